// MX quantizer kernels for sm_100a: row-wise, transposed / two-axis, Q-EMA, dequantize.
// All are HBM-bound element passes: 128-bit global accesses, one thread (or four lanes) per
// 32-element group, scales written straight into the 128x4 tiled order the GEMM consumes.
#include "common.cuh"

namespace mx {

// ------------------------------------------------------------------------------------------------
// Fill the padding entries (rows beyond `rows` up to a multiple of 128, blocks beyond `nblk` up to
// a multiple of 4) of a tiled scale buffer with 0x7F (= scale 1).
// ------------------------------------------------------------------------------------------------
__global__ void k_fill_scale_padding(uint8_t *scales, int64_t rows, int64_t nblk, int64_t nblk4)
{
    const int64_t rows_pad = ceil_div(rows, 128) * 128;
    const int64_t nb_pad = nblk4 * 4;
    const int64_t total = rows_pad * nb_pad;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / nb_pad, b = i - r * nb_pad;
        if (r >= rows || b >= nblk) scales[scale_offset(r, b, nblk4)] = 0x7F;
    }
}

static void fill_padding_if_needed(uint8_t *scales, int64_t rows, int64_t cols, cudaStream_t st)
{
    const int64_t nblk = cols / 32, nblk4 = ceil_div(nblk, 4);
    if (rows % 128 == 0 && nblk % 4 == 0) return;
    const int64_t total = ceil_div(rows, 128) * 128 * nblk4 * 4;
    int64_t nb = ceil_div(total, 256);
    int blocks = (int)(nb < 1184 ? nb : 1184);
    k_fill_scale_padding<<<blocks, 256, 0, st>>>(scales, rows, nblk, nblk4);
}

// 8 bf16 values held in one uint4, times the bf16 pair inv2 (2^-s in both halves) -> 8 codes (one u32, element 0 in
// the low nibble), round to nearest even.
__device__ __forceinline__ uint32_t rne8(const uint4 &q, uint32_t inv2)
{
    const uint32_t a = mul_bf16x2(q.x, inv2), b = mul_bf16x2(q.y, inv2), c = mul_bf16x2(q.z, inv2), d = mul_bf16x2(q.w, inv2);
    return rne_x8(bf16lo(a), bf16hi(a), bf16lo(b), bf16hi(b), bf16lo(c), bf16hi(c), bf16lo(d), bf16hi(d));
}

// The same with stochastic rounding; r0 / r1 are the random words of elements 0..3 / 4..7.
__device__ __forceinline__ uint32_t sr8(const uint4 &q, uint32_t inv2, uint32_t r0, uint32_t r1)
{
    const uint32_t a = mul_bf16x2(q.x, inv2), b = mul_bf16x2(q.y, inv2), c = mul_bf16x2(q.z, inv2), d = mul_bf16x2(q.w, inv2);
    const uint32_t lo = sr4(bf16lo(a), bf16hi(a), bf16lo(b), bf16hi(b), r0);
    const uint32_t hi = sr4(bf16lo(c), bf16hi(c), bf16lo(d), bf16hi(d), r1);
    return lo | (hi << 16);
}

// max of the 15-bit magnitudes of the 8 bf16 values in q (NaN/Inf patterns compare as large magnitudes)
__device__ __forceinline__ uint32_t absmax_u4(uint32_t acc, const uint4 &q)
{
    acc = absmax2(acc, q.x);
    acc = absmax2(acc, q.y);
    acc = absmax2(acc, q.z);
    return absmax2(acc, q.w);
}

// ------------------------------------------------------------------------------------------------
// Row-wise quantizer: one thread per 32-element group (Eq. 1 with 1x32 groups).
// ------------------------------------------------------------------------------------------------
template <int ROUNDING>
__global__ void __launch_bounds__(256) k_quantize_rows(const __nv_bfloat16 *__restrict__ src, int64_t rows, int nblk,
                                                       int64_t ld, uint8_t *__restrict__ packed,
                                                       uint8_t *__restrict__ scales, int nblk4, int scale_mode,
                                                       const SrStream sr, uint32_t *dev_status)
{
    const int64_t gid = blockIdx.x * (int64_t)256 + threadIdx.x;
    if (gid >= rows * nblk) return;
    const int64_t row = gid / nblk;
    const int blk = (int)(gid - row * nblk);
    const uint4 *p = reinterpret_cast<const uint4 *>(src + row * ld + blk * 32);
    uint4 q[4];
#pragma unroll
    for (int j = 0; j < 4; j++) q[j] = ld_nc_16(p + j);
    uint32_t am = 0;
#pragma unroll
    for (int j = 0; j < 4; j++) am = absmax_u4(am, q[j]);
    am = hmax_halves(am);
    uint4 out = make_uint4(0, 0, 0, 0);
    uint32_t byte;
    if (am >= 0x7F80u) {
        byte = 0xFFu;
        if (dev_status) atomicOr(dev_status, MXFP4_DEV_NONFINITE);
    } else {
        byte = scale_byte_from_amax(am, tf_add_of(scale_mode));
        const uint32_t inv = inv_scale_bf16x2(byte);
        if (ROUNDING == MXFP4_ROUND_NEAREST) {
            out = make_uint4(rne8(q[0], inv), rne8(q[1], inv), rne8(q[2], inv), rne8(q[3], inv));
        } else {
            const uint64_t q0 = ((uint64_t)row * ((uint64_t)nblk * 32) + (uint64_t)blk * 32) >> 4;
            const uint4 ra = sr_words(sr, q0), rb = sr_words(sr, q0 + 1);
            out.x = sr8(q[0], inv, ra.x, ra.y);
            out.y = sr8(q[1], inv, ra.z, ra.w);
            out.z = sr8(q[2], inv, rb.x, rb.y);
            out.w = sr8(q[3], inv, rb.z, rb.w);
        }
    }
    *reinterpret_cast<uint4 *>(packed + row * ((int64_t)nblk * 16) + blk * 16) = out;
    scales[scale_offset(row, blk, nblk4)] = (uint8_t)byte;
}

// ------------------------------------------------------------------------------------------------
// Two-axis tile quantizer.  A CTA owns a 128-row x 128-column tile of the source, which is exactly one
// 512-byte chunk of the tiled scale buffer of each output.  The tile is staged in shared memory as bf16
// (a bf16 source is copied; an MXFP4 source is dequantized exactly on the way in: double quantization,
// Sec. 3.3) and then read twice:
//   - row pass (optional): a thread takes 16 consecutive columns of one row, two lanes per group;
//   - column pass: a thread takes 16 consecutive rows of 4 columns, two lanes per group; the result is
//     the transposed matrix, staged in shared memory and written out in 64-byte rows.
// Each pass draws the random bits of 16 consecutive elements of ITS output with one Philox call.  Both
// scale chunks are assembled in shared memory (padding entries 0x7F) and written as whole chunks.
// ------------------------------------------------------------------------------------------------
constexpr int kTile = 128;
constexpr int kPitch = 2 * kTile + 16;   // bytes per staged row (16-byte skew against bank conflicts)

struct QuantSide {
    uint8_t *packed;
    uint8_t *scales;
    int nblk4;
    int scale_mode;
    SrStream sr;
};

// Packed pair of 15-bit group maxima (two columns) -> packed pair of scale bytes (bits 7:0 and 23:16).
// Non-finite maxima (>= 0x7F80) give 0xFF.
__device__ __forceinline__ uint32_t scale_bytes_x2(uint32_t am, uint32_t tf_add2)
{
    const uint32_t e = (am >> 7) & 0x00FF00FFu;
    const uint32_t up = (((am & 0x007F007Fu) + tf_add2) >> 7) & 0x00010001u;
    uint32_t b = __vmaxu2(e + up, 0x00020002u) - 0x00020002u;   // max(. - 2, 0) in each half, no borrow across
    b |= __vcmpeq2(am, 0u) & 0x00620062u;                        // all-zero group: byte 98
    b |= __vcmpgeu2(am, 0x7F807F80u) & 0x00FF00FFu;              // Inf/NaN in the group
    return b;
}

// DQ: the column pass quantizes the DEQUANTIZED result of the row pass instead of the source (double quantization of
// Sec. 3.3 in one kernel: the forward operand Q1(X) and the backward operand Q6(Q1(X)) from one read of X).
template <bool SRC_MXFP4, bool EMIT_ROW, bool SR_ROW, bool SR_T, bool DQ>
__global__ void __launch_bounds__(256, 4) k_quantize_tile(const void *__restrict__ src, const uint8_t *__restrict__ src_scales,
                                                          int src_nblk4, int rows, int cols, int64_t ld,
                                                          const __grid_constant__ QuantSide rw, const __grid_constant__ QuantSide tr,
                                                          uint32_t *dev_status)
{
    __shared__ __align__(16) uint8_t s_in[kTile * kPitch];
    __shared__ __align__(16) uint2 s_out[kTile * 8];          // [output row = source column][8-byte slot], slots XOR-swizzled
    __shared__ __align__(16) uint8_t s_sc_row[512], s_sc_t[512];

    const int tid = threadIdx.x;
    const int row0 = blockIdx.y * kTile, col0 = blockIdx.x * kTile;
    uint32_t nonfinite = 0;

    if (tid < 64) reinterpret_cast<uint4 *>(tid < 32 ? s_sc_row : s_sc_t)[tid & 31] = make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);

    // ---- stage the tile ----
    if (!SRC_MXFP4) {
        const int c16 = tid & 15, r0 = tid >> 4;
        const int gc = col0 + c16 * 8;
        const bool col_ok = gc < cols;
        const __nv_bfloat16 *gp = static_cast<const __nv_bfloat16 *>(src) + (int64_t)(row0 + r0) * ld + gc;
        uint8_t *sp = s_in + r0 * kPitch + c16 * 16;
#pragma unroll
        for (int k = 0; k < 8; k++) {
            uint4 q = make_uint4(0, 0, 0, 0);
            if (col_ok && row0 + r0 + k * 16 < rows) q = ld_nc_16(gp + (int64_t)k * 16 * ld);
            *reinterpret_cast<uint4 *>(sp + k * 16 * kPitch) = q;
        }
    } else {
        // packed source: one thread per (row, 32-element group): 16 bytes of codes + 1 scale byte
        const uint8_t *s = static_cast<const uint8_t *>(src);
        const uint8_t *sc_chunk = src_scales + ((size_t)(row0 >> 7) * src_nblk4 + (col0 >> 7)) * 512;
#pragma unroll
        for (int it = 0; it < 2; it++) {
            const int item = it * 256 + tid;
            const int r = item >> 2, g = item & 3;
            const int gr = row0 + r, gc = col0 + g * 32;
            uint32_t w[4] = {0, 0, 0, 0};
            uint32_t sc2 = 0u;
            if (gr < rows && gc < cols) {
                const uint4 q = ld_nc_16(s + (int64_t)gr * (cols >> 1) + (gc >> 1));
                w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
                const uint32_t sb = sc_chunk[(r & 31) * 16 + (r >> 5) * 4 + g];
                // a 0xFF scale marks a non-finite group of the first quantizer: propagate NaN
                sc2 = sb == 0xFFu ? 0x7FC07FC0u : scale_bf16x2(sb);
            }
#pragma unroll
            for (int j = 0; j < 4; j++) {
                uint32_t o[4];
                dequant_x8(w[j], sc2, o);   // P * 2^s is exact in bf16
                *reinterpret_cast<uint4 *>(s_in + r * kPitch + g * 64 + j * 16) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
    __syncthreads();

    // ---- row pass: thread = 16 consecutive columns of one row; lanes t, t^1 share a 32-element group ----
    if (EMIT_ROW) {
        const int cp = tid & 7, rr = tid >> 3;          // column chunk (16 columns), row within a 32-row pass
        const int gc = col0 + cp * 16;
        const bool col_ok = gc < cols;
        const uint32_t tfa = tf_add_of(rw.scale_mode);
        uint8_t *op = rw.packed + (int64_t)(row0 + rr) * (cols >> 1) + (gc >> 1);
        const uint64_t qi = ((uint64_t)(row0 + rr) * (uint64_t)cols + (uint64_t)gc) >> 4;
#pragma unroll 1
        for (int pass = 0; pass < 4; pass++) {
            const int r = pass * 32 + rr;
            const uint4 qa = *reinterpret_cast<const uint4 *>(s_in + r * kPitch + cp * 32);
            const uint4 qb = *reinterpret_cast<const uint4 *>(s_in + r * kPitch + cp * 32 + 16);
            uint32_t am = hmax_halves(absmax_u4(absmax_u4(0, qa), qb));
            am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
            const bool nf = am >= 0x7F80u;
            const uint32_t byte = nf ? 0xFFu : scale_byte_from_amax(am, tfa);
            const uint32_t inv = inv_scale_bf16x2(nf ? 127u : byte);
            uint2 codes;
            if (SR_ROW) {
                const uint4 rnd = sr_words(rw.sr, qi + (uint64_t)pass * 2u * (uint64_t)cols);
                codes.x = sr8(qa, inv, rnd.x, rnd.y);
                codes.y = sr8(qb, inv, rnd.z, rnd.w);
            } else {
                codes.x = rne8(qa, inv);
                codes.y = rne8(qb, inv);
            }
            if (nf) codes = make_uint2(0u, 0u);
            if (DQ) {
                // P * 2^s of the 16 codes back into the staged tile (exact in bf16); a non-finite group becomes NaN
                const uint32_t sc2 = nf ? 0x7FC07FC0u : scale_bf16x2(byte);
                uint32_t oa[4], ob[4];
                dequant_x8(codes.x, sc2, oa);
                dequant_x8(codes.y, sc2, ob);
                *reinterpret_cast<uint4 *>(s_in + r * kPitch + cp * 32) = make_uint4(oa[0], oa[1], oa[2], oa[3]);
                *reinterpret_cast<uint4 *>(s_in + r * kPitch + cp * 32 + 16) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
            }
            const bool ok = col_ok && row0 + r < rows;
            nonfinite |= (uint32_t)(nf && ok);
            if (ok) {
                *reinterpret_cast<uint2 *>(op + (int64_t)pass * 32 * (cols >> 1)) = codes;
                if ((cp & 1) == 0) s_sc_row[rr * 16 + pass * 4 + (cp >> 1)] = (uint8_t)byte;
            }
        }
    }

    if (DQ) __syncthreads();   // the column pass reads what the row pass wrote back

    // ---- column pass: warp = 32 rows x 64 columns; thread = 16 rows x 4 columns; lanes l, l^16 share the groups ----
    {
        const int warp = tid >> 5, lane = tid & 31;
        const int rg = warp >> 1, ch = warp & 1;
        const int h = lane >> 4, cl = lane & 15;
        const int c = ch * 64 + cl * 4;                 // first of this thread's 4 columns (tile-local)
        const int r = rg * 32 + h * 16;                 // first of its 16 rows
        uint2 v[16];
#pragma unroll
        for (int i = 0; i < 16; i++) v[i] = *reinterpret_cast<const uint2 *>(s_in + (r + i) * kPitch + c * 2);
        uint32_t am0 = 0, am1 = 0;
#pragma unroll
        for (int i = 0; i < 16; i++) {
            am0 = absmax2(am0, v[i].x);
            am1 = absmax2(am1, v[i].y);
        }
        am0 = __vmaxu2(am0, __shfl_xor_sync(0xFFFFFFFFu, am0, 16));
        am1 = __vmaxu2(am1, __shfl_xor_sync(0xFFFFFFFFu, am1, 16));
        // rows come in groups of 32 and columns in blocks of 32: a thread's 16 x 4 patch is inside the matrix or outside it
        if (row0 + r < rows && col0 + c < cols) {
            const uint32_t tfa2 = tf_add_of(tr.scale_mode) * 0x00010001u;
            const uint32_t b01 = scale_bytes_x2(am0, tfa2), b23 = scale_bytes_x2(am1, tfa2);
            // element index of (column, first row) in the transposed output, in units of 16
            const uint64_t qi = ((uint64_t)(col0 + c) * (uint64_t)rows + (uint64_t)(row0 + r)) >> 4;
#pragma unroll
            for (int jp = 0; jp < 2; jp++) {      // columns c + 2 jp and c + 2 jp + 1 share a word of every row
                const uint32_t b2 = jp ? b23 : b01;
                const uint32_t nfm = __vcmpeq2(b2, 0x00FF00FFu);                 // 0xFFFF in the half of a non-finite group
                nonfinite |= (uint32_t)(nfm != 0u);
                const uint32_t inv2 = (0x00FE00FEu - ((b2 & ~nfm) | (nfm & 0x007F007Fu))) << 7;   // 2^-s of both columns as bf16
                uint32_t lo0, hi0, lo1, hi1;   // codes of rows 0..7 / 8..15 of the two columns
                uint32_t x[16];
#pragma unroll
                for (int i = 0; i < 16; i++) x[i] = mul_bf16x2(jp ? v[i].y : v[i].x, inv2);
                if (SR_T) {
                    const uint4 ra = sr_words(tr.sr, qi + (uint64_t)(2 * jp) * (uint64_t)(rows >> 4));
                    const uint4 rb = sr_words(tr.sr, qi + (uint64_t)(2 * jp + 1) * (uint64_t)(rows >> 4));
                    lo0 = sr4(bf16lo(x[0]), bf16lo(x[1]), bf16lo(x[2]), bf16lo(x[3]), ra.x) | (sr4(bf16lo(x[4]), bf16lo(x[5]), bf16lo(x[6]), bf16lo(x[7]), ra.y) << 16);
                    hi0 = sr4(bf16lo(x[8]), bf16lo(x[9]), bf16lo(x[10]), bf16lo(x[11]), ra.z) | (sr4(bf16lo(x[12]), bf16lo(x[13]), bf16lo(x[14]), bf16lo(x[15]), ra.w) << 16);
                    lo1 = sr4(bf16hi(x[0]), bf16hi(x[1]), bf16hi(x[2]), bf16hi(x[3]), rb.x) | (sr4(bf16hi(x[4]), bf16hi(x[5]), bf16hi(x[6]), bf16hi(x[7]), rb.y) << 16);
                    hi1 = sr4(bf16hi(x[8]), bf16hi(x[9]), bf16hi(x[10]), bf16hi(x[11]), rb.z) | (sr4(bf16hi(x[12]), bf16hi(x[13]), bf16hi(x[14]), bf16hi(x[15]), rb.w) << 16);
                } else {
                    lo0 = rne_x8(bf16lo(x[0]), bf16lo(x[1]), bf16lo(x[2]), bf16lo(x[3]), bf16lo(x[4]), bf16lo(x[5]), bf16lo(x[6]), bf16lo(x[7]));
                    hi0 = rne_x8(bf16lo(x[8]), bf16lo(x[9]), bf16lo(x[10]), bf16lo(x[11]), bf16lo(x[12]), bf16lo(x[13]), bf16lo(x[14]), bf16lo(x[15]));
                    lo1 = rne_x8(bf16hi(x[0]), bf16hi(x[1]), bf16hi(x[2]), bf16hi(x[3]), bf16hi(x[4]), bf16hi(x[5]), bf16hi(x[6]), bf16hi(x[7]));
                    hi1 = rne_x8(bf16hi(x[8]), bf16hi(x[9]), bf16hi(x[10]), bf16hi(x[11]), bf16hi(x[12]), bf16hi(x[13]), bf16hi(x[14]), bf16hi(x[15]));
                }
                if (nfm & 0x0000FFFFu) lo0 = hi0 = 0u;
                if (nfm & 0xFFFF0000u) lo1 = hi1 = 0u;
                // output row c + j, bytes 16 rg + 8 h .. + 7: slot 2 rg + h, swizzled by the column quad
                const int j0 = 2 * jp;
                s_out[(c + j0) * 8 + ((2 * rg + h) ^ (cl & 7))] = make_uint2(lo0, hi0);
                s_out[(c + j0 + 1) * 8 + ((2 * rg + h) ^ (cl & 7))] = make_uint2(lo1, hi1);
                if (h == 0) {
                    s_sc_t[((c + j0) & 31) * 16 + ((c + j0) >> 5) * 4 + rg] = (uint8_t)(b2 & 0xFFu);
                    s_sc_t[((c + j0 + 1) & 31) * 16 + ((c + j0 + 1) >> 5) * 4 + rg] = (uint8_t)(b2 >> 16);
                }
            }
        }
    }
    __syncthreads();

    // ---- copy the transposed tile out: 128 output rows x 64 bytes, 16 bytes per thread and step ----
    {
#pragma unroll
        for (int it = 0; it < 2; it++) {
            const int id = it * 256 + tid;
            const int oc = id >> 2, g = id & 3;        // output row (source column), 16-byte group = source row group
            const int gc = col0 + oc, gr = row0 + g * 32;
            if (gc < cols && gr < rows) {
                const int x = (oc >> 2) & 7;
                const uint2 a = s_out[oc * 8 + ((2 * g) ^ x)], b = s_out[oc * 8 + ((2 * g + 1) ^ x)];
                *reinterpret_cast<uint4 *>(tr.packed + (int64_t)gc * (rows >> 1) + (gr >> 1)) = make_uint4(a.x, a.y, b.x, b.y);
            }
        }
        // the two scale chunks of this tile
        if (tid < 32) {
            if (EMIT_ROW)
                reinterpret_cast<uint4 *>(rw.scales + ((size_t)(row0 >> 7) * rw.nblk4 + (col0 >> 7)) * 512)[tid] =
                    reinterpret_cast<const uint4 *>(s_sc_row)[tid];
        } else if (tid < 64) {
            reinterpret_cast<uint4 *>(tr.scales + ((size_t)(col0 >> 7) * tr.nblk4 + (row0 >> 7)) * 512)[tid - 32] =
                reinterpret_cast<const uint4 *>(s_sc_t)[tid - 32];
        }
    }
    if (nonfinite && dev_status) atomicOr(dev_status, MXFP4_DEV_NONFINITE);
}

// ------------------------------------------------------------------------------------------------
// Q-EMA (Algorithm 1) fused with the EMA update (Eq. 10) and the oscillation counters (Sec. 6.1).

// ------------------------------------------------------------------------------------------------
struct OscPtrs {
    __nv_bfloat16 *w_prev;
    uint8_t *q_prev;
    uint8_t *s_prev;
    float *dist_w;
    float *dist_q;
};

// value of an E2M1 code as float
__device__ __forceinline__ float e2m1_value(uint32_t code)
{
    const uint32_t m = code & 7u;
    const uint32_t bits = m >= 2u ? (0x3F000000u + (m << 22)) : (m ? 0x3F000000u : 0u);
    return __uint_as_float(bits | ((code & 8u) << 28));
}

// The element step of Algorithm 1: propose the two neighbouring grid values q1 <= |w / S| <= q2, keep the one nearer
// to the EMA.  "The nearer of q1, q2 to e" is the round-to-nearest (ties to the even code, as everywhere) of e clamped
// to [q1, q2], because no grid value lies strictly between the two; a latent value on the grid has q1 = q2 and is
// kept.  Returns that clamped value with the sign of w, ready for the hardware convert.  v = w / S, ve = ema / S.
__device__ __forceinline__ float qema_target(float v, float ve)
{
    const uint32_t vb = __float_as_uint(v);
    const uint32_t ab = vb & 0x7FFFFFFFu;
    uint32_t lo, hi;
    if (ab >= 0x40C00000u) {            // 6 and beyond (floor scaling): saturates
        lo = hi = 0x40C00000u;
    } else if (ab >= 0x3F000000u) {     // [0.5, 6): one mantissa bit from 1 upwards, none below
        const uint32_t mask = ab >= 0x3F800000u ? 0x003FFFFFu : 0x007FFFFFu;
        lo = ab & ~mask;
        hi = ab == lo ? lo : lo + mask + 1u;
    } else {                            // [0, 0.5)
        lo = 0u;
        hi = ab == 0u ? 0u : 0x3F000000u;
    }
    const float es = (vb >> 31) ? -ve : ve;   // EMA mirrored to the side of w
    const float t = fminf(fmaxf(es, __uint_as_float(lo)), __uint_as_float(hi));
    return __uint_as_float(__float_as_uint(t) | (vb & 0x80000000u));
}

// Four consecutive lanes share a 32-element group: a thread owns 8 consecutive elements (the weight is contiguous).
template <bool OSC>
__global__ void __launch_bounds__(256) k_qema(const __nv_bfloat16 *__restrict__ w, float *__restrict__ ema, float beta,
                                              int update_ema, int64_t n, int nblk, uint8_t *__restrict__ packed,
                                              uint8_t *__restrict__ scales, int nblk4, int scale_mode, OscPtrs osc,
                                              uint32_t *dev_status)
{
    const int64_t total = n * nblk * 4;                       // threads with work (a multiple of 4)
    const int64_t gid = blockIdx.x * (int64_t)256 + threadIdx.x;
    const bool active = gid < total;
    const int64_t cid = active ? gid : 0;                     // idle lanes of the last warp shadow chunk 0 and store nothing
    const int64_t e0 = cid * 8;
    const int64_t grp = cid >> 2, row = grp / nblk;
    const int blk = (int)(grp - row * nblk);
    const float omb = __fsub_rn(1.0f, beta);

    const uint4 q = *reinterpret_cast<const uint4 *>(w + e0);
    float4 ea = *reinterpret_cast<const float4 *>(ema + e0), eb = *reinterpret_cast<const float4 *>(ema + e0 + 4);
    const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
    float wv[8];
#pragma unroll
    for (int t = 0; t < 4; t++) {
        wv[2 * t] = bf16lo(ww[t]);
        wv[2 * t + 1] = bf16hi(ww[t]);
    }
    if (update_ema) {
        ea.x = __fmaf_rn(beta, ea.x, __fmul_rn(omb, wv[0]));
        ea.y = __fmaf_rn(beta, ea.y, __fmul_rn(omb, wv[1]));
        ea.z = __fmaf_rn(beta, ea.z, __fmul_rn(omb, wv[2]));
        ea.w = __fmaf_rn(beta, ea.w, __fmul_rn(omb, wv[3]));
        eb.x = __fmaf_rn(beta, eb.x, __fmul_rn(omb, wv[4]));
        eb.y = __fmaf_rn(beta, eb.y, __fmul_rn(omb, wv[5]));
        eb.z = __fmaf_rn(beta, eb.z, __fmul_rn(omb, wv[6]));
        eb.w = __fmaf_rn(beta, eb.w, __fmul_rn(omb, wv[7]));
        if (active) {
            *reinterpret_cast<float4 *>(ema + e0) = ea;
            *reinterpret_cast<float4 *>(ema + e0 + 4) = eb;
        }
    }
    const float ev[8] = {ea.x, ea.y, ea.z, ea.w, eb.x, eb.y, eb.z, eb.w};
    uint32_t am = hmax_halves(absmax_u4(0, q));
    uint32_t badm = !(isfinite(ea.x) && isfinite(ea.y) && isfinite(ea.z) && isfinite(ea.w) && isfinite(eb.x) && isfinite(eb.y) &&
                      isfinite(eb.z) && isfinite(eb.w));
    am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
    am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 2));
    badm |= __shfl_xor_sync(0xFFFFFFFFu, badm, 1);
    badm |= __shfl_xor_sync(0xFFFFFFFFu, badm, 2);
    const bool bad = badm != 0u || am >= 0x7F80u;

    uint32_t byte, out = 0;
    if (bad) {
        byte = 0xFFu;
        if (dev_status && active) atomicOr(dev_status, MXFP4_DEV_NONFINITE);
    } else {
        byte = scale_byte_from_amax(am, tf_add_of(scale_mode));
        const float inv = inv_scale_from_byte(byte);
        float z[8];
#pragma unroll
        for (int i = 0; i < 8; i++) z[i] = qema_target(wv[i] * inv, ev[i] * inv);
        out = rne_x8(z[0], z[1], z[2], z[3], z[4], z[5], z[6], z[7]);
    }
    if (!active) return;

    const int64_t pk = row * ((int64_t)nblk * 16) + blk * 16 + (cid & 3) * 4;   // this thread's 4 bytes of codes
    if (OSC) {
        const uint32_t prev = *reinterpret_cast<const uint32_t *>(osc.q_prev + pk);
        const uint32_t sbp = osc.s_prev[scale_offset(row, blk, nblk4)];
        const float sc = byte == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(byte);
        const float scp = sbp == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(sbp);
        const uint4 wp = *reinterpret_cast<const uint4 *>(osc.w_prev + e0);
        const uint32_t wpw[4] = {wp.x, wp.y, wp.z, wp.w};
#pragma unroll
        for (int j = 0; j < 2; j++) {
            float4 dw = *reinterpret_cast<const float4 *>(osc.dist_w + e0 + 4 * j);
            float4 dq = *reinterpret_cast<const float4 *>(osc.dist_q + e0 + 4 * j);
            float *dwp = &dw.x, *dqp = &dq.x;
#pragma unroll
            for (int t = 0; t < 4; t++) {
                const int i = 4 * j + t;
                const float wpv = (i & 1) ? bf16hi(wpw[i >> 1]) : bf16lo(wpw[i >> 1]);
                const float qc = e2m1_value((out >> (4 * i)) & 15u) * sc;
                const float qo = e2m1_value((prev >> (4 * i)) & 15u) * scp;
                dwp[t] = __fadd_rn(dwp[t], fabsf(__fsub_rn(wv[i], wpv)));
                dqp[t] = __fadd_rn(dqp[t], fabsf(__fsub_rn(qc, qo)));
            }
            *reinterpret_cast<float4 *>(osc.dist_w + e0 + 4 * j) = dw;
            *reinterpret_cast<float4 *>(osc.dist_q + e0 + 4 * j) = dq;
        }
        __syncwarp();   // every lane of the group has read the previous scale before one of them replaces it
        *reinterpret_cast<uint4 *>(osc.w_prev + e0) = q;
        *reinterpret_cast<uint32_t *>(osc.q_prev + pk) = out;
        if ((cid & 3) == 0) osc.s_prev[scale_offset(row, blk, nblk4)] = (uint8_t)byte;
    }
    *reinterpret_cast<uint32_t *>(packed + pk) = out;
    if ((cid & 3) == 0) scales[scale_offset(row, blk, nblk4)] = (uint8_t)byte;
}

// ------------------------------------------------------------------------------------------------
// Exact dequantization, one thread per group.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_dequantize(const uint8_t *__restrict__ packed, const uint8_t *__restrict__ scales,
                                                    int64_t rows, int nblk, int nblk4, float *__restrict__ dst, int64_t ld)
{
    const int64_t gid = blockIdx.x * (int64_t)256 + threadIdx.x;
    if (gid >= rows * nblk) return;
    const int64_t row = gid / nblk;
    const int blk = (int)(gid - row * nblk);
    const uint4 q = *reinterpret_cast<const uint4 *>(packed + row * ((int64_t)nblk * 16) + blk * 16);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    const uint32_t sb = scales[scale_offset(row, blk, nblk4)];
    const float sc = sb == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(sb);
    float *o = dst + row * ld + blk * 32;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        float4 f;
        f.x = e2m1_value((w[i >> 3] >> (4 * (i & 7))) & 15u) * sc;
        f.y = e2m1_value((w[i >> 3] >> (4 * ((i + 1) & 7))) & 15u) * sc;
        f.z = e2m1_value((w[i >> 3] >> (4 * ((i + 2) & 7))) & 15u) * sc;
        f.w = e2m1_value((w[i >> 3] >> (4 * ((i + 3) & 7))) & 15u) * sc;
        *reinterpret_cast<float4 *>(o + i) = f;
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static mxfp4_status_t check_mat(const mxfp4_mat_t &m, int64_t rows, int64_t cols)
{
    if (!m.data || !m.scales) return MXFP4_INVALID_ARG;
    if (m.rows != rows || m.cols != cols) return MXFP4_BAD_SHAPE;
    if (!aligned16(m.data) || !aligned16(m.scales)) return MXFP4_MISALIGNED;
    return MXFP4_OK;
}

static mxfp4_status_t check_qp(const mxfp4_qparams_t *qp)
{
    if (!qp) return MXFP4_INVALID_ARG;
    if (qp->scale_mode != MXFP4_SCALE_TRUNCATION_FREE && qp->scale_mode != MXFP4_SCALE_FLOOR) return MXFP4_INVALID_ARG;
    if (qp->rounding != MXFP4_ROUND_NEAREST && qp->rounding != MXFP4_ROUND_STOCHASTIC) return MXFP4_INVALID_ARG;
    return MXFP4_OK;
}

mxfp4_status_t quantize_rows(const void *src, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                             const mxfp4_qparams_t *qp, uint32_t *dev_status, cudaStream_t st)
{
    if (rows < 0 || cols < 0) return MXFP4_INVALID_ARG;
    mxfp4_status_t s = check_qp(qp);
    if (s) return s;
    if (cols % 32 != 0 || ld < cols) return MXFP4_BAD_SHAPE;
    if (rows == 0 || cols == 0) return MXFP4_OK;  // nothing to do; pointers may be null
    if (!src) return MXFP4_INVALID_ARG;
    if ((s = check_mat(dst, rows, cols))) return s;
    if (!aligned16(src) || ld % 8 != 0) return MXFP4_MISALIGNED;
    if (rows == 0 || cols == 0) return MXFP4_OK;
    const int nblk = (int)(cols / 32), nblk4 = (nblk + 3) / 4;
    fill_padding_if_needed(dst.scales, rows, cols, st);
    const int64_t groups = rows * nblk;
    const unsigned blocks = (unsigned)ceil_div(groups, 256);
    if (qp->rounding == MXFP4_ROUND_STOCHASTIC)
        k_quantize_rows<MXFP4_ROUND_STOCHASTIC><<<blocks, 256, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(src), rows, nblk, ld, static_cast<uint8_t *>(dst.data), dst.scales, nblk4,
            qp->scale_mode, make_sr_stream(qp->seed, qp->stream_id), dev_status);
    else
        k_quantize_rows<MXFP4_ROUND_NEAREST><<<blocks, 256, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(src), rows, nblk, ld, static_cast<uint8_t *>(dst.data), dst.scales, nblk4,
            qp->scale_mode, make_sr_stream(qp->seed, qp->stream_id), dev_status);
    MX_CHECK_CUDA(cudaGetLastError());
    return MXFP4_OK;
}

static QuantSide make_side(const mxfp4_mat_t &m, const mxfp4_qparams_t *qp)
{
    QuantSide s;
    s.packed = static_cast<uint8_t *>(m.data);
    s.scales = m.scales;
    s.nblk4 = (int)ceil_div(m.cols / 32, 4);
    s.scale_mode = qp->scale_mode;
    s.sr = make_sr_stream(qp->seed, qp->stream_id);
    return s;
}

template <bool SRC_MXFP4, bool EMIT_ROW, bool SR_ROW, bool SR_T, bool DQ = false>
static void launch_tile(dim3 grid, cudaStream_t st, const void *src, const uint8_t *src_scales, int src_nblk4, int rows, int cols,
                        int64_t ld, const QuantSide &rw, const QuantSide &tr, uint32_t *dev_status)
{
    k_quantize_tile<SRC_MXFP4, EMIT_ROW, SR_ROW, SR_T, DQ><<<grid, 256, 0, st>>>(src, src_scales, src_nblk4, rows, cols, ld, rw, tr, dev_status);
}

// src_bf16 xor src_q; dst (row-wise) optional; dst_t required.  chain: dst_t is quantized from the dequantized dst
// (double quantization) instead of from the source; needs a bf16 source and dst.
mxfp4_status_t quantize_tile(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows, int64_t cols, int64_t ld,
                             const mxfp4_mat_t *dst, const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t,
                             const mxfp4_qparams_t *qp_t, uint32_t *dev_status, cudaStream_t st, bool chain)
{
    if (chain && (!dst || !src_bf16)) return MXFP4_INVALID_ARG;
    if ((src_bf16 == nullptr) == (src_q == nullptr) || rows < 0 || cols < 0) return MXFP4_INVALID_ARG;
    if (dst && src_q) return MXFP4_INVALID_ARG;
    mxfp4_status_t s = check_qp(qp_t);
    if (s) return s;
    if (dst && (s = check_qp(qp_row))) return s;
    if (rows % 32 != 0 || cols % 32 != 0) return MXFP4_BAD_SHAPE;
    if (rows > 0x7FFFFF80 || cols > 0x7FFFFF80) return MXFP4_BAD_SHAPE;
    if ((s = check_mat(dst_t, cols, rows))) return s;
    if (dst && (s = check_mat(*dst, rows, cols))) return s;
    if (src_bf16) {
        if (ld < cols) return MXFP4_BAD_SHAPE;
        if (!aligned16(src_bf16) || ld % 8 != 0) return MXFP4_MISALIGNED;
    } else {
        if ((s = check_mat(*src_q, rows, cols))) return s;
    }
    if (rows == 0 || cols == 0) return MXFP4_OK;
    // every tile writes its whole 512-byte scale chunk(s), padding entries included
    const dim3 grid((unsigned)ceil_div(cols, kTile), (unsigned)ceil_div(rows, kTile));
    if (grid.y > 65535u) return MXFP4_BAD_SHAPE;
    const QuantSide tr = make_side(dst_t, qp_t);
    const QuantSide rw = dst ? make_side(*dst, qp_row) : tr;
    const bool sr_t = qp_t->rounding == MXFP4_ROUND_STOCHASTIC;
    const bool sr_r = dst && qp_row->rounding == MXFP4_ROUND_STOCHASTIC;
    const int r = (int)rows, c = (int)cols;
    if (src_q) {
        const int nb4 = (int)ceil_div(cols / 32, 4);
        if (sr_t) launch_tile<true, false, false, true>(grid, st, src_q->data, src_q->scales, nb4, r, c, cols, rw, tr, dev_status);
        else launch_tile<true, false, false, false>(grid, st, src_q->data, src_q->scales, nb4, r, c, cols, rw, tr, dev_status);
    } else if (dst) {
        if (chain) {
            if (sr_r && sr_t) launch_tile<false, true, true, true, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
            else if (sr_r) launch_tile<false, true, true, false, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
            else if (sr_t) launch_tile<false, true, false, true, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
            else launch_tile<false, true, false, false, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
        } else if (sr_r && sr_t) launch_tile<false, true, true, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
        else if (sr_r) launch_tile<false, true, true, false>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
        else if (sr_t) launch_tile<false, true, false, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
        else launch_tile<false, true, false, false>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
    } else {
        if (sr_t) launch_tile<false, false, false, true>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
        else launch_tile<false, false, false, false>(grid, st, src_bf16, nullptr, 0, r, c, ld, rw, tr, dev_status);
    }
    MX_CHECK_CUDA(cudaGetLastError());
    return MXFP4_OK;
}

}  // namespace mx

using namespace mx;

extern "C" {

size_t mxfp4_scale_bytes(int64_t rows, int64_t cols)
{
    if (rows <= 0 || cols <= 0) return 0;
    return (size_t)(ceil_div(rows, 128) * ceil_div(ceil_div(cols, 32), 4) * 512);
}

size_t mxfp4_scale_offset(int64_t row, int64_t block, int64_t cols)
{
    return scale_offset(row, block, ceil_div(ceil_div(cols, 32), 4));
}

mxfp4_status_t mxfp4_quantize(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                              const mxfp4_qparams_t *qp, uint32_t *dev_status, void *stream)
{
    return quantize_rows(src_bf16, rows, cols, ld, dst, qp, dev_status, static_cast<cudaStream_t>(stream));
}

mxfp4_status_t mxfp4_quantize_t(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows, int64_t cols, int64_t ld,
                                mxfp4_mat_t dst_t, const mxfp4_qparams_t *qp, uint32_t *dev_status, void *stream)
{
    return quantize_tile(src_bf16, src_q, rows, cols, ld, nullptr, nullptr, dst_t, qp, dev_status,
                         static_cast<cudaStream_t>(stream), false);
}

mxfp4_status_t mxfp4_quantize_2axis(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                                    const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t, const mxfp4_qparams_t *qp_t,
                                    uint32_t *dev_status, void *stream)
{
    if (!src_bf16) return MXFP4_INVALID_ARG;
    return quantize_tile(src_bf16, nullptr, rows, cols, ld, &dst, qp_row, dst_t, qp_t, dev_status,
                         static_cast<cudaStream_t>(stream), false);
}

mxfp4_status_t mxfp4_quantize_chain(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                                    const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t, const mxfp4_qparams_t *qp_t,
                                    uint32_t *dev_status, void *stream)
{
    if (!src_bf16) return MXFP4_INVALID_ARG;
    return quantize_tile(src_bf16, nullptr, rows, cols, ld, &dst, qp_row, dst_t, qp_t, dev_status,
                         static_cast<cudaStream_t>(stream), true);
}

mxfp4_status_t mxfp4_qema_quantize(const void *w_bf16, float *ema, float beta, int32_t update_ema, int64_t n, int64_t k,
                                   mxfp4_mat_t dst, int32_t scale_mode, const mxfp4_osc_state_t *osc,
                                   uint32_t *dev_status, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!w_bf16 || !ema || n < 0 || k < 0) return MXFP4_INVALID_ARG;
    if (scale_mode != MXFP4_SCALE_TRUNCATION_FREE && scale_mode != MXFP4_SCALE_FLOOR) return MXFP4_INVALID_ARG;
    if (!(beta >= 0.f && beta <= 1.f)) return MXFP4_INVALID_ARG;
    if (k % 32 != 0) return MXFP4_BAD_SHAPE;
    mxfp4_status_t s = check_mat(dst, n, k);
    if (s) return s;
    if (!aligned16(w_bf16) || !aligned16(ema)) return MXFP4_MISALIGNED;
    OscPtrs op = {nullptr, nullptr, nullptr, nullptr, nullptr};
    if (osc) {
        if (!osc->w_prev || !osc->dist_w || !osc->dist_q) return MXFP4_INVALID_ARG;
        if ((s = check_mat(osc->wq_prev, n, k))) return s;
        if (!aligned16(osc->w_prev) || !aligned16(osc->dist_w) || !aligned16(osc->dist_q)) return MXFP4_MISALIGNED;
        op.w_prev = static_cast<__nv_bfloat16 *>(osc->w_prev);
        op.q_prev = static_cast<uint8_t *>(osc->wq_prev.data);
        op.s_prev = osc->wq_prev.scales;
        op.dist_w = osc->dist_w;
        op.dist_q = osc->dist_q;
    }
    if (n == 0 || k == 0) return MXFP4_OK;
    const int nblk = (int)(k / 32), nblk4 = (nblk + 3) / 4;
    fill_padding_if_needed(dst.scales, n, k, st);
    if (osc) fill_padding_if_needed(osc->wq_prev.scales, n, k, st);
    const unsigned blocks = (unsigned)ceil_div(n * nblk * 4, 256);
    if (osc)
        k_qema<true><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(w_bf16), ema, beta, update_ema, n, nblk,
                                             static_cast<uint8_t *>(dst.data), dst.scales, nblk4, scale_mode, op, dev_status);
    else
        k_qema<false><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(w_bf16), ema, beta, update_ema, n, nblk,
                                              static_cast<uint8_t *>(dst.data), dst.scales, nblk4, scale_mode, op, dev_status);
    MX_CHECK_CUDA(cudaGetLastError());
    return MXFP4_OK;
}

mxfp4_status_t mxfp4_dequantize(mxfp4_mat_t src, float *dst, int64_t ld, void *stream)
{
    if (!dst || src.rows < 0 || src.cols < 0) return MXFP4_INVALID_ARG;
    if (src.cols % 32 != 0 || ld < src.cols) return MXFP4_BAD_SHAPE;
    mxfp4_status_t s = check_mat(src, src.rows, src.cols);
    if (s) return s;
    if (!aligned16(dst) || ld % 4 != 0) return MXFP4_MISALIGNED;
    if (src.rows == 0 || src.cols == 0) return MXFP4_OK;
    const int nblk = (int)(src.cols / 32), nblk4 = (nblk + 3) / 4;
    const unsigned blocks = (unsigned)ceil_div(src.rows * nblk, 256);
    k_dequantize<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint8_t *>(src.data), src.scales,
                                                                        src.rows, nblk, nblk4, dst, ld);
    MX_CHECK_CUDA(cudaGetLastError());
    return MXFP4_OK;
}

}  // extern "C"
