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

// Quantize 8 bf16 values held in one uint4 to 8 codes (one u32, element 0 in the low nibble).
template <int ROUNDING>
__device__ __forceinline__ uint32_t quantize8(const uint4 &q, float inv, uint64_t seed, uint32_t stream, uint64_t elem_index)
{
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    uint32_t out = 0;
    if (ROUNDING == MXFP4_ROUND_NEAREST) {
#pragma unroll
        for (int j = 0; j < 4; j++) out |= rne_pair(bf16lo(w[j]) * inv, bf16hi(w[j]) * inv) << (8 * j);
    } else {
        const uint4 r = sr_words(seed, stream, elem_index >> 3);
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
        uint32_t sgn = 0;
#pragma unroll
        for (int j = 3; j >= 0; j--) {
            out = (out << 4) + sr_mag(bf16hi(w[j]) * inv, sr_c_odd(rw[j]));
            out = (out << 4) + sr_mag(bf16lo(w[j]) * inv, sr_c_even(rw[j]));
            // sign bits 15 / 31 of the source word -> bit 3 of nibbles 2j / 2j+1
            sgn |= (j == 0 ? (w[j] >> 12) : j == 1 ? (w[j] >> 4) : j == 2 ? (w[j] << 4) : (w[j] << 12)) & (0x8u << (8 * j));
            sgn |= (w[j] >> (24 - 8 * j)) & (0x80u << (8 * j));
        }
        out |= sgn;
    }
    return out;
}

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
                                                       uint64_t seed, uint32_t stream, uint32_t *dev_status)
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
        byte = scale_mode == MXFP4_SCALE_FLOOR ? scale_byte_from_amax<MXFP4_SCALE_FLOOR>(am)
                                               : scale_byte_from_amax<MXFP4_SCALE_TRUNCATION_FREE>(am);
        const float inv = inv_scale_from_byte(byte);
        const uint64_t e0 = (uint64_t)row * ((uint64_t)nblk * 32) + (uint64_t)blk * 32;
        out.x = quantize8<ROUNDING>(q[0], inv, seed, stream, e0);
        out.y = quantize8<ROUNDING>(q[1], inv, seed, stream, e0 + 8);
        out.z = quantize8<ROUNDING>(q[2], inv, seed, stream, e0 + 16);
        out.w = quantize8<ROUNDING>(q[3], inv, seed, stream, e0 + 24);
    }
    *reinterpret_cast<uint4 *>(packed + row * ((int64_t)nblk * 16) + blk * 16) = out;
    scales[scale_offset(row, blk, nblk4)] = (uint8_t)byte;
}

// ------------------------------------------------------------------------------------------------
// Two-axis tile quantizer.  A CTA stages a 128-row x 64-column tile of the source in shared memory
// (as bf16) and emits
//   - optionally the row-wise quantization of the tile (groups along columns), straight from the
//     registers that loaded it (4 lanes per group), and
//   - the quantization along rows (groups of 32 source rows), written as the transposed matrix.
// The source is bf16, or an MXFP4 matrix that is dequantized exactly on the way in (double
// quantization, Sec. 3.3).  Random words depend only on the source element index.
// ------------------------------------------------------------------------------------------------
constexpr int kTileR = 128, kTileC = 64;
constexpr int kPitch = 144;  // bytes per staged row: 128 + 16, keeps both access patterns conflict-free

struct QuantSide {
    uint8_t *packed;
    uint8_t *scales;
    int nblk4;
    int scale_mode;
    int rounding;
    uint32_t stream;
    uint64_t seed;
};

__device__ __forceinline__ uint32_t pick_scale_byte(uint32_t am, int scale_mode)
{
    return scale_mode == MXFP4_SCALE_FLOOR ? scale_byte_from_amax<MXFP4_SCALE_FLOOR>(am)
                                           : scale_byte_from_amax<MXFP4_SCALE_TRUNCATION_FREE>(am);
}

template <bool SRC_MXFP4, bool EMIT_ROW>
__global__ void __launch_bounds__(256) k_quantize_tile(const void *__restrict__ src, const uint8_t *__restrict__ src_scales,
                                                       int src_nblk4, int64_t rows, int64_t cols, int64_t ld,
                                                       QuantSide rw, QuantSide tr, uint32_t *dev_status)
{
    __shared__ __align__(16) uint8_t s_in[kTileR * kPitch];
    __shared__ __align__(16) uint8_t s_out[kTileC * (kTileR / 2)];

    const int tid = threadIdx.x;
    const int64_t row0 = (int64_t)blockIdx.y * kTileR;
    const int64_t col0 = (int64_t)blockIdx.x * kTileC;
    bool nonfinite = false;

    // ---- stage the tile (and emit the row-wise operand) ----
    if (!SRC_MXFP4) {
        const __nv_bfloat16 *s = static_cast<const __nv_bfloat16 *>(src);
#pragma unroll
        for (int it = 0; it < 4; it++) {
            const int id = it * 256 + tid;
            const int r = id >> 3, c16 = id & 7;  // 8 chunks of 8 elements per staged row
            const int64_t gr = row0 + r, gc = col0 + c16 * 8;
            const bool ok = gr < rows && gc < cols;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (ok) q = ld_nc_16(s + gr * ld + gc);
            *reinterpret_cast<uint4 *>(s_in + r * kPitch + c16 * 16) = q;
            if (EMIT_ROW) {
                // 4 consecutive lanes hold one 32-element group
                uint32_t am = hmax_halves(absmax_u4(0, q));
                am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
                am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, 2));
                if (ok) {
                    uint32_t byte, codes = 0;
                    if (am >= 0x7F80u) {
                        byte = 0xFFu;
                        nonfinite = true;
                    } else {
                        byte = pick_scale_byte(am, rw.scale_mode);
                        const float inv = inv_scale_from_byte(byte);
                        const uint64_t e0 = (uint64_t)gr * (uint64_t)cols + (uint64_t)gc;
                        codes = rw.rounding == MXFP4_ROUND_STOCHASTIC
                                    ? quantize8<MXFP4_ROUND_STOCHASTIC>(q, inv, rw.seed, rw.stream, e0)
                                    : quantize8<MXFP4_ROUND_NEAREST>(q, inv, 0, 0, 0);
                    }
                    *reinterpret_cast<uint32_t *>(rw.packed + gr * (cols >> 1) + (gc >> 1)) = codes;
                    if ((c16 & 3) == 0) rw.scales[scale_offset(gr, gc >> 5, rw.nblk4)] = (uint8_t)byte;
                }
            }
        }
    } else {
        // packed source: one thread per (row, 32-element group): 16 bytes of codes + 1 scale byte
        const uint8_t *s = static_cast<const uint8_t *>(src);
        const int r = tid >> 1, g = tid & 1;
        const int64_t gr = row0 + r, gc = col0 + g * 32;
        uint32_t w[4] = {0, 0, 0, 0};
        float sc = 0.f;
        if (gr < rows && gc < cols) {
            const uint4 q = ld_nc_16(s + gr * (cols >> 1) + (gc >> 1));
            w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
            const uint32_t sb = src_scales[scale_offset(gr, gc >> 5, src_nblk4)];
            // a 0xFF scale marks a non-finite group of the first quantizer: propagate NaN
            sc = sb == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(sb);
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            uint32_t o[4];
#pragma unroll
            for (int b = 0; b < 4; b++) {
                const uint32_t byte = (w[j] >> (8 * b)) & 0xFFu;
                uint32_t h2;
                asm("{\n\t.reg .b8 b;\n\tcvt.u8.u32 b, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}" : "=r"(h2) : "r"(byte));
                const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
                // P * 2^s is exact in FP32 and representable in bf16
                o[b] = (__float_as_uint(f.x * sc) >> 16) | (__float_as_uint(f.y * sc) & 0xFFFF0000u);
            }
            *reinterpret_cast<uint4 *>(s_in + r * kPitch + g * 64 + j * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
    __syncthreads();

    // ---- quantize along rows: warp = 32 rows x 32 columns, thread = 4 rows x 8 columns ----
    {
        const int warp = tid >> 5, lane = tid & 31;
        const int rg = warp >> 1, cb = warp & 1;
        const int lr = lane >> 2, lc = lane & 3;
        const int c = cb * 32 + lc * 8;           // first of this thread's 8 columns (tile-local)
        const int64_t gc = col0 + c;
        const int64_t grow0 = row0 + rg * 32;
        const bool ok = grow0 < rows && gc < cols;
        uint32_t v[4][4];                         // [row][column pair]
        uint32_t am[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const uint4 q = *reinterpret_cast<const uint4 *>(s_in + (rg * 32 + 4 * lr + i) * kPitch + c * 2);
            v[i][0] = q.x; v[i][1] = q.y; v[i][2] = q.z; v[i][3] = q.w;
#pragma unroll
            for (int j = 0; j < 4; j++) am[j] = absmax2(am[j], v[i][j]);
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            am[j] = __vmaxu2(am[j], __shfl_xor_sync(0xFFFFFFFFu, am[j], 4));
            am[j] = __vmaxu2(am[j], __shfl_xor_sync(0xFFFFFFFFu, am[j], 8));
            am[j] = __vmaxu2(am[j], __shfl_xor_sync(0xFFFFFFFFu, am[j], 16));
        }
        float inv[8];
        uint32_t byte[8];
#pragma unroll
        for (int j = 0; j < 8; j++) {
            const uint32_t a = (j & 1) ? (am[j >> 1] >> 16) : (am[j >> 1] & 0xFFFFu);
            if (a >= 0x7F80u) {
                byte[j] = 0xFFu;
                inv[j] = 0.f;
                if (ok) nonfinite = true;
            } else {
                byte[j] = pick_scale_byte(a, tr.scale_mode);
                inv[j] = inv_scale_from_byte(byte[j]);
            }
        }
        // per column pair: low 16 bits = codes of the even column (row i in nibble i), high 16 bits = odd column
        uint32_t outw[4] = {0, 0, 0, 0};
        if (tr.rounding == MXFP4_ROUND_STOCHASTIC) {
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const int64_t r = grow0 + 4 * lr + i;
                const uint4 rnd = sr_words(tr.seed, tr.stream, ((uint64_t)r * (uint64_t)cols + (uint64_t)gc) >> 3);
                const uint32_t rw4[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t m0 = sr_mag(bf16lo(v[i][j]) * inv[2 * j], sr_c_even(rw4[j]));
                    const uint32_t m1 = sr_mag(bf16hi(v[i][j]) * inv[2 * j + 1], sr_c_odd(rw4[j]));
                    outw[j] += (m0 << (4 * i)) + (m1 << (16 + 4 * i));
                    outw[j] |= (i == 3 ? v[i][j] : (v[i][j] >> (12 - 4 * i))) & (0x00080008u << (4 * i));
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; i++)
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t p = rne_pair(bf16lo(v[i][j]) * inv[2 * j], bf16hi(v[i][j]) * inv[2 * j + 1]);
                    outw[j] |= ((p & 15u) << (4 * i)) | ((p >> 4) << (16 + 4 * i));
                }
        }
        // bytes 2*lr, 2*lr+1 of the 16-byte group of each column hold rows 4*lr .. 4*lr+3
#pragma unroll
        for (int j = 0; j < 8; j++) {
            const uint32_t h = byte[j] == 0xFFu ? 0u : ((j & 1) ? (outw[j >> 1] >> 16) : (outw[j >> 1] & 0xFFFFu));
            *reinterpret_cast<uint16_t *>(s_out + (c + j) * (kTileR / 2) + rg * 16 + 2 * lr) = (uint16_t)h;
            if (lr == 0 && ok) tr.scales[scale_offset(gc + j, (grow0 >> 5), tr.nblk4)] = (uint8_t)byte[j];
        }
    }
    __syncthreads();

    // ---- copy the transposed tile out: 64 output rows x 64 bytes ----
    {
        const int c = tid >> 2, ch = tid & 3;
        const int64_t gc = col0 + c, gr = row0 + ch * 32;
        if (gc < cols && gr < rows)
            *reinterpret_cast<uint4 *>(tr.packed + gc * (rows >> 1) + (gr >> 1)) =
                *reinterpret_cast<const uint4 *>(s_out + c * (kTileR / 2) + ch * 16);
    }
    if (nonfinite && dev_status) atomicOr(dev_status, MXFP4_DEV_NONFINITE);
}

// ------------------------------------------------------------------------------------------------
// Q-EMA (Algorithm 1) fused with the EMA update (Eq. 10) and the oscillation counters (Sec. 6.1).
// One thread per 32-element group of the weight.
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

// Algorithm 1 lines 5-9 for one element: v = w / S, ve = ema / S.
__device__ __forceinline__ uint32_t qema_one(float v, float ve)
{
    const uint32_t vb = __float_as_uint(v);
    const uint32_t ab = vb & 0x7FFFFFFFu;
    uint32_t lo, hi;
    if (ab >= 0x40C00000u) return encode_on_grid(0x40C00000u, vb);  // beyond 6 (floor scaling): saturate
    if (ab >= 0x3F000000u) {
        const uint32_t mask = ab >= 0x3F800000u ? 0x003FFFFFu : 0x007FFFFFu;
        lo = ab & ~mask;
        hi = lo + mask + 1u;
    } else {
        lo = 0u;
        hi = 0x3F000000u;
    }
    if (ab == lo) return encode_on_grid(lo, vb);  // on the grid: kept
    const float flo = __uint_as_float(lo), fhi = __uint_as_float(hi);
    const float mid = 0.5f * (flo + fhi);
    const float es = (vb >> 31) ? -ve : ve;  // EMA mirrored to the side of w
    const uint32_t clo = encode_on_grid(lo, vb), chi = encode_on_grid(hi, vb);
    if (es < mid) return clo;
    if (es > mid) return chi;
    return (clo & 1u) ? chi : clo;  // tie: even code
}

template <bool OSC>
__global__ void __launch_bounds__(128) k_qema(const __nv_bfloat16 *__restrict__ w, float *__restrict__ ema, float beta,
                                              int update_ema, int64_t n, int nblk, uint8_t *__restrict__ packed,
                                              uint8_t *__restrict__ scales, int nblk4, int scale_mode, OscPtrs osc,
                                              uint32_t *dev_status)
{
    const int64_t gid = blockIdx.x * (int64_t)128 + threadIdx.x;
    if (gid >= n * nblk) return;
    const int64_t row = gid / nblk;
    const int blk = (int)(gid - row * nblk);
    const int64_t e0 = row * ((int64_t)nblk * 32) + (int64_t)blk * 32;
    const float omb = __fsub_rn(1.0f, beta);

    uint4 q[4];
#pragma unroll
    for (int j = 0; j < 4; j++) q[j] = *reinterpret_cast<const uint4 *>(w + e0 + 8 * j);
    uint32_t am = 0;
#pragma unroll
    for (int j = 0; j < 4; j++) am = absmax_u4(am, q[j]);
    am = hmax_halves(am);
    bool bad = am >= 0x7F80u;

    float wv[32], ev[32];
#pragma unroll
    for (int j = 0; j < 4; j++) {
        const uint32_t ww[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
        for (int t = 0; t < 4; t++) {
            wv[8 * j + 2 * t] = bf16lo(ww[t]);
            wv[8 * j + 2 * t + 1] = bf16hi(ww[t]);
        }
    }
#pragma unroll
    for (int j = 0; j < 8; j++) {
        float4 e = *reinterpret_cast<const float4 *>(ema + e0 + 4 * j);
        if (update_ema) {
            e.x = __fmaf_rn(beta, e.x, __fmul_rn(omb, wv[4 * j + 0]));
            e.y = __fmaf_rn(beta, e.y, __fmul_rn(omb, wv[4 * j + 1]));
            e.z = __fmaf_rn(beta, e.z, __fmul_rn(omb, wv[4 * j + 2]));
            e.w = __fmaf_rn(beta, e.w, __fmul_rn(omb, wv[4 * j + 3]));
            *reinterpret_cast<float4 *>(ema + e0 + 4 * j) = e;
        }
        ev[4 * j + 0] = e.x; ev[4 * j + 1] = e.y; ev[4 * j + 2] = e.z; ev[4 * j + 3] = e.w;
        bad = bad || !(isfinite(e.x) && isfinite(e.y) && isfinite(e.z) && isfinite(e.w));
    }

    uint32_t byte, out[4] = {0, 0, 0, 0};
    if (bad) {
        byte = 0xFFu;
        if (dev_status) atomicOr(dev_status, MXFP4_DEV_NONFINITE);
    } else {
        byte = pick_scale_byte(am, scale_mode);
        const float inv = inv_scale_from_byte(byte);
#pragma unroll
        for (int i = 0; i < 32; i++) out[i >> 3] |= qema_one(wv[i] * inv, ev[i] * inv) << (4 * (i & 7));
    }

    if (OSC) {
        const uint4 qp = *reinterpret_cast<const uint4 *>(osc.q_prev + row * ((int64_t)nblk * 16) + blk * 16);
        const uint32_t prev[4] = {qp.x, qp.y, qp.z, qp.w};
        const uint32_t sbp = osc.s_prev[scale_offset(row, blk, nblk4)];
        const float sc = byte == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(byte);
        const float scp = sbp == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(sbp);
#pragma unroll
        for (int j = 0; j < 8; j++) {
            float4 dw = *reinterpret_cast<const float4 *>(osc.dist_w + e0 + 4 * j);
            float4 dq = *reinterpret_cast<const float4 *>(osc.dist_q + e0 + 4 * j);
            const uint2 wp = *reinterpret_cast<const uint2 *>(osc.w_prev + e0 + 4 * j);
            const float wpv[4] = {bf16lo(wp.x), bf16hi(wp.x), bf16lo(wp.y), bf16hi(wp.y)};
            float *dwp = &dw.x, *dqp = &dq.x;
#pragma unroll
            for (int t = 0; t < 4; t++) {
                const int i = 4 * j + t;
                const float qc = e2m1_value((out[i >> 3] >> (4 * (i & 7))) & 15u) * sc;
                const float qo = e2m1_value((prev[i >> 3] >> (4 * (i & 7))) & 15u) * scp;
                dwp[t] = __fadd_rn(dwp[t], fabsf(__fsub_rn(wv[i], wpv[t])));
                dqp[t] = __fadd_rn(dqp[t], fabsf(__fsub_rn(qc, qo)));
            }
            *reinterpret_cast<float4 *>(osc.dist_w + e0 + 4 * j) = dw;
            *reinterpret_cast<float4 *>(osc.dist_q + e0 + 4 * j) = dq;
        }
#pragma unroll
        for (int j = 0; j < 4; j++) *reinterpret_cast<uint4 *>(osc.w_prev + e0 + 8 * j) = q[j];
        *reinterpret_cast<uint4 *>(osc.q_prev + row * ((int64_t)nblk * 16) + blk * 16) = make_uint4(out[0], out[1], out[2], out[3]);
        osc.s_prev[scale_offset(row, blk, nblk4)] = (uint8_t)byte;
    }
    *reinterpret_cast<uint4 *>(packed + row * ((int64_t)nblk * 16) + blk * 16) = make_uint4(out[0], out[1], out[2], out[3]);
    scales[scale_offset(row, blk, nblk4)] = (uint8_t)byte;
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
            qp->scale_mode, qp->seed, qp->stream_id, dev_status);
    else
        k_quantize_rows<MXFP4_ROUND_NEAREST><<<blocks, 256, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(src), rows, nblk, ld, static_cast<uint8_t *>(dst.data), dst.scales, nblk4,
            qp->scale_mode, qp->seed, qp->stream_id, dev_status);
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
    s.rounding = qp->rounding;
    s.stream = qp->stream_id;
    s.seed = qp->seed;
    return s;
}

// src_bf16 xor src_q; dst (row-wise) optional; dst_t required
mxfp4_status_t quantize_tile(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows, int64_t cols, int64_t ld,
                             const mxfp4_mat_t *dst, const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t,
                             const mxfp4_qparams_t *qp_t, uint32_t *dev_status, cudaStream_t st)
{
    if ((src_bf16 == nullptr) == (src_q == nullptr) || rows < 0 || cols < 0) return MXFP4_INVALID_ARG;
    if (dst && src_q) return MXFP4_INVALID_ARG;
    mxfp4_status_t s = check_qp(qp_t);
    if (s) return s;
    if (dst && (s = check_qp(qp_row))) return s;
    if (rows % 32 != 0 || cols % 32 != 0) return MXFP4_BAD_SHAPE;
    if ((s = check_mat(dst_t, cols, rows))) return s;
    if (dst && (s = check_mat(*dst, rows, cols))) return s;
    if (src_bf16) {
        if (ld < cols) return MXFP4_BAD_SHAPE;
        if (!aligned16(src_bf16) || ld % 8 != 0) return MXFP4_MISALIGNED;
    } else {
        if ((s = check_mat(*src_q, rows, cols))) return s;
    }
    if (rows == 0 || cols == 0) return MXFP4_OK;
    fill_padding_if_needed(dst_t.scales, cols, rows, st);
    if (dst) fill_padding_if_needed(dst->scales, rows, cols, st);
    const dim3 grid((unsigned)ceil_div(cols, kTileC), (unsigned)ceil_div(rows, kTileR));
    QuantSide tr = make_side(dst_t, qp_t);
    QuantSide rw = dst ? make_side(*dst, qp_row) : tr;
    if (src_q)
        k_quantize_tile<true, false><<<grid, 256, 0, st>>>(src_q->data, src_q->scales, (int)ceil_div(cols / 32, 4), rows,
                                                           cols, cols, rw, tr, dev_status);
    else if (dst)
        k_quantize_tile<false, true><<<grid, 256, 0, st>>>(src_bf16, nullptr, 0, rows, cols, ld, rw, tr, dev_status);
    else
        k_quantize_tile<false, false><<<grid, 256, 0, st>>>(src_bf16, nullptr, 0, rows, cols, ld, rw, tr, dev_status);
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
                         static_cast<cudaStream_t>(stream));
}

mxfp4_status_t mxfp4_quantize_2axis(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                                    const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t, const mxfp4_qparams_t *qp_t,
                                    uint32_t *dev_status, void *stream)
{
    if (!src_bf16) return MXFP4_INVALID_ARG;
    return quantize_tile(src_bf16, nullptr, rows, cols, ld, &dst, qp_row, dst_t, qp_t, dev_status,
                         static_cast<cudaStream_t>(stream));
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
    const unsigned blocks = (unsigned)ceil_div(n * nblk, 128);
    if (osc)
        k_qema<true><<<blocks, 128, 0, st>>>(static_cast<const __nv_bfloat16 *>(w_bf16), ema, beta, update_ema, n, nblk,
                                             static_cast<uint8_t *>(dst.data), dst.scales, nblk4, scale_mode, op, dev_status);
    else
        k_qema<false><<<blocks, 128, 0, st>>>(static_cast<const __nv_bfloat16 *>(w_bf16), ema, beta, update_ema, n, nblk,
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
