// MX quantizer kernels for sm_100a: row-wise, transposed / two-axis (a persistent TMA-fed tile kernel), double
// quantization of a packed source, Q-EMA, dequantize.  Element passes over HBM: scales are written straight into the
// 128x4 tiled order the GEMM consumes.
#include "common.cuh"
#include "quant_tile.cuh"
#include "tma.cuh"

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
    MX_LAUNCHED();
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
// Double quantization (Sec. 3.3) of an MXFP4 matrix along its other axis: Q4 and Q6 of Eq. 4-5.  A CTA owns a
// 128-row x 128-column tile of the packed source, which is exactly one 512-byte chunk of the tiled scale buffer of
// the source and of the output.  The tile is dequantized exactly into shared memory as bf16 on the way in, then the
// column pass re-quantizes it: a thread takes 16 consecutive rows of 4 columns, two lanes per group; the result is
// the transposed matrix, staged in shared memory and written out in 64-byte rows.  The random bits of 16
// consecutive elements of the output come from one Philox call.  The scale chunk is assembled in shared memory
// (padding entries 0x7F) and written whole.
// ------------------------------------------------------------------------------------------------
constexpr int kPitch = 2 * kTile + 16;   // bytes per staged row (16-byte skew against bank conflicts)

template <bool SR_T>
__global__ void __launch_bounds__(256, 4) k_requantize_tile(const void *__restrict__ src, const uint8_t *__restrict__ src_scales,
                                                            int src_nblk4, int rows, int cols, const __grid_constant__ QuantSide tr,
                                                            uint32_t *dev_status)
{
    __shared__ __align__(16) uint8_t s_in[kTile * kPitch];
    __shared__ __align__(16) uint2 s_out[kTile * 8];          // [output row = source column][8-byte slot], slots XOR-swizzled
    __shared__ __align__(16) uint8_t s_sc_t[512];

    const int tid = threadIdx.x;
    const int row0 = blockIdx.y * kTile, col0 = blockIdx.x * kTile;
    uint32_t nonfinite = 0;

    if (tid < 32) reinterpret_cast<uint4 *>(s_sc_t)[tid] = make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);

    // ---- stage the tile ----
    {
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
        // the scale chunk of this tile
        if (tid < 32)
            reinterpret_cast<uint4 *>(tr.scales + ((size_t)(col0 >> 7) * tr.nblk4 + (row0 >> 7)) * 512)[tid] =
                reinterpret_cast<const uint4 *>(s_sc_t)[tid];
    }
    if (nonfinite && dev_status) atomicOr(dev_status, MXFP4_DEV_NONFINITE);
}

// ------------------------------------------------------------------------------------------------
// Streaming two-axis quantizer for bf16 sources (Q3 + Q5 of Eq. 4-5, Q1 + Q6 by double quantization, or the
// transposed quantizer alone).  Persistent: two CTAs per SM walk over the 128 x 128 tiles; one thread feeds a ring of
// two tiles with TMA (each tile arrives as two 128B-swizzled boxes of 128 rows x 64 columns), so the next tile travels
// while this one is quantized, and nothing of the staging costs an instruction of the computing threads.
//   row pass   : a thread takes one whole 32-element group of a row (four 16-byte pieces) twice per tile and
//                stores its 16 bytes of codes straight to global memory;
//   column pass: a thread takes two adjacent columns x 32 rows (a bf16 pair per row), i.e. two whole groups of
//                the transposed output, scaled together by packed multiplies; the transposed codes are staged in a
//                64B-swizzled tile that leaves with one TMA store (clipped at the matrix edges).
// Both 512-byte scale chunks of a tile are assembled in shared memory (entries outside the matrix 0x7F) and leave
// as bulk copies.  The staging is double buffered: a tile's stores are read out while the next tile is computed.
// Random bits are drawn per 16 consecutive elements of each OUTPUT, as in every other quantizer here.
// ------------------------------------------------------------------------------------------------
constexpr int kQsThreads = 256;
constexpr int kQsStagingBytes = kTile * 64 + 1024;     // transposed codes (8 KB, 64B-swizzled) + the two scale chunks
constexpr int kQsBarOff = 2 * kTileBytes + 2 * kQsStagingBytes;
constexpr int kQsSmemBytes = kQsBarOff + 64 + 1024 /*align*/;
constexpr int kQsCtasPerSm = 2;

template <bool EMIT_ROW, bool SR_ROW, bool SR_T, bool DQ>
__global__ void __launch_bounds__(kQsThreads, kQsCtasPerSm)
k_quantize_stream(const __grid_constant__ CUtensorMap map_src, const __grid_constant__ CUtensorMap map_t, int rows, int cols,
                  const __grid_constant__ QuantSide rw, const __grid_constant__ QuantSide tr, uint32_t *dev_status, uint32_t spin_limit,
                  int withhold_loads)
{
    extern __shared__ uint8_t qs_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(qs_smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_full = smem_base + kQsBarOff;
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kQsBarOff + 32);

    const int tid = threadIdx.x;
    const int ntx = (cols + kTile - 1) / kTile, nty = (rows + kTile - 1) / kTile;
    const int total = ntx * nty;

    auto issue_load = [&](int tile, int stage) {
        const int ty = tile / ntx, tx = tile - ty * ntx;
        const uint32_t bar = bar_full + 8 * stage, dst = smem_base + stage * kTileBytes;
        mbar_expect_tx(bar, kTileBytes);
        tma_load_2d(dst, &map_src, tx * kTile, ty * kTile, bar);
        tma_load_2d(dst + kTileBytes / 2, &map_src, tx * kTile + 64, ty * kTile, bar);
    };

    if (tid == 0) {
        mbar_init(bar_full, 1);
        mbar_init(bar_full + 8, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // withhold_loads (self-test of the drain path): nothing is ever loaded, so the first bounded wait runs out
        for (int s = 0; s < 2; s++)
            if (!withhold_loads && (int)blockIdx.x + s * (int)gridDim.x < total) issue_load(blockIdx.x + s * gridDim.x, s);
    }
    __syncthreads();

    const QsGeom g = qs_geom(tid);
    const uint32_t tfa_r = tf_add_of(rw.scale_mode), tfa_t2 = tf_add_of(tr.scale_mode) * 0x00010001u;
    uint32_t nonfinite = 0;
    // tile coordinates advance by the grid size without a division per tile
    const int step_y = (int)gridDim.x / ntx, step_x = (int)gridDim.x - step_y * ntx;
    int ty = (int)blockIdx.x / ntx, tx = (int)blockIdx.x - ty * ntx;
    int it = 0;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x, it++) {
        const int stage = it & 1;
        const int row0 = ty * kTile, col0 = tx * kTile;
        const uint32_t st_base = smem_base + stage * kTileBytes;
        uint8_t *staging = smem + 2 * kTileBytes + stage * kQsStagingBytes;
        uint8_t *s_sc_row = staging + kTile * 64, *s_sc_t = s_sc_row + 512;

        const bool ok = mbar_wait(bar_full + 8 * stage, (uint32_t)(it >> 1) & 1u, abort_flag, dev_status, spin_limit);

        if (EMIT_ROW && ok) qs_row_pass<SR_ROW, DQ>(g, st_base, st_base, row0, col0, rows, cols, rw, tfa_r, s_sc_row, nonfinite);
        if (DQ) __syncwarp();      // the column pass reads what the row pass of the SAME warp wrote back

        if (ok) qs_col_pass<SR_T>(g, st_base, row0, col0, rows, cols, tr, tfa_t2, staging, s_sc_t, nonfinite);

        // ---- hand the tile's results to the copy engine, refill the ring ----
        fence_async_smem();                       // this thread's staging writes, before the asynchronous reads
        if (tid == 0) bulk_wait_read<0>();        // the previous tile's stores have left the other staging buffer
        if (__syncthreads_or(!ok)) break;          // a bounded wait ran out somewhere in the CTA: everybody leaves
        if (tid == 0) {
            tma_store_2d(&map_t, row0 >> 1, col0, smem_u32(staging));
            bulk_store(tr.scales + ((size_t)(col0 >> 7) * tr.nblk4 + (row0 >> 7)) * 512, smem_u32(s_sc_t), 512);
            if (EMIT_ROW) bulk_store(rw.scales + ((size_t)(row0 >> 7) * rw.nblk4 + (col0 >> 7)) * 512, smem_u32(s_sc_row), 512);
            bulk_commit();
            const int next = tile + 2 * (int)gridDim.x;
            if (next < total) issue_load(next, stage);
        }
        tx += step_x;
        ty += step_y;
        if (tx >= ntx) { tx -= ntx; ty++; }
    }
    if (tid == 0) bulk_wait0();                   // every store has completed before the shared memory goes away
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
    MX_CHECK_LAUNCH();
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

// bf16 source [rows, cols] (leading dimension ld) as a 2-D tensor of bf16; box = 64 columns x 128 rows, 128B swizzle.
static bool make_src_map(CUtensorMap *map, const void *src, int64_t rows, int64_t cols, int64_t ld)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    cuuint32_t estr[2] = {1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(src), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Packed transposed output [cols, rows / 2 bytes] as a 2-D byte tensor; box = 64 bytes x 128 rows, 64B swizzle.
static bool make_packed_t_map(CUtensorMap *map, void *packed, int64_t rows, int64_t cols)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)(rows / 2), (cuuint64_t)cols};
    cuuint64_t gstride[1] = {(cuuint64_t)(rows / 2)};
    cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    cuuint32_t estr[2] = {1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, packed, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool EMIT_ROW, bool SR_ROW, bool SR_T, bool DQ>
static mxfp4_status_t launch_stream(cudaStream_t st, const CUtensorMap &ms, const CUtensorMap &mt, int rows, int cols, const QuantSide &rw,
                                    const QuantSide &tr, uint32_t *dev_status, uint32_t spin_limit = kWaitSpinLimit, int withhold_loads = 0)
{
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_quantize_stream<EMIT_ROW, SR_ROW, SR_T, DQ>, kQsSmemBytes));
    const int64_t tiles = ceil_div(rows, kTile) * ceil_div(cols, kTile);
    const int64_t cap = kQsCtasPerSm * (int64_t)sm_count();
    const int grid = (int)(tiles < cap ? tiles : cap);
    k_quantize_stream<EMIT_ROW, SR_ROW, SR_T, DQ><<<grid, kQsThreads, kQsSmemBytes, st>>>(ms, mt, rows, cols, rw, tr, dev_status, spin_limit, withhold_loads);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

// src_bf16 xor src_q; dst (row-wise) optional; dst_t required.  chain: dst_t is quantized from the dequantized dst
// (double quantization) instead of from the source; needs a bf16 source and dst.
// spin_limit / withhold_loads: normal use kWaitSpinLimit / 0; the self-test of the drain path withholds the loads of the
// streaming kernel so that its bounded waits run out after spin_limit polls.
static mxfp4_status_t quantize_tile_ex(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows, int64_t cols, int64_t ld,
                                       const mxfp4_mat_t *dst, const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t,
                                       const mxfp4_qparams_t *qp_t, uint32_t *dev_status, cudaStream_t st, bool chain, uint32_t spin_limit,
                                       int withhold_loads)
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
    if (src_q && grid.y > 65535u) return MXFP4_BAD_SHAPE;
    const QuantSide tr = make_side(dst_t, qp_t);
    const QuantSide rw = dst ? make_side(*dst, qp_row) : tr;
    const bool sr_t = qp_t->rounding == MXFP4_ROUND_STOCHASTIC;
    const bool sr_r = dst && qp_row->rounding == MXFP4_ROUND_STOCHASTIC;
    const int r = (int)rows, c = (int)cols;
    if (src_q) {
        const int nb4 = (int)ceil_div(cols / 32, 4);
        if (sr_t) k_requantize_tile<true><<<grid, 256, 0, st>>>(src_q->data, src_q->scales, nb4, r, c, tr, dev_status);
        else k_requantize_tile<false><<<grid, 256, 0, st>>>(src_q->data, src_q->scales, nb4, r, c, tr, dev_status);
    } else {
        // bf16 source: the streaming kernel
        if (ceil_div(rows, kTile) * ceil_div(cols, kTile) > 0x7FFFFFFF) return MXFP4_BAD_SHAPE;
        CUtensorMap ms, mt;
        if (!make_src_map(&ms, src_bf16, rows, cols, ld) || !make_packed_t_map(&mt, dst_t.data, rows, cols)) return MXFP4_CUDA_ERROR;
        if (!dst) {
            return sr_t ? launch_stream<false, false, true, false>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads)
                        : launch_stream<false, false, false, false>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        }
        const int sel = (chain ? 4 : 0) | (sr_r ? 2 : 0) | (sr_t ? 1 : 0);
        switch (sel) {
        case 0: return launch_stream<true, false, false, false>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        case 1: return launch_stream<true, false, true, false>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        case 2: return launch_stream<true, true, false, false>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        case 3: return launch_stream<true, true, true, false>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        case 4: return launch_stream<true, false, false, true>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        case 5: return launch_stream<true, false, true, true>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        case 6: return launch_stream<true, true, false, true>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        default: return launch_stream<true, true, true, true>(st, ms, mt, r, c, rw, tr, dev_status, spin_limit, withhold_loads);
        }
    }
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

mxfp4_status_t quantize_tile(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows, int64_t cols, int64_t ld,
                             const mxfp4_mat_t *dst, const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t,
                             const mxfp4_qparams_t *qp_t, uint32_t *dev_status, cudaStream_t st, bool chain)
{
    return quantize_tile_ex(src_bf16, src_q, rows, cols, ld, dst, qp_row, dst_t, qp_t, dev_status, st, chain, kWaitSpinLimit, 0);
}

std::atomic<unsigned long long> g_launches{0};

}  // namespace mx

using namespace mx;

extern "C" {

uint64_t mxfp4_launch_count(void) { return (uint64_t)mx::g_launches.load(std::memory_order_relaxed); }

mxfp4_status_t mxfp4_quantize_wait_selftest(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                                            mxfp4_mat_t dst_t, uint32_t spin_limit, uint32_t *dev_status, void *stream)
{
    if (!src_bf16 || !dev_status || spin_limit < 128u || spin_limit > (1u << 16)) return MXFP4_INVALID_ARG;
    const mxfp4_qparams_t qp = {MXFP4_SCALE_TRUNCATION_FREE, MXFP4_ROUND_NEAREST, 0, 0, 0};
    return quantize_tile_ex(src_bf16, nullptr, rows, cols, ld, &dst, &qp, dst_t, &qp, dev_status, static_cast<cudaStream_t>(stream), false,
                            spin_limit, 1);
}

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
    MX_CHECK_LAUNCH();
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
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

}  // extern "C"
