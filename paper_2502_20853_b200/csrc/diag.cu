// Diagnostics of Sec. 4 and Appendix A computed on the device: the histogram of the quantization confidence of a
// weight matrix (Sec. 4.2, App. A.2) and the two sums behind the rate of change of a tensor (App. A.3).
// Single passes over the data; the reductions go through shared memory and a few atomics per block.
#include "common.cuh"

namespace mx {

// rounding thresholds of the E2M1 grid (midpoints of neighbouring values), framed by the mirror image of the first
// one and by the largest grid value: cell c of a latent magnitude is [c_thr[c], c_thr[c + 1]]
__constant__ float c_thr[9] = {-0.25f, 0.25f, 0.75f, 1.25f, 1.75f, 2.5f, 3.5f, 5.0f, 6.0f};
__constant__ float c_e2m1[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

// QuantConf(w) = min_i |a - thrd_i| / MaxDist(w_FP4) for the latent magnitude a = |w| / 2^s.  MaxDist is half the
// width of the cell; the cell of 6 is [5, 6] and counts from its only threshold; beyond 6 the confidence is 1.
__device__ __forceinline__ float quant_conf(float a)
{
    const int cell = (a > 0.25f) + (a > 0.75f) + (a > 1.25f) + (a > 1.75f) + (a > 2.5f) + (a > 3.5f) + (a > 5.0f);
    const float lo = c_thr[cell], hi = c_thr[cell + 1];
    float d, maxdist;
    if (cell == 7) {
        d = __fsub_rn(a, lo);
        maxdist = 1.0f;
    } else {
        d = fminf(__fsub_rn(a, lo), __fsub_rn(hi, a));
        maxdist = __fmul_rn(0.5f, __fsub_rn(hi, lo));
    }
    return fminf(__fdiv_rn(d, maxdist), 1.0f);
}

constexpr int kMaxBins = 64;

// One thread per 32-element group, as in the row-wise quantizer (same scale rule, Sec. 3.2).  Every thread counts into
// a private column of bytes in shared memory (a group has 32 elements, so a byte holds any count): no atomics while
// counting; the columns are added up per bin at the end and the block adds its totals to the global histogram.
__global__ void __launch_bounds__(256) k_quant_conf_hist(const __nv_bfloat16 *__restrict__ w, int64_t rows, int nblk, int scale_mode,
                                                         int bins, unsigned long long *__restrict__ hist)
{
    __shared__ __align__(16) uint8_t s_cnt[kMaxBins * 256];   // [bin][thread]
    for (int i = threadIdx.x; i < bins * 64; i += 256) reinterpret_cast<uint32_t *>(s_cnt)[i] = 0u;
    __syncthreads();
    const int64_t gid = blockIdx.x * (int64_t)256 + threadIdx.x;
    if (gid < rows * nblk) {
        const uint4 *p = reinterpret_cast<const uint4 *>(w + gid * 32);
        uint4 q[4];
#pragma unroll
        for (int j = 0; j < 4; j++) q[j] = ld_nc_16(p + j);
        uint32_t am = 0;
#pragma unroll
        for (int j = 0; j < 4; j++) {
            am = absmax2(am, q[j].x); am = absmax2(am, q[j].y); am = absmax2(am, q[j].z); am = absmax2(am, q[j].w);
        }
        am = hmax_halves(am);
        if (am < 0x7F80u) {   // groups with Inf / NaN are skipped
            const float inv = inv_scale_from_byte(scale_byte_from_amax(am, tf_add_of(scale_mode)));
            const float fb = (float)bins;
            uint8_t *mine = s_cnt + threadIdx.x;
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const uint32_t ws[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
                for (int t = 0; t < 4; t++) {
                    const float a0 = __fmul_rn(fabsf(bf16lo(ws[t])), inv), a1 = __fmul_rn(fabsf(bf16hi(ws[t])), inv);
                    const int b0 = min((int)floorf(__fmul_rn(quant_conf(a0), fb)), bins - 1);
                    const int b1 = min((int)floorf(__fmul_rn(quant_conf(a1), fb)), bins - 1);
                    mine[b0 * 256] += 1;
                    mine[b1 * 256] += 1;
                }
            }
        }
    }
    __syncthreads();
    // bin b: 256 bytes = 64 words; warp w takes bins w, w + 8, ...; a lane adds the bytes of two words
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int b = warp; b < bins; b += 8) {
        const uint2 v = reinterpret_cast<const uint2 *>(s_cnt + b * 256)[lane];
        uint32_t t = __dp4a(v.x, 0x01010101u, 0u);
        t = __dp4a(v.y, 0x01010101u, t);
        t = __reduce_add_sync(0xFFFFFFFFu, t);
        if (lane == 0 && t) atomicAdd(hist + b, (unsigned long long)t);
    }
}

// block-wide sum of two floats per thread into two doubles in global memory
__device__ __forceinline__ void block_add2(float a, float b, double *out)
{
    __shared__ float s_a[8], s_b[8];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
        b += __shfl_xor_sync(0xFFFFFFFFu, b, o);
    }
    if ((threadIdx.x & 31) == 0) { s_a[threadIdx.x >> 5] = a; s_b[threadIdx.x >> 5] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double ta = 0.0, tb = 0.0;
        for (int i = 0; i < 8; i++) { ta += (double)s_a[i]; tb += (double)s_b[i]; }
        atomicAdd(out, ta);
        atomicAdd(out + 1, tb);
    }
}

__global__ void __launch_bounds__(256) k_change_sums(const __nv_bfloat16 *__restrict__ cur, const __nv_bfloat16 *__restrict__ prev,
                                                     int64_t count, double *__restrict__ out)
{
    float d2 = 0.f, p2 = 0.f;
    const int64_t octs = count / 8;
    for (int64_t i = blockIdx.x * (int64_t)256 + threadIdx.x; i < octs; i += (int64_t)gridDim.x * 256) {
        const uint4 c = ld_nc_16(reinterpret_cast<const uint4 *>(cur) + i), p = ld_nc_16(reinterpret_cast<const uint4 *>(prev) + i);
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, pw[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
        for (int t = 0; t < 4; t++) {
            const float p0 = bf16lo(pw[t]), p1 = bf16hi(pw[t]);
            const float e0 = bf16lo(cw[t]) - p0, e1 = bf16hi(cw[t]) - p1;
            d2 = fmaf(e0, e0, d2); d2 = fmaf(e1, e1, d2);
            p2 = fmaf(p0, p0, p2); p2 = fmaf(p1, p1, p2);
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t i = octs * 8; i < count; i++) {
            const float p = __bfloat162float(prev[i]), e = __bfloat162float(cur[i]) - p;
            d2 = fmaf(e, e, d2);
            p2 = fmaf(p, p, p2);
        }
    }
    block_add2(d2, p2, out);
}

// the same for two quantized matrices of one shape: values = E2M1 value x 2^s; one thread per group
__global__ void __launch_bounds__(256) k_change_sums_q(const uint8_t *__restrict__ cp, const uint8_t *__restrict__ cs,
                                                       const uint8_t *__restrict__ pp, const uint8_t *__restrict__ ps, int64_t rows,
                                                       int nblk, int nblk4, double *__restrict__ out)
{
    float d2 = 0.f, p2 = 0.f;
    const int64_t gid = blockIdx.x * (int64_t)256 + threadIdx.x;
    if (gid < rows * nblk) {
        const int64_t row = gid / nblk;
        const int blk = (int)(gid - row * nblk);
        const uint4 c = *reinterpret_cast<const uint4 *>(cp + gid * 16), p = *reinterpret_cast<const uint4 *>(pp + gid * 16);
        const size_t so = scale_offset(row, blk, nblk4);
        const uint32_t cb = cs[so], pb = ps[so];
        const float csc = cb == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(cb);
        const float psc = pb == 0xFFu ? __uint_as_float(0x7FC00000u) : scale_from_byte(pb);
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, pw[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
        for (int t = 0; t < 4; t++)
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const uint32_t cc = (cw[t] >> (4 * i)) & 15u, pc = (pw[t] >> (4 * i)) & 15u;
                const float cv = (cc & 8u ? -c_e2m1[cc & 7u] : c_e2m1[cc & 7u]) * csc;
                const float pv = (pc & 8u ? -c_e2m1[pc & 7u] : c_e2m1[pc & 7u]) * psc;
                const float e = cv - pv;
                d2 = fmaf(e, e, d2);
                p2 = fmaf(pv, pv, p2);
            }
    }
    block_add2(d2, p2, out);
}

static bool al16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace mx

using namespace mx;

extern "C" {

mxfp4_status_t mxfp4_quant_conf_hist(const void *w_bf16, int64_t n, int64_t k, int32_t scale_mode, int32_t bins,
                                     unsigned long long *hist, void *stream)
{
    if (n < 0 || k < 0 || bins < 1 || bins > kMaxBins || !hist) return MXFP4_INVALID_ARG;
    if (scale_mode != MXFP4_SCALE_TRUNCATION_FREE && scale_mode != MXFP4_SCALE_FLOOR) return MXFP4_INVALID_ARG;
    if (k % 32 != 0) return MXFP4_BAD_SHAPE;
    if (n == 0 || k == 0) return MXFP4_OK;
    if (!w_bf16) return MXFP4_INVALID_ARG;
    if (!al16(w_bf16) || (reinterpret_cast<uintptr_t>(hist) & 7u)) return MXFP4_MISALIGNED;
    const int nblk = (int)(k / 32);
    const unsigned blocks = (unsigned)ceil_div(n * nblk, 256);
    k_quant_conf_hist<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const __nv_bfloat16 *>(w_bf16), n, nblk,
                                                                            scale_mode, bins, hist);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

mxfp4_status_t mxfp4_change_sums(const void *cur_bf16, const void *prev_bf16, int64_t count, double *out, void *stream)
{
    if (count < 0 || !out) return MXFP4_INVALID_ARG;
    if (count == 0) return MXFP4_OK;
    if (!cur_bf16 || !prev_bf16) return MXFP4_INVALID_ARG;
    if (!al16(cur_bf16) || !al16(prev_bf16) || (reinterpret_cast<uintptr_t>(out) & 7u)) return MXFP4_MISALIGNED;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms = 148;
    const int64_t want = ceil_div(ceil_div(count, 8), 256);
    const unsigned blocks = (unsigned)(want < (int64_t)sms * 8 ? (want > 0 ? want : 1) : (int64_t)sms * 8);
    k_change_sums<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const __nv_bfloat16 *>(cur_bf16),
                                                                        static_cast<const __nv_bfloat16 *>(prev_bf16), count, out);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

mxfp4_status_t mxfp4_change_sums_q(mxfp4_mat_t cur, mxfp4_mat_t prev, double *out, void *stream)
{
    if (!out || cur.rows < 0 || cur.cols < 0) return MXFP4_INVALID_ARG;
    if (cur.rows != prev.rows || cur.cols != prev.cols || cur.cols % 32 != 0) return MXFP4_BAD_SHAPE;
    if (cur.rows == 0 || cur.cols == 0) return MXFP4_OK;
    if (!cur.data || !cur.scales || !prev.data || !prev.scales) return MXFP4_INVALID_ARG;
    if (!al16(cur.data) || !al16(prev.data) || (reinterpret_cast<uintptr_t>(out) & 7u)) return MXFP4_MISALIGNED;
    const int nblk = (int)(cur.cols / 32), nblk4 = (nblk + 3) / 4;
    const unsigned blocks = (unsigned)ceil_div(cur.rows * nblk, 256);
    k_change_sums_q<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint8_t *>(cur.data), cur.scales,
                                                                          static_cast<const uint8_t *>(prev.data), prev.scales, cur.rows,
                                                                          nblk, nblk4, out);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

}  // extern "C"
