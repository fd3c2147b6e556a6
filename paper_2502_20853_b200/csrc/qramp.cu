// Q-Ramping (Sec. 6, Algorithm 2): the ramp factor of every weight element from its oscillation ratio, and the
// optimizer step that accumulates each element's gradient over its own number of steps.
// Both are single passes over per-element state: HBM-bound, 128-bit accesses, four elements per thread.
#include "common.cuh"
#include <math.h>

namespace mx {

// Algorithm 2, OscillationDetection: R_w = dist_Q / dist_W (Sec. 6.1), n_w = min(k2 floor(R_w / k1) + 1, N_max).
// Both quotients are single IEEE divisions in FP32.  dist_W = 0: R_w = +inf if dist_Q > 0, else 0; NaN: n_w = 1.
__device__ __forceinline__ uint32_t ramp_factor(float dw, float dq, float k1, float inv_k1, int k2, int n_max, bool &oscillating)
{
    const float r = dw == 0.0f ? (dq > 0.0f ? __int_as_float(0x7F800000) : 0.0f) : __fdiv_rn(dq, dw);
    oscillating = r > k1;                            // false for NaN
    if (!(r == r)) return 1u;
    // inv_k1 != 0: k1 is a power of two and multiplying by its reciprocal is the same correctly rounded quotient
    const float steps = floorf(inv_k1 != 0.0f ? __fmul_rn(r, inv_k1) : __fdiv_rn(r, k1));
    if (!(steps >= 1.0f)) return 1u;                 // also negative ratios (inputs that are not sums of magnitudes)
    if (steps >= (float)n_max) return (uint32_t)n_max;   // k2 >= 1: k2 * steps + 1 > N_max
    const int64_t n = (int64_t)k2 * (int64_t)steps + 1;
    return (uint32_t)(n < n_max ? n : n_max);
}

__global__ void __launch_bounds__(256) k_qramp_detect(const float *__restrict__ dist_w, const float *__restrict__ dist_q,
                                                      int64_t count, float k1, float inv_k1, int k2, int n_max,
                                                      uint8_t *__restrict__ n_w, unsigned long long *oscillating)
{
    // a fixed number of blocks walks the array, so that the count of oscillating elements costs one atomic per block
    __shared__ uint32_t s_osc[8];
    uint32_t osc = 0;
    const int64_t octs = (count + 7) / 8;     // eight elements per thread and turn: 64 bytes of loads in flight
    for (int64_t q = blockIdx.x * (int64_t)256 + threadIdx.x; q < octs; q += (int64_t)gridDim.x * 256) {
        const int64_t i0 = q * 8;
        if (i0 + 7 < count) {
            const float4 a0 = *reinterpret_cast<const float4 *>(dist_w + i0), a1 = *reinterpret_cast<const float4 *>(dist_w + i0 + 4);
            const float4 b0 = *reinterpret_cast<const float4 *>(dist_q + i0), b1 = *reinterpret_cast<const float4 *>(dist_q + i0 + 4);
            const float aw[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bq[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            uint32_t lo = 0, hi = 0;
#pragma unroll
            for (int j = 0; j < 8; j++) {
                bool o;
                const uint32_t n = ramp_factor(aw[j], bq[j], k1, inv_k1, k2, n_max, o);
                if (j < 4) lo |= n << (8 * j); else hi |= n << (8 * (j - 4));
                osc += (uint32_t)o;
            }
            *reinterpret_cast<uint2 *>(n_w + i0) = make_uint2(lo, hi);
        } else {
            for (int64_t i = i0; i < count; i++) {
                bool o;
                n_w[i] = (uint8_t)ramp_factor(dist_w[i], dist_q[i], k1, inv_k1, k2, n_max, o);
                osc += (uint32_t)o;
            }
        }
    }
    if (oscillating) {
        osc = __reduce_add_sync(0xFFFFFFFFu, osc);
        if ((threadIdx.x & 31) == 0) s_osc[threadIdx.x >> 5] = osc;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t t = 0;
            for (int i = 0; i < 8; i++) t += s_osc[i];
            if (t) atomicAdd(oscillating, (unsigned long long)t);
        }
    }
}

struct AdamW {
    float lr, b1, b2, eps, wd, c1, c2;
};

// One element of the customized AdamW (the reading stated with mxfp4_qramp_adamw).  Returns true if it was updated.
__device__ __forceinline__ bool adamw_one(float &w, float g, float &m, float &v, float &acc, uint32_t &cnt, uint32_t n, const AdamW &h)
{
    acc = __fadd_rn(acc, g);
    cnt += 1u;
    if (cnt < n) return false;
    const float gbar = __fdiv_rn(acc, (float)cnt);
    m = __fadd_rn(__fmul_rn(h.b1, m), __fmul_rn(__fsub_rn(1.0f, h.b1), gbar));
    v = __fadd_rn(__fmul_rn(h.b2, v), __fmul_rn(__fmul_rn(__fsub_rn(1.0f, h.b2), gbar), gbar));
    const float step = __fadd_rn(__fdiv_rn(__fdiv_rn(m, h.c1), __fadd_rn(__fsqrt_rn(__fdiv_rn(v, h.c2)), h.eps)), __fmul_rn(h.wd, w));
    w = __fsub_rn(w, __fmul_rn(__fmul_rn((float)n, h.lr), step));
    acc = 0.0f;
    cnt = 0u;
    return true;
}

__global__ void __launch_bounds__(256) k_qramp_adamw(float *__restrict__ w, __nv_bfloat16 *__restrict__ w_bf16,
                                                     const float *__restrict__ grad, float *__restrict__ m, float *__restrict__ v,
                                                     float *__restrict__ acc, uint8_t *__restrict__ cnt,
                                                     const uint8_t *__restrict__ n_w, int64_t count, const AdamW h)
{
    const int64_t i0 = (blockIdx.x * (int64_t)256 + threadIdx.x) * 4;
    if (i0 + 3 < count) {
        float4 W = *reinterpret_cast<const float4 *>(w + i0), G = *reinterpret_cast<const float4 *>(grad + i0);
        float4 M = *reinterpret_cast<const float4 *>(m + i0), V = *reinterpret_cast<const float4 *>(v + i0);
        float4 A = *reinterpret_cast<const float4 *>(acc + i0);
        const uint32_t c4 = *reinterpret_cast<const uint32_t *>(cnt + i0);
        const uint32_t n4 = n_w ? *reinterpret_cast<const uint32_t *>(n_w + i0) : 0x01010101u;
        uint32_t c0 = c4 & 0xFFu, c1 = (c4 >> 8) & 0xFFu, c2 = (c4 >> 16) & 0xFFu, c3 = c4 >> 24;
        bool u = adamw_one(W.x, G.x, M.x, V.x, A.x, c0, n4 & 0xFFu, h);
        u |= adamw_one(W.y, G.y, M.y, V.y, A.y, c1, (n4 >> 8) & 0xFFu, h);
        u |= adamw_one(W.z, G.z, M.z, V.z, A.z, c2, (n4 >> 16) & 0xFFu, h);
        u |= adamw_one(W.w, G.w, M.w, V.w, A.w, c3, n4 >> 24, h);
        *reinterpret_cast<float4 *>(acc + i0) = A;
        *reinterpret_cast<uint32_t *>(cnt + i0) = (c0 & 0xFFu) | ((c1 & 0xFFu) << 8) | ((c2 & 0xFFu) << 16) | (c3 << 24);
        if (u) {   // weights and moments change only where a window closed
            *reinterpret_cast<float4 *>(w + i0) = W;
            *reinterpret_cast<float4 *>(m + i0) = M;
            *reinterpret_cast<float4 *>(v + i0) = V;
            if (w_bf16) {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(W.x, W.y), hi = __floats2bfloat162_rn(W.z, W.w);
                uint2 o;
                o.x = *reinterpret_cast<const uint32_t *>(&lo);
                o.y = *reinterpret_cast<const uint32_t *>(&hi);
                *reinterpret_cast<uint2 *>(w_bf16 + i0) = o;
            }
        }
    } else {
        for (int64_t i = i0; i < count; i++) {
            float W = w[i], M = m[i], V = v[i], A = acc[i];
            uint32_t c = cnt[i];
            const bool u = adamw_one(W, grad[i], M, V, A, c, n_w ? n_w[i] : 1u, h);
            acc[i] = A;
            cnt[i] = (uint8_t)c;
            if (u) {
                w[i] = W; m[i] = M; v[i] = V;
                if (w_bf16) w_bf16[i] = __float2bfloat16_rn(W);
            }
        }
    }
}

static bool al16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool al4(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

}  // namespace mx

using namespace mx;

extern "C" {

mxfp4_status_t mxfp4_qramp_detect(const float *dist_w, const float *dist_q, int64_t count, float k1, int32_t k2, int32_t n_max,
                                  uint8_t *n_w, unsigned long long *oscillating, void *stream)
{
    if (count < 0 || !(k1 > 0.0f) || k2 < 1 || n_max < 1 || n_max > 255) return MXFP4_INVALID_ARG;
    if (count == 0) return MXFP4_OK;
    if (!dist_w || !dist_q || !n_w) return MXFP4_INVALID_ARG;
    if (!al16(dist_w) || !al16(dist_q) || (reinterpret_cast<uintptr_t>(n_w) & 7u) || (reinterpret_cast<uintptr_t>(oscillating) & 7u)) return MXFP4_MISALIGNED;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms = 148;
    int e = 0;
    const float inv_k1 = (frexpf(k1, &e) == 0.5f && e > -100 && e < 100) ? 1.0f / k1 : 0.0f;   // exact only for powers of two
    const int64_t want = ceil_div(ceil_div(count, 8), 256);
    const unsigned blocks = (unsigned)(want < (int64_t)sms * 8 ? want : (int64_t)sms * 8);
    k_qramp_detect<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(dist_w, dist_q, count, k1, inv_k1, k2, n_max, n_w, oscillating);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

mxfp4_status_t mxfp4_qramp_adamw(float *w, void *w_bf16, const float *grad, float *m, float *v, float *acc, uint8_t *cnt,
                                 const uint8_t *n_w, int64_t count, const mxfp4_adamw_t *hp, void *stream)
{
    if (count < 0 || !hp) return MXFP4_INVALID_ARG;
    if (!(hp->bias_corr1 > 0.0f) || !(hp->bias_corr2 > 0.0f) || !(hp->beta1 >= 0.0f && hp->beta1 < 1.0f) ||
        !(hp->beta2 >= 0.0f && hp->beta2 < 1.0f) || !(hp->eps >= 0.0f))
        return MXFP4_INVALID_ARG;
    if (count == 0) return MXFP4_OK;
    if (!w || !grad || !m || !v || !acc || !cnt) return MXFP4_INVALID_ARG;
    if (!al16(w) || !al16(grad) || !al16(m) || !al16(v) || !al16(acc) || !al4(cnt) || !al4(n_w) ||
        (reinterpret_cast<uintptr_t>(w_bf16) & 7u))
        return MXFP4_MISALIGNED;
    const AdamW h = {hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay, hp->bias_corr1, hp->bias_corr2};
    const unsigned blocks = (unsigned)ceil_div(ceil_div(count, 4), 256);
    k_qramp_adamw<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(w, static_cast<__nv_bfloat16 *>(w_bf16), grad, m, v, acc, cnt,
                                                                        n_w, count, h);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

}  // extern "C"
