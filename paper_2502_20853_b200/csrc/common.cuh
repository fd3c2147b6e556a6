// Device-side building blocks of the MXFP4 quantizers (sm_100a).
// Definitions follow Sec. 3.1-3.2 of the paper (E2M1 grid, shared power-of-two scale,
// deterministic and stochastic rounding); Philox4x32-10 is the random source.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxfp4.h"

namespace mx {

constexpr int kGroup = 32;

#define MX_CHECK_CUDA(expr)                                  \
    do {                                                     \
        cudaError_t e_ = (expr);                             \
        if (e_ != cudaSuccess) return MXFP4_CUDA_ERROR;      \
    } while (0)

__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Offset of scale (row, block) in the 128x4 tiled order; nblk4 = ceil(nblk / 4).
__host__ __device__ __forceinline__ size_t scale_offset(int64_t row, int64_t blk, int64_t nblk4)
{
    return (size_t)(((row >> 7) * nblk4 + (blk >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (blk & 3));
}

// ---- scale ------------------------------------------------------------------------------------
// E8M0 byte of a group from the bf16 bit pattern (sign cleared) of its largest magnitude.
//   truncation-free: s = ceil(log2(M/6)) = floor(log2 M) - 2 + [mantissa(M) > 1.5]
//   floor          : s = floor(log2 M) - 2
// M = 0 takes M~ = 1e-8, s = -29 in both; s is clamped to >= -127 (byte 0).  Callers test
// amax_bits >= 0x7F80 (Inf/NaN) first.
template <int SCALE_MODE>
__device__ __forceinline__ uint32_t scale_byte_from_amax(uint32_t amax_bits)
{
    if (amax_bits == 0) return 98u;
    int b = (int)(amax_bits >> 7) - 2;
    if (SCALE_MODE == MXFP4_SCALE_TRUNCATION_FREE) b += ((amax_bits & 0x7Fu) > 0x40u) ? 1 : 0;
    return (uint32_t)max(b, 0);
}

// 2^-s as a float for s = byte - 127; byte <= 253 always holds for finite bf16 inputs.
__device__ __forceinline__ float inv_scale_from_byte(uint32_t byte)
{
    return __uint_as_float((254u - byte) << 23);
}
// 2^s as a float (byte 0 gives the subnormal 2^-127).
__device__ __forceinline__ float scale_from_byte(uint32_t byte)
{
    return byte ? __uint_as_float(byte << 23) : __uint_as_float(0x00400000u);
}

// ---- rounding ---------------------------------------------------------------------------------
// Two latent values -> two E2M1 codes (v0 in the low nibble), round-to-nearest-even, saturating at 6,
// sign bit of the source kept.
__device__ __forceinline__ uint32_t rne_pair(float v0, float v1)
{
#ifndef MX_SOFT_RNE
    uint16_t r;
    asm("{\n\t.reg .b8 b;\n\tcvt.rn.satfinite.e2m1x2.f32 b, %1, %2;\n\tcvt.u16.u8 %0, b;\n\t}" : "=h"(r) : "f"(v1), "f"(v0));
    return (uint32_t)r;
#else
    auto one = [](float v) -> uint32_t {
        float a = fabsf(v);
        uint32_t m = (a > 0.25f) + (a >= 0.75f) + (a > 1.25f) + (a >= 1.75f) + (a > 2.5f) + (a >= 3.5f) + (a > 5.0f);
        return m | ((__float_as_uint(v) >> 28) & 8u);
    };
    return one(v0) | (one(v1) << 4);
#endif
}

// E2M1 code of a float that already lies on the grid (magnitude bits `mb`, sign from `vbits`).
__device__ __forceinline__ uint32_t encode_on_grid(uint32_t mb, uint32_t vbits)
{
    int m = max((int)(mb >> 22) - 252, (int)(mb != 0u));
    return (uint32_t)m | ((vbits >> 28) & 8u);
}

// Stochastic rounding (Sec. 3.2: q2 iff v + xi >= midpoint, xi = D (u - 1/2)  <=>  f + u >= 1) of one
// latent value; `c` holds the element's 16 random bits at bits [21:6] (u = u16 * 2^-16), other bits 0.
// Returns the magnitude code 0..7.
//   |v| >= 1: the grid points are the floats with one mantissa bit, f = low 22 mantissa bits / 2^22,
//             so f + u >= 1 is the carry out of (low22 + u16 * 64).
//   |v| <  1: the grid {0, .5, 1} + 1 is the same kind of grid in [1, 2]; |v| + 1 is taken with
//             round-toward-zero, which keeps floor(f * 2^22) and with it the decision (u16 * 64 is an integer).
// The shift by 22 drops the discarded bits; magnitudes above 6 (floor scaling) saturate.
__device__ __forceinline__ uint32_t sr_mag(float v, uint32_t c)
{
    const float a = fabsf(v);
    const bool lt1 = a < 1.0f;
    const float t = lt1 ? __fadd_rz(a, 1.0f) : a;
    const uint32_t code = ((__float_as_uint(t) + c) >> 22) - (lt1 ? 254u : 252u);
    return min(code, 7u);
}

// ---- Philox4x32-10 ----------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int i = 0; i < 10; i++) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c3 = (uint32_t)p0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The random bits of source elements 8q .. 8q+7: element j uses half (j & 1) of word j >> 1.
__device__ __forceinline__ uint4 sr_words(uint64_t seed, uint32_t stream_id, uint64_t q)
{
    return philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), stream_id, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
}
// 16 random bits moved to bits [21:6]
__device__ __forceinline__ uint32_t sr_c_even(uint32_t w) { return (w << 6) & 0x003FFFC0u; }
__device__ __forceinline__ uint32_t sr_c_odd(uint32_t w) { return (w >> 10) & 0x003FFFC0u; }

// ---- small helpers ------------------------------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// max over the two 15-bit magnitudes packed in each of two words
__device__ __forceinline__ uint32_t absmax2(uint32_t acc, uint32_t w) { return __vmaxu2(acc, w & 0x7FFF7FFFu); }
__device__ __forceinline__ uint32_t hmax_halves(uint32_t acc) { return max(acc & 0xFFFFu, acc >> 16); }

__device__ __forceinline__ uint4 ld_nc_16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

}  // namespace mx
