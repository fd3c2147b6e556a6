// Device-side building blocks of the MXFP4 quantizers (sm_100a).
// Definitions follow Sec. 3.1-3.2 of the paper (E2M1 grid, shared power-of-two scale,
// deterministic and stochastic rounding); Philox4x32-10 is the random source.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/mxfp4.h"

namespace mx {

constexpr int kGroup = 32;

#define MX_CHECK_CUDA(expr)                                  \
    do {                                                     \
        cudaError_t e_ = (expr);                             \
        if (e_ != cudaSuccess) return MXFP4_CUDA_ERROR;      \
    } while (0)

// Kernels this library has launched in this process (mxfp4_launch_count): counted where they are launched.
extern std::atomic<unsigned long long> g_launches;
#define MX_LAUNCHED() (::mx::g_launches.fetch_add(1ull, std::memory_order_relaxed))
// after a <<<...>>> launch: the launch error, if any, and the count
#define MX_CHECK_LAUNCH()                       \
    do {                                        \
        MX_CHECK_CUDA(cudaGetLastError());      \
        MX_LAUNCHED();                          \
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
// M = 0 takes M~ = 1e-8, s = -29 in both; s is clamped to >= -127 (byte 0).  Inf/NaN (amax_bits >=
// 0x7F80) are the caller's business.  tf_add = 63 for truncation-free scaling, 0 for floor scaling:
// (mantissa + 63) >> 7 is 1 exactly when the 7-bit mantissa exceeds 0x40.
__device__ __forceinline__ uint32_t scale_byte_from_amax(uint32_t amax_bits, uint32_t tf_add)
{
    const int b = (int)(amax_bits >> 7) - 2 + (int)(((amax_bits & 0x7Fu) + tf_add) >> 7);
    return amax_bits ? (uint32_t)max(b, 0) : 98u;
}
__device__ __forceinline__ uint32_t tf_add_of(int scale_mode) { return scale_mode == MXFP4_SCALE_FLOOR ? 0u : 63u; }

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

// Eight latent values -> eight codes in one word (v0 in the lowest nibble), round-to-nearest-even, saturating.
__device__ __forceinline__ uint32_t rne_x8(float v0, float v1, float v2, float v3, float v4, float v5, float v6, float v7)
{
#ifndef MX_SOFT_RNE
    uint32_t r;
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
        : "=r"(r) : "f"(v0), "f"(v1), "f"(v2), "f"(v3), "f"(v4), "f"(v5), "f"(v6), "f"(v7));
    return r;
#else
    return rne_pair(v0, v1) | (rne_pair(v2, v3) << 8) | (rne_pair(v4, v5) << 16) | (rne_pair(v6, v7) << 24);
#endif
}

// ---- packed bf16 arithmetic ---------------------------------------------------------------------
// Product of two bf16 pairs.  One factor is always a power of two here, so the product is exact unless it falls
// below the normal range, where it is far too small to round to anything but (signed) zero on the E2M1 grid.
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// 2^-s in both halves for s = byte - 127 (byte <= 253)
__device__ __forceinline__ uint32_t inv_scale_bf16x2(uint32_t byte) { return ((254u - byte) << 7) * 0x00010001u; }
// 2^s in both halves (byte 0 gives the subnormal 2^-127)
__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t byte) { return (byte ? (byte << 7) : 0x0040u) * 0x00010001u; }

// Eight E2M1 codes (one word, code 0 in the lowest nibble) times the bf16 pair `sc2` (the same power of two in both
// halves, or NaN) -> eight bf16 values in four words.  Exact: the products have at most two significant bits.
__device__ __forceinline__ void dequant_x8(uint32_t codes, uint32_t sc2, uint32_t (&o)[4])
{
    uint32_t h[4];
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\tmov.b32 {b0, b1, b2, b3}, %4;\n\t"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n\tcvt.rn.f16x2.e2m1x2 %1, b1;\n\tcvt.rn.f16x2.e2m1x2 %2, b2;\n\tcvt.rn.f16x2.e2m1x2 %3, b3;\n\t}"
        : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]) : "r"(codes));
#pragma unroll
    for (int j = 0; j < 4; j++) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h[j]));
        uint32_t b;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(b) : "f"(f.y), "f"(f.x));
        o[j] = mul_bf16x2(b, sc2);
    }
}

// Stochastic rounding (Sec. 3.2: q2 iff v + xi >= midpoint, xi = D (u - 1/2)  <=>  f + u >= 1, f the
// fraction of the way from the lower to the upper grid neighbour, u = u16 * 2^-16) of four consecutive
// latent values with the sm_100a stochastic-rounding convert.  `w` is the random word of these four
// elements: its low half is the 16-bit draw of the pair (v0, v1), its high half that of (v2, v3); within a
// pair the second element reads the draw with its bit order reversed.  The result has the code of v0 in
// its low nibble.  Magnitudes above 6 saturate; the sign of the source is kept, also on zero.
// The convert adds the 16 random bits below the last kept bit and truncates, which is exactly f + u >= 1.
// It expects the draw of the first pair in bytes 2 (high) and 0 (low) of its operand and that of the second
// pair in bytes 3 and 1, hence the byte permutation.
__device__ __forceinline__ uint32_t sr4(float v0, float v1, float v2, float v3, uint32_t w)
{
    uint32_t rb;
    asm("prmt.b32 %0, %1, %1, 0x3120;" : "=r"(rb) : "r"(w));
    uint16_t d;
    asm("cvt.rs.satfinite.e2m1x4.f32 %0, {%1, %2, %3, %4}, %5;" : "=h"(d) : "f"(v3), "f"(v2), "f"(v1), "f"(v0), "r"(rb));
    return (uint32_t)d;
}

// ---- Philox4x32-10 ----------------------------------------------------------------------------
// The ten round keys of one seed are computed on the host and travel as kernel parameters, so that
// each round reads its key straight from the constant bank.
struct SrStream {
    uint32_t k[20];      // k[2i] = seed_lo + i * 0x9E3779B9, k[2i+1] = seed_hi + i * 0xBB67AE85
    uint32_t stream_id;  // third counter word
    uint32_t pad;
};

inline SrStream make_sr_stream(uint64_t seed, uint32_t stream_id)
{
    SrStream s;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int i = 0; i < 10; i++) {
        s.k[2 * i] = k0;
        s.k[2 * i + 1] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    s.stream_id = stream_id;
    s.pad = 0;
    return s;
}

// The random words of elements 16q .. 16q+15 of a quantizer's output (counter = (q, stream_id, 0)):
// elements 4k .. 4k+3 use word k (see sr4).
__device__ __forceinline__ uint4 sr_words(const SrStream &s, uint64_t q)
{
    uint32_t c0 = (uint32_t)q, c1 = (uint32_t)(q >> 32), c2 = s.stream_id, c3 = 0u;
#pragma unroll
    for (int i = 0; i < 10; i++) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ s.k[2 * i];
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ s.k[2 * i + 1];
        c3 = (uint32_t)p0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// ---- small helpers ------------------------------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Running maximum of the magnitudes of packed bf16 pairs, as bit patterns: |.| and max are taken by the
// half-precision unit; a NaN operand gives the canonical NaN 0x7FFF, which compares as "not finite" like Inf (0x7F80).
__device__ __forceinline__ uint32_t absmax2(uint32_t acc, uint32_t w)
{
    uint32_t d;
    asm("{\n\t.reg .b32 t;\n\tabs.bf16x2 t, %2;\n\tmax.NaN.bf16x2 %0, %1, t;\n\t}" : "=r"(d) : "r"(acc), "r"(w));
    return d;
}
__device__ __forceinline__ uint32_t hmax_halves(uint32_t acc) { return max(acc & 0xFFFFu, acc >> 16); }

// The same running maximum in one instruction per word: max.xorsign.abs takes the larger magnitude of each half and
// gives it the product of the two signs, so the magnitudes accumulate and the sign bits are noise to be masked off at
// the end (absmax_fold_end).  NaN propagates as the canonical 0x7FFF.
__device__ __forceinline__ uint32_t absmax_fold(uint32_t acc, uint32_t w)
{
    uint32_t d;
    asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(acc), "r"(w));
    return d;
}
__device__ __forceinline__ uint32_t absmax_fold_end(uint32_t acc) { return acc & 0x7FFF7FFFu; }

__device__ __forceinline__ uint4 ld_nc_16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

}  // namespace mx
