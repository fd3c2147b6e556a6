// The two passes of the tile quantizer over a 128 x 128 bf16 tile held in shared memory, shared by the streaming
// two-axis quantizer (tiles loaded by TMA) and the quantizing epilogue of the GEMM (tiles written by the epilogue warps).
// Tile layout: two boxes of 128 rows x 64 columns, one after the other, each with the 128B swizzle of a TMA tile
// (the 16-byte piece j of row r sits at piece j ^ (r & 7)).  256 threads take part.
#pragma once
#include "common.cuh"

namespace mx {

constexpr int kTile = 128;
constexpr int kTileBytes = kTile * kTile * 2;   // 32 KB


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


// Per-thread geometry of the two passes (tile-local, the same for every tile).
//   row pass   : warps 0-3 take the left 64 columns, warps 4-7 the right; a lane pair shares a row (its two groups);
//                a thread handles rows r_row0 and r_row0 + 16
//   column pass: a warp takes the 32 rows x 64 columns it had in the row pass, a lane a pair of columns
struct QsGeom {
    int r_half, r_gg, r_row0;
    uint32_t r_off[4];   // the thread's four 16-byte pieces inside its swizzled row
    int c_rg, c_half, c_col;
    uint32_t c_off[8];   // the column pair's word inside rows with (row & 7) = k
};

__device__ __forceinline__ QsGeom qs_geom(int tid)
{
    QsGeom g;
    const int warp = tid >> 5, lane = tid & 31;
    g.r_half = warp >> 2;
    g.r_gg = lane & 1;
    g.r_row0 = (warp & 3) * 32 + (lane >> 1);
#pragma unroll
    for (int j = 0; j < 4; j++) g.r_off[j] = (uint32_t)(g.r_half * (kTileBytes / 2) + (((g.r_gg * 4 + j) ^ (g.r_row0 & 7)) << 4));
    g.c_rg = warp & 3;      // the same 32 rows x 64 columns this warp handled in the row pass: with DQ the column pass
    g.c_half = warp >> 2;   // reads only what its own warp wrote back, and a __syncwarp orders the two
    g.c_col = g.c_half * 64 + 2 * lane;
#pragma unroll
    for (int k = 0; k < 8; k++)
        g.c_off[k] = (uint32_t)(g.c_half * (kTileBytes / 2) + g.c_rg * 32 * 128 + ((((lane >> 2) ^ k) << 4) | ((lane & 3) << 2)));
    return g;
}

// Row pass: each thread quantizes two whole 32-element groups (Eq. 1, groups along the columns), stores their 16 bytes
// of codes straight to global memory and their scale bytes into the tile's 512-byte chunk `s_sc_row` (entries outside
// the matrix 0x7F).  st_base: shared-memory address of the tile; DQ: the exact dequantization P * 2^s of every group
// is written to the same position of the tile at dq_base (which may be st_base): double quantization, Sec. 3.3.
template <bool SR_ROW, bool DQ>
__device__ __forceinline__ void qs_row_pass(const QsGeom &g, uint32_t st_base, uint32_t dq_base, int row0, int col0, int rows, int cols,
                                            const QuantSide &rw, uint32_t tfa_r, uint8_t *s_sc_row, uint32_t &nonfinite)
{
    const int r_half = g.r_half, r_gg = g.r_gg, r_row0 = g.r_row0;
    const uint32_t *r_off = g.r_off;
#pragma unroll
    for (int item = 0; item < 2; item++) {
        const int r = r_row0 + item * 16;
        const uint32_t a0 = st_base + (uint32_t)r * 128u;
        const int gcol = col0 + r_half * 64 + r_gg * 32;
        uint4 q[4];
#pragma unroll
        for (int j = 0; j < 4; j++)
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(q[j].x), "=r"(q[j].y), "=r"(q[j].z), "=r"(q[j].w) : "r"(a0 + r_off[j]));
        uint32_t am4[4];
#pragma unroll
        for (int j = 0; j < 4; j++) am4[j] = absmax_fold(absmax_fold(q[j].x, q[j].y), absmax_fold(q[j].z, q[j].w));
        uint32_t am = hmax_halves(absmax_fold_end(absmax_fold(absmax_fold(am4[0], am4[1]), absmax_fold(am4[2], am4[3]))));
        const bool nf = am >= 0x7F80u;
        const uint32_t byte = nf ? 0xFFu : scale_byte_from_amax(am, tfa_r);
        const uint32_t inv = inv_scale_bf16x2(nf ? 127u : byte);
        uint4 codes;
        if (SR_ROW) {
            const uint64_t q0 = ((uint64_t)(row0 + r) * (uint64_t)cols + (uint64_t)gcol) >> 4;
            const uint4 ra = sr_words(rw.sr, q0), rb = sr_words(rw.sr, q0 + 1);
            codes = make_uint4(sr8(q[0], inv, ra.x, ra.y), sr8(q[1], inv, ra.z, ra.w), sr8(q[2], inv, rb.x, rb.y), sr8(q[3], inv, rb.z, rb.w));
        } else {
            codes = make_uint4(rne8(q[0], inv), rne8(q[1], inv), rne8(q[2], inv), rne8(q[3], inv));
        }
        if (nf) codes = make_uint4(0u, 0u, 0u, 0u);
        if (DQ) {
            // P * 2^s of the 32 codes back into the staged tile (exact in bf16); a non-finite group becomes NaN
            const uint32_t sc2 = nf ? 0x7FC07FC0u : scale_bf16x2(byte);
            const uint32_t cw[4] = {codes.x, codes.y, codes.z, codes.w};
#pragma unroll
            for (int j = 0; j < 4; j++) {
                uint32_t o[4];
                dequant_x8(cw[j], sc2, o);
                asm volatile("st.shared.v4.u32 [%4], {%0,%1,%2,%3};" ::"r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(dq_base + (uint32_t)r * 128u + r_off[j]) : "memory");
            }
        }
        const bool in = row0 + r < rows && gcol < cols;
        nonfinite |= (uint32_t)(nf && in);
        if (in) *reinterpret_cast<uint4 *>(rw.packed + (int64_t)(row0 + r) * (cols >> 1) + (gcol >> 1)) = codes;
        s_sc_row[(r & 31) * 16 + (r >> 5) * 4 + r_half * 2 + r_gg] = in ? (uint8_t)byte : (uint8_t)0x7F;
    }
}

// Column pass: each thread quantizes two adjacent columns x 32 rows, i.e. two whole groups of the transposed output
// (groups of 32 source rows, Sec. 3.3 "Block Format"), writes their codes into the 64B-swizzled staging tile
// `staging` (128 output rows x 64 bytes, for one TMA store) and their scale bytes into the chunk `s_sc_t`.
template <bool SR_T>
__device__ __forceinline__ void qs_col_pass(const QsGeom &g, uint32_t st_base, int row0, int col0, int rows, int cols, const QuantSide &tr,
                                            uint32_t tfa_t2, uint8_t *staging, uint8_t *s_sc_t, uint32_t &nonfinite)
{
    const int c_rg = g.c_rg, c_col = g.c_col;
    const uint32_t *c_off = g.c_off;
    uint32_t v[32];
#pragma unroll
    for (int i = 0; i < 32; i++) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v[i]) : "r"(st_base + c_off[i & 7] + (uint32_t)i * 128u));
    uint32_t am8[8];
#pragma unroll
    for (int k = 0; k < 8; k++) am8[k] = absmax_fold(absmax_fold(v[4 * k], v[4 * k + 1]), absmax_fold(v[4 * k + 2], v[4 * k + 3]));
    const uint32_t am = absmax_fold_end(absmax_fold(absmax_fold(absmax_fold(am8[0], am8[1]), absmax_fold(am8[2], am8[3])),
                                                    absmax_fold(absmax_fold(am8[4], am8[5]), absmax_fold(am8[6], am8[7]))));   // maxima of the two columns, one per half
    const uint32_t b2 = scale_bytes_x2(am, tfa_t2);
    const uint32_t nfm = __vcmpeq2(b2, 0x00FF00FFu);           // 0xFFFF in the half of a non-finite group
    const uint32_t inv2 = (0x00FE00FEu - ((b2 & ~nfm) | (nfm & 0x007F007Fu))) << 7;   // 2^-s of both columns as bf16
#pragma unroll
    for (int i = 0; i < 32; i++) v[i] = mul_bf16x2(v[i], inv2);
    uint32_t lo[4], hi[4];                                     // 32 codes of the first / second column
    if (SR_T) {
        const uint64_t qa = ((uint64_t)(col0 + c_col) * (uint64_t)rows + (uint64_t)(row0 + c_rg * 32)) >> 4;
        const uint64_t qb = qa + (uint64_t)(rows >> 4);
        const uint4 ra[2] = {sr_words(tr.sr, qa), sr_words(tr.sr, qa + 1)};
        const uint4 rb[2] = {sr_words(tr.sr, qb), sr_words(tr.sr, qb + 1)};
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const uint32_t *x = v + 16 * h;
            lo[2 * h] = sr4(bf16lo(x[0]), bf16lo(x[1]), bf16lo(x[2]), bf16lo(x[3]), ra[h].x) | (sr4(bf16lo(x[4]), bf16lo(x[5]), bf16lo(x[6]), bf16lo(x[7]), ra[h].y) << 16);
            lo[2 * h + 1] = sr4(bf16lo(x[8]), bf16lo(x[9]), bf16lo(x[10]), bf16lo(x[11]), ra[h].z) | (sr4(bf16lo(x[12]), bf16lo(x[13]), bf16lo(x[14]), bf16lo(x[15]), ra[h].w) << 16);
            hi[2 * h] = sr4(bf16hi(x[0]), bf16hi(x[1]), bf16hi(x[2]), bf16hi(x[3]), rb[h].x) | (sr4(bf16hi(x[4]), bf16hi(x[5]), bf16hi(x[6]), bf16hi(x[7]), rb[h].y) << 16);
            hi[2 * h + 1] = sr4(bf16hi(x[8]), bf16hi(x[9]), bf16hi(x[10]), bf16hi(x[11]), rb[h].z) | (sr4(bf16hi(x[12]), bf16hi(x[13]), bf16hi(x[14]), bf16hi(x[15]), rb[h].w) << 16);
        }
    } else {
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const uint32_t *x = v + 8 * k;
            lo[k] = rne_x8(bf16lo(x[0]), bf16lo(x[1]), bf16lo(x[2]), bf16lo(x[3]), bf16lo(x[4]), bf16lo(x[5]), bf16lo(x[6]), bf16lo(x[7]));
            hi[k] = rne_x8(bf16hi(x[0]), bf16hi(x[1]), bf16hi(x[2]), bf16hi(x[3]), bf16hi(x[4]), bf16hi(x[5]), bf16hi(x[6]), bf16hi(x[7]));
        }
    }
    if (nfm & 0x0000FFFFu) lo[0] = lo[1] = lo[2] = lo[3] = 0u;
    if (nfm & 0xFFFF0000u) hi[0] = hi[1] = hi[2] = hi[3] = 0u;
    // output rows c_col, c_col + 1 of the transposed tile: 16 bytes at piece c_rg, 64B swizzle (piece ^ ((row >> 1) & 3))
    const uint32_t piece = (uint32_t)((c_rg ^ ((c_col >> 1) & 3)) << 4);
    *reinterpret_cast<uint4 *>(staging + c_col * 64 + piece) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    *reinterpret_cast<uint4 *>(staging + (c_col + 1) * 64 + piece) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    const bool in = col0 + c_col < cols && row0 + c_rg * 32 < rows;     // columns come in blocks of 32: both or neither
    nonfinite |= (uint32_t)(in && nfm != 0u);
    s_sc_t[(c_col & 31) * 16 + (c_col >> 5) * 4 + c_rg] = in ? (uint8_t)(b2 & 0xFFu) : (uint8_t)0x7F;
    s_sc_t[((c_col + 1) & 31) * 16 + (c_col >> 5) * 4 + c_rg] = in ? (uint8_t)(b2 >> 16) : (uint8_t)0x7F;
}

}  // namespace mx
