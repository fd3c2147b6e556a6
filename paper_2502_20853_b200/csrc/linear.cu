// The MXFP4 linear layer (Sec. 3.3): Eq. 3 forward, Eq. 4-5 backward with double quantization.
// Pure composition of the quantizer and GEMM launches on the caller's stream.
#include "common.cuh"

namespace mx {
mxfp4_status_t quantize_rows(const void *src, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                             const mxfp4_qparams_t *qp, uint32_t *dev_status, cudaStream_t st);
mxfp4_status_t quantize_tile(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows, int64_t cols, int64_t ld,
                             const mxfp4_mat_t *dst, const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t,
                             const mxfp4_qparams_t *qp_t, uint32_t *dev_status, cudaStream_t st, bool chain);
mxfp4_status_t gemm(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int out_dtype, const void *bias, void *workspace,
                    size_t workspace_bytes, uint32_t *dev_status, cudaStream_t st, bool allow_split);
mxfp4_status_t gemm_check(mxfp4_mat_t a, mxfp4_mat_t b, const void *d, int64_t ldd, int out_dtype, const void *bias,
                          const void *workspace, size_t workspace_bytes, bool allow_split);
size_t gemm_workspace_bytes(int64_t m, int64_t n, int64_t kc);
mxfp4_status_t gemm_quant_check(mxfp4_mat_t a, mxfp4_mat_t b, const void *bias, const mxfp4_epilogue_t *epi);
mxfp4_status_t gemm_quant(mxfp4_mat_t a, mxfp4_mat_t b, const void *bias, const mxfp4_epilogue_t *epi, uint32_t *dev_status, cudaStream_t st);

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct BwdLayout {
    size_t dyq_p, dyq_s, dyqt_p, dyqt_s, wqt_p, wqt_s, xqt_p, xqt_s, gemm_ws, gemm_ws_bytes, total;
};

static BwdLayout bwd_layout(int64_t m, int64_t k, int64_t n)
{
    BwdLayout L;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
    L.dyq_p = take((size_t)m * n / 2);
    L.dyq_s = take(mxfp4_scale_bytes(m, n));
    L.dyqt_p = take((size_t)n * m / 2);
    L.dyqt_s = take(mxfp4_scale_bytes(n, m));
    L.wqt_p = take((size_t)k * n / 2);
    L.wqt_s = take(mxfp4_scale_bytes(k, n));
    L.xqt_p = take((size_t)k * m / 2);
    L.xqt_s = take(mxfp4_scale_bytes(k, m));
    const size_t g1 = gemm_workspace_bytes(m, k, n), g2 = gemm_workspace_bytes(n, k, m);
    L.gemm_ws_bytes = g1 > g2 ? g1 : g2;
    L.gemm_ws = take(L.gemm_ws_bytes);
    L.total = o;
    return L;
}

}  // namespace mx

using namespace mx;

extern "C" {

size_t mxfp4_linear_workspace_bytes(int64_t m, int64_t k, int64_t n)
{
    if (m <= 0 || k <= 0 || n <= 0) return 0;
    return bwd_layout(m, k, n).total;
}

mxfp4_status_t mxfp4_linear_fwd_ex(const void *x_bf16, int64_t ldx, int64_t m, int64_t k, const void *w_bf16, int64_t n,
                                   const void *bias_bf16, void *y_bf16, int64_t ldy, mxfp4_linear_ctx_t *ctx, int32_t scale_mode,
                                   const mxfp4_epilogue_t *epi, uint32_t *dev_status, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ctx || (!epi && !y_bf16)) return MXFP4_INVALID_ARG;
    if (ctx->xq.rows != m || ctx->xq.cols != k || ctx->wq.rows != n || ctx->wq.cols != k) return MXFP4_BAD_SHAPE;
    mxfp4_qparams_t qp = {scale_mode, MXFP4_ROUND_NEAREST, 0, 0, 0};
    mxfp4_status_t s;
    // The forward product takes no workspace, so it never splits the contraction; its arguments are checked before the
    // quantizers are enqueued, so that an error leaves the stream untouched.
    if (epi) {
        if ((s = gemm_quant_check(ctx->xq, ctx->wq, bias_bf16, epi))) return s;
    } else if ((s = gemm_check(ctx->xq, ctx->wq, y_bf16, ldy, MXFP4_OUT_BF16, bias_bf16, nullptr, 0, false))) {
        return s;
    }
    if (x_bf16) {
        if (k % 32 != 0 || ldx < k) return MXFP4_BAD_SHAPE;
        if ((reinterpret_cast<uintptr_t>(x_bf16) & 15u) || ldx % 8 != 0) return MXFP4_MISALIGNED;
        if (ctx->xq_t.data && (m % 32 != 0 || ctx->xq_t.rows != k || ctx->xq_t.cols != m)) return MXFP4_BAD_SHAPE;
        if (ctx->xq_t.data && (!ctx->xq_t.scales || ((reinterpret_cast<uintptr_t>(ctx->xq_t.data) | reinterpret_cast<uintptr_t>(ctx->xq_t.scales)) & 15u)))
            return ctx->xq_t.scales ? MXFP4_MISALIGNED : MXFP4_INVALID_ARG;
    }
    if (reinterpret_cast<uintptr_t>(w_bf16) & 15u) return MXFP4_MISALIGNED;
    // with the weight itself and a buffer for Q4 in the context, Q4 is made here too (one pass over W makes Q2 and Q4)
    const bool make_q4 = w_bf16 && ctx->wq_t.data && n % 32 == 0;
    if (make_q4) {
        if (ctx->wq_t.rows != k || ctx->wq_t.cols != n) return MXFP4_BAD_SHAPE;
        if (!ctx->wq_t.scales) return MXFP4_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(ctx->wq_t.data) | reinterpret_cast<uintptr_t>(ctx->wq_t.scales)) & 15u) return MXFP4_MISALIGNED;
    }
    if (x_bf16 && ctx->xq_t.data) {
        // Q1 and, from its dequantized result, Q6 (stream 6 of the seed the backward pass will use) in one pass over X
        const mxfp4_qparams_t q6 = {scale_mode, MXFP4_ROUND_STOCHASTIC, ctx->xq_t_seed, 6, 0};
        s = quantize_tile(x_bf16, nullptr, m, k, ldx, &ctx->xq, &qp, ctx->xq_t, &q6, dev_status, st, true);
        if (s) return s;
    } else if (x_bf16) {
        s = quantize_rows(x_bf16, m, k, ldx, ctx->xq, &qp, dev_status, st);  // Q1
        if (s) return s;
    }
    if (make_q4) {
        // Q2 and, from its dequantized result, Q4 (stream 4 of the seed the backward pass will use)
        const mxfp4_qparams_t q4 = {scale_mode, MXFP4_ROUND_STOCHASTIC, ctx->wq_t_seed, 4, 0};
        s = quantize_tile(w_bf16, nullptr, n, k, k, &ctx->wq, &qp, ctx->wq_t, &q4, dev_status, st, true);
        if (s) return s;
    } else if (w_bf16) {
        s = quantize_rows(w_bf16, n, k, k, ctx->wq, &qp, dev_status, st);  // Q2
        if (s) return s;
    }
    if (epi) return gemm_quant(ctx->xq, ctx->wq, bias_bf16, epi, dev_status, st);
    return gemm(ctx->xq, ctx->wq, y_bf16, ldy, MXFP4_OUT_BF16, bias_bf16, nullptr, 0, dev_status, st, false);
}

mxfp4_status_t mxfp4_linear_fwd(const void *x_bf16, int64_t ldx, int64_t m, int64_t k, const void *w_bf16, int64_t n,
                                const void *bias_bf16, void *y_bf16, int64_t ldy, mxfp4_linear_ctx_t *ctx,
                                int32_t scale_mode, uint32_t *dev_status, void *stream)
{
    if (!x_bf16 || !y_bf16) return MXFP4_INVALID_ARG;
    return mxfp4_linear_fwd_ex(x_bf16, ldx, m, k, w_bf16, n, bias_bf16, y_bf16, ldy, ctx, scale_mode, nullptr, dev_status, stream);
}

mxfp4_status_t mxfp4_linear_bwd_ex(const void *dy_bf16, int64_t lddy, const mxfp4_mat_t *dyq_in, const mxfp4_mat_t *dyq_t_in,
                                   const mxfp4_linear_ctx_t *ctx, uint64_t seed, int32_t scale_mode, void *dx_bf16, int64_t lddx,
                                   void *dw, int64_t lddw, int32_t dw_dtype, const mxfp4_epilogue_t *epi_dx, void *workspace,
                                   size_t workspace_bytes, uint32_t *dev_status, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ctx || !dw || !workspace || (!epi_dx && !dx_bf16)) return MXFP4_INVALID_ARG;
    if (!dy_bf16 && (!dyq_in || !dyq_t_in)) return MXFP4_INVALID_ARG;
    const int64_t m = ctx->xq.rows, k = ctx->xq.cols, n = ctx->wq.rows;
    if (ctx->wq.cols != k) return MXFP4_BAD_SHAPE;
    if (m % 32 != 0 || n % 32 != 0 || k % 32 != 0) return MXFP4_BAD_SHAPE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MXFP4_MISALIGNED;
    const BwdLayout L = bwd_layout(m, k, n);
    if (workspace_bytes < L.total) return MXFP4_WORKSPACE_TOO_SMALL;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    mxfp4_mat_t dyq = {ws + L.dyq_p, ws + L.dyq_s, m, n};
    mxfp4_mat_t dyq_t = {ws + L.dyqt_p, ws + L.dyqt_s, n, m};
    if (!dy_bf16) {
        // Q3(dY) and Q5(dY^T) come from the caller (the next layer's input-gradient product wrote them in its epilogue)
        if (dyq_in->rows != m || dyq_in->cols != n || dyq_t_in->rows != n || dyq_t_in->cols != m) return MXFP4_BAD_SHAPE;
        dyq = *dyq_in;
        dyq_t = *dyq_t_in;
    }
    mxfp4_mat_t wq_t = {ws + L.wqt_p, ws + L.wqt_s, k, n};
    mxfp4_mat_t xq_t = {ws + L.xqt_p, ws + L.xqt_s, k, m};
    const mxfp4_qparams_t q3 = {scale_mode, MXFP4_ROUND_STOCHASTIC, seed, 3, 0};
    const mxfp4_qparams_t q4 = {scale_mode, MXFP4_ROUND_STOCHASTIC, seed, 4, 0};
    const mxfp4_qparams_t q5 = {scale_mode, MXFP4_ROUND_STOCHASTIC, seed, 5, 0};
    const mxfp4_qparams_t q6 = {scale_mode, MXFP4_ROUND_STOCHASTIC, seed, 6, 0};
    mxfp4_status_t s;
    // both products are checked before anything is enqueued (the operands' buffers exist already; only their contents are to come)
    {
        const bool have4 = ctx->wq_t.data && ctx->wq_t_seed == seed, have6 = ctx->xq_t.data && ctx->xq_t_seed == seed;
        if (have4 && (ctx->wq_t.rows != k || ctx->wq_t.cols != n)) return MXFP4_BAD_SHAPE;
        if (have6 && (ctx->xq_t.rows != k || ctx->xq_t.cols != m)) return MXFP4_BAD_SHAPE;
        if (dy_bf16) {
            if (lddy < n || lddy % 8 != 0) return lddy < n ? MXFP4_BAD_SHAPE : MXFP4_MISALIGNED;
            if (reinterpret_cast<uintptr_t>(dy_bf16) & 15u) return MXFP4_MISALIGNED;
        }
        const mxfp4_mat_t b4 = have4 ? ctx->wq_t : wq_t;
        const mxfp4_mat_t b6 = have6 ? ctx->xq_t : xq_t;
        if (epi_dx) {
            if ((s = gemm_quant_check(dyq, b4, nullptr, epi_dx))) return s;
        } else if ((s = gemm_check(dyq, b4, dx_bf16, lddx, MXFP4_OUT_BF16, nullptr, ws + L.gemm_ws, L.gemm_ws_bytes, true))) {
            return s;
        }
        if ((s = gemm_check(dyq_t, b6, dw, lddw, dw_dtype, nullptr, ws + L.gemm_ws, L.gemm_ws_bytes, true))) return s;
    }
    // Q3 and Q5 from one read of dY
    if (dy_bf16 && (s = quantize_tile(dy_bf16, nullptr, m, n, lddy, &dyq, &q3, dyq_t, &q5, dev_status, st, false))) return s;
    // Q4: re-quantize Q2(W) along N;  Q6: re-quantize Q1(X) along M  (double quantization)
    if (ctx->wq_t.data && ctx->wq_t_seed == seed) {
        wq_t = ctx->wq_t;   // made ahead by the caller with this seed
    } else if ((s = quantize_tile(nullptr, &ctx->wq, n, k, k, nullptr, nullptr, wq_t, &q4, dev_status, st, false))) {
        return s;
    }
    if (ctx->xq_t.data && ctx->xq_t_seed == seed) {
        xq_t = ctx->xq_t;   // already made by the forward pass with this seed
    } else if ((s = quantize_tile(nullptr, &ctx->xq, m, k, k, nullptr, nullptr, xq_t, &q6, dev_status, st, false))) {
        return s;
    }
    // Eq. 5: dW[N,K] = dYq_t[N,M] * Xq_t[K,M]^T ;  Eq. 4: dX[M,K] = dYq[M,N] * Wq_t[K,N]^T.
    // dW first: its output is small, so the tail of Q3(dY) that the quantizer left in L2 is still there when dX reads it
    // (both products take the freshest part of their first operand first: the last K tiles, the last rows).
    if ((s = gemm(dyq_t, xq_t, dw, lddw, dw_dtype, nullptr, ws + L.gemm_ws, L.gemm_ws_bytes, dev_status, st, true))) return s;
    if (epi_dx) return gemm_quant(dyq, wq_t, nullptr, epi_dx, dev_status, st);
    return gemm(dyq, wq_t, dx_bf16, lddx, MXFP4_OUT_BF16, nullptr, ws + L.gemm_ws, L.gemm_ws_bytes, dev_status, st, true);
}

mxfp4_status_t mxfp4_linear_bwd(const void *dy_bf16, int64_t lddy, const mxfp4_linear_ctx_t *ctx, uint64_t seed,
                                int32_t scale_mode, void *dx_bf16, int64_t lddx, void *dw, int64_t lddw, int32_t dw_dtype,
                                void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream)
{
    if (!dy_bf16 || !dx_bf16) return MXFP4_INVALID_ARG;
    return mxfp4_linear_bwd_ex(dy_bf16, lddy, nullptr, nullptr, ctx, seed, scale_mode, dx_bf16, lddx, dw, lddw, dw_dtype, nullptr, workspace,
                               workspace_bytes, dev_status, stream);
}

}  // extern "C"
