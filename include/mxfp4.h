/*
 * mxfp4.h — C ABI of the B200 (sm_100a) MXFP4 quantized-linear library.
 *
 * The operations are those of "Oscillation-Reduced MXFP4 Training for Vision Transformers"
 * (arxiv 2502.20853): the MX quantizers of Sec. 3.1-3.2, the quantized linear layer of Sec. 3.3
 * (Eq. 3-5, block format, double quantization), the EMA quantizer of Sec. 5 / Algorithm 1 and
 * the oscillation counters of Sec. 6.1.
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, unless a comment says "host".
 *     Pointers must be 16-byte aligned; leading dimensions are in elements.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*); nothing synchronises and,
 *     except where stated, nothing allocates.
 *   - Return value: MXFP4_OK or an error code; on error nothing has been enqueued.
 *   - `dev_status` (optional, device uint32_t, caller-zeroed): conditions found on the device are
 *     OR-ed into it (MXFP4_DEV_* bits).
 *   - A "packed" matrix [rows, cols] holds two E2M1 codes per byte, element 2j in bits 3:0 of byte j,
 *     row pitch cols/2 bytes.  Its scales are one E8M0 byte (s + 127) per 32 consecutive columns,
 *     stored in the 128x4 tiled order that tcgen05 block-scaled MMA consumes (mxfp4_scale_offset).
 *     The grouped (contraction) axis is always `cols` and must be a multiple of 32.
 */
#ifndef MXFP4_H_
#define MXFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t mxfp4_status_t;
enum {
    MXFP4_OK = 0,
    MXFP4_INVALID_ARG = 1,         /* null pointer, negative size, unknown enum value */
    MXFP4_BAD_SHAPE = 2,           /* grouped axis not a multiple of 32, or shapes that do not match */
    MXFP4_MISALIGNED = 3,          /* pointer not 16-byte aligned, or pitch not a multiple of 16 bytes */
    MXFP4_WORKSPACE_TOO_SMALL = 4,
    MXFP4_UNSUPPORTED_DEVICE = 5,  /* current device is not compute capability 10.x */
    MXFP4_CUDA_ERROR = 6           /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
};

/* bits of *dev_status */
enum {
    MXFP4_DEV_NONFINITE = 1u,      /* an input group held Inf/NaN: its scale byte is 0xFF, codes 0 */
    MXFP4_DEV_TIMEOUT = 2u,        /* a bounded pipeline wait inside the GEMM expired; output invalid */
    MXFP4_DEV_SMEM_LAYOUT = 4u     /* a GEMM kernel that asks for a 1024-byte aligned shared-memory window did not get
                                      one and did nothing; output invalid (not seen on sm_100 with CUDA 12.9) */
};

enum { MXFP4_SCALE_TRUNCATION_FREE = 0,  /* s = ceil(log2(M/6)), Sec. 3.2 (the paper's rule) */
       MXFP4_SCALE_FLOOR = 1 };          /* s = floor(log2 M) - 2, Eq. 2 (Microscaling's rule) */
enum { MXFP4_ROUND_NEAREST = 0,          /* round_D of Sec. 3.2, ties to the even E2M1 code */
       MXFP4_ROUND_STOCHASTIC = 1 };     /* round_S of Sec. 3.2, Philox4x32-10 driven */
enum { MXFP4_OUT_BF16 = 0, MXFP4_OUT_FP32 = 1 };

/* A quantized matrix (device pointers).  `scales` must hold mxfp4_scale_bytes(rows, cols) bytes. */
typedef struct {
    void *data;       /* packed E2M1, rows * cols/2 bytes */
    uint8_t *scales;  /* E8M0 bytes in tiled order */
    int64_t rows, cols;
} mxfp4_mat_t;

/* Quantizer parameters.  Stochastic rounding (Sec. 3.2: q2 iff v + xi >= (q1+q2)/2, xi = D(u - 1/2)):
 * the larger neighbour is chosen iff f + u >= 1 with f = (|v| - lo) / (hi - lo) and u = u16 * 2^-16.
 * u16 of element i (row-major linear index in the quantizer's OUTPUT matrix, so consecutive i run along
 * the group axis): one Philox4x32-10 call (key = seed, counter = (i >> 4, stream_id, 0)) serves 16
 * elements; elements 2m and 2m+1 share the 16-bit field half (m & 1) (0 = low) of word (m & 7) >> 1; the
 * even element takes the field as it is, the odd element takes it with its 16 bits in reverse order. */
typedef struct {
    int32_t scale_mode;
    int32_t rounding;
    uint64_t seed;
    uint32_t stream_id;
    uint32_t reserved;
} mxfp4_qparams_t;

/* Oscillation-counter state of one weight matrix [n, k] (Sec. 6.1), all caller-owned device memory. */
typedef struct {
    void *w_prev;          /* bf16 [n, k]: weight of the previous step (read, then overwritten) */
    mxfp4_mat_t wq_prev;   /* quantized weight of the previous step (read, then overwritten) */
    float *dist_w;         /* [n, k] running sum of |w^t - w^(t-1)| */
    float *dist_q;         /* [n, k] running sum of |wQ^t - wQ^(t-1)| */
} mxfp4_osc_state_t;

/* What the forward pass leaves for the backward pass: the two forward operands (Eq. 3) and, optionally, the
 * backward operands Q6 (Eq. 5; made in the same pass over X) and Q4 (Eq. 4; made ahead from the quantized weight). */
typedef struct {
    mxfp4_mat_t xq;      /* Q1(X)  [M, K], groups along K */
    mxfp4_mat_t wq;      /* Q2(W)  [N, K], groups along K */
    mxfp4_mat_t xq_t;    /* optional (data == NULL: unused): Q6 = stochastic re-quantization of deq(Q1(X)) along M, [K, M] */
    uint64_t xq_t_seed;  /* the seed Q6 is drawn with (stream 6): the seed the backward pass of this step will be given */
    mxfp4_mat_t wq_t;    /* optional (data == NULL: unused): Q4 = stochastic re-quantization of deq(Q2(W)) along N, [K, N].
                          * Either made ahead by the caller with mxfp4_quantize_t(src_q = wq, stochastic, wq_t_seed,
                          * stream 4) (the weight changes once per optimizer step, so this small pass can run beside the
                          * activation quantizer on another stream instead of inside the backward pass), or, when the
                          * forward pass is given the weight itself (w_bf16) and N is a multiple of 32, written by the
                          * forward pass in its one pass over W, with wq_t_seed */
    uint64_t wq_t_seed;  /* the seed wq_t was (or is to be) drawn with */
} mxfp4_linear_ctx_t;

/* ---- host-side layout queries (pure functions) ------------------------------------------- */

/* Bytes of the scale buffer of a packed [rows, cols] matrix: rows padded to 128, 32-column blocks
 * padded to 4, one byte each. */
size_t mxfp4_scale_bytes(int64_t rows, int64_t cols);

/* Byte offset of the scale of (row, block) inside that buffer, block = column / 32:
 * ((row/128) * ceil(nblk/4) + block/4) * 512 + (row%32) * 16 + ((row%128)/32) * 4 + block%4.
 * Padding entries are written as 0x7F (scale 1) by the quantizers. */
size_t mxfp4_scale_offset(int64_t row, int64_t block, int64_t cols);

/* Number of kernels this library has launched in this process so far (all entry points, all streams; counted at the
 * launch sites).  For benchmarks that report how many launches a step takes. */
uint64_t mxfp4_launch_count(void);

/* Scratch bytes mxfp4_gemm needs for an [M, N] output with contraction length kc (0 if none). */
size_t mxfp4_gemm_workspace_bytes(int64_t m, int64_t n, int64_t kc);

/* The longest chain of tensor-core MMAs (64 contraction elements each) that mxfp4_gemm adds into one FP32
 * accumulator for this shape; the product's error bound is stated in terms of it (see mxfp4_gemm).  Split-K and
 * the kernels that alternate between two accumulators shorten it. */
int64_t mxfp4_gemm_chain_mmas(int64_t m, int64_t n, int64_t kc);

/* Scratch bytes mxfp4_linear_bwd needs (backward operands + GEMM scratch). */
size_t mxfp4_linear_workspace_bytes(int64_t m, int64_t k, int64_t n);

/* ---- quantizers --------------------------------------------------------------------------- */

/* Eq. 1 with 1x32 groups along columns (Sec. 3.1-3.2): dst = Q(src), src bf16 [rows, cols] with
 * leading dimension ld.  dst.rows/cols must equal rows/cols.  cols % 32 == 0, ld % 8 == 0. */
mxfp4_status_t mxfp4_quantize(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld,
                              mxfp4_mat_t dst, const mxfp4_qparams_t *qp, uint32_t *dev_status,
                              void *stream);

/* Quantization along the other axis (Sec. 3.3 "Block Format"): groups are 32 consecutive ROWS of the
 * source and the result is stored as the transposed matrix dst_t [cols, rows].
 * Exactly one source is given: src_bf16 (bf16 [rows, cols], ld) or src_q (an MXFP4 matrix
 * [rows, cols] whose exact dequantization is re-quantized: "Double Quantization", Sec. 3.3).
 * rows % 32 == 0, cols % 32 == 0. */
mxfp4_status_t mxfp4_quantize_t(const void *src_bf16, const mxfp4_mat_t *src_q, int64_t rows,
                                int64_t cols, int64_t ld, mxfp4_mat_t dst_t,
                                const mxfp4_qparams_t *qp, uint32_t *dev_status, void *stream);

/* Both layouts from ONE read of a bf16 source (the two gradient operands Q3, Q5 of Eq. 4-5):
 * dst = Q(src; qp_row) [rows, cols] and dst_t = Q(src^T; qp_t) [cols, rows].  Same results as
 * mxfp4_quantize followed by mxfp4_quantize_t.  rows % 32 == 0, cols % 32 == 0. */
mxfp4_status_t mxfp4_quantize_2axis(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld,
                                    mxfp4_mat_t dst, const mxfp4_qparams_t *qp_row,
                                    mxfp4_mat_t dst_t, const mxfp4_qparams_t *qp_t,
                                    uint32_t *dev_status, void *stream);

/* A quantizer and its double quantization (Sec. 3.3) in one pass: dst = Q(src; qp_row) [rows, cols] and
 * dst_t = Q(deq(dst)^T; qp_t) [cols, rows], i.e. the second output re-quantizes the already quantized first output
 * along the other axis.  Same results as mxfp4_quantize followed by mxfp4_quantize_t on its result.  This is how
 * the forward pass makes Q1(X) together with Q6 of Eq. 5.  rows % 32 == 0, cols % 32 == 0. */
mxfp4_status_t mxfp4_quantize_chain(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld, mxfp4_mat_t dst,
                                    const mxfp4_qparams_t *qp_row, mxfp4_mat_t dst_t, const mxfp4_qparams_t *qp_t,
                                    uint32_t *dev_status, void *stream);

/* Q-EMA (Sec. 5, Eq. 10, Algorithm 1) fused with the EMA update and, optionally, the oscillation
 * counters of Sec. 6.1.  w bf16 [n, k] contiguous; ema fp32 [n, k] in/out.
 *   update_ema != 0: ema <- fma(beta, ema, (1-beta)*w) in FP32 first (Eq. 10), then quantize;
 *   the scale of a group comes from the current weights; each element takes whichever of the two
 *   grid neighbours of w/S is nearer to ema/S (ties as round-to-nearest-even).
 *   osc != NULL: dist_w += |w - w_prev|, dist_q += |wQ - wQ_prev| (FP32), then w_prev, wq_prev take
 *   the current values. */
mxfp4_status_t mxfp4_qema_quantize(const void *w_bf16, float *ema, float beta, int32_t update_ema,
                                   int64_t n, int64_t k, mxfp4_mat_t dst, int32_t scale_mode,
                                   const mxfp4_osc_state_t *osc, uint32_t *dev_status, void *stream);

/* Exact dequantization P * 2^s (Sec. 3.1) into fp32 [rows, cols] with leading dimension ld. */
mxfp4_status_t mxfp4_dequantize(mxfp4_mat_t src, float *dst, int64_t ld, void *stream);

/* ---- block-scaled product ----------------------------------------------------------------- */

/* D[M, N] = deq(A)[M, kc] * deq(B)[N, kc]^T (+ bias[N]), FP32 accumulation on the tcgen05 tensor
 * cores (the three products of Eq. 3-5 all have this form).  a.cols == b.cols == kc, kc % 32 == 0.
 * d: bf16 or fp32 [M, N] with leading dimension ldd (bytes per row a multiple of 16).
 * bias_bf16: optional [N].  workspace: >= mxfp4_gemm_workspace_bytes(M, N, kc) bytes (may be NULL
 * when that is 0); used for split-K partial sums when M*N is small and kc long.
 * Accuracy.  The FP4 products are exact; the error is that of the FP32 accumulation.  The tensor core adds
 * each MMA's 64-term sum into its accumulator with truncation, which loses up to one ulp of the running sum
 * per MMA, always in the same direction.  With c = mxfp4_gemm_chain_mmas(M, N, kc) MMAs chained into one
 * accumulator the FP32 result d satisfies, against the exact product D of the dequantized operands,
 *     |d - D| <= max(1, c / 8) * 2^-20 * sum_k |a_k b_k|        per element
 * (a bf16 result is the rounding of such a d).  The ulp that is lost is one of the RUNNING sum: where the
 * terms cancel, as they do in the products of a layer (signed activations, weights and gradients), the
 * running sum is small against sum|a b| and the error stays within 2^-20 * sum|a b| at any length
 * (measured worst 0.5 * 2^-20 at kc = 50432); operands without cancellation and with scales spread over
 * many binades reach 2.4 * 2^-20 at c = 64 and c = 128. */
mxfp4_status_t mxfp4_gemm(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int32_t out_dtype,
                          const void *bias_bf16, void *workspace, size_t workspace_bytes,
                          uint32_t *dev_status, void *stream);

/* The product with the next quantization fused into its epilogue (Sec. 3.3: what one product writes, the next
 * product reads quantized; "Double Quantization" for the operand along the other axis).  Per output tile:
 *     Y  = bf16(deq(A) deq(B)^T + bias)                              the layer's result
 *     Z  = bf16(hook(Y))                                             hook: identity, GELU (0.5 y (1 + erf(y / sqrt 2)),
 *                                                                    in FP32, absolute error below 1e-6 |y|), or
 *                                                                    Y * aux elementwise (exact before the rounding)
 *     Zq   = Q(Z; qp_row)      [M, N], groups along N                (the next product's row operand, e.g. Q1 or Q3)
 *     Zq_t = Q(Z^T; qp_t)      [N, M], groups along M                (its transposed operand, e.g. Q5), or with
 *            chain != 0:  Q(deq(Zq)^T; qp_t)                          (double quantization, e.g. Q6)
 * Zq and Zq_t are bit for bit what mxfp4_quantize_2axis / mxfp4_quantize_chain give on Z (same rounding rules, same
 * random stream by (seed, stream_id, position in the output)).  Every output is optional (data / pointer NULL = not
 * written), at least one must be asked for; chain needs both Zq and Zq_t.  N % 32 == 0; M % 32 == 0 when Zq_t is
 * asked for; y, z, aux: bf16 [M, N], 16-byte aligned, leading dimensions multiples of 8.  No workspace: the
 * contraction is never split (see mxfp4_gemm for the accuracy bound with c = ceil(kc / 64)). */
enum { MXFP4_HOOK_IDENTITY = 0, MXFP4_HOOK_GELU = 1, MXFP4_HOOK_MULTIPLY = 2 };
typedef struct {
    int32_t hook;             /* MXFP4_HOOK_* */
    int32_t chain;            /* != 0: zq_t re-quantizes the dequantized zq instead of Z */
    const void *aux_bf16;     /* MXFP4_HOOK_MULTIPLY: the second factor, e.g. the derivative of the activation */
    int64_t ld_aux;
    void *y_bf16;             /* optional: Y */
    int64_t ldy;
    void *z_bf16;             /* optional: Z */
    int64_t ldz;
    mxfp4_mat_t zq;           /* optional: [M, N] */
    mxfp4_qparams_t qp_row;
    mxfp4_mat_t zq_t;         /* optional: [N, M] */
    mxfp4_qparams_t qp_t;
} mxfp4_epilogue_t;
mxfp4_status_t mxfp4_gemm_quant(mxfp4_mat_t a, mxfp4_mat_t b, const void *bias_bf16, const mxfp4_epilogue_t *epi,
                                uint32_t *dev_status, void *stream);

/* The same product for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a convenience of the library, not a step of the method).
 * Who needs it: code that is handed its tensors by someone else and may not call cudaMalloc or a
 * framework allocator itself -- an extension inside a runtime with a sealed memory pool, a step that
 * runs while allocation is forbidden.  mxfp4_gemm makes such a caller bring split-K scratch; here the
 * scratch is a fixed array of MXFP4_STATIC_SCRATCH_BYTES in the library's own device image.  Each GPU
 * that loads the library carries that array until the process ends.
 *   - Same arguments and results as mxfp4_gemm, without workspace / workspace_bytes.  The function
 *     calls no cudaMalloc, cudaFree or allocating library routine.
 *   - Shapes whose mxfp4_gemm_workspace_bytes(M, N, kc) exceeds MXFP4_STATIC_SCRATCH_BYTES are
 *     refused with MXFP4_WORKSPACE_TOO_SMALL and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (the device must be
 *     current); make that first call before any stream capture begins.
 *   - All calls on one GPU share the one array.  It keeps whatever the previous call left there;
 *     nothing in it needs to start at zero, because every partial sum that is read has been
 *     written by the same call.  Two calls that may overlap on the GPU (different streams) race on
 *     it: serialise them. */
#define MXFP4_STATIC_SCRATCH_BYTES (16u << 20)
mxfp4_status_t mxfp4_gemm_static(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int32_t out_dtype,
                                 const void *bias_bf16, uint32_t *dev_status, void *stream);

/* Measurement aid (the paper has no counterpart): runs, on every SM, `iters` x 4 block-scaled MXFP4 MMAs of
 * 128 x bn x 64 (bn = 128, 192 or 256) on operands that stay in shared memory, with no loads and no epilogue.
 * Timed by the caller (events on `stream`), 8 * 128 * bn * 64 * iters flops per SM give the tensor pipe's issue
 * ceiling on the part at hand, against which the GEMM kernels can be held.  Reads and writes no global memory
 * except *dev_status (optional, as elsewhere). */
mxfp4_status_t mxfp4_mma_issue_ceiling(int32_t bn, int32_t iters, uint32_t *dev_status, void *stream);

/* ---- self-tests of the bounded waits (the paper has no counterpart) ------------------------- */

/* Every wait on a barrier inside the GEMM kernels and the two-axis quantizer is bounded: after a fixed number of
 * polls it gives up, raises MXFP4_DEV_TIMEOUT in *dev_status and sets a flag that makes every other role of the
 * thread block leave its loop; the block then synchronises, frees its tensor memory and returns, so the context
 * stays usable.  In normal use the bound (about 0.3 s) is never reached.  These two calls exercise that path
 * without any fault: they launch the very kernels mxfp4_gemm / mxfp4_quantize_2axis would launch for these
 * arguments, with the operand loads withheld and the bound set to `spin_limit` polls (128 .. 65536), so that the
 * first wait of every block runs out within milliseconds.  Nothing is computed; the outputs (and the workspace)
 * are left undefined; *dev_status (required) has MXFP4_DEV_TIMEOUT set when the kernels have finished.  All waits
 * stay bounded: the calls return like any other and the next call on the stream runs normally. */
mxfp4_status_t mxfp4_gemm_wait_selftest(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int32_t out_dtype,
                                        void *workspace, size_t workspace_bytes, uint32_t spin_limit,
                                        uint32_t *dev_status, void *stream);
mxfp4_status_t mxfp4_quantize_wait_selftest(const void *src_bf16, int64_t rows, int64_t cols, int64_t ld,
                                            mxfp4_mat_t dst, mxfp4_mat_t dst_t, uint32_t spin_limit,
                                            uint32_t *dev_status, void *stream);

/* ---- Q-Ramping (Sec. 6, Algorithm 2) ------------------------------------------------------- */

/* Algorithm 2, OscillationDetection.  For each of `count` weight elements, from the trajectory
 * lengths that mxfp4_qema_quantize's counters (or the caller) accumulated over the detection window
 * (Sec. 6.1):  R_w = dist_q / dist_w,   n_w = min(k2 * floor(R_w / k1) + 1, n_max)   (1 <= n_max <= 255),
 * the factor by which the element's learning rate and gradient-accumulation length are multiplied.
 * Both quotients are single FP32 divisions.  dist_w = 0 gives n_max if dist_q > 0, else 1; a NaN
 * ratio gives 1.  dist_w, dist_q: device, FP32, 16-byte aligned, not modified (the caller zeroes
 * them when a new window starts).  n_w: device, one byte per element, 8-byte aligned.
 * oscillating: optional device counter to which the number of elements with R_w > k1 is ADDED
 * (the "oscillating weights" of Sec. 7.2 for k1 = 16).  Paper defaults: k1 = 16, k2 = 5. */
mxfp4_status_t mxfp4_qramp_detect(const float *dist_w, const float *dist_q, int64_t count, float k1,
                                  int32_t k2, int32_t n_max, uint8_t *n_w,
                                  unsigned long long *oscillating, void *stream);

/* Hyper-parameters of one optimizer step.  bias_corr1 = 1 - beta1^t and bias_corr2 = 1 - beta2^t
 * for the caller's global step count t (t >= 1). */
typedef struct {
    float lr, beta1, beta2, eps, weight_decay, bias_corr1, bias_corr2;
} mxfp4_adamw_t;

/* One step of Algorithm 2's customized AdamW over `count` elements.  The paper fixes LR_w = n_w LR and
 * an accumulation over n_w steps (Sec. 6.2) but prints no update rule; this library's reading, per element:
 *     acc += grad;  cnt += 1;
 *     if cnt >= n_w:  g = acc / cnt;  m = b1 m + (1 - b1) g;  v = b2 v + (1 - b2) g^2;
 *                     w -= n_w lr ((m / bias_corr1) / (sqrt(v / bias_corr2) + eps) + weight_decay w);
 *                     acc = 0;  cnt = 0
 * all in FP32, each operation rounded once.  With n_w == NULL (or all ones) this is AdamW.
 * w, m, v, acc: device FP32 state, updated in place (w, m, v only where a window closed); cnt: device,
 * one byte per element, the steps accumulated so far (start at 0); grad: device FP32, read only (the
 * dW of mxfp4_linear_bwd); w_bf16: optional bf16 copy of w for the quantizers, written where w changed.
 * FP32 arrays 16-byte aligned, byte arrays 4-byte aligned, w_bf16 8-byte aligned. */
mxfp4_status_t mxfp4_qramp_adamw(float *w, void *w_bf16, const float *grad, float *m, float *v,
                                 float *acc, uint8_t *cnt, const uint8_t *n_w, int64_t count,
                                 const mxfp4_adamw_t *hp, void *stream);

/* ---- diagnostics (Sec. 4, Appendix A) ------------------------------------------------------ */

/* Histogram of the quantization confidence (Sec. 4.2, App. A.2) of a weight matrix w bf16 [n, k], k % 32 == 0:
 *     QuantConf(w) = min_i |a - thrd_i| / MaxDist(w_FP4),   a = |w| / 2^s,
 * s the scale of the element's 1x32 group by the rule of Sec. 3.2 (scale_mode as in the quantizers), thrd_i the
 * midpoints of neighbouring E2M1 values, MaxDist half the width of the rounding cell (the cell of 0 reaches to
 * the threshold of the other sign: 0.25; the cell of 6 is [5, 6]: 1; latents beyond 6 count as confidence 1).
 * The count of every element is ADDED to hist[min(floor(conf * bins), bins - 1)]; hist: device, `bins` 64-bit
 * counters (1 <= bins <= 64), 8-byte aligned, zeroed by the caller when a new histogram starts.  Groups that
 * hold Inf or NaN are skipped.  w: device, 16-byte aligned, contiguous. */
mxfp4_status_t mxfp4_quant_conf_hist(const void *w_bf16, int64_t n, int64_t k, int32_t scale_mode, int32_t bins,
                                     unsigned long long *hist, void *stream);

/* One term of the rate of change r(X) of App. A.3, ||X^t - X^(t-1)||_F / ||X^(t-1)||_F: ADDS
 * sum (cur - prev)^2 to out[0] and sum prev^2 to out[1] (device doubles, 8-byte aligned, zeroed by the caller).
 * cur, prev: bf16, `count` elements, device, 16-byte aligned.  Partial sums are FP32 per thread, FP64 across
 * threads; the order of the additions is not fixed. */
mxfp4_status_t mxfp4_change_sums(const void *cur_bf16, const void *prev_bf16, int64_t count, double *out, void *stream);

/* The same for two quantized matrices of one shape (the quantized weights of two steps). */
mxfp4_status_t mxfp4_change_sums_q(mxfp4_mat_t cur, mxfp4_mat_t prev, double *out, void *stream);

/* ---- quantized linear layer (Sec. 3.3) ----------------------------------------------------- */

/* Forward, Eq. 3: Y = Q1(X) Q2(W)^T.  x bf16 [M, K] (ldx), y bf16 [M, N] (ldy).
 * ctx->xq and ctx->wq are caller-allocated; xq is always written.  If w_bf16 != NULL, wq is written
 * as round-to-nearest Q2(W); if w_bf16 == NULL, ctx->wq is taken as already quantized (e.g. by
 * mxfp4_qema_quantize, once per optimizer step).  If ctx->xq_t.data != NULL (needs M % 32 == 0), the same
 * kernel that makes Q1(X) also writes Q6 = Q(deq(Q1(X))^T; stochastic, seed ctx->xq_t_seed, stream 6) into
 * it, which saves the backward pass its second read of Q1(X).
 * The forward pass takes no workspace: its product never splits the contraction (for a small M with a very long
 * K, mxfp4_gemm with a workspace has more parallelism).  All arguments are checked before the first launch. */
mxfp4_status_t mxfp4_linear_fwd(const void *x_bf16, int64_t ldx, int64_t m, int64_t k,
                                const void *w_bf16, int64_t n, const void *bias_bf16, void *y_bf16,
                                int64_t ldy, mxfp4_linear_ctx_t *ctx, int32_t scale_mode,
                                uint32_t *dev_status, void *stream);

/* Backward, Eq. 4-5 with double quantization: dX = Q3(dY) Q4(deq(Wq)^T...) and dW = Q5(dY^T) Q6(deq(Xq)),
 * all four quantizers stochastic with Philox streams 3, 4, 5, 6 of `seed`.
 * dy bf16 [M, N] (lddy); dx bf16 [M, K] (lddx); dw [N, K] (lddw) in dw_dtype (MXFP4_OUT_*).
 * If ctx->xq_t.data != NULL and ctx->xq_t_seed == seed, ctx->xq_t is used as Q6 instead of being recomputed
 * (the result is the same either way); likewise ctx->wq_t with ctx->wq_t_seed == seed is used as Q4.
 * workspace: >= mxfp4_linear_workspace_bytes(M, K, N). */
mxfp4_status_t mxfp4_linear_bwd(const void *dy_bf16, int64_t lddy, const mxfp4_linear_ctx_t *ctx,
                                uint64_t seed, int32_t scale_mode, void *dx_bf16, int64_t lddx,
                                void *dw, int64_t lddw, int32_t dw_dtype, void *workspace,
                                size_t workspace_bytes, uint32_t *dev_status, void *stream);

/* The two passes with the quantizations at a layer boundary moved into the neighbouring product (Sec. 3.3: what one
 * product writes the next one reads quantized), so that a chain of layers skips its stand-alone quantizer passes.
 * mxfp4_linear_fwd_ex: as mxfp4_linear_fwd, and
 *   - x_bf16 == NULL: ctx->xq (and ctx->xq_t, if its data is set) already hold Q1(X) (and Q6), e.g. written by the
 *     previous layer's epilogue;
 *   - epi != NULL: the product runs as mxfp4_gemm_quant with *epi (y_bf16 / ldy are ignored: the epilogue names its
 *     own outputs, typically the next layer's ctx->xq and ctx->xq_t with chain = 1 and the hook between the layers).
 * mxfp4_linear_bwd_ex: as mxfp4_linear_bwd, and
 *   - dy_bf16 == NULL: *dyq = Q3(dY) [M, N] and *dyq_t = Q5(dY^T) [N, M] are given (written by the next layer's
 *     input-gradient epilogue with streams 3 and 5 of this layer's seed);
 *   - epi_dx != NULL: the input-gradient product runs as mxfp4_gemm_quant with *epi_dx (dx_bf16 / lddx are ignored),
 *     typically multiplying by the derivative of the activation and emitting the previous layer's Q3 and Q5. */
mxfp4_status_t mxfp4_linear_fwd_ex(const void *x_bf16, int64_t ldx, int64_t m, int64_t k, const void *w_bf16,
                                   int64_t n, const void *bias_bf16, void *y_bf16, int64_t ldy,
                                   mxfp4_linear_ctx_t *ctx, int32_t scale_mode, const mxfp4_epilogue_t *epi,
                                   uint32_t *dev_status, void *stream);
mxfp4_status_t mxfp4_linear_bwd_ex(const void *dy_bf16, int64_t lddy, const mxfp4_mat_t *dyq,
                                   const mxfp4_mat_t *dyq_t, const mxfp4_linear_ctx_t *ctx, uint64_t seed,
                                   int32_t scale_mode, void *dx_bf16, int64_t lddx, void *dw, int64_t lddw,
                                   int32_t dw_dtype, const mxfp4_epilogue_t *epi_dx, void *workspace,
                                   size_t workspace_bytes, uint32_t *dev_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MXFP4_H_ */
