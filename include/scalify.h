/*
 * scalify.h - C ABI of the B200 (sm_100a) scaled-array kernels.
 *
 * The operations are the scaled primitives of "Scalify: scale propagation for
 * efficient low-precision LLM training" (arxiv 2407.17353).  A ScaledArray is
 * a pair (data, scale) whose value is data * scale (Section 2).  Here `data`
 * is a device buffer in a low-precision format and `scale` is ONE fp32 power
 * of two kept in DEVICE memory (Section 2: E8M0 scale simulated in float32;
 * Section 3.1: scalar scale per tensor).  Every scale this library writes is a
 * power of two obtained by rounding DOWN (Section 3.2, last paragraph).
 *
 * General contract
 *   - All `scalify_array.data`, `.scale`, workspace, statistic, mean/rinv
 *     pointers are DEVICE pointers owned by the caller.  The library
 *     allocates no device memory and frees nothing.  Descriptor structs and
 *     the arrays of descriptors passed to the Adam call are HOST memory and
 *     are read before the call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls only enqueue work; they never synchronise, except
 *     scalify_check_status.
 *   - A NULL `scale` pointer on an INPUT means "unscaled array", scale 1
 *     (Section 3.1, get_data_and_scale).  A NULL `scale` on an OUTPUT means
 *     the propagated scale is not stored.
 *   - Input scale words must be finite positive powers of two within
 *     [2^-126, 2^126]; a violation detected on the device sets
 *     SCALIFY_DEV_BAD_SCALE in the workspace status word where a workspace
 *     is available.
 *   - Layout: row-major, `shape[0..ndim-1]` outermost first, `stride[]` in
 *     elements, innermost stride 1, data pointer 16-byte aligned and every
 *     outer stride a multiple of 16 bytes.
 *   - An output scale word must not alias an input scale word of the same
 *     call unless a function says otherwise (SCALIFY_ERR_ALIAS).
 *   - Return value: 0 on success, a negative scalify_error otherwise.  A call
 *     that fails validation enqueues nothing.  No call aborts, throws, or
 *     traps on the device; every device-side wait is bounded and reports
 *     SCALIFY_DEV_TIMEOUT in the status word when it expires.
 *   - Rounding: data are converted round-to-nearest-even; FP8 conversions
 *     saturate to the largest finite value; subnormals are kept.
 */
#ifndef SCALIFY_H_
#define SCALIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SCALIFY_E4M3 = 0, /* OCP FP8 E4M3 (finite only, max 448)  - forward operands (Section 1, Appendix A) */
  SCALIFY_E5M2 = 1, /* OCP FP8 E5M2 (max 57344)             - backward gradients (Section 1, Appendix A) */
  SCALIFY_F16 = 2,  /* IEEE binary16 */
  SCALIFY_BF16 = 3, /* bfloat16 */
  SCALIFY_F32 = 4   /* IEEE binary32 */
} scalify_dtype;

typedef enum {
  SCALIFY_STAT_NONE = 0,
  SCALIFY_STAT_AMAX = 1, /* max |data| */
  SCALIFY_STAT_L2 = 2    /* sqrt(mean(data^2)), the "L2 moment" of Section 3.3 */
} scalify_stat;

typedef enum {
  SCALIFY_OK = 0,
  SCALIFY_ERR_NULL = -1,        /* a required pointer is NULL */
  SCALIFY_ERR_DTYPE = -2,       /* dtype not valid for this argument */
  SCALIFY_ERR_SHAPE = -3,       /* shapes inconsistent or out of range */
  SCALIFY_ERR_ALIGNMENT = -4,   /* pointer or stride not 16-byte aligned, innermost stride not 1 */
  SCALIFY_ERR_WORKSPACE = -5,   /* workspace missing or too small */
  SCALIFY_ERR_UNSUPPORTED = -6, /* valid but not implemented combination */
  SCALIFY_ERR_CUDA = -7,        /* a CUDA runtime/driver call failed (see scalify_last_cuda_error) */
  SCALIFY_ERR_ALIAS = -8,       /* forbidden aliasing of scale words or buffers */
  SCALIFY_ERR_VALUE = -9        /* scalar argument out of range */
} scalify_error;

/* Bits of the device status word (first 4 bytes of any workspace). */
enum {
  SCALIFY_DEV_TIMEOUT = 1u,        /* a bounded device-side wait expired; results of that call are invalid */
  SCALIFY_DEV_BAD_SCALE = 2u,      /* an input scale word was not a finite positive power of two */
  SCALIFY_DEV_NONFINITE_STAT = 4u, /* a statistic was NaN or Inf; the rescale used factor 1 */
  SCALIFY_DEV_BAD_INDEX = 8u       /* a token id or target was out of range (treated as 0) */
};

typedef struct scalify_array {
  void* data;        /* device pointer, 16-byte aligned */
  int32_t dtype;     /* scalify_dtype */
  int32_t ndim;      /* 1..4 (4: only the attention calls, [batch, heads, T, hd]) */
  int64_t shape[4];  /* outermost first; unused entries ignored */
  int64_t stride[4]; /* in elements; stride[ndim-1] must be 1 */
  float* scale;      /* device pointer to one fp32 power of two, or NULL */
} scalify_array;

/* Operation codes for scalify_workspace_bytes. */
enum {
  SCALIFY_OP_MATMUL = 0,        /* d0 = batch*M, d1 = N */
  SCALIFY_OP_RESCALE = 1,       /* d0 = number of elements, d1 unused */
  SCALIFY_OP_LAYERNORM_BWD = 2, /* d0 = rows, d1 = row length */
  SCALIFY_OP_ADAM = 3,          /* d0 = number of tensors, d1 unused */
  SCALIFY_OP_STATISTIC = 4,     /* d0 = number of elements */
  SCALIFY_OP_CROSS_ENTROPY = 5, /* d0 = number of rows */
  SCALIFY_OP_COLSUM = 6,        /* d0 = rows, d1 = columns */
  SCALIFY_OP_MATMUL_SPLITK = 7  /* d0 = M, d1 = N: room for the partial products of a split contraction */
};

/* Bytes of workspace the given call needs (an upper bound; always >= 4096).
 * The first 256 bytes of a workspace form a header (status word, statistic
 * word, reduction tickets); scalify_workspace_init must have zeroed it once
 * before first use.  One workspace may serve successive calls on one stream;
 * two calls that may overlap on the GPU need separate workspaces.
 * For SCALIFY_OP_RESCALE and SCALIFY_OP_STATISTIC the figure grows with d0
 * (one fp64 partial per block of the statistic pass, at most 512 KiB); those
 * two calls also accept any smaller workspace of at least 4096 bytes and
 * then run the statistic pass with fewer, longer blocks (same result for
 * AMAX; for L2 the fp64 partial sums are combined in a different grouping). */
size_t scalify_workspace_bytes(int op, int64_t d0, int64_t d1);

/* Zero the workspace header (asynchronously, on `stream`). */
int scalify_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Synchronise `stream`, read and clear the status word of `workspace`.
 * Returns the SCALIFY_DEV_* bits (>= 0) or a negative scalify_error. */
int scalify_check_status(void* workspace, void* stream);

const char* scalify_status_string(int code);
/* The cudaError_t value recorded by the last call that returned SCALIFY_ERR_CUDA (per host thread). */
int scalify_last_cuda_error(void);
int scalify_version(void);

/*
 * Scaled matrix multiply (Section 3.2, the matmul rule of Algorithm 3; the
 * mixed-format FP8 operands and higher-precision output of Appendix A).
 *
 *   Y_s = A_s * B_s * kf(K),   Y_d = (op(A)_d . op(B)_d) / kf(K)
 *
 * with kf(K) = sqrt(K) rounded down to a power of two: under the paper's
 * assumption of independent unit-variance operands the contraction has
 * variance K, so dividing the data by kf(K) restores unit scale, and the
 * output scale depends only on the operand scales and the shape.
 *
 *   A : FP8 (E4M3 or E5M2), [M,K] (or [K,M] when transA != 0), ndim 2, or
 *       ndim 3 with a leading batch dimension.
 *   B : FP8 (E4M3 or E5M2, may differ from A), [K,N] (or [N,K] when transB).
 *       A 2-D B with a 3-D A is shared by all batches.
 *   Y : BF16, F16 or F32, [M,N] (or [batch,M,N]); receives the fp32
 *       accumulator times 1/kf(K), rounded once.  Y->scale receives Y_s.
 *   stat: statistic of the STORED Y data gathered in the epilogue (Section
 *       3.3).  SCALIFY_STAT_NONE: none.  Otherwise the statistic is left, as
 *       one fp32, at byte offset 16 of the workspace.
 *   Yq: optional (may be NULL; requires stat != NONE).  Receives the dynamic
 *       rescale of Y: r = statistic rounded down to a power of two,
 *       Yq_d = cast(Y_d / r), Yq_s = Y_s * r.  Any dtype; same shape as Y.
 *
 * Predicted rescale (Section 3.3: statistic and rebalancing are separate
 * primitives).  With stat = AMAX, a BF16/F16 Y, an FP8 Yq of its own and rows
 * of a multiple of 16 elements, the GEMM's epilogue already writes Yq with
 * the power of two of the statistic this workspace saw last (fp32 word at
 * byte offset 56 of the workspace), and the launch that follows rebuilds Yq
 * from Y only if this call's statistic has another power of two.  Y, Yq, both
 * scale words and the statistic word are the same bits either way and for any
 * content of that word; the call leaves its own statistic there.  Keep one
 * workspace per matmul of a training step for the prediction to hold.
 *
 * Y == NULL (FP8 output only): allowed with stat = AMAX and an FP8, contiguous
 * Yq with its own scale word and rows of a multiple of 16 elements.  The
 * values are still rounded to BF16 first and the statistic is still that of
 * the BF16 values, so Yq, Yq_s and the statistic word equal those of the call
 * with a BF16 Y bit for bit, but the intermediate is not stored: the epilogue
 * writes Yq with the predicted power of two, and a second launch of the same
 * kernel, whose thread blocks return at once when the prediction held,
 * computes the product again otherwise.  Never splits the contraction.
 *
 * Accumulation is fp32 on the tensor cores (tcgen05, kind::f8f6f4).  Row
 * strides must be multiples of 16 bytes.  Errors: see scalify_error.
  *
 * Split contraction: when the output has few tiles and K >= 2048 (a weight
 * gradient), and the workspace is at least scalify_workspace_bytes(
 * SCALIFY_OP_MATMUL_SPLITK, M, N), the K range is cut into up to 16 parts that
 * run as one batched launch writing fp32 partial products into the workspace; a
 * second launch adds them in a fixed order, rounds once and takes the statistic.
 * With the smaller SCALIFY_OP_MATMUL workspace the call never splits.  Results
 * of the two forms agree within the accumulation bar, not bit for bit.
 */
int scalify_scaled_matmul(const scalify_array* A, int transA, const scalify_array* B, int transB,
                          scalify_array* Y, int stat, scalify_array* Yq,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same product with a bias vector added in the kernel's epilogue (a linear
 * layer): the add rule applied to the product and the bias, rounded ONCE:
 *   Y_s = max(A_s B_s kf(K), bias_s)
 *   Y_d = (A_d B_d) / kf(K) * (A_s B_s kf(K) / Y_s)  +  bias_d[j] * (bias_s / Y_s)
 * (both factors are exact powers of two).  bias: [N], F16, BF16 or F32, contiguous.
 * Y may be F16, BF16, F32 or, as a static cast of the sum, E4M3 / E5M2.  stat, Yq,
 * workspace as for scalify_scaled_matmul; the contraction is never split.  The
 * unfused sequence (matmul, then scalify_scaled_add with the bias) rounds twice;
 * this call is its value with one rounding.
 * Errors: as scalify_scaled_matmul; NULL (no bias), DTYPE (bias not wide), SHAPE.
 */
int scalify_scaled_matmul_bias(const scalify_array* A, int transA, const scalify_array* B, int transB,
                               const scalify_array* bias, scalify_array* Y, int stat, scalify_array* Yq,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * scalify_scaled_matmul with stat = AMAX and a rebalanced FP8 output, made cheaper by a PREDICTION of the
 * statistic (Section 3.3 observes that statistics change slowly, which is what delayed rescaling exploits;
 * here the result stays that of the exact dynamic rescale).  *stat_hint (DEVICE) holds a predicted
 * statistic, typically the one this call produced last step.  The GEMM writes the 16-bit intermediate Y
 * and, in the same epilogue, Yq = fp8(stored Y / r_pred) with r_pred = the hint rounded down to a power of
 * two (1 if the hint cannot define a scale).  A second, small launch compares r_pred with the power of two
 * of the TRUE statistic of Y: if they agree (the common case) Yq is already the exact result and only its
 * scale word is written; if not, Yq is rebuilt from Y as scalify_scaled_matmul would.  Either way Y, Yq,
 * both scale words and the statistic word are bit-identical to scalify_scaled_matmul(..., AMAX, Yq), and
 * *stat_hint is overwritten with this call's statistic.  In the common case the separate pass over Y
 * (2 bytes read + 1 written per element) is replaced by 1 extra written byte per element in the GEMM.
 *   Y: F16 or BF16, contiguous; Yq: E4M3 or E5M2, contiguous, same shape; other arguments and errors as
 *   scalify_scaled_matmul; SCALIFY_ERR_NULL if stat_hint or Yq is NULL.
 */
int scalify_scaled_matmul_speculative(const scalify_array* A, int transA, const scalify_array* B, int transB,
                                      scalify_array* Y, scalify_array* Yq, float* stat_hint, void* workspace,
                                      size_t workspace_bytes, void* stream);

/*
 * Scaled matrix multiply with DELAYED rescaling (Section 3.3: "Delayed rescaling can be
 * similarly implemented by decoupling the compute of statistics and rebalancing ..., keeping
 * track of the first one in the model state").  One kernel, no intermediate, no second pass:
 *
 *   r   = *stat_in rounded down to a power of two (1 if *stat_in is zero, below 2^-126 or
 *         non-finite): the statistic of an EARLIER step, kept by the caller on the device;
 *   Y_d = cast((op(A)_d . op(B)_d) / kf(K) / r),   Y_s = A_s * B_s * kf(K) * r;
 *   *stat_out (and workspace offset 16) = statistic `stat` of THIS step's un-rebalanced fp32
 *         values (op(A)_d . op(B)_d)/kf(K), for the next step.
 *
 * Y may be FP8 (E4M3 / E5M2) as well as BF16 / F16 / F32.  stat_out may be NULL, and may be the
 * same word as stat_in (it is written after the kernel has finished).  stat = SCALIFY_STAT_NONE
 * gathers nothing (stat_out must then be NULL).  Other arguments as scalify_scaled_matmul.
 */
int scalify_scaled_matmul_delayed(const scalify_array* A, int transA, const scalify_array* B, int transB,
                                  const float* stat_in, scalify_array* Y, int stat, float* stat_out,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Statistic of the data component of X (Section 3.3: "L2 moment (or any other
 * statistic)"), written as one fp32 to `out_stat` (device) and to byte offset
 * 16 of the workspace.  X may be any dtype, contiguous.
 */
int scalify_statistic(const scalify_array* X, int stat, float* out_stat,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Rescaling family (Sections 3.1 and 3.3; Algorithm 4).  Y has the same shape
 * as X, any dtype; both contiguous.  Y may alias X (same buffer) only when the
 * two dtypes have the same size.
 *
 *   stat == AMAX or L2, new_scale == NULL, stat_in == NULL:
 *       dynamic_rescale: s = statistic(X_d); r = s rounded down to a power of
 *       two (r = 1 when s is zero, non-finite or below 2^-126);
 *       Y_d = cast(X_d / r); Y_s = X_s * r.  Needs a workspace.
 *   stat == AMAX or L2, stat_in != NULL (device fp32):
 *       delayed rescale: as above with s read from *stat_in instead of being
 *       computed (Section 3.3: statistic gathered elsewhere, kept in state).
 *   stat == NONE, new_scale != NULL (device fp32):
 *       set_scaling: s' = *new_scale rounded down to a power of two;
 *       Y_d = cast(X_d * X_s / s'); Y_s = s'.  With X->scale == NULL this is
 *       as_scaled_array of an unscaled input.  Y->scale must not alias X->scale.
 *   stat == NONE, new_scale == NULL:
 *       plain cast (cast_on_forward / cast_on_backward of Appendix A):
 *       Y_d = cast(X_d); Y_s = X_s.
 *
 * Y->scale may alias X->scale for the dynamic and delayed forms (in-place
 * rebalance of a state tensor).
 *
 * The dynamic form with an output buffer of its own reads X once when the power
 * of two can be predicted: while the statistic is gathered, Y is already written
 * with the power of two of the statistic this workspace saw last (fp32 word at
 * byte offset 56 of the workspace, any content), and X is read a second time
 * only if this call's statistic has another power of two.  Y, Y_s and the
 * statistic word do not depend on that word; the call leaves its statistic there.
 */
int scalify_rescale(const scalify_array* X, int stat, const float* new_scale, const float* stat_in,
                    scalify_array* Y, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Scaled add / subtract (Section 3.2, the add rule of Algorithm 3):
 *   Y_s = sqrt(A_s^2 + B_s^2) rounded down to a power of two (= max(A_s,B_s)),
 *   Y_d = cast(A_d*(A_s/Y_s) +- B_d*(B_s/Y_s)).
 * A: [M,N] (or any contiguous shape); B: same shape as A, or a vector [N]
 * broadcast over the rows of A (bias).  A and B: F16, BF16 or F32, same
 * dtype; Y any dtype.  Y may alias A's buffer when sizes match.
 */
int scalify_scaled_add(const scalify_array* A, const scalify_array* B, int subtract,
                       scalify_array* Y, void* stream);

/*
 * Scaled LayerNorm forward (Section 3.2.1 and Appendix C.2): the data
 * component is normalised and the result carries scale 1, whatever X_s is:
 *   n = (x_d - mean) / (sqrt(var) + eps)        (eps_inside_sqrt == 0, as printed)
 *   n = (x_d - mean) / sqrt(var + eps)          (eps_inside_sqrt != 0, textbook)
 * followed by the affine part through the ordinary mul and add rules:
 *   Y_s = max(gamma_s, beta_s),  Y_d = cast(n*gamma_d*(gamma_s/Y_s) + beta_d*(beta_s/Y_s)).
 * X: [R,d] F16/BF16/F32, d*elem_size a multiple of 16 bytes, d <= 16384.
 * gamma, beta: [d], same dtype as each other (F16/BF16/F32), or both NULL
 * (then Y_d = n, Y_s = 1).  Y: [R,d], any dtype.  mean, rinv: optional device
 * fp32 [R] outputs (row mean and 1/(sigma+eps) or 1/sqrt(var+eps)), needed by
 * the backward call.
 */
int scalify_scaled_layernorm(const scalify_array* X, const scalify_array* gamma, const scalify_array* beta,
                             float eps, int eps_inside_sqrt, scalify_array* Y,
                             float* mean, float* rinv, void* stream);

/*
 * Scaled LayerNorm backward with dynamic rescale of the input gradient
 * (Section 4 and Algorithm 5: one dynamic rescale per residual branch, placed
 * on the gradient that leaves the LayerNorm).
 *   ghat = G_d*gamma_d;  dx = LayerNorm'(ghat; x_d)  (exact derivative of the
 *   forward above);  dX_s = G_s*gamma_s / X_s;
 *   dgamma_d = sum_rows(G_d*n)/kf(R), dbeta_d = sum_rows(G_d)/kf(R), both with
 *   scale G_s*kf(R) (reduction over R rows treated like a contraction of size R).
 * G, X: [R,d], F16/BF16/F32 (same dtype); mean, rinv: from the forward call.
 * dX: [R,d] BF16/F16/F32: the un-rebalanced gradient (always written).
 * stat_dx: statistic of the stored dX data, left at workspace offset 16.
 * dXq: optional rescaled gradient (any dtype), as Yq of the matmul.
 * dgamma, dbeta: optional [d] outputs, F32/BF16/F16 (both or neither).
 *
 * dX == NULL (one pass, the un-rebalanced gradient is not stored): allowed with
 * stat_dx != NONE and a contiguous FP8 dXq.  The values are still rounded to
 * the dtype of X first and the statistic is still that of those rounded values,
 * so dXq, dXq_s, the statistic word, dgamma and dbeta equal those of the call
 * with a dX of X's dtype bit for bit; the gradient is written with the power
 * of two of the statistic this workspace saw last (fp32 word at byte offset 56
 * of the workspace, any content) and a second launch of the same kernel, whose
 * thread blocks return at once when that prediction held, writes it again
 * otherwise.  The call leaves its own statistic in that word: keep one
 * workspace per LayerNorm of a training step for the prediction to hold.
 * (Section 3.3: statistic and rebalancing are separate primitives.)
 */
int scalify_scaled_layernorm_bwd(const scalify_array* G, const scalify_array* X, const scalify_array* gamma,
                                 const float* mean, const float* rinv, float eps, int eps_inside_sqrt,
                                 int stat_dx, scalify_array* dX, scalify_array* dXq,
                                 scalify_array* dgamma, scalify_array* dbeta,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same backward pass with DELAYED rescaling of the input gradient (Section
 * 3.3: statistic and rebalancing decoupled, the statistic of an earlier step
 * kept in the caller's state), in ONE pass over G and X:
 *   r = the power of two at or below *stat_in (1 if *stat_in is zero,
 *   subnormal, Inf or NaN);  dX_d = cast(dx / r), rounded once from fp32;
 *   dX_s = G_s*gamma_s / X_s * r.
 * dX: [R,d] of ANY dtype (E5M2 for the gradient operand of the next matmul).
 * stat_dx (AMAX or L2; NONE: nothing gathered) is taken on this step's
 * un-rebalanced, unrounded dx and left at workspace offset 16 for the next
 * step; stat_in (device, fp32, not NULL) may be that same word.  Everything
 * else as scalify_scaled_layernorm_bwd.
 */
int scalify_scaled_layernorm_bwd_delayed(const scalify_array* G, const scalify_array* X, const scalify_array* gamma,
                                         const float* mean, const float* rinv, float eps, int eps_inside_sqrt,
                                         const float* stat_in, int stat_dx, scalify_array* dX,
                                         scalify_array* dgamma, scalify_array* dbeta,
                                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * Scaled GELU forward / backward (Section 3.2.1 and Appendix C.1):
 *   forward  (X_d * g(X_d*X_s), X_s);   backward  dX_d = G_d * f'(X_d*X_s), dX_s = G_s.
 * exact_erf == 0: tanh form; != 0: Gaussian-CDF form.  X, G: F16/BF16/F32
 * (same dtype), Y/dX any dtype, contiguous, same shape.
 */
int scalify_scaled_gelu(const scalify_array* X, int exact_erf, scalify_array* Y, void* stream);
int scalify_scaled_gelu_bwd(const scalify_array* G, const scalify_array* X, int exact_erf,
                            scalify_array* dX, void* stream);

/*
 * Diagnostic for the bounded device-side waits (no counterpart in the paper).  Enqueues a one-thread
 * kernel that waits, with the same routine and status path as the matmul pipeline, on a barrier that
 * nothing signals; after `limit_us` microseconds (1..1e6) the wait gives up, sets
 * SCALIFY_DEV_TIMEOUT in the workspace status word and the kernel ends normally.  `waited_us`
 * (optional device word) receives the time actually spent.  Nothing faults and the context stays
 * usable: this is how a lost copy or a lost MMA completion would surface.
 */
int scalify_debug_expire_wait(void* workspace, size_t workspace_bytes, uint32_t limit_us, uint32_t* waited_us,
                              void* stream);

/*
 * Diagnostic (no counterpart in the paper): y[i] = x[i] rounded to the nearest BF16 value (ties to even), as
 * fp32, computed by the routine the fused attention kernels use for the scores' BF16 intermediate (three fp32
 * operations instead of a conversion).  x, y: device fp32 arrays of n elements.  two_wide = 0: the scalar
 * form; 1: the form on two-wide fp32 instructions, which takes the elements in pairs (x[0], x[1]), ...
 * Lets a test compare both with the definition over any set of bit patterns.
 */
int scalify_debug_bf16_round(const float* x, float* y, int64_t n, int two_wide, void* stream);

/*
 * Diagnostics of the library's host-side state (no counterpart in the paper; host only, no GPU needed).
 * The library keeps two things between calls: the one-time set-up of each kernel PER DEVICE (dynamic
 * shared-memory limit, co-resident cluster count) and a cache of encoded TMA tensor maps keyed by pointer,
 * extents, strides and box.  scalify_debug_host_state_selftest drives both with made-up device numbers and a
 * stand-in encoder and returns 0 if each device was set up exactly once and the cache returned the right map
 * for every key; scalify_debug_tensor_map_cache reports how many encodes the real cache has saved (hits) and
 * made (misses) so far in this process.
 */
int scalify_debug_host_state_selftest(void);

/*
 * Bounds-checking build (no counterpart in the paper).  The library built with -DSCALIFY_DEBUG
 * (`libscalify_debug.so`) checks every global access of its memory-bound kernels that goes through their vector,
 * row-copy and scalar-tail helpers (the element-wise, LayerNorm, Adam, block-scale quantisation and support
 * kernels, and the split-K reduction; the tensor-core kernels move their tiles with TMA, which the hardware
 * bounds by the tensor map) against the byte spans of the arrays and workspaces its entry points have validated
 * so far.  An access outside all of them is counted, its address kept, and skipped (a load yields zeros), so
 * nothing faults.  Registration copies a table to the device synchronously: this build is for tests, not for
 * timing or stream capture.  Spans that touch are merged, and spans are never forgotten until reset.
 *
 * scalify_debug_bounds_report: synchronises the device; out[0] = accesses refused since the last report, out[1]
 * = address of the first, out[2] = its width in bytes; clears the counters.  reset_ranges != 0 also forgets every
 * registered span.  range_limit >= 0 caps the length of every span registered from now on (a self-test: accesses
 * past the cap, still inside the caller's buffers, are then refused and reported); -1 lifts the cap.
 * Returns SCALIFY_ERR_UNSUPPORTED in the ordinary build.
 */
int scalify_debug_bounds_report(uint64_t out[3], int reset_ranges, int64_t range_limit);
int scalify_debug_tensor_map_cache(uint64_t* hits, uint64_t* misses);

/*
 * Diagnostic (no counterpart in the paper): the launch shape the LayerNorm kernels would use for an
 * [R,d] input of dtype x_dtype on the current device, so that a test can state which code path it
 * exercised.  Host only, launches nothing.  plan[0] = thread blocks; plan[1] = rows every team of
 * warps walks one after another (forward: consecutive rows of its block's run; backward: the
 * persistent grid's stride loop); plan[2] = warps per row; plan[3] = rows kept in flight through
 * shared memory (0: the backward kernel prefetches one row in registers instead).
 */
int scalify_debug_layernorm_plan(int64_t R, int64_t d, int x_dtype, int backward, int32_t plan[4]);

/*
 * Multiply a ScaledArray by a scalar constant c that is a positive power of two (Section 3.4: a
 * broadcast scalar contributes the scale "c rounded down to a power of two" and its mantissa stays
 * in the data; for a power of two the mantissa is 1, so only the scale word changes: X_s *= c).
 * Other constants return SCALIFY_ERR_UNSUPPORTED.  Used for the 1/sqrt(head_dim) of attention.
 */
int scalify_scalar_mul_pow2(scalify_array* X, float c, void* stream);

/*
 * Support operations of a GPT-style training step.  The paper states no scale rule for these
 * (Section 3.2.1 only says that custom rules suit attention layers); the rules below are this
 * library's readings, chosen so that values follow the unscaled network exactly (model invariance,
 * Section 1) and bounded quantities carry scale 1 (as the gate of an activation, Appendix C.1).
 *
 * Embedding lookup through the add rule:  Y[i] = wte[ids[i]] + wpe[i mod seq_len],
 *   Y_s = max(wte_s, wpe_s).  ids: DEVICE int64 [n]; wte [vocab,d], wpe [>=seq_len,d] or NULL, same
 *   16/32-bit dtype; Y [n,d] any dtype; d*elem_size a multiple of 16 bytes.  An id outside
 *   [0,vocab) sets SCALIFY_DEV_BAD_INDEX in *status (optional device word) and reads row 0.
 * Backward: dwte[v] = sum of the rows of dY whose id is v, scale dY_s (the number of addends is data
 *   dependent, so no static factor; fp32 atomics, order not fixed); dwpe[p] = sum over the
 *   n/seq_len sequences divided by kf(n/seq_len), scale dY_s*kf(n/seq_len).  dwte [vocab,d] and
 *   dwpe [seq_len,d] (or NULL) are F32 and fully overwritten.
 */
int scalify_scaled_embedding(const int64_t* ids, int64_t n, int64_t seq_len, const scalify_array* wte,
                             const scalify_array* wpe, scalify_array* Y, uint32_t* status, void* stream);
int scalify_scaled_embedding_bwd(const int64_t* ids, int64_t n, int64_t seq_len, const scalify_array* dY,
                                 scalify_array* dwte, scalify_array* dwpe, void* stream);

/*
 * Row softmax of the VALUES S_d*S_s over the last dimension, optionally causal (row i of each
 * [Tq,Tk] matrix attends to columns j <= i + Tk - Tq; requires Tk >= Tq); P_d in [0,1], P_s = 1,
 * masked entries exactly 0.  S: [Tq,Tk] or [batch,Tq,Tk], F16/BF16/F32, contiguous, Tk*elem_size a
 * multiple of 16 bytes and at most 4096 bytes; P: same shape, any dtype.
 * Backward: dS_d = P_d*(dP_d - sum_j dP_d[j] P_d[j]), dS_s = dP_s*P_s (the Jacobian is bounded by 1,
 * so the gradient scale passes through).  dP: F16/BF16/F32; P: E4M3/F16/BF16/F32; dS any dtype.
 */
int scalify_scaled_softmax(const scalify_array* S, int causal, scalify_array* P, void* stream);
int scalify_scaled_softmax_bwd(const scalify_array* dP, const scalify_array* P, scalify_array* dS, void* stream);

/*
 * Mean cross-entropy of the values z = logits_d*logits_s through logsumexp (Appendix B) over the
 * first n_classes columns of logits [n, ld>=n_classes] (padding columns ignored), and its gradient
 * w.r.t. the values: dlogits_d = (softmax(z) - onehot(target)) * rem, dlogits_s = 1/n rounded down
 * to a power of two, rem = (1/n)/dlogits_s in [1,2); padding columns receive 0.
 * logits: F16/BF16/F32 (row stride = shape[1]); targets: DEVICE int64 [n]; loss: DEVICE fp32;
 * dlogits: same shape as logits, any dtype, or NULL.  A target outside [0,n_classes) sets
 * SCALIFY_DEV_BAD_INDEX in the workspace status word.  Workspace: SCALIFY_OP_CROSS_ENTROPY, n.
 */
int scalify_scaled_cross_entropy(const scalify_array* logits, int64_t n_classes, const int64_t* targets, float* loss,
                                 scalify_array* dlogits, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Scaled Adam step over a list of tensors (Sections 1, 3 and 4; Table 3 row 4:
 * FP8 gradients, FP16 scaled optimizer state and master weights).  In value
 * space this is textbook Adam with bias correction:
 *   m' = b1*m + (1-b1)*g;  v' = b2*v + (1-b2)*g^2;
 *   w' = w - lr * (m'/(1-b1^t)) / (sqrt(v'/(1-b2^t)) + eps)
 * and the new scales follow from tracing that expression with the static
 * rules (mul: product; add: max; div: ratio; sqrt: sqrt rounded down; a scalar
 * constant c carries the scale "|c| rounded down to a power of two",
 * Section 3.4):
 *   m'_s = max(p2(b1)*m_s, p2(1-b1)*g_s)
 *   v'_s = max(p2(b2)*v_s, p2(1-b2)*g_s^2)
 *   u_s  = p2(lr) * (m'_s/p2(1-b1^t)) / max(p2(sqrt(v'_s/p2(1-b2^t))), p2(eps))
 *   w'_s = max(w_s, u_s)
 * Each of m', v', w' is rounded once from fp32 arithmetic.
 *   grads[i]: any dtype (E5M2 typical); m[i], v[i]: F16 or F32 (same);
 *   w[i]: F16, BF16 or F32.  All four have the same element count, are
 *   contiguous, and m, v, w (data and scale words) are updated in place.
 *   Every m, v and w scale word of the whole list must be a word of its own
 *   (the kernels read the old scales while the new ones are written) and none
 *   of them a gradient's scale word; gradients may share one.  A repeated word
 *   returns SCALIFY_ERR_ALIAS and enqueues nothing.
 *   step >= 1 is t.  Needs a workspace (SCALIFY_OP_ADAM, n_tensors).
 */
int scalify_scaled_adam_step(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v,
                             scalify_array* w, float lr, float beta1, float beta2, float eps, int64_t step,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same step, which also writes the low-precision compute copy of every
 * updated weight that the next forward pass multiplies with (the static cast
 * on the forward path, Appendix A; Section 4: FP8 matmul operands, wider master
 * weights): w_cast[i]_d = cast(stored w'[i]_d), w_cast[i]_s = w'[i]_s.  The
 * cast starts from the value as stored in w[i] (already rounded to its dtype),
 * so the copy is bit-identical to a separate scalify_rescale(STAT_NONE) of
 * w[i], at one extra written byte per parameter instead of a 3-byte pass.
 *   w_cast[i]: E4M3, E5M2, F16 or BF16 (all the same, narrower than w[i]),
 *   contiguous, same element count as w[i], own scale word (no aliasing with
 *   g, m, v, w scale words; data must not alias w[i]).
 * Errors as scalify_scaled_adam_step; SCALIFY_ERR_NULL when w_cast is NULL.
 */
int scalify_scaled_adam_step_cast(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v,
                                  scalify_array* w, scalify_array* w_cast, float lr, float beta1, float beta2,
                                  float eps, int64_t step, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Block scales (Section 2: the scale component may be any array that broadcasts
 * against the data; the paper names the E8M0 exponent byte and the OCP
 * micro-scaling formats as the standard it follows, and works with one scalar
 * scale per tensor; this is the block form of the same representation).
 *
 * A block-scaled array is FP8 data [rows, K] (row-major, dense, K innermost),
 * one E8M0 exponent per 32 consecutive elements of a row, and the usual
 * tensor-wide fp32 power-of-two scale:
 *   value[i,k] = data[i,k] * 2^(exponent[i, k/32] - 127) * scale.
 * Only the tensor-wide scale takes part in the static scale rules; the
 * exponents belong to the data component.
 * K must be a multiple of 128.  `sf` holds the exponents in the order the
 * block-scaled tensor-core instruction consumes: tiles of 128 rows x 4 blocks
 * (512 bytes), tile (r, k) at byte ((r * (K/128)) + k) * 512, and inside a tile
 * row `row`, block `blk` at byte (row % 32) * 16 + (row / 32) * 4 + blk.  The
 * row count is padded up to a multiple of 256: scalify_mx_sf_bytes(rows, K)
 * bytes, 16-byte aligned; the exponents of the padding rows must be valid
 * (scalify_mx_quantize writes 127 there).  All pointers are DEVICE pointers
 * owned by the caller.
 */
typedef struct scalify_mx_array {
  void* data;     /* FP8 elements [rows, K], 16-byte aligned */
  int32_t dtype;  /* SCALIFY_E4M3 or SCALIFY_E5M2 */
  int64_t rows;
  int64_t K;
  uint8_t* sf;    /* E8M0 exponents, tiled as described above */
  float* scale;   /* one fp32 power of two, or NULL (scale 1) */
  int32_t transposed; /* 0: data [rows, K].  1: data stored [K, rows] (row-major, `rows` contiguous, rows a
                         multiple of 16): the form of an operand whose contraction dimension is the slow one
                         of the forward tensor (weight and activation gradients); a block is then 32
                         consecutive ROWS of the storage at one column.  The exponent tiles are the same. */
} scalify_mx_array;

size_t scalify_mx_sf_bytes(int64_t rows, int64_t K);

/*
 * Quantises the data component of X [rows, K] (F16, BF16 or F32; row stride
 * stride[0]) into Y: per block of 32 elements, exponent e = floor(log2(max|x|))
 * - emax (emax = 8 for E4M3, 15 for E5M2: the OCP MX rule, i.e. a dynamic
 * rescale with the AMAX statistic per block, Section 3.3, the power of two
 * rounded down), clamped to [-127, 127]; data = round-to-nearest-even of
 * x * 2^-e, saturating.  A block whose maximum is zero, infinite or NaN gets
 * e = 0.  Y_s = X_s.  `status`: optional DEVICE word that receives
 * SCALIFY_DEV_BAD_SCALE.  Errors: NULL, DTYPE, SHAPE (K % 128), ALIGNMENT.
 * With Y->transposed, X is [K, rows] like the data it is quantised into, and
 * the blocks run down the columns; the values and exponents are those of the
 * plain form applied to the transposed matrix.
 */
int scalify_mx_quantize(const scalify_array* X, scalify_mx_array* Y, uint32_t* status, void* stream);

/*
 * Block-scaled matmul with the static matmul rule (Section 3.2) on the
 * tensor-wide scales:  Y_s = A_s * B_s * kf(K),
 *   Y_d[i,j] = (sum_k A_d[i,k] 2^(Ea[i,k/32]-127) * B_d[j,k] 2^(Eb[j,k/32]-127)) / kf(K)
 * with fp32 accumulation on the tensor cores (tcgen05 kind::mxf8f6f4 with the
 * exponents in tensor memory).  A is [M,K], B is [N,K] (either may be stored
 * transposed, see scalify_mx_array: the tensor cores then read it MN-major and
 * no transposed copy is made); Y [M,N] is F16, BF16
 * or F32 (row stride stride[0]).  stat: NONE, AMAX or L2 of the stored Y, left
 * in the workspace's statistic word as by scalify_scaled_matmul.  Workspace:
 * SCALIFY_OP_MATMUL (M, N).
 */
int scalify_mx_matmul(const scalify_mx_array* A, const scalify_mx_array* B, scalify_array* Y, int stat,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Column sums of a scaled matrix: Y[j] = sum over the R rows of X[r, j], by the
 * rule for a sum of R independent terms (Section 3.2; the same rule as a matmul
 * with a ones operand and K = R, and as the dbeta of the LayerNorm backward):
 *   Y_s = X_s kf(R),   Y_d[j] = (sum_r X_d[r, j]) / kf(R)
 * This is the bias gradient of a linear layer.  X: any dtype, [R, N] (row stride
 * stride[0]); Y: F16, BF16 or F32, [N] contiguous.  Partial sums are fp32 per slab
 * of rows, the slabs are added in fp64 in a fixed order (results do not depend on
 * scheduling).  Workspace: SCALIFY_OP_COLSUM (R, N).
 * Errors: NULL, DTYPE, SHAPE, ALIGNMENT, WORKSPACE, ALIAS.
 */
int scalify_scaled_colsum(const scalify_array* X, scalify_array* Y, void* workspace, size_t workspace_bytes,
                          void* stream);

/*
 * The static cast of a gradient to FP8 (Appendix A: cast_on_backward) fused with the column sums of the cast
 * values: C = cast(X) with C_s = X_s, and Y = the column sums of C by the rule above, in one pass over X.  C, its
 * scale and Y are the bits scalify_rescale (plain cast) followed by scalify_scaled_colsum of its output give.
 * This is what the backward of a linear layer needs of the output gradient: its E5M2 copy for the two gradient
 * matmuls and the bias gradient.  X: BF16 or F16 [R, N]; C: E4M3 or E5M2 [R, N] (row stride a multiple of 16
 * bytes); Y: F16, BF16 or F32 [N].  Workspace: SCALIFY_OP_COLSUM (R, N).
 * Errors: NULL, DTYPE, SHAPE, ALIGNMENT, WORKSPACE, ALIAS.
 */
int scalify_scaled_cast_colsum(const scalify_array* X, scalify_array* C, scalify_array* Y, void* workspace,
                               size_t workspace_bytes, void* stream);

/*
 * Fused scaled attention forward: S = Q K^T, P = softmax(S c), O = P V in one
 * kernel per (head, 128 queries); the scores and the probabilities stay on chip.
 * The paper names attention as a place for a custom scale rule (Section 3.2.1)
 * and gives none; the rule here is the composition of the calls it replaces:
 *   S_s = Q_s K_s kf(hd),  S_d = (Q_d K_d^T) / kf(hd) rounded to BF16      (matmul rule)
 *   P   = softmax over the keys of the VALUES S_d S_s c, optionally causal
 *         (query i sees keys j <= i + Tk - Tq); bounded in [0,1], scale 1, rounded to E4M3
 *   O_s = V_s kf(Tk),      O_d = (P_d V_d) / kf(Tk)                          (matmul rule)
 * i.e. scalify_scaled_matmul, scalify_scalar_mul_pow2, scalify_scaled_softmax,
 * scalify_scaled_matmul.  The softmax is the exact two-sweep form (row maximum
 * and sum first, then the normalised probabilities), not an online rescaling.
 *   Q [heads, Tq, hd], K, V [heads, Tk, hd]: E4M3 or E5M2, hd = 64 or 128, 3-D views
 *   (row and head strides in stride[1], stride[0]; 2-D arrays are one head; 4-D
 *   arrays [batch, heads, T, hd] add a batch stride in front, so that the token-major
 *   buffers [batch * T, heads * hd] of a transformer are covered by ONE call);
 *   O [heads, Tq, hd]: F16, BF16 or F32, same kind of view; c: any finite
 *   scalar (a power of two only shifts the exponent; otherwise its mantissa is
 *   applied in fp32).  causal needs Tk >= Tq.
 *   S_dump (BF16) and P_dump (E4M3): optional dense [heads, Tq, Tk] DEVICE
 *   copies of S_d and P for checking (Tk % 32 == 0), normally NULL; with 4-D
 *   operands the leading dimension counts batch * heads (or is given as two).
 *   status: optional DEVICE word (SCALIFY_DEV_TIMEOUT, SCALIFY_DEV_BAD_SCALE).
 * Errors: NULL, DTYPE, SHAPE, ALIGNMENT, UNSUPPORTED (hd != 64, causal with
 * Tk < Tq), ALIAS (O_s aliasing an input scale word).
 */
int scalify_scaled_attention(const scalify_array* Q, const scalify_array* K, const scalify_array* V, float sm_scale,
                             int causal, scalify_array* O, scalify_array* S_dump, scalify_array* P_dump,
                             uint32_t* status, void* stream);

/*
 * Fused scaled attention backward: the gradients of scalify_scaled_attention with
 * respect to Q, K and V, from the gradient dO of its output and the probabilities
 * P it used (its P_dump).  Same custom rule (Section 3.2.1), i.e. the composition
 * of the calls it replaces:
 *   dP_s = dO_s V_s kf(hd),   dP_d = (dO_d V_d^T) / kf(hd) rounded to BF16       (matmul rule)
 *   dS_d = P_d (dP_d - sum_j dP_d[i,j] P_d[i,j]) rounded to E5M2,
 *   dS_s = dP_s P_s c                                  (softmax backward, scalar c)
 *   dQ_s = dS_s K_s kf(Tk),   dQ_d = (dS_d K_d) / kf(Tk)                          (matmul rule)
 *   dK_s = dS_s Q_s kf(Tq),   dK_d = (dS_d^T Q_d) / kf(Tq)
 *   dV_s = P_s dO_s kf(Tq),   dV_d = (P_d^T dO_d) / kf(Tq)
 * i.e. scalify_scaled_matmul, scalify_scaled_softmax_bwd, scalify_scalar_mul_pow2
 * and three more scalify_scaled_matmul.  Two launches: one CTA per (head, 128
 * queries) forms dP (twice, it never reaches memory), dS and dQ; one CTA per
 * (head, 128 keys) contracts P and dS over the queries into dV and dK.
 *   Q, dO [heads, Tq, hd], K, V [heads, Tk, hd]: E4M3 or E5M2, hd = 64 or 128, 3-D views
 *   as for the forward call.  P: E4M3, dense [heads, Tq, Tk], non-negative (the
 *   sign bit is ignored), exact zeros where the mask hides a key.  dS (output): E5M2, dense [heads, Tq, Tk], scale word
 *   required; with causal != 0 the 128 x 128 blocks wholly above the diagonal are
 *   not written.  dQ [heads, Tq, hd], dK, dV [heads, Tk, hd]: F16, BF16 or F32
 *   (one dtype), same kind of view.  c: the forward's scalar, a power of two.
 *   Tk % 32 == 0.  dP_dump (BF16, dense [heads, Tq, Tk]): optional copy of dP_d
 *   for checking, normally NULL.  status: optional DEVICE word.
 * Errors: NULL (also: dS without a scale word), DTYPE, SHAPE, ALIGNMENT,
 * UNSUPPORTED (hd != 64, causal with Tk < Tq, c not a power of two), ALIAS (an
 * output scale word aliasing another scale word of the call).
 */
int scalify_scaled_attention_bwd(const scalify_array* Q, const scalify_array* K, const scalify_array* V,
                                 const scalify_array* P, const scalify_array* dO, float sm_scale, int causal,
                                 scalify_array* dS, scalify_array* dQ, scalify_array* dK, scalify_array* dV,
                                 scalify_array* dP_dump, uint32_t* status, void* stream);

/*
 * Scaled Adam step without a workspace.  (No counterpart in the paper: this entry point exists
 * for the integration, not for the method.)
 *
 * Same operation, arguments and results as scalify_scaled_adam_step, for callers that cannot
 * allocate the workspace that call needs: code running after the application's own memory
 * pool has taken all device memory (a further cudaMalloc would fail), code on a path where
 * the device-wide synchronisation of cudaMalloc is not acceptable, and integrations that are
 * handed nothing but the tensors.  The scratch (old scale words and new reciprocals per
 * tensor, and the status word) is a fixed 33 KB array inside the library image; every GPU
 * that loads the library holds it until the process exits.  The call allocates nothing and
 * frees nothing.
 *
 *   n_tensors   at most 1024; more returns SCALIFY_ERR_WORKSPACE and enqueues nothing.
 *   status_out  optional DEVICE pointer to one uint32: receives the SCALIFY_DEV_* bits of this
 *               call (0 if none), written in stream order.  May be NULL.
 *
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call before starting any stream capture.  All calls on a device
 * share the one array, which keeps the previous call's contents (the call clears what it
 * needs to start from zero): two calls that may overlap on the GPU - different streams
 * without an ordering between them - race on it; order them or use
 * scalify_scaled_adam_step with separate workspaces.
 */
int scalify_scaled_adam_step_static(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v,
                                    scalify_array* w, float lr, float beta1, float beta2, float eps, int64_t step,
                                    uint32_t* status_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SCALIFY_H_ */
