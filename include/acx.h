/*
 * acx.h -- C ABI of libacx: the compressed linear-operator step on one B200 (sm_100a).
 *
 * The operation (paper: Definition 3.1 for a linear operator, and Section 4, "Activation-Gradient
 * Co-Compression"):
 *   forward    Z = X W^T is computed exactly; of X only the low-rank factor pair (U, V) with
 *              X_hat = U V^T is kept.  Here the compressor is the random projection named in the
 *              paper's experimental setup: V = S, U = X S, with S (d_in x r) a seeded Gaussian
 *              sketch, E[S S^T] = I, so that E[X_hat] = X (the premise of Theorem 3.2(a)).
 *   backward   dX = G W exactly (Theorem 3.3(a)); the weight gradient G^T X_hat = (G^T U) V^T is
 *              produced as its left factor A = G^T U (d_out x r); the right factor is S again.
 *   reconstruct  optimizer strategy (i) of Section 4: dW = A S^T.
 *
 * S is never an argument and is never kept between calls: it is a pure function of (seed, sketch_kind, i, j)
 * that every call regenerates on the GPU, inside its kernels or once into the call's workspace ("Gaussian v1":
 * Philox4x32-10 with key = seed and counter (i, j/4, 0, sketch_kind), then a Box-Muller transform made only of
 * binary32 +, -, * rounded to nearest even (no fused multiply-add, no library function; the reciprocal and the
 * reciprocal square root are fixed Newton iterations), then a multiplication by fp32(1/sqrt(r)); for ACX_BF16 the
 * operand is that value rounded to bfloat16, ties to even).  acx_sketch_materialize writes it out for inspection.
 * The calls with a _v suffix take an explicit second factor V^T from memory instead (Section 4's general pair).
 *
 * Conventions for every call
 *   - All matrix pointers are DEVICE pointers, row-major, densely packed, 16-byte aligned, owned by
 *     the caller, and must not overlap each other.  The descriptor is a HOST pointer.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     the call returns without synchronising.  The library allocates no memory.
 *   - Argument errors are reported before anything is launched; nothing is written in that case.
 *   - Shapes: tokens >= 0 (0 is a no-op); d_in, d_out >= 8 and multiples of 8; 16 <= r <= 256 and a
 *     multiple of 16; r <= d_in.  Anything else returns ACX_ERR_UNSUPPORTED_SHAPE.
 *   - io_dtype selects the element type of X, W, G, Y, dX, XS and of the S operand.  A and dW are
 *     always fp32.  All accumulation is fp32; each output element is rounded once, to nearest even.
 *   - The first call of an entry point on a device does one-time set-up for that device (it resolves the
 *     addresses of the library's device variables and sets kernel attributes).  Make that first call outside
 *     any stream capture; later calls can be captured.
 *   - State the library keeps (per process; nothing else survives a call): a device status word per GPU that
 *     kernels set when a bounded wait expires (read and cleared by acx_last_device_status: it reports for the
 *     whole device, whatever stream the kernel ran on); a count of kernel launches (acx_kernel_launches); the
 *     per-device caches of the set-up above; and the fixed scratch array of
 *     acx_linear_bwd_factor_builtin_scratch.
 */
#ifndef ACX_H_
#define ACX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ACX_VERSION 100 /* major*100 + minor */

#if defined(__GNUC__)
#define ACX_API __attribute__((visibility("default")))
#else
#define ACX_API
#endif

typedef enum acx_status {
  ACX_OK = 0,
  ACX_ERR_INVALID_ARG = 1,       /* null pointer, bad struct_size, unknown enum value */
  ACX_ERR_UNSUPPORTED_SHAPE = 2, /* see "Shapes" above */
  ACX_ERR_ALIGNMENT = 3,         /* a pointer is not 16-byte aligned */
  ACX_ERR_WORKSPACE = 4,         /* workspace missing or smaller than acx_workspace_bytes() */
  ACX_ERR_CUDA = 5,              /* a CUDA runtime call or launch failed */
  ACX_ERR_TIMEOUT = 6,           /* a bounded device-side wait expired (see acx_last_device_status) */
  ACX_ERR_SCRATCH_LIMIT = 7      /* the problem needs more than ACX_BUILTIN_SCRATCH_BYTES of built-in scratch */
} acx_status;

typedef enum acx_dtype { ACX_F32 = 0, ACX_BF16 = 1 } acx_dtype;

typedef enum acx_op {
  ACX_OP_FWD = 0, ACX_OP_BWD = 1, ACX_OP_RECONSTRUCT = 2,
  ACX_OP_BWD_BUILTIN_SCRATCH = 3, /* bytes of built-in scratch acx_linear_bwd_factor_builtin_scratch would use */
  ACX_OP_RSVD = 4,
  ACX_OP_BIAS_GRAD = 5,
  ACX_OP_BWD_BIAS = 6
} acx_op;

/* Problem descriptor: plain data, filled by the caller, read-only for the library. */
typedef struct acx_desc {
  uint32_t struct_size; /* sizeof(acx_desc); guards against layout drift */
  uint32_t sketch_kind; /* 0 = "Gaussian v1"; no other kind exists */
  int64_t tokens;       /* m: rows of X, G, Y, dX, XS */
  int64_t d_in;         /* columns of X and W, rows of S */
  int64_t d_out;        /* rows of W, columns of G and Y, rows of A */
  int32_t r;            /* sketch rank (the paper's k): columns of S, XS, A */
  int32_t io_dtype;     /* acx_dtype */
  uint64_t seed;        /* S = S(seed, sketch_kind); the same seed must be used in fwd, bwd, reconstruct */
} acx_desc;

/* Bytes of device scratch the given op needs for this descriptor (0 if none; 0 on a bad descriptor).
 * The scratch is only used during the call; its contents need no initialisation. */
ACX_API size_t acx_workspace_bytes(const acx_desc* desc, int op);

/* Forward (Definition 3.1; Section 4 with U = X S):  Y = X W^T,  XS = X S.
 *   X  [tokens x d_in]  io_dtype, in        W  [d_out x d_in] io_dtype, in
 *   Y  [tokens x d_out] io_dtype, out       XS [tokens x r]   io_dtype, out (the stored factor U)
 *   XS may be NULL: then only Y is computed.  Linears that read the same input (q/k/v, gate/up; the paper
 *   compresses such an input once, Section 5) share one factor: one of them stores XS, the others pass NULL
 *   and later hand that same XS (and the same seed) to acx_linear_bwd.
 *   ws/ws_bytes: scratch of at least acx_workspace_bytes(desc, ACX_OP_FWD) bytes (r x d_in io elements for
 *   ACX_BF16, else 0), or NULL.  With a workspace S^T is written there once per call by a small grid and the
 *   GEMM reads it back through L2; with ws == NULL every thread block regenerates its slices of S in shared
 *   memory instead (same bits in Y and XS, a few per cent slower, nothing to allocate).  A workspace that is
 *   given but too small is ACX_ERR_WORKSPACE. */
ACX_API acx_status acx_linear_fwd(const acx_desc* desc, const void* X, const void* W, void* Y, void* XS,
                          void* ws, size_t ws_bytes, void* cuda_stream);

/* Forward with an explicit second factor (Section 4: any factor pair X^ = U V^T of the stored activation, for
 * instance the orthonormal basis a randomized SVD of X yields, Section 5):  Y = X W^T,  XV = X V.
 *   Vt [r x d_in] io_dtype, in: V transposed, row j is the j-th basis vector.  The library does not check that
 *      V V^T approximates the identity; the gradient estimate is exact only on the row space of Vt.
 *   XV [tokens x r] io_dtype, out (the stored factor U = X V); must not be NULL.
 *   The other arguments are those of acx_linear_fwd; desc->seed is not read.  The backward of such a layer is
 *   acx_linear_bwd with XS := XV (it never touches the second factor), and the full gradient is
 *   acx_reconstruct_v with the same Vt.  The caller owns Vt and keeps it until then (r x d_in elements, which
 *   is what the seeded sketch saves). */
ACX_API acx_status acx_linear_fwd_v(const acx_desc* desc, const void* X, const void* W, const void* Vt, void* Y, void* XV,
                                    void* ws, size_t ws_bytes, void* cuda_stream);

/* Affine operator (appendix, "Bias term": Z = X W^T + B; the bias gradient equals the output gradient and does not
 * depend on X, so compression leaves it exact).  Reading taken here: B is one bias vector added to every token's row,
 * B = 1 b^T, whose gradient is the column sum of the output gradient.
 *   acx_linear_fwd_bias:  Y = X W^T + 1 b^T,  XS = X S.   bias [d_out] io_dtype, in; everything else as acx_linear_fwd.
 *      The bias is added to the fp32 accumulator in the GEMM's epilogue, before the one rounding of Y.
 *   acx_bias_grad:        db[c] = sum over the tokens of G_out[t][c].   G_out [tokens x d_out] io_dtype, in;
 *      db [d_out] fp32, out;  ws/ws_bytes: scratch of at least acx_workspace_bytes(desc, ACX_OP_BIAS_GRAD) bytes.
 *      A separate pass over G_out (it is not folded into acx_linear_bwd); fixed summation order, reproducible bits.
 *      tokens == 0 sets db to zero.
 *   acx_linear_bwd_bias:  acx_linear_bwd plus db in one call: the gradient-factor kernel, which stages every tile of
 *      G_out anyway, adds up its columns on the side (warps that would otherwise idle during the contraction), so db costs
 *      no second pass over G_out.  dW_A and db must not be NULL, dX may be; ws/ws_bytes: at least
 *      acx_workspace_bytes(desc, ACX_OP_BWD_BIAS) bytes.  Fixed summation order, reproducible bits; db differs from
 *      acx_bias_grad's only by the order of its fp32 additions.
 * All three need io_dtype == ACX_BF16 (else ACX_ERR_INVALID_ARG). */
ACX_API acx_status acx_linear_fwd_bias(const acx_desc* desc, const void* X, const void* W, const void* bias, void* Y, void* XS,
                                       void* ws, size_t ws_bytes, void* cuda_stream);
ACX_API acx_status acx_bias_grad(const acx_desc* desc, const void* G_out, float* db, void* ws, size_t ws_bytes, void* cuda_stream);
ACX_API acx_status acx_linear_bwd_bias(const acx_desc* desc, const void* G_out, const void* W, const void* XS, void* dX, float* dW_A,
                                       float* db, void* ws, size_t ws_bytes, void* cuda_stream);

/* Backward (Definition 3.1, Theorem 3.3(a); Section 4's factored gradient):
 *   dX = G_out W  (exact),   dW_A = G_out^T XS  (left gradient factor; right factor is S(seed)).
 *   G_out [tokens x d_out] io_dtype, in     W    [d_out x d_in] io_dtype, in
 *   XS    [tokens x r]     io_dtype, in     dX   [tokens x d_in] io_dtype, out
 *   dW_A  [d_out x r] fp32, out (overwritten)
 *   dX may be NULL to skip the input gradient (first layer); dW_A may be NULL to skip the factor.
 *   With both outputs (ACX_BF16) the factor's kernel is queued behind dX's without waiting for it (it reads nothing
 *   that dX writes), so its thread blocks fill the SMs that the last tiles of dX leave idle. */
ACX_API acx_status acx_linear_bwd(const acx_desc* desc, const void* G_out, const void* W, const void* XS,
                          void* dX, float* dW_A, void* ws, size_t ws_bytes, void* cuda_stream);

/* Gradient factor without a caller-supplied workspace (the paper has no counterpart: this entry point
 * exists for the sake of callers, not of the method).
 *
 *   dW_A = G_out^T XS        what acx_linear_bwd writes to dW_A for ACX_BF16: the same products in fp32; how the
 *                            token range is split, and so the last bits of the sums, may differ.
 *   G_out [tokens x d_out] bf16, in     XS [tokens x r] bf16, in     dW_A [d_out x r] fp32, out
 *
 * Who it is for: code that must not allocate device memory at the point where the backward pass runs.
 * Typical cases are a trainer whose memory pool already owns nearly all of the GPU, so that a fresh
 * allocation can fail or stall every stream while the driver makes room; a plug-in or callback that is
 * forbidden to call into the allocator it was called from; and a service with a fixed amount of memory
 * that is audited at start-up.  Such a caller cannot produce the workspace that acx_linear_bwd wants
 * for its split-K partial sums, so this call keeps those partial sums in a fixed array of
 * ACX_BUILTIN_SCRATCH_BYTES that is part of the library image: every GPU on which the library's
 * kernels are loaded holds that array until the process exits.  The call itself allocates nothing: it
 * makes no cudaMalloc/cudaFree and calls no allocating library routine.
 *
 * Limits and rules
 *   - io_dtype must be ACX_BF16 (else ACX_ERR_INVALID_ARG).
 *   - If the partial sums of this shape need more than ACX_BUILTIN_SCRATCH_BYTES, nothing is launched
 *     and ACX_ERR_SCRATCH_LIMIT is returned; acx_workspace_bytes(desc, ACX_OP_BWD_BUILTIN_SCRATCH) tells the need.
 *   - The first call on each device looks up the array's device address (the device must be current,
 *     as for every call).  Like every entry point's first call, make it outside any stream capture.
 *   - All calls on one device share the one array.  Two calls whose kernels may overlap on the GPU
 *     (different streams without an ordering between them, or different host threads) race on it and
 *     give undefined results: keep calls on one stream or order them with events.
 *   - The array keeps whatever the previous call left there.  Nothing has to start at zero: every
 *     partial sum that is read was written earlier in the same call.
 *   - tokens == 0 sets dW_A to zero, like acx_linear_bwd. */
#define ACX_BUILTIN_SCRATCH_BYTES (16u << 20)
ACX_API acx_status acx_linear_bwd_factor_builtin_scratch(const acx_desc* desc, const void* G_out, const void* XS,
                                                         float* dW_A, void* cuda_stream);

/* Reconstruct (Section 4, optimizer strategy (i)):  dW = beta * dW + dW_A S^T.
 *   dW_A [d_out x r] fp32, in        dW [d_out x d_in] fp32, in/out
 *   beta = 0 overwrites (dW is not read), beta = 1 accumulates.
 *   ws/ws_bytes: scratch of at least acx_workspace_bytes(desc, ACX_OP_RECONSTRUCT) bytes (may be NULL if 0).
 *   For ACX_BF16 the product is formed on the tensor cores from dW_A split into two bfloat16 terms
 *   (relative error of the split 2^-17) and from S rounded to bfloat16, with fp32 accumulation. */
ACX_API acx_status acx_reconstruct(const acx_desc* desc, const float* dW_A, float* dW, float beta, void* ws, size_t ws_bytes,
                                   void* cuda_stream);

/* Reconstruct with an explicit second factor (Section 4, optimizer strategy (i) for a factor pair U V^T):
 *   dW = beta * dW + dW_A Vt,   Vt [r x d_in] io_dtype as in acx_linear_fwd_v; everything else as acx_reconstruct.
 *   For ACX_BF16 Vt is bfloat16 and dW_A is split into two bfloat16 terms as above. */
ACX_API acx_status acx_reconstruct_v(const acx_desc* desc, const float* dW_A, const void* Vt, float* dW, float beta, void* ws,
                                     size_t ws_bytes, void* cuda_stream);

/* Hyper-parameters of one AdamW step (decoupled weight decay; Loshchilov & Hutter, ICLR 2019, Algorithm 2). */
typedef struct acx_adamw_params {
  uint32_t struct_size; /* sizeof(acx_adamw_params) */
  int32_t step;         /* t >= 1: number of this step, for the bias corrections 1 - beta^t */
  float lr, beta1, beta2, eps, weight_decay;
} acx_adamw_params;

/* Reconstruct fused with the optimizer update (Section 4, optimizer strategy (i): the full gradient A S^T is rebuilt
 * and handed to a standard update; the paper's experiments use AdamW).  The gradient only ever exists tile by tile in
 * tensor memory; dW is never written:
 *     g = dW_A S^T,   m <- beta1 m + (1 - beta1) g,   v <- beta2 v + (1 - beta2) g^2,
 *     W <- W - lr * ( (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps) + weight_decay * W ).
 *   dW_A [d_out x r] fp32, in          W [d_out x d_in] fp32 master weights, in/out
 *   m, v [d_out x d_in] fp32, in/out   W_lp [d_out x d_in] bfloat16, out: W rounded to nearest even (may be NULL)
 *   ws/ws_bytes: as for acx_reconstruct.  io_dtype must be ACX_BF16 (else ACX_ERR_INVALID_ARG); g is formed as in
 *   acx_reconstruct (dW_A as two bfloat16 terms, S rounded to bfloat16, fp32 accumulation); the update runs in fp32 with
 *   the approximate hardware square root and quotient (1-2 ulp). */
ACX_API acx_status acx_reconstruct_adamw(const acx_desc* desc, const float* dW_A, float* W, float* m, float* v, void* W_lp,
                                         const acx_adamw_params* hp, void* ws, size_t ws_bytes, void* cuda_stream);

/* Low-rank optimizer states (Section 4, optimizer strategy (ii): a GaLore-style update, Zhao et al., ICML 2024,
 * Algorithm 2 with the projection on the right and scale 1).  Adam's moments are kept for the gradient factor, not for
 * the weights (d_out x r each instead of d_out x d_in), and the normalised step is projected back through V^T:
 *     m_A <- beta1 m_A + (1 - beta1) dW_A,   v_A <- beta2 v_A + (1 - beta2) dW_A^2,
 *     N = (m_A / (1 - beta1^t)) / (sqrt(v_A / (1 - beta2^t)) + eps),
 *     W <- W - lr * (N V^T + weight_decay * W).
 *   dW_A [d_out x r] fp32, in            m_A, v_A [d_out x r] fp32, in/out
 *   Vt [r x d_in] bfloat16, in: the second factor as in acx_linear_fwd_v, or NULL for V = S(desc->seed)
 *   W [d_out x d_in] fp32 master weights, in/out
 *   ws/ws_bytes: as for acx_reconstruct.  io_dtype must be ACX_BF16 (else ACX_ERR_INVALID_ARG).
 *   The moments only make sense while V stays the same: keep the seed (or Vt) of a layer fixed over the steps that
 *   share one pair of moments, as GaLore keeps its projection between subspace switches.  The factor-space step is
 *   computed in fp32 with IEEE square root and quotient, then applied like acx_reconstruct with beta = 1 - lr *
 *   weight_decay (the step as two bfloat16 terms, V^T in bfloat16, fp32 accumulation). */
ACX_API acx_status acx_lowrank_adamw(const acx_desc* desc, const float* dW_A, float* m_A, float* v_A, const void* Vt, float* W,
                                     const acx_adamw_params* hp, void* ws, size_t ws_bytes, void* cuda_stream);

/* Randomized-SVD compressor (Section 5, set-up: the paper's low-error compressor; Halko, Martinsson, Tropp, SIAM Review
 * 2011, Algorithm 4.1 without power iterations and the projection step of Algorithm 5.1).  Its compressed activation is
 * the orthogonal projection of X on the range of the sketch U = X S, X^ = U (U^T U)^-1 U^T X.  The forward
 * (acx_linear_fwd) already stores that U; this call adds the matching second factor of Section 4,
 *     Vt = (U^T U + ridge I)^-1 U^T X        [r x d_in] io_dtype, out,
 * so that U Vt = X^ (the same X^ as Q Q^T X with Q an orthonormal basis of U's columns; Q is never formed, and the SVD
 * that Algorithm 5.1 ends with would only re-express the same X^).  ridge = 2^-20 times the largest diagonal entry of
 * U^T U keeps the r x r solve defined when X has rank below r.
 *   X [tokens x d_in] io_dtype, in      U [tokens x r] io_dtype, in (the XS of acx_linear_fwd for this X and seed)
 *   ws/ws_bytes: scratch of at least acx_workspace_bytes(desc, ACX_OP_RSVD) bytes.
 *   io_dtype must be ACX_BF16 (else ACX_ERR_INVALID_ARG), tokens > 0.
 * Afterwards the layer is used like one with an explicit second factor: acx_linear_bwd with XS := U, then
 * acx_reconstruct_v or acx_lowrank_adamw with this Vt.  d_out and seed of desc are not read. */
ACX_API acx_status acx_rsvd_factor(const acx_desc* desc, const void* X, const void* U, void* Vt, void* ws, size_t ws_bytes,
                                   void* cuda_stream);

/* Synchronises the stream and returns ACX_ERR_TIMEOUT if any kernel on this device since the last call gave up on
 * a bounded wait (its outputs are then undefined), ACX_ERR_CUDA on a CUDA error, else ACX_OK.  Clears the flag.  The
 * flag is one word per device: a kernel on any stream sets it, so the answer is about the device, not only about
 * `cuda_stream` (which is the stream that is synchronised first). */
ACX_API acx_status acx_last_device_status(void* cuda_stream);

ACX_API const char* acx_status_string(int status);
ACX_API int acx_version(void);

/* ---------------------------------------------------------------------------------------------------------------
 * Test and debug entry points.  None of them is needed to use the calls above.
 * --------------------------------------------------------------------------------------------------------------- */

/* Test/debug: write S (d_in x r, row-major, io_dtype) to S_out.  Not needed by the other calls. */
ACX_API acx_status acx_sketch_materialize(const acx_desc* desc, void* S_out, void* cuda_stream);

/* Test/debug: launches one warp that waits, with the same bounded wait the kernels use, on a barrier that is never
 * signalled, for limit_ns nanoseconds (1 .. 1e9).  The wait runs out, the kernel records that in the device status
 * word and returns normally; acx_last_device_status then reports ACX_ERR_TIMEOUT once.  This is how the error path
 * of the bounded waits is exercised without hanging or faulting the GPU. */
ACX_API acx_status acx_debug_expired_wait(uint64_t limit_ns, void* cuda_stream);

/* Test/debug: overrides how the forward and dX pick their tile shape, so that tests can run every kernel variant on any
 * shape: 0 = the cost models decide (default), 1 / 2 = one CTA per tile of 128 / 256 rows, 3 / 4 = a pair of CTAs
 * (tcgen05.mma.cta_group::2) per tile of 256 / 512 rows.  A variant that does not exist for a call (a pair on 256-row tiles
 * with the sketch generated in place) falls back to the cost model's choice among the others.  Process-wide; results do
 * not depend on the mode beyond the order of fp32 additions inside a tile, which is the same in all of them. */
ACX_API acx_status acx_debug_force_gemm_mode(int mode);

/* Test/debug: number of kernels this library has launched in this process so far (all streams, all devices). */
ACX_API unsigned long long acx_kernel_launches(void);


#ifdef __cplusplus
}
#endif
#endif /* ACX_H_ */
