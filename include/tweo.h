/*
 * tweo.h -- C ABI of the B200 (sm_100a) library for FP8 per-tensor-scaled
 * linear layers and the TWEO activation penalty.
 *
 * What the calls compute follows the TWEO paper (arXiv 2511.23225):
 *   - Sec. 3.3, Eq. 2-3: the penalty  L_TWEO = (1/L) sum_l mean((|A^(l)|/(tau+eps))^p)
 *     on every transformer block output A^(l), weighted by lambda(t);
 *   - Sec. 4.3 (the subsection on full FP8 pre-training of LLMs): every linear layer runs in FP8 with ONE scale per tensor,
 *     E4M3 for activations and weights, E5M2 for gradients (the HYBRID recipe),
 *     scales derived from the tensor's absolute maximum;
 *   - Sec. 4.4 (the subsection on post-training quantisation), Eq. 4 and the "W8(T)A8(T)" discussion: inference with static
 *     per-tensor scales for weights and activations.
 *
 * Conventions (all calls)
 *   - Every function returns a tweo_status_t and never throws or exits.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, valid until
 *     the work enqueued by the call has finished.  Scalars the device produces
 *     (amax, scale, scale_inv, loss) are DEVICE pointers too, so calls can be
 *     chained on a stream without a host synchronisation.  Hyper-parameters are
 *     passed by value.  `stream` is a cudaStream_t passed as void*.
 *   - Calls only enqueue work on `stream`; they do not synchronise and do not
 *     allocate device memory.  Scratch memory, where needed, is passed in as
 *     (ws, ws_bytes); size it with tweo_workspace_bytes().  A workspace must be
 *     zero-filled once before its first use (tweo_workspace_init); every call
 *     leaves it ready for the next one.  Two calls that overlap on the GPU must
 *     not share a workspace.
 *   - Tensors are row-major.  bf16 tensors are passed as uint16_t bit patterns,
 *     FP8 tensors as uint8_t codes (OCP FP8: E4M3 has no infinity, NaN = 0x7F /
 *     0xFF, max finite 448; E5M2 is IEEE-like, max finite 57344).
 *   - Leading dimensions (ld*) are in ELEMENTS.  All tensor bases must be
 *     16-byte aligned and every row must start 16-byte aligned (ld * element
 *     size is a multiple of 16), otherwise TWEO_ERR_ALIGNMENT.
 *   - Weights are stored one row per output feature: W is [N rows, K columns],
 *     K contiguous (the layout of a framework's Linear.weight).
 *   - Device-side waits are bounded; if one expires the kernel records it and
 *     returns, and tweo_read_device_status() reports TWEO_ERR_TIMEOUT.
 */
#ifndef TWEO_H_
#define TWEO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Exported symbols (the library is built with hidden default visibility). */
#if defined(__GNUC__)
#define TWEO_API __attribute__((visibility("default")))
#else
#define TWEO_API
#endif

typedef int32_t tweo_status_t;
enum {
  TWEO_OK = 0,
  TWEO_ERR_INVALID_ARG = 1,        /* NULL where a pointer is required, negative size, bad enum */
  TWEO_ERR_UNSUPPORTED_SHAPE = 2,  /* a dimension the kernels cannot tile (see each call)         */
  TWEO_ERR_ALIGNMENT = 3,          /* base pointer or row pitch not 16-byte aligned               */
  TWEO_ERR_WORKSPACE_TOO_SMALL = 4,
  TWEO_ERR_CUDA = 5,               /* a CUDA runtime/driver call failed; see tweo_last_cuda_error */
  TWEO_ERR_TIMEOUT = 6             /* a bounded device-side wait expired                          */
};

typedef enum { TWEO_E4M3 = 0, TWEO_E5M2 = 1 } tweo_fp8_t;
typedef enum { TWEO_SCALE_CURRENT = 0, TWEO_SCALE_GIVEN = 1 } tweo_scale_mode_t;
typedef enum { TWEO_BF16 = 0, TWEO_F32 = 1, TWEO_FP8_E4M3 = 2 } tweo_dtype_t;
typedef enum {
  TWEO_OP_QUANTIZE = 0,
  TWEO_OP_LINEAR_FWD = 1,
  TWEO_OP_LINEAR_DGRAD = 2,
  TWEO_OP_LINEAR_WGRAD = 3,
  TWEO_OP_LOSS = 4,
  TWEO_OP_W8A8 = 5,
  TWEO_OP_BLOCK_OUTPUT = 6,
  TWEO_OP_ABSMAX = 7
} tweo_op_t;
typedef enum { TWEO_GRAN_TENSOR = 0, TWEO_GRAN_ROW = 1 } tweo_granularity_t;
typedef enum { TWEO_ACT_NONE = 0, TWEO_ACT_GELU = 1, TWEO_ACT_GELU_TANH = 2, TWEO_ACT_SWIGLU = 3 } tweo_act_t;
typedef enum { TWEO_NORM_LAYER = 0, TWEO_NORM_RMS = 1 } tweo_norm_t;

/* Upper bound on the number of block outputs one tweo_loss_fwd_bwd call takes. */
#define TWEO_MAX_BLOCKS 128

/*
 * Optional fused outputs of a GEMM epilogue (Sec. 4.3: with delayed scaling the
 * next layer's scale is known before the GEMM runs, so the cast of the output
 * can ride on the epilogue instead of costing two more passes over it).
 * All three act on the bf16-ROUNDED output values, so that the fused result is
 * bit-identical to running tweo_quantize_per_tensor(GIVEN) on the stored output.
 *   out_amax : device float*, receives max |y| over the whole output, or NULL.
 *   out_q    : device uint8*, receives sat_rne_fp8(fl32(y * *q_scale)), or NULL;
 *              row pitch ldq elements (multiple of 16), format q_fmt.
 *   q_scale  : device const float*, required when out_q != NULL.
 */
typedef struct tweo_epilogue_t {
  float* out_amax;
  uint8_t* out_q;
  int64_t ldq;
  int32_t q_fmt; /* tweo_fp8_t */
  const float* q_scale;
} tweo_epilogue_t;

/*
 * tweo_quantize_per_tensor -- amax, scale and FP8 cast of one bf16 tensor
 * (Sec. 4.3: one scaling factor for the entire tensor; E4M3 range +-448).
 *   x [n] bf16 in.  q [n] uint8 out (same element order).  n >= 0; n == 0 yields
 *   amax 0, scale 1 (CURRENT) and writes nothing to q.
 *   mode CURRENT: amax = max|x_i|; scale = fl32(FP8MAX/amax) (1 if amax is 0 or
 *     not finite; clamped to FLT_MAX on overflow); *scale, *scale_inv, *amax are
 *     written; q_i = sat_rne_fp8(fl32(x_i * scale)).
 *   mode GIVEN: *scale is read (delayed or static scaling), one pass; *amax of x
 *     is still written (it feeds the next step's scale); *scale_inv is written.
 *   Rounding: one binary32 multiply, then round-to-nearest-even to FP8 with
 *     saturation to +-FP8MAX; NaN -> 0x7F (no sign).  amax skips NaN.
 *   sat_count: device uint32*, or NULL; receives the number of elements with
 *     |fl32(x_i * scale)| > FP8MAX.
 *   Workspace: optional.  With ws == NULL the call runs as separate kernels (reset, amax,
 *     cast).  With a workspace of tweo_workspace_bytes(TWEO_OP_QUANTIZE) bytes (any
 *     contents) a CURRENT-scaling call without sat_count runs as two kernels: per-CTA
 *     maxima go to workspace slots and every CTA of the cast reduces them itself, so
 *     there is no reset kernel and no atomic.  Results are identical bit for bit.
 */
TWEO_API tweo_status_t tweo_quantize_per_tensor(const uint16_t* x, int64_t n, int32_t fmt, int32_t mode,
                                       float* scale, float* scale_inv, float* amax, uint8_t* q,
                                       uint32_t* sat_count, void* ws, size_t ws_bytes, void* stream);

/*
 * tweo_quantize_per_tensor_batch -- tweo_quantize_per_tensor for up to
 * TWEO_MAX_QUANT_BATCH tensors in one pair of kernels (Sec. 4.3: a linear layer casts its
 * activation, its weight and, in the backward pass, its output gradient, each with its
 * own per-tensor scale; casting them together saves launches, which dominate for small
 * tensors).  Every tensor is treated exactly as tweo_quantize_per_tensor would treat it
 * (own amax, own scale, own format and mode; results bit-identical).
 *   descs: HOST array of `count` descriptors (read during the call, not kept).
 *   ws: tweo_workspace_bytes(TWEO_OP_QUANTIZE) bytes, any contents.  The tensors with
 *     CURRENT scaling and no sat_count share one amax kernel and one cast kernel per FP8
 *     format; GIVEN-scale tensors and those with a sat_count (and all of them when ws is
 *     NULL or too small) are launched one by one as tweo_quantize_per_tensor does.
 *   Errors: TWEO_ERR_INVALID_ARG (count out of range, NULL pointers, bad enums),
 *     TWEO_ERR_ALIGNMENT.
 */
#define TWEO_MAX_QUANT_BATCH 8
typedef struct tweo_quant_desc_t {
  const uint16_t* x;   /* bf16 [n], device */
  int64_t n;
  int32_t fmt;         /* tweo_fp8_t */
  int32_t mode;        /* tweo_scale_mode_t */
  float* scale;        /* device; out (CURRENT) or in (GIVEN) */
  float* scale_inv;    /* device out */
  float* amax;         /* device out */
  uint8_t* q;          /* uint8 [n], device out */
  uint32_t* sat_count; /* device out, or NULL */
} tweo_quant_desc_t;
TWEO_API tweo_status_t tweo_quantize_per_tensor_batch(const tweo_quant_desc_t* descs, int32_t count, void* ws,
                                             size_t ws_bytes, void* stream);

/*
 * tweo_fp8_linear_fwd -- forward GEMM of an FP8 linear layer (Sec. 4.3):
 *   Y[M,N] = (Xq[M,K] . Wq[N,K]^T) * (*sx_inv) * (*sw_inv), fp32 accumulation on
 *   the tensor cores, result rounded once to bf16.
 *   xq [M,K] codes (fmt_x), wq [N,K] codes (fmt_w), y [M,N] bf16.
 *   Shapes: M >= 1 (ragged M is zero-filled by the loader); N % 16 == 0,
 *   K % 16 == 0.  epi may be NULL.
 *   ws is optional for the three linear calls (NULL, 0 is valid).  With a zero-
 *   initialised workspace of tweo_workspace_bytes(TWEO_OP_LINEAR_*) bytes the
 *   kernel may split tiles along the contraction when whole tiles would leave SMs
 *   idle (few output tiles, long contraction); partial sums are added in a fixed
 *   order, so results stay bit-reproducible.
 */
TWEO_API tweo_status_t tweo_fp8_linear_fwd(const uint8_t* xq, int64_t ldx, const uint8_t* wq, int64_t ldw,
                                  const float* sx_inv, const float* sw_inv, uint16_t* y, int64_t ldy,
                                  int64_t M, int64_t N, int64_t K, int32_t fmt_x, int32_t fmt_w,
                                  const tweo_epilogue_t* epi, void* ws, size_t ws_bytes, void* stream);

/*
 * tweo_fp8_linear_fwd_act -- forward GEMM of an FP8 linear layer with the MLP's activation
 * applied in the epilogue (Sec. 3.2: the classic MLP with GELU and the gated MLP of the
 * Llama-style blocks; Sec. 4.3: the next linear consumes FP8, so its input can be cast here
 * instead of in two more passes over the activation):
 *   Z[m,n] = (Xq . Wq^T)[m,n] * (*sx_inv) * (*sw_inv)                (binary32)
 *   TWEO_ACT_GELU       Y = Z * Phi(Z)  (erf form)
 *   TWEO_ACT_GELU_TANH  Y = Z/2 * (1 + tanh( sqrt(2/pi) (Z + 0.044715 Z^3) ))
 *   TWEO_ACT_SWIGLU     Y[m,n] = SiLU(Z[m,n]) * Z[m,N+n], n < N: wq holds 2N rows, the N
 *                       gate rows first, then the N up rows
 *   TWEO_ACT_NONE       Y = Z (the call forwards to tweo_fp8_linear_fwd; y required)
 * Y is evaluated in binary32 (Phi through the Abramowitz-Stegun 7.1.26 approximation of erfc,
 * absolute error 1.5e-7; the tanh form with the hardware tanh, relative error 2^-11) and
 * rounded once to bf16; the optional outputs of epi act on the rounded values exactly as
 * in tweo_fp8_linear_fwd.  xq [M,K], wq [N,K] (SwiGLU: [2N,K]) codes; y [M,N] bf16, or NULL
 * when only the FP8 copy (epi->out_q) is wanted.  Shapes: M >= 1, N % 16 == 0, K % 16 == 0.
 * Errors: TWEO_ERR_INVALID_ARG (NULL pointers, bad enums, neither y nor epi->out_q),
 * TWEO_ERR_UNSUPPORTED_SHAPE, TWEO_ERR_ALIGNMENT.
 */
TWEO_API tweo_status_t tweo_fp8_linear_fwd_act(const uint8_t* xq, int64_t ldx, const uint8_t* wq, int64_t ldw,
                                      const float* sx_inv, const float* sw_inv, int32_t act, uint16_t* y,
                                      int64_t ldy, int64_t M, int64_t N, int64_t K, int32_t fmt_x,
                                      int32_t fmt_w, const tweo_epilogue_t* epi, void* stream);

/*
 * tweo_layernorm_fp8 -- LayerNorm (or RMSNorm) over the last dimension with the FP8 cast of
 * its output for the following linear in the same pass (Sec. 4.3: the LayerNorm components run
 * under FP8 together with the linears; with delayed scaling the scale is known beforehand):
 *   TWEO_NORM_LAYER  mu = mean_j x_j, var = mean_j (x_j - mu)^2,
 *                    y_j = (x_j - mu) / sqrt(var + eps) * gamma_j + beta_j
 *   TWEO_NORM_RMS    y_j = x_j / sqrt(mean_j x_j^2 + eps) * gamma_j (+ beta_j if given)
 * evaluated in binary32 and rounded once to bf16; then, on the rounded values,
 *   yq_j = sat_rne_fp8( fl32(y_j * *q_scale) ) and *amax = max |y_j| over the whole output
 * (bit-identical to tweo_quantize_per_tensor(GIVEN) on the stored y).
 *   x [rows, d] bf16 (row pitch ldx); gamma, beta: device float [d] (beta may be NULL);
 *   y [rows, d] bf16 or NULL; yq [rows, d] codes (q_fmt) or NULL, q_scale required with yq;
 *   amax: device float* or NULL; mean, rstd: device float [rows] or NULL (mu and
 *   1/sqrt(var + eps) per row, for a backward pass).  At least one of y, yq must be given.
 * Shapes: d % 8 == 0, 8 <= d <= 8192; ldx, ldy, ldq multiples of 8; rows >= 0 (0: only *amax = 0).
 * Errors: TWEO_ERR_INVALID_ARG, TWEO_ERR_UNSUPPORTED_SHAPE, TWEO_ERR_ALIGNMENT.
 */
TWEO_API tweo_status_t tweo_layernorm_fp8(const uint16_t* x, int64_t ldx, int64_t rows, int64_t d, int32_t kind,
                                 const float* gamma, const float* beta, float eps, uint16_t* y, int64_t ldy,
                                 uint8_t* yq, int64_t ldq, int32_t q_fmt, const float* q_scale, float* amax,
                                 float* mean, float* rstd, void* stream);

/*
 * tweo_fp8_linear_bwd_dgrad -- data gradient (Sec. 4.3, gradients in E5M2):
 *   dX[M,K] = (dYq[M,N] . Wq[N,K]) * (*sdy_inv) * (*sw_inv) -> bf16; the
 *   contraction runs over N.  wq is the same buffer the forward call used.
 *   Shapes: N % 16 == 0, K % 16 == 0.  epi may be NULL.
 */
TWEO_API tweo_status_t tweo_fp8_linear_bwd_dgrad(const uint8_t* dyq, int64_t lddy, int32_t fmt_dy,
                                        const uint8_t* wq, int64_t ldw, int32_t fmt_w,
                                        const float* sdy_inv, const float* sw_inv, uint16_t* dx,
                                        int64_t lddx, int64_t M, int64_t N, int64_t K,
                                        const tweo_epilogue_t* epi, void* ws, size_t ws_bytes,
                                        void* stream);

/*
 * tweo_fp8_linear_bwd_wgrad -- weight gradient (Sec. 4.3):
 *   dW[N,K] = (dYq[M,N]^T . Xq[M,K]) * (*sx_inv) * (*sdy_inv); the contraction
 *   runs over the tokens M.  dw has the layout of W.  dw_dtype TWEO_BF16
 *   (uint16_t*) or TWEO_F32 (float*); accumulate != 0 adds into dw instead of
 *   overwriting it (F32 only).  Shapes: N % 16 == 0, K % 16 == 0, any M >= 1.
 */
TWEO_API tweo_status_t tweo_fp8_linear_bwd_wgrad(const uint8_t* xq, int64_t ldx, int32_t fmt_x,
                                        const uint8_t* dyq, int64_t lddy, int32_t fmt_dy,
                                        const float* sx_inv, const float* sdy_inv, void* dw,
                                        int64_t lddw, int32_t dw_dtype, int32_t accumulate,
                                        int64_t M, int64_t N, int64_t K, void* ws, size_t ws_bytes,
                                        void* stream);

/*
 * tweo_fp8_linear_bwd -- both gradients of a linear layer in one call (Sec. 4.3): exactly
 *   tweo_fp8_linear_bwd_dgrad (dX, bf16) followed by tweo_fp8_linear_bwd_wgrad (dW, bf16,
 *   overwrite), without fused epilogue outputs; results are bit-identical to the two calls.
 *   When M, N and K all exceed 128 the two products run as ONE kernel launch: their tiles
 *   form one list, longest first, dealt to the CTA pairs so that each pair gets about the
 *   same work (the weight gradient has few, long tiles; the data gradient many short ones),
 *   which removes most of the idle SM time the two products have on their own at
 *   transformer-block sizes.  Otherwise it makes the two calls one after the other.
 *   Arguments as in the two calls; ws is only used on the two-call path (may be NULL).
 */
TWEO_API tweo_status_t tweo_fp8_linear_bwd(const uint8_t* dyq, int64_t lddy, int32_t fmt_dy,
                                  const uint8_t* xq, int64_t ldx, int32_t fmt_x, const uint8_t* wq,
                                  int64_t ldw, int32_t fmt_w, const float* sdy_inv, const float* sx_inv,
                                  const float* sw_inv, uint16_t* dx, int64_t lddx, uint16_t* dw,
                                  int64_t lddw, int64_t M, int64_t N, int64_t K, void* ws,
                                  size_t ws_bytes, void* stream);

/*
 * tweo_fp8_linear_group -- up to TWEO_MAX_GROUP products of FP8 linear layers that do not depend on each other,
 * in ONE kernel launch (Sec. 4.3: every linear of the network runs these three products; which of them are
 * independent is the caller's knowledge -- the forward products of projections that share an input, the weight
 * gradients of several layers, the data and weight gradient of one layer).  Each problem is exactly
 *   TWEO_PRODUCT_FWD    out = Y [M,N]  = tweo_fp8_linear_fwd       (xq, wq;  sx_inv, sw_inv)
 *   TWEO_PRODUCT_DGRAD  out = dX [M,K] = tweo_fp8_linear_bwd_dgrad (dyq, wq; sdy_inv, sw_inv)
 *   TWEO_PRODUCT_WGRAD  out = dW [N,K] = tweo_fp8_linear_bwd_wgrad (xq, dyq; sx_inv, sdy_inv; bf16, overwrite)
 * without a workspace; results are bit-identical to those calls.  A FWD or DGRAD problem may carry the fused
 * epilogue of the single call (`epi`: amax of the bf16 output, which the call resets first, and / or its FP8 copy
 * with a given scale; the descriptor is read during the call); a WGRAD problem may not.  A launch costs
 * a fixed few microseconds (set-up, first loads, last epilogue) and leaves SMs idle at its ragged end; the tiles of
 * all problems of a group form one list, longest first, dealt to the CTA pairs so that each gets about the same
 * work, with one ramp-up and one tail for the whole group.
 *   problems: HOST array of `count` descriptors (read during the call, not kept); only the operands the product
 *   uses need to be set.  No output may alias an operand or another output of the group.
 *   Shapes: as the single calls, and both dimensions of every output must exceed 128
 *   (else TWEO_ERR_UNSUPPORTED_SHAPE: make the single call).
 *   Errors: TWEO_ERR_INVALID_ARG (count, NULL pointers, enums), TWEO_ERR_UNSUPPORTED_SHAPE, TWEO_ERR_ALIGNMENT.
 */
#define TWEO_MAX_GROUP 8
typedef enum { TWEO_PRODUCT_FWD = 0, TWEO_PRODUCT_DGRAD = 1, TWEO_PRODUCT_WGRAD = 2 } tweo_product_t;
typedef struct tweo_linear_problem_t {
  int32_t product;                      /* tweo_product_t */
  int32_t fmt_x, fmt_w, fmt_dy;         /* tweo_fp8_t of the operands used */
  const uint8_t* xq;                    /* [M,K] codes: FWD, WGRAD */
  int64_t ldx;
  const uint8_t* wq;                    /* [N,K] codes: FWD, DGRAD */
  int64_t ldw;
  const uint8_t* dyq;                   /* [M,N] codes: DGRAD, WGRAD */
  int64_t lddy;
  const float* sx_inv;                  /* device scalars */
  const float* sw_inv;
  const float* sdy_inv;
  uint16_t* out;                        /* bf16: Y [M,N], dX [M,K] or dW [N,K] */
  int64_t ldo;
  int64_t M, N, K;
  const tweo_epilogue_t* epi;           /* optional fused outputs of Y (FWD) or dX (DGRAD); NULL: none */
} tweo_linear_problem_t;
TWEO_API tweo_status_t tweo_fp8_linear_group(const tweo_linear_problem_t* problems, int32_t count, void* stream);

/*
 * tweo_loss_fwd_bwd -- TWEO penalty and its gradient in one pass (Eq. 3, and
 * the derivative of Eq. 2's lambda(t) * L_TWEO term):
 *   loss_l = (1/n) sum_i (|a_i| / (tau+eps))^p,          l = 0..L-1
 *   *loss  = (1/L) sum_l loss_l                           (= L_TWEO)
 *   g_i    = grad_coeff * p * sign(a_i) |a_i|^(p-1) / (n (tau+eps)^p),  g = 0 at a = 0
 *   a: HOST array of L device pointers, each a bf16 tensor of n_per_tensor
 *      elements (a block output [batch, seq, hidden] flattened; the mean runs
 *      over all of them).  1 <= L <= TWEO_MAX_BLOCKS.
 *   grad_coeff folds lambda(t), the 1/L of Eq. 3 and any upstream gradient.
 *   loss: device float* out.  loss_per_block: device float[L] out, or NULL.
 *   grad: HOST array of L device pointers (bf16 or float according to
 *      grad_dtype), or NULL for loss only.  grad[l] may alias a[l] only if
 *      grad_dtype is bf16 (in-place).
 *   p = 4 (the paper's setting) runs a fast path; other p > 1 a generic one.
 *   Needs a workspace (TWEO_OP_LOSS, any contents); the sum is reduced in a fixed order,
 *   so results are bit-reproducible run to run.  Two kernels: the streaming pass and a
 *   one-CTA kernel that adds its partial sums.
 */
TWEO_API tweo_status_t tweo_loss_fwd_bwd(const uint16_t* const* a, int32_t L, int64_t n_per_tensor, float tau,
                                float eps, float p, float grad_coeff, float* loss,
                                float* loss_per_block, void* const* grad, int32_t grad_dtype, void* ws,
                                size_t ws_bytes, void* stream);

/*
 * tweo_block_output_fused -- the block output and everything that touches it once, in one pass
 * (Sec. 3.3: the penalty acts on A = x + f(x), the residual stream plus the block's branch;
 * Sec. 4.3: with delayed scaling the FP8 scale of A for the next block is known beforehand):
 *   a_i   = bf16( fl32(x_i + f_i) )                  written to a [n] (may alias x or f)
 *   *loss = (1/n) sum_i (|a_i| / (tau+eps))^p        this block's term of Eq. 3
 *   g_i   = grad_coeff * p * sign(a_i) |a_i|^(p-1) / (n (tau+eps)^p)   -> grad [n] bf16, or NULL
 *   *amax = max_i |a_i|                              (feeds tweo_delayed_scaling_update)
 *   aq_i  = sat_rne_fp8( fl32(a_i * *q_scale) )      -> aq [n] in format q_fmt, or NULL
 * Every output equals, bit for bit, what tweo_loss_fwd_bwd (L = 1, bf16 gradient) and
 * tweo_quantize_per_tensor (GIVEN) produce from the stored a.  x, f: bf16 [n], device.
 * loss, amax: device float*.  q_scale: device const float*, required with aq.  grad must
 * not alias x, f or a.  Needs a workspace of
 * tweo_workspace_bytes(TWEO_OP_BLOCK_OUTPUT) bytes (any contents); the reduction order is fixed, so results
 * are reproducible run to run.
 */
TWEO_API tweo_status_t tweo_block_output_fused(const uint16_t* x, const uint16_t* f, int64_t n, float tau,
                                      float eps, float p, float grad_coeff, uint16_t* a, uint16_t* grad,
                                      float* loss, float* amax, uint8_t* aq, int32_t q_fmt,
                                      const float* q_scale, void* ws, size_t ws_bytes, void* stream);

/*
 * tweo_delayed_scaling_update -- one step of delayed per-tensor scaling for n_tensors tensors of
 * one FP8 format (Sec. 4.3: amax history of length 16 in the paper's runs).  For every tensor t:
 * the history amax_history[t][0..history_len) moves one place (the oldest value drops out),
 * amax_new[t] enters at index 0, and scale[t] = fl32(FP8MAX / max(history)) (clamped to FLT_MAX)
 * becomes the scale for the NEXT step; if that maximum is zero or not finite scale[t] is kept.
 * scale_inv[t] = fl32(1 / scale[t]).  All pointers are device pointers; start from a zeroed
 * history and scale 1.  Under data parallelism amax_new must already be the maximum over ranks.
 */
TWEO_API tweo_status_t tweo_delayed_scaling_update(float* amax_history, int32_t history_len,
                                          const float* amax_new, float* scale, float* scale_inv,
                                          int32_t n_tensors, int32_t fmt, void* stream);

/*
 * tweo_loss_fwd_bwd_static -- tweo_loss_fwd_bwd without a workspace argument.
 * (The paper has no counterpart to this call; it exists for deployment reasons only.)
 *
 * Some programs that embed this library may not allocate GPU memory at the point where
 * they call it: an inference or training server that hands all device memory to its own
 * pool at start-up and forbids later cudaMalloc calls, a plug-in running inside a host
 * application that owns the allocator, or a control loop that cannot tolerate the latency
 * or the possible failure of an allocation.  For them the scratch memory of the loss
 * kernel (its per-CTA partial sums) is a fixed 33024-byte array
 * compiled into the library; every GPU that loads the library holds it until the process
 * exits.  Inputs and outputs are still the caller's.  Arguments, results and numerics are
 * those of tweo_loss_fwd_bwd (same kernel, same reduction order).
 *
 *   Limit: L * (CTAs per tensor) must not exceed 4096 partial sums; beyond that the call
 *     returns TWEO_ERR_WORKSPACE_TOO_SMALL and does nothing (on a 148-SM B200 the kernel
 *     uses at most 592 + L CTAs, so every L <= TWEO_MAX_BLOCKS fits).
 *   The call performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   First call on a device: looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   The array is shared by every call in the process and keeps the last call's contents;
 *     the call clears the part that must start at zero.  Two such calls that overlap on
 *     the GPU (different streams, or different threads) race on it: serialise them, or
 *     use tweo_loss_fwd_bwd with separate workspaces.
 */
TWEO_API tweo_status_t tweo_loss_fwd_bwd_static(const uint16_t* const* a, int32_t L, int64_t n_per_tensor,
                                                float tau, float eps, float p, float grad_coeff, float* loss,
                                                float* loss_per_block, void* const* grad, int32_t grad_dtype,
                                                void* stream);

/*
 * tweo_w8a8_static_gemm -- inference linear with static per-tensor scales for
 * both operands (Sec. 4.4: AbsMax static quantisation, W8(T)A8(T)), in the E4M3
 * flavour: Y[M,N] = (Xq . Wq^T) * (1 / *sx) * (*sw_inv) -> bf16.
 *   x: activations [M,K]; x_dtype TWEO_BF16 (cast inside with the static scale
 *      *sx, saturating; needs a workspace for the codes) or TWEO_FP8_E4M3
 *      (already cast by the caller with *sx).
 *   sx: device const float*, the calibrated activation scale (FP8MAX / amax_cal).
 *   wq [N,K] E4M3 codes, sw_inv device const float*.
 *   Shapes: N % 16 == 0, K % 16 == 0, any M >= 1 (small M takes a
 *   weight-streaming split-K path).
 */
TWEO_API tweo_status_t tweo_w8a8_static_gemm(const void* x, int32_t x_dtype, int64_t ldx, const float* sx,
                                    const uint8_t* wq, int64_t ldw, const float* sw_inv, uint16_t* y,
                                    int64_t ldy, int64_t M, int64_t N, int64_t K, void* ws,
                                    size_t ws_bytes, void* stream);

/*
 * FP4 (E2M1) with one scale per tensor -- the number format the paper's conclusion names as the step
 * after FP8 (it fixes no format; taken here: the 4-bit floating-point element of the OCP
 * Microscaling formats, 1 sign / 2 exponent (bias 1) / 1 mantissa bit, values +-{0, 0.5, 1, 1.5, 2,
 * 3, 4, 6}, no infinity, no NaN) with the per-tensor scaling of Sec. 4.3: scale = fl32(6 / amax).
 *
 * tweo_fp4_quantize -- code_i = rne_sat(fl32(x_i * scale)): one binary32 multiply, one saturating
 * round-to-nearest-even onto the E2M1 grid (ties to the even code; |v| >= 6 and infinities -> +-6;
 * NaN -> +6, the format having no NaN; zero and values that round to zero keep their sign).
 *   x: bf16 [n], 16-byte aligned.  mode CURRENT: amax = max|x| (NaN skipped), scale = 6 / amax
 *   (1 when amax is 0 or not finite, clamped to FLT_MAX), scale_inv = 1 / scale are written;
 *   mode GIVEN: *scale is read, *scale_inv and *amax (of this tensor) are written.
 *   q4 (optional): packed codes, (n + 1) / 2 bytes, element 2i in the low nibble and element 2i + 1
 *   in the high nibble of byte i (an odd n leaves the last high nibble 0); 8-byte aligned.
 *   q8 (optional): "carriers", n bytes, the E4M3 code of every ROUNDED value (each E2M1 value is an
 *   E4M3 value), 16-byte aligned: the operand form the FP8 GEMM entry points take, which then compute
 *   the FP4 product exactly (pass fmt TWEO_E4M3 and this tensor's scale_inv).  At least one of q4, q8.
 * All scalars are device pointers; nothing is read back by the host.
 * Errors: TWEO_ERR_INVALID_ARG, TWEO_ERR_ALIGNMENT.
 */
TWEO_API tweo_status_t tweo_fp4_quantize(const uint16_t* x, int64_t n, int32_t mode, float* scale, float* scale_inv,
                                float* amax, uint8_t* q4, uint8_t* q8, void* stream);

/*
 * tweo_fp4_unpack -- packed E2M1 codes (as tweo_fp4_quantize writes them) -> carriers: q8[i] = E4M3
 * code of the value of code i.  For weights kept packed at rest and expanded once when loaded.
 *   q4: (n + 1) / 2 bytes, 16-byte aligned; q8: n bytes, 16-byte aligned.
 */
TWEO_API tweo_status_t tweo_fp4_unpack(const uint8_t* q4, int64_t n, uint8_t* q8, void* stream);

/*
 * tweo_w4a4_static_gemm -- inference linear with static per-tensor scales and both operands on the
 * E2M1 grid (the W4A4 setting the paper's conclusion points to, in its floating-point form):
 *   Y[M,N] = (Xq . Wq^T) * (1 / *sx) * (*sw_inv) -> bf16,  Xq = tweo_fp4_quantize(x, GIVEN *sx).
 *   x: bf16 [M,K], dense (ldx == K); sx: device const float*, the calibrated scale (6 / amax_cal).
 *   wq8 [N,K]: carriers of the weight codes (tweo_fp4_quantize's q8, or tweo_fp4_unpack of the
 *   packed codes), row pitch ldw; sw_inv: device const float*.
 *   ws: tweo_workspace_bytes(TWEO_OP_W8A8, M, N, K) bytes (holds the activation carriers).
 *   Shapes and routes as tweo_w8a8_static_gemm: N % 16 == 0, K % 16 == 0, any M >= 1.
 */
TWEO_API tweo_status_t tweo_w4a4_static_gemm(const uint16_t* x, int64_t ldx, const float* sx, const uint8_t* wq8,
                                    int64_t ldw, const float* sw_inv, uint16_t* y, int64_t ldy, int64_t M,
                                    int64_t N, int64_t K, void* ws, size_t ws_bytes, void* stream);

/*
 * tweo_fp4_weight_linear -- the few-token inference linear with the weights kept PACKED in memory (two E2M1 codes
 * per byte): Y[M,N] = (Xq . Wq^T) * (*sx_inv) * (*sw_inv) -> bf16 for M <= 128, where streaming W once bounds the
 * call -- packed weights halve that stream.  The loads expand the codes on their way into shared memory and the
 * tensor core reads them as E2M1 operands beside the 8-bit activations, so the result equals
 * tweo_fp8_linear_fwd on the carriers of the same codes.
 *   xq [M,K]: E4M3 or E5M2 codes (fmt_x), or E2M1 carriers (fmt_x = TWEO_E4M3; then the product is W4A4), row
 *   pitch ldx; w4 [N, K/2 bytes]: tweo_fp4_quantize's packed codes of a [N,K] weight, row pitch ldw_bytes;
 *   sx_inv, sw_inv: device scalars (reciprocal scales).
 *   Shapes: 1 <= M <= 128 (else TWEO_ERR_UNSUPPORTED_SHAPE: expand the weights once with tweo_fp4_unpack and use
 *   the FP8 entry points, which are bound by the tensor core there, not by the weight stream), N % 16 == 0,
 *   K % 128 == 0.  w4 32-byte aligned, ldw_bytes % 32 == 0, xq 16-byte aligned, ldx % 16 == 0.
 */
TWEO_API tweo_status_t tweo_fp4_weight_linear(const uint8_t* xq, int64_t ldx, int32_t fmt_x, const float* sx_inv,
                                     const uint8_t* w4, int64_t ldw_bytes, const float* sw_inv, uint16_t* y,
                                     int64_t ldy, int64_t M, int64_t N, int64_t K, void* stream);

/*
 * tweo_absmax_quantize -- symmetric AbsMax b-bit quantisation (Sec. 4.4, Eq. 4):
 *   s = max|X| + eps,  X_q = round(X / s * Q_b),  Q_b = 2^(b-1) - 1   (Q_8 = 127, Q_6 = 31),
 * with one s for the whole tensor (TWEO_GRAN_TENSOR: the paper's "T") or one per row
 * (TWEO_GRAN_ROW: per output channel "C" for a weight [N,K], per token "K" for an activation
 * [M,K]).  x [rows, cols] bf16, row pitch ldx elements; q [rows, cols] int8 codes in
 * [-Q_b, Q_b], row pitch ldq; s: device float [1] or [rows].
 *   mode CURRENT: s is computed and written; mode GIVEN: s is read (static quantisation) and
 *   values beyond it clamp to +-Q_b.  Arithmetic: binary32, each operation rounded once,
 *   X / s * Q_b evaluated as X * (Q_b / s) -- s = fl32(amax + eps), c = fl32(Q_b / s),
 *   q = clamp(rne(fl32(x * c))); ties to even; NaN -> 0 and skipped by the maximum.  2 <= bits <= 8.
 *   TWEO_GRAN_TENSOR needs a dense tensor (ldx == cols == ldq) and, in CURRENT mode, a
 *   workspace of tweo_workspace_bytes(TWEO_OP_ABSMAX) bytes (any contents).
 */
TWEO_API tweo_status_t tweo_absmax_quantize(const uint16_t* x, int64_t rows, int64_t cols, int64_t ldx,
                                   int32_t bits, int32_t granularity, int32_t mode, float eps, float* s,
                                   int8_t* q, int64_t ldq, void* ws, size_t ws_bytes, void* stream);

/*
 * tweo_int8_linear -- the 8-bit (or b-bit) integer linear of Sec. 4.4 on Eq. 4's codes:
 *   Y[M,N] = (sum_k Xq[m,k] Wq[n,k]) * (sx[m or 0] / Q_b) * (sw[n or 0] / Q_b)  -> bf16,
 * the product of the dequantised operands.  Integer tensor cores, int32 accumulation (exact).
 * xq [M,K], wq [N,K] int8 codes (row pitches multiples of 16); sx: device float [1] (per tensor,
 * static or not) or [M] (per token) with sx_per_row != 0; sw: [1] or [N] (per channel) with
 * sw_per_row != 0.  Shapes: N % 16 == 0, K % 16 == 0, any M >= 1.
 */
TWEO_API tweo_status_t tweo_int8_linear(const int8_t* xq, int64_t ldx, const float* sx, int32_t sx_per_row,
                               const int8_t* wq, int64_t ldw, const float* sw, int32_t sw_per_row,
                               int32_t bits, uint16_t* y, int64_t ldy, int64_t M, int64_t N, int64_t K,
                               void* stream);

/*
 * tweo_int8_linear_q8 -- tweo_int8_linear with the output requantised in the epilogue (Sec. 4.4: with the
 * residual stream quantised too, a block's linear hands 8-bit codes to the next operation and no bf16
 * tensor exists in between).  With y the binary32 value tweo_int8_linear would round to bf16,
 *   yq[m,n] = clamp( rne_int( fl32(y * fl32(Q_b / *sy)) ), -Q_b, Q_b ),  NaN -> 0       (Eq. 4, static scale)
 * sy: device float [1], the static per-tensor AbsMax scale of the output.  yq [M,N] int8, row pitch ldq a
 * multiple of 16.  Other arguments, shapes and errors as tweo_int8_linear.
 */
TWEO_API tweo_status_t tweo_int8_linear_q8(const int8_t* xq, int64_t ldx, const float* sx, int32_t sx_per_row,
                                  const int8_t* wq, int64_t ldw, const float* sw, int32_t sw_per_row,
                                  int32_t bits, const float* sy, int8_t* yq, int64_t ldq, int64_t M, int64_t N,
                                  int64_t K, void* stream);

/*
 * tweo_residual_add_q8 -- the residual addition y = x + f(x) on a quantised residual stream (Sec. 4.4):
 * x, f(x) and y are Eq. 4 codes with static per-tensor scales.  Dequantise, add, quantise; Q_b cancels:
 *   a = fl32(*sx / *sy),  b = fl32(*sf / *sy)
 *   yq_i = clamp( rne_int( fl32( fq_i * b + fl32(xq_i * a) ) ), -Q_b, Q_b ),  NaN -> 0
 * (binary32: one product, one fused multiply-add).
 * xq, fq, yq: int8 [n], device, 16-byte aligned (yq may alias xq or fq); sx, sf, sy: device float [1].
 * 2 <= bits <= 8.  Errors: TWEO_ERR_INVALID_ARG, TWEO_ERR_ALIGNMENT.
 */
TWEO_API tweo_status_t tweo_residual_add_q8(const int8_t* xq, const float* sx, const int8_t* fq, const float* sf,
                                   int64_t n, int32_t bits, const float* sy, int8_t* yq, void* stream);

/*
 * tweo_residual_add_q8_rows -- the residual addition on a residual stream quantised per token (Sec. 4.4: the
 * "A8(K)" granularity, one Eq. 4 scale per row): for every row m of the [rows, cols] codes
 *   y_mj  = fl32( fq_mj * fl32(sf[m] / Q_b) + fl32(xq_mj * fl32(sx[m] / Q_b)) )
 *   sy[m] = fl32( max_j |y_mj| + eps )                     the row's own AbsMax scale, written to sy
 *   yq_mj = clamp( rne_int( fl32(y_mj * fl32(Q_b / sy[m])) ), -Q_b, Q_b ),  NaN -> 0
 * xq, fq, yq: int8 [rows, cols], dense, device, 16-byte aligned (yq may alias xq or fq); sx, sf, sy: device
 * float [rows].  cols % 16 == 0, cols <= 8192; 2 <= bits <= 8; eps >= 0.
 * Errors: TWEO_ERR_INVALID_ARG, TWEO_ERR_UNSUPPORTED_SHAPE, TWEO_ERR_ALIGNMENT.
 */
TWEO_API tweo_status_t tweo_residual_add_q8_rows(const int8_t* xq, const float* sx, const int8_t* fq,
                                        const float* sf, int64_t rows, int64_t cols, int32_t bits, float eps,
                                        int8_t* yq, float* sy, void* stream);

/* ---------------------------------------------------------------- helpers */

/* Bytes of workspace `op` needs for the given problem (n for QUANTIZE / LOSS is
 * passed in M, with N = number of tensors for LOSS; unused dims may be 0). */
TWEO_API size_t tweo_workspace_bytes(int32_t op, int64_t M, int64_t N, int64_t K);

/* Zero-fills a workspace (enqueued on stream); call once after allocating it. */
TWEO_API tweo_status_t tweo_workspace_init(void* ws, size_t ws_bytes, void* stream);

/* Synchronises `stream`, then returns TWEO_ERR_TIMEOUT if any kernel since the
 * last call recorded an expired wait (and clears the record), TWEO_ERR_CUDA if
 * the stream reports an error, else TWEO_OK. */
TWEO_API tweo_status_t tweo_read_device_status(void* stream);

/*
 * tweo_selftest_bounded_wait -- exercises the error path of the bounded device-side waits (the
 * conventions above; no passage of the paper).  Launches one small kernel in which one thread waits,
 * with the same wait routine the GEMM kernels use, for a barrier that nobody signals; after
 * limit_ns nanoseconds (1 us .. 100 ms, else TWEO_ERR_INVALID_ARG) the wait gives up, records
 * TWEO_ERR_TIMEOUT in the device status word and the kernel returns normally -- nothing traps and
 * the context stays usable.  gave_up: device uint32* (or NULL) that receives 1 if the wait expired.
 * The next tweo_read_device_status() returns TWEO_ERR_TIMEOUT once, then TWEO_OK again.
 */
TWEO_API tweo_status_t tweo_selftest_bounded_wait(uint64_t limit_ns, uint32_t* gave_up, void* stream);

/*
 * Diagnostics.  With TWEO_LOG=1 in the environment (read once per process) every entry point prints one line to
 * stderr before anything else: its name, shapes, formats, pitches and which optional pointers are set.  Nothing is
 * read from the device and nothing is synchronised.  Device-side by-products that serve as metrics are ordinary
 * outputs: amax of every cast and fused epilogue, the optional saturation counter, the loss scalars.
 */
TWEO_API const char* tweo_status_string(tweo_status_t s);
TWEO_API const char* tweo_last_cuda_error(void); /* text of the last failing CUDA call in this thread */
TWEO_API int32_t tweo_version(void);             /* major * 10000 + minor * 100 + patch */

/* Number of kernel launches this library has enqueued since it was loaded. */
TWEO_API uint64_t tweo_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TWEO_H_ */
