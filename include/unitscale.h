/*
 * libunitscale -- unit-scaled linear / FFN ops for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every matrix is row-major DEVICE memory owned by the caller; the
 * library allocates nothing on the device, keeps no reference to a buffer after
 * a call returns, and never synchronises: each call enqueues its kernels on the
 * given stream (a cudaStream_t passed as void*, NULL = the default stream) and
 * returns.  Errors are reported through the return value only; argument,
 * dtype, shape and alignment checks all run on the host before any launch, so
 * a call that returns an error other than US_ERR_CUDA has launched nothing.
 * There is no CPU fallback.
 *
 * Notation follows the paper: a scaled op is f* = alpha * f in the forward pass
 * and f*_grad_i = beta_i * f_grad_i in the backward pass (section "Scaled ops");
 * X is [b x m], W is [m x n] = [fan_in x fan_out], G is the gradient of the
 * output, [b x n] (section "Example").
 */
#ifndef UNITSCALE_H_
#define UNITSCALE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  US_OK = 0,
  US_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, ld < cols, bad enum, shape mismatch */
  US_ERR_UNSUPPORTED = 2, /* dtype combination that has no kernel */
  US_ERR_ALIGNMENT = 3,   /* pointer not 16-byte aligned, or row pitch not a multiple of 16 bytes */
  US_ERR_WORKSPACE = 4,   /* workspace missing or smaller than us_workspace_bytes() */
  US_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed (launch, tensor-map encode) */
  US_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (reported by us_workspace_status) */
} us_status;

/* Storage formats.  E4M3 / E5M2 are the OCP 8-bit formats (rows "FP8 E4 (b)" and
 * "FP8 E5 (b)" of the appendix table "Common floating point formats for deep
 * learning"): E4M3 for activations and weights, E5M2 for gradients. */
typedef enum { US_F32 = 0, US_BF16 = 1, US_F16 = 2, US_E4M3 = 3, US_E5M2 = 4 } us_dtype;

/* A row-major matrix in device memory.  ld = elements between consecutive rows
 * (ld >= cols).  ptr must be 16-byte aligned and ld * sizeof(element) a multiple
 * of 16 bytes for every matrix handed to a linear op. */
typedef struct {
  void* ptr;
  int32_t dtype; /* us_dtype */
  int64_t rows, cols, ld;
} us_mat;

typedef enum {
  US_ACT_NONE = 0,
  US_ACT_GELU = 1, US_ACT_GELU_GRAD = 2,
  US_ACT_RELU = 3, US_ACT_RELU_GRAD = 4,
  US_ACT_TANH = 5, US_ACT_TANH_GRAD = 6,
  US_ACT_SIGMOID = 7, US_ACT_SIGMOID_GRAD = 8
} us_act;

/*
 * Work fused after the scaled accumulator of a linear op, applied per element in
 * float32 and rounded once to the output dtype (round-to-nearest-even; the FP8
 * casts saturate to the largest finite value):
 *
 *   v = scale * acc
 *   US_ACT_GELU:       if aux.ptr, aux = round16(v)  (the pre-activation the backward pass reads);
 *                      v = act_out_scale * gelu(act_in_scale * v)
 *   US_ACT_GELU_GRAD:  h = aux (required);
 *                      v = act_out_scale * act_in_scale * gelu'(act_in_scale * h) * v
 *   skip.ptr != NULL:  v = skip_coef * skip + out_coef * v
 *   out = round_to(out dtype, v)
 *
 * The RELU / TANH / SIGMOID pairs do the same with f = max(x, 0), tanh, (1 + e^-x)^-1 (table section
 * "Activations"; us_scales_activation gives their factors): forward v = act_out_scale * f(act_in_scale * v),
 * gradient v = act_out_scale * act_in_scale * f'(act_in_scale * h) * v, relu'(0) = 0.
 * gelu(x) = x * Phi(x) with the exact normal CDF (table "Table of unit scaling
 * factors"); act_in_scale is the alignment pre-scale of appendix "Aligning a unit
 * scaled model with an existing model" (1 when unused).  The skip path is the
 * fixed(tau) residual of section "Weighted addition": skip_coef = sqrt(1 - tau),
 * out_coef = sqrt(tau).  aux and skip have the shape of the output; aux is BF16 or
 * F16, skip is F32, BF16 or F16.
 */
typedef struct {
  int32_t act; /* us_act */
  float act_in_scale;
  float act_out_scale;
  us_mat aux;
  us_mat skip;
  float skip_coef;
  float out_coef;
} us_epilogue;

/* ------------------------------------------------------------------ linear ops
 *
 * The three GEMMs of a unit-scaled linear layer (section "Example"; table row
 * "matmul"):
 *
 *   us_linear_fwd    Y  = alpha  * X  W      X [b x m], W [m x n]  ->  Y  [b x n]
 *   us_linear_bwd_x  dX = beta_x * G  W^T    G [b x n], W [m x n]  ->  dX [b x m]
 *   us_linear_bwd_w  dW = beta_w * X^T G     X [b x m], G [b x n]  ->  dW [m x n]
 *
 * W is always passed in the [fan_in x fan_out] orientation; no transposed copy is
 * needed or made.  Products are formed from the stored operand values and
 * accumulated in float32 (tensor-core accumulators); the scale is one float32
 * multiply on the accumulator, followed by the optional epilogue (NULL = none)
 * and a single rounding to the output dtype.  The unit-scaling values of the
 * scales are alpha = m^-1/2, beta_x = n^-1/2, beta_w = b^-1/2 (us_scales_linear).
 *
 * Operand dtypes: both 8-bit (any mix of US_E4M3 / US_E5M2), or both US_BF16, or
 * both US_F16.  Output dtype: any us_dtype.  Every dimension must be >= 1; rows
 * and columns need not be multiples of the tile sizes.  Alignment rule: see
 * us_mat (violations return US_ERR_ALIGNMENT).
 *
 * ws: device workspace of at least us_workspace_bytes() bytes, 16-byte aligned,
 * zeroed once by the caller before its first use (cudaMemsetAsync).  It holds a
 * status word that a kernel sets if one of its bounded waits runs out.  The word
 * is sticky and only ever set, atomically, to one constant, so linear calls may
 * share a workspace, also calls that run concurrently on different streams; it
 * then tells that some call since the last clearing timed out, not which one.
 * Read it with us_workspace_status (after the streams in question have been
 * joined or synchronised) and clear it with cudaMemsetAsync.
 */
us_status us_linear_fwd(const us_mat* X, const us_mat* W, float alpha, const us_epilogue* ep,
                        const us_mat* Y, void* ws, size_t ws_bytes, void* stream);
us_status us_linear_bwd_x(const us_mat* G, const us_mat* W, float beta_x, const us_epilogue* ep,
                          const us_mat* dX, void* ws, size_t ws_bytes, void* stream);
us_status us_linear_bwd_w(const us_mat* X, const us_mat* G, float beta_w, const us_epilogue* ep,
                          const us_mat* dW, void* ws, size_t ws_bytes, void* stream);

/*
 * Batched forms: count[0] x count[1] independent problems of one shape in a single launch, e.g. the
 * (sequence, head) problems of scaled dot-product attention (appendix "Unit scaling and attention":
 * alpha = beta_1 = beta_2 = 1 / sqrt(d) for the scores; the scaled softmax output then feeds an
 * ordinary scaled matmul).  The us_mat arguments describe problem (0, 0); problem (i, j) of an
 * operand starts stride[0] * i + stride[1] * j elements further.  Problems may be strided views of
 * larger tensors (a head is a 64-column slice of a [tokens x 3 d] QKV matrix: ld = 3 d, inner
 * stride 64, outer stride = sequence length * ld).  Every stride times the element size must be a
 * multiple of 16 bytes (US_ERR_ALIGNMENT), strides of dimensions with count > 1 must be positive.
 * No fused epilogue; otherwise dtypes, alignment, workspace and errors as for the single forms.
 */
typedef struct {
  int64_t count[2];      /* number of problems in the outer / inner batch dimension (>= 1 each) */
  int64_t a_stride[2];   /* first operand: elements between consecutive problems, outer / inner */
  int64_t b_stride[2];   /* second operand */
  int64_t out_stride[2]; /* output */
} us_batch;

us_status us_linear_fwd_batched(const us_mat* X, const us_mat* W, float alpha, const us_mat* Y, const us_batch* batch,
                                void* ws, size_t ws_bytes, void* stream);
us_status us_linear_bwd_x_batched(const us_mat* G, const us_mat* W, float beta_x, const us_mat* dX, const us_batch* batch,
                                  void* ws, size_t ws_bytes, void* stream);
us_status us_linear_bwd_w_batched(const us_mat* X, const us_mat* G, float beta_w, const us_mat* dW, const us_batch* batch,
                                  void* ws, size_t ws_bytes, void* stream);

/*
 * us_linear_group: count (1..4) independent linear ops as ONE kernel launch.
 *
 * Each call is one of the three GEMMs of section "Example" with the same arithmetic, rounding and
 * scale handling as the single entry points (bit-identical results: a tile is always accumulated by
 * one accumulator over its whole K range).  The ops must not depend on one another (no output of one
 * is an operand, skip tensor or output of another).  Meant for the tail of a training step, where
 * several GEMMs of different shapes are ready at once -- for the FFN block the second forward GEMM,
 * both weight-gradient GEMMs and the first layer's input-gradient GEMM -- and separate launches
 * would each leave a partly filled last wave: the tiles of all calls are dealt to the SMs together,
 * longest contraction first.
 *
 * a, b: the two operands in the order of the single entry point for `op` (X, W / G, W / X, G);
 * scale: alpha, beta_x or beta_w; ep: act must be US_ACT_NONE, the skip path (fixed(tau) residual) is
 * available; out as for the single entry points.
 *
 * Covered by this form: FP8 operands, outputs with more than 128 rows and more than 128 columns.
 * Any other valid call (16-bit operands, a fused activation, a small output, more tiles than the
 * work list holds) returns US_ERR_UNSUPPORTED and launches nothing: issue those calls one by one.
 * Other errors and the workspace as for us_linear_fwd.
 */
typedef enum { US_OP_FWD = 0, US_OP_BWD_X = 1, US_OP_BWD_W = 2 } us_linear_op;
typedef struct {
  int32_t op; /* us_linear_op */
  us_mat a, b;
  float scale;
  us_epilogue ep;
  us_mat out;
} us_linear_call;
us_status us_linear_group(int count, const us_linear_call* calls, void* ws, size_t ws_bytes, void* stream);

/*
 * us_ffn_hidden: both GEMMs that end in the hidden layer of the FFN block, as ONE kernel launch.
 *
 * The scaled FFN of the figure "PyTorch examples" is linear -> gelu -> linear; with the ops of section
 * "Example" and the table row "gelu" its hidden layer takes part in
 *
 *   forward    H  = alpha  * X W1                 X [b x m], W1 [m x f]       (us_linear_fwd)
 *              A  = act_out_scale * gelu(act_in_scale * H)                    (its US_ACT_GELU epilogue)
 *   backward   dA = beta_x * G W2^T               G [b x n], W2 [f x n]       (us_linear_bwd_x)
 *              dH = grad_out_scale * act_in_scale * gelu'(act_in_scale * H16) * dA   (its US_ACT_GELU_GRAD epilogue)
 *
 * where H16 is H rounded to h_dtype (US_BF16 or US_F16), the format in which the two separate calls hand the
 * pre-activation from the forward to the backward pass.  When the gradient G of the block's output is at hand
 * before the forward pass starts (a training step whose upstream gradient is an input, as in the benchmark of
 * the FFN block, or a recomputed block), both GEMMs can run tile by tile side by side: H stays on the SM,
 * rounded exactly as above, and is never written to or read from memory, which takes 4 bytes per element of
 * the block's largest tensor off the path.  A and dH are bit-identical to what the two separate calls give.
 *
 * X, W1, G, W2: 8-bit operands (any mix of US_E4M3 / US_E5M2).  A, dH [b x f]: 8-bit outputs, rounded once,
 * saturating.  H: NULL (or ptr NULL), or a [b x f] matrix of h_dtype that receives H16.
 * Covered: b > 128 and f > 128.  Other valid shapes return US_ERR_UNSUPPORTED and launch nothing: use the
 * two separate calls.  Alignment, workspace, status word and errors as for us_linear_fwd.
 */
us_status us_ffn_hidden(const us_mat* X, const us_mat* W1, float alpha, const us_mat* G, const us_mat* W2, float beta_x,
                        float act_in_scale, float act_out_scale, float grad_out_scale, int32_t h_dtype, const us_mat* H,
                        const us_mat* A, const us_mat* dH, void* ws, size_t ws_bytes, void* stream);

/* us_test_ffn_hidden_starved: us_test_linear_fwd_starved for the kernel of us_ffn_hidden (no operand loads, every
 * device-side wait gives up after `wait_limit` polls, 1 .. 65536): the kernel raises the status word, frees its
 * tensor memory and returns by itself; A and dH are not valid afterwards.  All scales are 1. */
us_status us_test_ffn_hidden_starved(const us_mat* X, const us_mat* W1, const us_mat* G, const us_mat* W2, const us_mat* A,
                                     const us_mat* dH, void* ws, size_t ws_bytes, unsigned int wait_limit, void* stream);

/* Bytes of device workspace the linear ops need. */
size_t us_workspace_bytes(void);

/* us_linear_fwd_check: the host-side checks of us_linear_fwd (arguments, dtypes, shapes, alignment,
 * workspace) without a launch: returns what us_linear_fwd would return before it reaches the device,
 * US_OK if it would launch.  Touches neither the device nor `ws` (only its address and size are looked at). */
us_status us_linear_fwd_check(const us_mat* X, const us_mat* W, const us_epilogue* ep, const us_mat* Y,
                              const void* ws, size_t ws_bytes);

/* Waits for `stream`, copies the workspace status word to the host and returns
 * US_OK, US_ERR_TIMEOUT (a device-side wait gave up: the outputs of that call are
 * not valid) or US_ERR_CUDA.  This is the only call that synchronises. */
us_status us_workspace_status(const void* ws, void* stream);

/*
 * us_linear_fwd_static_ws: us_linear_fwd for callers that cannot supply a workspace.
 * (The paper has no counterpart; this is a property of the library, not of the method.)
 *
 * Same computation, arguments and errors as us_linear_fwd, except that the scratch the kernel
 * needs comes from a fixed 1024-byte array built into the library instead of from the caller.
 * It is meant for code that has no way to allocate device memory: a plug-in that receives only
 * its input and output buffers from the runtime hosting it, a serving loop that bans allocation
 * once it is running because cudaMalloc stalls the device, a process whose framework has
 * claimed all device memory for its own pool.  The call allocates and frees nothing, directly
 * or through a library; each GPU that loads the library holds the 1024 bytes until exit.
 *
 *  - The first call on a device looks up the array's device address (a one-time set-up with
 *    that device current).  Make that first call before starting any stream capture.
 *  - All calls share the one array and it keeps the previous call's contents, so every call that
 *    passes the host-side checks first clears the status word on `stream` (a call that returns an
 *    argument, dtype, alignment or workspace error enqueues nothing and leaves the word as it was).  Two calls that overlap on the GPU (different
 *    streams) race on that word: keep calls to this entry point on one stream, or order them.
 *  - If the kernel's scratch requirement ever exceeds the built-in 1024 bytes the call returns
 *    US_ERR_WORKSPACE and launches nothing; the requirement does not depend on the matrix sizes.
 *  - ws_out (may be NULL) receives the device address of the built-in scratch; pass it to
 *    us_workspace_status to learn whether this call's kernel timed out, before the next call
 *    clears the word.
 */
us_status us_linear_fwd_static_ws(const us_mat* X, const us_mat* W, float alpha, const us_epilogue* ep,
                                  const us_mat* Y, void** ws_out, void* stream);

/*
 * us_test_linear_fwd_starved: exercises the failure path of the linear kernels (the paper has no counterpart;
 * this exists so that the bounded waits and their clean-up can be tested without faulting a GPU).
 * It launches the kernel of us_linear_fwd (no epilogue) with two changes: the warp that loads the
 * operands issues no loads, and every device-side wait gives up after `wait_limit` polls
 * (1 .. 65536) instead of the library's normal limit.  Nothing is in flight, so the waits of all roles run
 * out, the kernel raises the status word in `ws`, releases its tensor memory and returns by itself;
 * us_workspace_status(ws) then reports US_ERR_TIMEOUT and Y is not valid.  The device and the
 * context stay usable: clear the word (cudaMemsetAsync) and carry on.  Arguments and host-side
 * errors as for us_linear_fwd.
 */
us_status us_test_linear_fwd_starved(const us_mat* X, const us_mat* W, float alpha, const us_mat* Y, void* ws,
                                     size_t ws_bytes, unsigned int wait_limit, void* stream);

/* Activations of the table "Table of unit scaling factors", section Activations. */
typedef enum { US_FN_GELU = 0, US_FN_RELU = 1, US_FN_TANH = 2, US_FN_SIGMOID = 3 } us_fn;

/* ------------------------------------------------------------ elementwise ops
 *
 * Unfused forms of the ops between the GEMMs.  All tensors of a call have the
 * same rows x cols; any ld >= cols; pointers need only the natural alignment of
 * their element type (rows whose start is 16-byte aligned take the 128-bit path).
 *
 * us_gelu_fwd      A  = alpha * gelu(s_in * H)                      (table row "gelu")
 * us_gelu_bwd      dH = beta * s_in * gelu'(s_in * H) * dA
 * us_residual_add  out = sqrt(1 - tau) * skip + sqrt(tau) * branch  (section "Weighted
 *                  addition", scheme fixed(tau)); serves the backward pass too: there
 *                  skip = incoming gradient, branch = gradient at the branch entry.
 * us_activation_fwd  A  = alpha * f(s_in * H) for f = relu(x) = max(x, 0), tanh, sigmoid(x) = (1 + e^-x)^-1
 *                  or gelu (table rows relu / gelu / tanh / sigmoid: alpha = 1 / std f(Z), Z ~ N(0,1));
 * us_activation_bwd  dH = beta * s_in * f'(s_in * H) * dA (beta = 1 / rms f'(Z)); relu'(0) = 0.
 *                  US_FN_GELU gives the same values as us_gelu_fwd / us_gelu_bwd.
 * us_weighted_add  out = alpha * sum_i gamma_i * src_i over count (1..8) tensors of one shape (table row
 *                  weighted_add: alpha = (sum_i gamma_i^2)^-1/2 keeps unit scale; each input's gradient
 *                  is then the incoming gradient times alpha * gamma_i * beta_i with beta_i = 1 /
 *                  gamma_i, i.e. no kernel of its own).  The coefficient alpha * gamma_i is formed in
 *                  float32 and applied by one fused multiply-add per input, in the order given.
 *                  The running-mean residual of section "Weighted addition" is us_residual_add
 *                  with tau = 1 / (l + 1).  src, gamma: host arrays of count elements.
 * us_cast_fp8      dst = q(scale * src), q = nearest value of the FP8 format, ties to
 *                  even, saturating (section "Floating-point formats for deep learning",
 *                  paragraph "Quantisation error"); the product is one float32
 *                  multiply.  NaN stays NaN.
 *
 * us_cast_fp8_multi  count (1..8) casts dst[i] = q(scale[i] * src[i]) as ONE kernel launch: the
 *                  same arithmetic as count calls of us_cast_fp8 (bit-identical results), for
 *                  the casts that open a training step (weights, activations and the incoming
 *                  gradient all go to FP8 before the first matmul needs them, figure "PyTorch
 *                  examples": every matmul input is quantised), where four short launches cost
 *                  more than the bytes they move.  src, scale, dst: host arrays of count
 *                  elements.  Every tensor must be free of row padding (ld == cols) and start
 *                  on a 16-byte boundary: US_ERR_UNSUPPORTED / US_ERR_ALIGNMENT otherwise, and
 *                  nothing is launched.  Tensors must not overlap.
 *
 * Inputs may be F32, BF16 or F16 (us_weighted_add also takes E4M3 / E5M2 inputs: partial results that travelled
 * in 8 bits); outputs any us_dtype (us_cast_fp8, us_cast_fp8_multi: E4M3 or E5M2 only).  0 <= tau <= 1.
 */
us_status us_gelu_fwd(const us_mat* H, float s_in, float alpha, const us_mat* A, void* stream);
us_status us_gelu_bwd(const us_mat* H, const us_mat* dA, float s_in, float beta, const us_mat* dH,
                      void* stream);
us_status us_activation_fwd(us_fn fn, const us_mat* H, float s_in, float alpha, const us_mat* A, void* stream);
us_status us_activation_bwd(us_fn fn, const us_mat* H, const us_mat* dA, float s_in, float beta,
                            const us_mat* dH, void* stream);
us_status us_residual_add(const us_mat* skip, const us_mat* branch, float tau, const us_mat* out,
                          void* stream);
us_status us_weighted_add(int count, const us_mat* src, const float* gamma, float alpha, const us_mat* out,
                          void* stream);
us_status us_cast_fp8(const us_mat* src, float scale, const us_mat* dst, void* stream);
us_status us_cast_fp8_multi(int count, const us_mat* src, const float* scale, const us_mat* dst,
                            void* stream);

/* ------------------------------------------------------------ fused scaled dot-product attention (forward)
 *
 * Appendix "Unit scaling and attention" and paragraph "Softmax (followed by matmul)", for count[0] x
 * count[1] independent (sequence, head) problems in one launch:
 *
 *   S = alpha_scores * Q K^T                       Q [s_q x 64], K [s_k x 64]; S is never stored and never rounded
 *   P = softmax_scale * softmax(S), row by row     rounded to the operands' format (it is a matmul input)
 *   C = alpha_context * P V                        V [s_k x 64]; C [s_q x 64] rounded to C's dtype
 *
 * with alpha_scores = 1 / sqrt(64), softmax_scale = s_k and alpha_context = s_k^-1/2 for the
 * unconstrained unit-scaled layer (us_scales_attention).  The us_mat arguments describe problem (0, 0);
 * problem (i, j) of a tensor starts stride[0] * i + stride[1] * j elements further (heads are 64-column
 * slices of a [tokens x 3 d] QKV matrix, C a 64-column slice of a [tokens x d] matrix).  P may be NULL;
 * otherwise the rounded weights are also written to P [s_q x s_k] (the backward pass needs them).
 * Q, K, V (and P): all BF16, all F16 or all E4M3 (FP8 activations; weights above 448 saturate), device memory;
 * C: any us_dtype.  Head width must be 64 and
 * s_k at most 512, else US_ERR_UNSUPPORTED; s_k = 0 with s_q > 0 is US_ERR_INVALID_ARG, s_q = 0 is
 * a no-op.  Base addresses, row pitches and the strides of dimensions with count > 1 must be multiples
 * of 16 bytes (US_ERR_ALIGNMENT); those strides must be positive and counts lie in 1..65535
 * (US_ERR_INVALID_ARG).  Nothing is allocated and nothing owned; ws as for the linear ops (a wait that
 * runs out inside the kernel raises US_ERR_TIMEOUT there).
 */
typedef struct {
  int64_t count[2];      /* number of problems in the outer / inner batch dimension (>= 1 each) */
  int64_t q_stride[2];   /* elements between consecutive problems, outer / inner */
  int64_t k_stride[2];
  int64_t v_stride[2];
  int64_t c_stride[2];
  int64_t p_stride[2];   /* ignored when P is NULL */
} us_attention_batch;

us_status us_attention_fwd(const us_mat* Q, const us_mat* K, const us_mat* V, float alpha_scores, float softmax_scale,
                           float alpha_context, const us_mat* C, const us_mat* P, const us_attention_batch* batch,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * us_attention_bwd: the backward pass of us_attention_fwd down to the queries, in one launch:
 *
 *   dP = beta_p * dC V^T                                           score-sized, never stored and never rounded
 *   dS = softmax_beta * p (dP - sum_k p_k dP_k),  p = P / softmax_alpha    rounded to the gradients' format
 *   dQ = beta_q * dS K
 *
 * dC [s_q x 64] is the gradient of the context, P [s_q x s_k] the weights the forward call stored, K and V [s_k x 64].
 * dS [s_q x s_k] is written for the caller's dK = beta dS^T Q matmul (dV = beta P^T dC needs only P and dC); dQ
 * [s_q x 64] in any us_dtype.  dC, P, K, V and dS: all BF16 or all F16; or FP8: dC and dS E5M2 (gradients), P, K, V E4M3.  Shapes, limits, batch description (one stride
 * pair per tensor), alignment, workspace and errors as for us_attention_fwd; softmax_alpha must be positive.
 */
typedef struct {
  int64_t count[2];
  int64_t dc_stride[2];
  int64_t p_stride[2];
  int64_t k_stride[2];
  int64_t v_stride[2];
  int64_t ds_stride[2];
  int64_t dq_stride[2];
} us_attention_bwd_batch;

us_status us_attention_bwd(const us_mat* dC, const us_mat* P, const us_mat* K, const us_mat* V, float beta_p,
                           float softmax_alpha, float softmax_beta, float beta_q, const us_mat* dS, const us_mat* dQ,
                           const us_attention_bwd_batch* batch, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------ scaled softmax
 *
 * Row-wise scaled softmax and its gradient (table "Table of unit scaling factors", row softmax:
 * alpha = beta = s for rows of s elements; appendix paragraph "Softmax (followed by matmul)": the
 * output is then about one everywhere, and the following matmul uses its ordinary factor).
 *
 *   us_softmax_fwd   P_ij  = alpha * exp(S_ij - max_j S_ij) / sum_j exp(S_ij - max_j S_ij)
 *   us_softmax_bwd   dS_ij = beta * p_ij * (dP_ij - sum_k p_ik dP_ik),   p = P / alpha
 *
 * The backward pass takes the forward pass's scaled output P (as stored) and the gradient dP of
 * that output.  All tensors of a call have the same rows x cols; inputs F32, BF16 or F16 (P of
 * us_softmax_bwd may also be E4M3 / E5M2: an output stored for an FP8 matmul), outputs any us_dtype; any ld >= cols (rows that start 16-byte aligned, with cols a multiple of 8, take
 * the 128-bit path).  alpha must be positive in us_softmax_bwd.
 */
us_status us_softmax_fwd(const us_mat* S, float alpha, const us_mat* P, void* stream);
us_status us_softmax_bwd(const us_mat* P, const us_mat* dP, float alpha, float beta, const us_mat* dS, void* stream);

/* Softmax cross-entropy (table row softmax_xent: softmax_xent(x, t) = log softmax(x)_t, alpha = 1,
 * beta = s / sqrt(s - 1) for rows of s classes).
 *
 *   us_softmax_xent_fwd   out_i = x_{i,t_i} - log sum_j exp(x_ij)               (float32, one per row, <= 0)
 *   us_softmax_xent_bwd   dX_ij = beta * g_i * ([j == t_i] - softmax(x_i)_j)    (g == NULL: g_i = 1)
 *
 * X [rows x s]: F32, BF16 or F16, any ld >= s; targets: device array of rows int32 class indices in
 * [0, s) (an index outside gives NaN forward and no one-hot term backward); out, g: device float32
 * arrays of rows elements; dX: any us_dtype, shape of X.
 */
us_status us_softmax_xent_fwd(const us_mat* X, const int32_t* targets, float* out, void* stream);
us_status us_softmax_xent_bwd(const us_mat* X, const int32_t* targets, const float* g, float beta,
                              const us_mat* dX, void* stream);

/* ------------------------------------------------------------ scaled layer norm
 *
 * layer_norm(X, w, c)_ij = c_j + w_j (X_ij - mu_i) / sigma_i over the rows of X [b x n], mu_i the row
 * mean and sigma_i^2 = mean_j X_ij^2 - mu_i^2 (+ eps; the table's formula has no eps, pass 0 for it),
 * with the factors of table "Table of unit scaling factors", row layer_norm: alpha = 1, beta_x = 1,
 * beta_w = beta_c = b^-1/2 (appendix: the weight and bias are cut-edges and take their own factors).
 *
 * us_layer_norm_fwd   Y = c + w * xhat.
 * us_layer_norm_bwd   dX_ij = beta_x / sigma_i * (u_ij - mean_j u_ij - xhat_ij * mean_j(u_ij xhat_ij)),
 *                     u = G * w;  dw_j = beta_wc * sum_i G_ij xhat_ij;  dc_j = beta_wc * sum_i G_ij.
 *                     xhat and sigma are recomputed from X (nothing is saved by the forward call).
 *                     The column sums are formed without atomics, in a fixed order: the result does
 *                     not depend on scheduling.  Two launches.
 *
 * X, G: F32 / BF16 / F16, any ld >= cols.  w, c: 1 x n vectors, F32 / BF16 / F16.  Y, dX: any
 * us_dtype; dw, dc: 1 x n, F32 / BF16 / F16.  Arithmetic in float32; the variance is accumulated
 * about the mean.  Backward: n <= 4096 (US_ERR_UNSUPPORTED beyond) and a device workspace of
 * us_layer_norm_bwd_workspace_bytes(b, n) bytes, 16-byte aligned, owned by the caller, which must
 * not be used by another call that may run at the same time (US_ERR_WORKSPACE if too small).
 * The size depends on the current device's SM count.  eps >= 0.
 */
us_status us_layer_norm_fwd(const us_mat* X, const us_mat* w, const us_mat* c, float eps, const us_mat* Y,
                            void* stream);
size_t us_layer_norm_bwd_workspace_bytes(int64_t rows, int64_t cols);
us_status us_layer_norm_bwd(const us_mat* X, const us_mat* w, const us_mat* G, float eps, float beta_x,
                            float beta_wc, const us_mat* dX, const us_mat* dw, const us_mat* dc, void* ws,
                            size_t ws_bytes, void* stream);

/* ------------------------------------------------------------ quantisation diagnostics
 *
 * us_quant_stats: for v = scale * src (one float32 multiply per element) and a storage format fmt
 * (E4M3 / E5M2 saturating, BF16 / F16 IEEE), in one pass:
 *   sums[0] = sum v^2,  sums[1] = sum (q_fmt(v) - v)^2        (double; their ratio is the signal-to-noise
 *             ratio of section "Floating-point formats for deep learning", paragraph "Quantisation error")
 *   hist[0]         count of |v| < 2^exp_lo (zeros included)
 *   hist[1 + k]     count of 2^(exp_lo + k) <= |v| < 2^(exp_lo + k + 1),  k = 0 .. nbins - 1
 *   hist[nbins + 1] count of |v| >= 2^(exp_lo + nbins), infinities and NaNs
 *             (the histograms of floor(log2 |x|) of appendix "Histograms of tensor-scaling within BERT")
 * src: F32 / BF16 / F16, any ld >= cols.  1 <= nbins <= 64, -126 <= exp_lo, exp_lo + nbins <= 128.
 * sums (2 doubles) and hist (nbins + 2 64-bit counts) are device arrays; ws is a device workspace of
 * us_quant_stats_workspace_bytes() bytes owned by the caller (US_ERR_WORKSPACE if smaller).  Sums are
 * formed in a fixed order without atomics on global memory: repeated calls give identical results.
 */
size_t us_quant_stats_workspace_bytes(void);
us_status us_quant_stats(const us_mat* src, float scale, us_dtype fmt, int exp_lo, int nbins, double* sums,
                         unsigned long long* hist, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------- host helpers
 *
 * us_scales_linear: unit-scaling factors of matmul(X[b x m], W[m x n]).
 *   constrained == 0: alpha = m^-1/2, beta_x = n^-1/2, beta_w = b^-1/2 (table row "matmul").
 *   constrained != 0: alpha = beta_x = (m n)^-1/4 (geometric mean, section "Example").
 * us_scales_gelu: 1/std of gelu(z) and 1/rms of gelu'(z) for z ~ N(0,1) (the table prints
 *   them as 1.701 / 1.481); constrained: both equal their geometric mean.
 * us_scales_activation: the same pair for any us_fn (relu: sqrt(2 / (1 - 1/pi)), sqrt 2; tanh
 *   1.593 / 1.467; sigmoid 4.802 / 4.722 as printed, carried here to float precision).
 * us_scales_residual: the coefficients of the fixed(tau) residual of section "Weighted addition",
 *   sqrt(1 - tau) for the skip connection and sqrt(tau) for the branch, 0 <= tau <= 1 (tau = 1 / (l + 1)
 *   gives the running-mean scheme for layer l).
 * us_scales_attention: factors of scaled dot-product attention for sequences of s tokens and heads of
 *   d_head features (appendix "Unit scaling and attention"; table row "softmax"; paragraph "Softmax
 *   (followed by matmul)"): scores S = alpha_scores Q K^T with alpha_scores = beta_scores = d_head^-1/2 (beta for both
 *   dQ and dK); softmax_scale = s (alpha and beta of the scaled softmax); context C = alpha_context P V, an
 *   ordinary matmul with fan_in = s, fan_out = d_head, batch = s: alpha_context = s^-1/2, beta_p = d_head^-1/2
 *   (gradient of P), beta_v = s^-1/2 (gradient of V); constrained: alpha_context = beta_p = (s d_head)^-1/4.
 * Pure host arithmetic; output pointers must be non-NULL.
 */
us_status us_scales_linear(int64_t b, int64_t m, int64_t n, int constrained, float* alpha,
                           float* beta_x, float* beta_w);
us_status us_scales_gelu(int constrained, float* alpha, float* beta);
us_status us_scales_activation(us_fn fn, int constrained, float* alpha, float* beta);
us_status us_scales_residual(float tau, float* skip_coef, float* branch_coef);
us_status us_scales_attention(int64_t s, int64_t d_head, int constrained, float* alpha_scores, float* beta_scores,
                              float* softmax_scale, float* alpha_context, float* beta_p, float* beta_v);

const char* us_status_string(us_status s);
int us_version(void);

#ifdef __cplusplus
}
#endif
#endif /* UNITSCALE_H_ */
