// Front end of the linear ops: argument checks and the choice of operand layout and epilogue kind;
// tensor maps, tile configuration and the launch live with the kernel instantiations (gemm_inst.cu).
#include <cuda.h>

#include "gemm_kernel.cuh"
#include "gemm_launch.h"
#include "host.h"

namespace us {

static bool aligned16(const us_mat* m) {
  return reinterpret_cast<uintptr_t>(m->ptr) % 16 == 0 && (m->ld * dtype_size(m->dtype)) % 16 == 0;
}
static bool valid_mat(const us_mat* m) {
  return m && m->ptr && m->rows >= 1 && m->cols >= 1 && m->ld >= m->cols && m->rows < (1ll << 31) &&
         m->cols < (1ll << 31) && m->dtype >= US_F32 && m->dtype <= US_E5M2;
}
static bool is_fp8(int dt) { return dt == US_E4M3 || dt == US_E5M2; }

enum Op { kFwd, kBwdX, kBwdW };

// Failure-path test settings of one call: a short wait limit, and a producer that issues no loads.
struct WaitTest {
  uint32_t wait_limit;
  int no_loads;
};

// A, B: the two operands in call order; out [M x N].
static us_status linear(Op op, const us_mat* A, const us_mat* B, float scale, const us_epilogue* ep, const us_mat* out,
                        void* ws, size_t ws_bytes, void* stream, const us_batch* batch = nullptr,
                        const WaitTest* wt = nullptr, bool validate_only = false) {
  if (!valid_mat(A) || !valid_mat(B) || !valid_mat(out)) return US_ERR_INVALID_ARG;
  int64_t M, N, K;
  bool shapes_ok;
  switch (op) {
    case kFwd:  M = A->rows; K = A->cols; N = B->cols; shapes_ok = B->rows == K; break;                 // X[b,m] W[m,n]
    case kBwdX: M = A->rows; K = A->cols; N = B->rows; shapes_ok = B->cols == K; break;                 // G[b,n] W[m,n]
    default:    M = A->cols; K = A->rows; N = B->cols; shapes_ok = B->rows == K; break;                 // X[b,m] G[b,n]
  }
  if (!shapes_ok || out->rows != M || out->cols != N) return US_ERR_INVALID_ARG;
  const bool f8 = is_fp8(A->dtype) && is_fp8(B->dtype);
  const bool h16 = (A->dtype == US_BF16 || A->dtype == US_F16) && A->dtype == B->dtype;
  if (!f8 && !h16) return US_ERR_UNSUPPORTED;
  if (!aligned16(A) || !aligned16(B) || !aligned16(out)) return US_ERR_ALIGNMENT;

  GemmParams p{};
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.scale = scale;
  p.out = out->ptr; p.out_dt = out->dtype; p.out_ld = out->ld;
  p.out_coef = 1.f;
  p.wait_limit = wt ? wt->wait_limit : kWaitLimit;
  p.no_loads = wt ? wt->no_loads : 0;
  if (ep) {
    if (ep->act < US_ACT_NONE || ep->act > US_ACT_SIGMOID_GRAD) return US_ERR_INVALID_ARG;
    // the activation's class (forward: value from the accumulator; gradient: slope from the stored pre-activation)
    // and which function of the table it is
    const bool grad = ep->act != US_ACT_NONE && (ep->act % 2) == 0;
    p.act = ep->act == US_ACT_NONE ? US_ACT_NONE : grad ? US_ACT_GELU_GRAD : US_ACT_GELU;
    p.fn = ep->act <= US_ACT_GELU_GRAD ? US_FN_GELU : ep->act <= US_ACT_RELU_GRAD ? US_FN_RELU
         : ep->act <= US_ACT_TANH_GRAD ? US_FN_TANH : US_FN_SIGMOID;
    p.act_in = ep->act_in_scale; p.act_out = ep->act_out_scale;
    if (grad && !ep->aux.ptr) return US_ERR_INVALID_ARG;
    if (ep->act != US_ACT_NONE && ep->aux.ptr) {
      if (ep->aux.rows != M || ep->aux.cols != N || ep->aux.ld < N) return US_ERR_INVALID_ARG;
      if (ep->aux.dtype != US_BF16 && ep->aux.dtype != US_F16) return US_ERR_UNSUPPORTED;
      if (!aligned16(&ep->aux)) return US_ERR_ALIGNMENT;
      p.aux = ep->aux.ptr; p.aux_dt = ep->aux.dtype; p.aux_ld = ep->aux.ld;
    }
    if (ep->skip.ptr) {
      if (ep->skip.rows != M || ep->skip.cols != N || ep->skip.ld < N) return US_ERR_INVALID_ARG;
      if (ep->skip.dtype != US_F32 && ep->skip.dtype != US_BF16 && ep->skip.dtype != US_F16) return US_ERR_UNSUPPORTED;
      if (!aligned16(&ep->skip)) return US_ERR_ALIGNMENT;
      p.skip = ep->skip.ptr; p.skip_dt = ep->skip.dtype; p.skip_ld = ep->skip.ld;
      p.skip_coef = ep->skip_coef; p.out_coef = ep->out_coef;
    }
  }
  if (!ws || ws_bytes < us_workspace_bytes()) return US_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % 16) return US_ERR_ALIGNMENT;
  p.status = static_cast<unsigned int*>(ws);

  EpiMats em{out, p.aux ? &ep->aux : nullptr, p.skip ? &ep->skip : nullptr};
  // The specialised epilogues cover the combinations of the FFN path; anything else (an activation
  // together with a skip tensor) takes the general direct-access epilogue.
  int epi = kEpiLegacy;
  if (p.act == US_ACT_NONE && !p.skip) epi = kEpiPlain;
  else if (p.act == US_ACT_NONE) epi = kEpiSkip;
  else if (p.act == US_ACT_GELU && !p.skip) epi = kEpiGelu;
  else if (p.act == US_ACT_GELU_GRAD && !p.skip) epi = kEpiGeluGrad;
  BatchDesc bd;
  if (batch) {
    if (ep) return US_ERR_UNSUPPORTED;                  // batched problems take no fused epilogue
    const us_mat* ms[3] = {A, B, out};
    const int64_t* strides[3] = {batch->a_stride, batch->b_stride, batch->out_stride};
    int64_t* dst[3] = {bd.a, bd.b, bd.out};
    if (batch->count[0] < 1 || batch->count[1] < 1 || batch->count[0] * batch->count[1] > (1 << 20)) return US_ERR_INVALID_ARG;
    bd.nb0 = batch->count[0]; bd.nb1 = batch->count[1];
    for (int i = 0; i < 3; ++i) {
      const int es = dtype_size(ms[i]->dtype);
      for (int d = 0; d < 2; ++d) {
        int64_t st = strides[i][d];
        if (batch->count[d] == 1) st = ms[i]->rows * ms[i]->ld;    // unused dimension: any valid pitch
        if (st <= 0) return US_ERR_INVALID_ARG;
        if ((st * es) % 16) return US_ERR_ALIGNMENT;
        dst[i][d] = st;
      }
    }
    if ((long long)((M + 127) / 128) * ((N + 127) / 128) * bd.nb0 * bd.nb1 > 0x7fffffffll) return US_ERR_INVALID_ARG;
  }
  if (validate_only) return US_OK;                     // every host check has passed; nothing has been launched
  const bool a_mn = (op == kBwdW), b_mn = (op != kBwdX);
  const int a_fmt = f8 ? (A->dtype == US_E5M2) : (A->dtype == US_BF16);
  const int b_fmt = f8 ? (B->dtype == US_E5M2) : (B->dtype == US_BF16);
  p.idesc = make_idesc(a_fmt, b_fmt, a_mn, b_mn, kBM, 256);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (f8) {
    switch (op) {
      case kFwd:  return launch_gemm<1, false, true>(A, B, p, em, epi, bd, st);
      case kBwdX: return launch_gemm<1, false, false>(A, B, p, em, epi, bd, st);
      default:    return launch_gemm<1, true, true>(A, B, p, em, epi, bd, st);
    }
  }
  switch (op) {
    case kFwd:  return launch_gemm<2, false, true>(A, B, p, em, epi, bd, st);
    case kBwdX: return launch_gemm<2, false, false>(A, B, p, em, epi, bd, st);
    default:    return launch_gemm<2, true, true>(A, B, p, em, epi, bd, st);
  }
}

}  // namespace us

extern "C" us_status us_linear_fwd(const us_mat* X, const us_mat* W, float alpha, const us_epilogue* ep,
                                   const us_mat* Y, void* ws, size_t ws_bytes, void* stream) {
  return us::linear(us::kFwd, X, W, alpha, ep, Y, ws, ws_bytes, stream);
}
extern "C" us_status us_linear_bwd_x(const us_mat* G, const us_mat* W, float beta_x, const us_epilogue* ep,
                                     const us_mat* dX, void* ws, size_t ws_bytes, void* stream) {
  return us::linear(us::kBwdX, G, W, beta_x, ep, dX, ws, ws_bytes, stream);
}
extern "C" us_status us_linear_bwd_w(const us_mat* X, const us_mat* G, float beta_w, const us_epilogue* ep,
                                     const us_mat* dW, void* ws, size_t ws_bytes, void* stream) {
  return us::linear(us::kBwdW, X, G, beta_w, ep, dW, ws, ws_bytes, stream);
}

extern "C" us_status us_linear_fwd_batched(const us_mat* X, const us_mat* W, float alpha, const us_mat* Y,
                                           const us_batch* batch, void* ws, size_t ws_bytes, void* stream) {
  if (!batch) return US_ERR_INVALID_ARG;
  return us::linear(us::kFwd, X, W, alpha, nullptr, Y, ws, ws_bytes, stream, batch);
}
extern "C" us_status us_linear_bwd_x_batched(const us_mat* G, const us_mat* W, float beta_x, const us_mat* dX,
                                             const us_batch* batch, void* ws, size_t ws_bytes, void* stream) {
  if (!batch) return US_ERR_INVALID_ARG;
  return us::linear(us::kBwdX, G, W, beta_x, nullptr, dX, ws, ws_bytes, stream, batch);
}
extern "C" us_status us_linear_bwd_w_batched(const us_mat* X, const us_mat* G, float beta_w, const us_mat* dW,
                                             const us_batch* batch, void* ws, size_t ws_bytes, void* stream) {
  if (!batch) return US_ERR_INVALID_ARG;
  return us::linear(us::kBwdW, X, G, beta_w, nullptr, dW, ws, ws_bytes, stream, batch);
}

extern "C" us_status us_linear_fwd_check(const us_mat* X, const us_mat* W, const us_epilogue* ep, const us_mat* Y,
                                         const void* ws, size_t ws_bytes) {
  return us::linear(us::kFwd, X, W, 1.f, ep, Y, const_cast<void*>(ws), ws_bytes, nullptr, nullptr, nullptr, true);
}

extern "C" us_status us_test_linear_fwd_starved(const us_mat* X, const us_mat* W, float alpha, const us_mat* Y, void* ws,
                                                size_t ws_bytes, unsigned int wait_limit, void* stream) {
  if (wait_limit < 1 || wait_limit > (1u << 16)) return US_ERR_INVALID_ARG;
  const us::WaitTest wt = {wait_limit, 1};
  return us::linear(us::kFwd, X, W, alpha, nullptr, Y, ws, ws_bytes, stream, nullptr, &wt);
}

extern "C" size_t us_workspace_bytes(void) { return 256; }

extern "C" us_status us_workspace_status(const void* ws, void* stream) {
  if (!ws) return US_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned int word = 0;
  if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return US_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return US_ERR_CUDA;
  return word == 0 ? US_OK : US_ERR_TIMEOUT;
}
