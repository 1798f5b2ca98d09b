// Host side of the linear ops: argument checks, TMA tensor maps, kernel selection and launch.
#include <cuda.h>

#include "gemm_kernel.cuh"
#include "host.h"

namespace us {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// Tensor map over a row-major matrix [rows x cols] of ES-byte elements with a 128-byte-wide,
// 128-byte-swizzled box of `box_rows` rows.  Out-of-range parts of a box read as zero.
static bool make_tmap(CUtensorMap* tm, const us_mat* m, int es, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const CUtensorMapDataType type = es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : es == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32;
  cuuint64_t dims[2] = {(cuuint64_t)m->cols, (cuuint64_t)m->rows};
  cuuint64_t strides[1] = {(cuuint64_t)m->ld * es};
  cuuint32_t box[2] = {(cuuint32_t)(128 / es), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, type, 2, m->ptr, dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The matrices the epilogue reaches through TMA (aux / skip NULL when unused).
struct EpiMats {
  const us_mat* out;
  const us_mat* aux;
  const us_mat* skip;
};

template <int ES, bool A_MN, bool B_MN, int BN, int CG>
static us_status launch(const us_mat* A, const us_mat* B, const GemmParams& p, const EpiMats& em, cudaStream_t stream) {
  constexpr int kBK = kStageKBytes / ES;
  CUtensorMap ta, tb, t_out, t_aux, t_skip;
  if (!make_tmap(&ta, A, ES, A_MN ? kBK : kBM)) return US_ERR_CUDA;
  if (!make_tmap(&tb, B, ES, B_MN ? kBK : BN / CG)) return US_ERR_CUDA;
  // epilogue boxes: 32 rows x 128 bytes; unused maps alias the output's so that every parameter is valid
  if (!make_tmap(&t_out, em.out, dtype_size(em.out->dtype), 32)) return US_ERR_CUDA;
  t_aux = t_out; t_skip = t_out;
  if (p.staged && em.aux && !make_tmap(&t_aux, em.aux, dtype_size(em.aux->dtype), 32)) return US_ERR_CUDA;
  if (p.staged && em.skip && !make_tmap(&t_skip, em.skip, dtype_size(em.skip->dtype), 32)) return US_ERR_CUDA;
  auto kern = gemm_kernel<ES, A_MN, B_MN, BN, CG>;
  constexpr int smem = GemmSmem<BN, CG>::kTotal;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return US_ERR_CUDA;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const int tiles = p.tiles_m * p.tiles_n;
  const int groups = sms / CG;                        // one CTA per SM; pairs share a TPC
  const int grid = CG * (tiles < groups ? tiles : groups);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, ta, tb, t_out, t_aux, t_skip, p) == cudaSuccess ? US_OK : US_ERR_CUDA;
}

template <int ES, bool A_MN, bool B_MN>
static us_status pick_tile(const us_mat* A, const us_mat* B, GemmParams& p, const EpiMats& em, cudaStream_t stream) {
  const int bn = p.N <= 128 ? 128 : 256;
  const int cg = (bn == 256 && p.M > kBM) ? 2 : 1;    // CTA pairs whenever a 256 x 256 tile is not mostly empty
  p.tiles_m = (p.M + kBM * cg - 1) / (kBM * cg);
  p.tiles_n = (p.N + bn - 1) / bn;
  p.idesc = (p.idesc & ~((0x3fu << 17) | (0x1fu << 24))) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)((kBM * cg) >> 4) << 24);
  if (bn == 128) return launch<ES, A_MN, B_MN, 128, 1>(A, B, p, em, stream);
  if (cg == 1) return launch<ES, A_MN, B_MN, 256, 1>(A, B, p, em, stream);
  return launch<ES, A_MN, B_MN, 256, 2>(A, B, p, em, stream);
}

static bool aligned16(const us_mat* m) {
  return reinterpret_cast<uintptr_t>(m->ptr) % 16 == 0 && (m->ld * dtype_size(m->dtype)) % 16 == 0;
}
static bool valid_mat(const us_mat* m) {
  return m && m->ptr && m->rows >= 1 && m->cols >= 1 && m->ld >= m->cols && m->rows < (1ll << 31) &&
         m->cols < (1ll << 31) && m->dtype >= US_F32 && m->dtype <= US_E5M2;
}
static bool is_fp8(int dt) { return dt == US_E4M3 || dt == US_E5M2; }

enum Op { kFwd, kBwdX, kBwdW };

// A, B: the two operands in call order; out [M x N].
static us_status linear(Op op, const us_mat* A, const us_mat* B, float scale, const us_epilogue* ep, const us_mat* out,
                        void* ws, size_t ws_bytes, void* stream) {
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
  if (ep) {
    if (ep->act < US_ACT_NONE || ep->act > US_ACT_GELU_GRAD) return US_ERR_INVALID_ARG;
    p.act = ep->act; p.act_in = ep->act_in_scale; p.act_out = ep->act_out_scale;
    if (ep->act == US_ACT_GELU_GRAD && !ep->aux.ptr) return US_ERR_INVALID_ARG;
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
  // One input box and one output box per epilogue warp: combinations that need two inputs, or an
  // input next to the kept pre-activation, take the direct-access epilogue instead.
  const bool two_inputs = p.act == US_ACT_GELU_GRAD && p.skip;
  const bool aux_and_skip = p.act == US_ACT_GELU && p.aux && p.skip;
  p.staged = (two_inputs || aux_and_skip) ? 0 : 1;
  const bool a_mn = (op == kBwdW), b_mn = (op != kBwdX);
  const int a_fmt = f8 ? (A->dtype == US_E5M2) : (A->dtype == US_BF16);
  const int b_fmt = f8 ? (B->dtype == US_E5M2) : (B->dtype == US_BF16);
  p.idesc = make_idesc(a_fmt, b_fmt, a_mn, b_mn, kBM, 256);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (f8) {
    switch (op) {
      case kFwd:  return pick_tile<1, false, true>(A, B, p, em, st);
      case kBwdX: return pick_tile<1, false, false>(A, B, p, em, st);
      default:    return pick_tile<1, true, true>(A, B, p, em, st);
    }
  }
  switch (op) {
    case kFwd:  return pick_tile<2, false, true>(A, B, p, em, st);
    case kBwdX: return pick_tile<2, false, false>(A, B, p, em, st);
    default:    return pick_tile<2, true, true>(A, B, p, em, st);
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

extern "C" size_t us_workspace_bytes(void) { return 256; }

extern "C" us_status us_workspace_status(const void* ws, void* stream) {
  if (!ws) return US_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned int word = 0;
  if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return US_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return US_ERR_CUDA;
  return word == 0 ? US_OK : US_ERR_TIMEOUT;
}
