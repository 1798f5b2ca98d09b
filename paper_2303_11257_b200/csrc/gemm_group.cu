// us_linear_group: several independent linear ops in one launch (host side: checks, work list, launch).
#include <cuda.h>

#include <algorithm>
#include <vector>

#include "gemm_group.cuh"
#include "host.h"

namespace us {
namespace {

// Row-major [rows x cols] matrix of es-byte elements, boxes of box_rows rows x 128 bytes, 128-byte swizzle, zero fill.
bool make_tmap(CUtensorMap* tm, const us_mat* m, int es, int box_rows) {
  host::EncodeTiledFn fn = host::encode_tiled_fn();
  if (!fn) return false;
  const CUtensorMapDataType type = es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : es == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32;
  cuuint64_t dims[2] = {(cuuint64_t)m->cols, (cuuint64_t)m->rows};
  cuuint64_t strides[1] = {(cuuint64_t)m->ld * es};
  cuuint32_t box[2] = {(cuuint32_t)(128 / es), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, type, 2, m->ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const us_mat* m) {
  return reinterpret_cast<uintptr_t>(m->ptr) % 16 == 0 && (m->ld * dtype_size(m->dtype)) % 16 == 0;
}
bool valid_mat(const us_mat* m) {
  return m && m->ptr && m->rows >= 1 && m->cols >= 1 && m->ld >= m->cols && m->rows < (1ll << 31) && m->cols < (1ll << 31) &&
         m->dtype >= US_F32 && m->dtype <= US_E5M2;
}
bool is_fp8(int dt) { return dt == US_E4M3 || dt == US_E5M2; }

struct Shape { int64_t M, N, K; };

// Host checks of one call of the group; US_ERR_UNSUPPORTED for a valid call this launch form does not cover.
us_status check_call(const us_linear_call* c, Shape* sh) {
  if (c->op < US_OP_FWD || c->op > US_OP_BWD_W) return US_ERR_INVALID_ARG;
  if (!valid_mat(&c->a) || !valid_mat(&c->b) || !valid_mat(&c->out)) return US_ERR_INVALID_ARG;
  int64_t M, N, K;
  bool ok;
  switch (c->op) {
    case US_OP_FWD:   M = c->a.rows; K = c->a.cols; N = c->b.cols; ok = c->b.rows == K; break;
    case US_OP_BWD_X: M = c->a.rows; K = c->a.cols; N = c->b.rows; ok = c->b.cols == K; break;
    default:          M = c->a.cols; K = c->a.rows; N = c->b.cols; ok = c->b.rows == K; break;
  }
  if (!ok || c->out.rows != M || c->out.cols != N) return US_ERR_INVALID_ARG;
  if (!aligned16(&c->a) || !aligned16(&c->b) || !aligned16(&c->out)) return US_ERR_ALIGNMENT;
  if (!(is_fp8(c->a.dtype) && is_fp8(c->b.dtype))) {
    const bool h16 = (c->a.dtype == US_BF16 || c->a.dtype == US_F16) && c->a.dtype == c->b.dtype;
    return h16 ? US_ERR_UNSUPPORTED : US_ERR_UNSUPPORTED;
  }
  if (c->ep.act != US_ACT_NONE) return c->ep.act < US_ACT_NONE || c->ep.act > US_ACT_SIGMOID_GRAD ? US_ERR_INVALID_ARG : US_ERR_UNSUPPORTED;
  if (c->ep.skip.ptr) {
    const us_mat* s = &c->ep.skip;
    if (s->rows != M || s->cols != N || s->ld < N) return US_ERR_INVALID_ARG;
    if (s->dtype != US_F32 && s->dtype != US_BF16 && s->dtype != US_F16) return US_ERR_UNSUPPORTED;
    if (!aligned16(s)) return US_ERR_ALIGNMENT;
  }
  if (M <= 128 || N <= 128) return US_ERR_UNSUPPORTED;       // tiles of 256 x 256 only
  if (M > 4095ll * 256 || N > 4095ll * 256) return US_ERR_UNSUPPORTED;
  sh->M = M; sh->N = N; sh->K = K;
  return US_OK;
}

struct Item { int prob, tm, tn; int64_t kb; };

}  // namespace
}  // namespace us

using namespace us;

extern "C" us_status us_linear_group(int count, const us_linear_call* calls, void* ws, size_t ws_bytes, void* stream) {
  if (count < 1 || count > kGroupMaxProblems || !calls) return count >= 1 && calls ? US_ERR_UNSUPPORTED : US_ERR_INVALID_ARG;
  if (!ws || ws_bytes < us_workspace_bytes()) return US_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % 16) return US_ERR_ALIGNMENT;
  static_assert(sizeof(GroupParams) < 32000, "kernel parameter limit");
  GroupParams g{};
  std::vector<Item> items;
  for (int i = 0; i < count; ++i) {
    Shape sh;
    us_status s = check_call(&calls[i], &sh);
    if (s != US_OK) return s;
    GroupProblem& P = g.prob[i];
    const us_linear_call& c = calls[i];
    P.M = (int)sh.M; P.N = (int)sh.N; P.K = (int)sh.K;
    P.a_mn = c.op == US_OP_BWD_W; P.b_mn = c.op != US_OP_BWD_X;
    P.idesc = make_idesc(c.a.dtype == US_E5M2, c.b.dtype == US_E5M2, P.a_mn != 0, P.b_mn != 0, 256, 256);
    P.scale = c.scale;
    P.out_dt = c.out.dtype;
    P.has_skip = c.ep.skip.ptr != nullptr;
    P.skip_dt = P.has_skip ? c.ep.skip.dtype : US_F32;
    P.skip_coef = P.has_skip ? c.ep.skip_coef : 0.f;
    P.out_coef = P.has_skip ? c.ep.out_coef : 1.f;
    // operand tiles are 128-row x 128-byte boxes in either layout (FP8: 128 elements of K, or of M / N, per row)
    if (!make_tmap(&P.ta, &c.a, 1, 128) || !make_tmap(&P.tb, &c.b, 1, 128)) return US_ERR_CUDA;
    if (!make_tmap(&P.tout, &c.out, dtype_size(c.out.dtype), 32)) return US_ERR_CUDA;
    P.tskip = P.tout;
    if (P.has_skip && !make_tmap(&P.tskip, &c.ep.skip, dtype_size(c.ep.skip.dtype), 32)) return US_ERR_CUDA;
    const int tiles_m = (int)((sh.M + 255) / 256), tiles_n = (int)((sh.N + 255) / 256);
    const int64_t kb = (sh.K + 127) / 128;
    // column-major over the tiles of a problem: neighbours in the list share a B panel
    for (int tn = 0; tn < tiles_n; ++tn)
      for (int tm = 0; tm < tiles_m; ++tm) items.push_back({i, tm, tn, kb});
  }
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  int pairs = sms / 2;
  if (pairs > kGroupMaxPairs) pairs = kGroupMaxPairs;
  if ((int)items.size() < pairs) pairs = (int)items.size();
  // Longest first, each tile to the pair with the least work so far (ties: lowest pair), in a fixed order: the same
  // arguments always give the same work list, and a tile's result never depends on it anyway (one pair, one accumulator).
  std::stable_sort(items.begin(), items.end(), [](const Item& a, const Item& b) { return a.kb > b.kb; });
  std::vector<int64_t> load(pairs, 0);
  std::vector<int> filled(pairs, 0);
  for (int i = 0; i < kGroupMaxRounds * kGroupMaxPairs; ++i) g.table[i] = -1;
  int rounds = 0;
  for (const Item& it : items) {
    int best = 0;
    for (int p = 1; p < pairs; ++p)
      if (load[p] < load[best]) best = p;
    if (filled[best] >= kGroupMaxRounds) return US_ERR_UNSUPPORTED;      // too many tiles per pair for the work list
    g.table[filled[best] * pairs + best] = (it.prob << 24) | (it.tm << 12) | it.tn;
    load[best] += it.kb + 4;                                            // a tile costs its K blocks plus a change-over
    rounds = std::max(rounds, ++filled[best]);
  }
  g.count = count; g.rounds = rounds; g.pairs = pairs;
  g.status = static_cast<unsigned int*>(ws);
  g.wait_limit = kWaitLimit;

  constexpr int smem = GroupSmem::kTotal;
  if (cudaFuncSetAttribute(gemm_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return US_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(gemm_threads(kGroupEW));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_group_kernel, g) == cudaSuccess ? US_OK : US_ERR_CUDA;
}
