// Kernel instantiations of the unit-scaled GEMM for one (operand width, A layout, B layout)
// combination, selected by the macros US_INST_ES, US_INST_AMN, US_INST_BMN.  The build compiles
// this file once per combination, in parallel.
#include <cuda.h>

#include "gemm_kernel.cuh"
#include "gemm_launch.h"
#include "host.h"

#ifndef US_INST_ES
#error "compile with -DUS_INST_ES=<1|2> -DUS_INST_AMN=<0|1> -DUS_INST_BMN=<0|1>"
#endif

namespace us {
namespace {

// Tensor map over a row-major matrix [rows x cols] of ES-byte elements with a box of `box_rows` rows
// and `box_bytes` (128, or 64) bytes per row, swizzled with the pattern of that width.  Out-of-range parts of a box read as zero.
static bool make_tmap(CUtensorMap* tm, const us_mat* m, int es, int box_rows, int box_bytes = 128,
                      const BatchDesc* bd = nullptr, const int64_t* bstride = nullptr) {
  host::EncodeTiledFn fn = host::encode_tiled_fn();
  if (!fn) return false;
  const CUtensorMapDataType type = es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : es == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32;
  const CUtensorMapSwizzle swz = box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  CUresult r;
  if (!bd) {
    cuuint64_t dims[2] = {(cuuint64_t)m->cols, (cuuint64_t)m->rows};
    cuuint64_t strides[1] = {(cuuint64_t)m->ld * es};
    cuuint32_t box[2] = {(cuuint32_t)(box_bytes / es), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    r = fn(tm, type, 2, m->ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    // rank 4: (column, row, inner batch index, outer batch index); a box never spans problems
    cuuint64_t dims[4] = {(cuuint64_t)m->cols, (cuuint64_t)m->rows, (cuuint64_t)bd->nb1, (cuuint64_t)bd->nb0};
    cuuint64_t strides[3] = {(cuuint64_t)m->ld * es, (cuuint64_t)bstride[1] * es, (cuuint64_t)bstride[0] * es};
    cuuint32_t box[4] = {(cuuint32_t)(box_bytes / es), (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    r = fn(tm, type, 4, m->ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS;
}

template <int ES, bool A_MN, bool B_MN, int BN, int CG, int EPI, int EW, bool BATCHED = false>
static us_status launch(const us_mat* A, const us_mat* B, const GemmParams& p, const EpiMats& em, cudaStream_t stream,
                        const BatchDesc* bd = nullptr) {
  constexpr int kBK = kStageKBytes / ES;
  CUtensorMap ta, tb, t_out, t_aux, t_skip;
  const BatchDesc* b4 = BATCHED ? bd : nullptr;
  if (!make_tmap(&ta, A, ES, A_MN ? kBK : kBM, 128, b4, b4 ? bd->a : nullptr)) return US_ERR_CUDA;
  if (!make_tmap(&tb, B, ES, B_MN ? kBK : BN / CG, 128, b4, b4 ? bd->b : nullptr)) return US_ERR_CUDA;
  // epilogue boxes: 32 rows x 128 bytes; unused maps alias the output's so that every parameter is valid
  if (!make_tmap(&t_out, em.out, dtype_size(em.out->dtype), 32, EW == 16 ? 64 : 128, b4, b4 ? bd->out : nullptr)) return US_ERR_CUDA;
  t_aux = t_out; t_skip = t_out;
  // the 16-warp GELU-gradient epilogue reads the stored pre-activation as 32-row x 64-byte boxes (one per 32-column slice)
  if (EPI != kEpiLegacy && em.aux && !make_tmap(&t_aux, em.aux, dtype_size(em.aux->dtype), 32, (EW == 16 && EPI == kEpiGeluGrad) ? 64 : 128)) return US_ERR_CUDA;
  if (EPI != kEpiLegacy && em.skip && !make_tmap(&t_skip, em.skip, dtype_size(em.skip->dtype), 32)) return US_ERR_CUDA;
  auto kern = gemm_kernel<ES, A_MN, B_MN, BN, CG, EPI, EW, BATCHED>;
  constexpr int smem = GemmSmem<BN, CG, EW>::kTotal;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return US_ERR_CUDA;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const int tiles = p.tiles_m * p.tiles_n * p.nb0 * p.nb1;
  const int groups = sms / CG;                        // one CTA per SM; pairs share a TPC
  const int grid = CG * (tiles < groups ? tiles : groups);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(gemm_threads(EW));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, ta, tb, t_out, t_aux, t_skip, p) == cudaSuccess ? US_OK : US_ERR_CUDA;
}

template <int ES, bool A_MN, bool B_MN, int BN, int CG>
static us_status pick_epilogue(const us_mat* A, const us_mat* B, const GemmParams& p, const EpiMats& em, int epi,
                               const BatchDesc& bd, cudaStream_t stream) {
  if (bd.batched()) {                                  // batched problems: plain epilogue only (checked by the caller)
    return launch<ES, A_MN, B_MN, BN, CG, kEpiPlain, 8, true>(A, B, p, em, stream, &bd);
  }
  // The GELU epilogues with an FP8 output (the FFN's forward and backward hidden layer) are ALU
  // bound with eight epilogue warps; they run with sixteen.
  const bool fp8_out = (em.out->dtype == US_E4M3 || em.out->dtype == US_E5M2) && p.fn == US_FN_GELU;   // the 16-warp epilogue is the GELU pair's
  switch (epi) {
    case kEpiPlain:    return launch<ES, A_MN, B_MN, BN, CG, kEpiPlain, 8>(A, B, p, em, stream);
    case kEpiGelu:     return fp8_out ? launch<ES, A_MN, B_MN, BN, CG, kEpiGelu, 16>(A, B, p, em, stream)
                                      : launch<ES, A_MN, B_MN, BN, CG, kEpiGelu, 8>(A, B, p, em, stream);
    case kEpiGeluGrad: return fp8_out ? launch<ES, A_MN, B_MN, BN, CG, kEpiGeluGrad, 16>(A, B, p, em, stream)
                                      : launch<ES, A_MN, B_MN, BN, CG, kEpiGeluGrad, 8>(A, B, p, em, stream);
    case kEpiSkip:     return launch<ES, A_MN, B_MN, BN, CG, kEpiSkip, 8>(A, B, p, em, stream);
    default:           return launch<ES, A_MN, B_MN, BN, CG, kEpiLegacy, 8>(A, B, p, em, stream);
  }
}

}  // namespace

template <int ES, bool A_MN, bool B_MN>
us_status launch_gemm(const us_mat* A, const us_mat* B, GemmParams& p, const EpiMats& em, int epi, const BatchDesc& bd,
                      cudaStream_t stream) {
  // CTA pairs with 256 x 256 tiles whenever such a tile is not mostly empty and there are enough of them to occupy at
  // least half of the machine's CTA pairs; 128 x 128 tiles otherwise (a 1024 x 1024 output is 16 pair tiles on 74
  // pairs, but 64 single-CTA tiles).
  const int sms = host::sm_count();
  const long long pair_tiles = (long long)((p.M + 2 * kBM - 1) / (2 * kBM)) * ((p.N + 255) / 256) * bd.nb0 * bd.nb1;
  const bool pair = p.N > 128 && p.M > kBM && (sms <= 0 || 4 * pair_tiles >= sms);
  const int bn = pair ? 256 : 128, cg = pair ? 2 : 1;
  p.tiles_m = (p.M + kBM * cg - 1) / (kBM * cg);
  p.tiles_n = (p.N + bn - 1) / bn;
  p.nb0 = (int)bd.nb0; p.nb1 = (int)bd.nb1;
  // A (M x K operand) is re-read by every column of tiles: keep the plain order while it fits well
  // inside the 126 MB L2, switch to bands of 8 tile rows beyond that.
  p.band_m = ((long long)p.M * p.K * ES <= (80ll << 20)) ? p.tiles_m : 8;
  p.full_bands = p.tiles_m / p.band_m;
  p.d_problem = make_fast_div(p.tiles_m * p.tiles_n);
  p.d_band = make_fast_div(p.band_m * p.tiles_n);
  p.d_rows = make_fast_div(p.band_m);
  p.d_rows_last = make_fast_div(p.tiles_m % p.band_m ? p.tiles_m % p.band_m : 1);
  p.d_nb1 = make_fast_div(p.nb1);
  p.idesc = (p.idesc & ~((0x3fu << 17) | (0x1fu << 24))) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)((kBM * cg) >> 4) << 24);
  return pair ? pick_epilogue<ES, A_MN, B_MN, 256, 2>(A, B, p, em, epi, bd, stream)
              : pick_epilogue<ES, A_MN, B_MN, 128, 1>(A, B, p, em, epi, bd, stream);
}

template us_status launch_gemm<US_INST_ES, (US_INST_AMN != 0), (US_INST_BMN != 0)>(const us_mat*, const us_mat*, GemmParams&,
                                                                                 const EpiMats&, int, const BatchDesc&, cudaStream_t);

}  // namespace us
