// us_ffn_hidden: the two GEMMs that end in the hidden layer of the FFN block as ONE launch.
//
//   H  = alpha  * X W1                                   (first forward GEMM,          K = d_model)
//   A  = round_fp8(act_out * gelu(act_in * H))
//   dA = beta_x * G W2^T                                 (second layer's input gradient, K = d_model)
//   dH = round_fp8(grad_out * act_in * gelu'(act_in * round16(H)) * dA)
//
// Both GEMMs produce a [tokens x d_ff] matrix and the GELU gradient needs, element for element, the
// pre-activation H the forward GEMM has just produced.  Launched separately, H travels to memory in
// 16 bits and back (2 x 2 bytes per element of the largest tensor of the block), and both kernels'
// stores compete with their operand loads for the SM's memory path.  Here a CTA pair computes, for
// one 256 x 256 output tile, first X W1 into accumulator 0 and then G W2^T into accumulator 1 of
// tensor memory.  The sixteen epilogue warps turn accumulator 0 into A (stored as FP8) while the MMAs
// of accumulator 1 run, keep H -- rounded to the 16-bit format the unfused path stores it in -- in
// registers, and turn accumulator 1 into dH while the next tile's X W1 runs: the two
// accumulators alternate exactly as two consecutive tiles of gemm_kernel do, and H never leaves the SM
// (unless the caller asks for a copy).  Results are bit-identical to us_linear_fwd + GELU epilogue
// followed by us_linear_bwd_x + GELU-gradient epilogue.
#include <cuda.h>

#include "gemm_kernel.cuh"
#include "host.h"

namespace us {
namespace {

constexpr int kHidEW = 16;
// Shared-memory plan: 32 KB operand stages (this CTA's 128 rows of A and 128 rows of B, 128 bytes of K each) and one
// 32-row x 64-byte output box per epilogue warp.  The kept pre-activation lives in registers, which leaves room for
// six stages.
struct HidSmem {
  static constexpr int kABytes = kBM * kStageKBytes;
  static constexpr int kBBytes = 128 * kStageKBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiWarpBytes = 2048;
  static constexpr int kEpiBytes = kHidEW * kEpiWarpBytes;
  static constexpr int kStages = (229376 - kEpiBytes) / kStageBytes;
  static constexpr int kBarrierBytes = 512;
  static constexpr int kTotal = kStages * kStageBytes + kEpiBytes + kBarrierBytes + 1024;   // + alignment slack
};

struct HiddenParams {
  int M, N, K1, K2;                 // outputs are [M x N]; contraction lengths of X W1 and of G W2^T
  int tiles_m, tiles_n;
  FastDiv d_tiles_m;
  uint32_t idesc1, idesc2;
  float scale1, scale2;             // alpha, beta_x
  float act_in, act_out, grad_out;  // s_in, alpha_g, beta_g
  uint8_t* h_ptr; long long h_ld;   // optional copy of the rounded pre-activation (NULL: none); ld in elements
  unsigned int* status;
  uint32_t wait_limit;
  int no_loads;                     // test hook: no operand loads are issued, so that the waits run out
};

template <bool A_E5, bool D_E5, bool H_BF16>
__global__ void __launch_bounds__(gemm_threads(kHidEW), 1)
ffn_hidden_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w1,
                  const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_w2,
                  const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_dh,
                  const HiddenParams p) {
  using S = HidSmem;
  constexpr int BN = 256, kBK = 128;
  constexpr uint32_t kChunkBytes = kBK * 128;       // an MN-major operand tile: 128 rows of K x 128 bytes
  constexpr uint32_t kTmemCols = 2 * BN;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
  const uint32_t epi_base = smem_base + S::kStages * S::kStageBytes;
  const uint32_t bars = epi_base + S::kEpiBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S::kStages + s); };
  auto acc_full_bar = [&](int a) { return bars + 8u * (2 * S::kStages + a); };
  auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * S::kStages + 2 + a); };
  const uint32_t drained_bar = bars + 8u * (2 * S::kStages + 4);
  static_assert(8 * (2 * S::kStages + 5) + 8 <= S::kBarrierBytes, "barrier area too small");
  uint8_t* tail = smem_gen + S::kStages * S::kStageBytes + S::kEpiBytes + 8 * (2 * S::kStages + 5);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)ptx::cluster_ctarank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int kb1 = (p.K1 + kBK - 1) / kBK, kb2 = (p.K2 + kBK - 1) / kBK;
  // column-major over the tiles: pairs that run side by side share a panel of W1 and of W2
  auto tile_mn2 = [&](int tile, int& tm, int& tn) { tn = p.d_tiles_m.div(tile); tm = tile - tn * p.tiles_m; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full_bar(a), 1); ptx::mbar_init(acc_empty_bar(a), 2 * kHidEW); }
    ptx::mbar_init(drained_bar, 1);
    *abort_flag = 0;
    ptx::mbar_init_fence();
    ptx::prefetch_tensormap(&tm_x);
    ptx::prefetch_tensormap(&tm_w1);
    ptx::prefetch_tensormap(&tm_g);
    ptx::prefetch_tensormap(&tm_w2);
  }
  if (warp == 1) { ptx::tmem_alloc_pair(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols); ptx::tmem_relinquish_pair(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs of the pair)
    if (lane == 0) {
      uint32_t issued = 0;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; ok && !p.no_loads && tile < num_tiles; tile += num_pairs) {
        int tm, tn;
        tile_mn2(tile, tm, tn);
        const int m0 = tm * 256 + rank * 128, n0 = tn * 256 + rank * 128;
        for (int sub = 0; ok && sub < 2; ++sub) {
          const int num_kb = sub ? kb2 : kb1;
          for (int kb = 0; kb < num_kb; ++kb) {
            ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, p.wait_limit);
            if (!ok) break;
            const uint32_t a_dst = smem_base + stage * S::kStageBytes, b_dst = a_dst + S::kABytes;
            const int k0 = kb * kBK;
            const uint32_t fb = ptx::in_even_cta(full_bar(stage));
            if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), 2 * S::kStageBytes);
            if (sub == 0) {
              ptx::tma_load_2d_pair(a_dst, &tm_x, fb, k0, m0);      // X  [M x K1], K-major
              ptx::tma_load_2d_pair(b_dst, &tm_w1, fb, n0, k0);     // W1 [K1 x N], N-major
            } else {
              ptx::tma_load_2d_pair(a_dst, &tm_g, fb, k0, m0);      // G  [M x K2], K-major
              ptx::tma_load_2d_pair(b_dst, &tm_w2, fb, k0, n0);     // W2 [N x K2], K-major
            }
            ++issued;
            if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (*abort_flag && rank == 0) {
        // Let copies that are still in flight land before the CTA gives up its shared memory.
        const uint32_t n = issued < (uint32_t)S::kStages ? issued : (uint32_t)S::kStages;
        for (uint32_t i = 0; i < n; ++i) {
          if (stage == 0) { stage = S::kStages; phase ^= 1u; }
          --stage;
          for (uint32_t it = 0; it < p.wait_limit && !ptx::mbar_try_wait(full_bar(stage), phase); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0, local = 0;
      bool ok = true;
      constexpr uint32_t kStageStep = S::kStageBytes >> 4;
      const uint64_t a_desc = ptx::smem_desc_sw128(smem_base, 16, 1024);                              // K-major
      const uint64_t b_desc_mn = ptx::smem_desc_sw128(smem_base + S::kABytes, kChunkBytes, 1024);     // W1: N-major
      const uint64_t b_desc_k = ptx::smem_desc_sw128(smem_base + S::kABytes, 16, 1024);               // W2: K-major
      const uint32_t a_hi = (uint32_t)(a_desc >> 32), a_lo0 = (uint32_t)a_desc;
      for (int tile = pair; ok && tile < num_tiles; tile += num_pairs, ++local) {
        const uint32_t acc_phase = local & 1u;
        for (int sub = 0; ok && sub < 2; ++sub) {
          const uint64_t b_desc = sub ? b_desc_k : b_desc_mn;
          const uint32_t b_hi = (uint32_t)(b_desc >> 32), b_lo0 = (uint32_t)b_desc;
          const uint32_t b_step = (sub ? 32u : kChunkBytes / kKSteps) >> 4;
          const uint32_t idesc = sub ? p.idesc2 : p.idesc1;
          const int num_kb = sub ? kb2 : kb1;
          ok = wait_bounded(acc_empty_bar(sub), acc_phase ^ 1u, abort_flag, p.status, p.wait_limit);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + sub * BN;
          uint32_t accumulate = 0;
          for (int kb = 0; kb < num_kb; ++kb) {
            if (!ptx::mbar_try_wait(full_bar(stage), phase)) {
              ok = wait_bounded(full_bar(stage), phase, abort_flag, p.status, p.wait_limit);
              if (!ok) break;
            }
            ptx::tc_fence_after_sync();
            const uint32_t a_lo = a_lo0 + stage * kStageStep, b_lo = b_lo0 + stage * kStageStep;
#pragma unroll
            for (int k = 0; k < kKSteps; ++k) {
              const uint64_t adesc = ((uint64_t)a_hi << 32) | (a_lo + k * 2u);
              const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo + k * b_step);
              ptx::mma_ss_pair<true>(d_tmem, adesc, bdesc, idesc, accumulate);
              accumulate = 1;
            }
            ptx::mma_commit_pair(empty_bar(stage), 3);
            if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) ptx::mma_commit_pair(acc_full_bar(sub), 3);
        }
      }
      if (*abort_flag) {
        ptx::mma_commit_pair(drained_bar, 1);
        for (uint32_t it = 0; it < p.wait_limit && !ptx::mbar_try_wait(drained_bar, 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    // Warp (lane quarter q, part) owns 32 rows x 64 columns of the tile; a lane holds one row of them.  The rounded
    // pre-activation of a tile stays in 32 registers of packed 16-bit pairs (hst) between the two phases; staging
    // is one FP8 output box of 32 rows x 64 bytes (64-byte swizzle) per warp.
    const int q = warp & 3, part = (warp - 2) >> 2;
    const uint32_t buf_out = epi_base + (warp - 2) * S::kEpiWarpBytes;
    const uint32_t row64 = (uint32_t)lane * 64u, sw64 = (uint32_t)((lane >> 1) & 3);
    const f32x2 s1 = splat2(p.scale1), s2 = splat2(p.scale2), in2 = splat2(p.act_in), os2 = splat2(p.grad_out * p.act_in);
    const float tail_k = fabsf(p.act_in) * (1.0f / kTailRange), act_oi = p.act_out * p.act_in;

    auto release_acc = [&](int a) {
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(ptx::in_even_cta(acc_empty_bar(a)));
    };
    uint32_t hst[32];
    // One 32-column slice s of accumulator 0: scale, keep round16(H), GELU, round, stage.
    auto slice_fwd = [&](const uint32_t (&r)[32], int s) {
      uint32_t held[2];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        f32x2 x[4];
        float y[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          x[k] = mul2(pack2(__uint_as_float(r[8 * g + 2 * k]), __uint_as_float(r[8 * g + 2 * k + 1])), s1);
          float a, b;
          unpack2(x[k], a, b);
          hst[16 * s + 4 * g + k] = H_BF16 ? pack_bf16x2(a, b) : pack_f16x2(a, b);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) gelu_scaled2<true>(x[k], tail_k, act_oi, y[2 * k], y[2 * k + 1]);
        const uint32_t lo = cvt_fp8x4<A_E5>(y[0], y[1], y[2], y[3]);
        const uint32_t hi = cvt_fp8x4<A_E5>(y[4], y[5], y[6], y[7]);
        if ((g & 1) == 0) { held[0] = lo; held[1] = hi; }
        else ptx::sts128(buf_out + row64 + ((((uint32_t)(2 * s + (g >> 1))) ^ sw64) << 4), make_uint4(held[0], held[1], lo, hi));
      }
    };
    // The same slice of accumulator 1: scale, GELU gradient from the kept pre-activation, round, stage.
    auto slice_bwd = [&](const uint32_t (&r)[32], int s) {
      uint32_t held[2];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        float y[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const f32x2 x = mul2(pack2(__uint_as_float(r[8 * g + 2 * k]), __uint_as_float(r[8 * g + 2 * k + 1])), s2);
          const float2 h = H_BF16 ? unpack_bf16x2(hst[16 * s + 4 * g + k]) : unpack_f16x2(hst[16 * s + 4 * g + k]);
          unpack2(gelu_grad_scaled2(pack2(h.x, h.y), x, in2, os2), y[2 * k], y[2 * k + 1]);
        }
        const uint32_t lo = cvt_fp8x4<D_E5>(y[0], y[1], y[2], y[3]);
        const uint32_t hi = cvt_fp8x4<D_E5>(y[4], y[5], y[6], y[7]);
        if ((g & 1) == 0) { held[0] = lo; held[1] = hi; }
        else ptx::sts128(buf_out + row64 + ((((uint32_t)(2 * s + (g >> 1))) ^ sw64) << 4), make_uint4(held[0], held[1], lo, hi));
      }
    };

    uint32_t local = 0;
    bool ok = true;
    for (int tile = pair; ok && tile < num_tiles; tile += num_pairs, ++local) {
      int tm, tn;
      tile_mn2(tile, tm, tn);
      const int row0 = tm * 256 + rank * 128 + q * 32, n_w = tn * BN + part * 64;
      const bool active = n_w < p.N;                            // warp-uniform
      const uint32_t acc_phase = local & 1u;
#pragma unroll
      for (int sub = 0; sub < 2; ++sub) {
        ok = wait_bounded(acc_full_bar(sub), acc_phase, abort_flag, p.status, p.wait_limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + sub * BN + part * 64;
        uint32_t r0[32], r1[32];
        if (active) {
          ptx::tmem_ld_32x32_issue(t_row, r0);
          if (lane == 0) ptx::bulk_wait_group_read<0>();        // earlier stores have read the staging boxes
          __syncwarp();
          ptx::tmem_ld_fence(r0);
          ptx::tmem_ld_32x32_issue(t_row + 32, r1);
          if (sub == 0) slice_fwd(r0, 0); else slice_bwd(r0, 0);
          ptx::tmem_ld_fence(r1);
        }
        release_acc(sub);                                       // the values are in registers
        if (active) {
          if (sub == 0) slice_fwd(r1, 1); else slice_bwd(r1, 1);
          if (sub == 0 && p.h_ptr != nullptr && row0 + lane < p.M) {
            // the copy of the rounded pre-activation: this lane's 64 columns, 8 at a time (16 aligned bytes)
            uint8_t* dst = p.h_ptr + ((long long)(row0 + lane) * p.h_ld + n_w) * 2;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const int col = n_w + 8 * c;
              if (col + 8 <= p.N) {
                *reinterpret_cast<uint4*>(dst + 16 * c) = make_uint4(hst[4 * c], hst[4 * c + 1], hst[4 * c + 2], hst[4 * c + 3]);
              } else {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  if (col + j < p.N)
                    *reinterpret_cast<uint16_t*>(dst + 16 * c + 2 * j) = (uint16_t)(hst[4 * c + (j >> 1)] >> (16 * (j & 1)));
              }
            }
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (sub == 0) {
              ptx::tma_store_2d(&tm_a, buf_out, n_w, row0);
            } else {
              ptx::tma_store_2d(&tm_dh, buf_out, n_w, row0);
            }
            ptx::bulk_commit_group();
          }
        }
      }
    }
    // Leaving (early too, when a wait ran out somewhere in the CTA): tensor-memory loads have landed and
    // the stores have read shared memory before the CTA may give up its resources.
    ptx::tmem_ld_wait_all();
    if (lane == 0) ptx::bulk_wait_group_read<0>();
    __syncwarp();
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// Row-major [rows x cols] matrix of es-byte elements, boxes of box_rows rows x box_bytes, swizzled with the
// pattern of that width; out-of-range parts of a box read as zero and are not written.
bool make_tmap(CUtensorMap* tm, const us_mat* m, int es, int box_rows, int box_bytes) {
  host::EncodeTiledFn fn = host::encode_tiled_fn();
  if (!fn) return false;
  const CUtensorMapDataType type = es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16;
  cuuint64_t dims[2] = {(cuuint64_t)m->cols, (cuuint64_t)m->rows};
  cuuint64_t strides[1] = {(cuuint64_t)m->ld * es};
  cuuint32_t box[2] = {(cuuint32_t)(box_bytes / es), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, type, 2, m->ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
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

template <bool A_E5, bool D_E5, bool H_BF16>
us_status launch_hidden(const CUtensorMap* t, const HiddenParams& p, int grid, cudaStream_t stream) {
  auto kern = ffn_hidden_kernel<A_E5, D_E5, H_BF16>;
  constexpr int smem = HidSmem::kTotal;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return US_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(gemm_threads(kHidEW));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, t[0], t[1], t[2], t[3], t[4], t[5], p) == cudaSuccess ? US_OK : US_ERR_CUDA;
}

us_status hidden_impl(const us_mat* X, const us_mat* W1, float alpha, const us_mat* G, const us_mat* W2, float beta_x,
                      float act_in_scale, float act_out_scale, float grad_out_scale, int h_dtype, const us_mat* H,
                      const us_mat* A, const us_mat* dH, void* ws, size_t ws_bytes, void* stream, uint32_t wait_limit,
                      int no_loads) {
  if (!valid_mat(X) || !valid_mat(W1) || !valid_mat(G) || !valid_mat(W2) || !valid_mat(A) || !valid_mat(dH)) return US_ERR_INVALID_ARG;
  const bool keep_h = H && H->ptr;
  if (keep_h && !valid_mat(H)) return US_ERR_INVALID_ARG;
  if (h_dtype != US_BF16 && h_dtype != US_F16) return US_ERR_INVALID_ARG;
  const int64_t M = X->rows, K1 = X->cols, N = W1->cols, K2 = G->cols;
  if (W1->rows != K1 || G->rows != M || W2->rows != N || W2->cols != K2) return US_ERR_INVALID_ARG;
  if (A->rows != M || A->cols != N || dH->rows != M || dH->cols != N) return US_ERR_INVALID_ARG;
  if (keep_h && (H->rows != M || H->cols != N || H->dtype != h_dtype)) return US_ERR_INVALID_ARG;
  if (!ws || ws_bytes < us_workspace_bytes()) return US_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % 16) return US_ERR_ALIGNMENT;
  if (!aligned16(X) || !aligned16(W1) || !aligned16(G) || !aligned16(W2) || !aligned16(A) || !aligned16(dH) ||
      (keep_h && !aligned16(H)))
    return US_ERR_ALIGNMENT;
  if (!(is_fp8(X->dtype) && is_fp8(W1->dtype) && is_fp8(G->dtype) && is_fp8(W2->dtype) && is_fp8(A->dtype) && is_fp8(dH->dtype)))
    return US_ERR_UNSUPPORTED;
  if (M <= 128 || N <= 128) return US_ERR_UNSUPPORTED;          // tiles of 256 x 256 only

  HiddenParams p{};
  p.M = (int)M; p.N = (int)N; p.K1 = (int)K1; p.K2 = (int)K2;
  p.tiles_m = (int)((M + 255) / 256); p.tiles_n = (int)((N + 255) / 256);
  if ((int64_t)p.tiles_m * p.tiles_n >= (1ll << 30)) return US_ERR_UNSUPPORTED;
  p.d_tiles_m = make_fast_div(p.tiles_m);
  p.idesc1 = make_idesc(X->dtype == US_E5M2, W1->dtype == US_E5M2, false, true, 256, 256);
  p.idesc2 = make_idesc(G->dtype == US_E5M2, W2->dtype == US_E5M2, false, false, 256, 256);
  p.scale1 = alpha; p.scale2 = beta_x;
  p.act_in = act_in_scale; p.act_out = act_out_scale; p.grad_out = grad_out_scale;
  p.h_ptr = keep_h ? static_cast<uint8_t*>(H->ptr) : nullptr;
  p.h_ld = keep_h ? H->ld : 0;
  p.status = static_cast<unsigned int*>(ws);
  p.wait_limit = wait_limit;
  p.no_loads = no_loads;

  CUtensorMap t[6];
  if (!make_tmap(&t[0], X, 1, 128, 128) || !make_tmap(&t[1], W1, 1, 128, 128) || !make_tmap(&t[2], G, 1, 128, 128) ||
      !make_tmap(&t[3], W2, 1, 128, 128) || !make_tmap(&t[4], A, 1, 32, 64) || !make_tmap(&t[5], dH, 1, 32, 64))
    return US_ERR_CUDA;

  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const int tiles = p.tiles_m * p.tiles_n, pairs = sms / 2;
  const int grid = 2 * (tiles < pairs ? tiles : pairs);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool a5 = A->dtype == US_E5M2, d5 = dH->dtype == US_E5M2, bf = h_dtype == US_BF16;
  if (!a5 && d5) return bf ? launch_hidden<false, true, true>(t, p, grid, st) : launch_hidden<false, true, false>(t, p, grid, st);
  if (!a5 && !d5) return bf ? launch_hidden<false, false, true>(t, p, grid, st) : launch_hidden<false, false, false>(t, p, grid, st);
  if (a5 && d5) return bf ? launch_hidden<true, true, true>(t, p, grid, st) : launch_hidden<true, true, false>(t, p, grid, st);
  return bf ? launch_hidden<true, false, true>(t, p, grid, st) : launch_hidden<true, false, false>(t, p, grid, st);
}

}  // namespace
}  // namespace us

extern "C" us_status us_ffn_hidden(const us_mat* X, const us_mat* W1, float alpha, const us_mat* G, const us_mat* W2,
                                   float beta_x, float act_in_scale, float act_out_scale, float grad_out_scale,
                                   int32_t h_dtype, const us_mat* H, const us_mat* A, const us_mat* dH, void* ws,
                                   size_t ws_bytes, void* stream) {
  return us::hidden_impl(X, W1, alpha, G, W2, beta_x, act_in_scale, act_out_scale, grad_out_scale, h_dtype, H, A, dH, ws,
                         ws_bytes, stream, us::kWaitLimit, 0);
}

extern "C" us_status us_test_ffn_hidden_starved(const us_mat* X, const us_mat* W1, const us_mat* G, const us_mat* W2,
                                                const us_mat* A, const us_mat* dH, void* ws, size_t ws_bytes,
                                                uint32_t wait_limit, void* stream) {
  if (wait_limit == 0 || wait_limit > (1u << 16)) return US_ERR_INVALID_ARG;
  return us::hidden_impl(X, W1, 1.f, G, W2, 1.f, 1.f, 1.f, 1.f, US_BF16, nullptr, A, dH, ws, ws_bytes, stream, wait_limit, 1);
}
