// The unit-scaled GEMM of libunitscale for sm_100a.
//
//   out[M x N] = epilogue( scale * sum_k A(m, k) B(n, k) )
//
// One persistent CTA per SM walks over 128 x BN output tiles.  Warp roles:
//   warp 0   TMA producer: fills a ring of shared-memory stages (one 128-byte-swizzled
//            A tile + B tile per stage, 128 bytes of K each) with cp.async.bulk.tensor;
//   warp 1   MMA issuer: one thread issues tcgen05.mma (4 per stage) into one of two
//            float32 accumulators in tensor memory, commits stage release and
//            accumulator-ready barriers; the warp owns the TMEM allocation;
//   warps 2-5 epilogue: tcgen05.ld their 32-lane quarter of the finished accumulator,
//            apply scale / GELU / GELU-gradient / residual, round once, store.
// While the epilogue drains accumulator i, the MMA warp already fills accumulator i^1.
//
// Either operand may be stored K-major (row = M or N index, K contiguous) or MN-major
// (row = K index, M or N contiguous); the three linear ops differ only in that choice,
// so no operand is ever transposed in memory.
//
// Every wait is bounded: when a limit is hit the CTA raises a status word in the
// caller's workspace, all roles leave their loops, outstanding copies and MMAs are
// drained (bounded again), TMEM is freed and the kernel returns.
#pragma once

#include "common.cuh"
#include "sm100.cuh"

namespace us {

struct GemmParams {
  int M, N, K;
  int tiles_m, tiles_n;
  float scale;
  uint32_t idesc;
  void* out; int out_dt; int64_t out_ld;
  int act; float act_in, act_out;
  void* aux; int aux_dt; int64_t aux_ld;
  const void* skip; int skip_dt; int64_t skip_ld; float skip_coef, out_coef;
  unsigned int* status;
};

constexpr int kBM = 128;                 // tile rows = TMEM lanes
constexpr int kStageKBytes = 128;        // bytes of K per stage = one swizzle atom
constexpr int kKSteps = 4;               // MMAs per stage (32 bytes of K each)
constexpr int kGemmThreads = 192;
constexpr uint32_t kWaitLimit = 1u << 22;
constexpr unsigned int kStatusTimeout = 1;

template <int BN>
struct GemmSmem {
  static constexpr int kABytes = kBM * kStageKBytes;
  static constexpr int kBBytes = BN * kStageKBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kBarrierBytes = 256;
  static constexpr int kTotal = kStages * kStageBytes + kBarrierBytes + 1024;  // + alignment slack
};

// Bounded mbarrier wait.  Returns false if the CTA is aborting (this wait or another one timed out).
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             unsigned int* status) {
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  if (status) atomicExch(status, kStatusTimeout);
  return false;
}

// One 32-column slice of one output row: v holds scale * acc on entry.
template <bool kFull>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, float (&v)[32], int64_t row, int col, int ncols) {
  // kFull: all 32 columns are inside the matrix and every access is a 16-byte vector.
  if (p.act == US_ACT_GELU) {
    if (p.aux) {
      if (kFull) {
        store_vec<32>(static_cast<char*>(p.aux) + (row * p.aux_ld + col) * 2, p.aux_dt, v);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < ncols) store_one(p.aux, p.aux_dt, row * p.aux_ld + col + i, v[i]);
      }
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = gelu_scaled(v[i], p.act_in, p.act_out);
  } else if (p.act == US_ACT_GELU_GRAD) {
    float h[32];
    if (kFull) {
      load_vec<32>(static_cast<const char*>(p.aux) + (row * p.aux_ld + col) * 2, p.aux_dt, h);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) h[i] = (i < ncols) ? load_one(p.aux, p.aux_dt, row * p.aux_ld + col + i) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = gelu_grad_scaled(h[i], v[i], p.act_in, p.act_out);
  }
  if (p.skip) {
    float s[32];
    if (kFull) {
      load_vec<32>(static_cast<const char*>(p.skip) + (row * p.skip_ld + col) * dtype_size(p.skip_dt), p.skip_dt, s);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) s[i] = (i < ncols) ? load_one(p.skip, p.skip_dt, row * p.skip_ld + col + i) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = fmaf(p.skip_coef, s[i], p.out_coef * v[i]);
  }
  if (kFull) {
    store_vec<32>(static_cast<char*>(p.out) + (row * p.out_ld + col) * dtype_size(p.out_dt), p.out_dt, v);
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (i < ncols) store_one(p.out, p.out_dt, row * p.out_ld + col + i, v[i]);
  }
}

// ES: operand element size in bytes (1 = FP8, 2 = BF16 / F16).
// A_MN / B_MN: operand stored MN-major ([K x M] resp. [K x N] row-major) instead of K-major.
template <int ES, bool A_MN, bool B_MN, int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const GemmParams p) {
  using S = GemmSmem<BN>;
  constexpr int kBK = kStageKBytes / ES;            // K elements per stage
  constexpr int kChunkElems = 128 / ES;             // MN elements per 128-byte row of an MN-major tile
  constexpr uint32_t kChunkBytes = kBK * 128;       // one MN-major chunk: kBK rows of 128 bytes
  constexpr uint32_t kTmemCols = 2 * BN;            // two accumulators

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
  const uint32_t bars = smem_base + S::kStages * S::kStageBytes;
  // barrier layout (8 bytes each): full[kStages], empty[kStages], acc_full[2], acc_empty[2], drained
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S::kStages + s); };
  auto acc_full_bar = [&](int a) { return bars + 8u * (2 * S::kStages + a); };
  auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * S::kStages + 2 + a); };
  const uint32_t drained_bar = bars + 8u * (2 * S::kStages + 4);
  uint8_t* tail = smem_gen + S::kStages * S::kStageBytes + 8 * (2 * S::kStages + 5);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int num_kb = (p.K + kBK - 1) / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full_bar(a), 1); ptx::mbar_init(acc_empty_bar(a), 4); }
    ptx::mbar_init(drained_bar, 1);
    *abort_flag = 0;
    ptx::mbar_init_fence();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t issued = 0;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int m0 = (tile % p.tiles_m) * kBM;
        const int n0 = (tile / p.tiles_m) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status);
          if (!ok) break;
          const uint32_t a_dst = smem_base + stage * S::kStageBytes;
          const uint32_t b_dst = a_dst + S::kABytes;
          const int k0 = kb * kBK;
          ptx::mbar_expect_tx(full_bar(stage), S::kStageBytes);
          if (A_MN) {
#pragma unroll
            for (int c = 0; c < kBM / kChunkElems; ++c)
              ptx::tma_load_2d(a_dst + c * kChunkBytes, &tmap_a, full_bar(stage), m0 + c * kChunkElems, k0);
          } else {
            ptx::tma_load_2d(a_dst, &tmap_a, full_bar(stage), k0, m0);
          }
          if (B_MN) {
#pragma unroll
            for (int c = 0; c < BN / kChunkElems; ++c)
              ptx::tma_load_2d(b_dst + c * kChunkBytes, &tmap_b, full_bar(stage), n0 + c * kChunkElems, k0);
          } else {
            ptx::tma_load_2d(b_dst, &tmap_b, full_bar(stage), k0, n0);
          }
          ++issued;
          if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*abort_flag) {
        // Let copies that are still in flight land before the CTA gives up its shared memory.
        const uint32_t n = issued < (uint32_t)S::kStages ? issued : (uint32_t)S::kStages;
        for (uint32_t i = 0; i < n; ++i) {
          if (stage == 0) { stage = S::kStages; phase ^= 1u; }
          --stage;
          for (uint32_t it = 0; it < kWaitLimit && !ptx::mbar_try_wait(full_bar(stage), phase); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      uint32_t local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++local) {
        const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
        ok = wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = wait_bounded(full_bar(stage), phase, abort_flag, p.status);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t a_src = smem_base + stage * S::kStageBytes;
          const uint32_t b_src = a_src + S::kABytes;
#pragma unroll
          for (int k = 0; k < kKSteps; ++k) {
            // K-major: 32 bytes further along the swizzled row.  MN-major: kBK/4 rows of 128 bytes further.
            const uint64_t adesc = A_MN ? ptx::smem_desc_sw128(a_src + k * (kChunkBytes / kKSteps), kChunkBytes, 1024)
                                        : ptx::smem_desc_sw128(a_src + k * 32, 16, 1024);
            const uint64_t bdesc = B_MN ? ptx::smem_desc_sw128(b_src + k * (kChunkBytes / kKSteps), kChunkBytes, 1024)
                                        : ptx::smem_desc_sw128(b_src + k * 32, 16, 1024);
            ptx::mma_ss<ES == 1>(d_tmem, adesc, bdesc, p.idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::mma_commit(empty_bar(stage));        // stage reusable once these MMAs have read it
          if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) ptx::mma_commit(acc_full_bar(acc));  // accumulator complete
      }
      if (*abort_flag) {
        ptx::mma_commit(drained_bar);
        for (uint32_t it = 0; it < kWaitLimit && !ptx::mbar_try_wait(drained_bar, 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    uint32_t local = 0;
    bool ok = true;
    const bool vec_ok = true;                        // host guarantees 16-byte aligned rows
    for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++local) {
      const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
      const int m0 = (tile % p.tiles_m) * kBM;
      const int n0 = (tile / p.tiles_m) * BN;
      ok = wait_bounded(acc_full_bar(acc), acc_phase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const int64_t row = m0 + q * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
#pragma unroll 1
      for (int c = 0; c < BN; c += 32) {
        if (n0 + c >= p.N) break;                    // warp-uniform
        float v[32];
        ptx::tmem_ld_32x32(t_row + c, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= p.scale;
        if (row < p.M) {
          const int ncols = min(32, p.N - (n0 + c));
          if (vec_ok && ncols == 32) epilogue_chunk<true>(p, v, row, n0 + c, 32);
          else epilogue_chunk<false>(p, v, row, n0 + c, ncols);
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(acc_empty_bar(acc));
    }
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace us
