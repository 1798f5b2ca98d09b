// Several independent unit-scaled GEMMs in ONE launch (us_linear_group).
//
// The last four GEMMs of an FFN step (the second forward GEMM, the two weight-gradient GEMMs
// and the input-gradient GEMM of the first layer) depend on nothing but tensors that exist already.
// Launched one after the other, each pays its own set-up and tail and leaves a partly filled last
// wave (64 or 128 tiles of 256 x 256 on 74 CTA pairs).  Here the tiles of all problems form one
// list that the host deals out to the CTA pairs longest-first, so that every pair gets about the
// same number of K blocks; a pair walks its share with the usual roles (TMA producer, MMA issuer,
// eight epilogue warps), and the main loop of a pair's next tile runs while its previous tile's
// epilogue drains, across problem boundaries too.
//
// Scope: FP8 operands (either layout each), CTA-pair tiles of 256 x 256 (cta_group::2), plain
// or residual (skip) epilogue, any output dtype, up to kGroupMaxProblems problems.  Everything that
// differs between problems is run-time data here: tensor maps, operand layouts (a K-major and an
// MN-major FP8 tile are both one 128-row x 128-byte box, only the coordinate order and the
// descriptor strides differ), instruction descriptor, scale, epilogue kind.
#pragma once

#include "gemm_kernel.cuh"

namespace us {

constexpr int kGroupMaxProblems = 4;
constexpr int kGroupMaxRounds = 12;
constexpr int kGroupMaxPairs = 80;

struct GroupProblem {
  CUtensorMap ta, tb, tout, tskip;      // A and B: 128-row x 128-byte boxes; out / skip: 32-row x 128-byte boxes
  int M, N, K;
  int a_mn, b_mn;                       // operand stored MN-major ([K x M] resp. [K x N] row-major)
  uint32_t idesc;
  float scale;
  int out_dt;
  int has_skip, skip_dt;
  float skip_coef, out_coef;
};

struct GroupParams {
  GroupProblem prob[kGroupMaxProblems];
  int count, rounds, pairs;
  unsigned int* status;
  uint32_t wait_limit;
  // work list: entry [round * pairs + pair] = problem << 24 | tile row << 12 | tile column, or -1
  int32_t table[kGroupMaxRounds * kGroupMaxPairs];
};

__device__ __forceinline__ void group_decode(int32_t e, int& prob, int& tm, int& tn) {
  prob = e >> 24; tm = (e >> 12) & 0xfff; tn = e & 0xfff;
}

constexpr int kGroupEW = 8;
using GroupSmem = GemmSmem<256, 2, kGroupEW>;

__global__ void __launch_bounds__(gemm_threads(kGroupEW), 1)
gemm_group_kernel(const __grid_constant__ GroupParams g) {
  using S = GroupSmem;
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
  auto epi_in_bar = [&](int w) { return bars + 8u * (2 * S::kStages + 5 + w); };
  uint8_t* tail = smem_gen + S::kStages * S::kStageBytes + S::kEpiBytes + 8 * (2 * S::kStages + 5 + kGroupEW);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)ptx::cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  auto entry = [&](int r) { return g.table[r * g.pairs + pair]; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full_bar(a), 1); ptx::mbar_init(acc_empty_bar(a), 2 * 4 * (BN / 128)); }
    ptx::mbar_init(drained_bar, 1);
    for (int w = 0; w < kGroupEW; ++w) ptx::mbar_init(epi_in_bar(w), 1);
    *abort_flag = 0;
    ptx::mbar_init_fence();
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
      for (int r = 0; ok && r < g.rounds; ++r) {
        const int32_t e = entry(r);
        if (e < 0) continue;
        int pi, tm, tn;
        group_decode(e, pi, tm, tn);
        const GroupProblem& P = g.prob[pi];
        const int m0 = tm * 256 + rank * 128, n0 = tn * 256 + rank * 128;
        const int num_kb = (P.K + kBK - 1) / kBK;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, g.status, g.wait_limit);
          if (!ok) break;
          const uint32_t a_dst = smem_base + stage * S::kStageBytes, b_dst = a_dst + S::kABytes;
          const int k0 = kb * kBK;
          const uint32_t fb = ptx::in_even_cta(full_bar(stage));
          if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), 2 * S::kStageBytes);
          if (P.a_mn) ptx::tma_load_2d_pair(a_dst, &P.ta, fb, m0, k0); else ptx::tma_load_2d_pair(a_dst, &P.ta, fb, k0, m0);
          if (P.b_mn) ptx::tma_load_2d_pair(b_dst, &P.tb, fb, n0, k0); else ptx::tma_load_2d_pair(b_dst, &P.tb, fb, k0, n0);
          ++issued;
          if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*abort_flag && rank == 0) {
        const uint32_t n = issued < (uint32_t)S::kStages ? issued : (uint32_t)S::kStages;
        for (uint32_t i = 0; i < n; ++i) {
          if (stage == 0) { stage = S::kStages; phase ^= 1u; }
          --stage;
          for (uint32_t it = 0; it < g.wait_limit && !ptx::mbar_try_wait(full_bar(stage), phase); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0, local = 0;
      bool ok = true;
      constexpr uint32_t kStageStep = S::kStageBytes >> 4;
      for (int r = 0; ok && r < g.rounds; ++r) {
        const int32_t e = entry(r);
        if (e < 0) continue;
        int pi, tm, tn;
        group_decode(e, pi, tm, tn);
        const GroupProblem& P = g.prob[pi];
        const int num_kb = (P.K + kBK - 1) / kBK;
        const uint64_t a_desc0 = P.a_mn ? ptx::smem_desc_sw128(smem_base, kChunkBytes, 1024) : ptx::smem_desc_sw128(smem_base, 16, 1024);
        const uint64_t b_desc0 = P.b_mn ? ptx::smem_desc_sw128(smem_base + S::kABytes, kChunkBytes, 1024)
                                        : ptx::smem_desc_sw128(smem_base + S::kABytes, 16, 1024);
        const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), b_hi = (uint32_t)(b_desc0 >> 32);
        const uint32_t a_lo0 = (uint32_t)a_desc0, b_lo0 = (uint32_t)b_desc0;
        const uint32_t a_step = (P.a_mn ? kChunkBytes / kKSteps : 32u) >> 4, b_step = (P.b_mn ? kChunkBytes / kKSteps : 32u) >> 4;
        const uint32_t idesc = P.idesc;
        const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
        ++local;
        ok = wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, g.status, g.wait_limit);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        uint32_t accumulate = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_try_wait(full_bar(stage), phase)) {
            ok = wait_bounded(full_bar(stage), phase, abort_flag, g.status, g.wait_limit);
            if (!ok) break;
          }
          ptx::tc_fence_after_sync();
          const uint32_t a_lo = a_lo0 + stage * kStageStep, b_lo = b_lo0 + stage * kStageStep;
#pragma unroll
          for (int k = 0; k < kKSteps; ++k) {
            const uint64_t adesc = ((uint64_t)a_hi << 32) | (a_lo + k * a_step);
            const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo + k * b_step);
            ptx::mma_ss_pair<true>(d_tmem, adesc, bdesc, idesc, accumulate);
            accumulate = 1;
          }
          ptx::mma_commit_pair(empty_bar(stage), 3);
          if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) ptx::mma_commit_pair(acc_full_bar(acc), 3);
      }
      if (*abort_flag) {
        ptx::mma_commit_pair(drained_bar, 1);
        for (uint32_t it = 0; it < g.wait_limit && !ptx::mbar_try_wait(drained_bar, 0); ++it) {}
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    // Warp (quarter q, half) owns 32 rows x 128 columns of a tile, worked in 32-column slices.  Staging: box 0
    // (4 KB) receives the skip tensor's boxes by TMA, box 1 (4 KB) collects output and leaves by TMA store.
    const int q = warp & 3, half = (warp - 2) >> 2;
    const uint32_t buf_in = epi_base + (warp - 2) * epi_warp_bytes(kGroupEW), buf_out = buf_in + 4096u;
    const uint32_t in_bar = epi_in_bar(warp - 2);
    const uint32_t row_off = (uint32_t)lane * 128u, sw = (uint32_t)(lane & 7);
    uint32_t in_phase = 0, local = 0;
    bool in_pending = false, ok = true;

    auto issue_in = [&](const GroupProblem& P, int col, int row0) {
      if (lane == 0) {
        ptx::mbar_expect_tx(in_bar, 4096);
        ptx::tma_load_2d(buf_in, &P.tskip, in_bar, col, row0);
      }
      in_pending = true;
    };
    // first box of the skip tensor for the first tile at or after round r that has one for this warp
    auto prefetch_from = [&](int r) {
      for (; r < g.rounds; ++r) {
        const int32_t e = entry(r);
        if (e < 0) continue;
        int pi, tm, tn;
        group_decode(e, pi, tm, tn);
        const GroupProblem& P = g.prob[pi];
        const int n_w = tn * BN + half * 128;
        if (P.has_skip && n_w < P.N) issue_in(P, n_w, tm * 256 + rank * 128 + q * 32);
        return;                                                // only the very next tile is looked at
      }
    };
    prefetch_from(0);

    for (int r = 0; ok && r < g.rounds; ++r) {
      const int32_t e = entry(r);
      if (e < 0) continue;
      int pi, tm, tn;
      group_decode(e, pi, tm, tn);
      const GroupProblem& P = g.prob[pi];
      const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
      ++local;
      const int row0 = tm * 256 + rank * 128 + q * 32, n_w = tn * BN + half * 128;
      const bool skip = P.has_skip != 0;
      const int in_es = dtype_size(P.skip_dt), out_es = dtype_size(P.out_dt);
      const int in_box_cols = 128 / in_es, out_box_cols = 128 / out_es;
      ok = wait_bounded(acc_full_bar(acc), acc_phase, abort_flag, g.status, g.wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + half * 128;
      auto release_acc = [&]() {
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(ptx::in_even_cta(acc_empty_bar(acc)));
      };
      bool released = false, looked_ahead = false;
      if (n_w < P.N) {
        const f32x2 scale2 = splat2(P.scale), skip2 = splat2(P.skip_coef), oc2 = splat2(P.out_coef);
#pragma unroll 1
        for (int sl = 0; sl < 4; ++sl) {
          const int col = n_w + 32 * sl;
          if (col >= P.N) break;
          const bool last_slice = sl == 3 || col + 32 >= P.N;
          uint4 raw[8];
          if (skip) {
            const int off = (32 * sl) & (in_box_cols - 1);
            if (off == 0) {
              ok = wait_bounded(in_bar, in_phase, abort_flag, g.status, g.wait_limit);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              in_phase ^= 1u;
              in_pending = false;
            }
            const uint32_t cb = (uint32_t)(off * in_es) >> 4;
            const int nchunk = 2 * in_es;
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (j < nchunk) raw[j] = ptx::lds128(buf_in + row_off + (((cb + j) ^ sw) << 4));
            if (off + 32 == in_box_cols || last_slice) {
              __syncwarp();                                    // every lane has read the box
              if (!last_slice) issue_in(P, col + 32, row0);
              else { prefetch_from(r + 1); looked_ahead = true; }
            }
          }
          const int out_off = (32 * sl) & (out_box_cols - 1);
          if (out_off == 0) {                                  // the output box is about to be refilled
            if (lane == 0) ptx::bulk_wait_group_read<0>();
            __syncwarp();
          }
          float v[32];
          ptx::tmem_ld_32x32(t_row + 32 * sl, v);
          if (last_slice) { release_acc(); released = true; }
          const uint32_t out_cb = (uint32_t)(out_off * out_es) >> 4;
          const uint32_t dst = buf_out + row_off;
          uint32_t held[2];
#pragma unroll
          for (int gi = 0; gi < 4; ++gi) {
            f32x2 x[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) x[k] = mul2(pack2(v[8 * gi + 2 * k], v[8 * gi + 2 * k + 1]), scale2);
            float y[8];
            if (skip) {
              float sk[8];
              if (P.skip_dt == US_F32) {
                sk[0] = __uint_as_float(raw[2 * gi].x); sk[1] = __uint_as_float(raw[2 * gi].y);
                sk[2] = __uint_as_float(raw[2 * gi].z); sk[3] = __uint_as_float(raw[2 * gi].w);
                sk[4] = __uint_as_float(raw[2 * gi + 1].x); sk[5] = __uint_as_float(raw[2 * gi + 1].y);
                sk[6] = __uint_as_float(raw[2 * gi + 1].z); sk[7] = __uint_as_float(raw[2 * gi + 1].w);
              } else {
                const uint32_t w[4] = {raw[gi].x, raw[gi].y, raw[gi].z, raw[gi].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const float2 h = P.skip_dt == US_BF16 ? unpack_bf16x2(w[k]) : unpack_f16x2(w[k]);
                  sk[2 * k] = h.x; sk[2 * k + 1] = h.y;
                }
              }
#pragma unroll
              for (int k = 0; k < 4; ++k)
                unpack2(fma2(skip2, pack2(sk[2 * k], sk[2 * k + 1]), mul2(oc2, x[k])), y[2 * k], y[2 * k + 1]);
            } else {
#pragma unroll
              for (int k = 0; k < 4; ++k) unpack2(x[k], y[2 * k], y[2 * k + 1]);
            }
            if (P.out_dt == US_F32) {
              ptx::sts128(dst + (((out_cb + 2 * gi) ^ sw) << 4),
                          make_uint4(__float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3])));
              ptx::sts128(dst + (((out_cb + 2 * gi + 1) ^ sw) << 4),
                          make_uint4(__float_as_uint(y[4]), __float_as_uint(y[5]), __float_as_uint(y[6]), __float_as_uint(y[7])));
            } else if (P.out_dt == US_BF16 || P.out_dt == US_F16) {
              uint32_t w[4];
#pragma unroll
              for (int k = 0; k < 4; ++k)
                w[k] = P.out_dt == US_BF16 ? pack_bf16x2(y[2 * k], y[2 * k + 1]) : pack_f16x2(y[2 * k], y[2 * k + 1]);
              ptx::sts128(dst + (((out_cb + gi) ^ sw) << 4), make_uint4(w[0], w[1], w[2], w[3]));
            } else {
              const uint32_t lo = P.out_dt == US_E5M2 ? cvt_fp8x4<true>(y[0], y[1], y[2], y[3]) : cvt_fp8x4<false>(y[0], y[1], y[2], y[3]);
              const uint32_t hi = P.out_dt == US_E5M2 ? cvt_fp8x4<true>(y[4], y[5], y[6], y[7]) : cvt_fp8x4<false>(y[4], y[5], y[6], y[7]);
              if ((gi & 1) == 0) { held[0] = lo; held[1] = hi; }
              else ptx::sts128(dst + (((out_cb + (gi >> 1)) ^ sw) << 4), make_uint4(held[0], held[1], lo, hi));
            }
          }
          if (out_off + 32 == out_box_cols || last_slice) {
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) { ptx::tma_store_2d(&P.tout, buf_out, col - out_off, row0); ptx::bulk_commit_group(); }
          }
        }
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (!released) release_acc();
      if (!looked_ahead) prefetch_from(r + 1);                 // plain tile, or no columns here: the input box is free, fetch for the next tile
    }
    if (in_pending && lane == 0)
      for (uint32_t it = 0; it < g.wait_limit && !ptx::mbar_try_wait(in_bar, in_phase); ++it) {}
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

}  // namespace us
