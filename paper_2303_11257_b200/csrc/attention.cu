// Fused scaled dot-product attention, forward (appendix "Unit scaling and attention"; paragraph
// "Softmax (followed by matmul)"): per (sequence, head) problem
//     S = alpha_scores * Q K^T,   P = softmax_scale * softmax(S) per row,   C = alpha_context * P V
// in ONE persistent kernel (one CTA per SM walks the tiles).  A tile is 128 query rows of one problem and
// all of its (at most 512) keys:
//   * Q [128 x 64] and K [<=512 x 64] arrive by TMA (128-byte swizzle), V [<=512 x 64] behind them;
//   * tcgen05.mma (kind::f16, M = 128, N = 256, twice) leaves the whole score block, 128 x 512
//     float32, in tensor memory (all 512 columns): the scores never reach shared or global memory
//     and are never rounded;
//   * eight warps (two per TMEM lane quarter, one query row per lane, alternate 32-column chunks each)
//     make three passes over their rows in tensor memory: maximum; exponentials, written back over the
//     scores (tcgen05.st), and their sum; weights, scaled, rounded to the operand format and written
//     to shared memory in the K-major swizzled layout of an MMA A operand, a quarter of the keys (128)
//     at a time into two 32 KB buffers used in turn;
//   * as each quarter lands, a second chain of MMAs (M = 128, N = 64, K = 128 keys) multiplies it by V
//     into tensor memory columns 0..63 (whose scores are dead by then), and the same shared-memory
//     tiles leave by TMA store as the stored P the backward pass needs; a buffer is reused once its
//     MMAs and its store have read it;
//   * the eight warps scale the context and store it in the output format.
// The roles overlap across tiles: Q and K of the next tile are fetched as soon as the score MMAs have
// read the current ones, V as soon as the last context MMA has, and the weight stores of a tile drain
// while the next tile's softmax runs.
// Every wait on an mbarrier is bounded; a wait that runs out raises the status word (as in the GEMM
// kernels) and the CTA leaves after its own copies have landed and its tensor memory is freed.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/unitscale.h"
#include "common.cuh"
#include "gemm_kernel.cuh"
#include "host.h"
#include "sm100.cuh"

namespace us {
namespace {

constexpr int kAttnD = 64;                 // head width
constexpr int kAttnMaxKeys = 512;          // 128 x 512 float32 scores fill the 512 TMEM columns
constexpr int kSoftmaxWarps = 8;
constexpr int kAttnThreads = 64 + 32 * kSoftmaxWarps;   // warp 0: TMA + MMA issue; warp 1: TMEM owner; warps 2-9: softmax
constexpr uint32_t kQBytes = 128 * 128;    // 128 rows x 64 x 2 bytes
constexpr uint32_t kKeyBlockBytes = 128 * 128;   // P tile of one 64-key block: 128 rows x 128 bytes
constexpr uint32_t kQuarterBytes = 2 * kKeyBlockBytes;   // weights of 128 keys; two such buffers take the quarters of a tile in turn
constexpr uint32_t kKBytes = 512 * 128;
constexpr uint32_t kVBytes = 512 * 128;
constexpr uint32_t kAttnSmem = kQBytes + kKBytes + kVBytes + 2 * kQuarterBytes + 1024 /* alignment */ + 128 /* barriers, slots */ +
                               2048 /* row maxima and sums */;

struct AttnParams {
  int s_q, s_k;
  int q_tiles, nb1, nb0;    // 128-row query tiles per problem; problems in the inner / outer batch dimension
  float exp_scale;          // alpha_scores * log2(e)
  float softmax_scale;
  float alpha_context;
  void* c; int c_dt; int64_t c_ld, c_stride0, c_stride1;
  int op_bf16;              // operands (and stored P) are BF16 (1) or F16 (0)
  int store_p;
  uint32_t idesc_s, idesc_c;
  unsigned int* status;
  uint32_t wait_limit;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Tile n of a CTA: tiles blockIdx.x, blockIdx.x + gridDim.x, ... of q_tiles * nb1 * nb0, query tile fastest.
__device__ __forceinline__ void attn_tile_coords(const AttnParams& a, int tile, int& q0, int& b1, int& b0) {
  const int qt = tile % a.q_tiles, pr = tile / a.q_tiles;
  q0 = qt * 128; b1 = pr % a.nb1; b0 = pr / a.nb1;
}

// F8: operands (and the stored weights) are FP8 instead of 16-bit.  A head row is then 64 bytes: the TMA boxes stay 128
// bytes wide and the bytes beyond the head read as zeros, so Q and K tiles keep the 128-byte-swizzled layout (their
// MMAs stop after 64 bytes of K), a 128-byte row of weights holds 128 keys (one key block per quarter instead of
// two), and V, an MN-major operand whose rows are 128 bytes with the upper half zero, multiplies into 128 TMEM columns
// of which the first 64 are the context.
template <bool F8>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_fwd_kernel(const __grid_constant__ CUtensorMap tq, const __grid_constant__ CUtensorMap tk,
                     const __grid_constant__ CUtensorMap tv, const __grid_constant__ CUtensorMap tp, const AttnParams a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_addr(smem_raw));
  const uint32_t q_s = base, k_s = q_s + kQBytes, v_s = k_s + kKBytes, pq_s = v_s + kVBytes;
  constexpr uint32_t kData = kQBytes + kKBytes + kVBytes + 2 * kQuarterBytes;
  const uint32_t bars = base + kData;
  const uint32_t bar_qk = bars, bar_v = bars + 8, bar_s = bars + 16, bar_o = bars + 24, bar_tmem_free = bars + 32;
  auto bar_full = [&](int b) { return bars + 40u + 8u * b; };     // weights of a quarter are in buffer b
  auto bar_free = [&](int b) { return bars + 56u + 8u * b; };     // buffer b has been read by its MMAs and by its store
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + kData + 80);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + kData + 84);
  volatile float* row_max = reinterpret_cast<volatile float*>(gen + kData + 128);   // [2][128]
  volatile float* row_sum = row_max + 256;                                            // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = a.q_tiles * a.nb1 * a.nb0;
  constexpr int kBlockKeys = F8 ? 128 : 64;          // keys in a 128-byte row of weights
  constexpr int kQuarterBlocks = F8 ? 1 : 2;         // key blocks per quarter (128 keys)
  const int nkb = (a.s_k + kBlockKeys - 1) / kBlockKeys;   // key blocks with at least one key
  const int nq = (a.s_k + 127) >> 7;                 // quarters with at least one key
  const bool two_halves = a.s_k > 256;
  const uint32_t kv_bytes = (two_halves ? 2u : 1u) * 256u * 128u;

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_qk, 1); ptx::mbar_init(bar_v, 1); ptx::mbar_init(bar_s, 1); ptx::mbar_init(bar_o, 1);
    ptx::mbar_init(bar_tmem_free, kSoftmaxWarps);
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(bar_full(b), kSoftmaxWarps); ptx::mbar_init(bar_free(b), 2); }
    *abort_flag = 0;
    ptx::mbar_init_fence();
  }
  if (warp == 1) { ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA loads and both MMA chains
      auto load_qk = [&](int tile) {
        int q0, b1, b0;
        attn_tile_coords(a, tile, q0, b1, b0);
        ptx::mbar_expect_tx(bar_qk, kQBytes + kv_bytes);
        ptx::tma_load_4d(q_s, &tq, bar_qk, 0, q0, b1, b0);
        ptx::tma_load_4d(k_s, &tk, bar_qk, 0, 0, b1, b0);
        if (two_halves) ptx::tma_load_4d(k_s + 256u * 128u, &tk, bar_qk, 0, 256, b1, b0);
      };
      auto load_v = [&](int tile) {
        int q0, b1, b0;
        attn_tile_coords(a, tile, q0, b1, b0);
        ptx::mbar_expect_tx(bar_v, kv_bytes);
        ptx::tma_load_4d(v_s, &tv, bar_v, 0, 0, b1, b0);
        if (two_halves) ptx::tma_load_4d(v_s + 256u * 128u, &tv, bar_v, 0, 256, b1, b0);
      };
      bool qk_pending = false, v_pending = false;             // a load has been issued and not yet waited for ...
      uint32_t qk_phase = 0, v_phase = 0;                      // ... on this phase of its barrier
      if ((int)blockIdx.x < num_tiles) { load_qk(blockIdx.x); load_v(blockIdx.x); qk_pending = v_pending = true; }
      uint32_t fill0 = 0, fill1 = 0;                           // uses of each weight buffer so far
      bool ok = true;
      int n = 0;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++n) {
        const uint32_t ph = (uint32_t)n & 1u;
        const int next = tile + (int)gridDim.x;
        ok = wait_bounded(bar_qk, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        qk_pending = false;
        if (n > 0) {                                           // the previous tile's context has left tensor memory
          ok = wait_bounded(bar_tmem_free, ph ^ 1u, abort_flag, a.status, a.wait_limit);
          if (!ok) break;
        }
        ptx::tc_fence_after_sync();
        const uint64_t qd = ptx::smem_desc_sw128(q_s, 16, 1024);
        for (int h = 0; h < (two_halves ? 2 : 1); ++h) {
          const uint64_t kd = ptx::smem_desc_sw128(k_s + (uint32_t)h * 256u * 128u, 16, 1024);
#pragma unroll
          for (int k = 0; k < (F8 ? 2 : 4); ++k)               // 32 bytes of the head columns per MMA
            ptx::mma_ss<F8>(tmem + 256u * h, qd + 2u * k, kd + 2u * k, a.idesc_s, k > 0);
        }
        ptx::mma_commit(bar_s);
        // Q and K may be overwritten once those MMAs have read them: fetch the next tile's
        ok = wait_bounded(bar_s, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        if (next < num_tiles) { load_qk(next); qk_pending = true; qk_phase = ph ^ 1u; }
        ok = wait_bounded(bar_v, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        v_pending = false;
        // ---------------------------------------------------------------- C = P V, quarter by quarter
        for (int qd4 = 0; ok && qd4 < nq; ++qd4) {
          const int b = qd4 & 1;
          ok = wait_bounded(bar_full(b), (b ? fill1 : fill0) & 1u, abort_flag, a.status, a.wait_limit);
          if (!ok) break;
          if (b) ++fill1; else ++fill0;
          ptx::tc_fence_after_sync();
          for (int kbl = 0; kbl < kQuarterBlocks; ++kbl) {
            const int kb = kQuarterBlocks * qd4 + kbl;
            if (kb >= nkb) break;
            constexpr uint32_t kVBlock = (uint32_t)kBlockKeys * 128u;      // V rows of one key block, 128 bytes each
            const uint64_t pd = ptx::smem_desc_sw128(pq_s + (uint32_t)b * kQuarterBytes + (uint32_t)kbl * kKeyBlockBytes, 16, 1024);
            const uint64_t vd = ptx::smem_desc_sw128(v_s + (uint32_t)kb * kVBlock, kVBlock, 1024);
#pragma unroll
            for (int k = 0; k < 4; ++k)                        // 32 bytes along a P row = a quarter of the block's V rows per MMA
              ptx::mma_ss<F8>(tmem, pd + 2u * k, vd + (kVBlock / 64u) * k, a.idesc_c, (kb | k) != 0);
          }
          ptx::mma_commit(bar_free(b));                        // one of the two arrivals that free the buffer
        }
        if (!ok) break;
        ptx::mma_commit(bar_o);
        // V may be overwritten once the last of those MMAs has read it
        ok = wait_bounded(bar_o, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        if (next < num_tiles) { load_v(next); v_pending = true; v_phase = ph ^ 1u; }
      }
      if (*abort_flag) {
        // loads that were issued land before the CTA gives up its shared memory
        if (qk_pending) for (uint32_t it = 0; it < a.wait_limit && !ptx::mbar_try_wait(bar_qk, qk_phase); ++it) {}
        if (v_pending) for (uint32_t it = 0; it < a.wait_limit && !ptx::mbar_try_wait(bar_v, v_phase); ++it) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- the stored weights leave by TMA store
      uint32_t fill0 = 0, fill1 = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        int q0, b1, b0;
        attn_tile_coords(a, tile, q0, b1, b0);
        for (int qd4 = 0; ok && qd4 < nq; ++qd4) {
          const int b = qd4 & 1;
          ok = wait_bounded(bar_full(b), (b ? fill1 : fill0) & 1u, abort_flag, a.status, a.wait_limit);
          if (!ok) break;
          if (b) ++fill1; else ++fill0;
          if (a.store_p) {
            for (int kbl = 0; kbl < kQuarterBlocks; ++kbl) {
              const int kb = kQuarterBlocks * qd4 + kbl;
              if (kb < nkb)
                ptx::tma_store_4d(&tp, pq_s + (uint32_t)b * kQuarterBytes + (uint32_t)kbl * kKeyBlockBytes, kb * kBlockKeys, q0, b1, b0);
            }
            ptx::bulk_commit_group();
            ptx::bulk_wait_group_read<0>();                    // the store has read the buffer
          }
          ptx::mbar_arrive(bar_free(b));                       // the other arrival that frees it
        }
      }
      ptx::bulk_wait_group_read<0>();
    }
  } else {
    // ------------------------------------------------------------------ softmax and output
    // Two warps share each TMEM lane quarter (= 32 query rows, one per lane): warp (q, part) works on the
    // 32-column chunks c = 2 i + part of its rows, and the two exchange their partial row maximum and row
    // sum through shared memory.
    const int q = warp & 3, part = (warp - 2) >> 2, r = q * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(q * 32) << 16);
    const int c_end = 4 * nq;                                  // 32-column chunks, whole quarters
    // One sweep over this warp's chunks c = part, part + 2, ...
    auto sweep = [&](auto&& body) {
#pragma unroll 1
      for (int c = part; c < c_end; c += 2) {
        uint32_t x[32];
        ptx::tmem_ld_32x32_issue(t_row + 32u * c, x);
        ptx::tmem_ld_fence(x);
        body(c, x);
      }
    };
    // columns at and beyond s_k hold products with zero-filled key rows: they are kept out of the maximum and
    // the sum by replacing them with a very negative score, whose weight is exactly zero
    auto mask = [&](int c, uint32_t (&x)[32]) {
      if (32 * c + 32 > a.s_k) {
#pragma unroll
        for (int i = 0; i < 32; ++i) if (32 * c + i >= a.s_k) x[i] = __float_as_uint(-3.0e38f);
      }
    };
    uint32_t fill0 = 0, fill1 = 0;
    bool aborted = false;                                      // this warp gave up on a wait (it still joins the barriers below)
    int n = 0;
#pragma unroll 1
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++n) {
      const uint32_t ph = (uint32_t)n & 1u;
      const bool have_scores = !aborted && wait_bounded(bar_s, ph, abort_flag, a.status, a.wait_limit);
      // every softmax thread reaches this barrier in every tile whatever its waits returned, and the reduction
      // hands all of them the same answer, so either all or none go on to the barriers below
      if (ptx::named_barrier_any(1, 32 * kSoftmaxWarps, !have_scores)) break;
      ptx::tc_fence_after_sync();
      int q0, b1, b0;
      attn_tile_coords(a, tile, q0, b1, b0);
      float m4[4] = {-3.0e38f, -3.0e38f, -3.0e38f, -3.0e38f};
      sweep([&](int c, uint32_t (&x)[32]) {
        mask(c, x);
#pragma unroll
        for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(x[i]));
      });
      row_max[part * 128 + r] = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
      ptx::named_barrier_sync(1, 32 * kSoftmaxWarps);
      const float mk = fmaxf(row_max[r], row_max[128 + r]) * a.exp_scale;
      float s4[4] = {0.f, 0.f, 0.f, 0.f};
      sweep([&](int c, uint32_t (&x)[32]) {
        mask(c, x);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float e = ex2(fmaf(__uint_as_float(x[i]), a.exp_scale, -mk));
          s4[i & 3] += e;
          x[i] = __float_as_uint(e);
        }
        ptx::tmem_st_32x32_bits(t_row + 32u * c, x);           // the exponentials replace the scores
      });
      ptx::tmem_st_wait();
      row_sum[part * 128 + r] = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      ptx::named_barrier_sync(1, 32 * kSoftmaxWarps);
      const float inv = a.softmax_scale / (row_sum[r] + row_sum[128 + r]);
      const uint32_t row_off = (uint32_t)r * 128u, sw = (uint32_t)(r & 7);
      // weights, a quarter (128 keys, four chunks, two of them this warp's) at a time into the two buffers in turn
#pragma unroll 1
      for (int qd4 = 0; qd4 < nq && !aborted; ++qd4) {
        const int b = qd4 & 1;
        bool free_ok = wait_bounded(bar_free(b), ((b ? fill1 : fill0) & 1u) ^ 1u, abort_flag, a.status, a.wait_limit);
        free_ok = __all_sync(0xffffffffu, free_ok);
        if (!free_ok) { aborted = true; break; }
        if (b) ++fill1; else ++fill0;
#pragma unroll 1
        for (int c = 4 * qd4 + part; c < 4 * qd4 + 4 && c < c_end; c += 2) {
          float v[32];
          ptx::tmem_ld_32x32(t_row + 32u * c, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] *= inv;
          if (F8) {
            // one key block per quarter; this chunk's 32 weights are bytes 32 (c & 3) .. + 31 of the row
            const uint32_t blk = pq_s + (uint32_t)b * kQuarterBytes + row_off;
#pragma unroll
            for (int g = 0; g < 2; ++g) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                w[j] = cvt_fp8x4<false>(v[16 * g + 4 * j], v[16 * g + 4 * j + 1], v[16 * g + 4 * j + 2], v[16 * g + 4 * j + 3]);
              const uint32_t chunk16 = (uint32_t)((c & 3) * 2 + g);
              ptx::sts128(blk + ((chunk16 ^ sw) << 4), make_uint4(w[0], w[1], w[2], w[3]));
            }
          } else {
            const uint32_t blk = pq_s + (uint32_t)b * kQuarterBytes + (uint32_t)((c >> 1) & 1) * kKeyBlockBytes + row_off;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                w[j] = a.op_bf16 ? pack_bf16x2(v[8 * g + 2 * j], v[8 * g + 2 * j + 1]) : pack_f16x2(v[8 * g + 2 * j], v[8 * g + 2 * j + 1]);
              const uint32_t chunk16 = (uint32_t)((c & 1) * 4 + g);
              ptx::sts128(blk + ((chunk16 ^ sw) << 4), make_uint4(w[0], w[1], w[2], w[3]));
            }
          }
        }
        ptx::fence_proxy_async_smem();                         // the MMA and the TMA store read these bytes
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_full(b));
      }
      if (aborted) continue;
      // ---------------------------------------------------------------- context: this warp's 32 of the 64 columns
      bool ok = wait_bounded(bar_o, ph, abort_flag, a.status, a.wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { aborted = true; continue; }
      ptx::tc_fence_after_sync();
      {
        const int row = q0 + r;
        const int es = dtype_size(a.c_dt);
        char* dst = static_cast<char*>(a.c) +
                    ((int64_t)b0 * a.c_stride0 + (int64_t)b1 * a.c_stride1 + (int64_t)row * a.c_ld + 32 * part) * es;
        float v[32];
        ptx::tmem_ld_32x32(t_row + 32u * part, v);
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_tmem_free);        // the next tile's scores may overwrite the context
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= a.alpha_context;
        if (row < a.s_q) store_vec<32>(dst, a.c_dt, v);
      }
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) { ptx::tc_fence_after_sync(); ptx::tmem_dealloc(tmem, 512); }
}

// ---------------------------------------------------------------------------------------------------------------
// Backward pass down to the queries, one persistent kernel of the same shape as the forward one: per tile of 128
// query rows
//     dP = beta_p * dC V^T            score-sized, float32 in tensor memory only (never stored, never rounded)
//     dS = k * P (dP - sum_j P_j dP_j / alpha)     the scaled-softmax gradient, from the forward pass's stored P
//     dQ = beta_q * dS K
// dC [128 x 64] and V arrive by TMA, the MMAs of dC V^T fill the 512 TMEM columns; the tile of P (128 x 512, the layout
// the forward kernel stored it from) arrives in shared memory; eight warps pass twice over their rows (row sums of
// P dP; then dS, rounded and written over P in place); K replaces V in its buffer as soon as the first MMA chain has
// read V, and a second chain multiplies dS (A operand, from the same shared-memory tile) by K into TMEM columns
// 0..63; the tile of dS leaves by TMA store (the dK matmul reads it), the eight warps scale and store dQ.
struct AttnBwdParams {
  int s_q, s_k;
  int q_tiles, nb1, nb0;
  float inv_alpha;          // 1 / softmax_alpha
  float ds_scale;           // softmax_beta * beta_p / softmax_alpha
  float beta_q;
  void* dq; int dq_dt; int64_t dq_ld, dq_stride0, dq_stride1;
  int op_bf16;
  uint32_t idesc_s, idesc_c;
  unsigned int* status;
  uint32_t wait_limit;
};

constexpr uint32_t kTileBytes = 8 * kKeyBlockBytes;      // a 128 x 512 tile of 16-bit weights: 128 KB
constexpr uint32_t kAttnBwdSmem = kQBytes + kKBytes + kTileBytes + 1024 + 128 + 1024;

// F8: dC and dS are E5M2 (gradients), P, K and V E4M3 (activations); layouts as in the forward kernel's FP8 form
// (a 128-byte row of P / dS holds 128 keys; dC, V and K rows are 64 bytes in 128-byte boxes whose upper half is zero).
template <bool F8>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_bwd_kernel(const __grid_constant__ CUtensorMap tdc, const __grid_constant__ CUtensorMap tv,
                     const __grid_constant__ CUtensorMap tk, const __grid_constant__ CUtensorMap tp,
                     const __grid_constant__ CUtensorMap tds, const AttnBwdParams a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_addr(smem_raw));
  const uint32_t dc_s = base, kv_s = dc_s + kQBytes, ps_s = kv_s + kKBytes;
  constexpr uint32_t kData = kQBytes + kKBytes + kTileBytes;
  const uint32_t bars = base + kData;
  const uint32_t bar_in = bars, bar_pin = bars + 8, bar_dp = bars + 16, bar_k = bars + 24, bar_ds = bars + 32,
                 bar_dq = bars + 40, bar_tmem_free = bars + 48;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + kData + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + kData + 68);
  volatile float* row_sum = reinterpret_cast<volatile float*>(gen + kData + 128);     // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = a.q_tiles * a.nb1 * a.nb0;
  constexpr int kBlockKeys = F8 ? 128 : 64;          // keys in a 128-byte row of P / dS
  const int nkb = (a.s_k + kBlockKeys - 1) / kBlockKeys;
  const bool two_halves = a.s_k > 256;
  const uint32_t kv_bytes = (two_halves ? 2u : 1u) * 256u * 128u;
  auto coords = [&](int tile, int& q0, int& b1, int& b0) {
    const int qt = tile % a.q_tiles, pr = tile / a.q_tiles;
    q0 = qt * 128; b1 = pr % a.nb1; b0 = pr / a.nb1;
  };

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_in, 1); ptx::mbar_init(bar_pin, 1); ptx::mbar_init(bar_dp, 1); ptx::mbar_init(bar_k, 1);
    ptx::mbar_init(bar_ds, kSoftmaxWarps); ptx::mbar_init(bar_dq, 1); ptx::mbar_init(bar_tmem_free, kSoftmaxWarps);
    *abort_flag = 0;
    ptx::mbar_init_fence();
  }
  if (warp == 1) { ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA loads and both MMA chains
      auto load_in = [&](int tile) {                           // dC tile and V
        int q0, b1, b0;
        coords(tile, q0, b1, b0);
        ptx::mbar_expect_tx(bar_in, kQBytes + kv_bytes);
        ptx::tma_load_4d(dc_s, &tdc, bar_in, 0, q0, b1, b0);
        ptx::tma_load_4d(kv_s, &tv, bar_in, 0, 0, b1, b0);
        if (two_halves) ptx::tma_load_4d(kv_s + 256u * 128u, &tv, bar_in, 0, 256, b1, b0);
      };
      // phase of the latest load issued on each barrier (a wait on a phase that has completed returns at once)
      bool in_issued = false, k_issued = false;
      uint32_t in_phase = 0, k_phase = 0;
      if ((int)blockIdx.x < num_tiles) { load_in(blockIdx.x); in_issued = true; }
      bool ok = true;
      int n = 0;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++n) {
        const uint32_t ph = (uint32_t)n & 1u;
        const int next = tile + (int)gridDim.x;
        int q0, b1, b0;
        coords(tile, q0, b1, b0);
        ok = wait_bounded(bar_in, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        if (n > 0) {                                           // the previous tile's dQ has left tensor memory
          ok = wait_bounded(bar_tmem_free, ph ^ 1u, abort_flag, a.status, a.wait_limit);
          if (!ok) break;
        }
        ptx::tc_fence_after_sync();
        const uint64_t cd = ptx::smem_desc_sw128(dc_s, 16, 1024);
        for (int h = 0; h < (two_halves ? 2 : 1); ++h) {
          const uint64_t vd = ptx::smem_desc_sw128(kv_s + (uint32_t)h * 256u * 128u, 16, 1024);
#pragma unroll
          for (int k = 0; k < (F8 ? 2 : 4); ++k) ptx::mma_ss<F8>(tmem + 256u * h, cd + 2u * k, vd + 2u * k, a.idesc_s, k > 0);
        }
        ptx::mma_commit(bar_dp);
        // V has been read: K takes its place
        ok = wait_bounded(bar_dp, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        ptx::mbar_expect_tx(bar_k, kv_bytes);
        ptx::tma_load_4d(kv_s, &tk, bar_k, 0, 0, b1, b0);
        if (two_halves) ptx::tma_load_4d(kv_s + 256u * 128u, &tk, bar_k, 0, 256, b1, b0);
        k_issued = true; k_phase = ph;
        ok = wait_bounded(bar_k, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        ok = wait_bounded(bar_ds, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        for (int kb = 0; kb < nkb; ++kb) {
          constexpr uint32_t kKBlock = (uint32_t)kBlockKeys * 128u;        // K rows of one key block, 128 bytes each
          const uint64_t sd = ptx::smem_desc_sw128(ps_s + (uint32_t)kb * kKeyBlockBytes, 16, 1024);
          const uint64_t kd = ptx::smem_desc_sw128(kv_s + (uint32_t)kb * kKBlock, kKBlock, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) ptx::mma_ss<F8>(tmem, sd + 2u * k, kd + (kKBlock / 64u) * k, a.idesc_c, (kb | k) != 0);
        }
        ptx::mma_commit(bar_dq);
        // dC, K and (for the MMAs) the dS tile have been read once those MMAs are done
        ok = wait_bounded(bar_dq, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        if (next < num_tiles) { load_in(next); in_phase = ph ^ 1u; }
      }
      if (*abort_flag) {
        // loads that were issued land before the CTA gives up its shared memory
        if (in_issued) for (uint32_t it = 0; it < a.wait_limit && !ptx::mbar_try_wait(bar_in, in_phase); ++it) {}
        if (k_issued) for (uint32_t it = 0; it < a.wait_limit && !ptx::mbar_try_wait(bar_k, k_phase); ++it) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- the weight tile: P in by TMA load, dS out by TMA store
      auto load_p = [&](int tile) {                            // key block by key block
        int q0, b1, b0;
        coords(tile, q0, b1, b0);
        ptx::mbar_expect_tx(bar_pin, (uint32_t)nkb * kKeyBlockBytes);
        for (int kb = 0; kb < nkb; ++kb) ptx::tma_load_4d(ps_s + (uint32_t)kb * kKeyBlockBytes, &tp, bar_pin, kb * kBlockKeys, q0, b1, b0);
      };
      bool ok = true, p_issued = false;
      uint32_t p_phase = 0;
      if ((int)blockIdx.x < num_tiles) { load_p(blockIdx.x); p_issued = true; }
      int n = 0;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++n) {
        const uint32_t ph = (uint32_t)n & 1u;
        const int next = tile + (int)gridDim.x;
        int q0, b1, b0;
        coords(tile, q0, b1, b0);
        ok = wait_bounded(bar_ds, ph, abort_flag, a.status, a.wait_limit);
        if (!ok) break;
        for (int kb = 0; kb < nkb; ++kb) ptx::tma_store_4d(&tds, ps_s + (uint32_t)kb * kKeyBlockBytes, kb * kBlockKeys, q0, b1, b0);
        ptx::bulk_commit_group();
        ptx::bulk_wait_group_read<0>();                        // the store has read the tile ...
        ok = wait_bounded(bar_dq, ph, abort_flag, a.status, a.wait_limit);     // ... and so have the dQ MMAs
        if (!ok) break;
        if (next < num_tiles) { load_p(next); p_phase = ph ^ 1u; }
      }
      ptx::bulk_wait_group_read<0>();
      if (*abort_flag && p_issued)
        for (uint32_t it = 0; it < a.wait_limit && !ptx::mbar_try_wait(bar_pin, p_phase); ++it) {}
    }
  } else {
    // ------------------------------------------------------------------ softmax gradient and dQ
    const int q = warp & 3, part = (warp - 2) >> 2, r = q * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(q * 32) << 16);
    const int c_end = (kBlockKeys / 32) * nkb;                 // 32-column chunks, whole key blocks
    const uint32_t row_off = (uint32_t)r * 128u, sw = (uint32_t)(r & 7);
    constexpr int kPieces = F8 ? 2 : 4;                        // 16-byte pieces of a chunk: 16 FP8 or 8 16-bit values each
    auto p_addr = [&](int c, int g) {                          // piece g of chunk c of this row
      const int per_block = kBlockKeys / 32;                   // chunks in a key block
      return ps_s + (uint32_t)(c / per_block) * kKeyBlockBytes + row_off +
             ((((uint32_t)((c % per_block) * kPieces + g)) ^ sw) << 4);
    };
    // the values of one piece as floats (8, or 16 for FP8)
    auto piece_values = [&](const uint4& raw, float (&pv)[16]) {
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (F8) {
          const float2 lo = unpack_fp8x2((uint16_t)(w[j] & 0xffffu), false), hi = unpack_fp8x2((uint16_t)(w[j] >> 16), false);
          pv[4 * j] = lo.x; pv[4 * j + 1] = lo.y; pv[4 * j + 2] = hi.x; pv[4 * j + 3] = hi.y;
        } else {
          const float2 f = a.op_bf16 ? unpack_bf16x2(w[j]) : unpack_f16x2(w[j]);
          pv[2 * j] = f.x; pv[2 * j + 1] = f.y;
        }
      }
    };
    constexpr int kPieceVals = F8 ? 16 : 8;
    bool aborted = false;
    int n = 0;
#pragma unroll 1
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++n) {
      const uint32_t ph = (uint32_t)n & 1u;
      const bool have = !aborted && wait_bounded(bar_dp, ph, abort_flag, a.status, a.wait_limit) &&
                        wait_bounded(bar_pin, ph, abort_flag, a.status, a.wait_limit);
      if (ptx::named_barrier_any(1, 32 * kSoftmaxWarps, !have)) break;
      ptx::tc_fence_after_sync();
      int q0, b1, b0;
      coords(tile, q0, b1, b0);
      // pass 1: sum_j P_j dP_j over this warp's chunks (columns beyond s_k hold zeros in both factors)
      float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
      for (int c = part; c < c_end; c += 2) {
        float x[32];
        ptx::tmem_ld_32x32(t_row + 32u * c, x);
#pragma unroll
        for (int g = 0; g < kPieces; ++g) {
          float pv[16];
          piece_values(ptx::lds128(p_addr(c, g)), pv);
#pragma unroll
          for (int i = 0; i < kPieceVals; ++i) s4[i & 3] = fmaf(pv[i], x[kPieceVals * g + i], s4[i & 3]);
        }
      }
      row_sum[part * 128 + r] = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      ptx::named_barrier_sync(1, 32 * kSoftmaxWarps);
      const float mean = (row_sum[r] + row_sum[128 + r]) * a.inv_alpha;     // sum_j p_j dP_j in units of the raw accumulator
      // pass 2: dS = ds_scale * P * (dP - mean), rounded, over P in place
#pragma unroll 1
      for (int c = part; c < c_end; c += 2) {
        float x[32];
        ptx::tmem_ld_32x32(t_row + 32u * c, x);
#pragma unroll
        for (int g = 0; g < kPieces; ++g) {
          const uint32_t addr = p_addr(c, g);
          float pv[16], d[16];
          piece_values(ptx::lds128(addr), pv);
#pragma unroll
          for (int i = 0; i < kPieceVals; ++i) d[i] = a.ds_scale * pv[i] * (x[kPieceVals * g + i] - mean);
          uint32_t o[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (F8) o[j] = cvt_fp8x4<true>(d[4 * j], d[4 * j + 1], d[4 * j + 2], d[4 * j + 3]);     // gradients: E5M2
            else o[j] = a.op_bf16 ? pack_bf16x2(d[2 * j], d[2 * j + 1]) : pack_f16x2(d[2 * j], d[2 * j + 1]);
          }
          ptx::sts128(addr, make_uint4(o[0], o[1], o[2], o[3]));
        }
      }
      ptx::fence_proxy_async_smem();                           // the MMA and the TMA store read these bytes
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_ds);
      // ---------------------------------------------------------------- dQ: this warp's 32 of the 64 columns
      bool ok = wait_bounded(bar_dq, ph, abort_flag, a.status, a.wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { aborted = true; continue; }
      ptx::tc_fence_after_sync();
      {
        const int row = q0 + r;
        const int es = dtype_size(a.dq_dt);
        char* dst = static_cast<char*>(a.dq) +
                    ((int64_t)b0 * a.dq_stride0 + (int64_t)b1 * a.dq_stride1 + (int64_t)row * a.dq_ld + 32 * part) * es;
        float v[32];
        ptx::tmem_ld_32x32(t_row + 32u * part, v);
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_tmem_free);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= a.beta_q;
        if (row < a.s_q) store_vec<32>(dst, a.dq_dt, v);
      }
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) { ptx::tc_fence_after_sync(); ptx::tmem_dealloc(tmem, 512); }
}

// 4-d map (column, row, inner problem index, outer problem index) over elements of es bytes (2, or 1 for FP8); box of 128
// bytes (128-byte swizzle) x box_rows rows of one problem; columns of a box beyond the matrix read as zeros.
static bool attn_tmap(CUtensorMap* tm, const us_mat* m, const int64_t* stride, const int64_t* count, int box_rows, int es = 2) {
  host::EncodeTiledFn fn = host::encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)m->cols, (cuuint64_t)m->rows, (cuuint64_t)count[1], (cuuint64_t)count[0]};
  // a dimension of extent 1 still needs a valid (multiple of 16 bytes) stride
  const cuuint64_t s1 = count[1] > 1 ? (cuuint64_t)stride[1] * es : 16, s0 = count[0] > 1 ? (cuuint64_t)stride[0] * es : 16;
  cuuint64_t strides[3] = {(cuuint64_t)m->ld * es, s1, s0};
  cuuint32_t box[4] = {(cuuint32_t)(128 / es), (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(tm, es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16, 4, m->ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool ok16(const us_mat* m, const int64_t* stride, const int64_t* count, int es) {
  if (reinterpret_cast<uintptr_t>(m->ptr) % 16 || (m->ld * es) % 16) return false;
  for (int i = 0; i < 2; ++i)
    if (count[i] > 1 && (stride[i] * es) % 16) return false;
  return true;
}

}  // namespace
}  // namespace us

extern "C" us_status us_attention_fwd(const us_mat* Q, const us_mat* K, const us_mat* V, float alpha_scores,
                                      float softmax_scale, float alpha_context, const us_mat* C, const us_mat* P,
                                      const us_attention_batch* batch, void* ws, size_t ws_bytes, void* stream) {
  using namespace us;
  if (!Q || !K || !V || !C || !batch) return US_ERR_INVALID_ARG;
  const int64_t* cnt = batch->count;
  if (cnt[0] < 1 || cnt[1] < 1 || cnt[0] > 65535 || cnt[1] > 65535) return US_ERR_INVALID_ARG;
  const us_mat* all[5] = {Q, K, V, C, P};
  for (int i = 0; i < 5; ++i) {
    const us_mat* m = all[i];
    if (!m) continue;
    if (m->rows < 0 || m->cols < 0 || m->ld < m->cols) return US_ERR_INVALID_ARG;
    if (m->rows * m->cols > 0 && !m->ptr) return US_ERR_INVALID_ARG;
  }
  const int64_t s_q = Q->rows, s_k = K->rows;
  if (K->cols != Q->cols || V->cols != Q->cols || V->rows != s_k || C->rows != s_q || C->cols != Q->cols)
    return US_ERR_INVALID_ARG;
  if (P && (P->rows != s_q || P->cols != s_k)) return US_ERR_INVALID_ARG;
  if (!(alpha_scores > 0.f) || !(softmax_scale > 0.f)) return US_ERR_INVALID_ARG;
  const int64_t* strides[5] = {batch->q_stride, batch->k_stride, batch->v_stride, batch->c_stride, batch->p_stride};
  for (int i = 0; i < 5; ++i)
    for (int j = 0; j < 2; ++j)
      if (all[i] && cnt[j] > 1 && strides[i][j] <= 0) return US_ERR_INVALID_ARG;
  const bool h16 = (Q->dtype == US_BF16 || Q->dtype == US_F16) && K->dtype == Q->dtype && V->dtype == Q->dtype;
  const bool f8 = Q->dtype == US_E4M3 && K->dtype == US_E4M3 && V->dtype == US_E4M3;       // activations: E4M3
  if (!(h16 || f8) || (P && P->dtype != Q->dtype)) return US_ERR_UNSUPPORTED;
  const int es = f8 ? 1 : 2;
  if (C->dtype < US_F32 || C->dtype > US_E5M2) return US_ERR_UNSUPPORTED;
  if (Q->cols != kAttnD || s_k > kAttnMaxKeys) return US_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < us_workspace_bytes()) return US_ERR_WORKSPACE;
  if (s_q == 0 || s_k == 0) return s_k == 0 && s_q > 0 ? US_ERR_INVALID_ARG : US_OK;   // a softmax over no keys is undefined
  const int c_es = (int)dtype_size(C->dtype);
  if (!ok16(Q, batch->q_stride, cnt, es) || !ok16(K, batch->k_stride, cnt, es) || !ok16(V, batch->v_stride, cnt, es) ||
      !ok16(C, batch->c_stride, cnt, c_es) || (P && !ok16(P, batch->p_stride, cnt, es)))
    return US_ERR_ALIGNMENT;

  CUtensorMap tq, tk, tv, tp;
  if (!attn_tmap(&tq, Q, batch->q_stride, cnt, 128, es) || !attn_tmap(&tk, K, batch->k_stride, cnt, 256, es) ||
      !attn_tmap(&tv, V, batch->v_stride, cnt, 256, es))
    return US_ERR_CUDA;
  tp = tq;
  if (P && !attn_tmap(&tp, P, batch->p_stride, cnt, 128, es)) return US_ERR_CUDA;

  AttnParams a{};
  a.s_q = (int)s_q; a.s_k = (int)s_k;
  a.exp_scale = alpha_scores * 1.4426950408889634f;
  a.softmax_scale = softmax_scale;
  a.alpha_context = alpha_context;
  a.c = C->ptr; a.c_dt = C->dtype; a.c_ld = C->ld;
  a.c_stride0 = cnt[0] > 1 ? batch->c_stride[0] : 0; a.c_stride1 = cnt[1] > 1 ? batch->c_stride[1] : 0;
  a.op_bf16 = Q->dtype == US_BF16;
  a.store_p = P != nullptr;
  const int fmt = f8 ? 0 : a.op_bf16 ? 1 : 0;           // kind::f8f6f4: 0 = E4M3; kind::f16: 0 = F16, 1 = BF16
  a.idesc_s = make_idesc(fmt, fmt, false, false, 128, 256);
  a.idesc_c = make_idesc(fmt, fmt, false, true, 128, f8 ? 128 : 64);   // FP8: V rows are 128 bytes, the upper half zero
  a.status = static_cast<unsigned int*>(ws);
  a.wait_limit = kWaitLimit;

  auto kern = f8 ? attention_fwd_kernel<true> : attention_fwd_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmem) != cudaSuccess)
    return US_ERR_CUDA;
  a.q_tiles = (int)((s_q + 127) / 128); a.nb1 = (int)cnt[1]; a.nb0 = (int)cnt[0];
  const int64_t tiles = (int64_t)a.q_tiles * cnt[1] * cnt[0];
  if (tiles > 0x7fffffff) return US_ERR_INVALID_ARG;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);    // persistent: one CTA per SM walks the tiles
  kern<<<grid, kAttnThreads, kAttnSmem, static_cast<cudaStream_t>(stream)>>>(tq, tk, tv, tp, a);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

extern "C" us_status us_attention_bwd(const us_mat* dC, const us_mat* P, const us_mat* K, const us_mat* V, float beta_p,
                                      float softmax_alpha, float softmax_beta, float beta_q, const us_mat* dS,
                                      const us_mat* dQ, const us_attention_bwd_batch* batch, void* ws, size_t ws_bytes,
                                      void* stream) {
  using namespace us;
  if (!dC || !P || !K || !V || !dS || !dQ || !batch) return US_ERR_INVALID_ARG;
  const int64_t* cnt = batch->count;
  if (cnt[0] < 1 || cnt[1] < 1 || cnt[0] > 65535 || cnt[1] > 65535) return US_ERR_INVALID_ARG;
  const us_mat* all[6] = {dC, P, K, V, dS, dQ};
  const int64_t* strides[6] = {batch->dc_stride, batch->p_stride, batch->k_stride, batch->v_stride, batch->ds_stride,
                               batch->dq_stride};
  for (int i = 0; i < 6; ++i) {
    const us_mat* m = all[i];
    if (m->rows < 0 || m->cols < 0 || m->ld < m->cols) return US_ERR_INVALID_ARG;
    if (m->rows * m->cols > 0 && !m->ptr) return US_ERR_INVALID_ARG;
    for (int j = 0; j < 2; ++j)
      if (cnt[j] > 1 && strides[i][j] <= 0) return US_ERR_INVALID_ARG;
  }
  const int64_t s_q = dC->rows, s_k = K->rows;
  if (K->cols != dC->cols || V->cols != dC->cols || V->rows != s_k || P->rows != s_q || P->cols != s_k || dS->rows != s_q ||
      dS->cols != s_k || dQ->rows != s_q || dQ->cols != dC->cols)
    return US_ERR_INVALID_ARG;
  if (!(softmax_alpha > 0.f)) return US_ERR_INVALID_ARG;
  const bool h16 = (dC->dtype == US_BF16 || dC->dtype == US_F16) && K->dtype == dC->dtype && V->dtype == dC->dtype &&
                   P->dtype == dC->dtype && dS->dtype == dC->dtype;
  const bool f8 = dC->dtype == US_E5M2 && dS->dtype == US_E5M2 && P->dtype == US_E4M3 && K->dtype == US_E4M3 &&
                  V->dtype == US_E4M3;                 // gradients E5M2, activations E4M3
  if (!(h16 || f8)) return US_ERR_UNSUPPORTED;
  const int es = f8 ? 1 : 2;
  if (dQ->dtype < US_F32 || dQ->dtype > US_E5M2) return US_ERR_UNSUPPORTED;
  if (dC->cols != kAttnD || s_k > kAttnMaxKeys) return US_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < us_workspace_bytes()) return US_ERR_WORKSPACE;
  if (s_q == 0 || s_k == 0) return US_OK;              // no queries: nothing to do; no keys: dS is empty and dQ is not written
  const int q_es = (int)dtype_size(dQ->dtype);
  for (int i = 0; i < 5; ++i)
    if (!ok16(all[i], strides[i], cnt, es)) return US_ERR_ALIGNMENT;
  if (!ok16(dQ, batch->dq_stride, cnt, q_es)) return US_ERR_ALIGNMENT;

  CUtensorMap tdc, tv, tk, tp, tds;
  if (!attn_tmap(&tdc, dC, batch->dc_stride, cnt, 128, es) || !attn_tmap(&tv, V, batch->v_stride, cnt, 256, es) ||
      !attn_tmap(&tk, K, batch->k_stride, cnt, 256, es) || !attn_tmap(&tp, P, batch->p_stride, cnt, 128, es) ||
      !attn_tmap(&tds, dS, batch->ds_stride, cnt, 128, es))
    return US_ERR_CUDA;

  AttnBwdParams a{};
  a.s_q = (int)s_q; a.s_k = (int)s_k;
  a.q_tiles = (int)((s_q + 127) / 128); a.nb1 = (int)cnt[1]; a.nb0 = (int)cnt[0];
  a.inv_alpha = 1.0f / softmax_alpha;
  a.ds_scale = softmax_beta * beta_p / softmax_alpha;
  a.beta_q = beta_q;
  a.dq = dQ->ptr; a.dq_dt = dQ->dtype; a.dq_ld = dQ->ld;
  a.dq_stride0 = cnt[0] > 1 ? batch->dq_stride[0] : 0; a.dq_stride1 = cnt[1] > 1 ? batch->dq_stride[1] : 0;
  a.op_bf16 = dC->dtype == US_BF16;
  const int fmt = a.op_bf16 ? 1 : 0;
  // FP8 (kind::f8f6f4: 0 = E4M3, 1 = E5M2): the A operands dC and dS are gradients, the B operands V and K activations
  a.idesc_s = f8 ? make_idesc(1, 0, false, false, 128, 256) : make_idesc(fmt, fmt, false, false, 128, 256);
  a.idesc_c = f8 ? make_idesc(1, 0, false, true, 128, 128) : make_idesc(fmt, fmt, false, true, 128, 64);
  a.status = static_cast<unsigned int*>(ws);
  a.wait_limit = kWaitLimit;
  const int64_t tiles = (int64_t)a.q_tiles * cnt[1] * cnt[0];
  if (tiles > 0x7fffffff) return US_ERR_INVALID_ARG;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  auto kern = f8 ? attention_bwd_kernel<true> : attention_bwd_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnBwdSmem) != cudaSuccess)
    return US_ERR_CUDA;
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  kern<<<grid, kAttnThreads, kAttnBwdSmem, static_cast<cudaStream_t>(stream)>>>(tdc, tv, tk, tp, tds, a);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}
