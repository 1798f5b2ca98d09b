// The unit-scaled GEMM of libunitscale for sm_100a.
//
//   out[M x N] = epilogue( scale * sum_k A(m, k) B(n, k) )
//
// One persistent CTA per SM.  A CTA walks over 128 x BN output tiles on its own, or a cluster of
// two CTAs (cta_group::2) walks over 256 x BN tiles: each CTA then loads only its half of the B
// tile, which cuts the operand bytes per tensor-core cycle by a third.  Warp roles:
//   warp 0   TMA producer: fills a ring of shared-memory stages (one 128-byte-swizzled
//            A tile + B tile per stage, 128 bytes of K each) with cp.async.bulk.tensor;
//   warp 1   MMA issuer: one thread issues tcgen05.mma (4 per stage) into one of two
//            float32 accumulators in tensor memory, commits stage release and
//            accumulator-ready barriers; the warp owns the TMEM allocation;
//   warps 2-9 epilogue: tcgen05.ld 32-column slices of their 32-lane quarter of the finished
//            accumulator (two warps per quarter), apply scale / GELU / GELU-gradient /
//            residual, round once, store.
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

// Division of a non-negative int below 2^31 by a divisor fixed at launch: one multiply-high, one
// add and one shift instead of the ~30-instruction sequence of a hardware-less integer divide, which
// every epilogue warp would otherwise run several times per tile.  mul = floor(2^32 (2^shift - d) / d) + 1,
// shift = ceil(log2 d); floor(n / d) = (mulhi(n, mul) + n) >> shift.
struct FastDiv {
  uint32_t mul, shift;
  __device__ __forceinline__ int div(int n) const { return (int)((__umulhi((uint32_t)n, mul) + (uint32_t)n) >> shift); }
};
inline FastDiv make_fast_div(int d) {
  FastDiv f;
  uint32_t l = 0;
  while ((1ll << l) < d) ++l;
  f.shift = l;
  f.mul = (uint32_t)((((1ull << l) - (uint64_t)d) << 32) / (uint64_t)d + 1ull);
  return f;
}

struct GemmParams {
  int M, N, K;
  int tiles_m, tiles_n;
  int band_m;                               // tile rows per band of the tile order (see tile_mn)
  int nb0, nb1;                             // batch counts (outer, inner); 1, 1 for a single problem
  int full_bands;                           // bands that have band_m tile rows; a last, shorter one may follow
  FastDiv d_problem, d_band, d_rows, d_rows_last, d_nb1;   // by tiles_m * tiles_n, band_m * tiles_n, band_m, tiles_m % band_m, nb1
  float scale;
  uint32_t idesc;
  void* out; int out_dt; int64_t out_ld;
  int act; float act_in, act_out;          // act: US_ACT_NONE, or the forward / gradient class as US_ACT_GELU / US_ACT_GELU_GRAD
  int fn;                                   // us_fn of the activation (US_FN_GELU for the GELU pair)
  void* aux; int aux_dt; int64_t aux_ld;
  const void* skip; int skip_dt; int64_t skip_ld; float skip_coef, out_coef;
  unsigned int* status;
  uint32_t wait_limit;                      // polls a bounded wait makes before it gives up (kWaitLimit unless a test shortens it)
  int no_loads;                             // test hook: the producer issues no operand loads, so that the waits run out
};

constexpr int kBM = 128;                 // tile rows = TMEM lanes
constexpr int kStageKBytes = 128;        // bytes of K per stage = one swizzle atom
constexpr int kKSteps = 4;               // MMAs per stage (32 bytes of K each)
constexpr int kEpilogueWarps = 8;           // default: two per TMEM lane quarter
// Epilogue warps EW of a kernel: 8, or 16 for the ALU-heavy GELU epilogues with FP8 output (four
// per lane quarter, 64 columns each), which need more warps in flight to keep the pipes busy.
__host__ __device__ constexpr int gemm_threads(int ew) { return 64 + 32 * ew; }
// Staging per epilogue warp: EW = 8: two 32-row x 128-byte boxes; EW = 16: one such box (stored
// pre-activation in or out, 64 columns of 16 bits) and one 32-row x 64-byte box (64 FP8 outputs).
__host__ __device__ constexpr int epi_warp_bytes(int ew) { return ew == 16 ? 4096 + 2048 : 8192; }

// What the epilogue fuses, fixed at compile time so that each kernel carries one code path only.
enum EpiKind {
  kEpiPlain = 0,     // scale, round, store
  kEpiGelu = 1,      // + scaled GELU, optionally keeping the 16-bit pre-activation
  kEpiGeluGrad = 2,  // + scaled GELU gradient from the stored pre-activation
  kEpiSkip = 3,      // + weighted skip tensor (residual)
  kEpiLegacy = 4     // any other combination: direct global accesses, runtime switches
};
constexpr uint32_t kWaitLimit = 1u << 22;
constexpr unsigned int kStatusTimeout = 1;

// Shared-memory plan of one CTA.  CG = CTAs cooperating on a tile (1, or 2 = cta_group::2 pair):
// a pair computes 256 x BN, each CTA holding its 128 rows of A and its BN/2 rows of B.
template <int BN, int CG, int EW>
struct GemmSmem {
  static constexpr int kABytes = kBM * kStageKBytes;
  static constexpr int kBBytes = (BN / CG) * kStageKBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiBytes = EW * epi_warp_bytes(EW);          // 64 KB (EW = 8) or 96 KB (EW = 16)
  static constexpr int kStages = (229376 - kEpiBytes) / kStageBytes; // 32 KB stages: 5 (EW = 8) or 4 (EW = 16)
  static constexpr int kBarrierBytes = 512;
  static constexpr int kTotal = kStages * kStageBytes + kEpiBytes + kBarrierBytes + 1024;  // + alignment slack
};

// Tile order.  Tiles that run at the same time (consecutive indices) should share operand panels
// in L2: tiles are walked in bands of band_m tile-rows, down the band first and then across.  With
// band_m = tiles_m this is plain column-major order (all of A stays resident in L2 while B streams
// through once); when A is too large for that the host picks band_m = 8, so that a wave of ~74
// tiles touches 8 row panels of A and ~9 column panels of B.
__device__ __forceinline__ void tile_mn(const GemmParams& p, int tile, int& tm, int& tn) {
  tile -= p.d_problem.div(tile) * (p.tiles_m * p.tiles_n);   // position inside its problem of the batch
  const int band = p.d_band.div(tile);
  const int first_m = band * p.band_m;
  const bool last = band >= p.full_bands;
  const int rows = last ? p.tiles_m - first_m : p.band_m;
  const int r = tile - band * (p.band_m * p.tiles_n);
  tn = last ? p.d_rows_last.div(r) : p.d_rows.div(r);
  tm = first_m + r - tn * rows;
}
__device__ __forceinline__ int tile_m(const GemmParams& p, int tile) { int tm, tn; tile_mn(p, tile, tm, tn); return tm; }
__device__ __forceinline__ int tile_n(const GemmParams& p, int tile) { int tm, tn; tile_mn(p, tile, tm, tn); return tn; }
// Batched problems: consecutive groups of tiles_m * tiles_n tiles belong to consecutive problems,
// numbered outer * nb1 + inner.
__device__ __forceinline__ void tile_batch(const GemmParams& p, int tile, int& b0, int& b1) {
  const int b = p.d_problem.div(tile);
  b0 = p.d_nb1.div(b);
  b1 = b - b0 * p.nb1;
}

// Bounded mbarrier wait.  Returns false if the CTA is aborting (this wait or another one timed out).
// (Each attempt already suspends the thread in hardware for a while, so polling costs few issue
// slots: pausing between attempts made no measurable difference.)
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             unsigned int* status, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  if (status) atomicExch(status, kStatusTimeout);
  return false;
}

// Operands of the fused epilogue for one 32-column slice of one row, fetched as raw 16-byte
// vectors before the accumulator is read so that their latency overlaps the TMEM load.
struct EpiloguePrefetch {
  uint4 aux[4];    // 32 x 16-bit stored pre-activation (GELU-gradient only)
  uint4 skip[8];   // 32 x float32, or 32 x 16-bit in the first four
};

__device__ __forceinline__ void prefetch_full(const GemmParams& p, int64_t row, int col, EpiloguePrefetch& f) {
  if (p.act == US_ACT_GELU_GRAD) {
    const uint4* q = reinterpret_cast<const uint4*>(static_cast<const char*>(p.aux) + (row * p.aux_ld + col) * 2);
#pragma unroll
    for (int i = 0; i < 4; ++i) f.aux[i] = __ldg(q + i);
  }
  if (p.skip) {
    const int es = dtype_size(p.skip_dt);
    const uint4* q = reinterpret_cast<const uint4*>(static_cast<const char*>(p.skip) + (row * p.skip_ld + col) * es);
#pragma unroll
    for (int i = 0; i < 4; ++i) f.skip[i] = __ldg(q + i);
    if (es == 4) {
#pragma unroll
      for (int i = 4; i < 8; ++i) f.skip[i] = __ldg(q + i);
    }
  }
}

template <int N>
__device__ __forceinline__ void unpack16(const uint4* raw, int dt, float (&v)[N]) {
#pragma unroll
  for (int i = 0; i < N / 8; ++i) {
    const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 t = (dt == US_BF16) ? unpack_bf16x2(w[j]) : unpack_f16x2(w[j]);
      v[8 * i + 2 * j] = t.x; v[8 * i + 2 * j + 1] = t.y;
    }
  }
}

// Full 32-column slice of one output row, every access a 16-byte vector; v = scale * acc on entry.
__device__ __forceinline__ void epilogue_chunk_full(const GemmParams& p, float (&v)[32], const EpiloguePrefetch& f,
                                                    int64_t row, int col) {
  if (p.act == US_ACT_GELU) {
    if (p.aux) store_vec<32>(static_cast<char*>(p.aux) + (row * p.aux_ld + col) * 2, p.aux_dt, v);
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = act_scaled(p.fn, v[i], p.act_in, p.act_out);
  } else if (p.act == US_ACT_GELU_GRAD) {
    float h[32];
    unpack16<32>(f.aux, p.aux_dt, h);
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = act_grad_scaled(p.fn, h[i], v[i], p.act_in, p.act_out);
  }
  if (p.skip) {
    float sk[32];
    if (p.skip_dt == US_F32) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        sk[4 * i] = __uint_as_float(f.skip[i].x); sk[4 * i + 1] = __uint_as_float(f.skip[i].y);
        sk[4 * i + 2] = __uint_as_float(f.skip[i].z); sk[4 * i + 3] = __uint_as_float(f.skip[i].w);
      }
    } else {
      unpack16<32>(f.skip, p.skip_dt, sk);
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = fmaf(p.skip_coef, sk[i], p.out_coef * v[i]);
  }
  store_vec<32>(static_cast<char*>(p.out) + (row * p.out_ld + col) * dtype_size(p.out_dt), p.out_dt, v);
}

// Ragged 32-column slice (fewer than 32 columns inside the matrix): element-wise accesses.
__device__ __forceinline__ void epilogue_chunk_ragged(const GemmParams& p, float (&v)[32], int64_t row, int col, int ncols) {
  if (p.act == US_ACT_GELU) {
    if (p.aux) {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (i < ncols) store_one(p.aux, p.aux_dt, row * p.aux_ld + col + i, v[i]);
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = act_scaled(p.fn, v[i], p.act_in, p.act_out);
  } else if (p.act == US_ACT_GELU_GRAD) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float h = (i < ncols) ? load_one(p.aux, p.aux_dt, row * p.aux_ld + col + i) : 0.f;
      v[i] = act_grad_scaled(p.fn, h, v[i], p.act_in, p.act_out);
    }
  }
  if (p.skip) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float sk = (i < ncols) ? load_one(p.skip, p.skip_dt, row * p.skip_ld + col + i) : 0.f;
      v[i] = fmaf(p.skip_coef, sk, p.out_coef * v[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < 32; ++i)
    if (i < ncols) store_one(p.out, p.out_dt, row * p.out_ld + col + i, v[i]);
}

// Barrier addresses and identity the staged epilogue needs from the kernel.
struct EpiCtx {
  uint32_t tmem_base, acc_full0, acc_empty0, in_bar, buf0;   // buf0: this warp's two 4 KB boxes
  volatile int* abort_flag;
  int warp, lane, rank, group, num_groups, num_tiles;
};

// Epilogue through shared memory.  Each participating warp owns 32 rows x 128 columns of the
// tile and two private 32-row x 128-byte boxes (128-byte-swizzled, like the TMA maps).  A row of a
// box is written / read by the lane that owns that row, 16-byte chunk c at chunk (c ^ (row & 7)),
// which is conflict free; global memory is touched by TMA only: box loads for the stored
// pre-activation (GELU gradient) or the skip tensor, box stores for the output and for the
// pre-activation the GELU epilogue keeps.  TMA clips stores and zero-fills loads at the matrix
// edges, so ragged shapes need no special path.  No cross-warp synchronisation is involved.
template <int BN, int CG, int EPI, int EW, bool BATCHED>
__device__ __forceinline__ void epilogue_staged(const GemmParams& p, const CUtensorMap* tm_out, const CUtensorMap* tm_aux,
                                                const CUtensorMap* tm_skip, const EpiCtx& c) {
  constexpr int kWarpCols = EW == 16 ? 64 : 128;            // columns of the tile one warp handles
  constexpr bool kNarrowOut = EW == 16;                     // FP8 output box of 64 bytes per row (64-byte swizzle)
  const int q = c.warp & 3, half = (c.warp - 2) >> 2;       // lane quarter; which group of kWarpCols columns
  if (half >= BN / kWarpCols) return;                       // more warps than column groups: the rest sit out
  const int lane = c.lane;
  constexpr int in_kind = EPI == kEpiGeluGrad ? 1 : (EPI == kEpiSkip ? 2 : 0);
  const int in_dt = in_kind == 1 ? p.aux_dt : p.skip_dt;
  const int in_es = in_kind ? dtype_size(in_dt) : 4;
  const CUtensorMap* tm_in = in_kind == 1 ? tm_aux : tm_skip;
  const bool aux_out = EPI == kEpiGelu && p.aux != nullptr;
  const int out_es = dtype_size(p.out_dt);
  const int in_box_cols = 128 / in_es, out_box_cols = kNarrowOut ? 64 : 128 / out_es;
  const uint32_t buf_in = c.buf0, buf_aux = c.buf0;          // first box: input, or the kept pre-activation
  const uint32_t row_off = (uint32_t)lane * 128u;
  const uint32_t sw = (uint32_t)(lane & 7);
  // 64-byte output rows: pitch 64, 16-byte chunk c of row r at chunk c ^ ((r >> 1) & 3)
  const uint32_t out_row_off = kNarrowOut ? (uint32_t)lane * 64u : row_off;
  const uint32_t out_sw = kNarrowOut ? (uint32_t)((lane >> 1) & 3) : sw;
  uint32_t in_phase = 0;
  int plain_toggle = 0;
  uint32_t buf_out = c.buf0 + 4096u;

  auto tile_rows = [&](int tile) { return tile_m(p, tile) * (kBM * CG) + c.rank * kBM + q * 32; };
  auto tile_cols = [&](int tile) { return tile_n(p, tile) * BN + half * kWarpCols; };
  auto next_active_tile = [&](int tile) {
    while (tile < c.num_tiles && tile_cols(tile) >= p.N) tile += c.num_groups;
    return tile;
  };
  bool in_pending = false;                                   // an input box load has been issued and not yet waited for
  auto issue_in = [&](int col, int row0) {
    if (lane == 0) {
      ptx::mbar_expect_tx(c.in_bar, 4096);
      ptx::tma_load_2d(buf_in, tm_in, c.in_bar, col, row0);      // fused inputs exist for single problems only
    }
    in_pending = true;
  };
  // This warp is done reading accumulator a: its values are in registers, so the buffer is handed
  // back to the MMA warp before the arithmetic and the stores of the last slice, not after them.
  auto release_acc = [&](uint32_t a) {
    ptx::tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) {
      if (CG == 2) ptx::mbar_arrive_cluster(ptx::in_even_cta(c.acc_empty0 + 8u * a));
      else ptx::mbar_arrive(c.acc_empty0 + 8u * a);
    }
  };
  if (in_kind) {
    const int t0 = next_active_tile(c.group);
    if (t0 < c.num_tiles) issue_in(tile_cols(t0), tile_rows(t0));
  }

  uint32_t local = 0;
  bool ok = true;
  for (int tile = c.group; ok && tile < c.num_tiles; tile += c.num_groups, ++local) {
    const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
    const int row0 = tile_rows(tile), n_w = tile_cols(tile);
    ok = wait_bounded(c.acc_full0 + 8u * acc, acc_phase, c.abort_flag, p.status, p.wait_limit);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    ptx::tc_fence_after_sync();
    const uint32_t t_row = c.tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + half * kWarpCols;
    bool released = false;
    if (n_w < p.N) {
#pragma unroll 1
      for (int sl = 0; sl < kWarpCols / 32; ++sl) {
        const int col = n_w + 32 * sl;
        if (col >= p.N) break;                               // warp-uniform
        const bool last_slice = (sl == kWarpCols / 32 - 1) || (col + 32 >= p.N);
        // ---- fused-epilogue operand for this slice: read it from the input box up front, so that
        //      the box can be refilled while the slice is being computed
        uint4 raw[8];
        if (in_kind) {
          const int off = (32 * sl) & (in_box_cols - 1);       // box widths are powers of two
          if (off == 0) {
            ok = wait_bounded(c.in_bar, in_phase, c.abort_flag, p.status, p.wait_limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            in_phase ^= 1u;
            in_pending = false;
          }
          const uint32_t cb = (uint32_t)(off * in_es) >> 4;
          const int nchunk = 2 * in_es;                      // 32 values
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (j < nchunk) raw[j] = ptx::lds128(buf_in + row_off + (((cb + j) ^ sw) << 4));
          if (off + 32 == in_box_cols || last_slice) {       // box consumed: fetch the next one into it
            __syncwarp();
            if (!last_slice) {
              issue_in(col + 32, row0);
            } else {
              const int tn = next_active_tile(tile + c.num_groups);
              if (tn < c.num_tiles) issue_in(tile_cols(tn), tile_rows(tn));
            }
          }
        }
        // ---- staging boxes that start with this slice must have been read by their last TMA store
        const int aux_off = (32 * sl) & 63, out_off = (32 * sl) & (out_box_cols - 1);
        if (out_off == 0 || (aux_out && aux_off == 0)) {
          if (!in_kind && !aux_out) {                        // both boxes hold outputs, used alternately
            buf_out = c.buf0 + (plain_toggle ? 4096u : 0u);
            plain_toggle ^= 1;
            if (lane == 0) ptx::bulk_wait_group_read<1>();
          } else {
            if (lane == 0) ptx::bulk_wait_group_read<0>();
          }
          __syncwarp();
        }
        float v[32];
        ptx::tmem_ld_32x32(t_row + 32 * sl, v);
        if (last_slice) { release_acc(acc); released = true; }   // the MMA warp may refill it while this slice is worked on
        const f32x2 scale2 = splat2(p.scale), in2 = splat2(p.act_in);
        const float tail_k = fabsf(p.act_in) * (1.0f / kTailRange), act_oi = p.act_out * p.act_in;
        const f32x2 os2 = splat2(p.act_out * p.act_in), skip2 = splat2(p.skip_coef), oc2 = splat2(p.out_coef);
        const uint32_t aux_cb = (uint32_t)(aux_off * 2) >> 4, out_cb = (uint32_t)(out_off * out_es) >> 4;
        const uint32_t dst = buf_out + out_row_off;
        uint32_t held[2];                                    // first half of a 16-byte chunk of FP8 codes
        // Eight values at a time run through the whole chain (scale, kept pre-activation, activation,
        // residual, rounding, staging store), so that the different execution pipes overlap.
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          f32x2 x[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) x[k] = mul2(pack2(v[8 * g + 2 * k], v[8 * g + 2 * k + 1]), scale2);
          float y[8];
          if (EPI == kEpiGelu) {
            if (aux_out) {
              uint32_t w[4];
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                float a, b;
                unpack2(x[k], a, b);
                w[k] = p.aux_dt == US_BF16 ? pack_bf16x2(a, b) : pack_f16x2(a, b);
              }
              ptx::sts128(buf_aux + row_off + (((aux_cb + g) ^ sw) << 4), make_uint4(w[0], w[1], w[2], w[3]));
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              if (p.fn == US_FN_GELU) {
                gelu_scaled2<kNarrowOut>(x[k], tail_k, act_oi, y[2 * k], y[2 * k + 1]);
              } else {                                          // relu, tanh, sigmoid (table section "Activations")
                float a, b;
                unpack2(x[k], a, b);
                y[2 * k] = act_scaled(p.fn, a, p.act_in, p.act_out); y[2 * k + 1] = act_scaled(p.fn, b, p.act_in, p.act_out);
              }
            }
          } else if (EPI == kEpiGeluGrad) {
            const uint32_t w[4] = {raw[g].x, raw[g].y, raw[g].z, raw[g].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float2 h = in_dt == US_BF16 ? unpack_bf16x2(w[k]) : unpack_f16x2(w[k]);
              if (p.fn == US_FN_GELU) {
                unpack2(gelu_grad_scaled2(pack2(h.x, h.y), x[k], in2, os2), y[2 * k], y[2 * k + 1]);
              } else {
                float a, b;
                unpack2(x[k], a, b);
                y[2 * k] = act_grad_scaled(p.fn, h.x, a, p.act_in, p.act_out); y[2 * k + 1] = act_grad_scaled(p.fn, h.y, b, p.act_in, p.act_out);
              }
            }
          } else if (EPI == kEpiSkip) {
            float sk[8];
            if (in_dt == US_F32) {
              sk[0] = __uint_as_float(raw[2 * g].x); sk[1] = __uint_as_float(raw[2 * g].y);
              sk[2] = __uint_as_float(raw[2 * g].z); sk[3] = __uint_as_float(raw[2 * g].w);
              sk[4] = __uint_as_float(raw[2 * g + 1].x); sk[5] = __uint_as_float(raw[2 * g + 1].y);
              sk[6] = __uint_as_float(raw[2 * g + 1].z); sk[7] = __uint_as_float(raw[2 * g + 1].w);
            } else {
              const uint32_t w[4] = {raw[g].x, raw[g].y, raw[g].z, raw[g].w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float2 h = in_dt == US_BF16 ? unpack_bf16x2(w[k]) : unpack_f16x2(w[k]);
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
          // ---- rounding to the output format and staging store of these eight values
          if (p.out_dt == US_F32) {
            ptx::sts128(dst + (((out_cb + 2 * g) ^ out_sw) << 4),
                        make_uint4(__float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3])));
            ptx::sts128(dst + (((out_cb + 2 * g + 1) ^ out_sw) << 4),
                        make_uint4(__float_as_uint(y[4]), __float_as_uint(y[5]), __float_as_uint(y[6]), __float_as_uint(y[7])));
          } else if (p.out_dt == US_BF16 || p.out_dt == US_F16) {
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
              w[k] = p.out_dt == US_BF16 ? pack_bf16x2(y[2 * k], y[2 * k + 1]) : pack_f16x2(y[2 * k], y[2 * k + 1]);
            ptx::sts128(dst + (((out_cb + g) ^ out_sw) << 4), make_uint4(w[0], w[1], w[2], w[3]));
          } else {
            const uint32_t lo = p.out_dt == US_E5M2 ? cvt_fp8x4<true>(y[0], y[1], y[2], y[3]) : cvt_fp8x4<false>(y[0], y[1], y[2], y[3]);
            const uint32_t hi = p.out_dt == US_E5M2 ? cvt_fp8x4<true>(y[4], y[5], y[6], y[7]) : cvt_fp8x4<false>(y[4], y[5], y[6], y[7]);
            if ((g & 1) == 0) {
              held[0] = lo; held[1] = hi;
            } else {
              ptx::sts128(dst + (((out_cb + (g >> 1)) ^ out_sw) << 4), make_uint4(held[0], held[1], lo, hi));
            }
          }
        }
        // ---- boxes completed by this slice go out
        if (aux_out && (aux_off == 32 || last_slice)) {
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) { ptx::tma_store_2d(tm_aux, buf_aux, col - aux_off, row0); ptx::bulk_commit_group(); }
        }
        if (out_off + 32 == out_box_cols || last_slice) {
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (BATCHED) { int b0, b1; tile_batch(p, tile, b0, b1); ptx::tma_store_4d(tm_out, buf_out, col - out_off, row0, b1, b0); }
            else ptx::tma_store_2d(tm_out, buf_out, col - out_off, row0);
            ptx::bulk_commit_group();
          }
        }
      }
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    if (!released) release_acc(acc);                           // tile without columns for this warp
  }
  // Leaving early (a wait ran out somewhere in the CTA): an input box may still be in flight; let it
  // land before the CTA may give up its shared memory.
  if (in_kind && in_pending && lane == 0)
    for (uint32_t it = 0; it < p.wait_limit && !ptx::mbar_try_wait(c.in_bar, in_phase); ++it) {}
  if (lane == 0) ptx::bulk_wait_group_read<0>();             // stores have left shared memory before the CTA may exit
  __syncwarp();
}

// Epilogue of the two GELU kinds with an FP8 output, run by sixteen warps: warp (quarter q, part)
// owns the 32 rows of TMEM lane quarter q and 64 columns of the tile, as two 32-column slices.
// The per-tile chain of one warp is kept short, because with K = d_model the main loop of a tile
// lasts only a few thousand cycles:
//   * the second slice is loaded from tensor memory while the first is being worked on, and the
//     accumulator is handed back to the MMA warp as soon as both slices are in registers;
//   * the coordinates of the next tile are computed while the first load is in flight;
//   * GELU gradient: the stored pre-activation arrives as two 32-row x 64-byte boxes (one per
//     slice), each refilled for the next tile right after its slice has been read, so that a
//     load has a slice's worth of arithmetic and the tile change-over to land;
//   * one proxy fence and one bulk group per tile for all stores of the warp.
// Staging per warp (6 KB): GELU: [0, 4096) kept pre-activation, 32 rows x 128 bytes (128-byte
// swizzle), [4096, 6144) output; GELU gradient: [0, 2048) and [2048, 4096) the input boxes,
// [4096, 6144) output; 64-byte rows use the 64-byte swizzle: 16-byte chunk c of row r sits at
// chunk c ^ ((r >> 1) & 3).
template <int BN, int CG, int EPI, bool OUT_E5, bool AUX_BF16>
__device__ __forceinline__ void epilogue_act16(const GemmParams& p, const CUtensorMap* tm_out, const CUtensorMap* tm_aux,
                                               const EpiCtx& c, uint32_t in_bar1) {
  static_assert(EPI == kEpiGelu || EPI == kEpiGeluGrad, "GELU kinds only");
  constexpr bool kIn = EPI == kEpiGeluGrad;
  const int q = c.warp & 3, part = (c.warp - 2) >> 2;
  if (part >= BN / 64) return;
  const int lane = c.lane;
  const bool aux_out = EPI == kEpiGelu && p.aux != nullptr;
  const uint32_t buf_aux = c.buf0, buf_out = c.buf0 + 4096u;
  const uint32_t row128 = (uint32_t)lane * 128u, sw128 = (uint32_t)(lane & 7);
  const uint32_t row64 = (uint32_t)lane * 64u, sw64 = (uint32_t)((lane >> 1) & 3);
  const f32x2 scale2 = splat2(p.scale), in2 = splat2(p.act_in), os2 = splat2(p.act_out * p.act_in);
  const float tail_k = fabsf(p.act_in) * (1.0f / kTailRange), act_oi = p.act_out * p.act_in;

  auto coords = [&](int tile, int& row0, int& n_w) {
    int tm, tn;
    tile_mn(p, tile, tm, tn);
    row0 = tm * (kBM * CG) + c.rank * kBM + q * 32;
    n_w = tn * BN + part * 64;
  };
  auto issue_in = [&](int half, int n_w, int row0) {          // lane 0 only; a box wholly outside the matrix reads zeros
    const uint32_t bar = half ? in_bar1 : c.in_bar;
    ptx::mbar_expect_tx(bar, 2048);
    ptx::tma_load_2d(buf_aux + 2048u * half, tm_aux, bar, n_w + 32 * half, row0);
  };
  auto release_acc = [&](uint32_t a) {
    ptx::tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) {
      if (CG == 2) ptx::mbar_arrive_cluster(ptx::in_even_cta(c.acc_empty0 + 8u * a));
      else ptx::mbar_arrive(c.acc_empty0 + 8u * a);
    }
  };
  // One 32-column slice: scale, (kept pre-activation,) activation, rounding, staging stores.
  auto slice = [&](const uint32_t (&r)[32], int s) {
    uint32_t held[2];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      f32x2 x[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        x[k] = mul2(pack2(__uint_as_float(r[8 * g + 2 * k]), __uint_as_float(r[8 * g + 2 * k + 1])), scale2);
      float y[8];
      if (EPI == kEpiGelu) {
        if (aux_out) {
          uint32_t w[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            float a, b;
            unpack2(x[k], a, b);
            w[k] = AUX_BF16 ? pack_bf16x2(a, b) : pack_f16x2(a, b);
          }
          ptx::sts128(buf_aux + row128 + ((((uint32_t)(4 * s + g)) ^ sw128) << 4), make_uint4(w[0], w[1], w[2], w[3]));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) gelu_scaled2<true>(x[k], tail_k, act_oi, y[2 * k], y[2 * k + 1]);
      } else {
        const uint4 raw = ptx::lds128(buf_aux + 2048u * s + row64 + ((((uint32_t)g) ^ sw64) << 4));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 h = AUX_BF16 ? unpack_bf16x2(w[k]) : unpack_f16x2(w[k]);
          unpack2(gelu_grad_scaled2(pack2(h.x, h.y), x[k], in2, os2), y[2 * k], y[2 * k + 1]);
        }
      }
      const uint32_t lo = cvt_fp8x4<OUT_E5>(y[0], y[1], y[2], y[3]);
      const uint32_t hi = cvt_fp8x4<OUT_E5>(y[4], y[5], y[6], y[7]);
      if ((g & 1) == 0) {
        held[0] = lo; held[1] = hi;
      } else {
        ptx::sts128(buf_out + row64 + ((((uint32_t)(2 * s + (g >> 1))) ^ sw64) << 4), make_uint4(held[0], held[1], lo, hi));
      }
    }
  };

  int tile = c.group, row0 = 0, n_w = 0;
  bool pending[2] = {false, false};                          // an input box load is in flight
  if (tile < c.num_tiles) {
    coords(tile, row0, n_w);
    if (kIn) {
      if (lane == 0) { issue_in(0, n_w, row0); issue_in(1, n_w, row0); }
      pending[0] = pending[1] = true;
    }
  }
  uint32_t local = 0, ph0 = 0, ph1 = 0;                      // parities of the two input barriers
  bool ok = true;
  for (; tile < c.num_tiles; ++local) {
    const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
    ok = wait_bounded(c.acc_full0 + 8u * acc, acc_phase, c.abort_flag, p.status, p.wait_limit);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    ptx::tc_fence_after_sync();
    const uint32_t t_row = c.tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + part * 64;
    const bool active = n_w < p.N;                            // warp-uniform
    uint32_t r0[32], r1[32];
    if (active) ptx::tmem_ld_32x32_issue(t_row, r0);
    const int next = tile + c.num_groups;
    int next_row0 = 0, next_n_w = 0;
    if (next < c.num_tiles) coords(next, next_row0, next_n_w);
    if (active) {
      if (lane == 0) ptx::bulk_wait_group_read<0>();          // the previous tile's stores have read the staging boxes
      __syncwarp();
      ptx::tmem_ld_fence(r0);
      ptx::tmem_ld_32x32_issue(t_row + 32, r1);
    }
    if (kIn) {
      ok = wait_bounded(c.in_bar, ph0, c.abort_flag, p.status, p.wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      pending[0] = false;
      ph0 ^= 1u;
    }
    if (active) slice(r0, 0);
    if (kIn) {
      __syncwarp();                                           // every lane has read the first input box
      if (next < c.num_tiles) {
        if (lane == 0) issue_in(0, next_n_w, next_row0);
        pending[0] = true;
      }
    }
    if (active) ptx::tmem_ld_fence(r1);
    release_acc(acc);
    if (kIn) {
      ok = wait_bounded(in_bar1, ph1, c.abort_flag, p.status, p.wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      pending[1] = false;
      ph1 ^= 1u;
    }
    if (active) slice(r1, 1);
    if (kIn) {
      __syncwarp();
      if (next < c.num_tiles) {
        if (lane == 0) issue_in(1, next_n_w, next_row0);
        pending[1] = true;
      }
    }
    if (active) {
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        if (aux_out) ptx::tma_store_2d(tm_aux, buf_aux, n_w, row0);
        ptx::tma_store_2d(tm_out, buf_out, n_w, row0);
        ptx::bulk_commit_group();
      }
    }
    tile = next; row0 = next_row0; n_w = next_n_w;
  }
  // Leaving early (a wait ran out somewhere in the CTA): let tensor-memory loads and input boxes
  // that are still in flight land before the CTA may give up its resources.
  ptx::tmem_ld_wait_all();
  if (kIn && lane == 0) {
    if (pending[0]) for (uint32_t it = 0; it < p.wait_limit && !ptx::mbar_try_wait(c.in_bar, ph0); ++it) {}
    if (pending[1]) for (uint32_t it = 0; it < p.wait_limit && !ptx::mbar_try_wait(in_bar1, ph1); ++it) {}
  }
  if (lane == 0) ptx::bulk_wait_group_read<0>();             // stores have left shared memory before the CTA may exit
  __syncwarp();
}

// ES: operand element size in bytes (1 = FP8, 2 = BF16 / F16).
// A_MN / B_MN: operand stored MN-major ([K x M] resp. [K x N] row-major) instead of K-major.
// EPI: the fused epilogue (EpiKind).  EW: number of epilogue warps (8 or 16).
// CG: 1 = every CTA computes its own 128 x BN tiles; 2 = clusters of two CTAs compute 256 x BN
//     tiles with tcgen05.mma.cta_group::2 (the even CTA issues, both load and both run an epilogue).
template <int ES, bool A_MN, bool B_MN, int BN, int CG, int EPI, int EW, bool BATCHED>
__global__ void __launch_bounds__(gemm_threads(EW), 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_aux,
            const __grid_constant__ CUtensorMap tmap_skip, const GemmParams p) {
  using S = GemmSmem<BN, CG, EW>;
  static_assert(!BATCHED || EPI == kEpiPlain, "batched problems take the plain epilogue");
  static_assert(EW == 8 || (EW == 16 && (EPI == kEpiGelu || EPI == kEpiGeluGrad)), "16 epilogue warps serve the GELU epilogues only");
  constexpr int kBK = kStageKBytes / ES;            // K elements per stage
  constexpr int kChunkElems = 128 / ES;             // MN elements per 128-byte row of an MN-major tile
  constexpr uint32_t kChunkBytes = kBK * 128;       // one MN-major chunk: kBK rows of 128 bytes
  constexpr uint32_t kTmemCols = 2 * BN;            // two accumulators
  constexpr int kBRows = BN / CG;                   // B rows (N indices) this CTA loads
  static_assert(CG == 1 || (kBRows % kChunkElems) == 0, "pair tiles need whole 128-byte chunks of N per CTA");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
  const uint32_t epi_base = smem_base + S::kStages * S::kStageBytes;      // 1024-byte aligned staging boxes
  const uint32_t bars = epi_base + S::kEpiBytes;
  // barrier layout (8 bytes each): full[kStages], empty[kStages], acc_full[2], acc_empty[2], drained, epi_in[2 * EW]
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S::kStages + s); };
  auto acc_full_bar = [&](int a) { return bars + 8u * (2 * S::kStages + a); };
  auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * S::kStages + 2 + a); };
  const uint32_t drained_bar = bars + 8u * (2 * S::kStages + 4);
  auto epi_in_bar = [&](int w) { return bars + 8u * (2 * S::kStages + 5 + w); };   // epilogue warp w owns 2 w and 2 w + 1
  static_assert(8 * (2 * S::kStages + 5 + 2 * EW) + 8 <= S::kBarrierBytes, "barrier area too small");
  uint8_t* tail = smem_gen + S::kStages * S::kStageBytes + S::kEpiBytes + 8 * (2 * S::kStages + 5 + 2 * EW);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = (CG == 2) ? (int)ptx::cluster_ctarank() : 0;     // position in the pair
  const int group = blockIdx.x / CG, num_groups = gridDim.x / CG;   // tile-walking unit: CTA or pair
  const int num_tiles = p.tiles_m * p.tiles_n * p.nb0 * p.nb1;      // tiles of (128 * CG) x BN, all problems
  const int num_kb = (p.K + kBK - 1) / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    const int epi_arrivals = EPI != kEpiLegacy ? CG * 4 * (BN / (EW == 16 ? 64 : 128)) : CG * kEpilogueWarps;
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full_bar(a), 1); ptx::mbar_init(acc_empty_bar(a), epi_arrivals); }
    ptx::mbar_init(drained_bar, 1);
    for (int w = 0; w < 2 * EW; ++w) ptx::mbar_init(epi_in_bar(w), 1);
    *abort_flag = 0;
    ptx::mbar_init_fence();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    if (CG == 2) { ptx::tmem_alloc_pair(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (CG == 2) ptx::cluster_sync();                  // the partner's barriers and TMEM are ready too
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (every CTA)
    if (lane == 0) {
      uint32_t issued = 0;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = group; ok && !p.no_loads && tile < num_tiles; tile += num_groups) {
        const int m0 = tile_m(p, tile) * (kBM * CG) + rank * kBM;
        const int n0 = tile_n(p, tile) * BN + rank * kBRows;
        int b0 = 0, b1 = 0;
        if (BATCHED) tile_batch(p, tile, b0, b1);
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, p.wait_limit);
          if (!ok) break;
          const uint32_t a_dst = smem_base + stage * S::kStageBytes;
          const uint32_t b_dst = a_dst + S::kABytes;
          const int k0 = kb * kBK;
          // bytes of the whole tile stage are counted on the (even CTA's) full barrier
          const uint32_t fb = (CG == 2) ? ptx::in_even_cta(full_bar(stage)) : full_bar(stage);
          if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), CG * S::kStageBytes);
          auto load = [&](uint32_t dst, const void* tm, int x, int y) {
            if (BATCHED) {
              if (CG == 2) ptx::tma_load_4d_pair(dst, tm, fb, x, y, b1, b0); else ptx::tma_load_4d(dst, tm, fb, x, y, b1, b0);
            } else {
              if (CG == 2) ptx::tma_load_2d_pair(dst, tm, fb, x, y); else ptx::tma_load_2d(dst, tm, fb, x, y);
            }
          };
          if (A_MN) {
#pragma unroll
            for (int c = 0; c < kBM / kChunkElems; ++c) load(a_dst + c * kChunkBytes, &tmap_a, m0 + c * kChunkElems, k0);
          } else {
            load(a_dst, &tmap_a, k0, m0);
          }
          if (B_MN) {
#pragma unroll
            for (int c = 0; c < kBRows / kChunkElems; ++c) load(b_dst + c * kChunkBytes, &tmap_b, n0 + c * kChunkElems, k0);
          } else {
            load(b_dst, &tmap_b, k0, n0);
          }
          ++issued;
          if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
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
    // ------------------------------------------------------------ MMA issuer (even CTA of a pair only)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      uint32_t local = 0;
      bool ok = true;
      // The issuing thread is a single instruction stream that has to start four MMAs every ~500
      // cycles, so the loop body is kept minimal: descriptors differ from stage to stage and from
      // k-step to k-step only in their 14-bit start-address field, i.e. by adding a constant to the
      // low word (no carry: shared memory addresses / 16 stay below 2^14).
      const uint64_t a_desc0 = A_MN ? ptx::smem_desc_sw128(smem_base, kChunkBytes, 1024) : ptx::smem_desc_sw128(smem_base, 16, 1024);
      const uint64_t b_desc0 = B_MN ? ptx::smem_desc_sw128(smem_base + S::kABytes, kChunkBytes, 1024)
                                    : ptx::smem_desc_sw128(smem_base + S::kABytes, 16, 1024);
      const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), b_hi = (uint32_t)(b_desc0 >> 32);
      const uint32_t a_lo0 = (uint32_t)a_desc0, b_lo0 = (uint32_t)b_desc0;
      constexpr uint32_t kStageStep = S::kStageBytes >> 4;
      constexpr uint32_t kAStep = (A_MN ? kChunkBytes / kKSteps : 32u) >> 4;   // K-major: 32 bytes along the row
      constexpr uint32_t kBStep = (B_MN ? kChunkBytes / kKSteps : 32u) >> 4;   // MN-major: kBK/4 rows of 128 bytes
      const uint32_t idesc = p.idesc;
      for (int tile = group; ok && tile < num_tiles; tile += num_groups, ++local) {
        const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
        ok = wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, p.wait_limit);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
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
            const uint64_t adesc = ((uint64_t)a_hi << 32) | (a_lo + k * kAStep);
            const uint64_t bdesc = ((uint64_t)b_hi << 32) | (b_lo + k * kBStep);
            if (CG == 2) ptx::mma_ss_pair<ES == 1>(d_tmem, adesc, bdesc, idesc, accumulate);
            else ptx::mma_ss<ES == 1>(d_tmem, adesc, bdesc, idesc, accumulate);
            accumulate = 1;
          }
          // stage reusable (in both CTAs of a pair) once these MMAs have read it
          if (CG == 2) ptx::mma_commit_pair(empty_bar(stage), 3); else ptx::mma_commit(empty_bar(stage));
          if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) {                                     // accumulator complete
          if (CG == 2) ptx::mma_commit_pair(acc_full_bar(acc), 3); else ptx::mma_commit(acc_full_bar(acc));
        }
      }
      if (*abort_flag) {
        if (CG == 2) ptx::mma_commit_pair(drained_bar, 1); else ptx::mma_commit(drained_bar);
        for (uint32_t it = 0; it < p.wait_limit && !ptx::mbar_try_wait(drained_bar, 0); ++it) {}
      }
    }
  } else if (EPI != kEpiLegacy) {
    // ------------------------------------------------------------ epilogue warps, through shared memory + TMA
    EpiCtx c;
    c.tmem_base = tmem_base; c.acc_full0 = acc_full_bar(0); c.acc_empty0 = acc_empty_bar(0);
    c.in_bar = epi_in_bar(2 * (warp - 2)); c.buf0 = epi_base + (warp - 2) * epi_warp_bytes(EW);
    c.abort_flag = abort_flag; c.warp = warp; c.lane = lane; c.rank = rank;
    c.group = group; c.num_groups = num_groups; c.num_tiles = num_tiles;
    if constexpr (EW == 16) {
      const uint32_t in_bar1 = epi_in_bar(2 * (warp - 2) + 1);
      const bool e5 = p.out_dt == US_E5M2, bf = p.aux_dt == US_BF16;
      if (e5 && bf) epilogue_act16<BN, CG, EPI, true, true>(p, &tmap_out, &tmap_aux, c, in_bar1);
      else if (e5) epilogue_act16<BN, CG, EPI, true, false>(p, &tmap_out, &tmap_aux, c, in_bar1);
      else if (bf) epilogue_act16<BN, CG, EPI, false, true>(p, &tmap_out, &tmap_aux, c, in_bar1);
      else epilogue_act16<BN, CG, EPI, false, false>(p, &tmap_out, &tmap_aux, c, in_bar1);
    } else {
      epilogue_staged<BN, CG, EPI, EW, BATCHED>(p, &tmap_out, &tmap_aux, &tmap_skip, c);
    }
  } else {
    // ------------------------------------------------------------ epilogue warps, direct global accesses
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;                // which of the two interleaved sets of 32-column slices
    uint32_t local = 0;
    bool ok = true;
    for (int tile = group; ok && tile < num_tiles; tile += num_groups, ++local) {
      const uint32_t acc = local & 1u, acc_phase = (local >> 1) & 1u;
      const int m0 = tile_m(p, tile) * (kBM * CG) + rank * kBM;
      const int n0 = tile_n(p, tile) * BN;
      const int64_t row = m0 + q * 32 + lane;
      const bool row_ok = row < p.M;
      EpiloguePrefetch pf;
      const int c_first = 32 * half;
      if (row_ok && n0 + c_first + 32 <= p.N) prefetch_full(p, row, n0 + c_first, pf);
      ok = wait_bounded(acc_full_bar(acc), acc_phase, abort_flag, p.status, p.wait_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
#pragma unroll 1
      for (int c = c_first; c < BN; c += 64) {
        if (n0 + c >= p.N) break;                    // warp-uniform
        float v[32];
        ptx::tmem_ld_32x32(t_row + c, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= p.scale;
        const int ncols = min(32, p.N - (n0 + c));
        if (row_ok) {
          if (ncols == 32) epilogue_chunk_full(p, v, pf, row, n0 + c);
          else epilogue_chunk_ragged(p, v, row, n0 + c, ncols);
        }
        // operands of this warp's next slice, in flight while the next TMEM load is issued
        if (row_ok && c + 64 < BN && n0 + c + 64 + 32 <= p.N) prefetch_full(p, row, n0 + c + 64, pf);
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {                               // the issuing (even) CTA owns the accumulator-free barrier
        if (CG == 2) ptx::mbar_arrive_cluster(ptx::in_even_cta(acc_empty_bar(acc)));
        else ptx::mbar_arrive(acc_empty_bar(acc));
      }
    }
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (CG == 2) ptx::cluster_sync();                  // no CTA leaves while its partner may still signal it
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if (CG == 2) ptx::tmem_dealloc_pair(tmem_base, kTmemCols); else ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace us
