// Scaled layer norm over the rows of a matrix, forward and backward (table "Table of unit scaling
// factors", row layer_norm: alpha = 1, beta_x = 1, beta_w = beta_c = b^-1/2 for a b x n input).
//
// Forward and the input gradient are row-wise: one warp per row, 128-bit loads and stores, warp-shuffle
// reductions, the row held in registers when it has at most 1024 elements (re-read from cache otherwise).
// The variance is taken about the mean (sum of (x - mu)^2), which equals the table's
// mean(x^2) - mu^2 without its cancellation in float32.
//
// Weight and bias gradients are column sums over all rows.  The backward kernel keeps, per lane, the
// partial sums of the columns that lane owns (in registers, or in shared memory for long rows) over
// the rows its warp walks, combines the warps of a CTA in a fixed order and writes one partial row
// per CTA to the caller's workspace; a second kernel adds the CTAs' partials in a fixed order and
// applies beta.  No atomics: results do not depend on scheduling.
#include "common.cuh"
#include "host.h"
#include "rowwise.cuh"
#include "sm100.cuh"

namespace us {

constexpr int kLnThreads = 256;             // 8 warps = 8 rows in flight per CTA
constexpr int kLnWarps = kLnThreads / 32;
constexpr int kLnMaxBwdCols = 4096;         // backward, long rows: column partials of 4 warps in 128 KB of shared memory

struct LnArgs {
  const void* x; int x_dt; int64_t x_ld;
  const void* g; int g_dt; int64_t g_ld;    // backward only
  const void* w; int w_dt;                  // [cols]
  const void* c; int c_dt;                  // [cols], forward only
  void* out; int out_dt; int64_t out_ld;    // Y (forward) or dX (backward)
  float* partial;                           // backward: [gridDim.x][2][cols]
  int64_t rows; int cols;
  int vec_ok;                               // all row starts 16-byte aligned and cols % 8 == 0
  float eps, beta_x;
};

// Mean and reciprocal standard deviation of a row given as nch chunks per lane.
template <int NCH>
__device__ __forceinline__ void row_stats(const LnArgs& a, int64_t x_off, int lane, int nch, float (&x)[NCH > 0 ? NCH : 1][8],
                                          float& mu, float& rstd) {
  const bool vec = a.vec_ok != 0;
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    float t[8];
    if (col < a.cols) {
      load8(a.x, a.x_dt, x_off, col, a.cols, vec, 0.f, t);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) { s += t[i]; if (NCH > 0) x[c][i] = t[i]; }
  }
  mu = warp_sum(s) / (float)a.cols;
  float q = 0.f;
#pragma unroll
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    float t[8];
    if (NCH > 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = x[c][i];
    } else if (col < a.cols) {
      load8(a.x, a.x_dt, x_off, col, a.cols, vec, 0.f, t);
    }
    if (col < a.cols) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float d = (col + i < a.cols) ? t[i] - mu : 0.f;
        q = fmaf(d, d, q);
      }
    }
  }
  rstd = rsqrtf(warp_sum(q) / (float)a.cols + a.eps);
}

// NCH > 0: rows of up to 256 * NCH elements, held in registers.  NCH == 0: any length, re-read.
template <int NCH>
__global__ void __launch_bounds__(kLnThreads) ln_fwd_kernel(const LnArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kLnWarps + (threadIdx.x >> 5);
  if (row >= a.rows) return;
  const int64_t x_off = row * a.x_ld, out_off = row * a.out_ld;
  const bool vec = a.vec_ok != 0;
  const int nch = NCH > 0 ? NCH : (a.cols + 255) / 256;
  float x[NCH > 0 ? NCH : 1][8];
  float mu, rstd;
  row_stats<NCH>(a, x_off, lane, nch, x, mu, rstd);
#pragma unroll
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col >= a.cols) continue;
    float t[8], w[8], b[8];
    if (NCH > 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = x[c][i];
    } else {
      load8(a.x, a.x_dt, x_off, col, a.cols, vec, 0.f, t);
    }
    load8(a.w, a.w_dt, 0, col, a.cols, vec, 0.f, w);
    load8(a.c, a.c_dt, 0, col, a.cols, vec, 0.f, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) t[i] = fmaf(w[i], (t[i] - mu) * rstd, b[i]);
    store8(a.out, a.out_dt, out_off, col, a.cols, vec, t);
  }
}

// Input gradient of the rows this warp walks, and the CTA's partial column sums of G * xhat and G.
template <int NCH>
__global__ void __launch_bounds__(kLnThreads) ln_bwd_kernel(const LnArgs a) {
  extern __shared__ __align__(16) float ln_smem[];          // NCH > 0: [warps][cols] for the combine; NCH == 0: [warps][2][cols]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nw = blockDim.x >> 5;             // 8 warps per CTA, 4 for long rows
  const bool vec = a.vec_ok != 0;
  const int nch = NCH > 0 ? NCH : (a.cols + 255) / 256;
  const float inv_n = 1.0f / (float)a.cols;
  float sw[NCH > 0 ? NCH : 1][8], sc[NCH > 0 ? NCH : 1][8];
  float* my_w = ln_smem + (size_t)warp * 2 * a.cols;      // NCH == 0 only
  float* my_c = my_w + a.cols;
  if (NCH > 0) {
#pragma unroll
    for (int c = 0; c < (NCH > 0 ? NCH : 1); ++c)
#pragma unroll
      for (int i = 0; i < 8; ++i) { sw[c][i] = 0.f; sc[c][i] = 0.f; }
  } else {
    for (int j = lane; j < a.cols; j += 32) { my_w[j] = 0.f; my_c[j] = 0.f; }
    __syncwarp();
  }
  for (int64_t row = (int64_t)blockIdx.x * nw + warp; row < a.rows; row += (int64_t)gridDim.x * nw) {
    const int64_t x_off = row * a.x_ld, g_off = row * a.g_ld, out_off = row * a.out_ld;
    float x[NCH > 0 ? NCH : 1][8], u[NCH > 0 ? NCH : 1][8];
    float mu, rstd;
    row_stats<NCH>(a, x_off, lane, nch, x, mu, rstd);
    // pass 1: xhat, u = g w; row sums of u and u xhat; column partials of g xhat and g
    float su = 0.f, sux = 0.f;
#pragma unroll
    for (int c = 0; c < nch; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col >= a.cols) continue;
      float t[8], g[8], w[8];
      if (NCH > 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = x[c][i];
      } else {
        load8(a.x, a.x_dt, x_off, col, a.cols, vec, 0.f, t);
      }
      load8(a.g, a.g_dt, g_off, col, a.cols, vec, 0.f, g);
      load8(a.w, a.w_dt, 0, col, a.cols, vec, 0.f, w);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const bool in = col + i < a.cols;
        const float xh = in ? (t[i] - mu) * rstd : 0.f;
        const float uu = in ? g[i] * w[i] : 0.f;
        su += uu;
        sux = fmaf(uu, xh, sux);
        if (NCH > 0) {
          x[c][i] = xh; u[c][i] = uu;
          sw[c][i] = fmaf(g[i], xh, sw[c][i]);
          sc[c][i] += in ? g[i] : 0.f;
        } else if (in) {
          my_w[col + i] = fmaf(g[i], xh, my_w[col + i]);
          my_c[col + i] += g[i];
        }
      }
    }
    const float mean_u = warp_sum(su) * inv_n, mean_ux = warp_sum(sux) * inv_n;
    const float k = a.beta_x * rstd;
    // pass 2: dX = beta_x rstd (u - mean(u) - xhat mean(u xhat))
#pragma unroll
    for (int c = 0; c < nch; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col >= a.cols) continue;
      float d[8];
      if (NCH > 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) d[i] = k * (u[c][i] - mean_u - x[c][i] * mean_ux);
      } else {
        float t[8], g[8], w[8];
        load8(a.x, a.x_dt, x_off, col, a.cols, vec, 0.f, t);
        load8(a.g, a.g_dt, g_off, col, a.cols, vec, 0.f, g);
        load8(a.w, a.w_dt, 0, col, a.cols, vec, 0.f, w);
#pragma unroll
        for (int i = 0; i < 8; ++i) d[i] = k * (g[i] * w[i] - mean_u - (t[i] - mu) * rstd * mean_ux);
      }
      store8(a.out, a.out_dt, out_off, col, a.cols, vec, d);
    }
  }
  // ---- combine the CTA's warps in warp order; one partial row (G xhat sums, then G sums) per CTA
  float* dst = a.partial + (size_t)blockIdx.x * 2 * a.cols;
  if (NCH > 0) {
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      __syncthreads();
#pragma unroll
      for (int c = 0; c < (NCH > 0 ? NCH : 1); ++c) {
        const int col = (c * 32 + lane) * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (col + i < a.cols) ln_smem[(size_t)warp * a.cols + col + i] = pass == 0 ? sw[c][i] : sc[c][i];
      }
      __syncthreads();
      for (int j = threadIdx.x; j < a.cols; j += blockDim.x) {
        float s = 0.f;
        for (int wq = 0; wq < nw; ++wq) s += ln_smem[(size_t)wq * a.cols + j];
        dst[(size_t)pass * a.cols + j] = s;
      }
    }
  } else {
    __syncthreads();
    for (int j = threadIdx.x; j < 2 * a.cols; j += blockDim.x) {
      const int which = j >= a.cols, col = j - which * a.cols;
      float s = 0.f;
      for (int wq = 0; wq < nw; ++wq) s += ln_smem[((size_t)wq * 2 + which) * a.cols + col];
      dst[j] = s;
    }
  }
}

// ---------------------------------------------------------------- 16-bit inputs, rows in registers
// The common case (BF16 / F16 activations and gradients, rows of at most 2048 / 1024 elements, aligned)
// gets persistent warps that fetch their next row, still packed, before working on the current one,
// and read the weight (and bias) from a float32 copy in shared memory.

// Mean and reciprocal standard deviation of a row held as floats (zeros beyond the row's end).
template <int NCH>
__device__ __forceinline__ void stats_regs(const float (&x)[NCH][8], int lane, int cols, float eps, float& mu, float& rstd) {
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < NCH; ++c)
#pragma unroll
    for (int i = 0; i < 8; ++i) s += x[c][i];
  mu = warp_sum(s) / (float)cols;
  float q = 0.f;
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    if ((c * 32 + lane) * 8 < cols) {
#pragma unroll
      for (int i = 0; i < 8; ++i) { const float d = x[c][i] - mu; q = fmaf(d, d, q); }
    }
  }
  rstd = rsqrtf(warp_sum(q) / (float)cols + eps);
}

template <int NCH>
__global__ void __launch_bounds__(kLnThreads, 2) ln_fwd16_kernel(const LnArgs a) {
  extern __shared__ __align__(16) float ln_smem[];                         // w[cols], c[cols] as float32
  float* w_s = ln_smem;
  float* c_s = ln_smem + a.cols;
  for (int j = threadIdx.x; j < a.cols; j += blockDim.x) { w_s[j] = load_one(a.w, a.w_dt, j); c_s[j] = load_one(a.c, a.c_dt, j); }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int64_t stride = (int64_t)gridDim.x * nw;
  int64_t row = (int64_t)blockIdx.x * nw + warp;
  uint4 cur[NCH], nxt[NCH];
  if (row < a.rows) load_row16<NCH>(a.x, row * a.x_ld, lane, a.cols, cur);
  for (; row < a.rows; row += stride) {
    if (row + stride < a.rows) load_row16<NCH>(a.x, (row + stride) * a.x_ld, lane, a.cols, nxt);
    float x[NCH][8];
#pragma unroll
    for (int c = 0; c < NCH; ++c) unpack16x8(cur[c], a.x_dt, x[c]);
    float mu, rstd;
    stats_regs<NCH>(x, lane, a.cols, a.eps, mu, rstd);
    const int64_t out_off = row * a.out_ld;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        const float4 w0 = *reinterpret_cast<const float4*>(w_s + col), w1 = *reinterpret_cast<const float4*>(w_s + col + 4);
        const float4 b0 = *reinterpret_cast<const float4*>(c_s + col), b1 = *reinterpret_cast<const float4*>(c_s + col + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
        const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        float t[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = fmaf(w[i], (x[c][i] - mu) * rstd, b[i]);
        store8(a.out, a.out_dt, out_off, col, a.cols, true, t);
      }
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) cur[c] = nxt[c];
  }
}

// G32: the gradient is float32 (the gradient of a layer's output often is) instead of the 16-bit type of X.
//
// The rows reach the SM through a ring of kLnStages slots per warp in shared memory, filled by bulk
// copies (cp.async.bulk, completion counted on one mbarrier per slot): with one row per warp in
// registers the kernel is bound by memory latency (a few tens of KB in flight per SM), the ring keeps
// kLnStages rows per warp in flight.  A wait on a slot is bounded; if it ever runs out the warp reads
// that row and all later ones with ordinary loads (same result), and before leaving it gives the
// copies it issued time to land.
constexpr int kLnStages = 3;
constexpr uint32_t kLnWaitLimit = 1u << 20;

// XBF: X (and a 16-bit gradient) are BF16 rather than F16; fixed at compile time, because a run-time choice
// in the unpacking costs more instructions than the arithmetic it feeds.
template <int NCH, bool G32, bool XBF>
__global__ void __launch_bounds__(128, 3) ln_bwd16_kernel(const LnArgs a) {
  extern __shared__ __align__(16) float ln_smem[];             // w[cols] as float32, [warps][cols] for the combine, the ring, its mbarriers
  float* w_s = ln_smem;                                        // NCH * 256 floats
  float* comb = ln_smem + NCH * 256;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const uint32_t xb = (uint32_t)a.cols * 2u, gb = (uint32_t)a.cols * (G32 ? 4u : 2u), slot = xb + gb;
  char* ring_gen = reinterpret_cast<char*>(comb + (size_t)nw * a.cols) + (size_t)warp * kLnStages * slot;
  const uint32_t ring = ptx::smem_addr(ring_gen);
  const uint32_t bars = ptx::smem_addr(reinterpret_cast<char*>(comb + (size_t)nw * a.cols) + (size_t)nw * kLnStages * slot) +
                        8u * (uint32_t)(warp * kLnStages);
  if (!G32 && lane == 0) {                                     // (no ring, hence no mbarriers, with a float32 gradient)
    for (int st = 0; st < kLnStages; ++st) ptx::mbar_init(bars + 8u * st, 1);
    ptx::mbar_init_fence();
  }
  // w in shared memory, laid out for conflict-free 16-byte reads: a lane's eight consecutive weights
  // (columns 8 q .. 8 q + 7) are split into a low and a high half; low halves at [4 q, 4 q + 4), high halves
  // kLnHi floats further.
  const int kLnHi = NCH * 32 * 4;
  for (int j = threadIdx.x; j < a.cols; j += blockDim.x)
    w_s[(j >> 3) * 4 + (j & 3) + ((j & 4) ? kLnHi : 0)] = load_one(a.w, a.w_dt, j);
  __syncthreads();
  const int64_t stride = (int64_t)gridDim.x * nw;
  const float inv_n = 1.0f / (float)a.cols;
  f32x2 sw[NCH][4], sc[NCH][4];                                // column sums of g * xhat and of g, as float32 pairs
#pragma unroll
  for (int c = 0; c < NCH; ++c)
#pragma unroll
    for (int j = 0; j < 4; ++j) { sw[c][j] = pack2(0.f, 0.f); sc[c][j] = pack2(0.f, 0.f); }
  int64_t row = (int64_t)blockIdx.x * nw + warp;
  auto issue = [&](int64_t r, int st) {                        // lane 0
    const uint32_t bar = bars + 8u * st;
    ptx::mbar_expect_tx(bar, slot);
    ptx::bulk_load_1d(ring + st * slot, static_cast<const char*>(a.x) + r * a.x_ld * 2, xb, bar);
    ptx::bulk_load_1d(ring + st * slot + xb, static_cast<const char*>(a.g) + r * a.g_ld * (G32 ? 4 : 2), gb, bar);
  };
  int issued = 0;                                              // rows asked for so far (warp-uniform)
  if (!G32)
    for (; issued < kLnStages && row + issued * stride < a.rows; ++issued)
      if (lane == 0) issue(row + issued * stride, issued);
  // direct: ordinary loads instead of the ring -- after a wait ran out, and always for a float32 gradient
  // (rows of 6 bytes per element: the ring then costs a CTA per SM and measured slower than plain loads)
  bool direct = G32;
  int it = 0, unconsumed = 0;                                  // unconsumed: first row whose copy was never waited for
  uint4 cx[NCH], cg[G32 ? 1 : NCH], nx[G32 ? NCH : 1];
  for (; row < a.rows; row += stride, ++it) {
    const int st = it % kLnStages;
    const uint32_t parity = (uint32_t)(it / kLnStages) & 1u;
    float gf[G32 ? NCH : 1][8];
    if (!direct) {
      bool ok = false;
      for (uint32_t k = 0; k < kLnWaitLimit && !(ok = ptx::mbar_try_wait(bars + 8u * st, parity)); ++k) {}
      direct = !__all_sync(0xffffffffu, ok);
      if (direct) unconsumed = it;
    }
    if (!direct) {
      const char* sx = ring_gen + (size_t)st * slot;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int col = (c * 32 + lane) * 8;
        if (col < a.cols) {
          cx[c] = *reinterpret_cast<const uint4*>(sx + col * 2);
          if (G32) {
            const float4 g0 = *reinterpret_cast<const float4*>(sx + xb + col * 4), g1 = *reinterpret_cast<const float4*>(sx + xb + col * 4 + 16);
            gf[G32 ? c : 0][0] = g0.x; gf[G32 ? c : 0][1] = g0.y; gf[G32 ? c : 0][2] = g0.z; gf[G32 ? c : 0][3] = g0.w;
            gf[G32 ? c : 0][4] = g1.x; gf[G32 ? c : 0][5] = g1.y; gf[G32 ? c : 0][6] = g1.z; gf[G32 ? c : 0][7] = g1.w;
          } else {
            cg[G32 ? 0 : c] = *reinterpret_cast<const uint4*>(sx + xb + col * 2);
          }
        } else {
          cx[c] = make_uint4(0, 0, 0, 0);
          if (!G32) cg[G32 ? 0 : c] = make_uint4(0, 0, 0, 0);
        }
      }
      __syncwarp();                                            // every lane holds its part: the slot can be refilled
      const int64_t nxt = row + (int64_t)kLnStages * stride;
      if (nxt < a.rows) {
        if (lane == 0) issue(nxt, st);
        ++issued;
      }
    } else {
      if constexpr (G32) {
        // X of this row was fetched one iteration ahead (packed, in registers); the float32 gradient is read now
        if (it == 0) load_row16<NCH>(a.x, row * a.x_ld, lane, a.cols, cx);
        else {
#pragma unroll
          for (int c = 0; c < NCH; ++c) cx[c] = nx[c];
        }
        if (row + stride < a.rows) load_row16<NCH>(a.x, (row + stride) * a.x_ld, lane, a.cols, nx);
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const int col = (c * 32 + lane) * 8;
          if (col < a.cols) load_vec<8>(static_cast<const char*>(a.g) + (row * a.g_ld + col) * 4, US_F32, gf[c]);
        }
      } else {
        load_row16<NCH>(a.x, row * a.x_ld, lane, a.cols, cx);
        load_row16<NCH>(a.g, row * a.g_ld, lane, a.cols, cg);
      }
    }
    // From here on the row is worked on as pairs of float32 in 64-bit registers (add / mul / fma .f32x2):
    // the kernel is bound by instruction issue, and the packed forms halve the arithmetic instructions.
    f32x2 xp[NCH][4];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const uint32_t wx[4] = {cx[c].x, cx[c].y, cx[c].z, cx[c].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = XBF ? unpack_bf16x2(wx[j]) : unpack_f16x2(wx[j]);
        xp[c][j] = pack2(f.x, f.y);
      }
    }
    auto g_pair = [&](int c, int j) -> f32x2 {                 // gradient values 2 j, 2 j + 1 of chunk c
      if (G32) return pack2(gf[G32 ? c : 0][2 * j], gf[G32 ? c : 0][2 * j + 1]);
      const uint4& r = cg[G32 ? 0 : c];
      const uint32_t w = j == 0 ? r.x : j == 1 ? r.y : j == 2 ? r.z : r.w;
      const float2 f = XBF ? unpack_bf16x2(w) : unpack_f16x2(w);
      return pack2(f.x, f.y);
    };
    auto w_pairs = [&](int col, f32x2 (&w2)[4]) {
      const ulonglong2 lo = *reinterpret_cast<const ulonglong2*>(w_s + (col >> 1)), hi = *reinterpret_cast<const ulonglong2*>(w_s + (col >> 1) + kLnHi);
      w2[0] = lo.x; w2[1] = lo.y; w2[2] = hi.x; w2[3] = hi.y;
    };
    // mean, then variance about the mean (chunks beyond the row's end hold zeros and are left out of the second sum)
    f32x2 acc = pack2(0.f, 0.f);
#pragma unroll
    for (int c = 0; c < NCH; ++c)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc = add2(acc, xp[c][j]);
    float lo, hi;
    unpack2(acc, lo, hi);
    const float mu = warp_sum(lo + hi) * inv_n;
    const f32x2 neg_mu = splat2(-mu);
    acc = pack2(0.f, 0.f);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      if ((c * 32 + lane) * 8 < a.cols) {
#pragma unroll
        for (int j = 0; j < 4; ++j) { const f32x2 dm = add2(xp[c][j], neg_mu); acc = fma2(dm, dm, acc); }
      }
    }
    unpack2(acc, lo, hi);
    const float rstd = rsqrtf(warp_sum(lo + hi) * inv_n + a.eps);
    const f32x2 rstd2 = splat2(rstd), shift2 = splat2(-mu * rstd);
    f32x2 su2 = pack2(0.f, 0.f), sux2 = pack2(0.f, 0.f);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        f32x2 w2[4];
        w_pairs(col, w2);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const f32x2 g2 = g_pair(c, j);
          const f32x2 xh = fma2(xp[c][j], rstd2, shift2);      // normalised input, kept for the second loop
          xp[c][j] = xh;
          const f32x2 uu = mul2(g2, w2[j]);
          su2 = add2(su2, uu);
          sux2 = fma2(uu, xh, sux2);
          sw[c][j] = fma2(g2, xh, sw[c][j]);
          sc[c][j] = add2(sc[c][j], g2);
        }
      }
    }
    unpack2(su2, lo, hi);
    const float mean_u = warp_sum(lo + hi) * inv_n;
    unpack2(sux2, lo, hi);
    const float mean_ux = warp_sum(lo + hi) * inv_n;
    const float k = a.beta_x * rstd;
    const f32x2 k2 = splat2(k), c0 = splat2(-k * mean_u), c1 = splat2(-k * mean_ux);
    const int64_t out_off = row * a.out_ld;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        f32x2 w2[4];
        w_pairs(col, w2);
        float d[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          // k (g w - mean_u - xh mean_ux)
          const f32x2 t = fma2(mul2(g_pair(c, j), w2[j]), k2, c0);
          unpack2(fma2(xp[c][j], c1, t), d[2 * j], d[2 * j + 1]);
        }
        store8(a.out, a.out_dt, out_off, col, a.cols, true, d);
      }
    }
  }
  if (direct && lane == 0) {
    // copies issued but never consumed: one per slot at most
    for (int k = unconsumed; k < issued; ++k) {
      const uint32_t bar = bars + 8u * (k % kLnStages), parity = (uint32_t)(k / kLnStages) & 1u;
      for (uint32_t n = 0; n < kLnWaitLimit && !ptx::mbar_try_wait(bar, parity); ++n) {}
    }
  }
  float* dst = a.partial + (size_t)blockIdx.x * 2 * a.cols;
#pragma unroll
  for (int pass = 0; pass < 2; ++pass) {
    __syncthreads();
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<f32x2*>(comb + (size_t)warp * a.cols + col + 2 * j) = pass == 0 ? sw[c][j] : sc[c][j];
      }
    }
    __syncthreads();
    for (int j = threadIdx.x; j < a.cols; j += blockDim.x) {
      float s = 0.f;
      for (int wq = 0; wq < nw; ++wq) s += comb[(size_t)wq * a.cols + j];
      dst[(size_t)pass * a.cols + j] = s;
    }
  }
}

// dw_j = beta * sum over CTAs of partial[cta][0][j], dc_j likewise from partial[cta][1][j].
// One CTA per 32 columns of the 2 * cols sums: 32 groups of 32 threads each add every 32nd partial row
// in order (four independent partial sums per thread, combined in a fixed order), then the groups are
// added in order.
constexpr int kLnReduceGroups = 32;
__global__ void __launch_bounds__(32 * kLnReduceGroups) ln_bwd_reduce_kernel(const float* partial, int nparts, int cols, float beta,
                                                                             void* dw, int dw_dt, void* dc, int dc_dt) {
  __shared__ float acc[kLnReduceGroups][32];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + tx;               // index into [2][cols]
  float s4[4] = {0.f, 0.f, 0.f, 0.f};
  if (j < 2 * cols) {
    int p = ty;
    for (; p + 3 * kLnReduceGroups < nparts; p += 4 * kLnReduceGroups) {
#pragma unroll
      for (int u = 0; u < 4; ++u) s4[u] += partial[(size_t)(p + u * kLnReduceGroups) * 2 * cols + j];
    }
#pragma unroll
    for (int u = 0; u < 3; ++u)                     // at most three rows are left for this group
      if (p + u * kLnReduceGroups < nparts) s4[u] += partial[(size_t)(p + u * kLnReduceGroups) * 2 * cols + j];
  }
  acc[ty][tx] = (s4[0] + s4[1]) + (s4[2] + s4[3]);
  __syncthreads();
  if (ty == 0 && j < 2 * cols) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < kLnReduceGroups; ++q) t += acc[q][tx];
    t *= beta;
    if (j < cols) store_one(dw, dw_dt, j, t);
    else store_one(dc, dc_dt, j - cols, t);
  }
}

static bool ln_rows_aligned(const us_mat* m) {
  return reinterpret_cast<uintptr_t>(m->ptr) % 16 == 0 && (m->ld * dtype_size(m->dtype)) % 16 == 0;
}
static bool is_float_in(int dt) { return dt == US_F32 || dt == US_BF16 || dt == US_F16; }

static us_status check_matrix(const us_mat* m, const us_mat* like, bool input) {
  if (!m || m->rows < 0 || m->cols < 0 || m->ld < m->cols) return US_ERR_INVALID_ARG;
  if (like && (m->rows != like->rows || m->cols != like->cols)) return US_ERR_INVALID_ARG;
  if (m->rows * m->cols > 0 && !m->ptr) return US_ERR_INVALID_ARG;
  if (m->cols > 0x7ffffff0) return US_ERR_INVALID_ARG;
  if (input ? !is_float_in(m->dtype) : !(m->dtype >= US_F32 && m->dtype <= US_E5M2)) return US_ERR_UNSUPPORTED;
  if (m->ptr && reinterpret_cast<uintptr_t>(m->ptr) % dtype_size(m->dtype)) return US_ERR_ALIGNMENT;
  return US_OK;
}
// A parameter vector: 1 x cols.
static us_status check_vector(const us_mat* v, int64_t cols, bool input) {
  if (!v || v->rows != 1 || v->cols != cols || v->ld < v->cols) return US_ERR_INVALID_ARG;
  if (cols > 0 && !v->ptr) return US_ERR_INVALID_ARG;
  if (input ? !is_float_in(v->dtype) : !(v->dtype == US_F32 || v->dtype == US_BF16 || v->dtype == US_F16)) return US_ERR_UNSUPPORTED;
  if (v->ptr && reinterpret_cast<uintptr_t>(v->ptr) % dtype_size(v->dtype)) return US_ERR_ALIGNMENT;
  return US_OK;
}

// CTAs of the backward kernel: `warps` rows in flight per CTA, at most `per_sm` CTAs per SM.
static int ln_bwd_grid(int64_t rows, int warps = kLnWarps, int per_sm = 2) {
  const int sms = host::sm_count();
  if (sms <= 0) return 0;
  const int64_t want = (rows + warps - 1) / warps;
  const int64_t cap = (int64_t)sms * per_sm;
  return (int)(want < cap ? want : cap);
}
constexpr int kLnFastWarps = 4, kLnFastPerSm = 3;   // the 16-bit backward kernel: three CTAs of four warps per SM

}  // namespace us

using namespace us;

extern "C" us_status us_layer_norm_fwd(const us_mat* X, const us_mat* w, const us_mat* c, float eps, const us_mat* Y,
                                       void* stream) {
  us_status s = check_matrix(X, nullptr, true);
  if (s == US_OK) s = check_matrix(Y, X, false);
  if (s == US_OK) s = check_vector(w, X->cols, true);
  if (s == US_OK) s = check_vector(c, X->cols, true);
  if (s != US_OK) return s;
  if (!(eps >= 0.f)) return US_ERR_INVALID_ARG;
  if (X->rows == 0 || X->cols == 0) return US_OK;
  LnArgs a{};
  a.x = X->ptr; a.x_dt = X->dtype; a.x_ld = X->ld;
  a.w = w->ptr; a.w_dt = w->dtype; a.c = c->ptr; a.c_dt = c->dtype;
  a.out = Y->ptr; a.out_dt = Y->dtype; a.out_ld = Y->ld;
  a.rows = X->rows; a.cols = (int)X->cols; a.eps = eps; a.beta_x = 1.f;
  a.vec_ok = ln_rows_aligned(X) && ln_rows_aligned(Y) && ln_rows_aligned(w) && ln_rows_aligned(c) && X->cols % 8 == 0;
  const int64_t grid64 = (a.rows + kLnWarps - 1) / kLnWarps;
  if (grid64 > 0x7fffffff) return US_ERR_INVALID_ARG;
  const int grid = (int)grid64, nch = (a.cols + 255) / 256;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (a.vec_ok && (a.x_dt == US_BF16 || a.x_dt == US_F16) && nch <= 8) {
    const int sms = host::sm_count();
    if (sms <= 0) return US_ERR_CUDA;
    const int pgrid = grid < 2 * sms ? grid : 2 * sms;       // two resident CTAs per SM, warps walk the rows
    const size_t smem = (size_t)2 * a.cols * sizeof(float);
    if (nch <= 1) ln_fwd16_kernel<1><<<pgrid, kLnThreads, smem, st>>>(a);
    else if (nch <= 2) ln_fwd16_kernel<2><<<pgrid, kLnThreads, smem, st>>>(a);
    else if (nch <= 4) ln_fwd16_kernel<4><<<pgrid, kLnThreads, smem, st>>>(a);
    else ln_fwd16_kernel<8><<<pgrid, kLnThreads, smem, st>>>(a);
    return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
  }
  if (nch <= 1) ln_fwd_kernel<1><<<grid, kLnThreads, 0, st>>>(a);
  else if (nch <= 2) ln_fwd_kernel<2><<<grid, kLnThreads, 0, st>>>(a);
  else if (nch <= 4) ln_fwd_kernel<4><<<grid, kLnThreads, 0, st>>>(a);
  else if (nch <= 8) ln_fwd_kernel<8><<<grid, kLnThreads, 0, st>>>(a);
  else ln_fwd_kernel<0><<<grid, kLnThreads, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

extern "C" size_t us_layer_norm_bwd_workspace_bytes(int64_t rows, int64_t cols) {
  if (rows <= 0 || cols <= 0) return 0;
  const int g0 = ln_bwd_grid(rows), g1 = ln_bwd_grid(rows, kLnFastWarps, kLnFastPerSm);
  const int grid = g0 > g1 ? g0 : g1;                // whichever kernel the call takes
  return (size_t)(grid > 0 ? grid : 1) * 2 * (size_t)cols * sizeof(float);
}

extern "C" us_status us_layer_norm_bwd(const us_mat* X, const us_mat* w, const us_mat* G, float eps, float beta_x,
                                       float beta_wc, const us_mat* dX, const us_mat* dw, const us_mat* dc, void* ws,
                                       size_t ws_bytes, void* stream) {
  us_status s = check_matrix(X, nullptr, true);
  if (s == US_OK) s = check_matrix(G, X, true);
  if (s == US_OK) s = check_matrix(dX, X, false);
  if (s == US_OK) s = check_vector(w, X->cols, true);
  if (s == US_OK) s = check_vector(dw, X->cols, false);
  if (s == US_OK) s = check_vector(dc, X->cols, false);
  if (s != US_OK) return s;
  if (!(eps >= 0.f)) return US_ERR_INVALID_ARG;
  if (X->cols > kLnMaxBwdCols) return US_ERR_UNSUPPORTED;
  if (X->cols == 0) return US_OK;
  const int grid = ln_bwd_grid(X->rows > 0 ? X->rows : 1);
  if (grid <= 0) return US_ERR_CUDA;
  if (!ws || ws_bytes < us_layer_norm_bwd_workspace_bytes(X->rows > 0 ? X->rows : 1, X->cols)) return US_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % 16) return US_ERR_ALIGNMENT;
  LnArgs a{};
  a.x = X->ptr; a.x_dt = X->dtype; a.x_ld = X->ld;
  a.g = G->ptr; a.g_dt = G->dtype; a.g_ld = G->ld;
  a.w = w->ptr; a.w_dt = w->dtype;
  a.out = dX->ptr; a.out_dt = dX->dtype; a.out_ld = dX->ld;
  a.partial = static_cast<float*>(ws);
  a.rows = X->rows; a.cols = (int)X->cols; a.eps = eps; a.beta_x = beta_x;
  a.vec_ok = ln_rows_aligned(X) && ln_rows_aligned(G) && ln_rows_aligned(dX) && ln_rows_aligned(w) && X->cols % 8 == 0;
  const int nch = (a.cols + 255) / 256;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int nparts = grid;
  // With no rows the first kernel still runs (one CTA) and writes zero partials, so dw = dc = 0.
  if (a.vec_ok && nch <= 4 && (a.x_dt == US_BF16 || a.x_dt == US_F16) && (a.g_dt == a.x_dt || a.g_dt == US_F32)) {
    const bool g32 = a.g_dt == US_F32;
    nparts = ln_bwd_grid(X->rows > 0 ? X->rows : 1, kLnFastWarps, kLnFastPerSm);
    const size_t smem = ((size_t)(nch <= 1 ? 1 : nch <= 2 ? 2 : 4) * 256 + (size_t)kLnFastWarps * a.cols) * sizeof(float) +
                        (g32 ? (size_t)0 : (size_t)kLnFastWarps * kLnStages * (a.cols * 4 + 8));
    const bool xbf = a.x_dt == US_BF16;
    const int n = nch <= 1 ? 1 : nch <= 2 ? 2 : 4;
    void (*fn)(const LnArgs) = nullptr;
#define US_LN_PICK(N)                                                                                   \
  fn = g32 ? (xbf ? ln_bwd16_kernel<N, true, true> : ln_bwd16_kernel<N, true, false>)                   \
           : (xbf ? ln_bwd16_kernel<N, false, true> : ln_bwd16_kernel<N, false, false>)
    if (n == 1) US_LN_PICK(1);
    else if (n == 2) US_LN_PICK(2);
    else US_LN_PICK(4);
#undef US_LN_PICK
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return US_ERR_CUDA;
    fn<<<nparts, 32 * kLnFastWarps, smem, st>>>(a);
  } else if (nch <= 4) {
    const size_t smem = (size_t)kLnWarps * a.cols * sizeof(float);
    if (nch <= 1) ln_bwd_kernel<1><<<grid, kLnThreads, smem, st>>>(a);
    else if (nch <= 2) ln_bwd_kernel<2><<<grid, kLnThreads, smem, st>>>(a);
    else ln_bwd_kernel<4><<<grid, kLnThreads, smem, st>>>(a);
  } else {
    const size_t smem = (size_t)4 * 2 * a.cols * sizeof(float);
    if (cudaFuncSetAttribute(ln_bwd_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return US_ERR_CUDA;
    ln_bwd_kernel<0><<<grid, 128, smem, st>>>(a);
  }
  if (cudaGetLastError() != cudaSuccess) return US_ERR_CUDA;
  const int rgrid = (2 * a.cols + 31) / 32;
  ln_bwd_reduce_kernel<<<rgrid, 32 * kLnReduceGroups, 0, st>>>(a.partial, nparts, a.cols, beta_wc, dw->ptr, dw->dtype, dc->ptr, dc->dtype);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}
