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

// G32: the gradient is float32 (the gradient of a layer's output often is): it is loaded at the top of the
// iteration into float registers instead of being prefetched packed; X is still prefetched.
template <int NCH, bool G32>
__global__ void __launch_bounds__(128, 3) ln_bwd16_kernel(const LnArgs a) {
  extern __shared__ __align__(16) float ln_smem[];                         // w[cols] as float32, then [warps][cols] for the combine
  float* w_s = ln_smem;
  float* comb = ln_smem + a.cols;
  for (int j = threadIdx.x; j < a.cols; j += blockDim.x) w_s[j] = load_one(a.w, a.w_dt, j);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int64_t stride = (int64_t)gridDim.x * nw;
  const float inv_n = 1.0f / (float)a.cols;
  float sw[NCH][8], sc[NCH][8];
#pragma unroll
  for (int c = 0; c < NCH; ++c)
#pragma unroll
    for (int i = 0; i < 8; ++i) { sw[c][i] = 0.f; sc[c][i] = 0.f; }
  int64_t row = (int64_t)blockIdx.x * nw + warp;
  uint4 cx[NCH], cg[G32 ? 1 : NCH], nx[NCH], ng[G32 ? 1 : NCH];
  if (row < a.rows) {
    load_row16<NCH>(a.x, row * a.x_ld, lane, a.cols, cx);
    if (!G32) load_row16<G32 ? 1 : NCH>(a.g, row * a.g_ld, lane, a.cols, cg);
  }
  for (; row < a.rows; row += stride) {
    if (row + stride < a.rows) {
      load_row16<NCH>(a.x, (row + stride) * a.x_ld, lane, a.cols, nx);
      if (!G32) load_row16<G32 ? 1 : NCH>(a.g, (row + stride) * a.g_ld, lane, a.cols, ng);
    }
    float gf[G32 ? NCH : 1][8];
    if (G32) {
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int col = (c * 32 + lane) * 8;
        if (col < a.cols) load_vec<8>(static_cast<const char*>(a.g) + (row * a.g_ld + col) * 4, US_F32, gf[G32 ? c : 0]);
      }
    }
    float x[NCH][8];
#pragma unroll
    for (int c = 0; c < NCH; ++c) unpack16x8(cx[c], a.x_dt, x[c]);
    float mu, rstd;
    stats_regs<NCH>(x, lane, a.cols, a.eps, mu, rstd);
    float su = 0.f, sux = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        float g[8];
        if (G32) {
#pragma unroll
          for (int i = 0; i < 8; ++i) g[i] = gf[G32 ? c : 0][i];
        } else {
          unpack16x8(cg[G32 ? 0 : c], a.g_dt, g);
        }
        const float4 w0 = *reinterpret_cast<const float4*>(w_s + col), w1 = *reinterpret_cast<const float4*>(w_s + col + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float xh = (x[c][i] - mu) * rstd, uu = g[i] * w[i];
          x[c][i] = xh;
          su += uu;
          sux = fmaf(uu, xh, sux);
          sw[c][i] = fmaf(g[i], xh, sw[c][i]);
          sc[c][i] += g[i];
        }
      }
    }
    const float mean_u = warp_sum(su) * inv_n, mean_ux = warp_sum(sux) * inv_n;
    const float k = a.beta_x * rstd;
    const int64_t out_off = row * a.out_ld;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        float g[8], d[8];
        if (G32) {
#pragma unroll
          for (int i = 0; i < 8; ++i) g[i] = gf[G32 ? c : 0][i];
        } else {
          unpack16x8(cg[G32 ? 0 : c], a.g_dt, g);
        }
        const float4 w0 = *reinterpret_cast<const float4*>(w_s + col), w1 = *reinterpret_cast<const float4*>(w_s + col + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) d[i] = k * (g[i] * w[i] - mean_u - x[c][i] * mean_ux);
        store8(a.out, a.out_dt, out_off, col, a.cols, true, d);
      }
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) { cx[c] = nx[c]; if (!G32) cg[G32 ? 0 : c] = ng[G32 ? 0 : c]; }
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
        for (int i = 0; i < 8; ++i) comb[(size_t)warp * a.cols + col + i] = pass == 0 ? sw[c][i] : sc[c][i];
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
// One CTA per 32 columns of the 2 * cols sums: 8 groups of 32 threads each add every 8th partial row
// in order, then the groups are added in order.
__global__ void __launch_bounds__(256) ln_bwd_reduce_kernel(const float* partial, int nparts, int cols, float beta,
                                                            void* dw, int dw_dt, void* dc, int dc_dt) {
  __shared__ float acc[8][32];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + tx;               // index into [2][cols]
  float s = 0.f;
  if (j < 2 * cols)
    for (int p = ty; p < nparts; p += 8) s += partial[(size_t)p * 2 * cols + j];
  acc[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && j < 2 * cols) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) t += acc[q][tx];
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
    const size_t smem = (size_t)(1 + kLnFastWarps) * a.cols * sizeof(float);
#define US_LN_BWD16(N)                                                                             \
  do {                                                                                            \
    if (g32) ln_bwd16_kernel<N, true><<<nparts, 32 * kLnFastWarps, smem, st>>>(a);                \
    else ln_bwd16_kernel<N, false><<<nparts, 32 * kLnFastWarps, smem, st>>>(a);                   \
  } while (0)
    if (nch <= 1) US_LN_BWD16(1);
    else if (nch <= 2) US_LN_BWD16(2);
    else US_LN_BWD16(4);
#undef US_LN_BWD16
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
  ln_bwd_reduce_kernel<<<rgrid, 256, 0, st>>>(a.partial, nparts, a.cols, beta_wc, dw->ptr, dw->dtype, dc->ptr, dc->dtype);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}
