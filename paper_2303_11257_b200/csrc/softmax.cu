// Scaled softmax over the rows of a matrix, forward and backward (table "Table of unit scaling
// factors", row softmax: alpha = beta = s for rows of s elements; appendix paragraph "Softmax
// (followed by matmul)").  One warp per row, 128-bit loads and stores, warp-shuffle reductions;
// rows of up to 2048 elements are held in registers between the reduction and the write.
#include "common.cuh"
#include "host.h"
#include "rowwise.cuh"

namespace us {

constexpr int kSmThreads = 256;            // 8 rows per CTA
constexpr float kLog2e = 1.4426950408889634f;

struct SmArgs {
  const void* in0; int in0_dt; int64_t in0_ld;      // S (forward) or P (backward)
  const void* in1; int in1_dt; int64_t in1_ld;      // dP (backward only)
  void* out; int out_dt; int64_t out_ld;
  int64_t rows; int cols;
  int vec_ok;                                       // all row starts 16-byte aligned and cols % 8 == 0
  float alpha, beta;
};

// NCH > 0: the row fits in NCH chunks of 8 elements per lane, kept in registers.
// NCH == 0: any length; the row is re-read from global memory (cache) in each pass.
template <int NCH>
__global__ void __launch_bounds__(kSmThreads) softmax_fwd_kernel(const SmArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (kSmThreads / 32) + (threadIdx.x >> 5);
  if (row >= a.rows) return;
  const int64_t in_off = row * a.in0_ld, out_off = row * a.out_ld;
  const bool vec = a.vec_ok != 0;
  const int nch = NCH > 0 ? NCH : (a.cols + 255) / 256;
  float x[NCH > 0 ? NCH : 1][8];
  float m = -INFINITY;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    float t[8];
    if (col < a.cols) {
      load8(a.in0, a.in0_dt, in_off, col, a.cols, vec, -INFINITY, t);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = -INFINITY;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) { m = fmaxf(m, t[i]); if (NCH > 0) x[c][i] = t[i]; }
  }
  m = warp_max(m);
  const float mb = m * kLog2e;
  float sum = 0.f;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    float t[8];
    if (NCH > 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = x[c][i];
    } else if (col < a.cols) {
      load8(a.in0, a.in0_dt, in_off, col, a.cols, vec, -INFINITY, t);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = -INFINITY;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float e = ex2_approx(fmaf(t[i], kLog2e, -mb));    // exp(x - max); exp(-inf) = 0 for the padding
      sum += e;
      if (NCH > 0) x[c][i] = e;
    }
  }
  sum = warp_sum(sum);
  const float inv = a.alpha / sum;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col >= a.cols) continue;
    float t[8];
    if (NCH > 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = x[c][i] * inv;
    } else {
      load8(a.in0, a.in0_dt, in_off, col, a.cols, vec, -INFINITY, t);
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = ex2_approx(fmaf(t[i], kLog2e, -mb)) * inv;
    }
    store8(a.out, a.out_dt, out_off, col, a.cols, vec, t);
  }
}

template <int NCH>
__global__ void __launch_bounds__(kSmThreads) softmax_bwd_kernel(const SmArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (kSmThreads / 32) + (threadIdx.x >> 5);
  if (row >= a.rows) return;
  const int64_t p_off = row * a.in0_ld, g_off = row * a.in1_ld, out_off = row * a.out_ld;
  const bool vec = a.vec_ok != 0;
  const int nch = NCH > 0 ? NCH : (a.cols + 255) / 256;
  const float inv_alpha = 1.0f / a.alpha;
  float pt[NCH > 0 ? NCH : 1][8], g[NCH > 0 ? NCH : 1][8];
  float dot = 0.f;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    float tp[8], tg[8];
    if (col < a.cols) {
      load8(a.in0, a.in0_dt, p_off, col, a.cols, vec, 0.f, tp);
      load8(a.in1, a.in1_dt, g_off, col, a.cols, vec, 0.f, tg);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) { tp[i] = 0.f; tg[i] = 0.f; }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      tp[i] *= inv_alpha;                                   // softmax(S) recovered from the scaled output
      dot = fmaf(tp[i], tg[i], dot);
      if (NCH > 0) { pt[c][i] = tp[i]; g[c][i] = tg[i]; }
    }
  }
  dot = warp_sum(dot);
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col >= a.cols) continue;
    float tp[8], tg[8], t[8];
    if (NCH > 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) { tp[i] = pt[c][i]; tg[i] = g[c][i]; }
    } else {
      load8(a.in0, a.in0_dt, p_off, col, a.cols, vec, 0.f, tp);
      load8(a.in1, a.in1_dt, g_off, col, a.cols, vec, 0.f, tg);
#pragma unroll
      for (int i = 0; i < 8; ++i) tp[i] *= inv_alpha;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) t[i] = a.beta * tp[i] * (tg[i] - dot);
    store8(a.out, a.out_dt, out_off, col, a.cols, vec, t);
  }
}

// ---------------------------------------------------------------- 16-bit inputs, rows of at most 1024 elements
// Persistent warps: each walks rows grid-stride and fetches its next row, still packed, before working on
// the current one, so that a warp always has a row in flight.  Padding chunks (beyond the row) read as zero
// and are masked out of the maximum and the sums.
template <int NCH>
__global__ void __launch_bounds__(kSmThreads, 2) softmax_fwd16_kernel(const SmArgs a) {
  const int lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int64_t stride = (int64_t)gridDim.x * nw;
  int64_t row = (int64_t)blockIdx.x * nw + (threadIdx.x >> 5);
  uint4 cur[NCH], nxt[NCH];
  if (row < a.rows) load_row16<NCH>(a.in0, row * a.in0_ld, lane, a.cols, cur);
  for (; row < a.rows; row += stride) {
    if (row + stride < a.rows) load_row16<NCH>(a.in0, (row + stride) * a.in0_ld, lane, a.cols, nxt);
    float x[NCH][8];
    float m = -INFINITY;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      unpack16x8(cur[c], a.in0_dt, x[c]);
      if ((c * 32 + lane) * 8 < a.cols) {
#pragma unroll
        for (int i = 0; i < 8; ++i) m = fmaxf(m, x[c][i]);
      }
    }
    m = warp_max(m);
    const float mb = m * kLog2e;
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      if ((c * 32 + lane) * 8 < a.cols) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { x[c][i] = ex2_approx(fmaf(x[c][i], kLog2e, -mb)); sum += x[c][i]; }
      }
    }
    sum = warp_sum(sum);
    const float inv = a.alpha / sum;
    const int64_t out_off = row * a.out_ld;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        float t[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = x[c][i] * inv;
        store8(a.out, a.out_dt, out_off, col, a.cols, true, t);
      }
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) cur[c] = nxt[c];
  }
}

// dP 16-bit; P 16-bit of the same format, or (P8) FP8 codes as stored for an FP8 matmul.
template <int NCH, bool P8>
__global__ void __launch_bounds__(kSmThreads, 2) softmax_bwd16_kernel(const SmArgs a) {
  const int lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int64_t stride = (int64_t)gridDim.x * nw;
  const float inv_alpha = 1.0f / a.alpha;
  int64_t row = (int64_t)blockIdx.x * nw + (threadIdx.x >> 5);
  uint4 cp[P8 ? 1 : NCH], cg[NCH], np_[P8 ? 1 : NCH], ng[NCH];
  uint2 cp8[P8 ? NCH : 1], np8[P8 ? NCH : 1];
  if (row < a.rows) {
    if (P8) load_row8<P8 ? NCH : 1>(a.in0, row * a.in0_ld, lane, a.cols, cp8);
    else load_row16<P8 ? 1 : NCH>(a.in0, row * a.in0_ld, lane, a.cols, cp);
    load_row16<NCH>(a.in1, row * a.in1_ld, lane, a.cols, cg);
  }
  for (; row < a.rows; row += stride) {
    if (row + stride < a.rows) {
      if (P8) load_row8<P8 ? NCH : 1>(a.in0, (row + stride) * a.in0_ld, lane, a.cols, np8);
      else load_row16<P8 ? 1 : NCH>(a.in0, (row + stride) * a.in0_ld, lane, a.cols, np_);
      load_row16<NCH>(a.in1, (row + stride) * a.in1_ld, lane, a.cols, ng);
    }
    float pt[NCH][8], g[NCH][8];
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      if (P8) unpack8x8(cp8[P8 ? c : 0], a.in0_dt, pt[c]);
      else unpack16x8(cp[P8 ? 0 : c], a.in0_dt, pt[c]);
      unpack16x8(cg[c], a.in1_dt, g[c]);
#pragma unroll
      for (int i = 0; i < 8; ++i) { pt[c][i] *= inv_alpha; dot = fmaf(pt[c][i], g[c][i], dot); }   // padding: 0 * 0
    }
    dot = warp_sum(dot);
    const int64_t out_off = row * a.out_ld;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col = (c * 32 + lane) * 8;
      if (col < a.cols) {
        float t[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = a.beta * pt[c][i] * (g[c][i] - dot);
        store8(a.out, a.out_dt, out_off, col, a.cols, true, t);
      }
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      if (P8) cp8[P8 ? c : 0] = np8[P8 ? c : 0];
      else cp[P8 ? 0 : c] = np_[P8 ? 0 : c];
      cg[c] = ng[c];
    }
  }
}

// ---------------------------------------------------------------- softmax cross-entropy
// softmax_xent(x, t) = log softmax(x)_t (table row "softmax_xent": alpha = 1, beta = s / sqrt(s - 1)).
// One warp per row; the row is read twice (maximum, then sum of exponentials) from global memory /
// cache, which keeps any class count in one code path; the backward pass reads it a third time to write
// beta * g * (onehot(t) - softmax(x)).
struct XentArgs {
  const void* x; int x_dt; int64_t x_ld;
  const int32_t* t;
  const float* g;          // backward: one gradient per row, or null for ones
  void* out; int out_dt; int64_t out_ld;   // forward: float32 [rows]; backward: dX
  int64_t rows; int cols;
  int vec_ok;
  float beta;
};

template <bool BWD>
__global__ void __launch_bounds__(kSmThreads) softmax_xent_kernel(const XentArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (kSmThreads / 32) + (threadIdx.x >> 5);
  if (row >= a.rows) return;
  const int64_t x_off = row * a.x_ld;
  const bool vec = a.vec_ok != 0;
  const int nch = (a.cols + 255) / 256;
  float m = -INFINITY;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col >= a.cols) continue;
    float v[8];
    load8(a.x, a.x_dt, x_off, col, a.cols, vec, -INFINITY, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, v[i]);
  }
  m = warp_max(m);
  const float mb = m * kLog2e;
  float sum = 0.f;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col >= a.cols) continue;
    float v[8];
    load8(a.x, a.x_dt, x_off, col, a.cols, vec, -INFINITY, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += ex2_approx(fmaf(v[i], kLog2e, -mb));
  }
  sum = warp_sum(sum);
  const int t = a.t[row];
  const bool valid = t >= 0 && t < a.cols;                   // a target outside the row: NaN forward, no one-hot term backward
  if (!BWD) {
    if (lane == 0) {
      const float xt = valid ? load_one(a.x, a.x_dt, x_off + t) : __int_as_float(0x7fc00000);
      static_cast<float*>(a.out)[row] = (xt - m) - 0.6931471805599453f * __log2f(sum);
    }
    return;
  }
  const float k = a.beta * (a.g ? a.g[row] : 1.0f);
  const float inv = 1.0f / sum;
  const int64_t out_off = row * a.out_ld;
  for (int c = 0; c < nch; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col >= a.cols) continue;
    float v[8];
    load8(a.x, a.x_dt, x_off, col, a.cols, vec, -INFINITY, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float p = ex2_approx(fmaf(v[i], kLog2e, -mb)) * inv;
      v[i] = k * ((col + i == t ? 1.0f : 0.f) - p);
    }
    store8(a.out, a.out_dt, out_off, col, a.cols, vec, v);
  }
}

static bool rows_aligned(const us_mat* m) {
  return reinterpret_cast<uintptr_t>(m->ptr) % 16 == 0 && (m->ld * dtype_size(m->dtype)) % 16 == 0;
}

template <bool BWD>
static us_status launch_softmax(const SmArgs& a, cudaStream_t st) {
  if (a.rows == 0 || a.cols == 0) return US_OK;
  const int64_t grid64 = (a.rows + kSmThreads / 32 - 1) / (kSmThreads / 32);
  if (grid64 > 0x7fffffff) return US_ERR_INVALID_ARG;
  const int grid = (int)grid64;
  const int nch = (a.cols + 255) / 256;
  const bool in16 = a.in0_dt == US_BF16 || a.in0_dt == US_F16;
  const bool p8 = BWD && (a.in0_dt == US_E4M3 || a.in0_dt == US_E5M2) && (a.in1_dt == US_BF16 || a.in1_dt == US_F16);
  if (a.vec_ok && nch <= 4 && ((in16 && (!BWD || a.in1_dt == a.in0_dt)) || p8)) {
    const int sms = host::sm_count();
    if (sms <= 0) return US_ERR_CUDA;
    const int pgrid = grid < 2 * sms ? grid : 2 * sms;        // two resident CTAs per SM, warps walk the rows
#define US_SM16(N)                                                                   \
  do {                                                                               \
    if (BWD && p8) softmax_bwd16_kernel<N, true><<<pgrid, kSmThreads, 0, st>>>(a);   \
    else if (BWD) softmax_bwd16_kernel<N, false><<<pgrid, kSmThreads, 0, st>>>(a);   \
    else softmax_fwd16_kernel<N><<<pgrid, kSmThreads, 0, st>>>(a);                   \
  } while (0)
    if (nch <= 1) US_SM16(1);
    else if (nch <= 2) US_SM16(2);
    else US_SM16(4);
#undef US_SM16
    return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
  }
#define US_SM_LAUNCH(N)                                                          \
  do {                                                                           \
    if (BWD) softmax_bwd_kernel<N><<<grid, kSmThreads, 0, st>>>(a);              \
    else softmax_fwd_kernel<N><<<grid, kSmThreads, 0, st>>>(a);                  \
  } while (0)
  if (nch <= 1) US_SM_LAUNCH(1);
  else if (nch <= 2) US_SM_LAUNCH(2);
  else if (nch <= 4) US_SM_LAUNCH(4);
  else if (nch <= 8 && !BWD) US_SM_LAUNCH(8);
  else US_SM_LAUNCH(0);
#undef US_SM_LAUNCH
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

// input: a tensor the kernel reads (float formats; FP8 too where fp8_in says so).
static us_status check_mat(const us_mat* m, const us_mat* like, bool input, bool fp8_in = false) {
  if (!m || m->rows < 0 || m->cols < 0 || m->ld < m->cols) return US_ERR_INVALID_ARG;
  if (like && (m->rows != like->rows || m->cols != like->cols)) return US_ERR_INVALID_ARG;
  if (m->rows * m->cols > 0 && !m->ptr) return US_ERR_INVALID_ARG;
  if (m->cols > 0x7ffffff0) return US_ERR_INVALID_ARG;
  const bool is_fp8 = m->dtype == US_E4M3 || m->dtype == US_E5M2;
  if (input ? !(m->dtype == US_F32 || m->dtype == US_BF16 || m->dtype == US_F16 || (fp8_in && is_fp8)) : !(m->dtype >= US_F32 && m->dtype <= US_E5M2))
    return US_ERR_UNSUPPORTED;
  if (m->ptr && reinterpret_cast<uintptr_t>(m->ptr) % dtype_size(m->dtype)) return US_ERR_ALIGNMENT;
  return US_OK;
}

}  // namespace us

using namespace us;

extern "C" us_status us_softmax_fwd(const us_mat* S, float alpha, const us_mat* P, void* stream) {
  us_status s = check_mat(S, nullptr, true);
  if (s == US_OK) s = check_mat(P, S, false);
  if (s != US_OK) return s;
  SmArgs a{};
  a.in0 = S->ptr; a.in0_dt = S->dtype; a.in0_ld = S->ld;
  a.out = P->ptr; a.out_dt = P->dtype; a.out_ld = P->ld;
  a.rows = S->rows; a.cols = (int)S->cols; a.alpha = alpha; a.beta = 0.f;
  a.vec_ok = rows_aligned(S) && rows_aligned(P) && S->cols % 8 == 0;
  return launch_softmax<false>(a, static_cast<cudaStream_t>(stream));
}

extern "C" us_status us_softmax_bwd(const us_mat* P, const us_mat* dP, float alpha, float beta, const us_mat* dS,
                                    void* stream) {
  us_status s = check_mat(P, nullptr, true, true);           // the stored forward output may be FP8
  if (s == US_OK) s = check_mat(dP, P, true);
  if (s == US_OK) s = check_mat(dS, P, false);
  if (s != US_OK) return s;
  if (!(alpha > 0.f)) return US_ERR_INVALID_ARG;
  SmArgs a{};
  a.in0 = P->ptr; a.in0_dt = P->dtype; a.in0_ld = P->ld;
  a.in1 = dP->ptr; a.in1_dt = dP->dtype; a.in1_ld = dP->ld;
  a.out = dS->ptr; a.out_dt = dS->dtype; a.out_ld = dS->ld;
  a.rows = P->rows; a.cols = (int)P->cols; a.alpha = alpha; a.beta = beta;
  a.vec_ok = rows_aligned(P) && rows_aligned(dP) && rows_aligned(dS) && P->cols % 8 == 0;
  return launch_softmax<true>(a, static_cast<cudaStream_t>(stream));
}

static us_status check_xent(const us_mat* X, const int32_t* targets) {
  us_status s = check_mat(X, nullptr, true);
  if (s != US_OK) return s;
  if (X->rows > 0 && !targets) return US_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(targets) % 4) return US_ERR_ALIGNMENT;
  if (X->rows > 0 && X->cols < 1) return US_ERR_INVALID_ARG;
  return US_OK;
}

extern "C" us_status us_softmax_xent_fwd(const us_mat* X, const int32_t* targets, float* out, void* stream) {
  us_status s = check_xent(X, targets);
  if (s != US_OK) return s;
  if (X->rows == 0) return US_OK;
  if (!out || reinterpret_cast<uintptr_t>(out) % 4) return US_ERR_INVALID_ARG;
  XentArgs a{};
  a.x = X->ptr; a.x_dt = X->dtype; a.x_ld = X->ld; a.t = targets; a.out = out;
  a.rows = X->rows; a.cols = (int)X->cols;
  a.vec_ok = rows_aligned(X) && X->cols % 8 == 0;
  const int64_t grid = (a.rows + kSmThreads / 32 - 1) / (kSmThreads / 32);
  if (grid > 0x7fffffff) return US_ERR_INVALID_ARG;
  softmax_xent_kernel<false><<<(int)grid, kSmThreads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

extern "C" us_status us_softmax_xent_bwd(const us_mat* X, const int32_t* targets, const float* g, float beta,
                                         const us_mat* dX, void* stream) {
  us_status s = check_xent(X, targets);
  if (s == US_OK) s = check_mat(dX, X, false);
  if (s != US_OK) return s;
  if (g && reinterpret_cast<uintptr_t>(g) % 4) return US_ERR_ALIGNMENT;
  if (X->rows == 0) return US_OK;
  XentArgs a{};
  a.x = X->ptr; a.x_dt = X->dtype; a.x_ld = X->ld; a.t = targets; a.g = g;
  a.out = dX->ptr; a.out_dt = dX->dtype; a.out_ld = dX->ld;
  a.rows = X->rows; a.cols = (int)X->cols; a.beta = beta;
  a.vec_ok = rows_aligned(X) && rows_aligned(dX) && X->cols % 8 == 0;
  const int64_t grid = (a.rows + kSmThreads / 32 - 1) / (kSmThreads / 32);
  if (grid > 0x7fffffff) return US_ERR_INVALID_ARG;
  softmax_xent_kernel<true><<<(int)grid, kSmThreads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}
