// Unfused elementwise ops of libunitscale: FP8 cast, scaled GELU forward/backward,
// tau-weighted residual add.  All are HBM-bandwidth bound: each thread moves 16
// elements per iteration with 128-bit loads and stores; the grid is a multiple of
// the SM count and strides over the tensor.
#include "common.cuh"
#include "host.h"

namespace us {

constexpr int kVec = 16;       // elements per thread per iteration
constexpr int kThreads = 256;

struct EwTensor {
  void* ptr;
  int dt;
  int64_t ld;
};

struct EwArgs {
  EwTensor in0, in1, out;
  int64_t rows, cols;
  int64_t chunks_per_row;  // ceil(cols / kVec)
  int vec_ok;              // every row start of every tensor is 16-byte aligned
  float c0, c1, c2;        // op constants
  int fn;                  // us_fn of the activation ops
};

enum EwOp { kCast = 0, kGeluFwd = 1, kGeluBwd = 2, kResidual = 3, kActFwd = 4, kActBwd = 5 };

template <int OP>
__device__ __forceinline__ float ew_apply(float a, float b, const EwArgs& p) {
  if (OP == kActFwd)                                                          // c0 = s_in, c1 = alpha
    return p.fn == US_FN_GELU ? gelu_scaled(a, p.c0, p.c1) : p.c1 * act_value(p.fn, p.c0 * a);
  if (OP == kActBwd)                                                          // a = H, b = dA, c1 = beta
    return p.fn == US_FN_GELU ? gelu_grad_scaled(a, b, p.c0, p.c1) : (p.c1 * p.c0) * act_slope(p.fn, p.c0 * a) * b;
  if (OP == kCast) return p.c0 * a;                                   // scale * x, then the store rounds
  if (OP == kGeluFwd) {                                               // c0 = s_in, c1 = alpha; same arithmetic as the pair form
    float y0, y1;
    gelu_scaled2<false>(pack2(a, a), fabsf(p.c0) * (1.0f / kTailRange), p.c1 * p.c0, y0, y1);
    return y0;
  }
  if (OP == kGeluBwd) {                                               // a = H, b = dA, c1 = beta
    float y0, y1;
    unpack2(gelu_grad_scaled2(pack2(a, a), pack2(b, b), splat2(p.c0), splat2(p.c1 * p.c0)), y0, y1);
    return y0;
  }
  return fmaf(p.c0, a, p.c1 * b);                                     // c0 = sqrt(1-tau), c1 = sqrt(tau)
}

template <int OP>
__global__ void __launch_bounds__(kThreads) ew_kernel(const EwArgs p) {
  constexpr bool kTwoInputs = (OP == kGeluBwd || OP == kResidual || OP == kActBwd);
  const int64_t total = p.rows * p.chunks_per_row;
  for (int64_t c = blockIdx.x * (int64_t)kThreads + threadIdx.x; c < total;
       c += (int64_t)gridDim.x * kThreads) {
    const int64_t row = p.rows == 1 ? 0 : c / p.chunks_per_row;      // tensors without row padding arrive as one long row
    const int64_t col = (c - row * p.chunks_per_row) * kVec;
    const int64_t i0 = row * p.in0.ld + col, i1 = row * p.in1.ld + col, io = row * p.out.ld + col;
    if (p.vec_ok && col + kVec <= p.cols) {
      float a[kVec], b[kVec], o[kVec];
      load_vec<kVec>(static_cast<const char*>(p.in0.ptr) + i0 * dtype_size(p.in0.dt), p.in0.dt, a);
      if (kTwoInputs) load_vec<kVec>(static_cast<const char*>(p.in1.ptr) + i1 * dtype_size(p.in1.dt), p.in1.dt, b);
      if (OP == kGeluFwd) {                          // two values per instruction (packed float32 arithmetic)
        const float k = fabsf(p.c0) * (1.0f / kTailRange), oi = p.c1 * p.c0;
#pragma unroll
        for (int i = 0; i < kVec; i += 2) gelu_scaled2<false>(pack2(a[i], a[i + 1]), k, oi, o[i], o[i + 1]);
      } else if (OP == kGeluBwd) {
        const f32x2 in2 = splat2(p.c0), os2 = splat2(p.c1 * p.c0);
#pragma unroll
        for (int i = 0; i < kVec; i += 2)
          unpack2(gelu_grad_scaled2(pack2(a[i], a[i + 1]), pack2(b[i], b[i + 1]), in2, os2), o[i], o[i + 1]);
      } else {
#pragma unroll
        for (int i = 0; i < kVec; ++i) o[i] = ew_apply<OP>(a[i], kTwoInputs ? b[i] : 0.f, p);
      }
      store_vec<kVec>(static_cast<char*>(p.out.ptr) + io * dtype_size(p.out.dt), p.out.dt, o);
    } else {
      const int n = (int)min((int64_t)kVec, p.cols - col);
      for (int i = 0; i < n; ++i) {
        const float a = load_one(p.in0.ptr, p.in0.dt, i0 + i);
        const float b = kTwoInputs ? load_one(p.in1.ptr, p.in1.dt, i1 + i) : 0.f;
        store_one(p.out.ptr, p.out.dt, io + i, ew_apply<OP>(a, b, p));
      }
    }
  }
}

// Several casts in one launch: the chunks of all tensors are numbered consecutively and a thread finds
// the tensor of its chunk by scanning the (at most kMultiMax) cumulative counts.  Tensors are contiguous
// and 16-byte aligned (checked on the host), so every chunk but a tensor's last takes the vector path.
constexpr int kMultiMax = 8;
struct MultiCastArgs {
  const void* src[kMultiMax];
  void* dst[kMultiMax];
  int64_t elems[kMultiMax];
  int64_t chunk_end[kMultiMax];   // cumulative chunk counts
  float scale[kMultiMax];
  int src_dt[kMultiMax], dst_dt[kMultiMax];
  int count;
};

struct MultiChunk {
  const char* src; char* dst; float scale; int sdt, ddt, t; int64_t e0; bool full;
};
__device__ __forceinline__ MultiChunk multi_locate(const MultiCastArgs& p, int64_t c) {
  MultiChunk m;
  int t = 0;
  while (c >= p.chunk_end[t]) ++t;
  m.t = t;
  m.e0 = (c - (t ? p.chunk_end[t - 1] : 0)) * kVec;
  m.sdt = p.src_dt[t]; m.ddt = p.dst_dt[t];
  m.src = static_cast<const char*>(p.src[t]) + m.e0 * dtype_size(m.sdt);
  m.dst = static_cast<char*>(p.dst[t]) + m.e0;                          // FP8: one byte per element
  m.scale = p.scale[t];
  m.full = m.e0 + kVec <= p.elems[t];
  return m;
}
__device__ __forceinline__ void multi_tail(const MultiCastArgs& p, const MultiChunk& m) {
  for (int64_t i = 0; m.e0 + i < p.elems[m.t]; ++i)
    store_one(p.dst[m.t], m.ddt, m.e0 + i, m.scale * load_one(p.src[m.t], m.sdt, m.e0 + i));
}

// Two chunks per thread and iteration, both loaded before either is stored, to keep more loads in flight.
__global__ void __launch_bounds__(kThreads) multi_cast_kernel(const MultiCastArgs p) {
  const int64_t total = p.chunk_end[p.count - 1];
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t c = blockIdx.x * (int64_t)kThreads + threadIdx.x; c < total; c += 2 * stride) {
    const MultiChunk m0 = multi_locate(p, c);
    const bool two = c + stride < total;
    const MultiChunk m1 = two ? multi_locate(p, c + stride) : m0;
    float a[kVec], b[kVec];
    if (m0.full) load_vec<kVec>(m0.src, m0.sdt, a);
    if (two && m1.full) load_vec<kVec>(m1.src, m1.sdt, b);
    if (m0.full) {
#pragma unroll
      for (int i = 0; i < kVec; ++i) a[i] *= m0.scale;
      store_vec<kVec>(m0.dst, m0.ddt, a);
    } else {
      multi_tail(p, m0);
    }
    if (two) {
      if (m1.full) {
#pragma unroll
        for (int i = 0; i < kVec; ++i) b[i] *= m1.scale;
        store_vec<kVec>(m1.dst, m1.ddt, b);
      } else {
        multi_tail(p, m1);
      }
    }
  }
}

// alpha * sum_i gamma_i x_i over up to kMultiMax tensors of one shape (table row "weighted_add").
struct WeightedAddArgs {
  const void* src[kMultiMax];
  int src_dt[kMultiMax];
  int64_t src_ld[kMultiMax];
  float coef[kMultiMax];          // alpha * gamma_i
  void* out; int out_dt; int64_t out_ld;
  int count;
  int64_t rows, cols, chunks_per_row;
  int vec_ok;
};

__global__ void __launch_bounds__(kThreads) weighted_add_kernel(const WeightedAddArgs p) {
  const int64_t total = p.rows * p.chunks_per_row;
  for (int64_t c = blockIdx.x * (int64_t)kThreads + threadIdx.x; c < total; c += (int64_t)gridDim.x * kThreads) {
    const int64_t row = c / p.chunks_per_row;
    const int64_t col = (c - row * p.chunks_per_row) * kVec;
    if (p.vec_ok && col + kVec <= p.cols) {
      float acc[kVec];
#pragma unroll
      for (int i = 0; i < kVec; ++i) acc[i] = 0.f;
      for (int t = 0; t < p.count; ++t) {
        float a[kVec];
        load_vec<kVec>(static_cast<const char*>(p.src[t]) + (row * p.src_ld[t] + col) * dtype_size(p.src_dt[t]), p.src_dt[t], a);
#pragma unroll
        for (int i = 0; i < kVec; ++i) acc[i] = fmaf(p.coef[t], a[i], acc[i]);
      }
      store_vec<kVec>(static_cast<char*>(p.out) + (row * p.out_ld + col) * dtype_size(p.out_dt), p.out_dt, acc);
    } else {
      const int n = (int)min((int64_t)kVec, p.cols - col);
      for (int i = 0; i < n; ++i) {
        float acc = 0.f;
        for (int t = 0; t < p.count; ++t) acc = fmaf(p.coef[t], load_one(p.src[t], p.src_dt[t], row * p.src_ld[t] + col + i), acc);
        store_one(p.out, p.out_dt, row * p.out_ld + col + i, acc);
      }
    }
  }
}

static bool row_starts_aligned(const us_mat* m, bool contiguous) {
  const int es = dtype_size(m->dtype);
  if (reinterpret_cast<uintptr_t>(m->ptr) % 16) return false;
  return contiguous || (m->ld * es) % 16 == 0;
}

template <int OP>
static us_status ew_launch(const us_mat* in0, const us_mat* in1, const us_mat* out, float c0, float c1,
                           void* stream, int fn = 0) {
  EwArgs p{};
  p.fn = fn;
  // A tensor set without row padding is one long row: chunking then never straddles a row end.
  const bool contiguous = in0->ld == in0->cols && (!in1 || in1->ld == in1->cols) && out->ld == out->cols;
  p.rows = contiguous ? 1 : in0->rows;
  p.cols = contiguous ? in0->rows * in0->cols : in0->cols;
  p.in0 = {in0->ptr, in0->dtype, in0->ld};
  p.in1 = in1 ? EwTensor{in1->ptr, in1->dtype, in1->ld} : p.in0;
  p.out = {out->ptr, out->dtype, out->ld};
  p.chunks_per_row = (p.cols + kVec - 1) / kVec;
  p.vec_ok = row_starts_aligned(in0, contiguous) && (!in1 || row_starts_aligned(in1, contiguous)) &&
             row_starts_aligned(out, contiguous);
  p.c0 = c0; p.c1 = c1;
  const int64_t total = p.rows * p.chunks_per_row;
  if (total == 0) return US_OK;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const int64_t want = (total + kThreads - 1) / kThreads;
  const int64_t cap = (int64_t)sms * 8;                 // 8 resident CTAs of 256 threads per SM
  const int grid = (int)(want < cap ? want : cap);
  ew_kernel<OP><<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

}  // namespace us

using namespace us;

static bool is_float_in(int dt) { return dt == US_F32 || dt == US_BF16 || dt == US_F16; }
static bool is_dtype(int dt) { return dt >= US_F32 && dt <= US_E5M2; }

static us_status check_ew(const us_mat* a, const us_mat* b, const us_mat* out) {
  const us_mat* ms[3] = {a, b, out};
  for (int i = 0; i < 3; ++i) {
    const us_mat* m = ms[i];
    if (i == 1 && !m) continue;
    if (!m || m->rows < 0 || m->cols < 0 || m->ld < m->cols) return US_ERR_INVALID_ARG;
    if (m->rows != a->rows || m->cols != a->cols) return US_ERR_INVALID_ARG;
    if (m->rows * m->cols > 0 && !m->ptr) return US_ERR_INVALID_ARG;
    if (i < 2 ? !is_float_in(m->dtype) : !is_dtype(m->dtype)) return US_ERR_UNSUPPORTED;
    if (m->ptr && reinterpret_cast<uintptr_t>(m->ptr) % dtype_size(m->dtype)) return US_ERR_ALIGNMENT;
  }
  return US_OK;
}

extern "C" us_status us_cast_fp8(const us_mat* src, float scale, const us_mat* dst, void* stream) {
  us_status s = check_ew(src, nullptr, dst);
  if (s != US_OK) return s;
  if (dst->dtype != US_E4M3 && dst->dtype != US_E5M2) return US_ERR_UNSUPPORTED;
  return ew_launch<kCast>(src, nullptr, dst, scale, 0.f, stream);
}

extern "C" us_status us_cast_fp8_multi(int count, const us_mat* src, const float* scale, const us_mat* dst, void* stream) {
  if (count < 1 || count > kMultiMax || !src || !scale || !dst) return US_ERR_INVALID_ARG;
  MultiCastArgs p{};
  int64_t chunks = 0;
  int used = 0;
  for (int i = 0; i < count; ++i) {
    us_status s = check_ew(&src[i], nullptr, &dst[i]);
    if (s != US_OK) return s;
    if (dst[i].dtype != US_E4M3 && dst[i].dtype != US_E5M2) return US_ERR_UNSUPPORTED;
    const int64_t n = src[i].rows * src[i].cols;
    if (n == 0) continue;
    const bool dense = (src[i].ld == src[i].cols && dst[i].ld == dst[i].cols) || src[i].rows == 1;
    if (!dense) return US_ERR_UNSUPPORTED;                               // padded rows: use us_cast_fp8
    if (reinterpret_cast<uintptr_t>(src[i].ptr) % 16 || reinterpret_cast<uintptr_t>(dst[i].ptr) % 16) return US_ERR_ALIGNMENT;
    p.src[used] = src[i].ptr; p.dst[used] = dst[i].ptr; p.elems[used] = n; p.scale[used] = scale[i];
    p.src_dt[used] = src[i].dtype; p.dst_dt[used] = dst[i].dtype;
    chunks += (n + kVec - 1) / kVec;
    p.chunk_end[used] = chunks;
    ++used;
  }
  if (used == 0) return US_OK;
  p.count = used;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const int64_t want = (chunks + kThreads - 1) / kThreads;
  const int64_t cap = (int64_t)sms * 8;
  multi_cast_kernel<<<(int)(want < cap ? want : cap), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

extern "C" us_status us_weighted_add(int count, const us_mat* src, const float* gamma, float alpha, const us_mat* out,
                                      void* stream) {
  if (count < 1 || count > kMultiMax || !src || !gamma || !out) return US_ERR_INVALID_ARG;
  if (out->rows < 0 || out->cols < 0 || out->ld < out->cols || (out->rows * out->cols > 0 && !out->ptr)) return US_ERR_INVALID_ARG;
  if (!is_dtype(out->dtype)) return US_ERR_UNSUPPORTED;
  if (out->ptr && reinterpret_cast<uintptr_t>(out->ptr) % dtype_size(out->dtype)) return US_ERR_ALIGNMENT;
  WeightedAddArgs p{};
  bool vec = row_starts_aligned(out, false);
  for (int i = 0; i < count; ++i) {
    // inputs may also be FP8 tensors (partial results that travelled in 8 bits): checked like an output dtype
    const us_mat* m = &src[i];
    if (m->rows < 0 || m->cols < 0 || m->ld < m->cols || m->rows != out->rows || m->cols != out->cols) return US_ERR_INVALID_ARG;
    if (m->rows * m->cols > 0 && !m->ptr) return US_ERR_INVALID_ARG;
    if (!is_dtype(m->dtype)) return US_ERR_UNSUPPORTED;
    if (m->ptr && reinterpret_cast<uintptr_t>(m->ptr) % dtype_size(m->dtype)) return US_ERR_ALIGNMENT;
    p.src[i] = src[i].ptr; p.src_dt[i] = src[i].dtype; p.src_ld[i] = src[i].ld;
    p.coef[i] = alpha * gamma[i];
    vec = vec && row_starts_aligned(&src[i], false);
  }
  p.out = out->ptr; p.out_dt = out->dtype; p.out_ld = out->ld;
  p.count = count; p.rows = out->rows; p.cols = out->cols;
  p.chunks_per_row = (p.cols + kVec - 1) / kVec;
  p.vec_ok = vec;
  const int64_t total = p.rows * p.chunks_per_row;
  if (total == 0) return US_OK;
  const int sms = host::sm_count();
  if (sms <= 0) return US_ERR_CUDA;
  const int64_t want = (total + kThreads - 1) / kThreads, cap = (int64_t)sms * 8;
  weighted_add_kernel<<<(int)(want < cap ? want : cap), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}

extern "C" us_status us_gelu_fwd(const us_mat* H, float s_in, float alpha, const us_mat* A, void* stream) {
  us_status s = check_ew(H, nullptr, A);
  if (s != US_OK) return s;
  return ew_launch<kGeluFwd>(H, nullptr, A, s_in, alpha, stream);
}

extern "C" us_status us_gelu_bwd(const us_mat* H, const us_mat* dA, float s_in, float beta, const us_mat* dH,
                                 void* stream) {
  if (!dA) return US_ERR_INVALID_ARG;
  us_status s = check_ew(H, dA, dH);
  if (s != US_OK) return s;
  return ew_launch<kGeluBwd>(H, dA, dH, s_in, beta, stream);
}

extern "C" us_status us_activation_fwd(us_fn fn, const us_mat* H, float s_in, float alpha, const us_mat* A, void* stream) {
  if (fn < US_FN_GELU || fn > US_FN_SIGMOID) return US_ERR_INVALID_ARG;
  us_status s = check_ew(H, nullptr, A);
  if (s != US_OK) return s;
  if (fn == US_FN_GELU) return ew_launch<kGeluFwd>(H, nullptr, A, s_in, alpha, stream);
  return ew_launch<kActFwd>(H, nullptr, A, s_in, alpha, stream, fn);
}

extern "C" us_status us_activation_bwd(us_fn fn, const us_mat* H, const us_mat* dA, float s_in, float beta,
                                       const us_mat* dH, void* stream) {
  if (fn < US_FN_GELU || fn > US_FN_SIGMOID || !dA) return US_ERR_INVALID_ARG;
  us_status s = check_ew(H, dA, dH);
  if (s != US_OK) return s;
  if (fn == US_FN_GELU) return ew_launch<kGeluBwd>(H, dA, dH, s_in, beta, stream);
  return ew_launch<kActBwd>(H, dA, dH, s_in, beta, stream, fn);
}

extern "C" us_status us_residual_add(const us_mat* skip, const us_mat* branch, float tau, const us_mat* out,
                                     void* stream) {
  if (!branch) return US_ERR_INVALID_ARG;
  us_status s = check_ew(skip, branch, out);
  if (s != US_OK) return s;
  if (!(tau >= 0.f && tau <= 1.f)) return US_ERR_INVALID_ARG;
  const float c_skip = (float)sqrt(1.0 - (double)tau), c_branch = (float)sqrt((double)tau);
  return ew_launch<kResidual>(skip, branch, out, c_skip, c_branch, stream);
}
