// Quantisation diagnostics on device: the signal-to-noise ratio of a cast (section "Floating-point
// formats for deep learning", paragraph "Quantisation error": SNR = E[X^2] / E[(q(X) - X)^2]) and the
// histogram of floor(log2 |x|) (appendix "Histograms of tensor-scaling within BERT").
//
// One pass over the tensor (an analysis tool, not on the training path: 128-bit loads where the tensor has no row
// padding, a per-element update of a per-warp shared-memory histogram; bound by those updates and the double-precision
// sums, not by memory).  Every CTA accumulates its sums in double precision and its bin counts in shared-memory integers, and writes one partial record to the caller's workspace; a second,
// single-CTA kernel adds the records in order.  No global atomics and nothing to zero beforehand: the
// result is the same from run to run.
#include "common.cuh"
#include "host.h"

namespace us {

constexpr int kDiagThreads = 256;
constexpr int kDiagMaxBins = 64;
constexpr int kDiagRecord = 2 + kDiagMaxBins + 2;      // doubles / 64-bit words per CTA record

struct DiagArgs {
  const void* src; int src_dt; int64_t ld;
  int64_t rows, cols;
  float scale;
  int fmt;                 // format whose rounding error is measured
  int exp_lo, nbins;
  int vec_ok;              // no row padding and a 16-byte aligned base: 128-bit loads
  unsigned long long* partial;   // [gridDim.x][kDiagRecord]
};

// q(v) for the four storage formats: FP8 saturating, 16-bit IEEE (overflow -> infinity).
__device__ __forceinline__ float round_to(float v, int fmt) {
  if (fmt == US_E4M3) return unpack_fp8x2(cvt_e4m3x2(v, 0.f), false).x;
  if (fmt == US_E5M2) return unpack_fp8x2(cvt_e5m2x2(v, 0.f), true).x;
  if (fmt == US_BF16) return __bfloat162float(__float2bfloat16_rn(v));
  return __half2float(__float2half_rn(v));
}

__global__ void __launch_bounds__(kDiagThreads) quant_stats_kernel(const DiagArgs a) {
  // one histogram per warp (less contention on the few popular bins), added in warp order at the end
  __shared__ unsigned int bins[kDiagThreads / 32][kDiagMaxBins + 2];
  __shared__ double warp_sums[2][kDiagThreads / 32];
  for (int i = threadIdx.x; i < (kDiagThreads / 32) * (kDiagMaxBins + 2); i += kDiagThreads) (&bins[0][0])[i] = 0u;
  __syncthreads();
  unsigned int* my_bins = bins[threadIdx.x >> 5];
  double s_sig = 0.0, s_err = 0.0;
  auto take = [&](float x) {
    const float v = a.scale * x;
    const float e = round_to(v, a.fmt) - v;
    s_sig += (double)v * (double)v;
    s_err += (double)e * (double)e;
    // floor(log2 |v|) is the exponent field of a normal float32; zeros and subnormals fall below any bin
    const unsigned int bits = __float_as_uint(v) & 0x7fffffffu;
    const int ex = (int)(bits >> 23) - 127;
    int bin;
    if (bits >= 0x7f800000u) bin = a.nbins + 1;                       // infinity or NaN
    else if (ex < a.exp_lo) bin = 0;
    else if (ex >= a.exp_lo + a.nbins) bin = a.nbins + 1;
    else bin = 1 + ex - a.exp_lo;
    atomicAdd(&my_bins[bin], 1u);
  };
  const int64_t total = a.rows * a.cols;
  if (a.vec_ok) {
    // no row padding, 16-byte aligned: eight elements per thread and step with 128-bit loads
    const int64_t chunks = total / 8;
    const int es = dtype_size(a.src_dt);
    for (int64_t c = blockIdx.x * (int64_t)kDiagThreads + threadIdx.x; c < chunks; c += (int64_t)gridDim.x * kDiagThreads) {
      float x[8];
      load_vec<8>(static_cast<const char*>(a.src) + c * 8 * es, a.src_dt, x);
#pragma unroll
      for (int i = 0; i < 8; ++i) take(x[i]);
    }
    if (blockIdx.x == 0 && threadIdx.x < (int)(total - chunks * 8)) take(load_one(a.src, a.src_dt, chunks * 8 + threadIdx.x));
  } else {
    for (int64_t i = blockIdx.x * (int64_t)kDiagThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kDiagThreads) {
      const int64_t r = i / a.cols, c = i - r * a.cols;
      take(load_one(a.src, a.src_dt, r * a.ld + c));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s_sig += __shfl_xor_sync(0xffffffffu, s_sig, o);
    s_err += __shfl_xor_sync(0xffffffffu, s_err, o);
  }
  if ((threadIdx.x & 31) == 0) { warp_sums[0][threadIdx.x >> 5] = s_sig; warp_sums[1][threadIdx.x >> 5] = s_err; }
  __syncthreads();
  unsigned long long* rec = a.partial + (size_t)blockIdx.x * kDiagRecord;
  if (threadIdx.x < 2) {
    double t = 0.0;
    for (int w = 0; w < kDiagThreads / 32; ++w) t += warp_sums[threadIdx.x][w];
    rec[threadIdx.x] = (unsigned long long)__double_as_longlong(t);
  }
  for (int i = threadIdx.x; i < a.nbins + 2; i += kDiagThreads) {
    unsigned int t = 0u;
    for (int w = 0; w < kDiagThreads / 32; ++w) t += bins[w][i];
    rec[2 + i] = t;
  }
}

// sums[0..1] and hist[0 .. nbins + 1]: the CTAs' records added in CTA order.
__global__ void __launch_bounds__(128) quant_stats_reduce_kernel(const unsigned long long* partial, int nparts, int nbins,
                                                                 double* sums, unsigned long long* hist) {
  const int j = threadIdx.x;
  if (j < 2) {
    double t = 0.0;
    for (int p = 0; p < nparts; ++p) t += __longlong_as_double((long long)partial[(size_t)p * kDiagRecord + j]);
    sums[j] = t;
  } else if (j - 2 < nbins + 2) {
    unsigned long long t = 0ull;
    for (int p = 0; p < nparts; ++p) t += partial[(size_t)p * kDiagRecord + j];
    hist[j - 2] = t;
  }
}

static int diag_grid(int64_t total) {
  const int sms = host::sm_count();
  if (sms <= 0) return 0;
  const int64_t want = (total + kDiagThreads - 1) / kDiagThreads;
  const int64_t cap = (int64_t)sms * 8;
  const int64_t g = want < cap ? want : cap;
  return (int)(g < 1 ? 1 : g);
}

}  // namespace us

using namespace us;

extern "C" size_t us_quant_stats_workspace_bytes(void) {
  const int sms = host::sm_count();
  return (size_t)(sms > 0 ? sms : 1) * 8 * kDiagRecord * sizeof(unsigned long long);
}

extern "C" us_status us_quant_stats(const us_mat* src, float scale, us_dtype fmt, int exp_lo, int nbins, double* sums,
                                    unsigned long long* hist, void* ws, size_t ws_bytes, void* stream) {
  if (!src || src->rows < 0 || src->cols < 0 || src->ld < src->cols || !sums || !hist) return US_ERR_INVALID_ARG;
  if (src->rows * src->cols > 0 && !src->ptr) return US_ERR_INVALID_ARG;
  if (nbins < 1 || nbins > kDiagMaxBins || exp_lo < -126 || exp_lo + nbins > 128) return US_ERR_INVALID_ARG;
  if (src->dtype != US_F32 && src->dtype != US_BF16 && src->dtype != US_F16) return US_ERR_UNSUPPORTED;
  if (fmt != US_BF16 && fmt != US_F16 && fmt != US_E4M3 && fmt != US_E5M2) return US_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(sums) % 8 || reinterpret_cast<uintptr_t>(hist) % 8) return US_ERR_ALIGNMENT;
  if (src->ptr && reinterpret_cast<uintptr_t>(src->ptr) % dtype_size(src->dtype)) return US_ERR_ALIGNMENT;
  const int grid = diag_grid(src->rows * src->cols);
  if (grid <= 0) return US_ERR_CUDA;
  if (!ws || ws_bytes < us_quant_stats_workspace_bytes()) return US_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % 8) return US_ERR_ALIGNMENT;
  DiagArgs a{};
  a.src = src->ptr; a.src_dt = src->dtype; a.ld = src->ld; a.rows = src->rows; a.cols = src->cols;
  a.scale = scale; a.fmt = fmt; a.exp_lo = exp_lo; a.nbins = nbins;
  a.vec_ok = (src->ld == src->cols || src->rows <= 1) && reinterpret_cast<uintptr_t>(src->ptr) % 16 == 0;
  a.partial = static_cast<unsigned long long*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  quant_stats_kernel<<<grid, kDiagThreads, 0, st>>>(a);         // an empty tensor still writes one zero record
  if (cudaGetLastError() != cudaSuccess) return US_ERR_CUDA;
  quant_stats_reduce_kernel<<<1, 128, 0, st>>>(a.partial, grid, nbins, sums, hist);
  return cudaGetLastError() == cudaSuccess ? US_OK : US_ERR_CUDA;
}
