// Host-only entry points of libunitscale: scale-factor helpers, status strings, device queries.
#include <math.h>

#include "host.h"

namespace us {
namespace host {
int sm_count() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return -1;
    cached[dev] = n;
  }
  return cached[dev];
}

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;     // idempotent: concurrent first calls store the same pointer
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}
}  // namespace host
}  // namespace us

// 1 / std(gelu(z)) and 1 / rms(gelu'(z)) for z ~ N(0,1), gelu(x) = x Phi(x): the values the
// table of unit scaling factors prints as 1.701 and 1.481, here to double precision.
static const double kGeluAlpha = 1.7009262433633;
static const double kGeluBeta = 1.4811144127083;

extern "C" us_status us_scales_linear(int64_t b, int64_t m, int64_t n, int constrained, float* alpha,
                                      float* beta_x, float* beta_w) {
  if (b < 1 || m < 1 || n < 1 || !alpha || !beta_x || !beta_w) return US_ERR_INVALID_ARG;
  double a = 1.0 / sqrt((double)m), bx = 1.0 / sqrt((double)n), bw = 1.0 / sqrt((double)b);
  if (constrained) a = bx = sqrt(a * bx);  // geometric mean of the constrained pair
  *alpha = (float)a;
  *beta_x = (float)bx;
  *beta_w = (float)bw;
  return US_OK;
}

extern "C" us_status us_scales_gelu(int constrained, float* alpha, float* beta) {
  if (!alpha || !beta) return US_ERR_INVALID_ARG;
  double a = kGeluAlpha, b = kGeluBeta;
  if (constrained) a = b = sqrt(a * b);
  *alpha = (float)a;
  *beta = (float)b;
  return US_OK;
}

extern "C" us_status us_scales_activation(us_fn fn, int constrained, float* alpha, float* beta) {
  if (!alpha || !beta) return US_ERR_INVALID_ARG;
  // 1 / std f(Z) and 1 / rms f'(Z) for Z ~ N(0, 1): relu in closed form (sqrt(2 / (1 - 1/pi)), sqrt 2),
  // the others by numerical integration to the digits kept here (the table prints three of them).
  double a, b;
  switch (fn) {
    case US_FN_GELU: a = kGeluAlpha; b = kGeluBeta; break;
    case US_FN_RELU: a = 1.7128585504496627; b = 1.4142135623730951; break;
    case US_FN_TANH: a = 1.5925374197228314; b = 1.4674135916307951; break;
    case US_FN_SIGMOID: a = 4.8013133720399622; b = 4.7226460859379743; break;
    default: return US_ERR_INVALID_ARG;
  }
  if (constrained) a = b = sqrt(a * b);
  *alpha = (float)a;
  *beta = (float)b;
  return US_OK;
}

extern "C" us_status us_scales_residual(float tau, float* skip_coef, float* branch_coef) {
  if (!skip_coef || !branch_coef || !(tau >= 0.f && tau <= 1.f)) return US_ERR_INVALID_ARG;
  *skip_coef = (float)sqrt(1.0 - (double)tau);
  *branch_coef = (float)sqrt((double)tau);
  return US_OK;
}

extern "C" us_status us_scales_attention(int64_t s, int64_t d_head, int constrained, float* alpha_scores, float* beta_scores,
                                         float* softmax_scale, float* alpha_context, float* beta_p, float* beta_v) {
  if (s < 1 || d_head < 1 || !alpha_scores || !beta_scores || !softmax_scale || !alpha_context || !beta_p || !beta_v)
    return US_ERR_INVALID_ARG;
  // scores Q K^T: 1 / sqrt(d_head) in both passes; context P V is an ordinary matmul with fan_in = batch = s, fan_out = d_head
  const double a_s = 1.0 / sqrt((double)d_head);
  double a_c = 1.0 / sqrt((double)s), b_p = 1.0 / sqrt((double)d_head);
  if (constrained) a_c = b_p = sqrt(a_c * b_p);
  *alpha_scores = (float)a_s;
  *beta_scores = (float)a_s;
  *softmax_scale = (float)s;
  *alpha_context = (float)a_c;
  *beta_p = (float)b_p;
  *beta_v = (float)(1.0 / sqrt((double)s));
  return US_OK;
}

extern "C" const char* us_status_string(us_status s) {
  switch (s) {
    case US_OK: return "ok";
    case US_ERR_INVALID_ARG: return "invalid argument";
    case US_ERR_UNSUPPORTED: return "unsupported dtype combination";
    case US_ERR_ALIGNMENT: return "pointer or row pitch not 16-byte aligned";
    case US_ERR_WORKSPACE: return "workspace missing or too small";
    case US_ERR_CUDA: return "CUDA call failed";
    case US_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" int us_version(void) { return 100; }
