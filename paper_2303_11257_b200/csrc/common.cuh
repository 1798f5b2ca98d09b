// Shared device helpers of libunitscale: storage-format conversion and the scaled
// GELU arithmetic.  Everything here computes in float32.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/unitscale.h"

namespace us {

__host__ __device__ inline int dtype_size(int dt) {
  return dt == US_F32 ? 4 : (dt == US_BF16 || dt == US_F16) ? 2 : 1;
}

// ---------------------------------------------------------------- FP8 (OCP) casts
// Two float32 -> two 8-bit codes, round-to-nearest-even, saturating to the largest
// finite value, NaN -> NaN.  Element `lo` lands in the low byte.
__device__ __forceinline__ uint16_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint16_t cvt_e5m2x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
template <bool E5>
__device__ __forceinline__ uint32_t cvt_fp8x4(float a, float b, float c, float d) {
  const uint32_t lo = E5 ? cvt_e5m2x2(a, b) : cvt_e4m3x2(a, b);
  const uint32_t hi = E5 ? cvt_e5m2x2(c, d) : cvt_e4m3x2(c, d);
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, 0x5410;" : "=r"(r) : "r"(lo), "r"(hi));   // low halves of lo and hi, one instruction
  return r;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float2 unpack_bf16x2(uint32_t u) {
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}
__device__ __forceinline__ float2 unpack_f16x2(uint32_t u) {
  return __half22float2(*reinterpret_cast<__half2*>(&u));
}

// Two FP8 codes (low byte first) widened to float; exact.
__device__ __forceinline__ float2 unpack_fp8x2(uint16_t u, bool e5) {
  uint32_t h;
  if (e5) asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h) : "h"(u));
  else asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"(u));
  return unpack_f16x2(h);
}

// ---------------------------------------------------------------- row fragments
// Load N consecutive elements (N a multiple of 16 / element size) starting at a
// 16-byte aligned address and widen them to float.
template <int N>
__device__ __forceinline__ void load_vec(const void* p, int dt, float (&v)[N]) {
  if (dt == US_F32) {
    const float4* q = reinterpret_cast<const float4*>(p);
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      float4 t = __ldg(q + i);
      v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
    }
  } else if (dt == US_BF16 || dt == US_F16) {
    const uint4* q = reinterpret_cast<const uint4*>(p);
#pragma unroll
    for (int i = 0; i < N / 8; ++i) {
      uint4 t = __ldg(q + i);
      uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float2 f = (dt == US_BF16) ? unpack_bf16x2(w[j]) : unpack_f16x2(w[j]);
        v[8 * i + 2 * j] = f.x; v[8 * i + 2 * j + 1] = f.y;
      }
    }
  } else {                                             // FP8 codes, 16 per 16-byte vector (N a multiple of 16)
    const uint4* q = reinterpret_cast<const uint4*>(p);
#pragma unroll
    for (int i = 0; i < N / 16; ++i) {
      uint4 t = __ldg(q + i);
      uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 lo = unpack_fp8x2((uint16_t)(w[j] & 0xffffu), dt == US_E5M2), hi = unpack_fp8x2((uint16_t)(w[j] >> 16), dt == US_E5M2);
        v[16 * i + 4 * j] = lo.x; v[16 * i + 4 * j + 1] = lo.y; v[16 * i + 4 * j + 2] = hi.x; v[16 * i + 4 * j + 3] = hi.y;
      }
    }
  }
}

// Round N floats (N a multiple of 16) to `dt` and store them at a 16-byte aligned address.
template <int N>
__device__ __forceinline__ void store_vec(void* p, int dt, const float (&v)[N]) {
  if (dt == US_F32) {
    float4* q = reinterpret_cast<float4*>(p);
#pragma unroll
    for (int i = 0; i < N / 4; ++i) q[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  } else if (dt == US_BF16 || dt == US_F16) {
    uint4* q = reinterpret_cast<uint4*>(p);
#pragma unroll
    for (int i = 0; i < N / 8; ++i) {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        w[j] = (dt == US_BF16) ? pack_bf16x2(v[8 * i + 2 * j], v[8 * i + 2 * j + 1])
                               : pack_f16x2(v[8 * i + 2 * j], v[8 * i + 2 * j + 1]);
      q[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  } else {
    uint4* q = reinterpret_cast<uint4*>(p);
#pragma unroll
    for (int i = 0; i < N / 16; ++i) {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float* s = &v[16 * i + 4 * j];
        w[j] = (dt == US_E5M2) ? cvt_fp8x4<true>(s[0], s[1], s[2], s[3]) : cvt_fp8x4<false>(s[0], s[1], s[2], s[3]);
      }
      q[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

__device__ __forceinline__ float load_one(const void* base, int dt, int64_t idx) {
  if (dt == US_F32) return reinterpret_cast<const float*>(base)[idx];
  if (dt == US_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
  if (dt == US_F16) return __half2float(reinterpret_cast<const __half*>(base)[idx]);
  return unpack_fp8x2(reinterpret_cast<const uint8_t*>(base)[idx], dt == US_E5M2).x;
}

__device__ __forceinline__ void store_one(void* base, int dt, int64_t idx, float v) {
  switch (dt) {
    case US_F32: reinterpret_cast<float*>(base)[idx] = v; break;
    case US_BF16: reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(v); break;
    case US_F16: reinterpret_cast<__half*>(base)[idx] = __float2half_rn(v); break;
    case US_E4M3: reinterpret_cast<uint8_t*>(base)[idx] = (uint8_t)(cvt_e4m3x2(v, 0.f) & 0xff); break;
    default: reinterpret_cast<uint8_t*>(base)[idx] = (uint8_t)(cvt_e5m2x2(v, 0.f) & 0xff); break;
  }
}

// ---------------------------------------------------------------- scaled GELU
// Lower normal tail q(a) = Phi(-a), a = |z|, as 2^R(t) with t = min(a / 7.5, 1) and R a degree-6
// polynomial fitted to log2 Phi(-7.5 t) on [0, 1] (fit_normal_tail.py regenerates the coefficients):
// one saturating multiply, six FMAs and one ex2; |q error| <= 2.7e-7, |a q error| <= 1.5e-7 in
// float32.  Beyond a = 7.5 the tail is below 4e-14 and t stays at 1.  Phi(z) = z >= 0 ? 1 - q : q,
// and gelu(z) = z Phi(z) = max(z, 0) - |z| q(|z|).
constexpr float kTailRange = 7.5f;
constexpr float kTailC0 = -9.999993443e-01f, kTailC1 = -8.633527756e+00f, kTailC2 = -2.581697273e+01f,
                kTailC3 = -2.242405128e+01f, kTailC4 = 2.505270767e+01f, kTailC5 = -1.710954857e+01f,
                kTailC6 = 4.934150219e+00f;

__device__ __forceinline__ float ex2_approx(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
// min(|x| k, 1) for k > 0 in one instruction of the FMA pipe (the clamp is the multiply's saturation).
__device__ __forceinline__ float sat_mul_abs(float x, float k) {
  float r;
  asm("mul.rn.sat.f32 %0, %1, %2;" : "=f"(r) : "f"(fabsf(x)), "f"(k));
  return r;
}
__device__ __forceinline__ float normal_tail(float z) {
  const float t = sat_mul_abs(z, 1.0f / kTailRange);
  float r = kTailC6;
  r = fmaf(r, t, kTailC5);
  r = fmaf(r, t, kTailC4);
  r = fmaf(r, t, kTailC3);
  r = fmaf(r, t, kTailC2);
  r = fmaf(r, t, kTailC1);
  r = fmaf(r, t, kTailC0);
  return ex2_approx(r);
}

// out_scale * gelu(in_scale * h), gelu(x) = x Phi(x)
__device__ __forceinline__ float gelu_scaled(float h, float in_scale, float out_scale) {
  const float z = in_scale * h;
  const float q = normal_tail(z);
  const float oz = out_scale * z;
  return fmaf(-fabsf(oz), q, fmaxf(oz, 0.f));
}

// out_scale * in_scale * gelu'(in_scale * h) * g, gelu'(x) = Phi(x) + x phi(x)
__device__ __forceinline__ float gelu_grad_scaled(float h, float g, float in_scale, float out_scale) {
  const float z = in_scale * h;
  const float q = normal_tail(z);
  const float Phi = z >= 0.f ? 1.0f - q : q;
  const float e = ex2_approx((-0.72134752044448170f * z) * z);   // exp(-z^2 / 2) = 2^(-z^2 log2(e) / 2)
  const float d = fmaf(z * 0.39894228040143268f, e, Phi);
  return (out_scale * in_scale) * d * g;
}

// relu, tanh and sigmoid of the table "Activations" and their derivatives.  exp through ex2.approx and a
// correctly rounded division: absolute error about 2e-7 for the bounded functions.
__device__ __forceinline__ float sigmoid_f(float z) {
  const float e = ex2_approx(-1.4426950408889634f * fabsf(z));     // e^-|z| in (0, 1]
  const float r = __fdiv_rn(1.0f, 1.0f + e);
  return z >= 0.f ? r : e * r;
}
__device__ __forceinline__ float act_value(int fn, float z) {
  if (fn == US_FN_RELU) return fmaxf(z, 0.f);
  if (fn == US_FN_TANH) return 2.0f * sigmoid_f(2.0f * z) - 1.0f;
  if (fn == US_FN_SIGMOID) return sigmoid_f(z);
  return 0.f;   // gelu is dispatched before this point
}
__device__ __forceinline__ float act_slope(int fn, float z) {
  if (fn == US_FN_RELU) return z > 0.f ? 1.0f : 0.f;
  if (fn == US_FN_TANH) { const float s = sigmoid_f(2.0f * z), m = sigmoid_f(-2.0f * z); return 4.0f * s * m; }   // 1 - tanh^2
  if (fn == US_FN_SIGMOID) return sigmoid_f(z) * sigmoid_f(-z);
  return 0.f;
}

// out_scale * f(in_scale * h) and out_scale * in_scale * f'(in_scale * h) * g for any us_fn.
__device__ __forceinline__ float act_scaled(int fn, float h, float in_scale, float out_scale) {
  return fn == US_FN_GELU ? gelu_scaled(h, in_scale, out_scale) : out_scale * act_value(fn, in_scale * h);
}
__device__ __forceinline__ float act_grad_scaled(int fn, float h, float g, float in_scale, float out_scale) {
  return fn == US_FN_GELU ? gelu_grad_scaled(h, g, in_scale, out_scale) : (out_scale * in_scale) * act_slope(fn, in_scale * h) * g;
}

// ---------------------------------------------------------------- two floats per instruction
// sm_100 executes add / mul / fma on pairs of float32 held in a 64-bit register (same IEEE
// rounding per lane as the scalar forms); the GEMM epilogues use it to halve the number of
// issued arithmetic instructions.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 splat2(float x) { return pack2(x, x); }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// q for two arguments given t = min(|z| / 7.5, 1) of each (see normal_tail).
__device__ __forceinline__ void normal_tail2(float t0, float t1, float& q0, float& q1) {
  const f32x2 t = pack2(t0, t1);
  f32x2 r = splat2(kTailC6);
  r = fma2(r, t, splat2(kTailC5));
  r = fma2(r, t, splat2(kTailC4));
  r = fma2(r, t, splat2(kTailC3));
  r = fma2(r, t, splat2(kTailC2));
  r = fma2(r, t, splat2(kTailC1));
  r = fma2(r, t, splat2(kTailC0));
  float r0, r1;
  unpack2(r, r0, r1);
  q0 = ex2_approx(r0);
  q1 = ex2_approx(r1);
}

// out_scale * gelu(in_scale * x) for two values.  x holds the pre-activations, k = in_scale / 7.5,
// oi = out_scale * in_scale.  The arithmetic is laid out for the instruction mix of the GEMM
// epilogue: comparisons and min / max issue at half rate and do not overlap the packed FMAs there,
// so the clamp is a saturating multiply and, with CANCEL, max(.) is replaced by
//     gelu = h + |h| (1 - 2 q),  h = x / 2,
// which for negative x subtracts nearly equal numbers: the absolute error stays below
// 2^-24 |out_scale x|, harmless in front of a rounding to 8 or 16 bits but not for a float32 output,
// which takes the form max(x, 0) - |x| q instead (CANCEL = false).
template <bool CANCEL>
__device__ __forceinline__ void gelu_scaled2(f32x2 x, float k, float oi, float& y0, float& y1) {
  float x0, x1, q0, q1;
  unpack2(x, x0, x1);
  normal_tail2(sat_mul_abs(x0, k), sat_mul_abs(x1, k), q0, q1);
  if (CANCEL) {
    float h0, h1, w0, w1;
    unpack2(mul2(splat2(0.5f * oi), x), h0, h1);
    unpack2(fma2(pack2(q0, q1), splat2(-2.0f), splat2(1.0f)), w0, w1);
    y0 = fmaf(fabsf(h0), w0, h0);
    y1 = fmaf(fabsf(h1), w1, h1);
  } else {
    float o0, o1;
    unpack2(mul2(splat2(oi), x), o0, o1);
    y0 = fmaf(-fabsf(o0), q0, fmaxf(o0, 0.f));
    y1 = fmaf(-fabsf(o1), q1, fmaxf(o1, 0.f));
  }
}

// gelu_grad_scaled for two values: h = stored pre-activations, g = incoming gradients,
// in2 = splat(in_scale), os2 = splat(out_scale * in_scale).
__device__ __forceinline__ f32x2 gelu_grad_scaled2(f32x2 h, f32x2 g, f32x2 in2, f32x2 os2) {
  const f32x2 z = mul2(in2, h);
  float q0, q1, z0, z1;
  unpack2(z, z0, z1);
  normal_tail2(sat_mul_abs(z0, 1.0f / kTailRange), sat_mul_abs(z1, 1.0f / kTailRange), q0, q1);
  const f32x2 Phi = pack2(z0 >= 0.f ? 1.0f - q0 : q0, z1 >= 0.f ? 1.0f - q1 : q1);
  float e0, e1;
  unpack2(mul2(mul2(splat2(-0.72134752044448170f), z), z), e0, e1);
  const f32x2 e = pack2(ex2_approx(e0), ex2_approx(e1));
  const f32x2 d = fma2(mul2(z, splat2(0.39894228040143268f)), e, Phi);
  return mul2(mul2(os2, d), g);
}

}  // namespace us
