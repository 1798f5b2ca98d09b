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
  uint32_t lo = E5 ? cvt_e5m2x2(a, b) : cvt_e4m3x2(a, b);
  uint32_t hi = E5 ? cvt_e5m2x2(c, d) : cvt_e4m3x2(c, d);
  return lo | (hi << 16);
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
  } else {
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
  return __half2float(reinterpret_cast<const __half*>(base)[idx]);
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
// Lower normal tail q(a) = Phi(-a), a = |z|, as 2^R(a) with R a degree-6 polynomial fitted to
// log2 Phi(-a) on [0, 7.5] (fit_normal_tail.py regenerates the coefficients): one ex2 and six FMAs,
// |q error| <= 2.7e-7, |a q error| <= 1.5e-7 in float32.  Beyond 7.5 the tail is below 4e-14 and a
// is clamped.  Phi(z) = z >= 0 ? 1 - q : q, and gelu(z) = z Phi(z) = max(z, 0) - |z| q(|z|).
__device__ __forceinline__ float ex2_approx(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float normal_tail(float z) {
  const float a = fminf(fabsf(z), 7.5f);
  float r = 2.772329208e-05f;
  r = fmaf(r, a, -7.209949545e-04f);
  r = fmaf(r, a, 7.917892188e-03f);
  r = fmaf(r, a, -5.315330625e-02f);
  r = fmaf(r, a, -4.589684010e-01f);
  r = fmaf(r, a, -1.151137114e+00f);
  r = fmaf(r, a, -9.999993443e-01f);
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

}  // namespace us
