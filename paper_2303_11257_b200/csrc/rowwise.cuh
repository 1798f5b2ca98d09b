// Helpers of the row-wise kernels (softmax, layer norm): one warp per row, eight consecutive
// elements per lane and step, warp-shuffle reductions.
#pragma once

#include "common.cuh"

namespace us {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Eight consecutive elements starting at column `col` of a row (fill beyond the row's end).
__device__ __forceinline__ void load8(const void* base, int dt, int64_t row_off, int col, int cols, bool vec, float fill,
                                      float (&v)[8]) {
  if (vec && (dt == US_E4M3 || dt == US_E5M2)) {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(static_cast<const char*>(base) + row_off + col));
    const uint32_t w[2] = {r.x, r.y};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = unpack_fp8x2((uint16_t)(w[j >> 1] >> (16 * (j & 1))), dt == US_E5M2);
      v[2 * j] = f.x; v[2 * j + 1] = f.y;
    }
  } else if (vec) {
    load_vec<8>(static_cast<const char*>(base) + (row_off + col) * dtype_size(dt), dt, v);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = (col + i < cols) ? load_one(base, dt, row_off + col + i) : fill;
  }
}
__device__ __forceinline__ void store8(void* base, int dt, int64_t row_off, int col, int cols, bool vec, const float (&v)[8]) {
  if (vec) {
    char* p = static_cast<char*>(base) + (row_off + col) * dtype_size(dt);
    if (dt == US_E4M3 || dt == US_E5M2) {
      const uint32_t lo = dt == US_E5M2 ? cvt_fp8x4<true>(v[0], v[1], v[2], v[3]) : cvt_fp8x4<false>(v[0], v[1], v[2], v[3]);
      const uint32_t hi = dt == US_E5M2 ? cvt_fp8x4<true>(v[4], v[5], v[6], v[7]) : cvt_fp8x4<false>(v[4], v[5], v[6], v[7]);
      *reinterpret_cast<uint2*>(p) = make_uint2(lo, hi);
    } else {
      store_vec<8>(p, dt, v);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (col + i < cols) store_one(base, dt, row_off + col + i, v[i]);
  }
}

// ---- rows of 16-bit elements kept packed in registers (one 128-bit load per lane and chunk of 8)
__device__ __forceinline__ void unpack16x8(const uint4& r, int dt, float (&v)[8]) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = dt == US_BF16 ? unpack_bf16x2(w[j]) : unpack_f16x2(w[j]);
    v[2 * j] = f.x; v[2 * j + 1] = f.y;
  }
}
template <int NCH>
__device__ __forceinline__ void load_row16(const void* base, int64_t row_off, int lane, int cols, uint4 (&d)[NCH]) {
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    const int col = (c * 32 + lane) * 8;
    d[c] = col < cols ? __ldg(reinterpret_cast<const uint4*>(static_cast<const char*>(base) + (row_off + col) * 2))
                      : make_uint4(0u, 0u, 0u, 0u);
  }
}
// The same for rows of FP8 codes: one 64-bit load per lane and chunk of 8.
__device__ __forceinline__ void unpack8x8(const uint2& r, int dt, float (&v)[8]) {
  const uint32_t w[2] = {r.x, r.y};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = unpack_fp8x2((uint16_t)(w[j >> 1] >> (16 * (j & 1))), dt == US_E5M2);
    v[2 * j] = f.x; v[2 * j + 1] = f.y;
  }
}
template <int NCH>
__device__ __forceinline__ void load_row8(const void* base, int64_t row_off, int lane, int cols, uint2 (&d)[NCH]) {
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    const int col = (c * 32 + lane) * 8;
    d[c] = col < cols ? __ldg(reinterpret_cast<const uint2*>(static_cast<const char*>(base) + row_off + col)) : make_uint2(0u, 0u);
  }
}
}  // namespace us
