// 16-lane row slices: a key/value row of D elements is spread over 16 adjacent lanes,
// EPL = D/16 contiguous elements per lane, fetched with the widest load that fits.
#pragma once
#include "common.cuh"

namespace tca {

template <typename T, int EPL>
struct RowF;  // raw slice readable as float

template <>
struct RowF<__nv_bfloat16, 8> {
  uint4 raw;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { raw = __ldcs(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void load_cached(const __nv_bfloat16* p) { raw = *reinterpret_cast<const uint4*>(p); }
  __device__ __forceinline__ void zero() { raw = make_uint4(0, 0, 0, 0); }
  __device__ __forceinline__ float get(int e) const {
    uint32_t w = (e < 2) ? raw.x : (e < 4) ? raw.y : (e < 6) ? raw.z : raw.w;
    return (e & 1) ? bf16_hi(w) : bf16_lo(w);
  }
};
template <>
struct RowF<__nv_bfloat16, 4> {
  uint2 raw;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { raw = __ldcs(reinterpret_cast<const uint2*>(p)); }
  __device__ __forceinline__ void load_cached(const __nv_bfloat16* p) { raw = *reinterpret_cast<const uint2*>(p); }
  __device__ __forceinline__ void zero() { raw = make_uint2(0, 0); }
  __device__ __forceinline__ float get(int e) const {
    uint32_t w = (e < 2) ? raw.x : raw.y;
    return (e & 1) ? bf16_hi(w) : bf16_lo(w);
  }
};
template <>
struct RowF<float, 4> {
  float4 raw;
  __device__ __forceinline__ void load(const float* p) { raw = __ldcs(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void load_cached(const float* p) { raw = *reinterpret_cast<const float4*>(p); }
  __device__ __forceinline__ void zero() { raw = make_float4(0, 0, 0, 0); }
  __device__ __forceinline__ float get(int e) const { return e == 0 ? raw.x : e == 1 ? raw.y : e == 2 ? raw.z : raw.w; }
};
template <>
struct RowF<float, 8> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = __ldcs(reinterpret_cast<const float4*>(p));
    b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  }
  __device__ __forceinline__ void load_cached(const float* p) {
    a = *reinterpret_cast<const float4*>(p);
    b = *(reinterpret_cast<const float4*>(p) + 1);
  }
  __device__ __forceinline__ void zero() { a = b = make_float4(0, 0, 0, 0); }
  __device__ __forceinline__ float get(int e) const {
    const float4& v = e < 4 ? a : b;
    const int i = e & 3;
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
  }
};

__device__ __forceinline__ float elt_to_float(float x) { return x; }
__device__ __forceinline__ float elt_to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_elt(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_elt(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Transposing butterfly over a 16-lane group (float): on entry every lane holds 16
// partial sums, on exit lane i holds the group total of value index i.
__device__ __forceinline__ float butterfly16f(float (&v)[16], int lane16) {
  {
    const bool up = lane16 & 8;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float send = up ? v[i] : v[i + 8];
      float keep = up ? v[i + 8] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
  }
  {
    const bool up = lane16 & 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float send = up ? v[i] : v[i + 4];
      float keep = up ? v[i + 4] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
  }
  {
    const bool up = lane16 & 2;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      float send = up ? v[i] : v[i + 2];
      float keep = up ? v[i + 2] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
  }
  {
    const bool up = lane16 & 1;
    float send = up ? v[0] : v[1];
    float keep = up ? v[1] : v[0];
    v[0] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
  }
  return v[0];
}

}  // namespace tca
