// Warp-per-row helpers: a row of D floats (D % 4 == 0, D <= 2048) lives in the registers of one
// warp as float4 chunks, chunk index = lane + 32*j.
#pragma once
#include "common.cuh"

namespace et {

constexpr int ROW_MAX_VEC = 16;        // float4 chunks per lane -> D <= 2048
constexpr int ROW_MAX_D = ROW_MAX_VEC * 32 * 4;

template <typename T> __device__ __forceinline__ T to_out(float v);
template <> __device__ __forceinline__ float to_out<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 to_out<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <int NV>
__device__ __forceinline__ void load_row(const float* __restrict__ p, int D, int lane, float4 (&v)[NV]) {
  const int nvec = D >> 2;
  const float4* p4 = reinterpret_cast<const float4*>(p);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    v[j] = (i < nvec) ? __ldg(p4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

template <int NV>
__device__ __forceinline__ void store_row(float* __restrict__ p, int D, int lane, const float4 (&v)[NV]) {
  const int nvec = D >> 2;
  float4* p4 = reinterpret_cast<float4*>(p);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    if (i < nvec) p4[i] = v[j];
  }
}

template <int NV>
__device__ __forceinline__ void store_row(bf16* __restrict__ p, int D, int lane, const float4 (&v)[NV]) {
  const int nvec = D >> 2;
  uint2* p2 = reinterpret_cast<uint2*>(p);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    if (i < nvec) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(v[j].x, v[j].y);
      __nv_bfloat162 hi = __floats2bfloat162_rn(v[j].z, v[j].w);
      uint2 u;
      u.x = *reinterpret_cast<uint32_t*>(&lo);
      u.y = *reinterpret_cast<uint32_t*>(&hi);
      p2[i] = u;
    }
  }
}

// y = (x - mean) / sqrt(var + eps) * g + b, statistics in fp32 over the registers of the warp.
template <int NV>
__device__ __forceinline__ void layernorm_row_inplace(float4 (&v)[NV], int D, int lane,
                                                      const float* __restrict__ g, const float* __restrict__ b,
                                                      float eps) {
  const int nvec = D >> 2;
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < NV; ++j) s += (v[j].x + v[j].y) + (v[j].z + v[j].w);   // padding chunks are zero
  const float mean = warp_sum(s) / (float)D;
  float q = 0.f;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    if (lane + 32 * j < nvec) {
      const float a = v[j].x - mean, c = v[j].y - mean, d = v[j].z - mean, e = v[j].w - mean;
      q += (a * a + c * c) + (d * d + e * e);
    }
  }
  const float rstd = rsqrtf(warp_sum(q) / (float)D + eps);
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const float4* b4 = reinterpret_cast<const float4*>(b);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    if (i < nvec) {
      const float4 gg = __ldg(g4 + i), bb = __ldg(b4 + i);
      v[j].x = (v[j].x - mean) * rstd * gg.x + bb.x;
      v[j].y = (v[j].y - mean) * rstd * gg.y + bb.y;
      v[j].z = (v[j].z - mean) * rstd * gg.z + bb.z;
      v[j].w = (v[j].w - mean) * rstd * gg.w + bb.w;
    }
  }
}

// y = x / sqrt(mean(x^2) + eps) * g
template <int NV>
__device__ __forceinline__ void rmsnorm_row_inplace(float4 (&v)[NV], int D, int lane, const float* __restrict__ g,
                                                    float eps) {
  const int nvec = D >> 2;
  float q = 0.f;
#pragma unroll
  for (int j = 0; j < NV; ++j) q += (v[j].x * v[j].x + v[j].y * v[j].y) + (v[j].z * v[j].z + v[j].w * v[j].w);   // padding chunks are zero
  const float r = rsqrtf(warp_sum(q) / (float)D + eps);
  const float4* g4 = reinterpret_cast<const float4*>(g);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    if (i < nvec) {
      const float4 gg = __ldg(g4 + i);
      v[j].x = v[j].x * r * gg.x;
      v[j].y = v[j].y * r * gg.y;
      v[j].z = v[j].z * r * gg.z;
      v[j].w = v[j].w * r * gg.w;
    }
  }
}

__device__ __forceinline__ float gelu_f(float x, int tanh_approx) {
  if (tanh_approx) {
    const float c = 0.7978845608028654f;   // sqrt(2/pi)
    return 0.5f * x * (1.f + tanhf(c * (x + 0.044715f * x * x * x)));
  }
  return 0.5f * x * (1.f + erff(x * 0.7071067811865476f));
}

}  // namespace et
