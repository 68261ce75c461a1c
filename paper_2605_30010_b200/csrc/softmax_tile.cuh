// Register-level pieces of the online softmax that the tcgen05 attention kernels share: one thread owns one
// query row and holds a chunk of 32 logits of the current key tile in registers.
#pragma once

#include "tcgen05.cuh"

namespace et {
namespace tc {

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// maximum of the valid logits (columns lo <= c < nk of the tile) of one chunk of W = 32 or 16 columns whose first
// column is c0
template <bool MASK, int W>
__device__ __forceinline__ float row_max(const uint32_t (&r)[W], int c0, int nk, int lo = 0) {
  float a[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int i = 0; i < W; ++i)
    if (!MASK || (c0 + i < nk && c0 + i >= lo)) a[i & 3] = fmaxf(a[i & 3], __uint_as_float(r[i]));
  return fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
}

// The exponential phase of the softmax is bound by instruction issue: packed fp32 pairs (fma2 / add2) halve the FMA
// and ADD count, worth 4 % of the kernel; a three-input maximum and a cubic exp2 on the FMA pipe were measured slower.
template <bool MASK, int W>
__device__ __forceinline__ void probs(const uint32_t (&r)[W], int c0, int nk, float scale2, float m, float (&ls)[4],
                                      uint32_t p_addr, int lo = 0) {
  static_assert(W == 32 || W == 16, "chunk width");
  uint32_t pk[W / 2];
  const float neg_m = -m;
#pragma unroll
  for (int i = 0; i < W; i += 2) {
    float x0, x1;
    fma2(x0, x1, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), scale2, scale2, neg_m, neg_m);
    float p0 = ex2(x0), p1 = ex2(x1);
    if (MASK) {
      if (c0 + i >= nk || c0 + i < lo) p0 = 0.f;
      if (c0 + i + 1 >= nk || c0 + i + 1 < lo) p1 = 0.f;
    }
    const int a = ((i >> 1) & 1) * 2;                // two pairs of partial sums, alternating
    add2(ls[a], ls[a + 1], ls[a], ls[a + 1], p0, p1);
    pk[i >> 1] = pack_bf16(p0, p1);
  }
  if constexpr (W == 32) tmem_st16(p_addr, pk);
  else tmem_st8(p_addr, pk);
}

// P = 0 for a chunk of W keys none of which the row may see
template <int W>
__device__ __forceinline__ void zero_probs(const uint32_t (&)[W], uint32_t p_addr) {
  static_assert(W == 32 || W == 16, "chunk width");
  uint32_t z[W / 2];
#pragma unroll
  for (int i = 0; i < W / 2; ++i) z[i] = 0u;
  if constexpr (W == 32) tmem_st16(p_addr, z);
  else tmem_st8(p_addr, z);
}

}  // namespace tc
}  // namespace et
