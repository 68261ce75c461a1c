// Row-wise and elementwise steps of the language model's prefill: RMSNorm, rotary position embedding,
// SwiGLU gating, embedding lookup, fp32 -> bf16 cast, argmax of the logits.  All HBM-bound.
#include "common.cuh"
#include "rowops.cuh"

namespace et {

namespace {

// ---------------------------------------------------------------------------------------------
// RMSNorm: one warp per row, the row in registers (one read of x), fp32 statistics.
// ---------------------------------------------------------------------------------------------
template <int NV>
__global__ void __launch_bounds__(128)
rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ g, float eps, bf16* __restrict__ y, int rows, int D) {
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int nvec = D >> 2;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  for (int row = blockIdx.x * warps_per_block + (threadIdx.x >> 5); row < rows; row += gridDim.x * warps_per_block) {
    float4 v[NV];
    load_row<NV>(x + (size_t)row * D, D, lane, v);
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) q += (v[j].x * v[j].x + v[j].y * v[j].y) + (v[j].z * v[j].z + v[j].w * v[j].w);   // padding chunks are zero
    const float r = rsqrtf(warp_sum(q) / (float)D + eps);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const int i = lane + 32 * j;
      if (i < nvec) {
        const float4 gg = __ldg(g4 + i);
        v[j].x = v[j].x * r * gg.x; v[j].y = v[j].y * r * gg.y; v[j].z = v[j].z * r * gg.z; v[j].w = v[j].w * r * gg.w;
      }
    }
    store_row<NV>(y + (size_t)row * D, D, lane, v);
  }
}

// ---------------------------------------------------------------------------------------------
// Rotary embedding, rotate-half form: element i < dh/2 of a head pairs with element i + dh/2; the pair
// is turned by pos * theta^(-2i/dh).  The (cos, sin) of every (position, i) are tabulated once per model
// (rope_table_kernel: the angle is reduced to a fraction of a turn in double precision, since positions reach
// 10^4 and more, where a single-precision product loses that fraction; inv_turns[i] = theta^(-2i/dh) / (2 pi)
// comes from the host in double precision).  The rotation itself then only streams: one thread handles 8
// consecutive i of one (row, head), two 16-byte loads and stores plus 64 bytes of table from L2.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rope_table_kernel(float2* __restrict__ table, int L, int half, const double* __restrict__ inv_turns) {
  const long long total = (long long)L * half;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx % half);
    const long long pos = idx / half;
    const double turns = (double)pos * inv_turns[i];                          // angle / 2 pi
    const float frac = (float)(turns - floor(turns));
    float sn, cs;
    sincospif(2.f * frac, &sn, &cs);
    table[idx] = make_float2(cs, sn);
  }
}

__global__ void __launch_bounds__(256)
rope_kernel(bf16* __restrict__ qkv, int rows, int L, int rot_heads, int row_elems, int dh, const float2* __restrict__ table) {
  const int half = dh >> 1, chunks = half >> 3;
  const long long total = (long long)rows * rot_heads * chunks;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % chunks);
    const int h = (int)((idx / chunks) % rot_heads);
    const int row = (int)(idx / ((long long)chunks * rot_heads));
    const int pos = row % L;
    bf16* p = qkv + (size_t)row * row_elems + (size_t)h * dh + c * 8;
    uint4 a4 = *reinterpret_cast<const uint4*>(p), b4 = *reinterpret_cast<const uint4*>(p + half);
    const float4* t4 = reinterpret_cast<const float4*>(table + (size_t)pos * half + c * 8);     // (cos, sin) x 2 per float4
    __nv_bfloat162* a2 = reinterpret_cast<__nv_bfloat162*>(&a4);
    __nv_bfloat162* b2 = reinterpret_cast<__nv_bfloat162*>(&b4);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 a = __bfloat1622float2(a2[k]), b = __bfloat1622float2(b2[k]);
      const float4 t = __ldg(t4 + k);                       // cos0, sin0, cos1, sin1
      a2[k] = __floats2bfloat162_rn(a.x * t.x - b.x * t.y, a.y * t.z - b.y * t.w);
      b2[k] = __floats2bfloat162_rn(b.x * t.x + a.x * t.y, b.y * t.z + a.y * t.w);
    }
    *reinterpret_cast<uint4*>(p) = a4;
    *reinterpret_cast<uint4*>(p + half) = b4;
  }
}

// ---------------------------------------------------------------------------------------------
// SwiGLU: h = silu(gate) * up from one packed row [gate (M) | up (M)]; 8 elements per thread.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
swiglu_kernel(const bf16* __restrict__ gu, bf16* __restrict__ h, int rows, int M) {
  const int chunks = M >> 3;
  const long long total = (long long)rows * chunks;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % chunks);
    const long long row = idx / chunks;
    const bf16* p = gu + (size_t)row * 2 * M + c * 8;
    uint4 g4 = __ldg(reinterpret_cast<const uint4*>(p)), u4 = __ldg(reinterpret_cast<const uint4*>(p + M));
    const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&g4);
    const __nv_bfloat162* u2 = reinterpret_cast<const __nv_bfloat162*>(&u4);
    uint4 o4;
    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o4);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 g = __bfloat1622float2(g2[k]), u = __bfloat1622float2(u2[k]);
      o2[k] = __floats2bfloat162_rn(g.x / (1.f + __expf(-g.x)) * u.x, g.y / (1.f + __expf(-g.y)) * u.y);
    }
    *reinterpret_cast<uint4*>(h + (size_t)row * M + c * 8) = o4;
  }
}

__global__ void __launch_bounds__(256)
embed_rows_kernel(const bf16* __restrict__ table, const int* __restrict__ ids, float* __restrict__ x, int rows, int D, int vocab) {
  const int chunks = D >> 3;
  const long long total = (long long)rows * chunks;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % chunks);
    const long long row = idx / chunks;
    const int id = min(max(ids[row], 0), vocab - 1);
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(table + (size_t)id * D + c * 8));
    const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&v);
    float4* o = reinterpret_cast<float4*>(x + (size_t)row * D + c * 8);
    const float2 a = __bfloat1622float2(v2[0]), b = __bfloat1622float2(v2[1]), d = __bfloat1622float2(v2[2]), e = __bfloat1622float2(v2[3]);
    o[0] = make_float4(a.x, a.y, b.x, b.y);
    o[1] = make_float4(d.x, d.y, e.x, e.y);
  }
}

// dst[r][0..w) = src[r][0..w) for row pitches given in 16-byte units (a column block of a wider matrix)
__global__ void __launch_bounds__(256)
copy_columns_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int rows, int w16, int src_pitch16, int dst_pitch16) {
  const long long total = (long long)rows * w16;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % w16);
    const long long r = idx / w16;
    dst[r * dst_pitch16 + c] = __ldg(src + r * src_pitch16 + c);
  }
}

__global__ void __launch_bounds__(256)
cast_bf16_kernel(const float* __restrict__ x, bf16* __restrict__ y, size_t count) {
  const size_t n4 = count >> 2;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(x) + i);
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(y)[i] = u;
  }
  if (blockIdx.x == 0 && threadIdx.x < (count & 3)) y[(n4 << 2) + threadIdx.x] = __float2bfloat16_rn(x[(n4 << 2) + threadIdx.x]);
}

// One block: every thread scans a strided part, then a block reduction on (value, index) keeps the
// larger value and, between equal values, the smaller index.
__global__ void __launch_bounds__(1024)
argmax_kernel(const float* __restrict__ x, int n, int* __restrict__ out) {
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const float v = x[i];
    if (v > best || (v == best && i < bi)) { best = v; bi = i; }
  }
  __shared__ float sv[32];
  __shared__ int si[32];
  auto better = [](float v, int i, float w, int k) { return w > v || (w == v && k < i); };
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float w = __shfl_xor_sync(0xffffffffu, best, o);
    const int k = __shfl_xor_sync(0xffffffffu, bi, o);
    if (better(best, bi, w, k)) { best = w; bi = k; }
  }
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int nw = blockDim.x >> 5;
    best = threadIdx.x < nw ? sv[threadIdx.x] : -INFINITY;
    bi = threadIdx.x < nw ? si[threadIdx.x] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float w = __shfl_xor_sync(0xffffffffu, best, o);
      const int k = __shfl_xor_sync(0xffffffffu, bi, o);
      if (better(best, bi, w, k)) { best = w; bi = k; }
    }
    if (threadIdx.x == 0) *out = bi == 0x7fffffff ? 0 : bi;
  }
}

int grid_for(long long work_items, int threads) {
  const long long want = (work_items + threads - 1) / threads;
  return (int)std::max<long long>(1, std::min<long long>(want, 148 * 16));
}

}  // namespace

void launch_rmsnorm(const float* x, const float* g, float eps, bf16* y, int rows, int D, cudaStream_t s) {
  if (rows <= 0) return;
  ET_COUNT_LAUNCH();
  // 4 warps per block: a 3584-wide row takes 112 registers per thread, and three small blocks fit an SM where
  // one of 8 warps would
  const int threads = 128, wpb = threads / 32;
  const int blocks = std::min(cdiv(rows, wpb), 148 * 12);
  const int need = cdiv(D / 4, 32);
#define ET_RMS(NV) rmsnorm_kernel<NV><<<blocks, threads, 0, s>>>(x, g, eps, y, rows, D)
  if (need <= 2) ET_RMS(2);
  else if (need <= 4) ET_RMS(4);
  else if (need <= 8) ET_RMS(8);
  else if (need <= 16) ET_RMS(16);
  else if (need <= 28) ET_RMS(28);
  else ET_RMS(32);            // D <= 4096 (checked where the model is created)
#undef ET_RMS
}

void launch_rope_table(float2* table, int L, int dh, const double* inv_turns, cudaStream_t s) {
  if (L <= 0) return;
  ET_COUNT_LAUNCH();
  rope_table_kernel<<<grid_for((long long)L * (dh / 2), 256), 256, 0, s>>>(table, L, dh / 2, inv_turns);
}

void launch_rope(bf16* qkv, int rows, int L, int heads, int kv_heads, int dh, const float2* table, cudaStream_t s) {
  if (rows <= 0) return;
  ET_COUNT_LAUNCH();
  const int rot = heads + kv_heads;
  const long long items = (long long)rows * rot * (dh / 16);
  rope_kernel<<<grid_for(items, 256), 256, 0, s>>>(qkv, rows, L, rot, (heads + 2 * kv_heads) * dh, dh, table);
}

void launch_swiglu(const bf16* gu, bf16* h, int rows, int M, cudaStream_t s) {
  if (rows <= 0) return;
  ET_COUNT_LAUNCH();
  swiglu_kernel<<<grid_for((long long)rows * (M / 8), 256), 256, 0, s>>>(gu, h, rows, M);
}

void launch_embed_rows(const bf16* table, const int* ids, float* x, int rows, int D, int vocab, cudaStream_t s) {
  if (rows <= 0) return;
  ET_COUNT_LAUNCH();
  embed_rows_kernel<<<grid_for((long long)rows * (D / 8), 256), 256, 0, s>>>(table, ids, x, rows, D, vocab);
}

void launch_cast_bf16(const float* x, bf16* y, size_t count, cudaStream_t s) {
  if (count == 0) return;
  ET_COUNT_LAUNCH();
  cast_bf16_kernel<<<grid_for((long long)(count / 4 + 1), 256), 256, 0, s>>>(x, y, count);
}

void launch_copy_columns(const bf16* src, bf16* dst, int rows, int width, int src_pitch, int dst_pitch, cudaStream_t s) {
  if (rows <= 0 || width <= 0) return;
  ET_COUNT_LAUNCH();
  copy_columns_kernel<<<grid_for((long long)rows * (width / 8), 256), 256, 0, s>>>(
      reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), rows, width / 8, src_pitch / 8, dst_pitch / 8);
}

void launch_argmax(const float* x, int n, int* out, cudaStream_t s) {
  if (n <= 0) return;
  ET_COUNT_LAUNCH();
  argmax_kernel<<<1, 1024, 0, s>>>(x, n, out);
}

}  // namespace et
