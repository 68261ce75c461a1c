// Patch extraction and LayerNorm kernels (HBM/L2-bound helpers around the dense layers).
#include "common.cuh"
#include "rowops.cuh"

namespace et {

// ---------------------------------------------------------------------------------------------
// im2col: one thread per (token, channel, dy) copies the p contiguous pixels of one patch row.
// Patch feature index = c*p*p + dy*p + dx, i.e. the flattening of a [D][3][p][p] convolution
// weight; columns >= 3*p*p are zero (pad so that the row pitch is a multiple of 16 bytes).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void store_pair(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void store_pair(bf16* p, float a, float b) { *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b); }

// `tp` input frames form one encoder frame (temporal patch): feature index = ((c*tp + t)*p + dy)*p + dx, the
// flattening of a [D][3][tp][p][p] convolution weight.  With `int2raster` the tokens of an encoder frame are written
// in the encoder's internal order (token l of the output sits at raster position int2raster[l] of the patch grid).
template <typename T>
__global__ void im2col_kernel(const float* __restrict__ frames, T* __restrict__ patches, int T_frames, int image,
                              int patch, int grid, int k_pad, int tp, const int* __restrict__ int2raster,
                              const int* __restrict__ n_frames_dev) {
  const int n_frames = n_frames_dev ? min(*n_frames_dev, T_frames) : T_frames;      // encoder frames
  const int L = grid * grid;
  const int rows_per_tok = 3 * tp * patch + 1;  // 3*tp*p pixel rows + one job that writes the zero pad
  const long long total = (long long)n_frames * L * rows_per_tok;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int job = (int)(idx % rows_per_tok);
    const long long tok = idx / rows_per_tok;
    T* dst_row = patches + tok * k_pad;
    if (job == 3 * tp * patch) {
      for (int c = 3 * tp * patch * patch; c < k_pad; ++c) dst_row[c] = to_out<T>(0.f);
      continue;
    }
    const int ct = job / patch, dy = job % patch;       // ct = c*tp + t
    const int c = ct / tp, t = ct % tp;
    const int f = (int)(tok / L);
    int l = (int)(tok % L);
    if (int2raster) l = int2raster[l];
    const int gy = l / grid, gx = l % grid;
    const float* src = frames + ((((long long)f * tp + t) * 3 + c) * image + (gy * patch + dy)) * image + gx * patch;
    T* dst = dst_row + (ct * patch + dy) * patch;
    if ((patch & 1) == 0 && (image & 1) == 0 && (k_pad & 1) == 0 && (reinterpret_cast<size_t>(frames) & 7) == 0) {
      // pixel pairs: the patch row starts at an even pixel of an even-width image and at an even patch column
      const float2* s2 = reinterpret_cast<const float2*>(src);
      for (int dx = 0; dx < patch; dx += 2) {
        const float2 v = __ldg(s2 + (dx >> 1));
        store_pair(dst + dx, v.x, v.y);
      }
    } else {
      for (int dx = 0; dx < patch; ++dx) dst[dx] = to_out<T>(__ldg(src + dx));
    }
  }
}

// The same result with the work laid out along the image: a warp takes one pixel row of one channel of one input
// frame, reads it as consecutive pixel pairs (coalesced) and scatters the pairs to the patch rows they belong to (runs
// of `patch` elements); further warps write the zero pad of 32 tokens each.  Needs even patch, image and k_pad and
// 8-byte aligned frames; `raster2int` is the inverse of the order im2col_kernel takes (NULL: raster order).
template <typename T>
__global__ void im2col_rows_kernel(const float* __restrict__ frames, T* __restrict__ patches, int T_frames, int image,
                                   int patch, int grid, int k_pad, int tp, const int* __restrict__ raster2int,
                                   const int* __restrict__ n_frames_dev) {
  const int n_frames = n_frames_dev ? min(*n_frames_dev, T_frames) : T_frames;      // encoder frames
  const int L = grid * grid, crop = grid * patch, K = 3 * tp * patch * patch;
  const int lane = threadIdx.x & 31;
  const long long row_jobs = (long long)n_frames * tp * 3 * crop;
  const long long pad_jobs = K < k_pad ? ((long long)n_frames * L + 31) / 32 : 0;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long job = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); job < row_jobs + pad_jobs; job += warps) {
    if (job >= row_jobs) {
      const long long tok = (job - row_jobs) * 32 + lane;
      if (tok < (long long)n_frames * L)
        for (int c = K; c < k_pad; ++c) patches[tok * k_pad + c] = to_out<T>(0.f);
      continue;
    }
    const int y = (int)(job % crop);
    const long long fc = job / crop;                    // (input frame, channel)
    const int c = (int)(fc % 3);
    const long long f_in = fc / 3;
    const int t = (int)(f_in % tp);
    const long long f = f_in / tp;
    const int gy = y / patch, dy = y - gy * patch;
    const float2* src = reinterpret_cast<const float2*>(frames + ((f_in * 3 + c) * image + y) * image);
    T* const dst_frame = patches + f * L * (long long)k_pad + ((c * tp + t) * patch + dy) * patch;
    for (int x = 2 * lane; x < crop; x += 64) {
      const float2 v = __ldg(src + (x >> 1));
      const int gx = x / patch, dx = x - gx * patch;
      int l = gy * grid + gx;
      if (raster2int) l = raster2int[l];
      store_pair(dst_frame + (long long)l * k_pad + dx, v.x, v.y);
    }
  }
}

void launch_im2col(const float* frames, void* patches, int T, int image, int patch, int k_pad, bool out_bf16,
                   const int* n_frames_dev, cudaStream_t s, int tp, const int* int2raster, const int* raster2int) {
  const int grid = image / patch;
  if ((patch & 1) == 0 && (image & 1) == 0 && (k_pad & 1) == 0 && (reinterpret_cast<size_t>(frames) & 7) == 0 &&
      (int2raster == nullptr) == (raster2int == nullptr)) {
    const long long jobs = (long long)T * tp * 3 * grid * patch + ((long long)T * grid * grid + 31) / 32;
    const int threads = 256;
    const long long want = (jobs + 7) / 8;
    const int blocks = (int)(want < 148LL * 32 ? want : 148LL * 32);
    if (blocks == 0) return;
    ET_COUNT_LAUNCH();
    if (out_bf16)
      im2col_rows_kernel<bf16><<<blocks, threads, 0, s>>>(frames, (bf16*)patches, T, image, patch, grid, k_pad, tp, raster2int, n_frames_dev);
    else
      im2col_rows_kernel<float><<<blocks, threads, 0, s>>>(frames, (float*)patches, T, image, patch, grid, k_pad, tp, raster2int, n_frames_dev);
    return;
  }
  const long long total = (long long)T * grid * grid * (3 * tp * patch + 1);
  const int threads = 256;
  long long want = (total + threads - 1) / threads;
  const int blocks = (int)(want < 148LL * 32 ? want : 148LL * 32);
  if (blocks == 0) return;
  ET_COUNT_LAUNCH();
  if (out_bf16)
    im2col_kernel<bf16><<<blocks, threads, 0, s>>>(frames, (bf16*)patches, T, image, patch, grid, k_pad, tp, int2raster, n_frames_dev);
  else
    im2col_kernel<float><<<blocks, threads, 0, s>>>(frames, (float*)patches, T, image, patch, grid, k_pad, tp, int2raster, n_frames_dev);
}

// ---------------------------------------------------------------------------------------------
// LayerNorm: one warp per row, row held in registers, mean then centred variance (two passes over
// registers), fp32 statistics.  With b == NULL the kernel computes RMSNorm, y = x / sqrt(mean(x^2) + eps) * g.
// ---------------------------------------------------------------------------------------------
template <typename T, int NV>
__global__ void __launch_bounds__(256)
layernorm_kernel(const float* __restrict__ x, const float* __restrict__ g, const float* __restrict__ b, float eps,
                 T* __restrict__ y, int rows_cap, int D, const int* __restrict__ n_frames_dev, int rows_per_frame) {
  const int rows = n_frames_dev ? min(rows_cap, *n_frames_dev * rows_per_frame) : rows_cap;
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  for (int row = blockIdx.x * warps_per_block + (threadIdx.x >> 5); row < rows; row += gridDim.x * warps_per_block) {
    float4 v[NV];
    load_row<NV>(x + (size_t)row * D, D, lane, v);
    if (b) layernorm_row_inplace<NV>(v, D, lane, g, b, eps);
    else rmsnorm_row_inplace<NV>(v, D, lane, g, eps);          // no shift given: RMSNorm with gain g
    store_row<NV>(y + (size_t)row * D, D, lane, v);
  }
}

template <typename T>
void launch_layernorm_t(const float* x, const float* g, const float* b, float eps, T* y, int rows_cap, int D,
                        const int* n_frames_dev, int rows_per_frame, cudaStream_t s) {
  const int threads = 256, wpb = threads / 32;
  const int blocks = min(cdiv(rows_cap, wpb), 148 * 16);
  const int need = cdiv(D / 4, 32);      // float4 chunks per lane: the row lives in exactly that many registers
#define ET_LN(NV) layernorm_kernel<T, NV><<<blocks, threads, 0, s>>>(x, g, b, eps, y, rows_cap, D, n_frames_dev, rows_per_frame)
  if (need <= 1) ET_LN(1);
  else if (need <= 2) ET_LN(2);
  else if (need <= 4) ET_LN(4);
  else if (need <= 6) ET_LN(6);
  else if (need <= 9) ET_LN(9);
  else if (need <= 12) ET_LN(12);
  else ET_LN(16);
#undef ET_LN
}

void launch_layernorm(const float* x, const float* g, const float* b, float eps, void* y, int rows_cap, int D,
                      bool out_bf16, const int* n_frames_dev, int rows_per_frame, cudaStream_t s) {
  if (rows_cap <= 0) return;
  ET_COUNT_LAUNCH();
  if (out_bf16) launch_layernorm_t<bf16>(x, g, b, eps, (bf16*)y, rows_cap, D, n_frames_dev, rows_per_frame, s);
  else launch_layernorm_t<float>(x, g, b, eps, (float*)y, rows_cap, D, n_frames_dev, rows_per_frame, s);
}

// ---------------------------------------------------------------------------------------------
// 2-D rotary positions on the Q and K parts of packed rows [rows][3*D] (Q | K | V, head h at h*dh of its third):
// pair (x[i], x[i + dh/2]) of every head is turned by the angle of (token position in its frame, i); table
// [L][dh/2] holds (cos, sin).  One thread per (row, head, pair) for Q and K alike.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void rope_pairs_kernel(T* __restrict__ qkv, const float2* __restrict__ table, int rows_cap, int L, int heads,
                                  int dh, const int* __restrict__ n_frames_dev) {
  const int rows = n_frames_dev ? min(rows_cap, *n_frames_dev * L) : rows_cap;
  const int half = dh >> 1, D = heads * dh;
  const long long per_row = 2LL * heads * half;
  const long long total = (long long)rows * per_row;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(idx / per_row);
    int rem = (int)(idx % per_row);
    const int which = rem / (heads * half);             // 0 = Q, 1 = K
    rem %= heads * half;
    const int h = rem / half, i = rem % half;
    const float2 cs = __ldg(table + (size_t)(r % L) * half + i);
    T* p = qkv + (size_t)r * 3 * D + (size_t)which * D + h * dh + i;
    const float a = (float)p[0], b = (float)p[half];
    p[0] = to_out<T>(a * cs.x - b * cs.y);
    p[half] = to_out<T>(b * cs.x + a * cs.y);
  }
}

// The same, eight pairs per thread with 16-byte accesses (bf16 rows, dh/2 a multiple of 8).
__global__ void rope_pairs_vec8_kernel(bf16* __restrict__ qkv, const float2* __restrict__ table, int rows_cap, int L,
                                       int heads, int dh, const int* __restrict__ n_frames_dev) {
  const int rows = n_frames_dev ? min(rows_cap, *n_frames_dev * L) : rows_cap;
  const int half = dh >> 1, D = heads * dh, chunks = half >> 3;
  const long long per_row = 2LL * heads * chunks;
  const long long total = (long long)rows * per_row;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(idx / per_row);
    int rem = (int)(idx % per_row);
    const int which = rem / (heads * chunks);           // 0 = Q, 1 = K
    rem %= heads * chunks;
    const int h = rem / chunks, i0 = (rem % chunks) * 8;
    bf16* p = qkv + (size_t)r * 3 * D + (size_t)which * D + h * dh + i0;
    const float2* cs = table + (size_t)(r % L) * half + i0;
    uint4 va = *reinterpret_cast<const uint4*>(p), vb = *reinterpret_cast<const uint4*>(p + half);
    __nv_bfloat162* a2 = reinterpret_cast<__nv_bfloat162*>(&va);
    __nv_bfloat162* b2 = reinterpret_cast<__nv_bfloat162*>(&vb);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 a = __bfloat1622float2(a2[j]), b = __bfloat1622float2(b2[j]);
      const float2 c0 = __ldg(cs + 2 * j), c1 = __ldg(cs + 2 * j + 1);
      a2[j] = __floats2bfloat162_rn(a.x * c0.x - b.x * c0.y, a.y * c1.x - b.y * c1.y);
      b2[j] = __floats2bfloat162_rn(b.x * c0.x + a.x * c0.y, b.y * c1.x + a.y * c1.y);
    }
    *reinterpret_cast<uint4*>(p) = va;
    *reinterpret_cast<uint4*>(p + half) = vb;
  }
}

void launch_rope_pairs(void* qkv, const float2* table, int rows_cap, int L, int heads, int dh, bool is_bf16,
                       const int* n_frames_dev, cudaStream_t s) {
  if (rows_cap <= 0) return;
  ET_COUNT_LAUNCH();
  if (is_bf16 && (dh / 2) % 8 == 0 && (heads * dh) % 8 == 0) {
    const long long total = (long long)rows_cap * heads * (dh / 8);
    const int blocks = (int)min((total + 255) / 256, 148LL * 32);
    rope_pairs_vec8_kernel<<<blocks, 256, 0, s>>>((bf16*)qkv, table, rows_cap, L, heads, dh, n_frames_dev);
    return;
  }
  const long long total = (long long)rows_cap * heads * dh;
  const int blocks = (int)min((total + 255) / 256, 148LL * 32);
  if (is_bf16) rope_pairs_kernel<bf16><<<blocks, 256, 0, s>>>((bf16*)qkv, table, rows_cap, L, heads, dh, n_frames_dev);
  else rope_pairs_kernel<float><<<blocks, 256, 0, s>>>((float*)qkv, table, rows_cap, L, heads, dh, n_frames_dev);
}

// ---------------------------------------------------------------------------------------------
// Gated activation: h[r][j] = silu(gu[r][j]) * gu[r][Mp + j] for j < Mp (gu has 2*Mp columns: gate | up).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void gated_silu_kernel(const T* __restrict__ gu, T* __restrict__ h, int rows_cap, int Mp,
                                  const int* __restrict__ n_frames_dev, int rows_per_frame) {
  const int rows = n_frames_dev ? min(rows_cap, *n_frames_dev * rows_per_frame) : rows_cap;
  const long long total = (long long)rows * Mp;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const long long r = idx / Mp;
    const int j = (int)(idx % Mp);
    const float g = (float)gu[r * 2 * Mp + j], u = (float)gu[r * 2 * Mp + Mp + j];
    h[idx] = to_out<T>(g / (1.f + expf(-g)) * u);
  }
}

void launch_gated_silu(const void* gu, void* h, int rows_cap, int Mp, bool is_bf16, const int* n_frames_dev,
                       int rows_per_frame, cudaStream_t s) {
  if (rows_cap <= 0) return;
  const long long total = (long long)rows_cap * Mp;
  const int blocks = (int)min((total + 255) / 256, 148LL * 32);
  ET_COUNT_LAUNCH();
  if (is_bf16) gated_silu_kernel<bf16><<<blocks, 256, 0, s>>>((const bf16*)gu, (bf16*)h, rows_cap, Mp, n_frames_dev, rows_per_frame);
  else gated_silu_kernel<float><<<blocks, 256, 0, s>>>((const float*)gu, (float*)h, rows_cap, Mp, n_frames_dev, rows_per_frame);
}

// out[0] = in[0] * mult (the number of attention windows alive = frames alive * windows per frame)
__global__ void scale_count_kernel(const int* __restrict__ in, int mult, int* __restrict__ out) { out[0] = in[0] * mult; }
void launch_scale_count(const int* in, int mult, int* out, cudaStream_t s) {
  ET_COUNT_LAUNCH();
  scale_count_kernel<<<1, 1, 0, s>>>(in, mult, out);
}

}  // namespace et
