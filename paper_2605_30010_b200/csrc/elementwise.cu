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

template <typename T>
__global__ void im2col_kernel(const float* __restrict__ frames, T* __restrict__ patches, int T_frames, int image,
                              int patch, int grid, int k_pad, const int* __restrict__ n_frames_dev) {
  const int n_frames = n_frames_dev ? min(*n_frames_dev, T_frames) : T_frames;
  const int L = grid * grid;
  const int rows_per_tok = 3 * patch + 1;  // 3*p pixel rows + one job that writes the zero pad
  const long long total = (long long)n_frames * L * rows_per_tok;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int job = (int)(idx % rows_per_tok);
    const long long tok = idx / rows_per_tok;
    T* dst_row = patches + tok * k_pad;
    if (job == 3 * patch) {
      for (int c = 3 * patch * patch; c < k_pad; ++c) dst_row[c] = to_out<T>(0.f);
      continue;
    }
    const int c = job / patch, dy = job % patch;
    const int f = (int)(tok / L), l = (int)(tok % L);
    const int gy = l / grid, gx = l % grid;
    const float* src = frames + (((long long)f * 3 + c) * image + (gy * patch + dy)) * image + gx * patch;
    T* dst = dst_row + (c * patch + dy) * patch;
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

void launch_im2col(const float* frames, void* patches, int T, int image, int patch, int k_pad, bool out_bf16,
                   const int* n_frames_dev, cudaStream_t s) {
  const int grid = image / patch;
  const long long total = (long long)T * grid * grid * (3 * patch + 1);
  const int threads = 256;
  long long want = (total + threads - 1) / threads;
  const int blocks = (int)(want < 148LL * 32 ? want : 148LL * 32);
  if (blocks == 0) return;
  ET_COUNT_LAUNCH();
  if (out_bf16)
    im2col_kernel<bf16><<<blocks, threads, 0, s>>>(frames, (bf16*)patches, T, image, patch, grid, k_pad, n_frames_dev);
  else
    im2col_kernel<float><<<blocks, threads, 0, s>>>(frames, (float*)patches, T, image, patch, grid, k_pad, n_frames_dev);
}

// ---------------------------------------------------------------------------------------------
// LayerNorm: one warp per row, row held in registers, mean then centred variance (two passes over
// registers), fp32 statistics.
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
    layernorm_row_inplace<NV>(v, D, lane, g, b, eps);
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

}  // namespace et
