// Per-frame multi-head attention and the per-token attention score on the FFMA pipe.
// Used by the ET_F32 arithmetic path (and as the shape-agnostic fallback): online softmax over key
// chunks, fp32 everywhere.  Template parameter T is the storage type of qkv / out.
#include "common.cuh"
#include "rowops.cuh"

namespace et {

template <typename T> __device__ __forceinline__ float ld_f(const T* p);
template <> __device__ __forceinline__ float ld_f<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_f<bf16>(const bf16* p) { return __bfloat162float(*p); }

constexpr int AS_QB = 16;     // queries per CTA (4 per warp)
constexpr int AS_KC = 32;     // keys per chunk (one per lane)

// grid (ceil(L/AS_QB), heads, frames), 128 threads.  qkv [n*L][3*D] with D = heads*dh.
template <typename T>
__global__ void __launch_bounds__(128)
attention_simt_kernel(const T* __restrict__ qkv, T* __restrict__ out, float* __restrict__ lse, int n_cap, int L,
                      int heads, int dh, const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * AS_QB;
  if (f >= n) return;
  extern __shared__ float sm[];
  const int ld = dh + 1;
  float* Qs = sm;                    // [AS_QB][ld]
  float* Ks = Qs + AS_QB * ld;       // [AS_KC][ld]
  float* Vs = Ks + AS_KC * ld;       // [AS_KC][ld]
  const int D = heads * dh;
  const size_t row_stride = (size_t)3 * D;
  const T* base = qkv + (size_t)f * L * row_stride + (size_t)h * dh;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float scale = 1.0f / sqrtf((float)dh);

  for (int i = tid; i < AS_QB * dh; i += 128) {
    const int r = i / dh, d = i % dh;
    Qs[r * ld + d] = (q0 + r < L) ? ld_f<T>(base + (size_t)(q0 + r) * row_stride + d) : 0.f;
  }
  float m[4], lsum[4], o[4][4];
#pragma unroll
  for (int qi = 0; qi < 4; ++qi) {
    m[qi] = -INFINITY; lsum[qi] = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) o[qi][c] = 0.f;
  }
  for (int k0 = 0; k0 < L; k0 += AS_KC) {
    __syncthreads();
    for (int i = tid; i < AS_KC * dh; i += 128) {
      const int r = i / dh, d = i % dh;
      const bool ok = k0 + r < L;
      const T* rowp = base + (size_t)(k0 + r) * row_stride;
      Ks[r * ld + d] = ok ? ld_f<T>(rowp + D + d) : 0.f;
      Vs[r * ld + d] = ok ? ld_f<T>(rowp + 2 * D + d) : 0.f;
    }
    __syncthreads();
    const bool key_ok = k0 + lane < L;
#pragma unroll
    for (int qi = 0; qi < 4; ++qi) {
      const float* qrow = Qs + (wid * 4 + qi) * ld;
      const float* krow = Ks + lane * ld;
      float s = 0.f;
      for (int d = 0; d < dh; ++d) s = fmaf(qrow[d], krow[d], s);
      s = key_ok ? s * scale : -INFINITY;
      const float m_new = fmaxf(m[qi], warp_max(s));
      const float p = key_ok ? __expf(s - m_new) : 0.f;
      const float corr = __expf(m[qi] - m_new);      // first chunk: exp(-inf) = 0
      lsum[qi] = lsum[qi] * corr + warp_sum(p);
      m[qi] = m_new;
#pragma unroll
      for (int c = 0; c < 4; ++c) o[qi][c] *= corr;
      for (int j = 0; j < AS_KC; ++j) {
        const float pj = __shfl_sync(0xffffffffu, p, j);
        const float* vrow = Vs + j * ld;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int d = lane + 32 * c;
          if (d < dh) o[qi][c] = fmaf(pj, vrow[d], o[qi][c]);
        }
      }
    }
  }
#pragma unroll
  for (int qi = 0; qi < 4; ++qi) {
    const int q = q0 + wid * 4 + qi;
    if (q >= L) continue;
    const float inv = 1.f / lsum[qi];
    T* orow = out + ((size_t)f * L + q) * D + (size_t)h * dh;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int d = lane + 32 * c;
      if (d < dh) orow[d] = to_out<T>(o[qi][c] * inv);
    }
    if (lane == 0) lse[((size_t)f * heads + h) * L + q] = m[qi] + logf(lsum[qi]);
  }
}

template <typename T>
static void launch_attention_simt(const T* qkv, T* out, float* lse, int n_cap, int L, int heads, int dh,
                                  const int* n_frames_dev, cudaStream_t s) {
  if (n_cap <= 0) return;
  const size_t smem = sizeof(float) * (AS_QB + 2 * AS_KC) * (dh + 1);
  ET_COUNT_LAUNCH();
  attention_simt_kernel<T><<<dim3(cdiv(L, AS_QB), heads, n_cap), 128, smem, s>>>(qkv, out, lse, n_cap, L, heads, dh,
                                                                                 n_frames_dev);
}

void launch_attention_f32(const float* qkv, float* out, float* lse, int n_cap, int L, int heads, int dh,
                          const int* n_frames_dev, cudaStream_t s) {
  launch_attention_simt<float>(qkv, out, lse, n_cap, L, heads, dh, n_frames_dev, s);
}

// ---------------------------------------------------------------------------------------------
// Attention score, pass 1: partial[f][h][j] = sum_q exp(scale * q.k_j - lse[q]).
// grid (ceil(L/32), heads, frames), 128 threads; lane = key, warp w takes queries w, w+4, ...;
// the four warp sums are added in a fixed order.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128)
score_partial_simt_kernel(const T* __restrict__ qkv, const float* __restrict__ lse, float* __restrict__ partial,
                          int n_cap, int L, int heads, int dh, const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.z, h = blockIdx.y, k0 = blockIdx.x * 32;
  if (f >= n) return;
  extern __shared__ float sm[];
  const int ld = dh + 1;
  float* Ks = sm;              // [32][ld]
  float* Qs = Ks + 32 * ld;    // [32][ld]
  float* Ls = Qs + 32 * ld;    // [32]
  __shared__ float red[4][32];
  const int D = heads * dh;
  const size_t row_stride = (size_t)3 * D;
  const T* base = qkv + (size_t)f * L * row_stride + (size_t)h * dh;
  const float* lse_row = lse + ((size_t)f * heads + h) * L;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float scale = 1.0f / sqrtf((float)dh);
  for (int i = tid; i < 32 * dh; i += 128) {
    const int r = i / dh, d = i % dh;
    Ks[r * ld + d] = (k0 + r < L) ? ld_f<T>(base + (size_t)(k0 + r) * row_stride + D + d) : 0.f;
  }
  float acc = 0.f;
  for (int q0 = 0; q0 < L; q0 += 32) {
    __syncthreads();
    for (int i = tid; i < 32 * dh; i += 128) {
      const int r = i / dh, d = i % dh;
      Qs[r * ld + d] = (q0 + r < L) ? ld_f<T>(base + (size_t)(q0 + r) * row_stride + d) : 0.f;
    }
    if (tid < 32) Ls[tid] = (q0 + tid < L) ? lse_row[q0 + tid] : 0.f;
    __syncthreads();
    for (int r = wid; r < 32 && q0 + r < L; r += 4) {
      const float* qrow = Qs + r * ld;
      const float* krow = Ks + lane * ld;
      float s = 0.f;
      for (int d = 0; d < dh; ++d) s = fmaf(qrow[d], krow[d], s);
      acc += __expf(s * scale - Ls[r]);
    }
  }
  red[wid][lane] = acc;
  __syncthreads();
  if (wid == 0 && k0 + lane < L)
    partial[((size_t)f * heads + h) * L + k0 + lane] = (red[0][lane] + red[1][lane]) + (red[2][lane] + red[3][lane]);
}

// pass 2: score[f][j] = (sum_h partial[f][h][j]) / (heads * L), heads added in ascending order.
__global__ void score_finish_kernel(const float* __restrict__ partial, float* __restrict__ score, int n_cap, int L,
                                    int heads, const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.y;
  if (f >= n) return;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= L) return;
  float acc = 0.f;
  for (int h = 0; h < heads; ++h) acc += partial[((size_t)f * heads + h) * L + j];
  score[(size_t)f * L + j] = acc / ((float)heads * (float)L);
}

void launch_score_finish(const float* partial, float* score, int n_cap, int L, int heads, const int* n_frames_dev,
                         cudaStream_t s) {
  ET_COUNT_LAUNCH();
  score_finish_kernel<<<dim3(cdiv(L, 128), n_cap), 128, 0, s>>>(partial, score, n_cap, L, heads, n_frames_dev);
}

template <typename T>
static void launch_scores_simt(const T* qkv, const float* lse, float* partial, float* score, int n_cap, int L, int heads,
                               int dh, const int* n_frames_dev, cudaStream_t s) {
  if (n_cap <= 0) return;
  const size_t smem = sizeof(float) * (64 * (dh + 1) + 32);
  ET_COUNT_LAUNCH();
  score_partial_simt_kernel<T><<<dim3(cdiv(L, 32), heads, n_cap), 128, smem, s>>>(qkv, lse, partial, n_cap, L, heads,
                                                                                  dh, n_frames_dev);
  launch_score_finish(partial, score, n_cap, L, heads, n_frames_dev, s);
}

void launch_attention_scores_f32(const float* qkv, const float* lse, float* partial, float* score, int n_cap, int L,
                                 int heads, int dh, const int* n_frames_dev, cudaStream_t s) {
  launch_scores_simt<float>(qkv, lse, partial, score, n_cap, L, heads, dh, n_frames_dev, s);
}

// bf16 storage, FFMA arithmetic: fallback for shapes the tensor-core kernels do not cover.
void launch_attention_bf16_simt(const bf16* qkv, bf16* out, float* lse, int n_cap, int L, int heads, int dh,
                                const int* n_frames_dev, cudaStream_t s) {
  launch_attention_simt<bf16>(qkv, out, lse, n_cap, L, heads, dh, n_frames_dev, s);
}
void launch_attention_scores_bf16_simt(const bf16* qkv, const float* lse, float* partial, float* score, int n_cap, int L,
                                       int heads, int dh, const int* n_frames_dev, cudaStream_t s) {
  launch_scores_simt<bf16>(qkv, lse, partial, score, n_cap, L, heads, dh, n_frames_dev, s);
}

}  // namespace et
