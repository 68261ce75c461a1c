// fp32 dense layer on the FFMA pipe (the ET_F32 arithmetic path): c = epi(a[M][K] * w[K][N] + bias).
// 64x64 tile, 16-deep k slices, 256 threads with 4x4 register tiles; every load is bounds-checked so
// that any M, N, K works.  This path exists for fp32 parity, not for speed.
#include "common.cuh"
#include "rowops.cuh"

namespace et {

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;

__global__ void __launch_bounds__(256)
gemm_f32_kernel(const float* __restrict__ a, const float* __restrict__ w, const float* __restrict__ bias,
                float* __restrict__ c, int M_cap, int N, int K, int epilogue, int gelu_tanh,
                const float* __restrict__ table, int table_rows, const int* __restrict__ n_frames_dev,
                int rows_per_frame) {
  const int M = n_frames_dev ? min(M_cap, *n_frames_dev * rows_per_frame) : M_cap;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  if (m0 >= M) return;
  __shared__ float As[SG_BK][SG_BM + 4];
  __shared__ float Bs[SG_BK][SG_BN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;       // 16 x 16 threads, each a 4x4 block
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
    for (int i = tid; i < SG_BM * SG_BK; i += 256) {
      const int r = i / SG_BK, kk = i % SG_BK;
      const int gm = m0 + r, gk = k0 + kk;
      As[kk][r] = (gm < M && gk < K) ? a[(size_t)gm * K + gk] : 0.f;
    }
    for (int i = tid; i < SG_BK * SG_BN; i += 256) {
      const int kk = i / SG_BN, cidx = i % SG_BN;
      const int gk = k0 + kk, gn = n0 + cidx;
      Bs[kk][cidx] = (gk < K && gn < N) ? w[(size_t)gk * N + gn] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SG_BK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = acc[i][j] + (bias ? bias[gn] : 0.f);
      float* dst = c + (size_t)gm * N + gn;
      if (epilogue == EPI_GELU) v = gelu_f(v, gelu_tanh);
      else if (epilogue == EPI_RESIDUAL) v += *dst;
      else if (epilogue == EPI_TABLE) v += table[(size_t)(gm % table_rows) * N + gn];
      *dst = v;
    }
  }
}

void launch_gemm_f32(const float* a, const float* w, const float* bias, float* c, int M_cap, int N, int K,
                     int epilogue, int gelu_tanh, const float* table, int table_rows, const int* n_frames_dev,
                     int rows_per_frame, cudaStream_t s) {
  if (M_cap <= 0 || N <= 0) return;
  ET_COUNT_LAUNCH();
  dim3 grid(cdiv(N, SG_BN), cdiv(M_cap, SG_BM));
  gemm_f32_kernel<<<grid, 256, 0, s>>>(a, w, bias, c, M_cap, N, K, epilogue, gelu_tanh, table, table_rows,
                                       n_frames_dev, rows_per_frame);
}

}  // namespace et
