// Per-frame multi-head attention in bf16 on the tensor cores (warp-level m16n8k16 MMA, fp32
// accumulate) with online softmax, and the tensor-core pass that turns the last block's attention
// into per-token scores.  Head dims that are not a multiple of 16 (72 for SigLIP-so400m) are
// zero-padded in shared memory only; global memory keeps the packed [tokens][3*D] layout.
#include "common.cuh"
#include "rowops.cuh"

namespace et {

void launch_attention_bf16_simt(const bf16* qkv, bf16* out, float* lse, int n_cap, int L, int heads, int dh,
                                const int* n_frames_dev, cudaStream_t s);
void launch_attention_scores_bf16_simt(const bf16* qkv, const float* lse, float* partial, float* score, int n_cap, int L,
                                       int heads, int dh, const int* n_frames_dev, cudaStream_t s);
void launch_score_finish(const float* partial, float* score, int n_cap, int L, int heads, const int* n_frames_dev,
                         cudaStream_t s);

namespace {

constexpr int QT = 64;      // queries per CTA (16 per warp)
constexpr int KT = 64;      // keys per tile
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;       // src-size 0 -> 16 bytes of zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory row pitch (in bf16): head dim padded to a multiple of 16, plus 8 so that the eight
// rows of an ldmatrix phase fall into distinct 16-byte bank groups.
template <int DH> struct Geo {
  static constexpr int DHP = (DH + 15) / 16 * 16;
  static constexpr int PITCH = DHP + 8;
  static constexpr int CHUNKS = DH / 8;            // 16-byte chunks per row in global memory
  static constexpr int KSTEPS = DHP / 16;          // k-steps of Q K^T
  static constexpr int NT_O = DH / 8;              // n-tiles of the output
};

// Loads `rows` rows of one of Q/K/V (global row stride row_stride, DH valid columns) into a tile.
template <int DH>
__device__ __forceinline__ void load_tile(uint32_t tile_smem, const bf16* gbase, size_t row_stride, int row0, int rows,
                                          int L, int tid, int nthreads) {
  using G = Geo<DH>;
  for (int i = tid; i < rows * G::CHUNKS; i += nthreads) {
    const int r = i / G::CHUNKS, c = i % G::CHUNKS;
    const bool ok = row0 + r < L;
    const bf16* src = gbase + (size_t)(ok ? row0 + r : 0) * row_stride + c * 8;
    cp_async16(tile_smem + (uint32_t)(r * G::PITCH + c * 8) * 2u, src, ok);
  }
}

template <int DH>
__global__ void __launch_bounds__(128)
attention_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ out, float* __restrict__ lse, int n_cap, int L,
                     int heads, const int* __restrict__ n_frames_dev) {
  using G = Geo<DH>;
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * QT;
  if (f >= n) return;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);                  // [QT][PITCH]
  bf16* Ks = Qs + QT * G::PITCH;                                  // [2][KT][PITCH]
  bf16* Vs = Ks + 2 * KT * G::PITCH;                              // [2][KT][PITCH]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = heads * DH;
  const size_t row_stride = (size_t)3 * D;
  const bf16* qg = qkv + (size_t)f * L * row_stride + (size_t)h * DH;
  const bf16* kg = qg + D;
  const bf16* vg = qg + 2 * D;

  // zero the padded contraction columns [DH, DHP) of Q and K once (cp.async never writes them)
  if constexpr (G::DHP > DH) {
    constexpr int PADC = G::DHP - DH;
    for (int i = tid; i < (QT + 2 * KT) * PADC; i += 128) {
      const int r = i / PADC, c = DH + i % PADC;
      Qs[r * G::PITCH + c] = __float2bfloat16_rn(0.f);     // Qs and Ks are contiguous: rows QT.. are K rows
    }
  }
  const int n_tiles = (L + KT - 1) / KT;
  load_tile<DH>(smem_u32(Qs), qg, row_stride, q0, QT, L, tid, 128);
  load_tile<DH>(smem_u32(Ks), kg, row_stride, 0, KT, L, tid, 128);
  load_tile<DH>(smem_u32(Vs), vg, row_stride, 0, KT, L, tid, 128);
  cp_async_commit();

  const float scale2 = LOG2E / sqrtf((float)DH);      // logits are kept in the log2 domain
  uint32_t qf[G::KSTEPS][4];
  float o[G::NT_O][4];
#pragma unroll
  for (int j = 0; j < G::NT_O; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  for (int t = 0; t < n_tiles; ++t) {
    const int buf = t & 1;
    if (t + 1 < n_tiles) {
      load_tile<DH>(smem_u32(Ks + (buf ^ 1) * KT * G::PITCH), kg, row_stride, (t + 1) * KT, KT, L, tid, 128);
      load_tile<DH>(smem_u32(Vs + (buf ^ 1) * KT * G::PITCH), vg, row_stride, (t + 1) * KT, KT, L, tid, 128);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (t == 0) {
#pragma unroll
      for (int ks = 0; ks < G::KSTEPS; ++ks) {
        const int row = warp * 16 + (lane & 15), col = ks * 16 + (lane >> 4) * 8;
        ldsm_x4(smem_u32(Qs + row * G::PITCH + col), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const bf16* Kt = Ks + buf * KT * G::PITCH;
    const bf16* Vt = Vs + buf * KT * G::PITCH;
    // ---- S = Q K^T for 16 queries x 64 keys
    float sacc[KT / 8][4];
#pragma unroll
    for (int j = 0; j < KT / 8; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < G::KSTEPS; ++ks) {
#pragma unroll
      for (int jp = 0; jp < KT / 16; ++jp) {
        const int key = jp * 16 + (lane >> 4) * 8 + (lane & 7), col = ks * 16 + ((lane >> 3) & 1) * 8;
        uint32_t b0, b1, b2, b3;
        ldsm_x4(smem_u32(Kt + key * G::PITCH + col), b0, b1, b2, b3);
        mma_bf16(sacc[2 * jp], qf[ks], b0, b1);
        mma_bf16(sacc[2 * jp + 1], qf[ks], b2, b3);
      }
    }
    // ---- online softmax (rows lane/4 and lane/4 + 8 of this warp's 16 queries)
    const int key_base = t * KT + (lane & 3) * 2;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < KT / 8; ++j) {
      const int k0 = key_base + j * 8;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool ok = k0 + (e & 1) < L;
        sacc[j][e] = ok ? sacc[j][e] * scale2 : -INFINITY;
      }
      mx[0] = fmaxf(mx[0], fmaxf(sacc[j][0], sacc[j][1]));
      mx[1] = fmaxf(mx[1], fmaxf(sacc[j][2], sacc[j][3]));
    }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);      // finite: every tile holds at least one valid key
      corr[r] = exp2f(m_run[r] - m_new);
      m_run[r] = m_new;
    }
    float rs[2] = {0.f, 0.f};
    uint32_t pf[KT / 16][4];
#pragma unroll
    for (int j = 0; j < KT / 8; ++j) {
      const float p0 = exp2f(sacc[j][0] - m_run[0]), p1 = exp2f(sacc[j][1] - m_run[0]);
      const float p2 = exp2f(sacc[j][2] - m_run[1]), p3 = exp2f(sacc[j][3] - m_run[1]);
      rs[0] += p0 + p1;
      rs[1] += p2 + p3;
      pf[j >> 1][(j & 1) * 2 + 0] = pack2(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = pack2(p2, p3);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + rs[r];   // per-thread partial row sums
#pragma unroll
    for (int j = 0; j < G::NT_O; ++j) {
      o[j][0] *= corr[0]; o[j][1] *= corr[0];
      o[j][2] *= corr[1]; o[j][3] *= corr[1];
    }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < KT / 16; ++kk) {
      const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int jp = 0; jp < G::NT_O / 2; ++jp) {
        const int col = jp * 16 + (lane >> 4) * 8;
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(smem_u32(Vt + key * G::PITCH + col), b0, b1, b2, b3);
        mma_bf16(o[2 * jp], pf[kk], b0, b1);
        mma_bf16(o[2 * jp + 1], pf[kk], b2, b3);
      }
      if (G::NT_O & 1) {
        const int col = (G::NT_O - 1) * 8;
        uint32_t b0, b1;
        ldsm_x2_t(smem_u32(Vt + key * G::PITCH + col), b0, b1);
        mma_bf16(o[G::NT_O - 1], pf[kk], b0, b1);
      }
    }
    __syncthreads();     // all warps are done with this buffer before the next prefetch overwrites it
  }
  // ---- finish: full row sums across the quad, normalise, store
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int q = q0 + warp * 16 + (lane >> 2) + r * 8;
    if (q >= L) continue;
    const float inv = 1.f / l_run[r];
    bf16* orow = out + ((size_t)f * L + q) * D + (size_t)h * DH + (lane & 3) * 2;
#pragma unroll
    for (int j = 0; j < G::NT_O; ++j)
      *reinterpret_cast<uint32_t*>(orow + j * 8) = pack2(o[j][r * 2] * inv, o[j][r * 2 + 1] * inv);
    if ((lane & 3) == 0) lse[((size_t)f * heads + h) * L + q] = (m_run[r] + log2f(l_run[r])) * LN2;
  }
}

// ---------------------------------------------------------------------------------------------
// Score pass: partial[f][h][j] = sum_q exp(scale q.k_j - lse_q).  The CTA owns 64 keys of one
// (frame, head) and sweeps all query tiles: S^T = K Q^T on the tensor cores (keys are the MMA rows,
// so a thread's accumulator rows are keys and the sum over queries is a sum over its columns plus a
// quad reduction).  Query tiles are visited in a fixed order and the four warps own disjoint keys, so
// the result is bit-reproducible.
// ---------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(128)
score_mma_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse, float* __restrict__ partial, int n_cap,
                 int L, int heads, const int* __restrict__ n_frames_dev) {
  using G = Geo<DH>;
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.z, h = blockIdx.y, k0 = blockIdx.x * KT;
  if (f >= n) return;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);                  // [KT][PITCH]  (the MMA "A" operand)
  bf16* Qs = Ks + KT * G::PITCH;                                  // [2][QT][PITCH]
  float* Ls = reinterpret_cast<float*>(Qs + 2 * QT * G::PITCH);   // [2][QT] lse of the query tile (log2 domain)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = heads * DH;
  const size_t row_stride = (size_t)3 * D;
  const bf16* qg = qkv + (size_t)f * L * row_stride + (size_t)h * DH;
  const bf16* kg = qg + D;
  const float* lse_row = lse + ((size_t)f * heads + h) * L;
  if constexpr (G::DHP > DH) {
    constexpr int PADC = G::DHP - DH;
    for (int i = tid; i < (KT + 2 * QT) * PADC; i += 128) {
      const int r = i / PADC, c = DH + i % PADC;
      Ks[r * G::PITCH + c] = __float2bfloat16_rn(0.f);
    }
  }
  const int n_tiles = (L + QT - 1) / QT;
  load_tile<DH>(smem_u32(Ks), kg, row_stride, k0, KT, L, tid, 128);
  load_tile<DH>(smem_u32(Qs), qg, row_stride, 0, QT, L, tid, 128);
  cp_async_commit();
  if (tid < QT) Ls[tid] = (tid < L) ? lse_row[tid] * LOG2E : INFINITY;

  const float scale2 = LOG2E / sqrtf((float)DH);
  uint32_t kf[G::KSTEPS][4];
  float acc_rows[2] = {0.f, 0.f};
  for (int t = 0; t < n_tiles; ++t) {
    const int buf = t & 1;
    if (t + 1 < n_tiles) {
      load_tile<DH>(smem_u32(Qs + (buf ^ 1) * QT * G::PITCH), qg, row_stride, (t + 1) * QT, QT, L, tid, 128);
      cp_async_commit();
      if (tid < QT) {
        const int q = (t + 1) * QT + tid;
        Ls[(buf ^ 1) * QT + tid] = (q < L) ? lse_row[q] * LOG2E : INFINITY;    // exp2(-inf) = 0 for padded queries
      }
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (t == 0) {
#pragma unroll
      for (int ks = 0; ks < G::KSTEPS; ++ks) {
        const int row = warp * 16 + (lane & 15), col = ks * 16 + (lane >> 4) * 8;
        ldsm_x4(smem_u32(Ks + row * G::PITCH + col), kf[ks][0], kf[ks][1], kf[ks][2], kf[ks][3]);
      }
    }
    const bf16* Qt = Qs + buf * QT * G::PITCH;
    const float* Lt = Ls + buf * QT;
    float sacc[QT / 8][4];
#pragma unroll
    for (int j = 0; j < QT / 8; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < G::KSTEPS; ++ks) {
#pragma unroll
      for (int jp = 0; jp < QT / 16; ++jp) {
        const int qrow = jp * 16 + (lane >> 4) * 8 + (lane & 7), col = ks * 16 + ((lane >> 3) & 1) * 8;
        uint32_t b0, b1, b2, b3;
        ldsm_x4(smem_u32(Qt + qrow * G::PITCH + col), b0, b1, b2, b3);
        mma_bf16(sacc[2 * jp], kf[ks], b0, b1);
        mma_bf16(sacc[2 * jp + 1], kf[ks], b2, b3);
      }
    }
#pragma unroll
    for (int j = 0; j < QT / 8; ++j) {
      const int qc = j * 8 + (lane & 3) * 2;
      const float l0 = Lt[qc], l1 = Lt[qc + 1];
      acc_rows[0] += exp2f(sacc[j][0] * scale2 - l0) + exp2f(sacc[j][1] * scale2 - l1);
      acc_rows[1] += exp2f(sacc[j][2] * scale2 - l0) + exp2f(sacc[j][3] * scale2 - l1);
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    acc_rows[r] += __shfl_xor_sync(0xffffffffu, acc_rows[r], 1);
    acc_rows[r] += __shfl_xor_sync(0xffffffffu, acc_rows[r], 2);
    const int key = k0 + warp * 16 + (lane >> 2) + r * 8;
    if ((lane & 3) == 0 && key < L) partial[((size_t)f * heads + h) * L + key] = acc_rows[r];
  }
}

template <int DH> size_t attn_smem() { return (size_t)(QT + 4 * KT) * Geo<DH>::PITCH * 2; }
template <int DH> size_t score_smem() { return (size_t)(KT + 2 * QT) * Geo<DH>::PITCH * 2 + 2 * QT * sizeof(float); }

template <int DH>
void run_attention(const bf16* qkv, bf16* out, float* lse, int n_cap, int L, int heads, const int* n_frames_dev,
                   cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(attention_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem<DH>());
    configured = true;
  }
  ET_COUNT_LAUNCH();
  attention_mma_kernel<DH><<<dim3(cdiv(L, QT), heads, n_cap), 128, attn_smem<DH>(), s>>>(qkv, out, lse, n_cap, L, heads,
                                                                                       n_frames_dev);
}

template <int DH>
void run_scores(const bf16* qkv, const float* lse, float* partial, int n_cap, int L, int heads, const int* n_frames_dev,
                cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(score_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)score_smem<DH>());
    configured = true;
  }
  ET_COUNT_LAUNCH();
  score_mma_kernel<DH><<<dim3(cdiv(L, KT), heads, n_cap), 128, score_smem<DH>(), s>>>(qkv, lse, partial, n_cap, L, heads,
                                                                                    n_frames_dev);
}

}  // namespace

bool attention_bf16_supported(int L, int heads, int dh) {
  (void)heads;
  return L >= 1 && (dh == 16 || dh == 32 || dh == 64 || dh == 72 || dh == 80 || dh == 96 || dh == 128);
}

void launch_attention_bf16(const bf16* qkv, bf16* out, float* lse, int n_cap, int L, int heads, int dh,
                           const int* n_frames_dev, cudaStream_t s) {
  if (n_cap <= 0) return;
  switch (dh) {
    case 16: run_attention<16>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    case 32: run_attention<32>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    case 64: run_attention<64>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    case 72: run_attention<72>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    case 80: run_attention<80>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    case 96: run_attention<96>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    case 128: run_attention<128>(qkv, out, lse, n_cap, L, heads, n_frames_dev, s); break;
    default: launch_attention_bf16_simt(qkv, out, lse, n_cap, L, heads, dh, n_frames_dev, s);
  }
}

void launch_attention_scores_bf16(const bf16* qkv, const float* lse, float* partial, float* score, int n_cap, int L,
                                  int heads, int dh, const int* n_frames_dev, cudaStream_t s) {
  if (n_cap <= 0) return;
  switch (dh) {
    case 16: run_scores<16>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    case 32: run_scores<32>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    case 64: run_scores<64>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    case 72: run_scores<72>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    case 80: run_scores<80>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    case 96: run_scores<96>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    case 128: run_scores<128>(qkv, lse, partial, n_cap, L, heads, n_frames_dev, s); break;
    default: launch_attention_scores_bf16_simt(qkv, lse, partial, score, n_cap, L, heads, dh, n_frames_dev, s); return;
  }
  launch_score_finish(partial, score, n_cap, L, heads, n_frames_dev, s);
}

}  // namespace et
