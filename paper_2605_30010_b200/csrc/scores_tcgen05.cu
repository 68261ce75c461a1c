// Per-token attention score of the last block on the 5th-generation tensor cores.
//
//   partial[f][h][j] = sum_q exp(scale * q . k_j - lse[f][h][q])        (score = sum_h partial / (heads * L))
//
// One CTA owns 128 keys of one (frame, head) and sweeps the frame's queries in tiles of 128.  The logits are
// computed transposed, S^T = K Q^T (keys are the MMA rows, so a key is a TMEM lane and a consumer thread), which
// turns the sum over queries into a sum over the columns a thread reads from TMEM: no cross-thread reduction,
// fixed order, bit-reproducible.
//   warp 0      TMA producer: the K tile once, then a two-stage ring of Q tiles
//   warp 1      allocates TMEM (two 128-column accumulators) and issues the MMAs
//   warps 2..5  consumers: tcgen05.ld, exp2(s * scale - lse_q) with the query's log-sum-exp broadcast from a
//               per-warp copy in shared memory, running sum per key
// Head dim 64 or 72, operand tiles as in the attention kernel (64-element swizzled rows plus an 8-element tail
// whose contraction step is completed by a block of zeros).
#include "common.cuh"
#include "tcgen05.cuh"

namespace et {

void launch_score_finish(const float* partial, float* score, int n_cap, int L, int heads, const int* n_frames_dev,
                         cudaStream_t s);

namespace {

using namespace tc;

constexpr int TILE = 128;
constexpr int SC_THREADS = 192;
constexpr int MAIN_BYTES = 128 * 128, TAIL_BYTES = 128 * 16;
constexpr int Q_STAGES = 2;
constexpr float LOG2E = 1.4426950408889634f;

constexpr int OFF_K_MAIN = 0;
constexpr int OFF_Q_MAIN = OFF_K_MAIN + MAIN_BYTES;
constexpr int OFF_K_TAIL = OFF_Q_MAIN + Q_STAGES * MAIN_BYTES;
constexpr int OFF_Q_TAIL = OFF_K_TAIL + TAIL_BYTES;
constexpr int OFF_ZERO = OFF_Q_TAIL + Q_STAGES * TAIL_BYTES;
constexpr int OFF_LSE = OFF_ZERO + TAIL_BYTES;                 // [4 warps][2 buffers][128] floats: -lse * log2(e)
constexpr int OFF_BARS = OFF_LSE + 4 * 2 * TILE * 4;
constexpr int SC_SMEM_BYTES = OFF_BARS + 128 + 1024;
constexpr int B_K_FULL = 0, B_Q_FULL = 1, B_Q_EMPTY = B_Q_FULL + Q_STAGES, B_S_FULL = B_Q_EMPTY + Q_STAGES,
              B_S_EMPTY = B_S_FULL + 2, B_COUNT = B_S_EMPTY + 2;
static_assert(B_COUNT * 8 + 8 <= 128, "barrier area");
constexpr int TMEM_COLS = 256;

struct ScoreArgs {
  const float* lse;
  float* partial;
  int n_cap, L, heads;
  const int* n_frames_dev;
  int* status;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int DH>
__global__ void __launch_bounds__(SC_THREADS, 2)
scores_tc_kernel(const __grid_constant__ CUtensorMap tma_main, const __grid_constant__ CUtensorMap tma_tail, ScoreArgs g) {
  constexpr bool HAS_TAIL = DH > 64;
  static_assert(DH == 64 || DH == 72, "head dim");
  const int n = g.n_frames_dev ? min(*g.n_frames_dev, g.n_cap) : g.n_cap;
  const int f = blockIdx.z, h = blockIdx.y, k0 = blockIdx.x * TILE;
  if (f >= n) return;
  const int L = g.L, D = g.heads * DH;
  const int n_tiles = (L + TILE - 1) / TILE;
  const int row_base = f * L;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* const gen_base = smem_raw + (base - raw);
  const uint32_t bar_base = base + OFF_BARS;
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_ptr_slot = reinterpret_cast<volatile uint32_t*>(gen_base + OFF_BARS + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + OFF_BARS + 8 * B_COUNT + 4);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_K_FULL), 1);
    for (int s = 0; s < Q_STAGES; ++s) { mbar_init(bar(B_Q_FULL + s), 1); mbar_init(bar(B_Q_EMPTY + s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar(B_S_FULL + a), 1); mbar_init(bar(B_S_EMPTY + a), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = threadIdx.x; i < TAIL_BYTES / 16; i += SC_THREADS)
    reinterpret_cast<uint4*>(gen_base + OFF_ZERO)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_ptr_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem_base = *tmem_ptr_slot;
  auto queries_rounded = [&](int t) { return (min(TILE, L - t * TILE) + 15) & ~15; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      constexpr uint32_t TILE_TX = MAIN_BYTES + (HAS_TAIL ? TAIL_BYTES : 0);
      mbar_arrive_expect_tx(bar(B_K_FULL), TILE_TX);
      tma_load_2d(base + OFF_K_MAIN, &tma_main, bar(B_K_FULL), D + h * DH, row_base + k0);
      if (HAS_TAIL) tma_load_2d(base + OFF_K_TAIL, &tma_tail, bar(B_K_FULL), D + h * DH + 64, row_base + k0);
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t % Q_STAGES;
        if (!mbar_wait(bar(B_Q_EMPTY + s), ((uint32_t)(t / Q_STAGES) & 1u) ^ 1u, abort_flag)) break;
        mbar_arrive_expect_tx(bar(B_Q_FULL + s), TILE_TX);
        tma_load_2d(base + OFF_Q_MAIN + s * MAIN_BYTES, &tma_main, bar(B_Q_FULL + s), h * DH, row_base + t * TILE);
        if (HAS_TAIL) tma_load_2d(base + OFF_Q_TAIL + s * TAIL_BYTES, &tma_tail, bar(B_Q_FULL + s), h * DH + 64, row_base + t * TILE);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: S^T = K Q^T per query tile
    const uint32_t zero = base + OFF_ZERO;
    const uint64_t k_main = smem_desc(base + OFF_K_MAIN, 16, 1024, 2);
    const uint64_t k_tail = smem_desc(base + OFF_K_TAIL, zero - (base + OFF_K_TAIL), 128, 0);
    bool ok = mbar_wait_warp(bar(B_K_FULL), 0, abort_flag);
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int s = t % Q_STAGES, a = t & 1;
      if (!mbar_wait_warp(bar(B_Q_FULL + s), (uint32_t)(t / Q_STAGES) & 1u, abort_flag)) break;
      if (!mbar_wait_warp(bar(B_S_EMPTY + a), ((uint32_t)(t >> 1) & 1u) ^ 1u, abort_flag)) break;
      fence_after();
      const uint32_t idesc = idesc_bf16(128, queries_rounded(t), false, false);
      const uint64_t q_main = smem_desc(base + OFF_Q_MAIN + s * MAIN_BYTES, 16, 1024, 2);
      const uint32_t qt = base + OFF_Q_TAIL + s * TAIL_BYTES;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) mma_ss_elect(tmem_base + a * TILE, k_main + 2 * ks, q_main + 2 * ks, idesc, ks != 0 ? 1u : 0u);
      if (HAS_TAIL) mma_ss_elect(tmem_base + a * TILE, k_tail, smem_desc(qt, zero - qt, 128, 0), idesc, 1u);
      commit_elect(bar(B_S_FULL + a));
      commit_elect(bar(B_Q_EMPTY + s));
    }
  } else {
    // ------------------------------------------------------------------ consumers: one key per thread
    const int quarter = warp & 3;
    const int key = k0 + quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float* const my_lse = reinterpret_cast<float*>(gen_base + OFF_LSE) + (warp - 2) * 2 * TILE;
    const float* lse_row = g.lse + ((size_t)f * g.heads + h) * L;
    const float scale2 = LOG2E / sqrtf((float)DH);
    float acc0 = 0.f, acc1 = 0.f;
    for (int t = 0; t < n_tiles; ++t) {
      const int a = t & 1;
      float* nl = my_lse + a * TILE;                  // -lse * log2(e) of this tile's queries; -inf beyond the frame
#pragma unroll
      for (int i = 0; i < TILE / 32; ++i) {
        const int q = t * TILE + i * 32 + lane;
        nl[i * 32 + lane] = (q < L) ? -lse_row[q] * LOG2E : -INFINITY;
      }
      __syncwarp();
      if (!mbar_wait_warp(bar(B_S_FULL + a), (uint32_t)(t >> 1) & 1u, abort_flag)) break;
      fence_after();
      const int qr = queries_rounded(t);
      const int nch = (qr + 31) >> 5;
      for (int c = 0; c < nch; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_addr + a * TILE + c * 32, r);
        const float4* nl4 = reinterpret_cast<const float4*>(nl + c * 32);
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          if (c * 32 + i >= qr) break;                // columns beyond the MMA's width hold stale TMEM contents
          const float4 m = nl4[i >> 2];               // all lanes read the same address: a broadcast
          float x0, x1, x2, x3;
          fma2(x0, x1, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), scale2, scale2, m.x, m.y);
          fma2(x2, x3, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]), scale2, scale2, m.z, m.w);
          add2(acc0, acc1, acc0, acc1, ex2(x0), ex2(x1));
          add2(acc0, acc1, acc0, acc1, ex2(x2), ex2(x3));
        }
      }
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_S_EMPTY + a));
    }
    if (key < L) g.partial[((size_t)f * g.heads + h) * L + key] = acc0 + acc1;
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  fence_before();
  __syncthreads();
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    if (threadIdx.x == 0 && g.status) atomicExch(g.status, (int)DS_WAIT_EXPIRED);
    __syncthreads();
  }
  if (warp == 1) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}


template <int DH>
cudaError_t run(const AttnMaps& maps, const ScoreArgs& a, cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(scores_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, SC_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  ET_COUNT_LAUNCH();
  scores_tc_kernel<DH><<<dim3(cdiv(a.L, TILE), a.heads, a.n_cap), SC_THREADS, SC_SMEM_BYTES, s>>>(
      *reinterpret_cast<const CUtensorMap*>(maps.main.bytes), *reinterpret_cast<const CUtensorMap*>(maps.tail.bytes), a);
  return cudaGetLastError();
}

}  // namespace

bool attention_scores_tc_supported(int dh) { return dh == 64 || dh == 72; }

cudaError_t launch_attention_scores_tc(const AttnMaps& maps, const float* lse, float* partial, float* score, int n_cap,
                                       int L, int heads, int dh, const int* n_frames_dev, int* status_dev, cudaStream_t s) {
  if (n_cap <= 0) return cudaSuccess;
  ScoreArgs a{lse, partial, n_cap, L, heads, n_frames_dev, status_dev};
  cudaError_t e = dh == 72 ? run<72>(maps, a, s) : (dh == 64 ? run<64>(maps, a, s) : cudaErrorInvalidValue);
  if (e != cudaSuccess) return e;
  launch_score_finish(partial, score, n_cap, L, heads, n_frames_dev, s);
  return cudaGetLastError();
}

}  // namespace et
