// Dense layer on the 5th-generation tensor cores:  c = epi(a[M][K] * w[N][K]^T + bias[N]).
//
// Persistent, warp-specialised kernel.  Two SMs work as a pair (thread-block cluster of 2, tcgen05
// cta_group::2): the pair owns a 256 x BN output tile, each CTA holds its own 128 rows of a and one
// half (BN/2 rows) of the w tile in shared memory, and the MMA of the pair reads both halves, so
// every CTA fetches (128 + BN/2) x 64 operand elements per k-block instead of (128 + BN) x 64.
//   warp 0      TMA producer: per stage a 128 x 64 tile of a and a BN/2 x 64 tile of w (128-byte
//               swizzle); completion is signalled on the leader CTA's "full" barrier
//   warp 1      allocates TMEM; in the leader CTA issues tcgen05.mma (256 x BN x 16 per instruction,
//               bf16 in, fp32 accumulate in the TMEM of both CTAs), releases the shared-memory stage
//               of both CTAs and publishes accumulators through tcgen05.commit -> mbarrier
//   warps 2..9  epilogue: tcgen05.ld of the accumulator (each warp its 32 TMEM lanes and half of the
//               columns), bias / GELU in registers, staged through swizzled shared memory and written
//               with TMA stores (bf16 outputs) or TMA reduce-adds (fp32 residual: x += result, the add
//               happens at the L2, nothing is read back).  Two TMEM accumulators ping-pong so the
//               epilogue of tile i overlaps the main loop of tile i+1.
// The live row count M comes from device memory (frames alive * rows per frame), so no host
// synchronisation is needed when Stage I changes the number of frames.  The last row tile, whose rows
// beyond M must not be written, and the position-table epilogue take a plain per-row store path.
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA raises an abort flag, all
// roles leave their loops, in-flight copies are given time to land, TMEM is freed and the status word
// is set.
#include <cuda.h>

#include "common.cuh"
#include "rowops.cuh"
#include "tcgen05.cuh"

namespace et {

namespace {

using namespace tc;

constexpr int BM = 128;                // rows per CTA
constexpr int BK = 64;                 // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int CG = 2;                  // CTAs per MMA (tcgen05 cta_group)
constexpr int NUM_EPI_WARPS = 8;
constexpr int NUM_THREADS = 64 + 32 * NUM_EPI_WARPS;
constexpr int SLAB_BYTES = 4096;       // per epilogue warp: 32 rows x 128 bytes
constexpr int SMEM_LIMIT = 232448;     // 227 KB opt-in maximum per CTA

template <int BN> struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_ROWS = BN / CG;
  static constexpr int B_BYTES = B_ROWS * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int EPI_BYTES = NUM_EPI_WARPS * SLAB_BYTES;
  static constexpr int BAR_BYTES = 256;
  static constexpr int FIT = (SMEM_LIMIT - 1024 - BAR_BYTES - EPI_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = FIT > 8 ? 8 : FIT;
  static constexpr int TMEM_COLS = (2 * BN <= 256) ? 256 : 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*align slack*/ + BAR_BYTES;
  static_assert(STAGES >= 3, "too few pipeline stages");
  static_assert((2 * STAGES + 4) * 8 + 8 <= BAR_BYTES, "barrier area");
  static_assert(STAGE_BYTES % 1024 == 0, "operand tiles need 1024-byte alignment");
  static_assert(BN % 64 == 0 && BN <= 256, "tile width");
};

struct GemmArgs {
  const float* bias;
  void* c;
  int M_cap, N, K;
  int gelu_tanh;
  const float* table;
  int table_rows;
  const int* n_frames_dev;
  int rows_per_frame;
  int* status;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// arrive on a barrier given by its shared::cluster address (this CTA's or the peer's)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// Tile load into this CTA's shared memory; the completion bytes are counted on `bar`, which may be
// a barrier of the peer CTA of the pair (shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }


__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// The barrier at the same shared-memory offset in both CTAs of the pair receives one arrival once all
// MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}

// K-major operand tile written by TMA with 128-byte swizzle: rows of 128 bytes, groups of 8 rows
// 1024 bytes apart.  Fields: start address >> 4, leading byte offset (unused for swizzled K-major,
// set to 1), stride byte offset 1024 >> 4, descriptor version 1 (sm_100), layout 2 = SWIZZLE_128B.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))) in five FP32 operations and one MUFU
__device__ __forceinline__ float gelu_tanh_fast(float x) {
  const float c = 0.7978845608028654f;
  const float inner = x * fmaf(x * x, 0.044715f * c, c);
  const float hx = 0.5f * x;
  return fmaf(hx, tanh_fast(inner), hx);
}
// The same on two elements with packed instructions (identical operations per element, hence identical bits).
__device__ __forceinline__ void gelu_tanh_fast2(float& x0, float& x1) {
  const float c = 0.7978845608028654f, k = 0.044715f * c;
  float u0, u1, t0, t1, i0, i1, h0, h1;
  mul2(u0, u1, x0, x1, x0, x1);
  fma2(t0, t1, u0, u1, k, k, c, c);
  mul2(i0, i1, x0, x1, t0, t1);
  mul2(h0, h1, x0, x1, 0.5f, 0.5f);
  fma2(x0, x1, h0, h1, tanh_fast(i0), tanh_fast(i1), h0, h1);
}
// Both store paths of the epilogue go through this function, so a row gets the same bits whichever path writes it.
__device__ __forceinline__ float gelu_epi(float x, int tanh_approx) {
  if (tanh_approx) return gelu_tanh_fast(x);
  return 0.5f * x * (1.f + erff(x * 0.7071067811865476f));
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int BN, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b,
                 const __grid_constant__ CUtensorMap tma_bh,
                 const __grid_constant__ CUtensorMap tma_c, GemmArgs g) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // operand tiles need 1024-byte alignment
  uint8_t* const gen_base = smem_raw + (base - raw);
  const uint32_t epi_base = base + C::STAGES * C::STAGE_BYTES;
  uint8_t* const bar_mem = gen_base + C::STAGES * C::STAGE_BYTES + C::EPI_BYTES;
  const uint32_t bar_base = epi_base + C::EPI_BYTES;
  // barrier slots (8 bytes each): full[S], empty[S], tmem_full[2], tmem_empty[2]; then tmem ptr, abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 2 + a); };
  volatile uint32_t* tmem_ptr_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + 8 * (2 * C::STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * C::STAGES + 4) + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                      // 0 = leader of the pair
  const int pair = blockIdx.x / CG, n_pairs = gridDim.x / CG;
  const int M = g.n_frames_dev ? min(g.M_cap, *g.n_frames_dev * g.rows_per_frame) : g.M_cap;
  const int tiles_m = (M + BM * CG - 1) / (BM * CG);
  const int tiles_n = (g.N + BN - 1) / BN;
  const int total_tiles = tiles_m * tiles_n;
  const int num_kb = (g.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), CG * NUM_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_ptr_slot)), "r"((uint32_t)C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  cluster_sync_all();                 // the peer's barriers are initialised before anything arrives on them
  fence_after();
  const uint32_t tmem_base = *tmem_ptr_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_a) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_b) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_bh) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        const int m0 = (tile / tiles_n) * (BM * CG) + (int)rank * BM;
        // A last column tile of at most 128 valid columns is multiplied at that width: each CTA then holds 64 weight
        // rows, fetched through the 64-row box.
        const int nt0 = (tile % tiles_n) * BN;
        const bool narrow = BN == 256 && g.N - nt0 <= 128;
        const int n0 = nt0 + (int)rank * (narrow ? 64 : C::B_ROWS);
        const uint32_t stage_tx = narrow ? (uint32_t)(C::A_BYTES + 64 * BK * 2) : (uint32_t)C::STAGE_BYTES;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          const uint32_t full_leader = map_to_cta(full_bar(stage), 0);
          // the leader's barrier counts the bytes of both CTAs' tiles of this stage
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), CG * stage_tx);
          tma_load_2d_pair(sa, &tma_a, full_leader, kb * BK, m0);
          tma_load_2d_pair(sb, narrow ? &tma_bh : &tma_b, full_leader, kb * BK, n0);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      // instruction descriptor: D fp32 (bit 4), A and B bf16 (bits 7, 10), both K-major, N >> 3 at 17, M >> 4 at 24
      const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((BM * CG) >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        const bool narrow = BN == 256 && g.N - (tile % tiles_n) * BN <= 128;
        const uint32_t idesc = idesc0 | ((uint32_t)((narrow ? 128 : BN) >> 3) << 17);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          fence_after();
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advance 16 elements = 32 bytes along K inside the swizzle row: +2 in the (>>4) address field
            umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(stage));      // frees this stage in both CTAs once the MMAs have read it
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(tfull_bar(acc));          // accumulator complete -> epilogues of both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    const int e = warp - 2;
    const int quarter = warp & 3;                   // TMEM lanes this warp may read: 32*quarter ..
    const int half = e >> 2;                        // which half of the tile's 32-column chunks
    constexpr int CHUNKS = BN / 32, CH_PER = CHUNKS / 2;
    const uint32_t slab = epi_base + (uint32_t)e * SLAB_BYTES;
    const uint32_t tempty_leader0 = map_to_cta(tempty_bar(0), 0), tempty_leader1 = map_to_cta(tempty_bar(1), 0);
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t sub = 0;                               // bf16 outputs alternate between the two 2 KB halves of the slab
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
      const int m0 = (tile / tiles_n) * (BM * CG) + (int)rank * BM, n0 = (tile % tiles_n) * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      const bool staged = (EPI != EPI_TABLE) && (m0 + BM <= M);
      if (m0 < M) {
        if (staged) {
          // ---- full row tile: registers -> swizzled slab -> TMA store / reduce-add
          // The accumulator chunk after the current one is requested before the current one is processed,
          // and the bias loads of a chunk are issued while its TMEM load is in flight.
          uint32_t rr[2][32];
          const int c_first = half * CH_PER * 32;
          if (n0 + c_first < g.N) tmem_ld32_async(t_row + (uint32_t)c_first, rr[0]);
          if constexpr (EPI == EPI_SWIGLU) {
            // Chunks come in pairs (gate, up) of the same 32 outputs (the weight rows were interleaved that way):
            // h = silu(gate + b) * (up + b), half as many output columns as accumulator columns; the bias is in
            // weight-row order.
            float gate[32];
#pragma unroll
            for (int ch = 0; ch < CH_PER; ++ch) {
              const int c0 = (half * CH_PER + ch) * 32;
              tmem_wait_ld();
              tmem_regs_ready(rr[ch & 1]);
              if (ch + 1 < CH_PER) tmem_ld32_async(t_row + (uint32_t)(c0 + 32), rr[(ch + 1) & 1]);
              const uint32_t (&r)[32] = rr[ch & 1];
              float4 b[8];                              // bias of this chunk (weight-row order; zeros where a layer has none)
#pragma unroll
              for (int q = 0; q < 8; ++q) b[q] = __ldg(reinterpret_cast<const float4*>(g.bias + n0 + c0 + q * 4));
              const float* bf = reinterpret_cast<const float*>(b);
              if ((ch & 1) == 0) {
#pragma unroll
                for (int i = 0; i < 32; ++i) gate[i] = __uint_as_float(r[i]) + bf[i];
              } else {
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __fdividef(gate[i], 1.f + __expf(-gate[i])) * (__uint_as_float(r[i]) + bf[i]);
                if (lane == 0) bulk_wait_read<1>();   // the half written two stores ago has been read
                __syncwarp();
                const uint32_t buf = slab + sub * 2048u;
                const uint32_t rowp = buf + (uint32_t)lane * 64u;
                const uint32_t sw = (uint32_t)(lane >> 1) & 3u;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  st_shared_v4(rowp + ((((uint32_t)j) ^ sw) << 4), pack_bf16(v[j * 8 + 0], v[j * 8 + 1]), pack_bf16(v[j * 8 + 2], v[j * 8 + 3]),
                               pack_bf16(v[j * 8 + 4], v[j * 8 + 5]), pack_bf16(v[j * 8 + 6], v[j * 8 + 7]));
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { tma_store_2d(&tma_c, buf, (n0 + c0 - 32) >> 1, m0 + quarter * 32); bulk_commit(); }
                sub ^= 1u;
              }
            }
          } else {
#pragma unroll
          for (int ch = 0; ch < CH_PER; ++ch) {
            const int c0 = (half * CH_PER + ch) * 32;
            const int col0 = n0 + c0;
            if (col0 >= g.N) continue;              // warp-uniform (columns beyond N: nothing was requested either)
            float4 b[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const int col = col0 + q * 4;
              b[q] = (col < g.N) ? __ldg(reinterpret_cast<const float4*>(g.bias + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            tmem_wait_ld();
            tmem_regs_ready(rr[ch & 1]);
            if (ch + 1 < CH_PER && col0 + 32 < g.N) tmem_ld32_async(t_row + (uint32_t)(c0 + 32), rr[(ch + 1) & 1]);
            const uint32_t (&r)[32] = rr[ch & 1];
            float v[32];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              add2(v[q * 4 + 0], v[q * 4 + 1], __uint_as_float(r[q * 4 + 0]), __uint_as_float(r[q * 4 + 1]), b[q].x, b[q].y);
              add2(v[q * 4 + 2], v[q * 4 + 3], __uint_as_float(r[q * 4 + 2]), __uint_as_float(r[q * 4 + 3]), b[q].z, b[q].w);
            }
            if (EPI == EPI_GELU) {
              if (g.gelu_tanh) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) gelu_tanh_fast2(v[i], v[i + 1]);
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = gelu_epi(v[i], 0);
              }
            }
            if (EPI == EPI_STORE || EPI == EPI_GELU) {
              // bf16: 32 rows x 64 bytes, 64-byte swizzle: 16-byte chunk j of row r sits at j ^ ((r >> 1) & 3)
              if (lane == 0) bulk_wait_read<1>();   // the half written two chunks ago has been read
              __syncwarp();
              const uint32_t buf = slab + sub * 2048u;
              const uint32_t rowp = buf + (uint32_t)lane * 64u;
              const uint32_t sw = (uint32_t)(lane >> 1) & 3u;
#pragma unroll
              for (int j = 0; j < 4; ++j)
                st_shared_v4(rowp + ((((uint32_t)j) ^ sw) << 4), pack_bf16(v[j * 8 + 0], v[j * 8 + 1]), pack_bf16(v[j * 8 + 2], v[j * 8 + 3]),
                             pack_bf16(v[j * 8 + 4], v[j * 8 + 5]), pack_bf16(v[j * 8 + 6], v[j * 8 + 7]));
              fence_async_smem();
              __syncwarp();
              if (lane == 0) { tma_store_2d(&tma_c, buf, col0, m0 + quarter * 32); bulk_commit(); }
              sub ^= 1u;
            } else {
              // fp32: 32 rows x 128 bytes, 128-byte swizzle: chunk j of row r sits at j ^ (r & 7)
              if (lane == 0) bulk_wait_read<0>();
              __syncwarp();
              const uint32_t rowp = slab + (uint32_t)lane * 128u;
              const uint32_t sw = (uint32_t)lane & 7u;
#pragma unroll
              for (int j = 0; j < 8; ++j)
                st_shared_v4(rowp + ((((uint32_t)j) ^ sw) << 4), __float_as_uint(v[j * 4 + 0]), __float_as_uint(v[j * 4 + 1]),
                             __float_as_uint(v[j * 4 + 2]), __float_as_uint(v[j * 4 + 3]));
              fence_async_smem();
              __syncwarp();
              if (lane == 0) { tma_reduce_add_2d(&tma_c, slab, col0, m0 + quarter * 32); bulk_commit(); }
            }
          }
          }
        } else if constexpr (EPI == EPI_SWIGLU) {
          // ---- last row tile of the gated layer: per-row stores of silu(gate) * up, rows >= M untouched
          const int row = m0 + quarter * 32 + lane;
          const bool row_ok = row < M;
#pragma unroll 1
          for (int pr = 0; pr < CH_PER / 2; ++pr) {
            const int c0 = (half * CH_PER + 2 * pr) * 32;
            uint32_t rg[32], ru[32];
            tmem_ld32(t_row + (uint32_t)c0, rg);
            tmem_ld32(t_row + (uint32_t)(c0 + 32), ru);
            if (!row_ok) continue;
            bf16* dst = reinterpret_cast<bf16*>(g.c) + (size_t)row * (size_t)(g.N >> 1) + ((n0 + c0) >> 1);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float gt = __uint_as_float(rg[q * 8 + i]) + __ldg(g.bias + n0 + c0 + q * 8 + i);
                v[i] = __fdividef(gt, 1.f + __expf(-gt)) * (__uint_as_float(ru[q * 8 + i]) + __ldg(g.bias + n0 + c0 + 32 + q * 8 + i));
              }
              uint4 o;
              o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]);
              o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
              *reinterpret_cast<uint4*>(dst + q * 8) = o;
            }
          }
        } else {
          // ---- last row tile / position-table epilogue: per-row stores, rows >= M untouched
          const int row = m0 + quarter * 32 + lane;
          const bool row_ok = row < M;
          const float* table_row = (EPI == EPI_TABLE && row_ok) ? g.table + (size_t)(row % g.table_rows) * g.N : nullptr;
#pragma unroll 1
          for (int ch = 0; ch < CH_PER; ++ch) {
            const int c0 = (half * CH_PER + ch) * 32;
            if (n0 + c0 >= g.N) break;              // warp-uniform
            uint32_t r[32];
            tmem_ld32(t_row + (uint32_t)c0, r);
            if (!row_ok) continue;
#pragma unroll
            for (int q = 0; q < 4; ++q) {           // groups of 8 columns; N % 8 == 0
              const int col = n0 + c0 + q * 8;
              if (col >= g.N) break;
              float v[8];
              const float4 b0 = __ldg(reinterpret_cast<const float4*>(g.bias + col));
              const float4 b1 = __ldg(reinterpret_cast<const float4*>(g.bias + col + 4));
              v[0] = __uint_as_float(r[q * 8 + 0]) + b0.x; v[1] = __uint_as_float(r[q * 8 + 1]) + b0.y;
              v[2] = __uint_as_float(r[q * 8 + 2]) + b0.z; v[3] = __uint_as_float(r[q * 8 + 3]) + b0.w;
              v[4] = __uint_as_float(r[q * 8 + 4]) + b1.x; v[5] = __uint_as_float(r[q * 8 + 5]) + b1.y;
              v[6] = __uint_as_float(r[q * 8 + 6]) + b1.z; v[7] = __uint_as_float(r[q * 8 + 7]) + b1.w;
              if (EPI == EPI_STORE || EPI == EPI_GELU) {
                if (EPI == EPI_GELU) {
#pragma unroll
                  for (int i = 0; i < 8; ++i) v[i] = gelu_epi(v[i], g.gelu_tanh);
                }
                uint4 o;
                o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]);
                o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
                *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(g.c) + (size_t)row * g.N + col) = o;
              } else {
                float* dst = reinterpret_cast<float*>(g.c) + (size_t)row * g.N + col;
                float4 x0, x1;
                if (EPI == EPI_RESIDUAL) {
                  x0 = *reinterpret_cast<const float4*>(dst);
                  x1 = *reinterpret_cast<const float4*>(dst + 4);
                } else {
                  x0 = __ldg(reinterpret_cast<const float4*>(table_row + col));
                  x1 = __ldg(reinterpret_cast<const float4*>(table_row + col + 4));
                }
                *reinterpret_cast<float4*>(dst) = make_float4(v[0] + x0.x, v[1] + x0.y, v[2] + x0.z, v[3] + x0.w);
                *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4] + x1.x, v[5] + x1.y, v[6] + x1.z, v[7] + x1.w);
              }
            }
          }
        }
      }
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc == 0 ? tempty_leader0 : tempty_leader1);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();                 // the slab stays alive until its last store has been read
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  fence_before();
  __syncthreads();
  if (*abort_flag) {
    // Give copies that are still in flight time to land before the shared memory is released.
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    if (threadIdx.x == 0 && g.status) atomicExch(g.status, (int)DS_WAIT_EXPIRED);
    __syncthreads();
  }
  cluster_sync_all();                 // nothing of the pair is in flight towards this CTA any more
  if (warp == 1) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

template <int BN, int EPI>
cudaError_t launch_one(const TmaDesc& da, const WeightDesc& dw, const TmaDesc& dc, const GemmArgs& g, cudaStream_t s) {
  using C = Cfg<BN>;
  static int max_pairs = 0;           // CTA pairs that can be resident at once (one CTA per SM)
  if (max_pairs == 0) {
    cudaError_t e = cudaFuncSetAttribute(gemm_bf16_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t probe{};
    probe.gridDim = dim3(CG, 1, 1);
    probe.blockDim = dim3(NUM_THREADS, 1, 1);
    probe.dynamicSmemBytes = C::SMEM_BYTES;
    cudaLaunchAttribute pa[1];
    pa[0].id = cudaLaunchAttributeClusterDimension;
    pa[0].val.clusterDim.x = CG; pa[0].val.clusterDim.y = 1; pa[0].val.clusterDim.z = 1;
    probe.attrs = pa; probe.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, gemm_bf16_kernel<BN, EPI>, &probe);
    if (e != cudaSuccess) return e;
    if (n < 1) return cudaErrorLaunchOutOfResources;
    max_pairs = n;
  }
  const int tiles = cdiv(g.M_cap, BM * CG) * cdiv(g.N, BN);
  const int pairs = min(tiles, max_pairs);
  if (pairs <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(pairs * CG, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  ET_COUNT_LAUNCH();
  return cudaLaunchKernelEx(&cfg, gemm_bf16_kernel<BN, EPI>, *reinterpret_cast<const CUtensorMap*>(da.bytes),
                            *reinterpret_cast<const CUtensorMap*>(dw.full.bytes), *reinterpret_cast<const CUtensorMap*>(dw.half.bytes),
                            *reinterpret_cast<const CUtensorMap*>(dc.bytes), g);
}

template <int BN>
cudaError_t launch_bn(const TmaDesc& da, const WeightDesc& dw, const TmaDesc& dc, const GemmArgs& g, int epilogue, cudaStream_t s) {
  switch (epilogue) {
    case EPI_STORE: return launch_one<BN, EPI_STORE>(da, dw, dc, g, s);
    case EPI_GELU: return launch_one<BN, EPI_GELU>(da, dw, dc, g, s);
    case EPI_RESIDUAL: return launch_one<BN, EPI_RESIDUAL>(da, dw, dc, g, s);
    case EPI_TABLE: return launch_one<BN, EPI_TABLE>(da, dw, dc, g, s);
    case EPI_SWIGLU:
      // gate / up pairs are 32-column chunks of full 256-wide tiles
      if constexpr (BN == 256) { if (g.N % 256 == 0) return launch_one<BN, EPI_SWIGLU>(da, dw, dc, g, s); }
      return cudaErrorInvalidValue;
  }
  return cudaErrorInvalidValue;
}

bool encode_2d(TmaDesc* out, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t rows, uint64_t cols,
               uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle sw, const char** err) {
  static_assert(sizeof(CUtensorMap) <= sizeof(TmaDesc), "tensor map size");
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn) { if (err) *err = "cuTensorMapEncodeTiled is not available from the driver"; return false; }
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((cols * elem_bytes) & 15u)) {
    if (err) *err = "tensor map needs a 16-byte aligned base and a row pitch that is a multiple of 16 bytes";
    return false;
  }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * (cuuint64_t)elem_bytes};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(reinterpret_cast<CUtensorMap*>(out->bytes), dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (err) *err = "cuTensorMapEncodeTiled failed"; return false; }
  return true;
}

}  // namespace

namespace tc {
EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}
}  // namespace tc

bool make_tma_2d_bf16(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                      const char** err) {
  return encode_2d(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, rows, cols, BK, box_rows, CU_TENSOR_MAP_SWIZZLE_128B, err);
}

bool make_tma_weight(WeightDesc* out, const void* base, uint64_t n_rows, uint64_t k_cols, const char** err) {
  return make_tma_2d_bf16(&out->full, base, n_rows, k_cols, (uint32_t)gemm_bf16_w_box_rows((int)n_rows), err) &&
         make_tma_2d_bf16(&out->half, base, n_rows, k_cols, 64, err);
}

bool make_tma_out(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, bool fp32, const char** err) {
  if (fp32) return encode_2d(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, rows, cols, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B, err);
  return encode_2d(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, rows, cols, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B, err);
}

// Tile width.  256 columns per CTA pair keeps the operand traffic per FLOP lowest (each CTA fetches 128 rows of a
// and 128 rows of w per k-block) and the MMA at its widest; measured on B200 it beats 192-wide tiles even where
// 192 divides N and 256 does not (N = 1152, 3456: the clipped last tile costs less than the narrower MMA).
int gemm_bf16_pick_bn(int N) {
  return N <= 128 ? 128 : 256;
}

int gemm_bf16_w_box_rows(int N) { return gemm_bf16_pick_bn(N) / CG; }

cudaError_t launch_gemm_bf16(const TmaDesc& da, const WeightDesc& dw, const TmaDesc& dc, const float* bias, void* c, int M_cap,
                             int N, int K, int epilogue, int gelu_tanh, const float* table, int table_rows,
                             const int* n_frames_dev, int rows_per_frame, int* status_dev, cudaStream_t s) {
  GemmArgs g;
  g.bias = bias; g.c = c; g.M_cap = M_cap; g.N = N; g.K = K; g.gelu_tanh = gelu_tanh;
  g.table = table; g.table_rows = table_rows > 0 ? table_rows : 1;
  g.n_frames_dev = n_frames_dev; g.rows_per_frame = rows_per_frame; g.status = status_dev;
  switch (gemm_bf16_pick_bn(N)) {
    case 256: return launch_bn<256>(da, dw, dc, g, epilogue, s);
    default: return launch_bn<128>(da, dw, dc, g, epilogue, s);
  }
}

}  // namespace et
