// Dense layer on the 5th-generation tensor cores:  c = epi(a[M][K] * w[N][K]^T + bias[N]).
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0      TMA producer: 128 x 64 tile of a and BN x 64 tile of w per stage, 128-byte swizzle
//   warp 1      allocates TMEM, issues tcgen05.mma (128 x BN x 16, bf16 in, fp32 accumulate in TMEM),
//               releases smem stages and publishes accumulators through tcgen05.commit -> mbarrier
//   warps 2..5  epilogue: tcgen05.ld of the accumulator (each warp its own 32 TMEM lanes), bias,
//               GELU / residual / position-table add, stores.  Two TMEM accumulators ping-pong so the
//               epilogue of tile i overlaps the main loop of tile i+1.
// The live row count M comes from device memory (frames alive * rows per frame), so no host
// synchronisation is needed when Stage I changes the number of frames.
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA raises an abort flag, all
// roles leave their loops, in-flight copies are given time to land, TMEM is freed and the status word
// is set.
#include <cuda.h>

#include "common.cuh"
#include "rowops.cuh"

namespace et {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;                 // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr int EPI_WARP0 = 2;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s

template <int BN> struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : (BN == 192 ? 5 : 6);
  static constexpr int TMEM_COLS = (2 * BN <= 256) ? 256 : 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align slack*/ + 256 /*barriers*/;
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

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false if the limit ran out or another role aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  int spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 63) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// K-major operand tile written by TMA with 128-byte swizzle: rows of 128 bytes, groups of 8 rows
// 1024 bytes apart.  Fields: start address >> 4, leading byte offset (unused for swizzled K-major,
// set to 1), stride byte offset 1024 >> 4, descriptor version 1 (sm_100), layout 2 = SWIZZLE_128B.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gelu_epi(float x, int tanh_approx) {
  if (tanh_approx) return 0.5f * x * (1.f + tanh_fast(0.7978845608028654f * (x + 0.044715f * x * x * x)));
  return 0.5f * x * (1.f + erff(x * 0.7071067811865476f));
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int BN, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b, GemmArgs g) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // operand tiles need 1024-byte alignment
  uint8_t* const gen_base = smem_raw + (base - raw);
  uint8_t* const bar_mem = gen_base + C::STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = base + C::STAGES * C::STAGE_BYTES;
  // barrier slots (8 bytes each): full[S], empty[S], tmem_full[2], tmem_empty[2]; then tmem ptr, abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 2 + a); };
  volatile uint32_t* tmem_ptr_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + 8 * (2 * C::STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * C::STAGES + 4) + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int M = g.n_frames_dev ? min(g.M_cap, *g.n_frames_dev * g.rows_per_frame) : g.M_cap;
  const int tiles_m = (M + BM - 1) / BM;
  const int tiles_n = (g.N + BN - 1) / BN;
  const int total_tiles = tiles_m * tiles_n;
  const int num_kb = (g.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_ptr_slot)), "r"((uint32_t)C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_a) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_b) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / tiles_n) * BM, n0 = (tile % tiles_n) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          mbar_arrive_expect_tx(full_bar(stage), C::STAGE_BYTES);
          tma_load_2d(sa, &tma_a, full_bar(stage), kb * BK, m0);
          tma_load_2d(sb, &tma_b, full_bar(stage), kb * BK, n0);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: D fp32 (bit 4), A and B bf16 (bits 7, 10), both K-major, N >> 3 at 17, M >> 4 at 24
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advance 16 elements = 32 bytes along K inside the swizzle row: +2 in the (>>4) address field
            umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));           // frees the smem stage once these MMAs have read it
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));               // accumulator complete -> epilogue
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;                   // TMEM lanes this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile / tiles_n) * BM, n0 = (tile % tiles_n) * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const bool row_ok = row < M;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      const float* table_row = (EPI == EPI_TABLE && row_ok) ? g.table + (size_t)(row % g.table_rows) * g.N : nullptr;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        if (n0 + c0 >= g.N) break;                  // warp-uniform
        uint32_t r[32];
        tmem_ld32(t_row + (uint32_t)c0, r);
        if (!row_ok) continue;
#pragma unroll
        for (int q = 0; q < 4; ++q) {               // groups of 8 columns; N % 8 == 0
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
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // Give copies that are still in flight time to land before the shared memory is released.
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    if (threadIdx.x == 0 && g.status) atomicExch(g.status, (int)DS_WAIT_EXPIRED);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
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

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

template <int BN, int EPI>
cudaError_t launch_one(const TmaDesc& da, const TmaDesc& dw, const GemmArgs& g, cudaStream_t s) {
  using C = Cfg<BN>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_bf16_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int tiles = cdiv(g.M_cap, BM) * cdiv(g.N, BN);
  const int grid = min(tiles, sm_count());
  if (grid <= 0) return cudaSuccess;
  ET_COUNT_LAUNCH();
  gemm_bf16_kernel<BN, EPI><<<grid, NUM_THREADS, C::SMEM_BYTES, s>>>(
      *reinterpret_cast<const CUtensorMap*>(da.bytes), *reinterpret_cast<const CUtensorMap*>(dw.bytes), g);
  return cudaGetLastError();
}

template <int BN>
cudaError_t launch_bn(const TmaDesc& da, const TmaDesc& dw, const GemmArgs& g, int epilogue, cudaStream_t s) {
  switch (epilogue) {
    case EPI_STORE: return launch_one<BN, EPI_STORE>(da, dw, g, s);
    case EPI_GELU: return launch_one<BN, EPI_GELU>(da, dw, g, s);
    case EPI_RESIDUAL: return launch_one<BN, EPI_RESIDUAL>(da, dw, g, s);
    case EPI_TABLE: return launch_one<BN, EPI_TABLE>(da, dw, g, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

bool make_tma_2d_bf16(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                      const char** err) {
  static_assert(sizeof(CUtensorMap) <= sizeof(TmaDesc), "tensor map size");
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) { if (err) *err = "cuTensorMapEncodeTiled is not available from the driver"; return false; }
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((cols * 2) & 15u)) {
    if (err) *err = "tensor map needs a 16-byte aligned base and a row pitch that is a multiple of 16 bytes";
    return false;
  }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(reinterpret_cast<CUtensorMap*>(out->bytes), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                  dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (err) *err = "cuTensorMapEncodeTiled failed"; return false; }
  return true;
}

int gemm_bf16_pick_bn(int N) {
  if (N % 256 == 0) return 256;
  if (N % 192 == 0) return 192;
  if (N % 128 == 0) return 128;
  return 256;
}

cudaError_t launch_gemm_bf16(const TmaDesc& da, const TmaDesc& dw, const float* bias, void* c, int M_cap, int N, int K,
                             int epilogue, int gelu_tanh, const float* table, int table_rows, const int* n_frames_dev,
                             int rows_per_frame, int* status_dev, cudaStream_t s) {
  GemmArgs g;
  g.bias = bias; g.c = c; g.M_cap = M_cap; g.N = N; g.K = K; g.gelu_tanh = gelu_tanh;
  g.table = table; g.table_rows = table_rows > 0 ? table_rows : 1;
  g.n_frames_dev = n_frames_dev; g.rows_per_frame = rows_per_frame; g.status = status_dev;
  switch (gemm_bf16_pick_bn(N)) {
    case 256: return launch_bn<256>(da, dw, g, epilogue, s);
    case 192: return launch_bn<192>(da, dw, g, epilogue, s);
    default: return launch_bn<128>(da, dw, g, epilogue, s);
  }
}

}  // namespace et
