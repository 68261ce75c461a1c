// Causal grouped-query attention with head dim 128 on tcgen05 (the language model's prefill).
//
// Same organisation as the per-frame encoder attention (attention_tcgen05.cu): a persistent CTA per SM,
// work items of 256 queries of one (sequence, head), two softmax warpgroups (thread = query row = TMEM
// lane) that alternate on the tensor pipe, P written back into TMEM over S, O accumulated in TMEM.
// What differs:
//   * head dim 128 = two 128-byte swizzled 64-column boxes for Q, K and V; S = Q K^T takes 8 k-steps,
//     O += P V is one N = 128 MMA per 16 keys; TMEM holds S0 S1 O0 O1 = 4 x 128 columns exactly;
//   * query i sees keys 0..i: an item sweeps only the key tiles up to its diagonal, the number of valid
//     keys of a tile is a per-row quantity, and items are dealt longest first in alternating direction;
//   * several query heads share one key / value head; Q, K and V live in one packed row
//     [heads*128 | kv_heads*128 | kv_heads*128] and the row index is the position.
#include "common.cuh"
#include "softmax_tile.cuh"
#include "tcgen05.cuh"

namespace et {

namespace {

using namespace tc;

constexpr int DH = 128;
constexpr int QT = 128;                 // queries per softmax group
constexpr int QB = 2 * QT;              // queries per CTA
constexpr int KT = 128;                 // keys per tile
constexpr int KV_STAGES = 2;
constexpr int ATOM_BYTES = 128 * 128;   // 128 rows x 64 bf16, 128-byte swizzle
constexpr int TILE_BYTES = 2 * ATOM_BYTES;   // 128 rows x 128 bf16: columns 0..63, then 64..127
constexpr int ATT_THREADS = 384;        // warps 0..7 softmax, 8 TMA, 9 MMA, 10..11 idle (complete the third warpgroup)
constexpr int SOFTMAX_REGS = 200, CONTROL_REGS = 80;
// (nothing checks that a role's code fits its budget -- a path that needs more computes garbage silently; the
// parity tests validate these numbers)
// setmaxnreg.inc blocks until the registers exist: the budgets must fit into what the CTA was launched with
constexpr int LAUNCH_REGS = 160;
static_assert(SOFTMAX_REGS * 256 + CONTROL_REGS * 128 <= LAUNCH_REGS * ATT_THREADS, "register budgets exceed the CTA's allocation");
constexpr float LOG2E = 1.4426950408889634f;
constexpr float RESCALE_GAP = 8.f;

constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;
constexpr int OFF_V = OFF_K + KV_STAGES * TILE_BYTES;
constexpr int OFF_BARS = OFF_V + KV_STAGES * TILE_BYTES;
constexpr int SMEM_BYTES = OFF_BARS + 256 + 1024;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");

constexpr int B_Q_FULL = 0, B_K_FULL = 1, B_V_FULL = B_K_FULL + KV_STAGES, B_KV_EMPTY = B_V_FULL + KV_STAGES,
              B_S_FULL = B_KV_EMPTY + KV_STAGES, B_P_FULL = B_S_FULL + 2, B_O_READY = B_P_FULL + 2, B_Q_EMPTY = B_O_READY + 2,
              B_COUNT = B_Q_EMPTY + 1;
static_assert(B_COUNT * 8 + 8 <= 256, "barrier area");

constexpr int TMEM_COLS = 512;
constexpr int COL_O = 256;

struct CausalArgs {
  bf16* out;             // [n_seq * L][heads * 128]
  int n_seq, L, heads, group;   // group = query heads per key / value head
  int* status;
};

__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_causal_kernel(const __grid_constant__ CUtensorMap tma_qkv, CausalArgs g) {
  const int L = g.L;
  const int q_dim = g.heads * DH, kv_dim = (g.heads / g.group) * DH;
  const int tiles_all = (L + KT - 1) / KT;
  const int q_blocks = (L + QB - 1) / QB;
  const int n_items = g.n_seq * g.heads * q_blocks;
  // Items are numbered in order of decreasing length (the last query block first, heads and sequences fastest) and
  // dealt to the CTAs in rounds that alternate direction (0..G-1, then G-1..0, ...): every CTA then sweeps nearly the
  // same number of key tiles, where plain round-robin gives the first CTAs 15 % more than the average.
  const int G = (int)gridDim.x, rounds = (n_items + G - 1) / G;
  auto item_index = [&](int i) { return i * G + ((i & 1) ? G - 1 - (int)blockIdx.x : (int)blockIdx.x); };
  const int my_items = rounds == 0 ? 0 : rounds - 1 + (item_index(rounds - 1) < n_items ? 1 : 0);
  if (my_items == 0) return;
  auto item_coords = [&](int i, int& f, int& h, int& q0) {
    const int item = item_index(i);
    const int hs = g.heads * g.n_seq;
    q0 = (q_blocks - 1 - item / hs) * QB;
    h = (item % hs) % g.heads;
    f = (item % hs) / g.heads;
  };
  auto item_tiles = [&](int q0) { return min(tiles_all, q0 / KT + 2); };    // key tiles up to the diagonal of the block
  auto keys_rounded = [&](int j) { return (min(KT, L - j * KT) + 15) & ~15; };

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
    mbar_init(bar(B_Q_FULL), 1);
    mbar_init(bar(B_Q_EMPTY), 1);
    for (int s = 0; s < KV_STAGES; ++s) { mbar_init(bar(B_K_FULL + s), 1); mbar_init(bar(B_V_FULL + s), 1); mbar_init(bar(B_KV_EMPTY + s), 1); }
    for (int t = 0; t < 2; ++t) { mbar_init(bar(B_S_FULL + t), 1); mbar_init(bar(B_P_FULL + t), 4); mbar_init(bar(B_O_READY + t), 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_ptr_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem_base = *tmem_ptr_slot;

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CONTROL_REGS));
    if (warp == 8) {
      // ---------------------------------------------------------------- TMA producer
      if (lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_qkv) : "memory");
        bool ok = true;
        int gt = 0;                                      // key tiles loaded so far: ring stage and phase
        for (int i = 0; i < my_items && ok; ++i) {
          int f, h, q0;
          item_coords(i, f, h, q0);
          const int row_base = f * L, kvh = h / g.group;
          // Q of the previous item is free once its last Q K^T has completed
          if (i > 0 && !mbar_wait(bar(B_Q_EMPTY), (uint32_t)(i - 1) & 1u, abort_flag)) break;
          mbar_arrive_expect_tx(bar(B_Q_FULL), 2 * TILE_BYTES);
          for (int t = 0; t < 2; ++t)
            for (int c = 0; c < 2; ++c)
              tma_load_2d(base + OFF_Q + t * TILE_BYTES + c * ATOM_BYTES, &tma_qkv, bar(B_Q_FULL), h * DH + c * 64, row_base + q0 + t * QT);
          const int nt = item_tiles(q0);
          for (int j = 0; j < nt; ++j, ++gt) {
            const int s = gt % KV_STAGES;
            const uint32_t ph = (uint32_t)(gt / KV_STAGES) & 1u;
            if (!mbar_wait(bar(B_KV_EMPTY + s), ph ^ 1u, abort_flag)) { ok = false; break; }
            const int y = row_base + j * KT;
            mbar_arrive_expect_tx(bar(B_K_FULL + s), TILE_BYTES);
            for (int c = 0; c < 2; ++c)
              tma_load_2d(base + OFF_K + s * TILE_BYTES + c * ATOM_BYTES, &tma_qkv, bar(B_K_FULL + s), q_dim + kvh * DH + c * 64, y);
            mbar_arrive_expect_tx(bar(B_V_FULL + s), TILE_BYTES);
            for (int c = 0; c < 2; ++c)
              tma_load_2d(base + OFF_V + s * TILE_BYTES + c * ATOM_BYTES, &tma_qkv, bar(B_V_FULL + s), q_dim + kv_dim + kvh * DH + c * 64, y);
          }
        }
      }
    } else if (warp == 9) {
      // ---------------------------------------------------------------- MMA issuer
      // The whole warp runs the loop; one elected lane issues the MMAs and the commits.
      constexpr uint32_t IDESC_PV = idesc_bf16(128, DH, false, true);
      // Q / K: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart; the second 64 elements of the head
      // are a second box ATOM_BYTES further.  V: MN-major with 128-byte swizzle, 64 columns per atom, the
      // second atom ATOM_BYTES further (leading byte offset), 8-key groups 1024 bytes apart.
      const uint64_t q0d = smem_desc(base + OFF_Q, 16, 1024, 2), k0d = smem_desc(base + OFF_K, 16, 1024, 2),
                     v0d = smem_desc(base + OFF_V, ATOM_BYTES, 1024, 2);
      constexpr uint64_t TILE_STEP = TILE_BYTES >> 4, ATOM_STEP = ATOM_BYTES >> 4;
      bool ok = true;
      // O += P V of the key tile with running number gp (ring stage sp), jj its index inside its item
      auto pv = [&](int t, int gp, int jj) -> bool {
        const int sp = gp % KV_STAGES;
        if (t == 0 && !mbar_wait_warp(bar(B_V_FULL + sp), (uint32_t)(gp / KV_STAGES) & 1u, abort_flag)) return false;
        if (!mbar_wait_warp(bar(B_P_FULL + t), (uint32_t)gp & 1u, abort_flag)) return false;
        fence_after();
        const int ksteps = keys_rounded(jj) / 16;
        const uint32_t o_col = tmem_base + COL_O + t * DH;
        uint32_t a = tmem_base + t * 128;                     // 16 keys = 8 columns of packed bf16 pairs
        uint64_t dv = v0d + (uint64_t)sp * TILE_STEP;
#pragma unroll 1
        for (int ks = 0; ks < ksteps; ++ks) {
          mma_ts_elect(o_col, a, dv, IDESC_PV, (jj | ks) != 0 ? 1u : 0u);     // the first tile of an item overwrites O
          a += 8; dv += 2048 >> 4;                             // 16 keys = two 8-row groups; 16-byte units
        }
        commit_elect(bar(B_O_READY + t));
        if (t == 1) commit_elect(bar(B_KV_EMPTY + sp));        // K and V of that tile are no longer needed
        return true;
      };
      int gt = 0, prev_j = 0;
      for (int i = 0; i < my_items && ok; ++i) {
        int f, h, q0;
        item_coords(i, f, h, q0);
        const int nt = item_tiles(q0);
        for (int j = 0; j < nt && ok; ++j, ++gt) {
          const int s = gt % KV_STAGES;
          for (int t = 0; t < 2 && ok; ++t) {
            if (gt > 0 && !pv(t, gt - 1, prev_j)) { ok = false; break; }
            if (t == 0) {      // operands of this tile (waited for only now: the P V above must not wait for the next item's Q)
              if (j == 0 && !mbar_wait_warp(bar(B_Q_FULL), (uint32_t)i & 1u, abort_flag)) { ok = false; break; }
              if (!mbar_wait_warp(bar(B_K_FULL + s), (uint32_t)(gt / KV_STAGES) & 1u, abort_flag)) { ok = false; break; }
              fence_after();
            }
            const uint32_t idesc = idesc_bf16(128, keys_rounded(j), false, false);
            const uint64_t qd = q0d + (uint64_t)t * TILE_STEP, kd = k0d + (uint64_t)s * TILE_STEP;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {                    // 16 elements = 32 bytes inside the swizzle row
              const uint64_t off = (uint64_t)(ks >> 2) * ATOM_STEP + 2 * (ks & 3);
              mma_ss_elect(tmem_base + t * 128, qd + off, kd + off, idesc, ks != 0 ? 1u : 0u);
            }
            commit_elect(bar(B_S_FULL + t));
            if (t == 1 && j == nt - 1) commit_elect(bar(B_Q_EMPTY));   // the item's last read of Q
          }
          prev_j = j;
        }
      }
      for (int t = 0; t < 2 && ok; ++t)
        if (!pv(t, gt - 1, prev_j)) ok = false;
    }
  } else {
    // ------------------------------------------------------------------ softmax groups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(SOFTMAX_REGS));
    const int t = warp >> 2;
    const int quarter = warp & 3;                     // TMEM lanes 32*quarter .. +31
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_addr + t * 128, o_addr = lane_addr + COL_O + t * DH;
    const float scale2 = LOG2E / sqrtf((float)DH);    // logits are kept in the log2 domain
    bool ok = true;
    int gt = 0;                                       // key tiles processed so far (barrier phases)
    for (int i = 0; i < my_items && ok; ++i) {
      int f, h, q0;
      item_coords(i, f, h, q0);
      const int row_base = f * L, q = q0 + t * QT + row;
      const int nt = item_tiles(q0);
      float m = -INFINITY, l = 0.f;
      for (int j = 0; j < nt; ++j, ++gt) {
        const int nk_tile = min(KT, L - j * KT);
        const int nch = (nk_tile + 31) >> 5;
        const int nk = max(0, min(nk_tile, q - j * KT + 1));      // keys of this tile that query q sees
        if (!mbar_wait_warp(bar(B_S_FULL + t), (uint32_t)gt & 1u, abort_flag)) { ok = false; break; }
        fence_after();
        uint32_t r0[32], r1[32], r2[32], r3[32];
        tmem_ld32_async(s_addr, r0);
        if (nch > 1) tmem_ld32_async(s_addr + 32, r1);
        if (nch > 2) tmem_ld32_async(s_addr + 64, r2);
        if (nch > 3) tmem_ld32_async(s_addr + 96, r3);
        tmem_wait_ld();
        tmem_regs_ready(r0);
        if (nch > 1) tmem_regs_ready(r1);
        if (nch > 2) tmem_regs_ready(r2);
        if (nch > 3) tmem_regs_ready(r3);
        const bool full = __all_sync(0xffffffffu, nk == KT);
        float mx;
        if (full) {
          mx = fmaxf(fmaxf(row_max<false>(r0, 0, nk), row_max<false>(r1, 32, nk)), fmaxf(row_max<false>(r2, 64, nk), row_max<false>(r3, 96, nk)));
        } else {
          mx = row_max<true>(r0, 0, nk);
          if (nch > 1) mx = fmaxf(mx, row_max<true>(r1, 32, nk));
          if (nch > 2) mx = fmaxf(mx, row_max<true>(r2, 64, nk));
          if (nch > 3) mx = fmaxf(mx, row_max<true>(r3, 96, nk));
        }
        mx *= scale2;
        if (__any_sync(0xffffffffu, mx > m + RESCALE_GAP)) {
          const float m_new = fmaxf(m, mx);
          if (j > 0) {
            const float corr = ex2(m - m_new);
            if (!mbar_wait_warp(bar(B_O_READY + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
            fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t r[32];
              tmem_ld32(o_addr + c * 32, r);
#pragma unroll
              for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * corr);
              tmem_st32(o_addr + c * 32, r);
            }
            l *= corr;
          }
          m = m_new;
        }
        // P = exp2(S * scale - m) as packed bf16 over the first half of the S columns; a row that sees no
        // key of this tile (the upper group on the block's last tile) writes zeros
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
        if (full) {
          probs<false>(r0, 0, nk, scale2, m, ls, s_addr);
          probs<false>(r1, 32, nk, scale2, m, ls, s_addr + 16);
          probs<false>(r2, 64, nk, scale2, m, ls, s_addr + 32);
          probs<false>(r3, 96, nk, scale2, m, ls, s_addr + 48);
        } else {
          probs<true>(r0, 0, nk, scale2, m, ls, s_addr);
          if (nch > 1) probs<true>(r1, 32, nk, scale2, m, ls, s_addr + 16);
          if (nch > 2) probs<true>(r2, 64, nk, scale2, m, ls, s_addr + 32);
          if (nch > 3) probs<true>(r3, 96, nk, scale2, m, ls, s_addr + 48);
        }
        l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
        tmem_wait_st();
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_P_FULL + t));
      }
      if (!ok) break;
      if (!mbar_wait_warp(bar(B_O_READY + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
      fence_after();
      const float inv = 1.f / l;
      bf16* orow = g.out + ((size_t)row_base + q) * q_dim + (size_t)h * DH;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(o_addr + c * 32, r);
        if (q < L) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 o;
            o.x = pack_bf16(__uint_as_float(r[e + 0]) * inv, __uint_as_float(r[e + 1]) * inv);
            o.y = pack_bf16(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            o.z = pack_bf16(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
            o.w = pack_bf16(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c * 32 + e) = o;
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  fence_before();
  __syncthreads();
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);      // let copies in flight land
    if (threadIdx.x == 0 && g.status) atomicExch(g.status, (int)DS_WAIT_EXPIRED);
    __syncthreads();
  }
  if (warp == 9) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

}  // namespace

bool attention_causal_supported(int head_dim) { return head_dim == DH; }

bool make_causal_attention_map(TmaDesc* out, const bf16* qkv, long long rows, int heads, int kv_heads) {
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn) return false;
  const uint64_t cols = (uint64_t)(heads + 2 * kv_heads) * DH;
  if (reinterpret_cast<uintptr_t>(qkv) & 15u) return false;
  const cuuint64_t dims[2] = {cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  return fn(reinterpret_cast<CUtensorMap*>(out->bytes), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(qkv), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_attention_causal(const TmaDesc& map, bf16* out, int n_seq, int L, int heads, int kv_heads,
                                    int* status_dev, cudaStream_t s) {
  if (n_seq <= 0 || L <= 0) return cudaSuccess;
  if (kv_heads < 1 || heads % kv_heads != 0) return cudaErrorInvalidValue;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(attention_causal_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // setmaxnreg.inc waits for registers that only exist if the kernel was compiled with at least LAUNCH_REGS per
    // thread: refuse to launch (instead of blocking for ever) should a compiler ever assign fewer.
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, attention_causal_kernel);
    if (e != cudaSuccess) return e;
    if (fa.numRegs < LAUNCH_REGS) return cudaErrorLaunchOutOfResources;
    configured = true;
  }
  ET_COUNT_LAUNCH();
  static int sms = 0;
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  const long long items = (long long)cdiv(L, QB) * heads * n_seq;
  const int grid = (int)(items < sms ? items : sms);
  CausalArgs a{out, n_seq, L, heads, heads / kv_heads, status_dev};
  attention_causal_kernel<<<grid, ATT_THREADS, SMEM_BYTES, s>>>(*reinterpret_cast<const CUtensorMap*>(map.bytes), a);
  return cudaGetLastError();
}

}  // namespace et
