// Causal grouped-query attention with head dim 128 on tcgen05 (the language model's prefill).
//
// Same organisation as the per-frame encoder attention (attention_tcgen05.cu): a persistent CTA per SM,
// work items of 256 queries of one (sequence, head), two softmax warpgroups (thread = query row = TMEM
// lane), S, P and O of both groups in TMEM columns of their own, one warp issuing S = Q K^T and one warp per
// group issuing O += P V, so that the next S is computed under the current tile's exponentials.
// What differs:
//   * head dim 128 = two 128-byte swizzled 64-column boxes for Q, K and V; S = Q K^T takes 8 k-steps,
//     O += P V is one N = 128 MMA per 16 keys; the two O accumulators take 256 TMEM columns, which leaves
//     80-key tiles: S 2 x 80 + P 2 x 40 + O 2 x 128 = 496 of the 512 columns;
//   * query i sees keys 0..i: an item sweeps only the key tiles up to its diagonal, the number of valid
//     keys of a tile is a per-row quantity, and items are dealt longest first in alternating direction;
//   * several query heads share one key / value head; Q, K and V live in one packed row
//     [heads*128 | kv_heads*128 | kv_heads*128] and the row index is the position.
#include "common.cuh"
#include "softmax_tile.cuh"
#include "tcgen05.cuh"

#include <type_traits>

namespace et {

namespace {

using namespace tc;

constexpr int DH = 128;
constexpr int QT = 128;                 // queries per softmax group
constexpr int QB = 2 * QT;              // queries per CTA
constexpr int KT = 80;                  // keys per tile
constexpr int KV_STAGES = 4;
constexpr int ATOM_BYTES = 128 * 128;   // Q: 128 rows x 64 bf16, 128-byte swizzle
constexpr int TILE_BYTES = 2 * ATOM_BYTES;   // 128 rows x 128 bf16: columns 0..63, then 64..127
constexpr int KV_ATOM_BYTES = KT * 128;      // K / V: one key tile x 64 bf16 (a multiple of the 1024-byte swizzle atom)
constexpr int KV_TILE_BYTES = 2 * KV_ATOM_BYTES;
static_assert(KV_ATOM_BYTES % 1024 == 0, "swizzle atoms of a K / V stage");
constexpr int ATT_THREADS = 384;        // warps 0..7 softmax, 8 TMA, 9 S = Q K^T, 10 / 11 O += P V of group 0 / 1
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
constexpr int OFF_V = OFF_K + KV_STAGES * KV_TILE_BYTES;
constexpr int OFF_BARS = OFF_V + KV_STAGES * KV_TILE_BYTES;
constexpr int SMEM_BYTES = OFF_BARS + 256 + 1024;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");

constexpr int B_Q_FULL = 0, B_K_FULL = 1, B_V_FULL = B_K_FULL + KV_STAGES, B_KV_EMPTY = B_V_FULL + KV_STAGES,
              B_S_FULL = B_KV_EMPTY + KV_STAGES, B_S_FREE = B_S_FULL + 2, B_P_FULL = B_S_FREE + 2, B_O_READY = B_P_FULL + 2,
              B_Q_EMPTY = B_O_READY + 2, B_COUNT = B_Q_EMPTY + 1;
static_assert(B_COUNT * 8 + 8 <= 256, "barrier area");

// TMEM columns: S of group t at t*80, its P (packed bf16 pairs: 40 columns) at 160 + t*40, its O at 240 + t*128
constexpr int TMEM_COLS = 512;
constexpr int S_STRIDE = KT, COL_P = 2 * KT, P_STRIDE = KT / 2, COL_O = COL_P + 2 * P_STRIDE;
static_assert(COL_O + 2 * DH <= TMEM_COLS, "TMEM columns");

struct CausalArgs {
  bf16* out;             // [n_seq * L][heads * 128]
  int n_seq, L, heads, group;   // group = query heads per key / value head
  int* status;
};

__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_causal_kernel(const __grid_constant__ CUtensorMap tma_qkv, const __grid_constant__ CUtensorMap tma_kv, CausalArgs g) {
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
  auto item_tiles = [&](int q0) { return min(tiles_all, (q0 + QB - 1) / KT + 1); };    // key tiles up to the block's last query
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
    // a K / V stage is free once the three issuing warps are done with it
    for (int s = 0; s < KV_STAGES; ++s) { mbar_init(bar(B_K_FULL + s), 1); mbar_init(bar(B_V_FULL + s), 1); mbar_init(bar(B_KV_EMPTY + s), 3); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(bar(B_S_FULL + t), 1); mbar_init(bar(B_S_FREE + t), 4); mbar_init(bar(B_P_FULL + t), 4); mbar_init(bar(B_O_READY + t), 1);
    }
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
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_kv) : "memory");
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
            mbar_arrive_expect_tx(bar(B_K_FULL + s), KV_TILE_BYTES);
            for (int c = 0; c < 2; ++c)
              tma_load_2d(base + OFF_K + s * KV_TILE_BYTES + c * KV_ATOM_BYTES, &tma_kv, bar(B_K_FULL + s), q_dim + kvh * DH + c * 64, y);
            mbar_arrive_expect_tx(bar(B_V_FULL + s), KV_TILE_BYTES);
            for (int c = 0; c < 2; ++c)
              tma_load_2d(base + OFF_V + s * KV_TILE_BYTES + c * KV_ATOM_BYTES, &tma_kv, bar(B_V_FULL + s), q_dim + kv_dim + kvh * DH + c * 64, y);
          }
        }
      }
    } else if (warp == 9) {
      // ---------------------------------------------------------------- S = Q K^T of both groups
      // The whole warp runs the loop; one elected lane issues the MMAs and the commits.
      // Q / K: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart; the second 64 elements of the head
      // are a second box (ATOM_BYTES / KV_ATOM_BYTES further).
      const uint64_t q0d = smem_desc(base + OFF_Q, 16, 1024, 2), k0d = smem_desc(base + OFF_K, 16, 1024, 2);
      constexpr uint64_t Q_TILE_STEP = TILE_BYTES >> 4, Q_ATOM_STEP = ATOM_BYTES >> 4,
                         K_TILE_STEP = KV_TILE_BYTES >> 4, K_ATOM_STEP = KV_ATOM_BYTES >> 4;
      bool ok = true;
      int gt = 0;
      for (int i = 0; i < my_items && ok; ++i) {
        int f, h, q0;
        item_coords(i, f, h, q0);
        const int nt = item_tiles(q0);
        for (int j = 0; j < nt && ok; ++j, ++gt) {
          const int s = gt % KV_STAGES;
          if (j == 0 && !mbar_wait_warp(bar(B_Q_FULL), (uint32_t)i & 1u, abort_flag)) { ok = false; break; }
          if (!mbar_wait_warp(bar(B_K_FULL + s), (uint32_t)(gt / KV_STAGES) & 1u, abort_flag)) { ok = false; break; }
          const uint32_t idesc = idesc_bf16(128, keys_rounded(j), false, false);
          const uint64_t kd = k0d + (uint64_t)s * K_TILE_STEP;
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            // the group's softmax has taken the previous tile's logits out of the S columns
            if (gt > 0 && !mbar_wait_warp(bar(B_S_FREE + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
            fence_after();
            const uint64_t qd = q0d + (uint64_t)t * Q_TILE_STEP;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)                      // 16 elements = 32 bytes inside the swizzle row
              mma_ss_elect(tmem_base + t * S_STRIDE, qd + (uint64_t)(ks >> 2) * Q_ATOM_STEP + 2 * (ks & 3),
                           kd + (uint64_t)(ks >> 2) * K_ATOM_STEP + 2 * (ks & 3), idesc, ks != 0 ? 1u : 0u);
            commit_elect(bar(B_S_FULL + t));
          }
          if (!ok) break;
          commit_elect(bar(B_KV_EMPTY + s));                     // this warp's share: K of the tile has been read
          if (j == nt - 1) commit_elect(bar(B_Q_EMPTY));         // the item's last read of Q
        }
      }
    } else {
      // ---------------------------------------------------------------- O += P V of group t = warp - 10
      // V: MN-major with 128-byte swizzle, 64 columns per atom, the second atom KV_ATOM_BYTES further (leading byte
      // offset), 8-key groups 1024 bytes apart.  The group index is a compile-time constant on each path.
      constexpr uint32_t IDESC_PV = idesc_bf16(128, DH, false, true);
      const uint64_t v0d = smem_desc(base + OFF_V, KV_ATOM_BYTES, 1024, 2);
      auto pv_loop = [&](auto group) {
        constexpr int t = decltype(group)::value;
        const uint32_t o_col = tmem_base + COL_O + t * DH;
        int gp = 0;
        for (int i = 0; i < my_items; ++i) {
          int f, h, q0;
          item_coords(i, f, h, q0);
          const int nt = item_tiles(q0);
          for (int jj = 0; jj < nt; ++jj, ++gp) {
            const int sp = gp % KV_STAGES;
            if (!mbar_wait_warp(bar(B_V_FULL + sp), (uint32_t)(gp / KV_STAGES) & 1u, abort_flag)) return;
            if (!mbar_wait_warp(bar(B_P_FULL + t), (uint32_t)gp & 1u, abort_flag)) return;
            fence_after();
            const int ksteps = keys_rounded(jj) / 16;
            uint32_t a = tmem_base + COL_P + t * P_STRIDE;      // 16 keys = 8 columns of packed bf16 pairs
            uint64_t dv = v0d + (uint64_t)sp * (KV_TILE_BYTES >> 4);
#pragma unroll 1
            for (int ks = 0; ks < ksteps; ++ks) {
              mma_ts_elect(o_col, a, dv, IDESC_PV, (jj | ks) != 0 ? 1u : 0u);   // the first tile of an item overwrites O
              a += 8; dv += 2048 >> 4;                           // 16 keys = two 8-row groups; 16-byte units
            }
            commit_elect(bar(B_O_READY + t));                    // O holds the tile; the P columns are free again
            commit_elect(bar(B_KV_EMPTY + sp));                  // this warp's share: V of the tile has been read
          }
        }
      };
      if (warp == 10) pv_loop(std::integral_constant<int, 0>{});
      else pv_loop(std::integral_constant<int, 1>{});
    }
  } else {
    // ------------------------------------------------------------------ softmax groups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(SOFTMAX_REGS));
    const int t = warp >> 2;
    const int quarter = warp & 3;                     // TMEM lanes 32*quarter .. +31
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_addr + t * S_STRIDE, p_addr = lane_addr + COL_P + t * P_STRIDE,
                   o_addr = lane_addr + COL_O + t * DH;
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
        const int nch = (nk_tile + 31) >> 5;                      // chunks of 32, 32 and 16 keys
        const int nk = max(0, min(nk_tile, q - j * KT + 1));      // keys of this tile that query q sees
        if (!mbar_wait_warp(bar(B_S_FULL + t), (uint32_t)gt & 1u, abort_flag)) { ok = false; break; }
        fence_after();
        // the whole tile row goes to registers with one wait; the S columns are then free for the next tile's Q K^T
        uint32_t r0[32], r1[32], r2[16];
        tmem_ld32_async(s_addr, r0);
        if (nch > 1) tmem_ld32_async(s_addr + 32, r1);
        if (nch > 2) tmem_ld16_async(s_addr + 64, r2);
        tmem_wait_ld();
        tmem_regs_ready(r0);
        if (nch > 1) tmem_regs_ready(r1);
        if (nch > 2) tmem_regs_ready(r2);
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_S_FREE + t));
        const bool full = __all_sync(0xffffffffu, nk == KT);
        // Otherwise every chunk is, for the whole warp, visible (0: no masks needed), partly visible (1: masked) or
        // invisible (2: its P is zero, no exponentials).  Warp-uniform, as the TMEM stores must be.
        auto chunk_mode = [&](int c0, int w) {
          if (__all_sync(0xffffffffu, c0 + w <= nk)) return 0;
          if (__all_sync(0xffffffffu, c0 >= nk)) return 2;
          return 1;
        };
        int md0 = 0, md1 = 0, md2 = 0;
        float mx;
        if (full) {
          mx = fmaxf(fmaxf(row_max<false>(r0, 0, nk), row_max<false>(r1, 32, nk)), row_max<false>(r2, 64, nk));
        } else {
          mx = -INFINITY;
          auto chunk_max = [&](auto& r, int c0, int md) {
            if (md == 0) mx = fmaxf(mx, row_max<false>(r, c0, nk));
            else if (md == 1) mx = fmaxf(mx, row_max<true>(r, c0, nk));
          };
          md0 = chunk_mode(0, 32); chunk_max(r0, 0, md0);
          if (nch > 1) { md1 = chunk_mode(32, 32); chunk_max(r1, 32, md1); }
          if (nch > 2) { md2 = chunk_mode(64, 16); chunk_max(r2, 64, md2); }
        }
        mx *= scale2;
        // the P columns (and O, for a rescale) are free once the previous tile's P V has completed
        if (gt > 0 && !mbar_wait_warp(bar(B_O_READY + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
        fence_after();
        if (__any_sync(0xffffffffu, mx > m + RESCALE_GAP)) {
          const float m_new = fmaxf(m, mx);
          if (j > 0) {
            const float corr = ex2(m - m_new);
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
        // P = exp2(S * scale - m) as packed bf16; a row that sees no key of this tile (the upper rows of a block's last
        // tiles) writes zeros
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
        if (full) {
          probs<false>(r0, 0, nk, scale2, m, ls, p_addr);
          probs<false>(r1, 32, nk, scale2, m, ls, p_addr + 16);
          probs<false>(r2, 64, nk, scale2, m, ls, p_addr + 32);
        } else {
          auto chunk_probs = [&](auto& r, int c0, int md, uint32_t addr) {
            if (md == 0) probs<false>(r, c0, nk, scale2, m, ls, addr);
            else if (md == 1) probs<true>(r, c0, nk, scale2, m, ls, addr);
            else zero_probs(r, addr);
          };
          chunk_probs(r0, 0, md0, p_addr);
          if (nch > 1) chunk_probs(r1, 32, md1, p_addr + 16);
          if (nch > 2) chunk_probs(r2, 64, md2, p_addr + 32);
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

bool make_causal_attention_map(CausalMaps* out, const bf16* qkv, long long rows, int heads, int kv_heads) {
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn) return false;
  const uint64_t cols = (uint64_t)(heads + 2 * kv_heads) * DH;
  if (reinterpret_cast<uintptr_t>(qkv) & 15u) return false;
  const cuuint64_t dims[2] = {cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t estr[2] = {1, 1};
  auto encode = [&](TmaDesc* d, uint32_t box_rows) {
    const cuuint32_t box[2] = {64, box_rows};
    return fn(reinterpret_cast<CUtensorMap*>(d->bytes), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(qkv), dims,
              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  };
  return encode(&out->q, QT) && encode(&out->kv, KT);
}

cudaError_t launch_attention_causal(const CausalMaps& map, bf16* out, int n_seq, int L, int heads, int kv_heads,
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
  attention_causal_kernel<<<grid, ATT_THREADS, SMEM_BYTES, s>>>(*reinterpret_cast<const CUtensorMap*>(map.q.bytes),
                                                                *reinterpret_cast<const CUtensorMap*>(map.kv.bytes), a);
  return cudaGetLastError();
}

}  // namespace et
