// Per-frame multi-head attention on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
// Persistent kernel, one CTA per SM.  A work item is 256 queries of one (frame, head); the CTA sweeps the
// frame's keys in tiles of 112 and goes on to its next item without draining its pipelines:
//   warps 0..3  softmax group 0 (queries 0..127 of the CTA), warps 4..7 softmax group 1 (128..255):
//               thread = query row = TMEM lane; reads the 112 logits of a tile row into registers with
//               tcgen05.ld, releases the S columns at once (the next S = Q K^T is computed under this tile's
//               exponentials), keeps the running maximum and sum, writes P = exp2(S - m) as packed bf16 into
//               P columns of its own with tcgen05.st.
//   warp 8      TMA producer: Q (2 x 128 rows) once, then a ring of K / V tiles
//   warp 9      allocates TMEM and issues  S = Q K^T  for both groups (SS form, 128 x 112 x 16 per instruction)
//   warp 10/11  issue  O += P V  of group 0 / 1 (TS form: P is read from TMEM, V from shared memory, MN-major)
//   One thread sustains one tcgen05.mma per 130..180 cycles whatever its shape; three issuing warps with an
//   accumulator each, and no S -> P -> O -> S chain through one set of columns, keep that off the critical path:
//   a tile costs its exponentials.  112-key tiles are what makes S, P and O of two groups fit the 512 TMEM columns.
//   The control warpgroup (8..11) hands most of its registers to the softmax warpgroups (setmaxnreg).
// The running maximum is only raised when the tile maximum exceeds it by more than 8 (in the log2
// domain), so the rescale of O in TMEM is rare; P stays below 2^8, which bf16 represents without loss
// of relative precision.  The final division by the row sum makes the result independent of that choice.
//
// Head dim 64, 72 or 80.  A head row is 64 elements (one 128-byte swizzled row) plus a tail of 8 or 16 elements:
// for Q and K the tail is one contraction step (K = 16) made of two 16-byte-per-row column blocks, the second of
// which is a block of zeros for head dim 72 and the elements 72..79 for head dim 80; for V a second swizzled
// 64-column box, so that O += P V is one MMA of N = 80 per 16 keys (columns beyond the head are never read).
// Global memory keeps the packed [tokens][3*D] layout.
//
// Windowed attention (window_rows > 0): the tokens of a frame are ordered so that a window is a run of window_rows
// consecutive rows; the kernel sweeps the whole frame as usual and the softmax masks the keys outside the query's
// window (a tile without any key of the window contributes zeros).
#include "common.cuh"
#include "softmax_tile.cuh"
#include "tcgen05.cuh"

#include <type_traits>

namespace et {

namespace {

using namespace tc;

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

constexpr int QT = 128;                 // queries per softmax group
constexpr int QB = 2 * QT;              // queries per CTA
constexpr int KT = 112;                 // keys per tile
constexpr int KV_STAGES = 3;
constexpr int MAIN_BYTES = 128 * 128;   // Q: 128 rows x 64 bf16, 128-byte swizzle
constexpr int KV_MAIN_BYTES = KT * 128; // K / V: one key tile x 64 bf16, 128-byte swizzle (a multiple of the 1024-byte atom)
constexpr int TAIL_BYTES = 128 * 16;    // 128 rows x 8 bf16, rows 16 bytes apart
constexpr int KV_MAIN_TX = KV_MAIN_BYTES, KV_TAIL_TX = KT * 16;   // bytes one K / V box brings
static_assert(KV_MAIN_BYTES % 1024 == 0, "swizzle atoms of a K / V stage");
constexpr int ATT_THREADS = 384;         // warps 0..7 softmax, 8 TMA, 9 S = Q K^T, 10 / 11 O += P V of group 0 / 1
constexpr int SOFTMAX_REGS = 200, CONTROL_REGS = 80;   // per-thread register budgets after setmaxnreg
// Nothing checks that a role's code fits its budget: a path that needs more registers than it kept runs on with
// lost values and computes garbage without any error (seen when the MMA path was given a run-time group index).
// The parity tests are what validates these two numbers.
// setmaxnreg.inc blocks until the registers exist: the budgets must fit into what the CTA was launched with,
// which is at least LAUNCH_REGS per thread (the kernel is compiled for exactly one CTA of ATT_THREADS per SM).
constexpr int LAUNCH_REGS = 160;
static_assert(SOFTMAX_REGS * 256 + CONTROL_REGS * 128 <= LAUNCH_REGS * ATT_THREADS, "register budgets exceed the CTA's allocation");
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr float RESCALE_GAP = 8.f;      // raise the running maximum only when a tile exceeds it by this (log2 domain)

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q_MAIN = 0;
constexpr int OFF_K_MAIN = OFF_Q_MAIN + 2 * MAIN_BYTES;
constexpr int V_STAGE_BYTES = 2 * KV_MAIN_BYTES;                // columns 0..63 of the head, then the 64 columns from 64 on
constexpr int OFF_V_MAIN = OFF_K_MAIN + KV_STAGES * KV_MAIN_BYTES;
constexpr int TAIL_SLOT = 2 * TAIL_BYTES;                       // two column blocks (elements 64..71, 72..79) per Q group / K stage
constexpr int OFF_Q_TAIL = OFF_V_MAIN + KV_STAGES * V_STAGE_BYTES;
constexpr int OFF_K_TAIL = OFF_Q_TAIL + 2 * TAIL_SLOT;
constexpr int OFF_ZERO = OFF_K_TAIL + KV_STAGES * TAIL_SLOT;    // 2 KB of zeros: the second half of the tail step for head dim 72
constexpr int O_STAGE_BYTES = QT * 80 * 2;                      // one group's output rows (dense rows of head_dim bf16) for the TMA store
constexpr int OFF_O_STAGE = OFF_ZERO + TAIL_BYTES;
constexpr int OFF_BARS = OFF_O_STAGE + 2 * O_STAGE_BYTES;
constexpr int ATT_SMEM_BYTES = OFF_BARS + 256 + 1024;

// barrier slots
constexpr int B_Q_FULL = 0, B_K_FULL = 1, B_V_FULL = B_K_FULL + KV_STAGES, B_KV_EMPTY = B_V_FULL + KV_STAGES,
              B_S_FULL = B_KV_EMPTY + KV_STAGES, B_S_FREE = B_S_FULL + 2, B_P_FULL = B_S_FREE + 2, B_O_READY = B_P_FULL + 2,
              B_Q_EMPTY = B_O_READY + 2, B_COUNT = B_Q_EMPTY + 1;
static_assert(B_COUNT * 8 + 8 <= 256, "barrier area");
static_assert(ATT_SMEM_BYTES <= 232448, "shared memory");

// TMEM columns: S of group t at t*112, its P (packed bf16 pairs: 56 columns) at 224 + t*56, its O at 336 + t*80
constexpr int TMEM_COLS = 512;
constexpr int S_STRIDE = KT, COL_P = 2 * KT, P_STRIDE = KT / 2, COL_O = COL_P + 2 * P_STRIDE, O_STRIDE = 80;
static_assert(COL_O + 2 * O_STRIDE <= TMEM_COLS, "TMEM columns");

struct AttnArgs {
  float* lse;
  int n_cap, L, heads;
  const int* n_frames_dev;
  int* status;
  int window_rows;       // 0, or the rows of an attention window (a divisor of L)
};

template <int DH>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tma_main, const __grid_constant__ CUtensorMap tma_tail,
                    const __grid_constant__ CUtensorMap tma_kv_main, const __grid_constant__ CUtensorMap tma_kv_tail,
                    const __grid_constant__ CUtensorMap tma_out, AttnArgs g) {
  constexpr bool HAS_TAIL = DH > 64;
  constexpr bool TAIL2 = DH > 72;                    // the second column block of the tail step holds elements 72..79
  static_assert(DH == 64 || DH == 72 || DH == 80, "head dim");
  const int n = g.n_frames_dev ? min(*g.n_frames_dev, g.n_cap) : g.n_cap;
  const int L = g.L, D = g.heads * DH;
  const int n_tiles = (L + KT - 1) / KT;
  const int q_blocks = (L + QB - 1) / QB;
  // Work items (frame, head, block of 256 queries), query block fastest: the CTAs that run side by side
  // share the K / V of one (frame, head) in L2.  This CTA takes items blockIdx.x, + gridDim.x, ...
  const int n_items = n * g.heads * q_blocks;
  const int my_items = (int)blockIdx.x < n_items ? (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  if (my_items == 0) return;
  const int total_tiles = my_items * n_tiles;          // key tiles this CTA sweeps, over all its items
  auto item_coords = [&](int i, int& f, int& h, int& q0) {
    const int item = (int)blockIdx.x + i * (int)gridDim.x;
    q0 = (item % q_blocks) * QB;
    h = (item / q_blocks) % g.heads;
    f = item / (q_blocks * g.heads);
  };

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
  for (int i = threadIdx.x; i < TAIL_BYTES / 16; i += ATT_THREADS)
    reinterpret_cast<uint4*>(gen_base + OFF_ZERO)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();                   // the zeros are read by the tensor core (async proxy)
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_ptr_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem_base = *tmem_ptr_slot;

  auto keys_rounded = [&](int j) { return (min(KT, L - j * KT) + 15) & ~15; };   // MMA N / K extent of key tile j of an item

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CONTROL_REGS));
  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_main) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_kv_main) : "memory");
      if (HAS_TAIL) asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_tail) : "memory");
      if (HAS_TAIL) asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_kv_tail) : "memory");
      constexpr uint32_t Q_TX = MAIN_BYTES + (HAS_TAIL ? TAIL_BYTES : 0) + (TAIL2 ? TAIL_BYTES : 0);
      constexpr uint32_t K_TX = KV_MAIN_TX + (HAS_TAIL ? KV_TAIL_TX : 0) + (TAIL2 ? KV_TAIL_TX : 0);
      bool ok = true;
      int gt = 0;                                        // key tiles loaded so far: ring stage and phase
      for (int i = 0; i < my_items && ok; ++i) {
        int f, h, q0;
        item_coords(i, f, h, q0);
        const int row_base = f * L;
        // Q of the previous item is free once its last Q K^T has completed
        if (i > 0 && !mbar_wait(bar(B_Q_EMPTY), (uint32_t)(i - 1) & 1u, abort_flag)) break;
        mbar_arrive_expect_tx(bar(B_Q_FULL), 2 * Q_TX);
        for (int t = 0; t < 2; ++t) {
          tma_load_2d(base + OFF_Q_MAIN + t * MAIN_BYTES, &tma_main, bar(B_Q_FULL), h * DH, row_base + q0 + t * QT);
          if (HAS_TAIL) tma_load_2d(base + OFF_Q_TAIL + t * TAIL_SLOT, &tma_tail, bar(B_Q_FULL), h * DH + 64, row_base + q0 + t * QT);
          if (TAIL2) tma_load_2d(base + OFF_Q_TAIL + t * TAIL_SLOT + TAIL_BYTES, &tma_tail, bar(B_Q_FULL), h * DH + 72, row_base + q0 + t * QT);
        }
        for (int j = 0; j < n_tiles; ++j, ++gt) {
          const int s = gt % KV_STAGES;
          const uint32_t ph = (uint32_t)(gt / KV_STAGES) & 1u;
          if (!mbar_wait(bar(B_KV_EMPTY + s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const int y = row_base + j * KT;
          mbar_arrive_expect_tx(bar(B_K_FULL + s), K_TX);
          tma_load_2d(base + OFF_K_MAIN + s * KV_MAIN_BYTES, &tma_kv_main, bar(B_K_FULL + s), D + h * DH, y);
          if (HAS_TAIL) tma_load_2d(base + OFF_K_TAIL + s * TAIL_SLOT, &tma_kv_tail, bar(B_K_FULL + s), D + h * DH + 64, y);
          if (TAIL2) tma_load_2d(base + OFF_K_TAIL + s * TAIL_SLOT + TAIL_BYTES, &tma_kv_tail, bar(B_K_FULL + s), D + h * DH + 72, y);
          // V: a second 64-column box starting at column 64 of the head; only its first 8 or 16 columns belong to
          // the head, the rest (the next head, or zeros past the row end) lands in output columns nobody reads
          mbar_arrive_expect_tx(bar(B_V_FULL + s), (HAS_TAIL ? 2 : 1) * KV_MAIN_TX);
          tma_load_2d(base + OFF_V_MAIN + s * V_STAGE_BYTES, &tma_kv_main, bar(B_V_FULL + s), 2 * D + h * DH, y);
          if (HAS_TAIL) tma_load_2d(base + OFF_V_MAIN + s * V_STAGE_BYTES + KV_MAIN_BYTES, &tma_kv_main, bar(B_V_FULL + s), 2 * D + h * DH + 64, y);
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ S = Q K^T of both groups
    // The whole warp runs the loop (so that descriptors and addresses stay warp-uniform); one elected
    // lane issues the MMAs and the commits.
    // Descriptors of stage / group 0; the others differ by a multiple of the tile size in the address
    // field (16-byte units, bits 0..13) and, for the Q / K tails, in the offset to the zero block
    // (leading byte offset at bit 16).
    const uint32_t zero = base + OFF_ZERO;
    const uint64_t q_main0 = smem_desc(base + OFF_Q_MAIN, 16, 1024, 2), k_main0 = smem_desc(base + OFF_K_MAIN, 16, 1024, 2);
    // the second column block of a tail: the slot's own second block (head dim 80) or the shared block of zeros
    const uint64_t q_tail0 = smem_desc(base + OFF_Q_TAIL, TAIL2 ? (uint32_t)TAIL_BYTES : zero - (base + OFF_Q_TAIL), 128, 0),
                   k_tail0 = smem_desc(base + OFF_K_TAIL, TAIL2 ? (uint32_t)TAIL_BYTES : zero - (base + OFF_K_TAIL), 128, 0);
    constexpr uint64_t Q_STEP = MAIN_BYTES >> 4, K_STEP = KV_MAIN_BYTES >> 4, TAIL_STEP = TAIL_SLOT >> 4;
    // slot i: the address moves on by i slots; the distance to the shared zero block shrinks by as much
    auto tail_desc = [&](uint64_t d0, int i, int off_shift) {
      return d0 + (uint64_t)i * TAIL_STEP - (TAIL2 ? 0ull : (((uint64_t)i * TAIL_STEP) << off_shift));
    };
    bool ok = true;
    for (int gt = 0; gt < total_tiles && ok; ++gt) {     // gt counts the key tiles of all items of this CTA
      const int s = gt % KV_STAGES, j = gt % n_tiles;
      if (j == 0 && !mbar_wait_warp(bar(B_Q_FULL), (uint32_t)(gt / n_tiles) & 1u, abort_flag)) break;
      if (!mbar_wait_warp(bar(B_K_FULL + s), (uint32_t)(gt / KV_STAGES) & 1u, abort_flag)) break;
      const uint32_t idesc = idesc_bf16(128, keys_rounded(j), false, false);
      const uint64_t kd = k_main0 + (uint64_t)s * K_STEP;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        // the group's softmax has taken the previous tile's logits out of the S columns
        if (gt > 0 && !mbar_wait_warp(bar(B_S_FREE + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
        fence_after();
        const uint64_t qd = q_main0 + (uint64_t)t * Q_STEP;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)                       // 16 elements = 32 bytes inside the swizzle row
          mma_ss_elect(tmem_base + t * S_STRIDE, qd + 2 * ks, kd + 2 * ks, idesc, ks != 0 ? 1u : 0u);
        // elements 64..71 and 72..79 (or a block of zeros): two 8-element column blocks, the second one `lbo` bytes away
        if (HAS_TAIL) mma_ss_elect(tmem_base + t * S_STRIDE, tail_desc(q_tail0, t, 16), tail_desc(k_tail0, s, 16), idesc, 1u);
        commit_elect(bar(B_S_FULL + t));
      }
      if (!ok) break;
      commit_elect(bar(B_KV_EMPTY + s));                     // this warp's share: K of the tile has been read
      if (j == n_tiles - 1) commit_elect(bar(B_Q_EMPTY));    // the item's last read of Q
    }
  } else {
    // ------------------------------------------------------------------ O += P V of group t = warp - 10
    // V is MN-major with 128-byte swizzle: 64 columns per atom, the second atom KV_MAIN_BYTES further (leading byte
    // offset), 8-key groups 1024 bytes apart.  The group index is a compile-time constant on each path.
    constexpr uint32_t IDESC_PV = idesc_bf16(128, HAS_TAIL ? 80 : 64, false, true);
    const uint64_t v_main0 = smem_desc(base + OFF_V_MAIN, KV_MAIN_BYTES, 1024, 2);
    auto pv_loop = [&](auto group) {
      constexpr int t = decltype(group)::value;
      const uint32_t o_col = tmem_base + COL_O + t * O_STRIDE;
      for (int gp = 0; gp < total_tiles; ++gp) {
        const int jj = gp % n_tiles, sp = gp % KV_STAGES;
        if (!mbar_wait_warp(bar(B_V_FULL + sp), (uint32_t)(gp / KV_STAGES) & 1u, abort_flag)) break;
        if (!mbar_wait_warp(bar(B_P_FULL + t), (uint32_t)gp & 1u, abort_flag)) break;
        fence_after();
        const int ksteps = keys_rounded(jj) / 16;
        uint32_t a = tmem_base + COL_P + t * P_STRIDE;        // 16 keys = 8 columns of packed bf16 pairs
        uint64_t dv = v_main0 + (uint64_t)sp * (V_STAGE_BYTES >> 4);
#pragma unroll 1
        for (int ks = 0; ks < ksteps; ++ks) {
          mma_ts_elect(o_col, a, dv, IDESC_PV, (jj | ks) != 0 ? 1u : 0u);   // the first tile of an item overwrites O
          a += 8; dv += 2048 >> 4;                             // 16 keys = two 8-row groups; 16-byte units
        }
        commit_elect(bar(B_O_READY + t));                      // O holds the tile; the P columns are free again
        commit_elect(bar(B_KV_EMPTY + sp));                    // this warp's share: V of the tile has been read
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
                   o_addr = lane_addr + COL_O + t * O_STRIDE;
    const float scale2 = LOG2E / sqrtf((float)DH);    // logits are kept in the log2 domain
    bool ok = true;
    int gt = 0;                                       // key tiles processed so far (barrier phases)
    for (int i = 0; i < my_items && ok; ++i) {
    int f, h, q0;
    item_coords(i, f, h, q0);
    const int row_base = f * L, q = q0 + t * QT + row;
    float m = -INFINITY, l = 0.f;
    for (int j = 0; j < n_tiles; ++j, ++gt) {
      const int nk = min(KT, L - j * KT);
      const int nch = (nk + 31) >> 5;
      if (!mbar_wait_warp(bar(B_S_FULL + t), (uint32_t)gt & 1u, abort_flag)) { ok = false; break; }
      fence_after();
      // the whole tile row (up to 112 logits) goes to registers with one wait; the S columns are then free for
      // the next tile's Q K^T
      uint32_t r0[32], r1[32], r2[32], r3[16];
      tmem_ld32_async(s_addr, r0);
      if (nch > 1) tmem_ld32_async(s_addr + 32, r1);
      if (nch > 2) tmem_ld32_async(s_addr + 64, r2);
      if (nch > 3) tmem_ld16_async(s_addr + 96, r3);
      tmem_wait_ld();
      tmem_regs_ready(r0);
      if (nch > 1) tmem_regs_ready(r1);
      if (nch > 2) tmem_regs_ready(r2);
      if (nch > 3) tmem_regs_ready(r3);
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_S_FREE + t));
      // valid columns of this tile for this row: [lo, hi) (the keys of the row's window, or all nk keys)
      int lo = 0, hi = nk;
      if (g.window_rows > 0) {
        const int w0 = (min(q, L - 1) / g.window_rows) * g.window_rows - j * KT;
        lo = max(w0, 0);
        hi = min(nk, w0 + g.window_rows);
      }
      const bool full = nk == KT && g.window_rows == 0;
      // Otherwise every chunk of the tile is, for the whole warp, inside [lo, hi) (0: no masks needed), partly inside
      // (1: masked) or outside (2: its P is zero, no exponentials).  Warp-uniform, as the TMEM stores must be.
      auto chunk_mode = [&](int c0, int w) {
        if (__all_sync(0xffffffffu, c0 >= lo && c0 + w <= hi)) return 0;
        if (__all_sync(0xffffffffu, c0 >= hi || c0 + w <= lo)) return 2;
        return 1;
      };
      int md0 = 0, md1 = 0, md2 = 0, md3 = 0;
      float mx;
      if (full) {
        mx = fmaxf(fmaxf(row_max<false>(r0, 0, nk), row_max<false>(r1, 32, nk)), fmaxf(row_max<false>(r2, 64, nk), row_max<false>(r3, 96, nk)));
      } else {
        mx = -INFINITY;
        auto chunk_max = [&](auto& r, int c0, int md) {
          if (md == 0) mx = fmaxf(mx, row_max<false>(r, c0, hi));
          else if (md == 1) mx = fmaxf(mx, row_max<true>(r, c0, hi, lo));
        };
        md0 = chunk_mode(0, 32); chunk_max(r0, 0, md0);
        if (nch > 1) { md1 = chunk_mode(32, 32); chunk_max(r1, 32, md1); }
        if (nch > 2) { md2 = chunk_mode(64, 32); chunk_max(r2, 64, md2); }
        if (nch > 3) { md3 = chunk_mode(96, 16); chunk_max(r3, 96, md3); }
      }
      mx *= scale2;
      if (__any_sync(0xffffffffu, mx > m + RESCALE_GAP)) {
        const float m_new = fmaxf(m, mx);
        if (j > 0) {
          const float corr = ex2(m - m_new);
          if (!mbar_wait_warp(bar(B_O_READY + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
          fence_after();
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
            tmem_ld32(o_addr + c * 32, r);
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
            tmem_st32(o_addr + c * 32, r);
          }
          if (HAS_TAIL) {
            uint32_t r[16];
            tmem_ld16(o_addr + 64, r);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
            tmem_st16(o_addr + 64, r);
          }
          l *= corr;
        }
        m = m_new;
      }
      // the P columns are free once the previous tile's P V has completed
      if (gt > 0 && !mbar_wait_warp(bar(B_O_READY + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
      fence_after();
      // P = exp2(S * scale - m) as packed bf16
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
      if (full) {
        probs<false>(r0, 0, nk, scale2, m, ls, p_addr);
        probs<false>(r1, 32, nk, scale2, m, ls, p_addr + 16);
        probs<false>(r2, 64, nk, scale2, m, ls, p_addr + 32);
        probs<false>(r3, 96, nk, scale2, m, ls, p_addr + 48);
      } else {
        auto chunk_probs = [&](auto& r, int c0, int md, uint32_t addr) {
          if (md == 0) probs<false>(r, c0, hi, scale2, m, ls, addr);
          else if (md == 1) probs<true>(r, c0, hi, scale2, m, ls, addr, lo);
          else zero_probs(r, addr);
        };
        chunk_probs(r0, 0, md0, p_addr);
        if (nch > 1) chunk_probs(r1, 32, md1, p_addr + 16);
        if (nch > 2) chunk_probs(r2, 64, md2, p_addr + 32);
        if (nch > 3) chunk_probs(r3, 96, md3, p_addr + 48);
      }
      l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      tmem_wait_st();
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_P_FULL + t));
    }
    if (!ok) break;
    if (!mbar_wait_warp(bar(B_O_READY + t), (uint32_t)(gt - 1) & 1u, abort_flag)) { ok = false; break; }
    {
      // The group's 128 output rows go to shared memory (thread = row, dense rows of DH bf16) and from there to
      // global memory with one TMA store, which clips the rows beyond the frame.
      fence_after();
      const float inv = 1.f / l;
      uint8_t* const stage = gen_base + OFF_O_STAGE + t * O_STAGE_BYTES;
      uint4* const srow = reinterpret_cast<uint4*>(stage + row * (DH * 2));
      if (quarter == 0 && lane == 0) bulk_wait_read<0>();      // the previous item's store has read the staging rows
      named_barrier_sync(1 + t, QT);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
        tmem_ld32(o_addr + c * 32, r);
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
          uint4 o;
          o.x = pack_bf16(__uint_as_float(r[i + 0]) * inv, __uint_as_float(r[i + 1]) * inv);
          o.y = pack_bf16(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
          o.z = pack_bf16(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
          o.w = pack_bf16(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
          srow[(c * 32 + i) >> 3] = o;
        }
      }
      if (HAS_TAIL) {
        uint32_t r[16];
        tmem_ld16(o_addr + 64, r);
#pragma unroll
        for (int i = 0; i < (TAIL2 ? 16 : 8); i += 8) {
          uint4 o;
          o.x = pack_bf16(__uint_as_float(r[i + 0]) * inv, __uint_as_float(r[i + 1]) * inv);
          o.y = pack_bf16(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
          o.z = pack_bf16(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
          o.w = pack_bf16(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
          srow[(64 + i) >> 3] = o;
        }
      }
      fence_async_smem();                                      // the rows are read by the TMA unit (async proxy)
      named_barrier_sync(1 + t, QT);
      if (quarter == 0 && lane == 0) {
        tma_store_3d(&tma_out, smem_u32(stage), h * DH, q0 + t * QT, f);
        bulk_commit();
      }
      if (q < L) g.lse[((size_t)f * g.heads + h) * L + q] = (m + log2f(l)) * LN2;
    }
    }   // items
    if (quarter == 0 && lane == 0) bulk_wait_all();             // the staging rows stay alive until the last store is done
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

bool encode_map(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_cols, uint32_t box_rows,
                CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((cols * 2) & 15u)) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(reinterpret_cast<CUtensorMap*>(out->bytes), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The output [n][L][D] as a rank-3 tensor, so that a store of 128 rows is clipped at the end of its frame.
bool encode_out_map(TmaDesc* out, const void* base, uint64_t n, uint64_t L, uint64_t D, uint32_t dh) {
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((D * 2) & 15u) || ((dh * 2) & 15u)) return false;
  const cuuint64_t dims[3] = {D, L, n};
  const cuuint64_t strides[2] = {D * 2, L * D * 2};
  const cuuint32_t box[3] = {dh, QT, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(reinterpret_cast<CUtensorMap*>(out->bytes), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DH>
cudaError_t run(const AttnMaps& maps, const AttnArgs& a, cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // setmaxnreg.inc waits for registers that only exist if the kernel was compiled with at least LAUNCH_REGS per
    // thread: refuse to launch (instead of blocking for ever) should a compiler ever assign fewer.
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, attention_tc_kernel<DH>);
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
  const long long items_cap = (long long)cdiv(a.L, QB) * a.heads * a.n_cap;
  const int grid = (int)(items_cap < sms ? items_cap : sms);      // one CTA per SM, each loops over its items
  attention_tc_kernel<DH><<<grid, ATT_THREADS, ATT_SMEM_BYTES, s>>>(
      *reinterpret_cast<const CUtensorMap*>(maps.main.bytes), *reinterpret_cast<const CUtensorMap*>(maps.tail.bytes),
      *reinterpret_cast<const CUtensorMap*>(maps.kv_main.bytes), *reinterpret_cast<const CUtensorMap*>(maps.kv_tail.bytes),
      *reinterpret_cast<const CUtensorMap*>(maps.out.bytes), a);
  return cudaGetLastError();
}

}  // namespace

bool attention_tc_supported(int dh) { return dh == 64 || dh == 72 || dh == 80; }

bool make_attention_maps(AttnMaps* out, const bf16* qkv, long long rows, int heads, int dh, bf16* attn_out, int L) {
  if (!attention_tc_supported(dh)) return false;
  if (attn_out) {
    if (L < 1 || rows % L != 0) return false;
    if (!encode_out_map(&out->out, attn_out, (uint64_t)(rows / L), (uint64_t)L, (uint64_t)heads * dh, (uint32_t)dh)) return false;
  }
  const uint64_t cols = (uint64_t)3 * heads * dh;
  // Q in boxes of 128 rows, K / V in boxes of one key tile
  if (!encode_map(&out->main, qkv, (uint64_t)rows, cols, 64, QT, CU_TENSOR_MAP_SWIZZLE_128B)) return false;
  if (!encode_map(&out->kv_main, qkv, (uint64_t)rows, cols, 64, KT, CU_TENSOR_MAP_SWIZZLE_128B)) return false;
  if (dh > 64 && (!encode_map(&out->tail, qkv, (uint64_t)rows, cols, 8, QT, CU_TENSOR_MAP_SWIZZLE_NONE) ||
                  !encode_map(&out->kv_tail, qkv, (uint64_t)rows, cols, 8, KT, CU_TENSOR_MAP_SWIZZLE_NONE)))
    return false;
  if (dh <= 64) { out->tail = out->main; out->kv_tail = out->kv_main; }
  return true;
}

cudaError_t launch_attention_tc(const AttnMaps& maps, float* lse, int n_cap, int L, int heads, int dh,
                                const int* n_frames_dev, int* status_dev, cudaStream_t s, int window_rows) {
  if (n_cap <= 0) return cudaSuccess;
  if (window_rows < 0 || (window_rows > 0 && L % window_rows != 0)) return cudaErrorInvalidValue;
  AttnArgs a{lse, n_cap, L, heads, n_frames_dev, status_dev, window_rows == L ? 0 : window_rows};
  if (dh == 80) return run<80>(maps, a, s);
  if (dh == 72) return run<72>(maps, a, s);
  if (dh == 64) return run<64>(maps, a, s);
  return cudaErrorInvalidValue;
}

}  // namespace et
