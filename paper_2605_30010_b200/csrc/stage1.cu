// Stage I kernels: adjacent-frame token cosines, their mean, the merge plan (Eq. 1-2) and the
// weighted merge with frame compaction (Eq. 3).  All HBM-bound or latency-bound; no tensor cores.
#include "common.cuh"
#include "rowops.cuh"
#include "tcgen05.cuh"

namespace et {

ET_DEBUG_STATUS_WORD
ET_DEBUG_STATUS_READ(stage1_debug_status)

// ---------------------------------------------------------------------------------------------
// Token cosines.  One warp owns spatial position l over a run of consecutive frames: it keeps the
// previous frame's row (and its squared norm) in registers, so every row of X is read from memory
// once per run (plus one halo row per run), and writes cos[t][l] for every pair (t, t+1) of the run.
// Reductions: lane-local sums over a fixed chunk order, then a xor-shuffle tree -> bit-reproducible.
// ---------------------------------------------------------------------------------------------
constexpr int COS_RUN = 8;   // pairs per warp job

// One job: position l over the pairs t0 .. t1-1 (frames t0 .. t1).  `is_cross(t)` says that frames t and t+1
// belong to different videos: their cosine is never used, so it is not computed.  `emit(t, c)` receives the
// cosine of pair t (same value in every lane).
template <int NV, typename CrossFn, typename EmitFn>
__device__ __forceinline__ void cos_run(const float* __restrict__ x, int l, int t0, int t1, int L, int D, int lane,
                                        CrossFn is_cross, EmitFn emit) {
  const int nvec = D >> 2;
  const size_t frame_stride = (size_t)L * D;
  const float4* row = reinterpret_cast<const float4*>(x + (size_t)t0 * frame_stride + (size_t)l * D);
  float4 prev[NV], cur[NV];
  float np = 0.f;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    prev[j] = (i < nvec) ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  row = reinterpret_cast<const float4*>(x + (size_t)(t0 + 1) * frame_stride + (size_t)l * D);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int i = lane + 32 * j;
    cur[j] = (i < nvec) ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int j = 0; j < NV; ++j)
    np += (prev[j].x * prev[j].x + prev[j].y * prev[j].y) + (prev[j].z * prev[j].z + prev[j].w * prev[j].w);
  np = warp_sum(np);
  for (int t = t0; t < t1; ++t) {
    // the row after next is requested before this pair is reduced, so that loads stay in flight
    float4 nxt[NV];
    if (t + 1 < t1) {
      row = reinterpret_cast<const float4*>(x + (size_t)(t + 2) * frame_stride + (size_t)l * D);
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        const int i = lane + 32 * j;
        nxt[j] = (i < nvec) ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    float dot = 0.f, nc = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const float4 c = cur[j];
      dot += (prev[j].x * c.x + prev[j].y * c.y) + (prev[j].z * c.z + prev[j].w * c.w);
      nc += (c.x * c.x + c.y * c.y) + (c.z * c.z + c.w * c.w);
    }
    dot = warp_sum(dot);
    nc = warp_sum(nc);
    if (!is_cross(t)) emit(t, dot / fmaxf(sqrtf(np) * sqrtf(nc), 1e-8f));
    np = nc;
    if (t + 1 < t1) {
#pragma unroll
      for (int j = 0; j < NV; ++j) { prev[j] = cur[j]; cur[j] = nxt[j]; }
    }
  }
}

struct NoCross {
  __device__ __forceinline__ bool operator()(int) const { return false; }
};

template <int NV>
__global__ void __launch_bounds__(128)
token_cos_kernel(const float* __restrict__ x, float* __restrict__ cosbuf, int n_cap, int L, int D,
                 const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int n_pairs = n - 1;
  if (n_pairs <= 0) return;
  const int n_runs = (n_pairs + COS_RUN - 1) / COS_RUN;
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (blockDim.x >> 5);
  for (int job = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); job < n_runs * L; job += warps_total) {
    const int l = job % L, run = job / L;
    const int t0 = run * COS_RUN, t1 = min(t0 + COS_RUN, n_pairs);
    cos_run<NV>(x, l, t0, t1, L, D, lane, NoCross(),
                [=](int t, float c) { if (lane == 0) cosbuf[(size_t)t * L + l] = c; });
  }
}

void launch_token_cosines(const float* x, float* cos_scratch, int n_cap, int L, int D, const int* n_frames_dev,
                          cudaStream_t s) {
  if (n_cap < 2) return;
  const int runs = cdiv(n_cap - 1, COS_RUN);
  const int blocks = min(cdiv((long long)runs * L, 4), 148 * 16);
  const int need = cdiv(D / 4, 32);
  ET_COUNT_LAUNCH();
#define ET_COS(NV) token_cos_kernel<NV><<<blocks, 128, 0, s>>>(x, cos_scratch, n_cap, L, D, n_frames_dev)
  if (need <= 1) ET_COS(1);
  else if (need <= 2) ET_COS(2);
  else if (need <= 4) ET_COS(4);
  else if (need <= 6) ET_COS(6);
  else if (need <= 9) ET_COS(9);
  else if (need <= 12) ET_COS(12);
  else ET_COS(16);
#undef ET_COS
}

// sim[t] = (1/L) sum_l cos[t][l]: lane-strided partial sums, then the xor-shuffle tree (fixed order).
__device__ __forceinline__ float reduce_pair(const float* __restrict__ cos_row, int L, int lane) {
  float acc = 0.f;
  for (int l = lane; l < L; l += 32) acc += __ldcg(cos_row + l);
  acc = warp_sum(acc);
  return acc / (float)L;
}

// one warp per pair t < n - 1
__global__ void reduce_cos_kernel(const float* __restrict__ cosbuf, float* __restrict__ sim, int n_cap, int L,
                                  const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= n - 1) return;
  const float v = reduce_pair(cosbuf + (size_t)t * L, L, lane);
  if (lane == 0) sim[t] = v;
}

void launch_reduce_cosines(const float* cos_scratch, float* sim, int n_cap, int L, const int* n_frames_dev,
                           cudaStream_t s) {
  if (n_cap < 2) return;
  ET_COUNT_LAUNCH();
  reduce_cos_kernel<<<cdiv(n_cap - 1, 4), 128, 0, s>>>(cos_scratch, sim, n_cap, L, n_frames_dev);
}

// ---------------------------------------------------------------------------------------------
// Merge plan.  One thread per video walks its (at most a few hundred) frames: EMA segmentation
// (Eq. 1), the local-optimal pairing of middle frames (Eq. 2), the Eq. 3 weights, and the
// bookkeeping of the next frame list.  Decision arithmetic is double, comparisons are the
// paper's strict inequalities.
// ---------------------------------------------------------------------------------------------
constexpr int PLAN_STAGE_FRAMES = 2048;     // lists up to this length are planned out of shared memory
static inline size_t plan_smem_bytes(int n_videos, int n_cap) {
  return sizeof(int) * (n_videos + 1) + (size_t)min(n_cap, PLAN_STAGE_FRAMES) * (2 * sizeof(float) + 2 * sizeof(int) + 1);
}

// Per-frame flag byte while the plan is being made
enum : unsigned char { PF_START = 1, PF_MERGE = 2, PF_LAST = 4, PF_FIRST = 8 };

// The plan of one merge layer, executed by ALL threads of a block (it synchronises them).  Shared memory: sh_count
// [n_videos + 1] ints followed by the staging area for `stage_frames` frames (similarity, EMA, source range, flag byte).
//   phase A, a thread per video (the first videos on lane 0 of each warp, so that their chains do not diverge),
//            frames in order: the EMA recurrence of Eq. 1 with its restarts, and the pairing of Eq. 2 inside each
//            segment, are chains in which a step depends on the decision before it.  They only touch the staged
//            arrays (a chain of reads from global memory would cost a memory latency per frame);
//   phase B, a warp per video and a lane per frame: everything that depends on one frame and its neighbour -- the
//            output index (the video's offset plus a prefix sum of "this frame opens an output frame" by ballot /
//            popc), the Eq. 3 weights, the source ranges and roles of the next list, the trace.
// Lists longer than the staging area work on the global arrays (the trace arrays double as working storage).
// Similarities are read past the L1 (other SMs may have written them during the same kernel).
// Copies the list's similarities and source ranges into the staging area (any number of threads; the caller
// synchronises them before merge_plan_body runs).  Nothing is staged when the list does not fit.
__device__ __forceinline__ void merge_plan_stage(const PlanArgs& a, int tid, int nthr, int* sh_count, int stage_frames) {
  const int n = *a.cur.n;
  if (n > stage_frames) return;
  float* const st_sim = reinterpret_cast<float*>(sh_count + a.n_videos + 1);
  int* const st_lo = reinterpret_cast<int*>(st_sim + 2 * stage_frames);
  int* const st_hi = st_lo + stage_frames;
  for (int t = tid; t < n; t += nthr) {
    st_sim[t] = __ldcg(a.sim + t);
    st_lo[t] = a.cur.src_lo[t];
    st_hi[t] = a.cur.src_hi[t];
  }
}

__device__ void merge_plan_body(const PlanArgs& a, int tid, int nthr, int* sh_count, int stage_frames) {
  const int lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
  const int V = a.n_videos;
  const int n = *a.cur.n;
  const bool forced = a.forced_seg_start != nullptr;
  if (forced && tid == 0 && a.forced_n_in != n) atomicExch(a.status, (int)DS_FORCED_MISMATCH);
  const bool use_forced = forced && a.forced_n_in == n;
  const bool staged = n <= stage_frames;
  float* const st_sim = reinterpret_cast<float*>(sh_count + V + 1);
  float* const st_ema = st_sim + stage_frames;
  int* const st_lo = reinterpret_cast<int*>(st_ema + stage_frames);
  int* const st_hi = st_lo + stage_frames;
  unsigned char* const st_flag = reinterpret_cast<unsigned char*>(st_hi + stage_frames);
  float* const ema = staged ? st_ema : a.trace.ema;
  unsigned char* const flag = staged ? st_flag : a.trace.seg_start;
  auto sim_at = [&](int t) -> float { return staged ? st_sim[t] : __ldcg(a.sim + t); };
  auto lo_at = [&](int t) -> int { return staged ? st_lo[t] : a.cur.src_lo[t]; };
  auto hi_at = [&](int t) -> int { return staged ? st_hi[t] : a.cur.src_hi[t]; };

  // ---- phase A: per video, in frame order (video v on lane v / nwarps of warp v % nwarps)
  for (int v = warp + nwarps * lane; v < V; v += nwarps * 32) {
    const int g0 = a.cur.vid_off[v], g1 = a.cur.vid_off[v + 1];
    double prev = 0.0;
    bool have_prev = false;
    for (int t = g0; t < g1; ++t) {                    // Eq. 1
      unsigned char f = PF_START;
      float ema_out = 0.f;
      if (t > g0) {
        const double s = (double)sim_at(t - 1);
        // explicit roundings: no fused multiply-add, so the value is the same as a plain host evaluation
        const double cur = have_prev ? __dadd_rn(__dmul_rn(a.alpha, s), __dmul_rn(1.0 - a.alpha, prev)) : s;
        ema_out = (float)cur;
        const bool start = use_forced ? (a.forced_seg_start[t] != 0) : (cur < a.tau_seg);
        f = start ? PF_START : 0;
        if (start) have_prev = false;
        else { prev = cur; have_prev = true; }
      }
      if (t == g0) f |= PF_FIRST;
      if (t == g1 - 1) f |= PF_LAST;
      flag[t] = f;
      ema[t] = ema_out;
    }
    int out = g1 - g0;
    if (a.allow_merge && use_forced) {
      bool prev_merged = false;
      for (int t = g0; t < g1; ++t) {
        bool m = a.forced_merge_next[t] != 0;
        if (m && (t + 1 >= g1 || prev_merged)) { m = false; atomicExch(a.status, (int)DS_FORCED_MISMATCH); }
        if (m) { flag[t] |= PF_MERGE; --out; }
        prev_merged = m;
      }
    } else if (a.allow_merge) {                        // Eq. 2 inside each segment
      int seg_a = g0;
      while (seg_a < g1) {
        int seg_b = seg_a;                             // last frame of the segment
        while (seg_b + 1 < g1 && !(flag[seg_b + 1] & PF_START)) ++seg_b;
        const int k = seg_b - seg_a;
        int i = 1;
        while (i <= k - 2) {                           // both frames of a pair are middle frames g_1 .. g_{k-1}
          const int t = seg_a + i;
          const double ci = (double)sim_at(t), cn = (double)sim_at(t + 1);
          const bool m = (ci > a.tau_merge) && (ci > cn);
          if (m) { flag[t] |= PF_MERGE; --out; }
          i += m ? 2 : 1;
        }
        seg_a = seg_b + 1;
      }
    }
    sh_count[v] = out;
  }
  __syncthreads();
  if (tid == 0) {                                      // offsets of the next list
    int acc = 0;
    for (int v = 0; v < V; ++v) { const int c = sh_count[v]; sh_count[v] = acc; acc += c; }
    sh_count[V] = acc;
  }
  __syncthreads();

  // ---- phase B: per frame, a warp per video
  for (int v = warp; v < V; v += nwarps) {
  const int g0 = a.cur.vid_off[v], g1 = a.cur.vid_off[v + 1];
  int carry = sh_count[v];                             // output frames before this chunk of 32 input frames
  for (int base = g0; base < g1; base += 32) {
    const int t = base + lane;
    const bool live = t < g1;
    const unsigned char f = live ? flag[t] : 0;
    const unsigned char fp = (live && t > 0) ? flag[t - 1] : 0;
    const unsigned char fn = (live && t + 1 < n) ? flag[t + 1] : 0;
    const bool second = !(f & PF_FIRST) && (fp & PF_MERGE);      // the second frame of a merged pair
    const bool opens = live && !second;
    const unsigned m = __ballot_sync(0xffffffffu, opens);
    const int j = carry + __popc(m & ((1u << lane) - 1u));
    carry += __popc(m);
    if (!live) continue;
    const bool last = (f & PF_LAST) != 0;
    const bool mrg = (f & PF_MERGE) != 0;
    if (a.allow_merge && opens) {
      ET_CHECK(j >= 0 && j < n && (!mrg || !last), continue);
      if (mrg) {
        const double ca = (double)sim_at(t);
        const double cb = (fn & PF_LAST) ? 0.0 : (double)sim_at(t + 1);     // similarity to the following frame
        const double den = ca + cb;
        float wa = 0.5f, wb = 0.5f;
        if (a.weighted && den > 1e-6) { wa = (float)(ca / den); wb = (float)(cb / den); }
        a.plan.src_a[j] = t; a.plan.src_b[j] = t + 1;
        a.plan.w_a[j] = wa;  a.plan.w_b[j] = wb;
        a.nxt.src_lo[j] = lo_at(t);
        a.nxt.src_hi[j] = hi_at(t + 1);
        a.nxt.role[j] = 1;
      } else {
        const bool s0 = (f & PF_START) != 0;
        const bool s1 = last || (fn & PF_START);
        a.plan.src_a[j] = t; a.plan.src_b[j] = -1;
        a.plan.w_a[j] = 1.f; a.plan.w_b[j] = 0.f;
        a.nxt.src_lo[j] = lo_at(t);
        a.nxt.src_hi[j] = hi_at(t);
        a.nxt.role[j] = s0 ? (s1 ? 3 : 0) : (s1 ? 2 : 1);
      }
    }
    if (!a.allow_merge) {                              // segmentation only: roles of the unchanged list
      const bool s0 = (f & PF_START) != 0;
      const bool s1 = last || (fn & PF_START);
      a.cur.role[t] = s0 ? (s1 ? 3 : 0) : (s1 ? 2 : 1);
    }
    a.trace.sim[t] = last ? 0.f : sim_at(t);
    if (staged) a.trace.ema[t] = ema[t];
    a.trace.merge_next[t] = mrg ? 1 : 0;
  }
  }
  __syncthreads();                                     // every neighbour's flag has been read
  for (int t = tid; t < n; t += nthr) a.trace.seg_start[t] = (flag[t] & PF_START) ? 1 : 0;
  if (!a.allow_merge) {
    if (tid == 0 && a.n_hist_slot) *a.n_hist_slot = n;
    return;
  }
  for (int v = tid; v <= V; v += nthr) a.nxt.vid_off[v] = sh_count[v];
  if (tid == 0) {
    *a.nxt.n = sh_count[V];
    if (a.n_hist_slot) *a.n_hist_slot = sh_count[V];
  }
}

__global__ void merge_plan_kernel(PlanArgs a, int stage_frames) {
  extern __shared__ int sh_plan_count[];
  merge_plan_stage(a, threadIdx.x, blockDim.x, sh_plan_count, stage_frames);
  __syncthreads();
  merge_plan_body(a, threadIdx.x, blockDim.x, sh_plan_count, stage_frames);
}

void launch_merge_plan(const PlanArgs& a, int n_cap, cudaStream_t s) {
  ET_COUNT_LAUNCH();
  merge_plan_kernel<<<1, 128, plan_smem_bytes(a.n_videos, n_cap), s>>>(a, min(n_cap, PLAN_STAGE_FRAMES));
}

// ---------------------------------------------------------------------------------------------
// Similarities and plan in ONE launch (the encoder's path).  A block job is a run of 8 pairs over a strip of
// positions; the cosine of a (pair, position) is computed as in token_cos_kernel.  The mean over positions is accumulated without any scratch array and without any order:
// every cosine is scaled by 2^32, rounded to an integer and added to the pair's 64-bit accumulator with an atomic
// add.  Integer addition is exact and commutative, so the result does not depend on the order of arrival (bit-
// reproducible), and the rounding step (2^-32 per position) is far below the fp32 rounding of the cosine itself.
// No block waits for another: a block that has finished all its jobs takes one ticket; the block that takes the last
// ticket turns the accumulators into similarities (resetting them for the next launch) and runs the plan
// (Eq. 1-2, Eq. 3 weights, next list).  Pairs that straddle two videos are not computed.
// ---------------------------------------------------------------------------------------------
constexpr double SIM_FIXED_ONE = 4294967296.0;     // 2^32
// A pair's sum is spread over SIM_SLOTS accumulators (slot = position mod SIM_SLOTS, n_cap words apart): all warps
// work on the same few pairs at the same time, and thousands of atomic adds to one address queue up in one L2 slice.
constexpr int SIM_SLOTS = 16;

// The frames are streamed through shared memory by a producer warp: a block job is a strip of S consecutive positions
// over a run of frames; the strip of one frame is contiguous in memory (S rows of D floats) and comes in with ONE bulk
// copy (cp.async.bulk, completion on an mbarrier) into a ring of frame slots.  Consumer warp w owns position w of the
// strip: it reads its row of the current and of the previous frame from shared memory, reduces as cos_run does (same
// arithmetic, same order), and releases the previous frame's slot, which the producer refills at once.  The bytes in
// flight per SM are a whole slot, whatever the registers hold, and issuing the copies costs the consumers nothing
// (with plain loads, a row per warp under way, the kernel reached 0.55 of the copy bandwidth; a bulk copy per row
// issued by the consuming warp itself cost that warp 600 cycles per row).
constexpr int SIM_MAX_STRIP = 16;                  // consumer warps = positions per strip
constexpr int SIM_MAX_SLOTS = 8;
constexpr int SIM_SMEM_BUDGET = 222 * 1024;

__device__ __forceinline__ void bulk_load_rows(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

template <int NV>
__global__ void __launch_bounds__((SIM_MAX_STRIP + 1) * 32, 1)
similarity_plan_kernel(SimPlanArgs a, int plan_bytes, int strip, int slots) {
  extern __shared__ __align__(128) unsigned char sh_raw[];
  int* const sh_plan = reinterpret_cast<int*>(sh_raw);      // used only by the block that runs the plan
  __shared__ unsigned sh_last;
  __shared__ int sh_abort;
  const int n = min(*a.n_frames_dev, a.n_cap);
  const int n_pairs = n - 1;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int stage = min(a.n_cap, PLAN_STAGE_FRAMES);
  if (n_pairs <= 0) {                   // single frame: nothing to compare, the plan still sets roles and counts
    if (blockIdx.x == 0) {
      merge_plan_stage(a.plan, threadIdx.x, blockDim.x, sh_plan, stage);
      __syncthreads();
      merge_plan_body(a.plan, threadIdx.x, blockDim.x, sh_plan, stage);
    }
    return;
  }
  const int n_strips = (a.L + strip - 1) / strip;
  const int n_runs = (n_pairs + COS_RUN - 1) / COS_RUN;
  const int n_jobs = n_runs * n_strips;
  if ((int)blockIdx.x >= n_jobs) return;                // blocks without a job take no ticket
  const uint32_t row_bytes = (uint32_t)a.D * 4u;
  const size_t slot_bytes = (size_t)strip * row_bytes;
  const uint32_t bar_full = tc::smem_u32(sh_raw + plan_bytes), bar_empty = bar_full + 8u * SIM_MAX_SLOTS;
  unsigned char* const ring = sh_raw + plan_bytes + 1024;
  if (threadIdx.x == 0) {
    sh_abort = 0;
    for (int i = 0; i < slots; ++i) { tc::mbar_init(bar_full + 8u * i, 1); tc::mbar_init(bar_empty + 8u * i, (uint32_t)strip); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  bool ok = true;
  if (warp == strip) {
    // ---- producer: the frames t0 .. t1 of every job of this block, in order, one copy each
    int slot = 0, uses = 0;
    uint32_t phase = 1;                 // parity of the release that precedes a slot's use (none before its first)
    for (int job = blockIdx.x; job < n_jobs && ok; job += gridDim.x) {
      const int run = job / n_strips, l0 = (job % n_strips) * strip;
      const int t0 = run * COS_RUN, t1 = min(t0 + COS_RUN, n_pairs);
      const uint32_t bytes = (uint32_t)min(strip, a.L - l0) * row_bytes;
      ET_CHECK(t0 >= 0 && t1 <= a.n_cap - 1 && l0 < a.L, ok = false);
      if (!ok) break;
      for (int t = t0; t <= t1; ++t, ++uses) {
        if (uses >= slots && !tc::mbar_wait_warp(bar_empty + 8u * slot, phase, &sh_abort)) { ok = false; break; }
        if (lane == 0) {
          tc::mbar_arrive_expect_tx(bar_full + 8u * slot, bytes);
          bulk_load_rows(tc::smem_u32(ring + (size_t)slot * slot_bytes), a.x + ((size_t)t * a.L + l0) * a.D, bytes, bar_full + 8u * slot);
        }
        if (++slot == slots) { slot = 0; phase ^= 1u; }
      }
    }
  } else if (warp < strip) {
    // ---- consumers
    const int nvec = a.D >> 2;
    const int* vo = a.vid_off;
    int v = 0;                          // video of the current frame; the jobs of a block come in ascending frame order
    int slot = 0;                       // ring position and phase of the next frame
    uint32_t phase = 0;
    for (int job = blockIdx.x; job < n_jobs && ok; job += gridDim.x) {
      const int run = job / n_strips, l = (job % n_strips) * strip + warp;
      const int t0 = run * COS_RUN, t1 = min(t0 + COS_RUN, n_pairs);
      const bool mine = l < a.L;        // the last strip of a frame may be short: its spare warps only pass the slots on
      unsigned cross = 0;               // bit q: frames t0+q and t0+q+1 belong to different videos
      for (int t = t0; t < t1; ++t) {
        while (vo[v + 1] <= t) ++v;
        if (t + 1 == vo[v + 1]) cross |= 1u << (t - t0);
      }
      float4 prev[NV];                  // the previous frame's row stays in registers: a slot is free once it has been read
      float np = 0.f;
      float my_dot = 0.f, my_np = 1.f, my_nc = 1.f;      // lane q keeps the sums of pair t0 + q until the run is done
      for (int r = 0; r <= t1 - t0; ++r) {
        if (!tc::mbar_wait_warp(bar_full + 8u * slot, phase, &sh_abort)) { ok = false; break; }
        float4 cur[NV];
        if (mine) {
          const float4* row = reinterpret_cast<const float4*>(ring + (size_t)slot * slot_bytes + (size_t)warp * row_bytes);
#pragma unroll
          for (int j = 0; j < NV; ++j) {
            const int i = lane + 32 * j;
            cur[j] = (i < nvec) ? row[i] : make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        __syncwarp();                   // every lane has taken its part of the row
        if (lane == 0) tc::mbar_arrive(bar_empty + 8u * slot);
        if (++slot == slots) { slot = 0; phase ^= 1u; }
        if (mine) {
          float dot = 0.f, nc = 0.f;
          if (r == 0) {
#pragma unroll
            for (int j = 0; j < NV; ++j)
              nc += (cur[j].x * cur[j].x + cur[j].y * cur[j].y) + (cur[j].z * cur[j].z + cur[j].w * cur[j].w);
            nc = warp_sum(nc);
          } else {
#pragma unroll
            for (int j = 0; j < NV; ++j) {
              const float4 c = cur[j];
              dot += (prev[j].x * c.x + prev[j].y * c.y) + (prev[j].z * c.z + prev[j].w * c.w);
              nc += (c.x * c.x + c.y * c.y) + (c.z * c.z + c.w * c.w);
            }
            dot = warp_sum(dot);
            nc = warp_sum(nc);
            if (lane == r - 1) { my_dot = dot; my_np = np; my_nc = nc; }
          }
          np = nc;
#pragma unroll
          for (int j = 0; j < NV; ++j) prev[j] = cur[j];
        }
      }
      if (ok && mine && lane < t1 - t0 && !((cross >> lane) & 1u)) {
        // c * 2^32 is exact in fp32 (a power-of-two scaling), so the only rounding is the one to an integer
        const float c = my_dot / fmaxf(sqrtf(my_np) * sqrtf(my_nc), 1e-8f);
        atomicAdd(a.acc + (size_t)(l % SIM_SLOTS) * a.n_cap + (t0 + lane), (unsigned long long)__float2ll_rn(c * 4294967296.0f));
      }
    }
  }
  if (!ok) {                            // a wait ran out: report it, and give the copies in flight time to land
    if (lane == 0) atomicExch(a.plan.status, (int)DS_WAIT_EXPIRED);
    const unsigned long long t_begin = tc::global_ns();
    while (tc::global_ns() - t_begin < 200000ull) __nanosleep(1000);
  }
  if (lane == 0) __threadfence();       // this warp's additions before the block's ticket
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned blocks_with_jobs = (unsigned)min((int)gridDim.x, n_jobs);
    sh_last = atomicAdd(a.done, 1u) == blocks_with_jobs - 1u ? 1u : 0u;
  }
  __syncthreads();
  if (!sh_last) return;
  // the last block: accumulators -> similarities (and back to zero for the next launch), then the plan
  __threadfence();
  for (int t = threadIdx.x; t < n_pairs; t += blockDim.x) {
    unsigned long long part[SIM_SLOTS];
#pragma unroll
    for (int q = 0; q < SIM_SLOTS; ++q) part[q] = __ldcg(a.acc + (size_t)q * a.n_cap + t);   // the adds happened at the L2
    unsigned long long sum = 0;
#pragma unroll
    for (int q = 0; q < SIM_SLOTS; ++q) {
      sum += part[q];
      a.acc[(size_t)q * a.n_cap + t] = 0ull;
    }
    a.sim[t] = (float)((double)(long long)sum / (SIM_FIXED_ONE * (double)a.L));      // the mean, rounded once
  }
  if (threadIdx.x == 0) *a.done = 0u;
  __threadfence();
  __syncthreads();
  merge_plan_stage(a.plan, threadIdx.x, blockDim.x, sh_plan, stage);
  __syncthreads();
  merge_plan_body(a.plan, threadIdx.x, blockDim.x, sh_plan, stage);
}

int similarity_plan_words(int n_cap) { return SIM_SLOTS * n_cap + 1; }

void launch_similarity_plan(const SimPlanArgs& a, cudaStream_t s) {
  const int runs = max(1, cdiv(max(a.n_cap - 1, 1), COS_RUN));
  static int sms = 0;
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  const int need = cdiv(a.D / 4, 32);
  const int plan_bytes = (int)((plan_smem_bytes(a.n_videos, a.n_cap) + 127) & ~(size_t)127);
  const int row_bytes = a.D * 4;
  // the strip as wide as three slots (the frame being read, two on their way) allow; then as many slots as fit
  const int room = SIM_SMEM_BUDGET - plan_bytes - 1024;
  const int strip = max(1, min(min(SIM_MAX_STRIP, a.L), room / (3 * row_bytes)));
  const int slots = max(2, min(SIM_MAX_SLOTS, room / (strip * row_bytes)));
  const size_t smem = (size_t)plan_bytes + 1024 + (size_t)slots * strip * row_bytes;
  const int blocks = (int)max(1ll, min((long long)runs * cdiv(a.L, strip), (long long)sms));   // one block per SM
  ET_COUNT_LAUNCH();
#define ET_SP(NV)                                                                                                     \
  do {                                                                                                                \
    static bool configured = false;                                                                                   \
    if (!configured) {                                                                                                \
      cudaFuncSetAttribute(similarity_plan_kernel<NV>, cudaFuncAttributeMaxDynamicSharedMemorySize, SIM_SMEM_BUDGET); \
      configured = true;                                                                                              \
    }                                                                                                                 \
    similarity_plan_kernel<NV><<<blocks, (strip + 1) * 32, smem, s>>>(a, plan_bytes, strip, slots);                   \
  } while (0)
  if (need <= 1) ET_SP(1);
  else if (need <= 2) ET_SP(2);
  else if (need <= 4) ET_SP(4);
  else if (need <= 6) ET_SP(6);
  else if (need <= 9) ET_SP(9);
  else if (need <= 12) ET_SP(12);
  else ET_SP(16);
#undef ET_SP
}

// ---------------------------------------------------------------------------------------------
// Weighted merge + frame compaction (Eq. 3): y[j] = w_a x[src_a] + w_b x[src_b], or a copy.
// grid.y = output frame, grid.x = slices of the frame; float4 streaming.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
merge_frames_kernel(const float4* __restrict__ x, float4* __restrict__ y, int frame_vec4,
                    const int* __restrict__ n_out_dev, MergePlan plan) {
  const int j = blockIdx.y;
  if (j >= *n_out_dev) return;
  const int sa = plan.src_a[j], sb = plan.src_b[j];
  ET_CHECK(sa >= 0 && sa < (int)gridDim.y && sb >= -1 && sb < (int)gridDim.y, return);
  const float4* xa = x + (size_t)sa * frame_vec4;
  float4* yo = y + (size_t)j * frame_vec4;
  if (sb < 0) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < frame_vec4; i += gridDim.x * blockDim.x) yo[i] = __ldg(xa + i);
  } else {
    const float wa = plan.w_a[j], wb = plan.w_b[j];
    const float4* xb = x + (size_t)sb * frame_vec4;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < frame_vec4; i += gridDim.x * blockDim.x) {
      const float4 p = __ldg(xa + i), q = __ldg(xb + i);
      yo[i] = make_float4(wa * p.x + wb * q.x, wa * p.y + wb * q.y, wa * p.z + wb * q.z, wa * p.w + wb * q.w);
    }
  }
}

void launch_merge_frames(const float* x, float* y, int n_cap, int frame_elems, const int* n_out_dev,
                         const MergePlan& plan, cudaStream_t s) {
  if (n_cap <= 0) return;
  const int vec4 = frame_elems / 4;
  const int slices = max(1, min(cdiv(vec4, 256 * 4), 64));
  ET_COUNT_LAUNCH();
  merge_frames_kernel<<<dim3(slices, n_cap), 256, 0, s>>>((const float4*)x, (float4*)y, vec4, n_out_dev, plan);
}

__global__ void init_frames_kernel(FrameList fl, const int* __restrict__ vid_off_src, int V, int n) {
  for (int v = threadIdx.x; v <= V; v += blockDim.x) fl.vid_off[v] = vid_off_src[v];
  if (threadIdx.x == 0) *fl.n = n;
  for (int v = 0; v < V; ++v) {
    const int g0 = vid_off_src[v], g1 = vid_off_src[v + 1];
    for (int t = g0 + threadIdx.x; t < g1; t += blockDim.x) {
      fl.src_lo[t] = t - g0;
      fl.src_hi[t] = t - g0;
      fl.role[t] = 3;
    }
  }
}

void launch_init_frames(const FrameList& fl, const int* vid_off_src_dev, int n_videos, int n_frames, cudaStream_t s) {
  ET_COUNT_LAUNCH();
  init_frames_kernel<<<1, 256, 0, s>>>(fl, vid_off_src_dev, n_videos, n_frames);
}

}  // namespace et
