// Stage I kernels: adjacent-frame token cosines, their mean, the merge plan (Eq. 1-2) and the
// weighted merge with frame compaction (Eq. 3).  All HBM-bound or latency-bound; no tensor cores.
#include "common.cuh"
#include "rowops.cuh"

namespace et {

// ---------------------------------------------------------------------------------------------
// Token cosines.  One warp owns spatial position l over a run of consecutive frames: it keeps the
// previous frame's row (and its squared norm) in registers, so every row of X is read from memory
// once per run (plus one halo row per run), and writes cos[t][l] for every pair (t, t+1) of the run.
// Reductions: lane-local sums over a fixed chunk order, then a xor-shuffle tree -> bit-reproducible.
// ---------------------------------------------------------------------------------------------
constexpr int COS_RUN = 8;   // pairs per warp job

template <int NV>
__global__ void __launch_bounds__(128)
token_cos_kernel(const float* __restrict__ x, float* __restrict__ cosbuf, int n_cap, int L, int D,
                 const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int n_pairs = n - 1;
  if (n_pairs <= 0) return;
  const int n_runs = (n_pairs + COS_RUN - 1) / COS_RUN;
  const int lane = threadIdx.x & 31;
  const int nvec = D >> 2;
  const int warps_total = gridDim.x * (blockDim.x >> 5);
  const size_t frame_stride = (size_t)L * D;
  for (int job = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); job < n_runs * L; job += warps_total) {
    const int l = job % L, run = job / L;
    const int t0 = run * COS_RUN, t1 = min(t0 + COS_RUN, n_pairs);
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
      if (lane == 0) cosbuf[(size_t)t * L + l] = dot / fmaxf(sqrtf(np) * sqrtf(nc), 1e-8f);
      np = nc;
      if (t + 1 < t1) {
#pragma unroll
        for (int j = 0; j < NV; ++j) { prev[j] = cur[j]; cur[j] = nxt[j]; }
      }
    }
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

// sim[t] = (1/L) sum_l cos[t][l] for the pairs t < n - 1; one warp per pair, fixed order.
__global__ void reduce_cos_kernel(const float* __restrict__ cosbuf, float* __restrict__ sim, int n_cap, int L,
                                  const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= n - 1) return;
  float acc = 0.f;
  for (int l = lane; l < L; l += 32) acc += cosbuf[(size_t)t * L + l];
  acc = warp_sum(acc);
  if (lane == 0) sim[t] = acc / (float)L;
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
__global__ void merge_plan_kernel(PlanArgs a) {
  extern __shared__ int sh_count[];     // [n_videos + 1] output frames per video, then their scan
  const int V = a.n_videos;
  const int n = *a.cur.n;
  const bool forced = a.forced_seg_start != nullptr;
  if (forced && threadIdx.x == 0 && a.forced_n_in != n) atomicExch(a.status, (int)DS_FORCED_MISMATCH);
  const bool use_forced = forced && a.forced_n_in == n;
  unsigned char* const f_start = a.trace.seg_start;   // flags of the INPUT list (also the trace)
  unsigned char* const f_merge = a.trace.merge_next;

  // Pass 1 (per video): Eq. 1 segmentation, Eq. 2 pairing, count of output frames.
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    const int g0 = a.cur.vid_off[v], g1 = a.cur.vid_off[v + 1];
    double prev = 0.0;
    bool have_prev = false;
    for (int t = g0; t < g1; ++t) {
      unsigned char start = 1;
      float ema_out = 0.f;
      if (t > g0) {
        const double s = (double)a.sim[t - 1];
        // explicit roundings: no fused multiply-add, so the value is the same as a plain host evaluation
        const double cur = have_prev ? __dadd_rn(__dmul_rn(a.alpha, s), __dmul_rn(1.0 - a.alpha, prev)) : s;
        ema_out = (float)cur;
        start = use_forced ? (a.forced_seg_start[t] ? 1 : 0) : (cur < a.tau_seg ? 1 : 0);
        if (start) have_prev = false;
        else { prev = cur; have_prev = true; }
      }
      f_start[t] = start;
      a.trace.ema[t] = ema_out;
      a.trace.sim[t] = (t < g1 - 1) ? a.sim[t] : 0.f;
      f_merge[t] = 0;
    }
    if (a.allow_merge && use_forced) {
      for (int t = g0; t < g1; ++t) {
        bool m = a.forced_merge_next[t] != 0;
        if (m && (t + 1 >= g1 || (t > g0 && f_merge[t - 1]))) { m = false; atomicExch(a.status, (int)DS_FORCED_MISMATCH); }
        f_merge[t] = m ? 1 : 0;
      }
    } else if (a.allow_merge) {
      int seg_a = g0;
      while (seg_a < g1) {
        int seg_b = seg_a;                       // last frame of the segment
        while (seg_b + 1 < g1 && f_start[seg_b + 1] == 0) ++seg_b;
        const int k = seg_b - seg_a;
        int i = 1;
        while (i <= k - 1) {                     // middle frames g_1 .. g_{k-1}
          const int t = seg_a + i;
          bool m = false;
          if (i <= k - 2) {                      // both frames of the pair are middle frames
            const double ci = (double)a.sim[t], cn = (double)a.sim[t + 1];
            m = (ci > a.tau_merge) && (ci > cn);
          }
          f_merge[t] = m ? 1 : 0;
          i += m ? 2 : 1;
        }
        seg_a = seg_b + 1;
      }
    }
    int out = 0;
    for (int t = g0; t < g1; t += f_merge[t] ? 2 : 1) ++out;
    sh_count[v] = out;
  }
  __syncthreads();

  if (!a.allow_merge) {   // segmentation only: roles of the unchanged list
    for (int v = threadIdx.x; v < V; v += blockDim.x) {
      const int g0 = a.cur.vid_off[v], g1 = a.cur.vid_off[v + 1];
      for (int t = g0; t < g1; ++t) {
        const bool s0 = f_start[t] != 0;
        const bool s1 = (t + 1 >= g1) || f_start[t + 1] != 0;
        a.cur.role[t] = s0 ? (s1 ? 3 : 0) : (s1 ? 2 : 1);
      }
    }
    if (threadIdx.x == 0 && a.n_hist_slot) *a.n_hist_slot = n;
    return;
  }

  if (threadIdx.x == 0) {
    int acc = 0;
    for (int v = 0; v < V; ++v) { const int c = sh_count[v]; sh_count[v] = acc; acc += c; }
    sh_count[V] = acc;
  }
  __syncthreads();

  // Pass 2 (per video): emit the plan and the metadata of the next list, indexed by output frame.
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    const int g0 = a.cur.vid_off[v], g1 = a.cur.vid_off[v + 1];
    int j = sh_count[v];
    int t = g0;
    while (t < g1) {
      const bool mrg = f_merge[t] != 0;
      if (mrg) {
        const double ca = (double)a.sim[t];
        const double cb = (t + 1 < g1 - 1) ? (double)a.sim[t + 1] : 0.0;   // similarity to the following frame
        const double den = ca + cb;
        float wa = 0.5f, wb = 0.5f;
        if (a.weighted && den > 1e-6) { wa = (float)(ca / den); wb = (float)(cb / den); }
        a.plan.src_a[j] = t; a.plan.src_b[j] = t + 1;
        a.plan.w_a[j] = wa;  a.plan.w_b[j] = wb;
        a.nxt.src_lo[j] = a.cur.src_lo[t];
        a.nxt.src_hi[j] = a.cur.src_hi[t + 1];
        a.nxt.role[j] = 1;
      } else {
        const bool s0 = f_start[t] != 0;
        const bool s1 = (t + 1 >= g1) || f_start[t + 1] != 0;
        a.plan.src_a[j] = t; a.plan.src_b[j] = -1;
        a.plan.w_a[j] = 1.f; a.plan.w_b[j] = 0.f;
        a.nxt.src_lo[j] = a.cur.src_lo[t];
        a.nxt.src_hi[j] = a.cur.src_hi[t];
        a.nxt.role[j] = s0 ? (s1 ? 3 : 0) : (s1 ? 2 : 1);
      }
      ++j;
      t += mrg ? 2 : 1;
    }
  }
  for (int v = threadIdx.x; v <= V; v += blockDim.x) a.nxt.vid_off[v] = sh_count[v];
  if (threadIdx.x == 0) {
    *a.nxt.n = sh_count[V];
    if (a.n_hist_slot) *a.n_hist_slot = sh_count[V];
  }
}

void launch_merge_plan(const PlanArgs& a, cudaStream_t s) {
  ET_COUNT_LAUNCH();
  const int threads = min(1024, max(32, ((a.n_videos + 31) / 32) * 32));
  merge_plan_kernel<<<1, threads, sizeof(int) * (a.n_videos + 1), s>>>(a);
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
