// Stage II kernels: per-frame amounts (Eq. 5-6), decoupled selection (Eq. 4 / Eq. 6), the scan of
// the per-frame counts and the gather of the kept rows with warp-level prefix-sum compaction (Eq. 7).
#include "common.cuh"
#include "rowops.cuh"

namespace et {

ET_DEBUG_STATUS_WORD
ET_DEBUG_STATUS_READ(stage2_debug_status)

// ---------------------------------------------------------------------------------------------
// Selection: one CTA per frame, scores in shared memory.
//   dynamic frame: token j is kept iff fewer than k tokens precede it in the order
//                  (score descending, index ascending)  -> exact rank counting, O(L^2 / threads);
//   static frame : the first maximum of each window; windows are runs of w positions (window_mode 0,
//                  Eq. 6 as printed) or the k runs [floor(m L / k), floor((m+1) L / k)) (window_mode 1).
// A NaN score compares false against everything: it is ordered as the lowest value (after every number,
// ties to the lower index), so a frame never keeps more than k tokens and count[f] is the number of
// bytes set in the mask.  k and w are clamped to [1, L].
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float nan_to_lowest(float v) { return v != v ? -INFINITY : v; }

// The frame's scores are in sh_a (NaN already mapped); writes the mask row and returns the kept count (uniform).
__device__ __forceinline__ int select_frame(const float* sh_a, int L, bool dyn, int k_in, int w_in, int window_mode,
                                            unsigned char* __restrict__ kp) {
  const int k = max(1, min(k_in, L));
  if (dyn) {
    for (int j = threadIdx.x; j < L; j += blockDim.x) {
      const float aj = sh_a[j];
      int rank = 0;
      for (int i = 0; i < L; ++i) {
        const float ai = sh_a[i];
        rank += (ai > aj || (ai == aj && i < j)) ? 1 : 0;
      }
      kp[j] = rank < k ? 1 : 0;
    }
    return k;                                  // the order is total, so exactly k ranks are below k
  }
  const int w = max(1, min(w_in, L));
  const int M = window_mode == 1 ? k : (L + w - 1) / w;
  for (int j = threadIdx.x; j < L; j += blockDim.x) kp[j] = 0;
  __syncthreads();
  for (int m = threadIdx.x; m < M; m += blockDim.x) {
    const int lo = window_mode == 1 ? (int)(((long long)m * L) / k) : m * w;
    const int hi = window_mode == 1 ? (int)(((long long)(m + 1) * L) / k) : min(lo + w, L);
    ET_CHECK(lo >= 0 && lo < hi && hi <= L, continue);
    int best = lo;
    for (int j = lo + 1; j < hi; ++j)
      if (sh_a[j] > sh_a[best]) best = j;
    kp[best] = 1;
  }
  return M;                                    // windows are disjoint and non-empty: one byte set per window
}

// amounts given per frame (the single-step entry point)
__global__ void __launch_bounds__(256)
select_tokens_kernel(const float* __restrict__ scores, const unsigned char* __restrict__ dynamic,
                     const int* __restrict__ k_frame, const int* __restrict__ w_frame, int n_cap, int L,
                     int window_mode, unsigned char* __restrict__ keep, int* __restrict__ count) {
  extern __shared__ float sh_a[];
  const int f = blockIdx.x;
  if (f >= n_cap) return;
  const float* a = scores + (size_t)f * L;
  for (int j = threadIdx.x; j < L; j += blockDim.x) sh_a[j] = nan_to_lowest(a[j]);
  __syncthreads();
  const int c = select_frame(sh_a, L, dynamic[f] != 0, k_frame[f], w_frame[f], window_mode, keep + (size_t)f * L);
  if (threadIdx.x == 0) count[f] = c;
}

// The encoder's path: one CTA per frame finds its video, derives the video's amounts (Eq. 5 read as a per-frame
// token count k, window width w of Eq. 6; double arithmetic in the expression order of a plain host evaluation),
// the frame's dynamic flag (head / tail of its segment) and the mask, in one launch.
__global__ void __launch_bounds__(256) select_video_tokens_kernel(SelectArgs a) {
  extern __shared__ float sh_a[];
  __shared__ int sh_v;
  const int n = min(*a.fl.n, a.n_cap);
  const int f = blockIdx.x;
  if (f >= n) return;
  if (threadIdx.x == 0) {
    int lo = 0, hi = a.n_videos;               // invariant: vid_off[lo] <= f < vid_off[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (a.fl.vid_off[mid] <= f) lo = mid; else hi = mid;
    }
    sh_v = lo;
  }
  const float* sc = a.scores + (size_t)f * a.L;      // in the encoder's internal token order; selection is in raster order
  for (int j = threadIdx.x; j < a.L; j += blockDim.x) sh_a[j] = nan_to_lowest(sc[a.raster2int ? a.raster2int[j] : j]);
  __syncthreads();
  const int v = sh_v, L = a.L;
  ET_CHECK(v >= 0 && v < a.n_videos && a.fl.vid_off[v] <= f && f < a.fl.vid_off[v + 1], return);
  const int N = a.fl.vid_off[v + 1] - a.fl.vid_off[v];
  const int B = a.orig_vid_off[v + 1] - a.orig_vid_off[v];
  int k;
  if (a.retain_mode == 1) k = (int)floor(a.retain * (double)B * (double)L / (double)max(N, 1) + 1e-9);
  else k = (int)floor(a.retain * (double)L + 1e-9);
  k = max(1, min(L, k));
  const int w = max(1, L / k);                 // reported in both window modes; mode 1 cuts k near-equal windows
  const bool dyn = a.fl.role[f] != 1;
  if (threadIdx.x == 0) {
    a.dynamic[f] = dyn ? 1 : 0;
    if (f == a.fl.vid_off[v]) { a.video_k[v] = k; a.video_w[v] = w; }
  }
  if (a.mask_given) return;                    // the mask comes from the caller: only flags and amounts
  unsigned char* kp = a.keep + (size_t)f * L;
  if (a.selection == 0) {
    for (int j = threadIdx.x; j < L; j += blockDim.x) kp[j] = 1;
    if (threadIdx.x == 0) a.count[f] = L;
    return;
  }
  const int c = select_frame(sh_a, L, dyn || a.selection >= 2, k, w, a.window_mode, kp);
  if (threadIdx.x == 0) a.count[f] = c;
}

void launch_select_video_tokens(const SelectArgs& a, cudaStream_t s) {
  if (a.n_cap <= 0) return;
  ET_COUNT_LAUNCH();
  select_video_tokens_kernel<<<a.n_cap, 256, sizeof(float) * a.L, s>>>(a);
}

void launch_select_tokens(const float* scores, const unsigned char* dynamic, const int* k_frame, const int* w_frame,
                          int n_cap, int L, int window_mode, unsigned char* keep, int* count, cudaStream_t s) {
  if (n_cap <= 0) return;
  ET_COUNT_LAUNCH();
  select_tokens_kernel<<<n_cap, 256, sizeof(float) * L, s>>>(scores, dynamic, k_frame, w_frame, n_cap, L, window_mode,
                                                             keep, count);
}

// ---------------------------------------------------------------------------------------------
// Random-sampling ablation.  Philox-4x32 with 10 rounds (Salmon et al., SC'11), from its published
// definition: two 32x32->64 multiplications per round, key bumped by the Weyl constants.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                        uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

__global__ void random_scores_kernel(float* __restrict__ scores, const int* __restrict__ vid_off, int n_videos, int n_cap,
                                     int L, unsigned long long seed, const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.x;
  if (f >= n) return;
  int v = 0;
  while (v + 1 < n_videos && vid_off[v + 1] <= f) ++v;      // video of this frame (a few hundred at most)
  const uint32_t local = (uint32_t)(f - vid_off[v]);
  for (int j = threadIdx.x; j < L; j += blockDim.x) {
    const uint32_t x = philox4x32_10_word0((uint32_t)j, local, (uint32_t)v, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
    scores[(size_t)f * L + j] = (float)(x >> 8) * (1.0f / 16777216.0f);    // exact: 24 bits
  }
}

void launch_random_scores(float* scores, const int* vid_off, int n_videos, int n_cap, int L, unsigned long long seed,
                          const int* n_frames_dev, cudaStream_t s) {
  if (n_cap <= 0) return;
  ET_COUNT_LAUNCH();
  random_scores_kernel<<<n_cap, 256, 0, s>>>(scores, vid_off, n_videos, n_cap, L, seed, n_frames_dev);
}

// count[f] = number of set bytes of keep[f][:] (used when the mask is given, not decided)
__global__ void count_keep_kernel(const unsigned char* __restrict__ keep, int n_cap, int L, int* __restrict__ count,
                                  const int* __restrict__ n_frames_dev) {
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (f >= n) return;
  const int lane = threadIdx.x & 31;
  int c = 0;
  for (int j = lane; j < L; j += 32) c += keep[(size_t)f * L + j] ? 1 : 0;
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if (lane == 0) count[f] = c;
}

void launch_count_keep(const unsigned char* keep, int n_cap, int L, int* count, const int* n_frames_dev, cudaStream_t s) {
  if (n_cap <= 0) return;
  ET_COUNT_LAUNCH();
  count_keep_kernel<<<cdiv(n_cap, 4), 128, 0, s>>>(keep, n_cap, L, count, n_frames_dev);
}

// Exclusive scan of the per-frame counts by one CTA (warp-shuffle scan + carry across chunks).
__global__ void __launch_bounds__(1024)
scan_counts_kernel(const int* __restrict__ count, int* __restrict__ frame_offsets, int* __restrict__ totals, int n_cap,
                   const int* __restrict__ n_frames_dev) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < n ? count[i] : 0;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += u;
    }
    if (lane == 31) warp_tot[wid] = inc;
    __syncthreads();
    if (wid == 0) {
      int w = lane < (blockDim.x >> 5) ? warp_tot[lane] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += u;
      }
      warp_tot[lane] = w;     // inclusive scan of warp totals
    }
    __syncthreads();
    const int before = carry + (wid > 0 ? warp_tot[wid - 1] : 0) + inc - v;
    if (i < n) frame_offsets[i] = before;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry += warp_tot[(blockDim.x >> 5) - 1];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    frame_offsets[n] = carry;
    totals[0] = n;
    totals[1] = carry;
  }
}

void launch_scan_counts(const int* count, int* frame_offsets, int* totals, int n_cap, const int* n_frames_dev,
                        cudaStream_t s) {
  ET_COUNT_LAUNCH();
  scan_counts_kernel<<<1, 1024, 0, s>>>(count, frame_offsets, totals, n_cap, n_frames_dev);
}

// ---------------------------------------------------------------------------------------------
// Gather (Eq. 7) with optional LayerNorm.  grid = (slices, frames).  Each CTA sums the counts of the
// frames before its own (the frame's first output row; the CTA of slice 0 records it, and the last
// frame's also records the totals) and recomputes the frame's compaction map by a warp-level prefix
// sum: every warp ballots the keep bytes of its eighth of the positions, the warps' totals are
// scanned through shared memory, and popc of the ballot below a lane gives each kept position its
// rank; then the warps move their share of the kept rows: warp-per-row, row in registers, LayerNorm
// statistics by shuffles.
// ---------------------------------------------------------------------------------------------

template <int NV>
__global__ void __launch_bounds__(256)
gather_tokens_kernel(const float* __restrict__ x, const unsigned char* __restrict__ keep, const int* __restrict__ count,
                     int* __restrict__ frame_offsets, int* __restrict__ totals, int n_cap, int L, int D,
                     const float* __restrict__ ln_g, const float* __restrict__ ln_b, float eps, float* __restrict__ tokens,
                     int* __restrict__ token_pos, const int* __restrict__ n_frames_dev, const int* __restrict__ raster2int) {
  extern __shared__ unsigned short sh_pos[];   // [L] position of the r-th kept token of this frame
  __shared__ int sh_before[8], sh_wkept[8];
  const int n = n_frames_dev ? min(*n_frames_dev, n_cap) : n_cap;
  const int f = blockIdx.y;
  if (f >= n) return;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nwarps = blockDim.x >> 5;   // 8 warps
  const unsigned char* kp = keep + (size_t)f * L;
  // first output row of this frame: the counts of the frames before it (integer sum: any order gives the same)
  int before = 0;
  for (int g = threadIdx.x; g < f; g += blockDim.x) before += count[g];
  // compaction map: warp w owns the positions [w*chunk, (w+1)*chunk); ballots of its keep bytes stay in registers
  constexpr int MAX_STEPS = 16;                  // L <= 4096 -> chunk <= 512 positions = 16 ballots per warp
  const int chunk = ((L + nwarps * 32 - 1) / (nwarps * 32)) * 32;
  const int c0 = wid * chunk;
  unsigned masks[MAX_STEPS];
  int wkept = 0;
#pragma unroll
  for (int it = 0; it < MAX_STEPS; ++it) {
    const int j = c0 + it * 32 + lane;
    const bool k = it * 32 < chunk && j < L && kp[j] != 0;
    masks[it] = __ballot_sync(0xffffffffu, k);
    wkept += __popc(masks[it]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
  if (lane == 0) { sh_before[wid] = before; sh_wkept[wid] = wkept; }
  __syncthreads();
  int out0 = 0, kept = 0, woff = 0;
  for (int i = 0; i < nwarps; ++i) {
    out0 += sh_before[i];
    if (i < wid) woff += sh_wkept[i];
    kept += sh_wkept[i];
  }
#pragma unroll
  for (int it = 0; it < MAX_STEPS; ++it) {
    const unsigned m = masks[it];
    if ((m >> lane) & 1u) sh_pos[woff + __popc(m & ((1u << lane) - 1u))] = (unsigned short)(c0 + it * 32 + lane);
    woff += __popc(m);
  }
  __syncthreads();
  ET_CHECK(kept >= 0 && kept <= L && out0 >= 0 && (long long)out0 + kept <= (long long)n_cap * L, return);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    frame_offsets[f] = out0;
    if (f == n - 1) {
      frame_offsets[n] = out0 + kept;
      totals[0] = n;
      totals[1] = out0 + kept;
    }
  }
  for (int r = blockIdx.x * nwarps + wid; r < kept; r += gridDim.x * nwarps) {
    const int j = sh_pos[r];
    ET_CHECK(j < L, continue);
    float4 v[NV];
    load_row<NV>(x + ((size_t)f * L + (raster2int ? raster2int[j] : j)) * D, D, lane, v);   // the row of raster position j
    if (ln_g && ln_b) layernorm_row_inplace<NV>(v, D, lane, ln_g, ln_b, eps);
    else if (ln_g) rmsnorm_row_inplace<NV>(v, D, lane, ln_g, eps);
    store_row<NV>(tokens + (size_t)(out0 + r) * D, D, lane, v);
    if (lane == 0) token_pos[out0 + r] = j;
  }
}

void launch_gather_tokens(const float* x, const unsigned char* keep, const int* count, int* frame_offsets, int* totals,
                          int n_cap, int L, int D, const float* ln_g, const float* ln_b, float eps, float* tokens,
                          int* token_pos, const int* n_frames_dev, cudaStream_t s, const int* raster2int) {
  if (n_cap <= 0) return;
  // CTAs per frame: enough CTAs over all frames to fill the GPU a few times, few enough that a CTA's prologue (the
  // frame's compaction map) is spread over many rows (measured: 8 at 256 frames, 24 at 32 frames)
  const int slices = max(1, min(min(24, cdiv(L, 8)), max(6, 2048 / n_cap)));
  ET_COUNT_LAUNCH();
  const int need = cdiv(D / 4, 32);      // float4 chunks per lane
#define ET_GATHER(NV)                                                                                      \
  gather_tokens_kernel<NV><<<dim3(slices, n_cap), 256, sizeof(unsigned short) * L, s>>>(                   \
      x, keep, count, frame_offsets, totals, n_cap, L, D, ln_g, ln_b, eps, tokens, token_pos, n_frames_dev, raster2int)
  if (need <= 2) ET_GATHER(2);
  else if (need <= 4) ET_GATHER(4);
  else if (need <= 6) ET_GATHER(6);
  else if (need <= 9) ET_GATHER(9);
  else if (need <= 12) ET_GATHER(12);
  else ET_GATHER(16);
#undef ET_GATHER
}

}  // namespace et
