// C-ABI entry points and host orchestration: weights, workspace, the per-call launch sequence.
// No kernel here does arithmetic of the method; this file only sequences the kernels of the other
// translation units on one stream and moves the (tiny) result sizes back to the host.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <vector>

#include "common.cuh"
#include "rowops.cuh"

namespace et {
std::atomic<unsigned long long> g_kernel_launches{0};

void launch_score_finish(const float* partial, float* score, int n_cap, int L, int heads, const int* n_frames_dev,
                         cudaStream_t s);

namespace {

// Row of output j of a gated MLP ([gate | up]) in the order the fused epilogue of the dense layer wants: tiles of 256
// rows = 128 outputs, inside a tile four groups of (32 gate rows, 32 up rows) of the same 32 outputs.
__host__ __device__ inline int gated_row(int j, int up) { return (j >> 7) * 256 + ((j & 127) >> 5) * 64 + up * 32 + (j & 31); }

// dst[row(n)][k_pad] (bf16, zero padded for k >= K) = src[k][n] (fp32); row(n) = n, or, with gated_M > 0 (source
// columns [gate (gated_M) | up (gated_M)]), gated_row of the output (rows of padded outputs stay as they are)
__global__ void transpose_to_bf16_kernel(const float* __restrict__ src, bf16* __restrict__ dst, int K, int N, int k_pad,
                                         int gated_M) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int k = k0 + i, n = n0 + threadIdx.x;
    tile[i][threadIdx.x] = (k < K && n < N) ? src[(size_t)k * N + n] : 0.f;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int n = n0 + i, k = k0 + threadIdx.x;
    if (n < N && k < k_pad) {
      const int row = gated_M > 0 ? gated_row(n >= gated_M ? n - gated_M : n, n >= gated_M ? 1 : 0) : n;
      dst[(size_t)row * k_pad + k] = __float2bfloat16_rn(tile[threadIdx.x][i]);
    }
  }
}

// flag[0] = 1 if any of the `count` floats is NaN or infinite
__global__ void find_nonfinite_kernel(const float* __restrict__ w, size_t count, int* __restrict__ flag) {
  bool bad = false;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
    bad |= !isfinite(w[i]);
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicExch(flag, 1);
}

struct LayerOffsets { size_t ln1_g, ln1_b, wqkv, bqkv, wo, bo, ln2_g, ln2_b, w1, b1, w2, b2; };

struct LayerBf16 {
  bf16 *wqkv_t, *wo_t, *w1_t, *w2_t;       // arch 1: w1 = [gate | up] (each half padded to Mp rows), w2 = down
  WeightDesc d_wqkv, d_wo, d_w1, d_w2;
};

}  // namespace
}  // namespace et

using namespace et;

struct et_encoder {
  et_config cfg{};
  int L = 0, grid = 0, P = 0, Kp = 0, dh = 0, Fmax = 0, Vmax = 0;   // Fmax: capacity in ENCODER frames
  bool bf = false;
  // Qwen2.5-VL-style encoder (cfg.arch == 1)
  int arch = 0, tp = 1, ws = 0, wpf = 1, Lw = 0, Mp = 0;   // frames per temporal patch, window side, windows per frame,
                                                            // tokens per window, MLP width as stored (padded on the bf16 path)
  int *int2raster = nullptr, *raster2int = nullptr;         // [L] token orders (NULL: raster order is the internal order)
  std::vector<int> r2i_host;                                // host copy of raster2int (the trace reports scores in raster order)
  float* h_scores_int = nullptr;                            // staging for that permutation
  float2* rope_table = nullptr;                             // [L][dh/2] (cos, sin) by internal position
  float* zeros = nullptr;                                   // [max(D, 2*Mp)] zero bias / zero position row
  float* bgu_pad = nullptr;                                 // [layers][2*Mp] gate | up biases in the padded layout (bf16 path)
  int* n_windows = nullptr;                                 // [1] attention windows alive = frames alive * wpf
  void* GU = nullptr;                                       // fp32 path: [rows][2*M] gate | up pre-activations
  int device = 0;
  std::string last_error;
  std::vector<void*> dev_allocs, host_allocs;

  // weights
  float* w_blob = nullptr;                     // whole fp32 blob on the device (small params always read from here)
  size_t off_patch_w = 0, off_patch_b = 0, off_pos = 0, off_post_g = 0, off_post_b = 0;
  std::vector<LayerOffsets> lo;
  bf16* patch_w_t = nullptr;
  WeightDesc d_patch_w;
  std::vector<LayerBf16> lb;

  // activations
  float* X[2] = {nullptr, nullptr};
  void *Pm = nullptr, *Xn = nullptr, *QKV = nullptr, *O = nullptr, *Hm = nullptr;
  TmaDesc d_Pm, d_Xn, d_O, d_Hm;                   // operand (A) maps
  TmaDesc c_X[2], c_QKV, c_Hm;                      // output (C) maps
  AttnMaps attn_maps;                               // QKV as seen by the tcgen05 attention kernel
  bool attn_tc = false, scores_tc = false;
  float *lse = nullptr, *score_partial = nullptr, *scores = nullptr, *simbuf = nullptr;
  // Pipelined host calls (et_encode_batch_host_submit / _collect): two calls may be in flight; each owns a slot with
  // its own frame staging, result buffers and pinned words.  Slot 0's result buffers are the encoder's regular ones.
  struct HostSlot {
    float* frames_stage = nullptr;
    float* tokens = nullptr;
    int *token_pos = nullptr, *frame_offsets = nullptr, *src_lo = nullptr, *src_hi = nullptr, *vfo = nullptr;
    unsigned char* dynamic = nullptr;
    int *h_small = nullptr, *h_vid_off = nullptr;
    cudaEvent_t ev_h2d = nullptr, ev_done = nullptr;
    bool busy = false;                      // submitted and not collected yet
    void* stream = nullptr;                 // the stream its work was enqueued on
    et_params params{};
    et_host_buffers dst{};
    int V = 0, T = 0;
    unsigned long long ticket = 0;
  } slot[2];
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  unsigned long long next_ticket = 1;

  // frame lists, plans, traces
  FrameList fl[2]{};
  MergePlan plan{};
  LayerTrace tr[ET_MAX_MERGE_LAYERS]{};
  unsigned char* forced_seg[ET_MAX_MERGE_LAYERS]{};
  unsigned char* forced_mrg[ET_MAX_MERGE_LAYERS]{};
  int* orig_vid_off = nullptr;
  unsigned char *dynamic = nullptr, *keep = nullptr;
  int *video_k = nullptr, *video_w = nullptr, *count = nullptr;
  unsigned long long* sim_acc = nullptr;        // [Fmax] similarity accumulators + the ticket word (zero between launches)
  int *frame_offsets = nullptr, *token_pos = nullptr;
  float* tokens = nullptr;
  int* d_small = nullptr;   // [0] n_frames, [1] n_tokens, [2..9] n after merge layer i, [10] status
  // pinned host
  int* h_small = nullptr;
  int* h_vid_off = nullptr;
  unsigned char* h_forced = nullptr;           // [2*8*Fmax]
  unsigned char* h_keep_stage = nullptr;       // [Fmax*L]
  // trace (host)
  et_trace trace{};
  float* h_tr_f = nullptr;                     // sim/ema [2*8*Fmax]
  unsigned char* h_tr_b = nullptr;             // flags [2*8*Fmax]
  float* h_scores = nullptr;
  unsigned char* h_keep = nullptr;
  int* h_video_kw = nullptr;                   // [2*Vmax]
  // profiling
  bool prof_on = false;
  et_profile prof{};
  std::vector<cudaEvent_t> prof_events;
  struct Span { int cat; int ev; unsigned long long launches0, launches1; };
  std::vector<Span> prof_spans;
  size_t prof_next_event = 0;
};

namespace {

et_status fail(et_encoder* e, et_status st, const std::string& msg) {
  if (e) e->last_error = msg;
  return st;
}

void prof_begin(et_encoder* e, int cat, cudaStream_t s) {
  if (!e->prof_on) return;
  if (e->prof_next_event + 2 > e->prof_events.size()) {
    for (int i = 0; i < 2; ++i) {
      cudaEvent_t ev;
      if (cudaEventCreate(&ev) != cudaSuccess) return;
      e->prof_events.push_back(ev);
    }
  }
  et_encoder::Span sp{cat, (int)e->prof_next_event, g_kernel_launches.load(), 0};
  cudaEventRecord(e->prof_events[e->prof_next_event], s);
  e->prof_next_event += 2;
  e->prof_spans.push_back(sp);
}
void prof_end(et_encoder* e, cudaStream_t s) {
  if (!e->prof_on || e->prof_spans.empty()) return;
  et_encoder::Span& sp = e->prof_spans.back();
  sp.launches1 = g_kernel_launches.load();
  cudaEventRecord(e->prof_events[sp.ev + 1], s);
}
#define PROF(cat, ...)        \
  do {                        \
    prof_begin(e, (cat), s);  \
    __VA_ARGS__;              \
    prof_end(e, s);           \
  } while (0)

#define ET_CUDA(e, call)                                                                        \
  do {                                                                                          \
    cudaError_t err__ = (call);                                                                 \
    if (err__ != cudaSuccess)                                                                   \
      return fail((e), err__ == cudaErrorMemoryAllocation ? ET_ERR_OOM : ET_ERR_CUDA,           \
                  std::string(#call) + ": " + cudaGetErrorString(err__));                       \
  } while (0)

template <typename T>
et_status dalloc(et_encoder* e, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t err = cudaMalloc(&q, std::max<size_t>(count, 1) * sizeof(T));
  if (err != cudaSuccess) return fail(e, ET_ERR_OOM, std::string("cudaMalloc: ") + cudaGetErrorString(err));
  e->dev_allocs.push_back(q);
  *p = reinterpret_cast<T*>(q);
  return ET_OK;
}
template <typename T>
et_status halloc(et_encoder* e, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t err = cudaMallocHost(&q, std::max<size_t>(count, 1) * sizeof(T));
  if (err != cudaSuccess) return fail(e, ET_ERR_OOM, std::string("cudaMallocHost: ") + cudaGetErrorString(err));
  e->host_allocs.push_back(q);
  *p = reinterpret_cast<T*>(q);
  return ET_OK;
}
#define ET_TRY(x)                      \
  do {                                 \
    et_status st__ = (x);              \
    if (st__ != ET_OK) return st__;    \
  } while (0)

size_t blob_floats(const et_config& c, int L, int P) {
  const size_t D = c.hidden, M = c.mlp_dim;
  if (c.arch == 1) {
    const size_t per_layer = D + D * 3 * D + 3 * D + D * D + D + D + D * 2 * M + 2 * M + M * D + D;
    return (size_t)P * D + per_layer * c.num_layers + D;
  }
  size_t per_layer = 2 * D + D * 3 * D + 3 * D + D * D + D + 2 * D + D * M + M + M * D + D;
  return (size_t)P * D + D + (size_t)L * D + per_layer * c.num_layers + 2 * D;
}

et_status validate_config(const et_config* c) {
  if (!c) return ET_ERR_INVALID_ARG;
  if (c->image_size < 1 || c->patch_size < 1 || c->image_size < c->patch_size) return ET_ERR_SHAPE;
  if (c->num_layers < 1 || c->num_layers > 64) return ET_ERR_SHAPE;
  if (c->hidden < 4 || c->hidden % 4 != 0 || c->hidden > ROW_MAX_D) return ET_ERR_SHAPE;
  if (c->heads < 1 || c->hidden % c->heads != 0) return ET_ERR_SHAPE;
  if (c->hidden / c->heads > 128) return ET_ERR_SHAPE;
  if (c->mlp_dim < 1) return ET_ERR_SHAPE;
  if (c->dtype != ET_F32 && c->dtype != ET_BF16) return ET_ERR_INVALID_ARG;
  // (the gated MLP of arch 1 is stored padded to a multiple of 64 columns, so its width is free)
  if (c->dtype == ET_BF16 && (c->hidden % 8 != 0 || (c->arch != 1 && c->mlp_dim % 8 != 0) || (c->hidden / c->heads) % 8 != 0)) return ET_ERR_SHAPE;
  if (c->max_frames_total < 1 || c->max_videos < 1 || c->max_videos > 1024) return ET_ERR_INVALID_ARG;
  if (c->max_frames_total / (c->temporal_patch > 1 ? c->temporal_patch : 1) > 65535) return ET_ERR_CAPACITY;   // frames index gridDim.y
  if (c->arch == 1 && c->temporal_patch >= 1 && c->max_frames_total < c->temporal_patch) return ET_ERR_INVALID_ARG;
  const long long L = (long long)(c->image_size / c->patch_size) * (c->image_size / c->patch_size);
  if (L > 4096 || L * c->max_frames_total > (1ll << 30)) return ET_ERR_CAPACITY;
  if (!(c->ln_eps > 0.f)) return ET_ERR_INVALID_ARG;
  if (c->arch == 0) {
    if (c->temporal_patch > 1 || c->window != 0) return ET_ERR_INVALID_ARG;
  } else if (c->arch == 1) {
    const int g = c->image_size / c->patch_size, dh = c->hidden / c->heads;
    if (c->temporal_patch < 1 || c->temporal_patch > 8 || c->window < 0) return ET_ERR_INVALID_ARG;
    if (dh % 4 != 0 || !(c->rope_theta > 1.f)) return ET_ERR_SHAPE;
    if (c->window > 0) {
      if (g % c->window != 0) return ET_ERR_SHAPE;                                  // whole windows only
      if (!((c->full_attn_mask >> (c->num_layers - 1)) & 1ull)) return ET_ERR_SHAPE; // Stage II needs whole-frame scores
    }
  } else {
    return ET_ERR_INVALID_ARG;
  }
  return ET_OK;
}

et_status validate_params(const et_encoder* e, const et_params* p) {
  if (!p) return ET_ERR_INVALID_ARG;
  if (p->num_merge_layers < 0 || p->num_merge_layers > ET_MAX_MERGE_LAYERS) return ET_ERR_INVALID_ARG;
  for (int i = 0; i < p->num_merge_layers; ++i) {
    if (p->merge_layers[i] < 1 || p->merge_layers[i] > e->cfg.num_layers - 1) return ET_ERR_INVALID_ARG;
    if (i > 0 && p->merge_layers[i] <= p->merge_layers[i - 1]) return ET_ERR_INVALID_ARG;
  }
  if (!(p->ema_alpha > 0.0 && p->ema_alpha <= 1.0)) return ET_ERR_INVALID_ARG;
  if (!(p->retain > 0.0 && p->retain <= 1.0)) return ET_ERR_INVALID_ARG;
  if (isnan(p->tau_seg) || isnan(p->tau_merge)) return ET_ERR_INVALID_ARG;
  if (p->selection < 0 || p->selection > 3) return ET_ERR_INVALID_ARG;
  if (p->retain_mode < 0 || p->retain_mode > 1) return ET_ERR_INVALID_ARG;
  if (p->window_mode < 0 || p->window_mode > 1) return ET_ERR_INVALID_ARG;
  return ET_OK;
}

// One dense layer of the encoder on the arithmetic path the encoder was created with.
et_status dense(et_encoder* e, const void* a, const TmaDesc& da, const float* w_f32, const WeightDesc& dw,
                const TmaDesc& dc, const float* bias, void* c, int M_cap, int N, int K, int epi, const float* table, int table_rows,
                const int* n_dev, cudaStream_t s) {
  if (e->bf) {
    ET_CUDA(e, launch_gemm_bf16(da, dw, dc, bias, c, M_cap, N, K, epi, e->cfg.gelu_tanh, table, table_rows, n_dev, e->L,
                                e->d_small + 10, s));
  } else {
    launch_gemm_f32((const float*)a, w_f32, bias, (float*)c, M_cap, N, K, epi, e->cfg.gelu_tanh, table, table_rows,
                    n_dev, e->L, s);
  }
  return ET_OK;
}

SimPlanArgs sim_plan_args(et_encoder* e, const float* x, int n_cap, int lst, int V, const PlanArgs& plan) {
  SimPlanArgs a{};
  a.x = x; a.sim = e->simbuf; a.n_cap = n_cap; a.L = e->L; a.D = e->cfg.hidden;
  a.n_frames_dev = e->fl[lst].n; a.vid_off = e->fl[lst].vid_off; a.n_videos = V;
  a.acc = e->sim_acc; a.done = reinterpret_cast<unsigned*>(e->sim_acc + (similarity_plan_words(e->Fmax) - 1));
  a.plan = plan;
  return a;
}

et_status encode_finish(et_encoder* e, const et_params* p, int V, int T, int slot_idx, cudaStream_t s, et_result* out);

// slot_idx selects the result buffers; with defer the call returns after enqueueing its work (the caller waits for
// slot.ev_done and then calls encode_finish).
et_status encode_impl(et_encoder* e, const float* frames_dev, const int* vid_off_host, int V, const et_params* p,
                      cudaStream_t s, et_result* out, int slot_idx = 0, bool defer = false) {
  if (!e || !frames_dev || !vid_off_host || (!out && !defer)) return fail(e, ET_ERR_INVALID_ARG, "null argument");
  et_encoder::HostSlot& sl = e->slot[slot_idx];
  if (!defer && (e->slot[0].busy || e->slot[1].busy))
    return fail(e, ET_ERR_INVALID_ARG, "a submitted call has not been collected yet");
  ET_TRY(validate_params(e, p) == ET_OK ? ET_OK : fail(e, ET_ERR_INVALID_ARG, "invalid et_params"));
  if (V < 1 || V > e->Vmax) return fail(e, ET_ERR_CAPACITY, "number of videos outside [1, max_videos]");
  if (vid_off_host[0] != 0) return fail(e, ET_ERR_INVALID_ARG, "video_offsets[0] must be 0");
  for (int v = 0; v < V; ++v) {
    if (vid_off_host[v + 1] <= vid_off_host[v]) return fail(e, ET_ERR_INVALID_ARG, "every video needs at least one frame");
    if (vid_off_host[v + 1] % e->tp != 0) return fail(e, ET_ERR_INVALID_ARG, "frame counts must be multiples of temporal_patch");
  }
  // From here on a frame is an ENCODER frame (temporal_patch input frames; the same thing when temporal_patch is 1).
  const int T = vid_off_host[V] / e->tp;
  if (T > e->Fmax) return fail(e, ET_ERR_CAPACITY, "more frames than max_frames_total");
  const et_forced_plan* fp = p->forced_plan;
  if (fp) {
    for (int i = 0; i < p->num_merge_layers; ++i) {
      if (!fp->seg_start[i] || !fp->merge_next[i] || fp->n_in[i] < 1 || fp->n_in[i] > T)
        return fail(e, ET_ERR_INVALID_ARG, "forced plan: missing or oversized layer entry");
      for (int t = 0; t < fp->n_in[i]; ++t)
        if (fp->merge_next[i][t] && (t + 1 >= fp->n_in[i] || fp->merge_next[i][t + 1]))
          return fail(e, ET_ERR_INVALID_ARG, "forced plan: overlapping or dangling merge pair");
    }
    if (fp->keep && (fp->n_final < 1 || fp->n_final > T)) return fail(e, ET_ERR_INVALID_ARG, "forced plan: n_final");
  }
  ET_CUDA(e, cudaSetDevice(e->device));

  const et_config& c = e->cfg;
  const int L = e->L, D = c.hidden, Mlp = c.mlp_dim, H = c.heads, dh = e->dh;
  const int rows_cap = T * L;
  const float* W = e->w_blob;

  for (int v = 0; v <= V; ++v) sl.h_vid_off[v] = vid_off_host[v] / e->tp;
  ET_CUDA(e, cudaMemcpyAsync(e->orig_vid_off, sl.h_vid_off, sizeof(int) * (V + 1), cudaMemcpyHostToDevice, s));
  ET_CUDA(e, cudaMemsetAsync(e->d_small, 0, sizeof(int) * 16, s));
  if (fp) {
    for (int i = 0; i < p->num_merge_layers; ++i) {
      unsigned char* hs = e->h_forced + (size_t)(2 * i) * e->Fmax;
      unsigned char* hm = e->h_forced + (size_t)(2 * i + 1) * e->Fmax;
      memcpy(hs, fp->seg_start[i], fp->n_in[i]);
      memcpy(hm, fp->merge_next[i], fp->n_in[i]);
      ET_CUDA(e, cudaMemcpyAsync(e->forced_seg[i], hs, fp->n_in[i], cudaMemcpyHostToDevice, s));
      ET_CUDA(e, cudaMemcpyAsync(e->forced_mrg[i], hm, fp->n_in[i], cudaMemcpyHostToDevice, s));
    }
  }
  e->prof_spans.clear();
  e->prof_next_event = 0;
  int lst = 0, cur = 0;
  launch_init_frames(e->fl[0], e->orig_vid_off, V, T, s);

  // patch embedding: im2col + dense layer with the position table added in the epilogue
  const bool qw = e->arch == 1;           // Qwen2.5-VL-style blocks
  PROF(ET_CAT_IM2COL, launch_im2col(frames_dev, e->Pm, T, c.image_size, c.patch_size, e->Kp, e->bf, nullptr, s, e->tp, e->int2raster, e->raster2int));
  PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Pm, e->d_Pm, W + e->off_patch_w, e->d_patch_w, e->c_X[cur], qw ? e->zeros : W + e->off_patch_b, e->X[cur], rows_cap, D,
               e->bf ? e->Kp : e->P, EPI_TABLE, qw ? e->zeros : W + e->off_pos, qw ? 1 : L, nullptr, s)));
  if (e->ws > 0) launch_scale_count(e->fl[0].n, e->wpf, e->n_windows, s);

  int mi = 0;
  for (int layer = 0; layer < c.num_layers; ++layer) {
    if (mi < p->num_merge_layers && p->merge_layers[mi] == layer) {
      // Stage I at this block: similarities + plan (one launch) -> weighted merge + compaction
      PlanArgs a{};
      a.sim = e->simbuf; a.cur = e->fl[lst]; a.nxt = e->fl[lst ^ 1]; a.plan = e->plan; a.trace = e->tr[mi];
      a.forced_seg_start = fp ? e->forced_seg[mi] : nullptr;
      a.forced_merge_next = fp ? e->forced_mrg[mi] : nullptr;
      a.forced_n_in = fp ? fp->n_in[mi] : 0;
      a.alpha = p->ema_alpha; a.tau_seg = p->tau_seg; a.tau_merge = p->tau_merge;
      a.weighted = p->weighted_merge; a.allow_merge = 1; a.n_videos = V;
      a.n_hist_slot = e->d_small + 2 + mi; a.status = e->d_small + 10;
      PROF(ET_CAT_SIMILARITY, launch_similarity_plan(sim_plan_args(e, e->X[cur], T, lst, V, a), s));
      PROF(ET_CAT_MERGE, launch_merge_frames(e->X[cur], e->X[cur ^ 1], T, L * D, e->fl[lst ^ 1].n, e->plan, s));
      if (e->ws > 0) launch_scale_count(e->fl[lst ^ 1].n, e->wpf, e->n_windows, s);
      cur ^= 1; lst ^= 1; ++mi;
    }
    const int* n_dev = e->fl[lst].n;
    const LayerOffsets& o = e->lo[layer];
    const LayerBf16* b = e->bf ? &e->lb[layer] : nullptr;
    static const WeightDesc none{};
    PROF(ET_CAT_LAYERNORM, launch_layernorm(e->X[cur], W + o.ln1_g, qw ? nullptr : W + o.ln1_b, c.ln_eps, e->Xn, rows_cap, D, e->bf, n_dev, L, s));
    PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Xn, e->d_Xn, W + o.wqkv, b ? b->d_wqkv : none, e->c_QKV, W + o.bqkv, e->QKV, rows_cap, 3 * D, D, EPI_STORE,
                 nullptr, 1, n_dev, s)));
    if (qw) PROF(ET_CAT_ATTENTION, launch_rope_pairs(e->QKV, e->rope_table, rows_cap, L, H, dh, e->bf, n_dev, s));
    // attention items: whole frames, or (in a window block) the windows, which are runs of Lw rows in the internal order
    const bool windowed = e->ws > 0 && !((c.full_attn_mask >> layer) & 1ull);
    const int a_cap = windowed ? T * e->wpf : T, a_L = windowed ? e->Lw : L;
    const int* a_n = windowed ? e->n_windows : n_dev;
    PROF(ET_CAT_ATTENTION, {
      // the tensor-core kernel sweeps whole frames and masks the keys outside a query's window
      if (e->attn_tc) ET_CUDA(e, launch_attention_tc(e->attn_maps, e->lse, T, L, H, dh, n_dev, e->d_small + 10, s, windowed ? e->Lw : 0));
      else if (e->bf) launch_attention_bf16((const bf16*)e->QKV, (bf16*)e->O, e->lse, a_cap, a_L, H, dh, a_n, s);
      else launch_attention_f32((const float*)e->QKV, (float*)e->O, e->lse, a_cap, a_L, H, dh, a_n, s);
    });
    if (layer == c.num_layers - 1) {
      PROF(ET_CAT_SCORES, {
        if (e->scores_tc) ET_CUDA(e, launch_attention_scores_tc(e->attn_maps, e->lse, e->score_partial, e->scores, T, L, H, dh, n_dev, e->d_small + 10, s));
        else if (e->bf) launch_attention_scores_bf16((const bf16*)e->QKV, e->lse, e->score_partial, e->scores, T, L, H, dh, n_dev, s);
        else launch_attention_scores_f32((const float*)e->QKV, e->lse, e->score_partial, e->scores, T, L, H, dh, n_dev, s);
      });
    }
    PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->O, e->d_O, W + o.wo, b ? b->d_wo : none, e->c_X[cur], W + o.bo, e->X[cur], rows_cap, D, D, EPI_RESIDUAL,
                 nullptr, 1, n_dev, s)));
    PROF(ET_CAT_LAYERNORM, launch_layernorm(e->X[cur], W + o.ln2_g, qw ? nullptr : W + o.ln2_b, c.ln_eps, e->Xn, rows_cap, D, e->bf, n_dev, L, s));
    if (qw) {
      // gated MLP: [gate | up] pre-activations, silu(gate) * up, down projection added to the residual stream
      const int Mp = e->Mp;
      if (e->bf) {
        PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Xn, e->d_Xn, nullptr, b->d_w1, e->c_Hm, e->bgu_pad + (size_t)layer * 2 * Mp, e->Hm, rows_cap,
                     2 * Mp, D, EPI_SWIGLU, nullptr, 1, n_dev, s)));
      } else {
        PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Xn, e->d_Xn, W + o.w1, none, e->c_Hm, W + o.b1, e->GU, rows_cap, 2 * Mp, D, EPI_STORE, nullptr, 1,
                     n_dev, s)));
        PROF(ET_CAT_GEMM, launch_gated_silu(e->GU, e->Hm, rows_cap, Mp, false, n_dev, L, s));
      }
      PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Hm, e->d_Hm, W + o.w2, b ? b->d_w2 : none, e->c_X[cur], W + o.b2, e->X[cur], rows_cap, D, Mp, EPI_RESIDUAL,
                   nullptr, 1, n_dev, s)));
    } else {
      PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Xn, e->d_Xn, W + o.w1, b ? b->d_w1 : none, e->c_Hm, W + o.b1, e->Hm, rows_cap, Mlp, D, EPI_GELU, nullptr, 1,
                   n_dev, s)));
      PROF(ET_CAT_GEMM, ET_TRY(dense(e, e->Hm, e->d_Hm, W + o.w2, b ? b->d_w2 : none, e->c_X[cur], W + o.b2, e->X[cur], rows_cap, D, Mlp, EPI_RESIDUAL,
                   nullptr, 1, n_dev, s)));
    }
  }
  const int* n_dev = e->fl[lst].n;
  if (p->num_merge_layers == 0) {
    // Stage I off: the segment list of Stage II comes from the streaming segmentation of the final features
    PlanArgs a{};
    a.sim = e->simbuf; a.cur = e->fl[lst]; a.nxt = e->fl[lst ^ 1]; a.plan = e->plan; a.trace = e->tr[0];
    a.alpha = p->ema_alpha; a.tau_seg = p->tau_seg; a.tau_merge = p->tau_merge;
    a.weighted = p->weighted_merge; a.allow_merge = 0; a.n_videos = V; a.status = e->d_small + 10;
    PROF(ET_CAT_SIMILARITY, launch_similarity_plan(sim_plan_args(e, e->X[cur], T, lst, V, a), s));
  }
  // Stage II: amounts, flags and mask in one launch; offsets, totals and the gather in another
  SelectArgs sa{};
  sa.scores = e->scores; sa.fl = e->fl[lst]; sa.orig_vid_off = e->orig_vid_off; sa.n_cap = T; sa.n_videos = V; sa.L = L;
  sa.selection = p->selection; sa.retain_mode = p->retain_mode; sa.window_mode = p->window_mode; sa.retain = p->retain;
  sa.dynamic = e->dynamic; sa.keep = e->keep; sa.count = e->count; sa.video_k = e->video_k; sa.video_w = e->video_w;
  sa.raster2int = e->raster2int;
  if (fp && fp->keep) {
    memcpy(e->h_keep_stage, fp->keep, (size_t)fp->n_final * L);
    ET_CUDA(e, cudaMemcpyAsync(e->keep, e->h_keep_stage, (size_t)fp->n_final * L, cudaMemcpyHostToDevice, s));
    sa.mask_given = 1;
    PROF(ET_CAT_SELECT, launch_select_video_tokens(sa, s));
    PROF(ET_CAT_SELECT, launch_count_keep(e->keep, T, L, e->count, n_dev, s));
  } else {
    if (p->selection == 3) {          // random sampling: rank uniform numbers instead of attention scores
      PROF(ET_CAT_SELECT, launch_random_scores(e->score_partial, e->fl[lst].vid_off, V, T, L, p->sample_seed, n_dev, s));
      sa.scores = e->score_partial;
    }
    PROF(ET_CAT_SELECT, launch_select_video_tokens(sa, s));
  }
  PROF(ET_CAT_GATHER, launch_gather_tokens(e->X[cur], e->keep, e->count, sl.frame_offsets, e->d_small, T, L, D,
                       c.post_layernorm ? W + e->off_post_g : nullptr, (c.post_layernorm && !qw) ? W + e->off_post_b : nullptr,
                       c.ln_eps, sl.tokens, sl.token_pos, n_dev, s, e->raster2int));
  // per-frame results of this call: the frame list and flags are overwritten early in the next call
  ET_CUDA(e, cudaMemcpyAsync(sl.src_lo, e->fl[lst].src_lo, sizeof(int) * T, cudaMemcpyDeviceToDevice, s));
  ET_CUDA(e, cudaMemcpyAsync(sl.src_hi, e->fl[lst].src_hi, sizeof(int) * T, cudaMemcpyDeviceToDevice, s));
  ET_CUDA(e, cudaMemcpyAsync(sl.dynamic, e->dynamic, T, cudaMemcpyDeviceToDevice, s));
  ET_CUDA(e, cudaMemcpyAsync(sl.vfo, e->fl[lst].vid_off, sizeof(int) * (V + 1), cudaMemcpyDeviceToDevice, s));
  ET_CUDA(e, cudaMemcpyAsync(sl.h_small, e->d_small, sizeof(int) * 16, cudaMemcpyDeviceToHost, s));
  ET_CUDA(e, cudaGetLastError());
  if (defer) {
    ET_CUDA(e, cudaEventRecord(sl.ev_done, s));
    return ET_OK;
  }
  ET_CUDA(e, cudaStreamSynchronize(s));
  return encode_finish(e, p, V, T, slot_idx, s, out);
}

// After the call's work has completed: status, sizes, result struct, profile counters, trace.
et_status encode_finish(et_encoder* e, const et_params* p, int V, int T, int slot_idx, cudaStream_t s, et_result* out) {
  et_encoder::HostSlot& sl = e->slot[slot_idx];
  const et_config& c = e->cfg;
  const int L = e->L, D = c.hidden, Mlp = c.mlp_dim;
  const et_forced_plan* fp = p->forced_plan;
  const bool qw = e->arch == 1;
  const int status = sl.h_small[10];
  if (status == DS_WAIT_EXPIRED) return fail(e, ET_ERR_TIMEOUT, "a bounded device-side wait expired in a tensor-core kernel");
  if (status == DS_FORCED_MISMATCH) return fail(e, ET_ERR_INVALID_ARG, "forced plan does not fit the frame list");
  if (status != 0) return fail(e, ET_ERR_CUDA, "device status " + std::to_string(status));
  const int N = sl.h_small[0], n_tok = sl.h_small[1];
  if (fp && fp->keep && fp->n_final != N) return fail(e, ET_ERR_INVALID_ARG, "forced plan: n_final does not match");

  et_result r{};
  r.n_videos = V; r.n_frames_in = T; r.n_frames_out = N; r.n_tokens = n_tok; r.hidden = D; r.tokens_per_frame = L;
  r.tokens = sl.tokens; r.video_frame_offsets = sl.vfo; r.frame_offsets = sl.frame_offsets;
  r.frame_src_lo = sl.src_lo; r.frame_src_hi = sl.src_hi; r.frame_dynamic = sl.dynamic;
  r.token_pos = sl.token_pos; r.trace = nullptr;
  {
    int alive = T, m = 0;
    for (int layer = 0; layer < c.num_layers; ++layer) {
      if (m < p->num_merge_layers && p->merge_layers[m] == layer) { alive = sl.h_small[2 + m]; ++m; }
      r.frames_per_block[layer] = alive;
    }
  }
  if (e->prof_on) {
    for (const et_encoder::Span& sp : e->prof_spans) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, e->prof_events[sp.ev], e->prof_events[sp.ev + 1]) == cudaSuccess) e->prof.ms[sp.cat] += ms;
      e->prof.launches[sp.cat] += sp.launches1 - sp.launches0;
    }
    // algorithmic work of this call from the frame counts it actually ran with
    const double dL = L, dD = D, dM = Mlp, es = e->bf ? 2.0 : 4.0;
    double* wk = e->prof.work;
    wk[ET_CAT_IM2COL] += (double)T * e->tp * 3.0 * c.image_size * c.image_size * 4.0 + (double)T * dL * e->Kp * es;
    wk[ET_CAT_GEMM] += 2.0 * T * dL * dD * e->P;
    int n_in = T;
    for (int layer = 0, m = 0; layer < c.num_layers; ++layer) {
      if (m < p->num_merge_layers && p->merge_layers[m] == layer) {
        const int n_out = sl.h_small[2 + m];
        wk[ET_CAT_SIMILARITY] += (double)n_in * dL * dD * 4.0;
        wk[ET_CAT_MERGE] += ((double)n_in + n_out) * dL * dD * 4.0;
        n_in = n_out; ++m;
      }
      const double rows = (double)r.frames_per_block[layer] * dL;
      const bool windowed = e->ws > 0 && !((c.full_attn_mask >> layer) & 1ull);
      wk[ET_CAT_GEMM] += 2.0 * rows * (4.0 * dD * dD + (qw ? 3.0 : 2.0) * dD * dM);
      wk[ET_CAT_ATTENTION] += 4.0 * rows * (windowed ? (double)e->Lw : dL) * dD;
      wk[ET_CAT_LAYERNORM] += 2.0 * rows * dD * (4.0 + es);
    }
    if (p->num_merge_layers == 0) wk[ET_CAT_SIMILARITY] += (double)N * dL * dD * 4.0;
    wk[ET_CAT_SCORES] += 2.0 * N * dL * dL * dD;
    wk[ET_CAT_SELECT] += (double)N * dL * 5.0;
    wk[ET_CAT_GATHER] += 2.0 * n_tok * dD * 4.0;
    e->prof.calls += 1;
  }
  if (p->want_trace) {
    et_trace& t = e->trace;
    memset(&t, 0, sizeof(t));
    t.num_merge_layers = p->num_merge_layers;
    int n_in = T;
    for (int i = 0; i < p->num_merge_layers; ++i) {
      t.n_in[i] = n_in; t.n_out[i] = sl.h_small[2 + i];
      float* hs = e->h_tr_f + (size_t)(2 * i) * e->Fmax;
      float* he = e->h_tr_f + (size_t)(2 * i + 1) * e->Fmax;
      unsigned char* hb = e->h_tr_b + (size_t)(2 * i) * e->Fmax;
      unsigned char* hm = e->h_tr_b + (size_t)(2 * i + 1) * e->Fmax;
      ET_CUDA(e, cudaMemcpyAsync(hs, e->tr[i].sim, sizeof(float) * n_in, cudaMemcpyDeviceToHost, s));
      ET_CUDA(e, cudaMemcpyAsync(he, e->tr[i].ema, sizeof(float) * n_in, cudaMemcpyDeviceToHost, s));
      ET_CUDA(e, cudaMemcpyAsync(hb, e->tr[i].seg_start, n_in, cudaMemcpyDeviceToHost, s));
      ET_CUDA(e, cudaMemcpyAsync(hm, e->tr[i].merge_next, n_in, cudaMemcpyDeviceToHost, s));
      t.sim[i] = hs; t.ema[i] = he; t.seg_start[i] = hb; t.merge_next[i] = hm;
      n_in = t.n_out[i];
    }
    ET_CUDA(e, cudaMemcpyAsync(e->raster2int ? e->h_scores_int : e->h_scores, e->scores, sizeof(float) * (size_t)N * L, cudaMemcpyDeviceToHost, s));
    ET_CUDA(e, cudaMemcpyAsync(e->h_keep, e->keep, (size_t)N * L, cudaMemcpyDeviceToHost, s));
    ET_CUDA(e, cudaMemcpyAsync(e->h_video_kw, e->video_k, sizeof(int) * V, cudaMemcpyDeviceToHost, s));
    ET_CUDA(e, cudaMemcpyAsync(e->h_video_kw + e->Vmax, e->video_w, sizeof(int) * V, cudaMemcpyDeviceToHost, s));
    ET_CUDA(e, cudaStreamSynchronize(s));
    if (e->raster2int) {                // the device holds the scores in the internal token order; the trace is in raster order
      for (int f = 0; f < N; ++f)
        for (int j = 0; j < L; ++j) e->h_scores[(size_t)f * L + j] = e->h_scores_int[(size_t)f * L + e->r2i_host[j]];
    }
    t.scores = e->h_scores; t.keep = e->h_keep; t.video_k = e->h_video_kw; t.video_w = e->h_video_kw + e->Vmax;
    r.trace = &t;
  }
  *out = r;
  return ET_OK;
}

}  // namespace

extern "C" {

et_status et_encoder_create(const et_config* config, const et_weights* weights, et_encoder** out) {
  if (!config || !weights || !weights->data || !out) return ET_ERR_INVALID_ARG;
  et_status st = validate_config(config);
  if (st != ET_OK) return st;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return ET_ERR_CUDA;
  const int g = config->image_size / config->patch_size;
  const int tp = config->arch == 1 ? config->temporal_patch : 1;
  const int L = g * g, P = 3 * tp * config->patch_size * config->patch_size;
  if (weights->count != blob_floats(*config, L, P)) return ET_ERR_WEIGHTS;

  et_encoder* e = new (std::nothrow) et_encoder();
  if (!e) return ET_ERR_OOM;
  auto bail = [&](et_status s) { et_destroy(e); return s; };
  e->cfg = *config;
  e->L = L; e->grid = g; e->P = P; e->dh = config->hidden / config->heads;
  e->bf = config->dtype == ET_BF16;
  e->Kp = e->bf ? (P + 7) / 8 * 8 : P;
  e->arch = config->arch; e->tp = tp;
  e->ws = config->arch == 1 ? config->window : 0;
  e->wpf = e->ws > 0 ? (g / e->ws) * (g / e->ws) : 1;
  e->Lw = e->ws > 0 ? e->ws * e->ws : L;
  e->Mp = (config->arch == 1 && e->bf) ? (config->mlp_dim + 127) / 128 * 128 : config->mlp_dim;   // whole 128-output tiles
  e->Fmax = config->max_frames_total / tp; e->Vmax = config->max_videos;
  if (cudaGetDevice(&e->device) != cudaSuccess) return bail(ET_ERR_CUDA);
  const size_t D = config->hidden, M = config->mlp_dim, F = e->Fmax, rows = F * (size_t)L;
  const size_t Mp = e->Mp;

  // ---- weights
  {
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off += n; return o; };
    e->lo.resize(config->num_layers);
    if (e->arch == 1) {
      e->off_patch_w = take((size_t)P * D);
      for (auto& o : e->lo) {
        o.ln1_g = take(D); o.ln1_b = 0; o.wqkv = take(D * 3 * D); o.bqkv = take(3 * D);
        o.wo = take(D * D); o.bo = take(D); o.ln2_g = take(D); o.ln2_b = 0;
        o.w1 = take(D * 2 * M); o.b1 = take(2 * M); o.w2 = take(M * D); o.b2 = take(D);
      }
      e->off_post_g = take(D);
    } else {
      e->off_patch_w = take((size_t)P * D); e->off_patch_b = take(D); e->off_pos = take((size_t)L * D);
      for (auto& o : e->lo) {
        o.ln1_g = take(D); o.ln1_b = take(D); o.wqkv = take(D * 3 * D); o.bqkv = take(3 * D);
        o.wo = take(D * D); o.bo = take(D); o.ln2_g = take(D); o.ln2_b = take(D);
        o.w1 = take(D * M); o.b1 = take(M); o.w2 = take(M * D); o.b2 = take(D);
      }
      e->off_post_g = take(D); e->off_post_b = take(D);
    }
  }
  if ((st = dalloc(e, &e->w_blob, weights->count)) != ET_OK) return bail(st);
  if (cudaMemcpy(e->w_blob, weights->data, weights->count * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
    return bail(ET_ERR_CUDA);
  {
    int* flag = nullptr;
    int bad = 0;
    if ((st = dalloc(e, &flag, 1)) != ET_OK) return bail(st);
    cudaMemset(flag, 0, sizeof(int));
    ET_COUNT_LAUNCH();
    find_nonfinite_kernel<<<148 * 8, 256>>>(e->w_blob, weights->count, flag);
    if (cudaMemcpy(&bad, flag, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return bail(ET_ERR_CUDA);
    if (bad) return bail(ET_ERR_WEIGHTS);
  }
  const size_t es = e->bf ? 2 : 4;
  // ---- activations
#define ET_A(ptr, bytes)                                                     \
  do {                                                                       \
    unsigned char* q__ = nullptr;                                            \
    if ((st = dalloc(e, &q__, (bytes))) != ET_OK) return bail(st);           \
    ptr = reinterpret_cast<decltype(ptr)>(q__);                              \
  } while (0)
  ET_A(e->X[0], rows * D * 4); ET_A(e->X[1], rows * D * 4);
  ET_A(e->Pm, rows * e->Kp * es); ET_A(e->Xn, rows * D * es); ET_A(e->QKV, rows * 3 * D * es);
  ET_A(e->O, rows * D * es); ET_A(e->Hm, rows * Mp * es);
  if (e->arch == 1) {
    if (!e->bf) ET_A(e->GU, rows * 2 * Mp * es);      // the tensor-core path applies the gate inside the dense layer
    ET_A(e->zeros, std::max(D, 2 * Mp) * 4);
    ET_A(e->n_windows, 4);
    cudaMemset(e->zeros, 0, std::max(D, 2 * Mp) * 4);
    // rotary table and token orders.  Internal order = window-major (windows row-major over the grid, tokens
    // row-major inside a window), so that a window is a run of Lw consecutive rows; raster order otherwise.
    std::vector<int> i2r(L), r2i(L);
    for (int l = 0; l < L; ++l) i2r[l] = l;
    if (e->ws > 0) {
      const int ws = e->ws, wr = g / ws;
      for (int l = 0; l < L; ++l) {
        const int win = l / (ws * ws), in = l % (ws * ws);
        i2r[l] = ((win / wr) * ws + in / ws) * g + (win % wr) * ws + in % ws;
      }
      ET_A(e->int2raster, (size_t)L * 4); ET_A(e->raster2int, (size_t)L * 4);
      for (int l = 0; l < L; ++l) r2i[i2r[l]] = l;
      cudaMemcpy(e->int2raster, i2r.data(), (size_t)L * 4, cudaMemcpyHostToDevice);
      cudaMemcpy(e->raster2int, r2i.data(), (size_t)L * 4, cudaMemcpyHostToDevice);
      e->r2i_host = r2i;
    }
    const int half = e->dh / 2, quarter = e->dh / 4;
    std::vector<float2> tab((size_t)L * half);
    for (int l = 0; l < L; ++l) {
      const int gy = i2r[l] / g, gx = i2r[l] % g;
      for (int i = 0; i < half; ++i) {
        const double freq = pow((double)config->rope_theta, -2.0 * (double)(i % quarter) / (double)half);
        const double ang = (double)(i < quarter ? gy : gx) * freq;
        tab[(size_t)l * half + i] = make_float2((float)cos(ang), (float)sin(ang));
      }
    }
    ET_A(e->rope_table, tab.size() * sizeof(float2));
    cudaMemcpy(e->rope_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice);
  }
  ET_A(e->lse, F * config->heads * L * 4); ET_A(e->score_partial, F * config->heads * L * 4);
  ET_A(e->scores, rows * 4); ET_A(e->simbuf, F * 4);
  for (int i = 0; i < 2; ++i) {
    ET_A(e->fl[i].n, 4); ET_A(e->fl[i].vid_off, (e->Vmax + 1) * 4); ET_A(e->fl[i].src_lo, F * 4);
    ET_A(e->fl[i].src_hi, F * 4); ET_A(e->fl[i].role, F);
  }
  ET_A(e->plan.src_a, F * 4); ET_A(e->plan.src_b, F * 4); ET_A(e->plan.w_a, F * 4); ET_A(e->plan.w_b, F * 4);
  for (int i = 0; i < ET_MAX_MERGE_LAYERS; ++i) {
    ET_A(e->tr[i].sim, F * 4); ET_A(e->tr[i].ema, F * 4); ET_A(e->tr[i].seg_start, F); ET_A(e->tr[i].merge_next, F);
    ET_A(e->forced_seg[i], F); ET_A(e->forced_mrg[i], F);
  }
  ET_A(e->orig_vid_off, (e->Vmax + 1) * 4);
  ET_A(e->dynamic, F); ET_A(e->keep, rows);
  ET_A(e->sim_acc, (size_t)similarity_plan_words(e->Fmax) * 8);
  ET_A(e->video_k, e->Vmax * 4); ET_A(e->video_w, e->Vmax * 4); ET_A(e->count, F * 4);
  ET_A(e->frame_offsets, (F + 1) * 4); ET_A(e->token_pos, rows * 4); ET_A(e->tokens, rows * D * 4);
  ET_A(e->d_small, 16 * 4);
#undef ET_A
  if ((st = halloc(e, &e->h_small, 16)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_vid_off, e->Vmax + 1)) != ET_OK) return bail(st);
  {
    et_encoder::HostSlot& s0 = e->slot[0];            // the slot of the synchronous calls: the regular result buffers
    s0.tokens = e->tokens; s0.token_pos = e->token_pos; s0.frame_offsets = e->frame_offsets;
    s0.h_small = e->h_small; s0.h_vid_off = e->h_vid_off;
    if ((st = dalloc(e, &s0.src_lo, F)) != ET_OK || (st = dalloc(e, &s0.src_hi, F)) != ET_OK ||
        (st = dalloc(e, &s0.dynamic, F)) != ET_OK || (st = dalloc(e, &s0.vfo, (size_t)e->Vmax + 1)) != ET_OK)
      return bail(st);
  }
  if ((st = halloc(e, &e->h_forced, 2 * ET_MAX_MERGE_LAYERS * F)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_keep_stage, rows)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_tr_f, 2 * ET_MAX_MERGE_LAYERS * F)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_tr_b, 2 * ET_MAX_MERGE_LAYERS * F)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_scores, rows)) != ET_OK) return bail(st);
  if (e->raster2int && (st = halloc(e, &e->h_scores_int, rows)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_keep, rows)) != ET_OK) return bail(st);
  if ((st = halloc(e, &e->h_video_kw, 2 * (size_t)e->Vmax)) != ET_OK) return bail(st);
  // zero the activation buffers once: rows beyond the live count are read (never stored) by tile loads
  cudaMemset(e->Pm, 0, rows * e->Kp * es); cudaMemset(e->Xn, 0, rows * D * es); cudaMemset(e->O, 0, rows * D * es);
  cudaMemset(e->Hm, 0, rows * Mp * es); cudaMemset(e->QKV, 0, rows * 3 * D * es);
  cudaMemset(e->sim_acc, 0, (size_t)similarity_plan_words(e->Fmax) * 8);

  if (e->bf) {
    // transposed bf16 copies of the dense weights ([out][in], K contiguous) + their tensor maps
    const char* err = nullptr;
    // gated_M > 0: the [gate | up] weight of a gated MLP, rows_out >= N rows in the fused epilogue's order (the rest zero)
    auto convert = [&](size_t off, int K, int N, int k_pad, bf16** dst, int rows_out = 0, int gated_M = 0) -> et_status {
      if (rows_out <= 0) rows_out = N;
      et_status s2 = dalloc(e, dst, (size_t)rows_out * k_pad);
      if (s2 != ET_OK) return s2;
      if (rows_out != N && cudaMemset(*dst, 0, (size_t)rows_out * k_pad * sizeof(bf16)) != cudaSuccess) return ET_ERR_CUDA;
      ET_COUNT_LAUNCH();
      transpose_to_bf16_kernel<<<dim3(cdiv(N, 32), cdiv(k_pad, 32)), dim3(32, 8)>>>(e->w_blob + off, *dst, K, N, k_pad, gated_M);
      return cudaGetLastError() == cudaSuccess ? ET_OK : ET_ERR_CUDA;
    };
    if ((st = convert(e->off_patch_w, P, (int)D, e->Kp, &e->patch_w_t)) != ET_OK) return bail(st);
    if (!make_tma_weight(&e->d_patch_w, e->patch_w_t, D, e->Kp, &err)) return bail(fail(e, ET_ERR_CUDA, err));
    e->lb.resize(config->num_layers);
    for (int i = 0; i < config->num_layers; ++i) {
      LayerBf16& b = e->lb[i];
      const LayerOffsets& o = e->lo[i];
      if ((st = convert(o.wqkv, (int)D, (int)(3 * D), (int)D, &b.wqkv_t)) != ET_OK) return bail(st);
      if ((st = convert(o.wo, (int)D, (int)D, (int)D, &b.wo_t)) != ET_OK) return bail(st);
      if (e->arch == 1) {
        // [gate | up]: 2M source columns -> 2*Mp rows in the fused epilogue's order; down: K padded to Mp
        if ((st = convert(o.w1, (int)D, (int)(2 * M), (int)D, &b.w1_t, (int)(2 * Mp), (int)M)) != ET_OK) return bail(st);
        if ((st = convert(o.w2, (int)M, (int)D, (int)Mp, &b.w2_t)) != ET_OK) return bail(st);
      } else {
        if ((st = convert(o.w1, (int)D, (int)M, (int)D, &b.w1_t)) != ET_OK) return bail(st);
        if ((st = convert(o.w2, (int)M, (int)D, (int)M, &b.w2_t)) != ET_OK) return bail(st);
      }
      bool ok = make_tma_weight(&b.d_wqkv, b.wqkv_t, 3 * D, D, &err) &&
                make_tma_weight(&b.d_wo, b.wo_t, D, D, &err) &&
                make_tma_weight(&b.d_w1, b.w1_t, e->arch == 1 ? 2 * Mp : M, D, &err) &&
                make_tma_weight(&b.d_w2, b.w2_t, D, Mp, &err);
      if (!ok) return bail(fail(e, ET_ERR_CUDA, err ? err : "tensor map"));
    }
    bool ok = make_tma_2d_bf16(&e->d_Pm, e->Pm, rows, e->Kp, 128, &err) && make_tma_2d_bf16(&e->d_Xn, e->Xn, rows, D, 128, &err) &&
              make_tma_2d_bf16(&e->d_O, e->O, rows, D, 128, &err) && make_tma_2d_bf16(&e->d_Hm, e->Hm, rows, Mp, 128, &err) &&
              make_tma_out(&e->c_X[0], e->X[0], rows, D, true, &err) && make_tma_out(&e->c_X[1], e->X[1], rows, D, true, &err) &&
              make_tma_out(&e->c_QKV, e->QKV, rows, 3 * D, false, &err) && make_tma_out(&e->c_Hm, e->Hm, rows, Mp, false, &err);
    if (!ok) return bail(fail(e, ET_ERR_CUDA, err ? err : "tensor map"));
    if (e->arch == 1) {
      // gate | up biases in the order of the weight rows
      std::vector<float> hb((size_t)config->num_layers * 2 * Mp, 0.f);
      for (int i = 0; i < config->num_layers; ++i) {
        const float* src = weights->data + e->lo[i].b1;
        float* dst = hb.data() + (size_t)i * 2 * Mp;
        for (size_t j = 0; j < M; ++j) { dst[gated_row((int)j, 0)] = src[j]; dst[gated_row((int)j, 1)] = src[M + j]; }
      }
      if ((st = dalloc(e, &e->bgu_pad, hb.size())) != ET_OK) return bail(st);
      if (cudaMemcpy(e->bgu_pad, hb.data(), hb.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) return bail(ET_ERR_CUDA);
    }
    if (attention_tc_supported(e->dh)) {
      if (!make_attention_maps(&e->attn_maps, (const bf16*)e->QKV, (long long)rows, config->heads, e->dh, (bf16*)e->O, e->L))
        return bail(fail(e, ET_ERR_CUDA, "tensor map of the attention operands"));
      e->attn_tc = true;
      e->scores_tc = attention_scores_tc_supported(e->dh);
    }
  }
  if (cudaDeviceSynchronize() != cudaSuccess) return bail(ET_ERR_CUDA);
  *out = e;
  return ET_OK;
}

void et_destroy(et_encoder* e) {
  if (!e) return;
  for (void* p : e->dev_allocs) cudaFree(p);
  for (void* p : e->host_allocs) cudaFreeHost(p);
  for (cudaEvent_t ev : e->prof_events) cudaEventDestroy(ev);
  for (auto& sl : e->slot)
    for (cudaEvent_t ev : {sl.ev_h2d, sl.ev_done})
      if (ev) cudaEventDestroy(ev);
  if (e->h2d_stream) cudaStreamDestroy(e->h2d_stream);
  if (e->d2h_stream) cudaStreamDestroy(e->d2h_stream);
  delete e;
}

et_status et_encode_batch(et_encoder* enc, const float* frames_dev, const int* video_offsets_host, int V,
                          const et_params* params, void* cuda_stream, et_result* out) {
  return encode_impl(enc, frames_dev, video_offsets_host, V, params, (cudaStream_t)cuda_stream, out);
}

et_status et_encode_video(et_encoder* enc, const float* frames_dev, int T, const et_params* params, void* cuda_stream,
                          et_result* out) {
  if (T < 1) return fail(enc, ET_ERR_INVALID_ARG, "T < 1");
  const int offs[2] = {0, T};
  return encode_impl(enc, frames_dev, offs, 1, params, (cudaStream_t)cuda_stream, out);
}

}  // extern "C"

namespace {

// D2H of one call's results from its slot into the caller's host buffers, on stream s (not synchronised here)
et_status copy_result_to_host(et_encoder* e, const et_result& r, int V, const et_host_buffers* dst, cudaStream_t s) {
  if ((size_t)r.n_tokens > dst->capacity_tokens || (size_t)r.n_frames_out > dst->capacity_frames)
    return fail(e, ET_ERR_CAPACITY, "host buffers too small for the result");
  const size_t N = r.n_frames_out, nt = r.n_tokens;
  if (dst->tokens) ET_CUDA(e, cudaMemcpyAsync(dst->tokens, r.tokens, nt * r.hidden * sizeof(float), cudaMemcpyDeviceToHost, s));
  if (dst->token_pos) ET_CUDA(e, cudaMemcpyAsync(dst->token_pos, r.token_pos, nt * sizeof(int), cudaMemcpyDeviceToHost, s));
  if (dst->frame_offsets) ET_CUDA(e, cudaMemcpyAsync(dst->frame_offsets, r.frame_offsets, (N + 1) * sizeof(int), cudaMemcpyDeviceToHost, s));
  if (dst->frame_src_lo) ET_CUDA(e, cudaMemcpyAsync(dst->frame_src_lo, r.frame_src_lo, N * sizeof(int), cudaMemcpyDeviceToHost, s));
  if (dst->frame_src_hi) ET_CUDA(e, cudaMemcpyAsync(dst->frame_src_hi, r.frame_src_hi, N * sizeof(int), cudaMemcpyDeviceToHost, s));
  if (dst->frame_dynamic) ET_CUDA(e, cudaMemcpyAsync(dst->frame_dynamic, r.frame_dynamic, N, cudaMemcpyDeviceToHost, s));
  if (dst->video_frame_offsets)
    ET_CUDA(e, cudaMemcpyAsync(dst->video_frame_offsets, r.video_frame_offsets, (V + 1) * sizeof(int), cudaMemcpyDeviceToHost, s));
  return ET_OK;
}

et_status check_host_call(et_encoder* e, const float* frames_host, const int* video_offsets_host, int V, const et_host_buffers* dst) {
  if (!e || !frames_host || !video_offsets_host || !dst) return fail(e, ET_ERR_INVALID_ARG, "null argument");
  if (V < 1 || V > e->Vmax) return fail(e, ET_ERR_CAPACITY, "number of videos outside [1, max_videos]");
  const int T = video_offsets_host[V];                     // input frames
  if (T < 1 || T > e->Fmax * e->tp) return fail(e, ET_ERR_CAPACITY, "frames outside [1, max_frames_total]");
  return ET_OK;
}

// Everything a slot needs beyond what create gave slot 0: frame staging, events, and for slot 1 result buffers of its own.
et_status prepare_slot(et_encoder* e, int idx, bool events) {
  et_encoder::HostSlot& sl = e->slot[idx];
  const size_t F = e->Fmax, rows = F * (size_t)e->L, D = e->cfg.hidden;
  const size_t frame_floats = (size_t)3 * e->cfg.image_size * e->cfg.image_size;
  if (!sl.frames_stage) ET_TRY(dalloc(e, &sl.frames_stage, F * e->tp * frame_floats));
  if (!sl.tokens) {
    ET_TRY(dalloc(e, &sl.tokens, rows * D)); ET_TRY(dalloc(e, &sl.token_pos, rows)); ET_TRY(dalloc(e, &sl.frame_offsets, F + 1));
    ET_TRY(dalloc(e, &sl.src_lo, F)); ET_TRY(dalloc(e, &sl.src_hi, F)); ET_TRY(dalloc(e, &sl.dynamic, F));
    ET_TRY(dalloc(e, &sl.vfo, (size_t)e->Vmax + 1));
    ET_TRY(halloc(e, &sl.h_small, 16)); ET_TRY(halloc(e, &sl.h_vid_off, (size_t)e->Vmax + 1));
  }
  if (events && !sl.ev_done) {
    ET_CUDA(e, cudaEventCreateWithFlags(&sl.ev_h2d, cudaEventDisableTiming));
    ET_CUDA(e, cudaEventCreateWithFlags(&sl.ev_done, cudaEventDisableTiming));
  }
  return ET_OK;
}

}  // namespace

extern "C" {

et_status et_encode_batch_host(et_encoder* e, const float* frames_host, const int* video_offsets_host, int V,
                               const et_params* params, void* cuda_stream, const et_host_buffers* dst, et_result* out) {
  if (!out) return fail(e, ET_ERR_INVALID_ARG, "null argument");
  ET_TRY(check_host_call(e, frames_host, video_offsets_host, V, dst));
  const int T = video_offsets_host[V];
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const size_t frame_floats = (size_t)3 * e->cfg.image_size * e->cfg.image_size;
  ET_CUDA(e, cudaSetDevice(e->device));
  ET_TRY(prepare_slot(e, 0, false));
  ET_CUDA(e, cudaMemcpyAsync(e->slot[0].frames_stage, frames_host, (size_t)T * frame_floats * sizeof(float), cudaMemcpyHostToDevice, s));
  et_result r{};
  ET_TRY(encode_impl(e, e->slot[0].frames_stage, video_offsets_host, V, params, s, &r));
  ET_TRY(copy_result_to_host(e, r, V, dst, s));
  ET_CUDA(e, cudaStreamSynchronize(s));
  *out = r;
  return ET_OK;
}

et_status et_encode_batch_host_submit(et_encoder* e, const float* frames_host, const int* video_offsets_host, int V,
                                      const et_params* params, void* cuda_stream, const et_host_buffers* dst,
                                      unsigned long long* ticket) {
  if (!ticket || !params) return fail(e, ET_ERR_INVALID_ARG, "null argument");
  ET_TRY(check_host_call(e, frames_host, video_offsets_host, V, dst));
  if (params->forced_plan || params->want_trace) return fail(e, ET_ERR_INVALID_ARG, "forced plans and traces need the synchronous calls");
  if (e->prof_on) return fail(e, ET_ERR_INVALID_ARG, "per-category profiling needs the synchronous calls");
  const int idx = (int)(e->next_ticket & 1ull);
  et_encoder::HostSlot& sl = e->slot[idx];
  if (sl.busy) return fail(e, ET_ERR_CAPACITY, "two calls are in flight already: collect the older one first");
  if (e->slot[idx ^ 1].busy && e->slot[idx ^ 1].stream != cuda_stream)
    return fail(e, ET_ERR_INVALID_ARG, "calls in flight together must use one stream: they share the encoder's work buffers");
  const int T = video_offsets_host[V];
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const size_t frame_floats = (size_t)3 * e->cfg.image_size * e->cfg.image_size;
  ET_CUDA(e, cudaSetDevice(e->device));
  ET_TRY(prepare_slot(e, idx, true));
  if (!e->h2d_stream) {
    ET_CUDA(e, cudaStreamCreateWithFlags(&e->h2d_stream, cudaStreamNonBlocking));
    ET_CUDA(e, cudaStreamCreateWithFlags(&e->d2h_stream, cudaStreamNonBlocking));
  }
  // Upload on the copy stream, compute behind the upload.  The slot's previous call has been collected, so nothing
  // reads its staging area or result buffers any more.
  ET_CUDA(e, cudaMemcpyAsync(sl.frames_stage, frames_host, (size_t)T * frame_floats * sizeof(float), cudaMemcpyHostToDevice, e->h2d_stream));
  ET_CUDA(e, cudaEventRecord(sl.ev_h2d, e->h2d_stream));
  ET_CUDA(e, cudaStreamWaitEvent(s, sl.ev_h2d, 0));
  ET_TRY(encode_impl(e, sl.frames_stage, video_offsets_host, V, params, s, nullptr, idx, true));
  sl.params = *params; sl.dst = *dst; sl.V = V; sl.T = T / e->tp; sl.stream = cuda_stream; sl.busy = true;
  sl.ticket = e->next_ticket++;
  *ticket = sl.ticket;
  return ET_OK;
}

et_status et_encode_batch_host_collect(et_encoder* e, unsigned long long ticket, et_result* out) {
  if (!e || !out) return fail(e, ET_ERR_INVALID_ARG, "null argument");
  const int idx = (int)(ticket & 1ull);
  et_encoder::HostSlot& sl = e->slot[idx];
  if (!sl.busy || sl.ticket != ticket) return fail(e, ET_ERR_INVALID_ARG, "no such call in flight");
  const et_encoder::HostSlot& other = e->slot[idx ^ 1];
  if (other.busy && other.ticket < ticket) return fail(e, ET_ERR_INVALID_ARG, "collect the older call first");
  ET_CUDA(e, cudaSetDevice(e->device));
  sl.busy = false;                                 // whatever happens below, the slot is free again
  ET_CUDA(e, cudaEventSynchronize(sl.ev_done));
  et_result r{};
  ET_TRY(encode_finish(e, &sl.params, sl.V, sl.T, idx, nullptr, &r));
  ET_TRY(copy_result_to_host(e, r, sl.V, &sl.dst, e->d2h_stream));
  ET_CUDA(e, cudaStreamSynchronize(e->d2h_stream));
  *out = r;
  return ET_OK;
}

}  // extern "C"

extern "C" {

const char* et_status_string(et_status s) {
  switch (s) {
    case ET_OK: return "ok";
    case ET_ERR_INVALID_ARG: return "invalid argument";
    case ET_ERR_SHAPE: return "inconsistent shape";
    case ET_ERR_CAPACITY: return "capacity exceeded";
    case ET_ERR_OOM: return "out of memory";
    case ET_ERR_CUDA: return "CUDA error";
    case ET_ERR_TIMEOUT: return "device-side wait expired";
    case ET_ERR_WEIGHTS: return "bad weight blob";
  }
  return "unknown status";
}

const char* et_last_error(const et_encoder* enc) { return enc ? enc->last_error.c_str() : ""; }

unsigned long long et_kernel_launch_count(void) { return g_kernel_launches.load(); }

et_status et_profile_enable(et_encoder* enc, int on) {
  if (!enc) return ET_ERR_INVALID_ARG;
  enc->prof_on = on != 0;
  if (on) memset(&enc->prof, 0, sizeof(enc->prof));
  return ET_OK;
}

et_status et_profile_read(const et_encoder* enc, et_profile* out) {
  if (!enc || !out) return ET_ERR_INVALID_ARG;
  *out = enc->prof;
  return ET_OK;
}

// ------------------------------------------------------------------------------------------------
// single steps
// ------------------------------------------------------------------------------------------------
#define ET_CUDA0(call)                                 \
  do {                                                 \
    if ((call) != cudaSuccess) return ET_ERR_CUDA;     \
  } while (0)

et_status et_frame_similarity(const float* x_dev, int n, int L, int D, float* cos_scratch_dev, float* sim_dev,
                              void* cuda_stream) {
  if (!x_dev || !cos_scratch_dev || !sim_dev) return ET_ERR_INVALID_ARG;
  if (n < 1 || L < 1 || D < 4 || D % 4 != 0 || D > ROW_MAX_D) return ET_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  launch_token_cosines(x_dev, cos_scratch_dev, n, L, D, nullptr, s);
  launch_reduce_cosines(cos_scratch_dev, sim_dev, n, L, nullptr, s);
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

et_status et_merge_plan(const float* sim_dev, const int* video_offsets_dev, int n, int V, double ema_alpha, double tau_seg,
                        double tau_merge, int weighted_merge, unsigned char* seg_start_dev, unsigned char* merge_next_dev,
                        float* ema_dev, int* n_out_dev, int* src_a_dev, int* src_b_dev, float* w_a_dev, float* w_b_dev,
                        int* new_video_offsets_dev, void* cuda_stream) {
  if (!sim_dev || !video_offsets_dev || !seg_start_dev || !merge_next_dev || !ema_dev || !n_out_dev || !src_a_dev ||
      !src_b_dev || !w_a_dev || !w_b_dev || !new_video_offsets_dev)
    return ET_ERR_INVALID_ARG;
  if (n < 1 || V < 1 || V > 1024) return ET_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  // scratch for the list bookkeeping this entry point does not expose
  int* scratch = nullptr;
  const size_t ints = 2 + 4 * (size_t)n + (size_t)n /*sim copy as float*/ + 2;
  ET_CUDA0(cudaMalloc(&scratch, ints * sizeof(int) + 2 * (size_t)n));
  int* n_cur = scratch;
  int* status = scratch + 1;
  int* lo0 = scratch + 2; int* hi0 = lo0 + n; int* lo1 = hi0 + n; int* hi1 = lo1 + n;
  float* sim_tr = reinterpret_cast<float*>(hi1 + n);
  unsigned char* role0 = reinterpret_cast<unsigned char*>(sim_tr + n + 2);
  unsigned char* role1 = role0 + n;
  cudaMemsetAsync(scratch, 0, ints * sizeof(int) + 2 * (size_t)n, s);
  cudaMemcpyAsync(n_cur, &n, sizeof(int), cudaMemcpyHostToDevice, s);
  PlanArgs a{};
  a.sim = sim_dev;
  a.cur = FrameList{n_cur, const_cast<int*>(video_offsets_dev), lo0, hi0, role0};
  a.nxt = FrameList{n_out_dev, new_video_offsets_dev, lo1, hi1, role1};
  a.plan = MergePlan{src_a_dev, src_b_dev, w_a_dev, w_b_dev};
  a.trace = LayerTrace{sim_tr, ema_dev, seg_start_dev, merge_next_dev};
  a.alpha = ema_alpha; a.tau_seg = tau_seg; a.tau_merge = tau_merge; a.weighted = weighted_merge;
  a.allow_merge = 1; a.n_videos = V; a.status = status;
  launch_merge_plan(a, n, s);
  cudaError_t err = cudaStreamSynchronize(s);
  cudaFree(scratch);
  return err == cudaSuccess ? ET_OK : ET_ERR_CUDA;
}

et_status et_merge_frames(const float* x_dev, float* y_dev, int n_cap, int frame_elems, const int* n_out_dev,
                          const int* src_a_dev, const int* src_b_dev, const float* w_a_dev, const float* w_b_dev,
                          void* cuda_stream) {
  if (!x_dev || !y_dev || !n_out_dev || !src_a_dev || !src_b_dev || !w_a_dev || !w_b_dev || x_dev == y_dev) return ET_ERR_INVALID_ARG;
  if (n_cap < 1 || n_cap > 65535 || frame_elems < 4 || frame_elems % 4 != 0) return ET_ERR_SHAPE;
  MergePlan p{const_cast<int*>(src_a_dev), const_cast<int*>(src_b_dev), const_cast<float*>(w_a_dev), const_cast<float*>(w_b_dev)};
  launch_merge_frames(x_dev, y_dev, n_cap, frame_elems, n_out_dev, p, (cudaStream_t)cuda_stream);
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

et_status et_select_tokens(const float* scores_dev, const unsigned char* dynamic_dev, const int* k_dev, const int* w_dev,
                           int N, int L, int window_mode, unsigned char* keep_dev, int* count_dev, void* cuda_stream) {
  if (!scores_dev || !dynamic_dev || !k_dev || !w_dev || !keep_dev || !count_dev) return ET_ERR_INVALID_ARG;
  if (window_mode < 0 || window_mode > 1) return ET_ERR_INVALID_ARG;
  if (N < 1 || L < 1 || L > 4096) return ET_ERR_SHAPE;
  launch_select_tokens(scores_dev, dynamic_dev, k_dev, w_dev, N, L, window_mode, keep_dev, count_dev, (cudaStream_t)cuda_stream);
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

et_status et_gather_tokens(const float* x_dev, const unsigned char* keep_dev, int N, int L, int D, const float* ln_g_dev,
                           const float* ln_b_dev, float ln_eps, float* tokens_dev, size_t tokens_capacity_rows,
                           int* frame_offsets_dev, int* token_pos_dev, int* n_tokens_host, void* cuda_stream) {
  if (!x_dev || !keep_dev || !tokens_dev || !frame_offsets_dev || !token_pos_dev || !n_tokens_host) return ET_ERR_INVALID_ARG;
  if ((ln_g_dev == nullptr) != (ln_b_dev == nullptr)) return ET_ERR_INVALID_ARG;
  if (N < 1 || N > 65535 || L < 1 || L > 4096 || D < 4 || D % 4 != 0 || D > ROW_MAX_D) return ET_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int* scratch = nullptr;
  ET_CUDA0(cudaMalloc(&scratch, sizeof(int) * ((size_t)N + 2)));
  int* count = scratch + 2;
  launch_count_keep(keep_dev, N, L, count, nullptr, s);
  launch_scan_counts(count, frame_offsets_dev, scratch, N, nullptr, s);
  int totals[2] = {0, 0};
  cudaError_t err = cudaMemcpyAsync(totals, scratch, sizeof(totals), cudaMemcpyDeviceToHost, s);
  if (err == cudaSuccess) err = cudaStreamSynchronize(s);
  if (err != cudaSuccess) { cudaFree(scratch); return ET_ERR_CUDA; }
  if ((size_t)totals[1] > tokens_capacity_rows) { cudaFree(scratch); return ET_ERR_CAPACITY; }
  launch_gather_tokens(x_dev, keep_dev, count, frame_offsets_dev, scratch, N, L, D, ln_g_dev, ln_b_dev, ln_eps, tokens_dev,
                       token_pos_dev, nullptr, s);
  err = cudaStreamSynchronize(s);
  cudaFree(scratch);
  if (err != cudaSuccess) return ET_ERR_CUDA;
  *n_tokens_host = totals[1];
  return ET_OK;
}

et_status et_linear_bf16(const void* a_dev, const void* w_dev, const float* bias_dev, void* c_dev, int M, int N, int K,
                         int epilogue, int gelu_tanh, const float* table_dev, int table_rows, int* status_dev,
                         void* cuda_stream) {
  if (!a_dev || !w_dev || !bias_dev || !c_dev) return ET_ERR_INVALID_ARG;
  if (M < 1 || N < 8 || N % 8 != 0 || K < 8 || K % 8 != 0) return ET_ERR_SHAPE;
  if (epilogue < 0 || epilogue > 4 || (epilogue == 3 && (!table_dev || table_rows < 1))) return ET_ERR_INVALID_ARG;
  if (epilogue == 4 && N % 256 != 0) return ET_ERR_SHAPE;
  TmaDesc da, dc;
  WeightDesc dw;
  const char* err = nullptr;
  if (!make_tma_2d_bf16(&da, a_dev, M, K, 128, &err) || !make_tma_weight(&dw, w_dev, N, K, &err) ||
      !make_tma_out(&dc, c_dev, M, epilogue == 4 ? N / 2 : N, epilogue == 2 || epilogue == 3, &err))
    return ET_ERR_CUDA;
  ET_CUDA0(launch_gemm_bf16(da, dw, dc, bias_dev, c_dev, M, N, K, epilogue, gelu_tanh, table_dev, table_rows, nullptr, 1,
                            status_dev, (cudaStream_t)cuda_stream));
  return ET_OK;
}

et_status et_attention(const void* qkv_dev, void* out_dev, float* lse_dev, int n, int L, int heads, int head_dim,
                       int dtype, void* cuda_stream) {
  if (!qkv_dev || !out_dev || !lse_dev) return ET_ERR_INVALID_ARG;
  if (n < 1 || n > 65535 || L < 1 || heads < 1 || heads > 65535 || head_dim < 1 || head_dim > 128) return ET_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (dtype == ET_BF16) {
    if (head_dim % 8 != 0) return ET_ERR_SHAPE;
    if (attention_tc_supported(head_dim)) {
      AttnMaps maps;
      if (!make_attention_maps(&maps, (const bf16*)qkv_dev, (long long)n * L, heads, head_dim, (bf16*)out_dev, L)) return ET_ERR_CUDA;
      ET_CUDA0(launch_attention_tc(maps, lse_dev, n, L, heads, head_dim, nullptr, nullptr, s));
      return ET_OK;
    }
    launch_attention_bf16((const bf16*)qkv_dev, (bf16*)out_dev, lse_dev, n, L, heads, head_dim, nullptr, s);
  } else if (dtype == ET_F32) {
    launch_attention_f32((const float*)qkv_dev, (float*)out_dev, lse_dev, n, L, heads, head_dim, nullptr, s);
  } else {
    return ET_ERR_INVALID_ARG;
  }
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

et_status et_attention_windowed(const void* qkv_dev, void* out_dev, float* lse_scratch_dev, int n, int L, int heads,
                                int head_dim, int window_rows, int dtype, void* cuda_stream) {
  if (!qkv_dev || !out_dev || !lse_scratch_dev) return ET_ERR_INVALID_ARG;
  if (n < 1 || L < 1 || heads < 1 || heads > 65535 || head_dim < 1 || head_dim > 128) return ET_ERR_SHAPE;
  if (window_rows < 1 || L % window_rows != 0 || (long long)n * (L / window_rows) > 65535) return ET_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int items = n * (L / window_rows);
  if (dtype == ET_BF16) {
    if (head_dim % 8 != 0) return ET_ERR_SHAPE;
    if (attention_tc_supported(head_dim)) {
      AttnMaps maps;
      if (!make_attention_maps(&maps, (const bf16*)qkv_dev, (long long)n * L, heads, head_dim, (bf16*)out_dev, L)) return ET_ERR_CUDA;
      ET_CUDA0(launch_attention_tc(maps, lse_scratch_dev, n, L, heads, head_dim, nullptr, nullptr, s, window_rows));
      return ET_OK;
    }
    launch_attention_bf16((const bf16*)qkv_dev, (bf16*)out_dev, lse_scratch_dev, items, window_rows, heads, head_dim, nullptr, s);
  } else if (dtype == ET_F32) {
    launch_attention_f32((const float*)qkv_dev, (float*)out_dev, lse_scratch_dev, items, window_rows, heads, head_dim, nullptr, s);
  } else {
    return ET_ERR_INVALID_ARG;
  }
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

et_status et_attention_scores(const void* qkv_dev, const float* lse_dev, float* partial_dev, float* score_dev, int n, int L,
                              int heads, int head_dim, int dtype, void* cuda_stream) {
  if (!qkv_dev || !lse_dev || !partial_dev || !score_dev) return ET_ERR_INVALID_ARG;
  if (n < 1 || n > 65535 || L < 1 || heads < 1 || heads > 65535 || head_dim < 1 || head_dim > 128) return ET_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (dtype == ET_BF16) {
    if (head_dim % 8 != 0) return ET_ERR_SHAPE;
    if (attention_scores_tc_supported(head_dim)) {
      AttnMaps maps;
      if (!make_attention_maps(&maps, (const bf16*)qkv_dev, (long long)n * L, heads, head_dim)) return ET_ERR_CUDA;
      ET_CUDA0(launch_attention_scores_tc(maps, lse_dev, partial_dev, score_dev, n, L, heads, head_dim, nullptr, nullptr, s));
      return ET_OK;
    }
    launch_attention_scores_bf16((const bf16*)qkv_dev, lse_dev, partial_dev, score_dev, n, L, heads, head_dim, nullptr, s);
  } else if (dtype == ET_F32) {
    launch_attention_scores_f32((const float*)qkv_dev, lse_dev, partial_dev, score_dev, n, L, heads, head_dim, nullptr, s);
  } else {
    return ET_ERR_INVALID_ARG;
  }
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

et_status et_layernorm(const float* x_dev, const float* g_dev, const float* b_dev, float eps, void* y_dev, int rows, int D,
                       int dtype, void* cuda_stream) {
  if (!x_dev || !g_dev || !b_dev || !y_dev) return ET_ERR_INVALID_ARG;
  if (rows < 1 || D < 4 || D % 4 != 0 || D > ROW_MAX_D) return ET_ERR_SHAPE;
  if (dtype != ET_F32 && dtype != ET_BF16) return ET_ERR_INVALID_ARG;
  launch_layernorm(x_dev, g_dev, b_dev, eps, y_dev, rows, D, dtype == ET_BF16, nullptr, 1, (cudaStream_t)cuda_stream);
  ET_CUDA0(cudaGetLastError());
  return ET_OK;
}

}  // extern "C"
