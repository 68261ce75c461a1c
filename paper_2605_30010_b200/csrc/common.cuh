// Internal declarations shared by the translation units of libearlytom (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "earlytom.h"

namespace et {

typedef __nv_bfloat16 bf16;

extern std::atomic<unsigned long long> g_kernel_launches;
#define ET_COUNT_LAUNCH() (::et::g_kernel_launches.fetch_add(1, std::memory_order_relaxed))

// Codes written by kernels into the device status word (0 = fine).
enum DeviceStatus : int {
  DS_OK = 0,
  DS_WAIT_EXPIRED = 1,      // a bounded mbarrier wait ran out
  DS_FORCED_MISMATCH = 2,   // forced plan does not fit the frame list on the device
  DS_CAPACITY = 3,
  DS_BAD_INDEX = 4          // checked build only: an index left its array
};

// Index checks of the checked build (-DET_DEBUG, libearlytom_debug.so): a violated condition records DS_BAD_INDEX in
// a status word of the translation unit (read by et_debug_status) and the statement `skip` is executed instead
// of the access; nothing traps.  In the regular build the macro expands to nothing.
#ifdef ET_DEBUG
#define ET_DEBUG_STATUS_WORD static __device__ int g_debug_status_word = 0;
#define ET_CHECK(cond, skip)                                  \
  do {                                                        \
    if (!(cond)) {                                            \
      atomicExch(&g_debug_status_word, (int)::et::DS_BAD_INDEX); \
      skip;                                                   \
    }                                                         \
  } while (0)
#define ET_DEBUG_STATUS_READ(fn)                                                        \
  int fn() {                                                                            \
    int v = 0;                                                                          \
    if (cudaMemcpyFromSymbol(&v, g_debug_status_word, sizeof(int)) != cudaSuccess) return -1; \
    return v;                                                                           \
  }
#else
#define ET_DEBUG_STATUS_WORD
#define ET_CHECK(cond, skip) do { } while (0)
#define ET_DEBUG_STATUS_READ(fn) int fn() { return 0; }
#endif

static inline int cdiv(long long a, long long b) { return (int)((a + b - 1) / b); }

// Device-resident description of the current frame list (all videos of the call, concatenated).
struct FrameList {
  int* n;                // [1]  frames alive
  int* vid_off;          // [Vmax+1] first frame of each video in the list
  int* src_lo;           // [Fmax] first original frame merged into this frame (index inside its video)
  int* src_hi;           // [Fmax]
  unsigned char* role;   // [Fmax] 0 head, 1 middle, 2 tail, 3 single-frame segment
};

// The merge plan of one layer: how to build the next list from the current one.
struct MergePlan {
  int* src_a;    // [Fmax]
  int* src_b;    // [Fmax]  -1 = copy
  float* w_a;    // [Fmax]
  float* w_b;    // [Fmax]
};

// Trace slot of one merge layer (device arrays [Fmax]).
struct LayerTrace {
  float* sim;
  float* ema;
  unsigned char* seg_start;
  unsigned char* merge_next;
};

// EPI_SWIGLU: the N accumulator columns are pairs of 32-column chunks (gate, up) of the same 32 outputs; the layer
// writes c [M][N/2] = silu(gate + bias) * (up + bias) in bf16, bias [N] in the order of the weight rows.  N % 256 == 0.
enum Epilogue : int { EPI_STORE = 0, EPI_GELU = 1, EPI_RESIDUAL = 2, EPI_TABLE = 3, EPI_SWIGLU = 4 };

// ---- elementwise.cu ------------------------------------------------------------------------
// frames fp32 [T][3][H][W] -> patches [T*L][k_pad] (zero padded beyond 3*p*p), fp32 or bf16.
// tp input frames make one encoder frame (T counts encoder frames); int2raster: optional internal token order.
void launch_im2col(const float* frames, void* patches, int T, int image, int patch, int k_pad, bool out_bf16,
                   const int* n_frames_dev, cudaStream_t s, int tp = 1, const int* int2raster = nullptr,
                   const int* raster2int = nullptr);   // both token-order tables or neither
// 2-D rotary positions in place on the Q and K parts of packed rows [rows][3*heads*dh]; table [L][dh/2] (cos, sin)
void launch_rope_pairs(void* qkv, const float2* table, int rows_cap, int L, int heads, int dh, bool is_bf16,
                       const int* n_frames_dev, cudaStream_t s);
// h[r][j] = silu(gu[r][j]) * gu[r][Mp + j], j < Mp
void launch_gated_silu(const void* gu, void* h, int rows_cap, int Mp, bool is_bf16, const int* n_frames_dev,
                       int rows_per_frame, cudaStream_t s);
void launch_scale_count(const int* in, int mult, int* out, cudaStream_t s);
// LayerNorm of rows [rows_cap][D] (RMSNorm with gain g when b == NULL); live rows = *n_frames_dev * rows_per_frame
// when n_frames_dev != NULL.
void launch_layernorm(const float* x, const float* g, const float* b, float eps, void* y, int rows_cap, int D,
                      bool out_bf16, const int* n_frames_dev, int rows_per_frame, cudaStream_t s);

// ---- gemm_simt.cu --------------------------------------------------------------------------
// c = epi(a[M][K] * w[K][N] + bias) in fp32 FFMA.  live M as above.
void launch_gemm_f32(const float* a, const float* w, const float* bias, float* c, int M_cap, int N, int K,
                     int epilogue, int gelu_tanh, const float* table, int table_rows, const int* n_frames_dev,
                     int rows_per_frame, cudaStream_t s);

// ---- gemm_tcgen05.cu -----------------------------------------------------------------------
struct TmaDesc { alignas(64) unsigned char bytes[128]; };
// Build a 2-D bf16 tensor map: rows x cols (cols contiguous), box box_rows x 64 cols, 128-byte swizzle.
bool make_tma_2d_bf16(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                      const char** err);
// Weight operand w [N][K]: one map whose box holds a CTA's half of a full-width tile, one with a 64-row box for
// the narrow last column tile (N mod 256 <= 128), so that a narrow tile does not fetch weight rows it never uses.
struct WeightDesc { TmaDesc full, half; };
bool make_tma_weight(WeightDesc* out, const void* base, uint64_t n_rows, uint64_t k_cols, const char** err);
// Tensor map of a dense layer's output c [rows][cols] (fp32 or bf16): 32 x 32 boxes for the epilogue's
// TMA stores / reduce-adds.
bool make_tma_out(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, bool fp32, const char** err);
int gemm_bf16_pick_bn(int N);
// Rows of the w box: each CTA of a pair loads half of the tile's BN weight rows.
int gemm_bf16_w_box_rows(int N);
// c = epi(a[M][K] * w[N][K]^T + bias).  Descriptors must have been built for (a: M_cap x K, box 128),
// (w: make_tma_weight) and (c: make_tma_out; unused by EPI_TABLE).
cudaError_t launch_gemm_bf16(const TmaDesc& da, const WeightDesc& dw, const TmaDesc& dc, const float* bias, void* c,
                             int M_cap, int N, int K, int epilogue, int gelu_tanh, const float* table, int table_rows,
                             const int* n_frames_dev, int rows_per_frame, int* status_dev, cudaStream_t s);

// ---- attention_simt.cu / attention_mma.cu --------------------------------------------------
void launch_attention_f32(const float* qkv, float* out, float* lse, int n_cap, int L, int heads, int dh,
                          const int* n_frames_dev, cudaStream_t s);
void launch_attention_bf16(const bf16* qkv, bf16* out, float* lse, int n_cap, int L, int heads, int dh,
                           const int* n_frames_dev, cudaStream_t s);
bool attention_bf16_supported(int L, int heads, int dh);
// tcgen05 attention (attention_tcgen05.cu): head dims 64, 72 and 80.  The maps describe qkv [rows][3*D] bf16.
// Q boxes (128 rows), K / V boxes (one key tile), and the attention output as [frames][L][D] (stores clipped per frame)
struct AttnMaps { TmaDesc main, tail, kv_main, kv_tail, out; };
bool attention_tc_supported(int dh);
// attn_out (with the tokens per frame L) may be NULL for users that only read Q / K / V through the maps
bool make_attention_maps(AttnMaps* out, const bf16* qkv, long long rows, int heads, int dh, bf16* attn_out = nullptr, int L = 0);
// The output goes where maps.out points.  window_rows > 0: a query attends only to the keys of its run of
// window_rows consecutive rows of the frame
cudaError_t launch_attention_tc(const AttnMaps& maps, float* lse, int n_cap, int L, int heads, int dh,
                                const int* n_frames_dev, int* status_dev, cudaStream_t s, int window_rows = 0);
bool attention_scores_tc_supported(int dh);
// partial[f][h][j] = sum_q exp(s(q,j) - lse[f][h][q]);  score[f][j] = sum_h partial / (heads*L)
void launch_attention_scores_f32(const float* qkv, const float* lse, float* partial, float* score, int n_cap, int L,
                                 int heads, int dh, const int* n_frames_dev, cudaStream_t s);
void launch_attention_scores_bf16(const bf16* qkv, const float* lse, float* partial, float* score, int n_cap, int L,
                                  int heads, int dh, const int* n_frames_dev, cudaStream_t s);

// scores_tcgen05.cu: the score pass on tcgen05 (head dims 64 and 72), same maps as the attention kernel
cudaError_t launch_attention_scores_tc(const AttnMaps& maps, const float* lse, float* partial, float* score, int n_cap,
                                       int L, int heads, int dh, const int* n_frames_dev, int* status_dev, cudaStream_t s);

// attention_causal_tcgen05.cu: causal grouped-query attention, head dim 128, over packed rows
// [heads*128 | kv_heads*128 | kv_heads*128] of n_seq sequences of L positions each.
bool attention_causal_supported(int head_dim);
struct CausalMaps { TmaDesc q, kv; };     // the packed Q | K | V rows in boxes of 128 rows (Q) and of one key tile (K, V)
bool make_causal_attention_map(CausalMaps* out, const bf16* qkv, long long rows, int heads, int kv_heads);
cudaError_t launch_attention_causal(const CausalMaps& map, bf16* out, int n_seq, int L, int heads, int kv_heads,
                                    int* status_dev, cudaStream_t s);

// ---- llm_ops.cu: row-wise and elementwise steps of the language model --------------------------
// y = x * rsqrt(mean(x^2) + eps) * g, rows [rows][D] fp32 -> bf16
void launch_rmsnorm(const float* x, const float* g, float eps, bf16* y, int rows, int D, cudaStream_t s);
// rotate-half rotary embedding in place on the Q and K parts of packed rows [rows][(heads + 2*kv_heads)*dh];
// the position of a row is row % L; table [>= L][dh/2] holds (cos, sin) of position * theta^(-2i/dh), filled by
// launch_rope_table from inv_turns [dh/2] (device, double) = theta^(-2i/dh) / (2 pi)
void launch_rope_table(float2* table, int L, int dh, const double* inv_turns, cudaStream_t s);
void launch_rope(bf16* qkv, int rows, int L, int heads, int kv_heads, int dh, const float2* table, cudaStream_t s);
// h[r][j] = silu(gu[r][j]) * gu[r][M + j]
void launch_swiglu(const bf16* gu, bf16* h, int rows, int M, cudaStream_t s);
// x[r][:] = table[ids[r]][:]  (bf16 table -> fp32 rows)
void launch_embed_rows(const bf16* table, const int* ids, float* x, int rows, int D, int vocab, cudaStream_t s);
void launch_cast_bf16(const float* x, bf16* y, size_t count, cudaStream_t s);
// dst[r][0..width) = src[r][0..width); width and both pitches in elements, multiples of 8; 16-byte aligned pointers
void launch_copy_columns(const bf16* src, bf16* dst, int rows, int width, int src_pitch, int dst_pitch, cudaStream_t s);
// first index of the maximum of x[0..n)
void launch_argmax(const float* x, int n, int* out, cudaStream_t s);

// ---- stage1.cu -----------------------------------------------------------------------------
void launch_token_cosines(const float* x, float* cos_scratch, int n_cap, int L, int D, const int* n_frames_dev,
                          cudaStream_t s);
void launch_reduce_cosines(const float* cos_scratch, float* sim, int n_cap, int L, const int* n_frames_dev,
                           cudaStream_t s);
struct PlanArgs {
  const float* sim;              // [n] similarity of frames t, t+1
  FrameList cur, nxt;
  MergePlan plan;
  LayerTrace trace;              // may hold NULLs
  const unsigned char* forced_seg_start;   // NULL = decide
  const unsigned char* forced_merge_next;
  int forced_n_in;
  double alpha, tau_seg, tau_merge;
  int weighted;
  int allow_merge;               // 0 = segmentation only (roles), list unchanged
  int n_videos;
  int* n_hist_slot;              // receives the new frame count (may be NULL)
  int* status;
};
void launch_merge_plan(const PlanArgs& a, int n_cap, cudaStream_t s);
// Similarities of the current list and its plan in one launch (no scratch array, no kernel waits: see stage1.cu).
// acc: similarity_plan_words(n_cap) - 1 64-bit accumulators and done: [1] ticket counter, zero before the first
// launch; every launch leaves them at zero.
struct SimPlanArgs {
  const float* x;               // [n_cap][L][D] residual stream
  float* sim;                   // [n_cap]; must be plan.sim
  int n_cap, L, D;
  const int* n_frames_dev;      // live frames
  const int* vid_off;           // [n_videos+1] of the current list
  int n_videos;
  unsigned long long* acc;      // [slots][n_cap]
  unsigned* done;               // [1]
  PlanArgs plan;
};
void launch_similarity_plan(const SimPlanArgs& a, cudaStream_t s);
int similarity_plan_words(int n_cap);
void launch_merge_frames(const float* x, float* y, int n_cap, int frame_elems, const int* n_out_dev,
                         const MergePlan& plan, cudaStream_t s);
void launch_init_frames(const FrameList& fl, const int* vid_off_src_dev, int n_videos, int n_frames, cudaStream_t s);

// ---- stage2.cu -----------------------------------------------------------------------------
struct SelectArgs {
  const float* scores;       // [n_cap][L]
  FrameList fl;              // current list: live count, video offsets, roles
  const int* orig_vid_off;   // [V+1] offsets of the input videos (for B of Eq. 5)
  int n_cap, n_videos, L, selection, retain_mode, window_mode;
  int mask_given;            // 1: keep[] was provided by the caller; write only the flags and amounts
  const int* raster2int;     // NULL, or the internal position of raster position j (scores are in internal order)
  double retain;
  unsigned char* dynamic;    // [Fmax] out
  unsigned char* keep;       // [Fmax][L] out
  int* count;                // [Fmax] out
  int* video_k;              // [Vmax] out
  int* video_w;              // [Vmax] out
};
// per-video amounts (Eq. 5-6), per-frame dynamic flags and the keep mask in one launch
void launch_select_video_tokens(const SelectArgs& a, cudaStream_t s);
// keep mask from per-frame amounts given by the caller (the single-step entry point)
void launch_select_tokens(const float* scores, const unsigned char* dynamic, const int* k_frame, const int* w_frame,
                          int n_cap, int L, int window_mode, unsigned char* keep, int* count, cudaStream_t s);
// Random-sampling ablation: scores[f][j] = uniform number of Philox-4x32-10 with counter (j, frame inside its
// video, video, 0) and key = seed, for the frames of the current list.
void launch_random_scores(float* scores, const int* vid_off, int n_videos, int n_cap, int L, unsigned long long seed,
                          const int* n_frames_dev, cudaStream_t s);
void launch_count_keep(const unsigned char* keep, int n_cap, int L, int* count, const int* n_frames_dev, cudaStream_t s);
// frame_offsets[0..n] = exclusive scan of count; totals[0] = n_frames, totals[1] = n_tokens
void launch_scan_counts(const int* count, int* frame_offsets, int* totals, int n_cap, const int* n_frames_dev,
                        cudaStream_t s);
// gathers the kept rows; also writes frame_offsets[0..n] (exclusive scan of count) and totals[0] = n_frames,
// totals[1] = n_tokens
void launch_gather_tokens(const float* x, const unsigned char* keep, const int* count, int* frame_offsets, int* totals,
                          int n_cap, int L, int D, const float* ln_g, const float* ln_b, float eps, float* tokens,
                          int* token_pos, const int* n_frames_dev, cudaStream_t s, const int* raster2int = nullptr);
// (ln_b == NULL with ln_g != NULL: RMSNorm with gain ln_g; raster2int: the keep mask and token_pos are in raster
// order while the rows of x are in the encoder's internal order)

}  // namespace et
