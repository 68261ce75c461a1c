/*
 * earlytom.h - C ABI of the B200 (sm_100a) compressed video vision-encoder.
 *
 * The library runs a SigLIP-style ViT over the frames of a video and performs EarlyTom's
 * compression inside it:
 *   Stage I  (paper Sec. 3.2, Eq. 1-3, Algorithm 1): at selected blocks the frames are segmented
 *            by an EMA of adjacent-frame similarity, similar middle frames are merged pairwise
 *            (weighted by similarity) and the surviving frames are packed; the remaining blocks
 *            run on fewer frames.
 *   Stage II (paper Sec. 3.3, Eq. 4-7, Algorithm 2): at the encoder output, head/tail frames of
 *            each segment ("dynamic") keep their top-k tokens by attention score, middle frames
 *            ("static") keep the best token of each local window; kept tokens are gathered in
 *            temporal order into ragged per-frame lists.
 *
 * Conventions
 *   - every function returns et_status and never aborts or throws; on error outputs are untouched;
 *   - "dev" pointers are CUDA device memory of the current device, "host" pointers are host memory;
 *   - caller-owned inputs are only read; result pointers are owned by the encoder and stay valid
 *     until the next encode call on that encoder or et_destroy;
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = default stream);
 *   - one encoder serves one device and one call at a time (not re-entrant).
 *   - there is no CPU fallback: without a CUDA device every compute entry point returns ET_ERR_CUDA.
 */
#ifndef EARLYTOM_H_
#define EARLYTOM_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ET_API __attribute__((visibility("default")))
#else
#define ET_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct et_encoder et_encoder; /* opaque */

typedef enum {
  ET_OK = 0,
  ET_ERR_INVALID_ARG = 1, /* NULL pointer, value out of its documented range */
  ET_ERR_SHAPE = 2,       /* inconsistent architecture numbers */
  ET_ERR_CAPACITY = 3,    /* more frames / videos / tokens than the encoder or the buffer holds */
  ET_ERR_OOM = 4,         /* device or host allocation failed */
  ET_ERR_CUDA = 5,        /* a CUDA call failed; et_last_error() has the text */
  ET_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (kernel returned early) */
  ET_ERR_WEIGHTS = 7      /* weight blob has the wrong number of floats or non-finite values */
} et_status;

typedef enum { ET_F32 = 0, ET_BF16 = 1 } et_dtype;

#define ET_MAX_MERGE_LAYERS 8

/* Architecture and capacity.  Pre-LN ViT blocks, biases on every linear layer, learned position
 * embedding, no class token, patch embedding = stride-p valid convolution over the top-left
 * (image_size / patch_size * patch_size)^2 crop.  dtype selects the arithmetic of the dense
 * layers: ET_F32 = fp32 FFMA everywhere; ET_BF16 = bf16 tensor-core operands with fp32
 * accumulation, fp32 residual stream, fp32 LayerNorm / softmax / GELU.  Outputs are fp32. */
typedef struct {
  int image_size, patch_size, num_layers, hidden, heads, mlp_dim;
  float ln_eps;         /* LayerNorm epsilon, e.g. 1e-6 */
  int gelu_tanh;        /* 1 = tanh approximation of GELU, 0 = erf form */
  int post_layernorm;   /* 1 = final LayerNorm applied to the kept tokens */
  int dtype;            /* et_dtype */
  int max_frames_total; /* capacity: sum of (input) frames over the videos of one call; at most 65535 encoder frames */
  int max_videos;       /* capacity: videos per call */
  /* Architecture family (zero-initialised fields give the SigLIP-style encoder described above).
   * arch 1 = Qwen2.5-VL-style encoder, the architecture of the paper's generalisation study (supplementary
   * "Generalizability Analysis"): RMSNorm (gain only) instead of LayerNorm, gated SiLU MLP with biases, biases on
   * QKV / output projection, 2-D rotary positions on q and k (rotate-half pairing; the first dh/4 pairs turn with the
   * token's row in the patch grid, the next dh/4 with its column, frequencies rope_theta^(-2i/(dh/2))), no position
   * table, no patch-embedding bias; temporal_patch input frames form ONE encoder frame (a convolution over
   * temporal_patch x p x p pixels); attention runs inside windows of window x window patches except in the blocks
   * whose bit is set in full_attn_mask (bit b = 0-based block b), which attend over the whole encoder frame.
   * Requirements for arch 1: head dim a multiple of 4; window = 0 (no windows) or a divisor of the patch grid; the
   * last block in full_attn_mask (its attention scores feed Stage II); frame counts multiples of temporal_patch.
   * Every frame index and count the library reports (et_result, et_trace, Eq. 5's B and N) is then in ENCODER frames.
   * The final RMSNorm (post_layernorm) is the one that precedes the model's 2 x 2 patch merger; the merger itself is
   * not part of this library. */
  int arch;
  int temporal_patch;   /* arch 1: input frames per encoder frame (>= 1); arch 0: 0 or 1 */
  int window;           /* arch 1: window side in patches, 0 = full attention everywhere */
  unsigned long long full_attn_mask; /* arch 1 with window > 0: blocks with full attention */
  float rope_theta;     /* arch 1: base of the rotary frequencies, e.g. 10000 */
} et_config;

/* Host fp32 blob, row-major, y = x W + b with W [in][out], in this order:
 *   patch_w [3*p*p][D] (row = c*p*p + dy*p + dx), patch_b [D], pos [L][D],
 *   per layer: ln1_g, ln1_b [D]; wqkv [D][3D] (columns Q|K|V, head h at h*dh of its third),
 *   bqkv [3D]; wo [D][D], bo [D]; ln2_g, ln2_b [D]; w1 [D][M], b1 [M]; w2 [M][D], b2 [D];
 *   then post_g, post_b [D].
 * arch 1 (see et_config):
 *   patch_w [3*tp*p*p][D] (row = c*tp*p*p + t*p*p + dy*p + dx),
 *   per layer: n1_g [D]; wqkv [D][3D], bqkv [3D]; wo [D][D], bo [D]; n2_g [D]; wgu [D][2M] (columns gate | up),
 *   bgu [2M]; wd [M][D], bd [D];   then post_g [D].
 * The library converts and copies; the caller may free the blob after create returns. */
typedef struct {
  const float* data;
  size_t count;
} et_weights;

/* Decisions to replay instead of taking them (test hook; compares values under identical
 * decisions).  All pointers are host memory.  Entry i belongs to merge_layers[i] and describes
 * the frame list ENTERING that layer, concatenated over the videos of the call. */
typedef struct {
  int n_in[ET_MAX_MERGE_LAYERS];                           /* expected list length, checked */
  const unsigned char* seg_start[ET_MAX_MERGE_LAYERS];     /* [n_in] 1 = frame opens a segment */
  const unsigned char* merge_next[ET_MAX_MERGE_LAYERS];    /* [n_in] 1 = merged with its successor */
  int n_final;                                             /* frames at the encoder output */
  const unsigned char* keep;                               /* [n_final * L] or NULL = decide */
} et_forced_plan;

typedef struct {
  int num_merge_layers;
  int merge_layers[ET_MAX_MERGE_LAYERS]; /* 0-based block index the merge precedes; ascending; in [1, layers-1] */
  double ema_alpha;     /* Eq. 1 smoothing factor, (0, 1] */
  double tau_seg;       /* Eq. 1 threshold */
  double tau_merge;     /* Eq. 2 threshold */
  int weighted_merge;   /* 1 = Eq. 3, 0 = plain average */
  int selection;        /* 0 keep all tokens, 1 decoupled (Alg. 2), 2 per-frame top-k on every frame,
                           3 random sampling (the paper's sampling ablation): k tokens per frame drawn with
                           Philox-4x32-10, counter (position, output frame inside its video, video, 0), key = sample_seed */
  int retain_mode;      /* 0: keep floor(retain*L) per frame; 1: total budget, k = floor(retain*B*L/N) (Eq. 5) */
  double retain;        /* (0, 1] */
  const et_forced_plan* forced_plan; /* NULL = decide */
  int want_trace;       /* 1 = fill et_result.trace */
  unsigned long long sample_seed; /* selection 3 only */
  int window_mode;      /* local windows of a static frame (Eq. 6).  0: as printed, runs of w = floor(L/k) positions,
                           M = ceil(L/w) windows (M >= k; M = L once k > L/2, i.e. static frames keep everything);
                           1: k windows [floor(m*L/k), floor((m+1)*L/k)), so static and dynamic frames keep the same
                           amount and the total is N*k ~ retain*B*L.  Both coincide when k divides L. */
} et_params;

/* Decision trace, host memory owned by the encoder.  Per merge layer i the arrays cover the list
 * entering the layer: sim[t] = similarity of frames t and t+1 (0 for the last frame of a video),
 * ema[t] = smoothed value that decided whether frame t opens a segment (0 for first frames). */
typedef struct {
  int num_merge_layers;
  int n_in[ET_MAX_MERGE_LAYERS], n_out[ET_MAX_MERGE_LAYERS];
  const float* sim[ET_MAX_MERGE_LAYERS];
  const float* ema[ET_MAX_MERGE_LAYERS];
  const unsigned char* seg_start[ET_MAX_MERGE_LAYERS];
  const unsigned char* merge_next[ET_MAX_MERGE_LAYERS];
  const float* scores;          /* [n_frames_out * L] per-token attention score A */
  const unsigned char* keep;    /* [n_frames_out * L] */
  const int* video_k;           /* [n_videos] tokens kept per dynamic frame */
  const int* video_w;           /* [n_videos] window width on static frames */
} et_trace;

typedef struct {
  int n_videos, n_frames_in, n_frames_out, n_tokens, hidden, tokens_per_frame;
  /* device memory, owned by the encoder */
  const float* tokens;              /* [n_tokens][hidden] frames in temporal order, positions ascending */
  const int* video_frame_offsets;   /* [n_videos+1] into the output frames */
  const int* frame_offsets;         /* [n_frames_out+1] into tokens: the ragged per-frame lists */
  const int* frame_src_lo;          /* [n_frames_out] first original frame (index inside its video) merged in */
  const int* frame_src_hi;          /* [n_frames_out] last one */
  const unsigned char* frame_dynamic; /* [n_frames_out] 1 = dynamic (top-k), 0 = static (windows) */
  const int* token_pos;             /* [n_tokens] spatial index 0..L-1 of each kept token */
  const et_trace* trace;            /* host; NULL unless want_trace */
  int frames_per_block[64];         /* host: frames alive in each block (first num_layers entries) */
} et_result;

/* Host destination buffers for the *_host entry point (caller-owned; pinned memory makes the
 * copies asynchronous).  capacity_tokens / capacity_frames say how much they hold. */
typedef struct {
  float* tokens;                 /* [capacity_tokens][hidden] */
  int* token_pos;                /* [capacity_tokens] */
  int* frame_offsets;            /* [capacity_frames+1] */
  int* frame_src_lo;             /* [capacity_frames] */
  int* frame_src_hi;             /* [capacity_frames] */
  unsigned char* frame_dynamic;  /* [capacity_frames] */
  int* video_frame_offsets;      /* [n_videos+1] */
  size_t capacity_tokens, capacity_frames;
} et_host_buffers;

/* Paper: the vision encoder of Sec. 3.1 / 4.1 (pretrained SigLIP in the paper; random or real
 * weights here).  Validates the config, allocates every device buffer for the stated capacity,
 * converts the weights.  *out receives the encoder. */
ET_API et_status et_encoder_create(const et_config* config, const et_weights* weights, et_encoder** out);

/* Paper: the whole pipeline of Fig. 3 for one video: encoder blocks with Stage I (Alg. 1) at
 * params->merge_layers, then Stage II (Alg. 2).  frames_dev: fp32 [T][3][H][W] in device memory.
 * Work is enqueued on cuda_stream; the call synchronises that stream once at the end to read the
 * output sizes.  out: filled on success. */
ET_API et_status et_encode_video(et_encoder* enc, const float* frames_dev, int T, const et_params* params,
                          void* cuda_stream, et_result* out);

/* Same for V independent videos in one call (frames concatenated, video_offsets_host [V+1]);
 * every decision (segments, merges, Eq. 5 amounts) is taken per video. */
ET_API et_status et_encode_batch(et_encoder* enc, const float* frames_dev, const int* video_offsets_host, int V,
                          const et_params* params, void* cuda_stream, et_result* out);

/* Same as et_encode_batch with HOST frames and HOST results: copies the frames to the device,
 * encodes, copies tokens and index map into `dst`.  ET_ERR_CAPACITY if dst is too small. */
ET_API et_status et_encode_batch_host(et_encoder* enc, const float* frames_host, const int* video_offsets_host, int V,
                               const et_params* params, void* cuda_stream, const et_host_buffers* dst,
                               et_result* out);

/* The same host-to-host call split in two, so that the copies of neighbouring calls overlap the
 * encoder's work (no counterpart in the paper: serving plumbing around Fig. 3's pipeline).
 *
 * et_encode_batch_host_submit validates like et_encode_batch_host, enqueues the upload of
 * frames_host on a copy stream of the encoder's own and every kernel of the call on cuda_stream
 * behind it, and returns without waiting; *ticket names the call.  At most TWO calls may be in
 * flight (ET_ERR_CAPACITY on a third); each owns its own frame staging area and result buffers,
 * while the work buffers are shared, so calls in flight together must name the same cuda_stream
 * (ET_ERR_INVALID_ARG otherwise) and run one after the other on the device.  frames_host and the
 * buffers of dst stay the caller's and must remain valid and untouched until the call is collected;
 * pinned memory is needed for the upload to overlap.  params and video_offsets_host are copied.
 * params->forced_plan, params->want_trace and et_profile_enable need the synchronous calls
 * (ET_ERR_INVALID_ARG).  The synchronous encode calls are refused while a call is in flight.
 *
 * et_encode_batch_host_collect waits for that call's kernels, reads its status and sizes, copies
 * tokens and index map into the dst given at submit (ET_ERR_CAPACITY if too small), waits for those
 * copies and fills *out; out's device pointers name the call's slot and stay valid until the second
 * next submit or the next synchronous call.  Calls are collected in submission order (ET_ERR_INVALID_ARG otherwise, and for a
 * ticket that is not in flight).  A call that fails at collect is over: its slot is free again.
 * Results are bit-identical to et_encode_batch_host's on the same inputs. */
ET_API et_status et_encode_batch_host_submit(et_encoder* enc, const float* frames_host, const int* video_offsets_host,
                                      int V, const et_params* params, void* cuda_stream,
                                      const et_host_buffers* dst, unsigned long long* ticket);
ET_API et_status et_encode_batch_host_collect(et_encoder* enc, unsigned long long ticket, et_result* out);

ET_API void et_destroy(et_encoder* enc);
ET_API const char* et_status_string(et_status s);
ET_API const char* et_last_error(const et_encoder* enc); /* text of the last failure on this encoder */

/* Per-category device timings of the encode calls (no counterpart in the paper: measurement aid).
 * While enabled, every encode call brackets its kernel groups with CUDA events on the call's
 * stream and, after its final synchronisation, adds the elapsed times and the algorithmic work
 * (FLOPs for the tensor-core categories, bytes for the bandwidth categories, computed from the
 * frame counts the call actually ran with) to the counters. */
enum {
  ET_CAT_IM2COL = 0,    /* bytes: frames read + patch matrix written */
  ET_CAT_GEMM = 1,      /* flops: 2*M*N*K of every dense layer (patch embed, QKV, out-proj, MLP) */
  ET_CAT_ATTENTION = 2, /* flops: 4*L*L*D per frame per block */
  ET_CAT_LAYERNORM = 3, /* bytes: rows*D*(4 + output element size) */
  ET_CAT_SIMILARITY = 4,/* bytes: n*L*D*4 read once (includes the merge plan, same launch) */
  ET_CAT_PLAN = 5,      /* unused: the plan runs in the tail of the similarity launch */
  ET_CAT_MERGE = 6,     /* bytes: source frames read + output frames written */
  ET_CAT_SCORES = 7,    /* flops: 2*L*L*D per output frame */
  ET_CAT_SELECT = 8,    /* bytes: scores read + mask written */
  ET_CAT_GATHER = 9,    /* bytes: kept rows read + written */
  ET_PROF_CATS = 10
};
typedef struct {
  double ms[ET_PROF_CATS];
  double work[ET_PROF_CATS];
  unsigned long long launches[ET_PROF_CATS];
  int calls;
} et_profile;
/* on != 0: reset the counters and start collecting; 0: stop. */
ET_API et_status et_profile_enable(et_encoder* enc, int on);
ET_API et_status et_profile_read(const et_encoder* enc, et_profile* out);

/* Self-test of the failure-detection path (no counterpart in the paper).  Every tensor-core kernel of the library
 * waits on its barriers with a time limit and, when the limit runs out, records a status word, releases what it
 * holds and returns, which the encode calls report as ET_ERR_TIMEOUT.  This call runs that same bounded wait in a
 * one-warp kernel on a barrier that expects one arrival: with arrive = 0 nothing arrives, the wait runs out after
 * limit_ns (1 .. 1e9 nanoseconds) and the call returns ET_ERR_TIMEOUT; with arrive = 1 a lane arrives and the call
 * returns ET_OK.  Synchronous; the context stays usable either way. */
ET_API et_status et_selftest_bounded_wait(unsigned long long limit_ns, int arrive, void* cuda_stream);

/* The checked build (libearlytom_debug.so, compiled with -DET_DEBUG) verifies the indices the Stage I, Stage II and
 * gather kernels compute before using them; a bad index is recorded and the access skipped (nothing traps).
 * et_debug_build() says whether this library is that build; et_debug_status() returns 0 if no check has failed
 * since the library was loaded (always 0 in the regular build), non-zero otherwise. */
ET_API int et_debug_build(void);
ET_API int et_debug_status(void);

/* Number of kernels the library has launched in this process (all encoders); for benchmarks. */
ET_API unsigned long long et_kernel_launch_count(void);

/* ------------------------------------------------------------------------------------------
 * Single steps of the path on caller-owned device buffers (used by the per-kernel parity tests
 * and by the per-kernel roofline measurements).  All are asynchronous on cuda_stream unless
 * stated; shapes are checked, data is not.
 * ------------------------------------------------------------------------------------------ */

/* Paper Sec. 3.2 "Streaming frame segmentation": sim[t] = mean over the L positions of the cosine
 * between token l of frame t and token l of frame t+1 (denominator clamped at 1e-8), t = 0..n-2.
 * x_dev fp32 [n][L][D]; cos_scratch_dev fp32 [(n-1)*L] (per-position cosines, overwritten);
 * sim_dev fp32 [n-1].  Reductions run in a fixed order: results are bit-reproducible. */
ET_API et_status et_frame_similarity(const float* x_dev, int n, int L, int D, float* cos_scratch_dev, float* sim_dev,
                              void* cuda_stream);

/* The paper has no counterpart to this call: it is et_frame_similarity for callers that cannot
 * allocate device memory (an allocator that already owns the whole card, a thread that may not
 * take the device-wide synchronisation of cudaMalloc/cudaFree, a host that forbids allocation after
 * start-up).  The per-position cosines go to a fixed 256 KiB array inside the library image
 * instead of a caller buffer, so only x_dev (fp32 [n][L][D]) and sim_dev (fp32 [n-1]) are passed;
 * same arithmetic, same reduction order, same results as et_frame_similarity.
 *   - limit: (n-1)*L <= 65536, otherwise ET_ERR_CAPACITY and nothing is launched;
 *   - the call itself never allocates or frees; every GPU that loads the library holds the array
 *     until the process exits;
 *   - the first call on each device looks up the array's device address (host-side, once); make
 *     that first call before any stream capture begins; the address is remembered per device, so a
 *     process that calls cudaDeviceReset must not use this entry point on that device afterwards;
 *   - the array is shared by all calls and keeps the last call's cosines; nothing needs clearing
 *     (every value read is written first), but calls that overlap on the GPU race on it. */
ET_API et_status et_frame_similarity_static(const float* x_dev, int n, int L, int D, float* sim_dev,
                                            void* cuda_stream);

/* Paper Eq. 1-2 / Alg. 1 decisions for V videos from given similarities.  sim_dev [n] (entry t =
 * frames t,t+1; entries at video ends ignored), video_offsets_dev int [V+1].  Outputs (device):
 * seg_start [n], merge_next [n] bytes, ema [n] fp32, n_out int [1], and the plan of the merged
 * list: src_a, src_b int [n] (src_b = -1 for a copy), w_a, w_b fp32 [n] (Eq. 3 weights),
 * new_video_offsets int [V+1]. */
ET_API et_status et_merge_plan(const float* sim_dev, const int* video_offsets_dev, int n, int V, double ema_alpha,
                        double tau_seg, double tau_merge, int weighted_merge, unsigned char* seg_start_dev,
                        unsigned char* merge_next_dev, float* ema_dev, int* n_out_dev, int* src_a_dev,
                        int* src_b_dev, float* w_a_dev, float* w_b_dev, int* new_video_offsets_dev,
                        void* cuda_stream);

/* Paper Eq. 3 + frame compaction: y[j] = w_a[j] * x[src_a[j]] + w_b[j] * x[src_b[j]] (copy when
 * src_b[j] < 0) for j < *n_out_dev.  x_dev [n][L*D] fp32, y_dev [>= n_out][L*D] fp32, distinct. */
ET_API et_status et_merge_frames(const float* x_dev, float* y_dev, int n_cap, int frame_elems, const int* n_out_dev,
                          const int* src_a_dev, const int* src_b_dev, const float* w_a_dev, const float* w_b_dev,
                          void* cuda_stream);

/* Paper Eq. 4 / Eq. 6: keep mask of N frames from scores [N][L]; frame f keeps its k_dev[f]
 * highest scores (ties to the lower index) when dynamic_dev[f] != 0, else the first maximum of
 * each local window: runs of w_dev[f] positions (window_mode 0) or k_dev[f] near-equal runs
 * (window_mode 1, see et_params).  k and w are clamped to [1, L]; a NaN score ranks below every
 * number.  keep_dev bytes [N][L], count_dev int [N] = bytes set in each row. */
ET_API et_status et_select_tokens(const float* scores_dev, const unsigned char* dynamic_dev, const int* k_dev,
                           const int* w_dev, int N, int L, int window_mode, unsigned char* keep_dev, int* count_dev,
                           void* cuda_stream);

/* Paper Eq. 7: gather the kept rows of x_dev fp32 [N][L][D] in order into tokens_dev
 * [sum count][D] (optionally through LayerNorm with gain/shift ln_g_dev/ln_b_dev, NULL = none),
 * writing frame_offsets_dev int [N+1] and token_pos_dev int [sum count].  Synchronous: returns
 * the token count in *n_tokens_host. */
ET_API et_status et_gather_tokens(const float* x_dev, const unsigned char* keep_dev, int N, int L, int D,
                           const float* ln_g_dev, const float* ln_b_dev, float ln_eps, float* tokens_dev,
                           size_t tokens_capacity_rows, int* frame_offsets_dev, int* token_pos_dev,
                           int* n_tokens_host, void* cuda_stream);

/* Dense layer on the tensor cores (the GEMMs of the encoder blocks, paper Eq. 8's 4LD^2 + 2LDM
 * terms): c = epilogue(a[M][K] * w[N][K]^T + bias[N]).  a_dev, w_dev bf16 (K contiguous, K*2 bytes
 * a multiple of 16); epilogue 0: store bf16; 1: GELU then store bf16; 2: c fp32 += result
 * (residual, in place); 3: c fp32 = result + table[(row % table_rows)][N] (position embedding);
 * 4: gated feed-forward of the language model (earlytom_llm.h): the rows of w are ordered in tiles of
 * 256 = four groups of (32 gate rows, 32 up rows) of the same 32 outputs, bias [N] follows the same order, N % 256 == 0
 * and c is bf16 [M][N/2] = silu(gate + bias) * (up + bias).
 * status_dev int [1] receives a non-zero code if a bounded wait expired. */
ET_API et_status et_linear_bf16(const void* a_dev, const void* w_dev, const float* bias_dev, void* c_dev, int M, int N,
                         int K, int epilogue, int gelu_tanh, const float* table_dev, int table_rows,
                         int* status_dev, void* cuda_stream);

/* Per-frame multi-head attention (paper Sec. 3.1, softmax(QK^T/sqrt(d))V inside each frame).
 * qkv_dev [n*L][3D] (Q|K|V), out_dev [n*L][D], both fp32 (dtype 0) or bf16 (dtype 1);
 * lse_dev fp32 [n][heads][L] receives the row log-sum-exp (natural log, of the scaled logits). */
ET_API et_status et_attention(const void* qkv_dev, void* out_dev, float* lse_dev, int n, int L, int heads, int head_dim,
                       int dtype, void* cuda_stream);

/* The same inside windows (the Qwen2.5-VL-style encoder of et_config.arch 1): the rows of a frame are ordered so that a
 * window is a run of window_rows consecutive rows (window_rows divides L), and a query attends only to the keys of its
 * own window.  lse_scratch_dev fp32 [n][heads][L] is overwritten with values whose layout is not specified. */
ET_API et_status et_attention_windowed(const void* qkv_dev, void* out_dev, float* lse_scratch_dev, int n, int L, int heads,
                                int head_dim, int window_rows, int dtype, void* cuda_stream);

/* Per-token attention score of Alg. 2's input A: score[f][j] = mean over heads and queries of
 * softmax(QK^T/sqrt(d))[q][j], recomputed from qkv_dev and lse_dev.  partial_dev fp32
 * [n][heads][L] is scratch.  score_dev fp32 [n][L]. */
ET_API et_status et_attention_scores(const void* qkv_dev, const float* lse_dev, float* partial_dev, float* score_dev, int n,
                              int L, int heads, int head_dim, int dtype, void* cuda_stream);

/* LayerNorm over the last axis: x_dev fp32 [rows][D] -> y_dev fp32 (dtype 0) or bf16 (dtype 1). */
ET_API et_status et_layernorm(const float* x_dev, const float* g_dev, const float* b_dev, float eps, void* y_dev, int rows,
                       int D, int dtype, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* EARLYTOM_H_ */
