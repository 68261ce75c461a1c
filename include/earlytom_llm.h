/* earlytom_llm.h -- the stage downstream of the compressed encoder: projector and language-model prefill
 * up to the first generated token, i.e. the rest of the time-to-first-token that the paper profiles
 * (Sec. 3.1, "Video-LLM inference" and "Profiling of time-to-first-token"; Fig. 1 splits it into vision
 * encoding, visual token processing, LLM prefill and system overhead).
 *
 * The paper names the model (LLaVA-OneVision-7B) but prints nothing of its architecture; this library
 * follows the public architecture of that model: a two-layer GELU projector from the encoder's width to
 * the language model's, and a Qwen2-style pre-norm decoder -- RMSNorm, grouped-query causal attention with
 * rotate-half rotary position embedding on positions 0..n-1 and scale 1/sqrt(head_dim), biases on the
 * Q/K/V projection only, SwiGLU feed-forward, final RMSNorm, untied output head.  The sequence is
 * [text before the video | visual tokens in the encoder's output order | text after the video].
 *
 * Arithmetic: bf16 tensor-core GEMMs with fp32 accumulation, fp32 residual stream, fp32 norm statistics and
 * softmax, bf16 activations between kernels (the same scheme as the encoder's bf16 path).  There is no
 * fp32 path and no CPU fallback.  sm_100a only.
 *
 * Conventions are those of earlytom.h: every call returns et_status, nothing throws, device pointers are
 * marked _dev, host pointers _host.  One et_llm = one GPU = one call in flight.
 */
#ifndef EARLYTOM_LLM_H
#define EARLYTOM_LLM_H

#include "earlytom.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct et_llm et_llm; /* opaque */

typedef struct {
  int vision_hidden;      /* width of the encoder's tokens (1152 for SigLIP-so400m) */
  int hidden;             /* multiple of 8, <= 4096 */
  int num_layers;
  int heads, kv_heads;    /* heads % kv_heads == 0 */
  int head_dim;           /* 128 (the tensor-core attention kernel is written for it) */
  int mlp_dim;            /* multiple of 8 */
  int vocab;              /* multiple of 8 */
  float rms_eps;
  float rope_theta;
  int gelu_tanh;          /* projector activation: 1 tanh approximation, 0 erf form */
  int max_tokens;         /* workspace capacity: sequence length of one call */
  int keep_kv_cache;      /* 1: every layer's keys (after the rotary embedding) and values are kept for decoding */
} et_llm_config;

/* fp32 blob in this fixed order (row-major, a linear layer is y = x W + b with W [in][out]):
 *   embed [vocab][hidden]
 *   proj_w1 [vision_hidden][hidden], proj_b1 [hidden], proj_w2 [hidden][hidden], proj_b2 [hidden]
 *   per layer: rms1_g [hidden]; wqkv [hidden][(heads+2*kv_heads)*head_dim], bqkv [...];
 *              wo [heads*head_dim][hidden]; rms2_g [hidden];
 *              wgu [hidden][2*mlp_dim] (gate columns, then up columns); wd [mlp_dim][hidden]
 *   final_g [hidden]; lm_head [hidden][vocab]
 * wqkv's output columns are [Q | K | V]; query head h reads key / value head h / (heads / kv_heads).
 * on_device = 0: data is host memory; 1: data is device memory on the current device (for blobs too large
 * to stage through the host).  Either way the library converts into its own bf16 copies during create
 * and never touches data afterwards. */
typedef struct {
  const float* data;
  size_t count;
  int on_device;
} et_llm_weights;

/* Device pointers are owned by the model and valid until its next call or et_llm_destroy. */
typedef struct {
  int n_tokens;              /* sequence length = n_prefix + n_visual + n_suffix */
  int first_token;           /* argmax of the logits of the last position (lowest id among equals) */
  const float* logits;       /* device fp32 [vocab], last position */
  const float* hidden;       /* device fp32 [n_tokens][hidden]: residual stream after the last layer */
  const void* kv_cache;      /* NULL unless keep_kv_cache: device bf16 [num_layers][kv_cache_rows][2*kv_heads*head_dim],
                                row p of a layer = [keys of position p, rotated | values of position p]; rows >= n_tokens
                                are stale */
  int kv_cache_rows;         /* row count of one layer's slab (the capacity, a multiple of 256) */
} et_llm_result;

/* Errors: ET_ERR_SHAPE for widths the kernels do not cover, ET_ERR_WEIGHTS when count does not match the
 * layout, ET_ERR_OOM / ET_ERR_CUDA from the allocations and conversions. */
ET_API et_status et_llm_create(const et_llm_config* config, const et_llm_weights* weights, et_llm** out);

/* Prefill of one sequence.  prefix_ids_host / suffix_ids_host: token ids of the text before / after the
 * video (either may be empty: NULL with count 0); visual_tokens_dev: device fp32 [n_visual][vision_hidden],
 * e.g. et_result.tokens of the encoder on the same device (n_visual may be 0).  Runs on cuda_stream and
 * synchronises it once at the end to read the first token.  ET_ERR_CAPACITY if the sequence is longer than
 * max_tokens, ET_ERR_INVALID_ARG for an empty sequence or an id outside the vocabulary, ET_ERR_TIMEOUT if a
 * bounded device-side wait expired. */
ET_API et_status et_llm_prefill(et_llm* llm, const int* prefix_ids_host, int n_prefix, const float* visual_tokens_dev,
                                int n_visual, const int* suffix_ids_host, int n_suffix, void* cuda_stream,
                                et_llm_result* out);

ET_API void et_llm_destroy(et_llm* llm);
ET_API const char* et_llm_last_error(const et_llm* llm);

/* Per-stage device times (CUDA events) and launch counts summed over the calls since enable. */
enum { ET_LLM_EMBED = 0, ET_LLM_NORM = 1, ET_LLM_GEMM = 2, ET_LLM_ROPE = 3, ET_LLM_ATTENTION = 4, ET_LLM_SWIGLU = 5,
       ET_LLM_HEAD = 6, ET_LLM_CATS = 8 };
typedef struct {
  double ms[ET_LLM_CATS];
  unsigned long long launches[ET_LLM_CATS];
  int calls;
} et_llm_profile;
ET_API et_status et_llm_profile_enable(et_llm* llm, int on);
ET_API et_status et_llm_profile_read(const et_llm* llm, et_llm_profile* out);

/* ---- single steps on caller-owned device buffers (per-kernel parity tests and measurements) ---- */

/* y = x * rsqrt(mean(x^2) + eps) * g; x fp32 [rows][D], g fp32 [D], y bf16 [rows][D]; D % 4 == 0, D <= 4096. */
ET_API et_status et_rmsnorm(const float* x_dev, const float* g_dev, float eps, void* y_dev, int rows, int D, void* cuda_stream);

/* Rotary position embedding, rotate-half form, in place on the Q and K parts of packed bf16 rows
 * [rows][(heads + 2*kv_heads)*head_dim]; row r has position r % L; element i < head_dim/2 of a head pairs
 * with i + head_dim/2 and the pair turns by position * theta^(-2i/head_dim).  head_dim % 16 == 0, <= 256.
 * Allocates and frees its table of angles (min(L, rows) * head_dim/2 cosine / sine pairs) and synchronises the
 * stream; the model keeps such a table for its whole capacity instead. */
ET_API et_status et_rope(void* qkv_dev, int rows, int L, int heads, int kv_heads, int head_dim, float theta, void* cuda_stream);

/* h[r][j] = silu(gu[r][j]) * gu[r][M + j]; gu bf16 [rows][2M], h bf16 [rows][M]; M % 8 == 0. */
ET_API et_status et_swiglu(const void* gu_dev, void* h_dev, int rows, int M, void* cuda_stream);

/* Causal grouped-query attention (Sec. 3.1: softmax(Q K^T / sqrt(d)) V, query i sees keys 0..i) of n_seq
 * sequences of L positions; qkv bf16 [n_seq*L][(heads + 2*kv_heads)*128] packed [Q | K | V], out bf16
 * [n_seq*L][heads*128].  head_dim must be 128.  status_dev (int, may be NULL) receives a non-zero code if a
 * bounded wait inside the kernel expired. */
ET_API et_status et_attention_causal(const void* qkv_dev, void* out_dev, int n_seq, int L, int heads, int kv_heads,
                                     int head_dim, int* status_dev, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* EARLYTOM_LLM_H */
