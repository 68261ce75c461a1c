// C-ABI entry points and host orchestration of the stage downstream of the encoder: projector and
// language-model prefill up to the first token.  This file only converts weights, sequences the kernels
// of the other translation units on one stream and reads the first token back.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

#include "common.cuh"
#include "earlytom_llm.h"

namespace et {
namespace {

// dst[row(n)][K] (bf16) = src[k][n] (fp32).  row(n) = n, or, for a gated feed-forward weight with columns
// [gate (gated_M) | up (gated_M)], the order the fused epilogue wants: tiles of 256 rows = 128 outputs, inside a
// tile four groups of (32 gate rows, 32 up rows) of the same 32 outputs.
__global__ void transpose_weight_kernel(const float* __restrict__ src, bf16* __restrict__ dst, int K, int N, int gated_M) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int k = k0 + i, n = n0 + threadIdx.x;
    tile[i][threadIdx.x] = (k < K && n < N) ? src[(size_t)k * N + n] : 0.f;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int n = n0 + i, k = k0 + threadIdx.x;
    if (n < N && k < K) {
      int row = n;
      if (gated_M > 0) {
        const int up = n >= gated_M ? 1 : 0, j = n - up * gated_M;
        row = (j >> 7) * 256 + ((j & 127) >> 5) * 64 + up * 32 + (j & 31);
      }
      dst[(size_t)row * K + k] = __float2bfloat16_rn(tile[threadIdx.x][i]);
    }
  }
}

struct Dense {            // one linear layer: bf16 weight [N][K] and its tensor maps
  bf16* w = nullptr;
  WeightDesc d;
  int N = 0, K = 0;
};

struct LlmLayer {
  const float *rms1_g, *bqkv, *rms2_g;
  Dense qkv, o, gu, down;
};

}  // namespace
}  // namespace et

using namespace et;

struct et_llm {
  et_llm_config cfg{};
  int device = 0, cap = 0;
  bool fused_gate = false;
  int q_dim = 0, kv_dim = 0, qkv_dim = 0;
  std::string last_error;
  std::vector<void*> dev_allocs, host_allocs;

  float* small = nullptr;            // fp32 copies of the gains and biases, in blob order
  bf16* embed = nullptr;             // [vocab][hidden]
  const float *proj_b1 = nullptr, *proj_b2 = nullptr, *final_g = nullptr;
  Dense proj1, proj2, head;
  std::vector<LlmLayer> layers;
  float* zeros = nullptr;            // bias of the layers that have none
  double* inv_turns = nullptr;       // [head_dim/2] rotary frequencies in turns per position
  float2* rope_table = nullptr;      // [cap][head_dim/2] (cos, sin) of every position
  bf16* kv_cache = nullptr;          // [layers][cap][2*kv_dim] when the model keeps keys and values

  float *X = nullptr, *logits = nullptr;
  bf16 *Xn = nullptr, *QKV = nullptr, *O = nullptr, *GU = nullptr, *Hm = nullptr, *Vb = nullptr, *P1 = nullptr, *Xl = nullptr;
  TmaDesc a_Xn, a_O, a_Hm, a_Vb, a_P1, a_Xl;        // operand maps
  TmaDesc c_X, c_QKV, c_GU, c_Hm, c_P1, c_logits;    // output maps
  int* ids = nullptr;                // device [cap]
  int* d_small = nullptr;            // [0] first token, [1] status
  int *h_ids = nullptr, *h_small = nullptr;          // pinned

  bool prof_on = false;
  et_llm_profile prof{};
  std::vector<cudaEvent_t> events;
  struct Span { int cat, ev; unsigned long long l0, l1; };
  std::vector<Span> spans;
  size_t next_event = 0;
};

namespace {

et_status lfail(et_llm* m, et_status st, const std::string& msg) {
  if (m) m->last_error = msg;
  return st;
}

#define LLM_CUDA(m, call)                                                                          \
  do {                                                                                             \
    cudaError_t err__ = (call);                                                                    \
    if (err__ != cudaSuccess)                                                                      \
      return lfail((m), err__ == cudaErrorMemoryAllocation ? ET_ERR_OOM : ET_ERR_CUDA,             \
                   std::string(#call) + ": " + cudaGetErrorString(err__));                         \
  } while (0)
#define LLM_TRY(x)                     \
  do {                                 \
    et_status st__ = (x);              \
    if (st__ != ET_OK) return st__;    \
  } while (0)

template <typename T>
et_status dalloc(et_llm* m, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t err = cudaMalloc(&q, std::max<size_t>(count, 1) * sizeof(T));
  if (err != cudaSuccess) return lfail(m, ET_ERR_OOM, std::string("cudaMalloc: ") + cudaGetErrorString(err));
  m->dev_allocs.push_back(q);
  *p = reinterpret_cast<T*>(q);
  return ET_OK;
}

void span_begin(et_llm* m, int cat, cudaStream_t s) {
  if (!m->prof_on) return;
  while (m->next_event + 2 > m->events.size()) {
    cudaEvent_t ev;
    if (cudaEventCreate(&ev) != cudaSuccess) return;
    m->events.push_back(ev);
  }
  m->spans.push_back({cat, (int)m->next_event, g_kernel_launches.load(), 0});
  cudaEventRecord(m->events[m->next_event], s);
  m->next_event += 2;
}
void span_end(et_llm* m, cudaStream_t s) {
  if (!m->prof_on || m->spans.empty()) return;
  m->spans.back().l1 = g_kernel_launches.load();
  cudaEventRecord(m->events[m->spans.back().ev + 1], s);
}
#define SPAN(cat, ...)       \
  do {                       \
    span_begin(m, (cat), s); \
    __VA_ARGS__;             \
    span_end(m, s);          \
  } while (0)

et_status validate(const et_llm_config* c) {
  if (!c) return ET_ERR_INVALID_ARG;
  if (c->vision_hidden < 8 || c->vision_hidden % 8) return ET_ERR_SHAPE;
  if (c->hidden < 8 || c->hidden % 8 || c->hidden > 4096) return ET_ERR_SHAPE;
  if (c->num_layers < 1 || c->num_layers > 256) return ET_ERR_SHAPE;
  if (c->heads < 1 || c->kv_heads < 1 || c->heads % c->kv_heads) return ET_ERR_SHAPE;
  if (!attention_causal_supported(c->head_dim)) return ET_ERR_SHAPE;
  if (c->mlp_dim < 8 || c->mlp_dim % 8 || c->vocab < 8 || c->vocab % 8) return ET_ERR_SHAPE;
  if (!(c->rms_eps > 0.f) || !(c->rope_theta > 1.f)) return ET_ERR_INVALID_ARG;
  if (c->max_tokens < 1 || c->max_tokens > (1 << 20)) return ET_ERR_INVALID_ARG;
  if (c->keep_kv_cache != 0 && c->keep_kv_cache != 1) return ET_ERR_INVALID_ARG;
  return ET_OK;
}

size_t llm_blob_floats(const et_llm_config& c) {
  const size_t H = c.hidden, V = c.vocab, M = c.mlp_dim, q = (size_t)c.heads * c.head_dim,
               qkv = (size_t)(c.heads + 2 * c.kv_heads) * c.head_dim;
  const size_t per_layer = H + H * qkv + qkv + q * H + H + H * 2 * M + M * H;
  return V * H + (size_t)c.vision_hidden * H + H + H * H + H + per_layer * c.num_layers + H + H * V;
}

// c = epi(a w^T + bias) with live rows M
et_status dense(et_llm* m, const TmaDesc& a, const Dense& w, const TmaDesc& cmap, const float* bias, void* c, int M, int epi,
                cudaStream_t s) {
  LLM_CUDA(m, launch_gemm_bf16(a, w.d, cmap, bias ? bias : m->zeros, c, M, w.N, w.K, epi, m->cfg.gelu_tanh, nullptr, 1, nullptr, 1,
                               m->d_small + 1, s));
  return ET_OK;
}

}  // namespace

extern "C" {

et_status et_llm_create(const et_llm_config* config, const et_llm_weights* weights, et_llm** out) {
  if (!config || !weights || !weights->data || !out) return ET_ERR_INVALID_ARG;
  et_status st = validate(config);
  if (st != ET_OK) return st;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return ET_ERR_CUDA;
  if (weights->count != llm_blob_floats(*config)) return ET_ERR_WEIGHTS;

  et_llm* m = new (std::nothrow) et_llm();
  if (!m) return ET_ERR_OOM;
  auto bail = [&](et_status s2) { et_llm_destroy(m); return s2; };
  m->cfg = *config;
  const et_llm_config& c = m->cfg;
  if (cudaGetDevice(&m->device) != cudaSuccess) return bail(ET_ERR_CUDA);
  const size_t H = c.hidden, V = c.vocab, M = c.mlp_dim, vh = c.vision_hidden;
  m->q_dim = c.heads * c.head_dim; m->kv_dim = c.kv_heads * c.head_dim; m->qkv_dim = m->q_dim + 2 * m->kv_dim;
  const size_t qd = m->q_dim, qkv = m->qkv_dim;
  m->cap = (c.max_tokens + 255) / 256 * 256;          // whole row tiles: operand loads never leave the buffers
  m->fused_gate = c.mlp_dim % 128 == 0;               // SwiGLU inside the gate/up layer's epilogue (whole 128-output tiles)
  const size_t cap = m->cap;

  // ---- weights: a staging buffer for host blobs, bf16 copies of the matrices, fp32 copies of the vectors
  const size_t biggest = std::max<size_t>({V * H, H * 2 * M, H * qkv, vh * H});
  float* stage = nullptr;
  if (!weights->on_device && cudaMalloc(&stage, biggest * sizeof(float)) != cudaSuccess) return bail(ET_ERR_OOM);
  auto done_stage = [&]() { if (stage) cudaFree(stage); stage = nullptr; };
  auto bail2 = [&](et_status s2) { done_stage(); return bail(s2); };
  size_t off = 0;
  // device pointer to the next `n` floats of the blob (staged if the blob is host memory)
  auto next = [&](size_t n, const float** p) -> et_status {
    const float* src = weights->data + off;
    off += n;
    if (weights->on_device) { *p = src; return ET_OK; }
    if (cudaDeviceSynchronize() != cudaSuccess) return ET_ERR_CUDA;      // the previous conversion still reads the stage
    if (cudaMemcpy(stage, src, n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) return ET_ERR_CUDA;
    *p = stage;
    return ET_OK;
  };
  const char* err = nullptr;
  auto matrix = [&](int K, int N, Dense* d, int gated_M = 0) -> et_status {       // blob holds w [K][N]
    const float* src = nullptr;
    et_status s2 = next((size_t)K * N, &src);
    if (s2 != ET_OK) return s2;
    if ((s2 = dalloc(m, &d->w, (size_t)N * K)) != ET_OK) return s2;
    ET_COUNT_LAUNCH();
    transpose_weight_kernel<<<dim3(cdiv(N, 32), cdiv(K, 32)), dim3(32, 8)>>>(src, d->w, K, N, gated_M);
    if (cudaGetLastError() != cudaSuccess) return ET_ERR_CUDA;
    d->N = N; d->K = K;
    return make_tma_weight(&d->d, d->w, N, K, &err) ? ET_OK : ET_ERR_CUDA;
  };
  size_t n_small = H + H + H + (size_t)c.num_layers * (2 * H + qkv);
  if ((st = dalloc(m, &m->small, n_small)) != ET_OK) return bail2(st);
  size_t small_off = 0;
  auto vector_f32 = [&](size_t n, const float** p) -> et_status {
    float* dst = m->small + small_off;
    small_off += n;
    const float* src = weights->data + off;
    off += n;
    if (cudaMemcpy(dst, src, n * sizeof(float), weights->on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice) != cudaSuccess)
      return ET_ERR_CUDA;
    *p = dst;
    return ET_OK;
  };
  {
    const float* src = nullptr;
    if ((st = next(V * H, &src)) != ET_OK) return bail2(st);
    if ((st = dalloc(m, &m->embed, V * H)) != ET_OK) return bail2(st);
    launch_cast_bf16(src, m->embed, V * H, 0);
  }
  if ((st = matrix((int)vh, (int)H, &m->proj1)) != ET_OK) return bail2(st);
  if ((st = vector_f32(H, &m->proj_b1)) != ET_OK) return bail2(st);
  if ((st = matrix((int)H, (int)H, &m->proj2)) != ET_OK) return bail2(st);
  if ((st = vector_f32(H, &m->proj_b2)) != ET_OK) return bail2(st);
  m->layers.resize(c.num_layers);
  for (LlmLayer& l : m->layers) {
    if ((st = vector_f32(H, &l.rms1_g)) != ET_OK) return bail2(st);
    if ((st = matrix((int)H, (int)qkv, &l.qkv)) != ET_OK) return bail2(st);
    if ((st = vector_f32(qkv, &l.bqkv)) != ET_OK) return bail2(st);
    if ((st = matrix((int)qd, (int)H, &l.o)) != ET_OK) return bail2(st);
    if ((st = vector_f32(H, &l.rms2_g)) != ET_OK) return bail2(st);
    if ((st = matrix((int)H, (int)(2 * M), &l.gu, m->fused_gate ? (int)M : 0)) != ET_OK) return bail2(st);
    if ((st = matrix((int)M, (int)H, &l.down)) != ET_OK) return bail2(st);
  }
  if ((st = vector_f32(H, &m->final_g)) != ET_OK) return bail2(st);
  if ((st = matrix((int)H, (int)V, &m->head)) != ET_OK) return bail2(st);
  if (cudaDeviceSynchronize() != cudaSuccess) return bail2(ET_ERR_CUDA);
  done_stage();

  const size_t widest = std::max<size_t>({2 * M, V, H, qkv});
  if ((st = dalloc(m, &m->zeros, widest)) != ET_OK) return bail(st);
  cudaMemset(m->zeros, 0, widest * sizeof(float));
  {
    const int half = c.head_dim / 2;
    std::vector<double> t(half);
    for (int i = 0; i < half; ++i) t[i] = pow((double)c.rope_theta, -2.0 * i / (double)c.head_dim) / (2.0 * M_PI);
    if ((st = dalloc(m, &m->inv_turns, (size_t)half)) != ET_OK) return bail(st);
    if (cudaMemcpy(m->inv_turns, t.data(), half * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) return bail(ET_ERR_CUDA);
    if ((st = dalloc(m, &m->rope_table, cap * half)) != ET_OK) return bail(st);
    launch_rope_table(m->rope_table, (int)cap, c.head_dim, m->inv_turns, 0);
  }

  // ---- activations (zeroed once: rows beyond the live count are read, never stored, by tile loads)
#define LLM_A(ptr, count)                                                \
  do {                                                                   \
    if ((st = dalloc(m, &(ptr), (count))) != ET_OK) return bail(st);     \
    cudaMemset((ptr), 0, (count) * sizeof(*(ptr)));                      \
  } while (0)
  LLM_A(m->X, cap * H); LLM_A(m->Xn, cap * H); LLM_A(m->QKV, cap * qkv); LLM_A(m->O, cap * qd);
  LLM_A(m->GU, m->fused_gate ? 8 : cap * 2 * M); LLM_A(m->Hm, cap * M); LLM_A(m->Vb, cap * vh); LLM_A(m->P1, cap * H);
  if (c.keep_kv_cache) LLM_A(m->kv_cache, (size_t)c.num_layers * cap * 2 * m->kv_dim);
  LLM_A(m->Xl, 256 * H); LLM_A(m->logits, 32 * V); LLM_A(m->ids, cap); LLM_A(m->d_small, (size_t)4);
#undef LLM_A
  void* hp = nullptr;
  if (cudaMallocHost(&hp, cap * sizeof(int)) != cudaSuccess) return bail(ET_ERR_OOM);
  m->host_allocs.push_back(hp); m->h_ids = (int*)hp;
  if (cudaMallocHost(&hp, 4 * sizeof(int)) != cudaSuccess) return bail(ET_ERR_OOM);
  m->host_allocs.push_back(hp); m->h_small = (int*)hp;

  bool ok = make_tma_2d_bf16(&m->a_Xn, m->Xn, cap, H, 128, &err) && make_tma_2d_bf16(&m->a_O, m->O, cap, qd, 128, &err) &&
            make_tma_2d_bf16(&m->a_Hm, m->Hm, cap, M, 128, &err) && make_tma_2d_bf16(&m->a_Vb, m->Vb, cap, vh, 128, &err) &&
            make_tma_2d_bf16(&m->a_P1, m->P1, cap, H, 128, &err) && make_tma_2d_bf16(&m->a_Xl, m->Xl, 256, H, 128, &err) &&
            make_tma_out(&m->c_X, m->X, cap, H, true, &err) && make_tma_out(&m->c_QKV, m->QKV, cap, qkv, false, &err) &&
            (m->fused_gate ? make_tma_out(&m->c_Hm, m->Hm, cap, M, false, &err) : make_tma_out(&m->c_GU, m->GU, cap, 2 * M, false, &err)) &&
            make_tma_out(&m->c_P1, m->P1, cap, H, false, &err) &&
            make_tma_out(&m->c_logits, m->logits, 32, V, true, &err);
  if (!ok) return bail(lfail(m, ET_ERR_CUDA, err ? err : "tensor map"));
  if (cudaDeviceSynchronize() != cudaSuccess) return bail(ET_ERR_CUDA);
  *out = m;
  return ET_OK;
}

void et_llm_destroy(et_llm* m) {
  if (!m) return;
  for (void* p : m->dev_allocs) cudaFree(p);
  for (void* p : m->host_allocs) cudaFreeHost(p);
  for (cudaEvent_t ev : m->events) cudaEventDestroy(ev);
  delete m;
}

const char* et_llm_last_error(const et_llm* m) { return m ? m->last_error.c_str() : ""; }

et_status et_llm_prefill(et_llm* m, const int* prefix_ids_host, int n_prefix, const float* visual_tokens_dev, int n_visual,
                         const int* suffix_ids_host, int n_suffix, void* cuda_stream, et_llm_result* out) {
  if (!m || !out) return lfail(m, ET_ERR_INVALID_ARG, "null argument");
  if (n_prefix < 0 || n_visual < 0 || n_suffix < 0) return lfail(m, ET_ERR_INVALID_ARG, "negative count");
  if ((n_prefix > 0 && !prefix_ids_host) || (n_suffix > 0 && !suffix_ids_host) || (n_visual > 0 && !visual_tokens_dev))
    return lfail(m, ET_ERR_INVALID_ARG, "null pointer with a non-zero count");
  const long long n_ll = (long long)n_prefix + n_visual + n_suffix;
  if (n_ll < 1) return lfail(m, ET_ERR_INVALID_ARG, "empty sequence");
  if (n_ll > m->cfg.max_tokens) return lfail(m, ET_ERR_CAPACITY, "sequence longer than max_tokens");
  const et_llm_config& c = m->cfg;
  const int n = (int)n_ll, H = c.hidden, Mlp = c.mlp_dim;
  for (int i = 0; i < n_prefix; ++i)
    if (prefix_ids_host[i] < 0 || prefix_ids_host[i] >= c.vocab) return lfail(m, ET_ERR_INVALID_ARG, "token id outside the vocabulary");
  for (int i = 0; i < n_suffix; ++i)
    if (suffix_ids_host[i] < 0 || suffix_ids_host[i] >= c.vocab) return lfail(m, ET_ERR_INVALID_ARG, "token id outside the vocabulary");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  LLM_CUDA(m, cudaSetDevice(m->device));
  m->spans.clear();
  m->next_event = 0;
  LLM_CUDA(m, cudaMemsetAsync(m->d_small, 0, 4 * sizeof(int), s));

  // ---- the sequence: embeddings of the text, projected visual tokens between them
  const int n_text = n_prefix + n_suffix;
  if (n_text > 0) {
    if (n_prefix) memcpy(m->h_ids, prefix_ids_host, sizeof(int) * n_prefix);
    if (n_suffix) memcpy(m->h_ids + n_prefix, suffix_ids_host, sizeof(int) * n_suffix);
    LLM_CUDA(m, cudaMemcpyAsync(m->ids, m->h_ids, sizeof(int) * n_text, cudaMemcpyHostToDevice, s));
    SPAN(ET_LLM_EMBED, {
      launch_embed_rows(m->embed, m->ids, m->X, n_prefix, H, c.vocab, s);
      launch_embed_rows(m->embed, m->ids + n_prefix, m->X + (size_t)(n_prefix + n_visual) * H, n_suffix, H, c.vocab, s);
    });
  }
  if (n_visual > 0) {
    float* xv = m->X + (size_t)n_prefix * H;
    TmaDesc c_xv;
    const char* err = nullptr;
    if (!make_tma_out(&c_xv, xv, n_visual, H, true, &err)) return lfail(m, ET_ERR_CUDA, err ? err : "tensor map");
    SPAN(ET_LLM_EMBED, launch_cast_bf16(visual_tokens_dev, m->Vb, (size_t)n_visual * c.vision_hidden, s));
    SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_Vb, m->proj1, m->c_P1, m->proj_b1, m->P1, n_visual, EPI_GELU, s)));
    LLM_CUDA(m, cudaMemsetAsync(xv, 0, sizeof(float) * (size_t)n_visual * H, s));      // the residual epilogue adds into zeros
    SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_P1, m->proj2, c_xv, m->proj_b2, xv, n_visual, EPI_RESIDUAL, s)));
  }

  // ---- decoder layers
  CausalMaps attn_map;
  if (!make_causal_attention_map(&attn_map, m->QKV, n, c.heads, c.kv_heads)) return lfail(m, ET_ERR_CUDA, "tensor map of the attention operands");
  int layer_index = 0;
  for (const LlmLayer& l : m->layers) {
    SPAN(ET_LLM_NORM, launch_rmsnorm(m->X, l.rms1_g, c.rms_eps, m->Xn, n, H, s));
    SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_Xn, l.qkv, m->c_QKV, l.bqkv, m->QKV, n, EPI_STORE, s)));
    SPAN(ET_LLM_ROPE, launch_rope(m->QKV, n, n, c.heads, c.kv_heads, c.head_dim, m->rope_table, s));
    if (m->kv_cache)        // the K | V columns of the packed rows, as they are after the rotation
      SPAN(ET_LLM_ROPE, launch_copy_columns(m->QKV + m->q_dim, m->kv_cache + (size_t)layer_index * m->cap * 2 * m->kv_dim, n, 2 * m->kv_dim,
                                           m->qkv_dim, 2 * m->kv_dim, s));
    ++layer_index;
    SPAN(ET_LLM_ATTENTION, LLM_CUDA(m, launch_attention_causal(attn_map, m->O, 1, n, c.heads, c.kv_heads, m->d_small + 1, s)));
    SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_O, l.o, m->c_X, nullptr, m->X, n, EPI_RESIDUAL, s)));
    SPAN(ET_LLM_NORM, launch_rmsnorm(m->X, l.rms2_g, c.rms_eps, m->Xn, n, H, s));
    if (m->fused_gate) {
      SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_Xn, l.gu, m->c_Hm, nullptr, m->Hm, n, EPI_SWIGLU, s)));
    } else {
      SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_Xn, l.gu, m->c_GU, nullptr, m->GU, n, EPI_STORE, s)));
      SPAN(ET_LLM_SWIGLU, launch_swiglu(m->GU, m->Hm, n, Mlp, s));
    }
    SPAN(ET_LLM_GEMM, LLM_TRY(dense(m, m->a_Hm, l.down, m->c_X, nullptr, m->X, n, EPI_RESIDUAL, s)));
  }

  // ---- first token: final norm of the last position, output head, argmax
  SPAN(ET_LLM_HEAD, {
    launch_rmsnorm(m->X + (size_t)(n - 1) * H, m->final_g, c.rms_eps, m->Xl, 1, H, s);
    LLM_CUDA(m, cudaMemsetAsync(m->logits, 0, sizeof(float) * c.vocab, s));
    LLM_TRY(dense(m, m->a_Xl, m->head, m->c_logits, nullptr, m->logits, 1, EPI_RESIDUAL, s));
    launch_argmax(m->logits, c.vocab, m->d_small, s);
  });
  LLM_CUDA(m, cudaMemcpyAsync(m->h_small, m->d_small, 4 * sizeof(int), cudaMemcpyDeviceToHost, s));
  LLM_CUDA(m, cudaGetLastError());
  LLM_CUDA(m, cudaStreamSynchronize(s));
  if (m->h_small[1] == DS_WAIT_EXPIRED) return lfail(m, ET_ERR_TIMEOUT, "a bounded device-side wait expired in a tensor-core kernel");
  if (m->h_small[1] != 0) return lfail(m, ET_ERR_CUDA, "device status " + std::to_string(m->h_small[1]));

  if (m->prof_on) {
    for (const et_llm::Span& sp : m->spans) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, m->events[sp.ev], m->events[sp.ev + 1]) == cudaSuccess) m->prof.ms[sp.cat] += ms;
      m->prof.launches[sp.cat] += sp.l1 - sp.l0;
    }
    m->prof.calls += 1;
  }
  et_llm_result r{};
  r.n_tokens = n; r.first_token = m->h_small[0]; r.logits = m->logits; r.hidden = m->X;
  r.kv_cache = m->kv_cache; r.kv_cache_rows = m->kv_cache ? m->cap : 0;
  *out = r;
  return ET_OK;
}

et_status et_llm_profile_enable(et_llm* m, int on) {
  if (!m) return ET_ERR_INVALID_ARG;
  m->prof_on = on != 0;
  if (on) memset(&m->prof, 0, sizeof(m->prof));
  return ET_OK;
}

et_status et_llm_profile_read(const et_llm* m, et_llm_profile* out) {
  if (!m || !out) return ET_ERR_INVALID_ARG;
  *out = m->prof;
  return ET_OK;
}

// ---- single steps -------------------------------------------------------------------------------

et_status et_rmsnorm(const float* x_dev, const float* g_dev, float eps, void* y_dev, int rows, int D, void* cuda_stream) {
  if (!x_dev || !g_dev || !y_dev) return ET_ERR_INVALID_ARG;
  if (rows < 1 || D < 4 || D % 4 != 0 || D > 4096) return ET_ERR_SHAPE;
  launch_rmsnorm(x_dev, g_dev, eps, (bf16*)y_dev, rows, D, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? ET_OK : ET_ERR_CUDA;
}

et_status et_rope(void* qkv_dev, int rows, int L, int heads, int kv_heads, int head_dim, float theta, void* cuda_stream) {
  if (!qkv_dev) return ET_ERR_INVALID_ARG;
  if (rows < 1 || L < 1 || heads < 1 || kv_heads < 1 || head_dim < 16 || head_dim % 16 != 0 || head_dim > 256) return ET_ERR_SHAPE;
  if (!(theta > 1.f)) return ET_ERR_INVALID_ARG;
  const int half = head_dim / 2;
  std::vector<double> t(half);
  for (int i = 0; i < half; ++i) t[i] = pow((double)theta, -2.0 * i / (double)head_dim) / (2.0 * M_PI);
  const int Lt = L < rows ? L : rows;                     // positions that occur
  double* dev = nullptr;
  if (cudaMalloc(&dev, half * sizeof(double) + (size_t)Lt * half * sizeof(float2)) != cudaSuccess) return ET_ERR_OOM;
  float2* table = reinterpret_cast<float2*>(dev + half);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  cudaError_t e = cudaMemcpyAsync(dev, t.data(), half * sizeof(double), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) {
    launch_rope_table(table, Lt, head_dim, dev, s);
    launch_rope((bf16*)qkv_dev, rows, L, heads, kv_heads, head_dim, table, s);
    e = cudaGetLastError();
  }
  const cudaError_t e2 = cudaStreamSynchronize(s);
  cudaFree(dev);
  return (e == cudaSuccess && e2 == cudaSuccess) ? ET_OK : ET_ERR_CUDA;
}

et_status et_swiglu(const void* gu_dev, void* h_dev, int rows, int M, void* cuda_stream) {
  if (!gu_dev || !h_dev) return ET_ERR_INVALID_ARG;
  if (rows < 1 || M < 8 || M % 8 != 0) return ET_ERR_SHAPE;
  launch_swiglu((const bf16*)gu_dev, (bf16*)h_dev, rows, M, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? ET_OK : ET_ERR_CUDA;
}

et_status et_attention_causal(const void* qkv_dev, void* out_dev, int n_seq, int L, int heads, int kv_heads, int head_dim,
                              int* status_dev, void* cuda_stream) {
  if (!qkv_dev || !out_dev) return ET_ERR_INVALID_ARG;
  if (n_seq < 1 || L < 1 || heads < 1 || kv_heads < 1 || heads % kv_heads != 0 || !attention_causal_supported(head_dim)) return ET_ERR_SHAPE;
  if ((long long)n_seq * L > (1ll << 30)) return ET_ERR_CAPACITY;
  CausalMaps map;
  if (!make_causal_attention_map(&map, (const bf16*)qkv_dev, (long long)n_seq * L, heads, kv_heads)) return ET_ERR_CUDA;
  return launch_attention_causal(map, (bf16*)out_dev, n_seq, L, heads, kv_heads, status_dev, (cudaStream_t)cuda_stream) == cudaSuccess
             ? ET_OK : ET_ERR_CUDA;
}

}  // extern "C"
