// et_frame_similarity_static: adjacent-frame similarity for callers that must not allocate.
//
// Some users of this library run where device allocation is off the table: a serving loop whose
// memory was carved up at start-up by another allocator that has already claimed the whole card, a
// latency-critical thread that may not take the implicit device synchronisation of cudaMalloc or
// cudaFree, or a plug-in host that forbids allocation calls after initialisation.  The regular
// entry point leaves the (n-1)*L per-position cosines to a caller-provided scratch buffer; this
// variant keeps that scratch in a fixed array inside the library image instead, so the caller
// passes only the input and the output.
//
// The array lives in every CUDA context that loads the library, from load until the process exits
// (256 KiB per GPU).  All calls share it and it keeps the contents of the last call.  Nothing in it
// has to start at zero: the first kernel overwrites every cosine that the second kernel reads.
// Two calls that overlap on the GPU (different streams, or different host threads) race on it.
#include <mutex>

#include "common.cuh"
#include "rowops.cuh"

namespace {

constexpr size_t STATIC_COS_FLOATS = 64 * 1024;   // 256 KiB: (n-1)*L must not exceed this
static __device__ __align__(256) float g_static_cos[STATIC_COS_FLOATS];

constexpr int MAX_DEVICES = 64;
float* g_scratch_addr[MAX_DEVICES] = {};
bool g_scratch_ready[MAX_DEVICES] = {};
std::mutex g_scratch_mutex;

// In host code `g_static_cos` is only a handle for the runtime, not a device address.  The real
// address differs per device and is looked up once per device, with that device current.
et_status scratch_of_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return ET_ERR_CUDA;
  if (dev < 0 || dev >= MAX_DEVICES) return ET_ERR_CAPACITY;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    const cudaError_t err = cudaGetSymbolAddress(&p, g_static_cos);
    if (err != cudaSuccess || p == nullptr) return ET_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<float*>(p);
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_addr[dev];
  return ET_OK;
}

}  // namespace

extern "C" et_status et_frame_similarity_static(const float* x_dev, int n, int L, int D, float* sim_dev,
                                                void* cuda_stream) {
  if (!x_dev || !sim_dev) return ET_ERR_INVALID_ARG;
  if (n < 1 || L < 1 || D < 4 || D % 4 != 0 || D > et::ROW_MAX_D) return ET_ERR_SHAPE;
  if ((size_t)(n - 1) * (size_t)L > STATIC_COS_FLOATS) return ET_ERR_CAPACITY;   // beyond the built-in scratch
  float* scratch = nullptr;
  const et_status st = scratch_of_current_device(&scratch);
  if (st != ET_OK) return st;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  et::launch_token_cosines(x_dev, scratch, n, L, D, nullptr, s);
  et::launch_reduce_cosines(scratch, sim_dev, n, L, nullptr, s);
  return cudaGetLastError() == cudaSuccess ? ET_OK : ET_ERR_CUDA;
}
