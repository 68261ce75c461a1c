// Self-tests of the failure-detection path: a bounded device-side wait that nothing satisfies must run out,
// leave a status word behind and return, and the host must report ET_ERR_TIMEOUT with the context still usable.
#include "common.cuh"
#include "tcgen05.cuh"

namespace et {
int stage1_debug_status();
int stage2_debug_status();

namespace {

// One warp.  The barrier expects one arrival; lane 1 provides it only when `arrive` is set.  Every lane waits
// with the same bounded wait the tensor-core kernels use (no TMA, tcgen05 or TMEM involved), then the outcome
// goes to the status word exactly as those kernels report theirs.
__global__ void bounded_wait_kernel(unsigned long long limit_ns, int arrive, int* status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  const uint32_t b = tc::smem_u32(&bar);
  if (threadIdx.x == 0) {
    tc::mbar_init(b, 1);
    abort_flag = 0;
  }
  __syncwarp();
  if (arrive && threadIdx.x == 1) tc::mbar_arrive(b);
  const bool ok = tc::mbar_wait(b, 0, &abort_flag, limit_ns);
  if (!__all_sync(0xffffffffu, ok) && threadIdx.x == 0) atomicExch(status, (int)DS_WAIT_EXPIRED);
}

}  // namespace
}  // namespace et

extern "C" et_status et_selftest_bounded_wait(unsigned long long limit_ns, int arrive, void* cuda_stream) {
  if (limit_ns == 0 || limit_ns > 1000000000ull) return ET_ERR_INVALID_ARG;      // at most one second
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int* status = nullptr;
  if (cudaMalloc(&status, sizeof(int)) != cudaSuccess) return ET_ERR_OOM;
  int host = -1;
  cudaError_t err = cudaMemsetAsync(status, 0, sizeof(int), s);
  if (err == cudaSuccess) {
    ET_COUNT_LAUNCH();
    et::bounded_wait_kernel<<<1, 32, 0, s>>>(limit_ns, arrive, status);
    err = cudaMemcpyAsync(&host, status, sizeof(int), cudaMemcpyDeviceToHost, s);
  }
  if (err == cudaSuccess) err = cudaStreamSynchronize(s);
  cudaFree(status);
  if (err != cudaSuccess) return ET_ERR_CUDA;
  return host == et::DS_WAIT_EXPIRED ? ET_ERR_TIMEOUT : (host == 0 ? ET_OK : ET_ERR_CUDA);
}

extern "C" int et_debug_build(void) {
#ifdef ET_DEBUG
  return 1;
#else
  return 0;
#endif
}

extern "C" int et_debug_status(void) { return et::stage1_debug_status() | et::stage2_debug_status(); }
