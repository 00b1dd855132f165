// Self-test of the bounded device-side wait used by the tensor-core kernel: a one-block kernel waits on an
// mbarrier that nothing ever completes, gives up after its poll limit, and reports MARL_STATUS_TIMEOUT through
// a status word - the same path a lost hand-off inside the actor kernel takes.  The context stays usable.
#include "common.cuh"
#include "tcgen05.cuh"

namespace marl {

__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint32_t limit) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);  // expects one arrival; none will come
    abort_flag = 0;
    tc::mbar_init_fence();
  }
  __syncthreads();
  const bool ok = tc::mbar_wait(&bar, 0, &abort_flag, limit);
  __syncthreads();
  if (threadIdx.x == 0) status[0] = (ok ? 0u : MARL_STATUS_TIMEOUT) | (abort_flag ? 0x100u : 0u);
}

}  // namespace marl

extern "C" int marl_selftest_bounded_wait(void* stream, uint32_t poll_limit, uint32_t* status_out) {
  if (!status_out || poll_limit == 0 || poll_limit > 1000000u) return MARL_EINVAL;
  uint32_t* d = nullptr;
  if (cudaMalloc(&d, sizeof(uint32_t)) != cudaSuccess) return MARL_ENOMEM;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(d, 0xFF, sizeof(uint32_t), st);
  if (e == cudaSuccess) {
    marl::bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(d, poll_limit);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(status_out, d, sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(d);
  return e == cudaSuccess ? MARL_OK : MARL_ECUDA;
}
