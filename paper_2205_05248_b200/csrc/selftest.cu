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

// Dependency-free FFMA loop: 16 independent accumulators per thread, used to measure the fp32 FMA peak of the
// device under load (the bound of the fp32 actor path).
__global__ void __launch_bounds__(256) ffma_peak_kernel(float* out, int iters, float a, float b) {
  float acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = (float)(threadIdx.x + i);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], a, b);
  }
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) sum += acc[i];
  if (sum == 123.456f) out[0] = sum;  // never true in practice; keeps the loop alive
}

}  // namespace marl

extern "C" int marl_measure_ffma_tflops(void* stream, double* tflops_out) {
  if (!tflops_out) return MARL_EINVAL;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MARL_ECUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  float* d = nullptr;
  if (cudaMalloc(&d, sizeof(float)) != cudaSuccess) return MARL_ENOMEM;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  const int blocks = sms * 8, iters = 1 << 15;
  cudaError_t e = cudaSuccess;
  double best = 0.0;
  for (int rep = 0; rep < 4 && e == cudaSuccess; ++rep) {  // first repetition warms up
    cudaEventRecord(e0, st);
    marl::ffma_peak_kernel<<<blocks, 256, 0, st>>>(d, iters, 0.999f, 0.001f);
    cudaEventRecord(e1, st);
    e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    const double tf = 2.0 * 16.0 * iters * 256.0 * blocks / (ms * 1e-3) / 1e12;
    if (rep > 0 && tf > best) best = tf;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(d);
  *tflops_out = best;
  return e == cudaSuccess ? MARL_OK : MARL_ECUDA;
}

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
