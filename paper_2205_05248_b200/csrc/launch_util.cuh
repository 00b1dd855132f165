// Host-side launch helper shared by the actor kernels.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace marl {

constexpr int SMEM_OPTIN_DEVICES = 64;

// A kernel's opt-in dynamic shared-memory size is a per-device setting.  `table` (one per kernel variant, zero
// initialised) remembers the largest size set on each device, so that the attribute call is made once per device
// and size instead of once per launch; devices beyond the table are set on every launch.
inline cudaError_t ensure_dynamic_smem(const void* kernel, uint32_t bytes, uint32_t (&table)[SMEM_OPTIN_DEVICES]) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < SMEM_OPTIN_DEVICES;
  if (tracked && table[dev] >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && tracked) table[dev] = bytes;
  return e;
}

}  // namespace marl
