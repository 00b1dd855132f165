// marl_rollout_noalloc: the rollout against the synthetic environment for callers that must not allocate
// device memory.  The paper has no counterpart to this entry point; it exists for integration reasons only.
//
// Who needs it: a host program that has handed all device memory to its own pool up front (a simulator
// farm, an inference server, a real-time control loop), or that runs where cudaMalloc is unwelcome because
// it synchronises the whole device and can fail late.  Such a caller creates the actor on buffers carved
// from its own pool and then wants to run rollouts without the library ever asking the driver for memory.
// marl_rollout needs a staging window for the generated environment steps; here that window is a fixed
// array inside the library image instead of caller- or library-allocated memory.
//
// Consequences of the fixed array, all part of the contract:
//   * its size is MARL_NOALLOC_SCRATCH_BYTES.  CUDA loads the parts of a library image on first use, and this
//     file holds nothing but the array, so the driver places the array on a GPU - and takes that much of its
//     memory, until the process exits - when this entry point is first called with that GPU current.  That
//     first call is the set-up call: make it at start-up, BEFORE the rest of the device memory goes to the
//     caller's pool; a call with T = 0 does the set-up and nothing else.  Every later call on that device
//     touches no allocator at all;
//   * a configuration whose staging for ONE environment step does not fit is rejected with MARL_ENOMEM;
//     larger T simply runs in more windows;
//   * all actors and all calls on a device share the array.  It keeps whatever the previous call left in
//     it; nothing in it has to start at zero, because every window is completely rewritten by the
//     generator kernels before the actor kernel reads it.  Two calls whose GPU work overlaps (different
//     streams, different host threads) race on it: serialise them;
//   * the set-up call looks up the array's device address (cudaGetSymbolAddress), which synchronises.  Make
//     it outside any stream capture.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/marl_actor.h"

// The scratch itself.  In host code this name is only a handle for the runtime's symbol lookup, never an
// address a kernel could use: the device address is fetched once per device below.
static __device__ __align__(256) uint8_t g_noalloc_scratch[MARL_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
uint8_t* g_scratch_addr[kMaxDevices] = {};  // device address of g_noalloc_scratch, per device ordinal

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

// Device address of the scratch on the current device, or nullptr with *err set.
uint8_t* scratch_on_current_device(cudaError_t* err) {
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= kMaxDevices) {
    *err = cudaErrorInvalidDevice;
    return nullptr;
  }
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (*err != cudaSuccess) return nullptr;
    g_scratch_addr[dev] = static_cast<uint8_t*>(p);
  }
  return g_scratch_addr[dev];
}

}  // namespace

extern "C" int marl_rollout_noalloc(marl_actor_t* a, const marl_synth_env_t* env, int32_t T, double eps_start,
                                    double eps_end, int32_t anneal_steps) {
  if (T == 0) {  // set-up only: the driver places the array on the current device now
    cudaError_t e0 = cudaSuccess;
    return scratch_on_current_device(&e0) ? MARL_OK : MARL_ECUDA;
  }
  if (!a || !env || T < 1) return MARL_EINVAL;
  marl_ring_view_t rv;
  int rc = marl_ring_view(a, &rv);
  if (rc) return rc;
  const size_t rows = (size_t)rv.n_envs * rv.n_agents;
  // staging of w steps: obs | avail | reward | done, each part starting on a 256-byte boundary
  auto window_bytes = [&](size_t w) {
    return align256(sizeof(float) * rows * rv.obs_dim * w) + align256(rows * rv.n_actions * w) +
           align256(sizeof(float) * rv.n_envs * w) + align256((size_t)rv.n_envs * w);
  };
  if (window_bytes(1) > (size_t)MARL_NOALLOC_SCRATCH_BYTES) return MARL_ENOMEM;
  size_t W = 1;
  while (W < (size_t)T && window_bytes(W + 1) <= (size_t)MARL_NOALLOC_SCRATCH_BYTES) ++W;

  cudaError_t err = cudaSuccess;
  uint8_t* base = scratch_on_current_device(&err);
  if (!base) return MARL_ECUDA;
  float* d_obs = reinterpret_cast<float*>(base);
  uint8_t* d_avail = base + align256(sizeof(float) * rows * rv.obs_dim * W);
  float* d_reward = reinterpret_cast<float*>(d_avail + align256(rows * rv.n_actions * W));
  uint8_t* d_done = reinterpret_cast<uint8_t*>(d_reward) + align256(sizeof(float) * rv.n_envs * W);

  int32_t left = T;
  while (left > 0) {
    const int32_t w = left < (int32_t)W ? left : (int32_t)W;
    marl_state_view_t st;
    rc = marl_actor_get_state(a, &st);
    if (rc) return rc;
    rc = marl_env_generate(a, env, (uint32_t)st.step, w, d_obs, d_avail, d_reward, d_done);
    if (rc) return rc;
    rc = marl_rollout_staged(a, d_obs, d_avail, d_reward, d_done, w, eps_start, eps_end, anneal_steps);
    if (rc) return rc;
    left -= w;
  }
  return MARL_OK;
}
