// Synthetic-environment generator: the seeded stand-in for the simulator of Algorithm 1 (Env.step and
// Env.done).  Streams and their Philox counters are specified in include/marl_actor.h (marl_synth_env_t).
// Every value is derived from integers, so the output is reproducible bit for bit.
#include "common.cuh"

namespace marl {

struct EnvGenParams {
  marl_synth_env_t env;
  int32_t E, n, D, A;
  uint32_t t0;
  int32_t n_steps;
  float* obs;
  uint8_t* avail;
  float* reward;
  uint8_t* done;
};

__device__ __forceinline__ float irwin_hall12(const uint32_t a[4], const uint32_t b[4]) {
  int32_t s = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) s += (int32_t)(a[k] & 0xFFFFu) + (int32_t)(a[k] >> 16);
#pragma unroll
  for (int k = 0; k < 2; ++k) s += (int32_t)(b[k] & 0xFFFFu) + (int32_t)(b[k] >> 16);
  return (float)(s - 393210) * (1.0f / 65536.0f);
}

// One thread per group of four observation entries of one (step, env, agent) row.
__global__ void __launch_bounds__(256) env_obs_kernel(const __grid_constant__ EnvGenParams p) {
  const int groups = (p.D + 3) >> 2;
  const long long total = (long long)p.n_steps * p.E * p.n * groups;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int g = (int)(idx % groups);
    const long long row = idx / groups;  // (step, env, agent)
    const int i = (int)(row % p.n);
    const long long se = row / p.n;
    const uint32_t e = (uint32_t)(se % p.E);
    const uint32_t t = p.t0 + (uint32_t)(se / p.E);
    float v[4];
    if (p.env.obs_law == 0) {
      uint32_t w[4];
      philox_block(p.env.seed, t, e, (uint32_t)i, (uint32_t)g, TAG_OBS, w);
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = (float)((int32_t)(w[k] >> 8) - 8388608) * (1.0f / 8388608.0f);
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t d = (uint32_t)(4 * g + k);
        uint32_t w[4], w2[4];
        philox_block(p.env.seed, t, e, (uint32_t)i, 2 * d, TAG_OBS, w);
        philox_block(p.env.seed, t, e, (uint32_t)i, 2 * d + 1, TAG_OBS, w2);
        v[k] = fminf(3.0f, fmaxf(-3.0f, irwin_hall12(w, w2)));
      }
    }
    const int type = (i < p.env.n_type0) ? 0 : 1;
    const int other_lo = p.env.type_block_start + (type == 0 ? p.env.type_block_len : 0);
    float* dst = p.obs + row * p.D;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int d = 4 * g + k;
      if (d < p.D) {
        float x = v[k];
        if (p.env.type_block_len > 0 && d >= other_lo && d < other_lo + p.env.type_block_len) x = 0.0f;
        dst[d] = x;
      }
    }
  }
}

// One thread per group of four availability flags of one row.
__global__ void __launch_bounds__(256) env_avail_kernel(const __grid_constant__ EnvGenParams p) {
  const int groups = (p.A + 3) >> 2;
  const long long total = (long long)p.n_steps * p.E * p.n * groups;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int g = (int)(idx % groups);
    const long long row = idx / groups;
    const int i = (int)(row % p.n);
    const long long se = row / p.n;
    const uint32_t e = (uint32_t)(se % p.E);
    const uint32_t t = p.t0 + (uint32_t)(se / p.E);
    uint32_t w[4];
    philox_block(p.env.seed, t, e, (uint32_t)i, (uint32_t)g, TAG_AVAIL, w);
    uint8_t* dst = p.avail + row * p.A;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int a = 4 * g + k;
      if (a < p.A) {
        const uint32_t thr = (a < p.env.avail_split) ? p.env.avail_thresh_first : p.env.avail_thresh_rest;
        dst[a] = (a == 0) ? 1 : (((w[k] >> 8) < thr) ? 1 : 0);
      }
    }
  }
}

// One thread per (step, env): done flag and reward.
__global__ void __launch_bounds__(256) env_scalar_kernel(const __grid_constant__ EnvGenParams p) {
  const long long total = (long long)p.n_steps * p.E;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const uint32_t e = (uint32_t)(idx % p.E);
    const uint32_t t = p.t0 + (uint32_t)(idx / p.E);
    uint32_t w[4], w2[4];
    philox_block(p.env.seed, t, e, 0, 0, TAG_DONE_REWARD, w);
    p.done[idx] = ((w[0] >> 8) < p.env.done_thresh24) ? 1 : 0;
    philox_block(p.env.seed, t, e, 0, 1, TAG_DONE_REWARD, w);
    philox_block(p.env.seed, t, e, 0, 2, TAG_DONE_REWARD, w2);
    p.reward[idx] = irwin_hall12(w, w2);
  }
}

static int grid_for(long long items, int sms) {
  long long g = (items + 255) / 256;
  const long long cap = (long long)sms * 16;
  if (g > cap) g = cap;
  if (g < 1) g = 1;
  return (int)g;
}

// Returns the number of kernels launched (3) or a negative cudaError.
int launch_env_generate(const marl_synth_env_t& env, int E, int n, int D, int A, uint32_t t0, int n_steps,
                        float* obs, uint8_t* avail, float* reward, uint8_t* done, int sms,
                        cudaStream_t stream) {
  EnvGenParams p;
  p.env = env;
  p.E = E; p.n = n; p.D = D; p.A = A;
  p.t0 = t0;
  p.n_steps = n_steps;
  p.obs = obs; p.avail = avail; p.reward = reward; p.done = done;
  const long long rows = (long long)n_steps * E * n;
  env_obs_kernel<<<grid_for(rows * ((D + 3) / 4), sms), 256, 0, stream>>>(p);
  env_avail_kernel<<<grid_for(rows * ((A + 3) / 4), sms), 256, 0, stream>>>(p);
  env_scalar_kernel<<<grid_for((long long)n_steps * E, sms), 256, 0, stream>>>(p);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 3 : -(int)err;
}

}  // namespace marl
