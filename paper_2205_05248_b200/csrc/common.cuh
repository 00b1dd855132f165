// Shared device-side definitions of the actor library: kernel parameter block, Philox4x32-10, the
// exploration draw and the greedy rule.  Written from the published definition of Philox (Salmon et al.,
// SC'11) and from the conventions stated in include/marl_actor.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/marl_actor.h"

namespace marl {

enum : uint32_t { TAG_EPS = 0, TAG_DONE_REWARD = 1, TAG_AVAIL = 2, TAG_OBS = 3 };
enum { CNT_AGENT_STEPS = 0, CNT_EPISODES, CNT_EXPLORED, CNT_NO_AVAIL, CNT_TRUNCATED, CNT_N = 8 };

// Byte layout of one ring record (one environment step); every field starts on a 16-byte boundary.
struct RecordLayout {
  uint32_t off_obs, off_avail, off_action, off_q, off_reward, off_done, rec_bytes, pad;
};

// Everything a step kernel needs.  Passed by value (__grid_constant__).
struct ActorParams {
  int32_t E, n, D, A, H, I, L, S;
  int32_t prec;             // MARL_PRECISION_*
  int32_t T;                // steps in this launch
  uint32_t t0;              // global index of the first step
  int32_t ept;              // environments per tile
  int32_t num_tiles;
  int32_t eps_const_mode;   // 1: eps_const for every step; 0: linear schedule
  float eps_const;
  int32_t anneal_steps;
  double eps_start, eps_end;
  uint64_t seed;
  // FFMA-kernel weights, fp32 values (already rounded to bf16-representable values in bf16 precision),
  // k-major: W1T [I+4][H], WihT [H][3H], WhhT [H][3H]; W2 in [A][H]; biases.
  const float *W1T, *b1, *WihT, *bih, *WhhT, *bhh, *W2, *b2;
  // tensor-core kernel weights: one packed image (see actor_tc.cu)
  const void* wpack;
  // inputs; step k of the launch reads base + k * stride (elements)
  const float* obs;
  const uint8_t* avail;
  const float* reward;
  const uint8_t* done;
  long long obs_step_stride, avail_step_stride, env_step_stride;
  // state
  float* h;
  int32_t* last_action;
  int32_t* slot;
  int32_t* pos;
  long long* ep_count;
  // ring
  uint8_t* ring;
  RecordLayout rl;
  long long slot_stride;    // L * rec_bytes
  long long* slot_epid;
  int32_t* slot_len;
  uint8_t* slot_complete;
  // outputs
  int32_t* actions_out;     // [E][n] of the last step of the launch, may be null
  int32_t* trace_actions;   // may be null
  float* trace_q;           // may be null
  int32_t trace_first;      // trace index of the launch's first step
  int32_t trace_cap;
  unsigned long long* counters;
  uint32_t* status;
  // partial step (FFMA kernel only): the call's rows are the M listed environments; null: all E in order
  const int32_t* env_ids;
  int32_t M;
  // T == 1 over a list: reward/done are the outcome of each environment's PREVIOUS action (committed at pos - 1)
  int32_t lagged;
  // One network per unit type (FFMA kernel only): n_types > 1, the FFMA image of type k starts type_stride floats
  // after the one of type k - 1, and agent i's type is bits 2i, 2i+1 of agent_type_bits.
  int32_t n_types;
  uint32_t type_stride;
  uint64_t agent_type_bits;
};

// Everything the episode sampler needs (ring_sample.cu).  Passed by value.
struct SampleParams {
  int32_t B, C, L, n, D, A, E;
  uint64_t seed;
  uint32_t draw_index;
  const uint8_t* ring;
  RecordLayout rl;
  long long slot_stride;
  const long long* slot_epid;
  const int32_t* slot_len;
  const uint8_t* slot_complete;
  marl_sample_batch_t out;
};

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0;
    c1 = lo1;
    c2 = n2;
    c3 = lo0;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

__device__ __forceinline__ void philox_block(uint64_t seed, uint32_t step, uint32_t env, uint32_t agent,
                                             uint32_t block, uint32_t tag, uint32_t out[4]) {
  philox4x32_10(step, env, agent | (block << 16), tag, (uint32_t)seed, (uint32_t)(seed >> 32), out);
}

__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

// eps of global step t: s + (e - s) * min(t, N) / N in double with one rounding per operation.
__device__ __forceinline__ float eps_at(const ActorParams& p, uint32_t t) {
  if (p.eps_const_mode) return p.eps_const;
  if (p.anneal_steps <= 0) return (float)p.eps_start;
  const double N = (double)p.anneal_steps;
  const double tt = (double)t < N ? (double)t : N;
  const double frac = __ddiv_rn(tt, N);
  const double delta = __dmul_rn(__dsub_rn(p.eps_end, p.eps_start), frac);
  return (float)__dadd_rn(p.eps_start, delta);
}

// The epsilon draw of one row: Philox block (t, e, i, tag 0); word 0 -> u in [0,1), explore iff u < eps; word 1
// -> index among the K available actions (bit a of mask set = action a available), floor(w1 * K / 2^32).
// Returns -1 if the row does not explore, otherwise the random action.  K == 0 never explores.
__device__ __forceinline__ int draw_explore(uint32_t mask, float eps, uint64_t seed, uint32_t t, uint32_t e,
                                            uint32_t i) {
  uint32_t w[4];
  philox_block(seed, t, e, i, 0, TAG_EPS, w);
  const float u = (float)(w[0] >> 8) * (1.0f / 16777216.0f);
  const int K = __popc(mask);
  if (K == 0 || !(u < eps)) return -1;
  const uint32_t j = __umulhi(w[1], (uint32_t)K);
  return __fns(mask, 0, (int)j + 1);  // position of the (j+1)-th set bit, ascending
}

// Masked greedy choice with the lowest-index rule, then the epsilon draw (see marl_actor.h).
// q: A values; mask: bit a set = available.  Returns the action; sets flags bit0 = explored,
// bit1 = no action available.
template <typename QGet>
__device__ __forceinline__ int select_action(QGet q, int A, uint32_t mask, float eps, uint64_t seed, uint32_t t,
                                             uint32_t e, uint32_t i, uint32_t& flags) {
  flags = 0;
  if (mask == 0) {
    flags = 2;
    return 0;
  }
  const int pick = draw_explore(mask, eps, seed, t, e, i);
  if (pick >= 0) {
    flags = 1;
    return pick;
  }
  float m = -INFINITY;
  for (int a = 0; a < A; ++a)
    if (((mask >> a) & 1u) && q(a) > m) m = q(a);
  const float thr = __fsub_rn(m, 1e-4f);
  for (int a = 0; a < A; ++a)
    if (((mask >> a) & 1u) && q(a) >= thr) return a;
  return __ffs(mask) - 1;
}

}  // namespace marl
