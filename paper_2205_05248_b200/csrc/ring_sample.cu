// Learner-side episode sampler (Algorithm 3: the learner draws B samples from the experience replay pool):
// a draw kernel picks one complete episode per batch element from the stated Philox stream, a gather kernel copies
// the chosen episodes' records out of the ring into dense [B][L][...] arrays, zero beyond each episode's length.
// Both are plain streaming kernels: the gather reads every record once and writes every output element once.
#include "common.cuh"

namespace marl {

constexpr uint32_t TAG_SAMPLE = 5;


__global__ void ring_draw_kernel(const __grid_constant__ SampleParams p) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= p.B) return;
  int32_t slot = -1, len = 0;
  long long epid = -1;
  for (uint32_t a = 0; a < MARL_SAMPLE_ATTEMPTS; ++a) {
    uint32_t w[4];
    philox4x32_10(p.draw_index, (uint32_t)b, a, TAG_SAMPLE, (uint32_t)p.seed, (uint32_t)(p.seed >> 32), w);
    const int32_t s = (int32_t)__umulhi(w[0], (uint32_t)p.C);
    const int32_t l = p.slot_len[s];
    if (p.slot_complete[s] == 1 && l >= 1) {
      slot = s;
      len = l < p.L ? l : p.L;
      epid = p.slot_epid[s];
      break;
    }
  }
  p.out.slot[b] = slot;
  p.out.len[b] = len;
  p.out.epid[b] = epid;
}

// One block per (step, batch element): the record's fields go to their dense places, word by word (fields start on
// 16-byte boundaries but their lengths are arbitrary multiples of 4 bytes, the availability bytes of 1).
__global__ void __launch_bounds__(128) ring_gather_kernel(const __grid_constant__ SampleParams p) {
  const int l = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int32_t slot = p.out.slot[b], len = p.out.len[b];
  const bool live = slot >= 0 && l < len;
  const uint8_t* rec = p.ring + (size_t)(live ? slot : 0) * p.slot_stride + (size_t)l * p.rl.rec_bytes;
  const size_t row = (size_t)b * p.L + l;
  const int nD = p.n * p.D, nA = p.n * p.A;
  // fp32 fields: 16 bytes per thread where the row length allows it (record fields start on 16-byte boundaries)
  auto copy_f32 = [&](const float* src, float* dst, int count) {
    if ((count & 3) == 0) {
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int i = tid; i < count / 4; i += blockDim.x)
        reinterpret_cast<float4*>(dst)[i] = live ? reinterpret_cast<const float4*>(src)[i] : z;
    } else {
      for (int i = tid; i < count; i += blockDim.x) dst[i] = live ? src[i] : 0.f;
    }
  };
  copy_f32(reinterpret_cast<const float*>(rec + p.rl.off_obs), p.out.obs + row * nD, nD);
  copy_f32(reinterpret_cast<const float*>(rec + p.rl.off_q), p.out.q + row * nA, nA);
  const uint8_t* r_av = rec + p.rl.off_avail;
  uint8_t* o_av = p.out.avail + row * nA;
  for (int i = tid; i < nA; i += blockDim.x) o_av[i] = live ? r_av[i] : (uint8_t)0;
  const int32_t* r_act = reinterpret_cast<const int32_t*>(rec + p.rl.off_action);
  int32_t* o_act = p.out.action + row * p.n;
  for (int i = tid; i < p.n; i += blockDim.x) o_act[i] = live ? r_act[i] : 0;
  if (tid == 0) {
    p.out.reward[row] = live ? *reinterpret_cast<const float*>(rec + p.rl.off_reward) : 0.f;
    p.out.done[row] = live ? rec[p.rl.off_done] : (uint8_t)0;
  }
}

// Returns the number of kernels launched or a negative cudaError.
int launch_ring_sample(const SampleParams& p, cudaStream_t stream) {
  ring_draw_kernel<<<(p.B + 127) / 128, 128, 0, stream>>>(p);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return -(int)err;
  ring_gather_kernel<<<dim3((unsigned)p.L, (unsigned)p.B), 128, 0, stream>>>(p);
  err = cudaGetLastError();
  return err == cudaSuccess ? 2 : -(int)err;
}

}  // namespace marl
