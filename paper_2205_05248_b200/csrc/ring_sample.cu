// Learner-side episode sampler (Algorithm 3: the learner draws B samples from the experience replay pool):
// one kernel picks one complete episode per batch element from the stated Philox stream and copies the chosen
// episodes' records out of the ring into dense [B][L][...] arrays, zero beyond each episode's length.
// A plain streaming kernel: every sampled record is read once and every output element is written once.
#include <cstring>
#include "common.cuh"

namespace marl {

constexpr uint32_t TAG_SAMPLE = 5;


// The draw of batch element b: up to MARL_SAMPLE_ATTEMPTS proposals from the Philox blocks (draw, b, attempt, tag),
// the first complete episode with at least one step wins; none: slot -1.
__device__ __forceinline__ void draw_episode(const SampleParams& p, int b, int32_t& slot, int32_t& len, long long& epid) {
  slot = -1;
  len = 0;
  epid = -1;
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
}

// One field of one batch element over the steps [l0, l1): the steps of the episode (l < len) are copied from their
// records, a warp per step and a lane per unit V, the rest is one contiguous zero fill.  fb = the field's bytes per
// step, a multiple of sizeof(V); the dense rows and the record fields are aligned to V by the caller's choice of V.
template <typename V>
__device__ __forceinline__ void gather_field(uint8_t* out_rows, const uint8_t* rec0, size_t rec_stride, uint32_t off,
                                             uint32_t fb, int l0, int l1, int len, int tid, int nthreads) {
  const int units = (int)(fb / sizeof(V));
  const int le = len < l1 ? (len > l0 ? len : l0) : l1;  // first step of this range that is beyond the episode
  const int warp = tid >> 5, lane = tid & 31, nwarps = nthreads >> 5;
  for (int l = l0 + warp; l < le; l += nwarps) {
    const V* src = reinterpret_cast<const V*>(rec0 + (size_t)l * rec_stride + off);
    V* dst = reinterpret_cast<V*>(out_rows + (size_t)l * fb);
    for (int u = lane; u < units; u += 32) dst[u] = src[u];
  }
  V zero;
  memset(&zero, 0, sizeof(V));
  V* z = reinterpret_cast<V*>(out_rows + (size_t)le * fb);
  const int nz = (l1 - le) * units;
  for (int i = tid; i < nz; i += nthreads) z[i] = zero;
}

__device__ __forceinline__ void gather_any(uint8_t* out_rows, const uint8_t* rec0, size_t rec_stride, uint32_t off,
                                           uint32_t fb, int l0, int l1, int len, int tid, int nthreads) {
  if (fb % 16 == 0) gather_field<uint4>(out_rows, rec0, rec_stride, off, fb, l0, l1, len, tid, nthreads);
  else if (fb % 4 == 0) gather_field<uint32_t>(out_rows, rec0, rec_stride, off, fb, l0, l1, len, tid, nthreads);
  else gather_field<uint8_t>(out_rows, rec0, rec_stride, off, fb, l0, l1, len, tid, nthreads);
}

// One block per (batch element, range of steps): each record field goes to its dense place.  Record fields start on
// 16-byte boundaries and the dense arrays are 16-byte aligned, so a field whose bytes per step are a multiple of 16
// moves in 16-byte units; other lengths fall back to 4- or 1-byte units.
constexpr int GATHER_THREADS = 256;
__global__ void __launch_bounds__(GATHER_THREADS) ring_gather_kernel(const __grid_constant__ SampleParams p, int steps_per_block) {
  const int b = blockIdx.x, tid = threadIdx.x;
  const int l0 = blockIdx.y * steps_per_block;
  const int l1 = min(p.L, l0 + steps_per_block);
  // every block of an element repeats the element's draw (a few Philox blocks) instead of waiting for a kernel
  // that makes it; the first block of the element reports it
  __shared__ int32_t sh_slot, sh_len;
  if (tid == 0) {
    int32_t s_, l_;
    long long id_;
    draw_episode(p, b, s_, l_, id_);
    sh_slot = s_;
    sh_len = l_;
    if (blockIdx.y == 0) {
      p.out.slot[b] = s_;
      p.out.len[b] = l_;
      p.out.epid[b] = id_;
    }
  }
  __syncthreads();
  const int32_t slot = sh_slot;
  const int len = slot >= 0 ? sh_len : 0;
  const uint8_t* rec0 = p.ring + (size_t)(slot >= 0 ? slot : 0) * p.slot_stride;
  const size_t rec = p.rl.rec_bytes, row0 = (size_t)b * p.L;
  const uint32_t nD = (uint32_t)(p.n * p.D), nA = (uint32_t)(p.n * p.A);
  gather_any(reinterpret_cast<uint8_t*>(p.out.obs + row0 * nD), rec0, rec, p.rl.off_obs, 4u * nD, l0, l1, len, tid, GATHER_THREADS);
  gather_any(reinterpret_cast<uint8_t*>(p.out.q + row0 * nA), rec0, rec, p.rl.off_q, 4u * nA, l0, l1, len, tid, GATHER_THREADS);
  gather_any(p.out.avail + row0 * nA, rec0, rec, p.rl.off_avail, nA, l0, l1, len, tid, GATHER_THREADS);
  gather_any(reinterpret_cast<uint8_t*>(p.out.action + row0 * p.n), rec0, rec, p.rl.off_action, 4u * (uint32_t)p.n, l0, l1, len,
             tid, GATHER_THREADS);
  for (int l = l0 + tid; l < l1; l += GATHER_THREADS) {
    const bool live = l < len;
    const uint8_t* r = rec0 + (size_t)l * rec;
    p.out.reward[row0 + l] = live ? *reinterpret_cast<const float*>(r + p.rl.off_reward) : 0.f;
    p.out.done[row0 + l] = live ? r[p.rl.off_done] : (uint8_t)0;
  }
}

// Returns the number of kernels launched or a negative cudaError.
int launch_ring_sample(const SampleParams& p, cudaStream_t stream) {
  // whole episodes per block when the batch alone fills the device, else ranges of at least eight steps
  int spb = (int)(((long long)p.L * p.B + 1183) / 1184);
  if (spb < 8) spb = 8;
  if (spb > p.L) spb = p.L;
  ring_gather_kernel<<<dim3((unsigned)p.B, (unsigned)((p.L + spb - 1) / spb)), GATHER_THREADS, 0, stream>>>(p, spb);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 1 : -(int)err;
}

}  // namespace marl
