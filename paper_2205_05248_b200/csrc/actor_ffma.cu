// CUDA-core (FFMA) actor kernel: any shape, fp32 or bf16-rounded operands with fp32 accumulation.
//
// One thread block owns a tile of whole environments (up to 64 agent rows) and runs all T steps of the
// launch for that tile before taking the next tile: environments are independent (Sec. III-A, Fig. 3: one
// hidden state per environment and agent), so the hidden state, the last actions and the ring cursors of
// the tile stay in shared memory for the whole launch.  Per step the block runs the worker's decision
// (Algorithm 2: observations in, policy network, actions out) and the actor's recording of the step
// (Algorithm 1), in phases separated by block barriers:
//   A  stage obs (-> shared, and verbatim into the ring record), availability masks, open slot headers; a second set
//      of threads makes the epsilon draws, which need only the availability bytes
//   B  fc1 + one-hot column gathers + ReLU                       (register-tiled 4 rows x 4 columns)
//   C  GRU cell: both gate GEMMs, gate math, new hidden state    (same tiling, 64 accumulators)
//   D  fc2, masked greedy choice, ring/trace writes              (four threads per row, Q in registers)
//   F  reward/done, episode bookkeeping                          (one thread per environment); the hidden-state reset
//      of closed episodes shares the next step's phase A (a warp per eight rows)
// Weights are read through the read-only path from k-major copies, so a warp's load of four output
// columns for one k is one contiguous 256-byte segment.
#include <type_traits>

#include "common.cuh"
#include "launch_util.cuh"

namespace marl {

constexpr int FF_RMAX = 64;      // rows per tile
constexpr int FF_THREADS = 256;
constexpr int FF_PRE = 8;        // float4 registers per thread that hold the next step's observations

struct FfmaSmem {
  int Dp, Hp, wsmem;
  size_t off_xs, off_ys, off_hs, off_pick, off_mask, off_la, off_env, off_small, off_w, w_floats, total;
};

// Floats of the weight image kept in shared memory when it fits (hidden size 64): the k-major matrices
// W1T [I+4][H], WihT [H][3H] and WhhT [H][3H], in this order.
__host__ __device__ inline size_t ffma_weight_floats(int n, int D, int A, int H) {
  return (size_t)(D + n + A + 4) * H + 2 * (size_t)H * 3 * H;
}
// Floats of the small image that a shared network always keeps in shared memory: W2T [H][A rounded up to 4], then the
// biases b1 [H], b_ih [3H], b_hh [3H] and b2 [A rounded up to 4].
__host__ __device__ inline size_t ffma_small_floats(int A, int H) { return (size_t)((A + 3) & ~3) * (H + 1) + 7 * (size_t)H; }

__host__ __device__ inline FfmaSmem ffma_smem_layout(int n, int D, int A, int H) {
  FfmaSmem s;
  int Dp = (D + 3) & ~3;
  if ((Dp & 31) == 0) Dp += 4;
  s.Dp = Dp;
  s.Hp = H + 4;
  size_t o = 0;
  s.off_xs = o; o += sizeof(float) * FF_RMAX * s.Dp;
  s.off_ys = o; o += sizeof(float) * FF_RMAX * s.Hp;
  s.off_hs = o; o += sizeof(float) * 2 * FF_RMAX * s.Hp;
  s.off_pick = o; o += sizeof(int32_t) * FF_RMAX;
  s.off_mask = o; o += sizeof(uint32_t) * FF_RMAX;
  s.off_la = o; o += sizeof(int32_t) * FF_RMAX;
  s.off_env = o; o += 40 * FF_RMAX;  // per-environment scratch: see EnvSlot
  s.off_small = o; o += sizeof(float) * ffma_small_floats(A, H);
  s.off_w = o;
  s.w_floats = ffma_weight_floats(n, D, A, H);
  s.wsmem = (o + sizeof(float) * s.w_floats <= 227 * 1024) ? 1 : 0;  // resident weights if they fit
  if (s.wsmem) o += sizeof(float) * s.w_floats;
  s.total = o;
  return s;
}

struct EnvSlot {            // 40 bytes per environment of the tile
  long long epc;
  int32_t eid;              // the environment's index in the actor (not in the call)
  int32_t slot, pos;
  float reward;
  int32_t done;             // this step's done flag
  int32_t ok;               // cursor was in range at tile load
  int32_t reset;            // episode closed this step
};

static_assert(sizeof(EnvSlot) == 40, "the shared-memory plan reserves 40 bytes per environment");

__device__ __forceinline__ float sigmoid_accurate(float x) { return 1.0f / (1.0f + expf(-x)); }

// Weight loads: from the shared-memory copy (WS) or through the read-only global path.
template <bool WS>
__device__ __forceinline__ float4 wload4(const float* ptr) {
  if (WS) return *reinterpret_cast<const float4*>(ptr);
  return __ldg(reinterpret_cast<const float4*>(ptr));
}
// Two fp32 values in one 64-bit register and the packed multiply-add on them (fma.rn.f32x2: each half is the IEEE
// fused multiply-add of fmaf).  The FMA pipe does as many of them per clock as scalar ones would give - the peak is
// the same - but a packed instruction takes one issue slot for two, which leaves slots for the loads of the GEMM loops.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// Four weights as two packed pairs.
template <bool WS>
__device__ __forceinline__ ulonglong2 wload22(const float* ptr) {
  if (WS) return *reinterpret_cast<const ulonglong2*>(ptr);
  return __ldg(reinterpret_cast<const ulonglong2*>(ptr));
}
// Volatile, so that the request stays where it is written: a whole step before the value is used.
__device__ __forceinline__ float4 ldg_nc_v4(const float4* ptr) {
  float4 v;
  asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr));
  return v;
}
__device__ __forceinline__ float4 round4(float4 v, bool lowp) {
  if (lowp) { v.x = bf16_round(v.x); v.y = bf16_round(v.y); v.z = bf16_round(v.z); v.w = bf16_round(v.w); }
  return v;
}

// TYPED: one network per unit type (heterogeneous teams).  The tile's rows mix types, and a thread's register tile
// shares each weight value among its four rows, so the three products run once per type on that type's image with
// the operand of every row of another type replaced by zero: fma(0, w, acc) leaves acc as it is, so a row
// accumulates exactly the products of its own network.  Biases, the one-hot columns and fc2 (four threads per row)
// read the row's own image directly.  The images are read through the read-only path (they do not fit shared memory
// together).
// LOWP: operands rounded to bf16 (a template parameter: as a run-time flag it put a branch behind every operand
// load of the GEMM loops, and loads are not moved across branches).
template <bool WS, bool TYPED, bool LOWP>
__global__ void __launch_bounds__(FF_THREADS, 1) actor_ffma_kernel(const __grid_constant__ ActorParams p) {
  extern __shared__ __align__(16) uint8_t smem[];
  const FfmaSmem sl = ffma_smem_layout(p.n, p.D, p.A, p.H);
  float* xs = reinterpret_cast<float*>(smem + sl.off_xs);
  float* ys = reinterpret_cast<float*>(smem + sl.off_ys);
  float* hs = reinterpret_cast<float*>(smem + sl.off_hs);
  int32_t* picks = reinterpret_cast<int32_t*>(smem + sl.off_pick);  // the epsilon draw of every row: a random action or -1
  uint32_t* masks = reinterpret_cast<uint32_t*>(smem + sl.off_mask);
  int32_t* la = reinterpret_cast<int32_t*>(smem + sl.off_la);
  EnvSlot* envs = reinterpret_cast<EnvSlot*>(smem + sl.off_env);

  const int tid = threadIdx.x;
  const int n = p.n, D = p.D, A = p.A, H = p.H, Dp = sl.Dp, Hp = sl.Hp, H3 = 3 * p.H;
  constexpr bool lowp = LOWP;
  const int hbuf = FF_RMAX * Hp;  // floats per hidden buffer
  const int tx = tid & 15, ty = tid >> 4;
  const int ntypes = TYPED ? p.n_types : 1;
  const size_t tstride = TYPED ? p.type_stride : 0;
  auto row_type = [&](int r) -> int { return TYPED ? (int)((p.agent_type_bits >> (2 * (r % n))) & 3ull) : 0; };
  int rt[4];  // unit type of this thread's four rows
#pragma unroll
  for (int m = 0; m < 4; ++m) rt[m] = row_type(ty + 16 * m);

  unsigned long long c_steps = 0, c_explore = 0, c_noavail = 0, c_episodes = 0, c_trunc = 0;
  uint32_t st_bits = 0;

  for (int i = tid; i < (int)(sl.off_small / 4); i += FF_THREADS) reinterpret_cast<uint32_t*>(smem)[i] = 0;  // (the images follow)
  // weight pointers: the resident copy, or the k-major global arrays
  const float *W1T = p.W1T, *WihT = p.WihT, *WhhT = p.WhhT, *W2 = p.W2;
  const float *B1 = p.b1, *BIH = p.bih, *BHH = p.bhh, *B2 = p.b2;  // (a phase that starts with a load from global memory waits for it every step)
  constexpr bool SS = !TYPED;  // a shared network: W2 (transposed) and the biases are resident whatever the hidden size
  if (SS) {
    float* ssm = reinterpret_cast<float*>(smem + sl.off_small);
    const int AQ = (A + 3) & ~3;  // W2 transposed: the actions of one k side by side, padded with zeros
    for (size_t i = tid; i < (size_t)AQ * H; i += FF_THREADS) {
      const int k = (int)(i / AQ), a = (int)(i - (size_t)k * AQ);
      ssm[i] = a < A ? p.W2[(size_t)a * H + k] : 0.f;
    }
    float* bs = ssm + (size_t)AQ * H;
    for (int i = tid; i < H; i += FF_THREADS) bs[i] = p.b1[i];
    for (int i = tid; i < H3; i += FF_THREADS) { bs[H + i] = p.bih[i]; bs[H + H3 + i] = p.bhh[i]; }
    for (int i = tid; i < AQ; i += FF_THREADS) bs[H + 2 * H3 + i] = i < A ? p.b2[i] : 0.f;
    B1 = bs; BIH = bs + H; BHH = bs + H + H3; B2 = bs + H + 2 * H3;
    W2 = ssm;
  }
  if (WS) {
    float* wsm = reinterpret_cast<float*>(smem + sl.off_w);
    const size_t n1 = (size_t)(p.I + 4) * H, n2 = (size_t)H * H3;
    for (size_t i = tid; i < n1; i += FF_THREADS) wsm[i] = p.W1T[i];
    for (size_t i = tid; i < n2; i += FF_THREADS) { wsm[n1 + i] = p.WihT[i]; wsm[n1 + n2 + i] = p.WhhT[i]; }
    W1T = wsm; WihT = wsm + n1; WhhT = wsm + n1 + n2;
  }
  __syncthreads();

  // Observation tiles whose rows are whole float4s are requested one step ahead into registers, so that the
  // global-memory latency is hidden behind the previous step's arithmetic.
  const bool vec = (D % 4 == 0) && (reinterpret_cast<uintptr_t>(p.obs) % 16 == 0) && (FF_RMAX * D / 4 <= FF_THREADS * FF_PRE);
  float4 pre[FF_PRE];

  for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
    const int e0 = tile * p.ept;
    const int ne = min(p.ept, p.M - e0);  // environments in this tile (e0 counts the call's rows)
    // the environment behind row-of-the-call x: x itself, or the caller's list for a partial step
    auto env_of = [&](int x) { return p.env_ids ? __ldg(p.env_ids + x) : x; };
    const int R = ne * n;                 // live rows
    int cur = 0;
    auto prefetch_obs = [&](int s) {
      const float4* src4 = reinterpret_cast<const float4*>(p.obs + (size_t)s * p.obs_step_stride + (size_t)e0 * n * D);
      const int nv = R * D / 4;
#pragma unroll
      for (int u = 0; u < FF_PRE; ++u) {
        const int i4 = tid + u * FF_THREADS;
        if (i4 < nv) pre[u] = ldg_nc_v4(src4 + i4);
      }
    };
    if (vec) prefetch_obs(0);

    // ---- tile load: hidden state, last actions, ring cursors ----
    for (int idx = tid; idx < R * H; idx += FF_THREADS) {
      const int r = idx / H, j = idx - r * H;
      const int el = r / n;
      const float v = p.h[((size_t)env_of(e0 + el) * n + (r - el * n)) * H + j];
      hs[r * Hp + j] = v;
    }
    for (int r = tid; r < FF_RMAX; r += FF_THREADS) la[r] = (r < R) ? p.last_action[env_of(e0 + r / n) * n + r % n] : -1;
    if (tid < ne) {
      EnvSlot s;
      s.eid = env_of(e0 + tid);
      s.slot = p.slot[s.eid];
      s.pos = p.pos[s.eid];
      s.epc = p.ep_count[s.eid];
      s.reward = 0.f;
      s.done = 0;
      s.reset = 0;
      // (with late outcomes a full slot waits, at pos == L, for its last outcome before it is truncated)
      s.ok = (s.slot >= 0 && s.slot < p.E * p.S && s.pos >= 0 && s.pos < p.L + (p.lagged ? 1 : 0)) ? 1 : 0;
      if (!s.ok) st_bits |= MARL_STATUS_BAD_INDEX;
      if (p.lagged && s.ok && s.pos > 0) {
        // The outcome of the previous action arrives with this observation: it completes the record at pos - 1 and,
        // if the game ended or the slot is full, closes the episode before this step's decision.
        const float r = p.reward[e0 + tid];
        const int d = p.done[e0 + tid] ? 1 : 0;
        uint8_t* rec = p.ring + (size_t)s.slot * p.slot_stride + (size_t)(s.pos - 1) * p.rl.rec_bytes;
        *reinterpret_cast<float*>(rec + p.rl.off_reward) = r;
        rec[p.rl.off_done] = (uint8_t)d;
        if (d || s.pos == p.L) {
          p.slot_len[s.slot] = s.pos;
          p.slot_complete[s.slot] = 1;
          c_episodes += 1;
          if (!d) c_trunc += 1;
          s.epc += 1;
          s.slot = s.eid * p.S + (int)(s.epc % p.S);
          s.pos = 0;
          s.reset = 1;
        }
      }
      envs[tid] = s;
    }
    __syncthreads();
    if (p.lagged) {  // an episode closed above starts from a zero hidden state and no last action
      for (int idx = tid; idx < R * H; idx += FF_THREADS) {
        const int r = idx / H, j = idx - r * H;
        if (envs[r / n].reset) hs[r * Hp + j] = 0.f;
      }
      if (tid < R && envs[tid / n].reset) la[tid] = -1;
      __syncthreads();
    }

    // A closed episode starts from a zero hidden state and no last action.  Needs the flags of the bookkeeping phase
    // and touches neither what staging reads nor what it writes, so it shares a phase with the next step's staging.
    auto reset_closed = [&](int buf) {
      // each warp looks after eight rows: one lane per row reads the flag, the vote says whether anything is to do
      const int r8 = (tid >> 5) * 8 + (tid & 7);
      uint32_t todo = __ballot_sync(0xFFFFFFFFu, (tid & 31) < 8 && r8 < R && envs[r8 / n].reset) & 0xFFu;
      while (todo) {
        const int r = (tid >> 5) * 8 + __ffs(todo) - 1;
        todo &= todo - 1;
        for (int j = tid & 31; j < H; j += 32) hs[buf * hbuf + r * Hp + j] = 0.f;
      }
      if (tid < R && envs[tid / n].reset) la[tid] = -1;
    };

    for (int s = 0; s < p.T; ++s) {
      const uint32_t t = p.t0 + (uint32_t)s;
      const float eps = eps_at(p, t);
      const int nxt = cur ^ 1;

      // ---- phase A ----
      if (s > 0) reset_closed(cur);  // (the previous step's)
      {
        const float* src = p.obs + (size_t)s * p.obs_step_stride + (size_t)e0 * n * D;
        const int nD = n * D;
        const uint32_t inv_D = 0xFFFFFFFFu / (uint32_t)D + 1u, inv_nD = 0xFFFFFFFFu / (uint32_t)nD + 1u;
        // A row's availability bytes as aligned words (up to three bytes on either side are read and dropped), all
        // requested before the first is looked at: byte by byte, every load would wait for the one before it.
        auto load_avail_row = [&](const uint8_t* av, uint32_t (&w)[10]) -> uint32_t {
          const uintptr_t a0 = reinterpret_cast<uintptr_t>(av);
          const uint32_t* wp = reinterpret_cast<const uint32_t*>(a0 & ~(uintptr_t)3);
          const uint32_t sh = (uint32_t)(a0 & 3u), nw = (sh + (uint32_t)A + 3u) / 4u;
#pragma unroll
          for (int k = 0; k < 10; ++k) w[k] = (uint32_t)k < nw ? __ldg(wp + k) : 0u;
          return sh;
        };
        auto mask_of = [&](const uint32_t (&w)[10], uint32_t sh) -> uint32_t {
          unsigned long long bits = 0;
#pragma unroll
          for (int k = 0; k < 9; ++k) {
            const uint32_t v = w[k];
            const uint32_t nz = ((v | ((v & 0x7F7F7F7Fu) + 0x7F7F7F7Fu)) & 0x80808080u) >> 7;  // 0x01 per non-zero byte
            bits |= (unsigned long long)((nz * 0x01020408u) >> 24 & 0xFu) << (4 * k);
          }
          return (uint32_t)(bits >> sh) & (A >= 32 ? 0xFFFFFFFFu : ((1u << A) - 1u));
        };
        if (vec) {
          const int nv = R * D / 4;
#pragma unroll
          for (int u = 0; u < FF_PRE; ++u) {
            const int idx = (tid + u * FF_THREADS) * 4;
            if (idx < nv * 4) {
              asm volatile("" : "+f"(pre[u].x), "+f"(pre[u].y), "+f"(pre[u].z), "+f"(pre[u].w));  // first use is here
              const int r = (int)__umulhi((uint32_t)idx, inv_D), d = idx - r * D;  // (exact: idx < 2^16)
              const int el = (int)__umulhi((uint32_t)idx, inv_nD);
              const float4 v = pre[u];
              *reinterpret_cast<float4*>(xs + r * Dp + d) = round4(v, lowp);
              const EnvSlot& es = envs[el];
              if (es.ok)
                *reinterpret_cast<float4*>(p.ring + (size_t)es.slot * p.slot_stride + (size_t)es.pos * p.rl.rec_bytes +
                                           p.rl.off_obs + (size_t)(idx - el * nD) * 4) = v;
            }
          }
          if (s + 1 < p.T) prefetch_obs(s + 1);
        }
        for (int idx = tid; !vec && idx < R * D; idx += FF_THREADS) {
          const int r = idx / D, d = idx - r * D;
          const int el = idx / nD;
          const float v = src[idx];
          xs[r * Dp + d] = lowp ? bf16_round(v) : v;
          const EnvSlot& es = envs[el];
          if (es.ok) {
            float* dst = reinterpret_cast<float*>(p.ring + (size_t)es.slot * p.slot_stride +
                                                  (size_t)es.pos * p.rl.rec_bytes + p.rl.off_obs);
            dst[idx - el * nD] = v;
          }
        }
        if (s + 1 < p.T) {
          // the next step's availability rows, rewards and end flags are first touches of their lines: ask for them
          // now, so that the next phase A finds them in L2 instead of waiting for DRAM
          if (tid < R) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.avail + (size_t)(s + 1) * p.avail_step_stride + ((size_t)e0 * n + tid) * A));
          if (tid == FF_RMAX && !p.lagged) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.reward + (size_t)(s + 1) * p.env_step_stride + e0));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.done + (size_t)(s + 1) * p.env_step_stride + e0));
          }
        }
        if (tid < R) {
          const int el = tid / n, ai = tid - el * n;
          const uint8_t* av = p.avail + (size_t)s * p.avail_step_stride + ((size_t)e0 * n + tid) * A;
          const EnvSlot& es = envs[el];
          uint8_t* dst = p.ring + (size_t)es.slot * p.slot_stride + (size_t)es.pos * p.rl.rec_bytes +
                         p.rl.off_avail + ai * A;
          uint32_t w[10];
          const uint32_t sh = load_avail_row(av, w);
          masks[tid] = mask_of(w, sh);
          if (es.ok) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint32_t v = __funnelshift_r(w[j], w[j + 1], 8u * sh);  // bytes 4 j .. 4 j + 3 of the row
#pragma unroll
              for (int c = 0; c < 4; ++c)
                if (4 * j + c < A) dst[4 * j + c] = (uint8_t)(v >> (8 * c));
            }
          }
        }
        if (tid >= FF_RMAX && tid < FF_RMAX + R) {
          // The epsilon draw needs only the availability bytes (Algorithm 2 draws before it looks at Q): a second
          // set of threads reads them again and draws while the first set records them.
          const int r = tid - FF_RMAX, el = r / n, ai = r - el * n;
          const uint8_t* av = p.avail + (size_t)s * p.avail_step_stride + ((size_t)e0 * n + r) * A;
          uint32_t w[10];
          const uint32_t sh = load_avail_row(av, w);
          const uint32_t m = mask_of(w, sh);
          picks[r] = m ? draw_explore(m, eps, p.seed, t, (uint32_t)envs[el].eid, (uint32_t)ai) : -1;
        }
        if (tid < ne) {
          EnvSlot& es = envs[tid];
          es.reward = p.lagged ? 0.f : p.reward[(size_t)s * p.env_step_stride + e0 + tid];
          es.done = (!p.lagged && p.done[(size_t)s * p.env_step_stride + e0 + tid]) ? 1 : 0;
          if (es.ok && es.pos == 0) {  // an episode opens in this slot
            p.slot_epid[es.slot] = es.epc * (long long)p.E + es.eid;
            p.slot_len[es.slot] = 0;
            p.slot_complete[es.slot] = 0;
          }
        }
      }
      __syncthreads();

      // ---- phase B: fc1 ----
      for (int jb = 0; jb < H; jb += 64) {
        const int j0 = jb + tx * 4;
        f32x2 acc2[4][2];  // columns (0, 1) and (2, 3) of each row
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const ulonglong2 b = wload22<SS>(B1 + rt[m] * tstride + j0);
          acc2[m][0] = b.x; acc2[m][1] = b.y;
        }
        const int K4 = (D + 3) & ~3;
        for (int typ = 0; typ < ntypes; ++typ)
#pragma unroll 2
        for (int k = 0; k < K4; k += 4) {
          float4 xv[4];
#pragma unroll
          for (int m = 0; m < 4; ++m) {
            xv[m] = *reinterpret_cast<const float4*>(xs + (ty + 16 * m) * Dp + k);
            if (TYPED && rt[m] != typ) xv[m] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const ulonglong2 w = wload22<WS>(W1T + typ * tstride + (size_t)(k + kk) * H + j0);
#pragma unroll
            for (int m = 0; m < 4; ++m) {
              const float xk = kk == 0 ? xv[m].x : kk == 1 ? xv[m].y : kk == 2 ? xv[m].z : xv[m].w;
              const f32x2 xx = pack2(xk, xk);
              acc2[m][0] = fma2(xx, w.x, acc2[m][0]);
              acc2[m][1] = fma2(xx, w.y, acc2[m][1]);
            }
          }
        }
        float acc[4][4];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          unpack2(acc2[m][0], acc[m][0], acc[m][1]);
          unpack2(acc2[m][1], acc[m][2], acc[m][3]);
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int r = ty + 16 * m;
          const int ai = r % n;
          const float4 wid = wload4<WS>(W1T + rt[m] * tstride + (size_t)(D + ai) * H + j0);
          float4 o = make_float4(acc[m][0] + wid.x, acc[m][1] + wid.y, acc[m][2] + wid.z, acc[m][3] + wid.w);
          const int last = la[r];
          {  // (loaded whether or not there is a last action - row 0 then, dropped: a load under a condition is waited for)
            const float4 wl = wload4<WS>(W1T + rt[m] * tstride + (size_t)(D + n + max(last, 0)) * H + j0);
            if (last >= 0) { o.x += wl.x; o.y += wl.y; o.z += wl.z; o.w += wl.w; }
          }
          o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f);
          if (lowp) { o.x = bf16_round(o.x); o.y = bf16_round(o.y); o.z = bf16_round(o.z); o.w = bf16_round(o.w); }
          *reinterpret_cast<float4*>(ys + r * Hp + j0) = o;
        }
      }
      __syncthreads();

      // ---- phase C: GRU cell ----
      for (int jb = 0; jb < H; jb += 64) {
        const int j0 = jb + tx * 4;
        f32x2 ar2[4][2], az2[4][2], ai2[4][2], ah2[4][2];  // columns (0, 1) and (2, 3) of each row
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const float* bih = BIH + rt[m] * tstride;
          const float* bhh = BHH + rt[m] * tstride;
          const float4 bir = wload4<SS>(bih + j0);
          const float4 biz = wload4<SS>(bih + H + j0);
          const float4 bin = wload4<SS>(bih + 2 * H + j0);
          const float4 bhr = wload4<SS>(bhh + j0);
          const float4 bhz = wload4<SS>(bhh + H + j0);
          const float4 bhn = wload4<SS>(bhh + 2 * H + j0);
          ar2[m][0] = pack2(bir.x + bhr.x, bir.y + bhr.y); ar2[m][1] = pack2(bir.z + bhr.z, bir.w + bhr.w);
          az2[m][0] = pack2(biz.x + bhz.x, biz.y + bhz.y); az2[m][1] = pack2(biz.z + bhz.z, biz.w + bhz.w);
          ai2[m][0] = pack2(bin.x, bin.y); ai2[m][1] = pack2(bin.z, bin.w);
          ah2[m][0] = pack2(bhn.x, bhn.y); ah2[m][1] = pack2(bhn.z, bhn.w);
        }
        // (the pass is a compile-time constant of the loop body: chosen at run time, the products of the other pass'
        // candidate accumulators would be issued and predicated off)
        auto gemm_pass = [&](auto pass_c, int typ) {
          constexpr int pass = decltype(pass_c)::value;
          const float* act = pass == 0 ? ys : (hs + cur * hbuf);
          const float* WT = (pass == 0 ? WihT : WhhT) + typ * tstride;
          const bool rnd = lowp && pass == 1;  // the hidden state is stored in fp32; its operand copy is rounded here
          // Software pipeline: the weights of k + 1 and the activations of the next four k are requested before the
          // products of k are issued (indices past the end are clamped: loaded, never used), so that with two warps
          // per scheduler a shared-memory latency is not waited for at every k.
          auto load_act = [&](int k, float4 (&v)[4]) {
#pragma unroll
            for (int m = 0; m < 4; ++m) {
              v[m] = round4(*reinterpret_cast<const float4*>(act + (ty + 16 * m) * Hp + k), rnd);
              if (TYPED && rt[m] != typ) v[m] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
          };
          float4 v[4], vn[4];
          load_act(0, v);
          const float* wbase = WT + j0;
          ulonglong2 wr = wload22<WS>(wbase), wz = wload22<WS>(wbase + H), wn = wload22<WS>(wbase + 2 * H);
#pragma unroll 4  // (measured: 1 -> 21.5 k cycles per step for the gate GEMMs at H=64, 2 and 4 -> 18.0 k)
          for (int k = 0; k < H; k += 4) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const float* wrow = wbase + (size_t)min(k + kk + 1, H - 1) * H3;
              const ulonglong2 wr_n = wload22<WS>(wrow), wz_n = wload22<WS>(wrow + H), wn_n = wload22<WS>(wrow + 2 * H);
              if (kk == 1) load_act(min(k + 4, H - 4), vn);
#pragma unroll
              for (int m = 0; m < 4; ++m) {
                const float a = kk == 0 ? v[m].x : kk == 1 ? v[m].y : kk == 2 ? v[m].z : v[m].w;
                const f32x2 aa = pack2(a, a);
                ar2[m][0] = fma2(aa, wr.x, ar2[m][0]); ar2[m][1] = fma2(aa, wr.y, ar2[m][1]);
                az2[m][0] = fma2(aa, wz.x, az2[m][0]); az2[m][1] = fma2(aa, wz.y, az2[m][1]);
                if (pass == 0) {
                  ai2[m][0] = fma2(aa, wn.x, ai2[m][0]); ai2[m][1] = fma2(aa, wn.y, ai2[m][1]);
                } else {
                  ah2[m][0] = fma2(aa, wn.x, ah2[m][0]); ah2[m][1] = fma2(aa, wn.y, ah2[m][1]);
                }
              }
              wr = wr_n; wz = wz_n; wn = wn_n;
            }
#pragma unroll
            for (int m = 0; m < 4; ++m) v[m] = vn[m];
          }
        };
#pragma unroll 1
        for (int typ = 0; typ < ntypes; ++typ) {
          gemm_pass(std::integral_constant<int, 0>(), typ);
          gemm_pass(std::integral_constant<int, 1>(), typ);
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int r = ty + 16 * m;
          const float4 hp = *reinterpret_cast<const float4*>(hs + cur * hbuf + r * Hp + j0);
          const float hpv[4] = {hp.x, hp.y, hp.z, hp.w};
          float ar[4], az[4], ai_[4], ah[4];
          unpack2(ar2[m][0], ar[0], ar[1]); unpack2(ar2[m][1], ar[2], ar[3]);
          unpack2(az2[m][0], az[0], az[1]); unpack2(az2[m][1], az[2], az[3]);
          unpack2(ai2[m][0], ai_[0], ai_[1]); unpack2(ai2[m][1], ai_[2], ai_[3]);
          unpack2(ah2[m][0], ah[0], ah[1]); unpack2(ah2[m][1], ah[2], ah[3]);
          float o[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float rg = sigmoid_accurate(ar[c]);
            const float zg = sigmoid_accurate(az[c]);
            const float cand = tanhf(fmaf(rg, ah[c], ai_[c]));
            o[c] = fmaf(zg, hpv[c] - cand, cand);  // (1 - z) * cand + z * h
          }
          *reinterpret_cast<float4*>(hs + nxt * hbuf + r * Hp + j0) = make_float4(o[0], o[1], o[2], o[3]);
        }
      }
      __syncthreads();

      // ---- phase D: fc2, masked greedy choice and recording: four threads per row, each with the Q values of
      //      actions 4 part .. 4 part + 3 and 16 + 4 part .. 16 + 4 part + 3 in registers; the row's maximum and the
      //      set of near-maximal actions go round the four lanes by shuffles ----
      {
        const int r = tid >> 2, part = tid & 3;
        const bool live = r < R;
        const size_t toff = row_type(r) * tstride;  // this row's own network
        float q[2][4];
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int a = 16 * g + 4 * part + c;
            q[g][c] = a < A ? (SS ? B2[a] : __ldg(B2 + toff + a)) : 0.f;
          }
        const float* hv = hs + nxt * hbuf + r * Hp;
        if (SS) {
          const int AQ = (A + 3) & ~3;
          const float* wcol = W2 + 4 * part;  // W2T [k][AQ]
          // Unconditional loads, so that the four k of a pass are requested together (a load under a per-thread
          // condition is waited for where it stands).  A thread whose group lies beyond A reads the neighbouring
          // entries of the image - inside it: the biases follow the last row - and its sums are never used.
          if (A <= 16) {
#pragma unroll 2
            for (int k = 0; k < H; k += 4) {
              const float4 v = round4(*reinterpret_cast<const float4*>(hv + k), lowp);
              float4 w[4];
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) w[kk] = *reinterpret_cast<const float4*>(wcol + (size_t)(k + kk) * AQ);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                const float vk = kk == 0 ? v.x : kk == 1 ? v.y : kk == 2 ? v.z : v.w;
                q[0][0] = fmaf(vk, w[kk].x, q[0][0]); q[0][1] = fmaf(vk, w[kk].y, q[0][1]);
                q[0][2] = fmaf(vk, w[kk].z, q[0][2]); q[0][3] = fmaf(vk, w[kk].w, q[0][3]);
              }
            }
          } else {
#pragma unroll 2
            for (int k = 0; k < H; k += 4) {
              const float4 v = round4(*reinterpret_cast<const float4*>(hv + k), lowp);
              float4 w[4][2];
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                w[kk][0] = *reinterpret_cast<const float4*>(wcol + (size_t)(k + kk) * AQ);
                w[kk][1] = *reinterpret_cast<const float4*>(wcol + (size_t)(k + kk) * AQ + 16);
              }
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                const float vk = kk == 0 ? v.x : kk == 1 ? v.y : kk == 2 ? v.z : v.w;
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                  q[g][0] = fmaf(vk, w[kk][g].x, q[g][0]); q[g][1] = fmaf(vk, w[kk][g].y, q[g][1]);
                  q[g][2] = fmaf(vk, w[kk][g].z, q[g][2]); q[g][3] = fmaf(vk, w[kk][g].w, q[g][3]);
                }
              }
            }
          }
        } else {
          // weights from global memory, W2 [A][H]: the loads are unconditional (the action index clamped to A - 1; the
          // sums of actions beyond A are never used), so that those of one k-group are requested together
          const bool two = A > 16;
          for (int k = 0; k < H; k += 4) {
            const float4 v = round4(*reinterpret_cast<const float4*>(hv + k), lowp);
            float4 w[2][4];
#pragma unroll
            for (int g = 0; g < 2; ++g)
#pragma unroll
              for (int c = 0; c < 4; ++c)
                if (g == 0 || two) w[g][c] = wload4<false>(W2 + toff + (size_t)min(16 * g + 4 * part + c, A - 1) * H + k);
#pragma unroll
            for (int g = 0; g < 2; ++g)
#pragma unroll
              for (int c = 0; c < 4; ++c)
                if (g == 0 || two) {
                  q[g][c] = fmaf(v.x, w[g][c].x, q[g][c]);
                  q[g][c] = fmaf(v.y, w[g][c].y, q[g][c]);
                  q[g][c] = fmaf(v.z, w[g][c].z, q[g][c]);
                  q[g][c] = fmaf(v.w, w[g][c].w, q[g][c]);
                }
          }
        }
        // greedy rule: m = max over available, thr = m - 1e-4f, lowest available a with Q >= thr (a NaN never
        // compares greater or equal and fmaxf ignores it, like the "greater than" scan of select_action)
        const uint32_t mask = live ? masks[r] : 0u;
        float m = -INFINITY;
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int a = 16 * g + 4 * part + c;
            if (a < A && ((mask >> a) & 1u)) m = fmaxf(m, q[g][c]);
          }
        m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
        const float thr = __fsub_rn(m, 1e-4f);
        uint32_t ge = 0;
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int a = 16 * g + 4 * part + c;
            if (a < A && q[g][c] >= thr) ge |= 1u << a;
          }
        ge |= __shfl_xor_sync(0xFFFFFFFFu, ge, 1);
        ge |= __shfl_xor_sync(0xFFFFFFFFu, ge, 2);
        ge &= mask;
        if (live) {
          const int el = r / n, ai = r - el * n;
          const int pick = picks[r];
          const int greedy = ge ? __ffs(ge) - 1 : __ffs(mask) - 1;
          const int act = mask == 0 ? 0 : (pick >= 0 ? pick : greedy);
          const EnvSlot& es = envs[el];
          const int e = es.eid;
          uint8_t* rec = p.ring + (size_t)es.slot * p.slot_stride + (size_t)es.pos * p.rl.rec_bytes;
          const int tk = p.trace_first + s;
          const size_t grow = ((size_t)tk * p.E + e) * n + ai;
          const bool traced = tk < p.trace_cap;
          float* qd = reinterpret_cast<float*>(rec + p.rl.off_q) + ai * A;
#pragma unroll
          for (int g = 0; g < 2; ++g)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const int a = 16 * g + 4 * part + c;
              if (a < A) {
                if (es.ok) qd[a] = q[g][c];
                if (traced && p.trace_q) p.trace_q[grow * A + a] = q[g][c];
              }
            }
          if (part == 0) {
            c_steps += 1;
            c_explore += (mask != 0 && pick >= 0) ? 1u : 0u;
            if (mask == 0) { c_noavail += 1; st_bits |= MARL_STATUS_NO_AVAIL; }
            la[r] = act;
            if (es.ok) reinterpret_cast<int32_t*>(rec + p.rl.off_action)[ai] = act;
            if (traced && p.trace_actions) p.trace_actions[grow] = act;
            if (p.actions_out && s == p.T - 1) p.actions_out[(size_t)(e0 + el) * n + ai] = act;
          }
        }
      }
      __syncthreads();  // the rows above read the cursors that the environment threads advance below
      // ---- phase F (first half): reward/done and the episode cursor, one thread per environment ----
      if (tid < ne) {
        EnvSlot& es = envs[tid];
        if (es.ok) {
          uint8_t* rec = p.ring + (size_t)es.slot * p.slot_stride + (size_t)es.pos * p.rl.rec_bytes;
          *reinterpret_cast<float*>(rec + p.rl.off_reward) = es.reward;
          rec[p.rl.off_done] = (uint8_t)es.done;
          const bool full = !p.lagged && es.pos + 1 == p.L;  // (late outcomes: the next call truncates)
          if (es.done || full) {
            p.slot_len[es.slot] = es.pos + 1;
            p.slot_complete[es.slot] = 1;
            c_episodes += 1;
            if (!es.done) c_trunc += 1;
            es.epc += 1;
            es.slot = es.eid * p.S + (int)(es.epc % p.S);
            es.pos = 0;
            es.reset = 1;
          } else {
            es.pos += 1;
            es.reset = 0;
          }
        }
      }
      cur = nxt;
      __syncthreads();
    }
    reset_closed(cur);  // (the last step's)
    __syncthreads();

    // ---- tile store ----
    for (int idx = tid; idx < R * H; idx += FF_THREADS) {
      const int r = idx / H, j = idx - r * H;
      const int el = r / n;
      p.h[((size_t)envs[el].eid * n + (r - el * n)) * H + j] = hs[cur * hbuf + r * Hp + j];
    }
    if (tid < R) p.last_action[envs[tid / n].eid * n + tid % n] = la[tid];
    if (tid < ne) {
      const EnvSlot& es = envs[tid];
      if (es.ok) {
        p.slot[es.eid] = es.slot;
        p.pos[es.eid] = es.pos;
        p.ep_count[es.eid] = es.epc;
        if (es.pos > 0) p.slot_len[es.slot] = es.pos;
      }
    }
    __syncthreads();
  }

  if (c_steps) atomicAdd(p.counters + CNT_AGENT_STEPS, c_steps);
  if (c_explore) atomicAdd(p.counters + CNT_EXPLORED, c_explore);
  if (c_noavail) atomicAdd(p.counters + CNT_NO_AVAIL, c_noavail);
  if (c_episodes) atomicAdd(p.counters + CNT_EPISODES, c_episodes);
  if (c_trunc) atomicAdd(p.counters + CNT_TRUNCATED, c_trunc);
  if (st_bits) atomicOr(p.status, st_bits);
}

// Environments per tile and number of tiles for this kernel.
void ffma_tiling(int E, int n, int sms, int* ept, int* num_tiles) {
  int per = FF_RMAX / n;
  if (per < 1) per = 1;
  int spread = (E + sms - 1) / sms;  // small batches: one tile per SM before tiles grow
  if (spread < 1) spread = 1;
  if (per > spread) per = spread;
  *ept = per;
  *num_tiles = (E + per - 1) / per;
}

size_t ffma_smem_bytes(int n, int D, int A, int H) { return ffma_smem_layout(n, D, A, H).total; }

// Returns the number of kernels launched or a negative cudaError.
int launch_actor_ffma(const ActorParams& p, int sms, cudaStream_t stream) {
  const FfmaSmem sl = ffma_smem_layout(p.n, p.D, p.A, p.H);
  const bool typed = p.n_types > 1;
  const bool ws = sl.wsmem && !typed;
  const bool lowp = p.prec == MARL_PRECISION_BF16;
  auto kernel = typed ? (lowp ? actor_ffma_kernel<false, true, true> : actor_ffma_kernel<false, true, false>)
                : ws  ? (lowp ? actor_ffma_kernel<true, false, true> : actor_ffma_kernel<true, false, false>)
                      : (lowp ? actor_ffma_kernel<false, false, true> : actor_ffma_kernel<false, false, false>);
  const size_t smem_bytes = ws ? sl.total : sl.off_w;
  static uint32_t configured[6][SMEM_OPTIN_DEVICES];
  {
    const cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), (uint32_t)smem_bytes, configured[(typed ? 2 : (ws ? 1 : 0)) + (lowp ? 3 : 0)]);
    if (e != cudaSuccess) return -(int)e;
  }
  int grid = p.num_tiles < sms ? p.num_tiles : sms;
  if (grid < 1) grid = 1;
  kernel<<<grid, FF_THREADS, smem_bytes, stream>>>(p);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 1 : -(int)err;
}

}  // namespace marl
