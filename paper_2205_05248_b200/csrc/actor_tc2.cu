// Two-tile tensor-core actor kernel for sm_100a: bf16 operands, hidden size 64, two tiles of environments resident
// per thread block.
//
// The pipelined kernel (actor_tcp.cu) runs one 128-row tile per SM, and a step of that tile is a chain
//   epilogue 1 -> y-side GEMM -> epilogue 2 -> fc2 -> epilogue 3
// with nothing to overlap the GEMM round trips and the epilogues' latencies.  Environments are independent
// (Sec. III-A: nothing is shared between environments but the network), so this kernel keeps TWO tiles resident and
// lets their chains run side by side, about half a step apart: while one tile's GEMM is in flight or its threads wait
// for tensor memory, the other tile's epilogue has the SM.  The worker's decision step (Algorithm 2) and the actor's
// recording (Algorithm 1) are the ones of the pipelined kernel, with the same packed weight image and the same
// arithmetic; what is shared and what is doubled:
//
//   shared by both tiles   the 74 KB weight image, the one-hot operand tile, the staging ring of four-environment
//                          chunks with its load, converter and store warps, the tail warp, the MMA-issuing warp
//   per tile               256 columns of
//                          tensor memory (reset | update | candidate-input | candidate-hidden; the fc1 accumulator of
//                          the next step aliases candidate-input, the four Q parts alias candidate-hidden), the fc1
//                          operand, ONE operand buffer that holds y and then h' (a step's y-side GEMM has finished
//                          with y before the gate math writes h'), masks and draws, its own barriers.  The
//                          [action | Q | reward, done] part of a record is written straight to the ring (no
//                          shared-memory copy): the memory goes to the staging ring, whose depth - six chunks for
//                          two tiles - decides whether the inputs keep up
//
// The shared warps serve the two tiles in a fixed alternating order (tile A's step k, tile B's step k, A's k+1, ...),
// every dependency of which points backwards in that order, so the order cannot deadlock; it also keeps tile B
// half a step behind tile A.  The MMA warp issues, per step of a tile: the h-side candidate product (after the
// previous step's Q has been read), the y-side products, fc2, and - off the chain - fc1 and the h-side reset/update
// products of the next step.
//
// The epilogue threads (one agent row x 32 hidden columns, as in the pipelined kernel) serve both tiles as well, phase
// by phase: E1(A) E3(B) E2(A) E1(B) E3(A) E2(B).  (Giving each tile a warpgroup of its own - one thread per row, 64
// columns - was measured first: with one warp per scheduler a tile's gate math cannot keep the special-function unit
// busy, and a step took 9.4 k cycles against 6.0 k in the pipelined kernel.)
//
// Warp roles (512 threads): warps 0-7 epilogue (both tiles in turn), warps 8-11 converters,
// warp 12 issues every tcgen05.mma, warp 13 input loads and ring cursors ahead, warp 14 tails and headers,
// warp 15 observation stores.  All hand-offs are mbarriers with bounded waits; an expired wait sets
// MARL_STATUS_TIMEOUT and lets the block run to its end with every index in range.
//
// Taken: dense launches of at least 8 steps with more tiles than SMs, shapes whose per-environment blocks can be
// bulk-copied (observation width a multiple of 8, availability bytes per environment a multiple of 16), at most 16
// actions, at most seven chunks per tile-step.  Everything else stays on the pipelined kernel.
//
// Measured (workload 5, 65536 environments, 64-step rollouts): 8.4 ms against 6.15 ms for the pipelined kernel, so this
// kernel is offered as MARL_KERNEL_TENSOR_DUAL and never chosen automatically.  Timelines (clock stamps at the
// hand-offs) show why: the GEMM round trips are covered as planned, but with the epilogue threads busy all the time the
// converter warps slow down to about 5 k cycles per tile-step (the conversion alone from 1 k to 2.3 k cycles) and
// the MMA warp waits for the fc1 operand.  The pipelined kernel issues 9.7 k warp instructions and reads about 370 KB
// of shared memory per tile-step (175 KB of it tensor-core operand reads: small-N products re-read their 128-row
// operand for every product); two chains side by side ask the four schedulers and the shared-memory port for more
// than they give, whatever the staging depth (four or six chunks measured the same) or the code size (150 KB or 78 KB
// measured the same).
#include <cstring>

#include "actor_tc_layout.cuh"
#include "common.cuh"
#include "launch_util.cuh"
#include "tcgen05.cuh"

namespace marl {

constexpr int T2_THREADS = 512;
constexpr int T2_CONV = 128;       // converter threads
constexpr int T2_G = 4;            // environments per staging chunk
constexpr int T2_MAX_STAGES = 7;   // (the record addresses of T2_DEPTH = 8 steps are kept: a ragged tile's loads run up to 7 steps ahead)
constexpr int T2_DEPTH = 8;        // steps of record addresses and close flags kept per tile: the loads run at most
                                   // T2_MAX_STAGES chunks (of a ragged tile: steps) ahead
constexpr int T2_NQ = 16;
// Register split (setmaxnreg): launched with 128 registers per thread; 256 * 176 + 128 * 80 + 128 * 80 = 65536.
constexpr int T2_REGS_EPI = 176, T2_REGS_CONV = 80, T2_REGS_SVC = 80;
// tensor memory: 256 columns per resident tile
constexpr uint32_t T2_R = 0, T2_IN = 128, T2_HN = 192, T2_TILE_COLS = 256, T2_COLS = 512;
constexpr uint32_t T2_LBO_W1 = TC_H * 16, T2_LBO_G = 3 * TC_H * 16;
constexpr uint64_t T2_K_A = (2 * TC_LBO_A) >> 4, T2_K_X = (2 * TC_LBO_X) >> 4, T2_K_W1 = (2 * T2_LBO_W1) >> 4,
                   T2_K_G = (2 * T2_LBO_G) >> 4;

struct T2Layout {
  int32_t Dk, nchunk, ept, ohK, ohc, NS, pad0, pad1;
  uint32_t prefix_bytes, tail_bytes, chunk_bytes, obs_bytes, av_bytes;
  uint32_t off_W1, off_Wih, off_Whh, off_Bg, off_Bhn, off_W2, off_tab_la, wbytes;
  uint32_t off_oh, off_rowenv, off_tile0, tile_stride, off_bar, off_stage, total;
  uint32_t t_x, t_yh, t_sel, t_la, t_close, t_closeany, t_dstp, t_tdst;  // inside a tile's block
};

struct T2TileBars {
  uint64_t xready, fc1d, hsd, yready, grud, hready, fc2d, stepd, tiled, flags, selready[4];
};
struct T2Bars {
  uint64_t full[T2_MAX_STAGES], cfree[T2_MAX_STAGES], sfree[T2_MAX_STAGES];  // chunk loaded / converted / stored
  T2TileBars t[2];
  uint64_t wload;
  uint32_t tmem_base, abort;
};

static T2Layout t2_layout(int n, int D, int A, int rec_bytes) {
  const TcLayout W = tc_layout(n, D, A, rec_bytes);
  T2Layout L;
  memset(&L, 0, sizeof(L));
  L.Dk = W.Dk; L.nchunk = W.nchunk; L.ept = W.ept; L.ohK = W.ohK; L.ohc = W.ohc;
  L.off_W1 = W.off_W1; L.off_Wih = W.off_Wih; L.off_Whh = W.off_Whh; L.off_Bg = W.off_Bg; L.off_Bhn = W.off_Bhn;
  L.off_W2 = W.off_W2; L.off_tab_la = W.off_tab_la; L.wbytes = W.wbytes;
  L.obs_bytes = (uint32_t)(n * D) * 4u;
  L.av_bytes = (uint32_t)(n * A);
  L.prefix_bytes = L.obs_bytes + L.av_bytes;
  L.tail_bytes = (uint32_t)rec_bytes - (up16(L.obs_bytes) + up16(L.av_bytes));
  L.chunk_bytes = T2_G * L.prefix_bytes;
  uint32_t o = L.wbytes;
  L.off_oh = o; o += (uint32_t)L.ohc * TC_LBO_A;
  L.off_rowenv = o; o += TC_ROWS * 4;
  uint32_t t = 0;
  L.t_x = t; t += up16((uint32_t)L.nchunk * TC_LBO_X);
  L.t_yh = t; t += 8 * TC_LBO_A;
  L.t_sel = t; t += 4u * TC_ROWS * 4;
  L.t_la = t; t += TC_ROWS * 4;
  L.t_close = t; t += 2 * 32 * 4;
  L.t_closeany = t; t += T2_DEPTH * 4;
  L.t_dstp = t; t += T2_DEPTH * 32 * 8;
  L.t_tdst = t; t += 32 * 8;
  L.tile_stride = (t + 127u) & ~127u;
  L.off_tile0 = (o + 127u) & ~127u;
  o = L.off_tile0 + 2u * L.tile_stride;
  L.off_bar = o; o += (uint32_t)((sizeof(T2Bars) + 15) & ~15u);
  L.off_stage = o;
  const uint32_t room = o + 32 < TC_SMEM_MAX ? TC_SMEM_MAX - o - 32 : 0;  // (+32: the mask words read a few bytes past a row)
  int ns = (int)(room / L.chunk_bytes);
  if (ns > T2_MAX_STAGES) ns = T2_MAX_STAGES;
  // the ring holds at least one tile-step of chunks, so a slot's previous chunk always belongs to an earlier
  // tile-step (the converters finish a tile-step together before any of them starts the next)
  const int nck_max = (L.ept + T2_G - 1) / T2_G;
  if (ns < nck_max) ns = 0;
  L.NS = ns;
  L.total = o + (uint32_t)ns * L.chunk_bytes + 32;
  return L;
}

bool tc2_supported(int n, int D, int A, int H, int prec) {
  if (prec != MARL_PRECISION_BF16 || H != TC_H) return false;
  if (D < 1 || D > 256 || D % 8 != 0 || n < 4 || n > 32 || A < 1 || A > T2_NQ) return false;
  if ((n * A) % 16 != 0) return false;
  const T2Layout L = t2_layout(n, D, A, rec_bytes_of(n, D, A));
  return L.ept >= T2_G && L.NS >= 3 && L.total <= TC_SMEM_MAX;
}

__device__ __forceinline__ void t2_warp_arrive(uint64_t* bar, int lane) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
}

__global__ void __launch_bounds__(T2_THREADS, 1)
    actor_tc2_kernel(const __grid_constant__ ActorParams p, const __grid_constant__ T2Layout L) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using namespace tc;
  T2Bars* B = reinterpret_cast<T2Bars*>(smem + L.off_bar);
  uint8_t* oh = smem + L.off_oh;
  uint8_t* stage = smem + L.off_stage;
  int32_t* rowenv_s = reinterpret_cast<int32_t*>(smem + L.off_rowenv);
  const float* tab_la = reinterpret_cast<const float*>(smem + L.off_tab_la);
  volatile uint32_t* abortf = &B->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = p.n, D = p.D, A = p.A, T = p.T;
  const uint32_t rec_bytes = p.rl.rec_bytes;
  const int NS = L.NS;
  // This block's tiles are blockIdx.x, blockIdx.x + gridDim.x, ...; resident tile g (0 = A, 1 = B) takes those with
  // index g, g + 2, ... of that list and runs NK[g] tile-steps in all.
  const int my_tiles = blockIdx.x < p.num_tiles ? (p.num_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  const int NK0 = ((my_tiles + 1) / 2) * T, NK1 = (my_tiles / 2) * T;
  auto tile_of = [&](int g, int j) { return (int)blockIdx.x + (2 * j + g) * (int)gridDim.x; };  // j-th tile of resident tile g
  auto tmem_ptr = [&](int g) { return smem + L.off_tile0 + (uint32_t)g * L.tile_stride; };

  if (tid == 0) {
    for (int i = 0; i < T2_MAX_STAGES; ++i) {
      mbar_init(&B->full[i], 1);
      mbar_init(&B->cfree[i], 1);
      mbar_init(&B->sfree[i], 1);
    }
    for (int g = 0; g < 2; ++g) {
      T2TileBars& tb = B->t[g];
      mbar_init(&tb.xready, T2_CONV / 32);
      mbar_init(&tb.fc1d, 1);
      mbar_init(&tb.hsd, 1);
      mbar_init(&tb.yready, 8);
      mbar_init(&tb.grud, 1);
      mbar_init(&tb.hready, 8);
      mbar_init(&tb.fc2d, 1);
      mbar_init(&tb.stepd, 8);
      mbar_init(&tb.tiled, 8);
      mbar_init(&tb.flags, 1);
      for (int i = 0; i < 4; ++i) mbar_init(&tb.selready[i], T2_CONV / 32);
    }
    mbar_init(&B->wload, 1);
    B->abort = 0;
    mbar_init_fence();
  }
  if (warp == 12) tmem_alloc(&B->tmem_base, T2_COLS);
  // operands, tails and hand-off arrays start as zeros (padding bytes of every stored record stay zero)
  for (uint32_t i = L.off_oh / 16 + tid; i < L.off_bar / 16; i += T2_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (tid < TC_ROWS) {
    // one-hot operand tile: three ones (bias columns) and the agent's own column; the same for every tile
    const int ai = tid % n;
    auto oh_col = [&](int k) { return oh + (uint32_t)(k >> 3) * TC_LBO_A + (uint32_t)tid * 16u + (uint32_t)(k & 7) * 2u; };
    *reinterpret_cast<uint16_t*>(oh_col(0)) = 0x3F80;  // bf16 1.0
    *reinterpret_cast<uint16_t*>(oh_col(1)) = 0x3F80;
    *reinterpret_cast<uint16_t*>(oh_col(2)) = 0x3F80;
    *reinterpret_cast<uint16_t*>(oh_col(3 + ai)) = 0x3F80;
    rowenv_s[tid] = tid / n;
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = B->tmem_base;
  if (tid == 12 * 32) {
    mbar_arrive_expect_tx(&B->wload, L.wbytes);
    bulk_load(smem, p.wpack, L.wbytes, &B->wload);
  }
  mbar_wait(&B->wload, 0, abortf);

  if (warp >= 12) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(T2_REGS_SVC));
    if (warp == 12) {
      // =========================== MMA warp: lane 0 issues every tcgen05.mma of both tiles ===========================
      const uint32_t sb = smem_u32(smem);
      constexpr uint32_t id16 = idesc_bf16_f32(128, T2_NQ), id64 = idesc_bf16_f32(128, 64), id128 = idesc_bf16_f32(128, 128),
                         id192 = idesc_bf16_f32(128, 192);
      auto tbase = [&](int g) { return sb + L.off_tile0 + (uint32_t)g * L.tile_stride; };
      auto tcol = [&](int g) { return tmem + (uint32_t)g * T2_TILE_COLS; };
      // fc1 of one step into the candidate-input columns: observations x W1, then the one-hot tile x (bias pieces,
      // agent-id columns)
      auto issue_fc1 = [&](int g) {
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_x = smem_desc(tbase(g) + L.t_x, TC_LBO_X, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
          const uint64_t d_W1 = smem_desc(sb + L.off_W1, T2_LBO_W1, 128);
          const uint64_t d_W1oh = smem_desc(sb + L.off_W1 + (uint32_t)L.nchunk * T2_LBO_W1, T2_LBO_W1, 128);
          const int ks_obs = L.Dk / 16, ks_oh = L.ohK / 16;
          for (int ks = 0; ks < ks_obs; ++ks) mma_bf16(tcol(g) + T2_IN, d_x + ks * T2_K_X, d_W1 + ks * T2_K_W1, id64, ks > 0);
          for (int ks = 0; ks < ks_oh; ++ks) mma_bf16(tcol(g) + T2_IN, d_oh + ks * T2_K_A, d_W1oh + ks * T2_K_W1, id64, 1);
          mma_commit(&B->t[g].fc1d);
        }
        __syncwarp();
      };
      // h-side products of the reset and update gates, seeded with their biases
      auto issue_rz = [&](int g) {
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_h = smem_desc(tbase(g) + L.t_yh, TC_LBO_A, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
          mma_bf16(tcol(g) + T2_R, d_oh, smem_desc(sb + L.off_Bg, T2_LBO_G, 128), id128, 0);
          const uint64_t d_Whh = smem_desc(sb + L.off_Whh, T2_LBO_G, 128);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma_bf16(tcol(g) + T2_R, d_h + ks * T2_K_A, d_Whh + ks * T2_K_G, id128, 1);
        }
        __syncwarp();
      };
      // h-side product of the candidate plus its bias; then the operand buffer is free for y
      auto issue_hn = [&](int g) {
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_h = smem_desc(tbase(g) + L.t_yh, TC_LBO_A, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
          const uint64_t d_Whh_n = smem_desc(sb + L.off_Whh + 2 * TC_H * 16, T2_LBO_G, 128);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma_bf16(tcol(g) + T2_HN, d_h + ks * T2_K_A, d_Whh_n + ks * T2_K_G, id64, ks > 0);
          mma_bf16(tcol(g) + T2_HN, d_oh, smem_desc(sb + L.off_Bhn, T2_LBO_W1, 128), id64, 1);  // (bias last, as in the pipelined kernel)
          mma_commit(&B->t[g].hsd);
        }
        __syncwarp();
      };
      // One half-iteration serves tile g's step k (y-side, fc2) and, between the two, starts the other tile's coming
      // step: fc1 (off the chain), the h-side reset/update products early when no episode of that tile ends, then -
      // once that tile's previous step is through - the rest of the h-side.  Only the other tile's state is touched,
      // and the two states change places every half-iteration, so the code exists once.
      int ns_x = 0, ns_y = 0;          // step within its tile of the next step to begin: x = tile g, y = the other tile
      uint32_t tl_x = 0, tl_y = 0;     // tile prologues seen
      auto do_begin = [&](int o, int kn) {  // begin step kn of tile o
        mbar_wait(&B->t[o].xready, (uint32_t)kn & 1u, abortf);
        issue_fc1(o);  // (the candidate-input columns are free: fc2 of step kn - 1 was issued after its gate math)
        const bool first = ns_y == 0;
        bool rz = false;
        if (!first && reinterpret_cast<const int32_t*>(tmem_ptr(o) + L.t_closeany)[(kn - 1) & (T2_DEPTH - 1)] == 0) {
          issue_rz(o);  // the new hidden state is in place and no row will be cleared
          rz = true;
        }
        if (first) {
          mbar_wait(&B->t[o].tiled, tl_y & 1, abortf);
          ++tl_y;
        } else {
          mbar_wait(&B->t[o].stepd, (uint32_t)(kn - 1) & 1u, abortf);  // h' in place with closed episodes cleared, Q read
        }
        if (!rz) issue_rz(o);
        issue_hn(o);
        if (++ns_y == T) ns_y = 0;
      };
      auto do_yside = [&](int g, int k) {
        mbar_wait(&B->t[g].yready, (uint32_t)k & 1u, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_y = smem_desc(tbase(g) + L.t_yh, TC_LBO_A, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
          // the candidate-input columns (the fc1 accumulator until epilogue 1 has read it) start from their bias
          mma_bf16(tcol(g) + T2_IN, d_oh, smem_desc(sb + L.off_Bg + 2 * TC_H * 16, T2_LBO_G, 128), id64, 0);
          const uint64_t d_Wih = smem_desc(sb + L.off_Wih, T2_LBO_G, 128);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma_bf16(tcol(g) + T2_R, d_y + ks * T2_K_A, d_Wih + ks * T2_K_G, id192, 1);
          mma_commit(&B->t[g].grud);
        }
        __syncwarp();
      };
      auto do_fc2 = [&](int g, int k) {
        mbar_wait(&B->t[g].hready, (uint32_t)k & 1u, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_h = smem_desc(tbase(g) + L.t_yh, TC_LBO_A, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
          const uint64_t d_W2 = smem_desc(sb + L.off_W2, T2_NQ * 16, 128);
          mma_bf16(tcol(g) + T2_HN, d_oh, smem_desc(sb + L.off_W2 + 8u * T2_NQ * 16, T2_NQ * 16, 128), id16, 0);  // bias into part 0
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)  // four K-steps on four 16-column parts
            mma_bf16(tcol(g) + T2_HN + (uint32_t)ks * 16u, d_h + ks * T2_K_A, d_W2 + ks * ((2 * T2_NQ * 16) >> 4), id16, ks == 0 ? 1 : 0);
          mma_commit(&B->t[g].fc2d);
        }
        __syncwarp();
      };
      // half-iteration i: tile g = i & 1 at its step k = i >> 1 (i = -1: only the start of tile A's first step)
#pragma unroll 1
      for (int i = -1; i < 2 * NK0; ++i) {
        const int g = i & 1, k = i >> 1, o = g ^ 1;
        const int NKg = g ? NK1 : NK0, NKo = g ? NK0 : NK1;
        const int kn = g ? k + 1 : k;  // the other tile's step that begins now: A leads B by half a step
        if (k >= 0 && k < NKg) do_yside(g, k);
        if (kn < NKo) do_begin(o, kn);
        if (k >= 0 && k < NKg) do_fc2(g, k);
        const int tn = ns_x; ns_x = ns_y; ns_y = tn;
        const uint32_t tt = tl_x; tl_x = tl_y; tl_y = tt;
      }
    } else if (warp == 13) {
      // =========================== load warp: staging ring in, record addresses ahead ===========================
      // Lane el follows the ring cursor of environment el of each resident tile: the cursor sequence depends only on
      // the done flags, so it runs ahead of the network.  State of tile g of the half-iteration in *_x, of the other
      // tile in *_y; they change places every half-iteration.
      int32_t slot_x = 0, pos_x = 0, ok_x = 0, s_x = 0, j_x = 0, slot_y = 0, pos_y = 0, ok_y = 0, s_y = 0, j_y = 0;
      long long epc_x = 0, epc_y = 0;
      uint32_t dn_x = 0, dn_y = 0;
      uint32_t q = 0, qslot = 0, qpar = 1;
#pragma unroll 1
      for (int i = 0; i < 2 * NK0; ++i) {
        const int g = i & 1, k = i >> 1;
        if (k < (g ? NK1 : NK0)) {
          const int tile = tile_of(g, j_x);
          const int ne = min(L.ept, p.M - tile * L.ept);
          const int nck = (ne + T2_G - 1) / T2_G;
          const int e = tile * L.ept + lane;
          const bool mine = lane < ne;
          const int s = s_x;
          if (s == 0) {
            ok_x = 0;
            if (mine) {
              slot_x = p.slot[e];
              pos_x = p.pos[e];
              epc_x = p.ep_count[e];
              ok_x = (slot_x >= 0 && slot_x < p.E * p.S && pos_x >= 0 && pos_x < p.L) ? 1 : 0;
              dn_x = p.done[e];
            }
          }
          unsigned long long rec = 0;
          int closes = 0;
          if (mine && ok_x) {
            rec = reinterpret_cast<unsigned long long>(p.ring + (size_t)slot_x * p.slot_stride + (size_t)pos_x * rec_bytes);
            if (dn_x || pos_x + 1 == p.L) {  // the cursor after this step
              closes = 1;
              epc_x += 1;
              slot_x = e * p.S + (int)(epc_x % p.S);
              pos_x = 0;
            } else {
              pos_x += 1;
            }
          }
          uint8_t* tm = tmem_ptr(g);
          reinterpret_cast<unsigned long long*>(tm + L.t_dstp)[(k & (T2_DEPTH - 1)) * 32 + lane] = rec;
          closes = __any_sync(0xFFFFFFFFu, closes);
          if (lane == 0) reinterpret_cast<int32_t*>(tm + L.t_closeany)[k & (T2_DEPTH - 1)] = closes;
          if (mine && s + 1 < T) dn_x = p.done[(size_t)(s + 1) * p.env_step_stride + e];
          __syncwarp();
          for (int c = 0; c < nck; ++c) {
            const int ge = min(T2_G, ne - c * T2_G);
            if (q >= (uint32_t)NS) {  // the slot's previous chunk is converted and its observations are stored
              mbar_wait(&B->cfree[qslot], qpar, abortf);
              mbar_wait(&B->sfree[qslot], qpar, abortf);
            }
            if (lane == 0) mbar_arrive_expect_tx(&B->full[qslot], (uint32_t)ge * L.prefix_bytes);
            __syncwarp();
            const size_t env0 = (size_t)tile * L.ept + (size_t)(c * T2_G);
            uint8_t* dst = stage + qslot * L.chunk_bytes;
            if (lane == 0)
              bulk_load(dst, p.obs + (size_t)s * p.obs_step_stride + env0 * (size_t)(n * D), (uint32_t)ge * L.obs_bytes,
                        &B->full[qslot]);
            if (lane == 1)
              bulk_load(dst + T2_G * L.obs_bytes, p.avail + (size_t)s * p.avail_step_stride + env0 * (size_t)(n * A),
                        (uint32_t)ge * L.av_bytes, &B->full[qslot]);
            ++q;
            if (++qslot == (uint32_t)NS) {
              qslot = 0;
              qpar ^= 1u;
            }
          }
          if (++s_x == T) {
            s_x = 0;
            ++j_x;
          }
        }
        { int32_t t; long long tl_; uint32_t tu;
          t = slot_x; slot_x = slot_y; slot_y = t;  t = pos_x; pos_x = pos_y; pos_y = t;  t = ok_x; ok_x = ok_y; ok_y = t;
          t = s_x; s_x = s_y; s_y = t;  t = j_x; j_x = j_y; j_y = t;
          tl_ = epc_x; epc_x = epc_y; epc_y = tl_;  tu = dn_x; dn_x = dn_y; dn_y = tu; }
      }
    } else if (warp == 14) {
      // =========================== tail warp: cursors, slot headers, reward/done (lane = environment) ===========
      // Per resident tile: post(k) writes reward/done of step k into the record, publishes the close flags and the
      // record addresses and opens epilogue 3 of that step (which writes the chosen actions and Q rows into the record
      // itself); finish(k), once the step is through, closes the slot header where the episode ends and moves the
      // cursor.  post(k + 1) follows finish(k) directly, long before epilogue 3 of step k + 1.  State of tile g in *_x,
      // of the other tile in *_y, changing places every half-iteration.
      unsigned long long c_episodes = 0, c_trunc = 0;
      uint32_t st_bits = 0;
      int32_t slot_x = 0, pos_x = 0, ok_x = 0, s_x = 0, j_x = 0, cl_x = 0, dn_x = 0;
      int32_t slot_y = 0, pos_y = 0, ok_y = 0, s_y = 0, j_y = 0, cl_y = 0, dn_y = 0;
      long long epc_x = 0, epc_y = 0;
#pragma unroll 1
      for (int i = -2; i < 2 * NK0; ++i) {
        const int g = i & 1, k = i >> 1;  // (i = -2, -1: k = -1, only the first posts)
        const int NKg = g ? NK1 : NK0;
        if (k >= 0 && k < NKg) {
          // ---- finish(g, k) ----
          const int tile = tile_of(g, j_x);
          const int ne = min(L.ept, p.M - tile * L.ept);
          const bool mine = lane < ne;
          const int e = tile * L.ept + lane;
          mbar_wait(&B->t[g].stepd, (uint32_t)k & 1u, abortf);  // the step's choices are on their way to the records
          if (cl_x) {
            p.slot_len[slot_x] = pos_x + 1;
            p.slot_complete[slot_x] = 1;
            c_episodes += 1;
            if (!dn_x) c_trunc += 1;
            epc_x += 1;
            slot_x = e * p.S + (int)(epc_x % p.S);
            pos_x = 0;
          } else if (mine && ok_x) {
            pos_x += 1;
          }
          if (++s_x == T) {  // the tile is done: its cursors go back to global memory
            s_x = 0;
            ++j_x;
            if (mine && ok_x) {
              p.slot[e] = slot_x;
              p.pos[e] = pos_x;
              p.ep_count[e] = epc_x;
              if (pos_x > 0) p.slot_len[slot_x] = pos_x;
            }
          }
        }
        if (k + 1 < NKg) {
          // ---- post(g, k + 1) ----
          const int kp = k + 1;
          const int tile = tile_of(g, j_x);
          const int ne = min(L.ept, p.M - tile * L.ept);
          const bool mine = lane < ne;
          const int e = tile * L.ept + lane;
          const int s = s_x;
          if (s == 0) {
            ok_x = 0;
            if (mine) {
              slot_x = p.slot[e];
              pos_x = p.pos[e];
              epc_x = p.ep_count[e];
              ok_x = (slot_x >= 0 && slot_x < p.E * p.S && pos_x >= 0 && pos_x < p.L) ? 1 : 0;
              if (!ok_x) st_bits |= MARL_STATUS_BAD_INDEX;
            }
          }
          float reward = 0.f;
          int done = 0;
          if (mine) {
            reward = p.reward[(size_t)s * p.env_step_stride + e];
            done = p.done[(size_t)s * p.env_step_stride + e] ? 1 : 0;
          }
          const int close = (ok_x && (done || pos_x + 1 == p.L)) ? 1 : 0;
          uint8_t* tm = tmem_ptr(g);
          reinterpret_cast<int32_t*>(tm + L.t_close)[(kp & 1) * 32 + lane] = close;
          // the record of this step, for epilogue 3 (the previous step's epilogue 3 has finished: stepd was awaited)
          unsigned long long recaddr = 0;
          if (mine && ok_x) recaddr = reinterpret_cast<unsigned long long>(p.ring + (size_t)slot_x * p.slot_stride + (size_t)pos_x * rec_bytes);
          reinterpret_cast<unsigned long long*>(tm + L.t_tdst)[lane] = recaddr;
          if (mine && ok_x) {
            uint8_t* rec = reinterpret_cast<uint8_t*>(recaddr);
            if (pos_x == 0) {  // an episode opens in this slot
              p.slot_epid[slot_x] = epc_x * (long long)p.E + e;
              p.slot_len[slot_x] = 0;
              p.slot_complete[slot_x] = 0;
            }
            // reward and done go straight to the record (16 bytes with their padding)
            *reinterpret_cast<uint4*>(rec + p.rl.off_reward) = make_uint4(__float_as_uint(reward), (uint32_t)done, 0u, 0u);
          }
          cl_x = close;
          dn_x = done;
          __syncwarp();
          if (lane == 0) mbar_arrive(&B->t[g].flags);
        }
        { int32_t t; long long tl_;
          t = slot_x; slot_x = slot_y; slot_y = t;  t = pos_x; pos_x = pos_y; pos_y = t;  t = ok_x; ok_x = ok_y; ok_y = t;
          t = s_x; s_x = s_y; s_y = t;  t = j_x; j_x = j_y; j_y = t;  t = cl_x; cl_x = cl_y; cl_y = t;  t = dn_x; dn_x = dn_y; dn_y = t;
          tl_ = epc_x; epc_x = epc_y; epc_y = tl_; }
      }
      if (c_episodes) atomicAdd(p.counters + CNT_EPISODES, c_episodes);
      if (c_trunc) atomicAdd(p.counters + CNT_TRUNCATED, c_trunc);
      if (st_bits) atomicOr(p.status, st_bits);
    } else {
      // =========================== store warp: observations from staging to the ring records ===========================
      uint32_t q = 0, qslot = 0, qpar = 0, pslot = 0;
      int32_t s_x = 0, j_x = 0, s_y = 0, j_y = 0;
#pragma unroll 1
      for (int i = 0; i < 2 * NK0; ++i) {
        const int g = i & 1, k = i >> 1;
        if (k < (g ? NK1 : NK0)) {
          const int tile = tile_of(g, j_x);
          const int ne = min(L.ept, p.M - tile * L.ept);
          const int nck = (ne + T2_G - 1) / T2_G;
          const unsigned long long* dstp = reinterpret_cast<const unsigned long long*>(tmem_ptr(g) + L.t_dstp) + (k & (T2_DEPTH - 1)) * 32;
          for (int c = 0; c < nck; ++c) {
            const int ge = min(T2_G, ne - c * T2_G);
            mbar_wait(&B->full[qslot], qpar, abortf);
            if (lane < ge) {
              const unsigned long long rec = dstp[c * T2_G + lane];
              const uint8_t* from = stage + qslot * L.chunk_bytes + (uint32_t)lane * L.obs_bytes;
              if (rec) bulk_store(reinterpret_cast<void*>(rec), from, L.obs_bytes);
            }
            bulk_commit();
            // every lane commits one (possibly empty) group per chunk, so "all but the latest" covers chunk q - 1
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            __syncwarp();
            if (q > 0 && lane == 0) mbar_arrive(&B->sfree[pslot]);
            pslot = qslot;
            ++q;
            if (++qslot == (uint32_t)NS) {
              qslot = 0;
              qpar ^= 1u;
            }
          }
          if (++s_x == T) {
            s_x = 0;
            ++j_x;
          }
        }
        { int32_t t; t = s_x; s_x = s_y; s_y = t;  t = j_x; j_x = j_y; j_y = t; }
      }
      bulk_wait_read_all();
      __syncwarp();
      if (q > 0 && lane == 0) mbar_arrive(&B->sfree[pslot]);
      bulk_wait_all();
    }
  } else if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(T2_REGS_CONV));
    // =========================== converters: staged observations -> bf16 operand; masks and epsilon draws ==========
    // Each of the four warps takes whole chunks (chunk c of a tile-step goes to warp c % 4); thread ci then owns row ci
    // of the tile for the epsilon draw.  Tile-steps are taken in the alternating order A k, B k, A k + 1, ...
    const int ci = tid - 256, cw = warp - 8;
    const uint32_t inv_nchunk = 0xFFFFFFFFu / (uint32_t)L.nchunk + 1u;  // j / nchunk == umulhi(j, inv) for j < 2^16
    const uint32_t amask = (1u << A) - 1u;
    uint32_t qbase = 0;
    int32_t s_x = 0, j_x = 0, s_y = 0, j_y = 0;  // step within its tile and tile count: tile g of the half-iteration / the other
#pragma unroll 1
    for (int i = 0; i < 2 * NK0; ++i) {
      const int g = i & 1, k = i >> 1;
      if (k < (g ? NK1 : NK0)) {
        const int tile = tile_of(g, j_x);
        const int e0 = tile * L.ept;
        const int ne = min(L.ept, p.M - e0);
        const int nck = (ne + T2_G - 1) / T2_G;
        const uint32_t t = p.t0 + (uint32_t)s_x;
        const float eps = eps_at(p, t);
        uint8_t* tm = tmem_ptr(g);
        uint8_t* xb = tm + L.t_x;
        uint32_t* sel = reinterpret_cast<uint32_t*>(tm + L.t_sel) + (k & 3) * TC_ROWS;  // mask | (pick & 0xFF) << 16
        // the operand buffer is free once fc1 of the tile's previous step has finished reading it
        if (k > 0) mbar_wait(&B->t[g].fc1d, (uint32_t)(k - 1) & 1u, abortf);
        for (int c = cw; c < nck; c += T2_CONV / 32) {
          const int ge = min(T2_G, ne - c * T2_G);
          const int Rc = ge * n;
          const int r0 = c * T2_G * n;
          const uint32_t q = qbase + (uint32_t)c, qslot = q % (uint32_t)NS, qpar = (q / (uint32_t)NS) & 1u;
          const uint8_t* src = stage + qslot * L.chunk_bytes;
          const unsigned long long* recs = reinterpret_cast<const unsigned long long*>(tm + L.t_dstp) + (k & (T2_DEPTH - 1)) * 32 + c * T2_G;
          mbar_wait(&B->full[qslot], qpar, abortf);
          const int items = Rc * L.nchunk;
          // five items (8 columns of one row each) per lane and pass, all loads before the first store: the loop is
          // bound by shared-memory latency otherwise
          for (int j0 = lane; j0 < items; j0 += 32 * 5) {
            float4 v[5][2];
            uint32_t dsto[5];
#pragma unroll
            for (int u = 0; u < 5; ++u) {
              const int jj = j0 + 32 * u;
              const int rr = (int)__umulhi((uint32_t)jj, inv_nchunk), cc = jj - rr * L.nchunk;
              dsto[u] = jj < items ? (uint32_t)cc * TC_LBO_X + (uint32_t)(r0 + rr) * 16u : 0xFFFFFFFFu;
              v[u][0] = v[u][1] = make_float4(0.f, 0.f, 0.f, 0.f);
              if (jj < items && cc * 8 < D) {
                const float4* s4 = reinterpret_cast<const float4*>(src + (uint32_t)(rr * D) * 4u + (uint32_t)cc * 32u);
                v[u][0] = s4[0];
                v[u][1] = s4[1];
              }
            }
#pragma unroll
            for (int u = 0; u < 5; ++u)
              if (dsto[u] != 0xFFFFFFFFu)
                *reinterpret_cast<uint4*>(xb + dsto[u]) = make_uint4(pack_bf16x2(v[u][0].x, v[u][0].y), pack_bf16x2(v[u][0].z, v[u][0].w),
                                                                     pack_bf16x2(v[u][1].x, v[u][1].y), pack_bf16x2(v[u][1].z, v[u][1].w));
          }
          const uint8_t* avs = src + T2_G * L.obs_bytes;  // the chunk's availability bytes, rows contiguous
          const uint32_t per_env = L.av_bytes / 16u;
          for (uint32_t i = lane; i < (uint32_t)ge * per_env; i += 32) {
            const uint32_t envc = i / per_env;
            const unsigned long long rec = recs[envc];
            if (rec) reinterpret_cast<uint4*>(rec + L.obs_bytes)[i - envc * per_env] = reinterpret_cast<const uint4*>(avs)[i];
          }
          // availability masks: a row's A bytes read as aligned words, each word's four "byte is non-zero" flags
          // gathered with one multiply
          for (int rc = lane; rc < Rc; rc += 32) {
            const uint32_t off = (uint32_t)(rc * A);
            const uint32_t* w = reinterpret_cast<const uint32_t*>(avs + (off & ~3u));
            unsigned long long bits = 0;
#pragma unroll
            for (int kk = 0; kk < 5; ++kk) {
              const uint32_t v = w[kk];
              const uint32_t nz = ((v | ((v & 0x7F7F7F7Fu) + 0x7F7F7F7Fu)) & 0x80808080u) >> 7;  // 0x01 per non-zero byte
              bits |= (unsigned long long)((nz * 0x01020408u) >> 24 & 0xFu) << (4 * kk);
            }
            sel[r0 + rc] = (uint32_t)(bits >> (off & 3u)) & amask;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&B->cfree[qslot]);
        }
        qbase += (uint32_t)nck;
        fence_proxy_async_smem();
        t2_warp_arrive(&B->t[g].xready, lane);
        asm volatile("bar.sync 2, 128;" ::: "memory");  // the masks were written by the chunks' warps
        if (ci < ne * n) {
          const int rel = ci / n, rai = ci - rel * n;
          const uint32_t mask = sel[ci];
          int pick = -1;
          if (mask != 0) pick = draw_explore(mask, eps, p.seed, t, (uint32_t)(e0 + rel), (uint32_t)rai);
          sel[ci] = mask | (((uint32_t)pick & 0xFFu) << 16);
        }
        t2_warp_arrive(&B->t[g].selready[k & 3], lane);
        if (++s_x == T) {
          s_x = 0;
          ++j_x;
        }
      }
      { int32_t t; t = s_x; s_x = s_y; s_y = t;  t = j_x; j_x = j_y; j_y = t; }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(T2_REGS_EPI));
    // =========================== epilogue threads: (agent row, 32 hidden columns) of BOTH resident tiles in turn ===========================
    // Per pair of steps: E1(A) E3(B) E2(A) E1(B) E3(A) E2(B) - the order in which the MMA warp serves the tiles, so a
    // tile's GEMM round trip is always covered by an epilogue of the other tile.
    const int row = tid & 127, half = tid >> 7;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int el = row / n, ai = row - el * n;
    const int cb = half * 32;  // first hidden column of this thread
    unsigned long long c_steps = 0, c_explore = 0, c_noavail = 0;
    uint32_t st_bits = 0;
    // hx, cx, jx: hidden state, context and tile count of tile g of the half-iteration; hy, cy, jy: of the other tile.
    // They change places every half-iteration, so every phase exists once in the code.
    float hx[32], hy[32];
    struct TileCtx { bool live, is_row; int e, s; size_t grow; } cx = {false, false, 0, 0, 0}, cy = {false, false, 0, 0, 0};
    int jx = 0, jy = 0;

    // ---- tile prologue: hidden state and last actions from global memory ----
    auto prologue = [&](const int g, float (&h)[32], TileCtx& c, int j) {
      uint8_t* tm = tmem_ptr(g);
      uint8_t* yh = tm + L.t_yh;
      int32_t* la_s = reinterpret_cast<int32_t*>(tm + L.t_la);
      const int tile = tile_of(g, j);
      const int e0 = tile * L.ept;
      const int R = min(L.ept, p.M - e0) * n;
      c.live = row < R;
      c.is_row = c.live && half == 0;
      c.e = e0 + el;
      c.grow = (size_t)c.e * n + ai;
      c.s = 0;
      const int la_mem = c.is_row ? p.last_action[c.grow] : -1;
      const float4* src = reinterpret_cast<const float4*>(p.h + c.grow * TC_H + cb);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float4 v = c.live ? src[q] : make_float4(0.f, 0.f, 0.f, 0.f);
        h[4 * q] = v.x; h[4 * q + 1] = v.y; h[4 * q + 2] = v.z; h[4 * q + 3] = v.w;
      }
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        const uint4 o = make_uint4(pack_bf16x2(h[8 * cc], h[8 * cc + 1]), pack_bf16x2(h[8 * cc + 2], h[8 * cc + 3]),
                                   pack_bf16x2(h[8 * cc + 4], h[8 * cc + 5]), pack_bf16x2(h[8 * cc + 6], h[8 * cc + 7]));
        *reinterpret_cast<uint4*>(yh + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
      }
      if (half == 0) la_s[row] = la_mem >= A ? -1 : la_mem;
      fence_proxy_async_smem();
      tc_fence_before_sync();
      asm volatile("bar.sync 1, 256;" ::: "memory");  // la_s is read by both threads of a row
      t2_warp_arrive(&B->t[g].tiled, lane);
    };
    // ---- tile epilogue: state back to global memory ----
    auto tile_end = [&](const int g, float (&h)[32], TileCtx& c) {
      const int32_t* la_s = reinterpret_cast<const int32_t*>(tmem_ptr(g) + L.t_la);
      if (c.is_row) p.last_action[c.grow] = la_s[row];
      if (c.live) {
        float4* dsth = reinterpret_cast<float4*>(p.h + c.grow * TC_H + cb);
#pragma unroll
        for (int q = 0; q < 8; ++q) dsth[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
      }
    };
    // ---- epilogue 1: y = relu(fc1 + W1[:, last action]) -> bf16 operand.  Bias and agent-id column are inside the
    //      GEMM; the accumulator sits in the candidate-input columns. ----
    auto epi1 = [&](const int g, TileCtx& c, uint32_t k) {
      T2TileBars& tb = B->t[g];
      uint8_t* tm = tmem_ptr(g);
      uint8_t* yh = tm + L.t_yh;
      const uint32_t taddr = tmem + lane_addr + (uint32_t)g * T2_TILE_COLS;
      const uint32_t par = k & 1u;
      mbar_wait(&tb.fc1d, par, abortf);
      tc_fence_after_sync();
      const int last = reinterpret_cast<const int32_t*>(tm + L.t_la)[row];  // (-1 after an episode end: set in epilogue 3)
      const float* tlr = tab_la + (last >= 0 ? last : 0) * TC_TAB + cb;
      uint32_t yp[16];  // the thread's 32 values as bf16 pairs
      {
        uint32_t v2[2][16];
        tmem_ld16(taddr + T2_IN + cb, v2[0]);
        tmem_ld16(taddr + T2_IN + cb + 16, v2[1]);
        tmem_ld_wait();
#pragma unroll
        for (int c16 = 0; c16 < 2; ++c16) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float4 l4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (last >= 0) l4 = *reinterpret_cast<const float4*>(tlr + c16 * 16 + 4 * q);
            const float y0 = fmaxf(__uint_as_float(v2[c16][4 * q]) + l4.x, 0.f);
            const float y1 = fmaxf(__uint_as_float(v2[c16][4 * q + 1]) + l4.y, 0.f);
            const float y2 = fmaxf(__uint_as_float(v2[c16][4 * q + 2]) + l4.z, 0.f);
            const float y3 = fmaxf(__uint_as_float(v2[c16][4 * q + 3]) + l4.w, 0.f);
            yp[c16 * 8 + 2 * q] = pack_bf16x2(y0, y1);
            yp[c16 * 8 + 2 * q + 1] = pack_bf16x2(y2, y3);
          }
        }
      }
      // the operand buffer still holds h' until the step's h-side products have read it
      mbar_wait(&tb.hsd, par, abortf);
#pragma unroll
      for (int cc = 0; cc < 4; ++cc)
        *reinterpret_cast<uint4*>(yh + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) =
            make_uint4(yp[4 * cc], yp[4 * cc + 1], yp[4 * cc + 2], yp[4 * cc + 3]);
      fence_proxy_async_smem();
      tc_fence_before_sync();
      t2_warp_arrive(&tb.yready, lane);
    };
    // ---- epilogue 2: gate math, new hidden state (fp32 registers) and its bf16 operand (over y, which the y-side GEMM
    //      has finished reading).  The r and z accumulators hold half the pre-activation:
    //      sigmoid(v) = 0.5 * tanh(v / 2) + 0.5 ----
    auto epi2 = [&](const int g, float (&h)[32], uint32_t k) {
      T2TileBars& tb = B->t[g];
      uint8_t* yh = tmem_ptr(g) + L.t_yh;
      const uint32_t taddr = tmem + lane_addr + (uint32_t)g * T2_TILE_COLS;
      mbar_wait(&tb.grud, k & 1u, abortf);
      tc_fence_after_sync();
      uint32_t gb[2][4][8];  // [buffer][r, z, candidate-input, candidate-hidden][column]
      auto request = [&](int c8, uint32_t (&d)[4][8]) {
        const uint32_t col = (uint32_t)(cb + c8 * 8);
        tmem_ld8(taddr + T2_R + col, d[0]);
        tmem_ld8(taddr + T2_R + 64 + col, d[1]);
        tmem_ld8(taddr + T2_IN + col, d[2]);
        tmem_ld8(taddr + T2_HN + col, d[3]);
      };
      request(0, gb[0]);
#pragma unroll
      for (int c8 = 0; c8 < 4; ++c8) {
        tmem_ld_wait();
        if (c8 + 1 < 4) request(c8 + 1, gb[(c8 + 1) & 1]);
        uint32_t(&v)[4][8] = gb[c8 & 1];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const float rg = fmaf(0.5f, tanh_fast(__uint_as_float(v[0][jj])), 0.5f);
          const float zg = fmaf(0.5f, tanh_fast(__uint_as_float(v[1][jj])), 0.5f);
          const float cand = tanh_fast(fmaf(rg, __uint_as_float(v[3][jj]), __uint_as_float(v[2][jj])));
          const float hp = h[c8 * 8 + jj];
          h[c8 * 8 + jj] = fmaf(zg, hp - cand, cand);  // (1 - z) * cand + z * h
        }
        const float* hv = h + c8 * 8;
        const uint4 o = make_uint4(pack_bf16x2(hv[0], hv[1]), pack_bf16x2(hv[2], hv[3]), pack_bf16x2(hv[4], hv[5]),
                                   pack_bf16x2(hv[6], hv[7]));
        *reinterpret_cast<uint4*>(yh + (uint32_t)(half * 4 + c8) * TC_LBO_A + (uint32_t)row * 16u) = o;
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      t2_warp_arrive(&tb.hready, lane);
    };
    // ---- epilogue 3: the row owners choose and complete the record's tail; a closed episode restarts from a zero
    //      hidden state and no last action ----
    auto epi3 = [&](const int g, float (&h)[32], TileCtx& c, uint32_t k) {
      T2TileBars& tb = B->t[g];
      uint8_t* tm = tmem_ptr(g);
      uint8_t* yh = tm + L.t_yh;
      int32_t* la_s = reinterpret_cast<int32_t*>(tm + L.t_la);
      const uint32_t taddr = tmem + lane_addr + (uint32_t)g * T2_TILE_COLS;
      const uint32_t par = k & 1u;
      mbar_wait(&tb.flags, par, abortf);  // close flags of this step written
      mbar_wait(&tb.fc2d, par, abortf);   // (both halves: the hidden operand may be cleared below)
      tc_fence_after_sync();
      const bool closes = c.live && reinterpret_cast<const int32_t*>(tm + L.t_close)[par * 32 + el] != 0;
      if (half == 0) {
        uint32_t qv[16], q1[16], q2[16], q3[16];
        tmem_ld16(taddr + T2_HN, qv);
        tmem_ld16(taddr + T2_HN + 16, q1);
        tmem_ld16(taddr + T2_HN + 32, q2);
        tmem_ld16(taddr + T2_HN + 48, q3);
        tmem_ld_wait();
#pragma unroll
        for (int a = 0; a < 16; ++a)
          qv[a] = __float_as_uint((__uint_as_float(qv[a]) + __uint_as_float(q1[a])) + (__uint_as_float(q2[a]) + __uint_as_float(q3[a])));
        tc_fence_before_sync();
        if (c.is_row) {
          mbar_wait(&tb.selready[k & 3], (k >> 2) & 1, abortf);
          const uint32_t sp = reinterpret_cast<const uint32_t*>(tm + L.t_sel)[(k & 3) * TC_ROWS + row];
          const uint32_t mask = sp & 0xFFFFu;
          const int pick = (int)(int8_t)(sp >> 16);
          // greedy rule: m = max over available, thr = m - 1e-4f, lowest available a with Q >= thr
          float qm[16];
#pragma unroll
          for (int a = 0; a < 16; ++a) qm[a] = ((mask >> a) & 1u) ? __uint_as_float(qv[a]) : -INFINITY;
          float red[16];
#pragma unroll
          for (int a = 0; a < 16; ++a) red[a] = qm[a];
#pragma unroll
          for (int w = 8; w >= 1; w >>= 1)
#pragma unroll
            for (int a = 0; a < w; ++a) red[a] = fmaxf(red[a], red[a + w]);
          const float thr = __fsub_rn(red[0], 1e-4f);
          uint32_t ge = 0;
#pragma unroll
          for (int a = 0; a < 16; ++a) ge |= (qm[a] >= thr ? 1u : 0u) << a;
          ge &= mask;
          const int gsel = ge ? __ffs(ge) - 1 : __ffs(mask) - 1;
          const int act = mask == 0 ? 0 : (pick >= 0 ? pick : gsel);
          c_steps += 1;
          c_explore += pick >= 0 ? 1u : 0u;
          if (mask == 0) { c_noavail += 1; st_bits |= MARL_STATUS_NO_AVAIL; }
          la_s[row] = closes ? -1 : act;  // read by both threads of the row in the next step's epilogue 1
          // action and Q row go straight to the record (its address comes from the tail warp, with the close flags)
          const unsigned long long rec = reinterpret_cast<const unsigned long long*>(tm + L.t_tdst)[el];
          if (rec) {
            float* qrow = reinterpret_cast<float*>(rec + p.rl.off_q) + ai * A;
            if ((A & 1) == 0) {  // rows of an even number of floats start on 8-byte boundaries
#pragma unroll
              for (int a = 0; a < 16; a += 2)
                if (a < A) *reinterpret_cast<float2*>(qrow + a) = make_float2(__uint_as_float(qv[a]), __uint_as_float(qv[a + 1]));
            } else {
#pragma unroll
              for (int a = 0; a < 16; ++a)
                if (a < A) qrow[a] = __uint_as_float(qv[a]);
            }
            reinterpret_cast<int32_t*>(rec + p.rl.off_action)[ai] = act;
          }
          const int tk = p.trace_first + c.s;
          if (tk < p.trace_cap) {
            const size_t trow = ((size_t)tk * p.E + c.e) * n + ai;
            if (p.trace_actions) p.trace_actions[trow] = act;
            if (p.trace_q) {
#pragma unroll
              for (int a = 0; a < 16; ++a)
                if (a < A) p.trace_q[trow * A + a] = __uint_as_float(qv[a]);
            }
          }
          if (p.actions_out && c.s == T - 1) p.actions_out[c.grow] = act;
        }
      }
      if (closes) {
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) h[jj] = 0.f;
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
          *reinterpret_cast<uint4*>(yh + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      asm volatile("bar.sync 1, 256;" ::: "memory");  // la_s written before any thread of the row reads it
      t2_warp_arrive(&tb.stepd, lane);
      c.s += 1;
    };

    if (NK0 > 0) prologue(0, hx, cx, 0);
    if (NK1 > 0) prologue(1, hy, cy, 0);
    // half-iteration i: tile g = i & 1 at its step k = i >> 1: E1(g, k), E3 of the other tile's step in flight
    // (B's k - 1 for g = A, A's k for g = B), E2(g, k).  One extra half-iteration takes B's last E3.
#pragma unroll 1
    for (int i = 0; i < 2 * NK0 + 1; ++i) {
      const int g = i & 1, k = i >> 1, o = g ^ 1;
      const int NKg = g ? NK1 : NK0, NKo = g ? NK0 : NK1;
      const int ko = g ? k : k - 1;
      if (k < NKg) epi1(g, cx, (uint32_t)k);
      if (ko >= 0 && ko < NKo) {
        epi3(o, hy, cy, (uint32_t)ko);
        if (cy.s == T) {
          tile_end(o, hy, cy);
          ++jy;
          if (ko + 1 < NKo) prologue(o, hy, cy, jy);
        }
      }
      if (k < NKg) epi2(g, hx, (uint32_t)k);
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        const float t = hx[q];
        hx[q] = hy[q];
        hy[q] = t;
      }
      { const TileCtx t = cx; cx = cy; cy = t; const int tj = jx; jx = jy; jy = tj; }
    }
    if (c_steps) atomicAdd(p.counters + CNT_AGENT_STEPS, c_steps);
    if (c_explore) atomicAdd(p.counters + CNT_EXPLORED, c_explore);
    if (c_noavail) atomicAdd(p.counters + CNT_NO_AVAIL, c_noavail);
    if (st_bits) atomicOr(p.status, st_bits);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && B->abort) {
    atomicOr(p.status, MARL_STATUS_TIMEOUT);
    // diagnosis: which barrier (index inside the barrier block) and which warp gave up first
    atomicCAS(p.status + 1, 0u, ((((B->abort & 0xFFFFFu) - (smem_u32(B) & 0xFFFFFu)) >> 3) & 0xFFu) | (((B->abort >> 20) & 0xFFu) << 8));
  }
  if (warp == 12) tmem_dealloc(tmem, T2_COLS);
}

// Returns the number of kernels launched, 0 if this launch is not one the kernel takes (the caller then uses the
// pipelined kernel), or a negative cudaError.
int launch_actor_tc2(const ActorParams& p_in, int sms, cudaStream_t stream) {
  if (p_in.env_ids != nullptr || p_in.lagged || p_in.T < 8) return 0;
  if (!tc2_supported(p_in.n, p_in.D, p_in.A, p_in.H, p_in.prec)) return 0;
  const T2Layout L = t2_layout(p_in.n, p_in.D, p_in.A, (int)p_in.rl.rec_bytes);
  ActorParams p = p_in;
  p.ept = L.ept;
  p.num_tiles = (p.M + L.ept - 1) / L.ept;
  if (p.num_tiles <= sms) return 0;  // with one tile per SM there is nothing to pair
  if (reinterpret_cast<uintptr_t>(p.obs) % 16 || reinterpret_cast<uintptr_t>(p.avail) % 16) return 0;
  if ((p.obs_step_stride * 4) % 16 || p.avail_step_stride % 16) return 0;
  static uint32_t configured[SMEM_OPTIN_DEVICES];
  {
    const cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(actor_tc2_kernel), L.total, configured);
    if (e != cudaSuccess) return -(int)e;
  }
  const int grid = sms;
  actor_tc2_kernel<<<grid, T2_THREADS, L.total, stream>>>(p, L);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 1 : -(int)err;
}

}  // namespace marl
