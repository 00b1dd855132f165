// Pipelined tensor-core actor kernel for sm_100a: bf16 operands, hidden size 64.
//
// Same arithmetic, weight image, tensor-memory plan and tile-major schedule as the one-tile kernel in
// actor_tc.cu (one thread block owns a tile of whole environments - up to 128 agent rows - and runs all T steps
// of the launch for it, Sec. III-A: environments never exchange data).  What differs is how a step's data moves,
// so that nothing but the network itself is left on the per-step dependency chain:
//
//   * Everything about a step except Q and the chosen action is known before the network runs: the
//     observations, the availability bytes, reward and done (the worker "gets observations", Algorithm 2), and
//     with the done flags the whole sequence of ring cursors (Algorithm 1: a track ends when the environment
//     says so).  A ring record is therefore written in two pieces: its prefix [obs | avail] as soon as the
//     inputs have arrived, and its tail [action | Q | reward, done] after the choice.
//   * Staging is a ring of NS chunks of four environments, each filled by two bulk loads (the chunk's
//     observations and its availability bytes are contiguous in the input arrays) issued up to NS chunks ahead
//     of the network, across step and tile boundaries.  Bulk copies are kept few and large: their issue rate,
//     not their bandwidth, limits a kernel that moves a few kilobytes per environment.
//   * A warpgroup of converters (one warp per chunk, a step's chunks side by side) turns the fp32 observations
//     into the bf16 fc1 operand, stores the availability bytes to the records and builds from them the mask and
//     the Philox epsilon draw of every row; a store warp sends each environment's observations from staging to
//     its record with one bulk store.
//   * fc1 of step s+1 needs only that operand, and the h-side gate products of step s+1 only the new hidden
//     state (unless an episode of the tile ends with step s), so both are issued during step s; per step the
//     epilogue threads are left with: +last-action term, ReLU (epilogue 1) -> gate math (epilogue 2) -> masked arg-max (epilogue 3).
//
// Warp roles (512 threads): warps 0-7 epilogue (thread = one agent row x 32 hidden columns), warps 8-11
// converters, warp 12 issues every tcgen05.mma, warp 13 issues the loads and runs the ring cursors ahead
// (lane = environment) to publish each step's record addresses, warp 14 follows the same cursors in step with
// the network: slot headers, counters, reward/done and the copy of the tails to the ring, warp 15 stores the
// observations from staging to the records.  All
// hand-offs are mbarriers with bounded waits; an expired wait sets MARL_STATUS_TIMEOUT and lets the block run
// to its end with every index in range.
#include <cstring>
#include <type_traits>

#include "actor_tc_layout.cuh"
#include "common.cuh"
#include "launch_util.cuh"
#include "tcgen05.cuh"

namespace marl {

constexpr int TP_THREADS = 512;
constexpr int TP_CONV = 128;          // converter threads
constexpr int TP_G = 4;               // environments per staging chunk
constexpr int TP_MAX_STAGES = 8;
// fc2 is four K = 16 steps.  Dependent tcgen05.mma on one accumulator run one after the other at a few hundred
// cycles each whatever their width, so with 16 outputs the steps go to four accumulators (summed in epilogue 3).
constexpr int TP_QPARTS = 4;
constexpr int TP_DST_DEPTH = 16;      // steps of record addresses kept: the loads run at most TP_MAX_STAGES chunks (steps) ahead
// Register split (setmaxnreg): launched with 128 registers per thread (512 * 128 = 65536); afterwards
// 256 * 144 + 128 * 112 + 128 * 112 = 65536.
constexpr int TP_REGS_EPI = 144, TP_REGS_CONV = 112, TP_REGS_SVC = 112;

struct TpLayout {
  int32_t Dk, NQ, nchunk, ept, ohK, ohc, NS, plain;
  uint32_t prefix_bytes, tail_bytes, chunk_bytes, obs_bytes, av_bytes, rs_env, rs_bytes, off_rstage;
  uint32_t off_W1, off_Wih, off_Whh, off_Bg, off_Bhn, off_W2, off_tab_la, wbytes;
  uint32_t off_x, off_y, off_hb, off_oh, off_stage, off_tail, off_sel, off_la, off_close, off_closeany, off_rowenv, off_dstp, off_tdst, off_bar, total;
};

struct TpBars {
  uint64_t full[TP_MAX_STAGES], cfree[TP_MAX_STAGES], sfree[TP_MAX_STAGES];  // chunk loaded / converted / stored
  uint64_t xready, fc1d, yready, grud, hready, fc2d, stepd, wload, flags;
  // tile prologue done.  Its own barrier: as one more phase of stepd it could complete, together with the last
  // step's phase, before a waiter that is still busy with the next tile's fc1 has looked - two phases ahead of a
  // parity wait reads as none.
  uint64_t tiled;
  uint64_t selready[4];  // one per buffer of the four-deep draw hand-off: the converters run up to two steps ahead
  uint32_t tmem_base, abort;
};

// M, sms: the launch's batch and the number of blocks it may use (0: the largest tiles, for the shape check).
static TpLayout tp_layout(int n, int D, int A, int rec_bytes, int M = 0, int sms = 0) {
  const TcLayout W = tc_layout(n, D, A, rec_bytes);
  TpLayout L;
  memset(&L, 0, sizeof(L));
  L.Dk = W.Dk; L.NQ = W.NQ; L.nchunk = W.nchunk; L.ept = W.ept; L.ohK = W.ohK; L.ohc = W.ohc;
  L.off_W1 = W.off_W1; L.off_Wih = W.off_Wih; L.off_Whh = W.off_Whh; L.off_Bg = W.off_Bg; L.off_Bhn = W.off_Bhn;
  L.off_W2 = W.off_W2; L.off_tab_la = W.off_tab_la; L.wbytes = W.wbytes;
  L.obs_bytes = (uint32_t)(n * D) * 4u;
  L.av_bytes = (uint32_t)(n * A);
  L.prefix_bytes = L.obs_bytes + L.av_bytes;  // of one environment in staging: [obs of the chunk | avail of the chunk]
  // Shapes whose per-environment blocks are not 16-byte multiples ("plain"): a whole chunk's observations still are
  // (4 n D floats), so they load the same way, in tiles of whole chunks; the converters then lay observations and
  // availability bytes out as the records want them, for the store warp's bulk stores.
  // plain = 1: observation rows that are not 16-byte multiples (word-by-word path, tiles of whole chunks so that
  // every chunk starts on a 16-byte boundary); plain = 2: only the availability blocks are unaligned - observations
  // take the aligned path, availability bytes the shifted one.
  L.plain = D % 8 != 0 ? 1 : ((n * A) % 16 != 0 ? 2 : 0);
  if (L.plain == 1) L.ept = L.ept / TP_G * TP_G;
  // The plain shapes are bound by their converters, whose work grows with the tile: the smallest tile that keeps the
  // number of waves evens the blocks out (4096 environments of 5 agents: 164 tiles of 25 on 148 blocks take two
  // waves, and so do 293 tiles of 14, each at half the conversion).  The aligned shapes run at the step's dependency
  // chain whatever the tile holds, so they keep full tiles.
  if (L.plain != 0 && M > 0 && sms > 0) {
    const int tiles = (M + L.ept - 1) / L.ept, waves = (tiles + sms - 1) / sms;
    int e2 = (M + waves * sms - 1) / (waves * sms);
    if (L.plain == 1) e2 = (e2 + TP_G - 1) / TP_G * TP_G;
    if (e2 < TP_G) e2 = TP_G;
    if (e2 < L.ept) L.ept = e2;
  }
  L.tail_bytes = (uint32_t)rec_bytes - (up16(L.obs_bytes) + up16(L.av_bytes));
  // (plain shapes: a chunk's availability bytes need not start on a 16-byte boundary of the input array; the load
  // then covers the aligned range around them, at most 30 bytes more)
  L.chunk_bytes = L.plain ? TP_G * L.obs_bytes + up16(TP_G * L.av_bytes) + 16u : TP_G * L.prefix_bytes;
  uint32_t o = L.wbytes;
  L.off_x = o; o += up16((uint32_t)L.nchunk * TC_LBO_X);
  L.off_y = o; o += 8 * TC_LBO_A;
  L.off_hb = o; o += 8 * TC_LBO_A;
  L.off_oh = o; o += (uint32_t)L.ohc * TC_LBO_A;
  L.off_tail = o; o += 2u * (uint32_t)L.ept * L.tail_bytes;
  L.off_sel = o; o += 4u * TC_ROWS * 8;
  L.off_la = o; o += TC_ROWS * 4;
  L.off_close = o; o += 2 * 32 * 4;
  L.off_closeany = o; o += TP_DST_DEPTH * 4;
  L.off_rowenv = o; o += TC_ROWS * 4;
  L.off_dstp = o; o += TP_DST_DEPTH * 32 * 8;
  L.off_tdst = o; o += 32 * 8;
  L.off_bar = o; o += (uint32_t)((sizeof(TpBars) + 15) & ~15u);
  L.off_stage = o;
  // plain shapes: the converters also lay observations and availability bytes out as the records want them (each
  // block padded to 16 bytes), one image per staging slot, for the store warp's bulk stores
  L.rs_env = L.plain == 1 ? up16(L.obs_bytes) + up16(L.av_bytes) : 0;  // the record's prefix [obs | avail], padded as in the ring
  L.rs_bytes = TP_G * L.rs_env;
  const uint32_t room = o + 64 < TC_SMEM_MAX ? TC_SMEM_MAX - o - 64 : 0;
  int ns = (int)(room / (L.chunk_bytes + L.rs_bytes));
  if (ns > TP_MAX_STAGES) ns = TP_MAX_STAGES;
  if (ns < 0) ns = 0;
  // A converter warp waits for "the other phase" of a slot's barrier, which reads as complete while the slot's
  // previous chunk has not even arrived.  That previous chunk must therefore be behind the waiter in program order:
  // either it belongs to an earlier step (the ring holds a whole tile-step of chunks), or the same warp converts it
  // (a converter warp takes every fourth chunk, so the ring length is a multiple of four).
  const int nck_max = (L.ept + TP_G - 1) / TP_G;
  if (ns < nck_max) ns = ns / (TP_CONV / 32) * (TP_CONV / 32);
  L.NS = ns;
  L.off_rstage = o + (uint32_t)ns * L.chunk_bytes + 64;  // (+64: the mask words read a few bytes past a row)
  L.total = L.off_rstage + (uint32_t)ns * L.rs_bytes;
  return L;
}

// Shapes this kernel takes: at least 4 agents (tiles of at most 32 environments, one lane each) and a staging ring
// of at least three chunks of four environments.
bool tcp_supported(int n, int D, int A, int H, int prec) {
  if (prec != MARL_PRECISION_BF16 || H != TC_H) return false;
  if (D < 1 || D > 256 || n < 4 || n > 32 || A < 1 || A > 32) return false;
  const TpLayout L = tp_layout(n, D, A, rec_bytes_of(n, D, A));
  // enough staging for loads to run ahead of the network (tp_layout leaves 0 where the ring would be unsafe)
  return L.ept >= TP_G && L.NS >= 3 && L.total <= TC_SMEM_MAX;
}

// Tensor-memory columns of one Q buffer.
__host__ __device__ constexpr uint32_t tp_qstride(int NQ) { return NQ == 16 ? TP_QPARTS * 16u : (uint32_t)NQ; }

// One arrival per warp: every lane has made its writes (and proxy fences) before the warp-level barrier, lane 0
// then arrives for all of them.  Arrivals on one mbarrier are serialised, so 8 instead of 256 matters.
__device__ __forceinline__ void warp_arrive(uint64_t* bar, int lane) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
}

// ---- MMA issue helpers.  Descriptors are rebuilt from the layout (kernel parameter space) where they are used:
//      nothing is kept in local memory, whose loads would go to L2 - the L1 left beside 227 KB of shared memory is
//      tiny - and stall every tcgen05.mma behind them.
constexpr uint32_t TP_LBO_W1 = TC_H * 16, TP_LBO_G = 3 * TC_H * 16;   // k-chunk strides of the 64- and 192-row weight operands
constexpr uint64_t TP_K_A = (2 * TC_LBO_A) >> 4, TP_K_X = (2 * TC_LBO_X) >> 4, TP_K_W1 = (2 * TP_LBO_W1) >> 4,
                   TP_K_G = (2 * TP_LBO_G) >> 4;                       // descriptor increments of one K = 16 step

// fc1 of one step: observations x W1, then the one-hot tile x (bias pieces, agent-id columns); commits to fc1d.
__device__ __forceinline__ void tp_issue_fc1(const TpLayout& L, uint32_t sb, uint32_t tmem, int lane, uint64_t* fc1d) {
  using namespace tc;
  tc_fence_after_sync();
  if (lane == 0) {
    const uint64_t d_x = smem_desc(sb + L.off_x, TC_LBO_X, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
    const uint64_t d_W1 = smem_desc(sb + L.off_W1, TP_LBO_W1, 128);
    const uint64_t d_W1oh = smem_desc(sb + L.off_W1 + (uint32_t)L.nchunk * TP_LBO_W1, TP_LBO_W1, 128);
    const uint32_t id64 = idesc_bf16_f32(128, 64);
    const int ks_obs = L.Dk / 16, ks_oh = L.ohK / 16;
    for (int ks = 0; ks < ks_obs; ++ks) mma_bf16(tmem + TM_FC1, d_x + ks * TP_K_X, d_W1 + ks * TP_K_W1, id64, ks > 0);
    for (int ks = 0; ks < ks_oh; ++ks) mma_bf16(tmem + TM_FC1, d_oh + ks * TP_K_A, d_W1oh + ks * TP_K_W1, id64, 1);
    mma_commit(fc1d);
  }
  __syncwarp();
}

// h-side gate products of one step: the first MMA seeds r | z | candidate-input with their biases (contiguous in
// tensor memory: one N = 192 accumulator), the last one seeds the step's Q accumulator with the output bias.
template <int NQ>
__device__ __forceinline__ void tp_issue_hside(const TpLayout& L, uint32_t sb, uint32_t tmem, int lane, uint32_t qcol) {
  using namespace tc;
  tc_fence_after_sync();
  if (lane == 0) {
    const uint64_t d_h = smem_desc(sb + L.off_hb, TC_LBO_A, 128), d_oh = smem_desc(sb + L.off_oh, TC_LBO_A, 128);
    const uint64_t d_Whh = smem_desc(sb + L.off_Whh, TP_LBO_G, 128);
    const uint64_t d_Whh_n = smem_desc(sb + L.off_Whh + 2 * TC_H * 16, TP_LBO_G, 128);  // the candidate rows of each k-chunk
    const uint64_t d_Bg = smem_desc(sb + L.off_Bg, TP_LBO_G, 128), d_Bhn = smem_desc(sb + L.off_Bhn, TP_LBO_W1, 128);
    const uint64_t d_W2b = smem_desc(sb + L.off_W2 + 8u * NQ * 16, NQ * 16, 128);            // bias pieces of W2: k-chunks 8, 9
    const uint32_t id64 = idesc_bf16_f32(128, 64), id128 = idesc_bf16_f32(128, 128), id192 = idesc_bf16_f32(128, 192);
    mma_bf16(tmem + TM_R, d_oh, d_Bg, id192, 0);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      mma_bf16(tmem + TM_R, d_h + ks * TP_K_A, d_Whh + ks * TP_K_G, id128, 1);
      mma_bf16(tmem + TM_HN, d_h + ks * TP_K_A, d_Whh_n + ks * TP_K_G, id64, ks > 0);
    }
    mma_bf16(tmem + TM_HN, d_oh, d_Bhn, id64, 1);
    mma_bf16(tmem + qcol, d_oh, d_W2b, idesc_bf16_f32(128, NQ), 0);
  }
  __syncwarp();
}

// PM (TpLayout::plain) 1: the word-by-word path of shapes whose observation rows are not 16-byte multiples; 1 and 2:
// availability blocks that may start anywhere inside a 16-byte unit of the input array.
// MODE 1, 2 (LIST): the call's rows are the environments of p.env_ids (a partial step); inputs, the last step's
// actions and the tiling follow the row, state, ring cursors, the draw's key and the trace follow the environment.
// MODE 2 (LAG, one step per launch): reward/done are the outcome of each environment's previous action: they complete
// the record at pos - 1 and may close the episode BEFORE this step's decision; nothing closes after it.
// MODE 3: MODE 0 for launches of a few steps, where the tile-to-tile transition is a large part of the time: the
// hidden-state rows then move coalesced through a scratch and the next tile's rows are prefetched into L2 (modes 1
// and 2 do the same).  Launches of many steps keep the shorter transition code: its footprint in the step loop's
// instruction stream and registers costs them more (1.2 %) than the transition saves.
template <int NQ, int PM, int MODE>
__global__ void __launch_bounds__(TP_THREADS, 1)
    actor_tcp_kernel(const __grid_constant__ ActorParams p, const __grid_constant__ TpLayout L) {
  constexpr bool LIST = MODE == 1 || MODE == 2, LAG = MODE == 2, FASTX = MODE != 0;
  extern __shared__ __align__(1024) uint8_t smem[];
  using namespace tc;
  TpBars* B = reinterpret_cast<TpBars*>(smem + L.off_bar);
  uint8_t* xb = smem + L.off_x;
  uint8_t* yb = smem + L.off_y;
  uint8_t* hb = smem + L.off_hb;
  uint8_t* oh = smem + L.off_oh;
  uint8_t* stage = smem + L.off_stage;
  uint8_t* tails = smem + L.off_tail;                                  // [2][ept][tail_bytes]
  uint2* sel_s = reinterpret_cast<uint2*>(smem + L.off_sel);          // [4][128]: availability mask, random pick or -1
  int32_t* la_s = reinterpret_cast<int32_t*>(smem + L.off_la);        // last action of every row
  int32_t* close_s = reinterpret_cast<int32_t*>(smem + L.off_close);  // [2][32]: the environment's episode ends with this step
  int32_t* closeany_s = reinterpret_cast<int32_t*>(smem + L.off_closeany);  // [16] per step: some episode of the tile ends with it
  int32_t* rowenv_s = reinterpret_cast<int32_t*>(smem + L.off_rowenv);  // environment (within its chunk) of a chunk row
  unsigned long long* dstp_s = reinterpret_cast<unsigned long long*>(smem + L.off_dstp);  // [16][32] record address per step, environment
  unsigned long long* tdst_s = reinterpret_cast<unsigned long long*>(smem + L.off_tdst);  // [32] tail addresses of the step being copied
  const float* tab_la = reinterpret_cast<const float*>(smem + L.off_tab_la);
  volatile uint32_t* abortf = &B->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = p.n, D = p.D, A = p.A, T = p.T;
  const uint32_t rec_bytes = p.rl.rec_bytes;
  const int NS = L.NS;
  const uint32_t tail_set = (uint32_t)L.ept * L.tail_bytes;
  // tail-relative field offsets
  const uint32_t t_q = p.rl.off_q - p.rl.off_action, t_reward = p.rl.off_reward - p.rl.off_action,
                 t_done = p.rl.off_done - p.rl.off_action;
  const int my_tiles = blockIdx.x < p.num_tiles ? (p.num_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (tid == 0) {
    for (int i = 0; i < TP_MAX_STAGES; ++i) {
      mbar_init(&B->full[i], 1);
      mbar_init(&B->cfree[i], 1);
      mbar_init(&B->sfree[i], 1);
    }
    mbar_init(&B->xready, TP_CONV / 32);
    mbar_init(&B->fc1d, 1);
    mbar_init(&B->yready, 8);
    mbar_init(&B->grud, 1);
    mbar_init(&B->hready, 8);
    mbar_init(&B->fc2d, 1);
    mbar_init(&B->stepd, 8);
    mbar_init(&B->tiled, 8);
    mbar_init(&B->wload, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&B->selready[i], TP_CONV / 32);
    mbar_init(&B->flags, 1);
    B->abort = 0;
    mbar_init_fence();
  }
  if (warp == 12) tmem_alloc(&B->tmem_base, TM_COLS);
  // operands, tails and hand-off arrays start as zeros (padding bytes of every stored record stay zero)
  for (uint32_t i = L.off_x / 16 + tid; i < L.off_bar / 16; i += TP_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  for (uint32_t i = L.off_rstage / 16 + tid; i < L.total / 16; i += TP_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
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
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(TP_REGS_SVC));
    if (warp == 12) {
      // =========================== MMA warp: lane 0 issues every tcgen05.mma ===========================
      const uint32_t sb = smem_u32(smem);
      const int total = my_tiles * T;
      uint32_t tl = 0;
      bool hside_issued = false;
      if (total > 0) {
        mbar_wait(&B->xready, 0, abortf);
        tp_issue_fc1(L, sb, tmem, lane, &B->fc1d);
      }
      for (int g = 0, s = 0; g < total; ++g) {
        const uint32_t par = (uint32_t)g & 1u;
        const uint32_t qcol = TM_Q + par * tp_qstride(NQ);  // Q accumulators alternate, so the next step's can be seeded early
        if (!hside_issued) {
          // hidden operand in place: the tile prologue's, or the previous step's with closed episodes cleared
          if (s == 0) {
            mbar_wait(&B->tiled, tl & 1, abortf);
            ++tl;
          } else {
            mbar_wait(&B->stepd, par ^ 1u, abortf);
          }
          tp_issue_hside<NQ>(L, sb, tmem, lane, qcol);
        }
        mbar_wait(&B->yready, par, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_y = smem_desc(sb + L.off_y, TC_LBO_A, 128), d_Wih = smem_desc(sb + L.off_Wih, TP_LBO_G, 128);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma_bf16(tmem + TM_R, d_y + ks * TP_K_A, d_Wih + ks * TP_K_G, idesc_bf16_f32(128, 192), 1);
          mma_commit(&B->grud);
        }
        __syncwarp();
        // fc1 of the next step (possibly the next tile's first): its accumulator is free since epilogue 1 of
        // this step has read it; issue it now if the operand is already converted, else after fc2
        bool pending = g + 1 < total;
        if (pending) {
          // one lane looks (lanes looking separately could disagree and split the warp's control flow)
          const uint32_t ready = __shfl_sync(0xFFFFFFFFu, lane == 0 ? (uint32_t)mbar_test_wait(&B->xready, par ^ 1u) : 0u, 0);
          if (ready) {
            tp_issue_fc1(L, sb, tmem, lane, &B->fc1d);
            pending = false;
          }
        }
        mbar_wait(&B->hready, par, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t d_h = smem_desc(sb + L.off_hb, TC_LBO_A, 128), d_W2 = smem_desc(sb + L.off_W2, NQ * 16, 128);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)  // part 0 holds the bias already; parts 1..3 start from zero
            mma_bf16(tmem + qcol + (NQ == 16 ? ks * NQ : 0), d_h + ks * TP_K_A, d_W2 + ks * ((2 * NQ * 16) >> 4), idesc_bf16_f32(128, NQ),
                     (NQ == 16 && ks > 0) ? 0 : 1);
          mma_commit(&B->fc2d);
        }
        __syncwarp();
        if (pending) {
          mbar_wait(&B->xready, par ^ 1u, abortf);
          tp_issue_fc1(L, sb, tmem, lane, &B->fc1d);
        }
        // The next step's h-side products need only the new hidden state, which is in place unless an episode
        // of this tile ends with this step (its rows are cleared after fc2): issue them now, off the critical
        // path, whenever the tile goes on and nothing closes.
        hside_issued = false;
        if (++s == T) {
          s = 0;
        } else {
          // (published by the load warp before this step's inputs were requested: ordered before the fc1 operand)
          if (closeany_s[g & (TP_DST_DEPTH - 1)] == 0) {
            tp_issue_hside<NQ>(L, sb, tmem, lane, TM_Q + (par ^ 1u) * tp_qstride(NQ));
            hside_issued = true;
          }
        }
      }
    } else if (warp == 13) {
      // =========================== load warp: staging ring in, record addresses ahead ===========================
      // Chunks are numbered q = 0, 1, ... over (tile, step, chunk of four environments); chunk q lives in
      // staging slot q % NS as [observations of its environments | their availability bytes].  Lane el follows
      // the ring cursor of environment el of the tile being loaded: the cursor sequence depends only on the done
      // flags, so it runs ahead of the network, and the record address of every (step, environment) is published
      // for the converters before the step's first chunk is requested.
      int tile = blockIdx.x;
      int32_t slot = 0, pos = 0, ok = 0;
      long long epc = 0;
      uint32_t done_next = 0;
      uint32_t q = 0, qslot = 0, qpar = 1, kstep = 0;  // chunk index, q % NS, parity of the slot's previous use, global step
      for (; tile < p.num_tiles; tile += gridDim.x) {
        const int ne = min(L.ept, p.M - tile * L.ept);
        const int nck = (ne + TP_G - 1) / TP_G;
        const int x = tile * L.ept + lane;  // row of the call
        const bool mine = lane < ne;
        const int e = (LIST && mine) ? __ldg(p.env_ids + x) : x;
        ok = 0;
        if (mine) {
          slot = p.slot[e];
          pos = p.pos[e];
          epc = p.ep_count[e];
          ok = (slot >= 0 && slot < p.E * p.S && pos >= 0 && pos < p.L + (LAG ? 1 : 0)) ? 1 : 0;
          done_next = p.done[x];
          if (LAG && ok && pos > 0 && (done_next || pos == p.L)) {  // the late outcome closes the episode first
            epc += 1;
            slot = e * p.S + (int)(epc % p.S);
            pos = 0;
          }
        }
        for (int s = 0; s < T; ++s, ++kstep) {
          unsigned long long rec = 0;
          int closes = 0;
          if (mine && ok) {
            rec = reinterpret_cast<unsigned long long>(p.ring + (size_t)slot * p.slot_stride + (size_t)pos * rec_bytes);
            if (!LAG && (done_next || pos + 1 == p.L)) {  // the cursor after this step
              closes = 1;
              epc += 1;
              slot = e * p.S + (int)(epc % p.S);
              pos = 0;
            } else {
              pos += 1;
            }
          }
          dstp_s[(kstep & (TP_DST_DEPTH - 1)) * 32 + lane] = rec;
          closes = __any_sync(0xFFFFFFFFu, closes);
          if (lane == 0) closeany_s[kstep & (TP_DST_DEPTH - 1)] = closes;
          if (mine && s + 1 < T) done_next = p.done[(size_t)(s + 1) * p.env_step_stride + x];
          __syncwarp();
          for (int c = 0; c < nck; ++c) {
            const int ge = min(TP_G, ne - c * TP_G);
            if (q >= (uint32_t)NS) {  // the slot's previous chunk is converted and its observations are stored
              mbar_wait(&B->cfree[qslot], qpar, abortf);
              mbar_wait(&B->sfree[qslot], qpar, abortf);
            }
            const size_t env0 = (size_t)tile * L.ept + (size_t)(c * TP_G);
            // availability bytes of the chunk: [a0, a0 + ge n A) of the input array; plain shapes load the 16-byte
            // aligned range around them (inside the array: the launcher checks that the step's block ends aligned)
            const size_t a0 = (size_t)s * p.avail_step_stride + env0 * (size_t)(n * A);
            const size_t b0 = PM != 0 ? a0 & ~(size_t)15 : a0;
            const uint32_t av_load = PM != 0 ? (uint32_t)(((a0 + (size_t)ge * L.av_bytes + 15) & ~(size_t)15) - b0) : (uint32_t)ge * L.av_bytes;
            if (lane == 0) mbar_arrive_expect_tx(&B->full[qslot], (uint32_t)ge * L.obs_bytes + av_load);
            __syncwarp();
            uint8_t* dst = stage + qslot * L.chunk_bytes;
            if (lane == 0)
              bulk_load(dst, p.obs + (size_t)s * p.obs_step_stride + env0 * (size_t)(n * D), (uint32_t)ge * L.obs_bytes,
                        &B->full[qslot]);
            if (lane == 1) bulk_load(dst + TP_G * L.obs_bytes, p.avail + b0, av_load, &B->full[qslot]);
            ++q;
            if (++qslot == (uint32_t)NS) {
              qslot = 0;
              qpar ^= 1u;
            }
          }
        }
      }
    } else if (warp == 14) {
      // =========================== tail warp: cursors, slot headers, record tails (lane = environment) ===========
      unsigned long long c_episodes = 0, c_trunc = 0;
      uint32_t st_bits = 0, sd = 0, it = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        const int ne = min(L.ept, p.M - tile * L.ept);
        const bool mine = lane < ne;
        const int x = tile * L.ept + lane;  // row of the call
        const int e = (LIST && mine) ? __ldg(p.env_ids + x) : x;
        int32_t slot = 0, pos = 0, ok = 0;
        long long epc = 0;
        float reward_next = 0.f;
        uint32_t done_next = 0;
        if (mine) {
          slot = p.slot[e];
          pos = p.pos[e];
          epc = p.ep_count[e];
          ok = (slot >= 0 && slot < p.E * p.S && pos >= 0 && pos < p.L + (LAG ? 1 : 0)) ? 1 : 0;
          if (!ok) st_bits |= MARL_STATUS_BAD_INDEX;
          reward_next = p.reward[x];
          done_next = p.done[x];
          if (LAG) {
            if (ok && pos > 0) {  // the outcome of the previous action completes its record and may close the episode
              uint8_t* prev = p.ring + (size_t)slot * p.slot_stride + (size_t)(pos - 1) * rec_bytes;
              *reinterpret_cast<float*>(prev + p.rl.off_reward) = reward_next;
              prev[p.rl.off_done] = done_next ? 1 : 0;
              if (done_next || pos == p.L) {
                p.slot_len[slot] = pos;
                p.slot_complete[slot] = 1;
                c_episodes += 1;
                if (!done_next) c_trunc += 1;
                epc += 1;
                slot = e * p.S + (int)(epc % p.S);
                pos = 0;
              }
            }
            reward_next = 0.f;  // this step's own outcome is not known yet
            done_next = 0;
          }
        }
        // Copies the tails of one step (buffer bb, record addresses in tdst_s) to the ring: 16 bytes per lane, the
        // pieces of all environments in one flat loop.
        auto copy_tails = [&](uint32_t bb) {
          __syncwarp();
          const uint32_t pieces = L.tail_bytes / 16u, total = (uint32_t)ne * pieces;
          const uint32_t inv = 0xFFFFFFFFu / pieces + 1u;  // idx / pieces == umulhi(idx, inv) for idx < 2^16
          for (uint32_t idx = lane; idx < total; idx += 32) {
            const uint32_t env = __umulhi(idx, inv), pc = idx - env * pieces;
            const unsigned long long d = tdst_s[env];
            if (d) reinterpret_cast<uint4*>(d)[pc] = reinterpret_cast<const uint4*>(tails + bb * tail_set + env * L.tail_bytes)[pc];
          }
          __syncwarp();
        };
        for (int s = 0; s < T; ++s) {
          const uint32_t b = it & 1;
          const float reward = reward_next;
          const int done = done_next ? 1 : 0;
          const int close = (!LAG && ok && (done || pos + 1 == p.L)) ? 1 : 0;
          uint8_t* tl = tails + b * tail_set + (uint32_t)lane * L.tail_bytes;
          unsigned long long dst = 0;
          close_s[b * 32 + lane] = close;
          if (mine && ok) {
            dst = reinterpret_cast<unsigned long long>(p.ring + (size_t)slot * p.slot_stride + (size_t)pos * rec_bytes + p.rl.off_action);
            if (pos == 0) {  // an episode opens in this slot
              p.slot_epid[slot] = epc * (long long)p.E + e;
              p.slot_len[slot] = 0;
              p.slot_complete[slot] = 0;
            }
            *reinterpret_cast<float*>(tl + t_reward) = reward;
            tl[t_done] = (uint8_t)done;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&B->flags);  // first: epilogue 3 of this step waits for it
          if (s > 0) copy_tails(b ^ 1u);           // then the previous step's tails, off the critical path
          if (mine && s + 1 < T) {
            reward_next = p.reward[(size_t)(s + 1) * p.env_step_stride + x];
            done_next = p.done[(size_t)(s + 1) * p.env_step_stride + x];
          }
          mbar_wait(&B->stepd, sd & 1, abortf);  // action and Q of step s are in the tail
          ++sd;
          tdst_s[lane] = dst;
          if (close) {
            p.slot_len[slot] = pos + 1;
            p.slot_complete[slot] = 1;
            c_episodes += 1;
            if (!done) c_trunc += 1;
            epc += 1;
            slot = e * p.S + (int)(epc % p.S);
            pos = 0;
          } else if (mine && ok) {
            pos += 1;
          }
          ++it;
        }
        copy_tails((it - 1) & 1);  // the tile's last step
        if (mine && ok) {
          p.slot[e] = slot;
          p.pos[e] = pos;
          p.ep_count[e] = epc;
          if (pos > 0) p.slot_len[slot] = pos;
        }
      }
      if (c_episodes) atomicAdd(p.counters + CNT_EPISODES, c_episodes);
      if (c_trunc) atomicAdd(p.counters + CNT_TRUNCATED, c_trunc);
      if (st_bits) atomicOr(p.status, st_bits);
    } else {
      // =========================== store warp: observations from staging to the ring records ===========================
      // One bulk store per environment (its observation block is contiguous both in staging and in its record),
      // issued as soon as the chunk has arrived; a slot is handed back once its stores have been read out.
      uint32_t q = 0, qslot = 0, qpar = 0, pslot = 0, kstep = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        const int ne = min(L.ept, p.M - tile * L.ept);
        const int nck = (ne + TP_G - 1) / TP_G;
        for (int s = 0; s < T; ++s, ++kstep) {
          for (int c = 0; c < nck; ++c) {
            const int ge = min(TP_G, ne - c * TP_G);
            // plain shapes: the image the converters wrote, once they are done with the chunk; else the staged block
            mbar_wait(PM == 1 ? &B->cfree[qslot] : &B->full[qslot], qpar, abortf);
            if (lane < ge) {
              const unsigned long long rec = dstp_s[(kstep & (TP_DST_DEPTH - 1)) * 32 + c * TP_G + lane];
              const uint8_t* from = PM == 1 ? smem + L.off_rstage + qslot * L.rs_bytes + (uint32_t)lane * L.rs_env
                                            : stage + qslot * L.chunk_bytes + (uint32_t)lane * L.obs_bytes;
              if (rec) bulk_store(reinterpret_cast<void*>(rec), from, PM == 1 ? L.rs_env : L.obs_bytes);
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
        }
      }
      bulk_wait_read_all();
      __syncwarp();
      if (q > 0 && lane == 0) mbar_arrive(&B->sfree[pslot]);
      bulk_wait_all();
    }
  } else if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(TP_REGS_CONV));
    // =========================== converters: staged observations -> bf16 operand; masks and epsilon draws ==========
    // Each of the four warps takes whole chunks (chunk c of a step goes to warp c % 4), so a step's chunks are
    // converted side by side; thread ci then owns row ci of the tile for the epsilon draw.
    const int ci = tid - 256, cw = warp - 8;
    const int li = lane, ls = 32;
    const uint32_t inv_nchunk = 0xFFFFFFFFu / (uint32_t)L.nchunk + 1u;  // j / nchunk == umulhi(j, inv) for j < 2^16
    const uint32_t amask = A >= 32 ? 0xFFFFFFFFu : ((1u << A) - 1u);
    uint32_t it = 0, qbase = 0;  // steps and chunks before this step
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int e0 = tile * L.ept;
      const int ne = min(L.ept, p.M - e0);
      const int nck = (ne + TP_G - 1) / TP_G;
      for (int s = 0; s < T; ++s) {
        const uint32_t t = p.t0 + (uint32_t)s;
        const float eps = eps_at(p, t);
        uint2* sel = sel_s + (it & 3) * TC_ROWS;
        // the operand buffer is free once fc1 of the previous step has finished reading it
        if (it > 0) mbar_wait(&B->fc1d, (it - 1) & 1, abortf);
        for (int c = cw; c < nck; c += TP_CONV / 32) {
          const int ge = min(TP_G, ne - c * TP_G);
          const int Rc = ge * n;         // rows of this chunk
          const int r0 = c * TP_G * n;   // its first row in the tile
          const uint32_t q = qbase + (uint32_t)c, qslot = q % (uint32_t)NS, qpar = (q / (uint32_t)NS) & 1u;
          const uint8_t* src = stage + qslot * L.chunk_bytes;
          const unsigned long long* recs = dstp_s + (it & (TP_DST_DEPTH - 1)) * 32 + c * TP_G;  // this chunk's records
          mbar_wait(&B->full[qslot], qpar, abortf);
          const int items = Rc * L.nchunk;
          if (PM == 1) {
            // Rows are not 16-byte aligned: word by word, eight columns per item, to the operand and to the record
            // image.  Consecutive lanes take consecutive ROWS of one column group: a row stride of D words is odd for
            // most such shapes, so the lanes' words fall in different banks (lanes eight words apart would share four).
            const uint32_t inv_Rc = 0xFFFFFFFFu / (uint32_t)Rc + 1u;  // j / Rc == umulhi(j, inv) for j < 2^16
            for (int j = lane; j < items; j += 64) {  // two items per thread and pass: sixteen loads in flight
              float v[2][8];
              int cc[2], rr[2];
              bool on[2];
              float* drow[2];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int jj = j + 32 * u;
                on[u] = jj < items;
                cc[u] = on[u] ? (int)__umulhi((uint32_t)jj, inv_Rc) : 0;
                rr[u] = on[u] ? jj - cc[u] * Rc : 0;
                const int envc = rowenv_s[rr[u]];
                const float* srow = reinterpret_cast<const float*>(src) + rr[u] * D;
                drow[u] = reinterpret_cast<float*>(smem + L.off_rstage + qslot * L.rs_bytes + (uint32_t)envc * L.rs_env) + (rr[u] - envc * n) * D;
#pragma unroll
                for (int k = 0; k < 8; ++k) v[u][k] = (on[u] && cc[u] * 8 + k < D) ? srow[cc[u] * 8 + k] : 0.f;
              }
#pragma unroll
              for (int u = 0; u < 2; ++u) {  // (stores after all the loads: a store between them would order them one by one)
                if (on[u]) {
#pragma unroll
                  for (int k = 0; k < 8; ++k)
                    if (cc[u] * 8 + k < D) drow[u][cc[u] * 8 + k] = v[u][k];
                  *reinterpret_cast<uint4*>(xb + (uint32_t)cc[u] * TC_LBO_X + (uint32_t)(r0 + rr[u]) * 16u) =
                      make_uint4(pack_bf16x2(v[u][0], v[u][1]), pack_bf16x2(v[u][2], v[u][3]), pack_bf16x2(v[u][4], v[u][5]),
                                 pack_bf16x2(v[u][6], v[u][7]));
                }
              }
            }
          } else
          for (int j = lane; j < items; j += 64) {
            float4 v[2][2];
            int rr[2], cc[2];
            bool on[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const int jj = j + 32 * u;
              rr[u] = (int)__umulhi((uint32_t)jj, inv_nchunk);
              cc[u] = jj - rr[u] * L.nchunk;
              on[u] = jj < items;
              v[u][0] = v[u][1] = make_float4(0.f, 0.f, 0.f, 0.f);
              if (on[u] && cc[u] * 8 < D) {
                const uint32_t off = (uint32_t)(rr[u] * D) * 4u + (uint32_t)cc[u] * 32u;  // rows of a chunk are contiguous
                const float4* s4 = reinterpret_cast<const float4*>(src + off);
                v[u][0] = s4[0];
                v[u][1] = s4[1];
              }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              if (on[u]) {
                const uint4 o = make_uint4(pack_bf16x2(v[u][0].x, v[u][0].y), pack_bf16x2(v[u][0].z, v[u][0].w),
                                           pack_bf16x2(v[u][1].x, v[u][1].y), pack_bf16x2(v[u][1].z, v[u][1].w));
                *reinterpret_cast<uint4*>(xb + (uint32_t)cc[u] * TC_LBO_X + (uint32_t)(r0 + rr[u]) * 16u) = o;
              }
            }
          }
          // the chunk's availability bytes, rows contiguous; plain shapes: from byte `shift` of the loaded range
          const uint8_t* avs = src + TP_G * L.obs_bytes;
          const uint32_t shift = PM != 0 ? (uint32_t)(((size_t)(e0 + c * TP_G) * (size_t)(n * A)) & 15u) : 0u;
          if (PM != 0) {
            // To the record images (1) or straight to the records (2): word j of an environment's block is put
            // together from the two loaded words that hold its bytes; bytes beyond the block stay zero (padding of
            // the record).
            const uint32_t per_env = (L.av_bytes + 3u) / 4u;
            const uint32_t inv = 0xFFFFFFFFu / per_env + 1u;  // idx / per_env == umulhi(idx, inv) for idx < 2^16
            uint8_t* img = smem + L.off_rstage + qslot * L.rs_bytes + p.rl.off_avail;
            for (uint32_t i = li; i < (uint32_t)ge * per_env; i += ls) {
              const uint32_t envc = __umulhi(i, inv), j = i - envc * per_env;
              const uint32_t sb = shift + envc * L.av_bytes + 4u * j;  // first source byte of the word
              const uint32_t* w = reinterpret_cast<const uint32_t*>(avs + (sb & ~3u));
              uint32_t v = __funnelshift_r(w[0], w[1], 8u * (sb & 3u));
              const uint32_t left = L.av_bytes - 4u * j;  // bytes of the block from this word on
              if (left < 4u) v &= (1u << (8u * left)) - 1u;
              if (PM == 1) {
                reinterpret_cast<uint32_t*>(img + envc * L.rs_env)[j] = v;
              } else {
                const unsigned long long rec = recs[envc];
                if (rec) reinterpret_cast<uint32_t*>(rec + p.rl.off_avail)[j] = v;
              }
            }
          } else {
            const uint32_t per_env = L.av_bytes / 16u;
            for (uint32_t i = lane; i < (uint32_t)ge * per_env; i += 32) {
              const uint32_t envc = i / per_env;
              const unsigned long long rec = recs[envc];
              if (rec) reinterpret_cast<uint4*>(rec + L.obs_bytes)[i - envc * per_env] = reinterpret_cast<const uint4*>(avs)[i];
            }
          }
          // Availability masks of the chunk's rows.  A row's A bytes are read as aligned words (a few bytes beyond
          // the row are read and masked off) and each word's four "byte is non-zero" flags are gathered with one
          // multiply: short code, few loads.
          for (int rc = li; rc < Rc; rc += ls) {
            const uint32_t off = shift + (uint32_t)(rc * A);
            const uint32_t* w = reinterpret_cast<const uint32_t*>(avs + (off & ~3u));
            unsigned long long bits = 0;
#pragma unroll
            for (int k = 0; k < (NQ == 16 ? 5 : 9); ++k) {
              const uint32_t v = w[k];
              const uint32_t nz = ((v | ((v & 0x7F7F7F7Fu) + 0x7F7F7F7Fu)) & 0x80808080u) >> 7;  // 0x01 per non-zero byte
              bits |= (unsigned long long)((nz * 0x01020408u) >> 24 & 0xFu) << (4 * k);
            }
            sel[r0 + rc].x = (uint32_t)(bits >> (off & 3u)) & amask;
          }
          if (PM == 1) fence_proxy_async_smem();  // the record image is read by the store warp's bulk stores
          __syncwarp();
          if (lane == 0) mbar_arrive(&B->cfree[qslot]);
        }
        qbase += (uint32_t)nck;
        fence_proxy_async_smem();
        warp_arrive(&B->xready, lane);
        asm volatile("bar.sync 2, 128;" ::: "memory");  // the masks were written by the chunks' warps
        if (ci < ne * n) {
          const int rel = ci / n, rai = ci - rel * n;
          const uint32_t mask = sel[ci].x;
          int pick = -1;
          if (mask != 0)
            pick = draw_explore(mask, eps, p.seed, t, (uint32_t)(LIST ? __ldg(p.env_ids + e0 + rel) : e0 + rel), (uint32_t)rai);
          sel[ci].y = (uint32_t)pick;
        }
        warp_arrive(&B->selready[it & 3], lane);
        ++it;
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(TP_REGS_EPI));
    // =========================== epilogue threads ===========================
    const int row = tid & 127, half = tid >> 7;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int el = row / n, ai = row - el * n;
    const int cb = half * 32;  // first hidden column of this thread
    unsigned long long c_steps = 0, c_explore = 0, c_noavail = 0;
    uint32_t st_bits = 0, it = 0;
    float h[32];
    // this thread's half (32 floats) of tile row r's hidden state in global memory
    auto h_row = [&](int e0, int r) -> float* {
      if (!LIST) return p.h + ((size_t)e0 * n + (size_t)r) * TC_H + cb;  // a tile's rows are contiguous
      const int rel = rowenv_s[r];  // r / n
      const int env = __ldg(p.env_ids + e0 + rel);
      return p.h + ((size_t)env * n + (size_t)(r - rel * n)) * TC_H + cb;
    };

    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int e0 = tile * L.ept;
      const int ne = min(L.ept, p.M - e0);
      const int R = ne * n;
      const bool live = row < R;
      const bool is_row = live && half == 0;  // owner of the row's choice
      const int e = (LIST && live) ? __ldg(p.env_ids + e0 + el) : e0 + el;
      const size_t grow = (size_t)e * n + ai;  // global row
      int la = -1;

      // ---- tile prologue: hidden state and last actions from global memory ----
      {
        bool carry = live;  // the row continues an episode
        if (LAG && live) {  // ... unless the late outcome has just ended it
          const int ps = p.pos[e];
          if (ps > 0 && (p.done[e0 + el] || ps == p.L)) carry = false;
        }
        const int la_mem = (carry && half == 0) ? p.last_action[grow] : -1;  // in flight beside the rows below
        // A thread owns 128 bytes of its row, so a warp reading "its own" pieces would touch 32 lines per
        // instruction.  The rows go through a warp-private 2 KB scratch instead (the y operand buffer, idle
        // between tiles): eight lanes fetch one row's 128 bytes, the scratch's piece index is xor-ed with the row so
        // that neither side has bank conflicts, and each thread then takes its row, 16 rows per pass.
        if constexpr (FASTX) {
          uint4* sw = reinterpret_cast<uint4*>(yb) + warp * 128;  // this warp's scratch
          const int wrow0 = (warp & 3) * 32;                      // first tile row of this warp
          uint4 f[2][4];
#pragma unroll
          for (int ps = 0; ps < 2; ++ps)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int r = wrow0 + ps * 16 + 4 * j + (lane >> 3);
              f[ps][j] = make_uint4(0u, 0u, 0u, 0u);
              if (r < R) f[ps][j] = __ldg(reinterpret_cast<const uint4*>(h_row(e0, r)) + (lane & 7));
            }
#pragma unroll
          for (int ps = 0; ps < 2; ++ps) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int rl = 4 * j + (lane >> 3);
              sw[rl * 8 + ((lane & 7) ^ (rl & 7))] = f[ps][j];
            }
            __syncwarp();
            if ((lane >> 4) == ps) {
              const int rl = lane & 15;
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                const uint4 v = sw[rl * 8 + (q ^ (rl & 7))];
                h[4 * q] = __uint_as_float(v.x); h[4 * q + 1] = __uint_as_float(v.y);
                h[4 * q + 2] = __uint_as_float(v.z); h[4 * q + 3] = __uint_as_float(v.w);
              }
            }
            __syncwarp();
          }
          if (!carry) {
#pragma unroll
            for (int q = 0; q < 32; ++q) h[q] = 0.f;
          }
        } else {
          const float4* src = reinterpret_cast<const float4*>(p.h + grow * TC_H + cb);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 v = carry ? src[q] : make_float4(0.f, 0.f, 0.f, 0.f);
            h[4 * q] = v.x; h[4 * q + 1] = v.y; h[4 * q + 2] = v.z; h[4 * q + 3] = v.w;
          }
        }
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const uint4 o = make_uint4(pack_bf16x2(h[8 * cc], h[8 * cc + 1]), pack_bf16x2(h[8 * cc + 2], h[8 * cc + 3]),
                                     pack_bf16x2(h[8 * cc + 4], h[8 * cc + 5]), pack_bf16x2(h[8 * cc + 6], h[8 * cc + 7]));
          *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
        }
        if (half == 0) {
          la = la_mem;
          if (la >= A) la = -1;
          la_s[row] = la;
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        asm volatile("bar.sync 1, 256;" ::: "memory");  // la_s is read by both threads of a row
        warp_arrive(&B->tiled, lane);
        // The next tile's hidden state is a first touch of its lines (and often of its page): ask for it now, one
        // line per thread, so that the next prologue finds it in L2.
        const int tile_n = tile + (int)gridDim.x;
        if (FASTX && tile_n < p.num_tiles) {
          const int e0n = tile_n * L.ept;
          if (row < min(L.ept, p.M - e0n) * n) {
            const float* nx = h_row(e0n, row);
            asm volatile("prefetch.global.L2 [%0];" ::"l"(nx));
            if (half == 0 && ai == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.last_action + (nx - cb - p.h) / TC_H));
          }
        }
      }

      for (int s = 0; s < T; ++s) {
        const uint32_t b = it & 1, par = it & 1;
        uint8_t* tl = tails + b * tail_set + (uint32_t)el * L.tail_bytes;  // this row's environment tail

        // ---- epilogue 1: y = relu(fc1 + W1[:, last action]) -> bf16 operand.  Bias and agent-id column are
        //      inside the GEMM; fc1 itself finished during the previous step. ----
        mbar_wait(&B->fc1d, par, abortf);
        tc_fence_after_sync();
        {
          // an episode that just ended has no last action
          int last = (s > 0 && close_s[(b ^ 1u) * 32 + el]) ? -1 : la_s[row];
          const float* tlr = tab_la + (last >= 0 ? last : 0) * TC_TAB + cb;
          // both halves of the thread's 32 columns are requested before the one wait
          uint32_t v2[2][16];
          tmem_ld16(tmem + lane_addr + TM_FC1 + cb, v2[0]);
          tmem_ld16(tmem + lane_addr + TM_FC1 + cb + 16, v2[1]);
          tmem_ld_wait();
#pragma unroll
          for (int c16 = 0; c16 < 2; ++c16) {
            uint32_t(&v)[16] = v2[c16];
            float y[16];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float4 l4 = make_float4(0.f, 0.f, 0.f, 0.f);
              if (last >= 0) l4 = *reinterpret_cast<const float4*>(tlr + c16 * 16 + 4 * q);
              y[4 * q] = fmaxf(__uint_as_float(v[4 * q]) + l4.x, 0.f);
              y[4 * q + 1] = fmaxf(__uint_as_float(v[4 * q + 1]) + l4.y, 0.f);
              y[4 * q + 2] = fmaxf(__uint_as_float(v[4 * q + 2]) + l4.z, 0.f);
              y[4 * q + 3] = fmaxf(__uint_as_float(v[4 * q + 3]) + l4.w, 0.f);
            }
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              const uint4 o = make_uint4(pack_bf16x2(y[8 * cc], y[8 * cc + 1]), pack_bf16x2(y[8 * cc + 2], y[8 * cc + 3]),
                                         pack_bf16x2(y[8 * cc + 4], y[8 * cc + 5]), pack_bf16x2(y[8 * cc + 6], y[8 * cc + 7]));
              *reinterpret_cast<uint4*>(yb + (uint32_t)(half * 4 + c16 * 2 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
            }
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        warp_arrive(&B->yready, lane);

        // ---- epilogue 2: gate math, new hidden state (fp32 registers) and its bf16 operand.
        //      The r and z accumulators hold half the pre-activation: sigmoid(v) = 0.5 * tanh(v / 2) + 0.5 ----
        mbar_wait(&B->grud, par, abortf);
        tc_fence_after_sync();
        {
          // Eight columns at a time; the accumulators of the next eight are requested before the gate math of the
          // current ones (tcgen05.wait::ld waits for every load in flight, so the request follows the wait).
          uint32_t g[2][4][8];  // [buffer][r, z, candidate-input, candidate-hidden][column]
          auto request = [&](int c8, uint32_t (&d)[4][8]) {
            const uint32_t col = (uint32_t)(cb + c8 * 8);
            tmem_ld8(tmem + lane_addr + TM_R + col, d[0]);
            tmem_ld8(tmem + lane_addr + TM_Z + col, d[1]);
            tmem_ld8(tmem + lane_addr + TM_IN + col, d[2]);
            tmem_ld8(tmem + lane_addr + TM_HN + col, d[3]);
          };
          request(0, g[0]);
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            tmem_ld_wait();
            if (c8 + 1 < 4) request(c8 + 1, g[(c8 + 1) & 1]);
            uint32_t(&v)[4][8] = g[c8 & 1];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float rg = fmaf(0.5f, tanh_fast(__uint_as_float(v[0][j])), 0.5f);
              const float zg = fmaf(0.5f, tanh_fast(__uint_as_float(v[1][j])), 0.5f);
              const float cand = tanh_fast(fmaf(rg, __uint_as_float(v[3][j]), __uint_as_float(v[2][j])));
              const float hp = h[c8 * 8 + j];
              h[c8 * 8 + j] = fmaf(zg, hp - cand, cand);  // (1 - z) * cand + z * h
            }
            const float* hv = h + c8 * 8;
            const uint4 o = make_uint4(pack_bf16x2(hv[0], hv[1]), pack_bf16x2(hv[2], hv[3]), pack_bf16x2(hv[4], hv[5]),
                                       pack_bf16x2(hv[6], hv[7]));
            *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 4 + c8) * TC_LBO_A + (uint32_t)row * 16u) = o;
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        warp_arrive(&B->hready, lane);

        // ---- epilogue 3: the row owners choose and complete the record's tail ----
        mbar_wait(&B->flags, par, abortf);  // close flags of this step written, tail buffer free
        mbar_wait(&B->fc2d, par, abortf);   // (both halves: the hidden operand may be cleared below)
        tc_fence_after_sync();
        if (half == 0) {
          uint32_t qv[NQ];
          const uint32_t qcol = TM_Q + par * tp_qstride(NQ);
          tmem_ld16(tmem + lane_addr + qcol, *reinterpret_cast<uint32_t(*)[16]>(qv));
          if (NQ == 32) tmem_ld16(tmem + lane_addr + qcol + 16, *reinterpret_cast<uint32_t(*)[16]>(qv + NQ - 16));
          if (NQ == 16) {  // the four K-step parts: (bias + part 0) + part 1 + part 2 + part 3
            uint32_t q1[16], q2[16], q3[16];
            tmem_ld16(tmem + lane_addr + qcol + 16, q1);
            tmem_ld16(tmem + lane_addr + qcol + 32, q2);
            tmem_ld16(tmem + lane_addr + qcol + 48, q3);
            tmem_ld_wait();
#pragma unroll
            for (int a = 0; a < 16; ++a)
              qv[a] = __float_as_uint((__uint_as_float(qv[a]) + __uint_as_float(q1[a])) + (__uint_as_float(q2[a]) + __uint_as_float(q3[a])));
          }
          tmem_ld_wait();
          tc_fence_before_sync();
          if (is_row) {
            mbar_wait(&B->selready[it & 3], (it >> 2) & 1, abortf);
            const uint2 sp = sel_s[(it & 3) * TC_ROWS + row];
            const uint32_t mask = sp.x;
            const int pick = (int)sp.y;
            // greedy rule on registers: m = max over available, thr = m - 1e-4f, lowest available a with Q >= thr.
            // Unavailable (and padding) entries become -inf; NaN never compares greater or equal; fmaxf ignores
            // a NaN operand, like the "greater than" scan it replaces.
            float qm[NQ];
#pragma unroll
            for (int a = 0; a < NQ; ++a) qm[a] = ((mask >> a) & 1u) ? __uint_as_float(qv[a]) : -INFINITY;
            float red[NQ];
#pragma unroll
            for (int a = 0; a < NQ; ++a) red[a] = qm[a];
#pragma unroll
            for (int w = NQ / 2; w >= 1; w >>= 1)
#pragma unroll
              for (int a = 0; a < w; ++a) red[a] = fmaxf(red[a], red[a + w]);
            const float thr = __fsub_rn(red[0], 1e-4f);
            uint32_t ge = 0;
#pragma unroll
            for (int a = 0; a < NQ; ++a) ge |= (qm[a] >= thr ? 1u : 0u) << a;
            ge &= mask;
            const int g = ge ? __ffs(ge) - 1 : __ffs(mask) - 1;
            const int act = mask == 0 ? 0 : (pick >= 0 ? pick : g);
            c_steps += 1;
            c_explore += pick >= 0 ? 1u : 0u;
            if (mask == 0) { c_noavail += 1; st_bits |= MARL_STATUS_NO_AVAIL; }
            la = act;
            la_s[row] = act;  // read by both threads of the row in the next step's epilogue 1
            float* qrow = reinterpret_cast<float*>(tl + t_q) + ai * A;
            if ((A & 1) == 0) {  // rows of an even number of floats start on 8-byte boundaries
#pragma unroll
              for (int a = 0; a < NQ; a += 2)
                if (a < A) *reinterpret_cast<float2*>(qrow + a) = make_float2(__uint_as_float(qv[a]), __uint_as_float(qv[a + 1]));
            } else {
#pragma unroll
              for (int a = 0; a < NQ; ++a)
                if (a < A) qrow[a] = __uint_as_float(qv[a]);
            }
            reinterpret_cast<int32_t*>(tl)[ai] = act;
            const int tk = p.trace_first + s;
            if (tk < p.trace_cap) {
              const size_t trow = ((size_t)tk * p.E + e) * n + ai;
              if (p.trace_actions) p.trace_actions[trow] = act;
              if (p.trace_q) {
#pragma unroll
                for (int a = 0; a < NQ; ++a)  // unrolled: a run-time index would put the Q registers in local memory
                  if (a < A) p.trace_q[trow * A + a] = __uint_as_float(qv[a]);
              }
            }
            if (p.actions_out && s == T - 1) p.actions_out[LIST ? (size_t)(e0 + el) * n + ai : grow] = act;
          }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // ---- a closed episode restarts from a zero hidden state and no last action ----
        if (live && close_s[b * 32 + el]) {
#pragma unroll
          for (int j = 0; j < 32; ++j) h[j] = 0.f;
#pragma unroll
          for (int cc = 0; cc < 4; ++cc)
            *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) = make_uint4(0, 0, 0, 0);
          if (half == 0) la = -1;
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        warp_arrive(&B->stepd, lane);
        ++it;
      }

      // ---- tile epilogue: state back to global memory ----
      if (is_row) p.last_action[grow] = la;
      if constexpr (FASTX) {
        uint4* sw = reinterpret_cast<uint4*>(yb) + warp * 128;
        const int wrow0 = (warp & 3) * 32;
#pragma unroll
      for (int ps = 0; ps < 2; ++ps) {  // the rows leave through the same scratch, coalesced
        if ((lane >> 4) == ps) {
          const int rl = lane & 15;
#pragma unroll
          for (int q = 0; q < 8; ++q)
            sw[rl * 8 + (q ^ (rl & 7))] = make_uint4(__float_as_uint(h[4 * q]), __float_as_uint(h[4 * q + 1]),
                                                     __float_as_uint(h[4 * q + 2]), __float_as_uint(h[4 * q + 3]));
        }
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int rl = 4 * j + (lane >> 3), r = wrow0 + ps * 16 + rl;
          if (r < R) reinterpret_cast<uint4*>(h_row(e0, r))[lane & 7] = sw[rl * 8 + ((lane & 7) ^ (rl & 7))];
        }
        __syncwarp();
      }
      } else if (live) {
        float4* dsth = reinterpret_cast<float4*>(p.h + grow * TC_H + cb);
#pragma unroll
        for (int q = 0; q < 8; ++q) dsth[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");  // la_s is rewritten by the next tile's prologue
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
  if (warp == 12) tmem_dealloc(tmem, TM_COLS);
}

// Returns the number of kernels launched, 0 if this launch's pointers do not meet the kernel's alignment
// needs (the caller then uses the one-tile kernel), or a negative cudaError.
int launch_actor_tcp(const ActorParams& p_in, int sms, cudaStream_t stream) {
  const TpLayout L = tp_layout(p_in.n, p_in.D, p_in.A, (int)p_in.rl.rec_bytes, p_in.M, sms);
  ActorParams p = p_in;
  p.ept = L.ept;  // (tiles of whole chunks for the plain shapes)
  p.num_tiles = (p.M + L.ept - 1) / L.ept;
  if (reinterpret_cast<uintptr_t>(p.obs) % 16 || reinterpret_cast<uintptr_t>(p.avail) % 16) return 0;
  if ((p.obs_step_stride * 4) % 16 || p.avail_step_stride % 16) return 0;
  // plain shapes: a last chunk of fewer environments would not be a 16-byte multiple, and the aligned range around
  // the last chunk's availability bytes must end inside the step's block
  if (L.plain == 1 && p.M % TP_G != 0) return 0;
  if (L.plain != 0 && ((size_t)p.M * p.n * p.A) % 16 != 0) return 0;
  const int mode = p.env_ids == nullptr ? (p.T < 8 ? 3 : 0) : (p.lagged ? 2 : 1);
  if (p.lagged && (mode != 2 || p.T != 1)) return 0;  // late outcomes: one step per launch over a list
  auto pick = [&](auto nq) {
    constexpr int Q = decltype(nq)::value;
    auto of_mode = [&](auto md) {
      constexpr int MD = decltype(md)::value;
      return L.plain == 1 ? actor_tcp_kernel<Q, 1, MD> : L.plain == 2 ? actor_tcp_kernel<Q, 2, MD> : actor_tcp_kernel<Q, 0, MD>;
    };
    return mode == 3 ? of_mode(std::integral_constant<int, 3>()) : mode == 2 ? of_mode(std::integral_constant<int, 2>())
         : mode == 1 ? of_mode(std::integral_constant<int, 1>()) : of_mode(std::integral_constant<int, 0>());
  };
  auto kernel = L.NQ == 16 ? pick(std::integral_constant<int, 16>()) : pick(std::integral_constant<int, 32>());
  static uint32_t configured[24][SMEM_OPTIN_DEVICES];
  {
    const cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L.total,
                                              configured[(L.NQ == 16 ? 0 : 1) + 2 * L.plain + 6 * mode]);
    if (e != cudaSuccess) return -(int)e;
  }
  int grid = p.num_tiles < sms ? p.num_tiles : sms;
  if (grid < 1) grid = 1;
  kernel<<<grid, TP_THREADS, L.total, stream>>>(p, L);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 1 : -(int)err;
}

}  // namespace marl
