// Tensor-core actor kernel for hidden size 128 on sm_100a: bf16 operands, weights streamed through shared memory.
//
// The worker's decision step (Algorithm 2) and the actor's recording (Algorithm 1) for a tile of whole environments
// - up to 128 agent rows - with all T steps of the launch run tile by tile (Sec. III-A: environments never exchange
// data), exactly as in the pipelined kernel for hidden size 64 (actor_tcp.cu), whose data movement this kernel
// keeps: a staging ring of four-environment chunks filled by bulk loads that run ahead of the network, converter
// warps that write the bf16 fc1 operand, the masks and the epsilon draws, a store warp for the observation part of
// the ring records, a tail warp for headers, counters and the [action | Q | reward, done] part.
//
// What hidden size 128 changes:
//   * The bf16 network is 228 KB and does not fit one SM's shared memory.  The bias tiles, the candidate rows of W_hh,
//     W2 and the last-action table (60 KB) are resident; W1, W_ih and the reset/update rows of W_hh (185 KB) are packed
//     in global memory as a sequence of slices (at most 12 KB each: one to three K = 16 steps of one matrix) in the
//     order the tensor core consumes them, and a loader warp streams them from L2 through a ring of shared-memory
//     slots, one bulk load per slice, as far ahead as the ring allows.  The thread that issues the MMAs waits for a
//     slice, issues the MMAs that read it and hands the slot back with a tcgen05.commit.  Order per step: h-side r|z
//     products, h-side candidate product, y-side products, fc2, fc1 of the next step.
//   * Four 128-column accumulators (reset, update, candidate-input, candidate-hidden) fill tensor memory, so the
//     fc1 accumulator lives in the candidate-input columns (issued once the gate math has read them) and Q in the
//     candidate-hidden columns (read before the next step's candidate-hidden product is issued).
//   * An epilogue thread owns one agent row and 64 hidden columns.
//
// Warp roles (512 threads): warps 0-7 epilogue, warps 8-10 converters, warp 11 weight loader, warp 12 issues every
// tcgen05.mma, warp 13 input loads and ring cursors ahead, warp 14 tails and headers, warp 15 observation stores.
// All hand-offs are mbarriers with bounded waits; an expired wait sets MARL_STATUS_TIMEOUT and lets the block run
// to its end with every index in range.
//
// Shapes taken: bf16, hidden 128, at most 16 actions, at least 4 agents, observation width a multiple of 8 and
// availability bytes per environment a multiple of 16 (rows that can be bulk-copied).  Dense launches only; steps
// over a list of environments and other shapes run on the CUDA-core kernel.
#include <cstring>

#include "actor_tc_layout.cuh"
#include "common.cuh"
#include "launch_util.cuh"
#include "tcgen05.cuh"

namespace marl {

constexpr int TW_H = 128;
constexpr int TW_THREADS = 512;
constexpr int TW_NCONV = 3;        // converter warps
constexpr int TW_G = 4;            // environments per staging chunk
constexpr int TW_MAX_STAGES = 8;
constexpr int TW_DST_DEPTH = 16;   // steps of record addresses kept
constexpr uint32_t TW_WSLOT = 12288;  // bytes of one slot of the weight ring
constexpr int TW_MAX_WSLOTS = 8;
constexpr int TW_MAX_SLICES = 48;
constexpr int TW_NQ = 16;          // Q columns (actions padded)
constexpr int TW_TAB = TW_H + 4;   // row stride (floats) of the last-action table: conflict-free float4 rows
// Register split (setmaxnreg): launched with 128 registers per thread; 256 * 176 + 128 * 80 + 128 * 80 = 65536.
constexpr int TW_REGS_EPI = 176, TW_REGS_CONV = 80, TW_REGS_SVC = 80;
// tensor-memory columns: the fc1 accumulator aliases IN, the four Q parts alias the first 64 columns of HN
constexpr uint32_t TW_R = 0, TW_Z = 128, TW_IN = 256, TW_HN = 384, TW_COLS = 512;

struct TwLayout {
  int32_t Dk, nchunk, ept, ohK, ohc, NS, NW, n_slices;
  int32_t ks_obs, ks_oh, nC, pad0, pad1, pad2;         // K-steps of fc1; slices of the fc1 group
  uint32_t slice_off[TW_MAX_SLICES];                  // byte offset of a slice inside the streamed image
  uint32_t slice_bytes[TW_MAX_SLICES];
  // packed weights in global memory: [resident image | streamed image]; the resident part has the same offsets in
  // shared memory
  uint32_t off_Brz, off_Bin, off_Bhn, off_Whn, off_W2, off_tab_la, rbytes, stream_off, wbytes;
  uint32_t prefix_bytes, tail_bytes, chunk_bytes, obs_bytes, av_bytes;
  uint32_t off_x, off_y, off_hb, off_oh, off_tail, off_sel, off_la, off_close, off_closeany, off_rowenv, off_dstp, off_tdst,
      off_bar, off_wring, off_stage, total;
};

struct TwBars {
  uint64_t full[TW_MAX_STAGES], cfree[TW_MAX_STAGES], sfree[TW_MAX_STAGES];  // chunk loaded / converted / stored
  uint64_t wfull[TW_MAX_WSLOTS], wfree[TW_MAX_WSLOTS];                       // weight slice arrived / read by its MMAs
  uint64_t xready, fc1d, yready, grud, hready, fc2d, stepd, wload, flags, tiled;
  uint64_t selready[4];
  uint32_t tmem_base, abort;
};

// Resident: the bias tiles, the candidate rows of W_hh (32 KB), W2 (4.5 KB) and the last-action table.  Streamed
// groups, in the order of use within a step (fc1 belongs to the NEXT step):
//   D  W_hh rows r|z   (256 rows, K = 128): one K-step (8192 B) per slice
//   A  W_ih all rows   (384 rows):          one K-step (12288 B) per slice
//   C  W1              (128 rows, K = Dk + ohK): three K-steps (12288 B) per slice
// The stream starts with C (fc1 of the first step), then D A C repeat: 185 KB per tile-step.  Every kilobyte of
// shared memory is worth the same whether it keeps weights resident (less to stream) or deepens the ring (more
// streamed while the gate math holds tensor memory): measured, the L2-to-SM stream runs at about 19 bytes per
// clock and SM whatever the ring depth (2, 3 or 4 slots: 4.20, 3.98, 3.95 ms per rollout at 16384 environments),
// so the ring is two slots and the rest holds weights.
static TwLayout tw_layout(int n, int D, int A, int rec_bytes) {
  TwLayout L;
  memset(&L, 0, sizeof(L));
  L.Dk = (D + 15) & ~15;
  L.nchunk = L.Dk / 8;
  L.ept = TC_ROWS / n;
  L.ohK = (3 + n + 15) & ~15;
  L.ohc = L.ohK / 8;
  L.ks_obs = L.Dk / 16;
  L.ks_oh = L.ohK / 16;
  // ---- packed weights ----
  uint32_t o = 0;
  L.off_Brz = o; o += 2u * 256 * 16;
  L.off_Bin = o; o += 2u * 128 * 16;
  L.off_Bhn = o; o += 2u * 128 * 16;
  L.off_Whn = o; o += 8u * 2 * 128 * 16;     // W_hh rows n (128 rows, K = 128): resident
  L.off_W2 = o; o += 9u * 2 * TW_NQ * 16;    // W2 and its bias step (16 rows, K = 144): resident
  L.off_tab_la = o; o += up16((uint32_t)sizeof(float) * A * TW_TAB);
  L.rbytes = o;
  L.stream_off = o;
  uint32_t so = 0;
  int ns = 0;
  auto add_group = [&](int ksteps, uint32_t kstep_bytes, int per_slice) {
    int count = 0;
    for (int k = 0; k < ksteps; k += per_slice) {
      const int take = ksteps - k < per_slice ? ksteps - k : per_slice;
      if (ns < TW_MAX_SLICES) {
        L.slice_off[ns] = so;
        L.slice_bytes[ns] = (uint32_t)take * kstep_bytes;
      }
      so += (uint32_t)take * kstep_bytes;
      ++ns;
      ++count;
    }
    return count;
  };
  L.nC = add_group(L.ks_obs + L.ks_oh, 2u * 128 * 16, 3);  // C
  add_group(8, 2u * 256 * 16, 1);                           // D
  add_group(8, 2u * 384 * 16, 1);                           // A
  L.n_slices = ns;
  L.wbytes = L.stream_off + so;
  // ---- shared memory ----
  L.obs_bytes = (uint32_t)(n * D) * 4u;
  L.av_bytes = (uint32_t)(n * A);
  L.prefix_bytes = L.obs_bytes + L.av_bytes;
  L.tail_bytes = (uint32_t)rec_bytes - (up16(L.obs_bytes) + up16(L.av_bytes));
  L.chunk_bytes = TW_G * L.prefix_bytes;
  o = L.rbytes;
  L.off_x = o; o += up16((uint32_t)L.nchunk * TC_LBO_X);
  L.off_y = o; o += 16 * TC_LBO_A;
  L.off_hb = o; o += 16 * TC_LBO_A;
  L.off_oh = o; o += (uint32_t)L.ohc * TC_LBO_A;
  L.off_tail = o; o += (uint32_t)L.ept * L.tail_bytes;
  L.off_sel = o; o += 4u * TC_ROWS * 8;
  L.off_la = o; o += TC_ROWS * 4;
  L.off_close = o; o += 2 * 32 * 4;
  L.off_closeany = o; o += TW_DST_DEPTH * 4;
  L.off_rowenv = o; o += TC_ROWS * 4;
  L.off_dstp = o; o += TW_DST_DEPTH * 32 * 8;
  L.off_tdst = o; o += 32 * 8;
  L.off_bar = o; o += (uint32_t)((sizeof(TwBars) + 15) & ~15u);
  // Two slots of weight ring; the staging ring takes what is left, up to one tile-step of chunks.  A staging ring
  // shorter than a tile-step must be a multiple of the converter warps, so that the warp that waits for a slot is the
  // one that converted the slot's previous chunk (a wait on "the other phase" reads as complete before that chunk
  // has even arrived).
  const int nck_max = (L.ept + TW_G - 1) / TW_G;
  const int nw = 2;
  const uint32_t fixed = o + (uint32_t)nw * TW_WSLOT + 32;  // (+32: the mask words read a few bytes past a row)
  int nstage = fixed < TC_SMEM_MAX ? (int)((TC_SMEM_MAX - fixed) / L.chunk_bytes) : 0;
  const int want = nck_max < 3 ? 3 : nck_max;  // a tile-step of chunks, at least three
  if (nstage > want) nstage = want;
  if (nstage > TW_MAX_STAGES) nstage = TW_MAX_STAGES;
  if (nstage < nck_max) nstage = nstage / TW_NCONV * TW_NCONV;
  L.NS = nstage;
  const uint32_t stage_bytes = (uint32_t)L.NS * L.chunk_bytes + 32;
  L.NW = nw;
  L.off_wring = o;
  L.off_stage = o + (uint32_t)nw * TW_WSLOT;
  L.total = L.off_stage + stage_bytes;
  return L;
}

bool tcw_supported(int n, int D, int A, int H, int prec) {
  if (prec != MARL_PRECISION_BF16 || H != TW_H) return false;
  if (D < 1 || D > 256 || D % 8 != 0 || n < 4 || n > 32 || A < 1 || A > TW_NQ) return false;
  if ((n * A) % 16 != 0) return false;  // an environment's availability bytes are bulk-copied and stored as 16-byte pieces
  const TwLayout L = tw_layout(n, D, A, rec_bytes_of(n, D, A));
  return L.ept >= TW_G && L.NS >= 2 && L.NW >= 2 && L.n_slices <= TW_MAX_SLICES && L.total <= TC_SMEM_MAX;
}

size_t tcw_wpack_bytes(int n, int D, int A) {
  if (D < 1 || D > 256 || n < 1 || n > 32 || A < 1 || A > TW_NQ) return 0;
  return tw_layout(n, D, A, rec_bytes_of(n, D, A)).wbytes;
}

static uint16_t tw_bf16_bits(float v) {
  uint32_t u;
  memcpy(&u, &v, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}
static float tw_bf16_value(float v) {
  const uint32_t u = (uint32_t)tw_bf16_bits(v) << 16;
  float o;
  memcpy(&o, &u, 4);
  return o;
}

// Packs the network for this kernel: every matrix as an N-row K-major operand (k-chunks of all rows contiguous),
// the streamed groups one after the other in the order of tw_layout.  Biases enter the GEMMs as three bf16 pieces
// at k = 0..2 of a bias K-step (multiplied by the three ones of the one-hot operand tile); the reset and update rows
// and their biases are stored halved (sigmoid(v) = 0.5 tanh(v / 2) + 0.5).
void tcw_pack_weights(int n, int D, int A, const float* W1, const float* b1, const float* Wih, const float* bih,
                      const float* Whh, const float* bhh, const float* W2, const float* b2, void* dst_host) {
  const TwLayout L = tw_layout(n, D, A, rec_bytes_of(n, D, A));
  const int H = TW_H, I = D + n + A;
  uint8_t* o = static_cast<uint8_t*>(dst_host);
  memset(o, 0, L.wbytes);
  auto put = [&](uint32_t base, int N, int row, int k, float v) {
    const uint16_t b = tw_bf16_bits(v);
    memcpy(o + base + (size_t)(k / 8) * N * 16 + (size_t)row * 16 + (k % 8) * 2, &b, 2);
  };
  auto put3 = [&](uint32_t base, int N, int row, int k0, float v) {
    const float p0 = tw_bf16_value(v), p1 = tw_bf16_value(v - p0), p2 = tw_bf16_value(v - p0 - p1);
    put(base, N, row, k0, p0);
    put(base, N, row, k0 + 1, p1);
    put(base, N, row, k0 + 2, p2);
  };
  // resident bias tiles and the last-action table
  for (int r = 0; r < 2 * H; ++r) put3(L.off_Brz, 2 * H, r, 0, 0.5f * (bih[r] + bhh[r]));
  for (int j = 0; j < H; ++j) {
    put3(L.off_Bin, H, j, 0, bih[2 * H + j]);
    put3(L.off_Bhn, H, j, 0, bhh[2 * H + j]);
  }
  float* tla = reinterpret_cast<float*>(o + L.off_tab_la);
  for (int a = 0; a < A; ++a)
    for (int j = 0; j < H; ++j) tla[a * TW_TAB + j] = tw_bf16_value(W1[(size_t)j * I + D + n + a]);
  // streamed groups
  uint32_t g = L.stream_off;
  const uint32_t gC = g; g += (uint32_t)(L.ks_obs + L.ks_oh) * 2u * 128 * 16;
  const uint32_t gD = g; g += 8u * 2 * 256 * 16;
  const uint32_t gA = g;
  const uint32_t gE = L.off_Whn, gB = L.off_W2;  // resident
  for (int j = 0; j < H; ++j) {
    for (int k = 0; k < D; ++k) put(gC, H, j, k, W1[(size_t)j * I + k]);
    put3(gC, H, j, L.Dk, b1[j]);
    for (int i = 0; i < n; ++i) put(gC, H, j, L.Dk + 3 + i, W1[(size_t)j * I + D + i]);
  }
  for (int r = 0; r < 3 * H; ++r) {
    const float sc = r < 2 * H ? 0.5f : 1.0f;
    for (int k = 0; k < H; ++k) {
      put(gA, 3 * H, r, k, sc * tw_bf16_value(Wih[(size_t)r * H + k]));
      if (r < 2 * H) put(gD, 2 * H, r, k, sc * tw_bf16_value(Whh[(size_t)r * H + k]));
      else put(gE, H, r - 2 * H, k, Whh[(size_t)r * H + k]);
    }
  }
  for (int a = 0; a < A; ++a) {
    for (int k = 0; k < H; ++k) put(gB, TW_NQ, a, k, W2[(size_t)a * H + k]);
    put3(gB, TW_NQ, a, H, b2[a]);
  }
}

__device__ __forceinline__ void tw_warp_arrive(uint64_t* bar, int lane) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
}

__global__ void __launch_bounds__(TW_THREADS, 1)
    actor_tcw_kernel(const __grid_constant__ ActorParams p, const __grid_constant__ TwLayout L) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using namespace tc;
  TwBars* B = reinterpret_cast<TwBars*>(smem + L.off_bar);
  uint8_t* xb = smem + L.off_x;
  uint8_t* yb = smem + L.off_y;
  uint8_t* hb = smem + L.off_hb;
  uint8_t* oh = smem + L.off_oh;
  uint8_t* stage = smem + L.off_stage;
  uint8_t* tails = smem + L.off_tail;                                  // [ept][tail_bytes]
  uint2* sel_s = reinterpret_cast<uint2*>(smem + L.off_sel);          // [4][128]: availability mask, random pick or -1
  int32_t* la_s = reinterpret_cast<int32_t*>(smem + L.off_la);
  int32_t* close_s = reinterpret_cast<int32_t*>(smem + L.off_close);  // [2][32]
  int32_t* closeany_s = reinterpret_cast<int32_t*>(smem + L.off_closeany);
  int32_t* rowenv_s = reinterpret_cast<int32_t*>(smem + L.off_rowenv);
  unsigned long long* dstp_s = reinterpret_cast<unsigned long long*>(smem + L.off_dstp);  // [16][32]
  unsigned long long* tdst_s = reinterpret_cast<unsigned long long*>(smem + L.off_tdst);  // [32]
  const float* tab_la = reinterpret_cast<const float*>(smem + L.off_tab_la);
  volatile uint32_t* abortf = &B->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = p.n, D = p.D, A = p.A, T = p.T;
  const uint32_t rec_bytes = p.rl.rec_bytes;
  const int NS = L.NS, NW = L.NW;
  const uint32_t t_q = p.rl.off_q - p.rl.off_action, t_reward = p.rl.off_reward - p.rl.off_action,
                 t_done = p.rl.off_done - p.rl.off_action;
  const int my_tiles = blockIdx.x < p.num_tiles ? (p.num_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (tid == 0) {
    for (int i = 0; i < TW_MAX_STAGES; ++i) {
      mbar_init(&B->full[i], 1);
      mbar_init(&B->cfree[i], 1);
      mbar_init(&B->sfree[i], 1);
    }
    for (int i = 0; i < TW_MAX_WSLOTS; ++i) {
      mbar_init(&B->wfull[i], 1);
      mbar_init(&B->wfree[i], 1);
    }
    mbar_init(&B->xready, TW_NCONV);
    mbar_init(&B->fc1d, 1);
    mbar_init(&B->yready, 8);
    mbar_init(&B->grud, 1);
    mbar_init(&B->hready, 8);
    mbar_init(&B->fc2d, 1);
    mbar_init(&B->stepd, 8);
    mbar_init(&B->tiled, 8);
    mbar_init(&B->wload, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&B->selready[i], TW_NCONV);
    mbar_init(&B->flags, 1);
    B->abort = 0;
    mbar_init_fence();
  }
  if (warp == 12) tmem_alloc(&B->tmem_base, TW_COLS);
  // operands, tails and hand-off arrays start as zeros (padding bytes of every stored record stay zero)
  for (uint32_t i = L.off_x / 16 + tid; i < L.off_bar / 16; i += TW_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
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
    mbar_arrive_expect_tx(&B->wload, L.rbytes);
    bulk_load(smem, p.wpack, L.rbytes, &B->wload);
  }
  mbar_wait(&B->wload, 0, abortf);

  if (warp >= 12) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(TW_REGS_SVC));
    if (warp == 12) {
      // =========================== MMA warp: lane 0 issues every tcgen05.mma ===========================
      const uint32_t sb = smem_u32(smem);
      const int total = my_tiles * T;
      constexpr uint64_t K_A = (2 * TC_LBO_A) >> 4, K_X = (2 * TC_LBO_X) >> 4;
      constexpr uint32_t id256 = idesc_bf16_f32(128, 256), id128 = idesc_bf16_f32(128, 128), idq = idesc_bf16_f32(128, TW_NQ);
      uint32_t wslot = 0, wpar = 0;  // slot and parity of the next weight slice
      uint32_t tl = 0;
      // waits for the next slice of the stream and returns its shared-memory address
      auto slice_begin = [&]() -> uint32_t {
        mbar_wait(&B->wfull[wslot], wpar, abortf);
        tc_fence_after_sync();
        return sb + L.off_wring + wslot * TW_WSLOT;
      };
      // the slot is free again when the MMAs issued so far have completed
      auto slice_end = [&]() {
        if (lane == 0) mma_commit(&B->wfree[wslot]);
        __syncwarp();
        if (++wslot == (uint32_t)NW) {
          wslot = 0;
          wpar ^= 1u;
        }
      };
      // C: fc1 of one step into the candidate-input columns: observations x W1, then one-hot tile x (bias pieces,
      // agent-id columns)
      auto issue_fc1 = [&]() {
        const int ks_all = L.ks_obs + L.ks_oh;
        for (int ks0 = 0; ks0 < ks_all; ks0 += 3) {
          const uint32_t base = slice_begin();
          if (lane == 0) {
            for (int j = 0; j < 3 && ks0 + j < ks_all; ++j) {
              const int ks = ks0 + j;
              const uint64_t da = ks < L.ks_obs ? smem_desc(sb + L.off_x, TC_LBO_X, 128) + (uint64_t)ks * K_X
                                                : smem_desc(sb + L.off_oh, TC_LBO_A, 128) + (uint64_t)(ks - L.ks_obs) * K_A;
              mma_bf16(tmem + TW_IN, da, smem_desc(base + (uint32_t)j * 4096u, 2048, 128), id128, ks > 0);
            }
          }
          slice_end();
        }
        if (lane == 0) mma_commit(&B->fc1d);
        __syncwarp();
      };
      // D: h-side products of the reset and update gates, seeded with their biases
      auto issue_hside_rz = [&]() {
        tc_fence_after_sync();
        if (lane == 0)
          mma_bf16(tmem + TW_R, smem_desc(sb + L.off_oh, TC_LBO_A, 128), smem_desc(sb + L.off_Brz, 4096, 128), id256, 0);
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t base = slice_begin();
          if (lane == 0)
            mma_bf16(tmem + TW_R, smem_desc(sb + L.off_hb, TC_LBO_A, 128) + (uint64_t)ks * K_A, smem_desc(base, 4096, 128), id256, 1);
          slice_end();
        }
      };
      // h-side product of the candidate (resident weights), seeded with its bias
      auto issue_hside_n = [&]() {
        tc_fence_after_sync();
        if (lane == 0) {
          mma_bf16(tmem + TW_HN, smem_desc(sb + L.off_oh, TC_LBO_A, 128), smem_desc(sb + L.off_Bhn, 2048, 128), id128, 0);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_bf16(tmem + TW_HN, smem_desc(sb + L.off_hb, TC_LBO_A, 128) + (uint64_t)ks * K_A,
                     smem_desc(sb + L.off_Whn + (uint32_t)ks * 4096u, 2048, 128), id128, 1);
        }
        __syncwarp();
      };
      if (total > 0) {
        mbar_wait(&B->xready, 0, abortf);
        tc_fence_after_sync();
        issue_fc1();
      }
      bool rz_issued = false;
      for (int g = 0, s = 0; g < total; ++g) {
        const uint32_t par = (uint32_t)g & 1u;
        // hidden operand in place (the tile prologue's, or the previous step's with closed episodes cleared), and
        // the previous step's Q read out of the candidate-hidden columns
        if (s == 0) {
          mbar_wait(&B->tiled, tl & 1, abortf);
          ++tl;
        } else {
          mbar_wait(&B->stepd, par ^ 1u, abortf);
        }
        if (!rz_issued) issue_hside_rz();
        issue_hside_n();
        // A: y-side products: r|z accumulate, the candidate-input columns start from their bias
        mbar_wait(&B->yready, par, abortf);
        tc_fence_after_sync();
        if (lane == 0)
          mma_bf16(tmem + TW_IN, smem_desc(sb + L.off_oh, TC_LBO_A, 128), smem_desc(sb + L.off_Bin, 2048, 128), id128, 0);
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t base = slice_begin();
          if (lane == 0) {
            const uint64_t dy = smem_desc(sb + L.off_y, TC_LBO_A, 128) + (uint64_t)ks * K_A;
            mma_bf16(tmem + TW_R, dy, smem_desc(base, 6144, 128), id256, 1);
            mma_bf16(tmem + TW_IN, dy, smem_desc(base + 256u * 16u, 6144, 128), id128, 1);
          }
          slice_end();
        }
        if (lane == 0) mma_commit(&B->grud);
        __syncwarp();
        // fc2 (resident weights) into four 16-column parts (dependent MMAs on one accumulator run one after the other):
        // part ks % 4 takes K-steps ks and ks + 4, part 0 starts from the bias step
        mbar_wait(&B->hready, par, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
          const uint32_t base = sb + L.off_W2;
          const uint64_t dh = smem_desc(sb + L.off_hb, TC_LBO_A, 128);
          mma_bf16(tmem + TW_HN, smem_desc(sb + L.off_oh, TC_LBO_A, 128), smem_desc(base + 8u * 512u, 256, 128), idq, 0);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_bf16(tmem + TW_HN + (uint32_t)(ks & 3) * 16u, dh + (uint64_t)ks * K_A, smem_desc(base + (uint32_t)ks * 512u, 256, 128), idq,
                     (ks == 0 || ks >= 4) ? 1 : 0);
          mma_commit(&B->fc2d);
        }
        __syncwarp();
        // C: fc1 of the next step (possibly the next tile's first): the gate math of this step has read the
        // candidate-input columns
        if (g + 1 < total) {
          mbar_wait(&B->xready, par ^ 1u, abortf);
          tc_fence_after_sync();
          issue_fc1();
        }
        // D of the next step needs only the new hidden state, which is in place unless an episode of this tile ends
        // with this step (its rows are cleared after fc2)
        rz_issued = false;
        if (++s == T) {
          s = 0;
        } else if (closeany_s[g & (TW_DST_DEPTH - 1)] == 0) {
          issue_hside_rz();
          rz_issued = true;
        }
      }
    } else if (warp == 13) {
      // =========================== load warp: staging ring in, record addresses ahead ===========================
      int tile = blockIdx.x;
      int32_t slot = 0, pos = 0, ok = 0;
      long long epc = 0;
      uint32_t done_next = 0;
      uint32_t q = 0, qslot = 0, qpar = 1, kstep = 0;
      for (; tile < p.num_tiles; tile += gridDim.x) {
        const int ne = min(L.ept, p.M - tile * L.ept);
        const int nck = (ne + TW_G - 1) / TW_G;
        const int e = tile * L.ept + lane;
        const bool mine = lane < ne;
        ok = 0;
        if (mine) {
          slot = p.slot[e];
          pos = p.pos[e];
          epc = p.ep_count[e];
          ok = (slot >= 0 && slot < p.E * p.S && pos >= 0 && pos < p.L) ? 1 : 0;
          done_next = p.done[e];
        }
        for (int s = 0; s < T; ++s, ++kstep) {
          unsigned long long rec = 0;
          int closes = 0;
          if (mine && ok) {
            rec = reinterpret_cast<unsigned long long>(p.ring + (size_t)slot * p.slot_stride + (size_t)pos * rec_bytes);
            if (done_next || pos + 1 == p.L) {  // the cursor after this step
              closes = 1;
              epc += 1;
              slot = e * p.S + (int)(epc % p.S);
              pos = 0;
            } else {
              pos += 1;
            }
          }
          dstp_s[(kstep & (TW_DST_DEPTH - 1)) * 32 + lane] = rec;
          closes = __any_sync(0xFFFFFFFFu, closes);
          if (lane == 0) closeany_s[kstep & (TW_DST_DEPTH - 1)] = closes;
          if (mine && s + 1 < T) done_next = p.done[(size_t)(s + 1) * p.env_step_stride + e];
          __syncwarp();
          for (int c = 0; c < nck; ++c) {
            const int ge = min(TW_G, ne - c * TW_G);
            if (q >= (uint32_t)NS) {  // the slot's previous chunk is converted and its observations are stored
              mbar_wait(&B->cfree[qslot], qpar, abortf);
              mbar_wait(&B->sfree[qslot], qpar, abortf);
            }
            if (lane == 0) mbar_arrive_expect_tx(&B->full[qslot], (uint32_t)ge * L.prefix_bytes);
            __syncwarp();
            const size_t env0 = (size_t)tile * L.ept + (size_t)(c * TW_G);
            uint8_t* dst = stage + qslot * L.chunk_bytes;
            if (lane == 0)
              bulk_load(dst, p.obs + (size_t)s * p.obs_step_stride + env0 * (size_t)(n * D), (uint32_t)ge * L.obs_bytes,
                        &B->full[qslot]);
            if (lane == 1)
              bulk_load(dst + TW_G * L.obs_bytes, p.avail + (size_t)s * p.avail_step_stride + env0 * (size_t)(n * A),
                        (uint32_t)ge * L.av_bytes, &B->full[qslot]);
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
        const int e = tile * L.ept + lane;
        int32_t slot = 0, pos = 0, ok = 0;
        long long epc = 0;
        float reward_next = 0.f;
        uint32_t done_next = 0;
        if (mine) {
          slot = p.slot[e];
          pos = p.pos[e];
          epc = p.ep_count[e];
          ok = (slot >= 0 && slot < p.E * p.S && pos >= 0 && pos < p.L) ? 1 : 0;
          if (!ok) st_bits |= MARL_STATUS_BAD_INDEX;
          reward_next = p.reward[e];
          done_next = p.done[e];
        }
        // Copies the tails of the finished step (record addresses in tdst_s) to the ring: 16 bytes per lane, the
        // pieces of all environments in one flat loop.  One tail buffer: the copy follows the step directly, and the
        // next step's epilogue 3 is opened (flags) only after it.
        auto copy_tails = [&]() {
          __syncwarp();
          const uint32_t pieces = L.tail_bytes / 16u, total = (uint32_t)ne * pieces;
          const uint32_t inv = 0xFFFFFFFFu / pieces + 1u;  // idx / pieces == umulhi(idx, inv) for idx < 2^16
          for (uint32_t idx = lane; idx < total; idx += 32) {
            const uint32_t env = __umulhi(idx, inv), pc = idx - env * pieces;
            const unsigned long long d = tdst_s[env];
            if (d) reinterpret_cast<uint4*>(d)[pc] = reinterpret_cast<const uint4*>(tails + env * L.tail_bytes)[pc];
          }
          __syncwarp();
        };
        for (int s = 0; s < T; ++s) {
          const uint32_t b = it & 1;
          const float reward = reward_next;
          const int done = done_next ? 1 : 0;
          const int close = (ok && (done || pos + 1 == p.L)) ? 1 : 0;
          uint8_t* tl = tails + (uint32_t)lane * L.tail_bytes;
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
          if (lane == 0) mbar_arrive(&B->flags);  // epilogue 3 of this step may write the tails
          if (mine && s + 1 < T) {
            reward_next = p.reward[(size_t)(s + 1) * p.env_step_stride + e];
            done_next = p.done[(size_t)(s + 1) * p.env_step_stride + e];
          }
          mbar_wait(&B->stepd, sd & 1, abortf);  // action and Q of step s are in the tail
          ++sd;
          tdst_s[lane] = dst;
          copy_tails();
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
      uint32_t q = 0, qslot = 0, qpar = 0, pslot = 0, kstep = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        const int ne = min(L.ept, p.M - tile * L.ept);
        const int nck = (ne + TW_G - 1) / TW_G;
        for (int s = 0; s < T; ++s, ++kstep) {
          for (int c = 0; c < nck; ++c) {
            const int ge = min(TW_G, ne - c * TW_G);
            mbar_wait(&B->full[qslot], qpar, abortf);
            if (lane < ge) {
              const unsigned long long rec = dstp_s[(kstep & (TW_DST_DEPTH - 1)) * 32 + c * TW_G + lane];
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
        }
      }
      bulk_wait_read_all();
      __syncwarp();
      if (q > 0 && lane == 0) mbar_arrive(&B->sfree[pslot]);
      bulk_wait_all();
    }
  } else if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(TW_REGS_CONV));
    if (warp == 11) {
      // =========================== weight loader: the streamed image, slice by slice, through the ring ===========
      const uint8_t* stream = static_cast<const uint8_t*>(p.wpack) + L.stream_off;
      const uint32_t total = (uint32_t)(my_tiles * T) * (uint32_t)L.n_slices;
      uint32_t wslot = 0, wpar = 1, sl = 0;  // wpar: parity of the slot's previous use
      for (uint32_t q = 0; q < total; ++q) {
        if (q >= (uint32_t)NW) mbar_wait(&B->wfree[wslot], wpar, abortf);
        if (lane == 0) {
          const uint32_t bytes = L.slice_bytes[sl];
          mbar_arrive_expect_tx(&B->wfull[wslot], bytes);
          bulk_load(smem + L.off_wring + wslot * TW_WSLOT, stream + L.slice_off[sl], bytes, &B->wfull[wslot]);
        }
        __syncwarp();
        if (++sl == (uint32_t)L.n_slices) sl = 0;
        if (++wslot == (uint32_t)NW) {
          wslot = 0;
          wpar ^= 1u;
        }
      }
    } else {
      // =========================== converters: staged observations -> bf16 operand; masks and epsilon draws ==========
      // Each of the three warps takes whole chunks (chunk c of a step goes to warp c % 3); afterwards the rows of the
      // tile are shared out among the 96 threads for the epsilon draw.
      const int ci = tid - 256, cw = warp - 8;
      const uint32_t inv_nchunk = 0xFFFFFFFFu / (uint32_t)L.nchunk + 1u;  // j / nchunk == umulhi(j, inv) for j < 2^16
      const uint32_t amask = (1u << A) - 1u;
      uint32_t it = 0, qbase = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        const int e0 = tile * L.ept;
        const int ne = min(L.ept, p.M - e0);
        const int nck = (ne + TW_G - 1) / TW_G;
        for (int s = 0; s < T; ++s) {
          const uint32_t t = p.t0 + (uint32_t)s;
          const float eps = eps_at(p, t);
          uint2* sel = sel_s + (it & 3) * TC_ROWS;
          // the operand buffer is free once fc1 of the previous step has finished reading it
          if (it > 0) mbar_wait(&B->fc1d, (it - 1) & 1, abortf);
          for (int c = cw; c < nck; c += TW_NCONV) {
            const int ge = min(TW_G, ne - c * TW_G);
            const int Rc = ge * n;
            const int r0 = c * TW_G * n;
            const uint32_t q = qbase + (uint32_t)c, qslot = q % (uint32_t)NS, qpar = (q / (uint32_t)NS) & 1u;
            const uint8_t* src = stage + qslot * L.chunk_bytes;
            const unsigned long long* recs = dstp_s + (it & (TW_DST_DEPTH - 1)) * 32 + c * TW_G;
            mbar_wait(&B->full[qslot], qpar, abortf);
            const int items = Rc * L.nchunk;
            for (int j = lane; j < items; j += 32) {
              const int rr = (int)__umulhi((uint32_t)j, inv_nchunk), cc = j - rr * L.nchunk;
              float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f), v1 = v0;
              if (cc * 8 < D) {
                const float4* s4 = reinterpret_cast<const float4*>(src + (uint32_t)(rr * D) * 4u + (uint32_t)cc * 32u);
                v0 = s4[0];
                v1 = s4[1];
              }
              *reinterpret_cast<uint4*>(xb + (uint32_t)cc * TC_LBO_X + (uint32_t)(r0 + rr) * 16u) =
                  make_uint4(pack_bf16x2(v0.x, v0.y), pack_bf16x2(v0.z, v0.w), pack_bf16x2(v1.x, v1.y), pack_bf16x2(v1.z, v1.w));
            }
            const uint8_t* avs = src + TW_G * L.obs_bytes;  // the chunk's availability bytes, rows contiguous
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
              for (int k = 0; k < 5; ++k) {
                const uint32_t v = w[k];
                const uint32_t nz = ((v | ((v & 0x7F7F7F7Fu) + 0x7F7F7F7Fu)) & 0x80808080u) >> 7;  // 0x01 per non-zero byte
                bits |= (unsigned long long)((nz * 0x01020408u) >> 24 & 0xFu) << (4 * k);
              }
              sel[r0 + rc].x = (uint32_t)(bits >> (off & 3u)) & amask;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&B->cfree[qslot]);
          }
          qbase += (uint32_t)nck;
          fence_proxy_async_smem();
          tw_warp_arrive(&B->xready, lane);
          asm volatile("bar.sync 2, 96;" ::: "memory");  // the masks were written by the chunks' warps
          for (int r = ci; r < ne * n; r += 32 * TW_NCONV) {
            const int rel = r / n, rai = r - rel * n;
            const uint32_t mask = sel[r].x;
            int pick = -1;
            if (mask != 0) pick = draw_explore(mask, eps, p.seed, t, (uint32_t)(e0 + rel), (uint32_t)rai);
            sel[r].y = (uint32_t)pick;
          }
          tw_warp_arrive(&B->selready[it & 3], lane);
          ++it;
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(TW_REGS_EPI));
    // =========================== epilogue threads: one agent row x 64 hidden columns ===========================
    const int row = tid & 127, half = tid >> 7;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int el = row / n, ai = row - el * n;
    const int cb = half * 64;  // first hidden column of this thread
    unsigned long long c_steps = 0, c_explore = 0, c_noavail = 0;
    uint32_t st_bits = 0, it = 0;
    float h[64];

    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int e0 = tile * L.ept;
      const int ne = min(L.ept, p.M - e0);
      const int R = ne * n;
      const bool live = row < R;
      const bool is_row = live && half == 0;  // owner of the row's choice
      const int e = e0 + el;
      const size_t grow = (size_t)e * n + ai;
      int la = -1;

      // ---- tile prologue: hidden state and last actions from global memory ----
      {
        const int la_mem = is_row ? p.last_action[grow] : -1;
        const float4* src = reinterpret_cast<const float4*>(p.h + grow * TW_H + cb);
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          const float4 v = live ? src[q] : make_float4(0.f, 0.f, 0.f, 0.f);
          h[4 * q] = v.x; h[4 * q + 1] = v.y; h[4 * q + 2] = v.z; h[4 * q + 3] = v.w;
        }
#pragma unroll
        for (int cc = 0; cc < 8; ++cc) {
          const uint4 o = make_uint4(pack_bf16x2(h[8 * cc], h[8 * cc + 1]), pack_bf16x2(h[8 * cc + 2], h[8 * cc + 3]),
                                     pack_bf16x2(h[8 * cc + 4], h[8 * cc + 5]), pack_bf16x2(h[8 * cc + 6], h[8 * cc + 7]));
          *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 8 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
        }
        if (half == 0) {
          la = la_mem;
          if (la >= A) la = -1;
          la_s[row] = la;
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        asm volatile("bar.sync 1, 256;" ::: "memory");  // la_s is read by both threads of a row
        tw_warp_arrive(&B->tiled, lane);
      }

      for (int s = 0; s < T; ++s) {
        const uint32_t b = it & 1, par = it & 1;
        uint8_t* tl = tails + (uint32_t)el * L.tail_bytes;  // this row's environment tail

        // ---- epilogue 1: y = relu(fc1 + W1[:, last action]) -> bf16 operand (bias and agent-id column are inside
        //      the GEMM; the accumulator sits in the candidate-input columns) ----
        mbar_wait(&B->fc1d, par, abortf);
        tc_fence_after_sync();
        {
          const int last = (s > 0 && close_s[(b ^ 1u) * 32 + el]) ? -1 : la_s[row];  // an episode that just ended has none
          const float* tlr = tab_la + (last >= 0 ? last : 0) * TW_TAB + cb;
#pragma unroll
          for (int c32 = 0; c32 < 2; ++c32) {
            uint32_t v2[2][16];
            tmem_ld16(tmem + lane_addr + TW_IN + cb + c32 * 32, v2[0]);
            tmem_ld16(tmem + lane_addr + TW_IN + cb + c32 * 32 + 16, v2[1]);
            tmem_ld_wait();
#pragma unroll
            for (int c16 = 0; c16 < 2; ++c16) {
              uint32_t(&v)[16] = v2[c16];
              float y[16];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                float4 l4 = make_float4(0.f, 0.f, 0.f, 0.f);
                if (last >= 0) l4 = *reinterpret_cast<const float4*>(tlr + c32 * 32 + c16 * 16 + 4 * q);
                y[4 * q] = fmaxf(__uint_as_float(v[4 * q]) + l4.x, 0.f);
                y[4 * q + 1] = fmaxf(__uint_as_float(v[4 * q + 1]) + l4.y, 0.f);
                y[4 * q + 2] = fmaxf(__uint_as_float(v[4 * q + 2]) + l4.z, 0.f);
                y[4 * q + 3] = fmaxf(__uint_as_float(v[4 * q + 3]) + l4.w, 0.f);
              }
#pragma unroll
              for (int cc = 0; cc < 2; ++cc) {
                const uint4 o = make_uint4(pack_bf16x2(y[8 * cc], y[8 * cc + 1]), pack_bf16x2(y[8 * cc + 2], y[8 * cc + 3]),
                                           pack_bf16x2(y[8 * cc + 4], y[8 * cc + 5]), pack_bf16x2(y[8 * cc + 6], y[8 * cc + 7]));
                *reinterpret_cast<uint4*>(yb + (uint32_t)(half * 8 + c32 * 4 + c16 * 2 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
              }
            }
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        tw_warp_arrive(&B->yready, lane);

        // ---- epilogue 2: gate math, new hidden state (fp32 registers) and its bf16 operand.
        //      The r and z accumulators hold half the pre-activation: sigmoid(v) = 0.5 * tanh(v / 2) + 0.5 ----
        mbar_wait(&B->grud, par, abortf);
        tc_fence_after_sync();
        {
          uint32_t g[2][4][8];  // [buffer][r, z, candidate-input, candidate-hidden][column]
          auto request = [&](int c8, uint32_t (&d)[4][8]) {
            const uint32_t col = (uint32_t)(cb + c8 * 8);
            tmem_ld8(tmem + lane_addr + TW_R + col, d[0]);
            tmem_ld8(tmem + lane_addr + TW_Z + col, d[1]);
            tmem_ld8(tmem + lane_addr + TW_IN + col, d[2]);
            tmem_ld8(tmem + lane_addr + TW_HN + col, d[3]);
          };
          request(0, g[0]);
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8) {
            tmem_ld_wait();
            if (c8 + 1 < 8) request(c8 + 1, g[(c8 + 1) & 1]);
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
            *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 8 + c8) * TC_LBO_A + (uint32_t)row * 16u) = o;
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        tw_warp_arrive(&B->hready, lane);

        // ---- epilogue 3: the row owners choose and complete the record's tail ----
        mbar_wait(&B->flags, par, abortf);  // close flags of this step written, tail buffer free
        mbar_wait(&B->fc2d, par, abortf);   // (both halves: the hidden operand may be cleared below)
        tc_fence_after_sync();
        if (half == 0) {
          uint32_t qv[16], q1[16], q2[16], q3[16];
          tmem_ld16(tmem + lane_addr + TW_HN, qv);
          tmem_ld16(tmem + lane_addr + TW_HN + 16, q1);
          tmem_ld16(tmem + lane_addr + TW_HN + 32, q2);
          tmem_ld16(tmem + lane_addr + TW_HN + 48, q3);
          tmem_ld_wait();
#pragma unroll
          for (int a = 0; a < 16; ++a)
            qv[a] = __float_as_uint((__uint_as_float(qv[a]) + __uint_as_float(q1[a])) + (__uint_as_float(q2[a]) + __uint_as_float(q3[a])));
          tc_fence_before_sync();
          if (is_row) {
            mbar_wait(&B->selready[it & 3], (it >> 2) & 1, abortf);
            const uint2 sp = sel_s[(it & 3) * TC_ROWS + row];
            const uint32_t mask = sp.x;
            const int pick = (int)sp.y;
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
            la = act;
            la_s[row] = act;
            float* qrow = reinterpret_cast<float*>(tl + t_q) + ai * A;
            if ((A & 1) == 0) {
#pragma unroll
              for (int a = 0; a < 16; a += 2)
                if (a < A) *reinterpret_cast<float2*>(qrow + a) = make_float2(__uint_as_float(qv[a]), __uint_as_float(qv[a + 1]));
            } else {
#pragma unroll
              for (int a = 0; a < 16; ++a)
                if (a < A) qrow[a] = __uint_as_float(qv[a]);
            }
            reinterpret_cast<int32_t*>(tl)[ai] = act;
            const int tk = p.trace_first + s;
            if (tk < p.trace_cap) {
              const size_t trow = ((size_t)tk * p.E + e) * n + ai;
              if (p.trace_actions) p.trace_actions[trow] = act;
              if (p.trace_q) {
#pragma unroll
                for (int a = 0; a < 16; ++a)
                  if (a < A) p.trace_q[trow * A + a] = __uint_as_float(qv[a]);
              }
            }
            if (p.actions_out && s == T - 1) p.actions_out[grow] = act;
          }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // ---- a closed episode restarts from a zero hidden state and no last action ----
        if (live && close_s[b * 32 + el]) {
#pragma unroll
          for (int j = 0; j < 64; ++j) h[j] = 0.f;
#pragma unroll
          for (int cc = 0; cc < 8; ++cc)
            *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 8 + cc) * TC_LBO_A + (uint32_t)row * 16u) = make_uint4(0, 0, 0, 0);
          if (half == 0) la = -1;
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        tw_warp_arrive(&B->stepd, lane);
        ++it;
      }

      // ---- tile epilogue: state back to global memory ----
      if (is_row) p.last_action[grow] = la;
      if (live) {
        float4* dsth = reinterpret_cast<float4*>(p.h + grow * TW_H + cb);
#pragma unroll
        for (int q = 0; q < 16; ++q) dsth[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
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
  if (warp == 12) tmem_dealloc(tmem, TW_COLS);
}

// Returns the number of kernels launched, 0 if this launch cannot run here (a list step, or pointers that cannot be
// bulk-copied: the caller then uses the CUDA-core kernel), or a negative cudaError.
int launch_actor_tcw(const ActorParams& p_in, int sms, cudaStream_t stream) {
  if (p_in.env_ids != nullptr || p_in.lagged) return 0;
  const TwLayout L = tw_layout(p_in.n, p_in.D, p_in.A, (int)p_in.rl.rec_bytes);
  ActorParams p = p_in;
  p.ept = L.ept;
  p.num_tiles = (p.M + L.ept - 1) / L.ept;
  if (reinterpret_cast<uintptr_t>(p.obs) % 16 || reinterpret_cast<uintptr_t>(p.avail) % 16) return 0;
  if ((p.obs_step_stride * 4) % 16 || p.avail_step_stride % 16) return 0;
  if (reinterpret_cast<uintptr_t>(p.wpack) % 16) return 0;
  static uint32_t configured[SMEM_OPTIN_DEVICES];
  {
    const cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(actor_tcw_kernel), L.total, configured);
    if (e != cudaSuccess) return -(int)e;
  }
  int grid = p.num_tiles < sms ? p.num_tiles : sms;
  if (grid < 1) grid = 1;
  actor_tcw_kernel<<<grid, TW_THREADS, L.total, stream>>>(p, L);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 1 : -(int)err;
}

}  // namespace marl
