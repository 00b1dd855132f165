// Tensor-core actor kernel for sm_100a: bf16 operands, hidden size 64, observation width a multiple of 8.
//
// Schedule (as in the FFMA kernel): one thread block owns a tile of whole environments - up to 128 agent
// rows, the M of one tcgen05.mma - and runs all T steps of the launch for it before the next tile, because
// environments never exchange data (Sec. III-A, Fig. 3).  Hidden state (fp32, in registers), last actions
// and ring cursors stay on chip for the whole launch.
//
// Per step, the worker's decision (Algorithm 2) and the actor's recording (Algorithm 1) become:
//   bulk-async load of the tile's observations, one copy per environment, straight into that environment's
//   ring record being assembled in shared memory
//   -> bf16 copy of the observations in the UMMA operand layout
//   -> fc1 on the tensor core (accumulator in tensor memory) -> +bias, +one-hot columns, ReLU, bf16 (epilogue 1)
//   -> the two GRU gate GEMMs (r|z accumulate both products in one accumulator; the h-side products are
//      issued before epilogue 1 finishes, so they overlap it) -> gate math, new hidden state (epilogue 2)
//   -> fc2 -> Q row, masked greedy choice, Philox epsilon draw, record completion (epilogue 3)
//   -> one bulk store of the finished record per environment, episode bookkeeping, hidden-state reset.
//
// Thread roles: 256 epilogue threads - thread (row, half) owns one accumulator row (one agent) and 32 of its
// 64 hidden columns, so gate math, arg-max and the random draw need no cross-thread reduction - plus one
// warp whose lane 0 issues every tcgen05.mma and one warp whose lanes share the bulk copies.  The two halves
// split the third epilogue: half 0 chooses actions while half 1 converts the next step's observations.
// All hand-offs go through mbarriers with bounded waits; an expired wait sets MARL_STATUS_TIMEOUT and lets
// the block run to its end without touching anything out of range.
//
// Shared memory: the packed weights (bf16 matrices in operand layout, fp32 bias/one-hot tables), one x/y
// operand buffer, one hidden-state operand buffer, two sets of ring records (double-buffered over steps).
#include <cstring>
#include <vector>

#include "actor_tc_layout.cuh"
#include "common.cuh"
#include "launch_util.cuh"
#include "tcgen05.cuh"

namespace marl {

bool tc_supported(int n, int D, int A, int H, int prec) {
  if (prec != MARL_PRECISION_BF16 || H != TC_H) return false;
  if (D % 8 != 0 || D > 256 || n < 1 || n > 32 || A < 1 || A > 32) return false;
  return tc_layout(n, D, A, rec_bytes_of(n, D, A)).total <= TC_SMEM_MAX;
}

// (the packed image of the hidden-128 kernel: actor_tcw.cu)
size_t tcw_wpack_bytes(int n, int D, int A);
void tcw_pack_weights(int n, int D, int A, const float* W1, const float* b1, const float* Wih, const float* bih,
                      const float* Whh, const float* bhh, const float* W2, const float* b2, void* dst_host);

size_t tc_wpack_bytes(int n, int D, int A, int H) {
  if (H == 128) return tcw_wpack_bytes(n, D, A);
  if (H != TC_H || D < 1 || D > 256 || n < 1 || n > 32 || A < 1 || A > 32) return 0;  // (a layout question only)
  return tc_layout(n, D, A, rec_bytes_of(n, D, A)).wbytes;
}

static uint16_t bf16_bits(float v) {
  uint32_t u;
  memcpy(&u, &v, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}
static float bf16_value(float v) {
  const uint32_t u = (uint32_t)bf16_bits(v) << 16;
  float o;
  memcpy(&o, &u, 4);
  return o;
}

// Element (row, k) of an N-row K-major operand: k-chunks of all rows are contiguous (LBO = N * 16).
static size_t operand_offset(int N, int row, int k) { return (size_t)(k / 8) * N * 16 + (size_t)row * 16 + (k % 8) * 2; }

void tc_pack_weights(int n, int D, int A, int H, const float* W1, const float* b1, const float* Wih,
                     const float* bih, const float* Whh, const float* bhh, const float* W2, const float* b2,
                     void* dst_host) {
  if (H == 128) {
    tcw_pack_weights(n, D, A, W1, b1, Wih, bih, Whh, bhh, W2, b2, dst_host);
    return;
  }
  const TcLayout L = tc_layout(n, D, A, rec_bytes_of(n, D, A));
  const int I = D + n + A;
  uint8_t* o = static_cast<uint8_t*>(dst_host);
  memset(o, 0, L.wbytes);
  auto put = [&](uint32_t base, int N, int row, int k, float v) {
    const uint16_t b = bf16_bits(v);
    memcpy(o + base + operand_offset(N, row, k), &b, 2);
  };
  // a fp32 value as three bf16 pieces at k0, k0+1, k0+2
  auto put3 = [&](uint32_t base, int N, int row, int k0, float v) {
    const float p0 = bf16_value(v), p1 = bf16_value(v - p0), p2 = bf16_value(v - p0 - p1);
    put(base, N, row, k0, p0);
    put(base, N, row, k0 + 1, p1);
    put(base, N, row, k0 + 2, p2);
  };
  for (int j = 0; j < H; ++j) {
    for (int k = 0; k < D; ++k) put(L.off_W1, H, j, k, W1[(size_t)j * I + k]);
    put3(L.off_W1, H, j, L.Dk, b1[j]);
    for (int i = 0; i < n; ++i) put(L.off_W1, H, j, L.Dk + 3 + i, W1[(size_t)j * I + D + i]);
  }
  for (int r = 0; r < 3 * H; ++r) {
    const float sc = r < 2 * H ? 0.5f : 1.0f;  // reset and update rows are stored halved
    for (int k = 0; k < H; ++k) {
      put(L.off_Wih, 3 * H, r, k, sc * bf16_value(Wih[(size_t)r * H + k]));
      put(L.off_Whh, 3 * H, r, k, sc * bf16_value(Whh[(size_t)r * H + k]));
    }
    if (r < 2 * H) {
      put3(L.off_Bg, 3 * H, r, 0, 0.5f * (bih[r] + bhh[r]));
    } else {
      put3(L.off_Bg, 3 * H, r, 0, bih[r]);
      put3(L.off_Bhn, H, r - 2 * H, 0, bhh[r]);
    }
  }
  for (int a = 0; a < A; ++a) {
    for (int k = 0; k < H; ++k) put(L.off_W2, L.NQ, a, k, W2[(size_t)a * H + k]);
    put3(L.off_W2, L.NQ, a, H, b2[a]);
  }
  float* tla = reinterpret_cast<float*>(o + L.off_tab_la);
  for (int a = 0; a < A; ++a)
    for (int j = 0; j < H; ++j) tla[a * TC_TAB + j] = bf16_value(W1[(size_t)j * I + D + n + a]);
}

// Environments per tile: as many as fit 128 rows.  (Spreading a batch of fewer tiles than SMs over partly filled
// tiles was measured and gains nothing: a launch of T steps takes T times the per-step dependency chain of one
// tile however few rows the tile holds.)
void tc_tiling(int E, int n, int /*sms*/, int* ept, int* num_tiles) {
  *ept = TC_ROWS / n;
  *num_tiles = (E + *ept - 1) / *ept;
}

struct TcBars {
  uint64_t full[2], xready, fc1d, yready, grud, hready, fc2d, stepd, wload, selready;
  uint32_t tmem_base, abort;
};

template <int NQ>
__global__ void __launch_bounds__(TC_THREADS, 1)
    actor_tc_kernel(const __grid_constant__ ActorParams p, const __grid_constant__ TcLayout L) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using namespace tc;
  TcBars* B = reinterpret_cast<TcBars*>(smem + L.off_bar);
  uint8_t* xy = smem + L.off_xy;
  uint8_t* hb = smem + L.off_hb;
  uint8_t* oh = smem + L.off_oh;
  uint8_t* recs = smem + L.off_rec;
  unsigned long long* dst_s = reinterpret_cast<unsigned long long*>(smem + L.off_dst);  // [2][128]
  int32_t* reset_s = reinterpret_cast<int32_t*>(smem + L.off_reset);
  int32_t* la_s = reinterpret_cast<int32_t*>(smem + L.off_la);    // last action of every row, for the half-1 threads
  const float* tab_la = reinterpret_cast<const float*>(smem + L.off_tab_la);
  uint32_t* rowoff_s = reinterpret_cast<uint32_t*>(smem + L.off_rowoff);
  uint2* sel_s = reinterpret_cast<uint2*>(smem + L.off_sel);  // per row: availability mask, random pick or -1
  volatile uint32_t* abortf = &B->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = p.n, D = p.D, A = p.A;
  const uint32_t rec_bytes = p.rl.rec_bytes;
  const uint32_t buf_bytes = (uint32_t)L.ept * rec_bytes;

  if (tid == 0) {
    mbar_init(&B->full[0], 1);
    mbar_init(&B->full[1], 1);
    mbar_init(&B->xready, 128);
    mbar_init(&B->fc1d, 1);
    mbar_init(&B->yready, 256);
    mbar_init(&B->grud, 1);
    mbar_init(&B->hready, 256);
    mbar_init(&B->fc2d, 1);
    mbar_init(&B->stepd, 256);
    mbar_init(&B->wload, 1);
    mbar_init(&B->selready, 64);
    B->abort = 0;
    mbar_init_fence();
  }
  if (warp == 8) tmem_alloc(&B->tmem_base, TM_COLS);
  // record buffers start as zeros so that the padding bytes of every stored record are zero
  for (uint32_t i = tid; i < 2u * buf_bytes / 16u; i += TC_THREADS) reinterpret_cast<uint4*>(recs)[i] = make_uint4(0, 0, 0, 0);
  if (tid < TC_ROWS) rowoff_s[tid] = (uint32_t)(tid / n) * rec_bytes + (uint32_t)((tid % n) * D) * 4u;
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = B->tmem_base;
  if (tid == TC_EPI_THREADS) {
    mbar_arrive_expect_tx(&B->wload, L.wbytes);
    bulk_load(smem, p.wpack, L.wbytes, &B->wload);
  }
  mbar_wait(&B->wload, 0, abortf);

  uint32_t it = 0;  // steps processed so far by this block (all tiles): parity source of the per-step barriers
  uint32_t sd = 0;  // phases of the step_done barrier

  if (warp >= 8) {
   asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(TC_REGS_SERVICE));
   if (warp == 8) {
    // =========================== MMA warp: lane 0 issues every tcgen05.mma ===========================
    const uint32_t id64 = idesc_bf16_f32(128, 64), id128 = idesc_bf16_f32(128, 128), idq = idesc_bf16_f32(128, NQ), id192 = idesc_bf16_f32(128, 192);
    const uint32_t lbo_w1 = TC_H * 16, lbo_g = 3 * TC_H * 16, lbo_q = (uint32_t)NQ * 16;
    const uint32_t gate_n = 2 * TC_H * 16;  // byte offset of the candidate-gate rows inside a k-chunk of W_ih / W_hh
    // descriptors of the first k-step of every operand; a later k-step adds (2 * LBO) >> 4 to the address field
    const uint64_t d_x = smem_desc(smem_u32(xy), TC_LBO_X, 128), d_y = smem_desc(smem_u32(xy), TC_LBO_A, 128);
    const uint64_t d_h = smem_desc(smem_u32(hb), TC_LBO_A, 128), d_oh = smem_desc(smem_u32(oh), TC_LBO_A, 128);
    const uint64_t d_W1 = smem_desc(smem_u32(smem + L.off_W1), lbo_w1, 128);
    const uint64_t d_W1oh = smem_desc(smem_u32(smem + L.off_W1) + (uint32_t)L.nchunk * lbo_w1, lbo_w1, 128);
    const uint64_t d_Wih = smem_desc(smem_u32(smem + L.off_Wih), lbo_g, 128);
    const uint64_t d_Whh = smem_desc(smem_u32(smem + L.off_Whh), lbo_g, 128);
    const uint64_t d_Whh_n = smem_desc(smem_u32(smem + L.off_Whh) + gate_n, lbo_g, 128);
    const uint64_t d_Bg = smem_desc(smem_u32(smem + L.off_Bg), lbo_g, 128);
    const uint64_t d_Bhn = smem_desc(smem_u32(smem + L.off_Bhn), lbo_w1, 128);
    const uint64_t d_W2 = smem_desc(smem_u32(smem + L.off_W2), lbo_q, 128);
    const uint64_t k_x = (2 * TC_LBO_X) >> 4, k_a = (2 * TC_LBO_A) >> 4, k_w1 = (2 * lbo_w1) >> 4, k_g = (2 * lbo_g) >> 4,
                   k_q = (2 * lbo_q) >> 4;
    const int ks_obs = L.Dk / 16, ks_oh = L.ohK / 16;
    // fc1 of a step depends only on the converted observations (the last-action term is added in epilogue 1),
    // so it is issued as soon as those are ready - for step s+1 while step s is still in its third epilogue.
    auto issue_fc1 = [&]() {
      mbar_wait(&B->xready, it & 1, abortf);
      tc_fence_after_sync();
      if (lane == 0) {
        for (int ks = 0; ks < ks_obs; ++ks) mma_bf16(tmem + TM_FC1, d_x + ks * k_x, d_W1 + ks * k_w1, id64, ks > 0);
        for (int ks = 0; ks < ks_oh; ++ks) mma_bf16(tmem + TM_FC1, d_oh + ks * k_a, d_W1oh + ks * k_w1, id64, 1);
        mma_commit(&B->fc1d);
      }
      __syncwarp();
    };
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      issue_fc1();
      for (int s = 0; s < p.T; ++s) {
        const uint32_t par = it & 1;
        mbar_wait(&B->stepd, sd & 1, abortf);  // prologue or previous step: hidden operand in place
        ++sd;
        tc_fence_after_sync();
        if (lane == 0) {
          // h-side gate products; the first MMA seeds r | z | candidate-input with their biases (r, z and the
          // candidate's input part are contiguous in tensor memory: one N = 192 accumulator)
          mma_bf16(tmem + TM_R, d_oh, d_Bg, id192, 0);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            mma_bf16(tmem + TM_R, d_h + ks * k_a, d_Whh + ks * k_g, id128, 1);
            mma_bf16(tmem + TM_HN, d_h + ks * k_a, d_Whh_n + ks * k_g, id64, ks > 0);
          }
          mma_bf16(tmem + TM_HN, d_oh, d_Bhn, id64, 1);
        }
        __syncwarp();
        mbar_wait(&B->yready, par, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma_bf16(tmem + TM_R, d_y + ks * k_a, d_Wih + ks * k_g, id192, 1);
          mma_commit(&B->grud);
        }
        __syncwarp();
        mbar_wait(&B->hready, par, abortf);
        tc_fence_after_sync();
        if (lane == 0) {
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma_bf16(tmem + TM_Q, d_h + ks * k_a, d_W2 + ks * k_q, idq, ks > 0);
          mma_bf16(tmem + TM_Q, d_oh, d_W2 + 4 * k_q, idq, 1);
          mma_commit(&B->fc2d);
        }
        __syncwarp();
        ++it;
        if (s + 1 < p.T) issue_fc1();
      }
      mbar_wait(&B->stepd, sd & 1, abortf);  // last step of the tile
      ++sd;
    }
  } else if (warp == 9) {
    // =========================== copy warp: bulk loads of observations, bulk stores of records ==============
    // Observations of step i (counted over all tiles of this block) land in record buffer i & 1; they are
    // requested two steps ahead, as soon as the records of step i - 2 have been stored from that buffer.
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int e0 = tile * L.ept;
      const int ne = min(L.ept, p.E - e0);
      auto issue_loads = [&](int s, uint32_t b) {
        bulk_wait_read_all();  // this lane's earlier stores have left shared memory
        __syncwarp();
        const uint32_t env_bytes = (uint32_t)(n * D) * 4u, av_bytes = L.avail_bulk ? (uint32_t)(n * A) : 0u;
        if (lane == 0) mbar_arrive_expect_tx(&B->full[b], (env_bytes + av_bytes) * (uint32_t)ne);
        __syncwarp();
        const float* src = p.obs + (size_t)s * p.obs_step_stride + (size_t)e0 * n * D;
        const uint8_t* asrc = p.avail + (size_t)s * p.avail_step_stride + (size_t)e0 * n * A;
        for (int el = lane; el < ne; el += 32) {
          uint8_t* r = recs + b * buf_bytes + (uint32_t)el * rec_bytes;
          bulk_load(r, src + (size_t)el * n * D, env_bytes, &B->full[b]);
          if (av_bytes) bulk_load(r + p.rl.off_avail, asrc + (size_t)el * av_bytes, av_bytes, &B->full[b]);
        }
      };
      issue_loads(0, it & 1);
      if (p.T > 1) issue_loads(1, (it + 1) & 1);
      mbar_wait(&B->stepd, sd & 1, abortf);  // the tile prologue's phase
      ++sd;
      for (int s = 0; s < p.T; ++s) {
        const uint32_t b = it & 1;
        mbar_wait(&B->stepd, sd & 1, abortf);  // records of step s complete
        ++sd;
        for (int el = lane; el < ne; el += 32) {
          const unsigned long long dst = dst_s[b * TC_ROWS + el];
          if (dst) bulk_store(reinterpret_cast<void*>(dst), recs + b * buf_bytes + (uint32_t)el * rec_bytes, rec_bytes);
        }
        bulk_commit();
        if (s + 2 < p.T) issue_loads(s + 2, b);
        ++it;
      }
    }
    bulk_wait_all();
   } else if (L.avail_bulk) {
    // =========================== draw warps: availability mask and epsilon draw of every row ==============
    // Neither depends on the network, so two otherwise idle warps prepare them at the start of each step
    // from the availability bytes that arrived with the observations; epilogue 3 only reads the result.
    const int r0 = tid - 10 * 32;  // 0..63, rows r0 and r0 + 64
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int e0 = tile * L.ept;
      const int R = min(L.ept, p.E - e0) * n;
      for (int s = 0; s < p.T; ++s) {
        const uint32_t b = it & 1;
        mbar_wait(&B->stepd, sd & 1, abortf);  // prologue or previous step: the hand-off array is free again
        ++sd;
        mbar_wait(&B->full[b], (it >> 1) & 1, abortf);
        const uint32_t t = p.t0 + (uint32_t)s;
        const float eps = eps_at(p, t);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int r = r0 + 64 * u;
          if (r < R) {
            const int rel = r / n, rai = r - rel * n;
            const uint8_t* avd = recs + b * buf_bytes + (uint32_t)rel * rec_bytes + p.rl.off_avail + rai * A;
            uint32_t mask = 0;
            for (int a = 0; a < A; ++a) mask |= (avd[a] ? 1u : 0u) << a;
            int pick = -1;
            if (mask != 0) pick = draw_explore(mask, eps, p.seed, t, (uint32_t)(e0 + rel), (uint32_t)rai);
            sel_s[r] = make_uint2(mask, (uint32_t)pick);
          }
        }
        mbar_arrive(&B->selready);
        ++it;
      }
      mbar_wait(&B->stepd, sd & 1, abortf);  // last step of the tile
      ++sd;
    }
   }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(TC_REGS_EPILOGUE));
    // =========================== epilogue threads ===========================
    const int row = tid & 127, half = tid >> 7;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int el = row / n, ai = row - el * n;
    const int cb = half * 32;  // first hidden column of this thread
    const uint32_t inv_nchunk = 0xFFFFFFFFu / (uint32_t)L.nchunk + 1u;  // j / nchunk == umulhi(j, inv) for j < 2^16
    unsigned long long c_steps = 0, c_explore = 0, c_noavail = 0, c_episodes = 0, c_trunc = 0;
    uint32_t st_bits = 0;
    float h[32];

    // converts the observations of the record buffer `b` into the bf16 operand (threads of half 1)
    auto convert_x = [&](uint32_t b, int R) {
      const int items = TC_ROWS * L.nchunk;  // a multiple of 256: two items per pass keep four loads in flight
      const uint8_t* base = recs + b * buf_bytes;
      for (int j = row; j < items; j += 256) {
        float4 v[2][2];
        int rr[2], cc[2];
        bool on[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int jj = j + 128 * u;
          rr[u] = (int)__umulhi((uint32_t)jj, inv_nchunk);
          cc[u] = jj - rr[u] * L.nchunk;
          on[u] = rr[u] < R && cc[u] * 8 < D;
          if (on[u]) {
            const float4* src = reinterpret_cast<const float4*>(base + rowoff_s[rr[u]] + (uint32_t)cc[u] * 32u);
            v[u][0] = src[0];
            v[u][1] = src[1];
          }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          uint4 o = make_uint4(0, 0, 0, 0);
          if (on[u]) {
            o.x = pack_bf16x2(v[u][0].x, v[u][0].y);
            o.y = pack_bf16x2(v[u][0].z, v[u][0].w);
            o.z = pack_bf16x2(v[u][1].x, v[u][1].y);
            o.w = pack_bf16x2(v[u][1].z, v[u][1].w);
          }
          *reinterpret_cast<uint4*>(xy + (uint32_t)cc[u] * TC_LBO_X + (uint32_t)rr[u] * 16u) = o;
        }
      }
    };
    // one-hot operand tile of this thread's row: byte address of column k
    auto oh_col = [&](int k) { return oh + (uint32_t)(k >> 3) * TC_LBO_A + (uint32_t)row * 16u + (uint32_t)(k & 7) * 2u; };

    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int e0 = tile * L.ept;
      const int ne = min(L.ept, p.E - e0);
      const int R = ne * n;
      const bool live = row < R;
      const bool is_row = live && half == 0;             // owner of the row's choice
      const bool is_env = live && half == 1 && ai == 0;  // owner of the environment's cursor (half 1 has slack)
      const int e = e0 + el;
      const size_t grow = (size_t)e * n + ai;             // global row
      int32_t slot = 0, pos = 0, ok = 0, la = -1;
      long long epc = 0;
      uint32_t av_raw[32];      // availability bytes of the coming step (row owners)
      float reward_raw = 0.f;   // reward / done of the coming step (environment owners)
      uint32_t done_raw = 0;

      // ---- tile prologue ----
      {
        const float4* src = reinterpret_cast<const float4*>(p.h + grow * TC_H + cb);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 v = live ? src[q] : make_float4(0.f, 0.f, 0.f, 0.f);
          h[4 * q] = v.x; h[4 * q + 1] = v.y; h[4 * q + 2] = v.z; h[4 * q + 3] = v.w;
        }
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const uint4 o = make_uint4(pack_bf16x2(h[8 * cc], h[8 * cc + 1]), pack_bf16x2(h[8 * cc + 2], h[8 * cc + 3]),
                                     pack_bf16x2(h[8 * cc + 4], h[8 * cc + 5]), pack_bf16x2(h[8 * cc + 6], h[8 * cc + 7]));
          *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
        }
        if (half == 0) {
          reset_s[row] = 0;
          la_s[row] = live ? p.last_action[grow] : -1;
          for (int c = 0; c < L.ohc; ++c)
            *reinterpret_cast<uint4*>(oh + (uint32_t)c * TC_LBO_A + (uint32_t)row * 16u) = make_uint4(0, 0, 0, 0);
        }
        if (is_row) {
          la = p.last_action[grow];
          *reinterpret_cast<uint16_t*>(oh_col(0)) = 0x3F80;  // bf16 1.0: the three bias columns
          *reinterpret_cast<uint16_t*>(oh_col(1)) = 0x3F80;
          *reinterpret_cast<uint16_t*>(oh_col(2)) = 0x3F80;
          *reinterpret_cast<uint16_t*>(oh_col(3 + ai)) = 0x3F80;
          if (la >= A) la = -1;
          if (!L.avail_bulk) {
            const uint8_t* av = p.avail + grow * A;
#pragma unroll
            for (int a = 0; a < 32; ++a)
              if (a < A) av_raw[a] = av[a];
          }
        }
        if (is_env) {
          slot = p.slot[e];
          pos = p.pos[e];
          epc = p.ep_count[e];
          ok = (slot >= 0 && slot < p.E * p.S && pos >= 0 && pos < p.L) ? 1 : 0;
          if (!ok) st_bits |= MARL_STATUS_BAD_INDEX;
          reward_raw = p.reward[e];
          done_raw = p.done[e];
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        // fc1 of the tile's first step is issued as soon as the converted observations are ready (half 1 below);
        // it also reads the one-hot tile written above by half 0, so order the two halves first
        asm volatile("bar.sync 1, 256;" ::: "memory");
        mbar_arrive(&B->stepd);
        if (half == 1) {
          mbar_wait(&B->full[it & 1], (it >> 1) & 1, abortf);
          convert_x(it & 1, R);
          fence_proxy_async_smem();
          mbar_arrive(&B->xready);
        }
      }

      for (int s = 0; s < p.T; ++s) {
        const uint32_t b = it & 1, par = it & 1;
        const uint32_t t = p.t0 + (uint32_t)s;
        uint8_t* rec = recs + b * buf_bytes + (uint32_t)el * rec_bytes;  // this row's environment record

        // ---- epilogue 1: y = relu(fc1 + W1[:, last action]) -> bf16 operand.  Bias and agent-id column are
        //      inside the GEMM; fc1 itself finished during the previous step. ----
        mbar_wait(&B->fc1d, par, abortf);
        tc_fence_after_sync();
        {
          // both published before the previous step's closing barrier; an episode that just ended has no last action
          int last = reset_s[el] ? -1 : la_s[row];
          if (last >= A) last = -1;
          const float* tl = tab_la + (last >= 0 ? last : 0) * TC_TAB + cb;
#pragma unroll
          for (int c16 = 0; c16 < 2; ++c16) {
            uint32_t v[16];
            tmem_ld16(tmem + lane_addr + TM_FC1 + cb + c16 * 16, v);
            tmem_ld_wait();
            float y[16];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float4 l4 = make_float4(0.f, 0.f, 0.f, 0.f);
              if (last >= 0) l4 = *reinterpret_cast<const float4*>(tl + c16 * 16 + 4 * q);
              y[4 * q] = fmaxf(__uint_as_float(v[4 * q]) + l4.x, 0.f);
              y[4 * q + 1] = fmaxf(__uint_as_float(v[4 * q + 1]) + l4.y, 0.f);
              y[4 * q + 2] = fmaxf(__uint_as_float(v[4 * q + 2]) + l4.z, 0.f);
              y[4 * q + 3] = fmaxf(__uint_as_float(v[4 * q + 3]) + l4.w, 0.f);
            }
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              const uint4 o = make_uint4(pack_bf16x2(y[8 * cc], y[8 * cc + 1]), pack_bf16x2(y[8 * cc + 2], y[8 * cc + 3]),
                                         pack_bf16x2(y[8 * cc + 4], y[8 * cc + 5]), pack_bf16x2(y[8 * cc + 6], y[8 * cc + 7]));
              *reinterpret_cast<uint4*>(xy + (uint32_t)(half * 4 + c16 * 2 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
            }
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&B->yready);

        // ---- while the y-side gate products run: work that does not depend on the network - the environment's
        //      reward/done, record address and the requests for the next step's values ----
        uint32_t mask = 0;
        int pick = -1;
        float reward = 0.f;
        int done = 0;
        if (is_row && !L.avail_bulk) {
          // availability bytes fetched by this thread one step ahead (shapes whose rows cannot be bulk-copied)
          const float eps = eps_at(p, t);
          uint8_t* avd = rec + p.rl.off_avail + ai * A;
#pragma unroll
          for (int a = 0; a < 32; ++a)
            if (a < A) {
              asm volatile("" : "+r"(av_raw[a]));  // keeps the byte's use here, a whole step after its load
              mask |= (av_raw[a] ? 1u : 0u) << a;
              avd[a] = (uint8_t)av_raw[a];
            }
          if (s + 1 < p.T) {
            const uint8_t* av = p.avail + (size_t)(s + 1) * p.avail_step_stride + grow * A;
#pragma unroll
            for (int a = 0; a < 32; ++a)
              if (a < A) av_raw[a] = av[a];
          }
          if (mask != 0) pick = draw_explore(mask, eps, p.seed, t, (uint32_t)e, (uint32_t)ai);
        }
        if (is_env) {
          asm volatile("" : "+f"(reward_raw), "+r"(done_raw));
          reward = reward_raw;
          done = done_raw ? 1 : 0;
          if (s + 1 < p.T) {
            reward_raw = p.reward[(size_t)(s + 1) * p.env_step_stride + e];
            done_raw = p.done[(size_t)(s + 1) * p.env_step_stride + e];
          }
          unsigned long long dst = 0;
          if (ok) {
            dst = reinterpret_cast<unsigned long long>(p.ring + (size_t)slot * p.slot_stride + (size_t)pos * rec_bytes);
            if (pos == 0) {  // an episode opens in this slot
              p.slot_epid[slot] = epc * (long long)p.E + e;
              p.slot_len[slot] = 0;
              p.slot_complete[slot] = 0;
            }
          }
          dst_s[b * TC_ROWS + el] = dst;
        }

        // ---- epilogue 2: gate math, new hidden state (fp32 registers) and its bf16 operand.
        //      The r and z accumulators hold half the pre-activation: sigmoid(v) = 0.5 * tanh(v / 2) + 0.5 ----
        mbar_wait(&B->grud, par, abortf);
        tc_fence_after_sync();
#pragma unroll
        for (int c16 = 0; c16 < 2; ++c16) {
          uint32_t vr[16], vz[16], vi[16], vh[16];
          const uint32_t col = (uint32_t)(cb + c16 * 16);
          tmem_ld16(tmem + lane_addr + TM_R + col, vr);
          tmem_ld16(tmem + lane_addr + TM_Z + col, vz);
          tmem_ld16(tmem + lane_addr + TM_IN + col, vi);
          tmem_ld16(tmem + lane_addr + TM_HN + col, vh);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float rg = fmaf(0.5f, tanh_fast(__uint_as_float(vr[j])), 0.5f);
            const float zg = fmaf(0.5f, tanh_fast(__uint_as_float(vz[j])), 0.5f);
            const float cand = tanh_fast(fmaf(rg, __uint_as_float(vh[j]), __uint_as_float(vi[j])));
            const float hp = h[c16 * 16 + j];
            h[c16 * 16 + j] = fmaf(zg, hp - cand, cand);  // (1 - z) * cand + z * h
          }
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const float* hv = h + c16 * 16 + 8 * cc;
            const uint4 o = make_uint4(pack_bf16x2(hv[0], hv[1]), pack_bf16x2(hv[2], hv[3]), pack_bf16x2(hv[4], hv[5]),
                                       pack_bf16x2(hv[6], hv[7]));
            *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 4 + c16 * 2 + cc) * TC_LBO_A + (uint32_t)row * 16u) = o;
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&B->hready);

        // ---- epilogue 3: half 0 chooses and records; half 1 prepares the next step's operand ----
        if (half == 0) {
          mbar_wait(&B->fc2d, par, abortf);
          tc_fence_after_sync();
          uint32_t qv[NQ];
          tmem_ld16(tmem + lane_addr + TM_Q, *reinterpret_cast<uint32_t(*)[16]>(qv));
          if (NQ == 32) tmem_ld16(tmem + lane_addr + TM_Q + 16, *reinterpret_cast<uint32_t(*)[16]>(qv + NQ - 16));
          tmem_ld_wait();
          tc_fence_before_sync();
          if (is_row && L.avail_bulk) {
            mbar_wait(&B->selready, par, abortf);
            const uint2 sp = sel_s[row];
            mask = sp.x;
            pick = (int)sp.y;
          }
          if (is_row) {
            // greedy rule on registers: m = max over available, thr = m - 1e-4f, lowest available a with Q >= thr.
            // Unavailable (and padding) entries become -inf; NaN never compares greater or equal.
            // Written as independent operations and a reduction tree: one thread, so instruction-level
            // parallelism is all there is.  fmaxf ignores a NaN operand, like the "greater than" scan it replaces.
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
            float* qrow = reinterpret_cast<float*>(rec + p.rl.off_q) + ai * A;
            if ((A & 1) == 0) {  // rows of an even number of floats start on 8-byte boundaries
#pragma unroll
              for (int a = 0; a < NQ; a += 2)
                if (a < A) *reinterpret_cast<float2*>(qrow + a) = make_float2(__uint_as_float(qv[a]), __uint_as_float(qv[a + 1]));
            } else {
#pragma unroll
              for (int a = 0; a < NQ; ++a)
                if (a < A) qrow[a] = __uint_as_float(qv[a]);
            }
            reinterpret_cast<int32_t*>(rec + p.rl.off_action)[ai] = act;
            const int tk = p.trace_first + s;
            if (tk < p.trace_cap) {
              const size_t trow = ((size_t)tk * p.E + e) * n + ai;
              if (p.trace_actions) p.trace_actions[trow] = act;
              if (p.trace_q)
                for (int a = 0; a < A; ++a) p.trace_q[trow * A + a] = qrow[a];
            }
            if (p.actions_out && s == p.T - 1) p.actions_out[grow] = act;
          }
        } else {
          if (is_env) {
            int closed = 0;
            if (ok) {
              *reinterpret_cast<float*>(rec + p.rl.off_reward) = reward;
              rec[p.rl.off_done] = (uint8_t)done;
              if (done || pos + 1 == p.L) {
                p.slot_len[slot] = pos + 1;
                p.slot_complete[slot] = 1;
                c_episodes += 1;
                if (!done) c_trunc += 1;
                epc += 1;
                slot = e * p.S + (int)(epc % p.S);
                pos = 0;
                closed = 1;
              } else {
                pos += 1;
              }
            }
            reset_s[el] = closed;
          }
          if (s + 1 < p.T) {
            mbar_wait(&B->full[b ^ 1], ((it + 1) >> 1) & 1, abortf);
            convert_x(b ^ 1, R);
            fence_proxy_async_smem();
            mbar_arrive(&B->xready);
          }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // ---- a closed episode restarts from a zero hidden state and no last action ----
        if (live && reset_s[el]) {
#pragma unroll
          for (int j = 0; j < 32; ++j) h[j] = 0.f;
#pragma unroll
          for (int cc = 0; cc < 4; ++cc)
            *reinterpret_cast<uint4*>(hb + (uint32_t)(half * 4 + cc) * TC_LBO_A + (uint32_t)row * 16u) = make_uint4(0, 0, 0, 0);
          if (half == 0) la = -1;
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&B->stepd);
        ++it;
      }

      // ---- tile epilogue: state back to global memory ----
      if (live) {
        float4* dsth = reinterpret_cast<float4*>(p.h + grow * TC_H + cb);
#pragma unroll
        for (int q = 0; q < 8; ++q) dsth[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
      }
      if (is_row) p.last_action[grow] = la;
      if (is_env && ok) {
        p.slot[e] = slot;
        p.pos[e] = pos;
        p.ep_count[e] = epc;
        if (pos > 0) p.slot_len[slot] = pos;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");  // reset_s is rewritten by the next tile's prologue
    }
    if (c_steps) atomicAdd(p.counters + CNT_AGENT_STEPS, c_steps);
    if (c_explore) atomicAdd(p.counters + CNT_EXPLORED, c_explore);
    if (c_noavail) atomicAdd(p.counters + CNT_NO_AVAIL, c_noavail);
    if (c_episodes) atomicAdd(p.counters + CNT_EPISODES, c_episodes);
    if (c_trunc) atomicAdd(p.counters + CNT_TRUNCATED, c_trunc);
    if (st_bits) atomicOr(p.status, st_bits);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && B->abort) {
    atomicOr(p.status, MARL_STATUS_TIMEOUT);
    // diagnosis: which barrier (index inside the barrier block) and which warp gave up first
    atomicCAS(p.status + 1, 0u, ((((B->abort & 0xFFFFFu) - (smem_u32(B) & 0xFFFFFu)) >> 3) & 0xFFu) | (((B->abort >> 20) & 0xFFu) << 8));
  }
  if (warp == 8) tmem_dealloc(tmem, TM_COLS);
}

// Returns the number of kernels launched or a negative cudaError.
int launch_actor_tc(const ActorParams& p, int sms, cudaStream_t stream) {
  TcLayout L = tc_layout(p.n, p.D, p.A, (int)p.rl.rec_bytes);
  if (reinterpret_cast<uintptr_t>(p.obs) % 16) return -(int)cudaErrorMisalignedAddress;
  // availability bytes ride with the observation copies when every environment's block is 16-byte sized and
  // aligned; otherwise the row threads fetch them one step ahead
  L.avail_bulk = ((p.n * p.A) % 16 == 0 && reinterpret_cast<uintptr_t>(p.avail) % 16 == 0) ? 1 : 0;
  auto kernel = L.NQ == 16 ? actor_tc_kernel<16> : actor_tc_kernel<32>;
  static uint32_t configured[2][SMEM_OPTIN_DEVICES];
  {
    const cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L.total, configured[L.NQ == 16 ? 0 : 1]);
    if (e != cudaSuccess) return -(int)e;
  }
  int grid = p.num_tiles < sms ? p.num_tiles : sms;
  if (grid < 1) grid = 1;
  kernel<<<grid, TC_THREADS, L.total, stream>>>(p, L);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? 1 : -(int)err;
}

}  // namespace marl
