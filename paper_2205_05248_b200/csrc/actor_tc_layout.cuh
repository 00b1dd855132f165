// Layout shared by the tensor-core actor kernels: the packed weight image (bf16 matrices in the operand
// layout of tcgen05.mma, fp32 tables), tensor-memory columns, and the shared-memory plan of the one-tile kernel.
#pragma once

#include <cstring>

#include "common.cuh"

namespace marl {

constexpr int TC_ROWS = 128;
constexpr int TC_H = 64;
constexpr int TC_EPI_THREADS = 256;
constexpr int TC_THREADS = 384;  // two epilogue warpgroups + one service warpgroup (MMA warp, copy warp, two idle)
// Register split after start-up (setmaxnreg): the block is launched with 168 registers per thread
// (384 * 168 = 64512); the service warpgroup drops to 88 and each epilogue warpgroup rises to 208:
// 256 * 208 + 128 * 88 = 64512, exactly the launch total.
constexpr int TC_REGS_EPILOGUE = 208, TC_REGS_SERVICE = 88;
constexpr int TC_TAB = 68;                 // row stride (floats) of the last-action table: conflict-free float4 rows
constexpr uint32_t TC_LBO_A = 2048;        // k-chunk stride of a 128-row operand
constexpr uint32_t TC_LBO_X = 2048 + 16;   // padded for the observation operand: spreads the converter's stores
constexpr uint32_t TC_SMEM_MAX = 232448;   // 227 KB opt-in limit per block
// tensor-memory columns
constexpr uint32_t TM_FC1 = 0, TM_R = 64, TM_Z = 128, TM_IN = 192, TM_HN = 256, TM_Q = 320, TM_COLS = 512;

struct TcLayout {
  int32_t Dk, NQ, nchunk, ept, ohK, ohc, avail_bulk, pad_;
  // packed weight image (same offsets in global and shared memory)
  uint32_t off_W1, off_Wih, off_Whh, off_Bg, off_Bhn, off_W2, off_tab_la, wbytes;
  // shared memory only
  uint32_t off_xy, off_hb, off_oh, off_rec, off_dst, off_reset, off_la, off_rowoff, off_sel, off_bar, total;
};

// Operand K-columns beyond the data columns ("extension"): the fp32 biases and the two one-hot parts of
// the network input enter the GEMMs as extra K columns, so the epilogues add nothing.
//   one-hot operand tile (A side, per row, constant for a tile):  col 0..2 = 1, col 3+i = [agent == i]
//   fc1 weights (B side):    k = Dk+0..2: b1 split into three bf16 pieces (their sum is b1 to fp32 accuracy),
//                            k = Dk+3+i: W1[:, D+i]
//   gate-bias tile, candidate-hidden-bias tile and W2: bias pieces at k = 0..2 (resp. 64..66), multiplied by
//   the three ones of the one-hot tile; all other extension entries are zero.
// The last-action one-hot is the only input that depends on the previous step's choice; keeping it out of the
// GEMM lets fc1 of step s+1 run entirely during step s.  Its term W1[:, D+n+last] is added in epilogue 1 from
// a small fp32 table.
// The reset and update rows of W_ih / W_hh and their biases are stored halved (exact in bf16), so that
// sigmoid(v) = 0.5 * tanh(v / 2) + 0.5 needs no multiply in the epilogue.
static inline uint32_t up16(uint32_t v) { return (v + 15u) & ~15u; }

static inline TcLayout tc_layout(int n, int D, int A, int rec_bytes) {
  TcLayout L;
  memset(&L, 0, sizeof(L));
  L.Dk = (D + 15) & ~15;
  L.NQ = A <= 16 ? 16 : 32;
  L.nchunk = L.Dk / 8;
  L.ept = TC_ROWS / n;
  L.ohK = (3 + n + 15) & ~15;
  L.ohc = L.ohK / 8;
  uint32_t o = 0;
  L.off_W1 = o; o += (uint32_t)(L.nchunk + L.ohc) * TC_H * 16;
  L.off_Wih = o; o += 8u * 3 * TC_H * 16;
  L.off_Whh = o; o += 8u * 3 * TC_H * 16;
  L.off_Bg = o; o += 2u * 3 * TC_H * 16;   // gate biases: r, z (both sides summed, halved) and the candidate's input bias
  L.off_Bhn = o; o += 2u * TC_H * 16;      // the candidate's hidden bias
  L.off_W2 = o; o += 10u * L.NQ * 16;
  L.off_tab_la = o; o += up16(sizeof(float) * A * TC_TAB);  // W1[:, D+n+a] as fp32 rows: the last-action term
  L.wbytes = o;
  const uint32_t xbytes = (uint32_t)L.nchunk * TC_LBO_X;
  L.off_xy = o; o += up16(xbytes > 8 * TC_LBO_A ? xbytes : 8 * TC_LBO_A);
  L.off_hb = o; o += 8 * TC_LBO_A;
  L.off_oh = o; o += (uint32_t)L.ohc * TC_LBO_A;
  L.off_rec = o; o += 2u * L.ept * (uint32_t)rec_bytes;
  L.off_dst = o; o += 2u * TC_ROWS * 8;
  L.off_reset = o; o += TC_ROWS * 4;
  L.off_la = o; o += TC_ROWS * 4;
  L.off_rowoff = o; o += TC_ROWS * 4;
  L.off_sel = o; o += TC_ROWS * 8;
  L.off_bar = o; o += 128;
  L.total = o;
  return L;
}

static inline int rec_bytes_of(int n, int D, int A) {
  auto up = [](size_t v) { return (v + 15) / 16 * 16; };
  return (int)(up(4 * (size_t)n * D) + up((size_t)n * A) + up(4 * (size_t)n) + up(4 * (size_t)n * A) + 16);
}


__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

}  // namespace marl
