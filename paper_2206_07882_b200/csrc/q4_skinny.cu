// Weight-streaming LSTM step for a handful of rows (one utterance: at most 32 hypothesis rows,
// the regime of the paper's run-time study, Section 4.1).  With so few rows the step is bound by
// reading the weights once, so they are read as stored: packed 4-bit codes, 128-bit loads, no int8
// copies, no staging through shared memory.
//
// One CTA owns the 16 weight rows of 4 cells (their i, f, g, o rows); its 8 warps split K in chunks
// of 128 codes (the input part, then the recurrent part).  A lane loads 16 bytes (32 codes) of two
// weight rows and of one activation row per 8-row tile and chunk and turns every 32-bit word (8 codes)
// into two operand registers of the warp-level int8 MMA m16n8k32 by two masks and a shift: the
// even-numbered codes of the word, each in the high nibble of a byte (16 x code), and the odd-numbered
// ones.  Weights and activations are split the same way, so a weight code always meets the activation
// code of its own K index; which K index an MMA lane position stands for is immaterial to a dot
// product.  The accumulators are 256 x the true sums (|256 w x| <= 2^15 per product, K <= 2^12: no
// overflow).  Unsigned activation codes (the LM input quantizer, Eq. 2) enter as unsigned bytes; the
// zero point is taken out afterwards with the row sums of the weights, which a second MMA against an
// all-ones operand accumulates on the way.  Partial sums of the 8 warps meet in shared memory, then
// 32 to 128 threads de-quantize, apply the gates, update the cell state, quantize the cell output once
// (Sections 3.2, 3.4) and store codes, int8 codes for the projection kernels, and cell state.
#include <string.h>

#include "q4_internal.h"

namespace q4 {

constexpr int SK_WARPS = 8;
constexpr int SK_THREADS = 32 * SK_WARPS;

__device__ __forceinline__ void mma_s8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_s8u8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NT>
__global__ void __launch_bounds__(SK_THREADS) k_skinny_lstm(const SkinnyLstmArgs a) {
  // partial sums: [warp][part: input, recurrent][16 tile rows][8 NT rows], and the weight row sums
  __shared__ int part[SK_WARPS][2][16][8 * NT];
  __shared__ int wsum[SK_WARPS][16];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int e = g & 1, ci = g >> 1;
  const int H = a.H;
  const int cell0 = 4 * blockIdx.x;
  // tile row g = gate e of cell ci, tile row g + 8 = gate 2 + e of the same cell
  const long long r0 = (long long)e * H + cell0 + ci, r1 = (long long)(2 + e) * H + cell0 + ci;
  const int nxc = a.Kx >> 7, nhc = H >> 7;

  pdl_wait();   // nothing produced by an earlier kernel is read before this
  int n_act = a.N;
  if (a.n_active) n_act = min(n_act, *a.n_active);
  if (n_act <= 0) return;

  // activation row pointers of this lane: row 8 j + g of every tile (nullptr: no such row / zero state)
  const uint8_t* xrow[NT];
  const uint8_t* hrow[NT];
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const int n = 8 * j + g;
    xrow[j] = hrow[j] = nullptr;
    if (n < n_act && (a.dst_row ? a.dst_row[n] : n) >= 0) {
      const int xi = a.x_idx ? a.x_idx[n] : n;
      if (xi >= 0) xrow[j] = a.x + (long long)xi * a.x_stride;
      const int hi = a.src_row ? a.src_row[n] : n;
      if (hi >= 0) hrow[j] = a.hq_in + (long long)hi * (H >> 1);
    }
  }
  int acc[2][NT][4];
  int accs[4] = {0, 0, 0, 0};
#pragma unroll
  for (int p = 0; p < 2; ++p)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[p][j][r] = 0;
  const uint32_t M = 0xF0F0F0F0u;
  const bool x_unsigned = a.x_signed == 0;

  for (int q = warp; q < nxc + nhc; q += SK_WARPS) {
    const bool is_x = q < nxc;
    const int kb = ((is_x ? q : q - nxc) << 6) + 16 * t4;   // byte offset of this lane's 32 codes in a row
    const uint8_t* wbase = is_x ? a.w_ih : a.w_hh;
    const long long wpitch = is_x ? (a.Kx >> 1) : (H >> 1);
    const uint4 wa = *reinterpret_cast<const uint4*>(wbase + r0 * wpitch + kb);
    const uint4 wb = *reinterpret_cast<const uint4*>(wbase + r1 * wpitch + kb);
    uint4 xb[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const uint8_t* p = is_x ? xrow[j] : hrow[j];
      xb[j] = p ? *reinterpret_cast<const uint4*>(p + kb) : make_uint4(0, 0, 0, 0);
    }
    const uint32_t aw[4] = {wa.x, wa.y, wa.z, wa.w}, bw[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t a0 = (aw[i] << 4) & M, a2 = aw[i] & M, a1 = (bw[i] << 4) & M, a3 = bw[i] & M;
      if (is_x && x_unsigned) {
        mma_s8u8(accs, a0, a1, a2, a3, 0x01010101u, 0x01010101u);
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const uint32_t w = i == 0 ? xb[j].x : i == 1 ? xb[j].y : i == 2 ? xb[j].z : xb[j].w;
          mma_s8u8(acc[0][j], a0, a1, a2, a3, (w << 4) & M, w & M);
        }
      } else {
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const uint32_t w = i == 0 ? xb[j].x : i == 1 ? xb[j].y : i == 2 ? xb[j].z : xb[j].w;
          if (is_x)
            mma_s8s8(acc[0][j], a0, a1, a2, a3, (w << 4) & M, w & M);
          else
            mma_s8s8(acc[1][j], a0, a1, a2, a3, (w << 4) & M, w & M);
        }
      }
    }
  }
  pdl_trigger();
  // fragment (g, t4): rows g and g + 8, columns 2 t4 and 2 t4 + 1 of each tile
#pragma unroll
  for (int p = 0; p < 2; ++p)
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      part[warp][p][g][8 * j + 2 * t4] = acc[p][j][0];
      part[warp][p][g][8 * j + 2 * t4 + 1] = acc[p][j][1];
      part[warp][p][g + 8][8 * j + 2 * t4] = acc[p][j][2];
      part[warp][p][g + 8][8 * j + 2 * t4 + 1] = acc[p][j][3];
    }
  if (t4 == 0) {
    wsum[warp][g] = accs[0];
    wsum[warp][g + 8] = accs[2];
  }
  __syncthreads();
  if (tid >= 32 * NT) return;
  // item: cell c of the CTA's 4, row n
  const int c = tid & 3, n = tid >> 2;
  const int dst = (n < n_act) ? (a.dst_row ? a.dst_row[n] : n) : -1;
  int q = 0;
  if (dst >= 0) {
    const int cell = cell0 + c;
    float pre[4];
#pragma unroll
    for (int gate = 0; gate < 4; ++gate) {
      const int r = gate < 2 ? 2 * c + gate : 8 + 2 * c + (gate - 2);
      int ih = 0, hh = 0, ws = 0;
#pragma unroll
      for (int w = 0; w < SK_WARPS; ++w) {
        ih += part[w][0][r][n];
        hh += part[w][1][r][n];
        ws += wsum[w][r];
      }
      if (x_unsigned) ih -= 16 * a.x_zp * ws;   // 256 sum w (x - z) = 256 sum w x - 16 z (16 sum w)
      ih >>= 8;                                // both operands were 16 x code
      hh >>= 8;
      const long long row = (long long)gate * H + cell;
      const float b = a.bias ? a.bias[row] : 0.0f;
      const float v = __fmaf_rn((float)ih, __fmul_rn(a.x_scale, a.s_wih[row]), b);
      pre[gate] = __fmaf_rn((float)hh, __fmul_rn(a.hid_act.scale, a.s_whh[row]), v);
    }
    const int src = a.src_row ? a.src_row[n] : n;
    const float cprev = src >= 0 ? a.c_in[(long long)src * H + cell] : 0.0f;
    float cn, hn;
    cell_fixed(pre[0], pre[1], pre[2], pre[3], cprev, cn, hn);
    a.c_out[(long long)dst * H + cell] = cn;
    q = quantize1(hn, a.hid_act.inv_scale, a.hid_act.zero_point, act_lo(a.hid_act), act_hi(a.hid_act));
    if (a.h8_out) a.h8_out[(long long)n * a.h8_ld + cell] = (int8_t)q;
  }
  // two cells per byte: the even cell's thread writes
  const int qn = __shfl_down_sync(0xffffffffu, q, 1);
  if (dst >= 0 && (c & 1) == 0 && a.hq_out)
    a.hq_out[(long long)dst * (H >> 1) + ((cell0 + c) >> 1)] = (uint8_t)((q & 0xF) | ((qn & 0xF) << 4));
}

bool skinny_lstm_supported(int N, int H, int Kx, int w_bits_ih, int w_bits_hh, const q4_act& x_act,
                           const q4_act& hid_act) {
  return N >= 1 && N <= 32 && H % 128 == 0 && Kx % 128 == 0 && w_bits_ih == 4 && w_bits_hh == 4 && x_act.bits == 4 &&
         hid_act.bits == 4 && hid_act.is_signed && H <= 4096 && Kx <= 4096;
}

cudaError_t launch_skinny_lstm(const SkinnyLstmArgs& a, cudaStream_t s, bool dependent) {
  if (a.N <= 0) return cudaSuccess;
  const dim3 grid(a.H / 4), block(SK_THREADS);
  timing_begin(s);
  cudaError_t e;
  if (a.N <= 8)
    e = launch_ex(k_skinny_lstm<1>, grid, block, 0, s, dependent, 1, a);
  else if (a.N <= 16)
    e = launch_ex(k_skinny_lstm<2>, grid, block, 0, s, dependent, 1, a);
  else
    e = launch_ex(k_skinny_lstm<4>, grid, block, 0, s, dependent, 1, a);
  timing_end(s);
  ++g_launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace q4
