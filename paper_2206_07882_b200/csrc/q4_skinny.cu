// Weight-streaming LSTM step for a handful of rows (one utterance: at most 32 hypothesis rows,
// the regime of the paper's run-time study, Section 4.1).  With so few rows the step is bound by
// reading the weights once, so they are read as stored: packed 4-bit codes, 128-bit loads, no int8
// copies, no staging through shared memory.
//
// One CTA owns the 16 weight rows of 4 cells (their i, f, g, o rows); its 16 warps split K in chunks
// of 128 codes (the input part, then the recurrent part); a warp fetches its next chunk while it
// multiplies the present one.  Four CTAs fit an SM, so all CTAs of a layer (at most 512) are resident
// together and the whole weight matrix is requested within the first microsecond.  A lane loads 16 bytes (32 codes) of two
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
constexpr int SK_CTAS_PER_SM = 4;   // registers are capped so that every CTA of a layer is resident at once

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

__device__ __forceinline__ void cp_async4(float* dst_smem, const float* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src)
               : "memory");
}

template <int NT>
__global__ void __launch_bounds__(SK_THREADS, NT == 4 ? 2 : SK_CTAS_PER_SM) k_skinny_lstm(const SkinnyLstmArgs a) {
  // partial sums: [warp][part: input, recurrent][16 tile rows][8 NT rows], and the weight row sums
  extern __shared__ __align__(16) int sk_smem[];
  int (*part)[2][16][8 * NT] = reinterpret_cast<int (*)[2][16][8 * NT]>(sk_smem);
  int (*wsum)[16] = reinterpret_cast<int (*)[16]>(sk_smem + SK_WARPS * 2 * 16 * 8 * NT);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int e = g & 1, ci = g >> 1;
  const int H = a.H;
  const int cell0 = 4 * blockIdx.x;
  // tile row g = gate e of cell ci, tile row g + 8 = gate 2 + e of the same cell
  const long long r0 = (long long)e * H + cell0 + ci, r1 = (long long)(2 + e) * H + cell0 + ci;
  const int nxc = a.Kx >> 7, nhc = H >> 7;
  const uint32_t M = 0xF0F0F0F0u;
  const bool x_unsigned = a.x_signed == 0;

  // the de-quantization constants of the thread's item of the closing stage (cell ec of the CTA's 4,
  // row en) do not depend on the previous kernel of the stream: they are sent on their way to shared
  // memory first (row scales and bias of the item's four gate rows; no registers are held for them)
  const int ec = tid & 3, en = tid >> 2;
  float* ecst = reinterpret_cast<float*>(sk_smem + SK_WARPS * 2 * 16 * 8 * NT + SK_WARPS * 16);   // [12][32 NT]
  if (tid < 32 * NT) {
#pragma unroll
    for (int gate = 0; gate < 4; ++gate) {
      const long long row = (long long)gate * H + cell0 + ec;
      cp_async4(ecst + (gate * 3 + 0) * 32 * NT + tid, a.s_wih + row);
      cp_async4(ecst + (gate * 3 + 1) * 32 * NT + tid, a.s_whh + row);
      if (a.bias) cp_async4(ecst + (gate * 3 + 2) * 32 * NT + tid, a.bias + row);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  pdl_wait();   // nothing produced by an earlier kernel is read before this
  // row bookkeeping: every index is requested at once (the arrays hold an entry for each of the N launch
  // rows), the count of rows with work only masks them afterwards
  int n_act = a.N;
  int xrow[NT], hrow[NT], drow[NT];   // row indices of this lane's rows 8 j + g, negative = none
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const int n = 8 * j + g;
    const bool in = n < a.N;
    drow[j] = in ? (a.dst_row ? a.dst_row[n] : n) : -1;
    xrow[j] = in ? (a.x_idx ? a.x_idx[n] : n) : -1;
    hrow[j] = in ? (a.src_row ? a.src_row[n] : n) : -1;
  }
  int e_dst = -1, e_src = -1;
  if (tid < 32 * NT && en < a.N) {
    e_dst = a.dst_row ? a.dst_row[en] : en;
    e_src = a.src_row ? a.src_row[en] : en;
  }
  if (a.n_active) n_act = min(n_act, *a.n_active);
  if (n_act <= 0) return;
#pragma unroll
  for (int j = 0; j < NT; ++j)
    if (8 * j + g >= n_act || drow[j] < 0) xrow[j] = hrow[j] = -1;
  // the item's parent cell state, fetched beside the main loop
  float e_cprev = 0.0f;
  if (en >= n_act) e_dst = -1;
  if (e_dst >= 0 && e_src >= 0) e_cprev = a.c_in[(long long)e_src * H + cell0 + ec];

  // activation row pointers of this lane: row 8 j + g of every tile (nullptr: no such row / zero state)
  int acc[2][NT][4];
  int accs[4] = {0, 0, 0, 0};
#pragma unroll
  for (int p = 0; p < 2; ++p)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[p][j][r] = 0;

  // chunk q of this warp: weight pieces of two rows and activation pieces of NT rows, 16 bytes each
  auto fetch = [&](int q, uint4& wa, uint4& wb, uint4 (&xb)[NT]) {
    wa = wb = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int j = 0; j < NT; ++j) xb[j] = make_uint4(0, 0, 0, 0);
    if (q >= nxc + nhc) return;
    const bool is_x = q < nxc;
    const int kb = ((is_x ? q : q - nxc) << 6) + 16 * t4;   // byte offset of this lane's 32 codes in a row
    const uint8_t* wbase = is_x ? a.w_ih : a.w_hh;
    const long long wpitch = is_x ? (a.Kx >> 1) : (H >> 1);
    wa = *reinterpret_cast<const uint4*>(wbase + r0 * wpitch + kb);
    wb = *reinterpret_cast<const uint4*>(wbase + r1 * wpitch + kb);
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int r = is_x ? xrow[j] : hrow[j];
      if (r >= 0)
        xb[j] = *reinterpret_cast<const uint4*>((is_x ? a.x + (long long)r * a.x_stride : a.hq_in + (long long)r * (H >> 1)) + kb);
    }
  };
  uint4 wa, wb, xb[NT];
  fetch(warp, wa, wb, xb);
  for (int q = warp; q < nxc + nhc; q += SK_WARPS) {
    const bool is_x = q < nxc;
    const uint32_t aw[4] = {wa.x, wa.y, wa.z, wa.w}, bw[4] = {wb.x, wb.y, wb.z, wb.w};
    uint32_t xw[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      xw[j][0] = xb[j].x;
      xw[j][1] = xb[j].y;
      xw[j][2] = xb[j].z;
      xw[j][3] = xb[j].w;
    }
    fetch(q + SK_WARPS, wa, wb, xb);   // the next chunk is on its way while this one is multiplied
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t a0 = (aw[i] << 4) & M, a2 = aw[i] & M, a1 = (bw[i] << 4) & M, a3 = bw[i] & M;
      if (is_x && x_unsigned) {
        mma_s8u8(accs, a0, a1, a2, a3, 0x01010101u, 0x01010101u);
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_s8u8(acc[0][j], a0, a1, a2, a3, (xw[j][i] << 4) & M, xw[j][i] & M);
      } else if (is_x) {
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_s8s8(acc[0][j], a0, a1, a2, a3, (xw[j][i] << 4) & M, xw[j][i] & M);
      } else {
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_s8s8(acc[1][j], a0, a1, a2, a3, (xw[j][i] << 4) & M, xw[j][i] & M);
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
  asm volatile("cp.async.wait_all;" ::: "memory");   // this thread's constants have landed
  // item: cell c of the CTA's 4, row n
  const int c = ec, n = en;
  const int dst = e_dst;
  int q = 0;
  if (dst >= 0) {
    const int cell = cell0 + c;
    float pre[4];
#pragma unroll
    for (int gate = 0; gate < 4; ++gate) {
      const int r = gate < 2 ? 2 * c + gate : 8 + 2 * c + (gate - 2);
      int ih = 0, hh = 0, ws = 0;
#pragma unroll 4
      for (int w = 0; w < SK_WARPS; ++w) {
        ih += part[w][0][r][n];
        hh += part[w][1][r][n];
        ws += wsum[w][r];
      }
      if (x_unsigned) ih -= 16 * a.x_zp * ws;   // 256 sum w (x - z) = 256 sum w x - 16 z (16 sum w)
      ih >>= 8;                                // both operands were 16 x code
      hh >>= 8;
      const float sih = ecst[(gate * 3 + 0) * 32 * NT + tid], shh = ecst[(gate * 3 + 1) * 32 * NT + tid];
      const float bi = a.bias ? ecst[(gate * 3 + 2) * 32 * NT + tid] : 0.0f;
      const float v = __fmaf_rn((float)ih, __fmul_rn(a.x_scale, sih), bi);
      pre[gate] = __fmaf_rn((float)hh, __fmul_rn(a.hid_act.scale, shh), v);
    }
    float cn, hn;
    cell_fixed(pre[0], pre[1], pre[2], pre[3], e_cprev, cn, hn);
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
  auto smem = [](int nt) { return (size_t)(SK_WARPS * 2 * 16 * 8 * nt + SK_WARPS * 16 + 12 * 32 * nt) * sizeof(int); };
  static bool configured = false;
  if (!configured) {
    cudaError_t ce = cudaFuncSetAttribute(k_skinny_lstm<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem(4));
    if (ce != cudaSuccess) return ce;
    configured = true;
  }
  timing_begin(s);
  cudaError_t e;
  if (a.N <= 8)
    e = launch_ex(k_skinny_lstm<1>, grid, block, smem(1), s, dependent, 1, a);
  else if (a.N <= 16)
    e = launch_ex(k_skinny_lstm<2>, grid, block, smem(2), s, dependent, 1, a);
  else
    e = launch_ex(k_skinny_lstm<4>, grid, block, smem(4), s, dependent, 1, a);
  timing_end(s);
  ++g_launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace q4
