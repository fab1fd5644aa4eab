// Persistent encoder recurrence (Sections 3.2, 3.4): one launch runs all T steps of a layer.
//
// A cluster of 8 CTAs owns one (direction, batch group of BG sequences): CTA r keeps the
// recurrent weights of cells [r*H/8, (r+1)*H/8) (all four gates, int8, rows 4*cell+gate) in
// shared memory for the whole sequence, the cell state of its (cell, sequence) pairs in
// registers, and a double-buffered copy of the group's hidden codes h_{t-1} [BG, H] in shared
// memory.  Per step: warp w multiplies its 16 weight rows (4 cells) with h_{t-1} by warp-level
// int8 MMAs (m16n8k32, A fragments by ldmatrix from the resident weights), the four gate
// accumulators of every (cell, sequence) pair are brought into one lane by shuffles, that lane
// de-quantizes, applies the gates, updates its cell state, and quantizes the cell output once;
// the new codes are stored into the hidden buffers of all 8 CTAs through distributed shared
// memory, and one hardware cluster barrier ends the step.  Nothing is exchanged through global
// memory and no flag is polled.  The input contribution acc_ih (all frames, from the
// tensor-core GEMM) is prefetched at the top of each step.
#include <string.h>

#include "q4_internal.h"
#include "q4_mma.cuh"

namespace q4 {

constexpr int REC_CLUSTER = 8;
constexpr int REC_THREADS = 640;   // 20 warps: warp w owns weight rows 16w..16w+15 = 4 cells

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}
// Four 8x8 matrices of 16-bit elements = a 16 x 32 int8 A fragment.
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& a0, uint32_t& a1, uint32_t& a2,
                                            uint32_t& a3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t& a0, uint32_t& a1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(a0), "=r"(a1) : "r"(addr));
}
// c[16 x 8] += A[16 x 32] * B[32 x 8], signed 8-bit operands, int32 accumulate.
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                       uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int BG>
__global__ void __cluster_dims__(REC_CLUSTER, 1, 1) __launch_bounds__(REC_THREADS, 1)
k_enc_recurrent(const EncRecArgs a) {
  extern __shared__ __align__(16) uint8_t rec_smem[];
  constexpr int NT = BG / 8;                // 8-sequence MMA tiles = items finalised per lane
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const int cid = blockIdx.x / REC_CLUSTER;
  const int d = cid / a.n_groups, grp = cid % a.n_groups;
  const EncRecDir& D = a.d[d];
  const int H = a.H, T = a.T, B = a.B;
  const int cpc = H / REC_CLUSTER;          // cells per CTA
  const int rows = 4 * cpc;
  const int pitch = H + 16;                 // pitch % 128 == 16: ldmatrix rows and B words conflict-free
  int8_t* Ws = reinterpret_cast<int8_t*>(rec_smem);
  int8_t* hb = Ws + (size_t)rows * pitch;   // [2][BG][pitch]
  int8_t* stage = hb + (size_t)2 * BG * pitch;  // [BG][cpc] this CTA's new codes before the broadcast

  // resident weights: rows 4*cell+gate of this CTA's cells
  {
    const int per_row = H >> 4;
    const int8_t* src = D.w_hh + (size_t)rank * rows * H;
    for (int i = tid; i < rows * per_row; i += REC_THREADS) {
      const int r = i / per_row, c = i % per_row;
      *reinterpret_cast<uint4*>(Ws + (size_t)r * pitch + c * 16) =
          *reinterpret_cast<const uint4*>(src + (size_t)r * H + c * 16);
    }
    for (int i = tid; i < 2 * BG * pitch / 16; i += REC_THREADS)
      reinterpret_cast<uint4*>(hb)[i] = make_uint4(0, 0, 0, 0);   // h_0 = 0
  }
  __syncthreads();
  cluster_barrier();   // every CTA's buffers are initialised before anyone stores into them

  const int g = lane >> 2, t4 = lane & 3;   // MMA fragment coordinates
  const int ci = lane >> 3, n = lane & 7;   // this lane's item: cell ci of the warp's 4, sequence n
  const bool warp_valid = warp * 4 < cpc;
  const int cl = warp * 4 + ci;             // cell within the CTA
  const bool valid = cl < cpc;
  const int cell = (int)rank * cpc + cl;    // cell within the layer
  float4 s_ih = make_float4(0.f, 0.f, 0.f, 0.f), s_hh = s_ih, bb = s_ih;
  if (valid) {
    s_ih = reinterpret_cast<const float4*>(D.sc_ih)[cell];
    s_hh = reinterpret_cast<const float4*>(D.sc_hh)[cell];
    bb = reinterpret_cast<const float4*>(D.bias)[cell];
  }
  const float sh = a.hid_act.scale;
  const int hlo = act_lo(a.hid_act), hhi = act_hi(a.hid_act);
  const int ylo = act_lo(a.out_act), yhi = act_hi(a.out_act);
  float c_state[NT];
  float sx[NT];
  int last_q[NT];
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    c_state[j] = 0.0f;
    last_q[j] = 0;
    const int b = grp * BG + 8 * j + n;
    sx[j] = (a.x_scale_b && b < B) ? a.x_scale_b[b] : a.x_scale;
  }
  const uint32_t hb_addr = static_cast<uint32_t>(__cvta_generic_to_shared(hb));
  // ldmatrix: lane i supplies the row address of matrix i/8 (rows 0-7 | 8-15, k 0-15 | 16-31)
  const uint32_t a_addr = static_cast<uint32_t>(__cvta_generic_to_shared(
      Ws + (size_t)(16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * pitch + 16 * (lane >> 4)));
  const int G = 4 * H;
  // where the four gates of my item sit after the MMA: rows 4*ci+gate of the 16-row tile
  const int src_base = ((4 * (ci & 1)) << 2) | (n >> 1);
  const int ridx = 2 * (ci >> 1) + (n & 1);

  for (int step = 0; step < T; ++step) {
    const int t = d == 0 ? step : T - 1 - step;
    const int cur = step & 1, nxt = cur ^ 1;
    // input contribution of this step for my items (independent of the recurrence: prefetch)
    int4 pre[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int b = grp * BG + 8 * j + n;
      pre[j] = make_int4(0, 0, 0, 0);
      if (valid && b < B)
        pre[j] = *reinterpret_cast<const int4*>(D.acc_pre + ((size_t)t * B + b) * G + 4 * cell);
    }
    // recurrent MACs against the resident weights
    int acc[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[j][r] = 0;
    if (warp_valid) {
      // B fragments by ldmatrix as well: lane i supplies the row address of matrix i/8 = (sequence tile
      // i/16, k half (i/8)&1); thread (g, t4) receives bytes 4 t4 .. 4 t4 + 3 of sequence row g of each
      const uint32_t b_addr = hb_addr + (uint32_t)((cur * BG + (lane & 7) + 8 * (lane >> 4)) * pitch + 16 * ((lane >> 3) & 1));
#pragma unroll 4
      for (int k0 = 0; k0 < H; k0 += 32) {
        uint32_t a0, a1, a2, a3;
        ldmatrix_x4(a_addr + k0, a0, a1, a2, a3);
        uint32_t b[4];
        if (NT == 2)
          ldmatrix_x4(b_addr + k0, b[0], b[1], b[2], b[3]);
        else
          ldmatrix_x2(b_addr + k0, b[0], b[1]);
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_s8(acc[j], a0, a1, a2, a3, b[2 * j], b[2 * j + 1]);
      }
    }
    // cell update for my items
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int bl = 8 * j + n;
      const int b = grp * BG + bl;
      int hh[4];
#pragma unroll
      for (int gate = 0; gate < 4; ++gate) {
        const int src = src_base + (gate << 2);
        const int v0 = __shfl_sync(0xffffffffu, acc[j][0], src);
        const int v1 = __shfl_sync(0xffffffffu, acc[j][1], src);
        const int v2 = __shfl_sync(0xffffffffu, acc[j][2], src);
        const int v3 = __shfl_sync(0xffffffffu, acc[j][3], src);
        hh[gate] = ridx == 0 ? v0 : (ridx == 1 ? v1 : (ridx == 2 ? v2 : v3));
      }
      int q = 0, q2 = 0;
      const bool live = valid && b < B;
      if (live) {
        const float pi = __fmaf_rn((float)hh[0], __fmul_rn(sh, s_hh.x), __fmaf_rn((float)pre[j].x, __fmul_rn(sx[j], s_ih.x), bb.x));
        const float pf = __fmaf_rn((float)hh[1], __fmul_rn(sh, s_hh.y), __fmaf_rn((float)pre[j].y, __fmul_rn(sx[j], s_ih.y), bb.y));
        const float pg = __fmaf_rn((float)hh[2], __fmul_rn(sh, s_hh.z), __fmaf_rn((float)pre[j].z, __fmul_rn(sx[j], s_ih.z), bb.z));
        const float po = __fmaf_rn((float)hh[3], __fmul_rn(sh, s_hh.w), __fmaf_rn((float)pre[j].w, __fmul_rn(sx[j], s_ih.w), bb.w));
        float hval;
        cell_fixed(pi, pf, pg, po, c_state[j], c_state[j], hval);
        q = quantize1(hval, a.hid_act.inv_scale, a.hid_act.zero_point, hlo, hhi);
        q2 = quantize1(hval, a.out_act.inv_scale, a.out_act.zero_point, ylo, yhi);
        last_q[j] = q;
        if (D.dbg_ih) {
          const size_t o = ((size_t)t * B + b) * a.dbg_ld;
          D.dbg_ih[o + cell] = pre[j].x;
          D.dbg_ih[o + H + cell] = pre[j].y;
          D.dbg_ih[o + 2 * H + cell] = pre[j].z;
          D.dbg_ih[o + 3 * H + cell] = pre[j].w;
          D.dbg_hh[o + cell] = hh[0];
          D.dbg_hh[o + H + cell] = hh[1];
          D.dbg_hh[o + 2 * H + cell] = hh[2];
          D.dbg_hh[o + 3 * H + cell] = hh[3];
        }
      }
      if (valid) stage[bl * cpc + cl] = (int8_t)q;
      // layer output codes (out_act), two 4-bit cells per byte: the even cell's lane writes
      const int q2_next = __shfl_down_sync(0xffffffffu, q2, 8);
      if (live) {
        uint8_t* y = D.yq + ((size_t)t * B + b) * a.yq_ld;
        if (a.out_act.bits == 4) {
          if ((cl & 1) == 0) y[cell >> 1] = (uint8_t)((q2 & 0xF) | ((q2_next & 0xF) << 4));
        } else {
          y[cell] = (uint8_t)(q2 & 0xFF);
        }
      }
    }
    // the codes of h_t go to every CTA of the cluster (next step's operand): wide remote stores
    __syncthreads();
    if ((cpc & 15) == 0) {
      const int chunks = cpc >> 4;                       // 16-byte chunks per sequence row
      for (int i = tid; i < BG * chunks * REC_CLUSTER; i += REC_THREADS) {
        const uint32_t r = (uint32_t)(i % REC_CLUSTER);
        const int ch = (i / REC_CLUSTER) % chunks, bl = i / (REC_CLUSTER * chunks);
        const uint4 v = *reinterpret_cast<const uint4*>(stage + bl * cpc + ch * 16);
        st_cluster_v4(map_to_rank(hb_addr + (uint32_t)((nxt * BG + bl) * pitch + (int)rank * cpc + ch * 16), r), v);
      }
    } else {
      const int chunks = cpc >> 2;                       // 4-byte chunks
      for (int i = tid; i < BG * chunks * REC_CLUSTER; i += REC_THREADS) {
        const uint32_t r = (uint32_t)(i % REC_CLUSTER);
        const int ch = (i / REC_CLUSTER) % chunks, bl = i / (REC_CLUSTER * chunks);
        const uint32_t v = *reinterpret_cast<const uint32_t*>(stage + bl * cpc + ch * 4);
        st_cluster_u32(map_to_rank(hb_addr + (uint32_t)((nxt * BG + bl) * pitch + (int)rank * cpc + ch * 4), r), v);
      }
    }
    cluster_barrier();
  }
  // final states
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const int b = grp * BG + 8 * j + n;
    const int qn = __shfl_down_sync(0xffffffffu, last_q[j], 8);
    if (valid && b < B) {
      if (D.c_n) D.c_n[(size_t)b * H + cell] = c_state[j];
      if (D.hq_n) {
        if (a.hid_act.bits == 4) {
          if ((cl & 1) == 0) D.hq_n[(size_t)b * (H >> 1) + (cell >> 1)] = (uint8_t)((last_q[j] & 0xF) | ((qn & 0xF) << 4));
        } else {
          D.hq_n[(size_t)b * H + cell] = (uint8_t)(last_q[j] & 0xFF);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The same recurrence for 4-bit recurrent weights and 4-bit hidden codes (five of the six encoder
// layers, Section 3.2) with the weights held in REGISTERS for the whole sequence.
//
// A warp's 16 weight rows x H columns are 20 A fragments of the m16n8k32 MMA at H = 640; as 4-bit
// codes they fill 2 registers per fragment instead of 4, 40 registers per thread for the whole
// slice (102 KB per CTA).  Register 2s of thread (g, t4) holds, nibble 2i = W[row r(g)][32s + 4 t4 + i]
// and nibble 2i+1 = W[row r(g+8)][32s + 4 t4 + i] (register 2s+1 the same for columns + 16), so that
// two masks and one shift turn it into the fragment registers (a0, a1) with every code in the HIGH
// nibble of its byte: the int8 operand is 16 x code, exact, and the accumulator 16 x the true sum
// (|16 w h| <= 1024 per product, far from overflow); an arithmetic shift by 4 restores it.  The
// main loop therefore reads only the hidden codes from shared memory, not the weight slice (205 KB
// per step in the int8 kernel above: that kernel's limit).
//
// Tile row g holds gate (g & 1) of the warp's cell g >> 1 and tile row g + 8 gate 2 + (g & 1) of
// the same cell, so after the MMA the lanes g and g ^ 1 hold the four gates of one cell for two
// sequences: one exchange of two values with lane ^ 4 gives every lane the four gates of its item
// (cell g >> 1, sequence 2 t4 + (g & 1)).
//
// A cluster serves NU independent units of 8 sequences of one direction, one after the other within
// a step.  The hidden codes of a unit are laid out [source CTA][sequence][cells of that CTA], so a
// CTA's new codes are one contiguous block of 8 x H/8 bytes in every receiver: they travel as ONE
// bulk copy per destination through distributed shared memory (8 per unit and step instead of 320
// 16-byte stores), counted on an mbarrier of the receiving CTA; a CTA waits on its own mbarrier
// before the unit's next step.  (Rows of 80 bytes put the eight sequences of an ldmatrix on
// distinct banks.)  There is no cluster-wide barrier in the loop: while the
// codes of one unit are in flight the CTA computes the other unit.  Buffers are double buffered by
// step parity; a sender can only be a step ahead of a receiver after that receiver's own codes of
// the previous step have arrived, which it sends after its last read of the buffer in question.
// Every wait is bounded; when one expires the CTA records Q4_ERR_TIMEOUT, leaves the loop, and all
// CTAs still meet at the closing cluster barrier (the others' waits expire in turn).
// The input accumulators of the next step are fetched into shared memory by cp.async one step
// ahead.  The layer output codes leave through a staging buffer as 8-byte stores.
// `bytes` (a multiple of 16) from this CTA's shared memory into the shared memory of a CTA of the
// cluster by the bulk-copy engine; their arrival is counted on the mbarrier at `mbar_addr`, an
// address in the receiving CTA's window.  No multicast: one destination per copy.
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_addr, uint32_t src_addr, uint32_t bytes,
                                                     uint32_t mbar_addr) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_addr), "r"(src_addr), "r"(bytes), "r"(mbar_addr)
               : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int REC_BG = 8;   // sequences per unit of the register-resident kernel
constexpr int REC4_THREADS = REC_THREADS;

__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int count) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}

__host__ __device__ constexpr int rec_w4_ksmem(int nu) { return nu <= 2 ? 6 : 8; }
// k-steps of weights in shared memory, kernel whose clusters may take turns: packed 4-bit / int8
__host__ __device__ constexpr int rec_turns_ksmem(bool w8) { return w8 ? 13 : 6; }

template <int NU, int KS>
__global__ void __cluster_dims__(REC_CLUSTER, 1, 1) __launch_bounds__(REC4_THREADS, 1)
k_enc_recurrent_w4(const EncRecArgs a) {
  extern __shared__ __align__(16) uint8_t rec_smem[];
  constexpr int BG = REC_BG;
  constexpr int H = 32 * KS;
  constexpr int cpc = H / REC_CLUSTER;      // cells per CTA
  constexpr int rows = 4 * cpc;
  constexpr int chunks = cpc >> 4;          // 16-byte chunks of a sequence's new codes per CTA
  constexpr int UB = BG * H;                // bytes of one unit's hidden codes
  constexpr int CW = REC_THREADS / 32;      // warps
  constexpr int KR = KS - rec_w4_ksmem(NU);   // k-steps whose weight fragments stay in registers; the last
                                              // six or eight come from shared memory (8 bytes per thread and
                                              // k-step), which leaves the cell update enough registers: no spills
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const int cid = blockIdx.x / REC_CLUSTER;
  const int cpd = a.n_groups;               // clusters per direction
  const int d = cid / cpd;
  const int grp0 = (cid % cpd) * NU;        // first 8-sequence group of this cluster
  const EncRecDir& D = a.d[d];
  const int T = a.T, B = a.B;
  int8_t* hb = reinterpret_cast<int8_t*>(rec_smem);                       // [NU][2][source CTA][BG][cpc] h_{t-1}
  int4* pre_s = reinterpret_cast<int4*>(hb + (size_t)NU * 2 * UB);        // [2][NU][threads] input accumulators
  float4* cst = reinterpret_cast<float4*>(pre_s + (size_t)2 * NU * REC_THREADS);   // [3][cpc] per-cell constants
  int8_t* stage = reinterpret_cast<int8_t*>(cst + 3 * cpc);                // [2][NU][BG][cpc] new recurrent codes
  int8_t* stage_y = stage + (size_t)2 * NU * BG * cpc;                     // [2][NU][BG][cpc] new output codes
  uint64_t* full = reinterpret_cast<uint64_t*>(stage_y + (size_t)2 * NU * BG * cpc);   // [NU][2]
  volatile int* dead = reinterpret_cast<volatile int*>(full + NU * 2);     // a bounded wait has expired
  uint2* wsm = reinterpret_cast<uint2*>(full + NU * 2 + 2);                // [KS - KR][threads] packed weights

  const int g = lane >> 2, t4 = lane & 3;   // MMA fragment coordinates
  const int e = g & 1, ci = g >> 1;         // this lane's item: cell ci of the warp's 4 ...
  const int n = 2 * t4 + e;                 // ... and sequence n of the unit's 8
  const int cl = warp * 4 + ci;             // cell within the CTA
  const int cell = (int)rank * cpc + cl;    // cell within the layer
  const float sh = a.hid_act.scale;
  const uint32_t hb_addr = smem_u32(hb), pre_addr = smem_u32(pre_s), full_addr = smem_u32(full);

  // resident weights: this warp's 16 rows (stored in 4*cell+gate order), packed two codes per byte;
  // tile row g = gate e of cell ci, tile row g + 8 = gate 2 + e of cell ci
  uint32_t wreg[2 * KR];
  {
    const int8_t* W = D.w_hh + ((size_t)rank * rows + (size_t)(16 * warp)) * H;
    const int8_t* r0 = W + (size_t)(4 * ci + e) * H + 4 * t4;
    const int8_t* r1 = r0 + (size_t)2 * H;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint32_t q0 = *reinterpret_cast<const uint32_t*>(r0 + 32 * s);
      const uint32_t p0 = *reinterpret_cast<const uint32_t*>(r1 + 32 * s);
      const uint32_t q1 = *reinterpret_cast<const uint32_t*>(r0 + 32 * s + 16);
      const uint32_t p1 = *reinterpret_cast<const uint32_t*>(r1 + 32 * s + 16);
      const uint32_t w0 = (q0 & 0x0F0F0F0Fu) | ((p0 << 4) & 0xF0F0F0F0u);
      const uint32_t w1 = (q1 & 0x0F0F0F0Fu) | ((p1 << 4) & 0xF0F0F0F0u);
      if (s < KR) {
        wreg[2 * s] = w0;
        wreg[2 * s + 1] = w1;
      } else {
        wsm[(s - KR) * REC_THREADS + tid] = make_uint2(w0, w1);
      }
    }
  }
  for (int i = tid; i < NU * 2 * UB / 16; i += REC4_THREADS)
    reinterpret_cast<uint4*>(hb)[i] = make_uint4(0, 0, 0, 0);   // h_0 = 0
  for (int i = tid; i < cpc; i += REC4_THREADS) {
    // de-quantization products per gate row: input scale * row scale, hidden scale * row scale; bias
    const int c = (int)rank * cpc + i;
    const float4 w = reinterpret_cast<const float4*>(D.sc_hh)[c], v = reinterpret_cast<const float4*>(D.sc_ih)[c];
    const float sxs = a.x_scale;
    cst[i] = make_float4(__fmul_rn(sxs, v.x), __fmul_rn(sxs, v.y), __fmul_rn(sxs, v.z), __fmul_rn(sxs, v.w));
    cst[cpc + i] = make_float4(__fmul_rn(sh, w.x), __fmul_rn(sh, w.y), __fmul_rn(sh, w.z), __fmul_rn(sh, w.w));
    cst[2 * cpc + i] = reinterpret_cast<const float4*>(D.bias)[c];
  }
  if (tid == 0) {
    *dead = 0;
    for (int i = 0; i < NU * 2; ++i) mbar_init(&full[i], 1);
    fence_barrier_init();
    // the first fill of either buffer of every unit: BG x H bytes from the eight CTAs
    for (int i = 0; i < NU * 2; ++i) mbar_expect_tx(&full[i], (uint32_t)UB);
  }
  fence_proxy_async();   // the zeroed buffers are later written by the bulk-copy engine
  __syncthreads();
  cluster_barrier();   // every CTA's buffers and barriers are initialised before anyone stores into them

  float c_state[NU];
  bool live[NU];
#pragma unroll
  for (int u = 0; u < NU; ++u) {
    c_state[u] = 0.0f;
    live[u] = (grp0 + u) * BG + n < B;
  }
  constexpr int G = 4 * H;

  {
    const int hlo = act_lo(a.hid_act), hhi = act_hi(a.hid_act);
    const int ylo = act_lo(a.out_act), yhi = act_hi(a.out_act);
    const bool y4 = a.out_act.bits == 4;
#pragma unroll
    for (int u = 0; u < NU; ++u) {
      const int b = (grp0 + u) * BG + n;
      // input accumulators of the first step
      if (live[u]) {
        const int t = d == 0 ? 0 : T - 1;
        cp_async16(pre_addr + (uint32_t)((u * REC_THREADS + tid) * 16), D.acc_pre + ((size_t)t * B + b) * G + 4 * cell);
      }
      cp_async_commit();
    }
    bool ok = true;
    for (int step = 0; step < T; ++step) {
      const int t = d == 0 ? step : T - 1 - step;
      const int cur = step & 1, nxt = cur ^ 1;
#pragma unroll
      for (int u = 0; u < NU; ++u) {
        const int b = (grp0 + u) * BG + n;
        // the next step's input accumulators for this unit, one step ahead
        if (step + 1 < T && live[u]) {
          const int tn = d == 0 ? step + 1 : T - 2 - step;
          cp_async16(pre_addr + (uint32_t)(((nxt * NU + u) * REC_THREADS + tid) * 16),
                     D.acc_pre + ((size_t)tn * B + b) * G + 4 * cell);
        }
        cp_async_commit();
        // h_{t-1} of this unit is complete in this CTA once all eight CTAs' copies have landed.  Every
        // thread looks for itself (no block barrier: with several units the codes are long there).
        // After a wait has expired anywhere in the CTA nobody waits any more; the loop is walked to its
        // end all the same, so that every named barrier still gets its arrivals
        if (step > 0 && ok) {
          uint64_t* bar = &full[u * 2 + cur];
          const uint32_t parity = (uint32_t)(((step - 1) >> 1) & 1);
          bool got = false;
          for (uint32_t i = 0; i < (1u << 22); ++i) {
            if (mbar_try_wait(bar, parity)) {
              got = true;
              break;
            }
            if ((i & 255u) == 255u && *dead) break;
          }
          if (!got) {
            ok = false;
            *dead = 1;
            if (a.status) atomicExch(a.status, Q4_ERR_TIMEOUT);
          }
          // arm the barrier for the next fill of this buffer; nobody can send that fill before this
          // CTA's codes of the present step have arrived, which are sent after every thread got here
          if (tid == 0 && got) mbar_expect_tx(bar, (uint32_t)UB);
        }
        // recurrent MACs: weights from registers, hidden codes by ldmatrix
        int acc[2][4];
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int r = 0; r < 4; ++r) acc[c][r] = 0;
        {
          // lanes 0-15 supply the row addresses: matrix i/8 = k half, row i%8 = sequence; the 16-byte
          // chunk j = 2s + half of a sequence's codes lies in source block j / chunks at chunk j % chunks
          // (the second half's chunk is 16 bytes on, or in the next source block when j % chunks wraps)
          const uint32_t half = (uint32_t)((lane >> 3) & 1);
          const uint32_t b_addr = hb_addr + (uint32_t)((u * 2 + cur) * UB + (lane & 7) * cpc);
          const uint32_t b_in = b_addr + half * 16u, b_wrap = b_addr + half * (uint32_t)(BG * cpc - (chunks - 1) * 16);
#pragma unroll
          for (int s = 0; s < KS; ++s) {
            uint32_t w0, w1;
            if (s < KR) {
              w0 = wreg[2 * s];
              w1 = wreg[2 * s + 1];
            } else {
              const uint2 w = wsm[(s - KR) * REC_THREADS + tid];
              w0 = w.x;
              w1 = w.y;
            }
            const uint32_t a0 = (w0 << 4) & 0xF0F0F0F0u, a1 = w0 & 0xF0F0F0F0u;
            const uint32_t a2 = (w1 << 4) & 0xF0F0F0F0u, a3 = w1 & 0xF0F0F0F0u;
            const uint32_t o0 = (uint32_t)(((2 * s) / chunks) * BG * cpc + ((2 * s) % chunks) * 16);
            uint32_t b0, b1;
            ldmatrix_x2(((2 * s) % chunks == chunks - 1 ? b_wrap : b_in) + o0, b0, b1);
            mma_s8(acc[s & 1], a0, a1, a2, a3, b0, b1);
          }
        }
        // the four gates of my item: mine are rows g (gate e) and g + 8 (gate 2 + e) at column e of the
        // pair; the other two come from lane ^ 4, which needs my values at the other column
        int hh[4];
        {
          const int v0 = acc[0][0] + acc[1][0], v1 = acc[0][1] + acc[1][1];
          const int v2 = acc[0][2] + acc[1][2], v3 = acc[0][3] + acc[1][3];
          const int r0 = __shfl_xor_sync(0xffffffffu, e ? v0 : v1, 4);
          const int r1 = __shfl_xor_sync(0xffffffffu, e ? v2 : v3, 4);
          const int m0 = e ? v1 : v0, m1 = e ? v3 : v2;
          hh[0] = (e ? r0 : m0) >> 4;     // the operand was 16 x code
          hh[1] = (e ? m0 : r0) >> 4;
          hh[2] = (e ? r1 : m1) >> 4;
          hh[3] = (e ? m1 : r1) >> 4;
        }
        cp_async_wait<NU>();              // this thread's accumulators of the present step have landed
        int q = 0, q2 = 0;
        if (live[u]) {
          const int4 pre = pre_s[(cur * NU + u) * REC_THREADS + tid];
          const float4 s_ih = cst[cl], s_hh = cst[cpc + cl], bb = cst[2 * cpc + cl];
          const float pi = __fmaf_rn((float)hh[0], s_hh.x, __fmaf_rn((float)pre.x, s_ih.x, bb.x));
          const float pf = __fmaf_rn((float)hh[1], s_hh.y, __fmaf_rn((float)pre.y, s_ih.y, bb.y));
          const float pg = __fmaf_rn((float)hh[2], s_hh.z, __fmaf_rn((float)pre.z, s_ih.z, bb.z));
          const float po = __fmaf_rn((float)hh[3], s_hh.w, __fmaf_rn((float)pre.w, s_ih.w, bb.w));
          float hval;
          cell_fixed_p(pi, pf, pg, po, c_state[u], c_state[u], hval);
          q = quantize1(hval, a.hid_act.inv_scale, a.hid_act.zero_point, hlo, hhi);
          q2 = quantize1(hval, a.out_act.inv_scale, a.out_act.zero_point, ylo, yhi);
        }
        // staged by step parity: the engine may still be reading the other buffer (the previous step's
        // block), but not this one (its block of two steps ago has been received by every CTA)
        stage[((cur * NU + u) * BG + n) * cpc + cl] = (int8_t)q;
        stage_y[((cur * NU + u) * BG + n) * cpc + cl] = (int8_t)q2;
        if (step == T - 1 && D.hq_n) {   // final recurrent codes, two cells per byte: the even cell's lane writes
          const int qn = __shfl_down_sync(0xffffffffu, q, 8);
          if (live[u] && (cl & 1) == 0)
            D.hq_n[(size_t)b * (H >> 1) + (cell >> 1)] = (uint8_t)((q & 0xF) | ((qn & 0xF) << 4));
        }
        fence_proxy_async();   // the staged codes are read by the bulk-copy engine
        // One warp, a different one every time, waits until all threads have staged their codes (the
        // others only arrive at the named barrier and go on with the next unit), sends the staged
        // block [BG][cpc] to [source = this CTA] of every CTA's buffer for the next step (one bulk copy
        // per destination, counted on the receiver's mbarrier), and writes the CTA's share of the
        // layer output: 16 cells per lane and pass, packed when 4 bit
        if (warp != (step * NU + u) % CW) {
          named_bar_arrive(1 + u * 2 + cur, REC4_THREADS);
        } else {
          named_bar_sync(1 + u * 2 + cur, REC4_THREADS);
          if (lane < REC_CLUSTER) {
            const uint32_t r = (uint32_t)lane;
            bulk_copy_to_cluster(map_to_rank(hb_addr + (uint32_t)((u * 2 + nxt) * UB + (int)rank * BG * cpc), r),
                                 smem_u32(stage + (size_t)(cur * NU + u) * BG * cpc), (uint32_t)(BG * cpc),
                                 map_to_rank(full_addr + (uint32_t)((u * 2 + nxt) * 8), r));
          }
          for (int i = lane; i < BG * chunks; i += 32) {
            const int ch = i % chunks, bl = i / chunks;
            const int by = (grp0 + u) * BG + bl;
            if (by >= B) continue;
            const uint4 v = *reinterpret_cast<const uint4*>(stage_y + ((cur * NU + u) * BG + bl) * cpc + ch * 16);
            uint8_t* y = D.yq + ((size_t)t * B + by) * a.yq_ld;
            const int c0 = (int)rank * cpc + ch * 16;
            if (y4) {
              // bytes (c, c+1) -> one byte: low nibble c, high nibble c+1
              auto pk = [](uint32_t w) -> uint32_t {
                const uint32_t m = (w & 0x000F000Fu) | ((w >> 4) & 0x00F000F0u);   // bytes 0 and 2 hold the pairs
                return (m & 0xFFu) | ((m >> 8) & 0xFF00u);
              };
              *reinterpret_cast<uint2*>(y + (c0 >> 1)) = make_uint2(pk(v.x) | (pk(v.y) << 16), pk(v.z) | (pk(v.w) << 16));
            } else {
              *reinterpret_cast<uint4*>(y + c0) = v;
            }
          }
        }
      }
    }
  }
  cp_async_wait<0>();
  // the codes sent in the last step are still on their way into this CTA: wait for them (bounded), so
  // that nobody leaves while copies into its shared memory are in flight
  if (T > 0) {
#pragma unroll
    for (int u = 0; u < NU; ++u) {
      const uint32_t parity = (uint32_t)(((T - 1) >> 1) & 1);
      for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try_wait(&full[u * 2 + (T & 1)], parity)) break;
        if ((i & 255u) == 255u && *dead) break;
      }
    }
  }
  __syncthreads();
  cluster_barrier();
  // final states
#pragma unroll
  for (int u = 0; u < NU; ++u) {
    const int b = (grp0 + u) * BG + n;
    if (live[u] && D.c_n) D.c_n[(size_t)b * H + cell] = c_state[u];
  }
}

// ---------------------------------------------------------------------------------------------
// The same step with one group too many for the clusters that can be resident: G groups of 8
// sequences of a direction on G - 1 clusters.  Cluster j owns group j; group G - 1 is shared: it
// advances on cluster 0 during its first T / (G - 1) steps, then on cluster 1, and so on; while a
// cluster advances the shared group its own group rests.  Every cluster therefore walks
// T + T / (G - 1) steps of ONE group each instead of 2 T (two groups per cluster), and all clusters
// of the direction end together.  At a hand-over the shared group's cell states and hidden codes go
// through global memory: every CTA of the giving cluster stores its part, fences, and adds one to a
// counter; the taking cluster (always the next higher one, so a waiting cluster only ever waits for
// clusters that were dispatched before it) polls the counter, bounded, and loads the state.
// A direction with as many clusters as groups runs plain (sliced = 0).
// Slot 0 = the cluster's own group, slot 1 = the shared group while it is here.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

template <int KS, bool W8>
__global__ void __cluster_dims__(REC_CLUSTER, 1, 1) __launch_bounds__(REC4_THREADS, 1)
k_enc_recurrent_w4s(const EncRecArgs a) {
  extern __shared__ __align__(16) uint8_t rec_smem[];
  constexpr int BG = REC_BG;
  constexpr int NS = 2;                     // slots
  constexpr int H = 32 * KS;
  constexpr int cpc = H / REC_CLUSTER;      // cells per CTA
  constexpr int rows = 4 * cpc;
  constexpr int chunks = cpc >> 4;          // 16-byte chunks of a sequence's new codes per CTA
  constexpr int UB = BG * H;                // bytes of one group's hidden codes
  constexpr int CW = REC_THREADS / 32;      // warps
  constexpr int KR = KS - rec_turns_ksmem(W8);   // k-steps whose weight fragments stay in registers
  constexpr int WPK = W8 ? 4 : 2;                // 32-bit words of weights per thread and k-step
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const int cid = blockIdx.x / REC_CLUSTER;
  const int d = cid < a.ncl[0] ? 0 : 1;     // the clusters of direction 0 come first
  const int j = d == 0 ? cid : cid - a.ncl[0];
  const int C = a.ncl[d];
  const bool host = a.sliced[d] != 0;
  const EncRecDir& D = a.d[d];
  const int T = a.T, B = a.B;
  // the shared group's steps [w0, w1) run here
  const int w0 = host ? a.win[j] : 0, w1 = host ? a.win[j + 1] : 0;
  const int n_it = T + (w1 - w0);
  int8_t* hb = reinterpret_cast<int8_t*>(rec_smem);                       // [NS][2][source CTA][BG][cpc] h_{t-1}
  int4* pre_s = reinterpret_cast<int4*>(hb + (size_t)NS * 2 * UB);        // [2][threads] input accumulators
  float4* cst = reinterpret_cast<float4*>(pre_s + (size_t)2 * REC_THREADS);   // [3][cpc] per-cell constants
  int8_t* stage = reinterpret_cast<int8_t*>(cst + 3 * cpc);                // [NS][2][BG][cpc] new recurrent codes
  int8_t* stage_y = stage + (size_t)2 * NS * BG * cpc;                     // [NS][2][BG][cpc] new output codes
  uint64_t* full = reinterpret_cast<uint64_t*>(stage_y + (size_t)2 * NS * BG * cpc);   // [NS][2]
  volatile int* dead = reinterpret_cast<volatile int*>(full + NS * 2);     // a bounded wait has expired
  uint32_t* wsm = reinterpret_cast<uint32_t*>(full + NS * 2 + 2);          // [KS - KR][threads][WPK] weights

  const int g = lane >> 2, t4 = lane & 3;   // MMA fragment coordinates
  const int e = g & 1, ci = g >> 1;         // this lane's item: cell ci of the warp's 4 ...
  const int n = 2 * t4 + e;                 // ... and sequence n of the group's 8
  const int cl = warp * 4 + ci;             // cell within the CTA
  const int cell = (int)rank * cpc + cl;    // cell within the layer
  const float sh = a.hid_act.scale;
  const uint32_t hb_addr = smem_u32(hb), pre_addr = smem_u32(pre_s), full_addr = smem_u32(full);

  uint32_t wreg[WPK * KR];
  {
    const int8_t* W = D.w_hh + ((size_t)rank * rows + (size_t)(16 * warp)) * H;
    const int8_t* r0 = W + (size_t)(4 * ci + e) * H + 4 * t4;
    const int8_t* r1 = r0 + (size_t)2 * H;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint32_t q0 = *reinterpret_cast<const uint32_t*>(r0 + 32 * s);
      const uint32_t p0 = *reinterpret_cast<const uint32_t*>(r1 + 32 * s);
      const uint32_t q1 = *reinterpret_cast<const uint32_t*>(r0 + 32 * s + 16);
      const uint32_t p1 = *reinterpret_cast<const uint32_t*>(r1 + 32 * s + 16);
      if (W8) {   // one code per byte: the MMA fragment as it is
        if (s < KR) {
          wreg[WPK * s] = q0;
          wreg[WPK * s + 1] = p0;
          wreg[WPK * s + 2] = q1;
          wreg[WPK * s + 3] = p1;
        } else {
          reinterpret_cast<uint4*>(wsm)[(s - KR) * REC_THREADS + tid] = make_uint4(q0, p0, q1, p1);
        }
      } else {    // two codes per byte
        const uint32_t w0p = (q0 & 0x0F0F0F0Fu) | ((p0 << 4) & 0xF0F0F0F0u);
        const uint32_t w1p = (q1 & 0x0F0F0F0Fu) | ((p1 << 4) & 0xF0F0F0F0u);
        if (s < KR) {
          wreg[WPK * s] = w0p;
          wreg[WPK * s + 1] = w1p;
        } else {
          reinterpret_cast<uint2*>(wsm)[(s - KR) * REC_THREADS + tid] = make_uint2(w0p, w1p);
        }
      }
    }
  }
  for (int i = tid; i < NS * 2 * UB / 16; i += REC4_THREADS)
    reinterpret_cast<uint4*>(hb)[i] = make_uint4(0, 0, 0, 0);   // h_0 = 0
  for (int i = tid; i < cpc; i += REC4_THREADS) {
    const int c = (int)rank * cpc + i;
    const float4 w = reinterpret_cast<const float4*>(D.sc_hh)[c], v = reinterpret_cast<const float4*>(D.sc_ih)[c];
    cst[i] = v;   // multiplied with the sequence's input scale at every use (the same fp32 product)
    cst[cpc + i] = make_float4(__fmul_rn(sh, w.x), __fmul_rn(sh, w.y), __fmul_rn(sh, w.z), __fmul_rn(sh, w.w));
    cst[2 * cpc + i] = reinterpret_cast<const float4*>(D.bias)[c];
  }
  if (tid == 0) {
    *dead = 0;
    for (int i = 0; i < NS * 2; ++i) mbar_init(&full[i], 1);
    fence_barrier_init();
    for (int i = 0; i < NS * 2; ++i) mbar_expect_tx(&full[i], (uint32_t)UB);
  }
  fence_proxy_async();   // the zeroed buffers are later written by the bulk-copy engine
  __syncthreads();
  cluster_barrier();   // every CTA's buffers and barriers are initialised before anyone stores into them

  const int b_own = j * BG + n, b_shared = (a.groups - 1) * BG + n;
  const bool live_own = b_own < B, live_shared = host && b_shared < B;
  float c_own = 0.0f, c_shared = 0.0f;
  const float sx_own = (a.x_scale_b && live_own) ? a.x_scale_b[b_own] : a.x_scale;
  const float sx_shared = (a.x_scale_b && live_shared) ? a.x_scale_b[b_shared] : a.x_scale;
  const bool h4 = a.hid_act.bits == 4;
  constexpr int G = 4 * H;
  const int hlo = act_lo(a.hid_act), hhi = act_hi(a.hid_act);
  const int ylo = act_lo(a.out_act), yhi = act_hi(a.out_act);
  const bool y4 = a.out_act.bits == 4;
  int32_t* const flag_out = a.flags + d * 8 + j;

  // walk: own steps [0, w0), shared steps [w0, w1), own steps [w0, T)
  auto walk = [&](int i, int& u, int& step) {
    if (i < w0) {
      u = 0;
      step = i;
    } else if (i < w1) {
      u = 1;
      step = i;
    } else {
      u = 0;
      step = i - (w1 - w0);
    }
  };
  auto fetch_pre = [&](int i) {   // input accumulators of walk position i into buffer i & 1
    int u, step;
    walk(i, u, step);
    const int b = u ? b_shared : b_own;
    if (u ? live_shared : live_own) {
      const int t = d == 0 ? step : T - 1 - step;
      cp_async16(pre_addr + (uint32_t)(((i & 1) * REC_THREADS + tid) * 16), D.acc_pre + ((size_t)t * B + b) * G + 4 * cell);
    }
    cp_async_commit();
  };
  if (n_it > 0) fetch_pre(0);
  bool ok = true;
  for (int i = 0; i < n_it; ++i) {
    int u, step;
    walk(i, u, step);
    const int ls = u ? step - w0 : step;          // steps of this slot made here so far
    const int t = d == 0 ? step : T - 1 - step;
    const int cur = ls & 1, nxt = cur ^ 1;
    const int b = u ? b_shared : b_own;
    const bool live = u ? live_shared : live_own;
    if (i + 1 < n_it)
      fetch_pre(i + 1);
    else
      cp_async_commit();
    if (u == 1 && ls == 0 && j > 0) {
      // take the shared group over from cluster j - 1: all eight of its CTAs have stored their parts
      if (tid == 0 && ok) {
        bool got = false;
        for (uint32_t it = 0; it < (1u << 22); ++it) {
          if (ld_acquire_gpu(flag_out - 1) >= REC_CLUSTER) {
            got = true;
            break;
          }
          if (*dead) break;
          __nanosleep(100);
        }
        if (!got) {
          *dead = 1;
          if (a.status) atomicExch(a.status, Q4_ERR_TIMEOUT);
        }
      }
      __syncthreads();
      if (*dead) ok = false;
      if (ok) {
        const uint4* src = reinterpret_cast<const uint4*>(a.hand_h[d]);
        for (int k = tid; k < UB / 16; k += REC4_THREADS)
          reinterpret_cast<uint4*>(hb + (size_t)(1 * 2 + 0) * UB)[k] = __ldcg(src + k);
        c_shared = live_shared ? __ldcg(a.hand_c[d] + (size_t)n * H + cell) : 0.0f;
      }
      fence_proxy_async();   // this buffer is written by the bulk-copy engine two steps on
      __syncthreads();
    }
    if (ls > 0 && ok) {
      uint64_t* bar = &full[u * 2 + cur];
      const uint32_t parity = (uint32_t)(((ls - 1) >> 1) & 1);
      bool got = false;
      for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (mbar_try_wait(bar, parity)) {
          got = true;
          break;
        }
        if ((it & 255u) == 255u && *dead) break;
      }
      if (!got) {
        ok = false;
        *dead = 1;
        if (a.status) atomicExch(a.status, Q4_ERR_TIMEOUT);
      }
      if (tid == 0 && got) mbar_expect_tx(bar, (uint32_t)UB);
    }
    int acc[2][4];
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[c][r] = 0;
    {
      const uint32_t half = (uint32_t)((lane >> 3) & 1);
      const uint32_t b_addr = hb_addr + (uint32_t)((u * 2 + cur) * UB + (lane & 7) * cpc);
      const uint32_t b_in = b_addr + half * 16u, b_wrap = b_addr + half * (uint32_t)(BG * cpc - (chunks - 1) * 16);
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        uint32_t a0, a1, a2, a3;
        if (W8) {
          if (s < KR) {
            a0 = wreg[WPK * s];
            a1 = wreg[WPK * s + 1];
            a2 = wreg[WPK * s + 2];
            a3 = wreg[WPK * s + 3];
          } else {
            const uint4 w = reinterpret_cast<const uint4*>(wsm)[(s - KR) * REC_THREADS + tid];
            a0 = w.x;
            a1 = w.y;
            a2 = w.z;
            a3 = w.w;
          }
        } else {
          uint32_t w0p, w1p;
          if (s < KR) {
            w0p = wreg[WPK * s];
            w1p = wreg[WPK * s + 1];
          } else {
            const uint2 w = reinterpret_cast<const uint2*>(wsm)[(s - KR) * REC_THREADS + tid];
            w0p = w.x;
            w1p = w.y;
          }
          a0 = (w0p << 4) & 0xF0F0F0F0u;   // 16 x code
          a1 = w0p & 0xF0F0F0F0u;
          a2 = (w1p << 4) & 0xF0F0F0F0u;
          a3 = w1p & 0xF0F0F0F0u;
        }
        const uint32_t o0 = (uint32_t)(((2 * s) / chunks) * BG * cpc + ((2 * s) % chunks) * 16);
        uint32_t b0, b1;
        ldmatrix_x2(((2 * s) % chunks == chunks - 1 ? b_wrap : b_in) + o0, b0, b1);
        mma_s8(acc[s & 1], a0, a1, a2, a3, b0, b1);
      }
    }
    int hh[4];
    {
      const int v0 = acc[0][0] + acc[1][0], v1 = acc[0][1] + acc[1][1];
      const int v2 = acc[0][2] + acc[1][2], v3 = acc[0][3] + acc[1][3];
      const int r0 = __shfl_xor_sync(0xffffffffu, e ? v0 : v1, 4);
      const int r1 = __shfl_xor_sync(0xffffffffu, e ? v2 : v3, 4);
      const int m0 = e ? v1 : v0, m1 = e ? v3 : v2;
      constexpr int SH = W8 ? 0 : 4;   // the packed operand was 16 x code
      hh[0] = (e ? r0 : m0) >> SH;
      hh[1] = (e ? m0 : r0) >> SH;
      hh[2] = (e ? r1 : m1) >> SH;
      hh[3] = (e ? m1 : r1) >> SH;
    }
    cp_async_wait<1>();               // this thread's accumulators of the present step have landed
    int q = 0, q2 = 0;
    if (live) {
      const int4 pre = pre_s[(i & 1) * REC_THREADS + tid];
      const float4 s_ih = cst[cl], s_hh = cst[cpc + cl], bb = cst[2 * cpc + cl];
      const float sx = u ? sx_shared : sx_own;
      const float pi = __fmaf_rn((float)hh[0], s_hh.x, __fmaf_rn((float)pre.x, __fmul_rn(sx, s_ih.x), bb.x));
      const float pf = __fmaf_rn((float)hh[1], s_hh.y, __fmaf_rn((float)pre.y, __fmul_rn(sx, s_ih.y), bb.y));
      const float pg = __fmaf_rn((float)hh[2], s_hh.z, __fmaf_rn((float)pre.z, __fmul_rn(sx, s_ih.z), bb.z));
      const float po = __fmaf_rn((float)hh[3], s_hh.w, __fmaf_rn((float)pre.w, __fmul_rn(sx, s_ih.w), bb.w));
      float cs = u ? c_shared : c_own, hval;
      cell_fixed_p(pi, pf, pg, po, cs, cs, hval);
      if (u)
        c_shared = cs;
      else
        c_own = cs;
      q = quantize1(hval, a.hid_act.inv_scale, a.hid_act.zero_point, hlo, hhi);
      q2 = quantize1(hval, a.out_act.inv_scale, a.out_act.zero_point, ylo, yhi);
    }
    stage[((u * 2 + cur) * BG + n) * cpc + cl] = (int8_t)q;
    stage_y[((u * 2 + cur) * BG + n) * cpc + cl] = (int8_t)q2;
    if (step == T - 1 && D.hq_n) {   // final recurrent codes; at 4 bits two cells per byte: the even cell's lane writes
      const int qn = __shfl_down_sync(0xffffffffu, q, 8);
      if (live && !h4)
        D.hq_n[(size_t)b * H + cell] = (uint8_t)q;
      else if (live && (cl & 1) == 0)
        D.hq_n[(size_t)b * (H >> 1) + (cell >> 1)] = (uint8_t)((q & 0xF) | ((qn & 0xF) << 4));
    }
    fence_proxy_async();   // the staged codes are read by the bulk-copy engine
    const bool window_end = u == 1 && step == w1 - 1;   // the shared group leaves after this step
    if (warp != i % CW) {
      named_bar_arrive(1 + u * 2 + cur, REC4_THREADS);
    } else {
      named_bar_sync(1 + u * 2 + cur, REC4_THREADS);
      if (!window_end) {
        if (lane < REC_CLUSTER) {
          const uint32_t r = (uint32_t)lane;
          bulk_copy_to_cluster(map_to_rank(hb_addr + (uint32_t)((u * 2 + nxt) * UB + (int)rank * BG * cpc), r),
                               smem_u32(stage + (size_t)(u * 2 + cur) * BG * cpc), (uint32_t)(BG * cpc),
                               map_to_rank(full_addr + (uint32_t)((u * 2 + nxt) * 8), r));
        }
      } else if (w1 < T) {
        // this CTA's block of the shared group's codes, in the layout of a receiver's buffer
        const uint4* src = reinterpret_cast<const uint4*>(stage + (size_t)(u * 2 + cur) * BG * cpc);
        uint4* dst = reinterpret_cast<uint4*>(a.hand_h[d] + (size_t)rank * BG * cpc);
        for (int k = lane; k < BG * cpc / 16; k += 32) dst[k] = src[k];
      }
      for (int k = lane; k < BG * chunks; k += 32) {
        const int ch = k % chunks, bl = k / chunks;
        const int by = (u ? a.groups - 1 : j) * BG + bl;
        if (by >= B) continue;
        const uint4 v = *reinterpret_cast<const uint4*>(stage_y + ((u * 2 + cur) * BG + bl) * cpc + ch * 16);
        uint8_t* y = D.yq + ((size_t)t * B + by) * a.yq_ld;
        const int c0 = (int)rank * cpc + ch * 16;
        if (y4) {
          auto pk = [](uint32_t w) -> uint32_t {
            const uint32_t m = (w & 0x000F000Fu) | ((w >> 4) & 0x00F000F0u);   // bytes 0 and 2 hold the pairs
            return (m & 0xFFu) | ((m >> 8) & 0xFF00u);
          };
          *reinterpret_cast<uint2*>(y + (c0 >> 1)) = make_uint2(pk(v.x) | (pk(v.y) << 16), pk(v.z) | (pk(v.w) << 16));
        } else {
          *reinterpret_cast<uint4*>(y + c0) = v;
        }
      }
    }
    if (window_end && w1 < T) {
      // hand the shared group on: cell states by every thread, codes by the sending warp above
      a.hand_c[d][(size_t)n * H + cell] = c_shared;
      __threadfence();
      __syncthreads();
      if (tid == 0) atomicAdd(flag_out, 1);
    }
  }
  cp_async_wait<0>();
  // the own group's codes sent in its last step are still on their way into this CTA: wait for them
  // (bounded), so that nobody leaves while copies into its shared memory are in flight.  (The shared
  // group sends nothing in the last step of its stay.)
  if (T > 0) {
    const uint32_t parity = (uint32_t)(((T - 1) >> 1) & 1);
    for (uint32_t it = 0; it < (1u << 22); ++it) {
      if (mbar_try_wait(&full[0 * 2 + (T & 1)], parity)) break;
      if ((it & 255u) == 255u && *dead) break;
    }
  }
  __syncthreads();
  cluster_barrier();
  if (live_own && D.c_n) D.c_n[(size_t)b_own * H + cell] = c_own;
  if (live_shared && w1 == T && D.c_n) D.c_n[(size_t)b_shared * H + cell] = c_shared;
}

constexpr size_t REC_SMEM_MAX = 232448 - 128;   // 227 KB per CTA on sm_100, minus a margin

size_t enc_recurrent_smem(int H, int BG) {
  return (size_t)(4 * (H / REC_CLUSTER)) * (H + 16) + (size_t)2 * BG * (H + 16) +
         (size_t)BG * (H / REC_CLUSTER) + 16;
}

template <int BG>
static cudaError_t rec_launch(const EncRecArgs& a, size_t smem, cudaStream_t s) {
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(k_enc_recurrent<BG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  k_enc_recurrent<BG><<<(unsigned)(a.dirs * a.n_groups * REC_CLUSTER), REC_THREADS, smem, s>>>(a);
  return cudaGetLastError();
}

// How many 8-CTA clusters of this kernel can be resident at once on the current device
// (15 on a 148-SM B200: clusters do not straddle GPCs); asked once.
static int rec_max_clusters(int H) {
  static int cached = 0;
  if (cached > 0) return cached;
  const size_t smem = enc_recurrent_smem(H, 8);
  int n = 0;
  if (cudaFuncSetAttribute(k_enc_recurrent<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(REC_CLUSTER * 16);
    cfg.blockDim = dim3(REC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = REC_CLUSTER;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, k_enc_recurrent<8>, &cfg) != cudaSuccess) n = 0;
  }
  cached = n > 0 ? n : 15;
  return cached;
}

// The same question for the kernel whose clusters may take turns (its int8 variant, the one with the
// larger shared-memory footprint); asked once.  The plan takes the smaller of the two answers, so that
// every cluster of a launch is resident at once (a cluster that was not would only start later: a
// waiting cluster only waits for lower-numbered ones; but its direction would finish that much later).
static int rec_turns_max_clusters() {
  static int cached = 0;
  if (cached > 0) return cached;
  constexpr int H = 640, cpc = H / REC_CLUSTER;
  const size_t smem = (size_t)2 * 2 * REC_BG * H + (size_t)2 * REC_THREADS * sizeof(int4) + (size_t)3 * cpc * sizeof(float4) +
                      (size_t)4 * 2 * REC_BG * cpc + (size_t)2 * 2 * sizeof(uint64_t) + 32 +
                      (size_t)rec_turns_ksmem(true) * REC_THREADS * sizeof(uint4);
  int n = 0;
  if (cudaFuncSetAttribute(k_enc_recurrent_w4s<20, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(REC_CLUSTER * 16);
    cfg.blockDim = dim3(REC4_THREADS);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = REC_CLUSTER;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, k_enc_recurrent_w4s<20, true>, &cfg) != cudaSuccess) n = 0;
  }
  cached = n > 0 ? n : 15;
  return cached;
}

// Sequences per cluster: 8 or 16 (one or two MMA tiles), whichever gives the smaller estimated
// layer time = waves * (fixed cost + cost per sequence); a step's work grows with the group
// size, a second wave doubles everything.
int enc_recurrent_group(int B, int dirs, int H) {
  const int maxc = rec_max_clusters(H);
  int best = 8;
  double best_cost = 1e30;
  for (int bg = 8; bg <= 16; bg += 8) {
    if (enc_recurrent_smem(H, bg) > REC_SMEM_MAX) continue;
    const int clusters = dirs * ((B + bg - 1) / bg);
    const int waves = (clusters + maxc - 1) / maxc;
    const double cost = waves * (3.0 + bg);
    if (cost < best_cost) {
      best_cost = cost;
      best = bg;
    }
  }
  return best;
}

static int g_rec_sliced = 1;
int enc_recurrent_sliced_set(int enabled) {
  const int prev = g_rec_sliced;
  g_rec_sliced = enabled ? 1 : 0;
  return prev;
}

bool enc_recurrent_supported(int H, int B, int dirs) {
  (void)B;
  (void)dirs;
  if (H % 32 != 0 || H / REC_CLUSTER > 80) return false;
  return enc_recurrent_smem(H, 8) <= REC_SMEM_MAX;
}

static size_t enc_recurrent_w4_smem(int H, int NU) {
  const int cpc = H / REC_CLUSTER;
  return (size_t)NU * 2 * REC_BG * H + (size_t)2 * NU * REC_THREADS * sizeof(int4) +
         (size_t)3 * cpc * sizeof(float4) + (size_t)4 * NU * REC_BG * cpc + (size_t)NU * 2 * sizeof(uint64_t) + 32 + (size_t)rec_w4_ksmem(NU) * REC_THREADS * sizeof(uint2);
}

template <int KS, bool W8>
static cudaError_t rec_w4s_launch(const EncRecArgs& a, cudaStream_t s) {
  const int H = 32 * KS, cpc = H / REC_CLUSTER;
  const size_t smem = (size_t)2 * 2 * REC_BG * H + (size_t)2 * REC_THREADS * sizeof(int4) + (size_t)3 * cpc * sizeof(float4) +
                      (size_t)4 * 2 * REC_BG * cpc + (size_t)2 * 2 * sizeof(uint64_t) + 32 +
                      (size_t)rec_turns_ksmem(W8) * REC_THREADS * (W8 ? sizeof(uint4) : sizeof(uint2));
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_enc_recurrent_w4s<KS, W8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  k_enc_recurrent_w4s<KS, W8><<<(unsigned)((a.ncl[0] + a.ncl[1]) * REC_CLUSTER), REC4_THREADS, smem, s>>>(a);
  return cudaGetLastError();
}

template <int NU, int KS>
static cudaError_t rec_w4_launch(const EncRecArgs& a, cudaStream_t s) {
  const size_t smem = enc_recurrent_w4_smem(32 * KS, NU);
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_enc_recurrent_w4<NU, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  k_enc_recurrent_w4<NU, KS><<<(unsigned)(a.dirs * a.n_groups * REC_CLUSTER), REC4_THREADS, smem, s>>>(a);
  return cudaGetLastError();
}

EncRecPlan enc_recurrent_plan(int T, int B, int dirs, int H, int w_bits, int hid_bits, bool hid_signed,
                              bool per_sequence_scale, bool dump, bool scratch) {
  EncRecPlan p;
  memset(&p, 0, sizeof(p));
  const int groups = (B + REC_BG - 1) / REC_BG;
  p.groups = groups;
  p.max_clusters = rec_max_clusters(H);
  if (H == 640) p.max_clusters = p.max_clusters < rec_turns_max_clusters() ? p.max_clusters : rec_turns_max_clusters();
  // 640 cells, no accumulator dump: the kernels that keep (most of) a CTA's recurrent weights in
  // registers; the general kernel otherwise
  const bool regs_ok = hid_signed && H == 640 && !dump && (w_bits == 4 || w_bits == 8) && (hid_bits == 4 || hid_bits == 8);
  if (regs_ok) {
    // The kernel whose clusters may take turns: with one group more than clusters per sliced
    // direction, and (all directions plain) for what the packed kernel below does not take: int8
    // weights, 8-bit hidden codes, an input scale per sequence.
    const int lack = dirs * groups - p.max_clusters;
    const bool plain_only = w_bits == 8 || hid_bits == 8 || per_sequence_scale;
    const bool turns = g_rec_sliced && lack >= 1 && lack <= dirs && groups >= 2 && groups <= 8 && T >= 8 * groups && scratch;
    if (turns || (lack <= 0 && plain_only && groups <= 8 && scratch)) {
      p.kernel = 2;
      p.groups_per_cluster = 1;
      for (int d = 0; d < 2; ++d) {
        p.sliced[d] = turns && d < dirs && d < lack ? 1 : 0;
        p.ncl[d] = d < dirs ? groups - p.sliced[d] : 0;
      }
      if (turns)   // equal shares of the T steps, in cluster order
        for (int j = 0; j <= groups - 1; ++j) p.win[j] = (int)((long long)j * T / (groups - 1));
      return p;
    }
  }
  // packed 4-bit weights with as few groups of 8 sequences per cluster as keeps all clusters resident
  if (regs_ok && w_bits == 4 && hid_bits == 4 && !per_sequence_scale) {
    int nu = 1;
    while (nu <= 4 && dirs * ((groups + nu - 1) / nu) > p.max_clusters) ++nu;
    if (nu <= 4) {
      p.kernel = 1;
      p.groups_per_cluster = nu;
      p.ncl[0] = (groups + nu - 1) / nu;
      p.ncl[1] = dirs == 2 ? p.ncl[0] : 0;
      return p;
    }
  }
  p.kernel = 0;
  return p;
}

cudaError_t launch_enc_recurrent(EncRecArgs a, cudaStream_t s) {
  const EncRecPlan p = enc_recurrent_plan(a.T, a.B, a.dirs, a.H, a.w_bits, a.hid_act.bits, a.hid_act.is_signed != 0,
                                          a.x_scale_b != nullptr, a.d[0].dbg_ih != nullptr,
                                          a.flags && a.hand_h[0] && a.hand_c[0]);
  if (p.kernel == 2) {
    a.groups = p.groups;
    for (int d = 0; d < 2; ++d) {
      a.sliced[d] = p.sliced[d];
      a.ncl[d] = p.ncl[d];
    }
    for (int j = 0; j < 9; ++j) a.win[j] = p.win[j];
    timing_begin(s);
    cudaError_t e = a.w_bits == 8 ? rec_w4s_launch<20, true>(a, s) : rec_w4s_launch<20, false>(a, s);
    timing_end(s);
    ++g_launches;
    return e;
  }
  if (p.kernel == 1) {
    const int nu = p.groups_per_cluster;
    a.n_groups = p.ncl[0];   // clusters per direction
    timing_begin(s);
    cudaError_t e = nu == 1 ? rec_w4_launch<1, 20>(a, s) : nu == 2 ? rec_w4_launch<2, 20>(a, s)
                    : nu == 3 ? rec_w4_launch<3, 20>(a, s) : rec_w4_launch<4, 20>(a, s);
    timing_end(s);
    ++g_launches;
    return e;
  }
  const int BG = enc_recurrent_group(a.B, a.dirs, a.H);
  a.n_groups = (a.B + BG - 1) / BG;
  const size_t smem = enc_recurrent_smem(a.H, BG);
  timing_begin(s);
  cudaError_t e;
  if (BG == 8)
    e = rec_launch<8>(a, smem, s);
  else
    e = rec_launch<16>(a, smem, s);
  timing_end(s);
  ++g_launches;
  return e;
}

}  // namespace q4
