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

bool enc_recurrent_supported(int H, int B, int dirs) {
  (void)B;
  (void)dirs;
  if (H % 32 != 0 || H / REC_CLUSTER > 80) return false;
  return enc_recurrent_smem(H, 8) <= REC_SMEM_MAX;
}

cudaError_t launch_enc_recurrent(EncRecArgs a, cudaStream_t s) {
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
