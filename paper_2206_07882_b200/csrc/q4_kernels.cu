// Core kernels: quantize+pack (Eq. 2), the integer tile GEMM with fused epilogues
// (store / de-quantize+bias / re-quantize), the LSTM step with fused de-quantization,
// gates, cell update and output quantization (Sections 3.2, 3.4), joint element-wise
// stage, row log-softmax, and the feature prologue.
#include "q4_internal.h"

namespace q4 {

int64_t g_launches = 0;
int64_t g_quant_calls = 0;   // activation-quantizer applications (Section 3.4), see q4_quantizer_calls
int g_tag = TAG_NONE;
int g_dependent_launch = 1;

// Optional event timing of tagged launches: the caller lends pairs of CUDA events; every
// launch whose tag is enabled records one pair on its own stream.  Off by default.
struct Timing {
  uint32_t mask = 0;
  cudaEvent_t* start = nullptr;
  cudaEvent_t* stop = nullptr;
  int32_t* tags = nullptr;
  int cap = 0, n = 0;
  bool open = false;
} g_timing;

void timing_begin(cudaStream_t s) {
  Timing& t = g_timing;
  t.open = false;
  if (!(t.mask >> g_tag & 1u) || t.n >= t.cap) return;
  cudaEventRecord(t.start[t.n], s);
  t.open = true;
}
void timing_end(cudaStream_t s) {
  Timing& t = g_timing;
  if (!t.open) return;
  cudaEventRecord(t.stop[t.n], s);
  t.tags[t.n] = g_tag;
  ++t.n;
  t.open = false;
}
void timing_set(uint32_t mask, cudaEvent_t* start, cudaEvent_t* stop, int32_t* tags, int cap) {
  g_timing.mask = mask;
  g_timing.start = start;
  g_timing.stop = stop;
  g_timing.tags = tags;
  g_timing.cap = cap;
  g_timing.n = 0;
  g_timing.open = false;
}
int timing_count() { return g_timing.n; }

// =====================================================================================
// Integer tile GEMM: acc[m, j] = sum_k W[j,k] * (x[m,k] - z).  64 x 64 outputs per CTA,
// K staged through shared memory in chunks of 128 as int8, DP4A accumulation in int32.
// Thread (ty, tx) owns rows 4ty..4ty+3 and columns 4tx..4tx+3; column c is staged in
// shared row c/4 + 16*(c%4) so that the 16-byte reads of a quarter warp hit distinct banks.
// =====================================================================================
template <int EPI>
__global__ void __launch_bounds__(NT) k_gemm(const __grid_constant__ GemmArgs a) {
  __shared__ __align__(16) int8_t Xs[TILE * PITCH];
  __shared__ __align__(16) int8_t Ws[TILE * PITCH];
  __shared__ const uint8_t* xrow[TILE];
  __shared__ const uint8_t* wrow[TILE];
  __shared__ int orow[TILE];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.x * TILE, j0 = blockIdx.y * TILE;
  int active = 0;
  if (tid < TILE) {
    const int m = m0 + tid;
    const uint8_t* p = nullptr;
    int o = -1;
    if (m < a.M && !(a.n_active && m >= *a.n_active)) {
      o = a.out_idx ? a.out_idx[m] : m;
      const int r = a.x.idx ? a.x.idx[m] : m;
      if (o >= 0 && r >= 0) p = a.x.base + (long long)r * a.x.stride;
      if (r < 0) o = -1;
    }
    xrow[tid] = p;
    orow[tid] = o;
    active = o >= 0;
  } else if (tid < 2 * TILE) {
    const int s = tid - TILE;
    const int c = ((s & 15) << 2) | (s >> 4);
    const int j = j0 + c;
    wrow[s] = j < a.J ? a.w + (long long)j * (a.k_pad * a.w_bits / 8) : nullptr;
  }
  if (!__syncthreads_or(active)) return;

  const int ty = tid >> 4, tx = tid & 15;
  const uint32_t zp4 = (uint32_t)a.x_zp * 0x01010101u;
  int acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0;

  for (int k0 = 0; k0 < a.k_pad; k0 += KC) {
    stage_chunk(Xs, xrow, k0, a.k_pad, a.x_bits, a.x_signed != 0, zp4, tid);
    stage_chunk(Ws, wrow, k0, a.k_pad, a.w_bits, true, 0u, tid);
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < KC; kk += 16) {
      int4 xv[4], wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        xv[i] = *reinterpret_cast<const int4*>(Xs + (ty * 4 + i) * PITCH + kk);
        wv[i] = *reinterpret_cast<const int4*>(Ws + (tx + 16 * i) * PITCH + kk);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          int v = acc[i][j];
          v = dp4a(xv[i].x, wv[j].x, v);
          v = dp4a(xv[i].y, wv[j].y, v);
          v = dp4a(xv[i].z, wv[j].z, v);
          v = dp4a(xv[i].w, wv[j].w, v);
          acc[i][j] = v;
        }
    }
    __syncthreads();
  }

  const int jb = j0 + tx * 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    const int o = orow[ty * 4 + i];
    if (o < 0) continue;
    if (a.dbg_acc) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (jb + j < a.J) a.dbg_acc[(long long)m * a.J + jb + j] = acc[i][j];
    }
    if (EPI == EPI_I32) {
      int32_t* out = reinterpret_cast<int32_t*>(a.out) + (long long)o * a.out_stride;
      if (jb + 3 < a.J) {
        *reinterpret_cast<int4*>(out + jb) = make_int4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (jb + j < a.J) out[jb + j] = acc[i][j];
      }
    } else {
      float v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int jj = min(jb + j, a.J - 1);
        const float b = a.bias ? a.bias[jj] : 0.0f;
        v[j] = __fmaf_rn((float)acc[i][j], __fmul_rn(a.x_scale, a.w_scale[jj]), b);
      }
      if (EPI == EPI_F32) {
        float* out = reinterpret_cast<float*>(a.out) + (long long)o * a.out_stride;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (jb + j < a.J) out[jb + j] = v[j];
      } else {
        if (jb >= a.J) continue;  // J is a multiple of 4 here
        const int lo = act_lo(a.out_act), hi = act_hi(a.out_act);
        int q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
          q[j] = quantize1(v[j], a.out_act.inv_scale, a.out_act.zero_point, lo, hi);
        uint8_t* out = reinterpret_cast<uint8_t*>(a.out) + (long long)o * a.out_stride;
        if (a.out_act.bits == 4) {
          const uint16_t pk = (uint16_t)((q[0] & 0xF) | ((q[1] & 0xF) << 4) | ((q[2] & 0xF) << 8) |
                                         ((q[3] & 0xF) << 12));
          *reinterpret_cast<uint16_t*>(out + (jb >> 1)) = pk;
        } else {
          const uint32_t pk = (uint32_t)(q[0] & 0xFF) | ((uint32_t)(q[1] & 0xFF) << 8) |
                              ((uint32_t)(q[2] & 0xFF) << 16) | ((uint32_t)(q[3] & 0xFF) << 24);
          *reinterpret_cast<uint32_t*>(out + jb) = pk;
        }
      }
    }
  }
}

cudaError_t launch_gemm(const GemmArgs& a, int epi, cudaStream_t s) {
  if (a.M <= 0 || a.J <= 0) return cudaSuccess;
  dim3 grid((a.M + TILE - 1) / TILE, (a.J + TILE - 1) / TILE);
#define Q4_GEMM_CASE(E_)                               \
  if (epi == E_) {                                     \
    timing_begin(s);                                   \
    k_gemm<E_><<<grid, NT, 0, s>>>(a);                 \
    timing_end(s);                                     \
    ++g_launches;                                      \
    return cudaGetLastError();                         \
  }
  Q4_GEMM_CASE(EPI_I32)
  Q4_GEMM_CASE(EPI_F32)
  Q4_GEMM_CASE(EPI_QUANT)
#undef Q4_GEMM_CASE
  return cudaErrorInvalidValue;
}

// =====================================================================================
// LSTM step.  A CTA owns 16 cells (their i, f, g, o rows = 64 weight rows) for 64 rows
// of the batch; a thread owns 2 rows x 2 adjacent cells x 4 gates, so the whole cell
// update and the packing of two 4-bit codes into a byte stay in registers.
// Cell c of the tile is staged in shared row gate*16 + (c%2)*8 + c/2.
// =====================================================================================
__device__ __forceinline__ void lstm_mac(int (&acc)[2][2][4], const int8_t* Xs, const int8_t* Ws,
                                         int rp, int cp) {
#pragma unroll
  for (int kk = 0; kk < KC; kk += 16) {
    int4 xv[2], wv[2][4];
#pragma unroll
    for (int r = 0; r < 2; ++r) xv[r] = *reinterpret_cast<const int4*>(Xs + (2 * rp + r) * PITCH + kk);
#pragma unroll
    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
      for (int g = 0; g < 4; ++g)
        wv[cc][g] = *reinterpret_cast<const int4*>(Ws + (g * 16 + cc * 8 + cp) * PITCH + kk);
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int cc = 0; cc < 2; ++cc)
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          int v = acc[r][cc][g];
          v = dp4a(xv[r].x, wv[cc][g].x, v);
          v = dp4a(xv[r].y, wv[cc][g].y, v);
          v = dp4a(xv[r].z, wv[cc][g].z, v);
          v = dp4a(xv[r].w, wv[cc][g].w, v);
          acc[r][cc][g] = v;
        }
  }
}

__global__ void __launch_bounds__(NT) k_lstm(const __grid_constant__ LstmArgs2 args) {
  const LstmArgs& a = args.d[blockIdx.z];
  __shared__ __align__(16) int8_t Xs[TILE * PITCH];
  __shared__ __align__(16) int8_t Ws[TILE * PITCH];
  __shared__ const uint8_t* xrow[TILE];
  __shared__ const uint8_t* wrow[TILE];
  __shared__ int hrow[TILE];
  __shared__ int orow[TILE];
  const int tid = threadIdx.x;
  const int n0 = blockIdx.x * TILE, c0 = blockIdx.y * 16;
  const int H = a.H;
  int active = 0;
  if (tid < TILE) {
    const int n = n0 + tid;
    int hi = -1, oi = -1;
    const uint8_t* p = nullptr;
    if (n < a.N && !(a.n_active && n >= *a.n_active)) {
      oi = a.out_idx ? a.out_idx[n] : n;
      if (oi >= 0) {
        hi = a.hin.idx ? a.hin.idx[n] : n;
        if (!a.acc_pre) {
          const int xi = a.x.idx ? a.x.idx[n] : n;
          if (xi >= 0) p = a.x.base + (long long)xi * a.x.stride;
        }
      }
    }
    xrow[tid] = p;
    hrow[tid] = hi;
    orow[tid] = oi;
    active = oi >= 0;
  } else if (tid < 2 * TILE) {
    const int s = tid - TILE, g = s >> 4, q = s & 15;
    const int cell = c0 + (((q & 7) << 1) | (q >> 3));
    wrow[s] = cell < H ? a.w_ih + (long long)(g * H + cell) * (a.kx_pad * a.wih_bits / 8) : nullptr;
  }
  if (!__syncthreads_or(active)) return;

  const int cp = tid & 7, rp = tid >> 3;
  const int cell0 = c0 + 2 * cp;
  int acc[2][2][4];
  float pre[2][2][4];
#pragma unroll
  for (int r = 0; r < 2; ++r)
#pragma unroll
    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
      for (int g = 0; g < 4; ++g) acc[r][cc][g] = 0;

  // ---- input contribution
  if (a.acc_pre) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int n = n0 + 2 * rp + r;
      if (n < a.N && orow[2 * rp + r] >= 0 && cell0 < H) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const int2 v = *reinterpret_cast<const int2*>(a.acc_pre + (long long)n * a.acc_pre_stride +
                                                        g * H + cell0);
          acc[r][0][g] = v.x;
          acc[r][1][g] = v.y;
        }
      }
    }
  } else {
    const uint32_t zp4 = (uint32_t)a.x_zp * 0x01010101u;
    for (int k0 = 0; k0 < a.kx_pad; k0 += KC) {
      stage_chunk(Xs, xrow, k0, a.kx_pad, a.x_bits, a.x_signed != 0, zp4, tid);
      stage_chunk(Ws, wrow, k0, a.kx_pad, a.wih_bits, true, 0u, tid);
      __syncthreads();
      lstm_mac(acc, Xs, Ws, rp, cp);
      __syncthreads();
    }
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int n = n0 + 2 * rp + r;
    const bool ok = n < a.N && orow[2 * rp + r] >= 0;
    const float sx = (ok && a.x_scale_vec) ? a.x_scale_vec[n % a.x_scale_mod] : a.x_scale;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const int j = g * H + min(cell0 + cc, H - 1);
        const float b = a.bias ? a.bias[j] : 0.0f;
        pre[r][cc][g] = __fmaf_rn((float)acc[r][cc][g], __fmul_rn(sx, a.s_wih[j]), b);
        if (ok && a.dbg_ih && cell0 + cc < H) a.dbg_ih[(long long)n * a.dbg_stride + j] = acc[r][cc][g];
        acc[r][cc][g] = 0;
      }
  }

  // ---- recurrent contribution
  if (tid < TILE) {
    const int hi = hrow[tid];
    xrow[tid] = (orow[tid] >= 0 && hi >= 0) ? a.hin.base + (long long)hi * a.hin.stride : nullptr;
  } else if (tid < 2 * TILE) {
    const int s = tid - TILE, g = s >> 4, q = s & 15;
    const int cell = c0 + (((q & 7) << 1) | (q >> 3));
    wrow[s] = cell < H ? a.w_hh + (long long)(g * H + cell) * (a.kh_pad * a.whh_bits / 8) : nullptr;
  }
  __syncthreads();
  for (int k0 = 0; k0 < a.kh_pad; k0 += KC) {
    stage_chunk(Xs, xrow, k0, a.kh_pad, a.hid_act.bits, true, 0u, tid);
    stage_chunk(Ws, wrow, k0, a.kh_pad, a.whh_bits, true, 0u, tid);
    __syncthreads();
    lstm_mac(acc, Xs, Ws, rp, cp);
    __syncthreads();
  }

  // ---- gates, cell update, output quantization (once, at the cell output)
  const float sh = a.hid_act.scale;
  const int hlo = act_lo(a.hid_act), hhi = act_hi(a.hid_act);
  const int ylo = act_lo(a.out_act), yhi = act_hi(a.out_act);
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int n = n0 + 2 * rp + r;
    const int oi = orow[2 * rp + r];
    if (n >= a.N || oi < 0 || cell0 >= H) continue;
    const int hi = hrow[2 * rp + r];
    int q[2], q2[2];
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      const int cell = cell0 + cc;
      float g4[4];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const int j = g * H + cell;
        if (a.dbg_hh) a.dbg_hh[(long long)n * a.dbg_stride + j] = acc[r][cc][g];
        g4[g] = __fmaf_rn((float)acc[r][cc][g], __fmul_rn(sh, a.s_whh[j]), pre[r][cc][g]);
      }
      const float cprev = hi >= 0 ? a.c_in[(long long)hi * H + cell] : 0.0f;
      float c, h;
      cell_fixed(g4[0], g4[1], g4[2], g4[3], cprev, c, h);
      a.c_out[(long long)oi * H + cell] = c;
      if (a.h_f32) a.h_f32[(long long)n * H + cell] = h;
      q[cc] = quantize1(h, a.hid_act.inv_scale, a.hid_act.zero_point, hlo, hhi);
      q2[cc] = quantize1(h, a.out_act.inv_scale, a.out_act.zero_point, ylo, yhi);
    }
    if (a.hq_out == nullptr) {
      // Inner placement (Section 3.4): nothing is quantized at the cell output
    } else if (a.hid_act.bits == 4) {
      a.hq_out[(long long)oi * a.hq_stride + (cell0 >> 1)] = (uint8_t)((q[0] & 0xF) | ((q[1] & 0xF) << 4));
    } else {
      *reinterpret_cast<uint16_t*>(a.hq_out + (long long)oi * a.hq_stride + cell0) =
          (uint16_t)((q[0] & 0xFF) | ((q[1] & 0xFF) << 8));
    }
    if (a.yq_out) {
      if (a.out_act.bits == 4) {
        a.yq_out[(long long)n * a.yq_stride + (cell0 >> 1)] = (uint8_t)((q2[0] & 0xF) | ((q2[1] & 0xF) << 4));
      } else {
        *reinterpret_cast<uint16_t*>(a.yq_out + (long long)n * a.yq_stride + cell0) =
            (uint16_t)((q2[0] & 0xFF) | ((q2[1] & 0xFF) << 8));
      }
    }
  }
}

cudaError_t launch_lstm(const LstmArgs2& a, int dirs, cudaStream_t s) {
  const LstmArgs& a0 = a.d[0];
  if (a0.N <= 0) return cudaSuccess;
  dim3 grid((a0.N + TILE - 1) / TILE, (a0.H + 15) / 16, dirs);
  timing_begin(s);
  k_lstm<<<grid, NT, 0, s>>>(a);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}

// =====================================================================================
// Row log-softmax: out = x - max - log(sum(exp(x - max))).  One CTA per row; rows are
// addressed through idx (nullptr = identity, negative = skip); in place is allowed.
// =====================================================================================
__device__ __forceinline__ float block_reduce(float v, bool is_max, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float w = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, w) : v + w;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  v = lane < nw ? red[lane] : (is_max ? -INFINITY : 0.0f);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float w = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, w) : v + w;
  }
  return v;
}

__global__ void __launch_bounds__(256) k_logsoftmax(const float* in, float* out, int V,
                                                    long long stride, const int32_t* idx,
                                                    float* second, const int32_t* n_active) {
  __shared__ float red[32];
  if (n_active && (int)blockIdx.x >= *n_active) return;
  const int r = idx ? idx[blockIdx.x] : (int)blockIdx.x;
  if (r < 0) return;
  // blockIdx.y == 1 treats a second matrix with the same row indices, in place
  const float* x = (blockIdx.y ? second : in) + (long long)r * stride;
  float* y = (blockIdx.y ? second : out) + (long long)r * stride;
  float m = -INFINITY;
  for (int v = threadIdx.x; v < V; v += blockDim.x) m = fmaxf(m, x[v]);
  m = block_reduce(m, true, red);
  float s = 0.0f;
  for (int v = threadIdx.x; v < V; v += blockDim.x) s += expf(x[v] - m);
  s = block_reduce(s, false, red);
  const float lse = m + logf(s);
  for (int v = threadIdx.x; v < V; v += blockDim.x) y[v] = x[v] - lse;
}

cudaError_t launch_logsoftmax(const float* in, float* out, int rows, int V, long long stride,
                              const int32_t* idx, cudaStream_t s, float* second,
                              const int32_t* n_active) {
  if (rows <= 0) return cudaSuccess;
  timing_begin(s);
  k_logsoftmax<<<dim3(rows, second ? 2 : 1), 256, 0, s>>>(in, out, V, stride, idx, second, n_active);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}

// =====================================================================================
// Joint element-wise stage: z = tanh(e * p), quantized with z_act (Section 2: the two
// representations are combined multiplicatively).  Two adjacent elements per thread.
// Row n reads e row frame_idx[n] (or t_arr[n]*B + n/W when t_arr is given) and p row
// p_idx[n] (nullptr = n).  A row with a negative index writes zero codes and, when
// live_out is given, live_out[n] = -1 (else n).
// =====================================================================================
__global__ void __launch_bounds__(256) k_joint_z(const float* e, const int32_t* frame_idx,
                                                 const int32_t* t_arr, int B, int W, const float* p,
                                                 const int32_t* p_idx, int N, int D, q4_act za,
                                                 uint8_t* zq, int8_t* z8, int32_t* live_out) {
  pdl_trigger();
  pdl_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int half = D >> 1;
  if (i >= (long long)N * half) return;
  const int n = (int)(i / half), d = (int)(i % half) * 2;
  const int pr = p_idx ? p_idx[n] : n;
  int er = -1;
  if (pr >= 0) er = t_arr ? t_arr[n] * B + n / W : frame_idx[n];
  int q0 = 0, q1 = 0;
  if (pr >= 0 && er >= 0) {
    const float2 ev = *reinterpret_cast<const float2*>(e + (long long)er * D + d);
    const float2 pv = *reinterpret_cast<const float2*>(p + (long long)pr * D + d);
    const int lo = act_lo(za), hi = act_hi(za);
    q0 = quantize1(tanh_fixed(__fmul_rn(ev.x, pv.x)), za.inv_scale, za.zero_point, lo, hi);
    q1 = quantize1(tanh_fixed(__fmul_rn(ev.y, pv.y)), za.inv_scale, za.zero_point, lo, hi);
  }
  if (z8) {   // one code per byte, ready for the tensor-core GEMM
    *reinterpret_cast<uint16_t*>(z8 + (long long)n * D + d) = (uint16_t)((q0 & 0xFF) | ((q1 & 0xFF) << 8));
  } else if (za.bits == 4) {
    zq[(long long)n * half + (d >> 1)] = (uint8_t)((q0 & 0xF) | ((q1 & 0xF) << 4));
  } else {
    *reinterpret_cast<uint16_t*>(zq + (long long)n * D + d) = (uint16_t)((q0 & 0xFF) | ((q1 & 0xFF) << 8));
  }
  if (live_out && d == 0) live_out[n] = (pr >= 0 && er >= 0) ? n : -1;
}

cudaError_t launch_joint_z(const float* e, const int32_t* frame_idx, const int32_t* t_arr, int B,
                           int W, const float* p, const int32_t* p_idx, int N, int D,
                           const q4_act& za, uint8_t* zq, int8_t* z8, int32_t* live_out,
                           cudaStream_t s, bool dependent) {
  if (N <= 0) return cudaSuccess;
  const long long total = (long long)N * (D / 2);
  timing_begin(s);
  cudaError_t le = launch_ex(k_joint_z, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, s, dependent, 1, e,
                             frame_idx, t_arr, B, W, p, p_idx, N, D, za, zq, z8, live_out);
  timing_end(s);
  ++g_launches;
  return le != cudaSuccess ? le : cudaGetLastError();
}

// =====================================================================================
// quantize_pack: Eq. 2 on fp16/fp32 rows, eight output codes per thread.
// =====================================================================================
template <bool FP16>
__device__ __forceinline__ float ldx(const void* x, long long i) {
  return FP16 ? __half2float(reinterpret_cast<const __half*>(x)[i]) : reinterpret_cast<const float*>(x)[i];
}

// scale_mode 0: constants in `a`; 1: per-group scale vector (row % n_groups); 2: per-row scale.
template <bool FP16>
__global__ void __launch_bounds__(256) k_quantize(const void* x, long long rows, int k, int k_pad,
                                                  q4_act a, int scale_mode, int n_groups,
                                                  const float* scale_vec, uint8_t* out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = k_pad >> 3;
  if (i >= rows * per_row) return;
  const long long r = i / per_row;
  const int kb = (int)(i % per_row) * 8;
  float inv = a.inv_scale;
  if (scale_mode == 1) inv = __fdiv_rn(1.0f, scale_vec[r % n_groups]);
  if (scale_mode == 2) inv = __fdiv_rn(1.0f, scale_vec[r]);
  const int lo = act_lo(a), hi = act_hi(a);
  int q[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int kk = kb + j;
    q[j] = kk < k ? quantize1(ldx<FP16>(x, r * k + kk), inv, a.zero_point, lo, hi)
                  : (a.is_signed ? 0 : a.zero_point);
  }
  if (a.bits == 4) {
    uint32_t w = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) w |= (uint32_t)(q[j] & 0xF) << (4 * j);
    *reinterpret_cast<uint32_t*>(out + r * (k_pad >> 1) + (kb >> 1)) = w;
  } else if (a.bits == 2) {   // weights only: four codes per byte, element i in bits 2i, 2i+1
    uint32_t w = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) w |= (uint32_t)(q[j] & 0x3) << (2 * j);
    *reinterpret_cast<uint16_t*>(out + r * (k_pad >> 2) + (kb >> 2)) = (uint16_t)w;
  } else {
    uint2 w = make_uint2(0, 0);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      w.x |= (uint32_t)(q[j] & 0xFF) << (8 * j);
      w.y |= (uint32_t)(q[j + 4] & 0xFF) << (8 * j);
    }
    *reinterpret_cast<uint2*>(out + r * k_pad + kb) = w;
  }
}

// largest magnitude per group (row % n_groups); non-negative floats order like their bits
template <bool FP16>
__global__ void __launch_bounds__(256) k_absmax(const void* x, long long rows, int k, int n_groups,
                                                uint32_t* amax_bits) {
  const long long r = blockIdx.x;
  if (r >= rows) return;
  float m = 0.0f;
  for (int j = threadIdx.x; j < k; j += blockDim.x) m = fmaxf(m, fabsf(ldx<FP16>(x, r * k + j)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0 && m > 0.0f) atomicMax(amax_bits + (r % n_groups), __float_as_uint(m));
}

__global__ void k_amax_to_scale(uint32_t* amax_bits, int n_groups, int qmax) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= n_groups) return;
  float m = __uint_as_float(amax_bits[g]);
  if (m == 0.0f) m = 1.0f;
  reinterpret_cast<float*>(amax_bits)[g] = __fdiv_rn(m, (float)qmax);
}

cudaError_t launch_quantize(const void* x, bool fp16, long long rows, int k, int k_pad,
                            const q4_act& a, int mode, int n_groups, const float* scale_vec,
                            uint8_t* out, float* group_scale_out, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  const float* sv = scale_vec;
  if (mode == 1) {
    cudaError_t e = cudaMemsetAsync(group_scale_out, 0, sizeof(float) * n_groups, s);
    if (e != cudaSuccess) return e;
    if (fp16)
      k_absmax<true><<<(unsigned)rows, 256, 0, s>>>(x, rows, k, n_groups, (uint32_t*)group_scale_out);
    else
      k_absmax<false><<<(unsigned)rows, 256, 0, s>>>(x, rows, k, n_groups, (uint32_t*)group_scale_out);
    k_amax_to_scale<<<(n_groups + 255) / 256, 256, 0, s>>>((uint32_t*)group_scale_out, n_groups,
                                                           (1 << (a.bits - 1)) - 1);
    g_launches += 2;
    sv = group_scale_out;
  }
  const long long total = rows * (k_pad >> 3);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  timing_begin(s);
  if (fp16)
    k_quantize<true><<<blocks, 256, 0, s>>>(x, rows, k, k_pad, a, mode, n_groups, sv, out);
  else
    k_quantize<false><<<blocks, 256, 0, s>>>(x, rows, k, k_pad, a, mode, n_groups, sv, out);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}

// =====================================================================================
// Feature prologue: time differences with replicated edges, then frame stacking.
// =====================================================================================
__device__ __forceinline__ float mel_at(const float* m, int T, int M, int t, int j) {
  t = max(0, min(t, T - 1));
  return m[(long long)t * M + j];
}
__device__ __forceinline__ float delta_at(const float* m, int T, int M, int t, int j) {
  t = max(0, min(t, T - 1));
  return __fmul_rn(__fsub_rn(mel_at(m, T, M, t + 1, j), mel_at(m, T, M, t - 1, j)), 0.5f);
}

__global__ void __launch_bounds__(256) k_features(const float* mel, int B, int T100, int M,
                                                  __half* out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * T100 * M) return;
  const int j = (int)(i % M);
  const int t = (int)((i / M) % T100);
  const int b = (int)(i / ((long long)M * T100));
  if (t >= (T100 / 2) * 2) return;
  const float* m = mel + (long long)b * T100 * M;
  const float x = m[(long long)t * M + j];
  const float d = delta_at(m, T100, M, t, j);
  const float dd = __fmul_rn(__fsub_rn(delta_at(m, T100, M, t + 1, j), delta_at(m, T100, M, t - 1, j)), 0.5f);
  __half* o = out + (((long long)(t >> 1) * B + b) * 2 + (t & 1)) * 3 * M;
  o[j] = __float2half_rn(x);
  o[M + j] = __float2half_rn(d);
  o[2 * M + j] = __float2half_rn(dd);
}

cudaError_t launch_features(const float* mel, int B, int T100, int M, void* out, cudaStream_t s) {
  const long long total = (long long)B * T100 * M;
  if (total <= 0) return cudaSuccess;
  timing_begin(s);
  k_features<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(mel, B, T100, M, (__half*)out);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}

}  // namespace q4
