// Beam bookkeeping kernels: per-utterance log-softmax of the joint logits, the
// density-ratio score of Eq. 1 for every proposal, merging of equal label strings,
// the finished list, selection of the W best, state-row allocation and back-pointers.
// One CTA per utterance; nothing here leaves the GPU (the paper ran hypothesis sorting
// on the host CPU, Section 4.1).
#include <math.h>

#include "q4_internal.h"

namespace q4 {

constexpr int SEL_NT = 512;
constexpr int MAXW = 16;
constexpr uint64_t HASH0 = 0x243F6A8885A308D3ull;  // hash of the empty label string

__device__ __forceinline__ uint64_t hash_mix(uint64_t h, uint32_t k) {
  uint64_t z = h ^ (0x9E3779B97F4A7C15ull * (uint64_t)(k + 1u));
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Order-preserving key: larger score first, then smaller proposal index
// (index = parent slot * V + token, so parent ascending then token ascending).
__device__ __forceinline__ uint64_t make_key(float s, uint32_t idx) {
  uint32_t b = __float_as_uint(s);
  b = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ((uint64_t)b << 32) | (uint64_t)(~idx);
}
__device__ __forceinline__ float key_score(uint64_t key) {
  uint32_t b = (uint32_t)(key >> 32);
  b = (b & 0x80000000u) ? (b & 0x7FFFFFFFu) : ~b;
  return __uint_as_float(b);
}
__device__ __forceinline__ uint64_t u64max(uint64_t a, uint64_t b) { return a > b ? a : b; }
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = u64max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__global__ void __launch_bounds__(SEL_NT) k_beam_select(const __grid_constant__ BeamSelArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* cand = reinterpret_cast<float*>(smem_raw);  // [W * V]
  __shared__ float s_score[MAXW];
  __shared__ int s_t[MAXW], s_u[MAXW], s_row[MAXW], s_last[MAXW];
  __shared__ uint64_t s_hash[MAXW], s_prev[MAXW];
  __shared__ uint64_t slot_top[MAXW][MAXW];   // per slot: its W best proposals, best first (0 = none)
  __shared__ int win_idx[MAXW];
  __shared__ float win_score[MAXW];
  __shared__ int n_win_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x, W = a.W, V = a.V;
  const int base = b * W;
  const q4_beam_state& st = a.st;
  const float NEG = -INFINITY;

  if (tid < W) {
    const int o = base + tid;
    s_row[tid] = st.row[o];
    s_score[tid] = st.score[o];
    s_t[tid] = st.t[o];
    s_u[tid] = st.u[o];
    s_last[tid] = st.last_tok[o];
    s_hash[tid] = st.hash[o];
    s_prev[tid] = st.prev_hash[o];
  }
  if (tid < MAXW * MAXW) slot_top[tid / MAXW][tid % MAXW] = 0ull;
  __syncthreads();

  // ---- proposals: one warp per slot; the row of logits is read once and kept in registers
  for (int w = warp; w < W; w += SEL_NT / 32) {
    float* cw = cand + (size_t)w * V;
    const int row = s_row[w];
    if (row < 0) {
      for (int k = lane; k < V; k += 32) cw[k] = NEG;
      continue;
    }
    const float* x = a.logits + (size_t)(base + w) * V;
    const float* lt = a.tgt_lp + (size_t)row * V;
    const float* ls = a.src_lp + (size_t)row * V;
    const double S = (double)s_score[w];
    const bool labels = s_u[w] < a.u_max;
    for (int k0 = 0; k0 < V; k0 += 1024) {      // V <= 1024: a single trip
      float xv[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int k = k0 + lane + 32 * i;
        xv[i] = k < V ? x[k] : NEG;
      }
      if (k0 == 0 && V <= 1024) {
        float m = NEG;
#pragma unroll
        for (int i = 0; i < 32; ++i) m = fmaxf(m, xv[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float sum = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += expf(xv[i] - m);   // exp(-inf) = 0 for the padding
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const float lse = m + logf(sum);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int k = lane + 32 * i;
          if (k >= V) continue;
          const float lp = xv[i] - lse;
          float v;
          if (k == 0) {
            v = (float)(S + (double)lp);
          } else if (labels) {
            v = (float)(S + (double)lp + (double)a.lambda_t * (double)lt[k] -
                        (double)a.lambda_s * (double)ls[k] + (double)a.rho);
          } else {
            v = NEG;
          }
          cw[k] = v;
        }
      }
    }
    if (V > 1024) {   // general vocabulary size: three passes over the row
      float m = NEG;
      for (int k = lane; k < V; k += 32) m = fmaxf(m, x[k]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      float sum = 0.0f;
      for (int k = lane; k < V; k += 32) sum += expf(x[k] - m);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float lse = m + logf(sum);
      for (int k = lane; k < V; k += 32) {
        const float lp = x[k] - lse;
        float v;
        if (k == 0) {
          v = (float)(S + (double)lp);
        } else if (labels) {
          v = (float)(S + (double)lp + (double)a.lambda_t * (double)lt[k] -
                      (double)a.lambda_s * (double)ls[k] + (double)a.rho);
        } else {
          v = NEG;
        }
        cw[k] = v;
      }
    }
  }
  __syncthreads();

  // ---- merge: label proposal (w2, k) describing the same string as the blank proposal of w
  if (tid < W * W) {
    const int w = tid / W, w2 = tid % W;
    if (s_row[w] >= 0 && s_row[w2] >= 0 && s_u[w] == s_u[w2] + 1 && s_prev[w] == s_hash[w2] &&
        s_u[w2] < a.u_max) {
      const int k = s_last[w];
      const double x = (double)cand[(size_t)w * V], y = (double)cand[(size_t)w2 * V + k];
      const double mx = fmax(x, y);
      cand[(size_t)w * V] = (float)(mx + log1p(exp(-fabs(x - y))));
      cand[(size_t)w2 * V + k] = NEG;
    }
  }
  __syncthreads();

  // ---- finished hypotheses: blank proposals that consume the last frame
  if (tid == 0) {
    float* fs = st.fin_score + base;
    int* fi = st.fin_iter + base;
    int* fl = st.fin_slot + base;
    int n = st.fin_n[b];
    bool any = false;
    for (int w = 0; w < W; ++w) {
      if (s_row[w] < 0 || s_t[w] + 1 != a.T) continue;
      any = true;
      const float S = cand[(size_t)w * V];
      cand[(size_t)w * V] = NEG;
      int pos = n;
      while (pos > 0 && fs[pos - 1] < S) --pos;
      if (pos >= W) continue;
      const int last = min(n, W - 1);
      for (int i = last; i > pos; --i) {
        fs[i] = fs[i - 1];
        fi[i] = fi[i - 1];
        fl[i] = fl[i - 1];
      }
      fs[pos] = S;
      fi[pos] = a.iter;
      fl[pos] = w;
      n = min(n + 1, W);
    }
    if (any) st.fin_n[b] = n;
  }
  __syncthreads();

  // ---- the W best remaining proposals.  Stage 1: every slot's own W best (one warp per slot)
  for (int w = warp; w < W; w += SEL_NT / 32) {
    if (s_row[w] < 0) continue;
    float* cw = cand + (size_t)w * V;
    const uint32_t off = (uint32_t)w * (uint32_t)V;
    uint64_t best = 0;
    for (int k = lane; k < V; k += 32) best = u64max(best, make_key(cw[k], off + (uint32_t)k));
    for (int r = 0; r < W; ++r) {
      const uint64_t g = warp_max_u64(best);
      if (!(key_score(g) > NEG)) break;
      if (lane == 0) slot_top[w][r] = g;
      const int k = (int)(~(uint32_t)g - off);
      if ((k & 31) == lane) {
        cw[k] = NEG;
        best = 0;
        for (int kk = lane; kk < V; kk += 32) best = u64max(best, make_key(cw[kk], off + (uint32_t)kk));
      }
    }
  }
  __syncthreads();
  // Stage 2: the W best of the (at most W*W) survivors, one warp, eight keys per lane
  if (warp == 0) {
    uint64_t mine[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) mine[i] = slot_top[lane >> 1][(lane & 1) * 8 + i];
    int n_win = 0;
    for (int r = 0; r < W; ++r) {
      uint64_t lb = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) lb = u64max(lb, mine[i]);
      const uint64_t g = warp_max_u64(lb);
      if (g == 0ull) break;
      if (lane == 0) {
        win_idx[r] = (int)(~(uint32_t)g);
        win_score[r] = key_score(g);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (mine[i] == g) mine[i] = 0ull;
      n_win = r + 1;
    }
    if (lane == 0) n_win_s = n_win;
    __syncwarp();

    // ---- next beam, state rows, back-pointers: lane s writes slot s
    const int nw = n_win;
    const int row0 = b * 2 * W;
    uint32_t used = 0;
    for (int w = 0; w < W; ++w)
      if (s_row[w] >= 0) used |= 1u << (s_row[w] - row0);
    const uint32_t free_mask = ~used & (W >= 16 ? 0xFFFFFFFFu : ((1u << (2 * W)) - 1u));
    const int s = lane;
    int idx = 0, w = 0, k = 0;
    bool is_label = false;
    if (s < nw) {
      idx = win_idx[s];
      w = idx / V;
      k = idx % V;
      is_label = k != 0;
    }
    const unsigned lab = __ballot_sync(0xffffffffu, is_label);
    if (s < W) {
      const int o = base + s;
      const size_t hist = ((size_t)a.iter * a.B + b) * W + s;
      if (s < nw) {
        st.score[o] = win_score[s];
        if (!is_label) {
          st.t[o] = s_t[w] + 1;
          st.u[o] = s_u[w];
          st.hash[o] = s_hash[w];
          st.prev_hash[o] = s_prev[w];
          st.last_tok[o] = s_last[w];
          st.row[o] = s_row[w];
          st.adv_src[o] = -1;
          st.adv_dst[o] = -1;
          st.adv_tok[o] = -1;
        } else {
          // the j-th label extension (in slot order) takes the j-th state row not used by the
          // beam that is being replaced
          const int j = __popc(lab & ((1u << s) - 1u));
          const int f = (int)__fns(free_mask, 0, j + 1);
          st.t[o] = s_t[w];
          st.u[o] = s_u[w] + 1;
          st.hash[o] = hash_mix(s_hash[w], (uint32_t)k);
          st.prev_hash[o] = s_hash[w];
          st.last_tok[o] = k;
          st.row[o] = row0 + f;
          st.adv_src[o] = s_row[w];
          st.adv_dst[o] = row0 + f;
          st.adv_tok[o] = k;
        }
        st.bp_parent[hist] = w;
        st.bp_token[hist] = k;
        st.bp_score[hist] = win_score[s];
      } else {
        st.row[o] = -1;
        st.adv_src[o] = -1;
        st.adv_dst[o] = -1;
        st.adv_tok[o] = -1;
        st.bp_parent[hist] = -1;
        st.bp_token[hist] = -1;
        st.bp_score[hist] = 0.0f;
      }
    }
  }
}

cudaError_t launch_beam_select(const BeamSelArgs& a, cudaStream_t s) {
  const size_t smem = (size_t)a.W * a.V * sizeof(float);
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(k_beam_select, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  timing_begin(s);
  k_beam_select<<<a.B, SEL_NT, smem, s>>>(a);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}

// Compaction of the pending network advances: slots whose adv_dst >= 0 are listed first, in
// slot order, so that the advance kernels touch only tiles with work (most extensions of a
// beam are blanks, which advance nothing).  One CTA; deterministic order.
__global__ void __launch_bounds__(1024) k_compact(const int32_t* adv_src, const int32_t* adv_dst,
                                                  const int32_t* adv_tok, int N, int32_t* c_src,
                                                  int32_t* c_dst, int32_t* c_tok, int32_t* n_active) {
  __shared__ int wsum[32];
  __shared__ int base_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) base_s = 0;
  __syncthreads();
  for (int n0 = 0; n0 < N; n0 += 1024) {
    const int n = n0 + tid;
    const bool f = n < N && adv_dst[n] >= 0;
    const unsigned m = __ballot_sync(0xffffffffu, f);
    const int within = __popc(m & ((1u << lane) - 1u));
    if (lane == 0) wsum[warp] = __popc(m);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < 32; ++w) {
      const int c = wsum[w];
      if (w < warp) before += c;
      total += c;
    }
    const int base = base_s;
    if (f) {
      const int a = base + before + within;
      c_src[a] = adv_src[n];
      c_dst[a] = adv_dst[n];
      c_tok[a] = adv_tok[n];
    }
    __syncthreads();
    if (tid == 0) base_s = base + total;
    __syncthreads();
  }
  const int total = base_s;
  for (int a = total + tid; a < N; a += 1024) {
    c_src[a] = -1;
    c_dst[a] = -1;
    c_tok[a] = -1;
  }
  if (tid == 0) *n_active = total;
}

cudaError_t launch_compact(const q4_beam_state& st, int N, int32_t* c_src, int32_t* c_dst, int32_t* c_tok,
                           int32_t* n_active, cudaStream_t s) {
  timing_begin(s);
  k_compact<<<1, 1024, 0, s>>>(st.adv_src, st.adv_dst, st.adv_tok, N, c_src, c_dst, c_tok, n_active);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}

__global__ void k_beam_init(q4_beam_state st, int B, int W) {
  const int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o == 0) st.status[0] = 0;
  if (o >= B * W) return;
  const int b = o / W, s = o % W;
  const bool root = s == 0;
  st.score[o] = 0.0f;
  st.t[o] = 0;
  st.u[o] = 0;
  st.hash[o] = HASH0;
  st.prev_hash[o] = 0;
  st.last_tok[o] = 0;
  st.row[o] = root ? b * 2 * W : -1;
  st.adv_src[o] = -1;                      // zero state
  st.adv_dst[o] = root ? b * 2 * W : -1;
  st.adv_tok[o] = root ? 0 : -1;           // start symbol
  st.fin_score[o] = -INFINITY;
  st.fin_iter[o] = 0;
  st.fin_slot[o] = 0;
  if (s == 0) st.fin_n[b] = 0;
}

cudaError_t launch_beam_init(const q4_beam_state& st, int B, int W, int n_iters, cudaStream_t s) {
  (void)n_iters;
  k_beam_init<<<(B * W + 255) / 256, 256, 0, s>>>(st, B, W);
  ++g_launches;
  return cudaGetLastError();
}

__global__ void k_traceback(q4_beam_state st, int B, int W, int n_iters, int u_max,
                            int32_t* tokens, int32_t* lens, float* scores) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int j, s;
  float sc;
  if (st.fin_n[b] > 0) {
    sc = st.fin_score[b * W];
    j = st.fin_iter[b * W] - 1;
    s = st.fin_slot[b * W];
  } else if (n_iters > 0 && st.row[b * W] >= 0) {
    sc = st.score[b * W];
    j = n_iters - 1;
    s = 0;
  } else {
    sc = 0.0f;
    j = -1;
    s = -1;
  }
  int32_t* out = tokens + (size_t)b * u_max;
  int len = 0;
  while (j >= 0 && s >= 0) {
    const size_t h = ((size_t)j * B + b) * W + s;
    const int k = st.bp_token[h];
    if (k > 0 && len < u_max) out[len++] = k;
    s = st.bp_parent[h];
    --j;
  }
  for (int i = 0; i < len / 2; ++i) {
    const int32_t tmp = out[i];
    out[i] = out[len - 1 - i];
    out[len - 1 - i] = tmp;
  }
  for (int i = len; i < u_max; ++i) out[i] = 0;
  lens[b] = len;
  scores[b] = sc;
}

cudaError_t launch_traceback(const q4_beam_state& st, int B, int W, int n_iters, int u_max,
                             int32_t* tokens, int32_t* lens, float* scores, cudaStream_t s) {
  k_traceback<<<(B + 63) / 64, 64, 0, s>>>(st, B, W, n_iters, u_max, tokens, lens, scores);
  ++g_launches;
  return cudaGetLastError();
}

}  // namespace q4
