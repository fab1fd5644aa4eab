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

// Largest key of this lane's strided share of a shared array, and warp-wide arg-max helpers.
__device__ __forceinline__ uint64_t strided_max(const uint64_t* arr, int n, int lane) {
  uint64_t m = 0;
  for (int i = lane; i < n; i += 32) m = u64max(m, arr[i]);
  return m;
}

__global__ void __launch_bounds__(SEL_NT) k_beam_select(const __grid_constant__ BeamSelArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int W = a.W, V = a.V;
  float* cand = reinterpret_cast<float*>(smem_raw);                         // [W * V]
  uint64_t* list = reinterpret_cast<uint64_t*>(cand + (size_t)W * V);       // survivors of the filter
  __shared__ float s_score[MAXW];
  __shared__ int s_t[MAXW], s_u[MAXW], s_row[MAXW], s_last[MAXW];
  __shared__ uint64_t s_hash[MAXW], s_prev[MAXW];
  __shared__ int list_n;
  __shared__ int win_idx[MAXW];
  __shared__ float win_score[MAXW];
  __shared__ float s_gmax[SEL_NT / 32][16];   // per warp: best label proposal of lanes g and g + 16

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x;
  const int base = b * W;
  const q4_beam_state& st = a.st;
  const float NEG = -INFINITY;
  const int N = a.B * W;
  const bool fast = V <= 1024 && W <= SEL_NT / 32 && !a.exact_only;   // one warp per slot, row in registers

  pdl_wait();
  // the joint logits of slot `warp` do not depend on the beam state: request them first
  float v[32];
  if (fast && warp < W) {
    const float* x = a.logits + (size_t)(base + warp) * V;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int k = lane + 32 * i;
      v[i] = k < V ? x[k] : NEG;
    }
  }
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
  if (tid == 0) {
    list_n = 0;
    // the list of pending advances consumed by this iteration is free again
    if (b == 0) st.pend_n[a.iter & 1] = 0;
  }
  if (lane < 16) s_gmax[warp][lane] = NEG;
  __syncthreads();

  // ---- no slot of this utterance may emit a label (all at their label budget, or empty): the only
  // proposals are the blanks of the live slots, at most W of them, no two of which can describe the
  // same string.  One warp, lane = slot: the same score arithmetic, the same finished list and the
  // same order (score descending, then slot) as the general path below, without its passes over V.
  const int cap = 16 * ((V + 31) / 32);
  bool any_labels = false;
  for (int w = 0; w < W; ++w) any_labels |= s_row[w] >= 0 && s_u[w] < a.u_max;
  const bool blank_only = fast && a.normalized != 0 && !any_labels;
  if (blank_only) {
    if (warp == 0) {
      const int w = lane;
      const bool alive = w < W && s_row[w] >= 0;
      float sc = NEG;
      if (alive) sc = (float)((double)s_score[w] + (double)(a.logits[(size_t)(base + w) * V] - 0.0f));
      const bool fin = alive && s_t[w] + 1 == a.T;   // consumed the last frame: goes to the finished list
      if (__any_sync(0xffffffffu, fin)) {
        if (w < W) win_score[w] = sc;                // staging only; overwritten by the ranking below
        __syncwarp();
        if (lane == 0) {
          float* fs = st.fin_score + base;
          int* fi = st.fin_iter + base;
          int* fl = st.fin_slot + base;
          int n = st.fin_n[b];
          for (int x = 0; x < W; ++x) {
            if (s_row[x] < 0 || s_t[x] + 1 != a.T) continue;
            const float S = win_score[x];
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
            fl[pos] = x;
            n = min(n + 1, W);
          }
          st.fin_n[b] = n;
        }
        __syncwarp();
      }
      const bool cnd = alive && !fin && sc > NEG;
      const uint64_t key = cnd ? make_key(sc, (uint32_t)w * (uint32_t)V) : 0ull;
      int rank = 0;
      for (int x = 0; x < W; ++x) rank += __shfl_sync(0xffffffffu, key, x) > key;
      if (cnd) {
        win_idx[rank] = w * V;
        win_score[rank] = sc;
      }
      const int n_c = __popc(__ballot_sync(0xffffffffu, cnd));
      if (lane == 0) list_n = n_c;
    }
    __syncthreads();
  } else {
  // ---- proposals
  uint32_t skip = 0;   // fast path: bit i = element lane + 32 i is not a label proposal that can win
  if (fast) {
    if (warp < W) {
      const int w = warp;
      float* cw = cand + (size_t)w * V;
      const int row = s_row[w];
      const bool labels = row >= 0 && s_u[w] < a.u_max;
      if (row < 0) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int k = lane + 32 * i;
          if (k < V) cw[k] = NEG;
        }
        skip = 0xFFFFFFFFu;
      } else {
        // one round trip to memory for both LM rows
        float ltv[32], lsv[32];
        const float* lt = a.tgt_lp + (size_t)row * V;
        const float* ls = a.src_lp + (size_t)row * V;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int k = lane + 32 * i;
          ltv[i] = (k < V && labels) ? lt[k] : 0.0f;
          lsv[i] = (k < V && labels) ? ls[k] : 0.0f;
        }
        const double S = (double)s_score[w];
        const double S_rho = S + (double)a.rho;
        float lse = 0.0f;       // the joint kernel may already have normalised its rows
        if (!a.normalized) {
          float m = NEG;
#pragma unroll
          for (int i = 0; i < 32; ++i) m = fmaxf(m, v[i]);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          float sum = 0.0f;
#pragma unroll
          for (int i = 0; i < 32; ++i) sum += expf(v[i] - m);   // exp(-inf) = 0 for the padding
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          lse = m + logf(sum);
        }
        // label proposals of this slot that the merge below folds into another slot's blank: lane w1
        // tests slot w1 (all W tests at once), the few hits are then handed round the warp
        {
          const bool hit = lane < W && labels && s_row[lane] >= 0 && s_u[lane] == s_u[w] + 1 && s_prev[lane] == s_hash[w];
          const int tok = hit ? s_last[lane] : 0;
          unsigned hits = __ballot_sync(0xffffffffu, hit);
          while (hits) {
            const int src = __ffs(hits) - 1;
            hits &= hits - 1;
            const int t = __shfl_sync(0xffffffffu, tok, src);
            if ((t & 31) == lane) skip |= 1u << (t >> 5);
          }
        }
        float best = NEG;
        const float blank = (float)(S + (double)(v[0] - lse));   // element 0 of lane 0 is the blank proposal
        if (labels) {   // uniform per warp: a slot at its label budget skips the double-precision adds
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int k = lane + 32 * i;
            const float lp = v[i] - lse;
            float sc;
            if (k >= V) {
              sc = NEG;
              skip |= 1u << i;
            } else if (k == 0) {
              sc = blank;
              skip |= 1u << i;          // the blank proposal is read back after merge and finished list
            } else {
              // label increment in fp32 (magnitude of tens), one double add onto the running score
              const float inc = __fmaf_rn(a.lambda_t, ltv[i], __fmaf_rn(-a.lambda_s, lsv[i], lp));
              sc = (float)(S_rho + (double)inc);
            }
            v[i] = sc;
            if (k < V) cw[k] = sc;
            if (!((skip >> i) & 1u)) best = fmaxf(best, sc);
          }
        } else {
          skip = 0xFFFFFFFFu;       // no label proposals: only the blank, read back from shared memory
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int k = lane + 32 * i;
            const float sc = k == 0 ? blank : NEG;
            v[i] = sc;
            if (k < V) cw[k] = sc;
          }
        }
        best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, 16));
        if (lane < 16) s_gmax[w][lane] = best;
      }
    } else {
      skip = 0xFFFFFFFFu;
    }
  } else {
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
      const double S_rho = S + (double)a.rho;
      const bool labels = s_u[w] < a.u_max;
      // general vocabulary size: three passes over the row
      float lse = 0.0f;
      if (!a.normalized) {
        float m = NEG;
        for (int k = lane; k < V; k += 32) m = fmaxf(m, x[k]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float sum = 0.0f;
        for (int k = lane; k < V; k += 32) sum += expf(x[k] - m);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        lse = m + logf(sum);
      }
      for (int k = lane; k < V; k += 32) {
        const float lp = x[k] - lse;
        float sc;
        if (k == 0) {
          sc = (float)(S + (double)lp);
        } else if (labels) {
          // label increment in fp32 (magnitude of tens), one double add onto the running score
          const float inc = __fmaf_rn(a.lambda_t, lt[k], __fmaf_rn(-a.lambda_s, ls[k], lp));
          sc = (float)(S_rho + (double)inc);
        } else {
          sc = NEG;
        }
        cw[k] = sc;
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
  // fast path: a lower bound of the W-th best proposal.  The label proposals are split into 16
  // disjoint groups (by lane modulo 16); each group's best is a distinct proposal, so at least
  // 16 >= W proposals reach the smallest of the 16 group maxima.  An empty group (no slot may
  // emit labels) gives -inf: then only the at most W blank proposals exist and all pass.
  float bound = NEG;
  if (fast) {
    float g = NEG;
    if (lane < 16)
      for (int w = 0; w < W; ++w) g = fmaxf(g, s_gmax[w][lane]);
    g = __shfl_sync(0xffffffffu, g, lane & 15);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) g = fminf(g, __shfl_xor_sync(0xffffffffu, g, o));
    bound = g;
  }
  __syncthreads();

  // ---- finished hypotheses: blank proposals that consume the last frame
  if (tid == 0) {
    bool any = false;
    for (int w = 0; w < W; ++w) any |= s_row[w] >= 0 && s_t[w] + 1 == a.T;
    if (any) {
      float* fs = st.fin_score + base;
      int* fi = st.fin_iter + base;
      int* fl = st.fin_slot + base;
      int n = st.fin_n[b];
      for (int w = 0; w < W; ++w) {
        if (s_row[w] < 0 || s_t[w] + 1 != a.T) continue;
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
      st.fin_n[b] = n;
    }
  }
  __syncthreads();

  // ---- the W best remaining proposals
  bool exact = !fast;
  if (fast) {
    // everything at or above the bound goes to the short list (label proposals from registers,
    // the blank proposal from shared memory, where merge and finished list have updated it)
    if (warp < W && s_row[warp] >= 0) {   // uniform per warp: one list reservation per warp
      const uint32_t off = (uint32_t)warp * (uint32_t)V;
      uint32_t hit = 0;
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (!((skip >> i) & 1u) && v[i] >= bound) hit |= 1u << i;
      float vb = NEG;
      if (lane == 0) {
        vb = cand[(size_t)warp * V];
        if (!(vb >= bound)) vb = NEG;
      }
      const int mine = __popc(hit) + (vb > NEG ? 1 : 0);
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const int total = __shfl_sync(0xffffffffu, incl, 31);
      int p0 = 0;
      if (lane == 31 && total > 0) p0 = atomicAdd(&list_n, total);
      p0 = __shfl_sync(0xffffffffu, p0, 31) + incl - mine;
      if (vb > NEG) {
        if (p0 < cap) list[p0] = make_key(vb, off);
        ++p0;
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) {   // static register indices
        if ((hit >> i) & 1u) {
          if (p0 < cap) list[p0] = make_key(v[i], off + (uint32_t)(lane + 32 * i));
          ++p0;
        }
      }
    }
    __syncthreads();
    exact = list_n > cap;     // the bound was too loose for the list: take the exact threshold instead
    __syncthreads();
    if (exact && tid == 0) list_n = 0;
    if (exact) __syncthreads();
  }
  if (exact) {
    // Threshold filter.  (1) every thread's best proposal ("head") among its strided share of
    // its slot; (2) the W-th best head, found bit by bit with block-wide counts, is a lower bound
    // of the W-th best proposal, and only the threads owning the W best heads can hold anything
    // at or above it; (3) those go to the short list.
    uint64_t head = 0;
    for (int w = warp; w < W; w += SEL_NT / 32) {
      if (s_row[w] < 0) continue;
      const float* cw = cand + (size_t)w * V;
      const uint32_t off = (uint32_t)w * (uint32_t)V;
      for (int k = lane; k < V; k += 32) {
        const float x = cw[k];
        if (x > NEG) head = u64max(head, make_key(x, off + (uint32_t)k));
      }
    }
    // score bits first (32 counts); the index bits matter only if equal scores straddle the bound
    uint64_t th = 0;
    for (int bit = 63; bit >= 32; --bit) {
      const uint64_t c = th | (1ull << bit);
      if (__syncthreads_count(head >= c) >= W) th = c;
    }
    if (__syncthreads_count(head >= th) > W) {
      for (int bit = 31; bit >= 0; --bit) {
        const uint64_t c = th | (1ull << bit);
        if (__syncthreads_count(head >= c) >= W) th = c;
      }
    }
    // th = the W-th best head (0 if there are fewer than W heads: then everything valid passes)
    if (head != 0ull && head >= th) {
      for (int w = warp; w < W; w += SEL_NT / 32) {
        if (s_row[w] < 0) continue;
        const float* cw = cand + (size_t)w * V;
        const uint32_t off = (uint32_t)w * (uint32_t)V;
        for (int k = lane; k < V; k += 32) {
          const float x = cw[k];
          if (!(x > NEG)) continue;
          const uint64_t key = make_key(x, off + (uint32_t)k);
          if (key >= th) {
            const int p = atomicAdd(&list_n, 1);
            if (p < cap) list[p] = key;
          }
        }
      }
    }
    __syncthreads();
  }
  }
  // each list entry's rank is counted in parallel
  if (!blank_only) {
    const int ln = min(list_n, cap);
    for (int i = tid; i < ln; i += SEL_NT) {
      const uint64_t mine = list[i];
      int rank = 0;
      for (int j = 0; j < ln; ++j) rank += list[j] > mine;
      if (rank < W) {
        win_idx[rank] = (int)(~(uint32_t)mine);
        win_score[rank] = key_score(mine);
      }
    }
  }
  __syncthreads();
  pdl_trigger();   // only the bookkeeping is left: the next kernel of the stream may set itself up

  if (warp == 0) {
    const int n_win = min(min(list_n, cap), W);

    // ---- next beam, state rows, back-pointers, pending advances: lane s writes slot s
    const int nw = n_win;
    const int row0 = b * (st.rows_per_utt > 0 ? st.rows_per_utt : 2 * W);
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
    // reserve a range of the next iteration's pending list for this utterance's label extensions
    int pbase = 0;
    if (lane == 0 && lab != 0u) pbase = atomicAdd(st.pend_n + ((a.iter + 1) & 1), __popc(lab));
    pbase = __shfl_sync(0xffffffffu, pbase, 0);
    const size_t poff = (size_t)((a.iter + 1) & 1) * N;
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
          st.pend_src[poff + pbase + j] = s_row[w];
          st.pend_dst[poff + pbase + j] = row0 + f;
          st.pend_tok[poff + pbase + j] = k;
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

cudaError_t launch_beam_select(const BeamSelArgs& a, cudaStream_t s, bool dependent) {
  const size_t smem = (size_t)a.W * a.V * sizeof(float) + (size_t)16 * ((a.V + 31) / 32) * sizeof(uint64_t);
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(k_beam_select, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  timing_begin(s);
  cudaError_t le = launch_ex(k_beam_select, dim3(a.B), dim3(SEL_NT), smem, s, dependent, 1, a);
  timing_end(s);
  ++g_launches;
  return le != cudaSuccess ? le : cudaGetLastError();
}

// ------------------------------------------------------------------ time-synchronous search
// One call of the time-synchronous search for one utterance per CTA (the networks and the joint
// have already run for the hypotheses of the current set A, all at frame t).  Every live slot's
// blank proposal joins the candidate set of the next frame (global arrays nb_*, at most
// W (S+1) entries, equal label strings merged by log-addition in insertion order).  In an inner
// call (mode 1) the W best label proposals (score, parent slot, token) become the next set A at
// the same frame: fresh state rows, pending network advances, back-pointers, exactly like label
// extensions of the alignment-length synchronous search.  In the frame-closing call (mode 2) no
// label is proposed and the W best candidates (score, insertion order) open frame t + 1.
constexpr int TSD_MAXC = 64;
__global__ void __launch_bounds__(SEL_NT) k_tsd_select(const __grid_constant__ BeamSelArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int W = a.W, V = a.V;
  float* cand = reinterpret_cast<float*>(smem_raw);                         // [W * V] label proposals
  uint64_t* list = reinterpret_cast<uint64_t*>(cand + (size_t)W * V);
  __shared__ float s_score[MAXW], s_blank[MAXW];
  __shared__ int s_u[MAXW], s_row[MAXW], s_last[MAXW];
  __shared__ uint64_t s_hash[MAXW], s_prev[MAXW];
  __shared__ int list_n;
  __shared__ int win_idx[MAXW];
  __shared__ float win_score[MAXW];
  __shared__ float c_score[TSD_MAXC];
  __shared__ int c_u[TSD_MAXC], c_last[TSD_MAXC], c_row[TSD_MAXC], c_org[TSD_MAXC], c_n;
  __shared__ uint64_t c_hash[TSD_MAXC], c_prev[TSD_MAXC];
  __shared__ float s_gmax[SEL_NT / 32][16];   // per warp: best label proposal of lanes g and g + 16

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x;
  const int base = b * W;
  const q4_beam_state& st = a.st;
  const float NEG = -INFINITY;
  const int N = a.B * W;
  const int S = st.tsd_smax;
  const int CB = W * (S + 1);
  const int step = a.iter % (S + 1), frame = a.iter / (S + 1);
  const bool inner = a.mode == 1;
  const int RW = st.rows_per_utt;
  // inner calls with a vocabulary of at most 1024: one warp per slot keeps its proposals in registers
  // and the W best are found from a lower bound, as in k_beam_select
  const bool fast = inner && V <= 1024 && W <= SEL_NT / 32 && !a.exact_only;

  pdl_wait();
  if (tid < W) {
    const int o = base + tid;
    s_row[tid] = st.row[o];
    s_score[tid] = st.score[o];
    s_u[tid] = st.u[o];
    s_last[tid] = st.last_tok[o];
    s_hash[tid] = st.hash[o];
    s_prev[tid] = st.prev_hash[o];
  }
  const int cn0 = st.nb_n[b];
  for (int j = tid; j < cn0; j += SEL_NT) {
    const size_t o = (size_t)b * CB + j;
    c_score[j] = st.nb_score[o];
    c_u[j] = st.nb_u[o];
    c_last[j] = st.nb_last_tok[o];
    c_row[j] = st.nb_row[o];
    c_org[j] = st.nb_origin[o];
    c_hash[j] = st.nb_hash[o];
    c_prev[j] = st.nb_prev_hash[o];
  }
  if (tid == 0) {
    list_n = 0;
    c_n = cn0;
    if (b == 0) st.pend_n[a.iter & 1] = 0;   // the list consumed by this call is free again
  }
  if (lane < 16) s_gmax[warp][lane] = NEG;
  __syncthreads();

  // ---- proposals
  float v[32];
  uint32_t skip = 0xFFFFFFFFu;   // fast path: bit i = element lane + 32 i is not a label proposal
  if (!inner && a.normalized) {
    // a frame close proposes blanks only, and the joint kernel has normalised its rows
    if (tid < W)
      s_blank[tid] = s_row[tid] >= 0
                         ? (float)((double)s_score[tid] + (double)a.logits[(size_t)(base + tid) * V])
                         : NEG;
  } else if (fast) {
    if (warp < W) {
      const int w = warp;
      float* cw = cand + (size_t)w * V;
      const int row = s_row[w];
      if (row < 0) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int k = lane + 32 * i;
          if (k < V) cw[k] = NEG;
        }
        if (lane == 0) s_blank[w] = NEG;
      } else {
        const bool labels = s_u[w] < a.u_max;
        const float* x = a.logits + (size_t)(base + w) * V;
        const float* lt = a.tgt_lp + (size_t)row * V;
        const float* ls = a.src_lp + (size_t)row * V;
        float ltv[32], lsv[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int k = lane + 32 * i;
          v[i] = k < V ? x[k] : NEG;
          ltv[i] = (k < V && labels) ? lt[k] : 0.0f;
          lsv[i] = (k < V && labels) ? ls[k] : 0.0f;
        }
        const double S_rho = (double)s_score[w] + (double)a.rho;
        float lse = 0.0f;
        if (!a.normalized) {
          float m = NEG;
#pragma unroll
          for (int i = 0; i < 32; ++i) m = fmaxf(m, v[i]);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          float sum = 0.0f;
#pragma unroll
          for (int i = 0; i < 32; ++i) sum += expf(v[i] - m);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          lse = m + logf(sum);
        }
        skip = 0;
        float best = NEG;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int k = lane + 32 * i;
          const float lp = v[i] - lse;
          float sc = NEG;
          if (k >= V) {
            skip |= 1u << i;
          } else if (k == 0) {
            s_blank[w] = (float)((double)s_score[w] + (double)lp);
            skip |= 1u << i;
          } else if (labels) {
            const float inc = __fmaf_rn(a.lambda_t, ltv[i], __fmaf_rn(-a.lambda_s, lsv[i], lp));
            sc = (float)(S_rho + (double)inc);
            best = fmaxf(best, sc);
          } else {
            skip |= 1u << i;
          }
          v[i] = sc;
          if (k < V) cw[k] = sc;
        }
        best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, 16));
        if (lane < 16) s_gmax[w][lane] = best;
      }
    }
  } else
  for (int w = warp; w < W; w += SEL_NT / 32) {
    float* cw = cand + (size_t)w * V;
    const int row = s_row[w];
    if (row < 0) {
      for (int k = lane; k < V; k += 32) cw[k] = NEG;
      if (lane == 0) s_blank[w] = NEG;
      continue;
    }
    const float* x = a.logits + (size_t)(base + w) * V;
    const float* lt = a.tgt_lp + (size_t)row * V;
    const float* ls = a.src_lp + (size_t)row * V;
    const double S_rho = (double)s_score[w] + (double)a.rho;
    const bool labels = inner && s_u[w] < a.u_max;
    float lse = 0.0f;
    if (!a.normalized) {
      float m = NEG;
      for (int k = lane; k < V; k += 32) m = fmaxf(m, x[k]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      float sum = 0.0f;
      for (int k = lane; k < V; k += 32) sum += expf(x[k] - m);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      lse = m + logf(sum);
    }
    for (int k = lane; k < V; k += 32) {
      const float lp = x[k] - lse;
      float sc = NEG;
      if (k == 0) {
        s_blank[w] = (float)((double)s_score[w] + (double)lp);
      } else if (labels) {
        const float inc = __fmaf_rn(a.lambda_t, lt[k], __fmaf_rn(-a.lambda_s, ls[k], lp));
        sc = (float)(S_rho + (double)inc);
      }
      cw[k] = sc;
    }
  }
  __syncthreads();

  // ---- blanks join the candidate set, in slot order (warp 0; lanes search, lane 0 updates)
  if (warp == 0) {
    for (int w = 0; w < W; ++w) {
      if (s_row[w] < 0) continue;             // uniform
      const int n = c_n;
      const uint64_t h = s_hash[w];
      int found = -1;
      for (int j0 = 0; j0 < n; j0 += 32) {
        const int j = j0 + lane;
        const unsigned m = __ballot_sync(0xffffffffu, j < n && c_hash[j] == h);
        if (m) {
          found = j0 + __ffs(m) - 1;
          break;
        }
      }
      if (lane == 0) {
        if (found >= 0) {
          const double x = (double)c_score[found], y = (double)s_blank[w];
          c_score[found] = (float)(fmax(x, y) + log1p(exp(-fabs(x - y))));
        } else if (n < TSD_MAXC && n < CB) {
          c_score[n] = s_blank[w];
          c_u[n] = s_u[w];
          c_last[n] = s_last[w];
          c_row[n] = s_row[w];
          c_org[n] = (step << 8) | w;
          c_hash[n] = h;
          c_prev[n] = s_prev[w];
          c_n = n + 1;
        }
      }
      __syncwarp();
    }
  }
  // lower bound of the W-th best label proposal: the smallest of the 16 group maxima (k_beam_select)
  float bound = NEG;
  if (fast) {
    float g = NEG;
    if (lane < 16)
      for (int w = 0; w < W; ++w) g = fmaxf(g, s_gmax[w][lane]);
    g = __shfl_sync(0xffffffffu, g, lane & 15);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) g = fminf(g, __shfl_xor_sync(0xffffffffu, g, o));
    bound = g;
  }
  __syncthreads();

  if (inner) {
    const int cap = 16 * ((V + 31) / 32);
    bool exact = !fast;
    if (fast) {
      if (warp < W && s_row[warp] >= 0) {   // uniform per warp: one list reservation per warp
        const uint32_t off = (uint32_t)warp * (uint32_t)V;
        uint32_t hit = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (!((skip >> i) & 1u) && v[i] >= bound) hit |= 1u << i;
        const int mine = __popc(hit);
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        int p0 = 0;
        if (lane == 31 && total > 0) p0 = atomicAdd(&list_n, total);
        p0 = __shfl_sync(0xffffffffu, p0, 31) + incl - mine;
#pragma unroll
        for (int i = 0; i < 32; ++i) {   // static register indices
          if ((hit >> i) & 1u) {
            if (p0 < cap) list[p0] = make_key(v[i], off + (uint32_t)(lane + 32 * i));
            ++p0;
          }
        }
      }
      __syncthreads();
      exact = list_n > cap;     // the bound was too loose for the list: take the exact threshold instead
      __syncthreads();
      if (exact && tid == 0) list_n = 0;
      if (exact) __syncthreads();
    }
    // ---- otherwise the exact threshold search (see k_beam_select)
    uint64_t head = 0;
    if (exact) {
    for (int w = warp; w < W; w += SEL_NT / 32) {
      if (s_row[w] < 0) continue;
      const float* cw = cand + (size_t)w * V;
      const uint32_t off = (uint32_t)w * (uint32_t)V;
      for (int k = lane; k < V; k += 32) {
        const float x = cw[k];
        if (x > NEG) head = u64max(head, make_key(x, off + (uint32_t)k));
      }
    }
    uint64_t th = 0;
    for (int bit = 63; bit >= 32; --bit) {
      const uint64_t c = th | (1ull << bit);
      if (__syncthreads_count(head >= c) >= W) th = c;
    }
    if (__syncthreads_count(head >= th) > W) {
      for (int bit = 31; bit >= 0; --bit) {
        const uint64_t c = th | (1ull << bit);
        if (__syncthreads_count(head >= c) >= W) th = c;
      }
    }
    if (head != 0ull && head >= th) {
      for (int w = warp; w < W; w += SEL_NT / 32) {
        if (s_row[w] < 0) continue;
        const float* cw = cand + (size_t)w * V;
        const uint32_t off = (uint32_t)w * (uint32_t)V;
        for (int k = lane; k < V; k += 32) {
          const float x = cw[k];
          if (!(x > NEG)) continue;
          const uint64_t key = make_key(x, off + (uint32_t)k);
          if (key >= th) {
            const int p = atomicAdd(&list_n, 1);
            if (p < cap) list[p] = key;
          }
        }
      }
    }
    __syncthreads();
    }   // exact
    {
      const int ln = min(list_n, cap);
      for (int i = tid; i < ln; i += SEL_NT) {
        const uint64_t mine = list[i];
        int rank = 0;
        for (int j = 0; j < ln; ++j) rank += list[j] > mine;
        if (rank < W) {
          win_idx[rank] = (int)(~(uint32_t)mine);
          win_score[rank] = key_score(mine);
        }
      }
    }
    __syncthreads();
    pdl_trigger();
    if (warp == 0) {
      const int nw = min(min(list_n, cap), W);
      const int row0 = b * RW;
      // rows in use: those of the current set and those the candidates refer to
      uint64_t used = 0;
      for (int w = 0; w < W; ++w)
        if (s_row[w] >= 0) used |= 1ull << (s_row[w] - row0);
      for (int j = 0; j < c_n; ++j) used |= 1ull << (c_row[j] - row0);
      const uint64_t all = RW >= 64 ? ~0ull : ((1ull << RW) - 1ull);
      uint64_t free_mask = ~used & all;
      const int s = lane;
      // the j-th winner takes the j-th free row
      int f = -1;
      {
        uint64_t m = free_mask;
        for (int j = 0; j <= s && j < nw; ++j) {
          f = m ? __ffsll((long long)m) - 1 : -1;
          m &= m - 1;
        }
      }
      int pbase = 0;
      if (lane == 0 && nw > 0) pbase = atomicAdd(st.pend_n + ((a.iter + 1) & 1), nw);
      pbase = __shfl_sync(0xffffffffu, pbase, 0);
      const size_t poff = (size_t)((a.iter + 1) & 1) * N;
      if (s < W) {
        const int o = base + s;
        const size_t hist = ((size_t)a.iter * a.B + b) * W + s;
        if (s < nw && f >= 0) {
          const int idx = win_idx[s];
          const int w = idx / V, k = idx % V;
          st.score[o] = win_score[s];
          st.t[o] = frame;
          st.u[o] = s_u[w] + 1;
          st.hash[o] = hash_mix(s_hash[w], (uint32_t)k);
          st.prev_hash[o] = s_hash[w];
          st.last_tok[o] = k;
          st.row[o] = row0 + f;
          st.adv_src[o] = s_row[w];
          st.adv_dst[o] = row0 + f;
          st.adv_tok[o] = k;
          st.pend_src[poff + pbase + s] = s_row[w];
          st.pend_dst[poff + pbase + s] = row0 + f;
          st.pend_tok[poff + pbase + s] = k;
          st.bp_parent[hist] = w;
          st.bp_token[hist] = k;
          st.bp_score[hist] = win_score[s];
        } else {
          st.row[o] = -1;
          st.adv_src[o] = -1;
          st.adv_dst[o] = -1;
          st.adv_tok[o] = -1;
          st.bp_parent[hist] = -1;
          st.bp_token[hist] = 0;
          st.bp_score[hist] = 0.0f;
        }
      }
    }
    // the candidate set goes back to memory
    for (int j = tid; j < c_n; j += SEL_NT) {
      const size_t o = (size_t)b * CB + j;
      st.nb_score[o] = c_score[j];
      st.nb_u[o] = c_u[j];
      st.nb_last_tok[o] = c_last[j];
      st.nb_row[o] = c_row[j];
      st.nb_origin[o] = c_org[j];
      st.nb_hash[o] = c_hash[j];
      st.nb_prev_hash[o] = c_prev[j];
    }
    if (tid == 0) st.nb_n[b] = c_n;
  } else {
    // ---- frame close: the W best candidates (score descending, then insertion order)
    pdl_trigger();
    const int n = c_n;
    const int nw = min(n, W);
    if (tid < n) {
      const float mine = c_score[tid];
      int rank = 0;
      for (int j = 0; j < n; ++j) rank += (c_score[j] > mine) || (c_score[j] == mine && j < tid);
      if (rank < W) {
        const int o = base + rank;
        const size_t hist = ((size_t)a.iter * a.B + b) * W + rank;
        st.score[o] = mine;
        st.t[o] = frame + 1;
        st.u[o] = c_u[tid];
        st.hash[o] = c_hash[tid];
        st.prev_hash[o] = c_prev[tid];
        st.last_tok[o] = c_last[tid];
        st.row[o] = c_row[tid];
        st.adv_src[o] = -1;
        st.adv_dst[o] = -1;
        st.adv_tok[o] = -1;
        st.bp_parent[hist] = c_org[tid] & 0xFF;
        st.bp_token[hist] = -1 - (c_org[tid] >> 8);
        st.bp_score[hist] = mine;
        if (frame + 1 == a.T) {
          st.fin_score[base + rank] = mine;
          st.fin_iter[base + rank] = a.iter + 1;
          st.fin_slot[base + rank] = rank;
        }
      }
    }
    if (tid >= nw && tid < W) {
      const int o = base + tid;
      const size_t hist = ((size_t)a.iter * a.B + b) * W + tid;
      st.row[o] = -1;
      st.adv_src[o] = -1;
      st.adv_dst[o] = -1;
      st.adv_tok[o] = -1;
      st.bp_parent[hist] = -1;
      st.bp_token[hist] = 0;
      st.bp_score[hist] = 0.0f;
    }
    if (tid == 0) {
      st.nb_n[b] = 0;
      if (frame + 1 == a.T) st.fin_n[b] = nw;
    }
  }
}

cudaError_t launch_tsd_select(const BeamSelArgs& a, cudaStream_t s, bool dependent) {
  const size_t smem = (size_t)a.W * a.V * sizeof(float) + (size_t)16 * ((a.V + 31) / 32) * sizeof(uint64_t);
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(k_tsd_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  timing_begin(s);
  cudaError_t le = launch_ex(k_tsd_select, dim3(a.B), dim3(SEL_NT), smem, s, dependent, 1, a);
  timing_end(s);
  ++g_launches;
  return le != cudaSuccess ? le : cudaGetLastError();
}

// Trace-back of the time-synchronous search: a frame-closing call points at the call of the same
// frame whose blank created the entry; an inner call points at its parent slot of the call before.
__global__ void k_traceback_tsd(q4_beam_state st, int B, int W, int n_iters, int u_max, int32_t* tokens,
                                int32_t* lens, float* scores) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int S1 = st.tsd_smax + 1;
  int j = -1, s = -1;
  float sc = 0.0f;
  if (st.fin_n[b] > 0) {
    sc = st.fin_score[b * W];
    j = st.fin_iter[b * W] - 1;
    s = st.fin_slot[b * W];
  } else if (n_iters > 0 && st.row[b * W] >= 0) {
    sc = st.score[b * W];
    j = n_iters - 1;
    s = 0;
  }
  int32_t* out = tokens + (size_t)b * u_max;
  int len = 0;
  while (j >= 0 && s >= 0) {
    const size_t h = ((size_t)j * B + b) * W + s;
    const int k = st.bp_token[h];
    const int par = st.bp_parent[h];
    if (j % S1 == S1 - 1) {         // frame close: jump to the set the blank was proposed from
      j = j - (S1 - 1) + (-1 - k) - 1;
    } else {
      if (k > 0 && len < u_max) out[len++] = k;
      --j;
    }
    s = par;
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
  const int RW = st.rows_per_utt > 0 ? st.rows_per_utt : 2 * W;
  st.row[o] = root ? b * RW : -1;
  st.adv_src[o] = -1;                      // zero state
  st.adv_dst[o] = root ? b * RW : -1;
  st.adv_tok[o] = root ? 0 : -1;           // start symbol
  st.fin_score[o] = -INFINITY;
  st.fin_iter[o] = 0;
  st.fin_slot[o] = 0;
  if (s == 0) {
    st.fin_n[b] = 0;
    st.pend_src[b] = -1;               // pending list of iteration 0: every utterance's root,
    st.pend_dst[b] = b * RW;           // fed the start symbol from the zero state
    if (st.nb_n) st.nb_n[b] = 0;
    st.pend_tok[b] = 0;
  }
  if (o == 0) {
    st.pend_n[0] = B;
    st.pend_n[1] = 0;
  }
}

cudaError_t launch_beam_init(const q4_beam_state& st, int B, int W, int n_iters, cudaStream_t s) {
  (void)n_iters;
  k_beam_init<<<(B * W + 255) / 256, 256, 0, s>>>(st, B, W);
  ++g_launches;
  return cudaGetLastError();
}

// One warp per utterance.  The walk from the winning slot back to the root is a chain of
// dependent look-ups; to keep it off the memory latency, the warp first copies the back-pointer
// rows of 32 consecutive iterations into shared memory (one iteration per lane, all W slots),
// then lane 0 follows the chain there.
constexpr int TB_WARPS = 4;
__global__ void __launch_bounds__(32 * TB_WARPS) k_traceback(q4_beam_state st, int B, int W, int n_iters, int u_max,
                                                             int32_t* tokens, int32_t* lens, float* scores) {
  __shared__ int s_par[TB_WARPS][32][MAXW], s_tok[TB_WARPS][32][MAXW];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x * TB_WARPS + warp;
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
  while (j >= 0 && s >= 0) {   // uniform across the warp
    const int jl = j - lane;
    if (jl >= 0) {
      const size_t h = ((size_t)jl * B + b) * W;
      for (int i = 0; i < W; ++i) {
        s_par[warp][lane][i] = st.bp_parent[h + i];
        s_tok[warp][lane][i] = st.bp_token[h + i];
      }
    }
    __syncwarp();
    if (lane == 0) {
      for (int l = 0; l < 32 && j >= 0 && s >= 0; ++l, --j) {
        const int k = s_tok[warp][l][s];
        if (k > 0 && len < u_max) out[len++] = k;
        s = s_par[warp][l][s];
      }
    }
    j = __shfl_sync(0xffffffffu, j, 0);
    s = __shfl_sync(0xffffffffu, s, 0);
    __syncwarp();
  }
  if (lane == 0) {
    for (int i = 0; i < len / 2; ++i) {
      const int32_t tmp = out[i];
      out[i] = out[len - 1 - i];
      out[len - 1 - i] = tmp;
    }
    for (int i = len; i < u_max; ++i) out[i] = 0;
    lens[b] = len;
    scores[b] = sc;
  }
}

cudaError_t launch_traceback(const q4_beam_state& st, int B, int W, int n_iters, int u_max,
                             int32_t* tokens, int32_t* lens, float* scores, cudaStream_t s) {
  if (st.nb_score)   // the state of a time-synchronous search
    k_traceback_tsd<<<(B + 63) / 64, 64, 0, s>>>(st, B, W, n_iters, u_max, tokens, lens, scores);
  else
    k_traceback<<<(B + TB_WARPS - 1) / TB_WARPS, 32 * TB_WARPS, 0, s>>>(st, B, W, n_iters, u_max, tokens, lens, scores);
  ++g_launches;
  return cudaGetLastError();
}

}  // namespace q4
