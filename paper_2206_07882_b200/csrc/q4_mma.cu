// Tensor-core path (sm_100a): TMA-fed tcgen05 kind::i8 GEMMs with int32 accumulators in
// tensor memory.  Activations are the M operand (128 rows per tile), weight rows the N
// operand, both K-major int8 in shared memory under the 128-byte swizzle.
//   k_mma_gemm : D[128 x 256] tiles, epilogues: store int32 / de-quantize+bias / re-quantize.
//   k_mma_lstm : D_ih, D_hh[128 x 128] tiles (32 cells x 4 gates, gate-interleaved weight
//                rows) with the whole LSTM cell update fused into the epilogue.
// Warp roles per CTA: epilogue warps (one TMEM lane quarter each), one TMA producer thread,
// one MMA issuer thread.  4-bit codes are unpacked to int8 once per call by k_unpack_rows /
// k_prepare_w before they meet the tensor cores.
#include <string.h>

#include "q4_internal.h"
#include "q4_mma.cuh"

namespace q4 {

constexpr int BM = 128;          // activation rows per tile
constexpr int BK = 128;          // K bytes per pipeline stage (one swizzle row)
constexpr int GEMM_BN = 256;     // weight rows per tile, plain GEMM
constexpr int GEMM_STAGES = 4;
constexpr int LSTM_BN = 128;     // weight rows per tile, LSTM (32 cells x 4 gates)
constexpr int LSTM_STAGES = 3;
constexpr int LSTM_EPI_WARPS = 8;

// ------------------------------------------------------------------ operand preparation
// Gather + unpack activation rows to int8: dst[n, col0 + k] = code(src[idx[n], k]) - zero_point.
__global__ void __launch_bounds__(256) k_unpack_rows(const uint8_t* src, long long src_stride,
                                                     const int32_t* idx, int bits, int is_signed,
                                                     int zp, int k_pad, int n_rows, int8_t* dst,
                                                     long long dst_stride, int col0, int n_rows_pad, int32_t* clear64) {
  pdl_trigger();   // a dependent successor may set itself up; it reads nothing before this grid has completed
  pdl_wait();      // launched as a programmatic dependent itself: the source rows may be the predecessor's output
  if (clear64 && blockIdx.x == 0 && threadIdx.x < 64) clear64[threadIdx.x] = 0;   // the call's status block
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = k_pad >> 5;  // 32 elements per thread
  if (i >= (long long)n_rows_pad * per_row) return;
  const int n = (int)(i / per_row), k = (int)(i % per_row) * 32;
  uint4 o0 = make_uint4(0, 0, 0, 0), o1 = o0;
  int r = -1;
  if (n < n_rows) r = idx ? idx[n] : n;
  if (r >= 0) {
    const uint8_t* p = src + (long long)r * src_stride;
    if (bits == 4) {
      const uint4 v = *reinterpret_cast<const uint4*>(p + (k >> 1));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        // natural element order: byte b of the output word holds element 4*word + b
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          int a = (w[j] >> (4 * e)) & 0xF, c = (w[j] >> (4 * (e + 4))) & 0xF;
          if (is_signed) {
            a = (a ^ 8) - 8;
            c = (c ^ 8) - 8;
          } else {
            a -= zp;
            c -= zp;
          }
          lo |= (uint32_t)(a & 0xFF) << (8 * e);
          hi |= (uint32_t)(c & 0xFF) << (8 * e);
        }
        o[2 * j] = lo;
        o[2 * j + 1] = hi;
      }
      o0 = make_uint4(o[0], o[1], o[2], o[3]);
      o1 = make_uint4(o[4], o[5], o[6], o[7]);
    } else {
      o0 = *reinterpret_cast<const uint4*>(p + k);
      o1 = *reinterpret_cast<const uint4*>(p + k + 16);
    }
  }
  uint4* d = reinterpret_cast<uint4*>(dst + (long long)n * dst_stride + col0 + k);
  d[0] = o0;
  d[1] = o1;
}

cudaError_t launch_unpack_rows(const void* src, long long src_stride, const int32_t* idx,
                               const q4_act& act, int k_pad, int n_rows, int8_t* dst,
                               long long dst_stride, int col0, int n_rows_pad, cudaStream_t s,
                               int32_t* clear_status, bool dependent) {
  const long long total = (long long)n_rows_pad * (k_pad >> 5);
  if (total <= 0) return clear_status ? cudaMemsetAsync(clear_status, 0, 256, s) : cudaSuccess;
  timing_begin(s);
  cudaError_t le = launch_ex(k_unpack_rows, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, s, dependent, 1,
                             static_cast<const uint8_t*>(src), src_stride, idx, (int)act.bits, (int)act.is_signed,
                             (int)act.zero_point, k_pad, n_rows, dst, dst_stride, col0, n_rows_pad, clear_status);
  timing_end(s);
  ++g_launches;
  return le != cudaSuccess ? le : cudaGetLastError();
}

// Several gather+unpack jobs in one launch (blockIdx.y selects the job).  The grid is sized for
// the SMs, not for the padded row count: each thread strides over the 32-element pieces of the
// rows that carry work (their number is known on the device only).
__global__ void __launch_bounds__(256) k_unpack_multi(const UnpackJobs jobs) {
  pdl_trigger();
  pdl_wait();
  const UnpackJob& j = jobs.job[blockIdx.y];
  const int per_row = j.k_pad >> 5;
  int rows = jobs.n_rows_pad;
  if (!jobs.zero_tail) {   // rows without work need not be cleared every time
    rows = jobs.n_rows;
    if (jobs.n_active) rows = min(rows, *jobs.n_active);
  }
  const int n_work = jobs.n_active ? min(jobs.n_rows, *jobs.n_active) : jobs.n_rows;
  const uint32_t zp4 = (uint32_t)j.zp * 0x01010101u;
  const long long total = (long long)rows * per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(i / per_row), k = (int)(i % per_row) * 32;
    uint4 o0 = make_uint4(0, 0, 0, 0), o1 = o0;
    int r = -1;
    if (n < n_work) r = j.idx ? j.idx[n] : n;
    if (r >= 0) {
      const uint8_t* p = j.src + (long long)r * j.src_stride;
      if (j.bits == 4) {
        // eight codes per word -> two words of four int8 in natural element order
        const uint4 v = *reinterpret_cast<const uint4*>(p + (k >> 1));
        unpack8_natural(v.x, j.is_signed != 0, zp4, o0.x, o0.y);
        unpack8_natural(v.y, j.is_signed != 0, zp4, o0.z, o0.w);
        unpack8_natural(v.z, j.is_signed != 0, zp4, o1.x, o1.y);
        unpack8_natural(v.w, j.is_signed != 0, zp4, o1.z, o1.w);
      } else {
        o0 = *reinterpret_cast<const uint4*>(p + k);
        o1 = *reinterpret_cast<const uint4*>(p + k + 16);
      }
    }
    uint4* d = reinterpret_cast<uint4*>(j.dst + (long long)n * j.dst_stride + k);
    d[0] = o0;
    d[1] = o1;
  }
}

cudaError_t launch_unpack_multi(const UnpackJobs& jobs, cudaStream_t s, bool dependent) {
  if (jobs.n_jobs <= 0) return cudaSuccess;
  int kmax = 0;
  for (int i = 0; i < jobs.n_jobs; ++i) kmax = jobs.job[i].k_pad > kmax ? jobs.job[i].k_pad : kmax;
  const long long total = (long long)jobs.n_rows_pad * (kmax >> 5);
  long long blocks = (total + 255) / 256;
  const long long cap = (6 * 148 + jobs.n_jobs - 1) / jobs.n_jobs;   // about six CTAs per SM in all: one or two
                                                                     // pieces per thread at 1024 rows
  if (blocks > cap) blocks = cap;
  dim3 grid((unsigned)blocks, jobs.n_jobs);
  timing_begin(s);
  cudaError_t e = launch_ex(k_unpack_multi, grid, dim3(256), 0, s, dependent, 1, jobs);
  timing_end(s);
  ++g_launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Weight preparation: unpack to int8; with `interleave` the 4H rows (gate-major i,f,g,o) are
// reordered to row 4*cell + gate so that one thread of the epilogue owns all gates of a cell.
__global__ void __launch_bounds__(256) k_prepare_w(const uint8_t* src, int bits, int rows, int k_pad,
                                                   int interleave, int8_t* dst, long long dst_stride,
                                                   int col0) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = k_pad >> 3;
  if (i >= (long long)rows * per_row) return;
  const int r = (int)(i / per_row), k = (int)(i % per_row) * 8;
  int ro = r;
  if (interleave) {
    const int H = rows >> 2;
    ro = 4 * (r % H) + r / H;
  }
  uint2 o;
  if (bits == 4) {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(src + (long long)r * (k_pad >> 1) + (k >> 1));
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int a = (((w >> (4 * e)) & 0xF) ^ 8) - 8, c = (((w >> (4 * (e + 4))) & 0xF) ^ 8) - 8;
      lo |= (uint32_t)(a & 0xFF) << (8 * e);
      hi |= (uint32_t)(c & 0xFF) << (8 * e);
    }
    o = make_uint2(lo, hi);
  } else if (bits == 2) {   // four codes per byte, element i in bits 2i, 2i+1 of the 16-bit group
    const uint32_t w = *reinterpret_cast<const uint16_t*>(src + (long long)r * (k_pad >> 2) + (k >> 2));
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int a = (int)(((w >> (2 * e)) & 3u) ^ 2u) - 2, c = (int)(((w >> (2 * (e + 4))) & 3u) ^ 2u) - 2;
      lo |= (uint32_t)(a & 0xFF) << (8 * e);
      hi |= (uint32_t)(c & 0xFF) << (8 * e);
    }
    o = make_uint2(lo, hi);
  } else {
    o = *reinterpret_cast<const uint2*>(src + (long long)r * k_pad + k);
  }
  *reinterpret_cast<uint2*>(dst + (long long)ro * dst_stride + col0 + k) = o;
}
__global__ void k_prepare_vec(const float* src, int rows, int interleave, float* dst, float mul) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  int ro = r;
  if (interleave) {
    const int H = rows >> 2;
    ro = 4 * (r % H) + r / H;
  }
  dst[ro] = src ? __fmul_rn(mul, src[r]) : 0.0f;   // mul = 1 leaves the value as it is
}

cudaError_t launch_prepare_w(const q4_mat& w, int interleave, int8_t* dst, long long dst_stride,
                             int col0, cudaStream_t s) {
  const long long total = (long long)w.rows * (w.k_pad >> 3);
  timing_begin(s);
  k_prepare_w<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(static_cast<const uint8_t*>(w.q), w.bits,
                                                              w.rows, w.k_pad, interleave, dst,
                                                              dst_stride, col0);
  timing_end(s);
  ++g_launches;
  return cudaGetLastError();
}
cudaError_t launch_prepare_vec(const float* src, int rows, int interleave, float* dst, cudaStream_t s, float mul) {
  k_prepare_vec<<<(rows + 255) / 256, 256, 0, s>>>(src, rows, interleave, dst, mul);
  ++g_launches;
  return cudaGetLastError();
}

// ------------------------------------------------------------------ tensor maps (host)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// int8 matrix [rows, k] with row pitch `pitch` bytes; box = 128 bytes of K x box_rows rows.
bool make_tmap_i8(CUtensorMap* m, const void* base, uint64_t k, uint64_t rows, uint64_t pitch,
                  uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (pitch & 15u)) return false;
  const cuuint64_t dims[2] = {k, rows};
  const cuuint64_t strides[1] = {pitch};
  const cuuint32_t box[2] = {BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__device__ __forceinline__ void flag_timeout(int32_t* status) {
  if (status) atomicExch(status, Q4_ERR_TIMEOUT);
}

// ------------------------------------------------------------------ plain GEMM
struct MmaGemmArgs {
  int M, J, K, epi;
  void* out;
  long long ldo;            // elements (int32 / float) or bytes (codes) between output rows
  const int32_t* out_idx;   // output row of activation row m (nullptr = m, negative = skip)
  const float* w_scale;
  const float* bias;
  float x_scale;
  q4_act out_act;
  int32_t* status;
  const int32_t* n_active;
  const float* mul_e;       // EPI_JOINTZ: the other factor, row mul_idx[m] of [*, J] fp32
  const int32_t* mul_idx;
  uint32_t wait_limit;      // polls before a wait gives up
  int32_t skip_producer;    // test hook: the producer issues no copy, so the consumer's wait runs out
};

// Test hook (q4_test_wait_expiry_set): the next launches of k_mma_gemm get this limit and flag.
static uint32_t g_wait_limit = 1u << 22;
static int g_skip_producer = 0;
void test_wait_expiry_set(int skip_producer, uint32_t wait_limit) {
  g_skip_producer = skip_producer;
  g_wait_limit = wait_limit ? wait_limit : (1u << 22);
}

__global__ void __launch_bounds__(192, 1)
k_mma_gemm(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b,
           const MmaGemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int A_BYTES = BM * BK, B_BYTES = GEMM_BN * BK, STAGE = A_BYTES + B_BYTES;
  __shared__ uint64_t full[GEMM_STAGES], empty[GEMM_STAGES], acc_full;
  __shared__ uint32_t tmem_base_s;
  __shared__ float s_sc[GEMM_BN], s_bi[GEMM_BN];   // de-quantization constants of this tile's columns
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * GEMM_BN;   // row tiles slowest: tiles with work are dispatched first
  const int nk = (a.K + BK - 1) / BK;

  if (tid == 0) {
    for (int s = 0; s < GEMM_STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(&acc_full, 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 5) tmem_alloc(&tmem_base_s, GEMM_BN);
  if (warp == 4 && lane == 0) {
    prefetch_tmap(&tma_a);
    prefetch_tmap(&tma_b);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  pdl_wait();   // everything above overlaps the tail of the previous kernel of the stream
  const bool has_work = !(a.n_active && m0 >= *a.n_active);   // uniform per CTA

  if (!has_work) {
    // whole tile without work
  } else if (warp == 4 && lane == 0) {
    bool ok = true;
    for (int i = 0; i < nk && ok && !a.skip_producer; ++i) {
      const int s = i % GEMM_STAGES;
      if (i >= GEMM_STAGES) ok = mbar_wait(&empty[s], ((i / GEMM_STAGES) - 1) & 1, a.wait_limit);
      if (!ok) break;
      mbar_expect_tx(&full[s], STAGE);
      tma_load_2d(smem + s * STAGE, &tma_a, i * BK, m0, &full[s]);
      tma_load_2d(smem + s * STAGE + A_BYTES, &tma_b, i * BK, n0, &full[s]);
    }
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp == 5 && lane == 0) {
    const uint32_t idesc = umma_idesc_i8(BM, GEMM_BN);
    bool ok = true;
    for (int i = 0; i < nk && ok; ++i) {
      const int s = i % GEMM_STAGES;
      ok = mbar_wait(&full[s], (i / GEMM_STAGES) & 1, a.wait_limit);
      if (!ok) break;
      tc_fence_after();
      const uint64_t da = umma_desc_sw128(smem_u32(smem + s * STAGE));
      const uint64_t db = umma_desc_sw128(smem_u32(smem + s * STAGE + A_BYTES));
#pragma unroll
      for (int kk = 0; kk < BK / 32; ++kk) umma_i8(tmem, da + 2 * kk, db + 2 * kk, idesc, (i | kk) != 0);
      umma_commit(&empty[s]);
    }
    if (!ok) {   // recorded before the epilogue is released, so that it stores nothing
      flag_timeout(a.status);
      __threadfence();
    }
    umma_commit(&acc_full);
    pdl_trigger();
  } else if (warp < 4) {
    if (a.epi != EPI_I32) {   // stage scale * row scale and bias while the MMAs run
      for (int c = tid; c < GEMM_BN; c += 128) {
        const int j = min(n0 + c, a.J - 1);
        s_sc[c] = __fmul_rn(a.x_scale, __ldg(a.w_scale + j));
        s_bi[c] = a.bias ? __ldg(a.bias + j) : 0.0f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    bool ok = mbar_wait(&acc_full, 0, a.wait_limit);
    if (ok && a.status && *reinterpret_cast<volatile int32_t*>(a.status) != 0) ok = false;   // a wait gave up somewhere
    tc_fence_after();
    pdl_trigger();   // the main loop is over: the next kernel may set itself up
    if (!ok && lane == 0) flag_timeout(a.status);
    const int mi = m0 + warp * 32 + lane;
    int m = -1;
    if (mi < a.M && !(a.n_active && mi >= *a.n_active)) m = a.out_idx ? a.out_idx[mi] : mi;
    const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
    for (int c0 = 0; c0 < GEMM_BN; c0 += 32) {
      int r[32];
      tmem_ld32(taddr + c0, r);
      tmem_ld_wait();
      const int j0 = n0 + c0;
      if (!ok || m < 0 || j0 >= a.J) continue;
      if (a.epi == EPI_I32) {
        int32_t* o = reinterpret_cast<int32_t*>(a.out) + (long long)m * a.ldo + j0;
        if (j0 + 32 <= a.J) {
#pragma unroll
          for (int i = 0; i < 32; i += 4) *reinterpret_cast<int4*>(o + i) = make_int4(r[i], r[i + 1], r[i + 2], r[i + 3]);
        } else {
          for (int i = 0; i < 32 && j0 + i < a.J; ++i) o[i] = r[i];
        }
      } else {
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __fmaf_rn((float)r[i], s_sc[c0 + i], s_bi[c0 + i]);
        if (a.epi == EPI_JOINTZ) {
          // joint network: z = tanh(e * p) with p the projected value just formed; quantized below
          const float* er = a.mul_e + (long long)a.mul_idx[mi] * a.J + j0;
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 ev = *reinterpret_cast<const float4*>(er + i);
            v[i] = tanh_fixed(__fmul_rn(ev.x, v[i]));
            v[i + 1] = tanh_fixed(__fmul_rn(ev.y, v[i + 1]));
            v[i + 2] = tanh_fixed(__fmul_rn(ev.z, v[i + 2]));
            v[i + 3] = tanh_fixed(__fmul_rn(ev.w, v[i + 3]));
          }
        }
        if (a.epi == EPI_F32) {
          float* o = reinterpret_cast<float*>(a.out) + (long long)m * a.ldo + j0;
          if (j0 + 32 <= a.J && (reinterpret_cast<uintptr_t>(o) & 31) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 8)
              st_global_v8(o + i, make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]),
                           make_float4(v[i + 4], v[i + 5], v[i + 6], v[i + 7]));
          } else if (j0 + 32 <= a.J) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(o + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
          } else {
            for (int i = 0; i < 32 && j0 + i < a.J; ++i) o[i] = v[i];
          }
        } else {  // EPI_QUANT / EPI_QUANT8 (J a multiple of 32)
          const int lo = act_lo(a.out_act), hi = act_hi(a.out_act);
          uint8_t* o = reinterpret_cast<uint8_t*>(a.out) + (long long)m * a.ldo;
          if (a.epi == EPI_QUANT8 || a.epi == EPI_JOINTZ) {
            uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; ++i)
              w[i >> 2] |= (uint32_t)((quantize1(v[i], a.out_act.inv_scale, a.out_act.zero_point, lo, hi) -
                                       a.out_act.zero_point) & 0xFF) << (8 * (i & 3));
            *reinterpret_cast<uint4*>(o + j0) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(o + j0 + 16) = make_uint4(w[4], w[5], w[6], w[7]);
          } else if (a.out_act.bits == 4) {
            uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; ++i)
              w[i >> 3] |= (uint32_t)(quantize1(v[i], a.out_act.inv_scale, a.out_act.zero_point, lo, hi) & 0xF) << (4 * (i & 7));
            *reinterpret_cast<uint4*>(o + (j0 >> 1)) = make_uint4(w[0], w[1], w[2], w[3]);
          } else {
            uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; ++i)
              w[i >> 2] |= (uint32_t)(quantize1(v[i], a.out_act.inv_scale, a.out_act.zero_point, lo, hi) & 0xFF) << (8 * (i & 3));
            *reinterpret_cast<uint4*>(o + j0) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(o + j0 + 16) = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
      }
    }
  } else {
    pdl_trigger();   // idle lanes of the producer and issuer warps
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, GEMM_BN);
}

// ------------------------------------------------------------------ persistent GEMM, int32 out
// The encoder input projection is one large GEMM per layer and direction (thousands of tiles)
// whose int32 result (128 KB per tile) costs more time to write than its MMAs take.  One CTA per
// SM walks the tiles t = blockIdx.x, blockIdx.x + gridDim.x, ... (column tile fastest, so the
// CTAs working at the same time share activation rows and all weights in L2), with two
// accumulators in tensor memory: the epilogue warps drain one while the MMAs of the next tile
// fill the other, and the operand ring keeps streaming across tile boundaries.
constexpr int PG_STAGES = 4;

__global__ void __launch_bounds__(192, 1)
k_mma_gemm_persistent(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b,
                      const MmaGemmArgs a, const int tiles_m, const int tiles_n) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int A_BYTES = BM * BK, B_BYTES = GEMM_BN * BK, STAGE = A_BYTES + B_BYTES;
  __shared__ uint64_t full[PG_STAGES], empty[PG_STAGES], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nk = (a.K + BK - 1) / BK;
  const int n_tiles = tiles_m * tiles_n;

  if (tid == 0) {
    for (int s = 0; s < PG_STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 4);   // one arrival per epilogue warp
    }
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 5) tmem_alloc(&tmem_base_s, 2 * GEMM_BN);
  if (warp == 4 && lane == 0) {
    prefetch_tmap(&tma_a);
    prefetch_tmap(&tma_b);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  pdl_wait();

  if (warp == 4 && lane == 0) {
    // ---- TMA producer: the ring position runs on across tiles
    bool ok = true;
    int s = 0, g = 0;
    uint32_t ph = 0;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * GEMM_BN;
      for (int i = 0; i < nk; ++i, ++g) {
        if (g >= PG_STAGES) ok = mbar_wait(&empty[s], ph ^ 1);
        if (!ok) break;
        mbar_expect_tx(&full[s], STAGE);
        tma_load_2d(smem + s * STAGE, &tma_a, i * BK, m0, &full[s]);
        tma_load_2d(smem + s * STAGE + A_BYTES, &tma_b, i * BK, n0, &full[s]);
        if (++s == PG_STAGES) {
          s = 0;
          ph ^= 1;
        }
      }
    }
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp == 5 && lane == 0) {
    // ---- MMA issuer: tile `it` of this CTA accumulates into buffer it & 1
    const uint32_t idesc = umma_idesc_i8(BM, GEMM_BN);
    bool ok = true;
    int s = 0, it = 0;
    uint32_t ph = 0;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
      const int buf = it & 1, use = it >> 1;
      if (use >= 1) {   // the epilogue must have read the previous contents of this buffer
        ok = mbar_wait(&acc_empty[buf], (use - 1) & 1);
        if (!ok) break;
        tc_fence_after();
      }
      const uint32_t d = tmem + (uint32_t)(buf * GEMM_BN);
      for (int i = 0; i < nk; ++i) {
        ok = mbar_wait(&full[s], ph);
        if (!ok) break;
        tc_fence_after();
        const uint64_t da = umma_desc_sw128(smem_u32(smem + s * STAGE));
        const uint64_t db = umma_desc_sw128(smem_u32(smem + s * STAGE + A_BYTES));
#pragma unroll
        for (int kk = 0; kk < BK / 32; ++kk) umma_i8(d, da + 2 * kk, db + 2 * kk, idesc, (i | kk) != 0);
        umma_commit(&empty[s]);
        if (++s == PG_STAGES) {
          s = 0;
          ph ^= 1;
        }
      }
      if (ok) umma_commit(&acc_full[buf]);
    }
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp < 4) {
    // ---- epilogue: warp w drains TMEM lanes [32 w, 32 w + 32) of the finished accumulator
    bool ok = true;
    int it = 0;
    const bool wide = (reinterpret_cast<uintptr_t>(a.out) & 31) == 0 && ((a.ldo * 4) & 31) == 0;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
      const int buf = it & 1, use = it >> 1;
      const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * GEMM_BN;
      ok = mbar_wait(&acc_full[buf], use & 1);
      if (!ok) break;
      tc_fence_after();
      const int m = m0 + warp * 32 + lane;
      const uint32_t taddr = tmem + (uint32_t)(buf * GEMM_BN) + ((uint32_t)(warp * 32) << 16);
      // two register sets: the TMEM load of the next 32 columns is in flight while these are stored
      auto store32 = [&](const int (&r)[32], int c0) {
        const int j0 = n0 + c0;
        if (m >= a.M || j0 >= a.J) return;
        int32_t* o = reinterpret_cast<int32_t*>(a.out) + (long long)m * a.ldo + j0;
        if (j0 + 32 <= a.J && wide) {
#pragma unroll
          for (int i = 0; i < 32; i += 8)
            st_global_v8_b32(o + i, r[i], r[i + 1], r[i + 2], r[i + 3], r[i + 4], r[i + 5], r[i + 6], r[i + 7]);
        } else if (j0 + 32 <= a.J) {
#pragma unroll
          for (int i = 0; i < 32; i += 4) *reinterpret_cast<int4*>(o + i) = make_int4(r[i], r[i + 1], r[i + 2], r[i + 3]);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (j0 + i < a.J) o[i] = r[i];
        }
      };
      int r0[32], r1[32];
      tmem_ld32(taddr, r0);
#pragma unroll 1
      for (int c0 = 0; c0 < GEMM_BN; c0 += 64) {
        tmem_ld_wait();
        tmem_ld32(taddr + c0 + 32, r1);
        store32(r0, c0);
        tmem_ld_wait();
        if (c0 + 64 < GEMM_BN) {
          tmem_ld32(taddr + c0 + 64, r0);
        } else {
          // the accumulator has been read completely: hand it back before the last stores
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
        store32(r1, c0 + 32);
      }
    }
    pdl_trigger();
    if (!ok && lane == 0) flag_timeout(a.status);
  } else {
    pdl_trigger();   // idle lanes of the producer and issuer warps
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 2 * GEMM_BN);
}

static int g_sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

// x8: int8 activations [M, K] (pitch x_pitch), w8: int8 weights [J, K] (pitch w_pitch).
cudaError_t launch_mma_gemm(const int8_t* x8, long long x_pitch, int M, const int8_t* w8,
                            long long w_pitch, int J, int K, int epi, void* out, long long ldo,
                            const int32_t* out_idx, const float* w_scale, const float* bias,
                            float x_scale, const q4_act* out_act, int32_t* status,
                            const int32_t* n_active, cudaStream_t s, bool dependent, const float* mul_e,
                            const int32_t* mul_idx) {
  if (M <= 0 || J <= 0) return cudaSuccess;
  if (epi == EPI_JOINTZ && (!mul_e || !mul_idx || J % 32 != 0)) return cudaErrorInvalidValue;
  CUtensorMap ta, tb;
  if (!make_tmap_i8(&ta, x8, K, M, x_pitch, BM) || !make_tmap_i8(&tb, w8, K, J, w_pitch, GEMM_BN))
    return cudaErrorInvalidValue;
  MmaGemmArgs a;
  memset(&a, 0, sizeof(a));
  a.M = M;
  a.J = J;
  a.K = K;
  a.epi = epi;
  a.out = out;
  a.ldo = ldo;
  a.out_idx = out_idx;
  a.w_scale = w_scale;
  a.bias = bias;
  a.x_scale = x_scale;
  if (out_act) a.out_act = *out_act;
  a.status = status;
  a.n_active = n_active;
  a.mul_e = mul_e;
  a.mul_idx = mul_idx;
  a.wait_limit = g_wait_limit;
  a.skip_producer = g_skip_producer;
  const size_t smem = (size_t)GEMM_STAGES * (BM * BK + GEMM_BN * BK) + 1024;
  const size_t smem_p = (size_t)PG_STAGES * (BM * BK + GEMM_BN * BK) + 1024;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_mma_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_mma_gemm_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_p);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid((J + GEMM_BN - 1) / GEMM_BN, (M + BM - 1) / BM);
  if (epi == EPI_I32 && !out_idx && !n_active && (long long)grid.x * grid.y > 2 * g_sm_count()) {
    // more than two tiles per SM: one persistent CTA per SM with overlapped epilogue
    timing_begin(s);
    cudaError_t le = launch_ex(k_mma_gemm_persistent, dim3(g_sm_count()), dim3(192), smem_p, s, dependent, 1, ta, tb,
                               a, (int)grid.y, (int)grid.x);
    timing_end(s);
    ++g_launches;
    return le != cudaSuccess ? le : cudaGetLastError();
  }
  timing_begin(s);
  cudaError_t le = launch_ex(k_mma_gemm, grid, dim3(192), smem, s, dependent, 1, ta, tb, a);
  timing_end(s);
  ++g_launches;
  return le != cudaSuccess ? le : cudaGetLastError();
}

// ------------------------------------------------------------------ fused LM head
// One launch per language model (and one for the joint network's output layer) and iteration.
// A cluster of ceil(V/NB) CTAs serves one tile of 128 rows; every CTA computes the bottleneck
// GEMM (H -> D = 256, cheap, int32 in TMEM), de-quantizes + biases + re-quantizes it
// (asymmetric constants) straight into a swizzled shared-memory operand tile, multiplies it
// with its own block of NB output-layer rows, and keeps its NB logits per row in registers
// (NB/4 per thread).  Row maxima and sums of the blocks are exchanged through distributed
// shared memory, one cluster barrier later every thread knows the row's log-sum-exp and stores
// log-probabilities: one global write, no separate log-softmax pass.  With H = 0 there is no
// bottleneck: the 256-wide operand rows are read from memory (joint network).
constexpr int HEAD_D = 256;
constexpr int HEAD_STAGES = 4;
constexpr int HEAD_EPI_WARPS = 16;           // four warps per TMEM lane quarter, NB/4 columns each
constexpr int HEAD_THREADS = 32 * (HEAD_EPI_WARPS + 2);
constexpr int HEAD_MAX_BLOCKS = 8;           // portable cluster size: V <= 8 NB

__device__ __forceinline__ void cl_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cl_store_f32(const float* local, uint32_t rank, float v) {
  uint32_t addr = smem_u32(local), remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(addr), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

template <int NB>
__global__ void __launch_bounds__(HEAD_THREADS, 1)
k_mma_lmhead(const __grid_constant__ CUtensorMap tma_h, const __grid_constant__ CUtensorMap tma_wb,
             const __grid_constant__ CUtensorMap tma_wo, const LmHeadArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int A_BYTES = BM * BK, B_BYTES = HEAD_D * BK, STAGE = A_BYTES + B_BYTES;
  constexpr int B2_BYTES = NB * BK;            // one K chunk of my block of output-layer rows
  constexpr int CPT = NB / 4;                  // logits per thread
  __shared__ uint64_t full[HEAD_STAGES], empty[HEAD_STAGES], acc1_full, a2_ready, acc2_full;
  __shared__ uint32_t tmem_base_s;
  __shared__ __align__(16) float s_sc1[HEAD_D], s_b1[HEAD_D], s_sc2[NB], s_b2[NB];
  __shared__ float red_m[4][BM], red_s[4][BM];
  __shared__ float part_m[HEAD_MAX_BLOCKS][BM], part_s[HEAD_MAX_BLOCKS][BM];   // filled by every CTA of the cluster
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m0 = blockIdx.y * BM;
  const int nb = blockIdx.x;                    // my block of output columns = my cluster rank
  const int nblk = gridDim.x;
  const int nk1 = (a.H + BK - 1) / BK;
  const int nloads = nk1 + 2;

  if (tid == 0) {
    for (int s = 0; s < HEAD_STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(&acc1_full, 1);
    mbar_init(&a2_ready, HEAD_EPI_WARPS);
    mbar_init(&acc2_full, 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == HEAD_EPI_WARPS + 1) tmem_alloc(&tmem_base_s, 512);
  if (warp < HEAD_EPI_WARPS) {   // de-quantization constants: weights only, nothing of the previous kernel
    for (int c = tid; c < HEAD_D; c += 32 * HEAD_EPI_WARPS) {
      s_sc1[c] = nk1 > 0 ? __fmul_rn(a.x_scale, __ldg(a.sc_bott + c)) : 0.0f;
      s_b1[c] = (nk1 > 0 && a.b_bott) ? __ldg(a.b_bott + c) : 0.0f;
    }
    for (int c = tid; c < NB; c += 32 * HEAD_EPI_WARPS) {
      const int j = min(nb * NB + c, a.V - 1);
      s_sc2[c] = __fmul_rn(a.q_scale, __ldg(a.sc_out + j));
      s_b2[c] = a.b_out ? __ldg(a.b_out + j) : 0.0f;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  cl_barrier();   // every CTA of the cluster is running before anyone stores into a peer's shared memory
  pdl_wait();   // everything above (this barrier included) overlaps the tail of the previous kernel of the stream
  if (a.n_active && m0 >= *a.n_active) {   // whole row tile without work: the whole cluster leaves
    if (warp == HEAD_EPI_WARPS + 1) tmem_dealloc(tmem, 512);
    return;
  }

  if (warp == HEAD_EPI_WARPS && lane == 0) {
    // ---- TMA producer: bottleneck operands, then my block of output-layer weights
    bool ok = true;
    for (int i = 0; i < nloads && ok; ++i) {
      const int s = i % HEAD_STAGES;
      if (i >= HEAD_STAGES) ok = mbar_wait(&empty[s], ((i / HEAD_STAGES) - 1) & 1);
      if (!ok) break;
      if (i < nk1) {
        mbar_expect_tx(&full[s], STAGE);
        tma_load_2d(smem + s * STAGE, &tma_h, i * BK, m0, &full[s]);
        tma_load_2d(smem + s * STAGE + A_BYTES, &tma_wb, i * BK, 0, &full[s]);
      } else if (nk1 > 0) {
        // only the weight half of the stage is loaded: the activation halves of stages 0 and 1
        // receive the re-quantized bottleneck codes from the epilogue warps
        mbar_expect_tx(&full[s], B2_BYTES);
        tma_load_2d(smem + s * STAGE + A_BYTES, &tma_wo, (i - nk1) * BK, nb * NB, &full[s]);
      } else {
        // no bottleneck: the 256-wide operand rows come from memory (stage i holds chunk i)
        mbar_expect_tx(&full[s], A_BYTES + B2_BYTES);
        tma_load_2d(smem + s * STAGE, &tma_h, i * BK, m0, &full[s]);
        tma_load_2d(smem + s * STAGE + A_BYTES, &tma_wo, i * BK, nb * NB, &full[s]);
      }
    }
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp == HEAD_EPI_WARPS + 1 && lane == 0) {
    // ---- MMA issuer
    const uint32_t idesc1 = umma_idesc_i8(BM, HEAD_D), idesc2 = umma_idesc_i8(BM, NB);
    bool ok = true;
    for (int i = 0; i < nk1 && ok; ++i) {
      const int s = i % HEAD_STAGES;
      ok = mbar_wait(&full[s], (i / HEAD_STAGES) & 1);
      if (!ok) break;
      tc_fence_after();
      const uint64_t da = umma_desc_sw128(smem_u32(smem + s * STAGE));
      const uint64_t db = umma_desc_sw128(smem_u32(smem + s * STAGE + A_BYTES));
#pragma unroll
      for (int kk = 0; kk < BK / 32; ++kk) umma_i8(tmem, da + 2 * kk, db + 2 * kk, idesc1, (i | kk) != 0);
      umma_commit(&empty[s]);
    }
    umma_commit(&acc1_full);
    if (ok && nk1 > 0) ok = mbar_wait(&a2_ready, 0);
    tc_fence_after();
    for (int kc = 0; kc < 2 && ok; ++kc) {
      const int i = nk1 + kc;
      const int s = i % HEAD_STAGES;
      ok = mbar_wait(&full[s], (i / HEAD_STAGES) & 1);
      if (!ok) break;
      tc_fence_after();
      const uint64_t da = umma_desc_sw128(smem_u32(smem + kc * STAGE));      // bottleneck codes / operand rows
      const uint64_t db = umma_desc_sw128(smem_u32(smem + s * STAGE + A_BYTES));
#pragma unroll
      for (int kk = 0; kk < BK / 32; ++kk) umma_i8(tmem + HEAD_D, da + 2 * kk, db + 2 * kk, idesc2, (kc | kk) != 0);
      umma_commit(&empty[s]);
    }
    umma_commit(&acc2_full);
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp < HEAD_EPI_WARPS) {
    // ---- epilogue: warp = (lane quarter q, column share cs)
    const int q = warp & 3, cs = warp >> 2;
    const int rt = q * 32 + lane;
    const int n = m0 + rt;
    int dst = -1;
    if (n < a.N && !(a.n_active && n >= *a.n_active)) dst = a.dst_row ? a.dst_row[n] : n;
    bool ok = true;
    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
    if (nk1 > 0) {
      const int lo = act_lo(a.bott_act), hi = act_hi(a.bott_act), zp = a.bott_act.zero_point;
      ok = mbar_wait(&acc1_full, 0);
      tc_fence_after();
      // bottleneck codes of my row, columns [64 cs, 64 cs + 64), into the swizzled operand tiles
#pragma unroll 1
      for (int ch = 0; ch < 2; ++ch) {
        const int c0 = 64 * cs + 32 * ch;
        int r[32];
        tmem_ld32(taddr + c0, r);
        tmem_ld_wait();
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = 0;
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 sc = *reinterpret_cast<const float4*>(s_sc1 + c0 + i);
          const float4 bi = *reinterpret_cast<const float4*>(s_b1 + c0 + i);
          const float scv[4] = {sc.x, sc.y, sc.z, sc.w}, biv[4] = {bi.x, bi.y, bi.z, bi.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float x = __fmaf_rn((float)r[i + e], scv[e], biv[e]);
            const int code = quantize1(x, a.bott_act.inv_scale, zp, lo, hi) - zp;
            w[(i + e) >> 2] |= (uint32_t)(code & 0xFF) << (8 * ((i + e) & 3));
          }
        }
        const int kc = c0 >> 7, kb = c0 & 127;            // operand chunk and byte within its 128-byte row
        uint8_t* tile = smem + kc * STAGE + (rt >> 3) * 1024 + (rt & 7) * 128;
        *reinterpret_cast<uint4*>(tile + ((((kb >> 4) + 0) ^ (rt & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(tile + ((((kb >> 4) + 1) ^ (rt & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
      }
      fence_proxy_async();        // generic-proxy writes -> visible to the tensor core's async proxy
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&a2_ready);
    }

    // my CPT logits of this block, kept in registers until the row's log-sum-exp is known
    if (ok) ok = mbar_wait(&acc2_full, 0);
    tc_fence_after();
    pdl_trigger();   // both GEMMs are over: the next kernel may set itself up
    float v[CPT];
    float my_m = -INFINITY;
    const int col0 = nb * NB + CPT * cs;       // first vocabulary entry of my share
#pragma unroll
    for (int ch = 0; ch < CPT / 32; ++ch) {
      const int c0 = CPT * cs + 32 * ch;
      int r[32];
      tmem_ld32(taddr + HEAD_D + c0, r);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        const float4 sc = *reinterpret_cast<const float4*>(s_sc2 + c0 + i);
        const float4 bi = *reinterpret_cast<const float4*>(s_b2 + c0 + i);
        v[32 * ch + i + 0] = __fmaf_rn((float)r[i + 0], sc.x, bi.x);
        v[32 * ch + i + 1] = __fmaf_rn((float)r[i + 1], sc.y, bi.y);
        v[32 * ch + i + 2] = __fmaf_rn((float)r[i + 2], sc.z, bi.z);
        v[32 * ch + i + 3] = __fmaf_rn((float)r[i + 3], sc.w, bi.w);
      }
    }
#pragma unroll
    for (int i = 0; i < CPT; ++i)
      if (col0 + i < a.V) my_m = fmaxf(my_m, v[i]);
    // exponentials by the hardware base-2 unit: relative error near 1e-6, far inside what the
    // log-sum-exp of a thousand terms needs
    float my_s = 0.0f;
#pragma unroll
    for (int i = 0; i < CPT; ++i)
      if (col0 + i < a.V) my_s += __expf(v[i] - my_m);
    red_m[cs][rt] = my_m;
    red_s[cs][rt] = my_s;
    asm volatile("bar.sync 1, %0;" ::"n"(32 * HEAD_EPI_WARPS) : "memory");
    if (cs == 0) {   // this CTA's (max, sum) of the row goes to every CTA of the cluster
      const float m = fmaxf(fmaxf(red_m[0][rt], red_m[1][rt]), fmaxf(red_m[2][rt], red_m[3][rt]));
      float ssum = 0.0f;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (red_s[i][rt] > 0.0f) ssum += red_s[i][rt] * __expf(red_m[i][rt] - m);
      for (int r = 0; r < nblk; ++r) {
        cl_store_f32(&part_m[nb][rt], (uint32_t)r, m);
        cl_store_f32(&part_s[nb][rt], (uint32_t)r, ssum);
      }
    }
    cl_barrier();
    // all partials are fetched at once (at most HEAD_MAX_BLOCKS of them), then combined in block order
    float pm[HEAD_MAX_BLOCKS], ps[HEAD_MAX_BLOCKS];
#pragma unroll
    for (int r = 0; r < HEAD_MAX_BLOCKS; ++r) {
      pm[r] = r < nblk ? part_m[r][rt] : -INFINITY;
      ps[r] = r < nblk ? part_s[r][rt] : 0.0f;
    }
    float m = -INFINITY;
#pragma unroll
    for (int r = 0; r < HEAD_MAX_BLOCKS; ++r) m = fmaxf(m, pm[r]);
    float ssum = 0.0f;
#pragma unroll
    for (int r = 0; r < HEAD_MAX_BLOCKS; ++r)
      if (ps[r] > 0.0f) ssum += ps[r] * __expf(pm[r] - m);
    const float lse = m + logf(ssum);
    // A thread's 32 log-probabilities belong to one row and the rows of a warp's lanes are V floats
    // apart, so storing them directly touches 32 lines per instruction.  A full 128-column block goes
    // through shared memory instead (the operand stages are free: both GEMMs are complete) and leaves
    // as whole rows, one 512-byte row per warp-wide store.
    const bool staged = NB == 128 && nb * NB + NB <= a.V && (a.V & 3) == 0 &&
                        (reinterpret_cast<uintptr_t>(a.lp) & 15) == 0;   // uniform per CTA
    if (staged) {
      constexpr int TP = NB + 4;   // row pitch in floats: rows 16-byte aligned, 32 rows spread over the banks
      float* tile = reinterpret_cast<float*>(smem);
      int* tdst = reinterpret_cast<int*>(smem + (size_t)BM * TP * sizeof(float));
      float* trow = tile + rt * TP + CPT * cs;
#pragma unroll
      for (int i = 0; i < CPT; i += 4)
        *reinterpret_cast<float4*>(trow + i) = make_float4(v[i] - lse, v[i + 1] - lse, v[i + 2] - lse, v[i + 3] - lse);
      if (cs == 0) tdst[rt] = ok ? dst : -1;
      asm volatile("bar.sync 1, %0;" ::"n"(32 * HEAD_EPI_WARPS) : "memory");
      int d[BM / HEAD_EPI_WARPS];
      float4 t4[BM / HEAD_EPI_WARPS];
#pragma unroll
      for (int j = 0; j < BM / HEAD_EPI_WARPS; ++j) {   // this warp's 8 rows: fetch first, then store
        const int r = warp + j * HEAD_EPI_WARPS;
        d[j] = tdst[r];
        t4[j] = *reinterpret_cast<const float4*>(tile + r * TP + 4 * lane);
      }
#pragma unroll
      for (int j = 0; j < BM / HEAD_EPI_WARPS; ++j)
        if (d[j] >= 0) *reinterpret_cast<float4*>(a.lp + (long long)d[j] * a.V + nb * NB + 4 * lane) = t4[j];
    } else if (dst >= 0 && ok) {
      float* out = a.lp + (long long)dst * a.V + col0;
      const int left = a.V - col0;
      if (left >= CPT && (reinterpret_cast<uintptr_t>(out) & 31) == 0) {
#pragma unroll
        for (int i = 0; i < CPT; i += 8)   // rows of a warp's lanes are V floats apart: few, wide stores
          st_global_v8(out + i, make_float4(v[i] - lse, v[i + 1] - lse, v[i + 2] - lse, v[i + 3] - lse),
                       make_float4(v[i + 4] - lse, v[i + 5] - lse, v[i + 6] - lse, v[i + 7] - lse));
      } else if (left >= CPT) {
#pragma unroll
        for (int i = 0; i < CPT; i += 4)
          *reinterpret_cast<float4*>(out + i) = make_float4(v[i] - lse, v[i + 1] - lse, v[i + 2] - lse, v[i + 3] - lse);
      } else {
#pragma unroll
        for (int i = 0; i < CPT; ++i)
          if (i < left) out[i] = v[i] - lse;
      }
    }
    if (!ok && lane == 0) flag_timeout(a.status);
  }
  __syncwarp();
  if (warp >= HEAD_EPI_WARPS) {   // the producer and issuer warps join the cluster barrier too
    pdl_trigger();
    cl_barrier();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == HEAD_EPI_WARPS + 1) tmem_dealloc(tmem, 512);
  // no barrier at the exit: every store into a peer's shared memory precedes the exchange barrier above
  // (release on arrival, acquire on the wait), after which only local memory is touched
}

cudaError_t launch_mma_lmhead(const LmHeadArgs& a, const int8_t* h8, long long h_pitch, const int8_t* wb8,
                              const int8_t* wo8, cudaStream_t s, bool dependent) {
  if (a.N <= 0) return cudaSuccess;
  const int rows_pad = (a.N + BM - 1) / BM * BM;
  const int NB = a.V <= 128 * HEAD_MAX_BLOCKS ? 128 : 256;   // the narrower block spreads a row over more CTAs
  const int nblk = (a.V + NB - 1) / NB;
  if (nblk > HEAD_MAX_BLOCKS) return cudaErrorInvalidValue;
  CUtensorMap th, tb, to;
  const int Ka = a.H > 0 ? a.H : HEAD_D;
  if (!make_tmap_i8(&th, h8, Ka, rows_pad, h_pitch, BM) || !make_tmap_i8(&to, wo8, HEAD_D, a.V, HEAD_D, NB))
    return cudaErrorInvalidValue;
  if (a.H > 0) {
    if (!make_tmap_i8(&tb, wb8, a.H, HEAD_D, a.H, HEAD_D)) return cudaErrorInvalidValue;
  } else {
    tb = to;   // unused without a bottleneck
  }
  const size_t smem = (size_t)HEAD_STAGES * (BM * BK + HEAD_D * BK) + 1024;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_mma_lmhead<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_mma_lmhead<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  timing_begin(s);
  cudaError_t e;
  if (NB == 128)
    e = launch_ex(k_mma_lmhead<128>, dim3(nblk, rows_pad / BM), dim3(HEAD_THREADS), smem, s, dependent,
                  (unsigned)nblk, th, tb, to, a);
  else
    e = launch_ex(k_mma_lmhead<256>, dim3(nblk, rows_pad / BM), dim3(HEAD_THREADS), smem, s, dependent,
                  (unsigned)nblk, th, tb, to, a);
  timing_end(s);
  ++g_launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

// ------------------------------------------------------------------ fused LSTM step
// EXTRAS = false drops the second code (yq_out), the fp32 copy (h_f32) and the accumulator dumps
// from the cell loop: the search needs none of them, and without their branches the four cells
// of a thread are scheduled as one block.
// PREMUL = true: sc_ih / sc_hh already hold (input scale * row scale) and (hidden scale * row
// scale), the products the de-quantization needs (same fp32 multiplication, done once).
template <bool EXTRAS, bool PREMUL>
__global__ void __launch_bounds__(32 * (LSTM_EPI_WARPS + 2), 2)
k_mma_lstm(const __grid_constant__ CUtensorMap tma_xa, const __grid_constant__ CUtensorMap tma_xw,
           const __grid_constant__ CUtensorMap tma_ha, const __grid_constant__ CUtensorMap tma_hw,
           const MmaLstmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int A_BYTES = BM * BK, B_BYTES = LSTM_BN * BK, STAGE = A_BYTES + B_BYTES;
  constexpr int TCOLS = 2 * LSTM_BN;
  __shared__ uint64_t full[LSTM_STAGES], empty[LSTM_STAGES], acc_full;
  __shared__ uint32_t tmem_base_s;
  __shared__ float4 s_cst[3][LSTM_BN / 4];   // input scales, recurrent scales, bias of this tile's cells (4 gates each)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * LSTM_BN;   // row tiles slowest: tiles with work are dispatched first
  const int nkx = a.acc_pre ? 0 : (a.Kx_pad + BK - 1) / BK;
  const int nkh = (a.H + BK - 1) / BK;
  const int nk = nkx + nkh;

  if (tid == 0) {
    for (int s = 0; s < LSTM_STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(&acc_full, 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == LSTM_EPI_WARPS + 1) tmem_alloc(&tmem_base_s, TCOLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  // Everything above overlaps the tail of the previous kernel of the stream.  With h_first only
  // the input operand is that kernel's output: the recurrent half of the K loop (operands from
  // kernels further back, all complete) runs before the wait, the input half after it.
  const bool h_first = a.h_first != 0 && nkx > 0;
  if (!h_first) pdl_wait();
  const bool has_work = !(a.n_active && m0 >= *a.n_active);   // uniform per CTA
  if (a.trigger_early) pdl_trigger();   // the successor has a half it can run beside this kernel
  const int x_first = h_first ? nkh : 0, hh_first = h_first ? 0 : nkx;   // first chunk of each part

  if (!has_work) {
    if (h_first) pdl_wait();   // whole tile without work; still ordered behind the previous kernel
  } else if (warp == LSTM_EPI_WARPS && lane == 0) {
    bool ok = true;
    for (int i = 0; i < nk && ok; ++i) {
      const int s = i % LSTM_STAGES;
      if (i >= LSTM_STAGES) ok = mbar_wait(&empty[s], ((i / LSTM_STAGES) - 1) & 1);
      if (!ok) break;
      const bool xpart = h_first ? i >= nkh : i < nkx;
      if (h_first && i == x_first) pdl_wait();
      mbar_expect_tx(&full[s], STAGE);
      if (xpart) {
        tma_load_2d(smem + s * STAGE, &tma_xa, (i - x_first) * BK, m0, &full[s]);
        tma_load_2d(smem + s * STAGE + A_BYTES, &tma_xw, (i - x_first) * BK, n0, &full[s]);
      } else {
        tma_load_2d(smem + s * STAGE, &tma_ha, (i - hh_first) * BK, m0, &full[s]);
        tma_load_2d(smem + s * STAGE + A_BYTES, &tma_hw, (i - hh_first) * BK, n0, &full[s]);
      }
    }
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp == LSTM_EPI_WARPS + 1 && lane == 0) {
    const uint32_t idesc = umma_idesc_i8(BM, LSTM_BN);
    bool ok = true;
    for (int i = 0; i < nk && ok; ++i) {
      const int s = i % LSTM_STAGES;
      ok = mbar_wait(&full[s], (i / LSTM_STAGES) & 1);
      if (!ok) break;
      tc_fence_after();
      const uint64_t da = umma_desc_sw128(smem_u32(smem + s * STAGE));
      const uint64_t db = umma_desc_sw128(smem_u32(smem + s * STAGE + A_BYTES));
      const bool xpart = h_first ? i >= nkh : i < nkx;
      const uint32_t d = tmem + (xpart ? 0 : LSTM_BN);
      const int first = xpart ? x_first : hh_first;
#pragma unroll
      for (int kk = 0; kk < BK / 32; ++kk) umma_i8(d, da + 2 * kk, db + 2 * kk, idesc, (i != first) || kk != 0);
      umma_commit(&empty[s]);
    }
    umma_commit(&acc_full);
    pdl_trigger();
    if (!ok) flag_timeout(a.status);
  } else if (warp < LSTM_EPI_WARPS) {
    const int q = warp & 3, hf = warp >> 2;
    const int rt = q * 32 + lane;            // row within the tile
    const int n = m0 + rt;                   // row of this launch
    int src = -1, dst = -1;
    if (n < a.N && !(a.n_active && n >= *a.n_active)) {
      dst = a.dst_row ? a.dst_row[n] : n;
      src = a.src_row ? a.src_row[n] : n;
    }
    // previous cell states of all my cells: requested before the main loop ends (they belong to
    // rows no kernel of this iteration writes), so that their trip to memory costs the epilogue nothing
    float4 cprev_all[LSTM_BN / 32];
    // 16 cells = 64 contiguous bytes per row: two 256-bit accesses when the layout allows it
    const bool wide = (n0 >> 2) + hf * (LSTM_BN / 8) + LSTM_BN / 8 <= a.H && (a.H & 7) == 0 &&
                      ((reinterpret_cast<uintptr_t>(a.c_in) | reinterpret_cast<uintptr_t>(a.c_out)) & 31) == 0;
#pragma unroll
    for (int ch = 0; ch < LSTM_BN / 32; ++ch) cprev_all[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (wide) {
      if (dst >= 0 && src >= 0) {
        const float* cp0 = a.c_in + (long long)src * a.H + (n0 >> 2) + hf * (LSTM_BN / 8);
        ld_global_v8(cp0, cprev_all[0], cprev_all[1]);
        ld_global_v8(cp0 + 8, cprev_all[2], cprev_all[3]);
      }
    } else {
#pragma unroll
      for (int ch = 0; ch < LSTM_BN / 32; ++ch) {
        const int cell0 = (n0 >> 2) + hf * (LSTM_BN / 8) + ch * 4;
        if (dst >= 0 && src >= 0 && cell0 < a.H)
          cprev_all[ch] = *reinterpret_cast<const float4*>(a.c_in + (long long)src * a.H + cell0);
      }
    }
    // de-quantization constants of the tile's 32 cells: weights only (nothing of an earlier kernel),
    // fetched while the main loop runs so that the cell loop reads them from shared memory
    if (tid < 3 * (LSTM_BN / 4)) {
      const int which = tid / (LSTM_BN / 4), cell = (n0 >> 2) + tid % (LSTM_BN / 4);
      const float* src = which == 0 ? a.sc_ih : which == 1 ? a.sc_hh : a.bias;
      s_cst[which][tid % (LSTM_BN / 4)] =
          cell < a.H ? __ldg(reinterpret_cast<const float4*>(src) + cell) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    asm volatile("bar.sync 1, %0;" ::"n"(32 * LSTM_EPI_WARPS) : "memory");
    const bool ok = mbar_wait(&acc_full, 0);
    tc_fence_after();
    if (h_first) pdl_wait();   // before the first global write of this thread
    pdl_trigger();   // the main loop is over: the next kernel may set itself up
    if (!ok && lane == 0) flag_timeout(a.status);
    const bool live = ok && dst >= 0;
    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
    const int H = a.H;
    const float sx = (live && a.x_scale_vec) ? a.x_scale_vec[n % a.x_scale_mod] : a.x_scale;
    const float sh = a.hid_act.scale;
    const int hlo = act_lo(a.hid_act), hhi = act_hi(a.hid_act);
    const int ylo = act_lo(a.out_act), yhi = act_hi(a.out_act);
    constexpr int CELLS_PER_HALF = LSTM_BN / 4 / 2;   // 16
    // Without the extras the codes of all 16 cells of a thread are kept and stored once: the rows
    // of a warp's lanes lie far apart, so every store instruction touches 32 lines, and four small
    // stores per output cost the load/store unit four times as much as one wide one.
    const int cell_first = (n0 >> 2) + hf * CELLS_PER_HALF;
    const bool combine = !EXTRAS && cell_first + CELLS_PER_HALF <= H;
    uint32_t w8[CELLS_PER_HALF / 4];
#pragma unroll
    for (int ch = 0; ch < CELLS_PER_HALF / 4; ++ch) w8[ch] = 0;
    float4 c_even = make_float4(0.f, 0.f, 0.f, 0.f);   // new cell states of the even chunk, stored with the odd one
#pragma unroll
    for (int ch = 0; ch < CELLS_PER_HALF / 4; ++ch) {
      const int ct = hf * CELLS_PER_HALF + ch * 4;     // first cell of the chunk within the tile
      const int cell0 = (n0 >> 2) + ct;
      int ih[16], hh[16];
      if (nkx > 0) {
        tmem_ld16(taddr + 4 * ct, ih);
      }
      tmem_ld16(taddr + LSTM_BN + 4 * ct, hh);
      tmem_ld_wait();
      if (!live || cell0 >= H) continue;
      if (nkx == 0) {
        const int4* p = reinterpret_cast<const int4*>(a.acc_pre + (long long)n * a.acc_pre_ld + 4 * cell0);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int4 v = p[c];
          ih[4 * c] = v.x;
          ih[4 * c + 1] = v.y;
          ih[4 * c + 2] = v.z;
          ih[4 * c + 3] = v.w;
        }
      }
      const float4 cprev = cprev_all[ch];
      const float cp[4] = {cprev.x, cprev.y, cprev.z, cprev.w};
      float cn[4], hn[4];
      int qh[4], qy[4];
      // pre-activations of the four cells: acc_hh * s_hh + (acc_ih * s_ih + bias), gates (i, f) and (g, o)
      // as pairs on the paired fp32 instructions (the same two roundings per value as the scalar form)
      float pre[4][4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float4 s_ih = s_cst[0][ct + c], s_hh = s_cst[1][ct + c], bb = s_cst[2][ct + c];
        const uint64_t sih0 = PREMUL ? pk2(s_ih.x, s_ih.y) : pk2(__fmul_rn(sx, s_ih.x), __fmul_rn(sx, s_ih.y));
        const uint64_t sih1 = PREMUL ? pk2(s_ih.z, s_ih.w) : pk2(__fmul_rn(sx, s_ih.z), __fmul_rn(sx, s_ih.w));
        const uint64_t shh0 = PREMUL ? pk2(s_hh.x, s_hh.y) : pk2(__fmul_rn(sh, s_hh.x), __fmul_rn(sh, s_hh.y));
        const uint64_t shh1 = PREMUL ? pk2(s_hh.z, s_hh.w) : pk2(__fmul_rn(sh, s_hh.z), __fmul_rn(sh, s_hh.w));
        const uint64_t v0 = fma2(pk2((float)hh[4 * c + 0], (float)hh[4 * c + 1]), shh0,
                                 fma2(pk2((float)ih[4 * c + 0], (float)ih[4 * c + 1]), sih0, pk2(bb.x, bb.y)));
        const uint64_t v1 = fma2(pk2((float)hh[4 * c + 2], (float)hh[4 * c + 3]), shh1,
                                 fma2(pk2((float)ih[4 * c + 2], (float)ih[4 * c + 3]), sih1, pk2(bb.z, bb.w)));
        upk2(v0, pre[c][0], pre[c][1]);
        upk2(v1, pre[c][2], pre[c][3]);
      }
#pragma unroll
      for (int c = 0; c < 4; c += 2)   // two cells per call
        cell_fixed2(pre[c][0], pre[c][1], pre[c][2], pre[c][3], cp[c], pre[c + 1][0], pre[c + 1][1], pre[c + 1][2],
                    pre[c + 1][3], cp[c + 1], cn[c], hn[c], cn[c + 1], hn[c + 1]);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int cell = cell0 + c;
        qh[c] = quantize1(hn[c], a.hid_act.inv_scale, a.hid_act.zero_point, hlo, hhi);
        qy[c] = EXTRAS ? quantize1(hn[c], a.out_act.inv_scale, a.out_act.zero_point, ylo, yhi) : 0;
        if (EXTRAS && a.dbg_ih) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            a.dbg_ih[(long long)n * a.dbg_ld + g * H + cell] = ih[4 * c + g];
            a.dbg_hh[(long long)n * a.dbg_ld + g * H + cell] = hh[4 * c + g];
          }
        }
      }
      if (wide) {
        if (ch & 1)
          st_global_v8(a.c_out + (long long)dst * H + cell0 - 4, c_even, make_float4(cn[0], cn[1], cn[2], cn[3]));
        else
          c_even = make_float4(cn[0], cn[1], cn[2], cn[3]);
      } else {
        *reinterpret_cast<float4*>(a.c_out + (long long)dst * H + cell0) = make_float4(cn[0], cn[1], cn[2], cn[3]);
      }
      if (EXTRAS && a.h_f32) *reinterpret_cast<float4*>(a.h_f32 + (long long)n * H + cell0) = make_float4(hn[0], hn[1], hn[2], hn[3]);
      w8[ch] = (uint32_t)(qh[0] & 0xFF) | ((uint32_t)(qh[1] & 0xFF) << 8) | ((uint32_t)(qh[2] & 0xFF) << 16) |
               ((uint32_t)(qh[3] & 0xFF) << 24);
      if (combine) continue;
      if (a.hq_out) {
        if (a.hid_act.bits == 4)
          *reinterpret_cast<uint16_t*>(a.hq_out + (long long)dst * a.hq_ld + (cell0 >> 1)) =
              (uint16_t)((qh[0] & 0xF) | ((qh[1] & 0xF) << 4) | ((qh[2] & 0xF) << 8) | ((qh[3] & 0xF) << 12));
        else
          *reinterpret_cast<uint32_t*>(a.hq_out + (long long)dst * a.hq_ld + cell0) =
              (uint32_t)(qh[0] & 0xFF) | ((uint32_t)(qh[1] & 0xFF) << 8) | ((uint32_t)(qh[2] & 0xFF) << 16) | ((uint32_t)(qh[3] & 0xFF) << 24);
      }
      if (a.h8_out)
        *reinterpret_cast<uint32_t*>(a.h8_out + (long long)n * a.h8_ld + cell0) =
            (uint32_t)(qh[0] & 0xFF) | ((uint32_t)(qh[1] & 0xFF) << 8) | ((uint32_t)(qh[2] & 0xFF) << 16) | ((uint32_t)(qh[3] & 0xFF) << 24);
      if (EXTRAS && a.yq_out) {
        if (a.out_act.bits == 4)
          *reinterpret_cast<uint16_t*>(a.yq_out + (long long)n * a.yq_ld + (cell0 >> 1)) =
              (uint16_t)((qy[0] & 0xF) | ((qy[1] & 0xF) << 4) | ((qy[2] & 0xF) << 8) | ((qy[3] & 0xF) << 12));
        else
          *reinterpret_cast<uint32_t*>(a.yq_out + (long long)n * a.yq_ld + cell0) =
              (uint32_t)(qy[0] & 0xFF) | ((uint32_t)(qy[1] & 0xFF) << 8) | ((uint32_t)(qy[2] & 0xFF) << 16) | ((uint32_t)(qy[3] & 0xFF) << 24);
      }
    }
    if (combine && live) {
      static_assert(CELLS_PER_HALF == 16, "one uint4 of int8 codes per thread");
      if (a.h8_out)
        *reinterpret_cast<uint4*>(a.h8_out + (long long)n * a.h8_ld + cell_first) = make_uint4(w8[0], w8[1], w8[2], w8[3]);
      if (a.hq_out) {
        if (a.hid_act.bits == 4) {
          uint32_t lo = 0, hi = 0;   // 16 nibbles, cell order
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            lo |= ((w8[0] >> (8 * c)) & 0xFu) << (4 * c) | ((w8[1] >> (8 * c)) & 0xFu) << (16 + 4 * c);
            hi |= ((w8[2] >> (8 * c)) & 0xFu) << (4 * c) | ((w8[3] >> (8 * c)) & 0xFu) << (16 + 4 * c);
          }
          *reinterpret_cast<uint2*>(a.hq_out + (long long)dst * a.hq_ld + (cell_first >> 1)) = make_uint2(lo, hi);
        } else {
          *reinterpret_cast<uint4*>(a.hq_out + (long long)dst * a.hq_ld + cell_first) = make_uint4(w8[0], w8[1], w8[2], w8[3]);
        }
      }
    }
  } else {
    pdl_trigger();   // idle lanes of the producer and issuer warps
  }
  tc_fence_before();
  __syncthreads();
  if (warp == LSTM_EPI_WARPS + 1) tmem_dealloc(tmem, TCOLS);
}

// Operands: xa int8 [rows_pad, Kx_pad] (ignored with acc_pre), xw int8 [4H, Kx_pad] interleaved,
// ha int8 [rows_pad, H], hw int8 [4H, H] interleaved.  rows_pad = N rounded up to 128.
cudaError_t launch_mma_lstm(const MmaLstmArgs& a, const int8_t* xa, long long xa_pitch,
                            const int8_t* xw, long long xw_pitch, const int8_t* ha, long long ha_pitch,
                            const int8_t* hw, long long hw_pitch, cudaStream_t s, bool dependent) {
  if (a.N <= 0) return cudaSuccess;
  const int rows_pad = (a.N + BM - 1) / BM * BM;
  CUtensorMap txa, txw, tha, thw;
  if (!make_tmap_i8(&tha, ha, a.H, rows_pad, ha_pitch, BM) || !make_tmap_i8(&thw, hw, a.H, 4 * a.H, hw_pitch, LSTM_BN))
    return cudaErrorInvalidValue;
  if (a.acc_pre) {
    txa = tha;
    txw = thw;
  } else if (!make_tmap_i8(&txa, xa, a.Kx_pad, rows_pad, xa_pitch, BM) ||
             !make_tmap_i8(&txw, xw, a.Kx_pad, 4 * a.H, xw_pitch, LSTM_BN)) {
    return cudaErrorInvalidValue;
  }
  const size_t smem = (size_t)LSTM_STAGES * (BM * BK + LSTM_BN * BK) + 1024;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_mma_lstm<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_mma_lstm<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_mma_lstm<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid((4 * a.H + LSTM_BN - 1) / LSTM_BN, rows_pad / BM);
  const bool extras = a.yq_out || a.h_f32 || a.dbg_ih;
  if (a.premultiplied && (extras || a.x_scale_vec)) return cudaErrorInvalidValue;
  const dim3 block(32 * (LSTM_EPI_WARPS + 2));
  timing_begin(s);
  cudaError_t le;
  if (extras)
    le = launch_ex(k_mma_lstm<true, false>, grid, block, smem, s, dependent, 1, txa, txw, tha, thw, a);
  else if (a.premultiplied)
    le = launch_ex(k_mma_lstm<false, true>, grid, block, smem, s, dependent, 1, txa, txw, tha, thw, a);
  else
    le = launch_ex(k_mma_lstm<false, false>, grid, block, smem, s, dependent, 1, txa, txw, tha, thw, a);
  timing_end(s);
  ++g_launches;
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace q4
