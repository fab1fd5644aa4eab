// Shared device helpers of the CUDA library: operand tile staging (packed codes
// in global memory -> int8 in shared memory), the quantizer, launch accounting.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/q4rnnt.h"

namespace q4 {

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may
// start while its predecessor in the stream is still running; pdl_wait() returns once that
// predecessor has completed and its writes are visible (at once when the launch carries no such
// attribute), pdl_trigger() lets the successor's CTAs be scheduled once every CTA of this grid
// has called it or exited.  Nothing produced by an earlier kernel is read before pdl_wait().
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }


constexpr int TILE = 64;        // rows of each operand per CTA tile
constexpr int KC = 128;         // K elements staged per chunk
constexpr int PITCH = KC + 16;  // shared-memory row pitch in bytes (16 B aligned, conflict-free)
constexpr int NT = 256;         // threads per CTA of the tile kernels

extern int64_t g_launches;      // kernels launched by this process
extern int64_t g_quant_calls;   // activation-quantizer applications enqueued by this process

// Where the rows of an operand live: row n is at base + (idx ? idx[n] : n) * stride bytes;
// a negative index means "no row" (reads as zeros / is not written).
struct RowSrc {
  const uint8_t* base;
  long long stride;
  const int32_t* idx;
};

__device__ __forceinline__ int dp4a(int a, int b, int c) { return __dp4a(a, b, c); }

// 8 packed nibbles -> two words of 4 int8 each (even elements, odd elements).  Both
// operands of a dot product are unpacked the same way, so the element order inside a
// word does not matter.  sub = value subtracted from every element (8 via the xor trick
// for two's complement; the zero point for unsigned codes).
__device__ __forceinline__ void unpack8(uint32_t w, bool is_signed, uint32_t zp4, uint32_t& even,
                                        uint32_t& odd) {
  uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;
  if (is_signed) {
    even = __vsub4(lo ^ 0x08080808u, 0x08080808u);
    odd = __vsub4(hi ^ 0x08080808u, 0x08080808u);
  } else {
    even = __vsub4(lo, zp4);
    odd = __vsub4(hi, zp4);
  }
}

// 16 packed 2-bit codes (two's complement, element i in bits 2i, 2i+1) -> four words of 4 int8,
// natural element order.
__device__ __forceinline__ void unpack16x2(uint32_t w, uint32_t (&o)[4]) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint32_t v = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int c = (int)((w >> (2 * (4 * j + e))) & 3u);
      v |= (uint32_t)(((c ^ 2) - 2) & 0xFF) << (8 * e);
    }
    o[j] = v;
  }
}
// 8 packed nibbles -> two words of 4 int8 in natural element order (elements 0..3, 4..7).
__device__ __forceinline__ void unpack8_natural(uint32_t w, bool is_signed, uint32_t zp4, uint32_t& lo,
                                                uint32_t& hi) {
  uint32_t even, odd;
  unpack8(w, is_signed, zp4, even, odd);
  lo = __byte_perm(even, odd, 0x5140);   // e0 o0 e1 o1
  hi = __byte_perm(even, odd, 0x7362);   // e2 o2 e3 o3
}

// Stage one K chunk [k0, k0+KC) of a 64-row operand tile into shared memory as int8, natural
// element order whatever the storage width, so that operands of different widths can meet (2-bit
// or 4-bit weights with 4- or 8-bit activations).
// rowp[s] = first byte of the global row that belongs in shared row s (nullptr = zeros).
// Thread t handles 32 elements of row t/4.  bits = storage width of the codes (2: signed only).
__device__ __forceinline__ void stage_chunk(int8_t* smem, const uint8_t* const* rowp, int k0,
                                            int k_pad, int bits, bool is_signed, uint32_t zp4, int tid) {
  const int s = tid >> 2, seg = tid & 3;
  const int k = k0 + 32 * seg;
  uint4 o0 = make_uint4(0, 0, 0, 0), o1 = o0;
  const uint8_t* p = rowp[s];
  if (p != nullptr && k < k_pad) {
    if (bits == 4) {
      const uint4 v = *reinterpret_cast<const uint4*>(p + (k >> 1));
      unpack8_natural(v.x, is_signed, zp4, o0.x, o0.y);
      unpack8_natural(v.y, is_signed, zp4, o0.z, o0.w);
      unpack8_natural(v.z, is_signed, zp4, o1.x, o1.y);
      unpack8_natural(v.w, is_signed, zp4, o1.z, o1.w);
    } else if (bits == 2) {
      const uint2 v = *reinterpret_cast<const uint2*>(p + (k >> 2));
      uint32_t a[4], b[4];
      unpack16x2(v.x, a);
      unpack16x2(v.y, b);
      o0 = make_uint4(a[0], a[1], a[2], a[3]);
      o1 = make_uint4(b[0], b[1], b[2], b[3]);
    } else {
      o0 = *reinterpret_cast<const uint4*>(p + k);
      o1 = *reinterpret_cast<const uint4*>(p + k + 16);
    }
  }
  uint4* d = reinterpret_cast<uint4*>(smem + s * PITCH + 32 * seg);
  d[0] = o0;
  d[1] = o1;
}

// Eq. 2 in fp32: one multiply by the stored reciprocal, round half to even, add the zero
// point, clamp.  cvt.rni saturates and maps NaN to 0.
__device__ __forceinline__ int quantize1(float x, float inv_scale, int zp, int lo, int hi) {
  int q = __float2int_rn(__fmul_rn(x, inv_scale));
  q = max(min(q, 1000000000), -1000000000) + zp;
  return max(min(q, hi), lo);
}
__device__ __forceinline__ int act_lo(const q4_act& a) { return a.is_signed ? -(1 << (a.bits - 1)) : 0; }
__device__ __forceinline__ int act_hi(const q4_act& a) {
  return a.is_signed ? (1 << (a.bits - 1)) - 1 : (1 << a.bits) - 1;
}

// Gate non-linearities as a fixed sequence of IEEE fp32 operations (round-to-nearest add,
// multiply, fused multiply-add), so that the code a cell output quantizes to does
// not depend on a math library:
//   2^t for |t| <= 125: n = rne(t) by adding and subtracting 1.5 * 2^23; r = t - n (exact,
//   |r| <= 1/2); p = 1 + r (c1 + r (c2 + ... + r c6)) by Horner's rule with fused multiply-adds,
//   c1..c6 fixed constants (interpolation of (2^r - 1)/r at the six Chebyshev nodes of
//   [-1/2, 1/2], relative error below 1e-8); times 2^n by adding n to the exponent field.
__device__ __forceinline__ float exp2_fixed(float t) {
  const float nf = __fadd_rn(t, 12582912.0f);
  const float r = __fsub_rn(t, __fsub_rn(nf, 12582912.0f));
  float p = 0x1.44138ap-13f;
  p = __fmaf_rn(p, r, 0x1.5f0890p-10f);
  p = __fmaf_rn(p, r, 0x1.3b2a54p-7f);
  p = __fmaf_rn(p, r, 0x1.c6af6cp-5f);
  p = __fmaf_rn(p, r, 0x1.ebfbe0p-3f);
  p = __fmaf_rn(p, r, 0x1.62e430p-1f);
  p = __fmaf_rn(p, r, 1.0f);
  return __uint_as_float(__float_as_uint(p) + (__float_as_uint(nf) << 23));
}
//   1/d for d in [1, 2^118): seed from the exponent field (0x7EF311C7 - bits(d), within 12.5 %
//   of 1/d), then four Newton steps e = fma(-d, y, 1), y = fma(y, e, y).  No special cases, no
//   branch, no table: the same bits everywhere (the hardware reciprocal is rounded correctly but
//   costs a conditional slow path per call, which keeps the four cells of an epilogue thread
//   from being scheduled together: measured 20 % of the cell update).
__device__ __forceinline__ float rcp_fixed(float d) {
  float y = __uint_as_float(0x7EF311C7u - __float_as_uint(d));
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float e = __fmaf_rn(-d, y, 1.0f);
    y = __fmaf_rn(y, e, y);
  }
  return y;
}
constexpr float NEG_LOG2E = -0x1.715476p+0f;        // -log2(e) rounded to fp32
constexpr float NEG_2LOG2E = -0x1.715476p+1f;       // twice that
//   sigmoid(x) = 1 / (1 + 2^(-log2(e) x)), x clamped to [-40, 40]
__device__ __forceinline__ float sigmoid_fixed(float x) {
  x = fminf(fmaxf(x, -40.0f), 40.0f);
  return rcp_fixed(__fadd_rn(1.0f, exp2_fixed(__fmul_rn(x, NEG_LOG2E))));
}
//   tanh(x) = sign(x) (1 - e) * (1 / (1 + e)), e = 2^(-2 log2(e) min(|x|, 40))
__device__ __forceinline__ float tanh_fixed(float x) {
  const float e = exp2_fixed(__fmul_rn(fminf(fabsf(x), 40.0f), NEG_2LOG2E));
  return copysignf(__fmul_rn(__fsub_rn(1.0f, e), rcp_fixed(__fadd_rn(1.0f, e))), x);
}

// LSTM cell update with two reciprocals:
//   ei, ef, eo = 2^(-log2(e) pre), pre clamped to [-40, 40]; eg, ec = 2^(-2 log2(e) min(|.|, 40));
//   R = 1 / (((1 + ei)(1 + eg))(1 + ef));  i*g = sign(g) ((1 - eg)(1 + ef)) R;  f = ((1 + ei)(1 + eg)) R;
//   c = fma(f, c_prev, i*g);  h = sign(c) (1 - ec) * (1 / ((1 + eo)(1 + ec))).
// Every factor lies in [1, 2^58], so no product overflows.
__device__ __forceinline__ void cell_fixed(float pi, float pf, float pg, float po, float c_prev,
                                           float& c, float& h) {
  const float ei = exp2_fixed(__fmul_rn(fminf(fmaxf(pi, -40.0f), 40.0f), NEG_LOG2E));
  const float ef = exp2_fixed(__fmul_rn(fminf(fmaxf(pf, -40.0f), 40.0f), NEG_LOG2E));
  const float eo = exp2_fixed(__fmul_rn(fminf(fmaxf(po, -40.0f), 40.0f), NEG_LOG2E));
  const float eg = exp2_fixed(__fmul_rn(fminf(fabsf(pg), 40.0f), NEG_2LOG2E));
  const float ag = __fmul_rn(__fadd_rn(1.0f, ei), __fadd_rn(1.0f, eg));
  const float F = __fadd_rn(1.0f, ef);
  const float R = rcp_fixed(__fmul_rn(ag, F));
  const float ig = copysignf(__fmul_rn(__fmul_rn(__fsub_rn(1.0f, eg), F), R), pg);
  const float f = __fmul_rn(ag, R);
  c = __fmaf_rn(f, c_prev, ig);
  const float ec = exp2_fixed(__fmul_rn(fminf(fabsf(c), 40.0f), NEG_2LOG2E));
  const float R2 = rcp_fixed(__fmul_rn(__fadd_rn(1.0f, eo), __fadd_rn(1.0f, ec)));
  h = copysignf(__fmul_rn(__fsub_rn(1.0f, ec), R2), c);
}

// The same cell update for two cells at once on the paired fp32 instructions (two IEEE fp32
// operations per instruction, each rounded like its scalar form): the same operations on the same
// operands as cell_fixed, so the same bits, in about two thirds of the issue slots.  Pairs: the
// input and forget gates of a cell, its output and candidate gates, and the two cells' new states.
__device__ __forceinline__ uint64_t pk2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t exp2_fixed2(uint64_t t) {
  const uint64_t K = pk2(12582912.0f, 12582912.0f);
  const uint64_t nf = add2(t, K);
  const uint64_t r = sub2(t, sub2(nf, K));
  uint64_t p = pk2(0x1.44138ap-13f, 0x1.44138ap-13f);
  p = fma2(p, r, pk2(0x1.5f0890p-10f, 0x1.5f0890p-10f));
  p = fma2(p, r, pk2(0x1.3b2a54p-7f, 0x1.3b2a54p-7f));
  p = fma2(p, r, pk2(0x1.c6af6cp-5f, 0x1.c6af6cp-5f));
  p = fma2(p, r, pk2(0x1.ebfbe0p-3f, 0x1.ebfbe0p-3f));
  p = fma2(p, r, pk2(0x1.62e430p-1f, 0x1.62e430p-1f));
  p = fma2(p, r, pk2(1.0f, 1.0f));
  float p0, p1, n0, n1;
  upk2(p, p0, p1);
  upk2(nf, n0, n1);
  return pk2(__uint_as_float(__float_as_uint(p0) + (__float_as_uint(n0) << 23)),
             __uint_as_float(__float_as_uint(p1) + (__float_as_uint(n1) << 23)));
}
__device__ __forceinline__ uint64_t rcp_fixed2(uint64_t d) {
  float d0, d1;
  upk2(d, d0, d1);
  uint64_t y = pk2(__uint_as_float(0x7EF311C7u - __float_as_uint(d0)), __uint_as_float(0x7EF311C7u - __float_as_uint(d1)));
  const uint64_t nd = pk2(-d0, -d1), one = pk2(1.0f, 1.0f);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint64_t e = fma2(nd, y, one);
    y = fma2(y, e, y);
  }
  return y;
}
// pa, pb: pre-activations (i, f, g, o) of cells a and b
__device__ __forceinline__ void cell_fixed2(float pia, float pfa, float pga, float poa, float cpa,
                                            float pib, float pfb, float pgb, float pob, float cpb,
                                            float& ca, float& ha, float& cb, float& hb) {
  const uint64_t one = pk2(1.0f, 1.0f);
  // The arguments of 2^t are rounded products: scalar multiplications, because the assembler may
  // contract a paired multiplication with the paired addition that follows it inside exp2_fixed2
  // into one fused operation (observed), which skips that rounding.
  const uint64_t e_if_a = exp2_fixed2(pk2(__fmul_rn(fminf(fmaxf(pia, -40.0f), 40.0f), NEG_LOG2E),
                                          __fmul_rn(fminf(fmaxf(pfa, -40.0f), 40.0f), NEG_LOG2E)));
  const uint64_t e_og_a = exp2_fixed2(pk2(__fmul_rn(fminf(fmaxf(poa, -40.0f), 40.0f), NEG_LOG2E),
                                          __fmul_rn(fminf(fabsf(pga), 40.0f), NEG_2LOG2E)));
  const uint64_t e_if_b = exp2_fixed2(pk2(__fmul_rn(fminf(fmaxf(pib, -40.0f), 40.0f), NEG_LOG2E),
                                          __fmul_rn(fminf(fmaxf(pfb, -40.0f), 40.0f), NEG_LOG2E)));
  const uint64_t e_og_b = exp2_fixed2(pk2(__fmul_rn(fminf(fmaxf(pob, -40.0f), 40.0f), NEG_LOG2E),
                                          __fmul_rn(fminf(fabsf(pgb), 40.0f), NEG_2LOG2E)));
  float Ia, Fa, Oa, Ga, Ib, Fb, Ob, Gb, ta, ma, tb, mb;
  upk2(add2(one, e_if_a), Ia, Fa);      // 1 + ei, 1 + ef
  upk2(add2(one, e_og_a), Oa, Ga);      // 1 + eo, 1 + eg
  upk2(sub2(one, e_og_a), ta, ma);      // (unused), 1 - eg
  upk2(add2(one, e_if_b), Ib, Fb);
  upk2(add2(one, e_og_b), Ob, Gb);
  upk2(sub2(one, e_og_b), tb, mb);
  (void)ta;
  (void)tb;
  const float aga = __fmul_rn(Ia, Ga), agb = __fmul_rn(Ib, Gb);
  float Ra, Rb;
  upk2(rcp_fixed2(mul2(pk2(aga, agb), pk2(Fa, Fb))), Ra, Rb);
  const float iga = copysignf(__fmul_rn(__fmul_rn(ma, Fa), Ra), pga);
  const float igb = copysignf(__fmul_rn(__fmul_rn(mb, Fb), Rb), pgb);
  ca = __fmaf_rn(__fmul_rn(aga, Ra), cpa, iga);
  cb = __fmaf_rn(__fmul_rn(agb, Rb), cpb, igb);
  const uint64_t ec = exp2_fixed2(pk2(__fmul_rn(fminf(fabsf(ca), 40.0f), NEG_2LOG2E), __fmul_rn(fminf(fabsf(cb), 40.0f), NEG_2LOG2E)));
  const uint64_t R2 = rcp_fixed2(mul2(pk2(Oa, Ob), add2(one, ec)));
  float h0, h1;
  upk2(mul2(sub2(one, ec), R2), h0, h1);
  ha = copysignf(h0, ca);
  hb = copysignf(h1, cb);
}

// One cell on the paired instructions: the (input, forget) and (output, candidate) exponentials of the
// cell as pairs, the rest scalar; the same operations on the same operands as cell_fixed.
__device__ __forceinline__ void cell_fixed_p(float pi, float pf, float pg, float po, float c_prev, float& c, float& h) {
  const uint64_t one = pk2(1.0f, 1.0f);
  const uint64_t e_if = exp2_fixed2(pk2(__fmul_rn(fminf(fmaxf(pi, -40.0f), 40.0f), NEG_LOG2E),
                                        __fmul_rn(fminf(fmaxf(pf, -40.0f), 40.0f), NEG_LOG2E)));
  const uint64_t e_og = exp2_fixed2(pk2(__fmul_rn(fminf(fmaxf(po, -40.0f), 40.0f), NEG_LOG2E),
                                        __fmul_rn(fminf(fabsf(pg), 40.0f), NEG_2LOG2E)));
  float I, F, O, G, t, m;
  upk2(add2(one, e_if), I, F);
  upk2(add2(one, e_og), O, G);
  upk2(sub2(one, e_og), t, m);
  (void)t;
  const float ag = __fmul_rn(I, G);
  const float R = rcp_fixed(__fmul_rn(ag, F));
  const float ig = copysignf(__fmul_rn(__fmul_rn(m, F), R), pg);
  c = __fmaf_rn(__fmul_rn(ag, R), c_prev, ig);
  const float ec = exp2_fixed(__fmul_rn(fminf(fabsf(c), 40.0f), NEG_2LOG2E));
  const float R2 = rcp_fixed(__fmul_rn(O, __fadd_rn(1.0f, ec)));
  h = copysignf(__fmul_rn(__fsub_rn(1.0f, ec), R2), c);
}

// ---- argument blocks of the tile kernels -------------------------------------------
enum { EPI_I32 = 0, EPI_F32 = 1, EPI_QUANT = 2 };

struct GemmArgs {
  RowSrc x;                 // activation codes
  int32_t x_signed, x_zp, M;
  int32_t x_bits, w_bits;   // storage widths of the activation and weight codes
  const uint8_t* w;         // weight codes [J, k_pad]
  const float* w_scale;
  const float* bias;
  int32_t J, k_pad;
  float x_scale;
  void* out;                // EPI_I32: int32 [*, out_stride]; EPI_F32: float; EPI_QUANT: bytes
  long long out_stride;     // elements (I32/F32) or bytes (QUANT) between output rows
  const int32_t* out_idx;   // output row of x row m (nullptr = m; negative = skip)
  int32_t* dbg_acc;         // optional raw accumulators [M, J]
  q4_act out_act;           // EPI_QUANT
  const int32_t* n_active;  // optional device count: rows >= *n_active carry no work
};

struct LstmArgs {
  RowSrc x;                 // input codes (ignored when acc_pre is set)
  int32_t x_signed, x_zp, kx_pad;
  int32_t x_bits, wih_bits, whh_bits;   // storage widths: input codes, input weights, recurrent weights
  float x_scale;
  const float* x_scale_vec; // optional per-row input scale, indexed n % x_scale_mod
  int32_t x_scale_mod;
  const int32_t* acc_pre;   // optional precomputed input accumulators, row n at n*acc_pre_stride
  long long acc_pre_stride;
  RowSrc hin;               // previous cell-output codes
  const float* c_in;        // [*, H], indexed like hin
  const uint8_t* w_ih;
  const float* s_wih;
  const uint8_t* w_hh;
  const float* s_whh;
  const float* bias;
  int32_t H, N, kh_pad;
  q4_act hid_act, out_act;
  uint8_t* hq_out;          // recurrent codes, row stride hq_stride bytes, rows via out_idx
  long long hq_stride;
  const int32_t* out_idx;
  float* c_out;             // [*, H] rows via out_idx
  uint8_t* yq_out;          // optional second code (out_act), row n at n*yq_stride bytes
  long long yq_stride;
  float* h_f32;             // optional [N, H]
  int32_t* dbg_ih;          // optional, row n at n*dbg_stride
  int32_t* dbg_hh;
  long long dbg_stride;
  const int32_t* n_active;  // optional device count: rows >= *n_active carry no work
};
struct LstmArgs2 {
  LstmArgs d[2];
};

}  // namespace q4
