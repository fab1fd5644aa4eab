// CPU oracle for end-to-end 4-bit RNN-T inference with density-ratio LM fusion
// (arxiv 2206.07882).  TEST INFRASTRUCTURE ONLY: a plain, slow, single-purpose
// restatement of what the method computes, used by the tests, the smoke check
// and the timed CPU baseline.  It shares no code with the CUDA library and the
// product never calls it.
//
// Conventions
//   * integer codes are held one per int16 (activations) or int8 (weights);
//     integer accumulation is exact in int32;
//   * every floating-point value that is later quantized or carried as state
//     (de-quantized pre-activations, gates, cell state, cell output, linear
//     outputs, tanh(e*p)) is computed in fp32 by a fixed sequence of IEEE
//     operations (multiply, add, fused multiply-add, divide), including the
//     exponential behind sigmoid and tanh: a float decides an integer code
//     there, so the decision is taken in the precision the kernels use and
//     is reproducible bit for bit on any IEEE machine;
//   * the quantizer itself is fp32 by definition (one multiply by a stored
//     reciprocal, round-half-even, clamp);
//   * reductions whose order is free (log-softmax) and the hypothesis scores
//     of Eq. 1 are evaluated in double and rounded to float where stored;
//   * beside the fixed fp32 sequences stands a PLAIN path written from the
//     definitions alone (orc_lstm_step_plain, orc_joint_z_plain,
//     orc_linear_plain: the C library's exp and tanh in double, a value rounded
//     to fp32 only where the method stores or quantizes it).  It is what the
//     fixed sequences and the kernels are checked against under teacher
//     forcing: real values within 1e-5, codes equal except within 1e-3 code
//     units of a rounding boundary of Eq. 2, where they may differ by one.  A
//     change of the fixed sequences never touches the plain path;
//   * Section 3.4's quantizer-call counts are counted (g_quant_calls), under
//     both placements: Outer (orc_lstm_layer) and Inner (orc_lstm_layer_inner).
//
// Parity status: every function below is pinned by tests/test_oracle_*.py
// (hand tables, closed forms, brute force).  What no test can pin, because it
// needs trained weights and the NIST test sets, is recognition accuracy
// (Table 1): parity unpinned for WER, which nothing here computes.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

extern "C" {

// ---------------------------------------------------------------- quantizers
// Activation quantizer constants.  Eq. 2 / Eq. 3 with s = (a+ - a-)/(2^b - 1),
// z = -a-/s (rounded to an integer); the symmetric form (Section 3.1) has a
// single boundary, no zero point, and a signed code range.
struct OrcAct {
  float scale;
  float inv_scale;
  int32_t zero_point;
  int32_t bits;
  int32_t is_signed;
};

static inline float rne(float v) { return std::nearbyintf(v); }  // default mode: half to even

// Symmetric quantizer: s = alpha / (2^(b-1) - 1); codes in [-2^(b-1), 2^(b-1)-1].
void orc_act_symmetric(float alpha, int32_t bits, OrcAct* a) {
  const int32_t qmax = (1 << (bits - 1)) - 1;
  a->scale = alpha / (float)qmax;
  a->inv_scale = 1.0f / a->scale;
  a->zero_point = 0;
  a->bits = bits;
  a->is_signed = 1;
}

// Asymmetric quantizer, Eq. 2: s = (hi - lo)/(2^b - 1), z = round(-lo/s) in [0, 2^b-1].
void orc_act_asymmetric(float lo, float hi, int32_t bits, OrcAct* a) {
  const int32_t qmax = (1 << bits) - 1;
  a->scale = (hi - lo) / (float)qmax;
  a->inv_scale = 1.0f / a->scale;
  float z = rne(-lo / a->scale);
  z = std::fmin(std::fmax(z, 0.0f), (float)qmax);
  a->zero_point = (int32_t)z;
  a->bits = bits;
  a->is_signed = 0;
}

// MAX boundary (Section 3.1): the largest magnitude of the tensor; 1 if all zero.
float orc_absmax(const float* x, int64_t n) {
  float m = 0.0f;
  for (int64_t i = 0; i < n; ++i) m = std::fmax(m, std::fabs(x[i]));
  return m == 0.0f ? 1.0f : m;
}

static inline int32_t quantize_one(float x, const OrcAct& a) {
  const int32_t lo = a.is_signed ? -(1 << (a.bits - 1)) : 0;
  const int32_t hi = a.is_signed ? (1 << (a.bits - 1)) - 1 : (1 << a.bits) - 1;
  if (x != x) return std::min(std::max(a.zero_point, lo), hi);
  float r = rne(x * a.inv_scale);                       // Eq. 2: round(x / s)
  r = std::fmin(std::fmax(r, -1.0e9f), 1.0e9f);
  int32_t q = (int32_t)r + a.zero_point;                // + z
  return std::min(std::max(q, lo), hi);                 // clamp
}

// Number of activation-quantizer calls made so far: one call = the quantizer applied to one
// tensor handed to it (orc_quantize).  Section 3.4 counts these per time step and layer.
static std::atomic<int64_t> g_quant_calls{0};
void orc_quant_calls_reset() { g_quant_calls.store(0); }
int64_t orc_quant_calls() { return g_quant_calls.load(); }

// Eq. 2 on n values (one quantizer call).
void orc_quantize(const float* x, int64_t n, const OrcAct* a, int16_t* q) {
  g_quant_calls.fetch_add(1);
  for (int64_t i = 0; i < n; ++i) q[i] = (int16_t)quantize_one(x[i], *a);
}

// The network input [T, B, F] quantized frame by frame: one quantizer call per frame and
// sequence (the "T" of the T + T L calls of Section 3.4).
void orc_quantize_frames(const float* x, int64_t frames, int64_t F, const OrcAct* a, int16_t* q) {
  for (int64_t f = 0; f < frames; ++f) orc_quantize(x + f * F, F, a, q + f * F);
}

// Eq. 3: x_q = s (x_int - z).
void orc_dequantize(const int16_t* q, int64_t n, const OrcAct* a, float* x) {
  for (int64_t i = 0; i < n; ++i) x[i] = a->scale * (float)((int32_t)q[i] - a->zero_point);
}

// Per-row symmetric weight quantization with a given per-row scale:
// q = clamp(round(w / s_row)).
void orc_quantize_weights(const float* w, int64_t rows, int64_t k, const float* row_scale,
                          int32_t bits, int8_t* q) {
  for (int64_t r = 0; r < rows; ++r) {
    OrcAct a;
    a.scale = row_scale[r];
    a.inv_scale = 1.0f / a.scale;
    a.zero_point = 0;
    a.bits = bits;
    a.is_signed = 1;
    for (int64_t i = 0; i < k; ++i) q[r * k + i] = (int8_t)quantize_one(w[r * k + i], a);
  }
}

// Storage format for 4-bit codes: two per byte, element 2i in bits 0-3, element
// 2i+1 in bits 4-7, two's complement when signed; rows padded with zeros
// (signed) to k_pad elements.  `pad_code` fills the padding (the zero point for
// unsigned codes, so that padding contributes nothing after z is subtracted).
void orc_pack4(const int16_t* q, int64_t rows, int64_t k, int64_t k_pad, int32_t pad_code,
               uint8_t* out) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t i = 0; i < k_pad; i += 2) {
      int32_t lo = i < k ? q[r * k + i] : pad_code;
      int32_t hi = i + 1 < k ? q[r * k + i + 1] : pad_code;
      out[r * (k_pad / 2) + i / 2] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
    }
}

void orc_unpack4(const uint8_t* in, int64_t rows, int64_t k, int64_t k_pad, int32_t is_signed,
                 int16_t* q) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t i = 0; i < k; ++i) {
      int32_t v = (in[r * (k_pad / 2) + i / 2] >> ((i & 1) * 4)) & 0xF;
      if (is_signed && v >= 8) v -= 16;
      q[r * k + i] = (int16_t)v;
    }
}

// Storage format for 2-bit weight codes (the 2-bit weight rows of Table 1): four per byte,
// element 4i+j in bits 2j, 2j+1, two's complement (codes -2..1), rows padded with zeros.
void orc_pack2(const int16_t* q, int64_t rows, int64_t k, int64_t k_pad, uint8_t* out) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t i = 0; i < k_pad; i += 4) {
      uint32_t b = 0;
      for (int64_t j = 0; j < 4; ++j) {
        const int32_t v = i + j < k ? q[r * k + i + j] : 0;
        b |= (uint32_t)(v & 0x3) << (2 * j);
      }
      out[r * (k_pad / 4) + i / 4] = (uint8_t)b;
    }
}

void orc_unpack2(const uint8_t* in, int64_t rows, int64_t k, int64_t k_pad, int16_t* q) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t i = 0; i < k; ++i) {
      int32_t v = (in[r * (k_pad / 4) + i / 4] >> ((i & 3) * 2)) & 0x3;
      if (v >= 2) v -= 4;
      q[r * k + i] = (int16_t)v;
    }
}

// ------------------------------------------------------------ integer MACs
// acc[m, j] = sum_k W[j,k] * (xq[m,k] - z).  Weights are symmetric (no zero point).
void orc_int_matmul(const int8_t* w, int32_t J, int32_t K, const int16_t* xq, int32_t zero_point,
                    int32_t M, int32_t* acc) {
  for (int32_t m = 0; m < M; ++m)
    for (int32_t j = 0; j < J; ++j) {
      int32_t s = 0;
      for (int32_t k = 0; k < K; ++k)
        s += (int32_t)w[(int64_t)j * K + k] * ((int32_t)xq[(int64_t)m * K + k] - zero_point);
      acc[(int64_t)m * J + j] = s;
    }
}

struct OrcLinear {
  const int8_t* w;       // [J, K] integer codes
  const float* s_w;      // [J]
  const float* bias;     // [J] or null
  int32_t J, K;
};

// Quantized linear layer (Section 3.2: weight and input quantized, bias not):
// out[m,j] = fma(acc[m,j], s_x * s_w[j], bias[j]) in fp32.
void orc_linear(const OrcLinear* L, const int16_t* xq, const OrcAct* x_act, int32_t M, float* out,
                int32_t* acc_out) {
  std::vector<int32_t> acc((size_t)M * L->J);
  orc_int_matmul(L->w, L->J, L->K, xq, x_act->zero_point, M, acc.data());
  for (int32_t m = 0; m < M; ++m)
    for (int32_t j = 0; j < L->J; ++j) {
      const float sc = x_act->scale * L->s_w[j];
      out[(size_t)m * L->J + j] =
          std::fmaf((float)acc[(size_t)m * L->J + j], sc, L->bias ? L->bias[j] : 0.0f);
    }
  if (acc_out) std::memcpy(acc_out, acc.data(), acc.size() * sizeof(int32_t));
}


// ------------------------------------------------- fp32 activation functions
// 2^t for |t| <= 125 as a fixed sequence of fp32 operations: n = rne(t), obtained by adding
// and subtracting 1.5 * 2^23; r = t - n (exact, |r| <= 1/2); p = 1 + r (c1 + r (c2 + ... +
// r c6)) by Horner's rule with fused multiply-adds, c1..c6 being the interpolant of
// (2^r - 1)/r at the six Chebyshev nodes of [-1/2, 1/2] rounded to fp32; scaling by 2^n
// through the exponent field.
static inline float f32_from_bits(uint32_t b) {
  float f;
  std::memcpy(&f, &b, 4);
  return f;
}
static inline uint32_t bits_from_f32(float f) {
  uint32_t b;
  std::memcpy(&b, &f, 4);
  return b;
}
float orc_exp2(float t) {
  const float nf = t + 12582912.0f;
  const float n = nf - 12582912.0f;
  const float r = t - n;
  float p = 0x1.44138ap-13f;
  p = std::fmaf(p, r, 0x1.5f0890p-10f);
  p = std::fmaf(p, r, 0x1.3b2a54p-7f);
  p = std::fmaf(p, r, 0x1.c6af6cp-5f);
  p = std::fmaf(p, r, 0x1.ebfbe0p-3f);
  p = std::fmaf(p, r, 0x1.62e430p-1f);
  p = std::fmaf(p, r, 1.0f);
  return f32_from_bits(bits_from_f32(p) + (bits_from_f32(nf) << 23));
}
// 1/d for d in [1, 2^118) without a division: seed from the exponent field (0x7EF311C7 -
// bits(d), within 12.5 % of 1/d), then four Newton steps e = fma(-d, y, 1), y = fma(y, e, y).
static inline float orc_rcp(float d) {
  float y = f32_from_bits(0x7EF311C7u - bits_from_f32(d));
  for (int i = 0; i < 4; ++i) {
    const float e = std::fmaf(-d, y, 1.0f);
    y = std::fmaf(y, e, y);
  }
  return y;
}
static const float kNegLog2e = -0x1.715476p+0f;   // -log2(e) rounded to fp32
// sigmoid(x) = rcp(1 + 2^(-log2(e) x)), argument clamped to [-40, 40].
float orc_sigmoid(float x) {
  x = std::fmin(std::fmax(x, -40.0f), 40.0f);
  return orc_rcp(1.0f + orc_exp2(x * kNegLog2e));
}
// tanh(x) = sign(x) * (1 - e) * rcp(1 + e), e = 2^(-2 log2(e) min(|x|, 40)).
float orc_tanh(float x) {
  const float e = orc_exp2(std::fmin(std::fabs(x), 40.0f) * (2.0f * kNegLog2e));
  const float rcp = orc_rcp(1.0f + e);
  return std::copysign((1.0f - e) * rcp, x);
}
// LSTM cell update in fp32 with two reciprocals (orc_rcp, written 1 / (.) below).  With ei = 2^(-log2(e) i_pre) and likewise
// ef, eo (arguments clamped to [-40, 40]), eg = 2^(-2 log2(e) min(|g_pre|, 40)):
//   R   = 1 / (((1 + ei)(1 + eg))(1 + ef)),
//   i*g = sign(g) ((1 - eg)(1 + ef)) R,     f = ((1 + ei)(1 + eg)) R,
//   c   = fma(f, c_prev, i*g),
//   h   = sign(c) (1 - ec) (1 / ((1 + eo)(1 + ec))),   ec = 2^(-2 log2(e) min(|c|, 40)).
// Mathematically this is sigmoid(i) tanh(g), sigmoid(f), sigmoid(o) tanh(c); every factor
// lies in [1, 2^58], so no product overflows.
void orc_cell(float pi, float pf, float pg, float po, float c_prev, float* c_out, float* h_out) {
  const float ei = orc_exp2(std::fmin(std::fmax(pi, -40.0f), 40.0f) * kNegLog2e);
  const float ef = orc_exp2(std::fmin(std::fmax(pf, -40.0f), 40.0f) * kNegLog2e);
  const float eo = orc_exp2(std::fmin(std::fmax(po, -40.0f), 40.0f) * kNegLog2e);
  const float eg = orc_exp2(std::fmin(std::fabs(pg), 40.0f) * (2.0f * kNegLog2e));
  const float ag = (1.0f + ei) * (1.0f + eg);
  const float F = 1.0f + ef;
  const float R = orc_rcp(ag * F);
  const float ig = std::copysign(((1.0f - eg) * F) * R, pg);
  const float f = ag * R;
  const float c = std::fmaf(f, c_prev, ig);
  const float ec = orc_exp2(std::fmin(std::fabs(c), 40.0f) * (2.0f * kNegLog2e));
  const float R2 = orc_rcp((1.0f + eo) * (1.0f + ec));
  *c_out = c;
  *h_out = std::copysign((1.0f - ec) * R2, c);
}
// orc_cell on arrays (for the tests that pin it to the textbook formulas).
void orc_cells(const float* pre_i, const float* pre_f, const float* pre_g, const float* pre_o,
               const float* c_prev, int64_t n, float* c_out, float* h_out) {
  for (int64_t i = 0; i < n; ++i) orc_cell(pre_i[i], pre_f[i], pre_g[i], pre_o[i], c_prev[i], c_out + i, h_out + i);
}
void orc_activations(const float* x, int64_t n, float* ex, float* sg, float* th) {
  for (int64_t i = 0; i < n; ++i) {
    if (ex) ex[i] = orc_exp2(x[i]);
    if (sg) sg[i] = orc_sigmoid(x[i]);
    if (th) th[i] = orc_tanh(x[i]);
  }
}

// ---------------------------------------------------------------- LSTM cell
static inline double sigmoid(double v) { return 1.0 / (1.0 + std::exp(-v)); }  // plain paths only

struct OrcLstm {
  const int8_t* w_ih;    // [4H, K], gate blocks in the order i, f, g, o
  const float* s_wih;    // [4H]
  const int8_t* w_hh;    // [4H, H]
  const float* s_whh;    // [4H]
  const float* bias;     // [4H] or null (not quantized)
  int32_t K, H;
};

// De-quantized pre-activations and cell update of ONE row, without the output quantizer.
static void lstm_row(const OrcLstm* L, const int16_t* xq, const OrcAct* x_act, float s_x,
                     const int16_t* hq_in, const float* c_in, const OrcAct* hid_act, float* c_out,
                     float* h_out, int32_t* a_ih, int32_t* a_hh, float* pre) {
  const int32_t H = L->H, K = L->K, G = 4 * H;
  orc_int_matmul(L->w_ih, G, K, xq, x_act->zero_point, 1, a_ih);
  orc_int_matmul(L->w_hh, G, H, hq_in, hid_act->zero_point, 1, a_hh);
  const float s_h = hid_act->scale;
  for (int32_t j = 0; j < G; ++j) {
    // de-quantize: each accumulator times (activation scale * row scale), plus bias
    float v = std::fmaf((float)a_ih[j], s_x * L->s_wih[j], L->bias ? L->bias[j] : 0.0f);
    pre[j] = std::fmaf((float)a_hh[j], s_h * L->s_whh[j], v);
  }
  for (int32_t u = 0; u < H; ++u)
    orc_cell(pre[u], pre[H + u], pre[2 * H + u], pre[3 * H + u], c_in[u], c_out + u, h_out + u);
}

// One time step for N independent rows.  Cell state is kept in floating point
// and never quantized; the cell output o * tanh(c) lies in [-1,1] and is
// quantized ONCE, at the cell output ("Outer" placement, Section 3.4), with
// hid_act.  Optional outputs (may be null): h (float cell output), acc_ih,
// acc_hh (int32 [N,4H]), gates (float [N,4H]: i, f, g, o after activation),
// x_scale_row ([N], overrides x_act->scale per row when not null).
void orc_lstm_step(const OrcLstm* L, const int16_t* xq, const OrcAct* x_act,
                   const float* x_scale_row, const int16_t* hq_in, const float* c_in,
                   const OrcAct* hid_act, int32_t N, int16_t* hq_out, float* c_out, float* h_out,
                   int32_t* acc_ih_out, int32_t* acc_hh_out, float* gates_out) {
  const int32_t H = L->H, K = L->K, G = 4 * H;
  std::vector<int32_t> a_ih(G), a_hh(G);
  std::vector<float> pre(G), h(H);
  for (int32_t n = 0; n < N; ++n) {
    lstm_row(L, xq + (int64_t)n * K, x_act, x_scale_row ? x_scale_row[n] : x_act->scale,
             hq_in + (int64_t)n * H, c_in + (int64_t)n * H, hid_act, c_out + (int64_t)n * H, h.data(),
             a_ih.data(), a_hh.data(), pre.data());
    orc_quantize(h.data(), H, hid_act, hq_out + (int64_t)n * H);   // the one call at the cell output
    if (h_out) std::memcpy(h_out + (int64_t)n * H, h.data(), H * sizeof(float));
    if (acc_ih_out) std::memcpy(acc_ih_out + (int64_t)n * G, a_ih.data(), G * sizeof(int32_t));
    if (acc_hh_out) std::memcpy(acc_hh_out + (int64_t)n * G, a_hh.data(), G * sizeof(int32_t));
    if (gates_out)   // diagnostic: the four gate activations by themselves
      for (int32_t j = 0; j < G; ++j)
        gates_out[(int64_t)n * G + j] = (j >= 2 * H && j < 3 * H) ? orc_tanh(pre[j]) : orc_sigmoid(pre[j]);
  }
}

// ------------------------------------------------ the plain (textbook) LSTM step
// The same step written from the definitions alone, independent of the fixed fp32 sequences
// above: de-quantization (Eq. 3), the gates from the C library's exp and tanh, the cell
// update c = f c' + i g and the output h = o tanh(c), all in double; a value is rounded to
// fp32 only where the method stores it (the cell state, Section 3.2) or hands it to the
// quantizer (the cell output, Section 3.4; the quantizer is an fp32 operation by definition).
// tie_out [N,H] (nullable) receives how far h / s lies from the nearest rounding boundary of
// Eq. 2, in code units (0 = exactly between two codes, 0.5 = on a code): a code computed with
// other floating-point arithmetic may differ by one only where this is tiny.
void orc_lstm_step_plain(const OrcLstm* L, const int16_t* xq, const OrcAct* x_act,
                         const float* x_scale_row, const int16_t* hq_in, const float* c_in,
                         const OrcAct* hid_act, int32_t N, int16_t* hq_out, float* c_out,
                         float* h_out, float* tie_out) {
  const int32_t H = L->H, K = L->K, G = 4 * H;
  std::vector<double> pre(G);
  std::vector<float> h(H);
  for (int32_t n = 0; n < N; ++n) {
    const double s_x = x_scale_row ? (double)x_scale_row[n] : (double)x_act->scale;
    const double s_h = (double)hid_act->scale;
    for (int32_t j = 0; j < G; ++j) {
      double v = L->bias ? (double)L->bias[j] : 0.0;
      for (int32_t k = 0; k < K; ++k)     // W x with W = s_w Wq and x = s_x (xq - z)   (Eq. 3)
        v += (double)L->s_wih[j] * (double)L->w_ih[(int64_t)j * K + k] *
             (s_x * (double)((int32_t)xq[(int64_t)n * K + k] - x_act->zero_point));
      for (int32_t k = 0; k < H; ++k)
        v += (double)L->s_whh[j] * (double)L->w_hh[(int64_t)j * H + k] *
             (s_h * (double)((int32_t)hq_in[(int64_t)n * H + k] - hid_act->zero_point));
      pre[j] = v;
    }
    for (int32_t u = 0; u < H; ++u) {
      const double i = sigmoid(pre[u]), f = sigmoid(pre[H + u]);
      const double g = std::tanh(pre[2 * H + u]), o = sigmoid(pre[3 * H + u]);
      const float c = (float)(f * (double)c_in[(int64_t)n * H + u] + i * g);   // stored: fp32
      const double hd = o * std::tanh((double)c);
      h[u] = (float)hd;
      c_out[(int64_t)n * H + u] = c;
      if (tie_out) {
        const double t = hd * (double)hid_act->inv_scale;
        tie_out[(int64_t)n * H + u] = (float)std::fabs((t - std::floor(t)) - 0.5);
      }
    }
    orc_quantize(h.data(), H, hid_act, hq_out + (int64_t)n * H);
    if (h_out) std::memcpy(h_out + (int64_t)n * H, h.data(), H * sizeof(float));
  }
}

// A uni- or bidirectional layer over time-major input xq [T, B, K].
// Direction 1 runs t = T-1 .. 0 with its own weights; the output at t is the
// concatenation [fwd(t) | bwd(t)].  yq [T,B,dirs*H] holds the codes handed to
// the next layer (out_act); when out_act differs from hid_act (a precision
// change between layers) both codes are made from the same float h (a second
// quantizer call).  Optional: h_f [T,B,dirs*H]; hq_hid [T,B,dirs*H] (recurrent
// codes); c_n [dirs,B,H]; acc_ih/acc_hh [T,B,dirs,4H].
static void layer_one_sequence(const OrcLstm* L, int32_t dirs, const int16_t* xq,
                               const OrcAct* x_act, const float* x_scale_b, int32_t T, int32_t B,
                               int32_t b, const OrcAct* hid_act, const OrcAct* out_act,
                               int16_t* yq, int16_t* hq_hid, float* h_f, float* c_n,
                               int32_t* acc_ih, int32_t* acc_hh) {
  for (int32_t d = 0; d < dirs; ++d) {
    const int32_t H = L[d].H, K = L[d].K, G = 4 * H, OH = dirs * H;
    std::vector<int16_t> hq(H, 0), hq2(H), yo(H);
    std::vector<float> c(H, 0.0f), c2(H), h(H);
    const bool same = out_act->bits == hid_act->bits && out_act->scale == hid_act->scale;
    for (int32_t s = 0; s < T; ++s) {
      const int32_t t = d == 0 ? s : T - 1 - s;
      const int64_t row = (int64_t)t * B + b;
      orc_lstm_step(&L[d], xq + row * K, x_act, x_scale_b ? x_scale_b + b : nullptr, hq.data(),
                    c.data(), hid_act, 1, hq2.data(), c2.data(), h.data(),
                    acc_ih ? acc_ih + (row * dirs + d) * G : nullptr,
                    acc_hh ? acc_hh + (row * dirs + d) * G : nullptr, nullptr);
      hq.swap(hq2);
      c.swap(c2);
      if (!same) orc_quantize(h.data(), H, out_act, yo.data());
      for (int32_t u = 0; u < H; ++u) {
        const int64_t o = row * OH + (int64_t)d * H + u;
        yq[o] = same ? hq[u] : yo[u];
        if (hq_hid) hq_hid[o] = hq[u];
        if (h_f) h_f[o] = h[u];
      }
    }
    if (c_n) std::memcpy(c_n + ((int64_t)d * B + b) * H, c.data(), H * sizeof(float));
  }
}

void orc_lstm_layer(const OrcLstm* L, int32_t dirs, const int16_t* xq, const OrcAct* x_act,
                    const float* x_scale_b, int32_t T, int32_t B, const OrcAct* hid_act,
                    const OrcAct* out_act, int16_t* yq, int16_t* hq_hid, float* h_f, float* c_n,
                    int32_t* acc_ih, int32_t* acc_hh, int32_t n_threads) {
  n_threads = std::max(1, std::min(n_threads, B));
  std::vector<std::thread> pool;
  for (int32_t w = 0; w < n_threads; ++w)
    pool.emplace_back([=]() {
      for (int32_t b = w; b < B; b += n_threads)
        layer_one_sequence(L, dirs, xq, x_act, x_scale_b, T, B, b, hid_act, out_act, yq, hq_hid,
                           h_f, c_n, acc_ih, acc_hh);
    });
  for (auto& th : pool) th.join();
}

// The same layer under "Inner" placement of the activation quantizers (Section 3.4, the
// placement the paper rejects): nothing is quantized at a cell's output; instead every cell
// quantizes both of its inputs on entry, x_t with x_act and s_{t-1} with hid_act: two calls
// per cell and time step, 2 T L in a network of L cells.  Input x [T,B,K] and output h
// [T,B,dirs*H] are real-valued.  When x_act is the quantizer the producing layer would have
// applied at its output, the result equals that of the Outer placement (same codes reach the
// same integer MACs); only the number of quantizer calls differs.
void orc_lstm_layer_inner(const OrcLstm* L, int32_t dirs, const float* x, const OrcAct* x_act,
                          int32_t T, int32_t B, const OrcAct* hid_act, float* h_out) {
  for (int32_t b = 0; b < B; ++b)
    for (int32_t d = 0; d < dirs; ++d) {
      const int32_t H = L[d].H, K = L[d].K, G = 4 * H, OH = dirs * H;
      std::vector<int16_t> xq(K), hq(H);
      std::vector<float> c(H, 0.0f), c2(H), h(H, 0.0f), h2(H), pre(G);
      std::vector<int32_t> a_ih(G), a_hh(G);
      for (int32_t s = 0; s < T; ++s) {
        const int32_t t = d == 0 ? s : T - 1 - s;
        const int64_t row = (int64_t)t * B + b;
        orc_quantize(x + row * K, K, x_act, xq.data());       // x_t on entry
        orc_quantize(h.data(), H, hid_act, hq.data());         // s_{t-1} on entry
        lstm_row(&L[d], xq.data(), x_act, x_act->scale, hq.data(), c.data(), hid_act, c2.data(),
                 h2.data(), a_ih.data(), a_hh.data(), pre.data());
        c.swap(c2);
        h.swap(h2);
        std::memcpy(h_out + row * OH + (int64_t)d * H, h.data(), H * sizeof(float));
      }
    }
}

// Full-precision counterpart of the same layer: W = s_w * Wq as real numbers,
// no activation quantizer anywhere.  x [T,B,K] float, out h [T,B,dirs*H].
void orc_lstm_layer_fp32(const OrcLstm* L, int32_t dirs, const float* x, int32_t T, int32_t B,
                         float* h_out) {
  for (int32_t d = 0; d < dirs; ++d) {
    const int32_t H = L[d].H, K = L[d].K, G = 4 * H, OH = dirs * H;
    for (int32_t b = 0; b < B; ++b) {
      std::vector<double> h(H, 0.0), c(H, 0.0), act(G);
      for (int32_t s = 0; s < T; ++s) {
        const int32_t t = d == 0 ? s : T - 1 - s;
        const float* xr = x + ((int64_t)t * B + b) * K;
        for (int32_t j = 0; j < G; ++j) {
          double pre = L[d].bias ? (double)L[d].bias[j] : 0.0;
          for (int32_t k = 0; k < K; ++k)
            pre += (double)L[d].s_wih[j] * (double)L[d].w_ih[(int64_t)j * K + k] * (double)xr[k];
          for (int32_t k = 0; k < H; ++k)
            pre += (double)L[d].s_whh[j] * (double)L[d].w_hh[(int64_t)j * H + k] * h[k];
          act[j] = (j >= 2 * H && j < 3 * H) ? std::tanh(pre) : sigmoid(pre);
        }
        for (int32_t u = 0; u < H; ++u) {
          c[u] = act[H + u] * c[u] + act[u] * act[2 * H + u];
          h[u] = act[3 * H + u] * std::tanh(c[u]);
          h_out[((int64_t)t * B + b) * OH + (int64_t)d * H + u] = (float)h[u];
        }
      }
    }
  }
}

// -------------------------------------------------------------- softmax, joint
// lp = logits - max - log(sum(exp(logits - max))), evaluated in double.
void orc_log_softmax(const float* logits, int32_t M, int32_t V, float* lp) {
  for (int32_t m = 0; m < M; ++m) {
    const float* z = logits + (int64_t)m * V;
    double mx = z[0];
    for (int32_t v = 1; v < V; ++v) mx = std::max(mx, (double)z[v]);
    double s = 0.0;
    for (int32_t v = 0; v < V; ++v) s += std::exp((double)z[v] - mx);
    const double lse = mx + std::log(s);
    for (int32_t v = 0; v < V; ++v) lp[(int64_t)m * V + v] = (float)((double)z[v] - lse);
  }
}

struct OrcJoint {
  OrcAct z_act;      // quantizer of tanh(e * p): symmetric, boundary 1
  OrcLinear out;     // D -> V
};

// Joint network (Section 2): encoder and prediction representations are
// combined multiplicatively, z = tanh(e .* p), quantized, passed through the
// output layer and a log-softmax.  e [N,D], p [N,D] float.
void orc_joint(const OrcJoint* Jn, const float* e, const float* p, int32_t N, float* logp,
               int16_t* zq_out, int32_t* acc_out) {
  const int32_t D = Jn->out.K, V = Jn->out.J;
  std::vector<float> z((size_t)N * D), logits((size_t)N * V);
  std::vector<int16_t> zq((size_t)N * D);
  for (int64_t i = 0; i < (int64_t)N * D; ++i) z[i] = orc_tanh(e[i] * p[i]);
  orc_quantize(z.data(), (int64_t)N * D, &Jn->z_act, zq.data());
  orc_linear(&Jn->out, zq.data(), &Jn->z_act, N, logits.data(), acc_out);
  orc_log_softmax(logits.data(), N, V, logp);
  if (zq_out) std::memcpy(zq_out, zq.data(), zq.size() * sizeof(int16_t));
}

// Plain counterparts for the joint network's real-valued stages (definitions only, double):
// z = tanh(e p) rounded to fp32 for the quantizer, with the distance of z / s from the nearest
// rounding boundary (see orc_lstm_step_plain), and a linear layer W x + b with W = s_w Wq,
// x = s (xq - z) (Eq. 3).
void orc_joint_z_plain(const float* e, const float* p, int64_t n, const OrcAct* z_act, int16_t* zq,
                       float* tie_out) {
  std::vector<float> z(n);
  for (int64_t i = 0; i < n; ++i) {
    const double zd = std::tanh((double)e[i] * (double)p[i]);
    z[i] = (float)zd;
    if (tie_out) {
      const double t = zd * (double)z_act->inv_scale;
      tie_out[i] = (float)std::fabs((t - std::floor(t)) - 0.5);
    }
  }
  orc_quantize(z.data(), n, z_act, zq);
}
void orc_linear_plain(const OrcLinear* L, const int16_t* xq, const OrcAct* x_act, int32_t M,
                      double* out) {
  for (int32_t m = 0; m < M; ++m)
    for (int32_t j = 0; j < L->J; ++j) {
      double v = L->bias ? (double)L->bias[j] : 0.0;
      for (int32_t k = 0; k < L->K; ++k)
        v += (double)L->s_w[j] * (double)L->w[(int64_t)j * L->K + k] *
             ((double)x_act->scale * (double)((int32_t)xq[(int64_t)m * L->K + k] - x_act->zero_point));
      out[(int64_t)m * L->J + j] = v;
    }
}

// ------------------------------------------------ prediction network and LMs
struct OrcPred {
  const float* emb;   // [V, E]
  int32_t V, E;
  OrcAct emb_act;     // input quantizer of the LSTM (symmetric FIX)
  OrcLstm lstm;
  OrcAct hid_act;
  OrcLinear proj;     // Hp -> D
};

struct OrcLm {
  const float* emb;   // [V, E]
  int32_t V, E;
  OrcAct emb_act;     // learned-boundary input quantizer (asymmetric constants)
  int32_t n_layers;
  OrcLstm lstm[2];
  OrcAct hid_act[2];
  OrcLinear bott;     // H -> D
  OrcAct bott_act;    // learned-boundary quantizer of the bottleneck output
  OrcLinear out;      // D -> V
};

struct PredState {
  std::vector<int16_t> hq;
  std::vector<float> c, p;
};
struct LmState {
  std::vector<int16_t> hq[2];
  std::vector<float> c[2], lp;
};

static void pred_init(const OrcPred& P, PredState& s) {
  s.hq.assign(P.lstm.H, 0);
  s.c.assign(P.lstm.H, 0.0f);
  s.p.assign(P.proj.J, 0.0f);
}
static void lm_init(const OrcLm& M, LmState& s) {
  for (int l = 0; l < M.n_layers; ++l) {
    s.hq[l].assign(M.lstm[l].H, 0);
    s.c[l].assign(M.lstm[l].H, 0.0f);
  }
  s.lp.assign(M.out.J, 0.0f);
}

// Feed one symbol: embedding row -> quantize -> LSTM step -> linear to D.
static void pred_advance(const OrcPred& P, int32_t token, PredState& s) {
  std::vector<int16_t> xq(P.E), hq(P.lstm.H);
  std::vector<float> c(P.lstm.H);
  orc_quantize(P.emb + (int64_t)token * P.E, P.E, &P.emb_act, xq.data());
  orc_lstm_step(&P.lstm, xq.data(), &P.emb_act, nullptr, s.hq.data(), s.c.data(), &P.hid_act, 1,
                hq.data(), c.data(), nullptr, nullptr, nullptr, nullptr);
  s.hq.swap(hq);
  s.c.swap(c);
  orc_linear(&P.proj, s.hq.data(), &P.hid_act, 1, s.p.data(), nullptr);
}

// Feed one symbol to an LM: embedding -> LSTM layers (each cell output quantized
// once and used both by the next layer and the next step) -> bottleneck ->
// quantize -> output layer -> log-softmax over all V entries.
static void lm_advance(const OrcLm& M, int32_t token, LmState& s) {
  std::vector<int16_t> xq(M.E);
  orc_quantize(M.emb + (int64_t)token * M.E, M.E, &M.emb_act, xq.data());
  const int16_t* in = xq.data();
  const OrcAct* in_act = &M.emb_act;
  for (int l = 0; l < M.n_layers; ++l) {
    std::vector<int16_t> hq(M.lstm[l].H);
    std::vector<float> c(M.lstm[l].H);
    orc_lstm_step(&M.lstm[l], in, in_act, nullptr, s.hq[l].data(), s.c[l].data(), &M.hid_act[l], 1,
                  hq.data(), c.data(), nullptr, nullptr, nullptr, nullptr);
    s.hq[l].swap(hq);
    s.c[l].swap(c);
    in = s.hq[l].data();
    in_act = &M.hid_act[l];
  }
  std::vector<float> bo(M.bott.J), logits(M.out.J);
  std::vector<int16_t> bq(M.bott.J);
  orc_linear(&M.bott, in, in_act, 1, bo.data(), nullptr);
  orc_quantize(bo.data(), M.bott.J, &M.bott_act, bq.data());
  orc_linear(&M.out, bq.data(), &M.bott_act, 1, logits.data(), nullptr);
  orc_log_softmax(logits.data(), 1, M.out.J, s.lp.data());
}

// Teacher-forced prediction network + joint over label sequences:
// row n consumes tokens[n, 0..S-1] (tokens[n,0] is the start symbol), and at
// step s is scored against e[frame_idx[n*S+s]].  logp [N,S,V].  Optional dumps
// for per-step comparison: hq [N,S,Hp], c [N,S,Hp], p [N,S,D].
void orc_pred_joint_forced(const OrcPred* P, const OrcJoint* Jn, const float* e,
                           const int32_t* frame_idx, const int32_t* tokens, int32_t N, int32_t S,
                           float* logp, int16_t* hq_out, float* c_out, float* p_out,
                           int32_t n_threads) {
  const int32_t D = P->proj.J, V = Jn->out.J, Hp = P->lstm.H;
  n_threads = std::max(1, std::min(n_threads, N));
  std::vector<std::thread> pool;
  for (int32_t w = 0; w < n_threads; ++w)
    pool.emplace_back([=]() {
      for (int32_t n = w; n < N; n += n_threads) {
        PredState st;
        pred_init(*P, st);
        for (int32_t s = 0; s < S; ++s) {
          const int64_t r = (int64_t)n * S + s;
          pred_advance(*P, tokens[r], st);
          orc_joint(Jn, e + (int64_t)frame_idx[r] * D, st.p.data(), 1, logp + r * V, nullptr,
                    nullptr);
          if (hq_out) std::memcpy(hq_out + r * Hp, st.hq.data(), Hp * sizeof(int16_t));
          if (c_out) std::memcpy(c_out + r * Hp, st.c.data(), Hp * sizeof(float));
          if (p_out) std::memcpy(p_out + r * D, st.p.data(), D * sizeof(float));
        }
      }
    });
  for (auto& th : pool) th.join();
}

// LM log-probabilities along forced token sequences: lp [N,S,V].
void orc_lm_forced(const OrcLm* M, const int32_t* tokens, int32_t N, int32_t S, float* lp,
                   int32_t n_threads) {
  const int32_t V = M->out.J;
  n_threads = std::max(1, std::min(n_threads, N));
  std::vector<std::thread> pool;
  for (int32_t w = 0; w < n_threads; ++w)
    pool.emplace_back([=]() {
      for (int32_t n = w; n < N; n += n_threads) {
        LmState st;
        lm_init(*M, st);
        for (int32_t s = 0; s < S; ++s) {
          lm_advance(*M, tokens[(int64_t)n * S + s], st);
          std::memcpy(lp + ((int64_t)n * S + s) * V, st.lp.data(), V * sizeof(float));
        }
      }
    });
  for (auto& th : pool) th.join();
}

// ------------------------------------------------------------- beam search
struct OrcDecoder {
  OrcPred pred;
  OrcJoint joint;
  OrcLm src, tgt;
  float lambda_t, lambda_s, rho;   // Eq. 1: mu (external LM), lambda (source LM), rho (reward)
  int32_t W, U_max;
};

struct Hyp {
  std::vector<int32_t> y;
  int32_t t;
  float S;
  PredState pred;
  LmState src, tgt;
};

struct Cand {
  float S;
  int32_t parent, token;   // token 0 = blank
  bool dead;
};

static inline bool ranks_before(const Cand& a, const Cand& b) {
  if (a.S != b.S) return a.S > b.S;
  if (a.parent != b.parent) return a.parent < b.parent;
  return a.token < b.token;
}

static inline float log_add(float a, float b) {
  const double m = std::max((double)a, (double)b);
  return (float)(m + std::log1p(std::exp(-std::fabs((double)a - (double)b))));
}

struct Final {
  std::vector<int32_t> y;
  float S;
  int64_t order;
};

// Alignment-length synchronous beam search (Section 2) with the density-ratio
// score of Eq. 1 for ONE utterance.  e [T, D] are the projected encoder frames.
// Iteration i holds hypotheses with t + |y| = i.  Each live hypothesis proposes
// a blank (t+1, same labels; score + log P(blank)) and, while |y| < U_max, every
// label k (same t; score + log P(k) + lambda_t log P_tgt(k) - lambda_s log
// P_src(k) + rho): summed along a path this is Eq. 1, the LM terms and the
// reward applying to labels only.  Proposals that describe the same label
// string are merged by log-addition; those that consumed the last frame are
// final; the W best of the rest (score descending, then parent slot, then
// token) form the next beam.  T + U_max iterations are always executed.
//
// Outputs: best_tokens [U_max], best_len, best_score; trace arrays
// [T+U_max, W] (nullable): parent slot, token (0 blank), score, t, u of each
// slot of the beam selected in that iteration, slot count in trace_n [T+U_max];
// finals_n = number of final hypotheses kept (at most W), listed best first in
// finals_tokens [W,U_max], finals_len [W], finals_score [W] (nullable).
void orc_alsd(const OrcDecoder* Dc, const float* e, int32_t T, int32_t* best_tokens,
              int32_t* best_len, float* best_score, int32_t* trace_parent, int32_t* trace_token,
              float* trace_score, int32_t* trace_t, int32_t* trace_u, int32_t* trace_n,
              int32_t* finals_n, int32_t* finals_tokens, int32_t* finals_len,
              float* finals_score) {
  const int32_t W = Dc->W, U_max = Dc->U_max, V = Dc->joint.out.J, D = Dc->joint.out.K;
  std::vector<Hyp> beam(1);
  beam[0].t = 0;
  beam[0].S = 0.0f;
  pred_init(Dc->pred, beam[0].pred);
  lm_init(Dc->src, beam[0].src);
  lm_init(Dc->tgt, beam[0].tgt);
  pred_advance(Dc->pred, 0, beam[0].pred);   // start symbol = 0
  lm_advance(Dc->src, 0, beam[0].src);
  lm_advance(Dc->tgt, 0, beam[0].tgt);

  std::vector<Final> finals;
  int64_t order = 0;
  std::vector<float> lp(V);
  for (int32_t it = 0; it < T + U_max; ++it) {
    std::vector<Cand> cands;
    const int32_t nb = (int32_t)beam.size();
    std::vector<int32_t> blank_idx(nb), label_base(nb, -1);
    for (int32_t w = 0; w < nb; ++w) {
      const Hyp& h = beam[w];
      orc_joint(&Dc->joint, e + (int64_t)h.t * D, h.pred.p.data(), 1, lp.data(), nullptr, nullptr);
      blank_idx[w] = (int32_t)cands.size();
      cands.push_back({(float)((double)h.S + (double)lp[0]), w, 0, false});
      if ((int32_t)h.y.size() < U_max) {
        label_base[w] = (int32_t)cands.size();
        for (int32_t k = 1; k < V; ++k) {
          const double s = (double)h.S + (double)lp[k] + (double)Dc->lambda_t * (double)h.tgt.lp[k] -
                           (double)Dc->lambda_s * (double)h.src.lp[k] + (double)Dc->rho;
          cands.push_back({(float)s, w, k, false});
        }
      }
    }
    // merge: label proposal (w2, k) with y_w2 + k == y_w joins the blank proposal of w
    for (int32_t w = 0; w < nb; ++w)
      for (int32_t w2 = 0; w2 < nb; ++w2) {
        const auto& a = beam[w].y;
        const auto& b = beam[w2].y;
        if (a.size() != b.size() + 1 || label_base[w2] < 0) continue;
        if (!std::equal(b.begin(), b.end(), a.begin())) continue;
        Cand& lab = cands[label_base[w2] + (a.back() - 1)];
        Cand& blk = cands[blank_idx[w]];
        blk.S = log_add(blk.S, lab.S);
        lab.dead = true;
      }
    // finals: blank proposals that consumed the last frame
    std::vector<Cand> pool;
    for (const Cand& c : cands) {
      if (c.dead) continue;
      if (c.token == 0 && beam[c.parent].t + 1 == T) {
        finals.push_back({beam[c.parent].y, c.S, order++});
      } else {
        pool.push_back(c);
      }
    }
    std::stable_sort(finals.begin(), finals.end(), [](const Final& a, const Final& b) {
      if (a.S != b.S) return a.S > b.S;
      return a.order < b.order;
    });
    if ((int32_t)finals.size() > W) finals.resize(W);
    std::sort(pool.begin(), pool.end(), ranks_before);
    if ((int32_t)pool.size() > W) pool.resize(W);

    std::vector<Hyp> next;
    next.reserve(pool.size());
    for (size_t s = 0; s < pool.size(); ++s) {
      const Cand& c = pool[s];
      Hyp h = beam[c.parent];
      h.S = c.S;
      if (c.token == 0) {
        h.t += 1;
      } else {
        h.y.push_back(c.token);
        pred_advance(Dc->pred, c.token, h.pred);
        lm_advance(Dc->src, c.token, h.src);
        lm_advance(Dc->tgt, c.token, h.tgt);
      }
      if (trace_parent) {
        const int64_t o = (int64_t)it * W + (int64_t)s;
        trace_parent[o] = c.parent;
        trace_token[o] = c.token;
        trace_score[o] = c.S;
        trace_t[o] = h.t;
        trace_u[o] = (int32_t)h.y.size();
      }
      next.push_back(std::move(h));
    }
    if (trace_n) trace_n[it] = (int32_t)next.size();
    beam.swap(next);
  }
  const std::vector<int32_t>* by = nullptr;
  float bs = 0.0f;
  if (!finals.empty()) {
    by = &finals[0].y;
    bs = finals[0].S;
  } else if (!beam.empty()) {
    size_t bi = 0;
    for (size_t i = 1; i < beam.size(); ++i)
      if (beam[i].S > beam[bi].S) bi = i;
    by = &beam[bi].y;
    bs = beam[bi].S;
  }
  *best_len = by ? (int32_t)by->size() : 0;
  *best_score = bs;
  for (int32_t i = 0; i < *best_len && i < U_max; ++i) best_tokens[i] = (*by)[i];
  if (finals_n) *finals_n = (int32_t)finals.size();
  if (finals_tokens)
    for (size_t f = 0; f < finals.size(); ++f) {
      finals_len[f] = (int32_t)finals[f].y.size();
      finals_score[f] = finals[f].S;
      for (size_t i = 0; i < finals[f].y.size(); ++i) finals_tokens[f * U_max + i] = finals[f].y[i];
    }
}

// Batch of independent utterances, e [T, B, D] time-major; one utterance per
// thread.  `utts` lists which utterances to decode (n_utts of them); outputs
// are indexed by position in that list.
void orc_alsd_batch(const OrcDecoder* Dc, const float* e, int32_t T, int32_t B,
                    const int32_t* utts, int32_t n_utts, int32_t* best_tokens, int32_t* best_len,
                    float* best_score, int32_t* trace_parent, int32_t* trace_token,
                    float* trace_score, int32_t* trace_t, int32_t* trace_u, int32_t* trace_n,
                    int32_t* finals_n, int32_t* finals_tokens, int32_t* finals_len,
                    float* finals_score, int32_t n_threads) {
  const int32_t D = Dc->joint.out.K, W = Dc->W, U = Dc->U_max, IT = T + Dc->U_max;
  n_threads = std::max(1, std::min(n_threads, n_utts));
  std::vector<std::thread> pool;
  for (int32_t w = 0; w < n_threads; ++w)
    pool.emplace_back([=]() {
      for (int32_t i = w; i < n_utts; i += n_threads) {
        const int32_t b = utts[i];
        std::vector<float> eu((size_t)T * D);
        for (int32_t t = 0; t < T; ++t)
          std::memcpy(&eu[(size_t)t * D], e + ((int64_t)t * B + b) * D, D * sizeof(float));
        const int64_t o = (int64_t)i * IT * W;
        orc_alsd(Dc, eu.data(), T, best_tokens + (int64_t)i * U, best_len + i, best_score + i,
                 trace_parent ? trace_parent + o : nullptr, trace_token ? trace_token + o : nullptr,
                 trace_score ? trace_score + o : nullptr, trace_t ? trace_t + o : nullptr,
                 trace_u ? trace_u + o : nullptr, trace_n ? trace_n + (int64_t)i * IT : nullptr,
                 finals_n ? finals_n + i : nullptr,
                 finals_tokens ? finals_tokens + (int64_t)i * W * U : nullptr,
                 finals_tokens ? finals_len + (int64_t)i * W : nullptr,
                 finals_tokens ? finals_score + (int64_t)i * W : nullptr);
      }
    });
  for (auto& th : pool) th.join();
}

// Time-synchronous beam search with the score of Eq. 1 for ONE utterance: all hypotheses of
// the beam stand at the same frame t.  A frame takes S_max + 1 steps.  In step s every
// hypothesis of the current set A proposes its blank (score + log P(blank)): the string moves
// to the next frame and is collected in the set B, equal label strings merged by log-addition
// (the entry keeps the provenance of its first insertion); while s < S_max and |y| < U_max it
// also proposes every label k (score + log P(k) + lambda_t log P_tgt(k) - lambda_s log
// P_src(k) + rho), and the W best label proposals (score descending, then parent slot, then
// token) become the set A of step s + 1, still at frame t.  After step S_max the W best
// entries of B (score descending, then insertion order) are the beam of frame t + 1.  The
// entries of B after the last frame are the final hypotheses.  T (S_max + 1) steps in all.
//
// Trace arrays [T (S_max+1), W]: the set produced by each step.  For s < S_max: parent slot,
// token (> 0), score, |y| of each new member of A.  For s = S_max (frame close): parent = the
// slot the entry's blank was first proposed from, token = -1 - (step of that proposal within
// the frame), score, |y|.
void orc_tsd(const OrcDecoder* Dc, const float* e, int32_t T, int32_t S_max, int32_t* best_tokens,
             int32_t* best_len, float* best_score, int32_t* trace_parent, int32_t* trace_token,
             float* trace_score, int32_t* trace_u, int32_t* trace_n, int32_t* finals_n,
             int32_t* finals_tokens, int32_t* finals_len, float* finals_score) {
  const int32_t W = Dc->W, U_max = Dc->U_max, V = Dc->joint.out.J, D = Dc->joint.out.K;
  struct Entry {
    Hyp h;
    int32_t org_step, org_slot;
  };
  std::vector<Hyp> A(1);
  A[0].t = 0;
  A[0].S = 0.0f;
  pred_init(Dc->pred, A[0].pred);
  lm_init(Dc->src, A[0].src);
  lm_init(Dc->tgt, A[0].tgt);
  pred_advance(Dc->pred, 0, A[0].pred);   // start symbol = 0
  lm_advance(Dc->src, 0, A[0].src);
  lm_advance(Dc->tgt, 0, A[0].tgt);
  std::vector<Entry> Bset;
  std::vector<float> lp(V);
  int32_t it = 0;
  for (int32_t t = 0; t < T; ++t) {
    Bset.clear();
    for (int32_t s = 0; s <= S_max; ++s, ++it) {
      std::vector<Cand> labels;
      for (int32_t w = 0; w < (int32_t)A.size(); ++w) {
        const Hyp& h = A[w];
        orc_joint(&Dc->joint, e + (int64_t)t * D, h.pred.p.data(), 1, lp.data(), nullptr, nullptr);
        const float sb = (float)((double)h.S + (double)lp[0]);
        bool merged = false;
        for (Entry& b : Bset)
          if (b.h.y == h.y) {
            b.h.S = log_add(b.h.S, sb);
            merged = true;
            break;
          }
        if (!merged) {
          Entry b{h, s, w};
          b.h.S = sb;
          b.h.t = t + 1;
          Bset.push_back(std::move(b));
        }
        if (s < S_max && (int32_t)h.y.size() < U_max)
          for (int32_t k = 1; k < V; ++k) {
            const double sc = (double)h.S + (double)lp[k] + (double)Dc->lambda_t * (double)h.tgt.lp[k] -
                              (double)Dc->lambda_s * (double)h.src.lp[k] + (double)Dc->rho;
            labels.push_back({(float)sc, w, k, false});
          }
      }
      std::vector<Hyp> next;
      if (s < S_max) {
        std::sort(labels.begin(), labels.end(), ranks_before);
        if ((int32_t)labels.size() > W) labels.resize(W);
        for (size_t i = 0; i < labels.size(); ++i) {
          const Cand& c = labels[i];
          Hyp h = A[c.parent];
          h.S = c.S;
          h.y.push_back(c.token);
          pred_advance(Dc->pred, c.token, h.pred);
          lm_advance(Dc->src, c.token, h.src);
          lm_advance(Dc->tgt, c.token, h.tgt);
          if (trace_parent) {
            const int64_t o = (int64_t)it * W + (int64_t)i;
            trace_parent[o] = c.parent;
            trace_token[o] = c.token;
            trace_score[o] = c.S;
            trace_u[o] = (int32_t)h.y.size();
          }
          next.push_back(std::move(h));
        }
      } else {
        std::vector<int32_t> idx(Bset.size());
        for (size_t i = 0; i < idx.size(); ++i) idx[i] = (int32_t)i;
        std::stable_sort(idx.begin(), idx.end(),
                         [&](int32_t a, int32_t b) { return Bset[a].h.S > Bset[b].h.S; });
        if ((int32_t)idx.size() > W) idx.resize(W);
        for (size_t i = 0; i < idx.size(); ++i) {
          const Entry& b = Bset[idx[i]];
          if (trace_parent) {
            const int64_t o = (int64_t)it * W + (int64_t)i;
            trace_parent[o] = b.org_slot;
            trace_token[o] = -1 - b.org_step;
            trace_score[o] = b.h.S;
            trace_u[o] = (int32_t)b.h.y.size();
          }
          next.push_back(b.h);
        }
      }
      if (trace_n) trace_n[it] = (int32_t)next.size();
      A.swap(next);
    }
  }
  // A = the W best final hypotheses, best first
  *best_len = A.empty() ? 0 : (int32_t)A[0].y.size();
  *best_score = A.empty() ? 0.0f : A[0].S;
  for (int32_t i = 0; i < *best_len && i < U_max; ++i) best_tokens[i] = A[0].y[i];
  if (finals_n) *finals_n = (int32_t)A.size();
  if (finals_tokens)
    for (size_t f = 0; f < A.size(); ++f) {
      finals_len[f] = (int32_t)A[f].y.size();
      finals_score[f] = A[f].S;
      for (size_t i = 0; i < A[f].y.size(); ++i) finals_tokens[f * U_max + i] = A[f].y[i];
    }
}

void orc_tsd_batch(const OrcDecoder* Dc, const float* e, int32_t T, int32_t B, int32_t S_max,
                   const int32_t* utts, int32_t n_utts, int32_t* best_tokens, int32_t* best_len,
                   float* best_score, int32_t* trace_parent, int32_t* trace_token, float* trace_score,
                   int32_t* trace_u, int32_t* trace_n, int32_t* finals_n, int32_t* finals_tokens,
                   int32_t* finals_len, float* finals_score, int32_t n_threads) {
  const int32_t D = Dc->joint.out.K, W = Dc->W, U = std::max(Dc->U_max, 1), IT = T * (S_max + 1);
  n_threads = std::max(1, std::min(n_threads, n_utts));
  std::vector<std::thread> pool;
  for (int32_t w = 0; w < n_threads; ++w)
    pool.emplace_back([=]() {
      for (int32_t i = w; i < n_utts; i += n_threads) {
        const int32_t b = utts[i];
        std::vector<float> eu((size_t)T * D);
        for (int32_t t = 0; t < T; ++t)
          std::memcpy(&eu[(size_t)t * D], e + ((int64_t)t * B + b) * D, D * sizeof(float));
        const int64_t o = (int64_t)i * IT * W;
        orc_tsd(Dc, eu.data(), T, S_max, best_tokens + (int64_t)i * U, best_len + i, best_score + i,
                trace_parent ? trace_parent + o : nullptr, trace_token ? trace_token + o : nullptr,
                trace_score ? trace_score + o : nullptr, trace_u ? trace_u + o : nullptr,
                trace_n ? trace_n + (int64_t)i * IT : nullptr, finals_n ? finals_n + i : nullptr,
                finals_tokens ? finals_tokens + (int64_t)i * W * U : nullptr,
                finals_tokens ? finals_len + (int64_t)i * W : nullptr,
                finals_tokens ? finals_score + (int64_t)i * W : nullptr);
      }
    });
  for (auto& th : pool) th.join();
}

// Score of ONE given label string under Eq. 1, with log P(y|x) from the
// textbook transducer forward recursion over the (t,u) lattice:
//   a(0,0)=0; a(t,u) = logadd(a(t-1,u)+blank(t-1,u), a(t,u-1)+label(t,u-1));
//   log P = a(T-1,U) + blank(T-1,U).
// Used to check the search against brute-force enumeration.
void orc_sequence_score(const OrcDecoder* Dc, const float* e, int32_t T, const int32_t* y,
                        int32_t U, float* score_out, double* log_p_rnnt, double* log_p_tgt,
                        double* log_p_src) {
  const int32_t V = Dc->joint.out.J, D = Dc->joint.out.K;
  PredState ps;
  LmState ss, ts;
  pred_init(Dc->pred, ps);
  lm_init(Dc->src, ss);
  lm_init(Dc->tgt, ts);
  std::vector<std::vector<float>> lp((size_t)(U + 1) * T, std::vector<float>(V));
  double lt = 0.0, ls = 0.0;
  for (int32_t u = 0; u <= U; ++u) {
    const int32_t tok = u == 0 ? 0 : y[u - 1];
    pred_advance(Dc->pred, tok, ps);
    lm_advance(Dc->src, tok, ss);
    lm_advance(Dc->tgt, tok, ts);
    if (u < U) {
      lt += (double)ts.lp[y[u]];
      ls += (double)ss.lp[y[u]];
    }
    for (int32_t t = 0; t < T; ++t)
      orc_joint(&Dc->joint, e + (int64_t)t * D, ps.p.data(), 1, lp[(size_t)u * T + t].data(),
                nullptr, nullptr);
  }
  const double NEG = -1.0e300;
  std::vector<double> a((size_t)T * (U + 1), NEG);
  auto la = [](double p, double q) {
    if (p < -1.0e299) return q;
    if (q < -1.0e299) return p;
    const double m = std::max(p, q);
    return m + std::log1p(std::exp(-std::fabs(p - q)));
  };
  a[0] = 0.0;
  for (int32_t t = 0; t < T; ++t)
    for (int32_t u = 0; u <= U; ++u) {
      if (t == 0 && u == 0) continue;
      double v = NEG;
      if (t > 0) v = la(v, a[(size_t)(t - 1) * (U + 1) + u] + (double)lp[(size_t)u * T + t - 1][0]);
      if (u > 0)
        v = la(v, a[(size_t)t * (U + 1) + u - 1] + (double)lp[(size_t)(u - 1) * T + t][y[u - 1]]);
      a[(size_t)t * (U + 1) + u] = v;
    }
  const double lpr = a[(size_t)(T - 1) * (U + 1) + U] + (double)lp[(size_t)U * T + T - 1][0];
  *log_p_rnnt = lpr;
  *log_p_tgt = lt;
  *log_p_src = ls;
  *score_out = (float)(lpr + (double)Dc->lambda_t * lt - (double)Dc->lambda_s * ls +
                       (double)Dc->rho * (double)U);
}

// ------------------------------------------------------------ feature prologue
// log-mel [T100, M] at 100 frames/s -> first and second time differences
// (d_t = (x_{t+1} - x_{t-1})/2 with replicated edges, dd likewise on d) ->
// [T100, 3M]; then frames (2s, 2s+1) are concatenated -> [T100/2, 6M], fp32
// arithmetic, result rounded to fp16 precision by the caller.
void orc_features(const float* mel, int32_t T100, int32_t M, float* out) {
  std::vector<float> d((size_t)T100 * M), dd((size_t)T100 * M);
  auto at = [&](const float* a, int32_t t, int32_t m) {
    t = std::min(std::max(t, 0), T100 - 1);
    return a[(size_t)t * M + m];
  };
  for (int32_t t = 0; t < T100; ++t)
    for (int32_t m = 0; m < M; ++m) d[(size_t)t * M + m] = (at(mel, t + 1, m) - at(mel, t - 1, m)) * 0.5f;
  for (int32_t t = 0; t < T100; ++t)
    for (int32_t m = 0; m < M; ++m)
      dd[(size_t)t * M + m] = (at(d.data(), t + 1, m) - at(d.data(), t - 1, m)) * 0.5f;
  const int32_t T50 = T100 / 2;
  for (int32_t s = 0; s < T50; ++s)
    for (int32_t half = 0; half < 2; ++half) {
      const int32_t t = 2 * s + half;
      float* o = out + ((size_t)s * 2 + half) * 3 * M;
      for (int32_t m = 0; m < M; ++m) {
        o[m] = mel[(size_t)t * M + m];
        o[M + m] = d[(size_t)t * M + m];
        o[2 * M + m] = dd[(size_t)t * M + m];
      }
    }
}

}  // extern "C"
