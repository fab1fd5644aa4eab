// C ABI of the library (see include/q4rnnt.h): argument checking on the host, argument
// blocks for the kernels, launch sequencing.  Nothing here allocates or synchronises.
#include <math.h>
#include <string.h>

#include "q4_internal.h"

using namespace q4;

#define Q4_TRY(expr)                               \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return Q4_ERR_CUDA;    \
  } while (0)
#define Q4_CHECK(expr)        \
  do {                        \
    int r__ = (expr);         \
    if (r__ != Q4_OK) return r__; \
  } while (0)

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline cudaStream_t S(q4_stream s) { return reinterpret_cast<cudaStream_t>(s); }

int check_act(const q4_act* a) {
  if (!a) return Q4_ERR_NULL;
  if (a->bits != 4 && a->bits != 8) return Q4_ERR_BITS;
  if (!a->is_signed && a->bits != 4) return Q4_ERR_BITS;  // unsigned codes exist at 4 bit only
  if (!a->is_signed && (a->zero_point < 0 || a->zero_point > 15)) return Q4_ERR_DIM;
  if (a->is_signed && a->zero_point != 0) return Q4_ERR_DIM;
  if (!(a->scale > 0.0f) || !(a->inv_scale > 0.0f)) return Q4_ERR_DIM;
  return Q4_OK;
}

int check_mat(const q4_mat* m, int rows, int k_pad_expected) {
  if (!m || !m->q || !m->scale) return Q4_ERR_NULL;
  if (m->bits != 2 && m->bits != 4 && m->bits != 8) return Q4_ERR_BITS;
  if (m->rows <= 0 || m->k <= 0 || m->k_pad < m->k) return Q4_ERR_DIM;
  if (m->k_pad % (m->bits == 2 ? 64 : 32) != 0) return Q4_ERR_ALIGN;   // rows are 16-byte multiples
  if (rows > 0 && m->rows != rows) return Q4_ERR_DIM;
  if (k_pad_expected > 0 && m->k_pad != k_pad_expected) return Q4_ERR_DIM;
  if (!aligned16(m->q) || (reinterpret_cast<uintptr_t>(m->scale) & 3u)) return Q4_ERR_ALIGN;
  return Q4_OK;
}

inline long long row_bytes(int k_pad, int bits) { return (long long)k_pad * bits / 8; }

GemmArgs gemm_args(const void* x, long long x_stride, const int32_t* x_idx, const q4_act& xa, int M,
                   const q4_mat& w, const float* bias, void* out, long long out_stride,
                   const int32_t* out_idx) {
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.x.base = static_cast<const uint8_t*>(x);
  g.x.stride = x_stride;
  g.x.idx = x_idx;
  g.x_signed = xa.is_signed;
  g.x_zp = xa.zero_point;
  g.x_bits = xa.bits;
  g.w_bits = w.bits;
  g.M = M;
  g.w = static_cast<const uint8_t*>(w.q);
  g.w_scale = w.scale;
  g.bias = bias;
  g.J = w.rows;
  g.k_pad = w.k_pad;
  g.x_scale = xa.scale;
  g.out = out;
  g.out_stride = out_stride;
  g.out_idx = out_idx;
  return g;
}

}  // namespace

extern "C" {

int q4_version(void) { return 1; }

int q4_timing_set(uint32_t tag_mask, void** start_events, void** stop_events, int32_t* tags_out,
                  int32_t capacity) {
  if (tag_mask != 0 && (!start_events || !stop_events || !tags_out || capacity <= 0)) return Q4_ERR_NULL;
  timing_set(tag_mask, reinterpret_cast<cudaEvent_t*>(start_events),
             reinterpret_cast<cudaEvent_t*>(stop_events), tags_out, tag_mask ? capacity : 0);
  return Q4_OK;
}
int q4_timing_count(void) { return timing_count(); }
int64_t q4_launch_count(void) { return g_launches; }
int64_t q4_quantizer_calls(int32_t reset) {
  const int64_t n = g_quant_calls;
  if (reset) g_quant_calls = 0;
  return n;
}
static int g_select_exact = 0;
static int select_exact_only() { return g_select_exact; }
int q4_beam_select_exact_set(int32_t enabled) {
  const int prev = g_select_exact;
  g_select_exact = enabled ? 1 : 0;
  return prev;
}
int q4_test_wait_expiry_set(int32_t skip_producer, uint32_t wait_limit) {
  test_wait_expiry_set(skip_producer ? 1 : 0, wait_limit);
  return Q4_OK;
}
int q4_encoder_time_slicing_set(int32_t enabled) { return enc_recurrent_sliced_set(enabled ? 1 : 0); }
int q4_encoder_recurrence_plan(int32_t T, int32_t B, int32_t dirs, int32_t H, int32_t w_bits, int32_t hid_bits,
                               int32_t per_sequence_scale, int32_t* out) {
  if (!out) return Q4_ERR_NULL;
  if (T <= 0 || B <= 0 || dirs < 1 || dirs > 2 || H <= 0) return Q4_ERR_DIM;
  const EncRecPlan p = enc_recurrent_plan(T, B, dirs, H, w_bits, hid_bits, true, per_sequence_scale != 0, false, true);
  out[0] = p.kernel;
  out[1] = p.groups_per_cluster;
  out[2] = p.ncl[0];
  out[3] = p.ncl[1];
  out[4] = p.sliced[0];
  out[5] = p.sliced[1];
  out[6] = p.groups;
  out[7] = p.max_clusters;
  for (int j = 0; j < 9; ++j) out[8 + j] = p.win[j];
  return Q4_OK;
}
int q4_dependent_launch_set(int32_t enabled) {
  const int prev = g_dependent_launch;
  g_dependent_launch = enabled ? 1 : 0;
  return prev;
}

int q4_act_symmetric(float alpha, int32_t bits, q4_act* out) {
  if (!out) return Q4_ERR_NULL;
  if (bits != 4 && bits != 8) return Q4_ERR_BITS;
  if (!(alpha > 0.0f)) return Q4_ERR_DIM;
  const volatile float qmax = (float)((1 << (bits - 1)) - 1);
  const volatile float s = alpha / qmax;
  const volatile float inv = 1.0f / s;
  out->scale = s;
  out->inv_scale = inv;
  out->zero_point = 0;
  out->bits = bits;
  out->is_signed = 1;
  return Q4_OK;
}

int q4_act_asymmetric(float lo, float hi, int32_t bits, q4_act* out) {
  if (!out) return Q4_ERR_NULL;
  if (bits != 4) return Q4_ERR_BITS;
  if (!(hi > lo)) return Q4_ERR_DIM;
  const volatile float qmax = (float)((1 << bits) - 1);
  const volatile float s = (hi - lo) / qmax;
  const volatile float inv = 1.0f / s;
  const volatile float zr = -lo / s;
  float z = nearbyintf(zr);
  z = fminf(fmaxf(z, 0.0f), qmax);
  out->scale = s;
  out->inv_scale = inv;
  out->zero_point = (int32_t)z;
  out->bits = bits;
  out->is_signed = 0;
  return Q4_OK;
}

size_t q4_workspace_bytes(int32_t call_id, const int32_t* dims, int32_t ndims) {
  if (!dims) return 0;
  if (call_id == Q4_WS_LSTM_LAYER && ndims >= 4) {
    const size_t T = dims[0], B = dims[1], D = dims[2], H = dims[3];
    const size_t K = ndims >= 5 ? dims[4] : 0;
    size_t n = 256;                                      // status word
    n += align_up(D * T * B * 4 * H * sizeof(int32_t));  // input accumulators
    n += align_up(D * 2 * B * H);                        // recurrent codes, double buffered
    n += align_up(D * B * H * sizeof(float));            // cell state
    if (K > 0) {                                         // int8 operands of the tensor-core GEMM
      n += align_up(T * B * K);
      n += align_up(D * 4 * H * K);
      n += align_up(D * 4 * H * H);                      // resident recurrent weights, int8
      n += 3 * align_up(D * 4 * H * sizeof(float));      // row scales and bias, cell-major
    }
    return n;
  }
  if (call_id == Q4_WS_JOINT && ndims >= 2) {
    const size_t N = dims[0], D = dims[1];
    size_t n = align_up(N * D * sizeof(float)) + align_up(N * D);
    if (ndims >= 3) {   // tensor-core path: status word, int8 copies of the hidden codes and of z
      const size_t Np = (N + 127) / 128 * 128, Hp = dims[2];
      n += 256 + align_up(Np * Hp) + align_up(Np * D);
    }
    return n;
  }
  if (call_id == Q4_WS_LSTM_STEP && ndims >= 3) {   // status word, int8 copies of x and h rows
    const size_t Np = ((size_t)dims[0] + 127) / 128 * 128;
    return 256 + align_up(Np * (size_t)dims[1]) + align_up(Np * (size_t)dims[2]);
  }
  if (call_id == Q4_WS_LINEAR && ndims >= 2) {      // status word, int8 copy of the input rows
    const size_t Np = ((size_t)dims[0] + 127) / 128 * 128;
    return 256 + align_up(Np * (size_t)dims[1]);
  }
  if (call_id == Q4_WS_BEAM && ndims >= 4) {
    const size_t N = (size_t)dims[0] * dims[1], V = dims[2], D = dims[3];
    size_t n = align_up(N * D) * 3 + align_up(N * V * sizeof(float)) + align_up(N * sizeof(int32_t));
    if (ndims >= 8) {  // int8 operand scratch of the tensor-core path
      const size_t Np = (N + 127) / 128 * 128;
      const size_t E = dims[4], Hp = dims[5], Hs = dims[6], Ht = dims[7];
      const size_t Hmax = Hp > Hs ? (Hp > Ht ? Hp : Ht) : (Hs > Ht ? Hs : Ht);
      n += 3 * align_up(Np * E) + align_up(Np * Hp) + align_up(Np * Hs) + 2 * align_up(Np * Ht);  // gathered x / h operands
      (void)Hmax;
      n += align_up(Np * Hp) + align_up(Np * Hs) + 2 * align_up(Np * Ht); // new cell outputs, int8
      n += 3 * align_up(Np * D);                                         // bottleneck codes, z codes
    }
    return n;
  }
  return 0;
}

int q4_poll_status(const int32_t* device_status, q4_stream stream) {
  if (!device_status) return Q4_ERR_NULL;
  int32_t h = 0;
  if (cudaMemcpyAsync(&h, device_status, sizeof(h), cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess)
    return Q4_ERR_CUDA;
  if (cudaStreamSynchronize(S(stream)) != cudaSuccess) return Q4_ERR_CUDA;
  return h == 0 ? Q4_OK : (int)h;
}

int quantize_pack_int4(const void* x, int32_t x_is_fp16, int64_t rows, int32_t k, int32_t k_pad,
                       const q4_act* act, int32_t mode, int32_t n_groups,
                       const float* per_row_scale, void* q_out, float* group_scale_out,
                       q4_stream stream) {
  if (!act) return Q4_ERR_NULL;
  if (rows < 0 || k <= 0 || k_pad < k) return Q4_ERR_DIM;
  if (rows > 0 && (!x || !q_out)) return Q4_ERR_NULL;
  if (k_pad % 32 != 0 || !aligned16(q_out)) return Q4_ERR_ALIGN;
  if (mode < 0 || mode > 2) return Q4_ERR_UNSUPPORTED;
  if (act->bits != 4 && act->bits != 8 && !(act->bits == 2 && mode != 0)) return Q4_ERR_BITS;   // 2 bit: weights
  if (act->bits == 2 && k_pad % 64 != 0) return Q4_ERR_ALIGN;
  q4_act a = *act;
  if (mode == 0) {
    Q4_CHECK(check_act(act));
  } else {
    a.is_signed = 1;
    a.zero_point = 0;
    a.scale = a.inv_scale = 1.0f;
    if (mode == 1 && (!group_scale_out || n_groups <= 0)) return group_scale_out ? Q4_ERR_DIM : Q4_ERR_NULL;
    if (mode == 2 && !per_row_scale) return Q4_ERR_NULL;
  }
  if (rows == 0) return Q4_OK;
  TagScope tag(TAG_QUANT);
  if (mode != 2) ++g_quant_calls;   // an activation tensor (weights are quantized once, off line)
  Q4_TRY(launch_quantize(x, x_is_fp16 != 0, rows, k, k_pad, a, mode, n_groups, per_row_scale,
                         static_cast<uint8_t*>(q_out), group_scale_out, S(stream)));
  return Q4_OK;
}

int q4_linear_forward(const void* xq, const q4_act* x_act, int32_t M, const q4_mat* w,
                      const float* bias, float* out, int32_t* dbg_acc, const void* prepared,
                      void* workspace, size_t workspace_bytes, q4_stream stream) {
  if (!xq || !out) return Q4_ERR_NULL;
  Q4_CHECK(check_act(x_act));
  Q4_CHECK(check_mat(w, 0, 0));
  if (M < 0) return Q4_ERR_DIM;
  if (!aligned16(xq) || !aligned16(out)) return Q4_ERR_ALIGN;
  {
    const int32_t wd[2] = {M, w->k_pad};
    if (prepared && workspace && !dbg_acc && M >= 128 && aligned16(workspace) && aligned16(prepared) &&
        workspace_bytes >= q4_workspace_bytes(Q4_WS_LINEAR, wd, 2)) {
      // tensor cores: int8 copy of the input rows, then the tiled GEMM on the prepared int8 weights
      cudaStream_t s = S(stream);
      uint8_t* ws = static_cast<uint8_t*>(workspace);
      int32_t* status = reinterpret_cast<int32_t*>(ws);
      int8_t* x8 = reinterpret_cast<int8_t*>(ws + 256);
      const int Mp = (M + 127) / 128 * 128;
      TagScope tag(TAG_LINEAR);
      // the gather clears the status block and may start under the tail of whatever kernel precedes the call
      Q4_TRY(launch_unpack_rows(xq, row_bytes(w->k_pad, x_act->bits), nullptr, *x_act, w->k_pad, M, x8, w->k_pad, 0,
                                Mp, s, status, true));
      Q4_TRY(launch_mma_gemm(x8, w->k_pad, M, static_cast<const int8_t*>(prepared), w->k_pad, w->rows, w->k_pad,
                             EPI_F32, out, w->rows, nullptr, w->scale, bias, x_act->scale, nullptr, status, nullptr,
                             s, true));   // programmatic dependent of the gather before it
      return Q4_OK;
    }
  }
  GemmArgs g = gemm_args(xq, row_bytes(w->k_pad, x_act->bits), nullptr, *x_act, M, *w, bias, out,
                         w->rows, nullptr);
  g.dbg_acc = dbg_acc;
  TagScope tag(TAG_LINEAR);
  Q4_TRY(launch_gemm(g, EPI_F32, S(stream)));
  return Q4_OK;
}

static int check_lstm(const q4_mat* w_ih, const q4_mat* w_hh, const q4_act* x_act,
                      const q4_act* hid_act, int* H_out) {
  Q4_CHECK(check_act(x_act));
  Q4_CHECK(check_act(hid_act));
  if (!hid_act->is_signed) return Q4_ERR_UNSUPPORTED;
  Q4_CHECK(check_mat(w_ih, 0, 0));
  Q4_CHECK(check_mat(w_hh, 0, 0));
  if (w_ih->rows != w_hh->rows || w_ih->rows % 4 != 0) return Q4_ERR_DIM;
  const int H = w_ih->rows / 4;
  if (w_hh->k != H || w_hh->k_pad != H) return Q4_ERR_DIM;
  if (H % 32 != 0) return Q4_ERR_ALIGN;
  *H_out = H;
  return Q4_OK;
}

static void fill_lstm_weights(LstmArgs& a, const q4_mat& w_ih, const q4_mat& w_hh, const float* bias,
                              const q4_act& x_act, const q4_act& hid_act) {
  a.x_signed = x_act.is_signed;
  a.x_zp = x_act.zero_point;
  a.x_bits = x_act.bits;
  a.wih_bits = w_ih.bits;
  a.whh_bits = w_hh.bits;
  a.kx_pad = w_ih.k_pad;
  a.x_scale = x_act.scale;
  a.w_ih = static_cast<const uint8_t*>(w_ih.q);
  a.s_wih = w_ih.scale;
  a.w_hh = static_cast<const uint8_t*>(w_hh.q);
  a.s_whh = w_hh.scale;
  a.bias = bias;
  a.H = w_ih.rows / 4;
  a.kh_pad = w_hh.k_pad;
  a.hid_act = hid_act;
  a.out_act = hid_act;
}

int qlstm_step(const void* xq, const q4_act* x_act, const int32_t* x_row_idx, const void* hq_in,
               const float* c_in, int32_t N, const q4_mat* w_ih, const q4_mat* w_hh,
               const float* bias, const q4_act* hid_act, void* hq_out, float* c_out,
               float* h_f32_out, int32_t* dbg_acc_ih, int32_t* dbg_acc_hh, const void* prepared,
               void* workspace, size_t workspace_bytes, q4_stream stream) {
  if (!xq || !hq_in || !c_in || !c_out) return Q4_ERR_NULL;
  if (!hq_out && !h_f32_out) return Q4_ERR_NULL;   // Inner placement needs the real-valued output
  int H = 0;
  Q4_CHECK(check_lstm(w_ih, w_hh, x_act, hid_act, &H));
  if (N < 0) return Q4_ERR_DIM;
  if (hq_in == hq_out) return Q4_ERR_UNSUPPORTED;
  if (!aligned16(xq) || !aligned16(hq_in) || !aligned16(hq_out)) return Q4_ERR_ALIGN;
  if (N == 0) return Q4_OK;
  if (hq_out) ++g_quant_calls;   // the one quantizer call at the cell output (Outer placement)
  {
    const int32_t wd[3] = {N, w_ih->k_pad, H};
    if (prepared && workspace && hq_out && N >= 128 && H % 128 == 0 && aligned16(workspace) && aligned16(prepared) &&
        (dbg_acc_ih == nullptr) == (dbg_acc_hh == nullptr) && c_out != nullptr &&
        workspace_bytes >= q4_workspace_bytes(Q4_WS_LSTM_STEP, wd, 3)) {
      // tensor cores: int8 copies of the x rows (gathered) and h rows, then the fused LSTM kernel on the
      // prepared int8 weights (rows 4*cell+gate, scales and bias in the same order)
      cudaStream_t s = S(stream);
      const size_t G = 4 * (size_t)H, Kx = w_ih->k_pad;
      const uint8_t* pb = static_cast<const uint8_t*>(prepared);
      const int8_t* xw8 = reinterpret_cast<const int8_t*>(pb);
      const int8_t* hw8 = xw8 + align_up(G * Kx);
      const float* sc_ih = reinterpret_cast<const float*>(hw8 + align_up(G * H));
      const float* sc_hh = sc_ih + align_up(G * sizeof(float)) / sizeof(float);
      const float* bi = sc_hh + align_up(G * sizeof(float)) / sizeof(float);
      uint8_t* ws = static_cast<uint8_t*>(workspace);
      int32_t* status = reinterpret_cast<int32_t*>(ws);
      const int Np = (N + 127) / 128 * 128;
      int8_t* x8 = reinterpret_cast<int8_t*>(ws + 256);
      int8_t* h8 = x8 + align_up((size_t)Np * Kx);
      TagScope tag(TAG_PRED_LSTM);
      // every kernel of the call is a programmatic dependent of the one before (each waits for its
      // predecessor's completion before it reads anything); the first gather clears the status block
      Q4_TRY(launch_unpack_rows(xq, row_bytes(w_ih->k_pad, x_act->bits), x_row_idx, *x_act, (int)Kx, N, x8, (long long)Kx,
                                0, Np, s, status, true));
      Q4_TRY(launch_unpack_rows(hq_in, row_bytes(H, hid_act->bits), nullptr, *hid_act, H, N, h8, H, 0, Np, s, nullptr, true));
      MmaLstmArgs a;
      memset(&a, 0, sizeof(a));
      a.N = N;
      a.H = H;
      a.Kx_pad = (int)Kx;
      a.sc_ih = sc_ih;
      a.sc_hh = sc_hh;
      a.bias = bi;
      a.x_scale = x_act->scale;
      a.hid_act = *hid_act;
      a.out_act = *hid_act;
      a.c_in = c_in;
      a.c_out = c_out;
      a.hq_out = static_cast<uint8_t*>(hq_out);
      a.hq_ld = row_bytes(H, hid_act->bits);
      a.h_f32 = h_f32_out;
      a.dbg_ih = dbg_acc_ih;
      a.dbg_hh = dbg_acc_hh;
      a.dbg_ld = 4LL * H;
      a.status = status;
      // programmatic dependent of the second gather (which started after the first had completed)
      Q4_TRY(launch_mma_lstm(a, x8, (long long)Kx, xw8, (long long)Kx, h8, H, hw8, H, s, true));
      return Q4_OK;
    }
  }
  LstmArgs2 args;
  memset(&args, 0, sizeof(args));
  LstmArgs& a = args.d[0];
  fill_lstm_weights(a, *w_ih, *w_hh, bias, *x_act, *hid_act);
  a.x.base = static_cast<const uint8_t*>(xq);
  a.x.stride = row_bytes(w_ih->k_pad, x_act->bits);
  a.x.idx = x_row_idx;
  a.hin.base = static_cast<const uint8_t*>(hq_in);
  a.hin.stride = row_bytes(H, hid_act->bits);
  a.c_in = c_in;
  a.N = N;
  a.hq_out = static_cast<uint8_t*>(hq_out);
  a.hq_stride = a.hin.stride;
  a.c_out = c_out;
  a.h_f32 = h_f32_out;
  a.dbg_ih = dbg_acc_ih;
  a.dbg_hh = dbg_acc_hh;
  a.dbg_stride = 4LL * H;
  TagScope tag(TAG_PRED_LSTM);
  Q4_TRY(launch_lstm(args, 1, S(stream)));
  return Q4_OK;
}

int qlstm_layer_forward(const void* xq, const q4_act* x_act, const float* x_scale_b, int32_t T,
                        int32_t B, int32_t dirs, const q4_mat* w_ih, const q4_mat* w_hh,
                        const float* const* bias, const q4_act* hid_act, const q4_act* out_act,
                        void* yq, void* hq_n, float* c_n, int32_t* dbg_acc_ih,
                        int32_t* dbg_acc_hh, void* workspace, size_t workspace_bytes,
                        q4_stream stream) {
  if (!xq || !yq || !w_ih || !w_hh || !workspace) return Q4_ERR_NULL;
  if (T <= 0 || B <= 0 || dirs < 1 || dirs > 2) return Q4_ERR_DIM;
  int H = 0;
  for (int d = 0; d < dirs; ++d) {
    int Hd = 0;
    Q4_CHECK(check_lstm(&w_ih[d], &w_hh[d], x_act, hid_act, &Hd));
    if (d == 0) H = Hd;
    if (Hd != H || w_ih[d].k_pad != w_ih[0].k_pad || w_ih[d].bits != w_ih[0].bits) return Q4_ERR_DIM;
  }
  if (!out_act) out_act = hid_act;
  Q4_CHECK(check_act(out_act));
  if (!out_act->is_signed) return Q4_ERR_UNSUPPORTED;
  if (!aligned16(xq) || !aligned16(yq) || !aligned16(workspace)) return Q4_ERR_ALIGN;
  const int32_t dims[5] = {T, B, dirs, H, w_ih[0].k_pad};
  if (workspace_bytes < q4_workspace_bytes(Q4_WS_LSTM_LAYER, dims, 4)) return Q4_ERR_WORKSPACE;
  const long long TB = (long long)T * B;
  // tensor-core input projection when the caller's workspace has room for the int8 operands
  const bool use_mma = TB >= 128 && workspace_bytes >= q4_workspace_bytes(Q4_WS_LSTM_LAYER, dims, 5);

  cudaStream_t s = S(stream);
  const int G = 4 * H;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int32_t* status = reinterpret_cast<int32_t*>(ws);
  ws += 256;
  Q4_TRY(cudaMemsetAsync(status, 0, 256, s));
  int32_t* acc_ih = reinterpret_cast<int32_t*>(ws);
  ws += align_up((size_t)dirs * TB * G * sizeof(int32_t));
  uint8_t* hbuf = ws;  // [dirs][2][B*H bytes]
  ws += align_up((size_t)dirs * 2 * B * H);
  float* cbuf = reinterpret_cast<float*>(ws);  // [dirs][B][H]
  ws += align_up((size_t)dirs * B * H * sizeof(float));
  const int Kx = w_ih[0].k_pad;
  int8_t* x8 = reinterpret_cast<int8_t*>(ws);
  int8_t* w8 = x8 + align_up((size_t)TB * Kx);
  int8_t* whh8 = w8 + align_up((size_t)dirs * G * Kx);
  float* vec_ih = reinterpret_cast<float*>(whh8 + align_up((size_t)dirs * G * H));
  float* vec_hh = vec_ih + align_up((size_t)dirs * G * sizeof(float)) / sizeof(float);
  float* vec_b = vec_hh + align_up((size_t)dirs * G * sizeof(float)) / sizeof(float);
  // persistent recurrence: needs the tensor-core projection (cell-major accumulators)
  const bool persistent = use_mma && enc_recurrent_supported(H, B, dirs);
  const long long hb = row_bytes(H, hid_act->bits);
  const long long yb = row_bytes(dirs * H, out_act->bits);
  const long long xb = row_bytes(w_ih[0].k_pad, x_act->bits);

  // time-parallel input projections for all frames
  if (use_mma) {
    TagScope tag(TAG_QUANT);
    Q4_TRY(launch_unpack_rows(xq, xb, nullptr, *x_act, Kx, (int)TB, x8, Kx, 0, (int)TB, s));
    for (int d = 0; d < dirs; ++d)
      Q4_TRY(launch_prepare_w(w_ih[d], persistent ? 1 : 0, w8 + (size_t)d * G * Kx, Kx, 0, s));
    if (persistent) {
      for (int d = 0; d < dirs; ++d) {
        Q4_TRY(launch_prepare_w(w_hh[d], 1, whh8 + (size_t)d * G * H, H, 0, s));
        Q4_TRY(launch_prepare_vec(w_ih[d].scale, G, 1, vec_ih + (size_t)d * G, s));
        Q4_TRY(launch_prepare_vec(w_hh[d].scale, G, 1, vec_hh + (size_t)d * G, s));
        Q4_TRY(launch_prepare_vec(bias ? bias[d] : nullptr, G, 1, vec_b + (size_t)d * G, s));
      }
    }
  }
  for (int d = 0; d < dirs; ++d) {
    TagScope tag(TAG_ENC_GEMM);
    if (use_mma) {
      Q4_TRY(launch_mma_gemm(x8, Kx, (int)TB, w8 + (size_t)d * G * Kx, Kx, G, Kx, EPI_I32,
                             acc_ih + (size_t)d * TB * G, G, nullptr, nullptr, nullptr, 0.0f, nullptr,
                             status, nullptr, s));
    } else {
      GemmArgs g = gemm_args(xq, xb, nullptr, *x_act, (int)TB, w_ih[d], nullptr,
                             acc_ih + (size_t)d * TB * G, G, nullptr);
      Q4_TRY(launch_gemm(g, EPI_I32, s));
    }
  }
  // per step and direction one quantizer call at the cell output; a second one where the next
  // layer wants the same real value at another precision
  g_quant_calls += (int64_t)T * dirs *
                   ((out_act->bits == hid_act->bits && out_act->scale == hid_act->scale) ? 1 : 2);
  if (persistent) {
    EncRecArgs ra;
    memset(&ra, 0, sizeof(ra));
    ra.T = T;
    ra.B = B;
    ra.H = H;
    ra.dirs = dirs;
    ra.w_bits = w_hh[0].bits;
    ra.status = status;
    ra.x_scale = x_act->scale;
    ra.x_scale_b = x_scale_b;
    ra.hid_act = *hid_act;
    ra.out_act = *out_act;
    ra.yq_ld = yb;
    ra.dbg_ld = (long long)dirs * G;
    // scratch of the time-sliced kernel: counters in the status block (zeroed above), the shared
    // group's state in the buffers the step-by-step path would use
    ra.flags = status + 16;
    for (int d = 0; d < dirs && B >= 8; ++d) {
      ra.hand_h[d] = hbuf + (size_t)d * 2 * B * H;
      ra.hand_c[d] = cbuf + (size_t)d * B * H;
    }
    for (int d = 0; d < dirs; ++d) {
      EncRecDir& D = ra.d[d];
      D.w_hh = whh8 + (size_t)d * G * H;
      D.sc_ih = vec_ih + (size_t)d * G;
      D.sc_hh = vec_hh + (size_t)d * G;
      D.bias = vec_b + (size_t)d * G;
      D.acc_pre = acc_ih + (size_t)d * TB * G;
      D.yq = static_cast<uint8_t*>(yq) + row_bytes(d * H, out_act->bits);
      D.dbg_ih = dbg_acc_ih ? dbg_acc_ih + (size_t)d * G : nullptr;
      D.dbg_hh = dbg_acc_hh ? dbg_acc_hh + (size_t)d * G : nullptr;
      D.hq_n = hq_n ? static_cast<uint8_t*>(hq_n) + (size_t)d * B * hb : nullptr;
      D.c_n = c_n ? c_n + (size_t)d * B * H : nullptr;
    }
    if ((dbg_acc_ih == nullptr) != (dbg_acc_hh == nullptr)) return Q4_ERR_NULL;
    TagScope tag(TAG_ENC_STEP);
    Q4_TRY(launch_enc_recurrent(ra, s));
    return Q4_OK;
  }
  Q4_TRY(cudaMemsetAsync(hbuf, 0, (size_t)dirs * 2 * B * H, s));
  Q4_TRY(cudaMemsetAsync(cbuf, 0, (size_t)dirs * B * H * sizeof(float), s));

  for (int st = 0; st < T; ++st) {
    LstmArgs2 args;
    memset(&args, 0, sizeof(args));
    for (int d = 0; d < dirs; ++d) {
      const int t = d == 0 ? st : T - 1 - st;
      LstmArgs& a = args.d[d];
      fill_lstm_weights(a, w_ih[d], w_hh[d], bias ? bias[d] : nullptr, *x_act, *hid_act);
      a.out_act = *out_act;
      a.x_scale_vec = x_scale_b;
      a.x_scale_mod = B;
      a.acc_pre = acc_ih + ((size_t)d * TB + (size_t)t * B) * G;
      a.acc_pre_stride = G;
      a.hin.base = hbuf + ((size_t)d * 2 + (st & 1)) * B * H;
      a.hin.stride = hb;
      a.c_in = cbuf + (size_t)d * B * H;
      a.N = B;
      a.hq_out = hbuf + ((size_t)d * 2 + ((st + 1) & 1)) * B * H;
      a.hq_stride = hb;
      a.c_out = cbuf + (size_t)d * B * H;
      a.yq_out = static_cast<uint8_t*>(yq) + (size_t)t * B * yb + row_bytes(d * H, out_act->bits);
      a.yq_stride = yb;
      if (dbg_acc_ih) a.dbg_ih = dbg_acc_ih + ((size_t)t * B * dirs + d) * G;
      if (dbg_acc_hh) a.dbg_hh = dbg_acc_hh + ((size_t)t * B * dirs + d) * G;
      a.dbg_stride = (long long)dirs * G;
    }
    TagScope tag(TAG_ENC_STEP);
    Q4_TRY(launch_lstm(args, dirs, s));
  }
  for (int d = 0; d < dirs; ++d) {
    if (hq_n)
      Q4_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(hq_n) + (size_t)d * B * hb,
                             hbuf + ((size_t)d * 2 + (T & 1)) * B * H, (size_t)B * hb,
                             cudaMemcpyDeviceToDevice, s));
    if (c_n)
      Q4_TRY(cudaMemcpyAsync(c_n + (size_t)d * B * H, cbuf + (size_t)d * B * H,
                             (size_t)B * H * sizeof(float), cudaMemcpyDeviceToDevice, s));
  }
  return Q4_OK;
}

int qjoint_logprobs(const float* e, const int32_t* frame_idx, const void* pq, const q4_act* p_act,
                    int32_t N, const q4_mat* w_pred, const float* b_pred, const q4_act* z_act,
                    const q4_mat* w_out, const float* b_out, float* logp, const void* prepared_pred,
                    const void* prepared_out, void* workspace, size_t workspace_bytes, q4_stream stream) {
  if (!e || !frame_idx || !pq || !logp || !workspace) return Q4_ERR_NULL;
  Q4_CHECK(check_act(p_act));
  Q4_CHECK(check_act(z_act));
  Q4_CHECK(check_mat(w_pred, 0, 0));
  Q4_CHECK(check_mat(w_out, 0, 0));
  if (N < 0) return Q4_ERR_DIM;
  const int D = w_pred->rows, V = w_out->rows;
  if (w_out->k != D || w_out->k_pad != D || D % 32 != 0) return Q4_ERR_DIM;
  if (!aligned16(pq) || !aligned16(workspace) || !aligned16(e)) return Q4_ERR_ALIGN;
  const int32_t dims[2] = {N, D};
  if (workspace_bytes < q4_workspace_bytes(Q4_WS_JOINT, dims, 2)) return Q4_ERR_WORKSPACE;
  if (N == 0) return Q4_OK;
  cudaStream_t s = S(stream);
  TagScope tag(TAG_JOINT);
  ++g_quant_calls;   // tanh(e * p)
  const int32_t dims3[3] = {N, D, w_pred->k_pad};
  if (prepared_pred && prepared_out && N >= 128 && V % 32 == 0 && z_act->is_signed && aligned16(prepared_pred) &&
      aligned16(prepared_out) && workspace_bytes >= q4_workspace_bytes(Q4_WS_JOINT, dims3, 3)) {
    // tensor cores, three launches: int8 copy of the hidden codes; projection GEMM whose epilogue forms
    // tanh(e * p) and quantizes it; output layer with the log-softmax in its epilogue (fused head kernel
    // when D = 256, else GEMM + row log-softmax)
    const int Hp = w_pred->k_pad, Np = (N + 127) / 128 * 128;
    uint8_t* ws = static_cast<uint8_t*>(workspace) + align_up((size_t)N * D * sizeof(float)) + align_up((size_t)N * D);
    int32_t* status = reinterpret_cast<int32_t*>(ws);
    int8_t* p8 = reinterpret_cast<int8_t*>(ws + 256);
    int8_t* z8 = p8 + align_up((size_t)Np * Hp);
    Q4_TRY(launch_unpack_rows(pq, row_bytes(Hp, p_act->bits), nullptr, *p_act, Hp, N, p8, Hp, 0, Np, s, status, true));
    Q4_TRY(launch_mma_gemm(p8, Hp, N, static_cast<const int8_t*>(prepared_pred), Hp, D, Hp, EPI_JOINTZ, z8, D,
                           nullptr, w_pred->scale, b_pred, p_act->scale, z_act, status, nullptr, s, true, e,
                           frame_idx));   // each kernel of the call is a programmatic dependent of the one before
    if (D == 256 && V <= 2048) {
      LmHeadArgs ja;
      memset(&ja, 0, sizeof(ja));
      ja.N = N;
      ja.H = 0;
      ja.V = V;
      ja.q_scale = z_act->scale;
      ja.sc_out = w_out->scale;
      ja.b_out = b_out;
      ja.lp = logp;
      ja.status = status;
      Q4_TRY(launch_mma_lmhead(ja, z8, D, nullptr, static_cast<const int8_t*>(prepared_out), s, true));
    } else {
      Q4_TRY(launch_mma_gemm(z8, D, N, static_cast<const int8_t*>(prepared_out), D, V, D, EPI_F32, logp, V, nullptr,
                             w_out->scale, b_out, z_act->scale, nullptr, status, nullptr, s));
      Q4_TRY(launch_logsoftmax(logp, logp, N, V, V, nullptr, s));
    }
    return Q4_OK;
  }
  float* p = static_cast<float*>(workspace);
  uint8_t* zq = static_cast<uint8_t*>(workspace) + align_up((size_t)N * D * sizeof(float));
  GemmArgs g1 = gemm_args(pq, row_bytes(w_pred->k_pad, p_act->bits), nullptr, *p_act, N, *w_pred,
                          b_pred, p, D, nullptr);
  Q4_TRY(launch_gemm(g1, EPI_F32, s));
  Q4_TRY(launch_joint_z(e, frame_idx, nullptr, 1, 1, p, nullptr, N, D, *z_act, zq, nullptr, nullptr, s));
  GemmArgs g2 = gemm_args(zq, row_bytes(D, z_act->bits), nullptr, *z_act, N, *w_out, b_out, logp, V,
                          nullptr);
  Q4_TRY(launch_gemm(g2, EPI_F32, s));
  Q4_TRY(launch_logsoftmax(logp, logp, N, V, V, nullptr, s));
  return Q4_OK;
}

int q4_feature_prologue(const float* mel, int32_t B, int32_t T100, int32_t M, void* out_fp16,
                        q4_stream stream) {
  if (!mel || !out_fp16) return Q4_ERR_NULL;
  if (B <= 0 || T100 < 2 || M <= 0) return Q4_ERR_DIM;
  TagScope tag(TAG_MISC);
  Q4_TRY(launch_features(mel, B, T100, M, out_fp16, S(stream)));
  return Q4_OK;
}

// ------------------------------------------------------------------------ prepared weights
namespace {
struct PrepLstm {
  size_t xw, hw, sc_ih, sc_hh, bias;
};
struct PrepPlan {
  PrepLstm lstm[4];   // prediction, source LM, target LM layer 1, target LM layer 2
  size_t lin[6];      // pred_proj, src.bott, src.out, tgt.bott, tgt.out, joint_out
  size_t total;
};
const q4_lstm* model_lstm(const q4_model& m, int i) {
  switch (i) {
    case 0: return &m.pred_lstm;
    case 1: return &m.src.lstm[0];
    case 2: return &m.tgt.lstm[0];
    default: return m.tgt.n_layers == 2 ? &m.tgt.lstm[1] : nullptr;
  }
}
const q4_linear* model_linear(const q4_model& m, int i) {
  switch (i) {
    case 0: return &m.pred_proj;
    case 1: return &m.src.bott;
    case 2: return &m.src.out;
    case 3: return &m.tgt.bott;
    case 4: return &m.tgt.out;
    default: return &m.joint_out;
  }
}
PrepPlan plan_prepared(const q4_model& m) {
  PrepPlan p;
  memset(&p, 0, sizeof(p));
  size_t o = 0;
  for (int i = 0; i < 4; ++i) {
    const q4_lstm* L = model_lstm(m, i);
    if (!L) continue;
    const size_t G = L->w_ih.rows;
    p.lstm[i].xw = o;
    o += align_up(G * L->w_ih.k_pad);
    p.lstm[i].hw = o;
    o += align_up(G * L->w_hh.k_pad);
    p.lstm[i].sc_ih = o;
    o += align_up(G * sizeof(float));
    p.lstm[i].sc_hh = o;
    o += align_up(G * sizeof(float));
    p.lstm[i].bias = o;
    o += align_up(G * sizeof(float));
  }
  for (int i = 0; i < 6; ++i) {
    const q4_linear* L = model_linear(m, i);
    p.lin[i] = o;
    o += align_up((size_t)L->w.rows * L->w.k_pad);
  }
  p.total = o;
  return p;
}
}  // namespace

size_t q4_prepared_bytes(const q4_model* model) {
  if (!model) return 0;
  return plan_prepared(*model).total;
}

int q4_prepare_model(q4_model* model, void* buffer, size_t bytes, q4_stream stream) {
  if (!model || !buffer) return Q4_ERR_NULL;
  if (!aligned16(buffer)) return Q4_ERR_ALIGN;
  const PrepPlan p = plan_prepared(*model);
  if (bytes < p.total) return Q4_ERR_WORKSPACE;
  cudaStream_t s = S(stream);
  uint8_t* b = static_cast<uint8_t*>(buffer);
  TagScope tag(TAG_MISC);
  for (int i = 0; i < 4; ++i) {
    const q4_lstm* L = model_lstm(*model, i);
    if (!L) continue;
    Q4_CHECK(check_mat(&L->w_ih, 0, 0));
    Q4_CHECK(check_mat(&L->w_hh, 0, 0));
    Q4_TRY(launch_prepare_w(L->w_ih, 1, reinterpret_cast<int8_t*>(b + p.lstm[i].xw), L->w_ih.k_pad, 0, s));
    Q4_TRY(launch_prepare_w(L->w_hh, 1, reinterpret_cast<int8_t*>(b + p.lstm[i].hw), L->w_hh.k_pad, 0, s));
    // de-quantization products of the search (input scale * row scale, hidden scale * row scale)
    const q4_model& mm = *model;
    const float xs = i == 0 ? mm.pred_emb_act.scale : i == 1 ? mm.src.emb_act.scale
                     : i == 2 ? mm.tgt.emb_act.scale : mm.tgt.lstm[0].hid_act.scale;
    Q4_TRY(launch_prepare_vec(L->w_ih.scale, L->w_ih.rows, 1, reinterpret_cast<float*>(b + p.lstm[i].sc_ih), s, xs));
    Q4_TRY(launch_prepare_vec(L->w_hh.scale, L->w_hh.rows, 1, reinterpret_cast<float*>(b + p.lstm[i].sc_hh), s,
                              L->hid_act.scale));
    Q4_TRY(launch_prepare_vec(L->bias, L->w_ih.rows, 1, reinterpret_cast<float*>(b + p.lstm[i].bias), s));
  }
  for (int i = 0; i < 6; ++i) {
    const q4_linear* L = model_linear(*model, i);
    Q4_CHECK(check_mat(&L->w, 0, 0));
    Q4_TRY(launch_prepare_w(L->w, 0, reinterpret_cast<int8_t*>(b + p.lin[i]), L->w.k_pad, 0, s));
  }
  model->prepared = buffer;
  return Q4_OK;
}

// One-time int8 operands for the tensor-core variants of the step calls.
size_t q4_prepared_lstm_bytes(const q4_mat* w_ih, const q4_mat* w_hh) {
  if (!w_ih || !w_hh) return 0;
  const size_t G = w_ih->rows;
  return align_up(G * w_ih->k_pad) + align_up(G * w_hh->k_pad) + 3 * align_up(G * sizeof(float));
}
int q4_prepare_lstm(const q4_mat* w_ih, const q4_mat* w_hh, const float* bias, void* buffer, size_t bytes,
                    q4_stream stream) {
  if (!buffer) return Q4_ERR_NULL;
  Q4_CHECK(check_mat(w_ih, 0, 0));
  Q4_CHECK(check_mat(w_hh, 0, 0));
  if (w_ih->rows != w_hh->rows || w_ih->rows % 4 != 0) return Q4_ERR_DIM;
  if (!aligned16(buffer)) return Q4_ERR_ALIGN;
  if (bytes < q4_prepared_lstm_bytes(w_ih, w_hh)) return Q4_ERR_WORKSPACE;
  cudaStream_t s = S(stream);
  const size_t G = w_ih->rows;
  uint8_t* b = static_cast<uint8_t*>(buffer);
  int8_t* xw8 = reinterpret_cast<int8_t*>(b);
  int8_t* hw8 = xw8 + align_up(G * w_ih->k_pad);
  float* sc_ih = reinterpret_cast<float*>(hw8 + align_up(G * w_hh->k_pad));
  float* sc_hh = sc_ih + align_up(G * sizeof(float)) / sizeof(float);
  float* bi = sc_hh + align_up(G * sizeof(float)) / sizeof(float);
  TagScope tag(TAG_MISC);
  Q4_TRY(launch_prepare_w(*w_ih, 1, xw8, w_ih->k_pad, 0, s));
  Q4_TRY(launch_prepare_w(*w_hh, 1, hw8, w_hh->k_pad, 0, s));
  Q4_TRY(launch_prepare_vec(w_ih->scale, (int)G, 1, sc_ih, s));
  Q4_TRY(launch_prepare_vec(w_hh->scale, (int)G, 1, sc_hh, s));
  Q4_TRY(launch_prepare_vec(bias, (int)G, 1, bi, s));
  return Q4_OK;
}
size_t q4_prepared_linear_bytes(const q4_mat* w) { return w ? align_up((size_t)w->rows * w->k_pad) : 0; }
int q4_prepare_linear(const q4_mat* w, void* buffer, size_t bytes, q4_stream stream) {
  if (!buffer) return Q4_ERR_NULL;
  Q4_CHECK(check_mat(w, 0, 0));
  if (!aligned16(buffer)) return Q4_ERR_ALIGN;
  if (bytes < q4_prepared_linear_bytes(w)) return Q4_ERR_WORKSPACE;
  TagScope tag(TAG_MISC);
  Q4_TRY(launch_prepare_w(*w, 0, static_cast<int8_t*>(buffer), w->k_pad, 0, S(stream)));
  return Q4_OK;
}

// ------------------------------------------------------------------------ beam search
static int check_state(const q4_beam_state* st, int n_lm_layers) {
  if (!st) return Q4_ERR_NULL;
  const void* req[] = {st->pred_hq, st->pred_c, st->pred_p, st->src_hq, st->src_c, st->src_lp,
                       st->tgt_hq[0], st->tgt_c[0], st->tgt_lp, st->score, st->t, st->u, st->hash,
                       st->prev_hash, st->last_tok, st->row, st->adv_src, st->adv_dst, st->adv_tok,
                       st->bp_parent, st->bp_token, st->bp_score, st->fin_score, st->fin_iter,
                       st->fin_slot, st->fin_n, st->status, st->pend_src, st->pend_dst, st->pend_tok,
                       st->pend_n};
  for (const void* p : req)
    if (!p) return Q4_ERR_NULL;
  if (n_lm_layers > 1 && (!st->tgt_hq[1] || !st->tgt_c[1])) return Q4_ERR_NULL;
  return Q4_OK;
}

int q4_beam_init(q4_beam_state* state, int32_t B, int32_t W, int32_t n_iters, q4_stream stream) {
  Q4_CHECK(check_state(state, 1));
  if (B <= 0 || W <= 0 || W > 16 || n_iters < 0) return Q4_ERR_DIM;
  Q4_TRY(launch_beam_init(*state, B, W, n_iters, S(stream)));
  return Q4_OK;
}

// One network's pending advance for all slots: LSTM layers reading the parent's state row and
// writing the fresh row, then the projection(s).
static int advance_lstm(int tag_id, const q4_lstm& L, const void* x, long long x_stride,
                        const int32_t* x_idx, const q4_act& x_act, void* hq, float* c,
                        const q4_beam_state& st, int N, const int32_t* n_active, cudaStream_t s) {
  TagScope tag(tag_id);
  LstmArgs2 args;
  memset(&args, 0, sizeof(args));
  LstmArgs& a = args.d[0];
  fill_lstm_weights(a, L.w_ih, L.w_hh, L.bias, x_act, L.hid_act);
  const int H = a.H;
  a.x.base = static_cast<const uint8_t*>(x);
  a.x.stride = x_stride;
  a.x.idx = x_idx;
  a.hin.base = static_cast<const uint8_t*>(hq);
  a.hin.stride = row_bytes(H, L.hid_act.bits);
  a.hin.idx = st.adv_src;
  a.c_in = c;
  a.N = N;
  a.hq_out = static_cast<uint8_t*>(hq);
  a.hq_stride = a.hin.stride;
  a.out_idx = st.adv_dst;
  a.c_out = c;
  a.dbg_stride = 4LL * H;
  a.n_active = n_active;
  Q4_TRY(launch_lstm(args, 1, s));
  return Q4_OK;
}

static int check_model_lstm(const q4_lstm& L, const q4_act& x_act) {
  int H = 0;
  return check_lstm(&L.w_ih, &L.w_hh, &x_act, &L.hid_act, &H);
}

int dr_fusion_beam_step(const q4_model* model, q4_beam_state* state, const float* e, int32_t B,
                        int32_t T, int32_t W, int32_t iter, int32_t u_max, float lambda_t,
                        float lambda_s, float rho, int32_t mode, void* workspace,
                        size_t workspace_bytes, q4_stream stream) {
  if (!model || !e || !workspace) return Q4_ERR_NULL;
  if (mode < 0 || mode > 2) return Q4_ERR_UNSUPPORTED;
  if (B <= 0 || T <= 0 || W <= 0 || W > 16 || iter < 0 || u_max < 0) return Q4_ERR_DIM;
  const q4_model& m = *model;
  Q4_CHECK(check_state(state, m.tgt.n_layers));
  if (mode != 0) {   // time-synchronous search: candidate set, enough state rows, call number matches
    const q4_beam_state& ts = *state;
    if (!ts.nb_score || !ts.nb_u || !ts.nb_last_tok || !ts.nb_row || !ts.nb_origin || !ts.nb_hash ||
        !ts.nb_prev_hash || !ts.nb_n)
      return Q4_ERR_NULL;
    if (ts.tsd_smax < 0 || ts.tsd_smax > 3 || ts.rows_per_utt < W * (ts.tsd_smax + 1) || ts.rows_per_utt > 64)
      return Q4_ERR_DIM;
    const bool closing = iter % (ts.tsd_smax + 1) == ts.tsd_smax;
    if (closing != (mode == 2) || iter / (ts.tsd_smax + 1) >= T) return Q4_ERR_DIM;
  } else if (state->rows_per_utt != 0 && state->rows_per_utt < 2 * W) {
    return Q4_ERR_DIM;
  }
  const int V = m.V, D = m.D;
  if (V <= 1 || D <= 0 || D % 32 != 0 || m.E <= 0) return Q4_ERR_DIM;
  if (m.src.n_layers < 1 || m.src.n_layers > 2 || m.tgt.n_layers < 1 || m.tgt.n_layers > 2)
    return Q4_ERR_DIM;
  if (!m.pred_emb_q || !m.src.emb_q || !m.tgt.emb_q) return Q4_ERR_NULL;
  Q4_CHECK(check_model_lstm(m.pred_lstm, m.pred_emb_act));
  Q4_CHECK(check_mat(&m.pred_proj.w, D, m.pred_lstm.w_hh.k_pad));
  Q4_CHECK(check_act(&m.z_act));
  Q4_CHECK(check_mat(&m.joint_out.w, V, D));
  const q4_lm* lms[2] = {&m.src, &m.tgt};
  for (const q4_lm* lm : lms) {
    Q4_CHECK(check_model_lstm(lm->lstm[0], lm->emb_act));
    if (lm->n_layers == 2) Q4_CHECK(check_model_lstm(lm->lstm[1], lm->lstm[0].hid_act));
    const q4_lstm& last = lm->lstm[lm->n_layers - 1];
    Q4_CHECK(check_mat(&lm->bott.w, D, last.w_hh.k_pad));
    Q4_CHECK(check_act(&lm->bott_act));
    Q4_CHECK(check_mat(&lm->out.w, V, D));
  }
  if ((size_t)W * V * sizeof(float) > 200 * 1024) return Q4_ERR_UNSUPPORTED;
  const int32_t dims[4] = {B, W, V, D};
  if (workspace_bytes < q4_workspace_bytes(Q4_WS_BEAM, dims, 4)) return Q4_ERR_WORKSPACE;
  if (!aligned16(workspace) || !aligned16(e)) return Q4_ERR_ALIGN;

  cudaStream_t s = S(stream);
  const q4_beam_state& st = *state;
  const int N = B * W;
  // quantizer applications of one iteration: the cell outputs of the advanced networks, the two
  // bottleneck outputs, tanh(e * p)
  g_quant_calls += 1 + 1 + m.tgt.n_layers + 2 + 1;
  int joint_normalized = 0;   // the tensor-core joint kernel leaves log-probabilities, not logits
  // the first call of a frame of the time-synchronous search follows a frame close, which creates
  // no label extension: no network has anything to advance, only the joint runs
  const bool nets = !(mode != 0 && iter > 0 && iter % (state->tsd_smax + 1) == 0);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* zq = ws;
  ws += align_up((size_t)N * D);
  uint8_t* bq_src = ws;
  ws += align_up((size_t)N * D);
  uint8_t* bq_tgt = ws;
  ws += align_up((size_t)N * D);
  float* logits = reinterpret_cast<float*>(ws);
  ws += align_up((size_t)N * V * sizeof(float));
  int32_t* live = reinterpret_cast<int32_t*>(ws);
  ws += align_up((size_t)N * sizeof(int32_t));
  // pending advances of this iteration, compacted by the previous selection (or the reset)
  const int par = iter & 1;
  int32_t* c_src = st.pend_src + (size_t)par * N;
  int32_t* c_dst = st.pend_dst + (size_t)par * N;
  int32_t* c_tok = st.pend_tok + (size_t)par * N;
  const int32_t* n_active = st.pend_n + par;
  q4_beam_state cst = st;   // same state, pending advances in compacted order
  cst.adv_src = c_src;
  cst.adv_dst = c_dst;
  cst.adv_tok = c_tok;
  // tensor-core path: prepared int8 weights and room for the int8 operand scratch.  It is taken
  // for any number of rows: even 16 rows padded to one 128-row tile finish sooner than on the DP4A
  // kernels (measured 3x on a single utterance), since the time goes to streaming the weights
  const int Hp = m.pred_lstm.w_hh.k_pad, Hs = m.src.lstm[0].w_hh.k_pad, Ht = m.tgt.lstm[0].w_hh.k_pad;
  const int Ep = m.pred_lstm.w_ih.k_pad;
  const int32_t dims8[8] = {B, W, V, D, Ep, Hp, Hs, Ht};
  const bool use_mma = m.prepared != nullptr && m.src.n_layers == 1 &&
                       m.src.lstm[0].w_ih.k_pad == Ep && m.tgt.lstm[0].w_ih.k_pad == Ep &&
                       Hp % 128 == 0 && Hs % 128 == 0 && Ht % 128 == 0 && V % 32 == 0 &&
                       workspace_bytes >= q4_workspace_bytes(Q4_WS_BEAM, dims8, 8);
  if (use_mma) {
    const size_t Np = ((size_t)N + 127) / 128 * 128;
    const int Hmax = Hp > Hs ? (Hp > Ht ? Hp : Ht) : (Hs > Ht ? Hs : Ht);
    (void)Hmax;
    int8_t* xa8[3];   // embedding rows of the pending symbols: prediction, source LM, target LM
    for (int i = 0; i < 3; ++i) {
      xa8[i] = reinterpret_cast<int8_t*>(ws);
      ws += align_up(Np * Ep);
    }
    int8_t* ha8[4];   // previous cell outputs: prediction, source LM, target LM layers 1 and 2
    const int hdim[4] = {Hp, Hs, Ht, Ht};
    for (int i = 0; i < 4; ++i) {
      ha8[i] = reinterpret_cast<int8_t*>(ws);
      ws += align_up(Np * (size_t)hdim[i]);
    }
    int8_t* pred_h8 = reinterpret_cast<int8_t*>(ws);
    ws += align_up(Np * Hp);
    int8_t* src_h8 = reinterpret_cast<int8_t*>(ws);
    ws += align_up(Np * Hs);
    int8_t* tgt_h8[2];
    tgt_h8[0] = reinterpret_cast<int8_t*>(ws);
    ws += align_up(Np * Ht);
    tgt_h8[1] = reinterpret_cast<int8_t*>(ws);
    ws += align_up(Np * Ht);
    int8_t* bq8[2];
    bq8[0] = reinterpret_cast<int8_t*>(ws);
    ws += align_up(Np * D);
    bq8[1] = reinterpret_cast<int8_t*>(ws);
    ws += align_up(Np * D);
    int8_t* z8 = reinterpret_cast<int8_t*>(ws);
    const PrepPlan pp = plan_prepared(m);
    const uint8_t* pb = static_cast<const uint8_t*>(m.prepared);

    // at most 32 hypothesis rows (one utterance): the LSTM steps are bound by reading the weights once,
    // and a weight-streaming kernel reads them as stored (packed 4-bit), the state rows and embedding
    // rows too, so the gathers below are not needed
    const bool skinny =
        skinny_lstm_supported(N, Hp, Ep, m.pred_lstm.w_ih.bits, m.pred_lstm.w_hh.bits, m.pred_emb_act, m.pred_lstm.hid_act) &&
        skinny_lstm_supported(N, Hs, Ep, m.src.lstm[0].w_ih.bits, m.src.lstm[0].w_hh.bits, m.src.emb_act, m.src.lstm[0].hid_act) &&
        skinny_lstm_supported(N, Ht, Ep, m.tgt.lstm[0].w_ih.bits, m.tgt.lstm[0].w_hh.bits, m.tgt.emb_act, m.tgt.lstm[0].hid_act) &&
        (m.tgt.n_layers == 1 || skinny_lstm_supported(N, Ht, Ht, m.tgt.lstm[1].w_ih.bits, m.tgt.lstm[1].w_hh.bits,
                                                      m.tgt.lstm[0].hid_act, m.tgt.lstm[1].hid_act));
    // all gathers of the iteration in one launch: embedding rows by pending symbol, previous
    // cell-output codes by parent state row, unpacked to int8 operand rows
    if (nets && !skinny) {
      UnpackJobs uj;
      memset(&uj, 0, sizeof(uj));
      auto add = [&](const void* src, long long stride, const int32_t* idx, const q4_act& act, int k_pad,
                     int8_t* dst) {
        UnpackJob& j = uj.job[uj.n_jobs++];
        j.src = static_cast<const uint8_t*>(src);
        j.src_stride = stride;
        j.idx = idx;
        j.bits = act.bits;
        j.is_signed = act.is_signed;
        j.zp = act.zero_point;
        j.k_pad = k_pad;
        j.dst = dst;
        j.dst_stride = k_pad;
      };
      add(m.pred_emb_q, row_bytes(Ep, m.pred_emb_act.bits), cst.adv_tok, m.pred_emb_act, Ep, xa8[0]);
      add(m.src.emb_q, row_bytes(Ep, m.src.emb_act.bits), cst.adv_tok, m.src.emb_act, Ep, xa8[1]);
      add(m.tgt.emb_q, row_bytes(Ep, m.tgt.emb_act.bits), cst.adv_tok, m.tgt.emb_act, Ep, xa8[2]);
      add(st.pred_hq, row_bytes(Hp, m.pred_lstm.hid_act.bits), cst.adv_src, m.pred_lstm.hid_act, Hp, ha8[0]);
      add(st.src_hq, row_bytes(Hs, m.src.lstm[0].hid_act.bits), cst.adv_src, m.src.lstm[0].hid_act, Hs, ha8[1]);
      add(st.tgt_hq[0], row_bytes(Ht, m.tgt.lstm[0].hid_act.bits), cst.adv_src, m.tgt.lstm[0].hid_act, Ht, ha8[2]);
      if (m.tgt.n_layers == 2)
        add(st.tgt_hq[1], row_bytes(Ht, m.tgt.lstm[1].hid_act.bits), cst.adv_src, m.tgt.lstm[1].hid_act, Ht, ha8[3]);
      uj.n_rows = N;
      uj.n_rows_pad = (int)Np;
      uj.zero_tail = 0;   // rows beyond the pending advances feed tiles whose results are dropped
      uj.n_active = n_active;
      TagScope tag(TAG_MISC);
      Q4_TRY(launch_unpack_multi(uj, s, true));
    }
    // the three networks are independent until the selection: with two lent streams they run side
    // by side.  The call's own stream carries the chain that is critical: with many hypothesis rows
    // the target LM (two wide layers; the fork and the join would add to its path), with few rows
    // the prediction/joint chain, the only one with work in every iteration, which then runs
    // gather -> ... -> joint -> selection as programmatic dependents without an event in between
    // (measured: 16 utterances 18.8 -> 18.5 ms, one utterance 11.5 -> 11.2 ms; 64 utterances the other
    // way round, 49.7 -> 50.5 ms)
    const bool joint_on_call_stream = N <= 256;
    cudaStream_t sp = s, ss = s, stt = s;
    const bool forked = nets && st.aux_stream[0] && st.aux_stream[1] && st.aux_event[0] && st.aux_event[1] &&
                        st.aux_event[2];
    if (forked) {
      (joint_on_call_stream ? stt : sp) = reinterpret_cast<cudaStream_t>(st.aux_stream[0]);
      ss = reinterpret_cast<cudaStream_t>(st.aux_stream[1]);
      cudaEvent_t fork = reinterpret_cast<cudaEvent_t>(st.aux_event[0]);
      Q4_TRY(cudaEventRecord(fork, s));
      Q4_TRY(cudaStreamWaitEvent(joint_on_call_stream ? stt : sp, fork, 0));
      Q4_TRY(cudaStreamWaitEvent(ss, fork, 0));
    }
    // one LSTM layer of one network for every pending slot
    // `dep`: the previous launch on the same stream is a kernel of this library, so this one may
    // be launched as its programmatic dependent
    auto lstm_mma = [&](cudaStream_t s, bool dep, int tag_id, int li, const q4_lstm& L, const q4_act& x_act,
                        const int8_t* xa, const int8_t* ha, void* hq, float* c, int8_t* h8, int h_first = 0,
                        int trigger_early = 0) -> int {
      TagScope tag(tag_id);
      const int H = L.w_hh.k_pad, Kx = L.w_ih.k_pad;
      if (skinny) {
        // x rows: the embedding table by pending symbol, or (second layer) the first layer's fresh state rows
        const bool second = li == 3;
        SkinnyLstmArgs k;
        memset(&k, 0, sizeof(k));
        k.N = N;
        k.H = H;
        k.Kx = Kx;
        k.w_ih = static_cast<const uint8_t*>(L.w_ih.q);
        k.w_hh = static_cast<const uint8_t*>(L.w_hh.q);
        k.s_wih = L.w_ih.scale;
        k.s_whh = L.w_hh.scale;
        k.bias = L.bias;
        k.x = static_cast<const uint8_t*>(second ? st.tgt_hq[0] : li == 0 ? m.pred_emb_q : li == 1 ? m.src.emb_q : m.tgt.emb_q);
        k.x_stride = row_bytes(Kx, 4);
        k.x_idx = second ? cst.adv_dst : cst.adv_tok;
        k.x_signed = x_act.is_signed;
        k.x_zp = x_act.zero_point;
        k.x_scale = x_act.scale;
        k.hid_act = L.hid_act;
        k.hq_in = static_cast<const uint8_t*>(hq);
        k.c_in = c;
        k.src_row = cst.adv_src;
        k.dst_row = cst.adv_dst;
        k.hq_out = static_cast<uint8_t*>(hq);
        k.c_out = c;
        k.h8_out = h8;
        k.h8_ld = H;
        k.n_active = n_active;
        Q4_TRY(launch_skinny_lstm(k, s, dep));
        return Q4_OK;
      }
      MmaLstmArgs a;
      memset(&a, 0, sizeof(a));
      a.N = N;
      a.H = H;
      a.Kx_pad = Kx;
      a.sc_ih = reinterpret_cast<const float*>(pb + pp.lstm[li].sc_ih);
      a.sc_hh = reinterpret_cast<const float*>(pb + pp.lstm[li].sc_hh);
      a.bias = reinterpret_cast<const float*>(pb + pp.lstm[li].bias);
      a.x_scale = x_act.scale;
      a.hid_act = L.hid_act;
      a.out_act = L.hid_act;
      a.src_row = cst.adv_src;
      a.dst_row = cst.adv_dst;
      a.c_in = c;
      a.c_out = c;
      a.hq_out = static_cast<uint8_t*>(hq);
      a.hq_ld = row_bytes(H, L.hid_act.bits);
      a.h8_out = h8;
      a.h8_ld = H;
      a.status = st.status;
      a.n_active = n_active;
      a.premultiplied = 1;   // q4_prepare_model stored the products
      a.h_first = dep ? h_first : 0;
      a.trigger_early = trigger_early;
      Q4_TRY(launch_mma_lstm(a, xa, Kx, reinterpret_cast<const int8_t*>(pb + pp.lstm[li].xw), Kx, ha, H,
                             reinterpret_cast<const int8_t*>(pb + pp.lstm[li].hw), H, s, dep));
      return Q4_OK;
    };
    auto linear_mma = [&](cudaStream_t s, bool dep, int tag_id, int wi, const q4_linear& L, const int8_t* x8,
                          float x_scale, int epi, void* out, long long ldo, const int32_t* out_idx,
                          const q4_act* out_act, const int32_t* rows_active) -> int {
      TagScope tag(tag_id);
      Q4_TRY(launch_mma_gemm(x8, L.w.k_pad, N, reinterpret_cast<const int8_t*>(pb + pp.lin[wi]), L.w.k_pad,
                             L.w.rows, L.w.k_pad, epi, out, ldo, out_idx, L.w.scale, L.bias, x_scale, out_act,
                             st.status, rows_active, s, dep));
      return Q4_OK;
    };

    const bool fused_head = D == 256 && V <= 2048;   // the fused head kernel: 256-wide bottleneck, one cluster per row tile
    // 1a. prediction network, then the joint network for every live slot (stream sp)
    if (nets) {
      Q4_CHECK(lstm_mma(sp, !forked || joint_on_call_stream, TAG_PRED_LSTM, 0, m.pred_lstm, m.pred_emb_act, xa8[0], ha8[0], st.pred_hq,
                        st.pred_c, pred_h8));
      Q4_CHECK(linear_mma(sp, true, TAG_PRED_PROJ, 0, m.pred_proj, pred_h8, m.pred_lstm.hid_act.scale, EPI_F32,
                          st.pred_p, D, cst.adv_dst, nullptr, n_active));
    }
    {
      TagScope tag(TAG_JOINT);
      Q4_TRY(launch_joint_z(e, nullptr, st.t, B, W, st.pred_p, st.row, N, D, m.z_act, nullptr, z8, live, sp, true));
    }
    joint_normalized = fused_head ? 1 : 0;
    if (fused_head) {
      // output layer of the joint network with the log-softmax over the vocabulary in its epilogue
      TagScope tag(TAG_JOINT);
      LmHeadArgs ja;
      memset(&ja, 0, sizeof(ja));
      ja.N = N;
      ja.H = 0;
      ja.V = V;
      ja.q_scale = m.z_act.scale;
      ja.sc_out = m.joint_out.w.scale;
      ja.b_out = m.joint_out.bias;
      ja.lp = logits;
      ja.dst_row = live;
      ja.status = st.status;
      Q4_TRY(launch_mma_lmhead(ja, z8, D, nullptr, reinterpret_cast<const int8_t*>(pb + pp.lin[5]), sp, true));
    } else {
      Q4_CHECK(linear_mma(sp, true, TAG_JOINT, 5, m.joint_out, z8, m.z_act.scale, EPI_F32, logits, V, live, nullptr,
                          nullptr));
    }
    // 1b. source LM (stream ss) and target LM (stream stt)
    for (int which = 0; which < 2 && nets; ++which) {
      const q4_lm& lm = *lms[which];
      cudaStream_t sl = which == 0 ? ss : stt;
      const q4_lstm& L0 = lm.lstm[0];
      void* hq0 = which == 0 ? st.src_hq : st.tgt_hq[0];
      float* c0 = which == 0 ? st.src_c : st.tgt_c[0];
      int8_t* h8_0 = which == 0 ? src_h8 : tgt_h8[0];
      float* lp = which == 0 ? st.src_lp : st.tgt_lp;
      Q4_CHECK(lstm_mma(sl, (which == 1 && !joint_on_call_stream) || !forked, which == 0 ? TAG_SRC_LSTM : TAG_TGT_L1, which == 0 ? 1 : 2, L0, lm.emb_act,
                        xa8[which + 1], ha8[which + 1], hq0, c0, h8_0, 0, lm.n_layers == 2 ? 1 : 0));
      const int8_t* top8 = h8_0;
      const q4_lstm* last = &L0;
      if (lm.n_layers == 2) {
        const q4_lstm& L1 = lm.lstm[1];
        // layer 2 reads layer 1's output only as its input operand: its recurrent half starts
        // while layer 1 is still in its cell update
        Q4_CHECK(lstm_mma(sl, true, TAG_TGT_L2, 3, L1, L0.hid_act, h8_0, ha8[3], st.tgt_hq[1], st.tgt_c[1],
                          tgt_h8[1], 1, 0));
        top8 = tgt_h8[1];
        last = &L1;
      }
      const int head_tag = which == 0 ? TAG_SRC_HEAD : TAG_TGT_HEAD;
      if (fused_head) {
        // bottleneck, re-quantization, output layer and log-softmax in one kernel
        TagScope tag(head_tag);
        LmHeadArgs ha;
        memset(&ha, 0, sizeof(ha));
        ha.N = N;
        ha.H = last->w_hh.k_pad;
        ha.V = V;
        ha.x_scale = last->hid_act.scale;
        ha.sc_bott = lm.bott.w.scale;
        ha.b_bott = lm.bott.bias;
        ha.bott_act = lm.bott_act;
        ha.q_scale = lm.bott_act.scale;
        ha.sc_out = lm.out.w.scale;
        ha.b_out = lm.out.bias;
        ha.lp = lp;
        ha.dst_row = cst.adv_dst;
        ha.n_active = n_active;
        ha.status = st.status;
        Q4_TRY(launch_mma_lmhead(ha, top8, ha.H, reinterpret_cast<const int8_t*>(pb + pp.lin[which == 0 ? 1 : 3]),
                                 reinterpret_cast<const int8_t*>(pb + pp.lin[which == 0 ? 2 : 4]), sl, true));
      } else {
        Q4_CHECK(linear_mma(sl, true, head_tag, which == 0 ? 1 : 3, lm.bott, top8, last->hid_act.scale, EPI_QUANT8,
                            bq8[which], D, nullptr, &lm.bott_act, n_active));
        Q4_CHECK(linear_mma(sl, true, head_tag, which == 0 ? 2 : 4, lm.out, bq8[which], lm.bott_act.scale, EPI_F32, lp,
                            V, cst.adv_dst, nullptr, n_active));
      }
    }
    if (forked) {   // join: the call's stream waits for both side chains
      cudaEvent_t j0 = reinterpret_cast<cudaEvent_t>(st.aux_event[1]);
      cudaEvent_t j1 = reinterpret_cast<cudaEvent_t>(st.aux_event[2]);
      Q4_TRY(cudaEventRecord(j0, joint_on_call_stream ? stt : sp));
      Q4_TRY(cudaEventRecord(j1, ss));
      Q4_TRY(cudaStreamWaitEvent(s, j0, 0));
      Q4_TRY(cudaStreamWaitEvent(s, j1, 0));
    }
    if (!fused_head && nets) {  // log-softmax of both LMs' new rows in one launch
      TagScope tag(TAG_TGT_HEAD);
      Q4_TRY(launch_logsoftmax(st.src_lp, st.src_lp, N, V, V, cst.adv_dst, s, st.tgt_lp, n_active));
    }
  } else {
    // 1. pending advances -------------------------------------------------------------
    if (nets) {  // prediction network: embedding row -> LSTM -> projection to D
      const q4_lstm& L = m.pred_lstm;
      Q4_CHECK(advance_lstm(TAG_PRED_LSTM, L, m.pred_emb_q, row_bytes(L.w_ih.k_pad, m.pred_emb_act.bits), cst.adv_tok,
                            m.pred_emb_act, st.pred_hq, st.pred_c, cst, N, n_active, s));
      GemmArgs g = gemm_args(st.pred_hq, row_bytes(L.w_hh.k_pad, L.hid_act.bits), cst.adv_dst,
                             L.hid_act, N, m.pred_proj.w, m.pred_proj.bias, st.pred_p, D, cst.adv_dst);
      g.n_active = n_active;
      TagScope tag(TAG_PRED_PROJ);
      Q4_TRY(launch_gemm(g, EPI_F32, s));
    }
    for (int which = 0; which < 2 && nets; ++which) {
      const q4_lm& lm = *lms[which];
      void* hq0 = which == 0 ? st.src_hq : st.tgt_hq[0];
      float* c0 = which == 0 ? st.src_c : st.tgt_c[0];
      float* lp = which == 0 ? st.src_lp : st.tgt_lp;
      uint8_t* bq = which == 0 ? bq_src : bq_tgt;
      const q4_lstm& L0 = lm.lstm[0];
      Q4_CHECK(advance_lstm(which == 0 ? TAG_SRC_LSTM : TAG_TGT_L1, L0, lm.emb_q, row_bytes(L0.w_ih.k_pad, lm.emb_act.bits), cst.adv_tok,
                            lm.emb_act, hq0, c0, cst, N, n_active, s));
      const void* top = hq0;
      const q4_lstm* last = &L0;
      if (lm.n_layers == 2) {
        if (which == 0) return Q4_ERR_UNSUPPORTED;  // the state block holds one source-LM layer
        const q4_lstm& L1 = lm.lstm[1];
        Q4_CHECK(advance_lstm(TAG_TGT_L2, L1, hq0, row_bytes(L0.w_hh.k_pad, L0.hid_act.bits), cst.adv_dst,
                              L0.hid_act, st.tgt_hq[1], st.tgt_c[1], cst, N, n_active, s));
        top = st.tgt_hq[1];
        last = &L1;
      }
      GemmArgs gb = gemm_args(top, row_bytes(last->w_hh.k_pad, last->hid_act.bits), cst.adv_dst,
                              last->hid_act, N, lm.bott.w, lm.bott.bias, bq,
                              row_bytes(D, lm.bott_act.bits), nullptr);
      gb.out_act = lm.bott_act;
      gb.n_active = n_active;
      TagScope tag(which == 0 ? TAG_SRC_HEAD : TAG_TGT_HEAD);
      Q4_TRY(launch_gemm(gb, EPI_QUANT, s));
      GemmArgs go = gemm_args(bq, row_bytes(D, lm.bott_act.bits), nullptr, lm.bott_act, N, lm.out.w,
                              lm.out.bias, lp, V, cst.adv_dst);
      go.n_active = n_active;
      Q4_TRY(launch_gemm(go, EPI_F32, s));
      Q4_TRY(launch_logsoftmax(lp, lp, N, V, V, cst.adv_dst, s, nullptr, n_active));
    }

    // 2. joint network for every live slot at its frame -----------------------------------
    TagScope tag_joint(TAG_JOINT);
    Q4_TRY(launch_joint_z(e, nullptr, st.t, B, W, st.pred_p, st.row, N, D, m.z_act, zq, nullptr, live, s));
    GemmArgs gj = gemm_args(zq, row_bytes(D, m.z_act.bits), live, m.z_act, N, m.joint_out.w,
                            m.joint_out.bias, logits, V, nullptr);
    Q4_TRY(launch_gemm(gj, EPI_F32, s));
  }

  // 3. Eq. 1 proposals, merge, finished list, next beam --------------------------------
  BeamSelArgs sel;
  memset(&sel, 0, sizeof(sel));
  sel.logits = logits;
  sel.src_lp = st.src_lp;
  sel.tgt_lp = st.tgt_lp;
  sel.st = st;
  sel.B = B;
  sel.T = T;
  sel.W = W;
  sel.V = V;
  sel.iter = iter;
  sel.u_max = u_max;
  sel.lambda_t = lambda_t;
  sel.lambda_s = lambda_s;
  sel.rho = rho;
  sel.exact_only = select_exact_only();
  sel.normalized = joint_normalized;
  sel.mode = mode;
  TagScope tag_sel(TAG_SELECT);
  if (mode != 0)
    Q4_TRY(launch_tsd_select(sel, s, use_mma));
  else
    Q4_TRY(launch_beam_select(sel, s, use_mma));
  return Q4_OK;
}

int q4_traceback(const q4_beam_state* state, int32_t B, int32_t W, int32_t n_iters,
                 int32_t u_max, int32_t* tokens, int32_t* lens, float* scores, q4_stream stream) {
  Q4_CHECK(check_state(state, 1));
  if (!tokens || !lens || !scores) return Q4_ERR_NULL;
  if (B <= 0 || W <= 0 || W > 16 || n_iters < 0 || u_max <= 0) return Q4_ERR_DIM;
  Q4_TRY(launch_traceback(*state, B, W, n_iters, u_max, tokens, lens, scores, S(stream)));
  return Q4_OK;
}

}  // extern "C"
