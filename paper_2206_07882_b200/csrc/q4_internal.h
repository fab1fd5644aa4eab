// Internal launch interface between the translation units of the library.
#pragma once
#include "q4_common.cuh"

namespace q4 {

cudaError_t launch_gemm(const GemmArgs& a, int epi, cudaStream_t s);
cudaError_t launch_lstm(const LstmArgs2& a, int dirs, cudaStream_t s);
cudaError_t launch_logsoftmax(const float* in, float* out, int rows, int V, long long stride,
                              const int32_t* idx, cudaStream_t s, float* second = nullptr,
                              const int32_t* n_active = nullptr);
cudaError_t launch_joint_z(const float* e, const int32_t* frame_idx, const int32_t* t_arr, int B,
                           int W, const float* p, const int32_t* p_idx, int N, int D,
                           const q4_act& za, uint8_t* zq, int8_t* z8, int32_t* live_out,
                           cudaStream_t s, bool dependent = false);
cudaError_t launch_quantize(const void* x, bool fp16, long long rows, int k, int k_pad,
                            const q4_act& a, int mode, int n_groups, const float* scale_vec,
                            uint8_t* out, float* group_scale_out, cudaStream_t s);
cudaError_t launch_features(const float* mel, int B, int T100, int M, void* out, cudaStream_t s);

struct BeamSelArgs {
  const float* logits;      // [B*W, V] joint logits (bias included), rows of empty slots ignored
  const float* src_lp;      // [R, V]
  const float* tgt_lp;      // [R, V]
  q4_beam_state st;
  int32_t B, T, W, V, iter, u_max;
  float lambda_t, lambda_s, rho;
  int32_t mode;             // 0 alignment-length synchronous; 1 / 2 time-synchronous inner call / frame close
  int32_t normalized;       // 1 = `logits` already holds log-probabilities (rows sum to one)
  int32_t exact_only;       // 1 = skip the register-resident fast filter (the exact threshold path alone)
};
cudaError_t launch_beam_select(const BeamSelArgs& a, cudaStream_t s, bool dependent = false);
cudaError_t launch_tsd_select(const BeamSelArgs& a, cudaStream_t s, bool dependent = false);
cudaError_t launch_beam_init(const q4_beam_state& st, int B, int W, int n_iters, cudaStream_t s);
cudaError_t launch_traceback(const q4_beam_state& st, int B, int W, int n_iters, int u_max,
                             int32_t* tokens, int32_t* lens, float* scores, cudaStream_t s);

// Launch-site tags for the optional event timing hook (q4_timing_set).
enum { TAG_NONE = 0, TAG_QUANT = 1, TAG_ENC_GEMM = 2, TAG_ENC_STEP = 3, TAG_LINEAR = 4,
       TAG_PRED_LSTM = 5, TAG_PRED_PROJ = 6, TAG_SRC_LSTM = 7, TAG_SRC_HEAD = 8, TAG_TGT_L1 = 9,
       TAG_TGT_L2 = 10, TAG_TGT_HEAD = 11, TAG_JOINT = 12, TAG_SELECT = 13, TAG_MISC = 14,
       TAG_COUNT = 15 };
extern int g_tag;   // tag of the launches being issued
struct TagScope {
  int prev;
  explicit TagScope(int t) : prev(g_tag) { g_tag = t; }
  ~TagScope() { g_tag = prev; }
};
void timing_begin(cudaStream_t s);
void timing_end(cudaStream_t s);
void timing_set(uint32_t mask, cudaEvent_t* start, cudaEvent_t* stop, int32_t* tags, int cap);
int timing_count();

// ---- tensor-core path (q4_mma.cu)
struct MmaLstmArgs {
  int32_t N, H, Kx_pad;
  const int32_t* acc_pre;   // optional precomputed input accumulators [row, 4H] in 4*cell+gate order
  long long acc_pre_ld;
  const float* sc_ih;       // per weight row, 4*cell+gate order
  const float* sc_hh;
  const float* bias;
  float x_scale;
  const float* x_scale_vec;
  int32_t x_scale_mod;
  q4_act hid_act, out_act;
  const int32_t* src_row;   // state row read by launch row n (nullptr = n, negative = zero state)
  const int32_t* dst_row;   // state row written (nullptr = n, negative = row inactive)
  const float* c_in;
  float* c_out;
  uint8_t* hq_out;          // packed recurrent codes at dst row (nullable)
  long long hq_ld;
  int8_t* h8_out;           // int8 recurrent codes at launch row n (nullable)
  long long h8_ld;
  uint8_t* yq_out;          // packed out_act codes at launch row n (nullable)
  long long yq_ld;
  float* h_f32;
  int32_t* dbg_ih;          // optional [n, 4H] gate-major
  int32_t* dbg_hh;
  long long dbg_ld;
  int32_t* status;
  const int32_t* n_active;  // optional: rows >= *n_active carry no work (tiles beyond it exit at once)
  int32_t h_first;          // 1: only the input operand comes from the previous kernel of the stream, so
                            // the recurrent half of the K loop runs before waiting for that kernel
  int32_t trigger_early;    // 1: let the next kernel of the stream start beside this one
  int32_t premultiplied;    // 1: sc_ih = x_scale * row scale and sc_hh = hidden scale * row scale already
};
struct LmHeadArgs {
  int32_t N, H, V;            // launch rows, LSTM width (K of the bottleneck; 0 = no bottleneck: the
                              // operand h8 is [N, 256] and feeds the output layer directly), vocabulary
  float x_scale;              // scale of the cell-output codes feeding the bottleneck
  const float* sc_bott;       // [256] bottleneck row scales
  const float* b_bott;        // [256] bias (nullable)
  q4_act bott_act;            // quantizer of the bottleneck output
  float q_scale;              // = bott_act.scale
  const float* sc_out;        // [V] output-layer row scales
  const float* b_out;         // [V] bias (nullable)
  float* lp;                  // [*, V] log-probabilities, row dst_row[n]
  const int32_t* dst_row;     // nullptr = n, negative = skip
  const int32_t* n_active;
  int32_t* status;
};
cudaError_t launch_mma_lmhead(const LmHeadArgs& a, const int8_t* h8, long long h_pitch, const int8_t* wb8,
                              const int8_t* wo8, cudaStream_t s, bool dependent = false);
enum { EPI_QUANT8 = 3,      // re-quantize and store (code - zero_point) as int8, one per byte
       EPI_JOINTZ = 4 };    // tanh(other factor * value), quantized, stored like EPI_QUANT8
cudaError_t launch_unpack_rows(const void* src, long long src_stride, const int32_t* idx,
                               const q4_act& act, int k_pad, int n_rows, int8_t* dst,
                               long long dst_stride, int col0, int n_rows_pad, cudaStream_t s,
                               int32_t* clear_status = nullptr, bool dependent = false);
// clear_status: 64 status words zeroed by the kernel's first block (replaces a memset node in front of a
// call); dependent: launched as a programmatic dependent (the kernel waits for its predecessor itself)
struct UnpackJob {
  const uint8_t* src;       // packed code rows
  long long src_stride;
  const int32_t* idx;       // source row of launch row n (negative = zero row)
  int32_t bits, is_signed, zp, k_pad;
  int8_t* dst;              // int8 [n_rows_pad, k_pad], pitch dst_stride
  long long dst_stride;
};
struct UnpackJobs {
  UnpackJob job[8];
  int32_t n_jobs, n_rows, n_rows_pad, zero_tail;
  const int32_t* n_active;
};
cudaError_t launch_unpack_multi(const UnpackJobs& jobs, cudaStream_t s, bool dependent = false);
cudaError_t launch_prepare_w(const q4_mat& w, int interleave, int8_t* dst, long long dst_stride,
                             int col0, cudaStream_t s);
cudaError_t launch_prepare_vec(const float* src, int rows, int interleave, float* dst, cudaStream_t s,
                               float mul = 1.0f);
cudaError_t launch_mma_gemm(const int8_t* x8, long long x_pitch, int M, const int8_t* w8,
                            long long w_pitch, int J, int K, int epi, void* out, long long ldo,
                            const int32_t* out_idx, const float* w_scale, const float* bias,
                            float x_scale, const q4_act* out_act, int32_t* status,
                            const int32_t* n_active, cudaStream_t s, bool dependent = false,
                            const float* mul_e = nullptr, const int32_t* mul_idx = nullptr);
void test_wait_expiry_set(int skip_producer, uint32_t wait_limit);
cudaError_t launch_mma_lstm(const MmaLstmArgs& a, const int8_t* xa, long long xa_pitch,
                            const int8_t* xw, long long xw_pitch, const int8_t* ha, long long ha_pitch,
                            const int8_t* hw, long long hw_pitch, cudaStream_t s, bool dependent = false);

// ---- weight-streaming LSTM step for at most 32 rows (q4_skinny.cu)
struct SkinnyLstmArgs {
  int32_t N, H, Kx;         // launch rows (<= 32), cells, input width (both multiples of 128)
  const uint8_t* w_ih;      // packed 4-bit [4H, Kx], gate blocks i, f, g, o
  const uint8_t* w_hh;      // packed 4-bit [4H, H]
  const float* s_wih;       // [4H] row scales
  const float* s_whh;
  const float* bias;        // [4H] or null
  const uint8_t* x;         // packed 4-bit input code rows, row n at x + x_idx[n] * x_stride
  long long x_stride;
  const int32_t* x_idx;     // null = n, negative = zero row
  int32_t x_signed, x_zp;
  float x_scale;
  q4_act hid_act;
  const uint8_t* hq_in;     // packed state rows [*, H/2], row src_row[n] (negative = zero state)
  const float* c_in;        // [*, H], same rows
  const int32_t* src_row;   // null = n
  const int32_t* dst_row;   // null = n, negative = row inactive
  uint8_t* hq_out;          // packed codes at dst row
  float* c_out;
  int8_t* h8_out;           // int8 codes at launch row n (nullable)
  long long h8_ld;
  const int32_t* n_active;  // optional device count: rows >= *n_active carry no work
};
bool skinny_lstm_supported(int N, int H, int Kx, int w_bits_ih, int w_bits_hh, const q4_act& x_act,
                           const q4_act& hid_act);
cudaError_t launch_skinny_lstm(const SkinnyLstmArgs& a, cudaStream_t s, bool dependent = false);

// ---- persistent encoder recurrence (q4_recurrent.cu)
struct EncRecDir {
  const int8_t* w_hh;       // int8 [4H, H], rows in 4*cell+gate order
  const float* sc_ih;       // [4H] in the same order
  const float* sc_hh;
  const float* bias;
  const int32_t* acc_pre;   // input accumulators [T*B, 4H], columns in 4*cell+gate order
  uint8_t* yq;              // layer output codes, already offset to this direction's columns
  int32_t* dbg_ih;          // optional [T, B, dirs, 4H] gate-major, offset to this direction
  int32_t* dbg_hh;
  uint8_t* hq_n;            // optional final codes [B, H], this direction
  float* c_n;               // optional final cell state [B, H], this direction
};
struct EncRecArgs {
  EncRecDir d[2];
  int32_t T, B, H, dirs, n_groups;
  int32_t w_bits;           // storage width of the recurrent weights the int8 copies were made from
  int32_t* status;          // device status word: receives Q4_ERR_TIMEOUT when a bounded wait expires
  float x_scale;
  const float* x_scale_b;
  q4_act hid_act, out_act;
  long long yq_ld;          // bytes per (t, b) output row
  long long dbg_ld;         // elements per (t, b) debug row
  // One group of 8 sequences more than clusters (time-sliced kernel): set by the launcher from the
  // scratch below, which the caller provides (nullptr = that kernel is not used)
  int32_t ncl[2];           // clusters of each direction
  int32_t sliced[2];        // 1: the direction's clusters take turns at its last group
  int32_t groups;           // groups of 8 sequences per direction
  int32_t win[9];           // cluster j of a sliced direction advances the shared group over steps [win[j], win[j+1])
  int32_t* flags;           // [2][8] hand-over counters, zero before the launch
  uint8_t* hand_h[2];       // [8][8][H / 8] hidden codes of the shared group at a hand-over, per direction
  float* hand_c[2];         // [8][H] its cell states
};
bool enc_recurrent_supported(int H, int B, int dirs);
int enc_recurrent_sliced_set(int enabled);   // returns the previous setting
// Which recurrence kernel a layer takes and how its groups of sequences are laid on clusters (host only).
struct EncRecPlan {
  int32_t kernel;           // 0: general kernel (int8 weights in shared memory), 1: packed weights in registers,
                            // groups_per_cluster groups per cluster, 2: kernel whose clusters may take turns
  int32_t groups_per_cluster;
  int32_t ncl[2], sliced[2], groups, max_clusters;
  int32_t win[9];
};
EncRecPlan enc_recurrent_plan(int T, int B, int dirs, int H, int w_bits, int hid_bits, bool hid_signed,
                              bool per_sequence_scale, bool dump, bool scratch);
cudaError_t launch_enc_recurrent(EncRecArgs a, cudaStream_t s);

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

// Kernel launch with optional attributes: `dependent` asks for programmatic stream
// serialization (the kernel calls pdl_wait() before it touches its inputs), cluster_x > 1 for a
// thread-block cluster along x.
extern int g_dependent_launch;   // 0 switches the attribute off everywhere
template <typename... KA, typename... A>
inline cudaError_t launch_ex(void (*kern)(KA...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                             bool dependent, unsigned cluster_x, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[2];
  unsigned n = 0;
  if (cluster_x > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = cluster_x;
    at[n].val.clusterDim.y = 1;
    at[n].val.clusterDim.z = 1;
    ++n;
  }
  if (dependent && g_dependent_launch) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<A&&>(args)...);
}

}  // namespace q4
