// Internal launch interface between the translation units of the library.
#pragma once
#include "q4_common.cuh"

namespace q4 {

cudaError_t launch_gemm(const GemmArgs& a, int bits, int epi, cudaStream_t s);
cudaError_t launch_lstm(const LstmArgs2& a, int dirs, int x_bits, int h_bits, cudaStream_t s);
cudaError_t launch_logsoftmax(const float* in, float* out, int rows, int V, long long stride,
                              const int32_t* idx, cudaStream_t s);
cudaError_t launch_joint_z(const float* e, const int32_t* frame_idx, const int32_t* t_arr, int B,
                           int W, const float* p, const int32_t* p_idx, int N, int D,
                           const q4_act& za, uint8_t* zq, int32_t* live_out, cudaStream_t s);
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
};
cudaError_t launch_beam_select(const BeamSelArgs& a, cudaStream_t s);
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

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

}  // namespace q4
