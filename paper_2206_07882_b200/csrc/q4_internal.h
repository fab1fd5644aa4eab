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

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

}  // namespace q4
