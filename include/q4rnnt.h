/*
 * q4rnnt — INT4 x INT4 RNN-T inference with density-ratio LM fusion on one GPU.
 *
 * C ABI of the CUDA library.  All tensor pointers are DEVICE pointers owned by
 * the caller unless a parameter says "host"; they must be 16-byte aligned.  No
 * entry point allocates, frees, or keeps a copy of anything; work is enqueued
 * on the stream passed last and the call returns without synchronising (except
 * q4_poll_status).  Every function returns 0 on success or a negative Q4_ERR_*;
 * argument errors are detected on the host before anything is launched.
 *
 * Number formats
 *   codes, 4 bit : two per byte, element 2i in bits 0-3, element 2i+1 in bits
 *                  4-7; two's complement when signed, plain when unsigned.
 *   codes, 8 bit : one per byte, two's complement (signed only).
 *   codes, 2 bit : weights only (the 2-bit weight rows of the paper's Table 1): four per
 *                  byte, element 4i+j in bits 2j, 2j+1, two's complement (-2..1).
 *   rows         : row-major, k_pad elements per row, k_pad a multiple of 32 (of 64 for
 *                  2-bit weights: rows are multiples of 16 bytes), elements k..k_pad-1 hold
 *                  the code of the real value 0 (0 for signed codes, the zero point for
 *                  unsigned ones).
 *   weights      : symmetric signed codes with one fp32 scale per output row
 *                  (W[j,k] ~ scale[j] * q[j,k]); biases and LSTM cell states
 *                  are fp32 and never quantized (paper Section 3.2).
 *   LSTM gates   : the 4H rows of w_ih / w_hh / bias are ordered i, f, g, o.
 * Weights may be stored at 2, 4 or 8 bits and activations at 4 or 8 bits in any combination
 * (the paper's mixed assignments: 8-bit first layer, 2-bit weights with 4-bit activations);
 * a weight matrix and the activation rows it multiplies share k_pad.
 */
#ifndef Q4RNNT_H_
#define Q4RNNT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define Q4_OK 0
#define Q4_ERR_NULL (-1)        /* a required pointer is NULL */
#define Q4_ERR_DIM (-2)         /* a size is non-positive or inconsistent */
#define Q4_ERR_ALIGN (-3)       /* a pointer or k_pad breaks the alignment rule */
#define Q4_ERR_BITS (-4)        /* bit width not supported (weights 2/4/8, activations 4/8) */
#define Q4_ERR_WORKSPACE (-5)   /* workspace smaller than q4_workspace_bytes says */
#define Q4_ERR_UNSUPPORTED (-6) /* valid request this build does not implement */
#define Q4_ERR_CUDA (-7)        /* a CUDA runtime call failed (launch error) */
#define Q4_ERR_TIMEOUT (-8)     /* a bounded device-side wait expired */

typedef void* q4_stream; /* a cudaStream_t, passed as an opaque handle (NULL = default stream) */
/* All work of a call is enqueued on its stream, in stream order with whatever the caller enqueued before.
 * Kernels of the tensor-core paths are launched with programmatic stream serialization: one may be
 * scheduled while its predecessor in the stream is draining, but every kernel waits for the completion of
 * its predecessor (and the visibility of its writes) before it reads anything, so results never depend on
 * it. */

/* Integer weight matrix [rows, k_pad] with per-row scales (device pointers). */
typedef struct {
  const void* q;
  const float* scale;
  int32_t rows, k, k_pad, bits;
} q4_mat;

/* Constants of one activation quantizer (paper Eq. 2, Eq. 3):
 *   code = clamp(rne(x * inv_scale) + zero_point, lo, hi),  x_q = scale * (code - zero_point)
 * rne = round half to even; [lo,hi] = [-2^(b-1), 2^(b-1)-1] when is_signed (symmetric
 * quantizer, zero_point 0) or [0, 2^b-1] otherwise (asymmetric). */
typedef struct {
  float scale, inv_scale;
  int32_t zero_point, bits, is_signed;
} q4_act;

/* Fill *out (host) for a symmetric quantizer with boundary alpha (Section 3.1):
 * scale = alpha / (2^(b-1) - 1), inv_scale = 1 / scale, both rounded to fp32. */
int q4_act_symmetric(float alpha, int32_t bits, q4_act* out);
/* Fill *out (host) for the asymmetric quantizer of Eq. 2 with boundaries lo < hi:
 * scale = (hi - lo) / (2^b - 1), zero_point = clamp(rne(-lo / scale), 0, 2^b - 1). */
int q4_act_asymmetric(float lo, float hi, int32_t bits, q4_act* out);

/*
 * quantize_pack_int4 — Eq. 2 on a [rows, k] matrix of fp16 or fp32 values, written as
 * packed codes [rows, k_pad] (4 or 8 bit per act->bits).  (Section 3.1.)
 *   mode 0 (FIX / learned constants): `act` (host) gives the quantizer.
 *   mode 1 (MAX boundary): symmetric, boundary = largest magnitude over each group; row r
 *          belongs to group r % n_groups (time-major [T,B,*] data with n_groups = B gives one
 *          boundary per utterance).  The per-group scale is written to group_scale_out
 *          [n_groups] (device); an all-zero group gets boundary 1.  act->bits selects the width.
 *   mode 2 (weights): symmetric, row r uses scale per_row_scale[r] (device), act->bits wide.
 *   Modes 1 and 2 also accept act->bits = 2 (weight storage; k_pad a multiple of 64).
 * x_is_fp16: 1 = half precision input, 0 = fp32.  x rows are dense (k values per row).
 */
int quantize_pack_int4(const void* x, int32_t x_is_fp16, int64_t rows, int32_t k, int32_t k_pad,
                       const q4_act* act, int32_t mode, int32_t n_groups,
                       const float* per_row_scale, void* q_out, float* group_scale_out,
                       q4_stream stream);

/*
 * qlstm_layer_forward — one uni- or bidirectional quantized LSTM layer over a batch of
 * sequences (Sections 3.2 and 3.4).  Time-major.
 *   xq    [T, B, kx_pad] codes of the layer input, quantizer x_act (zero_point honoured);
 *         x_scale_b (nullable, [B]) overrides x_act.scale per sequence.
 *   w_ih  [dirs] host array of matrices [4H, kx_pad]; w_hh [dirs] of [4H, H]; bias [dirs]
 *         host array of device pointers [4H] (entries or the array may be NULL = no bias).
 *   Direction 1 consumes the sequence backwards with its own weights.
 *   Per step and direction: int32 MACs of the input and of the previous cell-output codes,
 *   de-quantization, sigmoid/tanh gates, c_t = f*c + i*g (fp32), h_t = o*tanh(c_t), and h_t
 *   is quantized ONCE at the cell output with hid_act; that code is the next step's
 *   recurrent input.  yq [T, B, dirs*H] receives the code of h_t under out_act (the next
 *   layer's input quantizer: same boundary, possibly another bit width; made from the same
 *   fp32 h_t), directions concatenated [forward | backward].
 *   hq_n [dirs, B, H] codes (hid_act) and c_n [dirs, B, H] fp32 receive the final states
 *   (nullable).  dbg_acc_ih / dbg_acc_hh [T, B, dirs, 4H] int32 (nullable) receive the raw
 *   accumulators for parity checks.  h0 = c0 = 0.
 *   workspace: scratch of q4_workspace_bytes(Q4_WS_LSTM_LAYER, {T,B,dirs,H}) bytes (DP4A input
 *   projection) or q4_workspace_bytes(Q4_WS_LSTM_LAYER, {T,B,dirs,H,kx_pad}) bytes (adds room for
 *   int8 operand copies, which selects the tensor-core input projection when T*B >= 128).
 *   Its first 4 bytes are a status word for q4_poll_status (bounded device waits).
 */
int qlstm_layer_forward(const void* xq, const q4_act* x_act, const float* x_scale_b, int32_t T,
                        int32_t B, int32_t dirs, const q4_mat* w_ih, const q4_mat* w_hh,
                        const float* const* bias, const q4_act* hid_act, const q4_act* out_act,
                        void* yq, void* hq_n, float* c_n, int32_t* dbg_acc_ih,
                        int32_t* dbg_acc_hh, void* workspace, size_t workspace_bytes,
                        q4_stream stream);

/*
 * qlstm_step — one LSTM time step for N independent rows (prediction network and LM
 * building block; Sections 2 and 3.2).
 *   xq [*, kx_pad] codes; row n reads xq row x_row_idx[n] when x_row_idx is given (an
 *   embedding lookup into a pre-quantized table), else row n.
 *   hq_in [N, H] codes (hid_act), c_in [N, H] fp32; c_out may alias c_in, hq_out must not
 *   alias hq_in (every output cell reads the whole previous row).
 *   h_f32_out [N, H] (nullable) receives the fp32 cell output before quantization;
 *   dbg_acc_ih / dbg_acc_hh [N, 4H] int32 (nullable).
 *   hq_out == NULL (then h_f32_out is required) leaves the cell output unquantized: the "Inner"
 *   placement of Section 3.4, where every cell quantizes its two inputs on entry instead
 *   (quantize_pack_int4 on x_t and on the previous real-valued cell output, then this call).
 *   prepared / workspace (all nullable): with the buffer filled by q4_prepare_lstm for these weights
 *   and a workspace of q4_workspace_bytes(Q4_WS_LSTM_STEP, {N, kx_pad, H}) bytes, calls with N >= 128
 *   and H a multiple of 128 run on the tensor cores (same results, bit for bit); otherwise, and
 *   always without them, the DP4A kernel reads the packed weights directly.
 */
int qlstm_step(const void* xq, const q4_act* x_act, const int32_t* x_row_idx, const void* hq_in,
               const float* c_in, int32_t N, const q4_mat* w_ih, const q4_mat* w_hh,
               const float* bias, const q4_act* hid_act, void* hq_out, float* c_out,
               float* h_f32_out, int32_t* dbg_acc_ih, int32_t* dbg_acc_hh, const void* prepared,
               void* workspace, size_t workspace_bytes, q4_stream stream);

/* One-time int8 operands of an LSTM's weights for the tensor-core path of qlstm_step (weights are
 * quantized once, activations at every step: Section 3.2): rows reordered to 4*cell+gate, row
 * scales and bias in the same order.  buffer: device, q4_prepared_lstm_bytes bytes, caller-owned.
 * q4_prepare_linear: the same for a linear layer (q4_linear_forward, qjoint_logprobs). */
size_t q4_prepared_lstm_bytes(const q4_mat* w_ih, const q4_mat* w_hh);
int q4_prepare_lstm(const q4_mat* w_ih, const q4_mat* w_hh, const float* bias, void* buffer, size_t bytes,
                    q4_stream stream);
size_t q4_prepared_linear_bytes(const q4_mat* w);
int q4_prepare_linear(const q4_mat* w, void* buffer, size_t bytes, q4_stream stream);

/*
 * q4_linear_forward — quantized linear layer (Section 3.2): out[m, j] = acc[m, j] *
 * (x_act.scale * w.scale[j]) + bias[j], fp32, out [M, w.rows].  Used for the encoder ->
 * joint projection.  dbg_acc [M, w.rows] int32 nullable.  prepared / workspace (nullable): with
 * the buffer of q4_prepare_linear and q4_workspace_bytes(Q4_WS_LINEAR, {M, k_pad}) bytes, calls
 * with M >= 128 and no dbg_acc run on the tensor cores.
 */
int q4_linear_forward(const void* xq, const q4_act* x_act, int32_t M, const q4_mat* w,
                      const float* bias, float* out, int32_t* dbg_acc, const void* prepared,
                      void* workspace, size_t workspace_bytes, q4_stream stream);

/*
 * qjoint_logprobs — joint network (Section 2): the prediction-network cell output codes pq
 * [N, Hp] (p_act) are projected to D dims (w_pred, b_pred), combined multiplicatively with
 * the projected encoder frame e[frame_idx[n]] ([*, D] fp32), z = tanh(e * p), z is quantized
 * with z_act, passed through the output layer (w_out [V, D], b_out) and a log-softmax.
 * logp [N, V] fp32.  workspace: q4_workspace_bytes(Q4_WS_JOINT, {N, D}).
 * prepared_pred / prepared_out (nullable): buffers of q4_prepare_linear for w_pred and w_out; with
 * both, a workspace of q4_workspace_bytes(Q4_WS_JOINT, {N, D, Hp_pad}) bytes, N >= 128 and V a
 * multiple of 32 the call runs on the tensor cores in three launches (the projection's epilogue forms
 * tanh(e * p) and quantizes it; the output layer's epilogue takes the log-softmax).
 */
int qjoint_logprobs(const float* e, const int32_t* frame_idx, const void* pq, const q4_act* p_act,
                    int32_t N, const q4_mat* w_pred, const float* b_pred, const q4_act* z_act,
                    const q4_mat* w_out, const float* b_out, float* logp, const void* prepared_pred,
                    const void* prepared_out, void* workspace, size_t workspace_bytes, q4_stream stream);

/*
 * qjoint_logprobs_static — qjoint_logprobs for callers that cannot allocate device memory when
 * they call (a latency-critical decoding thread that must not wait on the allocator, a host
 * that forbids allocations after start-up, a process in which another thread is capturing a
 * stream).  The paper has no counterpart: this is the same computation with the workspace
 * replaced by a fixed array inside the library's device image, so the call allocates nothing.
 *   Limit: N * D <= 65536 (D = w_pred->rows), about 320 KB of device memory that every GPU
 *   loading the library keeps until the process exits; larger problems get Q4_ERR_WORKSPACE.
 *   The first call on each device looks up the array's device address (with that device
 *   current); make that first call before starting any stream capture.  The address is
 *   kept for the life of the process: after a cudaDeviceReset reload the library.
 *   All calls on a device share the one array: calls that overlap on the GPU (different
 *   streams) race with each other; calls on one stream are ordered and safe.  Nothing in the
 *   array needs clearing, each call overwrites what it reads.
 */
int qjoint_logprobs_static(const float* e, const int32_t* frame_idx, const void* pq,
                           const q4_act* p_act, int32_t N, const q4_mat* w_pred,
                           const float* b_pred, const q4_act* z_act, const q4_mat* w_out,
                           const float* b_out, float* logp, q4_stream stream);

/* One LSTM layer / linear layer inside a model description. */
typedef struct {
  q4_mat w_ih, w_hh;
  const float* bias;
  q4_act hid_act;
} q4_lstm;
typedef struct {
  q4_mat w;
  const float* bias;
} q4_linear;
/* LSTM language model: embedding (pre-quantized table [V, E_pad] codes under emb_act) ->
 * n_layers LSTM -> bottleneck (H -> D, fp32) -> quantize (bott_act) -> output (D -> V). */
typedef struct {
  const void* emb_q;
  q4_act emb_act;
  int32_t n_layers;
  q4_lstm lstm[2];
  q4_linear bott;
  q4_act bott_act;
  q4_linear out;
} q4_lm;
/* Everything the beam step needs (host struct of device pointers). */
typedef struct {
  int32_t V, E, D;
  const void* pred_emb_q; /* [V, E_pad] codes under pred_emb_act */
  q4_act pred_emb_act;
  q4_lstm pred_lstm;
  q4_linear pred_proj; /* Hp -> D */
  q4_act z_act;
  q4_linear joint_out; /* D -> V */
  q4_lm src, tgt;
  void* prepared; /* NULL, or the buffer filled by q4_prepare_model (tensor-core operands) */
} q4_model;

/* Optional one-time weight preparation for the tensor-core search path (weights are
 * quantized once, activations at every step: Section 3.2).  Writes int8, gate-interleaved
 * copies of the step weights into `buffer` (device, q4_prepared_bytes(model) bytes, owned by
 * the caller, must outlive the model's use) and sets model->prepared.  With prepared == NULL
 * the search uses the DP4A kernels on the packed weights. */
size_t q4_prepared_bytes(const q4_model* model);
int q4_prepare_model(q4_model* model, void* buffer, size_t bytes, q4_stream stream);

/*
 * Caller-owned search state for B utterances x W beam slots.  R = B * 2W "state rows" hold
 * network states (a label extension writes a fresh row; a blank extension keeps its
 * parent's row, so nothing is copied).  Sizes in elements; codes packed as above.
 */
typedef struct {
  /* per state row */
  void* pred_hq;    /* [R, Hp] codes */
  float* pred_c;    /* [R, Hp] */
  float* pred_p;    /* [R, D]  projected prediction output */
  void* src_hq;     /* [R, Hs] codes */
  float* src_c;     /* [R, Hs] */
  float* src_lp;    /* [R, V]  log P_src(. | labels) */
  void* tgt_hq[2];  /* [R, Ht] codes per layer */
  float* tgt_c[2];  /* [R, Ht] */
  float* tgt_lp;    /* [R, V]  log P_tgt(. | labels) */
  /* per slot [B*W] */
  float* score;
  int32_t* t;         /* frames consumed */
  int32_t* u;         /* labels emitted */
  uint64_t* hash;     /* hash of the label string */
  uint64_t* prev_hash;/* hash of the string without its last label */
  int32_t* last_tok;
  int32_t* row;       /* state row of the slot, -1 = slot empty */
  int32_t* adv_src;   /* pending network advance: state row to read (-1 = zero state) */
  int32_t* adv_dst;   /* row to write (-1 = nothing pending) */
  int32_t* adv_tok;   /* symbol to feed */
  /* the pending advances again, compacted (only slots with adv_dst >= 0, any order), double
   * buffered by iteration parity: entry a of list p is at [p * B*W + a], pend_n[p] entries */
  int32_t* pend_src;  /* [2, B*W] */
  int32_t* pend_dst;  /* [2, B*W] */
  int32_t* pend_tok;  /* [2, B*W] */
  int32_t* pend_n;    /* [2] */
  /* history [n_iters, B, W] */
  int32_t* bp_parent; /* slot in the previous beam, -1 = empty */
  int32_t* bp_token;  /* 0 = blank */
  float* bp_score;
  /* finished hypotheses, best first [B, W] */
  float* fin_score;
  int32_t* fin_iter;  /* iteration at which it consumed the last frame */
  int32_t* fin_slot;  /* its slot in the beam entering that iteration */
  int32_t* fin_n;     /* [B] */
  int32_t* status;    /* [1] device status word, 0 = ok */
  /* Optional concurrency (host handles, all NULL = everything on the call's stream): two more
   * cudaStream_t and three cudaEvent_t (created without timing) owned by the caller.  The step
   * then runs the prediction/joint chain and the source-LM chain on the auxiliary streams,
   * forked from and joined back into the call's stream, so the call's stream still orders
   * the whole step. */
  void* aux_stream[2];
  void* aux_event[3];
  /* Time-synchronous search only (modes 1 and 2 of dr_fusion_beam_step; leave zero / NULL for the
   * alignment-length synchronous search).  tsd_smax: at most that many labels per frame (0..3).
   * rows_per_utt: state rows per utterance; 0 means 2W; the time-synchronous search needs
   * W (tsd_smax + 1) <= 64 of them (R = B * rows_per_utt then).  nb_*: the candidate set of the next
   * frame, CB = W (tsd_smax + 1) entries per utterance [B, CB], nb_n [B] entries in use. */
  int32_t tsd_smax;
  int32_t rows_per_utt;
  float* nb_score;
  int32_t* nb_u;
  int32_t* nb_last_tok;
  int32_t* nb_row;
  int32_t* nb_origin;      /* (step within the frame) << 8 | slot of the first proposal of the entry */
  uint64_t* nb_hash;
  uint64_t* nb_prev_hash;
  int32_t* nb_n;
} q4_beam_state;

/* Reset `state` for a new batch: slot 0 of every utterance holds the empty hypothesis with
 * the start symbol (0) pending, everything else empty. */
int q4_beam_init(q4_beam_state* state, int32_t B, int32_t W, int32_t n_iters, q4_stream stream);

/*
 * dr_fusion_beam_step — one iteration of alignment-length synchronous beam search with the
 * density-ratio score of Eq. 1 (Section 2) for B utterances x W slots:
 *   1. pending network advances: every newly created label extension feeds its label to the
 *      prediction network, the source LM and the target LM (LSTM steps, projections, LM
 *      log-softmax);
 *   2. joint network + log-softmax for every live hypothesis at its frame e[t, b];
 *   3. proposals: blank (t+1, score + log P(blank)) and, while u < u_max, every label k
 *      (score + log P(k) + lambda_t log P_tgt(k) - lambda_s log P_src(k) + rho);
 *      proposals describing the same label string are merged by log-addition; blank
 *      proposals that consumed the last frame go to the finished list (best W kept); the
 *      W best others (score descending, then parent slot, then token) become the next beam.
 * e [T, B, D] fp32 projected encoder frames.  `iter` counts from 0; hypotheses in the beam
 * entering iteration `iter` satisfy t + u = iter.
 * mode 0: the search above (the paper's, Section 2), T + u_max iterations.
 * modes 1 and 2: time-synchronous search over the same networks (the beam workload's wording):
 * all hypotheses stand at frame t = iter / (S + 1), S = state->tsd_smax; a frame takes S + 1 calls.
 * Call number s = iter % (S + 1) < S is mode 1: every blank proposal joins the candidate set of the
 * next frame (equal label strings merged by log-addition, state->nb_*), and the W best label
 * proposals become the hypotheses of the next call at the same frame.  Call s = S is mode 2: blanks
 * join the candidate set, no labels are proposed, and the W best candidates (score descending, then
 * order of insertion) open frame t + 1; after the last frame they are the finished list.
 * T (S + 1) iterations.  History of a mode-2 call: bp_parent = slot that first proposed the entry,
 * bp_token = -1 - (call number within the frame of that proposal).
 * workspace: q4_workspace_bytes(Q4_WS_BEAM, {B, W, V, D}), or, to enable the tensor-core path
 * (needs model->prepared, LSTM widths that are multiples of 128 and V a multiple of 32),
 * q4_workspace_bytes(Q4_WS_BEAM, {B, W, V, D, E_pad, Hp, Hs, Ht}).  A bounded device wait that expires sets state->status to Q4_ERR_TIMEOUT.
 */
int dr_fusion_beam_step(const q4_model* model, q4_beam_state* state, const float* e, int32_t B,
                        int32_t T, int32_t W, int32_t iter, int32_t u_max, float lambda_t,
                        float lambda_s, float rho, int32_t mode, void* workspace,
                        size_t workspace_bytes, q4_stream stream);

/* Label strings of the best finished hypothesis per utterance (the best live one if none
 * finished): tokens [B, u_max], lens [B], scores [B] (device). */
int q4_traceback(const q4_beam_state* state, int32_t B, int32_t W, int32_t n_iters,
                 int32_t u_max, int32_t* tokens, int32_t* lens, float* scores, q4_stream stream);

/*
 * q4_feature_prologue — log-mel [B, T100, M] fp32 at 100 frames/s -> first and second time
 * differences (d_t = (x_{t+1} - x_{t-1}) / 2, edges replicated; dd likewise on d) -> frames
 * (2s, 2s+1) concatenated -> out [T100/2, B, 6M] fp16, time-major.  (Section 2 gives only
 * the feature dimension; this is the reading documented with the workloads.)
 */
int q4_feature_prologue(const float* mel, int32_t B, int32_t T100, int32_t M, void* out_fp16,
                        q4_stream stream);

#define Q4_WS_LSTM_LAYER 1 /* dims = {T, B, dirs, H} or {T, B, dirs, H, kx_pad} */
#define Q4_WS_JOINT 2      /* dims = {N, D} or {N, D, Hp_pad} (tensor-core path) */
#define Q4_WS_BEAM 3       /* dims = {B, W, V, D} or {B, W, V, D, E_pad, Hp, Hs, Ht} */
#define Q4_WS_LSTM_STEP 4  /* dims = {N, kx_pad, H} (tensor-core path of qlstm_step) */
#define Q4_WS_LINEAR 5     /* dims = {M, k_pad} (tensor-core path of q4_linear_forward) */
size_t q4_workspace_bytes(int32_t call_id, const int32_t* dims, int32_t ndims);

/* Synchronise `stream`, read the device status word and return 0 or the error it holds. */
int q4_poll_status(const int32_t* device_status, q4_stream stream);

/* Library version and the number of kernels launched so far by this process (a counter the
 * benchmark reads to report its launch count). */
int q4_version(void);
int64_t q4_launch_count(void);
/* Number of activation-quantizer applications enqueued so far (Section 3.4 counts them: T + T L
 * per sequence with the quantizer at the cell outputs, 2 T L with quantizers at the cell inputs):
 * +1 per quantize_pack_int4 call on activations (modes 0 and 1), +1 per qlstm_step with hq_out,
 * +T*dirs per qlstm_layer_forward (twice that when out_act differs from hid_act), +1 per joint
 * call, and the corresponding sum per beam step.  A call covers all rows it is given (a batch of
 * sequences counts once).  reset != 0 sets the counter back to zero after reading it. */
int64_t q4_quantizer_calls(int32_t reset);

/* dr_fusion_beam_step launches consecutive kernels of one stream as programmatic dependents
 * (each kernel sets itself up while its predecessor drains and waits for the predecessor's
 * completion before it reads anything).  enabled = 0 switches this off (plain stream order),
 * non-zero switches it on (the default).  Returns the previous setting.  Results do not depend
 * on it.  Not an operation of the paper. */
int q4_dependent_launch_set(int32_t enabled);

/* The beam selection first bounds the W-th best proposal from below by the smallest of 16
 * group maxima and ranks the few proposals above that bound; if they overflow its short list
 * it falls back to an exact bit-by-bit threshold search.  enabled != 0 makes every selection
 * take the exact search (for tests; both give the same beam).  Returns the previous setting. */
int q4_beam_select_exact_set(int32_t enabled);

/* qlstm_layer_forward, 4-bit layers of 640 cells: when the sequences form one group of 8 more (per
 * direction) than thread-block clusters can be resident, the clusters of a direction take turns at
 * that group instead of every cluster serving two groups.  enabled = 0 switches this off (for tests
 * and measurements; the results are identical).  Returns the previous setting. */
int q4_encoder_time_slicing_set(int32_t enabled);

/* How qlstm_layer_forward lays a layer's recurrence on thread-block clusters (host logic only, no
 * launch; for tests and diagnostics; with no device present the cluster capacity defaults to 15).
 * out[17]: [0] kernel (0 general, 1 packed 4-bit weights in registers, 2 the kernel whose clusters
 * may take turns), [1] groups of 8 sequences per cluster, [2..3] clusters per direction, [4..5]
 * whether the direction's clusters take turns at its last group, [6] groups per direction, [7]
 * clusters that can be resident, [8..16] step bounds of the turns: cluster j of such a direction
 * advances the shared group over steps [out[8+j], out[9+j]).  Assumes a signed hidden quantizer,
 * no accumulator dump and a caller workspace (as qlstm_layer_forward provides). */
int q4_encoder_recurrence_plan(int32_t T, int32_t B, int32_t dirs, int32_t H, int32_t w_bits, int32_t hid_bits,
                               int32_t per_sequence_scale, int32_t* out);

/* Test hook for the bounded device-side waits (not an operation of the paper): while skip_producer
 * is non-zero the tiled tensor-core GEMM (the tensor-core paths of q4_linear_forward and of the
 * projections) launches with a producer that issues no copy at all, so that the consumer's wait
 * runs out after wait_limit polls (0 = the normal limit); nothing asynchronous is in flight, every
 * thread of the kernel still reaches its final barrier, tensor memory is freed, nothing is stored
 * and the status word reads Q4_ERR_TIMEOUT.  (0, 0) restores normal operation.  Process-wide. */
int q4_test_wait_expiry_set(int32_t skip_producer, uint32_t wait_limit);

/* Threads: the library keeps a few process-wide host variables (launch and quantizer counters, the
 * timing hook, the switches above); calls from several host threads must be serialised by the
 * caller. */

/* Optional timing of the library's own launches with CUDA events lent by the caller (host
 * arrays of cudaEvent_t, `capacity` entries each).  Every launch whose tag bit is set in
 * tag_mask records start_events[i] before and stop_events[i] after itself on the stream it
 * is launched on, and writes its tag to tags_out[i]; q4_timing_count() returns how many
 * pairs were used.  tag_mask 0 switches timing off (the default).  Tags: 1 quantize, 2
 * encoder input GEMM, 3 encoder recurrent step, 4 linear, 5 prediction LSTM, 6 prediction
 * projection, 7 source-LM LSTM, 8 source-LM head, 9 target-LM layer 1, 10 target-LM layer 2,
 * 11 target-LM head, 12 joint, 13 beam selection, 14 other. */
int q4_timing_set(uint32_t tag_mask, void** start_events, void** stop_events, int32_t* tags_out,
                  int32_t capacity);
int q4_timing_count(void);

#ifdef __cplusplus
}
#endif
#endif /* Q4RNNT_H_ */
