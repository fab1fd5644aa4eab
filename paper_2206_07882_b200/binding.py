"""Thin Python binding of the q4rnnt C ABI (include/q4rnnt.h).

Only argument marshalling happens here: torch provides device memory and the
current stream, ctypes passes raw pointers, and every arithmetic step runs in
the library's CUDA kernels.  There is no fallback: if the shared library is
missing, or CUDA is unavailable, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libq4rnnt.so")

ERRORS = {-1: "Q4_ERR_NULL", -2: "Q4_ERR_DIM", -3: "Q4_ERR_ALIGN", -4: "Q4_ERR_BITS",
          -5: "Q4_ERR_WORKSPACE", -6: "Q4_ERR_UNSUPPORTED", -7: "Q4_ERR_CUDA", -8: "Q4_ERR_TIMEOUT"}
WS_LSTM_LAYER, WS_JOINT, WS_BEAM, WS_LSTM_STEP, WS_LINEAR = 1, 2, 3, 4, 5


class Q4Error(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where} failed: {ERRORS.get(code, code)}")
        self.code = code


class Act(C.Structure):
    _fields_ = [("scale", C.c_float), ("inv_scale", C.c_float), ("zero_point", C.c_int32),
                ("bits", C.c_int32), ("is_signed", C.c_int32)]


class Mat(C.Structure):
    _fields_ = [("q", C.c_void_p), ("scale", C.c_void_p), ("rows", C.c_int32), ("k", C.c_int32),
                ("k_pad", C.c_int32), ("bits", C.c_int32)]


class LstmS(C.Structure):
    _fields_ = [("w_ih", Mat), ("w_hh", Mat), ("bias", C.c_void_p), ("hid_act", Act)]


class LinearS(C.Structure):
    _fields_ = [("w", Mat), ("bias", C.c_void_p)]


class LmS(C.Structure):
    _fields_ = [("emb_q", C.c_void_p), ("emb_act", Act), ("n_layers", C.c_int32),
                ("lstm", LstmS * 2), ("bott", LinearS), ("bott_act", Act), ("out", LinearS)]


class ModelS(C.Structure):
    _fields_ = [("V", C.c_int32), ("E", C.c_int32), ("D", C.c_int32), ("pred_emb_q", C.c_void_p),
                ("pred_emb_act", Act), ("pred_lstm", LstmS), ("pred_proj", LinearS),
                ("z_act", Act), ("joint_out", LinearS), ("src", LmS), ("tgt", LmS),
                ("prepared", C.c_void_p)]


class BeamStateS(C.Structure):
    _fields_ = [("pred_hq", C.c_void_p), ("pred_c", C.c_void_p), ("pred_p", C.c_void_p),
                ("src_hq", C.c_void_p), ("src_c", C.c_void_p), ("src_lp", C.c_void_p),
                ("tgt_hq", C.c_void_p * 2), ("tgt_c", C.c_void_p * 2), ("tgt_lp", C.c_void_p),
                ("score", C.c_void_p), ("t", C.c_void_p), ("u", C.c_void_p), ("hash", C.c_void_p),
                ("prev_hash", C.c_void_p), ("last_tok", C.c_void_p), ("row", C.c_void_p),
                ("adv_src", C.c_void_p), ("adv_dst", C.c_void_p), ("adv_tok", C.c_void_p),
                ("pend_src", C.c_void_p), ("pend_dst", C.c_void_p), ("pend_tok", C.c_void_p),
                ("pend_n", C.c_void_p),
                ("bp_parent", C.c_void_p), ("bp_token", C.c_void_p), ("bp_score", C.c_void_p),
                ("fin_score", C.c_void_p), ("fin_iter", C.c_void_p), ("fin_slot", C.c_void_p),
                ("fin_n", C.c_void_p), ("status", C.c_void_p),
                ("aux_stream", C.c_void_p * 2), ("aux_event", C.c_void_p * 3),
                ("tsd_smax", C.c_int32), ("rows_per_utt", C.c_int32),
                ("nb_score", C.c_void_p), ("nb_u", C.c_void_p), ("nb_last_tok", C.c_void_p),
                ("nb_row", C.c_void_p), ("nb_origin", C.c_void_p), ("nb_hash", C.c_void_p),
                ("nb_prev_hash", C.c_void_p), ("nb_n", C.c_void_p)]


EXPORTS = ["q4_act_symmetric", "q4_act_asymmetric", "quantize_pack_int4", "qlstm_layer_forward",
           "qlstm_step", "q4_linear_forward", "qjoint_logprobs", "q4_beam_init",
           "dr_fusion_beam_step", "q4_traceback", "q4_feature_prologue", "q4_workspace_bytes",
           "q4_poll_status", "q4_version", "q4_launch_count", "q4_dependent_launch_set", "q4_beam_select_exact_set", "q4_timing_set", "q4_timing_count", "q4_prepared_bytes", "q4_prepare_model", "qjoint_logprobs_static", "q4_quantizer_calls", "q4_prepared_lstm_bytes", "q4_prepare_lstm",
           "q4_prepared_linear_bytes", "q4_prepare_linear", "q4_test_wait_expiry_set", "q4_encoder_time_slicing_set", "q4_encoder_recurrence_plan"]

_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2206_07882_b200.build` (nvcc, sm_100a)")
        _lib = C.CDLL(LIB_PATH)
        _lib.q4_workspace_bytes.restype = C.c_size_t
        _lib.q4_launch_count.restype = C.c_int64
        _lib.q4_prepared_bytes.restype = C.c_size_t
        _lib.q4_quantizer_calls.restype = C.c_int64
        _lib.q4_prepared_lstm_bytes.restype = C.c_size_t
        _lib.q4_prepared_linear_bytes.restype = C.c_size_t
    return _lib


def _need_cuda():
    if not torch.cuda.is_available():
        raise RuntimeError("q4rnnt needs a CUDA device; there is no CPU path")


def _p(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _chk(code: int, where: str):
    if code != 0:
        raise Q4Error(code, where)


def pad32(k: int) -> int:
    return (k + 31) // 32 * 32


def pad_for(k: int, bits: int) -> int:
    """Row length in elements: rows are multiples of 16 bytes, so 2-bit rows pad to 64."""
    m = 64 if bits == 2 else 32
    return (k + m - 1) // m * m


def launch_count() -> int:
    return int(lib().q4_launch_count())


def quantizer_calls(reset: bool = False) -> int:
    """Activation-quantizer applications enqueued so far by the library (Section 3.4)."""
    return int(lib().q4_quantizer_calls(C.c_int32(1 if reset else 0)))


def dependent_launch_set(enabled: bool) -> bool:
    """Switch programmatic dependent launches of the beam step on or off; returns the previous setting."""
    return bool(lib().q4_dependent_launch_set(1 if enabled else 0))


def encoder_time_slicing_set(enabled: bool) -> bool:
    """Let the clusters of the encoder recurrence take turns at a surplus group of sequences (default) or not; returns the previous setting."""
    return bool(lib().q4_encoder_time_slicing_set(1 if enabled else 0))


def encoder_recurrence_plan(T: int, B: int, dirs: int, H: int, w_bits: int = 4, hid_bits: int = 4,
                            per_sequence_scale: bool = False) -> dict:
    """Host-side plan of a layer's recurrence (no launch): kernel, clusters per direction, turns."""
    out = (C.c_int32 * 17)()
    _chk(lib().q4_encoder_recurrence_plan(C.c_int32(T), C.c_int32(B), C.c_int32(dirs), C.c_int32(H), C.c_int32(w_bits),
                                          C.c_int32(hid_bits), C.c_int32(1 if per_sequence_scale else 0), out),
         "q4_encoder_recurrence_plan")
    v = list(out)
    return dict(kernel=v[0], groups_per_cluster=v[1], clusters=v[2:4], turns=v[4:6], groups=v[6], max_clusters=v[7],
                windows=v[8:17])


def beam_select_exact_set(enabled: bool) -> bool:
    """Force the exact threshold search in every beam selection (tests); returns the previous setting."""
    return bool(lib().q4_beam_select_exact_set(1 if enabled else 0))


def workspace_bytes(call_id: int, dims: Sequence[int]) -> int:
    arr = (C.c_int32 * len(dims))(*dims)
    return int(lib().q4_workspace_bytes(C.c_int32(call_id), arr, C.c_int32(len(dims))))


def q4_act_symmetric(alpha: float, bits: int) -> Act:
    a = Act()
    _chk(lib().q4_act_symmetric(C.c_float(alpha), C.c_int32(bits), C.byref(a)), "q4_act_symmetric")
    return a


def q4_act_asymmetric(lo: float, hi: float, bits: int = 4) -> Act:
    a = Act()
    _chk(lib().q4_act_asymmetric(C.c_float(lo), C.c_float(hi), C.c_int32(bits), C.byref(a)),
         "q4_act_asymmetric")
    return a


# ------------------------------------------------------------------ entry points
def quantize_pack_int4(x: torch.Tensor, act: Act, mode: int = 0, n_groups: int = 1,
                       per_row_scale: Optional[torch.Tensor] = None, k_pad: Optional[int] = None):
    """x [rows, k] fp16/fp32 on the device -> codes [rows, k_pad*bits/8] uint8.
    mode 1 also returns the per-group scales."""
    _need_cuda()
    assert x.is_cuda and x.dim() == 2 and x.is_contiguous()
    assert x.dtype in (torch.float16, torch.float32)
    rows, k = x.shape
    k_pad = pad32(k) if k_pad is None else k_pad
    out = torch.empty((rows, k_pad * act.bits // 8), dtype=torch.uint8, device=x.device)
    gs = torch.empty(n_groups, dtype=torch.float32, device=x.device) if mode == 1 else None
    _chk(lib().quantize_pack_int4(_p(x), C.c_int32(1 if x.dtype == torch.float16 else 0),
                                  C.c_int64(rows), C.c_int32(k), C.c_int32(k_pad), C.byref(act),
                                  C.c_int32(mode), C.c_int32(n_groups), _p(per_row_scale), _p(out),
                                  _p(gs), _stream()), "quantize_pack_int4")
    return (out, gs) if mode == 1 else out


class DeviceMat:
    """Integer weight matrix on the device in the library's storage format."""

    def __init__(self, q: torch.Tensor, scale: torch.Tensor, rows: int, k: int, k_pad: int, bits: int):
        self.q, self.scale, self.rows, self.k, self.k_pad, self.bits = q, scale, rows, k, k_pad, bits

    @staticmethod
    def from_codes(codes: np.ndarray, scale: np.ndarray, bits: int, device="cuda") -> "DeviceMat":
        """Pack integer codes with the library's own packer: the codes are handed over as
        floats with unit row scale, which quantize_pack_int4 (mode 2) maps back exactly."""
        rows, k = codes.shape
        x = torch.from_numpy(np.ascontiguousarray(codes, dtype=np.float32)).to(device)
        ones = torch.ones(rows, dtype=torch.float32, device=device)
        a = Act(1.0, 1.0, 0, bits, 1)
        q = quantize_pack_int4(x, a, mode=2, per_row_scale=ones, k_pad=pad_for(k, bits))
        s = torch.from_numpy(np.ascontiguousarray(scale, dtype=np.float32)).to(device)
        return DeviceMat(q, s, rows, k, pad_for(k, bits), bits)

    @staticmethod
    def from_float(w: np.ndarray, scale: np.ndarray, bits: int, device="cuda") -> "DeviceMat":
        """Symmetric per-row quantization of real-valued weights (mode 2)."""
        rows, k = w.shape
        x = torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).to(device)
        s = torch.from_numpy(np.ascontiguousarray(scale, dtype=np.float32)).to(device)
        a = Act(1.0, 1.0, 0, bits, 1)
        return DeviceMat(quantize_pack_int4(x, a, mode=2, per_row_scale=s, k_pad=pad_for(k, bits)), s, rows, k,
                         pad_for(k, bits), bits)

    @staticmethod
    def from_float_max(w: np.ndarray, bits: int, device="cuda") -> "DeviceMat":
        """Symmetric per-row quantization of real-valued weights with the MAX boundary of
        Section 3.1 taken per output row (boundary = the row's largest magnitude, an all-zero row
        gets 1): mode 1 with one group per row; the row scales come back from the device."""
        rows, k = w.shape
        x = torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).to(device)
        q, s = quantize_pack_int4(x, Act(1.0, 1.0, 0, bits, 1), mode=1, n_groups=rows, k_pad=pad_for(k, bits))
        return DeviceMat(q, s, rows, k, pad_for(k, bits), bits)

    def c(self) -> Mat:
        return Mat(self.q.data_ptr(), self.scale.data_ptr(), self.rows, self.k, self.k_pad, self.bits)

    def nbytes(self) -> int:
        return self.q.numel() + self.scale.numel() * 4


def _dev_f32(a: Optional[np.ndarray], device="cuda") -> Optional[torch.Tensor]:
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)


class DeviceLstm:
    def __init__(self, lw, device="cuda"):
        self.w_ih = DeviceMat.from_codes(lw.w_ih.codes, lw.w_ih.scale, lw.w_ih.bits, device)
        self.w_hh = DeviceMat.from_codes(lw.w_hh.codes, lw.w_hh.scale, lw.w_hh.bits, device)
        self.bias = _dev_f32(lw.bias, device)
        self.hid_act = q4_act_symmetric(lw.hid_alpha, lw.hid_bits)
        self.H = self.w_hh.k
        self.prepared = None
        self.ws = None

    def prepare(self):
        """One-time int8 operands for the tensor-core path of qlstm_step (q4_prepare_lstm)."""
        wi, wh = self.w_ih.c(), self.w_hh.c()
        n = int(lib().q4_prepared_lstm_bytes(C.byref(wi), C.byref(wh)))
        self.prepared = torch.empty(n, dtype=torch.uint8, device=self.w_ih.q.device)
        _chk(lib().q4_prepare_lstm(C.byref(wi), C.byref(wh), _p(self.bias), _p(self.prepared), C.c_size_t(n),
                                   _stream()), "q4_prepare_lstm")
        return self

    def c(self) -> LstmS:
        return LstmS(self.w_ih.c(), self.w_hh.c(), self.bias.data_ptr() if self.bias is not None else None,
                     self.hid_act)

    def nbytes(self):
        return self.w_ih.nbytes() + self.w_hh.nbytes() + (self.bias.numel() * 4 if self.bias is not None else 0)


class DeviceLinear:
    def __init__(self, lw, device="cuda"):
        self.w = DeviceMat.from_codes(lw.w.codes, lw.w.scale, lw.w.bits, device)
        self.bias = _dev_f32(lw.bias, device)
        self.prepared = None
        self.ws = None

    def prepare(self):
        """One-time int8 operand for the tensor-core paths (q4_prepare_linear)."""
        w = self.w.c()
        n = int(lib().q4_prepared_linear_bytes(C.byref(w)))
        self.prepared = torch.empty(n, dtype=torch.uint8, device=self.w.q.device)
        _chk(lib().q4_prepare_linear(C.byref(w), _p(self.prepared), C.c_size_t(n), _stream()), "q4_prepare_linear")
        return self

    def c(self) -> LinearS:
        return LinearS(self.w.c(), self.bias.data_ptr() if self.bias is not None else None)

    def nbytes(self):
        return self.w.nbytes() + (self.bias.numel() * 4 if self.bias is not None else 0)


def qlstm_layer_forward(xq: torch.Tensor, x_act: Act, T: int, B: int, layers: Sequence[DeviceLstm],
                        out_act: Optional[Act] = None, x_scale_b: Optional[torch.Tensor] = None,
                        want_state: bool = False, want_dbg: bool = False,
                        workspace: Optional[torch.Tensor] = None, tensor_cores: bool = True):
    """xq [T*B, kx_pad*bits/8] codes.  Returns dict(yq [, hq_n, c_n, acc_ih, acc_hh])."""
    _need_cuda()
    dirs, H = len(layers), layers[0].H
    hid_act = layers[0].hid_act
    out_act = out_act or hid_act
    dev = xq.device
    yq = torch.empty((T * B, dirs * H * out_act.bits // 8), dtype=torch.uint8, device=dev)
    need = workspace_bytes(WS_LSTM_LAYER, [T, B, dirs, H] + ([layers[0].w_ih.k_pad] if tensor_cores else []))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    r = {"yq": yq, "workspace": workspace}
    if want_state:
        r["hq_n"] = torch.empty((dirs, B, H * hid_act.bits // 8), dtype=torch.uint8, device=dev)
        r["c_n"] = torch.empty((dirs, B, H), dtype=torch.float32, device=dev)
    if want_dbg:
        r["acc_ih"] = torch.empty((T, B, dirs, 4 * H), dtype=torch.int32, device=dev)
        r["acc_hh"] = torch.empty((T, B, dirs, 4 * H), dtype=torch.int32, device=dev)
    wih = (Mat * dirs)(*[l.w_ih.c() for l in layers])
    whh = (Mat * dirs)(*[l.w_hh.c() for l in layers])
    bias = (C.c_void_p * dirs)(*[l.bias.data_ptr() if l.bias is not None else None for l in layers])
    _chk(lib().qlstm_layer_forward(_p(xq), C.byref(x_act), _p(x_scale_b), C.c_int32(T), C.c_int32(B),
                                   C.c_int32(dirs), wih, whh, bias, C.byref(hid_act),
                                   C.byref(out_act), _p(yq), _p(r.get("hq_n")), _p(r.get("c_n")),
                                   _p(r.get("acc_ih")), _p(r.get("acc_hh")), _p(workspace),
                                   C.c_size_t(workspace.numel()), _stream()), "qlstm_layer_forward")
    return r


def qlstm_step(xq: torch.Tensor, x_act: Act, hq_in: torch.Tensor, c_in: torch.Tensor,
               layer: DeviceLstm, x_row_idx: Optional[torch.Tensor] = None, want_dbg: bool = False,
               out: Optional[dict] = None):
    """One step for N rows.  Returns dict(hq, c, h [, acc_ih, acc_hh]).  `out` may hold
    preallocated tensors hq, c (c may be c_in itself) and optionally h; then nothing is allocated."""
    _need_cuda()
    N, H = c_in.shape
    dev = c_in.device
    if out is not None:
        r = dict(out)
    else:
        r = {"hq": torch.empty_like(hq_in), "c": torch.empty_like(c_in),
             "h": torch.empty((N, H), dtype=torch.float32, device=dev)}
    if want_dbg:
        r["acc_ih"] = torch.empty((N, 4 * H), dtype=torch.int32, device=dev)
        r["acc_hh"] = torch.empty((N, 4 * H), dtype=torch.int32, device=dev)
    wih, whh = layer.w_ih.c(), layer.w_hh.c()
    ws = None
    if layer.prepared is not None:      # tensor-core path (taken by the library from 128 rows on)
        need = workspace_bytes(WS_LSTM_STEP, [N, layer.w_ih.k_pad, H])
        if layer.ws is None or layer.ws.numel() < need:
            layer.ws = torch.empty(need, dtype=torch.uint8, device=dev)
        ws = layer.ws
    _chk(lib().qlstm_step(_p(xq), C.byref(x_act), _p(x_row_idx), _p(hq_in), _p(c_in), C.c_int32(N),
                          C.byref(wih), C.byref(whh), _p(layer.bias), C.byref(layer.hid_act),
                          _p(r.get("hq")), _p(r["c"]), _p(r.get("h")), _p(r.get("acc_ih")),
                          _p(r.get("acc_hh")), _p(layer.prepared), _p(ws),
                          C.c_size_t(ws.numel() if ws is not None else 0), _stream()), "qlstm_step")
    return r


def lstm_layer_inner(x: torch.Tensor, x_act: Act, layers: Sequence[DeviceLstm]) -> torch.Tensor:
    """One layer under the Inner placement of the activation quantizers (Section 3.4): real-valued
    x [T, B, K] in, real-valued cell outputs [T, B, dirs*H] out; every step of every direction
    quantizes its two inputs on entry (two quantize_pack_int4 calls) and runs qlstm_step without
    the output quantizer.  Marshalling only: a loop over library calls."""
    _need_cuda()
    T, B, K = x.shape
    dirs, H = len(layers), layers[0].H
    hid = layers[0].hid_act
    out = torch.empty((T, B, dirs * H), dtype=torch.float32, device=x.device)
    for d, L in enumerate(layers):
        h = torch.zeros((B, H), dtype=torch.float32, device=x.device)
        c = torch.zeros((B, H), dtype=torch.float32, device=x.device)
        for s in range(T):
            t = s if d == 0 else T - 1 - s
            xq = quantize_pack_int4(x[t].contiguous(), x_act, k_pad=L.w_ih.k_pad)     # x_t on entry
            hq = quantize_pack_int4(h, hid)                                            # s_{t-1} on entry
            r = qlstm_step(xq, x_act, hq, c, L, out=dict(c=c, h=torch.empty_like(h)))
            h = r["h"]
            out[t, :, d * H:(d + 1) * H] = h
    return out


def q4_poll_status(status: torch.Tensor) -> int:
    """Synchronise the stream and return the device status word (0 = ok)."""
    return int(lib().q4_poll_status(_p(status), _stream()))


def q4_linear_forward(xq: torch.Tensor, x_act: Act, lin: DeviceLinear, want_acc: bool = False):
    _need_cuda()
    M = xq.shape[0]
    out = torch.empty((M, lin.w.rows), dtype=torch.float32, device=xq.device)
    acc = torch.empty((M, lin.w.rows), dtype=torch.int32, device=xq.device) if want_acc else None
    w = lin.w.c()
    ws = None
    if getattr(lin, "prepared", None) is not None and not want_acc:
        need = workspace_bytes(WS_LINEAR, [M, lin.w.k_pad])
        if lin.ws is None or lin.ws.numel() < need:
            lin.ws = torch.empty(need, dtype=torch.uint8, device=xq.device)
        ws = lin.ws
    _chk(lib().q4_linear_forward(_p(xq), C.byref(x_act), C.c_int32(M), C.byref(w), _p(lin.bias),
                                 _p(out), _p(acc), _p(getattr(lin, "prepared", None)), _p(ws),
                                 C.c_size_t(ws.numel() if ws is not None else 0), _stream()), "q4_linear_forward")
    return (out, acc) if want_acc else out


def qjoint_logprobs(e: torch.Tensor, frame_idx: torch.Tensor, pq: torch.Tensor, p_act: Act,
                    proj: DeviceLinear, z_act: Act, out: DeviceLinear,
                    logp: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    _need_cuda()
    N = pq.shape[0]
    D, V = proj.w.rows, out.w.rows
    if logp is None:
        logp = torch.empty((N, V), dtype=torch.float32, device=pq.device)
    tc = proj.prepared is not None and out.prepared is not None
    need = workspace_bytes(WS_JOINT, [N, D] + ([proj.w.k_pad] if tc else []))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(need, dtype=torch.uint8, device=pq.device)
    wp, wo = proj.w.c(), out.w.c()
    _chk(lib().qjoint_logprobs(_p(e), _p(frame_idx), _p(pq), C.byref(p_act), C.c_int32(N),
                               C.byref(wp), _p(proj.bias), C.byref(z_act), C.byref(wo), _p(out.bias),
                               _p(logp), _p(proj.prepared if tc else None), _p(out.prepared if tc else None),
                               _p(workspace), C.c_size_t(workspace.numel()), _stream()),
         "qjoint_logprobs")
    return logp


def qjoint_logprobs_static(e: torch.Tensor, frame_idx: torch.Tensor, pq: torch.Tensor, p_act: Act,
                           proj: DeviceLinear, z_act: Act, out: DeviceLinear, logp: torch.Tensor):
    """Joint network without a caller workspace and without any allocation: the output tensor
    is passed in and the scratch is the library's built-in array (N * D <= 65536).  For callers
    that must not allocate at call time; overlapping calls on one GPU share that array."""
    _need_cuda()
    wp, wo = proj.w.c(), out.w.c()
    _chk(lib().qjoint_logprobs_static(_p(e), _p(frame_idx), _p(pq), C.byref(p_act),
                                      C.c_int32(pq.shape[0]), C.byref(wp), _p(proj.bias),
                                      C.byref(z_act), C.byref(wo), _p(out.bias), _p(logp), _stream()),
         "qjoint_logprobs_static")
    return logp


def q4_feature_prologue(mel: torch.Tensor) -> torch.Tensor:
    """mel [B, T100, M] fp32 -> [T100/2, B, 6M] fp16."""
    _need_cuda()
    B, T100, M = mel.shape
    out = torch.empty((T100 // 2, B, 6 * M), dtype=torch.float16, device=mel.device)
    _chk(lib().q4_feature_prologue(_p(mel), C.c_int32(B), C.c_int32(T100), C.c_int32(M), _p(out),
                                   _stream()), "q4_feature_prologue")
    return out


# ------------------------------------------------------------------ whole networks
class Encoder:
    """Device copy of the encoder weights plus the layer loop (one library call per layer)."""

    def __init__(self, enc, device="cuda"):
        self.layers = [[DeviceLstm(d, device) for d in dirs] for dirs in enc.layers]
        self.proj = DeviceLinear(enc.proj, device).prepare() if enc.proj is not None else None
        self.in_bits, self.in_max, self.in_clip = enc.in_bits, enc.in_max, enc.in_clip
        self.in_act = q4_act_symmetric(1.0 if enc.in_max else enc.in_clip, enc.in_bits)
        self.out_acts = []
        for l, dirs in enumerate(enc.layers):
            nxt = enc.layers[l + 1][0].w_ih.bits if l + 1 < len(enc.layers) else (
                enc.proj.w.bits if enc.proj is not None else dirs[0].hid_bits)
            self.out_acts.append(q4_act_symmetric(dirs[0].hid_alpha, nxt))
        self.ws = None

    def weight_bytes(self) -> int:
        n = sum(d.nbytes() for dirs in self.layers for d in dirs)
        return n + (self.proj.nbytes() if self.proj is not None else 0)

    def forward(self, features: torch.Tensor, want_layers: bool = False):
        """features [T, B, F] fp16/fp32 on the device.  Returns dict(yq, y_act, e [, layers])."""
        T, B, F = features.shape
        x2 = features.reshape(T * B, F)
        x_scale_b = None
        kp = self.layers[0][0].w_ih.k_pad          # rows padded like the first layer's weight rows
        if self.in_max:
            xq, x_scale_b = quantize_pack_int4(x2, self.in_act, mode=1, n_groups=B, k_pad=kp)
        else:
            xq = quantize_pack_int4(x2, self.in_act, k_pad=kp)
        x_act = self.in_act
        H = self.layers[0][0].H
        kmax = max(dirs[0].w_ih.k_pad for dirs in self.layers)
        need = workspace_bytes(WS_LSTM_LAYER, [T, B, 2, H, kmax])
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(need, dtype=torch.uint8, device=features.device)
        outs = []
        for l, dirs in enumerate(self.layers):
            r = qlstm_layer_forward(xq, x_act, T, B, dirs, self.out_acts[l], x_scale_b=x_scale_b,
                                    workspace=self.ws)
            xq, x_act, x_scale_b = r["yq"], self.out_acts[l], None
            if want_layers:
                outs.append(r["yq"])
        res = {"yq": xq, "y_act": x_act, "layers": outs}
        if self.proj is not None:
            res["e"] = q4_linear_forward(xq, x_act, self.proj).reshape(T, B, -1)
        return res


class DeviceLm:
    def __init__(self, m, device="cuda"):
        wide = getattr(m, "act_bits", 4) == 8     # 8 bits: symmetric with the wider boundary (signed codes)
        self.emb_act = q4_act_symmetric(max(-m.emb_lo, m.emb_hi), 8) if wide else q4_act_asymmetric(m.emb_lo, m.emb_hi, 4)
        emb = torch.from_numpy(np.ascontiguousarray(m.emb, dtype=np.float32)).to(device)
        self.lstm = [DeviceLstm(l, device) for l in m.lstm]
        self.emb_q = quantize_pack_int4(emb, self.emb_act, k_pad=self.lstm[0].w_ih.k_pad)   # table quantized once
        self.bott = DeviceLinear(m.bott, device)
        self.bott_act = q4_act_symmetric(max(-m.bott_lo, m.bott_hi), 8) if wide else q4_act_asymmetric(m.bott_lo, m.bott_hi, 4)
        self.out = DeviceLinear(m.out, device)

    def c(self) -> LmS:
        s = LmS()
        s.emb_q, s.emb_act, s.n_layers = self.emb_q.data_ptr(), self.emb_act, len(self.lstm)
        for i, l in enumerate(self.lstm):
            s.lstm[i] = l.c()
        s.bott, s.bott_act, s.out = self.bott.c(), self.bott_act, self.out.c()
        return s

    def nbytes(self):
        return self.emb_q.numel() + sum(l.nbytes() for l in self.lstm) + self.bott.nbytes() + self.out.nbytes()


class Decoder:
    """Device copy of prediction network, joint network and both fusion LMs, the search
    state, and the iteration loop (one library call per search iteration)."""

    def __init__(self, dw, device="cuda", tensor_cores: bool = True, concurrent: bool = True, share_from=None):
        self.dw = dw
        self.device = device
        self.tensor_cores = tensor_cores
        self.concurrent = concurrent and tensor_cores
        self.state = None
        self.S_max = None
        if share_from is not None:
            # a second search state over the same device weights (read-only, prepared operands included)
            for name in ("V", "E", "D", "pred_emb_act", "pred_emb_q", "pred_lstm", "pred_proj", "z_act", "joint_out",
                         "src", "tgt", "model", "prepared"):
                setattr(self, name, getattr(share_from, name))
            return
        self.V, self.E = dw.pred.emb.shape
        self.pred_emb_act = q4_act_symmetric(dw.pred.emb_alpha, getattr(dw, "emb_bits", 4))
        emb = torch.from_numpy(np.ascontiguousarray(dw.pred.emb, dtype=np.float32)).to(device)
        self.pred_lstm = DeviceLstm(dw.pred.lstm, device)
        self.pred_emb_q = quantize_pack_int4(emb, self.pred_emb_act, k_pad=self.pred_lstm.w_ih.k_pad)
        self.pred_proj = DeviceLinear(dw.pred.proj, device)
        self.D = self.pred_proj.w.rows
        self.z_act = q4_act_symmetric(1.0, dw.joint.z_bits)
        self.joint_out = DeviceLinear(dw.joint.out, device)
        self.src, self.tgt = DeviceLm(dw.src, device), DeviceLm(dw.tgt, device)
        m = self.model = ModelS()
        m.V, m.E, m.D = self.V, self.E, self.D
        m.pred_emb_q, m.pred_emb_act = self.pred_emb_q.data_ptr(), self.pred_emb_act
        m.pred_lstm, m.pred_proj = self.pred_lstm.c(), self.pred_proj.c()
        m.z_act, m.joint_out = self.z_act, self.joint_out.c()
        m.src, m.tgt = self.src.c(), self.tgt.c()
        m.prepared = None
        self.prepared = None
        if tensor_cores:
            self.q4_prepare_model()
        self.state = None
        self.S_max = None

    def q4_prepare_model(self):
        """One-time int8 / gate-interleaved copies of the step weights for the tensor cores."""
        n = int(lib().q4_prepared_bytes(C.byref(self.model)))
        self.prepared = torch.empty(n, dtype=torch.uint8, device=self.device)
        _chk(lib().q4_prepare_model(C.byref(self.model), _p(self.prepared), C.c_size_t(n), _stream()),
             "q4_prepare_model")

    def step_weight_bytes(self) -> int:
        return (self.pred_lstm.nbytes() + self.pred_proj.nbytes() + self.joint_out.nbytes() +
                self.src.nbytes() - self.src.emb_q.numel() + self.tgt.nbytes() - self.tgt.emb_q.numel())

    def alloc_state(self, B: int, W: int, n_iters: int, S_max: Optional[int] = None):
        """State for B utterances x W slots and n_iters calls; with S_max the layout of the
        time-synchronous search (W (S_max + 1) state rows per utterance and its candidate set)."""
        dev = self.device
        RW = 2 * W if S_max is None else max(2 * W, W * (S_max + 1))
        R, N = B * RW, B * W
        Hp, Hs, Ht = self.pred_lstm.H, self.src.lstm[0].H, self.tgt.lstm[0].H
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
        bp, bs, bt = (self.pred_lstm.hid_act.bits, self.src.lstm[0].hid_act.bits, self.tgt.lstm[0].hid_act.bits)
        t = self.tensors = dict(
            pred_hq=z((R, Hp * bp // 8), torch.uint8), pred_c=z((R, Hp), torch.float32),
            pred_p=z((R, self.D), torch.float32),
            src_hq=z((R, Hs * bs // 8), torch.uint8), src_c=z((R, Hs), torch.float32),
            src_lp=z((R, self.V), torch.float32),
            tgt_hq0=z((R, Ht * bt // 8), torch.uint8), tgt_c0=z((R, Ht), torch.float32),
            tgt_hq1=z((R, Ht * bt // 8), torch.uint8), tgt_c1=z((R, Ht), torch.float32),
            tgt_lp=z((R, self.V), torch.float32),
            score=z(N, torch.float32), t=z(N, torch.int32), u=z(N, torch.int32),
            hash=z(N, torch.int64), prev_hash=z(N, torch.int64), last_tok=z(N, torch.int32),
            row=z(N, torch.int32), adv_src=z(N, torch.int32), adv_dst=z(N, torch.int32),
            adv_tok=z(N, torch.int32),
            pend_src=z((2, N), torch.int32), pend_dst=z((2, N), torch.int32),
            pend_tok=z((2, N), torch.int32), pend_n=z(2, torch.int32),
            bp_parent=z((max(n_iters, 1), B, W), torch.int32),
            bp_token=z((max(n_iters, 1), B, W), torch.int32),
            bp_score=z((max(n_iters, 1), B, W), torch.float32),
            fin_score=z((B, W), torch.float32), fin_iter=z((B, W), torch.int32),
            fin_slot=z((B, W), torch.int32), fin_n=z(B, torch.int32), status=z(1, torch.int32))
        s = self.state = BeamStateS()
        for name in ("pred_hq", "pred_c", "pred_p", "src_hq", "src_c", "src_lp", "tgt_lp", "score",
                     "t", "u", "hash", "prev_hash", "last_tok", "row", "adv_src", "adv_dst", "adv_tok",
                     "pend_src", "pend_dst", "pend_tok", "pend_n",
                     "bp_parent", "bp_token", "bp_score", "fin_score", "fin_iter", "fin_slot",
                     "fin_n", "status"):
            setattr(s, name, t[name].data_ptr())
        s.tgt_hq[0], s.tgt_hq[1] = t["tgt_hq0"].data_ptr(), t["tgt_hq1"].data_ptr()
        s.tgt_c[0], s.tgt_c[1] = t["tgt_c0"].data_ptr(), t["tgt_c1"].data_ptr()
        self.S_max = S_max
        if S_max is not None:
            CB = W * (S_max + 1)
            t.update(nb_score=z((B, CB), torch.float32), nb_u=z((B, CB), torch.int32),
                     nb_last_tok=z((B, CB), torch.int32), nb_row=z((B, CB), torch.int32),
                     nb_origin=z((B, CB), torch.int32), nb_hash=z((B, CB), torch.int64),
                     nb_prev_hash=z((B, CB), torch.int64), nb_n=z(B, torch.int32))
            for name in ("nb_score", "nb_u", "nb_last_tok", "nb_row", "nb_origin", "nb_hash", "nb_prev_hash",
                         "nb_n"):
                setattr(s, name, t[name].data_ptr())
            s.tsd_smax, s.rows_per_utt = S_max, RW
        if self.concurrent:
            # two more streams and three untimed events lent to the library for fork / join
            self._aux_streams = [torch.cuda.Stream(device=dev) for _ in range(2)]
            self._aux_events = [torch.cuda.Event() for _ in range(3)]
            for ev in self._aux_events:
                ev.record()
            for i in range(2):
                s.aux_stream[i] = self._aux_streams[i].cuda_stream
            for i in range(3):
                s.aux_event[i] = self._aux_events[i].cuda_event
        self.B, self.W, self.n_iters = B, W, n_iters
        dims = [B, W, self.V, self.D]
        if self.tensor_cores:
            dims += [self.pred_lstm.w_ih.k_pad, Hp, Hs, Ht]
        self.ws = torch.empty(workspace_bytes(WS_BEAM, dims), dtype=torch.uint8, device=dev)

    def q4_beam_init(self):
        _chk(lib().q4_beam_init(C.byref(self.state), C.c_int32(self.B), C.c_int32(self.W),
                                C.c_int32(self.n_iters), _stream()), "q4_beam_init")

    def dr_fusion_beam_step(self, e: torch.Tensor, T: int, it: int, u_max: int, mode: int = 0):
        dw = self.dw
        _chk(lib().dr_fusion_beam_step(C.byref(self.model), C.byref(self.state), _p(e),
                                       C.c_int32(self.B), C.c_int32(T), C.c_int32(self.W),
                                       C.c_int32(it), C.c_int32(u_max), C.c_float(dw.lambda_t),
                                       C.c_float(dw.lambda_s), C.c_float(dw.rho), C.c_int32(mode),
                                       _p(self.ws), C.c_size_t(self.ws.numel()), _stream()),
             "dr_fusion_beam_step")

    def q4_traceback(self, n_iters: int, u_max: int):
        dev = self.device
        tokens = torch.zeros((self.B, max(u_max, 1)), dtype=torch.int32, device=dev)
        lens = torch.zeros(self.B, dtype=torch.int32, device=dev)
        scores = torch.zeros(self.B, dtype=torch.float32, device=dev)
        _chk(lib().q4_traceback(C.byref(self.state), C.c_int32(self.B), C.c_int32(self.W),
                                C.c_int32(n_iters), C.c_int32(max(u_max, 1)), _p(tokens), _p(lens),
                                _p(scores), _stream()), "q4_traceback")
        return tokens, lens, scores

    def decode(self, e: torch.Tensor, u_max: Optional[int] = None, W: Optional[int] = None):
        """e [T, B, D] fp32 on the device.  Runs T + u_max search iterations and returns
        (tokens [B,u_max], lens [B], scores [B]) on the device."""
        T, B, D = e.shape
        u_max = self.dw.U_max if u_max is None else u_max
        W = self.dw.W if W is None else W
        n_iters = T + u_max
        if self.state is None or (self.B, self.W) != (B, W) or self.n_iters < n_iters or self.S_max is not None:
            self.alloc_state(B, W, n_iters)
        self.q4_beam_init()
        for it in range(n_iters):
            self.dr_fusion_beam_step(e, T, it, u_max)
        return self.q4_traceback(n_iters, u_max)

    def decode_time_synchronous(self, e: torch.Tensor, S_max: int, u_max: Optional[int] = None,
                                W: Optional[int] = None):
        """Time-synchronous search with at most S_max labels per frame: T (S_max + 1) calls of
        dr_fusion_beam_step (mode 1, the last of every frame mode 2).  Returns like decode()."""
        T, B, D = e.shape
        u_max = self.dw.U_max if u_max is None else u_max
        W = self.dw.W if W is None else W
        n_iters = T * (S_max + 1)
        if (self.state is None or (self.B, self.W) != (B, W) or self.n_iters < n_iters or
                self.S_max != S_max):
            self.alloc_state(B, W, n_iters, S_max)
        self.q4_beam_init()
        for it in range(n_iters):
            self.dr_fusion_beam_step(e, T, it, u_max, mode=2 if it % (S_max + 1) == S_max else 1)
        return self.q4_traceback(n_iters, u_max)


class GroupedDecoder:
    """The fused search over a batch split into `groups` sets of utterances, each with its own search
    state and streams over ONE copy of the device weights.  Utterances are independent (Eq. 1 has no
    cross-utterance term), so the sets advance side by side: while one set's selection and LM heads (short,
    latency-bound kernels) run, the other set's LSTM GEMMs have the SMs.  Marshalling only."""

    def __init__(self, dw, groups: int = 2, device="cuda"):
        first = Decoder(dw, device)
        self.parts = [first] + [Decoder(dw, device, share_from=first) for _ in range(groups - 1)]
        self.dw, self.device = dw, device
        self.streams = [torch.cuda.Stream(device=device) for _ in range(groups)]
        for name in ("V", "E", "D", "pred_lstm", "pred_proj", "joint_out", "src", "tgt"):
            setattr(self, name, getattr(first, name))

    def step_weight_bytes(self) -> int:
        return self.parts[0].step_weight_bytes()

    def _bounds(self, B):
        G = len(self.parts)
        return [(g * B // G, (g + 1) * B // G) for g in range(G)]

    def alloc_state(self, B: int, W: int, n_iters: int):
        for part, (b0, b1) in zip(self.parts, self._bounds(B)):
            part.alloc_state(b1 - b0, W, n_iters)

    def history(self, name: str) -> torch.Tensor:
        """A history tensor [iter, B, W] of all sets, utterances in batch order."""
        return torch.cat([p.tensors[name] for p in self.parts], dim=1)

    def decode(self, e: torch.Tensor, u_max: Optional[int] = None, W: Optional[int] = None):
        T, B, D = e.shape
        u_max = self.dw.U_max if u_max is None else u_max
        W = self.dw.W if W is None else W
        n_iters = T + u_max
        bounds = self._bounds(B)
        main = torch.cuda.current_stream()
        es = [e[:, b0:b1].contiguous() for b0, b1 in bounds]     # each set's frames as one dense block
        for part, (b0, b1) in zip(self.parts, bounds):
            if part.state is None or (part.B, part.W) != (b1 - b0, W) or part.n_iters < n_iters or part.S_max is not None:
                part.alloc_state(b1 - b0, W, n_iters)
        for st in self.streams:
            st.wait_stream(main)
        for part, st in zip(self.parts, self.streams):
            with torch.cuda.stream(st):
                part.q4_beam_init()
        for it in range(n_iters):
            for part, st, eg in zip(self.parts, self.streams, es):
                with torch.cuda.stream(st):
                    part.dr_fusion_beam_step(eg, T, it, u_max)
        res = []
        for part, st in zip(self.parts, self.streams):
            with torch.cuda.stream(st):
                res.append(part.q4_traceback(n_iters, u_max))
        for st in self.streams:
            main.wait_stream(st)
        return tuple(torch.cat([r[i] for r in res], dim=0) for i in range(3))


class GraphedStep:
    """Replays one whole pass (any callable that only enqueues library calls on the current
    stream) as a CUDA graph: the pass is run eagerly once (so that every kernel attribute is
    configured), captured once, then replayed.  The callable must read its input from the
    static tensors it closes over; results are the tensors it returned during capture."""

    def __init__(self, fn):
        self.fn = fn
        self.graph = None
        self.result = None

    def __call__(self):
        if self.graph is None:
            self.fn()                                   # eager warm-up
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self.result = self.fn()
            self.graph = g
        self.graph.replay()
        return self.result
