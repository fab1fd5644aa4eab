"""ctypes front end of the CPU oracle (oracle/q4_oracle.cpp).

TEST INFRASTRUCTURE ONLY.  Imported by the tests, the smoke check and the timed
CPU baseline; the product package never imports it.  It marshals numpy arrays
into the oracle's plain C structs and orchestrates whole-network passes (layer
loops); all arithmetic lives in the C++ file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "q4_oracle.cpp")
_LIB = os.path.join(_HERE, "libq4oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with plain -O2 (no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
                               "-pthread", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class Act(C.Structure):
    _fields_ = [("scale", C.c_float), ("inv_scale", C.c_float), ("zero_point", C.c_int32),
                ("bits", C.c_int32), ("is_signed", C.c_int32)]

    def lo(self):
        return -(1 << (self.bits - 1)) if self.is_signed else 0

    def hi(self):
        return (1 << (self.bits - 1)) - 1 if self.is_signed else (1 << self.bits) - 1


class _Linear(C.Structure):
    _fields_ = [("w", C.c_void_p), ("s_w", C.c_void_p), ("bias", C.c_void_p),
                ("J", C.c_int32), ("K", C.c_int32)]


class _Lstm(C.Structure):
    _fields_ = [("w_ih", C.c_void_p), ("s_wih", C.c_void_p), ("w_hh", C.c_void_p),
                ("s_whh", C.c_void_p), ("bias", C.c_void_p), ("K", C.c_int32), ("H", C.c_int32)]


class _Joint(C.Structure):
    _fields_ = [("z_act", Act), ("out", _Linear)]


class _Pred(C.Structure):
    _fields_ = [("emb", C.c_void_p), ("V", C.c_int32), ("E", C.c_int32), ("emb_act", Act),
                ("lstm", _Lstm), ("hid_act", Act), ("proj", _Linear)]


class _Lm(C.Structure):
    _fields_ = [("emb", C.c_void_p), ("V", C.c_int32), ("E", C.c_int32), ("emb_act", Act),
                ("n_layers", C.c_int32), ("lstm", _Lstm * 2), ("hid_act", Act * 2),
                ("bott", _Linear), ("bott_act", Act), ("out", _Linear)]


class _Decoder(C.Structure):
    _fields_ = [("pred", _Pred), ("joint", _Joint), ("src", _Lm), ("tgt", _Lm),
                ("lambda_t", C.c_float), ("lambda_s", C.c_float), ("rho", C.c_float),
                ("W", C.c_int32), ("U_max", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_absmax.restype = C.c_float
        _lib.orc_quant_calls.restype = C.c_int64
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


# ------------------------------------------------------------- quantizers
def act_symmetric(alpha: float, bits: int) -> Act:
    a = Act()
    lib().orc_act_symmetric(C.c_float(alpha), C.c_int32(bits), C.byref(a))
    return a


def act_asymmetric(lo: float, hi: float, bits: int) -> Act:
    a = Act()
    lib().orc_act_asymmetric(C.c_float(lo), C.c_float(hi), C.c_int32(bits), C.byref(a))
    return a


def absmax(x: np.ndarray) -> float:
    x = _c(x, np.float32)
    return float(lib().orc_absmax(_p(x), C.c_int64(x.size)))


def quantize(x: np.ndarray, act: Act) -> np.ndarray:
    x = _c(x, np.float32)
    q = np.empty(x.shape, dtype=np.int16)
    lib().orc_quantize(_p(x), C.c_int64(x.size), C.byref(act), _p(q))
    return q


def quantize_frames(x: np.ndarray, act: Act) -> np.ndarray:
    """Eq. 2 on [..., F], one quantizer call per frame (leading dimensions)."""
    x = _c(x, np.float32)
    q = np.empty(x.shape, dtype=np.int16)
    F = x.shape[-1]
    lib().orc_quantize_frames(_p(x), C.c_int64(x.size // F), C.c_int64(F), C.byref(act), _p(q))
    return q


def quant_calls_reset() -> None:
    lib().orc_quant_calls_reset()


def quant_calls() -> int:
    """Activation-quantizer calls made by the oracle since the last reset (Section 3.4)."""
    return int(lib().orc_quant_calls())


def dequantize(q: np.ndarray, act: Act) -> np.ndarray:
    q = _c(q, np.int16)
    x = np.empty(q.shape, dtype=np.float32)
    lib().orc_dequantize(_p(q), C.c_int64(q.size), C.byref(act), _p(x))
    return x


def quantize_weights(w: np.ndarray, row_scale: np.ndarray, bits: int) -> np.ndarray:
    w = _c(w, np.float32)
    s = _c(row_scale, np.float32)
    q = np.empty(w.shape, dtype=np.int8)
    lib().orc_quantize_weights(_p(w), C.c_int64(w.shape[0]), C.c_int64(w.shape[1]), _p(s),
                               C.c_int32(bits), _p(q))
    return q


def pack4(q: np.ndarray, k_pad: int, pad_code: int = 0) -> np.ndarray:
    q = _c(q, np.int16)
    rows, k = q.shape
    out = np.empty((rows, k_pad // 2), dtype=np.uint8)
    lib().orc_pack4(_p(q), C.c_int64(rows), C.c_int64(k), C.c_int64(k_pad), C.c_int32(pad_code),
                    _p(out))
    return out


def unpack4(b: np.ndarray, k: int, is_signed: bool) -> np.ndarray:
    b = _c(b, np.uint8)
    rows, kp2 = b.shape
    q = np.empty((rows, k), dtype=np.int16)
    lib().orc_unpack4(_p(b), C.c_int64(rows), C.c_int64(k), C.c_int64(kp2 * 2),
                      C.c_int32(1 if is_signed else 0), _p(q))
    return q


def pack2(q: np.ndarray, k_pad: int) -> np.ndarray:
    """2-bit codes (-2..1) -> four per byte."""
    q = _c(q, np.int16)
    rows, k = q.shape
    out = np.empty((rows, k_pad // 4), dtype=np.uint8)
    lib().orc_pack2(_p(q), C.c_int64(rows), C.c_int64(k), C.c_int64(k_pad), _p(out))
    return out


def unpack2(b: np.ndarray, k: int) -> np.ndarray:
    b = _c(b, np.uint8)
    rows, kp4 = b.shape
    q = np.empty((rows, k), dtype=np.int16)
    lib().orc_unpack2(_p(b), C.c_int64(rows), C.c_int64(k), C.c_int64(kp4 * 4), _p(q))
    return q


def activations(x: np.ndarray):
    """The oracle's fp32 2^x, sigmoid and tanh on an array."""
    x = _c(x, np.float32)
    ex, sg, th = np.empty_like(x), np.empty_like(x), np.empty_like(x)
    lib().orc_activations(_p(x), C.c_int64(x.size), _p(ex), _p(sg), _p(th))
    return ex, sg, th


def cells(pre_i, pre_f, pre_g, pre_o, c_prev):
    """The oracle's fp32 LSTM cell update on arrays of pre-activations: returns (c, h)."""
    a = [_c(v, np.float32) for v in (pre_i, pre_f, pre_g, pre_o, c_prev)]
    c, h = np.empty_like(a[0]), np.empty_like(a[0])
    lib().orc_cells(*[_p(v) for v in a], C.c_int64(a[0].size), _p(c), _p(h))
    return c, h


def int_matmul(w: np.ndarray, xq: np.ndarray, zero_point: int = 0) -> np.ndarray:
    w = _c(w, np.int8)
    xq = _c(xq, np.int16)
    J, K = w.shape
    M = xq.shape[0]
    acc = np.empty((M, J), dtype=np.int32)
    lib().orc_int_matmul(_p(w), C.c_int32(J), C.c_int32(K), _p(xq), C.c_int32(zero_point),
                         C.c_int32(M), _p(acc))
    return acc


# ------------------------------------------------- struct builders (keep refs)
class _Keep:
    """Owns the numpy buffers a C struct points into."""

    def __init__(self):
        self.refs = []

    def arr(self, a, dtype):
        a = _c(a, dtype)
        self.refs.append(a)
        return a.ctypes.data


def _mk_linear(keep: _Keep, lw) -> _Linear:
    J, K = lw.w.codes.shape
    return _Linear(keep.arr(lw.w.codes, np.int8), keep.arr(lw.w.scale, np.float32),
                   keep.arr(lw.bias, np.float32) if lw.bias is not None else None, J, K)


def _mk_lstm(keep: _Keep, lw) -> _Lstm:
    G, K = lw.w_ih.codes.shape
    return _Lstm(keep.arr(lw.w_ih.codes, np.int8), keep.arr(lw.w_ih.scale, np.float32),
                 keep.arr(lw.w_hh.codes, np.int8), keep.arr(lw.w_hh.scale, np.float32),
                 keep.arr(lw.bias, np.float32) if lw.bias is not None else None, K, G // 4)


class Lstm:
    """A list of per-direction LSTM weights as a contiguous C array."""

    def __init__(self, dirs: Sequence):
        self.keep = _Keep()
        self.n = len(dirs)
        self.c = (_Lstm * self.n)(*[_mk_lstm(self.keep, d) for d in dirs])
        self.H = self.c[0].H
        self.K = self.c[0].K


class Linear:
    def __init__(self, lw):
        self.keep = _Keep()
        self.c = _mk_linear(self.keep, lw)
        self.J, self.K = self.c.J, self.c.K


def linear(L: Linear, xq: np.ndarray, act: Act, want_acc: bool = False):
    xq = _c(xq, np.int16)
    M = xq.shape[0]
    out = np.empty((M, L.J), dtype=np.float32)
    acc = np.empty((M, L.J), dtype=np.int32) if want_acc else None
    lib().orc_linear(C.byref(L.c), _p(xq), C.byref(act), C.c_int32(M), _p(out), _p(acc))
    return (out, acc) if want_acc else out


def lstm_step(L: Lstm, xq, x_act: Act, hq_in, c_in, hid_act: Act, x_scale_row=None, d: int = 0):
    """One step for N rows; returns dict(hq, c, h, acc_ih, acc_hh, gates)."""
    xq = _c(xq, np.int16)
    hq_in = _c(hq_in, np.int16)
    c_in = _c(c_in, np.float32)
    N, H = hq_in.shape
    G = 4 * H
    r = dict(hq=np.empty((N, H), np.int16), c=np.empty((N, H), np.float32),
             h=np.empty((N, H), np.float32), acc_ih=np.empty((N, G), np.int32),
             acc_hh=np.empty((N, G), np.int32), gates=np.empty((N, G), np.float32))
    xs = None if x_scale_row is None else _c(x_scale_row, np.float32)
    lib().orc_lstm_step(C.byref(L.c[d]), _p(xq), C.byref(x_act), _p(xs), _p(hq_in), _p(c_in),
                        C.byref(hid_act), C.c_int32(N), _p(r["hq"]), _p(r["c"]), _p(r["h"]),
                        _p(r["acc_ih"]), _p(r["acc_hh"]), _p(r["gates"]))
    return r


def lstm_step_plain(L: Lstm, xq, x_act: Act, hq_in, c_in, hid_act: Act, x_scale_row=None, d: int = 0):
    """The textbook step in double (libm gates); returns dict(hq, c, h, tie) where tie is the
    distance of h / s from the nearest rounding boundary in code units."""
    xq = _c(xq, np.int16)
    hq_in = _c(hq_in, np.int16)
    c_in = _c(c_in, np.float32)
    N, H = hq_in.shape
    r = dict(hq=np.empty((N, H), np.int16), c=np.empty((N, H), np.float32),
             h=np.empty((N, H), np.float32), tie=np.empty((N, H), np.float32))
    xs = None if x_scale_row is None else _c(x_scale_row, np.float32)
    lib().orc_lstm_step_plain(C.byref(L.c[d]), _p(xq), C.byref(x_act), _p(xs), _p(hq_in), _p(c_in),
                              C.byref(hid_act), C.c_int32(N), _p(r["hq"]), _p(r["c"]), _p(r["h"]),
                              _p(r["tie"]))
    return r


def lstm_layer_inner(L: Lstm, x, x_act: Act, hid_act: Act) -> np.ndarray:
    """Layer under Inner quantizer placement: real-valued x [T,B,K] in, real-valued h out."""
    x = _c(x, np.float32)
    T, B, K = x.shape
    assert K == L.K
    h = np.empty((T, B, L.n * L.H), dtype=np.float32)
    lib().orc_lstm_layer_inner(L.c, C.c_int32(L.n), _p(x), C.byref(x_act), C.c_int32(T), C.c_int32(B),
                               C.byref(hid_act), _p(h))
    return h


def joint_z_plain(e, p, z_act: Act):
    """tanh(e * p) in double -> fp32 -> codes; returns (zq, tie)."""
    e = _c(e, np.float32)
    p = _c(p, np.float32)
    zq = np.empty(e.shape, np.int16)
    tie = np.empty(e.shape, np.float32)
    lib().orc_joint_z_plain(_p(e), _p(p), C.c_int64(e.size), C.byref(z_act), _p(zq), _p(tie))
    return zq, tie


def linear_plain(L: Linear, xq: np.ndarray, act: Act) -> np.ndarray:
    """W x + b on de-quantized operands, in double."""
    xq = _c(xq, np.int16)
    M = xq.shape[0]
    out = np.empty((M, L.J), dtype=np.float64)
    lib().orc_linear_plain(C.byref(L.c), _p(xq), C.byref(act), C.c_int32(M), _p(out))
    return out


def lstm_layer(L: Lstm, xq, x_act: Act, hid_act: Act, out_act: Optional[Act] = None,
               x_scale_b=None, want=("h",), n_threads: int = 8):
    """Whole layer over xq [T,B,K]; returns dict with yq and the requested extras
    among h, hq_hid, c_n, acc_ih, acc_hh."""
    xq = _c(xq, np.int16)
    T, B, K = xq.shape
    assert K == L.K
    dirs, H = L.n, L.H
    out_act = out_act or hid_act
    r = dict(yq=np.empty((T, B, dirs * H), np.int16))
    if "h" in want:
        r["h"] = np.empty((T, B, dirs * H), np.float32)
    if "hq_hid" in want:
        r["hq_hid"] = np.empty((T, B, dirs * H), np.int16)
    if "c_n" in want:
        r["c_n"] = np.empty((dirs, B, H), np.float32)
    if "acc_ih" in want:
        r["acc_ih"] = np.empty((T, B, dirs, 4 * H), np.int32)
    if "acc_hh" in want:
        r["acc_hh"] = np.empty((T, B, dirs, 4 * H), np.int32)
    xs = None if x_scale_b is None else _c(x_scale_b, np.float32)
    lib().orc_lstm_layer(L.c, C.c_int32(dirs), _p(xq), C.byref(x_act), _p(xs), C.c_int32(T),
                         C.c_int32(B), C.byref(hid_act), C.byref(out_act), _p(r["yq"]),
                         _p(r.get("hq_hid")), _p(r.get("h")), _p(r.get("c_n")),
                         _p(r.get("acc_ih")), _p(r.get("acc_hh")), C.c_int32(n_threads))
    return r


def lstm_layer_fp32(L: Lstm, x: np.ndarray) -> np.ndarray:
    x = _c(x, np.float32)
    T, B, K = x.shape
    h = np.empty((T, B, L.n * L.H), dtype=np.float32)
    lib().orc_lstm_layer_fp32(L.c, C.c_int32(L.n), _p(x), C.c_int32(T), C.c_int32(B), _p(h))
    return h


def log_softmax(logits: np.ndarray) -> np.ndarray:
    z = _c(logits, np.float32)
    M, V = z.shape
    lp = np.empty((M, V), dtype=np.float32)
    lib().orc_log_softmax(_p(z), C.c_int32(M), C.c_int32(V), _p(lp))
    return lp


# ------------------------------------------------------------ encoder pass
def encoder_forward_inner(enc, features: np.ndarray):
    """The encoder's LSTM stack under Inner quantizer placement (Section 3.4): real-valued
    tensors travel between cells and every cell quantizes its two inputs on entry.  FIX
    boundaries only.  Returns the real-valued output of the last layer [T,B,2H]."""
    x = np.asarray(features, dtype=np.float32)
    assert not enc.in_max
    x_act = act_symmetric(enc.in_clip, enc.in_bits)
    for dirs in enc.layers:
        hid_act = act_symmetric(dirs[0].hid_alpha, dirs[0].hid_bits)
        x = lstm_layer_inner(Lstm(dirs), x, x_act, hid_act)
        x_act = hid_act
    return x


def encoder_forward(enc, features: np.ndarray, n_threads: int = 8, want_layers: bool = False):
    """Features [T,B,F] (fp16/fp32) -> quantize -> L bidirectional layers ->
    projection.  The first layer's input boundary is FIX (enc.in_clip) or, with
    enc.in_max, the per-utterance MAX boundary.  Layer l's cell output is
    quantized once with boundary hid_alpha[l]; when layer l+1 runs at another
    precision a second code at that precision is made from the same float."""
    x = np.asarray(features, dtype=np.float32)
    T, B, F = x.shape
    x_scale_b = None
    if enc.in_max:
        x_act = act_symmetric(1.0, enc.in_bits)
        xq = np.empty((T, B, F), dtype=np.int16)
        x_scale_b = np.empty(B, dtype=np.float32)
        for b in range(B):
            a = act_symmetric(absmax(x[:, b, :]), enc.in_bits)
            xq[:, b, :] = quantize_frames(x[:, b, :], a)
            x_scale_b[b] = a.scale
    else:
        x_act = act_symmetric(enc.in_clip, enc.in_bits)
        xq = quantize_frames(x, x_act)          # the network input: one call per frame
    outs = []
    for l, dirs in enumerate(enc.layers):
        lw = dirs[0]
        hid_act = act_symmetric(lw.hid_alpha, lw.hid_bits)
        nxt_bits = enc.layers[l + 1][0].w_ih.bits if l + 1 < len(enc.layers) else (
            enc.proj.w.bits if enc.proj is not None else lw.hid_bits)
        out_act = act_symmetric(lw.hid_alpha, nxt_bits)
        L = Lstm(dirs)
        r = lstm_layer(L, xq, x_act, hid_act, out_act, x_scale_b=x_scale_b,
                       want=("h",) if want_layers else (), n_threads=n_threads)
        xq, x_act, x_scale_b = r["yq"], out_act, None
        if want_layers:
            outs.append(r)
    res = {"yq": xq, "y_act": x_act, "layers": outs}
    if enc.proj is not None:
        P = Linear(enc.proj)
        res["e"] = linear(P, xq.reshape(T * B, -1), x_act).reshape(T, B, -1)
    return res


# ------------------------------------------------------------ decoder side
class Decoder:
    def __init__(self, dw):
        k = self.keep = _Keep()
        d = self.c = _Decoder()
        self.dw = dw
        V, E = dw.pred.emb.shape
        d.pred = _Pred(k.arr(dw.pred.emb, np.float32), V, E,
                       act_symmetric(dw.pred.emb_alpha, getattr(dw, "emb_bits", 4)),
                       _mk_lstm(k, dw.pred.lstm),
                       act_symmetric(dw.pred.lstm.hid_alpha, dw.pred.lstm.hid_bits),
                       _mk_linear(k, dw.pred.proj))
        d.joint = _Joint(act_symmetric(1.0, dw.joint.z_bits), _mk_linear(k, dw.joint.out))
        d.src = self._lm(dw.src)
        d.tgt = self._lm(dw.tgt)
        d.lambda_t, d.lambda_s, d.rho = dw.lambda_t, dw.lambda_s, dw.rho
        d.W, d.U_max = dw.W, dw.U_max
        self.V, self.D = V, dw.pred.proj.w.codes.shape[0]

    def _lm(self, m) -> _Lm:
        k = self.keep
        V, E = m.emb.shape
        lm = _Lm()
        lm.emb, lm.V, lm.E = k.arr(m.emb, np.float32), V, E
        # learned-boundary input quantizers: asymmetric at 4 bits (Eq. 2); at 8 bits symmetric with
        # the wider of the two boundaries (no clipping is added, codes stay signed)
        wide = getattr(m, "act_bits", 4) == 8
        lm.emb_act = act_symmetric(max(-m.emb_lo, m.emb_hi), 8) if wide else act_asymmetric(m.emb_lo, m.emb_hi, 4)
        lm.n_layers = len(m.lstm)
        for i, l in enumerate(m.lstm):
            lm.lstm[i] = _mk_lstm(k, l)
            lm.hid_act[i] = act_symmetric(l.hid_alpha, l.hid_bits)
        lm.bott = _mk_linear(k, m.bott)
        lm.bott_act = act_symmetric(max(-m.bott_lo, m.bott_hi), 8) if wide else act_asymmetric(m.bott_lo, m.bott_hi, 4)
        lm.out = _mk_linear(k, m.out)
        return lm


def joint(dec: Decoder, e: np.ndarray, p: np.ndarray, want_zq: bool = False):
    e = _c(e, np.float32)
    p = _c(p, np.float32)
    N, D = e.shape
    lp = np.empty((N, dec.V), dtype=np.float32)
    zq = np.empty((N, D), dtype=np.int16) if want_zq else None
    acc = np.empty((N, dec.V), dtype=np.int32) if want_zq else None
    lib().orc_joint(C.byref(dec.c.joint), _p(e), _p(p), C.c_int32(N), _p(lp), _p(zq), _p(acc))
    return (lp, zq, acc) if want_zq else lp


def pred_joint_forced(dec: Decoder, e: np.ndarray, frame_idx: np.ndarray, tokens: np.ndarray,
                      want_state: bool = False, n_threads: int = 8):
    """e [R,D]; frame_idx, tokens [N,S].  Returns logp [N,S,V] (and hq, c, p)."""
    e = _c(e, np.float32)
    fi = _c(frame_idx, np.int32)
    tk = _c(tokens, np.int32)
    N, S = tk.shape
    Hp = dec.c.pred.lstm.H
    lp = np.empty((N, S, dec.V), dtype=np.float32)
    hq = np.empty((N, S, Hp), np.int16) if want_state else None
    c = np.empty((N, S, Hp), np.float32) if want_state else None
    p = np.empty((N, S, dec.D), np.float32) if want_state else None
    lib().orc_pred_joint_forced(C.byref(dec.c.pred), C.byref(dec.c.joint), _p(e), _p(fi), _p(tk),
                                C.c_int32(N), C.c_int32(S), _p(lp), _p(hq), _p(c), _p(p),
                                C.c_int32(n_threads))
    return (lp, hq, c, p) if want_state else lp


def lm_forced(dec: Decoder, which: str, tokens: np.ndarray, n_threads: int = 8) -> np.ndarray:
    tk = _c(tokens, np.int32)
    N, S = tk.shape
    lp = np.empty((N, S, dec.V), dtype=np.float32)
    m = dec.c.src if which == "src" else dec.c.tgt
    lib().orc_lm_forced(C.byref(m), _p(tk), C.c_int32(N), C.c_int32(S), _p(lp),
                        C.c_int32(n_threads))
    return lp


def alsd(dec: Decoder, e: np.ndarray, utts: Optional[Sequence[int]] = None, trace: bool = True,
         n_threads: int = 8):
    """e [T,B,D].  Decodes the listed utterances (default all).  Returns dict:
    tokens [n,U_max], len [n], score [n], finals_n [n] and, with trace, parent /
    token / score / t / u [n, T+U_max, W] and n_slots [n, T+U_max]."""
    e = _c(e, np.float32)
    T, B, D = e.shape
    utts = np.arange(B, dtype=np.int32) if utts is None else _c(utts, np.int32)
    n = len(utts)
    W, U = dec.c.W, dec.c.U_max
    IT = T + U
    r = dict(tokens=np.zeros((n, max(U, 1)), np.int32), len=np.zeros(n, np.int32),
             score=np.zeros(n, np.float32), finals_n=np.zeros(n, np.int32),
             finals_tokens=np.zeros((n, W, max(U, 1)), np.int32),
             finals_len=np.zeros((n, W), np.int32), finals_score=np.zeros((n, W), np.float32))
    if trace:
        r.update(parent=np.full((n, IT, W), -1, np.int32), token=np.full((n, IT, W), -1, np.int32),
                 tscore=np.zeros((n, IT, W), np.float32), t=np.zeros((n, IT, W), np.int32),
                 u=np.zeros((n, IT, W), np.int32), n_slots=np.zeros((n, IT), np.int32))
    lib().orc_alsd_batch(C.byref(dec.c), _p(e), C.c_int32(T), C.c_int32(B), _p(utts), C.c_int32(n),
                         _p(r["tokens"]), _p(r["len"]), _p(r["score"]), _p(r.get("parent")),
                         _p(r.get("token")), _p(r.get("tscore")), _p(r.get("t")), _p(r.get("u")),
                         _p(r.get("n_slots")), _p(r["finals_n"]), _p(r["finals_tokens"]),
                         _p(r["finals_len"]), _p(r["finals_score"]), C.c_int32(n_threads))
    return r


def tsd(dec: Decoder, e: np.ndarray, S_max: int, utts: Optional[Sequence[int]] = None, trace: bool = True,
        n_threads: int = 8):
    """Time-synchronous search, at most S_max labels per frame.  e [T,B,D].  Returns dict like alsd():
    tokens, len, score, finals_* and, with trace, parent / token / tscore / u [n, T (S_max+1), W] and
    n_slots [n, T (S_max+1)] (frame-close steps hold parent = first proposing slot, token = -1 - step)."""
    e = _c(e, np.float32)
    T, B, D = e.shape
    utts = np.arange(B, dtype=np.int32) if utts is None else _c(utts, np.int32)
    n = len(utts)
    W, U = dec.c.W, dec.c.U_max
    IT = T * (S_max + 1)
    r = dict(tokens=np.zeros((n, max(U, 1)), np.int32), len=np.zeros(n, np.int32),
             score=np.zeros(n, np.float32), finals_n=np.zeros(n, np.int32),
             finals_tokens=np.zeros((n, W, max(U, 1)), np.int32),
             finals_len=np.zeros((n, W), np.int32), finals_score=np.zeros((n, W), np.float32))
    if trace:
        r.update(parent=np.full((n, IT, W), -1, np.int32), token=np.zeros((n, IT, W), np.int32),
                 tscore=np.zeros((n, IT, W), np.float32), u=np.zeros((n, IT, W), np.int32),
                 n_slots=np.zeros((n, IT), np.int32))
    lib().orc_tsd_batch(C.byref(dec.c), _p(e), C.c_int32(T), C.c_int32(B), C.c_int32(S_max), _p(utts),
                        C.c_int32(n), _p(r["tokens"]), _p(r["len"]), _p(r["score"]), _p(r.get("parent")),
                        _p(r.get("token")), _p(r.get("tscore")), _p(r.get("u")), _p(r.get("n_slots")),
                        _p(r["finals_n"]), _p(r["finals_tokens"]), _p(r["finals_len"]),
                        _p(r["finals_score"]), C.c_int32(n_threads))
    return r


def sequence_score(dec: Decoder, e_utt: np.ndarray, y: Sequence[int]):
    """Eq. 1 score of one label string via the transducer forward recursion."""
    e = _c(e_utt, np.float32)
    T = e.shape[0]
    yy = _c(np.asarray(y, dtype=np.int32).reshape(-1), np.int32)
    s = C.c_float()
    a, b, c = C.c_double(), C.c_double(), C.c_double()
    lib().orc_sequence_score(C.byref(dec.c), _p(e), C.c_int32(T), _p(yy), C.c_int32(len(yy)),
                             C.byref(s), C.byref(a), C.byref(b), C.byref(c))
    return s.value, a.value, b.value, c.value


def features(mel: np.ndarray) -> np.ndarray:
    """[T100, M] fp32 -> [T100/2, 6M] fp32 (caller rounds to fp16)."""
    mel = _c(mel, np.float32)
    T100, M = mel.shape
    out = np.empty((T100 // 2, 6 * M), dtype=np.float32)
    lib().orc_features(_p(mel), C.c_int32(T100), C.c_int32(M), _p(out))
    return out
