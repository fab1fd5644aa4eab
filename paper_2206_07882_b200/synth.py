"""Seeded synthetic inputs for the INT4 RNN-T workloads.

This module only draws numbers: a counter-based SplitMix64 stream keyed by
(seed, tensor name, element index), uniforms from the top 24 bits, normals by
Box-Muller in double.  It holds none of the method's arithmetic (no quantizer,
no packing, no network code), so that the CPU oracle and the CUDA library can
both be fed from it without sharing anything else.

The recipes follow the shapes of the paper's model (Section 2: six
bidirectional LSTM encoder layers, an embedding + LSTM + linear prediction
network, a multiplicative joint network, and two LSTM language models for
density-ratio fusion) at the synthetic dimensions used for measurement.  The
paper's audio (Switchboard / Hub5 / RT-03) and trained weights are not
available; these tensors stand in for them.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function (Steele, Lea, Flood 2014) on uint64 arrays."""
    with np.errstate(over="ignore"):
        z = (z + _GOLDEN).astype(_U64)
        z = ((z ^ (z >> _U64(30))) * _M1).astype(_U64)
        z = ((z ^ (z >> _U64(27))) * _M2).astype(_U64)
        return (z ^ (z >> _U64(31))).astype(_U64)


class Stream:
    """Counter-based generator: element i of tensor `name` under `seed` is a
    pure function of (seed, name, i); shapes and draw order do not matter."""

    def __init__(self, seed: int):
        self.seed = int(seed)

    def _key(self, name: str) -> np.uint64:
        tid = zlib.crc32(name.encode("utf-8"))
        k = _mix(np.array([self.seed], dtype=_U64))
        k = _mix(k ^ _U64(tid))
        return k[0]

    def bits(self, name: str, n: int, lane: int = 0) -> np.ndarray:
        idx = np.arange(n, dtype=_U64)
        with np.errstate(over="ignore"):
            ctr = (idx * _U64(4) + _U64(lane)) * _GOLDEN + self._key(name)
        return _mix(ctr.astype(_U64))

    def uniform01(self, name: str, n: int, lane: int = 0) -> np.ndarray:
        """Uniform in [0,1) with 24-bit resolution, as float64."""
        return (self.bits(name, n, lane) >> _U64(40)).astype(np.float64) / float(1 << 24)

    def uniform(self, name: str, shape, lo: float, hi: float) -> np.ndarray:
        n = int(np.prod(shape))
        return (lo + (hi - lo) * self.uniform01(name, n)).reshape(shape)

    def normal(self, name: str, shape, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
        n = int(np.prod(shape))
        u1 = 1.0 - self.uniform01(name, n, 0)          # (0,1]
        u2 = self.uniform01(name, n, 1)
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        return (mean + std * z).reshape(shape)

    def integers(self, name: str, shape, lo: int, hi: int) -> np.ndarray:
        """Uniform integers in [lo, hi] inclusive, as int64."""
        n = int(np.prod(shape))
        span = hi - lo + 1
        v = (self.bits(name, n) >> _U64(11)).astype(np.float64) / float(1 << 53)
        return (lo + np.floor(v * span).astype(np.int64)).reshape(shape)


# --------------------------------------------------------------------------
# Plain containers (numbers only).  Weight codes are signed integers held one
# per int8; each side packs them into its own storage format.
# --------------------------------------------------------------------------
@dataclass
class QMat:
    """Integer weight matrix [rows, k] with one fp32 scale per output row."""
    codes: np.ndarray          # int8 [rows, k]
    scale: np.ndarray          # float32 [rows]
    bits: int = 4


@dataclass
class LstmW:
    w_ih: QMat                 # [4H, K]
    w_hh: QMat                 # [4H, H]
    bias: np.ndarray           # float32 [4H]
    hid_alpha: float = 1.0     # FIX boundary of the hidden-state quantizer
    hid_bits: int = 4


@dataclass
class LinearW:
    w: QMat                    # [J, K]
    bias: np.ndarray           # float32 [J]


@dataclass
class EncoderW:
    layers: List[List[LstmW]]  # [L][dirs]
    in_clip: float             # FIX boundary of the feature quantizer (ignored with in_max)
    in_bits: int
    in_max: bool               # per-utterance MAX boundary for the features
    proj: Optional[LinearW]    # encoder -> joint projection (2H -> D)


@dataclass
class PredW:
    emb: np.ndarray            # float32 [V, E]
    emb_alpha: float           # FIX +-alpha, symmetric
    lstm: LstmW
    proj: LinearW              # Hp -> D


@dataclass
class JointW:
    out: LinearW               # D -> V
    z_bits: int = 4            # precision of the quantized tanh(e*p) (boundary FIX +-1)


@dataclass
class LmW:
    emb: np.ndarray            # float32 [V, E]
    emb_lo: float              # learned-boundary (PACT-style) constants, asymmetric
    emb_hi: float
    lstm: List[LstmW]
    bott: LinearW              # H -> D
    bott_lo: float
    bott_hi: float
    out: LinearW               # D -> V
    act_bits: int = 4          # width of the two input quantizers; at 8 bits they are symmetric with
                               # the boundary max(|lo|, hi) (signed codes), at 4 bits asymmetric


@dataclass
class DecoderW:
    pred: PredW
    joint: JointW
    src: LmW
    tgt: LmW
    lambda_t: float = 0.5
    lambda_s: float = 0.3
    rho: float = 0.2
    W: int = 16
    U_max: int = 0
    emb_bits: int = 4          # width of the prediction network's input quantizer


def _qmat(st: Stream, name: str, rows: int, k: int, bits: int = 4) -> QMat:
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    codes = st.integers(name + ".q", (rows, k), lo, hi).astype(np.int8)
    scale = st.uniform(name + ".s", (rows,), 0.01, 0.05).astype(np.float32)
    if bits == 8:
        # keep the dequantized weight range of the 4-bit layers (same alpha)
        scale = (scale * np.float32(7.0 / 127.0)).astype(np.float32)
    if bits == 2:
        # codes -2..1 with the same boundary: one step is the whole boundary
        scale = (scale * np.float32(7.0)).astype(np.float32)
    return QMat(codes, scale, bits)


def _lstm(st: Stream, name: str, k: int, h: int, bits: int = 4, bias_std: float = 0.1,
          hid_alpha: float = 1.0, hid_bits: Optional[int] = None, wscale: float = 1.0) -> LstmW:
    w_ih = _qmat(st, name + ".w_ih", 4 * h, k, bits)
    w_hh = _qmat(st, name + ".w_hh", 4 * h, h, bits)
    if wscale != 1.0:
        w_ih.scale = (w_ih.scale * np.float32(wscale)).astype(np.float32)
        w_hh.scale = (w_hh.scale * np.float32(wscale)).astype(np.float32)
    if bias_std > 0:
        bias = st.normal(name + ".b", (4 * h,), 0.0, bias_std).astype(np.float32)
    else:
        bias = np.zeros(4 * h, dtype=np.float32)
    return LstmW(w_ih, w_hh, bias, hid_alpha, hid_bits if hid_bits is not None else bits)


def _linear(st: Stream, name: str, j: int, k: int, bits: int = 4, bias_std: float = 0.1,
            wscale: float = 1.0) -> LinearW:
    w = _qmat(st, name + ".w", j, k, bits)
    if wscale != 1.0:
        w.scale = (w.scale * np.float32(wscale)).astype(np.float32)
    bias = st.normal(name + ".b", (j,), 0.0, bias_std).astype(np.float32)
    return LinearW(w, bias)


# --------------------------------------------------------------------------
# Workload recipes
# --------------------------------------------------------------------------
def single_layer(seed: int = 0, T: int = 50, B: int = 4, K: int = 64, H: int = 128,
                 bits: int = 4, dirs: int = 1):
    """One LSTM layer: x ~ N(0,1) fp32 (clip 3.0 on the consumer's side), weight
    integers uniform over the code range, per-row scales U(.01,.05), zero bias."""
    st = Stream(seed)
    x = st.normal("x", (T, B, K)).astype(np.float32)
    layers = [_lstm(st, f"l0.d{d}", K, H, bits, bias_std=0.0) for d in range(dirs)]
    return {"x": x, "x_clip": 3.0, "layers": layers, "T": T, "B": B, "K": K, "H": H}


def encoder(seed: int = 1, T: int = 500, B: int = 32, F: int = 240, H: int = 640, L: int = 6,
            D: int = 256, first_layer_bits: int = 4, in_max: bool = False,
            with_proj: bool = True, features: bool = True, w_bits: int = 4, proj_bits: int = 4,
            layer_bits: int = 4):
    """Bidirectional LSTM encoder.  Features fp16 ~ N(0,1); input clip U(2.5,3.5);
    per-layer hidden boundary U(.9,1.0) (the paper observes MAX boundaries of LSTM
    outputs in [0.9,1], Section 3.2); biases N(0,.1)."""
    st = Stream(seed)
    out = {}
    if features:
        out["features"] = st.normal("features", (T, B, F)).astype(np.float16)
    in_clip = float(st.uniform("enc.in_clip", (1,), 2.5, 3.5)[0])
    alphas = st.uniform("enc.hid_alpha", (L,), 0.9, 1.0)
    layers = []
    for l in range(L):
        k = F if l == 0 else 2 * H
        bits = first_layer_bits if l == 0 else layer_bits
        # w_bits < 4: weight codes stored narrower than the activation codes (Table 1's 2/4 rows)
        wb = bits if bits == 8 else w_bits
        layers.append([_lstm(st, f"enc.l{l}.d{d}", k, H, wb, 0.1, float(alphas[l]), bits)
                       for d in range(2)])
    proj = _linear(st, "enc.proj", D, 2 * H, proj_bits) if with_proj else None
    out["enc"] = EncoderW(layers, in_clip, first_layer_bits, in_max, proj)
    out.update(T=T, B=B, F=F, H=H, L=L, D=D)
    return out


def _lm(st: Stream, name: str, V: int, E: int, H: int, n_layers: int, D: int, bits: int = 4) -> LmW:
    emb = st.normal(name + ".emb", (V, E), 0.0, 0.5).astype(np.float32)
    lo = -float(st.uniform(name + ".emb_lo", (1,), 1.0, 2.0)[0])
    hi = float(st.uniform(name + ".emb_hi", (1,), 1.0, 2.0)[0])
    alphas = st.uniform(name + ".hid_alpha", (n_layers,), 0.9, 1.0)
    lstm = [_lstm(st, f"{name}.l{l}", E if l == 0 else H, H, bits, 0.1, float(alphas[l]))
            for l in range(n_layers)]
    bott = _linear(st, name + ".bott", D, H, bits)
    blo = -float(st.uniform(name + ".bott_lo", (1,), 1.0, 2.0)[0])
    bhi = float(st.uniform(name + ".bott_hi", (1,), 1.0, 2.0)[0])
    out = _linear(st, name + ".out", V, D, bits)
    return LmW(emb, lo, hi, lstm, bott, blo, bhi, out, bits)


def decoder(seed: int = 3, V: int = 1024, E: int = 256, Hp: int = 1024, D: int = 256,
            Hs: int = 1024, Ht: int = 2048, tgt_layers: int = 2, out_bits: int = 4,
            W: int = 16, U_max: int = 150, lambda_t: float = 0.5, lambda_s: float = 0.3,
            rho: float = 0.2, rnnt_w_bits: int = 4, proj_bits: int = 4, all_bits: int = 4) -> DecoderW:
    """Prediction network, joint network and the two fusion LMs.  Embeddings
    N(0,.5); prediction-input boundary 1.25 and hidden boundary 1 (Section 3.2);
    learned LM input boundaries stand-ins alpha- ~ -U(1,2), alpha+ ~ U(1,2)."""
    st = Stream(seed)
    if all_bits == 8:      # the all-8-bit point of the paper's run-time figure: every weight and quantizer at 8
        rnnt_w_bits = out_bits = proj_bits = 8
    pred = PredW(st.normal("pred.emb", (V, E), 0.0, 0.5).astype(np.float32), 1.25,
                 _lstm(st, "pred.lstm", E, Hp, rnnt_w_bits, 0.1, 1.0, all_bits),
                 _linear(st, "pred.proj", D, Hp, proj_bits if proj_bits != 4 else rnnt_w_bits))
    joint = JointW(_linear(st, "joint.out", V, D, out_bits if out_bits != 4 else rnnt_w_bits), out_bits)
    src = _lm(st, "src", V, E, Hs, 1, D, all_bits)
    tgt = _lm(st, "tgt", V, E, Ht, tgt_layers, D, all_bits)
    return DecoderW(pred, joint, src, tgt, lambda_t, lambda_s, rho, W, U_max, all_bits)


def enc_frames(seed: int, T: int, B: int, dim: int = 1280) -> np.ndarray:
    """Stand-in for the last encoder layer's output: fp16 ~ N(0,1), [T, B, dim]."""
    return Stream(seed).normal("enc_out", (T, B, dim)).astype(np.float16)


def labels(seed: int, rows: int, steps: int, V: int) -> np.ndarray:
    """Teacher-forced label sequences, uniform in 1..V-1 (0 is blank / start)."""
    return Stream(seed).integers("labels", (rows, steps), 1, V - 1).astype(np.int32)


def logmel(seed: int, B: int, T100: int = 1000, n_mel: int = 40) -> np.ndarray:
    """log-mel stand-in, fp32 ~ N(0,1), [B, T100, n_mel] at 100 frames/s."""
    return Stream(seed).normal("logmel", (B, T100, n_mel)).astype(np.float32)


def paper_dimensions(seed: int = 5, T: int = 12, B: int = 2, U_max: int = 6, section_3_2: bool = False):
    """The model sizes the paper states in Section 2: 340-d encoder input, 6 bidirectional layers of
    640 cells, 256-d encoder/prediction outputs, prediction LSTM of 768 cells behind a small
    embedding (10-d reproduces the 2.6 M parameters quoted), 46 output characters, external LM of
    two 2048-cell layers with a 256 bottleneck, source LM shaped like the prediction network;
    fusion weights 0.7 / 0.5 / 0.2 as after Eq. 1.  section_3_2 = the precision assignment of
    Section 3.2: first encoder layer at 8 bits with the per-utterance MAX boundary on its input, the
    linear layers of the RNN-T (encoder and prediction projections, joint output) at 8 bits,
    everything else, both LMs included, at 4 bits."""
    kw_e = dict(first_layer_bits=8, in_max=True, proj_bits=8) if section_3_2 else {}
    kw_d = dict(out_bits=8, proj_bits=8) if section_3_2 else {}
    enc = encoder(seed, T=T, B=B, F=340, H=640, L=6, D=256, **kw_e)
    dec = decoder(seed + 1000, V=46, E=10, Hp=768, D=256, Hs=768, Ht=2048, tgt_layers=2, U_max=U_max,
                  lambda_t=0.7, lambda_s=0.5, rho=0.2, **kw_d)
    return enc, dec


def weight_storage(enc: EncoderW, dec: DecoderW, with_src_lm: bool = False) -> dict:
    """Weight-matrix parameters by storage width (biases and embeddings aside): count, the share
    held at 4 bits, bytes as stored and the ratio to fp32 storage."""
    mats = [m for layer in enc.layers for l in layer for m in (l.w_ih, l.w_hh)]
    if enc.proj is not None:
        mats.append(enc.proj.w)
    mats += [dec.pred.lstm.w_ih, dec.pred.lstm.w_hh, dec.pred.proj.w, dec.joint.out.w]
    for m in [dec.tgt] + ([dec.src] if with_src_lm else []):
        mats += [w for l in m.lstm for w in (l.w_ih, l.w_hh)] + [m.bott.w, m.out.w]
    n = sum(m.codes.size for m in mats)
    by = sum(m.codes.size * m.bits / 8 for m in mats)
    return {"params": n, "frac_4bit": sum(m.codes.size for m in mats if m.bits == 4) / n, "bytes": by,
            "compression": 4.0 * n / by}


def parameter_counts(enc: EncoderW, dec: DecoderW) -> dict:
    """Trainable parameters of a weight set (matrices, biases, embeddings) by component."""
    def lstm(l: LstmW) -> int:
        return l.w_ih.codes.size + l.w_hh.codes.size + l.bias.size

    def linear(l: LinearW) -> int:
        return l.w.codes.size + (l.bias.size if l.bias is not None else 0)

    def lm(m: LmW) -> int:
        return m.emb.size + sum(lstm(l) for l in m.lstm) + linear(m.bott) + linear(m.out)

    n_enc = sum(lstm(l) for layer in enc.layers for l in layer) + (linear(enc.proj) if enc.proj else 0)
    n_pred = dec.pred.emb.size + lstm(dec.pred.lstm) + linear(dec.pred.proj) + linear(dec.joint.out)
    return {"encoder": n_enc, "prediction": n_pred, "rnnt": n_enc + n_pred, "lm_ext": lm(dec.tgt),
            "lm_src": lm(dec.src)}


# Reduced-dimension suite for whole-search comparisons over many utterances.
def parity_suite(seed: int = 7, n_utt: int = 256, T: int = 32, V: int = 64):
    enc = encoder(seed, T=T, B=n_utt, F=48, H=64, L=2, D=32)
    dec = decoder(seed + 1000, V=V, E=32, Hp=128, D=32, Hs=128, Ht=256, tgt_layers=2,
                  U_max=T // 2)
    return enc, dec
