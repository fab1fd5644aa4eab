"""Pins for the oracle's quantized LSTM (CPU only).

The library routine is torch.nn.LSTM / LSTMCell in float64 (gate order i,f,g,o,
no peepholes, no projection).  On already-quantized inputs the integer form
acc * (s_x * s_w) equals the real-valued product of the dequantized operands
(Eq. 3), so one oracle step must reproduce LSTMCell on dequantized tensors; the
cell output must lie in [-1,1] (Section 3.2) and its code must be the quantizer
applied once to that output (Section 3.4).
"""
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2206_07882_b200 import synth
from test_oracle_quantizers import gold


def torch_cell(lw, dtype=torch.float64):
    G, K = lw.w_ih.codes.shape
    H = G // 4
    cell = torch.nn.LSTMCell(K, H, bias=True).to(dtype)
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(lw.w_ih.codes.astype(np.float64) * lw.w_ih.scale.astype(np.float64)[:, None]))
        cell.weight_hh.copy_(torch.from_numpy(lw.w_hh.codes.astype(np.float64) * lw.w_hh.scale.astype(np.float64)[:, None]))
        cell.bias_ih.copy_(torch.from_numpy(lw.bias.astype(np.float64)))
        cell.bias_hh.zero_()
    return cell


@pytest.mark.parametrize("signed_in", [True, False])
def test_step_equals_library_cell_on_dequantized_operands(signed_in):
    st = synth.Stream(5)
    K, H, N = 24, 16, 5
    lw = synth._lstm(st, "cell", K, H, 4, bias_std=0.3)
    rng = np.random.default_rng(0)
    x_act = O.act_symmetric(3.0, 4) if signed_in else O.act_asymmetric(-2.5, 3.5, 4)
    hid = O.act_symmetric(1.0, 4)
    xq = rng.integers(x_act.lo(), x_act.hi() + 1, (N, K)).astype(np.int16)
    hq = rng.integers(-7, 8, (N, H)).astype(np.int16)
    c = rng.normal(0, 1, (N, H)).astype(np.float32)
    r = O.lstm_step(O.Lstm([lw]), xq, x_act, hq, c, hid)
    cell = torch_cell(lw)
    with torch.no_grad():
        h1, c1 = cell(torch.from_numpy(O.dequantize(xq, x_act)).double(),
                      (torch.from_numpy(O.dequantize(hq, hid)).double(), torch.from_numpy(c).double()))
    np.testing.assert_allclose(r["c"], c1.numpy(), rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(r["h"], h1.numpy(), rtol=1e-6, atol=1e-6)
    assert np.abs(r["h"]).max() <= 1.0                                   # Section 3.2
    np.testing.assert_array_equal(r["hq"], O.quantize(r["h"], hid))      # quantized once, at the output
    # integer accumulators by 64-bit library matmul
    np.testing.assert_array_equal(r["acc_ih"], (xq.astype(np.int64) - x_act.zero_point) @ lw.w_ih.codes.astype(np.int64).T)
    np.testing.assert_array_equal(r["acc_hh"], hq.astype(np.int64) @ lw.w_hh.codes.astype(np.int64).T)
    # gate dump: i,f,o in (0,1), g in (-1,1), and c = f*c0 + i*g
    g = r["gates"].astype(np.float64)
    i_, f_, g_, o_ = g[:, :H], g[:, H:2 * H], g[:, 2 * H:3 * H], g[:, 3 * H:]
    np.testing.assert_allclose(f_ * c + i_ * g_, r["c"], atol=1e-6)
    np.testing.assert_allclose(o_ * np.tanh(r["c"].astype(np.float64)), r["h"], atol=1e-6)


def test_hand_case_one_cell_two_steps():
    # K = H = 1.  All numbers written out by hand: w_ih codes (i,f,g,o) = (2,-3,4,1),
    # w_hh = (1,2,-2,3), all row scales 0.5, bias (0.1,-0.2,0.3,0), x code 3 at s_x=0.5,
    # hidden quantizer alpha=1,b=4 (s=1/7).
    lw = synth.LstmW(synth.QMat(np.array([[2], [-3], [4], [1]], np.int8), np.full(4, 0.5, np.float32)),
                     synth.QMat(np.array([[1], [2], [-2], [3]], np.int8), np.full(4, 0.5, np.float32)),
                     np.array([0.1, -0.2, 0.3, 0.0], np.float32))
    L = O.Lstm([lw])
    x_act = O.act_symmetric(3.5, 4)          # s = 0.5
    hid = O.act_symmetric(1.0, 4)
    xq = np.array([[3]], np.int16)
    r1 = O.lstm_step(L, xq, x_act, np.zeros((1, 1), np.int16), np.zeros((1, 1), np.float32), hid)
    # step 1: pre = acc_ih*0.25 + bias = (1.6, -2.45, 3.3, 0.75)
    sig = lambda v: 1 / (1 + np.exp(-v))
    c1 = sig(1.6) * np.tanh(3.3)
    h1 = sig(0.75) * np.tanh(c1)
    assert r1["acc_ih"].tolist() == [[6, -9, 12, 3]] and r1["acc_hh"].tolist() == [[0, 0, 0, 0]]
    assert abs(r1["c"][0, 0] - c1) < 1e-6 and abs(r1["h"][0, 0] - h1) < 1e-6
    assert abs(c1 - 0.83202 * 0.99728) < 1e-4 and abs(h1 - 0.67918 * 0.68045) < 1e-4   # table values of sigmoid/tanh
    assert r1["hq"][0, 0] == 3                                          # 0.4619*7 = 3.23 -> 3
    r2 = O.lstm_step(L, xq, x_act, r1["hq"], r1["c"], hid)
    # step 2: h code 3 at s_h = 1/7 -> acc_hh = (3,6,-6,9), scaled by 0.5/7
    pre = np.array([6, -9, 12, 3]) * 0.25 + np.array([3, 6, -6, 9]) * (0.5 / 7) + np.array([0.1, -0.2, 0.3, 0.0])
    c2 = sig(pre[1]) * c1 + sig(pre[0]) * np.tanh(pre[2])
    h2 = sig(pre[3]) * np.tanh(c2)
    assert r2["acc_hh"].tolist() == [[3, 6, -6, 9]]
    assert abs(r2["c"][0, 0] - c2) < 1e-6 and abs(r2["h"][0, 0] - h2) < 1e-6
    assert r2["hq"][0, 0] == int(np.rint(h2 * 7))


def test_fp32_layer_equals_library_bidirectional_lstm():
    w = synth.single_layer(seed=3, T=9, B=3, K=10, H=6, dirs=2)
    for l in w["layers"]:
        l.bias[:] = np.linspace(-0.3, 0.3, l.bias.size)
    L = O.Lstm(w["layers"])
    got = O.lstm_layer_fp32(L, w["x"])
    ref = torch.nn.LSTM(10, 6, num_layers=1, bidirectional=True).double()
    with torch.no_grad():
        for d, suffix in enumerate(["", "_reverse"]):
            c = torch_cell(w["layers"][d])
            getattr(ref, "weight_ih_l0" + suffix).copy_(c.weight_ih)
            getattr(ref, "weight_hh_l0" + suffix).copy_(c.weight_hh)
            getattr(ref, "bias_ih_l0" + suffix).copy_(c.bias_ih)
            getattr(ref, "bias_hh_l0" + suffix).zero_()
        want, _ = ref(torch.from_numpy(w["x"]).double())
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-6, atol=1e-6)


def test_quantized_layer_is_the_step_iterated_and_concatenated():
    # the layer routine = the (pinned) step applied along time, direction 1 reversed,
    # outputs concatenated [fwd | bwd]; checked against a python loop over the step.
    w = synth.single_layer(seed=4, T=7, B=2, K=12, H=8, dirs=2)
    L = O.Lstm(w["layers"])
    x_act = O.act_symmetric(3.0, 4)
    hid = O.act_symmetric(1.0, 4)
    xq = O.quantize(w["x"], x_act)
    r = O.lstm_layer(L, xq, x_act, hid, want=("h", "c_n", "acc_ih", "acc_hh", "hq_hid"))
    T, B, H = 7, 2, 8
    for d in range(2):
        hq = np.zeros((B, H), np.int16)
        c = np.zeros((B, H), np.float32)
        order = range(T) if d == 0 else range(T - 1, -1, -1)
        for t in order:
            s = O.lstm_step(L, xq[t], x_act, hq, c, hid, d=d)
            hq, c = s["hq"], s["c"]
            np.testing.assert_array_equal(r["yq"][t, :, d * H:(d + 1) * H], hq)
            np.testing.assert_array_equal(r["h"][t, :, d * H:(d + 1) * H], s["h"])
            np.testing.assert_array_equal(r["acc_ih"][t, :, d], s["acc_ih"])
            np.testing.assert_array_equal(r["acc_hh"][t, :, d], s["acc_hh"])
        np.testing.assert_array_equal(r["c_n"][d], c)
    assert np.abs(r["h"]).max() <= 1.0
    # with boundary 1 no code is ever clamped: |code| <= 7
    assert r["yq"].min() >= -7 and r["yq"].max() <= 7


def test_second_code_at_other_precision_comes_from_same_float():
    w = synth.single_layer(seed=6, T=6, B=2, K=12, H=8, bits=8)
    L = O.Lstm(w["layers"])
    x_act = O.act_symmetric(3.0, 8)
    hid8, out4 = O.act_symmetric(1.0, 8), O.act_symmetric(1.0, 4)
    xq = O.quantize(w["x"], x_act)
    r = O.lstm_layer(L, xq, x_act, hid8, out4, want=("h", "hq_hid"))
    np.testing.assert_array_equal(r["hq_hid"], O.quantize(r["h"], hid8))
    np.testing.assert_array_equal(r["yq"], O.quantize(r["h"], out4))     # no double rounding
    same = O.lstm_layer(L, xq, x_act, hid8, hid8, want=("h",))
    np.testing.assert_array_equal(same["h"], r["h"])                     # recurrence unaffected by out_act


def test_int4_tracks_fp32_and_int8_tracks_closer():
    # Section 3.1: s is proportional to 1/(2^(b-1)-1), so going from 4 to 8 bits shrinks
    # the deviation from the unquantized network by about 127/7 = 18x.
    T, B, K, H = 50, 4, 64, 128
    dev = {}
    for bits in (4, 8):
        w = synth.single_layer(seed=0, T=T, B=B, K=K, H=H, bits=4)
        for l in w["layers"]:            # gentle weights: stay out of gate saturation
            l.w_ih.scale *= np.float32(0.2)
            l.w_hh.scale *= np.float32(0.2)
        L = O.Lstm(w["layers"])
        x_act = O.act_symmetric(3.0, bits)
        hid = O.act_symmetric(1.0, bits)
        xc = np.clip(w["x"], -3.0, 3.0)
        r = O.lstm_layer(L, O.quantize(w["x"], x_act), x_act, hid, want=("h",))
        ref = O.lstm_layer_fp32(L, xc)
        dev[bits] = float(np.sqrt(np.mean((r["h"] - ref) ** 2)))
        if bits == 4:
            cc = np.corrcoef(r["h"].ravel(), ref.ravel())[0, 1]
            assert cc > 0.95, cc
    ratio = dev[4] / dev[8]
    assert 9.0 < ratio < 36.0, (dev, ratio)


def test_outer_vs_inner_quantizer_calls():
    # Section 3.4: Inner 2*T*L, Outer T + T*L, ratio (L+1)/(2L); 45 % fewer in the encoder.
    # Both numbers are COUNTED: every call of the oracle's activation quantizer increments a
    # counter, and the two placements are two code paths that must give the same network output.
    g = gold()
    T, Lc = 5, int(g["outer_inner_L"])           # L = 12 cells: 6 layers x 2 directions
    enc = synth.encoder(seed=1, T=T, B=1, F=16, H=8, L=6, D=8, with_proj=False)
    O.quant_calls_reset()
    r = O.encoder_forward(enc["enc"], enc["features"], want_layers=True)
    outer = O.quant_calls()
    O.quant_calls_reset()
    h_inner = O.encoder_forward_inner(enc["enc"], enc["features"])
    inner = O.quant_calls()
    assert inner == 2 * T * Lc and outer == T + T * Lc
    assert abs(outer / inner - g["outer_inner_ratio"]) < 1e-9
    assert round(100 * (1 - outer / inner)) in (45, 46)
    assert abs(100 * (1 - outer / inner) - g["outer_inner_saving_percent"]) < 1.0
    # the placement changes the number of calls, not the result
    np.testing.assert_array_equal(h_inner, r["layers"][-1]["h"])
    # a batch of B sequences makes B times the calls (the count is per sequence)
    enc3 = synth.encoder(seed=1, T=T, B=3, F=16, H=8, L=6, D=8, with_proj=False)
    O.quant_calls_reset()
    O.encoder_forward(enc3["enc"], enc3["features"])
    assert O.quant_calls() == 3 * (T + T * Lc)


def test_encoder_layers_chain_and_projection():
    enc = synth.encoder(seed=2, T=6, B=3, F=16, H=8, L=3, D=8)
    E = enc["enc"]
    r = O.encoder_forward(E, enc["features"], want_layers=True)
    # layer l+1 consumes exactly layer l's output codes (Outer: the same tensor feeds both)
    x_act = O.act_symmetric(E.in_clip, 4)
    xq = O.quantize(enc["features"].astype(np.float32), x_act)
    for l in range(3):
        hid = O.act_symmetric(E.layers[l][0].hid_alpha, 4)
        rr = O.lstm_layer(O.Lstm(E.layers[l]), xq, x_act, hid)
        np.testing.assert_array_equal(rr["yq"], r["layers"][l]["yq"])
        xq, x_act = rr["yq"], hid
    want = O.dequantize(xq, x_act).astype(np.float64).reshape(18, 16) @ \
        (E.proj.w.codes.astype(np.float64) * E.proj.w.scale.astype(np.float64)[:, None]).T + E.proj.bias
    np.testing.assert_allclose(r["e"].reshape(18, 8), want, rtol=1e-5, atol=1e-6)


def test_encoder_per_utterance_max_input():
    # INT8 first layer with the MAX boundary per utterance (Section 3.2).
    enc = synth.encoder(seed=8, T=6, B=3, F=16, H=8, L=2, D=8, first_layer_bits=8, in_max=True)
    E = enc["enc"]
    f = enc["features"].astype(np.float32)
    r = O.encoder_forward(E, f, want_layers=True)
    # utterance b alone gives the same result as inside the batch
    for b in range(3):
        rb = O.encoder_forward(E, f[:, b:b + 1, :])
        np.testing.assert_array_equal(rb["yq"][:, 0], r["yq"][:, b])
    # MAX boundary: no clipping, the largest magnitude of each utterance maps to code 127
    for b in range(3):
        a = O.act_symmetric(O.absmax(f[:, b, :]), 8)
        assert abs(a.scale - np.abs(f[:, b, :]).max() / 127) < 1e-7
        assert np.abs(O.quantize(f[:, b, :], a)).max() == 127


def test_features_prologue_by_hand():
    # 4 frames of 1 mel bin: x = (1, 4, 9, 16); d = ((x1-x0)/2, (x2-x0)/2, (x3-x1)/2, (x3-x2)/2)
    mel = np.array([[1.0], [4.0], [9.0], [16.0]], np.float32)
    out = O.features(mel)
    d = np.array([1.5, 4.0, 6.0, 3.5])
    dd = np.array([(d[1] - d[0]) / 2, (d[2] - d[0]) / 2, (d[3] - d[1]) / 2, (d[3] - d[2]) / 2])
    want = np.array([[1, d[0], dd[0], 4, d[1], dd[1]], [9, d[2], dd[2], 16, d[3], dd[3]]])
    np.testing.assert_allclose(out, want, atol=1e-6)


def test_cell_update_against_textbook_formulas():
    # c = sigmoid(f) c_prev + sigmoid(i) tanh(g), h = sigmoid(o) tanh(c) evaluated in double
    st = synth.Stream(77)
    n = 200000
    pre = [st.normal(f"p{k}", (n,)).astype(np.float32) * np.float32(s) for k, s in enumerate((3, 3, 3, 3))]
    cp = (st.normal("c", (n,)) * 2).astype(np.float32)
    # extremes: saturated gates in every combination, huge cell state
    ext = np.array([-1e4, -100.0, -41.0, -40.0, 0.0, 40.0, 41.0, 100.0, 1e4], dtype=np.float32)
    gi, gf, gg, go = [v.ravel() for v in np.meshgrid(ext, ext, ext, ext)]
    pre = [np.concatenate([p, e]) for p, e in zip(pre, (gi, gf, gg, go))]
    cp = np.concatenate([cp, np.resize(np.array([-50.0, -1.0, 0.0, 1.0, 50.0], dtype=np.float32), gi.size)])
    c, h = O.cells(pre[0], pre[1], pre[2], pre[3], cp)
    assert np.isfinite(c).all() and np.isfinite(h).all()
    d = [p.astype(np.float64) for p in pre]
    sig = lambda v: 1 / (1 + np.exp(-np.clip(v, -700, 700)))
    c_ref = sig(d[1]) * cp.astype(np.float64) + sig(d[0]) * np.tanh(d[2])
    h_ref = sig(d[3]) * np.tanh(c_ref)
    # a handful of fp32 roundings on f and i*g, the first scaled by |c_prev|
    assert np.max(np.abs(c - c_ref) / np.maximum(1.0, np.abs(cp.astype(np.float64)))) < 4e-7
    assert np.max(np.abs(h - h_ref)) < 4e-7
    assert (np.abs(h) <= 1).all()
    # a cell whose forget gate is open and input gate shut keeps its state exactly
    c2, _ = O.cells(np.float32([-100.0]), np.float32([100.0]), np.float32([0.3]), np.float32([0.0]), np.float32([1.2345678]))
    assert c2[0] == np.float32(1.2345678)


def test_fp32_activation_functions_against_libm():
    # The gate non-linearities are fixed fp32 operation sequences (so that codes are
    # reproducible); here they are pinned to the real functions evaluated in double.
    x = np.concatenate([np.linspace(-30, 30, 400001), np.linspace(-1e-3, 1e-3, 2001),
                        np.array([-1e4, -90.0, 90.0, 1e4, 0.0])]).astype(np.float32)
    ex, sg, th = O.activations(x)
    xd = x.astype(np.float64)
    inr = np.abs(xd) <= 30
    assert np.max(np.abs(ex[inr] / np.exp2(xd[inr]) - 1)) < 2e-7
    # the power of two over its whole range, and exactly at the integers
    t = np.linspace(-125, 125, 500001).astype(np.float32)
    e2, _, _ = O.activations(t)
    assert np.max(np.abs(e2 / np.exp2(t.astype(np.float64)) - 1)) < 2e-7
    ti = np.arange(-125, 126).astype(np.float32)
    np.testing.assert_array_equal(O.activations(ti)[0], np.exp2(ti.astype(np.float64)).astype(np.float32))
    assert np.max(np.abs(sg - 1 / (1 + np.exp(-np.clip(xd, -700, 700))))) < 2e-7
    assert np.max(np.abs(th - np.tanh(xd))) < 2e-7
    assert (sg >= 0).all() and (sg <= 1).all() and (np.abs(th) <= 1).all()
    assert th[-1] == 0.0 and sg[-1] == 0.5 and ex[-1] == 1.0
    # monotone where it matters for quantization: no inversions on a fine grid
    g = np.linspace(-12, 12, 200001).astype(np.float32)
    _, sg, th = O.activations(g)
    assert (np.diff(sg) >= -1.2e-7).all() and (np.diff(th) >= -1.2e-7).all()
    # odd symmetry of tanh, and sigmoid(x) + sigmoid(-x) = 1 within rounding
    _, s1, t1 = O.activations(g)
    _, s2, t2 = O.activations(-g)
    np.testing.assert_array_equal(t1, -t2)
    assert np.max(np.abs(s1 + s2 - 1)) < 2e-7


# ------------------------------------------------------------------ plain (textbook) step
def _forced_fixed_vs_plain(layers, xq, x_act, hid, eps=1e-3):
    """Walks the fixed-sequence step along time (both directions) and, on the very same inputs
    (teacher forcing), evaluates the plain step: libm gates in double.  Returns counts."""
    T, B, K = xq.shape
    L = O.Lstm(layers)
    H = L.H
    n = near = moved_at_tie = outside = 0
    for d in range(L.n):
        hq = np.zeros((B, H), np.int16)
        c = np.zeros((B, H), np.float32)
        for s in range(T):
            t = s if d == 0 else T - 1 - s
            f = O.lstm_step(L, xq[t], x_act, hq, c, hid, d=d)
            p = O.lstm_step_plain(L, xq[t], x_act, hq, c, hid, d=d)
            np.testing.assert_allclose(f["c"], p["c"], rtol=1e-5, atol=1e-6)
            np.testing.assert_allclose(f["h"], p["h"], rtol=1e-5, atol=1e-6)
            tie = p["tie"] < eps
            diff = f["hq"].astype(np.int32) - p["hq"].astype(np.int32)
            assert np.abs(diff).max() <= 1
            n += diff.size
            near += int(tie.sum())
            moved_at_tie += int(((diff != 0) & tie).sum())
            outside += int(((diff != 0) & ~tie).sum())
            hq, c = f["hq"], f["c"]
    return n, near, moved_at_tie, outside


def test_fixed_sequence_step_against_plain_step_config0():
    # config 0: one layer, K=64, H=128, B=4, T=50, clip 3.0
    w = synth.single_layer(seed=0)
    x_act, hid = O.act_symmetric(w["x_clip"], 4), O.act_symmetric(1.0, 4)
    n, near, moved, outside = _forced_fixed_vs_plain(w["layers"], O.quantize(w["x"], x_act), x_act, hid)
    print(f"config 0: {n} codes, {near} within 1e-3 of a rounding boundary, {moved} of those differ by one, "
          f"{outside} differ elsewhere")
    assert outside == 0
    assert near < 0.01 * n


def test_fixed_sequence_step_against_plain_step_encoder_layer():
    # one bidirectional 640-cell layer with the encoder's inner-layer shape (K = 1280), 4 and 8 bit
    for bits in (4, 8):
        st = synth.Stream(41 + bits)
        layers = [synth._lstm(st, f"d{d}", 1280, 640, bits, 0.1, 0.95, bits) for d in range(2)]
        x_act, hid = O.act_symmetric(0.97, bits), O.act_symmetric(0.95, bits)
        lo, hi = x_act.lo() + 1, x_act.hi()
        xq = st.integers("xq", (6, 2, 1280), lo, hi).astype(np.int16)
        n, near, moved, outside = _forced_fixed_vs_plain(layers, xq, x_act, hid)
        print(f"{bits} bit: {n} codes, {near} near a boundary, {moved} of those differ, {outside} elsewhere")
        assert outside == 0


def test_plain_step_is_the_library_cell():
    # the plain step itself against torch's LSTMCell in float64 (gate order, transposes, Eq. 3)
    st = synth.Stream(5)
    K, H, N = 24, 16, 5
    lw = synth._lstm(st, "cell", K, H, 4, bias_std=0.3)
    rng = np.random.default_rng(1)
    x_act, hid = O.act_asymmetric(-2.5, 3.5, 4), O.act_symmetric(1.0, 4)
    xq = rng.integers(0, 16, (N, K)).astype(np.int16)
    hq = rng.integers(-7, 8, (N, H)).astype(np.int16)
    c = rng.normal(0, 1, (N, H)).astype(np.float32)
    p = O.lstm_step_plain(O.Lstm([lw]), xq, x_act, hq, c, hid)
    with torch.no_grad():
        h1, c1 = torch_cell(lw)(torch.from_numpy(O.dequantize(xq, x_act)).double(),
                                (torch.from_numpy(O.dequantize(hq, hid)).double(), torch.from_numpy(c).double()))
    # de-quantized operands are fp32 products s * q here and exact reals inside the plain step
    np.testing.assert_allclose(p["c"], c1.numpy(), rtol=2e-6, atol=2e-6)
    np.testing.assert_allclose(p["h"], h1.numpy(), rtol=2e-6, atol=2e-6)
    np.testing.assert_array_equal(p["hq"], O.quantize(p["h"], hid))
    t = p["h"].astype(np.float64) * hid.inv_scale
    np.testing.assert_allclose(p["tie"], np.abs(t - np.floor(t) - 0.5), atol=1e-5)
