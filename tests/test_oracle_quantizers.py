"""Pins for the oracle's quantizers, packing and integer MACs (CPU only).

Each check compares the oracle with something the paper or the mathematics
fixes: Eq. 2 / Eq. 3 evaluated by hand on a grid with a power-of-two scale, the
s/2 residual bound of Section 3.1, the end points alpha- -> 0 and alpha+ ->
2^b-1, the round trip Q(Dq(q)) == q, 64-bit brute force for the MACs.
"""
import os

import numpy as np
import pytest

from oracle import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def gold():
    d = {}
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            d[k.strip()] = float(v)
    return d


def test_symmetric_hand_table_half_to_even():
    # alpha = 3.5, b = 4 -> s = 0.5 exactly, so x/s is exact and ties are real ties.
    a = O.act_symmetric(3.5, 4)
    assert a.scale == 0.5 and a.inv_scale == 2.0 and a.zero_point == 0
    x = np.array([0.0, 0.25, 0.75, 1.25, 1.75, -0.25, -0.75, -1.25, 0.26, 0.74, 3.5, 3.74, 3.76,
                  100.0, -3.5, -3.75, -4.0, -4.3, -100.0], dtype=np.float32)
    want = np.array([0, 0, 2, 2, 4, 0, -2, -2, 1, 1, 7, 7, 7, 7, -7, -8, -8, -8, -8])
    np.testing.assert_array_equal(O.quantize(x, a), want)


def test_symmetric_clip3_bits4_codes():
    # s = 3/7; thresholds between codes sit at (n + 1/2) * 3/7.
    a = O.act_symmetric(3.0, 4)
    assert abs(a.scale - 3.0 / 7.0) < 1e-7
    x = np.array([0.0, 0.2142, 0.2144, 3.0, -3.0, 10.0, -10.0, 0.6428, 0.6430, -3.3, -3.22],
                 dtype=np.float32)
    want = np.array([0, 0, 1, 7, -7, 7, -8, 1, 2, -8, -8])
    np.testing.assert_array_equal(O.quantize(x, a), want)


def test_asymmetric_endpoints_and_zero_point():
    # Eq. 2: x = alpha- maps to 0 and x = alpha+ to 2^b - 1.
    for lo, hi, bits in [(-2.5, 3.5, 4), (-1.0, 2.0, 4), (-1.3, 1.9, 8), (0.0, 6.0, 4)]:
        a = O.act_asymmetric(lo, hi, bits)
        qmax = (1 << bits) - 1
        assert abs(a.scale - (hi - lo) / qmax) < 1e-6
        assert a.zero_point == int(np.rint(-lo / a.scale))
        q = O.quantize(np.array([lo, hi, lo - 5, hi + 5, 0.0], dtype=np.float32), a)
        assert list(q[:4]) == [0, qmax, 0, qmax]
        assert q[4] == a.zero_point           # zero is representable exactly ...
        assert O.dequantize(q[4:5], a)[0] == 0.0


def test_asymmetric_hand_table():
    # lo = -2, hi = 5.5, b = 4 -> s = 0.5, z = 4.
    a = O.act_asymmetric(-2.0, 5.5, 4)
    assert a.scale == 0.5 and a.zero_point == 4
    x = np.array([-2.0, -1.75, -1.25, 0.0, 0.25, 0.75, 5.5, 9.0, -9.0], dtype=np.float32)
    want = np.array([0, 0, 2, 4, 4, 6, 15, 15, 0])   # ties to even BEFORE adding z
    np.testing.assert_array_equal(O.quantize(x, a), want)
    np.testing.assert_array_equal(O.dequantize(want, a),
                                  0.5 * (want - 4).astype(np.float32))   # Eq. 3


@pytest.mark.parametrize("bits", [4, 8])
def test_roundtrip_all_codes(bits):
    rng = np.random.default_rng(0)
    for _ in range(50):
        a = O.act_symmetric(float(rng.uniform(0.1, 5.0)), bits)
        q = np.arange(a.lo(), a.hi() + 1, dtype=np.int16)
        np.testing.assert_array_equal(O.quantize(O.dequantize(q, a), a), q)
        lo = -float(rng.uniform(0.1, 3.0))
        a = O.act_asymmetric(lo, float(rng.uniform(0.1, 3.0)), bits)
        q = np.arange(0, (1 << bits), dtype=np.int16)
        np.testing.assert_array_equal(O.quantize(O.dequantize(q, a), a), q)


@pytest.mark.parametrize("bits", [4, 8])
def test_residual_bound_in_range(bits):
    # Section 3.1: inside [alpha-, alpha+] the residual |x - x_q| is at most s/2.
    g = gold()
    rng = np.random.default_rng(1)
    a = O.act_symmetric(1.0, bits)
    x = rng.uniform(-1.0, 1.0, 20000).astype(np.float32)
    r = np.abs(O.dequantize(O.quantize(x, a), a).astype(np.float64) - x)
    assert r.max() <= g["residual_bound_in_s"] * a.scale * (1 + 1e-5)
    assert r.max() > 0.45 * a.scale             # and the bound is approached
    a = O.act_asymmetric(-1.5, 2.0, bits)
    # the grid is anchored at z, an integer: in-range means within the grid's span
    glo, ghi = a.scale * (0 - a.zero_point), a.scale * ((1 << bits) - 1 - a.zero_point)
    x = rng.uniform(glo, ghi, 20000).astype(np.float32)
    r = np.abs(O.dequantize(O.quantize(x, a), a).astype(np.float64) - x)
    assert r.max() <= 0.5 * a.scale * (1 + 1e-5)


def test_absmax_and_zero_tensor():
    assert O.absmax(np.array([0.5, -3.25, 2.0], dtype=np.float32)) == 3.25
    assert O.absmax(np.zeros(7, dtype=np.float32)) == 1.0


def test_weight_quantizer_recovers_integer_codes():
    rng = np.random.default_rng(2)
    for bits in (4, 8):
        lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
        q = rng.integers(lo, hi + 1, (33, 70)).astype(np.int8)
        s = rng.uniform(0.01, 0.05, 33).astype(np.float32)
        w = (q.astype(np.float32) * s[:, None]).astype(np.float32)
        np.testing.assert_array_equal(O.quantize_weights(w, s, bits), q)


def test_pack4_nibble_order_by_hand():
    # element 2i in bits 0-3, element 2i+1 in bits 4-7, two's complement.
    q = np.array([[1, -1, 7, -8, 3]], dtype=np.int16)
    b = O.pack4(q, 8)
    assert b.tolist() == [[0xF1, 0x87, 0x03, 0x00]]
    u = np.array([[15, 0, 9]], dtype=np.int16)
    assert O.pack4(u, 4, pad_code=5).tolist() == [[0x0F, 0x59]]


def test_pack_unpack_roundtrip():
    rng = np.random.default_rng(3)
    q = rng.integers(-8, 8, (17, 45)).astype(np.int16)
    np.testing.assert_array_equal(O.unpack4(O.pack4(q, 64), 45, True), q)
    u = rng.integers(0, 16, (5, 31)).astype(np.int16)
    np.testing.assert_array_equal(O.unpack4(O.pack4(u, 32, 3), 31, False), u)


def test_int_matmul_brute_force_and_zero_point():
    rng = np.random.default_rng(4)
    w = rng.integers(-8, 8, (37, 129)).astype(np.int8)
    x = rng.integers(-8, 8, (9, 129)).astype(np.int16)
    want = x.astype(np.int64) @ w.astype(np.int64).T          # library matmul, 64-bit
    np.testing.assert_array_equal(O.int_matmul(w, x), want)
    # transposition check: a one-hot input picks out a weight column
    e = np.zeros((1, 129), dtype=np.int16)
    e[0, 5] = 1
    np.testing.assert_array_equal(O.int_matmul(w, e)[0], w[:, 5])
    # unsigned codes with zero point z equal signed codes pre-shifted by z
    u = rng.integers(0, 16, (9, 129)).astype(np.int16)
    np.testing.assert_array_equal(O.int_matmul(w, u, 6), O.int_matmul(w, u - 6, 0))
    # extreme magnitudes stay exact in int32 (8*8*K, 128*128*K)
    K = 4096
    w8 = np.full((1, K), -128, dtype=np.int8)
    x8 = np.full((1, K), -128, dtype=np.int16)
    assert O.int_matmul(w8, x8)[0, 0] == 128 * 128 * K


def test_linear_matches_dequantized_float_matmul():
    rng = np.random.default_rng(5)
    from paper_2206_07882_b200 import synth
    lw = synth._linear(synth.Stream(11), "t", 24, 40)
    L = O.Linear(lw)
    a = O.act_asymmetric(-1.5, 1.2, 4)
    xq = rng.integers(0, 16, (6, 40)).astype(np.int16)
    out, acc = O.linear(L, xq, a, want_acc=True)
    wd = lw.w.codes.astype(np.float64) * lw.w.scale.astype(np.float64)[:, None]
    xd = O.dequantize(xq, a).astype(np.float64)                # Eq. 3
    want = xd @ wd.T + lw.bias
    np.testing.assert_allclose(out, want, rtol=1e-5, atol=1e-6)
    np.testing.assert_array_equal(acc, (xq.astype(np.int64) - a.zero_point) @ lw.w.codes.astype(np.int64).T)


def test_log_softmax_properties_and_library():
    import torch
    rng = np.random.default_rng(6)
    z = rng.normal(0, 3, (7, 100)).astype(np.float32)
    lp = O.log_softmax(z)
    np.testing.assert_allclose(np.exp(lp.astype(np.float64)).sum(1), 1.0, atol=1e-6)
    np.testing.assert_allclose(O.log_softmax(z + 11.0), lp, atol=2e-6)   # shift invariance
    want = torch.log_softmax(torch.from_numpy(z).double(), dim=1).numpy()
    np.testing.assert_allclose(lp, want, rtol=0, atol=1e-6)
    big = np.array([[1000.0, 999.0, -1000.0]], dtype=np.float32)        # no overflow
    assert np.isfinite(O.log_softmax(big)).all()


def test_size_accounting_matches_paper():
    # Section 3.2: 94.9 % of parameters at 4 bits, the rest at 8 -> 7.6x vs fp32.
    g = gold()
    f4 = g["frac_params_4bit"]
    ratio = 32.0 / (f4 * 4 + (1 - f4) * 8)
    assert abs(ratio - g["compression_full"]) < 0.05
    assert abs(g["size_fp32_mb"] / g["size_int4_mb"] - g["compression_full"]) < 0.05
    # packed bytes of a matrix = rows * k_pad * bits / 8 in the oracle's storage format
    q = np.zeros((10, 64), dtype=np.int16)
    assert O.pack4(q, 64).nbytes == 10 * 64 * 4 // 8


def test_two_bit_weight_storage_by_hand_and_round_trip():
    # four codes per byte, element 4i+j in bits 2j, 2j+1, two's complement: -2..1 -> 10, 11, 00, 01
    q = np.array([[1, -1, 0, -2, -2, 1, 1, 0, 0, 0, -1]], dtype=np.int16)
    b = O.pack2(q, 12)
    #   byte 0: 1 | (-1&3)<<2 | 0<<4 | (-2&3)<<6 = 1 + 12 + 0 + 128 = 141
    #   byte 1: (-2&3) | 1<<2 | 1<<4 | 0<<6 = 2 + 4 + 16 = 22
    #   byte 2: 0 | 0 | (-1&3)<<4 | padding 0 = 48
    assert b.tolist() == [[141, 22, 48]]
    np.testing.assert_array_equal(O.unpack2(b, 11), q)
    rng = np.random.default_rng(3)
    q = rng.integers(-2, 2, (7, 130)).astype(np.int16)
    np.testing.assert_array_equal(O.unpack2(O.pack2(q, 192), 130), q)
    # the symmetric weight quantizer at 2 bits: step = boundary, codes clamp to -2..1
    w = np.array([[0.0, 0.49, 0.51, 1.0, 1.6, -0.6, -1.4, -1.6, -9.0]], dtype=np.float32)
    codes = O.quantize_weights(w, np.array([1.0], np.float32), 2)
    assert codes.tolist() == [[0, 0, 1, 1, 1, -1, -1, -2, -2]]
