"""GPU parity: quantize_pack_int4 and the feature prologue against the oracle (bit-exact:
the quantizer is defined in fp32 on both sides)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2206_07882_b200 import synth
from _parity import gpu_codes, to_act

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def Bd():
    from paper_2206_07882_b200 import binding
    binding.lib()
    return binding


CASES = [("sym4", lambda: O.act_symmetric(3.0, 4)), ("sym8", lambda: O.act_symmetric(2.7, 8)),
         ("asym4", lambda: O.act_asymmetric(-2.5, 3.5, 4)), ("pred", lambda: O.act_symmetric(1.25, 4))]


@pytest.mark.parametrize("name,mk", CASES)
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("rows,k", [(1, 32), (7, 45), (200, 240), (1000, 1280), (0, 64)])
def test_fixed_boundary(Bd, name, mk, dtype, rows, k):
    a = mk()
    x = synth.Stream(3).normal(f"x{rows}.{k}", (rows, k), 0.0, 1.5).astype(dtype)
    if rows:
        x[0, :min(k, 6)] = np.array([0.0, a.scale * 0.5, -a.scale * 1.5, 100.0, -100.0, a.scale * 2.5], dtype)[:min(k, 6)]
    got = Bd.quantize_pack_int4(torch.from_numpy(x).cuda(), to_act(a))
    k_pad = Bd.pad32(k)
    assert got.shape == (rows, k_pad * a.bits // 8)
    if rows == 0:
        return
    want = O.quantize(x.astype(np.float32), a)
    np.testing.assert_array_equal(gpu_codes(got, k, a), want)
    # padding holds the code of the real value 0
    if k_pad > k:
        full = gpu_codes(got, k_pad, a)
        assert (full[:, k:] == (0 if a.is_signed else a.zero_point)).all()
    # byte-identical to the oracle's storage format
    if a.bits == 4:
        np.testing.assert_array_equal(got.cpu().numpy(), O.pack4(want, k_pad, 0 if a.is_signed else a.zero_point))


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("T,B,F", [(6, 3, 40), (50, 8, 240)])
def test_max_boundary_per_utterance(Bd, bits, T, B, F):
    x = synth.Stream(4).normal("feat", (T, B, F)).astype(np.float16)
    x[:, 1, :] = 0                                     # an all-zero utterance: boundary 1
    base = Bd.q4_act_symmetric(1.0, bits)
    got, scales = Bd.quantize_pack_int4(torch.from_numpy(x).cuda().reshape(T * B, F), base, mode=1, n_groups=B)
    codes = gpu_codes(got, F, base).reshape(T, B, F)
    for b in range(B):
        a = O.act_symmetric(O.absmax(x[:, b, :].astype(np.float32)), bits)
        assert scales[b].item() == a.scale
        np.testing.assert_array_equal(codes[:, b, :], O.quantize(x[:, b, :].astype(np.float32), a))


@pytest.mark.parametrize("bits", [4, 8])
def test_weight_mode_per_row_scale(Bd, bits):
    st = synth.Stream(5)
    rows, k = 130, 200
    w = st.normal("w", (rows, k), 0.0, 0.1).astype(np.float32)
    s = st.uniform("s", (rows,), 0.01, 0.05).astype(np.float32)
    m = Bd.DeviceMat.from_float(w, s, bits)
    a = O.act_symmetric(1.0, bits)
    np.testing.assert_array_equal(gpu_codes(m.q, k, a), O.quantize_weights(w, s, bits))
    # integer codes handed over as floats come back exactly
    q = st.integers("q", (rows, k), -(1 << (bits - 1)), (1 << (bits - 1)) - 1).astype(np.int8)
    m2 = Bd.DeviceMat.from_codes(q, s, bits)
    np.testing.assert_array_equal(gpu_codes(m2.q, k, a), q)


@pytest.mark.parametrize("bits", [4, 8])
def test_weight_mode_max_boundary_per_row(Bd, bits):
    # real-valued weights -> codes with the MAX boundary (Section 3.1) of every output row: the
    # row's largest magnitude maps to the largest code, an all-zero row gets boundary 1
    from _parity import pack_codes
    st = synth.Stream(6)
    rows, k = 77, 150
    w = (st.normal("w", (rows, k), 0.0, 0.2) * st.uniform("g", (rows, 1), 0.1, 3.0)).astype(np.float32)
    w[5, :] = 0
    m = Bd.DeviceMat.from_float_max(w, bits)
    scales = m.scale.cpu().numpy()
    qmax = (1 << (bits - 1)) - 1
    got = gpu_codes(m.q, k, O.act_symmetric(1.0, bits))
    for r in range(rows):
        a = O.act_symmetric(O.absmax(w[r:r + 1]), bits)
        assert scales[r] == a.scale
        np.testing.assert_array_equal(got[r], O.quantize(w[r:r + 1], a)[0])
        if r != 5:
            assert np.abs(got[r]).max() == qmax          # the boundary itself reaches the last code
    # de-quantized weights lie within half a step of the originals (Section 3.1)
    deq = got.astype(np.float64) * scales[:, None]
    assert (np.abs(deq - w) <= 0.5 * scales[:, None] * (1 + 1e-6)).all()
    # the matrix serves a quantized linear layer as it stands
    xa = O.act_symmetric(1.0, bits)     # the linear entry point takes codes of the weights' width
    xq = O.quantize(st.normal("x", (9, k)).astype(np.float32), xa)
    lin = Bd.DeviceLinear.__new__(Bd.DeviceLinear)
    lin.w, lin.bias = m, None
    out = Bd.q4_linear_forward(pack_codes(xq, xa), to_act(xa), lin).cpu().numpy()
    want = (xq.astype(np.int64) @ got.astype(np.int64).T).astype(np.float64) * \
        (np.float64(xa.scale) * scales.astype(np.float64))[None, :]
    np.testing.assert_allclose(out, want, rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("B,T100,M", [(1, 4, 1), (3, 20, 40), (2, 1000, 40), (2, 7, 5)])
def test_feature_prologue(Bd, B, T100, M):
    mel = synth.logmel(9, B, T100, M)
    got = Bd.q4_feature_prologue(torch.from_numpy(mel).cuda()).cpu().numpy()
    assert got.shape == (T100 // 2, B, 6 * M) and got.dtype == np.float16
    for b in range(B):
        want = O.features(mel[b]).astype(np.float16)
        np.testing.assert_array_equal(got[:, b, :], want)


def test_weight_mode_two_bit_storage(Bd):
    # symmetric per-row quantization to 2-bit codes, four per byte: byte-identical to the oracle's packing
    st = synth.Stream(31)
    rows, k = 37, 200
    w = st.normal("w", (rows, k), 0, 1.0).astype(np.float32)
    sc = st.uniform("s", (rows,), 0.5, 1.5).astype(np.float32)
    dm = Bd.DeviceMat.from_float(w, sc, 2)
    assert dm.k_pad == 256 and dm.q.shape == (rows, 64)
    want = O.pack2(O.quantize_weights(w, sc, 2).astype(np.int16), 256)
    np.testing.assert_array_equal(dm.q.cpu().numpy(), want)
    # MAX boundary per row at 2 bits: the row's largest magnitude maps to code 1 (or -1 / -2 by sign)
    dm2 = Bd.DeviceMat.from_float_max(w, 2)
    amax = np.abs(w).max(1)
    np.testing.assert_array_equal(dm2.scale.cpu().numpy(), amax.astype(np.float32))
    want2 = O.pack2(O.quantize_weights(w, amax.astype(np.float32), 2).astype(np.int16), 256)
    np.testing.assert_array_equal(dm2.q.cpu().numpy(), want2)
