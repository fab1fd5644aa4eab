"""Host-side checks of the CUDA library that need no GPU: it loads, exports every symbol
the header declares, computes quantizer constants identically to the oracle, sizes its
workspaces, and turns bad arguments into error codes before touching the device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def Bd():
    from paper_2206_07882_b200 import build
    build.build()
    from paper_2206_07882_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(Bd):
    hdr = open(os.path.join(ROOT, "include", "q4rnnt.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"^(?:int|size_t|int64_t)\s+(\w+)\s*\(", hdr, flags=re.M))
    assert {"quantize_pack_int4", "qlstm_layer_forward", "qlstm_step", "qjoint_logprobs",
            "dr_fusion_beam_step"} <= names
    lib = Bd.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(Bd.EXPORTS)
    assert lib.q4_version() >= 1


def test_struct_layouts_match_header_sizes(Bd):
    assert C.sizeof(Bd.Act) == 20 and C.sizeof(Bd.Mat) == 32
    assert C.sizeof(Bd.LstmS) == 2 * 32 + 8 + 20 + 4          # two mats, pointer, act, padding
    assert C.sizeof(Bd.BeamStateS) == 47 * 8   # 38 pointers, two int32, 8 pointers of the candidate set


def test_quantizer_constants_equal_oracle(Bd):
    rng = np.random.default_rng(0)
    for bits in (4, 8):
        for alpha in [1.0, 1.25, 3.0, 0.9371] + list(rng.uniform(0.05, 9, 20)):
            a, b = Bd.q4_act_symmetric(float(alpha), bits), O.act_symmetric(float(alpha), bits)
            assert (a.scale, a.inv_scale, a.zero_point, a.bits, a.is_signed) == \
                   (b.scale, b.inv_scale, b.zero_point, b.bits, b.is_signed)
    for _ in range(30):
        lo, hi = -float(rng.uniform(0.1, 3)), float(rng.uniform(0.1, 3))
        a, b = Bd.q4_act_asymmetric(lo, hi, 4), O.act_asymmetric(lo, hi, 4)
        assert (a.scale, a.inv_scale, a.zero_point, a.bits, a.is_signed) == \
               (b.scale, b.inv_scale, b.zero_point, b.bits, b.is_signed)


def test_argument_errors_are_reported_on_the_host(Bd):
    lib = Bd.lib()
    a = Bd.Act()
    assert lib.q4_act_symmetric(C.c_float(1.0), C.c_int32(5), C.byref(a)) == -4
    assert lib.q4_act_symmetric(C.c_float(-1.0), C.c_int32(4), C.byref(a)) == -2
    assert lib.q4_act_symmetric(C.c_float(1.0), C.c_int32(4), None) == -1
    assert lib.q4_act_asymmetric(C.c_float(1.0), C.c_float(0.5), C.c_int32(4), C.byref(a)) == -2
    ok = Bd.q4_act_symmetric(1.0, 4)
    # NULL tensors
    assert lib.quantize_pack_int4(None, 0, C.c_int64(4), 32, 32, C.byref(ok), 0, 1, None, None, None, None) == -1
    fake = C.c_void_p(4096)           # aligned, never dereferenced: checks fail first
    assert lib.quantize_pack_int4(fake, 0, C.c_int64(4), 33, 48, C.byref(ok), 0, 1, None, fake, None, None) == -3
    assert lib.quantize_pack_int4(fake, 0, C.c_int64(4), 40, 32, C.byref(ok), 0, 1, None, fake, None, None) == -2
    assert lib.quantize_pack_int4(fake, 0, C.c_int64(4), 32, 32, C.byref(ok), 7, 1, None, fake, None, None) == -6
    assert lib.quantize_pack_int4(fake, 0, C.c_int64(4), 32, 32, C.byref(ok), 2, 1, None, fake, None, None) == -1
    bad_bits = Bd.Act(1.0, 1.0, 0, 3, 1)
    assert lib.quantize_pack_int4(fake, 0, C.c_int64(4), 32, 32, C.byref(bad_bits), 0, 1, None, fake, None, None) == -4
    # LSTM: unsupported weight width, misaligned k_pad (2-bit rows need multiples of 64), aliasing
    w_ih = Bd.Mat(4096, 4096, 128, 64, 64, 4)
    w_hh = Bd.Mat(4096, 4096, 128, 32, 32, 4)
    args = lambda x_act, wi=w_ih, wh=w_hh, hin=fake, hout=C.c_void_p(8192): lib.qlstm_step(
        fake, C.byref(x_act), None, hin, fake, 4, C.byref(wi), C.byref(wh), None, C.byref(ok), hout,
        fake, None, None, None, None, None, C.c_size_t(0), None)
    assert args(ok, wi=Bd.Mat(4096, 4096, 128, 64, 64, 3)) == -4
    assert args(ok, wi=Bd.Mat(4096, 4096, 128, 32, 32, 2)) == -3
    assert args(ok, wi=Bd.Mat(4096, 4096, 128, 60, 60, 4)) == -3
    assert args(ok, wh=Bd.Mat(4096, 4096, 128, 64, 64, 4)) == -2
    assert args(ok, hout=fake) == -6
    assert args(ok, hin=C.c_void_p(4100)) == -3
    # layer: workspace too small
    wih = (Bd.Mat * 1)(w_ih)
    whh = (Bd.Mat * 1)(w_hh)
    r = lib.qlstm_layer_forward(fake, C.byref(ok), None, 5, 2, 1, wih, whh, None, C.byref(ok), None,
                                fake, None, None, None, None, fake, C.c_size_t(16), None)
    assert r == -5
    r = lib.qlstm_layer_forward(fake, C.byref(ok), None, 5, 2, 3, wih, whh, None, C.byref(ok), None,
                                fake, None, None, None, None, fake, C.c_size_t(1 << 30), None)
    assert r == -2


def test_workspace_sizes(Bd):
    T, B, dirs, H = 50, 4, 2, 128
    n = Bd.workspace_bytes(Bd.WS_LSTM_LAYER, [T, B, dirs, H])
    assert n >= dirs * T * B * 4 * H * 4 + dirs * 2 * B * H + dirs * B * H * 4
    assert n % 256 == 0
    assert Bd.workspace_bytes(Bd.WS_JOINT, [256, 256]) >= 256 * 256 * 5
    assert Bd.workspace_bytes(Bd.WS_BEAM, [16, 16, 1024, 256]) >= 256 * 1024 * 4
    assert Bd.workspace_bytes(99, [1, 2, 3, 4]) == 0


def test_no_cpu_fallback(Bd):
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    x = torch.zeros((2, 32))
    with pytest.raises((RuntimeError, AssertionError)):
        Bd.quantize_pack_int4(x, Bd.q4_act_symmetric(1.0, 4))


def test_encoder_recurrence_plan_lays_groups_on_clusters():
    # host logic of qlstm_layer_forward's recurrence: which kernel, how many clusters, whose turn when
    from paper_2206_07882_b200 import binding as Bd
    plan = Bd.encoder_recurrence_plan
    p = plan(500, 32, 2, 640)                      # 4 groups x 2 directions: one group per cluster
    cap = p["max_clusters"]
    assert cap >= 8 and p["kernel"] == 1 and p["groups_per_cluster"] == 1 and p["clusters"] == [4, 4]
    for T, B in ((500, 64), (64, 57), (152, 60)):   # 8 groups x 2 directions
        p = plan(T, B, 2, 640)
        lack = 16 - cap
        if 1 <= lack <= 2:                          # one group more than clusters in `lack` directions: turns
            assert p["kernel"] == 2 and p["groups"] == 8
            assert p["turns"] == [1, 1 if lack == 2 else 0]
            assert sum(p["clusters"]) == cap and p["clusters"][0] == 7
            w = p["windows"][:8]
            assert w[0] == 0 and w[-1] == T and all(b > a for a, b in zip(w, w[1:]))      # a partition of the steps
            assert max(b - a for a, b in zip(w, w[1:])) - min(b - a for a, b in zip(w, w[1:])) <= 1
    p = plan(20, 64, 2, 640)                        # too few steps for turns: several groups per cluster
    assert p["kernel"] == 1 and p["groups_per_cluster"] * sum(p["clusters"]) >= 16 and sum(p["clusters"]) <= cap
    p = plan(500, 128, 2, 640)                      # 16 groups per direction
    assert p["kernel"] == 1 and sum(p["clusters"]) <= cap and p["groups_per_cluster"] * p["clusters"][0] >= 16
    # 8-bit weights or codes, or an input scale per sequence: the kernel with int8 fragments / per-sequence
    # scales while one group per cluster fits, the general kernel beyond
    assert plan(500, 32, 2, 640, w_bits=8, hid_bits=8)["kernel"] == 2
    assert plan(500, 32, 2, 640, per_sequence_scale=True)["kernel"] == 2
    assert plan(500, 64, 2, 640, w_bits=8, hid_bits=8)["kernel"] == (2 if 1 <= 16 - cap <= 2 else 0)
    assert plan(500, 128, 2, 640, w_bits=8, hid_bits=8)["kernel"] == 0
    assert plan(500, 32, 2, 320)["kernel"] == 0     # other widths: general kernel
    import ctypes as C
    assert Bd.lib().q4_encoder_recurrence_plan(C.c_int32(0), C.c_int32(4), C.c_int32(2), C.c_int32(640), C.c_int32(4),
                                               C.c_int32(4), C.c_int32(0), (C.c_int32 * 17)()) == -2
    assert Bd.lib().q4_encoder_recurrence_plan(C.c_int32(5), C.c_int32(4), C.c_int32(2), C.c_int32(640), C.c_int32(4),
                                               C.c_int32(4), C.c_int32(0), None) == -1
