"""The allocation-free joint entry point against the regular one.

qjoint_logprobs_static serves callers that cannot allocate device memory at call time (a
decoding thread that must not stall on the allocator, a host that fixes its memory budget
at start-up).  It must give what qjoint_logprobs gives, call after call, although all its
calls share one built-in scratch array that keeps the previous call's contents.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2206_07882_b200 import synth

pytestmark = pytest.mark.gpu

LP_ATOL = 1e-5      # the tolerance the other joint tests use for log-probabilities


def test_static_scratch_joint_matches_workspace_joint_twice():
    from paper_2206_07882_b200 import binding as Bd
    lib = Bd.lib()
    dw = synth.decoder(seed=5, V=1024, E=32, Hp=1024, D=256, Hs=32, Ht=32)
    dd = Bd.Decoder(dw, tensor_cores=False)
    st = synth.Stream(12)
    hid = dd.pred_lstm.hid_act
    R = 64
    e_host = st.normal("e", (R, 256)).astype(np.float32)
    e = torch.from_numpy(e_host).cuda()
    dec, o_hid = O.Decoder(dw), O.act_symmetric(dw.pred.lstm.hid_alpha, 4)
    for call, N in enumerate((200, 37)):          # second call is smaller: stale scratch behind it
        fi_host = st.integers(f"fi{call}", (N,), 0, R - 1).astype(np.int32)
        fi = torch.from_numpy(fi_host).cuda()
        codes = st.integers(f"pq{call}", (N, 1024), -7, 7).astype(np.float32)
        pq = Bd.quantize_pack_int4(torch.from_numpy(codes).cuda(), Bd.Act(1.0, 1.0, 0, 4, 1))
        want = Bd.qjoint_logprobs(e, fi, pq, hid, dd.pred_proj, dd.z_act, dd.joint_out)
        got = torch.full((N, 1024), float("nan"), dtype=torch.float32, device="cuda")
        before = torch.cuda.memory_allocated()
        Bd.qjoint_logprobs_static(e, fi, pq, hid, dd.pred_proj, dd.z_act, dd.joint_out, got)
        assert torch.cuda.memory_allocated() == before          # nothing was allocated through torch
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert (got - want).abs().max().item() <= LP_ATOL
        # and against the CPU oracle's joint network on the same inputs
        p_ref = O.linear(O.Linear(dw.pred.proj), codes.astype(np.int16), o_hid)
        assert np.abs(got.cpu().numpy() - O.joint(dec, e_host[fi_host], p_ref)).max() <= LP_ATOL
    # beyond the built-in limit: a clear error instead of an allocation (N * D > 65536)
    N = 300
    pq = torch.zeros((N, 512), dtype=torch.uint8, device="cuda")
    fi = torch.zeros(N, dtype=torch.int32, device="cuda")
    out = torch.zeros((N, 1024), dtype=torch.float32, device="cuda")
    with pytest.raises(Bd.Q4Error) as err:
        Bd.qjoint_logprobs_static(e, fi, pq, hid, dd.pred_proj, dd.z_act, dd.joint_out, out)
    assert err.value.code == -5
