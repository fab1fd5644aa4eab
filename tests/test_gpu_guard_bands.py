"""Guard bands around every device buffer the binding allocates for the library.

Stand-in for a memory checker on the write side: every output, state and workspace buffer that
the Python binding allocates is carved out of a larger allocation whose 4 KB margins on both
sides hold a byte pattern; after the calls the margins must be untouched.  A kernel that stores
past the end of a tile, a ragged row, a padded workspace or a state array would leave its mark
there.  (Reads are not covered, and neither are the read-only weight and input tensors.)
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2206_07882_b200 import synth
from _parity import pack_codes, to_act

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


class GuardedTorch:
    """Forwards to torch, but empty/zeros/full and their _like forms on a CUDA device return the
    inside of a guarded allocation."""

    def __init__(self):
        self.blocks = []          # (flat allocation, payload bytes)

    def __getattr__(self, name):
        return getattr(torch, name)

    def _guarded(self, shape, dtype, device, fill):
        if isinstance(shape, int):
            shape = (shape,)
        shape = tuple(int(s) for s in shape)
        dtype = dtype or torch.float32
        n = int(np.prod(shape)) if len(shape) else 1
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        pad = (-nbytes) % 256
        flat = torch.full((GUARD + nbytes + pad + GUARD,), PATTERN, dtype=torch.uint8, device=device)
        inner = flat[GUARD:GUARD + nbytes]
        if fill is not None:
            inner.zero_()
        t = inner.view(dtype).reshape(shape)
        if fill not in (None, 0):
            t.fill_(fill)
        self.blocks.append((flat, nbytes))
        return t

    def _on_cuda(self, device):
        return device is not None and torch.device(device).type == "cuda"

    def empty(self, *shape, dtype=None, device=None, **kw):
        shape = shape[0] if len(shape) == 1 and not isinstance(shape[0], int) else shape
        if not self._on_cuda(device):
            return torch.empty(shape, dtype=dtype, device=device, **kw)
        return self._guarded(shape, dtype, device, None)

    def zeros(self, *shape, dtype=None, device=None, **kw):
        shape = shape[0] if len(shape) == 1 and not isinstance(shape[0], int) else shape
        if not self._on_cuda(device):
            return torch.zeros(shape, dtype=dtype, device=device, **kw)
        return self._guarded(shape, dtype, device, 0)

    def full(self, shape, value, dtype=None, device=None, **kw):
        if not self._on_cuda(device):
            return torch.full(shape, value, dtype=dtype, device=device, **kw)
        return self._guarded(shape, dtype, device, value)

    def empty_like(self, t, **kw):
        return self.empty(tuple(t.shape), dtype=t.dtype, device=t.device) if t.is_cuda else torch.empty_like(t, **kw)

    def zeros_like(self, t, **kw):
        return self.zeros(tuple(t.shape), dtype=t.dtype, device=t.device) if t.is_cuda else torch.zeros_like(t, **kw)

    def check(self):
        torch.cuda.synchronize()
        assert self.blocks, "nothing was allocated through the guarded allocator"
        for flat, nbytes in self.blocks:
            head = flat[:GUARD]
            tail = flat[GUARD + nbytes:]
            assert bool((head == PATTERN).all()), f"write before a buffer of {nbytes} bytes"
            assert bool((tail == PATTERN).all()), f"write behind a buffer of {nbytes} bytes"
        return len(self.blocks)


@pytest.fixture()
def guarded(monkeypatch):
    from paper_2206_07882_b200 import binding
    binding.lib()
    g = GuardedTorch()
    monkeypatch.setattr(binding, "torch", g)
    return binding, g


def test_the_allocator_catches_a_stray_write():
    g = GuardedTorch()
    t = g.empty((5, 7), dtype=torch.float32, device="cuda")
    assert t.shape == (5, 7) and t.data_ptr() % 256 == 0
    g.check()
    flat, nbytes = g.blocks[0]
    flat[GUARD + nbytes + 3] = 0          # one byte behind the payload, planted by the test on the host side
    with pytest.raises(AssertionError):
        g.check()


def test_quantize_steps_layers_and_linear_layers_stay_inside_their_buffers(guarded):
    Bd, g = guarded
    st = synth.Stream(901)
    # quantize + pack: ragged row lengths, both widths, per-group boundary
    for bits, K, rows in ((4, 37, 5), (8, 200, 33), (4, 1280, 130)):
        x = torch.from_numpy(st.normal(f"x{bits}{K}", (rows, K)).astype(np.float32)).cuda()
        Bd.quantize_pack_int4(x, Bd.q4_act_symmetric(2.0, bits))
        Bd.quantize_pack_int4(x, Bd.q4_act_symmetric(1.0, bits), mode=1, n_groups=1)
    # one step: DP4A kernel (ragged rows and widths), tensor-core kernel (prepared operands, ragged tile)
    for N, K, H, prep in ((70, 200, 96, False), (5, 32, 32, False), (130, 256, 128, True), (300, 96, 256, True)):
        lw = synth._lstm(st, f"l{N}", K, H, 4, bias_std=0.2, hid_alpha=0.95, hid_bits=4)
        x_act, hid = O.act_symmetric(3.0, 4), O.act_symmetric(0.95, 4)
        xq = st.integers(f"xq{N}", (N, K), x_act.lo(), x_act.hi()).astype(np.int16)
        hq = st.integers(f"hq{N}", (N, H), hid.lo() + 1, hid.hi()).astype(np.int16)
        c = torch.from_numpy(st.normal(f"c{N}", (N, H)).astype(np.float32)).cuda()
        dl = Bd.DeviceLstm(lw)
        if prep:
            dl.prepare()
        Bd.qlstm_step(pack_codes(xq, x_act, dl.w_ih.k_pad), to_act(x_act), pack_codes(hq, hid), c, dl, want_dbg=not prep)
    # whole layers: step-by-step kernels, the general persistent kernel, the register-resident kernels
    # (one group per cluster; clusters taking turns at 57 sequences x 2 directions; int8 weights)
    for T, B, K, H, dirs, bits in ((9, 3, 48, 32, 2, 4), (20, 70, 240, 64, 2, 8), (12, 33, 128, 96, 1, 4),
                                   (6, 20, 64, 640, 2, 4), (64, 57, 64, 640, 2, 4), (64, 57, 64, 640, 2, 8)):
        w = synth.single_layer(seed=T + B, T=T, B=B, K=K, H=H, bits=bits, dirs=dirs)
        for lw in w["layers"]:
            lw.hid_bits = bits
        x_act, out = O.act_symmetric(3.0, bits), O.act_symmetric(1.0, 4)
        xq = pack_codes(O.quantize(w["x"], x_act).reshape(T * B, K), x_act)
        layers = [Bd.DeviceLstm(lw) for lw in w["layers"]]
        r = Bd.qlstm_layer_forward(xq, to_act(x_act), T, B, layers, to_act(out), want_state=True)
        assert Bd.q4_poll_status(r["workspace"]) == 0
    # linear layers: DP4A and tensor-core path (ragged rows, ragged output width)
    for M, K, J, prep in ((7, 96, 50, False), (257, 1280, 256, True), (130, 128, 72, True)):
        lin = synth._linear(st, f"lin{M}", J, K, 4)
        act = O.act_symmetric(1.0, 4)
        xq = st.integers(f"lx{M}", (M, K), -7, 7).astype(np.int16)
        dlin = Bd.DeviceLinear(lin)
        if prep:
            dlin.prepare()
        Bd.q4_linear_forward(pack_codes(xq, act, dlin.w.k_pad), to_act(act), dlin)
    assert g.check() > 30


@pytest.mark.parametrize("tensor_cores", [True, False])
def test_the_search_stays_inside_its_state_and_workspace(guarded, tensor_cores):
    Bd, g = guarded
    # fused heads (V = 1024, D = 256) with 9 utterances x 16 slots = two ragged row tiles; odd sizes on the DP4A path
    for V, D, utts in ((1024, 256, 9), (200, 64, 3)):
        dw = synth.decoder(seed=77, V=V, E=32, Hp=128, D=D, Hs=128, Ht=128, tgt_layers=2, U_max=5, W=16)
        e = torch.from_numpy(synth.Stream(5).normal("e", (9, utts, D)).astype(np.float32)).cuda()
        dec = Bd.Decoder(dw, tensor_cores=tensor_cores)
        dec.decode(e)
        dec.decode_time_synchronous(e, 2)
    # one utterance: the weight-streaming step kernel
    dw = synth.decoder(seed=78, V=1024, E=32, Hp=256, D=256, Hs=256, Ht=256, tgt_layers=2, U_max=5, W=16)
    e = torch.from_numpy(synth.Stream(6).normal("e", (9, 1, 256)).astype(np.float32)).cuda()
    Bd.Decoder(dw, tensor_cores=tensor_cores).decode(e)
    assert g.check() > 20


def test_the_encoder_stays_inside_its_buffers(guarded):
    Bd, g = guarded
    w = synth.encoder(seed=2, T=30, B=5, F=80, H=32, L=3, D=32, first_layer_bits=8, in_max=True)
    Bd.Encoder(w["enc"]).forward(torch.from_numpy(w["features"]).cuda())
    Bd.q4_feature_prologue(torch.from_numpy(synth.logmel(13, 3, 50, 40)).cuda())
    assert g.check() > 5
