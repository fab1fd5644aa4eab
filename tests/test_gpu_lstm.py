"""GPU parity: qlstm_step (teacher-forced, every step fed the oracle's state) and
qlstm_layer_forward / the encoder (free-running) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2206_07882_b200 import synth
from _parity import assert_close, assert_codes_match, gpu_codes, near_tie, pack_codes, to_act

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def Bd():
    from paper_2206_07882_b200 import binding
    binding.lib()
    return binding


def step_case(Bd, lw, x_act, hid, xq, hq, c, prepare=False):
    L = O.Lstm([lw])
    want = O.lstm_step(L, xq, x_act, hq, c, hid)
    dl = Bd.DeviceLstm(lw)
    if prepare:
        dl.prepare()
    assert dl.hid_act.scale == hid.scale
    got = Bd.qlstm_step(pack_codes(xq, x_act, dl.w_ih.k_pad), to_act(x_act), pack_codes(hq, hid),
                        torch.from_numpy(c).cuda(), dl, want_dbg=True)
    H = c.shape[1]
    np.testing.assert_array_equal(got["acc_ih"].cpu().numpy(), want["acc_ih"])     # bit-exact
    np.testing.assert_array_equal(got["acc_hh"].cpu().numpy(), want["acc_hh"])
    # the float stages are a fixed fp32 operation sequence on both sides: bit-exact
    np.testing.assert_array_equal(got["c"].cpu().numpy(), want["c"])
    np.testing.assert_array_equal(got["h"].cpu().numpy(), want["h"])
    np.testing.assert_array_equal(gpu_codes(got["hq"], H, hid), want["hq"])
    return 0


def test_config0_teacher_forced_every_step(Bd):
    # Single unidirectional INT4 layer: K=64, H=128, B=4, T=50, clip 3.0, seed 0.
    w = synth.single_layer(seed=0)
    lw = w["layers"][0]
    x_act, hid = O.act_symmetric(w["x_clip"], 4), O.act_symmetric(1.0, 4)
    xq = O.quantize(w["x"], x_act)
    ref = O.lstm_layer(O.Lstm([lw]), xq, x_act, hid, want=("h", "hq_hid", "c_n"))
    hq = np.zeros((4, 128), np.int16)
    c = np.zeros((4, 128), np.float32)
    ties = 0
    L = O.Lstm([lw])
    for t in range(50):
        ties += step_case(Bd, lw, x_act, hid, xq[t], hq, c)
        s = O.lstm_step(L, xq[t], x_act, hq, c, hid)          # oracle state feeds the next step
        hq, c = s["hq"], s["c"]
    np.testing.assert_array_equal(hq, ref["yq"][49])
    assert ties == 0


@pytest.mark.parametrize("N,K,H,xb,hb,signed", [(70, 200, 96, 4, 4, True), (5, 32, 32, 4, 4, False),
                                                 (130, 240, 64, 8, 8, True), (33, 256, 160, 4, 4, False),
                                                 (64, 64, 32, 8, 4, True), (1, 1280, 640, 4, 4, True)])
def test_step_shapes_and_formats(Bd, N, K, H, xb, hb, signed):
    st = synth.Stream(100 + N)
    lw = synth._lstm(st, "l", K, H, 4, bias_std=0.2, hid_alpha=0.95, hid_bits=hb)
    if xb == 8:
        lw.w_ih = synth._qmat(st, "w8", 4 * H, K, 8)
    if hb == 8:
        lw.w_hh = synth._qmat(st, "h8", 4 * H, H, 8)
    x_act = O.act_symmetric(3.0, xb) if signed else O.act_asymmetric(-1.7, 1.4, 4)
    hid = O.act_symmetric(0.95, hb)
    lo, hi = x_act.lo(), x_act.hi()
    xq = st.integers("xq", (N, K), lo, hi).astype(np.int16)
    hq = st.integers("hq", (N, H), -(1 << (hb - 1)) + 1, (1 << (hb - 1)) - 1).astype(np.int16)
    c = st.normal("c", (N, H)).astype(np.float32)
    step_case(Bd, lw, x_act, hid, xq, hq, c)


def test_step_embedding_lookup(Bd):
    st = synth.Stream(7)
    V, E, H, N = 50, 32, 64, 20
    lw = synth._lstm(st, "l", E, H, 4, bias_std=0.1)
    emb = st.normal("emb", (V, E), 0, 0.5).astype(np.float32)
    a = O.act_asymmetric(-1.2, 1.6, 4)
    table = Bd.quantize_pack_int4(torch.from_numpy(emb).cuda(), to_act(a))
    tok = st.integers("tok", (N,), 0, V - 1).astype(np.int32)
    hid = O.act_symmetric(1.0, 4)
    hq = st.integers("hq", (N, H), -7, 7).astype(np.int16)
    c = st.normal("c", (N, H)).astype(np.float32)
    got = Bd.qlstm_step(table, to_act(a), pack_codes(hq, hid), torch.from_numpy(c).cuda(),
                        Bd.DeviceLstm(lw), x_row_idx=torch.from_numpy(tok).cuda(), want_dbg=True)
    want = O.lstm_step(O.Lstm([lw]), O.quantize(emb[tok], a), a, hq, c, hid)
    np.testing.assert_array_equal(got["acc_ih"].cpu().numpy(), want["acc_ih"])
    np.testing.assert_array_equal(gpu_codes(got["hq"], H, hid), want["hq"])


def layer_case(Bd, T, B, K, H, dirs, xb=4, hb=4, ob=None, seed=0, x_clip=3.0, max_off=1e-4):
    w = synth.single_layer(seed=seed, T=T, B=B, K=K, H=H, bits=4, dirs=dirs)
    st = synth.Stream(seed + 77)
    for d, lw in enumerate(w["layers"]):
        lw.bias[:] = st.normal(f"b{d}", (4 * H,), 0, 0.1)
        if xb == 8:
            lw.w_ih = synth._qmat(st, f"w8{d}", 4 * H, K, 8)
        if hb == 8:
            lw.w_hh = synth._qmat(st, f"h8{d}", 4 * H, H, 8)
        lw.hid_bits = hb
    ob = ob or hb
    x_act, hid, out = O.act_symmetric(x_clip, xb), O.act_symmetric(1.0, hb), O.act_symmetric(1.0, ob)
    xq = O.quantize(w["x"], x_act)
    ref = O.lstm_layer(O.Lstm(w["layers"]), xq, x_act, hid, out, want=("h", "hq_hid", "c_n", "acc_ih", "acc_hh"))
    layers = [Bd.DeviceLstm(lw) for lw in w["layers"]]
    got = Bd.qlstm_layer_forward(pack_codes(xq.reshape(T * B, K), x_act), to_act(x_act), T, B, layers,
                                 to_act(out), want_state=True, want_dbg=True)
    assert Bd.q4_poll_status(got["workspace"]) == 0          # no bounded wait expired
    # input accumulators depend on the input only: bit-exact over the whole sequence
    np.testing.assert_array_equal(got["acc_ih"].cpu().numpy(), ref["acc_ih"])
    if T * B >= 128:                                         # tensor-core and DP4A projections agree
        alt = Bd.qlstm_layer_forward(pack_codes(xq.reshape(T * B, K), x_act), to_act(x_act), T, B, layers,
                                     to_act(out), want_dbg=True, tensor_cores=False)
        assert torch.equal(alt["acc_ih"], got["acc_ih"]) and torch.equal(alt["yq"], got["yq"])
    # the same call without the accumulator dumps (at 640 cells and 4 bits this takes the kernel that
    # keeps the recurrent weights in registers)
    lean = Bd.qlstm_layer_forward(pack_codes(xq.reshape(T * B, K), x_act), to_act(x_act), T, B, layers,
                                  to_act(out), want_state=True)
    assert Bd.q4_poll_status(lean["workspace"]) == 0
    for k in ("yq", "hq_n", "c_n"):
        assert torch.equal(lean[k], got[k]), k
    yq = gpu_codes(got["yq"], dirs * H, out).reshape(T, B, dirs * H)
    # free-running over the whole sequence and still bit-exact: codes, accumulators, states
    np.testing.assert_array_equal(yq, ref["yq"])
    np.testing.assert_array_equal(got["acc_hh"].cpu().numpy(), ref["acc_hh"])
    np.testing.assert_array_equal(got["c_n"].cpu().numpy(), ref["c_n"])
    hqn = gpu_codes(got["hq_n"].reshape(dirs * B, -1), H, hid).reshape(dirs, B, H)
    last = np.stack([ref["hq_hid"][T - 1, :, :H]] + ([ref["hq_hid"][0, :, H:]] if dirs == 2 else []))
    np.testing.assert_array_equal(hqn, last)
    return np.abs(yq.astype(np.int32) - ref["yq"])


def test_config0_layer_forward(Bd):
    diff = layer_case(Bd, T=50, B=4, K=64, H=128, dirs=1, seed=0)
    assert (diff > 0).sum() == 0


@pytest.mark.parametrize("T,B,K,H,dirs,xb,hb,ob", [(9, 3, 48, 32, 2, 4, 4, 4), (20, 70, 240, 64, 2, 8, 8, 4),
                                                   (12, 33, 128, 96, 1, 4, 4, 8), (7, 1, 1280, 160, 2, 4, 4, 4),
                                                   # 64 and 60 sequences x 2 directions of 640 cells: groups of 16
                                                   # sequences per cluster, full and ragged
                                                   (6, 64, 64, 640, 2, 4, 4, 4), (5, 60, 32, 640, 2, 8, 8, 4),
                                                   # 8-bit layers of 640 cells, one group of 8 per cluster: int8
                                                   # weights split between registers and shared memory
                                                   (9, 20, 32, 640, 2, 8, 8, 4), (7, 30, 32, 640, 1, 8, 8, 8),
                                                   # 7620 rows x 1280 gate rows: 298 tiles of the input projection with a
                                                   # ragged last row tile, more than two per SM (the persistent GEMM)
                                                   (60, 127, 32, 320, 1, 4, 4, 4)])
def test_layer_shapes_directions_precisions(Bd, T, B, K, H, dirs, xb, hb, ob):
    layer_case(Bd, T, B, K, H, dirs, xb, hb, ob, seed=11)


def test_layer_clusters_taking_turns_at_a_surplus_group(Bd):
    # 57 sequences x 2 directions of 640 cells = 16 groups of 8 for the 15 clusters that fit: the seven
    # clusters of one direction take turns at its eighth group (9 of 64 steps each, one more on the
    # last; the group holds one live sequence), the other direction runs one group per cluster
    diff = layer_case(Bd, T=64, B=57, K=64, H=640, dirs=2, seed=23)
    assert (diff > 0).sum() == 0


def test_layer_clusters_taking_turns_eight_bit(Bd):
    # the same with 8-bit weights and codes (the first encoder layer of the end-to-end workload)
    diff = layer_case(Bd, T=64, B=57, K=64, H=640, dirs=2, xb=8, hb=8, ob=4, seed=37)
    assert (diff > 0).sum() == 0


def test_layer_time_slicing_equals_two_groups_per_cluster(Bd):
    # longer windows, full groups: codes and final states of the time-sliced launch against the launch
    # that gives every cluster two groups
    T, B, K, H = 150, 64, 64, 640
    w = synth.single_layer(seed=29, T=T, B=B, K=K, H=H, bits=4, dirs=2)
    x_act, out = O.act_symmetric(3.0, 4), O.act_symmetric(1.0, 4)
    xq = pack_codes(O.quantize(w["x"], x_act).reshape(T * B, K), x_act)
    layers = [Bd.DeviceLstm(lw) for lw in w["layers"]]
    run = lambda: Bd.qlstm_layer_forward(xq, to_act(x_act), T, B, layers, to_act(out), want_state=True)
    a = run()
    assert Bd.q4_poll_status(a["workspace"]) == 0
    prev = Bd.encoder_time_slicing_set(False)
    try:
        b = run()
    finally:
        Bd.encoder_time_slicing_set(prev)
    assert Bd.q4_poll_status(b["workspace"]) == 0
    for k in ("yq", "hq_n", "c_n"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("T,B,K,H", [(8, 5, 64, 32),
                                     # 640 cells: int8 weights mostly in registers; 20 sequences = one group per
                                     # cluster, 57 over 64 steps = the clusters of one direction take turns
                                     (8, 20, 64, 640), (64, 57, 64, 640)])
def test_layer_per_sequence_input_scale(Bd, T, B, K, H):
    w = synth.single_layer(seed=5, T=T, B=B, K=K, H=H, bits=8, dirs=2)
    base = O.act_symmetric(1.0, 8)
    xq = np.empty((T, B, K), np.int16)
    sc = np.empty(B, np.float32)
    for b in range(B):
        a = O.act_symmetric(O.absmax(w["x"][:, b]), 8)
        xq[:, b] = O.quantize(w["x"][:, b], a)
        sc[b] = a.scale
    hid = O.act_symmetric(1.0, 8)
    ref = O.lstm_layer(O.Lstm(w["layers"]), xq, base, hid, x_scale_b=sc)
    for lw in w["layers"]:
        lw.hid_bits = 8
    got = Bd.qlstm_layer_forward(pack_codes(xq.reshape(T * B, K), base), to_act(base), T, B,
                                 [Bd.DeviceLstm(lw) for lw in w["layers"]],
                                 x_scale_b=torch.from_numpy(sc).cuda())
    assert Bd.q4_poll_status(got["workspace"]) == 0
    yq = gpu_codes(got["yq"], 2 * H, hid).reshape(T, B, 2 * H)
    np.testing.assert_array_equal(yq, ref["yq"])


def encoder_case(Bd, enc_w, feats, utts=None):
    E = enc_w["enc"]
    T, B, F = feats.shape
    dev = Bd.Encoder(E)
    got = dev.forward(torch.from_numpy(feats).cuda(), want_layers=True)
    sel = list(range(B)) if utts is None else utts
    ref = O.encoder_forward(E, feats[:, sel, :], want_layers=True)
    H2 = 2 * enc_w["H"]
    for l, yq in enumerate(got["layers"]):
        a = dev.out_acts[l]
        g = gpu_codes(yq, H2, a).reshape(T, B, H2)[:, sel]
        np.testing.assert_array_equal(g, ref["layers"][l]["yq"], err_msg=f"layer {l}")
    np.testing.assert_array_equal(got["e"].cpu().numpy()[:, sel], ref["e"])
    return 0.0


def test_encoder_reduced(Bd):
    enc = synth.encoder(seed=1, T=40, B=6, F=48, H=64, L=3, D=32)
    encoder_case(Bd, enc, enc["features"])


def test_encoder_reduced_int8_first_layer_max_input(Bd):
    enc = synth.encoder(seed=2, T=30, B=5, F=80, H=32, L=3, D=32, first_layer_bits=8, in_max=True)
    encoder_case(Bd, enc, enc["features"])


def test_config1_full_size_sampled_utterances(Bd):
    # 6-layer bidirectional encoder, 640 cells/direction, 240-dim input, T=500, B=32; the
    # oracle recomputes two of the 32 utterances (they are independent).
    enc = synth.encoder(seed=1)
    encoder_case(Bd, enc, enc["features"], utts=[3, 28])


def test_config4_encoder_full_size_sampled_utterances(Bd):
    # The encoder of the end-to-end workload at its full size and in its launch configuration: 64
    # utterances x 1000 log-mel frames (500 encoder steps), per-utterance MAX boundary, 8-bit first layer,
    # 4-bit layers 2-6, replayed as a CUDA graph.  16 groups of 8 sequences on 15 clusters: the clusters of
    # direction 0 take turns at the group of utterances 56-63 (71 or 72 steps each).  The oracle recomputes
    # utterance 5 (a cluster's own group) and utterance 58 (the shared group).
    B, T100 = 64, 1000
    T = T100 // 2
    enc_w = synth.encoder(4, T=T, B=B, first_layer_bits=8, in_max=True, features=False)
    mel = synth.logmel(4, B, T100, 40)
    mel_dev = torch.from_numpy(mel).cuda()
    enc = Bd.Encoder(enc_w["enc"])
    plan = Bd.encoder_recurrence_plan(T, B, 2, 640, 8, 8, True)
    if plan["max_clusters"] == 15:
        assert plan["kernel"] == 2 and plan["turns"] == [1, 0] and plan["clusters"] == [7, 8]
    run = Bd.GraphedStep(lambda: enc.forward(Bd.q4_feature_prologue(mel_dev), want_layers=True))
    got = run()
    got = run()
    torch.cuda.synchronize()
    assert Bd.q4_poll_status(enc.ws) == 0
    utts = [5, 58]
    feats_ref = np.stack([O.features(mel[b]) for b in utts], axis=1).astype(np.float16)
    ref = O.encoder_forward(enc_w["enc"], feats_ref, want_layers=True)
    for l, yq in enumerate(got["layers"]):
        g = gpu_codes(yq, 1280, enc.out_acts[l]).reshape(T, B, 1280)[:, utts]
        np.testing.assert_array_equal(g, ref["layers"][l]["yq"], err_msg=f"encoder layer {l}")
    np.testing.assert_array_equal(got["e"].cpu().numpy()[:, utts], ref["e"])


# ------------------------------------------------------------------ against the PLAIN oracle path
def plain_step_case(Bd, lw, x_act, hid, xq, hq, c):
    """qlstm_step against the textbook step (libm gates in double): real values within the
    tolerance, codes equal except within 1e-3 code units of a rounding boundary (+-1 there)."""
    want = O.lstm_step_plain(O.Lstm([lw]), xq, x_act, hq, c, hid)
    got = Bd.qlstm_step(pack_codes(xq, x_act), to_act(x_act), pack_codes(hq, hid),
                        torch.from_numpy(c).cuda(), Bd.DeviceLstm(lw))
    H = c.shape[1]
    assert_close(got["c"].cpu().numpy(), want["c"], "cell state")
    assert_close(got["h"].cpu().numpy(), want["h"], "cell output")
    g = gpu_codes(got["hq"], H, hid)
    diff = g.astype(np.int32) - want["hq"]
    tie = want["tie"] < 1e-3
    assert np.abs(diff).max() <= 1
    assert not ((diff != 0) & ~tie).any(), "code mismatch away from a rounding boundary"
    return diff.size, int(tie.sum()), int((diff != 0).sum())


def test_config0_teacher_forced_against_plain_step(Bd):
    w = synth.single_layer(seed=0)
    lw = w["layers"][0]
    x_act, hid = O.act_symmetric(w["x_clip"], 4), O.act_symmetric(1.0, 4)
    xq = O.quantize(w["x"], x_act)
    hq, c = np.zeros((4, 128), np.int16), np.zeros((4, 128), np.float32)
    L = O.Lstm([lw])
    tot = np.zeros(3, np.int64)
    for t in range(50):
        tot += plain_step_case(Bd, lw, x_act, hid, xq[t], hq, c)
        s = O.lstm_step_plain(L, xq[t], x_act, hq, c, hid)      # the plain path's own state feeds the next step
        hq, c = s["hq"], s["c"]
    print(f"config 0 vs plain step: {tot[0]} codes, {tot[1]} near a rounding boundary, {tot[2]} differ by one")


@pytest.mark.parametrize("bits", [4, 8])
def test_encoder_shaped_step_against_plain_step(Bd, bits):
    # 130 rows of the encoder's inner-layer shape (K = 1280, H = 640)
    st = synth.Stream(51 + bits)
    lw = synth._lstm(st, "l", 1280, 640, bits, 0.1, 0.95, bits)
    x_act, hid = O.act_symmetric(0.97, bits), O.act_symmetric(0.95, bits)
    N = 130
    xq = st.integers("xq", (N, 1280), x_act.lo() + 1, x_act.hi()).astype(np.int16)
    hq = st.integers("hq", (N, 640), hid.lo() + 1, hid.hi()).astype(np.int16)
    c = st.normal("c", (N, 640)).astype(np.float32)
    n, near, moved = plain_step_case(Bd, lw, x_act, hid, xq, hq, c)
    print(f"{bits} bit: {n} codes, {near} near a rounding boundary, {moved} differ by one")


# ------------------------------------------------------------------ 2-bit weights, mixed widths
@pytest.mark.parametrize("N,K,H,wb,xb,hb", [(70, 200, 64, 2, 4, 4), (130, 256, 128, 2, 8, 4), (9, 64, 64, 4, 8, 8),
                                             (33, 96, 64, 8, 4, 4), (5, 1280, 640, 2, 4, 4)])
def test_step_weight_and_activation_widths_mix(Bd, N, K, H, wb, xb, hb):
    # weights stored at 2, 4 or 8 bits under activations of 4 or 8 bits (Table 1's 2/4 rows; the
    # 8-bit first layer): integer accumulators, cell state and codes exact
    st = synth.Stream(300 + N)
    lw = synth._lstm(st, "l", K, H, wb, bias_std=0.2, hid_alpha=0.95, hid_bits=hb)
    x_act, hid = O.act_symmetric(3.0, xb), O.act_symmetric(0.95, hb)
    xq = st.integers("xq", (N, K), x_act.lo(), x_act.hi()).astype(np.int16)
    hq = st.integers("hq", (N, H), hid.lo() + 1, hid.hi()).astype(np.int16)
    c = st.normal("c", (N, H)).astype(np.float32)
    assert lw.w_ih.codes.min() == -(1 << (wb - 1)) and lw.w_ih.codes.max() == (1 << (wb - 1)) - 1
    step_case(Bd, lw, x_act, hid, xq, hq, c)


def test_layer_two_bit_weights(Bd):
    # bidirectional layer with 2-bit weights under 4-bit activations, 160 rows: tensor-core input
    # projection and persistent recurrence from int8 operand copies of the 2-bit codes
    T, B, K, H = 20, 8, 128, 64
    w = synth.single_layer(seed=21, T=T, B=B, K=K, H=H, bits=2, dirs=2)
    for lw in w["layers"]:
        lw.hid_bits = 4
    x_act, hid = O.act_symmetric(3.0, 4), O.act_symmetric(1.0, 4)
    xq = O.quantize(w["x"], x_act)
    ref = O.lstm_layer(O.Lstm(w["layers"]), xq, x_act, hid, want=("c_n", "acc_ih"))
    layers = [Bd.DeviceLstm(lw) for lw in w["layers"]]
    assert layers[0].w_ih.bits == 2 and layers[0].w_ih.q.shape[1] == K // 4
    for tc in (True, False):
        got = Bd.qlstm_layer_forward(pack_codes(xq.reshape(T * B, K), x_act), to_act(x_act), T, B, layers,
                                     want_state=True, want_dbg=True, tensor_cores=tc)
        np.testing.assert_array_equal(got["acc_ih"].cpu().numpy(), ref["acc_ih"])
        np.testing.assert_array_equal(gpu_codes(got["yq"], 2 * H, hid).reshape(T, B, 2 * H), ref["yq"])
        np.testing.assert_array_equal(got["c_n"].cpu().numpy(), ref["c_n"])


def test_outer_and_inner_quantizer_placement_counted_on_the_device(Bd):
    # Section 3.4 on the device: the library counts its activation-quantizer applications.  Outer
    # placement (quantize once at each cell output; the input once per frame): T + T L.  Inner
    # placement (every cell quantizes its two inputs on entry): 2 T L.  L = 12 cells (6 layers x 2
    # directions).  Both placements give the same network output; the oracle's two paths agree
    # with both, value for value.
    T, B, Lc = 5, 3, 12
    enc = synth.encoder(seed=1, T=T, B=B, F=32, H=32, L=6, D=32, with_proj=False)
    E = enc["enc"]
    feats = torch.from_numpy(enc["features"].astype(np.float32)).cuda()
    dev = Bd.Encoder(E)
    # Outer, input quantized frame by frame
    Bd.quantizer_calls(reset=True)
    frames = [Bd.quantize_pack_int4(feats[t].contiguous(), dev.in_act) for t in range(T)]
    xq, x_act = torch.cat(frames, 0), dev.in_act
    for l, dirs in enumerate(dev.layers):
        r = Bd.qlstm_layer_forward(xq, x_act, T, B, dirs, dev.out_acts[l])
        xq, x_act = r["yq"], dev.out_acts[l]
    outer = Bd.quantizer_calls(reset=True)
    # Inner
    x = feats
    x_act = dev.in_act
    for l, dirs in enumerate(dev.layers):
        x = Bd.lstm_layer_inner(x, x_act, dirs)
        x_act = dirs[0].hid_act
    inner = Bd.quantizer_calls(reset=True)
    assert outer == T + T * Lc and inner == 2 * T * Lc
    assert round(100 * (1 - outer / inner)) in (45, 46)
    ref = O.encoder_forward(E, enc["features"], want_layers=True)
    np.testing.assert_array_equal(gpu_codes(xq, 64, dev.out_acts[-1]).reshape(T, B, 64), ref["yq"])
    np.testing.assert_array_equal(x.cpu().numpy(), ref["layers"][-1]["h"])
    np.testing.assert_array_equal(x.cpu().numpy(), O.encoder_forward_inner(E, enc["features"]))


@pytest.mark.parametrize("N,K,H,xb,hb,signed", [(130, 256, 128, 4, 4, True), (300, 96, 256, 4, 4, False),
                                                 (128, 240, 128, 8, 8, True), (257, 64, 384, 4, 8, True)])
def test_step_on_the_tensor_cores_with_prepared_weights(Bd, N, K, H, xb, hb, signed):
    # qlstm_step with the one-time int8 operands: tcgen05 kernel, same integers and floats as the oracle
    st = synth.Stream(400 + N)
    lw = synth._lstm(st, "l", K, H, 4, bias_std=0.2, hid_alpha=0.95, hid_bits=hb)
    if xb == 8:
        lw.w_ih = synth._qmat(st, "w8", 4 * H, K, 8)
    if hb == 8:
        lw.w_hh = synth._qmat(st, "h8", 4 * H, H, 8)
    x_act = O.act_symmetric(3.0, xb) if signed else O.act_asymmetric(-1.7, 1.4, 4)
    hid = O.act_symmetric(0.95, hb)
    xq = st.integers("xq", (N, K), x_act.lo(), x_act.hi()).astype(np.int16)
    hq = st.integers("hq", (N, H), hid.lo() + 1, hid.hi()).astype(np.int16)
    c = st.normal("c", (N, H)).astype(np.float32)
    n0 = Bd.launch_count()
    step_case(Bd, lw, x_act, hid, xq, hq, c, prepare=True)
    # packing of the test operands aside: two gathers and one fused kernel (not the DP4A kernel alone)
    assert Bd.launch_count() - n0 >= 3


def test_bounded_wait_runs_out_and_the_stream_stays_usable(Bd):
    # The consumer of the tiled tensor-core GEMM waits for operand tiles a bounded number of polls.  With
    # the test hook the producer issues nothing (so nothing asynchronous is in flight): the wait runs
    # out, every role of the kernel returns, the status word reads Q4_ERR_TIMEOUT, nothing was stored,
    # and the next call on the same stream is correct.
    import ctypes as C
    st = synth.Stream(77)
    M, K, J = 200, 256, 256
    lw = synth._linear(st, "lin", J, K)
    a = O.act_symmetric(1.0, 4)
    xq = st.integers("xq", (M, K), -7, 7).astype(np.int16)
    want = O.linear(O.Linear(lw), xq, a)
    lin = Bd.DeviceLinear(lw).prepare()
    x_dev = pack_codes(xq, a)
    lib = Bd.lib()
    assert lib.q4_test_wait_expiry_set(C.c_int32(1), C.c_uint32(1 << 12)) == 0
    try:
        out = Bd.q4_linear_forward(x_dev, to_act(a), lin)
        assert Bd.q4_poll_status(lin.ws) == -8                      # Q4_ERR_TIMEOUT
    finally:
        lib.q4_test_wait_expiry_set(C.c_int32(0), C.c_uint32(0))
    torch.cuda.synchronize()
    out = Bd.q4_linear_forward(x_dev, to_act(a), lin)               # same stream, same buffers
    assert Bd.q4_poll_status(lin.ws) == 0
    np.testing.assert_array_equal(out.cpu().numpy(), want)
