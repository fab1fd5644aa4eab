"""Pins for the oracle's prediction network, LMs, joint, Eq. 1 and beam search.

The search is pinned by brute force: with a beam at least as wide as the number
of live label strings nothing is pruned, so every final score must equal Eq. 1
with log P(y|x) from the textbook transducer forward recursion, written here in
numpy independently of the oracle's search code.
"""
import itertools

import numpy as np
import pytest

from oracle import oracle as O
from paper_2206_07882_b200 import synth


def tiny_decoder(seed=21, V=3, U_max=2, W=16, **kw):
    dw = synth.decoder(seed, V=V, E=8, Hp=8, D=8, Hs=8, Ht=8, tgt_layers=2, U_max=U_max, W=W, **kw)
    return dw, O.Decoder(dw)


def tiny_e(seed, T, D=8):
    return synth.Stream(seed).normal("e", (T, 1, D), 0.0, 1.0).astype(np.float32)


def logadd(a, b):
    if a == -np.inf:
        return b
    if b == -np.inf:
        return a
    m = max(a, b)
    return m + np.log1p(np.exp(-abs(a - b)))


def brute_force_score(dec, dw, e_utt, y):
    """Eq. 1 for label string y: forward recursion over the (t,u) lattice in numpy."""
    T, U = e_utt.shape[0], len(y)
    toks = np.array([[0] + list(y)], dtype=np.int32)                  # start symbol, then labels
    # joint log-probs for every (u, t): run the forced routine once per frame
    lp = np.zeros((U + 1, T, dec.V))
    for t in range(T):
        fi = np.full((1, U + 1), t, dtype=np.int32)
        lp[:, t, :] = O.pred_joint_forced(dec, e_utt, fi, toks)[0]
    alpha = np.full((T, U + 1), -np.inf)
    alpha[0, 0] = 0.0
    for t in range(T):
        for u in range(U + 1):
            if t == 0 and u == 0:
                continue
            v = -np.inf
            if t > 0:
                v = logadd(v, alpha[t - 1, u] + lp[u, t - 1, 0])
            if u > 0:
                v = logadd(v, alpha[t, u - 1] + lp[u - 1, t, y[u - 1]])
            alpha[t, u] = v
    log_p = alpha[T - 1, U] + lp[U, T - 1, 0]
    lt = ls = 0.0
    if U:
        lpt = O.lm_forced(dec, "tgt", toks)[0]
        lps = O.lm_forced(dec, "src", toks)[0]
        lt = sum(float(lpt[u, y[u]]) for u in range(U))
        ls = sum(float(lps[u, y[u]]) for u in range(U))
    return log_p + dw.lambda_t * lt - dw.lambda_s * ls + dw.rho * U, log_p, lt, ls


def all_strings(V, U_max):
    for n in range(U_max + 1):
        yield from itertools.product(range(1, V), repeat=n)


def finals_dict(r, i=0):
    return {tuple(r["finals_tokens"][i, f, :r["finals_len"][i, f]].tolist()): float(r["finals_score"][i, f])
            for f in range(r["finals_n"][i])}


@pytest.mark.parametrize("T,U_max,seed", [(1, 2, 0), (2, 2, 1), (3, 2, 2), (3, 1, 3), (2, 3, 4)])
def test_unpruned_search_equals_brute_force_eq1(T, U_max, seed):
    dw, dec = tiny_decoder(seed=30 + seed, U_max=U_max, W=16)
    e = tiny_e(seed, T)
    r = O.alsd(dec, e)
    got = finals_dict(r)
    strings = list(all_strings(3, U_max))
    assert len(strings) <= 16 and set(got) == set(strings)
    for y in strings:
        want = brute_force_score(dec, dw, e[:, 0, :], y)[0]
        assert abs(got[y] - want) < 2e-5, (y, got[y], want)
    best = max(strings, key=lambda y: got[y])
    assert tuple(r["tokens"][0, :r["len"][0]].tolist()) == best
    assert abs(r["score"][0] - got[best]) == 0.0


def test_sequence_score_routine_matches_numpy_recursion():
    dw, dec = tiny_decoder(seed=41, V=5, U_max=3)
    e = tiny_e(9, 4)
    for y in [(), (2,), (1, 4), (3, 3, 1)]:
        want = brute_force_score(dec, dw, e[:, 0, :], y)
        got = O.sequence_score(dec, e[:, 0, :], y)
        np.testing.assert_allclose(got, want, rtol=1e-6, atol=2e-6)


def test_fusion_weights_zero_give_plain_transducer_scores():
    dw, dec = tiny_decoder(seed=50, lambda_t=0.0, lambda_s=0.0, rho=0.0)
    e = tiny_e(5, 3)
    got = finals_dict(O.alsd(dec, e))
    for y, s in got.items():
        assert abs(s - brute_force_score(dec, dw, e[:, 0, :], y)[1]) < 2e-5
    # all label strings of a transducer with the search unpruned and U unbounded sum to 1;
    # with U_max = 2 they sum to at most 1
    assert np.logaddexp.reduce(list(got.values())) <= 1e-5


def test_lm_terms_cancel_when_both_lms_are_the_same():
    # Eq. 1 with P_ext == P_src and mu == lambda: the LM terms drop out exactly.
    dw, _ = tiny_decoder(seed=60, lambda_t=0.4, lambda_s=0.4, rho=0.1)
    dw.tgt = dw.src
    dec = O.Decoder(dw)
    e = tiny_e(6, 3)
    got = finals_dict(O.alsd(dec, e))
    for y, s in got.items():
        assert abs(s - (brute_force_score(dec, dw, e[:, 0, :], y)[1] + 0.1 * len(y))) < 2e-5


def test_length_reward_is_rho_times_length():
    dw0, dec0 = tiny_decoder(seed=70, rho=0.0)
    dw1, dec1 = tiny_decoder(seed=70, rho=0.35)
    e = tiny_e(7, 2)
    a, b = finals_dict(O.alsd(dec0, e)), finals_dict(O.alsd(dec1, e))
    for y in a:
        assert abs((b[y] - a[y]) - 0.35 * len(y)) < 2e-5


def test_beam_one_is_greedy():
    # W = 1: one hypothesis survives each iteration, the best proposal under Eq. 1
    # increments; on the last frame the blank proposal is final (finals bypass pruning)
    # and the best label proposal carries on.
    dw, dec = tiny_decoder(seed=80, V=6, U_max=3, W=1)
    T = 4
    e = tiny_e(8, T)
    r = O.alsd(dec, e)
    y, t, S = [], 0, 0.0
    finals = []
    alive = True
    for it in range(T + 3):
        if not alive:
            assert r["n_slots"][0, it] == 0
            continue
        toks = np.array([[0] + y], dtype=np.int32)
        u = len(y)
        lp = O.pred_joint_forced(dec, e[:, 0, :], np.full((1, u + 1), t, np.int32), toks)[0, u]
        cand = {}
        if t + 1 == T:
            finals.append((S + float(lp[0]), list(y)))
        else:
            cand[0] = S + float(lp[0])
        if u < 3:
            lt = O.lm_forced(dec, "tgt", toks)[0, u]
            ls = O.lm_forced(dec, "src", toks)[0, u]
            for k in range(1, 6):
                cand[k] = S + float(lp[k]) + dw.lambda_t * float(lt[k]) - dw.lambda_s * float(ls[k]) + dw.rho
        if not cand:
            alive = False
            assert r["n_slots"][0, it] == 0
            continue
        k = max(cand, key=lambda k: (cand[k], -k))
        S = cand[k]
        assert r["token"][0, it, 0] == k and abs(r["tscore"][0, it, 0] - S) < 2e-5
        if k == 0:
            t += 1
        else:
            y.append(k)
    best = max(finals, key=lambda f: f[0])
    assert r["tokens"][0, :r["len"][0]].tolist() == best[1]
    assert abs(r["score"][0] - best[0]) < 2e-5


def test_pruned_beam_trace_invariants():
    dw, dec = tiny_decoder(seed=90, V=12, U_max=6, W=4)
    T = 8
    e = tiny_e(10, T)
    r = O.alsd(dec, e)
    IT = T + 6
    for it in range(IT):
        n = r["n_slots"][0, it]
        assert 0 <= n <= 4
        sc = r["tscore"][0, it, :n]
        assert (np.diff(sc) <= 0).all()                       # slots are in rank order
        assert ((r["t"][0, it, :n] + r["u"][0, it, :n]) == it + 1).all()   # alignment length
        assert (r["t"][0, it, :n] < T).all() and (r["u"][0, it, :n] <= 6).all()
        # label strings within a beam are distinct (merging): rebuild them from back-pointers
        strings = set()
        for s in range(n):
            y, ss = [], s
            for j in range(it, -1, -1):
                k = r["token"][0, j, ss]
                if k > 0:
                    y.append(int(k))
                ss = r["parent"][0, j, ss]
            strings.add(tuple(reversed(y)))
        assert len(strings) == n
    # the reported best is one of the finals and its score is Eq. 1-consistent: not above
    # the unpruned total for that string
    y = tuple(r["tokens"][0, :r["len"][0]].tolist())
    full = brute_force_score(dec, dw, e[:, 0, :], y)[0]
    assert r["score"][0] <= full + 2e-5


def test_joint_is_multiplicative_tanh_quantize_linear_logsoftmax():
    dw, dec = tiny_decoder(seed=100, V=7)
    rng = np.random.default_rng(0)
    e = rng.normal(0, 1, (5, 8)).astype(np.float32)
    p = rng.normal(0, 1, (5, 8)).astype(np.float32)
    lp, zq, acc = O.joint(dec, e, p, want_zq=True)
    a = O.act_symmetric(1.0, 4)
    z = np.tanh(e.astype(np.float64) * p.astype(np.float64)).astype(np.float32)
    np.testing.assert_array_equal(zq, O.quantize(z, a))
    out = dw.joint.out
    logits = (zq.astype(np.float64) * a.scale) @ (out.w.codes.astype(np.float64) * out.w.scale.astype(np.float64)[:, None]).T + out.bias
    import torch
    want = torch.log_softmax(torch.from_numpy(logits), dim=1).numpy()
    np.testing.assert_allclose(lp, want, atol=2e-6)
    # symmetric in its two inputs (a product), unlike an additive joint with separate weights
    np.testing.assert_array_equal(O.joint(dec, p, e), lp)


def test_lm_step_chain_by_parts():
    # LM = embedding -> quantize (asymmetric constants) -> LSTM layers -> bottleneck ->
    # quantize -> output -> log-softmax; rebuilt here from the separately pinned parts.
    dw, dec = tiny_decoder(seed=110, V=9)
    m = dw.tgt
    toks = np.array([[0, 4, 2]], dtype=np.int32)
    got = O.lm_forced(dec, "tgt", toks)[0]
    ea = O.act_asymmetric(m.emb_lo, m.emb_hi, 4)
    ba = O.act_asymmetric(m.bott_lo, m.bott_hi, 4)
    hq = [np.zeros((1, 8), np.int16) for _ in m.lstm]
    c = [np.zeros((1, 8), np.float32) for _ in m.lstm]
    for s in range(3):
        x, xa = O.quantize(m.emb[toks[0, s]][None, :], ea), ea
        for l, lw in enumerate(m.lstm):
            ha = O.act_symmetric(lw.hid_alpha, 4)
            r = O.lstm_step(O.Lstm([lw]), x, xa, hq[l], c[l], ha)
            hq[l], c[l] = r["hq"], r["c"]
            x, xa = r["hq"], ha
        b = O.linear(O.Linear(m.bott), x, xa)
        logits = O.linear(O.Linear(m.out), O.quantize(b, ba), ba)
        np.testing.assert_array_equal(got[s], O.log_softmax(logits)[0])
    assert ea.is_signed == 0 and 0 < ea.zero_point < 15


def test_slot_order_does_not_matter():
    # permuting nothing but the thread count / utterance order leaves results unchanged
    dw, dec = tiny_decoder(seed=120, V=8, U_max=4, W=4)
    e = synth.Stream(3).normal("e", (6, 5, 8)).astype(np.float32)
    a = O.alsd(dec, e, n_threads=1)
    b = O.alsd(dec, e, utts=[4, 3, 2, 1, 0], n_threads=3)
    for k in ("tokens", "len", "score"):
        np.testing.assert_array_equal(a[k], b[k][::-1])


# ---------------------------------------------------------------- time-synchronous search
@pytest.mark.parametrize("T,U_max,seed", [(1, 2, 0), (2, 2, 1), (3, 2, 2), (3, 1, 3), (2, 3, 4)])
def test_time_synchronous_unpruned_equals_brute_force_eq1(T, U_max, seed):
    # beam >= number of label strings and as many labels per frame as the budget allows: nothing is
    # pruned, every alignment is reachable, so every final score is Eq. 1 by the forward recursion
    dw, dec = tiny_decoder(seed=30 + seed, U_max=U_max, W=16)
    e = tiny_e(seed, T)
    r = O.tsd(dec, e, S_max=U_max)
    got = finals_dict(r)
    strings = list(all_strings(3, U_max))
    assert set(got) == set(strings)
    for y in strings:
        want = brute_force_score(dec, dw, e[:, 0, :], y)[0]
        assert abs(got[y] - want) < 2e-5, (y, got[y], want)
    # the two search orders agree when neither prunes
    ref = finals_dict(O.alsd(dec, e))
    for y in strings:
        assert abs(got[y] - ref[y]) < 2e-5
    best = max(strings, key=lambda y: got[y])
    assert tuple(r["tokens"][0, :r["len"][0]].tolist()) == best
    # finals are listed best first
    fs = r["finals_score"][0, :r["finals_n"][0]]
    assert (np.diff(fs) <= 0).all()


def test_time_synchronous_label_limit_per_frame():
    dw, dec = tiny_decoder(seed=52, V=4, U_max=3, W=16)
    e = tiny_e(5, 2)
    # no labels at all: the empty string, scored by the blanks alone
    r0 = O.tsd(dec, e, S_max=0)
    assert finals_dict(r0).keys() == {()}
    assert abs(finals_dict(r0)[()] - brute_force_score(dec, dw, e[:, 0, :], ())[0]) < 2e-5
    # one frame, one label per frame: strings of length <= 1, each with its single alignment
    e1 = tiny_e(6, 1)
    r1 = O.tsd(dec, e1, S_max=1)
    got = finals_dict(r1)
    assert set(got) == {(), (1,), (2,), (3,)}
    for y in got:
        assert abs(got[y] - brute_force_score(dec, dw, e1[:, 0, :], y)[0]) < 2e-5
    # two frames, one label per frame: "ab" needs a at frame 0 and b at frame 1 -- one alignment of the
    # three the lattice has, so its score stays below the full sum
    r2 = O.tsd(dec, e, S_max=1)
    got2 = finals_dict(r2)
    full = brute_force_score(dec, dw, e[:, 0, :], (1, 2))[0]
    assert (1, 2) in got2 and got2[(1, 2)] < full
    assert max(len(y) for y in got2) == 2


def test_time_synchronous_pruned_trace_invariants():
    dw, dec = tiny_decoder(seed=61, V=6, U_max=5, W=3)
    T, S = 6, 2
    e = tiny_e(8, T)
    r = O.tsd(dec, e, S_max=S)
    par, tok, sc, u, ns = r["parent"][0], r["token"][0], r["tscore"][0], r["u"][0], r["n_slots"][0]
    assert ns.shape == (T * (S + 1),) and (ns <= 3).all() and ns[-1] >= 1
    for it in range(T * (S + 1)):
        s = it % (S + 1)
        n = ns[it]
        prev_n = 1 if it == 0 else ns[it - 1]
        prev_u = np.zeros(1, np.int32) if it == 0 else u[it - 1]
        assert (np.diff(sc[it, :n]) <= 0).all()                      # ranked by score
        if s < S:
            assert ((tok[it, :n] >= 1) & (tok[it, :n] < 6)).all()
            assert ((par[it, :n] >= 0) & (par[it, :n] < prev_n)).all()
            assert (u[it, :n] == prev_u[par[it, :n]] + 1).all()
            assert (u[it, :n] <= 5).all()
        else:
            org = -1 - tok[it, :n]
            assert ((org >= 0) & (org <= S)).all()                   # the step the blank was proposed in
            assert (par[it, :n] >= 0).all()
    # the best final is the first slot of the last frame close
    assert abs(r["score"][0] - sc[-1, 0]) == 0.0 and r["len"][0] == u[-1, 0]


# ---------------------------------------------------------------- prediction network by parts
def test_prediction_network_chain_by_parts():
    # prediction network = embedding row -> symmetric quantizer with the FIX boundary 1.25
    # (Section 3.2) -> LSTM step -> linear to D fed with the hidden-state codes under the hidden
    # quantizer; rebuilt here from the separately pinned parts and compared with the forced routine.
    dw, dec = tiny_decoder(seed=130, V=9)
    P = dw.pred
    assert P.emb_alpha == 1.25
    toks = np.array([[0, 5, 3, 8]], dtype=np.int32)
    e = synth.Stream(9).normal("e", (4, 8)).astype(np.float32)
    fi = np.array([[2, 0, 3, 1]], dtype=np.int32)
    lp, hq_g, c_g, p_g = O.pred_joint_forced(dec, e, fi, toks, want_state=True)
    ea = O.act_symmetric(P.emb_alpha, 4)
    ha = O.act_symmetric(P.lstm.hid_alpha, P.lstm.hid_bits)
    assert ea.is_signed == 1 and ea.zero_point == 0 and abs(ea.scale - 1.25 / 7) < 1e-7
    hq, c = np.zeros((1, 8), np.int16), np.zeros((1, 8), np.float32)
    L, proj = O.Lstm([P.lstm]), O.Linear(P.proj)
    for s in range(4):
        xq = O.quantize(P.emb[toks[0, s]][None, :], ea)
        r = O.lstm_step(L, xq, ea, hq, c, ha)
        hq, c = r["hq"], r["c"]
        p = O.linear(proj, hq, ha)                       # hidden codes with the HIDDEN quantizer's scale
        np.testing.assert_array_equal(hq_g[0, s], hq[0])
        np.testing.assert_array_equal(c_g[0, s], c[0])
        np.testing.assert_array_equal(p_g[0, s], p[0])
        np.testing.assert_array_equal(lp[0, s], O.joint(dec, e[fi[0, s]][None, :], p)[0])
    # the two quantizers differ, so feeding the projection with the wrong one would show
    assert not np.array_equal(O.linear(proj, hq, ea), p)


def test_joint_and_linear_fixed_sequences_against_plain_definitions():
    # tanh(e p) by the fixed fp32 sequence vs libm in double: codes equal away from rounding
    # boundaries; the fp32 linear layer vs W x + b in double
    dw, dec = tiny_decoder(seed=140, V=11)
    st = synth.Stream(12)
    e = st.normal("e", (400, 8)).astype(np.float32)
    p = (st.normal("p", (400, 8)) * 1.5).astype(np.float32)
    a = O.act_symmetric(1.0, 4)
    _, zq, _ = O.joint(dec, e, p, want_zq=True)
    zq_p, tie = O.joint_z_plain(e, p, a)
    d = zq.astype(np.int32) - zq_p
    assert np.abs(d).max() <= 1 and not ((d != 0) & (tie >= 1e-3)).any()
    out = O.Linear(dw.joint.out)
    got = O.linear(out, zq, a)
    want = O.linear_plain(out, zq, a)
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-6)
