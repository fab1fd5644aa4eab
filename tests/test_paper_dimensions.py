"""The model sizes the paper states (Section 2): parameter counts on the CPU, and the GPU path against
the oracle at exactly those sizes (odd ones: 46 output characters, 340-d input, 10-d embedding)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2206_07882_b200 import synth
from test_oracle_quantizers import gold as _gold


def gold(name):
    return _gold()[name]


def test_parameter_counts_match_section_2():
    enc, dec = synth.paper_dimensions(T=2, B=1, U_max=1)
    n = synth.parameter_counts(enc["enc"], dec)
    # the paper prints millions with one decimal; one bias vector per LSTM here (two would add 0.03 M)
    assert abs(n["encoder"] / 1e6 - gold("params_encoder_m")) < 0.1
    assert abs(n["prediction"] / 1e6 - gold("params_prediction_m")) < 0.05
    assert abs(n["rnnt"] / 1e6 - gold("params_rnnt_m")) < 0.15
    assert abs(n["lm_ext"] / 1e6 - gold("params_lm_ext_m")) < 0.05
    assert abs(n["lm_src"] / 1e6 - gold("params_prediction_m")) < 0.05     # "same building blocks and size"
    assert (dec.lambda_t, dec.lambda_s, dec.rho) == (gold("mu"), gold("lambda"), gold("rho"))


@pytest.fixture(scope="module")
def Bd():
    from paper_2206_07882_b200 import binding
    return binding


@pytest.mark.gpu
def test_paper_sized_model_end_to_end(Bd):
    # 2 utterances, 8 encoder frames, label budget 4, beam 16: encoder output exact, then every beam of
    # every iteration identical to the oracle's
    from test_gpu_decode import compare_search, run_search
    T, B, U = 8, 2, 4
    enc, dec = synth.paper_dimensions(T=T, B=B, U_max=U)
    got = Bd.Encoder(enc["enc"]).forward(torch.from_numpy(enc["features"]).cuda())
    ref_e = O.encoder_forward(enc["enc"], enc["features"])["e"]
    np.testing.assert_array_equal(got["e"].cpu().numpy(), ref_e)
    dd, tokens, lens, scores, ref = run_search(Bd, dec, ref_e)
    frac, tr = compare_search(dd, tokens, lens, scores, ref, list(range(B)), T, U, dec.W, min_same=1.0)
    assert tr == 1.0
