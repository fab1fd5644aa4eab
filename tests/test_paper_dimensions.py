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


def test_precision_assignment_of_section_3_2_gives_the_printed_shares():
    # first encoder layer and the RNN-T's linear layers at 8 bits, the rest at 4: the paper prints
    # 94.9 % of the parameters at 4 bits, a 7.6x smaller model, 432.5 MB -> 57.2 MB (Table 1: RNN-T
    # plus the external LM).  Counted here from the weight matrices of the paper-sized model.
    enc, dec = synth.paper_dimensions(T=2, B=1, U_max=1, section_3_2=True)
    E = enc["enc"]
    assert E.layers[0][0].w_ih.bits == 8 and E.layers[1][0].w_ih.bits == 4 and E.in_max
    assert E.proj.w.bits == 8 and dec.pred.proj.w.bits == 8 and dec.joint.out.w.bits == 8
    assert dec.tgt.out.w.bits == 4 and dec.pred.lstm.w_hh.bits == 4
    st = synth.weight_storage(E, dec)
    assert abs(st["frac_4bit"] - gold("frac_params_4bit")) < 0.002
    assert abs(st["compression"] - gold("compression_full")) < 0.05
    assert abs(st["params"] * 4 / 1e6 - gold("size_fp32_mb")) < 1.0
    assert abs(st["bytes"] / 1e6 - gold("size_int4_mb")) < 0.6


@pytest.fixture(scope="module")
def Bd():
    from paper_2206_07882_b200 import binding
    return binding


@pytest.mark.gpu
@pytest.mark.parametrize("section_3_2", [False, True])
def test_paper_sized_model_end_to_end(Bd, section_3_2):
    # 2 utterances, 8 encoder frames, label budget 4, beam 16: encoder output exact, then every beam of
    # every iteration identical to the oracle's; all at 4 bits, and with Section 3.2's assignment
    # (8-bit first layer with the MAX input boundary, 8-bit linear layers)
    from test_gpu_decode import compare_search, run_search
    T, B, U = 8, 2, 4
    enc, dec = synth.paper_dimensions(T=T, B=B, U_max=U, section_3_2=section_3_2)
    got = Bd.Encoder(enc["enc"]).forward(torch.from_numpy(enc["features"]).cuda())
    ref_e = O.encoder_forward(enc["enc"], enc["features"])["e"]
    np.testing.assert_array_equal(got["e"].cpu().numpy(), ref_e)
    dd, tokens, lens, scores, ref = run_search(Bd, dec, ref_e)
    frac, tr = compare_search(dd, tokens, lens, scores, ref, list(range(B)), T, U, dec.W, min_same=1.0)
    assert tr == 1.0
