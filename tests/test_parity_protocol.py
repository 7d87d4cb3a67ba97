"""The whole-head comparison protocol itself (tests/parity.py), on the CPU: an output that took a near-decision
the other way is accepted through the oracle's report, anything else that exceeds the tolerance is refused."""
import numpy as np
import pytest

from oracle import attention as A
from oracle import quantize as Qz
from paper_2609_04105_b200 import inputs as I

import parity


def _one_hot_case():
    """One head whose rows are close to one-hot (outlier channels as in configuration 4), N = 512."""
    w = I.shrink(I.WORKLOADS["cfg4"], H=1, N=512)
    q, k, v = I.make_qkv(w)
    return w, Qz.quantize_qk(q, "mx"), Qz.quantize_qk(k, "mx"), Qz.quantize_v(v)


def test_default_evaluation_passes_and_a_flipped_near_decision_is_accepted():
    w, qd, kd, vd = _one_hot_case()
    O, L = A.direct_p_forward(qd, kd, vd)
    st = parity.compare_head(A.bf16_round(O[0]), L[0], qd, kd, vd, 0, 0, chunk=200)
    assert st["rows_failing_strict"] == 0 and st["rel_fro"] < 2.5e-3

    # plant the alternative: find a reported near-decision whose flip moves its row beyond the tolerance
    c32 = A.score_constant(qd, kd, w.d)
    s32 = A.scores_fp32(qd, kd, 0, 0)
    Vhat = parity._vhat(vd, 0, 0)
    rep = {}
    A.direct_p_rows(s32, c32, Vhat, report=rep, ambiguity=dict(rel=2.0 ** -9))      # wide net, to have candidates
    planted = None
    for i, j in zip(*np.nonzero(rep["code"])):
        fl = {"code": np.zeros((1, w.N), bool)}
        fl["code"][0, j] = True
        O2, L2, _, _, _ = A.direct_p_rows(s32[i:i + 1], c32, Vhat, flips=fl)
        if np.abs(O2[0] - O[0, i]).max() > 1.5 * parity.MAX_ABS:
            planted = (i, O2[0], L2[0])
            break
    assert planted is not None, "no visible near-decision in the test head"
    i, o_alt, l_alt = planted
    Og, Lg = A.bf16_round(O[0]), L[0].copy()
    Og[i], Lg[i] = A.bf16_round(o_alt), l_alt
    with pytest.raises(AssertionError):                                             # default thresholds do not list it ...
        parity.compare_head(Og, Lg, qd, kd, vd, 0, 0, chunk=200)
    st = parity.compare_head(Og, Lg, qd, kd, vd, 0, 0, chunk=200, ambiguity=dict(rel=2.0 ** -9))   # ... the wide net does
    assert st["rows_failing_strict"] == 1 and st["accepted_with_flips"] == 1
    assert st["max_abs_strict"] > parity.MAX_ABS >= st["max_abs"]


def test_an_error_that_is_no_near_decision_is_refused():
    w, qd, kd, vd = _one_hot_case()
    O, L = A.direct_p_forward(qd, kd, vd)
    Og = A.bf16_round(O[0])
    Og[17, 3] += 0.05
    with pytest.raises(AssertionError):
        parity.compare_head(Og, L[0], qd, kd, vd, 0, 0)
    Lg = L[0].copy()
    Lg[200] += 0.01
    with pytest.raises(AssertionError):
        parity.compare_head(A.bf16_round(O[0]), Lg, qd, kd, vd, 0, 0)
