"""Pins for the bookkeeping that decides what the GPU parity harness may excuse.

A step whose decisions differ between the library and the oracle is excused only when the first
differing decision sits near its boundary on the oracle's side.  The distances come from
`invcdf_margin` and from the `ratio_margin` / `row_top2` / `final_margin` / `draft_margin` /
`draft_top2` fields of `PassOracle.decide`; the classification is `parity_util.classify`.  Every
value below is worked out by hand from laws with known interval edges, so a helper that
returned 0 (everything excused) or infinity (nothing excused) fails here, on the CPU.
"""
import math

import numpy as np
import pytest

from oracle import pass_oracle as po
import parity_util as pu


class _Backend:
    vocab = 4


def _oracle(drafts, top_k=0):
    orc = po.PassOracle.__new__(po.PassOracle)
    orc.be, orc.len, orc.pending = _Backend(), 10, 1
    orc.drafts = list(drafts)
    orc.Q_dft = np.zeros((0, 4))
    orc.k_prev = orc.T_prev = None
    orc.top_k = orc.top_k_prev = top_k
    orc.last_logits = None
    return orc


def _logits(p):
    return np.log(np.asarray(p, dtype=np.float64))


# --------------------------------------------------------------------------- invcdf_margin
@pytest.mark.parametrize("u,token,margin", [
    (0.30, 1, 0.05),     # interval of token 1 is (0.25, 0.75]: nearest edge 0.25
    (0.70, 1, 0.05),     # nearest edge 0.75
    (0.50, 1, 0.25),     # the middle
    (0.10, 0, 0.15),     # interval of token 0 is [0, 0.25): only its upper edge can flip the token
    (0.76, 2, 0.01),
    (0.999, 2, 0.001),   # the last edge, 1.0
])
def test_invcdf_margin_is_the_distance_to_the_nearest_interval_edge(u, token, margin):
    w = np.array([1.0, 2.0, 1.0])            # unnormalised on purpose: edges at 0.25, 0.75, 1
    assert po.invcdf(w, u) == token
    assert po.invcdf_margin(w, u) == pytest.approx(margin, abs=1e-12)


def test_invcdf_margin_ignores_scale_and_zero_weights():
    w = np.array([0.0, 3.0, 0.0, 1.0])       # edges 0, 0.75, 0.75, 1
    assert po.invcdf_margin(w, 0.7) == pytest.approx(0.05, abs=1e-12)
    assert po.invcdf_margin(10 * w, 0.7) == pytest.approx(0.05, abs=1e-12)
    assert po.invcdf_margin(w, 0.8) == pytest.approx(0.05, abs=1e-12)


# --------------------------------------------------------------------------- decide(): margins
def test_decide_reports_ratio_cdf_and_top2_margins_of_known_laws():
    # one pending draft (token 0) drawn from Q = [.8 .1 .05 .05]; targets P0 = [.5 .25 .125 .125], P1 = [.1 .2 .3 .4]
    Q = np.array([[0.8, 0.1, 0.05, 0.05]])
    P0, P1 = [0.5, 0.25, 0.125, 0.125], [0.1, 0.2, 0.3, 0.4]
    la = [0.25, 0.25, 0.25, 0.25]
    Z = np.stack([_logits(P0), _logits(P1), _logits(la)])
    orc = _oracle([0])
    # accept: ratio 0.5/0.8 = 0.625 against u = 0.6; final token from P1 with u = 0.35 (edges .1 .3 .6 1)
    dec = orc.decide(Z, Q, 1, 1.0, [0.6, 0.35, 0.9])
    info = dec["info"]
    assert dec["n_accepted"] == 1 and dec["emitted"] == [0, 2]
    assert info["ratio_margin"] == [pytest.approx(0.025, abs=1e-12)]
    assert info["final_margin"] == pytest.approx(0.05, abs=1e-12)
    assert info["row_top2"][0] == pytest.approx(math.log(2.0), abs=1e-12)        # .5 against .25
    assert info["row_top2"][1] == pytest.approx(math.log(4.0 / 3.0), abs=1e-12)  # .4 against .3
    assert info["top2_margin"] == info["row_top2"][1]                            # the row that chose the final token
    assert dec["new_drafts"] == [3]                                              # uniform law, u = 0.9
    assert info["draft_margin"] == [pytest.approx(0.1, abs=1e-12)]
    assert info["draft_top2"] == [pytest.approx(0.0, abs=1e-12)]
    # reject: u = 0.65 >= 0.625; residual max(0, P0 - Q) = [0 .15 .075 .075] -> edges .5 .75 1; u = 0.55 -> token 2
    dec = orc.decide(Z, Q, 1, 1.0, [0.65, 0.55, 0.9])
    info = dec["info"]
    assert dec["n_accepted"] == 0 and dec["emitted"] == [2] and dec["new_drafts"] == []
    assert info["ratio_margin"] == [pytest.approx(0.025, abs=1e-12)]
    assert info["final_margin"] == pytest.approx(0.05, abs=1e-12)
    assert info["top2_margin"] == info["row_top2"][0]


def test_greedy_margins_are_per_row():
    Z = np.array([[0.0, 1.0, 0.995, -1.0],      # near tie (gap 0.005), argmax 1
                  [3.0, 0.0, 0.0, 0.0],         # clear
                  [0.0, 0.0, 2.0, 1.5]])        # look-ahead row, gap 0.5
    orc = _oracle([1])
    Q = po.softmax_T(np.array([0.0, 5.0, 0.0, 0.0]), 0.0)[None]
    dec = orc.decide(Z, Q, 1, 0.0, [0.0, 0.0, 0.0])
    assert dec["emitted"] == [1, 0] and dec["new_drafts"] == [2]
    info = dec["info"]
    assert info["row_top2"] == [pytest.approx(0.005), pytest.approx(3.0)]
    assert info["draft_top2"] == [pytest.approx(0.5)]


# --------------------------------------------------------------------------- first_difference / classify
def _dec(emitted, new_drafts, **info):
    return {"emitted": emitted, "new_drafts": new_drafts, "info": info}


def test_first_difference_names_the_decision():
    d = _dec([5, 6, 7], [1, 2])
    assert pu.first_difference(d, [5, 6, 7], [1, 2]) is None
    assert pu.first_difference(d, [5, 6, 9], [1, 2]) == ("final", 2)      # same accepts, other final token
    assert pu.first_difference(d, [5, 9], []) == ("accept", 1)             # the library rejected draft 2
    assert pu.first_difference(_dec([5, 9], []), [5, 6, 7], [1, 2]) == ("accept", 1)
    assert pu.first_difference(d, [5, 6, 7], [1, 3]) == ("draft", 1)
    assert pu.first_difference(d, [8], []) == ("accept", 0)


def test_classify_uses_the_margin_of_the_first_differing_decision_only():
    info = dict(ratio_margin=[0.5, 2e-4], final_margin=0.3, draft_margin=[0.2, 5e-5],
                row_top2=[4.0, 0.004, 2.0], draft_top2=[1.0, 0.003])
    d = _dec([5, 6, 7], [1, 2], **info)
    # sampled: accept test of draft 1 is far from its boundary, of draft 2 near
    assert pu.classify(d, [9], [], 1.0, 1e-4)[0] == "mismatch"
    assert pu.classify(d, [5, 9], [], 1.0, 1e-4)[0] == "excused"
    # final token: CDF distance 0.3 -> never excused, whatever other margins say
    assert pu.classify(d, [5, 6, 9], [1, 2], 1.0, 1e-4)[0] == "mismatch"
    # drafts: the second one is 5e-5 from an edge
    assert pu.classify(d, [5, 6, 7], [3, 2], 1.0, 1e-4)[0] == "mismatch"
    assert pu.classify(d, [5, 6, 7], [1, 3], 1.0, 1e-4)[0] == "excused"
    assert pu.classify(d, [5, 6, 7], [1, 3], 1.0, 1e-5)[0] == "mismatch"
    # greedy: the deciding row's own top-2 gap, not the smallest gap of the step
    assert pu.classify(d, [9], [], 0.0, 1e-4)[0] == "mismatch"              # row 0: gap 4.0
    assert pu.classify(d, [5, 9], [], 0.0, 1e-4)[0] == "excused"            # row 1: gap 0.004
    assert pu.classify(d, [5, 6, 9], [1, 2], 0.0, 1e-4)[0] == "mismatch"    # row 2: gap 2.0
    assert pu.classify(d, [5, 6, 7], [1, 3], 0.0, 1e-4)[0] == "excused"     # look-ahead row 2: gap 0.003
    assert pu.classify(d, [5, 6, 7], [1, 2], 0.0, 1e-4) == ("match", None)


def test_a_margin_helper_stuck_at_zero_or_infinity_would_be_noticed(monkeypatch):
    """The planted mistake lives on the CPU: with invcdf_margin forced to 0 the pins above no longer
    hold (here: one of them re-checked), and the harness's cap on excused steps bounds the damage."""
    monkeypatch.setattr(po, "invcdf_margin", lambda w, u: 0.0)
    assert po.invcdf_margin(np.array([1.0, 2.0, 1.0]), 0.5) != pytest.approx(0.25)
    assert pu.excuse_cap(3) == 0 and pu.excuse_cap(19) == 0 and pu.excuse_cap(20) == 1 and pu.excuse_cap(64) == 3
