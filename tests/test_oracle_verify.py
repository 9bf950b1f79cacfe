"""Pins of the oracle's sampling rule and schedules against what the paper fixes.

The paper states that the rejection scheme leaves the output distributed exactly
as the target model (Introduction; Speculative Sampling; Parallel Speculative
Sampling: "guaranteeing the same loss-less quality").  On a toy vocabulary this
is checked by exact enumeration with rational arithmetic, through the oracle's
own code path.  No expected value here comes from any implementation.
"""
import itertools
from fractions import Fraction as F

import numpy as np
import pytest

from oracle import pass_oracle as po


def lattice(n):
    return [(i + 0.5) / n for i in range(n)]


# ---------------------------------------------------------------- invcdf / softmax
def test_invcdf_interval_lengths_equal_probabilities():
    w = np.array([1, 0, 3, 2, 0, 2]) / 8.0
    counts = np.zeros(6, dtype=int)
    prev = -1
    for u in lattice(64):
        i = po.invcdf(w, u)
        assert i >= prev          # monotone in u
        prev = i
        counts[i] += 1
    assert counts.tolist() == [8, 0, 24, 16, 0, 16]


def test_invcdf_edges():
    w = np.array([0.0, 0.0, 0.25, 0.75, 0.0])
    assert po.invcdf(w, 0.0) == 2            # first index with mass
    assert po.invcdf(w, 0.25) == 3           # "sum > u*total" is strict
    assert po.invcdf(w, np.nextafter(1.0, 0.0)) == 3
    assert po.invcdf(w * 7.0, 0.2) == 2      # unnormalised weights are fine


def test_softmax_T_against_library_and_limits():
    from scipy.special import softmax
    rng = np.random.default_rng(0)
    z = rng.normal(size=50)
    for T in (1.0, 0.8, 0.2):
        np.testing.assert_allclose(po.softmax_T(z, T), softmax(z / T), rtol=1e-13, atol=0)
    z[7] = z[31] = z.max() + 1.0             # tie: lowest index wins at T = 0
    p0 = po.softmax_T(z, 0.0)
    assert p0[7] == 1.0 and p0.sum() == 1.0
    assert np.argmax(po.softmax_T(z, 1e-3)) in (7, 31)


# ---------------------------------------------------------------- verify: closed forms
P8 = [F(1, 4), F(1, 4), F(1, 8), F(1, 8), F(1, 8), F(1, 16), F(1, 32), F(1, 32)]
Q8 = [F(1, 2), F(1, 4), F(1, 8), F(1, 8), F(0), F(0), F(0), F(0)]


def _np(v):
    return np.array([float(x) for x in v])


def test_verify_single_draft_exact_law_dyadic_lattice():
    """Vocabulary 8, dyadic laws: the output of one draft + verify has law P exactly."""
    N = 64
    P, Q = _np(P8), _np(Q8)
    law = [F(0)] * 8
    acc = F(0)
    for d in range(8):
        if Q8[d] == 0:
            continue
        for ua, uf in itertools.product(lattice(N), lattice(N)):
            a, y, _ = po.verify(np.stack([P, P]), Q[None], [d], [ua], uf)
            out = d if a == 1 else y
            law[out] += Q8[d] * F(1, N * N)
            if a == 1:
                acc += Q8[d] * F(1, N * N)
    assert law == P8
    # acceptance probability = sum min(P, Q) = 1 - TV(P, Q)
    assert acc == sum(min(p, q) for p, q in zip(P8, Q8))
    assert acc == 1 - sum(abs(p - q) for p, q in zip(P8, Q8)) / 2


def _exact_law_single(Pf, Qf):
    """Exact output law for arbitrary rational P, Q by integrating over cells.

    For a fixed draft d the outcome is piecewise constant in (u_accept, u_final);
    the break points are the acceptance ratio and the edges of the final law's
    CDF.  One evaluation at each cell's midpoint, weighted by the cell's exact area.
    """
    V = len(Pf)
    P, Q = _np(Pf), _np(Qf)
    law = [F(0)] * V
    for d in range(V):
        if Qf[d] == 0:
            continue
        ratio = min(F(1), Pf[d] / Qf[d])
        # accepted part
        if ratio > 0:
            a, y, _ = po.verify(np.stack([P, P]), Q[None], [d], [float(ratio) / 2], 0.5)
            assert a == 1
            law[d] += Qf[d] * ratio
        if ratio < 1:
            res = [max(F(0), p - q) for p, q in zip(Pf, Qf)]
            tot = sum(res)
            edges = [F(0)]
            for r in res:
                edges.append(edges[-1] + r / tot)
            for i in range(V):
                lo, hi = edges[i], edges[i + 1]
                if hi == lo:
                    continue
                a, y, _ = po.verify(np.stack([P, P]), Q[None], [d],
                                    [float((ratio + 1) / 2)], float((lo + hi) / 2))
                assert a == 0
                law[y] += Qf[d] * (1 - ratio) * (hi - lo)
    return law


def test_verify_single_draft_exact_law_random_rationals():
    rng = np.random.default_rng(1)
    for _ in range(20):
        V = 6
        p = rng.integers(0, 9, size=V)
        q = rng.integers(0, 9, size=V)
        p[rng.integers(V)] += 1
        q[rng.integers(V)] += 1
        Pf = [F(int(x), int(p.sum())) for x in p]
        Qf = [F(int(x), int(q.sum())) for x in q]
        assert _exact_law_single(Pf, Qf) == Pf


def test_verify_special_cases():
    P = _np(P8)
    # Q == P: every draft is accepted whatever u < 1, final token from P_tgt[m]
    for d in range(8):
        for u in (0.0, 0.5, np.nextafter(1.0, 0.0)):
            a, y, _ = po.verify(np.stack([P, P]), P[None], [d], [u], 0.3)
            assert a == 1 and y == po.invcdf(P, 0.3)
    # Q one-hot on a token the target gives no mass: always rejected, residual law is P
    Pz = P.copy()
    Pz[3] += Pz[0]
    Pz[0] = 0.0
    Q = np.zeros(8)
    Q[0] = 1.0
    for uf in lattice(32):
        a, y, info = po.verify(np.stack([Pz, Pz]), Q[None], [0], [0.0], uf)
        assert a == 0 and y == po.invcdf(Pz, uf)
    # strictness: ratio exactly 1/2, u = 1/2 is a rejection
    a, _, _ = po.verify(np.stack([P, P]), _np(Q8)[None], [0], [0.5], 0.1)
    assert a == 0
    a, _, _ = po.verify(np.stack([P, P]), _np(Q8)[None], [0], [np.nextafter(0.5, 0)], 0.1)
    assert a == 1


def test_verify_stops_at_first_rejection_and_uses_matching_rows():
    """Three drafts; target rows differ, so a wrong row index shows."""
    V = 4
    P = np.array([[0.1, 0.2, 0.3, 0.4], [0.4, 0.3, 0.2, 0.1], [0.25, 0.25, 0.25, 0.25],
                  [0.7, 0.1, 0.1, 0.1]])
    Q = np.array([[0.4, 0.3, 0.2, 0.1], [0.1, 0.2, 0.3, 0.4], [0.25, 0.25, 0.25, 0.25]])
    drafts = [0, 3, 1]
    # draft 1: ratio 0.25; draft 2: ratio 0.25; draft 3: ratio 1
    a, y, info = po.verify(P, Q, drafts, [0.2, 0.2, 0.99], 0.5)
    assert a == 3 and y == po.invcdf(P[3], 0.5)
    a, y, info = po.verify(P, Q, drafts, [0.2, 0.3, 0.0], 0.5)
    assert a == 1
    resid = np.maximum(0, P[1] - Q[1])
    assert y == po.invcdf(resid, 0.5)
    np.testing.assert_allclose(info["final_law"], resid)
    a, y, _ = po.verify(P, Q, drafts, [0.26, 0.0, 0.0], 0.9)
    assert a == 0 and y == po.invcdf(np.maximum(0, P[0] - Q[0]), 0.9)


# ---------------------------------------------------------------- schedules on a table model
# prob[j][t]: law of the row that follows real token t and j look-ahead rows.
TGT = [[F(1, 4), F(1, 4), F(1, 4), F(1, 4)],
       [F(1, 2), F(1, 4), F(1, 8), F(1, 8)],
       [F(0), F(1, 2), F(1, 4), F(1, 4)],
       [F(1, 2), F(0), F(1, 2), F(0)]]
DFT = [[F(1, 2), F(1, 4), F(1, 8), F(1, 8)]] * 4


def _table(k):
    prob = np.zeros((k + 1, 4, 4))
    for t in range(4):
        prob[0][t] = _np(TGT[t])
        for j in range(1, k + 1):
            prob[j][t] = _np(DFT[t])
    return prob


def _true_pair_law(first):
    return {(a, b): first[a] * TGT[a][b] for a in range(4) for b in range(4)}


def test_fused_schedule_two_token_law_exact():
    """k = 1: the first two emitted tokens have law P(x1) P(x2 | x1), exactly."""
    N = 8
    prob = _table(1)
    first = TGT[2]                      # prompt ends with token 2
    law = {}
    for u1y, u1d, u2a, u2f in itertools.product(lattice(N), repeat=4):
        orc = po.PassOracle(po.TableBackend(prob), [1, 2])
        e1, a1, _ = orc.step(1, 1.0, [0.0, u1y, u1d])
        assert a1 == 0 and len(e1) == 1          # drafting call: one token (Alg. 1)
        e2, a2, _ = orc.step(1, 1.0, [u2a, u2f, 0.0])
        assert len(e2) == a2 + 1 and 1 <= len(e2) <= 2
        key = (e1[0], e2[0])
        law[key] = law.get(key, F(0)) + F(1, N ** 4)
    want = {k: v for k, v in _true_pair_law(first).items() if v}
    assert law == want


def test_two_call_algorithm1_two_token_law_exact():
    N = 8
    prob = _table(1)
    first = TGT[2]
    law = {}
    for us in itertools.product(lattice(N), repeat=4):
        out, calls = po.alg1_two_call(po.TableBackend(prob), [1, 2], 1, 1.0, 2,
                                      lambda it, n: np.array(us))
        assert calls == 2 and 2 <= len(out) <= 3     # at least one token per call
        key = (out[0], out[1])
        law[key] = law.get(key, F(0)) + F(1, N ** 4)
    want = {k: v for k, v in _true_pair_law(first).items() if v}
    assert law == want


def test_fused_schedule_three_token_law_monte_carlo_k2():
    """k = 2 exercises chained accepts; 3-token law within 5 sigma of the product law."""
    rng = np.random.default_rng(7)
    prob = _table(2)
    # make the second look-ahead law differ from the first
    for t in range(4):
        prob[2][t] = np.array([0.125, 0.125, 0.25, 0.5])
    n_run = 6000
    counts = {}
    for _ in range(n_run):
        orc = po.PassOracle(po.TableBackend(prob), [3, 1])
        toks = []
        while len(toks) < 3:
            e, a, info = orc.step(2, 1.0, rng.random(5))
            assert len(e) == a + 1 and 1 <= len(e) <= 3
            toks += e
        key = tuple(toks[:3])
        counts[key] = counts.get(key, 0) + 1
    for a in range(4):
        for b in range(4):
            for c in range(4):
                p = float(TGT[1][a] * TGT[a][b] * TGT[b][c])
                got = counts.get((a, b, c), 0) / n_run
                sigma = np.sqrt(max(p * (1 - p), 1e-9) / n_run)
                assert abs(got - p) <= 5 * sigma + 1e-12, ((a, b, c), got, p)


def test_changing_k_or_temperature_drops_pending_drafts():
    prob = _table(2)
    orc = po.PassOracle(po.TableBackend(prob), [1, 2])
    orc.step(2, 1.0, [0.1] * 5)
    assert len(orc.drafts) == 2
    e, a, info = orc.step(1, 1.0, [0.1] * 3)
    assert info["m"] == 0 and a == 0 and len(e) == 1
    assert len(orc.drafts) == 1
    e, a, info = orc.step(1, 0.5, [0.1] * 3)
    assert info["m"] == 0


# ---------------------------------------------------------------- top-k sampling (Experiments, setup)
def test_top_k_law_against_library_and_special_cases():
    from scipy.special import softmax
    rng = np.random.default_rng(3)
    z = rng.normal(size=50)
    z[11] = z[40] = z[5]                      # a three-way tie somewhere in the row
    for T in (1.0, 0.8, 0.2):
        for k in (1, 2, 10, 49):
            idx = np.argsort(-z, kind="stable")[:k]          # library sort; stable = lower index first
            want = np.zeros(50)
            want[idx] = softmax(z[idx] / T)
            got = po.softmax_T(z, T, k)
            np.testing.assert_allclose(got, want, rtol=1e-13, atol=0)
            assert np.count_nonzero(got) == k and abs(got.sum() - 1.0) < 1e-15
            assert set(po.top_k_set(z, k).tolist()) == set(idx.tolist())
    # k >= V and k = 0: no filter; k = 1: the greedy law
    np.testing.assert_array_equal(po.softmax_T(z, 0.7, 50), po.softmax_T(z, 0.7))
    np.testing.assert_array_equal(po.softmax_T(z, 0.7, 0), po.softmax_T(z, 0.7))
    np.testing.assert_array_equal(po.softmax_T(z, 0.7, 1), po.softmax_T(z, 0.0))
    # a tie across the cut: the lower index stays
    t = np.array([1.0, 3.0, 3.0, 3.0, 0.0])
    assert po.top_k_set(t, 2).tolist() == [1, 2]
    np.testing.assert_allclose(po.softmax_T(t, 1.0, 2), [0, 0.5, 0.5, 0, 0], rtol=1e-15)
    # greedy is untouched by the filter
    np.testing.assert_array_equal(po.softmax_T(z, 0.0, 3), po.softmax_T(z, 0.0))


# laws whose two largest entries renormalise to dyadic numbers, so that a lattice enumerates them exactly
TGT_K = [[F(9, 16), F(3, 16), F(1, 8), F(1, 8)],      # top-2 -> [3/4, 1/4, 0, 0]
         [F(1, 8), F(3, 8), F(3, 8), F(1, 8)],        #       -> [0, 1/2, 1/2, 0]
         [F(1, 8), F(1, 8), F(3, 16), F(9, 16)],      #       -> [0, 0, 1/4, 3/4]
         [F(3, 8), F(1, 8), F(1, 8), F(3, 8)]]        #       -> [1/2, 0, 0, 1/2]
DFT_K = [F(3, 8), F(3, 8), F(1, 8), F(1, 8)]          #       -> [1/2, 1/2, 0, 0]


def _filtered(row, k):
    keep = sorted(range(len(row)), key=lambda i: (-row[i], i))[:k]
    tot = sum(row[i] for i in keep)
    return [row[i] / tot if i in keep else F(0) for i in range(len(row))]


def test_fused_schedule_with_top_k_emits_the_filtered_target_law_exactly():
    """Top-2 sampling on vocabulary 4, k = 1 look-ahead: the first two emitted tokens follow
    P_2(x1) P_2(x2 | x1) with P_2 the top-2 renormalised target law - the filter is applied to
    target and look-ahead rows alike, and the rejection scheme stays exact for the filtered law."""
    N = 8
    prob = np.zeros((2, 4, 4))
    for t in range(4):
        prob[0][t] = _np(TGT_K[t])
        prob[1][t] = _np(DFT_K)
    assert _filtered(TGT_K[0], 2) == [F(3, 4), F(1, 4), F(0), F(0)]
    assert _filtered(DFT_K, 2) == [F(1, 2), F(1, 2), F(0), F(0)]
    first = _filtered(TGT_K[2], 2)
    want = {}
    for a in range(4):
        for b in range(4):
            v = first[a] * _filtered(TGT_K[a], 2)[b]
            if v:
                want[(a, b)] = v
    law = {}
    n_two = 0
    for u1y, u1d, u2a, u2f in itertools.product(lattice(N), repeat=4):
        orc = po.PassOracle(po.TableBackend(prob), [1, 2])
        e1, a1, _ = orc.step(1, 1.0, [0.0, u1y, u1d], top_k=2)
        assert a1 == 0 and len(e1) == 1
        assert orc.drafts[0] in (0, 1)                       # drafts come from the filtered draft law
        e2, a2, _ = orc.step(1, 1.0, [u2a, u2f, 0.0])
        n_two += len(e2) == 2
        key = (e1[0], e2[0])
        law[key] = law.get(key, F(0)) + F(1, N ** 4)
    assert law == want
    assert n_two > 0
    # the unfiltered law is a different one
    assert want != {k: v for k, v in {(a, b): TGT_K[2][a] * TGT_K[a][b] for a in range(4) for b in range(4)}.items() if v}


def test_changing_top_k_drops_pending_drafts():
    prob = _table(2)
    orc = po.PassOracle(po.TableBackend(prob), [1, 2])
    orc.step(2, 1.0, [0.1] * 5, top_k=3)
    assert len(orc.drafts) == 2
    e, a, info = orc.step(2, 1.0, [0.1] * 5, top_k=2)
    assert info["m"] == 0 and a == 0 and len(e) == 1
    e, a, info = orc.step(2, 1.0, [0.1] * 5)                 # top_k stays 2: drafts are used
    assert info["m"] == 2
