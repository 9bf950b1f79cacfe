"""Lockstep comparison of the CUDA library with the CPU oracle.

Both sides start every step from the same committed tokens, pending token and
drafts.  Compared per step:
  * logits of the live rows (max-abs for float32 models, per-row relative L2 for bf16);
  * level A: the oracle's decisions from its OWN logits against the library's.  A step that
    differs is excused only if the FIRST decision that differs sits near its boundary on the
    oracle's side: an accept test with |P/Q - u| < 1e-3, an argmax (greedy) whose row has a
    top-2 logit gap < 1e-2, a sampled token with CDF distance < cdf_tol;
  * level B: the oracle's float64 verify replayed on the LIBRARY's float32 logits and the
    same uniforms - must agree exactly unless the CDF distance is < 1e-9.
Excused steps are counted, printed, and capped (see `lockstep`).  Afterwards the oracle
adopts the library's outcome, so one excused step cannot cascade.
"""
import math

import numpy as np

import synthetic_inputs as si
from oracle import pass_oracle as po

RATIO_TOL = 1e-3        # |P_tgt/Q_dft - u| below which an accept test counts as near its boundary
TOP2_TOL = 1e-2         # top-2 logit gap below which an argmax counts as near a tie
REPORT = []             # one line per lockstep run, printed at the end of the test session


def logits_error(Zg, Zo, fp32):
    if fp32:
        return float(np.max(np.abs(Zg - Zo)))
    num = np.linalg.norm(Zg - Zo, axis=-1)
    den = np.linalg.norm(Zo, axis=-1)
    return float(np.max(num / den))


def first_difference(dec, g_emitted, g_drafts):
    """Which decision of a step differs first between the oracle's outcome `dec` and the library's.

    Returns None (same outcome) or (kind, index): ("accept", j) the accept test of draft j+1,
    ("final", a) the final token after a accepted drafts, ("draft", t) new draft t.
    Emitted tokens are the accepted drafts followed by the final token, and both sides hold the
    same drafts, so position i of the two lists can differ only if at least one side ended there.
    """
    eo, eg = list(dec["emitted"]), list(g_emitted)
    n = min(len(eo), len(eg))
    for i in range(n):
        if eo[i] != eg[i]:
            if len(eo) == len(eg) == i + 1:
                return ("final", i)
            return ("accept", i)
    if len(eo) != len(eg):
        return ("accept", n - 1)
    do, dg = list(dec["new_drafts"]), list(g_drafts)
    if do != dg:
        if len(do) != len(dg):
            return ("draft", 0)
        return ("draft", next(t for t in range(len(do)) if do[t] != dg[t]))
    return None


def decision_margin(dec, diff, T):
    """Distance of the oracle's decision `diff` from its boundary, and the tolerance it is held
    against: (margin, kind) with kind in {"ratio", "top2", "cdf"}."""
    info = dec["info"]
    kind, i = diff
    if T == 0:
        if kind == "draft":
            return float(info["draft_top2"][i]) if "draft_top2" in info else math.inf, "top2"
        return float(info["row_top2"][i]), "top2"
    if kind == "accept":
        return (float(info["ratio_margin"][i]) if i < len(info["ratio_margin"]) else math.inf), "ratio"
    if kind == "final":
        return float(info["final_margin"]), "cdf"
    return (float(info["draft_margin"][i]) if "draft_margin" in info else math.inf), "cdf"


def classify(dec, g_emitted, g_drafts, T, cdf_tol):
    """"match", "excused" or "mismatch" for one step and one sequence."""
    diff = first_difference(dec, g_emitted, g_drafts)
    if diff is None:
        return "match", None
    margin, kind = decision_margin(dec, diff, T)
    tol = {"ratio": RATIO_TOL, "top2": TOP2_TOL, "cdf": cdf_tol}[kind]
    return ("excused" if margin < tol else "mismatch"), (diff, kind, margin)


def excuse_cap(decisions):
    """At most 5 % of the compared (step, sequence) pairs may be excused at level A."""
    return int(math.floor(0.05 * decisions))


def lockstep(ctx, oracles, k, T, n_steps, seed=0, step0=0, cdf_tol_A=1e-4, check_A=True, top_k=0,
             max_excused_A=None, label=""):
    import paper_2311_13581_b200 as pb
    B, V, M = ctx.B, ctx.vocab, 1 + 2 * k
    ctx.set_top_k(top_k)
    for orc in oracles:
        orc.top_k = top_k
    T = float(np.float32(T))            # the library takes the temperature as a C float
    fp32 = ctx.shape.dtype == "fp32"
    stats = {"steps": 0, "tokens": 0, "accepted": 0, "max_logit_err": 0.0, "A_excused": 0,
             "A_mismatch": 0, "B_excused": 0, "B_mismatch": 0, "multi_accept_steps": 0, "details": []}
    prev_la = getattr(ctx, "_prev_la", [None] * B)
    streams = [[] for _ in range(B)]
    for step in range(step0, step0 + n_steps):
        u = np.stack([si.step_uniforms(seed, b, step, 2 * k + 1).numpy() for b in range(B)])
        emitted, n_out = ctx.step(k, T, None if T == 0 else u)
        Zg_all = ctx.get_debug(pb.PASS_DBG_LOGITS, rows=B * M).reshape(B, M, V)
        m_after = ctx.get_debug(pb.PASS_DBG_N_DRAFT)
        d_after = ctx.get_debug(pb.PASS_DBG_DRAFTS)
        lens = ctx.get_debug(pb.PASS_DBG_KV_LEN)
        n_acc = ctx.get_debug(pb.PASS_DBG_N_ACCEPTED)
        for b, orc in enumerate(oracles):
            Zo = orc.forward_step(k, T)
            m = len(orc.drafts)
            live = 1 + m + k
            Zg = Zg_all[b, :live].astype(np.float64)
            err = logits_error(Zg, Zo, fp32)
            stats["max_logit_err"] = max(stats["max_logit_err"], err)
            g_em = emitted[b]
            g_nd = [int(x) for x in d_after[b][:m_after[b]]]
            assert 1 <= len(g_em) <= k + 1 and len(g_em) == n_out[b] == n_acc[b] + 1
            # level B: float64 verify on the library's own logits
            if m:
                Qg = np.stack([po.softmax_T(prev_la[b][t], T, top_k) for t in range(m)])
            else:
                Qg = np.zeros((0, V))
            decB = orc.decide(Zg, Qg, k, T, u[b])
            verdict, why = classify(decB, g_em, g_nd, T, 1e-9)
            if verdict != "match" and why[1] != "cdf":
                verdict = "mismatch"            # same logits on both sides: only a CDF edge may round apart
            if verdict != "match":
                stats["B_" + verdict] += 1
                stats["details"].append(("B", step, b) + why)
            # level A: the oracle's own logits
            decA = orc.decide(Zo, orc.Q_dft, k, T, u[b])
            verdict, why = classify(decA, g_em, g_nd, T, cdf_tol_A)
            if verdict != "match":
                stats["A_" + verdict] += 1
                stats["details"].append(("A", step, b) + why)
            # adopt the library's outcome
            Qn = np.stack([po.softmax_T(Zo[m + 1 + t], T, top_k) for t in range(k)]) if g_nd else np.zeros((0, V))
            orc.commit(g_em, g_nd, Qn)
            if g_nd:
                prev_la[b] = Zg[m + 1:m + 1 + k].copy()
            assert orc.len == lens[b], (orc.len, lens[b])
            streams[b] += g_em
            stats["tokens"] += len(g_em)
            stats["accepted"] += len(g_em) - 1
            stats["multi_accept_steps"] += int(len(g_em) > 1)
        stats["steps"] += 1
    ctx._prev_la = prev_la
    decisions = stats["steps"] * B
    cap = excuse_cap(decisions) if max_excused_A is None else max_excused_A
    line = (f"{label or ctx.shape.dtype} k={k} T={T:g} top_k={top_k} steps={stats['steps']} B={B}: "
            f"max_logit_err={stats['max_logit_err']:.3g} A_excused={stats['A_excused']}/{decisions} "
            f"(cap {cap if check_A else 'n/a'}) A_mismatch={stats['A_mismatch']} B_excused={stats['B_excused']} "
            f"B_mismatch={stats['B_mismatch']} multi_accept_steps={stats['multi_accept_steps']}")
    print("[parity] " + line)
    REPORT.append(line)
    if check_A:
        assert stats["A_mismatch"] == 0, stats
        assert stats["A_excused"] <= cap, stats
    assert stats["B_mismatch"] == 0, stats
    assert stats["B_excused"] == 0, stats
    return stats, streams


def make_pair(shape, max_batch, kv_capacity, prompts, seed=0, weights=None, device="cuda:0"):
    """Weights generated once on the CPU, handed to both sides; prompt run on both."""
    import paper_2311_13581_b200 as pb
    w_cpu = weights if weights is not None else si.make_weights(shape, seed=seed)
    ctx = pb.PassContext(shape, si.weights_to(w_cpu, device), max_batch, kv_capacity, device=device)
    oracles = []
    for b, p in enumerate(prompts):
        ctx.prefill(b, p)
        be = po.TransformerBackend(shape, w_cpu, kv_capacity)
        oracles.append(po.PassOracle(be, p))
    return ctx, oracles, w_cpu
