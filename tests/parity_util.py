"""Lockstep comparison of the CUDA library with the CPU oracle.

Both sides start every step from the same committed tokens, pending token and
drafts.  Compared per step:
  * logits of the live rows (max-abs for float32 models, per-row relative L2 for bf16);
  * level A: the oracle's decisions from its OWN logits against the library's, excusing
    steps the oracle flags as near a boundary (|P/Q - u| < 1e-3, top-2 logit margin
    < 1e-2 for greedy, CDF distance < cdf_tol for sampled tokens);
  * level B: the oracle's float64 verify replayed on the LIBRARY's float32 logits and the
    same uniforms - must agree exactly unless the CDF distance is < 1e-9.
Afterwards the oracle adopts the library's outcome, so one excused step cannot cascade.
"""
import numpy as np

import synthetic_inputs as si
from oracle import pass_oracle as po
import paper_2311_13581_b200 as pb


def logits_error(Zg, Zo, fp32):
    if fp32:
        return float(np.max(np.abs(Zg - Zo)))
    num = np.linalg.norm(Zg - Zo, axis=-1)
    den = np.linalg.norm(Zo, axis=-1)
    return float(np.max(num / den))


def lockstep(ctx, oracles, k, T, n_steps, seed=0, step0=0, cdf_tol_A=1e-4, check_A=True, top_k=0):
    B, V, M = ctx.B, ctx.vocab, 1 + 2 * k
    ctx.set_top_k(top_k)
    for orc in oracles:
        orc.top_k = top_k
    T = float(np.float32(T))            # the library takes the temperature as a C float
    fp32 = ctx.shape.dtype == "fp32"
    stats = {"steps": 0, "tokens": 0, "accepted": 0, "max_logit_err": 0.0, "A_excused": 0,
             "A_mismatch": 0, "B_excused": 0, "B_mismatch": 0, "multi_accept_steps": 0}
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
            if decB["emitted"] != g_em or decB["new_drafts"] != g_nd:
                info = decB["info"]
                margins = [info["final_margin"]] + list(info.get("draft_margin", []))
                if T > 0 and min(margins) < 1e-9:
                    stats["B_excused"] += 1
                else:
                    stats["B_mismatch"] += 1
            # level A: the oracle's own logits
            decA = orc.decide(Zo, orc.Q_dft, k, T, u[b])
            if decA["emitted"] != g_em or decA["new_drafts"] != g_nd:
                info = decA["info"]
                near = False
                if any(x < 1e-3 for x in info["ratio_margin"]):
                    near = True
                if T == 0:
                    srt = np.sort(Zo, axis=-1)
                    near |= bool(np.min(srt[:, -1] - srt[:, -2]) < 1e-2)
                else:
                    margins = [info["final_margin"]] + list(info.get("draft_margin", []))
                    near |= min(margins) < cdf_tol_A
                if near:
                    stats["A_excused"] += 1
                else:
                    stats["A_mismatch"] += 1
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
    if check_A:
        assert stats["A_mismatch"] == 0, stats
    assert stats["B_mismatch"] == 0, stats
    return stats, streams


def make_pair(shape, max_batch, kv_capacity, prompts, seed=0, weights=None, device="cuda:0"):
    """Weights generated once on the CPU, handed to both sides; prompt run on both."""
    w_cpu = weights if weights is not None else si.make_weights(shape, seed=seed)
    ctx = pb.PassContext(shape, si.weights_to(w_cpu, device), max_batch, kv_capacity, device=device)
    oracles = []
    for b, p in enumerate(prompts):
        ctx.prefill(b, p)
        be = po.TransformerBackend(shape, w_cpu, kv_capacity)
        oracles.append(po.PassOracle(be, p))
    return ctx, oracles, w_cpu
