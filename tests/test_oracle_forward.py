"""Pins of the oracle's decoder forward and of the schedules run on it.

What the paper fixes without any implementation to compare with:
  * a forward pass on n tokens equals n sequential single-token passes
    (Speculative Sampling, first paragraph);
  * greedy PaSS emits exactly the greedy auto-regressive stream (loss-less
    claim, Introduction / Parallel Speculative Sampling), for the one-call
    schedule and for Algorithm 1 as printed;
  * every model call adds at least one token; the two-call scheme gains at most
    (L + 2) / 2 (Parallel Speculative Sampling).
The single operations are pinned on closed forms and library routines.
"""
import math

import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import pass_oracle as po

TINY = si.SHAPES["tiny"]


@pytest.fixture(scope="module")
def tiny_weights():
    return si.make_weights(TINY, seed=0)


# ---------------------------------------------------------------- single operations
def test_linear_matches_library_matmul_fp32_and_bf16():
    rng = np.random.default_rng(0)
    W = rng.normal(size=(37, 53)).astype(np.float32)
    x = rng.normal(size=(5, 53))
    pc = po.Pieces(TINY, wdtype=0)
    np.testing.assert_allclose(pc.linear(W, x), x @ W.astype(np.float64).T, rtol=1e-12, atol=1e-12)
    Wb = torch.from_numpy(W).to(torch.bfloat16)
    bits = Wb.view(torch.int16).numpy().view(np.uint16)
    pcb = po.Pieces(TINY, wdtype=1)
    np.testing.assert_allclose(pcb.linear(bits, x), x @ Wb.double().numpy().T, rtol=1e-12, atol=1e-12)
    # operand order: a non-square W with a one-hot x picks a column of W
    e = np.zeros((1, 53))
    e[0, 7] = 1.0
    np.testing.assert_array_equal(pc.linear(W, e)[0], W[:, 7].astype(np.float64))


def test_linear_rows_are_independent_bitwise():
    rng = np.random.default_rng(1)
    W = rng.normal(size=(64, 300)).astype(np.float32)
    x = rng.normal(size=(9, 300))
    pc = po.Pieces(TINY)
    full = pc.linear(W, x)
    for r in range(9):
        np.testing.assert_array_equal(pc.linear(W, x[r:r + 1])[0], full[r])


def test_rmsnorm_closed_forms():
    pc = po.Pieces(TINY)
    d = TINY.d_model
    g = np.ones(d, dtype=np.float32)
    x = np.full((1, d), 2.0)
    np.testing.assert_allclose(pc.rmsnorm(g, x), 1.0, rtol=1e-6)   # constant vector -> gains
    rng = np.random.default_rng(2)
    x = rng.normal(size=(3, d)) * 5
    y = pc.rmsnorm(g, x)
    np.testing.assert_allclose((y ** 2).mean(axis=1), 1.0, rtol=1e-6)   # unit mean square
    np.testing.assert_allclose(pc.rmsnorm(g, 3.0 * x), y, rtol=1e-6)     # scale invariance
    g2 = rng.normal(size=d).astype(np.float32)
    np.testing.assert_allclose(pc.rmsnorm(g2, x), y * g2.astype(np.float64), rtol=1e-12)
    # eps matters for tiny inputs: x = 1e-3 -> x / sqrt(1e-6 + 1e-6)
    np.testing.assert_allclose(pc.rmsnorm(g, np.full((1, d), 1e-3)), 1e-3 / math.sqrt(2e-6),
                               rtol=1e-12)


def test_rope_known_values_and_group_properties():
    pc = po.Pieces(TINY)
    d, dh = TINY.d_model, TINY.d_head
    v = np.zeros(d)
    v[0] = 1.0                       # pair 0 of head 0: frequency 1
    r = pc.rope(v, 1)
    assert r[0] == pytest.approx(0.5403023058681398, abs=1e-15)    # cos 1
    assert r[1] == pytest.approx(0.8414709848078965, abs=1e-15)    # sin 1
    v = np.zeros(d)
    v[dh + dh - 2] = 1.0             # last pair of head 1: frequency theta^(-(dh-2)/dh)
    f = 1e4 ** (-(dh - 2) / dh)
    r = pc.rope(v, 1000)
    assert r[dh + dh - 2] == pytest.approx(math.cos(1000 * f), abs=1e-12)
    assert r[dh + dh - 1] == pytest.approx(math.sin(1000 * f), abs=1e-12)
    rng = np.random.default_rng(3)
    q, k = rng.normal(size=d), rng.normal(size=d)
    np.testing.assert_array_equal(pc.rope(q, 0), q)                                  # identity at 0
    np.testing.assert_allclose(pc.rope(pc.rope(q, 5), 12), pc.rope(q, 17), atol=1e-12)  # additive
    np.testing.assert_allclose(np.linalg.norm(pc.rope(q, 99)), np.linalg.norm(q), rtol=1e-13)
    # scores depend on the position difference only
    a = pc.rope(q, 40) @ pc.rope(k, 33)
    b = pc.rope(q, 1007) @ pc.rope(k, 1000)
    assert a == pytest.approx(b, abs=1e-10)


def test_swiglu_known_values():
    pc = po.Pieces(TINY)
    g = np.array([0.0, 1.0, -1.0, 40.0, -40.0])
    u = np.array([3.0, 2.0, 2.0, 1.0, 1.0])
    out = pc.swiglu(g, u)
    sig1 = 0.7310585786300049        # 1 / (1 + e^-1)
    np.testing.assert_allclose(out, [0.0, 2 * sig1, -2 * (1 - sig1), 40.0, -40.0 * math.exp(-40.0)],
                               rtol=1e-13, atol=1e-300)


def test_attention_closed_forms_and_library():
    from scipy.special import softmax
    pc = po.Pieces(TINY)
    d, H, dh = TINY.d_model, TINY.n_heads, TINY.d_head
    rng = np.random.default_rng(4)
    n_ctx, n_rows = 11, 3
    kc = rng.normal(size=(n_ctx + n_rows, d))
    vc = rng.normal(size=(n_ctx + n_rows, d))
    # q = 0: uniform weights over the causal window -> running mean of V
    o = pc.attention(np.zeros((n_rows, d)), kc, vc, n_ctx)
    for r in range(n_rows):
        np.testing.assert_allclose(o[r], vc[:n_ctx + r + 1].mean(axis=0), rtol=1e-12, atol=1e-14)
    # a single key: the output is that value
    o = pc.attention(rng.normal(size=(1, d)), kc, vc, 0)
    np.testing.assert_allclose(o[0], vc[0], rtol=1e-13)
    # general case against scipy softmax per head
    q = rng.normal(size=(n_rows, d))
    o = pc.attention(q, kc, vc, n_ctx)
    for r in range(n_rows):
        n = n_ctx + r + 1
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            w = softmax(kc[:n, sl] @ q[r, sl] / math.sqrt(dh))
            np.testing.assert_allclose(o[r, sl], w @ vc[:n, sl], rtol=1e-11, atol=1e-13)


# ---------------------------------------------------------------- whole forward
def _torch_forward(shape, w, x, pos0, kc, vc, store=lambda t: t):
    """float64 transcription with library matmul / softmax (a cross-check, all rows at once)."""
    W = lambda t: t.double()
    d, H, dh = shape.d_model, shape.n_heads, shape.d_head
    h = torch.from_numpy(x).clone()
    n = h.shape[0]
    pos = torch.arange(pos0, pos0 + n, dtype=torch.float64)
    inv = shape.rope_theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = pos[:, None] * inv[None]
    rot = torch.polar(torch.ones_like(ang), ang)          # e^{i pos f}

    def rope(t):
        c = torch.view_as_complex(t.reshape(n, H, dh // 2, 2).contiguous())
        return torch.view_as_real(c * rot[:, None]).reshape(n, d)

    def norm(t, g):
        return t * torch.rsqrt((t * t).mean(-1, keepdim=True) + shape.rms_eps) * W(g)

    for l in range(shape.n_layers):
        a = norm(h, w["norm_attn"][l])
        q, k, v = rope(a @ W(w["wq"][l]).T), rope(a @ W(w["wk"][l]).T), a @ W(w["wv"][l]).T
        kc[l][pos0:pos0 + n], vc[l][pos0:pos0 + n] = store(k), store(v)
        K = kc[l][:pos0 + n].reshape(-1, H, dh).transpose(0, 1)
        V = vc[l][:pos0 + n].reshape(-1, H, dh).transpose(0, 1)
        s = q.reshape(n, H, dh).transpose(0, 1) @ K.transpose(1, 2) / math.sqrt(dh)
        mask = torch.arange(pos0 + n)[None, :] > (pos0 + torch.arange(n))[:, None]
        s = s.masked_fill(mask[None], float("-inf"))
        o = (torch.softmax(s, -1) @ V).transpose(0, 1).reshape(n, d)
        h = h + o @ W(w["wo"][l]).T
        b = norm(h, w["norm_ffn"][l])
        h = h + (torch.nn.functional.silu(b @ W(w["wg"][l]).T) * (b @ W(w["wu"][l]).T)) @ W(w["wd"][l]).T
    return (norm(h, w["final_norm"]) @ W(w["lm_head"]).T).numpy()


def test_forward_against_torch_float64_transcription(tiny_weights):
    be = po.TransformerBackend(TINY, tiny_weights, 64)
    prompt = si.make_prompt(TINY, 20)
    rows = [("tok", t) for t in prompt[:17]]
    z0 = be.forward(rows, 0)
    rows2 = [("tok", prompt[17]), ("tok", prompt[18]), ("la", 0), ("la", 1), ("la", 2)]
    z1 = be.forward(rows2, 17)
    kc = torch.zeros(TINY.n_layers, 64, TINY.d_model, dtype=torch.float64)
    vc = torch.zeros_like(kc)
    t0 = _torch_forward(TINY, tiny_weights, be.embed(rows), 0, kc, vc)
    t1 = _torch_forward(TINY, tiny_weights, be.embed(rows2), 17, kc, vc)
    np.testing.assert_allclose(z0, t0, rtol=0, atol=1e-11)
    np.testing.assert_allclose(z1, t1, rtol=0, atol=1e-11)
    assert np.abs(z1).max() > 0.1                    # not a vacuous comparison


def _nearest_bf16(t):
    """bfloat16 has 8 significant bits: x = m 2^e with m in [0.5, 1) -> rint(256 m) 2^(e-8), ties to even."""
    m, e = np.frexp(t.numpy())
    return torch.from_numpy(np.ldexp(np.rint(m * 256.0), e - 8))


def test_bf16_cache_stores_rounded_rows_and_attention_reads_them(tiny_weights):
    prompt = si.make_prompt(TINY, 20)
    rows = [("tok", t) for t in prompt[:17]]
    rows2 = [("tok", prompt[17]), ("tok", prompt[18]), ("la", 0), ("la", 1), ("la", 2)]
    be = po.TransformerBackend(TINY, tiny_weights, 64, kv_dtype="bf16")
    ref = po.TransformerBackend(TINY, tiny_weights, 64)
    z0, z1 = be.forward(rows, 0), be.forward(rows2, 17)
    r0, r1 = ref.forward(rows, 0), ref.forward(rows2, 17)
    # what is stored is representable in 8 significant bits, and is the nearest such value: layer 0 sees
    # the same input in both backends, so its rows are the unrounded ones, rounded
    for c, cr in ((be.k, ref.k), (be.v, ref.v)):
        t = torch.from_numpy(c[:, :22])
        assert torch.equal(t.to(torch.bfloat16).double(), t)
        assert torch.equal(torch.from_numpy(c[0, :22]), _nearest_bf16(torch.from_numpy(cr[0, :22])))
        assert np.all(np.abs(c[0, :22] - cr[0, :22]) <= 2.0 ** -8 * np.abs(cr[0, :22]))   # half a step: 2^-9 x / m, m >= 1/2
    assert _nearest_bf16(torch.tensor([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -0.75, 0.0],
                                      dtype=torch.float64)).tolist() == [1.0, 1.0 + 2.0 ** -6, -0.75, 0.0]
    # the forward with that cache, transcribed
    kc = torch.zeros(TINY.n_layers, 64, TINY.d_model, dtype=torch.float64)
    vc = torch.zeros_like(kc)
    t0 = _torch_forward(TINY, tiny_weights, be.embed(rows), 0, kc, vc, store=_nearest_bf16)
    t1 = _torch_forward(TINY, tiny_weights, be.embed(rows2), 17, kc, vc, store=_nearest_bf16)
    np.testing.assert_allclose(z0, t0, rtol=0, atol=1e-11)
    np.testing.assert_allclose(z1, t1, rtol=0, atol=1e-11)
    # and it is a different computation from the unrounded one, by about the format's step
    err = np.linalg.norm(z1 - r1) / np.linalg.norm(r1)
    assert 1e-5 < err < 1e-2, err


def test_forward_reduces_to_head_of_embedding_when_blocks_are_zero():
    """Wo = 0 and Wd = 0: logits = rmsnorm(embedding) Wlm^T (residual plumbing)."""
    w = si.make_weights(TINY, seed=3)
    for l in range(TINY.n_layers):
        w["wo"][l].zero_()
        w["wd"][l].zero_()
    be = po.TransformerBackend(TINY, w, 16)
    rows = [("tok", 5), ("la", 1), ("tok", 900)]
    z = be.forward(rows, 0)
    x = be.embed(rows)
    xn = x / np.sqrt((x * x).mean(-1, keepdims=True) + TINY.rms_eps)
    np.testing.assert_allclose(z, xn @ w["lm_head"].double().numpy().T, rtol=1e-12, atol=1e-13)


def test_multi_token_forward_equals_sequential_single_token_forwards(tiny_weights):
    prompt = si.make_prompt(TINY, 12)
    rows = [("tok", t) for t in prompt] + [("la", 0), ("la", 1)]
    be1 = po.TransformerBackend(TINY, tiny_weights, 32)
    z_all = be1.forward(rows, 0)
    be2 = po.TransformerBackend(TINY, tiny_weights, 32)
    for i, row in enumerate(rows):
        z_i = be2.forward([row], i)
        np.testing.assert_array_equal(z_i[0], z_all[i])      # bit for bit
    np.testing.assert_array_equal(be1.k, be2.k)
    # split 5 + 9 rows, and a rollback that overwrites the tail
    be3 = po.TransformerBackend(TINY, tiny_weights, 32)
    be3.forward(rows[:5], 0)
    be3.forward([("tok", 1), ("tok", 2), ("tok", 3)], 5)      # to be rolled back
    z_b = be3.forward(rows[5:], 5)
    np.testing.assert_array_equal(z_b, z_all[5:])


# ---------------------------------------------------------------- schedules on the transformer
def _greedy_reference(weights, prompt, n):
    be = po.TransformerBackend(TINY, weights, len(prompt) + n + 24)
    return po.autoregressive(be, prompt, 0.0, n, lambda i: 0.0)[0]


@pytest.mark.parametrize("k", [1, 2, 4])
def test_greedy_pass_equals_greedy_autoregressive(tiny_weights, k):
    prompt = si.make_prompt(TINY, 32)
    G = 64 if k == 2 else 24
    ar = _greedy_reference(tiny_weights, prompt, G)
    be = po.TransformerBackend(TINY, tiny_weights, len(prompt) + G + 24)
    orc = po.PassOracle(be, prompt)
    out, steps = [], 0
    while len(out) < G:
        before = orc.len
        e, a, info = orc.step(k, 0.0, [0.0] * (2 * k + 1))
        steps += 1
        assert len(e) == a + 1 and 1 <= len(e) <= k + 1       # >= 1 token per call
        assert orc.len == before + len(e)
        out += e
    assert out[:G] == ar
    be2 = po.TransformerBackend(TINY, tiny_weights, len(prompt) + G + 24)
    out2, calls = po.alg1_two_call(be2, prompt, k, 0.0, G, lambda it, n: np.zeros(n))
    assert out2[:G] == ar
    assert len(out2) <= calls * (k + 2) / 2                    # speed-up ceiling (L+2)/2
    assert len(out2) >= calls                                  # at least one token per call


def test_greedy_accepts_when_lookahead_rows_predict_the_future():
    """With look-ahead rows built so that drafts are right, several tokens per call come out,
    and the stream still equals the auto-regressive one."""
    # Identity-like toy: zero blocks, so logits depend on the row's own embedding only.
    w = si.make_weights(TINY, seed=5)
    for l in range(TINY.n_layers):
        w["wo"][l].zero_()
        w["wd"][l].zero_()
    prompt = [3, 4]
    ar = _greedy_reference(w, prompt, 6)
    # the stream is a fixed chain t -> next(t); make LA_j's embedding equal to the embedding of
    # the token that is j steps ahead of prompt[-1]... only valid for the first call, enough here
    chain = [prompt[-1]] + ar
    for j in range(3):
        w["la_emb"][j] = w["tok_emb"][chain[j + 1]]
    be = po.TransformerBackend(TINY, w, 32)
    orc = po.PassOracle(be, prompt)
    e1, a1, _ = orc.step(3, 0.0, [0.0] * 7)
    assert e1 == ar[:1] and orc.drafts == ar[1:4]              # drafts predict tokens 2..4
    e2, a2, _ = orc.step(3, 0.0, [0.0] * 7)
    assert a2 == 3 and e2 == ar[1:5]                           # all accepted + one extra token


def test_sampled_pass_with_temperature_runs_and_keeps_invariants(tiny_weights):
    prompt = si.make_prompt(TINY, 32)
    be = po.TransformerBackend(TINY, tiny_weights, 32 + 64 + 24)
    orc = po.PassOracle(be, prompt)
    n, accepted = 0, 0
    for step in range(30):
        u = si.step_uniforms(0, 0, step, 5).numpy()
        e, a, info = orc.step(2, 1.0, u)
        assert len(e) == a + 1 and 1 <= len(e) <= 3
        assert all(0 <= t < TINY.vocab for t in e)
        n += len(e)
        accepted += a
    assert accepted > 0          # flat random-init laws: some drafts do get accepted at T = 1
