"""Pins for the CPU oracle of the look-ahead-embedding training step (oracle/la_training_oracle.py).

The oracle's gradient is a hand-written backward pass, so it is held against things that are not itself:
central differences of its own loss (the definition of a derivative), the forward of the other,
independently written decoder oracle (C, float64), torch autograd on a separate transcription built
from library operations, torch.optim.AdamW, and closed-form values of the learning-rate schedule.
"""
import math

import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import la_training_oracle as lo
from oracle import pass_oracle as po

SMALL = si.ModelShape(2, 128, 2, 64, 344, 300, k_max=4, dtype="fp32")


@pytest.fixture(scope="module")
def setup():
    w = si.make_weights(SMALL, seed=3, std=0.08)         # larger than 0.02 so that attention and SwiGLU are far from linear
    toks = si.make_prompt(SMALL, 24, seq=5)
    la = _la0(w, 3)
    return w, toks, la


def _la0(w, L, seed=0):
    rng = np.random.default_rng(seed)
    return w["tok_emb"][:L].double().numpy() + 0.05 * rng.standard_normal((L, SMALL.d_model))


def test_forward_agrees_with_the_decoder_oracle(setup):
    w, toks, la = setup
    n = 11
    _, _, Z = lo.sequence_loss_and_grad(SMALL, w, toks, n, la)
    w2 = dict(w)
    w2["la_emb"] = torch.zeros(SMALL.k_max, SMALL.d_model)
    w2["la_emb"][:3] = torch.from_numpy(la).float()
    # float32 storage of the look-ahead rows on that side: compare with the same rounded rows
    _, _, Z32 = lo.sequence_loss_and_grad(SMALL, w, toks, n, w2["la_emb"][:3].double().numpy())
    be = po.TransformerBackend(SMALL, w2, 64)
    Zc = be.forward([("tok", t) for t in toks[:n + 1]] + [("la", i) for i in range(3)], 0)[n + 1:]
    assert np.max(np.abs(Zc - Z32)) < 1e-10
    assert np.max(np.abs(Z)) > 0.05


def test_gradient_matches_central_differences(setup):
    w, toks, la = setup
    n = 9
    loss, grad, _ = lo.sequence_loss_and_grad(SMALL, w, toks, n, la)
    assert loss > 1.0 and np.linalg.norm(grad) > 1e-4
    rng = np.random.default_rng(1)
    eps = 1e-5
    for _ in range(14):
        t, j = int(rng.integers(0, 3)), int(rng.integers(0, SMALL.d_model))
        lp, lm = la.copy(), la.copy()
        lp[t, j] += eps
        lm[t, j] -= eps
        fd = (lo.sequence_loss_and_grad(SMALL, w, toks, n, lp)[0] - lo.sequence_loss_and_grad(SMALL, w, toks, n, lm)[0]) / (2 * eps)
        assert abs(fd - grad[t, j]) <= 1e-6 * max(1.0, abs(fd)) + 2e-9, (t, j, fd, grad[t, j])


def _torch_loss(w, toks, n, la_t):
    """The same model written with torch operations (float64), for autograd."""
    s = SMALL
    dd = lambda t: t.double()
    x = torch.cat([dd(w["tok_emb"])[toks[:n + 1]], la_t], dim=0)
    T = x.shape[0]
    half = s.d_head // 2
    inv = torch.pow(torch.tensor(float(s.rope_theta), dtype=torch.float64), -2.0 * torch.arange(half, dtype=torch.float64) / s.d_head)
    ang = torch.arange(T, dtype=torch.float64)[:, None] * inv[None]
    rot = torch.polar(torch.ones_like(ang), ang)                       # e^{i angle}

    def rope(v):
        c = torch.view_as_complex(v.reshape(T, s.n_heads, half, 2).contiguous())
        return torch.view_as_real(c * rot[:, None, :]).reshape(T, s.d_model)

    def norm(v, g):
        return v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + s.rms_eps) * dd(g)

    h = x
    for l in range(s.n_layers):
        a = norm(h, w["norm_attn"][l])
        q, k, v = rope(a @ dd(w["wq"][l]).T), rope(a @ dd(w["wk"][l]).T), a @ dd(w["wv"][l]).T
        sp = lambda t: t.reshape(T, s.n_heads, s.d_head).transpose(0, 1)
        o = torch.nn.functional.scaled_dot_product_attention(sp(q), sp(k), sp(v), is_causal=True)
        h = h + o.transpose(0, 1).reshape(T, s.d_model) @ dd(w["wo"][l]).T
        b = norm(h, w["norm_ffn"][l])
        h = h + (torch.nn.functional.silu(b @ dd(w["wg"][l]).T) * (b @ dd(w["wu"][l]).T)) @ dd(w["wd"][l]).T
    logits = norm(h, w["final_norm"]) @ dd(w["lm_head"]).T
    L = la_t.shape[0]
    tgt = torch.tensor([toks[n + 1 + t] for t in range(1, L + 1)])
    return torch.nn.functional.cross_entropy(logits[n + 1:n + 1 + L], tgt)


def test_gradient_matches_torch_autograd(setup):
    w, toks, la = setup
    for n in (0, 7, 19):
        la_t = torch.tensor(la, dtype=torch.float64, requires_grad=True)
        loss_t = _torch_loss(w, toks, n, la_t)
        loss_t.backward()
        loss, grad, _ = lo.sequence_loss_and_grad(SMALL, w, toks, n, la)
        assert abs(loss - float(loss_t)) < 1e-10
        assert np.max(np.abs(grad - la_t.grad.numpy())) < 1e-10 * max(1.0, float(la_t.grad.abs().max()))


def test_targets_are_the_tokens_after_the_next_one(setup):
    """The output at LA_t drafts the token t + 1 places after w_n: a model whose target is moved by one
    place has another loss, and the loss does not look at w_{n+1} at all."""
    w, toks, la = setup
    n = 6
    base = lo.sequence_loss_and_grad(SMALL, w, toks, n, la)[0]
    t2 = list(toks)
    t2[n + 1] = (t2[n + 1] + 1) % SMALL.vocab
    assert lo.sequence_loss_and_grad(SMALL, w, t2, n, la)[0] == base
    t3 = list(toks)
    t3[n + 2] = (t3[n + 2] + 1) % SMALL.vocab
    assert lo.sequence_loss_and_grad(SMALL, w, t3, n, la)[0] != base
    with pytest.raises(AssertionError):
        lo.sequence_loss_and_grad(SMALL, w, toks, len(toks) - 4, la)      # the last target would lie beyond the sequence


def test_batch_is_the_mean_over_sequences(setup):
    w, toks, la = setup
    seqs = [si.make_prompt(SMALL, 20, seq=b) for b in range(3)]
    pos = [4, 9, 13]
    loss, grad = lo.batch_loss_and_grad(SMALL, w, seqs, pos, la)
    parts = [lo.sequence_loss_and_grad(SMALL, w, s, n, la) for s, n in zip(seqs, pos)]
    assert loss == pytest.approx(np.mean([p[0] for p in parts]), rel=1e-13)
    assert np.allclose(grad, np.mean([p[1] for p in parts], axis=0), rtol=1e-13, atol=0)


def test_adamw_matches_the_library_optimizer():
    rng = np.random.default_rng(4)
    p0 = rng.standard_normal((3, 16))
    pt = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([pt], lr=0.01, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    p, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
    for t in range(1, 8):
        g = rng.standard_normal(p0.shape)
        lr = 0.01 * t / 7
        for grp in opt.param_groups:
            grp["lr"] = lr
        pt.grad = torch.tensor(g)
        opt.step()
        p, m, v = lo.adamw_update(p, g, m, v, t, lr)
        assert np.max(np.abs(p - pt.detach().numpy())) < 1e-14


def test_learning_rate_schedule_closed_forms():
    base, wu, tot = 0.01, 2000, 10000            # the paper's values
    assert lo.lr_at(0, base, wu, tot) == pytest.approx(base / wu)
    assert lo.lr_at(wu - 1, base, wu, tot) == pytest.approx(base)
    assert lo.lr_at(wu, base, wu, tot) == pytest.approx(base)
    assert lo.lr_at((wu + tot) // 2, base, wu, tot) == pytest.approx(base / 2)
    assert lo.lr_at(wu + (tot - wu) // 4, base, wu, tot) == pytest.approx(base * (1 + math.sqrt(0.5)) / 2)
    assert lo.lr_at(tot, base, wu, tot) == 0.0
    assert all(lo.lr_at(s, base, wu, tot) >= lo.lr_at(s + 1, base, wu, tot) for s in range(wu, tot, 97))


def test_trainer_lowers_the_loss_on_a_fixed_batch(setup):
    w, toks, la = setup
    seqs = [si.make_prompt(SMALL, 20, seq=b) for b in range(2)]
    tr = lo.LATrainer(SMALL, w, la, base_lr=0.02, warmup_steps=2, total_steps=40)
    losses = [tr.step(seqs, [5, 8])[0] for _ in range(12)]
    assert losses[-1] < losses[0] - 0.05
    assert tr.t == 12
