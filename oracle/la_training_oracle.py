"""CPU oracle of the look-ahead-embedding training step.  TEST INFRASTRUCTURE ONLY.

Only tests, ``__graft_entry__.smoke()`` and the CPU-baseline legs of ``bench.py`` may import this module;
the CUDA library shares no code with it.

What it computes (Supplementary material, "Training details"; section "Look-ahead embeddings"):
the model is frozen, the only parameters are the L look-ahead input embeddings.  For a training
sequence w_0 .. w_{S-1} and a chosen position n, the model reads (w_0, .., w_n, LA_1, .., LA_L) in one
causal forward pass; the output at LA_t is the draft for the token t + 1 places after w_n (Algorithm 1:
the output at w_n is x_{n+1}, the output at LA_t is the draft of the place after it), so the loss is
the mean over t = 1..L of the cross entropy of that output against w_{n+1+t}, averaged over the
sequences of the batch.  The gradient is taken with respect to the look-ahead rows only and applied
with AdamW under a linear warm-up followed by a cosine decay.

Everything is float64 numpy with the forward written out as the definition and the backward as its
derivative, step by step; no blocking and no reuse of the structure the CUDA path exploits (it
differentiates only the look-ahead rows; here every row goes through the backward pass).
Pins: tests/test_oracle_training.py (central differences of the loss, torch autograd on a separate
transcription, torch.optim.AdamW, closed-form values of the schedule).
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np


def _f64(t) -> np.ndarray:
    return t.detach().cpu().double().numpy()


def rope_tables(shape, n_pos: int) -> Tuple[np.ndarray, np.ndarray]:
    """cos / sin of pos * theta^(-2i/d_head), [n_pos, d_head/2] (adjacent pairs rotate together)."""
    half = shape.d_head // 2
    inv = np.power(float(shape.rope_theta), -2.0 * np.arange(half) / shape.d_head)
    ang = np.arange(n_pos)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray, n_heads: int, transpose: bool = False) -> np.ndarray:
    """Rotate the pairs (2i, 2i+1) of every head of x [T, d]; transpose=True applies the inverse rotation,
    which is the derivative of the rotation (it is linear and orthogonal)."""
    T, d = x.shape
    v = x.reshape(T, n_heads, -1, 2)
    c, s = cos[:T, None, :], (-sin if transpose else sin)[:T, None, :]
    out = np.empty_like(v)
    out[..., 0] = v[..., 0] * c - v[..., 1] * s
    out[..., 1] = v[..., 1] * c + v[..., 0] * s
    return out.reshape(T, d)


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float):
    r = 1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return x * r * g, r


def rmsnorm_backward(dy: np.ndarray, x: np.ndarray, g: np.ndarray, r: np.ndarray) -> np.ndarray:
    """y = x r g with r = (mean x^2 + eps)^(-1/2): dx = r g dy - x r^3 mean(g dy x)."""
    u = dy * g
    return r * u - x * (r ** 3) * np.mean(u * x, axis=-1, keepdims=True)


def silu(x):
    return x / (1.0 + np.exp(-x))


def silu_grad(x):
    s = 1.0 / (1.0 + np.exp(-x))
    return s * (1.0 + x * (1.0 - s))


def forward(shape, weights: Dict[str, object], x: np.ndarray):
    """Causal forward of input rows x [T, d] at positions 0..T-1.  Returns (logits [T, V], tape)."""
    T, d = x.shape
    H, dh = shape.n_heads, shape.d_head
    cos, sin = rope_tables(shape, T)
    mask = np.tril(np.ones((T, T), dtype=bool))
    tape: List[dict] = []
    h = x.copy()
    for l in range(shape.n_layers):
        Wq, Wk, Wv, Wo = (_f64(weights[n][l]) for n in ("wq", "wk", "wv", "wo"))
        Wg, Wu, Wd = (_f64(weights[n][l]) for n in ("wg", "wu", "wd"))
        g1, g2 = _f64(weights["norm_attn"][l]), _f64(weights["norm_ffn"][l])
        a, r1 = rmsnorm(h, g1, shape.rms_eps)
        q = rope(a @ Wq.T, cos, sin, H)
        k = rope(a @ Wk.T, cos, sin, H)
        v = a @ Wv.T
        qh, kh, vh = (t.reshape(T, H, dh).transpose(1, 0, 2) for t in (q, k, v))
        S = qh @ kh.transpose(0, 2, 1) / math.sqrt(dh)
        S = np.where(mask[None], S, -np.inf)
        P = np.exp(S - S.max(axis=-1, keepdims=True))
        P /= P.sum(axis=-1, keepdims=True)
        attn = (P @ vh).transpose(1, 0, 2).reshape(T, d)
        h2 = h + attn @ Wo.T
        b, r2 = rmsnorm(h2, g2, shape.rms_eps)
        G, U = b @ Wg.T, b @ Wu.T
        act = silu(G) * U
        h3 = h2 + act @ Wd.T
        tape.append(dict(h=h, r1=r1, a=a, qh=qh, kh=kh, vh=vh, P=P, attn=attn, h2=h2, r2=r2, b=b, G=G, U=U, act=act))
        h = h3
    gf = _f64(weights["final_norm"])
    xf, rf = rmsnorm(h, gf, shape.rms_eps)
    logits = xf @ _f64(weights["lm_head"]).T
    return logits, dict(layers=tape, h_last=h, rf=rf, xf=xf, cos=cos, sin=sin)


def backward(shape, weights: Dict[str, object], tape: dict, dlogits: np.ndarray) -> np.ndarray:
    """Gradient of a scalar with respect to the input rows, given its gradient with respect to the logits."""
    T = dlogits.shape[0]
    H, dh, d = shape.n_heads, shape.d_head, shape.d_model
    gf = _f64(weights["final_norm"])
    dxf = dlogits @ _f64(weights["lm_head"])
    dh_ = rmsnorm_backward(dxf, tape["h_last"], gf, tape["rf"])
    for l in reversed(range(shape.n_layers)):
        t = tape["layers"][l]
        Wq, Wk, Wv, Wo = (_f64(weights[n][l]) for n in ("wq", "wk", "wv", "wo"))
        Wg, Wu, Wd = (_f64(weights[n][l]) for n in ("wg", "wu", "wd"))
        g1, g2 = _f64(weights["norm_attn"][l]), _f64(weights["norm_ffn"][l])
        dact = dh_ @ Wd
        dG = dact * t["U"] * silu_grad(t["G"])
        dU = dact * silu(t["G"])
        db = dG @ Wg + dU @ Wu
        dh2 = dh_ + rmsnorm_backward(db, t["h2"], g2, t["r2"])
        dattn = (dh2 @ Wo).reshape(T, H, dh).transpose(1, 0, 2)
        P, qh, kh, vh = t["P"], t["qh"], t["kh"], t["vh"]
        dP = dattn @ vh.transpose(0, 2, 1)
        dv = P.transpose(0, 2, 1) @ dattn
        dS = P * (dP - np.sum(dP * P, axis=-1, keepdims=True))
        dq = dS @ kh / math.sqrt(dh)
        dk = dS.transpose(0, 2, 1) @ qh / math.sqrt(dh)
        dq = rope(dq.transpose(1, 0, 2).reshape(T, d), tape["cos"], tape["sin"], H, transpose=True)
        dk = rope(dk.transpose(1, 0, 2).reshape(T, d), tape["cos"], tape["sin"], H, transpose=True)
        dv = dv.transpose(1, 0, 2).reshape(T, d)
        da = dq @ Wq + dk @ Wk + dv @ Wv
        dh_ = dh2 + rmsnorm_backward(da, t["h"], g1, t["r1"])
    return dh_


def sequence_loss_and_grad(shape, weights, tokens: Sequence[int], n: int, la: np.ndarray):
    """One sequence: rows (w_0..w_n, LA_1..LA_L); loss = mean_t CE(output at LA_t, w_{n+1+t}).
    Returns (loss, d loss / d la [L, d], logits of the look-ahead rows [L, V])."""
    L = la.shape[0]
    assert n >= 0 and n + 1 + L < len(tokens), "the sequence must hold the L targets after w_{n+1}"
    emb = _f64(weights["tok_emb"])
    x = np.concatenate([emb[[int(t) for t in tokens[:n + 1]]], np.asarray(la, dtype=np.float64)], axis=0)
    logits, tape = forward(shape, weights, x)
    Z = logits[n + 1:n + 1 + L]
    tgt = np.array([int(tokens[n + 1 + t]) for t in range(1, L + 1)])
    m = Z.max(axis=-1, keepdims=True)
    lse = m[:, 0] + np.log(np.sum(np.exp(Z - m), axis=-1))
    loss = float(np.mean(lse - Z[np.arange(L), tgt]))
    dZ = np.exp(Z - lse[:, None])
    dZ[np.arange(L), tgt] -= 1.0
    dlogits = np.zeros_like(logits)
    dlogits[n + 1:n + 1 + L] = dZ / L
    dx = backward(shape, weights, tape, dlogits)
    return loss, dx[n + 1:n + 1 + L], Z


def batch_loss_and_grad(shape, weights, batch_tokens: Sequence[Sequence[int]], positions: Sequence[int], la: np.ndarray):
    """Mean over the sequences of the batch."""
    B = len(batch_tokens)
    loss, grad = 0.0, np.zeros_like(np.asarray(la, dtype=np.float64))
    for toks, n in zip(batch_tokens, positions):
        l, g, _ = sequence_loss_and_grad(shape, weights, toks, n, la)
        loss += l / B
        grad += g / B
    return loss, grad


def lr_at(step: int, base_lr: float, warmup_steps: int, total_steps: int) -> float:
    """Learning rate of update number `step` (0-based): linear warm-up to base_lr over warmup_steps updates,
    then half a cosine from base_lr down to 0 at total_steps."""
    if warmup_steps > 0 and step < warmup_steps:
        return base_lr * (step + 1) / warmup_steps
    if step >= total_steps:
        return 0.0
    prog = (step - warmup_steps) / max(1, total_steps - warmup_steps)
    return 0.5 * base_lr * (1.0 + math.cos(math.pi * prog))


def adamw_update(p: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, t: int, lr: float,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.01):
    """AdamW (decoupled weight decay), update number t >= 1.  Returns (p, m, v) after the update."""
    p = p * (1.0 - lr * weight_decay)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mh = m / (1.0 - beta1 ** t)
    vh = v / (1.0 - beta2 ** t)
    return p - lr * mh / (np.sqrt(vh) + eps), m, v


class LATrainer:
    """State of the training: the look-ahead table (float64 here), AdamW moments, update count."""

    def __init__(self, shape, weights, la0: np.ndarray, base_lr=0.01, warmup_steps=2000, total_steps=10000,
                 beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01):
        self.shape, self.weights = shape, weights
        self.la = np.asarray(la0, dtype=np.float64).copy()
        self.m, self.v = np.zeros_like(self.la), np.zeros_like(self.la)
        self.t = 0
        self.hp = dict(base_lr=base_lr, warmup_steps=warmup_steps, total_steps=total_steps, beta1=beta1, beta2=beta2,
                       eps=eps, weight_decay=weight_decay)

    def step(self, batch_tokens, positions):
        loss, grad = batch_loss_and_grad(self.shape, self.weights, batch_tokens, positions, self.la)
        lr = lr_at(self.t, self.hp["base_lr"], self.hp["warmup_steps"], self.hp["total_steps"])
        self.t += 1
        self.la, self.m, self.v = adamw_update(self.la, grad, self.m, self.v, self.t, lr, self.hp["beta1"],
                                               self.hp["beta2"], self.hp["eps"], self.hp["weight_decay"])
        return loss, grad
