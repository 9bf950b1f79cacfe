"""The look-ahead-embedding training step against its CPU oracle, through the C ABI (needs a B200).

Tolerances: both sides compute the same loss and the same gradient; the library carries activations as bf16
hi + lo pairs (about 16 significand bits) with fp32 accumulation and stores the look-ahead rows' keys and
values in a bf16 cache (2^-9 per element, which the float64 oracle does not do), so the logits agree to a few
1e-3 (the step's bound is 1e-2) and a gradient row to a few 1e-3 of its norm.  The loss is a mean of
lse(z) - z_target over as few as three rows, and moves by up to twice the largest logit error of a row, so its
bound is the logits' own, 1e-2 absolute (observed: up to 4e-3 with one sequence, below 1e-3 with batches);
gradient: 2e-2 relative L2 per look-ahead row.
"""
import dataclasses

import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import la_training_oracle as lo

pytestmark = pytest.mark.gpu

TINY_BF16 = dataclasses.replace(si.SHAPES["tiny"], dtype="bf16")
SEVENB_2L = dataclasses.replace(si.SHAPES["7b"], n_layers=2)


def _batch(shape, lengths, stride, seed=0):
    toks = np.zeros((len(lengths), stride), dtype=np.int32)
    for b in range(len(lengths)):
        toks[b] = si.make_prompt(shape, stride, seq=b + 10 * seed)
    return toks


def _rel_rows(a, b):
    return float(np.max(np.linalg.norm(a - b, axis=-1) / np.linalg.norm(b, axis=-1)))


def test_tiny_bf16_loss_and_gradient_match_the_oracle():
    import paper_2311_13581_b200 as pb
    w = si.make_weights(TINY_BF16, seed=1, std=0.05)
    L, pos = 3, [5, 12, 30]
    toks = _batch(TINY_BF16, pos, 48)
    ctx = pb.PassContext(TINY_BF16, si.weights_to(w, "cuda:0"), 3, 64)
    ctx.train_init(L, 3, warmup_steps=2, total_steps=20)
    loss = ctx.train_step(toks, pos, apply_update=False)
    grad = ctx.train_get(pb.PASS_TRAIN_GRAD).astype(np.float64)
    la0 = w["la_emb"][:L].double().numpy()
    assert np.array_equal(ctx.train_get(pb.PASS_TRAIN_LA).astype(np.float64), la0)      # no update was asked for
    want_loss, want_grad = lo.batch_loss_and_grad(TINY_BF16, w, [t.tolist() for t in toks], pos, la0)
    print(f"[training parity] tiny bf16 batch of 3: loss {loss:.5f} vs {want_loss:.5f}, gradient rows rel {_rel_rows(grad, want_grad):.3g}")
    assert abs(loss - want_loss) <= 1e-2, (loss, want_loss)
    assert _rel_rows(grad, want_grad) <= 2e-2, _rel_rows(grad, want_grad)
    # one sequence alone, the shortest possible prompt (a single token) and the longest the cache takes
    for p in ([0], [64 - 1 - L]):
        t1 = _batch(TINY_BF16, p, 70, seed=2)
        loss = ctx.train_step(t1, p, apply_update=False)
        grad = ctx.train_get(pb.PASS_TRAIN_GRAD).astype(np.float64)
        want_loss, want_grad = lo.batch_loss_and_grad(TINY_BF16, w, [t1[0].tolist()], p, la0)
        print(f"[training parity] tiny bf16, one sequence, n = {p[0]}: loss {loss:.5f} vs {want_loss:.5f}, gradient rows rel {_rel_rows(grad, want_grad):.3g}")
        assert abs(loss - want_loss) <= 1e-2, (p, loss, want_loss)
        assert _rel_rows(grad, want_grad) <= 2e-2, (p, _rel_rows(grad, want_grad))
    ctx.close()


def test_tiny_bf16_updates_follow_the_oracle_trainer():
    """Six AdamW updates under warm-up and cosine decay: losses and the learned rows against the oracle's
    trainer fed the same batches.  AdamW divides by the root of the second moment, so in the first updates
    every element moves by about the learning rate whatever the size of its gradient; an element whose
    gradient is within the arithmetic's error of zero may move the other way, hence the bound on the rows'
    CHANGE (5e-2 relative L2) rather than on single elements."""
    import paper_2311_13581_b200 as pb
    w = si.make_weights(TINY_BF16, seed=1, std=0.05)
    L, B = 4, 4
    ctx = pb.PassContext(TINY_BF16, si.weights_to(w, "cuda:0"), B, 64)
    hp = dict(lr=0.01, warmup_steps=3, total_steps=10)
    ctx.train_init(L, B, **hp)
    la0 = w["la_emb"][:L].double().numpy()
    tr = lo.LATrainer(TINY_BF16, w, la0, base_lr=0.01, warmup_steps=3, total_steps=10)
    rng = np.random.default_rng(0)
    for step in range(6):
        toks = _batch(TINY_BF16, [0] * B, 40, seed=step)
        pos = [int(x) for x in rng.integers(0, 40 - 2 - L, size=B)]
        loss = ctx.train_step(toks, pos)
        want_loss, _ = tr.step([t.tolist() for t in toks], pos)
        assert abs(loss - want_loss) <= 1e-2, (step, loss, want_loss)
    la = ctx.train_get(pb.PASS_TRAIN_LA).astype(np.float64)
    change, want_change = la - la0, tr.la - la0
    assert np.linalg.norm(want_change) > 1e-2
    assert np.linalg.norm(change - want_change) / np.linalg.norm(want_change) <= 5e-2
    # the trained rows, rounded to bf16, go into the table that steps read
    table = si.weights_to(w, "cuda:0")["la_emb"].clone()
    ctx.train_export(table)
    assert torch.equal(table[:L].cpu(), torch.from_numpy(la).to(torch.bfloat16))
    assert torch.equal(table[L:].cpu(), w["la_emb"][L:])
    ctx.close()


def test_7b_layer_shape_gradient_matches_the_oracle():
    """Two layers of the 7B layer shape, two sequences, prompts of 41 and 201 tokens (the second one goes
    through the large-chunk prompt path), four look-ahead rows."""
    import paper_2311_13581_b200 as pb
    shape = SEVENB_2L
    w = si.make_weights(shape, seed=0, device="cuda:0")
    w_cpu = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in w.items()}
    L, pos = 4, [40, 200]
    toks = _batch(shape, pos, 208)
    ctx = pb.PassContext(shape, w, 2, 256)
    ctx.train_init(L, 2)
    loss = ctx.train_step(toks, pos, apply_update=False)
    grad = ctx.train_get(pb.PASS_TRAIN_GRAD).astype(np.float64)
    la0 = w_cpu["la_emb"][:L].double().numpy()
    want_loss, want_grad = lo.batch_loss_and_grad(shape, w_cpu, [t.tolist() for t in toks], pos, la0)
    print(f"[training parity] 7B layer shape, 2 layers: loss {loss:.5f} vs {want_loss:.5f}, gradient rows rel {_rel_rows(grad, want_grad):.3g}")
    assert abs(loss - want_loss) <= 1e-2, (loss, want_loss)
    assert _rel_rows(grad, want_grad) <= 2e-2
    ctx.close()


def test_training_error_paths():
    import paper_2311_13581_b200 as pb
    w = si.make_weights(TINY_BF16, seed=1)
    ctx = pb.PassContext(TINY_BF16, si.weights_to(w, "cuda:0"), 2, 64)
    toks = _batch(TINY_BF16, [3, 3], 40)
    with pytest.raises(pb.PassError) as e:
        ctx.train_L = 2
        ctx.train_step(toks, [3, 3])                       # before pass_train_init
    assert e.value.code == -3
    with pytest.raises(pb.PassError):
        ctx.train_init(9, 2)                               # more rows than the look-ahead table has
    with pytest.raises(pb.PassError):
        ctx.train_init(2, 3)                               # more sequences than the context holds
    ctx.train_init(2, 2)
    with pytest.raises(pb.PassError) as e:
        ctx.train_step(toks, [38, 3])                      # targets beyond the sequence
    assert e.value.code == -1
    with pytest.raises(pb.PassError) as e:
        ctx.train_step(_batch(TINY_BF16, [0] * 3, 40), [1, 2, 3])      # more sequences than set up
    assert e.value.code == -2
    assert ctx.train_step(toks, [3, 9]) > 0.0
    ctx.close()
