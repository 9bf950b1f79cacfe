"""The long-cache attention kernel (scores on tcgen05, Section 3's one model call over a long cache) against the
oracle: whole PaSS steps in lockstep, on caches cut at and around its 128-key blocks, with ragged batches,
with slices that hold no key at all, and with its bounded waits made to run out."""
import dataclasses

import numpy as np
import pytest

import synthetic_inputs as si
from oracle import pass_oracle as po

pytestmark = pytest.mark.gpu

# d_head 128 (what the kernel is written for), everything else small: 4 heads, 2 layers
SMALL_DH128 = si.ModelShape(2, 512, 4, 128, 1408, 1024, k_max=8, dtype="bf16")


def _pair(shape, B, ctx_len, cap, lens, kv_dtype="f64"):
    import paper_2311_13581_b200 as pb
    w = si.make_weights(shape, seed=3, device="cuda:0")
    w_cpu = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in w.items()}
    ctx = pb.PassContext(shape, w, B, cap)
    bes = [po.TransformerBackend(shape, w_cpu, cap, kv_dtype=kv_dtype) for _ in range(B)]
    orcs = []
    for b, be in enumerate(bes):
        for layer in range(shape.n_layers):
            k, v = si.make_kv(shape, layer, ctx_len, seq=b)
            ctx.set_kv(b, layer, 0, k, v)
            be.k[layer, :ctx_len] = k.double().numpy()
            be.v[layer, :ctx_len] = v.double().numpy()
        ctx.set_state(b, lens[b], 5 + b)
        orc = po.PassOracle.__new__(po.PassOracle)
        orc.be, orc.len, orc.pending, orc.drafts = be, lens[b], 5 + b, []
        orc.Q_dft, orc.k_prev, orc.T_prev, orc.last_logits = np.zeros((0, shape.vocab)), None, None, None
        orcs.append(orc)
    return ctx, orcs


@pytest.mark.parametrize("k,length", [(4, 119), (4, 120), (4, 118), (0, 127), (0, 128), (1, 381), (7, 1009), (4, 1300),
                                      (2, 6)])
def test_small_model_every_step_through_the_long_cache_kernel(k, length):
    """1 + 2k rows on a cache of `length` positions, chosen so that the keys end exactly on a block of 128,
    one short of it, one past it; a cache shorter than one block (most of the 16 slices are empty); 15 rows
    (k = 7, the most the kernel takes); one row (k = 0)."""
    import paper_2311_13581_b200 as pb
    from parity_util import lockstep
    ctx, orcs = _pair(SMALL_DH128, 1, length, length + 80, [length])
    ctx.debug_set(pb.PASS_HOOK_ATTN_LONG_FROM, 0)
    stats, _ = lockstep(ctx, orcs, k, 0.8, 4, check_A=False, label=f"long-cache kernel len={length}")
    assert stats["max_logit_err"] <= 1e-2, stats
    stats, _ = lockstep(ctx, orcs, k, 0.0, 2, step0=4, check_A=True, label=f"long-cache kernel len={length} greedy")
    assert stats["max_logit_err"] <= 1e-2, stats
    ctx.close()


def test_ragged_batch_through_the_long_cache_kernel():
    """Three sequences of different lengths in one step: each has its own slices, mask and merge."""
    import paper_2311_13581_b200 as pb
    from parity_util import lockstep
    lens = [700, 333, 1025]
    ctx, orcs = _pair(SMALL_DH128, 3, 1025, 1100, lens)
    ctx.debug_set(pb.PASS_HOOK_ATTN_LONG_FROM, 0)
    stats, _ = lockstep(ctx, orcs, 4, 1.0, 4, check_A=False, label="long-cache kernel B=3")
    assert stats["max_logit_err"] <= 1e-2, stats
    assert sorted(ctx.get_debug(pb.PASS_DBG_KV_LEN).tolist()) != sorted(lens)      # the caches grew
    ctx.close()


def test_13b_layer_shape_long_cache_without_any_hook():
    """40 heads (3 slices each), 3700 cached positions: past the default threshold, so this is the path a
    user gets."""
    from parity_util import lockstep
    shape = dataclasses.replace(si.SHAPES["13b"], n_layers=1)
    ctx, orcs = _pair(shape, 1, 3700, 3800, [3700])
    stats, _ = lockstep(ctx, orcs, 4, 1.0, 3, check_A=False, label="13B-1L ctx3700")
    assert stats["max_logit_err"] <= 1e-2, stats
    ctx.close()


def test_long_cache_kernel_gives_up_cleanly_when_its_scores_never_arrive():
    """The kernel's waits are bounded: with the announcement of the scores withheld they run out, the step
    returns the time-out error with the sequence state as it was, and the steps after it are right again
    (the slice counters and the status word are scrubbed)."""
    import paper_2311_13581_b200 as pb
    from parity_util import lockstep
    ctx, orcs = _pair(SMALL_DH128, 1, 600, 700, [600])
    ctx.debug_set(pb.PASS_HOOK_ATTN_LONG_FROM, 0)
    stats, _ = lockstep(ctx, orcs, 4, 0.0, 2)
    len_before = ctx.get_debug(pb.PASS_DBG_KV_LEN).copy()
    ctx.debug_set(pb.PASS_HOOK_ATTN_STUCK, 1)
    with pytest.raises(pb.PassError) as e:
        ctx.step(4, 0.0, None)
    assert "timed out" in str(e.value)
    ctx.debug_set(pb.PASS_HOOK_ATTN_STUCK, 0)
    assert (ctx.get_debug(pb.PASS_DBG_KV_LEN) == len_before).all()
    stats, _ = lockstep(ctx, orcs, 4, 0.0, 3, step0=2)
    assert stats["max_logit_err"] <= 1e-2, stats
    ctx.close()
