"""The seeded input generator: determinism, ranges and first moments."""
import numpy as np
import torch

import synthetic_inputs as si


def test_hash_is_counter_based_and_deterministic():
    a = si.hash_u64(0, 5, 0, 100)
    b = si.hash_u64(0, 5, 40, 10)
    assert torch.equal(a[40:50], b)
    assert not torch.equal(si.hash_u64(1, 5, 0, 100), a)
    assert not torch.equal(si.hash_u64(0, 6, 0, 100), a)
    assert a.unique().numel() == 100


def test_uniforms_are_24_bit_in_unit_interval():
    u = si.uniforms(0, 9, 0, 200000)
    assert u.dtype == torch.float32 and float(u.min()) >= 0.0 and float(u.max()) < 1.0
    assert torch.equal(u * 16777216.0, torch.round(u * 16777216.0))
    assert abs(float(u.double().mean()) - 0.5) < 5e-3
    hist = torch.histc(u, bins=10, min=0, max=1) / u.numel()
    assert float((hist - 0.1).abs().max()) < 5e-3


def test_normals_have_the_requested_moments():
    z = si.normal(0, 3, 400000, 0.02)
    assert abs(float(z.mean())) < 2e-4
    assert abs(float(z.std()) - 0.02) < 2e-4
    assert abs(float(((z / 0.02) ** 4).mean()) - 3.0) < 0.1


def test_weights_shapes_dtypes_and_prompt():
    sh = si.SHAPES["tiny"]
    w = si.make_weights(sh, seed=0)
    assert w["tok_emb"].shape == (1024, 256) and w["tok_emb"].dtype == torch.float32
    assert w["la_emb"].shape == (sh.k_max, 256)
    assert len(w["wq"]) == 2 and w["wg"][0].shape == (688, 256) and w["wd"][1].shape == (256, 688)
    assert torch.equal(w["norm_attn"][0], torch.ones(256))
    w2 = si.make_weights(sh, seed=0)
    assert torch.equal(w["wd"][1], w2["wd"][1])
    assert not torch.equal(w["wq"][0], w["wk"][0])
    p = si.make_prompt(sh, 32)
    assert len(p) == 32 and all(0 <= t < 1024 for t in p) and len(set(p)) > 20
    assert si.make_prompt(sh, 32, seq=1) != p
    u = si.step_uniforms(0, 0, 3, 5)
    assert u.shape == (5,) and torch.equal(u, si.step_uniforms(0, 0, 3, 5))
