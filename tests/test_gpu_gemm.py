"""The tensor-core weight-streaming GEMM on its own, through the C ABI (needs a B200)."""
import dataclasses

import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import pass_oracle as po

pytestmark = pytest.mark.gpu

# d_model multiple of 128; d_ffn and vocab deliberately NOT multiples of 64 / 128 (ragged tiles)
MID = si.ModelShape(2, 512, 4, 128, 1384, 2000, k_max=8, dtype="bf16")
TINY_BF16 = dataclasses.replace(si.SHAPES["tiny"], dtype="bf16")
NAMES = ["wq", "wk", "wv", "wo", "wg", "wu", "wd", "lm_head"]


def _ctx(shape, seed=2):
    import paper_2311_13581_b200 as pb
    w = si.make_weights(shape, seed=seed)
    return pb.PassContext(shape, si.weights_to(w, "cuda:0"), 1, 64), w


def _weight(w, which, layer):
    return w["lm_head"] if which == 7 else w[NAMES[which]][layer]


@pytest.mark.parametrize("shape", [TINY_BF16, MID], ids=["tiny", "mid"])
@pytest.mark.parametrize("R", [1, 9, 17, 72, 128])
def test_linear_matches_float64_matmul(shape, R):
    ctx, w = _ctx(shape)
    g = torch.Generator().manual_seed(R)
    for which in range(8):
        layer = 1 if which != 7 else 0
        W = _weight(w, which, layer)
        x = torch.randn(R, W.shape[1], generator=g, dtype=torch.float32)
        y = ctx.debug_linear(which, layer, x.cuda()).cpu().double()
        ref = x.double() @ W.double().T
        rel = (y - ref).norm(dim=1) / ref.norm(dim=1)
        assert float(rel.max()) < 1e-4, (NAMES[which], R, float(rel.max()))
    ctx.close()


def test_gate_up_interleaved_layout():
    ctx, w = _ctx(MID)
    f = MID.d_ffn
    x = torch.randn(9, MID.d_model, generator=torch.Generator().manual_seed(5))
    y = ctx.debug_linear(8, 0, x.cuda()).cpu().double()
    nt = (f + 63) // 64
    y = y.view(9, nt, 2, 64)
    gate = y[:, :, 0, :].reshape(9, nt * 64)[:, :f]
    up = y[:, :, 1, :].reshape(9, nt * 64)[:, :f]
    rg = x.double() @ w["wg"][0].double().T
    ru = x.double() @ w["wu"][0].double().T
    assert float(((gate - rg).norm(dim=1) / rg.norm(dim=1)).max()) < 1e-4
    assert float(((up - ru).norm(dim=1) / ru.norm(dim=1)).max()) < 1e-4
    ctx.close()


def test_linear_against_oracle_piece_and_determinism():
    ctx, w = _ctx(MID)
    x = torch.randn(17, MID.d_ffn, generator=torch.Generator().manual_seed(6))
    y1 = ctx.debug_linear(6, 0, x.cuda())
    y2 = ctx.debug_linear(6, 0, x.cuda())
    assert torch.equal(y1, y2)                       # split-K partials are summed in a fixed order
    bits = w["wd"][0].view(torch.int16).numpy().view(np.uint16)
    ref = po.Pieces(MID, wdtype=1).linear(bits, x.double().numpy())
    err = np.linalg.norm(y1.cpu().double().numpy() - ref, axis=1) / np.linalg.norm(ref, axis=1)
    assert err.max() < 1e-4
    ctx.close()
