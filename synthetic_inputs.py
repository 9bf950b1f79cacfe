"""Seeded synthetic inputs for the PaSS decoder step: weights, prompts, uniforms.

This module holds no arithmetic of the method itself. It only turns
(seed, stream id, element index) into numbers, so that the CPU oracle and the
CUDA path can be fed the very same tensors. It stands in for the paper's
trained LLaMA-7B weights and its Wikipedia / The Stack prompts (Experiments,
"Data"), none of which ship with this repository: only shapes carry over.

Generator: a counter-based hash. The 64-bit counter
``seed * C_SEED + stream * C_STREAM + index`` is passed through the SplitMix64
finaliser (Steele, Lea, Flood 2014).  Normals are Box-Muller in float64 on two
hashes per element; uniforms keep the top 24 bits so that they are exact in
float32 and lie in [0, 1).

Everything is written with torch integer ops so it runs on CPU or on a CUDA
device alike; a given run generates each tensor once and hands copies of that
one tensor to both sides.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List

import torch

_C_SEED = -7046029254386353131      # 0x9E3779B97F4A7C15 as int64
_C_STREAM = -4658895280553007687    # 0xBF58476D1CE4E5B9 as int64
_M1 = -4658895280553007687          # 0xBF58476D1CE4E5B9
_M2 = -7723592293110705685          # 0x94D049BB133111EB


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _wrap64(v: int) -> int:
    v &= (1 << 64) - 1
    return v - (1 << 64) if v >= (1 << 63) else v


def hash_u64(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """Hash of counters start..start+count-1 of one stream (int64 bit patterns)."""
    base = _wrap64(seed * (_C_SEED & ((1 << 64) - 1)) + stream * (_C_STREAM & ((1 << 64) - 1)))
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix64(idx + base)


def uniforms(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """float32 uniforms in [0,1): top 24 bits of the hash times 2^-24."""
    h = hash_u64(seed, stream, start, count, device)
    return (_lsr(h, 40).to(torch.float32)) * (1.0 / 16777216.0)


def normal(seed: int, stream: int, count: int, std: float, device="cpu",
           chunk: int = 1 << 25) -> torch.Tensor:
    """float64 N(0, std) by Box-Muller; element i uses counters 2i and 2i+1."""
    out = torch.empty(count, dtype=torch.float64, device=device)
    for s in range(0, count, chunk):
        n = min(chunk, count - s)
        h = hash_u64(seed, stream, 2 * s, 2 * n, device).view(n, 2)
        u1 = (_lsr(h[:, 0], 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)
        u2 = (_lsr(h[:, 1], 11).to(torch.float64)) * (1.0 / 9007199254740992.0)
        out[s:s + n] = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2) * std
    return out


def token_ids(seed: int, stream: int, count: int, vocab: int, device="cpu") -> torch.Tensor:
    """int32 ids uniform on [0, vocab)."""
    h = _lsr(hash_u64(seed, stream, 0, count, device), 33)   # 31 bits
    return (h % vocab).to(torch.int32)


# ---------------------------------------------------------------------------
# Model shapes (the paper's "7B LLaMa" re-implementation and neighbours)
# ---------------------------------------------------------------------------

@dataclasses.dataclass
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    d_head: int
    d_ffn: int
    vocab: int
    k_max: int = 8            # rows in the look-ahead embedding table
    dtype: str = "bf16"       # "fp32" or "bf16"
    rms_eps: float = 1e-6
    rope_theta: float = 1e4


SHAPES: Dict[str, ModelShape] = {
    "tiny": ModelShape(2, 256, 4, 64, 688, 1024, k_max=8, dtype="fp32"),
    "7b": ModelShape(32, 4096, 32, 128, 11008, 32000),
    "13b": ModelShape(40, 5120, 40, 128, 13824, 32000),
}

# stream ids
_S_TOK, _S_LA, _S_LM = 1, 2, 3
_S_LAYER0, _S_PER_LAYER = 16, 8      # wq wk wv wo wg wu wd
_S_PROMPT, _S_UNIF = 1 << 20, 1 << 21

_TORCH_DTYPE = {"fp32": torch.float32, "bf16": torch.bfloat16}


_LAYER_NAMES = ["wq", "wk", "wv", "wo", "wg", "wu", "wd"]


def make_layer_weights(shape: ModelShape, layer: int, seed: int = 0, device="cpu", std: float = 0.02
                       ) -> Dict[str, torch.Tensor]:
    """The seven matrices and two norm gains of one decoder layer (same values as in make_weights)."""
    dt = _TORCH_DTYPE[shape.dtype]
    d, f = shape.d_model, shape.d_ffn
    dims = [(d, d), (d, d), (d, d), (d, d), (f, d), (f, d), (d, f)]
    out: Dict[str, torch.Tensor] = {}
    for j, (n, (r, c)) in enumerate(zip(_LAYER_NAMES, dims)):
        out[n] = normal(seed, _S_LAYER0 + layer * _S_PER_LAYER + j, r * c, std, device).view(r, c).to(dt)
    out["norm_attn"] = torch.ones(d, dtype=dt, device=device)
    out["norm_ffn"] = torch.ones(d, dtype=dt, device=device)
    return out


def make_weights(shape: ModelShape, seed: int = 0, device="cpu", std: float = 0.02
                 ) -> Dict[str, object]:
    """All tensors of a random-init decoder, canonical [out, in] row-major.

    Matrices, embeddings and look-ahead rows are N(0, std) rounded to the model
    dtype; norm gains are exactly 1.
    """
    dt = _TORCH_DTYPE[shape.dtype]
    d, v = shape.d_model, shape.vocab

    def mat(stream, rows, cols):
        return normal(seed, stream, rows * cols, std, device).view(rows, cols).to(dt)

    w: Dict[str, object] = {
        "tok_emb": mat(_S_TOK, v, d),
        "la_emb": mat(_S_LA, shape.k_max, d),
        "lm_head": mat(_S_LM, v, d),
        "final_norm": torch.ones(d, dtype=dt, device=device),
    }
    for n in _LAYER_NAMES + ["norm_attn", "norm_ffn"]:
        w[n] = []
    for l in range(shape.n_layers):
        for n, t in make_layer_weights(shape, l, seed, device, std).items():
            w[n].append(t)
    return w


def weights_to(w: Dict[str, object], device) -> Dict[str, object]:
    out = {}
    for k, v in w.items():
        out[k] = [t.to(device) for t in v] if isinstance(v, list) else v.to(device)
    return out


def make_prompt(shape: ModelShape, length: int, seq: int = 0, seed: int = 0) -> List[int]:
    return token_ids(seed, _S_PROMPT + seq, length, shape.vocab).tolist()


def step_uniforms(seed: int, seq: int, step: int, n_slots: int) -> torch.Tensor:
    """The uniforms of one PaSS step of one sequence: float32 [n_slots]."""
    return uniforms(seed, _S_UNIF + seq, step * 64, n_slots)


_S_KV = 1 << 22


def make_kv(shape: ModelShape, layer: int, n_pos: int, seq: int = 0, seed: int = 0, std: float = 1.0,
            device="cpu"):
    """Synthetic cached keys and values of one layer, [n_pos, d_model] each in the model dtype.

    Stands in for the cache a long prompt would leave behind, so that long contexts can be
    checked without paying for the prompt pass on the CPU side.
    """
    dt = _TORCH_DTYPE[shape.dtype]
    base = _S_KV + (seq * 4096 + layer) * 2
    k = normal(seed, base, n_pos * shape.d_model, std, device).view(n_pos, shape.d_model).to(dt)
    v = normal(seed, base + 1, n_pos * shape.d_model, std, device).view(n_pos, shape.d_model).to(dt)
    return k, v
