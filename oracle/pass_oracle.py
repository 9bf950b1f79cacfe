"""CPU oracle of PaSS (Parallel Speculative Sampling): TEST INFRASTRUCTURE only.

Nothing here is a product path.  Only the tests, the smoke check and the
CPU-baseline leg of the benchmark may import this module; the CUDA library
never does, and this module imports nothing from it.

What it holds, each part written from the paper in float64:

* ``TransformerBackend``  - the decoder forward (C, ``pass_oracle.c``) behind a
  tiny "rows in, logits out" interface with a KV cache that can be truncated
  (section "Baselines": after each model call the cache is cut back to what the
  accepted tokens need).
* ``softmax_T``, ``invcdf``, ``verify`` - the speculative-sampling rule of
  Algorithm 1 / Algorithm 2: accept draft t when r < min(1, target/draft), else
  sample from the positive part of (target - draft) and stop; if every draft is
  accepted, sample one more token from the last target row.
* ``PassOracle``          - the one-call-per-iteration schedule of Algorithm 1
  (validation of the previous drafts and drafting of the next ones share one
  forward pass of 1 + m + k rows).
* ``alg1_two_call``       - Algorithm 1 exactly as printed (a drafting call and a
  validation call per iteration).
* ``autoregressive``      - the auto-regressive baseline (Baselines).

Naming: the paper calls the target distribution q and the draft p; other texts
swap them.  To stay unambiguous this file says P_tgt and Q_dft.

Pins (tests/test_oracle_*.py): exact enumeration of ``verify`` and of both
schedules on a toy vocabulary with a table model (output law == target law),
greedy PaSS == greedy auto-regressive, multi-row forward == one-row forwards
bit for bit, the forward against a float64 torch transcription built from
library matmul/softmax, closed forms of the acceptance probability.
The paper prints no worked numeric example of a step, so no printed values pin
the forward: parity for the printed tables is unpinned (they need trained
weights and datasets).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpass_oracle.so")
_SRC_PATH = os.path.join(_HERE, "pass_oracle.c")

Row = Tuple[str, int]          # ("tok", token id)  or  ("la", look-ahead index 0..k-1)


def build_oracle(force: bool = False) -> str:
    """Compile pass_oracle.c into libpass_oracle.so next to it (gcc + OpenMP)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC_PATH)):
        return _LIB_PATH
    cmd = ["gcc", "-O3", "-march=native", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
           "-o", _LIB_PATH, _SRC_PATH, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB_PATH


class _CModel(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("n_layers", "d_model", "n_heads", "d_head", "d_ffn", "vocab", "wdtype", "kvdtype")] + \
               [("rms_eps", ctypes.c_double), ("rope_theta", ctypes.c_double),
                ("lm_head", ctypes.c_void_p), ("final_norm", ctypes.c_void_p)] + \
               [(n, ctypes.POINTER(ctypes.c_void_p)) for n in
                ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm_attn", "norm_ffn")]


_lib = None


def _load():
    global _lib
    if _lib is None:
        build_oracle()
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.oracle_forward.restype = ctypes.c_int
        _lib.oracle_forward.argtypes = [ctypes.POINTER(_CModel), ctypes.c_void_p, ctypes.c_int,
                                        ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _widen(t) -> np.ndarray:
    """Exact float64 copy of a small torch tensor (fp32 or bf16)."""
    return t.detach().cpu().double().numpy()


class TransformerBackend:
    """Decoder forward with a float64 KV cache for ONE sequence.

    ``weights``: dict of CPU torch tensors as produced by the synthetic input
    generator (canonical [out, in] row-major; float32 or bfloat16).
    ``forward(rows, pos0)`` places the rows at positions pos0, pos0+1, ... (plain
    causal mask, look-ahead rows appended after the real tokens - Look-ahead
    embeddings) and returns float64 logits [len(rows), vocab].  Whatever the cache
    held at positions >= pos0 is overwritten: that is the rollback.

    ``kv_dtype`` is the storage format of the cache.  The paper does not fix one
    (Experiments, setup), so the default "f64" keeps every row as computed.
    "bf16" models a bfloat16 cache: each K/V row is rounded (nearest, ties to even)
    when it is stored, and attention reads the stored values - the arithmetic stays
    float64.  That isolates the one error a bf16 cache makes by construction.
    """

    def __init__(self, shape, weights, kv_capacity: int, kv_dtype: str = "f64"):
        import torch
        self.shape = shape
        self.w = weights
        self.cap = int(kv_capacity)
        self.vocab = shape.vocab
        d = shape.d_model
        self.k = np.zeros((shape.n_layers, self.cap, d), dtype=np.float64)
        self.v = np.zeros((shape.n_layers, self.cap, d), dtype=np.float64)
        dt = weights["lm_head"].dtype
        assert dt in (torch.float32, torch.bfloat16)
        for name, val in weights.items():
            for t in (val if isinstance(val, list) else [val]):
                assert t.device.type == "cpu" and t.is_contiguous() and t.dtype == dt, name
        cm = _CModel()
        cm.n_layers, cm.d_model, cm.n_heads = shape.n_layers, d, shape.n_heads
        cm.d_head, cm.d_ffn, cm.vocab = shape.d_head, shape.d_ffn, shape.vocab
        cm.wdtype = 0 if dt == torch.float32 else 1
        cm.kvdtype = {"f64": 0, "bf16": 1}[kv_dtype]
        cm.rms_eps, cm.rope_theta = float(shape.rms_eps), float(shape.rope_theta)
        cm.lm_head = weights["lm_head"].data_ptr()
        cm.final_norm = weights["final_norm"].data_ptr()
        self._arrays = []
        for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm_attn", "norm_ffn"):
            arr = (ctypes.c_void_p * shape.n_layers)(*[t.data_ptr() for t in weights[n]])
            self._arrays.append(arr)
            setattr(cm, n, ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p)))
        self._cm = cm
        self._lib = _load()

    def embed(self, rows: Sequence[Row]) -> np.ndarray:
        x = np.empty((len(rows), self.shape.d_model), dtype=np.float64)
        for i, (kind, idx) in enumerate(rows):
            src = self.w["tok_emb"] if kind == "tok" else self.w["la_emb"]
            x[i] = _widen(src[int(idx)])
        return x

    def forward(self, rows: Sequence[Row], pos0: int, want_logits: bool = True
                ) -> Optional[np.ndarray]:
        n = len(rows)
        if pos0 + n > self.cap:
            raise ValueError("KV capacity exceeded")
        x = self.embed(rows)
        logits = np.empty((n, self.vocab), dtype=np.float64) if want_logits else None
        rc = self._lib.oracle_forward(
            ctypes.byref(self._cm), x.ctypes.data, n, int(pos0), self.k.ctypes.data,
            self.v.ctypes.data, self.cap, logits.ctypes.data if want_logits else None, None)
        if rc != 0:
            raise RuntimeError("oracle_forward failed")
        return logits

    def prefill(self, tokens: Sequence[int], chunk: int = 256) -> None:
        """Cache K/V of ``tokens`` at positions 0.. (no logits)."""
        for s in range(0, len(tokens), chunk):
            part = tokens[s:s + chunk]
            self.forward([("tok", t) for t in part], s, want_logits=False)


class Pieces:
    """The single operations of the forward, one call each (for pinning them)."""

    def __init__(self, shape, wdtype: int = 0):
        cm = _CModel()
        cm.n_layers, cm.d_model, cm.n_heads = shape.n_layers, shape.d_model, shape.n_heads
        cm.d_head, cm.d_ffn, cm.vocab = shape.d_head, shape.d_ffn, shape.vocab
        cm.wdtype, cm.kvdtype = wdtype, 0
        cm.rms_eps, cm.rope_theta = float(shape.rms_eps), float(shape.rope_theta)
        self._cm, self._lib, self.shape = cm, _load(), shape

    def linear(self, W: np.ndarray, x: np.ndarray) -> np.ndarray:
        """x [n, in] (float64) times W^T, W [out, in] float32 (or uint16 bf16 bits)."""
        W = np.ascontiguousarray(W)
        x = np.ascontiguousarray(x, dtype=np.float64)
        y = np.empty((x.shape[0], W.shape[0]))
        self._lib.oracle_linear(ctypes.byref(self._cm), ctypes.c_void_p(W.ctypes.data),
                                W.shape[0], W.shape[1], ctypes.c_void_p(x.ctypes.data),
                                x.shape[0], ctypes.c_void_p(y.ctypes.data))
        return y

    def rmsnorm(self, g: np.ndarray, x: np.ndarray) -> np.ndarray:
        g = np.ascontiguousarray(g)
        x = np.ascontiguousarray(x, dtype=np.float64)
        y = np.empty_like(x)
        self._lib.oracle_rmsnorm(ctypes.byref(self._cm), ctypes.c_void_p(g.ctypes.data),
                                 ctypes.c_void_p(x.ctypes.data), x.shape[0],
                                 ctypes.c_void_p(y.ctypes.data))
        return y

    def rope(self, v: np.ndarray, pos: int) -> np.ndarray:
        out = np.array(v, dtype=np.float64, copy=True)
        self._lib.oracle_rope(ctypes.byref(self._cm), ctypes.c_void_p(out.ctypes.data), int(pos))
        return out

    def attention(self, q: np.ndarray, kc: np.ndarray, vc: np.ndarray, pos0: int) -> np.ndarray:
        q = np.ascontiguousarray(q, dtype=np.float64)
        kc = np.ascontiguousarray(kc, dtype=np.float64)
        vc = np.ascontiguousarray(vc, dtype=np.float64)
        o = np.empty_like(q)
        self._lib.oracle_attention(ctypes.byref(self._cm), ctypes.c_void_p(q.ctypes.data),
                                   ctypes.c_void_p(kc.ctypes.data), ctypes.c_void_p(vc.ctypes.data),
                                   q.shape[0], int(pos0), ctypes.c_void_p(o.ctypes.data))
        return o

    def swiglu(self, g: np.ndarray, u: np.ndarray) -> np.ndarray:
        out = np.array(g, dtype=np.float64, copy=True)
        u = np.ascontiguousarray(u, dtype=np.float64)
        self._lib.oracle_swiglu(ctypes.c_void_p(out.ctypes.data), ctypes.c_void_p(u.ctypes.data),
                                ctypes.c_long(out.size))
        return out


class TableBackend:
    """A lookup-table "model" for exact enumeration on a toy vocabulary.

    The distribution of a row depends only on the last real token before (or at)
    the row and on how many look-ahead rows follow it:
    ``prob[j][t]`` is a length-V law for "last real token t, j look-ahead rows".
    j = 0 is the target model q(. | ..., t) itself.  Logits are log(prob).
    """

    def __init__(self, prob: np.ndarray, cap: int = 64):
        self.prob = np.asarray(prob, dtype=np.float64)   # [k+1][V][V]
        self.vocab = self.prob.shape[-1]
        self.sym: List[Optional[Row]] = [None] * cap

    def prefill(self, tokens: Sequence[int], chunk: int = 0) -> None:
        for i, t in enumerate(tokens):
            self.sym[i] = ("tok", int(t))

    def forward(self, rows: Sequence[Row], pos0: int, want_logits: bool = True):
        out = np.empty((len(rows), self.vocab))
        for r, row in enumerate(rows):
            self.sym[pos0 + r] = (row[0], int(row[1]))
            p, n_la = pos0 + r, 0
            while self.sym[p][0] == "la":
                n_la += 1
                p -= 1
            with np.errstate(divide="ignore"):
                out[r] = np.log(self.prob[n_la][self.sym[p][1]])
        return out


# ---------------------------------------------------------------------------
# Sampling primitives
# ---------------------------------------------------------------------------

def top_k_set(z: np.ndarray, top_k: int) -> np.ndarray:
    """Indices of the top_k largest entries of z; among equal values the lower index ranks first."""
    z = np.asarray(z, dtype=np.float64)
    order = sorted(range(z.size), key=lambda i: (-z[i], i))
    return np.array(sorted(order[:top_k]), dtype=np.int64)


def softmax_T(z: np.ndarray, temperature: float, top_k: int = 0) -> np.ndarray:
    """softmax(z / T) in float64; T == 0 is the one-hot law at the first argmax.

    top_k > 0 is top-k sampling (Experiments, setup: "top-k sampling" with a
    temperature): the law is the softmax over the top_k largest logits only,
    every other token has probability exactly 0.  The same filter is applied to
    every row, target rows and look-ahead rows alike, before any ratio is formed.
    """
    z = np.asarray(z, dtype=np.float64)
    if temperature == 0.0:
        p = np.zeros_like(z)
        p[int(np.argmax(z))] = 1.0
        return p
    s = z / float(temperature)
    e = np.exp(s - np.max(s))
    if 0 < top_k < z.size:
        keep = np.zeros(z.size, dtype=bool)
        keep[top_k_set(z, top_k)] = True
        e = np.where(keep, e, 0.0)
    return e / np.sum(e)


def invcdf(w: np.ndarray, u: float) -> int:
    """Smallest index i with w_0 + ... + w_i > u * sum(w), vocabulary order.

    If rounding leaves no such index, the last index with w > 0.
    """
    c = np.cumsum(np.asarray(w, dtype=np.float64))
    hit = np.nonzero(c > float(u) * c[-1])[0]
    if hit.size:
        return int(hit[0])
    return int(np.nonzero(w > 0)[0][-1])


def invcdf_margin(w: np.ndarray, u: float) -> float:
    """Distance of u from the nearest edge of the chosen token's CDF interval."""
    c = np.cumsum(np.asarray(w, dtype=np.float64))
    c = c / c[-1]
    return float(np.min(np.abs(c - float(u))))


def verify(P_tgt: np.ndarray, Q_dft: np.ndarray, drafts: Sequence[int],
           u_accept: Sequence[float], u_final: float):
    """The accept / resample rule shared by Algorithm 1 and Algorithm 2.

    P_tgt: [m+1, V] target laws; row j-1 is the target law at the position of
    draft j.  Q_dft: [m, V] laws the drafts were drawn from.  Returns
    (n_accepted, final_token, info).  Draft j is kept when
    u_accept[j-1] < min(1, P_tgt[j-1][d_j] / Q_dft[j-1][d_j]) (strict).  On the
    first failure the final token comes from the normalised positive part of
    P_tgt[j-1] - Q_dft[j-1]; if it has no mass (the laws coincide) from P_tgt[j-1].
    With every draft kept, the final token comes from P_tgt[m].
    """
    m = len(drafts)
    info = {"ratio_margin": [], "final_law": None}
    for j in range(m):
        d = int(drafts[j])
        ratio = P_tgt[j][d] / Q_dft[j][d]
        info["ratio_margin"].append(abs(float(ratio) - float(u_accept[j])))
        if float(u_accept[j]) < min(1.0, ratio):
            continue
        resid = np.maximum(0.0, P_tgt[j] - Q_dft[j])
        if np.sum(resid) == 0.0:
            resid = P_tgt[j]
        info["final_law"] = resid
        return j, invcdf(resid, u_final), info
    info["final_law"] = P_tgt[m]
    return m, invcdf(P_tgt[m], u_final), info


# ---------------------------------------------------------------------------
# Schedules
# ---------------------------------------------------------------------------

class PassOracle:
    """One-call-per-iteration PaSS for one sequence.

    State: ``len`` cached positions, ``pending`` (last emitted token, not yet in
    the cache), and either m = 0 or m = k pending drafts with the laws Q_dft they
    were drawn from.  One step feeds rows
    [pending, d_1..d_m, LA_1..LA_k] at positions len, len+1, ...; rows 0..m give
    the target laws that validate the drafts (Algorithm 1, validation phase) and
    rows m+1..m+k are the drafting phase for the next step.  When a draft is
    rejected the look-ahead rows were conditioned on rejected tokens and their
    outputs are dropped: the next step is then exactly the drafting call of
    Algorithm 1.

    Uniform slots of a step, u[0 .. 2k]: u[j-1] accept test of draft j;
    u[k] the final token (residual resample or extra token); u[k+t] draft t of
    the next step.
    """

    def __init__(self, backend, prompt: Sequence[int]):
        self.be = backend
        prompt = [int(t) for t in prompt]
        self.be.prefill(prompt[:-1])
        self.len = len(prompt) - 1
        self.pending = prompt[-1]
        self.drafts: List[int] = []
        self.Q_dft = np.zeros((0, backend.vocab))
        self.k_prev: Optional[int] = None
        self.T_prev: Optional[float] = None
        self.top_k = 0                      # 0 = plain temperature sampling
        self.top_k_prev = 0
        self.last_logits: Optional[np.ndarray] = None

    def rows(self, k: int) -> List[Row]:
        return ([("tok", self.pending)] + [("tok", d) for d in self.drafts]
                + [("la", i) for i in range(k)])

    def forward_step(self, k: int, temperature: float) -> np.ndarray:
        """Run the model call of a step; returns float64 logits [1 + m + k, V]."""
        top_k = getattr(self, "top_k", 0)
        if k != self.k_prev or temperature != self.T_prev or top_k != getattr(self, "top_k_prev", 0):
            self.drafts, self.Q_dft = [], np.zeros((0, self.be.vocab))   # drawn under other settings
        self.k_prev, self.T_prev, self.top_k_prev = k, temperature, top_k
        Z = self.be.forward(self.rows(k), self.len)
        self.last_logits = Z
        return Z

    def decide(self, Z: np.ndarray, Q_dft: np.ndarray, k: int, temperature: float,
               u: Sequence[float]) -> dict:
        """Pure decision of a step from logits Z and the stored draft laws Q_dft.

        Touches no state, so the same rule can be replayed on logits that some
        other implementation computed.
        """
        m = len(self.drafts)
        top_k = getattr(self, "top_k", 0)
        Z = np.asarray(Z, dtype=np.float64)
        P_tgt = np.stack([softmax_T(Z[j], temperature, top_k) for j in range(m + 1)])
        a, y, info = verify(P_tgt, Q_dft, self.drafts, u[:m], u[k])
        info["final_margin"] = invcdf_margin(info["final_law"], u[k])
        # top-2 logit gap of every target row (row j decides draft j+1, row a the final token)
        info["row_top2"] = [float(np.diff(np.sort(Z[j])[-2:])[0]) for j in range(m + 1)]
        info["top2_margin"] = info["row_top2"][a]
        info["m"] = m
        dec = {"m": m, "n_accepted": a, "final": y, "emitted": list(self.drafts[:a]) + [y],
               "new_drafts": [], "Qn": np.zeros((0, self.be.vocab)), "info": info}
        if a == m and k > 0:
            Qn = np.stack([softmax_T(Z[m + 1 + t], temperature, top_k) for t in range(k)])
            dec["Qn"] = Qn
            dec["new_drafts"] = [invcdf(Qn[t], u[k + 1 + t]) for t in range(k)]
            info["draft_margin"] = [invcdf_margin(Qn[t], u[k + 1 + t]) for t in range(k)]
            info["draft_top2"] = [float(np.diff(np.sort(Z[m + 1 + t])[-2:])[0]) for t in range(k)]
        return dec

    def commit(self, emitted: Sequence[int], new_drafts: Sequence[int], Qn: np.ndarray) -> None:
        """Advance the state: keep K/V of the old pending token and of the accepted
        drafts, drop everything after them, and install the next drafts (or none)."""
        self.len += len(emitted)
        self.pending = int(emitted[-1])
        self.drafts = [int(d) for d in new_drafts]
        self.Q_dft = np.asarray(Qn, dtype=np.float64) if len(new_drafts) else \
            np.zeros((0, self.be.vocab))

    def step(self, k: int, temperature: float, u: Sequence[float], top_k: Optional[int] = None):
        """Returns (emitted tokens, n_accepted, info).  1 <= len(emitted) <= k+1."""
        if top_k is not None:
            self.top_k = int(top_k)
        Z = self.forward_step(k, temperature)
        dec = self.decide(Z, self.Q_dft, k, temperature, u)
        self.commit(dec["emitted"], dec["new_drafts"], dec["Qn"])
        return dec["emitted"], dec["n_accepted"], dec["info"]


def alg1_two_call(backend, prompt: Sequence[int], L: int, temperature: float,
                  n_tokens: int, uniform_fn: Callable[[int, int], np.ndarray], top_k: int = 0):
    """Algorithm 1 as printed: per iteration a drafting call on
    [x_n, LA_1..LA_L], then a validation call on [x_{n+1}, d_1..d_L].

    ``uniform_fn(it, n)`` returns n uniforms for iteration ``it``: slot 0 samples
    x_{n+1}, slots 1..L the drafts, slots L+1..2L the accept tests, slot 2L+1 the
    final token.  Returns (generated tokens, number of model calls).
    """
    prompt = [int(t) for t in prompt]
    backend.prefill(prompt[:-1])
    n_cached, pending = len(prompt) - 1, prompt[-1]
    out: List[int] = []
    calls = it = 0
    while len(out) < n_tokens:
        u = uniform_fn(it, 2 * L + 2)
        it += 1
        # drafting phase
        Z = backend.forward([("tok", pending)] + [("la", i) for i in range(L)], n_cached)
        calls += 1
        x_next = invcdf(softmax_T(Z[0], temperature, top_k), u[0])
        Q_dft = np.stack([softmax_T(Z[1 + t], temperature, top_k) for t in range(L)])
        drafts = [invcdf(Q_dft[t], u[1 + t]) for t in range(L)]
        out.append(x_next)
        n_cached += 1                      # keep K/V of the old pending token only
        pending = x_next
        # validation phase
        Z = backend.forward([("tok", pending)] + [("tok", d) for d in drafts], n_cached)
        calls += 1
        P_tgt = np.stack([softmax_T(Z[j], temperature, top_k) for j in range(L + 1)])
        a, y, _ = verify(P_tgt, Q_dft, drafts, u[L + 1:2 * L + 1], u[2 * L + 1])
        out.extend(drafts[:a] + [y])
        n_cached += 1 + a
        pending = y
    return out, calls


def autoregressive(backend, prompt: Sequence[int], temperature: float, n_tokens: int,
                   uniform_fn: Callable[[int], float], top_k: int = 0):
    """One token per model call with the KV cache (Baselines)."""
    prompt = [int(t) for t in prompt]
    backend.prefill(prompt[:-1])
    n_cached, pending = len(prompt) - 1, prompt[-1]
    out: List[int] = []
    all_logits = []
    for i in range(n_tokens):
        Z = backend.forward([("tok", pending)], n_cached)
        all_logits.append(Z[0])
        pending = invcdf(softmax_T(Z[0], temperature, top_k), uniform_fn(i))
        out.append(pending)
        n_cached += 1
    return out, all_logits
