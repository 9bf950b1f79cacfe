"""ctypes binding of libpass_b200.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch is used for
device memory (KV cache, workspace, weights) and for the stream; there is no
CPU fallback - if the library is missing or no CUDA device is present, calls
raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpass_b200.so")

PASS_DBG_LOGITS, PASS_DBG_DRAFT_LOGITS, PASS_DBG_KV_LEN, PASS_DBG_N_DRAFT = 0, 1, 2, 3
PASS_DBG_DRAFTS, PASS_DBG_PENDING, PASS_DBG_N_ACCEPTED, PASS_DBG_STATUS, PASS_DBG_HIDDEN = 4, 5, 6, 7, 8
PASS_DBG_FOOTPRINT = 10
PASS_DBG_ATTN_TRACE = 11
PASS_MAX_ROWS = 128
PASS_HOOK_GEMM_STUCK, PASS_HOOK_ATTN_STALE, PASS_HOOK_ATTN_LONG_FROM, PASS_HOOK_ATTN_STUCK = 0, 1, 2, 3
PASS_PROMPT_HI_LO, PASS_PROMPT_BF16 = 0, 1
PASS_TRAIN_LA, PASS_TRAIN_GRAD = 0, 1
PASS_MAX_TOP_K = 1024

EXPORTS = ["pass_kv_bytes", "pass_workspace_bytes", "pass_create", "pass_load_weights", "pass_prefill",
           "pass_step", "pass_step_enqueue", "pass_step_collect", "pass_forward_tokens", "pass_reset",
           "pass_set_top_k", "pass_step_two_call", "pass_debug_schedule",
           "pass_set_kv", "pass_get_kv", "pass_set_state", "pass_get_debug", "pass_last_step_launches",
           "pass_stream", "pass_destroy", "pass_strerror", "pass_debug_linear",
           "pass_debug_time_linear", "pass_linear_noalloc", "pass_debug_set", "pass_set_prompt_precision",
           "pass_train_workspace_bytes", "pass_train_init", "pass_train_step", "pass_train_get", "pass_train_export"]


class PassError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{msg} (code {code})")
        self.code = code


class _Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("n_layers", "d_model", "n_heads", "d_head", "d_ffn", "vocab", "k_max", "max_batch",
                 "kv_capacity", "dtype")] + [("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)]


class _TrainConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_float) for n in ("lr", "beta1", "beta2", "eps", "weight_decay")] + \
               [("warmup_steps", ctypes.c_int), ("total_steps", ctypes.c_int)]


class _Weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("tok_emb", "la_emb", "lm_head", "final_norm")] + \
               [(n, ctypes.POINTER(ctypes.c_void_p)) for n in
                ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm_attn", "norm_ffn")]


_lib = None


def load_library(path: str = LIB_PATH):
    """dlopen the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} not built: run __graft_entry__.build() "
                                "(python -m paper_2311_13581_b200.build)")
    lib = ctypes.CDLL(path)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.pass_kv_bytes.restype = ctypes.c_size_t
    lib.pass_kv_bytes.argtypes = [ctypes.POINTER(_Config)]
    lib.pass_workspace_bytes.restype = ctypes.c_size_t
    lib.pass_workspace_bytes.argtypes = [ctypes.POINTER(_Config)]
    lib.pass_create.argtypes = [ctypes.POINTER(_Config), vp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp,
                                ctypes.POINTER(vp)]
    lib.pass_load_weights.argtypes = [vp, ctypes.POINTER(_Weights)]
    lib.pass_prefill.argtypes = [vp, ci, vp, ci]
    lib.pass_step.argtypes = [vp, ci, cf, vp, vp, vp]
    lib.pass_step_two_call.argtypes = [vp, ci, cf, vp, vp, vp]
    lib.pass_step_enqueue.argtypes = [vp, ci, cf, vp]
    lib.pass_step_collect.argtypes = [vp, vp, vp]
    lib.pass_forward_tokens.argtypes = [vp, ci, vp, ci, vp, ci]
    lib.pass_reset.argtypes = [vp, ci]
    lib.pass_set_top_k.argtypes = [vp, ci]
    lib.pass_debug_schedule.argtypes = [ci, ci, ci, ci, ci, vp]
    lib.pass_set_kv.argtypes = [vp, ci, ci, ci, ci, vp, vp]
    lib.pass_get_kv.argtypes = [vp, ci, ci, ci, ci, vp, vp]
    lib.pass_set_state.argtypes = [vp, ci, ci, ctypes.c_int32]
    lib.pass_get_debug.argtypes = [vp, ci, vp, ctypes.c_size_t]
    lib.pass_last_step_launches.argtypes = [vp]
    lib.pass_debug_linear.argtypes = [vp, ci, ci, vp, ci, vp]
    lib.pass_debug_time_linear.argtypes = [vp, ci, ci, ci, vp]
    lib.pass_linear_noalloc.argtypes = [vp, ci, ci, vp, ci, vp]
    lib.pass_debug_set.argtypes = [vp, ci, ci]
    lib.pass_set_prompt_precision.argtypes = [vp, ci]
    lib.pass_train_workspace_bytes.restype = ctypes.c_size_t
    lib.pass_train_workspace_bytes.argtypes = [ctypes.POINTER(_Config), ci, ci]
    lib.pass_train_init.argtypes = [vp, vp, ctypes.c_size_t, ctypes.POINTER(_TrainConfig), ci, ci]
    lib.pass_train_step.argtypes = [vp, vp, ci, vp, ci, ci, vp]
    lib.pass_train_get.argtypes = [vp, ci, vp, ctypes.c_size_t]
    lib.pass_train_export.argtypes = [vp, vp]
    lib.pass_stream.restype = vp
    lib.pass_stream.argtypes = [vp]
    lib.pass_destroy.restype = None
    lib.pass_destroy.argtypes = [vp]
    lib.pass_strerror.restype = ctypes.c_char_p
    lib.pass_strerror.argtypes = [ci]
    _lib = lib
    return lib


def _check(lib, rc: int):
    if rc != 0:
        raise PassError(rc, lib.pass_strerror(rc).decode())


class PassContext:
    """One library context: owns the torch buffers it lends to the library.

    ``shape`` carries n_layers, d_model, n_heads, d_head, d_ffn, vocab, k_max, dtype
    ("fp32" / "bf16"), rms_eps, rope_theta.  ``weights``: dict of CUDA torch tensors,
    canonical [out, in] row-major (per-layer entries are lists).
    """

    def __init__(self, shape, weights: Dict[str, object], max_batch: int, kv_capacity: int,
                 device="cuda:0", stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("PaSS step needs a CUDA device (sm_100a); there is no CPU path")
        self.lib = load_library()
        self.torch = torch
        self.shape = shape
        self.device = torch.device(device)
        self.B = int(max_batch)
        self.k_max = int(shape.k_max)
        # result buffers of step / step_collect, made once: building arrays and their ctypes views per call costs
        # the caller some 15 us of a 2.8 ms step
        self._out = np.full((self.B, self.k_max + 1), -1, dtype=np.int32)
        self._n = np.zeros(self.B, dtype=np.int32)
        self._out_ptr, self._n_ptr = self._out.ctypes.data, self._n.ctypes.data
        self.vocab = int(shape.vocab)
        cfg = _Config(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab,
                      shape.k_max, self.B, int(kv_capacity), 0 if shape.dtype == "fp32" else 1,
                      float(shape.rms_eps), float(shape.rope_theta))
        self.cfg = cfg
        kvb = self.lib.pass_kv_bytes(ctypes.byref(cfg))
        wsb = self.lib.pass_workspace_bytes(ctypes.byref(cfg))
        if kvb == 0 or wsb == 0:
            raise PassError(-1, "unsupported configuration")
        with torch.cuda.device(self.device):
            self.kv_k = torch.zeros(kvb, dtype=torch.uint8, device=self.device)
            self.kv_v = torch.zeros(kvb, dtype=torch.uint8, device=self.device)
            self.ws = torch.zeros(wsb, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.Stream(device=self.device)
            torch.cuda.synchronize(self.device)
            h = ctypes.c_void_p()
            _check(self.lib, self.lib.pass_create(ctypes.byref(cfg), self.kv_k.data_ptr(), self.kv_v.data_ptr(),
                                                  kvb, self.ws.data_ptr(), wsb, self.stream.cuda_stream,
                                                  ctypes.byref(h)))
        self.h = h
        self.weights = weights
        want = torch.float32 if shape.dtype == "fp32" else torch.bfloat16
        cw = _Weights()
        self._keep = []
        for n in ("tok_emb", "la_emb", "lm_head", "final_norm"):
            t = weights[n]
            assert t.is_cuda and t.is_contiguous() and t.dtype == want, n
            setattr(cw, n, t.data_ptr())
        for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm_attn", "norm_ffn"):
            for t in weights[n]:
                assert t.is_cuda and t.is_contiguous() and t.dtype == want, n
            arr = (ctypes.c_void_p * shape.n_layers)(*[t.data_ptr() for t in weights[n]])
            self._keep.append(arr)
            setattr(cw, n, ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p)))
        _check(self.lib, self.lib.pass_load_weights(self.h, ctypes.byref(cw)))

    # -- the calls of include/pass.h -------------------------------------------------------
    def prefill(self, seq: int, tokens: Sequence[int]) -> None:
        a = np.ascontiguousarray(tokens, dtype=np.int32)
        _check(self.lib, self.lib.pass_prefill(self.h, seq, a.ctypes.data, len(a)))

    def step(self, k: int, temperature: float, uniforms: Optional[np.ndarray]
             ) -> Tuple[List[List[int]], np.ndarray]:
        """uniforms: [B][2k+1] float32 host array (None iff temperature == 0)."""
        out, n = self._out, self._n
        up = None
        if uniforms is not None:
            u = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(self.B, 2 * k + 1)
            up = u.ctypes.data
        _check(self.lib, self.lib.pass_step(self.h, k, float(temperature), up, self._out_ptr, self._n_ptr))
        return [out[b, :n[b]].tolist() for b in range(self.B)], n.copy()

    def step_enqueue(self, k: int, temperature: float, uniforms_device=None) -> None:
        p = None if uniforms_device is None else uniforms_device.data_ptr()
        _check(self.lib, self.lib.pass_step_enqueue(self.h, k, float(temperature), p))

    def step_collect(self) -> Tuple[List[List[int]], np.ndarray]:
        out, n = self._out, self._n
        _check(self.lib, self.lib.pass_step_collect(self.h, self._out_ptr, self._n_ptr))
        return [out[b, :n[b]].tolist() for b in range(self.B)], n.copy()

    def forward_tokens(self, seq: int, tokens: Sequence[int], commit: int, want_logits: bool = True):
        a = np.ascontiguousarray(tokens, dtype=np.int32)
        logits = None
        if want_logits:
            logits = self.torch.empty((len(a), self.vocab), dtype=self.torch.float32, device=self.device)
        _check(self.lib, self.lib.pass_forward_tokens(self.h, seq, a.ctypes.data, len(a),
                                                      None if logits is None else logits.data_ptr(), commit))
        return logits

    def reset(self, seq: int) -> None:
        _check(self.lib, self.lib.pass_reset(self.h, seq))

    def step_two_call(self, L: int, temperature: float, uniforms):
        """uniforms: numpy float32 [B][2L+2] or None (greedy). Returns (list of emitted lists, n_out)."""
        out = np.zeros((self.B, self.k_max + 2), dtype=np.int32)
        n_out = np.zeros(self.B, dtype=np.int32)
        if uniforms is not None:
            uniforms = np.ascontiguousarray(uniforms, dtype=np.float32)
            assert uniforms.shape == (self.B, 2 * L + 2)
            up = uniforms.ctypes.data
        else:
            up = None
        _check(self.lib, self.lib.pass_step_two_call(self.h, int(L), ctypes.c_float(temperature), up,
                                                     out.ctypes.data, n_out.ctypes.data))
        return [out[b, :n_out[b]].tolist() for b in range(self.B)], n_out

    def set_top_k(self, top_k: int) -> None:
        _check(self.lib, self.lib.pass_set_top_k(self.h, int(top_k)))

    def set_state(self, seq: int, length: int, pending: int) -> None:
        _check(self.lib, self.lib.pass_set_state(self.h, seq, length, pending))

    def _np_dtype_view(self, t):
        """host torch tensor [n][d] in the model dtype -> contiguous buffer pointer"""
        want = self.torch.float32 if self.shape.dtype == "fp32" else self.torch.bfloat16
        assert t.device.type == "cpu" and t.dtype == want and t.is_contiguous()
        return t.data_ptr()

    def set_kv(self, seq: int, layer: int, pos0: int, k_host, v_host) -> None:
        n = k_host.shape[0]
        _check(self.lib, self.lib.pass_set_kv(self.h, seq, layer, pos0, n, self._np_dtype_view(k_host),
                                              self._np_dtype_view(v_host)))

    def get_kv(self, seq: int, layer: int, pos0: int, n: int):
        want = self.torch.float32 if self.shape.dtype == "fp32" else self.torch.bfloat16
        k = self.torch.empty((n, self.shape.d_model), dtype=want)
        v = self.torch.empty((n, self.shape.d_model), dtype=want)
        _check(self.lib, self.lib.pass_get_kv(self.h, seq, layer, pos0, n, k.data_ptr(), v.data_ptr()))
        return k, v

    def get_debug(self, what: int, rows: int = 0) -> np.ndarray:
        B, km, V = self.B, self.k_max, self.vocab
        if what == PASS_DBG_LOGITS:
            a = np.empty((rows, V), dtype=np.float32)
        elif what == PASS_DBG_HIDDEN:
            a = np.empty((rows, self.shape.d_model), dtype=np.float32)
        elif what == PASS_DBG_DRAFT_LOGITS:
            a = np.empty((B, km, V), dtype=np.float32)
        elif what == PASS_DBG_DRAFTS:
            a = np.empty((B, km), dtype=np.int32)
        elif what == PASS_DBG_STATUS:
            a = np.empty(1, dtype=np.int32)
        elif what == PASS_DBG_FOOTPRINT:
            a = np.empty(9, dtype=np.int32)
        else:
            a = np.empty(B, dtype=np.int32)
        _check(self.lib, self.lib.pass_get_debug(self.h, what, a.ctypes.data, a.nbytes))
        return a

    def debug_linear(self, which: int, layer: int, x):
        """x: CUDA float32 [R][K]; returns CUDA float32 [R][N] (see pass_debug_linear)."""
        d, f = self.shape.d_model, self.shape.d_ffn
        N = {4: f, 5: f, 7: self.vocab, 8: ((f + 63) // 64) * 128}.get(which, d)
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.torch.float32
        y = self.torch.empty((x.shape[0], N), dtype=self.torch.float32, device=self.device)
        _check(self.lib, self.lib.pass_debug_linear(self.h, which, layer, x.data_ptr(), x.shape[0], y.data_ptr()))
        return y

    def linear_noalloc(self, which: int, layer: int, x, y):
        """pass_linear_noalloc: same result as debug_linear, split-K scratch inside the library image.

        For callers that may not allocate device memory: ``y`` (CUDA float32 [R][N]) is passed in
        rather than created here, and at most 16 rows are accepted."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.torch.float32
        assert y.is_cuda and y.is_contiguous() and y.dtype == self.torch.float32
        _check(self.lib, self.lib.pass_linear_noalloc(self.h, which, layer, x.data_ptr(), x.shape[0], y.data_ptr()))
        return y

    def train_init(self, L: int, max_seqs: int, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
                   warmup_steps=2000, total_steps=10000) -> None:
        """pass_train_init: the training workspace is a torch buffer owned by this object."""
        need = self.lib.pass_train_workspace_bytes(ctypes.byref(self.cfg), L, max_seqs)
        if need == 0:
            raise PassError(-1, "unsupported training configuration")
        self.train_ws = self.torch.empty(need, dtype=self.torch.uint8, device=self.device)
        hp = _TrainConfig(lr, beta1, beta2, eps, weight_decay, warmup_steps, total_steps)
        self.train_L = L
        _check(self.lib, self.lib.pass_train_init(self.h, self.train_ws.data_ptr(), need, ctypes.byref(hp), L, max_seqs))

    def train_step(self, tokens, positions, apply_update: bool = True) -> float:
        """tokens: [n_seqs][stride] int32 host array, positions: [n_seqs]; returns the batch loss."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        p = np.ascontiguousarray(positions, dtype=np.int32)
        loss = ctypes.c_float(0.0)
        _check(self.lib, self.lib.pass_train_step(self.h, t.ctypes.data, t.shape[1], p.ctypes.data, t.shape[0],
                                                  1 if apply_update else 0, ctypes.byref(loss)))
        return float(loss.value)

    def train_get(self, what: int) -> np.ndarray:
        a = np.empty((self.train_L, self.shape.d_model), dtype=np.float32)
        _check(self.lib, self.lib.pass_train_get(self.h, what, a.ctypes.data, a.nbytes))
        return a

    def train_export(self, la_emb) -> None:
        _check(self.lib, self.lib.pass_train_export(self.h, la_emb.data_ptr()))

    def set_prompt_precision(self, mode: int) -> None:
        """pass_set_prompt_precision: PASS_PROMPT_HI_LO (default) or PASS_PROMPT_BF16 for long prompts."""
        _check(self.lib, self.lib.pass_set_prompt_precision(self.h, mode))

    def debug_set(self, hook: int, value: int) -> None:
        """pass_debug_set: per-context switches for the tests of the library's error handling."""
        _check(self.lib, self.lib.pass_debug_set(self.h, hook, value))

    def debug_time_linear(self, which: int, R: int, n_launches: int) -> float:
        """Milliseconds for n_launches back-to-back launches of one GEMM, cycling over layers."""
        ms = ctypes.c_float(0.0)
        _check(self.lib, self.lib.pass_debug_time_linear(self.h, which, R, n_launches, ctypes.byref(ms)))
        return float(ms.value)

    def last_step_launches(self) -> int:
        return int(self.lib.pass_last_step_launches(self.h))

    def close(self) -> None:
        if getattr(self, "h", None):
            self.lib.pass_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
