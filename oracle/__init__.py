"""ctypes front end of the CPU oracle (test infrastructure only).

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It builds ``liborc.so`` from ``knnssd_oracle.c`` with gcc on first
use and exposes the oracle's functions on numpy / torch CPU arrays.  It imports
nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "knnssd_oracle.c")
_LIB = os.path.join(_HERE, "liborc.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Config(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim",
                                       "d_ff", "vocab", "max_seq")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("dtype", C.c_int)]


class _Weights(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo",
                                                     "mlp_norm", "w_gate", "w_up", "w_down")]


class Stats(C.Structure):
    _fields_ = [("rounds", C.c_int), ("drafted", C.c_int), ("accepted", C.c_int), ("tokens", C.c_int),
                ("min_margin", C.c_float)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_create.restype = C.c_void_p
        _lib.orc_create.argtypes = [C.POINTER(_Config), C.POINTER(_Weights)]
        _lib.orc_destroy.argtypes = [C.c_void_p]
        _lib.orc_len.argtypes = [C.c_void_p]
        _lib.orc_set_len.argtypes = [C.c_void_p, C.c_int]
        _lib.orc_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
        _lib.orc_linear.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        _lib.orc_pool_mean.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        _lib.orc_knn_select.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                        C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_float)]
        _lib.orc_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        _lib.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.POINTER(C.c_int),
                                     C.POINTER(C.c_float)]
        _lib.orc_generate.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                      C.POINTER(Stats), C.c_void_p, C.c_void_p, C.c_int]
        _lib.orc_greedy_full.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.POINTER(C.c_float)]
    return _lib


def _ptr(a) -> Optional[int]:
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        assert a.device.type == "cpu" and a.is_contiguous()
        return a.data_ptr()
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


class OracleModel:
    """A decoder with its KV cache.  ``weights`` is the dict of CPU torch tensors made by
    ``synthetic_inputs.make_model_weights`` (borrowed: kept alive by this object)."""

    def __init__(self, shape, weights: Dict[str, object], max_seq: int):
        L = shape.n_layers
        self.shape, self.max_seq, self._keep = shape, max_seq, weights
        self.cfg = _Config(L, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff,
                           shape.vocab, max_seq, shape.rms_eps, shape.rope_theta,
                           0 if shape.dtype == "fp32" else 1)
        w = _Weights()
        w.tok_embed, w.final_norm, w.lm_head = (_ptr(weights[k]) for k in ("tok_embed", "final_norm", "lm_head"))
        self._arrays = []
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down"):
            arr = (C.c_void_p * L)(*[_ptr(t) for t in weights[name]])
            self._arrays.append(arr)
            setattr(w, name, arr)
        self._w = w
        self.h = lib().orc_create(C.byref(self.cfg), C.byref(w))
        if not self.h:
            raise MemoryError("orc_create failed")

    def close(self):
        if self.h:
            lib().orc_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    @property
    def length(self) -> int:
        return lib().orc_len(self.h)

    @length.setter
    def length(self, n: int):
        lib().orc_set_len(self.h, int(n))

    def forward(self, tokens, pos0: int, skip_mask=None, want_logits=True, want_hidden=False, head_rows=None):
        """Returns dict(logits [M][V], hidden [M][d], argmax [M], margin [M]) for the rows asked."""
        tok = _i32(tokens)
        M = tok.shape[0]
        V, d = self.shape.vocab, self.shape.d_model
        head_rows = M if head_rows is None else head_rows
        logits = np.zeros((M, V), dtype=np.float32) if want_logits else None
        hidden = np.zeros((M, d), dtype=np.float32) if want_hidden else None
        am = np.full(M, -1, dtype=np.int32)
        mg = np.zeros(M, dtype=np.float32)
        mask = None if skip_mask is None else np.ascontiguousarray(np.asarray(skip_mask, dtype=np.uint8))
        rc = lib().orc_forward(self.h, _ptr(tok), M, int(pos0), _ptr(mask), _ptr(logits), _ptr(hidden),
                               _ptr(am), _ptr(mg), int(head_rows))
        if rc:
            raise ValueError(f"orc_forward rc={rc}")
        return {"logits": logits, "hidden": hidden, "argmax": am, "margin": mg}

    def prefill(self, prompt):
        tok = _i32(prompt)
        pooled = np.zeros(self.shape.d_model, dtype=np.float32)
        first, mg = C.c_int(), C.c_float()
        rc = lib().orc_prefill(self.h, _ptr(tok), tok.shape[0], _ptr(pooled), C.byref(first), C.byref(mg))
        if rc:
            raise ValueError(f"orc_prefill rc={rc}")
        return pooled, first.value, mg.value

    def generate(self, first_token: int, max_new: int, k: int, skip_mask=None):
        out = np.zeros(max_new, dtype=np.int32)
        cap = max_new + 1
        acc = np.full(cap, -1, dtype=np.int32)
        drafts = np.full((cap, max(k, 1)), -1, dtype=np.int32)
        st = Stats()
        mask = None if skip_mask is None else np.ascontiguousarray(np.asarray(skip_mask, dtype=np.uint8))
        rc = lib().orc_generate(self.h, int(first_token), int(max_new), int(k), _ptr(mask), _ptr(out),
                                C.byref(st), _ptr(acc), _ptr(drafts) if k > 0 else None, cap)
        if rc:
            raise ValueError(f"orc_generate rc={rc}")
        return {"tokens": out, "accepts": acc[:st.rounds].copy(), "drafts": drafts[:st.rounds, :k].copy(),
                "rounds": st.rounds, "drafted": st.drafted, "accepted": st.accepted,
                "min_margin": st.min_margin}

    def greedy_full(self, first_token: int, max_new: int):
        out = np.zeros(max_new, dtype=np.int32)
        mm = C.c_float()
        rc = lib().orc_greedy_full(self.h, int(first_token), int(max_new), _ptr(out), C.byref(mm))
        if rc:
            raise ValueError(f"orc_greedy_full rc={rc}")
        return out, mm.value


def linear(W: torch.Tensor, x: np.ndarray) -> np.ndarray:
    """y = x . W^T with fp64 accumulation; W a CPU torch tensor (fp32 or bf16) [n_out][n_in], x fp32 [M][n_in]."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    M, n_in = x.shape
    n_out = W.shape[0]
    assert W.shape[1] == n_in and M <= 64
    y = np.zeros((M, n_out), dtype=np.float32)
    lib().orc_linear(_ptr(W), 0 if W.dtype == torch.float32 else 1, n_out, n_in, _ptr(x), M, _ptr(y))
    return y


def pool_mean(hidden: np.ndarray) -> np.ndarray:
    hidden = np.ascontiguousarray(hidden, dtype=np.float32)
    T, d = hidden.shape
    v = np.zeros(d, dtype=np.float32)
    lib().orc_pool_mean(_ptr(hidden), T, d, _ptr(v))
    return v


def knn_select(v, anchors, n_domains: int, per_domain: int):
    """(domain, anchor, cosine) or None for a degenerate (zero / non-finite norm) input."""
    v = np.ascontiguousarray(np.asarray(v, dtype=np.float32))
    a = np.ascontiguousarray(np.asarray(anchors, dtype=np.float32))
    assert a.shape == (n_domains * per_domain, v.shape[0])
    dom, anc, cs = C.c_int(), C.c_int(), C.c_float()
    rc = lib().orc_knn_select(_ptr(v), _ptr(a), n_domains, per_domain, v.shape[0],
                              C.byref(dom), C.byref(anc), C.byref(cs))
    return None if rc else (dom.value, anc.value, cs.value)


def accept(draft: Sequence[int], target: Sequence[int]):
    d, t = _i32(draft), _i32(target)
    assert t.shape[0] == d.shape[0] + 1
    a, nx = C.c_int(), C.c_int()
    lib().orc_accept(_ptr(d) if d.shape[0] else None, _ptr(t), d.shape[0], C.byref(a), C.byref(nx))
    return a.value, nx.value
