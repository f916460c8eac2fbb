"""Thin ctypes binding of libknnssd.so: argument marshalling only.

The functions and the ``Session`` methods carry the names of the C ABI
(``include/knnssd.h``).  torch is used for device memory and streams; every step
of the path runs in the library's CUDA kernels.  There is no CPU fallback: if the
library cannot be loaded the import of this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libknnssd.so")

STATUS = {0: "OK", 1: "ERR_INVALID_ARG", 2: "ERR_SHAPE", 3: "ERR_CAPACITY", 4: "ERR_STATE",
          5: "ERR_DEGENERATE", 6: "ERR_CUDA", 7: "ERR_TIMEOUT"}

EXPORTS = ["knnssd_init", "knnssd_destroy", "knnssd_prefill", "knnssd_select_skipset", "knnssd_set_skipmask",
           "knnssd_draft", "knnssd_verify", "knnssd_generate", "knnssd_decode", "knnssd_get_launch_count", "knnssd_get_length", "knnssd_set_length",
           "knnssd_set_pending", "knnssd_mask_objective", "knnssd_get_stats", "knnssd_last_error", "knnssd_time_pass", "knnssd_trace_pass", "knnssd_linear",
           "knnssd_gemm_split", "knnssd_linear_tc", "knnssd_build_anchors", "knnssd_cosine_top1", "knnssd_cosine_top1_static",
           "knnssd_debug_barrier_timeout", "knnssd_filtered_probs", "knnssd_sample_token", "knnssd_spec_accept",
           "knnssd_decode_sampled"]


class KnnssdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"knnssd: {STATUS.get(status, status)}: {message}")
        self.status = status


class Config(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff",
                                       "vocab", "max_seq", "max_draft")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int) for n in ("dtype", "n_domains", "anchors_per_domain", "pool_mode")]


class Weights(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo",
                                                     "mlp_norm", "w_gate", "w_up", "w_down")]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("rounds", "drafted", "accepted", "tokens")] + \
               [(n, C.c_float) for n in ("ms_prefill", "ms_select", "ms_draft", "ms_verify")]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_16162_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    P, I, F = C.c_void_p, C.c_int, C.c_float
    PI, PF = C.POINTER(C.c_int), C.POINTER(C.c_float)
    sigs = {
        "knnssd_init": (I, [C.POINTER(Config), C.POINTER(Weights), P, P, P, C.POINTER(P)]),
        "knnssd_destroy": (None, [P]),
        "knnssd_prefill": (I, [P, P, I, P, PI]),
        "knnssd_select_skipset": (I, [P, P, PI, PI, PF]),
        "knnssd_set_skipmask": (I, [P, P]),
        "knnssd_draft": (I, [P, I, P, P]),
        "knnssd_verify": (I, [P, P, I, PI, PI, P, P]),
        "knnssd_generate": (I, [P, P, I, I, I, I, P, PI, P, PI, C.POINTER(Stats)]),
        "knnssd_decode": (I, [P, I, I, I, P, PI, P, PI, C.POINTER(Stats)]),
        "knnssd_get_launch_count": (C.c_longlong, [P]),
        "knnssd_get_length": (I, [P]),
        "knnssd_set_length": (I, [P, I]),
        "knnssd_set_pending": (I, [P, I]),
        "knnssd_mask_objective": (I, [P, P, I, P, P, I, I, I, P, P, P]),
        "knnssd_get_stats": (I, [P, C.POINTER(Stats)]),
        "knnssd_last_error": (C.c_char_p, [P]),
        "knnssd_time_pass": (I, [P, I, I, I, PF, PI, PF, PI]),
        "knnssd_trace_pass": (I, [P, I, I, I, PI, PI, PF, PF, PI]),
        "knnssd_linear": (I, [P, I, I, I, P, I, P, P]),
        "knnssd_gemm_split": (I, [P, P, I, I, P, I, I, P, P]),
        "knnssd_build_anchors": (I, [P, I, I, I, P, I, I, P, P, P, PI, PF, P]),
        "knnssd_linear_tc": (I, [P, I, I, P, I, P, PF, P]),
        "knnssd_cosine_top1": (I, [P, P, I, I, PI, PF, P]),
        "knnssd_cosine_top1_static": (I, [P, P, I, I, PI, PF, P]),
        "knnssd_debug_barrier_timeout": (I, [P, C.c_uint]),
        "knnssd_filtered_probs": (I, [P, I, I, F, F, P, P]),
        "knnssd_sample_token": (I, [P, I, F, PI, P]),
        "knnssd_spec_accept": (I, [P, P, P, I, I, P, F, PI, PI, P]),
        "knnssd_decode_sampled": (I, [P, I, I, F, F, P, I, P, PI, P, C.POINTER(Stats)]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


_lib = _load()


def _dev_ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _host_i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    return None if stream is None else stream.cuda_stream


def knnssd_linear(W: torch.Tensor, x: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """y = x @ W^T through the weight-streaming kernel.  W [n_out][n_in] fp32/bf16, x fp32 [M][n_in]."""
    dtype = {torch.float32: 0, torch.bfloat16: 1}[W.dtype]
    M, n_in = x.shape
    n_out = W.shape[0]
    y = torch.empty((M, n_out), dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        cur = torch.cuda.current_stream() if stream is None else stream
        rc = _lib.knnssd_linear(_dev_ptr(W), dtype, n_out, n_in, _dev_ptr(x, torch.float32), M, _dev_ptr(y),
                                cur.cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_linear")
    return y


def knnssd_gemm_split(W0: torch.Tensor, x: torch.Tensor, mode: int = 0, W1: Optional[torch.Tensor] = None,
                      y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The prompt pass's tensor-core contraction over T rows.  W0 (and W1 for mode 2) bf16 [n_out][n_in], x fp32 [T][n_in].
    mode 0: y = x W0^T; 1: y += x W0^T (y given); 2: silu(x W0^T) * (x W1^T), rounded to two bf16 terms."""
    T, n_in = x.shape
    n_out = W0.shape[0]
    if y is None:
        y = torch.zeros((T, n_out), dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = _lib.knnssd_gemm_split(_dev_ptr(W0, torch.bfloat16), None if W1 is None else _dev_ptr(W1, torch.bfloat16), n_out, n_in,
                                    _dev_ptr(x, torch.float32), T, mode, _dev_ptr(y, torch.float32),
                                    torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_gemm_split")
    return y


def knnssd_linear_tc(W: torch.Tensor, x: torch.Tensor):
    """y = x @ W^T for up to 16 rows through the tensor-core weight-streaming kernel; returns (y, ms of its kernels)."""
    M, n_in = x.shape
    n_out = W.shape[0]
    y = torch.empty((M, n_out), dtype=torch.float32, device=x.device)
    ms = C.c_float()
    with torch.cuda.device(x.device):
        rc = _lib.knnssd_linear_tc(_dev_ptr(W, torch.bfloat16), n_out, n_in, _dev_ptr(x, torch.float32), M, _dev_ptr(y), C.byref(ms),
                                   torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_linear_tc")
    return y, ms.value


def knnssd_build_anchors(x: torch.Tensor, init_centroids: torch.Tensor, max_rounds: int, k: int):
    """Sec. 4.1: K-means over the rows of x (fp32 [N][d], CUDA) from ``init_centroids`` (fp32 [n][d]), then Eq. (2).
    Returns dict(labels int32 [N], centroids fp64 CUDA [n][d], anchors int32 [n][k], rounds, ms_rounds)."""
    N, d = x.shape
    n = init_centroids.shape[0]
    labels = np.zeros(N, dtype=np.int32)
    anchors = np.zeros((n, k), dtype=np.int32)
    mu = torch.empty((n, d), dtype=torch.float64, device=x.device)
    rounds, ms = C.c_int(), C.c_float()
    with torch.cuda.device(x.device):
        rc = _lib.knnssd_build_anchors(_dev_ptr(x, torch.float32), N, d, n, _dev_ptr(init_centroids, torch.float32), max_rounds, k,
                                       labels.ctypes.data, _dev_ptr(mu), anchors.ctypes.data, C.byref(rounds), C.byref(ms),
                                       torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_build_anchors")
    return {"labels": labels, "centroids": mu, "anchors": anchors, "rounds": rounds.value, "ms_rounds": ms.value}


def _check_query(query: torch.Tensor, anchors: torch.Tensor):
    # the C entry points get raw pointers and cannot see a query shorter than the anchors' rows
    if anchors.dim() != 2 or query.numel() != anchors.shape[1]:
        raise ValueError("anchors must be [n][d] and the query must hold d values")


def knnssd_cosine_top1(query: torch.Tensor, anchors: torch.Tensor):
    """(best flat index, cosine) of Eq. (4); raises KnnssdError(ERR_DEGENERATE) on zero / non-finite norms."""
    _check_query(query, anchors)
    n, d = anchors.shape
    best, cs = C.c_int(), C.c_float()
    with torch.cuda.device(query.device):
        rc = _lib.knnssd_cosine_top1(_dev_ptr(query, torch.float32), _dev_ptr(anchors, torch.float32), n, d,
                                     C.byref(best), C.byref(cs), torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_cosine_top1")
    return best.value, cs.value


def knnssd_filtered_probs(logits: torch.Tensor, temperature: float, top_p: float) -> torch.Tensor:
    """Temperature + nucleus filtering of logits [rows][vocab] (App. C.1's decoding settings); returns probabilities."""
    rows, V = logits.shape
    probs = torch.empty_like(logits)
    with torch.cuda.device(logits.device):
        rc = _lib.knnssd_filtered_probs(_dev_ptr(logits, torch.float32), rows, V, float(temperature), float(top_p), _dev_ptr(probs),
                                        torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_filtered_probs")
    return probs


def knnssd_sample_token(weights: torch.Tensor, u: float) -> int:
    """Inverse-CDF draw in token-id order from non-negative weights [vocab] with the uniform u."""
    tok = C.c_int()
    with torch.cuda.device(weights.device):
        rc = _lib.knnssd_sample_token(_dev_ptr(weights, torch.float32), weights.shape[0], float(u), C.byref(tok),
                                      torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_sample_token")
    return tok.value


def knnssd_spec_accept(p: torch.Tensor, q: Optional[torch.Tensor], drafts, u_accept, u_final: float):
    """One verification round of speculative sampling: (n_accepted, next_token).  p [k+1][V], q [k][V] filtered."""
    d = _host_i32(drafts)
    k = d.shape[0]
    ua = np.ascontiguousarray(np.asarray(u_accept, dtype=np.float32))
    if p.dim() != 2 or p.shape[0] != k + 1 or (k > 0 and (q is None or tuple(q.shape) != (k, p.shape[1]))) or ua.shape[0] != k:
        raise ValueError("p must be [k+1][V], q [k][V], drafts and u_accept [k]")
    a, nx = C.c_int(), C.c_int()
    with torch.cuda.device(p.device):
        rc = _lib.knnssd_spec_accept(_dev_ptr(p, torch.float32), _dev_ptr(q, torch.float32) if k else None,
                                     d.ctypes.data if k else None, k, p.shape[1], ua.ctypes.data if k else None, float(u_final),
                                     C.byref(a), C.byref(nx), torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_spec_accept")
    return a.value, nx.value


STATIC_MAX_ANCHORS = 4096


def knnssd_cosine_top1_static(query: torch.Tensor, anchors: torch.Tensor):
    """Same search and same result as ``knnssd_cosine_top1``, for callers that may not allocate device memory
    (a serving loop living inside a pre-sized pool, a process under a fixed memory reservation): the library keeps
    the per-anchor cosines in a fixed array of its own, so nothing is allocated or freed here either - the inputs
    are used in place and the two results come back as Python numbers.  At most ``STATIC_MAX_ANCHORS`` anchors
    (ERR_CAPACITY beyond that).  All calls on a GPU share that array: do not overlap them."""
    _check_query(query, anchors)
    n, d = anchors.shape
    best, cs = C.c_int(), C.c_float()
    with torch.cuda.device(query.device):
        rc = _lib.knnssd_cosine_top1_static(_dev_ptr(query, torch.float32), _dev_ptr(anchors, torch.float32), n, d,
                                            C.byref(best), C.byref(cs), torch.cuda.current_stream().cuda_stream)
    if rc:
        raise KnnssdError(rc, "knnssd_cosine_top1_static")
    return best.value, cs.value


class Session:
    """One model + one request at a time; wraps a knnssd_ctx.  ``weights`` is a dict of CUDA tensors with
    the keys of ``knnssd_weights`` (lists of per-layer tensors for the per-layer entries); they are borrowed,
    so this object keeps references to them."""

    def __init__(self, *, n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab, max_seq, max_draft,
                 rms_eps, rope_theta, dtype: str, weights: Dict[str, object],
                 anchors: Optional[torch.Tensor] = None, skip_masks=None, anchors_per_domain: int = 0,
                 pool_mode: int = 0, stream: Optional[torch.cuda.Stream] = None):
        self._keep = (weights, anchors)
        self.vocab, self.d_model, self.n_layers = vocab, d_model, n_layers
        self.device = weights["tok_embed"].device
        n_domains = 0
        masks_ptr = None
        if anchors is not None:
            n_domains = anchors.shape[0] // anchors_per_domain
            self._masks = np.ascontiguousarray(np.asarray(skip_masks, dtype=np.uint8))
            if self._masks.shape != (n_domains, 2 * n_layers):
                raise ValueError("skip_masks must be [n_domains][2*n_layers]")
            masks_ptr = self._masks.ctypes.data
        cfg = Config(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab, max_seq, max_draft,
                     rms_eps, rope_theta, {"fp32": 0, "bf16": 1}[dtype], n_domains, anchors_per_domain, pool_mode)
        w = Weights()
        w.tok_embed, w.final_norm, w.lm_head = (_dev_ptr(weights[k]) for k in ("tok_embed", "final_norm", "lm_head"))
        self._tables = []
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down"):
            arr = (C.c_void_p * n_layers)(*[_dev_ptr(t) for t in weights[name]])
            self._tables.append(arr)
            setattr(w, name, arr)
        self._stream = stream
        self.h = C.c_void_p()
        with torch.cuda.device(self.device):
            sh = (torch.cuda.current_stream() if stream is None else stream).cuda_stream
            rc = _lib.knnssd_init(C.byref(cfg), C.byref(w), _dev_ptr(anchors, torch.float32), masks_ptr, sh,
                                  C.byref(self.h))
        if rc:
            self.h = None
            raise KnnssdError(rc, "knnssd_init")

    @classmethod
    def from_shape(cls, shape, weights, max_seq, max_draft=8, **kw):
        return cls(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads,
                   n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ff=shape.d_ff, vocab=shape.vocab,
                   max_seq=max_seq, max_draft=max_draft, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                   dtype=shape.dtype, weights=weights, **kw)

    def _check(self, rc: int):
        if rc:
            raise KnnssdError(rc, _lib.knnssd_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            _lib.knnssd_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    # ---- the calls of the C ABI, same names ----
    def prefill(self, tokens, want_pooled: bool = False):
        tok = _host_i32(tokens)
        pooled = torch.empty(self.d_model, dtype=torch.float32, device=self.device) if want_pooled else None
        first = C.c_int()
        self._check(_lib.knnssd_prefill(self.h, tok.ctypes.data, tok.shape[0], _dev_ptr(pooled), C.byref(first)))
        return (first.value, pooled) if want_pooled else first.value

    def select_skipset(self, query: Optional[torch.Tensor] = None):
        dom, anc, cs = C.c_int(), C.c_int(), C.c_float()
        self._check(_lib.knnssd_select_skipset(self.h, _dev_ptr(query, torch.float32) if query is not None else None,
                                               C.byref(dom), C.byref(anc), C.byref(cs)))
        return dom.value, anc.value, cs.value

    def set_skipmask(self, mask):
        m = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
        if m.shape != (2 * self.n_layers,):
            raise ValueError("mask must have 2*n_layers entries")
        self._check(_lib.knnssd_set_skipmask(self.h, m.ctypes.data))

    def draft(self, k: int, want_logits: bool = False):
        out = np.zeros(max(k, 1), dtype=np.int32)
        logits = torch.empty((k, self.vocab), dtype=torch.float32, device=self.device) if want_logits else None
        self._check(_lib.knnssd_draft(self.h, k, out.ctypes.data, _dev_ptr(logits)))
        return (out[:k], logits) if want_logits else out[:k]

    def verify(self, draft_tokens, want_logits: bool = False, want_hidden: bool = False):
        d = _host_i32(draft_tokens)
        k = d.shape[0]
        logits = torch.empty((k + 1, self.vocab), dtype=torch.float32, device=self.device) if want_logits else None
        hidden = torch.empty((k + 1, self.d_model), dtype=torch.float32, device=self.device) if want_hidden else None
        a, nx = C.c_int(), C.c_int()
        self._check(_lib.knnssd_verify(self.h, d.ctypes.data if k else None, k, C.byref(a), C.byref(nx),
                                       _dev_ptr(logits), _dev_ptr(hidden)))
        return {"n_accepted": a.value, "next_token": nx.value, "logits": logits, "hidden": hidden}

    def generate(self, prompt, max_new: int, k: int, use_selection: bool = False):
        p = _host_i32(prompt)
        out = np.zeros(max_new, dtype=np.int32)
        acc = np.full(max_new, -1, dtype=np.int32)
        n_out, dom, st = C.c_int(), C.c_int(), Stats()
        self._check(_lib.knnssd_generate(self.h, p.ctypes.data, p.shape[0], max_new, k, int(use_selection),
                                         out.ctypes.data, C.byref(n_out), acc.ctypes.data, C.byref(dom), C.byref(st)))
        return {"tokens": out[:n_out.value], "accepts": acc[:st.rounds].copy(), "domain": dom.value,
                "stats": {f: getattr(st, f) for f, _ in Stats._fields_}}

    def decode(self, max_new: int, k: int, use_selection: bool = False):
        out = np.zeros(max_new, dtype=np.int32)
        acc = np.full(max_new, -1, dtype=np.int32)
        n_out, dom, st = C.c_int(), C.c_int(), Stats()
        self._check(_lib.knnssd_decode(self.h, max_new, k, int(use_selection), out.ctypes.data, C.byref(n_out),
                                       acc.ctypes.data, C.byref(dom), C.byref(st)))
        return {"tokens": out[:n_out.value], "accepts": acc[:st.rounds].copy(), "domain": dom.value,
                "stats": {f: getattr(st, f) for f, _ in Stats._fields_}}

    def decode_sampled(self, max_new: int, k: int, temperature: float, top_p: float, uniforms):
        """Sampled draft-and-verify loop; ``uniforms``: (max_new - 1) * (2k + 1) values in [0, 1), layout as in the header."""
        u = np.ascontiguousarray(np.asarray(uniforms, dtype=np.float32))
        out = np.zeros(max_new, dtype=np.int32)
        acc = np.full(max_new, -1, dtype=np.int32)
        n_out, st = C.c_int(), Stats()
        self._check(_lib.knnssd_decode_sampled(self.h, max_new, k, float(temperature), float(top_p), u.ctypes.data, u.shape[0],
                                               out.ctypes.data, C.byref(n_out), acc.ctypes.data, C.byref(st)))
        return {"tokens": out[:n_out.value], "accepts": acc[:st.rounds].copy(),
                "stats": {f: getattr(st, f) for f, _ in Stats._fields_}}

    @property
    def launch_count(self) -> int:
        return _lib.knnssd_get_launch_count(self.h)

    @property
    def length(self) -> int:
        return _lib.knnssd_get_length(self.h)

    def set_length(self, n: int):
        self._check(_lib.knnssd_set_length(self.h, int(n)))

    def set_pending(self, token: int):
        self._check(_lib.knnssd_set_pending(self.h, int(token)))

    def mask_objective(self, masks, prompts, max_new: int, k: int):
        """Eq. (3)'s objective for each candidate mask over the given sample prompts: (ms per verified token [n_masks],
        accepted [n_masks], drafted [n_masks])."""
        m = np.ascontiguousarray(np.asarray(masks, dtype=np.uint8))
        lens = _host_i32([len(p) for p in prompts])
        toks = _host_i32(np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts]))
        n = m.shape[0]
        ms = np.zeros(n, dtype=np.float32)
        acc, drf = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.int32)
        self._check(_lib.knnssd_mask_objective(self.h, m.ctypes.data, n, toks.ctypes.data, lens.ctypes.data, len(prompts), max_new, k,
                                               ms.ctypes.data, acc.ctypes.data, drf.ctypes.data))
        return ms, acc, drf

    def debug_barrier_timeout(self, spin_limit: int = 4000):
        """Makes one bounded grid-barrier wait run out (test hook); raises KnnssdError(ERR_TIMEOUT)."""
        self._check(_lib.knnssd_debug_barrier_timeout(self.h, int(spin_limit)))

    def get_stats(self):
        st = Stats()
        self._check(_lib.knnssd_get_stats(self.h, C.byref(st)))
        return {f: getattr(st, f) for f, _ in Stats._fields_}

    def trace_pass(self, which: int, k: int, cap: int = 512):
        """Per-operation (type, layer, us of work, us at the barrier) of one pass, as stamped by CTA 0."""
        ty, ly = (C.c_int * cap)(), (C.c_int * cap)()
        uw, ub = (C.c_float * cap)(), (C.c_float * cap)()
        n = C.c_int()
        self._check(_lib.knnssd_trace_pass(self.h, which, k, cap, ty, ly, uw, ub, C.byref(n)))
        return [(ty[i], ly[i], uw[i], ub[i]) for i in range(n.value)]

    def time_pass(self, which: int, k: int, iters: int):
        ms, n, msl, nl = C.c_float(), C.c_int(), C.c_float(), C.c_int()
        self._check(_lib.knnssd_time_pass(self.h, which, k, iters, C.byref(ms), C.byref(n), C.byref(msl), C.byref(nl)))
        return {"ms_per_pass": ms.value, "launches": n.value, "ms_linear": msl.value, "linear_launches": nl.value}
