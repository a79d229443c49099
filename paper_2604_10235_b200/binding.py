"""ctypes binding of libcodecomp.so: argument marshalling only.

Every function here has the name of the C entry point it forwards to (see
``include/codecomp.h`` for what each computes); tensors are ``torch`` CUDA tensors whose
``data_ptr()`` is handed to the library, and the work is enqueued on torch's current
stream.  There is no CPU implementation behind these calls: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

CC_OK = 0
CC_ERR_INVALID_ARG, CC_ERR_UNSUPPORTED, CC_ERR_WORKSPACE, CC_ERR_CUDA = -1, -2, -3, -4
CC_ERR_TIMEOUT, CC_ERR_DEVICE_FLAG = -5, -6
CC_BF16 = 1
CC_F32 = 2
CC_MODE_BF16, CC_MODE_FP32 = 0, 1
CC_POOL_NONE, CC_POOL_MAX, CC_POOL_AVG = 0, 1, 2
CC_MAX_SEQS = 64
CC_FILL_ATTENTION, CC_FILL_NEAREST = 0, 1

EXPORTS = ("cc_create", "cc_destroy", "cc_status_string", "cc_last_error", "cc_poll_status",
           "cc_workspace_bytes", "cc_score_window", "cc_fuse_prior_pool", "cc_topk_select",
           "cc_compact_kv", "cc_compress_layer", "cc_workspace_views", "cc_topk_select_static",
           "cc_structural_score", "cc_plan_budgets", "cc_select_spans", "cc_ppl_chunk_scores",
           "cc_select_chunks", "cc_exp_rate_probe", "cc_compress_layers")
CC_STATIC_SELECT_MAX_ITEMS = 1 << 20


class CodecompError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"libcodecomp status {status}: {text}")
        self.status = status


class cc_layer_desc(C.Structure):
    _fields_ = [
        ("n_heads_q", C.c_int32), ("n_heads_kv", C.c_int32), ("head_dim", C.c_int32),
        ("window", C.c_int32), ("dtype", C.c_int32), ("compute_mode", C.c_int32),
        ("pool_kind", C.c_int32), ("pool_size", C.c_int32), ("chunk_size", C.c_int32),
        ("alpha", C.c_float), ("beta", C.c_float), ("force_threshold", C.c_float),
        ("span_ratio", C.c_double), ("span_min", C.c_int32),
        ("n", C.c_int32), ("budget", C.c_int32),
        ("q_stride_seq", C.c_int64), ("q_stride_row", C.c_int64), ("q_stride_head", C.c_int64),
        ("kv_stride_tok", C.c_int64), ("kv_stride_head", C.c_int64),
        ("out_stride_tok", C.c_int64), ("out_stride_head", C.c_int64),
        ("num_seqs", C.c_int32), ("page_size", C.c_int32),
        ("seq_lens", C.POINTER(C.c_int32)), ("budgets", C.POINTER(C.c_int32)),
        ("page_table", C.c_void_p),
        ("page_table_stride", C.c_int32), ("pool_pages", C.c_int32),
        ("out_page_table_stride", C.c_int32),
        ("causal", C.c_int32), ("fill_mode", C.c_int32),
    ]


_LIB = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads (building first if the sources are newer) the in-tree shared library."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    if path is None:
        path = _build.LIB_PATH
        if not os.path.exists(path) or _build._stale():
            try:
                _build.build()
            except Exception as exc:                      # no nvcc: a stale library is still usable
                if not os.path.exists(path):
                    raise RuntimeError(f"libcodecomp.so is missing and cannot be built: {exc}")
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    dp = C.POINTER(cc_layer_desc)
    lib.cc_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.cc_destroy.argtypes = [vp]
    lib.cc_status_string.argtypes = [C.c_int]
    lib.cc_status_string.restype = C.c_char_p
    lib.cc_last_error.argtypes = [vp]
    lib.cc_last_error.restype = C.c_char_p
    lib.cc_poll_status.argtypes = [vp, vp, C.POINTER(C.c_int)]
    lib.cc_workspace_bytes.argtypes = [vp, dp]
    lib.cc_workspace_bytes.restype = sz
    lib.cc_score_window.argtypes = [vp, dp, vp, vp, vp, vp, vp, sz, vp]
    lib.cc_fuse_prior_pool.argtypes = [vp, dp, vp, vp, vp, vp]
    lib.cc_topk_select.argtypes = [vp, dp, vp, vp, vp, vp, vp, sz, vp]
    lib.cc_topk_select_static.argtypes = [vp, dp, vp, vp, vp, vp, vp]
    lib.cc_structural_score.argtypes = [vp, dp, vp, vp, C.c_float, vp, vp, vp]
    lib.cc_compact_kv.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.cc_ppl_chunk_scores.argtypes = [vp, vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64,
                                        C.c_int64, vp, vp, vp, vp]
    lib.cc_select_chunks.argtypes = [vp, vp, C.c_int32, C.c_int32, vp, vp]
    lib.cc_plan_budgets.argtypes = [vp, vp, C.c_int32, C.POINTER(cc_budget_params), vp, vp]
    lib.cc_select_spans.argtypes = [vp, vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, C.c_double,
                                    C.c_int32, vp, vp, vp]
    lib.cc_compress_layer.argtypes = [vp, dp] + [vp] * 10 + [vp, sz, vp]
    lib.cc_exp_rate_probe.argtypes = [vp, C.c_int32, C.c_int32, C.POINTER(C.c_double), vp]
    lib.cc_compress_layers.argtypes = [vp, dp, C.c_int32] + [vp] * 3 + [vp] + [vp] * 6 + [vp, sz, vp]
    lib.cc_workspace_views.argtypes = [vp, dp, vp, C.POINTER(vp), C.POINTER(vp)]
    for name in EXPORTS:
        if name not in ("cc_status_string", "cc_last_error", "cc_workspace_bytes"):
            getattr(lib, name).restype = C.c_int
    if path == _build.LIB_PATH:
        _LIB = lib
    return lib


class cc_budget_params(C.Structure):
    _fields_ = [("r", C.c_double), ("r_max", C.c_double), ("m_min", C.c_double),
                ("m_max", C.c_double), ("eps", C.c_double)]


class Context:
    """Owns a ``cc_ctx`` (one per stream / thread)."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("libcodecomp needs a CUDA device; there is no CPU path")
        torch.cuda.init()
        self.device = device
        h = C.c_void_p()
        rc = self.lib.cc_create(C.byref(h), device)
        if rc != CC_OK:
            raise CodecompError(rc, self.lib.cc_status_string(rc).decode())
        self.handle = h

    def close(self) -> None:
        if getattr(self, "handle", None):
            self.lib.cc_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self, rc: int) -> None:
        if rc != CC_OK:
            raise CodecompError(rc, self.lib.cc_last_error(self.handle).decode() or
                                self.lib.cc_status_string(rc).decode())

    def workspace_bytes(self, desc: "Desc") -> int:
        n = self.lib.cc_workspace_bytes(self.handle, C.byref(desc.c))
        if n == 0:
            raise CodecompError(CC_ERR_INVALID_ARG, self.lib.cc_last_error(self.handle).decode())
        return int(n)

    def workspace(self, desc: "Desc") -> torch.Tensor:
        return torch.empty(self.workspace_bytes(desc), dtype=torch.uint8,
                           device=f"cuda:{self.device}")

    def poll(self, stream: Optional[int] = None) -> int:
        """Synchronises the stream and returns the device-side status (0 = ok)."""
        st = C.c_int(0)
        self.check(self.lib.cc_poll_status(self.handle, _stream(stream), C.byref(st)))
        return int(st.value)


class Desc:
    """A ``cc_layer_desc`` plus the host arrays it points to (kept alive here)."""

    def __init__(self, n_heads_q: int, n_heads_kv: int, window: int, *, n: int = 0,
                 budget: int = 0, seq_lens: Optional[Sequence[int]] = None,
                 budgets: Optional[Sequence[int]] = None, head_dim: int = 128,
                 compute_mode: int = CC_MODE_BF16, pool_kind: int = CC_POOL_MAX,
                 pool_size: int = 7, chunk_size: int = 1, alpha: float = 1.0, beta: float = 0.0,
                 force_threshold: float = math.inf, span_ratio: float = 0.0, span_min: int = 0,
                 page_size: int = 0, page_table: Optional[torch.Tensor] = None, pool_pages: int = 0,
                 out_page_table_stride: int = 0, causal: bool = False, fill_mode: int = 0,
                 q_strides=None,
                 kv_strides=None,
                 out_strides=(0, 0)):
        c = cc_layer_desc()
        c.n_heads_q, c.n_heads_kv, c.head_dim, c.window = n_heads_q, n_heads_kv, head_dim, window
        c.dtype, c.compute_mode = CC_BF16, compute_mode
        c.pool_kind, c.pool_size, c.chunk_size = pool_kind, pool_size, chunk_size
        c.alpha, c.beta, c.force_threshold = alpha, beta, force_threshold
        c.span_ratio, c.span_min = span_ratio, span_min
        c.n, c.budget = n, budget
        if q_strides is None:
            q_strides = (window * n_heads_q * head_dim, n_heads_q * head_dim, head_dim)
        if kv_strides is None:
            kv_strides = (n_heads_kv * head_dim, head_dim)
        c.q_stride_seq, c.q_stride_row, c.q_stride_head = q_strides
        c.kv_stride_tok, c.kv_stride_head = kv_strides
        c.out_stride_tok, c.out_stride_head = out_strides
        self._keep = []
        if seq_lens is not None:
            lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
            buds = np.ascontiguousarray(budgets, dtype=np.int32)
            assert lens.shape == buds.shape and lens.ndim == 1
            self._keep += [lens, buds]
            c.num_seqs = len(lens)
            c.seq_lens = lens.ctypes.data_as(C.POINTER(C.c_int32))
            c.budgets = buds.ctypes.data_as(C.POINTER(C.c_int32))
        c.page_size = page_size
        if page_table is not None:
            assert page_table.dtype == torch.int32 and page_table.is_cuda and page_table.is_contiguous()
            self._keep.append(page_table)
            c.page_table = page_table.data_ptr()
            c.page_table_stride = page_table.shape[-1]
        c.pool_pages = pool_pages
        c.out_page_table_stride = out_page_table_stride
        c.causal = 1 if causal else 0
        c.fill_mode = fill_mode
        self.c = c

    # sizes the caller needs to allocate outputs
    @property
    def lens(self):
        return [int(x) for x in self._keep[0]] if self.c.num_seqs else [self.c.n]

    @property
    def buds(self):
        return [int(x) for x in self._keep[1]] if self.c.num_seqs else [self.c.budget]

    @property
    def n_tot(self) -> int:
        return sum(self.lens)

    @property
    def b_tot(self) -> int:
        return sum(self.buds)

    @property
    def m_tot(self) -> int:
        ch = max(1, self.c.chunk_size)
        return sum((n + ch - 1) // ch for n in self.lens)


def _stream(stream: Optional[int]) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    return C.c_void_p(stream)


def _ptr(t: Optional[torch.Tensor], pinned_ok: bool = False) -> C.c_void_p:
    """Address of a CUDA tensor; with ``pinned_ok`` also of a page-locked host tensor (its address
    is valid on the device: the V rows of a compaction may be gathered straight from it)."""
    if t is None:
        return C.c_void_p(0)
    if not t.is_cuda and not (pinned_ok and t.is_pinned()):
        raise ValueError("libcodecomp takes CUDA tensors only" +
                         (" (or page-locked host memory here)" if pinned_ok else ""))
    return C.c_void_p(t.data_ptr())


def cc_score_window(ctx: Context, desc: Desc, q_win, k, scores, lse=None, ws=None, stream=None):
    ws = ctx.workspace(desc) if ws is None else ws
    ctx.check(ctx.lib.cc_score_window(ctx.handle, C.byref(desc.c), _ptr(q_win), _ptr(k),
                                      _ptr(scores), _ptr(lse), _ptr(ws), ws.numel(),
                                      _stream(stream)))


def cc_fuse_prior_pool(ctx: Context, desc: Desc, scores, prior, fused, stream=None):
    ctx.check(ctx.lib.cc_fuse_prior_pool(ctx.handle, C.byref(desc.c), _ptr(scores), _ptr(prior),
                                         _ptr(fused), _stream(stream)))


def cc_topk_select(ctx: Context, desc: Desc, fused, prior, idx, count, ws=None, stream=None):
    ws = ctx.workspace(desc) if ws is None else ws
    ctx.check(ctx.lib.cc_topk_select(ctx.handle, C.byref(desc.c), _ptr(fused), _ptr(prior),
                                     _ptr(idx), _ptr(count), _ptr(ws), ws.numel(),
                                     _stream(stream)))


def cc_topk_select_static(ctx: Context, desc: Desc, fused, prior, idx, count, stream=None):
    """cc_topk_select without a workspace: for callers that cannot allocate device memory when
    they need a selection.  The kernel's flag scratch is a fixed array inside the library
    (CC_STATIC_SELECT_MAX_ITEMS bytes per GPU, shared by every call, so overlapping calls must
    be ordered by the caller); larger batches raise CodecompError(CC_ERR_UNSUPPORTED).  The
    first call on a device resolves the array's address and belongs outside stream capture."""
    ctx.check(ctx.lib.cc_topk_select_static(ctx.handle, C.byref(desc.c), _ptr(fused), _ptr(prior),
                                            _ptr(idx), _ptr(count), _stream(stream)))


def cc_compact_kv(ctx: Context, desc: Desc, k, v, idx, k_out, v_out, free_pages=None,
                  out_page_table=None, stream=None):
    ctx.check(ctx.lib.cc_compact_kv(ctx.handle, C.byref(desc.c), _ptr(k, True), _ptr(v, True), _ptr(idx),
                                    _ptr(k_out), _ptr(v_out), _ptr(free_pages),
                                    _ptr(out_page_table), _stream(stream)))


def cc_structural_score(ctx: Context, desc: Desc, idx, prior, threshold: float, score,
                        counts=None, stream=None):
    ctx.check(ctx.lib.cc_structural_score(ctx.handle, C.byref(desc.c), _ptr(idx), _ptr(prior),
                                          C.c_float(threshold), _ptr(score), _ptr(counts),
                                          _stream(stream)))


def cc_ppl_chunk_scores(ctx: Context, logits: torch.Tensor, targets: torch.Tensor,
                        nll: torch.Tensor, score: torch.Tensor, stream=None):
    """logits [chunks][T][V] (bf16 or f32, last dimension contiguous), targets i32 [T]."""
    chunks, t, v = logits.shape
    assert logits.stride(2) == 1
    dtype = CC_F32 if logits.dtype == torch.float32 else CC_BF16
    ctx.check(ctx.lib.cc_ppl_chunk_scores(ctx.handle, _ptr(logits), dtype, chunks, t, v,
                                          logits.stride(0), logits.stride(1), _ptr(targets),
                                          _ptr(nll), _ptr(score), _stream(stream)))


def cc_select_chunks(ctx: Context, score: torch.Tensor, k: int, chosen: torch.Tensor, stream=None):
    ctx.check(ctx.lib.cc_select_chunks(ctx.handle, _ptr(score), score.numel(), k, _ptr(chosen),
                                       _stream(stream)))


def _host(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def cc_plan_budgets(sigma, lens, r: float, r_max: float = 1.0, m_min: float = 0.5,
                    m_max: float = 1.5, eps: float = 1e-6, lib=None):
    """Host call (no GPU): per-chunk budgets and capacity multipliers (numpy arrays)."""
    lib = lib or load_library()
    sigma = np.ascontiguousarray(sigma, dtype=np.float64)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    budgets = np.zeros(len(sigma), dtype=np.int32)
    mult = np.zeros(len(sigma), dtype=np.float64)
    p = cc_budget_params(r, r_max, m_min, m_max, eps)
    rc = lib.cc_plan_budgets(_host(sigma), _host(lens), len(sigma), C.byref(p), _host(budgets),
                             _host(mult))
    if rc != CC_OK:
        raise CodecompError(rc, lib.cc_status_string(rc).decode())
    return budgets, mult


def cc_select_spans(starts, ends, scores, protected, n: int, budget: int, span_ratio: float,
                    span_min: int, lib=None):
    """Host call (no GPU): prior mask [n] of the tokens covered by the selected spans and the
    indices of the spans in the order taken."""
    lib = lib or load_library()
    starts = np.ascontiguousarray(starts, dtype=np.int32)
    ends = np.ascontiguousarray(ends, dtype=np.int32)
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    prot = np.ascontiguousarray(protected, dtype=np.uint8)
    mask = np.zeros(max(n, 1), dtype=np.float32)
    taken = np.zeros(max(len(starts), 1), dtype=np.int32)
    count = C.c_int32(0)
    rc = lib.cc_select_spans(_host(starts), _host(ends), _host(scores), _host(prot), len(starts), n,
                             budget, span_ratio, span_min, _host(mask), _host(taken),
                             C.cast(C.byref(count), C.c_void_p))
    if rc != CC_OK:
        raise CodecompError(rc, lib.cc_status_string(rc).decode())
    return mask[:n], taken[:count.value]


def cc_compress_layer(ctx: Context, desc: Desc, q_win, k, v, prior, k_out, v_out, idx, count,
                      free_pages=None, out_page_table=None, ws=None, stream=None):
    ws = ctx.workspace(desc) if ws is None else ws
    ctx.check(ctx.lib.cc_compress_layer(ctx.handle, C.byref(desc.c), _ptr(q_win), _ptr(k), _ptr(v, True),
                                        _ptr(prior), _ptr(k_out), _ptr(v_out), _ptr(idx),
                                        _ptr(count), _ptr(free_pages), _ptr(out_page_table),
                                        _ptr(ws), ws.numel(), _stream(stream)))


def cc_exp_rate_probe(ctx: Context, from_tmem: bool, iters: int = 4000, stream=None) -> float:
    """Values per clock per SM of the score kernel's inner loop run alone (synchronises)."""
    rate = C.c_double(0.0)
    ctx.check(ctx.lib.cc_exp_rate_probe(ctx.handle, 1 if from_tmem else 0, iters, C.byref(rate),
                                        _stream(stream)))
    return float(rate.value)


def _ptr_array(tensors):
    """Host array of the device pointers of a list of tensors (None -> NULL array)."""
    if tensors is None:
        return None
    arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    return arr


def cc_compress_layers(ctx: Context, desc: Desc, q_win, k, v, prior, k_out, v_out, idx, count,
                       free_pages=None, out_page_table=None, ws=None, stream=None):
    """cc_compress_layer for a list of layers in one call: every tensor argument except ``prior``
    and ``ws`` is a list with one tensor per layer."""
    ws = ctx.workspace(desc) if ws is None else ws
    n = len(k)
    arrays = [_ptr_array(x) for x in (q_win, k, v)]
    outs = [_ptr_array(x) for x in (k_out, v_out, idx, count, free_pages, out_page_table)]
    ctx.check(ctx.lib.cc_compress_layers(ctx.handle, C.byref(desc.c), n, *arrays, _ptr(prior), *outs,
                                         _ptr(ws), ws.numel(), _stream(stream)))


def cc_workspace_views(ctx: Context, desc: Desc, ws: torch.Tensor):
    """Views of the intermediate scores / fused values inside a workspace tensor."""
    s, f = C.c_void_p(), C.c_void_p()
    ctx.check(ctx.lib.cc_workspace_views(ctx.handle, C.byref(desc.c), _ptr(ws), C.byref(s),
                                         C.byref(f)))
    base = ws.data_ptr()
    hkv = desc.c.n_heads_kv
    so, fo = s.value - base, f.value - base
    scores = ws[so:so + 4 * hkv * desc.n_tot].view(torch.float32).view(hkv, desc.n_tot)
    fused = ws[fo:fo + 4 * hkv * desc.m_tot].view(torch.float32).view(hkv, desc.m_tot)
    return scores, fused
