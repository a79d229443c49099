"""User-facing wrapper: compress one layer's KV cache starting from host or device tensors.

``LayerCompressor`` owns the device buffers (inputs, outputs, workspace) for one layer
geometry so that repeated calls allocate nothing, and forwards to ``cc_compress_layer``.
All arithmetic happens in libcodecomp's kernels; this file only moves bytes.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from dataclasses import dataclass, fields
from typing import Tuple

from . import binding as cc


@dataclass(frozen=True)
class LayerSpec:
    """Geometry and settings of one layer's compression step (what ``cc_layer_desc`` holds,
    minus pointers): heads, window, pooling, prior fusion, protection and its cap, the
    sequences of the batch with their budgets, and the K/V layout."""

    n_heads_q: int
    n_heads_kv: int
    window: int
    lens: Tuple[int, ...]                 # tokens per sequence
    budgets: Tuple[int, ...]              # tokens kept per KV head, per sequence
    head_dim: int = 128
    pool_kind: int = cc.CC_POOL_MAX
    pool_size: int = 7
    chunk_size: int = 1
    alpha: float = 1.0
    beta: float = 0.0
    force_threshold: float = float("inf")
    span_ratio: float = 0.0
    span_min: int = 0
    page_size: int = 0                    # 0 = contiguous K/V
    causal: bool = False
    fill_mode: int = cc.CC_FILL_ATTENTION

    @classmethod
    def like(cls, obj) -> "LayerSpec":
        """A spec with the values of the equally named attributes of ``obj`` (any object that
        describes a layer: a benchmark workload, a model configuration, ...)."""
        kw = {f.name: getattr(obj, f.name) for f in fields(cls) if hasattr(obj, f.name)}
        kw["lens"], kw["budgets"] = tuple(kw["lens"]), tuple(kw["budgets"])
        return cls(**kw)

    @property
    def group(self) -> int:
        return self.n_heads_q // self.n_heads_kv


def desc_from_spec(wl: LayerSpec, mode: int = cc.CC_MODE_BF16,
                   page_table: Optional[torch.Tensor] = None, pool_pages: int = 0,
                   out_pt_stride: int = 0) -> cc.Desc:
    kw = dict(head_dim=wl.head_dim, compute_mode=mode, pool_kind=wl.pool_kind,
              pool_size=wl.pool_size, chunk_size=wl.chunk_size, alpha=wl.alpha, beta=wl.beta,
              force_threshold=wl.force_threshold, span_ratio=wl.span_ratio, span_min=wl.span_min,
              page_size=wl.page_size, page_table=page_table, pool_pages=pool_pages,
              out_page_table_stride=out_pt_stride, causal=wl.causal, fill_mode=wl.fill_mode)
    if len(wl.lens) > 1 or wl.page_size:
        return cc.Desc(wl.n_heads_q, wl.n_heads_kv, wl.window, seq_lens=wl.lens,
                       budgets=wl.budgets, **kw)
    return cc.Desc(wl.n_heads_q, wl.n_heads_kv, wl.window, n=wl.lens[0], budget=wl.budgets[0], **kw)


def to_bf16(bits: np.ndarray, device: str = "cuda", pin: bool = False) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if device == "cpu":
        return t.pin_memory() if pin else t
    return t.to(device)


class LayerCompressor:
    """Pre-allocated state for repeated ``cc_compress_layer`` calls on one geometry.

    ``spec`` is a ``LayerSpec`` (or any object with its attributes).  Contiguous K/V: the
    compacted cache lands in ``k_out`` / ``v_out``.  Paged K/V (``spec.page_size > 0``):
    ``layout`` supplies ``page_table`` [S][pages] (int32, numpy), ``free_pages`` (fresh page
    ids, int32, numpy) and ``pool_pages``; the retained rows are written into fresh pages of the
    same pool and ``out_page_table`` names them."""

    def __init__(self, ctx: cc.Context, spec, mode: int = cc.CC_MODE_BF16, layout=None):
        wl = spec if isinstance(spec, LayerSpec) else LayerSpec.like(spec)
        self.ctx, self.wl = ctx, wl
        dev = f"cuda:{ctx.device}"
        self.paged = wl.page_size > 0
        S, hq, hkv, d = len(wl.lens), wl.n_heads_q, wl.n_heads_kv, wl.head_dim
        bf = torch.bfloat16
        if self.paged:
            if layout is None or layout.page_table is None:
                raise ValueError("a paged layout needs page_table, free_pages and pool_pages")
            ps = wl.page_size
            self.page_table = torch.from_numpy(layout.page_table).to(dev)
            self.free_pages = torch.from_numpy(layout.free_pages).to(dev)
            self.out_pt_stride = max((min(b, n) + ps - 1) // ps
                                     for b, n in zip(wl.budgets, wl.lens)) + 1
            self.desc = desc_from_spec(wl, mode, self.page_table, layout.pool_pages,
                                           self.out_pt_stride)
            rows = layout.pool_pages * ps
            self.out_page_table = torch.empty((S, self.out_pt_stride), dtype=torch.int32, device=dev)
            self.h_out_page_table = torch.empty(self.out_page_table.shape, dtype=torch.int32).pin_memory()
        else:
            self.desc = desc_from_spec(wl, mode)
            rows = self.desc.n_tot
            self.page_table = self.free_pages = self.out_page_table = None
        n_tot, b_tot = self.desc.n_tot, self.desc.b_tot
        self.q = torch.empty((S, wl.window, hq, d), dtype=bf, device=dev)
        self.k = torch.empty((rows, hkv, d), dtype=bf, device=dev)
        self.v = torch.empty((rows, hkv, d), dtype=bf, device=dev)
        self.prior = torch.empty((n_tot,), dtype=torch.float32, device=dev)
        if self.paged:
            self.k_out = self.v_out = None          # the pool itself receives the retained rows
        else:
            self.k_out = torch.empty((b_tot, hkv, d), dtype=bf, device=dev)
            self.v_out = torch.empty((b_tot, hkv, d), dtype=bf, device=dev)
        self.idx = torch.empty((hkv, b_tot), dtype=torch.int32, device=dev)
        self.count = torch.empty((S, hkv), dtype=torch.int32, device=dev)
        self.ws = ctx.workspace(self.desc)
        # pinned landing buffers for the results
        if self.paged:
            ps = wl.page_size
            n_out_rows = sum((min(b, n) + ps - 1) // ps for b, n in zip(wl.budgets, wl.lens)) * ps
            self.out_rows = (self.free_pages[: n_out_rows // ps, None].long() * ps
                             + torch.arange(ps, device=dev)[None, :]).reshape(-1)
            self.h_k_out = torch.empty((n_out_rows, hkv, d), dtype=bf).pin_memory()
            self.h_v_out = torch.empty((n_out_rows, hkv, d), dtype=bf).pin_memory()
            self.k_stage = torch.empty((n_out_rows, hkv, d), dtype=bf, device=dev)
            self.v_stage = torch.empty((n_out_rows, hkv, d), dtype=bf, device=dev)
        else:
            self.h_k_out = torch.empty(self.k_out.shape, dtype=bf).pin_memory()
            self.h_v_out = torch.empty(self.v_out.shape, dtype=bf).pin_memory()
        self.h_idx = torch.empty(self.idx.shape, dtype=torch.int32).pin_memory()
        self.h_count = torch.empty(self.count.shape, dtype=torch.int32).pin_memory()
        self._side = None               # stream of the overlapped copies back to the host
        self._readback_done = None      # event recorded after the last of them

    def h2d_bytes_of(self, v_in_place: bool) -> int:
        """Bytes that cross to the device per run_host call: Q, K and the prior, plus all of V or,
        when V is gathered in place from page-locked host memory, only its retained rows."""
        n = sum(t.numel() * t.element_size() for t in (self.q, self.k, self.prior))
        if not v_in_place:
            return n + self.v.numel() * self.v.element_size()
        kept = sum(min(b, m) for b, m in zip(self.wl.budgets, self.wl.lens))
        return n + kept * self.wl.n_heads_kv * self.wl.head_dim * self.v.element_size()

    @property
    def h2d_bytes(self) -> int:
        return self.h2d_bytes_of(False)

    @property
    def d2h_bytes(self) -> int:
        outs = [self.h_k_out, self.h_v_out, self.idx, self.count]
        if self.paged:
            outs.append(self.out_page_table)
        return sum(t.numel() * t.element_size() for t in outs)

    def run_device(self, q, k, v, prior, v_src=None) -> None:
        """Inputs already on the device; outputs land in self.k_out / v_out (contiguous) or in
        fresh pages of k / v (paged), plus idx / count / out_page_table.  ``v_src`` (page-locked
        host memory laid out like v) makes the compaction read the retained V rows from there."""
        if self.paged:
            cc.cc_compress_layer(self.ctx, self.desc, q, k, v if v_src is None else v_src, prior,
                                 k, v, self.idx, self.count,
                                 self.free_pages, self.out_page_table, ws=self.ws)
        else:
            cc.cc_compress_layer(self.ctx, self.desc, q, k, v if v_src is None else v_src, prior,
                                 self.k_out, self.v_out, self.idx, self.count, ws=self.ws)

    def run_host(self, q_h, k_h, v_h, prior_h, v_in_place: bool = False,
                 overlap_readback: bool = False) -> Dict[str, torch.Tensor]:
        """Inputs in (pinned) host memory: copy in, compress, copy the compacted cache back.
        Everything is enqueued on the current stream; the caller synchronises.

        V takes no part in the scoring: with ``v_in_place`` (v_h page-locked) it is not copied;
        the compaction kernel reads the retained rows of v_h across the bus and writes them to
        the device-side result, which cuts the bytes copied in by almost half.

        With ``overlap_readback`` the copies back to the host run on a stream of the compressor's
        own, so that they share the bus (which carries both directions at once) with the next
        call's copies in; the next call's kernels wait for them before they overwrite the device
        results.  Call ``finish()`` (or synchronise the device) before reading the host tensors."""
        main = torch.cuda.current_stream()
        self.q.copy_(q_h, non_blocking=True)
        self.k.copy_(k_h, non_blocking=True)
        if v_in_place:
            if not v_h.is_pinned() or v_h.shape != self.v.shape or not v_h.is_contiguous():
                raise ValueError("v_in_place needs a contiguous page-locked tensor shaped like the V pool")
        else:
            self.v.copy_(v_h, non_blocking=True)
        self.prior.copy_(prior_h, non_blocking=True)
        if self._readback_done is not None:          # the previous call's results are still going out
            main.wait_event(self._readback_done)
            self._readback_done = None
        self.run_device(self.q, self.k, self.v, self.prior, v_src=v_h if v_in_place else None)
        out = {"k_out": self.h_k_out, "v_out": self.h_v_out, "idx": self.h_idx,
               "count": self.h_count}
        if self.paged:
            # the retained rows sit in the fresh pages of the pool: gather just those (on the main
            # stream, before the next call refills the pool) and bring them back
            torch.index_select(self.k, 0, self.out_rows, out=self.k_stage)
            torch.index_select(self.v, 0, self.out_rows, out=self.v_stage)
            k_res, v_res = self.k_stage, self.v_stage
            out["out_page_table"] = self.h_out_page_table
        else:
            k_res, v_res = self.k_out, self.v_out
        back = main
        if overlap_readback:
            if self._side is None:
                self._side = torch.cuda.Stream()
            back = self._side
            back.wait_stream(main)
        with torch.cuda.stream(back):
            self.h_k_out.copy_(k_res, non_blocking=True)
            self.h_v_out.copy_(v_res, non_blocking=True)
            if self.paged:
                self.h_out_page_table.copy_(self.out_page_table, non_blocking=True)
            self.h_idx.copy_(self.idx, non_blocking=True)
            self.h_count.copy_(self.count, non_blocking=True)
            if overlap_readback:
                self._readback_done = torch.cuda.Event()
                self._readback_done.record(back)
        return out

    def finish(self) -> None:
        """Makes the current stream wait for copies back to the host that are still in flight."""
        if self._readback_done is not None:
            torch.cuda.current_stream().wait_event(self._readback_done)
            self._readback_done = None
