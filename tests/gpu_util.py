"""Helpers shared by the GPU parity tests: tensor marshalling and oracle-side staging."""
from __future__ import annotations

import math

import numpy as np
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen

_CTX = None


def ctx() -> cc.Context:
    global _CTX
    if _CTX is None:
        _CTX = cc.Context(0)
    return _CTX


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bits_host(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def f32_dev(x) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()


def desc_for(wl: gen.Workload, mode: int, page_table=None, out_pt_stride: int = 0,
             force: bool = True, pool_pages: int = 0) -> cc.Desc:
    kw = dict(head_dim=wl.head_dim, compute_mode=mode, pool_kind=wl.pool_kind,
              pool_size=wl.pool_size, chunk_size=wl.chunk_size, alpha=wl.alpha, beta=wl.beta,
              force_threshold=wl.force_threshold if force else math.inf,
              span_ratio=wl.span_ratio, span_min=wl.span_min, page_size=wl.page_size,
              page_table=page_table, out_page_table_stride=out_pt_stride,
              pool_pages=pool_pages, causal=wl.causal, fill_mode=wl.fill_mode)
    if wl.seq_lens:
        return cc.Desc(wl.n_heads_q, wl.n_heads_kv, wl.window, seq_lens=wl.lens,
                       budgets=wl.budgets, **kw)
    return cc.Desc(wl.n_heads_q, wl.n_heads_kv, wl.window, n=wl.n, budget=wl.budget, **kw)


def score_tolerance(u_ref: np.ndarray, rows: int, n: int, tol: float) -> np.ndarray:
    """|u - u_ref| <= tol * |u_ref| + tol * (w * G / n): relative, with a floor at the mean score."""
    return tol * np.abs(u_ref) + tol * rows / max(n, 1)


def assert_scores_close(u: np.ndarray, u_ref: np.ndarray, rows: int, n: int, tol: float):
    err = np.abs(u.astype(np.float64) - u_ref)
    bound = score_tolerance(u_ref, rows, n, tol)
    bad = err > bound
    assert not bad.any(), (f"{bad.sum()} of {bad.size} scores off; worst ratio "
                           f"{(err / bound).max():.3g} at {np.unravel_index((err / bound).argmax(), err.shape)}")
    # The floor above (one mean score) only matters for scores far below the mean.  Every score
    # that is not negligible (above a thousandth of the mean) must also meet the relative bound
    # with hardly any help from the floor: the kernels' error sources are relative.
    mean = rows / max(n, 1)
    sizable = np.abs(u_ref) > 1e-3 * mean
    rel_bad = sizable & (err > tol * np.abs(u_ref) + tol * 1e-3 * mean)
    assert not rel_bad.any(), (f"{rel_bad.sum()} of {sizable.sum()} sizable scores miss the relative "
                               f"bound; worst {(err[sizable] / np.abs(u_ref[sizable])).max():.3g}")


def seq_kv(x: gen.LayerInputs, s: int):
    """Contiguous K/V bit patterns of sequence s (undoing the paging)."""
    wl = x.workload
    n = wl.lens[s]
    if wl.page_size:
        rows = orc.paged_rows(x.page_table[s], n, wl.page_size)
    else:
        rows = np.arange(x.tok_offsets[s], x.tok_offsets[s] + n)
    return x.k[rows], (x.v[rows] if x.v.shape[0] else None)


def check_selection(idx: np.ndarray, fused_ref: np.ndarray, forced: np.ndarray, keep: int,
                    band: np.ndarray, n: int, chunk: int = 1):
    """Index-set comparison that forgives only items (tokens or chunks) whose reference value
    is within the tolerance band of the reference cut-off: every item clearly above it is
    kept whole, every item clearly below it is dropped, the token count is exact, indices
    ascend, each item keeps a prefix of its tokens and at most one item is cut short."""
    assert len(idx) == keep
    assert np.all(np.diff(idx) > 0)
    assert keep == 0 or (idx[0] >= 0 and idx[-1] < n)
    lens = orc.chunk_lengths(n, chunk)
    m = len(lens)
    take = np.bincount(idx // chunk, minlength=m) if keep else np.zeros(m, np.int64)
    np.testing.assert_array_equal(orc.expand_items(take, chunk), idx)      # prefixes of items
    assert np.sum((take > 0) & (take < lens)) <= 1
    forced_tokens = int(lens[forced].sum())
    if forced_tokens >= keep:
        ref = orc.select_items(np.zeros(m), forced.astype(np.float32), lens, keep, 0.5)
        np.testing.assert_array_equal(take, ref)          # first B tokens of the protected set
        return
    assert np.all(take[forced] == lens[forced])
    free = ~forced
    ref_take = orc.select_items(fused_ref, forced.astype(np.float32), lens, keep, 0.5)
    kept_free = free & (ref_take > 0)
    if not kept_free.any() or np.all(ref_take[free] == lens[free]):
        return
    cut = fused_ref[kept_free].min()              # reference value of the last retained item
    clearly_in = free & (fused_ref > cut + band)
    clearly_out = free & (fused_ref < cut - band)
    assert np.all(take[clearly_in] == lens[clearly_in]), "an item clearly above the cut-off was dropped"
    assert not take[clearly_out].any(), "an item clearly below the cut-off was kept"
