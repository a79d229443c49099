"""Seeded synthetic inputs for the CodeComp compression hot path.

This module only draws random numbers and lays them out; it contains none of the
method's arithmetic, so both the CUDA path's tests and the CPU oracle's tests can
take their inputs from it.  Everything is NumPy on the host; bf16 tensors are
carried as ``uint16`` bit patterns so that every consumer sees identical bits.

Workloads stand in for the long-code contexts the paper evaluates on (8B-class GQA
models, tens of thousands of context tokens, Appendix "Experimental Setup"): only
the shapes and the line-level statistics of structural anchors (Section 4.4,
"Structural span construction") are taken from it; no benchmark item is reproduced.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2

# line labels used by the structural-prior generator
LABELS = ("call", "branch", "assign", "return", "other")
LABEL_P = (0.08, 0.06, 0.12, 0.03, 0.71)


@dataclass(frozen=True)
class Workload:
    """One configuration of the hot path (one layer's worth of shapes)."""

    name: str
    cfg_id: int
    layers: int
    n_heads_q: int
    n_heads_kv: int
    head_dim: int
    window: int
    pool_kind: int
    pool_size: int
    budget: int                      # tokens kept per KV head (single sequence)
    n: int = 0                       # prefix length (single sequence)
    seq_lens: Tuple[int, ...] = ()   # ragged batch; empty = single sequence of n
    budget_frac: float = 0.0         # ragged: B_s = floor(frac * n_s)
    chunk_size: int = 1              # 1 = token level
    page_size: int = 0               # 0 = contiguous K/V
    outlier_frac: float = 0.0        # fraction of key channels scaled
    outlier_scale: float = 8.0
    p_structural: float = 1.0 - LABEL_P[-1]   # P(line is not "other")
    flagged_per_line: int = 3
    alpha: float = 1.0
    beta: float = 0.0
    force_threshold: float = 0.5     # prior >= threshold -> forced retention
    span_ratio: float = 0.0          # 0 = no cap on forced tokens
    span_min: int = 16
    causal: bool = False             # window = last w tokens of the sequence itself (masked)
    fill_mode: int = 0               # 1 = the budget left by the protected tokens goes to their nearest neighbours
    seq_budgets: Tuple[int, ...] = ()   # ragged batch: explicit per-sequence budgets (else budget_frac)

    @property
    def group(self) -> int:
        return self.n_heads_q // self.n_heads_kv

    @property
    def lens(self) -> Tuple[int, ...]:
        return self.seq_lens if self.seq_lens else (self.n,)

    @property
    def budgets(self) -> Tuple[int, ...]:
        if self.seq_budgets:
            return self.seq_budgets
        if self.seq_lens:
            return tuple(int(np.floor(self.budget_frac * s)) for s in self.seq_lens)
        return (self.budget,)


def _ragged_lengths(seed: int, count: int, lo: int, hi: int) -> Tuple[int, ...]:
    rng = np.random.Generator(np.random.PCG64(seed))
    return tuple(int(x) for x in rng.integers(lo, hi + 1, size=count))


def workloads() -> Dict[str, Workload]:
    """The five benchmark configurations plus the paper's own pooling setting."""
    w: Dict[str, Workload] = {}
    w["tiny"] = Workload("tiny", 0, 1, 8, 2, 128, 32, POOL_MAX, 7, 512, n=2048)
    w["llama3_8b"] = Workload("llama3_8b", 1, 32, 32, 8, 128, 64, POOL_MAX, 7, 2048,
                              n=32768, outlier_frac=0.01)
    w["qwen25_coder_7b"] = Workload("qwen25_coder_7b", 2, 28, 28, 4, 128, 64, POOL_MAX, 7,
                                    4096, n=65536)
    w["chunk10"] = Workload("chunk10", 3, 32, 32, 8, 128, 64, POOL_NONE, 1, 2048, n=32768,
                            outlier_frac=0.01, chunk_size=10)
    w["ragged_paged"] = Workload("ragged_paged", 4, 32, 32, 8, 128, 64, POOL_MAX, 7, 0,
                                 seq_lens=_ragged_lengths(4004, 8, 8192, 65536),
                                 budget_frac=0.10, page_size=16)
    # Appendix "Compression settings": average pooling of width 5, window of 128 rows,
    # span budget ratio 0.5 with a 16-token minimum.
    w["paper_avg5_w128"] = Workload("paper_avg5_w128", 5, 32, 32, 8, 128, 128, POOL_AVG, 5,
                                    1638, n=4096, span_ratio=0.5, span_min=16)
    return w


def qwen_variant(base: Workload, budget: int, density: str) -> Workload:
    """Budget / prior-density sweep of the Qwen-shaped configuration.

    Densities keep the call:branch:assign:return ratio and change how many lines are
    structural; 30 % needs six flagged tokens per line because three flagged tokens of
    a mean-12 line cap the density near 23 %.
    """
    p, flagged = {"5": (0.2176, 3), "15": (0.6529, 3), "30": (0.7377, 6)}[density]
    return replace(base, name=f"{base.name}_B{budget}_p{density}", budget=budget,
                   p_structural=p, flagged_per_line=flagged)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of float32 values to bf16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + rounding) >> np.uint32(16)).astype(np.uint16)


def structural_prior(seed: int, n: int, p_structural: float = 1.0 - LABEL_P[-1],
                     flagged_per_line: int = 3, mean_line: float = 12.0
                     ) -> Tuple[np.ndarray, np.ndarray]:
    """Per-token prior in {0, 1} and the per-token line label (index into LABELS).

    Tokens are split into lines of geometric length; each line is labelled, and the
    first ``flagged_per_line`` tokens of every structural line carry prior 1.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    struct_p = np.array(LABEL_P[:4], dtype=np.float64)
    probs = np.concatenate([struct_p / struct_p.sum() * p_structural, [1.0 - p_structural]])
    prior = np.zeros(n, dtype=np.float32)
    label = np.full(n, len(LABELS) - 1, dtype=np.int8)
    pos = 0
    while pos < n:
        length = int(rng.geometric(1.0 / mean_line))
        lab = int(rng.choice(len(LABELS), p=probs))
        end = min(n, pos + length)
        label[pos:end] = lab
        if lab != len(LABELS) - 1:
            prior[pos:min(end, pos + flagged_per_line)] = 1.0
        pos = end
    return prior, label


@dataclass
class LayerInputs:
    """Host-side tensors for one layer of a workload (bf16 carried as uint16 bits)."""

    workload: Workload
    layer: int
    q_win: np.ndarray          # [S][w][H_q][d] uint16
    k: np.ndarray              # contiguous: [N_tot][H_kv][d]; paged: [pool_tokens][H_kv][d]
    v: np.ndarray
    prior: np.ndarray          # [N_tot] float32, sequences back to back
    label: np.ndarray          # [N_tot] int8
    page_table: Optional[np.ndarray] = None   # [S][max_pages] int32, -1 padded
    free_pages: Optional[np.ndarray] = None   # fresh page ids for the compacted cache
    pool_pages: int = 0
    tok_offsets: np.ndarray = field(default_factory=lambda: np.zeros(1, np.int64))


def make_layer(wl: Workload, layer: int = 0, with_v: bool = True) -> LayerInputs:
    """Draw one layer's Q window, K, V and priors for ``wl`` from its seeds."""
    rng = np.random.Generator(np.random.PCG64(1000 * wl.cfg_id + layer))
    lens = wl.lens
    S, d, Hq, Hkv = len(lens), wl.head_dim, wl.n_heads_q, wl.n_heads_kv
    n_tot = int(sum(lens))
    q = rng.standard_normal((S, wl.window, Hq, d), dtype=np.float32)
    k = rng.standard_normal((n_tot, Hkv, d), dtype=np.float32)
    if wl.outlier_frac > 0.0:
        n_out = int(np.ceil(wl.outlier_frac * d))
        for h in range(Hkv):
            ch = rng.choice(d, size=n_out, replace=False)
            k[:, h, ch] *= np.float32(wl.outlier_scale)
    v = rng.standard_normal((n_tot, Hkv, d), dtype=np.float32) if with_v else None
    q_b, k_b = f32_to_bf16_bits(q), f32_to_bf16_bits(k)
    v_b = f32_to_bf16_bits(v) if with_v else np.zeros((0, Hkv, d), np.uint16)
    del q, k, v

    priors, labels = [], []
    for s, n_s in enumerate(lens):
        p, lab = structural_prior(7919 * wl.cfg_id + s, n_s, wl.p_structural,
                                  wl.flagged_per_line)
        priors.append(p)
        labels.append(lab)
    tok_off = np.zeros(S + 1, dtype=np.int64)
    tok_off[1:] = np.cumsum(lens)

    out = LayerInputs(wl, layer, q_b, k_b, v_b, np.concatenate(priors),
                      np.concatenate(labels), tok_offsets=tok_off)
    if wl.page_size > 0:
        _scatter_into_pages(out, rng)
    return out


def _scatter_into_pages(x: LayerInputs, rng: np.random.Generator) -> None:
    """Move the back-to-back sequences of ``x`` into a shuffled paged pool (in place)."""
    wl = x.workload
    ps = wl.page_size
    lens = wl.lens
    n_pages = [(n + ps - 1) // ps for n in lens]
    out_pages = [(b + ps - 1) // ps for b in wl.budgets]
    used = int(sum(n_pages))
    pool_pages = used + int(sum(out_pages)) + 8
    perm = rng.permutation(pool_pages).astype(np.int32)
    table = np.full((len(lens), max(n_pages)), -1, dtype=np.int32)
    Hkv, d = wl.n_heads_kv, wl.head_dim
    k_pool = np.zeros((pool_pages * ps, Hkv, d), dtype=np.uint16)
    v_pool = np.zeros((pool_pages * ps, Hkv, d), dtype=np.uint16) if x.v.shape[0] else x.v
    cursor = 0
    for s, n_s in enumerate(lens):
        ids = perm[cursor:cursor + n_pages[s]]
        cursor += n_pages[s]
        table[s, :n_pages[s]] = ids
        tok = np.arange(n_s)
        dst = ids[tok // ps].astype(np.int64) * ps + tok % ps
        src = x.tok_offsets[s] + tok
        k_pool[dst] = x.k[src]
        if x.v.shape[0]:
            v_pool[dst] = x.v[src]
    x.k, x.v = k_pool, v_pool
    x.page_table = table
    x.free_pages = perm[used:].copy()
    x.pool_pages = pool_pages


def repage(x: LayerInputs, ref: LayerInputs) -> None:
    """Re-scatter the paged K/V of ``x`` so that it uses the page table of ``ref`` (same
    workload).  Lets several layers share one page layout (in place)."""
    wl = x.workload
    ps = wl.page_size
    k_new, v_new = np.zeros_like(x.k), np.zeros_like(x.v)
    for s, n_s in enumerate(wl.lens):
        tok = np.arange(n_s)
        src = x.page_table[s][tok // ps].astype(np.int64) * ps + tok % ps
        dst = ref.page_table[s][tok // ps].astype(np.int64) * ps + tok % ps
        k_new[dst] = x.k[src]
        if x.v.shape[0]:
            v_new[dst] = x.v[src]
    x.k, x.v = k_new, v_new
    x.page_table, x.free_pages = ref.page_table, ref.free_pages


def small_case(seed: int, n: int, window: int, n_heads_q: int, n_heads_kv: int,
               head_dim: int = 128, scale: float = 1.0
               ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Q window, K and V bit patterns of arbitrary small shape, for shape sweeps."""
    rng = np.random.Generator(np.random.PCG64(seed))
    q = rng.standard_normal((window, n_heads_q, head_dim), dtype=np.float32) * np.float32(scale)
    k = rng.standard_normal((n, n_heads_kv, head_dim), dtype=np.float32)
    v = rng.standard_normal((n, n_heads_kv, head_dim), dtype=np.float32)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


@dataclass
class ChunkBatch:
    """Synthetic retrieved chunks of one request, as the planner sees them (Sections 4.3, 4.4):
    lengths, chunk-level structural scores, and per chunk the structural spans (half-open token
    ranges with an importance score and a protected flag for signatures / query matches)."""

    lens: Tuple[int, ...]
    sigma: np.ndarray                      # [chunks] float64 in [0, 1]
    spans: List[Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]]   # starts, ends, scores, protected


def chunk_batch(seed: int, count: int = 32, lo: int = 128, hi: int = 4096) -> ChunkBatch:
    """``count`` chunks of ``lo``..``hi`` tokens (Appendix "Compression settings": method-level
    chunks of at most 4096 tokens).  Spans: one per structural line of the chunk's seeded
    line-label layout, from the line's first token over a local context of 6 to 40 tokens (spans
    overlap, and together cover more tokens than a span budget admits); the score is the
    label's weight of the appendix (call .20, branch .18, return .14, assignment .14) plus a
    seeded term below .24 standing for the query-alignment and def-use terms; the first line of
    a chunk (the signature) and about 3 % of the others are protected."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = tuple(int(x) for x in rng.integers(lo, hi + 1, size=count))
    sigma = rng.random(count)
    weight = {0: 0.20, 1: 0.18, 2: 0.14, 3: 0.14}
    spans = []
    for c, n in enumerate(lens):
        _, label = structural_prior(seed * 1000 + c, n)
        starts, ends, scores, prot = [0], [min(n, 8)], [0.5], [True]       # the signature line
        line_start = np.flatnonzero(np.diff(np.concatenate([[-1], label.astype(np.int64)])) != 0)
        for j in line_start:
            lab = int(label[j])
            if lab == len(LABELS) - 1 or j == 0:
                continue
            starts.append(int(j))
            ends.append(int(min(n, j + rng.integers(6, 41))))
            scores.append(weight[lab] + float(rng.random()) * 0.24)
            prot.append(bool(rng.random() < 0.03))
        spans.append((np.asarray(starts, np.int32), np.asarray(ends, np.int32),
                      np.asarray(scores, np.float32), np.asarray(prot, bool)))
    return ChunkBatch(lens, sigma, spans)
