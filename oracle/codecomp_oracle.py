"""CPU oracle for the CodeComp per-layer KV-compression step.  TEST INFRASTRUCTURE ONLY.

A plain, slow NumPy restatement of what the hot path computes, written from the
paper's definitions.  It shares no code with the CUDA library and must never be
imported by it; only the tests, the smoke check and the benchmark's CPU-baseline leg
call it.  Floating point is fp64 unless a ``dtype`` argument says otherwise: the
pooling / fusing stages can also be evaluated in fp32, in a fixed operation order, so
that a selection (an integer decision taken on fp32 keys by the kernels) can be
compared bit for bit on identical fp32 inputs.

What each function follows:

* ``window_scores``   - Section 4.5, the equation defining A = softmax(QK^T/sqrt(d))
                        and u(j) = sum_t A(t, j); summed over the query heads that
                        share a KV head (grouped-query attention).
* ``pool_scores``     - Appendix "Compression settings" (sliding-window pooling of the
                        attention scores; the paper uses average pooling of width 5).
* ``fuse_prior``      - Section 4.4 "Span scoring" (importance is a weighted sum of
                        structural indicators and an attention term, Appendix
                        "Structural prior configuration").
* ``nearest_fill_values`` - Section 4.4 "Token-level protection", last sentence: when the
                        protected tokens do not fill the budget, the rest goes to the tokens
                        nearest to them (the alternative to the attention fill of Section 4.5).
* ``chunk_reduce``    - chunk-level aggregation of scores and prior (benchmark variant).
* ``span_budget``     - Section 4.4, the equation for B^span.
* ``select_tokens``   - Section 4.4 "Token-level protection" (protected tokens first,
                        first B of them if they exceed the budget) and Section 4.5
                        (remaining capacity filled by top-ranked attention scores).
* ``compact_kv``      - the retained K/V rows in original order (Section 4.6: chunks
                        keep their original position indices).
* ``ppl_chunk_scores`` / ``select_chunks`` - Section 4.1 "Query-Conditioned Chunk Selection":
                        mean negative log-likelihood of the query tokens given each chunk,
                        and the k chunks with the lowest value.
* ``plan_budgets``    - Section 4.3 "Structure-Aware Budget Allocation": normalised chunk
                        scores, capacity multipliers and the per-chunk token budgets B_i.
* ``select_spans``    - Section 4.4 "Span selection under budget": protected spans first,
                        the others greedily by score within B^span; returns the tokens
                        they cover (the set P_i that "Token-level protection" starts from).
* ``structural_score`` - Section 5.3, caption of the bug-localization table: the fraction
                        of structurally critical tokens that a retained set contains
                        (the table averages it over layers and chunks; the average is
                        the caller's).

Readings of the paper that are choices rather than statements of it ("parity
unpinned" by the paper, pinned here only by self-consistency tests):
  - the normalisation of the attention term inside ``fuse_prior`` (alpha is a free
    caller-chosen factor);
  - the edge rule of average pooling (zero padding, always divide by the width);
  - the ``causal`` option of ``window_scores`` (window inside the sequence) is an extension;
    the paper's window follows the context and needs no mask;
  - ``select_spans``: the greedy filling of the span budget (Section 4.4, "Span selection
    under budget") is read as: spans
    are taken whole, in rank order (score descending, earlier start first), while the
    tokens covered so far are fewer than B^span, so the last span taken may overshoot it;
  - ``structural_score`` of a sequence without structurally critical tokens is taken
    as 1 (nothing could be lost); the paper does not say;
  - ``nearest_fill_values``: "nearest" is the distance in token positions to the closest token
    whose prior reaches the threshold (before any cap of the protected set), equal distances go
    to the lower index, and a sequence without such a token keeps its first tokens.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2


# --------------------------------------------------------------------------- inputs
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- A1 score
def window_scores(q_win: np.ndarray, k: np.ndarray, n_heads_kv: int, causal: bool = False
                  ) -> Tuple[np.ndarray, np.ndarray]:
    """Window attention scores per KV head.

    q_win: [w][H_q][d] float64, k: [n][H_kv][d] float64.
    Returns (u [H_kv][n], lse [H_q][w]) with
      s_{g,t}(j) = q_{g,t} . k_j / sqrt(d),  A = softmax over the n keys (no mask),
      u_h(j) = sum over the G query heads of KV head h and the w window rows of A,
      lse = log sum_j exp(s) for every (query head, window row).
    ``causal`` (an extension, not in the paper, whose window follows the context): the window
    is the last w tokens of the sequence itself, so row t sits at position n - w + t and
    attends to the keys j <= n - w + t only (A = 0 beyond).
    """
    w, hq, d = q_win.shape
    n = k.shape[0]
    if causal and n < w:
        raise ValueError("a causal window needs n >= w")
    g = hq // n_heads_kv
    u = np.zeros((n_heads_kv, n), dtype=np.float64)
    lse = np.zeros((hq, w), dtype=np.float64)
    for h in range(n_heads_kv):
        kh = k[:, h, :]                                   # [n][d]
        for gi in range(g):
            qh = q_win[:, h * g + gi, :]                  # [w][d]
            s = (qh @ kh.T) / math.sqrt(d)                # [w][n]
            if causal:
                for t in range(w):
                    s[t, n - w + t + 1:] = -np.inf
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            l = e.sum(axis=1, keepdims=True)
            a = e / l                                     # rows sum to 1
            u[h] += a.sum(axis=0)
            lse[h * g + gi] = (m + np.log(l))[:, 0]
    return u, lse


# --------------------------------------------------------------------------- A2 pool
def pool_scores(u: np.ndarray, kind: int, width: int, dtype=np.float64) -> np.ndarray:
    """Centred stride-1 pooling along the last axis, output length unchanged.

    max: the window is clipped to the valid range.
    avg: zero padded; the ``width`` taps are added left to right and the sum is
         divided by ``width`` (also at the edges).
    """
    u = np.asarray(u, dtype=dtype)
    if kind == POOL_NONE or width == 1:
        return u.copy()
    assert width % 2 == 1
    half = width // 2
    n = u.shape[-1]
    fill = -np.inf if kind == POOL_MAX else 0.0
    pad = np.full(u.shape[:-1] + (n + 2 * half,), fill, dtype=dtype)
    pad[..., half:half + n] = u
    acc = pad[..., 0:n].copy()
    for o in range(1, width):
        tap = pad[..., o:o + n]
        acc = np.maximum(acc, tap) if kind == POOL_MAX else (acc + tap).astype(dtype)
    if kind == POOL_AVG:
        acc = (acc / dtype(width)).astype(dtype)
    return acc


# --------------------------------------------------------------------------- A3 fuse
def fuse_prior(pooled: np.ndarray, prior: np.ndarray, alpha: float, beta: float,
               dtype=np.float64) -> np.ndarray:
    """f(j) = alpha * pooled(j) + beta * prior(j); two products, then one sum."""
    a, b = dtype(alpha), dtype(beta)
    t1 = (a * np.asarray(pooled, dtype=dtype)).astype(dtype)
    t2 = (b * np.asarray(prior, dtype=dtype)).astype(dtype)
    return (t1 + t2).astype(dtype)


def nearest_fill_values(prior: np.ndarray, force_threshold: float) -> np.ndarray:
    """Ranking value of every token when the budget left by the protected tokens is filled with
    the tokens nearest to them: minus the distance (in positions) to the closest token with
    prior >= force_threshold, found with one forward and one backward sweep.  Larger is better,
    so the usual order (value descending, index ascending) takes nearer tokens first and the
    lower index among equally near ones.  Without any such token every value is minus the
    sequence length (the order is then by index)."""
    n = len(prior)
    hit = np.asarray(prior).astype(np.float32) >= np.float32(force_threshold)
    dist = np.full(n, n, dtype=np.int64)
    last = -1
    for j in range(n):                         # distance to the closest protected token at or before j
        if hit[j]:
            last = j
        if last >= 0:
            dist[j] = j - last
    nxt = -1
    for j in range(n - 1, -1, -1):             # ... and at or after j
        if hit[j]:
            nxt = j
        if nxt >= 0:
            dist[j] = min(dist[j], nxt - j)
    return -dist.astype(np.float64)


# --------------------------------------------------------------------------- A6 chunks
def chunk_lengths(n: int, chunk: int) -> np.ndarray:
    """Token count of every fixed-size chunk of a length-n sequence (last one ragged)."""
    chunk = max(1, chunk)
    m = (n + chunk - 1) // chunk
    lens = np.full(m, chunk, dtype=np.int64)
    if m:
        lens[-1] = n - (m - 1) * chunk
    return lens


def chunk_reduce(u: np.ndarray, prior: np.ndarray, chunk: int, dtype=np.float64
                 ) -> Tuple[np.ndarray, np.ndarray]:
    """Chunk score = sum of token scores (in index order); chunk prior = max token prior."""
    u = np.asarray(u, dtype=dtype)
    n = u.shape[-1]
    lens = chunk_lengths(n, chunk)
    m = len(lens)
    # lay the tokens out as [m][chunk]; the ragged tail is padded with +0.0 (adding it
    # changes nothing) and with -inf for the prior maximum
    pad_u = np.zeros(u.shape[:-1] + (m * chunk,), dtype=dtype)
    pad_u[..., :n] = u
    pad_u = pad_u.reshape(u.shape[:-1] + (m, chunk))
    acc = pad_u[..., 0].copy()
    for c in range(1, chunk):                      # token order inside the chunk
        acc = (acc + pad_u[..., c]).astype(dtype)
    pad_p = np.full(m * chunk, -np.inf, dtype=np.float64)
    pad_p[:n] = prior
    ps = pad_p.reshape(m, chunk).max(axis=1).astype(np.asarray(prior).dtype)
    return acc, ps


# --------------------------------------------------------------------------- A4 select
def span_budget(budget: int, span_ratio: float, span_min: int) -> int:
    """B^span = min(B, max(B_min, floor(rho * B))); the floor is taken after a 1e-9 nudge
    so that products such as 0.7 * 10 that are integers on paper stay integers."""
    return int(min(budget, max(span_min, math.floor(span_ratio * budget + 1e-9))))


def protected_items(prior: np.ndarray, lens: np.ndarray, budget: int, force_threshold: float,
                    span_ratio: float = 0.0, span_min: int = 0) -> np.ndarray:
    """Mask of the protected items (Section 4.4, "Token-level protection" and "Span selection
    under budget"): prior >= force_threshold; with span_ratio > 0 only the longest prefix of
    them, ranked by (prior descending, index ascending), whose token count stays within B^span."""
    m = len(prior)
    lens = np.asarray(lens, dtype=np.int64)
    idx = np.arange(m)
    # the prior is an fp32 input, so the threshold test is an fp32 comparison
    forced = np.asarray(prior).astype(np.float32) >= np.float32(force_threshold)
    if span_ratio > 0.0:
        cap = span_budget(int(budget), span_ratio, span_min)
        cand = idx[forced]
        order = cand[np.lexsort((cand, -np.asarray(prior, dtype=np.float64)[cand]))]
        cum = np.cumsum(lens[order])
        forced = np.zeros(m, dtype=bool)
        forced[order[cum <= cap]] = True
    return forced


def select_items(fused: np.ndarray, prior: np.ndarray, lens: np.ndarray, budget: int,
                 force_threshold: float, span_ratio: float = 0.0, span_min: int = 0
                 ) -> np.ndarray:
    """How many leading tokens of each item (token or chunk) are retained.

    Items are ranked by: protected first (among themselves by position), then larger
    fused score, then smaller index.
    Items are taken in rank order until ``min(budget, total tokens)`` tokens are kept;
    the item that crosses the budget keeps only its first tokens.  Protected items are
    those of ``protected_items``.
    """
    m = len(fused)
    lens = np.asarray(lens, dtype=np.int64)
    total = int(lens.sum())
    b_eff = max(0, min(int(budget), total))
    idx = np.arange(m)
    forced = protected_items(prior, lens, budget, force_threshold, span_ratio, span_min)
    f = np.asarray(fused, dtype=np.float64) + 0.0          # -0.0 ranks equal to +0.0
    f = np.where(forced, np.inf, f)                        # protected items rank by position only
    order = np.lexsort((idx, -f, ~forced))                 # last key is the primary one
    before = np.cumsum(lens[order]) - lens[order]
    take_sorted = np.clip(b_eff - before, 0, lens[order])
    take = np.zeros(m, dtype=np.int64)
    take[order] = take_sorted
    return take


def expand_items(take: np.ndarray, chunk: int) -> np.ndarray:
    """Ascending token indices of the retained tokens given per-item retained counts."""
    chunk = max(1, chunk)
    out: List[np.ndarray] = [np.arange(c * chunk, c * chunk + t)
                             for c, t in enumerate(take) if t > 0]
    return np.concatenate(out).astype(np.int32) if out else np.zeros(0, np.int32)


def select_tokens(fused: np.ndarray, prior: np.ndarray, n: int, budget: int,
                  force_threshold: float, span_ratio: float = 0.0, span_min: int = 0,
                  chunk: int = 1) -> np.ndarray:
    """Retained token indices (ascending) of one head; ``fused``/``prior`` are per item."""
    lens = chunk_lengths(n, chunk)
    take = select_items(fused, prior, lens, budget, force_threshold, span_ratio, span_min)
    return expand_items(take, chunk)


# --------------------------------------------------------------------------- A5 compact
def compact_kv(k_bits: np.ndarray, v_bits: np.ndarray, idx: Sequence[np.ndarray]
               ) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Per KV head h: K_out[s] = K[idx_h[s]][h], same for V (bit copies)."""
    k_out = [k_bits[np.asarray(ix, dtype=np.int64), h, :] for h, ix in enumerate(idx)]
    v_out = [v_bits[np.asarray(ix, dtype=np.int64), h, :] for h, ix in enumerate(idx)]
    return k_out, v_out


# --------------------------------------------------------------------------- chunk selection
def ppl_chunk_scores(logits: np.ndarray, targets: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Query-conditioned perplexity score of every chunk (Section 4.1).

    logits [chunks][T][V] (any float type, used as fp64): row (i, t) holds the model's
    next-token logits for query position t when the context is prefix + chunk i;
    targets [T]: the query tokens q_t.  -log p(q_t | ...) = logsumexp(row) - row[q_t].
    Returns (s_ppl [chunks] = mean over t, nll [chunks][T])."""
    x = np.asarray(logits, dtype=np.float64)
    m = x.max(axis=2, keepdims=True)
    lse = (m + np.log(np.exp(x - m).sum(axis=2, keepdims=True)))[:, :, 0]
    tgt = np.take_along_axis(x, np.asarray(targets, dtype=np.int64)[None, :, None], axis=2)[:, :, 0]
    nll = lse - tgt
    return nll.mean(axis=1), nll


def select_chunks(scores: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k chunks with the lowest score, best first; equal scores: lower index
    first (the paper is silent on ties); NaN ranks last."""
    s = np.asarray(scores, dtype=np.float64)
    key = np.where(np.isnan(s), np.inf, s)
    order = sorted(range(len(s)), key=lambda i: (key[i], i))
    return np.asarray(order[:max(0, min(k, len(s)))], dtype=np.int64)


# --------------------------------------------------------------------------- budget planner
def plan_budgets(sigma: Sequence[float], lens: Sequence[int], r: float, r_max: float,
                 m_min: float, m_max: float, eps: float) -> Tuple[np.ndarray, np.ndarray]:
    """Per-chunk token budgets from the chunk-level structural scores (Section 4.3).

    s~_i = 0.5 if all scores are equal, else (sigma_i - min) / max(eps, max - min);
    m_i = m_min + (m_max - m_min) * clip(s~_i, 0, 1);  B_i = floor(|C_i| * min(r_max, r * m_i)).
    Everything in fp64, in exactly this operation order.  Returns (B [int64], m [float64])."""
    sig = np.asarray(sigma, dtype=np.float64)
    budgets = np.zeros(len(sig), dtype=np.int64)
    mult = np.zeros(len(sig), dtype=np.float64)
    if len(sig) == 0:
        return budgets, mult
    lo, hi = float(sig.min()), float(sig.max())
    for i, (sg, length) in enumerate(zip(sig, lens)):
        st = 0.5 if hi == lo else (float(sg) - lo) / max(float(eps), hi - lo)
        st = min(1.0, max(0.0, st))
        mult[i] = float(m_min) + (float(m_max) - float(m_min)) * st
        # same 1e-9 nudge as span_budget: products that are integers on paper stay integers
        budgets[i] = math.floor(float(length) * min(float(r_max), float(r) * mult[i]) + 1e-9)
    return budgets, mult


def select_spans(starts: Sequence[int], ends: Sequence[int], scores: Sequence[float],
                 protected: Sequence[bool], n: int, budget: int, span_ratio: float,
                 span_min: int) -> Tuple[np.ndarray, List[int]]:
    """Tokens covered by the spans selected under the span budget (Section 4.4).

    Spans are half-open token ranges [start, end) inside [0, n).  Protected spans are all
    taken; the others follow in rank order (score descending, earlier start, lower index) while
    fewer than B^span = min(B, max(B_min, floor(rho * B))) tokens are covered.
    Returns (mask [n] of covered tokens, indices of the spans taken in the order taken)."""
    cap = span_budget(budget, span_ratio, span_min) if span_ratio > 0 else budget
    mask = np.zeros(n, dtype=bool)
    taken: List[int] = []
    for i in range(len(starts)):
        if protected[i]:
            mask[starts[i]:ends[i]] = True
            taken.append(i)
    rest = [i for i in range(len(starts)) if not protected[i]]
    rest.sort(key=lambda i: (-float(np.float32(scores[i])), starts[i], i))
    for i in rest:
        if int(mask.sum()) >= cap:
            break
        mask[starts[i]:ends[i]] = True
        taken.append(i)
    return mask, taken


# --------------------------------------------------------------------------- Str. Score
def structural_score(idx: np.ndarray, prior: np.ndarray, threshold: float
                     ) -> Tuple[float, int, int]:
    """Fraction of the structurally critical tokens {j : prior[j] >= threshold} that the
    retained index set ``idx`` (entries < 0 are padding) contains; also the two counts
    (retained critical tokens, critical tokens).  Defined as 1.0 when there are none."""
    critical = set(int(j) for j in np.flatnonzero(np.asarray(prior, dtype=np.float64) >= threshold))
    kept = set(int(j) for j in np.asarray(idx).ravel() if j >= 0)
    hit = len(critical & kept)
    return (hit / len(critical) if critical else 1.0), hit, len(critical)


# --------------------------------------------------------------------------- paged layout
def paged_rows(page_table_row: np.ndarray, n: int, page_size: int) -> np.ndarray:
    """Pool row of every token 0..n-1 of one sequence."""
    tok = np.arange(n, dtype=np.int64)
    return page_table_row[tok // page_size].astype(np.int64) * page_size + tok % page_size


def assign_output_pages(budgets: Sequence[int], totals: Sequence[int], page_size: int,
                        free_pages: np.ndarray) -> List[np.ndarray]:
    """Fresh pages per sequence: ceil(min(B_s, n_s)/page) ids taken in order from the list."""
    out, cur = [], 0
    for b, n in zip(budgets, totals):
        cnt = (min(b, n) + page_size - 1) // page_size
        out.append(np.asarray(free_pages[cur:cur + cnt], dtype=np.int32))
        cur += cnt
    return out


# --------------------------------------------------------------------------- A8 whole path
def compress_sequence(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: Optional[np.ndarray],
                      prior: np.ndarray, n_heads_kv: int, pool_kind: int, pool_size: int,
                      budget: int, alpha: float, beta: float, force_threshold: float,
                      span_ratio: float = 0.0, span_min: int = 0, chunk: int = 1,
                      stage_dtype=np.float64, causal: bool = False,
                      nearest_fill: bool = False) -> dict:
    """The whole per-layer step for one contiguous sequence.

    q_bits [w][H_q][d], k_bits/v_bits [n][H_kv][d] as bf16 bit patterns, prior [n].
    ``stage_dtype`` is the precision of everything after the scores (fp64 by default;
    fp32 reproduces the kernels' post-score arithmetic on the oracle's own scores).
    """
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    n = k.shape[0]
    u, lse = window_scores(q, k, n_heads_kv, causal)
    u_s = u.astype(stage_dtype)
    prior_s = np.asarray(prior, dtype=stage_dtype)
    if chunk > 1:
        item_u, item_p = chunk_reduce(u_s, prior_s, chunk, dtype=stage_dtype)
        pooled = item_u
    else:
        pooled = pool_scores(u_s, pool_kind, pool_size, dtype=stage_dtype)
        item_p = prior_s
    fused = fuse_prior(pooled, item_p[None, :], alpha, beta, dtype=stage_dtype)
    if nearest_fill:
        # Section 4.4 fill rule instead of the attention scores (token level only)
        assert chunk == 1
        fused = np.repeat(nearest_fill_values(prior, force_threshold)[None, :], n_heads_kv, axis=0
                          ).astype(stage_dtype)
    idx = [select_tokens(fused[h], item_p, n, budget, force_threshold, span_ratio,
                         span_min, chunk) for h in range(n_heads_kv)]
    res = {"scores": u, "lse": lse, "pooled": pooled, "fused": fused, "idx": idx,
           "item_prior": item_p}
    if v_bits is not None:
        res["k_out"], res["v_out"] = compact_kv(k_bits, v_bits, idx)
    return res
