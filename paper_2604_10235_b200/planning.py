"""From the planner to the compression call: per-chunk budgets (Section 4.3) and the protected
token sets of the selected structural spans (Section 4.4) for a batch of chunks, in the form
``cc_layer_desc`` and ``cc_compress_layer`` take them (budgets per sequence; one prior array,
chunks back to back, 1.0 on the protected tokens).  The arithmetic is the library's
(``cc_plan_budgets``, ``cc_select_spans``: host calls of the C ABI); this file only loops over
the chunks."""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from . import binding as cc


def plan_chunk_batch(lens: Sequence[int], sigma, spans: List[Tuple], capacity: float,
                     r_max: float = 1.0, m_min: float = 0.5, m_max: float = 1.5,
                     span_ratio: float = 0.5, span_min: int = 16
                     ) -> Tuple[Tuple[int, ...], np.ndarray]:
    """Budgets B_i of every chunk at base ratio ``capacity`` with capacity multipliers in
    [m_min, m_max], and the prior array whose 1.0 entries are the tokens covered by the spans
    selected under each chunk's span budget B^span = min(B_i, max(span_min, floor(span_ratio B_i))).
    ``spans[i]`` = (starts, ends, scores, protected) of chunk i."""
    budgets, _ = cc.cc_plan_budgets(sigma, lens, r=capacity, r_max=r_max, m_min=m_min, m_max=m_max)
    masks = []
    for n, b, (starts, ends, scores, prot) in zip(lens, budgets, spans):
        mask, _ = cc.cc_select_spans(starts, ends, scores, prot, int(n), int(b), span_ratio, span_min)
        masks.append(mask.astype(np.float32))
    prior = np.concatenate(masks) if masks else np.zeros(0, np.float32)
    return tuple(int(b) for b in budgets), prior


def paper_chunks(capacity: float, seed: int = 5005, count: int = 32):
    """The paper's own configuration as a benchmark workload (Appendix "Compression settings" and
    "Structural prior configuration"): ``count`` synthetic chunks of 128..4096 tokens as one
    ragged batch, average pooling of width 5, a window of 128 rows, budgets planned at the given
    capacity with multipliers in [0.5, 1.5], span ratio 0.5 with a minimum of 16 tokens, the
    protected tokens of the selected spans as the prior.  Returns (workload, prior): the prior
    replaces the generic one of ``inputs.make_layer``."""
    from . import inputs as gen
    cb = gen.chunk_batch(seed, count)
    budgets, prior = plan_chunk_batch(cb.lens, cb.sigma, cb.spans, capacity)
    wl = gen.Workload(f"paper_chunks_c{int(round(capacity * 100))}", 6, 32, 32, 8, 128, 128,
                      gen.POOL_AVG, 5, 0, seq_lens=cb.lens, seq_budgets=budgets,
                      span_ratio=0.5, span_min=16)
    return wl, prior
