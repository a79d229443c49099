"""Host-side planning calls of the C ABI (cc_plan_budgets, cc_select_spans) against the oracle.
They touch no GPU, so they run everywhere; integer outputs are compared bit for bit."""
import numpy as np
import pytest

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc


def test_plan_budgets_paper_like_case():
    """Appendix "Structural prior configuration": multipliers in [0.5, 1.5]; capacity 0.4."""
    b, m = cc.cc_plan_budgets([0.2, 0.5, 0.8], [1000, 2000, 4096], r=0.4)
    assert b.tolist() == [200, 800, 2457]
    np.testing.assert_allclose(m, [0.5, 1.0, 1.5], rtol=1e-12)


@pytest.mark.parametrize("seed", range(6))
def test_plan_budgets_matches_oracle(seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    k = int(rng.integers(1, 40))
    sigma = rng.random(k)
    if seed == 0:
        sigma[:] = sigma[0]                                   # all equal
    if seed == 1:
        sigma = 0.5 + rng.random(k) * 1e-7
    lens = rng.integers(0, 4097, size=k)
    r = float(rng.choice([0.4, 0.6, 0.8]))
    got_b, got_m = cc.cc_plan_budgets(sigma, lens, r=r, r_max=0.9, m_min=0.5, m_max=1.5, eps=1e-6)
    ref_b, ref_m = orc.plan_budgets(sigma, lens, r, 0.9, 0.5, 1.5, 1e-6)
    assert got_b.tolist() == ref_b.tolist()
    assert np.array_equal(got_m, ref_m)                       # same double operations, same bits


def test_plan_budgets_rejects_bad_input():
    with pytest.raises(cc.CodecompError):
        cc.cc_plan_budgets([float("nan")], [10], r=0.4)
    with pytest.raises(cc.CodecompError):
        cc.cc_plan_budgets([0.1], [-1], r=0.4)
    with pytest.raises(cc.CodecompError):
        cc.cc_plan_budgets([0.1], [10], r=0.4, m_min=2.0, m_max=1.0)
    b, m = cc.cc_plan_budgets([], [], r=0.4)
    assert b.size == 0 and m.size == 0


def test_select_spans_hand_case():
    mask, taken = cc.cc_select_spans([0, 5, 10, 20], [3, 9, 12, 25], [0.2, 0.9, 0.9, 0.5],
                                     [1, 0, 0, 0], 30, 10, 0.5, 2)
    assert taken.tolist() == [0, 1]
    assert np.flatnonzero(mask).tolist() == [0, 1, 2, 5, 6, 7, 8]


@pytest.mark.parametrize("seed", range(8))
def test_select_spans_matches_oracle(seed):
    rng = np.random.Generator(np.random.PCG64(50 + seed))
    n, k = 300, int(rng.integers(0, 40))
    starts = rng.integers(0, n - 12, size=k)
    ends = starts + rng.integers(0, 12, size=k)               # empty spans included
    scores = (rng.integers(0, 6, size=k) / 5.0).astype(np.float32)
    prot = rng.random(k) < 0.1
    budget = int(rng.integers(0, 120))
    rho = float(rng.choice([0.0, 0.5, 1.0]))
    got_mask, got_taken = cc.cc_select_spans(starts, ends, scores, prot, n, budget, rho, 16)
    ref_mask, ref_taken = orc.select_spans(starts, ends, scores, prot, n, budget, rho, 16)
    assert got_taken.tolist() == ref_taken
    assert np.array_equal(got_mask > 0, ref_mask)


def test_select_spans_rejects_bad_ranges():
    with pytest.raises(cc.CodecompError):
        cc.cc_select_spans([5], [3], [0.1], [0], 10, 4, 0.5, 1)        # end before start
    with pytest.raises(cc.CodecompError):
        cc.cc_select_spans([5], [12], [0.1], [0], 10, 4, 0.5, 1)       # beyond the chunk


def test_planned_protection_feeds_the_selection():
    """The mask of cc_select_spans, used as the prior, is what the selection keeps first
    (Section 4.4 "Token-level protection"): all of it when it fits the budget."""
    rng = np.random.Generator(np.random.PCG64(9))
    n, budget = 400, 60
    mask, _ = cc.cc_select_spans([10, 100, 300], [20, 112, 305], [0.5, 0.4, 0.3], [0, 0, 0], n,
                                 budget, 0.5, 16)
    assert 16 <= int(mask.sum()) <= 30 + 12                   # B_span = 30, last span may overshoot
    fused = rng.random(n).astype(np.float32)
    kept = orc.select_tokens(fused, mask.astype(np.float32), n, budget, 0.5, 0.0, 0, 1)
    assert set(np.flatnonzero(mask)) <= set(kept.tolist())


@pytest.mark.parametrize("capacity", [0.4, 0.6])
def test_planned_chunk_batch_matches_the_oracle(capacity):
    """Budgets and protected-token masks of a 32-chunk batch, as `planning.plan_chunk_batch` hands
    them to the compression call, against the oracle's planner (Sections 4.3 and 4.4)."""
    from paper_2604_10235_b200 import inputs as gen
    from paper_2604_10235_b200 import planning
    cb = gen.chunk_batch(5005)
    budgets, prior = planning.plan_chunk_batch(cb.lens, cb.sigma, cb.spans, capacity)
    ref_b, _ = orc.plan_budgets(cb.sigma, cb.lens, capacity, 1.0, 0.5, 1.5, 1e-6)
    assert list(budgets) == ref_b.tolist()
    off, binding_caps = 0, 0
    for n, b, (st, en, sc, pr) in zip(cb.lens, budgets, cb.spans):
        ref_mask, _ = orc.select_spans(st, en, sc, pr, n, b, 0.5, 16)
        assert np.array_equal(prior[off:off + n] > 0, ref_mask)
        binding_caps += int(ref_mask.sum() >= orc.span_budget(b, 0.5, 16))
        off += n
    assert off == len(prior)
    assert binding_caps >= len(cb.lens) // 2          # the span budget is what limits most chunks
    wl, p2 = planning.paper_chunks(capacity)
    assert wl.lens == cb.lens and wl.budgets == budgets and np.array_equal(p2, prior)
