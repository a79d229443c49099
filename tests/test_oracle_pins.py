"""Pins the CPU oracle to things other than itself: closed forms, library routines,
hand-worked fixtures, brute force on tiny inputs and invariants.  No GPU needed."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import inputs as gen

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    return np.random.Generator(np.random.PCG64(seed)).standard_normal(shape)


# ------------------------------------------------------------------ bf16 widening
def test_bf16_widening_matches_torch():
    bits = np.arange(0, 65536, 7, dtype=np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]          # finite patterns only
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(orc.bf16_bits_to_f64(bits), ref)


def test_generator_bf16_rounding_matches_torch():
    x = _rand(4096, 3).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(gen.f32_to_bf16_bits(x), ref)


# ------------------------------------------------------------------ window scores
def brute_scores(q, k, n_heads_kv):
    """Triple-loop restatement of Section 4.5 with grouped heads, pure Python floats."""
    w, hq, d = q.shape
    n = k.shape[0]
    g = hq // n_heads_kv
    u = [[0.0] * n for _ in range(n_heads_kv)]
    for head in range(hq):
        h = head // g
        for t in range(w):
            s = [sum(float(q[t, head, c]) * float(k[j, h, c]) for c in range(d)) / math.sqrt(d)
                 for j in range(n)]
            z = sum(math.exp(x) for x in s)
            for j in range(n):
                u[h][j] += math.exp(s[j]) / z
    return np.array(u)


@pytest.mark.parametrize("w,hq,hkv,n,d", [(1, 1, 1, 5, 4), (3, 4, 2, 9, 8), (2, 6, 2, 17, 16),
                                          (4, 3, 3, 7, 8)])
def test_scores_vs_brute_force(w, hq, hkv, n, d):
    q, k = _rand((w, hq, d), 11), _rand((n, hkv, d), 12)
    u, _ = orc.window_scores(q, k, hkv)
    np.testing.assert_allclose(u, brute_scores(q, k, hkv), rtol=1e-12, atol=1e-14)


def test_single_row_is_library_softmax():
    d, n = 128, 300
    q, k = _rand((1, 1, d), 1), _rand((n, 1, d), 2)
    u, lse = orc.window_scores(q, k, 1)
    s = torch.from_numpy(k[:, 0, :] @ q[0, 0]) / math.sqrt(d)
    np.testing.assert_allclose(u[0], torch.softmax(s, 0).numpy(), rtol=1e-12)
    np.testing.assert_allclose(lse[0, 0], torch.logsumexp(s, 0).item(), rtol=1e-13)


def test_two_key_closed_form_golden():
    with open(os.path.join(GOLD, "two_key_softmax.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        d = c["d"]
        q = np.zeros((c["w"], 1, d)); q[:, 0, 0] = c["q"]
        k = np.zeros((2, 1, d)); k[0, 0, 0] = c["a"]; k[1, 0, 0] = c["b"]
        u, _ = orc.window_scores(q, k, 1)
        np.testing.assert_allclose(u[0], c["u"], rtol=1e-13)


def test_scores_invariants_and_special_cases():
    w, hq, hkv, n, d = 5, 6, 2, 40, 32
    q, k = _rand((w, hq, d), 5), _rand((n, hkv, d), 6)
    u, _ = orc.window_scores(q, k, hkv)
    g = hq // hkv
    np.testing.assert_allclose(u.sum(axis=1), w * g, rtol=1e-12)        # rows of A sum to 1
    # identical keys or a zero query -> uniform attention
    u_c, _ = orc.window_scores(q, np.broadcast_to(k[:1], k.shape).copy(), hkv)
    np.testing.assert_allclose(u_c, w * g / n, rtol=1e-12)
    u_0, _ = orc.window_scores(np.zeros_like(q), k, hkv)
    np.testing.assert_allclose(u_0, w * g / n, rtol=1e-12)
    # adding one vector to every key shifts each softmax row by a constant
    u_s, _ = orc.window_scores(q, k + _rand((1, hkv, d), 7), hkv)
    np.testing.assert_allclose(u_s, u, rtol=1e-10)
    # a key far in the query's direction takes all the mass of that head's rows
    qpos = np.abs(q)
    k3 = np.abs(k); k3[3, 0, :] = 1e3
    u_p, _ = orc.window_scores(qpos, k3, hkv)
    np.testing.assert_allclose(u_p[0, 3], w * g, rtol=1e-9)
    # permuting the keys permutes the scores
    perm = np.random.Generator(np.random.PCG64(9)).permutation(n)
    u_perm, _ = orc.window_scores(q, k[perm], hkv)
    np.testing.assert_allclose(u_perm, u[:, perm], rtol=1e-12)


def test_gqa_head_mapping():
    """Query head i belongs to KV head i // G: give KV head 1 identical keys (uniform
    scores) and KV head 0 distinct ones."""
    w, hq, hkv, n, d = 2, 4, 2, 12, 8
    q, k = _rand((w, hq, d), 21), _rand((n, hkv, d), 22)
    k[:, 1, :] = k[0, 1, :]
    u, lse = orc.window_scores(q, k, hkv)
    np.testing.assert_allclose(u[1], w * 2 / n, rtol=1e-12)
    assert np.ptp(u[0]) > 1e-3
    # lse of the uniform head: s + log n
    s = (q[:, 2:, :] * k[0, 1, :]).sum(-1) / math.sqrt(d)            # [w][2]
    np.testing.assert_allclose(lse[2:], (s + math.log(n)).T, rtol=1e-12)


# ------------------------------------------------------------------ pooling
@pytest.mark.parametrize("width", [1, 3, 5, 7])
@pytest.mark.parametrize("n", [1, 2, 6, 50])
def test_pool_matches_library(width, n):
    u = np.abs(_rand((3, n), 30 + n))
    t = torch.from_numpy(u)[None]
    mx = torch.nn.functional.max_pool1d(t, width, 1, width // 2)[0].numpy()
    av = torch.nn.functional.avg_pool1d(t, width, 1, width // 2, count_include_pad=True)[0].numpy()
    np.testing.assert_array_equal(orc.pool_scores(u, orc.POOL_MAX, width), mx)
    np.testing.assert_allclose(orc.pool_scores(u, orc.POOL_AVG, width), av, rtol=1e-13)
    np.testing.assert_array_equal(orc.pool_scores(u, orc.POOL_NONE, width), u)


def test_pool_closed_forms():
    delta = np.zeros((1, 21)); delta[0, 10] = 2.0
    mx = orc.pool_scores(delta, orc.POOL_MAX, 7)
    assert mx[0].tolist() == [0.0] * 7 + [2.0] * 7 + [0.0] * 7          # plateau of width k
    const = np.full((1, 9), 3.0)
    av = orc.pool_scores(const, orc.POOL_AVG, 5)[0]
    np.testing.assert_allclose(av, [3 * 3 / 5, 3 * 4 / 5, 3, 3, 3, 3, 3, 3 * 4 / 5, 3 * 3 / 5])
    u32 = np.abs(_rand((2, 33), 31)).astype(np.float32)
    out = orc.pool_scores(u32, orc.POOL_AVG, 5, dtype=np.float32)
    assert out.dtype == np.float32
    j = 7                                            # left-to-right fp32 sum, then divide
    acc = np.float32(0)
    for o in range(-2, 3):
        acc = np.float32(acc + u32[1, j + o])
    assert out[1, j] == np.float32(acc / np.float32(5))


# ------------------------------------------------------------------ fuse
def test_fuse_hand_values():
    out = orc.fuse_prior(np.array([[2.0, 4.0]]), np.array([1.0, 0.5]), 0.25, 3.0)
    assert out.tolist() == [[3.5, 2.5]]
    a, b = np.float32(0.1), np.float32(0.7)
    x, p = np.float32(1.2345678), np.float32(0.3333333)
    out32 = orc.fuse_prior(np.array([[x]], np.float32), np.array([p], np.float32), 0.1, 0.7,
                           dtype=np.float32)
    assert out32.dtype == np.float32 and out32[0, 0] == np.float32(np.float32(a * x) + np.float32(b * p))


# ------------------------------------------------------------------ selection
def brute_select(fused, prior, lens, budget, theta, span_ratio, span_min):
    """Rank every item by counting the items that precede it (O(m^2)), then walk ranks."""
    m = len(fused)
    forced = [np.float32(prior[i]) >= np.float32(theta) for i in range(m)]
    if span_ratio > 0:
        cap = min(budget, max(span_min, math.floor(span_ratio * budget + 1e-9)))
        cand = [i for i in range(m) if forced[i]]

        def before_p(a, b):
            return prior[a] > prior[b] or (prior[a] == prior[b] and a < b)
        ranked = sorted(cand, key=lambda i: sum(before_p(o, i) for o in cand))
        forced = [False] * m
        tot = 0
        for i in ranked:
            tot += lens[i]
            if tot > cap:
                break
            forced[i] = True

    def before(a, b):
        if forced[a] != forced[b]:
            return forced[a]
        if forced[a]:
            return a < b                      # protected tokens: sequence order only
        if fused[a] != fused[b]:
            return fused[a] > fused[b]
        return a < b
    rank = [sum(before(o, i) for o in range(m) if o != i) for i in range(m)]
    by_rank = sorted(range(m), key=lambda i: rank[i])
    take = [0] * m
    left = min(budget, sum(lens))
    for i in by_rank:
        take[i] = min(lens[i], left)
        left -= take[i]
    return np.array(take)


def test_select_golden_cases():
    with open(os.path.join(GOLD, "select_cases.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        n = c.get("n", len(c["fused"]))
        idx = orc.select_tokens(np.array(c["fused"]), np.array(c["prior"], np.float32), n,
                                c["budget"], c["theta"], c["span_ratio"], c["span_min"],
                                c["chunk"])
        assert idx.tolist() == c["idx"], c["name"]


@pytest.mark.parametrize("seed", range(12))
def test_select_vs_brute_force(seed):
    rng = np.random.Generator(np.random.PCG64(100 + seed))
    m = int(rng.integers(1, 40))
    chunk = int(rng.choice([1, 1, 3, 4]))
    n = m * chunk - int(rng.integers(0, chunk))
    lens = orc.chunk_lengths(n, chunk)
    m = len(lens)
    fused = rng.choice(np.round(rng.random(6), 2), size=m)            # many exact ties
    prior = rng.choice([0.0, 0.0, 0.3, 0.6, 0.9], size=m).astype(np.float32)
    budget = int(rng.integers(0, n + 3))
    ratio = float(rng.choice([0.0, 0.5, 0.7]))
    take = orc.select_items(fused, prior, lens, budget, 0.5, ratio, 2)
    ref = brute_select(fused, prior, lens, budget, 0.5, ratio, 2)
    np.testing.assert_array_equal(take, ref)


def test_select_invariants():
    rng = np.random.Generator(np.random.PCG64(77))
    n = 500
    fused = rng.random(n)
    prior = (rng.random(n) < 0.1).astype(np.float32)
    forced = np.flatnonzero(prior >= 0.5)
    for budget in [0, 1, len(forced) - 1, len(forced), len(forced) + 10, n - 1, n, n + 5]:
        idx = orc.select_tokens(fused, prior, n, budget, 0.5)
        assert len(idx) == min(budget, n)                               # count = B exactly
        assert np.all(np.diff(idx) > 0)                                 # ascending, unique
        if budget >= len(forced):
            assert set(forced) <= set(idx.tolist())                     # all protected kept
            rest = np.setdiff1d(idx, forced)
            out = np.setdiff1d(np.arange(n), idx)
            if len(rest) and len(out):
                assert fused[rest].min() >= fused[out].max()
        else:
            assert idx.tolist() == forced[:budget].tolist()             # first B of P


def test_span_budget_hand_values():
    assert orc.span_budget(100, 0.5, 16) == 50
    assert orc.span_budget(20, 0.5, 16) == 16
    assert orc.span_budget(10, 0.5, 16) == 10
    assert orc.span_budget(10, 0.7, 0) == 7
    assert orc.span_budget(100, 0.29, 0) == 29


# ------------------------------------------------------------------ chunks
def test_chunk_reduce_definition():
    u = _rand((2, 23), 40)
    p = np.zeros(23, np.float32); p[[4, 22]] = [0.7, 0.2]
    us, ps = orc.chunk_reduce(u, p, 10)
    for c, (lo, hi) in enumerate([(0, 10), (10, 20), (20, 23)]):
        acc = u[:, lo].copy()
        for j in range(lo + 1, hi):
            acc = acc + u[:, j]
        np.testing.assert_array_equal(us[:, c], acc)
    assert ps.tolist() == [np.float32(0.7), 0.0, np.float32(0.2)]
    np.testing.assert_allclose(us.sum(1), u.sum(1), rtol=1e-12)
    assert orc.chunk_lengths(23, 10).tolist() == [10, 10, 3]
    assert orc.chunk_lengths(20, 10).tolist() == [10, 10]


# ------------------------------------------------------------------ compaction / paged layout
def test_compact_is_row_gather():
    k = np.arange(6 * 2 * 4, dtype=np.uint16).reshape(6, 2, 4)
    v = k + 1000
    idx = [np.array([0, 5]), np.array([2, 3, 4])]
    ko, vo = orc.compact_kv(k, v, idx)
    for h in range(2):
        for s, j in enumerate(idx[h]):
            assert ko[h][s].tolist() == k[j, h].tolist()
            assert vo[h][s].tolist() == v[j, h].tolist()


def test_paged_helpers():
    table = np.array([7, 2, 9], dtype=np.int32)
    rows = orc.paged_rows(table, 10, 4)
    assert rows.tolist() == [28, 29, 30, 31, 8, 9, 10, 11, 36, 37]
    pages = orc.assign_output_pages([5, 0, 9], [100, 100, 6], 4, np.arange(50, 60))
    assert [p.tolist() for p in pages] == [[50, 51], [], [52, 53]]


# ------------------------------------------------------------------ whole path
def test_compress_sequence_invariants_on_tiny_workload():
    wl = gen.workloads()["tiny"]
    x = gen.make_layer(wl)
    res = orc.compress_sequence(x.q_win[0], x.k, x.v, x.prior, wl.n_heads_kv, wl.pool_kind,
                                wl.pool_size, wl.budget, wl.alpha, wl.beta, wl.force_threshold)
    g = wl.group
    np.testing.assert_allclose(res["scores"].sum(1), wl.window * g, rtol=1e-12)
    forced = np.flatnonzero(x.prior >= 0.5)
    assert 0 < len(forced) < wl.budget
    for h in range(wl.n_heads_kv):
        idx = res["idx"][h]
        assert len(idx) == wl.budget and np.all(np.diff(idx) > 0)
        assert set(forced) <= set(idx.tolist())
        np.testing.assert_array_equal(res["k_out"][h], x.k[idx, h])
        np.testing.assert_array_equal(res["v_out"][h], x.v[idx, h])
        assert np.all(res["pooled"][h] >= res["scores"][h])             # max-pool dominates


def _compose_by_hand(q_bits, k_bits, prior, hkv, pool_kind, pool_size, budget, alpha, beta, theta,
                     span_ratio, span_min, chunk):
    """The whole path written out from the stage functions that the tests above pin one by one
    (scalar loops for the chunk level and the fusion, so that no helper of compress_sequence's
    wiring is reused)."""
    u, _ = orc.window_scores(orc.bf16_bits_to_f64(q_bits), orc.bf16_bits_to_f64(k_bits), hkv)
    n = u.shape[1]
    out = []
    for h in range(hkv):
        if chunk > 1:
            m = (n + chunk - 1) // chunk
            item = [sum(u[h, c * chunk:min(n, (c + 1) * chunk)]) for c in range(m)]
            item_p = [max(prior[c * chunk:min(n, (c + 1) * chunk)]) for c in range(m)]
        else:
            item = list(orc.pool_scores(u[h:h + 1], pool_kind, pool_size)[0])
            item_p = list(prior)
        fused = [alpha * a + beta * p for a, p in zip(item, item_p)]
        out.append(orc.select_tokens(np.array(fused), np.array(item_p, np.float32), n, budget,
                                     theta, span_ratio, span_min, chunk))
    return out


@pytest.mark.parametrize("chunk,span_ratio,span_min,beta", [(1, 0.5, 2, 0.0), (5, 0.0, 0, 0.3),
                                                          (5, 0.5, 2, 0.0), (4, 0.4, 5, 0.7)])
def test_compress_sequence_wiring_with_chunks_and_span_cap(chunk, span_ratio, span_min, beta):
    """30 tokens; priors of several sizes placed so that a chunk's prior (its maximum) differs
    from the prior of its first token, and more protected tokens than the span budget: taking
    the token prior for the chunk prior, dropping the cap arguments or swapping alpha and beta
    changes the retained set."""
    n, hq, hkv, w, budget = 30, 4, 2, 3, 12
    q, k, v = gen.small_case(77, n, w, hq, hkv)
    prior = np.zeros(n, np.float32)
    prior[[3, 7, 8, 14, 21, 22, 23, 29]] = [0.9, 0.6, 1.0, 0.8, 0.7, 0.55, 0.95, 0.65]
    res = orc.compress_sequence(q, k, v, prior, hkv, orc.POOL_MAX if chunk == 1 else orc.POOL_NONE,
                                3 if chunk == 1 else 1, budget, 1.0, beta, 0.5, span_ratio,
                                span_min, chunk)
    ref = _compose_by_hand(q, k, prior, hkv, orc.POOL_MAX if chunk == 1 else orc.POOL_NONE,
                           3 if chunk == 1 else 1, budget, 1.0, beta, 0.5, span_ratio, span_min, chunk)
    for h in range(hkv):
        assert len(res["idx"][h]) == budget
        assert res["idx"][h].tolist() == ref[h].tolist()
        np.testing.assert_array_equal(res["k_out"][h], k[res["idx"][h], h])
    if chunk > 1:
        # the chunk prior is the maximum over the chunk, not the prior of its first token
        m = (n + chunk - 1) // chunk
        assert res["item_prior"].tolist() == [float(prior[c * chunk:(c + 1) * chunk].max()) for c in range(m)]
        assert any(res["item_prior"][c] != prior[c * chunk] for c in range(m))
    if span_ratio > 0:
        cap = orc.span_budget(budget, span_ratio, span_min)
        lens = orc.chunk_lengths(n, chunk)
        prot = orc.protected_items(res["item_prior"], lens, budget, 0.5, span_ratio, span_min)
        uncapped = orc.protected_items(res["item_prior"], lens, budget, 0.5)
        assert lens[prot].sum() <= cap < lens[uncapped].sum()      # the cap is what limits them
        # the retained set differs from what the uncapped rule would keep
        other = orc.compress_sequence(q, k, v, prior, hkv, orc.POOL_MAX if chunk == 1 else orc.POOL_NONE,
                                      3 if chunk == 1 else 1, budget, 1.0, beta, 0.5, 0.0, 0, chunk)
        assert any(other["idx"][h].tolist() != res["idx"][h].tolist() for h in range(hkv))


def test_workload_recipe_statistics():
    wls = gen.workloads()
    p, lab = gen.structural_prior(1, 200000)
    assert abs(p.mean() - 0.0666) < 0.004                 # 0.29 * E[min(3, len)] / 12
    assert set(np.unique(p)) == {0.0, 1.0}
    assert wls["ragged_paged"].lens == gen.workloads()["ragged_paged"].lens   # seeded
    assert all(8192 <= s <= 65536 for s in wls["ragged_paged"].lens)
    for dens, target in [("5", 0.05), ("15", 0.15), ("30", 0.30)]:
        v = gen.qwen_variant(wls["qwen25_coder_7b"], 4096, dens)
        pp, _ = gen.structural_prior(2, 200000, v.p_structural, v.flagged_per_line)
        assert abs(pp.mean() - target) < 0.012
    small = gen.Workload("s", 9, 1, 4, 2, 128, 8, gen.POOL_MAX, 3, 8, seq_lens=(40, 70),
                         budget_frac=0.1, page_size=16)
    x = gen.make_layer(small)
    assert x.page_table.shape == (2, 5) and x.k.shape[0] == x.pool_pages * 16
    y = gen.make_layer(gen.Workload("s", 9, 1, 4, 2, 128, 8, gen.POOL_MAX, 3, 8, seq_lens=(40, 70),
                                    budget_frac=0.1))
    rows = orc.paged_rows(x.page_table[1], 70, 16)
    np.testing.assert_array_equal(x.k[rows], y.k[40:110])                  # same bits, scattered
    assert len(set(x.free_pages.tolist()) & set(x.page_table[x.page_table >= 0].tolist())) == 0


# --------------------------------------------------------------------------- Str. Score
def test_structural_score_hand_values():
    """Section 5.3 (table caption): fraction of structurally critical tokens retained.
    Worked by hand: critical = {0, 2, 3, 6}; a retained set {0, 1, 3} holds two of the four."""
    prior = np.array([1, 0, 1, 1, 0, 0, 1], dtype=np.float32)
    frac, hit, tot = orc.structural_score(np.array([0, 1, 3, -1]), prior, 0.5)
    assert (frac, hit, tot) == (0.5, 2, 4)
    assert orc.structural_score(np.array([0, 2, 3, 6]), prior, 0.5) == (1.0, 4, 4)
    assert orc.structural_score(np.array([1, 4, 5]), prior, 0.5) == (0.0, 0, 4)
    # no critical token at all: nothing can be lost
    assert orc.structural_score(np.array([1, 4]), prior, 2.0) == (1.0, 0, 0)
    # the threshold is inclusive, like the protection rule of the selection
    assert orc.structural_score(np.array([0]), np.array([0.5, 0.49]), 0.5) == (1.0, 1, 1)


@pytest.mark.parametrize("seed", range(4))
def test_structural_score_vs_counting_loop(seed):
    rng = np.random.Generator(np.random.PCG64(900 + seed))
    n = 300
    prior = (rng.random(n) < 0.2).astype(np.float32)
    idx = np.sort(rng.choice(n, size=60, replace=False))
    hit = tot = 0
    for j in range(n):
        if prior[j] >= 0.5:
            tot += 1
            hit += int(j in idx)
    assert orc.structural_score(idx, prior, 0.5) == (hit / tot, hit, tot)


def test_structural_score_is_one_when_protected_tokens_fit_the_budget():
    """Section 4.4 "Token-level protection": protected tokens are kept first, so when they fit
    the budget the retained set of every head contains all of them."""
    wl = gen.workloads()["tiny"]
    x = gen.make_layer(wl)
    res = orc.compress_sequence(x.q_win[0], x.k, None, x.prior, wl.n_heads_kv, wl.pool_kind,
                                wl.pool_size, wl.budget, wl.alpha, wl.beta, wl.force_threshold)
    assert int((x.prior >= wl.force_threshold).sum()) <= wl.budget
    for h in range(wl.n_heads_kv):
        frac, hit, tot = orc.structural_score(res["idx"][h], x.prior, wl.force_threshold)
        assert frac == 1.0 and hit == tot > 0
    # without protection (threshold out of reach for the selection) attention alone keeps fewer
    res2 = orc.compress_sequence(x.q_win[0], x.k, None, x.prior, wl.n_heads_kv, wl.pool_kind,
                                 wl.pool_size, wl.budget, wl.alpha, wl.beta, float("inf"))
    assert orc.structural_score(res2["idx"][0], x.prior, wl.force_threshold)[0] < 1.0


# --------------------------------------------------------------------------- causal window
def test_causal_window_closed_form_with_identical_keys():
    """All keys equal: row t spreads its mass evenly over the n - w + t + 1 keys it sees, so
    u(j) = G * sum over the rows that see j of 1 / (keys the row sees)."""
    n, w, hq, hkv, d = 40, 6, 4, 2, 128
    rng = np.random.Generator(np.random.PCG64(5))
    q = rng.standard_normal((w, hq, d))
    k = np.broadcast_to(rng.standard_normal((1, hkv, d)), (n, hkv, d)).copy()
    u, lse = orc.window_scores(q, k, hkv, causal=True)
    g = hq // hkv
    want = np.zeros(n)
    for t in range(w):
        seen = n - w + t + 1
        want[:seen] += g / seen
    np.testing.assert_allclose(u[0], want, rtol=1e-12)
    np.testing.assert_allclose(u.sum(axis=1), w * g, rtol=1e-12)
    # lse of row t = s + log(keys seen)
    s00 = q[0, 0] @ k[0, 0] / math.sqrt(d)
    np.testing.assert_allclose(lse[0, 0], s00 + math.log(n - w + 1), rtol=1e-12)


@pytest.mark.parametrize("seed", range(3))
def test_causal_window_vs_scalar_loops(seed):
    rng = np.random.Generator(np.random.PCG64(700 + seed))
    n, w, hq, hkv, d = 11, 4, 2, 1, 128
    q = rng.standard_normal((w, hq, d))
    k = rng.standard_normal((n, hkv, d))
    u, _ = orc.window_scores(q, k, hkv, causal=True)
    ref = np.zeros(n)
    for gi in range(hq):
        for t in range(w):
            last = n - w + t
            s = [sum(q[t, gi, c] * k[j, 0, c] for c in range(d)) / math.sqrt(d) for j in range(last + 1)]
            z = sum(math.exp(x) for x in s)
            for j in range(last + 1):
                ref[j] += math.exp(s[j]) / z
    np.testing.assert_allclose(u[0], ref, rtol=1e-10)
    # the last key is seen by the last row only; keys before the window are seen by all rows
    assert u[0, n - 1] <= hq and np.all(u[0] > 0)


def test_causal_window_differs_from_unmasked_only_through_the_last_keys():
    rng = np.random.Generator(np.random.PCG64(77))
    n, w, hq, hkv, d = 64, 8, 2, 2, 128
    q, k = rng.standard_normal((w, hq, d)), rng.standard_normal((n, hkv, d))
    u_c, lse_c = orc.window_scores(q, k, hkv, causal=True)
    u_f, lse_f = orc.window_scores(q, k, hkv, causal=False)
    # the last row sees every key: identical log-sum-exp; earlier rows see fewer: smaller
    np.testing.assert_allclose(lse_c[:, w - 1], lse_f[:, w - 1], rtol=1e-13)
    assert np.all(lse_c[:, :w - 1] < lse_f[:, :w - 1])
    with pytest.raises(ValueError):
        orc.window_scores(q, k[:4], hkv, causal=True)


# --------------------------------------------------------------------------- budget planner
def test_plan_budgets_hand_values():
    """Section 4.3, worked by hand with the appendix's multiplier range [0.5, 1.5]:
    sigma = (.2, .5, .8) -> s~ = (0, .5, 1) -> m = (.5, 1, 1.5) -> ratios (.2, .4, .6)."""
    b, m = orc.plan_budgets([0.2, 0.5, 0.8], [1000, 2000, 4096], 0.4, 1.0, 0.5, 1.5, 1e-6)
    np.testing.assert_allclose(m, [0.5, 1.0, 1.5], rtol=1e-12)
    assert b.tolist() == [200, 800, 2457]                     # floor(2457.6)
    # equal scores: s~ = 0.5 for everyone, the multiplier is the middle of the range
    b, m = orc.plan_budgets([0.3, 0.3], [512, 4096], 0.6, 1.0, 0.5, 1.5, 1e-6)
    assert m.tolist() == [1.0, 1.0] and b.tolist() == [307, 2457]
    # the ratio is capped at r_max: 0.8 * 1.5 = 1.2 -> 1.0 -> the whole chunk
    b, _ = orc.plan_budgets([0.0, 1.0], [100, 100], 0.8, 1.0, 0.5, 1.5, 1e-6)
    assert b.tolist() == [40, 100]
    # a spread below eps is divided by eps, not by itself
    _, m = orc.plan_budgets([0.5, 0.5 + 1e-9], [10, 10], 0.5, 1.0, 0.5, 1.5, 1e-6)
    np.testing.assert_allclose(m, [0.5, 0.5 + 1e-3], rtol=1e-6)
    assert orc.plan_budgets([], [], 0.4, 1.0, 0.5, 1.5, 1e-6)[0].size == 0


def test_plan_budgets_invariants():
    rng = np.random.Generator(np.random.PCG64(31))
    sigma = rng.random(50)
    lens = np.full(50, 3000)
    b, m = orc.plan_budgets(sigma, lens, 0.4, 0.9, 0.5, 1.5, 1e-6)
    order = np.argsort(sigma)
    assert np.all(np.diff(b[order]) >= 0)                      # more structure, more capacity
    assert m.min() == 0.5 and m.max() == 1.5                   # the extremes map to the range ends
    assert np.all(b <= np.floor(lens * 0.9 + 1e-9)) and np.all(b >= np.floor(lens * 0.4 * 0.5))


def test_select_spans_hand_case():
    """Section 4.4: B = 10, rho = 0.5, B_min = 2 -> B^span = 5.  The protected span (3 tokens)
    comes first; of the two spans with score .9 the earlier one follows (7 covered >= 5: stop)."""
    starts, ends = [0, 5, 10, 20], [3, 9, 12, 25]
    mask, taken = orc.select_spans(starts, ends, [0.2, 0.9, 0.9, 0.5], [True, False, False, False],
                                   30, 10, 0.5, 2)
    assert taken == [0, 1]
    assert np.flatnonzero(mask).tolist() == [0, 1, 2, 5, 6, 7, 8]
    # protected spans are taken even beyond the span budget; nothing else follows then
    mask, taken = orc.select_spans(starts, ends, [0.2, 0.9, 0.9, 0.5], [True, False, False, True],
                                   30, 10, 0.5, 2)
    assert taken == [0, 3] and int(mask.sum()) == 8
    # overlapping spans count their union
    mask, taken = orc.select_spans([0, 2], [4, 6], [0.5, 0.4], [False, False], 10, 10, 1.0, 1)
    assert taken == [0, 1] and int(mask.sum()) == 6
    assert orc.select_spans([], [], [], [], 5, 3, 0.5, 1)[1] == []


@pytest.mark.parametrize("seed", range(5))
def test_select_spans_properties(seed):
    rng = np.random.Generator(np.random.PCG64(400 + seed))
    n, k = 200, 25
    starts = rng.integers(0, n - 10, size=k)
    ends = starts + rng.integers(1, 10, size=k)
    scores = rng.integers(0, 5, size=k) / 4.0                  # many ties
    prot = rng.random(k) < 0.15
    budget, rho, bmin = 60, 0.5, 16
    cap = orc.span_budget(budget, rho, bmin)
    mask, taken = orc.select_spans(starts, ends, scores, prot, n, budget, rho, bmin)
    n_prot = int(prot.sum())
    assert taken[:n_prot] == [i for i in range(k) if prot[i]]
    rest = taken[n_prot:]
    rank = sorted((i for i in range(k) if not prot[i]), key=lambda i: (-scores[i], starts[i], i))
    assert rest == rank[:len(rest)]                            # a prefix of the rank order
    cover = np.zeros(n, dtype=bool)
    for i in taken[:-1] if rest else taken:
        cover[starts[i]:ends[i]] = True
    if rest:
        assert cover.sum() < cap                               # the last one was still needed
    if len(rest) < len(rank):
        assert mask.sum() >= cap                               # stopped because the budget is used
    want = np.zeros(n, dtype=bool)
    for i in taken:
        want[starts[i]:ends[i]] = True
    assert np.array_equal(mask, want)


# --------------------------------------------------------------------------- chunk selection
def test_ppl_scores_closed_forms():
    """Section 4.1.  Uniform logits: p = 1/V for every token, so the score is log V.  One-hot
    logits of height a on the target: -log p = log(1 + (V - 1) e^-a)."""
    chunks, t, v = 3, 5, 11
    tgt = np.array([0, 3, 10, 3, 7])
    s, nll = orc.ppl_chunk_scores(np.zeros((chunks, t, v)), tgt)
    np.testing.assert_allclose(s, math.log(v), rtol=1e-14)
    a = 2.5
    x = np.zeros((1, t, v))
    x[0, np.arange(t), tgt] = a
    s, nll = orc.ppl_chunk_scores(x, tgt)
    np.testing.assert_allclose(nll, math.log(1 + (v - 1) * math.exp(-a)), rtol=1e-13)
    # adding a constant to a row changes nothing; the score is the mean over the query tokens
    y = x + np.arange(t)[None, :, None] * 100.0
    np.testing.assert_allclose(orc.ppl_chunk_scores(y, tgt)[1], nll, rtol=1e-12)
    x[0, 0, :] = 0.0
    s2, nll2 = orc.ppl_chunk_scores(x, tgt)
    np.testing.assert_allclose(s2[0], (math.log(v) + (t - 1) * nll[0, 1]) / t, rtol=1e-13)


def test_ppl_scores_vs_scalar_loops():
    rng = np.random.Generator(np.random.PCG64(12))
    x = rng.standard_normal((2, 3, 7)) * 3
    tgt = np.array([6, 0, 2])
    s, nll = orc.ppl_chunk_scores(x, tgt)
    for i in range(2):
        acc = 0.0
        for t in range(3):
            z = sum(math.exp(x[i, t, j]) for j in range(7))
            want = -math.log(math.exp(x[i, t, tgt[t]]) / z)
            assert abs(nll[i, t] - want) < 1e-12
            acc += want
        assert abs(s[i] - acc / 3) < 1e-12


def test_select_chunks_lowest_first_with_ties():
    s = np.array([2.0, 0.5, 2.0, 0.5, np.nan, 1.0])
    assert orc.select_chunks(s, 3).tolist() == [1, 3, 5]
    assert orc.select_chunks(s, 6).tolist() == [1, 3, 5, 0, 2, 4]
    assert orc.select_chunks(s, 9).tolist() == [1, 3, 5, 0, 2, 4]
    assert orc.select_chunks(s, 0).tolist() == []
    rng = np.random.Generator(np.random.PCG64(3))
    r = rng.integers(0, 6, size=40).astype(np.float64)
    got = orc.select_chunks(r, 10)
    assert np.array_equal(np.sort(r)[:10], r[got])           # against the library sort
    assert all(r[a] < r[b] or (r[a] == r[b] and a < b) for a, b in zip(got[:-1], got[1:]))


# ------------------------------------------------------------------ nearest-to-protected fill
def test_nearest_fill_hand_cases():
    """Section 4.4, last sentence of "Token-level protection": worked by hand."""
    #            0  1  2  3  4  5  6  7  8  9
    prior = np.array([0, 0, 1, 0, 0, 0, 0, 1, 0, 0], np.float32)
    assert (-orc.nearest_fill_values(prior, 0.5)).tolist() == [2, 1, 0, 1, 2, 2, 1, 0, 1, 2]
    # budget 6: the two protected tokens, then distance 1 (1, 3, 6, 8 in index order)
    assert orc.select_tokens(orc.nearest_fill_values(prior, 0.5), prior, 10, 6, 0.5).tolist() == [1, 2, 3, 6, 7, 8]
    # budget 5: of the four tokens at distance 1 the three with the lowest index
    assert orc.select_tokens(orc.nearest_fill_values(prior, 0.5), prior, 10, 5, 0.5).tolist() == [1, 2, 3, 6, 7]
    # no protected token: the first tokens of the sequence
    none = np.zeros(7, np.float32)
    assert (-orc.nearest_fill_values(none, 0.5)).tolist() == [7] * 7
    assert orc.select_tokens(orc.nearest_fill_values(none, 0.5), none, 7, 3, 0.5).tolist() == [0, 1, 2]
    # protected token at one end only
    end = np.array([0, 0, 0, 0, 1], np.float32)
    assert (-orc.nearest_fill_values(end, 0.5)).tolist() == [4, 3, 2, 1, 0]


@pytest.mark.parametrize("seed", range(6))
def test_nearest_fill_vs_quadratic_loop(seed):
    rng = np.random.Generator(np.random.PCG64(900 + seed))
    n = int(rng.integers(1, 120))
    prior = (rng.random(n) < rng.choice([0.0, 0.05, 0.3])).astype(np.float32) * np.float32(0.8)
    got = -orc.nearest_fill_values(prior, 0.5)
    prot = [j for j in range(n) if prior[j] >= 0.5]
    want = [min((abs(j - p) for p in prot), default=n) for j in range(n)]
    assert got.tolist() == want
    # the retained set: every protected token, then by (distance, index)
    b = int(rng.integers(0, n + 1))
    ref = sorted(sorted(range(n), key=lambda j: (0 if prior[j] >= 0.5 else 1, want[j], j))[:b]) \
        if len(prot) <= b else prot[:b]
    assert orc.select_tokens(-got, prior, n, b, 0.5).tolist() == ref
