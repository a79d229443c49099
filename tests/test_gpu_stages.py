"""Stage-by-stage parity of the CUDA path against the oracle, through the C ABI.
Integer and byte outputs are compared bit for bit on identical fp32 inputs."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen

from gpu_util import bf16_dev, bits_host, ctx, desc_for, f32_dev

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")
GUARD = 64


def guarded(shape, dtype, fill):
    """Output tensor with guard words on both sides; returns (view, full, fill)."""
    n = int(np.prod(shape))
    full = torch.full((n + 2 * GUARD,), fill, dtype=dtype, device="cuda")
    return full[GUARD:GUARD + n].view(*shape), full


def guards_intact(full, fill):
    return bool((full[:GUARD] == fill).all() and (full[-GUARD:] == fill).all())


# ------------------------------------------------------------------ A2 + A3
@pytest.mark.parametrize("n", [1, 2, 15, 129, 2048, 4099])
@pytest.mark.parametrize("kind,width", [(cc.CC_POOL_NONE, 1), (cc.CC_POOL_MAX, 7), (cc.CC_POOL_MAX, 3),
                                        (cc.CC_POOL_AVG, 5), (cc.CC_POOL_AVG, 1), (cc.CC_POOL_MAX, 63)])
def test_fuse_prior_pool_token_level(n, kind, width):
    rng = np.random.Generator(np.random.PCG64(n * 100 + width))
    hkv = 3
    u = np.abs(rng.standard_normal((hkv, n))).astype(np.float32) * np.float32(1e-3)
    prior = (rng.random(n) < 0.2).astype(np.float32) * rng.random(n).astype(np.float32)
    alpha, beta = 0.37, 1.25
    d = cc.Desc(hkv * 2, hkv, 4, n=n, budget=1, pool_kind=kind, pool_size=width, alpha=alpha, beta=beta)
    out, full = guarded((hkv, n), torch.float32, -7.0)
    cc.cc_fuse_prior_pool(ctx(), d, f32_dev(u), f32_dev(prior), out)
    ref = orc.fuse_prior(orc.pool_scores(u, kind, width, dtype=np.float32), prior[None, :], alpha,
                         beta, dtype=np.float32)
    np.testing.assert_array_equal(out.cpu().numpy(), ref)
    assert guards_intact(full, -7.0)


@pytest.mark.parametrize("n,chunk", [(23, 10), (20, 10), (5, 10), (32768, 10), (1000, 3)])
def test_fuse_prior_pool_chunk_level(n, chunk):
    rng = np.random.Generator(np.random.PCG64(n + chunk))
    hkv = 2
    u = np.abs(rng.standard_normal((hkv, n))).astype(np.float32)
    prior = (rng.random(n) < 0.1).astype(np.float32)
    d = cc.Desc(hkv, hkv, 4, n=n, budget=1, pool_kind=cc.CC_POOL_NONE, pool_size=1,
                chunk_size=chunk, alpha=0.5, beta=2.0)
    m = d.m_tot
    out, full = guarded((hkv, m), torch.float32, -7.0)
    cc.cc_fuse_prior_pool(ctx(), d, f32_dev(u), f32_dev(prior), out)
    cu, cp = orc.chunk_reduce(u, prior, chunk, dtype=np.float32)
    ref = orc.fuse_prior(cu, cp[None, :], 0.5, 2.0, dtype=np.float32)
    np.testing.assert_array_equal(out.cpu().numpy(), ref)
    assert guards_intact(full, -7.0)


# ------------------------------------------------------------------ A4
def run_select(fused, prior, n, budget, theta, span_ratio=0.0, span_min=0, chunk=1):
    hkv = fused.shape[0]
    d = cc.Desc(hkv, hkv, 4, n=n, budget=budget, pool_kind=cc.CC_POOL_NONE, pool_size=1,
                chunk_size=chunk, force_threshold=theta, span_ratio=span_ratio, span_min=span_min)
    idx_c, full = guarded((hkv, budget), torch.int32, -99)
    count = torch.full((hkv,), -5, dtype=torch.int32, device="cuda")
    cc.cc_topk_select(ctx(), d, f32_dev(fused), f32_dev(prior), idx_c, count)
    assert ctx().poll() == 0
    assert guards_intact(full, -99)
    return idx_c.cpu().numpy(), count.cpu().numpy()


def test_select_golden_cases():
    with open(os.path.join(GOLD, "select_cases.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        n = c.get("n", len(c["fused"]))
        fused = np.array([c["fused"]], dtype=np.float32)
        idx, count = run_select(fused, np.array(_token_prior(c, n), np.float32), n, c["budget"],
                                c["theta"], c["span_ratio"], c["span_min"], c["chunk"])
        keep = min(c["budget"], n)
        assert count[0] == keep, c["name"]
        assert idx[0, :keep].tolist() == c["idx"], c["name"]
        assert (idx[0, keep:] == -1).all()


def _token_prior(c, n):
    """The fixtures give one prior per item; put it on the first token of each chunk."""
    if c["chunk"] == 1:
        return c["prior"]
    p = [0.0] * n
    for i, v in enumerate(c["prior"]):
        p[i * c["chunk"]] = v
    return p


@pytest.mark.parametrize("n", [1, 15, 16, 17, 127, 128, 129, 2048, 4099, 32768, 65536])
def test_select_matches_oracle_bit_exact(n):
    rng = np.random.Generator(np.random.PCG64(n))
    hkv = 2
    u = (np.abs(rng.standard_normal((hkv, n))) * 1e-3).astype(np.float32)
    fused = orc.pool_scores(u, orc.POOL_MAX, 7, dtype=np.float32)      # runs of exact ties
    prior = (rng.random(n) < 0.07).astype(np.float32)
    n_forced = int(prior.sum())
    for budget in sorted({0, 1, n // 16, max(0, n_forced - 1), n_forced, n_forced + 3, n - 1, n, n + 5}):
        if budget < 0:
            continue
        idx, count = run_select(fused, prior, n, budget, 0.5)
        keep = min(budget, n)
        for h in range(hkv):
            ref = orc.select_tokens(fused[h], prior, n, budget, 0.5)
            assert count[h] == keep
            np.testing.assert_array_equal(idx[h, :keep], ref, err_msg=f"n={n} B={budget} h={h}")
            assert (idx[h, keep:] == -1).all()


@pytest.mark.parametrize("seed", range(6))
def test_select_with_span_cap_and_graded_prior(seed):
    rng = np.random.Generator(np.random.PCG64(500 + seed))
    n = int(rng.integers(200, 5000))
    hkv = 2
    fused = rng.choice(rng.random(50).astype(np.float32), size=(hkv, n)).astype(np.float32)
    prior = rng.choice(np.array([0, 0, 0, 0, 0.2, 0.6, 0.6, 0.8, 0.95], np.float32), size=n)
    for budget in [n // 10, n // 3]:
        for ratio, smin in [(0.5, 16), (0.25, 0), (1.0, 0)]:
            idx, count = run_select(fused, prior, n, budget, 0.5, ratio, smin)
            for h in range(hkv):
                ref = orc.select_tokens(fused[h], prior, n, budget, 0.5, ratio, smin)
                np.testing.assert_array_equal(idx[h, :len(ref)], ref)


@pytest.mark.parametrize("n,chunk,budget", [(32768, 10, 2048), (1003, 10, 100), (95, 10, 95),
                                            (4099, 7, 500), (64, 10, 7)])
def test_select_chunk_level(n, chunk, budget):
    rng = np.random.Generator(np.random.PCG64(n + budget))
    hkv = 2
    u = np.abs(rng.standard_normal((hkv, n))).astype(np.float32)
    prior = (rng.random(n) < 0.02).astype(np.float32)
    cu, cp = orc.chunk_reduce(u, prior, chunk, dtype=np.float32)
    idx, count = run_select(cu, prior, n, budget, 0.5, chunk=chunk)
    for h in range(hkv):
        ref = orc.select_tokens(cu[h], cp, n, budget, 0.5, chunk=chunk)
        np.testing.assert_array_equal(idx[h, :len(ref)], ref)
        assert count[h] == len(ref) == min(budget, n)


def test_select_negative_and_zero_scores():
    n = 300
    rng = np.random.Generator(np.random.PCG64(3))
    fused = rng.standard_normal((1, n)).astype(np.float32)
    fused[0, ::5] = 0.0
    fused[0, 1::7] = -0.0
    prior = np.zeros(n, np.float32)
    for budget in [10, 150, 290]:
        idx, _ = run_select(fused, prior, n, budget, 0.5)
        np.testing.assert_array_equal(idx[0], orc.select_tokens(fused[0], prior, n, budget, 0.5))


# ------------------------------------------------------------------ A5
# the last five cases reach the forms of the kernel that move a run of heads per thread group:
# 2, 4 and all 8 heads of a slot (the batch fills the GPU with fewer units), and head counts that
# are not powers of two (one unit per slot, the last trip of a unit shorter than the others)
@pytest.mark.parametrize("n,budget,hkv", [(1, 1, 1), (129, 40, 2), (4099, 4099, 8), (2048, 512, 2),
                                          (6000, 5000, 8), (12000, 10000, 8), (20000, 19000, 8),
                                          (700, 650, 6), (700, 300, 3)])
def test_compact_contiguous(n, budget, hkv):
    rng = np.random.Generator(np.random.PCG64(n + budget))
    k = rng.integers(0, 65535, size=(n, hkv, 128), dtype=np.uint16)
    v = rng.integers(0, 65535, size=(n, hkv, 128), dtype=np.uint16)
    idx = np.stack([np.sort(rng.choice(n, size=budget, replace=False)) for _ in range(hkv)]).astype(np.int32)
    d = cc.Desc(hkv, hkv, 4, n=n, budget=budget)
    ko, kfull = guarded((budget, hkv, 128), torch.int16, 0x1111)
    vo, vfull = guarded((budget, hkv, 128), torch.int16, 0x1111)
    cc.cc_compact_kv(ctx(), d, bf16_dev(k), bf16_dev(v), torch.from_numpy(idx).cuda(),
                     ko.view(torch.bfloat16), vo.view(torch.bfloat16))
    assert ctx().poll() == 0
    rk, rv = orc.compact_kv(k, v, idx)
    got_k, got_v = bits_host(ko), bits_host(vo)
    for h in range(hkv):
        np.testing.assert_array_equal(got_k[:, h], rk[h])
        np.testing.assert_array_equal(got_v[:, h], rv[h])
    assert guards_intact(kfull, 0x1111) and guards_intact(vfull, 0x1111)


def test_compact_rejects_in_place_and_bad_index():
    n, hkv = 64, 2
    k = bf16_dev(np.zeros((n, hkv, 128), np.uint16))
    d = cc.Desc(hkv, hkv, 4, n=n, budget=8)
    idx = torch.zeros((hkv, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(cc.CodecompError) as e:
        cc.cc_compact_kv(ctx(), d, k, k, idx, k, k)
    assert e.value.status == cc.CC_ERR_INVALID_ARG
    idx[1, 3] = n + 7                                   # out of range: flagged and skipped
    out = torch.zeros((8, hkv, 128), dtype=torch.bfloat16, device="cuda")
    cc.cc_compact_kv(ctx(), d, k, k, idx, out, out.clone())
    assert ctx().poll() == cc.CC_ERR_DEVICE_FLAG
    assert ctx().poll() == 0                            # the status word is cleared by the poll


@pytest.mark.parametrize("wl", [
    gen.Workload("p", 11, 1, 4, 2, 128, 8, gen.POOL_MAX, 3, 0, seq_lens=(100, 37, 260),
                 budget_frac=0.25, page_size=16),
    # enough slots that a thread group moves four heads of a slot, two groups per slot
    gen.Workload("p4", 12, 1, 8, 8, 128, 8, gen.POOL_MAX, 3, 0, seq_lens=(9000, 700, 5000, 6300),
                 budget_frac=0.5, page_size=16),
], ids=lambda w: w.name)
def test_compact_paged(wl):
    x = gen.make_layer(wl)
    rng = np.random.Generator(np.random.PCG64(5))
    buds = wl.budgets
    b_tot = sum(buds)
    idx = np.full((wl.n_heads_kv, b_tot), -1, np.int32)
    off = 0
    for s, (n, b) in enumerate(zip(wl.lens, buds)):
        for h in range(wl.n_heads_kv):
            idx[h, off:off + b] = np.sort(rng.choice(n, size=b, replace=False))
        off += b
    pt = torch.from_numpy(x.page_table).cuda()
    stride = max((b + 15) // 16 for b in buds) + 2
    d = desc_for(wl, cc.CC_MODE_FP32, page_table=pt, out_pt_stride=stride, pool_pages=x.pool_pages)
    k_pool, v_pool = bf16_dev(x.k), bf16_dev(x.v)
    before_k = bits_host(k_pool).copy()
    out_pt = torch.full((len(buds), stride), -7, dtype=torch.int32, device="cuda")
    cc.cc_compact_kv(ctx(), d, k_pool, v_pool, torch.from_numpy(idx).cuda(), k_pool, v_pool,
                     torch.from_numpy(x.free_pages).cuda(), out_pt)
    assert ctx().poll() == 0
    pages = orc.assign_output_pages(buds, wl.lens, 16, x.free_pages)
    got_pt = out_pt.cpu().numpy()
    after_k, after_v = bits_host(k_pool), bits_host(v_pool)
    off = 0
    touched = np.zeros(x.pool_pages, bool)
    for s, (n, b) in enumerate(zip(wl.lens, buds)):
        assert got_pt[s, :len(pages[s])].tolist() == pages[s].tolist()
        assert (got_pt[s, len(pages[s]):] == -1).all()
        src = orc.paged_rows(x.page_table[s], n, 16)
        dst = orc.paged_rows(pages[s], b, 16)
        touched[pages[s]] = True
        for h in range(wl.n_heads_kv):
            tok = idx[h, off:off + b]
            np.testing.assert_array_equal(after_k[dst, h], x.k[src[tok], h])
            np.testing.assert_array_equal(after_v[dst, h], x.v[src[tok], h])
        off += b
    untouched_rows = np.repeat(~touched, 16)
    np.testing.assert_array_equal(after_k[untouched_rows], before_k[untouched_rows])


def test_page_ids_outside_the_pool_are_skipped_and_flagged():
    """A page id equal to pool_pages (one past the pool) in the page table or in the list of fresh
    pages: the kernels skip the access and record CC_ERR_DEVICE_FLAG.  The pool tensors carry
    guard pages behind the pool, which must stay untouched."""
    wl = gen.Workload("p", 12, 1, 4, 2, 128, 8, gen.POOL_MAX, 3, 0, seq_lens=(100, 37),
                      budget_frac=0.25, page_size=16)
    x = gen.make_layer(wl)
    buds = wl.budgets
    b_tot = sum(buds)
    idx = np.full((wl.n_heads_kv, b_tot), -1, np.int32)
    off = 0
    for n, b in zip(wl.lens, buds):
        idx[:, off:off + b] = np.arange(b)[None, :]
        off += b
    guard_pages = 4
    hkv = wl.n_heads_kv

    def padded(bits):
        pad = np.full((guard_pages * 16, hkv, 128), 0x7FC0, np.uint16)
        return bf16_dev(np.concatenate([bits, pad]))

    stride = max((b + 15) // 16 for b in buds) + 2
    for where in ("page_table", "free_pages"):
        table = x.page_table.copy()
        free = x.free_pages.copy()
        if where == "page_table":
            table[0, 0] = x.pool_pages              # tokens 0..15 of sequence 0 point past the pool
        else:
            free[0] = x.pool_pages
        pt = torch.from_numpy(table).cuda()
        d = desc_for(wl, cc.CC_MODE_FP32, page_table=pt, out_pt_stride=stride, pool_pages=x.pool_pages)
        k_pool, v_pool = padded(x.k), padded(x.v)
        out_pt = torch.full((len(buds), stride), -7, dtype=torch.int32, device="cuda")
        cc.cc_compact_kv(ctx(), d, k_pool, v_pool, torch.from_numpy(idx).cuda(), k_pool, v_pool,
                         torch.from_numpy(free).cuda(), out_pt)
        assert ctx().poll() == cc.CC_ERR_DEVICE_FLAG
        assert (bits_host(k_pool)[x.pool_pages * 16:] == 0x7FC0).all()
        assert (bits_host(v_pool)[x.pool_pages * 16:] == 0x7FC0).all()
        if where == "free_pages":
            assert out_pt.cpu().numpy()[0, 0] == -1       # the bad page is not published
    # the fp32 score kernel reads K through the same table
    table = x.page_table.copy()
    table[1, 1] = x.pool_pages
    pt = torch.from_numpy(table).cuda()
    d = desc_for(wl, cc.CC_MODE_FP32, page_table=pt, out_pt_stride=stride, pool_pages=x.pool_pages)
    scores = torch.zeros((hkv, sum(wl.lens)), device="cuda")
    cc.cc_score_window(ctx(), d, bf16_dev(x.q_win), padded(x.k), scores)
    assert ctx().poll() == cc.CC_ERR_DEVICE_FLAG
    d = desc_for(wl, cc.CC_MODE_BF16, page_table=pt, out_pt_stride=stride, pool_pages=x.pool_pages)
    cc.cc_score_window(ctx(), d, bf16_dev(x.q_win), padded(x.k), scores)
    assert ctx().poll() == cc.CC_ERR_DEVICE_FLAG


# ------------------------------------------------------------------ argument checks
def test_descriptor_validation():
    c = ctx()
    ok = cc.Desc(8, 2, 32, n=128, budget=16)
    assert c.workspace_bytes(ok) >= 256
    for bad, status in [
        (cc.Desc(8, 3, 32, n=128, budget=16), cc.CC_ERR_INVALID_ARG),
        (cc.Desc(8, 2, 32, n=128, budget=16, head_dim=64), cc.CC_ERR_UNSUPPORTED),
        (cc.Desc(8, 2, 32, n=128, budget=16, pool_size=4), cc.CC_ERR_UNSUPPORTED),
        (cc.Desc(64, 1, 32, n=128, budget=16), cc.CC_ERR_UNSUPPORTED),          # w * G = 2048 rows
        (cc.Desc(8, 2, 32, n=-1, budget=16), cc.CC_ERR_INVALID_ARG),
        (cc.Desc(8, 2, 32, n=128, budget=16, page_size=12), cc.CC_ERR_UNSUPPORTED),
    ]:
        scores = torch.zeros(2, 128, device="cuda")
        with pytest.raises(cc.CodecompError) as e:
            cc.cc_fuse_prior_pool(c, bad, scores, scores[0], scores.clone())
        assert e.value.status == status
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    big = cc.Desc(8, 2, 32, n=4096, budget=16)
    with pytest.raises(cc.CodecompError) as e:
        cc.cc_topk_select(c, big, torch.zeros(2, 4096, device="cuda"), torch.zeros(4096, device="cuda"),
                          torch.zeros(2, 16, dtype=torch.int32, device="cuda"),
                          torch.zeros(2, dtype=torch.int32, device="cuda"), ws=small)
    assert e.value.status == cc.CC_ERR_WORKSPACE


# ------------------------------------------------------------------ Str. Score
@pytest.mark.parametrize("lens,budgets", [((1,), (1,)), ((700,), (64,)), ((4099,), (4099,)),
                                          ((300, 1, 129, 2050, 64), (30, 1, 12, 205, 6)),
                                          ((65536,), (2048,))])
@pytest.mark.parametrize("density,threshold", [(0.07, 0.5), (0.0, 0.5), (1.0, 0.5), (0.3, math.inf)])
def test_structural_score_matches_oracle(lens, budgets, density, threshold):
    """Counts bit for bit, fraction as the correctly rounded f32 quotient of the counts."""
    rng = np.random.Generator(np.random.PCG64(sum(lens) + int(density * 100)))
    hkv, n_tot, b_tot = 3, sum(lens), sum(min(b, n) for b, n in zip(budgets, lens))
    prior = (rng.random(n_tot) < density).astype(np.float32) * np.float32(0.75)
    if density > 0:
        prior[rng.integers(n_tot)] = 0.5                  # a token exactly at the threshold
    idx = np.full((hkv, b_tot), -1, dtype=np.int32)
    off = 0
    for n, b in zip(lens, budgets):
        keep = min(b, n)
        for h in range(hkv):
            idx[h, off:off + keep] = np.sort(rng.choice(n, size=keep, replace=False))
        off += keep
    idx[1, b_tot - 1] = -1                                # padding entries are skipped
    if len(lens) > 1:
        d = cc.Desc(hkv, hkv, 4, seq_lens=lens, budgets=budgets)
    else:
        d = cc.Desc(hkv, hkv, 4, n=lens[0], budget=budgets[0])
    score, full_s = guarded((len(lens), hkv), torch.float32, -3.0)
    counts, full_c = guarded((len(lens), hkv, 2), torch.int32, -3)
    cc.cc_structural_score(ctx(), d, torch.from_numpy(idx).cuda(), f32_dev(prior), threshold,
                           score, counts)
    assert ctx().poll() == 0
    got_s, got_c = score.cpu().numpy(), counts.cpu().numpy()
    tok = off = 0
    for s, (n, b) in enumerate(zip(lens, budgets)):
        keep = min(b, n)
        for h in range(hkv):
            frac, hit, tot = orc.structural_score(idx[h, off:off + keep], prior[tok:tok + n], threshold)
            assert (got_c[s, h, 0], got_c[s, h, 1]) == (hit, tot)
            assert got_s[s, h] == np.float32(frac)
        tok += n
        off += keep
    assert guards_intact(full_s, -3.0) and guards_intact(full_c, -3)


def test_structural_score_of_the_fused_path_on_tiny():
    """The retained sets of cc_compress_layer keep every protected token when they fit the budget."""
    wl = gen.workloads()["tiny"]
    x = gen.make_layer(wl)
    d = desc_for(wl, cc.CC_MODE_BF16)
    hkv, b = wl.n_heads_kv, wl.budget
    idx = torch.empty((hkv, b), dtype=torch.int32, device="cuda")
    count = torch.empty((1, hkv), dtype=torch.int32, device="cuda")
    k_out = torch.empty((b, hkv, 128), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    prior = f32_dev(x.prior)
    cc.cc_compress_layer(ctx(), d, bf16_dev(x.q_win), bf16_dev(x.k), bf16_dev(x.v), prior, k_out,
                         v_out, idx, count)
    score = torch.empty((1, hkv), dtype=torch.float32, device="cuda")
    cc.cc_structural_score(ctx(), d, idx, prior, wl.force_threshold, score)
    assert ctx().poll() == 0
    assert (score.cpu().numpy() == 1.0).all()
    res = orc.compress_sequence(x.q_win[0], x.k, None, x.prior, hkv, wl.pool_kind, wl.pool_size,
                                wl.budget, wl.alpha, wl.beta, wl.force_threshold)
    for h in range(hkv):
        assert orc.structural_score(res["idx"][h], x.prior, wl.force_threshold)[0] == 1.0


def test_exp_rate_probe_reports_a_plausible_rate():
    """Between the special-function unit alone (16 per clock per SM, minus the share that the
    polynomial takes over) and what both pipes could do if nothing else limited them."""
    reg = cc.cc_exp_rate_probe(ctx(), False, 2000)
    tm = cc.cc_exp_rate_probe(ctx(), True, 2000)
    assert 12.0 < reg < 40.0, reg
    assert 8.0 < tm < 40.0, tm
    assert ctx().poll() == 0


@pytest.mark.parametrize("n", [1, 31, 1024, 1025, 5000, 70001])
@pytest.mark.parametrize("density", [0.0, 0.002, 0.07, 1.0])
def test_nearest_fill_values_bit_exact(n, density):
    """cc_fuse_prior_pool with CC_FILL_NEAREST against the oracle's two-sweep distances."""
    rng = np.random.Generator(np.random.PCG64(n + int(1000 * density)))
    prior = (rng.random(n) < density).astype(np.float32)
    hkv = 3
    d = cc.Desc(hkv, hkv, 4, n=n, budget=max(1, n // 10), pool_kind=cc.CC_POOL_NONE, pool_size=1,
                force_threshold=0.5, fill_mode=cc.CC_FILL_NEAREST)
    fused_c, full = guarded((hkv, n), torch.float32, -77.0)
    cc.cc_fuse_prior_pool(ctx(), d, None, f32_dev(prior), fused_c)
    assert ctx().poll() == 0
    assert guards_intact(full, -77.0)
    ref = orc.nearest_fill_values(prior, 0.5).astype(np.float32)
    for h in range(hkv):
        np.testing.assert_array_equal(fused_c[h].cpu().numpy(), ref)
