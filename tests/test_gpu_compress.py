"""A8 parity: the fused per-layer call against the oracle's whole path.

Scores are floating point, so the retained index sets may differ only for items whose
oracle value lies within the score tolerance of the oracle's cut-off; everything else -
count, order, protected tokens, gathered K/V bits - must agree exactly."""
import numpy as np
import pytest
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen

from gpu_util import (assert_scores_close, bf16_dev, bits_host, check_selection, ctx, desc_for,
                      score_tolerance, seq_kv)

pytestmark = pytest.mark.gpu
MODES = [(cc.CC_MODE_FP32, 1e-5), (cc.CC_MODE_BF16, 2e-3)]


def run_layer(wl, x, mode):
    paged = wl.page_size > 0
    pt = torch.from_numpy(x.page_table).cuda() if paged else None
    buds, lens = wl.budgets, wl.lens
    b_tot = sum(buds)
    stride = max((min(b, n) + wl.page_size - 1) // wl.page_size for b, n in zip(buds, lens)) + 1 if paged else 0
    d = desc_for(wl, mode, page_table=pt, out_pt_stride=stride, pool_pages=x.pool_pages)
    k, v = bf16_dev(x.k), bf16_dev(x.v)
    idx = torch.full((wl.n_heads_kv, b_tot), -9, dtype=torch.int32, device="cuda")
    count = torch.full((len(lens), wl.n_heads_kv), -9, dtype=torch.int32, device="cuda")
    ws = ctx().workspace(d)
    if paged:
        k_out, v_out = k, v
        out_pt = torch.full((len(lens), stride), -9, dtype=torch.int32, device="cuda")
        free = torch.from_numpy(x.free_pages).cuda()
    else:
        k_out = torch.zeros((b_tot, wl.n_heads_kv, 128), dtype=torch.bfloat16, device="cuda")
        v_out = torch.zeros_like(k_out)
        out_pt = free = None
    cc.cc_compress_layer(ctx(), d, bf16_dev(x.q_win), k, v, f32_dev_prior(x), k_out, v_out, idx,
                         count, free, out_pt, ws)
    assert ctx().poll() == 0, ctx().lib.cc_last_error(ctx().handle)
    scores, fused = cc.cc_workspace_views(ctx(), d, ws)
    return dict(idx=idx.cpu().numpy(), count=count.cpu().numpy(), k_out=bits_host(k_out),
                v_out=bits_host(v_out), scores=scores.cpu().numpy(), fused=fused.cpu().numpy(),
                out_pt=None if out_pt is None else out_pt.cpu().numpy())


def f32_dev_prior(x):
    return torch.from_numpy(x.prior).cuda()


def check_layer(wl, x, mode, tol):
    got = run_layer(wl, x, mode)
    rows = wl.window * wl.group
    chunk = max(1, wl.chunk_size)
    pages = orc.assign_output_pages(wl.budgets, wl.lens, wl.page_size, x.free_pages) if wl.page_size else None
    off_b = off_i = 0
    for s, (n, b) in enumerate(zip(wl.lens, wl.budgets)):
        keep = min(n, b)
        if n == 0:                               # an empty sequence keeps nothing
            assert (got["count"][s] == 0).all() and (got["idx"][:, off_b:off_b + b] == -1).all()
            off_b += b
            continue
        k_s, v_s = seq_kv(x, s)
        lo = int(x.tok_offsets[s])
        prior = x.prior[lo:lo + n]
        ref = orc.compress_sequence(x.q_win[s], k_s, v_s, prior, wl.n_heads_kv, wl.pool_kind,
                                    wl.pool_size, b, wl.alpha, wl.beta, wl.force_threshold,
                                    wl.span_ratio, wl.span_min, chunk, causal=wl.causal,
                                    nearest_fill=bool(wl.fill_mode))
        if not wl.fill_mode:                  # (the nearest-token fill does not compute scores)
            assert_scores_close(got["scores"][:, lo:lo + n], ref["scores"], rows, n, tol)
        m = len(ref["item_prior"])
        # the protected set (capped to the span budget when a span ratio is set) depends on the
        # prior alone, so it is taken from the oracle; what the scores decide is checked below
        forced_items = orc.protected_items(ref["item_prior"], orc.chunk_lengths(n, chunk), b,
                                           wl.force_threshold, wl.span_ratio, wl.span_min)
        # how far a fused value may move when every score in its pooling window (or chunk)
        # moves by its tolerance: alpha * (sum or max of the per-score bounds)
        tol_u = score_tolerance(ref["scores"], rows, n, tol)
        if chunk > 1:
            band_u, _ = orc.chunk_reduce(tol_u, prior, chunk)
        elif wl.pool_kind == orc.POOL_AVG:
            band_u = orc.pool_scores(tol_u, orc.POOL_AVG, wl.pool_size)
        else:
            band_u = orc.pool_scores(tol_u, wl.pool_kind, wl.pool_size)
        # ... plus the rounding of the kernels' fp32 fusion (two products and a sum, half an ulp
        # each) against the fp64 reference: it decides the order when beta * p dominates
        band = abs(wl.alpha) * band_u * 2 + 1e-12 + 3 * 2.0 ** -24 * np.abs(ref["fused"])
        if wl.fill_mode:
            band = np.zeros_like(ref["fused"])          # distances are integers: nothing to forgive
            np.testing.assert_array_equal(got["fused"][:, off_i:off_i + m], ref["fused"])
        for h in range(wl.n_heads_kv):
            assert got["count"][s, h] == keep
            idx = got["idx"][h, off_b:off_b + keep]
            assert (got["idx"][h, off_b + keep:off_b + b] == -1).all()
            check_selection(idx, ref["fused"][h], forced_items, keep, band[h], n, chunk)
            # gathered rows are bit copies of the rows the GPU selected
            if wl.page_size:
                dst = orc.paged_rows(pages[s], keep, wl.page_size)
                np.testing.assert_array_equal(got["k_out"][dst, h], k_s[idx, h])
                np.testing.assert_array_equal(got["v_out"][dst, h], v_s[idx, h])
            else:
                np.testing.assert_array_equal(got["k_out"][off_b:off_b + keep, h], k_s[idx, h])
                np.testing.assert_array_equal(got["v_out"][off_b:off_b + keep, h], v_s[idx, h])
        if wl.page_size:
            assert got["out_pt"][s, :len(pages[s])].tolist() == pages[s].tolist()
        off_b += b
        off_i += m


@pytest.mark.parametrize("mode,tol", MODES)
def test_tiny_config(mode, tol):
    wl = gen.workloads()["tiny"]
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("n,budget", [(1, 1), (17, 0), (129, 129), (129, 200), (4099, 300)])
def test_edge_sizes(mode, tol, n, budget):
    wl = gen.Workload("edge", 30, 1, 8, 2, 128, 32, gen.POOL_MAX, 7, budget, n=n)
    check_layer(wl, gen.make_layer(wl, layer=n), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_paper_setting_avg_pool(mode, tol):
    from dataclasses import replace
    wl = replace(gen.workloads()["paper_avg5_w128"], span_ratio=0.0, n_heads_q=8, n_heads_kv=2)
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_weighted_prior_mode(mode, tol):
    from dataclasses import replace
    wl = replace(gen.workloads()["tiny"], alpha=0.06 / (32 * 4), beta=1.0, force_threshold=float("inf"))
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_causal_window_fused_path(mode, tol):
    wl = gen.Workload("causal", 33, 1, 8, 2, 128, 32, gen.POOL_MAX, 7, 200, n=1500, causal=True)
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_chunk_level(mode, tol):
    wl = gen.Workload("chunk", 31, 1, 8, 2, 128, 32, gen.POOL_NONE, 1, 256, n=3003, chunk_size=10)
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_ragged_paged(mode, tol):
    wl = gen.Workload("rp", 32, 1, 8, 2, 128, 16, gen.POOL_MAX, 7, 0,
                      seq_lens=(300, 40, 2050, 129), budget_frac=0.1, page_size=16)
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("ratio,smin", [(0.5, 16), (0.25, 0), (0.3, 64)])
def test_span_cap_through_the_fused_call(mode, tol, ratio, smin):
    """Protected tokens limited to B_span = min(B, max(B_min, floor(rho * B))) (Section 4.4, "Span
    selection under budget"): more protected tokens than the cap, the attention scores fill the rest."""
    from dataclasses import replace
    wl = replace(gen.workloads()["tiny"], span_ratio=ratio, span_min=smin, budget=200)
    check_layer(wl, gen.make_layer(wl, layer=7), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_span_cap_ragged_paged_and_chunked(mode, tol):
    wl = gen.Workload("rpcap", 34, 1, 8, 2, 128, 16, gen.POOL_AVG, 5, 0,
                      seq_lens=(700, 40, 2050, 129), budget_frac=0.3, page_size=16,
                      span_ratio=0.5, span_min=16)
    check_layer(wl, gen.make_layer(wl), mode, tol)
    wl = gen.Workload("chcap", 35, 1, 8, 2, 128, 32, gen.POOL_NONE, 1, 300, n=3003, chunk_size=10,
                      span_ratio=0.5, span_min=16)
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("n,pool,k", [(140000, gen.POOL_MAX, 7), (140000, gen.POOL_AVG, 5),
                                      (270000, gen.POOL_MAX, 7)])
def test_more_items_than_a_cluster_stages_or_holds(n, pool, k):
    """140000 items: more than 16 per thread of the widest cluster, so the cluster kernel pools
    straight from global memory instead of staging the raw scores.  270000 items: more than a
    cluster holds (262144), so the fused call and cc_topk_select take the single-CTA selection
    kernel and the stand-alone pooling kernel instead."""
    wl = gen.Workload("long", 36, 1, 2, 1, 128, 8, pool, k, 9000, n=n)
    x = gen.make_layer(wl)
    check_layer(wl, x, cc.CC_MODE_BF16, 2e-3)
    # selection stage alone on the oracle's fp32 stage values: bit for bit
    from test_gpu_stages import run_select
    rng = np.random.Generator(np.random.PCG64(9))
    u = (np.abs(rng.standard_normal((1, wl.n))) * 1e-3).astype(np.float32)
    fused = orc.pool_scores(u, pool, k, dtype=np.float32)
    idx, count = run_select(fused, x.prior, wl.n, wl.budget, wl.force_threshold, 0.5, 16)
    ref = orc.select_tokens(fused[0], x.prior, wl.n, wl.budget, wl.force_threshold, 0.5, 16)
    assert count[0] == len(ref) == wl.budget
    np.testing.assert_array_equal(idx[0, :len(ref)], ref)


@pytest.mark.parametrize("mode,tol", MODES)
def test_nearest_token_fill_through_the_fused_call(mode, tol):
    """Section 4.4, last sentence of "Token-level protection": the budget left by the protected
    tokens goes to the tokens nearest to them; bit for bit (the ranking values are integers)."""
    from dataclasses import replace
    wl = replace(gen.workloads()["tiny"], fill_mode=cc.CC_FILL_NEAREST)
    check_layer(wl, gen.make_layer(wl, layer=11), mode, tol)
    wl = gen.Workload("rpnear", 37, 1, 8, 2, 128, 16, gen.POOL_AVG, 5, 0,
                      seq_lens=(700, 40, 2050, 129, 5000), budget_frac=0.3, page_size=16,
                      span_ratio=0.5, span_min=16, fill_mode=cc.CC_FILL_NEAREST)
    check_layer(wl, gen.make_layer(wl), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_nearest_fill_edge_batches(mode, tol):
    """Empty and one-token sequences, a budget above the length, and a sequence without any
    protected token, in one ragged batch with the nearest-token fill."""
    wl = gen.Workload("nearedge", 38, 1, 8, 2, 128, 8, gen.POOL_MAX, 3, 0,
                      seq_lens=(0, 1, 33, 500), seq_budgets=(4, 1, 40, 77),
                      fill_mode=cc.CC_FILL_NEAREST)
    x = gen.make_layer(wl)
    x.prior[1:34] = 0.0                       # sequences 1 and 2 have no protected token
    check_layer(wl, x, mode, tol)


def test_all_layers_call_with_no_layers_is_a_no_op():
    wl = gen.workloads()["tiny"]
    d = desc_for(wl, cc.CC_MODE_BF16)
    cc.cc_compress_layers(ctx(), d, [], [], [], torch.zeros(wl.n, device="cuda"), [], [], [], [],
                          ws=ctx().workspace(d))
    assert ctx().poll() == 0
