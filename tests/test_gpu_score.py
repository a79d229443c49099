"""A1 parity: window attention scores of the CUDA path against the fp64 oracle.
Tolerances: |u - u_ref| <= tol * |u_ref| + tol * (w G / n) with tol = 2e-3 for the bf16
tensor-core mode and 1e-5 for the fp32 verification mode."""
import numpy as np
import pytest
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen

from gpu_util import assert_scores_close, bf16_dev, ctx, desc_for, seq_kv

pytestmark = pytest.mark.gpu
MODES = [(cc.CC_MODE_FP32, 1e-5), (cc.CC_MODE_BF16, 2e-3)]


def run_scores(wl, x, mode, want_lse=True):
    pt = torch.from_numpy(x.page_table).cuda() if wl.page_size else None
    d = desc_for(wl, mode, page_table=pt, pool_pages=x.pool_pages)
    n_tot = sum(wl.lens)
    scores = torch.full((wl.n_heads_kv, n_tot), -1.0, device="cuda")
    lse = torch.full((len(wl.lens), wl.n_heads_q, wl.window), -1.0, device="cuda") if want_lse else None
    cc.cc_score_window(ctx(), d, bf16_dev(x.q_win), bf16_dev(x.k), scores, lse)
    assert ctx().poll() == 0, ctx().lib.cc_last_error(ctx().handle)
    return scores.cpu().numpy(), (lse.cpu().numpy() if want_lse else None)


def check_against_oracle(wl, x, mode, tol):
    u, lse = run_scores(wl, x, mode)
    rows = wl.window * wl.group
    for s, n in enumerate(wl.lens):
        k_s, _ = seq_kv(x, s)
        ref, lse_ref = orc.window_scores(orc.bf16_bits_to_f64(x.q_win[s]), orc.bf16_bits_to_f64(k_s),
                                         wl.n_heads_kv, causal=wl.causal)
        lo = int(x.tok_offsets[s])
        assert_scores_close(u[:, lo:lo + n], ref, rows, n, tol)
        np.testing.assert_allclose(lse[s], lse_ref, atol=20 * tol, rtol=0)
        np.testing.assert_allclose(u[:, lo:lo + n].sum(1), rows, rtol=20 * tol)   # rows of A sum to 1


@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("n", [1, 15, 16, 17, 127, 128, 129, 2048, 4099])
def test_scores_length_sweep(mode, tol, n):
    wl = gen.Workload("sweep", 20, 1, 8, 2, 128, 32, gen.POOL_MAX, 7, 1, n=n)
    check_against_oracle(wl, gen.make_layer(wl, layer=n, with_v=False), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("w,hq,hkv", [(1, 1, 1), (1, 7, 1), (32, 8, 2), (64, 4, 1), (128, 4, 1),
                                      (64, 28, 4), (64, 32, 8), (3, 6, 2), (128, 8, 2)])
def test_scores_shape_sweep(mode, tol, w, hq, hkv):
    wl = gen.Workload("shape", 21, 1, hq, hkv, 128, w, gen.POOL_MAX, 7, 1, n=1000,
                      outlier_frac=0.01)
    check_against_oracle(wl, gen.make_layer(wl, layer=w + hq, with_v=False), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_scores_tiny_config(mode, tol):
    wl = gen.workloads()["tiny"]
    check_against_oracle(wl, gen.make_layer(wl, with_v=False), mode, tol)


@pytest.mark.parametrize("w,hq,hkv,page", [(96, 8, 2, 0), (48, 14, 2, 16)])
def test_scores_three_stage_ring(w, hq, hkv, page):
    """Row counts of 384 and 336: the shared-memory ring of the tensor-core kernel has three K
    stages then (four below 313 rows, two above 440), and 40000 keys give every CTA more tiles than
    the ring has stages, so it wraps."""
    wl = gen.Workload("ring3", 26, 1, hq, hkv, 128, w, gen.POOL_MAX, 7, 1,
                      seq_lens=(40000,), budget_frac=0.1, page_size=page)
    check_against_oracle(wl, gen.make_layer(wl, with_v=False), cc.CC_MODE_BF16, 2e-3)


@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("page", [0, 8, 16, 32, 64, 128])      # every supported page size
def test_scores_ragged_batch(mode, tol, page):
    wl = gen.Workload("ragged", 22, 1, 8, 2, 128, 16, gen.POOL_MAX, 7, 0,
                      seq_lens=(300, 1, 129, 2050, 64), budget_frac=0.1, page_size=page)
    check_against_oracle(wl, gen.make_layer(wl, with_v=False), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
def test_scores_peaked_and_uniform_rows(mode, tol):
    """Degenerate softmax rows: identical keys (uniform) and one dominant key (all mass)."""
    wl = gen.Workload("deg", 23, 1, 4, 2, 128, 8, gen.POOL_MAX, 7, 1, n=700)
    x = gen.make_layer(wl, with_v=False)
    x.k[:, 1, :] = x.k[0, 1, :]                       # KV head 1: identical keys
    x.k[123, 0, :] = gen.f32_to_bf16_bits(np.full(128, 6.0, np.float32))
    x.q_win[:, :, :2, :] = gen.f32_to_bf16_bits(np.full((1, 8, 2, 128), 2.0, np.float32))
    check_against_oracle(wl, x, mode, tol)
    u, _ = run_scores(wl, x, mode, want_lse=False)
    np.testing.assert_allclose(u[1], 8 * 2 / 700, rtol=max(tol, 1e-5))
    assert abs(u[0, 123] - 16.0) < 16 * 10 * tol


@pytest.mark.parametrize("mode,tol", MODES)
def test_scores_large_logits_do_not_overflow(mode, tol):
    wl = gen.Workload("big", 24, 1, 2, 1, 128, 8, gen.POOL_MAX, 7, 1, n=500)
    x = gen.make_layer(wl, with_v=False)
    q = orc.bf16_bits_to_f64(x.q_win).astype(np.float32) * 12.0       # logits of order +-150
    x.q_win = gen.f32_to_bf16_bits(q)
    check_against_oracle(wl, x, mode, tol)


# ------------------------------------------------------------------ causal in-sequence window
@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("n,w,hq,hkv", [(32, 32, 8, 2), (33, 32, 8, 2), (127, 16, 4, 1), (128, 64, 4, 1),
                                        (129, 64, 32, 8), (300, 128, 4, 1), (1000, 64, 28, 4),
                                        (4099, 32, 8, 2), (200, 3, 6, 2), (512, 128, 8, 2)])
def test_scores_causal_window(mode, tol, n, w, hq, hkv):
    """The window is the last w tokens of the sequence: row t attends to keys <= n - w + t."""
    wl = gen.Workload("causal", 24, 1, hq, hkv, 128, w, gen.POOL_MAX, 7, 1, n=n, causal=True)
    check_against_oracle(wl, gen.make_layer(wl, layer=n + w, with_v=False), mode, tol)


@pytest.mark.parametrize("mode,tol", MODES)
@pytest.mark.parametrize("page", [0, 16])
def test_scores_causal_ragged_batch(mode, tol, page):
    wl = gen.Workload("causal_ragged", 25, 1, 8, 2, 128, 16, gen.POOL_MAX, 7, 0,
                      seq_lens=(300, 16, 129, 2050, 64), budget_frac=0.1, page_size=page, causal=True)
    check_against_oracle(wl, gen.make_layer(wl, with_v=False), mode, tol)


def test_causal_window_shorter_than_the_window_is_rejected():
    d = cc.Desc(8, 2, 32, n=20, budget=4, causal=True)
    scores = torch.empty((2, 20), device="cuda")
    q = torch.empty((1, 32, 8, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.empty((20, 2, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cc.CodecompError):
        cc.cc_score_window(ctx(), d, q, k, scores, None)
