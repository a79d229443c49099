"""Chunk selection by query-conditioned perplexity (Section 4.1): CUDA path against the oracle.
Tolerance of the negative log-likelihoods: 5e-5 absolute (fp32 sums of up to 2^17 exponentials,
approximate exp2 with relative error <= 8e-5 on one element in eight and 2^-22 on the others,
whose errors largely cancel in the sum; values are of order 10).  The chosen chunks are integers:
the selection is compared bit for bit on the same fp32 scores."""
import numpy as np
import pytest
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc

from gpu_util import ctx

pytestmark = pytest.mark.gpu
TOL = 5e-5


def make_logits(seed, chunks, t, v, dtype):
    rng = np.random.Generator(np.random.PCG64(seed))
    x = (rng.standard_normal((chunks, t, v)) * 3.0).astype(np.float32)
    tgt = rng.integers(0, v, size=t).astype(np.int32)
    boost = rng.random((chunks, t)).astype(np.float32) * 12.0          # how well each chunk explains q_t
    x[np.arange(chunks)[:, None], np.arange(t)[None, :], tgt[None, :]] += boost
    dev = torch.from_numpy(x).cuda().to(dtype)
    return dev, dev.float().cpu().numpy().astype(np.float64), tgt


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("chunks,t,v", [(1, 1, 1), (2, 3, 7), (3, 5, 8), (4, 2, 4099), (6, 16, 32000),
                                        (2, 4, 128256), (1, 2, 151936)])
def test_ppl_scores_match_oracle(dtype, chunks, t, v):
    dev, host, tgt = make_logits(chunks * 1000 + v, chunks, t, v, dtype)
    nll = torch.full((chunks, t), -1.0, device="cuda")
    score = torch.full((chunks,), -1.0, device="cuda")
    cc.cc_ppl_chunk_scores(ctx(), dev, torch.from_numpy(tgt).cuda(), nll, score)
    assert ctx().poll() == 0, ctx().lib.cc_last_error(ctx().handle)
    ref_s, ref_nll = orc.ppl_chunk_scores(host, tgt)
    np.testing.assert_allclose(nll.cpu().numpy(), ref_nll, atol=TOL, rtol=0)
    np.testing.assert_allclose(score.cpu().numpy(), ref_s, atol=TOL, rtol=0)


def test_ppl_scores_strided_rows_and_extreme_logits():
    """Rows inside a wider buffer; one row with a huge spread (no overflow, exact target term)."""
    chunks, t, v, pitch = 3, 4, 1000, 1024
    dev, host, tgt = make_logits(5, chunks, t, pitch, torch.float32)
    dev[1, 2, :v] = -300.0
    dev[1, 2, 17] = 250.0
    host = dev.cpu().numpy().astype(np.float64)
    view = dev[:, :, :v]
    tgt = (tgt % v).astype(np.int32)
    nll = torch.empty((chunks, t), device="cuda")
    score = torch.empty((chunks,), device="cuda")
    cc.cc_ppl_chunk_scores(ctx(), view, torch.from_numpy(tgt).cuda(), nll, score)
    assert ctx().poll() == 0
    ref_s, ref_nll = orc.ppl_chunk_scores(host[:, :, :v], tgt)
    np.testing.assert_allclose(nll.cpu().numpy(), ref_nll, atol=TOL, rtol=1e-6)


def test_ppl_scores_flag_a_bad_token_id():
    dev, _, tgt = make_logits(6, 2, 3, 64, torch.float32)
    tgt[1] = 64
    nll = torch.zeros((2, 3), device="cuda")
    score = torch.zeros((2,), device="cuda")
    cc.cc_ppl_chunk_scores(ctx(), dev, torch.from_numpy(tgt).cuda(), nll, score)
    assert ctx().poll() == cc.CC_ERR_DEVICE_FLAG
    out = nll.cpu().numpy()
    assert np.isnan(out[:, 1]).all() and np.isfinite(out[:, [0, 2]]).all()


@pytest.mark.parametrize("n,k", [(1, 1), (6, 3), (6, 9), (100, 6), (1000, 20), (8192, 64)])
def test_select_chunks_matches_oracle(n, k):
    rng = np.random.Generator(np.random.PCG64(n + k))
    s = (rng.integers(0, max(2, n // 3), size=n) / 7.0).astype(np.float32)       # many ties
    if n >= 6:
        s[4] = np.nan
    chosen = torch.full((max(k, 1),), -7, dtype=torch.int32, device="cuda")
    cc.cc_select_chunks(ctx(), torch.from_numpy(s).cuda(), k, chosen)
    assert ctx().poll() == 0
    ref = orc.select_chunks(s, k)
    got = chosen.cpu().numpy()
    assert got[:len(ref)].tolist() == ref.tolist()
    assert (got[len(ref):] == -7).all()


def test_scores_then_selection_pick_the_best_explained_query():
    """End to end on synthetic logits: the chunk whose logits favour the query tokens most has
    the lowest perplexity and comes first."""
    chunks, t, v = 8, 12, 5000
    rng = np.random.Generator(np.random.PCG64(77))
    x = rng.standard_normal((chunks, t, v)).astype(np.float32)
    tgt = rng.integers(0, v, size=t).astype(np.int32)
    x[5, np.arange(t), tgt] += 20.0
    x[2, np.arange(t), tgt] += 10.0
    dev = torch.from_numpy(x).cuda()
    nll = torch.empty((chunks, t), device="cuda")
    score = torch.empty((chunks,), device="cuda")
    chosen = torch.empty((2,), dtype=torch.int32, device="cuda")
    cc.cc_ppl_chunk_scores(ctx(), dev, torch.from_numpy(tgt).cuda(), nll, score)
    cc.cc_select_chunks(ctx(), score, 2, chosen)
    assert ctx().poll() == 0
    assert chosen.cpu().tolist() == [5, 2]
    assert orc.select_chunks(orc.ppl_chunk_scores(x, tgt)[0], 2).tolist() == [5, 2]
