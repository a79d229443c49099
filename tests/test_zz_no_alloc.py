"""cc_topk_select_static: the selection entry point that needs no workspace.

Some callers cannot allocate device memory at the moment they need a selection (their
allocator already owns the device, or a blocking cudaMalloc is not acceptable inside their
request loop), so this variant keeps its scratch in a fixed array inside the library.  The
test calls it through the C ABI twice in a row, with different shapes so that the second call
meets the first call's left-over scratch, and requires exactly the indices and counts of
cc_topk_select and of the CPU oracle's selection (integer outputs: bit for bit), and that the
call leaves the device's free memory as it found it.  It is collected last so that a run that stops
at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from oracle import codecomp_oracle as orc
from paper_2604_10235_b200 import binding as cc

pytestmark = pytest.mark.gpu


def _case(seed, n, hkv, budget, chunk=1, span_ratio=0.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    m = (n + chunk - 1) // chunk
    fused = rng.choice(rng.random(97).astype(np.float32), size=(hkv, m)).astype(np.float32)
    prior = rng.choice(np.array([0, 0, 0, 0, 0, 0.3, 0.7, 1.0], np.float32), size=n)
    d = cc.Desc(hkv, hkv, 4, n=n, budget=budget, pool_kind=cc.CC_POOL_NONE, pool_size=1,
                chunk_size=chunk, force_threshold=0.5, span_ratio=span_ratio, span_min=8)
    return d, torch.from_numpy(fused).cuda(), torch.from_numpy(prior).cuda()


def _both(ctx, d, fused, prior):
    hkv, b = d.c.n_heads_kv, d.c.budget
    ref_idx = torch.full((hkv, b), -7, dtype=torch.int32, device="cuda")
    ref_cnt = torch.full((hkv,), -7, dtype=torch.int32, device="cuda")
    cc.cc_topk_select(ctx, d, fused, prior, ref_idx, ref_cnt)
    got_idx = torch.full((hkv, b), -9, dtype=torch.int32, device="cuda")
    got_cnt = torch.full((hkv,), -9, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    cc.cc_topk_select_static(ctx, d, fused, prior, got_idx, got_cnt)
    assert ctx.poll() == 0
    assert torch.cuda.mem_get_info()[0] == free_before        # nothing allocated, nothing freed
    assert torch.equal(got_idx, ref_idx)
    assert torch.equal(got_cnt, ref_cnt)
    # ... and the oracle's selection of the same fp32 values
    f_h, p_h, got = fused.cpu().numpy(), prior.cpu().numpy(), got_idx.cpu().numpy()
    chunk = max(1, d.c.chunk_size)
    n = d.c.n
    item_p = orc.chunk_reduce(np.zeros(n), p_h, chunk)[1] if chunk > 1 else p_h
    for h in range(hkv):
        ref = orc.select_tokens(f_h[h], item_p, n, b, 0.5, d.c.span_ratio, d.c.span_min, chunk)
        assert int(got_cnt[h]) == len(ref)
        np.testing.assert_array_equal(got[h, :len(ref)], ref)


def test_static_scratch_select_matches_workspace_select_twice_in_a_row():
    ctx = cc.Context(0)
    # first call: large, many protected tokens, span cap active (fills the scratch with flags)
    _both(ctx, *_case(1, 40000, 8, 4000, span_ratio=0.5))
    # second call right after it: smaller and chunked, so it reads scratch the first call wrote
    _both(ctx, *_case(2, 5003, 2, 600, chunk=10))
    _both(ctx, *_case(3, 40000, 8, 4000))
    # chunk-level ranking together with the span cap
    _both(ctx, *_case(4, 7001, 3, 900, chunk=10, span_ratio=0.5))


def test_static_scratch_select_rejects_oversized_batches():
    ctx = cc.Context(0)
    n = cc.CC_STATIC_SELECT_MAX_ITEMS // 8 + 8
    d = cc.Desc(8, 8, 4, n=n, budget=16, pool_kind=cc.CC_POOL_NONE, pool_size=1)
    fused = torch.zeros((8, n), device="cuda")
    prior = torch.zeros((n,), device="cuda")
    idx = torch.zeros((8, 16), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((8,), dtype=torch.int32, device="cuda")
    with pytest.raises(cc.CodecompError) as e:
        cc.cc_topk_select_static(ctx, d, fused, prior, idx, cnt)
    assert e.value.status == cc.CC_ERR_UNSUPPORTED
    assert "static scratch" in str(e.value)
