"""Calls enqueued back to back, with no synchronisation in between and replayed from a CUDA graph
as `bench.py` does: the kernels of consecutive calls overlap through programmatic dependent
launch (a kernel may start while its predecessor drains), so every output is compared bit for
bit with what the same call produces when it runs alone."""
import pytest
import torch

from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen
from paper_2604_10235_b200.api import LayerCompressor, to_bf16

from gpu_util import ctx

pytestmark = pytest.mark.gpu


def _inputs(wl, layer):
    x = gen.make_layer(wl, layer=layer)
    return (to_bf16(x.q_win), to_bf16(x.k), to_bf16(x.v), torch.from_numpy(x.prior).cuda())


def _snapshot(comp):
    scores, fused = cc.cc_workspace_views(comp.ctx, comp.desc, comp.ws)
    return [t.clone() for t in (comp.idx, comp.count, comp.k_out, comp.v_out, scores, fused)]


@pytest.mark.parametrize("wl", [
    gen.workloads()["tiny"],
    gen.workloads()["llama3_8b"],
    gen.Workload("b2b", 40, 1, 8, 2, 128, 32, gen.POOL_MAX, 7, 600, n=6000),
    gen.Workload("b2b_rows", 41, 1, 28, 4, 128, 64, gen.POOL_AVG, 5, 300, n=3000),
    gen.Workload("b2b_chunks", 42, 1, 8, 2, 128, 32, gen.POOL_NONE, 1, 250, n=3003, chunk_size=10),
], ids=lambda w: w.name)
def test_back_to_back_calls_match_single_calls(wl):
    n_sets = 3
    sets = [_inputs(wl, layer) for layer in range(n_sets)]
    # one compressor (one workspace, one set of outputs) per input set, so that the outputs of
    # every call survive until the end; plus one shared compressor that all inputs go through
    comps = [LayerCompressor(ctx(), wl) for _ in range(n_sets)]
    shared = LayerCompressor(ctx(), wl)
    want = []
    for comp, s in zip(comps, sets):
        comp.run_device(*s)
        torch.cuda.synchronize()
        want.append(_snapshot(comp))
        for t in (comp.idx, comp.count, comp.k_out, comp.v_out, comp.ws):
            t.zero_()
    torch.cuda.synchronize()

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for _ in range(3):
                for comp, s in zip(comps, sets):
                    comp.run_device(*s)
                    shared.run_device(*s)          # same workspace and outputs, call after call
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert ctx().poll() == 0, ctx().lib.cc_last_error(ctx().handle)
    for comp, ref in zip(comps, want):
        for got, exp in zip(_snapshot(comp), ref):
            assert torch.equal(got, exp)
    for got, exp in zip(_snapshot(shared), want[-1]):          # the last call through the shared one
        assert torch.equal(got, exp)


def test_all_layers_call_equals_separate_calls():
    """cc_compress_layers on three layers: indices, counts and gathered K/V of every layer equal
    those of three cc_compress_layer calls, bit for bit; contiguous and paged."""
    from gpu_util import bf16_dev, ctx, desc_for
    for wl in (gen.workloads()["tiny"],
               gen.Workload("rp", 32, 1, 8, 2, 128, 16, gen.POOL_MAX, 7, 0,
                            seq_lens=(300, 40, 2050, 129), budget_frac=0.1, page_size=16)):
        paged = wl.page_size > 0
        xs = [gen.make_layer(wl, layer=l) for l in range(3)]
        if paged:
            for x in xs[1:]:
                gen.repage(x, xs[0])
        pt = torch.from_numpy(xs[0].page_table).cuda() if paged else None
        b_tot = sum(wl.budgets)
        stride = max((b + 15) // 16 for b in wl.budgets) + 1 if paged else 0
        d = desc_for(wl, cc.CC_MODE_BF16, page_table=pt, out_pt_stride=stride, pool_pages=xs[0].pool_pages)
        ws = ctx().workspace(d)
        prior = torch.from_numpy(xs[0].prior).cuda()

        def fresh():
            q = [bf16_dev(x.q_win) for x in xs]
            k = [bf16_dev(x.k) for x in xs]
            v = [bf16_dev(x.v) for x in xs]
            idx = [torch.full((wl.n_heads_kv, b_tot), -9, dtype=torch.int32, device="cuda") for _ in xs]
            cnt = [torch.full((len(wl.lens), wl.n_heads_kv), -9, dtype=torch.int32, device="cuda") for _ in xs]
            if paged:
                ko, vo = k, v
                free = [torch.from_numpy(x.free_pages).cuda() for x in xs]
                opt = [torch.full((len(wl.lens), stride), -9, dtype=torch.int32, device="cuda") for _ in xs]
            else:
                ko = [torch.zeros((b_tot, wl.n_heads_kv, 128), dtype=torch.bfloat16, device="cuda") for _ in xs]
                vo = [torch.zeros_like(t) for t in ko]
                free = opt = None
            return q, k, v, ko, vo, idx, cnt, free, opt

        a = fresh()
        for l in range(3):
            cc.cc_compress_layer(ctx(), d, a[0][l], a[1][l], a[2][l], prior, a[3][l], a[4][l], a[5][l],
                                 a[6][l], a[7][l] if paged else None, a[8][l] if paged else None, ws)
        b = fresh()
        cc.cc_compress_layers(ctx(), d, b[0], b[1], b[2], prior, b[3], b[4], b[5], b[6], b[7], b[8], ws)
        assert ctx().poll() == 0
        for l in range(3):
            for j in (3, 4, 5, 6):
                assert torch.equal(a[j][l].view(torch.int16) if a[j][l].dtype == torch.bfloat16 else a[j][l],
                                   b[j][l].view(torch.int16) if b[j][l].dtype == torch.bfloat16 else b[j][l])
            if paged:
                assert torch.equal(a[8][l], b[8][l])
