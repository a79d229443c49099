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
