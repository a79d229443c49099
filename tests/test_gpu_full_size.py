"""Parity at the full benchmark sizes: the fused call on the workloads `bench.py` times (same
entry point, same launch configuration), every output checked against the fp64 oracle exactly as
in the small cases (all scores within tolerance, retained sets equal outside the tolerance band
of the cut-off, counts, order, protected tokens, gathered K/V bits, page tables).  The oracle
needs a few seconds per workload at these sizes."""
import pytest

from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen

from test_gpu_compress import check_layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["llama3_8b", "qwen25_coder_7b", "chunk10", "paper_avg5_w128"])
def test_benchmark_workload_full_size(name):
    wl = gen.workloads()[name]
    if wl.span_ratio:
        from dataclasses import replace
        wl = replace(wl, span_ratio=0.0)      # check_layer's tolerance band assumes uncapped protection
    check_layer(wl, gen.make_layer(wl, layer=1), cc.CC_MODE_BF16, 2e-3)


def test_ragged_paged_full_size():
    """293 k tokens in 8 sequences of 8192..65536 tokens, 16-token pages scattered over the pool,
    output into fresh pages."""
    wl = gen.workloads()["ragged_paged"]
    check_layer(wl, gen.make_layer(wl), cc.CC_MODE_BF16, 2e-3)


@pytest.mark.parametrize("density", ["5", "15", "30"])
@pytest.mark.parametrize("budget", [1024, 4096, 8192])
def test_qwen_shape_budget_and_prior_density_sweep(budget, density):
    """65536 tokens, 28 / 4 heads: budgets below and above the number of protected tokens (5 %
    of the tokens = 3277 protected: the attention scores fill the rest for B = 4096 and 8192;
    15 % and 30 % exceed every budget, so the first B protected tokens are kept)."""
    wl = gen.qwen_variant(gen.workloads()["qwen25_coder_7b"], budget, density)
    check_layer(wl, gen.make_layer(wl, layer=2), cc.CC_MODE_BF16, 2e-3)
