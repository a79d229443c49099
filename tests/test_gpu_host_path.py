"""`LayerCompressor.run_host`: inputs in page-locked host memory, the compacted cache copied back.
With `v_in_place` the V tensor is never copied to the device: the compaction kernel gathers the
retained rows straight from host memory.  Both forms must return the same bits, and those bits
must be the rows of the host K / V that the returned indices name."""
import numpy as np
import pytest
import torch

from paper_2604_10235_b200 import binding as cc
from paper_2604_10235_b200 import inputs as gen
from paper_2604_10235_b200.api import LayerCompressor, to_bf16

from gpu_util import ctx

pytestmark = pytest.mark.gpu

CASES = [
    gen.workloads()["tiny"],
    gen.Workload("host_rows", 51, 1, 28, 4, 128, 64, gen.POOL_AVG, 5, 300, n=3000),
    gen.Workload("host_paged", 52, 1, 8, 2, 128, 16, gen.POOL_MAX, 7, 0,
                 seq_lens=(300, 40, 2050, 129), budget_frac=0.1, page_size=16),
]


def _bits(t):
    return t.view(torch.int16) if t.dtype == torch.bfloat16 else t


def _valid_rows(wl):
    """Rows of k_out / v_out that hold a retained token (the tail of a sequence's last fresh page
    holds whatever the pool held there, which is not part of the result)."""
    ps = wl.page_size
    valid, row0 = [], 0
    for n, bud in zip(wl.lens, wl.budgets):
        keep = min(n, bud)
        valid.extend(range(row0, row0 + keep))
        row0 += (keep + ps - 1) // ps * ps if ps else bud
    return torch.tensor(valid, dtype=torch.long)


def _assert_same(a, b, valid):
    assert a.keys() == b.keys()
    for key in a:
        if key in ("k_out", "v_out"):
            assert torch.equal(_bits(a[key])[valid], _bits(b[key])[valid]), key
        else:
            assert torch.equal(a[key], b[key]), key


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_v_gathered_from_host_memory_equals_the_copying_form(wl):
    x = gen.make_layer(wl, layer=0)
    layout = x if wl.page_size else None
    host = (to_bf16(x.q_win, "cpu", pin=True), to_bf16(x.k, "cpu", pin=True),
            to_bf16(x.v, "cpu", pin=True), torch.from_numpy(x.prior).pin_memory())
    results = []
    for in_place in (False, True):
        comp = LayerCompressor(ctx(), wl, layout=layout)
        comp.v.fill_(7.0)                       # whatever the V pool holds must not leak into the result
        out = comp.run_host(*host, v_in_place=in_place)
        torch.cuda.synchronize()
        assert ctx().poll() == 0, ctx().lib.cc_last_error(ctx().handle)
        results.append({k: v.clone() for k, v in out.items()})
        if in_place:
            assert comp.h2d_bytes_of(True) < comp.h2d_bytes_of(False)
    a, b = results
    ps = wl.page_size
    _assert_same(a, b, _valid_rows(wl))

    # the returned rows are the host rows that idx names (bit copies)
    idx, count = b["idx"].numpy(), b["count"].numpy()
    k_h, v_h = _bits(host[1]).numpy(), _bits(host[2]).numpy()
    k_o, v_o = _bits(b["k_out"]).numpy(), _bits(b["v_out"]).numpy()
    off, page_off = 0, 0
    for s, (n, bud) in enumerate(zip(wl.lens, wl.budgets)):
        keep = min(n, bud)
        for h in range(wl.n_heads_kv):
            assert count[s, h] == keep
            toks = idx[h, off:off + keep]
            if ps:
                src = x.page_table[s][toks // ps].astype(np.int64) * ps + toks % ps
                dst = page_off * ps + np.arange(keep)      # h_k_out holds the sequences' new pages in order
            else:
                src = toks                                  # one sequence, rows = tokens
                dst = off + np.arange(keep)
            assert np.array_equal(k_o[dst, h], k_h[src, h])
            assert np.array_equal(v_o[dst, h], v_h[src, h])
        off += bud
        page_off += (keep + ps - 1) // ps if ps else 0


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_overlapped_readback_returns_every_call_s_results(wl):
    """Copies back to the host on the compressor's own stream, overlapping the next call's copies
    in: after finish() the host tensors hold the last call's results, and the results of the call
    before it were complete before its device buffers were overwritten."""
    xs = [gen.make_layer(wl, layer=l) for l in range(3)]
    if wl.page_size:
        for x in xs[1:]:
            gen.repage(x, xs[0])
    layout = xs[0] if wl.page_size else None
    hosts = [(to_bf16(x.q_win, "cpu", pin=True), to_bf16(x.k, "cpu", pin=True),
              to_bf16(x.v, "cpu", pin=True), torch.from_numpy(x.prior).pin_memory()) for x in xs]
    plain = LayerCompressor(ctx(), wl, layout=layout)
    want = []
    for h in hosts:
        out = plain.run_host(*h, v_in_place=True)
        torch.cuda.synchronize()
        want.append({k: v.clone() for k, v in out.items()})
    over = LayerCompressor(ctx(), wl, layout=layout)
    valid = _valid_rows(wl)
    for i, h in enumerate(hosts):
        out = over.run_host(*h, v_in_place=True, overlap_readback=True)
        if i == 1:
            # results of call 1 once they have landed; call 2 is enqueued only afterwards here
            over.finish()
            torch.cuda.synchronize()
            _assert_same(out, want[1], valid)
    over.finish()
    torch.cuda.synchronize()
    assert ctx().poll() == 0
    _assert_same(out, want[2], valid)
    # back to back without waiting in between: the last results still arrive intact
    for h in hosts:
        out = over.run_host(*h, v_in_place=True, overlap_readback=True)
    over.finish()
    torch.cuda.synchronize()
    _assert_same(out, want[2], valid)


def test_v_in_place_needs_page_locked_memory():
    wl = gen.workloads()["tiny"]
    x = gen.make_layer(wl, layer=0)
    comp = LayerCompressor(ctx(), wl)
    host = (to_bf16(x.q_win, "cpu", pin=True), to_bf16(x.k, "cpu", pin=True),
            to_bf16(x.v, "cpu", pin=False), torch.from_numpy(x.prior).pin_memory())
    with pytest.raises(ValueError):
        comp.run_host(*host, v_in_place=True)
    with pytest.raises(ValueError):                          # the binding refuses pageable memory too
        cc.cc_compact_kv(ctx(), comp.desc, comp.k, host[2], comp.idx, comp.k_out, comp.v_out)
