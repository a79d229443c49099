#!/usr/bin/env python
"""Benchmark of the CodeComp per-layer KV-compression hot path on B200.

One "step" is one call of the fused path (score -> pool -> prior fuse -> select -> compact)
on one layer of the workload.  The metric is prefix tokens compressed per second per layer;
with N GPUs every rank compresses its own layer stream (weak scaling, no data-path
collective) and the value is the sum over ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama3_8b] [--impl reference]

Prints one JSON line (rank 0).  ``--impl reference`` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "prefix tokens compressed/sec per layer (score+prior+topk+gather)"
UNIT = "tokens/s/layer"
N_LAYER_SETS = 4          # distinct K/V sets cycled through so that no step finds its keys in L2


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def algorithmic_work(wl):
    """Bytes and flops one layer needs on paper: K read once, Q, prior, the gathered K/V rows
    read and written once, the index lists; 2*w*G*d flops per (key, KV head)."""
    d, hkv, hq, w = wl.head_dim, wl.n_heads_kv, wl.n_heads_q, wl.window
    n_tot = sum(wl.lens)
    keep = sum(min(b, n) for b, n in zip(wl.budgets, wl.lens))
    row = d * 2
    k_bytes = n_tot * hkv * row
    q_bytes = len(wl.lens) * w * hq * row
    score_bytes = k_bytes + q_bytes + 4 * n_tot * hkv            # the score kernel alone
    gather_bytes = 4 * keep * hkv * row + 4 * keep * hkv          # K,V rows read + written, idx
    bytes_total = k_bytes + q_bytes + 4 * n_tot + gather_bytes
    flops = 2.0 * w * wl.group * d * n_tot * hkv
    return {"bytes": float(bytes_total), "flops": flops, "score_bytes": float(score_bytes),
            "gather_bytes": float(gather_bytes), "tokens": n_tot}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while timing runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle arm
_ORACLE_INPUTS = {}


def oracle_throughput(wl, budget_s: float):
    """Times the oracle (as it stands) on a bounded sample of one layer: a subset of the KV
    heads, all keys, whole path.  Returns tokens/s/layer scaled to all heads."""
    from oracle import codecomp_oracle as orc
    from paper_2604_10235_b200 import inputs as gen
    if wl.name not in _ORACLE_INPUTS:
        _ORACLE_INPUTS[wl.name] = gen.make_layer(wl, layer=0)
    x = _ORACLE_INPUTS[wl.name]
    s = 0
    n = wl.lens[s]
    lo = int(x.tok_offsets[s])
    if wl.page_size:
        rows = orc.paged_rows(x.page_table[s], n, wl.page_size)
    else:
        rows = np.arange(lo, lo + n)
    g = wl.group

    def run(heads: int) -> float:
        k = x.k[rows][:, :heads]
        v = x.v[rows][:, :heads]
        q = x.q_win[s][:, :heads * g]
        t0 = time.perf_counter()
        orc.compress_sequence(q, k, v, x.prior[lo:lo + n], heads, wl.pool_kind, wl.pool_size,
                              wl.budgets[s], wl.alpha, wl.beta, wl.force_threshold,
                              wl.span_ratio, wl.span_min, max(1, wl.chunk_size))
        return time.perf_counter() - t0

    t1 = run(1)
    heads = int(max(1, min(wl.n_heads_kv, budget_s // max(t1, 1e-3))))
    t = run(heads) if heads > 1 else t1
    t_layer = t * wl.n_heads_kv / heads
    try:
        import threadpoolctl
        cores = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    return {"value": n / t_layer, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"sequence 0 ({n} tokens), {heads} of {wl.n_heads_kv} KV heads, whole path, "
                      f"time scaled to all heads", "seconds": t}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total_budget = 150.0
    per_step = max(0.3, min(8.0, total_budget / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_throughput(wl, per_step)
    times, last = [], None
    t0 = time.perf_counter()
    for _ in range(args.steps):
        last = oracle_throughput(wl, per_step)
        times.append(last["value"])
        if time.perf_counter() - t0 > total_budget:
            break
    value = float(np.mean(times))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": len(times), "warmup": args.warmup,
            "ms_per_step": 1e3 * sum(wl.lens) / value, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "note": "CPU oracle, NumPy fp64, host cores"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- CUDA arm
def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2604_10235_b200 import binding as cc
    from paper_2604_10235_b200 import inputs as gen
    from paper_2604_10235_b200 import sharding
    from paper_2604_10235_b200.api import LayerCompressor, to_bf16

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    ctx = cc.Context(local)
    layers = sharding.rank_layers(rank, N_LAYER_SETS)
    layout0 = gen.make_layer(wl, layer=layers[0]) if wl.page_size else None
    comp = LayerCompressor(ctx, wl, layout=layout0)
    work = algorithmic_work(wl)
    peaks = load_peaks()

    # inputs: N_LAYER_SETS layers, resident in HBM before timing, plus pinned host copies
    dev_sets, host_sets = [], []
    for i, layer in enumerate(layers):
        x = gen.make_layer(wl, layer=layer)
        if wl.page_size and i > 0:
            gen.repage(x, layout0)          # every layer set uses the page layout of the first
        hs = (to_bf16(x.q_win, "cpu", pin=True), to_bf16(x.k, "cpu", pin=True),
              to_bf16(x.v, "cpu", pin=True), torch.from_numpy(x.prior).pin_memory())
        host_sets.append(hs)
        dev_sets.append(tuple(t.cuda() for t in hs))
    set_bytes = sum(t.numel() * t.element_size() for t in dev_sets[0])

    def barrier():
        sharding.barrier(world)
        torch.cuda.synchronize()

    def max_over_ranks(ms: float) -> float:
        return sharding.max_over_ranks(ms, world, "cuda")

    # ---- device-resident timing: the fused call on each of the layer sets is captured once in
    # a CUDA graph (one replay = N_LAYER_SETS steps), so the timed region holds kernel time and
    # launch dependencies, not the Python binding's host time between calls
    for i in range(args.warmup):
        comp.run_device(*dev_sets[i % N_LAYER_SETS])
    assert ctx.poll() == 0
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for j in range(N_LAYER_SETS):
                comp.run_device(*dev_sets[j])
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    n_replays, n_rest = divmod(args.steps, N_LAYER_SETS)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_replays):
        graph.replay()
    for j in range(n_rest):
        comp.run_device(*dev_sets[j])
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    status = ctx.poll()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")
    ms_step = ms_total / args.steps
    value = sharding.job_throughput(work["tokens"], world, ms_step)

    # ---- per-stage durations: each stage entry point captured the same way and replayed
    d = comp.desc
    scores = torch.empty((wl.n_heads_kv, d.n_tot), device="cuda")
    fused = torch.empty((wl.n_heads_kv, d.m_tot), device="cuda")

    def stage_call(k, q_d, k_d, v_d, p_d):
        if k == 0:
            cc.cc_score_window(ctx, d, q_d, k_d, scores, None, ws=comp.ws)
        elif k == 1:
            cc.cc_fuse_prior_pool(ctx, d, scores, p_d, fused)
        elif k == 2:
            cc.cc_topk_select(ctx, d, fused, p_d, comp.idx, comp.count, ws=comp.ws)
        elif k == 3:
            if comp.paged:
                cc.cc_compact_kv(ctx, d, k_d, v_d, comp.idx, k_d, v_d, comp.free_pages,
                                 comp.out_page_table)
            else:
                cc.cc_compact_kv(ctx, d, k_d, v_d, comp.idx, comp.k_out, comp.v_out)
        else:
            # not part of a step: the retained fraction of the structurally critical tokens
            cc.cc_structural_score(ctx, d, comp.idx, p_d, wl.force_threshold, str_score)

    str_score = torch.empty((len(wl.lens), wl.n_heads_kv), device="cuda")
    stage_ms = np.zeros(5)
    stage_reps = max(1, min(args.steps, 200) // N_LAYER_SETS)
    for k in range(5):
        for j in range(N_LAYER_SETS):
            stage_call(k, *dev_sets[j])
        torch.cuda.synchronize()
        side.wait_stream(torch.cuda.current_stream())
        g_stage = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g_stage, stream=side):
                for j in range(N_LAYER_SETS):
                    stage_call(k, *dev_sets[j])
        torch.cuda.current_stream().wait_stream(side)
        g_stage.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(stage_reps):
            g_stage.replay()
        e1.record()
        torch.cuda.synchronize()
        stage_ms[k] = e0.elapsed_time(e1) / (stage_reps * N_LAYER_SETS)
    score_s = stage_ms[0] * 1e-3
    achieved_tf = work["flops"] / score_s / 1e12
    t_bytes = work["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_flops = work["flops"] / (peaks["bf16_tflops"] * 1e12)
    t_roof = max(t_bytes, t_flops)

    # ---- end to end: pinned host inputs in, compacted cache back out, every step
    n_e2e = max(3, min(args.steps, 40))
    for i in range(2):
        comp.run_host(*host_sets[i % N_LAYER_SETS])
    barrier()
    e0.record()
    for i in range(n_e2e):
        comp.run_host(*host_sets[i % N_LAYER_SETS])
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1)) / n_e2e
    e2e_value = sharding.job_throughput(work["tokens"], world, ms_e2e)

    aux = chunk_scoring_bandwidth(ctx, peaks) if rank == 0 and world == 1 else None
    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = oracle_throughput(wl, 12.0)
            cpu.pop("seconds", None)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "layers_cycled": N_LAYER_SETS,
                       "launch": f"CUDA graph of {N_LAYER_SETS} fused steps, replayed",
                       "n": list(wl.lens), "heads_q": wl.n_heads_q, "heads_kv": wl.n_heads_kv,
                       "window": wl.window, "pool": [wl.pool_kind, wl.pool_size],
                       "budget": list(wl.budgets), "chunk": wl.chunk_size,
                       "l2": f"inputs larger than L2: {N_LAYER_SETS} layer sets of "
                             f"{set_bytes / 1e6:.0f} MB cycled, no set reused within "
                             f"{(N_LAYER_SETS - 1) * set_bytes / 1e6:.0f} MB of traffic"},
            "roofline": {"bound": "tensor", "kernel": "score_tc_kernel<1> + score_tc_kernel<2> (the two launches of the score stage)",
                         "achieved": achieved_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": achieved_tf / peaks["bf16_tflops"], "traffic": score_traffic(wl),
                         "peak_source": f"{peaks['source']} bf16 burst",
                         "flops_per_launch_pair": work["flops"]},
            "path_roofline": {"t_roof_us": t_roof * 1e6, "t_bytes_us": t_bytes * 1e6,
                              "t_flops_us": t_flops * 1e6, "t_path_us": ms_step * 1e3,
                              "frac": t_roof / (ms_step * 1e-3), "bytes": work["bytes"],
                              "flops": work["flops"], "hbm_peak_gbs": peaks["hbm_gbs"]},
            "stage_us": {"score": stage_ms[0] * 1e3, "fuse_pool": stage_ms[1] * 1e3,
                         "select": stage_ms[2] * 1e3, "compact": stage_ms[3] * 1e3,
                         "str_score_diagnostic": stage_ms[4] * 1e3},
            "str_score": [round(float(v), 4) for v in str_score.flatten().tolist()],
            "chunk_scoring": aux,
            "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": comp.h2d_bytes,
                    "d2h_bytes_per_step": comp.d2h_bytes, "ms_per_step": ms_e2e, "steps": n_e2e},
            # per step: score pass 1, score pass 2, pool + fuse + select (one cluster kernel), compact
            "gpu_launches": 4 * args.steps,
            "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def chunk_scoring_bandwidth(ctx, peaks):
    """Not part of a step: the chunk-selection kernel (cc_ppl_chunk_scores) on synthetic bf16 and
    f32 logits of a 128256-token vocabulary, as achieved bytes/s against the HBM peak.  Two logit
    sets larger than L2 alternate, so no call finds its input cached."""
    import torch
    from paper_2604_10235_b200 import binding as cc
    chunks, t, v = 32, 64, 128256
    out = {"shape": [chunks, t, v], "bound": "hbm", "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    tgt = torch.randint(0, v, (t,), device="cuda", dtype=torch.int32)
    nll = torch.empty((chunks, t), device="cuda")
    score = torch.empty((chunks,), device="cuda")
    for name, dtype in (("bf16", torch.bfloat16), ("f32", torch.float32)):
        gen_ = torch.Generator(device="cuda").manual_seed(7)
        sets = [torch.randn((chunks, t, v), device="cuda", generator=gen_).to(dtype) for _ in range(2)]
        for x in sets:
            cc.cc_ppl_chunk_scores(ctx, x, tgt, nll, score)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 10
        e0.record()
        for _ in range(reps):
            for x in sets:
                cc.cc_ppl_chunk_scores(ctx, x, tgt, nll, score)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (2 * reps)
        gbs = sets[0].numel() * sets[0].element_size() / ms * 1e-6
        out[name] = {"us": ms * 1e3, "achieved": gbs, "frac": gbs / peaks["hbm_gbs"]}
        del sets
    if ctx.poll() != 0:
        raise RuntimeError("device status after the chunk-scoring measurement")
    return out


# DRAM bytes (read + write) of one launch pair of the score stage, from the ncu capture that
# is summarised under profiles/ (llama3_8b: 67.67 + 0.81 MB for pass 1,
# 68.00 + 1.44 MB for pass 2).  The counters were taken on the kernel as it stands in this tree;
# other workloads have no capture and report null.
SCORE_TRAFFIC_BYTES = {"llama3_8b": 137.93e6}


def score_traffic(wl):
    return SCORE_TRAFFIC_BYTES.get(wl.name)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3_8b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2604_10235_b200 import inputs as gen
    wl = gen.workloads()[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
