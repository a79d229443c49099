"""The multi-process plumbing on CPU: two gloo ranks take disjoint layer streams, meet at the
barrier, and agree on the slowest rank's time and on the job throughput.  No GPU needed."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_10235_b200 import inputs as gen
from paper_2604_10235_b200 import sharding


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out) -> None:
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        layers = sharding.rank_layers(rank, 4)
        wl = gen.workloads()["tiny"]
        x = gen.make_layer(wl, layer=layers[0], with_v=False)
        sharding.barrier(world)
        ms_local = 2.0 + rank                                  # rank 1 is the slow one
        ms = sharding.max_over_ranks(ms_local, world)
        out.put((rank, layers, int(x.k.astype(np.int64).sum()), ms,
                 sharding.job_throughput(1000, world, ms)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_layers_and_reduce_timings():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, l0, sum0, ms0, v0), (_, l1, sum1, ms1, v1) = got
    assert not set(l0) & set(l1)                  # disjoint layer streams
    assert sum0 != sum1                           # and therefore different synthetic inputs
    assert ms0 == ms1 == 3.0                      # everyone reports the slowest rank's time
    assert v0 == v1 == 2 * 1000 / 3.0e-3          # whole-job tokens/s: both ranks' tokens


def test_single_rank_needs_no_process_group():
    assert sharding.max_over_ranks(1.5, 1) == 1.5
    sharding.barrier(1)
    assert sharding.rank_layers(3, 2) == [300, 301]
    assert abs(sharding.job_throughput(32768, 1, 0.0689) - 32768 / 0.0689e-3) < 1e-3


def test_bench_launcher_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a torchrun environment starts two ranks (here: gloo ranks with
    a host stub in place of the CUDA step) and rank 0 reports both of them."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "3",
                          "--warmup", "1", "--impl", "stub"], capture_output=True, text=True,
                         timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                      # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["steps"] == 3
    assert lines[0]["ms_per_step"] >= 2.0 / 3   # the slower rank's time (rank 1 adds 2 ms)


def test_bench_roofline_arithmetic():
    """The host arithmetic behind the benchmark's roofline figures, against hand values for the
    Llama-shaped workload: K once + Q + prior + gathered rows; 2 w G d flops and w G exponentials
    per (key, KV head)."""
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    import bench
    wl = gen.workloads()["llama3_8b"]
    work = bench.algorithmic_work(wl)
    assert work["tokens"] == 32768
    assert work["flops"] == 2.0 * 64 * 4 * 128 * 32768 * 8                    # 17.18 GFLOP
    assert work["exps"] == 64 * 4 * 32768 * 8                                 # 67.1 M per pass
    k_bytes = 32768 * 8 * 256
    assert work["bytes"] == k_bytes + 64 * 32 * 256 + 4 * 32768 + 4 * 2048 * 8 * 256 + 4 * 2048 * 8
    peaks = {"hbm_gbs": 6532.9, "bf16_tflops": 1628.0}
    r = bench.roofline_of(work, peaks, 62.0e-6, clock_mhz=1965.0)
    assert r["bound"] == "hbm" and abs(r["t_roof_us"] - 12.95) < 0.01 and abs(r["t_flops_us"] - 10.55) < 0.01
    assert abs(r["frac"] - 12.95 / 62.0) < 1e-3
    rate = bench.EXP_RATE["registers"]
    assert abs(r["exp_bound_us"] - 2 * 67108864 / (rate * 148 * 1965e6) * 1e6) < 1e-6
    # dominant kernels: the binding one of bytes, flops and exponentials, each at its own peak
    k = bench.score_kernel_roofline(work, dict(peaks, source="measured"), 50.0e-6)
    t_alu = 2 * 67108864 / (25.6 * 148 * 1965e6)
    assert k["bound"] == "alu" and abs(k["frac"] - t_alu / 50.0e-6) < 1e-9
    assert abs(k["achieved"] - 2 * 67108864 / 50.0e-6 / 1e9) < 1e-6 and k["unit"] == "Gexp/s"
    assert abs(k["frac_of"]["tensor"] - 10.55 / 50.0) < 1e-3 and abs(k["frac_of"]["hbm"] - 10.513 / 50.0) < 1e-4
    slow_alu = dict(work, exps=work["exps"] / 100)        # without the exponentials the flops bind
    assert bench.score_kernel_roofline(slow_alu, dict(peaks, source="measured"), 50.0e-6)["bound"] == "tensor"
    cfg = bench.bench_config(gen.workloads()["ragged_paged"])
    assert cfg["workload"] == "ragged_paged" and cfg["layers_cycled"] == 2 and "larger than L2" in cfg["l2"]
