"""Host-side plumbing of a multi-process run: which layers a rank compresses and how the
ranks' timings become one job figure.

The hot path shards with no exchange: the units (layer, sequence, KV head) are independent
(Section 4.5: scoring and selection are per layer and per KV head), so every rank compresses
its own stream of layers and the only communication is a barrier and a max over the ranks'
device timings.  The process group may be NCCL (one rank per GPU) or gloo (CPU tests).
"""
from typing import List

import torch
import torch.distributed as dist

LAYER_STRIDE = 100      # rank r works on layers 100 r, 100 r + 1, ...: disjoint for < 100 layer sets


def rank_layers(rank: int, n_sets: int) -> List[int]:
    """Layer ids (seeds of the synthetic inputs) of the layer sets a rank cycles through."""
    if not 0 < n_sets <= LAYER_STRIDE:
        raise ValueError(f"n_sets must be in 1..{LAYER_STRIDE}")
    return [LAYER_STRIDE * rank + i for i in range(n_sets)]


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(ms: float, world: int, device: str = "cpu") -> float:
    """The slowest rank's duration: the job is done when the last rank is."""
    if world == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job tokens/s/layer: every rank processes ``tokens_per_step`` per step (weak
    scaling) and a step lasts as long as the slowest rank's."""
    return world * tokens_per_step / (ms_per_step * 1e-3)
