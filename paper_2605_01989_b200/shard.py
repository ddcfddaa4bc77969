"""Host-side logic for running the receive path on several GPUs, one process per GPU.

The path shards like a parameter server split by offset range: rank r owns a contiguous run of gradient tensors,
keeps its own rings, bitmap and aggregate for them, and runs the four calls without looking at another GPU's memory.
The only exchange is a sum of the per-worker (received, missing, total) chunk counts, after which every rank takes the
same stop / continue decision with the library's own rule (dblp_bound_ok)."""
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def partition_tensors(numel: Sequence[int], world: int) -> List[Tuple[int, int]]:
    """Splits tensors 0..T-1 into `world` contiguous runs [lo, hi) of nearly equal element count: the cut between
    run r-1 and run r is the tensor boundary whose prefix sum is closest to r / world of the total.  Runs may be empty
    when there are fewer tensors than ranks."""
    prefix = [0]
    for n in numel:
        prefix.append(prefix[-1] + n)
    total, cuts = prefix[-1], [0]
    for r in range(1, world):
        target = total * r / world
        best = min(range(cuts[-1], len(prefix)), key=lambda i: (abs(prefix[i] - target), i))
        cuts.append(best)
    cuts.append(len(numel))
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def shard_offsets(numel: Sequence[int], parts: Sequence[Tuple[int, int]]) -> List[Tuple[int, int]]:
    """Element range [first, last) of the flat gradient that each run of tensors covers."""
    prefix = [0]
    for n in numel:
        prefix.append(prefix[-1] + n)
    return [(prefix[lo], prefix[hi]) for lo, hi in parts]


def exchange_counts(recv_cnt: torch.Tensor, missing_cnt: torch.Tensor, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Sums the per-worker counts over all ranks (in place on copies widened to int64).  Works on CPU tensors with
    gloo and on CUDA tensors with NCCL."""
    r = recv_cnt.to(torch.int64).clone()
    m = missing_cnt.to(torch.int64).clone()
    dist.all_reduce(r, group=group)
    dist.all_reduce(m, group=group)
    return r, m


def decide(bound_ok, recv_total: torch.Tensor, missing_total: torch.Tensor, bound_ppm: int) -> Tuple[List[int], int]:
    """Per-worker decisions and their conjunction from the summed counts; `bound_ok(missing, total, ppm)` is the
    library's rule (binding.dblp_bound_ok)."""
    ok = [int(bound_ok(int(m), int(r) + int(m), bound_ppm)) for r, m in zip(recv_total.flatten().tolist(),
                                                                            missing_total.flatten().tolist())]
    return ok, int(all(ok))
