"""The receive path on several GPUs, one process per GPU: a parameter server split by offset range.

Rank r owns a contiguous run of the gradient tensors.  It keeps its own rings, claim table, bitmap columns and
aggregate range for them and runs the whole round (dblp_round_device) without looking at another GPU's memory.
The loss process is drawn by each packet's number in the whole worker stream (dblp_plan_set_shard), so the shards'
bitmaps side by side are the bitmap of the unsplit round and the stitched aggregate is the unsplit aggregate.

Two exchanges per round, both plain collectives of torch.distributed (NCCL on GPUs, gloo on CPU):
  * the per-worker (received, missing) chunk counts are summed over the ranks, after which every rank takes the same
    stop / continue decision with the library's own rule (dblp_bound_ok) -- a worker stream is judged as a whole
    (Section III-B), not per server shard;
  * for the broadcast half (Algorithm 3: the server sends the mean back), the aggregate ranges are all-gathered.

`sharded_round` is the one function that runs a round this way.  The per-rank work is behind a small runner interface
so that the same function serves the CUDA library (GpuShardRunner, below) and, in the CPU tests, a stand-in runner.
"""
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

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


@dataclass
class ShardSpec:
    """What rank `rank` of `world` owns: tensors [tensor_lo, tensor_hi), flat elements [elem_lo, elem_hi), and the
    chunks [seq_offset, seq_offset + chunks) of worker streams that are stream_chunks long in all."""
    rank: int
    world: int
    tensor_lo: int
    tensor_hi: int
    elem_lo: int
    elem_hi: int
    seq_offset: int
    chunks: int
    stream_chunks: int
    numel: List[int]

    @property
    def empty(self) -> bool:
        return self.tensor_hi == self.tensor_lo


def shard_specs(numel: Sequence[int], elems_per_chunk: int, world: int) -> List[ShardSpec]:
    """The specs of all ranks.  Chunking is per tensor, so a tensor boundary is also a chunk boundary."""
    parts = partition_tensors(numel, world)
    offs = shard_offsets(numel, parts)
    chunks_of = [-(-int(n) // elems_per_chunk) for n in numel]
    cprefix = [0]
    for c in chunks_of:
        cprefix.append(cprefix[-1] + c)
    return [ShardSpec(r, world, lo, hi, offs[r][0], offs[r][1], cprefix[lo], cprefix[hi] - cprefix[lo], cprefix[-1],
                      [int(n) for n in numel[lo:hi]]) for r, (lo, hi) in enumerate(parts)]


def exchange_counts(recv_cnt: torch.Tensor, missing_cnt: torch.Tensor, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Sums the per-worker counts over all ranks (on copies widened to int64).  Works on CPU tensors with gloo and on
    CUDA tensors with NCCL."""
    both = torch.stack([recv_cnt.to(torch.int64).flatten(), missing_cnt.to(torch.int64).flatten()])
    dist.all_reduce(both, group=group)
    return both[0], both[1]


def decide(bound_ok, recv_total: torch.Tensor, missing_total: torch.Tensor, bound_ppm: int) -> Tuple[List[int], int]:
    """Per-worker decisions and their conjunction from the summed counts; `bound_ok(missing, total, ppm)` is the
    library's rule (binding.dblp_bound_ok)."""
    ok = [int(bound_ok(int(m), int(r) + int(m), bound_ppm)) for r, m in zip(recv_total.flatten().tolist(),
                                                                            missing_total.flatten().tolist())]
    return ok, int(all(ok))


def gather_ranges(local: torch.Tensor, specs: Sequence[ShardSpec], group=None) -> torch.Tensor:
    """All-gathers the ranks' aggregate ranges into the full aggregate (every rank gets all of it).  Ranges differ in
    length, so each is padded to the longest before the collective and cut back afterwards."""
    sizes = [s.elem_hi - s.elem_lo for s in specs]
    longest = max(sizes)
    padded = local if local.numel() == longest else torch.cat([local, local.new_zeros(longest - local.numel())])
    parts = [torch.empty_like(padded) for _ in specs]
    dist.all_gather(parts, padded.contiguous(), group=group)
    return torch.cat([p[:n] for p, n in zip(parts, sizes)])


def sharded_round(runner, specs: Sequence[ShardSpec], rnd: int, bound_ppm: int, gather: bool = True, group=None,
                  marks=None) -> dict:
    """One round of the split server on this rank; enqueues work and collectives and does not wait for them.
    `runner.round(rnd, bound_ppm, marks)` does the rank's own work and returns (aggregate range as a 1-D fp32 tensor,
    per-worker received counts, per-worker missing counts), all on the device the process group communicates on; a rank
    whose spec is empty passes runner=None.  Returns the counts summed over the ranks ("recv", "missing", int64), the
    rank's own range ("agg_range") and, with gather, the full aggregate ("agg").  `decision` turns the summed counts
    into the stop / continue decision."""
    if runner is not None:
        agg, recv, miss = runner.round(rnd, bound_ppm, marks)
    else:
        agg = recv = miss = None
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        if runner is None:                       # nothing owned: zeros of the right shape join the collectives
            W, device = _peer_shape(group)
            recv = torch.zeros(W, dtype=torch.int64, device=device)
            miss = torch.zeros(W, dtype=torch.int64, device=device)
            agg = torch.zeros(0, dtype=torch.float32, device=device)
        recv_t, miss_t = exchange_counts(recv, miss, group)
        full = gather_ranges(agg, specs, group) if gather else None
    else:
        recv_t, miss_t = recv.flatten(), miss.flatten()
        full = agg if gather else None
    return {"recv": recv_t, "missing": miss_t, "agg_range": agg, "agg": full}


def decision(result: dict, bound_ok, bound_ppm: int) -> Tuple[List[int], int]:
    """Reads the summed counts of a `sharded_round` back to the host (this waits for the round) and applies the
    library's rule to every worker stream."""
    return decide(bound_ok, result["recv"], result["missing"], bound_ppm)


_peer = {}


def set_peer_shape(W: int, device) -> None:
    """For ranks that own nothing: the worker count and device their zero contributions must have."""
    _peer["W"], _peer["device"] = W, device


def _peer_shape(group):
    if "W" not in _peer:
        raise RuntimeError("a rank without tensors must call set_peer_shape(W, device) first")
    return _peer["W"], _peer["device"]


class GpuShardRunner:
    """Rank-local work of `sharded_round` on the CUDA library: a plan over the rank's tensors, marked as a shard of the
    whole stream, its buffers, and the rank's slices of the workers' gradients (the same values the unsplit workload
    has at those offsets).  world = 1 gives the plain single-GPU round."""

    def __init__(self, work, spec: ShardSpec, device, flags=None, grads: Optional[list] = None):
        from . import binding as dblp
        from . import workloads as wl
        self.dblp, self.work, self.spec, self.device = dblp, work, spec, device
        self.W = work.W
        self.flags = dblp.DBLP_MEAN if flags is None else flags
        self.plan = dblp.Plan(spec.numel, work.dtype, work.payload_bytes, work.W)
        if spec.world > 1:
            self.plan.set_shard(spec.stream_chunks, spec.seq_offset)
        self.buf = self.plan.alloc_round(device)
        self.grads = grads if grads is not None else wl.make_grads(work, device, elem_range=(spec.elem_lo, spec.elem_hi))
        self.model = dblp.loss_model(work.loss.kind, **work.loss.thresholds(spec.stream_chunks))

    def round(self, rnd, bound_ppm, marks=None):
        self.dblp.dblp_round_device(self.plan, self.grads, self.model, self.work.seed, rnd, bound_ppm, self.flags,
                                    self.buf, marks)
        return self.buf["agg"], self.buf["recv_cnt"], self.buf["missing_cnt"]

    def close(self):
        self.plan.close()
        self.buf = self.grads = None
