"""The multi-GPU host logic on CPU: two gloo ranks, each a server shard that owns a run of tensors.  The shards'
per-worker counts are summed with the product's exchange, the decision is taken with the library's host rule, and
everything is compared with one unsharded round of the CPU oracle."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_01989_b200 import shard

NUMEL = [1000, 7, 352 * 40, 353, 100003, 2, 352 * 9, 50000]
W, P, ES = 3, 1408, 4


def test_partition_covers_every_tensor_once_and_balances():
    for world in (1, 2, 3, 4, 8, 16):
        parts = shard.partition_tensors(NUMEL, world)
        assert len(parts) == world and parts[0][0] == 0 and parts[-1][1] == len(NUMEL)
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:])) and all(lo <= hi for lo, hi in parts)
        offs = shard.shard_offsets(NUMEL, parts)
        assert offs[0][0] == 0 and offs[-1][1] == sum(NUMEL)
    sizes = [b - a for a, b in shard.shard_offsets([10] * 100, shard.partition_tensors([10] * 100, 4))]
    assert sizes == [250] * 4
    assert shard.partition_tensors([1000, 1, 1, 1, 1000], 2) == [(0, 2), (2, 5)]      # total 2003: prefix 1001 is nearest to the half
    assert shard.partition_tensors([5, 5], 4) == [(0, 0), (0, 1), (1, 1), (1, 2)]      # fewer tensors than ranks


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import dblp_oracle as orc
        from paper_2605_01989_b200 import binding
        lo, hi = shard.partition_tensors(NUMEL, world)[rank]
        first, last = shard.shard_offsets(NUMEL, shard.partition_tensors(NUMEL, world))[rank]
        rng = np.random.default_rng(5)
        full = [(rng.standard_normal(sum(NUMEL)) * 1e-3).astype(np.float32) for _ in range(W)]
        mine = [np.ascontiguousarray(g[first:last]) for g in full]
        op = orc.Plan(NUMEL[lo:hi], ES, P, W)
        hdr, pay = op.packetize(mine, 1)
        model = orc.loss_model("iid", t_drop=int(0.1 * 2 ** 32))
        d, _ = op.loss_mask(model, 100 + rank, 1)
        arr, n = op.arrival(d, 100 + rank, 1)
        st = op.book(hdr, arr, n, 1, op.new_state())
        recv, miss, ok, _ = op.check_bound(st["bitmap"], 100000)
        r, m = shard.exchange_counts(torch.from_numpy(recv.astype(np.int64)), torch.from_numpy(miss.astype(np.int64)))
        oks, all_ok = shard.decide(binding.dblp_bound_ok, r, m, 100000)
        # zero-loss aggregate of the shard, to be stitched by the parent
        st0 = op.book(hdr, np.arange(op.M, dtype=np.uint32), op.M, 1, op.new_state())
        agg = op.reduce(pay, st0)
        gathered = [None] * world
        dist.all_gather_object(gathered, {"recv": recv[:, 0].tolist(), "miss": miss[:, 0].tolist(), "C": op.C,
                                          "agg": agg, "sum_recv": r.flatten().tolist(), "sum_miss": m.flatten().tolist(),
                                          "oks": oks, "all_ok": all_ok})
        if rank == 0:
            torch.save(gathered, out)
    finally:
        dist.destroy_process_group()


def test_two_ranks_sum_their_counts_and_agree_on_the_decision(tmp_path):
    from oracle import dblp_oracle as orc
    from paper_2605_01989_b200 import build as b
    b.build()
    out = str(tmp_path / "g.pt")
    mp.start_processes(_rank, args=(2, _free_port(), out), nprocs=2, join=True, start_method="spawn")
    g = torch.load(out, weights_only=False)
    for k in ("sum_recv", "sum_miss", "oks", "all_ok"):
        assert g[0][k] == g[1][k]                                   # every rank ends with the same totals and decision
    assert g[0]["sum_recv"] == [a + b_ for a, b_ in zip(g[0]["recv"], g[1]["recv"])]
    assert g[0]["sum_miss"] == [a + b_ for a, b_ in zip(g[0]["miss"], g[1]["miss"])]
    total_c = g[0]["C"] + g[1]["C"]
    assert all(r + m == total_c for r, m in zip(g[0]["sum_recv"], g[0]["sum_miss"]))
    assert g[0]["oks"] == [int(m * 1000000 <= 100000 * total_c) for m in g[0]["sum_miss"]]
    # stitched zero-loss aggregates of the shards = unsharded oracle sum
    rng = np.random.default_rng(5)
    full = [(rng.standard_normal(sum(NUMEL)) * 1e-3).astype(np.float32) for _ in range(W)]
    op = orc.Plan(NUMEL, ES, P, W)
    hdr, pay = op.packetize(full, 1)
    st = op.book(hdr, np.arange(op.M, dtype=np.uint32), op.M, 1, op.new_state())
    assert op.C == total_c
    assert np.concatenate([g[0]["agg"], g[1]["agg"]]).tobytes() == op.reduce(pay, st).tobytes()
