"""The split server on CPU: gloo ranks run the product's `shard.sharded_round` with the CPU oracle standing in for the
rank-local work, under every loss process, and the stitched result (full aggregate, summed counts, per-worker
decisions) is compared with ONE unsplit round of the oracle.  That pins the partition, the stream-wide packet
numbering of the loss draws, the count exchange, the decision rule and the gather of the aggregate ranges."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_01989_b200 import shard
from paper_2605_01989_b200 import workloads as wl

NUMEL = [1000, 7, 352 * 40, 353, 100003, 2, 352 * 9, 50000]
W, P, ES = 3, 1408, 4
E = P // ES
SEED, ROUND, BOUND = 77, 4, 100000
LOSSES = {"iid": wl.LossSpec("iid", 0.1), "ge": wl.LossSpec("ge", 0.1, 6.0),
          "microburst": wl.LossSpec("microburst", window_frac=0.3, p_in=0.5, p_out=0.02), "none": wl.LossSpec("none")}


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


def test_shard_specs_tile_the_stream():
    for world in (1, 2, 3, 5, 8, 11):
        specs = shard.shard_specs(NUMEL, E, world)
        total_c = sum(-(-n // E) for n in NUMEL)
        assert specs[0].seq_offset == 0 and specs[0].elem_lo == 0 and specs[-1].elem_hi == sum(NUMEL)
        for a, b in zip(specs, specs[1:]):
            assert a.seq_offset + a.chunks == b.seq_offset and a.elem_hi == b.elem_lo and a.tensor_hi == b.tensor_lo
        assert specs[-1].seq_offset + specs[-1].chunks == total_c and all(s.stream_chunks == total_c for s in specs)
        assert [n for s in specs for n in s.numel] == NUMEL


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _columns(bits, lo, n):
    """Columns lo .. lo + n - 1 of a (rows, words) little-endian bitmap, as a bitmap of ceil(n / 32) words."""
    rows = np.unpackbits(bits.view(np.uint8).reshape(bits.shape[0], -1), axis=1, bitorder="little")[:, lo:lo + n]
    pad = (-n) % 32
    rows = np.pad(rows, ((0, 0), (0, pad)))
    return np.packbits(rows, axis=1, bitorder="little").view(np.uint32).reshape(bits.shape[0], -1)


def _full_grads():
    rng = np.random.default_rng(5)
    return [(rng.standard_normal(sum(NUMEL)) * 1e-3).astype(np.float32) for _ in range(W)]


class OracleShardRunner:
    """The rank-local round, by the oracle: the delivered bitmap is the rank's columns of the stream-wide loss mask
    (what dblp_plan_set_shard makes the CUDA library draw), the arrival order is the shard's own permutation."""

    def __init__(self, spec, loss):
        from oracle import dblp_oracle as orc
        self.orc, self.spec, self.W = orc, spec, W
        self.op = orc.Plan(spec.numel, ES, P, W)
        self.mine = [np.ascontiguousarray(g[spec.elem_lo:spec.elem_hi]) for g in _full_grads()]
        self.stream = orc.Plan(NUMEL, ES, P, W)
        self.model = orc.loss_model(loss.kind, **loss.thresholds(spec.stream_chunks))

    def round(self, rnd, bound_ppm, marks=None):
        op = self.op
        hdr, pay = op.packetize(self.mine, rnd)
        whole, _ = self.stream.loss_mask(self.model, SEED, rnd)
        d = _columns(whole, self.spec.seq_offset, self.spec.chunks)
        arr, n = op.arrival(d, SEED, rnd)
        st = op.book(hdr, arr, n, rnd, op.new_state())
        agg = op.reduce(pay, st, mean=True)
        recv, miss, _, _ = op.check_bound(st["bitmap"], bound_ppm)
        return (torch.from_numpy(agg), torch.from_numpy(recv[:, 0].astype(np.int64)),
                torch.from_numpy(miss[:, 0].astype(np.int64)))


def _rank(rank, world, port, out, kind):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2605_01989_b200 import binding
        specs = shard.shard_specs(NUMEL, E, world)
        shard.set_peer_shape(W, "cpu")
        runner = None if specs[rank].empty else OracleShardRunner(specs[rank], LOSSES[kind])
        res = shard.sharded_round(runner, specs, ROUND, BOUND, gather=True)
        ok, all_ok = shard.decision(res, binding.dblp_bound_ok, BOUND)
        gathered = [None] * world
        dist.all_gather_object(gathered, {"recv": res["recv"].tolist(), "missing": res["missing"].tolist(),
                                          "ok": ok, "all_ok": all_ok, "agg": res["agg"].numpy()})
        if rank == 0:
            torch.save(gathered, out)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("kind,world", [("iid", 2), ("ge", 2), ("microburst", 2), ("none", 2), ("ge", 3)])
def test_split_server_equals_the_unsplit_round(tmp_path, kind, world):
    from oracle import dblp_oracle as orc
    from paper_2605_01989_b200 import build as b
    b.build()
    out = str(tmp_path / "g.pt")
    mp.start_processes(_rank, args=(world, _free_port(), out, kind), nprocs=world, join=True, start_method="spawn")
    g = torch.load(out, weights_only=False)
    for r in range(1, world):                                        # every rank ends with the same totals, decision
        for k in ("recv", "missing", "ok", "all_ok"):                # and full aggregate
            assert g[0][k] == g[r][k]
        assert g[0]["agg"].tobytes() == g[r]["agg"].tobytes()
    # one unsplit round of the oracle
    op = orc.Plan(NUMEL, ES, P, W)
    loss = LOSSES[kind]
    model = orc.loss_model(loss.kind, **loss.thresholds(op.C))
    hdr, pay = op.packetize(_full_grads(), ROUND)
    d, _ = op.loss_mask(model, SEED, ROUND)
    arr, n = op.arrival(d, SEED, ROUND)
    st = op.book(hdr, arr, n, ROUND, op.new_state())
    recv, miss, ok, all_ok = op.check_bound(st["bitmap"], BOUND)
    assert g[0]["recv"] == recv[:, 0].tolist() and g[0]["missing"] == miss[:, 0].tolist()
    assert g[0]["ok"] == ok[:, 0].tolist() and g[0]["all_ok"] == all_ok
    assert g[0]["agg"].tobytes() == op.reduce(pay, st, mean=True).tobytes()
    if kind != "none":
        assert 0 < sum(g[0]["missing"]) < W * op.C                  # the comparison is not vacuous


def test_more_ranks_than_tensors_leaves_some_ranks_empty(tmp_path):
    """Ranks that own nothing still join the collectives (with zeros) and reach the same decision."""
    global NUMEL
    out = str(tmp_path / "g.pt")
    mp.start_processes(_rank_few, args=(3, _free_port(), out), nprocs=3, join=True, start_method="spawn")
    g = torch.load(out, weights_only=False)
    assert g[0]["ok"] == g[1]["ok"] == g[2]["ok"] and len(g[0]["agg"]) == 7000


def _rank_few(rank, world, port, out):
    global NUMEL
    NUMEL = [5000, 2000]                                              # two tensors, three ranks
    _rank(rank, world, port, out, "iid")
