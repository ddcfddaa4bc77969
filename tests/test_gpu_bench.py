"""The bench's own record on a GPU: one short run of `bench.measure` per case, checked for the keys of the output
contract, for the check of the last timed round against the CPU oracle, for the launch count, and -- with a stand-in
for the process group -- for the byte accounting of the split server (every rank of a world of 2 and 3 in turn on the
one device; the collectives themselves are covered by the gloo tests)."""
import argparse
import os
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2605_01989_b200 import workloads as wl  # noqa: E402

pytestmark = pytest.mark.gpu


class OneProcessJob:
    """What bench.Job offers, for rank `rank` of `world` without a process group: reductions over ranks see one rank."""

    def __init__(self, rank=0, world=1):
        self.rank, self.world, self.local, self.dev, self.dist = rank, world, 0, "cuda:0", None
        self.args = argparse.Namespace(no_verify=False, no_e2e=False, e2e_steps=3, extras=False)
        torch.cuda.set_device(0)

    def barrier(self):
        pass

    def max_over_ranks(self, x):
        return x

    def sum_over_ranks(self, x):
        return x


def test_record_of_a_small_workload_has_the_contract_keys_and_is_verified():
    rec, work, bytes_all = bench.measure(OneProcessJob(), "flat", steps=5, warmup=3, full=True)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "vs_baseline",
                "dtype", "data", "config", "roofline", "clocks", "gpu_launches", "e2e", "verified", "step_GBps"):
        assert key in rec, key
    assert "scaling" not in rec                                   # one GPU: nothing scales
    assert rec["config"]["workload"] == work.name == "flat-1M-f32" and rec["dtype"] == "f32" and rec["vs_baseline"] is None
    assert rec["verified"]["ok"] and all(rec["verified"]["checks"].values())
    assert rec["gpu_launches"] == 5 * 10                          # pointwise loss model: ten kernels per round (one of them the round reset)
    roof = rec["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["achieved"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-12
    assert abs(roof["achieved"] - roof["algorithmic_bytes_per_launch"] / roof["ms_per_launch"] / 1e6) < 1e-6 * roof["achieved"]
    assert rec["value"] > 0 and abs(rec["value"] - bytes_all["aggregate_path"] / rec["aggregate_path"]["ms"] / 1e6) < 1e-6 * rec["value"]
    e2e = rec["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] == work.W * work.N * 4 and e2e["d2h_bytes_per_step"] > work.N * 4
    assert e2e["value"] < rec["value"]                            # the copies are inside its timed region


def test_traffic_carries_its_provenance():
    rec, work, _ = bench.measure(OneProcessJob(), "resnet50", steps=3, warmup=3, full=False)
    roof = rec["roofline"]
    assert roof["kernel"] == "k_reduce_tiled<4, 8, 1, false>"
    if roof["traffic"] is not None:
        src = roof["traffic_source"]
        assert os.path.exists(os.path.join(ROOT, src["source"])) and src["commit"] and src["captured_on"]
        assert abs(roof["traffic"] - src["dram_bytes_per_algorithmic_byte"] * roof["algorithmic_bytes_per_launch"]) < 1.0
    assert rec["verified"]["ok"]


@pytest.mark.parametrize("world", [2, 3])
def test_split_server_accounting_adds_up_to_the_unsplit_round(world):
    whole, work, bytes_whole = bench.measure(OneProcessJob(), "resnet50", steps=2, warmup=3, full=False)
    elements, sums = 0, {}
    for rank in range(world):
        rec, _, bytes_rank = bench.measure(OneProcessJob(rank, world), "resnet50", steps=2, warmup=3, full=False)
        assert rec["scaling"] == "strong" and rec["n_gpus"] == world and rec["verified"] is None
        assert rec["per_rank"]["rank"] == rank and "aggregate_path_with_exchange" in rec["stage_ms"]
        elements += rec["per_rank"]["elements"]
        for k, v in bytes_rank.items():
            sums[k] = sums.get(k, 0) + v
    assert elements == work.N
    # the same rounds (100, 101) draw the same packet fates on the split server, so the byte counts agree exactly
    # where they count packets and elements; the bitmap words are rounded up per shard
    for k in ("packetize", "reduce"):
        assert sums[k] == bytes_whole[k], k
    for k in ("apply_loss", "book", "check_bound"):
        assert 0 <= sums[k] - bytes_whole[k] <= 64 * world * work.W, k
