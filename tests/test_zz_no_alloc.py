"""The allocation-free variant of apply_loss (scratch inside the library instead of a caller workspace) must give
exactly what the ordinary entry point gives.  It serves callers that cannot allocate device memory -- code inside a
memory pool that forbids side allocations, plug-ins in a process whose device memory belongs to another runtime,
latency-critical loops -- so the test also checks that an oversized plan is refused with a clear message rather than
served from memory the library does not have.  Collected last on purpose: a failure here cannot hide the other tests
from a run that stops at the first failure."""
import pytest
import torch

from paper_2605_01989_b200 import binding as dblp
from paper_2605_01989_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _round_both_ways(work, rnd, attempt):
    plan = dblp.Plan(work.numel, work.dtype, work.payload_bytes, work.W)
    assert plan.workspace_bytes <= dblp.STATIC_SCRATCH_BYTES
    model = dblp.loss_model(work.loss.kind, **work.loss.thresholds(plan.C))
    a, b = plan.alloc_round(DEV), plan.alloc_round(DEV)
    b["delivered_bits"].fill_(-1)
    b["arrival"].fill_(-1)
    b["n_arrived"].fill_(-1)
    dblp.dblp_apply_loss(plan, model, work.seed, rnd, attempt, a["delivered_bits"], a["arrival"], a["n_arrived"], a["ws"])
    dblp.dblp_apply_loss_static(plan, model, work.seed, rnd, attempt, b["delivered_bits"], b["arrival"], b["n_arrived"])
    torch.cuda.synchronize()
    n = int(a["n_arrived"].item())
    assert int(b["n_arrived"].item()) == n and 0 < n <= plan.M
    assert torch.equal(a["delivered_bits"], b["delivered_bits"])
    assert torch.equal(a["arrival"][:n], b["arrival"][:n])
    plan.close()
    return n


def test_static_scratch_variant_matches_on_two_calls_in_a_row():
    torch.cuda.set_device(0)
    # two different plans back to back, so the second call finds the first call's leftovers in the shared scratch
    big = wl.Workload("a", 8, "f32", 1408, [352 * 20000, 1000, 7, 353], 1e-3, wl.LossSpec("ge", 0.1, 8.0), seed=5)
    small = wl.Workload("b", 3, "bf16", 4096, [2048 * 70, 5, 4099], 1e-3,
                        wl.LossSpec("microburst", window_frac=0.3, p_in=0.5, p_out=0.02), seed=6)
    n1 = _round_both_ways(big, rnd=1, attempt=0)
    n2 = _round_both_ways(small, rnd=2, attempt=1)
    n3 = _round_both_ways(big, rnd=3, attempt=0)
    assert n1 != n3 and n2 < n1


def test_static_scratch_variant_refuses_plans_beyond_its_limit():
    torch.cuda.set_device(0)
    plan = dblp.Plan([256 * (1 << 19)], "f32", 1024, 4)          # 2^21 packets: twice what the built-in scratch holds
    assert plan.workspace_bytes > dblp.STATIC_SCRATCH_BYTES
    buf = {"d": torch.zeros(plan.W * plan.row_words, dtype=torch.int32, device=DEV),
           "a": torch.zeros(plan.M, dtype=torch.int32, device=DEV), "n": torch.zeros(1, dtype=torch.int64, device=DEV)}
    with pytest.raises(dblp.DblpError) as e:
        dblp.dblp_apply_loss_static(plan, dblp.loss_model("none"), 1, 1, 0, buf["d"], buf["a"], buf["n"])
    assert e.value.status == -3 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    plan.close()
