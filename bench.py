#!/usr/bin/env python
"""Throughput of the DBLP receive path on synthetic gradients.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload gpt2xl|bert|resnet50|flat|sweep] [--impl reference]

One step = one communication round through the library's whole-round call (dblp_round_device): round_reset,
packetize, apply_loss, aggregate (bookkeeping + masked reduce) and check_bound on gradients already resident in device
memory, in the library's two-stream schedule.

The metric is the bounded-loss aggregate rate: algorithmic bytes read plus written by the aggregate path (bookkeeping,
masked reduce, tolerance test) divided by the time of that path inside the step, in GB/s.  `ms_per_step` is the whole
step and `step_GBps` the whole step's bytes over it.  With no --workload the headline is the GPT-2-XL-shaped workload
(the largest that fits one GPU) and `per_config` carries the ResNet-50- and BERT-large-shaped ones.  Prints one JSON
line.

With --impl reference the same round is run by the plain CPU checker on the host cores (a reported baseline).
Under torchrun (N > 1) the server is split by offset range over the ranks (strong scaling): every rank runs the round
on its own run of tensors, the per-worker loss counts are summed over the ranks and the aggregate ranges all-gathered.
"""
import argparse
import copy
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_01989_b200 import workloads as wl  # noqa: E402

METRIC = "bounded-loss aggregate GB/s (bytes read+written)"
WORKLOADS = {"flat": 0, "resnet50": 1, "bert": 2, "gpt2xl": 3, "sweep": 4}
HEADLINE, PER_CONFIG = "gpt2xl", ("resnet50", "bert")
DEFAULT_STEPS = {"flat": 2000, "resnet50": 500, "bert": 100, "gpt2xl": 40, "sweep": 300}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (read + write) that ncu counted for one launch of the reduce kernel, as a ratio to that launch's
# algorithmic bytes.  The ResNet-50-shaped workload was captured itself; the two large ones are too big to capture, so
# their ratio comes from a point of the size sweep that runs the same kernel with the same payload size on about 2 GB,
# and `traffic` scales it to the launch timed here (traffic grows in proportion to the bytes moved).  `commit` is the
# revision of the kernels the counters were taken on: an entry is removed whenever its kernel changes.
NCU_TRAFFIC = {
    "resnet50-f32": {"kernel": "k_reduce_tiled<4, 8, 1, false>", "dram_bytes_per_algorithmic_byte": 0.969,
                     "captured_on": "resnet50-f32", "commit": "5ca6832", "source": "profiles/k_reduce_tiled_resnet50.md"},
    "bert-large-bf16": {"kernel": "k_reduce_tiled<2, 8, 1, false>", "dram_bytes_per_algorithmic_byte": 0.956,
                        "captured_on": "point:bf16:64:16:4096", "commit": "ffeeae1",
                        "source": "profiles/k_reduce_tiled_sweep_points_bf16_f32.md"},
    "gpt2-xl-f32": {"kernel": "k_reduce_tiled<4, 8, 1, false>", "dram_bytes_per_algorithmic_byte": 0.978,
                    "captured_on": "point:f32:128:8:4096", "commit": "5ca6832",
                    "source": "profiles/k_reduce_tiled_sweep_points_bf16_f32.md"},
}


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def byte_model(W, N, s, C, n_arrived, payload_recv_bytes):
    """Algorithmic bytes of each stage for one round (what the method has to move, not what a kernel happens to)."""
    M, R = W * C, n_arrived
    stages = {
        "packetize": 2 * W * N * s + 32 * M,                       # read gradients, write payloads + headers
        "apply_loss": M // 8 + 4 * R,                              # delivered bitmap + arrival list
        "book": (4 + 32) * R + 4 * R + M // 8,                     # arrival entry + header per packet, slot entry, bitmap
        "reduce": payload_recv_bytes + 4 * N + 4 * M + 8 * C,      # received payloads, aggregate, slot entries, chunk table
        "check_bound": M // 8,
    }
    stages["aggregate_path"] = stages["book"] + stages["reduce"] + stages["check_bound"]
    stages["total"] = stages["packetize"] + stages["apply_loss"] + stages["aggregate_path"]
    return stages


def chunk_lengths(numel, E):
    return np.concatenate([np.minimum(E, n - np.arange(-(-n // E), dtype=np.int64) * E) for n in numel])


def workload_by_name(name):
    """A named workload, or one point of the size sweep written as point:DTYPE:MiB:W:PAYLOAD (for instance
    point:bf16:64:16:4096 = 16 workers with 64 MiB of bf16 each in 4096-byte packets, 5 % bursty loss, seed 10): the
    bounded cases that profiler captures run on."""
    if name.startswith("point:"):
        _, dtype, mib, W, P = name.split(":")
        work = wl.sweep_point(int(mib) << 20, int(W), int(P), 0.05, "ge", 10)
        if dtype == "bf16":                                   # same bytes per worker, twice the elements
            work.dtype, work.numel = "bf16", [2 * work.numel[0]]
        elif dtype != "f32":
            raise SystemExit("point: dtype must be f32 or bf16")
        work.name = name
        work.bounds_ppm = (80000,)
        return work
    return wl.config(WORKLOADS[name])


def reduce_kernel_name(work):
    W, es = work.W, work.elem_size
    if W > 6000:
        return "k_reduce<%d>" % es
    wb, j = (1, 8) if W == 1 else (2, 4) if W <= 2 else (4, 2) if W <= 4 else (8, 1)
    kind = "k_reduce_rows" if W <= 4 and work.payload_bytes >= 2048 else "k_reduce_tiled"
    return "%s<%d, %d, %d, false>" % (kind, es, wb, j)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:                                   # the device CUDA uses, by UUID; NVML's numbering may differ
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap", nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown"}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                break
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ----------------------------------------------------------------------------------------------------------------------
class Job:
    """Process-wide state of a GPU run: rank, world, device, process group."""

    def __init__(self):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dev = "cuda:%d" % self.local
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device(self.dev))
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, x):
        if self.dist is None:
            return x
        t = torch.tensor([x], device=self.dev, dtype=torch.float64)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, x):
        if self.dist is None:
            return x
        t = torch.tensor([x], device=self.dev, dtype=torch.float64)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return float(t.item())


def measure(job, name, steps, warmup, full):
    """Times `steps` rounds of workload `name` (after `warmup` untimed ones) and returns its record.  `full` adds the
    legs that only the headline carries: end to end from host buffers, and the CPU baseline."""
    from paper_2605_01989_b200 import binding as dblp
    from paper_2605_01989_b200 import shard
    dev, world, rank = job.dev, job.world, job.rank
    work = workload_by_name(name)
    specs = shard.shard_specs(work.numel, work.E, world)
    spec = specs[rank]
    bound = work.bounds_ppm[-1] if name == "gpt2xl" else work.bounds_ppm[0]
    shard.set_peer_shape(work.W, dev)
    n_local = spec.elem_hi - spec.elem_lo
    runner = None
    if not spec.empty:
        # one contiguous buffer for all workers' gradients: the end-to-end leg copies into the same memory
        grads_dev = torch.empty(work.W * n_local, dtype=torch.float32 if work.dtype == "f32" else torch.bfloat16, device=dev)
        grads = wl.make_grads(work, dev, elem_range=(spec.elem_lo, spec.elem_hi) if world > 1 else None, out=grads_dev)
        runner = shard.GpuShardRunner(work, spec, dev, grads=grads)
        runner.grads_dev = grads_dev
    torch.cuda.synchronize()

    exchanged = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]

    def step(rnd, marks=None, k=None):
        res = shard.sharded_round(runner, specs, rnd, bound, gather=world > 1, marks=marks)
        if k is not None:
            exchanged[k].record()
        return res

    for i in range(warmup):
        step(1 + i)
    torch.cuda.synchronize()
    job.barrier()

    marks = [dblp.RoundMarks() for _ in range(steps)] if runner is not None else [None] * steps
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(job.local))
    launches0 = dblp.dblp_launch_count()
    torch.cuda.synchronize()
    job.barrier()
    sampler.start()
    t_begin.record()
    for k in range(steps):
        last = step(100 + k, marks[k], k)
    t_end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = dblp.dblp_launch_count() - launches0
    job.barrier()
    last_round = 100 + steps - 1
    ms_step = job.max_over_ranks(t_begin.elapsed_time(t_end)) / steps

    # realised loss of the last round -> algorithmic bytes of this rank's shard
    if runner is not None:
        plan, buf = runner.plan, runner.buf
        n_arrived = int(buf["n_arrived"].item())
        bm = buf["recv_bitmap"].cpu().numpy().view("uint32").reshape(plan.W, plan.row_words)
        bits = np.unpackbits(bm.view(np.uint8), axis=1, bitorder="little")[:, :plan.C]
        payload_recv = int((bits.astype(np.int64) * chunk_lengths(spec.numel, work.E)[None, :]).sum()) * work.elem_size
        mine = byte_model(work.W, n_local, work.elem_size, plan.C, n_arrived, payload_recv)
        stage = lambda a, b: sum(m.ms(a, b) for m in marks) / steps                                  # noqa: E731
        stage_ms = {"packetize": stage("begin", "packetize_end"), "apply_loss": stage("loss_begin", "loss_end"),
                    "book": stage("receive_begin", "claim_end"), "reduce": stage("claim_end", "reduce_end"),
                    "check_bound": stage("bound_begin", "bound_end"), "aggregate_path": stage("receive_begin", "end")}
        if world > 1:                                        # the split server's aggregate path ends with its exchanges
            stage_ms["aggregate_path_with_exchange"] = sum(
                m.events["receive_begin"].elapsed_time(e) for m, e in zip(marks, exchanged)) / steps
    else:
        mine = byte_model(work.W, 0, work.elem_size, 0, 0, 0)
        stage_ms = {k: 0.0 for k in ("packetize", "apply_loss", "book", "reduce", "check_bound", "aggregate_path")}
        n_arrived = 0
    bytes_all = {k: int(job.sum_over_ranks(v)) for k, v in mine.items()}
    agg_key = "aggregate_path_with_exchange" if world > 1 else "aggregate_path"
    agg_ms = job.max_over_ranks(stage_ms[agg_key])
    arrived_all = job.sum_over_ranks(n_arrived)

    verified = None
    if world == 1 and not job.args.no_verify:
        verified = verify_last_round(work, runner, last_round, bound, last)

    peak, peak_kind = measured_peak()
    red_gbs = mine["reduce"] / stage_ms["reduce"] / 1e6 if stage_ms["reduce"] else 0.0
    agg_gbs = bytes_all["aggregate_path"] / agg_ms / 1e6
    kernel = reduce_kernel_name(work)
    ncu = NCU_TRAFFIC.get(work.name) if world == 1 else None
    if ncu is not None and ncu["kernel"] != kernel:
        ncu = None
    rec = {
        "metric": METRIC, "value": agg_gbs, "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "vs_baseline": None, "dtype": work.dtype, "data": "synthetic",
        "config": {"workload": work.name, "W": work.W, "payload_bytes": work.payload_bytes, "tensors": len(work.numel),
                   "elements_per_worker": work.N, "packets": work.W * specs[0].stream_chunks, "loss": work.loss.kind,
                   "realised_loss": 1.0 - arrived_all / (work.W * specs[0].stream_chunks), "bound_ppm": bound,
                   "reduce": "mean, fixed worker order", "launch": "dblp_round_device, eager",
                   "streams": "the library's schedule: apply_loss beside packetize, bitmap + check_bound beside the reduce, on the plan's high-priority stream",
                   "l2": "inputs per step (%.0f MB) exceed the 126 MB L2; no flush" % (bytes_all["total"] / 1e6)
                         if bytes_all["total"] > 4 * 126e6 else
                         "inputs per step (%.0f MB) do not exceed the L2 by much: L2-resident, launch-bound" % (bytes_all["total"] / 1e6),
                   "parallelism": "server split by offset range over %d GPUs" % world if world > 1 else "1 GPU"},
        "value_is": "aggregate path (bookkeeping + masked reduce + tolerance test): its bytes / its time inside the step",
        "pct_of_nominal_8TBs": 100.0 * agg_gbs / NOMINAL_HBM_GBS / world,
        "pct_of_%s_peak" % peak_kind: 100.0 * agg_gbs / peak / world,
        "step_GBps": bytes_all["total"] / ms_step / 1e6,
        "bytes_per_step": bytes_all, "stage_ms": stage_ms,
        "aggregate_path": {"what": "bookkeeping + masked reduce + bound check only", "GBps": agg_gbs, "ms": agg_ms,
                           "pct_of_nominal_8TBs": 100.0 * agg_gbs / NOMINAL_HBM_GBS / world,
                           "pct_of_%s_peak" % peak_kind: 100.0 * agg_gbs / peak / world},
        "roofline": {"kernel": kernel, "bound": "hbm", "achieved": red_gbs, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": red_gbs / peak,
                     "traffic": ncu["dram_bytes_per_algorithmic_byte"] * mine["reduce"] if ncu else None,
                     "traffic_source": {k: ncu[k] for k in ("source", "captured_on", "commit", "dram_bytes_per_algorithmic_byte")}
                     if ncu else None,
                     "algorithmic_bytes_per_launch": mine["reduce"], "ms_per_launch": stage_ms["reduce"]},
        "clocks": clocks, "gpu_launches": launches, "verified": verified,
    }
    if world > 1:
        rec["scaling"] = "strong"
        rec["per_rank"] = {"rank": rank, "elements": n_local, "bytes_per_step": mine}

    if full:
        rec["e2e"] = end_to_end(job, work, runner, bound, mine, steps) if not job.args.no_e2e else None
        if rank == 0 and world == 1 and job.args.extras:
            rec["round_loop"], rec["reduce_extras"] = side_sections(work, runner, bound)
    if runner is not None:
        runner.close()
        del grads, grads_dev
    torch.cuda.empty_cache()
    return rec, work, bytes_all


def verify_last_round(work, runner, rnd, bound, result):
    """Outside the timed region: the state the last timed round left on the device against the CPU checker -- arrival
    count, received bitmap, all counters, the tolerance outputs, and a sample of aggregate elements (random ones, both
    ends of every tensor, every tensor's short last chunk)."""
    from oracle import dblp_oracle as orc
    from paper_2605_01989_b200 import binding as dblp
    t0 = time.perf_counter()
    plan, buf = runner.plan, runner.buf
    op = orc.Plan(work.numel, work.elem_size, work.payload_bytes, work.W)
    om = orc.loss_model(work.loss.kind, **work.loss.thresholds(op.C))
    o_del, _ = op.loss_mask(om, work.seed, rnd)
    o_arr, o_n = op.arrival(o_del, work.seed, rnd)
    st = op.book(op.headers(rnd), o_arr, o_n, rnd, op.new_state())
    checks = {}
    checks["n_arrived"] = int(buf["n_arrived"].item()) == o_n
    checks["received_bitmap"] = buf["recv_bitmap"].cpu().numpy().view(np.uint32).tobytes() == st["bitmap"].tobytes()
    c = dblp.counters_dict(buf["counters"])
    checks["counters"] = {k: c[k] for k in dblp.COUNTER_FIELDS} == st["counters"].as_dict() and c["status"] == 0
    recv, miss, ok, all_ok = op.check_bound(st["bitmap"], bound)
    checks["bound_outputs"] = (buf["recv_cnt"].cpu().numpy().view(np.uint32).tolist() == recv[:, 0].tolist() and
                               buf["missing_cnt"].cpu().numpy().view(np.uint32).tolist() == miss[:, 0].tolist() and
                               buf["ok"].cpu().numpy().tolist() == ok[:, 0].tolist() and
                               int(buf["all_ok"].item()) == all_ok)
    from paper_2605_01989_b200 import shard
    checks["decision"] = shard.decision(result, dblp.dblp_bound_ok, bound) == (ok[:, 0].tolist(), all_ok)
    rng = np.random.default_rng(rnd)
    base, numel, E = op.base.astype(np.int64), op.numel.astype(np.int64), op.E
    tails = [np.arange(base[t] + (numel[t] // E) * E, base[t] + numel[t]) for t in range(op.T) if numel[t] % E]
    elem = np.unique(np.concatenate([rng.integers(0, op.N, 100000), base, base + numel - 1] + tails))
    idx = torch.from_numpy(elem).to(buf["agg"].device)
    vals = torch.stack([x[idx] for x in runner.grads])
    vals = vals.view(torch.int16).cpu().numpy().view(np.uint16) if work.elem_size == 2 else vals.cpu().numpy()
    want = op.reduce_at(st["bitmap"], elem, vals, mean=True)
    checks["aggregate_sample"] = buf["agg"][idx].cpu().numpy().tobytes() == want.tobytes()
    return {"ok": all(checks.values()), "checks": checks, "round": rnd, "sampled_elements": int(len(elem)),
            "seconds": time.perf_counter() - t0}


def end_to_end(job, work, runner, bound, mine, steps):
    """The same round through dblp_round_host: every step copies all workers' gradients from pinned host memory and
    reads the aggregate, the counters and the tolerance outputs back."""
    from paper_2605_01989_b200 import binding as dblp
    if runner is None:
        return None
    dev = job.dev
    plan, buf = runner.plan, runner.buf
    n_local = runner.spec.elem_hi - runner.spec.elem_lo
    dtype = runner.grads[0].dtype
    pinned = True
    try:
        grads_host = [torch.empty(n_local, dtype=dtype, pin_memory=True) for _ in range(work.W)]
        agg_host = torch.empty(n_local, dtype=torch.float32, pin_memory=True)
    except RuntimeError:
        pinned = False
        grads_host = agg_host = None
        try:
            grads_host = [torch.empty(n_local, dtype=dtype) for _ in range(work.W)]
            agg_host = torch.empty(n_local, dtype=torch.float32)
        except (RuntimeError, MemoryError) as e:       # the host cannot hold a copy of the gradients at all
            del grads_host, agg_host
            return {"value": None, "unit": "GB/s", "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                    "unavailable": "host memory for %d x %d bytes of gradients: %s" % (work.W, n_local * work.elem_size,
                                                                                       str(e)[:160])}
    for h, g in zip(grads_host, runner.grads):
        h.copy_(g)
    grads_dev = runner.grads_dev                  # the workers' gradients back to back: the copies land where they already are
    cnt_host = torch.zeros(7, dtype=torch.int64).pin_memory()
    small = [torch.zeros(work.W, dtype=torch.int32).pin_memory() for _ in range(2)]
    ok_host = torch.zeros(work.W, dtype=torch.uint8).pin_memory()
    all_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    h2d = work.W * n_local * work.elem_size
    Ke = max(3, min(steps, job.args.e2e_steps, int(30e9 / max(1, h2d)) + 3))      # about half a minute of copies at most

    def e2e_step(rnd):
        dblp.dblp_round_host(plan, grads_host, runner.model, work.seed, rnd, bound, dblp.DBLP_MEAN, buf, grads_dev,
                             agg_host, cnt_host, small[0], small[1], ok_host, all_host)

    for i in range(3):
        e2e_step(50 + i)
    torch.cuda.synchronize()
    job.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for k in range(Ke):
        e2e_step(100 + k)
    b.record()
    torch.cuda.synchronize()
    ms_e2e = job.max_over_ranks(a.elapsed_time(b) / Ke)
    agg_bytes = job.sum_over_ranks(mine["aggregate_path"])
    return {"value": agg_bytes / ms_e2e / 1e6, "unit": "GB/s", "ms_per_step": ms_e2e, "steps": Ke,
            "what": "dblp_round_host: the metric's bytes over the whole call, host-to-device copies of all gradients and "
                    "device-to-host copy of the aggregate included",
            "step_GBps": job.sum_over_ranks(mine["total"]) / ms_e2e / 1e6,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": n_local * 4 + 56 + work.W * 9 + 4, "pinned": pinned,
            "h2d_GBps": h2d / ms_e2e / 1e6}


def side_sections(work, runner, bound):
    """Untimed extras (--extras): the control loop under heavy loss (attempts until every worker passes, low against
    high tolerance: the mechanism behind the paper's latency tables) and the reduce with its fused norm / update."""
    from paper_2605_01989_b200 import binding as dblp
    plan, buf, grads = runner.plan, runner.buf, runner.grads
    p_low, p_high = bound, bound + 400000
    round_loop = []
    dblp.dblp_packetize(plan, grads, 7, buf["hdr_ring"], buf["payload_ring"])
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for burst in (0.6, 0.7, 0.8, 0.9):
        m = dblp.loss_model("iid", t_drop=wl.threshold(burst))
        row = {"loss": burst}
        for name, ppm in (("p_low", p_low), ("p_high", p_high)):
            dblp.dblp_round_reset(plan, buf["recv_bitmap"], buf["slot_key"], buf["counters"])
            a.record()
            attempts, ok = dblp.dblp_round_until_stop(plan, m, work.seed, 7, ppm, 400, True, buf)
            b.record()
            torch.cuda.synchronize()
            row[name] = {"ppm": ppm, "attempts": attempts, "all_ok": ok, "ms": a.elapsed_time(b)}
        row["attempt_ratio"] = row["p_low"]["attempts"] / max(1, row["p_high"]["attempts"])
        round_loop.append(row)

    dblp.dblp_round_device(plan, grads, runner.model, work.seed, 7, bound, dblp.DBLP_MEAN, buf)
    dev = buf["agg"].device
    scratch = torch.empty(max(1, dblp.dblp_norm_scratch_count(plan)), dtype=torch.float64, device=dev)
    norm_out = torch.zeros(2, dtype=torch.float64, device=dev)
    params = torch.zeros(plan.N, dtype=torch.float32, device=dev)

    def timed(fn, reps=20):
        for _ in range(3):
            fn()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    ring, keys, agg = buf["payload_ring"], buf["slot_key"], buf["agg"]
    extras = {
        "reduce_ms": timed(lambda: dblp.dblp_aggregate_reduce(plan, ring, keys, agg, dblp.DBLP_MEAN)),
        "reduce_norm_ms": timed(lambda: dblp.dblp_aggregate_reduce_ex(plan, ring, keys, agg, dblp.DBLP_MEAN, scratch, norm_out)),
        "reduce_norm_update_ms": timed(lambda: dblp.dblp_aggregate_reduce_ex(plan, ring, keys, agg, dblp.DBLP_MEAN, scratch,
                                                                             norm_out, params, 0.01)),
        "reduce_atomic_order_free_ms": timed(lambda: dblp.dblp_aggregate_reduce_atomic(plan, ring, keys, agg, dblp.DBLP_MEAN)),
        "grad_norm": float(norm_out[1].item()),
    }
    return round_loop, extras


def run_gpu(args):
    job = Job()
    job.args = args
    names = [args.workload] if args.workload else [HEADLINE] + list(PER_CONFIG)
    left_out = []
    if not args.workload:
        # the headline is the largest workload that fits in what is free on this device (a rank holds 1 / world of it)
        free, _ = torch.cuda.mem_get_info()
        need = lambda n: workload_by_name(n).device_bytes() // job.world + (4 << 30)                     # noqa: E731
        left_out = [n for n in names if need(n) > free]
        names = sorted([n for n in names if n not in left_out], key=need, reverse=True)
        if not names:
            raise SystemExit("bench.py: no workload fits in %.1f GB of free device memory" % (free / 1e9))
    # the smaller workloads run first, on a device that has held nothing large yet; names[0] is the headline
    out, others = None, []
    keep = ("value", "unit", "ms_per_step", "steps", "warmup", "dtype", "config", "pct_of_nominal_8TBs", "step_GBps",
            "bytes_per_step", "stage_ms", "aggregate_path", "roofline", "clocks", "gpu_launches", "verified")
    for name in reversed(names):
        steps = args.steps if args.steps is not None else DEFAULT_STEPS.get(name, 50)
        warmup = max(3, 5 if args.warmup is None else args.warmup)
        rec, work, bytes_all = measure(job, name, steps, warmup, full=(name == names[0]))
        if name == names[0]:
            out = rec
            if job.rank == 0 and job.world == 1 and not args.no_cpu_baseline:
                out["cpu_baseline"] = cpu_baseline(work)
        else:
            others.append({k: rec[k] for k in keep} | {k: v for k, v in rec.items() if k.startswith("pct_of_")})
    if len(names) > 1:
        out["per_config"] = others
    if left_out:
        out["config"]["left_out"] = "%s: not enough free device memory" % ", ".join(left_out)
    if job.dist is not None:
        job.barrier()
        job.dist.destroy_process_group()
    if job.rank == 0:
        print(json.dumps(out))


def run_sweep(args):
    """Stand-alone timing of packetize and of the aggregate path (bookkeeping + reduce + bound check) over the size
    sweep: per-worker buffer 1 MiB * 4^k, W in {1, 2, 8, 32}, payload {1024, 4096}, fp32 and bf16, 5 % bursty loss.
    Points that do not fit in device memory are left out.  Prints one JSON line."""
    from paper_2605_01989_b200 import binding as dblp
    torch.cuda.set_device(0)
    dev = "cuda:0"
    peak, peak_kind = measured_peak()
    rows = []
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for dtype in ("f32", "bf16"):
        for k in range(6):
            for W in (1, 2, 8, 32):
                for P in (1024, 4096):
                    if dtype == "bf16" and k % 2 == 0:
                        continue                          # bf16: every other size
                    work = wl.sweep_point((1 << 20) * 4 ** k, W, P, 0.05, "ge", 10)
                    if dtype == "bf16":                   # same bytes per worker, twice the elements
                        work.dtype = "bf16"
                        work.numel = [2 * work.numel[0]]
                    free, _ = torch.cuda.mem_get_info()
                    if work.device_bytes() + (2 << 30) > free:
                        rows.append({"dtype": dtype, "buffer_MiB": 4 ** k, "W": W, "P": P, "skipped": "does not fit"})
                        continue
                    plan = dblp.Plan(work.numel, work.dtype, work.payload_bytes, work.W)
                    buf = plan.alloc_round(dev)
                    grads = wl.make_grads(work, dev)
                    model = dblp.loss_model(work.loss.kind, **work.loss.thresholds(plan.C))
                    reps = max(3, min(50, int(2e10 / work.device_bytes())))

                    def timed(fn):
                        for _ in range(2):
                            fn()
                        a.record()
                        for _ in range(reps):
                            fn()
                        b.record()
                        torch.cuda.synchronize()
                        return a.elapsed_time(b) / reps

                    t_pack = timed(lambda: dblp.dblp_packetize(plan, grads, 1, buf["hdr_ring"], buf["payload_ring"]))
                    dblp.dblp_round_send(plan, grads, model, work.seed, 1, buf)
                    t_agg = timed(lambda: (dblp.dblp_round_reset(plan, buf["recv_bitmap"], buf["slot_key"], buf["counters"]),
                                           dblp.dblp_round_receive(plan, 1, 50000, dblp.DBLP_MEAN, buf)))
                    t_red = timed(lambda: dblp.dblp_aggregate_reduce(plan, buf["payload_ring"], buf["slot_key"], buf["agg"],
                                                                     dblp.DBLP_MEAN))
                    n = int(buf["n_arrived"].item())
                    by = byte_model(work.W, work.N, work.elem_size, plan.C, n, int(n / plan.M * work.W * work.N * work.elem_size))
                    rows.append({"dtype": dtype, "buffer_MiB": 4 ** k, "W": W, "P": P, "packets": plan.M, "loss": 1 - n / plan.M,
                                 "kernel": reduce_kernel_name(work),
                                 "packetize_GBps": by["packetize"] / t_pack / 1e6,
                                 "aggregate_path_GBps": by["aggregate_path"] / t_agg / 1e6,
                                 "reduce_GBps": by["reduce"] / t_red / 1e6,
                                 "reduce_frac_of_%s" % peak_kind: by["reduce"] / t_red / 1e6 / peak,
                                 "aggregate_path_us": t_agg * 1e3})
                    plan.close()
                    del buf, grads
                    torch.cuda.empty_cache()
    print(json.dumps({"sweep": rows, "peak": peak, "peak_kind": peak_kind}))


# ----------------------------------------------------------------------------------------------------------------------
def oracle_round(op, om, grads, work, rnd, bound):
    """One whole round by the CPU checker; returns (arrivals, seconds of the whole round, seconds of its aggregate path:
    bookkeeping + reduce + tolerance test)."""
    t0 = time.perf_counter()
    hdr, pay = op.packetize(grads, rnd)
    d, _ = op.loss_mask(om, work.seed, rnd)
    arr, n = op.arrival(d, work.seed, rnd)
    t1 = time.perf_counter()
    st = op.book(hdr, arr, n, rnd, op.new_state())
    op.reduce(pay, st, mean=True)
    op.check_bound(st["bitmap"], bound)
    t2 = time.perf_counter()
    return n, t2 - t0, t2 - t1


def oracle_setup(work, threads):
    from oracle import dblp_oracle as orc
    op = orc.Plan(work.numel, work.elem_size, work.payload_bytes, work.W)
    om = orc.loss_model(work.loss.kind, **work.loss.thresholds(op.C))
    grads = wl.make_grads(work, "cpu")
    if work.dtype == "bf16":
        grads = [g.view(torch.int16).numpy().view("uint16") for g in grads]
    else:
        grads = [g.numpy() for g in grads]
    return op, om, grads, orc.set_threads(threads)


def sample_of(work, max_elems):
    """A bounded sample of the workload: its leading tensors, up to max_elems elements per worker."""
    if work.N <= max_elems:
        return work, "full workload"
    numel, tot = [], 0
    for n in work.numel:
        if tot + n > max_elems and numel:
            break
        numel.append(min(n, max_elems))
        tot += numel[-1]
    s = copy.copy(work)
    s.numel = numel
    return s, "leading %d of %d tensors (%d of %d elements per worker)" % (len(numel), len(work.numel), tot, work.N)


def time_oracle(work, sample, what, threads, budget_s, max_reps):
    from oracle import dblp_oracle as orc
    op, om, grads, used = oracle_setup(sample, threads)
    bound = work.bounds_ppm[0]
    oracle_round(op, om, grads, sample, 1, bound)                   # first call pays for page faults of fresh buffers
    t0 = time.perf_counter()
    reps, t_round, t_agg = 0, 0.0, 0.0
    while reps < 2 or (time.perf_counter() - t0 < budget_s and reps < max_reps):
        n, a, b = oracle_round(op, om, grads, sample, 2 + reps, bound)
        t_round, t_agg, reps = t_round + a, t_agg + b, reps + 1
    t_round, t_agg = t_round / reps, t_agg / reps
    by = byte_model(sample.W, sample.N, sample.elem_size, op.C, n, int(n / op.M * sample.W * sample.N * sample.elem_size))
    orc.set_threads(os.cpu_count() or 1)
    return {"value": by["aggregate_path"] / t_agg / 1e9, "unit": "GB/s", "cores": used, "kind": "oracle",
            "sample": "%s, %d rounds, %.2f s per round of which %.2f s in bookkeeping + reduce + tolerance test; only the "
                      "reduce loop is multi-threaded" % (what, reps, t_round, t_agg),
            "step_GBps": by["total"] / t_round / 1e9, "ms_per_step": t_round * 1e3}


def cpu_baseline(work):
    """The CPU checker, as it stands, on a bounded sample of the same workload: on all host cores and on one."""
    sample, what = sample_of(work, 32_000_000)
    allc = time_oracle(work, sample, what, os.cpu_count() or 1, 10.0, 12)
    one = time_oracle(work, sample, what, 1, 8.0, 6)
    allc["single_thread"] = {k: one[k] for k in ("value", "unit", "cores", "sample", "step_GBps")}
    return allc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload or HEADLINE
    work = workload_by_name(name)
    total_steps = args.steps + args.warmup
    budget_s = 150.0
    # about 65 ns per element-worker on one core for packetize + reduce: size the sample so the run fits the budget
    per_step = budget_s / max(1, total_steps)
    max_elems = int(max(1_000_000, min(work.N, per_step / (8e-9 * work.W))))
    sample, what = sample_of(work, max_elems)
    op, om, grads, threads = oracle_setup(sample, os.cpu_count() or 1)
    bound = work.bounds_ppm[0]
    for i in range(args.warmup):
        oracle_round(op, om, grads, sample, 1 + i, bound)
    t_round = t_agg = 0.0
    for k in range(args.steps):
        n, a, b = oracle_round(op, om, grads, sample, 100 + k, bound)
        t_round, t_agg = t_round + a, t_agg + b
    t_round, t_agg = t_round / args.steps, t_agg / args.steps
    by = byte_model(sample.W, sample.N, sample.elem_size, op.C, n, int(n / op.M * sample.W * sample.N * sample.elem_size))
    v = by["aggregate_path"] / t_agg / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_round * 1e3, "higher_is_better": True,
        "vs_baseline": None, "dtype": work.dtype, "data": "synthetic",
        "config": {"workload": work.name, "W": work.W, "payload_bytes": work.payload_bytes, "tensors": len(work.numel),
                   "elements_per_worker": work.N, "loss": work.loss.kind},
        "value_is": "aggregate path (bookkeeping + masked reduce + tolerance test): its bytes / its time inside the step",
        "step_GBps": by["total"] / t_round / 1e9,
        "cpu_baseline": {"value": v, "unit": "GB/s", "kind": "oracle", "cores": threads,
                         "sample": what + "; only the reduce loop is multi-threaded"},
        "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=None,
                    help="one workload only (%s, or point:DTYPE:MiB:W:PAYLOAD for one point of the size sweep); default: "
                         "gpt2xl as the headline with resnet50 and bert under per_config" % ", ".join(sorted(WORKLOADS)))
    ap.add_argument("--impl", choices=["dblp", "reference"], default="dblp")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-verify", action="store_true", help="skip the check of the last round against the CPU checker")
    ap.add_argument("--extras", action="store_true", help="also run the control-loop and fused-reduce side sections")
    ap.add_argument("--sweep", action="store_true", help="time the size sweep instead of the default step")
    args = ap.parse_args()
    if args.workload is not None and args.workload not in WORKLOADS and not args.workload.startswith("point:"):
        ap.error("unknown workload %r" % args.workload)
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
