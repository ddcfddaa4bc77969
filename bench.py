#!/usr/bin/env python
"""Throughput of the DBLP receive path on synthetic gradients.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50|flat|bert|gpt2xl|sweep] [--impl reference]

One step = one communication round through the library: round_reset, packetize, apply_loss, aggregate (bookkeeping +
masked reduce) and check_bound, on gradients already resident in device memory.  The metric is algorithmic bytes read
plus written per step divided by the step time (GB/s).  Prints one JSON line.

With --impl reference the same round is run by the plain CPU checker on the host cores (a reported baseline).
Under torchrun (N > 1) every rank runs its own independent round on its own GPU (weak scaling); the per-worker loss
counts are summed across ranks once per step, the only exchange the sharded path has.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_01989_b200 import workloads as wl  # noqa: E402

METRIC = "bounded-loss aggregate GB/s (bytes read+written)"
WORKLOADS = {"flat": 0, "resnet50": 1, "bert": 2, "gpt2xl": 3, "sweep": 4}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def byte_model(work, C, n_arrived, payload_recv_bytes):
    """Algorithmic bytes of each stage for one round (what the method has to move, not what a kernel happens to)."""
    W, N, s, M = work.W, work.N, work.elem_size, work.W * C
    R = n_arrived
    stages = {
        "packetize": 2 * W * N * s + 32 * M,                       # read gradients, write payloads + headers
        "apply_loss": M // 8 + 4 * R,                              # delivered bitmap + arrival list
        "book": (4 + 32) * R + 4 * R + M // 8,                     # arrival entry + header per packet, slot entry, bitmap
        "reduce": payload_recv_bytes + 4 * N + 4 * M + 8 * C,      # received payloads, aggregate, slot entries, chunk table
        "check_bound": M // 8,
    }
    stages["total"] = sum(stages.values())
    return stages


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
def run_gpu(args):
    from paper_2605_01989_b200 import binding as dblp
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    work = wl.config(WORKLOADS[args.workload])
    if world > 1:
        work.seed = work.seed + 100 * rank            # every rank is an independent server shard with its own workers
    plan = dblp.Plan(work.numel, work.dtype, work.payload_bytes, work.W)
    buf = plan.alloc_round(dev)
    grads = wl.make_grads(work, dev)
    model = dblp.loss_model(work.loss.kind, **work.loss.thresholds(plan.C))
    bound = work.bounds_ppm[0]
    from paper_2605_01989_b200 import shard

    # The loss process and the arrival order do not depend on the gradients, so apply_loss (ALU-bound) runs on a side
    # stream while packetize (HBM-bound) runs on the main one; bookkeeping joins the two.  --serial puts all on one.
    side = None if args.serial else torch.cuda.Stream(priority=-1)   # high priority: its small kernels slot in between packetize blocks
    fork = torch.cuda.Event()
    join = torch.cuda.Event()
    booked = torch.cuda.Event()

    def lossy_channel(rnd, ev):
        dblp.dblp_round_reset(plan, buf["recv_bitmap"], buf["slot_key"], buf["counters"])
        if ev: ev[6].record()
        dblp.dblp_apply_loss(plan, model, work.seed, rnd, 0, buf["delivered_bits"], buf["arrival"], buf["n_arrived"],
                             buf["ws"])
        if ev: ev[7].record()

    def step(rnd, ev=None):
        if ev: ev[0].record()
        if side is not None:
            fork.record()
            with torch.cuda.stream(side):
                side.wait_event(fork)
                lossy_channel(rnd, ev)
                join.record()
        dblp.dblp_packetize(plan, grads, rnd, buf["hdr_ring"], buf["payload_ring"])
        if ev: ev[1].record()
        if side is not None:
            torch.cuda.current_stream().wait_event(join)
        else:
            lossy_channel(rnd, ev)
        if ev: ev[2].record()
        if side is None:
            dblp.dblp_aggregate_book(plan, buf["hdr_ring"], plan.M, buf["arrival"], buf["n_arrived"], plan.M, rnd,
                                     buf["recv_bitmap"], buf["slot_key"], buf["counters"])
        else:
            dblp.dblp_aggregate_claim(plan, buf["hdr_ring"], plan.M, buf["arrival"], buf["n_arrived"], plan.M, rnd,
                                      buf["slot_key"], buf["counters"])
        if ev: ev[3].record()
        if side is not None:                           # bitmap and tolerance test need the claims only: beside the reduce
            booked.record()
            with torch.cuda.stream(side):
                side.wait_event(booked)
                if ev: ev[8].record()
                dblp.dblp_aggregate_bitmap(plan, buf["slot_key"], buf["n_arrived"], plan.M, buf["recv_bitmap"],
                                           buf["counters"])
                dblp.dblp_check_bound(plan, buf["recv_bitmap"], bound, buf["recv_cnt"], buf["missing_cnt"], buf["ok"],
                                      buf["all_ok"])
                if ev: ev[5].record()
                join.record()
        dblp.dblp_aggregate_reduce(plan, buf["payload_ring"], buf["slot_key"], buf["agg"], dblp.DBLP_MEAN)
        if ev: ev[4].record()
        if side is not None:
            torch.cuda.current_stream().wait_event(join)
            if ev: ev[9].record()
        else:
            if ev: ev[8].record()
            dblp.dblp_check_bound(plan, buf["recv_bitmap"], bound, buf["recv_cnt"], buf["missing_cnt"], buf["ok"],
                                  buf["all_ok"])
            if ev: ev[5].record()
            if ev: ev[9].record()
        if dist is not None:                           # the sharded path's one exchange: loss counts per worker
            shard.exchange_counts(buf["recv_cnt"], buf["missing_cnt"])

    for i in range(args.warmup):
        step(1 + i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()

    K = args.steps
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local))
    graph = None
    if args.graph:
        # Launch-bound sizes: the step (both streams, fork and join included) is captured once into a CUDA graph and
        # replayed, so the host issues one launch per step.  Every replay redoes all the work with the captured round
        # number; the per-stage times then come from a short eager pass after the timed region.
        assert dist is None, "--graph is a single-GPU mode"
        graph = torch.cuda.CUDAGraph()
        launches0 = dblp.dblp_launch_count()
        with torch.cuda.graph(graph):
            step(100)
        launches_per_step = dblp.dblp_launch_count() - launches0
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        sampler.start()
        t_begin.record()
        for k in range(K):
            graph.replay()
        t_end.record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        launches = launches_per_step * K
        Ke = min(K, 50)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(10)] for _ in range(Ke)]
        for k in range(Ke):
            step(100, evs[k])
        torch.cuda.synchronize()
    else:
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(10)] for _ in range(K)]
        launches0 = dblp.dblp_launch_count()
        torch.cuda.synchronize()
        sampler.start()
        t_begin.record()
        for k in range(K):
            step(100 + k, evs[k])
        t_end.record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        launches = dblp.dblp_launch_count() - launches0
    if dist is not None:
        dist.barrier()
    ms_total = t_begin.elapsed_time(t_end)
    if dist is not None:
        t = torch.tensor([ms_total], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / K

    spans = {"packetize": (0, 1), "apply_loss": (6, 7), "book": (2, 3), "reduce": (3, 4), "check_bound": (8, 5)}
    stage_ms = {n: sum(e[a].elapsed_time(e[b]) for e in evs) / len(evs) for n, (a, b) in spans.items()}

    # realised loss of the last round -> algorithmic bytes
    n_arrived = int(buf["n_arrived"].item())
    bm = buf["recv_bitmap"].cpu().numpy().view("uint32").reshape(plan.W, plan.row_words)
    import numpy as np
    bits = np.unpackbits(bm.view(np.uint8), axis=1, bitorder="little")[:, :plan.C]
    E = work.E
    chunk_len = np.concatenate([np.minimum(E, n - np.arange(-(-n // E), dtype=np.int64) * E) for n in work.numel])
    payload_recv = int((bits.astype(np.int64) * chunk_len[None, :]).sum()) * work.elem_size
    bytes_ = byte_model(work, plan.C, n_arrived, payload_recv)

    # end to end from host memory: pinned gradients in, aggregate + counts out, every step
    e2e = None
    if not args.no_e2e and work.W * work.N * work.elem_size > (16 << 30):
        e2e = {"skipped": "host copies of %.0f GB of gradients: run with a smaller workload" % (work.W * work.N * work.elem_size / 1e9)}
    elif not args.no_e2e:
        grads_host = [g.cpu().pin_memory() for g in grads]
        grads_dev = torch.empty(work.W * work.N, dtype=plan.torch_dtype, device=dev)
        agg_host = torch.empty(work.N, dtype=torch.float32).pin_memory()
        cnt_host = torch.zeros(7, dtype=torch.int64).pin_memory()
        small = [torch.zeros(work.W, dtype=torch.int32).pin_memory() for _ in range(2)]
        ok_host = torch.zeros(work.W, dtype=torch.uint8).pin_memory()
        all_host = torch.zeros(1, dtype=torch.int32).pin_memory()
        Ke = min(K, args.e2e_steps)

        def e2e_step(rnd):
            dblp.dblp_round_host(plan, grads_host, model, work.seed, rnd, bound, dblp.DBLP_MEAN, buf, grads_dev,
                                 agg_host, cnt_host, small[0], small[1], ok_host, all_host)

        for i in range(3):
            e2e_step(50 + i)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for k in range(Ke):
            e2e_step(100 + k)
        b.record()
        torch.cuda.synchronize()
        ms_e2e = a.elapsed_time(b) / Ke
        if dist is not None:
            t = torch.tensor([ms_e2e], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e2e = float(t.item())
        e2e = {"value": world * bytes_["total"] / ms_e2e / 1e6, "unit": "GB/s", "ms_per_step": ms_e2e, "steps": Ke,
               "h2d_bytes_per_step": work.W * work.N * work.elem_size,
               "d2h_bytes_per_step": work.N * 4 + 56 + work.W * 9 + 4}
        del grads_host, grads_dev

    # the control loop under heavy i.i.d. bursts: attempts until every worker passes, low vs high tolerance
    # (the mechanism behind the paper's latency tables; not part of the timed step)
    round_loop = None
    if rank == 0 and world == 1 and not args.no_round_loop:
        p_low = bound
        p_high = bound + 400000
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

    # the reduce with its fused extras (norm for Eq. 1, worker update), timed alone; not part of the timed step
    extras = None
    if rank == 0 and world == 1 and not args.no_round_loop:
        dblp.dblp_round_reset(plan, buf["recv_bitmap"], buf["slot_key"], buf["counters"])
        step(7)
        scratch = torch.empty(max(1, dblp.dblp_norm_scratch_count(plan)), dtype=torch.float64, device=dev)
        norm_out = torch.zeros(2, dtype=torch.float64, device=dev)
        params = torch.zeros(work.N, dtype=torch.float32, device=dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def timed(fn, reps=50):
            for _ in range(3):
                fn()
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        extras = {
            "reduce_ms": timed(lambda: dblp.dblp_aggregate_reduce(plan, buf["payload_ring"], buf["slot_key"], buf["agg"],
                                                                  dblp.DBLP_MEAN)),
            "reduce_norm_ms": timed(lambda: dblp.dblp_aggregate_reduce_ex(plan, buf["payload_ring"], buf["slot_key"],
                                                                          buf["agg"], dblp.DBLP_MEAN, scratch, norm_out)),
            "reduce_norm_update_ms": timed(lambda: dblp.dblp_aggregate_reduce_ex(
                plan, buf["payload_ring"], buf["slot_key"], buf["agg"], dblp.DBLP_MEAN, scratch, norm_out, params, 0.01)),
            "reduce_atomic_order_free_ms": timed(lambda: dblp.dblp_aggregate_reduce_atomic(
                plan, buf["payload_ring"], buf["slot_key"], buf["agg"], dblp.DBLP_MEAN)),
            "grad_norm": float(norm_out[1].item()),
        }
        del scratch, params

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(work, bytes_["total"])

    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    peak, peak_kind = measured_peak()
    red_gbs = bytes_["reduce"] / stage_ms["reduce"] / 1e6
    agg_ms = sum(e[2].elapsed_time(e[9]) for e in evs) / len(evs)      # bookkeeping start to the end of reduce and bound check
    agg_gbs = (bytes_["book"] + bytes_["reduce"] + bytes_["check_bound"]) / agg_ms / 1e6
    out = {
        "metric": METRIC, "value": world * bytes_["total"] / ms_step / 1e6, "unit": "GB/s", "n_gpus": world,
        "steps": K, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": work.dtype, "data": "synthetic",
        "config": {"workload": work.name, "W": work.W, "payload_bytes": work.payload_bytes, "tensors": len(work.numel),
                   "elements_per_worker": work.N, "packets": plan.M, "loss": work.loss.kind,
                   "realised_loss": 1.0 - n_arrived / plan.M, "bound_ppm": bound, "reduce": "mean, fixed worker order",
                   "launch": "CUDA graph replay" if graph is not None else "eager",
                   "streams": "one" if side is None else "apply_loss beside packetize, bitmap + check_bound beside the reduce, on a high-priority side stream",
                   "l2": "inputs per step (%.0f MB) exceed the 126 MB L2; no flush" % (bytes_["total"] / 1e6),
                   "parallelism": "independent server shard per GPU" if world > 1 else "1 GPU"},
        "bytes_per_step": bytes_, "stage_ms": stage_ms,
        "pct_of_nominal_8TBs": 100.0 * bytes_["total"] / ms_step / 1e6 / NOMINAL_HBM_GBS,
        "aggregate_path": {"what": "bookkeeping + masked reduce + bound check only", "GBps": agg_gbs, "ms": agg_ms,
                           "pct_of_nominal_8TBs": 100.0 * agg_gbs / NOMINAL_HBM_GBS,
                           "pct_of_%s_peak" % peak_kind: 100.0 * agg_gbs / peak},
        "roofline": {"kernel": "k_reduce_rows" if work.W <= 4 and work.payload_bytes >= 2048 else "k_reduce_tiled", "bound": "hbm", "achieved": red_gbs, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": red_gbs / peak, "traffic": TRAFFIC.get(work.name),
                     "algorithmic_bytes_per_launch": bytes_["reduce"], "ms_per_launch": stage_ms["reduce"]},
        "clocks": clocks, "gpu_launches": launches, "e2e": e2e, "cpu_baseline": cpu, "round_loop": round_loop, "reduce_extras": extras,
    }
    print(json.dumps(out))


def run_sweep(args):
    """Stand-alone timing of packetize and of the aggregate path (bookkeeping + reduce + bound check) over the size
    sweep: per-worker buffer 1 MiB * 4^k, W in {2, 8, 32}, payload {1024, 4096}, 5 % bursty loss.  Points that do not
    fit in device memory are left out.  Prints one JSON line."""
    from paper_2605_01989_b200 import binding as dblp
    torch.cuda.set_device(0)
    dev = "cuda:0"
    peak, peak_kind = measured_peak()
    rows = []
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for k in range(6):
        for W in (2, 8, 32):
            for P in (1024, 4096):
                work = wl.sweep_point((1 << 20) * 4 ** k, W, P, 0.05, "ge", 10)
                free, _ = torch.cuda.mem_get_info()
                if work.device_bytes() + (2 << 30) > free:
                    rows.append({"buffer_MiB": 4 ** k, "W": W, "P": P, "skipped": "does not fit"})
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
                dblp.dblp_apply_loss(plan, model, work.seed, 1, 0, buf["delivered_bits"], buf["arrival"],
                                     buf["n_arrived"], buf["ws"])

                def agg_path():
                    dblp.dblp_round_reset(plan, buf["recv_bitmap"], buf["slot_key"], buf["counters"])
                    dblp.dblp_aggregate(plan, buf["hdr_ring"], buf["payload_ring"], plan.M, buf["arrival"],
                                        buf["n_arrived"], plan.M, 1, buf["recv_bitmap"], buf["slot_key"],
                                        buf["counters"], buf["agg"], dblp.DBLP_MEAN)
                    dblp.dblp_check_bound(plan, buf["recv_bitmap"], 50000, buf["recv_cnt"], buf["missing_cnt"],
                                          buf["ok"], buf["all_ok"])

                t_agg = timed(agg_path)
                t_red = timed(lambda: dblp.dblp_aggregate_reduce(plan, buf["payload_ring"], buf["slot_key"], buf["agg"],
                                                                 dblp.DBLP_MEAN))
                n = int(buf["n_arrived"].item())
                by = byte_model(work, plan.C, n, int(n / plan.M * work.W * work.N * work.elem_size))
                rows.append({"buffer_MiB": 4 ** k, "W": W, "P": P, "packets": plan.M, "loss": 1 - n / plan.M,
                             "packetize_GBps": by["packetize"] / t_pack / 1e6,
                             "aggregate_path_GBps": (by["book"] + by["reduce"] + by["check_bound"]) / t_agg / 1e6,
                             "reduce_GBps": by["reduce"] / t_red / 1e6, "reduce_frac_of_%s" % peak_kind: by["reduce"] / t_red / 1e6 / peak,
                             "aggregate_path_us": t_agg * 1e3})
                plan.close()
                del buf, grads
                torch.cuda.empty_cache()
    print(json.dumps({"sweep": rows, "peak": peak, "peak_kind": peak_kind}))


# DRAM bytes (read + write) per k_reduce launch from an ncu capture of this same workload; None until captured, and
# reset to None whenever the kernel changes.
TRAFFIC = {"resnet50-f32": 883.6e6}


# ----------------------------------------------------------------------------------------------------------------------
def oracle_round(op, om, grads, work, rnd):
    from oracle import dblp_oracle as orc  # noqa: F401
    hdr, pay = op.packetize(grads, rnd)
    d, _ = op.loss_mask(om, work.seed, rnd)
    arr, n = op.arrival(d, work.seed, rnd)
    st = op.book(hdr, arr, n, rnd, op.new_state())
    agg = op.reduce(pay, st, mean=True)
    res = op.check_bound(st["bitmap"], work.bounds_ppm[0])
    return n, agg, res


def oracle_setup(work):
    from oracle import dblp_oracle as orc
    op = orc.Plan(work.numel, work.elem_size, work.payload_bytes, work.W)
    om = orc.loss_model(work.loss.kind, **work.loss.thresholds(op.C))
    grads = wl.make_grads(work, "cpu")
    if work.dtype == "bf16":
        grads = [g.view(torch.int16).numpy().view("uint16") for g in grads]
    else:
        grads = [g.numpy() for g in grads]
    threads = orc.set_threads(os.cpu_count() or 1)
    return op, om, grads, threads


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
    import copy
    s = copy.copy(work)
    s.numel = numel
    return s, "leading %d of %d tensors (%d of %d elements per worker)" % (len(numel), len(work.numel), tot, work.N)


def cpu_baseline(work, gpu_total_bytes):
    """The CPU checker, as it stands, on a bounded sample of the same workload (about 10-30 s of CPU work)."""
    sample, what = sample_of(work, 32_000_000)
    op, om, grads, threads = oracle_setup(sample)
    oracle_round(op, om, grads, sample, 1)                       # first call pays for page faults of fresh buffers
    t0 = time.perf_counter()
    reps = 0
    while reps < 3 or (time.perf_counter() - t0 < 10.0 and reps < 20):
        n, _, _ = oracle_round(op, om, grads, sample, 2 + reps)
        reps += 1
    dt = (time.perf_counter() - t0) / reps
    bits_recv = n / op.M
    b = byte_model(sample, op.C, n, int(bits_recv * sample.W * sample.N * sample.elem_size))
    return {"value": b["total"] / dt / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": "%s, %d rounds, %.2f s per round; only the reduce loop is multi-threaded" % (what, reps, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    work = wl.config(WORKLOADS[args.workload])
    total_steps = args.steps + args.warmup
    budget_s = 150.0
    # about 65 ns per element-worker on one core for packetize + reduce: size the sample so the run fits the budget
    per_step = budget_s / max(1, total_steps)
    max_elems = int(max(1_000_000, min(work.N, per_step / (8e-9 * work.W))))
    sample, what = sample_of(work, max_elems)
    op, om, grads, threads = oracle_setup(sample)
    for i in range(args.warmup):
        oracle_round(op, om, grads, sample, 1 + i)
    t0 = time.perf_counter()
    for k in range(args.steps):
        n, _, _ = oracle_round(op, om, grads, sample, 100 + k)
    dt = (time.perf_counter() - t0) / args.steps
    b = byte_model(sample, op.C, n, int(n / op.M * sample.W * sample.N * sample.elem_size))
    v = b["total"] / dt / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": work.dtype, "data": "synthetic",
        "config": {"workload": work.name, "W": work.W, "payload_bytes": work.payload_bytes, "loss": work.loss.kind},
        "cpu_baseline": {"value": v, "unit": "GB/s", "kind": "oracle", "cores": threads,
                         "sample": what + "; only the reduce loop is multi-threaded"},
        "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="resnet50")
    ap.add_argument("--impl", choices=["dblp", "reference"], default="dblp")
    ap.add_argument("--e2e-steps", type=int, default=30)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-round-loop", action="store_true")
    ap.add_argument("--serial", action="store_true", help="all stages on one stream")
    ap.add_argument("--graph", action="store_true", help="replay the step as a CUDA graph (for launch-bound sizes)")
    ap.add_argument("--sweep", action="store_true", help="time the size sweep instead of the default step")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 1000 if args.steps is None else args.steps
        args.warmup = max(3, 10 if args.warmup is None else args.warmup)
        run_gpu(args)


if __name__ == "__main__":
    main()
