"""Helpers shared by the GPU parity tests: run one round through the C-ABI on the device, run the same round
through the CPU oracle on the same seeded inputs, and compare field by field.  Nothing the oracle consumes comes from
the CUDA path."""
import numpy as np
import torch

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import binding as dblp
from paper_2605_01989_b200 import workloads as wl

DEV = "cuda:0"


def models_for(work, C):
    """The same integer thresholds for both sides."""
    th = work.loss.thresholds(C)
    return dblp.loss_model(work.loss.kind, **th), orc.loss_model(work.loss.kind, **th)


def to_host(grads_dev, dtype):
    if dtype == "bf16":
        return [g.view(torch.int16).cpu().numpy().view(np.uint16) for g in grads_dev]
    return [g.cpu().numpy() for g in grads_dev]


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def hdr_np(t):
    return t.cpu().numpy().view(orc.HDR_DTYPE)


class GpuRound:
    """One round on the device through the public binding."""

    def __init__(self, work, bucket_bounds=None, n_slots=None, arrival_cap=None):
        self.work = work
        self.plan = dblp.Plan(work.numel, work.dtype, work.payload_bytes, work.W, bucket_bounds)
        self.buf = self.plan.alloc_round(DEV, n_slots, arrival_cap)
        self.reset()

    def reset(self):
        b = self.buf
        dblp.dblp_round_reset(self.plan, b["recv_bitmap"], b["slot_key"], b["counters"])

    def packetize(self, grads, rnd):
        dblp.dblp_packetize(self.plan, grads, rnd, self.buf["hdr_ring"], self.buf["payload_ring"])

    def apply_loss(self, model, seed, rnd, attempt=0):
        b = self.buf
        dblp.dblp_apply_loss(self.plan, model, seed, rnd, attempt, b["delivered_bits"], b["arrival"], b["n_arrived"],
                             b["ws"])

    def aggregate(self, rnd, flags=dblp.DBLP_SUM):
        b = self.buf
        dblp.dblp_aggregate(self.plan, b["hdr_ring"], b["payload_ring"], b["n_slots"], b["arrival"], b["n_arrived"],
                            b["arrival_cap"], rnd, b["recv_bitmap"], b["slot_key"], b["counters"], b["agg"], flags)

    def reduce(self, flags):
        b = self.buf
        dblp.dblp_aggregate_reduce(self.plan, b["payload_ring"], b["slot_key"], b["agg"], flags)

    def check_bound(self, bound_ppm):
        b = self.buf
        dblp.dblp_check_bound(self.plan, b["recv_bitmap"], bound_ppm, b["recv_cnt"], b["missing_cnt"], b["ok"],
                              b["all_ok"])
        torch.cuda.synchronize()
        W, B = self.plan.W, self.plan.B
        return (u32(b["recv_cnt"]).reshape(W, B), u32(b["missing_cnt"]).reshape(W, B),
                b["ok"].cpu().numpy().reshape(W, B), int(u32(b["all_ok"])[0]))

    def n_arrived(self):
        return int(self.buf["n_arrived"].item())

    def slot_key(self):
        k = self.buf["slot_key"].cpu().numpy().view(np.uint64)
        return (k & np.uint64(0xFFFFFFFF)).astype(np.uint32), (k >> np.uint64(32)).astype(np.uint32)

    def close(self):
        self.plan.close()
        self.buf = None


def assert_bits_equal(a, b, what):
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    assert a.shape == b.shape, "%s: shape %s vs %s" % (what, a.shape, b.shape)
    if a.tobytes() != b.tobytes():
        av, bv = a.reshape(-1).view(np.uint8), b.reshape(-1).view(np.uint8)
        bad = np.flatnonzero(av != bv)
        raise AssertionError("%s: %d differing bytes, first at byte %d" % (what, len(bad), bad[0]))


def full_round_parity(work, bounds=None, bucket_bounds=None, flags_list=(dblp.DBLP_SUM, dblp.DBLP_MEAN)):
    """Whole round on both sides from the same seeded gradients; every output compared bit for bit."""
    grads = wl.make_grads(work, DEV)
    host = to_host(grads, work.dtype)
    g = GpuRound(work, bucket_bounds)
    op = orc.Plan(work.numel, work.elem_size, work.payload_bytes, work.W)
    assert (g.plan.C, g.plan.N, g.plan.M, g.plan.row_words) == (op.C, op.N, op.M, op.row_words)
    gm, om = models_for(work, op.C)
    rnd, seed = work.round, work.seed

    g.packetize(grads, rnd)
    o_hdr, o_pay = op.packetize(host, rnd)
    assert_bits_equal(hdr_np(g.buf["hdr_ring"]), o_hdr, "header ring")
    assert_bits_equal(g.buf["payload_ring"].cpu().numpy(), o_pay, "payload ring")

    g.apply_loss(gm, seed, rnd)
    o_del, _ = op.loss_mask(om, seed, rnd)
    o_arr, o_n = op.arrival(o_del, seed, rnd)
    assert g.n_arrived() == o_n
    assert_bits_equal(u32(g.buf["delivered_bits"]).reshape(op.W, op.row_words), o_del, "delivered bitmap")
    assert_bits_equal(u32(g.buf["arrival"])[:o_n], o_arr[:o_n], "arrival list")

    st = op.book(o_hdr, o_arr, o_n, rnd, op.new_state())
    for i, flags in enumerate(flags_list):
        if i == 0:
            g.aggregate(rnd, flags)
        else:
            g.reduce(flags)
        torch.cuda.synchronize()
        assert_bits_equal(g.buf["agg"].cpu().numpy(), op.reduce(o_pay, st, mean=(flags == dblp.DBLP_MEAN)),
                          "aggregate (flags %d)" % flags)
    compare_state(g, st, op)
    for ppm in (bounds if bounds is not None else work.bounds_ppm):
        compare_bound(g, op, st["bitmap"], ppm, bucket_bounds)
    out = {"loss": 1.0 - o_n / op.M, "n_arrived": o_n}
    g.close()
    return out


def compare_state(g, st, op):
    assert_bits_equal(u32(g.buf["recv_bitmap"]).reshape(op.W, op.row_words), st["bitmap"], "received bitmap")
    slot, number = g.slot_key()
    assert_bits_equal(slot, st["slot_of"], "slot table")
    got = st["slot_of"] != orc.NONE
    assert_bits_equal(number[got], st["first_arrival"][got], "first-arrival numbers")
    assert (number[~got] == 0xFFFFFFFF).all()
    c = dblp.counters_dict(g.buf["counters"])
    assert {k: c[k] for k in dblp.COUNTER_FIELDS} == st["counters"].as_dict() and c["status"] == 0


def compare_bound(g, op, bitmap, ppm, bucket_bounds=None):
    recv, miss, ok, allok = g.check_bound(ppm)
    o = op.check_bound(bitmap, ppm, bucket_bounds)
    assert_bits_equal(recv, o[0], "recv counts")
    assert_bits_equal(miss, o[1], "missing counts")
    assert_bits_equal(ok, o[2], "ok flags")
    assert allok == o[3]
    return o


def oracle_round(op, om, host_grads, seed, rnd):
    """One whole round by the oracle: headers, payloads, delivered bitmap, arrival list, booked state."""
    o_hdr, o_pay = op.packetize(host_grads, rnd)
    o_del, _ = op.loss_mask(om, seed, rnd)
    o_arr, o_n = op.arrival(o_del, seed, rnd)
    st = op.book(o_hdr, o_arr, o_n, rnd, op.new_state())
    return o_hdr, o_pay, o_del, o_arr, o_n, st


def device_round_parity(work, rounds, bound_ppm, flags=dblp.DBLP_MEAN, marks=None):
    """`rounds` consecutive whole rounds through dblp_round_device (the library's two-stream schedule, every buffer
    reused from one round to the next), each compared with the oracle bit for bit: rings, delivered bitmap, arrival
    list, received bitmap, slot table, counters, bound outputs and the aggregate."""
    grads = wl.make_grads(work, DEV)
    host = to_host(grads, work.dtype)
    g = GpuRound(work)
    op = orc.Plan(work.numel, work.elem_size, work.payload_bytes, work.W)
    gm, om = models_for(work, op.C)
    for k in range(rounds):
        rnd = work.round + k
        dblp.dblp_round_device(g.plan, grads, gm, work.seed, rnd, bound_ppm, flags, g.buf, marks)
        torch.cuda.synchronize()
        o_hdr, o_pay, o_del, o_arr, o_n, st = oracle_round(op, om, host, work.seed, rnd)
        assert_bits_equal(hdr_np(g.buf["hdr_ring"]), o_hdr, "header ring, round %d" % rnd)
        assert_bits_equal(g.buf["payload_ring"].cpu().numpy(), o_pay, "payload ring, round %d" % rnd)
        assert g.n_arrived() == o_n
        assert_bits_equal(u32(g.buf["delivered_bits"]).reshape(op.W, op.row_words), o_del, "delivered bitmap")
        assert_bits_equal(u32(g.buf["arrival"])[:o_n], o_arr[:o_n], "arrival list")
        compare_state(g, st, op)
        assert_bits_equal(g.buf["agg"].cpu().numpy(), op.reduce(o_pay, st, mean=(flags == dblp.DBLP_MEAN)),
                          "aggregate, round %d" % rnd)
        W, B = op.W, 1
        o = op.check_bound(st["bitmap"], bound_ppm)
        assert_bits_equal(u32(g.buf["recv_cnt"]).reshape(W, B), o[0], "recv counts")
        assert_bits_equal(u32(g.buf["missing_cnt"]).reshape(W, B), o[1], "missing counts")
        assert_bits_equal(g.buf["ok"].cpu().numpy().reshape(W, B), o[2], "ok flags")
        assert int(u32(g.buf["all_ok"])[0]) == o[3]
    g.close()


def compare_bound_outputs(g, op, bitmap, ppm, saved=None):
    """Two-step check of the bound outputs that a whole-round call leaves in its buffers: called with g right after the
    round, it returns a host copy; called later with that copy and the oracle's bitmap, it compares."""
    if saved is None:
        W, B = g.plan.W, g.plan.B
        b = g.buf
        return (u32(b["recv_cnt"]).reshape(W, B).copy(), u32(b["missing_cnt"]).reshape(W, B).copy(),
                b["ok"].cpu().numpy().reshape(W, B).copy(), int(u32(b["all_ok"])[0]))
    o = op.check_bound(bitmap, ppm)
    assert_bits_equal(saved[0], o[0], "recv counts of the round")
    assert_bits_equal(saved[1], o[1], "missing counts of the round")
    assert_bits_equal(saved[2], o[2], "ok flags of the round")
    assert saved[3] == o[3]
    return o
