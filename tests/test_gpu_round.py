"""GPU parity for the round state machine: retransmission attempts (send set = what the bitmap reports missing), early
stop (each worker's receiver stops the moment its tolerance is met) and the control loop that strings them together.
Everything here is integer work and must match the CPU oracle bit for bit; the aggregate after the loop too."""
import numpy as np
import pytest
import torch

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import binding as dblp
from paper_2605_01989_b200 import workloads as wl

import harness as H

pytestmark = pytest.mark.gpu

RAGGED = [1000, 1, 352 * 40, 353, 7, 100003, 2, 352]
LOSSES = [wl.LossSpec("iid", 0.4), wl.LossSpec("ge", 0.3, 6.0),
          wl.LossSpec("microburst", window_frac=0.3, p_in=0.8, p_out=0.05)]


def work(numel, dtype, P, W, loss, seed):
    return wl.Workload("t", W, dtype, P, list(numel), 1e-3, loss, seed, round=seed + 2)


@pytest.mark.parametrize("loss", LOSSES, ids=["iid", "ge", "mb"])
def test_retransmission_attempts_match_step_by_step(loss):
    w = work(RAGGED, "f32", 1408, 5, loss, 17)
    op = orc.Plan(w.numel, 4, 1408, 5)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    grads = wl.make_grads(w, H.DEV)
    g.packetize(grads, w.round)
    o_hdr = op.headers(w.round)
    st = op.new_state()
    b = g.buf
    for attempt in range(4):
        dblp.dblp_missing_bits(g.plan, b["recv_bitmap"], b["sent_bits"])
        o_sent = op.missing_bits(st["bitmap"])
        H.assert_bits_equal(H.u32(b["sent_bits"]).reshape(op.W, op.row_words), o_sent, "send set")
        dblp.dblp_apply_loss_resend(g.plan, gm, w.seed, w.round, attempt, b["sent_bits"], b["delivered_bits"],
                                    b["arrival"], b["n_arrived"], b["ws"])
        o_del, _ = op.loss_mask(om, w.seed, w.round, attempt, o_sent)
        o_arr, o_n = op.arrival(o_del, w.seed, w.round, attempt)
        assert g.n_arrived() == o_n
        H.assert_bits_equal(H.u32(b["delivered_bits"]).reshape(op.W, op.row_words), o_del, "delivered, attempt %d" % attempt)
        H.assert_bits_equal(H.u32(b["arrival"])[:o_n], o_arr[:o_n], "arrival, attempt %d" % attempt)
        dblp.dblp_aggregate_book(g.plan, b["hdr_ring"], op.M, b["arrival"], b["n_arrived"], op.M, w.round,
                                 b["recv_bitmap"], b["slot_key"], b["counters"])
        st = op.book(o_hdr, o_arr, o_n, w.round, st)
        H.compare_state(g, st, op)
    assert st["counters"].n_dup == 0                     # nothing that had arrived was sent again
    g.close()


@pytest.mark.parametrize("ppm", [0, 8000, 100000, 408000, 1000000])
@pytest.mark.parametrize("W", [1, 5, 33])
def test_early_stop_matches_the_sequential_receiver(ppm, W):
    w = work(RAGGED, "f32", 1408, W, wl.LossSpec("iid", 0.05), 23)
    op = orc.Plan(w.numel, 4, 1408, W)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w, arrival_cap=2 * op.M)
    b = g.buf
    g.packetize(wl.make_grads(w, H.DEV), w.round)
    o_hdr = op.headers(w.round)
    o_del, _ = op.loss_mask(om, w.seed, w.round)
    o_arr, o_n = op.arrival(o_del, w.seed, w.round)
    # the arrival list with 10 % of its entries repeated somewhere later (duplicates before and after the stops)
    rng = np.random.default_rng(1)
    extra = rng.choice(o_arr[:o_n], o_n // 10)
    mixed = np.concatenate([o_arr[:o_n], extra])
    tail = mixed[o_n // 2:].copy()
    rng.shuffle(tail)
    mixed[o_n // 2:] = tail
    b["arrival"][:len(mixed)].copy_(torch.from_numpy(mixed.view(np.int32)))
    b["n_arrived"].fill_(len(mixed))
    dblp.dblp_aggregate_book_stop(g.plan, b["hdr_ring"], op.M, b["arrival"], b["n_arrived"], b["arrival_cap"], w.round, ppm,
                                  b["recv_bitmap"], b["slot_key"], b["counters"], b["ws"])
    st = op.book(o_hdr, mixed, len(mixed), w.round, op.new_state(), stop_ppm=ppm)
    H.compare_state(g, st, op)
    c = st["counters"].as_dict()
    if ppm in (100000, 408000):                     # 5 % loss: tighter tolerances are not met in the first attempt
        assert c["n_late"] > 0 and c["n_dup"] > 0
    # a second attempt continues the same round: stopped receivers ignore it, the others go on
    dblp.dblp_apply_loss(g.plan, gm, w.seed, w.round, 1, b["delivered_bits"], b["arrival"], b["n_arrived"], b["ws"])
    o_del1, _ = op.loss_mask(om, w.seed, w.round, 1)
    o_arr1, o_n1 = op.arrival(o_del1, w.seed, w.round, 1)
    dblp.dblp_aggregate_book_stop(g.plan, b["hdr_ring"], op.M, b["arrival"], b["n_arrived"], b["arrival_cap"], w.round, ppm,
                                  b["recv_bitmap"], b["slot_key"], b["counters"], b["ws"])
    st = op.book(o_hdr, o_arr1, o_n1, w.round, st, stop_ppm=ppm)
    H.compare_state(g, st, op)
    H.compare_bound(g, op, st["bitmap"], ppm)
    g.close()


@pytest.mark.parametrize("early", [False, True], ids=["probe", "early-stop"])
@pytest.mark.parametrize("loss,ppm", [(wl.LossSpec("iid", 0.7), 8000), (wl.LossSpec("iid", 0.7), 408000),
                                      (wl.LossSpec("ge", 0.5, 10.0), 24000),
                                      (wl.LossSpec("microburst", window_frac=0.5, p_in=0.9, p_out=0.01), 8000)],
                         ids=["iid-low", "iid-high", "ge", "mb"])
def test_control_loop_attempts_state_and_aggregate(loss, ppm, early):
    w = work(RAGGED, "bf16", 4096, 4, loss, 29)
    op = orc.Plan(w.numel, 2, 4096, 4)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    grads = wl.make_grads(w, H.DEV)
    g.packetize(grads, w.round)
    attempts, ok = dblp.dblp_round_until_stop(g.plan, gm, w.seed, w.round, ppm, 60, early, g.buf)
    o_hdr, o_pay = op.packetize(H.to_host(grads, w.dtype), w.round)
    st, o_attempts, o_ok, _ = op.round_until_stop(o_hdr, om, w.seed, w.round, ppm, 60, early)
    assert (attempts, ok) == (o_attempts, o_ok) and ok == 1
    H.compare_state(g, st, op)
    g.reduce(dblp.DBLP_MEAN)
    torch.cuda.synchronize()
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), op.reduce(o_pay, st, mean=True), "aggregate after the loop")
    g.close()


def test_control_loop_gives_up_after_max_attempts():
    w = work([256 * 500], "f32", 1024, 2, wl.LossSpec("iid", 1.0), 3)
    g = H.GpuRound(w)
    g.packetize(wl.make_grads(w, H.DEV), w.round)
    gm, _ = H.models_for(w, g.plan.C)
    assert dblp.dblp_round_until_stop(g.plan, gm, 3, w.round, 8000, 3, True, g.buf) == (3, 0)
    assert dblp.counters_dict(g.buf["counters"])["n_arrived"] == 0
    g.close()


def test_early_stop_at_the_bench_workload_size():
    w = wl.config(1)
    op = orc.Plan(w.numel, 4, w.payload_bytes, w.W)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    g.packetize(wl.make_grads(w, H.DEV), w.round)
    o_hdr = op.headers(w.round)
    for ppm, early in ((408000, True), (0, True)):
        g.reset()
        attempts, ok = dblp.dblp_round_until_stop(g.plan, gm, w.seed, w.round, ppm, 40, early, g.buf)
        st, o_attempts, o_ok, _ = op.round_until_stop(o_hdr, om, w.seed, w.round, ppm, 40, early)
        assert (attempts, ok) == (o_attempts, o_ok)
        H.compare_state(g, st, op)
    g.close()
