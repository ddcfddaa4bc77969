"""GPU parity for the work fused behind the masked reduce: the L2 norm of the aggregate (input of Eq. 1) and the
worker-side update w <- w - lr * g (Algorithm 4), including the broadcast half of a round run as a W = 1 plan.
The update is fp32 multiply-then-subtract on both sides: bit-exact.  The norm is an fp64 sum of exact squares of
non-negative terms; the device adds them along a fixed tree of depth < 400 (per thread, warp, block, tiles), each
addition off by at most 2^-53 relative, so it must agree with the oracle's exactly rounded sum to 1e-12 relative
(bound: 400 * 1.1e-16 = 4.4e-14)."""
import numpy as np
import pytest
import torch

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import binding as dblp
from paper_2605_01989_b200 import workloads as wl

import harness as H

pytestmark = pytest.mark.gpu
NORM_RTOL = 1e-12
RAGGED = [1000, 1, 352 * 40, 353, 7, 100003, 2, 352]


def _round(w):
    op = orc.Plan(w.numel, w.elem_size, w.payload_bytes, w.W)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    grads = wl.make_grads(w, H.DEV)
    g.packetize(grads, w.round)
    g.apply_loss(gm, w.seed, w.round)
    b = g.buf
    dblp.dblp_aggregate_book(g.plan, b["hdr_ring"], op.M, b["arrival"], b["n_arrived"], op.M, w.round, b["recv_bitmap"],
                             b["slot_key"], b["counters"])
    o_hdr, o_pay = op.packetize(H.to_host(grads, w.dtype), w.round)
    o_del, _ = op.loss_mask(om, w.seed, w.round)
    o_arr, o_n = op.arrival(o_del, w.seed, w.round)
    st = op.book(o_hdr, o_arr, o_n, w.round, op.new_state())
    return g, op, o_pay, st


@pytest.mark.parametrize("dtype,P,W", [("f32", 1408, 5), ("bf16", 4096, 3), ("f32", 1024, 2), ("f32", 4096, 17),
                                       ("f32", 4096, 1), ("bf16", 2048, 2)])
@pytest.mark.parametrize("flags", [dblp.DBLP_SUM, dblp.DBLP_MEAN])
def test_fused_norm_and_update(dtype, P, W, flags):
    w = wl.Workload("t", W, dtype, P, RAGGED, 1e-3, wl.LossSpec("ge", 0.1, 5.0), seed=W, round=4)
    g, op, o_pay, st = _round(w)
    n_scratch = dblp.dblp_norm_scratch_count(g.plan)
    assert n_scratch > 0
    scratch = torch.full((n_scratch,), float("nan"), dtype=torch.float64, device=H.DEV)
    norm = torch.zeros(2, dtype=torch.float64, device=H.DEV)
    gen = torch.Generator(device="cpu").manual_seed(3)
    params0 = torch.randn(op.N, generator=gen, dtype=torch.float32)
    params = params0.to(H.DEV)
    lr = 0.05
    dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], flags, scratch, norm,
                                  params, lr)
    torch.cuda.synchronize()
    agg = op.reduce(o_pay, st, mean=(flags == dblp.DBLP_MEAN))
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), agg, "aggregate")
    H.assert_bits_equal(params.cpu().numpy(), orc.sgd_apply(params0.numpy(), agg, lr), "updated parameters")
    s, nrm = orc.norm(agg)
    got_s, got_n = norm.cpu().tolist()
    assert abs(got_s - s) <= NORM_RTOL * s and abs(got_n - nrm) <= NORM_RTOL * nrm
    assert got_n == float(np.sqrt(np.float64(got_s)))
    # same plan, same data: the fixed tree gives the same bits again
    norm2 = torch.zeros(2, dtype=torch.float64, device=H.DEV)
    dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], flags, scratch, norm2)
    assert torch.equal(norm, norm2)
    # the regime decision taken from the device's norm equals the one taken from the oracle's
    for prev in (nrm * 2.0, nrm / 2.0, nrm * 1.1, nrm * 3.0, 0.0):
        assert dblp.dblp_clr(prev, got_n, 0.5) == orc.clr(prev, nrm, 0.5)
    # extras off: identical aggregate, parameters untouched
    dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], flags)
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), agg, "aggregate, extras off")
    g.close()


@pytest.mark.parametrize("dtype,P,W", [("f32", 1408, 5), ("bf16", 4096, 3), ("f32", 1024, 2)])
def test_bf16_output_is_the_rounded_fp32_aggregate(dtype, P, W):
    w = wl.Workload("t", W, dtype, P, RAGGED, 1e-3, wl.LossSpec("iid", 0.1), seed=W + 40, round=2)
    g, op, o_pay, st = _round(w)
    out16 = torch.full((op.N + 3,), 0x1234, dtype=torch.int16, device=H.DEV)
    scratch = torch.empty(dblp.dblp_norm_scratch_count(g.plan), dtype=torch.float64, device=H.DEV)
    norm = torch.zeros(2, dtype=torch.float64, device=H.DEV)
    for view in (out16[:op.N], out16[1:op.N + 1]):                   # second view: only 2-byte aligned
        view.fill_(0x1234)
        dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], view,
                                      dblp.DBLP_MEAN | dblp.DBLP_OUT_BF16, scratch, norm)
        agg = op.reduce(o_pay, st, mean=True)
        H.assert_bits_equal(view.cpu().numpy().view(np.uint16), orc.to_bf16(agg), "bf16 aggregate")
        s, _ = orc.norm(agg)
        assert abs(norm[0].item() - s) <= NORM_RTOL * s                 # the norm is taken before the rounding
    assert int(out16[op.N + 1].item()) == 0x1234                        # nothing written past the end
    g.close()


@pytest.mark.parametrize("dtype,P,W", [("f32", 1408, 5), ("bf16", 4096, 3), ("f32", 1024, 32)])
@pytest.mark.parametrize("flags", [dblp.DBLP_SUM, dblp.DBLP_MEAN])
def test_order_free_reduce_is_within_the_rounding_bound(dtype, P, W, flags):
    """Any order of W fp32 additions is within (W-1) * 2^-24 * sum|x| of the exact sum, so the atomic result and the
    oracle's fixed-order result differ by at most twice that (the mean's division adds one more rounding)."""
    w = wl.Workload("t", W, dtype, P, RAGGED, 1e-3, wl.LossSpec("iid", 0.15), seed=W + 60, round=2)
    g, op, o_pay, st = _round(w)
    dblp.dblp_aggregate_reduce_atomic(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], flags)
    got = g.buf["agg"].cpu().numpy().astype(np.float64)
    ref = op.reduce(o_pay, st, mean=(flags == dblp.DBLP_MEAN)).astype(np.float64)
    # sum over the workers that delivered of |x_w|, per element, from the oracle's own packets
    pay = o_pay.reshape(op.M, op.P)
    if dtype == "f32":
        vals = np.abs(pay.view(np.float32).astype(np.float64))
    else:
        vals = np.abs(torch.from_numpy(pay.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy())
    E = op.E
    mag = np.zeros(op.N)
    recv = st["slot_of"].reshape(op.W, op.C) != orc.NONE
    for t in range(op.T):
        n, b, c0 = int(op.numel[t]), int(op.base[t]), int(op.chunkbase[t])
        nch = -(-n // E)
        for wk in range(op.W):
            rows = vals[wk * op.C + c0: wk * op.C + c0 + nch] * recv[wk, c0:c0 + nch, None]
            mag[b:b + n] += rows.reshape(-1)[:n]
    scale = 1.0 / W if flags == dblp.DBLP_MEAN else 1.0
    bound = (2 * (W - 1) + 2) * 2.0 ** -24 * mag * scale + 1e-45
    assert (np.abs(got - ref) <= bound).all()
    assert (got[mag == 0] == 0).all()                                   # chunks nobody delivered are exactly zero
    g.close()


def test_norm_of_an_all_lost_round_is_zero():
    w = wl.Workload("t", 3, "f32", 1408, RAGGED, 1e-3, wl.LossSpec("iid", 1.0), seed=1, round=1)
    g, op, o_pay, st = _round(w)
    scratch = torch.empty(dblp.dblp_norm_scratch_count(g.plan), dtype=torch.float64, device=H.DEV)
    norm = torch.ones(2, dtype=torch.float64, device=H.DEV)
    params = torch.ones(op.N, dtype=torch.float32, device=H.DEV)
    dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], dblp.DBLP_MEAN, scratch,
                                  norm, params, 0.5)
    assert norm.cpu().tolist() == [0.0, 0.0] and bool((params == 1.0).all())
    g.close()


def test_broadcast_half_reconstructs_and_updates_in_one_pass():
    """Server -> worker: the mean travels as packets of a single sender (W = 1), is lossy, and the worker applies
    w <- w - lr * (what arrived, zero where nothing did)."""
    numel = RAGGED
    N = sum(numel)
    gen = torch.Generator(device="cpu").manual_seed(11)
    mean_grad = (torch.randn(N, generator=gen) * 1e-3).to(torch.float32)
    weights0 = torch.randn(N, generator=gen, dtype=torch.float32)
    w = wl.Workload("bcast", 1, "f32", 1408, numel, 1e-3, wl.LossSpec("microburst", window_frac=0.2, p_in=0.6, p_out=0.01),
                    seed=9, round=12)
    op = orc.Plan(numel, 4, 1408, 1)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    g.packetize([mean_grad.to(H.DEV)], w.round)
    g.apply_loss(gm, w.seed, w.round)
    b = g.buf
    dblp.dblp_aggregate_book(g.plan, b["hdr_ring"], op.M, b["arrival"], b["n_arrived"], op.M, w.round, b["recv_bitmap"],
                             b["slot_key"], b["counters"])
    weights = weights0.to(H.DEV)
    dblp.dblp_aggregate_reduce_ex(g.plan, b["payload_ring"], b["slot_key"], b["agg"], dblp.DBLP_SUM, None, None, weights, 0.1)
    o_hdr, o_pay = op.packetize([mean_grad.numpy()], w.round)
    o_del, _ = op.loss_mask(om, w.seed, w.round)
    o_arr, o_n = op.arrival(o_del, w.seed, w.round)
    st = op.book(o_hdr, o_arr, o_n, w.round, op.new_state())
    recon = op.reduce(o_pay, st)
    assert 0.05 < 1 - o_n / op.M < 0.3
    H.assert_bits_equal(b["agg"].cpu().numpy(), recon, "reconstructed mean")
    H.assert_bits_equal(weights.cpu().numpy(), orc.sgd_apply(weights0.numpy(), recon, 0.1), "updated weights")
    lost = recon == 0
    assert bool((weights.cpu().numpy()[lost] == weights0.numpy()[lost]).all())
    g.close()


def test_norm_at_the_bench_workload_size():
    w = wl.config(1)
    g, op, o_pay, st = _round(w)
    scratch = torch.empty(dblp.dblp_norm_scratch_count(g.plan), dtype=torch.float64, device=H.DEV)
    norm = torch.zeros(2, dtype=torch.float64, device=H.DEV)
    dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], dblp.DBLP_MEAN, scratch, norm)
    agg = op.reduce(o_pay, st, mean=True)
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), agg, "aggregate")
    s, nrm = orc.norm(agg)
    assert abs(norm[0].item() - s) <= NORM_RTOL * s and abs(norm[1].item() - nrm) <= NORM_RTOL * nrm
    g.close()
