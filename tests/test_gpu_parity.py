"""GPU parity: the CUDA path, called through the C-ABI binding, against the CPU oracle on the same seeded inputs.
Bar: bit-exact for headers, payloads, masks, arrival lists, bitmaps, slot tables, counters and bound decisions, and
bit-exact for the fp32 aggregate (fixed worker order on both sides, bf16 widened exactly)."""
import numpy as np
import pytest
import torch

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import binding as dblp
from paper_2605_01989_b200 import workloads as wl

import harness as H

pytestmark = pytest.mark.gpu

RAGGED = [1000, 1, 352 * 40, 353, 7, 100003, 2, 352]          # sizes that are not multiples of the vector width
ALIGNED = [1024, 4096 * 3, 64, 352 * 64, 8]


def work(numel, dtype, P, W, loss, seed, bounds=(0, 8000, 50000, 408000)):
    return wl.Workload("t", W, dtype, P, list(numel), 1e-3, loss, seed, bounds_ppm=bounds, round=seed + 3)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P", [1408, 4096, 16])
@pytest.mark.parametrize("loss", [wl.LossSpec("none"), wl.LossSpec("iid", 0.1), wl.LossSpec("ge", 0.1, 5.0),
                                  wl.LossSpec("microburst", window_frac=0.2, p_in=0.5, p_out=0.01)],
                         ids=["none", "iid", "ge", "mb"])
def test_ragged_multi_tensor_round(dtype, P, loss):
    numel = RAGGED if P != 16 else [37, 1, 8, 5, 4096]
    H.full_round_parity(work(numel, dtype, P, 5, loss, 11))


@pytest.mark.parametrize("W", [1, 2, 8, 9, 17, 32])
def test_worker_counts(W):
    H.full_round_parity(work(ALIGNED, "f32", 1024, W, wl.LossSpec("iid", 0.2), 5))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P", [2048, 4096, 65536])
@pytest.mark.parametrize("W", [1, 2, 3, 4])
def test_few_workers_long_payloads(W, P, dtype):
    """The shape that takes the warp-per-chunk reduce kernel: ragged tensors, short last chunks, unaligned bases."""
    numel = [100003, 1, 4096, 5, 16384 * 3 + 7, 31, 2048]
    H.full_round_parity(work(numel, dtype, P, W, wl.LossSpec("iid", 0.2), 70 + W))


def test_random_shapes():
    """Forty seeded random plans: tensor counts and sizes (tiny, ragged, exact multiples of a chunk, large), payload
    sizes from 16 B to 64 KiB, 1 to 40 workers, both dtypes, every loss process."""
    rng = np.random.default_rng(2024)
    for case in range(40):
        P = int(rng.choice([16, 48, 256, 1024, 1408, 2048, 4096, 8192, 65536]))
        dtype = str(rng.choice(["f32", "bf16"]))
        E = P // (4 if dtype == "f32" else 2)
        numel = []
        for _ in range(int(rng.integers(1, 13))):
            kind = rng.integers(0, 4)
            if kind == 0:
                numel.append(int(rng.integers(1, 50)))
            elif kind == 1:
                numel.append(int(rng.integers(100, 5000)))
            elif kind == 2:
                numel.append(E * int(rng.integers(1, 6)))
            else:
                numel.append(int(rng.integers(5000, 200000)))
        W = int(rng.integers(1, 41))
        loss = [wl.LossSpec("none"), wl.LossSpec("iid", float(rng.uniform(0, 0.6))),
                wl.LossSpec("ge", float(rng.uniform(0.01, 0.5)), float(rng.uniform(1.0, 30.0))),
                wl.LossSpec("microburst", window_frac=float(rng.uniform(0, 1)), p_in=float(rng.uniform(0, 1)),
                            p_out=float(rng.uniform(0, 0.2)))][int(rng.integers(0, 4))]
        try:
            H.full_round_parity(work(numel, dtype, P, W, loss, 1000 + case, bounds=(int(rng.integers(0, 500000)),)))
        except AssertionError as e:
            raise AssertionError("case %d: P=%d %s W=%d numel=%s loss=%s: %s" % (case, P, dtype, W, numel, loss, e))


def test_thousands_of_workers_take_the_simple_reduce_kernel():
    """More workers than one chunk's slot entries fit in shared memory: the reduce falls back to its simple form, the
    fused extras say so instead of running, packetize goes through its worker groups."""
    w = work([100, 7, 64], "f32", 64, 6200, wl.LossSpec("iid", 0.3), 5, bounds=(0, 300000, 1000000))
    H.full_round_parity(w)
    g = H.GpuRound(w)
    assert dblp.dblp_norm_scratch_count(g.plan) == 0
    with pytest.raises(dblp.DblpError) as e:
        dblp.dblp_aggregate_reduce_ex(g.plan, g.buf["payload_ring"], g.buf["slot_key"], g.buf["agg"], dblp.DBLP_SUM)
    assert e.value.status == -3
    g.close()


def test_total_loss_and_zero_loss():
    r = H.full_round_parity(work(RAGGED, "f32", 1408, 3, wl.LossSpec("iid", 1.0), 2))
    assert r["n_arrived"] == 0
    r = H.full_round_parity(work(RAGGED, "bf16", 1408, 3, wl.LossSpec("iid", 0.0), 2))
    assert r["loss"] == 0.0


def test_single_chunk_and_word_boundaries():
    for n_chunks in (1, 31, 32, 33, 64, 65):
        H.full_round_parity(work([256 * n_chunks], "f32", 1024, 2, wl.LossSpec("ge", 0.3, 3.0), n_chunks))


def test_per_tensor_buckets_and_per_bucket_bounds():
    w = work(RAGGED, "f32", 1408, 4, wl.LossSpec("iid", 0.05), 8)
    op = orc.Plan(w.numel, 4, 1408, 4)
    bb = [int(x) for x in op.chunkbase]
    per_bucket = [0, 1000000, 50000, 20000, 0, 60000, 1000000, 0]
    H.full_round_parity(w, bounds=[50000, per_bucket], bucket_bounds=bb)


def test_config0_flat_fp32():
    r = H.full_round_parity(wl.config(0))
    assert 0.005 < r["loss"] < 0.015


def test_config1_resnet50_shaped():
    r = H.full_round_parity(wl.config(1), bounds=(24000, 8000, 0, 424000))
    assert 0.004 < r["loss"] < 0.02


def test_sweep_points_small():
    pts = [wl.sweep_point(sz, W, P, loss, kind, seed)
           for sz, W, P, loss, kind, seed in [(1 << 20, 2, 1024, 0.0, "iid", 10), (1 << 20, 32, 4096, 0.2, "ge", 11),
                                              (1 << 22, 8, 1024, 0.05, "iid", 12), (1 << 22, 32, 1024, 0.01, "ge", 13),
                                              (1 << 24, 2, 4096, 0.2, "iid", 14), (1 << 24, 8, 4096, 0.05, "ge", 10)]]
    for p in pts:
        H.full_round_parity(p, flags_list=(dblp.DBLP_SUM,))


def test_sweep_sample_across_every_axis():
    """A stride through the cartesian sweep (sizes x workers x payloads x loss rates x processes x seeds), limited to
    points whose rings the host can hold: every value of every axis occurs at least once."""
    pts = [p for p in wl.sweep(max_device_bytes=600e6)]
    sample = pts[::19]
    assert len(sample) >= 30
    for axis in ("W", "payload_bytes", "seed"):
        assert {getattr(p, axis) for p in sample} == {getattr(p, axis) for p in pts}
    assert {p.loss.kind for p in sample} >= {"none", "iid", "ge"}
    assert {p.loss.mean_loss for p in sample} >= {0.0, 0.01, 0.05, 0.2}
    assert len({p.N for p in sample}) >= 4
    for p in sample:
        H.full_round_parity(p, flags_list=(dblp.DBLP_MEAN,))


def _aggregate(g, rnd, flags, grouped):
    """dblp_aggregate, or the same with the claims grouped by slot range first."""
    if not grouped:
        return g.aggregate(rnd, flags)
    b = g.buf
    dblp.dblp_aggregate_claim_grouped(g.plan, b["hdr_ring"], b["n_slots"], b["arrival"], b["n_arrived"], b["arrival_cap"], rnd,
                                      b["slot_key"], b["counters"], b["ws"])
    dblp.dblp_aggregate_bitmap(g.plan, b["slot_key"], b["n_arrived"], b["arrival_cap"], b["recv_bitmap"], b["counters"])
    dblp.dblp_aggregate_reduce(g.plan, b["payload_ring"], b["slot_key"], b["agg"], flags)


@pytest.mark.parametrize("grouped", [False, True], ids=["claims in arrival order", "claims grouped by slot range"])
def test_stale_duplicate_and_invalid_packets_and_second_attempt(grouped):
    w = work(RAGGED, "f32", 1408, 4, wl.LossSpec("iid", 0.3), 21)
    rnd = w.round
    grads = wl.make_grads(w, H.DEV)
    host = H.to_host(grads, w.dtype)
    op = orc.Plan(w.numel, 4, 1408, 4)
    M, P = op.M, op.P
    n_junk = 600
    g = H.GpuRound(w, n_slots=M + n_junk, arrival_cap=2 * M)
    gm, om = H.models_for(w, op.C)

    # both sides packetize their own rings; the junk recipe below is applied to each side's ring separately
    g.packetize(grads, rnd)
    o_hdr, o_pay = op.packetize(host, rnd)
    rng = np.random.default_rng(7)
    src = rng.integers(0, M, n_junk)
    kinds = rng.integers(0, 8, n_junk)

    def add_junk(hdr, pay):
        hdr = np.concatenate([hdr, hdr[src]])
        pay = np.concatenate([pay.reshape(M, P), pay.reshape(M, P)[src]])
        j = hdr[M:]
        j["round"][kinds == 0] = rnd - 1
        j["round"][kinds == 1] = rnd + 1
        # kinds 2, 3: plain duplicates (payload of the copy is altered so that taking the wrong copy shows up)
        pay[M:][np.isin(kinds, (2, 3))] ^= 0x5A
        j["worker"][kinds == 4] = w.W + 3
        j["tensor_id"][kinds == 5] = op.T
        j["offset_elems"][kinds == 6] += 1
        j["len_bytes"][kinds == 7] += 4
        return hdr, pay.reshape(-1)

    o_hdr2, o_pay2 = add_junk(o_hdr, o_pay)
    g_hdr2, g_pay2 = add_junk(H.hdr_np(g.buf["hdr_ring"])[:M], g.buf["payload_ring"].cpu().numpy()[:M * P])
    H.assert_bits_equal(g_hdr2, o_hdr2, "ring headers with junk")
    g.buf["hdr_ring"].copy_(torch.from_numpy(g_hdr2.view(np.uint8).copy()))
    g.buf["payload_ring"].copy_(torch.from_numpy(g_pay2.copy()))

    # attempt 0: survivors of the loss process plus all junk slots plus an out-of-ring slot, shuffled
    g.apply_loss(gm, w.seed, rnd)
    o_del, _ = op.loss_mask(om, w.seed, rnd)
    o_arr, o_n = op.arrival(o_del, w.seed, rnd)
    H.assert_bits_equal(H.u32(g.buf["arrival"])[:o_n], o_arr[:o_n], "arrival list")
    mixed = np.concatenate([o_arr[:o_n], np.arange(M, M + n_junk, dtype=np.uint32),
                            np.array([M + n_junk, 0xFFFFFFFE], np.uint32)])
    rng.shuffle(mixed)
    g.buf["arrival"][:len(mixed)].copy_(torch.from_numpy(mixed.view(np.int32)))
    g.buf["n_arrived"].fill_(len(mixed))
    _aggregate(g, rnd, dblp.DBLP_SUM, grouped)
    st = op.book(o_hdr2, mixed, len(mixed), rnd, op.new_state())
    c = st["counters"].as_dict()
    assert c["n_stale"] > 50 and c["n_dup"] > 50 and c["n_invalid"] > 100
    H.compare_state(g, st, op)
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), op.reduce(o_pay2, st), "aggregate with junk")

    # attempt 1 of the same round: the sender re-sends what the bitmap says is missing; a new loss draw applies
    g.apply_loss(gm, w.seed, rnd, attempt=1)
    o_del1, _ = op.loss_mask(om, w.seed, rnd, attempt=1)
    o_arr1, o_n1 = op.arrival(o_del1, w.seed, rnd, attempt=1)
    H.assert_bits_equal(H.u32(g.buf["arrival"])[:o_n1], o_arr1[:o_n1], "arrival list, attempt 1")
    _aggregate(g, rnd, dblp.DBLP_MEAN, grouped)
    st = op.book(o_hdr2, o_arr1, o_n1, rnd, st)
    H.compare_state(g, st, op)
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), op.reduce(o_pay2, st, mean=True), "aggregate after attempt 1")
    assert st["counters"].as_dict()["n_dup"] > c["n_dup"]
    H.compare_bound(g, op, st["bitmap"], 100000)
    g.close()


@pytest.mark.parametrize("C", [1, 63, 64, 65, 4097, 70001])
def test_grouped_claims_leave_the_same_table_as_plain_claims(C):
    """Ring sizes around the limits of the grouping (fewer slots than ranges, one more than a power of two times the
    range count), with repeats and out-of-ring entries in the arrival list: claim table, bitmap and counters must be
    identical, byte for byte, to those of dblp_aggregate_claim."""
    w = work([C * 4], "f32", 16, 3, wl.LossSpec("iid", 0.2), 5 + C)
    grads = wl.make_grads(w, H.DEV)
    a, b = H.GpuRound(w, arrival_cap=2 * 3 * C + 8), H.GpuRound(w, arrival_cap=2 * 3 * C + 8)
    gm, _ = H.models_for(w, a.plan.C)
    M = a.plan.M
    rng = np.random.default_rng(C)
    for attempt in range(2):                             # the second call continues the arrival numbers of the first
        for g in (a, b):
            g.packetize(grads, w.round)
            g.apply_loss(gm, w.seed, w.round, attempt)
        n = a.n_arrived()
        extra = np.concatenate([rng.integers(0, M, n // 3 + 1), [M, M + 7, 0xFFFFFFFF]]).astype(np.uint32)
        mixed = np.concatenate([H.u32(a.buf["arrival"])[:n], extra])
        rng.shuffle(mixed)
        for g in (a, b):
            g.buf["arrival"][:len(mixed)].copy_(torch.from_numpy(mixed.view(np.int32)))
            g.buf["n_arrived"].fill_(len(mixed))
        _aggregate(a, w.round, dblp.DBLP_SUM, False)
        _aggregate(b, w.round, dblp.DBLP_SUM, True)
        torch.cuda.synchronize()
        for name in ("slot_key", "recv_bitmap", "counters", "agg"):
            assert torch.equal(a.buf[name].view(torch.uint8), b.buf[name].view(torch.uint8)), (name, attempt)
        assert dblp.counters_dict(b.buf["counters"])["n_invalid"] == 3 * (attempt + 1)
    a.close()
    b.close()


def test_physically_permuted_ring():
    """Packets stored in the ring at their arrival position instead of slot w*C+seq: the receive path trusts headers
    and the slot table only, so the aggregate must not change."""
    w = work(ALIGNED + [100003], "bf16", 4096, 6, wl.LossSpec("ge", 0.1, 4.0), 31)
    rnd = w.round
    grads = wl.make_grads(w, H.DEV)
    host = H.to_host(grads, w.dtype)
    op = orc.Plan(w.numel, 2, 4096, 6)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    g.packetize(grads, rnd)
    g.apply_loss(gm, w.seed, rnd)
    n = g.n_arrived()
    arr = g.buf["arrival"][:n].long()
    # move payloads and headers of the survivors to ring positions 0..n-1 in arrival order (plumbing, torch indexing)
    pay = g.buf["payload_ring"].view(op.M, op.P)
    hdr = g.buf["hdr_ring"].view(op.M, 32)
    pay[:n] = pay[arr].clone()
    hdr[:n] = hdr[arr].clone()
    pay[n:] = 0xEE
    hdr[n:] = 0xEE                       # garbage in the rest of the ring must never be touched
    g.buf["arrival"][:n] = torch.arange(n, dtype=torch.int32, device=H.DEV)
    g.aggregate(rnd)
    # oracle: its own round on the unpermuted ring -- the aggregate is defined by what arrived, not where it is stored
    o_hdr, o_pay = op.packetize(host, rnd)
    o_del, _ = op.loss_mask(om, w.seed, rnd)
    o_arr, o_n = op.arrival(o_del, w.seed, rnd)
    st = op.book(o_hdr, o_arr, o_n, rnd, op.new_state())
    assert o_n == n
    H.assert_bits_equal(g.buf["agg"].cpu().numpy(), op.reduce(o_pay, st), "aggregate from a permuted ring")
    H.assert_bits_equal(H.u32(g.buf["recv_bitmap"]).reshape(op.W, op.row_words), st["bitmap"], "bitmap")
    g.close()


@pytest.mark.parametrize("dtype,P", [("f32", 1408), ("bf16", 4096)])
def test_datagram_wire_format(dtype, P):
    """Header and payload interleaved in one ring, as a packet looks on the wire: same results, different addresses."""
    w = work(RAGGED, dtype, P, 4, wl.LossSpec("ge", 0.1, 5.0), 51)
    rnd = w.round
    grads = wl.make_grads(w, H.DEV)
    op = orc.Plan(w.numel, w.elem_size, P, 4)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    g.plan.set_wire_format(True)
    b = g.buf
    ring = torch.full((op.M * (32 + P) + 16,), 0xCD, dtype=torch.uint8, device=H.DEV)
    dblp.dblp_packetize(g.plan, grads, rnd, ring, ring)
    o_hdr, o_pay = op.packetize(H.to_host(grads, dtype), rnd)
    expect = np.concatenate([o_hdr.view(np.uint8).reshape(op.M, 32), o_pay.reshape(op.M, P)], axis=1).reshape(-1)
    H.assert_bits_equal(ring.cpu().numpy()[:op.M * (32 + P)], expect, "datagram ring")
    assert bool((ring[op.M * (32 + P):] == 0xCD).all())
    g.apply_loss(gm, w.seed, rnd)
    dblp.dblp_aggregate(g.plan, ring, ring, op.M, b["arrival"], b["n_arrived"], op.M, rnd, b["recv_bitmap"], b["slot_key"],
                        b["counters"], b["agg"], dblp.DBLP_MEAN)
    o_del, _ = op.loss_mask(om, w.seed, rnd)
    o_arr, o_n = op.arrival(o_del, w.seed, rnd)
    st = op.book(o_hdr, o_arr, o_n, rnd, op.new_state())
    H.compare_state(g, st, op)
    H.assert_bits_equal(b["agg"].cpu().numpy(), op.reduce(o_pay, st, mean=True), "aggregate from datagrams")
    dblp.dblp_aggregate_reduce_atomic(g.plan, ring, b["slot_key"], b["agg"], dblp.DBLP_SUM)
    ref = op.reduce(o_pay, st)
    assert np.allclose(b["agg"].cpu().numpy(), ref, rtol=0, atol=1e-8)
    g.close()


def _round_host_parity(w, bound_ppm=60000, reps=2):
    """dblp_round_host on workload w, `reps` calls in a row on the same buffers: everything it hands back to the host
    and the state it leaves on the device, against the oracle."""
    op = orc.Plan(w.numel, w.elem_size, w.payload_bytes, w.W)
    gm, om = H.models_for(w, op.C)
    grads_host = [x.pin_memory() for x in wl.make_grads(w, "cpu")]
    g = H.GpuRound(w)
    grads_dev = torch.empty(w.W * w.N, dtype=grads_host[0].dtype, device=H.DEV)
    agg_host = torch.empty(w.N, dtype=torch.float32).pin_memory()
    cnt_host = torch.zeros(7, dtype=torch.int64).pin_memory()
    recv_host = torch.zeros(w.W, dtype=torch.int32).pin_memory()
    miss_host = torch.zeros(w.W, dtype=torch.int32).pin_memory()
    ok_host = torch.zeros(w.W, dtype=torch.uint8).pin_memory()
    all_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    host = H.to_host(grads_host, w.dtype)
    for rep in range(reps):                    # later calls reuse every buffer
        rnd = w.round + rep
        agg_host.fill_(float("nan"))
        dblp.dblp_round_host(g.plan, grads_host, gm, w.seed, rnd, bound_ppm, dblp.DBLP_MEAN, g.buf, grads_dev,
                             agg_host, cnt_host, recv_host, miss_host, ok_host, all_host)
        o_hdr, o_pay = op.packetize(host, rnd)
        o_del, _ = op.loss_mask(om, w.seed, rnd)
        o_arr, o_n = op.arrival(o_del, w.seed, rnd)
        st = op.book(o_hdr, o_arr, o_n, rnd, op.new_state())
        want = op.reduce(o_pay, st, mean=True)
        H.assert_bits_equal(agg_host.numpy(), want, "aggregate via round_host")
        H.assert_bits_equal(g.buf["agg"].cpu().numpy(), want, "aggregate left on the device")
        H.assert_bits_equal(H.hdr_np(g.buf["hdr_ring"]), o_hdr, "header ring")
        assert g.buf["payload_ring"].cpu().numpy().tobytes() == o_pay.tobytes(), "payload ring"
        H.compare_state(g, st, op)
        o = op.check_bound(st["bitmap"], bound_ppm)
        assert recv_host.numpy().view(np.uint32).tolist() == o[0][:, 0].tolist()
        assert miss_host.numpy().view(np.uint32).tolist() == o[1][:, 0].tolist()
        assert ok_host.numpy().tolist() == o[2][:, 0].tolist() and int(all_host[0]) == o[3]
        assert dict(zip(dblp.COUNTER_FIELDS, cnt_host.tolist()[:6])) == st["counters"].as_dict()
    g.close()


def test_round_host_entry_point_matches_the_oracle():
    _round_host_parity(work(RAGGED, "f32", 1408, 3, wl.LossSpec("ge", 0.05, 6.0), 41))


@pytest.mark.parametrize("name,w", [
    ("resnet50: six parts", wl.config(1)),
    ("sixteen parts that cut through tensors, fp32", work([40_000_003, 17, 90_000_001, 4096 * 3 + 5], "f32", 4096, 2,
                                                        wl.LossSpec("iid", 0.03), 43)),
    ("sixteen parts, bf16, short payloads", work([100_000_001, 3, 70_000_000], "bf16", 1408, 2,
                                             wl.LossSpec("ge", 0.05, 6.0), 44)),
], ids=["resnet50", "f32-many-parts", "bf16-many-parts"])
def test_round_host_in_several_parts_matches_the_oracle(name, w):
    """Gradients of 32 MiB and more per worker go through dblp_round_host part by part (copy in, packetize, claim,
    reduce, copy out, pipelined): the results must be those of the unsplit round."""
    assert w.N * w.elem_size > (64 << 20)
    _round_host_parity(w, bound_ppm=w.bounds_ppm[0], reps=2)


def test_round_device_schedule_on_the_resnet50_shaped_workload():
    """The schedule the bench times (apply_loss beside packetize, bitmap + check_bound beside the reduce, on the plan's
    side stream), three consecutive rounds with every buffer reused, against the oracle."""
    H.device_round_parity(wl.config(1), rounds=3, bound_ppm=24000)


@pytest.mark.parametrize("dtype,P,W,flags", [("bf16", 4096, 3, dblp.DBLP_SUM), ("f32", 1408, 9, dblp.DBLP_MEAN),
                                              ("f32", 16, 2, dblp.DBLP_MEAN)])
def test_round_device_schedule_small_shapes(dtype, P, W, flags):
    numel = RAGGED if P != 16 else [37, 1, 8, 5, 4096]
    H.device_round_parity(work(numel, dtype, P, W, wl.LossSpec("ge", 0.1, 5.0), 23), rounds=4, bound_ppm=100000,
                          flags=flags)


def test_round_device_records_the_stage_marks():
    marks = dblp.RoundMarks()
    H.device_round_parity(wl.config(0), rounds=2, bound_ppm=8000, marks=marks)
    order = [("begin", "packetize_end"), ("loss_begin", "loss_end"), ("receive_begin", "claim_end"),
             ("claim_end", "reduce_end"), ("bound_begin", "bound_end"), ("reduce_end", "end"), ("begin", "end")]
    for a, b in order:
        assert marks.ms(a, b) >= 0.0, (a, b)
    assert marks.ms("begin", "end") > 0.0


def test_send_and_receive_halves_equal_the_whole_round():
    w = work(RAGGED, "f32", 1408, 5, wl.LossSpec("iid", 0.1), 77)
    grads = wl.make_grads(w, H.DEV)
    a, b = H.GpuRound(w), H.GpuRound(w)
    gm, _ = H.models_for(w, a.plan.C)
    dblp.dblp_round_device(a.plan, grads, gm, w.seed, 9, 50000, dblp.DBLP_MEAN, a.buf)
    dblp.dblp_round_send(b.plan, grads, gm, w.seed, 9, b.buf)
    dblp.dblp_round_receive(b.plan, 9, 50000, dblp.DBLP_MEAN, b.buf)
    torch.cuda.synchronize()
    for name in ("hdr_ring", "payload_ring", "delivered_bits", "recv_bitmap", "slot_key", "counters", "agg", "recv_cnt",
                 "missing_cnt", "ok", "all_ok"):
        assert torch.equal(a.buf[name].view(torch.uint8), b.buf[name].view(torch.uint8)), name
    a.close()
    b.close()


@pytest.mark.parametrize("W,P", [(766, 16), (766, 64), (761, 48), (1500, 32), (6134, 16)])
def test_worker_counts_at_the_shared_memory_limit_of_the_tiled_reduce(W, P):
    """Worker counts whose slot entries for a tile land on or just under the 48 KiB shared-memory limit."""
    H.full_round_parity(work([100, 7, 64, 333], "f32", P, W, wl.LossSpec("iid", 0.3), W, bounds=(0, 300000)))


@pytest.mark.parametrize("loss", [wl.LossSpec("iid", 0.1), wl.LossSpec("ge", 0.1, 5.0),
                                  wl.LossSpec("microburst", window_frac=0.2, p_in=0.5, p_out=0.01)], ids=["iid", "ge", "mb"])
@pytest.mark.parametrize("world", [2, 3, 5])
def test_shard_plans_side_by_side_equal_the_unsplit_round(loss, world):
    """A server split over `world` devices, its shards run here one after the other on one device (they do not depend
    on each other): delivered and received bitmaps side by side, counts summed and aggregates stitched must equal the
    unsplit round of the oracle -- the loss draws use stream-wide packet numbers."""
    from paper_2605_01989_b200 import shard
    numel = [1000, 1, 352 * 40, 353, 7, 100003, 2, 352, 5000, 33]
    w = work(numel, "f32", 1408, 4, loss, 19, bounds=(50000,))
    op = orc.Plan(w.numel, 4, 1408, 4)
    _, om = H.models_for(w, op.C)
    host = H.to_host(wl.make_grads(w, H.DEV), "f32")        # the runners draw the same values on the device
    o_hdr, o_pay, o_del, o_arr, o_n, st = H.oracle_round(op, om, host, w.seed, w.round)
    want_bits = np.unpackbits(st["bitmap"].view(np.uint8).reshape(op.W, -1), axis=1, bitorder="little")[:, :op.C]
    o_recv, o_miss, o_ok, o_all = op.check_bound(st["bitmap"], 50000)

    specs = shard.shard_specs(w.numel, w.E, world)
    bits, aggs, recv, miss = [], [], 0, 0
    for spec in specs:
        if spec.empty:
            continue
        r = shard.GpuShardRunner(w, spec, H.DEV)
        agg, rc, ms = r.round(w.round, 50000)
        torch.cuda.synchronize()
        for name in ("delivered_bits", "recv_bitmap"):               # no junk in this round: the two are equal
            b = H.u32(r.buf[name]).reshape(op.W, -1)
            got = np.unpackbits(b.view(np.uint8).reshape(op.W, -1), axis=1, bitorder="little")
            assert not got[:, spec.chunks:].any(), "padding bits of " + name
            if name == "recv_bitmap":
                bits.append(got[:, :spec.chunks])
        aggs.append(agg.cpu().numpy())
        recv = recv + H.u32(rc).astype(np.int64)
        miss = miss + H.u32(ms).astype(np.int64)
        r.close()
    H.assert_bits_equal(np.concatenate(bits, axis=1), want_bits, "shards' bitmaps side by side")
    H.assert_bits_equal(np.concatenate(aggs), op.reduce(o_pay, st, mean=True), "stitched aggregate")
    assert recv.tolist() == o_recv[:, 0].tolist() and miss.tolist() == o_miss[:, 0].tolist()
    ok, all_ok = shard.decide(dblp.dblp_bound_ok, torch.from_numpy(recv), torch.from_numpy(miss), 50000)
    assert ok == o_ok[:, 0].tolist() and all_ok == o_all


def test_argument_errors_are_reported_not_faulted():
    w = work(ALIGNED, "f32", 1024, 2, wl.LossSpec("iid", 0.1), 1)
    g = H.GpuRound(w)
    b = g.buf
    with pytest.raises(dblp.DblpError) as e:
        dblp.Plan([100], "f32", 1000, 2)                     # payload not a multiple of 16
    assert e.value.status == -2
    with pytest.raises(dblp.DblpError) as e:
        dblp.Plan([100, 0], "f32", 1024, 2)                  # empty tensor
    assert e.value.status == -1
    with pytest.raises(dblp.DblpError) as e:
        dblp.Plan([100], "f32", 1024, 2, bucket_seq_bounds=[0, 5])   # bounds must end at C
    assert e.value.status == -1
    with pytest.raises(dblp.DblpError) as e:                 # misaligned ring
        dblp.dblp_packetize(g.plan, wl.make_grads(w, H.DEV), 1, b["hdr_ring"], b["payload_ring"][4:])
    assert e.value.status == -2
    with pytest.raises(dblp.DblpError) as e:                 # workspace too small
        dblp.dblp_apply_loss(g.plan, dblp.loss_model("none"), 1, 1, 0, b["delivered_bits"], b["arrival"],
                             b["n_arrived"], b["ws"][:1])
    assert e.value.status == -3
    with pytest.raises(dblp.DblpError) as e:                 # threshold above 2^32
        dblp.dblp_apply_loss(g.plan, dblp.loss_model("iid", t_drop=(1 << 32) + 1), 1, 1, 0, b["delivered_bits"],
                             b["arrival"], b["n_arrived"], b["ws"])
    assert e.value.status == -1
    with pytest.raises(dblp.DblpError) as e:
        dblp.dblp_check_bound(g.plan, b["recv_bitmap"], [1, 2, 3], b["recv_cnt"], b["missing_cnt"], b["ok"], b["all_ok"])
    assert e.value.status == -1
    torch.cuda.synchronize()                                  # the context is still healthy
    g.close()


def test_claim_then_bitmap_equals_book():
    w = work(RAGGED, "f32", 1408, 4, wl.LossSpec("iid", 0.2), 61)
    op = orc.Plan(w.numel, 4, 1408, 4)
    gm, om = H.models_for(w, op.C)
    g = H.GpuRound(w)
    b = g.buf
    g.packetize(wl.make_grads(w, H.DEV), w.round)
    o_hdr = op.headers(w.round)
    st = op.new_state()
    for attempt in range(2):                                   # the second call sees cells already claimed
        g.apply_loss(gm, w.seed, w.round, attempt)
        dblp.dblp_aggregate_claim(g.plan, b["hdr_ring"], op.M, b["arrival"], b["n_arrived"], op.M, w.round, b["slot_key"],
                                  b["counters"])
        dblp.dblp_aggregate_bitmap(g.plan, b["slot_key"], b["n_arrived"], op.M, b["recv_bitmap"], b["counters"])
        o_del, _ = op.loss_mask(om, w.seed, w.round, attempt)
        o_arr, o_n = op.arrival(o_del, w.seed, w.round, attempt)
        st = op.book(o_hdr, o_arr, o_n, w.round, st)
        H.compare_state(g, st, op)
    g.close()


def test_library_counts_its_launches():
    w = work(ALIGNED, "f32", 1024, 2, wl.LossSpec("ge", 0.1, 5.0), 1)
    g = H.GpuRound(w)
    gm, _ = H.models_for(w, g.plan.C)
    n0 = dblp.dblp_launch_count()
    g.packetize(wl.make_grads(w, H.DEV), 1)
    g.apply_loss(gm, 1, 1)
    g.aggregate(1)
    g.check_bound(1000)
    assert dblp.dblp_launch_count() - n0 == 1 + 6 + 3 + 1
    n0 = dblp.dblp_launch_count()
    dblp.dblp_round_device(g.plan, wl.make_grads(w, H.DEV), gm, 1, 2, 1000, dblp.DBLP_SUM, g.buf)
    assert dblp.dblp_launch_count() - n0 == 1 + 1 + 6 + 3 + 1          # the whole round starts with the reset kernel
    torch.cuda.synchronize()
    g.close()
