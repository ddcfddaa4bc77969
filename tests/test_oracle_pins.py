"""Pins for the CPU oracle: each checks it against something other than itself -- published known answers,
closed forms, identities that the definitions force, library routines on special cases, brute force on tiny
inputs.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import workloads as wl

TWO32 = 1 << 32


def popcount(a):
    return int(np.unpackbits(np.ascontiguousarray(a).view(np.uint8)).sum())


def bits_of(row_words, C):
    """Bitmap rows -> bool array [W, C] (bit seq%32 of word seq//32)."""
    b = np.unpackbits(np.ascontiguousarray(row_words).view(np.uint8).reshape(row_words.shape[0], -1),
                      axis=1, bitorder="little")
    return b[:, :C].astype(bool)


def rand_grads(plan, seed, dtype=np.float32):
    rng = np.random.default_rng(seed)
    if dtype == np.float32:
        return [(rng.standard_normal(plan.N) * 1e-3).astype(np.float32) for _ in range(plan.W)]
    t = [(torch.from_numpy(rng.standard_normal(plan.N).astype(np.float32)) * 1e-3).to(torch.bfloat16)
         for _ in range(plan.W)]
    return [x.view(torch.uint16).numpy().copy() for x in t]


# ------------------------------------------------------------------------------------------------ Philox
def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert orc.philox(v[0:4], v[4:6]) == v[6:10]


def test_philox_counter_and_key_sensitivity():
    base = orc.philox([1, 2, 3, 4], [5, 6])
    for i in range(4):
        c = [1, 2, 3, 4]
        c[i] ^= 1
        assert orc.philox(c, [5, 6]) != base
    assert orc.philox([1, 2, 3, 4], [5, 7]) != base and orc.philox([1, 2, 3, 4], [4, 6]) != base


# ------------------------------------------------------------------------------------------------ plan
@pytest.mark.parametrize("numel,es,P", [([1 << 20], 4, 1024), ([1000, 1, 352, 353, 7], 4, 1408),
                                        ([5000, 2048, 2049, 3], 2, 4096)])
def test_plan_closed_form(numel, es, P):
    p = orc.Plan(numel, es, P, 3)
    E = P // es
    assert p.C == sum(-(-n // E) for n in numel)
    assert list(p.base) == list(np.cumsum([0] + numel[:-1]))
    assert list(p.chunkbase) == list(np.cumsum([0] + [-(-n // E) for n in numel]))


def test_plan_counts_of_named_architectures():
    # parameter totals of the three architectures are public facts; C follows from them by the closed form
    for i, (T, N) in {1: (161, 25557032), 2: (391, 335141888), 3: (580, 1557611200)}.items():
        c = wl.config(i)
        p = orc.Plan(c.numel, c.elem_size, c.payload_bytes, c.W)
        assert (p.T, p.N) == (T, N)
        assert p.C == sum(-(-n // c.E) for n in c.numel) == c.C


# ------------------------------------------------------------------------------------------------ packetize
@pytest.mark.parametrize("es", [4, 2])
def test_packetize_reassembly_is_identity(es):
    numel = [1000, 1, 352 * 3, 353, 7, 4096]
    p = orc.Plan(numel, es, 1408, 3)
    grads = rand_grads(p, 1, np.float32 if es == 4 else np.uint16)
    hdr, pay = p.packetize(grads, rnd=7)
    pay = pay.reshape(p.M, p.P)
    assert int(hdr["len_bytes"].sum()) == p.W * p.N * es
    rebuilt = [np.zeros(p.N * es, np.uint8) for _ in range(p.W)]
    for s in range(p.M):                       # place every packet by what its header says, nothing else
        h = hdr[s]
        dst = (int(p.base[h["tensor_id"]]) + int(h["offset_elems"])) * es
        rebuilt[h["worker"]][dst:dst + h["len_bytes"]] = pay[s, :h["len_bytes"]]
        assert not pay[s, h["len_bytes"]:].any()                    # padding of short chunks is zero
        assert h["round"] == 7 and h["reserved"] == 0
    for w in range(p.W):
        assert rebuilt[w].tobytes() == grads[w].tobytes()
    # sequence numbers are unique per worker and cover [0, C)
    for w in range(p.W):
        assert sorted(hdr["seq"][hdr["worker"] == w]) == list(range(p.C))
    # slot of packet (w, seq) is w*C + seq
    assert np.array_equal(hdr["worker"].astype(np.int64) * p.C + hdr["seq"], np.arange(p.M))


def test_packetize_single_tensor_is_a_reshape():
    p = orc.Plan([256 * 37], 4, 1024, 2)
    grads = rand_grads(p, 2)
    hdr, pay = p.packetize(grads, rnd=0)
    assert np.array_equal(pay.view(np.float32).reshape(2, 37, 256), np.stack(grads).reshape(2, 37, 256))
    assert np.array_equal(hdr["offset_elems"], np.tile(np.arange(37) * 256, 2))
    assert (hdr["len_bytes"] == 1024).all() and (hdr["tensor_id"] == 0).all()


def test_header_at_matches_full_packetize():
    p = orc.Plan([1000, 1, 352, 353, 7], 4, 1408, 2)
    hdr, _ = p.packetize(rand_grads(p, 3), rnd=5)
    for w in range(2):
        for s in range(p.C):
            h, base = p.header_at(w, s, 5)
            assert h == hdr[w * p.C + s] and base == int(p.base[h["tensor_id"]])


# ------------------------------------------------------------------------------------------------ loss masks
def test_loss_thresholds_extremes():
    p = orc.Plan([256 * 1000], 4, 1024, 3)
    for kind, lo, hi in (("iid", dict(t_drop=0), dict(t_drop=TWO32)),
                         ("microburst", dict(window_len=50, t_drop_in=0, t_drop_out=0),
                          dict(window_len=50, t_drop_in=TWO32, t_drop_out=TWO32))):
        d, _ = p.loss_mask(orc.loss_model(kind, **lo), 1, 1)
        assert popcount(d) == p.M
        d, _ = p.loss_mask(orc.loss_model(kind, **hi), 1, 1)
        assert popcount(d) == 0
    d, _ = p.loss_mask(orc.loss_model("none"), 1, 1)
    assert popcount(d) == p.M
    # padding bits of the last word of a row stay zero
    assert p.C % 32 != 0 and not (d[:, -1] >> (p.C % 32)).any()


def test_iid_rate_within_binomial_interval():
    p = orc.Plan([256 * 200000], 4, 1024, 4)
    for prob in (0.01, 0.05, 0.2):
        d, _ = p.loss_mask(orc.loss_model("iid", t_drop=wl.threshold(prob)), 11, 3)
        lost = p.M - popcount(d)
        assert abs(lost - prob * p.M) < 5 * math.sqrt(p.M * prob * (1 - prob))
    # different seed / round / attempt give different masks
    m = orc.loss_model("iid", t_drop=wl.threshold(0.2))
    a = p.loss_mask(m, 11, 3, 0)[0]
    assert not np.array_equal(a, p.loss_mask(m, 12, 3, 0)[0])
    assert not np.array_equal(a, p.loss_mask(m, 11, 4, 0)[0])
    assert not np.array_equal(a, p.loss_mask(m, 11, 3, 1)[0])
    assert np.array_equal(a, p.loss_mask(m, 11, 3, 0)[0])


def test_microburst_window():
    C = 100000
    p = orc.Plan([256 * C], 4, 1024, 4)
    spec = wl.LossSpec("microburst", window_frac=0.05, p_in=0.30, p_out=0.001)
    th = spec.thresholds(C)
    assert th["window_len"] == 5000
    d, s0 = p.loss_mask(orc.loss_model("microburst", **th), 2, 1)
    assert 0 <= s0 <= C - 5000
    lost = ~bits_of(d, C)
    inside = lost[:, s0:s0 + 5000].sum()
    outside = lost.sum() - inside
    n_in, n_out = 4 * 5000, 4 * (C - 5000)
    assert abs(inside - 0.30 * n_in) < 5 * math.sqrt(n_in * 0.3 * 0.7)
    assert abs(outside - 0.001 * n_out) < 5 * math.sqrt(n_out * 0.001)
    # with certain loss inside and none outside the lost set is exactly one window, identical for every worker
    d, s0 = p.loss_mask(orc.loss_model("microburst", window_len=5000, t_drop_in=TWO32, t_drop_out=0), 2, 1)
    lost = ~bits_of(d, C)
    for w in range(4):
        assert np.array_equal(np.flatnonzero(lost[w]), np.arange(s0, s0 + 5000))


def test_gilbert_elliott_degenerate_chains():
    C = 1000
    p = orc.Plan([256 * C], 4, 1024, 3)
    ge = lambda **kw: orc.loss_model("ge", t_drop_good=0, t_drop_bad=TWO32, **kw)
    # never enters Bad
    assert popcount(p.loss_mask(ge(t_gb=0, t_bg=TWO32, t_init_bad=0), 5, 1)[0]) == p.M
    # starts Bad and never leaves
    assert popcount(p.loss_mask(ge(t_gb=0, t_bg=0, t_init_bad=TWO32), 5, 1)[0]) == 0
    # starts Good, always flips: G B G B ... -> odd seqs lost (the state is read before it is advanced)
    lost = ~bits_of(p.loss_mask(ge(t_gb=TWO32, t_bg=TWO32, t_init_bad=0), 5, 1)[0], C)
    assert np.array_equal(lost, np.tile(np.arange(C) % 2 == 1, (3, 1)))
    # starts Bad, leaves at once, never returns: exactly seq 0 lost
    lost = ~bits_of(p.loss_mask(ge(t_gb=0, t_bg=TWO32, t_init_bad=TWO32), 5, 1)[0], C)
    assert np.array_equal(np.argwhere(lost), [[0, 0], [1, 0], [2, 0]])
    # drop probabilities per state are honoured: Good drops everything, Bad nothing, chain stuck in Good
    m = orc.loss_model("ge", t_gb=0, t_bg=TWO32, t_init_bad=0, t_drop_good=TWO32, t_drop_bad=0)
    assert popcount(p.loss_mask(m, 5, 1)[0]) == 0


def test_gilbert_elliott_statistics_match_the_two_state_chain():
    C, W = 400000, 4
    p = orc.Plan([256 * C], 4, 1024, W)
    for pi, L in ((0.01, 20.0), (0.05, 20.0), (0.2, 20.0)):
        th = wl.LossSpec("ge", pi, L).thresholds(C)
        lost = ~bits_of(p.loss_mask(orc.loss_model("ge", **th), 7, 2)[0], C)
        # stationary loss = pi; runs of drops are geometric with mean L
        runs = []
        for w in range(W):
            x = np.concatenate(([0], lost[w].astype(np.int8), [0]))
            edges = np.flatnonzero(np.diff(x))
            runs.append(edges[1::2] - edges[0::2])
        runs = np.concatenate(runs)
        n_runs = len(runs)
        # a run's length has std ~ L, the loss count is a sum of n_runs such lengths
        assert abs(runs.mean() - L) < 5 * L / math.sqrt(n_runs)
        expect = pi * C * W
        assert abs(lost.sum() - expect) < 5 * L * math.sqrt(2 * expect / L)


# ------------------------------------------------------------------------------------------------ permutation
def test_permutation_is_a_bijection_for_every_small_M():
    for M in list(range(1, 600)) + [1023, 1024, 1025, 4095, 4096, 4097, 16384, 16385, 65537]:
        p = orc.Plan([M], 4, 4, 1)            # one element per packet: C = M
        assert p.M == M
        full = np.full((1, p.row_words), 0xFFFFFFFF, np.uint32)
        arr, n = p.arrival(full, seed=M, rnd=1)
        assert n == M and np.array_equal(np.sort(arr[:n]), np.arange(M))


def test_permutation_depends_on_seed_round_attempt_and_is_not_the_identity():
    p = orc.Plan([5000], 4, 4, 1)
    full = np.full((1, p.row_words), 0xFFFFFFFF, np.uint32)
    a = p.arrival(full, 1, 1, 0)[0]
    assert (a != np.arange(5000)).mean() > 0.99
    for other in (p.arrival(full, 2, 1, 0)[0], p.arrival(full, 1, 2, 0)[0], p.arrival(full, 1, 1, 1)[0]):
        assert (a != other).mean() > 0.99
    assert all(p.perm(1, 1, 0, i) == a[i] for i in range(0, 5000, 97))
    # roughly uniform: position of element i is uncorrelated with i
    assert abs(np.corrcoef(a.astype(float), np.arange(5000))[0, 1]) < 0.05


def test_arrival_list_is_the_delivered_set_in_permuted_order():
    p = orc.Plan([256 * 777], 4, 1024, 3)
    d, _ = p.loss_mask(orc.loss_model("iid", t_drop=wl.threshold(0.2)), 9, 1)
    arr, n = p.arrival(d, 9, 1)
    assert n == popcount(d)
    assert len(set(arr[:n].tolist())) == n
    got = np.zeros(p.M, bool)
    got[arr[:n]] = True
    assert np.array_equal(got.reshape(3, p.C), bits_of(d, p.C))
    order = [p.perm(9, 1, 0, a) for a in range(p.M)]
    assert arr[:n].tolist() == [x for x in order if got[x]]


# ------------------------------------------------------------------------------------------------ bookkeeping
def _round(p, grads, model, seed, rnd=1):
    hdr, pay = p.packetize(grads, rnd)
    d, _ = p.loss_mask(model, seed, rnd)
    arr, n = p.arrival(d, seed, rnd)
    st = p.book(hdr, arr, n, rnd, p.new_state())
    return hdr, pay, d, arr, n, st


def test_book_counts_each_received_packet_exactly_once():
    p = orc.Plan([1000, 1, 352 * 40, 353, 7], 4, 1408, 4)
    hdr, pay, d, arr, n, st = _round(p, rand_grads(p, 4), orc.loss_model("iid", t_drop=wl.threshold(0.1)), 21)
    c = st["counters"].as_dict()
    assert c == {"n_arrived": n, "n_accepted": n, "n_dup": 0, "n_stale": 0, "n_invalid": 0, "n_late": 0}
    assert np.array_equal(st["bitmap"], d)                      # received bitmap = delivered mask
    assert popcount(st["bitmap"]) == n                          # loss fraction = popcount of the mask
    sel = st["slot_of"] != orc.NONE
    assert sel.sum() == n and np.array_equal(np.flatnonzero(sel), np.sort(arr[:n]))
    assert np.array_equal(st["slot_of"][sel], np.flatnonzero(sel))
    pos = np.empty(p.M, np.int64)
    pos[arr[:n]] = np.arange(n)
    assert np.array_equal(st["first_arrival"][sel], pos[sel])


def test_book_drops_stale_duplicate_and_invalid_packets():
    p = orc.Plan([1000, 352 * 10, 7], 4, 1408, 2)
    grads = rand_grads(p, 5)
    hdr, pay = p.packetize(grads, rnd=3)
    M = p.M
    junk = np.zeros(8, orc.HDR_DTYPE)
    junk[0] = hdr[2]; junk[0]["round"] = 2                      # stale (older round)
    junk[1] = hdr[3]; junk[1]["round"] = 4                      # stale (newer round)
    junk[2] = hdr[5]                                            # duplicate of slot 5, arrives after it
    junk[3] = hdr[6]; junk[3]["worker"] = 2                     # worker out of range
    junk[4] = hdr[6]; junk[4]["tensor_id"] = 3                  # tensor out of range
    junk[5] = hdr[6]; junk[5]["offset_elems"] += 1              # not on a chunk boundary
    junk[6] = hdr[6]; junk[6]["len_bytes"] -= 4                 # wrong length
    junk[7] = hdr[6]; junk[7]["seq"] += 1                       # seq contradicts (tensor, offset)
    ring = np.concatenate([hdr, junk])
    arrival = np.array([5, 0, M + 0, M + 1, M + 2, M + 3, M + 4, M + 5, M + 6, M + 7, M + 8, 1, 5, M + 2],
                       np.uint32)                               # M+8 is outside the ring
    st = p.book(ring, arrival, len(arrival), 3, p.new_state())
    assert st["counters"].as_dict() == {"n_arrived": 14, "n_accepted": 3, "n_dup": 3, "n_stale": 2, "n_invalid": 6, "n_late": 0}
    assert popcount(st["bitmap"]) == 3
    assert st["slot_of"][5] == 5 and st["first_arrival"][5] == 0          # first arrival keeps the slot
    # a duplicate that arrives BEFORE the original wins the slot instead
    st = p.book(ring, np.array([M + 2, 5], np.uint32), 2, 3, p.new_state())
    assert st["slot_of"][5] == M + 2 and st["counters"].n_dup == 1
    # continuing the round: arrival numbers go on counting, earlier attempt keeps its slots
    st = p.book(ring, np.array([5, 7], np.uint32), 2, 3, st)
    assert st["slot_of"][5] == M + 2 and st["slot_of"][7] == 7 and st["first_arrival"][7] == 3
    assert st["counters"].as_dict() == {"n_arrived": 4, "n_accepted": 2, "n_dup": 2, "n_stale": 0, "n_invalid": 0, "n_late": 0}


# ------------------------------------------------------------------------------------------------ reduce
def test_zero_loss_is_the_plain_left_to_right_sum():
    p = orc.Plan([1000, 1, 352 * 5, 353, 7], 4, 1408, 5)
    grads = rand_grads(p, 6)
    hdr, pay, d, arr, n, st = _round(p, grads, orc.loss_model("none"), 1)
    expect = np.zeros(p.N, np.float32)
    for g in grads:                                            # textbook: acc += g[w], fp32, worker order
        expect = expect + g
    assert p.reduce(pay, st).tobytes() == expect.tobytes()
    assert p.reduce(pay, st, mean=True).tobytes() == (expect / np.float32(5)).tobytes()


def test_total_loss_is_positive_zero_everywhere():
    p = orc.Plan([1000, 7], 4, 1408, 3)
    hdr, pay, d, arr, n, st = _round(p, rand_grads(p, 7), orc.loss_model("iid", t_drop=TWO32), 1)
    assert n == 0
    for mean in (False, True):
        assert not p.reduce(pay, st, mean).view(np.uint32).any()            # +0.0 has the all-zero pattern


def test_lone_negative_zero_sums_to_positive_zero():
    p = orc.Plan([8], 4, 16, 2)
    grads = [np.full(8, -0.0, np.float32), np.full(8, -0.0, np.float32)]
    hdr, pay, d, arr, n, st = _round(p, grads, orc.loss_model("none"), 1)
    assert not p.reduce(pay, st).view(np.uint32).any()


def test_single_worker_reconstruction_zero_fills_lost_chunks():
    p = orc.Plan([1000, 1, 352 * 50, 353], 4, 1408, 1)
    grads = rand_grads(p, 8)
    hdr, pay, d, arr, n, st = _round(p, grads, orc.loss_model("iid", t_drop=wl.threshold(0.3)), 3)
    got = p.reduce(pay, st)
    keep = np.zeros(p.N, bool)
    for s in range(p.M):
        if bits_of(d, p.C)[0, hdr[s]["seq"]]:
            b = int(p.base[hdr[s]["tensor_id"]]) + int(hdr[s]["offset_elems"])
            keep[b:b + hdr[s]["len_bytes"] // 4] = True
    assert 0.5 < keep.mean() < 0.9
    assert got.tobytes() == np.where(keep, grads[0] + np.float32(0), np.float32(0)).tobytes()


@pytest.mark.parametrize("es", [4, 2])
def test_result_is_invariant_to_arrival_order_and_matches_masked_sum(es):
    p = orc.Plan([1000, 1, 352 * 20, 353, 7], es, 1408, 6)
    grads = rand_grads(p, 9, np.float32 if es == 4 else np.uint16)
    model = orc.loss_model("iid", t_drop=wl.threshold(0.25))
    hdr, pay = p.packetize(grads, 1)
    d, _ = p.loss_mask(model, 5, 1)
    ref = None
    for perm_seed in (5, 6, 7, 8):
        arr, n = p.arrival(d, perm_seed, 1)
        st = p.book(hdr, arr, n, 1, p.new_state())
        out = p.reduce(pay, st)
        if ref is None:
            ref, ref_bm = out, st["bitmap"].copy()
        assert out.tobytes() == ref.tobytes() and np.array_equal(st["bitmap"], ref_bm)
        assert st["counters"].as_dict()["n_accepted"] == n
    # independent formulation: sum_w mask_w * g_w in float64
    E = p.E
    elem_chunk = np.concatenate([int(p.chunkbase[t]) + np.arange(int(p.numel[t])) // E for t in range(p.T)])
    mask = bits_of(d, p.C)[:, elem_chunk]
    if es == 4:
        g64 = np.stack(grads).astype(np.float64)
    else:
        g64 = np.stack([torch.from_numpy(g.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
                        for g in grads])
    exact = (mask * g64).sum(0)
    scale = np.abs(g64).sum(0) + 1e-30
    assert np.max(np.abs(ref - exact) / scale) <= 1e-6
    # the per-element entry point states the same definition
    elem = np.arange(0, p.N, 13)
    vals = np.stack(grads)[:, elem]
    assert p.reduce_at(d, elem, vals).tobytes() == ref[elem].tobytes()


def test_bf16_is_widened_exactly():
    p = orc.Plan([4096], 2, 4096, 1)
    pat = np.arange(0, 65536, 16, dtype=np.uint16)            # every 16th bf16 pattern incl. zeros, inf, nan
    assert len(pat) == 4096
    hdr, pay, d, arr, n, st = _round(p, [pat], orc.loss_model("none"), 1)
    got = p.reduce(pay, st)
    lib = torch.from_numpy(pat.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    finite = np.isfinite(lib)
    assert np.array_equal((lib[finite] + np.float32(0)).view(np.uint32), got[finite].view(np.uint32))
    assert np.array_equal(np.isnan(lib), np.isnan(got))


def test_mean_divides_by_all_workers_not_by_received_count():
    p = orc.Plan([256], 4, 1024, 4)
    grads = [np.full(256, float(w + 1), np.float32) for w in range(4)]
    hdr, pay = p.packetize(grads, 1)
    st = p.book(hdr, np.array([1, 3], np.uint32), 2, 1, p.new_state())   # only workers 1 and 3 arrive
    assert (p.reduce(pay, st) == 6.0).all() and (p.reduce(pay, st, mean=True) == 1.5).all()


# ------------------------------------------------------------------------------------------------ tolerance
def test_bound_equality_passes_with_the_papers_tolerances(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "tolerance_table.txt")) if l.strip() and l[0] != "#"]
    C = 1000
    p = orc.Plan([C], 4, 4, 2)
    for _, _, base, lo, hi in rows:
        assert abs(float(hi) - float(lo) - 40.0) < 1e-9 and base == lo       # P_high = p + 40 %, P_low = p
        for pct in (float(lo), float(hi)):
            ppm = round(pct * 10000)
            allowed = int(pct * 10)                     # chunks of 1000 that may be missing
            for missing, expect in ((allowed, 1), (allowed + 1, 0)):
                bm = bits_of(np.full((2, p.row_words), 0xFFFFFFFF, np.uint32), C)
                bm[1, 17:17 + missing] = False
                words = np.packbits(np.pad(bm, ((0, 0), (0, p.row_words * 32 - C))), axis=1,
                                    bitorder="little").view(np.uint32)
                recv, miss, ok, allok = p.check_bound(words, ppm)
                assert recv[:, 0].tolist() == [C, C - missing] and miss[:, 0].tolist() == [0, missing]
                assert ok[:, 0].tolist() == [1, expect] and allok == expect


def test_bound_zero_tolerance_and_buckets():
    C = 100
    p = orc.Plan([C], 4, 4, 1)
    bm = np.ones((1, 128), bool); bm[0, C:] = False; bm[0, [3, 40, 41, 99]] = False
    words = np.packbits(bm, axis=1, bitorder="little").view(np.uint32)
    assert p.check_bound(words, 0)[3] == 0
    recv, miss, ok, allok = p.check_bound(words, [0, 50000, 500000, 10000], bucket_bounds=[0, 3, 40, 42, 100])
    assert recv[0].tolist() == [3, 36, 0, 57] and miss[0].tolist() == [0, 1, 2, 1]
    assert ok[0].tolist() == [1, 1, 0, 0] and allok == 0
    assert p.check_bound(words, 1000000)[3] == 1


def test_clr_rule_boundaries():
    assert orc.clr(1.0, 0.5) and not orc.clr(1.0, 0.6) and orc.clr(1.0, 1.6) and orc.clr(1.0, 1.5)
    assert not orc.clr(1.0, 1.4) and orc.clr(0.0, 1.0) and orc.clr(2.0, 0.0) and not orc.clr(3.0, 3.0)


def test_bound_schedule_truth_table():
    lo, hi = 8000, 408000
    sb = lambda prev, cur, epoch, first, current: orc.select_bound(prev, cur, 0.5, lo, hi, epoch, first, current)
    assert sb(0, 0, True, True, hi) == lo                  # training starts at P_low
    assert sb(1.0, 0.9, False, False, lo) == lo            # mid-epoch: keep
    assert sb(1.0, 0.1, False, False, hi) == hi            # mid-epoch: keep even if the norm moved
    assert sb(1.0, 0.9, True, False, lo) == hi             # epoch start, calm: P_high
    assert sb(1.0, 0.4, True, False, hi) == lo             # epoch start, regime detected: P_low
    assert sb(1.0, 2.0, True, False, hi) == lo             # a rise triggers as well
