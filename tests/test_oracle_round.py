"""Pins for the oracle's round state machine: early stop (Algorithm 2, stop without a probe) and retransmission
attempts (Algorithm 1 + Section III-B).  Each is checked against an independent statement of the same rule in numpy,
closed forms of the geometric decay of the missing set, and degenerate chains.  CPU only."""
import math

import numpy as np
import pytest

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import workloads as wl

from test_oracle_pins import bits_of, popcount, rand_grads

TWO32 = 1 << 32


def need_of(C, ppm):
    """Fewest received chunks with missing / C <= ppm / 10^6."""
    return C - (ppm * C) // 1000000


def test_need_is_tight_for_the_papers_tolerances():
    for C in (1000, 72672, 163753, 7):
        for ppm in (0, 8000, 24000, 408000, 424000, 1000000):
            n = need_of(C, ppm)
            assert (C - n) * 1000000 <= ppm * C and (n == 0 or (C - n + 1) * 1000000 > ppm * C)


@pytest.mark.parametrize("ppm", [0, 8000, 100000, 408000, 1000000])
def test_early_stop_keeps_each_workers_first_arrivals_and_nothing_else(ppm):
    p = orc.Plan([352 * 200, 1000, 7], 4, 1408, 5)
    hdr = p.headers(3)
    full = np.full((p.W, p.row_words), 0xFFFFFFFF, np.uint32)
    arr, n = p.arrival(p.loss_mask(orc.loss_model("none"), 1, 3)[0], 9, 3)
    assert n == p.M
    st = p.book(hdr, arr, n, 3, p.new_state(), stop_ppm=ppm)
    need = need_of(p.C, ppm)
    # independent statement: of each worker's own arrival sequence, the first `need` entries are kept
    keep = np.zeros(p.M, bool)
    for w in range(p.W):
        mine = arr[arr // p.C == w]
        keep[mine[:need]] = True
    assert np.array_equal(bits_of(st["bitmap"], p.C).reshape(-1), keep.reshape(p.W, p.C).reshape(-1))
    c = st["counters"].as_dict()
    assert c["n_accepted"] == p.W * need and c["n_late"] == p.M - p.W * need and c["n_dup"] == 0
    recv, miss, ok, allok = p.check_bound(st["bitmap"], ppm)
    assert allok == 1 and (miss[:, 0] == p.C - need).all()
    if ppm == 0:
        ref = p.book(hdr, arr, n, 3, p.new_state())
        assert np.array_equal(ref["bitmap"], st["bitmap"]) and np.array_equal(ref["slot_of"], st["slot_of"])


def test_early_stop_counts_duplicates_before_the_stop_and_late_after_it():
    p = orc.Plan([256 * 10], 4, 1024, 1)                       # C = 10, need 8 at 20 %
    hdr = p.headers(1)
    arrival = np.array([0, 1, 1, 2, 3, 4, 5, 0, 6, 7, 7, 8, 9, 3], np.uint32)
    st = p.book(hdr, arrival, len(arrival), 1, p.new_state(), stop_ppm=200000)
    # accepted: 0 1 2 3 4 5 6 7 (the stop falls on the first 7); dups before it: second 1, second 0; late: 7 8 9 3
    assert st["counters"].as_dict() == {"n_arrived": 14, "n_accepted": 8, "n_dup": 2, "n_stale": 0, "n_invalid": 0,
                                        "n_late": 4}
    assert bits_of(st["bitmap"], 10)[0].tolist() == [True] * 8 + [False] * 2
    # a receiver that has already stopped ignores a whole further attempt
    st = p.book(hdr, np.array([8, 9], np.uint32), 2, 1, st, stop_ppm=200000)
    assert st["counters"].n_late == 6 and popcount(st["bitmap"]) == 8


def test_retransmission_sends_exactly_the_missing_chunks():
    p = orc.Plan([256 * 5000], 4, 1024, 3)
    m = orc.loss_model("iid", t_drop=wl.threshold(0.5))
    d0, _ = p.loss_mask(m, 4, 1, 0)
    sent = p.missing_bits(d0)
    assert np.array_equal(bits_of(sent, p.C), ~bits_of(d0, p.C))
    assert not (sent[:, -1] >> (p.C % 32)).any()                         # padding bits are not "missing"
    d1, _ = p.loss_mask(m, 4, 1, 1, sent)
    assert not (bits_of(d1, p.C) & ~bits_of(sent, p.C)).any()           # nothing arrives that was not sent
    n_sent = popcount(sent)
    assert abs(popcount(d1) - 0.5 * n_sent) < 5 * math.sqrt(n_sent * 0.25)
    # a sent packet's fate does not depend on what else is sent (memoryless process, per-packet draw)
    dall, _ = p.loss_mask(m, 4, 1, 1)
    assert np.array_equal(bits_of(d1, p.C), bits_of(dall, p.C) & bits_of(sent, p.C))


def test_burst_chain_advances_only_over_sent_packets():
    C = 2000
    p = orc.Plan([256 * C], 4, 1024, 2)
    flip = orc.loss_model("ge", t_gb=TWO32, t_bg=TWO32, t_init_bad=0, t_drop_good=0, t_drop_bad=TWO32)
    rng = np.random.default_rng(3)
    sent_bool = rng.random((2, C)) < 0.3
    sent = np.packbits(np.pad(sent_bool, ((0, 0), (0, p.row_words * 32 - C))), axis=1, bitorder="little").view(np.uint32)
    d, _ = p.loss_mask(flip, 1, 1, 2, sent)
    got = bits_of(d, C)
    for w in range(2):
        idx = np.flatnonzero(sent_bool[w])                      # Good, Bad, Good, ... over the packets actually sent
        assert np.array_equal(got[w, idx], np.arange(len(idx)) % 2 == 0)
        assert not got[w, ~sent_bool[w]].any()


@pytest.mark.parametrize("loss,ppm", [(0.6, 8000), (0.6, 408000), (0.9, 8000), (0.9, 408000), (0.7, 24000),
                                      (0.7, 424000)])
def test_attempts_follow_the_geometric_decay_of_the_missing_set(loss, ppm):
    """With i.i.d. loss q the missing share after k attempts is q^k, so the round needs about
    ceil(log(p) / log(q)) attempts: the mechanism behind the paper's latency tables (a high tolerance ends the round
    several times sooner under 60-90 % bursts)."""
    p = orc.Plan([256 * 20000], 4, 1024, 3)
    hdr = p.headers(1)
    m = orc.loss_model("iid", t_drop=wl.threshold(loss))
    st, attempts, ok, arrived = p.round_until_stop(hdr, m, 11, 1, ppm, 200, early_stop=False)
    expect = math.ceil(math.log(ppm / 1e6) / math.log(loss))
    assert ok == 1 and abs(attempts - expect) <= max(1, math.ceil(0.06 * expect))   # all three workers must pass
    assert sum(arrived) == popcount(st["bitmap"]) == st["counters"].n_accepted     # nothing is re-sent once it arrived
    assert st["counters"].n_dup == 0
    # early stop ends in the same attempt and leaves exactly the tolerated number missing where enough arrived
    st2, attempts2, ok2, _ = p.round_until_stop(hdr, m, 11, 1, ppm, 200, early_stop=True)
    assert ok2 == 1 and attempts2 == attempts
    miss = p.check_bound(st2["bitmap"], ppm)[1][:, 0]
    assert (miss == p.C - need_of(p.C, ppm)).all()
    assert not (bits_of(st2["bitmap"], p.C) & ~bits_of(st["bitmap"], p.C)).any()   # a subset of what arrived


def test_high_tolerance_ends_the_round_several_times_sooner():
    p = orc.Plan([256 * 20000], 4, 1024, 3)
    hdr = p.headers(1)
    speedups = []
    for loss in (0.6, 0.7, 0.8, 0.9):
        m = orc.loss_model("iid", t_drop=wl.threshold(loss))
        low = p.round_until_stop(hdr, m, 5, 1, 8000, 300, False)[1]
        high = p.round_until_stop(hdr, m, 5, 1, 408000, 300, False)[1]
        speedups.append(low / high)
    assert all(3.5 <= s <= 6.5 for s in speedups)               # the paper's Tables II-V report 4.0x - 5.97x


def test_round_gives_up_after_max_attempts():
    p = orc.Plan([256 * 100], 4, 1024, 2)
    st, attempts, ok, _ = p.round_until_stop(p.headers(1), orc.loss_model("iid", t_drop=TWO32), 1, 1, 8000, 4, False)
    assert attempts == 4 and ok == 0 and popcount(st["bitmap"]) == 0


# ------------------------------------------------------------------------------------------------ norm and update
def test_norm_is_the_exactly_rounded_sum_of_squares():
    rng = np.random.default_rng(0)
    for n, scale in ((1, 1.0), (7, 1e-3), (100003, 1e-3), (1 << 20, 1e-4), (50000, 1e10)):
        g = (rng.standard_normal(n) * scale).astype(np.float32)
        exact = math.fsum((g.astype(np.float64) ** 2).tolist())         # correctly rounded sum of the exact squares
        s, nrm = orc.norm(g)
        assert abs(s - exact) <= 2 * np.spacing(exact)
        assert nrm == math.sqrt(s)
    assert orc.norm(np.array([3.0, 4.0], np.float32)) == (25.0, 5.0)
    assert orc.norm(np.ones(4096, np.float32)) == (4096.0, 64.0)
    assert orc.norm(np.zeros(10, np.float32)) == (0.0, 0.0)
    g = (rng.standard_normal(1000) * 1e-3).astype(np.float32)
    assert orc.norm(2 * g)[0] == 4 * orc.norm(g)[0]                     # scaling by two is exact
    # a sum where naive accumulation loses the small terms: one large value and a million small ones
    g = np.concatenate([[4096.0], np.full(1 << 20, 2.0 ** -12)]).astype(np.float32)
    assert orc.norm(g)[0] == 4096.0 ** 2 + (1 << 20) * 2.0 ** -24


def test_sgd_apply_is_multiply_then_subtract_in_fp32():
    rng = np.random.default_rng(1)
    w = rng.standard_normal(100000).astype(np.float32)
    g = (rng.standard_normal(100000) * 1e-3).astype(np.float32)
    lr = np.float32(0.1)
    out = orc.sgd_apply(w, g, float(lr))
    two_step = w - (lr * g)                                              # numpy: two separately rounded fp32 operations
    assert out.tobytes() == two_step.tobytes()
    fused = (w.astype(np.float64) - np.float64(lr) * g.astype(np.float64)).astype(np.float32)
    assert (out != fused).any()                                          # it is NOT the fused multiply-add result
    assert orc.sgd_apply(w, g, 0.0).tobytes() == w.tobytes()
    assert orc.sgd_apply(w, np.zeros_like(g), 0.5).tobytes() == w.tobytes()   # lost chunks (zero-filled) change nothing


def test_bf16_rounding_matches_the_library_conversion():
    import torch
    rng = np.random.default_rng(2)
    x = np.concatenate([(rng.standard_normal(200000) * 1e-3).astype(np.float32),
                        rng.integers(0, 1 << 32, 200000, dtype=np.uint64).astype(np.uint32).view(np.float32),
                        np.array([0.0, -0.0, 1.0, np.inf, -np.inf, 3.3895314e38, 1.00390625, 1.01171875, 1e-40],
                                 np.float32)])
    got = orc.to_bf16(x)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    finite = ~np.isnan(x)
    assert np.array_equal(got[finite], lib[finite])
    assert ((got[~finite] & 0x7F80) == 0x7F80).all() and ((got[~finite] & 0x7F) != 0).all()     # NaN stays NaN
    # ties go to the even neighbour: 1 + 2^-8 is halfway between 1.0 (even) and 1 + 2^-7; 1 + 3*2^-8 rounds up to even
    assert orc.to_bf16(np.array([1.00390625, 1.01171875], np.float32)).tolist() == [0x3F80, 0x3F82]
