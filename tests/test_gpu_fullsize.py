"""GPU parity at the full sizes of the BERT-large-shaped (bf16) and GPT-2-XL-shaped (fp32) workloads, in the launch
configuration the bench times: the whole round goes through dblp_round_device (the library's two-stream schedule).  All integer results (headers, delivered bitmap, arrival list, received bitmap, slot
table, counters, bound decisions) are compared in full against the CPU oracle.  The payload ring and the fp32
aggregate are too large for the host, so they are checked (a) on sampled elements that the oracle computes one by
one from the workers' own values, and (b) in full on the device against properties that hold at any size: every
payload slot equals the gradient slice its oracle header names (padding zero), and the aggregate equals the
left-to-right fp32 sum over workers of (oracle mask ? g_w : 0), for the sum and for the mean, evaluated with elementwise
torch ops.  The sample always contains the places where a wrong chunk table would show: both ends of every tensor, every
element of every tensor's short last chunk, and the first element of each chunk that lost a packet and of the chunk
after it."""
import numpy as np
import pytest
import torch

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import binding as dblp
from paper_2605_01989_b200 import workloads as wl

import harness as H

pytestmark = pytest.mark.gpu


def _expand_mask(bits_row, chunk_len, N):
    """Per-chunk bool [C] -> per-element bool [N] on the device."""
    return torch.repeat_interleave(bits_row, chunk_len, output_size=N)


def _fullsize(work, n_samples=200000):
    free, _ = torch.cuda.mem_get_info()
    need = work.device_bytes() + 3 * work.N * 4 + 2 * work.N + (2 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of device memory, %.0f GB free" % (need / 1e9, free / 1e9))
    op = orc.Plan(work.numel, work.elem_size, work.payload_bytes, work.W)
    gm, om = H.models_for(work, op.C)
    rnd, seed = work.round, work.seed
    grads = wl.make_grads(work, H.DEV)
    g = H.GpuRound(work)
    dblp.dblp_round_device(g.plan, grads, gm, seed, rnd, work.bounds_ppm[0], dblp.DBLP_SUM, g.buf)
    torch.cuda.synchronize()
    first = H.compare_bound_outputs(g, op, None, work.bounds_ppm[0])     # as the round itself left them; checked below

    # ---- integer results, in full
    o_hdr = op.headers(rnd)
    H.assert_bits_equal(H.hdr_np(g.buf["hdr_ring"]), o_hdr, "header ring")
    o_del, _ = op.loss_mask(om, seed, rnd)
    o_arr, o_n = op.arrival(o_del, seed, rnd)
    assert g.n_arrived() == o_n
    H.assert_bits_equal(H.u32(g.buf["delivered_bits"]).reshape(op.W, op.row_words), o_del, "delivered bitmap")
    H.assert_bits_equal(H.u32(g.buf["arrival"])[:o_n], o_arr[:o_n], "arrival list")
    st = op.book(o_hdr, o_arr, o_n, rnd, op.new_state())
    H.compare_state(g, st, op)
    H.compare_bound_outputs(None, op, st["bitmap"], work.bounds_ppm[0], first)
    for ppm in work.bounds_ppm:
        H.compare_bound(g, op, st["bitmap"], ppm)

    # ---- payload ring, in full, on the device: slot (w, seq) holds the slice named by the oracle's header
    E, es, P = op.E, op.es, op.P
    ring = g.buf["payload_ring"].view(op.W, op.C, P)
    for t in range(op.T):
        n, b, c0 = int(op.numel[t]), int(op.base[t]), int(op.chunkbase[t])
        nch = -(-n // E)
        for w in range(op.W):
            rows = ring[w, c0:c0 + nch].reshape(-1)
            src = grads[w][b:b + n].view(torch.uint8)
            assert torch.equal(rows[:n * es], src), "payload of tensor %d worker %d" % (t, w)
            assert not rows[n * es:].any(), "padding of tensor %d worker %d" % (t, w)

    # ---- aggregate on sampled elements, one by one by the oracle
    rng = np.random.default_rng(seed)
    base, numel = op.base.astype(np.int64), op.numel.astype(np.int64)
    edges = np.concatenate([base, base + numel - 1])
    tails = [np.arange(base[t] + (numel[t] // E) * E, base[t] + numel[t]) for t in range(op.T) if numel[t] % E]
    chunk_first = np.concatenate([base[t] + np.arange(-(-int(numel[t]) // E), dtype=np.int64) * E for t in range(op.T)])
    got_all = np.unpackbits(o_del.view(np.uint8).reshape(op.W, -1), axis=1, bitorder="little")[:, :op.C].all(axis=0)
    lossy = np.flatnonzero(~got_all)                       # chunks that lost at least one worker's packet
    after = np.minimum(lossy + 1, op.C - 1)
    elem = np.unique(np.concatenate([rng.integers(0, op.N, n_samples), edges, [0, op.N - 1], chunk_first[lossy],
                                     chunk_first[after]] + tails))
    idx = torch.from_numpy(elem).to(H.DEV)
    vals = torch.stack([x[idx] for x in grads])
    vals = vals.view(torch.int16).cpu().numpy().view(np.uint16) if es == 2 else vals.cpu().numpy()
    for flags in (dblp.DBLP_SUM, dblp.DBLP_MEAN):
        g.reduce(flags)
        got = g.buf["agg"][idx].cpu().numpy()
        H.assert_bits_equal(got, op.reduce_at(o_del, elem, vals, mean=(flags == dblp.DBLP_MEAN)),
                            "sampled aggregate (flags %d)" % flags)

    # ---- aggregate, in full, against the masked left-to-right sum built from the oracle's bitmap
    chunk_len = torch.from_numpy(np.concatenate([
        np.minimum(E, int(op.numel[t]) - np.arange(-(-int(op.numel[t]) // E), dtype=np.int64) * E)
        for t in range(op.T)])).to(H.DEV)
    bits = np.unpackbits(o_del.view(np.uint8).reshape(op.W, -1), axis=1, bitorder="little")[:, :op.C].astype(bool)
    acc = torch.zeros(op.N, dtype=torch.float32, device=H.DEV)
    zero = torch.zeros((), dtype=torch.float32, device=H.DEV)
    for w in range(op.W):
        m = _expand_mask(torch.from_numpy(bits[w]).to(H.DEV), chunk_len, op.N)
        acc += torch.where(m, grads[w].float(), zero)
        del m
    g.reduce(dblp.DBLP_SUM)
    assert torch.equal(acc.view(torch.int32), g.buf["agg"].view(torch.int32)), "full aggregate vs masked sum"
    g.reduce(dblp.DBLP_MEAN)
    acc /= float(op.W)                                     # IEEE fp32 division, as the definition of the mean
    assert torch.equal(acc.view(torch.int32), g.buf["agg"].view(torch.int32)), "full mean vs masked sum / W"
    loss = 1.0 - o_n / op.M
    g.close()
    return loss


def test_config2_bert_large_shaped_bf16():
    loss = _fullsize(wl.config(2))
    assert 0.012 < loss < 0.02                      # 5 % of packets at 30 %, the rest at 0.1 %


def test_config3_gpt2_xl_shaped_fp32():
    loss = _fullsize(wl.config(3))
    assert 0.015 < loss < 0.025


def test_sweep_largest_points_that_fit():
    """The sweep's heaviest corners: 256 MiB buffers with 32 workers, 1 GiB buffers with 8."""
    for sz, W, P, lossrate, kind, seed in [(1 << 28, 32, 1024, 0.20, "ge", 13), (1 << 30, 8, 4096, 0.05, "iid", 14)]:
        _fullsize(wl.sweep_point(sz, W, P, lossrate, kind, seed), n_samples=50000)
