"""ctypes access to the CPU oracle (oracle/dblp_oracle.c).  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only tests, the smoke check and the bench's CPU-baseline leg import this module.  It holds argument
marshalling between numpy arrays and the C functions and nothing of the method itself.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

HDR_DTYPE = np.dtype([("seq", "<u4"), ("round", "<u4"), ("len_bytes", "<u4"), ("tensor_id", "<u4"),
                      ("offset_elems", "<u8"), ("worker", "<u4"), ("reserved", "<u4")])
assert HDR_DTYPE.itemsize == 32

NONE = 0xFFFFFFFF


class LossModel(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("pad", C.c_uint32), ("t_drop", C.c_uint64), ("t_gb", C.c_uint64),
                ("t_bg", C.c_uint64), ("t_init_bad", C.c_uint64), ("t_drop_good", C.c_uint64),
                ("t_drop_bad", C.c_uint64), ("window_len", C.c_uint64), ("t_drop_in", C.c_uint64),
                ("t_drop_out", C.c_uint64)]


class Counters(C.Structure):
    _fields_ = [("n_arrived", C.c_uint64), ("n_accepted", C.c_uint64), ("n_dup", C.c_uint64),
                ("n_stale", C.c_uint64), ("n_invalid", C.c_uint64), ("n_late", C.c_uint64), ("status", C.c_uint32),
                ("pad", C.c_uint32)]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k in ("n_arrived", "n_accepted", "n_dup", "n_stale", "n_invalid", "n_late")}


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.dblp_oracle_perm.restype = C.c_uint64
        _lib.dblp_oracle_perm.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
        _lib.dblp_oracle_clr.argtypes = [C.c_double, C.c_double, C.c_double]
        _lib.dblp_oracle_select_bound.restype = C.c_uint32
        _lib.dblp_oracle_select_bound.argtypes = [C.c_double, C.c_double, C.c_double, C.c_uint32, C.c_uint32,
                                                  C.c_int, C.c_int, C.c_uint32]
    return _lib


def set_threads(n):
    """Threads the one OpenMP loop (the reduce) may use; returns the count in effect."""
    omp = C.CDLL("libgomp.so.1")
    omp.omp_set_num_threads(int(n))
    return int(omp.omp_get_max_threads())


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _u64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint64))


def _check(rc, what):
    if rc != 0:
        raise RuntimeError("oracle %s failed: %d" % (what, rc))


def loss_model(kind, **kw):
    m = LossModel()
    m.kind = {"none": 0, "iid": 1, "ge": 2, "microburst": 3}[kind]
    for k, v in kw.items():
        setattr(m, k, int(v))
    return m


def philox(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().dblp_oracle_philox4x32_10(c, k, o)
    return [int(x) for x in o]


class Plan:
    """The constants of Section IV-A: tensor sizes, element size, payload size, worker count."""

    def __init__(self, numel, elem_size, payload_bytes, W):
        self.numel = _u64(numel)
        self.T = len(self.numel)
        self.es = int(elem_size)
        self.P = int(payload_bytes)
        self.W = int(W)
        self.base = np.zeros(self.T, np.uint64)
        self.chunkbase = np.zeros(self.T + 1, np.uint64)
        _check(lib().dblp_oracle_plan(_p(self.numel), C.c_uint32(self.T), C.c_uint32(self.es), C.c_uint32(self.P),
                                      _p(self.base), _p(self.chunkbase)), "plan")
        self.E = self.P // self.es
        self.C = int(self.chunkbase[self.T])
        self.N = int(self.numel.sum())
        self.M = self.C * self.W
        self.row_words = (self.C + 31) // 32

    def _args(self):
        return (_p(self.numel), C.c_uint32(self.T), C.c_uint32(self.es), C.c_uint32(self.P))

    def packetize(self, grads, rnd):
        """grads: list of W contiguous numpy arrays (float32 or uint16 for bf16 bit patterns)."""
        hdr = np.zeros(self.M, HDR_DTYPE)
        payload = np.empty(self.M * self.P, np.uint8)
        ptrs = (C.c_void_p * self.W)(*[g.ctypes.data for g in grads])
        _check(lib().dblp_oracle_packetize(*self._args(), C.c_uint32(self.W), ptrs, C.c_uint32(rnd),
                                           _p(hdr), _p(payload)), "packetize")
        return hdr, payload

    def headers(self, rnd):
        """Headers of all M packets without the payloads."""
        hdr = np.zeros(self.M, HDR_DTYPE)
        _check(lib().dblp_oracle_packetize(*self._args(), C.c_uint32(self.W), None, C.c_uint32(rnd), _p(hdr), None),
               "packetize(headers)")
        return hdr

    def header_at(self, w, seq, rnd):
        h = np.zeros(1, HDR_DTYPE)
        b = C.c_uint64()
        _check(lib().dblp_oracle_header_at(*self._args(), C.c_uint32(w), C.c_uint64(seq), C.c_uint32(rnd),
                                           _p(h), C.byref(b)), "header_at")
        return h[0], int(b.value)

    def loss_mask(self, model, seed, rnd, attempt=0, sent=None):
        """sent: bitmap of the chunks that are transmitted in this attempt (None = all)."""
        d = np.zeros(self.W * self.row_words, np.uint32)
        s0 = C.c_uint64()
        sp = None if sent is None else _p(np.ascontiguousarray(sent, np.uint32))
        _check(lib().dblp_oracle_loss_mask_sent(C.byref(model), C.c_uint64(self.C), C.c_uint32(self.W), C.c_uint64(seed),
                                                C.c_uint32(rnd), C.c_uint32(attempt), sp, _p(d), C.byref(s0)),
               "loss_mask")
        return d.reshape(self.W, self.row_words), int(s0.value)

    def missing_bits(self, bitmap):
        """The set a sender retransmits after a bitmap reply: chunks whose bit is 0."""
        out = np.zeros((self.W, self.row_words), np.uint32)
        lib().dblp_oracle_missing_bits(C.c_uint64(self.C), C.c_uint32(self.W),
                                       _p(np.ascontiguousarray(bitmap, np.uint32)), _p(out))
        return out

    def perm(self, seed, rnd, attempt, a, M=None):
        return int(lib().dblp_oracle_perm(self.M if M is None else M, seed, rnd, attempt, a))

    def arrival(self, delivered, seed, rnd, attempt=0):
        arr = np.zeros(self.M, np.uint32)
        n = C.c_uint64()
        d = np.ascontiguousarray(delivered, np.uint32)
        _check(lib().dblp_oracle_arrival(C.c_uint64(self.C), C.c_uint32(self.W), C.c_uint64(seed), C.c_uint32(rnd),
                                         C.c_uint32(attempt), _p(d), _p(arr), C.byref(n)), "arrival")
        return arr, int(n.value)

    def new_state(self):
        """Round state at its start (Algorithm 2: bitmap <- 0)."""
        return {"bitmap": np.zeros((self.W, self.row_words), np.uint32),
                "slot_of": np.full(self.W * self.C, NONE, np.uint32),
                "first_arrival": np.full(self.W * self.C, NONE, np.uint32),
                "counters": Counters()}

    def book(self, hdr, arrival, n_arrived, rnd, state, stop_ppm=None):
        """stop_ppm: None = every arrival is examined; a tolerance in ppm = each worker's receiver stops as soon as
        its own missing / total <= p holds (Algorithm 2) and later arrivals of that worker count as late."""
        hdr = np.ascontiguousarray(hdr)
        arrival = np.ascontiguousarray(arrival, np.uint32)
        _check(lib().dblp_oracle_book_stop(*self._args(), C.c_uint32(self.W), _p(hdr), C.c_uint64(len(hdr)),
                                           _p(arrival), C.c_uint64(n_arrived), C.c_uint32(rnd),
                                           C.c_int(0 if stop_ppm is None else 1),
                                           C.c_uint32(0 if stop_ppm is None else stop_ppm), _p(state["bitmap"]),
                                           _p(state["slot_of"]), _p(state["first_arrival"]),
                                           C.byref(state["counters"])), "book")
        return state

    def round_until_stop(self, hdr, model, seed, rnd, bound_ppm, max_attempts, early_stop, state=None):
        """Algorithm 1 + 2 as one loop: attempt k sends what the bitmap reports missing, the loss process and the
        arrival order are redrawn with the attempt number, the receiver books the arrivals, and the round ends when
        every worker's missing / total <= p (stop signal) or after max_attempts.  Returns (state, attempts used,
        all_ok, per-attempt arrival counts)."""
        state = self.new_state() if state is None else state
        arrived = []
        all_ok = 0
        attempts = 0
        for k in range(max_attempts):
            sent = self.missing_bits(state["bitmap"])
            d, _ = self.loss_mask(model, seed, rnd, k, sent)
            arr, n = self.arrival(d, seed, rnd, k)
            self.book(hdr, arr, n, rnd, state, bound_ppm if early_stop else None)
            arrived.append(n)
            attempts = k + 1
            all_ok = self.check_bound(state["bitmap"], bound_ppm)[3]
            if all_ok:
                break
        return state, attempts, all_ok, arrived

    def reduce(self, payload, state, mean=False):
        agg = np.empty(self.N, np.float32)
        _check(lib().dblp_oracle_reduce(*self._args(), C.c_uint32(self.W), _p(payload), _p(state["bitmap"]),
                                        _p(state["slot_of"]), C.c_int(int(mean)), _p(agg)), "reduce")
        return agg

    def reduce_at(self, bitmap, elem, vals, mean=False):
        """vals[w, k] = worker w's value at flat element elem[k] (float32, or uint16 bf16 patterns)."""
        elem = _u64(elem)
        vals = np.ascontiguousarray(vals)
        assert vals.shape == (self.W, len(elem)) and vals.dtype.itemsize == self.es
        out = np.empty(len(elem), np.float32)
        bitmap = np.ascontiguousarray(bitmap, np.uint32)
        _check(lib().dblp_oracle_reduce_at(*self._args(), C.c_uint32(self.W), _p(bitmap), C.c_uint64(len(elem)),
                                           _p(elem), _p(vals), C.c_int(int(mean)), _p(out)), "reduce_at")
        return out

    def check_bound(self, bitmap, bound_ppm, bucket_bounds=None):
        bitmap = np.ascontiguousarray(bitmap, np.uint32)
        if bucket_bounds is None:
            B, bb = 1, None
        else:
            bbv = _u64(bucket_bounds)
            B, bb = len(bbv) - 1, _p(bbv)
        ppm = np.ascontiguousarray(np.atleast_1d(np.asarray(bound_ppm, np.uint32)))
        recv = np.zeros((self.W, B), np.uint32)
        miss = np.zeros((self.W, B), np.uint32)
        ok = np.zeros((self.W, B), np.uint8)
        allok = C.c_uint32()
        _check(lib().dblp_oracle_check_bound(C.c_uint64(self.C), C.c_uint32(self.W), _p(bitmap), bb, C.c_uint32(B),
                                             _p(ppm), C.c_uint32(len(ppm)), _p(recv), _p(miss), _p(ok),
                                             C.byref(allok)), "check_bound")
        return recv, miss, ok, int(allok.value)


def clr(norm_prev, norm_curr, eta=0.5):
    return bool(lib().dblp_oracle_clr(norm_prev, norm_curr, eta))


def select_bound(norm_prev, norm_curr, eta, p_low_ppm, p_high_ppm, at_epoch_start, first_iteration, current_ppm):
    return int(lib().dblp_oracle_select_bound(norm_prev, norm_curr, eta, p_low_ppm, p_high_ppm,
                                              int(at_epoch_start), int(first_iteration), current_ppm))


def norm(g):
    """(sum of squares, L2 norm) of a float32 array, fp64."""
    g = np.ascontiguousarray(g, np.float32)
    s, n = C.c_double(), C.c_double()
    _check(lib().dblp_oracle_norm(_p(g), C.c_uint64(g.size), C.byref(s), C.byref(n)), "norm")
    return float(s.value), float(n.value)


def sgd_apply(params, g, lr):
    """params - lr * g per element in fp32 (multiply, then subtract); returns a new array."""
    out = np.ascontiguousarray(params, np.float32).copy()
    g = np.ascontiguousarray(g, np.float32)
    assert out.shape == g.shape
    lib().dblp_oracle_sgd_apply(_p(out), _p(g), C.c_float(lr), C.c_uint64(out.size))
    return out


def to_bf16(x):
    """float32 array -> uint16 bf16 patterns, round to nearest even."""
    x = np.ascontiguousarray(x, np.float32)
    out = np.empty(x.shape, np.uint16)
    lib().dblp_oracle_to_bf16(_p(x), _p(out), C.c_uint64(x.size))
    return out
