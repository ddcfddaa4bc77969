"""Thin ctypes binding of libdblp.so: argument marshalling only, same names as include/dblp.h.

Device buffers are torch tensors (torch is used for device memory and streams, nothing else).  Every step of the path
runs in the library's kernels; if the library has not been built, loading fails with an error -- there is no fallback.
"""
import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdblp.so")

DBLP_F32, DBLP_BF16 = 0, 1
DBLP_LOSS_NONE, DBLP_LOSS_IID, DBLP_LOSS_GE, DBLP_LOSS_MICROBURST = 0, 1, 2, 3
DBLP_SUM, DBLP_MEAN, DBLP_OUT_BF16 = 0, 1, 2
LOSS_KINDS = {"none": DBLP_LOSS_NONE, "iid": DBLP_LOSS_IID, "ge": DBLP_LOSS_GE, "microburst": DBLP_LOSS_MICROBURST}
HDR_BYTES = 32
COUNTER_FIELDS = ("n_arrived", "n_accepted", "n_dup", "n_stale", "n_invalid", "n_late")


class dblp_loss_model_t(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("pad", C.c_uint32), ("t_drop", C.c_uint64), ("t_gb", C.c_uint64),
                ("t_bg", C.c_uint64), ("t_init_bad", C.c_uint64), ("t_drop_good", C.c_uint64),
                ("t_drop_bad", C.c_uint64), ("window_len", C.c_uint64), ("t_drop_in", C.c_uint64),
                ("t_drop_out", C.c_uint64)]


class dblp_counters_t(C.Structure):
    _fields_ = [("n_arrived", C.c_uint64), ("n_accepted", C.c_uint64), ("n_dup", C.c_uint64),
                ("n_stale", C.c_uint64), ("n_invalid", C.c_uint64), ("n_late", C.c_uint64), ("status", C.c_uint32),
                ("pad", C.c_uint32)]


class dblp_device_buffers_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("grads", "hdr_ring", "payload_ring", "delivered_bits", "arrival",
                                          "n_arrived", "recv_bitmap", "slot_key", "counters", "agg", "recv_cnt",
                                          "missing_cnt", "ok", "all_ok", "ws")] + [("ws_bytes", C.c_size_t),
                                                                                   ("sent_bits", C.c_void_p)]


MARK_FIELDS = ("begin", "packetize_end", "loss_begin", "loss_end", "receive_begin", "claim_end", "reduce_end",
               "bound_begin", "bound_end", "end")


class dblp_round_marks_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in MARK_FIELDS]


class RoundMarks:
    """Timing events for the stages of a whole-round call (torch events; the library records them)."""

    def __init__(self):
        self.events = {n: torch.cuda.Event(enable_timing=True) for n in MARK_FIELDS}
        for e in self.events.values():
            e.record()                      # torch creates the CUDA event on first use; the library needs the handle
        self.struct = dblp_round_marks_t(**{n: e.cuda_event for n, e in self.events.items()})

    def ms(self, first, last):
        return self.events[first].elapsed_time(self.events[last])


class DblpError(RuntimeError):
    def __init__(self, status, what):
        super().__init__("%s: %s (%d): %s" % (what, lib().dblp_strerror(status).decode(), status,
                                              lib().dblp_last_error().decode()))
        self.status = status


_lib = None
EXPORTS = ("dblp_plan_create", "dblp_plan_destroy", "dblp_plan_query", "dblp_plan_tune_reduce", "dblp_plan_set_wire_format",
           "dblp_plan_set_shard",
           "dblp_workspace_bytes",
           "dblp_loss_model_from_rates", "dblp_packetize", "dblp_apply_loss", "dblp_apply_loss_static",
           "dblp_apply_loss_resend", "dblp_missing_bits", "dblp_stop_workspace_bytes", "dblp_aggregate_book_stop",
           "dblp_round_until_stop",
           "dblp_aggregate_book",
           "dblp_aggregate_claim", "dblp_aggregate_claim_grouped", "dblp_claim_workspace_bytes", "dblp_aggregate_bitmap", "dblp_aggregate_reduce", "dblp_aggregate_reduce_ex", "dblp_aggregate_reduce_atomic", "dblp_norm_scratch_count", "dblp_aggregate", "dblp_round_reset", "dblp_check_bound", "dblp_bound_ok", "dblp_clr",
           "dblp_select_bound", "dblp_round_send", "dblp_round_receive", "dblp_round_device", "dblp_round_host",
           "dblp_strerror", "dblp_last_error", "dblp_launch_count")


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libdblp.so is not built: run `python -m paper_2605_01989_b200.build` "
                              "(needs nvcc); there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        L.dblp_strerror.restype = C.c_char_p
        L.dblp_last_error.restype = C.c_char_p
        L.dblp_launch_count.restype = C.c_uint64
        L.dblp_select_bound.restype = C.c_uint32
        L.dblp_select_bound.argtypes = [C.c_double, C.c_double, C.c_double, C.c_uint32, C.c_uint32, C.c_int, C.c_int,
                                        C.c_uint32]
        L.dblp_clr.argtypes = [C.c_double, C.c_double, C.c_double]
        L.dblp_loss_model_from_rates.argtypes = [C.c_int, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double,
                                                 C.c_uint64, C.POINTER(dblp_loss_model_t)]
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc, what):
    if rc != 0:
        raise DblpError(rc, what)


def loss_model(kind, **fields):
    m = dblp_loss_model_t()
    m.kind = LOSS_KINDS[kind] if isinstance(kind, str) else int(kind)
    for k, v in fields.items():
        setattr(m, k, int(v))
    return m


def dblp_loss_model_from_rates(kind, mean_loss=0.0, mean_burst_len=20.0, window_frac=0.05, p_in=0.3, p_out=0.001, C_=0):
    m = dblp_loss_model_t()
    _check(lib().dblp_loss_model_from_rates(LOSS_KINDS[kind] if isinstance(kind, str) else kind, mean_loss,
                                            mean_burst_len, window_frac, p_in, p_out, C_, C.byref(m)),
           "dblp_loss_model_from_rates")
    return m


class Plan:
    """Owns a dblp_plan_t.  Create it with the CUDA device that holds the buffers current."""

    def __init__(self, tensor_numel, dtype, payload_bytes, W, bucket_seq_bounds=None):
        numel = (C.c_uint64 * len(tensor_numel))(*[int(n) for n in tensor_numel])
        dt = {"f32": DBLP_F32, "bf16": DBLP_BF16}[dtype] if isinstance(dtype, str) else int(dtype)
        if bucket_seq_bounds is None:
            bb, B = None, 1
        else:
            bb, B = (C.c_uint64 * len(bucket_seq_bounds))(*[int(b) for b in bucket_seq_bounds]), len(bucket_seq_bounds) - 1
        self.handle = C.c_void_p()
        _check(lib().dblp_plan_create(numel, C.c_uint32(len(tensor_numel)), C.c_int(dt), C.c_uint32(payload_bytes),
                                      C.c_uint32(W), bb, C.c_uint32(B), C.byref(self.handle)), "dblp_plan_create")
        c, n, m, rw = C.c_uint64(), C.c_uint64(), C.c_uint64(), C.c_uint64()
        _check(lib().dblp_plan_query(self.handle, C.byref(c), C.byref(n), C.byref(m), C.byref(rw)), "dblp_plan_query")
        self.C, self.N, self.M, self.row_words = int(c.value), int(n.value), int(m.value), int(rw.value)
        self.T, self.W, self.B, self.P = len(tensor_numel), int(W), B, int(payload_bytes)
        self.es = 4 if dt == DBLP_F32 else 2
        self.torch_dtype = torch.float32 if dt == DBLP_F32 else torch.bfloat16
        ws = C.c_size_t()
        _check(lib().dblp_workspace_bytes(self.handle, C.byref(ws)), "dblp_workspace_bytes")
        self.workspace_bytes = int(ws.value)

    def set_wire_format(self, datagrams):
        """True: one ring of (32 + P)-byte datagrams (pass it as both hdr_ring and payload_ring); False: two rings."""
        _check(lib().dblp_plan_set_wire_format(self.handle, C.c_int(1 if datagrams else 0)), "dblp_plan_set_wire_format")
        self.datagrams = bool(datagrams)

    def set_shard(self, stream_chunks, seq_offset):
        """This plan is the chunks seq_offset .. seq_offset + C - 1 of worker streams of stream_chunks chunks."""
        _check(lib().dblp_plan_set_shard(self.handle, C.c_uint64(stream_chunks), C.c_uint64(seq_offset)), "dblp_plan_set_shard")
        ws = C.c_size_t()
        _check(lib().dblp_workspace_bytes(self.handle, C.byref(ws)), "dblp_workspace_bytes")
        self.workspace_bytes = int(ws.value)

    def tune_reduce(self, chunks_per_tile=0, grid_blocks=0):
        _check(lib().dblp_plan_tune_reduce(self.handle, C.c_uint32(chunks_per_tile), C.c_uint32(grid_blocks)),
               "dblp_plan_tune_reduce")

    def close(self):
        if self.handle:
            lib().dblp_plan_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def alloc_round(self, device, n_slots=None, arrival_cap=None):
        """Device buffers of one round, sized from the plan (torch is the allocator)."""
        n_slots = self.M if n_slots is None else n_slots
        cap = self.M if arrival_cap is None else arrival_cap
        stop_ws = C.c_size_t()
        _check(lib().dblp_stop_workspace_bytes(self.handle, C.c_uint64(cap), C.byref(stop_ws)), "dblp_stop_workspace_bytes")
        claim_ws = C.c_size_t()
        _check(lib().dblp_claim_workspace_bytes(self.handle, C.c_uint64(n_slots), C.c_uint64(cap), C.byref(claim_ws)),
               "dblp_claim_workspace_bytes")
        ws_bytes = max(self.workspace_bytes, int(stop_ws.value), int(claim_ws.value))
        u8, u32, i64 = torch.uint8, torch.int32, torch.int64
        z = lambda n, dt: torch.zeros(n, dtype=dt, device=device)
        return {
            "hdr_ring": z(n_slots * HDR_BYTES, u8), "payload_ring": torch.empty(n_slots * self.P, dtype=u8, device=device),
            "delivered_bits": z(self.W * self.row_words, u32), "arrival": z(cap, u32), "n_arrived": z(1, i64),
            "recv_bitmap": z(self.W * self.row_words, u32), "slot_key": z(self.W * self.C, i64),
            "counters": z(7, i64), "agg": torch.empty(self.N, dtype=torch.float32, device=device),
            "recv_cnt": z(self.W * self.B, u32), "missing_cnt": z(self.W * self.B, u32),
            "ok": z(self.W * self.B, u8), "all_ok": z(1, u32),
            "ws": z((ws_bytes + 7) // 8, i64), "sent_bits": z(self.W * self.row_words, u32),
            "n_slots": n_slots, "arrival_cap": cap,
        }


def dblp_packetize(plan, grads, round, hdr_ring, payload_ring, stream=None):
    ptrs = (C.c_void_p * plan.W)(*[g.data_ptr() for g in grads])
    _check(lib().dblp_packetize(plan.handle, ptrs, C.c_uint32(round), _ptr(hdr_ring), _ptr(payload_ring),
                                _stream(stream)), "dblp_packetize")


def dblp_apply_loss(plan, model, seed, round, attempt, delivered_bits, arrival, n_arrived_dev, ws, stream=None):
    _check(lib().dblp_apply_loss(plan.handle, C.byref(model), C.c_uint64(seed), C.c_uint32(round), C.c_uint32(attempt),
                                 _ptr(delivered_bits), _ptr(arrival), _ptr(n_arrived_dev), _ptr(ws),
                                 C.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "dblp_apply_loss")


STATIC_SCRATCH_BYTES = 4 * 1024 * 1024 + 64 * 1024


def dblp_apply_loss_static(plan, model, seed, round, attempt, delivered_bits, arrival, n_arrived_dev, stream=None):
    """dblp_apply_loss for callers that may not allocate device memory: the scratch is a fixed array inside the
    library (plans up to STATIC_SCRATCH_BYTES of workspace).  All calls on a device share that array, so calls that
    could overlap on the GPU must be ordered by the caller."""
    _check(lib().dblp_apply_loss_static(plan.handle, C.byref(model), C.c_uint64(seed), C.c_uint32(round),
                                        C.c_uint32(attempt), _ptr(delivered_bits), _ptr(arrival), _ptr(n_arrived_dev),
                                        _stream(stream)), "dblp_apply_loss_static")


def dblp_missing_bits(plan, recv_bitmap, sent_bits, stream=None):
    _check(lib().dblp_missing_bits(plan.handle, _ptr(recv_bitmap), _ptr(sent_bits), _stream(stream)), "dblp_missing_bits")


def dblp_apply_loss_resend(plan, model, seed, round, attempt, sent_bits, delivered_bits, arrival, n_arrived_dev, ws,
                           stream=None):
    _check(lib().dblp_apply_loss_resend(plan.handle, C.byref(model), C.c_uint64(seed), C.c_uint32(round),
                                        C.c_uint32(attempt), _ptr(sent_bits), _ptr(delivered_bits), _ptr(arrival),
                                        _ptr(n_arrived_dev), _ptr(ws), C.c_size_t(ws.numel() * ws.element_size()),
                                        _stream(stream)), "dblp_apply_loss_resend")


def dblp_aggregate_book_stop(plan, hdr_ring, n_slots, arrival, n_arrived_dev, arrival_cap, round, bound_ppm,
                             recv_bitmap, slot_key, counters, ws, stream=None):
    _check(lib().dblp_aggregate_book_stop(plan.handle, _ptr(hdr_ring), C.c_uint64(n_slots), _ptr(arrival),
                                          _ptr(n_arrived_dev), C.c_uint64(arrival_cap), C.c_uint32(round),
                                          C.c_uint32(bound_ppm), _ptr(recv_bitmap), _ptr(slot_key), _ptr(counters),
                                          _ptr(ws), C.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "dblp_aggregate_book_stop")


def _device_buffers(dev, grads_dev=None):
    b = dblp_device_buffers_t()
    b.grads = grads_dev.data_ptr() if grads_dev is not None else 0
    for name in ("hdr_ring", "payload_ring", "delivered_bits", "arrival", "n_arrived", "recv_bitmap", "slot_key",
                 "counters", "agg", "recv_cnt", "missing_cnt", "ok", "all_ok", "ws", "sent_bits"):
        setattr(b, name, dev[name].data_ptr())
    b.ws_bytes = dev["ws"].numel() * dev["ws"].element_size()
    return b


def dblp_round_until_stop(plan, model, seed, round, bound_ppm, max_attempts, early_stop, dev, stream=None):
    """Returns (attempts used, all_ok).  Blocks: the decision is read back after every attempt."""
    b = _device_buffers(dev)
    attempts, ok = C.c_uint32(), C.c_uint32()
    _check(lib().dblp_round_until_stop(plan.handle, C.byref(model), C.c_uint64(seed), C.c_uint32(round),
                                       C.c_uint32(bound_ppm), C.c_uint32(max_attempts), C.c_int(int(early_stop)),
                                       C.byref(b), C.byref(attempts), C.byref(ok), _stream(stream)),
           "dblp_round_until_stop")
    return int(attempts.value), int(ok.value)


def dblp_aggregate_book(plan, hdr_ring, n_slots, arrival, n_arrived_dev, arrival_cap, round, recv_bitmap, slot_key,
                        counters, stream=None):
    _check(lib().dblp_aggregate_book(plan.handle, _ptr(hdr_ring), C.c_uint64(n_slots), _ptr(arrival),
                                     _ptr(n_arrived_dev), C.c_uint64(arrival_cap), C.c_uint32(round), _ptr(recv_bitmap),
                                     _ptr(slot_key), _ptr(counters), _stream(stream)), "dblp_aggregate_book")


def dblp_aggregate_claim(plan, hdr_ring, n_slots, arrival, n_arrived_dev, arrival_cap, round, slot_key, counters,
                         stream=None):
    _check(lib().dblp_aggregate_claim(plan.handle, _ptr(hdr_ring), C.c_uint64(n_slots), _ptr(arrival), _ptr(n_arrived_dev),
                                      C.c_uint64(arrival_cap), C.c_uint32(round), _ptr(slot_key), _ptr(counters),
                                      _stream(stream)), "dblp_aggregate_claim")


def dblp_aggregate_claim_grouped(plan, hdr_ring, n_slots, arrival, n_arrived_dev, arrival_cap, round, slot_key, counters,
                                 ws, stream=None):
    _check(lib().dblp_aggregate_claim_grouped(plan.handle, _ptr(hdr_ring), C.c_uint64(n_slots), _ptr(arrival),
                                              _ptr(n_arrived_dev), C.c_uint64(arrival_cap), C.c_uint32(round), _ptr(slot_key),
                                              _ptr(counters), _ptr(ws), C.c_size_t(ws.numel() * ws.element_size()),
                                              _stream(stream)), "dblp_aggregate_claim_grouped")


def dblp_aggregate_bitmap(plan, slot_key, n_arrived_dev, arrival_cap, recv_bitmap, counters, stream=None):
    _check(lib().dblp_aggregate_bitmap(plan.handle, _ptr(slot_key), _ptr(n_arrived_dev), C.c_uint64(arrival_cap),
                                       _ptr(recv_bitmap), _ptr(counters), _stream(stream)), "dblp_aggregate_bitmap")


def dblp_aggregate_reduce(plan, payload_ring, slot_key, agg_out, flags=DBLP_SUM, stream=None):
    _check(lib().dblp_aggregate_reduce(plan.handle, _ptr(payload_ring), _ptr(slot_key), _ptr(agg_out),
                                       C.c_uint32(flags), _stream(stream)), "dblp_aggregate_reduce")


def dblp_aggregate_reduce_atomic(plan, payload_ring, slot_key, agg_out, flags=DBLP_SUM, stream=None):
    _check(lib().dblp_aggregate_reduce_atomic(plan.handle, _ptr(payload_ring), _ptr(slot_key), _ptr(agg_out),
                                              C.c_uint32(flags), _stream(stream)), "dblp_aggregate_reduce_atomic")


def dblp_norm_scratch_count(plan):
    n = C.c_uint64()
    _check(lib().dblp_norm_scratch_count(plan.handle, C.byref(n)), "dblp_norm_scratch_count")
    return int(n.value)


def dblp_aggregate_reduce_ex(plan, payload_ring, slot_key, agg_out, flags=DBLP_SUM, norm_scratch=None, norm_out=None,
                             params=None, lr=0.0, stream=None):
    _check(lib().dblp_aggregate_reduce_ex(plan.handle, _ptr(payload_ring), _ptr(slot_key), _ptr(agg_out),
                                          C.c_uint32(flags), _ptr(norm_scratch), _ptr(norm_out), _ptr(params),
                                          C.c_float(lr), _stream(stream)), "dblp_aggregate_reduce_ex")


def dblp_aggregate(plan, hdr_ring, payload_ring, n_slots, arrival, n_arrived_dev, arrival_cap, round, recv_bitmap,
                   slot_key, counters, agg_out, flags=DBLP_SUM, stream=None):
    _check(lib().dblp_aggregate(plan.handle, _ptr(hdr_ring), _ptr(payload_ring), C.c_uint64(n_slots), _ptr(arrival),
                                _ptr(n_arrived_dev), C.c_uint64(arrival_cap), C.c_uint32(round), _ptr(recv_bitmap),
                                _ptr(slot_key), _ptr(counters), _ptr(agg_out), C.c_uint32(flags), _stream(stream)),
           "dblp_aggregate")


def dblp_round_reset(plan, recv_bitmap, slot_key, counters, stream=None):
    _check(lib().dblp_round_reset(plan.handle, _ptr(recv_bitmap), _ptr(slot_key), _ptr(counters), _stream(stream)),
           "dblp_round_reset")


def dblp_check_bound(plan, recv_bitmap, bound_ppm, recv_cnt, missing_cnt, ok, all_ok, stream=None):
    bounds = [int(bound_ppm)] if isinstance(bound_ppm, int) else [int(b) for b in bound_ppm]
    arr = (C.c_uint32 * len(bounds))(*bounds)
    _check(lib().dblp_check_bound(plan.handle, _ptr(recv_bitmap), arr, C.c_uint32(len(bounds)), _ptr(recv_cnt),
                                  _ptr(missing_cnt), _ptr(ok), _ptr(all_ok), _stream(stream)), "dblp_check_bound")


def dblp_bound_ok(missing, total, bound_ppm):
    return bool(lib().dblp_bound_ok(C.c_uint64(missing), C.c_uint64(total), C.c_uint32(bound_ppm)))


def dblp_clr(norm_prev, norm_curr, eta=0.5):
    return bool(lib().dblp_clr(norm_prev, norm_curr, eta))


def dblp_select_bound(norm_prev, norm_curr, eta, p_low_ppm, p_high_ppm, at_epoch_start, first_iteration, current_ppm):
    return int(lib().dblp_select_bound(norm_prev, norm_curr, eta, p_low_ppm, p_high_ppm, int(at_epoch_start),
                                       int(first_iteration), current_ppm))


def _marks(marks):
    return C.byref(marks.struct) if marks is not None else None


def _grad_ptrs(plan, grads):
    return (C.c_void_p * plan.W)(*[g.data_ptr() for g in grads])


def dblp_round_send(plan, grads, model, seed, round, dev, marks=None, stream=None):
    b = _device_buffers(dev)
    _check(lib().dblp_round_send(plan.handle, _grad_ptrs(plan, grads), C.byref(model), C.c_uint64(seed), C.c_uint32(round),
                                 C.byref(b), _marks(marks), _stream(stream)), "dblp_round_send")


def dblp_round_receive(plan, round, bound_ppm, flags, dev, marks=None, stream=None):
    b = _device_buffers(dev)
    _check(lib().dblp_round_receive(plan.handle, C.c_uint32(round), C.c_uint32(bound_ppm), C.c_uint32(flags), C.byref(b),
                                    _marks(marks), _stream(stream)), "dblp_round_receive")


def dblp_round_device(plan, grads, model, seed, round, bound_ppm, flags, dev, marks=None, stream=None):
    """One whole round on device-resident gradients with the library's two-stream schedule."""
    b = _device_buffers(dev)
    _check(lib().dblp_round_device(plan.handle, _grad_ptrs(plan, grads), C.byref(model), C.c_uint64(seed),
                                   C.c_uint32(round), C.c_uint32(bound_ppm), C.c_uint32(flags), C.byref(b),
                                   _marks(marks), _stream(stream)), "dblp_round_device")


def dblp_round_host(plan, grads_host, model, seed, round, bound_ppm, flags, dev, grads_dev, agg_host=None,
                    counters_host=None, recv_cnt_host=None, missing_cnt_host=None, ok_host=None, all_ok_host=None,
                    stream=None):
    """grads_host: W host tensors (pinned recommended); dev: buffers from Plan.alloc_round; grads_dev: one device
    tensor of W*N elements; *_host: host tensors that receive the results (None to skip)."""
    ptrs = (C.c_void_p * plan.W)(*[g.data_ptr() for g in grads_host])
    b = _device_buffers(dev, grads_dev)
    _check(lib().dblp_round_host(plan.handle, ptrs, C.byref(model), C.c_uint64(seed), C.c_uint32(round),
                                 C.c_uint32(bound_ppm), C.c_uint32(flags), C.byref(b), _ptr(agg_host),
                                 _ptr(counters_host), _ptr(recv_cnt_host), _ptr(missing_cnt_host), _ptr(ok_host),
                                 _ptr(all_ok_host), _stream(stream)), "dblp_round_host")


def dblp_launch_count():
    return int(lib().dblp_launch_count())


def counters_dict(counters_tensor):
    v = counters_tensor.cpu().tolist()
    d = dict(zip(COUNTER_FIELDS, v[:6]))
    d["status"] = v[6] & 0xFFFFFFFF
    return d
