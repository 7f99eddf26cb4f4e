"""ctypes binding of libblink.so: argument marshalling only, same names as the C ABI.

Every step of the serving path runs in the CUDA library; this module only fills
structs, keeps the caller-owned torch buffers alive and decodes what comes back.
There is no CPU fallback: loading fails loudly when the library is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libblink.so")

BLINK_OK, BLINK_EAGAIN, BLINK_EINVAL, BLINK_ESTOPPED, BLINK_EDEVICE = 0, -1, -2, -3, -4
BLINK_ETIMEDOUT, BLINK_ENOMEM, BLINK_ECUDA, BLINK_ETOOBIG = -5, -6, -7, -8
SAMPLE_NOALLOC_MAX_ROWS = 1024
DTYPE_BF16, DTYPE_FP32 = 0, 1
EXEC_PERSISTENT, EXEC_STEPPED, EXEC_MANUAL, EXEC_HOST_GRAPH, EXEC_HOST_LAUNCHES = 0, 1, 2, 3, 4
GEMM_AUTO, GEMM_SIMT, GEMM_TC, GEMM_TC_PAIR = 0, 1, 2, 3
WEIGHTS_ROW_MAJOR, WEIGHTS_STREAMING = 0, 1
FUSION_AUTO, FUSION_OFF, FUSION_ON = 0, 1, 2
POLICY_CHUNKED, POLICY_PAUSE_RESUME = 0, 1
LOOP_NOT_STARTED, LOOP_RUNNING, LOOP_EXIT_STOP, LOOP_EXIT_BUDGET, LOOP_EXIT_IDLE, LOOP_EXIT_ERROR = range(6)
TRACE_MAGIC = 0x424C4B31
TRACE_HDR_WORDS = 12


class blink_model_cfg(C.Structure):
    _fields_ = [("size", C.c_uint32), ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32),
                ("n_experts", C.c_int32), ("top_k_experts", C.c_int32), ("rope_theta", C.c_float),
                ("rms_eps", C.c_float), ("dtype", C.c_int32), ("weights_layout", C.c_int32), ("weights", C.c_void_p),
                ("weights_bytes", C.c_uint64)]


class blink_sched_cfg(C.Structure):
    _fields_ = [("size", C.c_uint32), ("max_batch", C.c_int32), ("prefill_chunk_tokens", C.c_int32),
                ("n_slots", C.c_int32), ("max_prompt", C.c_int32), ("max_new", C.c_int32), ("exec_mode", C.c_int32),
                ("gemm_impl", C.c_int32), ("control_only", C.c_int32), ("start_paused", C.c_int32),
                ("wait_limit_ms", C.c_int32), ("iteration_budget", C.c_int64), ("idle_exit_us", C.c_int64),
                ("trace_capacity_words", C.c_int64), ("stats_capacity_iters", C.c_int64),
                ("logits_capture", C.c_void_p), ("logits_capture_rows", C.c_int64), ("epilogue_fusion", C.c_int32),
                ("policy", C.c_int32)]


class blink_kv_pool(C.Structure):
    _fields_ = [("size", C.c_uint32), ("block_size", C.c_int32), ("base", C.c_void_p), ("bytes", C.c_uint64)]


class blink_request(C.Structure):
    _fields_ = [("size", C.c_uint32), ("n_prompt", C.c_int32), ("prompt", C.POINTER(C.c_int32)),
                ("max_new_tokens", C.c_int32), ("top_k", C.c_int32), ("temperature", C.c_float),
                ("eos_id", C.c_int32), ("seed", C.c_uint64), ("user_tag", C.c_uint64),
                ("forced_tokens", C.POINTER(C.c_int32)), ("top_p", C.c_float), ("reserved0", C.c_int32)]


class blink_token_event(C.Structure):
    _fields_ = [("ticket", C.c_uint64), ("user_tag", C.c_uint64), ("index", C.c_int32), ("token", C.c_int32),
                ("is_first", C.c_int32), ("is_last", C.c_int32), ("t_device_ns", C.c_uint64),
                ("t_host_ns", C.c_uint64), ("t_submit_ns", C.c_uint64)]


class blink_stats(C.Structure):
    _fields_ = [("size", C.c_uint32), ("loop_state", C.c_int32), ("device_status", C.c_int32),
                ("n_blocks", C.c_int32), ("iterations", C.c_int64), ("launches", C.c_int64),
                ("tokens_out", C.c_int64), ("prompt_tokens", C.c_int64), ("trace_words", C.c_int64),
                ("device_clock_offset_ns", C.c_int64), ("free_blocks", C.c_int32), ("reserved_blocks", C.c_int32),
                ("batch_live", C.c_int32), ("reserved1", C.c_int32), ("bytes_to_device", C.c_int64),
                ("bytes_from_device", C.c_int64)]


class blink_iter_stat(C.Structure):
    _fields_ = [("t_begin_ns", C.c_uint64), ("t_forward_ns", C.c_uint64), ("t_end_ns", C.c_uint64),
                ("n_tokens", C.c_int32), ("n_decode", C.c_int32), ("n_sample_rows", C.c_int32),
                ("n_items", C.c_int32), ("ctx_tokens", C.c_int64), ("kv_tokens", C.c_int64),
                ("phase_ns", C.c_uint64 * 16)]


ITER_STAT_DTYPE = np.dtype([("t_begin_ns", "<u8"), ("t_forward_ns", "<u8"), ("t_end_ns", "<u8"),
                            ("n_tokens", "<i4"), ("n_decode", "<i4"), ("n_sample_rows", "<i4"),
                            ("n_items", "<i4"), ("ctx_tokens", "<i8"), ("kv_tokens", "<i8"),
                            ("phase_ns", "<u8", (16,))])
PHASE_NAMES = ["norm1", "qkv", "rope_kv", "attention", "o", "norm2", "gate_up", "swiglu", "down", "final_norm",
               "lm_head", "sample", "moe_group"]
EVENT_DTYPE = np.dtype([("ticket", "<u8"), ("user_tag", "<u8"), ("index", "<i4"), ("token", "<i4"),
                        ("is_first", "<i4"), ("is_last", "<i4"), ("t_device_ns", "<u8"), ("t_host_ns", "<u8"),
                        ("t_submit_ns", "<u8")])

EXPORTS = ["blink_weights_bytes", "blink_weight_offset", "blink_convert_weights", "blink_kv_blocks_for_bytes", "blink_create",
           "blink_start", "blink_submit", "blink_cancel", "blink_poll", "blink_step", "blink_run", "blink_stop", "blink_destroy",
           "blink_get_stats", "blink_get_trace", "blink_get_iter_stats", "blink_sample", "blink_sample_top_p",
           "blink_sample_noalloc",
           "blink_strerror"]

_lib = None


def lib():
    """Load libblink.so (built in-tree by paper_2604_07609_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_07609_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    P = C.POINTER
    L.blink_weights_bytes.restype = C.c_uint64
    L.blink_weights_bytes.argtypes = [P(blink_model_cfg)]
    L.blink_weight_offset.restype = C.c_uint64
    L.blink_weight_offset.argtypes = [P(blink_model_cfg), C.c_int]
    L.blink_convert_weights.restype = C.c_int
    L.blink_convert_weights.argtypes = [P(blink_model_cfg), C.c_void_p, C.c_int]
    L.blink_kv_blocks_for_bytes.restype = C.c_int64
    L.blink_kv_blocks_for_bytes.argtypes = [P(blink_model_cfg), C.c_int, C.c_uint64]
    L.blink_create.restype = C.c_int
    L.blink_create.argtypes = [P(blink_model_cfg), P(blink_sched_cfg), P(blink_kv_pool), P(C.c_void_p)]
    L.blink_start.restype = C.c_int
    L.blink_start.argtypes = [C.c_void_p]
    L.blink_submit.restype = C.c_int
    L.blink_submit.argtypes = [C.c_void_p, P(blink_request), P(C.c_uint64)]
    L.blink_cancel.restype = C.c_int
    L.blink_cancel.argtypes = [C.c_void_p, C.c_uint64]
    L.blink_poll.restype = C.c_int
    L.blink_poll.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int]
    L.blink_step.restype = C.c_int
    L.blink_step.argtypes = [C.c_void_p, C.c_int]
    L.blink_run.restype = C.c_int
    L.blink_run.argtypes = [C.c_void_p, C.c_int64, P(C.c_float)]
    L.blink_stop.restype = C.c_int
    L.blink_stop.argtypes = [C.c_void_p, C.c_int, C.c_int]
    L.blink_destroy.restype = C.c_int
    L.blink_destroy.argtypes = [C.c_void_p, C.c_int]
    L.blink_get_stats.restype = C.c_int
    L.blink_get_stats.argtypes = [C.c_void_p, P(blink_stats)]
    L.blink_get_trace.restype = C.c_int
    L.blink_get_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, P(C.c_int64)]
    L.blink_get_iter_stats.restype = C.c_int
    L.blink_get_iter_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, P(C.c_int64)]
    L.blink_sample.restype = C.c_int
    L.blink_sample.argtypes = [C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 6
    L.blink_sample_top_p.restype = C.c_int
    L.blink_sample_top_p.argtypes = [C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 7
    L.blink_sample_noalloc.restype = C.c_int
    L.blink_sample_noalloc.argtypes = [C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 6
    L.blink_strerror.restype = C.c_char_p
    L.blink_strerror.argtypes = [C.c_int]
    _lib = L
    return L


class BlinkError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib().blink_strerror(code).decode()} ({code})")


def make_model_cfg(m, weights_ptr=0, weights_bytes=0, weights_layout=0) -> blink_model_cfg:
    """m: synth.ModelCfg-like object (n_layers, d_model, ..., dtype 'bf16'|'fp32')."""
    return blink_model_cfg(C.sizeof(blink_model_cfg), m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim,
                           m.d_ff, m.vocab, m.n_experts, m.top_k_experts, m.rope_theta, m.rms_eps,
                           DTYPE_BF16 if m.dtype == "bf16" else DTYPE_FP32, weights_layout, weights_ptr, weights_bytes)


def blink_weights_bytes(m) -> int:
    cfg = make_model_cfg(m)
    return int(lib().blink_weights_bytes(C.byref(cfg)))


def blink_weight_offset(m, tensor_id: int) -> int:
    cfg = make_model_cfg(m)
    return int(lib().blink_weight_offset(C.byref(cfg), tensor_id))


def blink_convert_weights(m, weights, from_layout: int, to_layout: int, raise_on_error=True) -> int:
    """weights: torch CUDA tensor holding the flat weight buffer; converted in place."""
    cfg = make_model_cfg(m, weights.data_ptr(), weights.numel() * weights.element_size(), from_layout)
    rc = lib().blink_convert_weights(C.byref(cfg), weights.data_ptr(), to_layout)
    if rc != BLINK_OK and raise_on_error:
        raise BlinkError(rc, "blink_convert_weights")
    return rc


def blink_kv_blocks_for_bytes(m, block_size: int, nbytes: int) -> int:
    cfg = make_model_cfg(m)
    return int(lib().blink_kv_blocks_for_bytes(C.byref(cfg), block_size, nbytes))


def blink_sample(logits, top_k, temperature, ticket, gen_index, seed) -> np.ndarray:
    """logits: torch CUDA float32 [rows, vocab]; the rest: per-row sequences (host)."""
    rows, vocab = logits.shape
    assert logits.is_cuda and logits.is_contiguous() and logits.dtype.is_floating_point and logits.element_size() == 4
    a = lambda v, dt: np.ascontiguousarray(v, dtype=dt)
    tk, tp, ti, gi, sd = a(top_k, np.int32), a(temperature, np.float32), a(ticket, np.uint64), \
        a(gen_index, np.int32), a(seed, np.uint64)
    out = np.zeros(rows, dtype=np.int32)
    rc = lib().blink_sample(logits.data_ptr(), rows, vocab, tk.ctypes.data, tp.ctypes.data, ti.ctypes.data,
                            gi.ctypes.data, sd.ctypes.data, out.ctypes.data)
    if rc != BLINK_OK:
        raise BlinkError(rc, "blink_sample")
    return out


def blink_sample_top_p(logits, top_k, temperature, top_p, ticket, gen_index, seed) -> np.ndarray:
    """blink_sample with a per-row nucleus cut (top_p in (0, 1); 0 or >= 1 = off)."""
    rows, vocab = logits.shape
    assert logits.is_cuda and logits.is_contiguous() and logits.dtype.is_floating_point and logits.element_size() == 4
    a = lambda v, dt: np.ascontiguousarray(v, dtype=dt)
    tk, tp, pp, ti, gi, sd = a(top_k, np.int32), a(temperature, np.float32), a(top_p, np.float32), a(ticket, np.uint64), \
        a(gen_index, np.int32), a(seed, np.uint64)
    out = np.zeros(rows, dtype=np.int32)
    rc = lib().blink_sample_top_p(logits.data_ptr(), rows, vocab, tk.ctypes.data, tp.ctypes.data, pp.ctypes.data,
                                  ti.ctypes.data, gi.ctypes.data, sd.ctypes.data, out.ctypes.data)
    if rc != BLINK_OK:
        raise BlinkError(rc, "blink_sample_top_p")
    return out


def blink_sample_noalloc(logits, top_k, temperature, ticket, gen_index, seed, raise_on_error=True):
    """Same sampling as blink_sample, for callers that cannot allocate device memory (a server
    whose memory budget is fixed at start-up, or code that must avoid the device-wide
    synchronisation of cudaFree): the per-row parameters go through a fixed scratch array inside
    the library, so at most SAMPLE_NOALLOC_MAX_ROWS rows per call.  Returns the tokens, or the
    negative error code when raise_on_error is false."""
    rows, vocab = logits.shape
    assert logits.is_cuda and logits.is_contiguous() and logits.dtype.is_floating_point and logits.element_size() == 4
    a = lambda v, dt: np.ascontiguousarray(v, dtype=dt)
    tk, tp, ti, gi, sd = a(top_k, np.int32), a(temperature, np.float32), a(ticket, np.uint64), \
        a(gen_index, np.int32), a(seed, np.uint64)
    out = np.zeros(rows, dtype=np.int32)
    rc = lib().blink_sample_noalloc(logits.data_ptr(), rows, vocab, tk.ctypes.data, tp.ctypes.data, ti.ctypes.data,
                                    gi.ctypes.data, sd.ctypes.data, out.ctypes.data)
    if rc != BLINK_OK:
        if raise_on_error:
            raise BlinkError(rc, "blink_sample_noalloc")
        return rc
    return out


def kv_bytes_per_block(m, block_size: int = 16) -> int:
    return m.n_layers * 2 * m.n_kv_heads * block_size * m.head_dim * (2 if m.dtype == "bf16" else 4)


@dataclass
class TraceRecord:
    iter: int
    W: int
    admitted: list
    scheduled: list
    allocated: list
    sampled: list
    finished: list
    freed: list
    free_count: int
    reserved: int

    def as_dict(self):
        return dict(iter=self.iter, W=self.W, admitted=self.admitted, scheduled=self.scheduled,
                    allocated=self.allocated, sampled=self.sampled, finished=self.finished, freed=self.freed,
                    free_count=self.free_count, reserved=self.reserved)


def parse_trace(words: np.ndarray) -> list[dict]:
    """Decode the device trace.  One record per traced iteration:
    header[12] = magic, iter, W, n_admitted, n_scheduled, n_allocated, n_sampled, n_finished,
    n_freed, free_count, reserved, record_words; then admitted (ticket, batch slot) pairs,
    scheduled (batch slot, ticket, phase, start_pos, n_tokens) 5-tuples, allocated (batch slot,
    logical index, physical block) triples, sampled (batch slot, token) pairs, finished tickets,
    freed blocks."""
    out = []
    p = 0
    w = [int(v) for v in words]
    n = len(w)
    while p < n:
        assert w[p] == TRACE_MAGIC, f"bad trace magic at word {p}"
        _, it, W, na, ns, nal, nsm, nf, nfr, fc, rs, total = w[p:p + TRACE_HDR_WORDS]
        q = p + TRACE_HDR_WORDS
        adm = [(w[q + 2 * i], w[q + 2 * i + 1]) for i in range(na)]; q += 2 * na
        sch = [tuple(w[q + 5 * i:q + 5 * i + 5]) for i in range(ns)]; q += 5 * ns
        alc = [tuple(w[q + 3 * i:q + 3 * i + 3]) for i in range(nal)]; q += 3 * nal
        smp = [(w[q + 2 * i], w[q + 2 * i + 1]) for i in range(nsm)]; q += 2 * nsm
        fin = w[q:q + nf]; q += nf
        fre = w[q:q + nfr]; q += nfr
        assert q - p == total, "trace record length mismatch"
        out.append(dict(iter=it, W=W, admitted=adm, scheduled=sch, allocated=alc, sampled=smp, finished=fin,
                        freed=fre, free_count=fc, reserved=rs))
        p = q
    return out


class Blink:
    """Thin owner of one blink_ctx.  `weights` and `kv_pool` are caller-owned torch CUDA
    tensors (any dtype, used as raw bytes); they are kept referenced while the context lives."""

    def __init__(self, model, sched, weights=None, kv_pool=None, *, exec_mode=EXEC_PERSISTENT, gemm_impl=GEMM_AUTO,
                 control_only=False, start_paused=False, iteration_budget=0, idle_exit_us=0, trace_words=0,
                 stats_iters=0, logits_capture=None, kv_bytes=None, weights_layout=WEIGHTS_ROW_MAJOR, wait_limit_ms=0,
                 epilogue_fusion=FUSION_AUTO, policy=POLICY_CHUNKED):
        L = lib()
        self.model, self.sched = model, sched
        self._keep = (weights, kv_pool, logits_capture)
        wptr = weights.data_ptr() if weights is not None else 0
        wbytes = weights.numel() * weights.element_size() if weights is not None else 0
        mc = make_model_cfg(model, wptr, wbytes, weights_layout)
        cap_ptr = logits_capture.data_ptr() if logits_capture is not None else 0
        cap_rows = logits_capture.shape[0] if logits_capture is not None else 0
        sc = blink_sched_cfg(C.sizeof(blink_sched_cfg), sched.max_batch, sched.prefill_chunk_tokens, sched.n_slots,
                             sched.max_prompt, sched.max_new, exec_mode, gemm_impl, int(control_only),
                             int(start_paused), wait_limit_ms, iteration_budget, idle_exit_us, trace_words, stats_iters,
                             cap_ptr, cap_rows, epilogue_fusion, policy)
        if kv_pool is not None:
            kv = blink_kv_pool(C.sizeof(blink_kv_pool), sched.block_size, kv_pool.data_ptr(),
                               kv_pool.numel() * kv_pool.element_size())
        else:  # control-only: no memory behind the pool, only its size
            kv = blink_kv_pool(C.sizeof(blink_kv_pool), sched.block_size, 0,
                               kv_bytes if kv_bytes is not None else sched.n_blocks * kv_bytes_per_block(model))
        h = C.c_void_p()
        rc = L.blink_create(C.byref(mc), C.byref(sc), C.byref(kv), C.byref(h))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_create")
        self._h = h
        self._ev = np.zeros(4096, dtype=EVENT_DTYPE)

    # -- C ABI, same names -----------------------------------------------------------------
    def blink_start(self):
        rc = lib().blink_start(self._h)
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_start")

    def blink_submit(self, prompt, max_new_tokens, top_k=0, temperature=1.0, eos_id=-1, seed=0, user_tag=0,
                     forced_tokens=None, raise_on_error=True, top_p=0.0):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        f = None if forced_tokens is None else np.ascontiguousarray(forced_tokens, dtype=np.int32)
        r = blink_request(C.sizeof(blink_request), p.shape[0], p.ctypes.data_as(C.POINTER(C.c_int32)),
                          max_new_tokens, top_k, temperature, eos_id, seed, user_tag,
                          f.ctypes.data_as(C.POINTER(C.c_int32)) if f is not None else None, top_p, 0)
        t = C.c_uint64()
        rc = lib().blink_submit(self._h, C.byref(r), C.byref(t))
        if rc != BLINK_OK:
            if raise_on_error:
                raise BlinkError(rc, "blink_submit")
            return rc
        return int(t.value)

    def blink_cancel(self, ticket: int) -> int:
        return int(lib().blink_cancel(self._h, ticket))

    def blink_poll(self, max_events=4096, timeout_us=0) -> np.ndarray:
        max_events = min(max_events, self._ev.shape[0])
        n = lib().blink_poll(self._h, self._ev.ctypes.data, max_events, timeout_us)
        if n < 0:
            raise BlinkError(n, "blink_poll")
        return self._ev[:n].copy()

    def blink_step(self, n=1):
        rc = lib().blink_step(self._h, n)
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_step")

    def blink_run(self, n_iterations: int) -> float:
        """Manual mode: one launch of the loop kernel for up to n_iterations steps; returns its
        duration in ms (CUDA events on the library's stream)."""
        ms = C.c_float()
        rc = lib().blink_run(self._h, n_iterations, C.byref(ms))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_run")
        return float(ms.value)

    def blink_stop(self, final=False, timeout_ms=10000):
        return lib().blink_stop(self._h, int(final), timeout_ms)

    def blink_destroy(self, timeout_ms=20000):
        if self._h is None:
            return BLINK_OK
        rc = lib().blink_destroy(self._h, timeout_ms)
        if rc == BLINK_OK:
            self._h = None
            self._keep = None
        return rc

    def blink_get_stats(self) -> blink_stats:
        s = blink_stats(C.sizeof(blink_stats))
        rc = lib().blink_get_stats(self._h, C.byref(s))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_get_stats")
        return s

    def blink_get_trace(self) -> np.ndarray:
        n = C.c_int64()
        rc = lib().blink_get_trace(self._h, None, 0, C.byref(n))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_get_trace")
        buf = np.zeros(max(1, n.value), dtype=np.int32)
        rc = lib().blink_get_trace(self._h, buf.ctypes.data, n.value, C.byref(n))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_get_trace")
        return buf[:n.value]

    def blink_get_iter_stats(self) -> np.ndarray:
        n = C.c_int64()
        rc = lib().blink_get_iter_stats(self._h, None, 0, C.byref(n))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_get_iter_stats")
        buf = np.zeros(max(1, n.value), dtype=ITER_STAT_DTYPE)
        rc = lib().blink_get_iter_stats(self._h, buf.ctypes.data, n.value, C.byref(n))
        if rc != BLINK_OK:
            raise BlinkError(rc, "blink_get_iter_stats")
        return buf[:n.value]

    # -- conveniences built only from the calls above ---------------------------------------
    def submit_request(self, r, forced_tokens=None, **kw):
        return self.blink_submit(r.prompt, r.max_new, r.top_k, r.temperature, r.eos_id, r.seed, r.user_tag,
                                 forced_tokens, top_p=getattr(r, "top_p", 0.0), **kw)

    def drain(self, n_tokens_expected: int, timeout_s: float = 60.0, step_iters: int = 0):
        """Poll (persistent mode) or step+poll (stepped mode, step_iters per round) until
        n_tokens_expected events arrived.  Returns the concatenated event array."""
        import time
        evs, got = [], 0
        t0 = time.monotonic()
        while got < n_tokens_expected:
            if step_iters:
                self.blink_step(step_iters)
            e = self.blink_poll(4096, 0 if step_iters else 2000)
            if len(e):
                evs.append(e)
                got += len(e)
            if time.monotonic() - t0 > timeout_s:
                raise TimeoutError(f"drain: {got}/{n_tokens_expected} tokens after {timeout_s}s "
                                   f"(device_status={self.blink_get_stats().device_status})")
        return np.concatenate(evs) if evs else np.zeros(0, dtype=EVENT_DTYPE)

    def __del__(self):
        try:
            if getattr(self, "_h", None) is not None:
                lib().blink_destroy(self._h, 20000)
        except Exception:
            pass


def tokens_by_ticket(events: np.ndarray) -> dict:
    out = {}
    for ev in np.sort(events, order=["ticket", "index"]):
        out.setdefault(int(ev["ticket"]), []).append(int(ev["token"]))
    return out
