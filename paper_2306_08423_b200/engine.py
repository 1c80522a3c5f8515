"""Thin ctypes binding of the engine's C ABI (``include/distsim.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Device buffers are PyTorch tensors (PyTorch is used for device memory
and streams, nothing else); their ``data_ptr()`` is what crosses the boundary.
There is no fallback: if ``libdistsim.so`` has not been built, importing this
module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("DISTSIM_LIBRARY", os.path.join(_PKG, "libdistsim.so"))   # another build of the same ABI
MAX_PP = 64

OK, E_ARG, E_STATE, E_RANGE, E_CAPACITY, E_OVERFLOW, E_CUDA, E_TIMEOUT, E_UNSUPPORTED = (
    0, -1, -2, -3, -4, -5, -6, -7, -8)

EXPORTS = ("distsim_create", "distsim_destroy", "distsim_last_error",
           "distsim_load_event_table", "distsim_set_space", "distsim_decode",
           "distsim_eval_strategies", "distsim_eval_select", "distsim_argmin", "distsim_topk",
           "distsim_merge_topk",
           "distsim_emit_timelines", "distsim_emit_shape_of_last_plan", "distsim_emit_timelines_async",
           "distsim_checksum_timelines", "distsim_search_host",
           "distsim_topk_static")
# hooks of include/distsim_testing.h (test-suite and benchmark accounting; not the stable ABI)
TESTING_EXPORTS = ("distsim_testing_set_stage_wait_polls", "distsim_testing_launch_count",
                   "distsim_testing_space_cells", "distsim_testing_lockstep_pieces",
                   "distsim_testing_bidirectional_order",
                   "distsim_testing_time_phases", "distsim_testing_last_phase_ms")
TOPK_STATIC_MAX_K = 1024

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2306_08423_b200.build` "
                      "(there is no CPU fallback)")
_lib = C.CDLL(LIB_PATH)


class DistsimError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"distsim error {code}: {msg}")
        self.code = code


class _Table(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_classes", C.c_int32), ("n_devices", C.c_int32),
                ("gpus_per_node", C.c_int32), ("global_batch", C.c_int64), ("seq", C.c_int64),
                ("hidden", C.c_int64), ("alpha_intra_ns", C.c_int64), ("beta_intra", C.c_int64),
                ("alpha_inter_ns", C.c_int64), ("beta_inter", C.c_int64),
                ("dp_bucket_bytes", C.c_int64), ("dp_overlap", C.c_int32),
                ("act_bytes_per_elem", C.c_int32), ("class_mp", C.c_void_p),
                ("class_b", C.c_void_p), ("fwd_ns", C.c_void_p), ("bwd_ns", C.c_void_p),
                ("layer_is_expert", C.c_void_p), ("grad_bytes", C.c_void_p),
                ("allreduce_profile_max", C.c_int32), ("n_jitter", C.c_int32),
                ("jitter_stages", C.c_int32), ("reserved", C.c_int32),
                ("jitter_fwd_ns", C.c_void_p), ("jitter_bwd_ns", C.c_void_p)]


class _Space(C.Structure):
    _fields_ = [("mp_max", C.c_int32), ("pp_max", C.c_int32), ("n_m", C.c_int32),
                ("m_list", C.c_void_p), ("m_rule", C.c_int32), ("partition_mode", C.c_int32),
                ("sched_mask", C.c_int32), ("v_max", C.c_int32)]


class _Candidate(C.Structure):
    _fields_ = [("mp", C.c_int32), ("pp", C.c_int32), ("dp", C.c_int32), ("m", C.c_int32),
                ("sched", C.c_int32), ("micro_batch_size", C.c_int32), ("class_index", C.c_int32),
                ("bounds", C.c_int32 * (MAX_PP + 1)), ("v", C.c_int32)]


_lib.distsim_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
_lib.distsim_destroy.argtypes = [C.c_void_p]
_lib.distsim_destroy.restype = None
_lib.distsim_last_error.argtypes = [C.c_void_p]
_lib.distsim_last_error.restype = C.c_char_p
_lib.distsim_testing_launch_count.argtypes = [C.c_void_p]
_lib.distsim_testing_launch_count.restype = C.c_int64
_lib.distsim_testing_set_stage_wait_polls.argtypes = [C.c_void_p, C.c_int32]
_lib.distsim_testing_lockstep_pieces.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_int64, C.c_int64,
                                                 C.c_void_p, C.c_void_p, C.c_void_p]
_lib.distsim_testing_lockstep_pieces.restype = C.c_int64
_lib.distsim_testing_bidirectional_order.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.POINTER(C.c_int32)]
_lib.distsim_testing_time_phases.argtypes = [C.c_void_p, C.c_int32]
_lib.distsim_testing_last_phase_ms.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_float)]
_lib.distsim_load_event_table.argtypes = [C.c_void_p, C.POINTER(_Table)]
_lib.distsim_set_space.argtypes = [C.c_void_p, C.POINTER(_Space), C.POINTER(C.c_int64)]
_lib.distsim_decode.argtypes = [C.c_void_p, C.c_int64, C.POINTER(_Candidate)]
_lib.distsim_eval_strategies.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
_lib.distsim_eval_select.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
_lib.distsim_argmin.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
_lib.distsim_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32,
                              C.c_void_p, C.c_void_p]
_lib.distsim_merge_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32,
                                    C.c_void_p, C.c_void_p]
_lib.distsim_emit_timelines.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                        C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.POINTER(C.c_int64)]
_lib.distsim_emit_shape_of_last_plan.argtypes = [C.c_void_p, C.c_void_p]
_lib.distsim_emit_timelines_async.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                              C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.distsim_checksum_timelines.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
_lib.distsim_search_host.argtypes = [C.c_void_p, C.POINTER(_Table), C.POINTER(_Space), C.c_int32,
                                     C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                     C.c_void_p, C.c_void_p]


_lib.distsim_topk_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32,
                                     C.c_void_p, C.c_void_p]


_lib.distsim_testing_space_cells.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _table_struct(t):
    arrs = [np.ascontiguousarray(t.class_mp, np.int32), np.ascontiguousarray(t.class_b, np.int32),
            np.ascontiguousarray(t.fwd_ns, np.int64), np.ascontiguousarray(t.bwd_ns, np.int64),
            np.ascontiguousarray(t.layer_is_expert, np.uint8),
            np.ascontiguousarray(t.grad_bytes, np.int64)]
    s = _Table(t.n_layers, arrs[0].shape[0], t.n_devices, t.gpus_per_node, t.global_batch, t.seq,
               t.hidden, t.alpha_intra_ns, t.beta_intra, t.alpha_inter_ns, t.beta_inter,
               t.dp_bucket_bytes, t.dp_overlap, t.act_bytes_per_elem, *[_np_ptr(a) for a in arrs],
               int(getattr(t, "allreduce_profile_max", 0)), 0, 0, 0, None, None)
    jf = getattr(t, "jitter_fwd_ns", None)
    if jf is not None and np.size(jf) > 0:
        jf = np.ascontiguousarray(jf, np.int64)
        jb = np.ascontiguousarray(t.jitter_bwd_ns, np.int64)
        s.n_jitter, s.jitter_stages = jf.shape
        s.jitter_fwd_ns, s.jitter_bwd_ns = _np_ptr(jf), _np_ptr(jb)
        arrs += [jf, jb]
    return s, arrs


def _space_struct(sp):
    ml = np.ascontiguousarray(sp.m_list, np.int32)
    return _Space(sp.mp_max, sp.pp_max, ml.shape[0], _np_ptr(ml), sp.m_rule, sp.partition_mode,
                  sp.sched_mask, int(getattr(sp, "v_max", 0))), ml


def _dev_ptr(t, dtype_name: str, min_elems: int, what: str):
    """Device pointer of a contiguous CUDA tensor after checking dtype and size."""
    import torch
    if t is None:
        return None
    want = getattr(torch, dtype_name)
    if not t.is_cuda or t.dtype != want or not t.is_contiguous():
        raise ValueError(f"{what}: need a contiguous CUDA tensor of {dtype_name}")
    if t.numel() < min_elems:
        raise ValueError(f"{what}: need at least {min_elems} elements, got {t.numel()}")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


class Context:
    """Owns one ``distsim_ctx`` on a CUDA device."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        rc = _lib.distsim_create(C.byref(self._h), device)
        if rc != OK:
            raise DistsimError(rc, "distsim_create failed (no CUDA device of compute capability 10.x?)")
        self.device = device
        self.n_candidates = 0
        self.n_devices = 0
        self.pp_max = 0

    def close(self):
        if self._h:
            _lib.distsim_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            raise DistsimError(rc, _lib.distsim_last_error(self._h).decode())

    @property
    def launch_count(self) -> int:
        return int(_lib.distsim_testing_launch_count(self._h))


def distsim_load_event_table(ctx: Context, table) -> None:
    s, _keep = _table_struct(table)
    ctx._check(_lib.distsim_load_event_table(ctx._h, C.byref(s)))
    ctx.n_devices = int(table.n_devices)
    ctx.n_candidates = 0


def distsim_set_space(ctx: Context, space) -> int:
    s, _keep = _space_struct(space)
    n = C.c_int64(0)
    ctx._check(_lib.distsim_set_space(ctx._h, C.byref(s), C.byref(n)))
    ctx.n_candidates = int(n.value)
    ctx.pp_max = int(space.pp_max)
    return ctx.n_candidates


def distsim_decode(ctx: Context, index: int) -> dict:
    c = _Candidate()
    ctx._check(_lib.distsim_decode(ctx._h, index, C.byref(c)))
    return dict(mp=c.mp, pp=c.pp, dp=c.dp, m=c.m, sched=c.sched, micro_batch_size=c.micro_batch_size,
                class_index=c.class_index, bounds=tuple(c.bounds[: c.pp * c.v + 1]), v=c.v)


def distsim_eval_strategies(ctx: Context, first: int, count: int, d_batch_ns,
                            d_stage_busy_ns=None, stream=None) -> None:
    pb = _dev_ptr(d_batch_ns, "int64", count, "d_batch_ns")
    ps = _dev_ptr(d_stage_busy_ns, "int64", count * ctx.pp_max, "d_stage_busy_ns")
    ctx._check(_lib.distsim_eval_strategies(ctx._h, _stream(stream), first, count, pb, ps))


def distsim_eval_select(ctx: Context, first: int, count: int, d_batch_ns, k: int = 0, d_indices=None,
                        d_times=None, d_best=None, stream=None, to_host: bool = True):
    """Evaluation with the best candidate and the k fastest in one call.  With ``to_host`` it
    synchronises and returns (best index, best batch time); without, it is asynchronous, returns
    None, and ``d_best`` (int64 [2] on the device: batch time, index) receives the best candidate."""
    pb = _dev_ptr(d_batch_ns, "int64", count, "d_batch_ns")
    pi = _dev_ptr(d_indices, "int64", k, "d_indices")
    pt = _dev_ptr(d_times, "int64", k, "d_times")
    pd = _dev_ptr(d_best, "int64", 2, "d_best")
    bi, bt = C.c_int64(0), C.c_int64(0)
    rc = _lib.distsim_eval_select(ctx._h, _stream(stream), first, count, pb, k, pi, pt, pd,
                                  C.byref(bi) if to_host else None, C.byref(bt) if to_host else None)
    if rc == E_TIMEOUT and b"outputs are exact" in _lib.distsim_last_error(ctx._h):
        e = DistsimError(rc, _lib.distsim_last_error(ctx._h).decode())
        e.result = (int(bi.value), int(bt.value))
        raise e
    ctx._check(rc)
    return (int(bi.value), int(bt.value)) if to_host else None


def distsim_argmin(ctx: Context, d_batch_ns, first: int, count: int, stream=None):
    pb = _dev_ptr(d_batch_ns, "int64", count, "d_batch_ns")
    bi, bt = C.c_int64(0), C.c_int64(0)
    rc = _lib.distsim_argmin(ctx._h, _stream(stream), pb, first, count, C.byref(bi), C.byref(bt))
    if rc == E_TIMEOUT and b"outputs are exact" in _lib.distsim_last_error(ctx._h):
        e = DistsimError(rc, _lib.distsim_last_error(ctx._h).decode())
        e.result = (int(bi.value), int(bt.value))       # the outputs were written before the code was returned
        raise e
    ctx._check(rc)
    return int(bi.value), int(bt.value)


def distsim_topk(ctx: Context, d_batch_ns, first: int, count: int, k: int, d_indices,
                 d_times=None, stream=None) -> None:
    pb = _dev_ptr(d_batch_ns, "int64", count, "d_batch_ns")
    pi = _dev_ptr(d_indices, "int64", k, "d_indices")
    pt = _dev_ptr(d_times, "int64", k, "d_times")
    ctx._check(_lib.distsim_topk(ctx._h, _stream(stream), pb, first, count, k, pi, pt))


def distsim_merge_topk(ctx: Context, d_times_in, d_indices_in, n: int, k: int, d_indices, d_times=None,
                       stream=None) -> None:
    """The k smallest of n given (time, index) pairs, ascending: merges the lists of several ranks."""
    pt = _dev_ptr(d_times_in, "int64", n, "d_times_in")
    pi = _dev_ptr(d_indices_in, "int64", n, "d_indices_in")
    po = _dev_ptr(d_indices, "int64", k, "d_indices")
    pq = _dev_ptr(d_times, "int64", k, "d_times")
    ctx._check(_lib.distsim_merge_topk(ctx._h, _stream(stream), pt, pi, n, k, po, pq))


def distsim_emit_timelines(ctx: Context, d_indices, n: int, d_records, capacity_records: int,
                           d_offsets=None, d_busy_ns=None, d_util=None, stream=None) -> int:
    """Returns the number of records needed; raises DistsimError(E_CAPACITY) if
    ``d_records`` is given but too small.  ``d_records`` is an int64 tensor of
    at least ``5 * capacity_records`` elements (or None for a sizing pass).  Offsets, busy
    times and utilisations are final on return; the records are written in stream order
    (complete once the work enqueued on the stream has finished).  A DistsimError with code
    E_TIMEOUT that carries ``total_records`` reports a stalled table copy: all outputs were
    written and are exact."""
    pi = _dev_ptr(d_indices, "int64", n, "d_indices")
    pr = _dev_ptr(d_records, "int64", 5 * capacity_records, "d_records")
    nn = n * ctx.n_devices
    po = _dev_ptr(d_offsets, "int64", nn + 1, "d_offsets")
    pbz = _dev_ptr(d_busy_ns, "int64", nn, "d_busy_ns")
    pu = _dev_ptr(d_util, "float64", nn, "d_util")
    total = C.c_int64(0)
    rc = _lib.distsim_emit_timelines(ctx._h, _stream(stream), pi, n, pr, capacity_records, po, pbz, pu,
                                     C.byref(total))
    if rc == E_CAPACITY or (rc == E_TIMEOUT and b"outputs are exact" in _lib.distsim_last_error(ctx._h)):
        e = DistsimError(rc, _lib.distsim_last_error(ctx._h).decode())
        e.total_records = int(total.value)
        raise e
    ctx._check(rc)
    return int(total.value)


class EmitShape(C.Structure):
    """distsim_emit_shape: what an emission needs, as upper bounds an asynchronous call provisions for."""
    _fields_ = [("records", C.c_int64), ("item_tiles", C.c_int64), ("bucket_tiles", C.c_int64),
                ("tmpl_words", C.c_int64), ("bucket_recs", C.c_int64), ("run_words", C.c_int64)]


def distsim_emit_shape_of_last_plan(ctx: Context) -> EmitShape:
    """The shape of the context's most recent synchronising emission call (a sizing call, say)."""
    shape = EmitShape()
    ctx._check(_lib.distsim_emit_shape_of_last_plan(ctx._h, C.byref(shape)))
    return shape


def distsim_emit_timelines_async(ctx: Context, d_indices, n: int, d_records, capacity_records: int, shape: EmitShape,
                                 d_offsets=None, d_busy_ns=None, d_util=None, stream=None) -> None:
    """Emission without any wait on the host: plans and writes in stream order, provisioned by
    ``shape``.  If the selection needs more than the shape or the capacity allow, nothing is written
    to ``d_records`` and the next synchronising call on the context raises E_CAPACITY;
    ``d_offsets[n * N]`` is the number of records needed either way."""
    pi = _dev_ptr(d_indices, "int64", n, "d_indices")
    pr = _dev_ptr(d_records, "int64", 5 * capacity_records, "d_records")
    nn = n * ctx.n_devices
    po = _dev_ptr(d_offsets, "int64", nn + 1, "d_offsets")
    pbz = _dev_ptr(d_busy_ns, "int64", nn, "d_busy_ns")
    pu = _dev_ptr(d_util, "float64", nn, "d_util")
    ctx._check(_lib.distsim_emit_timelines_async(ctx._h, _stream(stream), pi, n, pr, capacity_records, C.byref(shape),
                                                 po, pbz, pu))


def distsim_checksum_timelines(ctx: Context, d_records, d_offsets, n_lists: int, d_checksums, stream=None) -> None:
    """Order-sensitive 64-bit checksum of each of the ``n_lists`` record streams delimited by
    ``d_offsets`` into ``d_checksums`` (an int64 tensor holding the 64-bit sums' bit patterns)."""
    total = 0 if n_lists == 0 else 1
    pr = _dev_ptr(d_records, "int64", total, "d_records")
    po = _dev_ptr(d_offsets, "int64", n_lists + 1, "d_offsets")
    pc = _dev_ptr(d_checksums, "int64", n_lists, "d_checksums")
    ctx._check(_lib.distsim_checksum_timelines(ctx._h, _stream(stream), pr, po, n_lists, pc))


def distsim_search_host(ctx: Context, table, space, k: int = 0):
    """Whole search from host memory.  Returns (n_candidates, best_index,
    best_batch_ns, topk_indices, topk_times) with numpy arrays for the last two."""
    ts, _k1 = _table_struct(table)
    ss, _k2 = _space_struct(space)
    n, bi, bt = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    idx = np.zeros(max(k, 1), np.int64)
    tim = np.zeros(max(k, 1), np.int64)
    ctx._check(_lib.distsim_search_host(ctx._h, C.byref(ts), C.byref(ss), k, C.byref(n), C.byref(bi),
                                        C.byref(bt), _np_ptr(idx) if k else None,
                                        _np_ptr(tim) if k else None))
    ctx.n_devices = int(table.n_devices)
    ctx.n_candidates = int(n.value)
    ctx.pp_max = int(space.pp_max)
    kk = min(k, ctx.n_candidates, 4096)
    return ctx.n_candidates, int(bi.value), int(bt.value), idx[:kk], tim[:kk]


def distsim_topk_static(d_batch_ns, first: int, count: int, k: int, d_indices, d_times=None,
                        stream=None) -> None:
    """The k fastest candidates without a context and without any device allocation.

    For callers that cannot call cudaMalloc (a latency-critical loop, a process whose device
    memory is all owned by a pool, a plug-in whose host forbids it): the scratch is a fixed
    array inside the library, so
    ``k`` is limited to ``TOPK_STATIC_MAX_K``.  The tensors are the caller's; this wrapper
    creates none.  Runs on the current device; calls that may overlap on the GPU must be
    ordered by the caller because they share the scratch.
    """
    pb = _dev_ptr(d_batch_ns, "int64", count, "d_batch_ns")
    pi = _dev_ptr(d_indices, "int64", k, "d_indices")
    pt = _dev_ptr(d_times, "int64", k, "d_times")
    rc = _lib.distsim_topk_static(_stream(stream), pb, first, count, k, pi, pt)
    if rc == E_CAPACITY:
        raise DistsimError(rc, f"k = {k} exceeds the fixed scratch (at most {TOPK_STATIC_MAX_K})")
    if rc != OK:
        raise DistsimError(rc, "distsim_topk_static failed")


def distsim_testing_bidirectional_order(pp: int, m: int):
    """(order, kept): the library's merged item order of the bidirectional schedule for (pp, m) as a
    list per device of ('F'|'B', micro-batch, pipeline), and its kept-item count.  Host logic only."""
    buf = (C.c_uint16 * (pp * 2 * m))()
    kept = C.c_int32(0)
    rc = _lib.distsim_testing_bidirectional_order(pp, m, buf, C.byref(kept))
    if rc != OK:
        raise DistsimError(rc, "distsim_testing_bidirectional_order failed")
    half = m // 2
    order = []
    for d in range(pp):
        items = []
        for k in range(2 * m):
            w = buf[d * 2 * m + k]
            u = w >> 15
            items.append(("B" if w & (1 << 14) else "F", (w & 0x3FFF) + u * half, u))
        order.append(items)
    return order, int(kept.value)


def distsim_testing_space_cells(ctx: Context):
    """(recurrence cells of the space, cells the engine evaluates in 32-bit arithmetic)."""
    a, b = C.c_int64(0), C.c_int64(0)
    ctx._check(_lib.distsim_testing_space_cells(ctx._h, C.byref(a), C.byref(b)))
    return int(a.value), int(b.value)


def distsim_testing_lockstep_pieces(pp: int, lo: int, hi: int, max_blocks: int, max_pieces: int = 64):
    """(number of pieces, [(lo, hi, blocks) of the first max_pieces])."""
    a, b = np.zeros(max(1, max_pieces), np.int64), np.zeros(max(1, max_pieces), np.int64)
    c = np.zeros(max(1, max_pieces), np.int32)
    n = int(_lib.distsim_testing_lockstep_pieces(pp, lo, hi, max_blocks, max_pieces, _np_ptr(a), _np_ptr(b), _np_ptr(c)))
    if n < 0:
        raise DistsimError(n, "bad arguments")
    k = min(n, max_pieces)
    return n, list(zip(a[:k].tolist(), b[:k].tolist(), c[:k].tolist()))


def distsim_testing_time_phases(ctx: Context, enable: bool) -> None:
    ctx._check(_lib.distsim_testing_time_phases(ctx._h, 1 if enable else 0))


def distsim_testing_last_phase_ms(ctx: Context):
    """(evaluation ms, selection ms) of the most recent timed distsim_eval_select call."""
    a, b = C.c_float(0), C.c_float(0)
    ctx._check(_lib.distsim_testing_last_phase_ms(ctx._h, C.byref(a), C.byref(b)))
    return float(a.value), float(b.value)


def distsim_testing_launch_count(ctx: Context) -> int:
    return ctx.launch_count


def distsim_testing_set_stage_wait_polls(ctx: Context, polls: int) -> None:
    """Polls of the evaluation kernels' first wait for their staged tables (0: give up at once
    and take the global-memory path; the library's default is 65 536)."""
    ctx._check(_lib.distsim_testing_set_stage_wait_polls(ctx._h, polls))
