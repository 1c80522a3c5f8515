"""ctypes wrapper of the C oracle -- TEST INFRASTRUCTURE ONLY (see distsim_oracle.c).

Tables and spaces are passed as any object with the attributes of
``EventTable`` / ``SearchSpace`` (numpy arrays and ints); this module does not
import the engine package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "distsim_oracle.c")
_LIB = os.path.join(_HERE, "_liborc.so")
_MAX_PP = 64

KINDS = {"COMPUTE_F": 0, "COMPUTE_B": 1, "MP_AR_F": 2, "MP_AR_B": 3, "A2A_F": 4, "A2A_B": 5,
         "SEND_F": 6, "SEND_B": 7, "DP_AR": 8, "JITTER_F": 9, "JITTER_B": 10}


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}")
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
                ("jitter_stages", C.c_int32), ("pad", C.c_int32),
                ("jitter_fwd_ns", C.c_void_p), ("jitter_bwd_ns", C.c_void_p)]


class _Space(C.Structure):
    _fields_ = [("mp_max", C.c_int32), ("pp_max", C.c_int32), ("n_m", C.c_int32),
                ("m_list", C.c_void_p), ("m_rule", C.c_int32), ("partition_mode", C.c_int32),
                ("sched_mask", C.c_int32), ("v_max", C.c_int32)]


class _Cand(C.Structure):
    _fields_ = [("mp", C.c_int32), ("pp", C.c_int32), ("dp", C.c_int32), ("m", C.c_int32),
                ("sched", C.c_int32), ("bounds", C.c_int32 * (_MAX_PP + 1)), ("v", C.c_int32)]


@dataclass
class Candidate:
    mp: int
    pp: int
    dp: int
    m: int
    sched: int
    bounds: tuple
    v: int = 1               # model chunks per device (interleaved 1F1B, sched 3)

    def _c(self) -> _Cand:
        c = _Cand(self.mp, self.pp, self.dp, self.m, self.sched)
        for i, b in enumerate(self.bounds):
            c.bounds[i] = b
        c.v = self.v
        return c


@dataclass
class SimResult:
    batch_ns: int
    offsets: np.ndarray      # int64 [n_lists + 1], in records
    records: np.ndarray      # int64 [total, 5] = (kind, layer, microbatch, start_ns, end_ns)
    busy_ns: np.ndarray      # int64 [n_lists]
    util: np.ndarray         # float64 [n_lists]


_lib = None


def build(force: bool = False) -> str:
    """Compiles the C oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", _LIB, _SRC])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.orc_count.restype = C.c_int64
        lib.orc_simulate.restype = C.c_void_p
        lib.orc_result_batch.restype = C.c_int64
        lib.orc_result_total_records.restype = C.c_int64
        lib.orc_result_n_lists.restype = C.c_int32
        for f in (lib.orc_ring_allreduce_ns, lib.orc_all_to_all_ns, lib.orc_p2p_ns, lib.orc_allreduce_ns):
            f.restype = C.c_int64
        assert lib.orc_sizeof_candidate() == C.sizeof(_Cand)
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _table(t):
    """Returns (struct, keepalive) for an EventTable-like object."""
    arrs = [np.ascontiguousarray(t.class_mp, np.int32), np.ascontiguousarray(t.class_b, np.int32),
            np.ascontiguousarray(t.fwd_ns, np.int64), np.ascontiguousarray(t.bwd_ns, np.int64),
            np.ascontiguousarray(t.layer_is_expert, np.uint8),
            np.ascontiguousarray(t.grad_bytes, np.int64)]
    s = _Table(t.n_layers, arrs[0].shape[0], t.n_devices, t.gpus_per_node, t.global_batch, t.seq,
               t.hidden, t.alpha_intra_ns, t.beta_intra, t.alpha_inter_ns, t.beta_inter,
               t.dp_bucket_bytes, t.dp_overlap, t.act_bytes_per_elem, *[_ptr(a) for a in arrs],
               int(getattr(t, "allreduce_profile_max", 0)), 0, 0, 0, None, None)
    jf = getattr(t, "jitter_fwd_ns", None)
    if jf is not None and np.size(jf) > 0:
        jf = np.ascontiguousarray(jf, np.int64)
        jb = np.ascontiguousarray(t.jitter_bwd_ns, np.int64)
        assert jf.ndim == 2 and jf.shape == jb.shape
        s.n_jitter, s.jitter_stages = jf.shape
        s.jitter_fwd_ns, s.jitter_bwd_ns = _ptr(jf), _ptr(jb)
        arrs += [jf, jb]
    return s, arrs


def _space(sp):
    ml = np.ascontiguousarray(sp.m_list, np.int32)
    return _Space(sp.mp_max, sp.pp_max, ml.shape[0], _ptr(ml), sp.m_rule, sp.partition_mode,
                  sp.sched_mask, int(getattr(sp, "v_max", 0))), ml


def ring_allreduce_ns(n, nbytes, alpha, beta):
    return _load().orc_ring_allreduce_ns(C.c_int64(n), C.c_int64(nbytes), C.c_int64(alpha), C.c_int64(beta))


def allreduce_ns(k, n, nbytes, alpha, beta):
    return _load().orc_allreduce_ns(C.c_int64(k), C.c_int64(n), C.c_int64(nbytes), C.c_int64(alpha), C.c_int64(beta))


def all_to_all_ns(n, nbytes, alpha, beta):
    return _load().orc_all_to_all_ns(C.c_int64(n), C.c_int64(nbytes), C.c_int64(alpha), C.c_int64(beta))


def p2p_ns(nbytes, alpha, beta):
    return _load().orc_p2p_ns(C.c_int64(nbytes), C.c_int64(alpha), C.c_int64(beta))


def count(table, space) -> int:
    t, _k1 = _table(table)
    s, _k2 = _space(space)
    return int(_load().orc_count(C.byref(t), C.byref(s)))


def enumerate_at(table, space, indices) -> list:
    """Candidates at the given ascending indices of the canonical order."""
    idx = np.ascontiguousarray(indices, np.int64)
    t, _k1 = _table(table)
    s, _k2 = _space(space)
    out = (_Cand * max(1, idx.shape[0]))()
    e = _load().orc_enumerate_at(C.byref(t), C.byref(s), _ptr(idx), C.c_int64(idx.shape[0]), out)
    if e:
        raise OracleError(e)
    return [Candidate(c.mp, c.pp, c.dp, c.m, c.sched, tuple(c.bounds[: c.pp * (c.v if c.sched == 3 else 1) + 1]),
                      c.v if c.sched == 3 else 1)
            for c in out[: idx.shape[0]]]


def simulate(table, cand: Candidate, replicate: bool = True, reverse_scan: bool = False,
             want_records: bool = True) -> SimResult:
    lib = _load()
    t, _k1 = _table(table)
    err = C.c_int(0)
    c = cand._c()
    h = lib.orc_simulate(C.byref(t), C.byref(c), int(replicate), int(reverse_scan), C.byref(err))
    if not h:
        raise OracleError(err.value)
    h = C.c_void_p(h)
    try:
        n = lib.orc_result_n_lists(h)
        total = lib.orc_result_total_records(h)
        offsets = np.zeros(n + 1, np.int64)
        records = np.zeros((total if want_records else 0, 5), np.int64)
        busy = np.zeros(n, np.int64)
        util = np.zeros(n, np.float64)
        lib.orc_result_copy(h, _ptr(offsets), _ptr(records) if want_records else None,
                            _ptr(busy), _ptr(util))
        return SimResult(int(lib.orc_result_batch(h)), offsets, records, busy, util)
    finally:
        lib.orc_result_free(h)


def eval_indices(table, space, indices, replicate: bool = False, pp_stride: int = 0):
    """(batch_ns[n], stage_busy[n, pp_stride] or None) for ascending indices; one thread."""
    idx = np.ascontiguousarray(indices, np.int64)
    t, _k1 = _table(table)
    s, _k2 = _space(space)
    batch = np.zeros(idx.shape[0], np.int64)
    busy = np.zeros((idx.shape[0], pp_stride), np.int64) if pp_stride else None
    e = _load().orc_eval_indices(C.byref(t), C.byref(s), _ptr(idx), C.c_int64(idx.shape[0]),
                                 int(replicate), _ptr(batch), _ptr(busy) if pp_stride else None,
                                 C.c_int32(pp_stride))
    if e:
        raise OracleError(e)
    return batch, busy


def eval_indices_parallel(table, space, indices, threads: int, replicate: bool = False,
                          pp_stride: int = 0):
    """Farms ``eval_indices`` over host threads (the C call releases the GIL).
    Each candidate is still simulated by one thread."""
    idx = np.ascontiguousarray(indices, np.int64)
    _load()
    if threads <= 1 or idx.shape[0] < 2 * threads:
        return eval_indices(table, space, idx, replicate, pp_stride)
    chunks = np.array_split(np.arange(idx.shape[0]), threads * 4)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        parts = list(ex.map(lambda c: eval_indices(table, space, idx[c], replicate, pp_stride), chunks))
    batch = np.concatenate([p[0] for p in parts])
    busy = np.concatenate([p[1] for p in parts]) if pp_stride else None
    return batch, busy
