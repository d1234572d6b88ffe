"""ctypes access to ``llmem_oracle.c`` (TEST INFRASTRUCTURE ONLY).

Argument marshalling only; every number comes from the C file.  Inputs are
numpy arrays of 64-byte configuration records (any structured dtype of
itemsize 64 with the documented field order).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "llmem_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
# Tests of the pins' strength point this at a deliberately broken build of the oracle.
_OVERRIDE = os.environ.get("LLMEM_ORACLE_LIB")

SELECT_ALLZERO = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if _OVERRIDE:
        return _OVERRIDE
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", tmp, _SRC,
             "-lpthread"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_max_batch.restype = ctypes.c_int32
        _lib.oracle_max_batch_bisect.restype = ctypes.c_int32
    return _lib


def _cfgs(cfg: np.ndarray) -> np.ndarray:
    cfg = np.ascontiguousarray(cfg)
    if cfg.dtype.itemsize != 64:
        raise ValueError("configuration records must be 64 bytes")
    return cfg.reshape(-1)


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _rec(cfg: np.ndarray, i: int = 0):
    return ctypes.c_void_p(cfg.ctypes.data + 64 * i)


# ---- single-configuration calls ------------------------------------------
def validate(cfg: np.ndarray) -> int:
    cfg = _cfgs(cfg)
    return int(lib().oracle_validate(_rec(cfg)))


def inventory(cfg: np.ndarray) -> dict:
    cfg = _cfgs(cfg)
    out = np.zeros(10, dtype=np.int64)
    st = lib().oracle_inventory(_rec(cfg), _p(out))
    if st:
        raise ValueError(f"invalid configuration (status {st})")
    keys = ("e_n", "K", "C", "embed_p", "other_p", "lm_p", "tok_p", "pos_p", "hh_p", "hf_p")
    return dict(zip(keys, (int(v) for v in out)))


def event_count(cfg: np.ndarray, formula: bool = False) -> tuple[int, int]:
    """(status, number of events)."""
    cfg = _cfgs(cfg)
    n = ctypes.c_int64(0)
    f = lib().oracle_event_count_formula if formula else lib().oracle_event_count
    st = f(_rec(cfg), ctypes.byref(n))
    return int(st), int(n.value)


def expand_events(cfg: np.ndarray) -> np.ndarray:
    """Raw signed byte deltas of one configuration."""
    cfg = _cfgs(cfg)
    st, n = event_count(cfg)
    if st:
        raise ValueError(f"status {st}")
    out = np.zeros(n, dtype=np.int64)
    st = lib().oracle_expand_events(_rec(cfg), _p(out), ctypes.c_int64(n))
    assert st == 0
    return out


def round_events(delta: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(delta, dtype=np.int64).copy()
    lib().oracle_round_events(_p(out), ctypes.c_int64(out.size))
    return out


def scan_peak(delta: np.ndarray) -> tuple[int, int]:
    """(max prefix sum, first index attaining it); (0, -1) for an empty list."""
    d = np.ascontiguousarray(delta, dtype=np.int64)
    best, arg = ctypes.c_int64(0), ctypes.c_int64(0)
    lib().oracle_scan_peak(_p(d), ctypes.c_int64(d.size), ctypes.byref(best), ctypes.byref(arg))
    return int(best.value), int(arg.value)


def peak_offset(cfg: np.ndarray) -> tuple[int, int]:
    cfg = _cfgs(cfg)
    off = ctypes.c_int64(0)
    st = lib().oracle_peak_offset(_rec(cfg), ctypes.byref(off))
    return int(st), int(off.value)


# ---- batched calls ---------------------------------------------------------
def estimate(cfg: np.ndarray, level: int = 1, threads: int = 1):
    """Returns dict(peak, index, status, count); index and count are level-1 only."""
    cfg = _cfgs(cfg)
    n = cfg.size
    peak = np.full(n, -1, dtype=np.int64)
    index = np.full(n, -1, dtype=np.int64)
    status = np.zeros(n, dtype=np.uint8)
    count = np.zeros(n, dtype=np.int64)
    lib().oracle_estimate_many(_p(cfg), ctypes.c_int64(n), _p(peak), _p(index), _p(status),
                               _p(count), ctypes.c_int(level), ctypes.c_int(threads))
    return {"peak": peak, "index": index, "status": status, "count": count}


# ---- the DNNMem-style second estimator (Section 3.1) ---------------------------
def dnn_event_count(cfg: np.ndarray) -> tuple[int, int]:
    cfg = _cfgs(cfg)
    n = ctypes.c_int64(0)
    st = lib().oracle_dnn_event_count(_rec(cfg), ctypes.byref(n))
    return int(st), int(n.value)


def dnn_expand_events(cfg: np.ndarray) -> np.ndarray:
    """Raw byte counts of the second estimator's allocations, in order."""
    cfg = _cfgs(cfg)
    st, n = dnn_event_count(cfg)
    if st:
        raise ValueError(f"status {st}")
    out = np.zeros(n, dtype=np.int64)
    st = lib().oracle_dnn_expand_events(_rec(cfg), _p(out), ctypes.c_int64(n))
    assert st == 0
    return out


def dnn_round_events(delta: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(delta, dtype=np.int64).copy()
    lib().oracle_dnn_round_events(_p(out), ctypes.c_int64(out.size))
    return out


def dnn_estimate(cfg: np.ndarray, threads: int = 1):
    """Returns dict(peak, index, status, count) of the second estimator."""
    cfg = _cfgs(cfg)
    n = cfg.size
    peak = np.full(n, -1, dtype=np.int64)
    index = np.full(n, -1, dtype=np.int64)
    status = np.zeros(n, dtype=np.uint8)
    count = np.zeros(n, dtype=np.int64)
    lib().oracle_dnn_estimate_many(_p(cfg), ctypes.c_int64(n), _p(peak), _p(index), _p(status), _p(count),
                                   ctypes.c_int(threads))
    return {"peak": peak, "index": index, "status": status, "count": count}


def list_digest(cfg: np.ndarray, threads: int = 1):
    """Two position-weighted checksums (mod 2^64) of each configuration's page-rounded event
    list: sum d[k] (k + 1) and sum d[k] (k + 1)^2 over the positions k of the list (zeros where
    status != 0).  Returns dict(a, b uint64; status uint8)."""
    cfg = _cfgs(cfg)
    n = cfg.size
    a = np.zeros(n, dtype=np.uint64)
    b = np.zeros(n, dtype=np.uint64)
    status = np.zeros(n, dtype=np.uint8)
    lib().oracle_list_digest_many(_p(cfg), ctypes.c_int64(n), _p(a), _p(b), _p(status), ctypes.c_int(threads))
    return {"a": a, "b": b, "status": status}


def max_batch(cfg: np.ndarray, capacities, bmax: int, level: int = 1, threads: int = 1):
    """Returns (bs[n, n_cap] int32, status[n] uint8)."""
    cfg = _cfgs(cfg)
    caps = np.ascontiguousarray(capacities, dtype=np.int64).reshape(-1)
    n = cfg.size
    bs = np.full((n, caps.size), -1, dtype=np.int32)
    status = np.zeros(n, dtype=np.uint8)
    lib().oracle_max_batch_many(_p(cfg), ctypes.c_int64(n), _p(caps), ctypes.c_int32(caps.size),
                                ctypes.c_int32(bmax), _p(bs), _p(status), ctypes.c_int(level),
                                ctypes.c_int(threads))
    return bs, status


def select_method(cfg: np.ndarray, capacities, bmax: int, flags: int = 0, level: int = 1,
                  threads: int = 1):
    """Returns dict(method[n, n_cap], batch[n, n_cap], bs_list[n, n_cap, 4], status[n])."""
    cfg = _cfgs(cfg)
    caps = np.ascontiguousarray(capacities, dtype=np.int64).reshape(-1)
    n = cfg.size
    method = np.full((n, caps.size), -1, dtype=np.int32)
    batch = np.full((n, caps.size), -1, dtype=np.int32)
    bs_list = np.full((n, caps.size, 4), -1, dtype=np.int32)
    status = np.zeros(n, dtype=np.uint8)
    lib().oracle_select_many(_p(cfg), ctypes.c_int64(n), _p(caps), ctypes.c_int32(caps.size),
                             ctypes.c_int32(bmax), ctypes.c_uint32(flags), _p(method), _p(batch),
                             _p(bs_list), _p(status), ctypes.c_int(level), ctypes.c_int(threads))
    return {"method": method, "batch": batch, "bs_list": bs_list, "status": status}


def decide(bs_list, gpu_n: int, tp_n: int, flags: int = 0) -> tuple[int, int]:
    """Decision step of Algorithm 1 for given per-method largest batches."""
    bl = np.ascontiguousarray(bs_list, dtype=np.int32)
    assert bl.size == 4
    m, b = ctypes.c_int32(0), ctypes.c_int32(0)
    lib().oracle_decide(_p(bl), ctypes.c_int32(gpu_n), ctypes.c_int32(tp_n),
                        ctypes.c_uint32(flags), ctypes.byref(m), ctypes.byref(b))
    return int(m.value), int(b.value)


def select_segmented(item_cfg: np.ndarray, bs: np.ndarray, group_offsets):
    """Decision of Algorithm 1 over arbitrary candidate groups.
    Returns dict(item[n_groups, n_cap] int64, method, batch int32)."""
    item_cfg = _cfgs(item_cfg)
    bs = np.ascontiguousarray(bs, dtype=np.int32)
    assert bs.ndim == 2 and bs.shape[0] == item_cfg.size
    offs = np.ascontiguousarray(group_offsets, dtype=np.int64)
    n_groups, n_cap = offs.size - 1, bs.shape[1]
    item = np.full((n_groups, n_cap), -2, dtype=np.int64)
    method = np.full((n_groups, n_cap), -2, dtype=np.int32)
    batch = np.full((n_groups, n_cap), -2, dtype=np.int32)
    lib().oracle_select_segmented(_p(item_cfg), _p(bs), _p(offs), ctypes.c_int64(n_groups),
                                  ctypes.c_int32(n_cap), _p(item), _p(method), _p(batch))
    return {"item": item, "method": method, "batch": batch}


def chunk_search(cfg: np.ndarray, cs_min: int, cs_step: int, n_candidates: int):
    """Least-waste chunk size per configuration.  Returns dict(chunk, waste int64; status uint8)."""
    cfg = _cfgs(cfg)
    n = cfg.size
    chunk = np.full(n, -1, dtype=np.int64)
    waste = np.full(n, -1, dtype=np.int64)
    status = np.zeros(n, dtype=np.uint8)
    f = lib().oracle_chunk_search
    for i in range(n):
        a, b = ctypes.c_int64(0), ctypes.c_int64(0)
        status[i] = f(_rec(cfg, i), ctypes.c_int64(cs_min), ctypes.c_int64(cs_step),
                      ctypes.c_int32(n_candidates), ctypes.byref(a), ctypes.byref(b))
        chunk[i], waste[i] = a.value, b.value
    return {"chunk": chunk, "waste": waste, "status": status}
