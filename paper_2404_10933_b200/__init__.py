"""Batched LLMem peak-memory estimation on NVIDIA B200.

Thin Python binding of ``csrc/libllmem.so`` (C ABI declared in
``include/llmem.h``).  The functions here only marshal arguments: they allocate
output and scratch tensors with PyTorch, pass raw device pointers and the current
CUDA stream, and check return codes.  Every step of the estimation runs in the
library's CUDA kernels.  There is no CPU fallback: if the shared library is
missing or fails to load, importing a function that needs it raises.

Configurations are 64-byte records (``grids.CONFIG_DTYPE``); on the device they
are ``torch.uint8`` tensors of shape ``[n, 64]``.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

from . import grids  # noqa: F401  (input generators; no part of the model)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libllmem.so")
# the checked build (-DLLMEM_DEBUG); set LLMEM_CHECKED=1 before the first call to load it instead
DEBUG_LIB_PATH = os.path.join(_HERE, "csrc", "libllmem_debug.so")
if os.environ.get("LLMEM_CHECKED") == "1":
    LIB_PATH = DEBUG_LIB_PATH

OK, ERR_ARG, ERR_SCRATCH, ERR_CUDA, ERR_TIMEOUT, ERR_CHECK = 0, 1, 2, 3, 4, 5
OP_ESTIMATE, OP_EVENT_COUNTS, OP_EXPAND, OP_ROUND, OP_SCAN_PEAK, OP_MAX_BATCH, OP_SELECT, OP_EXPAND_SCAN = range(8)
SELECT_ALLZERO = 1
FUSE_ROUND = 2
ESTIMATOR_DNNMEM = 4   # the DNNMem-style estimator of Section 3.1 instead of LLMem
METHOD_OFFLOAD = 4


def _estimator_flag(estimator: str) -> int:
    if estimator == "llmem":
        return 0
    if estimator == "dnnmem":
        return ESTIMATOR_DNNMEM
    raise ValueError("estimator must be 'llmem' or 'dnnmem'")

EXPORTS = (
    "llmem_scratch_bytes", "llmem_estimate_batch", "llmem_event_counts", "llmem_expand_events",
    "llmem_round_events", "llmem_scan_peak", "llmem_max_batch", "llmem_select_method",
    "llmem_scratch_status", "llmem_last_error", "llmem_version", "llmem_event_counts_static",
    "llmem_select_segmented", "llmem_expand_scan", "llmem_chunk_search",
    "llmem_selftest_wait_limit", "llmem_selftest_int_rate", "llmem_checked_build", "llmem_slab_bounds",
)
STATIC_MAX_CONFIGS = 4194304


class LlmemError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"llmem status {code}: {text}")
        self.code = code


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            # a source checkout without build artefacts: compile in-tree if nvcc is at hand
            try:
                from . import _build
                if LIB_PATH == DEBUG_LIB_PATH:
                    _build.build_checked()
                else:
                    _build.build()
            except Exception as e:  # noqa: BLE001
                raise ImportError(
                    f"{LIB_PATH} is missing and could not be built ({e}): build it with "
                    "`python -m paper_2404_10933_b200._build` (needs nvcc); this package has no CPU "
                    "fallback") from e
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, u32, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32,
                                 ctypes.c_size_t)
        L.llmem_scratch_bytes.restype = sz
        L.llmem_scratch_bytes.argtypes = [ctypes.c_int, i64, i64]
        L.llmem_estimate_batch.argtypes = [vp, i64, vp, vp, vp, vp, sz, u32, vp]
        L.llmem_event_counts.argtypes = [vp, i64, vp, vp, vp, sz, u32, vp]
        L.llmem_event_counts_static.argtypes = [vp, i64, vp, vp, u32, vp]
        L.llmem_expand_events.argtypes = [vp, i64, vp, i64, vp, vp, sz, u32, vp]
        L.llmem_round_events.argtypes = [vp, i64, vp, sz, u32, vp]
        L.llmem_scan_peak.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, sz, u32, vp]
        L.llmem_max_batch.argtypes = [vp, i64, vp, i32, i32, vp, vp, vp, sz, u32, vp]
        L.llmem_select_method.argtypes = [vp, i64, vp, i32, i32, vp, vp, vp, vp, vp, sz, u32, vp]
        L.llmem_chunk_search.argtypes = [vp, i64, i64, i64, i32, vp, vp, vp, vp, sz, u32, vp]
        L.llmem_expand_scan.argtypes = [vp, i64, vp, i64, vp, vp, vp, vp, sz, u32, vp]
        L.llmem_select_segmented.argtypes = [vp, vp, vp, i64, i64, i32, vp, vp, vp, vp, sz, u32, vp]
        L.llmem_slab_bounds.argtypes = [vp, i64, i64, i64, vp, vp, i64, vp, vp]
        L.llmem_selftest_wait_limit.argtypes = [vp, sz, u32, vp]
        L.llmem_selftest_int_rate.argtypes = [ctypes.c_int, u32, vp, ctypes.POINTER(i64), vp]
        L.llmem_scratch_status.argtypes = [vp, vp]
        L.llmem_last_error.restype = ctypes.c_char_p
        L.llmem_version.restype = ctypes.c_int
        L.llmem_checked_build.restype = ctypes.c_int
        for name in EXPORTS:
            getattr(L, name)  # every declared entry point must be exported
        _lib = L
    return _lib


def _check(code: int) -> None:
    if code != OK:
        raise LlmemError(code, lib().llmem_last_error().decode())


def _torch():
    import torch
    return torch


def _stream_ptr(stream) -> int:
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def to_device(cfg: np.ndarray, device="cuda", non_blocking: bool = False):
    """Copy 64-byte configuration records to a ``[n, 64]`` uint8 device tensor."""
    torch = _torch()
    cfg = np.ascontiguousarray(cfg)
    if cfg.dtype.itemsize != 64:
        raise ValueError("configuration records must be 64 bytes")
    host = torch.from_numpy(cfg.reshape(-1).view(np.uint8).reshape(-1, 64))
    return host.to(device, non_blocking=non_blocking)


def _as_cfg(cfg):
    torch = _torch()
    if isinstance(cfg, np.ndarray):
        cfg = to_device(cfg)
    if cfg.dtype != torch.uint8 or cfg.dim() != 2 or cfg.shape[1] != 64 or not cfg.is_cuda:
        raise ValueError("cfg must be a CUDA uint8 tensor of shape [n, 64]")
    return cfg.contiguous()


def scratch_bytes(op: int, n: int, total_events: int = 0) -> int:
    return int(lib().llmem_scratch_bytes(op, n, total_events))


def _scratch(op: int, n: int, total: int, device):
    torch = _torch()
    nbytes = scratch_bytes(op, n, total)
    if nbytes == 0:
        return None, 0
    return torch.empty(nbytes, dtype=torch.uint8, device=device), nbytes


def estimate_batch(cfg, *, want_index: bool = True, want_status: bool = True, stream=None, estimator: str = "llmem"):
    """Fused estimate.  ``estimator="dnnmem"`` evaluates the DNNMem-style procedure of the paper's
    Section 3.1 instead.  Returns dict(peak[n] int64, index[n] int64 | None, status[n] uint8 | None)."""
    torch = _torch()
    cfg = _as_cfg(cfg)
    n = cfg.shape[0]
    peak = torch.empty(n, dtype=torch.int64, device=cfg.device)
    index = torch.empty(n, dtype=torch.int64, device=cfg.device) if want_index else None
    status = torch.empty(n, dtype=torch.uint8, device=cfg.device) if want_status else None
    _check(lib().llmem_estimate_batch(_ptr(cfg), n, _ptr(peak), _ptr(index), _ptr(status), None, 0,
                                      _estimator_flag(estimator), _stream_ptr(stream)))
    return {"peak": peak, "index": index, "status": status}


def event_counts(cfg, *, want_status: bool = True, stream=None, estimator: str = "llmem"):
    """Returns (offsets[n+1] int64 exclusive scan of event counts, status[n] | None)."""
    torch = _torch()
    cfg = _as_cfg(cfg)
    n = cfg.shape[0]
    offsets = torch.empty(n + 1, dtype=torch.int64, device=cfg.device)
    status = torch.empty(n, dtype=torch.uint8, device=cfg.device) if want_status else None
    scratch, nbytes = _scratch(OP_EVENT_COUNTS, n, 0, cfg.device)
    _check(lib().llmem_event_counts(_ptr(cfg), n, _ptr(offsets), _ptr(status), _ptr(scratch), nbytes,
                                    _estimator_flag(estimator), _stream_ptr(stream)))
    return offsets, status


def event_counts_static(cfg, offsets_out, status_out=None, *, stream=None):
    """``event_counts`` for callers that must not allocate device memory at the point of
    the call (for instance code running inside a framework callback that may not re-enter
    the allocator, or a service whose device memory is fixed at start-up).  The caller
    passes every tensor, ``offsets_out`` ([n+1] int64) and optionally ``status_out`` ([n]
    uint8); the library's own fixed device array serves as scratch, so neither this
    function nor the library allocates anything.  ``n`` may not exceed
    ``STATIC_MAX_CONFIGS``.  Calls that can overlap on the GPU share that array and race:
    keep them in one stream."""
    torch = _torch()
    if cfg.dtype != torch.uint8 or cfg.dim() != 2 or cfg.shape[1] != 64 or not cfg.is_cuda \
            or not cfg.is_contiguous():
        raise ValueError("cfg must be a contiguous CUDA uint8 tensor of shape [n, 64]")
    n = cfg.shape[0]
    _check_buffer(offsets_out, "offsets_out", torch.int64, n + 1, cfg.device)
    if status_out is not None:
        _check_buffer(status_out, "status_out", torch.uint8, n, cfg.device)
    _check(lib().llmem_event_counts_static(_ptr(cfg), n, _ptr(offsets_out), _ptr(status_out), 0,
                                           _stream_ptr(stream)))
    return offsets_out


def expand_events(cfg, offsets, total_events: Optional[int] = None, *, fuse_round: bool = False,
                  out=None, scratch=None, stream=None, estimator: str = "llmem"):
    """Materialise the signed event list.  ``total_events`` defaults to ``offsets[-1]`` (one
    device-to-host read).  ``scratch`` (optional, 256 bytes) is allocated when not given."""
    torch = _torch()
    cfg = _as_cfg(cfg)
    n = cfg.shape[0]
    if total_events is None:
        total_events = int(offsets[-1].item())
    _check_buffer(offsets, "offsets", torch.int64, n + 1, cfg.device)
    if out is None:
        out = torch.empty(total_events, dtype=torch.int64, device=cfg.device)
    else:
        _check_buffer(out, "out", torch.int64, total_events, cfg.device)
    if scratch is None:
        scratch = torch.empty(scratch_bytes(OP_EXPAND, n, total_events), dtype=torch.uint8, device=cfg.device)
    else:
        _check_buffer(scratch, "scratch", torch.uint8, 0, cfg.device)
    _check(lib().llmem_expand_events(_ptr(cfg), n, _ptr(offsets), total_events, _ptr(out), _ptr(scratch),
                                     scratch.numel(), (FUSE_ROUND if fuse_round else 0) | _estimator_flag(estimator),
                                     _stream_ptr(stream)))
    return out[:total_events] if out.numel() != total_events else out


def round_events(delta, stream=None):
    """Round every magnitude up to the 2 MiB page, in place."""
    _check(lib().llmem_round_events(_ptr(delta), delta.numel(), None, 0, 0, _stream_ptr(stream)))
    return delta


def scan_peak(delta, offsets, cfg=None, *, fuse_round: bool = False, want_index: bool = True,
              scratch=None, stream=None, check_status: bool = False, estimator: str = "llmem"):
    """Segmented prefix-sum + max.  Returns dict(peak[n], index[n] | None, scratch)."""
    torch = _torch()
    if not isinstance(offsets, torch.Tensor) or not offsets.is_cuda:
        raise ValueError("offsets must be a CUDA tensor")
    n = offsets.numel() - 1
    total = delta.numel()
    _check_buffer(offsets, "offsets", torch.int64, 1, offsets.device)
    _check_buffer(delta, "delta", torch.int64, 0, offsets.device)
    if cfg is not None:
        cfg = _as_cfg(cfg)
    peak = torch.empty(n, dtype=torch.int64, device=offsets.device)
    index = torch.empty(n, dtype=torch.int64, device=offsets.device) if want_index else None
    if scratch is None:
        scratch, nbytes = _scratch(OP_SCAN_PEAK, n, total, offsets.device)
    else:
        _check_buffer(scratch, "scratch", torch.uint8, 0, offsets.device)
        nbytes = scratch.numel()
    _check(lib().llmem_scan_peak(_ptr(delta), _ptr(offsets), n, total, _ptr(cfg), _ptr(peak), _ptr(index),
                                 _ptr(scratch), nbytes, (FUSE_ROUND if fuse_round else 0) | _estimator_flag(estimator),
                                 _stream_ptr(stream)))
    if check_status:
        _check(lib().llmem_scratch_status(_ptr(scratch), _stream_ptr(stream)))
    return {"peak": peak, "index": index, "scratch": scratch}


def expand_scan(cfg, offsets, total_events: Optional[int] = None, *, fuse_round: bool = True, out=None,
                want_index: bool = True, scratch=None, stream=None, peak_out=None, index_out=None,
                estimator: str = "llmem"):
    """Materialise the event list and compute the peaks in one pass (the list is written
    once and not read back).  ``peak_out`` / ``index_out`` ([n] int64) receive the results when
    given.  Returns dict(delta, peak[n], index[n] | None, scratch)."""
    torch = _torch()
    cfg = _as_cfg(cfg)
    n = cfg.shape[0]
    if total_events is None:
        total_events = int(offsets[-1].item())
    _check_buffer(offsets, "offsets", torch.int64, n + 1, cfg.device)
    if out is None:
        out = torch.empty(total_events, dtype=torch.int64, device=cfg.device)
    else:
        _check_buffer(out, "out", torch.int64, total_events, cfg.device)
    if peak_out is not None:
        _check_buffer(peak_out, "peak_out", torch.int64, n, cfg.device)
    if index_out is not None:
        _check_buffer(index_out, "index_out", torch.int64, n, cfg.device)
    peak = peak_out if peak_out is not None else torch.empty(n, dtype=torch.int64, device=cfg.device)
    index = index_out if index_out is not None else (
        torch.empty(n, dtype=torch.int64, device=cfg.device) if want_index else None)
    if scratch is None:
        scratch, nbytes = _scratch(OP_EXPAND_SCAN, n, total_events, cfg.device)
    else:
        _check_buffer(scratch, "scratch", torch.uint8, 0, cfg.device)
        nbytes = scratch.numel()
    _check(lib().llmem_expand_scan(_ptr(cfg), n, _ptr(offsets), total_events, _ptr(out), _ptr(peak), _ptr(index),
                                   _ptr(scratch), nbytes, (FUSE_ROUND if fuse_round else 0) | _estimator_flag(estimator),
                                   _stream_ptr(stream)))
    delta = out[:total_events] if out.numel() != total_events else out
    return {"delta": delta, "peak": peak, "index": index, "scratch": scratch}


def max_batch(shape, capacities, bmax: int, *, want_status: bool = True, stream=None):
    """Largest fitting batch.  Returns (bs[n, n_cap] int32, status[n] | None)."""
    torch = _torch()
    shape = _as_cfg(shape)
    n = shape.shape[0]
    caps = _caps(capacities, shape.device)
    bs = torch.empty((n, caps.numel()), dtype=torch.int32, device=shape.device)
    status = torch.empty(n, dtype=torch.uint8, device=shape.device) if want_status else None
    _check(lib().llmem_max_batch(_ptr(shape), n, _ptr(caps), caps.numel(), bmax, _ptr(bs), _ptr(status),
                                 None, 0, 0, _stream_ptr(stream)))
    return bs, status


def select_method(shape, capacities, bmax: int, *, allzero: bool = False, want_bs_list: bool = True,
                  want_status: bool = True, stream=None):
    """Algorithm 1.  Returns dict(method[n, n_cap], batch[n, n_cap], bs_list[n, n_cap, 4] | None,
    status[n] | None)."""
    torch = _torch()
    shape = _as_cfg(shape)
    n = shape.shape[0]
    caps = _caps(capacities, shape.device)
    m = caps.numel()
    method = torch.empty((n, m), dtype=torch.int32, device=shape.device)
    batch = torch.empty((n, m), dtype=torch.int32, device=shape.device)
    bs_list = torch.empty((n, m, 4), dtype=torch.int32, device=shape.device) if want_bs_list else None
    status = torch.empty(n, dtype=torch.uint8, device=shape.device) if want_status else None
    _check(lib().llmem_select_method(_ptr(shape), n, _ptr(caps), m, bmax, _ptr(method), _ptr(batch),
                                     _ptr(bs_list), _ptr(status), None, 0,
                                     SELECT_ALLZERO if allzero else 0, _stream_ptr(stream)))
    return {"method": method, "batch": batch, "bs_list": bs_list, "status": status}


def select_segmented(item_cfg, bs, group_offsets, *, stream=None):
    """Algorithm 1's decision over arbitrary candidate groups.  ``bs`` is the [n_items, n_cap]
    matrix written by ``max_batch`` for ``item_cfg``; ``group_offsets`` ([n_groups+1] int64)
    delimits the groups.  Returns dict(item[n_groups, n_cap] int64, method, batch int32)."""
    torch = _torch()
    item_cfg = _as_cfg(item_cfg)
    n_items, n_cap = bs.shape
    if not isinstance(group_offsets, torch.Tensor):
        group_offsets = torch.as_tensor(np.asarray(group_offsets, dtype=np.int64))
    group_offsets = group_offsets.to(device=item_cfg.device, dtype=torch.int64).contiguous()
    n_groups = group_offsets.numel() - 1
    item = torch.empty((n_groups, n_cap), dtype=torch.int64, device=item_cfg.device)
    method = torch.empty((n_groups, n_cap), dtype=torch.int32, device=item_cfg.device)
    batch = torch.empty((n_groups, n_cap), dtype=torch.int32, device=item_cfg.device)
    _check(lib().llmem_select_segmented(_ptr(item_cfg), _ptr(bs.contiguous()), _ptr(group_offsets), n_groups,
                                        n_items, n_cap, _ptr(item), _ptr(method), _ptr(batch), None, 0, 0,
                                        _stream_ptr(stream)))
    return {"item": item, "method": method, "batch": batch}


def chunk_search(cfg, cs_min: int, cs_step: int, n_candidates: int, *, stream=None):
    """Least-waste chunk size among cs_min + k cs_step.  Returns dict(chunk[n], waste[n] int64,
    status[n] uint8)."""
    torch = _torch()
    cfg = _as_cfg(cfg)
    n = cfg.shape[0]
    chunk = torch.empty(n, dtype=torch.int64, device=cfg.device)
    waste = torch.empty(n, dtype=torch.int64, device=cfg.device)
    status = torch.empty(n, dtype=torch.uint8, device=cfg.device)
    _check(lib().llmem_chunk_search(_ptr(cfg), n, cs_min, cs_step, n_candidates, _ptr(chunk), _ptr(waste),
                                    _ptr(status), None, 0, 0, _stream_ptr(stream)))
    return {"chunk": chunk, "waste": waste, "status": status}


def _check_buffer(t, name: str, dtype, min_numel: int, device) -> None:
    """A tensor supplied by the caller that a kernel will write: it has to be device memory
    of the configurations' GPU, contiguous, of the right type and long enough (a pointer to
    anything else would be written all the same)."""
    torch = _torch()
    if not isinstance(t, torch.Tensor) or not t.is_cuda or t.device != device:
        raise ValueError(f"{name} must be a CUDA tensor on {device}")
    if t.dtype != dtype or not t.is_contiguous() or t.numel() < min_numel:
        raise ValueError(f"{name} must be a contiguous {dtype} tensor with at least {min_numel} elements")


def _caps(capacities, device):
    torch = _torch()
    if isinstance(capacities, torch.Tensor):
        caps = capacities.to(device=device, dtype=torch.int64).contiguous().reshape(-1)
    else:
        caps = torch.as_tensor(np.asarray(capacities, dtype=np.int64).reshape(-1)).to(device)
    return caps


def estimate_materialized(cfg, *, fuse_round: bool = True, stream=None, estimator: str = "llmem"):
    """The materialised path end to end: event counts -> expansion -> (rounding) ->
    segmented scan.  Returns dict(peak, index, status, offsets, total_events)."""
    cfg = _as_cfg(cfg)
    if estimator != "llmem" and not fuse_round:
        raise ValueError("the separate rounding pass rounds to the 2 MiB page: use fuse_round with this estimator")
    offsets, status = event_counts(cfg, stream=stream, estimator=estimator)
    total = int(offsets[-1].item())
    delta = expand_events(cfg, offsets, total, fuse_round=fuse_round, stream=stream, estimator=estimator)
    if not fuse_round:
        round_events(delta, stream=stream)
    r = scan_peak(delta, offsets, cfg, stream=stream, estimator=estimator)
    return {"peak": r["peak"], "index": r["index"], "status": status, "offsets": offsets,
            "total_events": total}


def slab_bounds(offsets, max_events: int, first_config: int = 0, *, max_slabs: int = 4096, stream=None):
    """Cut configurations [first_config, n) into contiguous slabs of at most ``max_events``
    events (``llmem_slab_bounds``; the cut runs on the device, only the few boundaries come
    back).  Returns (bounds, events): numpy int64 arrays, slab k = configurations
    bounds[k] .. bounds[k+1]-1 with events[k+1] - events[k] events."""
    torch = _torch()
    _check_buffer(offsets, "offsets", torch.int64, 1, offsets.device)
    n = offsets.numel() - 1
    out = torch.empty(2 * (max_slabs + 1) + 1, dtype=torch.int64, device=offsets.device)
    bounds, events, count = out[:max_slabs + 1], out[max_slabs + 1:2 * (max_slabs + 1)], out[-1:]
    _check(lib().llmem_slab_bounds(_ptr(offsets), n, max_events, first_config, _ptr(bounds), _ptr(events), max_slabs,
                                   _ptr(count), _stream_ptr(stream)))
    host = out.cpu().numpy()
    k = int(host[-1])
    if k < 0:
        raise ValueError(f"more than {max_slabs} slabs of {max_events} events: raise max_slabs or max_events")
    return host[:k + 1].copy(), host[max_slabs + 1:max_slabs + 2 + k].copy()


def estimate_in_slabs(cfg, max_events: int, *, first_config: int = 0, on_slab=None, stream=None):
    """The materialised path for grids whose event lists do not fit in device memory at
    once: the configurations are cut into contiguous slabs of at most ``max_events`` events
    (``llmem_slab_bounds``), and every slab is expanded, page-rounded and scanned by
    ``llmem_expand_scan`` through one list buffer and one scratch buffer that are reused.
    ``first_config`` restarts an interrupted run at a slab boundary (earlier results are then
    left at -1).  ``on_slab(lo, hi, delta, offsets)`` is called after each slab with its
    configuration range, its event list (valid until the next slab) and its local offsets.
    Returns dict(peak[n], index[n], status[n], bounds): ``bounds`` are the slab boundaries."""
    torch = _torch()
    cfg = _as_cfg(cfg)
    n = cfg.shape[0]
    offsets, status = event_counts(cfg, stream=stream)
    bounds, events = slab_bounds(offsets, max_events, first_config, stream=stream)
    sizes = np.diff(events)
    capacity = int(sizes.max()) if len(sizes) else 0
    delta = torch.empty(max(capacity, 1), dtype=torch.int64, device=cfg.device)
    nbytes = max([scratch_bytes(OP_EXPAND_SCAN, int(hi - lo), int(t))
                  for lo, hi, t in zip(bounds[:-1], bounds[1:], sizes)] + [scratch_bytes(OP_EXPAND_SCAN, 0, 0)])
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=cfg.device)
    peak = torch.full((n,), -1, dtype=torch.int64, device=cfg.device)
    index = torch.full((n,), -1, dtype=torch.int64, device=cfg.device)
    for lo, hi, total in zip(bounds[:-1].tolist(), bounds[1:].tolist(), sizes.tolist()):
        part = cfg[lo:hi]
        local, _ = event_counts(part, want_status=False, stream=stream)
        r = expand_scan(part, local, int(total), fuse_round=True, out=delta, scratch=scratch, stream=stream,
                        peak_out=peak[lo:hi], index_out=index[lo:hi])
        if on_slab is not None:
            on_slab(lo, hi, r["delta"], local)
    return {"peak": peak, "index": index, "status": status, "bounds": bounds}


def int_rate(kind: int = 0, iters: int = 4096, reps: int = 3, stream=None) -> float:
    """Warp instructions per second of the issue-rate probe (``llmem_selftest_int_rate``):
    kind 0 add/xor, 1 multiply-add, 2 alternating.  Timed with CUDA events, best of ``reps``."""
    torch = _torch()
    count = ctypes.c_int64(0)
    best = None
    for _ in range(reps + 1):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        _check(lib().llmem_selftest_int_rate(kind, iters, None, ctypes.byref(count), _stream_ptr(stream)))
        b.record(stream)
        b.synchronize()
        ms = a.elapsed_time(b)
        best = ms if best is None or ms < best else best
    return count.value / (best * 1e-3)
