"""CPU-side checks: the C-ABI library loads and exports what the header declares,
the input generators are deterministic and well-formed, and argument errors are
reported by return code without touching a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2404_10933_b200 as llmem
from paper_2404_10933_b200 import grids

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "llmem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(llmem_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2404_10933_b200 import _build
    _build.build()
    L = llmem.lib()
    names = declared_symbols()
    assert len(names) >= 11
    for name in names:
        assert hasattr(L, name), name
    assert sorted(llmem.EXPORTS) == names
    assert L.llmem_version() >= 100


def test_scratch_bytes_and_argument_errors_need_no_gpu():
    L = llmem.lib()
    assert L.llmem_scratch_bytes(llmem.OP_ESTIMATE, 1000, 0) == 0
    assert L.llmem_scratch_bytes(llmem.OP_EXPAND, 1000, 10 ** 9) == 256  # optional: the work counter
    # lists of short segments: a descriptor per configuration for the expansion by segment owners
    assert L.llmem_scratch_bytes(llmem.OP_EXPAND, 1000, 10 ** 6) == L.llmem_scratch_bytes(llmem.OP_EXPAND_SCAN, 1000, 10 ** 6)
    assert L.llmem_scratch_bytes(llmem.OP_EXPAND_SCAN, 1000, 10 ** 6) > 1000 * 800
    assert L.llmem_scratch_bytes(llmem.OP_EVENT_COUNTS, 5000, 0) >= 256 + 8 * 6
    assert L.llmem_scratch_bytes(llmem.OP_SCAN_PEAK, 5000, 10 ** 9) >= 256 + 64
    # call-level errors are detected before any CUDA call
    assert L.llmem_estimate_batch(None, -1, None, None, None, None, 0, 0, None) == llmem.ERR_ARG
    assert b"n < 0" in L.llmem_last_error()
    assert L.llmem_estimate_batch(None, 5, None, None, None, None, 0, 0, None) == llmem.ERR_ARG
    assert L.llmem_max_batch(ctypes.c_void_p(16), 5, ctypes.c_void_p(16), 1, 0, ctypes.c_void_p(16),
                             None, None, 0, 0, None) == llmem.ERR_ARG          # bmax < 1
    assert L.llmem_estimate_batch(ctypes.c_void_p(8), 5, ctypes.c_void_p(16), None, None, None, 0, 0,
                                  None) == llmem.ERR_ARG                        # cfg misaligned
    assert L.llmem_scan_peak(ctypes.c_void_p(16), ctypes.c_void_p(16), 5, 10, None, ctypes.c_void_p(16),
                             None, None, 0, 0, None) == llmem.ERR_SCRATCH
    assert L.llmem_event_counts(ctypes.c_void_p(16), 5, ctypes.c_void_p(16), None, ctypes.c_void_p(256), 8,
                                0, None) == llmem.ERR_SCRATCH
    # chunk-size candidates beyond 2^40 are refused even where cs_min + k cs_step wraps 64 bits
    for n_cand, step in ((1 << 24, 1 << 40), ((1 << 24) + 1, 1 << 40), (1 << 30, (1 << 34) + 1), (2, 1 << 40)):
        assert L.llmem_chunk_search(ctypes.c_void_p(16), 1, 1, step, n_cand, ctypes.c_void_p(16), None, None,
                                    None, 0, 0, None) == llmem.ERR_ARG, (n_cand, step)
    assert b"2^40" in L.llmem_last_error()
    # empty calls succeed
    assert L.llmem_chunk_search(None, 0, 1, (1 << 40) - 1, 2, None, None, None, None, 0, 0, None) == llmem.OK
    assert L.llmem_estimate_batch(None, 0, None, None, None, None, 0, 0, None) == llmem.OK
    assert L.llmem_round_events(None, 0, None, 0, 0, None) == llmem.OK
    assert L.llmem_last_error() == b""


def test_wrappers_refuse_buffers_a_kernel_could_not_write():
    """Tensors the caller supplies for a kernel to write are checked before any launch: host
    memory, another device, the wrong type, a strided view or too few elements raise."""
    torch = pytest.importorskip("torch")
    dev = torch.device("cuda", 0)
    host = torch.zeros(16, dtype=torch.int64)
    with pytest.raises(ValueError, match="CUDA tensor"):
        llmem._check_buffer(host, "offsets_out", torch.int64, 4, dev)
    with pytest.raises(ValueError, match="CUDA tensor"):
        llmem._check_buffer(None, "out", torch.int64, 4, dev)
    with pytest.raises(ValueError, match="CUDA tensor"):
        llmem._check_buffer(host.numpy(), "out", torch.int64, 4, dev)
    # the public wrappers reach that check (or the one on cfg) before touching the library
    cfg_host = torch.zeros((4, 64), dtype=torch.uint8)
    with pytest.raises(ValueError):
        llmem.event_counts_static(cfg_host, host)
    with pytest.raises(ValueError):
        llmem.expand_scan(cfg_host, host, 8, out=host)
    with pytest.raises(ValueError):
        llmem.expand_events(cfg_host, host, 8, out=host)
    with pytest.raises(ValueError):
        llmem.scan_peak(host, host)


def test_record_layout_matches_header():
    text = open(os.path.join(ROOT, "include", "llmem.h")).read()
    body = text[text.index("typedef struct __attribute__((aligned(16))) llmem_config {"):text.index("} llmem_config;")]
    fields = re.findall(r"^\s*(int32_t|int64_t|uint8_t)\s+(\w+)(\[\d+\])?;", body, flags=re.M)
    assert [f[1] for f in fields] == list(grids.CONFIG_DTYPE.names)
    size = {"int32_t": 4, "int64_t": 8, "uint8_t": 1}
    off = 0
    for ctype, name, arr in fields:
        assert grids.CONFIG_DTYPE.fields[name][1] == off, name
        off += size[ctype] * (int(arr[1:-1]) if arr else 1)
    assert off == 64 == grids.CONFIG_DTYPE.itemsize


def test_grids_are_deterministic_and_sliceable():
    a = grids.g3_sweep(1000, 50)
    b = grids.g3_sweep(0, 2000)[1000:1050]
    assert a.tobytes() == b.tobytes()
    assert grids.g5_stress(10, 5).tobytes() == grids.g5_stress(0, 20)[10:15].tobytes()
    assert grids.g5_stress(0, 8, seed_offset=1).tobytes() != grids.g5_stress(0, 8).tobytes()


def test_grid_shapes_and_ranges():
    g1 = grids.g1_small()
    assert len(g1) == 64 and g1["batch"].tolist() == list(range(1, 65))
    combos = grids.g2_combos()
    assert len(combos) == 29
    assert [(n, t) for m, n, t in combos if m == 3] == [(4, 2), (6, 2), (6, 3), (8, 2), (8, 4)]
    g2 = grids.g2_shape_grid(0, 3)
    assert len(g2) == 3 * 32 * 29
    assert set(np.unique(g2["hidden"]) % 256) == {0}
    assert g2["layers"].min() >= 4 and g2["layers"].max() <= 48
    assert ((g2["hidden"] % g2["heads"]) == 0).all()
    g3 = grids.g3_sweep(0, 20000)
    assert g3["gpu_n"].min() == 1 and g3["gpu_n"].max() == 16
    assert set(np.unique(g3["seq"])) == {128, 256, 512, 1024, 2048, 4096}
    dptp = g3[g3["method"] == 3]
    assert len(dptp) > 0
    assert ((dptp["gpu_n"] % dptp["tp_n"]) == 0).all() and (dptp["tp_n"] >= 2).all()
    assert (2 * dptp["tp_n"].astype(int) <= dptp["gpu_n"]).all()
    assert set(np.unique(g3["method"])) == {0, 1, 2, 3}
    g4 = grids.g4_search_grid(0, 2)
    assert len(g4) == 2 * 64
    g4s = grids.g4_select_grid(0, 2)
    assert len(g4s) == 2 * 16 and g4s["tp_n"][:16].tolist() == [0, 0, 0, 2, 0, 2, 0, 2, 3, 2, 0, 2, 0, 2, 3, 2]
    g5 = grids.g5_stress(0, 1000)
    assert g5["layers"].min() >= 64 and g5["hidden"].min() >= 8192 and (g5["chunk_elems"] == 1 << 23).all()
    assert grids.g4_capacities().tolist() == [g << 30 for g in (16, 24, 40, 48, 80, 96, 141, 180, 192)]


def test_shard_bounds_balance_weights():
    w = np.array([5, 1, 1, 1, 1, 1, 5, 5], dtype=np.int64)
    b = grids.shard_bounds(w, 2)
    assert b[0] == 0 and b[-1] == len(w) and (np.diff(b) >= 0).all()
    left = w[b[0]:b[1]].sum()
    assert abs(left - w.sum() / 2) <= w.max()
    assert grids.shard_bounds(w, 1).tolist() == [0, 8]
    assert grids.shard_bounds(np.ones(3), 8)[-1] == 3


def test_slab_bounds_cover_and_respect_the_budget():
    from paper_2404_10933_b200 import grids
    rng = np.random.default_rng(4)
    counts = rng.integers(0, 5000, size=300)
    counts[[17, 140]] = 60000                      # larger than the budget: slabs of their own
    counts[50:60] = 0                              # inadmissible records have no events
    off = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    for budget in (1, 4999, 20000, 10 ** 9):
        for first in (0, 23, 300):
            b = grids.slab_bounds(off, budget, first)
            assert b[0] == first and b[-1] == 300 and (np.diff(b) > 0).all()
            assert len(b) > 1 or first == 300
            for lo, hi in zip(b[:-1], b[1:]):
                events = off[hi] - off[lo]
                assert events <= budget or hi == lo + 1
                # greedy: the next configuration would not have fitted
                if hi < 300 and hi > lo + 1:
                    assert off[hi + 1] - off[lo] > budget
    with pytest.raises(ValueError):
        grids.slab_bounds(off, 0)
    with pytest.raises(ValueError):
        grids.slab_bounds(off, 10, 301)


def test_checked_build_exports_the_same_entry_points():
    from paper_2404_10933_b200 import _build
    assert llmem.lib().llmem_checked_build() == 0
    if not os.path.exists(_build.DEBUG_LIB):
        _build.build_checked()
    D = ctypes.CDLL(_build.DEBUG_LIB)
    for name in declared_symbols():
        getattr(D, name)
    D.llmem_checked_build.restype = ctypes.c_int
    assert D.llmem_checked_build() == 1


def test_bench_constants_are_the_figures_of_the_committed_profiles():
    """bench.py scales profiler counters (DRAM bytes per event, lane instructions per unit) that
    were captured on reduced cases; the figures it uses must be the ones the summaries under
    profiles/ state, so that neither can be updated without the other."""
    import importlib.util
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)

    def rows(name):
        with open(os.path.join(root, "profiles", name)) as f:
            return [[c.strip() for c in line.strip().strip("|").split("|")] for line in f if line.startswith("|")]

    g5 = [r for r in rows("expand_scan_g5_4096cfg_ncu.md") if r[0].startswith("traffic per event")]
    assert len(g5) == 1
    one_pass, expand, scan = (float(c.split()[0]) for c in g5[0][1:4])
    assert bench.NCU_TRAFFIC_BYTES_PER_EVENT == {"expand": expand, "scan": scan, "expand_scan": one_pass}
    owners = [r for r in rows("expand_scan_owned_g2_64shapes_ncu.md") if r[0].startswith("traffic per event")]
    assert len(owners) == 1 and float(owners[0][2].split()[0]) == bench.NCU_TRAFFIC_BYTES_PER_EVENT_OWNERS
    table = rows("register_kernels_g3_g4_ncu.md")
    head = next(r for r in table if r[0] == "kernel" and "lane instr / 32 / unit" in r)
    col = head.index("lane instr / 32 / unit")
    for kernel, value in bench.NCU_LANE_INSTR_PER_UNIT.items():
        row = next(r for r in table if r[0].startswith(kernel) and len(r) == len(head))
        assert float(row[col]) == value, kernel
