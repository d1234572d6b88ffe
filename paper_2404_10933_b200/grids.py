"""Seeded synthetic configuration grids (inputs only).

This module draws decoder shapes and fine-tuning settings and packs them into
the 64-byte configuration record that the estimator consumes.  It contains no
part of the memory model itself: no parameter counts, no event sizes, no
rounding.  The only method-related knowledge it holds is which
(method, gpu_n, tp_n) triples are admissible inputs, so that a grid can be
restricted to them.

Every draw is a pure function of ``(seed, index, field)`` through a 64-bit
counter-based mixer (the SplitMix64 output function of Steele, Lea and Flood,
"Fast splittable pseudorandom number generators", OOPSLA 2014), so any slice
of any grid can be regenerated without generating what precedes it.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# record layout (64 bytes, little endian, no padding)
# --------------------------------------------------------------------------
CONFIG_DTYPE = np.dtype(
    [
        ("layers", "<i4"),
        ("hidden", "<i4"),
        ("heads", "<i4"),
        ("ffn", "<i4"),
        ("vocab", "<i4"),
        ("pos_len", "<i4"),
        ("seq", "<i4"),
        ("batch", "<i4"),
        ("chunk_elems", "<i8"),
        ("base_bytes", "<i8"),
        ("method", "u1"),
        ("gpu_n", "u1"),
        ("tp_n", "u1"),
        ("lm_bytes", "u1"),
        ("ffn_kind", "u1"),
        ("has_bias", "u1"),
        ("iters", "u1"),
        ("act_mode", "u1"),
        ("reserved", "u1", (8,)),
    ]
)
assert CONFIG_DTYPE.itemsize == 64

METHOD_CDP, METHOD_ADP, METHOD_TP, METHOD_DPTP = 0, 1, 2, 3
METHOD_NAMES = ("CDP", "ADP", "TP", "DP+TP")

SEED_BASE = 0x240410933
GIB = 1 << 30
MIB = 1 << 20

# Device capacities of the max-batch grid, in GiB.
G4_CAPACITIES_GIB = (16, 24, 40, 48, 80, 96, 141, 180, 192)

# field ids for the mixer
(_F_LAYERS, _F_HIDDEN, _F_HEADS, _F_FFNKIND, _F_VOCAB, _F_POS, _F_SEQ, _F_BATCH,
 _F_CHUNK, _F_BASE, _F_METHOD, _F_GPUN, _F_TPN, _F_LMB) = range(14)


def _mix(seed: int, index, field: int) -> np.ndarray:
    """SplitMix64 output function applied to a (seed, index, field) counter."""
    idx = np.asarray(index, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
             + idx * np.uint64(0x9E3779B97F4A7C15)
             + np.uint64(field + 1) * np.uint64(0xD1B54A32D192ED03))
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def _uniform(seed: int, index, field: int, lo: int, hi: int) -> np.ndarray:
    """Integers in [lo, hi] (inclusive)."""
    span = np.uint64(hi - lo + 1)
    return ((_mix(seed, index, field) >> np.uint64(11)) % span).astype(np.int64) + lo


def _choice(seed: int, index, field: int, values) -> np.ndarray:
    values = np.asarray(values, dtype=np.int64)
    return values[_uniform(seed, index, field, 0, len(values) - 1)]


def valid_tp_degrees(gpu_n: int) -> list[int]:
    """tp_n values admissible for DP+TP on gpu_n devices: 2 <= t <= n/2, t | n."""
    return [t for t in range(2, gpu_n // 2 + 1) if gpu_n % t == 0]


def empty(n: int) -> np.ndarray:
    return np.zeros(n, dtype=CONFIG_DTYPE)


def _round_up(x, m):
    return (x + m - 1) // m * m


def _draw_shapes(seed: int, index: np.ndarray, *, layers, hidden_lo, hidden_hi, hidden_step,
                 vocab, seqs, chunks) -> np.ndarray:
    """Common shape draw: the fields that describe a decoder, not how it is fine-tuned."""
    n = len(index)
    c = empty(n)
    c["layers"] = _uniform(seed, index, _F_LAYERS, *layers)
    hidden = hidden_lo + hidden_step * _uniform(
        seed, index, _F_HIDDEN, 0, (hidden_hi - hidden_lo) // hidden_step)
    c["hidden"] = hidden
    head_dim = _choice(seed, index, _F_HEADS, (64, 128))
    c["heads"] = hidden // head_dim
    gated = _uniform(seed, index, _F_FFNKIND, 0, 1)
    c["ffn_kind"] = gated
    c["has_bias"] = 1 - gated
    c["ffn"] = np.where(gated == 1, _round_up(8 * hidden // 3, 256), 4 * hidden)
    c["vocab"] = _uniform(seed, index, _F_VOCAB, *vocab)
    c["pos_len"] = _choice(seed, index, _F_POS, (0, 2048))
    c["seq"] = _choice(seed, index, _F_SEQ, seqs)
    c["chunk_elems"] = _choice(seed, index, _F_CHUNK, chunks)
    c["base_bytes"] = _uniform(seed, index, _F_BASE, 256 * MIB, 1 * GIB)
    c["lm_bytes"] = _choice(seed, index, _F_LMB, (2, 4))
    c["iters"] = 2
    c["batch"] = 1
    c["gpu_n"] = 1
    return c


def _draw_method(seed: int, index: np.ndarray, c: np.ndarray, n_max: int) -> None:
    """gpu_n uniform in 1..n_max; method uniform over those admissible for it."""
    gpu_n = _uniform(seed, index, _F_GPUN, 1, n_max)
    r_method = _mix(seed, index, _F_METHOD) >> np.uint64(11)
    r_tp = _mix(seed, index, _F_TPN) >> np.uint64(11)
    method = np.zeros(len(index), dtype=np.int64)
    tp_n = np.zeros(len(index), dtype=np.int64)
    for n in range(1, n_max + 1):
        sel = gpu_n == n
        if not sel.any():
            continue
        degs = valid_tp_degrees(n)
        n_methods = 4 if degs else 3
        m = (r_method[sel] % np.uint64(n_methods)).astype(np.int64)
        method[sel] = m
        if degs:
            t = np.asarray(degs, dtype=np.int64)[(r_tp[sel] % np.uint64(len(degs))).astype(np.int64)]
            tp_n[sel] = np.where(m == METHOD_DPTP, t, 0)
    c["gpu_n"] = gpu_n
    c["method"] = method
    c["tp_n"] = tp_n


# --------------------------------------------------------------------------
# G1: one small decoder, batch 1..64
# --------------------------------------------------------------------------
def g1_small() -> np.ndarray:
    c = empty(64)
    c["layers"], c["hidden"], c["heads"], c["ffn"] = 12, 768, 12, 3072
    c["vocab"], c["pos_len"], c["seq"] = 50257, 1024, 512
    c["batch"] = np.arange(1, 65)
    c["chunk_elems"] = 1 << 20
    c["base_bytes"] = 0
    c["method"], c["gpu_n"], c["tp_n"] = METHOD_CDP, 1, 0
    c["lm_bytes"], c["ffn_kind"], c["has_bias"], c["iters"] = 2, 0, 1, 2
    return c


# --------------------------------------------------------------------------
# G2: shape grid x batch 1..32 x (method, degree)
# --------------------------------------------------------------------------
G2_SHAPES = 4096
G2_BATCHES = 32


def g2_combos() -> list[tuple[int, int, int]]:
    """(method, gpu_n, tp_n) triples of the shape grid: 3 methods x n=1..8 plus admissible DP+TP."""
    out = [(m, n, 0) for m in (METHOD_CDP, METHOD_ADP, METHOD_TP) for n in range(1, 9)]
    out += [(METHOD_DPTP, n, t) for n in range(1, 9) for t in valid_tp_degrees(n)]
    return out


def g2_shapes(first: int = 0, count: int = G2_SHAPES) -> np.ndarray:
    idx = np.arange(first, first + count, dtype=np.uint64)
    return _draw_shapes(SEED_BASE + 2, idx, layers=(4, 48), hidden_lo=512, hidden_hi=8192,
                        hidden_step=256, vocab=(32000, 128000), seqs=(256, 512, 1024, 2048),
                        chunks=[1 << k for k in range(20, 25)])


def g2_shape_grid(first: int = 0, count: int = G2_SHAPES) -> np.ndarray:
    """Configs ordered [shape][batch][combo]."""
    shapes = g2_shapes(first, count)
    combos = g2_combos()
    nb, nc = G2_BATCHES, len(combos)
    c = np.repeat(shapes, nb * nc)
    c["batch"] = np.tile(np.repeat(np.arange(1, nb + 1), nc), count)
    cm = np.asarray(combos, dtype=np.int64)
    c["method"] = np.tile(cm[:, 0], count * nb)
    c["gpu_n"] = np.tile(cm[:, 1], count * nb)
    c["tp_n"] = np.tile(cm[:, 2], count * nb)
    return c


# --------------------------------------------------------------------------
# G3: large i.i.d. sweep
# --------------------------------------------------------------------------
G3_CONFIGS = 1 << 20


def _g3_like_shapes(seed: int, idx: np.ndarray) -> np.ndarray:
    return _draw_shapes(seed, idx, layers=(12, 80), hidden_lo=1024, hidden_hi=8192,
                        hidden_step=256, vocab=(32000, 256000),
                        seqs=[1 << k for k in range(7, 13)],
                        chunks=[1 << k for k in range(22, 26)])


def g3_sweep(first: int = 0, count: int = G3_CONFIGS) -> np.ndarray:
    idx = np.arange(first, first + count, dtype=np.uint64)
    c = _g3_like_shapes(SEED_BASE + 3, idx)
    c["batch"] = _uniform(SEED_BASE + 3, idx, _F_BATCH, 1, 256)
    _draw_method(SEED_BASE + 3, idx, c, 16)
    return c


# --------------------------------------------------------------------------
# G4: max-batch search and method selection
# --------------------------------------------------------------------------
G4_SHAPES = 1 << 17
G4_BMAX = 4096
G4_DEGREES = 16


def g4_capacities() -> np.ndarray:
    return np.asarray(G4_CAPACITIES_GIB, dtype=np.int64) * GIB


def g4_shapes(first: int = 0, count: int = G4_SHAPES) -> np.ndarray:
    idx = np.arange(first, first + count, dtype=np.uint64)
    return _g3_like_shapes(SEED_BASE + 4, idx)


def _smallest_tp(n: int) -> int:
    degs = valid_tp_degrees(n)
    return degs[0] if degs else 0


def g4_search_grid(first: int = 0, count: int = G4_SHAPES) -> np.ndarray:
    """Configs ordered [shape][method][gpu_n]; DP+TP uses the smallest admissible tp_n
    (tp_n = 0, an inadmissible input, where gpu_n has none)."""
    shapes = g4_shapes(first, count)
    per = 4 * G4_DEGREES
    c = np.repeat(shapes, per)
    method = np.repeat(np.arange(4), G4_DEGREES)
    gpu_n = np.tile(np.arange(1, G4_DEGREES + 1), 4)
    tp_n = np.where(method == METHOD_DPTP, [_smallest_tp(int(n)) for n in gpu_n], 0)
    c["method"] = np.tile(method, count)
    c["gpu_n"] = np.tile(gpu_n, count)
    c["tp_n"] = np.tile(tp_n, count)
    return c


def g4_select_grid(first: int = 0, count: int = G4_SHAPES) -> np.ndarray:
    """Configs ordered [shape][gpu_n]; tp_n = smallest admissible divisor or 0."""
    shapes = g4_shapes(first, count)
    c = np.repeat(shapes, G4_DEGREES)
    gpu_n = np.arange(1, G4_DEGREES + 1)
    c["gpu_n"] = np.tile(gpu_n, count)
    c["tp_n"] = np.tile([_smallest_tp(int(n)) for n in gpu_n], count)
    return c


def all_split_candidates(n_max: int = G4_DEGREES) -> list[tuple[int, int, int]]:
    """Every (method, gpu_n, tp_n) candidate on up to n_max devices, ordered by degree,
    then CDP, ADP, TP, then the DP+TP splits by increasing tp_n (67 candidates for 16)."""
    out = []
    for n in range(1, n_max + 1):
        out += [(METHOD_CDP, n, 0), (METHOD_ADP, n, 0), (METHOD_TP, n, 0)]
        out += [(METHOD_DPTP, n, t) for t in valid_tp_degrees(n)]
    return out


def g4_all_splits_grid(first: int = 0, count: int = G4_SHAPES, n_max: int = G4_DEGREES):
    """Configs ordered [shape][candidate] and the group offsets (one group per shape)."""
    shapes = g4_shapes(first, count)
    cand = np.asarray(all_split_candidates(n_max), dtype=np.int64)
    k = len(cand)
    c = np.repeat(shapes, k)
    c["method"] = np.tile(cand[:, 0], count)
    c["gpu_n"] = np.tile(cand[:, 1], count)
    c["tp_n"] = np.tile(cand[:, 2], count)
    return c, np.arange(count + 1, dtype=np.int64) * k


# --------------------------------------------------------------------------
# G5: deep/wide stress grid with long event lists
# --------------------------------------------------------------------------
G5_CONFIGS = 1 << 16


def g5_stress(first: int = 0, count: int = G5_CONFIGS, seed_offset: int = 0) -> np.ndarray:
    seed = SEED_BASE + 5 + (seed_offset << 8)
    idx = np.arange(first, first + count, dtype=np.uint64)
    c = _draw_shapes(seed, idx, layers=(64, 128), hidden_lo=8192, hidden_hi=16384,
                     hidden_step=1024, vocab=(32000, 256000),
                     seqs=(4096, 8192, 16384, 32768), chunks=(1 << 23,))
    c["batch"] = _uniform(seed, idx, _F_BATCH, 1, 8)
    _draw_method(seed, idx, c, 16)
    return c


# --------------------------------------------------------------------------
# sharding of independent configs over ranks (no exchange step exists)
# --------------------------------------------------------------------------
def shard_bounds(weights: np.ndarray, world_size: int) -> np.ndarray:
    """Split range(len(weights)) into world_size contiguous pieces of near-equal total
    weight.  Returns world_size+1 boundaries.  Weights are per-config costs (for
    materialised lists: event counts)."""
    n = len(weights)
    if world_size <= 0:
        raise ValueError("world_size must be positive")
    csum = np.concatenate([[0], np.cumsum(np.asarray(weights, dtype=np.float64))])
    total = csum[-1]
    targets = total * np.arange(1, world_size) / world_size
    cuts = np.searchsorted(csum, targets, side="left")
    bounds = np.concatenate([[0], np.clip(cuts, 0, n), [n]]).astype(np.int64)
    return np.maximum.accumulate(bounds)


def slab_bounds(offsets: np.ndarray, max_events: int, first: int = 0) -> np.ndarray:
    """Cut configurations [first, n) into contiguous slabs whose event lists hold at most
    ``max_events`` events each, greedily; a configuration with more events than that forms a
    slab of its own.  ``offsets`` is the exclusive prefix sum of the event counts ([n+1]).
    Returns the slab boundaries, starting with ``first`` and ending with n (just [first] if
    first == n)."""
    offsets = np.asarray(offsets, dtype=np.int64)
    n = len(offsets) - 1
    if max_events < 1:
        raise ValueError("max_events must be positive")
    if not 0 <= first <= n:
        raise ValueError("first must lie in 0 .. n")
    bounds = [first]
    a = first
    while a < n:
        # largest b with offsets[b] - offsets[a] <= max_events, at least a + 1
        b = int(np.searchsorted(offsets, offsets[a] + max_events, side="right")) - 1
        b = min(max(b, a + 1), n)
        bounds.append(b)
        a = b
    return np.asarray(bounds, dtype=np.int64)
