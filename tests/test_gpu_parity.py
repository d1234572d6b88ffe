"""Parity of the CUDA library with the CPU oracle, element by element, on the same
seeded inputs.  All quantities are integers: the bar is bit-exact equality.
Sizes here are ones the level-1 oracle finishes in seconds; they still span many
chunks of the expansion and scan kernels (576 and 832 events) with ragged tails."""
import numpy as np
import pytest

import oracle
from paper_2404_10933_b200 import grids

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

G = 2 * 1024 * 1024


@pytest.fixture(scope="module")
def llmem():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2404_10933_b200 as m
    m.lib()
    return m


def oracle_lists(cfgs, rounded):
    """Concatenated oracle event lists and offsets (status != 0 contributes nothing)."""
    parts, counts = [], []
    for i in range(len(cfgs)):
        st, n = oracle.event_count(cfgs[i:i + 1])
        if st == 0:
            ev = oracle.expand_events(cfgs[i:i + 1])
            parts.append(oracle.round_events(ev) if rounded else ev)
            counts.append(n)
        else:
            counts.append(0)
    offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    delta = np.concatenate(parts) if parts else np.zeros(0, dtype=np.int64)
    return delta, offsets


def mixed_small_grid():
    """All methods and degrees on small shapes, plus inadmissible records."""
    c = grids.g2_shape_grid(40, 3)           # 3 shapes x 32 batches x 29 combos
    c = c[::7].copy()                        # 398 configs, every method / degree appears
    c["chunk_elems"] = np.where(np.arange(len(c)) % 3 == 0, 1 << 22, c["chunk_elems"])
    c["iters"] = 1 + (np.arange(len(c)) % 3)
    c["act_mode"] = (np.arange(len(c)) // 2) % 2          # half of them keep every operator output
    bad = grids.g2_shape_grid(41, 1)[:12].copy()
    bad["layers"][0] = 0
    bad["heads"][1] = 7
    bad["method"][2] = 9
    bad["method"][3], bad["gpu_n"][3], bad["tp_n"][3] = 3, 4, 3      # inadmissible DP+TP
    bad["method"][4], bad["gpu_n"][4], bad["tp_n"][4] = 3, 2, 2
    bad["batch"][5], bad["seq"][5], bad["vocab"][5] = 1 << 26, 1 << 26, 1 << 26   # >= 2^62 bytes
    bad["layers"][6], bad["hidden"][6], bad["heads"][6], bad["ffn"][6] = 48, 8192, 64, 32768
    bad["chunk_elems"][6] = 1                                         # >= 2^31 events
    bad["reserved"][7, 7] = 1
    bad["lm_bytes"][8] = 3
    bad["act_mode"][8] = 2
    bad["seq"][9] = 1                                                 # valid: zero-byte shifted logits
    bad["method"][10], bad["gpu_n"][10] = 2, 1                        # valid: zero-byte TP buffers
    bad["method"][11], bad["gpu_n"][11] = 1, 1                        # valid: zero-byte gathers
    out = np.concatenate([c[:150], bad, c[150:]])
    return out


def check_estimate(llmem, cfgs, threads=8):
    want = oracle.estimate(cfgs, threads=threads)
    got = llmem.estimate_batch(cfgs)
    torch.cuda.synchronize()
    assert np.array_equal(got["status"].cpu().numpy(), want["status"])
    assert np.array_equal(got["peak"].cpu().numpy(), want["peak"])
    assert np.array_equal(got["index"].cpu().numpy(), want["index"])
    return want


def check_materialized(llmem, cfgs, want):
    dev = llmem.to_device(cfgs)
    offsets, status = llmem.event_counts(dev)
    raw_want, off_want = oracle_lists(cfgs, rounded=False)
    assert np.array_equal(offsets.cpu().numpy(), off_want)
    assert np.array_equal(status.cpu().numpy(), want["status"])
    total = int(off_want[-1])
    raw = llmem.expand_events(dev, offsets, total)
    assert np.array_equal(raw.cpu().numpy(), raw_want)
    rounded_want = oracle.round_events(raw_want)
    fused = llmem.expand_events(dev, offsets, total, fuse_round=True)
    assert np.array_equal(fused.cpu().numpy(), rounded_want)
    # scan of raw deltas with rounding fused into the read
    r1 = llmem.scan_peak(raw, offsets, dev, fuse_round=True, check_status=True)
    # separate rounding kernel, then plain scan
    rounded = llmem.round_events(raw.clone())
    assert np.array_equal(rounded.cpu().numpy(), rounded_want)
    r2 = llmem.scan_peak(rounded, offsets, dev, check_status=True)
    r3 = llmem.scan_peak(fused, offsets, dev, check_status=True)
    # one-pass expansion + scan, list written rounded and raw
    r4 = llmem.expand_scan(dev, offsets, total, fuse_round=True)
    assert np.array_equal(r4["delta"].cpu().numpy(), rounded_want)
    r5 = llmem.expand_scan(dev, offsets, total, fuse_round=False)
    assert np.array_equal(r5["delta"].cpu().numpy(), raw_want)
    for r in (r1, r2, r3, r4, r5):
        assert np.array_equal(r["peak"].cpu().numpy(), want["peak"])
        assert np.array_equal(r["index"].cpu().numpy(), want["index"])
    return total


def test_g1_small_grid_all_entry_points(llmem):
    cfgs = grids.g1_small()
    want = check_estimate(llmem, cfgs)
    assert (want["count"] == 308).all()
    total = check_materialized(llmem, cfgs, want)
    assert total == 64 * 308
    pipe = llmem.estimate_materialized(cfgs)
    assert np.array_equal(pipe["peak"].cpu().numpy(), want["peak"])


def test_mixed_methods_and_inadmissible_records(llmem):
    cfgs = mixed_small_grid()
    want = check_estimate(llmem, cfgs)
    assert set(np.unique(want["status"])) == {0, 1, 2, 3}
    total = check_materialized(llmem, cfgs, want)
    assert total > 50 * 4608          # spans many tiles


def test_tiny_segments_many_per_tile(llmem):
    # 21 .. ~100 events per configuration: dozens of segments inside every tile
    c = grids.g2_shape_grid(7, 1)
    c["layers"] = 1 + (np.arange(len(c)) % 3)
    c["hidden"], c["heads"], c["ffn"] = 256, 4, 1024
    c["chunk_elems"] = 1 << 22
    want = check_estimate(llmem, c)
    assert want["count"][want["status"] == 0].max() < 200
    total = check_materialized(llmem, c, want)
    assert total > 3 * 4608


def test_empty_and_degenerate_calls(llmem):
    z = grids.empty(0)
    r = llmem.estimate_batch(z)
    assert r["peak"].numel() == 0
    offsets, _ = llmem.event_counts(z)
    assert offsets.cpu().tolist() == [0]
    # every record inadmissible: no events at all, scan must still define the outputs
    c = grids.g1_small()[:5].copy()
    c["layers"] = 0
    want = oracle.estimate(c)
    pipe = llmem.estimate_materialized(c)
    assert pipe["total_events"] == 0
    assert np.array_equal(pipe["peak"].cpu().numpy(), want["peak"])
    assert np.array_equal(pipe["index"].cpu().numpy(), want["index"])
    assert (want["peak"] == -1).all()
    # a single configuration
    one = grids.g1_small()[3:4]
    check_materialized(llmem, one, check_estimate(llmem, one))


def test_scan_of_arbitrary_lists_and_alignments(llmem):
    """llmem_scan_peak on lists it did not produce: random signed values, segment
    lengths from 0 to several tiles (including exact tile multiples), and a delta
    pointer that is only 8-byte aligned."""
    rng = np.random.default_rng(2404)
    lens = [0, 1, 2, 4607, 4608, 4609, 0, 0, 9216, 13824, 5, 70000, 3, 0, 4608 * 3 - 1, 1, 18, 17, 19,
            250000, 0]
    # around the limits of the scan by owners: a lane's segment (768), a warp's part (4096), its chunks (832)
    lens += [383, 384, 385, 767, 768, 769, 831, 832, 833, 4095, 4096, 4097, 8191, 8192, 8193, 2 * 4096 + 833]
    lens += rng.integers(0, 300, size=400).tolist()
    lens += [0]
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(offsets[-1])
    delta = rng.integers(-(1 << 40), 1 << 40, size=total, dtype=np.int64)
    delta[rng.integers(0, total, size=total // 10)] = 0
    want_peak = np.zeros(len(lens), dtype=np.int64)
    want_idx = np.zeros(len(lens), dtype=np.int64)
    want_peak_r = np.zeros(len(lens), dtype=np.int64)
    want_idx_r = np.zeros(len(lens), dtype=np.int64)
    for i in range(len(lens)):
        seg = delta[offsets[i]:offsets[i + 1]]
        want_peak[i], want_idx[i] = oracle.scan_peak(seg)
        want_peak_r[i], want_idx_r[i] = oracle.scan_peak(oracle.round_events(seg))
    off_dev = torch.from_numpy(offsets).cuda()
    for shift in (0, 1):
        buf = torch.zeros(total + 3, dtype=torch.int64, device="cuda")
        view = buf[shift:shift + total]
        assert view.data_ptr() % 16 == 8 * shift
        view.copy_(torch.from_numpy(delta))
        r = llmem.scan_peak(view, off_dev, None, check_status=True)
        assert np.array_equal(r["peak"].cpu().numpy(), want_peak)
        assert np.array_equal(r["index"].cpu().numpy(), want_idx)
        r = llmem.scan_peak(view, off_dev, None, fuse_round=True, check_status=True)
        assert np.array_equal(r["peak"].cpu().numpy(), want_peak_r)
        assert np.array_equal(r["index"].cpu().numpy(), want_idx_r)
        # in-place rounding on the same (mis)aligned view
        llmem.round_events(view)
        assert np.array_equal(view.cpu().numpy(), oracle.round_events(delta))
        assert int(buf[shift + total:].abs().sum()) == 0 and (shift == 0 or int(buf[0]) == 0)


def test_expand_into_unaligned_output(llmem):
    cfgs = mixed_small_grid()[:60]
    dev = llmem.to_device(cfgs)
    offsets, _ = llmem.event_counts(dev)
    want, off_want = oracle_lists(cfgs, rounded=True)
    total = int(off_want[-1])
    buf = torch.full((total + 4,), -7, dtype=torch.int64, device="cuda")
    out = llmem.expand_events(dev, offsets, total, fuse_round=True, out=buf[1:1 + total])
    assert out.data_ptr() % 16 == 8
    assert np.array_equal(out.cpu().numpy(), want)
    assert buf[0].item() == -7 and (buf[1 + total:] == -7).all()
    # the one-pass variant into the same unaligned view
    buf.fill_(-7)
    r = llmem.expand_scan(dev, offsets, total, fuse_round=True, out=buf[1:1 + total])
    est = oracle.estimate(cfgs, threads=4)
    assert np.array_equal(r["delta"].cpu().numpy(), want)
    assert np.array_equal(r["peak"].cpu().numpy(), est["peak"])
    assert np.array_equal(r["index"].cpu().numpy(), est["index"])
    assert buf[0].item() == -7 and (buf[1 + total:] == -7).all()


def test_long_runs_all_store_paths(llmem):
    """Lists made of long runs of equal or alternating events (deep/wide decoders): most chunks
    are issued from a buffer that is not refilled and folded in closed form.  Both kernels,
    rounded and raw lists, aligned and unaligned outputs, with and without the work counter."""
    cfgs = grids.g5_stress(3, 40)
    cfgs["iters"][::3] = 1                     # lists that end with the optimizer states
    cfgs["iters"][1::7] = 3
    cfgs["act_mode"][::4] = 1                  # periodic operator-output runs between the long ones
    dev = llmem.to_device(cfgs)
    offsets, _ = llmem.event_counts(dev)
    est = oracle.estimate(cfgs, threads=8)
    assert (est["status"] == 0).all()
    total = int(offsets[-1].item())
    assert total > 1000 * 576
    no_scratch = torch.empty(0, dtype=torch.uint8, device="cuda")
    for rounded in (True, False):
        want, off_want = oracle_lists(cfgs, rounded=rounded)
        assert np.array_equal(offsets.cpu().numpy(), off_want)
        for shift in (0, 1):
            buf = torch.full((total + 4,), -7, dtype=torch.int64, device="cuda")
            view = buf[shift:shift + total]
            for scratch in (None, no_scratch):
                buf.fill_(-7)
                out = llmem.expand_events(dev, offsets, total, fuse_round=rounded, out=view, scratch=scratch)
                assert np.array_equal(out.cpu().numpy(), want), (rounded, shift, scratch is None)
                assert (buf[:shift] == -7).all() and (buf[shift + total:] == -7).all()
            buf.fill_(-7)
            r = llmem.expand_scan(dev, offsets, total, fuse_round=rounded, out=view)
            assert np.array_equal(r["delta"].cpu().numpy(), want), (rounded, shift)
            assert np.array_equal(r["peak"].cpu().numpy(), est["peak"]), (rounded, shift)
            assert np.array_equal(r["index"].cpu().numpy(), est["index"]), (rounded, shift)
            assert (buf[:shift] == -7).all() and (buf[shift + total:] == -7).all()


def test_max_batch_and_select_small(llmem):
    shapes = grids.g4_search_grid(0, 8)              # 8 shapes x 4 methods x 16 degrees
    shapes["chunk_elems"] = 1 << 25                  # keeps the literal (level-1) oracle quick
    caps = grids.g4_capacities()
    bmax = 40
    want_bs, want_st = oracle.max_batch(shapes, caps, bmax, level=1, threads=8)
    got_bs, got_st = llmem.max_batch(shapes, caps, bmax)
    assert np.array_equal(got_st.cpu().numpy(), want_st)
    assert np.array_equal(got_bs.cpu().numpy(), want_bs)
    assert (want_bs == 0).any() and (want_bs == bmax).any() and ((want_bs > 0) & (want_bs < bmax)).any()
    sel_shapes = grids.g4_select_grid(0, 8)
    sel_shapes["chunk_elems"] = 1 << 25
    for allzero in (False, True):
        want = oracle.select_method(sel_shapes, caps, bmax, flags=1 if allzero else 0, level=1, threads=8)
        got = llmem.select_method(sel_shapes, caps, bmax, allzero=allzero)
        for k in ("method", "batch", "bs_list", "status"):
            assert np.array_equal(got[k].cpu().numpy(), want[k]), k
    # inadmissible shapes and the full batch range against the bisecting oracle
    bad = shapes[:6].copy()
    bad["hidden"][0] = 0
    bad["method"][1] = 7
    bad["layers"][2], bad["hidden"][2], bad["heads"][2], bad["ffn"][2] = 48, 8192, 64, 32768
    bad["chunk_elems"][2] = 1            # >= 2^31 events
    bad["batch"][3] = -5                 # ignored by the search
    want_bs, want_st = oracle.max_batch(bad, caps, 4096, level=2)
    got_bs, got_st = llmem.max_batch(bad, caps, 4096)
    assert np.array_equal(got_st.cpu().numpy(), want_st) and want_st.tolist()[:3] == [1, 1, 3]
    assert np.array_equal(got_bs.cpu().numpy(), want_bs)
    want = oracle.select_method(bad, caps, 4096, level=2)
    got = llmem.select_method(bad, caps, 4096)
    for k in ("method", "batch", "bs_list", "status"):
        assert np.array_equal(got[k].cpu().numpy(), want[k]), k


def test_aligned_family_on_device(llmem):
    # the page-aligned family of the oracle pins, straight through the CUDA path
    c = grids.empty(4)
    for k, v in dict(layers=4, hidden=2048, heads=16, ffn=8192, vocab=65536, pos_len=0, seq=1024, batch=32,
                     chunk_elems=1 << 24, base_bytes=123456789, lm_bytes=2, iters=2).items():
        c[k] = v
    c["method"] = [0, 1, 2, 3]
    c["gpu_n"] = [1, 4, 4, 4]
    c["tp_n"] = [0, 0, 0, 2]
    want = oracle.estimate(c)
    got = llmem.estimate_batch(c)
    assert np.array_equal(got["peak"].cpu().numpy(), want["peak"])
    assert ((want["peak"] - 123456789 - 65536 * 2048 * 2) % G == 0).all()


def test_search_edge_capacities_and_ranges(llmem):
    """Capacities below the fixed part, equal to a peak, one byte less, negative, at and
    beyond 2^62; one-iteration lists; TP on a single device; the largest admissible bmax."""
    base = grids.g4_search_grid(3, 2)                       # 2 shapes x 4 methods x 16 degrees
    one_iter = base.copy(); one_iter["iters"] = 1
    tiny = base[:32].copy()
    tiny["layers"], tiny["hidden"], tiny["heads"], tiny["ffn"], tiny["vocab"] = 1, 64, 1, 256, 1000
    tiny["seq"], tiny["chunk_elems"], tiny["base_bytes"] = 1, 1 << 20, 0   # zero-byte shifted copies
    shapes = np.concatenate([base, one_iter, tiny])
    probe = shapes.copy(); probe["batch"] = 3
    est = oracle.estimate(probe, level=2)
    exact = est["peak"][est["status"] == 0]
    caps = np.array([-5, 0, 1, int(exact.min()), int(exact.min()) - 1, int(np.median(exact)),
                     int(exact.max()), int(exact.max()) - 1, (1 << 62) - 1, 1 << 62, (1 << 63) - 1,
                     16 << 30, 80 << 30], dtype=np.int64)
    for bmax in (1, 7, 1 << 26):
        want_bs, want_st = oracle.max_batch(shapes, caps, bmax, level=2, threads=8)
        got_bs, got_st = llmem.max_batch(shapes, caps, bmax)
        assert np.array_equal(got_st.cpu().numpy(), want_st)
        assert np.array_equal(got_bs.cpu().numpy(), want_bs), bmax
    want_bs, _ = oracle.max_batch(shapes, caps, 9, level=1, threads=8)
    got_bs, _ = llmem.max_batch(shapes, caps, 9)
    assert np.array_equal(got_bs.cpu().numpy(), want_bs)
    # a capacity equal to the peak at batch 3 admits exactly batch 3 (strict exit test)
    ok = np.flatnonzero(est["status"] == 0)[::7]
    for i in ok:
        cap = np.array([int(est["peak"][i])], dtype=np.int64)
        got, _ = llmem.max_batch(shapes[i:i + 1], cap, 64)
        want, _ = oracle.max_batch(shapes[i:i + 1], cap, 64, level=1)
        assert got.cpu().numpy().tolist() == want.tolist()
        assert want[0, 0] >= 3
    sel_shapes = np.concatenate([grids.g4_select_grid(3, 2), grids.g4_select_grid(5, 1)])
    sel_shapes["iters"][::3] = 1
    for allzero in (False, True):
        want = oracle.select_method(sel_shapes, caps, 1 << 26, flags=1 if allzero else 0, level=2, threads=8)
        got = llmem.select_method(sel_shapes, caps, 1 << 26, allzero=allzero)
        for k in ("method", "batch", "bs_list", "status"):
            assert np.array_equal(got[k].cpu().numpy(), want[k]), k


def test_search_bracket_at_its_boundaries(llmem):
    """The search cuts a floating-point bracket to integers and probes only inside it: capacities
    exactly at, one byte below and one page below the peak of a batch, for batches from 1 to
    2^20, on shapes whose bytes per sample range from a few bytes (wide brackets) to gigabytes
    (brackets of one candidate), every method, TP degrees that do not divide the output."""
    rng = np.random.default_rng(606)
    shapes = fuzz_configs(40, 7)
    small = shapes[:12].copy()
    small["seq"], small["hidden"], small["heads"], small["vocab"] = 1, 3, 1, 5      # few bytes per sample
    small["layers"] = rng.integers(1, 40, size=12)
    odd = shapes[12:24].copy()
    odd["method"], odd["gpu_n"], odd["tp_n"] = 2, rng.choice([3, 5, 7, 11, 13], size=12), 0
    odd["seq"] = rng.choice([1, 3, 7, 129], size=12)
    shapes = np.concatenate([shapes, small, odd])
    bmax = 1 << 20
    checked = 0
    for i in range(len(shapes)):
        one = shapes[i:i + 1]
        caps = []
        for b in (1, 2, 3, 17, 255, 4097, 65535, (1 << 20) - 1, 1 << 20):
            at = one.copy(); at["batch"] = b
            est = oracle.estimate(at, level=2)
            if est["status"][0] == 0:
                pk = int(est["peak"][0])
                caps += [pk, pk - 1, pk - (1 << 21), pk + (1 << 21) - 1]
        if not caps:
            continue
        caps = np.array(sorted(set(caps)), dtype=np.int64)
        want_bs, want_st = oracle.max_batch(one, caps, bmax, level=2)
        got_bs, got_st = llmem.max_batch(one, caps, bmax)
        assert np.array_equal(got_st.cpu().numpy(), want_st)
        assert np.array_equal(got_bs.cpu().numpy(), want_bs), (i, caps, got_bs.cpu().numpy(), want_bs)
        checked += caps.size
    assert checked > 1000


def configs_near_the_byte_limit(n_per=256):
    """Records whose peak crosses 2^62 bytes as the batch grows: through the logits, through
    the score-sized operator outputs, through m_base; every method."""
    base = grids.g1_small()[:1].copy()
    k = np.arange(n_per)
    a = np.repeat(base, n_per)
    a["lm_bytes"], a["seq"], a["vocab"], a["hidden"], a["heads"], a["ffn"], a["layers"] = 4, 1 << 26, 1 << 26, 64, 1, 256, 2
    a["batch"], a["method"] = k + 1, k % 4
    a["gpu_n"] = np.where(a["method"] == 3, 4, 1 + k % 7)
    a["tp_n"] = np.where(a["method"] == 3, 2, 0)
    b = np.repeat(base, n_per)
    b["act_mode"], b["seq"], b["hidden"], b["heads"], b["ffn"], b["vocab"] = 1, 1 << 20, 1 << 10, 1 << 10, 1 << 12, 1000
    b["layers"], b["batch"], b["method"] = 1 + k % 64, 1 + k // 4, k % 4
    b["gpu_n"] = np.where(b["method"] == 3, 4, 1 + k % 5)
    b["tp_n"] = np.where(b["method"] == 3, 2, 0)
    c = np.repeat(base, n_per)
    c["base_bytes"], c["lm_bytes"], c["seq"], c["vocab"] = 1 << 60, 4, 1 << 25, 1 << 26
    c["batch"], c["iters"] = k + 1, 1 + k % 2
    out = np.concatenate([a, b, c])
    out["chunk_elems"] = 1 << 30
    return out


def test_results_around_the_byte_limit(llmem):
    """Status 3 exactly from 2^62 bytes on, the exact peak below: the fused estimate remembers
    an overflow instead of clamping, the counts clamp, the searches exclude such batches."""
    cfgs = configs_near_the_byte_limit()
    want = oracle.estimate(cfgs, level=2, threads=8)
    for part in range(3):
        st = want["status"][part * 256:(part + 1) * 256]
        assert (st == 0).sum() > 60 and (st == 3).sum() > 60
    assert want["peak"].max() > 0.98 * 2.0 ** 62
    got = llmem.estimate_batch(cfgs)
    assert np.array_equal(got["status"].cpu().numpy(), want["status"])
    assert np.array_equal(got["peak"].cpu().numpy(), want["peak"])
    offsets, status = llmem.event_counts(cfgs)
    assert np.array_equal(status.cpu().numpy(), want["status"])
    caps = np.array([(1 << 62) - 1, 1 << 61, 1 << 60, 3 << 59], dtype=np.int64)
    for bmax in (300, 1 << 26):
        want_bs, want_st = oracle.max_batch(cfgs, caps, bmax, level=2, threads=8)
        got_bs, got_st = llmem.max_batch(cfgs, caps, bmax)
        assert np.array_equal(got_st.cpu().numpy(), want_st)
        assert np.array_equal(got_bs.cpu().numpy(), want_bs), bmax
    want_sel = oracle.select_method(cfgs, caps, 1 << 26, level=2, threads=8)
    got_sel = llmem.select_method(cfgs, caps, 1 << 26)
    for key in ("method", "batch", "bs_list", "status"):
        assert np.array_equal(got_sel[key].cpu().numpy(), want_sel[key]), key


def test_segmented_selection_random_groups(llmem):
    rng = np.random.default_rng(10933)
    sizes = rng.integers(0, 40, size=300)
    sizes[[0, 17, 299]] = 0                              # empty groups, first and last included
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    n_items, n_cap = int(offsets[-1]), 7
    items = grids.empty(n_items)
    items["method"] = rng.integers(0, 6, size=n_items)   # 4 and 5 are not methods: score 0
    items["gpu_n"] = rng.integers(1, 64, size=n_items)
    items["tp_n"] = rng.integers(0, 9, size=n_items)     # 0 with DP+TP: score 0
    bs = rng.integers(-1, 6, size=(n_items, n_cap)).astype(np.int32)   # many ties
    bs[rng.random((n_items, n_cap)) < 0.05] = 1 << 26
    want = oracle.select_segmented(items, bs, offsets)
    got = llmem.select_segmented(items, torch.from_numpy(bs).cuda(), offsets)
    for k in ("item", "method", "batch"):
        assert np.array_equal(got[k].cpu().numpy(), want[k]), k
    assert (want["item"] == -1).any() and (want["method"] == 3).any()


def test_chunk_search(llmem):
    cfgs = np.concatenate([grids.g2_shapes(0, 300), grids.g3_sweep(0, 200), grids.g5_stress(0, 100)])
    cfgs["layers"][5] = 0
    cfgs["chunk_elems"][6] = -3            # ignored
    for cs_min, step, count in ((1 << 20, 1 << 16, 257), (1 << 22, 1 << 22, 8), (12345, 1, 33), (1 << 40, 1, 1)):
        want = oracle.chunk_search(cfgs, cs_min, step, count)
        got = llmem.chunk_search(cfgs, cs_min, step, count)
        for k in ("chunk", "waste", "status"):
            assert np.array_equal(got[k].cpu().numpy(), want[k]), (k, cs_min)
    L = llmem.lib()
    assert L.llmem_chunk_search(None, 0, 0, 1, 1, None, None, None, None, 0, 0, None) == llmem.ERR_ARG
    assert L.llmem_chunk_search(None, 0, 1 << 40, 1, 2, None, None, None, None, 0, 0, None) == llmem.ERR_ARG


def fuzz_configs(n, seed):
    """Random admissible and inadmissible records over wide field ranges, small enough for
    the level-1 oracle: every method, degrees up to 255, up to 40 iterations, both FFN kinds,
    with and without biases and position embeddings, sequence length 1 included."""
    rng = np.random.default_rng(seed)
    c = grids.empty(n)
    heads = rng.choice([1, 2, 4, 8], size=n)
    c["heads"] = heads
    c["hidden"] = heads * rng.integers(8, 129, size=n)
    c["layers"] = rng.integers(1, 13, size=n)
    c["ffn"] = rng.integers(16, 4097, size=n)
    c["vocab"] = rng.integers(1, 70000, size=n)
    c["pos_len"] = rng.choice([0, 0, 1, 77, 4096], size=n)
    c["seq"] = rng.choice([1, 2, 17, 512, 4096, 100000], size=n)
    c["batch"] = rng.integers(1, 300, size=n)
    c["chunk_elems"] = rng.choice([1 << 16, 1 << 18, 100003, 1 << 22, 1 << 30], size=n)
    c["base_bytes"] = rng.integers(0, 1 << 34, size=n)
    c["method"] = rng.integers(0, 4, size=n)
    gpu_n = rng.choice([1, 2, 3, 4, 6, 8, 12, 16, 60, 64, 240, 255], size=n)
    c["gpu_n"] = gpu_n
    tp = np.zeros(n, dtype=np.int64)
    for i in range(n):
        degs = grids.valid_tp_degrees(int(gpu_n[i]))
        tp[i] = rng.choice(degs) if degs and rng.random() < 0.9 else rng.integers(0, 9)
    c["tp_n"] = tp
    c["lm_bytes"] = rng.choice([2, 4], size=n)
    c["ffn_kind"] = rng.integers(0, 2, size=n)
    c["has_bias"] = rng.integers(0, 2, size=n)
    c["iters"] = rng.choice([1, 2, 3, 7, 40], size=n)
    c["act_mode"] = rng.integers(0, 2, size=n)
    return c


def test_fuzz_all_entry_points(llmem):
    cfgs = fuzz_configs(2500, 42)
    want = check_estimate(llmem, cfgs)
    assert (want["status"] == 2).any() and (want["status"] == 0).sum() > 1500
    assert want["count"].max() < 200000
    total = check_materialized(llmem, cfgs, want)
    assert total > 10 * 4608
    caps = np.array([1 << 28, 1 << 31, 3 << 32, 1 << 36, 1 << 40], dtype=np.int64)
    sub = cfgs[::5]
    want_bs, want_st = oracle.max_batch(sub, caps, 12, level=1, threads=8)
    got_bs, got_st = llmem.max_batch(sub, caps, 12)
    assert np.array_equal(got_st.cpu().numpy(), want_st) and np.array_equal(got_bs.cpu().numpy(), want_bs)
    want_bs, want_st = oracle.max_batch(cfgs, caps, 1 << 20, level=2, threads=8)
    got_bs, got_st = llmem.max_batch(cfgs, caps, 1 << 20)
    assert np.array_equal(got_st.cpu().numpy(), want_st) and np.array_equal(got_bs.cpu().numpy(), want_bs)
    for allzero in (False, True):
        want_sel = oracle.select_method(cfgs, caps, 1 << 20, flags=1 if allzero else 0, level=2, threads=8)
        got_sel = llmem.select_method(cfgs, caps, 1 << 20, allzero=allzero)
        for k in ("method", "batch", "bs_list", "status"):
            assert np.array_equal(got_sel[k].cpu().numpy(), want_sel[k]), k


def heads_and_hidden_pairs(n, seed):
    """hidden in 1 .. 2^20 against divisors, near-divisors, itself, heads above hidden and heads
    up to 2^31 - 1; records with tiny event lists."""
    rng = np.random.default_rng(seed)
    c = np.repeat(grids.g1_small()[:1], n)
    lo = np.arange(n) % 2 == 0
    h = np.where(lo, rng.integers(1, 1 << 10, size=n), rng.integers(1, 1 << 5, size=n))
    k = np.where(lo, rng.integers(1, 1 << 10, size=n), rng.integers(1, 1 << 15, size=n))
    hidden = h * k                                              # <= 2^20
    kind = (np.arange(n) // 2) % 8
    heads = np.select(
        [kind == 0, kind == 1, kind == 2, kind == 3, kind == 4, kind == 5, kind == 6],
        [h, k, h + 1, np.maximum(1, k - 1), hidden, hidden + rng.integers(1, 1 << 20, size=n),
         rng.integers(1 << 21, 1 << 31, size=n)],
        default=rng.integers(1, (1 << 20) + 1, size=n))
    hidden[:4] = [1, 1 << 20, (1 << 20) - 1, 720720]
    heads[:4] = [1, 1 << 20, (1 << 20) - 1, (1 << 31) - 1]
    c["hidden"], c["heads"] = hidden, heads
    c["layers"], c["ffn"], c["vocab"], c["seq"], c["batch"] = 1, 64, 64, 8, 1
    c["chunk_elems"] = 1 << 40
    return c


def test_heads_must_divide_hidden_every_pair_class(llmem):
    """The field check decides hidden % heads == 0 without an integer division."""
    c = heads_and_hidden_pairs(1 << 18, 77)
    want = oracle.estimate(c, threads=16)
    ok = (c["hidden"] % c["heads"]) == 0
    assert np.array_equal(want["status"] == 0, ok) and 0.3 < ok.mean() < 0.7
    got = llmem.estimate_batch(c)
    assert np.array_equal(got["status"].cpu().numpy(), want["status"])
    assert np.array_equal(got["peak"].cpu().numpy(), want["peak"])
    caps = np.array([1 << 34], dtype=np.int64)
    got_bs, got_st = llmem.max_batch(c[:4096], caps, 64)
    want_bs, want_st = oracle.max_batch(c[:4096], caps, 64, level=2, threads=8)
    assert np.array_equal(got_st.cpu().numpy(), want_st) and np.array_equal(got_bs.cpu().numpy(), want_bs)


def test_bounded_wait_gives_up_and_reports(llmem):
    """Failure handling without a fault: a wait on a barrier that nothing completes runs out
    after its limit, the status word says so, and the context keeps working."""
    import time
    L = llmem.lib()
    scratch = torch.zeros(256, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert L.llmem_scratch_status(scratch.data_ptr(), stream) == llmem.OK
    t0 = time.perf_counter()
    assert L.llmem_selftest_wait_limit(scratch.data_ptr(), 256, 50, stream) == llmem.OK
    assert L.llmem_scratch_status(scratch.data_ptr(), stream) == llmem.ERR_TIMEOUT
    dt = time.perf_counter() - t0
    assert 0.045 < dt < 1.0, dt
    assert b"wait" in L.llmem_last_error()
    # argument checks
    assert L.llmem_selftest_wait_limit(scratch.data_ptr(), 256, 0, stream) == llmem.ERR_ARG
    assert L.llmem_selftest_wait_limit(None, 256, 50, stream) == llmem.ERR_SCRATCH
    # the context is intact: a scan on the same stream right afterwards is correct
    cfgs = grids.g1_small()[:8]
    want = oracle.estimate(cfgs)
    pipe = llmem.estimate_materialized(cfgs)
    assert np.array_equal(pipe["peak"].cpu().numpy(), want["peak"])


def test_materialised_path_in_slabs(llmem):
    """Slab by slab through one reused list buffer: same peaks as the oracle, every slab's
    list bit for bit, restart from a slab boundary."""
    cfgs = np.concatenate([mixed_small_grid(), grids.g5_stress(11, 3)])
    want = oracle.estimate(cfgs, threads=8)
    lists, off = oracle_lists(cfgs, rounded=True)
    budget = 150_000                                   # the stress-grid lists are larger: slabs of their own
    assert np.diff(off).max() > budget
    seen = []

    def on_slab(lo, hi, delta, local):
        assert np.array_equal(delta.cpu().numpy(), lists[off[lo]:off[hi]])
        assert np.array_equal(local.cpu().numpy(), off[lo:hi + 1] - off[lo])
        seen.append((lo, hi))

    r = llmem.estimate_in_slabs(cfgs, budget, on_slab=on_slab)
    torch.cuda.synchronize()
    b = r["bounds"]
    assert len(b) > 10 and seen == list(zip(b[:-1].tolist(), b[1:].tolist()))
    assert np.array_equal(b, grids.slab_bounds(off, budget))
    assert np.array_equal(r["status"].cpu().numpy(), want["status"])
    assert np.array_equal(r["peak"].cpu().numpy(), want["peak"])
    assert np.array_equal(r["index"].cpu().numpy(), want["index"])
    # restart at the fifth slab: earlier results stay at -1
    again = llmem.estimate_in_slabs(cfgs, budget, first_config=int(b[4]))
    k = int(b[4])
    assert (again["peak"][:k] == -1).all()
    assert np.array_equal(again["peak"].cpu().numpy()[k:], want["peak"][k:])
    assert np.array_equal(again["index"].cpu().numpy()[k:], want["index"][k:])


def test_slab_bounds_on_device_equal_the_host_cut(llmem):
    """llmem_slab_bounds against the greedy cut written out on the host, for budgets from one
    event (every configuration a slab of its own) to more than the whole grid, restarts, empty
    segments, and the refusal when the slabs do not fit the output."""
    cfgs = mixed_small_grid()
    offsets, _ = llmem.event_counts(cfgs)
    off = offsets.cpu().numpy()
    n = len(cfgs)
    for budget in (1, 300, 5000, 40_000, int(off[-1]), int(off[-1]) * 3):
        for first in (0, 7, n - 1, n):
            b, ev = llmem.slab_bounds(offsets, budget, first)
            assert np.array_equal(b, grids.slab_bounds(off, budget, first))
            assert np.array_equal(ev, off[b])
    with pytest.raises(ValueError, match="slabs"):
        llmem.slab_bounds(offsets, 1, 0, max_slabs=16)
    L = llmem.lib()
    assert L.llmem_slab_bounds(offsets.data_ptr(), n, 0, 0, offsets.data_ptr(), offsets.data_ptr(), 4,
                               offsets.data_ptr(), None) == llmem.ERR_ARG


def test_second_estimator_all_paths(llmem):
    """The DNNMem-style estimator of Section 3.1: fused estimate, event counts, the list raw
    and aligned to 512 bytes (both expansion kernels), its scan and the one-pass path against
    the oracle, on G1, a mixed grid with inadmissible records, long lists and every operator
    output kept; the searches refuse the flag."""
    mixed = mixed_small_grid()
    mixed["method"][::2] = 0                       # the estimator takes the conventional method only
    long_lists = grids.g5_stress(3, 12).copy()
    long_lists["method"], long_lists["act_mode"] = 0, np.arange(12) % 2
    long_lists["layers"] = 40000                   # lists long enough for the chunk kernels
    for cfgs in (grids.g1_small(), mixed, long_lists):
        want = oracle.dnn_estimate(cfgs, threads=8)
        got = llmem.estimate_batch(cfgs, estimator="dnnmem")
        for k in ("status", "peak", "index"):
            assert np.array_equal(got[k].cpu().numpy(), want[k]), k
        assert (want["status"] == 0).any()
        dev = llmem.to_device(cfgs)
        offsets, status = llmem.event_counts(dev, estimator="dnnmem")
        off = offsets.cpu().numpy()
        assert np.array_equal(status.cpu().numpy(), want["status"])
        assert np.array_equal(np.diff(off), np.where(want["status"] == 0, want["count"], 0))
        total = int(off[-1])
        raw_want = np.concatenate([oracle.dnn_expand_events(cfgs[i:i + 1]) for i in range(len(cfgs))
                                   if want["status"][i] == 0])
        aligned_want = oracle.dnn_round_events(raw_want)
        raw = llmem.expand_events(dev, offsets, total, estimator="dnnmem")
        assert np.array_equal(raw.cpu().numpy(), raw_want)
        header = torch.zeros(256, dtype=torch.uint8, device="cuda")
        for scratch in (None, header):             # segment owners / chunks of the list
            aligned = llmem.expand_events(dev, offsets, total, fuse_round=True, estimator="dnnmem", scratch=scratch)
            assert np.array_equal(aligned.cpu().numpy(), aligned_want)
        two = llmem.scan_peak(aligned, offsets, dev, estimator="dnnmem", check_status=True)
        one = llmem.expand_scan(dev, offsets, total, fuse_round=True, estimator="dnnmem")
        assert np.array_equal(one["delta"].cpu().numpy(), aligned_want)
        pipe = llmem.estimate_materialized(dev, estimator="dnnmem")
        for r in (two, one, pipe):
            assert np.array_equal(r["peak"].cpu().numpy(), want["peak"])
            assert np.array_equal(r["index"].cpu().numpy(), want["index"])
        with pytest.raises(llmem.LlmemError):
            llmem.expand_scan(dev, offsets, total, fuse_round=False, estimator="dnnmem")
        with pytest.raises(llmem.LlmemError):
            llmem.scan_peak(raw, offsets, dev, fuse_round=True, estimator="dnnmem")
    L = llmem.lib()
    caps = llmem._caps(grids.g4_capacities(), dev.device)
    out = torch.zeros((len(cfgs), caps.numel()), dtype=torch.int32, device="cuda")
    assert L.llmem_max_batch(dev.data_ptr(), len(cfgs), caps.data_ptr(), caps.numel(), 8, out.data_ptr(), None, None, 0,
                             llmem.ESTIMATOR_DNNMEM, None) == llmem.ERR_ARG
    assert L.llmem_select_method(dev.data_ptr(), len(cfgs), caps.data_ptr(), caps.numel(), 8, out.data_ptr(),
                                 out.data_ptr(), None, None, None, 0, llmem.ESTIMATOR_DNNMEM, None) == llmem.ERR_ARG


CHECKED_SCRIPT = r"""
import numpy as np, torch
import oracle
import paper_2404_10933_b200 as llmem
from paper_2404_10933_b200 import grids
L = llmem.lib()
assert L.llmem_checked_build() == 1
import tests.test_gpu_parity as t
tiny = grids.g2_shape_grid(7, 1)
tiny["layers"] = 1 + (np.arange(len(tiny)) % 3)
tiny["hidden"], tiny["heads"], tiny["ffn"] = 256, 4, 1024
for cfgs in (t.mixed_small_grid(), grids.g5_stress(5, 48), tiny, grids.g2_shape_grid(3, 6)):
    want = oracle.estimate(cfgs, threads=8)
    dev = llmem.to_device(cfgs)
    offsets, _ = llmem.event_counts(dev)
    total = int(offsets[-1].item())
    for shift in (0, 1):
        buf = torch.zeros(total + 2, dtype=torch.int64, device="cuda")
        view = buf[shift:shift + total]
        header = torch.zeros(256, dtype=torch.uint8, device="cuda")
        llmem.expand_events(dev, offsets, total, fuse_round=True, out=view, scratch=header)
        assert L.llmem_scratch_status(header.data_ptr(), None) == llmem.OK, L.llmem_last_error()
        r = llmem.scan_peak(view, offsets, dev)
        assert L.llmem_scratch_status(r["scratch"].data_ptr(), None) == llmem.OK, L.llmem_last_error()
        one = llmem.expand_scan(dev, offsets, total, fuse_round=True, out=view)
        assert L.llmem_scratch_status(one["scratch"].data_ptr(), None) == llmem.OK, L.llmem_last_error()
        for res in (r, one):
            assert np.array_equal(res["peak"].cpu().numpy(), want["peak"])
            assert np.array_equal(res["index"].cpu().numpy(), want["index"])
print("checked build ok")
"""


def test_checked_build_finds_nothing_and_agrees(llmem):
    """The library compiled with its index checks on (every offset, block and segment index the
    streaming kernels derive is tested before use) runs the same grids: no check fires and the
    results are those of the oracle.  It runs in a process of its own because a process loads
    one build of the library."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, LLMEM_CHECKED="1", PYTHONPATH=root)
    p = subprocess.run([sys.executable, "-c", CHECKED_SCRIPT], cwd=root, env=env, capture_output=True, text=True,
                       timeout=600)
    assert p.returncode == 0 and "checked build ok" in p.stdout, p.stdout + p.stderr


def test_issue_rate_probe(llmem):
    import ctypes
    L = llmem.lib()
    count = ctypes.c_int64(0)
    stream = llmem._stream_ptr(None)
    assert L.llmem_selftest_int_rate(0, 16, None, ctypes.byref(count), stream) == llmem.OK
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert count.value == sms * 8 * 8 * 16 * 64          # CTAs x warps x iterations x counted instructions
    assert L.llmem_selftest_int_rate(3, 16, None, None, stream) == llmem.ERR_ARG
    assert L.llmem_selftest_int_rate(0, 0, None, None, stream) == llmem.ERR_ARG
    rates = [llmem.int_rate(kind, iters=512, reps=1) for kind in range(3)]
    torch.cuda.synchronize()
    assert all(r > 1e11 for r in rates)
    assert rates[1] < rates[0]                            # 32-bit multiplies issue more slowly than adds


def test_all_operator_outputs_mode(llmem):
    """act_mode = 1 (no gradient checkpointing) on realistic shapes: estimate, materialised
    paths, searches and selection against the oracle; the mode must change the result."""
    base = grids.g3_sweep(5000, 300)
    base["chunk_elems"] = 1 << 25
    on = base.copy(); on["act_mode"] = 1
    want_off = oracle.estimate(base, threads=8)
    want_on = check_estimate(llmem, on)
    assert (want_on["peak"] > want_off["peak"]).all()
    check_materialized(llmem, on[:60], {k: v[:60] for k, v in want_on.items()})
    caps = grids.g4_capacities()
    shapes = grids.g4_search_grid(20, 4); shapes["act_mode"] = 1
    want_bs, want_st = oracle.max_batch(shapes, caps, grids.G4_BMAX, level=2, threads=8)
    got_bs, got_st = llmem.max_batch(shapes, caps, grids.G4_BMAX)
    assert np.array_equal(got_st.cpu().numpy(), want_st) and np.array_equal(got_bs.cpu().numpy(), want_bs)
    small = shapes[::9].copy(); small["chunk_elems"] = 1 << 25
    want_bs, _ = oracle.max_batch(small, caps, 10, level=1, threads=8)
    got_bs, _ = llmem.max_batch(small, caps, 10)
    assert np.array_equal(got_bs.cpu().numpy(), want_bs)
    sel = grids.g4_select_grid(20, 4); sel["act_mode"] = 1
    want = oracle.select_method(sel, caps, grids.G4_BMAX, level=2, threads=8)
    got = llmem.select_method(sel, caps, grids.G4_BMAX)
    for k in ("method", "batch", "bs_list", "status"):
        assert np.array_equal(got[k].cpu().numpy(), want[k]), k
    # attention scores that overflow 2^62 bytes: status 3, nothing fits
    huge = on[:2].copy(); huge["seq"] = 1 << 26; huge["heads"] = huge["hidden"]; huge["batch"] = 1 << 10
    check_estimate(llmem, huge)
    want_bs, want_st = oracle.max_batch(huge, caps, 64, level=2)
    got_bs, got_st = llmem.max_batch(huge, caps, 64)
    assert np.array_equal(got_bs.cpu().numpy(), want_bs) and np.array_equal(got_st.cpu().numpy(), want_st)
