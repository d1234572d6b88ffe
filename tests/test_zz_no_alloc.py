"""llmem_event_counts_static: the event-count entry point for callers that cannot
allocate device memory when they call (framework callbacks that may not re-enter the
allocator, services with device memory fixed at start-up).  It must give exactly what
llmem_event_counts gives -- and what the CPU oracle counts -- call after call, although
all calls share one fixed scratch array inside the library that still holds the previous
call's partial sums, and it must leave the device's free memory untouched.

Collected last on purpose (file name): a failure here cannot hide other tests from a run
that stops at the first failure.  It has to pass alone in a fresh process (then its first
call performs the per-device address look-up) and after the rest of the suite."""
import ctypes
import os

import numpy as np
import pytest

import oracle
from paper_2404_10933_b200 import grids

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def llmem():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2404_10933_b200 as m
    m.lib()
    return m


def reference_counts(llmem, dev_cfg):
    """The existing entry point, with caller-provided scratch."""
    offsets, status = llmem.event_counts(dev_cfg)
    torch.cuda.synchronize()
    return offsets.cpu().numpy(), status.cpu().numpy()


def static_counts(llmem, dev_cfg, offsets_buf, status_buf):
    """The new entry point, straight through the C ABI with raw pointers; the output
    buffers were allocated by the caller beforehand, nothing is allocated here."""
    n = dev_cfg.shape[0]
    rc = llmem.lib().llmem_event_counts_static(
        ctypes.c_void_p(dev_cfg.data_ptr()), ctypes.c_int64(n), ctypes.c_void_p(offsets_buf.data_ptr()),
        ctypes.c_void_p(status_buf.data_ptr()), ctypes.c_uint32(0),
        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == llmem.OK, llmem.lib().llmem_last_error()
    torch.cuda.synchronize()


def oracle_counts(cfgs):
    """Status and event count of every record from the CPU oracle (it walks the explicit
    list), as the exclusive prefix sum the entry points return."""
    want = oracle.estimate(cfgs, level=1, threads=os.cpu_count() or 8)
    counts = np.where(want["status"] == 0, want["count"], 0)
    return np.concatenate([[0], np.cumsum(counts)]).astype(np.int64), want["status"]


def test_static_event_counts_match_on_consecutive_calls(llmem):
    # first call: a large batch (293 partial sums, a ragged last block)
    big = grids.g3_sweep(0, 300_000)
    big["layers"][::1000] = 0                       # some inadmissible records
    # second call: a smaller batch with a ragged last block; the array still holds the
    # first call's sums beyond what this call uses
    small = np.concatenate([grids.g1_small(), grids.g2_shape_grid(5, 1)[::3]])[:-5]
    # third call: big again, after the small one
    batches = (big, small, big)
    dev = [llmem.to_device(c) for c in batches]
    want = [reference_counts(llmem, d) for d in dev]
    from_oracle = [oracle_counts(c) for c in (big, small)]
    from_oracle.append(from_oracle[0])
    offsets_buf = torch.full((len(big) + 1,), -1, dtype=torch.int64, device="cuda")
    status_buf = torch.full((len(big),), 255, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    free_before = None
    for k, (cfgs, d, (want_off, want_st), (orc_off, orc_st)) in enumerate(zip(batches, dev, want, from_oracle)):
        n = len(cfgs)
        offsets_buf.fill_(-1)
        status_buf.fill_(255)
        torch.cuda.synchronize()
        if k >= 1:
            free_before = torch.cuda.mem_get_info()[0]
        static_counts(llmem, d, offsets_buf, status_buf)
        if k >= 1:
            # the address look-up happened in the first call; from then on a call leaves the
            # device's free memory exactly as it found it
            assert torch.cuda.mem_get_info()[0] == free_before
        got_off, got_st = offsets_buf[:n + 1].cpu().numpy(), status_buf[:n].cpu().numpy()
        assert np.array_equal(got_off, want_off)       # integers: bit-exact, as everywhere
        assert np.array_equal(got_st, want_st)
        assert np.array_equal(got_off, orc_off)        # and equal to the oracle's own counts
        assert np.array_equal(got_st, orc_st)
        assert got_off[0] == 0 and (np.diff(got_off) >= 0).all()
        assert int(offsets_buf[n + 1:].max().item()) == -1 if n < len(big) else True
    # the closed-form count of the oracle on a sample of single records
    for i in range(0, len(small), 17):
        st, cnt = oracle.event_count(small[i:i + 1], formula=True)
        assert st == want[1][1][i] and (cnt if st == 0 else 0) == want[1][0][i + 1] - want[1][0][i]
    # the binding wrapper takes the same caller-owned buffers
    out = llmem.event_counts_static(dev[1], offsets_buf, status_buf)
    torch.cuda.synchronize()
    assert np.array_equal(out[:len(small) + 1].cpu().numpy(), want[1][0])


def test_static_event_counts_at_the_size_limit(llmem):
    """n = LLMEM_STATIC_MAX_CONFIGS exactly: the only size that uses the last entry of the
    library's array (4096 block sums plus the grand total)."""
    n = llmem.STATIC_MAX_CONFIGS
    part = grids.g3_sweep(0, 1 << 16)
    part["seq"][5::97] = 0                          # some inadmissible records
    cfgs = np.tile(part, n // len(part))
    assert len(cfgs) == n
    part_off, part_st = oracle_counts(part)
    dev = llmem.to_device(cfgs)
    offsets_buf = torch.full((n + 1,), -1, dtype=torch.int64, device="cuda")
    status_buf = torch.full((n,), 255, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        offsets_buf.fill_(-1)
        static_counts(llmem, dev, offsets_buf, status_buf)
        got = offsets_buf.cpu().numpy()
        counts = np.diff(got)
        assert np.array_equal(counts, np.tile(np.diff(part_off), n // len(part)))
        assert got[0] == 0 and got[-1] == part_off[-1] * (n // len(part))
        assert np.array_equal(status_buf.cpu().numpy(), np.tile(part_st, n // len(part)))
    want_off, _ = reference_counts(llmem, dev)
    assert np.array_equal(got, want_off)


def test_static_event_counts_rejects_oversize_and_handles_empty(llmem):
    L = llmem.lib()
    buf = torch.zeros(8, dtype=torch.int64, device="cuda")
    cfg = llmem.to_device(grids.g1_small()[:1])
    too_many = llmem.STATIC_MAX_CONFIGS + 1
    rc = L.llmem_event_counts_static(ctypes.c_void_p(cfg.data_ptr()), ctypes.c_int64(too_many),
                                     ctypes.c_void_p(buf.data_ptr()), None, 0, None)
    assert rc == llmem.ERR_ARG
    assert b"LLMEM_STATIC_MAX_CONFIGS" in L.llmem_last_error()
    buf.fill_(7)
    rc = L.llmem_event_counts_static(None, ctypes.c_int64(0), ctypes.c_void_p(buf.data_ptr()), None, 0,
                                     ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == llmem.OK
    torch.cuda.synchronize()
    assert buf.cpu().tolist() == [0, 7, 7, 7, 7, 7, 7, 7]
