"""llmem_event_counts_static: the event-count entry point for callers that cannot
allocate device memory when they call (framework callbacks that may not re-enter the
allocator, services with device memory fixed at start-up).  It must give exactly what
llmem_event_counts gives, call after call, although all calls share one fixed scratch
array inside the library that still holds the previous call's partial sums.

Collected last on purpose (file name): a failure here cannot hide other tests from a run
that stops at the first failure.  It has to pass alone in a fresh process (then its first
call performs the per-device address look-up) and after the rest of the suite."""
import ctypes

import numpy as np
import pytest

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
    return offsets_buf[:n + 1].cpu().numpy(), status_buf[:n].cpu().numpy()


def test_static_event_counts_match_on_consecutive_calls(llmem):
    # first call: a large batch that fills several thousand partial sums
    big = grids.g3_sweep(0, 300_000)
    big["layers"][::1000] = 0                       # some inadmissible records
    # second call: a smaller batch with a ragged last block; the array still holds the
    # first call's sums beyond what this call uses
    small = np.concatenate([grids.g1_small(), grids.g2_shape_grid(5, 1)[::3]])[:-5]
    # third call: big again, after the small one
    offsets_buf = torch.full((len(big) + 1,), -1, dtype=torch.int64, device="cuda")
    status_buf = torch.full((len(big),), 255, dtype=torch.uint8, device="cuda")
    for cfgs in (big, small, big):
        dev = llmem.to_device(cfgs)
        want_off, want_st = reference_counts(llmem, dev)
        offsets_buf.fill_(-1)
        status_buf.fill_(255)
        got_off, got_st = static_counts(llmem, dev, offsets_buf, status_buf)
        assert np.array_equal(got_off, want_off)       # integers: bit-exact, as everywhere
        assert np.array_equal(got_st, want_st)
        assert got_off[0] == 0 and (np.diff(got_off) >= 0).all()
    # the binding wrapper takes the same caller-owned buffers
    dev = llmem.to_device(small)
    want_off, _ = reference_counts(llmem, dev)
    out = llmem.event_counts_static(dev, offsets_buf, status_buf)
    torch.cuda.synchronize()
    assert np.array_equal(out[:len(small) + 1].cpu().numpy(), want_off)


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
