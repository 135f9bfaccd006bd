"""gs_risk_scan_noalloc -- the risk scan for callers that are not allowed to allocate device
memory (all of it already belongs to a KV-cache pool, or an allocation's implicit
synchronisation would stall a serving loop).  Its scratch is a fixed array inside the
library instead of a context's buffers; the results must equal gs_risk_scan's bit for bit,
and the oracle's, on back-to-back calls that reuse that one array with different inputs, and
no call after the first may change the amount of free device memory.

Collected last on purpose: if this file fails, every other test has already run."""
import ctypes as C

import numpy as np
import pytest

import workloads as W

torch = pytest.importorskip("torch")


def _scan_both_ways(gs, wl, n_active, capacity, with_status=True, check_free_memory=False):
    import oracle
    from paper_2605_16867_b200 import InstancePool, risk_scan_noalloc
    dev = gs.device
    pool = InstancePool.from_host(wl.types, wl.instances, dev)
    cols = [torch.from_numpy(np.ascontiguousarray(c[:n_active])).to(dev) for c in wl.active.columns()]
    words = (n_active + 31) // 32

    def buffers():
        return (torch.full((max(words, 1),), -1, dtype=torch.int32, device=dev),
                torch.full((max(capacity, 1),), -9, dtype=torch.int32, device=dev),
                torch.full((1,), -1, dtype=torch.int64, device=dev))

    bits_a, cand_a, count_a = buffers()
    gs.risk_scan(*cols, pool, bits_a, cand_a, count_a, cand_capacity=capacity)
    bits_b, cand_b, count_b = buffers()
    status = torch.zeros(1, dtype=torch.int32, device=dev) if with_status else None
    torch.cuda.synchronize(dev)
    free_before = torch.cuda.mem_get_info(dev)[0]
    risk_scan_noalloc(*cols, pool, bits_b, cand_b, count_b, status, cand_capacity=capacity)
    torch.cuda.synchronize(dev)
    if check_free_memory:                          # (the very first call on a GPU may load the kernels' module)
        assert torch.cuda.mem_get_info(dev)[0] == free_before
    assert int(count_a.item()) == int(count_b.item()) >= 0
    assert torch.equal(bits_a[:words], bits_b[:words])
    assert torch.equal(cand_a, cand_b)             # including the untouched tail past the count
    # ... and against the CPU oracle directly, not only against the other entry point
    tab = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32")
    flags = oracle.risk(tab, *(c[:n_active] for c in wl.active.columns())).flag
    ref_bits, ref_cand, ref_count = oracle.compact(flags)
    assert int(count_b.item()) == ref_count
    assert np.array_equal(bits_b[:words].cpu().numpy().view(np.uint32), ref_bits)
    n_listed = min(ref_count, capacity)
    assert np.array_equal(cand_b[:n_listed].cpu().numpy(), ref_cand[:n_listed])
    return int(count_b.item()), int(status.item()) if with_status else None, gs.device_status()


@pytest.mark.gpu
def test_noalloc_scan_equals_context_scan_on_consecutive_calls():
    from paper_2605_16867_b200 import GoodServe
    assert torch.cuda.is_available()
    gs = GoodServe(0)
    big = W.make_workload(2, n_requests=16, n_active=1_500_000)
    small = W.make_workload(0, n_requests=16, n_active=1024)
    # first call: large; second: a different pool and a much smaller, ragged population, so
    # whatever the first call left in the shared scratch (chunk counts, group totals) would show up
    c1, s1, ctx1 = _scan_both_ways(gs, big, 1_500_000, 1_500_000)
    c2, s2, ctx2 = _scan_both_ways(gs, small, 1001, 1001, check_free_memory=True)
    c3, s3, ctx3 = _scan_both_ways(gs, big, 700_001, 1000, check_free_memory=True)      # truncated candidate list
    assert 0 < c2 < 1001 and c1 > c3 > 1000
    assert s1 == ctx1 == 0 and s2 == ctx2 == 0
    assert s3 == ctx3 == 16                                      # GS_DEV_CAND_TRUNCATED on both paths
    c0, _, _ = _scan_both_ways(gs, small, 0, 0)                  # empty scan
    assert c0 == 0
    # without a status word the bits are dropped, the results are the same
    c4, s4, _ = _scan_both_ways(gs, big, 300_000, 300_000, with_status=False, check_free_memory=True)
    assert c4 > 0 and s4 is None
    gs.close()


def test_noalloc_scan_rejects_oversized_input_before_touching_the_gpu():
    from paper_2605_16867_b200 import NOALLOC_MAX_ACTIVE, load_library
    from paper_2605_16867_b200.binding import _Instances, _Types
    lib = load_library()
    inst = _Instances(16, 16, 16, 16, 16, 4)
    types = _Types(16, 16, 16, 2)
    rc = lib.gs_risk_scan_noalloc(16, 16, 16, 16, 16, NOALLOC_MAX_ACTIVE + 1, C.byref(inst), C.byref(types),
                                  16, 16, 0, 16, None, None)
    assert rc == -6
    assert b"GS_NOALLOC_MAX_ACTIVE" in lib.gs_strerror(rc)
