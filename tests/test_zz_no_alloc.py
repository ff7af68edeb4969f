"""The workspace-free decode entry point.  Some callers cannot allocate device memory at all (a
callback inside a runtime that owns every allocation, a loop that must never reach the
allocator), so lora_mixed_linear_decode_static keeps its scratch in a fixed array inside the
library.  Here it is called through the C ABI and must reproduce the regular entry point's
output on two calls in a row that use different inputs, so that contents left in the shared
array by the first call would show up as a mismatch in the second.

Collected last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Site, to_bits

pytestmark = pytest.mark.gpu


def run_static(site, w):
    import torch
    from paper_2608_15241_b200 import binding as b
    so = torch.from_numpy(w.seg_offsets).cuda()
    ids = torch.from_numpy(site.slot_ids()).cuda()
    pm = None if w.perm is None else torch.from_numpy(w.perm).cuda()
    y = torch.full((w.T, w.d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
    b.lora_mixed_linear_decode_static(site.table.handle, site.x.data_ptr(), site.W0.data_ptr(), w.T,
                                      so.data_ptr(), ids.data_ptr(), w.G, 0 if pm is None else pm.data_ptr(),
                                      y.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return to_bits(y), site.table.device_status()


def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row():
    # first call: 16 rows, every row on an adapter; second call: 5 shuffled rows, some without
    first = wl.ragged(T=16, d_in=520, d_out=264, ranks=(16, 4, 64, 8, 33))
    first.seg_offsets = np.array([0, 7, 16], np.int32)
    first.seg_entry = np.array([2, 0], np.int32)
    second = wl.ragged(seed=3, T=5, d_in=520, d_out=264, ranks=(16, 4, 64, 8, 33), shuffled=True)
    for w in (first, second):
        site = Site(w)
        try:
            y_static, flags = run_static(site, w)
            y_regular, flags2 = site.run()
            assert flags == 0 and flags2 == 0
            # same kernels, same scratch contents: the outputs agree bit for bit ...
            assert np.array_equal(y_static, y_regular)
            # ... and both sit within the parity tolerance of the oracle
            ref, _ = oracle.forward_workload(w)
            r = oracle.compare(y_static, ref)
            assert r["ok"], r
        finally:
            site.close()


def test_static_scratch_entry_point_rejects_oversized_calls():
    import torch
    from paper_2608_15241_b200 import binding as b
    w = wl.ragged(T=17, d_in=256, d_out=264)
    site = Site(w)
    try:
        y = torch.empty((w.T, w.d_out), dtype=torch.bfloat16, device="cuda")
        so = torch.from_numpy(w.seg_offsets).cuda()
        ids = torch.from_numpy(site.slot_ids()).cuda()
        with pytest.raises(b.LmlError) as e:
            b.lora_mixed_linear_decode_static(site.table.handle, site.x.data_ptr(), site.W0.data_ptr(), w.T,
                                              so.data_ptr(), ids.data_ptr(), w.G, 0, y.data_ptr(), 0)
        assert e.value.status == 10 and "TOO_LARGE" in str(e.value)
    finally:
        site.close()
