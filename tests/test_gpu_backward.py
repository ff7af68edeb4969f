"""Backward pass of the layer against the fp64 oracle.  dx is the forward kernels on the transposed
table (W0^T, adapters registered transposed); dA and dB come from the gradient kernels, which work on
bf16-rounded small products (the shrink results), hence the looser bound on them: relative Frobenius
error 1e-2 and every element within 2e-2 of the largest magnitude of its matrix."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,K,N", [(300, 264, 136), (8, 520, 264), (1100, 1024, 512), (129, 200, 1032)])
def test_backward_matches_the_oracle(T, K, N):
    import torch
    from paper_2608_15241_b200.binding import Table
    w = wl.ragged(T=T, d_in=K, d_out=N, ranks=(4, 16, 1, 33, 64))
    dy_bits = wl.normal_bf16(77, 3, (T, N), 1.0)
    tbl, tbl_T = Table(K, N, len(w.entries) + 1), Table(N, K, len(w.entries) + 2)
    slots, slots_T = [], []
    filler = tbl_T.register_adapter_transposed(99, 1, to_dev(w.entries[0].A), to_dev(w.entries[0].B), 1.0)   # slots differ between the tables
    for e in w.entries:
        slots.append(tbl.register_adapter(e.adapter_id, e.version, to_dev(e.A), to_dev(e.B), e.scale))
        slots_T.append(tbl_T.register_adapter_transposed(e.adapter_id, e.version, to_dev(e.A), to_dev(e.B), e.scale))
    assert filler not in slots_T
    ids = np.array([slots[e] if e >= 0 else -1 for e in w.seg_entry], np.int32)
    ids_T = np.array([slots_T[e] if e >= 0 else -1 for e in w.seg_entry], np.int32)
    x, dy = to_dev(w.x), to_dev(dy_bits)
    W0T = to_dev(np.ascontiguousarray(w.W0.T))
    so, d_ids, d_ids_T = (torch.from_numpy(a).cuda() for a in (w.seg_offsets, ids, ids_T))

    ref_dx, ref_dA, ref_dB, _ = oracle.backward(w.x, dy_bits, w.W0, w.entries, w.seg_offsets, w.seg_entry)

    # dx: the layer on the transposed problem
    dx = to_bits(tbl_T.lora_mixed_linear(dy, W0T, so, d_ids_T))
    torch.cuda.synchronize()
    assert tbl_T.device_status() == 0
    r = oracle.compare(dx, ref_dx)
    assert r["ok"], r

    # dA, dB: two calls accumulate (second batch = the same tokens again: twice the gradient)
    dA = torch.zeros((tbl.max_slots, 64, K), dtype=torch.float32, device="cuda")
    dB = torch.zeros((tbl.max_slots, N, 64), dtype=torch.float32, device="cuda")
    tbl.backward_adapters(tbl_T, x, dy, so, d_ids, d_ids_T, dA, dB)
    torch.cuda.synchronize()
    assert tbl.device_status() == 0 and tbl_T.device_status() == 0
    dA1, dB1 = dA.cpu().numpy().astype(np.float64), dB.cpu().numpy().astype(np.float64)
    used = set(int(e) for g, e in enumerate(w.seg_entry) if e >= 0 and w.seg_offsets[g + 1] > w.seg_offsets[g])
    for e, ent in enumerate(w.entries):
        gA, gB = dA1[slots[e], :ent.rank, :], dB1[slots[e], :, :ent.rank]
        assert not dA1[slots[e], ent.rank:, :].any() and not dB1[slots[e], :, ent.rank:].any()
        if e not in used:
            assert not gA.any() and not gB.any()
            continue
        for got, ref in ((gA, ref_dA[e]), (gB, ref_dB[e])):
            scale = max(np.abs(ref).max(), 1.0)
            assert np.linalg.norm(got - ref) <= 1e-2 * max(np.linalg.norm(ref), 1e-30), (e, np.linalg.norm(got - ref) / np.linalg.norm(ref))
            assert np.abs(got - ref).max() <= 2e-2 * scale, (e, np.abs(got - ref).max(), scale)
    tbl.backward_adapters(tbl_T, x, dy, so, d_ids, d_ids_T, dA, dB)
    torch.cuda.synchronize()
    assert np.array_equal(dA.cpu().numpy().astype(np.float64), 2.0 * dA1) and np.array_equal(dB.cpu().numpy().astype(np.float64), 2.0 * dB1)
    tbl.close(); tbl_T.close()
