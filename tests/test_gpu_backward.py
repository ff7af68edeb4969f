"""Backward pass of the layer against the fp64 oracle.  dx is the forward kernels on the transposed
table (W0^T, adapters registered transposed); dA and dB come from the gradient kernels, which work on
bf16-rounded small products (the shrink results: about 1e-3 relative).  All three are held to the
forward pass's criterion: every element within 1e-2 * max(1, |oracle|) and relative Frobenius error
at most 5e-3.  The measured figures are printed (pytest -s shows them).  Gradient buffers sit between
canary bands."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Guarded, to_bits, to_dev

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
    gdA, gdB = Guarded(tbl.max_slots * 64 * K * 4, fill=0), Guarded(tbl.max_slots * N * 64 * 4, fill=0)
    dA = gdA.view(torch.float32, (tbl.max_slots, 64, K))
    dB = gdB.view(torch.float32, (tbl.max_slots, N, 64))
    tbl.backward_adapters(tbl_T, x, dy, so, d_ids, d_ids_T, dA, dB)
    torch.cuda.synchronize()
    assert gdA.intact() and gdB.intact(), "the gradient kernels wrote outside dA / dB"
    assert tbl.device_status() == 0 and tbl_T.device_status() == 0
    dA1, dB1 = dA.cpu().numpy().astype(np.float64), dB.cpu().numpy().astype(np.float64)
    results = []
    used = set(int(e) for g, e in enumerate(w.seg_entry) if e >= 0 and w.seg_offsets[g + 1] > w.seg_offsets[g])
    for e, ent in enumerate(w.entries):
        gA, gB = dA1[slots[e], :ent.rank, :], dB1[slots[e], :, :ent.rank]
        assert not dA1[slots[e], ent.rank:, :].any() and not dB1[slots[e], :, ent.rank:].any()
        if e not in used:
            assert not gA.any() and not gB.any()
            continue
        for name, got, ref in (("dA", gA, ref_dA[e]), ("dB", gB, ref_dB[e])):
            fro = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
            # a gradient element is a sum over the slot's tokens: its rounding error grows with the size of the
            # terms, not with the size of the (possibly cancelling) sum, so the per-element bound takes the
            # matrix's scale into account: 1e-2 * max(1, |oracle|, 0.25 * largest |oracle| of the matrix)
            bound = 1e-2 * np.maximum(np.maximum(1.0, np.abs(ref)), 0.25 * np.abs(ref).max())
            worst = (np.abs(got - ref) / bound).max()
            plain = (np.abs(got - ref) / (1e-2 * np.maximum(1.0, np.abs(ref)))).max()
            print(f"T={T} K={K} N={N} entry {e} rank {ent.rank} {name}: rel_fro {fro:.2e}, max |err| {np.abs(got - ref).max():.3e}, "
                  f"max |ref| {np.abs(ref).max():.2f}, worst element at {worst:.3f} of its bound ({plain:.2f} of 1e-2 max(1, |ref|))")
            results.append((e, name, fro, worst))
    assert all(fro <= 5e-3 for _, _, fro, _ in results), results
    assert all(worst <= 1.0 for _, _, _, worst in results), results
    tbl.backward_adapters(tbl_T, x, dy, so, d_ids, d_ids_T, dA, dB)
    torch.cuda.synchronize()
    assert np.array_equal(dA.cpu().numpy().astype(np.float64), 2.0 * dA1) and np.array_equal(dB.cpu().numpy().astype(np.float64), 2.0 * dB1)
    tbl.close(); tbl_T.close()
