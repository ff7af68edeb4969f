"""lora_mixed_linear_tokens (one slot id per token) against the two-call form it replaces:
lml_segment_tokens followed by lora_mixed_linear with the perm it produced.  Both forms run the
same arithmetic per output element, so the results must agree bit for bit; the oracle is checked
on top.  Covers the one-launch decode form (T <= 16), the form for a few blocks of 16 tokens (the decode kernel
again: bit for bit a decode call per block), the one-tile form (up to 128 tokens in their order: agreement with the
two-call form to the last place), the prefill form, ids that name no live adapter (flagged, treated as -1) and the
all-base case."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import to_bits, to_dev

pytestmark = pytest.mark.gpu


def _table(K, N, ranks, seed):
    from paper_2608_15241_b200.binding import Table
    tbl = Table(K, N, len(ranks) + 2)
    entries = []
    for s, r in enumerate(ranks):
        A = wl.normal_bf16(seed, 100 + s, (r, K), 0.05)
        B = wl.normal_bf16(seed, 200 + s, (N, r), 0.05)
        slot = tbl.register_adapter(s, 1, to_dev(A), to_dev(B), 1.5)
        entries.append((slot, wl.AdapterEntry(s, 1, r, 1.5, A, B)))
    return tbl, entries


@pytest.mark.parametrize("T,K,N", [(1, 264, 136), (8, 520, 264), (16, 1024, 512), (13, 4096, 520), (300, 256, 384),
                                   (17, 264, 136), (24, 1032, 520), (32, 1032, 16400), (33, 1032, 16400), (32, 4104, 4200), (48, 520, 264), (64, 520, 264), (65, 520, 264), (100, 520, 264), (128, 2048, 1000), (127, 1032, 264), (40, 1032, 16400), (129, 1024, 512), (256, 256, 384), (257, 256, 384),
                                   (200, 1536, 520)])
def test_tokens_call_equals_segment_then_layer(T, K, N):
    import torch
    tbl, entries = _table(K, N, (4, 16, 33), seed=21)
    rng = np.random.default_rng(T * 7 + 1)
    slots = np.array([e[0] for e in entries] + [-1], np.int32)
    token_slots = slots[rng.integers(0, len(slots), size=T)].astype(np.int32)
    x_bits = wl.normal_bf16(21, 1, (T, K), 1.0)
    W_bits = wl.normal_bf16(21, 2, (N, K), 0.05)
    x, W, ts = to_dev(x_bits), to_dev(W_bits), torch.from_numpy(token_slots).cuda()

    y_tok = to_bits(tbl.lora_mixed_linear_tokens(x, W, ts))
    launches_tok = tbl.last_launch_count()
    perm, so, ids = tbl.segment_tokens(ts)
    y_two = to_bits(tbl.lora_mixed_linear(x, W, so, ids, perm=perm))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    blocks = 16 < T <= (48 if K * N <= 1 << 24 else (32 if K > 4096 else 16))
    # (the two forms differ in the bf16 rounding of u, whose size grows with the length of the dot products)
    last_place = 2.0 ** -7 if K <= 2048 else 2.0 ** -6
    if blocks:
        # a few blocks of 16 tokens: one launch of the decode kernel, every block's rows exactly those of a decode call
        # on that block alone; against the two-call form (the GEMM path) equal to the last place of bf16
        assert launches_tok == 1
        for t0 in range(0, T, 16):
            y_blk = to_bits(tbl.lora_mixed_linear_tokens(x[t0:t0 + 16].contiguous(), W, ts[t0:t0 + 16].contiguous()))
            assert np.array_equal(y_tok[t0:t0 + 16], y_blk), t0
        a, b2 = wl.bf16_bits_to_f64(y_tok), wl.bf16_bits_to_f64(y_two)
        assert (np.abs(a - b2) <= last_place * np.maximum(1.0, np.abs(b2))).all()
    elif 16 < T <= (256 if K <= 4096 else 128):
        # one or two row tiles: binding and shrink in one launch with the tokens in their order, then the GEMM; the shrink sums
        # in another order than the grouped path's, so the two forms agree to the last place of bf16
        assert launches_tok == 2
        a, b2 = wl.bf16_bits_to_f64(y_tok), wl.bf16_bits_to_f64(y_two)
        assert (np.abs(a - b2) <= last_place * np.maximum(1.0, np.abs(b2))).all()
    else:
        assert np.array_equal(y_tok, y_two)
    if T <= 16:
        assert launches_tok == 1

    # oracle on the same problem: one segment per token, rows in their original order
    slot_to_entry = {slot: i for i, (slot, _) in enumerate(entries)}
    seg_entry = np.array([slot_to_entry.get(int(s), -1) for s in token_slots], np.int32)
    ref, _ = oracle.forward(x_bits, W_bits, [e for _, e in entries], np.arange(T + 1, dtype=np.int32), seg_entry)
    cmp = oracle.compare(y_tok, ref)
    assert cmp["ok"], cmp
    tbl.close()


@pytest.mark.parametrize("reps", [1, 4, 10, 20])
def test_tokens_call_flags_ids_without_adapter(reps):
    import torch
    K, N, T = 264, 136, 8 * reps
    tbl, entries = _table(K, N, (8,), seed=5)
    good = entries[0][0]
    free = [s for s in range(tbl.max_slots) if s != good][0]
    token_slots = np.tile(np.array([good, free, -1, 99, good, -7, good, -1], np.int32), reps)
    x, W = to_dev(wl.normal_bf16(5, 1, (T, K), 1.0)), to_dev(wl.normal_bf16(5, 2, (N, K), 0.05))
    y = to_bits(tbl.lora_mixed_linear_tokens(x, W, torch.from_numpy(token_slots).cuda()))
    torch.cuda.synchronize()
    from paper_2608_15241_b200.binding import FLAG_BAD_SLOT
    assert tbl.device_status() == FLAG_BAD_SLOT
    cleaned = np.where(token_slots == good, good, -1).astype(np.int32)
    y_ref = to_bits(tbl.lora_mixed_linear_tokens(x, W, torch.from_numpy(cleaned).cuda()))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    assert np.array_equal(y, y_ref)
    tbl.close()


def test_tokens_call_all_base_equals_no_segments():
    import torch
    K, N, T = 520, 264, 16
    tbl, _ = _table(K, N, (8,), seed=9)
    x, W = to_dev(wl.normal_bf16(9, 1, (T, K), 1.0)), to_dev(wl.normal_bf16(9, 2, (N, K), 0.05))
    ts = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    y = to_bits(tbl.lora_mixed_linear_tokens(x, W, ts))
    y0 = to_bits(tbl.lora_mixed_linear(x, W, None, None))
    torch.cuda.synchronize()
    assert np.array_equal(y, y0)
    tbl.close()


@pytest.mark.parametrize("T,K,N,n_adapters", [(40, 1032, 16400, 1),     # wide output: the one-tile path from 17 tokens on
                                               (17, 1032, 16400, 17),    # every token its own slot
                                               (128, 264, 136, 62)])     # a full tile, nearly every slot of a 64-slot table
def test_one_tile_path_edge_cases(T, K, N, n_adapters):
    """The path that keeps the tokens in their order (one launch binds them and computes the shrink, the GEMM follows):
    a batch without any adapter, as many distinct slots as tokens, a full tile with dozens of slots."""
    import torch
    tbl, entries = _table(K, N, (4,) * n_adapters, seed=33)
    slots = np.array([e[0] for e in entries], np.int32)
    if n_adapters == 1:
        token_slots = np.full(T, -1, np.int32)
    else:
        token_slots = slots[np.arange(T) % len(slots)].astype(np.int32)
        token_slots[::7] = -1
        if n_adapters == 17:
            token_slots = slots[:T].copy()
    x_bits = wl.normal_bf16(33, 1, (T, K), 1.0)
    W_bits = wl.normal_bf16(33, 2, (N, K), 0.02)
    x, W, ts = to_dev(x_bits), to_dev(W_bits), torch.from_numpy(token_slots).cuda()
    y_tok = to_bits(tbl.lora_mixed_linear_tokens(x, W, ts))
    assert tbl.last_launch_count() == 2
    y_again = to_bits(tbl.lora_mixed_linear_tokens(x, W, ts))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    assert np.array_equal(y_tok, y_again)
    if n_adapters == 1:
        y0 = to_bits(tbl.lora_mixed_linear(x, W, None, None))
        assert np.array_equal(y_tok, y0)
    slot_to_entry = {slot: i for i, (slot, _) in enumerate(entries)}
    seg_entry = np.array([slot_to_entry.get(int(s), -1) for s in token_slots], np.int32)
    ref, _ = oracle.forward(x_bits, W_bits, [e for _, e in entries], np.arange(T + 1, dtype=np.int32), seg_entry)
    cmp = oracle.compare(y_tok, ref)
    assert cmp["ok"], cmp
    tbl.close()
