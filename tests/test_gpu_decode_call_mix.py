"""Decode-range calls of different kinds on ONE table, back to back on one stream with no host synchronisation in
between: the plain call (one part), a dual-version call (two parts), token-form calls of 32 and 48 tokens (two and three
blocks of 16 as parts), the no-workspace call, a call without adapters.  Each kind uses the table's exchange blocks (the
marked entries through which the CTAs of a launch hand one another the shrink result) in its own way, and every launch
must find them as the launch before left them.  A few hundred calls in random order; every kind's output must stay,
bit for bit, what its first call produced, and that first output agrees with the oracle."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import to_bits, to_dev

pytestmark = pytest.mark.gpu


def test_many_decode_calls_of_mixed_kinds_on_one_table():
    import torch
    from paper_2608_15241_b200.binding import Table
    K, N, ranks = 1032, 520, (16, 4, 33, 8, 64, 16)
    tbl = Table(K, N, len(ranks) + 1)
    entries, slots = [], []
    for s, r in enumerate(ranks):
        A = wl.normal_bf16(61, 100 + s, (r, K), 0.02)
        B = wl.normal_bf16(61, 200 + s, (N, r), 0.02)
        slots.append(tbl.register_adapter(s, 1, to_dev(A), to_dev(B), 2.0))
        entries.append(wl.AdapterEntry(s, 1, r, 2.0, A, B))
    rng = np.random.default_rng(61)
    T_max = 48
    x_bits = wl.normal_bf16(61, 1, (T_max, K), 1.0)
    W_bits = wl.normal_bf16(61, 2, (N, K), 0.02)
    x, W = to_dev(x_bits), to_dev(W_bits)
    choice = np.array(slots + [-1], np.int32)
    tok = choice[rng.integers(0, len(choice), size=T_max)].astype(np.int32)
    tok_d = torch.from_numpy(tok).cuda()
    # segments form of the first 13 tokens: one segment per token
    so13 = torch.arange(14, dtype=torch.int32, device="cuda")
    ids13_a = tok_d[:13].contiguous()
    ids13_b = torch.from_numpy(np.roll(tok[:13], 3).astype(np.int32)).cuda()

    x13 = x[:13].contiguous()

    def static13():
        from paper_2608_15241_b200 import binding as b
        y = torch.empty((13, N), dtype=torch.bfloat16, device="cuda")
        b.lora_mixed_linear_decode_static(tbl.handle, x13.data_ptr(), W.data_ptr(), 13, so13.data_ptr(), ids13_a.data_ptr(), 13, 0,
                                          y.data_ptr(), b._stream(None))
        return y

    kinds = {
        "plain8": lambda: [tbl.lora_mixed_linear_tokens(x[:8].contiguous(), W, tok_d[:8].contiguous())],
        "plain16": lambda: [tbl.lora_mixed_linear_tokens(x[:16].contiguous(), W, tok_d[:16].contiguous())],
        "segments13": lambda: [tbl.lora_mixed_linear(x[:13].contiguous(), W, so13, ids13_a)],
        "dual13": lambda: list(tbl.lora_mixed_linear_dual(x[:13].contiguous(), W, so13, ids13_a, ids13_b)),
        "blocks32": lambda: [tbl.lora_mixed_linear_tokens(x[:32].contiguous(), W, tok_d[:32].contiguous())],
        "blocks48": lambda: [tbl.lora_mixed_linear_tokens(x[:48].contiguous(), W, tok_d[:48].contiguous())],
        "base16": lambda: [tbl.lora_mixed_linear(x[:16].contiguous(), W, None, None)],
        "static13": lambda: [static13()],
    }
    first = {}
    for name, fn in kinds.items():
        first[name] = [to_bits(y) for y in fn()]
    torch.cuda.synchronize()
    assert tbl.device_status() == 0

    # kinds that promise the same bits: the no-workspace call and the first binding of the dual call against the plain call
    assert np.array_equal(first["static13"][0], first["segments13"][0])
    assert np.array_equal(first["dual13"][0], first["segments13"][0])

    # the oracle on two of the kinds
    slot_to_entry = {s: i for i, s in enumerate(slots)}
    seg_entry = np.array([slot_to_entry.get(int(s), -1) for s in tok], np.int32)
    for name, T in (("plain16", 16), ("blocks48", 48)):
        ref, _ = oracle.forward(x_bits[:T], W_bits, entries, np.arange(T + 1, dtype=np.int32), seg_entry[:T])
        r = oracle.compare(first[name][0], ref)
        assert r["ok"], (name, r)

    names = list(kinds)
    order = rng.integers(0, len(names), size=400)
    held = {}
    for step, k in enumerate(order):
        held[names[k]] = kinds[names[k]]()          # (no synchronisation: the launches follow one another on the stream)
        if step % 40 == 39:
            torch.cuda.synchronize()
            for name, ys in held.items():
                for y, y0 in zip(ys, first[name]):
                    assert np.array_equal(to_bits(y), y0), (name, step)
            held = {}
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    tbl.close()
