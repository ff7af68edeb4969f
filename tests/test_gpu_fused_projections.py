"""Several projections that read the same x (q/k/v of one layer) as one call: concatenated base
weight, adapters fused into a block-diagonal B.  The fused call must reproduce the separate calls
bit for bit (the extra K-steps only ever add exact zeros) and match the oracle on the fused problem."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T", [8, 300])
def test_fused_qkv_equals_separate_calls(T):
    import torch
    from paper_2608_15241_b200.binding import Table, fuse_projection_adapters
    K, Ns, ranks, scale = 256, (256, 128, 192), (16, 16, 8), 2.0
    x_bits = wl.normal_bf16(11, 1, (T, K), 1.0)
    W_bits = [wl.normal_bf16(11, 10 + p, (n, K), 0.05) for p, n in enumerate(Ns)]
    # two adapters (slots), each with its own A/B per projection
    adapters = []
    for s in range(2):
        adapters.append([(wl.normal_bf16(11, 100 + 10 * s + p, (ranks[p], K), 0.05),
                          wl.normal_bf16(11, 200 + 10 * s + p, (Ns[p], ranks[p]), 0.05)) for p in range(3)])
    so = np.array([0, T // 3, T], np.int32)
    x = to_dev(x_bits)
    d_so = torch.from_numpy(so).cuda()

    # separate calls, one table per projection
    ys = []
    for p in range(3):
        tbl = Table(K, Ns[p], 2)
        slots = [tbl.register_adapter(s, 1, to_dev(adapters[s][p][0]), to_dev(adapters[s][p][1]), scale) for s in range(2)]
        ids = torch.tensor(slots, dtype=torch.int32, device="cuda")
        ys.append(to_bits(tbl.lora_mixed_linear(x, to_dev(W_bits[p]), d_so, ids)))
        torch.cuda.synchronize()
        tbl.close()
    y_sep = np.concatenate(ys, axis=1)

    # one fused call
    tbl = Table(K, sum(Ns), 2)
    Wcat = to_dev(np.concatenate(W_bits, axis=0))
    fused_entries, slots = [], []
    for s in range(2):
        A, B = fuse_projection_adapters([(to_dev(a), to_dev(b)) for a, b in adapters[s]])
        slots.append(tbl.register_adapter(s, 1, A, B, scale))
        fused_entries.append(wl.AdapterEntry(s, 1, int(A.shape[0]), scale, to_bits(A), to_bits(B)))
    ids = torch.tensor(slots, dtype=torch.int32, device="cuda")
    y_fused = to_bits(tbl.lora_mixed_linear(x, Wcat, d_so, ids))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    tbl.close()

    assert np.array_equal(y_fused, y_sep)
    # each projection's columns against the oracle on that projection's own (A_p, B_p): no helper of the
    # product stands between the raw adapters and the expected values
    n0 = 0
    for p in range(3):
        ents = [wl.AdapterEntry(s, 1, ranks[p], scale, adapters[s][p][0], adapters[s][p][1]) for s in range(2)]
        ref_p, _ = oracle.forward(x_bits, W_bits[p], ents, so, np.array([0, 1], np.int32))
        r = oracle.compare(np.ascontiguousarray(y_fused[:, n0:n0 + Ns[p]]), ref_p)
        assert r["ok"], (p, r)
        n0 += Ns[p]
    ref, _ = oracle.forward(x_bits, np.concatenate(W_bits, axis=0), fused_entries, so, np.array([0, 1], np.int32))
    assert oracle.compare(y_fused, ref)["ok"]
