"""lora_mixed_linear_multi: several projections of the same x (q/k/v, gate/up) in one call, every projection
with its own table (ranks up to 64, its own scales, its own slot numbering).  Each output is compared with
the oracle run on that projection alone and, bit for bit, with the separate lora_mixed_linear_tokens calls: up to
16 tokens are one launch of the decode kernel for all projections, whose CTAs each work on one projection exactly as
in a call of its own (a row's arithmetic does not depend on how the rows are dealt out)."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Guarded, to_bits, to_dev

pytestmark = pytest.mark.gpu


def _case(seed, K, Ns, ranks_per_proj, scales_per_proj, T, none_every=5):
    """Adapters a = 0..n-1; projection p holds (A, B) of rank ranks_per_proj[p][a] for adapter a."""
    n_ad = len(ranks_per_proj[0])
    x = wl.normal_bf16(seed, 1, (T, K), 1.0)
    W = [wl.normal_bf16(seed, 10 + p, (n, K), 0.02) for p, n in enumerate(Ns)]
    ents = []
    for p, n in enumerate(Ns):
        ents.append([wl.AdapterEntry(a, 1, ranks_per_proj[p][a], scales_per_proj[p][a],
                                     wl.normal_bf16(seed, 100 + 20 * p + a, (ranks_per_proj[p][a], K), 0.02),
                                     wl.normal_bf16(seed, 500 + 20 * p + a, (n, ranks_per_proj[p][a]), 0.02))
                     for a in range(n_ad)])
    rng = np.random.default_rng(seed)
    tok_adapter = rng.integers(0, n_ad, size=T).astype(np.int32)
    tok_adapter[::none_every] = -1
    return x, W, ents, tok_adapter


def _run_multi(K, Ns, x, W, ents, tok_adapter, max_slots=None, reorder=True):
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table
    T = x.shape[0]
    tables, slots = [], []
    for p, n in enumerate(Ns):
        tbl = Table(K, n, max_slots or len(ents[p]))
        order = list(range(len(ents[p])))
        if reorder and p % 2 == 1:
            order.reverse()                      # slot numbering differs between the tables
        sl = {}
        for a in order:
            e = ents[p][a]
            sl[a] = tbl.register_adapter(e.adapter_id, e.version, to_dev(e.A), to_dev(e.B), e.scale)
        tables.append(tbl)
        slots.append(sl)
    torch.cuda.synchronize()
    xd = to_dev(x)
    Wd = [to_dev(w) for w in W]
    toks = [torch.from_numpy(np.array([slots[p][a] if a >= 0 else -1 for a in tok_adapter], np.int32)).cuda()
            for p in range(len(Ns))]
    gys = [Guarded(T * n * 2) for n in Ns]
    ys = [g.view(torch.bfloat16, (T, n)) for g, n in zip(gys, Ns)]
    handles = [t.handle for t in tables]
    gws = Guarded(max(b.lml_multi_workspace_bytes(handles, T), 256))
    b.multi_projection(tables, xd, Wd, toks, ys=ys, workspace=gws.payload)
    torch.cuda.synchronize()
    assert all(g.intact() for g in gys) and gws.intact()
    flags = [t.device_status() for t in tables]
    out = [to_bits(y) for y in ys]
    # the same projections one call each
    sep = [to_bits(tables[p].lora_mixed_linear_tokens(xd, Wd[p], toks[p])) for p in range(len(Ns))]
    torch.cuda.synchronize()
    launches = tables[0].last_launch_count()
    for t in tables:
        t.close()
    return out, sep, flags


def _check(out, sep, flags, x, W, ents, tok_adapter, last_place=True):
    T = x.shape[0]
    assert flags == [0] * len(W), flags
    for p in range(len(W)):
        ref, _ = oracle.forward(x, W[p], ents[p], np.arange(T + 1, dtype=np.int32), tok_adapter)
        r = oracle.compare(out[p], ref)
        assert r["ok"], (p, r)
        if last_place:
            assert np.array_equal(out[p], sep[p]), p


@pytest.mark.parametrize("T", [1, 8, 16, 128, 2048])
def test_three_projections_with_their_own_ranks_and_scales(T):
    K, Ns = 520, (264, 136, 1000)
    ranks = [(16, 64, 4, 8), (8, 16, 64, 1), (64, 33, 16, 2)]
    scales = [(2.0, 0.5, 1.0, 4.0), (1.0, 2.0, 0.25, 3.0), (0.5, 1.5, 2.0, 1.0)]
    x, W, ents, tok = _case(40 + T, K, Ns, ranks, scales, T)
    out, sep, flags = _run_multi(K, Ns, x, W, ents, tok)
    _check(out, sep, flags, x, W, ents, tok)


@pytest.mark.parametrize("T", [3, 16])
def test_wide_projections_take_one_launch(T):
    """q/k/v-like widths of unequal size: one launch, the CTAs dealt out over the projections in proportion to their
    rows."""
    import torch
    from paper_2608_15241_b200 import binding as b
    K, Ns = 1032, (4104, 2056, 3080)
    ranks = [(16, 16, 8, 4)] * 3
    scales = [(2.0, 2.0, 1.0, 0.5), (1.0, 2.0, 0.25, 3.0), (0.5, 1.5, 2.0, 1.0)]
    x, W, ents, tok = _case(7 + T, K, Ns, ranks, scales, T)
    out, sep, flags = _run_multi(K, Ns, x, W, ents, tok)
    _check(out, sep, flags, x, W, ents, tok)


@pytest.mark.parametrize("T,ranks", [(8, (16, 16, 16, 16)), (16, (16, 8, 16, 4)), (16, (64, 33, 64, 16))])
def test_rows_of_x_wider_than_a_staged_pass_keep_their_bits(T, ranks):
    """d_in beyond the width of one pass through the staging buffer.  In the one-launch call a projection has a
    share of the SMs only, so its dot products are dealt out in larger groups than in a call of its own (singles
    against pairs, pairs against staged groups of four): whatever the grouping, a dot product is summed in the same
    order, and the outputs are equal bit for bit."""
    K, Ns = 7944, (520, 264)
    scales = [(2.0, 0.5, 1.0, 4.0), (1.0, 2.0, 0.25, 3.0)]
    x, W, ents, tok = _case(300 + T + ranks[0], K, Ns, [ranks, ranks], scales, T, none_every=7)
    out, sep, flags = _run_multi(K, Ns, x, W, ents, tok)
    _check(out, sep, flags, x, W, ents, tok)


@pytest.mark.parametrize("T", [2, 16])
def test_four_projections_some_with_very_few_rows(T):
    """LML_MAX_PROJECTIONS projections, two of them with fewer pairs of rows than their share of the SMs."""
    K, Ns = 264, (3080, 16, 1032, 40)
    ranks = [(16, 8, 64), (4, 16, 1), (64, 2, 16), (8, 8, 8)]
    scales = [(2.0, 0.5, 1.0), (1.0, 2.0, 0.25), (0.5, 1.5, 2.0), (1.0, 1.0, 3.0)]
    x, W, ents, tok = _case(90 + T, K, Ns, ranks, scales, T)
    out, sep, flags = _run_multi(K, Ns, x, W, ents, tok)
    _check(out, sep, flags, x, W, ents, tok)


def test_multi_launch_count_and_bad_ids():
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table
    K, Ns, T = 264, (1032, 520), 8
    ranks = [(16, 8), (4, 16)]
    scales = [(2.0, 1.0), (1.0, 2.0)]
    x, W, ents, tok = _case(3, K, Ns, ranks, scales, T)
    tables = [Table(K, n, 4) for n in Ns]
    for p in range(2):
        for e in ents[p]:
            tables[p].register_adapter(e.adapter_id, e.version, to_dev(e.A), to_dev(e.B), e.scale)
    xd, Wd = to_dev(x), [to_dev(w) for w in W]
    good = torch.from_numpy(np.where(tok >= 0, tok, -1).astype(np.int32)).cuda()
    ys = b.multi_projection(tables, xd, Wd, good)
    torch.cuda.synchronize()
    assert tables[0].last_launch_count() == 1 and tables[1].last_launch_count() == 0   # one launch for both
    assert [t.device_status() for t in tables] == [0, 0]
    # an id that names no live adapter in the second table only: that table's flag, base output for that token there
    bad1 = good.clone()
    bad1[1] = 3
    ys_bad = b.multi_projection(tables, xd, Wd, [good, bad1])
    torch.cuda.synchronize()
    assert [t.device_status() for t in tables] == [0, b.FLAG_BAD_SLOT]
    assert np.array_equal(to_bits(ys_bad[0]), to_bits(ys[0]))
    tok1 = tok.copy()
    tok1[1] = -1
    ref, _ = oracle.forward(x, W[1], ents[1], np.arange(T + 1, dtype=np.int32), tok1)
    assert oracle.compare(to_bits(ys_bad[1]), ref)["ok"]
    # argument errors are refused on the host
    with pytest.raises(b.LmlError):
        b.lora_mixed_linear_multi([t.handle for t in tables], xd.data_ptr(), [w.data_ptr() for w in Wd], T,
                                  [good.data_ptr()] * 2, [ys[0].data_ptr(), ys[0].data_ptr()], 0, 0)
    for t in tables:
        t.close()


def test_tables_with_many_wide_adapters():
    K, Ns, T = 264, (520, 264), 8
    ranks = [(64,) * 12, (64,) * 12]          # 768 rows of A per table: more than the weights have rows
    scales = [(1.0,) * 12, (2.0,) * 12]
    x, W, ents, tok = _case(11, K, Ns, ranks, scales, T)
    out, sep, flags = _run_multi(K, Ns, x, W, ents, tok)
    _check(out, sep, flags, x, W, ents, tok)


def test_seven_b_class_qkv_decode():
    K, Ns, T = 4096, (4096, 4096, 4096), 8
    ranks = [(16,) * 5] * 3
    scales = [(2.0,) * 5] * 3
    x, W, ents, tok = _case(0, K, Ns, ranks, scales, T, none_every=100)
    out, sep, flags = _run_multi(K, Ns, x, W, ents, tok, reorder=False)
    _check(out, sep, flags, x, W, ents, tok)
