"""Publication of adapter versions (Section 4.2: requests bind to the last committed adapter;
Section 5.3: the staged version runs privately while the old one serves).  Calls that name adapters
are resolved on the device at the moment they run in stream order; calls that name slots reach any
resident entry, staged ones included.  Outputs are checked against the oracle with the entry each
token should have been bound to."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import to_bits, to_dev

pytestmark = pytest.mark.gpu


def _entry(seed, aid, ver, rank, K, N):
    return wl.AdapterEntry(aid, ver, rank, 2.0, wl.normal_bf16(seed, 10 * aid + ver, (rank, K), 0.05),
                           wl.normal_bf16(seed, 100 + 10 * aid + ver, (N, rank), 0.05))


def _ref(x_bits, W_bits, entries, token_entry):
    T = x_bits.shape[0]
    return oracle.forward(x_bits, W_bits, entries, np.arange(T + 1, dtype=np.int32),
                          np.asarray(token_entry, np.int32))[0]


@pytest.mark.parametrize("T", [8, 30, 100, 200])   # (decode kernel, two blocks of 16 on the decode kernel, one-tile path, grouped GEMM path)
def test_publish_switches_resolution_at_a_point_of_the_stream(T):
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table, LmlError
    K, N = 264, 136
    tbl = Table(K, N, 6)
    x_bits, W_bits = wl.normal_bf16(3, 1, (T, K), 1.0), wl.normal_bf16(3, 2, (N, K), 0.05)
    x, W = to_dev(x_bits), to_dev(W_bits)
    e = {(0, 1): _entry(3, 0, 1, 8, K, N), (0, 2): _entry(3, 0, 2, 16, K, N), (1, 1): _entry(3, 1, 1, 4, K, N)}
    order = [(0, 1), (0, 2), (1, 1)]
    entries = [e[k] for k in order]
    idx = {k: i for i, k in enumerate(order)}
    slot = {k: tbl.register_adapter(k[0], k[1], to_dev(e[k].A), to_dev(e[k].B), e[k].scale) for k in [(0, 1), (1, 1)]}
    rng = np.random.default_rng(T)
    ids_np = rng.integers(-1, 2, size=T).astype(np.int32)      # adapter ids -1, 0, 1
    ids = torch.from_numpy(ids_np).cuda()

    # nothing published yet: adapters resolve to nothing, tokens get base output and the flag goes up
    y = to_bits(tbl.lora_mixed_linear_adapters(x, W, ids))
    torch.cuda.synchronize()
    assert tbl.device_status() == (b.FLAG_BAD_SLOT if (ids_np >= 0).any() else 0)
    assert oracle.compare(y, _ref(x_bits, W_bits, entries, [-1] * T))["ok"]
    with pytest.raises(LmlError):
        tbl.resolve(0)

    assert tbl.publish(0, 1) == -1 and tbl.publish(1, 1) == -1
    assert tbl.resolve(0) == (slot[(0, 1)], 1)
    assert tbl.slot_state(slot[(0, 1)]) == (b.STATE_SERVING, 0)
    bound_v1 = [idx[(0, 1)] if a == 0 else (idx[(1, 1)] if a == 1 else -1) for a in ids_np]
    y1 = to_bits(tbl.lora_mixed_linear_adapters(x, W, ids))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    assert oracle.compare(y1, _ref(x_bits, W_bits, entries, bound_v1))["ok"]

    # version 2 of adapter 0 is staged: resident, reachable by its slot, invisible to calls that name the adapter
    slot[(0, 2)] = tbl.register_adapter(0, 2, to_dev(e[(0, 2)].A), to_dev(e[(0, 2)].B), e[(0, 2)].scale)
    assert tbl.slot_state(slot[(0, 2)]) == (b.STATE_RESIDENT, 0)
    y1b = to_bits(tbl.lora_mixed_linear_adapters(x, W, ids))
    staged_slots = torch.full((T,), slot[(0, 2)], dtype=torch.int32, device="cuda")
    y_staged = to_bits(tbl.lora_mixed_linear_tokens(x, W, staged_slots))
    torch.cuda.synchronize()
    assert np.array_equal(y1b, y1)
    assert oracle.compare(y_staged, _ref(x_bits, W_bits, entries, [idx[(0, 2)]] * T))["ok"]

    # a request is still running under version 1 when version 2 is published: version 1 stays resident
    tbl.pin(slot[(0, 1)])
    # calls enqueued before the publication see version 1, calls after it version 2, all on one stream
    y_before = tbl.lora_mixed_linear_adapters(x, W, ids)
    assert tbl.publish(0, 2) == 1
    y_after = tbl.lora_mixed_linear_adapters(x, W, ids)
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    assert np.array_equal(to_bits(y_before), y1)
    bound_v2 = [idx[(0, 2)] if a == 0 else (idx[(1, 1)] if a == 1 else -1) for a in ids_np]
    assert oracle.compare(to_bits(y_after), _ref(x_bits, W_bits, entries, bound_v2))["ok"]
    assert tbl.resolve(0) == (slot[(0, 2)], 2)
    assert tbl.slot_state(slot[(0, 1)]) == (b.STATE_RETIRING, 1)
    # the pinned old version still serves whoever names its slot
    old_slots = torch.full((T,), slot[(0, 1)], dtype=torch.int32, device="cuda")
    y_old = to_bits(tbl.lora_mixed_linear_tokens(x, W, old_slots))
    torch.cuda.synchronize()
    assert oracle.compare(y_old, _ref(x_bits, W_bits, entries, [idx[(0, 1)]] * T))["ok"]
    # the request ends: the old version is retired and its slot is free again
    tbl.unpin(slot[(0, 1)])
    with pytest.raises(LmlError):
        tbl.lookup(0, 1)
    with pytest.raises(LmlError):
        tbl.unpin(slot[(0, 1)])
    again = tbl.register_adapter(7, 1, to_dev(e[(1, 1)].A), to_dev(e[(1, 1)].B), 1.0)
    assert again == slot[(0, 1)]
    tbl.close()


def test_publish_errors_and_retire_of_the_serving_version():
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table, LmlError
    K, N, T = 264, 136, 8
    tbl = Table(K, N, 4)
    en = _entry(9, 2, 5, 8, K, N)
    s = tbl.register_adapter(2, 5, to_dev(en.A), to_dev(en.B), en.scale)
    for bad in [(2, 6), (3, 5)]:
        with pytest.raises(LmlError) as ei:
            tbl.publish(*bad)
        assert ei.value.status == b.ERR_NOT_FOUND
    with pytest.raises(LmlError) as ei:
        tbl.publish(b.MAX_ADAPTER_IDS, 1)
    assert ei.value.status == b.ERR_INVALID_ARG
    assert tbl.publish(2, 5) == -1 and tbl.publish(2, 5) == -1      # publishing the serving version again changes nothing
    x, W = to_dev(wl.normal_bf16(9, 1, (T, K), 1.0)), to_dev(wl.normal_bf16(9, 2, (N, K), 0.05))
    ids = torch.full((T,), 2, dtype=torch.int32, device="cuda")
    y_served = to_bits(tbl.lora_mixed_linear_adapters(x, W, ids))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    tbl.pin(s)
    tbl.retire_version(2, 5)          # pinned: stays resident for its slot, but no longer serves the adapter
    assert tbl.slot_state(s) == (b.STATE_RETIRING, 1)
    y_none = to_bits(tbl.lora_mixed_linear_adapters(x, W, ids))
    y_base = to_bits(tbl.lora_mixed_linear(x, W, None, None))
    y_slot = to_bits(tbl.lora_mixed_linear_tokens(x, W, torch.full((T,), s, dtype=torch.int32, device="cuda")))
    torch.cuda.synchronize()
    assert tbl.device_status() == b.FLAG_BAD_SLOT
    assert np.array_equal(y_none, y_base) and np.array_equal(y_slot, y_served)
    tbl.unpin(s)
    with pytest.raises(LmlError):
        tbl.slot_state(s)
    tbl.close()


@pytest.mark.parametrize("ordered", [False, True])
def test_retired_serving_entry_never_resolves_to_the_slots_next_tenant(ordered):
    """An adapter is published on a busy non-blocking stream and retired while that publish is still
    queued; another adapter is then registered and takes over the slot.  A call that names the retired
    adapter must get base output and the flag, never the new tenant's delta: with the retire ordered on
    the publishing stream (the device map is cleared behind the publish) and also with the plain
    retire_version, whose clear on the legacy stream overtakes the publish and leaves a stale word in
    the map (the word names the old registration, which the slot no longer holds)."""
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table
    K, N, T = 264, 136, 8
    tbl = Table(K, N, 2)
    old, new = _entry(21, 5, 1, 8, K, N), _entry(21, 9, 1, 16, K, N)
    x_bits, W_bits = wl.normal_bf16(21, 1, (T, K), 1.0), wl.normal_bf16(21, 2, (N, K), 0.05)
    x, W = to_dev(x_bits), to_dev(W_bits)
    s_old = tbl.register_adapter(5, 1, to_dev(old.A), to_dev(old.B), old.scale)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()                 # a non-blocking stream: the legacy stream does not order against it
    big = torch.randn((4096, 4096), device="cuda")
    with torch.cuda.stream(side):
        for _ in range(40):                    # keeps the stream busy for a few milliseconds
            big = big @ big * 1e-3
        tbl.publish(5, 1, stream=side)         # queued behind the products
    if ordered:
        tbl.retire_version(5, 1, stream=side)
    else:
        tbl.retire_version(5, 1)               # its clear runs at once, before the publish lands
    with torch.cuda.stream(side):
        s_new = tbl.register_adapter(9, 1, to_dev(new.A), to_dev(new.B), new.scale, stream=side)
    assert s_new == s_old                      # lowest free index: the retired entry's slot
    side.synchronize()
    torch.cuda.synchronize()
    ids = torch.full((T,), 5, dtype=torch.int32, device="cuda")
    y = to_bits(tbl.lora_mixed_linear_adapters(x, W, ids))
    torch.cuda.synchronize()
    assert tbl.device_status() == b.FLAG_BAD_SLOT
    base = _ref(x_bits, W_bits, [old, new], [-1] * T)
    assert oracle.compare(y, base)["ok"]
    with_new = _ref(x_bits, W_bits, [old, new], [1] * T)
    assert not oracle.compare(y, with_new)["ok"]          # the other adapter's delta would show
    # the new tenant itself is reachable by its slot, and by its adapter id once published
    y_slot = to_bits(tbl.lora_mixed_linear_tokens(x, W, torch.full((T,), s_new, dtype=torch.int32, device="cuda")))
    tbl.publish(9, 1)
    y_id = to_bits(tbl.lora_mixed_linear_adapters(x, W, torch.full((T,), 9, dtype=torch.int32, device="cuda")))
    torch.cuda.synchronize()
    assert tbl.device_status() == 0
    assert oracle.compare(y_slot, with_new)["ok"] and np.array_equal(y_slot, y_id)
    tbl.close()


def test_two_step_form_across_a_publish_keeps_its_version_when_pinned():
    """Ids resolved by lml_segment_tokens_adapters, the layer run by lora_mixed_linear after a publish of
    the same adapter: with the resolved slot pinned the tokens run under the version they were bound to;
    without the pin the replaced entry is free by then and they fall back to base output with the flag."""
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table
    K, N, T = 264, 136, 200
    e1, e2 = _entry(33, 4, 1, 8, K, N), _entry(33, 4, 2, 16, K, N)
    x_bits, W_bits = wl.normal_bf16(33, 1, (T, K), 1.0), wl.normal_bf16(33, 2, (N, K), 0.05)
    x, W = to_dev(x_bits), to_dev(W_bits)
    ids = torch.full((T,), 4, dtype=torch.int32, device="cuda")
    for pinned in (True, False):
        tbl = Table(K, N, 4)
        s1 = tbl.register_adapter(4, 1, to_dev(e1.A), to_dev(e1.B), e1.scale)
        tbl.register_adapter(4, 2, to_dev(e2.A), to_dev(e2.B), e2.scale)
        tbl.publish(4, 1)
        if pinned:
            tbl.pin(s1)
        perm = torch.empty(T, dtype=torch.int32, device="cuda")
        so = torch.empty(tbl.max_slots + 2, dtype=torch.int32, device="cuda")
        sid = torch.empty(tbl.max_slots + 1, dtype=torch.int32, device="cuda")
        b.lml_segment_tokens_adapters(tbl.handle, ids.data_ptr(), T, perm.data_ptr(), so.data_ptr(), sid.data_ptr(),
                                      b._stream(None))
        tbl.publish(4, 2)                                   # the adapter moves on between the two steps
        y = to_bits(tbl.lora_mixed_linear(x, W, so, sid, perm))
        torch.cuda.synchronize()
        flags = tbl.device_status()
        if pinned:
            assert flags == 0
            assert oracle.compare(y, _ref(x_bits, W_bits, [e1, e2], [0] * T))["ok"]
            tbl.unpin(s1)
        else:
            assert flags == b.FLAG_BAD_SLOT
            assert oracle.compare(y, _ref(x_bits, W_bits, [e1, e2], [-1] * T))["ok"]
        tbl.close()
