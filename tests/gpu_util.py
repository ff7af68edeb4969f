"""Helpers for the GPU parity tests: push a Workload through the C-ABI binding."""
import numpy as np


def to_dev(bits: np.ndarray, device="cuda:0"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def to_bits(t) -> np.ndarray:
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Guarded:
    """A device buffer between two canary bands.  The library is handed the middle; after the call the
    bands must still hold the canary byte: a write before or behind a buffer is caught even without a
    memory checker.  The payload starts out as 0xFF bytes (a bf16 / fp32 NaN), so an element the
    library should have written and did not shows up in any comparison."""

    BAND = 4096
    CANARY = 0xA5

    def __init__(self, nbytes, device="cuda:0", fill=0xFF):
        import torch
        self.nbytes = int(nbytes)
        pad = (-self.nbytes) % 256
        self.raw = torch.full((2 * self.BAND + self.nbytes + pad,), self.CANARY, dtype=torch.uint8, device=device)
        self.payload = self.raw[self.BAND:self.BAND + self.nbytes]
        if self.nbytes:
            self.payload.fill_(fill)

    def view(self, dtype, shape):
        return self.payload.view(dtype).view(*shape)

    def intact(self) -> bool:
        head = self.raw[:self.BAND]
        tail = self.raw[self.BAND + self.nbytes:]
        return bool((head == self.CANARY).all().item()) and bool((tail == self.CANARY).all().item())


class Site:
    """A table with a workload's entries registered and its tensors resident on the GPU."""

    def __init__(self, w, max_slots=None, device="cuda:0"):
        import torch
        from paper_2608_15241_b200.binding import Table
        self.w = w
        self.device = device
        self.table = Table(w.d_in, w.d_out, max_slots or max(len(w.entries), 1))
        self.slots = []
        for e in w.entries:
            self.slots.append(self.table.register_adapter(e.adapter_id, e.version, to_dev(e.A), to_dev(e.B), e.scale))
        torch.cuda.synchronize()
        self.x = to_dev(w.x)
        self.W0 = to_dev(w.W0)

    def slot_ids(self, seg_entry=None):
        se = self.w.seg_entry if seg_entry is None else seg_entry
        return np.array([self.slots[e] if 0 <= e < len(self.slots) else e for e in se], dtype=np.int32)

    def run(self, seg_offsets=None, seg_entry=None, perm="workload", x=None, raw_slot_ids=None):
        import torch
        w = self.w
        so = w.seg_offsets if seg_offsets is None else np.asarray(seg_offsets, np.int32)
        ids = self.slot_ids(seg_entry) if raw_slot_ids is None else np.asarray(raw_slot_ids, np.int32)
        pm = w.perm if isinstance(perm, str) else perm
        dso = torch.from_numpy(np.ascontiguousarray(so, dtype=np.int32)).to(self.device)
        dids = torch.from_numpy(ids).to(self.device) if len(ids) else None
        dpm = None if pm is None else torch.from_numpy(np.ascontiguousarray(pm, dtype=np.int32)).to(self.device)
        xx = self.x if x is None else x
        # output and workspace sit between canary bands; the workspace is exactly as large as the library asks
        T, G = int(xx.shape[0]), len(ids)
        gy = Guarded(T * w.d_out * 2, self.device)
        gws = Guarded(max(self.table.workspace_bytes(T, G), 256), self.device)
        y = gy.view(torch.bfloat16, (T, w.d_out))
        self.table.lora_mixed_linear(xx, self.W0, dso, dids, dpm, y=y, workspace=gws.payload)
        torch.cuda.synchronize()
        assert gy.intact(), "the call wrote outside y"
        assert gws.intact(), "the call wrote outside its workspace"
        return to_bits(y), self.table.device_status()

    def close(self):
        self.table.close()


def sample_positions_every_tile(w, count, tile=128, seed=0):
    """At least `count` positions: one in every `tile`-row band (so that no row tile of the GEMM goes
    unchecked), every segment's first and last row, and random ones."""
    rng = np.random.default_rng(seed)
    pos = set()
    for t0 in range(0, w.T, tile):
        pos.add(int(rng.integers(t0, min(t0 + tile, w.T))))
    for g in range(w.G):
        a, b = int(w.seg_offsets[g]), int(w.seg_offsets[g + 1])
        if b > a:
            pos.update((a, b - 1))
    while len(pos) < min(count, w.T):
        pos.add(int(rng.integers(0, w.T)))
    return np.array(sorted(pos), dtype=np.int32)


def sample_positions(w, count, seed=0):
    """Positions covering every segment's first and last row plus random ones."""
    pos = set()
    for g in range(w.G):
        a, b = int(w.seg_offsets[g]), int(w.seg_offsets[g + 1])
        if b > a:
            pos.update((a, b - 1))
    rng = np.random.default_rng(seed)
    while len(pos) < min(count, w.T):
        pos.add(int(rng.integers(0, w.T)))
    return np.array(sorted(pos), dtype=np.int32)
