"""Seeded synthetic workloads for the mixed-adapter LoRA linear layer.

This module only *draws inputs*: bf16 bit patterns for x, W0, A, B and the integer
token -> adapter-entry assignment.  It contains none of the layer's arithmetic and is
the one module shared by the CPU oracle's tests and the CUDA path's tests / bench, so
both sides consume exactly the same bits.

The workloads stand in for the paper's multi-agent serving batches (several agents'
tokens on one frozen base model, a handful of resident adapters, an old and a freshly
published version of one adapter resident together right after a publish — Section 5.3,
"stale-coverage prefill", and Section 4.2, "last committed serving adapter") at 7B-class
projection shapes.  Value distributions: x ~ N(0,1); W0, A, B ~ N(0, 0.02); every tensor
is rounded once to bf16 (round-to-nearest-even) and handed around as uint16.

Random numbers come from numpy's counter-based Philox generator keyed by
(seed, stream id), one stream per tensor, so a tensor's bits do not depend on which
other tensors were drawn first.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np

BF16_DTYPE = np.uint16

# Stream ids (second Philox key word).  Adapter entry e uses ADAPTER_A + e / ADAPTER_B + e.
_STREAM_X = 1
_STREAM_W0 = 2
_STREAM_ASSIGN = 3
_STREAM_ADAPTER_A = 1000
_STREAM_ADAPTER_B = 2000


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def normal_bf16(seed: int, stream: int, shape: Sequence[int], std: float) -> np.ndarray:
    g = _rng(seed, stream)
    a = g.standard_normal(size=tuple(shape), dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return f32_to_bf16_bits(a)


@dataclasses.dataclass
class AdapterEntry:
    """One resident (adapter, version) pair: A is [rank][d_in], B is [d_out][rank]."""

    adapter_id: int
    version: int
    rank: int
    scale: float
    A: np.ndarray  # uint16 [rank, d_in]
    B: np.ndarray  # uint16 [d_out, rank]


@dataclasses.dataclass
class Workload:
    """One call's worth of inputs.

    seg_offsets[G+1] / seg_entry[G] describe contiguous *positions*; position p is row
    perm[p] of x and y when perm is given, else row p.  seg_entry holds an index into
    `entries`, or -1 for "no adapter".  token_entry[T] is the same binding seen per row
    of x (what the token-segmentation pass takes as input).
    """

    name: str
    d_in: int
    d_out: int
    T: int
    x: np.ndarray  # uint16 [T, d_in]
    W0: np.ndarray  # uint16 [d_out, d_in]
    entries: List[AdapterEntry]
    seg_offsets: np.ndarray  # int32 [G+1]
    seg_entry: np.ndarray  # int32 [G]
    token_entry: np.ndarray  # int32 [T]
    perm: Optional[np.ndarray] = None  # int32 [T] or None

    @property
    def G(self) -> int:
        return int(self.seg_entry.shape[0])

    def flops(self) -> float:
        """Algorithmic FLOPs: base GEMM plus true-rank shrink and expand."""
        f = 2.0 * self.T * self.d_in * self.d_out
        for g in range(self.G):
            e = int(self.seg_entry[g])
            if e >= 0:
                n = int(self.seg_offsets[g + 1] - self.seg_offsets[g])
                f += 2.0 * n * self.entries[e].rank * (self.d_in + self.d_out)
        return f

    def bytes(self) -> float:
        """Algorithmic bytes: W0, x, y once; each adapter entry that serves >=1 token once;
        the segment arrays (and perm when present)."""
        b = 2.0 * self.d_in * self.d_out + 2.0 * self.T * (self.d_in + self.d_out)
        used = set()
        for g in range(self.G):
            e = int(self.seg_entry[g])
            if e >= 0 and self.seg_offsets[g + 1] > self.seg_offsets[g]:
                used.add(e)
        for e in used:
            b += 2.0 * self.entries[e].rank * (self.d_in + self.d_out)
        b += 4.0 * (self.G + 1) + 4.0 * self.G
        if self.perm is not None:
            b += 4.0 * self.T
        return b


def make_entries(seed: int, d_in: int, d_out: int, specs: Sequence[tuple], std: float = 0.02
                 ) -> List[AdapterEntry]:
    """specs: (adapter_id, version, rank, scale) per resident entry, in entry order."""
    out = []
    for e, (aid, ver, rank, scale) in enumerate(specs):
        A = normal_bf16(seed, _STREAM_ADAPTER_A + e, (rank, d_in), std)
        B = normal_bf16(seed, _STREAM_ADAPTER_B + e, (d_out, rank), std)
        out.append(AdapterEntry(int(aid), int(ver), int(rank), float(scale), A, B))
    return out


def segments_from_lengths(lengths: Sequence[int], entry_of_segment: Sequence[int]):
    off = np.zeros(len(lengths) + 1, dtype=np.int32)
    off[1:] = np.cumsum(np.asarray(lengths, dtype=np.int64))
    seg_entry = np.asarray(entry_of_segment, dtype=np.int32)
    token_entry = np.repeat(seg_entry, np.asarray(lengths, dtype=np.int64)).astype(np.int32)
    return off, seg_entry, token_entry


def group_tokens(token_entry: np.ndarray, num_entries: int):
    """Host-side statement of the grouping rule used to build grouped workloads: stable,
    entries ascending, -1 last.  Returns (perm, seg_offsets, seg_entry) with one segment per
    entry that has at least one token."""
    key = np.where(token_entry < 0, num_entries, token_entry).astype(np.int64)
    perm = np.argsort(key, kind="stable").astype(np.int32)
    counts = np.bincount(key, minlength=num_entries + 1)
    seg_entry, lengths = [], []
    for s in range(num_entries + 1):
        if counts[s] > 0:
            seg_entry.append(s if s < num_entries else -1)
            lengths.append(int(counts[s]))
    off = np.zeros(len(lengths) + 1, dtype=np.int32)
    off[1:] = np.cumsum(lengths)
    return perm, off, np.asarray(seg_entry, dtype=np.int32)


def _base(seed: int, T: int, d_in: int, d_out: int):
    x = normal_bf16(seed, _STREAM_X, (T, d_in), 1.0)
    W0 = normal_bf16(seed, _STREAM_W0, (d_out, d_in), 0.02)
    return x, W0


def tiny(seed: int = 0, scale_numerator: float = 2.0, zero_base: bool = False) -> Workload:
    """d_in = d_out = 256, 64 tokens in segments 30/20/14 on entries 0,1,2 with ranks
    4,8,8 and scale = scale_numerator / rank.  zero_base=True sets W0 = 0 so the output is
    the LoRA term alone; scale_numerator=100 makes the LoRA term as large as the base term."""
    K = N = 256
    T = 64
    x, W0 = _base(seed, T, K, N)
    if zero_base:
        W0 = np.zeros_like(W0)
    ranks = (4, 8, 8)
    entries = make_entries(seed, K, N, [(i, 1, r, scale_numerator / r) for i, r in enumerate(ranks)])
    off, seg_entry, tok = segments_from_lengths((30, 20, 14), (0, 1, 2))
    return Workload("tiny", K, N, T, x, W0, entries, off, seg_entry, tok)


def decode_q_proj(seed: int = 0, split_versions: bool = False) -> Workload:
    """d_in = d_out = 4096, 8 tokens = 4 agents x 2.  Entries: 0 = (adapter 0, v1, old),
    1..3 = (adapters 1..3, v1), 4 = (adapter 0, v2, new).  Agent 0's two in-flight tokens
    stay on the old version; the new one is resident with no token.  split_versions=True
    puts one of agent 0's tokens on the new version instead."""
    K = N = 4096
    T = 8
    x, W0 = _base(seed, T, K, N)
    specs = [(0, 1, 16, 2.0), (1, 1, 16, 2.0), (2, 1, 16, 2.0), (3, 1, 16, 2.0), (0, 2, 16, 2.0)]
    entries = make_entries(seed, K, N, specs)
    if split_versions:
        off, seg_entry, tok = segments_from_lengths((1, 1, 2, 2, 2), (0, 4, 1, 2, 3))
    else:
        off, seg_entry, tok = segments_from_lengths((2, 2, 2, 2), (0, 1, 2, 3))
    return Workload("decode_q_proj", K, N, T, x, W0, entries, off, seg_entry, tok)


def prefill_q_proj(seed: int = 0) -> Workload:
    """d_in = d_out = 4096, 2048 tokens in segments 1024/512/384/128.  Entry 0 = (adapter 0,
    v2, freshly published) serves the 1024-token segment; entries 1..3 = adapters 1..3;
    entry 4 = (adapter 0, v1, old) stays resident with no token."""
    K = N = 4096
    T = 2048
    x, W0 = _base(seed, T, K, N)
    specs = [(0, 2, 16, 2.0), (1, 1, 16, 2.0), (2, 1, 16, 2.0), (3, 1, 16, 2.0), (0, 1, 16, 2.0)]
    entries = make_entries(seed, K, N, specs)
    off, seg_entry, tok = segments_from_lengths((1024, 512, 384, 128), (0, 1, 2, 3))
    return Workload("prefill_q_proj", K, N, T, x, W0, entries, off, seg_entry, tok)


def shuffle_rows(w: Workload, seed: int = 3) -> Workload:
    """The same batch with its rows in arrival order instead of grouped: row r of the result is a
    random row of `w`; perm / seg_offsets / seg_entry are the stable grouping of the shuffled
    per-token binding (what the token-segmentation pass has to produce)."""
    assert w.perm is None
    order = _rng(seed, _STREAM_ASSIGN + 2).permutation(w.T).astype(np.int32)
    tok = w.token_entry[order].astype(np.int32)
    perm, off, seg_entry = group_tokens(tok, len(w.entries))
    return Workload(w.name + "_shuffled", w.d_in, w.d_out, w.T, np.ascontiguousarray(w.x[order]), w.W0,
                    w.entries, off, seg_entry, tok, perm)


def zipf_assign(seed: int, stream: int, count: int, num: int, s: float) -> np.ndarray:
    """count i.i.d. draws from p_i proportional to (i+1)^-s over i = 0..num-1."""
    p = np.arange(1, num + 1, dtype=np.float64) ** (-s)
    p /= p.sum()
    return _rng(seed, stream).choice(num, size=count, p=p).astype(np.int32)


def mlp_up_gate(seed: int = 0, shuffled: bool = False, T: int = 4096, d_in: int = 4096,
                d_out: int = 11008) -> Workload:
    """d_in = 4096, d_out = 11008, 4096 tokens over 8 entries with ranks 8,16,32,64,8,16,32,64;
    10 % of the tokens (410 of 4096) carry no adapter, the rest draw their entry from
    Zipf(1.2).  shuffled=False: rows already grouped (contiguous segments, entries
    ascending, -1 last).  shuffled=True: rows in random order with a grouping perm, the
    form the token-segmentation pass produces."""
    K, N = d_in, d_out
    x, W0 = _base(seed, T, K, N)
    ranks = (8, 16, 32, 64, 8, 16, 32, 64)
    entries = make_entries(seed, K, N, [(i, 1, r, 2.0) for i, r in enumerate(ranks)])
    n_none = int(round(0.1 * T))
    tok_sorted = np.concatenate([
        np.sort(zipf_assign(seed, _STREAM_ASSIGN, T - n_none, len(ranks), 1.2)),
        np.full(n_none, -1, dtype=np.int32)]).astype(np.int32)
    if not shuffled:
        _, off, seg_entry = group_tokens(tok_sorted, len(ranks))
        return Workload("mlp_up_gate", K, N, T, x, W0, entries, off, seg_entry, tok_sorted)
    order = _rng(seed, _STREAM_ASSIGN + 1).permutation(T)
    tok = tok_sorted[order].astype(np.int32)
    perm, off, seg_entry = group_tokens(tok, len(ranks))
    return Workload("mlp_up_gate_shuffled", K, N, T, x, W0, entries, off, seg_entry, tok, perm)


LAYER_PROJECTIONS = {
    # name: (d_in, d_out)
    "q": (4096, 4096), "k": (4096, 4096), "v": (4096, 4096), "o": (4096, 4096),
    "gate": (4096, 11008), "up": (4096, 11008), "down": (11008, 4096),
}
SWEEP_TOKENS = (1, 16, 128, 1024, 8192)


def layer_sweep(proj: str, T: int, seed: int = 0) -> Workload:
    """One cell of the decoder-layer sweep: 16 adapters of rank 16 (scale 2.0), adapters 0
    and 1 resident in two versions each (18 entries); tokens draw their adapter from
    Zipf(1.1) and, for a two-version adapter, old or new with probability 1/2; rows are
    grouped by entry."""
    K, N = LAYER_PROJECTIONS[proj]
    pidx = list(LAYER_PROJECTIONS).index(proj)
    x, W0 = _base(seed + 7919 * (pidx + 1), T, K, N)
    specs = [(a, 1, 16, 2.0) for a in range(16)] + [(0, 2, 16, 2.0), (1, 2, 16, 2.0)]
    entries = make_entries(seed + 7919 * (pidx + 1), K, N, specs)
    adapter = zipf_assign(seed, _STREAM_ASSIGN + 10 + pidx, T, 16, 1.1)
    coin = _rng(seed, _STREAM_ASSIGN + 100 + pidx).integers(0, 2, size=T)
    entry = adapter.copy()
    entry[(adapter == 0) & (coin == 1)] = 16
    entry[(adapter == 1) & (coin == 1)] = 17
    tok = np.sort(entry).astype(np.int32)
    _, off, seg_entry = group_tokens(tok, len(specs))
    return Workload(f"sweep_{proj}_T{T}", K, N, T, x, W0, entries, off, seg_entry, tok)


def lattice(seed: int = 0, T: int = 200, d_in: int = 512, d_out: int = 384) -> Workload:
    """Rounding-free case: every entry of W0, A, B is in {-1, 0, 1}; each row of x has exactly
    16 non-zeros of +-1; rank 4, scale 1.  Every intermediate and every output is a small
    integer, exactly representable in bf16 and fp32, so any correct implementation must
    reproduce the outputs with zero error whatever its summation order."""
    K, N = d_in, d_out
    g = _rng(seed, _STREAM_X)
    xf = np.zeros((T, K), dtype=np.float32)
    for t in range(T):
        cols = g.choice(K, size=16, replace=False)
        xf[t, cols] = g.choice(np.array([-1.0, 1.0], dtype=np.float32), size=16)
    # keep |base| <= 16: at most one non-zero W0 entry is hit per non-zero of x anyway
    W0f = _rng(seed, _STREAM_W0).integers(-1, 2, size=(N, K)).astype(np.float32)
    entries = []
    for e in range(4):
        Af = _rng(seed, _STREAM_ADAPTER_A + e).integers(-1, 2, size=(4, K)).astype(np.float32)
        Bf = _rng(seed, _STREAM_ADAPTER_B + e).integers(-1, 2, size=(N, 4)).astype(np.float32)
        entries.append(AdapterEntry(e % 3, 1 + e // 3, 4, 1.0, f32_to_bf16_bits(Af), f32_to_bf16_bits(Bf)))
    l0, l2 = T // 3, T // 4
    l3 = min(17, T - l0 - l2)
    lens = (l0, 0, l2, l3, T - l0 - l2 - l3)
    off, seg_entry, tok = segments_from_lengths(lens, (0, 1, 3, -1, 2))
    return Workload("lattice", K, N, T, f32_to_bf16_bits(xf), f32_to_bf16_bits(W0f), entries,
                    off, seg_entry, tok)


def ragged(seed: int = 0, T: int = 333, d_in: int = 320, d_out: int = 456,
           ranks: Sequence[int] = (4, 16, 1, 33, 64), shuffled: bool = False) -> Workload:
    """Mid-size case for element-by-element parity: sizes that are not multiples of any
    tile, segments that cross row tiles, odd ranks, no-adapter rows, an empty segment and
    two segments on the same entry."""
    K, N = d_in, d_out
    x, W0 = _base(seed, T, K, N)
    entries = make_entries(seed, K, N, [(i, 1, r, 2.0) for i, r in enumerate(ranks)])
    ne = len(ranks)
    cuts = np.sort(_rng(seed, _STREAM_ASSIGN).integers(0, T + 1, size=ne + 2))
    bounds = np.concatenate([[0], cuts, [T]])
    lens = np.diff(bounds).tolist() + [0]
    ents = [i % ne for i in range(ne)] + [-1, 0, ne - 1, 1]
    lens = lens[: len(ents)]
    lens[-1] += T - sum(lens)
    off, seg_entry, tok_grouped = segments_from_lengths(lens, ents)
    if not shuffled:
        return Workload("ragged", K, N, T, x, W0, entries, off, seg_entry, tok_grouped)
    perm = _rng(seed, _STREAM_ASSIGN + 1).permutation(T).astype(np.int32)
    tok = np.empty(T, dtype=np.int32)
    tok[perm] = tok_grouped
    return Workload("ragged_shuffled", K, N, T, x, W0, entries, off, seg_entry, tok, perm)
