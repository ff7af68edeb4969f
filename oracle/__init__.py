"""ctypes front end of the fp64 CPU oracle (oracle/lml_oracle.c).

TEST INFRASTRUCTURE ONLY.  Nothing in the CUDA package imports this; only tests, the
smoke check and the benchmark's CPU-baseline leg may.  It shares no code with the CUDA
path: inputs arrive as numpy uint16 (bf16 bit patterns) and int32 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lml_oracle.c")
_LIB = os.path.join(_HERE, "liblml_oracle.so")

FLAG_BAD_SLOT = 1
FLAG_BAD_OFFSETS = 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no fp contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.lml_oracle_forward.restype = ctypes.c_int
        _lib.lml_oracle_forward_brute.restype = ctypes.c_int
        _lib.lml_oracle_backward.restype = ctypes.c_int
        _lib.lml_oracle_segment.restype = ctypes.c_int
        _lib.lml_oracle_threads.restype = ctypes.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _entry_arrays(entries, K, N):
    ne = len(entries)
    keep = []
    Ap = (ctypes.c_void_p * max(ne, 1))()
    Bp = (ctypes.c_void_p * max(ne, 1))()
    rank = np.zeros(max(ne, 1), dtype=np.int32)
    scale = np.zeros(max(ne, 1), dtype=np.float32)
    for i, e in enumerate(entries):
        A = _u16(e.A)
        B = _u16(e.B)
        assert A.shape == (e.rank, K) and B.shape == (N, e.rank), (A.shape, B.shape)
        keep += [A, B]
        Ap[i] = A.ctypes.data
        Bp[i] = B.ctypes.data
        rank[i] = e.rank
        scale[i] = e.scale
    return Ap, Bp, rank, scale, keep


def threads() -> int:
    return int(_load().lml_oracle_threads())


def forward(x, W0, entries, seg_offsets, seg_entry, perm=None, positions=None, live=None,
            nthreads: int = 0, out: Optional[np.ndarray] = None):
    """fp64 reference output.  Returns (y64 [T, N] float64, flags).  With `positions`, only
    the rows those positions address are computed (the others stay zero / untouched)."""
    lib = _load()
    x = _u16(x)
    W0 = _u16(W0)
    T, K = x.shape
    N = W0.shape[0]
    assert W0.shape == (N, K)
    Ap, Bp, rank, scale, keep = _entry_arrays(entries, K, N)
    ne = len(entries)
    live_a = np.ones(max(ne, 1), dtype=np.int32) if live is None else _i32(live)
    so = _i32(seg_offsets)
    se = _i32(seg_entry)
    G = int(se.shape[0])
    assert so.shape[0] == G + 1 or G == 0
    pm = None if perm is None else _i32(perm)
    pos = None if positions is None else _i32(positions)
    y = np.zeros((T, N), dtype=np.float64) if out is None else out
    flags = ctypes.c_uint32(0)
    rc = lib.lml_oracle_forward(_p(x), _p(W0), T, K, N, ne, Ap, Bp, _p(rank), _p(scale), _p(live_a),
                                G, _p(so), _p(se), _p(pm), _p(pos),
                                0 if pos is None else int(pos.shape[0]),
                                _p(y), ctypes.byref(flags), int(nthreads))
    if rc != 0:
        raise ValueError("lml_oracle_forward: invalid argument")
    del keep
    return y, int(flags.value)


def forward_workload(w, positions=None, nthreads: int = 0):
    return forward(w.x, w.W0, w.entries, w.seg_offsets, w.seg_entry, w.perm, positions,
                   nthreads=nthreads)


def backward(x, dy, W0, entries, seg_offsets, seg_entry, perm=None, live=None):
    """fp64 reference gradients of the layer.  Returns (dx [T, K], [dA_e [rank_e, K]], [dB_e [N, rank_e]], flags)."""
    lib = _load()
    x, dy, W0 = _u16(x), _u16(dy), _u16(W0)
    T, K = x.shape
    N = W0.shape[0]
    assert W0.shape == (N, K) and dy.shape == (T, N)
    Ap, Bp, rank, scale, keep = _entry_arrays(entries, K, N)
    ne = len(entries)
    live_a = np.ones(max(ne, 1), dtype=np.int32) if live is None else _i32(live)
    so, se = _i32(seg_offsets), _i32(seg_entry)
    pm = None if perm is None else _i32(perm)
    dx = np.zeros((T, K), dtype=np.float64)
    dA = [np.zeros((e.rank, K), dtype=np.float64) for e in entries]
    dB = [np.zeros((N, e.rank), dtype=np.float64) for e in entries]
    PP = ctypes.c_void_p * max(ne, 1)
    dAp = PP(*[a.ctypes.data for a in dA]) if ne else PP()
    dBp = PP(*[b.ctypes.data for b in dB]) if ne else PP()
    flags = ctypes.c_uint32(0)
    rc = lib.lml_oracle_backward(_p(x), _p(dy), _p(W0), T, K, N, ne, Ap, Bp, _p(rank), _p(scale), _p(live_a),
                                 int(se.shape[0]), _p(so), _p(se), _p(pm), _p(dx), dAp, dBp, ctypes.byref(flags))
    del keep
    if rc != 0:
        raise ValueError("lml_oracle_backward: bad argument")
    return dx, dA, dB, int(flags.value)


def forward_brute(x, W0, entries, seg_offsets, seg_entry, perm=None):
    lib = _load()
    x = _u16(x)
    W0 = _u16(W0)
    T, K = x.shape
    N = W0.shape[0]
    Ap, Bp, rank, scale, keep = _entry_arrays(entries, K, N)
    so, se = _i32(seg_offsets), _i32(seg_entry)
    pm = None if perm is None else _i32(perm)
    y = np.zeros((T, N), dtype=np.float64)
    lib.lml_oracle_forward_brute(_p(x), _p(W0), T, K, N, len(entries), Ap, Bp, _p(rank), _p(scale),
                                 int(se.shape[0]), _p(so), _p(se), _p(pm), _p(y))
    del keep
    return y


def segment(token_entry: Sequence[int], num_entries: int):
    """Reference token grouping.  Returns (perm, seg_offsets, seg_entry, flags)."""
    lib = _load()
    te = _i32(token_entry)
    T = int(te.shape[0])
    perm = np.zeros(max(T, 1), dtype=np.int32)
    so = np.zeros(num_entries + 2, dtype=np.int32)
    se = np.zeros(num_entries + 1, dtype=np.int32)
    ns = ctypes.c_int32(0)
    flags = ctypes.c_uint32(0)
    lib.lml_oracle_segment(_p(te), T, int(num_entries), _p(perm), _p(so), _p(se),
                           ctypes.byref(ns), ctypes.byref(flags))
    n = int(ns.value)
    return perm[:T].copy(), so[: n + 1].copy(), se[:n].copy(), int(flags.value)


def compare(y_gpu_bf16_bits: np.ndarray, y64: np.ndarray, rows=None):
    """The parity criterion: per element |g - o| <= 1e-2 * max(1, |o|) and relative Frobenius
    error <= 5e-3.  y_gpu is bf16 bit patterns.  Returns a dict of the measured figures."""
    g16 = np.ascontiguousarray(y_gpu_bf16_bits, dtype=np.uint16)
    g = (g16.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    o = y64
    if rows is not None:
        g = g[rows]
        o = o[rows]
    diff = np.abs(g - o)
    tol = 1e-2 * np.maximum(1.0, np.abs(o))
    worst = float((diff / tol).max()) if diff.size else 0.0
    den = float(np.sqrt((o * o).sum()))
    fro = float(np.sqrt((diff * diff).sum())) / den if den > 0 else float(np.sqrt((diff * diff).sum()))
    return {"max_abs": float(diff.max()) if diff.size else 0.0, "worst_tol_ratio": worst,
            "rel_fro": fro, "ok": bool(worst <= 1.0 and fro <= 5e-3)}
