"""Thin ctypes binding of the C-ABI library (include/lora_mixed_linear.h).

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.
PyTorch supplies device memory and streams.  There is no CPU fallback: if the shared
library is missing, or a call returns an error status, this module raises.

Module-level functions carry the C names (lml_table_create, register_adapter,
retire_version, lml_segment_tokens, lora_mixed_linear, ...) and take raw pointers/ints;
`Table` wraps them for torch tensors.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblora_mixed_linear.so")

LML_OK = 0
STATUS_NAMES = {0: "LML_OK", 1: "LML_ERR_INVALID_ARG", 2: "LML_ERR_BAD_SLOT", 3: "LML_ERR_TABLE_FULL",
                4: "LML_ERR_DUPLICATE", 5: "LML_ERR_NOT_FOUND", 6: "LML_ERR_UNSUPPORTED",
                7: "LML_ERR_CUDA", 8: "LML_ERR_TIMEOUT", 9: "LML_ERR_WORKSPACE", 10: "LML_ERR_TOO_LARGE"}
FLAG_BAD_SLOT, FLAG_BAD_OFFSETS, FLAG_BAD_PERM, FLAG_TIMEOUT = 1, 2, 4, 8
MAX_SLOTS, MAX_RANK, DECODE_MAX_TOKENS, MAX_ADAPTER_IDS = 64, 64, 16, 4096
ERR_INVALID_ARG, ERR_BAD_SLOT, ERR_NOT_FOUND = 1, 2, 5

EXPORTS = ("lml_status_string", "lml_table_create", "lml_table_destroy", "register_adapter",
           "retire_version", "lml_lookup", "lml_slot_info", "lml_workspace_bytes",
           "lml_segment_tokens", "lora_mixed_linear", "lml_host_workspace_bytes",
           "lora_mixed_linear_host", "lml_device_status", "lml_last_launch_count",
           "lora_mixed_linear_decode_static", "lml_tokens_workspace_bytes", "lora_mixed_linear_tokens",
           "lml_publish", "lml_pin", "lml_unpin", "lml_resolve", "lml_slot_state",
           "lml_segment_tokens_adapters", "lora_mixed_linear_adapters",
           "lml_dual_workspace_bytes", "lora_mixed_linear_dual", "register_adapter_transposed",
           "lml_backward_workspace_bytes", "lora_mixed_linear_backward_adapters", "retire_version_on",
           "lml_multi_workspace_bytes", "lora_mixed_linear_multi")


class LmlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with "
                              "`python -m paper_2608_15241_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.lml_status_string.restype = ctypes.c_char_p
        L.lml_status_string.argtypes = [i32]
        L.lml_table_create.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32]
        L.lml_table_destroy.argtypes = [vp]
        L.register_adapter.argtypes = [vp, i32, i32, vp, vp, i32, ctypes.c_float, vp, ctypes.POINTER(i32)]
        L.retire_version.argtypes = [vp, i32, i32]
        L.retire_version_on.argtypes = [vp, i32, i32, vp]
        L.lml_lookup.argtypes = [vp, i32, i32, ctypes.POINTER(i32)]
        L.lml_slot_info.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                    ctypes.POINTER(ctypes.c_float)]
        L.lml_workspace_bytes.restype = sz
        L.lml_workspace_bytes.argtypes = [vp, i32, i32]
        L.lml_host_workspace_bytes.restype = sz
        L.lml_host_workspace_bytes.argtypes = [vp, i32, i32]
        L.lml_segment_tokens.argtypes = [vp, vp, i32, vp, vp, vp, vp]
        L.lora_mixed_linear.argtypes = [vp, vp, vp, i32, vp, vp, i32, vp, vp, vp, sz, vp]
        L.lora_mixed_linear_host.argtypes = [vp, vp, vp, i32, vp, vp, i32, vp, vp, vp, sz, vp]
        L.lora_mixed_linear_decode_static.argtypes = [vp, vp, vp, i32, vp, vp, i32, vp, vp, vp]
        L.lml_tokens_workspace_bytes.restype = sz
        L.lml_tokens_workspace_bytes.argtypes = [vp, i32]
        L.lora_mixed_linear_tokens.argtypes = [vp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.lora_mixed_linear_adapters.argtypes = [vp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.lml_segment_tokens_adapters.argtypes = [vp, vp, i32, vp, vp, vp, vp]
        L.register_adapter_transposed.argtypes = [vp, i32, i32, vp, vp, i32, ctypes.c_float, vp, ctypes.POINTER(i32)]
        L.lml_backward_workspace_bytes.restype = sz
        L.lml_backward_workspace_bytes.argtypes = [vp, i32, i32]
        L.lora_mixed_linear_backward_adapters.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.lml_dual_workspace_bytes.restype = sz
        L.lml_dual_workspace_bytes.argtypes = [vp, i32, i32]
        L.lora_mixed_linear_dual.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.lml_multi_workspace_bytes.restype = sz
        L.lml_multi_workspace_bytes.argtypes = [ctypes.POINTER(vp), i32, i32]
        L.lora_mixed_linear_multi.argtypes = [ctypes.POINTER(vp), i32, vp, ctypes.POINTER(vp), i32, ctypes.POINTER(vp),
                                              ctypes.POINTER(vp), vp, sz, vp]
        L.lml_publish.argtypes = [vp, i32, i32, vp, ctypes.POINTER(i32)]
        L.lml_pin.argtypes = [vp, i32]
        L.lml_unpin.argtypes = [vp, i32]
        L.lml_resolve.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.lml_slot_state.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.lml_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
        L.lml_last_launch_count.argtypes = [vp]
        for name in EXPORTS:
            if name not in ("lml_status_string", "lml_workspace_bytes", "lml_host_workspace_bytes",
                            "lml_tokens_workspace_bytes", "lml_dual_workspace_bytes", "lml_backward_workspace_bytes",
                            "lml_multi_workspace_bytes"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != LML_OK:
        raise LmlError(status, where)


# ---- C names, raw arguments ---------------------------------------------------------------------

def lml_status_string(status: int) -> str:
    return lib().lml_status_string(status).decode()


def lml_table_create(device: int, d_in: int, d_out: int, max_slots: int) -> int:
    h = ctypes.c_void_p()
    _check(lib().lml_table_create(ctypes.byref(h), device, d_in, d_out, max_slots), "lml_table_create")
    return h.value


def lml_table_destroy(table: int) -> None:
    _check(lib().lml_table_destroy(table), "lml_table_destroy")


def register_adapter(table: int, adapter_id: int, version: int, A_ptr: int, B_ptr: int, rank: int,
                     scale: float, stream: int = 0) -> int:
    slot = ctypes.c_int(-1)
    _check(lib().register_adapter(table, adapter_id, version, A_ptr, B_ptr, rank, scale, stream,
                                  ctypes.byref(slot)), "register_adapter")
    return slot.value


def retire_version(table: int, adapter_id: int, version: int) -> None:
    _check(lib().retire_version(table, adapter_id, version), "retire_version")


def retire_version_on(table: int, adapter_id: int, version: int, stream: int = 0) -> None:
    """retire_version whose device-side part (the serving entry leaves the adapter map) runs on `stream`."""
    _check(lib().retire_version_on(table, adapter_id, version, stream), "retire_version_on")


def lml_lookup(table: int, adapter_id: int, version: int) -> int:
    slot = ctypes.c_int(-1)
    _check(lib().lml_lookup(table, adapter_id, version, ctypes.byref(slot)), "lml_lookup")
    return slot.value


def lml_slot_info(table: int, slot: int) -> Tuple[int, int, int, float]:
    a, v, r, s = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_float()
    _check(lib().lml_slot_info(table, slot, ctypes.byref(a), ctypes.byref(v), ctypes.byref(r), ctypes.byref(s)),
           "lml_slot_info")
    return a.value, v.value, r.value, s.value


def lml_workspace_bytes(table: int, max_tokens: int, max_segments: int) -> int:
    return int(lib().lml_workspace_bytes(table, max_tokens, max_segments))


def lml_host_workspace_bytes(table: int, max_tokens: int, max_segments: int) -> int:
    return int(lib().lml_host_workspace_bytes(table, max_tokens, max_segments))


def lml_segment_tokens(table: int, token_slots_ptr: int, T: int, perm_ptr: int, seg_offsets_ptr: int,
                       seg_slot_ids_ptr: int, stream: int = 0) -> None:
    _check(lib().lml_segment_tokens(table, token_slots_ptr, T, perm_ptr, seg_offsets_ptr, seg_slot_ids_ptr,
                                    stream), "lml_segment_tokens")


def lora_mixed_linear(table: int, x_ptr: int, W0_ptr: int, T: int, seg_offsets_ptr: int, slot_ids_ptr: int,
                      G: int, perm_ptr: int, y_ptr: int, workspace_ptr: int, workspace_bytes: int,
                      stream: int = 0) -> None:
    _check(lib().lora_mixed_linear(table, x_ptr, W0_ptr, T, seg_offsets_ptr, slot_ids_ptr, G, perm_ptr, y_ptr,
                                   workspace_ptr, workspace_bytes, stream), "lora_mixed_linear")


def lora_mixed_linear_host(table: int, x_host_ptr: int, W0_ptr: int, T: int, seg_offsets_host_ptr: int,
                           slot_ids_host_ptr: int, G: int, perm_host_ptr: int, y_host_ptr: int,
                           workspace_ptr: int, workspace_bytes: int, stream: int = 0) -> None:
    _check(lib().lora_mixed_linear_host(table, x_host_ptr, W0_ptr, T, seg_offsets_host_ptr, slot_ids_host_ptr, G,
                                        perm_host_ptr, y_host_ptr, workspace_ptr, workspace_bytes, stream),
           "lora_mixed_linear_host")


def lml_tokens_workspace_bytes(table: int, max_tokens: int) -> int:
    return int(lib().lml_tokens_workspace_bytes(table, max_tokens))


def lora_mixed_linear_tokens(table: int, x_ptr: int, W0_ptr: int, T: int, token_slots_ptr: int, y_ptr: int,
                             workspace_ptr: int, workspace_bytes: int, stream: int = 0) -> None:
    """Segmentation and layer in one call: one slot id per token instead of segments."""
    _check(lib().lora_mixed_linear_tokens(table, x_ptr, W0_ptr, T, token_slots_ptr, y_ptr, workspace_ptr,
                                          workspace_bytes, stream), "lora_mixed_linear_tokens")


def _ptr_array(values):
    arr = (ctypes.c_void_p * len(values))()
    for i, v in enumerate(values):
        arr[i] = v
    return arr


def lml_multi_workspace_bytes(tables, max_tokens: int) -> int:
    return int(lib().lml_multi_workspace_bytes(_ptr_array(tables), len(tables), max_tokens))


def lora_mixed_linear_multi(tables, x_ptr: int, W0_ptrs, T: int, token_slots_ptrs, y_ptrs, workspace_ptr: int,
                            workspace_bytes: int, stream: int = 0) -> None:
    """Several projections of the same x in one call (table handles and per-projection pointers as lists)."""
    P = len(tables)
    assert len(W0_ptrs) == P and len(token_slots_ptrs) == P and len(y_ptrs) == P
    _check(lib().lora_mixed_linear_multi(_ptr_array(tables), P, x_ptr, _ptr_array(W0_ptrs), T,
                                         _ptr_array(token_slots_ptrs), _ptr_array(y_ptrs), workspace_ptr,
                                         workspace_bytes, stream), "lora_mixed_linear_multi")


def register_adapter_transposed(table_T: int, adapter_id: int, version: int, A_ptr: int, B_ptr: int, rank: int,
                                scale: float, stream: int = 0) -> int:
    """Register the forward adapter (A [rank][K], B [N][rank]) in the transposed table (d_in = N, d_out = K)."""
    slot = ctypes.c_int32(-1)
    _check(lib().register_adapter_transposed(table_T, adapter_id, version, A_ptr, B_ptr, rank, scale, stream,
                                             ctypes.byref(slot)), "register_adapter_transposed")
    return int(slot.value)


def lml_backward_workspace_bytes(table: int, max_tokens: int, max_segments: int) -> int:
    return int(lib().lml_backward_workspace_bytes(table, max_tokens, max_segments))


def lora_mixed_linear_backward_adapters(table: int, table_T: int, x_ptr: int, dy_ptr: int, T: int, seg_offsets_ptr: int,
                                        slot_ids_ptr: int, slot_ids_T_ptr: int, G: int, dA_ptr: int, dB_ptr: int,
                                        workspace_ptr: int, workspace_bytes: int, stream: int = 0) -> None:
    """dA, dB (fp32, packed like the arena) += this batch's adapter gradients."""
    _check(lib().lora_mixed_linear_backward_adapters(table, table_T, x_ptr, dy_ptr, T, seg_offsets_ptr, slot_ids_ptr,
                                                     slot_ids_T_ptr, G, dA_ptr, dB_ptr, workspace_ptr, workspace_bytes,
                                                     stream), "lora_mixed_linear_backward_adapters")


def lml_dual_workspace_bytes(table: int, max_tokens: int, max_segments: int) -> int:
    return int(lib().lml_dual_workspace_bytes(table, max_tokens, max_segments))


def lora_mixed_linear_dual(table: int, x_ptr: int, W0_ptr: int, T: int, seg_offsets_ptr: int, slot_ids_a_ptr: int,
                           slot_ids_b_ptr: int, G: int, perm_ptr: int, y_a_ptr: int, y_b_ptr: int, workspace_ptr: int,
                           workspace_bytes: int, stream: int = 0) -> None:
    """The same tokens under two slot bindings in one call; the base product is shared for T > 16."""
    _check(lib().lora_mixed_linear_dual(table, x_ptr, W0_ptr, T, seg_offsets_ptr, slot_ids_a_ptr, slot_ids_b_ptr, G,
                                        perm_ptr, y_a_ptr, y_b_ptr, workspace_ptr, workspace_bytes, stream),
           "lora_mixed_linear_dual")


STATE_RESIDENT, STATE_SERVING, STATE_RETIRING = 0, 1, 2


def lml_publish(table: int, adapter_id: int, version: int, stream: int = 0) -> int:
    """Make (adapter_id, version) the adapter's serving version from this point of the stream on.
    Returns the version that served before, or -1."""
    prev = ctypes.c_int32(-1)
    _check(lib().lml_publish(table, adapter_id, version, stream, ctypes.byref(prev)), "lml_publish")
    return int(prev.value)


def lml_pin(table: int, slot: int) -> None:
    _check(lib().lml_pin(table, slot), "lml_pin")


def lml_unpin(table: int, slot: int) -> None:
    _check(lib().lml_unpin(table, slot), "lml_unpin")


def lml_resolve(table: int, adapter_id: int):
    """(slot, version) of the adapter's serving entry; raises LmlError(NOT_FOUND) if none."""
    slot, ver = ctypes.c_int32(-1), ctypes.c_int32(-1)
    _check(lib().lml_resolve(table, adapter_id, ctypes.byref(slot), ctypes.byref(ver)), "lml_resolve")
    return int(slot.value), int(ver.value)


def lml_slot_state(table: int, slot: int):
    """(state, pins) of a live slot."""
    st, pins = ctypes.c_int32(-1), ctypes.c_int32(-1)
    _check(lib().lml_slot_state(table, slot, ctypes.byref(st), ctypes.byref(pins)), "lml_slot_state")
    return int(st.value), int(pins.value)


def lml_segment_tokens_adapters(table: int, token_adapter_ids_ptr: int, T: int, perm_ptr: int, seg_offsets_ptr: int,
                                seg_slot_ids_ptr: int, stream: int = 0) -> None:
    _check(lib().lml_segment_tokens_adapters(table, token_adapter_ids_ptr, T, perm_ptr, seg_offsets_ptr,
                                             seg_slot_ids_ptr, stream), "lml_segment_tokens_adapters")


def lora_mixed_linear_adapters(table: int, x_ptr: int, W0_ptr: int, T: int, token_adapter_ids_ptr: int, y_ptr: int,
                               workspace_ptr: int, workspace_bytes: int, stream: int = 0) -> None:
    """lora_mixed_linear_tokens with adapter ids, resolved on the device to each adapter's serving slot."""
    _check(lib().lora_mixed_linear_adapters(table, x_ptr, W0_ptr, T, token_adapter_ids_ptr, y_ptr, workspace_ptr,
                                            workspace_bytes, stream), "lora_mixed_linear_adapters")


def lora_mixed_linear_decode_static(table: int, x_ptr: int, W0_ptr: int, T: int, seg_offsets_ptr: int,
                                    slot_ids_ptr: int, G: int, perm_ptr: int, y_ptr: int, stream: int = 0) -> None:
    """Decode form (T <= 16) that takes no workspace: its scratch is a fixed array inside the
    library, so the call allocates nothing.  For callers that cannot obtain device memory."""
    _check(lib().lora_mixed_linear_decode_static(table, x_ptr, W0_ptr, T, seg_offsets_ptr, slot_ids_ptr, G,
                                                 perm_ptr, y_ptr, stream), "lora_mixed_linear_decode_static")


def lml_device_status(table: int, stream: int = 0) -> int:
    f = ctypes.c_uint32(0)
    _check(lib().lml_device_status(table, ctypes.byref(f), stream), "lml_device_status")
    return int(f.value)


def lml_last_launch_count(table: int) -> int:
    return int(lib().lml_last_launch_count(table))


# ---- torch convenience ------------------------------------------------------------------------------

def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _stream(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def fuse_projection_adapters(parts):
    """Adapters of several projections that read the same x (q/k/v, or gate/up) as ONE adapter of
    the projection with the concatenated weight: parts = [(A_p [r_p, d_in], B_p [d_out_p, r_p]), ...]
    gives A = cat(A_p) [sum r_p, d_in] and B = blockdiag(B_p) [sum d_out_p, sum r_p], so that
    x.W0cat + s (x.A^T).B^T equals the per-projection results side by side (same scale for all
    parts; sum r_p <= 64).  One call then reads x once and launches once instead of once per
    projection.  Layout plumbing only (torch cat / copy); the arithmetic stays in the kernels."""
    import torch
    A = torch.cat([a for a, _ in parts], dim=0).contiguous()
    rank = int(A.shape[0])
    assert rank <= MAX_RANK, "fused rank exceeds the table's maximum"
    n_total = sum(int(b.shape[0]) for _, b in parts)
    B = torch.zeros((n_total, rank), dtype=parts[0][1].dtype, device=parts[0][1].device)
    n0 = r0 = 0
    for a, b in parts:
        r, n = int(a.shape[0]), int(b.shape[0])
        B[n0:n0 + n, r0:r0 + r] = b
        n0 += n
        r0 += r
    return A, B


def multi_projection(tables, x, W0s, token_slots, ys=None, workspace=None, stream=None):
    """lora_mixed_linear_multi for torch tensors: tables = [Table, ...], W0s / token_slots per projection
    (token_slots may also be one tensor for all).  Returns the list of outputs."""
    import torch
    P, T = len(tables), int(x.shape[0])
    if not isinstance(token_slots, (list, tuple)):
        token_slots = [token_slots] * P
    if ys is None:
        ys = [torch.empty((T, t.d_out), dtype=torch.bfloat16, device=x.device) for t in tables]
    handles = [t.handle for t in tables]
    if workspace is None:
        workspace = torch.empty(max(lml_multi_workspace_bytes(handles, T), 256), dtype=torch.uint8, device=x.device)
    lora_mixed_linear_multi(handles, _ptr(x), [_ptr(w) for w in W0s], T, [_ptr(s) for s in token_slots],
                            [_ptr(y) for y in ys], _ptr(workspace), int(workspace.numel()), _stream(stream))
    return ys


class Table:
    """Adapter slot table of one linear site, for torch tensors (bf16 CUDA, contiguous)."""

    def __init__(self, d_in: int, d_out: int, max_slots: int = MAX_SLOTS, device: int = 0):
        self.d_in, self.d_out, self.max_slots, self.device = d_in, d_out, max_slots, device
        self.handle = lml_table_create(device, d_in, d_out, max_slots)
        self._ws = None

    def close(self) -> None:
        if self.handle:
            lml_table_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def register_adapter(self, adapter_id: int, version: int, A, B, scale: float, stream=None) -> int:
        import torch
        assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and A.is_cuda and B.is_cuda
        assert A.is_contiguous() and B.is_contiguous()
        rank = int(A.shape[0])
        assert A.shape == (rank, self.d_in) and B.shape == (self.d_out, rank), (A.shape, B.shape)
        return register_adapter(self.handle, adapter_id, version, _ptr(A), _ptr(B), rank, float(scale),
                                _stream(stream))

    def retire_version(self, adapter_id: int, version: int, stream="legacy") -> None:
        """stream="legacy": the C call retire_version (legacy default stream); a torch stream or None (the
        current stream): retire_version_on."""
        if isinstance(stream, str):
            retire_version(self.handle, adapter_id, version)
        else:
            retire_version_on(self.handle, adapter_id, version, _stream(stream))

    def lookup(self, adapter_id: int, version: int) -> int:
        return lml_lookup(self.handle, adapter_id, version)

    def slot_info(self, slot: int):
        return lml_slot_info(self.handle, slot)

    def workspace_bytes(self, max_tokens: int, max_segments: int) -> int:
        return lml_workspace_bytes(self.handle, max_tokens, max_segments)

    def workspace(self, T: int, G: int, host: bool = False):
        """A cached torch byte buffer large enough for (T, G); grown on demand (outside the hot call)."""
        import torch
        need = (lml_host_workspace_bytes if host else lml_workspace_bytes)(self.handle, T, G)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(max(need, 1024), dtype=torch.uint8, device=f"cuda:{self.device}")
        return self._ws

    def segment_tokens(self, token_slots, stream=None):
        """token_slots int32[T] (cuda) -> (perm int32[T], seg_offsets int32[max_slots+2],
        seg_slot_ids int32[max_slots+1]); G = max_slots + 1."""
        import torch
        assert token_slots.dtype == torch.int32 and token_slots.is_cuda and token_slots.is_contiguous()
        T = int(token_slots.shape[0])
        dev = token_slots.device
        perm = torch.empty(max(T, 1), dtype=torch.int32, device=dev)
        seg_offsets = torch.empty(self.max_slots + 2, dtype=torch.int32, device=dev)
        seg_slot_ids = torch.empty(self.max_slots + 1, dtype=torch.int32, device=dev)
        lml_segment_tokens(self.handle, _ptr(token_slots), T, _ptr(perm), _ptr(seg_offsets), _ptr(seg_slot_ids),
                           _stream(stream))
        return perm[:T], seg_offsets, seg_slot_ids

    def lora_mixed_linear(self, x, W0, seg_offsets, slot_ids, perm=None, y=None, workspace=None, stream=None):
        import torch
        assert x.dtype == torch.bfloat16 and W0.dtype == torch.bfloat16 and x.is_cuda and W0.is_cuda
        assert x.is_contiguous() and W0.is_contiguous()
        T = int(x.shape[0])
        assert x.shape[1] == self.d_in and W0.shape == (self.d_out, self.d_in)
        G = 0 if slot_ids is None else int(slot_ids.shape[0])
        if G:
            assert seg_offsets.dtype == torch.int32 and slot_ids.dtype == torch.int32
            assert seg_offsets.shape[0] == G + 1 and seg_offsets.is_cuda and slot_ids.is_cuda
        if perm is not None:
            assert perm.dtype == torch.int32 and perm.shape[0] == T and perm.is_cuda
        if y is None:
            y = torch.empty((T, self.d_out), dtype=torch.bfloat16, device=x.device)
        if workspace is None:
            workspace = self.workspace(T, G)
        lora_mixed_linear(self.handle, _ptr(x), _ptr(W0), T, _ptr(seg_offsets) if G else 0,
                          _ptr(slot_ids) if G else 0, G, _ptr(perm), _ptr(y), _ptr(workspace),
                          int(workspace.numel()), _stream(stream))
        return y

    def publish(self, adapter_id: int, version: int, stream=None) -> int:
        return lml_publish(self.handle, adapter_id, version, _stream(stream))

    def pin(self, slot: int) -> None:
        lml_pin(self.handle, slot)

    def unpin(self, slot: int) -> None:
        lml_unpin(self.handle, slot)

    def resolve(self, adapter_id: int):
        return lml_resolve(self.handle, adapter_id)

    def slot_state(self, slot: int):
        return lml_slot_state(self.handle, slot)

    def register_adapter_transposed(self, adapter_id: int, version: int, A, B, scale: float, stream=None) -> int:
        """On the TRANSPOSED table (d_in = N, d_out = K): A [rank][K], B [N][rank] of the forward layer."""
        rank = int(A.shape[0])
        assert A.shape[1] == self.d_out and B.shape == (self.d_in, rank)
        return register_adapter_transposed(self.handle, adapter_id, version, _ptr(A), _ptr(B), rank, float(scale),
                                           _stream(stream))

    def backward_adapters(self, table_T, x, dy, seg_offsets, slot_ids, slot_ids_T, dA, dB, stream=None):
        """dA fp32 [max_slots][64][d_in], dB fp32 [max_slots][d_out][64] += gradients of this batch."""
        import torch
        T, G = int(x.shape[0]), int(slot_ids.shape[0])
        assert dA.dtype == torch.float32 and dB.dtype == torch.float32
        assert tuple(dA.shape) == (self.max_slots, 64, self.d_in) and tuple(dB.shape) == (self.max_slots, self.d_out, 64)
        ws = torch.empty(max(lml_backward_workspace_bytes(self.handle, T, G), 256), dtype=torch.uint8, device=x.device)
        lora_mixed_linear_backward_adapters(self.handle, table_T.handle, _ptr(x), _ptr(dy), T, _ptr(seg_offsets),
                                            _ptr(slot_ids), _ptr(slot_ids_T), G, _ptr(dA), _ptr(dB), _ptr(ws),
                                            int(ws.numel()), _stream(stream))

    def lora_mixed_linear_dual(self, x, W0, seg_offsets, slot_ids_a, slot_ids_b, perm=None, stream=None):
        """-> (y_a, y_b): the layer under two slot bindings of the same segments."""
        import torch
        T, G = int(x.shape[0]), int(slot_ids_a.shape[0])
        assert slot_ids_b.shape[0] == G and seg_offsets.shape[0] == G + 1
        y_a = torch.empty((T, self.d_out), dtype=torch.bfloat16, device=x.device)
        y_b = torch.empty_like(y_a)
        ws = torch.empty(max(lml_dual_workspace_bytes(self.handle, T, G), 256), dtype=torch.uint8, device=x.device)
        lora_mixed_linear_dual(self.handle, _ptr(x), _ptr(W0), T, _ptr(seg_offsets), _ptr(slot_ids_a), _ptr(slot_ids_b),
                               G, _ptr(perm), _ptr(y_a), _ptr(y_b), _ptr(ws), int(ws.numel()), _stream(stream))
        return y_a, y_b

    def lora_mixed_linear_adapters(self, x, W0, token_adapter_ids, y=None, workspace=None, stream=None):
        """As lora_mixed_linear_tokens, with one ADAPTER id per token (resolved on the device)."""
        return self.lora_mixed_linear_tokens(x, W0, token_adapter_ids, y, workspace, stream, by_adapter=True)

    def lora_mixed_linear_tokens(self, x, W0, token_slots, y=None, workspace=None, stream=None, by_adapter=False):
        """x bf16 [T][d_in], W0 bf16 [d_out][d_in], token_slots int32[T] (all cuda) -> y bf16 [T][d_out]."""
        import torch
        assert x.dtype == torch.bfloat16 and W0.dtype == torch.bfloat16 and token_slots.dtype == torch.int32
        assert x.is_cuda and W0.is_cuda and token_slots.is_cuda and x.is_contiguous() and W0.is_contiguous()
        T = int(x.shape[0])
        assert token_slots.shape[0] == T and x.shape[1] == self.d_in and W0.shape == (self.d_out, self.d_in)
        if y is None:
            y = torch.empty((T, self.d_out), dtype=torch.bfloat16, device=x.device)
        if workspace is None:
            workspace = torch.empty(max(lml_tokens_workspace_bytes(self.handle, T), 256), dtype=torch.uint8,
                                    device=x.device)
        fn = lora_mixed_linear_adapters if by_adapter else lora_mixed_linear_tokens
        fn(self.handle, _ptr(x), _ptr(W0), T, _ptr(token_slots), _ptr(y), _ptr(workspace), int(workspace.numel()),
           _stream(stream))
        return y

    def lora_mixed_linear_host(self, x_host, W0, seg_offsets_host, slot_ids_host, y_host, perm_host=None,
                               workspace=None, stream=None):
        """x_host / y_host: CPU bf16 tensors (pinned for asynchronous copies); W0 on the device."""
        T = int(x_host.shape[0])
        G = 0 if slot_ids_host is None else int(slot_ids_host.shape[0])
        assert not x_host.is_cuda and not y_host.is_cuda and W0.is_cuda
        if workspace is None:
            workspace = self.workspace(T, G, host=True)
        lora_mixed_linear_host(self.handle, _ptr(x_host), _ptr(W0), T, _ptr(seg_offsets_host) if G else 0,
                               _ptr(slot_ids_host) if G else 0, G, _ptr(perm_host), _ptr(y_host),
                               _ptr(workspace), int(workspace.numel()), _stream(stream))
        return y_host

    def device_status(self, stream=None) -> int:
        return lml_device_status(self.handle, _stream(stream))

    def last_launch_count(self) -> int:
        return lml_last_launch_count(self.handle)
