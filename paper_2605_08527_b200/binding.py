"""Python binding of the C-ABI library: same names as include/marlaas.h, argument marshalling only.

Every step of the layer runs in the library's CUDA kernels; torch is used here for device memory
(tensors own the buffers) and for the current stream.  There is no CPU fallback: if the library is
missing or the device is not a B200-class (sm_100) GPU, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmarlaas.so")

MARLAAS_OK = 0
MARLAAS_ERR_INVALID_ARG = -1
MARLAAS_ERR_BAD_SEGMENT_TABLE = -2
MARLAAS_ERR_UNKNOWN_TENANT = -3
MARLAAS_ERR_RANK_TOO_LARGE = -4
MARLAAS_ERR_POOL_FULL = -5
MARLAAS_ERR_UNSUPPORTED_DEVICE = -6
MARLAAS_ERR_CUDA = -7
MARLAAS_ERR_DEVICE_TIMEOUT = -8
MARLAAS_ERR_DEVICE_BAD_INDEX = -9
MARLAAS_ERR_WORKSPACE_TOO_SMALL = -10

MARLAAS_FLAG_ACCUMULATE = 1
MARLAAS_FLAG_HOST_TABLE = 2
MARLAAS_FLAG_VALIDATE_SYNC = 4
MARLAAS_FLAG_CUDA_CORE_PATH = 8
MARLAAS_FLAG_REUSE_PLAN = 16
MARLAAS_FLAG_OVERLAP_PREVIOUS = 32

EXPORTED_SYMBOLS = [
    "marlaas_adapter_pool_storage_bytes", "marlaas_adapter_pool_create", "marlaas_adapter_pool_destroy",
    "marlaas_adapter_pool_register", "marlaas_adapter_pool_unregister", "marlaas_adapter_pool_lookup",
    "marlaas_adapter_pool_export", "marlaas_adapter_pool_rank_stride", "marlaas_lora_workspace_bytes",
    "marlaas_lora_forward_workspace_bytes", "marlaas_debug_wait_runs_out", "marlaas_lora_forward_multi",
    "marlaas_lora_forward", "marlaas_lora_backward", "marlaas_lora_build_index", "marlaas_check_status",
    "marlaas_last_error", "marlaas_kernel_launch_count", "marlaas_kernel_timing_begin", "marlaas_kernel_timing_end",
    "marlaas_lora_static_workspace_limit", "marlaas_lora_forward_static_ws", "marlaas_adapter_pool_adamw_commit",
    "marlaas_lora_forward_workspace_min_bytes", "marlaas_adapter_pool_storage_bytes_segmented", "marlaas_adapter_pool_create_segmented", "marlaas_adapter_pool_parts",
]


class MarlaasError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"marlaas status {status}: {message}")
        self.status = status


class marlaas_adamw_t(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
                ("weight_decay", ctypes.c_float), ("grad_scale", ctypes.c_float), ("step", ctypes.c_int64)]


class marlaas_segments_t(ctypes.Structure):
    _fields_ = [("num_segments", ctypes.c_int32), ("seg_offsets", ctypes.c_void_p), ("seg_slot", ctypes.c_void_p)]


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """dlopen the in-tree libmarlaas.so (built by paper_2605_08527_b200/build.py); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise MarlaasError(MARLAAS_ERR_CUDA, f"{LIB_PATH} is not built; run `python -m paper_2605_08527_b200.build` "
                           "(needs nvcc); there is no fallback path")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u32, u64, f32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32,
                                       ctypes.c_uint64, ctypes.c_float, ctypes.c_size_t)
    P = ctypes.POINTER
    L.marlaas_adapter_pool_storage_bytes.restype = sz
    L.marlaas_adapter_pool_storage_bytes.argtypes = [i64, i64, i32, i32]
    L.marlaas_adapter_pool_create.restype = i32
    L.marlaas_adapter_pool_create.argtypes = [P(vp), ctypes.c_int, i64, i64, i32, i32, vp, sz, vp]
    L.marlaas_adapter_pool_destroy.restype = i32
    L.marlaas_adapter_pool_destroy.argtypes = [vp]
    L.marlaas_adapter_pool_storage_bytes_segmented.restype = sz
    L.marlaas_adapter_pool_storage_bytes_segmented.argtypes = [i64, i32, P(i64), i32, i32]
    L.marlaas_adapter_pool_create_segmented.restype = i32
    L.marlaas_adapter_pool_create_segmented.argtypes = [P(vp), ctypes.c_int, i64, i32, P(i64), i32, i32, vp, sz, vp]
    L.marlaas_adapter_pool_parts.restype = i32
    L.marlaas_adapter_pool_parts.argtypes = [vp]
    L.marlaas_adapter_pool_register.restype = i32
    L.marlaas_adapter_pool_register.argtypes = [vp, u64, u64, i32, f32, vp, vp, P(i32), vp]
    L.marlaas_adapter_pool_unregister.restype = i32
    L.marlaas_adapter_pool_unregister.argtypes = [vp, u64, vp]
    L.marlaas_adapter_pool_lookup.restype = i32
    L.marlaas_adapter_pool_lookup.argtypes = [vp, u64, P(i32), P(i32), P(f32), P(u64)]
    L.marlaas_adapter_pool_export.restype = i32
    L.marlaas_adapter_pool_export.argtypes = [vp, i32, vp, vp, vp]
    L.marlaas_adapter_pool_adamw_commit.restype = i32
    L.marlaas_adapter_pool_adamw_commit.argtypes = [vp, i32, P(u64), P(u64)] + [P(vp)] * 8 + [P(marlaas_adamw_t), vp]
    L.marlaas_adapter_pool_rank_stride.restype = i32
    L.marlaas_adapter_pool_rank_stride.argtypes = [vp]
    L.marlaas_lora_workspace_bytes.restype = sz
    L.marlaas_lora_workspace_bytes.argtypes = [vp, i64]
    L.marlaas_lora_forward_workspace_bytes.restype = sz
    L.marlaas_lora_forward_workspace_bytes.argtypes = [vp, i64]
    L.marlaas_lora_forward_workspace_min_bytes.restype = sz
    L.marlaas_lora_forward_workspace_min_bytes.argtypes = [vp, i64]
    L.marlaas_lora_forward.restype = i32
    L.marlaas_lora_forward.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, P(marlaas_segments_t), vp, vp, sz, u32, vp]
    L.marlaas_lora_static_workspace_limit.restype = sz
    L.marlaas_lora_static_workspace_limit.argtypes = []
    L.marlaas_lora_forward_static_ws.restype = i32
    L.marlaas_lora_forward_static_ws.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, P(marlaas_segments_t), vp, u32, vp]
    L.marlaas_lora_backward.restype = i32
    L.marlaas_lora_backward.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, vp,
                                        P(marlaas_segments_t), vp, vp, sz, u32, vp]
    L.marlaas_lora_build_index.restype = i32
    L.marlaas_lora_build_index.argtypes = [vp, i64, P(marlaas_segments_t), vp, vp, vp, vp, vp, sz, u32, vp]
    L.marlaas_check_status.restype = i32
    L.marlaas_check_status.argtypes = [vp, vp]
    L.marlaas_lora_forward_multi.restype = i32
    L.marlaas_lora_forward_multi.argtypes = [ctypes.c_int32, vp, ctypes.c_uint32, vp]
    L.marlaas_debug_wait_runs_out.restype = i32
    L.marlaas_debug_wait_runs_out.argtypes = [vp, ctypes.c_uint64, vp]
    L.marlaas_kernel_timing_begin.restype = i32
    L.marlaas_kernel_timing_begin.argtypes = [vp]
    L.marlaas_kernel_timing_end.restype = i32
    L.marlaas_kernel_timing_end.argtypes = [vp, P(f32), P(i32)]
    L.marlaas_last_error.restype = ctypes.c_char_p
    L.marlaas_last_error.argtypes = []
    L.marlaas_kernel_launch_count.restype = u64
    L.marlaas_kernel_launch_count.argtypes = []
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != MARLAAS_OK:
        raise MarlaasError(rc, load_library().marlaas_last_error().decode())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _dptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(None if t is None else t.data_ptr())


def marlaas_last_error() -> str:
    return load_library().marlaas_last_error().decode()


def marlaas_kernel_launch_count() -> int:
    return int(load_library().marlaas_kernel_launch_count())


class marlaas_forward_call_t(ctypes.Structure):
    _fields_ = [("pool", ctypes.c_void_p), ("T", ctypes.c_int64), ("x", ctypes.c_void_p), ("ldx", ctypes.c_int64),
                ("W", ctypes.c_void_p), ("ldw", ctypes.c_int64), ("y", ctypes.c_void_p), ("ldy", ctypes.c_int64),
                ("seg", ctypes.c_void_p), ("h_save", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t)]


class Segments:
    """The token-to-adapter segment table of one mixed batch (int32 tensors, on the device or -- with
    MARLAAS_FLAG_HOST_TABLE -- on the host)."""

    def __init__(self, seg_offsets: torch.Tensor, seg_slot: torch.Tensor):
        assert seg_offsets.dtype == torch.int32 and seg_slot.dtype == torch.int32
        assert seg_offsets.is_contiguous() and seg_slot.is_contiguous()
        assert seg_offsets.numel() == seg_slot.numel() + 1
        assert seg_offsets.device == seg_slot.device
        self.seg_offsets, self.seg_slot = seg_offsets, seg_slot
        self.on_host = seg_offsets.device.type == "cpu"
        self.c = marlaas_segments_t(seg_slot.numel(), seg_offsets.data_ptr(), seg_slot.data_ptr())

    @property
    def flags(self) -> int:
        return MARLAAS_FLAG_HOST_TABLE if self.on_host else 0


class AdapterPool:
    """marlaas_pool_t plus the torch tensor that owns its device storage.  With `parts` (the widths of several
    projections that read the same activations) the pool is made by marlaas_adapter_pool_create_segmented and d_out
    is their sum."""

    def __init__(self, d_in: int, d_out: int, max_rank: int, capacity: int, device="cuda:0", stream=None,
                 parts: Optional[Sequence[int]] = None):
        L = load_library()
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise MarlaasError(MARLAAS_ERR_UNSUPPORTED_DEVICE, "the layer runs on a CUDA device only")
        idx = self.device.index if self.device.index is not None else torch.cuda.current_device()
        self.parts = None if parts is None else [int(p) for p in parts]
        if self.parts is not None:
            assert d_out == sum(self.parts)
        self.n_parts = 1 if self.parts is None else len(self.parts)
        self.d_in, self.d_out, self.max_rank, self.capacity = d_in, d_out, max_rank, capacity
        if self.parts is None:
            nbytes = L.marlaas_adapter_pool_storage_bytes(d_in, d_out, max_rank, capacity)
        else:
            widths = (ctypes.c_int64 * len(self.parts))(*self.parts)
            nbytes = L.marlaas_adapter_pool_storage_bytes_segmented(d_in, len(self.parts), widths, max_rank, capacity)
        if nbytes == 0:
            raise MarlaasError(MARLAAS_ERR_INVALID_ARG, "invalid pool dimensions")
        with torch.cuda.device(idx):
            self.storage = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            h = ctypes.c_void_p()
            if self.parts is None:
                _check(L.marlaas_adapter_pool_create(ctypes.byref(h), idx, d_in, d_out, max_rank, capacity,
                                                     _dptr(self.storage), nbytes, _stream(stream)))
            else:
                _check(L.marlaas_adapter_pool_create_segmented(ctypes.byref(h), idx, d_in, len(self.parts), widths, max_rank,
                                                               capacity, _dptr(self.storage), nbytes, _stream(stream)))
        self.handle = h
        self.rank_stride = int(L.marlaas_adapter_pool_rank_stride(h))
        self._workspaces = {}

    def close(self):
        if getattr(self, "handle", None):
            load_library().marlaas_adapter_pool_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, T: int) -> torch.Tensor:
        """A cached workspace tensor large enough for T tokens (one per pool; not for overlapping calls)."""
        need = marlaas_lora_workspace_bytes(self, T)
        ws = self._workspaces.get("ws")
        if ws is None or ws.numel() < need:
            ws = torch.empty(need, dtype=torch.uint8, device=self.device)
            self._workspaces["ws"] = ws
        return ws


def marlaas_adapter_pool_register(pool: AdapterPool, tenant_id: int, version: int, rank: int, alpha: float,
                                  A: Optional[torch.Tensor], B: Optional[torch.Tensor], stream=None) -> int:
    if rank > 0 and pool.parts is not None:
        # one pair per projection, handed to the library as blocks one after another
        assert len(A) == pool.n_parts and len(B) == pool.n_parts
        for p in range(pool.n_parts):
            assert tuple(A[p].shape) == (pool.d_in, rank) and tuple(B[p].shape) == (rank, pool.parts[p])
        A = torch.cat([a.contiguous().reshape(-1) for a in A])
        B = torch.cat([b.contiguous().reshape(-1) for b in B])
        assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and A.device == pool.device and B.device == pool.device
    elif rank > 0:
        assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and A.is_contiguous() and B.is_contiguous()
        assert tuple(A.shape) == (pool.d_in, rank) and tuple(B.shape) == (rank, pool.d_out)
        assert A.device == pool.device and B.device == pool.device
    slot = ctypes.c_int32(-1)
    _check(load_library().marlaas_adapter_pool_register(pool.handle, tenant_id, version, rank, alpha, _dptr(A), _dptr(B),
                                                        ctypes.byref(slot), _stream(stream)))
    return int(slot.value)


def marlaas_adapter_pool_adamw_commit(pool: AdapterPool, tenant_ids: Sequence[int], dA, dB, A, B, m_A, v_A, m_B, v_B, *,
                                      lr: float, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                                      weight_decay: float = 0.0, grad_scale: float = 1.0, step: int = 1,
                                      new_versions: Optional[Sequence[int]] = None, stream=None) -> None:
    """AdamW on the fp32 masters of the listed tenants and commit of their bf16 rounding into the pool.  Each of the
    eight arguments dA .. v_B is a list (one entry per tenant) of contiguous fp32 device tensors, updated in place
    (A, m_A, v_A: [d_in][rank]; B, m_B, v_B: [rank][d_out])."""
    n = len(tenant_ids)
    tables = []
    for name, lst in (("dA", dA), ("dB", dB), ("A", A), ("B", B), ("m_A", m_A), ("v_A", v_A), ("m_B", m_B), ("v_B", v_B)):
        assert len(lst) == n, name
        tab = (ctypes.c_void_p * max(n, 1))()
        for i, t in enumerate(lst):
            assert t.dtype == torch.float32 and t.is_contiguous() and t.device == pool.device, name
            tab[i] = t.data_ptr()
        tables.append(tab)
    ids = (ctypes.c_uint64 * max(n, 1))(*tenant_ids)
    vers = None if new_versions is None else (ctypes.c_uint64 * max(n, 1))(*new_versions)
    hp = marlaas_adamw_t(lr, beta1, beta2, eps, weight_decay, grad_scale, step)
    _check(load_library().marlaas_adapter_pool_adamw_commit(pool.handle, n, ids, vers, *tables, ctypes.byref(hp),
                                                            _stream(stream)))


def marlaas_adapter_pool_unregister(pool: AdapterPool, tenant_id: int, stream=None) -> None:
    _check(load_library().marlaas_adapter_pool_unregister(pool.handle, tenant_id, _stream(stream)))


def marlaas_adapter_pool_lookup(pool: AdapterPool, tenant_id: int):
    s, r, sc, v = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_float(), ctypes.c_uint64()
    _check(load_library().marlaas_adapter_pool_lookup(pool.handle, tenant_id, ctypes.byref(s), ctypes.byref(r),
                                                      ctypes.byref(sc), ctypes.byref(v)))
    return int(s.value), int(r.value), float(sc.value), int(v.value)


def marlaas_adapter_pool_export(pool: AdapterPool, slot: int, rank: int, stream=None):
    """The slot's adapter in the caller's layout; for a pool over several projections, two lists (one A and one B per
    projection)."""
    A = torch.empty((pool.n_parts * pool.d_in, rank), dtype=torch.bfloat16, device=pool.device)
    B = torch.empty(rank * pool.d_out, dtype=torch.bfloat16, device=pool.device)
    _check(load_library().marlaas_adapter_pool_export(pool.handle, slot, _dptr(A), _dptr(B), _stream(stream)))
    if pool.parts is None:
        return A, B.view(rank, pool.d_out)
    As = [A[p * pool.d_in:(p + 1) * pool.d_in] for p in range(pool.n_parts)]
    Bs, o = [], 0
    for w in pool.parts:
        Bs.append(B[o:o + rank * w].view(rank, w))
        o += rank * w
    return As, Bs


def marlaas_lora_workspace_bytes(pool: AdapterPool, T: int) -> int:
    return int(load_library().marlaas_lora_workspace_bytes(pool.handle, T))


def marlaas_lora_forward_workspace_bytes(pool: AdapterPool, T: int) -> int:
    return int(load_library().marlaas_lora_forward_workspace_bytes(pool.handle, T))


def marlaas_lora_forward_workspace_min_bytes(pool: AdapterPool, T: int) -> int:
    return int(load_library().marlaas_lora_forward_workspace_min_bytes(pool.handle, T))


def _mat(t: torch.Tensor, cols: int, name: str):
    assert t.dtype == torch.bfloat16 and t.dim() == 2 and t.shape[1] == cols and t.stride(1) == 1, name
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), cols)


def marlaas_lora_forward(pool: AdapterPool, x: torch.Tensor, W: torch.Tensor, seg: Segments,
                         y: Optional[torch.Tensor] = None, h_save: Optional[torch.Tensor] = None,
                         workspace: Optional[torch.Tensor] = None, flags: int = 0, stream=None) -> torch.Tensor:
    T = x.shape[0]
    if y is None:
        y = torch.empty((T, pool.d_out), dtype=torch.bfloat16, device=x.device)
    ws = workspace if workspace is not None else pool.workspace(T)
    ldx, ldw, ldy = _mat(x, pool.d_in, "x"), _mat(W, pool.d_out, "W"), _mat(y, pool.d_out, "y")
    assert W.shape[0] == pool.d_in
    if h_save is not None:
        assert h_save.dtype == torch.float32 and h_save.is_contiguous() and h_save.numel() == pool.n_parts * T * pool.rank_stride
    _check(load_library().marlaas_lora_forward(pool.handle, T, _dptr(x), ldx, _dptr(W), ldw, _dptr(y), ldy,
                                               ctypes.byref(seg.c), _dptr(h_save), _dptr(ws), ws.numel(),
                                               flags | seg.flags, _stream(stream)))
    return y


def marlaas_lora_forward_multi(calls, flags: int = 0, stream=None):
    """Independent forward calls as one (see marlaas.h): `calls` is a list of dicts with the keyword arguments of
    marlaas_lora_forward (pool, x, W, seg, and y / h_save / workspace, which must be distinct per call; missing y and
    workspace are allocated).  Returns the list of outputs."""
    n = len(calls)
    arr = (marlaas_forward_call_t * max(n, 1))()
    keep, ys = [], []
    fl = flags
    for i, c in enumerate(calls):
        pool, x, W, seg = c["pool"], c["x"], c["W"], c["seg"]
        T = x.shape[0]
        y = c.get("y")
        if y is None:
            y = torch.empty((T, pool.d_out), dtype=torch.bfloat16, device=x.device)
        ws = c.get("workspace")
        if ws is None:
            ws = torch.empty(max(marlaas_lora_forward_workspace_bytes(pool, T), 256), dtype=torch.uint8, device=x.device)
        hs = c.get("h_save")
        if hs is not None:
            assert hs.dtype == torch.float32 and hs.is_contiguous() and hs.numel() == pool.n_parts * T * pool.rank_stride
        assert W.shape[0] == pool.d_in
        arr[i] = marlaas_forward_call_t(pool.handle, T, _dptr(x), _mat(x, pool.d_in, "x"), _dptr(W), _mat(W, pool.d_out, "W"),
                                        _dptr(y), _mat(y, pool.d_out, "y"), ctypes.cast(ctypes.byref(seg.c), ctypes.c_void_p),
                                        _dptr(hs), _dptr(ws), ws.numel())
        fl |= seg.flags
        keep.append((ws, hs, seg))
        ys.append(y)
    _check(load_library().marlaas_lora_forward_multi(n, ctypes.cast(arr, ctypes.c_void_p), fl, _stream(stream)))
    return ys


def marlaas_lora_static_workspace_limit() -> int:
    return int(load_library().marlaas_lora_static_workspace_limit())


def marlaas_lora_forward_static_ws(pool: AdapterPool, x: torch.Tensor, W: torch.Tensor, seg: Segments,
                                   y: torch.Tensor, h_save: Optional[torch.Tensor] = None, flags: int = 0,
                                   stream=None) -> torch.Tensor:
    """Forward for callers that may not allocate on the device: the scratch is the library's built-in array, and
    this wrapper allocates nothing either (y is the caller's).  Raises for batches beyond the array's size."""
    T = x.shape[0]
    ldx, ldw, ldy = _mat(x, pool.d_in, "x"), _mat(W, pool.d_out, "W"), _mat(y, pool.d_out, "y")
    assert W.shape[0] == pool.d_in and y.shape[0] == T
    if h_save is not None:
        assert h_save.dtype == torch.float32 and h_save.is_contiguous() and h_save.numel() == pool.n_parts * T * pool.rank_stride
    _check(load_library().marlaas_lora_forward_static_ws(pool.handle, T, _dptr(x), ldx, _dptr(W), ldw, _dptr(y), ldy,
                                                         ctypes.byref(seg.c), _dptr(h_save), flags | seg.flags,
                                                         _stream(stream)))
    return y


def _ptr_table(ts: Optional[Sequence[Optional[torch.Tensor]]], cap: int):
    if ts is None:
        return None
    tab = (ctypes.c_void_p * cap)()
    for i in range(cap):
        t = ts[i] if i < len(ts) else None
        if t is not None:
            assert t.dtype == torch.float32 and t.is_contiguous()
            tab[i] = t.data_ptr()
    return tab


def marlaas_lora_backward(pool: AdapterPool, x: torch.Tensor, W: torch.Tensor, dy: torch.Tensor, seg: Segments,
                          dx: Optional[torch.Tensor] = None, dA: Optional[Sequence[Optional[torch.Tensor]]] = None,
                          dB: Optional[Sequence[Optional[torch.Tensor]]] = None,
                          h_saved: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                          flags: int = 0, stream=None) -> None:
    T = dy.shape[0]
    ws = workspace if workspace is not None else pool.workspace(T)
    ldx = _mat(x, pool.d_in, "x") if x is not None else 0
    ldw, lddy = _mat(W, pool.d_out, "W"), _mat(dy, pool.d_out, "dy")
    lddx = _mat(dx, pool.d_in, "dx") if dx is not None else 0
    ta, tb = _ptr_table(dA, pool.capacity), _ptr_table(dB, pool.capacity)
    _check(load_library().marlaas_lora_backward(pool.handle, T, _dptr(x), ldx, _dptr(W), ldw, _dptr(dy), lddy,
                                                _dptr(dx), lddx, ta, tb, ctypes.byref(seg.c), _dptr(h_saved),
                                                _dptr(ws), ws.numel(), flags | seg.flags, _stream(stream)))


def marlaas_lora_build_index(pool: AdapterPool, T: int, seg: Segments, workspace: Optional[torch.Tensor] = None,
                             flags: int = 0, stream=None):
    dev = pool.device
    tok_slot = torch.empty(max(T, 1), dtype=torch.int32, device=dev)
    slot_count = torch.empty(pool.capacity + 1, dtype=torch.int32, device=dev)
    slot_offset = torch.empty(pool.capacity + 2, dtype=torch.int32, device=dev)
    perm = torch.empty(max(T, 1), dtype=torch.int32, device=dev)
    ws = workspace if workspace is not None else pool.workspace(T)
    _check(load_library().marlaas_lora_build_index(pool.handle, T, ctypes.byref(seg.c), _dptr(tok_slot),
                                                   _dptr(slot_count), _dptr(slot_offset), _dptr(perm), _dptr(ws),
                                                   ws.numel(), flags | seg.flags, _stream(stream)))
    return tok_slot[:T], slot_count, slot_offset, perm[:T]


def marlaas_check_status(pool: AdapterPool, stream=None) -> None:
    _check(load_library().marlaas_check_status(pool.handle, _stream(stream)))


def marlaas_debug_wait_runs_out(pool: AdapterPool, limit_ns: int = 1_000_000, stream=None) -> None:
    """Diagnostic: one small CTA lets a bounded wait run out; the next marlaas_check_status raises DEVICE_TIMEOUT."""
    _check(load_library().marlaas_debug_wait_runs_out(pool.handle, int(limit_ns), _stream(stream)))


def marlaas_kernel_timing_begin(pool: AdapterPool) -> None:
    _check(load_library().marlaas_kernel_timing_begin(pool.handle))


def marlaas_kernel_timing_end(pool: AdapterPool):
    """(summed device milliseconds, launches) of the dominant kernel since marlaas_kernel_timing_begin."""
    ms, n = ctypes.c_float(), ctypes.c_int32()
    _check(load_library().marlaas_kernel_timing_end(pool.handle, ctypes.byref(ms), ctypes.byref(n)))
    return float(ms.value), int(n.value)
