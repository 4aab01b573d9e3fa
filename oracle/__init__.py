"""CPU oracle for the multi-tenant LoRA linear layer (numpy front end to plain C loops).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's cpu_baseline / reference
legs may import this package; the product path never does, and this package never imports the
CUDA path.  The arithmetic lives in marlaas_oracle.c / marlaas_oracle_impl.inc; this file only
marshals numpy arrays.

Layer definition (frozen shared base weight W, per-tenant adapters A_t, B_t with scale s_t; the
paper's Multi-Task Manager and Multi-LoRA Rollout sections): y_i = x_i W + s_t (x_i A_t) B_t,
dx_i = dy_i W^T + s_t (dy_i B_t^T) A_t^T, dA_t = s_t sum_i x_i^T (dy_i B_t^T),
dB_t = s_t sum_i (x_i A_t)^T dy_i, sums over the tokens routed to tenant t.

adamw_step (the policy update that precedes the commit of a new adapter version in Algorithm 1; the paper names no
optimizer, AdamW is this build's choice) is written out below in float64 numpy.
"""
from __future__ import annotations

import ctypes
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.marlaas_oracle_num_threads.restype = ctypes.c_int
        _lib.marlaas_oracle_build_index.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().marlaas_oracle_num_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _ptr_table(arrs: Sequence[Optional[np.ndarray]]):
    tab = (ctypes.c_void_p * max(1, len(arrs)))()
    for i, a in enumerate(arrs):
        tab[i] = None if a is None else a.ctypes.data
    return tab


def _prep(dtype, ranks, scales, As, Bs):
    sfx = {np.dtype(np.float32): "_f32", np.dtype(np.float64): "_f64"}[np.dtype(dtype)]
    ranks = np.ascontiguousarray(ranks, dtype=np.int32)
    scales = np.ascontiguousarray(scales, dtype=dtype)
    As = [None if a is None else np.ascontiguousarray(a, dtype=dtype) for a in As]
    Bs = [None if b is None else np.ascontiguousarray(b, dtype=dtype) for b in Bs]
    for t, r in enumerate(ranks):
        if r > 0:
            assert As[t].shape[1] == r and Bs[t].shape[0] == r, "adapter shape does not match its rank"
    return sfx, ranks, scales, As, Bs


def build_index(T: int, seg_offsets, seg_slot, cap: int):
    """Segment table -> (tok_slot[T], slot_count[cap+1], slot_offset[cap+2], perm[T]); raises on a bad table."""
    so = np.ascontiguousarray(seg_offsets, dtype=np.int32)
    ss = np.ascontiguousarray(seg_slot, dtype=np.int32)
    S = len(ss)
    assert len(so) == S + 1
    tok_slot = np.empty(max(T, 1), dtype=np.int32)
    count = np.empty(cap + 1, dtype=np.int32)
    offset = np.empty(cap + 2, dtype=np.int32)
    perm = np.empty(max(T, 1), dtype=np.int32)
    rc = lib().marlaas_oracle_build_index(ctypes.c_int(T), ctypes.c_int(S), _ptr(so), _ptr(ss), ctypes.c_int(cap),
                                          _ptr(tok_slot), _ptr(count), _ptr(offset), _ptr(perm))
    if rc != 0:
        raise ValueError("malformed segment table")
    return tok_slot[:T], count, offset, perm[:T]


def forward(x, W, ranks, scales, As, Bs, tok_slot, dtype=np.float32) -> Tuple[np.ndarray, np.ndarray]:
    """y[T][N] and h[T][max rank] (h_i = x_i A_t, zero beyond r_t) for the given per-token slots."""
    sfx, ranks, scales, As, Bs = _prep(dtype, ranks, scales, As, Bs)
    x = np.ascontiguousarray(x, dtype=dtype)
    W = np.ascontiguousarray(W, dtype=dtype)
    ts = np.ascontiguousarray(tok_slot, dtype=np.int32)
    T, K = x.shape
    N = W.shape[1]
    assert W.shape[0] == K and len(ts) == T
    hl = max(1, int(ranks.max()) if len(ranks) else 1)
    y = np.empty((T, N), dtype=dtype)
    h = np.empty((T, hl), dtype=dtype)
    getattr(lib(), "marlaas_oracle_forward" + sfx)(
        ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(N), _ptr(x), _ptr(W), ctypes.c_int(len(ranks)),
        _ptr(ranks), _ptr(scales), _ptr_table(As), _ptr_table(Bs), _ptr(ts), _ptr(y), _ptr(h), ctypes.c_int(hl))
    return y, h


def backward_dx(dy, W, ranks, scales, As, Bs, tok_slot, dtype=np.float32) -> Tuple[np.ndarray, np.ndarray]:
    """dx[T][K] and g[T][max rank] (g_i = dy_i B_t^T)."""
    sfx, ranks, scales, As, Bs = _prep(dtype, ranks, scales, As, Bs)
    dy = np.ascontiguousarray(dy, dtype=dtype)
    W = np.ascontiguousarray(W, dtype=dtype)
    ts = np.ascontiguousarray(tok_slot, dtype=np.int32)
    T, N = dy.shape
    K = W.shape[0]
    assert W.shape[1] == N and len(ts) == T
    gl = max(1, int(ranks.max()) if len(ranks) else 1)
    dx = np.empty((T, K), dtype=dtype)
    g = np.empty((T, gl), dtype=dtype)
    getattr(lib(), "marlaas_oracle_backward_dx" + sfx)(
        ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(N), _ptr(dy), _ptr(W), ctypes.c_int(len(ranks)),
        _ptr(ranks), _ptr(scales), _ptr_table(As), _ptr_table(Bs), _ptr(ts), _ptr(dx), _ptr(g), ctypes.c_int(gl))
    return dx, g


def backward_dAdB(x, dy, ranks, scales, As, Bs, tok_slot, dtype=np.float32):
    """Per-slot adapter gradients: lists dA[t] (K x r_t) and dB[t] (r_t x N); None for rank-0 slots."""
    sfx, ranks, scales, As, Bs = _prep(dtype, ranks, scales, As, Bs)
    x = np.ascontiguousarray(x, dtype=dtype)
    dy = np.ascontiguousarray(dy, dtype=dtype)
    ts = np.ascontiguousarray(tok_slot, dtype=np.int32)
    T, K = x.shape
    N = dy.shape[1]
    assert dy.shape[0] == T and len(ts) == T
    dA: List[Optional[np.ndarray]] = [np.zeros((K, r), dtype=dtype) if r > 0 else None for r in ranks]
    dB: List[Optional[np.ndarray]] = [np.zeros((r, N), dtype=dtype) if r > 0 else None for r in ranks]
    getattr(lib(), "marlaas_oracle_backward_dAdB" + sfx)(
        ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(N), _ptr(x), _ptr(dy), ctypes.c_int(len(ranks)),
        _ptr(ranks), _ptr(scales), _ptr_table(As), _ptr_table(Bs), _ptr(ts), _ptr_table(dA), _ptr_table(dB))
    return dA, dB


def adapters_of(proj, dtype=np.float32):
    """(ranks, scales, As, Bs) of a workload projection, scale = alpha / rank formed in ``dtype``."""
    ranks = [a.rank for a in proj.adapters]
    scales = [np.dtype(dtype).type(a.alpha) / np.dtype(dtype).type(a.rank) if a.rank > 0 else 0 for a in proj.adapters]
    return ranks, scales, [a.A for a in proj.adapters], [a.B for a in proj.adapters]


def adamw_step(theta, grad, m, v, *, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, grad_scale=1.0, step=1):
    """One AdamW step (Adam with decoupled weight decay), from its definition, in float64:
        g = grad_scale * grad;  m' = beta1 m + (1 - beta1) g;  v' = beta2 v + (1 - beta2) g^2
        theta' = theta - lr * ( (m' / (1 - beta1^step)) / (sqrt(v' / (1 - beta2^step)) + eps) + weight_decay * theta )
    Returns (theta', m', v')."""
    theta, m, v = (np.asarray(a, dtype=np.float64) for a in (theta, m, v))
    g = float(grad_scale) * np.asarray(grad, dtype=np.float64)
    m1 = beta1 * m + (1.0 - beta1) * g
    v1 = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m1 / (1.0 - beta1 ** step)
    v_hat = v1 / (1.0 - beta2 ** step)
    theta1 = theta - lr * (m_hat / (np.sqrt(v_hat) + eps) + weight_decay * theta)
    return theta1, m1, v1
