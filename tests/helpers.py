"""Shared helpers of the GPU parity tests: upload seeded workloads, run the C-ABI path, compare with the oracle."""
import numpy as np
import torch

import paper_2605_08527_b200 as ml
from paper_2605_08527_b200 import binding as B

TOL_ABS, TOL_REL = 1e-2, 1e-2      # |gpu - ref| <= 1e-2 + 1e-2 |ref| for bf16-in / fp32-accumulate results


def dev_bf16(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def assert_close(got: np.ndarray, ref: np.ndarray, what: str, atol=TOL_ABS, rtol=TOL_REL):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    err = np.abs(got - ref)
    bound = atol + rtol * np.abs(ref)
    bad = err > bound
    if np.any(bad):
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())}/{bad.size} elements outside |gpu-ref| <= {atol} + {rtol}|ref|; "
                             f"worst at {i}: gpu={got[i]:.6g} ref={ref[i]:.6g}")


class DeviceCase:
    """One projection of a workload resident on the GPU with its adapters registered (slot t = adapter t)."""

    def __init__(self, w, proj, capacity=None, max_rank=None, register=True):
        self.w, self.p = w, proj
        n = len(proj.adapters)
        self.capacity = capacity or max(1, n)
        self.max_rank = max_rank or max([a.rank for a in proj.adapters] + [1])
        self.pool = B.AdapterPool(proj.d_in, proj.d_out, self.max_rank, self.capacity)
        self.W = dev_bf16(proj.W_bits)
        self.x = dev_bf16(proj.x_bits)
        self.dy = None if proj.dy_bits is None else dev_bf16(proj.dy_bits)
        self.A = [dev_bf16(a.A_bits) if a.rank > 0 else None for a in proj.adapters]
        self.Bm = [dev_bf16(a.B_bits) if a.rank > 0 else None for a in proj.adapters]
        if register:
            for t, a in enumerate(proj.adapters):
                slot = B.marlaas_adapter_pool_register(self.pool, a.tenant_id, 0, a.rank, a.alpha, self.A[t], self.Bm[t])
                assert slot == t
        self.seg = B.Segments(torch.from_numpy(w.seg_offsets.astype(np.int32)).cuda(),
                              torch.from_numpy(w.seg_slot.astype(np.int32)).cuda())
        self.seg_host = B.Segments(torch.from_numpy(w.seg_offsets.astype(np.int32).copy()),
                                   torch.from_numpy(w.seg_slot.astype(np.int32).copy()))

    def seg_prefix(self, T):
        """Segment table restricted to the first T tokens (the backward rows of a mixed batch)."""
        so, ss = self.w.seg_offsets, self.w.seg_slot
        keep = [s for s in range(len(ss)) if so[s] < T]
        off = np.array([min(int(so[s]), T) for s in keep] + [T], dtype=np.int32)
        sl = np.array([ss[s] for s in keep], dtype=np.int32)
        return B.Segments(torch.from_numpy(off).cuda(), torch.from_numpy(sl).cuda())

    def grads(self, fill=None):
        dA, dB = [], []
        for a in self.p.adapters:
            if a.rank > 0:
                mk = (lambda *s: torch.full(s, fill, dtype=torch.float32, device="cuda:0")) if fill is not None else \
                     (lambda *s: torch.empty(s, dtype=torch.float32, device="cuda:0"))
                dA.append(mk(self.p.d_in, a.rank))
                dB.append(mk(a.rank, self.p.d_out))
            else:
                dA.append(None)
                dB.append(None)
        return dA, dB

    def forward(self, flags=0, h_save=None, seg=None, x=None):
        x = self.x if x is None else x
        y = B.marlaas_lora_forward(self.pool, x, self.W, seg or self.seg, h_save=h_save, flags=flags)
        return y

    def backward(self, flags=0, h_saved=None, seg=None, want_dx=True, dA=None, dB=None, T=None):
        T = T or self.dy.shape[0]
        dx = torch.empty((T, self.p.d_in), dtype=torch.bfloat16, device="cuda:0") if want_dx else None
        if dA is None and dB is None:
            dA, dB = self.grads()
        B.marlaas_lora_backward(self.pool, self.x[:T], self.W, self.dy[:T], seg or self.seg, dx=dx, dA=dA, dB=dB,
                                h_saved=h_saved, flags=flags)
        return dx, dA, dB
