"""Projections that share their input (q, k, v; gate, up) served by ONE layer call: the base weights side by side, the
tenants' A side by side and their B block diagonal.  The GPU runs the fused projection; the oracle runs every
projection on its own, from the definition; the fused outputs must be the concatenation (y, dA, the diagonal blocks
of dB) resp. the sum (dx) of the separate ones, within the layer's tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu


def _separate_case(seed, T, K, Ns, n, rank, per_token):
    w0 = wl.small_random_case(seed, T, K, Ns[0], [rank] * n, n_segments=7)
    if per_token:
        ts = wl.uniform_token_slots(seed, T, n).astype(np.int32)
        ts[3] = -1
        w0.seg_offsets, w0.seg_slot = wl.per_token_table(ts)
    projs = [w0.projections[0]]
    projs[0].name = "p0"
    for i, N in enumerate(Ns[1:], start=1):
        wi = wl.small_random_case(seed + 50 * i, T, K, N, [rank] * n, n_segments=7)
        pi = wi.projections[0]
        pi.name, pi.x_bits = f"p{i}", projs[0].x_bits
        for a, a0 in zip(pi.adapters, projs[0].adapters):
            a.tenant_id = a0.tenant_id
        projs.append(pi)
    w0.projections = projs
    return w0


@pytest.mark.parametrize("T,K,Ns,n,rank,per_token", [
    (200, 256, (256, 128, 128), 5, 16, True),       # q, k, v shaped, decode batch (one token per segment)
    (96, 192, (384, 384), 3, 8, True),              # gate, up shaped; rank 8 blocks inside one 16-rank unit
    (700, 128, (128, 256), 4, 16, False),           # training-shaped batch with backward
])
def test_fused_projection_equals_the_separate_projections(T, K, Ns, n, rank, per_token):
    w = _separate_case(640 + T, T, K, Ns, n, rank, per_token)
    f = wl.fuse_projections(w)
    pf = f.projections[0]
    ts = w.tok_slot()
    offs = np.concatenate([[0], np.cumsum(Ns)])
    P = len(Ns)
    # oracle: every projection on its own
    ys, dxs, dAs, dBs = [], [], [], []
    for p in w.projections:
        r, s, A, Bm = oracle.adapters_of(p)
        ys.append(oracle.forward(p.x, p.W, r, s, A, Bm, ts)[0])
        if not per_token:
            dxs.append(oracle.backward_dx(p.dy, p.W, r, s, A, Bm, ts)[0])
            a, b = oracle.backward_dAdB(p.x, p.dy, r, s, A, Bm, ts)
            dAs.append(a)
            dBs.append(b)
    dc = DeviceCase(f, pf, capacity=n + 1)
    hs = torch.empty((T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    y = dc.forward(h_save=hs)
    assert_close(to_np(y), np.concatenate(ys, axis=1), "fused forward = separate forwards side by side")
    if not per_token:
        dx, dA, dB = dc.backward(h_saved=hs)
        assert_close(to_np(dx), sum(dxs), "fused dx = sum of the separate dx")
        for t in range(n):
            if t in set(ts.tolist()) or True:
                got_A, got_B = to_np(dA[t]), to_np(dB[t])
                for i in range(P):
                    assert_close(got_A[:, i * rank:(i + 1) * rank], dAs[i][t], f"dA of tenant {t}, projection {i}")
                    assert_close(got_B[i * rank:(i + 1) * rank, offs[i]:offs[i + 1]], dBs[i][t],
                                 f"dB of tenant {t}, projection {i} (diagonal block)")
    B.marlaas_check_status(dc.pool)


def test_independent_projections_as_one_multi_call():
    # q, k, v shaped: three pools, one decode batch, one call; every output against the oracle of its own projection,
    # and bit for bit against the three single calls (the same kernels, only on side streams)
    T, K, Ns, n, rank = 130, 256, (256, 128, 320), 5, 16
    w = _separate_case(977, T, K, Ns, n, rank, True)
    ts = w.tok_slot()
    dcs = [DeviceCase(w, p, capacity=n + 1) for p in w.projections]
    calls = [dict(pool=dc.pool, x=dc.x, W=dc.W, seg=dc.seg,
                  h_save=torch.empty((T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")) for dc in dcs]
    ys = B.marlaas_lora_forward_multi(calls)
    torch.cuda.synchronize()
    for dc, p, y, c in zip(dcs, w.projections, ys, calls):
        r, s, A, Bm = oracle.adapters_of(p)
        ry, rh = oracle.forward(p.x, p.W, r, s, A, Bm, ts)
        assert_close(to_np(y), ry, f"multi call: y of {p.name}")
        hs = torch.empty_like(c["h_save"])
        y1 = dc.forward(h_save=hs)
        assert torch.equal(y1, y) and torch.equal(hs, c["h_save"])
        B.marlaas_check_status(dc.pool)
    # two entries on one pool, or sharing a workspace, are refused before anything is launched
    n0 = B.marlaas_kernel_launch_count()
    with pytest.raises(B.MarlaasError):
        B.marlaas_lora_forward_multi([calls[0], dict(calls[0])])
    shared = torch.empty(1 << 22, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.MarlaasError):
        B.marlaas_lora_forward_multi([dict(calls[0], workspace=shared), dict(calls[1], workspace=shared)])
    assert B.marlaas_kernel_launch_count() == n0


@pytest.mark.parametrize("T,K,Ns,n,rank", [
    (1300, 128, (256, 128, 192), 5, 16),      # 2-CTA GEMM, tensor-core gradient reductions on the side stream
    (600, 192, (128, 256), 4, 8),             # 1-CTA GEMM
])
def test_a_layers_projections_reuse_the_plan_of_the_first(T, K, Ns, n, rank):
    # Projections of one layer see the same mixed batch: the first forward (backward) builds the plan in the shared
    # workspace, the others run with MARLAAS_FLAG_REUSE_PLAN.  Every projection's outputs against its own oracle run.
    w = _separate_case(1200 + T, T, K, Ns, n, rank, False)
    ts = w.tok_slot()
    dcs = [DeviceCase(w, p, capacity=n + 1) for p in w.projections]
    ws = torch.empty(max(B.marlaas_lora_workspace_bytes(dc.pool, T) for dc in dcs), dtype=torch.uint8, device="cuda:0")
    hs = [torch.empty((T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0") for dc in dcs]
    ys = []
    for j, dc in enumerate(dcs):
        ys.append(B.marlaas_lora_forward(dc.pool, dc.x, dc.W, dc.seg, h_save=hs[j], workspace=ws,
                                         flags=B.MARLAAS_FLAG_REUSE_PLAN if j else 0))
    outs = []
    for j, dc in enumerate(dcs):
        dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda:0")
        dA, dB = dc.grads(fill=3.0)
        B.marlaas_lora_backward(dc.pool, dc.x, dc.W, dc.dy, dc.seg, dx=dx, dA=dA, dB=dB, h_saved=hs[j], workspace=ws,
                                flags=B.MARLAAS_FLAG_REUSE_PLAN if j else 0)
        outs.append((dx, dA, dB))
    torch.cuda.synchronize()
    for j, (dc, p) in enumerate(zip(dcs, w.projections)):
        r, s, A, Bm = oracle.adapters_of(p)
        assert_close(to_np(ys[j]), oracle.forward(p.x, p.W, r, s, A, Bm, ts)[0], f"{p.name}: y with a reused plan")
        assert_close(to_np(outs[j][0]), oracle.backward_dx(p.dy, p.W, r, s, A, Bm, ts)[0], f"{p.name}: dx with a reused plan")
        rdA, rdB = oracle.backward_dAdB(p.x, p.dy, r, s, A, Bm, ts)
        for t in range(n):
            assert_close(to_np(outs[j][1][t]), rdA[t], f"{p.name}: dA[{t}] with a reused plan")
            assert_close(to_np(outs[j][2][t]), rdB[t], f"{p.name}: dB[{t}] with a reused plan")
        B.marlaas_check_status(dc.pool)
