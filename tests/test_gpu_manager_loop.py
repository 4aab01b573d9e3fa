"""Algorithm 1 driving the layer on the GPU: rollout threads (decode forward under each task's current adapter) and
one training thread (forward + backward on the task's batch, AdamW step, commit) run asynchronously under the
multi-task manager.  Tasks only touch their own adapters, so whatever the interleaving was, each task's sequence of
rollout outputs must match the oracle replaying that task's loop on its own; the pool's version counters must agree
with the manager's.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import manager as M
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, dev_bf16, to_np

pytestmark = pytest.mark.gpu

HP = dict(lr=2e-2, beta1=0.9, beta2=0.99, eps=1e-6, weight_decay=0.0, grad_scale=1.0 / 64)


def _bf16_round(a64):
    return wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(np.asarray(a64, dtype=np.float32)))


def test_asynchronous_loop_matches_per_task_oracle_replay():
    K, N, ranks, versions = 128, 192, (16, 8, 16, 4), 3
    n = len(ranks)
    base = wl.small_random_case(905, 64, K, N, list(ranks), n_segments=2)
    p = base.projections[0]
    dc = DeviceCase(base, p, capacity=n)
    ids = [a.tenant_id for a in p.adapters]
    scales = [a.alpha / a.rank for a in p.adapters]
    # per task: a rollout batch of 40 decode tokens and a training batch of 96 tokens, all its own
    xr_bits = [wl.normal_bf16(920 + t, wl.TID_X, (40, K), 1.0)[0] for t in range(n)]
    xt_bits = [wl.normal_bf16(940 + t, wl.TID_X, (96, K), 1.0)[0] for t in range(n)]
    dy_bits = [wl.normal_bf16(960 + t, wl.TID_DY, (96, N), 1.0)[0] for t in range(n)]
    xr, xt, dy = [dev_bf16(b) for b in xr_bits], [dev_bf16(b) for b in xt_bits], [dev_bf16(b) for b in dy_bits]

    def seg_of(task, T, per_token):
        off = np.arange(T + 1, dtype=np.int32) if per_token else np.array([0, T], dtype=np.int32)
        sl = np.full(len(off) - 1, task, dtype=np.int32)
        return B.Segments(torch.from_numpy(off).cuda(), torch.from_numpy(sl).cuda())

    seg_r = [seg_of(t, 40, True) for t in range(n)]
    seg_t = [seg_of(t, 96, False) for t in range(n)]
    mA = [torch.from_numpy(wl.bf16_bits_to_f32(a.A_bits)).cuda() for a in p.adapters]
    mB = [torch.from_numpy(wl.bf16_bits_to_f32(a.B_bits)).cuda() for a in p.adapters]
    st = [[torch.zeros_like(mA[t]), torch.zeros_like(mA[t]), torch.zeros_like(mB[t]), torch.zeros_like(mB[t])] for t in range(n)]
    rollouts = {}

    def rollout(task, version, device_lock):
        with device_lock:
            y = B.marlaas_lora_forward(dc.pool, xr[task], dc.W, seg_r[task])
            out = to_np(y)                         # synchronises: the trajectory leaves the device
            assert B.marlaas_adapter_pool_lookup(dc.pool, ids[task])[3] == version
        rollouts[(task, version)] = out
        return out

    def update(task, tau, version, device_lock):
        with device_lock:
            hs = torch.empty((96, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
            B.marlaas_lora_forward(dc.pool, xt[task], dc.W, seg_t[task], h_save=hs)
            dA, dB = dc.grads()
            B.marlaas_lora_backward(dc.pool, xt[task], dc.W, dy[task], seg_t[task], dx=None, dA=dA, dB=dB, h_saved=hs)
            B.marlaas_adapter_pool_adamw_commit(dc.pool, [ids[task]], [dA[task]], [dB[task]], [mA[task]], [mB[task]],
                                                [st[task][0]], [st[task][1]], [st[task][2]], [st[task][3]], step=version + 1, **HP)
            torch.cuda.synchronize()

    mgr = M.MultiTaskManager(kv_budget_bytes=3 * M.kv_cache_bytes(40, 64, 4, 2, 64))       # three of the four tasks at a time
    for t in range(n):
        mgr.add_task(t, M.kv_cache_bytes(40, 64, 4, 2, 64))
    M.run_loop(mgr, list(range(n)), versions, rollout, update)
    B.marlaas_check_status(dc.pool)

    # oracle: every task's loop replayed on its own
    for t in range(n):
        A64 = wl.bf16_bits_to_f32(p.adapters[t].A_bits).astype(np.float64)
        B64 = wl.bf16_bits_to_f32(p.adapters[t].B_bits).astype(np.float64)
        s = [np.zeros_like(A64), np.zeros_like(A64), np.zeros_like(B64), np.zeros_like(B64)]
        for v in range(versions):
            Ab, Bb = _bf16_round(A64), _bf16_round(B64)
            ref, _ = oracle.forward(wl.bf16_bits_to_f32(xr_bits[t]), p.W, [ranks[t]], [scales[t]], [Ab], [Bb], np.zeros(40, np.int32))
            assert_close(rollouts[(t, v)], ref, f"task {t}: rollout under version {v}")
            x64, d64 = wl.bf16_bits_to_f32(xt_bits[t]), wl.bf16_bits_to_f32(dy_bits[t])
            gA, gB = oracle.backward_dAdB(x64, d64, [ranks[t]], [scales[t]], [Ab], [Bb], np.zeros(96, np.int32))
            A64, s[0], s[1] = oracle.adamw_step(A64, gA[0], s[0], s[1], step=v + 1, **HP)
            B64, s[2], s[3] = oracle.adamw_step(B64, gB[0], s[2], s[3], step=v + 1, **HP)
        assert mgr.tasks[t].version == versions
        assert B.marlaas_adapter_pool_lookup(dc.pool, ids[t])[3] == versions
        np.testing.assert_allclose(mA[t].cpu().numpy(), A64, rtol=0, atol=2e-2 * HP["lr"] * versions + 1e-6)
        np.testing.assert_allclose(mB[t].cpu().numpy(), B64, rtol=0, atol=2e-2 * HP["lr"] * versions + 1e-6)
