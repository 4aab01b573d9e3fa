"""Several policy iterations over the whole hot path, GPU against oracle: rollout forward on a mixed decode batch ->
training forward + backward on a mixed training batch -> AdamW step and commit of the new adapter version -> the
next rollout must already run on the committed adapters (Algorithm 1: rollout under version v, policy update,
commit of version v + 1; every call is ordered on one stream, nothing synchronises in between).

The oracle side repeats the loop in float64 / bf16 exactly as the definitions say: after each update its adapters are
the bf16 rounding of its own float64 masters.  Both sides therefore drift apart only by rounding: fp32 vs float64
optimizer arithmetic, and the rare master that rounds to the neighbouring bf16 value; the bars below allow for that.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, dev_bf16, to_np

pytestmark = pytest.mark.gpu

HP = dict(lr=2e-2, beta1=0.9, beta2=0.99, eps=1e-6, weight_decay=0.01, grad_scale=1.0 / 64)


def _bf16_round(a64):
    return wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(np.asarray(a64, dtype=np.float32)))


def test_three_policy_iterations_track_the_oracle():
    K, N, ranks = 256, 320, (16, 8, 32)
    n = len(ranks)
    train = wl.small_random_case(811, 640, K, N, list(ranks), n_segments=7, with_base_only=False)
    p = train.projections[0]
    dc = DeviceCase(train, p, capacity=n)
    ids = [a.tenant_id for a in p.adapters]
    # rollout batch: 96 decode tokens, tenants unsorted, one base-only token
    ts_roll = wl.uniform_token_slots(812, 96, n).astype(np.int32)
    ts_roll[7] = -1
    x_roll_bits = wl.normal_bf16(813, wl.TID_X, (96, K), 1.0)[0]
    off, sl = wl.per_token_table(ts_roll)
    seg_roll = B.Segments(torch.from_numpy(off.astype(np.int32)).cuda(), torch.from_numpy(sl.astype(np.int32)).cuda())
    x_roll = dev_bf16(x_roll_bits)
    ts_train = train.tok_slot()
    scales = [a.alpha / a.rank for a in p.adapters]

    # optimizer state on both sides; masters start at the registered bf16 values
    hA = [wl.bf16_bits_to_f32(a.A_bits).astype(np.float64) for a in p.adapters]
    hB = [wl.bf16_bits_to_f32(a.B_bits).astype(np.float64) for a in p.adapters]
    hst = [[np.zeros_like(hA[t]), np.zeros_like(hA[t]), np.zeros_like(hB[t]), np.zeros_like(hB[t])] for t in range(n)]
    dA_m = [torch.from_numpy(hA[t].astype(np.float32)).cuda() for t in range(n)]
    dB_m = [torch.from_numpy(hB[t].astype(np.float32)).cuda() for t in range(n)]
    dst = [[torch.zeros_like(dA_m[t]), torch.zeros_like(dA_m[t]), torch.zeros_like(dB_m[t]), torch.zeros_like(dB_m[t])]
           for t in range(n)]

    for it in range(1, 4):
        As = [_bf16_round(hA[t]) for t in range(n)]
        Bs = [_bf16_round(hB[t]) for t in range(n)]
        # ---- rollout under the current version ----
        y_roll = B.marlaas_lora_forward(dc.pool, x_roll, dc.W, seg_roll)
        ref_roll, _ = oracle.forward(wl.bf16_bits_to_f32(x_roll_bits), p.W, list(ranks), scales, As, Bs, ts_roll)
        assert_close(to_np(y_roll), ref_roll, f"iteration {it}: rollout forward")
        for t in range(n):
            assert B.marlaas_adapter_pool_lookup(dc.pool, ids[t])[3] == it - 1
        # ---- training step on the mixed batch ----
        hs = torch.empty((train.T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
        y = dc.forward(h_save=hs)
        ref_y, _ = oracle.forward(p.x, p.W, list(ranks), scales, As, Bs, ts_train)
        assert_close(to_np(y), ref_y, f"iteration {it}: training forward")
        dx, gA, gB = dc.backward(h_saved=hs)
        ref_dx, _ = oracle.backward_dx(p.dy, p.W, list(ranks), scales, As, Bs, ts_train)
        ref_gA, ref_gB = oracle.backward_dAdB(p.x, p.dy, list(ranks), scales, As, Bs, ts_train)
        assert_close(to_np(dx), ref_dx, f"iteration {it}: dx")
        for t in range(n):
            assert_close(to_np(gA[t]), ref_gA[t], f"iteration {it}: dA[{t}]")
            assert_close(to_np(gB[t]), ref_gB[t], f"iteration {it}: dB[{t}]")
        # ---- policy update and commit ----
        B.marlaas_adapter_pool_adamw_commit(dc.pool, ids, gA, gB, dA_m, dB_m, [s[0] for s in dst], [s[1] for s in dst],
                                            [s[2] for s in dst], [s[3] for s in dst], step=it, **HP)
        for t in range(n):
            hA[t], hst[t][0], hst[t][1] = oracle.adamw_step(hA[t], ref_gA[t], hst[t][0], hst[t][1], step=it, **HP)
            hB[t], hst[t][2], hst[t][3] = oracle.adamw_step(hB[t], ref_gB[t], hst[t][2], hst[t][3], step=it, **HP)
            # masters: the two sides saw gradients that differ by up to the layer's tolerance, the update divides by
            # sqrt(v) ~ |g|, so the steps agree to about that tolerance times lr
            np.testing.assert_allclose(dA_m[t].cpu().numpy(), hA[t], rtol=0, atol=2e-2 * HP["lr"] * it + 1e-6,
                                       err_msg=f"iteration {it}: master A[{t}]")
            np.testing.assert_allclose(dB_m[t].cpu().numpy(), hB[t], rtol=0, atol=2e-2 * HP["lr"] * it + 1e-6,
                                       err_msg=f"iteration {it}: master B[{t}]")
    B.marlaas_check_status(dc.pool)
