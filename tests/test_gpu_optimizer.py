"""GPU parity of the fused policy update + commit (AdamW on the fp32 masters, bf16 rounding written into the pooled
adapter store) against the float64 oracle, through the C ABI.

Bar: fp32 masters and moments within 2e-5 relative / 1e-7 absolute of the float64 oracle (fp32 arithmetic of a dozen
operations per element); the committed bf16 rows are bit-exact the round-to-nearest-even of the GPU's own fp32
masters; the layer's forward after the commit matches the oracle's forward on the committed adapters.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu

HP = dict(lr=2e-2, beta1=0.9, beta2=0.98, eps=1e-6, weight_decay=0.05, grad_scale=0.5)


def _f32(bits):
    return wl.bf16_bits_to_f32(bits).astype(np.float32)


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def _grad(shape, seed):
    return _f32(wl.normal_bf16(seed, wl.TID_PERTURB, shape, 1.0)[0])


@pytest.mark.parametrize("K,N,ranks", [(192, 136, (16, 5, 64)), (4096, 320, (16,) * 18)])
def test_adamw_commit_matches_the_oracle_and_the_pool_holds_the_rounded_masters(K, N, ranks):
    w = wl.small_random_case(700 + K, 96, K, N, list(ranks), n_segments=9)
    p = w.projections[0]
    dc = DeviceCase(w, p, capacity=len(ranks) + 1)
    n = len(ranks)
    ids = [a.tenant_id for a in p.adapters]
    # host (float64) and device (fp32) optimizer state; masters start at the registered bf16 values
    hA = [_f32(a.A_bits).astype(np.float64) for a in p.adapters]
    hB = [_f32(a.B_bits).astype(np.float64) for a in p.adapters]
    hs = [[np.zeros_like(hA[t]), np.zeros_like(hA[t]), np.zeros_like(hB[t]), np.zeros_like(hB[t])] for t in range(n)]
    dA_m = [_dev(hA[t]) for t in range(n)]
    dB_m = [_dev(hB[t]) for t in range(n)]
    ds = [[torch.zeros_like(dA_m[t]), torch.zeros_like(dA_m[t]), torch.zeros_like(dB_m[t]), torch.zeros_like(dB_m[t])]
          for t in range(n)]
    for step in range(1, 4):
        gA = [_grad((K, r), 1000 * step + 2 * t) for t, r in enumerate(ranks)]
        gB = [_grad((r, N), 1000 * step + 2 * t + 1) for t, r in enumerate(ranks)]
        B.marlaas_adapter_pool_adamw_commit(dc.pool, ids, [_dev(g) for g in gA], [_dev(g) for g in gB], dA_m, dB_m,
                                            [s[0] for s in ds], [s[1] for s in ds], [s[2] for s in ds], [s[3] for s in ds],
                                            step=step, **HP)
        for t in range(n):
            hA[t], hs[t][0], hs[t][1] = oracle.adamw_step(hA[t], gA[t], hs[t][0], hs[t][1], step=step, **HP)
            hB[t], hs[t][2], hs[t][3] = oracle.adamw_step(hB[t], gB[t], hs[t][2], hs[t][3], step=step, **HP)
    B.marlaas_check_status(dc.pool)
    for t, r in enumerate(ranks):
        for got, ref, nm in ((dA_m[t], hA[t], "A"), (dB_m[t], hB[t], "B"), (ds[t][0], hs[t][0], "m_A"),
                             (ds[t][1], hs[t][1], "v_A"), (ds[t][2], hs[t][2], "m_B"), (ds[t][3], hs[t][3], "v_B")):
            np.testing.assert_allclose(got.cpu().numpy(), ref, rtol=2e-5, atol=1e-7, err_msg=f"tenant {t} {nm}")
        slot, rank, _, version = B.marlaas_adapter_pool_lookup(dc.pool, ids[t])
        assert (slot, rank, version) == (t, r, 3)                     # registered at version 0, three commits
        eA, eB = B.marlaas_adapter_pool_export(dc.pool, slot, r)
        assert torch.equal(eA, dA_m[t].to(torch.bfloat16)), f"tenant {t}: committed A is not the rounded master"
        assert torch.equal(eB, dB_m[t].to(torch.bfloat16)), f"tenant {t}: committed B is not the rounded master"
    # the layer now runs on the committed adapters
    ts = w.tok_slot()
    r_, s_, _, _ = oracle.adapters_of(p)
    As = [to_np(B.marlaas_adapter_pool_export(dc.pool, t, r)[0]) for t, r in enumerate(ranks)]
    Bs = [to_np(B.marlaas_adapter_pool_export(dc.pool, t, r)[1]) for t, r in enumerate(ranks)]
    ref, _ = oracle.forward(p.x, p.W, r_, s_, As, Bs, ts)
    assert_close(to_np(dc.forward()), ref, "forward after commit")


def test_adamw_commit_versions_and_errors():
    w = wl.small_random_case(731, 32, 64, 64, [8, 0, 4], n_segments=4)
    p = w.projections[0]
    dc = DeviceCase(w, p, capacity=4)
    ids = [a.tenant_id for a in p.adapters]

    def tensors(r):
        return [torch.zeros((64, r), dtype=torch.float32, device="cuda:0"), torch.zeros((r, 64), dtype=torch.float32, device="cuda:0")]

    def call(tenants, ranks, **kw):
        t = [tensors(r) for r in ranks]
        a = [x[0] for x in t]
        b = [x[1] for x in t]
        B.marlaas_adapter_pool_adamw_commit(dc.pool, tenants, a, b, [x.clone() for x in a], [x.clone() for x in b],
                                            [x.clone() for x in a], [x.clone() for x in a], [x.clone() for x in b],
                                            [x.clone() for x in b], lr=1e-3, **kw)

    call([ids[0], ids[2]], [8, 4], new_versions=[41, 7])
    assert B.marlaas_adapter_pool_lookup(dc.pool, ids[0])[3] == 41 and B.marlaas_adapter_pool_lookup(dc.pool, ids[2])[3] == 7
    call([ids[2]], [4])
    assert B.marlaas_adapter_pool_lookup(dc.pool, ids[2])[3] == 8
    n0 = B.marlaas_kernel_launch_count()
    for tenants, ranks, kw, status in (([987654321], [8], {}, B.MARLAAS_ERR_UNKNOWN_TENANT),
                                       ([ids[1]], [1], {}, B.MARLAAS_ERR_INVALID_ARG),            # rank-0 tenant
                                       ([ids[0], ids[0]], [8, 8], {}, B.MARLAAS_ERR_INVALID_ARG),  # listed twice
                                       ([ids[0]], [8], {"step": 0}, B.MARLAAS_ERR_INVALID_ARG)):
        with pytest.raises(B.MarlaasError) as e:
            call(tenants, ranks, **kw)
        assert e.value.status == status
    assert B.marlaas_kernel_launch_count() == n0                      # nothing was launched
    assert B.marlaas_adapter_pool_lookup(dc.pool, ids[0])[3] == 41
