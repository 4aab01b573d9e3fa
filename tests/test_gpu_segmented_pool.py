"""A pool over several projections that read the same activations (q, k, v; gate, up): one layer call over the
side-by-side base weights, the tenants' adapters kept per projection (no block-diagonal zeros stored or streamed).
The GPU runs the one call; the oracle runs every projection on its own, from the definition.  y must be the separate
outputs side by side, dx their sum, dA_t / dB_t the separate gradients block after block.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import assert_close, dev_bf16, to_np

pytestmark = pytest.mark.gpu


def _case(seed, T, K, Ns, ranks, per_token, n_segments=7):
    """Projections of widths Ns over one x and one segment table; tenant t has rank ranks[t] on every projection."""
    n = len(ranks)
    w0 = wl.small_random_case(seed, T, K, Ns[0], list(ranks), n_segments=n_segments)
    if per_token:
        ts = wl.uniform_token_slots(seed, T, n).astype(np.int32)
        ts[min(3, T - 1)] = -1
        w0.seg_offsets, w0.seg_slot = wl.per_token_table(ts)
    projs = [w0.projections[0]]
    for i, N in enumerate(Ns[1:], start=1):
        wi = wl.small_random_case(seed + 50 * i, T, K, N, list(ranks), n_segments=n_segments)
        pi = wi.projections[0]
        pi.x_bits = projs[0].x_bits
        for a, a0 in zip(pi.adapters, projs[0].adapters):
            a.tenant_id, a.alpha = a0.tenant_id, a0.alpha
        projs.append(pi)
    w0.projections = projs
    return w0


class SegCase:
    def __init__(self, w, capacity=None):
        self.w = w
        ps = w.projections
        self.Ns = [p.d_out for p in ps]
        self.K = ps[0].d_in
        n = len(ps[0].adapters)
        self.ranks = [a.rank for a in ps[0].adapters]
        self.pool = B.AdapterPool(self.K, sum(self.Ns), max(self.ranks + [1]), capacity or n, parts=self.Ns)
        self.W = dev_bf16(np.concatenate([p.W_bits for p in ps], axis=1))
        self.x = dev_bf16(ps[0].x_bits)
        self.dy = None if ps[0].dy_bits is None else dev_bf16(np.concatenate([p.dy_bits for p in ps], axis=1))
        for t in range(n):
            a0 = ps[0].adapters[t]
            As = [dev_bf16(p.adapters[t].A_bits) for p in ps] if a0.rank > 0 else None
            Bs = [dev_bf16(p.adapters[t].B_bits) for p in ps] if a0.rank > 0 else None
            assert B.marlaas_adapter_pool_register(self.pool, a0.tenant_id, 0, a0.rank, a0.alpha, As, Bs) == t
        self.seg = B.Segments(torch.from_numpy(w.seg_offsets.astype(np.int32)).cuda(),
                              torch.from_numpy(w.seg_slot.astype(np.int32)).cuda())

    def grads(self, fill=None):
        mk = (lambda n: torch.full((n,), fill, dtype=torch.float32, device="cuda:0")) if fill is not None else \
             (lambda n: torch.empty(n, dtype=torch.float32, device="cuda:0"))
        dA = [mk(len(self.Ns) * self.K * r) if r > 0 else None for r in self.ranks]
        dB = [mk(r * sum(self.Ns)) if r > 0 else None for r in self.ranks]
        return dA, dB

    def split_dA(self, t, dA):
        r = self.ranks[t]
        return [to_np(dA[p * self.K * r:(p + 1) * self.K * r]).reshape(self.K, r) for p in range(len(self.Ns))]

    def split_dB(self, t, dB):
        r, out, o = self.ranks[t], [], 0
        for N in self.Ns:
            out.append(to_np(dB[o:o + r * N]).reshape(r, N))
            o += r * N
        return out


def _oracle_forward(w, ts):
    ys, hs = [], []
    for p in w.projections:
        r, s, A, Bm = oracle.adapters_of(p)
        y, h = oracle.forward(p.x, p.W, r, s, A, Bm, ts)
        ys.append(y)
        hs.append(h)
    return np.concatenate(ys, axis=1), hs


def test_store_roundtrip_of_a_pool_over_three_projections():
    w = _case(31, 64, 256, (512, 256, 256), (16, 8, 40, 0, 64), True)
    sc = SegCase(w, capacity=6)
    assert sc.pool.n_parts == 3
    for t, r in enumerate(sc.ranks):
        if r == 0:
            continue
        As, Bs = B.marlaas_adapter_pool_export(sc.pool, t, r)
        for p, proj in enumerate(w.projections):
            assert np.array_equal(As[p].view(torch.int16).cpu().numpy().view(np.uint16), proj.adapters[t].A_bits)
            assert np.array_equal(Bs[p].view(torch.int16).cpu().numpy().view(np.uint16), proj.adapters[t].B_bits)
    # part widths that would let a 256-column tile straddle two projections are refused
    with pytest.raises(B.MarlaasError):
        B.AdapterPool(256, 384, 16, 4, parts=[128, 256])
    B.marlaas_check_status(sc.pool)


@pytest.mark.parametrize("T,K,Ns,ranks,per_token,flags", [
    (200, 256, (512, 256, 256), (16, 16, 32, 8, 64), True, 0),            # q, k, v; decode batch
    (96, 4096, (8192, 8192), (16, 64, 8), True, 0),                       # gate, up over a large weight (wide decode kernel)
    (64, 2048, (9728, 9728), (16, 32, 8), True, 0),                       # 76 strips on 74 CTA pairs: tiles cut between pairs
    (1, 128, (256, 256), (16,), True, 0),                                 # a single token
    (333, 192, (256, 512, 256), (16, 0, 40, 8), True, 0),                 # a registered tenant of rank 0 (base weight only)
    (700, 128, (256, 512), (16, 8, 24, 16), False, 0),                    # training shape below 1024 rows
    (1500, 192, (256, 256, 512), (16, 32, 8, 64, 16), False, 0),          # training shape, several row tiles
    (300, 136, (256, 256), (16, 8, 24), False, B.MARLAAS_FLAG_CUDA_CORE_PATH),
    # one shrink over all projections' adapter rows, the contraction cut over a cluster: three planes of rank stride 64
    (1500, 4096, (256, 512, 256), (16, 32, 8, 64, 16), False, 0),
    # every token its own tenant: eight and more units per 128-token tile, four per work item with two projections; a tenant
    # of three units lies across two items
    (900, 2048, (512, 256), (16, 8, 16, 40, 16, 16, 24, 16, 16), True, 0),
    (640, 1024, (256, 256, 256, 256), (16, 24, 8), True, 0),              # four projections: two units per work item
    (600, 512, (256, 256, 256, 256), (128, 16), False, 0),                # rank stride 128 x 4 planes: one shrink per projection
    (777, 1024, (256, 512), (16, 16), False, 0),                          # last tile with 9 rows
])
def test_forward_of_a_pool_over_several_projections(T, K, Ns, ranks, per_token, flags):
    w = _case(900 + T, T, K, Ns, ranks, per_token)
    ts = w.tok_slot()
    sc = SegCase(w, capacity=len(ranks) + 1)
    P = len(Ns)
    hs = torch.full((P, T, sc.pool.rank_stride), 7.0, dtype=torch.float32, device="cuda:0")
    y = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, h_save=hs, flags=flags)
    ry, rh = _oracle_forward(w, ts)
    assert_close(to_np(y), ry, "y = the projections' outputs side by side")
    for p in range(P):
        got = to_np(hs[p])
        assert_close(got[:, :rh[p].shape[1]], rh[p], f"h of projection {p}", atol=1e-3, rtol=1e-3)
        assert np.all(got[:, rh[p].shape[1]:] == 0)
    # the same call again is bit-identical (nothing depends on what the workspace held)
    y2 = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, flags=flags)
    assert torch.equal(y, y2)
    B.marlaas_check_status(sc.pool)


@pytest.mark.parametrize("T,K,Ns,ranks,flags,saved", [
    (1300, 128, (256, 256, 512), (16, 32, 8, 64), 0, True),       # 2-CTA GEMM, gradient reductions on the side stream
    (1300, 128, (256, 256, 512), (16, 32, 8, 64), 0, False),      # h recomputed
    (600, 192, (256, 512), (16, 8, 24), 0, True),
    (150, 64, (256, 256), (16, 8), 0, True),
    (1100, 128, (512, 256), (16, 0, 24, 8), 0, True),             # a tenant of rank 0: no gradient arrays, base-only rows
    (300, 136, (256, 256), (16, 8, 24), B.MARLAAS_FLAG_CUDA_CORE_PATH, True),
    (1300, 2048, (256, 256, 512), (16, 32, 8, 64), 0, True),      # forward through one shrink over the three projections
])
def test_backward_of_a_pool_over_several_projections(T, K, Ns, ranks, flags, saved):
    w = _case(1700 + T, T, K, Ns, ranks, False)
    ts = w.tok_slot()
    sc = SegCase(w, capacity=len(ranks) + 1)
    P, n = len(Ns), len(ranks)
    hs = torch.empty((P, T, sc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, h_save=hs, flags=flags)
    dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda:0")
    dA, dB = sc.grads(fill=3.0)
    B.marlaas_lora_backward(sc.pool, sc.x, sc.W, sc.dy, sc.seg, dx=dx, dA=dA, dB=dB, h_saved=hs if saved else None, flags=flags)
    rdx, rdA, rdB = 0.0, [], []
    for p in w.projections:
        r, s, A, Bm = oracle.adapters_of(p)
        rdx = rdx + oracle.backward_dx(p.dy, p.W, r, s, A, Bm, ts)[0]
        a, b = oracle.backward_dAdB(p.x, p.dy, r, s, A, Bm, ts)
        rdA.append(a)
        rdB.append(b)
    assert_close(to_np(dx), rdx, "dx = sum over the projections")
    for t in range(n):
        if ranks[t] == 0:
            continue
        gA, gB = sc.split_dA(t, dA[t]), sc.split_dB(t, dB[t])
        for p in range(P):
            assert_close(gA[p], rdA[p][t], f"dA of tenant {t}, projection {p}")
            assert_close(gB[p], rdB[p][t], f"dB of tenant {t}, projection {p}")
    # accumulate: a second pass adds the same contribution
    B.marlaas_lora_backward(sc.pool, sc.x, sc.W, sc.dy, sc.seg, dx=None, dA=dA, dB=dB, h_saved=hs if saved else None,
                            flags=flags | B.MARLAAS_FLAG_ACCUMULATE)
    for t in range(n):
        if ranks[t] == 0:
            continue
        gA = sc.split_dA(t, dA[t])
        for p in range(P):
            assert_close(gA[p], 2 * rdA[p][t], f"accumulated dA of tenant {t}, projection {p}", atol=2e-2)
    B.marlaas_check_status(sc.pool)


def test_adamw_commit_on_a_pool_over_two_projections():
    T, K, Ns, ranks = 64, 128, (256, 512), (16, 8)
    w = _case(77, T, K, Ns, ranks, True)
    sc = SegCase(w, capacity=3)
    rng = np.random.default_rng(5)
    ids = [w.projections[0].adapters[t].tenant_id for t in range(2)]
    tabs = {k: [] for k in ("dA", "dB", "A", "B", "mA", "vA", "mB", "vB")}
    ref = []
    for t, r in enumerate(ranks):
        nA, nB = len(Ns) * K * r, r * sum(Ns)
        host = {"dA": rng.standard_normal(nA), "dB": rng.standard_normal(nB), "A": rng.standard_normal(nA) * 0.1,
                "B": rng.standard_normal(nB) * 0.1, "mA": np.zeros(nA), "vA": np.zeros(nA), "mB": np.zeros(nB), "vB": np.zeros(nB)}
        for k, v in host.items():
            tabs[k].append(torch.from_numpy(v.astype(np.float32)).cuda())
        ref.append({k: v.astype(np.float32).astype(np.float64) for k, v in host.items()})
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01, grad_scale=0.5, step=1)
    B.marlaas_adapter_pool_adamw_commit(sc.pool, ids, tabs["dA"], tabs["dB"], tabs["A"], tabs["B"], tabs["mA"], tabs["vA"],
                                        tabs["mB"], tabs["vB"], **hp)
    for t, r in enumerate(ranks):
        As, Bs = B.marlaas_adapter_pool_export(sc.pool, t, r)
        newA = oracle.adamw_step(ref[t]["A"], ref[t]["dA"], ref[t]["mA"], ref[t]["vA"], **hp)[0]
        newB = oracle.adamw_step(ref[t]["B"], ref[t]["dB"], ref[t]["mB"], ref[t]["vB"], **hp)[0]
        assert_close(to_np(tabs["A"][t]), newA, "fp32 master A", atol=1e-5, rtol=1e-5)
        assert_close(to_np(tabs["B"][t]), newB, "fp32 master B", atol=1e-5, rtol=1e-5)
        # the store holds the bf16 rounding of the new masters, block by block
        gotA = torch.cat([a.reshape(-1) for a in As]).float()
        gotB = torch.cat([b.reshape(-1) for b in Bs]).float()
        assert torch.equal(gotA, tabs["A"][t].to(torch.bfloat16).float())
        assert torch.equal(gotB, tabs["B"][t].to(torch.bfloat16).float())
    B.marlaas_check_status(sc.pool)


def test_plan_shared_between_a_pool_over_two_projections_and_a_plain_pool():
    # One layer, one mixed batch, one workspace: the pool over (p0, p1) builds the plan, the plain pool of p2 reuses it
    # (forward and backward), then the other way round.  The plan's place in the workspace must not depend on how many
    # projections a pool holds.
    from helpers import DeviceCase
    T, K, Ns, ranks = 1300, 128, (256, 512, 384), (16, 8, 16, 16)
    w = _case(2100, T, K, Ns, ranks, False)
    ts = w.tok_slot()
    import copy
    w2 = copy.copy(w)
    w2.projections = w.projections[:2]
    sc = SegCase(w2, capacity=len(ranks) + 1)
    p2 = w.projections[2]
    dc = DeviceCase(w, p2, capacity=len(ranks) + 1, max_rank=max(ranks))
    ws = torch.empty(max(B.marlaas_lora_workspace_bytes(sc.pool, T), B.marlaas_lora_workspace_bytes(dc.pool, T)),
                     dtype=torch.uint8, device="cuda:0")
    r2, s2, A2, B2 = oracle.adapters_of(p2)
    ry2 = oracle.forward(p2.x, p2.W, r2, s2, A2, B2, ts)[0]
    rdx2 = oracle.backward_dx(p2.dy, p2.W, r2, s2, A2, B2, ts)[0]
    rdA2, rdB2 = oracle.backward_dAdB(p2.x, p2.dy, r2, s2, A2, B2, ts)
    ry01 = _oracle_forward(w2, ts)[0]
    for first_seg in (True, False):
        hs_s = torch.empty((2, T, sc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
        hs_p = torch.empty((T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
        ws.fill_(0x5a)
        fl = lambda second: B.MARLAAS_FLAG_REUSE_PLAN if second else 0
        if first_seg:
            y01 = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, h_save=hs_s, workspace=ws, flags=fl(False))
            y2 = B.marlaas_lora_forward(dc.pool, dc.x, dc.W, dc.seg, h_save=hs_p, workspace=ws, flags=fl(True))
        else:
            y2 = B.marlaas_lora_forward(dc.pool, dc.x, dc.W, dc.seg, h_save=hs_p, workspace=ws, flags=fl(False))
            y01 = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, h_save=hs_s, workspace=ws, flags=fl(True))
        assert_close(to_np(y01), ry01, "pool over two projections, shared plan: y")
        assert_close(to_np(y2), ry2, "plain pool, shared plan: y")
        dx2 = torch.empty((T, K), dtype=torch.bfloat16, device="cuda:0")
        dA2, dB2 = dc.grads(fill=1.0)
        dxs = torch.empty((T, K), dtype=torch.bfloat16, device="cuda:0")
        dAs, dBs = sc.grads(fill=1.0)
        calls = [lambda f: B.marlaas_lora_backward(sc.pool, sc.x, sc.W, sc.dy, sc.seg, dx=dxs, dA=dAs, dB=dBs, h_saved=hs_s,
                                                   workspace=ws, flags=f),
                 lambda f: B.marlaas_lora_backward(dc.pool, dc.x, dc.W, dc.dy, dc.seg, dx=dx2, dA=dA2, dB=dB2, h_saved=hs_p,
                                                   workspace=ws, flags=f)]
        if not first_seg:
            calls.reverse()
        calls[0](fl(False))
        calls[1](fl(True))
        assert_close(to_np(dx2), rdx2, "plain pool, shared plan: dx")
        for t in range(len(ranks)):
            assert_close(to_np(dA2[t]), rdA2[t], f"plain pool, shared plan: dA[{t}]")
            assert_close(to_np(dB2[t]), rdB2[t], f"plain pool, shared plan: dB[{t}]")
        rdx = 0.0
        for p in w2.projections:
            r, s, A, Bm = oracle.adapters_of(p)
            rdx = rdx + oracle.backward_dx(p.dy, p.W, r, s, A, Bm, ts)[0]
        assert_close(to_np(dxs), rdx, "pool over two projections, shared plan: dx")
        for pi, p in enumerate(w2.projections):
            r, s, A, Bm = oracle.adapters_of(p)
            rdA, rdB = oracle.backward_dAdB(p.x, p.dy, r, s, A, Bm, ts)
            for t in range(len(ranks)):
                assert_close(sc.split_dA(t, dAs[t])[pi], rdA[t], f"pool over two projections, shared plan: dA[{t}] of {pi}")
                assert_close(sc.split_dB(t, dBs[t])[pi], rdB[t], f"pool over two projections, shared plan: dB[{t}] of {pi}")
    B.marlaas_check_status(sc.pool)
    B.marlaas_check_status(dc.pool)


def _draw_seg(rng):
    kind = rng.choice(["decode", "mid", "train"])
    P = int(rng.integers(1, 5))
    Ns = tuple(256 * int(rng.integers(1, 4)) for _ in range(P))
    if kind == "decode":
        T, K = int(rng.integers(1, 257)), 64 * int(rng.integers(1, 7))
    elif kind == "mid":
        T, K = int(rng.integers(257, 1025)), 8 * int(rng.integers(4, 40))
    else:
        T, K = int(rng.integers(1024, 2300)), 8 * int(rng.integers(8, 40))
    n = int(rng.integers(1, 7))
    ranks = [int(rng.choice([0, 1, 4, 8, 16, 17, 32, 48, 64])) for _ in range(n)]
    if max(ranks) == 0:
        ranks[0] = 8
    return kind, T, K, Ns, ranks, int(rng.integers(1, 1 << 30)), bool(rng.integers(0, 2)), int(rng.integers(1, 10)), \
        int(rng.integers(0, 3)), bool(rng.integers(0, 2))


@pytest.mark.parametrize("batch", range(2))
def test_random_pools_over_several_projections_match_the_oracle(batch):
    # seeded random draws of the number and widths of the projections, token count, depth, rank mix (rank 0 and odd
    # ranks included), table form, spare capacity, backward with and without the saved h; every output against the
    # per-projection oracle runs
    rng = np.random.default_rng(77100 + batch)
    for ci in range(12):
        kind, T, K, Ns, ranks, seed, per_token, nseg, extra, use_saved = _draw_seg(rng)
        w = _case(seed % 100000, T, K, Ns, ranks, per_token, n_segments=nseg)
        tag = f"batch {batch} case {ci} ({kind}) T={T} K={K} Ns={Ns} ranks={ranks} per_token={per_token} seed={seed}"
        ts = w.tok_slot()
        sc = SegCase(w, capacity=len(ranks) + extra)
        P, n = len(Ns), len(ranks)
        hs = torch.full((P, T, sc.pool.rank_stride), 9.0, dtype=torch.float32, device="cuda:0")
        y = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, h_save=hs)
        ry, rh = _oracle_forward(w, ts)
        assert_close(to_np(y), ry, tag + ": y")
        for p in range(P):
            hr = np.zeros((T, sc.pool.rank_stride), np.float32)
            hr[:, :rh[p].shape[1]] = rh[p]
            assert_close(to_np(hs[p]), hr, tag + f": h_save of projection {p}", atol=1e-3, rtol=1e-3)
        dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda:0")
        dA, dB = sc.grads(fill=2.0)
        B.marlaas_lora_backward(sc.pool, sc.x, sc.W, sc.dy, sc.seg, dx=dx, dA=dA, dB=dB, h_saved=hs if use_saved else None)
        rdx = 0.0
        for pi, p in enumerate(w.projections):
            r, s, A, Bm = oracle.adapters_of(p)
            rdx = rdx + oracle.backward_dx(p.dy, p.W, r, s, A, Bm, ts)[0]
            rdA, rdB = oracle.backward_dAdB(p.x, p.dy, r, s, A, Bm, ts)
            for t in range(n):
                if ranks[t] > 0:
                    assert_close(sc.split_dA(t, dA[t])[pi], rdA[t], tag + f": dA[{t}] of projection {pi}")
                    assert_close(sc.split_dB(t, dB[t])[pi], rdB[t], tag + f": dB[{t}] of projection {pi}")
        assert_close(to_np(dx), rdx, tag + ": dx")
        B.marlaas_check_status(sc.pool)


def test_unregister_and_reregister_on_a_pool_over_two_projections():
    # a freed slot serves the base weight only on every projection; registering again (another rank) brings it back
    T, K, Ns, ranks = 180, 128, (256, 512), (16, 8, 32)
    w = _case(4100, T, K, Ns, ranks, True)
    ts = w.tok_slot()
    sc = SegCase(w, capacity=4)
    t0 = w.projections[0].adapters[0]
    B.marlaas_adapter_pool_unregister(sc.pool, t0.tenant_id)
    y = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg)
    ts_freed = np.where(ts == 0, -1, ts).astype(np.int32)
    assert_close(to_np(y), _oracle_forward(w, ts_freed)[0], "after unregister: slot 0 serves the base weight only")
    with pytest.raises(B.MarlaasError):
        B.marlaas_adapter_pool_lookup(sc.pool, t0.tenant_id)
    As = [dev_bf16(p.adapters[0].A_bits) for p in w.projections]
    Bs = [dev_bf16(p.adapters[0].B_bits) for p in w.projections]
    assert B.marlaas_adapter_pool_register(sc.pool, t0.tenant_id, 7, t0.rank, t0.alpha, As, Bs) == 0      # lowest free slot
    y2 = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg)
    assert_close(to_np(y2), _oracle_forward(w, ts)[0], "after registering again")
    assert B.marlaas_adapter_pool_lookup(sc.pool, t0.tenant_id)[3] == 7
    B.marlaas_check_status(sc.pool)


@pytest.mark.parametrize("T,K,Ns", [
    (96, 4096, (8192, 8192)),        # one tile per CTA pair, both projections' planes of hd
    (64, 2048, (9728, 9728)),        # more tiles than CTA pairs
    (200, 256, (512, 256, 256)),     # the token-major decode kernel
])
def test_overlapped_decode_calls_on_pools_over_several_projections(T, K, Ns):
    # MARLAAS_FLAG_OVERLAP_PREVIOUS on pools over several projections: two pools used in turn, bit-identical to serial calls
    w = _case(2300 + T, T, K, Ns, (16, 8, 32), True)
    cases = [SegCase(w, capacity=4) for _ in range(2)]
    ref = B.marlaas_lora_forward(cases[0].pool, cases[0].x, cases[0].W, cases[0].seg).clone()
    torch.cuda.synchronize()
    ys = [torch.empty_like(ref) for _ in range(6)]
    for j in range(6):
        c = cases[j % 2]
        B.marlaas_lora_forward(c.pool, c.x, c.W, c.seg, y=ys[j], flags=B.MARLAAS_FLAG_OVERLAP_PREVIOUS)
    torch.cuda.synchronize()
    for y in ys:
        assert torch.equal(y, ref)
    for c in cases:
        B.marlaas_check_status(c.pool)
