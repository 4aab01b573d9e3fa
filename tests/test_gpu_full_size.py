"""GPU parity at the full configured sizes, through the same calls bench.py times (forward with h_save, backward with
the saved h).  y and dx are checked, over all columns, on at least one token row of every 128-row block (the rows one
CTA of a 256-row tile owns, so every CTA of every tile of the launch has a checked row) plus the tile-edge rows; each
oracle row is computed on its own, from the definition.  The adapter gradients, which sum over every token of a
tenant, are checked in full, and one slow test checks every row of y at the largest size.  Index outputs are compared
bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu


def _sample_rows(T, n, seed):
    """Edge rows, one seeded row inside every 128-row block, and n more seeded rows anywhere."""
    edge = [0, 1, 63, 64, 127, 128, 255, 256, 257, T // 2, T - 257, T - 256, T - 129, T - 128, T - 2, T - 1]
    nblk = (T + 127) // 128
    off = (wl.hash_u64(seed, wl.TID_PERTURB, np.arange(nblk, dtype=np.uint64) + np.uint64(1 << 20)) % np.uint64(128)).astype(np.int64)
    per_block = np.minimum(np.arange(nblk, dtype=np.int64) * 128 + off, T - 1)
    rnd = (wl.hash_u64(seed, wl.TID_PERTURB, np.arange(n, dtype=np.uint64)) % np.uint64(T)).astype(np.int64)
    rows = sorted({int(r) for r in edge if 0 <= r < T} | {int(r) for r in per_block} | {int(r) for r in rnd})
    assert len({r // 128 for r in rows}) == nblk
    return np.array(rows, dtype=np.int64)


def _check_full(w, p, n_rows=40):
    ts = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    dc = DeviceCase(w, p)
    T, Tb = w.T, w.T_bwd
    hs = torch.empty((T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    y = dc.forward(h_save=hs)
    rows = _sample_rows(T, n_rows, 7 + len(p.name))
    ry, rh = oracle.forward(p.x[rows], p.W, r, s, A, Bm, ts[rows])
    assert_close(to_np(y[torch.from_numpy(rows).cuda()]), ry, f"{w.name}/{p.name} y (sampled rows)")
    hr = np.zeros((len(rows), dc.pool.rank_stride), np.float32)
    hr[:, :rh.shape[1]] = rh
    assert_close(to_np(hs[torch.from_numpy(rows).cuda()]), hr, f"{w.name}/{p.name} h_save (sampled rows)", atol=1e-3, rtol=1e-3)
    if Tb:
        seg = dc.seg if Tb == T else dc.seg_prefix(Tb)
        dx, dA, dB = dc.backward(seg=seg, T=Tb, h_saved=hs[:Tb])
        rb = rows[rows < Tb]
        rdx, _ = oracle.backward_dx(p.dy[rb], p.W, r, s, A, Bm, ts[rb])
        assert_close(to_np(dx[torch.from_numpy(rb).cuda()]), rdx, f"{w.name}/{p.name} dx (sampled rows)")
        rdA, rdB = oracle.backward_dAdB(p.x[:Tb], p.dy[:Tb], r, s, A, Bm, ts[:Tb])
        for t, a in enumerate(p.adapters):
            if a.rank > 0:
                assert_close(to_np(dA[t]), rdA[t], f"{w.name}/{p.name} dA[{t}]")
                assert_close(to_np(dB[t]), rdB[t], f"{w.name}/{p.name} dB[{t}]")
    exp = oracle.build_index(T, w.seg_offsets, w.seg_slot, dc.capacity)
    got = B.marlaas_lora_build_index(dc.pool, T, dc.seg)
    for g_, e, nm in zip(got, exp, ("tok_slot", "slot_count", "slot_offset", "perm")):
        assert np.array_equal(g_.cpu().numpy(), e), (w.name, nm)
    B.marlaas_check_status(dc.pool)


def test_cfg3_training_shaped_full_size():
    w = wl.make_workload(3)
    _check_full(w, w.projections[0])


@pytest.mark.slow
def test_cfg3_every_row_of_y():
    """All 16384 x 11008 outputs of the largest forward against the oracle (about a minute of host time)."""
    w = wl.make_workload(3)
    p = w.projections[0]
    ts = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    dc = DeviceCase(w, p)
    y = to_np(dc.forward())
    B.marlaas_check_status(dc.pool)
    step = 2048
    for r0 in range(0, w.T, step):
        ry, _ = oracle.forward(p.x[r0:r0 + step], p.W, r, s, A, Bm, ts[r0:r0 + step])
        assert_close(y[r0:r0 + step], ry, f"{w.name}/{p.name} y rows {r0}..{r0 + step - 1}")


def test_cfg4_heterogeneous_full_size():
    w = wl.make_workload(4)
    _check_full(w, w.projections[0])


def test_cfg5_decoder_layer_full_size():
    w = wl.make_workload(5)
    for p in w.projections:
        _check_full(w, p, n_rows=24)
        torch.cuda.empty_cache()


def _check_fused_full(w, names, n_rows=24):
    """Projections `names` of the layer through ONE pool over them, at the full size: sampled rows of y and dx over all
    columns, the adapter gradients of every projection in full."""
    import copy
    from test_gpu_segmented_pool import SegCase
    w2 = copy.copy(w)
    w2.projections = [p for p in w.projections if p.name in names]
    assert all(np.array_equal(p.x_bits, w2.projections[0].x_bits) for p in w2.projections)
    sc = SegCase(w2)
    ts = w.tok_slot()
    T, Tb, P = w.T, w.T_bwd, len(w2.projections)
    tag = f"{w.name}/{'+'.join(names)} through one pool"
    hs = torch.empty((P, T, sc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    y = B.marlaas_lora_forward(sc.pool, sc.x, sc.W, sc.seg, h_save=hs)
    rows = _sample_rows(T, n_rows, 11 + P)
    ridx = torch.from_numpy(rows).cuda()
    ry = []
    for pi, p in enumerate(w2.projections):
        r, s, A, Bm = oracle.adapters_of(p)
        yy, rh = oracle.forward(p.x[rows], p.W, r, s, A, Bm, ts[rows])
        ry.append(yy)
        hr = np.zeros((len(rows), sc.pool.rank_stride), np.float32)
        hr[:, :rh.shape[1]] = rh
        assert_close(to_np(hs[pi][ridx]), hr, f"{tag}: h_save of {p.name} (sampled rows)", atol=1e-3, rtol=1e-3)
    assert_close(to_np(y[ridx]), np.concatenate(ry, axis=1), f"{tag}: y (sampled rows)")
    if Tb:
        so, ss = w.seg_offsets, w.seg_slot
        keep = [s_ for s_ in range(len(ss)) if so[s_] < Tb]
        seg = B.Segments(torch.from_numpy(np.array([min(int(so[s_]), Tb) for s_ in keep] + [Tb], dtype=np.int32)).cuda(),
                         torch.from_numpy(np.array([ss[s_] for s_ in keep], dtype=np.int32)).cuda())
        dx = torch.empty((Tb, sc.K), dtype=torch.bfloat16, device="cuda:0")
        dA, dB = sc.grads()
        B.marlaas_lora_backward(sc.pool, sc.x[:Tb], sc.W, sc.dy[:Tb], seg, dx=dx, dA=dA, dB=dB, h_saved=hs[:, :Tb].contiguous())
        rb = rows[rows < Tb]
        rdx = 0.0
        for pi, p in enumerate(w2.projections):
            r, s, A, Bm = oracle.adapters_of(p)
            rdx = rdx + oracle.backward_dx(p.dy[rb], p.W, r, s, A, Bm, ts[rb])[0]
            rdA, rdB = oracle.backward_dAdB(p.x[:Tb], p.dy[:Tb], r, s, A, Bm, ts[:Tb])
            for t, a in enumerate(p.adapters):
                if a.rank > 0:
                    assert_close(sc.split_dA(t, dA[t])[pi], rdA[t], f"{tag}: dA[{t}] of {p.name}")
                    assert_close(sc.split_dB(t, dB[t])[pi], rdB[t], f"{tag}: dB[{t}] of {p.name}")
        assert_close(to_np(dx[torch.from_numpy(rb).cuda()]), rdx, f"{tag}: dx (sampled rows)")
    B.marlaas_check_status(sc.pool)


def test_cfg5_layer_through_pools_over_projections_full_size():
    # the configurations bench.py reports as cfg5-fused and cfg5-decode-fused: q, k, v and gate, up through one pool each,
    # on the mixed training + decode batch (forward over 4352 rows, backward over 4096) and on the 256 decode rows alone
    # (48 and 86 column strips: the one-tile-per-pair and the balanced decode kernels)
    w = wl.make_workload(5)
    for names in (("q", "k", "v"), ("gate", "up")):
        _check_fused_full(w, names)
        torch.cuda.empty_cache()
    wd = wl.make_variant("cfg5-decode", w)
    for names in (("q", "k", "v"), ("gate", "up")):
        _check_fused_full(wd, names, n_rows=64)
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name", [
    "decode5120x17408-256-32",     # 68 strips, one tile per CTA pair, 256-token tiles
    "decode5120x17408-64-32",      # the same weight with 64-token tiles
    "decode12288x4096-64-32",      # 16 strips, 64 tokens: the steps spread over all pairs, 4-5 pieces per tile
    "decode5120x25600-64-32",      # 100 strips on 74 pairs, 64-token tiles
])
def test_decode_over_wide_weights_every_row(name):
    # the decode configurations bench.py reports beside the configured workloads: every row of y against the oracle
    w = wl.make_named_workload(name)
    p = w.projections[0]
    ts = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    dc = DeviceCase(w, p)
    y = dc.forward()
    ry, _ = oracle.forward(p.x, p.W, r, s, A, Bm, ts)
    assert_close(to_np(y), ry, f"{name}: y (every row)")
    assert torch.equal(y, dc.forward())
    B.marlaas_check_status(dc.pool)
