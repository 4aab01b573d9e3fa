"""The seeded input generators (no GPU): named workloads are reproducible, well formed and shaped as documented."""
import numpy as np
import pytest

from paper_2605_08527_b200 import workloads as wl


def _well_formed(w):
    off, sl = w.seg_offsets, w.seg_slot
    assert off[0] == 0 and off[-1] == w.T and len(off) == len(sl) + 1
    assert np.all(np.diff(off) >= 0)
    assert sl.min() >= -1 and sl.max() < w.n_tenants
    ts = w.tok_slot()
    assert ts.shape == (w.T,)
    return ts


def test_decode_sweep_point_is_one_token_per_segment_and_uniform_over_tenants():
    w = wl.make_named_workload("decode-512-8")
    ts = _well_formed(w)
    assert w.T == 512 and w.T_bwd == 0 and len(w.seg_slot) == 512 and w.n_tenants == 8
    assert set(np.unique(ts)) == set(range(8))                      # every tenant appears
    assert not np.all(np.diff(ts) >= 0)                             # unsorted
    p = w.projections[0]
    assert (p.d_in, p.d_out) == (4096, 4096) and all(a.rank == 16 for a in p.adapters) and p.dy_bits is None
    again = wl.make_named_workload("decode-512-8")
    assert np.array_equal(again.seg_slot, w.seg_slot) and np.array_equal(again.projections[0].x_bits[:4], p.x_bits[:4])


def test_prefill_sweep_point_has_whole_prompt_segments():
    w = wl.make_named_workload("prefill-8192-8")
    _well_formed(w)
    lens = np.diff(w.seg_offsets)
    assert w.T == 8192 and w.T_bwd == 0
    assert lens.min() >= 128 and lens.max() <= 4096 + 127           # clipped lognormal; the last may absorb a short tail
    assert len(lens) < 64


def test_named_workload_covers_the_configs_and_rejects_other_names():
    assert wl.make_named_workload("cfg1").name == wl.make_workload(1).name
    for bad in ("cfg", "decode-0-4", "decode-16", "prefill-64-0", "train-64-4"):
        with pytest.raises(ValueError):
            wl.make_named_workload(bad)


def test_decode_sweep_point_over_another_weight_shape():
    w = wl.make_named_workload("decode512x768-48-4")
    _well_formed(w)
    p = w.projections[0]
    assert (p.d_in, p.d_out) == (512, 768) and w.T == 48 and w.T_bwd == 0 and p.x_bits.shape == (48, 512)
    for bad in ("decode512x-48-4", "decode513x768-48-4", "decodex768-48-4"):
        with pytest.raises(ValueError):
            wl.make_named_workload(bad)


def test_layer_through_pools_over_projections_keeps_the_tensors_of_the_separate_projections():
    # a scaled-down 7-projection layer: q, k, v and gate, up as one projection each, o and down as they are
    w = wl.make_workload(5, scale_down=8)
    f = wl._fuse_layer(w, "fused")
    _well_formed(f)
    by = {p.name: p for p in w.projections}
    assert [p.name for p in f.projections] == ["q+k+v", "o", "gate+up", "down"]
    qkv, gu = f.projections[0], f.projections[2]
    assert qkv.parts == [by[n].d_out for n in "qkv"] and qkv.d_out == sum(qkv.parts)
    assert gu.parts == [by["gate"].d_out, by["up"].d_out]
    assert np.array_equal(qkv.W_bits, np.concatenate([by[n].W_bits for n in "qkv"], axis=1))
    assert np.array_equal(qkv.dy_bits, np.concatenate([by[n].dy_bits for n in "qkv"], axis=1))
    r = by["q"].adapters[0].rank
    a = qkv.adapters[0]
    assert a.rank == r and a.alpha == by["q"].adapters[0].alpha            # rank and scale of ONE projection
    assert a.A_bits.shape == (qkv.d_in, 3 * r) and a.B_bits.shape == (r, qkv.d_out)
    assert np.array_equal(a.A_bits[:, r:2 * r], by["k"].adapters[0].A_bits)
    assert np.array_equal(a.B_bits[:, qkv.parts[0]:qkv.parts[0] + qkv.parts[1]], by["k"].adapters[0].B_bits)
    # the block-diagonal form of the same projections, for comparison: rank 3 r, zeros off the diagonal
    d = wl.fuse_projections(w, ["q", "k", "v"]).projections[0]
    assert d.parts is None and d.adapters[0].rank == 3 * r and d.adapters[0].B_bits.shape == (3 * r, qkv.d_out)
    assert not d.adapters[0].B_bits[:r, qkv.parts[0]:].any()
