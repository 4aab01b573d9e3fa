"""The oracle against its own stored values on cfg1 (tests/golden/cfg1_oracle_values.txt, written by
tests/golden/make_golden.py from the seeded inputs and oracle/ alone): a change to the oracle's arithmetic or to the input
generators shows up here and has to be justified.  The GPU case checks the CUDA path against the same stored numbers."""
import importlib.util
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
GOLDEN = os.path.join(HERE, "golden", "cfg1_oracle_values.txt")


def _maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


def _stored():
    shapes, sums, points = {}, {}, {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if f[1] == "shape":
            shapes[f[0]] = tuple(int(v) for v in f[2:])
        elif f[1] == "sum":
            sums[f[0]] = float(f[2])
        else:
            points.setdefault(f[0], []).append((tuple(int(v) for v in f[2:-1]), float(f[-1])))
    return shapes, sums, points


def test_oracle_reproduces_its_stored_values():
    shapes, sums, points = _stored()
    vals = _maker().oracle_values()
    assert set(vals) == set(shapes) and {"y", "h", "dx", "g"} <= set(shapes)
    for name, (arr, _) in vals.items():
        assert arr.shape == shapes[name], name
        scale = 1.0 + float(np.abs(arr).sum())
        assert abs(float(arr.sum()) - sums[name]) <= 1e-12 * scale, name      # float64 sums in another thread order
        assert len(points[name]) == 6
        for ix, v in points[name]:
            assert abs(float(arr[ix]) - v) <= 1e-12 * (1.0 + abs(v)), (name, ix)


def test_stored_file_is_what_the_script_writes():
    assert [l.split()[:2] for l in _maker().lines()] == [l.split()[:2] for l in open(GOLDEN).read().splitlines()]


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_oracle_values():
    import torch
    from paper_2605_08527_b200 import workloads as wl
    from helpers import DeviceCase, to_np, TOL_ABS, TOL_REL
    shapes, _, points = _stored()
    w = wl.make_workload(1)
    p = w.projections[0]
    dc = DeviceCase(w, p)
    hs = torch.empty((w.T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    y = to_np(dc.forward(h_save=hs))
    dx, dA, dB = dc.backward(h_saved=hs)
    got = {"y": y, "dx": to_np(dx), "h": to_np(hs)}
    for t in range(len(p.adapters)):
        if dA[t] is not None:
            got[f"dA[{t}]"], got[f"dB[{t}]"] = to_np(dA[t]), to_np(dB[t])
    checked = 0
    for name, arr in got.items():
        if name not in points:
            continue
        # the layer's tolerance, as in the element-wise parity tests (the saved h is fp32: the tighter bound used there)
        atol, rtol = (1e-3, 1e-3) if name == "h" else (TOL_ABS, TOL_REL)
        for ix, v in points[name]:
            assert abs(float(arr[ix]) - v) <= atol + rtol * abs(v), (name, ix, float(arr[ix]), v)
            checked += 1
    assert checked >= 30
