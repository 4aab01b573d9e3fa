"""GPU parity on seeded random shapes: token counts, dimensions, rank mixes (rank 0 and odd ranks included), segment
tables (coarse segments or one token per segment with a base-only token) drawn so that every kernel family is hit
-- the two-kernel decode path (up to 1024 tokens, K a multiple of 64), the 1-CTA and 2-CTA GEMM paths, the
tensor-core and CUDA-core reductions, backward with and without the saved h (side-stream and in-order forms).
Forward, saved h, dx, dA and dB are compared element by element with the oracle at the layer's tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu


def _draw(rng):
    kind = rng.choice(["decode", "mid", "train", "odd"])
    if kind == "decode":
        T, K, N = int(rng.integers(1, 257)), 64 * int(rng.integers(1, 9)), 8 * int(rng.integers(8, 100))
    elif kind == "mid":
        T, K, N = int(rng.integers(257, 1025)), 64 * int(rng.integers(1, 7)), 8 * int(rng.integers(8, 80))
    elif kind == "train":
        T, K, N = int(rng.integers(1024, 2600)), 8 * int(rng.integers(8, 60)), 8 * int(rng.integers(8, 60))
    else:
        T, K, N = int(rng.integers(1, 1500)), 8 * int(rng.integers(1, 40)), 8 * int(rng.integers(1, 40))
    n = int(rng.integers(1, 9))
    ranks = [int(rng.choice([0, 1, 3, 4, 8, 16, 17, 32, 48, 64])) for _ in range(n)]
    if max(ranks) == 0:
        ranks[0] = 8
    return kind, T, K, N, ranks, int(rng.integers(1, 1 << 30)), bool(rng.integers(0, 2)), int(rng.integers(1, 12)), \
        int(rng.integers(0, 3)), bool(rng.integers(0, 2))


@pytest.mark.parametrize("batch", range(4))
def test_random_shapes_match_the_oracle(batch):
    rng = np.random.default_rng(20260 + batch)
    for ci in range(20):
        kind, T, K, N, ranks, seed, per_token, nseg, extra, use_saved = _draw(rng)
        w = wl.small_random_case(seed, T, K, N, ranks, n_segments=nseg)
        if per_token:
            ts = wl.uniform_token_slots(seed, T, len(ranks)).astype(np.int32)
            ts[seed % T] = -1
            w.seg_offsets, w.seg_slot = wl.per_token_table(ts)
        p = w.projections[0]
        tag = f"batch {batch} case {ci} ({kind}) T={T} K={K} N={N} ranks={ranks} per_token={per_token} seed={seed}"
        ts = w.tok_slot()
        r, s, A, Bm = oracle.adapters_of(p)
        dc = DeviceCase(w, p, capacity=len(ranks) + extra)
        hs = torch.full((T, dc.pool.rank_stride), 9.0, dtype=torch.float32, device="cuda:0")
        y = dc.forward(h_save=hs)
        ry, rh = oracle.forward(p.x, p.W, r, s, A, Bm, ts)
        assert_close(to_np(y), ry, tag + ": y")
        hr = np.zeros((T, dc.pool.rank_stride), np.float32)
        hr[:, :rh.shape[1]] = rh
        assert_close(to_np(hs), hr, tag + ": h_save", atol=1e-3, rtol=1e-3)
        dx, dA, dB = dc.backward(h_saved=hs if use_saved else None)
        rdx, _ = oracle.backward_dx(p.dy, p.W, r, s, A, Bm, ts)
        rdA, rdB = oracle.backward_dAdB(p.x, p.dy, r, s, A, Bm, ts)
        assert_close(to_np(dx), rdx, tag + ": dx")
        for t, a in enumerate(p.adapters):
            if a.rank > 0:
                assert_close(to_np(dA[t]), rdA[t], tag + f": dA[{t}]")
                assert_close(to_np(dB[t]), rdB[t], tag + f": dB[{t}]")
        B.marlaas_check_status(dc.pool)
