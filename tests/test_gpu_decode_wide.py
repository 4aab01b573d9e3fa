"""GPU parity of the decode-shaped forward over large weights (the kernel with W columns on the MMA's M side), which
only weights of 64 MB and more reach: one case per way it cuts the contraction -- no split (33 or more tiles), two
slices and four slices (partial accumulators exchanged through the workspace), and more tiles than CTA pairs (the tiles'
steps spread evenly over all pairs, partial tiles summed by the pair holding a tile's last steps) -- each element-wise
against the oracle, plus repeated calls on one pool (the exchange flags carry an epoch from call to call) and bit-identity of two runs.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu


def _case(seed, T, K, N, ranks, per_token):
    w = wl.small_random_case(seed, T, K, N, list(ranks), n_segments=min(9, T + 1))
    if per_token:
        ts = wl.uniform_token_slots(seed, T, len(ranks)).astype(np.int32)
        ts[T // 3] = -1                                   # one token served by the base weight only
        w.seg_offsets, w.seg_slot = wl.per_token_table(ts)
    return w


@pytest.mark.parametrize("seed,T,K,N,ranks,per_token", [
    (801, 100, 4096, 11008, (16, 16, 8, 16, 4), True),     # 43 tiles: no split; last strip complete, ragged token tile
    (802, 70, 11008, 4096, (16, 32, 16), True),            # 16 tiles: four slices of 43 steps each (uneven: 172 = 4 x 43)
    (803, 300, 11008, 4096, (16, 8, 16, 16), False),       # 2 x 16 tiles: two slices; second token tile has 44 rows
    (804, 256, 4096, 8200, (16, 16, 16, 16, 16, 16), True),   # 33 tiles; N not a multiple of 64: per-chunk copies, 8-column tail
    (805, 90, 2048, 19200, (16, 8, 16, 32), True),         # 75 tiles on 74 pairs: every pair but the first cuts a tile
    (806, 257, 4096, 11008, (16, 16, 8, 16), False),       # 2 x 43 tiles; the second token tile has one row
    (807, 40, 1664, 24584, (16, 16), True),                # 97 tiles, N not a multiple of 64, K / 64 = 26 steps: pairs span 2-3 tiles
    (808, 40, 16384, 4864, (16, 8, 16), True),             # 19 tiles, 256 steps each, spread over 74 pairs: 3-5 pieces per tile
    (809, 40, 4096, 13312, (16, 8, 16, 4), True),          # 52 tiles, no split, 64-token tiles: the second CTA's rows 32..39 only
    (810, 64, 4096, 12808, (16, 16, 32), True),            # 51 tiles of 64 tokens, all rows; N not a multiple of 64
    (811, 17, 4096, 14336, (16, 16), True),                # 56 tiles of 64 tokens whose second half holds no token at all
    (812, 128, 4096, 11008, (16, 8, 16, 16), False),       # 128-token tiles, every row a token
    (813, 17, 4096, 11008, (16, 16), True),                # 43 tiles, up to 64 tokens: steps spread over all pairs, 1-2 pieces per tile
    (814, 64, 11008, 4096, (16, 8, 32), False),            # 16 tiles, 64 tokens: 4-5 pieces per tile
    (815, 150, 4096, 11008, (16, 8, 16), True),            # 43 tiles of 192 tokens (96 per CTA; the second CTA's last 42 rows empty)
    (816, 190, 2048, 19200, (16, 16, 8), True),            # 75 tiles of 192 tokens on 74 pairs
])
def test_decode_over_large_weights_matches_the_oracle(seed, T, K, N, ranks, per_token):
    w = _case(seed, T, K, N, ranks, per_token)
    p = w.projections[0]
    ts = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    ry, rh = oracle.forward(p.x, p.W, r, s, A, Bm, ts)
    dc = DeviceCase(w, p, capacity=len(ranks) + 1)
    hs = torch.full((T, dc.pool.rank_stride), 7.0, dtype=torch.float32, device="cuda:0")
    y1 = dc.forward(h_save=hs)
    assert_close(to_np(y1), ry, f"large-weight decode {T}x{K}x{N}: y")
    hr = np.zeros((T, dc.pool.rank_stride), np.float32)
    hr[:, :rh.shape[1]] = rh
    assert_close(to_np(hs), hr, f"large-weight decode {T}x{K}x{N}: h_save", atol=1e-3, rtol=1e-3)
    # again on the same pool and workspace (the exchange flags of the first call are still there), and once more
    # after a call on different activations: every call must stand on its own and repeat bit for bit
    y2 = dc.forward()
    assert torch.equal(y1, y2)
    x3 = torch.flip(dc.x, dims=[0]).contiguous()
    y3 = dc.forward(x=x3)
    y4 = dc.forward()
    assert torch.equal(y1, y4) and not torch.equal(y1, y3)
    ry3, _ = oracle.forward(p.x[::-1], p.W, r, s, A, Bm, ts)
    assert_close(to_np(y3), ry3, f"large-weight decode {T}x{K}x{N}: y of the second batch")
    B.marlaas_check_status(dc.pool)
