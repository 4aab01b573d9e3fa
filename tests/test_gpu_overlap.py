"""MARLAAS_FLAG_OVERLAP_PREVIOUS: decode-shaped forward calls whose predecessor on the stream is independent of them
(another micro-batch: its own pool, workspace and outputs) start their shrink beside the end of that predecessor.  The
results must be bit-identical to the same calls without the flag, whichever decode kernel serves the shape, with two
pools used in turn (the least the flag's condition allows) and with three; the entry points that cannot honour the flag
refuse it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu


def _case(seed, T, K, N, ranks):
    w = wl.small_random_case(seed, T, K, N, list(ranks), n_segments=min(9, T + 1))
    ts = wl.uniform_token_slots(seed, T, len(ranks)).astype(np.int32)
    ts[T // 2] = -1
    w.seg_offsets, w.seg_slot = wl.per_token_table(ts)
    return w


@pytest.mark.parametrize("seed,T,K,N,ranks,npools", [
    (901, 96, 512, 768, (16, 8, 32, 4), 2),          # the token-major decode kernel, two slices
    (902, 256, 4096, 4096, (16,) * 8, 3),            # the configured decode shape
    (903, 100, 4096, 11008, (16, 16, 8), 2),         # one tile per CTA pair, 128-token tiles
    (904, 90, 2048, 19200, (16, 8, 16, 32), 2),      # more tiles than CTA pairs
    (905, 70, 11008, 4096, (16, 32, 16), 3),         # four slices per tile
    (906, 300, 1024, 1024, (16, 16), 2),             # two token tiles
])
def test_overlapped_calls_are_bit_identical_to_serial_ones(seed, T, K, N, ranks, npools):
    w = _case(seed, T, K, N, ranks)
    p = w.projections[0]
    cases = [DeviceCase(w, p, capacity=len(ranks) + 1) for _ in range(npools)]
    ncall = 7
    xs = [torch.roll(cases[0].x, shifts=3 * j, dims=0).contiguous() for j in range(ncall)]
    # serial reference: the same calls, no flag, one at a time
    ref, ref_h = [], []
    for j in range(ncall):
        h = torch.empty((T, cases[0].pool.rank_stride), dtype=torch.float32, device="cuda:0")
        ref.append(cases[j % npools].forward(x=xs[j], h_save=h).clone())
        ref_h.append(h)
        torch.cuda.synchronize()
    r, s, A, Bm = oracle.adapters_of(p)
    ry, _ = oracle.forward(p.x, p.W, r, s, A, Bm, w.tok_slot())
    assert_close(to_np(ref[0]), ry, f"serial decode {T}x{K}x{N}")
    # back to back with the flag: call j runs beside the end of call j - 1, which uses another pool and workspace
    for rep in range(2):
        ys = [torch.empty((T, N), dtype=torch.bfloat16, device="cuda:0") for _ in range(ncall)]
        hs = [torch.empty((T, cases[0].pool.rank_stride), dtype=torch.float32, device="cuda:0") for _ in range(ncall)]
        for j in range(ncall):
            c = cases[j % npools]
            B.marlaas_lora_forward(c.pool, xs[j], c.W, c.seg, y=ys[j], h_save=hs[j], flags=B.MARLAAS_FLAG_OVERLAP_PREVIOUS)
        torch.cuda.synchronize()
        for j in range(ncall):
            assert torch.equal(ys[j], ref[j]), (rep, j)
            assert torch.equal(hs[j], ref_h[j]), (rep, j)
    for c in cases:
        B.marlaas_check_status(c.pool)


def test_overlapped_calls_inside_a_captured_graph():
    w = _case(911, 128, 4096, 4096, (16, 16, 16, 16))
    p = w.projections[0]
    cases = [DeviceCase(w, p, capacity=5) for _ in range(2)]
    ref = cases[0].forward().clone()
    ys = [torch.empty_like(ref) for _ in range(6)]
    for c in cases:
        c.forward()                                  # first calls (workspace allocation, attributes) outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for j in range(6):
                c = cases[j % 2]
                B.marlaas_lora_forward(c.pool, c.x, c.W, c.seg, y=ys[j], flags=B.MARLAAS_FLAG_OVERLAP_PREVIOUS)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        for y in ys:
            y.zero_()
        g.replay()
        torch.cuda.synchronize()
        for y in ys:
            assert torch.equal(y, ref)
    for c in cases:
        B.marlaas_check_status(c.pool)


def test_entry_points_that_cannot_honour_the_flag_refuse_it():
    w = _case(921, 64, 256, 256, (16, 8))
    dc = DeviceCase(w, w.projections[0], capacity=3)
    y = torch.empty((w.T, 256), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_lora_forward_static_ws(dc.pool, dc.x, dc.W, dc.seg, y, flags=B.MARLAAS_FLAG_OVERLAP_PREVIOUS)
    assert e.value.status == B.MARLAAS_ERR_INVALID_ARG
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_lora_forward_multi([dict(pool=dc.pool, x=dc.x, W=dc.W, seg=dc.seg)], flags=B.MARLAAS_FLAG_OVERLAP_PREVIOUS)
    assert e.value.status == B.MARLAAS_ERR_INVALID_ARG
    # a training-shaped batch ignores the flag
    w2 = wl.small_random_case(922, 1300, 128, 256, [16, 8], n_segments=5)
    d2 = DeviceCase(w2, w2.projections[0], capacity=3)
    assert torch.equal(d2.forward(), d2.forward(flags=B.MARLAAS_FLAG_OVERLAP_PREVIOUS))
