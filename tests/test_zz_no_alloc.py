"""The allocation-free forward entry point against the regular one.

Collected last on purpose (file name): a run that stops at the first failure has then already run every other test.
Some users of the layer cannot allocate device memory -- their memory pool is frozen once serving starts, or they
are a plug-in that only ever sees its input and output buffers -- so marlaas_lora_forward_static_ws takes its
scratch from an array built into the library.  It must give what marlaas_lora_forward gives with a caller
workspace, call after call, although the built-in array still holds the previous call's intermediates.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, to_np

pytestmark = pytest.mark.gpu


def _run_both(dc, w, x):
    y_ref = B.marlaas_lora_forward(dc.pool, x, dc.W, dc.seg)
    h_ref = torch.empty((w.T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    B.marlaas_lora_forward(dc.pool, x, dc.W, dc.seg, h_save=h_ref)
    y = torch.full((w.T, dc.p.d_out), 3.0, dtype=torch.bfloat16, device="cuda:0")
    h = torch.full((w.T, dc.pool.rank_stride), 5.0, dtype=torch.float32, device="cuda:0")
    B.marlaas_lora_forward_static_ws(dc.pool, x, dc.W, dc.seg, y, h_save=h)
    B.marlaas_check_status(dc.pool)
    return y_ref, h_ref, y, h


def test_static_workspace_forward_matches_regular_forward_twice_in_a_row():
    # decode-shaped batch at reduced width: 64 unsorted tokens, 8 tenants of mixed rank, one base-only token
    w = wl.small_random_case(91, 64, 256, 320, [16, 8, 32, 4, 16, 16, 8, 2], n_segments=9)
    ts = wl.uniform_token_slots(91, 64, 8).astype(np.int32)
    ts[5] = -1
    w.seg_offsets, w.seg_slot = wl.per_token_table(ts)
    dc = DeviceCase(w, w.projections[0], capacity=10)
    assert B.marlaas_lora_forward_workspace_bytes(dc.pool, w.T) <= B.marlaas_lora_static_workspace_limit()

    # first call, then a second one on different activations: the array still holds the first call's contents
    y_ref1, h_ref1, y1, h1 = _run_both(dc, w, dc.x)
    x2 = torch.flip(dc.x, dims=[0]).contiguous()
    y_ref2, h_ref2, y2, h2 = _run_both(dc, w, x2)
    # Both entry points run the same deterministic kernels (every sum has a fixed order), so the results must agree
    # bit for bit, not merely within the layer's tolerance.
    for tag, (yr, hr, y, h) in {"first": (y_ref1, h_ref1, y1, h1), "second": (y_ref2, h_ref2, y2, h2)}.items():
        assert torch.equal(y, yr), f"static-workspace forward, {tag} call: y differs from the regular entry point"
        assert torch.equal(h, hr), f"static-workspace forward, {tag} call: h_save differs from the regular entry point"
    assert not torch.equal(y1, y2)      # the two calls really computed different batches

    # one comparison with the oracle, so that the pair of entry points is not only checked against itself
    p = dc.p
    r, s, A, Bm = oracle.adapters_of(p)
    ry, rh = oracle.forward(p.x, p.W, r, s, A, Bm, ts.astype(np.int64))
    assert_close(to_np(y1), ry, "static-workspace forward vs oracle: y")
    hr = np.zeros((w.T, dc.pool.rank_stride), np.float32)
    hr[:, :rh.shape[1]] = rh
    assert_close(to_np(h1), hr, "static-workspace forward vs oracle: h_save", atol=1e-3, rtol=1e-3)

    # a call after the first one on this device takes no device memory: the driver's free-byte count is unchanged
    # (torch's own allocations for the outputs come from its cache, warmed by the first pair of calls)
    y3 = torch.empty_like(y2)
    torch.cuda.synchronize()
    free_mid = torch.cuda.mem_get_info()[0]
    B.marlaas_lora_forward_static_ws(dc.pool, x2, dc.W, dc.seg, y3)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_mid, "the static-workspace call changed the device's free memory"
    assert torch.equal(y3, y2)


def test_static_workspace_rejects_batches_beyond_its_size():
    w = wl.small_random_case(92, 64, 64, 64, [64] * 4, n_segments=4)
    dc = DeviceCase(w, w.projections[0], capacity=64, max_rank=64)
    T_big = 4096
    assert B.marlaas_lora_forward_workspace_bytes(dc.pool, T_big) > B.marlaas_lora_static_workspace_limit()
    x = torch.zeros((T_big, 64), dtype=torch.bfloat16, device="cuda:0")
    y = torch.empty((T_big, 64), dtype=torch.bfloat16, device="cuda:0")
    seg = B.Segments(torch.tensor([0, T_big], dtype=torch.int32, device="cuda:0"),
                     torch.tensor([0], dtype=torch.int32, device="cuda:0"))
    n0 = B.marlaas_kernel_launch_count()
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_lora_forward_static_ws(dc.pool, x, dc.W, seg, y)
    assert e.value.status == B.MARLAAS_ERR_WORKSPACE_TOO_SMALL
    assert B.marlaas_kernel_launch_count() == n0      # nothing was launched
