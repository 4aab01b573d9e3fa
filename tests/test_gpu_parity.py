"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on identical seeded inputs.

Bar: integer / index outputs bit-exact; floating-point outputs within |gpu - ref| <= 1e-2 + 1e-2 |ref| per
element (bf16 inputs, fp32 accumulation), the tolerance stated for this layer.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08527_b200 import binding as B
from paper_2605_08527_b200 import workloads as wl

from helpers import DeviceCase, assert_close, dev_bf16, to_np

pytestmark = pytest.mark.gpu


def _oracle_all(w, p, T_bwd=None):
    ts = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    y, h = oracle.forward(p.x, p.W, r, s, A, Bm, ts)
    out = {"y": y, "h": h, "ts": ts}
    if p.dy_bits is not None:
        Tb = p.dy.shape[0] if T_bwd is None else T_bwd
        out["dx"], out["g"] = oracle.backward_dx(p.dy[:Tb], p.W, r, s, A, Bm, ts[:Tb])
        out["dA"], out["dB"] = oracle.backward_dAdB(p.x[:Tb], p.dy[:Tb], r, s, A, Bm, ts[:Tb])
    return out


def _check_case(w, p, flags=0, capacity=None, max_rank=None):
    ref = _oracle_all(w, p, w.T_bwd if w.T_bwd else None)
    dc = DeviceCase(w, p, capacity=capacity, max_rank=max_rank)
    hs = torch.full((w.T, dc.pool.rank_stride), 7.0, dtype=torch.float32, device="cuda:0")
    y = dc.forward(flags=flags, h_save=hs)
    assert_close(to_np(y), ref["y"], f"{w.name}/{p.name} y")
    hr = np.zeros((w.T, dc.pool.rank_stride), np.float32)
    hr[:, :ref["h"].shape[1]] = ref["h"]
    assert_close(to_np(hs), hr, f"{w.name}/{p.name} h_save", atol=1e-3, rtol=1e-3)
    if p.dy_bits is not None:
        Tb = p.dy.shape[0]
        seg = dc.seg if Tb == w.T else dc.seg_prefix(Tb)
        dx, dA, dB = dc.backward(flags=flags, seg=seg, T=Tb)
        assert_close(to_np(dx), ref["dx"], f"{w.name}/{p.name} dx")
        for t, a in enumerate(p.adapters):
            if a.rank > 0:
                assert_close(to_np(dA[t]), ref["dA"][t], f"{w.name}/{p.name} dA[{t}]")
                assert_close(to_np(dB[t]), ref["dB"][t], f"{w.name}/{p.name} dB[{t}]")
        # reuse of the saved h must give the same dB
        _, _, dB2 = dc.backward(flags=flags, seg=seg, T=Tb, h_saved=hs[:Tb].contiguous(), want_dx=False)
        for t, a in enumerate(p.adapters):
            if a.rank > 0:
                assert_close(to_np(dB2[t]), ref["dB"][t], f"{w.name}/{p.name} dB[{t}] (saved h)")
    B.marlaas_check_status(dc.pool)
    return dc, ref


@pytest.mark.parametrize("flags", [0, B.MARLAAS_FLAG_CUDA_CORE_PATH])
def test_cfg1_tiny_forward_backward(flags):
    w = wl.make_workload(1)
    _check_case(w, w.projections[0], flags=flags)


@pytest.mark.parametrize("flags", [0, B.MARLAAS_FLAG_CUDA_CORE_PATH])
@pytest.mark.parametrize("seed,T,K,N,ranks", [
    (1, 37, 24, 40, (3, 1, 5, 2)),            # tiny, odd token count, dims multiples of 8 only
    (2, 300, 136, 264, (8, 16, 32, 64)),      # ragged tails in every dimension, mixed ranks
    (3, 129, 512, 72, (16, 16, 7)),           # one token past a 128-row tile
    (4, 1, 64, 64, (4,)),                     # single token
    (5, 640, 200, 328, (64, 33, 1, 12, 9)),   # several row tiles, odd ranks
    (6, 1100, 264, 392, (16, 8, 32, 5)),      # 2-CTA tiles with ragged tails in rows, columns and depth
    (7, 1290, 128, 136, (8, 64)),             # second CTA of the last pair has only 10 rows; its column half is empty
])
def test_small_ragged_cases(flags, seed, T, K, N, ranks):
    w = wl.small_random_case(seed, T, K, N, list(ranks), n_segments=min(9, T + 1))
    _check_case(w, w.projections[0], flags=flags, capacity=len(ranks) + 2)


@pytest.mark.parametrize("seed,T,K,N,ranks", [
    # 5 x 16 = 80 tiles on 74 CTA pairs in forward and in dx: a second, nearly empty round.  Depths not multiples of 64
    # (one panel per step); last tile of y: 160 columns, of dx: 200
    (61, 1280, 4040, 4000, (16, 8, 32)),
    # depths in whole panels (two per step); last tile of y has 64 columns, of dx 192
    (62, 1280, 4032, 3904, (16, 16, 64, 4)),
    # 9 x 9 = 81 tiles forward (7 in the last round), dx in a single round; 10 rows in the last row tile
    (63, 2058, 1024, 2304, (32, 8)),
])
def test_more_tiles_than_cta_pairs_with_ragged_edges(seed, T, K, N, ranks):
    w = wl.small_random_case(seed, T, K, N, list(ranks), n_segments=9)
    _check_case(w, w.projections[0], capacity=len(ranks) + 1)


def test_finely_interleaved_tenants_with_backward():
    # every token its own segment, tenants drawn uniformly: the per-block tenant copies of the tensor-core gradient
    # reduction do not fit, so the device-side switch to the CUDA-core reduction is exercised
    T, n = 700, 12
    w = wl.small_random_case(61, T, 128, 136, [8] * n, n_segments=4)
    w.seg_offsets, w.seg_slot = wl.per_token_table(wl.uniform_token_slots(61, T, n))
    _check_case(w, w.projections[0])


@pytest.mark.parametrize("K,N", [(64, 64), (128, 320), (256, 320), (320, 1024)])
def test_decode_shallow_contraction_repeated_calls(K, N):
    # few 64-deep blocks of K: the decode GEMM may not cut the contraction into more slices than it has steps, and a
    # second call on other activations must not see anything the first one left in tensor memory
    w = wl.small_random_case(33 + K, 96, K, N, [16, 8, 32, 4], n_segments=9)
    w.seg_offsets, w.seg_slot = wl.per_token_table(wl.uniform_token_slots(33 + K, 96, 4))
    p = w.projections[0]
    dc = DeviceCase(w, p, capacity=6)
    ts = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    for rep in range(3):
        xs = np.roll(p.x_bits, 7 * rep, axis=0)
        ref, _ = oracle.forward(wl.bf16_bits_to_f32(xs), p.W, r, s, A, Bm, ts)
        y = dc.forward(x=dev_bf16(xs))
        assert_close(to_np(y), ref, f"decode K={K} N={N} call {rep}")
    B.marlaas_check_status(dc.pool)


def test_cfg2_decode_full_size():
    w = wl.make_workload(2)
    dc, _ = _check_case(w, w.projections[0])
    # the forward of this batch is two kernels (shrink, and the GEMM launched as its programmatic dependent)
    n0 = B.marlaas_kernel_launch_count()
    dc.forward()
    assert B.marlaas_kernel_launch_count() - n0 == 2


@pytest.mark.parametrize("T,K,N,ranks,cap", [
    (256, 256, 512, (32, 8, 17, 0, 32, 5), 8),      # mixed ranks over two 16-rank units; a rank-0 tenant; unused slots
    (100, 192, 384, (16, 16, 16), 3),               # second half of the 256-token tile empty
    (200, 128, 200, (64, 1, 40), 4),                # ragged last strip; four units per tenant
    (256, 512, 128, (16,) * 12, 12),                # a single 128-column strip
    (300, 128, 384, (16, 8), 2),                    # two 256-token tiles, the second with 44 rows
    (777, 192, 320, (32,), 1),                      # one tenant: its 16-token passes are shared by several clusters
    (1024, 256, 512, (16, 16, 16), 3),              # four full token tiles
])
def test_decode_mixed_ranks_and_base_only_tokens(T, K, N, ranks, cap):
    # decode-shaped batches with base-only tokens, tenants of several rank units and repeated calls on changing
    # activations, y and the saved h both checked
    w = wl.small_random_case(400 + T + N, T, K, N, list(ranks), n_segments=9)
    ts = wl.uniform_token_slots(400 + T + N, T, len(ranks)).astype(np.int32)
    ts[::11] = -1
    w.seg_offsets, w.seg_slot = wl.per_token_table(ts)
    p = w.projections[0]
    dc = DeviceCase(w, p, capacity=cap)
    tsl = w.tok_slot()
    r, s, A, Bm = oracle.adapters_of(p)
    for rep in range(3):
        xs = np.roll(p.x_bits, 5 * rep, axis=0)
        ref, rh = oracle.forward(wl.bf16_bits_to_f32(xs), p.W, r, s, A, Bm, tsl)
        hs = torch.full((T, dc.pool.rank_stride), 7.0, dtype=torch.float32, device="cuda:0")
        y = dc.forward(x=dev_bf16(xs), h_save=hs)
        assert_close(to_np(y), ref, f"decode units T={T} N={N} call {rep}: y")
        hr = np.zeros((T, dc.pool.rank_stride), np.float32)
        hr[:, :rh.shape[1]] = rh
        assert_close(to_np(hs), hr, f"decode units T={T} N={N} call {rep}: h_save", atol=1e-3, rtol=1e-3)
    B.marlaas_check_status(dc.pool)


@pytest.mark.parametrize("cfg,sd", [(3, 8), (4, 8), (5, 8)])
def test_scaled_down_configs(cfg, sd):
    w = wl.make_workload(cfg, scale_down=sd)
    for p in w.projections:
        _check_case(w, p)


def test_index_build_bit_exact():
    cases = [wl.make_workload(c, scale_down=4) for c in (2, 3, 4, 5)]
    cases.append(wl.small_random_case(8, 1000, 64, 64, [4, 4, 4, 4, 4, 4, 4], n_segments=40))
    for w in cases:
        p = w.projections[0]
        dc = DeviceCase(w, p, capacity=len(p.adapters) + 3)
        exp = oracle.build_index(w.T, w.seg_offsets, w.seg_slot, dc.capacity)
        for seg in (dc.seg, dc.seg_host):
            got = B.marlaas_lora_build_index(dc.pool, w.T, seg)
            torch.cuda.synchronize()
            for g, e, nm in zip(got, exp, ("tok_slot", "slot_count", "slot_offset", "perm")):
                assert np.array_equal(g.cpu().numpy(), e), (w.name, nm)
        B.marlaas_check_status(dc.pool)
    # zero-length segments and an empty batch
    w = wl.small_random_case(3, 50, 64, 64, [4, 4, 4], n_segments=5)
    dc = DeviceCase(w, w.projections[0])
    so = np.array([0, 0, 10, 10, 10, 31, 50, 50], np.int32)
    ss = np.array([1, 0, 2, -1, 1, 0, 2], np.int32)
    exp = oracle.build_index(50, so, ss, dc.capacity)
    got = B.marlaas_lora_build_index(dc.pool, 50, B.Segments(torch.from_numpy(so).cuda(), torch.from_numpy(ss).cuda()))
    for g, e in zip(got, exp):
        assert np.array_equal(g.cpu().numpy(), e)
    got = B.marlaas_lora_build_index(dc.pool, 0, B.Segments(torch.zeros(1, dtype=torch.int32).cuda(),
                                                           torch.zeros(0, dtype=torch.int32).cuda()))
    assert got[0].numel() == 0 and int(got[2][-1]) == 0 and int(got[1].sum()) == 0


@pytest.mark.parametrize("flags", [0, B.MARLAAS_FLAG_CUDA_CORE_PATH])
def test_P1_zero_B_is_bit_identical_to_base_only(flags):
    w = wl.small_random_case(21, 333, 256, 320, [8, 16, 32], n_segments=7)
    p = w.projections[0]
    for a in p.adapters:
        a.B_bits = np.zeros_like(a.B_bits)
    dc = DeviceCase(w, p)
    y0 = dc.forward(flags=flags)
    base = B.Segments(torch.tensor([0, w.T], dtype=torch.int32).cuda(), torch.tensor([-1], dtype=torch.int32).cuda())
    yb = dc.forward(flags=flags, seg=base)
    assert torch.equal(y0.view(torch.int16), yb.view(torch.int16))
    dx0, dA0, _ = dc.backward(flags=flags)
    dxb, _, _ = dc.backward(flags=flags, seg=base)
    assert torch.equal(dx0.view(torch.int16), dxb.view(torch.int16))
    assert all(float(a.abs().max()) == 0.0 for a in dA0 if a is not None)
    # second opinion on the base product from a library GEMM (not the oracle)
    ref = (dc.x.float() @ dc.W.float())
    assert_close(to_np(yb), to_np(ref), "base GEMM vs torch.matmul")


@pytest.mark.parametrize("flags", [0, B.MARLAAS_FLAG_CUDA_CORE_PATH])
def test_P7_routing_probe_exact(flags):
    T, K, N, n = 200, 64, 72, 5
    w = wl.small_random_case(13, T, K, N, [1] * n, n_segments=12)
    p = w.projections[0]
    p.W_bits = np.zeros_like(p.W_bits)
    xb = np.zeros((T, K), np.float32)
    xb[np.arange(T), np.arange(T) % K] = 1.0
    p.x_bits = wl.f32_to_bf16_bits(xb)
    dyv = np.zeros((T, N), np.float32)
    dyv[:, 5] = 1.0
    p.dy_bits = wl.f32_to_bf16_bits(dyv)
    for t, a in enumerate(p.adapters):
        a.alpha = 1.0
        a.A_bits = wl.f32_to_bf16_bits(np.ones((K, 1), np.float32))
        a.B_bits = wl.f32_to_bf16_bits(np.full((1, N), t + 1.0, np.float32))
    ts = w.tok_slot()
    dc = DeviceCase(w, p)
    y = to_np(dc.forward(flags=flags))
    assert np.array_equal(y, np.repeat((ts + 1).astype(np.float32)[:, None], N, axis=1))
    _, dA, dB = dc.backward(flags=flags)
    for t in range(n):
        cnt = int(np.sum(ts == t))
        assert float(dB[t][0, 5]) == cnt and float(dB[t].abs().sum()) == cnt
        e = np.zeros(K, np.float32)
        for i in range(T):
            if ts[i] == t:
                e[i % K] += t + 1
        assert np.array_equal(to_np(dA[t])[:, 0], e)


def test_accumulate_flag_and_absent_tenants():
    w = wl.small_random_case(31, 260, 128, 136, [8, 4, 16, 8], n_segments=6)
    p = w.projections[0]
    dc, ref = _check_case(w, p)
    ts = w.tok_slot()
    absent = [t for t in range(4) if not np.any(ts == t)]
    assert absent, "the generator leaves the last tenant without tokens"
    dA, dB = dc.grads(fill=3.0)
    dc.backward(dA=dA, dB=dB, want_dx=False)
    for t in absent:
        assert float(dA[t].abs().max()) == 0.0 and float(dB[t].abs().max()) == 0.0     # overwritten with exact zeros
    dA2, dB2 = dc.grads(fill=3.0)
    dc.backward(dA=dA2, dB=dB2, want_dx=False, flags=B.MARLAAS_FLAG_ACCUMULATE)
    for t in range(4):
        assert_close(to_np(dA2[t]), ref["dA"][t] + 3.0, f"accumulated dA[{t}]")
        assert_close(to_np(dB2[t]), ref["dB"][t] + 3.0, f"accumulated dB[{t}]")
    # NULL entries are skipped
    dA3, dB3 = dc.grads(fill=5.0)
    keepA = dA3[0].clone()
    dc.backward(dA=[None] + dA3[1:], dB=None, want_dx=False)
    assert torch.equal(dA3[0], keepA)


def test_two_runs_are_bit_identical():
    w = wl.make_workload(4, scale_down=8)
    p = w.projections[0]
    dc = DeviceCase(w, p)
    y1 = dc.forward()
    dx1, dA1, dB1 = dc.backward()
    y2 = dc.forward()
    dx2, dA2, dB2 = dc.backward()
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    assert torch.equal(dx1.view(torch.int16), dx2.view(torch.int16))
    for a, b in zip(dA1 + dB1, dA2 + dB2):
        if a is not None:
            assert torch.equal(a, b)


def test_pool_store_roundtrip_versions_and_errors():
    w = wl.small_random_case(41, 64, 72, 88, [8, 5, 16], n_segments=4)
    p = w.projections[0]
    dc = DeviceCase(w, p, capacity=4, max_rank=16)
    for t, a in enumerate(p.adapters):
        A, Bm = B.marlaas_adapter_pool_export(dc.pool, t, a.rank)
        assert torch.equal(A.view(torch.int16), dc.A[t].view(torch.int16))
        assert torch.equal(Bm.view(torch.int16), dc.Bm[t].view(torch.int16))
        assert B.marlaas_adapter_pool_lookup(dc.pool, a.tenant_id) == (t, a.rank, float(np.float32(a.alpha) / np.float32(a.rank)), 0)
    # committing a new version of tenant 1 reuses its slot and changes the output of its tokens only
    y0 = dc.forward()
    a1 = p.adapters[1]
    newB = dev_bf16(wl.normal_bf16(77, wl.TID_B, (a1.rank, p.d_out), 0.02)[0])
    assert B.marlaas_adapter_pool_register(dc.pool, a1.tenant_id, 1, a1.rank, a1.alpha, dc.A[1], newB) == 1
    assert B.marlaas_adapter_pool_lookup(dc.pool, a1.tenant_id)[3] == 1
    y1 = dc.forward()
    ts = torch.from_numpy(w.tok_slot()).cuda()
    same = (y0.view(torch.int16) == y1.view(torch.int16)).all(dim=1)
    assert bool(same[ts != 1].all()) and (int((ts == 1).sum()) == 0 or not bool(same[ts == 1].all()))
    # a fourth tenant takes the free slot, a fifth does not fit, too large a rank is refused
    assert B.marlaas_adapter_pool_register(dc.pool, 5000, 0, 0, 0.0, None, None) == 3
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_adapter_pool_register(dc.pool, 5001, 0, 0, 0.0, None, None)
    assert e.value.status == B.MARLAAS_ERR_POOL_FULL
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_adapter_pool_register(dc.pool, a1.tenant_id, 2, 17, 1.0,
                                        torch.zeros((p.d_in, 17), dtype=torch.bfloat16, device="cuda:0"),
                                        torch.zeros((17, p.d_out), dtype=torch.bfloat16, device="cuda:0"))
    assert e.value.status == B.MARLAAS_ERR_RANK_TOO_LARGE
    B.marlaas_adapter_pool_unregister(dc.pool, 5000)
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_adapter_pool_unregister(dc.pool, 5000)
    assert e.value.status == B.MARLAAS_ERR_UNKNOWN_TENANT
    # an unregistered tenant's slot behaves as "no adapter"
    B.marlaas_adapter_pool_unregister(dc.pool, p.adapters[0].tenant_id)
    y2 = dc.forward()
    base = B.Segments(torch.tensor([0, w.T], dtype=torch.int32).cuda(), torch.tensor([-1], dtype=torch.int32).cuda())
    yb = dc.forward(seg=base)
    rows0 = ts == 0
    assert torch.equal(y2[rows0].view(torch.int16), yb[rows0].view(torch.int16))


def test_malformed_calls_return_status_codes_and_launch_nothing():
    w = wl.small_random_case(51, 40, 64, 64, [4, 4], n_segments=3)
    p = w.projections[0]
    dc = DeviceCase(w, p)
    n0 = B.marlaas_kernel_launch_count()

    def expect(status, fn):
        with pytest.raises(B.MarlaasError) as e:
            fn()
        assert e.value.status == status, str(e.value)

    bad_off = B.Segments(torch.tensor([0, 30, 20, 40], dtype=torch.int32), torch.tensor([0, 1, 0], dtype=torch.int32))
    expect(B.MARLAAS_ERR_BAD_SEGMENT_TABLE, lambda: dc.forward(seg=bad_off))
    short = B.Segments(torch.tensor([0, 30], dtype=torch.int32), torch.tensor([0], dtype=torch.int32))
    expect(B.MARLAAS_ERR_BAD_SEGMENT_TABLE, lambda: dc.forward(seg=short))
    bad_slot = B.Segments(torch.tensor([0, 40], dtype=torch.int32), torch.tensor([9], dtype=torch.int32))
    expect(B.MARLAAS_ERR_BAD_SEGMENT_TABLE, lambda: dc.forward(seg=bad_slot))
    small_ws = torch.empty(256, dtype=torch.uint8, device="cuda:0")
    expect(B.MARLAAS_ERR_WORKSPACE_TOO_SMALL,
           lambda: B.marlaas_lora_forward(dc.pool, dc.x, dc.W, dc.seg, workspace=small_ws))
    xm = torch.empty(40 * 64 + 8, dtype=torch.bfloat16, device="cuda:0")[1:1 + 40 * 64].view(40, 64)   # 2-byte offset
    expect(B.MARLAAS_ERR_INVALID_ARG, lambda: B.marlaas_lora_forward(dc.pool, xm, dc.W, dc.seg))
    assert B.marlaas_kernel_launch_count() == n0
    # device-resident tables are checked by the kernels: out-of-range slots fall back to the base weight and set
    # the status word, without any fault
    dev_bad = B.Segments(torch.tensor([0, 20, 40], dtype=torch.int32).cuda(), torch.tensor([1, 7], dtype=torch.int32).cuda())
    y = dc.forward(seg=dev_bad)
    expect(B.MARLAAS_ERR_DEVICE_BAD_INDEX, lambda: B.marlaas_check_status(dc.pool))
    B.marlaas_check_status(dc.pool)                       # cleared
    base = B.Segments(torch.tensor([0, 40], dtype=torch.int32).cuda(), torch.tensor([-1], dtype=torch.int32).cuda())
    yb = dc.forward(seg=base)
    assert torch.equal(y[20:].view(torch.int16), yb[20:].view(torch.int16))
    dev_off = B.Segments(torch.tensor([0, 30, 20, 40], dtype=torch.int32).cuda(), torch.tensor([0, 1, 0], dtype=torch.int32).cuda())
    dc.forward(seg=dev_off)
    expect(B.MARLAAS_ERR_BAD_SEGMENT_TABLE, lambda: B.marlaas_check_status(dc.pool))
    # an empty batch is a no-op
    e = B.marlaas_lora_forward(dc.pool, dc.x[:0], dc.W, B.Segments(torch.zeros(1, dtype=torch.int32).cuda(),
                                                                  torch.zeros(0, dtype=torch.int32).cuda()))
    assert e.shape[0] == 0


def test_backward_inside_a_stream_capture_replays_to_the_same_bits():
    # training-shaped batch large enough for the 2-CTA GEMM, saved h given: the adapter-gradient kernels go to the
    # pool's side stream (fork / join by events), which a capture must be able to hold; the replayed graph has to
    # reproduce the directly issued call bit for bit, twice
    w = wl.make_workload(4, scale_down=4)
    p = w.projections[0]
    dc = DeviceCase(w, p)
    hs = torch.empty((w.T, dc.pool.rank_stride), dtype=torch.float32, device="cuda:0")
    dc.forward(h_save=hs)
    dx0, dA0, dB0 = dc.backward(h_saved=hs)
    torch.cuda.synchronize()
    dx = torch.zeros_like(dx0)
    dA, dB = dc.grads(fill=0.0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            B.marlaas_lora_backward(dc.pool, dc.x, dc.W, dc.dy, dc.seg, dx=dx, dA=dA, dB=dB, h_saved=hs)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        dx.fill_(7.0)
        for t in dA + dB:
            if t is not None:
                t.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(dx, dx0)
        for a, b in zip(dA + dB, dA0 + dB0):
            if a is not None:
                assert torch.equal(a, b)
    B.marlaas_check_status(dc.pool)


def test_a_wait_that_runs_out_is_reported_and_the_pool_stays_usable():
    # A bounded wait inside a kernel gives up after its limit, the kernel returns normally and the status word says
    # DEVICE_TIMEOUT.  No product kernel is starved for this: a diagnostic CTA waits 1 ms on a barrier nobody arrives on.
    w = wl.make_workload(1)
    p = w.projections[0]
    dc, ref = _check_case(w, p)
    B.marlaas_debug_wait_runs_out(dc.pool, limit_ns=1_000_000)
    with pytest.raises(B.MarlaasError) as e:
        B.marlaas_check_status(dc.pool)
    assert e.value.status == B.MARLAAS_ERR_DEVICE_TIMEOUT
    assert "site 99" in str(e.value)
    B.marlaas_check_status(dc.pool)                      # the finding was cleared by the read
    y = dc.forward()                                     # and the pool computes as before
    assert_close(to_np(y), ref["y"], "forward after a reported timeout")
    B.marlaas_check_status(dc.pool)
    with pytest.raises(B.MarlaasError):
        B.marlaas_debug_wait_runs_out(dc.pool, limit_ns=10**12)      # limits beyond 100 ms are refused on the host
