"""Pins for the CPU oracle: facts that the layer's definition fixes, each written independently
of the oracle's own loops (numpy library routines, closed forms, finite differences, brute force),
chosen so that a dropped term, a wrong sign or index, or a transposed operand fails at least one.

The paper prints no worked numeric example of the layer, so there are no printed values to pin to;
the definition (shared frozen base weight + per-tenant low-rank adapters, Multi-Task Manager /
Multi-LoRA Rollout sections) and mathematics are the pins.
"""
import numpy as np
import pytest

import oracle
from paper_2605_08527_b200 import workloads as wl


def _case(seed=11, T=37, K=24, N=20, ranks=(3, 1, 5, 2), nseg=7, base_only=True, sigma_w=0.3, alphas=None):
    w = wl.small_random_case(seed, T, K, N, list(ranks), alphas=alphas, n_segments=nseg,
                             with_base_only=base_only, sigma_w=sigma_w)
    return w, w.projections[0]


def _args(p, dtype=np.float64):
    return oracle.adapters_of(p, dtype)


def _np_forward(x, W, ranks, scales, As, Bs, ts):
    """Independent restatement with numpy matmul in float64, token by token."""
    y = x.astype(np.float64) @ W.astype(np.float64)
    for i, t in enumerate(ts):
        if t >= 0 and ranks[t] > 0:
            y[i] += float(scales[t]) * ((x[i].astype(np.float64) @ As[t].astype(np.float64)) @ Bs[t].astype(np.float64))
    return y


def test_forward_matches_numpy_matmul_f32_and_f64():
    w, p = _case()
    ts = w.tok_slot()
    for dt, tol in ((np.float32, 2e-6), (np.float64, 1e-12)):
        r, s, A, B = _args(p, dt)
        y, h = oracle.forward(p.x, p.W, r, s, A, B, ts, dtype=dt)
        ref = _np_forward(p.x, p.W, r, s, A, B, ts)
        assert np.max(np.abs(y - ref)) <= tol * (1 + np.max(np.abs(ref)))
        for i, t in enumerate(ts):
            if t >= 0:
                hr = p.x[i].astype(np.float64) @ A[t].astype(np.float64)
                assert np.allclose(h[i, :r[t]], hr, rtol=tol * 10, atol=tol * 10)
                assert np.all(h[i, r[t]:] == 0)
            else:
                assert np.all(h[i] == 0)


def test_P1_zero_B_gives_base_output_exactly():
    w, p = _case()
    ts = w.tok_slot()
    r, s, A, B = _args(p, np.float32)
    B0 = [np.zeros_like(b) for b in B]
    y0, _ = oracle.forward(p.x, p.W, r, s, A, B0, ts)
    ybase, _ = oracle.forward(p.x, p.W, r, s, A, B0, np.full(w.T, -1, np.int32))
    assert np.array_equal(y0, ybase)
    assert np.allclose(ybase, p.x.astype(np.float64) @ p.W.astype(np.float64), rtol=2e-6, atol=2e-6)
    dx0, g0 = oracle.backward_dx(p.dy, p.W, r, s, A, B0, ts)
    dxb, _ = oracle.backward_dx(p.dy, p.W, r, s, A, B0, np.full(w.T, -1, np.int32))
    assert np.array_equal(dx0, dxb) and np.all(g0 == 0)
    assert np.allclose(dxb, p.dy.astype(np.float64) @ p.W.astype(np.float64).T, rtol=2e-6, atol=2e-5)
    dA, dB = oracle.backward_dAdB(p.x, p.dy, r, s, A, B0, ts)
    assert all(np.all(a == 0) for a in dA)
    assert any(np.any(b != 0) for b in dB)          # dB does not vanish with B


def test_P2_single_tenant_equals_merged_weight():
    w, p = _case(nseg=1, ranks=(4,), base_only=False)
    ts = np.zeros(w.T, np.int32)
    r, s, A, B = _args(p)
    y, _ = oracle.forward(p.x, p.W, r, s, A, B, ts, dtype=np.float64)
    Wm = p.W.astype(np.float64) + s[0] * (A[0].astype(np.float64) @ B[0].astype(np.float64))
    assert np.allclose(y, p.x.astype(np.float64) @ Wm, rtol=1e-12, atol=1e-12)
    dx, _ = oracle.backward_dx(p.dy, p.W, r, s, A, B, ts, dtype=np.float64)
    assert np.allclose(dx, p.dy.astype(np.float64) @ Wm.T, rtol=1e-12, atol=1e-12)
    # dense chain rule for the merged form: dWm = x^T dy, dA = s dWm B^T, dB = s A^T dWm
    dWm = p.x.astype(np.float64).T @ p.dy.astype(np.float64)
    dA, dB = oracle.backward_dAdB(p.x, p.dy, r, s, A, B, ts, dtype=np.float64)
    assert np.allclose(dA[0], s[0] * dWm @ B[0].astype(np.float64).T, rtol=1e-11, atol=1e-11)
    assert np.allclose(dB[0], s[0] * A[0].astype(np.float64).T @ dWm, rtol=1e-11, atol=1e-11)


def test_P3_token_permutation_and_segment_splitting():
    w, p = _case(T=41)
    ts = w.tok_slot()
    r, s, A, B = _args(p, np.float32)
    y, _ = oracle.forward(p.x, p.W, r, s, A, B, ts)
    dx, _ = oracle.backward_dx(p.dy, p.W, r, s, A, B, ts)
    dA, dB = oracle.backward_dAdB(p.x, p.dy, r, s, A, B, ts)
    perm = np.argsort(wl.hash_u64(3, 9, np.arange(w.T, dtype=np.uint64)))
    y2, _ = oracle.forward(p.x[perm], p.W, r, s, A, B, ts[perm])
    dx2, _ = oracle.backward_dx(p.dy[perm], p.W, r, s, A, B, ts[perm])
    dA2, dB2 = oracle.backward_dAdB(p.x[perm], p.dy[perm], r, s, A, B, ts[perm])
    assert np.array_equal(y2, y[perm]) and np.array_equal(dx2, dx[perm])   # rows are independent: bit-exact
    for t in range(len(r)):
        assert np.allclose(dA2[t], dA[t], rtol=1e-6, atol=1e-6 * np.abs(dA[t]).max() + 1e-30)
        assert np.allclose(dB2[t], dB[t], rtol=1e-6, atol=1e-6 * np.abs(dB[t]).max() + 1e-30)
    # the index build gives the same per-token slots whether a segment is whole or split in pieces
    so, ss = w.seg_offsets, w.seg_slot
    so2, ss2 = [0], []
    for a, b, t in zip(so[:-1], so[1:], ss):
        mid = (a + b) // 2
        so2 += [mid, mid, b]          # split in two with an empty segment in between
        ss2 += [t, (t + 1) % len(r), t]
    a1 = oracle.build_index(w.T, so, ss, len(r))
    a2 = oracle.build_index(w.T, so2, ss2, len(r))
    for u, v in zip(a1, a2):
        assert np.array_equal(u, v)


def test_P4_rank1_closed_form():
    w, p = _case(ranks=(1, 1, 1), nseg=5, T=23)
    ts = w.tok_slot()
    r, s, A, B = _args(p)
    x, W, dy = p.x.astype(np.float64), p.W.astype(np.float64), p.dy.astype(np.float64)
    y, _ = oracle.forward(x, W, r, s, A, B, ts, dtype=np.float64)
    dx, _ = oracle.backward_dx(dy, W, r, s, A, B, ts, dtype=np.float64)
    dA, dB = oracle.backward_dAdB(x, dy, r, s, A, B, ts, dtype=np.float64)
    K, N = W.shape
    ey, edx = x @ W, dy @ W.T
    eA = [np.zeros(K) for _ in r]
    eB = [np.zeros(N) for _ in r]
    for i, t in enumerate(ts):
        if t < 0:
            continue
        a = A[t][:, 0].astype(np.float64)
        b = B[t][0, :].astype(np.float64)
        ey[i] += s[t] * np.dot(x[i], a) * b
        edx[i] += s[t] * np.dot(dy[i], b) * a
        eA[t] += s[t] * np.dot(dy[i], b) * x[i]
        eB[t] += s[t] * np.dot(x[i], a) * dy[i]
    assert np.allclose(y, ey, rtol=1e-12, atol=1e-12)
    assert np.allclose(dx, edx, rtol=1e-12, atol=1e-12)
    for t in range(len(r)):
        assert np.allclose(dA[t][:, 0], eA[t], rtol=1e-11, atol=1e-11)
        assert np.allclose(dB[t][0, :], eB[t], rtol=1e-11, atol=1e-11)


def test_P5_finite_differences_in_double():
    # 3 tenants of ranks 1,2,3 (+ a fourth that never appears), one tenant in two segments, one -1 segment
    K, N, T = 12, 10, 7
    w, p = _case(seed=5, T=T, K=K, N=N, ranks=(1, 2, 3, 2), nseg=5, sigma_w=0.5)
    ts = np.array([0, 1, 1, -1, 2, 1, 2], np.int32)
    r, s, A, B = _args(p)
    A = [a.astype(np.float64) * 10 for a in A]
    B = [b.astype(np.float64) * 10 for b in B]
    x, W, dy = p.x.astype(np.float64), p.W.astype(np.float64), p.dy.astype(np.float64)

    def loss(x_, A_, B_):
        y, _ = oracle.forward(x_, W, r, s, A_, B_, ts, dtype=np.float64)
        return float(np.sum(y * dy))

    dx, _ = oracle.backward_dx(dy, W, r, s, A, B, ts, dtype=np.float64)
    dA, dB = oracle.backward_dAdB(x, dy, r, s, A, B, ts, dtype=np.float64)
    eps = 1e-3   # the loss is linear in each argument separately, so central differences are exact up to rounding

    def fd(arr, setter):
        out = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            plus, minus = arr.copy(), arr.copy()
            plus[idx] += eps
            minus[idx] -= eps
            out[idx] = (setter(plus) - setter(minus)) / (2 * eps)
        return out

    assert np.allclose(fd(x, lambda v: loss(v, A, B)), dx, rtol=1e-8, atol=1e-8)
    for t in range(4):
        fA = fd(A[t], lambda v: loss(x, [v if u == t else A[u] for u in range(4)], B))
        fB = fd(B[t], lambda v: loss(x, A, [v if u == t else B[u] for u in range(4)]))
        assert np.allclose(fA, dA[t], rtol=1e-8, atol=1e-8)
        assert np.allclose(fB, dB[t], rtol=1e-8, atol=1e-8)
    assert np.all(dA[3] == 0) and np.all(dB[3] == 0)       # registered tenant with no token: exact zeros
    assert np.any(dA[1] != 0)


def test_P6_adjoint_identities_moderate_size():
    w = wl.make_workload(4, scale_down=16)
    p = w.projections[0]
    ts = w.tok_slot()
    r, s, A, B = _args(p, np.float32)
    K, N = p.d_in, p.d_out
    x, dy = p.x, p.dy
    dx, _ = oracle.backward_dx(dy, p.W, r, s, A, B, ts)
    dA, dB = oracle.backward_dAdB(x, dy, r, s, A, B, ts)
    y0, _ = oracle.forward(x, p.W, r, s, A, B, ts, dtype=np.float64)
    _, ex = wl.normal_bf16(99, wl.TID_PERTURB, x.shape, 1.0)
    y1, _ = oracle.forward(x.astype(np.float64) + ex, p.W, r, s, A, B, ts, dtype=np.float64)
    lhs = np.sum(dy.astype(np.float64) * (y1 - y0))
    rhs = np.sum(dx.astype(np.float64) * ex)
    assert abs(lhs - rhs) <= 1e-5 * (abs(lhs) + abs(rhs) + 1)
    eA = [wl.normal_bf16(99, wl.TID_PERTURB, a.shape, 0.02, sub=1 + t)[1].astype(np.float64) for t, a in enumerate(A)]
    eB = [wl.normal_bf16(99, wl.TID_PERTURB, b.shape, 0.02, sub=100 + t)[1].astype(np.float64) for t, b in enumerate(B)]
    yA, _ = oracle.forward(x, p.W, r, s, [a + e for a, e in zip(A, eA)], B, ts, dtype=np.float64)
    yB, _ = oracle.forward(x, p.W, r, s, A, [b + e for b, e in zip(B, eB)], ts, dtype=np.float64)
    lhsA = np.sum(dy.astype(np.float64) * (yA - y0))
    rhsA = sum(np.sum(d.astype(np.float64) * e) for d, e in zip(dA, eA))
    lhsB = np.sum(dy.astype(np.float64) * (yB - y0))
    rhsB = sum(np.sum(d.astype(np.float64) * e) for d, e in zip(dB, eB))
    assert abs(lhsA - rhsA) <= 1e-5 * (abs(lhsA) + abs(rhsA) + 1)
    assert abs(lhsB - rhsB) <= 1e-5 * (abs(lhsB) + abs(rhsB) + 1)
    assert abs(lhsA) > 1e-3 and abs(lhsB) > 1e-3


def test_P7_routing_probe_exact_integers():
    T, K, N, n = 29, 16, 12, 5
    so = np.array([0, 4, 4, 9, 15, 22, 29], np.int32)
    ss = np.array([2, 0, 4, -1, 0, 3], np.int32)
    ts, cnt, off, perm = oracle.build_index(T, so, ss, n)
    W = np.zeros((K, N), np.float32)
    x = np.zeros((T, K), np.float32)
    x[np.arange(T), np.arange(T) % K] = 1.0                      # one-hot rows
    r = [1] * n
    s = [1.0] * n
    A = [np.ones((K, 1), np.float32) for _ in range(n)]
    B = [np.full((1, N), t + 1.0, np.float32) for t in range(n)]
    y, _ = oracle.forward(x, W, r, s, A, B, ts)
    assert np.array_equal(y, np.repeat((ts + 1).astype(np.float32)[:, None], N, axis=1))
    dy = np.zeros((T, N), np.float32)
    dy[:, 3] = 1.0
    dA, dB = oracle.backward_dAdB(x, dy, r, s, A, B, ts)
    for t in range(n):
        assert dB[t][0, 3] == cnt[t] and np.all(np.delete(dB[t][0], 3) == 0)      # token counts of tenant t
        # dA_t[k] = (t+1) * number of tenant-t tokens whose hot index is k
        e = np.zeros(K)
        for i in range(T):
            if ts[i] == t:
                e[i % K] += t + 1
        assert np.array_equal(dA[t][:, 0], e.astype(np.float32))


def test_P8_scale_doubling_is_exact():
    w, p = _case()
    ts = w.tok_slot()
    r, s, A, B = _args(p, np.float32)
    s2 = [2 * v for v in s]
    base = np.full(w.T, -1, np.int32)
    y, _ = oracle.forward(p.x, p.W, r, s, A, B, ts, dtype=np.float64)
    y2, _ = oracle.forward(p.x, p.W, r, s2, A, B, ts, dtype=np.float64)
    yb, _ = oracle.forward(p.x, p.W, r, s, A, B, base, dtype=np.float64)
    assert np.allclose(y2 - yb, 2 * (y - yb), rtol=1e-12, atol=1e-13)
    dA, dB = oracle.backward_dAdB(p.x, p.dy, r, s, A, B, ts)
    dA2, dB2 = oracle.backward_dAdB(p.x, p.dy, r, s2, A, B, ts)
    for t in range(len(r)):
        assert np.array_equal(dA2[t], 2 * dA[t]) and np.array_equal(dB2[t], 2 * dB[t])


def test_P9_rank_zero_padding_changes_nothing():
    w, p = _case()
    ts = w.tok_slot()
    r, s, A, B = _args(p, np.float32)
    pad = 3
    r2 = [v + pad for v in r]
    A2 = [np.concatenate([a, np.zeros((a.shape[0], pad), np.float32)], axis=1) for a in A]
    B2 = [np.concatenate([b, np.zeros((pad, b.shape[1]), np.float32)], axis=0) for b in B]
    y, _ = oracle.forward(p.x, p.W, r, s, A, B, ts)
    y2, _ = oracle.forward(p.x, p.W, r2, s, A2, B2, ts)
    dx, _ = oracle.backward_dx(p.dy, p.W, r, s, A, B, ts)
    dx2, _ = oracle.backward_dx(p.dy, p.W, r2, s, A2, B2, ts)
    assert np.array_equal(y, y2) and np.array_equal(dx, dx2)
    dA, dB = oracle.backward_dAdB(p.x, p.dy, r, s, A, B, ts)
    dA2, dB2 = oracle.backward_dAdB(p.x, p.dy, r2, s, A2, B2, ts)
    for t in range(len(r)):
        assert np.array_equal(dA2[t][:, :r[t]], dA[t]) and np.array_equal(dB2[t][:r[t]], dB[t])


def _brute_index(T, so, ss, cap):
    tok = np.full(T, -7, np.int32)
    for i in range(T):
        for s_ in range(len(ss)):
            if so[s_] <= i < so[s_ + 1]:
                tok[i] = ss[s_]
    key = np.where(tok < 0, cap, tok)
    cnt = np.array([int(np.sum(key == t)) for t in range(cap + 1)], np.int32)
    off = np.zeros(cap + 2, np.int32)
    for t in range(cap + 1):
        off[t + 1] = off[t] + cnt[t]
    perm = np.array(sorted(range(T), key=lambda i: (key[i], i)), np.int32)
    return tok, cnt, off, perm


@pytest.mark.parametrize("seed", range(6))
def test_P10_index_build_brute_force(seed):
    T = [0, 1, 17, 64, 129, 300][seed]
    cap = [1, 3, 4, 7, 33, 5][seed]
    S = [1, 1, 9, 64, 40, 300][seed]
    if S == T and T > 0:
        so = np.arange(T + 1, dtype=np.int32)
    else:
        cuts = np.sort(wl.hash_u64(seed, 1, np.arange(max(S - 1, 0), dtype=np.uint64)) % np.uint64(T + 1)).astype(np.int32)
        so = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    ss = (wl.hash_u64(seed, 2, np.arange(S, dtype=np.uint64)) % np.uint64(cap + 1)).astype(np.int32) - 1
    got = oracle.build_index(T, so, ss, cap)
    exp = _brute_index(T, so, ss, cap)
    for g, e in zip(got, exp):
        assert np.array_equal(g, e)


def test_index_build_rejects_malformed_tables():
    with pytest.raises(ValueError):
        oracle.build_index(8, [0, 5, 3, 8], [0, 1, 0], 2)       # decreasing offsets
    with pytest.raises(ValueError):
        oracle.build_index(8, [0, 4, 7], [0, 1], 2)             # does not cover T
    with pytest.raises(ValueError):
        oracle.build_index(8, [0, 4, 8], [0, 2], 2)             # slot out of range


def test_float_accumulation_agrees_with_double_on_cfg1():
    # an fp32-accumulating restatement (numpy float32 matmul) stays within 1e-5 * sum|terms| of the oracle
    w = wl.make_workload(1)
    p = w.projections[0]
    ts = w.tok_slot()
    r, s, A, B = _args(p, np.float32)
    y, _ = oracle.forward(p.x, p.W, r, s, A, B, ts)
    y32 = p.x @ p.W
    for i, t in enumerate(ts):
        y32[i] += np.float32(s[t]) * ((p.x[i] @ A[t]) @ B[t])
    bound = 1e-5 * (np.abs(p.x) @ np.abs(p.W) + 1.0)
    assert np.all(np.abs(y32 - y) <= bound)


# ---- AdamW (policy update before the commit of a new adapter version) ------------------------------------------
def _rand(shape, seed):
    return wl.bf16_bits_to_f32(wl.normal_bf16(seed, wl.TID_PERTURB, shape, 1.0)[0]).astype(np.float64)


def test_adamw_first_step_closed_form():
    # from zero moments the bias corrections cancel the (1 - beta) factors exactly: m_hat = g, v_hat = g^2
    th, g = _rand((7, 5), 901), _rand((7, 5), 902)
    lr, eps, wd = 0.05, 1e-3, 0.1
    t1, m1, v1 = oracle.adamw_step(th, g, np.zeros_like(th), np.zeros_like(th), lr=lr, beta1=0.9, beta2=0.99, eps=eps,
                                   weight_decay=wd, step=1)
    np.testing.assert_allclose(t1, th - lr * (g / (np.abs(g) + eps) + wd * th), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(m1, 0.1 * g, rtol=1e-12)
    np.testing.assert_allclose(v1, 0.01 * g * g, rtol=1e-12)


def test_adamw_constant_gradient_and_pure_decay_closed_forms():
    th0, g = _rand((4, 6), 903), _rand((4, 6), 904)
    lr, eps, n = 0.01, 1e-4, 9
    # constant gradient, no decay: m_hat = g and v_hat = g^2 at every step, so each step moves by lr g / (|g| + eps)
    th, m, v = th0, np.zeros_like(th0), np.zeros_like(th0)
    for t in range(1, n + 1):
        th, m, v = oracle.adamw_step(th, g, m, v, lr=lr, beta1=0.8, beta2=0.95, eps=eps, step=t)
    np.testing.assert_allclose(th, th0 - n * lr * g / (np.abs(g) + eps), rtol=1e-10, atol=1e-12)
    # zero gradient: only the decoupled decay acts, theta_n = theta_0 (1 - lr wd)^n, and the moments stay zero
    th, m, v = th0, np.zeros_like(th0), np.zeros_like(th0)
    for t in range(1, n + 1):
        th, m, v = oracle.adamw_step(th, np.zeros_like(th0), m, v, lr=lr, weight_decay=0.3, step=t)
    np.testing.assert_allclose(th, th0 * (1 - lr * 0.3) ** n, rtol=1e-12)
    assert not m.any() and not v.any()


def test_adamw_gradient_scale_is_a_scale_of_the_gradient():
    th, g = _rand((3, 8), 905), _rand((3, 8), 906)
    a = oracle.adamw_step(th, g, 0 * th, 0 * th, lr=0.02, grad_scale=0.25, step=1)
    b = oracle.adamw_step(th, 0.25 * g, 0 * th, 0 * th, lr=0.02, step=1)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=1e-14)


def test_adamw_agrees_with_the_library_optimizer_over_several_steps():
    import torch
    th0 = _rand((6, 9), 907)
    hp = dict(lr=3e-2, beta1=0.9, beta2=0.98, eps=1e-6, weight_decay=0.05)
    p = torch.nn.Parameter(torch.from_numpy(th0.copy()))
    opt = torch.optim.AdamW([p], lr=hp["lr"], betas=(hp["beta1"], hp["beta2"]), eps=hp["eps"],
                            weight_decay=hp["weight_decay"])
    th, m, v = th0, np.zeros_like(th0), np.zeros_like(th0)
    for t in range(1, 7):
        g = _rand((6, 9), 910 + t)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        th, m, v = oracle.adamw_step(th, g, m, v, step=t, **hp)
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-11, atol=1e-13)
