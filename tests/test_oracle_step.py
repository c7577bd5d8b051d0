"""Pins for the oracle's step (Algorithm 1, Eq. 3, Eq. 4, Eq. 5): closed forms,
invariants, textbook reductions and a hand-worked example, none of which call the
oracle to produce the expected value."""
import math

import numpy as np
import pytest

import oracle
from oracle import MODE_CHANNEL, MODE_TENSOR, DT_BF16, DT_F32, MatrixOracle


def _rng(seed=0):
    return np.random.default_rng(seed)


def _grads(rows, cols, steps, seed=0, scale=1e-3):
    r = _rng(seed)
    return [(r.standard_normal((rows, cols)) * scale).astype(np.float32) for _ in range(steps)]


def test_contraction_matches_numpy_matmul():
    r = _rng(1)
    P = r.standard_normal((5, 13))
    G = r.standard_normal((13, 29))
    np.testing.assert_allclose(oracle.project(P, G), P @ G, rtol=1e-13, atol=1e-13)
    # a transposed operand or swapped index would fail on this asymmetric case
    e = np.zeros((2, 3)); e[1, 2] = 1.0
    G2 = np.arange(12.0).reshape(3, 4)
    assert np.array_equal(oracle.project(e, G2), np.vstack([np.zeros(4), G2[2]]))


def test_hand_worked_2x3_rank1_step():
    # P = [1 2], G = [[1,2,3],[4,5,6]] -> R = [9,12,15]; M = 0.1 R; V = 0.001 R^2;
    # R~ = 0.1 R / sqrt(0.001 R^2) = sqrt(10) sign(R); s_j = sqrt(10)/|R_j|.
    mo = MatrixOracle(2, 3, rank=1, mode=MODE_CHANNEL, gamma=1.01, eps=0.0)
    W = np.zeros((2, 3), dtype=np.float32)
    G = np.array([[1, 2, 3], [4, 5, 6]], dtype=np.float32)
    res = mo.step(W, G, lr=0.5, wd=0.0, P=np.array([[1.0, 2.0]]), want_R=True)
    np.testing.assert_allclose(res.R, [[9.0, 12.0, 15.0]], rtol=1e-14)
    s = np.array([0.35136418446315326, 0.26352313834736496, 0.21081851067789195])
    np.testing.assert_allclose(res.s, s, rtol=1e-12)
    # scaled gradient G diag(s): columns (1,4)s0, (2,5)s1, (3,6)s2
    norm = math.sqrt(17 * s[0] ** 2 + 29 * s[1] ** 2 + 45 * s[2] ** 2)
    assert res.c == 1.0 and abs(res.norm - norm) < 1e-12
    np.testing.assert_allclose(res.dW, -0.5 * G * s[None, :], rtol=1e-12)
    np.testing.assert_allclose(res.W, (-0.5 * G * s[None, :]).astype(np.float32), rtol=1e-6)


def test_identity_projection_reduces_to_full_rank_channel_scaling():
    # With P = I_m the low-rank scale (Eq. 5) is the full-rank one (Eq. 3) built from
    # textbook Adam moments of G itself.
    m, n, steps = 6, 11, 5
    b1, b2, eps = 0.9, 0.999, 1e-8
    mo = MatrixOracle(m, n, rank=m, mode=MODE_CHANNEL, gamma=0.0, beta1=b1, beta2=b2, eps=eps)
    W = np.zeros((m, n), dtype=np.float32)
    M = np.zeros((m, n)); V = np.zeros((m, n))
    for G in _grads(m, n, steps, seed=2, scale=1.0):
        res = mo.step(W, G, lr=0.1, wd=0.0, P=np.eye(m), want_R=True)
        g = G.astype(np.float64)
        M = b1 * M + (1 - b1) * g
        V = b2 * V + (1 - b2) * g * g
        Gt = M / (np.sqrt(V) + eps)
        s = np.linalg.norm(Gt, axis=0) / np.linalg.norm(g, axis=0)
        np.testing.assert_allclose(res.R, g, rtol=1e-14)
        np.testing.assert_allclose(res.s, s, rtol=1e-12)
        np.testing.assert_allclose(res.dW, -0.1 * g * s[None, :], rtol=1e-12)
        W = res.W


def test_low_rank_first_moment_is_projection_of_full_moment_and_second_moment_l1_identity():
    # Appendix, first-moment analysis: M^R_t = P M_t for a fixed P and zero init; second
    # moment: |V^R_t[:, j]|_1 = (1 - beta2) sum_k beta2^k |R_{t-k}[:, j]|^2.
    m, n, r, steps = 16, 19, 4, 7
    b1, b2 = 0.8, 0.95
    mo = MatrixOracle(m, n, rank=r, seed=5, T=1000, beta1=b1, beta2=b2, p_round_bf16=False)
    P = oracle.projection(5, 0, 0, r, m, round_bf16=False)
    W = np.zeros((m, n), dtype=np.float32)
    Mfull = np.zeros((m, n))
    Rs = []
    for G in _grads(m, n, steps, seed=3, scale=1.0):
        mo.step(W, G, lr=0.0, wd=0.0)
        Mfull = b1 * Mfull + (1 - b1) * G.astype(np.float64)
        Rs.append(P @ G.astype(np.float64))
        np.testing.assert_allclose(mo.M, P @ Mfull, rtol=1e-11, atol=1e-13)
        t = len(Rs)
        l1 = (1 - b2) * sum(b2 ** k * np.sum(Rs[t - 1 - k] ** 2, axis=0) for k in range(t))
        np.testing.assert_allclose(np.sum(mo.V, axis=0), l1, rtol=1e-11)


@pytest.mark.parametrize("bias_correction", [False, True])
def test_constant_gradient_closed_form_scale(bias_correction):
    # Constant G, eps = 0: M = (1-b1^t) R, V = (1-b2^t) R^2, so every entry of R~ has
    # magnitude (1-b1^t)/sqrt(1-b2^t) (1 with bias correction) and
    # s_j = that * sqrt(r) / |R[:, j]|.
    m, n, r = 7, 12, 3
    b1, b2 = 0.9, 0.999
    G = (_rng(4).standard_normal((m, n))).astype(np.float32)
    P = oracle.projection(8, 2, 0, r, m)
    R = P @ G.astype(np.float64)
    mo = MatrixOracle(m, n, rank=r, seed=8, matrix_id=2, T=1000, gamma=0.0, eps=0.0, beta1=b1, beta2=b2,
                      bias_correction=bias_correction)
    W = np.zeros((m, n), dtype=np.float32)
    for t in range(1, 5):
        res = mo.step(W, G, lr=0.0, wd=0.0)
        f = 1.0 if bias_correction else (1 - b1 ** t) / math.sqrt(1 - b2 ** t)
        np.testing.assert_allclose(res.s, f * math.sqrt(r) / np.linalg.norm(R, axis=0), rtol=1e-10)
    assert abs((1 - b1) / math.sqrt(1 - b2) - 3.1622776601683795) < 1e-12


def test_scales_are_one_when_moments_reproduce_R():
    # beta1 = 0 gives M = R; beta2 = 1 keeps V = 0; eps = 1 then makes R~ = R exactly.
    for mode in (MODE_CHANNEL, MODE_TENSOR):
        mo = MatrixOracle(8, 20, rank=4, mode=mode, gamma=0.0, beta1=0.0, beta2=1.0, eps=1.0)
        W = np.zeros((8, 20), dtype=np.float32)
        for G in _grads(8, 20, 3, seed=5):
            res = mo.step(W, G, lr=1.0, wd=0.0)
            np.testing.assert_allclose(res.s, np.ones(20), rtol=1e-14)
            np.testing.assert_allclose(res.dW, -G.astype(np.float64), rtol=1e-14)
    # eps is added to sqrt(V), not placed under the root: eps = 0.5 gives R~ = 2 R, s = 2
    mo = MatrixOracle(8, 20, rank=4, gamma=0.0, beta1=0.0, beta2=1.0, eps=0.5)
    res = mo.step(np.zeros((8, 20), dtype=np.float32), _grads(8, 20, 1, seed=5)[0], lr=1.0, wd=0.0)
    np.testing.assert_allclose(res.s, np.full(20, 2.0), rtol=1e-14)


def test_mini_is_one_tensor_wise_scale_equal_to_the_flattened_channel_formula():
    m, n = 10, 33
    mo = MatrixOracle(m, n, rank=1, mode=MODE_TENSOR, seed=3, gamma=0.0, alpha=math.sqrt(128))
    W = np.zeros((m, n), dtype=np.float32)
    for G in _grads(m, n, 4, seed=6):
        res = mo.step(W, G, lr=0.01, wd=0.0, want_R=True)
        assert np.all(res.s == res.s[0])
        Rt = mo.M / (np.sqrt(mo.V) + 1e-8)
        want = np.linalg.norm(Rt.reshape(-1)) / np.linalg.norm(res.R.reshape(-1))
        assert abs(res.s[0] - want) < 1e-12 * want
        np.testing.assert_allclose(res.dW, -0.01 * math.sqrt(128) * want * G.astype(np.float64), rtol=1e-11)


def test_tensor_mode_with_rank_above_one_uses_frobenius_norms():
    m, n, r = 8, 12, 3
    mo = MatrixOracle(m, n, rank=r, mode=MODE_TENSOR, seed=3, gamma=0.0)
    W = np.zeros((m, n), dtype=np.float32)
    G = _grads(m, n, 1, seed=7)[0]
    res = mo.step(W, G, lr=0.01, wd=0.0, want_R=True)
    Rt = mo.M / (np.sqrt(mo.V) + 1e-8)
    want = math.sqrt(np.sum(Rt ** 2)) / math.sqrt(np.sum(res.R ** 2))
    np.testing.assert_allclose(res.s, np.full(n, want), rtol=1e-12)


def test_limiter_caps_growth_and_only_acts_above_gamma():
    # Eq. 4: if |G~_t| / |G~_{t-1}| > gamma, rescale to gamma |G~_{t-1}|.
    m, n, r, gamma = 8, 16, 4, 1.01
    lim = MatrixOracle(m, n, rank=r, seed=1, gamma=gamma)
    free = MatrixOracle(m, n, rank=r, seed=1, gamma=0.0)
    W = np.zeros((m, n), dtype=np.float32)
    base = _grads(m, n, 12, seed=8, scale=1.0)
    growth = [1.0, 3.0, 0.2, 0.21, 5.0, 5.0, 1.0, 1.004, 1.2, 0.9, 0.95, 2.0]
    prev = None
    saw_limited = saw_free = False
    for t, (G, f) in enumerate(zip(base, growth)):
        G = (G * f).astype(np.float32)
        a = lim.step(W, G, lr=1.0, wd=0.0)
        b = free.step(W, G, lr=1.0, wd=0.0)
        assert b.c == 1.0
        np.testing.assert_allclose(a.s, b.s, rtol=1e-14)     # the limiter does not touch s
        raw = math.sqrt(np.sum((G.astype(np.float64) * b.s[None, :]) ** 2))
        assert abs(b.norm - raw) < 1e-12 * raw
        if t == 0:
            assert a.c == 1.0                                  # first step is never limited
        else:
            if raw / prev > gamma:
                saw_limited = True
                assert a.c < 1.0
                assert abs(a.c - gamma * prev / raw) < 1e-14
                assert abs(a.norm - gamma * prev) < 1e-12 * prev
            else:
                saw_free = True
                assert a.c == 1.0 and abs(a.norm - raw) < 1e-12 * raw
            assert a.norm <= gamma * prev * (1 + 1e-12)
        # the applied update has exactly the limited norm
        assert abs(np.linalg.norm(a.dW) - a.norm) < 1e-10 * a.norm
        prev = a.norm
    assert saw_limited and saw_free


def test_huge_gamma_never_limits():
    mo = MatrixOracle(4, 6, rank=2, gamma=1e30)
    W = np.zeros((4, 6), dtype=np.float32)
    for t, G in enumerate(_grads(4, 6, 4, seed=9, scale=1.0)):
        assert mo.step(W, (G * 10.0 ** t).astype(np.float32), lr=1.0, wd=0.0).c == 1.0


def test_zero_gradient_leaves_only_weight_decay():
    W = (_rng(10).standard_normal((5, 9)) * 0.02).astype(np.float32)
    mo = MatrixOracle(5, 9, rank=2)
    res = mo.step(W, np.zeros_like(W), lr=0.1, wd=0.5)
    assert np.all(res.s == 0.0)
    np.testing.assert_allclose(res.dW, -0.05 * W.astype(np.float64), rtol=1e-14)
    np.testing.assert_allclose(res.W, W * np.float32(0.95), rtol=1e-6)


def test_zero_learning_rate_keeps_weights_but_advances_state():
    W = (_rng(11).standard_normal((5, 9)) * 0.02).astype(np.float32)
    mo = MatrixOracle(5, 9, rank=2)
    res = mo.step(W, _grads(5, 9, 1, seed=12)[0], lr=0.0, wd=0.3)
    assert np.array_equal(res.W, W)
    assert mo.t == 1 and np.any(mo.M != 0) and np.any(mo.V != 0) and mo.prev_norm.value > 0


def test_gradient_scale_invariance_without_eps():
    # Scaling every gradient by k scales R, M and sqrt(V) by k: R~ is unchanged, s is
    # divided by k, and the update G diag(s) is unchanged.
    a = MatrixOracle(6, 10, rank=3, seed=2, eps=0.0)
    b = MatrixOracle(6, 10, rank=3, seed=2, eps=0.0)
    W = np.zeros((6, 10), dtype=np.float32)
    for G in _grads(6, 10, 4, seed=13, scale=1.0):
        ra = a.step(W, G, lr=0.1, wd=0.0)
        rb = b.step(W, (G * 8.0).astype(np.float32), lr=0.1, wd=0.0)   # 8 is exact in fp32
        np.testing.assert_allclose(ra.s, rb.s * 8.0, rtol=1e-12)
        np.testing.assert_allclose(ra.dW, rb.dW, rtol=1e-12, atol=1e-18)


def test_channel_permutation_equivariance():
    perm = _rng(14).permutation(10)
    a = MatrixOracle(6, 10, rank=3, seed=2)
    b = MatrixOracle(6, 10, rank=3, seed=2)
    W = (_rng(15).standard_normal((6, 10)) * 0.02).astype(np.float32)
    Wa, Wb = W, W[:, perm]
    for G in _grads(6, 10, 3, seed=16):
        ra = a.step(Wa, G, lr=0.1, wd=0.01)
        rb = b.step(Wb, G[:, perm], lr=0.1, wd=0.01)
        np.testing.assert_allclose(ra.s[perm], rb.s, rtol=1e-13)
        np.testing.assert_allclose(ra.dW[:, perm], rb.dW, rtol=1e-12)
        Wa, Wb = ra.W, rb.W


def test_tall_matrix_is_the_transposed_wide_problem():
    # The paper states the method for m <= n; a tall stored matrix is handled as its
    # transpose: project along the shorter side, one scale per stored row.
    rows, cols, r = 14, 5, 2
    tall = MatrixOracle(rows, cols, rank=r, seed=4, matrix_id=7, T=2)
    wide = MatrixOracle(cols, rows, rank=r, seed=4, matrix_id=7, T=2)
    W = (_rng(17).standard_normal((rows, cols)) * 0.02).astype(np.float32)
    Wt, Ww = W, np.ascontiguousarray(W.T)
    for G in _grads(rows, cols, 5, seed=18):
        rt = tall.step(Wt, G, lr=0.05, wd=0.1)
        rw = wide.step(Ww, np.ascontiguousarray(G.T), lr=0.05, wd=0.1)
        assert rt.s.shape == (rows,)
        np.testing.assert_allclose(rt.s, rw.s, rtol=1e-14)
        np.testing.assert_allclose(rt.dW, rw.dW.T, rtol=1e-14)
        assert np.array_equal(rt.W, rw.W.T)
        Wt, Ww = rt.W, rw.W


def test_square_matrix_projects_rows_and_scales_columns():
    mo = MatrixOracle(6, 6, rank=6, gamma=0.0, eps=0.0)
    G = _grads(6, 6, 1, seed=19, scale=1.0)[0]
    res = mo.step(np.zeros((6, 6), dtype=np.float32), G, lr=1.0, wd=0.0, P=np.eye(6))
    want = (0.1 / math.sqrt(0.001)) * math.sqrt(6) / np.linalg.norm(G.astype(np.float64), axis=0)
    np.testing.assert_allclose(res.s, want, rtol=1e-12)


def test_refresh_changes_the_projection_every_T_steps_and_keeps_moments():
    m, n, r, T = 5, 8, 2, 3
    mo = MatrixOracle(m, n, rank=r, seed=6, matrix_id=1, T=T, p_round_bf16=False)
    W = np.zeros((m, n), dtype=np.float32)
    G = _grads(m, n, 1, seed=20, scale=1.0)[0]
    M = np.zeros((r, n))
    for t in range(7):
        res = mo.step(W, G, lr=0.0, wd=0.0, want_R=True)
        P = oracle.projection(6, 1, t // T, r, m, round_bf16=False)
        np.testing.assert_allclose(res.R, P @ G.astype(np.float64), rtol=1e-12)
        M = 0.9 * M + 0.1 * res.R
        np.testing.assert_allclose(mo.M, M, rtol=1e-12)       # no reset at the refresh
    assert not np.allclose(oracle.projection(6, 1, 0, r, m), oracle.projection(6, 1, 1, r, m))


def test_bf16_store_rounds_old_weight_plus_update():
    import torch
    W = (torch.randn(7, 12, generator=torch.Generator().manual_seed(1)) * 0.02).to(torch.bfloat16)
    G = (torch.randn(7, 12, generator=torch.Generator().manual_seed(2)) * 1e-3).to(torch.bfloat16)
    mo = MatrixOracle(7, 12, rank=3, dtype=DT_BF16)
    res = mo.step(W.float().numpy(), G.float().numpy(), lr=0.01, wd=0.01)
    want = np.array([[oracle.round_bf16(float(W[i, j]) + res.dW[i, j]) for j in range(12)] for i in range(7)])
    assert np.array_equal(res.W.astype(np.float64), want)
    # every stored value is a bfloat16
    assert np.array_equal(torch.from_numpy(res.W).to(torch.bfloat16).float().numpy(), res.W)
    f32 = MatrixOracle(7, 12, rank=3, dtype=DT_F32)
    r32 = f32.step(W.float().numpy(), G.float().numpy(), lr=0.01, wd=0.01)
    np.testing.assert_allclose(r32.W, W.float().numpy() + r32.dW, rtol=1e-6)


def test_scale_ratio_between_low_rank_and_full_rank_is_sqrt_r_over_m():
    # Theorem on the bounded update ratio: s^R_j / s_j concentrates near sqrt(r/m)
    # (the paper's sqrt(r/n) with n read as the projected dimension).
    m, n, steps = 64, 200, 6
    W = np.zeros((m, n), dtype=np.float32)
    gs = _grads(m, n, steps, seed=21, scale=1.0)
    full = MatrixOracle(m, n, rank=m, gamma=0.0)
    for G in gs:
        s_full = full.step(W, G, lr=0.0, wd=0.0, P=np.eye(m)).s
    for r in (16, 32):
        low = MatrixOracle(m, n, rank=r, seed=3, T=1000, gamma=0.0)
        for G in gs:
            s_low = low.step(W, G, lr=0.0, wd=0.0).s
        ratio = np.mean(s_low / s_full)
        assert abs(ratio / math.sqrt(r / m) - 1.0) < 0.1


def test_rank_above_short_side_is_rejected():
    mo = MatrixOracle(4, 9, rank=5)
    with pytest.raises(ValueError):
        mo.step(np.zeros((4, 9), dtype=np.float32), np.zeros((4, 9), dtype=np.float32), 0.1, 0.0)


def test_bf16_state_variant_rounds_the_moments_after_each_update():
    # Table 3's optimizer-state size (1.6 G at r = 256 for the 7B model) is two bytes per moment entry.
    import torch
    m, n, r = 6, 9, 3
    P = oracle.projection(4, 0, 0, r, m)
    mo = MatrixOracle(m, n, rank=r, seed=4, T=1000, gamma=0.0, state_bf16=True)
    W = np.zeros((m, n), dtype=np.float32)
    M = np.zeros((r, n)); V = np.zeros((r, n))
    rb = lambda a: torch.from_numpy(a).float().to(torch.bfloat16).double().numpy()
    for G in _grads(m, n, 4, seed=23, scale=1.0):
        res = mo.step(W, G, lr=0.1, wd=0.0, want_R=True)
        R = P @ G.astype(np.float64)
        Mn = 0.9 * M + 0.1 * R
        Vn = 0.999 * V + 0.001 * R * R
        s = np.linalg.norm(Mn / (np.sqrt(Vn) + 1e-8), axis=0) / np.linalg.norm(R, axis=0)   # from the unrounded values
        np.testing.assert_allclose(res.s, s, rtol=1e-12)
        M, V = rb(Mn), rb(Vn)
        assert np.array_equal(mo.M, M) and np.array_equal(mo.V, V)
