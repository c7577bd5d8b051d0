"""Pins for the oracle's Gaussian projection P ~ N(0, 1/r) (Algorithm 1; Appendix,
"Norm Preservation" theorem: E[P^T P] = I_m and r |Px|^2 / |x|^2 ~ chi-square with r
degrees of freedom) and for its bfloat16 rounding."""
import numpy as np
import scipy.stats
import torch

import oracle


def test_standard_normals_pass_a_kolmogorov_smirnov_test():
    z = oracle.standard_normals(42, 0, 0, 256, 4096).reshape(-1)
    assert z.size == 2**20
    assert abs(z.mean()) < 4e-3
    assert abs(z.var() - 1.0) < 5e-3
    assert abs(scipy.stats.kurtosis(z, fisher=False) - 3.0) < 0.03
    assert abs(scipy.stats.skew(z)) < 0.01
    assert scipy.stats.kstest(z[:200000], "norm").pvalue > 1e-3


def test_box_muller_pairs_share_a_radius_fixed_by_the_first_word():
    # z[4q]^2 + z[4q+1]^2 = -2 ln u1 with u1 from the top 23 bits of word 0; same for words 2, 3.
    r, m = 3, 24
    z = oracle.standard_normals(9, 1, 2, r, m).reshape(r, m // 4, 4)
    d = oracle.philox_draws(9, 1, 2, r, m)
    for h in range(2):
        u1 = 1.0 - (d[..., 2 * h] >> np.uint32(9)).astype(np.float64) / 2.0**23
        rad2 = z[..., 2 * h] ** 2 + z[..., 2 * h + 1] ** 2
        np.testing.assert_allclose(rad2, -2.0 * np.log(u1), rtol=1e-12)
        u2 = (d[..., 2 * h + 1] >> np.uint32(9)).astype(np.float64) / 2.0**23
        ang = np.arctan2(z[..., 2 * h + 1], z[..., 2 * h])
        want = 2 * np.pi * (u2 - 0.5)
        np.testing.assert_allclose(np.mod(ang - want + np.pi, 2 * np.pi) - np.pi, 0.0, atol=1e-9)


def test_ragged_m_drops_the_tail_of_the_last_quad():
    a = oracle.standard_normals(5, 0, 0, 4, 10)
    b = oracle.standard_normals(5, 0, 0, 4, 12)
    assert np.array_equal(a, b[:, :10])


def test_entries_have_variance_one_over_r():
    for r in (1, 16, 128):
        P = oracle.projection(1, 0, 0, r, 8192 // r * 16, round_bf16=False)
        assert abs(P.var() * r - 1.0) < 0.02
        Pb = oracle.projection(1, 0, 0, r, 8192 // r * 16, round_bf16=True)
        assert abs(Pb.var() * r - 1.0) < 0.02
        # rounding to bf16 moves an entry by at most 2^-9 relative
        np.testing.assert_allclose(Pb, P, rtol=2.0**-8, atol=0)


def test_expected_gram_matrix_is_identity():
    r, m, trials = 8, 12, 4000
    acc = np.zeros((m, m))
    for seed in range(trials):
        P = oracle.projection(seed, 0, 0, r, m, round_bf16=False)
        acc += P.T @ P
    acc /= trials
    # each entry of the average has standard deviation <= sqrt(2 / (r trials))
    assert np.max(np.abs(acc - np.eye(m))) < 6.0 * np.sqrt(2.0 / (r * trials))


def test_projected_norm_follows_chi_square_r():
    r, m, trials = 16, 40, 3000
    x = np.random.default_rng(0).standard_normal(m)
    zs = np.empty(trials)
    for seed in range(trials):
        P = oracle.projection(1000 + seed, 3, 1, r, m, round_bf16=False)
        zs[seed] = r * np.sum((P @ x) ** 2) / np.sum(x**2)
    assert abs(zs.mean() - r) < 5 * np.sqrt(2.0 * r / trials)
    assert abs(zs.var() - 2 * r) < 0.15 * 2 * r
    assert scipy.stats.kstest(zs, "chi2", args=(r,)).pvalue > 1e-3


def test_round_bf16_matches_torch_on_float_inputs():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(20000, generator=g) * torch.pow(10.0, torch.rand(20000, generator=g) * 8 - 4)
    want = x.to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.round_bf16(float(v)) for v in x.to(torch.float64).numpy()])
    assert np.array_equal(got, want)


def test_round_bf16_ties_and_no_double_rounding():
    ulp = 2.0**-7                      # bf16 spacing in [1, 2)
    assert oracle.round_bf16(1.0 + ulp / 2) == 1.0                 # tie -> even mantissa
    assert oracle.round_bf16(1.0 + ulp + ulp / 2) == 1.0 + 2 * ulp   # tie -> even mantissa
    assert oracle.round_bf16(1.0 + ulp / 2 + 2.0**-30) == 1.0 + ulp  # above the tie in double only
    assert oracle.round_bf16(1.0 + ulp / 2 - 2.0**-30) == 1.0
    assert oracle.round_bf16(-(1.0 + ulp / 2 + 2.0**-30)) == -(1.0 + ulp)
    assert oracle.round_bf16(0.0) == 0.0
    assert oracle.round_bf16(2.0 - 2.0**-10) == 2.0                  # carries into the next binade
