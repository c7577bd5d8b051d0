"""Pins for the oracle's Philox4x32-10 and its mapping onto the entries of P."""
from pathlib import Path

import numpy as np

import oracle

GOLDEN = Path(__file__).resolve().parent / "golden" / "philox4x32_10_kat.txt"


def _kat_rows():
    for line in GOLDEN.read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        v = [int(x, 16) for x in line.split()]
        yield v[:4], v[4:6], v[6:]


def test_known_answer_vectors():
    rows = list(_kat_rows())
    assert len(rows) >= 2
    for ctr, key, want in rows:
        assert list(oracle.philox4x32_10(ctr, key)) == want


def _philox_limbs(ctr, key):
    """Second coding: 16-bit limb products on Python integers, no 64-bit multiply."""
    def mulhilo(a, b):
        a0, a1, b0, b1 = a & 0xFFFF, a >> 16, b & 0xFFFF, b >> 16
        p00, p01, p10, p11 = a0 * b0, a0 * b1, a1 * b0, a1 * b1
        mid = (p00 >> 16) + (p01 & 0xFFFF) + (p10 & 0xFFFF)
        lo = (p00 & 0xFFFF) | ((mid & 0xFFFF) << 16)
        hi = p11 + (p01 >> 16) + (p10 >> 16) + (mid >> 16)
        return hi & 0xFFFFFFFF, lo & 0xFFFFFFFF
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        hi0, lo0 = mulhilo(0xD2511F53, c[0])
        hi1, lo1 = mulhilo(0xCD9E8D57, c[2])
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_second_coding_agrees_on_random_inputs():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        assert list(oracle.philox4x32_10(ctr, key)) == _philox_limbs(ctr, key)


def test_limb_coding_matches_known_answers():
    for ctr, key, want in _kat_rows():
        assert _philox_limbs(ctr, key) == want


def test_draw_layout_counter_is_quad_row_matrix_epoch():
    seed = 0x0123456789ABCDEF
    d = oracle.philox_draws(seed, 5, 9, 3, 10)          # m=10 -> 3 quads
    assert d.shape == (3, 3, 4)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for k in range(3):
        for q in range(3):
            assert list(d[k, q]) == list(oracle.philox4x32_10([q, k, 5, 9], key))


def test_streams_differ_across_matrix_epoch_seed_and_repeat_exactly():
    a = oracle.philox_draws(42, 0, 0, 4, 16)
    assert np.array_equal(a, oracle.philox_draws(42, 0, 0, 4, 16))
    for other in (oracle.philox_draws(42, 1, 0, 4, 16), oracle.philox_draws(42, 0, 1, 4, 16),
                  oracle.philox_draws(43, 0, 0, 4, 16), oracle.philox_draws(42 + (1 << 32), 0, 0, 4, 16)):
        assert not np.array_equal(a, other)
        assert np.mean(a == other) < 0.01


def test_rows_of_a_wider_matrix_extend_the_narrower_one():
    # P[k][i] depends only on (k, i): same leading entries for any m, any r.
    a = oracle.philox_draws(3, 2, 1, 2, 8)
    b = oracle.philox_draws(3, 2, 1, 5, 40)
    assert np.array_equal(a, b[:2, :2])


def test_output_words_are_uniform():
    d = oracle.philox_draws(11, 0, 0, 64, 4096).reshape(-1).astype(np.float64)
    u = d / 2.0**32
    assert abs(u.mean() - 0.5) < 2e-3
    assert abs(u.var() - 1.0 / 12.0) < 1e-3
    # every bit is set about half of the time
    w = oracle.philox_draws(11, 0, 0, 64, 4096).reshape(-1)
    for bit in range(32):
        frac = np.mean((w >> np.uint32(bit)) & np.uint32(1))
        assert abs(frac - 0.5) < 0.01
