"""Pins for the oracle's noise stream: published Philox4x32-10 known answers, a second
Philox written with python integers, closed-form Box-Muller values, and the
distribution the paper asks for, N(0,1) scaled by sigma*C (section 2)."""
import math
import os
import numpy as np
from scipy import stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def _philox_python(ctr, key):
    """Independent restatement with python big integers (mulhi via >> 32)."""
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        lo0, hi0 = (0xD2511F53 * c[0]) & 0xFFFFFFFF, (0xD2511F53 * c[0]) >> 32
        lo1, hi1 = (0xCD9E8D57 * c[2]) & 0xFFFFFFFF, (0xCD9E8D57 * c[2]) >> 32
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_published_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert oracle.philox4x32_10(ctr, key) == out
        assert _philox_python(ctr, key) == out


def test_matches_python_restatement_on_random_inputs():
    rng = np.random.default_rng(0)
    for _ in range(200):
        ctr = [int(v) for v in rng.integers(0, 2 ** 32, 4)]
        key = [int(v) for v in rng.integers(0, 2 ** 32, 2)]
        assert oracle.philox4x32_10(ctr, key) == _philox_python(ctr, key)


def test_counter_and_key_layout():
    seed, step, block = 0x0123456789ABCDEF, 0x0FEDCBA987654321, (5 << 32) | 17
    w = oracle.philox_blocks(seed, step, block, 2)
    assert list(w[0]) == _philox_python([17, 5, 0x87654321, 0x0FEDCBA9], [0x89ABCDEF, 0x01234567])
    assert list(w[1]) == _philox_python([18, 5, 0x87654321, 0x0FEDCBA9], [0x89ABCDEF, 0x01234567])


def test_box_muller_closed_form():
    """z from the raw words by the textbook transform, done here with python floats."""
    for seed, step, i0 in [(0, 0, 0), (42, 3, 20), (2 ** 40 + 1, 2 ** 33, 2 ** 34 + 4)]:
        w = _philox_python([(i0 // 4) & 0xFFFFFFFF, (i0 // 4) >> 32, step & 0xFFFFFFFF, step >> 32],
                           [seed & 0xFFFFFFFF, seed >> 32])
        z = oracle.noise_z(seed, step, i0, 4)
        for pair in range(2):
            u1 = ((w[2 * pair] >> 9) + 0.5) / 2 ** 23
            u2 = (w[2 * pair + 1] >> 8) / 2 ** 24
            assert 0.0 < u1 < 1.0 and 0.0 <= u2 < 1.0
            r = math.sqrt(-2.0 * math.log(u1))
            assert abs(z[2 * pair] - r * math.cos(2 * math.pi * u2)) < 1e-14
            assert abs(z[2 * pair + 1] - r * math.sin(2 * math.pi * u2)) < 1e-14


def test_first_values_of_the_default_stream():
    # seed 0, step 0, block 0 is the all-zero known-answer vector: 6627e8d5 e169c58d bc57ac4c 9b00dbd8
    u1 = ((0x6627E8D5 >> 9) + 0.5) / 2 ** 23
    u2 = (0xE169C58D >> 8) / 2 ** 24
    z = oracle.noise_z(0, 0, 0, 4)
    assert abs(u1 - 0.3990464807) < 1e-9 and abs(u2 - 0.8805201650) < 1e-9
    assert abs(z[0] - math.sqrt(-2 * math.log(u1)) * math.cos(2 * math.pi * u2)) < 1e-14
    assert abs(z[0] - 0.9911374751) < 1e-8 and abs(z[1] + 0.9246627804) < 1e-8


def test_values_depend_only_on_the_global_index():
    a = oracle.noise_z(3, 4, 0, 103)
    b = np.concatenate([oracle.noise_z(3, 4, 0, 5), oracle.noise_z(3, 4, 5, 62), oracle.noise_z(3, 4, 67, 36)])
    np.testing.assert_array_equal(a, b)


def test_standard_normal_statistics():
    n = 2_000_000
    z = oracle.noise_z(0, 0, 0, n)
    assert abs(z.mean()) < 5 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 5 * math.sqrt(2.0 / n)
    assert np.abs(z).max() <= math.sqrt(-2 * math.log(2.0 ** -24)) + 1e-12   # truncation of the tail
    assert abs(stats.skew(z)) < 0.01 and abs(stats.kurtosis(z)) < 0.02
    assert stats.kstest(z[:200_000], "norm").pvalue > 1e-3
    for lane in range(4):                                                    # each lane is N(0,1) by itself
        assert abs(z[lane::4].var() - 1.0) < 0.01
    assert abs(np.corrcoef(z[0::4], z[1::4])[0, 1]) < 0.005                  # cos/sin partners
    assert abs(np.corrcoef(z[:-1], z[1:])[0, 1]) < 0.005


def test_streams_of_different_seed_or_step_are_uncorrelated():
    n = 400_000
    a = oracle.noise_z(0, 0, 0, n)
    b = oracle.noise_z(1, 0, 0, n)
    c = oracle.noise_z(0, 1, 0, n)
    for x, y in [(a, b), (a, c), (b, c)]:
        assert abs(np.corrcoef(x, y)[0, 1]) < 5 / math.sqrt(n)
    assert not np.array_equal(a, b) and not np.array_equal(a, c)


def test_scaled_noise_has_std_sigma_C_and_per_example_form_has_the_same_variance():
    """Section 2: N(0, sigma^2 C^2) on the sum; |B| draws of variance sigma^2 C^2/|B| add up to the same."""
    P, sigma, C, Bt = 300_000, 1.3, 0.7, 16
    out = oracle.noise_average(np.zeros(P), 0, sigma, C, Bt, 5, 0)
    assert abs(out.std() * Bt - sigma * C) < 5 * sigma * C / math.sqrt(2 * P)
    per_example = sum(oracle.noise_z(100 + n, 0, 0, P) for n in range(Bt)) * (sigma * C / math.sqrt(Bt))
    assert abs(per_example.std() - sigma * C) < 5 * sigma * C / math.sqrt(2 * P)


def test_example_stream_layout_and_independence():
    """Per-example noise (section 2, the paper's own variant): counter word 1 carries 0x80000000 | example."""
    seed, step, e, g0 = 77, 5, 9, 40
    w = _philox_python([g0 // 4, 0x80000000 | e, step, 0], [seed, 0])
    z = oracle.example_noise_z(seed, step, e, g0, 4)
    for pair in range(2):
        u1 = ((w[2 * pair] >> 9) + 0.5) / 2 ** 23
        u2 = (w[2 * pair + 1] >> 8) / 2 ** 24
        r = math.sqrt(-2.0 * math.log(u1))
        assert abs(z[2 * pair] - r * math.cos(2 * math.pi * u2)) < 1e-14
        assert abs(z[2 * pair + 1] - r * math.sin(2 * math.pi * u2)) < 1e-14
    n = 200_000
    a, b, c = oracle.example_noise_z(1, 0, 0, 0, n), oracle.example_noise_z(1, 0, 1, 0, n), oracle.noise_z(1, 0, 0, n)
    for x, y in [(a, b), (a, c), (b, c)]:
        assert abs(np.corrcoef(x, y)[0, 1]) < 5 / math.sqrt(n)
    assert abs(a.var() - 1.0) < 0.02 and abs(a.mean()) < 0.02


def test_per_example_noised_sum_is_the_clipped_sum_plus_the_example_draws():
    B, P, sd = 5, 64, 0.3
    G = np.random.default_rng(3).standard_normal((B, P)).astype(np.float32)
    f = np.linspace(0.2, 1.0, B)
    acc = oracle.clip_accumulate_noised(G, f, np.zeros(P), sd, 8, 2, 10, 100)
    want = np.einsum("n,np->p", f, G.astype(np.float64)) + sd * sum(oracle.example_noise_z(8, 2, 10 + n, 100, P) for n in range(B))
    np.testing.assert_allclose(acc, want, rtol=1e-13, atol=1e-13)
    # sd = sigma*C/sqrt(|B|) over |B| examples gives total variance (sigma*C)^2
    Bt, Pn = 16, 100_000
    tot = sum(oracle.example_noise_z(4, 0, e, 0, Pn) for e in range(Bt)) * (1.3 * 0.7 / math.sqrt(Bt))
    assert abs(tot.std() - 1.3 * 0.7) < 5 * 1.3 * 0.7 / math.sqrt(2 * Pn)
