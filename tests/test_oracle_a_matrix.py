"""Pins for the measurement matrix A = sigma_k * Z used by the oracle (CPU only).

The paper fixes only A's law: i.i.d. zero-mean normal entries of standard deviation 1/sqrt(k)
(Section 3.3).  These tests check that law on the generated values (moments, Kolmogorov distance,
independence along rows and columns, Gram-matrix statistics, column-norm concentration) and keep
the generator frozen through golden vectors.
"""
import itertools

import numpy as np
import pytest
from scipy.stats import norm

import oracle
from golden_util import read_z_golden


@pytest.mark.parametrize("seed", [0, 1, 0x123456789ABCDEF])
def test_golden_vectors(seed):
    blocks, xor, total = read_z_golden(seed)
    assert len(blocks) == 2
    for (r0, c0), want in blocks.items():
        got = oracle.z_block(seed, r0, 32, c0, 32).astype(np.float16).view(np.uint16)
        assert np.array_equal(got, want)
    big = oracle.z_block(seed, 0, 1024, 1000, 1024).astype(np.float16).view(np.uint16)
    assert int(np.bitwise_xor.reduce(big.ravel())) == xor
    assert int(big.ravel().astype(np.uint64).sum()) == total


def test_values_are_binary16_and_block_offsets_consistent():
    z = oracle.z_block(1, 0, 256, 0, 256)
    assert np.array_equal(z.astype(np.float16).astype(np.float32), z)
    sub = oracle.z_block(1, 100, 50, 37, 60)
    assert np.array_equal(sub, z[100:150, 37:97])
    # odd starting rows: the two rows of a pair come from one word, whichever row the block starts at
    assert np.array_equal(oracle.z_block(1, 101, 7, 5, 9), z[101:108, 5:14])


def _all_finite_halves():
    bits = np.arange(1 << 16, dtype=np.uint16)
    vals = bits.view(np.float16).astype(np.float64)
    keep = np.isfinite(vals)
    return bits[keep], vals[keep]


def test_binary16_rounding_matches_numpy_conversion():
    # the oracle restates binary16 arithmetic with doubles; numpy's float64 -> float16 conversion is an
    # independent, correctly rounded implementation of the same rounding
    L = oracle.lib()
    rng = np.random.default_rng(0)
    samples = np.concatenate([
        rng.standard_normal(20000) * 10.0 ** rng.integers(-9, 5, size=20000),
        rng.uniform(-2.0 ** -14, 2.0 ** -14, size=5000),                  # subnormal range
        np.array([0.0, -0.0, 2.0 ** -25, 2.0 ** -24, 3 * 2.0 ** -25, 65504.0, 65519.0, 1.00048828125, 1.0009765625 + 2.0 ** -12]),
    ])
    bits, vals = _all_finite_halves()
    mids = (vals[:-1] + vals[1:]) / 2                                      # exact ties of neighbouring halves
    samples = np.concatenate([samples, mids[np.abs(mids) < 65504][::17]])
    samples = samples[np.abs(samples) < 65519.0]
    want = samples.astype(np.float16).view(np.uint16)
    got = np.array([L.orc_half_round(float(v)) for v in samples], dtype=np.uint16)
    same = (got == want) | ((samples == 0) & ((got & 0x7FFF) == 0) & ((want & 0x7FFF) == 0))
    assert same.all(), samples[~same][:5]
    for b in bits[::37]:
        assert L.orc_half_value(int(b)) == float(np.uint16(b).view(np.float16))


def test_binary16_fma_matches_exact_rational_arithmetic():
    # brute force: the exact value a*b + c as a fraction, rounded by searching the sorted list of all halves
    from fractions import Fraction
    L = oracle.lib()
    bits, vals = _all_finite_halves()
    order = np.argsort(vals, kind="stable")
    sbits, svals = bits[order], vals[order]
    fr = [Fraction(float(v)) for v in svals]

    def nearest_even(x):
        lo, hi = 0, len(fr) - 1
        while hi - lo > 1:
            mid = (lo + hi) // 2
            if fr[mid] <= x:
                lo = mid
            else:
                hi = mid
        dl, dh = x - fr[lo], fr[hi] - x
        if dl < dh:
            return sbits[lo]
        if dh < dl:
            return sbits[hi]
        return sbits[lo] if (int(sbits[lo]) & 1) == 0 else sbits[hi]

    rng = np.random.default_rng(1)
    pool = np.concatenate([rng.integers(0, 1 << 16, size=300).astype(np.uint16), np.array([0x40c2, 0xbad9, 0x3f89], dtype=np.uint16)])
    pool = pool[np.isfinite(pool.view(np.float16).astype(np.float64))]
    # the generator's own operands: x = (S-255)/256, w = x*x, and the polynomial coefficients
    xs = ((np.arange(0, 511, 7) - 255) / 256.0).astype(np.float16).view(np.uint16)
    checked = 0
    for a in np.concatenate([pool[:40], xs[:30]]):
        for b in pool[40:60]:
            for c in pool[60:75]:
                exact = Fraction(float(np.uint16(a).view(np.float16))) * Fraction(float(np.uint16(b).view(np.float16))) + \
                    Fraction(float(np.uint16(c).view(np.float16)))
                if abs(exact) >= 65504:
                    continue
                w = int(nearest_even(exact))
                g = L.orc_half_fma(int(a), int(b), int(c))
                assert (g == w) or ((g & 0x7FFF) == 0 and (w & 0x7FFF) == 0), (hex(a), hex(b), hex(c), hex(g), hex(w))
                checked += 1
    assert checked > 10000


def test_quantile_map_follows_its_definition_on_every_lattice_point():
    # step 5 of the definition, restated with numpy float16 products (exact in float32, one rounding) and
    # float64 sums (exact here), for all 511 byte sums; also: Z is odd and monotone in S
    L = oracle.lib()
    C0, C1, C2 = (np.uint16(v).view(np.float16) for v in (0x40c2, 0xbad9, 0x3f89))
    z = np.array([L.orc_z_of_byte_sum(S) for S in range(511)], dtype=np.uint16).view(np.float16)
    for S in range(511):
        x = np.float16((S - 255) / 256.0)
        w = np.float16(np.float32(x) * np.float32(x))
        q = np.float16(np.float64(w) * np.float64(C2) + np.float64(C1))
        q = np.float16(np.float64(q) * np.float64(w) + np.float64(C0))
        assert np.float16(np.float32(x) * np.float32(q)) == z[S], S
    zf = z.astype(np.float64)
    assert np.array_equal(zf, -zf[::-1]) and np.all(np.diff(zf) > 0) and zf[255] == 0
    pmf = (256 - np.abs(np.arange(511) - 255)) / 65536.0
    assert abs((pmf * zf ** 2).sum() - 1.0) < 1e-4 and abs((pmf * zf ** 4).sum() - 3.0) < 5e-3


def test_sigma_is_rounded_inverse_sqrt():
    for k in (1, 2, 256, 1000, 1024, 2048, 16384):
        assert oracle.sigma(k) == np.float32(1.0 / np.sqrt(np.float64(k)))


@pytest.mark.parametrize("seed,col0", [(0, 0), (1, 0), (1, 16_000_000), (7, 4_000_000_000)])
def test_standard_normal_law(seed, col0):
    z = oracle.z_block(seed, 0, 2048, col0, 1024).astype(np.float64).ravel()
    n = z.size
    assert abs(z.mean()) < 4.0 / np.sqrt(n)
    assert abs(z.var() - 1.0) < 5e-3
    assert abs((z ** 3).mean()) < 0.02
    assert abs((z ** 4).mean() / z.var() ** 2 - 3.0) < 0.03
    assert abs(np.abs(z).mean() - np.sqrt(2 / np.pi)) < 3e-3
    zs = np.sort(z)
    ks = np.max(np.abs(norm.cdf(zs) - (np.arange(n) + 0.5) / n))
    assert ks < 6e-3      # 511 lattice values (largest atom 1/256: 3.5e-3 to the normal) + sampling noise ~ 1e-3
    assert 3.2 < np.abs(z).max() <= 3.37


def test_independence_and_gram_statistics():
    k, ncol = 2048, 1024
    z = oracle.z_block(1, 0, k, 123456, ncol).astype(np.float64)
    assert abs(np.mean(z[:-1] * z[1:])) < 4.0 / np.sqrt(z.size)       # adjacent rows
    assert abs(np.mean(z[:, :-1] * z[:, 1:])) < 4.0 / np.sqrt(z.size)  # adjacent columns
    assert abs(np.mean(z[:-2] * z[2:])) < 4.0 / np.sqrt(z.size)
    a = z * float(oracle.sigma(k))
    G = a.T @ a
    off = G[~np.eye(ncol, dtype=bool)]
    assert abs(off.std() * np.sqrt(k) - 1.0) < 0.02                   # <a_i,a_j> ~ N(0, 1/k)
    assert np.abs(off).max() * np.sqrt(k) < 6.0                        # no coherent column pairs
    assert abs(np.diag(G).mean() - 1.0) < 5e-3                         # column norms concentrate at 1
    assert abs(np.diag(G).std() * np.sqrt(k / 2.0) - 1.0) < 0.1


def test_seed_halves_and_columns_decorrelate():
    k = 1024
    base = oracle.z_block(5, 0, k, 0, 256).astype(np.float64)
    for other_seed in (4, 5 + (1 << 32), 6):
        o = oracle.z_block(other_seed, 0, k, 0, 256).astype(np.float64)
        assert abs(np.mean(base * o)) < 5.0 / np.sqrt(base.size)
    shifted = oracle.z_block(5, 0, k, 1, 256).astype(np.float64)
    assert abs(np.mean(base * shifted)) < 5.0 / np.sqrt(base.size)


def test_restricted_isometry_on_random_supports():
    # Section 3.3: with k >= kappa*s the matrix acts as a near-isometry on s-sparse vectors.
    k, s = 512, 16
    rng = np.random.default_rng(0)
    a = oracle.z_block(3, 0, k, 0, 4096).astype(np.float64) * float(oracle.sigma(k))
    for _ in range(20):
        S = rng.choice(4096, size=s, replace=False)
        sv = np.linalg.svd(a[:, S], compute_uv=False)
        assert 0.6 < sv.min() and sv.max() < 1.4
