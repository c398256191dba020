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
        got = oracle.z_block(seed, r0, 32, c0, 32).view(np.uint32)
        assert np.array_equal(got, want)
    big = oracle.z_block(seed, 0, 1024, 1000, 1024).view(np.uint32)
    assert int(np.bitwise_xor.reduce(big.ravel())) == xor
    assert int(big.ravel().astype(np.uint64).sum()) == total


def test_values_are_bf16_and_block_offsets_consistent():
    z = oracle.z_block(1, 0, 256, 0, 256)
    assert not np.any(z.view(np.uint32) & 0xFFFF)
    sub = oracle.z_block(1, 100, 50, 37, 60)
    assert np.array_equal(sub, z[100:150, 37:97])


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
    assert ks < 4e-3      # lattice of ~850 values + sampling noise 1.36/sqrt(n) ~ 1e-3
    assert 4.0 < np.abs(z).max() <= 4.4375


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
