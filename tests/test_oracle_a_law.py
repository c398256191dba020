"""Does the generated measurement matrix behave like the Gaussian one of Section 3.3 where the method is sensitive?

The paper takes A with i.i.d. N(0, 1/k) entries.  The library's A is a counter-based function whose entries take 511
lattice values with |Z| <= 3.37 (binary16-exact, so that the tensor cores consume it without rounding).  Moments and
Kolmogorov distance are checked elsewhere; what matters for the method is recovery: OMP's success near its phase
transition and the size of the cross-talk that wrong columns produce.  Both are measured here for the oracle's A and for
numpy's standard_normal A of the same shape, with the same plain OMP, and must agree within sampling error.
"""
import numpy as np

import oracle

D, S = 4096, 16


def dense_omp_support(A, norms, y, s):
    """Plain OMP on a dense matrix: normalised argmax, least squares on the support (numpy)."""
    r = y.copy()
    lam = []
    for _ in range(s):
        c = np.abs(A.T @ r) / norms
        c[lam] = -1.0
        lam.append(int(np.argmax(c)))
        x = np.linalg.lstsq(A[:, lam], y, rcond=None)[0]
        r = y - A[:, lam] @ x
    return lam


def matrices(k, law, n_mat):
    for m in range(n_mat):
        if law == "oracle":
            A = float(oracle.sigma(k)) * oracle.z_block(1000 + m, 0, k, 0, D).astype(np.float64)
        else:
            A = np.random.default_rng(5000 + m).standard_normal((k, D)) / np.sqrt(k)
        yield A, np.sqrt((A * A).sum(axis=0))


def success_rate(k, law, n_mat=6, trials=100):
    rng = np.random.default_rng(77 + k)                     # the same planted vectors for both laws
    ok = 0
    for A, norms in matrices(k, law, n_mat):
        for _ in range(trials):
            supp = rng.choice(D, size=S, replace=False)
            x = rng.uniform(1.0, 2.0, size=S) * rng.choice([-1.0, 1.0], size=S)
            y = A[:, supp] @ x
            ok += set(dense_omp_support(A, norms, y, S)) == set(supp.tolist())
    return ok / (n_mat * trials), n_mat * trials


def test_planted_recovery_rate_matches_a_gaussian_matrix_across_the_phase_transition():
    rates = {}
    for k in (64, 96, 128, 192):
        po, n = success_rate(k, "oracle")
        pg, _ = success_rate(k, "gauss")
        rates[k] = (po, pg)
        pbar = 0.5 * (po + pg)
        sigma = np.sqrt(max(2.0 * pbar * (1.0 - pbar) / n, 1e-4))          # std of the difference of two binomial rates
        assert abs(po - pg) <= 4.0 * sigma + 0.01, (k, po, pg, sigma)
    # the sweep really crosses the transition (otherwise equal rates of 0 or 1 would say nothing)
    assert rates[64][1] < 0.2 and rates[192][1] > 0.9, rates
    assert 0.15 < rates[96][1] < 0.95 or 0.15 < rates[128][1] < 0.95, rates


def test_cross_talk_of_wrong_columns_matches_a_gaussian_matrix():
    # For y = A x the score of a column outside the support is ~ N(0, ||y||^2 / k); its maximum over the d columns, in
    # units of ||y|| / sqrt(k), is what decides whether OMP's first picks are right (about sqrt(2 ln 2d) = 4.25).
    k = 256
    stats = {}
    for law in ("oracle", "gauss"):
        rng = np.random.default_rng(9)
        vals = []
        for A, norms in matrices(k, law, 8):
            for _ in range(25):
                supp = rng.choice(D, size=S, replace=False)
                x = rng.uniform(1.0, 2.0, size=S) * rng.choice([-1.0, 1.0], size=S)
                y = A[:, supp] @ x
                c = np.abs(A.T @ y) / norms
                c[supp] = 0.0
                vals.append(c.max() / (np.linalg.norm(y) / np.sqrt(k)))
        stats[law] = (float(np.mean(vals)), float(np.std(vals) / np.sqrt(len(vals))))
    (mo, eo), (mg, eg) = stats["oracle"], stats["gauss"]
    assert abs(mo - mg) <= 4.0 * np.hypot(eo, eg) + 0.02, stats
    target = np.sqrt(2.0 * np.log(2.0 * D))
    assert 0.85 * target < mo < 1.1 * target and 0.85 * target < mg < 1.1 * target, (stats, target)
