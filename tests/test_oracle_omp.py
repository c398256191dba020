"""Pins for the oracle's recovery step a4 (OMP, Eq. 7 / Appendix B) and for the whole step (CPU only)."""
import itertools

import numpy as np
import pytest

import oracle


def dense_A(seed, k, d):
    return oracle.z_block(seed, 0, k, 0, d).astype(np.float64) * np.float64(oracle.sigma(k))


def numpy_omp(A, y, s):
    """Dense restatement with library routines: argmax of |A^T r| / ||A_i||, numpy lstsq on the support."""
    k, d = A.shape
    nrm = np.linalg.norm(A, axis=0)
    r = y.copy()
    lam = []
    for _ in range(s):
        c = np.abs(A.T @ r) / nrm
        c[lam] = -1.0
        lam.append(int(np.argmax(c)))
        x, *_ = np.linalg.lstsq(A[:, lam], y, rcond=None)
        r = y - A[:, lam] @ x
    return lam, x, r


def test_exact_recovery_of_planted_sparse_vector():
    # k comfortably above s*log(d/s): OMP returns the planted support and values (Section 3.3).
    seed, d, k, s = 11, 4096, 512, 8
    rng = np.random.default_rng(5)
    supp = np.sort(rng.choice(d, size=s, replace=False))
    xs = rng.uniform(1.0, 2.0, size=s) * rng.choice([-1.0, 1.0], size=s)
    A = dense_A(seed, k, d)
    y = A[:, supp] @ xs
    out = oracle.omp(seed, d, k, s, y)
    assert out["done"] == s
    order = np.argsort(out["lam"])
    assert np.array_equal(out["lam"][order], supp.astype(np.uint32))
    np.testing.assert_allclose(out["x"][order], xs, rtol=1e-9)
    assert out["rnorm"][-1] < 1e-10 * np.linalg.norm(y)
    assert np.all(np.diff(out["rnorm"]) <= 1e-12)                 # residual norm never increases
    assert np.all(out["top1"] >= out["top2"])


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_brute_force_over_every_support(seed):
    # On a tiny problem with exact recovery the OMP support is the global least-squares minimiser
    # over all supports of size s, and x is the least-squares solution on it.
    d, k, s = 18, 12, 3
    rng = np.random.default_rng(100 + seed)
    supp = np.sort(rng.choice(d, size=s, replace=False))
    xs = rng.uniform(1.0, 2.0, size=s) * rng.choice([-1.0, 1.0], size=s)
    A = dense_A(seed, k, d)
    y = A[:, supp] @ xs
    best, best_S = np.inf, None
    for S in itertools.combinations(range(d), s):
        x, *_ = np.linalg.lstsq(A[:, S], y, rcond=None)
        res = np.linalg.norm(y - A[:, S] @ x)
        if res < best:
            best, best_S = res, S
    out = oracle.omp(seed, d, k, s, y)
    lam_np, x_np, _ = numpy_omp(A, y, s)
    assert out["lam"].tolist() == lam_np                               # same greedy path as the dense restatement
    if best < 1e-9 and sorted(lam_np) == list(supp):
        assert sorted(out["lam"].tolist()) == list(best_S)
    xls, *_ = np.linalg.lstsq(A[:, out["lam"].astype(int)], y, rcond=None)
    np.testing.assert_allclose(out["x"], xls, rtol=1e-9, atol=1e-12)


def test_matches_dense_numpy_restatement_on_noisy_target():
    # inexact regime: y is not s-sparse in A; every pick, the coefficients and residual norms must still agree
    seed, d, k, s = 6, 700, 48, 10
    rng = np.random.default_rng(2)
    A = dense_A(seed, k, d)
    y = rng.standard_normal(k)
    out = oracle.omp(seed, d, k, s, y)
    lam_np, x_np, r_np = numpy_omp(A, y, s)
    assert out["lam"].tolist() == lam_np
    np.testing.assert_allclose(out["x"], x_np, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(out["rnorm"][-1], np.linalg.norm(r_np), rtol=1e-10)
    # residual orthogonal to the selected columns
    r = y - A[:, lam_np] @ out["x"]
    assert np.abs(A[:, lam_np].T @ r).max() < 1e-12
    # top1/top2 records are the two largest normalised correlations of the first iteration
    c = np.sort(np.abs(A.T @ y) / np.linalg.norm(A, axis=0))[::-1]
    np.testing.assert_allclose([out["top1"][0], out["top2"][0]], c[:2], rtol=1e-12)


def test_scale_invariance():
    seed, d, k, s = 8, 2000, 96, 12
    rng = np.random.default_rng(9)
    y = rng.standard_normal(k)
    a = oracle.omp(seed, d, k, s, y)
    b = oracle.omp(seed, d, k, s, 37.5 * y)
    assert np.array_equal(a["lam"], b["lam"])
    np.testing.assert_allclose(b["x"], 37.5 * a["x"], rtol=1e-10)


def test_lowest_index_wins_exact_ties_and_no_reselection():
    # y = 0 gives all-zero correlations: every pick is an exact tie -> lowest unselected index; the
    # columns are independent so all s iterations complete with zero coefficients.
    out = oracle.omp(3, 50, 16, 4, np.zeros(16))
    assert out["lam"].tolist() == [0, 1, 2, 3] and not out["x"].any()


def test_dependent_column_stops_early():
    # k = 2 rows: two picked columns span the plane, so whichever column the third iteration picks is a combination of
    # them.  Algorithm 3's gamma = 1/sqrt(g_ll - c^H c) would divide by ~0 there; the oracle's reading is that the
    # recovery ends with the picks made so far.  s = 3 > k reaches that branch (s = 2 never does).
    y = np.array([1.0, -2.0])
    two = oracle.omp(3, 6, 2, 2, y)
    assert two["done"] == 2
    out = oracle.omp(3, 6, 2, 3, y)
    assert out["done"] == 2
    assert out["lam"][2] == 0xFFFFFFFF and out["x"][2] == 0.0 and out["rnorm"][2] == 0.0
    # the picks before the stop are those of the shorter run, and so is the least-squares fit
    assert np.array_equal(out["lam"][:2], two["lam"]) and np.array_equal(out["x"][:2], two["x"])
    # the fit on two independent columns of the plane is exact
    A = _columns(3, 2, out["lam"][:2])
    np.testing.assert_allclose(A @ out["x"][:2], y, atol=1e-12)
    # the same with k = 3: three picks complete (the stop does not fire on independent columns), the fourth cannot
    y3 = np.array([0.5, -1.0, 2.0])
    for seed in range(5):
        assert oracle.omp(seed, 40, 3, 3, y3)["done"] == 3
        o4 = oracle.omp(seed, 40, 3, 4, y3)
        assert o4["done"] == 3 and o4["lam"][3] == 0xFFFFFFFF
        assert len(set(o4["lam"][:3].tolist())) == 3


def _sin2_of_first_two_columns(seed):
    Z = oracle.z_block(seed, 0, 2, 0, 2).astype(np.float64)
    a, b = Z[:, 0], Z[:, 1]
    return (a[0] * b[1] - a[1] * b[0]) ** 2 / ((a @ a) * (b @ b))


def test_dependence_threshold_from_both_sides():
    # The stop is for a column whose component outside the span of the support is below 1e-5 of its norm (1e-10 in the
    # squared, relative pivot).  With k = 2 and d = 2 the second pick is forced, so the angle between the two columns
    # decides: seeds found by search whose first two columns are exactly parallel, at sin^2 = 6.2e-11 (stop) and at
    # sin^2 = 1.5e-9 (an ordinary, if ill-conditioned, pick).  A threshold off by a factor of 20 either way fails.
    y = np.array([0.3, 1.0])
    assert _sin2_of_first_two_columns(66855) == 0.0
    assert oracle.omp(66855, 2, 2, 2, y)["done"] == 1
    s2 = _sin2_of_first_two_columns(112200)
    assert 5e-11 < s2 < 1e-10
    out = oracle.omp(112200, 2, 2, 2, y)
    assert out["done"] == 1 and out["lam"][1] == 0xFFFFFFFF and out["x"][1] == 0.0
    s2 = _sin2_of_first_two_columns(143364)
    assert 1e-9 < s2 < 2e-9
    out = oracle.omp(143364, 2, 2, 2, y)
    assert out["done"] == 2 and sorted(out["lam"].tolist()) == [0, 1]
    A = _columns(143364, 2, out["lam"])
    np.testing.assert_allclose(A @ out["x"], y, rtol=0, atol=1e-7)      # condition number ~ 5e4


def _columns(seed, k, lam):
    return float(oracle.sigma(k)) * np.stack([oracle.z_block(seed, 0, k, int(c), 1)[:, 0] for c in lam], axis=1).astype(np.float64)


def test_whole_step_constant_sparse_gradient_closed_form():
    # A gradient with exactly s non-zeros, held constant: Mhat = A g, Vhat = A g^2 for all t, OMP recovers
    # both exactly, so N = alpha * g / (|g| + eps) = alpha * sign(g) and W_t = W_0 - t*eta*alpha*sign(g).
    d, k, s, seed = 2048, 256, 6, 21
    lr, alpha = np.float32(1e-3), 2.0
    rng = np.random.default_rng(4)
    supp = np.sort(rng.choice(d, size=s, replace=False))
    g = np.zeros(d, dtype=np.float32)
    g[supp] = (rng.uniform(1.0, 2.0, size=s) * rng.choice([-1.0, 1.0], size=s)).astype(np.float32)
    W0 = rng.standard_normal(d).astype(np.float32)
    W = W0.copy()
    st = oracle.Oracle(d, k, s, seed, lr, 0.9, 0.999, 1e-8, alpha=alpha)
    for t in range(1, 6):
        st.step(g, W)
        assert st.get("t") == t
        assert np.array_equal(st.get("sel_idx"), supp.astype(np.uint32))
        assert sorted(st.get("lamM").tolist()) == supp.tolist() == sorted(st.get("lamV").tolist())
        assert st.get("mismatch") == 0 and st.get("negv") == 0 and st.get("n_upd") == s
        order = np.argsort(st.get("lamM"))
        np.testing.assert_allclose(st.get("xM")[order], g[supp], rtol=2e-6)      # fp32 state rounding
        want = W0.astype(np.float64)
        want[supp] -= t * np.float64(lr) * alpha * np.sign(g[supp])
        np.testing.assert_allclose(W, want, rtol=0, atol=3e-6)
        untouched = np.ones(d, dtype=bool)
        untouched[supp] = False
        assert np.array_equal(W[untouched], W0[untouched])
    st.close()


def test_step_split_equals_whole_step():
    d, k, s = 512, 64, 4
    rng = np.random.default_rng(12)
    a = oracle.Oracle(d, k, s, 1, 1e-3, 0.9, 0.999, 1e-8)
    b = oracle.Oracle(d, k, s, 1, 1e-3, 0.9, 0.999, 1e-8)
    Wa = rng.standard_normal(d).astype(np.float32)
    Wb = Wa.copy()
    for _ in range(3):
        g = rng.standard_normal(d).astype(np.float32)
        a.step(g, Wa)
        b.step_compress(g)
        b.step_recover(Wb)
    assert np.array_equal(Wa, Wb) and np.array_equal(a.get("M"), b.get("M"))


def test_create_rejects_bad_arguments():
    for (d, k, s) in [(0, 4, 1), (10, 0, 1), (10, 4, 0), (10, 4, 5), (3, 8, 4), (1 << 32, 8, 4)]:
        with pytest.raises(ValueError):
            oracle.Oracle(d, k, s, 0, 1e-3, 0.9, 0.999, 1e-8)


# ---- opt-in variant: shared support and early stop (remark after Eq. (8)) -----------------------------------
def test_least_squares_on_a_support_is_numpy_lstsq():
    seed, d, k = 3, 1000, 96
    rng = np.random.default_rng(8)
    lam = rng.choice(d, size=7, replace=False).astype(np.uint32)
    y = rng.standard_normal(k)
    A = dense_A(seed, k, d)
    want, *_ = np.linalg.lstsq(A[:, lam.astype(np.int64)], y, rcond=None)
    np.testing.assert_allclose(oracle.least_squares(seed, k, lam, y), want, rtol=1e-10, atol=1e-12)


def test_early_stop_ends_at_the_sparsity_of_an_exactly_sparse_target():
    # y has 5 non-zeros in the A-basis; with k this large OMP finds them in 5 picks and the residual drops to rounding
    # noise, so a tolerance of 1e-9 stops there, while tolerance 0 runs all s iterations (Algorithm 3 as printed)
    seed, d, k, s, s0 = 17, 3000, 400, 12, 5
    rng = np.random.default_rng(3)
    supp = rng.choice(d, size=s0, replace=False)
    A = dense_A(seed, k, d)
    y = A[:, supp] @ rng.uniform(1.0, 2.0, size=s0)
    full = oracle.omp(seed, d, k, s, y)
    early = oracle.omp(seed, d, k, s, y, residual_tol=1e-9)
    assert full["done"] == s and early["done"] == s0
    assert np.array_equal(early["lam"][:s0], full["lam"][:s0]) and sorted(early["lam"][:s0].tolist()) == sorted(supp.tolist())
    assert np.all(early["lam"][s0:] == 0xFFFFFFFF) and np.all(early["x"][s0:] == 0.0)
    # a tolerance the first residual already meets stops after one pick; the stop never changes the picks made before it
    one = oracle.omp(seed, d, k, s, y, residual_tol=1.0)
    assert one["done"] == 1 and one["lam"][0] == full["lam"][0]
    # the coefficients at the stop are the least-squares fit on the picks made so far
    np.testing.assert_allclose(early["x"][:s0], oracle.least_squares(seed, k, early["lam"][:s0], y), rtol=1e-9)


def test_shared_support_step_against_its_definition():
    # noisy gradients: the two printed recoveries pick different columns late on; the variant keeps OMP_A(M^)'s picks
    # for both moments and fits V^ on them by least squares (numpy restatement), then applies Eq. (8) on that support
    d, k, s, seed = 1500, 128, 10, 9
    lr, eps, alpha = np.float32(1e-3), np.float32(1e-8), 2.0
    rng = np.random.default_rng(31)
    plain = oracle.Oracle(d, k, s, seed, lr, 0.9, 0.999, eps, alpha=alpha)
    var = oracle.Oracle(d, k, s, seed, lr, 0.9, 0.999, eps, alpha=alpha)
    var.set_recovery(True)
    A = dense_A(seed, k, d)
    Wp = rng.standard_normal(d).astype(np.float32)
    Wv = Wp.copy()
    differed = False
    for _ in range(4):
        g = (rng.standard_t(3.0, size=d) * 1e-2).astype(np.float32)
        W_before = Wv.copy()
        plain.step(g, Wp)
        var.step(g, Wv)
        # a1-a3 and the recovery of M^ do not depend on the variant
        for name in ("sel_idx", "M", "V", "lamM", "xM", "Mhat", "Vhat"):
            assert np.array_equal(plain.get(name), var.get(name)), name
        lam = var.get("lamM").astype(np.int64)
        assert np.array_equal(var.get("lamV"), var.get("lamM")) and var.get("doneV") == var.get("doneM") == s
        want, *_ = np.linalg.lstsq(A[:, lam], var.get("Vhat"), rcond=None)
        np.testing.assert_allclose(var.get("xV"), want, rtol=1e-8, atol=1e-14)
        differed |= sorted(plain.get("lamV").tolist()) != sorted(lam.tolist())
        # Eq. (8) on the one support, guarded where x^V <= 0
        xM, xV = var.get("xM"), var.get("xV")
        ok = xV > 0
        assert var.get("mismatch") == 0 and var.get("negv") == int((~ok).sum()) and var.get("n_upd") == int(ok.sum())
        expect = W_before.astype(np.float64)
        expect[lam[ok]] -= np.float64(lr) * alpha * xM[ok] / (np.sqrt(xV[ok]) + np.float64(eps))
        np.testing.assert_allclose(Wv, expect.astype(np.float32), rtol=0, atol=1e-7)
    assert differed          # otherwise this test would not tell the variant from Algorithm 2 as printed
    plain.close()
    var.close()


def test_shared_support_equals_the_printed_algorithm_when_the_supports_coincide():
    # constant exactly sparse gradient: both printed recoveries return the planted support (the premise of the remark after
    # Eq. (8)), so the variant must reproduce the printed step up to the order in which x^V is listed
    d, k, s, seed = 2048, 256, 6, 21
    rng = np.random.default_rng(4)
    supp = np.sort(rng.choice(d, size=s, replace=False))
    g = np.zeros(d, dtype=np.float32)
    g[supp] = (rng.uniform(1.0, 2.0, size=s) * rng.choice([-1.0, 1.0], size=s)).astype(np.float32)
    a = oracle.Oracle(d, k, s, seed, 1e-3, 0.9, 0.999, 1e-8)
    b = oracle.Oracle(d, k, s, seed, 1e-3, 0.9, 0.999, 1e-8)
    b.set_recovery(True, 0.0)
    Wa = rng.standard_normal(d).astype(np.float32)
    Wb = Wa.copy()
    for _ in range(3):
        a.step(g, Wa)
        b.step(g, Wb)
        assert np.array_equal(a.get("upd_idx"), b.get("upd_idx"))
        np.testing.assert_allclose(b.get("upd_val"), a.get("upd_val"), rtol=1e-9)
        np.testing.assert_allclose(Wb, Wa, rtol=0, atol=1e-9)
    a.close()
    b.close()


# ---- the batched Select (used to check picks at full size, where s whole iterations are out of reach) --------------
def test_select_is_the_dense_normalised_argmax_for_every_residual():
    seed, d, k, n = 12, 3000, 48, 7
    rng = np.random.default_rng(0)
    R = rng.standard_normal((n, k))
    R[3] = 0.0                                                          # all scores tie at zero: lowest free index
    skip = [sorted(rng.choice(d, size=q, replace=False).tolist()) for q in (0, 1, 5, 2, 0, 9, 3)]
    skip[3] = [0, 1]
    out = oracle.select(seed, d, k, R, skip)
    Z = oracle.z_block(seed, 0, k, 0, d).astype(np.float64)
    A = float(oracle.sigma(k)) * Z
    sc = np.abs(R @ A) / np.sqrt((A * A).sum(axis=0))                   # n x d, the definition with A written out
    for i in range(n):
        s_i = sc[i].copy()
        s_i[skip[i]] = -1.0
        order = np.argsort(-s_i, kind="stable")                         # stable: ties keep the lower index first
        assert out["idx"][i] == order[0], i
        np.testing.assert_allclose(out["best"][i], s_i[order[0]], rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(out["second"][i], s_i[order[1]], rtol=1e-12, atol=1e-300)
    assert out["idx"][3] == 2
    # without skip lists
    out0 = oracle.select(seed, d, k, R)
    assert np.array_equal(out0["idx"], np.argmax(sc, axis=1))


def test_select_reproduces_every_iteration_of_omp():
    # feeding Select the residual before each iteration of a full OMP run (with the support so far excluded) must give
    # that run's picks and scores back: the batch is s independent copies of one iteration
    seed, d, k, s = 5, 20_000, 96, 12
    rng = np.random.default_rng(3)
    supp = rng.choice(d, size=s, replace=False)
    A_s = _columns(seed, k, supp)
    y = A_s @ rng.uniform(1.0, 2.0, size=s) + 0.05 * rng.standard_normal(k)
    run = oracle.omp(seed, d, k, s, y)
    R, skip = [], []
    for j in range(s):
        lam = run["lam"][:j]
        r = y if j == 0 else y - _columns(seed, k, lam) @ oracle.least_squares(seed, k, lam, y)
        R.append(r)
        skip.append(lam.tolist())
    out = oracle.select(seed, d, k, np.array(R), skip)
    assert np.array_equal(out["idx"], run["lam"].astype(np.int64))
    np.testing.assert_allclose(out["best"], run["top1"], rtol=1e-9)
    np.testing.assert_allclose(out["second"], run["top2"], rtol=1e-9)
