"""Pins for the oracle's steps a1-a3 and a5 (CPU only): plain definitions on dense matrices,
closed forms and invariants that the paper states."""
import numpy as np
import pytest

import oracle


def dense_A(seed, k, d):
    return oracle.z_block(seed, 0, k, 0, d).astype(np.float64) * np.float64(oracle.sigma(k))


# ---- a1 Sparsify_s --------------------------------------------------------------------------------
@pytest.mark.parametrize("d,s", [(1, 1), (17, 5), (1000, 16), (4096, 64), (100003, 256)])
def test_sparsify_is_full_sort_definition(d, s):
    rng = np.random.default_rng(d)
    g = rng.standard_normal(d).astype(np.float32)
    idx, val = oracle.sparsify(g, s)
    order = np.argsort(-np.abs(g).astype(np.float64), kind="stable")[:s]   # |g| descending, index ascending
    assert np.array_equal(idx, np.sort(order).astype(np.uint32))
    assert np.array_equal(val, g[idx])
    assert np.all(np.diff(idx.astype(np.int64)) > 0)


def test_sparsify_ties_zeros_and_signed_zero():
    g = np.array([0.5, -0.5, 0.5, 0.0, -0.0, 0.25, -0.5], dtype=np.float32)
    idx, val = oracle.sparsify(g, 3)
    assert idx.tolist() == [0, 1, 2]                 # four entries tie at 0.5: the three lowest indices win
    idx, _ = oracle.sparsify(g, 6)
    assert idx.tolist() == [0, 1, 2, 3, 5, 6]        # +0 and -0 tie: index 3 before index 4
    g = np.zeros(10, dtype=np.float32)
    idx, val = oracle.sparsify(g, 4)
    assert idx.tolist() == [0, 1, 2, 3] and not val.any()


# ---- a2 projection ---------------------------------------------------------------------------------
def test_projection_equals_dense_matvec():
    seed, k, d, s = 2, 64, 300, 9
    rng = np.random.default_rng(1)
    g = rng.standard_normal(d).astype(np.float32)
    idx, val = oracle.sparsify(g, s)
    A = dense_A(seed, k, d)
    gt = np.zeros(d)
    gt[idx] = val.astype(np.float64)
    p, q = oracle.project(seed, k, idx, val)
    np.testing.assert_allclose(p, A @ gt, rtol=0, atol=1e-14)
    np.testing.assert_allclose(q, A @ (gt * gt), rtol=0, atol=1e-14)


def test_projection_is_linear():
    seed, k = 9, 128
    idx = np.array([3, 77, 1000, 50000, 4_000_000_000], dtype=np.uint32)
    x = np.array([1.0, -2.0, 0.5, 4.0, -0.25], dtype=np.float32)
    y = np.array([0.5, 0.25, -8.0, 1.0, 2.0], dtype=np.float32)
    px, _ = oracle.project(seed, k, idx, x)
    py, _ = oracle.project(seed, k, idx, y)
    pxy, _ = oracle.project(seed, k, idx, (2 * x + 4 * y).astype(np.float32))   # exact in fp32
    np.testing.assert_allclose(pxy, 2 * px + 4 * py, rtol=0, atol=1e-13)
    # q is the projection of the squared entries on the same support
    _, qx = oracle.project(seed, k, idx, x)
    px2, _ = oracle.project(seed, k, idx, (x * x).astype(np.float32))
    np.testing.assert_allclose(qx, px2, rtol=0, atol=1e-14)


# ---- a3 Adam in k-space ----------------------------------------------------------------------------
def test_adam_constant_input_closed_form():
    # Algorithm 2 with M_0 = V_0 = 0 and constant p, q:  M_t = (1-b1^t) p,  Mhat_t = p.
    k, b1, b2 = 50, np.float32(0.9), np.float32(0.999)
    rng = np.random.default_rng(0)
    p = rng.standard_normal(k)
    q = rng.random(k)
    M = np.zeros(k, dtype=np.float32)
    V = np.zeros(k, dtype=np.float32)
    for t in range(1, 40):
        Mh, Vh = oracle.adam(M, V, p, q, b1, b2, t)
        np.testing.assert_allclose(M, (1 - np.float64(b1) ** t) * p, rtol=3e-6, atol=0)
        np.testing.assert_allclose(V, (1 - np.float64(b2) ** t) * q, rtol=2e-5, atol=0)
        np.testing.assert_allclose(Mh, p, rtol=3e-6, atol=0)
        np.testing.assert_allclose(Vh, q, rtol=2e-5, atol=0)


def test_adam_second_moment_uses_beta2():
    M = np.zeros(1, dtype=np.float32)
    V = np.zeros(1, dtype=np.float32)
    oracle.adam(M, V, np.array([1.0]), np.array([1.0]), np.float32(0.5), np.float32(0.75), 1)
    assert M[0] == np.float32(0.5) and V[0] == np.float32(0.25)
    Mh, Vh = oracle.adam(M, V, np.array([1.0]), np.array([1.0]), np.float32(0.5), np.float32(0.75), 2)
    assert M[0] == np.float32(0.75) and V[0] == np.float32(0.4375)       # stored state is NOT bias corrected
    assert Mh[0] == 1.0 and Vh[0] == 1.0


def test_kspace_ema_is_projection_of_dspace_ema():
    # Eq. (9): M_t = A sum_i h_i(beta1) G~_i.
    seed, k, d, s, b1, b2 = 4, 32, 200, 6, np.float32(0.9), np.float32(0.999)
    A = dense_A(seed, k, d)
    rng = np.random.default_rng(3)
    M = np.zeros(k, dtype=np.float32)
    V = np.zeros(k, dtype=np.float32)
    Md = np.zeros(d)
    Vd = np.zeros(d)
    for t in range(1, 8):
        g = rng.standard_normal(d).astype(np.float32)
        idx, val = oracle.sparsify(g, s)
        gt = np.zeros(d)
        gt[idx] = val
        Md = np.float64(b1) * Md + (1 - np.float64(b1)) * gt
        Vd = np.float64(b2) * Vd + (1 - np.float64(b2)) * gt * gt
        p, q = oracle.project(seed, k, idx, val)
        oracle.adam(M, V, p, q, b1, b2, t)
        np.testing.assert_allclose(M, A @ Md, rtol=0, atol=2e-6 * np.abs(A @ Md).max())
        np.testing.assert_allclose(V, A @ Vd, rtol=0, atol=2e-6 * np.abs(A @ Vd).max())


# ---- a5 combine + scatter --------------------------------------------------------------------------
def test_combine_scatter_definition_and_guards():
    W = np.arange(10, dtype=np.float32)
    lamM = np.array([7, 2, 5, 9], dtype=np.uint32)
    xM = np.array([1.0, -2.0, 3.0, 4.0])
    lamV = np.array([2, 7, 9, 4], dtype=np.uint32)
    xV = np.array([4.0, 0.25, -1.0, 1.0])
    ui, uv, mis, neg = oracle.combine_scatter(lamM, xM, lamV, xV, np.float32(2.0), np.float32(1e-8), np.float32(0.5),
                                              W)
    assert ui.tolist() == [2, 7] and mis == 1 and neg == 1        # 5 is not in Lam_V; x^V at 9 is negative
    np.testing.assert_allclose(uv, [0.5 * 2.0 * -2.0 / (2.0 + 1e-8), 0.5 * 2.0 * 1.0 / (0.5 + 1e-8)], rtol=1e-12)
    want = np.arange(10, dtype=np.float64)
    want[2] -= uv[0]
    want[7] -= uv[1]
    assert np.array_equal(W, want.astype(np.float32))


# ---- SGCA re-projection (Appendix C, Algorithm 4) ------------------------------------------------
def test_reprojection_moves_an_exactly_sparse_state_to_the_new_matrix():
    # constant sparse gradient: M_t = (1 - b1^t) A g and V_t = (1 - b2^t) A g^2 exactly (closed form of the EMA), so
    # OMP recovers (1 - b^t) g and the re-projected states must be (1 - b^t) A' g, A' materialised with numpy
    d, k, s, seed, new_seed = 3000, 256, 6, 3, 0xABCDEF0123
    rng = np.random.default_rng(5)
    supp = np.sort(rng.choice(d, size=s, replace=False)).astype(np.uint32)
    g = np.zeros(d, dtype=np.float32)
    g[supp] = (rng.uniform(1.0, 2.0, size=s) * rng.choice([-1.0, 1.0], size=s)).astype(np.float32)
    o = oracle.Oracle(d, k, s, seed, 1e-3, 0.9, 0.999, 1e-8)
    w = np.zeros(d, dtype=np.float32)
    steps = 3
    for _ in range(steps):
        o.step(g, w)
    o.reproject(new_seed)
    Anew = oracle.z_block(new_seed, 0, k, 0, d).astype(np.float64) * float(oracle.sigma(k))
    gd = g.astype(np.float64)
    b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))          # the betas are fp32 numbers
    np.testing.assert_allclose(o.get("M"), (1 - b1 ** steps) * (Anew @ gd), rtol=0, atol=2e-6 * np.abs(Anew @ gd).max())
    np.testing.assert_allclose(o.get("V"), (1 - b2 ** steps) * (Anew @ (gd * gd)), rtol=0,
                               atol=2e-6 * (1 - b2 ** steps) * np.abs(Anew @ (gd * gd)).max())
    # the method carries on under the new matrix: same support, same update direction
    w2 = np.zeros(d, dtype=np.float32)
    o.step(g, w2)
    assert sorted(o.get("lamM").tolist()) == supp.tolist() == sorted(o.get("lamV").tolist())
    np.testing.assert_allclose(w2[supp], -1e-3 * np.sign(g[supp]), rtol=0, atol=2e-8)
    o.close()


# ---- CESGC (Section 4.4): SGC on the projected gradient, update back through B^T --------------------------------
def test_cesgc_with_an_identity_projection_is_the_chunked_step_itself():
    # r = m and B = I: B G = G and B^T N = N, so the step must equal the chunk oracles run on G directly
    m, n, c, k, sc, seed = 8, 64, 4, 24, 2, 3
    rng = np.random.default_rng(1)
    G = (rng.standard_t(3.0, size=(m, n)) * 1e-2).astype(np.float32)
    W0 = rng.standard_normal((m, n)).astype(np.float32)
    a = [oracle.Oracle(m * n // c, k, sc, seed, 1e-3, 0.9, 0.999, 1e-8) for _ in range(c)]
    b = [oracle.Oracle(m * n // c, k, sc, seed, 1e-3, 0.9, 0.999, 1e-8) for _ in range(c)]
    Wa, Wb = W0.copy(), W0.copy()
    for _ in range(2):
        oracle.cesgc_step(a, np.eye(m, dtype=np.float32), G, Wa)
        flat = Wb.reshape(-1)
        dc = m * n // c
        for i, ch in enumerate(b):
            ch.step(np.ascontiguousarray(G.reshape(-1)[i * dc:(i + 1) * dc]), flat[i * dc:(i + 1) * dc])
        for x, y in zip(a, b):
            assert np.array_equal(x.get("lamM"), y.get("lamM")) and np.array_equal(x.get("M"), y.get("M"))
        np.testing.assert_allclose(Wa, Wb, rtol=0, atol=2e-7)
    for ch in a + b:
        ch.close()


def test_cesgc_update_lives_in_the_row_space_of_the_projection_and_matches_its_formula():
    # orthonormal B (first r left-singular vectors of G): the weight change is B^T U with U = -eta N at most s-sparse,
    # so it is orthogonal to every direction outside the span of B's rows, and B (W1 - W0) returns U itself
    m, n, r, c, k, sc, seed = 48, 40, 6, 3, 32, 3, 5
    rng = np.random.default_rng(2)
    G = (rng.standard_normal((m, 4)) @ rng.standard_normal((4, n)) + 0.05 * rng.standard_normal((m, n))).astype(np.float32)
    Um, _, _ = np.linalg.svd(G.astype(np.float64), full_matrices=True)
    B = np.ascontiguousarray(Um[:, :r].T).astype(np.float32)
    chunks = [oracle.Oracle(r * n // c, k, sc, seed, 1e-3, 0.9, 0.999, 1e-8) for _ in range(c)]
    W0 = rng.standard_normal((m, n)).astype(np.float32)
    W1 = W0.copy()
    P, U = oracle.cesgc_step(chunks, B, G, W1)
    np.testing.assert_allclose(P, B.astype(np.float64) @ G, rtol=1e-6, atol=1e-7)
    assert 0 < np.count_nonzero(U) <= c * sc
    dW = W1.astype(np.float64) - W0
    np.testing.assert_allclose(Um[:, r:].T @ dW, 0.0, atol=2e-6)                  # nothing outside the row space of B
    np.testing.assert_allclose(B.astype(np.float64) @ dW, U, rtol=0, atol=2e-6)   # B B^T = I on that space
    # the non-zeros of U are each chunk's update record
    dc = r * n // c
    for i, ch in enumerate(chunks):
        nz = np.nonzero(U.reshape(-1)[i * dc:(i + 1) * dc])[0]
        assert np.array_equal(nz, np.sort(ch.get("upd_idx")[:ch.get("n_upd")]))
    for ch in chunks:
        ch.close()
