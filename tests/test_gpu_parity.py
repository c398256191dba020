"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on seeded inputs.

Bar: index sets (top-s support, OMP supports, updated positions) bit-exact; p, q, M, V within 1e-5 and the
recovered update within 1e-4, both as max-abs error relative to the largest reference magnitude.
"""
import numpy as np
import pytest

import oracle
from golden_util import read_z_golden
from paper_2502_00311_b200 import inputs

pytestmark = pytest.mark.gpu

TOL_STATE = 1e-5
TOL_UPDATE = 1e-4


@pytest.fixture(scope="module")
def sgc():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_00311_b200 import binding
    binding.lib()
    return binding


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)


def cuda(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# ---- the A generator ----------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1, 0x123456789ABCDEF])
def test_z_generator_bit_exact(sgc, seed):
    blocks, xor, total = read_z_golden(seed)
    for (r0, c0), want in blocks.items():
        got = sgc.z_block(seed, r0, 32, c0, 32).cpu().numpy()
        assert np.array_equal(got.astype(np.float16).astype(np.float32), got)         # every Z is a binary16 number
        assert np.array_equal(got.astype(np.float16).view(np.uint16), want)
    for (r0, nr, c0, nc) in [(0, 300, 0, 257), (65000, 536, 4294967000, 296), (7, 1, 123456789, 1), (1, 4, 5, 3)]:
        got = sgc.z_block(seed, r0, nr, c0, nc).cpu().numpy()
        assert np.array_equal(got.view(np.uint32), oracle.z_block(seed, r0, nr, c0, nc).view(np.uint32))


# ---- a1 top-s -------------------------------------------------------------------------------------------
def run_select(sgc, g, s, k=None):
    d = g.size
    k = k or max(s, 8)
    st = sgc.Sgc(d, k, s, 3, 1e-3, 0.9, 0.999, 1e-8)
    w = cuda(np.zeros(d, dtype=np.float32))
    st.step(cuda(g), w)
    idx, val, status = st.get("sel_idx"), st.get("sel_val"), st.get("status")
    st.close()
    return idx, val, status


@pytest.mark.parametrize("d,s", [(1, 1), (5, 5), (1023, 7), (4096, 16), (32768, 64), (32769, 64), (100003, 33),
                                 (1 << 20, 256), (3_000_001, 1024)])
def test_select_matches_oracle(sgc, d, s):
    rng = np.random.default_rng(d + s)
    g = (rng.standard_t(3.0, size=d) * 1e-3).astype(np.float32)
    idx, val, status = run_select(sgc, g, s, k=max(s, 16))
    widx, wval = oracle.sparsify(g, s)
    assert np.array_equal(idx, widx) and np.array_equal(val, wval)
    assert not status & sgc.STATUS_SELECT_FALLBACK


def test_select_ties_and_degenerate_distributions(sgc):
    # many equal magnitudes: the sampled threshold cannot separate them -> exact fallback, lowest indices win
    d, s = 200_000, 20
    g = np.full(d, 0.5, dtype=np.float32)
    g[::3] *= -1
    g[[17, 99_999, 150_000]] = [2.0, -3.0, 2.0]
    idx, val, status = run_select(sgc, g, s)
    widx, wval = oracle.sparsify(g, s)
    assert np.array_equal(idx, widx) and np.array_equal(val, wval)
    assert status & sgc.STATUS_SELECT_FALLBACK
    # all zeros, signed zeros
    g = np.zeros(70_000, dtype=np.float32)
    g[1::2] = -0.0
    idx, val, _ = run_select(sgc, g, 9)
    assert idx.tolist() == list(range(9))
    # Gaussian (light tails) and a constant-plus-spikes vector
    rng = np.random.default_rng(0)
    g = rng.standard_normal(2_000_000).astype(np.float32)
    idx, val, status = run_select(sgc, g, 128, k=128)
    widx, _ = oracle.sparsify(g, 128)
    assert np.array_equal(idx, widx) and not status & sgc.STATUS_SELECT_FALLBACK


def test_select_flags_non_finite_input(sgc):
    g = np.random.default_rng(1).standard_normal(50_000).astype(np.float32)
    g[1234] = np.nan
    g[4321] = np.inf
    _, _, status = run_select(sgc, g, 8)
    assert status & sgc.STATUS_NONFINITE_INPUT


# ---- whole step, config-1 shape and relatives -------------------------------------------------------------
def run_both(sgc, d, k, s, seed, kind, steps, cfg_id=1, alpha=None, redraw_support=False, compare_every=1, mode=None,
             stats=None, list_rounds=None, recovery=None, n_planted=None):
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=alpha)
    if mode is not None:
        st.set_mode(mode)
    ref = oracle.Oracle(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=alpha or 1.0)
    if recovery is not None:                     # the opt-in variant, on both sides
        st.set_recovery(*recovery)
        ref.set_recovery(*recovery)
    supp, sign = inputs.planted_support(d, n_planted or s, inputs.support_seed(cfg_id, 0))
    w0 = inputs.weights(d, 99)
    w_gpu = cuda(w0.copy())
    w_ref = w0.copy()
    worst = dict(p=0.0, q=0.0, M=0.0, V=0.0, upd=0.0, x=0.0)
    for step in range(1, steps + 1):
        if redraw_support:
            supp, sign = inputs.planted_support(d, n_planted or s, inputs.support_seed(cfg_id, 0) + 7919 * step)
        g = inputs.gradient(d, kind, supp, sign, inputs.step_seed(cfg_id, 0, step))
        w_before = w_ref.copy()
        st.step(cuda(g), w_gpu)
        ref.step(g, w_ref)
        assert st.get("t") == step == ref.get("t")
        if stats is not None:
            stats.append((int(st.get("rounds")), int(st.get("fallback")), int(st.get("n_cand"))))
        if list_rounds is not None:
            list_rounds.append(int(st.get("list_rounds")))
        assert np.array_equal(st.get("sel_idx"), ref.get("sel_idx"))
        assert np.array_equal(st.get("sel_val"), ref.get("sel_val"))
        for name in ("p", "q", "M", "V"):
            worst[name] = max(worst[name], rel(st.get(name), ref.get(name)))
        assert st.get("doneM") == ref.get("doneM") and st.get("doneV") == ref.get("doneV")
        assert np.array_equal(st.get("lamM"), ref.get("lamM")), "OMP(M^) selection order differs at step %d" % step
        assert np.array_equal(st.get("lamV"), ref.get("lamV")), "OMP(V^) selection order differs at step %d" % step
        worst["x"] = max(worst["x"], rel(st.get("xM"), ref.get("xM")), rel(st.get("xV"), ref.get("xV")))
        n = int(ref.get("n_upd"))
        assert st.get("n_upd") == n and st.get("mismatch") == ref.get("mismatch") and st.get("negv") == ref.get("negv")
        assert np.array_equal(st.get("upd_idx")[:n], ref.get("upd_idx")[:n])
        if n:
            worst["upd"] = max(worst["upd"], rel(st.get("upd_val")[:n], ref.get("upd_val")[:n]))
        wg = w_gpu.cpu().numpy()
        touched = np.zeros(d, dtype=bool)
        touched[ref.get("upd_idx")[:n]] = True
        assert np.array_equal(wg[~touched], w_before[~touched])            # nothing else is written
        if n:
            dw_g = wg[touched].astype(np.float64) - w_before[touched]
            dw_r = w_ref[touched].astype(np.float64) - w_before[touched]
            assert np.abs(dw_g - dw_r).max() <= TOL_UPDATE * np.abs(dw_r).max() + 1.2e-7 * np.abs(w_before[touched]).max()
    for name in ("p", "q", "M", "V"):
        assert worst[name] < TOL_STATE, (name, worst[name])
    assert worst["x"] < TOL_UPDATE and worst["upd"] < TOL_UPDATE, worst
    status = st.get("status")
    st.close()
    ref.close()
    return worst, status


def test_config1_ten_steps(sgc):
    # 64x64 matrix, k=256, s=16, N(0, 0.1^2) noise + 16 planted U(1,2) entries, seed 0, 10 steps
    worst, status = run_both(sgc, 4096, 256, 16, 0, "gauss", 10, cfg_id=1)
    assert not status & (sgc.STATUS_CANDIDATE_OVERFLOW | sgc.STATUS_SELECT_FALLBACK | sgc.STATUS_NONFINITE_INPUT)


@pytest.mark.parametrize("d,k,s", [(1000, 64, 1), (4099, 96, 12), (70_001, 333, 17), (1 << 17, 512, 64)])
def test_awkward_shapes(sgc, d, k, s):
    # d not a multiple of 4 or of the tile, k not a multiple of 32, s = 1 and s = k/8
    run_both(sgc, d, k, s, 5, "student", 3, cfg_id=2)


# ---- speculative recovery (candidate-list OMP confirmed by tensor-core screening passes) ---------------------
@pytest.mark.parametrize("d,k,s,kind", [(4096, 256, 16, "gauss"), (1 << 17, 512, 64, "student"), (70_001, 320, 17, "student"),
                                        (200_000, 128, 5, "student"), (50_000, 2048, 130, "student")])
def test_speculative_recovery_matches_the_oracle(sgc, d, k, s, kind):
    # same bar as the lock-step path: supports in selection order bit-exact, values within tolerance; the planted
    # support is fixed, so after the first step the candidate list holds it and one screening pass per step suffices
    stats = []
    worst, status = run_both(sgc, d, k, s, 5, kind, 4, cfg_id=2, mode=2, stats=stats)
    assert not status & sgc.STATUS_CANDIDATE_OVERFLOW
    assert all(fb == 0 for _, fb, _ in stats), stats
    assert all(r >= 1 for r, _, _ in stats), stats


def test_speculative_recovery_with_redrawn_supports_and_alpha(sgc):
    # every step is a cold start for the candidate list, and the recovery is inexact (picks among noise columns)
    stats = []
    run_both(sgc, 150_000, 256, 8, 11, "student", 5, cfg_id=2, alpha=2.0, redraw_support=True, mode=2, stats=stats)
    assert all(fb == 0 for _, fb, _ in stats), stats


@pytest.mark.parametrize("d,k,s,max_rounds", [(150_000, 256, 32, 1), (150_000, 256, 32, 2), (150_000, 256, 32, 3),
                                              (100_000, 768, 96, 2)])
def test_lockstep_finishes_what_a_bounded_number_of_rounds_leaves_open(sgc, d, k, s, max_rounds):
    # Two steady steps, then a new support every step, so that every later step needs several rounds of speculation and
    # its first refuted pick gets a prescribed column.  With the rounds bounded, the lock-step path takes over from a
    # state that the speculation left behind -- stored columns, F, coefficients and the prescribed pick included -- and
    # must still end with Algorithm 3's supports and update.  (s = 96: the bounded steps screen in half-width passes.)
    seed = 3
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    st.set_mode(sgc.MODE_SPECULATIVE)
    st.set_max_rounds(max_rounds)
    ref = oracle.Oracle(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    w0 = inputs.weights(d, 99)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    open_steps = 0
    for step in range(1, 6):
        supp, sign = inputs.planted_support(d, s, 1000 * seed + (0 if step <= 2 else step))
        g = inputs.gradient(d, "student", supp, sign, 50 * seed + step)
        st.step(cuda(g), w_gpu)
        ref.step(g, w_ref)
        assert np.array_equal(st.get("lamM"), ref.get("lamM")), step
        assert np.array_equal(st.get("lamV"), ref.get("lamV")), step
        assert int(st.get("rounds")) <= max_rounds
        trace = st.get("round_trace").reshape(-1, 3)
        open_steps += int(trace[int(st.get("rounds")) - 1, 0] < s or trace[int(st.get("rounds")) - 1, 1] < s)
        np.testing.assert_allclose(w_gpu.cpu().numpy(), w_ref, rtol=0, atol=1e-6)
    assert open_steps >= 1, open_steps              # the bound really cut a step short
    with pytest.raises(sgc.SgcError):
        st.set_max_rounds(-1)
    st.close()
    ref.close()


def test_steps_after_a_refuted_pick_screen_in_passes_of_half_the_width(sgc):
    # s = 96: both streams fill a pass of 192 residual rows.  After a step in which a full pass refuted a pick, the
    # next step screens 48 residuals per stream and round in the 96-row pass (half the cost per round); the supports
    # must not depend on which width a step used.
    d, k, s, seed = 100_000, 768, 96, 5
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    st.set_mode(sgc.MODE_SPECULATIVE)
    ref = oracle.Oracle(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    w0 = inputs.weights(d, 99)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    widths = []
    for step in range(1, 7):
        supp, sign = inputs.planted_support(d, s, 77 + (0 if step <= 2 else step))      # new supports from step 3 on
        g = inputs.gradient(d, "student", supp, sign, 900 + step)
        st.step(cuda(g), w_gpu)
        ref.step(g, w_ref)
        assert np.array_equal(st.get("lamM"), ref.get("lamM")), step
        assert np.array_equal(st.get("lamV"), ref.get("lamV")), step
        np.testing.assert_allclose(w_gpu.cpu().numpy(), w_ref, rtol=0, atol=1e-6)
        assert int(st.get("fallback")) == 0
        widths.append((int(st.get("rounds")), int(st.get("pass_rows"))))
    assert widths[0][1] >= 192, widths                                    # a fresh state starts with the pass over all 192 rows
    assert any(r >= 2 and rows == 96 * r for r, rows in widths[1:]), widths
    st.close()
    ref.close()


@pytest.mark.parametrize("d,k,s,steps", [(400_000, 256, 48, 7), (500_000, 512, 100, 4)])
def test_two_level_screening_matches_the_oracle(sgc, d, k, s, steps):
    # inexact regime (supports redrawn every step, k small): steps need several passes over all columns, which switches
    # on the wide lists and the list passes between full passes; the picks must not depend on any of that
    stats, lists = [], []
    run_both(sgc, d, k, s, 21, "student", steps, cfg_id=2, redraw_support=True, mode=2, stats=stats, list_rounds=lists)
    assert all(fb == 0 for _, fb, _ in stats), stats
    assert max(r for r, _, _ in stats) >= 3, stats               # the regime this test is about
    assert sum(lists) > 0, (stats, lists)                        # list passes ran and were resolved


# ---- opt-in recovery variant: shared support, early stop (remark after Eq. (8)) ----------------------------------
@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("d,k,s,kind,redraw", [(70_001, 320, 17, "student", True), (1 << 17, 512, 64, "student", False),
                                               (4096, 256, 16, "gauss", False)])
def test_shared_support_variant_matches_its_oracle(sgc, mode, d, k, s, kind, redraw):
    # OMP(M^) alone selects; x^V is the least-squares fit of V^ on its support.  Redrawn supports make the two printed
    # recoveries disagree, so this is not the printed algorithm in disguise.
    if mode == 2 and k % 64:
        pytest.skip("speculative recovery needs k to be a multiple of 64")
    run_both(sgc, d, k, s, 5, kind, 4, cfg_id=2, mode=mode, redraw_support=redraw, recovery=(True, 0.0))


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("shared", [False, True])
def test_early_stop_on_the_residual_matches_its_oracle(sgc, mode, shared):
    # gradients with 10 non-zeros while s = 16: M^ and V^ are exactly 10-sparse in the A-basis, the residual falls to
    # rounding noise after 10 picks, and a tolerance of 1e-6 ends both recoveries there on both sides (the later picks
    # of an uncut run would be decided by that noise)
    d, k, s = 50_000, 512, 16
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, 3, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    st.set_mode(mode)
    st.set_recovery(shared, 1e-6)
    run_both(sgc, d, k, s, 3, "zero", 3, cfg_id=2, mode=mode, recovery=(shared, 1e-6), n_planted=10)
    # the cut is visible in the records
    supp, sign = inputs.planted_support(d, 10, inputs.support_seed(2, 0))
    w = cuda(inputs.weights(d, 99))
    st.step(cuda(inputs.gradient(d, "zero", supp, sign, inputs.step_seed(2, 0, 1))), w)
    assert st.get("doneM") == 10 == st.get("doneV")
    assert sorted(st.get("lamM")[:10].tolist()) == sorted(supp.tolist()) and np.all(st.get("lamM")[10:] == 0xFFFFFFFF)
    assert np.all(st.get("xM")[10:] == 0.0) and st.get("n_upd") == 10
    st.close()


def test_set_recovery_rejects_bad_arguments(sgc):
    st = sgc.Sgc(4096, 64, 4, 1, 1e-3, 0.9, 0.999, 1e-8)
    for args in [(2, 0.0), (0, -1.0), (1, float("nan")), (0, float("inf"))]:
        assert sgc.lib().sgc_set_recovery(st._h, args[0], args[1]) != 0
    assert sgc.lib().sgc_set_recovery(st._h, 1, 0.5) == 0
    st.close()


def test_speculative_and_lockstep_agree_bit_for_bit_on_supports(sgc):
    d, k, s = 300_000, 2048, 24          # k large enough for exact recovery: the picks are the planted support
    hp = inputs.ADAM
    supp, sign = inputs.planted_support(d, s, 77)
    a = sgc.Sgc(d, k, s, 6, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    b = sgc.Sgc(d, k, s, 6, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    a.set_mode(sgc.MODE_LOCKSTEP)
    b.set_mode(sgc.MODE_SPECULATIVE)
    wa, wb = cuda(inputs.weights(d, 3)), cuda(inputs.weights(d, 3))
    for step in range(1, 6):
        g = cuda(inputs.gradient(d, "student", supp, sign, 900 + step))
        a.step(g, wa)
        b.step(g, wb)
        assert a.get("fallback") == 1 and b.get("fallback") == 0
        for name in ("lamM", "lamV", "upd_idx"):
            assert np.array_equal(a.get(name), b.get(name)), (name, step)
        assert rel(b.get("xM"), a.get("xM")) < 1e-9 and rel(b.get("xV"), a.get("xV")) < 1e-9
        assert rel(wb.cpu().numpy(), wa.cpu().numpy()) < 1e-7
    assert b.get("rounds") == 1          # warm candidate list: one confirming pass per step
    a.close()
    b.close()


def test_alpha_and_redrawn_supports(sgc):
    # alpha = 2 as in the paper's experiments; the planted support is redrawn every step so that M^ and V^
    # stop being s-sparse and the recovery is inexact (supports of the two recoveries may differ)
    run_both(sgc, 20_000, 256, 8, 11, "student", 6, cfg_id=2, alpha=2.0, redraw_support=True)


def test_constant_sparse_gradient_closed_form(sgc):
    # exactly s non-zeros held constant: N = alpha*sign(g) on the support, W_t = W_0 - t*lr*alpha*sign(g)
    d, k, s, lr = 50_000, 512, 10, 1e-3
    rng = np.random.default_rng(8)
    supp = np.sort(rng.choice(d, size=s, replace=False))
    g = np.zeros(d, dtype=np.float32)
    g[supp] = (rng.uniform(1.0, 2.0, size=s) * rng.choice([-1.0, 1.0], size=s)).astype(np.float32)
    w0 = rng.standard_normal(d).astype(np.float32)
    st = sgc.Sgc(d, k, s, 2, lr, 0.9, 0.999, 1e-8)
    w = cuda(w0.copy())
    gd = cuda(g)
    for t in range(1, 5):
        st.step(gd, w)
        assert sorted(st.get("lamM").tolist()) == supp.tolist() == sorted(st.get("lamV").tolist())
    want = w0.astype(np.float64)
    want[supp] -= 4 * lr * np.sign(g[supp])
    np.testing.assert_allclose(w.cpu().numpy(), want, rtol=0, atol=3e-6)
    st.close()


def test_dependent_column_stops_like_the_oracle(sgc):
    # With s <= k (which sgc_create enforces) the stop needs columns that are dependent although there are at most k of
    # them.  Seeds whose first two columns at k = 2 are exactly parallel (66855), nearly so (112200: sin^2 = 6.2e-11,
    # under the 1e-10 pivot bound) and merely ill-conditioned (143364: sin^2 = 1.5e-9) reach it from both sides with
    # d = 2, s = 2, where the second pick is forced.
    d, k, s = 2, 2, 2
    g = np.array([0.75, -1.25], dtype=np.float32)
    for seed, want_done in ((66855, 1), (112200, 1), (143364, 2)):
        st = sgc.Sgc(d, k, s, seed, 1e-3, 0.9, 0.999, 1e-8)
        ref = oracle.Oracle(d, k, s, seed, 1e-3, 0.9, 0.999, 1e-8)
        w = cuda(np.zeros(4, dtype=np.float32))
        wr = np.zeros(d, dtype=np.float32)
        st.step(cuda(np.concatenate([g, np.zeros(2, dtype=np.float32)])), w)
        ref.step(g, wr)
        for m in "MV":
            assert st.get("done" + m) == ref.get("done" + m) == want_done, (seed, m)
            assert np.array_equal(st.get("lam" + m), ref.get("lam" + m)), (seed, m)
        assert bool(st.get("status") & sgc.STATUS_DEPENDENT_COLUMN) == (want_done < s)
        assert st.status() == int(st.get("status"))
        np.testing.assert_allclose(w.cpu().numpy()[:d], wr, rtol=1e-4, atol=1e-12)
        st.close()
        ref.close()
    # the generic small case: k = 2, s = 2 among 64 columns completes both picks
    d = 64
    g = np.random.default_rng(3).standard_normal(d).astype(np.float32)
    st = sgc.Sgc(d, k, s, 3, 1e-3, 0.9, 0.999, 1e-8)
    ref = oracle.Oracle(d, k, s, 3, 1e-3, 0.9, 0.999, 1e-8)
    w = cuda(np.zeros(d, dtype=np.float32))
    wr = np.zeros(d, dtype=np.float32)
    st.step(cuda(g), w)
    ref.step(g, wr)
    assert st.get("doneM") == ref.get("doneM") == 2 and np.array_equal(st.get("lamM"), ref.get("lamM"))
    st.close()


def test_lockstep_three_near_tied_columns_in_one_block(sgc):
    # The lock-step screen runs in fp32 and every block forwards only its best two columns per residual to the fp64
    # decision.  Three columns of one block's range whose scores agree to ~1e-7 (far inside the 2e-3 rescoring window, far
    # above fp64 noise) must still be ordered as the oracle orders them: the block reports that it kept a third one back and
    # its range is screened again.  M^ = a_c1 x1 + a_c2 x2 + a_c3 x3 with x solving "equal normalised correlations".
    d, k, s = 4096, 256, 3
    hp = inputs.ADAM
    rng = np.random.default_rng(17)
    for trial in range(12):
        seed = 100 + trial
        cols = np.sort(rng.choice(2048, size=3, replace=False))              # one tile of the screen: one block
        A = float(oracle.sigma(k)) * np.stack([oracle.z_block(seed, 0, k, int(c), 1)[:, 0] for c in cols], axis=1).astype(np.float64)
        G = (A.T @ A) / np.sqrt((A * A).sum(axis=0))[:, None]
        x = np.linalg.solve(G, np.ones(3))
        g = np.zeros(d, dtype=np.float32)
        g[cols] = x.astype(np.float32)
        st = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
        ref = oracle.Oracle(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
        w, wr = cuda(np.zeros(d, dtype=np.float32)), np.zeros(d, dtype=np.float32)
        st.step(cuda(g), w)
        ref.step(g, wr)
        assert int(st.get("fallback")) == 1                                   # d < 65536: lock-step
        top = ref.get("top1M")[0], ref.get("top2M")[0]
        assert abs(top[0] - top[1]) < 1e-5 * top[0]                           # the premise: a near-tie at the first pick
        assert np.array_equal(st.get("lamM"), ref.get("lamM")), (trial, st.get("lamM"), ref.get("lamM"))
        assert np.array_equal(st.get("lamV"), ref.get("lamV")), trial
        assert not int(st.get("status")) & sgc.STATUS_CANDIDATE_OVERFLOW
        st.close()
        ref.close()


def test_state_set_get_roundtrip_and_resume(sgc):
    d, k, s = 30_000, 128, 6
    hp = inputs.ADAM
    supp, sign = inputs.planted_support(d, s, 5)
    gs = [inputs.gradient(d, "student", supp, sign, 100 + i) for i in range(4)]
    a = sgc.Sgc(d, k, s, 9, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    wa = cuda(inputs.weights(d, 1))
    for g in gs[:2]:
        a.step(cuda(g), wa)
    b = sgc.Sgc(d, k, s, 9, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    b.set_state(a.get("M"), a.get("V"), int(a.get("t")))
    wb = wa.clone()
    for g in gs[2:]:
        a.step(cuda(g), wa)
        b.step(cuda(g), wb)
    assert np.array_equal(a.get("M"), b.get("M")) and np.array_equal(wa.cpu().numpy(), wb.cpu().numpy())
    a.close()
    b.close()


def test_group_equals_independent_steps(sgc):
    d, k, s, n = 40_000, 256, 8, 3
    hp = inputs.ADAM
    solo = [sgc.Sgc(d, k, s, 4, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(n)]
    grp = [sgc.Sgc(d, k, s, 4, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(n)]
    ws = [cuda(inputs.weights(d, 10 + i)) for i in range(n)]
    wg = [w.clone() for w in ws]
    for step in range(2):
        gr = []
        for i in range(n):
            supp, sign = inputs.planted_support(d, s, 50 + i)
            gr.append(cuda(inputs.gradient(d, "student", supp, sign, 1000 * i + step)))
        for i in range(n):
            solo[i].step(gr[i], ws[i])
        sgc.step_group(grp, gr, wg)
        for i in range(n):
            assert np.array_equal(solo[i].get("lamM"), grp[i].get("lamM"))
            assert np.array_equal(ws[i].cpu().numpy(), wg[i].cpu().numpy())
    with pytest.raises(sgc.SgcError):
        other = sgc.Sgc(d, k, s, 5, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
        sgc.step_group([grp[0], other], gr[:2], wg[:2])
    for st in solo + grp:
        st.close()


@pytest.mark.parametrize("d,k,s,n", [(300_000, 512, 64, 3), (200_000, 256, 8, 5), (150_000, 2048, 128, 2)])
def test_group_shares_screening_passes_and_equals_independent_steps(sgc, d, k, s, n):
    # speculative recovery: the residuals of several same-A states are screened by one tensor-core pass per batch
    # (two states at s = 64, up to eight at s <= 16, one at s = 128); supports and weights must equal independent steps
    hp = inputs.ADAM
    solo = [sgc.Sgc(d, k, s, 4, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(n)]
    grp = [sgc.Sgc(d, k, s, 4, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(n)]
    for st in solo + grp:
        st.set_mode(sgc.MODE_SPECULATIVE)
    ws = [cuda(inputs.weights(d, 10 + i)) for i in range(n)]
    wg = [w.clone() for w in ws]
    supports = [inputs.planted_support(d, s, 50 + i) for i in range(n)]
    for step in range(3):
        gr = [cuda(inputs.gradient(d, "student", supports[i][0], supports[i][1], 1000 * i + step)) for i in range(n)]
        for i in range(n):
            solo[i].step(gr[i], ws[i])
        sgc.step_group(grp, gr, wg)
        for i in range(n):
            assert grp[i].get("fallback") == 0
            for name in ("sel_idx", "lamM", "lamV", "upd_idx"):
                assert np.array_equal(solo[i].get(name), grp[i].get(name)), (name, i, step)
            assert rel(grp[i].get("xM"), solo[i].get("xM")) < 1e-9
            assert np.array_equal(ws[i].cpu().numpy(), wg[i].cpu().numpy())
            assert grp[i].get("t") == step + 1
    for st in solo + grp:
        st.close()


def test_mesgc_chunks_share_one_matrix_and_match_independent_oracles(sgc):
    # Section 4.4: c chunks, s_c entries each, one A of size k x d/c; every chunk is an SGC problem of its own
    c, dc, k, sc = 6, 70_000, 256, 4
    d = c * dc
    hp = inputs.ADAM
    m = sgc.Mesgc(d, c, k, sc, 8, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    for st in m.chunks:
        st.set_mode(sgc.MODE_SPECULATIVE)
    refs = [oracle.Oracle(dc, k, sc, 8, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(c)]
    supp, sign = inputs.planted_support(d, c * sc, 17)
    w0 = inputs.weights(d, 2)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    for step in range(1, 4):
        g = inputs.gradient(d, "student", supp, sign, 40 + step)
        m.step(cuda(g), w_gpu)
        for i in range(c):
            refs[i].step(g[i * dc:(i + 1) * dc], w_ref[i * dc:(i + 1) * dc])
            for name in ("sel_idx", "lamM", "lamV"):
                assert np.array_equal(m.chunks[i].get(name), refs[i].get(name)), (name, i, step)
            assert rel(m.chunks[i].get("M"), refs[i].get("M")) < TOL_STATE
        wg = w_gpu.cpu().numpy()
        changed = wg != w0
        assert np.array_equal(changed, w_ref != w0)
        assert np.abs(wg[changed].astype(np.float64) - w_ref[changed]).max() <= TOL_UPDATE * np.abs(w_ref[changed] - w0[changed]).max() + 2e-9
    with pytest.raises(sgc.SgcError):
        odd = sgc.Mesgc(6 * 1002, 6, 64, 2, 0, 1e-3, 0.9, 0.999, 1e-8)       # chunks of 1002 floats are not 16-byte aligned
        import torch
        odd.step(torch.zeros(6 * 1002, device="cuda"), torch.zeros(6 * 1002, device="cuda"))
    m.close()
    for r in refs:
        r.close()


@pytest.mark.parametrize("c,dc,k,sc,kind", [(6, 70_000, 56, 4, "student"), (40, 4096, 8, 1, "student"), (9, 65_536, 112, 16, "student"),
                                             (300, 2048, 14, 2, "gauss"), (5, 10_000, 128, 16, "student"), (3, 5_000, 33, 7, "student"),
                                             (64, 2048, 217, 31, "student"), (1100, 1024, 200, 2, "student"), (4, 30_000, 256, 32, "student")])
def test_mesgc_small_chunks_batched_path_matches_independent_oracles(sgc, c, dc, k, sc, kind):
    # the regime the paper runs MESGC in (s_c of 1 to 16, k_c = 7 or 8 times s_c): all chunks go through one set of
    # launches; every chunk must still equal an SGC problem of its own, record by record
    d = c * dc
    hp = inputs.ADAM
    m = sgc.Mesgc(d, c, k, sc, 8, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=2.0)
    refs = [oracle.Oracle(dc, k, sc, 8, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=2.0) for _ in range(c)]
    w0 = inputs.weights(d, 2)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    check = sorted(set(range(0, c, max(1, c // 12))) | {c - 1})          # chunks compared record by record
    for step in range(1, 4):
        supp, sign = inputs.planted_support(d, c * sc, 17 + step)          # redrawn: M^ and V^ have more than s_c columns
        g = inputs.gradient(d, kind, supp, sign, 40 + step)
        w_before = w_ref.copy()
        m.step(cuda(g), w_gpu)
        # the batched path ran: 2 + 2 s_c launches, or, with phase A on the tensor cores (k_c > 32), 4 + passes per pick
        passes = -(-(-(-2 * c // 32) * 32) // 256)
        kp = next(v for v in (8, 16, 32, 64, 128, 256) if k <= v)
        tensor = kp >= 64 and 2 * c <= 2048 and dc * kp * 2 * c >= 1e9
        assert m.chunks[0].last_launches() == (2 + sc * (4 + passes) if tensor else 2 + 2 * sc)
        for i in range(c):
            refs[i].step(g[i * dc:(i + 1) * dc], w_ref[i * dc:(i + 1) * dc])
        for i in check:
            st, ref = m.chunks[i], refs[i]
            assert st.get("t") == step
            for name in ("sel_idx", "sel_val", "lamM", "lamV", "upd_idx"):
                assert np.array_equal(st.get(name), ref.get(name)), (name, i, step)
            for name in ("p", "q", "M", "V"):
                assert rel(st.get(name), ref.get(name)) < TOL_STATE, (name, i, step)
            for name in ("doneM", "doneV", "n_upd", "mismatch", "negv"):
                assert st.get(name) == ref.get(name), (name, i, step)
            assert rel(st.get("xM"), ref.get("xM")) < TOL_UPDATE and rel(st.get("xV"), ref.get("xV")) < TOL_UPDATE
            assert rel(st.get("rnormM"), ref.get("rnormM")) < 1e-6
        wg = w_gpu.cpu().numpy()
        changed = w_ref != w_before
        assert np.array_equal(wg[~changed], w_before[~changed])           # nothing else is written
        if changed.any():
            dw_g = wg[changed].astype(np.float64) - w_before[changed]
            dw_r = w_ref[changed].astype(np.float64) - w_before[changed]
            assert np.abs(dw_g - dw_r).max() <= TOL_UPDATE * np.abs(dw_r).max() + 1.2e-7 * np.abs(w_before[changed]).max()
    m.close()
    for r in refs:
        r.close()


def test_mesgc_batched_path_edge_cases(sgc):
    import torch
    hp = inputs.ADAM
    # tiny chunks: as many kept entries as a chunk can give (s_c = d/c), k_c barely above s_c
    c, dc, k, sc = 5, 8, 12, 8
    m = sgc.Mesgc(c * dc, c, k, sc, 4, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    refs = [oracle.Oracle(dc, k, sc, 4, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(c)]
    rng = np.random.default_rng(0)
    w0 = rng.standard_normal(c * dc).astype(np.float32)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    for step in range(2):
        g = rng.standard_normal(c * dc).astype(np.float32)
        m.step(cuda(g), w_gpu)
        assert m.chunks[0].last_launches() == 2 + 2 * sc
        for i in range(c):
            refs[i].step(g[i * dc:(i + 1) * dc], w_ref[i * dc:(i + 1) * dc])
            assert np.array_equal(m.chunks[i].get("sel_idx"), np.arange(dc, dtype=np.uint32))
            for name in ("lamM", "lamV", "upd_idx"):
                assert np.array_equal(m.chunks[i].get(name), refs[i].get(name)), (name, i)
            assert m.chunks[i].get("doneM") == refs[i].get("doneM") and m.chunks[i].get("doneV") == refs[i].get("doneV")
        assert rel(w_gpu.cpu().numpy(), w_ref) < 1e-5
    m.close()
    for r in refs:
        r.close()
    # a NaN is flagged in the chunk that holds it and nowhere else; equal magnitudes go to the lower index
    c, dc = 4, 4096
    m = sgc.Mesgc(c * dc, c, 16, 2, 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    g = np.full(c * dc, 0.25, dtype=np.float32)
    g[1::2] *= -1
    g[2 * dc + 77] = np.nan
    m.step(cuda(g), cuda(np.zeros(c * dc, dtype=np.float32)))
    flags = [int(st.get("status")) & sgc.STATUS_NONFINITE_INPUT for st in m.chunks]
    assert flags[2] and not (flags[0] or flags[1] or flags[3])
    for i in (0, 1, 3):
        assert np.array_equal(m.chunks[i].get("sel_idx"), np.array([0, 1], dtype=np.uint32))
    m.close()


def test_mesgc_batched_path_on_a_side_stream(sgc):
    # the first call builds the chunk table and the norm table; a stream that does not synchronise with the default
    # stream must still find them complete
    import torch
    hp = inputs.ADAM
    c, dc, k, sc = 8, 16_384, 56, 4
    d = c * dc
    supp, sign = inputs.planted_support(d, c * sc, 5)
    g = cuda(inputs.gradient(d, "student", supp, sign, 6))
    outs = []
    for side in (False, True):
        m = sgc.Mesgc(d, c, k, sc, 2, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
        w = cuda(inputs.weights(d, 1))
        if side:
            stream = torch.cuda.Stream()
            stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(stream):
                m.step(g, w, stream=stream)
            stream.synchronize()
        else:
            m.step(g, w)
        outs.append(([st.get("lamM").copy() for st in m.chunks], [st.get("lamV").copy() for st in m.chunks], w.cpu().numpy()))
        m.close()
    for a, b in zip(outs[0][0] + outs[0][1], outs[1][0] + outs[1][1]):
        assert np.array_equal(a, b)
    assert np.array_equal(outs[0][2], outs[1][2])


def test_small_states_are_created_without_speculative_buffers(sgc):
    import torch
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    states = [sgc.Sgc(4096, 64, 8, 1, 1e-3, 0.9, 0.999, 1e-8) for _ in range(64)]      # k a multiple of 64: could speculate
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < 64 * (4 << 20), (free0 - free1) / 64                     # a few MB each at most, not 50
    states[0].set_mode(sgc.MODE_SPECULATIVE)                                        # this one gets them now
    free2, _ = torch.cuda.mem_get_info()
    assert free1 - free2 > (30 << 20)
    g = cuda((np.random.default_rng(0).standard_normal(4096) * 0.1).astype(np.float32))
    wa, wb = cuda(np.zeros(4096, dtype=np.float32)), cuda(np.zeros(4096, dtype=np.float32))
    states[0].step(g, wa)
    states[1].step(g, wb)
    assert states[0].get("fallback") == 0 and states[1].get("fallback") == 1
    assert np.array_equal(states[0].get("lamM"), states[1].get("lamM")) and np.array_equal(wa.cpu().numpy(), wb.cpu().numpy())
    for st in states:
        st.close()


def test_mesgc_batched_path_rejects_a_repeated_state(sgc):
    import torch
    m = sgc.Mesgc(4 * 4096, 4, 16, 2, 1, 1e-3, 0.9, 0.999, 1e-8)
    hs = (sgc.C.c_void_p * 4)(m.chunks[0]._h, m.chunks[1]._h, m.chunks[1]._h, m.chunks[3]._h)
    g, w = torch.zeros(4 * 4096, device="cuda"), torch.zeros(4 * 4096, device="cuda")
    assert sgc.lib().sgc_step_chunked(hs, 4, g.data_ptr(), w.data_ptr(), None) != 0
    assert m.chunks[0].get("t") == 0
    m.close()


@pytest.mark.parametrize("m,n,r,c,k,sc", [(512, 256, 8, 4, 28, 4), (1000, 384, 32, 16, 56, 8), (4096, 512, 32, 8, 217, 31),
                                          (300, 128, 8, 1, 320, 8),          # a core too large for the batched chunk path
                                          (560, 100, 8, 2, 28, 4)])         # ragged columns; the last CTA of the projection's cluster has no rows
def test_cesgc_step_matches_its_oracle(sgc, m, n, r, c, k, sc):
    # Section 4.4: SGC (chunked) on B G, update back through B^T; B = first r left-singular vectors of the first gradient
    hp = inputs.ADAM
    rng = np.random.default_rng(m + r)
    low = rng.standard_normal((m, 6)) @ rng.standard_normal((6, n))
    ce = sgc.Cesgc(m, n, r, c, k, sc, 9, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=2.0)
    refs = [oracle.Oracle(r * n // c, k, sc, 9, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], alpha=2.0) for _ in range(c)]
    W_ref = (rng.standard_normal((m, n)) * 0.02).astype(np.float32)
    w_gpu = cuda(W_ref.copy())
    B = None
    for step in range(1, 4):
        G = (low * (1.0 + 0.1 * step) + 0.3 * rng.standard_t(3.0, size=(m, n))).astype(np.float32)
        if B is None:
            U, _, _ = np.linalg.svd(G.astype(np.float64), full_matrices=False)
            B = np.ascontiguousarray(U[:, :r].T).astype(np.float32)
            ce.set_projection(cuda(B))
        W_before = W_ref.copy()
        P, Uref = oracle.cesgc_step(refs, B, G, W_ref)
        ce.step(cuda(G), w_gpu)
        import torch
        torch.cuda.synchronize()
        got_P = ce.scratch[: r * n].cpu().numpy().reshape(r, n)
        # the projection rounds a two-float sum once: the fp64 product of the oracle gives the same fp32 numbers but for
        # a few elements in ten thousand, which differ by one ulp (more for entries that are tiny against their terms,
        # never by more than the ulp of the largest entries)
        off = got_P != P
        assert off.sum() <= max(1, 1e-3 * off.size) and np.abs(got_P[off] - P[off]).max(initial=0.0) <= np.spacing(np.abs(P).max())
        for i in range(c):
            st = ce.core.chunks[i]
            for name in ("sel_idx", "lamM", "lamV", "upd_idx"):
                assert np.array_equal(st.get(name), refs[i].get(name)), (name, i, step)
        got_U = ce.scratch[r * n:].cpu().numpy().reshape(r, n)
        assert np.array_equal(got_U != 0, Uref != 0)
        assert rel(got_U, Uref) < TOL_UPDATE
        wg = w_gpu.cpu().numpy()
        dw_g = wg.astype(np.float64) - W_before
        dw_r = W_ref.astype(np.float64) - W_before
        cols = np.nonzero(np.any(Uref != 0, axis=0))[0]
        other = np.setdiff1d(np.arange(n), cols)
        assert np.array_equal(wg[:, other], W_before[:, other])          # columns without an update are not written
        assert np.abs(dw_g - dw_r).max() <= TOL_UPDATE * np.abs(dw_r).max() + 1.2e-7 * np.abs(W_before).max()
    ce.close()
    for rf in refs:
        rf.close()


def test_cesgc_step_rejects_bad_shapes(sgc):
    import torch
    ce = sgc.Cesgc(64, 32, 4, 2, 16, 2, 1, 1e-3, 0.9, 0.999, 1e-8)
    g, w = torch.zeros(64, 32, device="cuda"), torch.zeros(64, 32, device="cuda")
    B = torch.zeros(4, 64, device="cuda")
    call = lambda r, m, n: sgc.lib().sgc_cesgc_step(ce.core._hs, 2, B.data_ptr(), r, m, n, g.data_ptr(), w.data_ptr(),
                                                      ce.scratch.data_ptr(), None)
    assert call(0, 64, 32) != 0 and call(65, 64, 32) != 0 and call(4, 64, 31) != 0 and call(4, 0, 32) != 0
    assert ce.core.chunks[0].get("t") == 0
    ce.close()


@pytest.mark.parametrize("mode", [1, 2])
def test_sgca_reprojection_matches_the_oracle(sgc, mode):
    # Algorithm 4: every T = 2 steps the matrix is replaced and M, V are re-aligned; the steps after that run under the
    # new matrix on both sides (the oracle recovers the stored moments afresh, the GPU rescales the step's recoveries)
    d, k, s = 120_000, 512, 12
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, 21, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    st.set_mode(mode)
    ref = oracle.Oracle(d, k, s, 21, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    supp, sign = inputs.planted_support(d, s, 31)
    w_gpu, w_ref = cuda(inputs.weights(d, 4)), inputs.weights(d, 4)
    for step in range(1, 7):
        g = inputs.gradient(d, "student", supp, sign, 500 + step)
        st.step(cuda(g), w_gpu)
        ref.step(g, w_ref)
        assert np.array_equal(st.get("lamM"), ref.get("lamM")) and np.array_equal(st.get("lamV"), ref.get("lamV")), step
        assert rel(st.get("p"), ref.get("p")) < TOL_STATE
        if step % 2 == 0:
            new_seed = 1000 + step
            st.reproject(new_seed)
            ref.reproject(new_seed)
        assert rel(st.get("M"), ref.get("M")) < TOL_STATE and rel(st.get("V"), ref.get("V")) < TOL_STATE, step
        assert rel(w_gpu.cpu().numpy(), w_ref) < 1e-6
    st.close()
    ref.close()
    fresh = sgc.Sgc(1000, 64, 2, 0, 1e-3, 0.9, 0.999, 1e-8)
    with pytest.raises(sgc.SgcError) as e:
        fresh.reproject(5)
    assert e.value.code == -8
    fresh.close()


def test_step_rejects_misaligned_pointers(sgc):
    import torch
    st = sgc.Sgc(1000, 16, 2, 0, 1e-3, 0.9, 0.999, 1e-8)
    buf = torch.zeros(1001, dtype=torch.float32, device="cuda")
    good = torch.zeros(1000, dtype=torch.float32, device="cuda")
    with pytest.raises(sgc.SgcError) as e:
        st.step(buf[1:], good)
    assert e.value.code == -4
    with pytest.raises(sgc.SgcError):
        st.get("p")          # no step has run yet
    st.close()
