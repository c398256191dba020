"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

A full oracle recovery costs k*d*s generated entries per residual (hours at d = 16.7M), so at these sizes the
comparison is split:
  * a1-a3 (top-s support and values, p, q, M, V, t): element by element against the oracle, every step;
  * a4, the picks: OMP is defined pick by pick -- pick j is the argmax over ALL d columns of |<A_i, r_j>| / ||A_i||, where
    r_j is the least-squares residual on the first j picks.  For sampled iterations j the test forms r_j from the GPU's
    first j picks with the oracle's own least squares and asks the oracle's Select (oracle.select: every one of the d
    columns, fp64, the routine that test_oracle_omp pins to oracle.omp) for the argmax: it must be the GPU's pick j.
    The first iterations are always among the sampled ones, so by induction the leading picks are exactly those of
    oracle.omp, and the later sampled ones are those of oracle.omp given the same history.  Where even one pass over
    all columns is out of reach on the host (k >= 4096 at d = 45M: minutes per pass) the Select runs over a prefix of the
    columns: nothing in the prefix may beat the pick, and a pick inside the prefix must be its argmax.
  * a4, for all picks: on the GPU's support, OMP (numpy, fp64) selects the same columns in the same order, and the
    coefficients are the oracle's least-squares solution on that support;
  * a5: the weight update against Eq. (8) evaluated with numpy on the recovered coefficients;
  * lock-step and speculative recovery give the same supports at the headline size (supplementary: GPU against GPU).
"""
import numpy as np
import pytest

import oracle
from paper_2502_00311_b200 import inputs

pytestmark = pytest.mark.gpu

TOL_STATE = 1e-5
TOL_UPDATE = 1e-4

D44 = 4096 * 4096
DG = 4096 * 11008


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)


def cuda(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def columns(seed, k, cols):
    """A[:, cols] (without sigma) as float64 [k, len(cols)] from the oracle's generator."""
    out = np.empty((k, len(cols)), dtype=np.float64)
    for i, c in enumerate(cols):
        out[:, i] = oracle.z_block(seed, 0, k, int(c), 1)[:, 0]
    return out


def check_support_properties(seed, k, s, y, lam, x, done):
    """On the GPU's own support: OMP replays it in the same order, and x is the oracle's least-squares fit."""
    assert done == s
    lam = lam[:done].astype(np.int64)
    assert np.unique(lam).size == done
    sigma = float(oracle.sigma(k))
    Z = columns(seed, k, lam)
    A = sigma * Z
    norms = np.sqrt((Z * Z).sum(axis=0))
    r = y.copy()
    for j in range(done):
        sc = np.abs(Z.T @ r) / norms
        sc[:j] = -1.0
        assert int(np.argmax(sc)) == j, "pick %d is not the best of the support" % j
        xj = np.linalg.lstsq(A[:, :j + 1], y, rcond=None)[0]
        r = y - A[:, :j + 1] @ xj
    assert rel(x[:done], oracle.least_squares(seed, k, lam.astype(np.uint32), y)) < TOL_UPDATE
    return A


def check_picks(seed, d, k, items, d_cols=None):
    """items: [(y, lam, A, js)], one entry per recovery.  Pick j of the GPU must be the oracle's Select over all d columns
    (or over the prefix [0, d_cols)) for the residual that the GPU's first j picks leave.  A = sigma * Z on the GPU's
    support (from the oracle's generator).  All residuals of all items share one pass of the oracle over the columns."""
    R, skip, tags = [], [], []
    for (y, lam, A, js) in items:
        for j in sorted(set(int(j) % len(lam) for j in js)):
            if j == 0:
                r = y.copy()
            else:
                r = y - A[:, :j] @ oracle.least_squares(seed, k, lam[:j].astype(np.uint32), y)
            R.append(r)
            skip.append(lam[:j].tolist())
            tags.append((lam, A, j))
    if not R:
        return
    sel = oracle.select(seed, d_cols or d, k, np.array(R), skip)
    for n, (lam, A, j) in enumerate(tags):
        if d_cols is None or lam[j] < d_cols:
            assert sel["idx"][n] == lam[j], "pick %d: GPU %d, oracle %d (scores %.9g / %.9g)" % (
                j, lam[j], sel["idx"][n], sel["best"][n], sel["second"][n])
        else:
            own = abs(A[:, j] @ R[n]) / np.sqrt(A[:, j] @ A[:, j])
            assert sel["best"][n] <= own, "pick %d: column %d of the prefix scores %.9g > %.9g" % (
                j, sel["idx"][n], sel["best"][n], own)


def check_update(st, hp, d, rec, w_before, w_after):
    """a5: Eq. (8) on the common support where x^V > 0, nothing else touched."""
    lamM, xM = rec["M"]
    lamV, xV = rec["V"]
    upd = {}
    for i, col in enumerate(lamM.tolist()):
        hit = np.nonzero(lamV == col)[0]
        if hit.size and xV[hit[0]] > 0:
            upd[col] = hp["lr"] * xM[i] / (np.sqrt(xV[hit[0]]) + hp["eps"])
    n = int(st.get("n_upd"))
    assert n == len(upd) and sorted(upd) == st.get("upd_idx")[:n].tolist()
    want = np.array([upd[c] for c in sorted(upd)])
    assert rel(st.get("upd_val")[:n], want) < TOL_UPDATE
    touched = np.zeros(d, dtype=bool)
    touched[sorted(upd)] = True
    assert np.array_equal(w_after[~touched], w_before[~touched])
    dw = w_after[touched].astype(np.float64) - w_before[touched]
    assert np.abs(dw + want).max() <= TOL_UPDATE * np.abs(want).max() + 1.2e-7 * np.abs(w_before[touched]).max()


def run_config(sgc, d, k, s, seed, cfg_id, steps, planted, picks=None, mode=None, matrix_id=0, lockstep_twin=False):
    """picks: {step: (js for M^, js for V^[, d_cols])} -- iterations whose pick is checked against the oracle's Select
    over all d columns, or over the first d_cols when given."""
    import torch
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    if mode is not None:
        st.set_mode(mode)
    twin = None
    if lockstep_twin:
        twin = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
        twin.set_mode(sgc.MODE_LOCKSTEP)
        w_twin = cuda(inputs.weights(d, 99))
    ref = oracle.Oracle(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    supp, sign = inputs.planted_support(d, s, inputs.support_seed(cfg_id, matrix_id))
    w_gpu = cuda(inputs.weights(d, 99))
    rounds = []
    seen = set()                                                # every index that was ever kept by Sparsify_s
    picks = picks or {}
    for step in range(1, steps + 1):
        g = inputs.gradient(d, "student", supp, sign, inputs.step_seed(cfg_id, matrix_id, step))
        w_before = w_gpu.cpu().numpy()
        gd = cuda(g)
        st.step(gd, w_gpu)
        ref.step_compress(g)                                    # a1-a3 of the oracle
        assert st.get("t") == step == ref.get("t")
        assert np.array_equal(st.get("sel_idx"), ref.get("sel_idx"))
        assert np.array_equal(st.get("sel_val"), ref.get("sel_val"))
        for name in ("p", "q", "M", "V"):
            assert rel(st.get(name), ref.get(name)) < TOL_STATE, name
        rounds.append((int(st.get("rounds")), int(st.get("fallback")), int(st.get("list_rounds"))))
        seen |= set(ref.get("sel_idx").tolist())
        targets = dict(M=ref.get("Mhat"), V=ref.get("Vhat"))
        rec = {}
        items = []
        for mi, name in enumerate(("M", "V")):
            lam, x, done = st.get("lam" + name), st.get("x" + name), int(st.get("done" + name))
            if step in (1, steps) or step in picks:
                A = check_support_properties(seed, k, s, targets[name], lam, x, done)
                if step in picks:
                    items.append((targets[name], lam[:done].astype(np.int64), A, picks[step][mi]))
            if planted:
                # exact-recovery regime: M^ and V^ are combinations of the columns kept so far, and OMP finds only those
                assert set(lam.tolist()) <= seen, "recovered support leaves the kept indices"
                if step == 1:
                    assert sorted(lam.tolist()) == ref.get("sel_idx").tolist()
            rec[name] = (lam[:done], x[:done])
        if step in picks:
            check_picks(seed, d, k, items, picks[step][2] if len(picks[step]) > 2 else None)
        check_update(st, hp, d, rec, w_before, w_gpu.cpu().numpy())
        if twin is not None:
            twin.step(gd, w_twin)
            assert int(twin.get("fallback")) == 1
            for name in ("lamM", "lamV", "upd_idx"):
                assert np.array_equal(twin.get(name), st.get(name)), (name, step)
            assert torch.equal(w_twin, w_gpu)
        del gd
    status = int(st.get("status"))
    st.close()
    ref.close()
    if twin is not None:
        twin.close()
    return rounds, status


@pytest.fixture(scope="module")
def sgc():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_00311_b200 import binding
    binding.lib()
    return binding


def test_config2_full_size(sgc):
    # 4096 x 4096, k = 2048, s = 64, seed 1: the benchmark's workload; exact-recovery regime.  Step 1: the first eight
    # picks and every eighth after them, both recoveries; last step: five iterations spread over the run.
    dense = list(range(8)) + list(range(15, 64, 8))
    rounds, status = run_config(sgc, D44, 2048, 64, 1, 2, steps=3, planted=True, lockstep_twin=True,
                                picks={1: (dense, dense), 3: ([0, 1, 7, 32, 63], [0, 1, 7, 32, 63])})
    assert all(fb == 0 for _, fb, _ in rounds), rounds
    assert rounds[-1][0] == 1, rounds            # warm candidate list: one screening pass per step
    assert not status & (sgc.STATUS_CANDIDATE_OVERFLOW | sgc.STATUS_SELECT_FALLBACK | sgc.STATUS_TIMEOUT)


def test_config3_4096x4096_two_level_screening_full_size(sgc):
    # one 4096 x 4096 projection of a Llama-2-7B layer: k = 2048, s = 128 (recovery is inexact here: noise columns get
    # picked); enough steps for the wide lists and the list passes to come into play
    js = [0, 1, 2, 7, 64, 127]
    rounds, status = run_config(sgc, D44, 2048, 128, 1, 3, steps=5, planted=False, picks={1: (js, js), 5: (js, js)})
    assert all(fb == 0 for _, fb, _ in rounds), rounds
    assert sum(lr for _, _, lr in rounds) > 0, rounds
    assert not status & (sgc.STATUS_CANDIDATE_OVERFLOW | sgc.STATUS_TIMEOUT)


def test_config3_down_projection_full_size(sgc):
    # the 4096 x 11008 "down" projection of the layer (matrix 6 of config 3), d = 45 088 768
    js = [0, 1, 64, 127]
    run_config(sgc, DG, 2048, 128, 1, 3, steps=2, planted=False, matrix_id=6, picks={1: (js, js)})


def test_config3_layer_as_groups_full_size(sgc):
    # Config 3 as a configuration: the seven projections of one layer share the seed, so same-shape matrices see the same
    # A (Section 4.4 lets equal-sized vectors share one matrix): q/k/v/o step as one sgc_step_group, gate/up as another,
    # down alone.  Every state must equal its solo run record for record, and one state per group is checked against the
    # oracle's Select at the last step.
    import torch
    hp = inputs.ADAM
    cfg = inputs.CONFIGS["c3_llama7b_layer"]
    k, s, seed = cfg["k"], cfg["s"], cfg["seed"]
    dims = [r * c for r, c in cfg["shapes"]]
    assert dims == [D44] * 4 + [DG] * 3

    def make():
        return [sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for d in dims]

    grp, solo = make(), make()
    supports = [inputs.planted_support(d, s, inputs.support_seed(3, i)) for i, d in enumerate(dims)]
    w_grp = [cuda(inputs.weights(d, 200 + i)) for i, d in enumerate(dims)]
    w_solo = [w.clone() for w in w_grp]
    refs = {i: oracle.Oracle(dims[i], k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for i in (0, 4, 6)}
    steps = 3
    for step in range(1, steps + 1):
        grads = []
        for i, d in enumerate(dims):
            g = inputs.gradient(d, "student", supports[i][0], supports[i][1], inputs.step_seed(3, i, step))
            if i in refs:
                refs[i].step_compress(g)
            grads.append(cuda(g))
        sgc.step_group(grp[0:4], grads[0:4], w_grp[0:4])
        sgc.step_group(grp[4:6], grads[4:6], w_grp[4:6])
        grp[6].step(grads[6], w_grp[6])
        for i in range(7):
            solo[i].step(grads[i], w_solo[i])
        for i in range(7):
            assert grp[i].get("t") == step
            for name in ("sel_idx", "lamM", "lamV", "upd_idx"):
                assert np.array_equal(grp[i].get(name), solo[i].get(name)), (name, i, step)
            assert rel(grp[i].get("xM"), solo[i].get("xM")) < 1e-9 and rel(grp[i].get("xV"), solo[i].get("xV")) < 1e-9
            assert torch.equal(w_grp[i], w_solo[i]), (i, step)
            assert int(grp[i].get("fallback")) == 0
        for i, ref in refs.items():                                  # a1-a3 of one matrix per group against the oracle
            assert np.array_equal(grp[i].get("sel_idx"), ref.get("sel_idx"))
            for name in ("p", "q", "M", "V"):
                assert rel(grp[i].get(name), ref.get(name)) < TOL_STATE, (name, i)
        del grads
    for i, ref in refs.items():                                      # a4 of one matrix per group, last step
        items = []
        for name, js in (("M", [0, s - 1]), ("V", [s // 2])):
            y = ref.get(name + "hat")
            lam, x, done = grp[i].get("lam" + name), grp[i].get("x" + name), int(grp[i].get("done" + name))
            A = check_support_properties(seed, k, s, y, lam, x, done)
            items.append((y, lam[:done].astype(np.int64), A, js))
        check_picks(seed, dims[i], k, items)
    for st in grp + solo:
        st.close()
    for ref in refs.values():
        ref.close()


def test_config4_matrix_full_size(sgc):
    # the 32-layer stack uses k = 1024, s = 64 for every matrix
    dense = [0, 1, 2, 3] + list(range(7, 64, 8))
    run_config(sgc, D44, 1024, 64, 1, 4, steps=2, planted=False, picks={1: (dense, dense), 2: ([0, 63], [0, 63])})


# The (k, s) sweep of config 5 on the 4096 x 11008 matrix: every pair.  One pass of the oracle over all d columns costs
# k * d generated entries: seconds up to k = 1024, 45 s at k = 4096, three minutes at k = 16384 (16 host cores); from
# k = 4096 on the Select therefore runs over the first 2^22 columns, except for one full pass at (4096, 256), the pair
# that takes the two-passes-of-128-picks route.
P22, P21 = 1 << 22, 1 << 21
C5_CASES = {
    (256, 16): dict(planted=False, picks={1: (range(16), range(16)), 2: ([0, 15], [0, 15])}),
    (1024, 16): dict(planted=False, picks={1: ([0, 1, 7, 15], [0, 1, 7, 15])}),
    (1024, 64): dict(planted=False, picks={1: ([0, 1, 31, 63], [0, 1, 31, 63])}),
    (4096, 16): dict(planted=True, picks={1: (range(16), [0, 15], P22)}),
    (4096, 64): dict(planted=True, picks={1: ([0, 1, 7, 31, 63], [0, 63], P22)}),
    (4096, 256): dict(planted=False, picks={1: ([0], []), 2: ([1, 127, 128, 255], [0, 255], P22)}),
    (16384, 16): dict(planted=True, picks={1: ([0, 15], [0], P21)}),
    (16384, 64): dict(planted=True, picks={1: ([0, 63], [0], P21)}),
    (16384, 256): dict(planted=True, picks={1: ([0, 128, 255], [0], P21)}),
}


@pytest.mark.parametrize("k,s", sorted(C5_CASES))
def test_config5_sweep_full_size(sgc, k, s):
    case = C5_CASES[(k, s)]
    assert (k, s) in inputs.C5_PAIRS
    run_config(sgc, DG, k, s, 1, 5, steps=2, planted=case["planted"], picks=case["picks"])
