"""The failure path of the tensor-core screening pass, exercised without breaking anything.

Every wait on a hardware barrier inside the pass is bounded.  With the bound set to one nanosecond (sgc_set_wait_limit)
ordinary waits run out: the kernel is intact, its warps merely give up early, flag the error, let what is in flight
finish, return their tensor memory and exit.  The caller must see the flag, the step must still produce Algorithm 3's
result (finished in lock-step) with SGC_STATUS_TIMEOUT set, and the next ordinary step must be an ordinary one again.
"""
import numpy as np
import pytest

import oracle
from paper_2502_00311_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sgc():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_00311_b200 import binding
    binding.lib()
    return binding


def cuda(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def screen_case(sgc, seed, d, k, n):
    import torch
    rng = np.random.default_rng(5)
    R = rng.standard_normal((n, k)).astype(np.float16)
    tau = np.full(n, 4.0 * np.sqrt(k) * 1.0, dtype=np.float32)           # ~4 noise deviations of a unit-variance residual
    return torch.from_numpy(R.view(np.int16)).cuda(), torch.from_numpy(tau).cuda()


def test_screen_reports_an_expired_wait_and_the_next_pass_is_clean(sgc):
    import torch
    seed, d, k, n = 4, 100_003, 256, 64
    rt, tau = screen_case(sgc, seed, d, k, n)
    ref_count, _, err = sgc.screen(seed, d, k, rt, tau, 256)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    try:
        sgc.set_screen_wait_limit(1)
        _, _, err = sgc.screen(seed, d, k, rt, tau, 256)
        torch.cuda.synchronize()                                        # the kernel returned: nothing hangs, nothing faults
        assert int(err.item()) == 1
    finally:
        sgc.set_screen_wait_limit(0)
    count, _, err = sgc.screen(seed, d, k, rt, tau, 256)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert np.array_equal(count.cpu().numpy(), ref_count.cpu().numpy())


def compare_step(st, ref, g, w_gpu, w_ref):
    st.step(cuda(g), w_gpu)
    ref.step(g, w_ref)
    for name in ("sel_idx", "lamM", "lamV"):
        assert np.array_equal(st.get(name), ref.get(name)), name
    n = int(ref.get("n_upd"))
    assert st.get("n_upd") == n and np.array_equal(st.get("upd_idx")[:n], ref.get("upd_idx")[:n])
    a, b = st.get("upd_val")[:n], ref.get("upd_val")[:n]
    assert np.abs(a - b).max() <= 1e-4 * np.abs(b).max()


def test_step_survives_an_expired_wait_and_recovers(sgc):
    d, k, s, seed = 1 << 17, 512, 16, 2
    hp = inputs.ADAM
    st = sgc.Sgc(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    ref = oracle.Oracle(d, k, s, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    supp, sign = inputs.planted_support(d, s, 31)
    w0 = inputs.weights(d, 3)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    grads = [inputs.gradient(d, "student", supp, sign, 900 + i) for i in range(5)]
    for i in range(2):
        compare_step(st, ref, grads[i], w_gpu, w_ref)
    assert int(st.get("fallback")) == 0 and not st.status() & sgc.STATUS_TIMEOUT
    st.set_wait_limit(1)
    compare_step(st, ref, grads[2], w_gpu, w_ref)                       # the pass gives up; lock-step finishes the step
    assert st.status() & sgc.STATUS_TIMEOUT
    assert int(st.get("fallback")) == 1
    st.set_wait_limit(0)
    st.clear_status()
    compare_step(st, ref, grads[3], w_gpu, w_ref)
    compare_step(st, ref, grads[4], w_gpu, w_ref)
    assert int(st.get("fallback")) == 0 and int(st.get("rounds")) == 1   # one screening pass confirms every pick again
    assert not st.status() & sgc.STATUS_TIMEOUT
    st.close()
    ref.close()


def test_chunked_tensor_route_survives_an_expired_wait(sgc):
    # MESGC chunks with k_c > 32 and at least 1e9 multiply-adds per OMP iteration screen on the tensor cores (steps 0 and
    # 2 check that route against the oracles); an expired wait (step 1) sends every recovery of that step through the
    # fp32 kernels and is reported in the chunks' status words
    c, dc, k, sc, seed = 64, 65_536, 112, 4, 9
    hp = inputs.ADAM
    me = sgc.Mesgc(c * dc, c, k, sc, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
    refs = [oracle.Oracle(dc, k, sc, seed, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]) for _ in range(c)]
    supp, sign = inputs.planted_support(c * dc, c * sc, 77)
    w0 = inputs.weights(c * dc, 5)
    w_gpu, w_ref = cuda(w0.copy()), w0.copy()
    for step in range(3):
        g = inputs.gradient(c * dc, "student", supp, sign, 300 + step)
        me.chunks[0].set_wait_limit(1 if step == 1 else 0)               # the first state of the list owns the passes
        me.step(cuda(g), w_gpu)
        for i, ref in enumerate(refs):
            ref.step(g[i * dc:(i + 1) * dc], w_ref[i * dc:(i + 1) * dc])
            assert np.array_equal(me.chunks[i].get("lamM"), ref.get("lamM")), (step, i)
            assert np.array_equal(me.chunks[i].get("lamV"), ref.get("lamV")), (step, i)
        timed_out = any(ch.status() & sgc.STATUS_TIMEOUT for ch in me.chunks)
        assert timed_out == (step == 1)
        for ch in me.chunks:
            ch.clear_status()
        np.testing.assert_allclose(w_gpu.cpu().numpy(), w_ref, rtol=0, atol=1e-6)
    me.close()
    for ref in refs:
        ref.close()


def test_states_of_very_different_k_live_side_by_side(sgc):
    # the lock-step kernel's shared-memory opt-in belongs to the kernel, not to a state: creating a small-k state must
    # not take away what a large-k state needs
    hp = inputs.ADAM
    big = dict(d=1 << 16, k=16384, s=2, seed=5)
    small = dict(d=1 << 16, k=256, s=4, seed=6)
    sts, refs, ws, wr = [], [], [], []
    for cfg in (big, small):                                             # the small state is created second
        st = sgc.Sgc(cfg["d"], cfg["k"], cfg["s"], cfg["seed"], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"])
        st.set_mode(sgc.MODE_LOCKSTEP)
        sts.append(st)
        refs.append(oracle.Oracle(cfg["d"], cfg["k"], cfg["s"], cfg["seed"], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"]))
        w0 = inputs.weights(cfg["d"], 11)
        ws.append(cuda(w0.copy()))
        wr.append(w0.copy())
    for step in range(2):
        for cfg, st, ref, w_gpu, w_ref in zip((big, small), sts, refs, ws, wr):
            supp, sign = inputs.planted_support(cfg["d"], cfg["s"], 40 + cfg["k"])
            g = inputs.gradient(cfg["d"], "student", supp, sign, 700 + step)
            compare_step(st, ref, g, w_gpu, w_ref)
    for st, ref in zip(sts, refs):
        st.close()
        ref.close()
