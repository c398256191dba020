"""The tensor-core screening pass (sgc_screen) against the plain definition computed from the oracle's A generator.

For every residual j the pass must report exactly the columns i with |<Z_i, R_j>| / ||Z_i|| >= tau_j.  The reference
takes Z from the oracle (bit-identical generator), R as the very binary16 values handed to the GPU, and evaluates the
definition in fp64.  The pass accumulates the column norm ||Z_i||^2 in short binary16 partial sums, which the library
documents as a relative score error of at most 1e-3: pairs whose exact score lies within 1e-3 (relative) of the
threshold may fall on either side; every other pair must match, and reported scores must agree to 1e-3.
"""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


def half_round(x):
    """float32 array -> (the nearest binary16 values as float32, their 16-bit patterns)."""
    h = np.ascontiguousarray(x, dtype=np.float32).astype(np.float16)
    return h.astype(np.float32), h.view(np.uint16)


@pytest.mark.parametrize("d,k,n,seed", [(5000, 256, 32, 0), (100_003, 256, 128, 1), (40_000, 128, 256, 7),
                                        (300, 64, 32, 3), (77_777, 1024, 64, 2)])
def test_screen_reports_exactly_the_columns_above_threshold(d, k, n, seed):
    import torch
    from paper_2502_00311_b200 import binding
    rng = np.random.default_rng(d + k + n)
    Z = oracle.z_block(seed, 0, k, 0, d).astype(np.float64)              # k x d
    R, bits = half_round(rng.standard_normal((n, k)).astype(np.float32) * rng.uniform(0.01, 3.0, size=(n, 1)).astype(np.float32))
    norms = np.sqrt((Z * Z).sum(axis=0))
    scores = np.abs(R.astype(np.float64) @ Z) / norms                       # n x d
    # thresholds: a few dozen expected reports per residual; one residual disabled, one reporting nothing
    tau = np.quantile(scores, 1.0 - min(0.5, 40.0 / d), axis=1).astype(np.float32)
    tau[n // 2] = np.inf
    tau[n - 1] = np.float32(scores[n - 1].max() * 1.5)
    rep_cap = 512
    rep_count, rep, err = binding.screen(seed, d, k, torch.from_numpy(bits.view(np.int16)).cuda(), torch.from_numpy(tau).cuda(),
                                         rep_cap)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    rep_count = rep_count.cpu().numpy()
    rep = rep.cpu().numpy()
    assert rep_count[n // 2] == 0 and rep_count[n - 1] == 0
    for j in range(n):
        c = int(rep_count[j])
        assert c <= rep_cap
        cols = rep[j, :c, 0].view(np.uint32).astype(np.int64)
        got_sc = rep[j, :c, 1].copy().view(np.float32)
        assert cols.size == np.unique(cols).size and (cols < d).all()
        sure = set(np.nonzero(scores[j] >= tau[j] * (1 + 1e-3))[0].tolist())
        maybe = set(np.nonzero(scores[j] >= tau[j] * (1 - 1e-3))[0].tolist())
        got = set(cols.tolist())
        assert sure <= got <= maybe, (j, sorted(sure - got)[:5], sorted(got - maybe)[:5])
        if c:
            np.testing.assert_allclose(got_sc, scores[j][cols], rtol=1e-3)


def test_screen_rejects_bad_arguments():
    import torch
    from paper_2502_00311_b200 import binding
    rt = torch.zeros((32, 96), dtype=torch.int16, device="cuda")
    tau = torch.zeros(32, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.SgcError) as e:
        binding.screen(0, 1000, 96, rt, tau, 16)            # k not a multiple of 64
    assert e.value.code == -2
    rt = torch.zeros((48, 128), dtype=torch.int16, device="cuda")
    with pytest.raises(binding.SgcError) as e:
        binding.screen(0, 1000, 128, rt, torch.zeros(48, device="cuda"), 16)   # n not a multiple of 32
    assert e.value.code == -2
