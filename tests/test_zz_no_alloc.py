"""sgc_sparsify_static: the allocation-free top-s selection must agree with the selection inside sgc_step and with
the CPU oracle's definition of Sparsify_s (full sort by magnitude, ties to the lower index).

The entry point exists for callers that cannot call cudaMalloc when they need a selection (a framework that
owns all device memory through its own pool, or a thread that must avoid cudaMalloc's device-wide
synchronisation).  Its scratch is a static device array shared by every call, so the test runs two calls in a
row on different gradients: stale contents from the first call must not leak into the second.  Index sets and
values are compared bit for bit, the bar the other selection tests use.  Collected last on purpose.
"""
import numpy as np
import pytest

import oracle
from paper_2502_00311_b200 import inputs

pytestmark = pytest.mark.gpu


def reference_selection(binding, g_dev, d, s):
    st = binding.Sgc(d, max(s, 16), s, 3, 1e-3, 0.9, 0.999, 1e-8)
    import torch
    w = torch.zeros(d, dtype=torch.float32, device="cuda")
    st.step(g_dev, w)
    idx, val = st.get("sel_idx"), st.get("sel_val")
    st.close()
    return idx, val


def test_static_selection_matches_step_selection_twice_in_a_row():
    import torch
    from paper_2502_00311_b200 import binding
    binding.lib()
    cases = [(1_000_003, 64, "student", 11), (1_000_003, 64, "student", 12), (300_000, 1024, "gauss", 13),
             (5000, 16, "gauss", 14)]
    out_idx = torch.empty(1024, dtype=torch.int32, device="cuda")
    out_val = torch.empty(1024, dtype=torch.float32, device="cuda")
    out_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for (d, s, kind, seed) in cases:
        supp, sign = inputs.planted_support(d, min(s, 64), seed)
        g = torch.from_numpy(inputs.gradient(d, kind, supp, sign, 100 + seed)).cuda()
        out_idx.fill_(-1)
        out_val.fill_(float("nan"))
        binding.sparsify_static(g, s, out_idx, out_val, out_status)
        torch.cuda.synchronize()
        got_idx = out_idx[:s].cpu().numpy().view(np.uint32)
        got_val = out_val[:s].cpu().numpy()
        want_idx, want_val = reference_selection(binding, g, d, s)
        assert np.array_equal(got_idx, want_idx), (d, s)
        assert np.array_equal(got_val.view(np.uint32), want_val.view(np.uint32)), (d, s)
        # the independent reference: the oracle sorts the whole vector
        orc_idx, orc_val = oracle.sparsify(g.cpu().numpy(), s)
        assert np.array_equal(got_idx, orc_idx), (d, s)
        assert np.array_equal(got_val.view(np.uint32), orc_val.view(np.uint32)), (d, s)
        assert int(out_status.item()) == 0
        del g
    # a degenerate vector (all magnitudes equal) takes the exact fallback and says so
    g = torch.full((100_000,), 0.25, dtype=torch.float32, device="cuda")
    binding.sparsify_static(g, 8, out_idx, out_val, out_status)
    torch.cuda.synchronize()
    assert out_idx[:8].cpu().tolist() == list(range(8))
    assert int(out_status.item()) & binding.STATUS_SELECT_FALLBACK
    # and the next ordinary call is clean again
    supp, sign = inputs.planted_support(200_000, 32, 1)
    g = torch.from_numpy(inputs.gradient(200_000, "student", supp, sign, 5)).cuda()
    binding.sparsify_static(g, 32, out_idx, out_val, out_status)
    torch.cuda.synchronize()
    want_idx, _ = reference_selection(binding, g, 200_000, 32)
    assert np.array_equal(out_idx[:32].cpu().numpy().view(np.uint32), want_idx)
    orc_idx, orc_val = oracle.sparsify(g.cpu().numpy(), 32)
    assert np.array_equal(out_idx[:32].cpu().numpy().view(np.uint32), orc_idx)
    assert np.array_equal(out_val[:32].cpu().numpy().view(np.uint32), orc_val.view(np.uint32))
    assert int(out_status.item()) == 0


def test_static_selection_rejects_oversized_requests():
    import torch
    from paper_2502_00311_b200 import binding
    g = torch.zeros(4096, dtype=torch.float32, device="cuda")
    out_idx = torch.empty(2048, dtype=torch.int32, device="cuda")
    out_val = torch.empty(2048, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.SgcError) as e:
        binding.sparsify_static(g, 1025, out_idx, out_val)        # s beyond the static capacity
    assert e.value.code == -2
    with pytest.raises(binding.SgcError) as e:
        binding.sparsify_static(g[:100], 101, out_idx, out_val)   # s > d
    assert e.value.code == -2
    with pytest.raises(binding.SgcError) as e:
        binding.sparsify_static(torch.zeros(1001, device="cuda")[1:], 4, out_idx, out_val)   # misaligned
    assert e.value.code == -4
