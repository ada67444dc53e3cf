"""The allocation-free column sum (gcnsa_op_colsum_static) against the regular
entry point, through the C-ABI.  Some callers cannot allocate device memory
while they run (code inside another framework's memory pool, or next to a CUDA
graph capture, or under a fixed memory budget); for them the library carries
its own scratch array.  The array is shared by all calls and keeps the last
call's contents, so the check is made on two calls in a row with different
inputs.  Collected last on purpose: a failure here must not hide another."""
import numpy as np
import pytest
import torch

from paper_2012_04930_b200 import gcnsa

pytestmark = pytest.mark.gpu


def _ld(f):
    return (f + 3) // 4 * 4


def test_static_colsum_matches_regular_entry_point_twice_in_a_row():
    rng = np.random.default_rng(42)
    # the second call is smaller than the first: stale partials of call one stay in the array
    for n, f, accumulate in ((50_001, 128, 0), (777, 41, 1)):
        g = torch.zeros((n, _ld(f)), device="cuda")
        g[:, :f] = torch.from_numpy(rng.standard_normal((n, f)).astype(np.float32)).cuda()
        start = torch.from_numpy(rng.standard_normal(f).astype(np.float32)).cuda()
        want, got = start.clone(), start.clone()
        sc = torch.empty(gcnsa.op_colsum_scratch(n, f) // 4 + 1, device="cuda")
        gcnsa.op_colsum(g, f, want, accumulate, sc)
        before = torch.cuda.memory_allocated()
        gcnsa.op_colsum_static(g, f, got, accumulate)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        ref = g[:, :f].double().sum(0).cpu().numpy() + (start.double().cpu().numpy() if accumulate else 0.0)
        assert np.abs(got.cpu().numpy() - ref).max() <= 1e-4 * np.abs(ref).max()
        assert torch.equal(got, want), "same kernels in the same order: the results must be identical"


def test_static_colsum_rejects_sizes_beyond_its_scratch():
    f = gcnsa.COLSUM_STATIC_MAX_F + 1
    g = torch.zeros((4, _ld(f)), device="cuda")
    out = torch.zeros(f, device="cuda")
    with pytest.raises(gcnsa.GcnsaError) as ei:
        gcnsa.op_colsum_static(g, f, out, 0)
    assert ei.value.code == gcnsa.ERR_TOO_LARGE
    assert "GCNSA_COLSUM_STATIC_MAX_F" in str(ei.value)
    gcnsa.op_colsum_static(g, gcnsa.COLSUM_STATIC_MAX_F, out, 0)   # the largest allowed width works
    torch.cuda.synchronize()
    assert torch.all(out == 0)
