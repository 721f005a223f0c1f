"""gc_compress_noalloc against gc_compress.

Some callers cannot allocate device memory at all (a hook running inside a framework whose
allocator owns the device, a latency-bound loop), so they cannot create a plan.  The
entry point they use keeps its scratch in a fixed array inside the library; this test calls
it through the C ABI and requires bit-identical indices, values and residual to what the
plan-based gc_compress gives on the same inputs -- twice in a row, because the second call
meets the first call's leftovers in the shared array.  The file name keeps it last in
collection order, so a failure here cannot hide the other tests from a stop-at-first run.
"""
import numpy as np
import pytest
import torch

from paper_2104_01981_b200 import api, build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    api.lib()


def reference_compress(n, k_density, g, r):
    """The existing entry point on private copies; returns (k, idx, val, residual)."""
    plan = api.Plan([n], k_density, device=0)
    k = plan.total_cap
    idx, val, cnt = plan.alloc_outputs()
    ws = plan.alloc_workspace()
    r2 = r.clone()
    plan.compress(g, r2, idx, val, None, ws)
    torch.cuda.synchronize()
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK
    return k, idx[:k].clone(), val[:k].clone(), r2


def test_two_calls_in_a_row_match_the_plan_based_entry_point():
    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(99)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    # first call: a large tensor (many tiles, ragged tail); second: a smaller one with ties, so
    # stale tile words and histogram bins from the first call would show
    cases = [(3_000_001, 0.01, False), (70_003, 0.2, True)]
    r_keep = None
    for n, density, quantise in cases:
        g = torch.randn(n + 3, device="cuda", generator=gen)[:n + 3]
        if quantise:
            g = torch.round(g * 4) / 4
        g = g[:n].contiguous() if (g.data_ptr() % 16 == 0) else g.clone()[:n]
        r = torch.randn(n, device="cuda", generator=gen) * 0.3
        k, want_idx, want_val, want_r = reference_compress(n, density, g, r)
        out_idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        out_val = torch.full((k,), float("nan"), device="cuda")
        rc = api.compress_noalloc(g, r, n, k, out_idx, out_val, status)
        assert rc == api.GC_OK
        torch.cuda.synchronize()
        assert status.item() == api.GC_OK
        assert torch.equal(out_idx, want_idx)
        assert torch.equal(out_val.view(torch.int32), want_val.view(torch.int32))
        assert torch.equal(r.view(torch.int32), want_r.view(torch.int32))
        r_keep = r
    # third call reusing the residual the second call left (error feedback carried over)
    n, density = cases[-1][0], cases[-1][1]
    g = torch.randn(n, device="cuda", generator=gen)
    k, want_idx, want_val, want_r = reference_compress(n, density, g, r_keep)
    out_idx = torch.empty(k, dtype=torch.int32, device="cuda")
    out_val = torch.empty(k, device="cuda")
    assert api.compress_noalloc(g, r_keep, n, k, out_idx, out_val, None) == api.GC_OK
    torch.cuda.synchronize()
    assert torch.equal(out_idx, want_idx) and torch.equal(r_keep.view(torch.int32), want_r.view(torch.int32))
    assert torch.equal(out_val.view(torch.int32), want_val.view(torch.int32))


def test_sizes_beyond_the_fixed_scratch_are_refused():
    torch.cuda.set_device(0)
    g = torch.zeros(16, device="cuda")
    i = torch.zeros(16, dtype=torch.int32, device="cuda")
    assert api.compress_noalloc(g, g.clone(), api.GC_NOALLOC_MAX_N + 1, 1, i, g.clone()) == api.GC_E_TOO_LARGE
    assert api.compress_noalloc(g, g.clone(), 8, 9, i, g.clone()) == api.GC_E_INVALID
    assert api.compress_noalloc(g, g.clone(), 0, 0, i, g.clone()) == api.GC_OK
    torch.cuda.synchronize()
