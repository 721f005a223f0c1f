"""gc_compress_noalloc against gc_compress and against the CPU oracle.

Some callers cannot allocate device memory at all (a hook running inside a framework whose
allocator owns the device, a latency-bound loop), so they cannot create a plan.  The
entry point they use keeps its scratch in a fixed array inside the library; this test calls
it through the C ABI and requires bit-identical indices, values and residual to what the
plan-based gc_compress gives on the same inputs -- twice in a row, because the second call
meets the first call's leftovers in the shared array -- and to what the oracle gives.  The
file name keeps it last in collection order, so a failure here cannot hide the other tests
from a stop-at-first run.
"""
import numpy as np
import pytest
import torch

import oracle
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


def oracle_compress(n, k, g, r):
    """The CPU definition on host copies; returns (idx, val, residual) as uint32 bit patterns."""
    r_cpu = r.cpu().numpy().copy()
    oi, ov = oracle.topk_compress_tensors([n], [k], g.cpu().numpy(), r_cpu)
    return oi, ov.view(np.uint32), r_cpu.view(np.uint32)


def u32(t):
    return t.cpu().numpy().view(np.uint32)


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
        o_idx, o_val, o_r = oracle_compress(n, k, g, r)
        out_idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        out_val = torch.full((k,), float("nan"), device="cuda")
        rc = api.compress_noalloc(g, r, n, k, out_idx, out_val, status)
        assert rc == api.GC_OK
        torch.cuda.synchronize()
        assert status.item() == api.GC_OK
        assert torch.equal(out_idx, want_idx)
        assert torch.equal(out_val.view(torch.int32), want_val.view(torch.int32))
        assert torch.equal(r.view(torch.int32), want_r.view(torch.int32))
        assert np.array_equal(u32(out_idx), o_idx) and np.array_equal(u32(out_val), o_val)
        assert np.array_equal(u32(r), o_r)
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


@pytest.mark.parametrize("n,k", [(api.GC_NOALLOC_MAX_N, 16_778), (4093, 4093), (4093, 1), (1000, 1000), (17, 1),
                                 (300_007, 300_007)])
def test_extreme_k_and_the_largest_size_match_the_oracle(n, k):
    """k = n, k = 1, a tensor shorter than one tile and the largest size the fixed scratch
    takes (every tile word of the array in use), each bit for bit against the CPU oracle."""
    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(n % 1000 + k % 7)
    g = torch.randn(n, device="cuda", generator=gen)
    r = torch.randn(n, device="cuda", generator=gen) * 0.5
    o_idx, o_val, o_r = oracle_compress(n, k, g, r)
    out_idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
    out_val = torch.full((k,), float("nan"), device="cuda")
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    assert api.compress_noalloc(g, r, n, k, out_idx, out_val, status) == api.GC_OK
    torch.cuda.synchronize()
    assert status.item() == api.GC_OK
    assert np.array_equal(u32(out_idx), o_idx) and np.array_equal(u32(out_val), o_val)
    assert np.array_equal(u32(r), o_r)


def test_k_zero_still_folds_the_gradient_into_the_residual():
    """Nothing is sent, but the gradient must not be lost: r' = fl32(g + r), and the status word
    is written."""
    torch.cuda.set_device(0)
    n = 70_001
    gen = torch.Generator(device="cuda").manual_seed(5)
    g = torch.randn(n, device="cuda", generator=gen)
    r = torch.randn(n, device="cuda", generator=gen)
    o_idx, o_val, o_r = oracle_compress(n, 0, g, r)
    assert o_idx.size == 0
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    assert api.compress_noalloc(g, r, n, 0, None, None, status) == api.GC_OK
    torch.cuda.synchronize()
    assert status.item() == api.GC_OK
    assert np.array_equal(u32(r), o_r)
    status.fill_(77)
    assert api.compress_noalloc(g, r, 0, 0, None, None, status) == api.GC_OK       # n = 0: only the status
    torch.cuda.synchronize()
    assert status.item() == api.GC_OK


def test_a_warmed_up_call_allocates_no_device_memory():
    torch.cuda.set_device(0)
    n, k = 1_000_003, 1000
    g = torch.randn(n, device="cuda")
    r = torch.zeros(n, device="cuda")
    out_idx = torch.empty(k, dtype=torch.int32, device="cuda")
    out_val = torch.empty(k, device="cuda")
    assert api.compress_noalloc(g, r, n, k, out_idx, out_val, None) == api.GC_OK     # set-up happens here
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        assert api.compress_noalloc(g, r, n, k, out_idx, out_val, None) == api.GC_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_sizes_beyond_the_fixed_scratch_are_refused():
    torch.cuda.set_device(0)
    g = torch.zeros(16, device="cuda")
    i = torch.zeros(16, dtype=torch.int32, device="cuda")
    assert api.compress_noalloc(g, g.clone(), api.GC_NOALLOC_MAX_N + 1, 1, i, g.clone()) == api.GC_E_TOO_LARGE
    assert api.compress_noalloc(g, g.clone(), 8, 9, i, g.clone()) == api.GC_E_INVALID
    assert api.compress_noalloc(g, g.clone(), 0, 0, i, g.clone()) == api.GC_OK
    torch.cuda.synchronize()
