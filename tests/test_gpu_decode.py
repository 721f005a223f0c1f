"""GPU parity of gc_decompress_accumulate against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_01981_b200 import api, build, synth
from helpers import GpuWorker, bits, to_np_u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    api.lib()


ROUTES = {"auto": api.GC_DECODE_AUTO, "narrow": api.GC_DECODE_NARROW, "wide": api.GC_DECODE_WIDE}


def routed_plan(route, *args, **kwargs):
    """A plan whose tiled decode is pinned to one of its two kernels (or left to choose)."""
    plan = api.Plan(*args, **kwargs)
    plan.set_option(api.GC_OPT_DECODE_ROUTE, ROUTES[route])
    return plan


def run_workers(sizes, density, W, seed, steps=1, dist_scale=None):
    """W workers compress `steps` times on GPU; returns plan, workers, last gradients (cpu)."""
    plan = api.Plan(sizes, density, device=0)
    workers = [GpuWorker(plan) for _ in range(W)]
    n = plan.total_n
    grads = []
    for w, wk in enumerate(workers):
        for s in range(steps):
            gen = torch.Generator().manual_seed(seed + 1000 * w + s)
            g = torch.randn(n, generator=gen) * (dist_scale[w] if dist_scale else 1.0)
            wk.step(g.cuda())
        grads.append(g)
    return plan, workers, grads


def synthetic_sets(plan, sizes, W, seed, share_every=0):
    """W seeded sparse sets shaped like this plan's top-k output, as numpy pairs and as device
    tensors.  They come from the input generator, never from the CUDA compress path.  With
    share_every = s, groups of s consecutive workers use the same indices (collisions)."""
    ks = plan.tensor_k()
    pairs, d_idx, d_val = [], [], []
    for w in range(W):
        iseed = seed + (w // share_every if share_every else w)
        idx, _ = synth.sparse_set(sizes, ks, iseed)
        _, val = synth.sparse_set(sizes, ks, 7919 * seed + w, scale=10.0 ** (w % 5 - 2))
        pairs.append((idx, val))
        d_idx.append(torch.from_numpy(idx.view(np.int32)).cuda())
        d_val.append(torch.from_numpy(val).cuda())
    return pairs, d_idx, d_val


@pytest.mark.parametrize("W", [1, 2, 8])
@pytest.mark.parametrize("sizes,density", [([100_000], 0.01), ([5, 3, 1000, 7, 8193, 64, 70001], 0.02),
                                           ([40_000], 0.5)])
@pytest.mark.parametrize("route", list(ROUTES))
def test_decode_matches_oracle_bitwise(W, sizes, density, route):
    plan = routed_plan(route, sizes, density, device=0)
    ws = plan.alloc_workspace()
    pairs, d_idx, d_val = synthetic_sets(plan, sizes, W, seed=3, share_every=2)
    n = plan.total_n
    out = torch.full((n,), 7.0, device="cuda")
    plan.decompress_accumulate(d_idx, d_val, None, out, True, ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))
    # with explicit count arrays (one launch per worker) the result is the same
    T = len(sizes)
    cnt = torch.tensor(plan.tensor_k() * 2, dtype=torch.int32, device="cuda")
    out2 = torch.full((n,), 7.0, device="cuda")
    plan.decompress_accumulate(d_idx, d_val, [cnt] * W, out2, True, ws)
    assert torch.equal(out, out2)
    # accumulate mode adds on top of the existing content
    plan.decompress_accumulate(d_idx, d_val, None, out2, False, ws)
    want2 = oracle.decode_accumulate(pairs, want.copy(), False)
    assert np.array_equal(to_np_u32(out2), bits(want2))
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK


@pytest.mark.parametrize("W", [3, 16, 33, 64])
@pytest.mark.parametrize("route", list(ROUTES))
def test_decode_many_workers_and_unaligned_output(W, route):
    """Worker counts that are not powers of two, more than 32 workers, duplicate indices across
    workers, and a dense buffer that is only 4-byte aligned (no bulk copies)."""
    sizes = [70_001, 9, 20_000]
    plan = routed_plan(route, sizes, 0.03, device=0)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val = synthetic_sets(plan, sizes, W, seed=5, share_every=3)
    for shift in (0, 1):
        backing = torch.full((n + 8,), 3.0, device="cuda")
        out = backing[shift:shift + n]
        for zero_first in (True, False):
            before = out.cpu().numpy().copy()
            plan.decompress_accumulate(d_idx, d_val, None, out, zero_first, ws)
            want = oracle.decode_accumulate(pairs, before, zero_first)
            assert np.array_equal(to_np_u32(out), bits(want)), (W, shift, zero_first)
        assert backing[shift + n:].eq(3.0).all() and backing[:shift].eq(3.0).all()
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK


@pytest.mark.parametrize("W,density", [(16, 0.01), (32, 0.01), (64, 0.004), (8, 0.04)])
@pytest.mark.parametrize("route", list(ROUTES))
def test_decode_many_workers_at_one_percent(W, density, route):
    """Sixteen and more workers at 1 % density (the all-gathered lists of as many ranks): a
    worker's share of a tile exceeds four entries per thread, so the wider pre-load is taken;
    plain decode in both modes and the fused momentum step."""
    sizes = [1_000_003]
    plan = routed_plan(route, sizes, density, device=0)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val = synthetic_sets(plan, sizes, W, seed=17, share_every=5)
    out = torch.full((n,), 2.0, device="cuda")
    for zero_first in (True, False):
        before = out.cpu().numpy().copy()
        plan.decompress_accumulate(d_idx, d_val, None, out, zero_first, ws)
        want = oracle.decode_accumulate(pairs, before, zero_first)
        assert np.array_equal(to_np_u32(out), bits(want)), (W, zero_first)
    gen = torch.Generator().manual_seed(3)
    p = torch.randn(n, generator=gen); v = torch.randn(n, generator=gen) * 0.1
    d_p, d_v = p.cuda(), v.cuda()
    h_p, h_v = p.numpy().copy(), v.numpy().copy()
    plan.decompress_apply_momentum(d_idx, d_val, None, d_p, d_v, 0.05, 0.9, 1.0 / W, ws)
    oracle.decode_apply_momentum(pairs, h_p, h_v, 0.05, 0.9, 1.0 / W)
    assert np.array_equal(to_np_u32(d_v), bits(h_v)) and np.array_equal(to_np_u32(d_p), bits(h_p))
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK


def test_config5_sixteen_workers_full_size_decode():
    """The 355M-element workload: 16 seeded sparse sets of k = 354,824 pairs each, decoded in one
    call; every element is checked against the oracle."""
    w = synth.workload(4)
    plan = api.Plan(w.sizes, w.density, device=0)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val = synthetic_sets(plan, w.sizes, w.workers, seed=11, share_every=4)
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate(d_idx, d_val, None, out, True, ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK


def test_density_one_reproduces_the_dense_sum():
    sizes, W = [9, 30_000, 4097], 5
    plan, workers, grads = run_workers(sizes, 1.0, W, seed=11, dist_scale=[1.0, 1e3, 1e-3, 50.0, 0.1])
    n = plan.total_n
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate([w.idx for w in workers], [w.val for w in workers], None, out, True,
                               workers[0].ws)
    dense = np.zeros(n, np.float32)
    for g in grads:
        dense = (dense + g.numpy()).astype(np.float32)
    assert np.array_equal(to_np_u32(out), bits(dense))
    for w in workers:
        assert not w.residual.any()


@pytest.mark.parametrize("route", list(ROUTES))
def test_worker_order_is_observable_and_fixed(route):
    plan = routed_plan(route, [8], 1.0, device=0)
    ws = plan.alloc_workspace()
    idx = torch.arange(8, dtype=torch.int32, device="cuda")
    a = torch.full((8,), 1e8, device="cuda")
    b = torch.ones(8, device="cuda")
    out = torch.empty(8, device="cuda")
    plan.decompress_accumulate([idx, idx, idx], [a, b, -a], None, out, True, ws)
    assert out.tolist() == [0.0] * 8
    plan.decompress_accumulate([idx, idx, idx], [a, -a, b], None, out, True, ws)
    assert out.tolist() == [1.0] * 8


@pytest.mark.parametrize("route", list(ROUTES))
def test_out_of_range_index_is_skipped_and_reported(route):
    plan = routed_plan(route, [100], 0.04, device=0)          # k = 4
    ws = plan.alloc_workspace()
    idx = torch.tensor([1, 50, 99, 100], dtype=torch.int32, device="cuda")
    val = torch.ones(4, device="cuda")
    out = torch.empty(100, device="cuda")
    plan.decompress_accumulate([idx], [val], None, out, True, ws)
    st, det = plan.last_status(ws)
    assert st == api.GC_E_INVALID and det == 3          # position of the bad entry in the list
    assert out.sum().item() == 3.0
    # the per-worker launch path (count arrays given) reports the same
    ws.zero_()
    cnt = torch.tensor([4, 4], dtype=torch.int32, device="cuda")
    plan.decompress_accumulate([idx], [val], [cnt], out, True, ws)
    st, det = plan.last_status(ws)
    assert st == api.GC_E_INVALID and det == 3
    assert out.sum().item() == 3.0


@pytest.mark.parametrize("route", list(ROUTES))
def test_list_that_is_not_ascending_is_reported_and_stays_in_bounds(route):
    """A list whose indices step backwards across a tile boundary: the call ends, writes only
    inside the dense buffer and leaves GC_E_INVALID in the status word."""
    plan = routed_plan(route, [20_000], 0.0002, device=0)          # k = 4
    assert plan.total_cap == 4
    ws = plan.alloc_workspace()
    idx = torch.tensor([9000, 5, 9001, 9002], dtype=torch.int32, device="cuda")
    val = torch.ones(4, device="cuda")
    backing = torch.full((20_000 + 64,), 7.0, device="cuda")
    out = backing[32:32 + 20_000]
    plan.decompress_accumulate([idx], [val], None, out, True, ws)
    st, _ = plan.last_status(ws)
    assert st == api.GC_E_INVALID
    assert backing[:32].eq(7.0).all() and backing[32 + 20_000:].eq(7.0).all()
    assert 0.0 <= out.sum().item() <= 4.0


def test_config4_eight_resnet_workers_decode():
    w = synth.workload(3)
    plan = api.Plan(w.sizes, w.density, device=0)
    ks = plan.tensor_k()
    n = plan.total_n
    workers = [GpuWorker(plan) for _ in range(w.workers)]
    pairs = []
    for i, wk in enumerate(workers):
        g = synth.gradient(w, i, 0, device="cuda")
        wk.step(g)
        r = np.zeros(n, np.float32)
        oi, ov = oracle.topk_compress_tensors(w.sizes, ks, g.cpu().numpy(), r)
        assert np.array_equal(to_np_u32(wk.idx[:plan.total_cap]), oi)
        assert np.array_equal(to_np_u32(wk.val[:plan.total_cap]), bits(ov))
        assert np.array_equal(to_np_u32(wk.residual[:n]), bits(r))
        pairs.append((oi, ov))
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate([x.idx for x in workers], [x.val for x in workers], None, out, True,
                               workers[0].ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))


@pytest.mark.parametrize("W", [1, 3, 8])
@pytest.mark.parametrize("route", list(ROUTES))
def test_one_tensor_lists_with_counts_use_their_length(W, route):
    """Threshold-mode lists of a one-tensor plan: the slots hold `cap` pairs but only the first
    count[0] are valid; whatever lies behind them (here: junk indices) must not be applied."""
    n = 3_000_001
    plan = routed_plan(route, [n], 0.001, mode=api.GC_THRESHOLD, device=0)
    cap = plan.tensor_cap()[0]
    ws = plan.alloc_workspace()
    pairs, d_idx, d_val, d_cnt = [], [], [], []
    for w in range(W):
        m = [cap, cap // 2 + 17 * w, 0, 1][(w + 1) % 4] if W > 1 else cap // 3
        idx, val = synth.sparse_set([n], [m], seed=40 + w)
        pairs.append((idx, val))
        full_idx = np.full(cap, 0xFFFFFFFF, np.uint32); full_idx[:m] = idx
        full_idx[m:] = np.arange(cap - m, dtype=np.uint32)[::-1] * 3 % n          # junk, not even ascending
        full_val = np.full(cap, 1e30, np.float32); full_val[:m] = val
        d_idx.append(torch.from_numpy(full_idx.view(np.int32)).cuda())
        d_val.append(torch.from_numpy(full_val).cuda())
        d_cnt.append(torch.tensor([m, m], dtype=torch.int32, device="cuda"))
    out = torch.full((n,), 2.0, device="cuda")
    for zero_first in (True, False):
        before = out.cpu().numpy().copy()
        plan.decompress_accumulate(d_idx, d_val, d_cnt, out, zero_first, ws)
        want = oracle.decode_accumulate(pairs, before, zero_first)
        assert np.array_equal(to_np_u32(out), bits(want)), (W, zero_first)
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK


def lists_with_counts(plan, sizes, W, seed, fill):
    """W threshold-mode lists of a many-tensor plan built from the input generator: worker w sends
    m[w][t] <= cap[t] pairs of tensor t (from nothing to the full capacity), laid out at the tensor's
    output offset; the unused slots behind them hold junk (indices that are not ascending and lie
    in other tensors, huge values) that must never be applied.  Returns oracle pairs and device
    idx / val / count tensors."""
    rng = np.random.default_rng(seed)
    caps, offs = plan.tensor_cap(), plan.tensor_out_offset()
    T, n, total_cap = len(sizes), plan.total_n, plan.total_cap
    pairs, d_idx, d_val, d_cnt = [], [], [], []
    for w in range(W):
        m = []
        for t in range(T):
            mode = (w + t) % 4 if fill == "mixed" else fill
            m.append(int({0: caps[t], 1: caps[t] // 2, 2: 0, 3: min(caps[t], 1), "full": caps[t]}[mode]))
        idx, val = synth.sparse_set(sizes, m, seed + 31 * w, scale=10.0 ** (w % 4 - 2))
        pairs.append((idx, val))
        full_idx = ((rng.integers(0, max(n, 1), size=max(total_cap, 1))).astype(np.uint32))[:total_cap]
        full_val = np.full(total_cap, 3e30, np.float32)
        pos = 0
        for t in range(T):
            full_idx[offs[t]:offs[t] + m[t]] = idx[pos:pos + m[t]]
            full_val[offs[t]:offs[t] + m[t]] = val[pos:pos + m[t]]
            pos += m[t]
        d_idx.append(torch.from_numpy(full_idx.view(np.int32)).cuda())
        d_val.append(torch.from_numpy(full_val).cuda())
        d_cnt.append(torch.tensor(m + [x + 5 for x in m], dtype=torch.int32, device="cuda"))    # [T + t] = hits: unused here
    return pairs, d_idx, d_val, d_cnt


@pytest.mark.parametrize("W", [1, 2, 3, 8, 17, 64])
@pytest.mark.parametrize("sizes,density,fill", [
    ([5, 3, 1000, 7, 8193, 64, 1, 0, 2, 70_001, 300_000, 0, 6, 131_073], 0.01, "mixed"),
    ([0, 0, 40_000, 0, 8192, 8192, 16_384, 3, 0], 0.05, "mixed"),
    ([300_007, 64, 64, 128, 2_000_001, 512, 512], 0.002, "full"),
    ([20_000] * 40, 0.3, "mixed"),
])
def test_many_tensor_lists_with_counts_match_the_oracle(W, sizes, density, fill):
    """Threshold-mode lists of plans with several tensors: every tensor's pairs start at its output
    offset and only count[t] of its slots are live.  Plain decode in both modes and the fused
    momentum step, bit for bit, through the tile kernel that walks the tensors' segments."""
    plan = api.Plan(sizes, density, mode=api.GC_THRESHOLD, device=0, cap_factor=1.5)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val, d_cnt = lists_with_counts(plan, sizes, W, seed=90 + W, fill=fill)
    launches0 = plan.launches()
    out = torch.full((n,), 2.0, device="cuda")
    for zero_first in (True, False):
        before = out.cpu().numpy().copy()
        plan.decompress_accumulate(d_idx, d_val, d_cnt, out, zero_first, ws)
        want = oracle.decode_accumulate(pairs, before, zero_first)
        assert np.array_equal(to_np_u32(out), bits(want)), (W, zero_first)
    assert plan.launches() - launches0 == 2            # one tile kernel per call, no per-worker launches
    gen = torch.Generator().manual_seed(3)
    p = torch.randn(n, generator=gen); v = torch.randn(n, generator=gen) * 0.1
    d_p, d_v = p.cuda(), v.cuda()
    h_p, h_v = p.numpy().copy(), v.numpy().copy()
    plan.decompress_apply_momentum(d_idx, d_val, d_cnt, d_p, d_v, 0.05, 0.9, 1.0 / W, ws)
    oracle.decode_apply_momentum(pairs, h_p, h_v, 0.05, 0.9, 1.0 / W)
    assert np.array_equal(to_np_u32(d_v), bits(h_v)) and np.array_equal(to_np_u32(d_p), bits(h_p))
    st, det = plan.last_status(ws)
    assert st == api.GC_OK, (st, det)


def test_many_tensor_lists_with_counts_report_an_index_outside_its_tensor():
    """A live pair whose index lies beyond its tensor's last element is skipped and reported."""
    sizes = [10_000, 10_000]
    plan = api.Plan(sizes, 0.001, mode=api.GC_THRESHOLD, device=0)       # cap 20 per tensor
    caps, offs = plan.tensor_cap(), plan.tensor_out_offset()
    ws = plan.alloc_workspace()
    idx = torch.zeros(plan.total_cap, dtype=torch.int32, device="cuda")
    val = torch.ones(plan.total_cap, device="cuda")
    idx[offs[0]:offs[0] + 3] = torch.tensor([5, 9_000, 10_500], dtype=torch.int32)    # the third belongs to tensor 1
    idx[offs[1]:offs[1] + 2] = torch.tensor([12_000, 19_999], dtype=torch.int32)
    cnt = torch.tensor([3, 2, 3, 2], dtype=torch.int32, device="cuda")
    out = torch.empty(plan.total_n, device="cuda")
    plan.decompress_accumulate([idx], [val], [cnt], out, True, ws)
    st, _ = plan.last_status(ws)
    assert st == api.GC_E_INVALID
    assert out.sum().item() == 4.0 and out[10_500].item() == 0.0


@pytest.mark.parametrize("W", [0, 1, 3, 16])
@pytest.mark.parametrize("sizes,density", [([100_003], 0.01), ([5, 3, 1000, 7, 8193, 64, 70001], 0.02)])
@pytest.mark.parametrize("route", list(ROUTES))
def test_decode_apply_momentum_matches_oracle_bitwise(W, sizes, density, route):
    """The decode with momentum SGD fused behind it: parameter and velocity after three steps."""
    plan = routed_plan(route, sizes, density, device=0)
    ws = plan.alloc_workspace()
    n = plan.total_n
    gen = torch.Generator().manual_seed(7)
    p = torch.randn(n, generator=gen); v = torch.randn(n, generator=gen) * 0.1
    d_p, d_v = p.cuda(), v.cuda()
    h_p, h_v = p.numpy().copy(), v.numpy().copy()
    for step in range(3):
        pairs, d_idx, d_val = synthetic_sets(plan, sizes, W, seed=60 + step, share_every=2) if W else ([], [], [])
        plan.decompress_apply_momentum(d_idx, d_val, None, d_p, d_v, 0.05, 0.9, 1.0 / max(W, 1), ws)
        oracle.decode_apply_momentum(pairs, h_p, h_v, 0.05, 0.9, 1.0 / max(W, 1))
        assert np.array_equal(to_np_u32(d_v), bits(h_v)), (W, step)
        assert np.array_equal(to_np_u32(d_p), bits(h_p)), (W, step)
    st, _ = plan.last_status(ws)
    assert st == api.GC_OK


def test_decode_apply_momentum_full_size_matches_the_unfused_pair():
    """110M-element workload, W = 1: the fused call gives the same bits as decode into a dense
    buffer followed by the same momentum step written with torch ops that round once each."""
    w = synth.workload(2)
    plan = api.Plan(w.sizes, w.density, device=0)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val = synthetic_sets(plan, w.sizes, 1, seed=13)
    gen = torch.Generator(device="cuda").manual_seed(1)
    p = torch.randn(n, device="cuda", generator=gen); v = torch.randn(n, device="cuda", generator=gen)
    p2, v2 = p.clone(), v.clone()
    plan.decompress_apply_momentum(d_idx, d_val, None, p, v, 0.01, 0.9, 1.0, ws)
    dense = torch.empty(n, device="cuda")
    plan.decompress_accumulate(d_idx, d_val, None, dense, True, ws)
    v2 = torch.mul(v2, 0.9) + torch.mul(dense, 1.0)          # separate kernels: no contraction into an fma
    p2 = p2 - torch.mul(v2, 0.01)
    assert torch.equal(v.view(torch.int32), v2.view(torch.int32))
    assert torch.equal(p.view(torch.int32), p2.view(torch.int32))


@pytest.mark.parametrize("seed", list(range(12)))
def test_random_plans_and_worker_counts_match_the_oracle(seed):
    """Seeded random plans (1-5 tensors with sizes around the tile boundaries), densities from
    0.01 % to 100 %, 1-64 workers with and without shared index sets, each of the decode routes:
    plain decode in both modes and the fused momentum step, bit for bit."""
    rng = np.random.default_rng(777 + seed)
    menu = [1, 5, 64, 1000, 4097, 8191, 8192, 8193, 16385, 50001, 131072, 300007]
    sizes = [int(menu[int(rng.integers(0, len(menu)))]) for _ in range(int(rng.integers(1, 6)))]
    density = float(rng.choice([1e-4, 1e-3, 0.01, 0.03, 0.1, 0.4, 1.0]))
    W = int(rng.choice([1, 2, 3, 5, 8, 13, 16, 24, 32, 47, 64]))
    share = int(rng.choice([0, 0, 2, 7]))
    route = ["auto", "narrow", "wide"][int(rng.integers(0, 3))]
    plan = routed_plan(route, sizes, density, device=0)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val = synthetic_sets(plan, sizes, W, seed=1000 + seed, share_every=share)
    out = torch.full((max(n, 4),), 2.5, device="cuda")[:n]
    for zero_first in (True, False):
        before = out.cpu().numpy().copy()
        plan.decompress_accumulate(d_idx, d_val, None, out, zero_first, ws)
        want = oracle.decode_accumulate(pairs, before, zero_first)
        assert np.array_equal(to_np_u32(out), bits(want)), (sizes, density, W, share, route, zero_first)
    p0 = np.random.default_rng(seed).standard_normal(n).astype(np.float32)
    v0 = (p0 * np.float32(0.1)).astype(np.float32)
    d_p, d_v = torch.from_numpy(p0.copy()).cuda(), torch.from_numpy(v0.copy()).cuda()
    plan.decompress_apply_momentum(d_idx, d_val, None, d_p, d_v, 0.05, 0.9, 1.0 / W, ws)
    oracle.decode_apply_momentum(pairs, p0, v0, 0.05, 0.9, 1.0 / W)
    assert np.array_equal(to_np_u32(d_p), bits(p0)) and np.array_equal(to_np_u32(d_v), bits(v0))
    st, det = plan.last_status(ws)
    assert st == api.GC_OK, (st, det)


@pytest.mark.parametrize("W,density,share", [(1, 0.01, 0), (4, 0.02, 2), (16, 0.01, 0), (16, 0.01, 4), (8, 0.3, 0)])
def test_any_order_decode_stays_within_the_rounding_bound(W, density, share):
    """GC_ORDER_ANY: elements hit by one worker equal the fixed-order result bit for bit; the
    others lie within (hits - 1) x 2^-24 x sum |values| of it, which is below the 1e-6 relative
    bound for up to 16 workers.  Plain decode, accumulate mode and the fused momentum step."""
    sizes = [300_007, 8193]
    plan = api.Plan(sizes, density, device=0)
    plan.set_option(api.GC_OPT_DECODE_ORDER, api.GC_ORDER_ANY)
    ws = plan.alloc_workspace()
    n = plan.total_n
    pairs, d_idx, d_val = synthetic_sets(plan, sizes, W, seed=31, share_every=share)
    hits = np.zeros(n, np.int64)
    mag = np.zeros(n, np.float64)
    for i, v in pairs:
        np.add.at(hits, i, 1)
        np.add.at(mag, i, np.abs(v.astype(np.float64)))
    out = torch.full((n,), 0.5, device="cuda")
    for zero_first in (True, False):
        before = out.cpu().numpy().copy()
        plan.decompress_accumulate(d_idx, d_val, None, out, zero_first, ws)
        want = oracle.decode_accumulate(pairs, before.copy(), zero_first)
        got = out.cpu().numpy()
        lone = hits <= (1 if zero_first else 0)
        assert np.array_equal(got[lone].view(np.uint32), want[lone].view(np.uint32))
        bound = 1e-6 * (mag + np.abs(before.astype(np.float64)) * (0 if zero_first else 1))
        assert np.all(np.abs(got.astype(np.float64) - want.astype(np.float64)) <= bound + 1e-30), (W, zero_first)
    p0 = np.random.default_rng(5).standard_normal(n).astype(np.float32)
    v0 = (p0 * np.float32(0.1)).astype(np.float32)
    d_p, d_v = torch.from_numpy(p0.copy()).cuda(), torch.from_numpy(v0.copy()).cuda()
    plan.decompress_apply_momentum(d_idx, d_val, None, d_p, d_v, 0.05, 0.9, 1.0, ws)
    oracle.decode_apply_momentum(pairs, p0, v0, 0.05, 0.9, 1.0)
    assert np.all(np.abs(d_v.cpu().numpy().astype(np.float64) - v0) <= 1e-6 * (mag + np.abs(v0)) + 1e-30)
    assert np.all(np.abs(d_p.cpu().numpy().astype(np.float64) - p0) <= 1e-6 * (mag + np.abs(p0) + np.abs(v0)) + 1e-30)
    st, det = plan.last_status(ws)
    assert st == api.GC_OK, (st, det)
