"""GPU parity of gc_compress (top-k mode) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_01981_b200 import api, build, synth
from helpers import GpuWorker, bits, check_topk_against_oracle, to_np_u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    api.lib()


def randn(n, seed, scale=1.0):
    gen = torch.Generator().manual_seed(seed)
    return torch.randn(n, generator=gen) * scale


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 31, 32, 33, 1023, 1024, 1025, 8191, 8192, 8193, 8196,
                               16384, 16385, 100_003, (1 << 20) - 1, (1 << 20) + 1])
@pytest.mark.parametrize("density", [1e-9, 0.01, 1.0])
def test_single_tensor_sizes_and_extreme_k(n, density):
    grads = [randn(n, 17 * n + s) for s in range(2)]
    check_topk_against_oracle([n], density, grads, r0=randn(n, 5 * n + 1, 0.3))


def test_many_ragged_tensors_misaligned_offsets():
    sizes = [5, 3, 1000, 7, 8193, 64, 1, 0, 2, 16384, 9, 70001, 0, 6]
    n = sum(sizes)
    grads = [randn(n, 100 + s) for s in range(3)]
    for density in (0.001, 0.05, 0.5):
        check_topk_against_oracle(sizes, density, grads)


def test_tie_stress_quantised_values():
    n = 300_000
    grads = [synth.quantised_gradient(n, 40 + s) for s in range(3)]
    for density in (0.01, 0.2):
        check_topk_against_oracle([n], density, grads)
        check_topk_against_oracle([100_000, 100_000, 100_000], density, grads)


@pytest.mark.parametrize("step,expect_no_redo", [(2.0 ** -12, True), (2.0 ** -8, True), (2.0 ** -6, True),
                                                   (2.0 ** -4, False)])
def test_one_tensor_ties_at_the_threshold(step, expect_no_redo):
    """One large tensor whose values sit on a grid: from a dozen to thousands of elements share the
    threshold magnitude, so the tie cut (lowest indices win) decides; up to a few thousand ties the
    one-tensor kernel has to settle it without the exact redo."""
    n = 2_000_000
    grads = [synth.quantised_gradient(n, 70 + s, step=step) for s in range(2)]
    seen = []
    check_topk_against_oracle([n], 0.01, grads, expect_counters=seen.append)
    if expect_no_redo:
        assert all(c[1] == 0 and c[2] == 0 for c in seen), seen


def test_degenerate_values():
    n = 20_000
    for g in (torch.zeros(n), torch.full((n,), -2.5), torch.cat([torch.ones(n // 2), -torch.ones(n // 2)])):
        check_topk_against_oracle([n], 0.01, [g, g])
    g = randn(n, 9)
    g[::7] = float("inf")
    g[3::11] = float("nan")
    g[5::13] = -0.0
    g[1::17] = 1e-42                  # denormal
    check_topk_against_oracle([n], 0.05, [g])


def test_config1_three_steps_error_feedback():
    w = synth.workload(0)
    grads = [synth.gradient(w, 0, s, device="cuda") for s in range(w.steps)]
    check_topk_against_oracle(w.sizes, w.density, grads)


class LazyGrads:
    """The gradients of one worker, generated step by step (one full-size buffer alive at a time)."""

    def __init__(self, w, worker, steps):
        self.w, self.worker, self.steps = w, worker, steps

    def __iter__(self):
        for s in range(self.steps):
            yield synth.gradient(self.w, self.worker, s, device="cuda")


def test_config2_resnet50_layerwise_ten_steps():
    w = synth.workload(1)
    assert w.steps == 10
    seen = []
    check_topk_against_oracle(w.sizes, w.density, LazyGrads(w, 0, w.steps), expect_counters=seen.append)
    assert all(c[1] == 0 for c in seen), seen            # no candidate-list overflow on the workload itself


def test_config3_bert_full_size_ten_steps():
    """All ten error-feedback steps at full size: the unsent entries pile up under the threshold
    from step to step, which is what strains the sampled bracket."""
    w = synth.workload(2)
    assert w.steps == 10
    seen = []
    check_topk_against_oracle(w.sizes, w.density, LazyGrads(w, 0, w.steps), expect_counters=seen.append)
    assert all(c[1] == 0 and c[2] == 0 for c in seen), seen     # the safety net stayed idle


def test_config5_gpt2_medium_two_workers_five_steps():
    w = synth.workload(4)
    assert w.steps == 5
    for worker in (0, 15):
        check_topk_against_oracle(w.sizes, w.density, LazyGrads(w, worker, w.steps))
        torch.cuda.empty_cache()


def test_config5_gpt2_medium_sixteen_workers_compress_then_decode():
    """All 16 workers of the 355M-element workload, one step each: every worker's pairs and residual
    against the oracle, then ONE decode call over the 16 lists the CUDA compress produced against
    the oracle's sequential aggregation of the oracle's own lists."""
    w = synth.workload(4)
    assert w.workers == 16
    plan = api.Plan(w.sizes, w.density, device=0)
    ks, n, cap = plan.tensor_k(), plan.total_n, plan.total_cap
    wk = GpuWorker(plan)
    lists, pairs = [], []
    g = torch.empty(n, device="cuda")
    for worker in range(w.workers):
        synth.gradient(w, worker, 0, device="cuda", out=g)
        wk.residual.zero_()
        wk.step(g)
        wk.check_status()
        r_cpu = np.zeros(n, np.float32)
        oi, ov = oracle.topk_compress_tensors(w.sizes, ks, g.cpu().numpy(), r_cpu)
        assert np.array_equal(to_np_u32(wk.idx[:cap]), oi), worker
        assert np.array_equal(to_np_u32(wk.val[:cap]), bits(ov)), worker
        assert np.array_equal(to_np_u32(wk.residual[:n]), bits(r_cpu)), worker
        lists.append((wk.idx[:cap].clone(), wk.val[:cap].clone()))
        pairs.append((oi, ov))
    del g
    wk.residual = None
    torch.cuda.empty_cache()
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate([x[0] for x in lists], [x[1] for x in lists], None, out, True, wk.ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))
    wk.check_status()


@pytest.mark.parametrize("n,density,quantised", [(24_000_001, 0.01, True), (21_823_500, 0.003, False),
                                                (47_999_999, 0.01, False)])
def test_one_tensor_with_unequal_shares_per_cta(n, density, quantised):
    """Tensors of twelve and more rows of tiles per CTA column: the one-tensor kernel gives the
    three CTAs of an SM unequal numbers of rows (the last rows are only partly filled).  Three
    error-feedback steps, one of them with values quantised to 1/8 (thousands of ties at the
    threshold); also the safety-net routes on the same geometry."""
    gen = torch.Generator(device="cuda").manual_seed(n % 1000)
    grads = []
    for s in range(3):
        g = torch.randn(n, device="cuda", generator=gen)
        if quantised and s == 1:
            g = torch.round(g * 8) / 8
        grads.append(g)
    check_topk_against_oracle([n], density, grads)
    if quantised:
        check_topk_against_oracle([n], density, grads[:2], options={api.GC_OPT_SAMPLE_RANK_PERMILLE: 30})
        check_topk_against_oracle([n], density, grads[:1], options={api.GC_OPT_CANDIDATE_CAPACITY: 100})


PATHS = {
    "auto": {},
    "exact": {api.GC_OPT_PATH: api.GC_PATH_EXACT},
    "staged": {api.GC_OPT_PATH: api.GC_PATH_STAGED},
    "staged_starved": {api.GC_OPT_PATH: api.GC_PATH_STAGED, api.GC_OPT_SAMPLE_RANK_PERMILLE: 30},
    "staged_overflow": {api.GC_OPT_PATH: api.GC_PATH_STAGED, api.GC_OPT_CANDIDATE_CAPACITY: 100},
    "auto_starved": {api.GC_OPT_SAMPLE_RANK_PERMILLE: 30},      # candidate sets too small -> redo per tensor
    "auto_overflow": {api.GC_OPT_CANDIDATE_CAPACITY: 100},      # candidate list too short -> redo everything
}


@pytest.mark.parametrize("sizes", [[300_000, 5, 1_500_001, 131_072, 64, 131_071, 2_000_003], [3_000_001]],
                         ids=["many_tensors", "one_tensor"])
@pytest.mark.parametrize("path", list(PATHS))
def test_every_route_gives_the_same_bits(path, sizes):
    n = sum(sizes)
    grads = [randn(n, 900 + s) for s in range(3)]
    seen = []
    options = dict(PATHS[path])
    if path == "auto_overflow" and len(sizes) == 1:
        options[api.GC_OPT_CANDIDATE_CAPACITY] = 4        # the one-tensor kernel splits the list per CTA
    for density in (0.001, 0.01):
        check_topk_against_oracle(sizes, density, grads, options=options, expect_counters=seen.append)
    if path in ("auto", "staged"):
        assert all(c[1] == 0 and c[2] == 0 for c in seen), seen     # the safety net stayed idle
    if path.endswith("_starved"):
        assert all(c[2] >= 1 for c in seen), seen
    if path.endswith("_overflow"):
        assert all(c[1] == 1 for c in seen), seen


def run_workers_call(sizes, density, W, steps, seed, options=None, grads_fn=None, with_counts=True):
    """`steps` calls of gc_compress_workers for W workers; every worker's pairs, counts and residual
    against the oracle after every step.  Returns plan, workers and the oracle's last pairs."""
    plan = api.Plan(sizes, density, device=0)
    for opt, value in (options or {}).items():
        plan.set_option(opt, value)
    ks, n, T = plan.tensor_k(), plan.total_n, len(sizes)
    workers = [GpuWorker(plan) for _ in range(W)]
    r_cpu = [np.zeros(n, np.float32) for _ in range(W)]
    pairs = None
    for step in range(steps):
        if grads_fn is not None:
            grads = [grads_fn(w, step) for w in range(W)]
        else:
            grads = [randn(n, seed + 100 * w + step, scale=10.0 ** (w % 3 - 1)).cuda() for w in range(W)]
        for wk in workers:
            wk.idx.fill_(-1); wk.val.fill_(float("nan")); wk.count.fill_(-1)
        plan.compress_workers(grads, [wk.residual for wk in workers], [wk.idx for wk in workers],
                              [wk.val for wk in workers], [wk.count for wk in workers] if with_counts else None,
                              [wk.ws for wk in workers])
        pairs = []
        for w, wk in enumerate(workers):
            wk.check_status()
            oi, ov = oracle.topk_compress_tensors(list(sizes), ks, grads[w].cpu().numpy(), r_cpu[w])
            tot = sum(ks)
            assert np.array_equal(to_np_u32(wk.idx[:tot]), oi), (step, w)
            assert np.array_equal(to_np_u32(wk.val[:tot]), bits(ov)), (step, w)
            assert np.array_equal(to_np_u32(wk.residual[:n]), bits(r_cpu[w])), (step, w)
            if with_counts:
                cnt = wk.count.cpu().numpy()
                assert cnt[:T].tolist() == ks and cnt[T:2 * T].tolist() == ks, (step, w)
            pairs.append((oi, ov))
    return plan, workers, pairs


@pytest.mark.parametrize("W", [1, 2, 3, 8, 13, 27])
def test_workers_call_many_tensors_matches_the_oracle(W):
    """gc_compress_workers on a plan of several tensors (ragged sizes, misaligned starts, an empty
    tensor, single-tile tensors): the workers share cooperative launches -- from two to twelve per
    launch, a lone leftover worker on its own -- and each must come out exactly as a call of its own."""
    sizes = [300_000, 5, 1_500_001, 131_072, 64, 0, 131_071, 2_000_003, 4097, 1000]
    plan, workers, _ = run_workers_call(sizes, 0.003, W, steps=3, seed=4000 + W)
    seen = [plan.last_counters(wk.ws) for wk in workers]
    assert all(c[1] == 0 and c[2] == 0 for c in seen), seen


@pytest.mark.parametrize("options", [{api.GC_OPT_SAMPLE_RANK_PERMILLE: 30}, {api.GC_OPT_CANDIDATE_CAPACITY: 100},
                                     {api.GC_OPT_PATH: api.GC_PATH_EXACT}, {api.GC_OPT_PATH: api.GC_PATH_STAGED}],
                         ids=["starved", "overflow", "exact", "staged"])
def test_workers_call_safety_net_and_other_routes(options):
    """The redo routes inside the shared launch (brackets that miss, candidate regions that
    overflow) run per group of CTAs; plans on the other routes take one call per worker."""
    sizes = [300_000, 5, 1_500_001, 131_072, 64, 131_071, 2_000_003]
    plan, workers, _ = run_workers_call(sizes, 0.01, 4, steps=2, seed=4100, options=options)
    seen = [plan.last_counters(wk.ws) for wk in workers]
    if api.GC_OPT_SAMPLE_RANK_PERMILLE in options:
        assert all(c[2] >= 1 for c in seen), seen
    if api.GC_OPT_CANDIDATE_CAPACITY in options:
        assert all(c[1] == 1 for c in seen), seen


def test_workers_call_one_tensor_plan_and_ties():
    """One-tensor plans are served worker by worker; quantised values put thousands of ties at the
    thresholds of a many-tensor plan."""
    run_workers_call([3_000_001], 0.01, 3, steps=2, seed=4200, with_counts=False)
    n = 300_000
    run_workers_call([n, n, n], 0.01, 5, steps=2, seed=0,
                     grads_fn=lambda w, s: synth.quantised_gradient(3 * n, 40 + 7 * w + s).cuda())


def test_workers_call_rejects_shared_buffers():
    plan = api.Plan([100_000, 50_000], 0.01, device=0)
    a, b = GpuWorker(plan), GpuWorker(plan)
    g = torch.zeros(plan.total_n, device="cuda")
    with pytest.raises(api.GcError) as e:
        plan.compress_workers([g, g], [a.residual, b.residual], [a.idx, b.idx], [a.val, b.val], None, [a.ws, a.ws])
    assert e.value.code == api.GC_E_INVALID
    with pytest.raises(api.GcError):
        plan.compress_workers([g, g], [a.residual, a.residual], [a.idx, b.idx], [a.val, b.val], None, [a.ws, b.ws])
    plan.compress_workers([], [], [], [], None, [])            # no workers: nothing happens
    torch.cuda.synchronize()


def test_config4_eight_resnet_workers_in_one_call_then_decode():
    """The 8-worker ResNet-50 workload as one gc_compress_workers call per step (two steps, so the
    error feedback of every worker is exercised), then the decode of the 8 lists."""
    w = synth.workload(3)
    assert w.workers == 8
    plan, workers, pairs = run_workers_call(w.sizes, w.density, w.workers, steps=2, seed=0,
                                            grads_fn=lambda wk, s: synth.gradient(w, wk, s, device="cuda"))
    n = plan.total_n
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate([x.idx for x in workers], [x.val for x in workers], None, out, True, workers[0].ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))


def test_which_plans_take_which_route():
    """The five workloads take the one-tensor or the many-tensor kernel; a candidate set too large
    for the per-CTA regions (20 % of 20M elements) takes the general candidate kernel, and that
    route is exact too; the path option and the mode pick the others."""
    for cfg, want in ((0, api.GC_ROUTE_TOPK_ONE), (1, api.GC_ROUTE_TOPK_MANY), (2, api.GC_ROUTE_TOPK_ONE),
                      (3, api.GC_ROUTE_TOPK_MANY), (4, api.GC_ROUTE_TOPK_ONE)):
        w = synth.workload(cfg)
        assert api.Plan(w.sizes, w.density, device=0).query(api.GC_Q_COMPRESS_ROUTE) == want, cfg
        thr = api.Plan(w.sizes, w.density, mode=api.GC_THRESHOLD, device=0).query(api.GC_Q_COMPRESS_ROUTE)
        assert thr == (api.GC_ROUTE_THRESHOLD_ONE if len(w.sizes) == 1 else api.GC_ROUTE_THRESHOLD_MANY), cfg
    n = 20_000_000
    plan = api.Plan([n], 0.2, device=0)
    assert plan.query(api.GC_Q_COMPRESS_ROUTE) == api.GC_ROUTE_TOPK_GENERAL
    gen = torch.Generator(device="cuda").manual_seed(12)
    grads = [torch.randn(n, device="cuda", generator=gen) for _ in range(2)]
    seen = []
    check_topk_against_oracle([n], 0.2, grads, expect_counters=seen.append)
    assert all(c[1] == 0 and c[2] == 0 for c in seen), seen
    many = api.Plan([3_000_000] * 4, 0.3, device=0)
    assert many.query(api.GC_Q_COMPRESS_ROUTE) in (api.GC_ROUTE_TOPK_MANY, api.GC_ROUTE_TOPK_GENERAL)
    for opt, want in ((api.GC_PATH_EXACT, api.GC_ROUTE_EXACT), (api.GC_PATH_STAGED, api.GC_ROUTE_TOPK_STAGED)):
        plan.set_option(api.GC_OPT_PATH, opt)
        assert plan.query(api.GC_Q_COMPRESS_ROUTE) == want
    assert api.Plan([100], 0.1, device=-1).query(api.GC_Q_COMPRESS_ROUTE) == api.GC_ROUTE_NONE


@pytest.mark.parametrize("options", [{}, {api.GC_OPT_SAMPLE_RANK_PERMILLE: 30}, {api.GC_OPT_CANDIDATE_CAPACITY: 4}],
                         ids=["plain", "starved", "overflow"])
def test_private_workspace_skips_the_clearing_launch_and_stays_exact(options):
    """GC_OPT_WORKSPACE_PRIVATE: from the second call on a workspace, the one-tensor kernel runs
    without the clearing launch in front of it (one launch per call) because it leaves the control
    block clean itself -- also when the safety net ran.  Five error-feedback steps, alternating two
    workspaces, every step against the oracle."""
    n = 3_000_001
    plan = api.Plan([n], 0.01, device=0)
    plan.set_option(api.GC_OPT_WORKSPACE_PRIVATE, 1)
    for opt, value in options.items():
        plan.set_option(opt, value)
    k = plan.total_cap
    wss = [plan.alloc_workspace(), plan.alloc_workspace()]
    idx, val, cnt = plan.alloc_outputs()
    r = torch.zeros(n, device="cuda")
    r_cpu = np.zeros(n, np.float32)
    for step in range(6):
        ws = wss[step % 2]
        g = randn(n, 5000 + step)
        idx.fill_(-1); val.fill_(float("nan"))
        before = plan.launches()
        plan.compress(g.cuda(), r, idx, val, cnt, ws)
        assert plan.launches() - before == (2 if step < 2 else 1), step        # first use of a workspace: cleared once
        st, det = plan.last_status(ws)
        assert st == api.GC_OK, (step, st, det)
        oi, ov = oracle.topk_compress_tensors([n], [k], g.numpy(), r_cpu)
        assert np.array_equal(to_np_u32(idx[:k]), oi), step
        assert np.array_equal(to_np_u32(val[:k]), bits(ov)), step
        assert np.array_equal(to_np_u32(r), bits(r_cpu)), step
        if step == 3:                                  # a decode of this plan in between is fine (status word only)
            dense = torch.empty(n, device="cuda")
            plan.decompress_accumulate([idx], [val], None, dense, True, ws)


@pytest.mark.parametrize("options", [{}, {api.GC_OPT_SAMPLE_RANK_PERMILLE: 30}, {api.GC_OPT_CANDIDATE_CAPACITY: 100}],
                         ids=["plain", "starved", "overflow"])
def test_private_workspace_many_tensors_and_workers_call(options):
    """The same promise for plans of several tensors: gc_compress runs one launch per call from the
    second call on a workspace, gc_compress_workers one launch for all its workers; every step of
    every worker against the oracle, with the safety-net routes forced as well."""
    sizes = [300_000, 5, 1_500_001, 131_072, 64, 0, 131_071, 700_003, 4097, 1000]
    plan = api.Plan(sizes, 0.005, device=0)
    plan.set_option(api.GC_OPT_WORKSPACE_PRIVATE, 1)
    for opt, value in options.items():
        plan.set_option(opt, value)
    ks, n, W = plan.tensor_k(), plan.total_n, 3
    tot = sum(ks)
    workers = [GpuWorker(plan) for _ in range(W)]
    r_cpu = [np.zeros(n, np.float32) for _ in range(W)]

    def check(w, g):
        workers[w].check_status()
        oi, ov = oracle.topk_compress_tensors(sizes, ks, g.numpy(), r_cpu[w])
        assert np.array_equal(to_np_u32(workers[w].idx[:tot]), oi)
        assert np.array_equal(to_np_u32(workers[w].val[:tot]), bits(ov))
        assert np.array_equal(to_np_u32(workers[w].residual[:n]), bits(r_cpu[w]))

    for step in range(4):                              # one worker, plain calls
        g = randn(n, 7000 + step)
        before = plan.launches()
        workers[0].step(g.cuda())
        # (the plan has an empty tensor, so the counts are pre-zeroed by a memset per call)
        assert plan.launches() - before == (3 if step == 0 else 2), step
        check(0, g)
    for step in range(3):                              # all workers in one call
        gs = [randn(n, 7100 + 10 * step + w) for w in range(W)]
        before = plan.launches()
        plan.compress_workers([g.cuda() for g in gs], [wk.residual for wk in workers], [wk.idx for wk in workers],
                              [wk.val for wk in workers], [wk.count for wk in workers], [wk.ws for wk in workers])
        assert plan.launches() - before == W + (2 if step == 0 else 1), step  # workers 1 and 2 are new to the plan at first
        for w in range(W):
            check(w, gs[w])
    # a foreign write to one worker's workspace: that call reports it, the next one is exact again
    workers[1].ws.fill_(0x33)
    gs = [randn(n, 7200 + w) for w in range(W)]
    r_keep = workers[1].residual.clone()
    plan.compress_workers([g.cuda() for g in gs], [wk.residual for wk in workers], [wk.idx for wk in workers],
                          [wk.val for wk in workers], None, [wk.ws for wk in workers])
    assert plan.last_status(workers[1].ws)[0] == api.GC_E_INVALID
    assert torch.equal(workers[1].residual, r_keep)
    check(0, gs[0]); check(2, gs[2])
    gs2 = [randn(n, 7300 + w) for w in range(W)]
    plan.compress_workers([g.cuda() for g in gs2], [wk.residual for wk in workers], [wk.idx for wk in workers],
                          [wk.val for wk in workers], None, [wk.ws for wk in workers])
    for w in range(W):
        check(w, gs2[w])


def test_private_workspace_broken_promise_is_caught():
    """The caller overwrites a workspace it promised to leave alone: the next call must end at once
    with GC_E_INVALID in the device status (no barrier is entered on counters that cannot be
    trusted), and the call after that -- cleared again -- is exact."""
    n = 1_000_003
    plan = api.Plan([n], 0.01, device=0)
    plan.set_option(api.GC_OPT_WORKSPACE_PRIVATE, 1)
    k = plan.total_cap
    ws = plan.alloc_workspace()
    idx, val, cnt = plan.alloc_outputs()
    r = torch.zeros(n, device="cuda")
    r_cpu = np.zeros(n, np.float32)
    g = randn(n, 1)
    plan.compress(g.cuda(), r, idx, val, None, ws)
    assert plan.last_status(ws)[0] == api.GC_OK
    oracle.topk_compress_tensors([n], [k], g.numpy(), r_cpu)
    for fill in (0x5A, 0):                             # junk, and a zero fill (the mark is gone either way)
        ws.fill_(fill)
        r_keep = r.clone()
        plan.compress(g.cuda(), r, idx, val, None, ws)
        st, det = plan.last_status(ws)
        assert st == api.GC_E_INVALID, (fill, st, det)
        assert torch.equal(r, r_keep)                  # the kernel left before touching anything
        g2 = randn(n, 2 + fill)
        plan.compress(g2.cuda(), r, idx, val, None, ws)
        assert plan.last_status(ws)[0] == api.GC_OK
        oi, ov = oracle.topk_compress_tensors([n], [k], g2.numpy(), r_cpu)
        assert np.array_equal(to_np_u32(idx[:k]), oi) and np.array_equal(to_np_u32(r), bits(r_cpu))


def test_candidate_path_needs_no_redo_in_error_feedback_steady_state():
    """Re-using a few gradients makes unsent entries pile up just below the threshold (a cliff in
    the magnitude distribution).  The sampled threshold is an exact order statistic, so the
    candidate set must still come out large enough -- and small enough -- at every step."""
    n = 3_000_000
    base = [randn(n, 300 + s) for s in range(2)]
    grads = [base[s % 2] for s in range(10)]
    seen = []
    check_topk_against_oracle([n], 0.01, grads, expect_counters=seen.append)
    assert all(c[1] == 0 and c[2] == 0 for c in seen), seen
    k = 30_000
    assert all(k <= c[0] <= 4 * k + 600_000 for c in seen), seen


def test_sample_blind_spot_falls_back_and_stays_exact():
    """All large values sit where the sample never looks (groups that are not a multiple of the
    stride), so the sampled threshold is far too low or too high; the result must not care."""
    n = 1 << 21
    g = randn(n, 77) * 1e-3
    grp = torch.arange(n) // 4
    hidden = (grp % 64) != 0
    big = hidden & (torch.rand(n, generator=torch.Generator().manual_seed(5)) < 0.02)
    g[big] = torch.sign(g[big]) * 5.0
    for density in (0.001, 0.01, 0.03):
        check_topk_against_oracle([n], density, [g, -g, g])


def test_rejects_misaligned_and_null_buffers():
    plan = api.Plan([1024], 0.1, device=0)
    wk = GpuWorker(plan)
    g = torch.zeros(1028, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    base = dict(grad=g.data_ptr(), residual=wk.residual.data_ptr(), out_idx=wk.idx.data_ptr(),
                out_val=wk.val.data_ptr(), out_count=None, workspace=wk.ws.data_ptr(), stream=s)
    assert plan.compress_ptr(**base) == api.GC_OK
    for key, bad in (("grad", g.data_ptr() + 4), ("residual", 0), ("workspace", wk.ws.data_ptr() + 16),
                     ("out_idx", 0)):
        args = dict(base)
        args[key] = bad
        assert plan.compress_ptr(**args) == api.GC_E_INVALID
    torch.cuda.synchronize()


def test_maximum_size_properties():
    """The largest plan the ABI accepts (2^31 - 1 elements, 8.6 GB per buffer): far beyond what
    the CPU oracle can rank in a test, so the result is checked through the properties that
    define it -- exactly k pairs, ascending indices, values are bit copies of a = g + r, every
    sent magnitude key >= every unsent one with ties going to the lower index, residual = a with
    +0 at the sent indices -- all evaluated with plain torch ops on the device."""
    n = (1 << 31) - 1
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * (1 << 30):
        pytest.skip("needs about 70 GB of device memory")
    plan = api.Plan([n], 1e-4, device=0)
    k = plan.tensor_k()[0]
    assert k == oracle.k_from_density(n, 1e-4) and plan.total_n == n
    gen = torch.Generator(device="cuda").manual_seed(2024)
    g = torch.empty(n, device="cuda")
    chunk = 1 << 28
    for lo in range(0, n, chunk):
        g[lo:lo + chunk].normal_(0.0, 1.0, generator=gen)
    r = torch.zeros(n, device="cuda")
    ws = plan.alloc_workspace()
    idx, val, cnt = plan.alloc_outputs()
    for step in range(2):
        a = g + r                                           # what the fold computes (one rounded add)
        plan.compress(g, r, idx, val, cnt, ws)
        st, det = plan.last_status(ws)
        assert st == api.GC_OK, (st, det)
        assert cnt.cpu().tolist()[:2] == [k, k]
        i64 = idx[:k].to(torch.int64) & 0xFFFFFFFF
        assert bool((i64[1:] > i64[:-1]).all()) and int(i64[-1]) < n
        assert torch.equal(val[:k].view(torch.int32), a[i64].view(torch.int32))
        sent = torch.zeros(n, dtype=torch.bool, device="cuda")
        sent[i64] = True
        assert bool((r[i64].view(torch.int32) == 0).all())                  # +0.0 exactly
        assert torch.equal(r[~sent].view(torch.int32), a[~sent].view(torch.int32))
        key = a.view(torch.int32) & 0x7FFFFFFF
        t_key = int(key[i64].min())
        unsent_max = int(key[~sent].max())
        assert unsent_max <= t_key
        if unsent_max == t_key:                             # ties at the threshold: lower indices were taken
            tie = key == t_key
            last_sent_tie = int(torch.nonzero(tie & sent).max())
            first_unsent_tie = int(torch.nonzero(tie & ~sent).min())
            assert last_sent_tie < first_unsent_tie
        del a, sent, key
    torch.cuda.empty_cache()


@pytest.mark.parametrize("seed", list(range(10)))
def test_random_plans_match_the_oracle(seed):
    """Seeded random plans: tensor counts, sizes around the tile and small-tensor boundaries,
    empty tensors, misaligned offsets, densities from one in a million to one half, values on
    very different scales per tensor.  Three error-feedback steps each, bit-exact."""
    rng = np.random.default_rng(1000 + seed)
    T = int(rng.integers(1, 40))
    menu = [0, 1, 2, 3, 5, 63, 64, 1000, 4091, 4092, 4093, 4095, 4096, 4097, 8191, 8192, 8193, 12_289,
            16_384, 50_001, 131_072, 300_007, 1_048_577]
    sizes = [int(menu[int(rng.integers(0, len(menu)))]) for _ in range(T)]
    if sum(sizes) == 0:
        sizes[0] = 4097
    density = float(rng.choice([1e-6, 1e-4, 1e-3, 0.01, 0.07, 0.5]))
    n = sum(sizes)
    scales = torch.cat([torch.full((s,), float(10.0 ** rng.integers(-3, 3))) for s in sizes])
    grads = [randn(n, 5000 + 10 * seed + s) * scales for s in range(3)]
    check_topk_against_oracle(sizes, density, grads)


@pytest.mark.parametrize("sizes,density", [([3_000_001], 0.01), ([70_001], 0.001),
                                           ([300_000, 5, 1_500_001, 131_072, 64, 131_071, 4093, 0, 2_000_003], 0.001),
                                           ([5, 3, 1000, 7], 0.3)])
def test_bf16_gradient_matches_the_oracle_on_the_widened_values(sizes, density):
    """gc_compress_bf16: the gradient arrives as bfloat16, is widened exactly and folded into the
    fp32 residual; indices, values and residual must be the oracle's on the widened gradient."""
    plan = api.Plan(sizes, density, device=0)
    n, ks = plan.total_n, plan.tensor_k()
    wk = GpuWorker(plan)
    r_cpu = np.zeros(n, np.float32)
    for step in range(3):
        g16 = (randn(n, 8000 + step) * 0.37).to(torch.bfloat16)
        pad = torch.zeros(8, dtype=torch.bfloat16)
        d_g = torch.cat([g16, pad]).cuda()[:n]
        plan.compress_bf16(d_g, wk.residual, wk.idx, wk.val, wk.count, wk.ws)
        oi, ov = oracle.topk_compress_tensors(sizes, ks, g16.float().numpy(), r_cpu)
        tot = plan.total_cap
        assert np.array_equal(to_np_u32(wk.idx[:tot]), oi), step
        assert np.array_equal(to_np_u32(wk.val[:tot]), bits(ov)), step
        assert np.array_equal(to_np_u32(wk.residual[:n]), bits(r_cpu)), step
        st, det = plan.last_status(wk.ws)
        assert st == api.GC_OK, (st, det)


def test_bf16_gradient_is_refused_where_no_kernel_reads_it():
    plan = api.Plan([100_000], 0.01, device=0)
    plan.set_option(api.GC_OPT_PATH, api.GC_PATH_EXACT)
    wk = GpuWorker(plan)
    g = torch.zeros(100_000, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.GcError):
        plan.compress_bf16(g, wk.residual, wk.idx, wk.val, wk.count, wk.ws)
    thr = api.Plan([100_000], 0.01, mode=api.GC_THRESHOLD, device=0)
    wt = GpuWorker(thr)
    with pytest.raises(api.GcError):
        thr.compress_bf16(g, wt.residual, wt.idx, wt.val, wt.count, wt.ws)


@pytest.mark.parametrize("sizes", [[3_000_001], [300_000, 5, 1_500_001, 64, 131_071]])
def test_host_buffer_entry_point_with_alternating_staging_buffers(sizes):
    """gc_compress_host: pinned host gradient in, pairs back in pinned host memory.  Five
    error-feedback steps are enqueued back to back with two staging buffers and two host gradient
    buffers alternating (the copy of the next gradient overlaps the current compress); every
    step's pairs and the final residual must equal the oracle's, and so must a run with the
    per-kernel timing on (copy on the caller's stream)."""
    density = 0.01
    plan = api.Plan(sizes, density, device=0)
    n, ks = plan.total_n, plan.tensor_k()
    for profiled in (False, True):
        plan.profile_enable(256 if profiled else 0)
        ws = plan.alloc_workspace()
        idx, val, cnt = plan.alloc_outputs()
        resid = torch.zeros(n, device="cuda")
        staging = [torch.empty(n, device="cuda") for _ in range(2)]
        steps = 5
        host_g = [torch.randn(n, generator=torch.Generator().manual_seed(90 + s)).pin_memory() for s in range(steps)]
        host_idx = [torch.empty(plan.total_cap, dtype=torch.int32).pin_memory() for _ in range(steps)]
        host_val = [torch.empty(plan.total_cap, dtype=torch.float32).pin_memory() for _ in range(steps)]
        for s in range(steps):
            plan.compress_host(host_g[s], staging[s % 2], resid, idx, val, None, host_idx[s], host_val[s], ws)
        torch.cuda.synchronize()
        r_cpu = np.zeros(n, np.float32)
        for s in range(steps):
            oi, ov = oracle.topk_compress_tensors(sizes, ks, host_g[s].numpy(), r_cpu)
            assert np.array_equal(host_idx[s].numpy().view(np.uint32), oi), (profiled, s)
            assert np.array_equal(host_val[s].numpy().view(np.uint32), ov.view(np.uint32)), (profiled, s)
        assert np.array_equal(resid.cpu().numpy().view(np.uint32), r_cpu.view(np.uint32)), profiled
        st, det = plan.last_status(ws)
        assert st == api.GC_OK, (st, det)
    plan.profile_enable(0)


@pytest.mark.parametrize("mode", [api.GC_TOPK, api.GC_THRESHOLD], ids=["topk", "threshold"])
def test_private_workspaces_under_changing_call_patterns(mode):
    """Sixty steps on private workspaces that are served in turn by one gc_compress_workers call,
    by one gc_compress call per worker, and by a two-worker call plus single calls, with a decode on
    one of the workspaces in between, quantised (tie-heavy) gradients every fifth step and thirty
    times larger ones every seventh: every step bit-equal to a second plan that clears its one
    shared workspace before every call (that plan's route is what the tests above hold against
    the oracle)."""
    rng = np.random.default_rng(11)
    sizes = [int(rng.integers(1, 200_000)) for _ in range(30)] + [5, 0, 4096, 4097]
    W, n = 5, None
    pa = api.Plan(sizes, 0.004, mode=mode, device=0)
    pa.set_option(api.GC_OPT_WORKSPACE_PRIVATE, 1)
    pb = api.Plan(sizes, 0.004, mode=mode, device=0)
    n = pa.total_n
    wa, wsb = [GpuWorker(pa) for _ in range(W)], pb.alloc_workspace()
    wb = [GpuWorker(pb) for _ in range(W)]
    da, db = torch.empty(n, device="cuda"), torch.empty(n, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(5)
    scale = torch.rand(n, device="cuda", generator=gen) * 2 + 0.01
    for s in range(60):
        g = [torch.randn(n, device="cuda", generator=gen) * scale * (1.0 if s % 7 else 30.0) for _ in range(W)]
        if s % 5 == 3:
            g = [torch.round(x * 4) / 4 for x in g]
        for wk in wa + wb:
            wk.idx.fill_(-1); wk.val.fill_(float("nan"))
        first = 0 if s % 3 == 0 else (W if s % 3 == 1 else 2)      # workers served by the shared call
        if first:
            pa.compress_workers(g[:first] if first < W else g, [wk.residual for wk in wa[:first]],
                                [wk.idx for wk in wa[:first]], [wk.val for wk in wa[:first]],
                                [wk.count for wk in wa[:first]], [wk.ws for wk in wa[:first]])
        for w in range(first, W):
            pa.compress(g[w], wa[w].residual, wa[w].idx, wa[w].val, wa[w].count, wa[w].ws)
        for w in range(W):
            pb.compress(g[w], wb[w].residual, wb[w].idx, wb[w].val, wb[w].count, wsb)
        pa.decompress_accumulate([wk.idx for wk in wa], [wk.val for wk in wa], [wk.count for wk in wa], da, True,
                                 wa[s % W].ws)
        pb.decompress_accumulate([wk.idx for wk in wb], [wk.val for wk in wb], [wk.count for wk in wb], db, True, wsb)
        for w in range(W):
            assert pa.last_status(wa[w].ws)[0] >= 0, (s, w)
            assert torch.equal(wa[w].count, wb[w].count), (s, w)
            assert torch.equal(wa[w].idx, wb[w].idx), (s, w)
            assert torch.equal(wa[w].val.view(torch.int32), wb[w].val.view(torch.int32)), (s, w)
            assert torch.equal(wa[w].residual.view(torch.int32), wb[w].residual.view(torch.int32)), (s, w)
        assert torch.equal(da.view(torch.int32), db.view(torch.int32)), s


@pytest.mark.parametrize("tiles", [296, 297, 593, 2999, 3000, 3001])
def test_one_tensor_plans_around_the_grid_rule(tiles):
    """One-tensor plans of up to 3000 tiles run on two CTAs per SM, larger ones on three: sizes on
    both sides of that rule and where a CTA's share of tiles changes (296 CTAs), with a ragged
    last tile, two steps each against the oracle."""
    n = tiles * 4096 - 5
    check_topk_against_oracle([n], 0.004, [randn(n, 9100 + tiles), randn(n, 9200 + tiles)])


def test_calls_on_a_side_stream():
    """Every call enqueues on the stream it is given and on no other: compress, the workers call,
    decode and the fused optimizer step on a non-blocking side stream that is held back by a
    long-running kernel, while the default stream stays idle; the results are read after the
    side stream alone has been waited for, and compared with the oracle."""
    sizes = [250_000, 0, 7, 1_200_003, 4096, 66_000]
    plan = api.Plan(sizes, 0.004, device=0)
    ks, n, W = plan.tensor_k(), plan.total_n, 3
    tot = sum(ks)
    workers = [GpuWorker(plan) for _ in range(W)]
    gs = [randn(n, 9500 + w) for w in range(W)]
    gd = [g.cuda() for g in gs]
    dense = torch.empty(n, device="cuda")
    param, vel = torch.ones(n, device="cuda"), torch.zeros(n, device="cuda")
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        torch.cuda._sleep(20_000_000)                       # about 10 ms: everything below queues up behind it
        plan.compress(gd[0], workers[0].residual, workers[0].idx, workers[0].val, workers[0].count, workers[0].ws, side)
        plan.compress_workers(gd[1:], [wk.residual for wk in workers[1:]], [wk.idx for wk in workers[1:]],
                              [wk.val for wk in workers[1:]], [wk.count for wk in workers[1:]],
                              [wk.ws for wk in workers[1:]], side)
        plan.decompress_accumulate([wk.idx for wk in workers], [wk.val for wk in workers], None, dense, True,
                                   workers[0].ws, side)
        plan.decompress_apply_momentum([wk.idx for wk in workers], [wk.val for wk in workers], None, param, vel,
                                       0.1, 0.9, 0.5, workers[0].ws, side)
    side.synchronize()
    lists = []
    for w in range(W):
        r_cpu = np.zeros(n, np.float32)
        oi, ov = oracle.topk_compress_tensors(sizes, ks, gs[w].numpy(), r_cpu)
        assert np.array_equal(to_np_u32(workers[w].idx[:tot]), oi), w
        assert np.array_equal(to_np_u32(workers[w].val[:tot]), bits(ov)), w
        assert np.array_equal(to_np_u32(workers[w].residual[:n]), bits(r_cpu)), w
        lists.append((oi, ov))
    want = oracle.decode_accumulate(lists, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(dense), bits(want))
    p_cpu, v_cpu = np.ones(n, np.float32), np.zeros(n, np.float32)
    oracle.decode_apply_momentum(lists, p_cpu, v_cpu, 0.1, 0.9, 0.5)
    assert np.array_equal(to_np_u32(param), bits(p_cpu)) and np.array_equal(to_np_u32(vel), bits(v_cpu))


@pytest.mark.parametrize("sizes", [[1_300_001], [200_000, 3, 0, 900_001, 4096]], ids=["one", "many"])
def test_step_captured_in_a_cuda_graph(sizes):
    """A compress + decode step captured once in a CUDA graph (cooperative launch included) and
    replayed on fresh gradients copied into the captured buffer: every replay against the oracle.
    The workspace is private and warmed, so the captured step holds no clearing launch."""
    plan = api.Plan(sizes, 0.005, device=0)
    plan.set_option(api.GC_OPT_WORKSPACE_PRIVATE, 1)
    ks, n = plan.tensor_k(), plan.total_n
    tot = sum(ks)
    wk = GpuWorker(plan)
    g_dev = torch.zeros(n, device="cuda")
    dense = torch.empty(n, device="cuda")
    side = torch.cuda.Stream()
    r_cpu = np.zeros(n, np.float32)

    def step():
        plan.compress(g_dev, wk.residual, wk.idx, wk.val, wk.count, wk.ws, side)
        plan.decompress_accumulate([wk.idx], [wk.val], None, dense, True, wk.ws, side)

    def check(g):
        oi, ov = oracle.topk_compress_tensors(sizes, ks, g.numpy(), r_cpu)
        assert np.array_equal(to_np_u32(wk.idx[:tot]), oi)
        assert np.array_equal(to_np_u32(wk.val[:tot]), bits(ov))
        assert np.array_equal(to_np_u32(wk.residual[:n]), bits(r_cpu))
        assert np.array_equal(to_np_u32(dense), bits(oracle.decode_accumulate([(oi, ov)], np.empty(n, np.float32), True)))

    g0 = randn(n, 9600)
    g_dev.copy_(g0.cuda())
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        step()                                              # warm: clears once, leaves the workspace clean
    side.synchronize()
    check(g0)
    graph = torch.cuda.CUDAGraph()
    before = plan.launches()
    with torch.cuda.graph(graph, stream=side):
        step()
    assert plan.launches() - before == (2 if len(sizes) == 1 else 3)    # (many: the plan has an empty tensor, counts pre-zeroed)
    for i in range(3):
        g = randn(n, 9601 + i)
        g_dev.copy_(g.cuda())
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert plan.last_status(wk.ws)[0] == api.GC_OK
        check(g)
