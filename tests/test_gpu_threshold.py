"""GPU parity of the threshold-estimation variant (GC_THRESHOLD) against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2104_01981_b200 import api, build, synth
from helpers import GpuWorker, bits, same_f32_bits, to_np_u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    api.lib()


def randn(n, seed, scale=1.0):
    return torch.randn(n, generator=torch.Generator().manual_seed(seed)) * scale


def check_threshold(sizes, density, grads, stride=0, cap_factor=0.0, expect_truncated=None):
    plan = api.Plan(sizes, density, mode=api.GC_THRESHOLD, device=0, sample_stride=stride,
                    cap_factor=cap_factor)
    w = GpuWorker(plan)
    T = len(sizes)
    caps, offs = plan.tensor_cap(), plan.tensor_out_offset()
    strides = [plan.query(api.GC_Q_TENSOR_STRIDE, t) for t in range(T)]
    n = plan.total_n
    r_cpu = np.zeros(n, np.float32)
    for step, g in enumerate(grads):
        gd = g.cuda()
        if gd.numel() < 4:
            gd = torch.cat([gd, torch.zeros(4 - gd.numel(), device="cuda")])
        w.step(gd)
        st, det = plan.last_status(w.ws)
        g_cpu = g.numpy()
        cnt = w.count.cpu().numpy()
        gi, gv = to_np_u32(w.idx), to_np_u32(w.val)
        off, truncated = 0, False
        for t, sz in enumerate(sizes):
            oi, ov, hits, tau = oracle.threshold_compress(g_cpu[off:off + sz], r_cpu[off:off + sz], density,
                                                          strides[t], caps[t], index_base=off)
            assert cnt[t] == oi.size and cnt[T + t] == hits, (step, t, cnt[t], oi.size, cnt[T + t], hits)
            assert np.array_equal(gi[offs[t]:offs[t] + oi.size], oi), (step, t)
            assert same_f32_bits(gv[offs[t]:offs[t] + oi.size], bits(ov)), (step, t)
            truncated |= hits > caps[t]
            off += sz
        assert same_f32_bits(to_np_u32(w.residual[:n]), bits(r_cpu)), f"step {step}: residual differs"
        assert st == (api.GC_W_TRUNCATED if truncated else api.GC_OK), (st, det)
        if expect_truncated is not None:
            assert truncated == expect_truncated
    return plan, w


@pytest.mark.parametrize("n", [1, 3, 4, 5, 33, 1025, 8193, 65536, 65537, 100_003, (1 << 20) + 1])
@pytest.mark.parametrize("density", [0.001, 0.05])
def test_threshold_single_tensor_sizes(n, density):
    check_threshold([n], density, [randn(n, 3 * n + s) for s in range(2)])


@pytest.mark.parametrize("stride,cap_factor", [(0, 0.0), (1, 1.0), (3, 1.5), (16, 4.0), (64, 1.0)])
def test_threshold_many_ragged_tensors(stride, cap_factor):
    sizes = [5, 3, 1000, 7, 8193, 64, 1, 0, 2, 70_001, 300_000, 0, 6, 131_073]
    n = sum(sizes)
    check_threshold(sizes, 0.01, [randn(n, 500 + s) for s in range(3)], stride=stride, cap_factor=cap_factor)


def test_threshold_truncation_keeps_a_prefix():
    # the sample (stride 64) only sees tiny values, so nearly everything is a hit and the
    # capacity cuts it to the first `cap` in index order
    n = 400_000
    g = randn(n, 8)
    grp = torch.arange(n) // 4
    g[(grp % 64) == 0] *= 1e-3
    check_threshold([n], 0.01, [g, g], expect_truncated=True)


def test_threshold_ties_at_tau():
    n = 300_000
    g = synth.quantised_gradient(n, 21)
    check_threshold([n, n // 3], 0.02, [torch.cat([g, g[:n // 3]])] * 2, cap_factor=8.0)


def test_threshold_config4_resnet_workers_and_decode():
    w = synth.workload(3)
    plan = api.Plan(w.sizes, w.density, mode=api.GC_THRESHOLD, device=0)
    T, n = len(w.sizes), plan.total_n
    caps, offs = plan.tensor_cap(), plan.tensor_out_offset()
    strides = [plan.query(api.GC_Q_TENSOR_STRIDE, t) for t in range(T)]
    assert w.workers == 8
    workers, pairs = [GpuWorker(plan) for _ in range(w.workers)], []
    for i, wk in enumerate(workers):
        g = synth.gradient(w, i, 0, device="cuda")
        wk.step(g)
        g_cpu, r_cpu = g.cpu().numpy(), np.zeros(n, np.float32)
        cnt, gi, gv = wk.count.cpu().numpy(), to_np_u32(wk.idx), to_np_u32(wk.val)
        off, all_i, all_v = 0, [], []
        for t, sz in enumerate(w.sizes):
            oi, ov, hits, _ = oracle.threshold_compress(g_cpu[off:off + sz], r_cpu[off:off + sz], w.density,
                                                        strides[t], caps[t], index_base=off)
            assert cnt[t] == oi.size and cnt[T + t] == hits
            assert np.array_equal(gi[offs[t]:offs[t] + oi.size], oi)
            assert np.array_equal(gv[offs[t]:offs[t] + oi.size], bits(ov))
            all_i.append(oi); all_v.append(ov)
            off += sz
        assert np.array_equal(to_np_u32(wk.residual[:n]), bits(r_cpu))
        pairs.append((np.concatenate(all_i), np.concatenate(all_v)))
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate([x.idx for x in workers], [x.val for x in workers], [x.count for x in workers],
                               out, True, workers[0].ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))


def check_threshold_workers(sizes, density, W, grads_fn, steps=2, cap_factor=0.0):
    """`steps` gc_compress_workers calls of a threshold plan for W workers; every worker's pairs,
    counts, residual and status against the oracle after every step."""
    plan = api.Plan(sizes, density, mode=api.GC_THRESHOLD, device=0, cap_factor=cap_factor)
    T, n = len(sizes), plan.total_n
    caps, offs = plan.tensor_cap(), plan.tensor_out_offset()
    strides = [plan.query(api.GC_Q_TENSOR_STRIDE, t) for t in range(T)]
    workers = [GpuWorker(plan) for _ in range(W)]
    r_cpu = [np.zeros(n, np.float32) for _ in range(W)]
    for step in range(steps):
        grads = [grads_fn(w, step) for w in range(W)]
        for wk in workers:
            wk.idx.fill_(-1); wk.val.fill_(float("nan")); wk.count.fill_(-1)
        plan.compress_workers([g.cuda() for g in grads], [wk.residual for wk in workers], [wk.idx for wk in workers],
                              [wk.val for wk in workers], [wk.count for wk in workers], [wk.ws for wk in workers])
        for w, wk in enumerate(workers):
            st, det = plan.last_status(wk.ws)
            g_cpu = grads[w].cpu().numpy()
            cnt, gi, gv = wk.count.cpu().numpy(), to_np_u32(wk.idx), to_np_u32(wk.val)
            off, truncated = 0, False
            for t, sz in enumerate(sizes):
                oi, ov, hits, _ = oracle.threshold_compress(g_cpu[off:off + sz], r_cpu[w][off:off + sz], density,
                                                            strides[t], caps[t], index_base=off)
                assert cnt[t] == oi.size and cnt[T + t] == hits, (step, w, t)
                assert np.array_equal(gi[offs[t]:offs[t] + oi.size], oi), (step, w, t)
                assert same_f32_bits(gv[offs[t]:offs[t] + oi.size], bits(ov)), (step, w, t)
                truncated |= hits > caps[t]
                off += sz
            assert same_f32_bits(to_np_u32(wk.residual[:n]), bits(r_cpu[w])), (step, w)
            assert st == (api.GC_W_TRUNCATED if truncated else api.GC_OK), (st, det)
    return plan, workers


@pytest.mark.parametrize("W", [2, 5, 8, 13])
def test_threshold_workers_call_matches_the_oracle(W):
    """gc_compress_workers in threshold mode on a plan of several tensors: the workers share
    cooperative launches (groups of CTAs), each exactly as a call of its own; a tight capacity
    factor makes some workers truncate."""
    sizes = [300_000, 5, 1_500_001, 131_072, 64, 0, 131_071, 700_003, 4097, 1000]
    n = sum(sizes)
    check_threshold_workers(sizes, 0.004, W, lambda w, s: randn(n, 9000 + 50 * w + s, 10.0 ** (w % 3 - 1)),
                            steps=2, cap_factor=1.0)


def test_threshold_workers_call_on_the_resnet_workload():
    w = synth.workload(3)
    check_threshold_workers(w.sizes, w.density, w.workers, lambda wk, s: synth.gradient(w, wk, s, device="cuda"), steps=2)


@pytest.mark.parametrize("config_id", [2, 4], ids=["bert_110m", "gpt2_medium_355m"])
def test_threshold_full_size_one_tensor_workloads(config_id):
    """One full-size step of the threshold variant on the 110M- and the 355M-element workload (the
    one-tensor kernel at the sizes the benchmark quotes it on), then the decode of that list by
    its count against the oracle."""
    w = synth.workload(config_id)
    g = synth.gradient(w, 0, 0, device="cuda")
    plan, wk = check_threshold(w.sizes, w.density, [g.cpu()])
    del g
    n = plan.total_n
    m = int(wk.count[0].item())
    pairs = [(to_np_u32(wk.idx[:m]), wk.val[:m].cpu().numpy())]
    wk.residual = None
    torch.cuda.empty_cache()
    out = torch.empty(n, device="cuda")
    plan.decompress_accumulate([wk.idx], [wk.val], [wk.count], out, True, wk.ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert np.array_equal(to_np_u32(out), bits(want))


def test_threshold_one_tensor_mild_truncation_and_two_valued_input():
    """One large tensor (the fused one-tensor kernel).  cap_factor 1.0: the hits exceed the
    capacity by a little in some steps, so the kernel itself cuts the tail and puts those
    values back.  Two-valued input: tens of thousands of sampled keys are equal to tau (the
    8192-bin route of the sample select) and every element is a hit (the hit list overflows,
    the look-back pass takes over)."""
    n = 2_000_003
    grads = [randn(n, 900 + s) for s in range(4)]
    check_threshold([n], 0.01, grads, cap_factor=1.0)
    check_threshold([n], 0.02, grads[:2], stride=16, cap_factor=1.25)
    g = torch.ones(n)
    g[torch.rand(n, generator=torch.Generator().manual_seed(3)) < 0.1] = -3.0
    check_threshold([n], 0.5, [g, g])
    check_threshold([n], 0.05, [g])


def test_threshold_many_tensors_hit_list_overflow_and_truncation():
    """Several tensors in one plan (the fused many-tensor kernel).  In the large ones the sample
    only sees tiny values, so nearly every element is a hit: the hit list overflows, the
    look-back pass takes over (leaving the single-tile tensors, which are already done, alone),
    and the capacity cuts every large tensor to a prefix."""
    sizes = [70_001, 5, 300_000, 1000, 64, 131_073, 4092, 4093, 0, 9000]
    n = sum(sizes)
    g = randn(n, 77)
    off = 0
    for sz in sizes:
        if sz > 65536:                      # stride 64 applies (smaller tensors are sampled in full)
            loc = torch.arange(sz)
            g[off:off + sz][((loc >> 2) % 64) == 0] *= 1e-3
        off += sz
    check_threshold(sizes, 0.01, [g, g], expect_truncated=True)
    # the same plan on ordinary data: no overflow, mild or no truncation
    check_threshold(sizes, 0.01, [randn(n, 78 + s) for s in range(3)], cap_factor=1.0)


@pytest.mark.parametrize("seed", list(range(6)))
def test_threshold_random_plans_match_the_oracle(seed):
    """Seeded random plans for the threshold variant (sizes around the tile boundaries, empty
    tensors, misaligned offsets, several densities, strides and capacity factors)."""
    rng = np.random.default_rng(2000 + seed)
    T = int(rng.integers(1, 30))
    menu = [0, 1, 2, 5, 64, 1000, 4092, 4093, 4096, 4097, 8193, 16_384, 65_536, 65_537, 131_072, 300_007, 1_048_577]
    sizes = [int(menu[int(rng.integers(0, len(menu)))]) for _ in range(T)]
    if sum(sizes) == 0:
        sizes[0] = 4097
    density = float(rng.choice([1e-4, 1e-3, 0.01, 0.07]))
    stride = int(rng.choice([0, 1, 7, 64]))
    cap_factor = float(rng.choice([0.0, 1.0, 1.5, 3.0]))
    n = sum(sizes)
    scales = torch.cat([torch.full((s,), float(10.0 ** rng.integers(-2, 2))) for s in sizes])
    grads = [randn(n, 6000 + 10 * seed + s) * scales for s in range(2)]
    check_threshold(sizes, density, grads, stride=stride, cap_factor=cap_factor)


@pytest.mark.parametrize("tiles", [296, 297, 2500, 2501])
def test_threshold_one_tensor_plans_around_the_grid_rule(tiles):
    """The one-tensor threshold kernel runs on two CTAs per SM up to 2500 tiles and on three beyond:
    both sides of the rule and of the 296-CTA grid, ragged last tile, two steps against the oracle."""
    n = tiles * 4096 - 7
    check_threshold([n], 0.004, [randn(n, 9300 + tiles), randn(n, 9400 + tiles)])
