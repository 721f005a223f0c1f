"""GPU parity of the multi-GPU aggregation path (compress into the exchange block, all-gather,
decode over the gathered lists) against the CPU oracle.  One GPU is available to the tests, so
(a) a one-rank NCCL group runs the real collective and (b) R ranks are emulated by R compress
calls whose blocks are laid side by side exactly as the all-gather lays them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_01981_b200 import api, build, exchange, synth
from helpers import bits, same_f32_bits, to_np_u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    api.lib()


def _grad(n, seed):
    gen = torch.Generator().manual_seed(seed)
    return torch.randn(n, generator=gen)


def _emulated_ranks(plan, R, seed, steps=2):
    """R ranks on one GPU: every rank owns a residual and a send block; returns the exchange
    object holding the gathered blocks, and the CPU copies of the gradients and residuals."""
    n = plan.total_n
    ws = plan.alloc_workspace()
    ranks = [exchange.PairExchange.for_plan(plan) for _ in range(R)]
    resid = [torch.zeros(n, device="cuda") for _ in range(R)]
    r_cpu = [np.zeros(n, np.float32) for _ in range(R)]
    g_cpu = []
    for r, ex in enumerate(ranks):
        for s in range(steps):
            g = _grad(n, seed + 100 * r + s)
            oi, ov, oc = ex.outputs()
            oi.fill_(-1); ov.fill_(float("nan"))
            plan.compress(g.cuda(), resid[r], oi, ov, oc, ws)
            g_cpu.append((r, s, g.numpy()))
    gathered = exchange.PairExchange.for_plan(plan)
    gathered.world = R
    gathered.recv = torch.cat([ex.send for ex in ranks])
    return gathered, ranks, g_cpu, resid, ws


@pytest.mark.parametrize("sizes,density", [([300_001], 0.01), ([5, 3, 1000, 7, 8193, 64, 70_001], 0.02)])
@pytest.mark.parametrize("R", [1, 3, 8])
def test_emulated_ranks_topk_gather_then_decode(sizes, density, R):
    plan = api.Plan(sizes, density, device=0)
    n, ks = plan.total_n, plan.tensor_k()
    gathered, ranks, g_cpu, resid, ws = _emulated_ranks(plan, R, seed=11)
    # oracle: the same two steps per rank, then the rank-ordered sum of the last step's sets
    pairs = []
    for r in range(R):
        rc = np.zeros(n, np.float32)
        for (rr, s, g) in g_cpu:
            if rr == r:
                oi, ov = oracle.topk_compress_tensors(sizes, ks, g, rc)
        pairs.append((oi, ov))
        assert same_f32_bits(to_np_u32(resid[r]), bits(rc))
    li, lv, lc = gathered.lists()
    assert lc is None
    for r in range(R):
        assert np.array_equal(to_np_u32(li[r])[:plan.total_cap], pairs[r][0])
        assert same_f32_bits(to_np_u32(lv[r])[:plan.total_cap], bits(pairs[r][1]))
    dense = torch.full((n,), 3.0, device="cuda")
    gathered.decode(plan, dense, True, ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert same_f32_bits(to_np_u32(dense), bits(want))
    # the optimizer step fused behind the same gathered lists
    gen = torch.Generator().manual_seed(5)
    p0, v0 = torch.randn(n, generator=gen), torch.randn(n, generator=gen) * 0.1
    p, v = p0.cuda(), v0.cuda()
    gathered.decode_apply_momentum(plan, p, v, 0.05, 0.9, 1.0 / R, ws)
    pc, vc = p0.numpy().copy(), v0.numpy().copy()
    oracle.decode_apply_momentum(pairs, pc, vc, 0.05, 0.9, 1.0 / R)
    assert same_f32_bits(to_np_u32(p), bits(pc)) and same_f32_bits(to_np_u32(v), bits(vc))
    st, det = plan.last_status(ws)
    assert st == api.GC_OK, (st, det)


@pytest.mark.parametrize("sizes", [[200_003], [5, 1000, 8193, 0, 70_001, 64]])
def test_emulated_ranks_threshold_counts_travel_in_the_block(sizes):
    density, R = 0.01, 3
    plan = api.Plan(sizes, density, mode=api.GC_THRESHOLD, device=0)
    n, T = plan.total_n, len(sizes)
    caps, offs = plan.tensor_cap(), plan.tensor_out_offset()
    strides = [plan.query(api.GC_Q_TENSOR_STRIDE, t) for t in range(T)]
    gathered, ranks, g_cpu, resid, ws = _emulated_ranks(plan, R, seed=23, steps=1)
    li, lv, lc = gathered.lists()
    assert lc is not None
    pairs = []
    for r in range(R):
        g = [x for (rr, s, x) in g_cpu if rr == r][0]
        rc = np.zeros(n, np.float32)
        oi_all, ov_all, off = [], [], 0
        cnt = lc[r].cpu().numpy()
        for t, sz in enumerate(sizes):
            oi, ov, hits, _ = oracle.threshold_compress(g[off:off + sz], rc[off:off + sz], density, strides[t],
                                                        caps[t], index_base=off)
            assert cnt[t] == oi.size
            assert np.array_equal(to_np_u32(li[r])[offs[t]:offs[t] + oi.size], oi)
            oi_all.append(oi); ov_all.append(ov)
            off += sz
        pairs.append((np.concatenate(oi_all), np.concatenate(ov_all)))
    dense = torch.full((n,), 3.0, device="cuda") if n else torch.zeros(4, device="cuda")
    gathered.decode(plan, dense, True, ws)
    want = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    assert same_f32_bits(to_np_u32(dense)[:n], bits(want))


def test_one_rank_nccl_group_runs_the_collective(tmp_path):
    """The real collective on the one GPU there is: a one-rank NCCL group."""
    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method=f"file://{tmp_path}/rendezvous", rank=0, world_size=1,
                            device_id=torch.device("cuda:0"))
    try:
        sizes, density = [5, 70_001, 8193, 64], 0.01
        plan = api.Plan(sizes, density, device=0)
        n, ks = plan.total_n, plan.tensor_k()
        ex = exchange.PairExchange.for_plan(plan)
        assert ex.world == 1 and ex.bytes_on_wire_per_rank() == 0
        ws = plan.alloc_workspace()
        r, rc = torch.zeros(n, device="cuda"), np.zeros(n, np.float32)
        dense = torch.empty(n, device="cuda")
        for s in range(2):
            g = _grad(n, 77 + s)
            oi, ov, oc = ex.outputs()
            plan.compress(g.cuda(), r, oi, ov, oc, ws)
            ex.all_gather()
            ex.decode(plan, dense, True, ws)
            wi, wv = oracle.topk_compress_tensors(sizes, ks, g.numpy(), rc)
            want = oracle.decode_accumulate([(wi, wv)], np.empty(n, np.float32), True)
            assert same_f32_bits(to_np_u32(dense), bits(want))
    finally:
        dist.destroy_process_group()
