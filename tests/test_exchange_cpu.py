"""The exchange step of the multi-GPU path on two gloo ranks on CPU: block layout, one
all-gather of fixed-size blocks, worker order = rank order.  The sparse sets and the decode
come from the CPU oracle here; the GPU tests run the same object against the CUDA library."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SIZES, DENSITY = [5, 7001, 4096, 64, 12345], 0.01


def _rank_grad(rank: int, n: int) -> np.ndarray:
    rng = np.random.default_rng(1234 + rank)
    return (rng.standard_t(3, n) * 0.02).astype(np.float32)


def _rank_pairs(rank: int, ks):
    import oracle
    n = sum(SIZES)
    r = np.zeros(n, np.float32)
    return oracle.topk_compress_tensors(SIZES, ks, _rank_grad(rank, n), r)


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2104_01981_b200 import api, exchange
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    try:
        plan = api.Plan(SIZES, DENSITY, device=-1)              # host-only plan: sizes and capacities
        ks = plan.tensor_k()
        ex = exchange.PairExchange(plan.total_cap, plan.n_tensors, False, "cpu")
        assert ex.world == world and ex.rank == rank
        oi, ov = _rank_pairs(rank, ks)
        idx, val, cnt = ex.outputs()
        idx.copy_(torch.from_numpy(oi.view(np.int32)))
        val.copy_(torch.from_numpy(ov))
        cnt[:len(ks)].copy_(torch.tensor(ks, dtype=torch.int32))
        ex.all_gather()
        li, lv, lc = ex.lists()
        assert lc is None and len(li) == world
        pairs = [(li[r].numpy().view(np.uint32), lv[r].numpy()) for r in range(world)]
        dense = oracle.decode_accumulate(pairs, np.empty(plan.total_n, np.float32), True)
        np.save(os.path.join(out_dir, f"dense{rank}.npy"), dense)
        np.save(os.path.join(out_dir, f"recv{rank}.npy"), ex.recv.numpy())
        assert ex.bytes_on_wire_per_rank() == 4 * ex.layout.words * (world - 1)
    finally:
        torch.distributed.destroy_process_group()


def test_two_gloo_ranks_gather_blocks_in_rank_order_and_agree(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2104_01981_b200 import api
    port = 31000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    plan = api.Plan(SIZES, DENSITY, device=-1)
    ks = plan.tensor_k()
    pairs = [_rank_pairs(r, ks) for r in range(2)]
    want = oracle.decode_accumulate(pairs, np.empty(plan.total_n, np.float32), True)
    d0, d1 = np.load(tmp_path / "dense0.npy"), np.load(tmp_path / "dense1.npy")
    assert np.array_equal(d0.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(d1.view(np.uint32), want.view(np.uint32))          # every rank ends with the same bits
    assert np.array_equal(np.load(tmp_path / "recv0.npy"), np.load(tmp_path / "recv1.npy"))


def test_block_layout_sections_are_16_byte_aligned_and_disjoint():
    sys.path.insert(0, ROOT)
    from paper_2104_01981_b200 import exchange
    for cap, T in [(0, 1), (1, 1), (5, 3), (4096, 161), (1094823, 1)]:
        L = exchange.BlockLayout(cap, T)
        assert L.off_val % 4 == 0 and L.off_cnt % 4 == 0 and L.words % 4 == 0
        assert L.off_val >= max(cap, 1) and L.off_cnt >= L.off_val + max(cap, 1)
        assert L.words >= L.off_cnt + max(2 * T, 1)
        block = torch.arange(L.words, dtype=torch.int32)
        idx, val, cnt = L.views(block)
        assert idx.numel() == max(cap, 1) and val.numel() == max(cap, 1) and cnt.numel() == max(2 * T, 1)
        assert idx.data_ptr() % 16 == val.data_ptr() % 16 == cnt.data_ptr() % 16 == block.data_ptr() % 16
        assert val.dtype == torch.float32 and int(cnt[0]) == L.off_cnt


def test_single_process_exchange_is_a_copy():
    sys.path.insert(0, ROOT)
    from paper_2104_01981_b200 import exchange
    ex = exchange.PairExchange(10, 2, True, "cpu")
    ex.send.copy_(torch.arange(ex.layout.words, dtype=torch.int32))
    ex.all_gather()
    assert torch.equal(ex.recv, ex.send)
    li, lv, lc = ex.lists()
    assert len(li) == 1 and lc is not None and lc[0].numel() == 4
