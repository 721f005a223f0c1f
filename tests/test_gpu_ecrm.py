"""GPU parity of the erasure-coded embedding-table kernels against the CPU oracle, through the
C ABI: bit-exact for every operation (fixed order, one rounding per operation)."""
import numpy as np
import pytest
import torch

from oracle import ecrm_oracle as eo
from paper_2104_01981_b200 import build, ecrm, synth
from helpers import bits, to_np_u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    ecrm.lib()


def same(dev: torch.Tensor, ref: np.ndarray) -> bool:
    return np.array_equal(to_np_u32(dev.reshape(-1)), bits(ref.reshape(-1)))


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 8, 9, 32])
@pytest.mark.parametrize("n", [1, 3, 4, 1000, 4099, 1 << 20, (1 << 22) + 7])
def test_encode_decode_match_oracle_bitwise(k, n):
    if k == 32 and n > (1 << 20):
        pytest.skip("covered by the smaller sizes")
    gen = torch.Generator().manual_seed(k * 1000 + n % 977)
    shards = [torch.randn(n, generator=gen) * (10.0 ** (s % 3 - 1)) for s in range(k)]
    d_shards = [s.cuda() for s in shards]
    parity = torch.full((n + 4,), 7.0, device="cuda")
    ecrm.encode(d_shards, parity[:n])
    want = eo.encode([s.numpy() for s in shards])
    assert same(parity[:n], want) and parity[n:].eq(7.0).all()
    for lost in sorted({0, k // 2, k - 1}):
        out = torch.empty(n, device="cuda")
        others = [s for i, s in enumerate(d_shards) if i != lost]
        ecrm.decode(others, parity[:n], out)
        assert same(out, eo.decode(want, [s.numpy() for i, s in enumerate(shards) if i != lost]))
    # recovery in place (out aliases the parity)
    work = parity[:n].clone()
    ecrm.decode(d_shards[1:], work, work)
    assert same(work, eo.decode(want, [s.numpy() for s in shards[1:]]))


@pytest.mark.parametrize("optimizer,lr,hyper", [(ecrm.ECRM_ADAGRAD, 0.05, 1e-8), (ecrm.ECRM_MOMENTUM, 0.01, 0.9)])
@pytest.mark.parametrize("n_rows,p_rows,m,dim", [(1, 1, 1, 4), (100, 40, 30, 128), (5000, 1300, 1237, 128),
                                                 (999, 333, 333, 132), (200_000, 50_000, 20_000, 128)])
def test_fused_rows_step_and_parity_match_oracle_bitwise(optimizer, lr, hyper, n_rows, p_rows, m, dim):
    """The optimizer step with the parity update fused behind it (data shard and parity shard on
    one GPU): entry, state, parity entry and parity state after three steps equal the oracle's
    step followed by its parity update, bit for bit; rows out of range are skipped and counted."""
    entry = synth.ecrm_tables(n_rows, dim, 1, seed=n_rows + dim)[0]
    state = torch.zeros(n_rows, dim)
    p_entry, p_state = synth.ecrm_tables(p_rows, dim, 1, seed=7)[0] * 3.0, torch.zeros(p_rows, dim)
    d = [t.cuda() for t in (entry, state, p_entry, p_state)]
    h = [t.numpy().copy() for t in (entry, state, p_entry, p_state)]
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(m)
    for step in range(3):
        rows, g = synth.ecrm_batch(n_rows, m, dim, seed=100 * step + m)
        prow = torch.from_numpy(rng.permutation(p_rows)[:m].astype(np.uint32).view(np.int32))   # distinct parity rows
        ecrm.rows_step_parity(optimizer, rows.cuda(), prow.cuda(), g.cuda(), d[0], d[1], d[2], d[3], lr, hyper, bad)
        rows_np, prow_np = rows.numpy().view(np.uint32), prow.numpy().view(np.uint32)
        wde, wds = eo.rows_step(optimizer, rows_np, g.numpy(), h[0], h[1], lr, hyper)
        eo.parity_add(prow_np, wde, wds, h[2], h[3])
        assert same(d[0], h[0]) and same(d[1], h[1]) and same(d[2], h[2]) and same(d[3], h[3]), step
    assert bad.item() == 0
    if m >= 3:                                     # a data row and a parity row out of range: both skipped
        rows, g = synth.ecrm_batch(n_rows, m, dim, seed=999)
        prow = torch.from_numpy(rng.permutation(p_rows)[:m].astype(np.uint32).view(np.int32))
        rows_bad, prow_bad = rows.clone(), prow.clone()
        rows_bad[1] = n_rows
        prow_bad[2] = p_rows + 5
        ecrm.rows_step_parity(optimizer, rows_bad.cuda(), prow_bad.cuda(), g.cuda(), d[0], d[1], d[2], d[3], lr, hyper, bad)
        keep = np.ones(m, bool); keep[[1, 2]] = False
        wde, wds = eo.rows_step(optimizer, rows.numpy().view(np.uint32)[keep], g.numpy()[keep], h[0], h[1], lr, hyper)
        eo.parity_add(prow.numpy().view(np.uint32)[keep], wde, wds, h[2], h[3])
        assert same(d[0], h[0]) and same(d[1], h[1]) and same(d[2], h[2]) and same(d[3], h[3])
        assert bad.item() == 2


def test_integer_valued_shards_are_recovered_exactly():
    shards = synth.ecrm_tables(5000, 128, 4, seed=3, device="cuda", integer_valued=True)
    parity = torch.empty_like(shards[0])
    ecrm.encode(shards, parity)
    for lost in range(4):
        out = torch.empty_like(parity)
        ecrm.decode([s for i, s in enumerate(shards) if i != lost], parity, out)
        assert torch.equal(out, shards[lost])


@pytest.mark.parametrize("optimizer,lr,hyper", [(ecrm.ECRM_ADAGRAD, 0.05, 1e-8), (ecrm.ECRM_MOMENTUM, 0.01, 0.9)])
@pytest.mark.parametrize("n_rows,m,dim", [(1, 1, 4), (100, 100, 128), (5000, 1237, 128), (3000, 700, 64),
                                          (999, 333, 132), (200_000, 20_000, 128)])
def test_rows_step_and_parity_add_match_oracle_bitwise(optimizer, lr, hyper, n_rows, m, dim):
    """Three steps of: optimizer on the batch's rows (differences out), parity host adds them."""
    entry = synth.ecrm_tables(n_rows, dim, 1, seed=n_rows + dim)[0]
    state = torch.zeros(n_rows, dim)
    p_entry, p_state = entry * 3.0, torch.zeros(n_rows, dim)        # some parity content
    d = [t.cuda() for t in (entry, state, p_entry, p_state)]
    h = [t.numpy().copy() for t in (entry, state, p_entry, p_state)]
    de, ds = torch.empty(m, dim, device="cuda"), torch.empty(m, dim, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step in range(3):
        rows, g = synth.ecrm_batch(n_rows, m, dim, seed=100 * step + m)
        ecrm.rows_step(optimizer, rows.cuda(), g.cuda(), d[0], d[1], lr, hyper, de, ds, bad)
        rows_np = rows.numpy().view(np.uint32)
        wde, wds = eo.rows_step(optimizer, rows_np, g.numpy(), h[0], h[1], lr, hyper)
        assert same(de, wde) and same(ds, wds) and same(d[0], h[0]) and same(d[1], h[1]), step
        ecrm.parity_add(rows.cuda(), de, ds, d[2], d[3], bad)
        eo.parity_add(rows_np, wde, wds, h[2], h[3])
        assert same(d[2], h[2]) and same(d[3], h[3]), step
    # stateless form of the parity update
    ecrm.parity_add(rows.cuda(), de, None, d[2], None, bad)
    eo.parity_add(rows_np, wde, None, h[2], None)
    assert same(d[2], h[2]) and bad.item() == 0


def test_out_of_range_rows_are_skipped_and_counted():
    n_rows, dim = 50, 128
    entry, state = torch.ones(n_rows, dim, device="cuda"), torch.zeros(n_rows, dim, device="cuda")
    rows = torch.tensor([3, 50, 7, 4_000_000_000 - (1 << 32)], dtype=torch.int32, device="cuda")
    g = torch.ones(4, dim, device="cuda")
    de, ds = torch.zeros(4, dim, device="cuda"), torch.zeros(4, dim, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    ecrm.rows_step(ecrm.ECRM_MOMENTUM, rows, g, entry, state, 0.5, 0.0, de, ds, bad)
    assert bad.item() == 2
    touched = (entry != 1.0).any(dim=1).nonzero().flatten().tolist()
    assert touched == [3, 7] and de[1].eq(0).all() and de[3].eq(0).all()
    ecrm.parity_add(rows, de, ds, entry, state, bad)
    assert bad.item() == 4


def test_degraded_read_matches_oracle_and_the_lost_rows():
    k, n_rows, dim, m = 4, 20_000, 128, 3000
    shards = synth.ecrm_tables(n_rows, dim, k, seed=9, device="cuda", integer_valued=True)
    parity = torch.empty_like(shards[0])
    ecrm.encode(shards, parity)
    rows, _ = synth.ecrm_batch(n_rows, m, dim, seed=4)
    rows = torch.cat([rows, rows[:5]]).cuda()                       # reads may repeat
    out = torch.empty(rows.numel(), dim, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    lost = 2
    survivors = [s for i, s in enumerate(shards) if i != lost]
    ecrm.degraded_read(rows, None, survivors, parity, out, bad)
    idx = rows.cpu().numpy().view(np.uint32)
    want = eo.degraded_read(idx, None, [s.cpu().numpy() for s in survivors], parity.cpu().numpy())
    assert same(out, want) and torch.equal(out, shards[lost][rows.long()]) and bad.item() == 0
    # a survivor kept under permuted row numbers
    perm = torch.randperm(n_rows, generator=torch.Generator().manual_seed(1)).cuda()
    moved = torch.empty_like(survivors[1]); moved[perm] = survivors[1]
    srows = [None, perm[rows.long()].to(torch.int32), None]
    ecrm.degraded_read(rows, srows, [survivors[0], moved, survivors[2]], parity, out, bad)
    assert torch.equal(out, shards[lost][rows.long()])
    # real-valued data: bitwise equal to the oracle's rounding
    real = synth.ecrm_tables(n_rows, dim, k, seed=10, device="cuda")
    ecrm.encode(real, parity)
    ecrm.degraded_read(rows, None, real[1:], parity, out, bad)
    want = eo.degraded_read(idx, None, [s.cpu().numpy() for s in real[1:]], parity.cpu().numpy())
    assert same(out, want)


def test_end_to_end_three_servers_stay_recoverable():
    """k = 3 data servers and a parity host through several batches, then a server is lost:
    full recovery (decode over the whole shard) and degraded reads return its rows.  Momentum
    with dyadic constants on integer data keeps every sum exact, so equality is bitwise."""
    k, n_rows, dim, m = 3, 4096, 128, 900
    entries = synth.ecrm_tables(n_rows, dim, k, seed=21, device="cuda", integer_valued=True)
    states = [torch.zeros(n_rows, dim, device="cuda") for _ in range(k)]
    p_entry, p_state = torch.empty_like(entries[0]), torch.empty_like(entries[0])
    ecrm.encode(entries, p_entry)
    ecrm.encode(states, p_state)
    de, ds = torch.empty(m, dim, device="cuda"), torch.empty(m, dim, device="cuda")
    for step in range(4):
        for s in range(k):
            rows, g = synth.ecrm_batch(n_rows, m, dim, seed=50 * step + s, device="cpu", integer_valued=True)
            rows, g = rows.cuda(), g.cuda()
            ecrm.rows_step(ecrm.ECRM_MOMENTUM, rows, g, entries[s], states[s], 0.25, 0.5, de, ds)
            ecrm.parity_add(rows, de, ds, p_entry, p_state)
    for lost in range(k):
        out = torch.empty_like(p_entry)
        ecrm.decode([e for i, e in enumerate(entries) if i != lost], p_entry, out)
        assert torch.equal(out, entries[lost])
        ecrm.decode([e for i, e in enumerate(states) if i != lost], p_state, out)
        assert torch.equal(out, states[lost])


def test_argument_checks():
    a = torch.zeros(64, device="cuda")
    with pytest.raises(ecrm.EcrmError):
        ecrm.encode([], a)
    with pytest.raises(ecrm.EcrmError):
        ecrm.encode([a[1:33]], a[:32])                     # misaligned shard
    with pytest.raises(ecrm.EcrmError):
        ecrm.encode([a], a)                                # parity aliases a shard
    e = torch.zeros(4, 6, device="cuda")                   # dim not a multiple of 4
    r = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(ecrm.EcrmError):
        ecrm.rows_step(ecrm.ECRM_ADAGRAD, r, e[:1], e, e.clone(), 0.1, 0.0, e[:1].clone(), e[:1].clone())
    with pytest.raises(ecrm.EcrmError):
        ecrm.rows_step(7, r, a[:4].view(1, 4), a.view(16, 4), a.clone().view(16, 4), 0.1, 0.0,
                       a[:4].clone().view(1, 4), a[:4].clone().view(1, 4))
