"""Pins of the erasure-coded embedding-table oracle against what the source states and what the
arithmetic fixes (no GPU): the k = 3 worked example, closed forms of the optimizers, the parity
invariant of server-side propagation, the appendix timeline, rotating placement."""
import numpy as np
import pytest

from oracle import ecrm_oracle as eo

f32 = np.float32


def test_worked_example_k3_sum_and_subtraction():
    """Section 2 / Section 3.2: p = e1 + e2 + e3; with e2 lost, e2 = p - e1 - e3."""
    e1, e2, e3 = (np.array(v, f32) for v in ([1, -2, 3, 0.5], [4, 5, -6, 0.25], [-7, 8, 9, 2]))
    p = eo.encode([e1, e2, e3])
    assert p.tolist() == [-2.0, 11.0, 6.0, 2.75]
    assert np.array_equal(eo.decode(p, [e1, e3]), e2)
    assert np.array_equal(eo.decode(p, [e2, e3]), e1)
    assert np.array_equal(eo.decode(p, [e1, e2]), e3)
    assert np.array_equal(eo.decode(p, []), p) and np.array_equal(eo.encode([e1]), e1)     # k = 1: a replica


@pytest.mark.parametrize("k", [2, 3, 4, 8])
def test_any_one_of_k_plus_one_units_is_recoverable(k):
    """r = 1: any k of the k+1 units give the missing one.  Integer-valued data: exact."""
    rng = np.random.default_rng(k)
    shards = [rng.integers(-1000, 1000, size=257).astype(f32) for _ in range(k)]
    p = eo.encode(shards)
    assert np.array_equal(p, np.sum(np.stack(shards).astype(np.float64), axis=0).astype(f32))
    for lost in range(k):
        assert np.array_equal(eo.decode(p, [s for i, s in enumerate(shards) if i != lost]), shards[lost])
    # general floats: within a few roundings of the parity's magnitude
    shards = [rng.standard_normal(257).astype(f32) for _ in range(k)]
    p = eo.encode(shards)
    for lost in range(k):
        got = eo.decode(p, [s for i, s in enumerate(shards) if i != lost])
        bound = (k + 1) * np.finfo(f32).eps * np.sum(np.abs(np.stack(shards)), axis=0)
        assert np.all(np.abs(got.astype(np.float64) - shards[lost]) <= bound)


def test_adagrad_step_matches_the_written_update():
    """Section 3.3.1: G' = G + g^2, e' = e - lr / sqrt(G' + eps) * g.  Hand values that are exact:
    g = 2, G = 0, eps = 0, lr = 1 -> G' = 4, e' = e - 1; then g = 1.5: G' = 6.25, step = 0.4."""
    entry, state = np.full((3, 4), 10.0, f32), np.zeros((3, 4), f32)
    de, ds = eo.rows_step(eo.ADAGRAD, [1], np.full((1, 4), 2.0, f32), entry, state, lr=1.0, hyper=0.0)
    assert entry[1].tolist() == [9.0] * 4 and state[1].tolist() == [4.0] * 4
    assert entry[0].tolist() == [10.0] * 4 and entry[2].tolist() == [10.0] * 4          # other rows untouched
    assert de.tolist() == [[-1.0] * 4] and ds.tolist() == [[4.0] * 4]
    eo.rows_step(eo.ADAGRAD, [1], np.full((1, 4), 1.5, f32), entry, state, lr=1.0, hyper=0.0)
    assert state[1].tolist() == [6.25] * 4
    assert np.allclose(entry[1], 9.0 - 0.4 * 1.5, rtol=0, atol=1e-6)
    # against float64 over many steps with a varying gradient
    rng = np.random.default_rng(0)
    e64, s64 = np.zeros(8), np.zeros(8)
    entry, state = np.zeros((1, 8), f32), np.zeros((1, 8), f32)
    for _ in range(50):
        g = rng.standard_normal((1, 8)).astype(f32)
        eo.rows_step(eo.ADAGRAD, [0], g, entry, state, lr=0.1, hyper=1e-8)
        s64 += g[0].astype(np.float64) ** 2
        e64 -= 0.1 / np.sqrt(s64 + 1e-8) * g[0]
    assert np.allclose(entry[0], e64, rtol=1e-5, atol=1e-6) and np.allclose(state[0], s64, rtol=1e-5)


def test_momentum_closed_form():
    """Constant gradient 1, mu = 0.5: v_t = 2 - 2^(1-t); e_t = e_0 - lr * sum v (all exact in fp32)."""
    entry, state = np.zeros((1, 4), f32), np.zeros((1, 4), f32)
    g = np.ones((1, 4), f32)
    total = 0.0
    for t in range(1, 11):
        de, ds = eo.rows_step(eo.MOMENTUM, [0], g, entry, state, lr=0.25, hyper=0.5)
        v = 2.0 - 2.0 ** (1 - t)
        total += v
        assert state[0].tolist() == [v] * 4 and entry[0].tolist() == [-0.25 * total] * 4
        assert de[0].tolist() == [-0.25 * v] * 4


def simulate(optimizer, k, steps, lr, hyper, integer, seed):
    """k data servers + one parity host for the same row range; returns data, parity (entry, state)."""
    rng = np.random.default_rng(seed)
    n_rows, dim = 40, 8
    def draw(shape):
        return rng.integers(-8, 9, size=shape).astype(f32) if integer else rng.standard_normal(shape).astype(f32)
    entries = [draw((n_rows, dim)) for _ in range(k)]
    states = [np.zeros((n_rows, dim), f32) for _ in range(k)]
    p_entry, p_state = eo.encode(entries), eo.encode(states)
    for _ in range(steps):
        for s in range(k):
            rows = rng.choice(n_rows, size=7, replace=False)
            de, ds = eo.rows_step(optimizer, rows, draw((7, dim)), entries[s], states[s], lr, hyper)
            eo.parity_add(rows, de, ds, p_entry, p_state)        # same row number on the parity host
    return entries, states, p_entry, p_state


def test_server_side_propagation_keeps_parity_equal_to_the_sum():
    """Section 3.3.2: adding the DIFFERENCES keeps p = sum of entries (and of optimizer state).
    Momentum with mu = 0.5, lr = 0.25 on integer data stays in dyadic rationals: bit-exact."""
    entries, states, p_entry, p_state = simulate(eo.MOMENTUM, 3, 6, 0.25, 0.5, True, 1)
    assert np.array_equal(p_entry, eo.encode(entries)) and np.array_equal(p_state, eo.encode(states))
    for lost in range(3):       # hence any server's rows and state can be rebuilt exactly
        others = [e for i, e in enumerate(entries) if i != lost]
        assert np.array_equal(eo.decode(p_entry, others), entries[lost])
    # Adagrad on real-valued data: equal up to the roundings of the float sum
    entries, states, p_entry, p_state = simulate(eo.ADAGRAD, 4, 10, 0.1, 1e-8, False, 2)
    assert np.allclose(p_entry, eo.encode(entries), rtol=0, atol=2e-5)
    assert np.allclose(p_state, eo.encode(states), rtol=1e-5, atol=1e-5)


def test_worker_side_propagation_with_a_parity_accumulator_is_wrong():
    """Section 3.3.1: applying the optimizer on the parity host with the PARITY accumulator
    (sum of the k accumulators) does not keep p = e1 + e2 + e3, because G_p != G_1."""
    e = [np.full((1, 4), v, f32) for v in (1.0, 2.0, 3.0)]
    G = [np.full((1, 4), v, f32) for v in (4.0, 9.0, 16.0)]
    p, Gp = eo.encode(e), eo.encode(G)
    g = np.full((1, 4), 2.0, f32)
    eo.rows_step(eo.ADAGRAD, [0], g, e[0], G[0], lr=1.0, hyper=0.0)          # the data server
    eo.rows_step(eo.ADAGRAD, [0], g, p, Gp, lr=1.0, hyper=0.0)               # the parity host, same gradient
    assert np.array_equal(Gp, eo.encode(G))                                  # the accumulator parity is fine ...
    assert not np.allclose(p, eo.encode(e))                                  # ... the entry parity is not


def test_appendix_timeline_recovers_the_last_propagated_value():
    """Table 1 of the appendix: x is updated but its difference never leaves server 1; y is
    updated and propagated; server 1 fails; decoding x gives x_t (the value before the lost
    update) next to y_{t+1} -- a state asynchronous training could have produced."""
    x, y = np.array([[3.0, -1.0, 2.0, 5.0]], f32), np.array([[1.0, 4.0, -2.0, 0.0]], f32)
    sx, sy = np.zeros((1, 4), f32), np.zeros((1, 4), f32)
    p, ps = eo.encode([x, y]), eo.encode([sx, sy])
    x_t = x.copy()
    dx = eo.rows_step(eo.MOMENTUM, [0], np.array([[1.0, 2.0, -1.0, 4.0]], f32), x, sx, 0.5, 0.5)    # time 0
    y_read = y.copy()                                                                                 # time 1
    dy = eo.rows_step(eo.MOMENTUM, [0], np.array([[2.0, -2.0, 1.0, 1.0]], f32), y, sy, 0.5, 0.5)    # time 2
    eo.parity_add([0], dy[0], dy[1], p, ps)                                                           # time 3
    assert not np.array_equal(x, x_t) and not np.array_equal(y, y_read)
    recovered = eo.decode(p, [y])                                                                     # times 4, 5
    assert np.array_equal(recovered, x_t)
    assert np.array_equal(eo.decode(ps, [sy]), np.zeros((1, 4), f32))
    # had the difference been propagated, the new value would come back
    eo.parity_add([0], dx[0], dx[1], p, ps)
    assert np.array_equal(eo.decode(p, [y]), x)


def test_rotating_placement_balances_parities():
    """Section 3.2 (figure: k = 3, four servers): the parity host rotates, the k entries sit on the
    other servers, every server hosts the same number of parities."""
    for k in (2, 3, 4, 7):
        hosts = [eo.placement(k, g)[0] for g in range(5 * (k + 1))]
        assert hosts[:k + 1] == list(range(k + 1))
        assert all(hosts.count(s) == 5 for s in range(k + 1))
        for g in range(k + 1):
            ps, ds = eo.placement(k, g)
            assert ps not in ds and sorted(ds + [ps]) == list(range(k + 1)) and ds == sorted(ds)


def test_degraded_read_is_the_decoder_on_rows():
    rng = np.random.default_rng(5)
    shards = [rng.integers(-50, 50, size=(30, 8)).astype(f32) for _ in range(3)]
    p = eo.encode(shards)
    rows = np.array([29, 0, 7, 7, 15])
    assert np.array_equal(eo.degraded_read(rows, None, [shards[0], shards[2]], p), shards[1][rows])
    # survivors stored under other row numbers (placement maps a group to different rows per server)
    perm = rng.permutation(30)
    moved = np.empty_like(shards[2]); moved[perm] = shards[2]
    assert np.array_equal(eo.degraded_read(rows, [None, perm[rows]], [shards[0], moved], p), shards[1][rows])
