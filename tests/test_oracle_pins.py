"""Pins of the CPU oracle against things other than itself: brute force in numpy, closed
forms, hand-worked examples, printed figures and invariants.  No GPU needed."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2104_01981_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def keys(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def brute_topk(a, k):
    """Full sort of every index by (key descending, index ascending); first k, then by index."""
    ky = keys(a).astype(np.int64)
    order = np.lexsort((np.arange(a.size), -ky))
    return np.sort(order[:k]).astype(np.uint32)


def f32_add(x, y):
    return (np.asarray(x, np.float32) + np.asarray(y, np.float32)).astype(np.float32)


# ------------------------------------------------------------------ k rule
def test_k_matches_printed_figure():
    for line in open(os.path.join(GOLD, "k_from_density.txt")):
        if line.startswith("#") or not line.strip():
            continue
        n, d, k = line.split()
        assert oracle.k_from_density(int(n), float(d)) == int(k)


@pytest.mark.parametrize("cfg", [0, 1, 2, 4])
def test_k_equals_exact_rational_ceiling_on_all_workload_sizes(cfg):
    w = synth.workload(cfg)
    d = Fraction(str(w.density))
    for n in set(w.sizes):
        exact = min(n, max(1, math.ceil(d * n)))
        assert oracle.k_from_density(n, w.density) == exact


def test_k_edges():
    assert oracle.k_from_density(0, 0.5) == 0
    assert oracle.k_from_density(64, 0.001) == 1        # tiny tensors still send one entry
    assert oracle.k_from_density(7, 1.0) == 7
    assert oracle.k_from_density(1000, 0.001) == 1
    assert oracle.k_from_density(2048000, 0.001) == 2048


def test_resnet50_totals():
    w = synth.workload(1)
    assert len(w.sizes) == 161 and w.total_n == 25_557_032
    assert sum(oracle.k_from_density(n, w.density) for n in w.sizes) == 25_670
    assert synth.workload(2).total_n == 109_482_240
    assert synth.workload(4).total_n == 354_823_168


# ------------------------------------------------------------------ selection vs brute force
@pytest.mark.parametrize("seed", range(40))
def test_topk_matches_bruteforce_random(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 4097))
    k = int(rng.integers(1, n + 1))
    g = rng.standard_normal(n).astype(np.float32)
    r0 = (rng.standard_normal(n) * 0.5).astype(np.float32)
    a = f32_add(g, r0)
    r = r0.copy()
    idx, val = oracle.topk_compress(g, r, k)
    want = brute_topk(a, k)
    assert np.array_equal(idx, want)
    assert np.array_equal(val.view(np.uint32), a[want].view(np.uint32))
    exp_r = a.copy()
    exp_r[want] = 0.0
    assert np.array_equal(r.view(np.uint32), exp_r.view(np.uint32))


@pytest.mark.parametrize("seed", range(20))
def test_topk_matches_bruteforce_tie_heavy(seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(2, 3000))
    k = int(rng.integers(1, n + 1))
    levels = int(rng.integers(1, 6))
    g = (rng.integers(-levels, levels + 1, n) * 0.25).astype(np.float32)   # few distinct magnitudes
    r = np.zeros(n, np.float32)
    idx, _ = oracle.topk_compress(g, r, k)
    assert np.array_equal(idx, brute_topk(g, k))


def test_closed_form_distinct_magnitudes_pick_the_last_k():
    n, k = 1000, 37
    sign = np.where(np.arange(n) % 3 == 0, -1.0, 1.0)
    g = (sign * (np.arange(n) + 1)).astype(np.float32)
    r = np.zeros(n, np.float32)
    idx, val = oracle.topk_compress(g, r, k)
    assert np.array_equal(idx, np.arange(n - k, n, dtype=np.uint32))
    assert np.array_equal(val, g[n - k:])
    assert np.all(r[n - k:] == 0) and np.array_equal(r[:n - k], g[:n - k])


def test_closed_form_all_equal_picks_the_first_k():
    for value in (0.0, 2.5, -2.5):
        g = np.full(257, value, np.float32)
        r = np.zeros(257, np.float32)
        idx, _ = oracle.topk_compress(g, r, 19)
        assert np.array_equal(idx, np.arange(19, dtype=np.uint32))


def test_closed_form_sign_does_not_matter_for_ties():
    g = np.array([1, -1, 1, -1, 1, -1], np.float32)
    r = np.zeros(6, np.float32)
    idx, val = oracle.topk_compress(g, r, 4)
    assert idx.tolist() == [0, 1, 2, 3] and val.tolist() == [1, -1, 1, -1]


def test_closed_form_two_values_all_large_plus_lowest_index_small():
    n = 500
    big = np.array([7, 50, 123, 400, 499])
    g = np.full(n, 0.5, np.float32)
    g[big] = -3.0
    r = np.zeros(n, np.float32)
    k = 9
    idx, _ = oracle.topk_compress(g, r, k)
    small = [i for i in range(n) if i not in set(big.tolist())][:k - big.size]
    assert sorted(idx.tolist()) == sorted(big.tolist() + small)


def test_k_equals_n_sends_everything_and_k_zero_sends_nothing():
    g = np.arange(1, 9, dtype=np.float32)
    r = np.ones(8, np.float32)
    idx, val = oracle.topk_compress(g, r, 8)
    assert idx.tolist() == list(range(8)) and np.array_equal(val, g + 1) and not r.any()
    r = np.ones(8, np.float32)
    idx, val = oracle.topk_compress(g, r, 0)
    assert idx.size == 0 and np.array_equal(r, g + 1)


def test_index_base_offsets_emitted_indices():
    g = np.array([0, 5, 0, 0], np.float32)
    idx, _ = oracle.topk_compress(g, np.zeros(4, np.float32), 1, index_base=1000)
    assert idx.tolist() == [1001]


# ------------------------------------------------------------------ fold arithmetic / special values
def test_fold_is_a_single_fp32_rounding():
    # 1 + 2^-24 is a tie in fp32 and rounds to even (1.0); 1 + 3*2^-25 rounds up to 1+2^-23.
    g = np.array([1.0, 1.0, 16777216.0], np.float32)
    r = np.array([2.0 ** -24, 3 * 2.0 ** -25, 1.0], np.float32)
    rr = r.copy()
    idx, val = oracle.topk_compress(g, rr, 3)
    assert val.tolist() == [1.0, float(np.float32(1 + 2.0 ** -23)), 16777216.0]


def test_negative_zero_and_nonfinite_ordering():
    a = np.array([-0.0, 1.0, np.inf, np.nan, -np.inf, 3.0], np.float32)
    r = np.zeros(6, np.float32)
    idx, val = oracle.topk_compress(a, r, 3)
    # NaN's key exceeds Inf's; the two infinities tie and both fit
    assert idx.tolist() == [2, 3, 4]
    r = np.zeros(6, np.float32)
    r[0] = -0.0                                           # IEEE: -0 + +0 = +0, only -0 + -0 = -0
    idx, val = oracle.topk_compress(a, r, 6)
    assert val.view(np.uint32)[0] == 0x80000000          # -0.0 travels as a bit copy
    assert r.view(np.uint32).tolist() == [0] * 6          # and leaves +0.0 behind


def test_denormals_are_kept():
    tiny = np.float32(1e-45)
    g = np.array([tiny, 0.0, -tiny, 0.0], np.float32)
    r = np.zeros(4, np.float32)
    idx, val = oracle.topk_compress(g, r, 2)
    assert idx.tolist() == [0, 2] and val.view(np.uint32).tolist() == [1, 0x80000001]


# ------------------------------------------------------------------ error feedback across steps
def test_hand_example_two_steps():
    r = np.zeros(4, np.float32)
    for line in open(os.path.join(GOLD, "error_feedback_hand_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, g, si, sv, rafter = [p.strip() for p in line.split("|")]
        g = np.array(g.split(), np.float32)
        idx, val = oracle.topk_compress(g, r, 1)
        assert idx.tolist() == [int(si)] and val.tolist() == [float(sv)]
        assert r.tolist() == [float(x) for x in rafter.split()]


def test_conservation_with_integer_valued_gradients():
    """With small integers every fp32 add is exact, so sent + residual == sum of gradients."""
    rng = np.random.default_rng(7)
    n, k, steps = 5000, 50, 12
    r = np.zeros(n, np.float32)
    sent = np.zeros(n, np.float64)
    total = np.zeros(n, np.float64)
    for _ in range(steps):
        g = rng.integers(-8, 9, n).astype(np.float32)
        total += g
        idx, val = oracle.topk_compress(g, r, k)
        assert idx.size == k and np.all(np.diff(idx.astype(np.int64)) > 0)
        np.add.at(sent, idx, val)
    assert np.array_equal(sent + r, total)


def test_invariants_every_selected_key_dominates():
    rng = np.random.default_rng(11)
    n, k = 20000, 200
    g = np.round(rng.standard_normal(n) * 8).astype(np.float32) / 8      # tie stress
    r0 = np.round(rng.standard_normal(n) * 8).astype(np.float32) / 8
    a = f32_add(g, r0)
    r = r0.copy()
    idx, val = oracle.topk_compress(g, r, k)
    ky = keys(a)
    sel = np.zeros(n, bool)
    sel[idx] = True
    T = ky[sel].min()
    assert ky[~sel].max() <= T
    # among keys equal to the threshold, the selected ones are exactly the lowest indices
    eq = np.nonzero(ky == T)[0]
    m = sel[eq].sum()
    assert sel[eq[:m]].all() and not sel[eq[m:]].any()
    # residual + transmitted == accumulated gradient
    back = r.copy()
    back[idx] += val
    assert np.array_equal(back, a)


def test_layerwise_is_independent_per_tensor():
    rng = np.random.default_rng(5)
    sizes = [64, 1000, 7, 4096, 1]
    ks = [oracle.k_from_density(n, 0.01) for n in sizes]
    g = rng.standard_normal(sum(sizes)).astype(np.float32)
    r = np.zeros_like(g)
    idx, val = oracle.topk_compress_tensors(sizes, ks, g, r)
    off = ooff = 0
    for n, k in zip(sizes, ks):
        want = brute_topk(g[off:off + n], k) + off
        assert np.array_equal(idx[ooff:ooff + k], want)
        off += n
        ooff += k
    assert np.all(np.diff(idx.astype(np.int64)) > 0)       # globally ascending as well


# ------------------------------------------------------------------ decode
def test_decode_single_worker_is_a_scatter():
    out = np.full(10, 9.0, np.float32)
    oracle.decode_accumulate([(np.array([1, 4, 9]), np.array([1.5, -2.0, 3.0]))], out, True)
    assert out.tolist() == [0, 1.5, 0, 0, -2.0, 0, 0, 0, 0, 3.0]


def test_decode_accumulates_when_not_zeroed():
    out = np.ones(4, np.float32)
    oracle.decode_accumulate([(np.array([0, 3]), np.array([1.0, 2.0]))], out, False)
    assert out.tolist() == [2, 1, 1, 3]


def test_density_one_reproduces_dense_left_to_right_sum():
    rng = np.random.default_rng(3)
    n, W = 3000, 7
    grads = [rng.standard_normal(n).astype(np.float32) * (10.0 ** rng.integers(-3, 4)) for _ in range(W)]
    pairs = []
    for g in grads:
        idx, val = oracle.topk_compress(g, np.zeros(n, np.float32), n)
        pairs.append((idx, val))
    out = oracle.decode_accumulate(pairs, np.empty(n, np.float32), True)
    dense = np.zeros(n, np.float32)
    for g in grads:                                      # fixed worker order, fp32 throughout
        dense = f32_add(dense, g)
    assert np.array_equal(out.view(np.uint32), dense.view(np.uint32))


def test_decode_worker_order_matters_and_is_0_to_W_minus_1():
    # (1e8 + 1) - 1e8 = 0 in fp32 but (1e8 - 1e8) + 1 = 1: order is observable
    i = np.array([0])
    a, b, c = np.array([1e8], np.float32), np.array([1.0], np.float32), np.array([-1e8], np.float32)
    out = oracle.decode_accumulate([(i, a), (i, b), (i, c)], np.empty(1, np.float32))
    assert out[0] == 0.0
    out = oracle.decode_accumulate([(i, a), (i, c), (i, b)], np.empty(1, np.float32))
    assert out[0] == 1.0


def test_decode_disjoint_sets_give_the_union_and_minus_zero_becomes_plus_zero():
    out = oracle.decode_accumulate([(np.array([0, 2]), np.array([1.0, -0.0])),
                                    (np.array([1, 3]), np.array([5.0, 6.0]))], np.empty(4, np.float32))
    assert out.tolist() == [1, 5, 0, 6] and out.view(np.uint32)[2] == 0      # +0 + -0 = +0


# ------------------------------------------------------------------ threshold variant (own reading)
def brute_threshold(a, density, stride, cap):
    n = a.size
    ky = keys(a)
    samp = ky[((np.arange(n) >> 2) % stride) == 0]
    ks = min(samp.size, max(1, math.ceil(density * samp.size)))
    tau = np.sort(samp)[::-1][ks - 1]
    hits = np.nonzero(ky >= tau)[0]
    return hits[:cap].astype(np.uint32), hits.size, int(tau)


@pytest.mark.parametrize("seed", range(20))
def test_threshold_matches_bruteforce(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 5000))
    stride = int(rng.choice([1, 2, 3, 8, 64]))
    density = float(rng.choice([0.001, 0.01, 0.1, 0.5]))
    cap = int(rng.integers(1, n + 1))
    g = rng.standard_normal(n).astype(np.float32)
    if seed % 3 == 0:
        g = np.round(g * 4) / 4
    g = f32_add(g, np.zeros(n, np.float32))               # the fold turns -0 + +0 into +0
    r = np.zeros(n, np.float32)
    idx, val, hits, tau = oracle.threshold_compress(g, r, density, stride, cap)
    widx, whits, wtau = brute_threshold(g, density, stride, cap)
    assert np.array_equal(idx, widx) and hits == whits and tau == wtau
    exp_r = g.copy()
    exp_r[widx] = 0
    assert np.array_equal(r.view(np.uint32), exp_r.view(np.uint32))
    assert np.array_equal(val.view(np.uint32), g[widx].view(np.uint32))


def test_threshold_with_full_sample_equals_topk_threshold():
    rng = np.random.default_rng(2)
    n, density = 4096, 0.01
    g = rng.standard_normal(n).astype(np.float32)          # continuous: no ties
    k = oracle.k_from_density(n, density)
    tidx, _ = oracle.topk_compress(g, np.zeros(n, np.float32), k)
    idx, val, hits, tau = oracle.threshold_compress(g, np.zeros(n, np.float32), density, 1, n)
    assert tau == keys(g)[tidx].min() and hits == k and np.array_equal(idx, tidx)


def test_threshold_truncation_keeps_a_prefix_and_leaves_the_rest_in_the_residual():
    g = np.array([5, 0, 5, 0, 5, 0, 5, 0], np.float32)
    r = np.zeros(8, np.float32)
    idx, val, hits, tau = oracle.threshold_compress(g, r, 0.5, 1, 2)
    assert idx.tolist() == [0, 2] and hits == 4 and r.tolist() == [0, 0, 0, 0, 5, 0, 5, 0]


def test_sample_definition():
    assert oracle.sample_count(16, 1) == 16
    assert oracle.sample_count(16, 2) == 8             # groups 0 and 2
    assert oracle.sample_count(10, 2) == 6             # group 0 (4) + group 2 (2 of 4)
    assert oracle.sample_count(1 << 20, 64) == (1 << 20) // 64
    assert oracle.effective_stride(65536, 64) == 1 and oracle.effective_stride(65537, 64) == 64


def test_decode_apply_momentum_hand_values_and_torch_sgd():
    """Fused decode + momentum SGD: hand values (dyadic, exact), the untouched elements still
    take their momentum step, and many steps agree with torch.optim.SGD on the dense sum."""
    import torch
    p = np.array([1.0, 2.0, 3.0, 4.0], np.float32)
    v = np.array([0.5, 0.0, -1.0, 2.0], np.float32)
    pairs = [(np.array([1, 3], np.uint32), np.array([4.0, -2.0], np.float32)),
             (np.array([3], np.uint32), np.array([6.0], np.float32))]
    oracle.decode_apply_momentum(pairs, p, v, lr=0.25, momentum=0.5, scale=0.5)
    # s = [0, 4, 0, 4]; v' = 0.5 v + 0.5 s = [0.25, 2, -0.5, 3]; p' = p - 0.25 v'
    assert v.tolist() == [0.25, 2.0, -0.5, 3.0]
    assert p.tolist() == [0.9375, 1.5, 3.125, 3.25]
    rng = np.random.default_rng(3)
    n, W = 500, 3
    p = rng.standard_normal(n).astype(np.float32); v = np.zeros(n, np.float32)
    tp = torch.nn.Parameter(torch.from_numpy(p.copy()))
    opt = torch.optim.SGD([tp], lr=0.1, momentum=0.9)
    for step in range(20):
        pairs = []
        dense = np.zeros(n, np.float32)
        for w in range(W):
            idx = np.sort(rng.choice(n, size=40, replace=False)).astype(np.uint32)
            val = rng.standard_normal(40).astype(np.float32)
            pairs.append((idx, val))
            dense[idx] = (dense[idx] + val).astype(np.float32)
        oracle.decode_apply_momentum(pairs, p, v, lr=0.1, momentum=0.9, scale=1.0)
        tp.grad = torch.from_numpy(dense.copy())
        opt.step()
    assert np.allclose(p, tp.detach().numpy(), rtol=1e-5, atol=1e-6)
