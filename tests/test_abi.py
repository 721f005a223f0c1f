"""The C-ABI library loads, exports every symbol the header declares, and its host-side
logic (k rule, offsets, capacities, argument checks) is right.  No GPU needed."""
import ctypes
import math
import os
import re

import pytest

import oracle
from paper_2104_01981_b200 import api, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def declared_symbols():
    syms = set()
    inc = os.path.join(ROOT, "include")
    for name in sorted(os.listdir(inc)):
        text = open(os.path.join(inc, name)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        syms |= set(re.findall(r"\b((?:gc|ecrm)_[a-z_0-9]+)\s*\(", text))
    return sorted(syms)


def test_every_declared_symbol_is_exported(lib):
    syms = declared_symbols()
    assert {"gc_plan", "gc_compress", "gc_decompress_accumulate", "gc_destroy"} <= set(syms)
    assert {"ecrm_encode", "ecrm_decode", "ecrm_rows_step", "ecrm_parity_add", "ecrm_degraded_read",
            "ecrm_placement"} <= set(syms)
    for s in syms:
        assert hasattr(lib, s), s
    assert lib.gc_version() >= 1


def test_host_plan_k_offsets_match_the_oracle_rule(lib):
    for cfg in (0, 1, 2, 4):
        w = synth.workload(cfg)
        p = api.Plan(w.sizes, w.density, device=-1)
        ks = p.tensor_k()
        assert ks == [oracle.k_from_density(n, w.density) for n in w.sizes]
        offs = p.tensor_out_offset()
        assert offs == [sum(ks[:t]) for t in range(len(ks))]
        assert p.total_n == w.total_n and p.total_cap == sum(ks)
        assert p.workspace_bytes % 256 == 0
        p.destroy()
    p = api.Plan([1 << 20], 0.01, device=-1)
    assert p.tensor_k() == [10486]


def test_threshold_plan_capacity_and_stride(lib):
    sizes = [64, 65536, 65537, 1_000_000]
    p = api.Plan(sizes, 0.001, mode=api.GC_THRESHOLD, device=-1)
    ks = [oracle.k_from_density(n, 0.001) for n in sizes]
    assert p.tensor_cap() == [min(n, math.ceil(2.0 * k)) for n, k in zip(sizes, ks)]
    assert [p.query(api.GC_Q_TENSOR_STRIDE, t) for t in range(4)] == \
        [oracle.effective_stride(n, 64) for n in sizes]
    p2 = api.Plan(sizes, 0.001, mode=api.GC_THRESHOLD, device=-1, sample_stride=16, cap_factor=1.5)
    assert p2.tensor_cap() == [min(n, math.ceil(1.5 * k)) for n, k in zip(sizes, ks)]
    assert p2.query(api.GC_Q_TENSOR_STRIDE, 3) == 16


def test_plan_rejects_bad_arguments(lib):
    for density in (0.0, -0.1, 1.5, float("nan")):
        with pytest.raises(api.GcError) as e:
            api.Plan([10], density, device=-1)
        assert e.value.code == api.GC_E_INVALID
    with pytest.raises(api.GcError) as e:
        api.Plan([1 << 30, 1 << 30], 0.01, device=-1)
    assert e.value.code == api.GC_E_TOO_LARGE
    with pytest.raises(api.GcError):
        api.Plan([10], 0.5, mode=7, device=-1)
    with pytest.raises(api.GcError):
        api.Plan([10], 0.5, mode=api.GC_THRESHOLD, device=-1, cap_factor=0.5)


def test_empty_and_zero_sized_tensors(lib):
    p = api.Plan([], 0.5, device=-1)
    assert p.total_n == 0 and p.total_cap == 0
    p = api.Plan([0, 5, 0], 0.5, device=-1)
    assert p.tensor_k() == [0, 3, 0] and p.tensor_out_offset() == [0, 0, 3]
    with pytest.raises(api.GcError):
        p.query(api.GC_Q_TENSOR_K, 3)


def test_plan_options_accept_their_values_and_reject_others(lib):
    p = api.Plan([1000], 0.01, device=-1)
    for opt, good, bad in [(api.GC_OPT_PATH, (api.GC_PATH_AUTO, api.GC_PATH_EXACT, api.GC_PATH_STAGED), 3),
                           (api.GC_OPT_DECODE_ROUTE, (api.GC_DECODE_AUTO, api.GC_DECODE_NARROW, api.GC_DECODE_WIDE), 3),
                           (api.GC_OPT_DECODE_ORDER, (api.GC_ORDER_FIXED, api.GC_ORDER_ANY), 2)]:
        for v in good:
            p.set_option(opt, v)
        with pytest.raises(api.GcError) as e:
            p.set_option(opt, bad)
        assert e.value.code == api.GC_E_INVALID
    with pytest.raises(api.GcError):
        p.set_option(99, 0)


def test_workspace_size_survives_the_sample_rank_option(lib):
    """At densities near 1 a tensor's default sample rank reaches its sample size and the tensor is
    left unsampled; a smaller rank option samples it after all.  The workspace size reported at
    plan creation must already cover the sample keys kept then."""
    for sizes, density in (([300_000, 5, 1_500_001, 131_072], 0.9), ([300_000, 70_000], 0.99),
                           ([2_000_000], 0.95), ([300_000, 5, 1_500_001], 0.01)):
        p = api.Plan(sizes, density, device=-1)
        before = p.query(api.GC_Q_WORKSPACE_BYTES)
        for permille in (30, 500, 1000, 5000):
            p.set_option(api.GC_OPT_SAMPLE_RANK_PERMILLE, permille)
            assert p.query(api.GC_Q_WORKSPACE_BYTES) <= before, (sizes, density, permille)
        p.destroy()


def test_host_only_plan_refuses_compute(lib):
    p = api.Plan([16], 0.5, device=-1)
    assert p.compress_ptr(16, 16, 16, 16, None, 256, 0) == api.GC_E_UNSUPPORTED
    assert lib.gc_destroy(None) == api.GC_OK


def test_ecrm_placement_matches_the_oracle_rule(lib):
    from oracle import ecrm_oracle
    from paper_2104_01981_b200 import ecrm
    for k in (1, 3, 4, 32):
        for group in (0, 1, k, k + 1, 12345678901):
            assert ecrm.placement(k, group) == ecrm_oracle.placement(k, group)
    with pytest.raises(ecrm.EcrmError):
        ecrm.placement(0, 1)
    with pytest.raises(ecrm.EcrmError):
        ecrm.placement(33, 1)
