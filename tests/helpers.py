"""Shared plumbing of the GPU parity tests: run the CUDA library and the CPU oracle on the
same input bytes and compare bit for bit."""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np
import torch

import oracle
from paper_2104_01981_b200 import api


def bits(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x).view(np.uint32)


def to_np_u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def same_f32_bits(x_bits: np.ndarray, y_bits: np.ndarray) -> bool:
    """Bitwise equality, except that any NaN equals any NaN: the payload an fp32 adder gives a
    NaN result is left open by IEEE 754 and differs between x86 (operand payload) and the GPU
    (canonical 0x7FFFFFFF)."""
    if np.array_equal(x_bits, y_bits):
        return True
    nan_x = (x_bits & 0x7FFFFFFF) > 0x7F800000
    nan_y = (y_bits & 0x7FFFFFFF) > 0x7F800000
    return bool(np.all((x_bits == y_bits) | (nan_x & nan_y)))


class GpuWorker:
    """One simulated worker on the GPU: residual, outputs, workspace."""

    def __init__(self, plan: api.Plan):
        self.plan = plan
        dev = f"cuda:{plan.device}"
        self.residual = torch.zeros(max(plan.total_n, 4), dtype=torch.float32, device=dev)
        self.idx, self.val, self.count = plan.alloc_outputs()
        self.ws = plan.alloc_workspace()

    def step(self, g: torch.Tensor) -> None:
        # poison outputs so that a slot the kernels fail to write is caught
        self.idx.fill_(-1)
        self.val.fill_(float("nan"))
        self.plan.compress(g, self.residual, self.idx, self.val, self.count, self.ws)

    def check_status(self, expect: int = api.GC_OK):
        st, det = self.plan.last_status(self.ws)
        assert st == expect, f"device status {st} (detail {det})"
        return st, det


def check_topk_against_oracle(sizes: Sequence[int], density: float, grads,
                              r0: Optional[torch.Tensor] = None, device: int = 0, options=None,
                              expect_counters=None):
    """Runs one step per gradient in `grads` (a list, or any iterable that yields them one at a
    time) of one worker on GPU and oracle; asserts bitwise
    equality of indices, values, counts and residual after every step.  Returns the plan
    worker (for decode tests) and the oracle's last (idx, val)."""
    plan = api.Plan(sizes, density, device=device)
    for opt, value in (options or {}).items():
        plan.set_option(opt, value)
    w = GpuWorker(plan)
    ks = plan.tensor_k()
    n = plan.total_n
    r_cpu = np.zeros(n, np.float32)
    if r0 is not None:
        w.residual[:n].copy_(r0.to(w.residual.device))
        r_cpu = r0.cpu().numpy().astype(np.float32).copy()
    last = None
    for step, g in enumerate(grads):
        g_dev = g.to(f"cuda:{device}")
        if g_dev.numel() < 4:
            g_dev = torch.cat([g_dev, torch.zeros(4 - g_dev.numel(), device=g_dev.device)])
        w.step(g_dev)
        w.check_status()
        if expect_counters is not None:
            expect_counters(plan.last_counters(w.ws))
        g_cpu = g.cpu().numpy()
        del g_dev
        oi, ov = oracle.topk_compress_tensors(list(sizes), ks, g_cpu, r_cpu)
        tot = sum(ks)
        gi = to_np_u32(w.idx[:tot])
        gv = to_np_u32(w.val[:tot])
        assert np.array_equal(gi, oi), f"step {step}: index sets differ"
        assert same_f32_bits(gv, bits(ov)), f"step {step}: values differ"
        assert same_f32_bits(to_np_u32(w.residual[:n]), bits(r_cpu)), f"step {step}: residual differs"
        cnt = w.count.cpu().numpy()
        T = len(sizes)
        assert cnt[:T].tolist() == ks and cnt[T:2 * T].tolist() == ks
        last = (oi, ov)
    return plan, w, last
