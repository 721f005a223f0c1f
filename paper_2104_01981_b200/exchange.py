"""Multi-GPU aggregation of the sparse sets: one all-gather of every rank's block of pairs, then a
local decode over the gathered lists in rank order.

Each rank compresses its own gradient into ONE contiguous block of 32-bit words

    [ idx : cap_pad | val : cap_pad | count : cnt_pad ]

(``cap`` = the plan's output capacity, sections padded to 16 bytes), so the exchange is a single
``all_gather_into_tensor`` of fixed-size blocks: with exact top-k the lists have a fixed length,
and in threshold mode the lists are padded to their capacity and the per-tensor counts travel in
the same block.  The gathered blocks land in this GPU's own memory before any kernel reads them;
the decode then takes rank r's sections as worker r's lists, so every rank adds the contributions
in the same order and all ranks end with bit-identical dense buffers.

The layout and the collective are device-agnostic (the CPU tests run them on ``gloo`` ranks);
``decode``/``decode_apply_momentum`` call the CUDA library and need the plan's GPU.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import torch
import torch.distributed as dist


def _pad4(words: int) -> int:
    return (words + 3) // 4 * 4


class BlockLayout:
    """Word offsets of the three sections inside one rank's block."""

    def __init__(self, total_cap: int, n_tensors: int):
        self.cap = int(total_cap)
        self.n_tensors = int(n_tensors)
        self.cap_pad = _pad4(max(self.cap, 1))
        self.cnt_words = max(2 * self.n_tensors, 1)
        self.off_idx = 0
        self.off_val = self.cap_pad
        self.off_cnt = 2 * self.cap_pad
        self.words = 2 * self.cap_pad + _pad4(self.cnt_words)

    def views(self, block: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """(idx as int32 bit patterns, val as float32, count as int32) views of one block."""
        assert block.dtype == torch.int32 and block.numel() == self.words
        idx = block[self.off_idx:self.off_idx + max(self.cap, 1)]
        val = block[self.off_val:self.off_val + max(self.cap, 1)].view(torch.float32)
        cnt = block[self.off_cnt:self.off_cnt + self.cnt_words]
        return idx, val, cnt


class PairExchange:
    """Send block, receive buffer and the collective for one plan and one process group.

    ``with_counts`` says whether the decode reads the per-tensor counts (threshold mode) or takes
    every list at its fixed length k (top-k mode).
    """

    def __init__(self, total_cap: int, n_tensors: int, with_counts: bool, device, group=None):
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.layout = BlockLayout(total_cap, n_tensors)
        self.with_counts = bool(with_counts)
        self.send = torch.zeros(self.layout.words, dtype=torch.int32, device=device)
        self.recv = torch.zeros(self.world * self.layout.words, dtype=torch.int32, device=device)

    @classmethod
    def for_plan(cls, plan, group=None) -> "PairExchange":
        from . import api
        return cls(plan.total_cap, plan.n_tensors, plan.mode == api.GC_THRESHOLD, f"cuda:{plan.device}", group)

    def outputs(self) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """The (out_idx, out_val, out_count) arguments of this rank's compress call."""
        return self.layout.views(self.send)

    def all_gather(self, async_op: bool = False):
        """Gather every rank's block into ``recv`` (rank order).  A single-process job copies."""
        if self.world == 1 and not dist.is_initialized():
            self.recv.copy_(self.send)
            return None
        return dist.all_gather_into_tensor(self.recv, self.send, group=self.group, async_op=async_op)

    def lists(self) -> Tuple[List[torch.Tensor], List[torch.Tensor], Optional[List[torch.Tensor]]]:
        """Per-worker (idx, val, count) views of the gathered blocks, worker = rank."""
        idx, val, cnt = [], [], []
        L = self.layout.words
        for r in range(self.world):
            i, v, c = self.layout.views(self.recv[r * L:(r + 1) * L])
            idx.append(i); val.append(v); cnt.append(c)
        return idx, val, (cnt if self.with_counts else None)

    def bytes_on_wire_per_rank(self) -> int:
        """Bytes each rank receives from its peers in one exchange."""
        return 4 * self.layout.words * (self.world - 1)

    # --- the two consumers of the gathered lists (CUDA library)
    def decode(self, plan, dense_out: torch.Tensor, zero_first: bool, workspace: torch.Tensor, stream=None) -> int:
        idx, val, cnt = self.lists()
        return plan.decompress_accumulate(idx, val, cnt, dense_out, zero_first, workspace, stream)

    def decode_apply_momentum(self, plan, param: torch.Tensor, velocity: torch.Tensor, lr: float, momentum: float,
                              scale: float, workspace: torch.Tensor, stream=None) -> int:
        idx, val, cnt = self.lists()
        return plan.decompress_apply_momentum(idx, val, cnt, param, velocity, lr, momentum, scale, workspace, stream)
