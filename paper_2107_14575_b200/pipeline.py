"""One DQ-SGD communication round on one GPU: buffers plus the four library calls.

``Round`` owns the device buffers (torch tensors) of a fixed layout and worker
count and issues norms -> bit rule -> quantize+pack -> unpack+average on the
current stream.  It adds no arithmetic of its own: every step is a kernel of
the C-ABI library.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import dq


class Round:
    def __init__(self, seg_elems: Sequence[int], bucket: int, M: int, max_bits: int = 16,
                 device: str = "cuda", worker_stride: Optional[int] = None):
        self.device = torch.device(device)
        self.layout = dq.Layout(seg_elems, bucket).bind(self.device)
        self.M = int(M)
        L = self.layout
        self.stride = L.D32 if worker_stride is None else int(worker_stride)
        self.packed_stride = (L.packed_words(max_bits) + 3) // 4 * 4
        self.norms = torch.empty((M, L.nb), dtype=torch.float32, device=self.device)
        self.packed = torch.empty((M, self.packed_stride), dtype=torch.int32, device=self.device)
        self.out = torch.empty(L.D32, dtype=torch.float32, device=self.device)
        self.dev_b = torch.zeros(2, dtype=torch.int32, device=self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.scratch_bytes = dq.choose_bits_scratch_bytes(L, M)
        self.scratch = torch.empty(max(self.scratch_bytes, 256), dtype=torch.uint8, device=self.device)
        self._host_in = None
        self._host_out = None
        self._dev_in = None

    # ---- the four calls, on device-resident gradients [M, stride] fp32 ----
    def norms_(self, grads) -> None:
        dq.bucket_norms(self.layout, grads, self.stride, self.M, self.norms, self.status)

    def bits_(self, rule: dq.Rule) -> None:
        dq.choose_bits(self.layout, self.norms, self.M, rule, self.dev_b, self.scratch, self.scratch_bytes,
                       self.status)

    def quantize_(self, grads, seed: int, step: int) -> None:
        dq.quantize_pack(self.layout, grads, self.stride, self.M, self.norms, self.dev_b, seed, step,
                         self.packed, self.packed_stride, self.status)

    def norms_quantize_(self, grads, seed: int, step: int) -> None:
        """Norms and quantize+pack in one pass, with the b already in ``dev_b``."""
        dq.norms_quantize_pack(self.layout, grads, self.stride, self.M, self.dev_b, seed, step, self.norms,
                               self.packed, self.packed_stride, self.status)

    def average_(self) -> None:
        dq.unpack_dequant_average(self.layout, self.packed, self.packed_stride, self.norms, self.M, self.dev_b,
                                  self.out, self.status)

    def step(self, grads, rule: dq.Rule, seed: int, step: int) -> torch.Tensor:
        """Whole round on device gradients; returns the averaged gradient [D32] (device)."""
        self.norms_(grads)
        self.bits_(rule)
        self.quantize_(grads, seed, step)
        self.average_()
        return self.out

    def step_fused(self, grads, next_rule: dq.Rule, seed: int, step: int) -> torch.Tensor:
        """One round in the order of Algorithm 1: quantize with the b chosen after the
        previous round (one pass over the gradients), average, then choose the next b from
        this round's norms.  ``dev_b`` must hold a b (a first call to ``bits_`` with the
        initial b_0 does that)."""
        self.norms_quantize_(grads, seed, step)
        self.average_()
        self.bits_(next_rule)
        return self.out

    def step_host(self, host_grads: torch.Tensor, next_rule: dq.Rule, seed: int, step: int) -> torch.Tensor:
        """``step_fused`` on pinned host gradients [M, stride]; returns a pinned host tensor [D32].

        Copies the gradients to the device, runs the round and copies the
        average back, all on the current stream; the caller synchronises.
        """
        if self._dev_in is None:
            self._dev_in = torch.empty((self.M, self.stride), dtype=torch.float32, device=self.device)
            self._host_out = torch.empty(self.layout.D32, dtype=torch.float32).pin_memory()
        self._dev_in.copy_(host_grads, non_blocking=True)
        self.step_fused(self._dev_in, next_rule, seed, step)
        self._host_out.copy_(self.out, non_blocking=True)
        return self._host_out

    def bits(self) -> int:
        """b chosen by the last bits_ call (synchronises)."""
        return int(self.dev_b[0].item())

    def read_status(self) -> int:
        return int(self.status.item())
