"""One DQ-SGD communication round on one GPU: buffers plus the library calls.

``Round`` owns the device buffers (torch tensors) of a fixed layout and worker
count and issues norms -> bit rule -> quantize+pack -> unpack+average on the
current stream, or, in the order of Algorithm 1, norms+quantize+pack -> average
with the next bit width chosen on a second stream meanwhile.  It adds no
arithmetic of its own: every step is a kernel of the C-ABI library.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import dq


class Round:
    def __init__(self, seg_elems: Sequence[int], bucket: int, M: int, max_bits: int = 16,
                 device: str = "cuda", worker_stride: Optional[int] = None, norm: int = dq.NORM_L2):
        self.device = torch.device(device)
        self.layout = dq.Layout(seg_elems, bucket, norm).bind(self.device)
        self.M = int(M)
        L = self.layout
        self.stride = L.D32 if worker_stride is None else int(worker_stride)
        self.packed_stride = (L.packed_words(max_bits) + 3) // 4 * 4
        self.norms = torch.empty((M, L.nb), dtype=torch.float32, device=self.device)
        self.packed = torch.empty((M, self.packed_stride), dtype=torch.int32, device=self.device)
        self.out = torch.empty(L.D32, dtype=torch.float32, device=self.device)
        # two (b, s) slots of 16 bytes: the rounds of ``step_fused`` alternate between them, so that
        # the next b can be written while the average still reads the current one
        self._b = torch.zeros((2, 4), dtype=torch.int32, device=self.device)
        self._cur = 0
        self._side = None
        self._ev_norms = None
        self._ev_bits = None
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.scratch_bytes = dq.choose_bits_scratch_bytes(L, M)
        self.scratch = torch.empty(max(self.scratch_bytes, 256), dtype=torch.uint8, device=self.device)
        self.norm_scratch_bytes = dq.tensor_norms_scratch_bytes(L, M)
        self.norm_scratch = (torch.empty(self.norm_scratch_bytes, dtype=torch.uint8, device=self.device)
                             if self.norm_scratch_bytes else None)
        self._host_in = None
        self._host_out = None
        self._dev_in = None

    @property
    def dev_b(self) -> torch.Tensor:
        """The (b, s) slot the calls read and ``bits_`` writes."""
        return self._b[self._cur]

    # ---- the four calls, on device-resident gradients [M, stride] fp32 ----
    def norms_(self, grads) -> None:
        if self.layout.whole_tensor:
            dq.tensor_norms(self.layout, grads, self.stride, self.M, self.norms, self.norm_scratch,
                            self.norm_scratch_bytes, self.status)
        else:
            dq.bucket_norms(self.layout, grads, self.stride, self.M, self.norms, self.status)

    def bits_(self, rule: dq.Rule) -> None:
        dq.choose_bits(self.layout, self.norms, self.M, rule, self.dev_b, self.scratch, self.scratch_bytes,
                       self.status)

    def quantize_(self, grads, seed: int, step: int) -> None:
        dq.quantize_pack(self.layout, grads, self.stride, self.M, self.norms, self.dev_b, seed, step,
                         self.packed, self.packed_stride, self.status)

    def norms_quantize_(self, grads, seed: int, step: int) -> None:
        """Norms and quantize+pack in one pass, with the b already in ``dev_b`` (two passes for a
        whole-tensor layout, whose codes need the norm of the whole tensor)."""
        if self.layout.whole_tensor:
            self.norms_(grads)
            self.quantize_(grads, seed, step)
            return
        dq.norms_quantize_pack(self.layout, grads, self.stride, self.M, self.dev_b, seed, step, self.norms,
                               self.packed, self.packed_stride, self.status)

    def average_(self) -> None:
        dq.unpack_dequant_average(self.layout, self.packed, self.packed_stride, self.norms, self.M, self.dev_b,
                                  self.out, self.status)

    def update_(self, params, lr: float) -> None:
        """``params <- params - lr * average`` (Eq. 2) from the packed codes; the average itself is not stored."""
        dq.unpack_average_update(self.layout, self.packed, self.packed_stride, self.norms, self.M, self.dev_b, lr,
                                 params, self.status)

    def step(self, grads, rule: dq.Rule, seed: int, step: int) -> torch.Tensor:
        """Whole round on device gradients; returns the averaged gradient [D32] (device)."""
        self.norms_(grads)
        self.bits_(rule)
        self.quantize_(grads, seed, step)
        self.average_()
        return self.out

    # below this many norms the bit rule takes a few microseconds and the hand-over between two
    # streams costs more than running it behind the average on the same stream
    OVERLAP_MIN_NORMS = 1 << 20

    def step_fused(self, grads, next_rule: dq.Rule, seed: int, step: int, overlap: Optional[bool] = None,
                   events=None, params=None, lr: float = 0.0) -> torch.Tensor:
        """One round in the order of Algorithm 1: quantize with the b chosen after the
        previous round (one pass over the gradients), average, and choose the next b from
        this round's norms.  ``dev_b`` must hold a b (a first call to ``bits_`` with the
        initial b_0 does that); on return it holds the next one.

        With ``overlap`` the bit rule runs on a second stream next to the average: it needs
        only the norms, and writes the other (b, s) slot.  The current stream waits for it
        before it goes on.  ``overlap=None`` decides by size: a second stream for
        ``OVERLAP_MIN_NORMS`` norms or more, one stream below (measured on the ResNet-18
        shape, 175k norms: 102.5 us per step on one stream, 104.2 us with two; at 4.2M
        norms the second stream hides 85 us of bit rule).  ``events`` = (e0, e1, e2, s0, s1) are recorded around the three
        calls (e* on the current stream, s* around the bit rule on its own stream).

        With ``params`` (fp32 [D32] in the padded layout) the server step also applies the
        update of Eq. 2, ``params <- params - lr * average``, in the same kernel; ``out`` is
        then not written and ``params`` is returned.
        """
        def server_step():
            if params is None:
                self.average_()
            else:
                self.update_(params, lr)
        result = self.out if params is None else params
        if overlap is None:
            overlap = self.M * self.layout.nb >= self.OVERLAP_MIN_NORMS
        main = torch.cuda.current_stream(self.device)
        if events:
            events[0].record(main)
        self.norms_quantize_(grads, seed, step)
        if events:
            events[1].record(main)
        if not overlap:
            server_step()
            if events:
                events[2].record(main)
                events[3].record(main)
            self.bits_(next_rule)
            if events:
                events[4].record(main)
            return result
        if self._side is None:
            self._side = torch.cuda.Stream(self.device)
            self._ev_norms = torch.cuda.Event()
            self._ev_bits = torch.cuda.Event()
        self._ev_norms.record(main)
        self._side.wait_event(self._ev_norms)
        if events:
            events[3].record(self._side)
        dq.choose_bits(self.layout, self.norms, self.M, next_rule, self._b[1 - self._cur], self.scratch,
                       self.scratch_bytes, self.status, stream=self._side)
        if events:
            events[4].record(self._side)
        self._ev_bits.record(self._side)
        server_step()                        # reads the current slot
        if events:
            events[2].record(main)
        main.wait_event(self._ev_bits)
        self._cur = 1 - self._cur
        return result

    def step_host(self, host_grads: torch.Tensor, next_rule: dq.Rule, seed: int, step: int) -> torch.Tensor:
        """``step_fused`` on pinned host gradients [M, stride]; returns a pinned host tensor [D32].

        The gradients travel to the device on a copy stream, the round runs on the current
        stream and the average travels back on a second copy stream, with two device input
        buffers and two host output buffers used in turn: in a loop of calls the upload of
        step i + 1 runs beside the round and the download of step i (the link is full duplex).
        The caller synchronises before it reads the returned tensor, leaves ``host_grads``
        untouched until then, and finds the result of a call intact until the call after next.
        """
        if self._dev_in is None:
            self._dev_in = [torch.empty((self.M, self.stride), dtype=torch.float32, device=self.device) for _ in range(2)]
            self._host_out = [torch.empty(self.layout.D32, dtype=torch.float32).pin_memory() for _ in range(2)]
            self._s_in = torch.cuda.Stream(self.device)
            self._s_out = torch.cuda.Stream(self.device)
            self._ev_in = [torch.cuda.Event() for _ in range(2)]       # upload into buffer i has landed
            self._ev_used = [torch.cuda.Event() for _ in range(2)]     # the round that read buffer i is done
            self._ev_avg = torch.cuda.Event()                           # this round's average is in self.out
            self._ev_out = torch.cuda.Event()                           # the last download has left self.out
            self._host_calls = 0
        i = self._host_calls % 2
        self._host_calls += 1
        main = torch.cuda.current_stream(self.device)
        self._s_in.wait_event(self._ev_used[i])          # (a wait on an event never recorded returns at once)
        with torch.cuda.stream(self._s_in):
            self._dev_in[i].copy_(host_grads, non_blocking=True)
            self._ev_in[i].record(self._s_in)
        main.wait_event(self._ev_in[i])
        main.wait_event(self._ev_out)                    # the previous average has been read out of self.out
        self.step_fused(self._dev_in[i], next_rule, seed, step)
        self._ev_used[i].record(main)
        self._ev_avg.record(main)
        self._s_out.wait_event(self._ev_avg)
        with torch.cuda.stream(self._s_out):
            self._host_out[i].copy_(self.out, non_blocking=True)
            self._ev_out.record(self._s_out)
        return self._host_out[i]

    def join_host(self) -> None:
        """Makes the current stream wait (on the device) for the last download ``step_host`` queued."""
        if self._dev_in is not None:
            torch.cuda.current_stream(self.device).wait_event(self._ev_out)

    def sync_host(self) -> None:
        """Waits for everything ``step_host`` has queued (its copy streams included)."""
        if self._dev_in is not None:
            self._s_in.synchronize()
            self._s_out.synchronize()
        torch.cuda.current_stream(self.device).synchronize()

    def bits(self) -> int:
        """b chosen by the last bits_ call (synchronises)."""
        return int(self.dev_b[0].item())

    def read_status(self) -> int:
        return int(self.status.item())
