"""Algorithm 1 with one worker per GPU: the "send / collect / average" steps cut across ranks.

Every rank quantizes its own gradient over the whole layout (worker index = rank).  The
padded buffer is cut into ``world`` contiguous ranges of whole buckets
(``dq_layout_shard_bounds``); rank r receives range r of every rank's packed words
(an all-to-all), averages the ``world`` workers over that range with the slice layout
(``dq_layout_slice``) and the ranks put their ranges together again (an all-gather).  The
norms travel whole (they are small): every rank sees all of them, so the bit rule gives
the same b everywhere without a reduction of its own.  All arithmetic is the C-ABI
library's; this module moves bytes.

Two transports carry the exchange.  ``DistTransport`` uses ``torch.distributed`` (NCCL
between GPUs, gloo between CPU processes); received data lands in this rank's own memory
and is read from there by ordinary loads and bulk copies.  ``LoopbackTransport`` holds
all ranks in one process and copies between their buffers, so that the whole sharded path
can be run, rank after rank, on a single GPU.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import dq


class ShardPlan:
    """Which buckets, elements and packed words each rank averages."""

    def __init__(self, layout: dq.Layout, world: int):
        self.world = int(world)
        self.bounds = layout.shard_bounds(self.world)
        self.first_elem: List[int] = []
        self.n_elems: List[int] = []
        self.slices: List[Optional[dq.Layout]] = []
        for r in range(self.world):
            k0, k1 = self.bounds[r], self.bounds[r + 1]
            if k1 > k0:
                sub, first = layout.slice(k0, k1)
                self.slices.append(sub)
                self.first_elem.append(first)
                self.n_elems.append(sub.D32)
            else:                                    # fewer buckets than ranks: this rank averages nothing
                self.slices.append(None)
                self.first_elem.append(self.first_elem[-1] + self.n_elems[-1] if r else 0)
                self.n_elems.append(0)
        assert sum(self.n_elems) == layout.D32

    def buckets(self, r: int):
        return self.bounds[r], self.bounds[r + 1]

    def word_range(self, r: int, b: int):
        """First word and number of words of range r in a worker's packed stream at b bits."""
        return b * self.first_elem[r] // 32, b * self.n_elems[r] // 32

    def max_elems(self) -> int:
        return max(self.n_elems)


class DistTransport:
    """The exchange over ``torch.distributed`` (any backend that has all_to_all_single and all_gather)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self._stage = None

    def gather_rows(self, row: torch.Tensor, all_rows: torch.Tensor) -> None:
        """all_rows[q] <- rank q's row (rows of equal length)."""
        self.dist.all_gather_into_tensor(all_rows.view(-1), row.contiguous().view(-1), group=self.group)

    def exchange(self, send: torch.Tensor, send_ranges: Sequence, recv: torch.Tensor, recv_len: int) -> None:
        """recv[q, :recv_len] <- elements send_ranges[self.rank] of rank q's ``send``; rank q gets
        send[send_ranges[q]] of this rank.  ``send_ranges`` = (start, length) per destination, contiguous
        and ascending, so the send side needs no staging.  The receive side lands straight in ``recv``
        when its rows are exactly ``recv_len`` long; otherwise the rows of ``recv`` keep their aligned
        stride and the data passes through a staging buffer that is allocated once and reused."""
        world = self.world
        lo = send_ranges[0][0]
        hi = send_ranges[-1][0] + send_ranges[-1][1]
        flat_in = send.view(-1)[lo:hi]
        direct = recv.is_contiguous() and recv.shape[1] == recv_len
        if direct:
            flat_out = recv.view(-1)
        else:
            need = world * recv.shape[1]
            if (self._stage is None or self._stage.numel() < need or self._stage.dtype != send.dtype
                    or self._stage.device != send.device):
                self._stage = torch.empty(need, dtype=send.dtype, device=send.device)
            flat_out = self._stage[: world * recv_len]
        self.dist.all_to_all_single(flat_out, flat_in, output_split_sizes=[recv_len] * world,
                                    input_split_sizes=[n for _, n in send_ranges], group=self.group)
        if not direct:
            recv[:, :recv_len].copy_(flat_out.view(world, recv_len))


class LoopbackTransport:
    """All ranks in one process: the collectives become copies between the ranks' buffers.

    Each collective is called once per rank like the real one; a rank's call deposits its
    contribution and the last rank's call delivers everything."""

    def __init__(self, world: int):
        self.world = int(world)
        self._rows = {}
        self._ex = {}

    def bind(self, rank: int) -> "_LoopbackEnd":
        return _LoopbackEnd(self, rank)


class _LoopbackEnd:
    def __init__(self, hub: LoopbackTransport, rank: int):
        self.hub, self.rank, self.world = hub, rank, hub.world

    def gather_rows(self, row, all_rows) -> None:
        h = self.hub
        h._rows[self.rank] = (row, all_rows)
        if len(h._rows) == self.world:
            for q in range(self.world):
                for r in range(self.world):
                    h._rows[r][1][q].view(-1).copy_(h._rows[q][0].view(-1))
            h._rows = {}

    def exchange(self, send, send_ranges, recv, recv_len) -> None:
        h = self.hub
        h._ex[self.rank] = (send, send_ranges, recv, recv_len)
        if len(h._ex) == self.world:
            for q in range(self.world):                     # sender
                send_q, ranges_q, _, _ = h._ex[q]
                for r in range(self.world):                 # receiver
                    start, n = ranges_q[r]
                    recv_r = h._ex[r][2]
                    assert n == h._ex[r][3]
                    recv_r[q, :n].copy_(send_q.view(-1)[start: start + n])
            h._ex = {}


class ShardedRound:
    """One rank of the sharded path.  ``grad`` is this rank's gradient [D32] in the padded layout.

    The steps of a round, in order (each a method so that a single process can drive several
    ranks turn by turn): ``quantize_`` (local norms and packed words), ``share_norms_`` and
    ``exchange_`` (the two collectives), ``average_`` (this rank's range), ``gather_`` and ``assemble_`` (the
    ranges collected and put in place), ``bits_`` (b for the next round, the same on every rank).  ``step`` runs them all.
    The bit width is passed in as a host integer: the sizes of the all-to-all depend on it.
    """

    def __init__(self, seg_elems: Sequence[int], bucket: int, transport, rank: int, world: int,
                 max_bits: int = 16, device: str = "cuda", norm: int = dq.NORM_L2):
        self.device = torch.device(device)
        self.rank, self.world = int(rank), int(world)
        self.t = transport
        self.layout = dq.Layout(seg_elems, bucket, norm).bind(self.device)
        L = self.layout
        self.plan = ShardPlan(L, world)
        self.sub = self.plan.slices[self.rank]
        if self.sub is not None:
            self.sub.bind(self.device)
        self.n_mine = self.plan.n_elems[self.rank]
        k0, k1 = self.plan.buckets(self.rank)
        self.k0, self.k1 = k0, k1
        i32, f32 = torch.int32, torch.float32
        self.pstride = (L.packed_words(max_bits) + 3) // 4 * 4
        self.rstride = max(4, (max_bits * self.n_mine // 32 + 3) // 4 * 4)
        self.norms_local = torch.zeros((1, L.nb), dtype=f32, device=self.device)
        self.norms_all = torch.zeros((world, L.nb), dtype=f32, device=self.device)
        self.norms_mine = torch.zeros((world, max(k1 - k0, 1)), dtype=f32, device=self.device)
        self.packed_local = torch.zeros(self.pstride, dtype=i32, device=self.device)
        self.packed_recv = torch.zeros((world, self.rstride), dtype=i32, device=self.device)
        self.out_mine = torch.zeros(max(self.n_mine, 32), dtype=f32, device=self.device)
        self.out_pad = torch.zeros(self.plan.max_elems(), dtype=f32, device=self.device)
        self.out_all = torch.zeros((world, self.plan.max_elems()), dtype=f32, device=self.device)
        self.out = torch.zeros(L.D32, dtype=f32, device=self.device)
        self.dev_b = torch.zeros(4, dtype=i32, device=self.device)
        self.status = torch.zeros(1, dtype=i32, device=self.device)
        self.scratch_bytes = dq.choose_bits_scratch_bytes(L, world)
        self.scratch = torch.empty(max(self.scratch_bytes, 256), dtype=torch.uint8, device=self.device)
        self.norm_scratch_bytes = dq.tensor_norms_scratch_bytes(L, 1)
        self.norm_scratch = (torch.empty(self.norm_scratch_bytes, dtype=torch.uint8, device=self.device)
                             if self.norm_scratch_bytes else None)

    def set_bits(self, b: int) -> None:
        """Puts (b, s) into ``dev_b``: the library's bit rule with a fixed b writes both numbers."""
        dq.choose_bits(self.layout, self.norms_all, self.world, dq.Rule.fixed(b), self.dev_b, self.scratch,
                       self.scratch_bytes, self.status)

    def quantize_(self, grad: torch.Tensor, seed: int, step: int) -> None:
        if self.layout.whole_tensor:             # one norm per tensor: norms first, then the codes
            dq.tensor_norms(self.layout, grad, self.layout.D32, 1, self.norms_local, self.norm_scratch,
                            self.norm_scratch_bytes, self.status)
            dq.quantize_pack_worker(self.layout, grad, self.layout.D32, 1, self.norms_local, self.dev_b, seed, step,
                                    self.rank, self.packed_local, self.pstride, self.status)
            return
        dq.norms_quantize_pack_worker(self.layout, grad, self.layout.D32, 1, self.dev_b, seed, step, self.rank,
                                      self.norms_local, self.packed_local, self.pstride, self.status)

    def share_norms_(self) -> None:
        self.t.gather_rows(self.norms_local, self.norms_all)

    def exchange_(self, b: int) -> None:
        ranges = [self.plan.word_range(q, b) for q in range(self.world)]
        self.t.exchange(self.packed_local, ranges, self.packed_recv, ranges[self.rank][1])

    def average_(self) -> None:
        if self.sub is None:
            return
        self.norms_mine.copy_(self.norms_all[:, self.k0: self.k1])
        dq.unpack_dequant_average(self.sub, self.packed_recv, self.rstride, self.norms_mine, self.world, self.dev_b,
                                  self.out_mine, self.status)

    def gather_(self) -> None:
        self.out_pad[: self.n_mine].copy_(self.out_mine[: self.n_mine])
        self.t.gather_rows(self.out_pad, self.out_all)

    def assemble_(self) -> None:
        for q in range(self.world):
            n = self.plan.n_elems[q]
            if n:
                f = self.plan.first_elem[q]
                self.out[f: f + n].copy_(self.out_all[q, :n])

    def bits_(self, rule: dq.Rule) -> None:
        dq.choose_bits(self.layout, self.norms_all, self.world, rule, self.dev_b, self.scratch, self.scratch_bytes,
                       self.status)

    def step(self, grad: torch.Tensor, b: int, seed: int, step: int, next_rule: Optional[dq.Rule] = None):
        """One round with bit width ``b`` (what ``dev_b`` holds); returns the averaged gradient [D32]."""
        self.quantize_(grad, seed, step)
        self.share_norms_()
        self.exchange_(b)
        self.average_()
        self.gather_()
        self.assemble_()
        if next_rule is not None:
            self.bits_(next_rule)
        return self.out

    def read_bits(self) -> int:
        return int(self.dev_b[0].item())

    def read_status(self) -> int:
        return int(self.status.item())
