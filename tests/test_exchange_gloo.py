"""The sharded path's plumbing on CPU: shard plans against the layout, and the two collectives
of ``exchange.DistTransport`` between two gloo ranks (rendezvous on 127.0.0.1).  No kernel runs
here; what the ranks exchange are tagged integers, so a misplaced range shows up as a wrong tag."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2107_14575_b200 import dq, exchange

RAGGED = [70, 32, 1, 100, 4097, 31, 0, 64, 1000, 5, 12345]


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("segs,bucket,world", [(RAGGED, 64, 4), (RAGGED, 4096, 3), ([1 << 16], 512, 8),
                                               ([100], 32, 8), (RAGGED, dq.BUCKET_WHOLE_TENSOR, 2)])
def test_shard_plan_tiles_the_layout(dqlib, segs, bucket, world):
    lay = dq.Layout(segs, bucket)
    plan = exchange.ShardPlan(lay, world)
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs) if bucket == 0 else bucket)
    assert plan.bounds[0] == 0 and plan.bounds[-1] == lay.nb == ref.nb
    assert all(a <= b for a, b in zip(plan.bounds, plan.bounds[1:]))
    pos = 0
    for r in range(world):
        k0, k1 = plan.buckets(r)
        assert plan.first_elem[r] == pos
        if k1 > k0:
            sub = plan.slices[r]
            assert pos == int(ref.bucket_start[k0]) and sub.nb == k1 - k0
            for j in (0, (k1 - k0) // 2, k1 - k0 - 1):           # bucket j of the slice is bucket k0 + j
                s0, n0 = sub.bucket_range(j)
                assert (s0 + pos, n0) == (int(ref.bucket_start[k0 + j]), int(ref.bucket_len[k0 + j]))
        else:
            assert plan.n_elems[r] == 0 and plan.slices[r] is None
        for b in (1, 5, 16):                                     # the words of a range are contiguous
            w0, wn = plan.word_range(r, b)
            assert w0 == b * pos // 32 and wn == b * plan.n_elems[r] // 32
        pos += plan.n_elems[r]
    assert pos == lay.D32
    if lay.nb >= 8 * world:                                      # balance: no shard above twice the mean
        assert max(plan.n_elems) <= 2 * lay.D32 / world + 2 * max(lay.bucket, 4096)


def test_slice_errors(dqlib):
    lay = dq.Layout(RAGGED, 64)
    for k0, k1 in ((-1, 3), (3, 3), (5, 2), (0, lay.nb + 1)):
        with pytest.raises(dq.DQError) as e:
            lay.slice(k0, k1)
        assert e.value.code == dq.ERR_RANGE
    with pytest.raises(dq.DQError):
        lay.shard_bounds(0)


def _worker(rank: int, world: int, port: int, out_dir: str) -> None:
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lay = dq.Layout(RAGGED, 64)
        plan = exchange.ShardPlan(lay, world)
        t = exchange.DistTransport()
        assert (t.rank, t.world) == (rank, world)
        for b in (3, 8):
            nw = lay.packed_words(b)
            # word i of rank q's stream carries the tag q * 2^24 + i
            send = (torch.arange(nw + 5, dtype=torch.int32) + (rank << 24))
            ranges = [plan.word_range(q, b) for q in range(world)]
            mine = ranges[rank][1]
            recv = torch.full((world, (mine + 3) // 4 * 4 + 4), -1, dtype=torch.int32)
            t.exchange(send, ranges, recv, mine)
            w0 = ranges[rank][0]
            for q in range(world):
                want = torch.arange(w0, w0 + mine, dtype=torch.int32) + (q << 24)
                assert torch.equal(recv[q, :mine], want), (rank, q, b)
                assert torch.all(recv[q, mine:] == -1)             # nothing beyond the range is touched
        row = torch.full((1, 7), float(rank + 1))
        rows = torch.zeros((world, 7))
        t.gather_rows(row, rows)
        assert torch.equal(rows, torch.arange(1, world + 1, dtype=torch.float32)[:, None].expand(world, 7))
        open(os.path.join(out_dir, "ok%d" % rank), "w").write("ok")
    finally:
        dist.barrier()
        dist.destroy_process_group()


def test_two_gloo_ranks_exchange_their_ranges(dqlib, tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok0").exists() and (tmp_path / "ok1").exists()


def test_loopback_transport_matches_the_collectives_definition():
    world = 3
    hub = exchange.LoopbackTransport(world)
    ends = [hub.bind(r) for r in range(world)]
    ranges = [(0, 4), (4, 2), (6, 6)]
    sends = [torch.arange(12, dtype=torch.int32) + 100 * q for q in range(world)]
    recvs = [torch.full((world, 8), -1, dtype=torch.int32) for _ in range(world)]
    for r in range(world):
        ends[r].exchange(sends[r], ranges, recvs[r], ranges[r][1])
    for r in range(world):
        st, n = ranges[r]
        for q in range(world):
            assert torch.equal(recvs[r][q, :n], sends[q][st: st + n])
            assert torch.all(recvs[r][q, n:] == -1)
    rows = [torch.zeros((world, 2)) for _ in range(world)]
    for r in range(world):
        ends[r].gather_rows(torch.full((2,), float(r)), rows[r])
    for r in range(world):
        assert torch.equal(rows[r][:, 0], torch.arange(world, dtype=torch.float32))
