"""Randomised layouts through the whole CUDA path against the oracle.

Tensor lists with empty, tiny and large tensors, every kind of bucket size (32 * 2^k and not),
odd worker counts, padded worker strides and all bit widths: the cases where tiles straddle
tensor ends, buckets are short and the regular-tile shortcuts must hand over to the general
routes.  Seeds are fixed; tolerances are those of test_gpu_parity.py.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_14575_b200 import dq

pytestmark = pytest.mark.gpu

BUCKETS = [32, 64, 96, 128, 160, 256, 512, 1024, 2048, 4096]


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


def _case(seed):
    rng = np.random.default_rng(1000 + seed)
    n_seg = int(rng.integers(1, 13))
    kinds = rng.integers(0, 6, size=n_seg)
    segs = []
    for k in kinds:
        segs.append(int({0: 0, 1: rng.integers(1, 40), 2: rng.integers(40, 700), 3: rng.integers(700, 6000),
                         4: rng.integers(6000, 40000), 5: rng.integers(40000, 150000)}[int(k)]))
    if sum(segs) == 0:
        segs[0] = 77
    bucket = int(BUCKETS[rng.integers(0, len(BUCKETS))])
    M = int([1, 2, 3, 5, 8][rng.integers(0, 5)])
    b = int(rng.integers(1, 17))
    extra = int(rng.integers(0, 3)) * 32
    return rng, segs, bucket, M, b, extra


@pytest.mark.parametrize("seed", range(40))
def test_random_layout_whole_path(G, seed):
    rng, segs, bucket, M, b, extra = _case(seed)
    ref = oracle.Layout(segs, bucket)
    stride = ref.D32 + extra
    g = np.full((M, stride), np.float32(1e30), np.float32)          # padding and the stride's slack hold garbage
    for i, n in enumerate(segs):
        scale = 10.0 ** rng.uniform(-6, 3)
        g[:, ref.offsets[i]: ref.offsets[i] + n] = (rng.standard_normal((M, n)) * scale).astype(np.float32)
    r = G.GpuRound(segs, bucket, M, stride=stride)
    r.set_grads(g)

    want_norms = oracle.bucket_norms(ref, g)
    norms = r.norms().copy()
    np.testing.assert_allclose(norms, want_norms, rtol=1e-6, atol=0)

    r.set_b(b)
    nw = ref.packed_words(b)
    packed = r.quantize(seed, 3, fill=-1).copy()
    assert np.array_equal(packed[:, :nw], oracle.quantize_pack(ref, g, norms, b, seed, 3))
    assert np.all(packed[:, nw:] == 0xFFFFFFFF)

    norms_f, packed_f = r.norms_quantize(seed, 3, fill=-1)
    assert np.array_equal(norms_f, norms) and np.array_equal(packed_f, packed)

    out = r.average(fill=7.0)
    want = oracle.unpack_dequant_average(ref, packed[:, :nw], norms, b)
    assert G.rel_l2(out, want) <= 1e-6
    valid = np.zeros(ref.D32, bool)
    for i, n in enumerate(segs):
        valid[ref.offsets[i]: ref.offsets[i] + n] = True
    assert np.all(out[~valid] == 0)

    x = rng.standard_normal(ref.D32).astype(np.float32)
    lr = 0.25
    got = r.update(lr, x)
    want_x = oracle.unpack_average_update(ref, packed[:, :nw], norms, b, lr, x)
    tol = 1e-6 * lr * max(float(np.abs(want).max()), 1e-30) + 2.0 ** -23 * np.abs(want_x) + 1e-30
    assert np.all(np.abs(got.astype(np.float64) - want_x) <= tol)
    assert np.array_equal(got[~valid], x[~valid])
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("seed", range(40, 64))
def test_random_layout_norm_family_and_slices(G, seed):
    """The same random layouts with the l_inf norm or one norm per tensor, a worker offset, and the
    average taken range by range on slices of the layout: all must reproduce the oracle / the
    whole-layout result."""
    rng, segs, bucket, M, b, _ = _case(seed)
    linf = bool(rng.integers(0, 2))
    whole = bool(rng.integers(0, 3) == 0)
    first = int(rng.integers(0, 50))
    kind_g, kind_o = (dq.NORM_LINF, oracle.NORM_LINF) if linf else (dq.NORM_L2, oracle.NORM_L2)
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs) if whole else bucket)
    g = np.zeros((first + M, ref.D32), np.float32)
    for i, n in enumerate(segs):
        scale = 10.0 ** rng.uniform(-4, 2)
        g[:, ref.offsets[i]: ref.offsets[i] + n] = (rng.standard_normal((first + M, n)) * scale).astype(np.float32)
    r = G.GpuRound(segs, dq.BUCKET_WHOLE_TENSOR if whole else bucket, M, norm=kind_g)
    assert r.lay.nb == ref.nb
    r.set_grads(np.ascontiguousarray(g[first:]))
    want_norms = oracle.bucket_norms(ref, g, kind_o)
    norms = r.norms().copy()
    if linf:
        assert np.array_equal(norms, want_norms[first:])
    else:
        np.testing.assert_allclose(norms, want_norms[first:], rtol=1e-6, atol=0)

    # words of workers first .. first + M - 1 with the GPU's norms in their rows of the oracle's call
    all_norms = want_norms.copy()
    all_norms[first:] = norms
    want = oracle.quantize_pack(ref, g, all_norms, b, seed, 11)[first:]
    r.set_b(b)
    nw = ref.packed_words(b)
    dq.quantize_pack_worker(r.lay, r.grads, r.stride, M, r.g_norms.view, r.g_b.view, seed, 11, first,
                            r.g_packed.view, r.pstride, r.status)
    packed = r.g_packed.view.cpu().numpy().view(np.uint32).reshape(M, r.pstride).copy()
    assert np.array_equal(packed[:, :nw], want)
    if not whole:
        dq.norms_quantize_pack_worker(r.lay, r.grads, r.stride, M, r.g_b.view, seed, 11, first, r.g_norms.view,
                                      r.g_packed.view, r.pstride, r.status)
        assert np.array_equal(r.g_packed.view.cpu().numpy().view(np.uint32).reshape(M, r.pstride)[:, :nw], want)
        assert np.array_equal(r.g_norms.view.cpu().numpy().reshape(M, ref.nb), norms)

    out = r.average(fill=-3.0).copy()
    assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, norms, b)) <= 1e-6

    # the average over 1..4 ranges of whole buckets, each through its slice layout, is the same array
    n_shards = int(rng.integers(1, 5))
    bounds = r.lay.shard_bounds(n_shards)
    pieces = np.full(ref.D32, np.float32(9.0), np.float32)
    dev_packed = r.g_packed.view.view(torch.int32).reshape(M, r.pstride)
    dev_norms = r.g_norms.view.reshape(M, ref.nb)
    for j in range(n_shards):
        k0, k1 = bounds[j], bounds[j + 1]
        if k0 == k1:
            continue
        sub, f0 = r.lay.slice(k0, k1)
        sub.bind()
        w0, wn = b * f0 // 32, b * sub.D32 // 32
        rs = (wn + 3) // 4 * 4 + 4
        sub_packed = torch.zeros((M, rs), dtype=torch.int32, device="cuda")
        sub_packed[:, :wn].copy_(dev_packed[:, w0: w0 + wn])
        sub_norms = dev_norms[:, k0:k1].contiguous()
        sub_out = G.Guarded(sub.D32, torch.float32)
        dq.unpack_dequant_average(sub, sub_packed, rs, sub_norms, M, r.g_b.view, sub_out.view, r.status)
        pieces[f0: f0 + sub.D32] = sub_out.view.cpu().numpy()
        assert sub_out.intact()
    assert np.array_equal(pieces, out)
    assert r.read_status() == 0 and r.guards_intact()
