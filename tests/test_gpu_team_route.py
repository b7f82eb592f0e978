"""GPU parity of the fused quantizer's route for buckets of 2048 and 4096 elements.

A team of two or four warps shares every bucket, one 1024-element tile per warp.  The layouts
here are chosen for what that route has to get right besides the common case: tensors much
shorter than a bucket (most warps of the team have an empty share), tensors that end inside a
warp's tile or exactly on its edge, a single bucket (more teams than buckets), and ranges of a
team that cross from one worker to the next.  Norms are compared with the oracle's, words bit
for bit with the oracle's when it is driven with the GPU's norms, and the separate passes must
give the same norms and words.
"""
import zlib

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

SEED = 0x7EA3_0F_3A7C


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


LAYOUTS = {
    "one-short-bucket": [100],
    "one-full-bucket": [4096],
    "tiny-tensors": [1, 7, 32, 33, 64, 5, 1000, 1023, 1024, 1025, 2047, 2048, 2049, 3, 3071, 3072, 3073, 4095, 4097],
    "edges": [1024, 2048, 3072, 4096, 5120, 8192 + 1024, 8192 + 1],
    "long-and-short": [9 * 4096 + 1500, 12, 5 * 4096, 1, 7 * 4096 + 4095],
    "with-empty-tensors": [0, 2048, 0, 0, 4096 + 17, 0],
}


@pytest.mark.parametrize("b", [2, 5, 8, 16])
@pytest.mark.parametrize("bucket", [2048, 4096])
@pytest.mark.parametrize("name", sorted(LAYOUTS))
def test_team_route_matches_the_oracle(G, name, bucket, b):
    segs = LAYOUTS[name]
    M = 3
    ref = oracle.Layout(segs, bucket)
    rng = np.random.default_rng(zlib.crc32(("%s/%d/%d" % (name, bucket, b)).encode()))
    g = np.full((M, ref.D32), 3e30, np.float32)                  # padding holds a value that must be ignored
    for o, n in zip(ref.offsets, segs):
        g[:, o: o + n] = (rng.standard_normal((M, n)) * rng.choice([1e-3, 1.0, 50.0])).astype(np.float32)
    if ref.nb > 1:                                                 # one bucket of zeros
        k = int(rng.integers(0, ref.nb))
        g[1, int(ref.bucket_start[k]): int(ref.bucket_start[k]) + int(ref.bucket_len[k])] = 0.0
    r = G.GpuRound(segs, bucket, M)
    r.set_grads(g)
    r.set_b(b)
    norms, packed = r.norms_quantize(SEED, 11, fill=-1)
    norms, packed = norms.copy(), packed.copy()
    want_norms = oracle.bucket_norms(ref, g)
    assert np.all(np.abs(norms.astype(np.float64) - want_norms) <= 1e-6 * want_norms.astype(np.float64))
    nw = ref.packed_words(b)
    want = oracle.quantize_pack(ref, g, norms, b, SEED, 11)
    assert np.array_equal(packed[:, :nw], want)
    assert np.all(packed[:, nw:] == 0xFFFFFFFF)                    # nothing written past the stream
    assert r.read_status() == 0 and r.guards_intact()
    # the two separate passes: identical norms and words
    assert np.array_equal(r.norms(), norms)
    assert np.array_equal(r.quantize(SEED, 11)[:, :nw], want)
    # and the average of those words
    out = r.average(fill=1e30)
    ref_out = oracle.unpack_dequant_average(ref, want, norms, b)
    assert G.rel_l2(out, ref_out) <= 1e-6
    assert r.read_status() == 0 and r.guards_intact()
