"""The allocation-free bit rule (``dq_choose_bits_noalloc``) against ``dq_choose_bits``.

Some users of the library cannot hand it a scratch buffer: their device memory was
divided up once at start-up (a caching allocator or a fixed budget owns all of it), or
they sit on a path where ``cudaMalloc`` is ruled out because it stalls the device for an
unpredictable time.  For them the library carries its own 64 KB of scratch.  This test
drives both entry points through the C ABI with the same inputs and expects the same
``(b, s)`` -- integers, so the comparison is exact -- on two calls in a row, the second
with different norms and rule so that anything left in the shared array by the first
call would show.  It also checks that a problem too large for the built-in array is
refused.  The file sorts last on purpose: a run that stops at the first failure has then
already been through every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _both(dq, lay, M, norms_np, rule):
    """(b, s) from the caller-scratch entry point and from the allocation-free one."""
    norms = torch.from_numpy(np.ascontiguousarray(norms_np, np.float32)).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_ref = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    out_new = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    nbytes = dq.choose_bits_scratch_bytes(lay, M)
    scratch = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    dq.choose_bits(lay, norms, M, rule, out_ref, scratch, nbytes, status)
    dq.choose_bits_noalloc(lay, norms, M, rule, out_new, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return tuple(out_ref.cpu().tolist()), tuple(out_new.cpu().tolist())


def test_noalloc_bit_rule_matches_on_two_calls_in_a_row(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    dq = dqlib
    rng = np.random.default_rng(2107)
    # several reduction chunks (3 * 40000 norms), so the shared array really is used
    M, nb = 3, 40000
    lay = dq.Layout([32 * nb], 32)
    assert lay.nb == nb
    norms1 = np.abs(rng.standard_normal((M, nb))).astype(np.float32)
    G2 = float((norms1.astype(np.float64) ** 2).sum() / M)
    T, alpha = 100, 0.95
    eps_hat = T * alpha ** (T - 1) * G2 / 36.0                    # b = 4 at t = 0
    ref1, new1 = _both(dq, lay, M, norms1, dq.Rule.dynamic(T, 0, eps_hat, alpha))
    assert ref1 == new1 and ref1[0] == 4 and ref1[1] == 7
    # and both agree with the CPU checker's rule on the same norms
    assert new1 == oracle.choose_bits(norms1, T, 0, eps_hat, alpha)[:2]

    # second call: much smaller norms, a later step, another layout size sharing the array
    M2, nb2 = 2, 9000
    lay2 = dq.Layout([32 * nb2], 32)
    norms2 = (np.abs(rng.standard_normal((M2, nb2))) * 1e-3).astype(np.float32)
    ref2, new2 = _both(dq, lay2, M2, norms2, dq.Rule.dynamic(T, 60, eps_hat * 1e-7, alpha))
    assert ref2 == new2 and ref2 != ref1
    assert new2 == oracle.choose_bits(norms2, T, 60, eps_hat * 1e-7, alpha)[:2]

    # fixed b never touches the array; and the first problem again gives the first answer
    ref3, new3 = _both(dq, lay, M, norms1, dq.Rule.fixed(9))
    assert ref3 == new3 == (9, 255)
    ref4, new4 = _both(dq, lay, M, norms1, dq.Rule.dynamic(T, 0, eps_hat, alpha))
    assert ref4 == new4 == ref1


def test_noalloc_refuses_more_norms_than_its_array_covers(dqlib):
    dq = dqlib
    limit = int(dq.lib().dq_choose_bits_noalloc_max_norms())
    assert limit == 8192 * 8192
    # 2^21 buckets per worker * 64 workers = 2 * limit norms; refused on the host, nothing is launched
    lay = dq.Layout([32 << 21], 32)
    rule = dq.Rule.fixed(4)
    fake = 0x7f0000001000                                          # never dereferenced
    rc = dq.lib().dq_choose_bits_noalloc(lay.handle, fake, 64, C.byref(rule), fake, fake, 0)
    assert rc == dq.ERR_TOO_LARGE
    assert "larger" in dq.status_string(rc)
    rc = dq.lib().dq_choose_bits_noalloc(lay.handle, fake, 32, C.byref(rule), 0, fake, 0)
    assert rc == dq.ERR_ARG
