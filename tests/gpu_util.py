"""Helpers of the GPU parity tests: run the library on numpy inputs, return numpy."""
from __future__ import annotations

import numpy as np
import torch

from paper_2107_14575_b200 import dq

CANARY = np.int32(0x5EEDC0DE - (1 << 32) if 0x5EEDC0DE >= (1 << 31) else 0x5EEDC0DE)
GUARD = 64        # guard words before and after every output buffer


class Guarded:
    """A device buffer with canary words on both sides, to catch out-of-bounds writes."""

    def __init__(self, n: int, dtype):
        assert dtype in (torch.int32, torch.float32)
        self.n = n
        self.raw = torch.full((n + 2 * GUARD,), int(CANARY), dtype=torch.int32, device="cuda")
        self.view = self.raw[GUARD: GUARD + n].view(dtype)

    def intact(self) -> bool:
        r = self.raw.cpu().numpy()
        return bool(np.all(r[:GUARD] == CANARY) and np.all(r[GUARD + self.n:] == CANARY))


class GpuRound:
    """Device state for one layout and worker count, driven through the C ABI."""

    def __init__(self, segs, bucket, M, stride=None, packed_stride=None, max_bits=16, norm=dq.NORM_L2):
        self.lay = dq.Layout(segs, bucket, norm).bind()
        self.M = M
        self.stride = self.lay.D32 if stride is None else stride
        self.pstride = ((self.lay.packed_words(max_bits) + 3) // 4 * 4) if packed_stride is None else packed_stride
        self.g_norms = Guarded(M * self.lay.nb, torch.float32)
        self.g_packed = Guarded(M * self.pstride, torch.int32)
        self.g_out = Guarded(self.lay.D32, torch.float32)
        self.g_b = Guarded(2, torch.int32)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.sbytes = dq.choose_bits_scratch_bytes(self.lay, M)
        self.scratch = torch.empty(max(self.sbytes, 256), dtype=torch.uint8, device="cuda")
        self.nbytes = dq.tensor_norms_scratch_bytes(self.lay, M)
        self.g_nscratch = Guarded(max(self.nbytes // 4, 4), torch.float32)
        self.grads = None

    # -- inputs
    def set_grads(self, g: np.ndarray):
        assert g.shape == (self.M, self.stride) and g.dtype == np.float32
        self.grads = torch.from_numpy(np.ascontiguousarray(g)).cuda()

    def set_norms(self, n: np.ndarray):
        assert n.shape == (self.M, self.lay.nb)
        self.g_norms.view.copy_(torch.from_numpy(np.ascontiguousarray(n, np.float32)).reshape(-1))

    def set_b(self, b: int):
        self.g_b.view.copy_(torch.tensor([b, (1 << (b - 1)) - 1 if 1 <= b <= 31 else 0], dtype=torch.int32))

    def set_packed(self, p: np.ndarray):
        assert p.shape == (self.M, self.pstride)
        self.g_packed.view.copy_(torch.from_numpy(p.view(np.int32).reshape(-1)))

    # -- calls
    def norms(self) -> np.ndarray:
        if self.lay.whole_tensor:
            dq.tensor_norms(self.lay, self.grads, self.stride, self.M, self.g_norms.view, self.g_nscratch.view,
                            self.nbytes, self.status)
        else:
            dq.bucket_norms(self.lay, self.grads, self.stride, self.M, self.g_norms.view, self.status)
        return self.g_norms.view.cpu().numpy().reshape(self.M, self.lay.nb)

    def bits(self, rule) -> tuple:
        dq.choose_bits(self.lay, self.g_norms.view, self.M, rule, self.g_b.view, self.scratch, self.sbytes,
                       self.status)
        b = self.g_b.view.cpu().numpy()
        return int(b[0]), int(b[1])

    def quantize(self, seed, step, fill=None) -> np.ndarray:
        if fill is not None:
            self.g_packed.view.fill_(fill)
        dq.quantize_pack(self.lay, self.grads, self.stride, self.M, self.g_norms.view, self.g_b.view, seed, step,
                         self.g_packed.view, self.pstride, self.status)
        return self.g_packed.view.cpu().numpy().view(np.uint32).reshape(self.M, self.pstride)

    def norms_quantize(self, seed, step, fill=None):
        """Fused call: returns (norms [M, nb], packed [M, pstride])."""
        if fill is not None:
            self.g_packed.view.fill_(fill)
        dq.norms_quantize_pack(self.lay, self.grads, self.stride, self.M, self.g_b.view, seed, step,
                               self.g_norms.view, self.g_packed.view, self.pstride, self.status)
        return (self.g_norms.view.cpu().numpy().reshape(self.M, self.lay.nb),
                self.g_packed.view.cpu().numpy().view(np.uint32).reshape(self.M, self.pstride))

    def average(self, fill=None) -> np.ndarray:
        if fill is not None:
            self.g_out.view.fill_(fill)
        dq.unpack_dequant_average(self.lay, self.g_packed.view, self.pstride, self.g_norms.view, self.M,
                                  self.g_b.view, self.g_out.view, self.status)
        return self.g_out.view.cpu().numpy()

    def update(self, lr: float, x: np.ndarray) -> np.ndarray:
        """Average and parameter update in one call; the parameters live in the guarded output buffer."""
        assert x.shape == (self.lay.D32,) and x.dtype == np.float32
        self.g_out.view.copy_(torch.from_numpy(x))
        dq.unpack_average_update(self.lay, self.g_packed.view, self.pstride, self.g_norms.view, self.M,
                                 self.g_b.view, lr, self.g_out.view, self.status)
        return self.g_out.view.cpu().numpy()

    def read_status(self) -> int:
        return int(self.status.item())

    def clear_status(self):
        self.status.zero_()

    def guards_intact(self) -> bool:
        return (self.g_norms.intact() and self.g_packed.intact() and self.g_out.intact() and self.g_b.intact()
                and self.g_nscratch.intact())


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))
