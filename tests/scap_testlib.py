"""Helpers shared by the GPU parity tests: move seeded inputs to the device, call the C ABI through the
Python binding, and compare with the CPU oracle.  Nothing here computes the method."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import scap_inputs as si

REL_L2_TOL = 2e-3          # y vs the oracle's binary64 result, per batch row
CANARY = 0x7FC0DEAD        # a NaN pattern: any read of a guard word poisons the result too


def dev(bits: np.ndarray, dt: int) -> torch.Tensor:
    """uint16 patterns -> fp16/bf16 CUDA tensor (bytes unchanged)."""
    return si.as_torch(bits, dt).cuda()


def f32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).cuda()


def rel_l2_rows(y_gpu: np.ndarray, y64: np.ndarray) -> float:
    y_gpu = np.asarray(y_gpu, np.float64)
    num = np.linalg.norm(y_gpu - y64, axis=-1)
    den = np.maximum(np.linalg.norm(y64, axis=-1), 1e-300)
    return float(np.max(num / den))


class Guarded:
    """A device buffer with guard words on both sides, to catch out-of-bounds writes without a sanitizer."""
    PAD = 64  # int32 words = 256 bytes, keeps the payload 256-byte aligned

    def __init__(self, nbytes: int):
        words = (nbytes + 3) // 4
        self.words = words
        self.raw = torch.full((words + 2 * self.PAD,), CANARY, dtype=torch.int32, device="cuda")
        self.payload = self.raw[self.PAD:self.PAD + words]

    def view(self, dtype, shape):
        n = int(np.prod(shape)) if len(shape) else 1
        return self.payload.view(torch.uint8)[: n * torch.empty((), dtype=dtype).element_size()].view(dtype).view(*shape)

    def intact(self) -> bool:
        torch.cuda.synchronize()
        lo = self.raw[: self.PAD]
        hi = self.raw[self.PAD + self.words:]
        return bool((lo == CANARY).all().item() and (hi == CANARY).all().item())


def workspace(nbytes: int) -> Guarded:
    return Guarded(max(nbytes, 4))


def oracle_fc(d: dict, m, tau, bf64, x_bits=None, threads: int = 8):
    """Oracle y (binary64, with a binary64 fused bias), keep mask and kept-channel list."""
    dt = d["dt"]
    xf = si.to_f32(d["x"] if x_bits is None else x_bits, dt)
    y = oracle.sparse_fc(xf, d["W"], dt, m, tau, None, threads=threads)
    if bf64 is not None:
        y = y + np.asarray(bf64, np.float64)[None, :]
    keep, U, idx = oracle.mask(xf, m, tau)
    return y, keep, idx
