"""Helpers for the GPU parity tests: guarded device buffers and numpy <-> device transfers."""
import numpy as np
import torch

GUARD = 512
CANARY = 0x5A


class DevBuf:
    """A byte buffer on the device with canary bands before and after; `off` shifts the payload start."""

    def __init__(self, nbytes: int, off: int = 0, fill: int = 0xA5):
        self.nbytes = nbytes
        self.off = off
        self.raw = torch.full((GUARD + off + nbytes + GUARD,), CANARY, dtype=torch.uint8, device="cuda")
        self.view = self.raw[GUARD + off:GUARD + off + nbytes]
        if nbytes:
            self.view.fill_(fill)
        # the fills run on torch's current stream; tests hand these buffers to calls on other (non-blocking) streams, which are
        # not ordered behind it, so the buffer is made ready here
        torch.cuda.current_stream().synchronize()

    @property
    def ptr(self) -> int:
        return self.raw.data_ptr() + GUARD + self.off

    def data_ptr(self) -> int:
        return self.ptr

    def put(self, arr: np.ndarray):
        b = torch.from_numpy(arr.view(np.uint8).copy())
        assert b.numel() == self.nbytes
        self.view.copy_(b)
        torch.cuda.current_stream().synchronize()
        return self

    def get(self, dtype) -> np.ndarray:
        return self.view.cpu().numpy().view(dtype).copy()

    def guards_intact(self) -> bool:
        head = self.raw[:GUARD + self.off]
        tail = self.raw[GUARD + self.off + self.nbytes:]
        return bool((head == CANARY).all().item()) and bool((tail == CANARY).all().item())


def np_dtype(dtype: str):
    return np.float32 if dtype == "fp32" else np.uint16


def same_bits(a: np.ndarray, b: np.ndarray, dtype: str) -> bool:
    """Bit equality, except that any NaN matches any NaN (payloads are not part of the contract)."""
    if a.shape != b.shape:
        return False
    if dtype == "fp32":
        ua, ub = a.view(np.uint32), b.view(np.uint32)
        nan_a = (ua & 0x7FFFFFFF) > 0x7F800000
        nan_b = (ub & 0x7FFFFFFF) > 0x7F800000
    else:
        ua, ub = a.view(np.uint16), b.view(np.uint16)
        nan_a = (ua & 0x7FFF) > 0x7F80
        nan_b = (ub & 0x7FFF) > 0x7F80
    return bool(((ua == ub) | (nan_a & nan_b)).all()) and bool((nan_a == nan_b).all())
