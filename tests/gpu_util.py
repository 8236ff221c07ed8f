"""Helpers for the GPU parity tests: device buffers with canary padding, oracle wrappers."""
import numpy as np

CANARY = 0xA5
PAD = 256          # bytes of canary on each side of every output buffer


def torch_mod():
    import torch
    return torch


def dev(a: np.ndarray):
    torch = torch_mod()
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class Guarded:
    """A device output buffer with canary bytes before and after it."""

    def __init__(self, nbytes: int):
        torch = torch_mod()
        self.nbytes = int(nbytes)
        body = (self.nbytes + 255) // 256 * 256
        self.raw = torch.full((PAD + body + PAD,), CANARY, dtype=torch.uint8, device="cuda")
        self.view = self.raw[PAD:PAD + self.nbytes]

    def data_ptr(self):
        return self.view.data_ptr()

    def numpy(self, dtype, shape):
        return self.view.cpu().numpy().view(dtype).reshape(shape).copy()

    def check(self):
        torch = torch_mod()
        head = self.raw[:PAD]
        tail = self.raw[PAD + self.nbytes:]
        assert bool(torch.all(head == CANARY)), "write before the buffer"
        assert bool(torch.all(tail == CANARY)), "write past the buffer"
