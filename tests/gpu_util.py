"""Helpers of the GPU parity tests: run the CUDA path through the C-ABI binding on numpy
inputs and hand back numpy results.  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

from paper_2112_04291_b200 import binding

GUARD = 4096        # canary bytes on each side of every output buffer
CANARY = 0xA5


def dev():
    return torch.device("cuda", 0)


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev())


class Guarded:
    """A device byte buffer with canaries before and after the part handed to the library."""

    def __init__(self, nbytes: int, fill: int = 0):
        self.nbytes = int(nbytes)
        pad = (-self.nbytes) % 256
        self.raw = torch.full((GUARD + self.nbytes + pad + GUARD,), CANARY, dtype=torch.uint8, device=dev())
        self.view = self.raw[GUARD:GUARD + self.nbytes]
        self.view.fill_(fill)

    def intact(self) -> bool:
        head = self.raw[:GUARD]
        tail = self.raw[GUARD + self.nbytes:]
        return bool((head == CANARY).all().item()) and bool((tail == CANARY).all().item())


def gpu_compress(v: np.ndarray, p: binding.Params, cap: int | None = None, fill: int = 0):
    """-> (rc, header status, stream bytes (numpy), guard intact)"""
    g = to_dev(v.astype(np.float32, copy=False))
    n = g.numel()
    binding.ensure_workspace(n, p)
    if cap is None:
        cap = binding.compress_bound(n, p)
    buf = Guarded(cap, fill)
    rc = binding.compress(g, p, buf.view)
    if rc != 0:
        return rc, None, None, buf.intact()
    total, d, status = binding.stream_info(buf.view)
    torch.cuda.synchronize()
    assert total <= cap
    return rc, status, buf.view[:total].cpu().numpy().copy(), buf.intact()


def gpu_decompress(stream: np.ndarray, n: int, p: binding.Params, dense0: np.ndarray | None = None,
                   nbytes: int | None = None):
    """-> (rc, decoder status, dense (numpy), guard intact)"""
    binding.ensure_workspace(n, p)
    s = np.ascontiguousarray(stream, np.uint8)
    pad = (-s.size) % 16
    sd = to_dev(np.concatenate([s, np.zeros(pad + 16, np.uint8)]))
    buf = Guarded(4 * n)
    dense = buf.view.view(torch.float32)
    if dense0 is not None:
        dense.copy_(torch.from_numpy(dense0))
    rc = binding.decompress_accumulate(sd, s.size if nbytes is None else nbytes, n, p, dense)
    if rc != 0:
        return rc, None, None, buf.intact()
    st = binding.decode_status()
    torch.cuda.synchronize()
    return rc, st, dense.cpu().numpy().copy(), buf.intact()
