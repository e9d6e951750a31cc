"""Helpers for the GPU-vs-oracle parity tests."""
import numpy as np
import torch

SENTINEL = 12345.0


def rel_l2(got, want) -> float:
    """||got - want||_2 / ||want||_2 in float64."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    denom = np.linalg.norm(want)
    if denom == 0.0:
        return float(np.linalg.norm(got))
    return float(np.linalg.norm(got - want) / denom)


def f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a tensor's bit pattern to float64 on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()


class Guarded:
    """A device buffer with sentinel-filled guard bands before and after the payload
    (stands in for a memory checker: out-of-bounds writes of a kernel show up here)."""

    def __init__(self, n, dtype=torch.float32, pad=64, offset=0, device="cuda"):
        self.pad, self.n, self.offset = pad, n, offset
        self.buf = torch.full((pad + offset + n + pad,), SENTINEL, dtype=dtype, device=device)
        self.view = self.buf[pad + offset: pad + offset + n]

    def fill(self, src: torch.Tensor):
        self.view.copy_(src.reshape(-1))
        return self

    def zero(self):
        self.view.zero_()
        return self

    def check(self):
        lo = self.buf[: self.pad + self.offset]
        hi = self.buf[self.pad + self.offset + self.n:]
        assert bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all()), "guard band overwritten"
