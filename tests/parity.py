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


def max_abs_rel(got, want) -> float:
    """max|got - want| / max|want| in float64: one wrong element (a chunk, a row, a tile edge)
    shows here even when it would vanish in the L2 norm of a large matrix."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    if got.size == 0:
        return 0.0
    denom = float(np.max(np.abs(want)))
    err = float(np.max(np.abs(got - want)))
    return err if denom == 0.0 else err / denom


def assert_close(got, want, tol, what="", elementwise=True):
    """The parity bar of a whole tensor or sample: relative L2 error <= tol AND the largest
    single deviation <= tol * the largest magnitude.

    elementwise=False drops the second bound.  It is for ONE case: the weights after the very
    first update of a run with a single micro-batch and inexact (non-integer) inputs.  There
    m_hat / sqrt(v_hat) = G / |G| is the sign of the gradient, so an element whose G is at
    rounding level (a few in 10^7 are) legitimately lands on w - lr or w + lr depending on the
    summation order; m and v of the same element stay within the bound."""
    l2 = rel_l2(got, want)
    assert l2 <= tol, f"{what}: relative L2 error {l2:.3e} > {tol:.1e}"
    if elementwise:
        mx = max_abs_rel(got, want)
        assert mx <= tol, f"{what}: max |error| / max |value| = {mx:.3e} > {tol:.1e}"


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
