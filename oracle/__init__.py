"""fp64 CPU oracle for AdamA (arXiv 2305.19982) -- TEST INFRASTRUCTURE ONLY.

This package wraps ``adama_oracle.c`` (plain C, fp64) with ctypes.  It is the
checker, not the product: only the test-suite, the smoke check and the
CPU-baseline leg of the benchmark may import it.  It imports nothing from the
CUDA package and the CUDA package imports nothing from here.

``AdamAOracle`` strings the C functions together in the order Algorithm 2 of
the paper gives: ``begin_minibatch`` (t <- t+1 and the beta-decay of m, v),
``fold`` once per (micro-batch, layer), ``update`` at the end of the
mini-batch.  All state is numpy float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "adama_oracle.c"
_LIB = _HERE / "libadama_oracle.so"

_c_double_p = ctypes.POINTER(ctypes.c_double)
_c_int64_p = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> Path:
    """Compile adama_oracle.c with gcc into libadama_oracle.so beside it."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fvisibility=hidden",
           # no -ffast-math: IEEE semantics, no reassociation
           "-o", str(_LIB) + ".tmp", str(_SRC), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(str(_LIB) + ".tmp", _LIB)
    return _LIB


_lib = None


def load(path) -> ctypes.CDLL:
    """dlopen one build of the oracle and declare its signatures."""
    L = ctypes.CDLL(str(path))
    L.oracle_num_threads.restype = ctypes.c_int
    L.oracle_set_num_threads.argtypes = [ctypes.c_int]
    L.oracle_set_num_threads.restype = None
    L.oracle_decay.argtypes = [_c_double_p, _c_double_p, ctypes.c_size_t,
                               ctypes.c_double, ctypes.c_double]
    L.oracle_fold.argtypes = [_c_double_p, _c_double_p, _c_double_p, ctypes.c_size_t,
                              ctypes.c_int, ctypes.c_double, ctypes.c_double]
    L.oracle_update.argtypes = [_c_double_p, _c_double_p, _c_double_p, ctypes.c_size_t,
                                ctypes.c_long, ctypes.c_double, ctypes.c_double,
                                ctypes.c_double, ctypes.c_double]
    L.oracle_update_decoupled_decay.argtypes = [_c_double_p, _c_double_p, _c_double_p,
                                                ctypes.c_size_t, ctypes.c_long, ctypes.c_double,
                                                ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                                ctypes.c_double]
    L.oracle_update_decoupled_decay.restype = None
    L.oracle_closed_form_moments.argtypes = [_c_double_p, _c_double_p, _c_double_p,
                                             ctypes.c_size_t, ctypes.c_int, ctypes.c_double,
                                             ctypes.c_double, ctypes.c_int]
    L.oracle_linear_wgrad.argtypes = [_c_double_p, _c_double_p, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_size_t, ctypes.c_size_t,
                                      _c_double_p]
    L.oracle_linear_wgrad_entries.argtypes = [_c_double_p, _c_double_p, ctypes.c_int,
                                              ctypes.c_size_t, ctypes.c_size_t, _c_int64_p,
                                              _c_int64_p, ctypes.c_size_t, _c_double_p]
    L.oracle_ddp_decay.argtypes = [_c_double_p, _c_double_p, ctypes.c_size_t, ctypes.c_int,
                                   ctypes.c_double, ctypes.c_double]
    L.oracle_ddp_allreduce.argtypes = [_c_double_p, _c_double_p, ctypes.c_size_t,
                                       ctypes.c_int, _c_double_p, _c_double_p]
    L.oracle_coefficient_stats.argtypes = [_c_double_p, _c_double_p, ctypes.c_size_t,
                                           ctypes.c_long, ctypes.c_double, _c_double_p]
    L.oracle_sgdm_decay.argtypes = [_c_double_p, ctypes.c_size_t, ctypes.c_double]
    L.oracle_sgdm_fold.argtypes = [_c_double_p, _c_double_p, ctypes.c_size_t, ctypes.c_int]
    L.oracle_sgdm_update.argtypes = [_c_double_p, _c_double_p, ctypes.c_size_t, ctypes.c_double]
    for f in (L.oracle_coefficient_stats, L.oracle_sgdm_decay, L.oracle_sgdm_fold,
              L.oracle_sgdm_update):
        f.restype = None
    for f in (L.oracle_decay, L.oracle_fold, L.oracle_update, L.oracle_closed_form_moments,
              L.oracle_linear_wgrad, L.oracle_linear_wgrad_entries, L.oracle_ddp_decay,
              L.oracle_ddp_allreduce):
        f.restype = None
    return L


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = load(build())
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(threads: int) -> None:
    """Thread count of the oracle's loops from now on (timing only; results do not change)."""
    lib().oracle_set_num_threads(int(threads))


def _f64(a) -> np.ndarray:
    """C-contiguous float64 view/copy (exact widening for float32 inputs)."""
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags.c_contiguous
    return a.ctypes.data_as(_c_double_p)


def linear_wgrad(X, dY) -> np.ndarray:
    """G = X^T.dY by the naive triple loop; X [T, d_in], dY [T, d_out] (any real dtype)."""
    X = _f64(X)
    dY = _f64(dY)
    T, d_in = X.shape
    T2, d_out = dY.shape
    assert T == T2
    G = np.empty((d_in, d_out), dtype=np.float64)
    lib().oracle_linear_wgrad(_p(X), _p(dY), T, d_in, d_out, d_in, d_out, _p(G))
    return G


def linear_wgrad_entries(X, dY, p, q) -> np.ndarray:
    """G[p[s], q[s]] for sampled entries, same definition as linear_wgrad."""
    X = _f64(X)
    dY = _f64(dY)
    p = np.ascontiguousarray(np.asarray(p, dtype=np.int64))
    q = np.ascontiguousarray(np.asarray(q, dtype=np.int64))
    assert p.shape == q.shape and p.ndim == 1
    assert p.size == 0 or (p.min() >= 0 and p.max() < X.shape[1])
    assert q.size == 0 or (q.min() >= 0 and q.max() < dY.shape[1])
    out = np.empty(p.shape[0], dtype=np.float64)
    lib().oracle_linear_wgrad_entries(_p(X), _p(dY), X.shape[0], X.shape[1], dY.shape[1],
                                      p.ctypes.data_as(_c_int64_p), q.ctypes.data_as(_c_int64_p),
                                      p.shape[0], _p(out))
    return out


def closed_form_moments(m, v, grads, beta1, beta2, adam_variant: bool):
    """Algorithm 1's two moment lines for one mini-batch; grads is [N, n] raw gradients.

    Returns new (m, v); ``adam_variant`` picks standard Adam's (sum g)^2 instead
    of AdamA's sum(g^2)."""
    m = _f64(m).copy()
    v = _f64(v).copy()
    grads = _f64(grads)
    N, n = grads.shape
    assert m.shape == (n,) and v.shape == (n,)
    lib().oracle_closed_form_moments(_p(m), _p(v), _p(grads), n, N, beta1, beta2,
                                     1 if adam_variant else 0)
    return m, v


def coefficient_stats(v_adama, v_adam, t: int, beta2: float) -> dict:
    """Section 4.1: mean and range over the elements of sqrt(v_hat)/sqrt(v_hat') at step t, from
    AdamA's second moment ``v_adama`` and standard Adam's ``v_adam`` (both as they stand after the
    mini-batch's accumulation, before bias correction).  Elements with v_adam == 0 are left out."""
    a = _f64(v_adama).reshape(-1)
    b = _f64(v_adam).reshape(-1)
    assert a.shape == b.shape
    out = np.zeros(4)
    lib().oracle_coefficient_stats(_p(a), _p(b), a.shape[0], int(t), float(beta2), _p(out))
    count = int(out[3])
    return {"sum": out[0], "min": out[1], "max": out[2], "count": count,
            "mean": out[0] / count if count else float("nan")}


class SGDMOracle:
    """SGD with momentum on the same pipeline as Algorithm 2 (an extension, see the C source):
    ``begin_minibatch`` decays the buffer by mu, ``fold`` adds grad/N, ``update`` steps."""

    def __init__(self, theta, momentum=0.9):
        self.theta = _f64(theta).reshape(-1).copy()
        self.buf = np.zeros_like(self.theta)
        self.mu = float(momentum)
        self.N = None

    @property
    def n(self) -> int:
        return self.theta.shape[0]

    def begin_minibatch(self, N: int) -> None:
        assert N >= 1
        self.N = int(N)
        lib().oracle_sgdm_decay(_p(self.buf), self.n, self.mu)

    def fold(self, grad, lo: int = 0) -> None:
        g = _f64(grad).reshape(-1)
        hi = lo + g.shape[0]
        assert 0 <= lo and hi <= self.n and self.N is not None
        lib().oracle_sgdm_fold(_p(self.buf[lo:hi]), _p(g), g.shape[0], self.N)

    def update(self, lr: float) -> None:
        lib().oracle_sgdm_update(_p(self.theta), _p(self.buf), self.n, float(lr))


class AdamAOracle:
    """Algorithm 2 of the paper on one flat parameter vector, in fp64.

    theta, m, v are float64 numpy arrays of the same length; m0 = v0 = 0, t = 0.
    """

    def __init__(self, theta, beta1=0.9, beta2=0.999, eps=1e-8):
        self.theta = _f64(theta).reshape(-1).copy()
        self.m = np.zeros_like(self.theta)
        self.v = np.zeros_like(self.theta)
        self.t = 0
        self.N = None
        self.beta1, self.beta2, self.eps = float(beta1), float(beta2), float(eps)

    @property
    def n(self) -> int:
        return self.theta.shape[0]

    def begin_minibatch(self, N: int) -> None:
        """t <- t+1, m <- beta1*m, v <- beta2*v; fixes N for this mini-batch."""
        assert N >= 1
        self.t += 1
        self.N = int(N)
        lib().oracle_decay(_p(self.m), _p(self.v), self.n, self.beta1, self.beta2)

    def fold(self, grad, lo: int = 0) -> None:
        """Accumulate one raw micro-batch gradient into m, v at [lo, lo+len(grad))."""
        g = _f64(grad).reshape(-1)
        hi = lo + g.shape[0]
        assert 0 <= lo and hi <= self.n and self.N is not None
        m = self.m[lo:hi]
        v = self.v[lo:hi]
        lib().oracle_fold(_p(m), _p(v), _p(g), g.shape[0], self.N, self.beta1, self.beta2)

    def fold_linear(self, X, dY, lo: int = 0) -> None:
        """Weight gradient of a linear layer (G = X^T.dY), then fold; the layer's
        [d_in, d_out] weights live at [lo, lo + d_in*d_out)."""
        self.fold(linear_wgrad(X, dY), lo)

    def update(self, lr: float, weight_decay: float = 0.0) -> None:
        """Bias-corrected Adam step with the current t; weight_decay > 0 adds AdamW's
        decoupled decay (an extension, not part of the paper's algorithms)."""
        assert self.t >= 1
        if weight_decay == 0.0:
            lib().oracle_update(_p(self.theta), _p(self.m), _p(self.v), self.n, self.t, float(lr),
                                self.beta1, self.beta2, self.eps)
        else:
            lib().oracle_update_decoupled_decay(_p(self.theta), _p(self.m), _p(self.v), self.n,
                                                self.t, float(lr), self.beta1, self.beta2,
                                                self.eps, float(weight_decay))


class AdamADDPOracle:
    """Section 3.3: R data-parallel devices, each folding its own N micro-batches,
    with v pre-scaled by R*beta2 and one state all-reduce per mini-batch
    (m summed / R, v summed / R^2)."""

    def __init__(self, theta, devices: int, beta1=0.9, beta2=0.999, eps=1e-8):
        self.R = int(devices)
        self.theta = _f64(theta).reshape(-1).copy()
        n = self.theta.shape[0]
        self.m = np.zeros((self.R, n))
        self.v = np.zeros((self.R, n))
        self.t = 0
        self.N = None
        self.beta1, self.beta2, self.eps = float(beta1), float(beta2), float(eps)

    def begin_minibatch(self, N: int) -> None:
        self.t += 1
        self.N = int(N)
        n = self.theta.shape[0]
        for r in range(self.R):
            lib().oracle_ddp_decay(_p(self.m[r]), _p(self.v[r]), n, self.R, self.beta1, self.beta2)

    def fold(self, rank: int, grad) -> None:
        g = _f64(grad).reshape(-1)
        lib().oracle_fold(_p(self.m[rank]), _p(self.v[rank]), _p(g), g.shape[0], self.N,
                          self.beta1, self.beta2)

    def allreduce_and_update(self, lr: float) -> None:
        n = self.theta.shape[0]
        m_out = np.empty(n)
        v_out = np.empty(n)
        lib().oracle_ddp_allreduce(_p(self.m), _p(self.v), n, self.R, _p(m_out), _p(v_out))
        self.m[:] = m_out
        self.v[:] = v_out
        lib().oracle_update(_p(self.theta), _p(m_out), _p(v_out), n, self.t, float(lr),
                            self.beta1, self.beta2, self.eps)
