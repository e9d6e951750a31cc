"""ctypes binding with the same names as the C ABI (include/adama.h).

Argument marshalling only: tensors become raw device pointers, the stream is
torch's current CUDA stream, doubles stay doubles.
"""
from __future__ import annotations

import ctypes
import enum
from pathlib import Path
from typing import Optional

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libadama.so"

EXPORTED_SYMBOLS = [
    "adama_init", "adama_destroy", "adama_begin_minibatch", "adama_fold",
    "adama_linear_wgrad_fold", "adama_linear_wgrad_bias_fold", "adama_apply", "adama_apply_bf16_copy", "adama_apply_allreduced", "adama_apply_sharded", "adama_apply_sharded_peers", "adama_fold_multi", "adama_apply_multi", "adama_bias_grad_fold",
    "adama_fold_host", "adama_linear_wgrad_fold_host",
    "adama_apply_to_host", "adama_linear_wgrad_fold_noalloc", "adama_linear_wgrad_fold_multi", "adama_sgdm_fold", "adama_sgdm_apply",
    "adama_coefficient_stats", "adama_get_step", "adama_set_step", "adama_get_n_micro", "adama_set_weight_decay",
    "adama_sync_status", "adama_debug_set_status", "adama_debug_wgrad_expire_wait",
    "adama_debug_set_wgrad_variant", "adama_debug_setup_state", "adama_last_error", "adama_launch_count", "adama_host_constants",
    "adama_host_constants_allreduced", "adama_host_constants_sharded",
    "adama_version",
]


class Status(enum.IntEnum):
    OK = 0
    ERR_INVALID_ARG = 1
    ERR_BAD_STATE = 2
    ERR_MISALIGNED = 3
    ERR_UNSUPPORTED = 4
    ERR_CUDA = 5
    ERR_TIMEOUT = 6


F32, BF16 = 0, 1
GRADS_PRESCALED = 1
ASYNC_COPYBACK = 2
INPUTS_SETTLED = 4


class AdamAError(RuntimeError):
    def __init__(self, status: int, message: str):
        self.status = Status(status)
        super().__init__(f"{self.status.name}: {message}")


class _LinearItem(ctypes.Structure):
    _fields_ = [("X", ctypes.c_void_p), ("dY", ctypes.c_void_p), ("tokens", ctypes.c_int),
                ("d_in", ctypes.c_int), ("d_out", ctypes.c_int), ("ldx", ctypes.c_int64),
                ("ldy", ctypes.c_int64), ("m", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("ldmv", ctypes.c_int64), ("m_bias", ctypes.c_void_p), ("v_bias", ctypes.c_void_p)]


class _Config(ctypes.Structure):
    _fields_ = [("beta1", ctypes.c_double), ("beta2", ctypes.c_double), ("eps", ctypes.c_double),
                ("device", ctypes.c_int), ("flags", ctypes.c_uint)]


_lib: Optional[ctypes.CDLL] = None


def library_path() -> Path:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """dlopen libadama.so (built in-tree by paper_2305_19982_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists() and _LIB_PATH == _PKG / "libadama.so":
        # a source-only checkout: compile once, in-tree (needs nvcc); never a substitute path
        try:
            from . import build as _build
            _build.build()
        except Exception as exc:  # noqa: BLE001 - reported below with the way out
            raise FileNotFoundError(
                f"{_LIB_PATH} is missing and could not be built ({exc}): build it with "
                "`python -m paper_2305_19982_b200.build` (there is no fallback path)") from exc
    if not _LIB_PATH.exists():
        raise FileNotFoundError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2305_19982_b200.build` "
            "(there is no fallback path)")
    L = ctypes.CDLL(str(_LIB_PATH))
    vp, i64, sz, dbl, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_double, ctypes.c_int
    L.adama_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(_Config)]
    L.adama_destroy.argtypes = [vp]
    L.adama_begin_minibatch.argtypes = [vp, ci]
    L.adama_fold.argtypes = [vp, vp, ci, vp, vp, sz, vp]
    L.adama_linear_wgrad_fold.argtypes = [vp, vp, vp, ci, ci, ci, i64, i64, vp, vp, i64, vp]
    L.adama_linear_wgrad_bias_fold.argtypes = [vp, vp, vp, ci, ci, ci, i64, i64, vp, vp, i64, vp, vp, vp]
    L.adama_linear_wgrad_fold_multi.argtypes = [vp, ctypes.POINTER(_LinearItem), ci, vp]
    L.adama_apply.argtypes = [vp, vp, vp, vp, sz, dbl, vp]
    L.adama_apply_bf16_copy.argtypes = [vp, vp, vp, vp, vp, sz, dbl, vp]
    L.adama_apply_allreduced.argtypes = [vp, vp, vp, vp, sz, dbl, ci, vp]
    L.adama_host_constants_allreduced.argtypes = [ctypes.POINTER(_Config), ci, i64, dbl, ci,
                                                  ctypes.POINTER(ctypes.c_float)]
    L.adama_apply_sharded.argtypes = [vp, vp, vp, vp, sz, dbl, ci, vp]
    L.adama_host_constants_sharded.argtypes = L.adama_host_constants_allreduced.argtypes
    L.adama_fold_multi.argtypes = [vp, ctypes.POINTER(vp), ci, ctypes.POINTER(vp),
                                   ctypes.POINTER(vp), ctypes.POINTER(sz), ci, vp]
    L.adama_apply_multi.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp),
                                    ctypes.POINTER(sz), ci, dbl, vp]
    L.adama_apply_sharded_peers.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp),
                                            ctypes.POINTER(vp), ci, ci, sz, dbl, vp]
    L.adama_bias_grad_fold.argtypes = [vp, vp, ci, ci, i64, vp, vp, vp]
    L.adama_fold_host.argtypes = [vp, vp, ci, vp, vp, sz, vp, sz, vp]
    L.adama_linear_wgrad_fold_host.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp, i64, vp, sz, vp]
    L.adama_apply_to_host.argtypes = [vp, vp, vp, vp, sz, dbl, vp, vp]
    L.adama_linear_wgrad_fold_noalloc.argtypes = [ctypes.POINTER(_Config), ci, vp, vp, ci, ci, ci,
                                                  i64, i64, vp, vp, i64, vp, ctypes.c_char_p, sz, vp]
    L.adama_sgdm_fold.argtypes = [vp, vp, ci, vp, sz, vp]
    L.adama_sgdm_apply.argtypes = [vp, vp, vp, sz, dbl, dbl, vp]
    L.adama_coefficient_stats.argtypes = [vp, vp, vp, vp, vp, sz, vp, vp]
    L.adama_get_step.argtypes = [vp]
    L.adama_get_step.restype = i64
    L.adama_set_step.argtypes = [vp, i64]
    L.adama_get_n_micro.argtypes = [vp]
    L.adama_set_weight_decay.argtypes = [vp, dbl]
    L.adama_sync_status.argtypes = [vp, vp]
    L.adama_debug_set_status.argtypes = [vp, ctypes.c_uint, ctypes.c_uint, ctypes.c_uint, vp]
    L.adama_debug_wgrad_expire_wait.argtypes = [vp, vp, vp, ci, ci, ci, i64, i64, vp, vp, i64,
                                                ctypes.c_uint64, vp]
    L.adama_debug_set_wgrad_variant.argtypes = [vp, ci, ci, ci, ci]
    L.adama_debug_setup_state.argtypes = [ci]
    L.adama_debug_setup_state.restype = ci
    L.adama_last_error.argtypes = [vp]
    L.adama_last_error.restype = ctypes.c_char_p
    L.adama_launch_count.argtypes = [vp]
    L.adama_launch_count.restype = i64
    L.adama_host_constants.argtypes = [ctypes.POINTER(_Config), ci, i64, dbl,
                                       ctypes.POINTER(ctypes.c_float)]
    L.adama_version.restype = ctypes.c_char_p
    _lib = L
    return L


def host_constants(beta1, beta2, eps, n_micro, t, lr, flags=0, world_size=1, sharded=False):
    """adama_host_constants[_allreduced|_sharded]: the nine fp32 constants the kernels receive
    (no GPU needed)."""
    L = load_library()
    cfg = _Config(beta1, beta2, eps, 0, flags)
    out = (ctypes.c_float * 9)()
    fn = L.adama_host_constants_sharded if sharded else L.adama_host_constants_allreduced
    st = fn(ctypes.byref(cfg), n_micro, t, lr, world_size, out)
    if st != 0:
        raise AdamAError(st, "adama_host_constants")
    return [float(x) for x in out]


def _stream_ptr(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _dev_ptr(t: torch.Tensor, dtype: torch.dtype, name: str) -> int:
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


class TensorList:
    """Device pointers and sizes of a list of contiguous CUDA tensors, marshalled once for
    repeated multi-tensor calls (keeps the tensors alive)."""

    def __init__(self, tensors, dtype=None):
        self.tensors = list(tensors)
        self.dtype = dtype if dtype is not None else (self.tensors[0].dtype if self.tensors else torch.float32)
        self.ptrs = (ctypes.c_void_p * len(self.tensors))()
        for i, t in enumerate(self.tensors):
            if not t.is_contiguous():
                raise ValueError(f"tensor {i} must be contiguous")
            self.ptrs[i] = _dev_ptr(t, self.dtype, f"tensor {i}")
        self.numels = [t.numel() for t in self.tensors]
        self.ns = (ctypes.c_size_t * len(self.tensors))(*self.numels)

    def __len__(self):
        return len(self.tensors)


class AdamA:
    """One AdamA context (adama_ctx) bound to a CUDA device.

    Methods mirror the C ABI one to one; tensors are torch CUDA tensors owned by
    the caller, work is queued on torch's current stream of the context's device.
    The keyword flags are adama_config.flags: grads_prescaled = ADAMA_GRADS_PRESCALED,
    async_copyback = ADAMA_ASYNC_COPYBACK, inputs_settled = ADAMA_INPUTS_SETTLED (the caller
    promises that X, dY of the fused calls are not written by the kernel enqueued just before
    the call; see include/adama.h).
    """

    def __init__(self, beta1=0.9, beta2=0.999, eps=1e-8, device=0, grads_prescaled=False,
                 async_copyback=False, inputs_settled=False):
        self._L = load_library()
        self._h = ctypes.c_void_p()
        self.device = torch.device("cuda", int(device))
        cfg = _Config(beta1, beta2, eps, int(device),
                      (GRADS_PRESCALED if grads_prescaled else 0) |
                      (ASYNC_COPYBACK if async_copyback else 0) |
                      (INPUTS_SETTLED if inputs_settled else 0))
        st = self._L.adama_init(ctypes.byref(self._h), ctypes.byref(cfg))
        if st != 0:
            self._h = ctypes.c_void_p()
            raise AdamAError(st, "adama_init failed (needs a compute-capability-10.x GPU)")

    # -- plumbing ---------------------------------------------------------------------------
    def _check(self, st: int) -> None:
        if st != 0:
            raise AdamAError(st, self._L.adama_last_error(self._h).decode())

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._L.adama_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- Algorithm 2 --------------------------------------------------------------------------
    def begin_minibatch(self, n_micro: int) -> None:
        self._check(self._L.adama_begin_minibatch(self._h, int(n_micro)))

    def fold(self, grad: torch.Tensor, m: torch.Tensor, v: torch.Tensor) -> None:
        """adama_fold on contiguous tensors of equal numel; grad is fp32 or bf16."""
        if grad.dtype == torch.float32:
            gdt = F32
        elif grad.dtype == torch.bfloat16:
            gdt = BF16
        else:
            raise TypeError("grad must be float32 or bfloat16")
        if not (grad.is_contiguous() and m.is_contiguous() and v.is_contiguous()):
            raise ValueError("fold needs contiguous tensors")
        n = grad.numel()
        if m.numel() != n or v.numel() != n:
            raise ValueError("grad, m, v must have the same number of elements")
        self._check(self._L.adama_fold(self._h, _dev_ptr(grad, grad.dtype, "grad"), gdt,
                                       _dev_ptr(m, torch.float32, "m"),
                                       _dev_ptr(v, torch.float32, "v"), n,
                                       _stream_ptr(self.device)))

    def linear_wgrad_fold(self, X: torch.Tensor, dY: torch.Tensor, m: torch.Tensor,
                          v: torch.Tensor, m_bias: Optional[torch.Tensor] = None,
                          v_bias: Optional[torch.Tensor] = None) -> None:
        """adama_linear_wgrad_fold: X [tokens, d_in], dY [tokens, d_out] bf16 (unit stride in
        the last dim), m, v [d_in, d_out] fp32 views with a common row pitch.  With m_bias and
        v_bias (contiguous, d_out fp32 each): adama_linear_wgrad_bias_fold, which folds the
        bias gradient (column sums of dY) in the same launch."""
        if X.dim() != 2 or dY.dim() != 2 or m.dim() != 2 or v.dim() != 2:
            raise ValueError("linear_wgrad_fold takes 2-D tensors")
        tokens, d_in = X.shape
        if dY.shape[0] != tokens:
            raise ValueError("X and dY must have the same number of tokens")
        d_out = dY.shape[1]
        if tuple(m.shape) != (d_in, d_out) or tuple(v.shape) != (d_in, d_out):
            raise ValueError("m, v must be [d_in, d_out]")
        for name, t in (("X", X), ("dY", dY), ("m", m), ("v", v)):
            if t.shape[1] > 1 and t.stride(1) != 1:
                raise ValueError(f"{name} must have unit stride in its last dimension")
        if m.stride(0) != v.stride(0):
            raise ValueError("m and v must share one row pitch")
        ldx = X.stride(0) if tokens > 1 else max(d_in, X.stride(0))
        ldy = dY.stride(0) if tokens > 1 else max(d_out, dY.stride(0))
        ldmv = m.stride(0) if d_in > 1 else max(d_out, m.stride(0))
        if (m_bias is None) != (v_bias is None):
            raise ValueError("m_bias and v_bias go together")
        if m_bias is not None:
            if m_bias.numel() != d_out or v_bias.numel() != d_out or not (
                    m_bias.is_contiguous() and v_bias.is_contiguous()):
                raise ValueError("m_bias, v_bias must be contiguous with d_out elements")
            self._check(self._L.adama_linear_wgrad_bias_fold(
                self._h, _dev_ptr(X, torch.bfloat16, "X"), _dev_ptr(dY, torch.bfloat16, "dY"),
                tokens, d_in, d_out, ldx, ldy, _dev_ptr(m, torch.float32, "m"),
                _dev_ptr(v, torch.float32, "v"), ldmv, _dev_ptr(m_bias, torch.float32, "m_bias"),
                _dev_ptr(v_bias, torch.float32, "v_bias"), _stream_ptr(self.device)))
            return
        self._check(self._L.adama_linear_wgrad_fold(
            self._h, _dev_ptr(X, torch.bfloat16, "X"), _dev_ptr(dY, torch.bfloat16, "dY"),
            tokens, d_in, d_out, ldx, ldy, _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), ldmv, _stream_ptr(self.device)))

    def linear_wgrad_fold_multi(self, layers) -> None:
        """adama_linear_wgrad_fold_multi: `layers` is a sequence of (X, dY, m, v) or
        (X, dY, m, v, m_bias, v_bias) tuples, tensors as for linear_wgrad_fold; they are folded
        in the given order by as few launches as possible.  Keep X and dY alive until the
        stream has run the call."""
        arr = (_LinearItem * len(layers))()
        for it, layer in zip(arr, layers):
            X, dY, m, v = layer[:4]
            mb, vb = (layer[4], layer[5]) if len(layer) > 4 else (None, None)
            if X.dim() != 2 or dY.dim() != 2 or m.dim() != 2 or v.dim() != 2:
                raise ValueError("linear_wgrad_fold_multi takes 2-D tensors")
            tokens, d_in = X.shape
            d_out = dY.shape[1]
            if dY.shape[0] != tokens or tuple(m.shape) != (d_in, d_out) or tuple(v.shape) != (d_in, d_out):
                raise ValueError("shapes must be X [T, d_in], dY [T, d_out], m, v [d_in, d_out]")
            for name, t in (("X", X), ("dY", dY), ("m", m), ("v", v)):
                if t.shape[1] > 1 and t.stride(1) != 1:
                    raise ValueError(f"{name} must have unit stride in its last dimension")
            if m.stride(0) != v.stride(0):
                raise ValueError("m and v must share one row pitch")
            it.X, it.dY = _dev_ptr(X, torch.bfloat16, "X"), _dev_ptr(dY, torch.bfloat16, "dY")
            it.tokens, it.d_in, it.d_out = tokens, d_in, d_out
            it.ldx = X.stride(0) if tokens > 1 else max(d_in, X.stride(0))
            it.ldy = dY.stride(0) if tokens > 1 else max(d_out, dY.stride(0))
            it.m, it.v = _dev_ptr(m, torch.float32, "m"), _dev_ptr(v, torch.float32, "v")
            it.ldmv = m.stride(0) if d_in > 1 else max(d_out, m.stride(0))
            if mb is not None:
                if mb.numel() != d_out or vb.numel() != d_out or not (mb.is_contiguous() and vb.is_contiguous()):
                    raise ValueError("m_bias, v_bias must be contiguous with d_out elements")
                it.m_bias, it.v_bias = _dev_ptr(mb, torch.float32, "m_bias"), _dev_ptr(vb, torch.float32, "v_bias")
        self._check(self._L.adama_linear_wgrad_fold_multi(self._h, arr, len(layers),
                                                          _stream_ptr(self.device)))

    def apply(self, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor, lr: float) -> None:
        if not (w.is_contiguous() and m.is_contiguous() and v.is_contiguous()):
            raise ValueError("apply needs contiguous tensors")
        n = w.numel()
        if m.numel() != n or v.numel() != n:
            raise ValueError("w, m, v must have the same number of elements")
        self._check(self._L.adama_apply(self._h, _dev_ptr(w, torch.float32, "w"),
                                        _dev_ptr(m, torch.float32, "m"),
                                        _dev_ptr(v, torch.float32, "v"), n, float(lr),
                                        _stream_ptr(self.device)))

    def apply_sharded_peers(self, w_ptrs, m_ptrs, v_ptrs, rank: int, n: int, lr: float) -> None:
        """adama_apply_sharded_peers: lists of raw device pointers (ints), one per rank, to the
        peer-mapped full-size w, m, v buffers; `rank` is this process's index."""
        world = len(w_ptrs)
        if len(m_ptrs) != world or len(v_ptrs) != world:
            raise ValueError("pointer lists must have equal length")
        arr = lambda ps: (ctypes.c_void_p * world)(*[int(p) for p in ps])
        self._check(self._L.adama_apply_sharded_peers(
            self._h, arr(w_ptrs), arr(m_ptrs), arr(v_ptrs), world, int(rank), int(n), float(lr),
            _stream_ptr(self.device)))

    def bias_grad_fold(self, dY: torch.Tensor, m: torch.Tensor, v: torch.Tensor) -> None:
        """adama_bias_grad_fold: dY [tokens, d_out] bf16 (unit stride in the last dim), m, v [d_out]."""
        tokens, d_out = dY.shape
        if dY.shape[1] > 1 and dY.stride(1) != 1:
            raise ValueError("dY must have unit stride in its last dimension")
        if m.numel() != d_out or v.numel() != d_out or not (m.is_contiguous() and v.is_contiguous()):
            raise ValueError("m, v must be contiguous with d_out elements")
        ldy = dY.stride(0) if tokens > 1 else max(d_out, dY.stride(0))
        self._check(self._L.adama_bias_grad_fold(
            self._h, _dev_ptr(dY, torch.bfloat16, "dY"), tokens, d_out, ldy,
            _dev_ptr(m, torch.float32, "m"), _dev_ptr(v, torch.float32, "v"),
            _stream_ptr(self.device)))

    def fold_multi(self, grads, ms, vs) -> None:
        """adama_fold_multi over lists of tensors (all gradients of one dtype); pass TensorList
        objects to skip the per-call marshalling."""
        grads = grads if isinstance(grads, TensorList) else TensorList(grads)
        ms = ms if isinstance(ms, TensorList) else TensorList(ms, torch.float32)
        vs = vs if isinstance(vs, TensorList) else TensorList(vs, torch.float32)
        if not (len(grads) == len(ms) == len(vs)):
            raise ValueError("lists must have equal length")
        if len(grads) == 0:
            return
        if grads.numels != ms.numels or grads.numels != vs.numels:
            raise ValueError("grad, m, v must have the same number of elements")
        gdt = {torch.float32: F32, torch.bfloat16: BF16}[grads.dtype]
        self._check(self._L.adama_fold_multi(self._h, grads.ptrs, gdt, ms.ptrs, vs.ptrs, grads.ns,
                                             len(grads), _stream_ptr(self.device)))

    def apply_multi(self, ws, ms, vs, lr: float) -> None:
        """adama_apply_multi over lists of tensors (or TensorList objects)."""
        ws = ws if isinstance(ws, TensorList) else TensorList(ws, torch.float32)
        ms = ms if isinstance(ms, TensorList) else TensorList(ms, torch.float32)
        vs = vs if isinstance(vs, TensorList) else TensorList(vs, torch.float32)
        if not (len(ws) == len(ms) == len(vs)):
            raise ValueError("lists must have equal length")
        if len(ws) == 0:
            return
        if ws.numels != ms.numels or ws.numels != vs.numels:
            raise ValueError("w, m, v must have the same number of elements")
        self._check(self._L.adama_apply_multi(self._h, ws.ptrs, ms.ptrs, vs.ptrs, ws.ns, len(ws),
                                              float(lr), _stream_ptr(self.device)))

    def sgdm_fold(self, grad: torch.Tensor, buf: torch.Tensor) -> None:
        """adama_sgdm_fold: buf += grad/N (SGD with momentum on the same pipeline)."""
        if not (grad.is_contiguous() and buf.is_contiguous()):
            raise ValueError("sgdm_fold needs contiguous tensors")
        if grad.numel() != buf.numel():
            raise ValueError("grad and buf must have the same number of elements")
        if grad.dtype == torch.float32:
            gdt = F32
        elif grad.dtype == torch.bfloat16:
            gdt = BF16
        else:
            raise TypeError(f"gradient dtype {grad.dtype} not supported (float32 or bfloat16)")
        if not grad.is_cuda:
            raise TypeError("grad must be a CUDA tensor")
        self._check(self._L.adama_sgdm_fold(self._h, grad.data_ptr(), gdt,
                                            _dev_ptr(buf, torch.float32, "buf"), buf.numel(),
                                            _stream_ptr(self.device)))

    def sgdm_apply(self, w: torch.Tensor, buf: torch.Tensor, lr: float, momentum: float) -> None:
        """adama_sgdm_apply: w -= lr*buf, then buf *= momentum for the next mini-batch."""
        if not (w.is_contiguous() and buf.is_contiguous()):
            raise ValueError("sgdm_apply needs contiguous tensors")
        if w.numel() != buf.numel():
            raise ValueError("w and buf must have the same number of elements")
        self._check(self._L.adama_sgdm_apply(self._h, _dev_ptr(w, torch.float32, "w"),
                                             _dev_ptr(buf, torch.float32, "buf"), w.numel(),
                                             float(lr), float(momentum), _stream_ptr(self.device)))

    def coefficient_stats(self, m: torch.Tensor, m_begin: Optional[torch.Tensor], v: torch.Tensor,
                          v_adam: torch.Tensor, stats: torch.Tensor) -> None:
        """adama_coefficient_stats: `stats` (4 float64 on the device) receives
        {sum, min, max, count} of sqrt(v_hat)/sqrt(v_hat'); `v_adam` is updated in place."""
        ts = [m, v, v_adam] + ([m_begin] if m_begin is not None else [])
        if not all(t.is_contiguous() for t in ts):
            raise ValueError("coefficient_stats needs contiguous tensors")
        n = m.numel()
        if any(t.numel() != n for t in ts):
            raise ValueError("m, m_begin, v, v_adam must have the same number of elements")
        if stats.numel() != 4:
            raise ValueError("stats must hold 4 float64 values")
        self._check(self._L.adama_coefficient_stats(
            self._h, _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(m_begin, torch.float32, "m_begin") if m_begin is not None else None,
            _dev_ptr(v, torch.float32, "v"), _dev_ptr(v_adam, torch.float32, "v_adam"), n,
            _dev_ptr(stats, torch.float64, "stats"), _stream_ptr(self.device)))

    def apply_bf16_copy(self, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor,
                        w_bf16: torch.Tensor, lr: float) -> None:
        """adama_apply_bf16_copy: apply, and write the updated weights to `w_bf16` as bf16."""
        if not (w.is_contiguous() and m.is_contiguous() and v.is_contiguous() and w_bf16.is_contiguous()):
            raise ValueError("apply needs contiguous tensors")
        n = w.numel()
        if m.numel() != n or v.numel() != n or w_bf16.numel() != n:
            raise ValueError("w, m, v, w_bf16 must have the same number of elements")
        self._check(self._L.adama_apply_bf16_copy(
            self._h, _dev_ptr(w, torch.float32, "w"), _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), _dev_ptr(w_bf16, torch.bfloat16, "w_bf16"), n,
            float(lr), _stream_ptr(self.device)))

    def apply_allreduced(self, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor, lr: float,
                         world_size: int) -> None:
        """adama_apply_allreduced: m, v hold the sums over `world_size` data-parallel ranks."""
        if not (w.is_contiguous() and m.is_contiguous() and v.is_contiguous()):
            raise ValueError("apply needs contiguous tensors")
        n = w.numel()
        if m.numel() != n or v.numel() != n:
            raise ValueError("w, m, v must have the same number of elements")
        self._check(self._L.adama_apply_allreduced(
            self._h, _dev_ptr(w, torch.float32, "w"), _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), n, float(lr), int(world_size),
            _stream_ptr(self.device)))

    def apply_sharded(self, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor, lr: float,
                      world_size: int) -> None:
        """adama_apply_sharded: w, m, v are this rank's shard; m, v hold the reduce-scattered
        sums over `world_size` ranks."""
        if not (w.is_contiguous() and m.is_contiguous() and v.is_contiguous()):
            raise ValueError("apply needs contiguous tensors")
        n = w.numel()
        if m.numel() != n or v.numel() != n:
            raise ValueError("w, m, v must have the same number of elements")
        self._check(self._L.adama_apply_sharded(
            self._h, _dev_ptr(w, torch.float32, "w"), _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), n, float(lr), int(world_size),
            _stream_ptr(self.device)))

    # -- host-buffer variants ---------------------------------------------------------------
    def fold_host(self, grad_host: torch.Tensor, m: torch.Tensor, v: torch.Tensor,
                  staging: torch.Tensor) -> None:
        if grad_host.is_cuda or not grad_host.is_contiguous():
            raise TypeError("grad_host must be a contiguous CPU tensor (pinned for full speed)")
        gdt = {torch.float32: F32, torch.bfloat16: BF16}[grad_host.dtype]
        n = grad_host.numel()
        if m.numel() != n or v.numel() != n:
            raise ValueError("grad, m, v must have the same number of elements")
        self._check(self._L.adama_fold_host(
            self._h, grad_host.data_ptr(), gdt, _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), n, staging.data_ptr(),
            staging.numel() * staging.element_size(), _stream_ptr(self.device)))

    def linear_wgrad_fold_host(self, X_host: torch.Tensor, dY_host: torch.Tensor, m: torch.Tensor,
                               v: torch.Tensor, staging: torch.Tensor) -> None:
        if X_host.is_cuda or dY_host.is_cuda:
            raise TypeError("X_host, dY_host must be CPU tensors")
        if not (X_host.is_contiguous() and dY_host.is_contiguous()):
            raise ValueError("X_host, dY_host must be dense")
        if X_host.dtype != torch.bfloat16 or dY_host.dtype != torch.bfloat16:
            raise TypeError("X_host, dY_host must be bfloat16")
        tokens, d_in = X_host.shape
        d_out = dY_host.shape[1]
        if tuple(m.shape) != (d_in, d_out) or tuple(v.shape) != (d_in, d_out):
            raise ValueError("m, v must be [d_in, d_out]")
        self._check(self._L.adama_linear_wgrad_fold_host(
            self._h, X_host.data_ptr(), dY_host.data_ptr(), tokens, d_in, d_out,
            _dev_ptr(m, torch.float32, "m"), _dev_ptr(v, torch.float32, "v"), m.stride(0),
            staging.data_ptr(), staging.numel() * staging.element_size(),
            _stream_ptr(self.device)))

    def apply_to_host(self, w: torch.Tensor, m: torch.Tensor, v: torch.Tensor, lr: float,
                      w_host: torch.Tensor) -> None:
        n = w.numel()
        if w_host.is_cuda or w_host.dtype != torch.float32 or w_host.numel() != n:
            raise TypeError("w_host must be a CPU float32 tensor of w's size")
        self._check(self._L.adama_apply_to_host(
            self._h, _dev_ptr(w, torch.float32, "w"), _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), n, float(lr), w_host.data_ptr(),
            _stream_ptr(self.device)))

    # -- state ------------------------------------------------------------------------------
    @property
    def step(self) -> int:
        return int(self._L.adama_get_step(self._h))

    def set_step(self, t: int) -> None:
        self._check(self._L.adama_set_step(self._h, int(t)))

    def set_weight_decay(self, weight_decay: float) -> None:
        """adama_set_weight_decay: decoupled (AdamW) decay for all later applies; 0 turns it off."""
        self._check(self._L.adama_set_weight_decay(self._h, float(weight_decay)))

    @property
    def n_micro(self) -> int:
        return int(self._L.adama_get_n_micro(self._h))

    def sync_status(self) -> None:
        """Waits for the current stream and raises AdamAError(ERR_TIMEOUT) if a bounded
        device-side wait expired."""
        self._check(self._L.adama_sync_status(self._h, _stream_ptr(self.device)))

    def debug_set_status(self, code: int, wait: int = 0, tile: int = 0) -> None:
        """adama_debug_set_status (test hook for the time-out reporting path)."""
        self._check(self._L.adama_debug_set_status(self._h, code, wait, tile,
                                                   _stream_ptr(self.device)))

    def debug_wgrad_expire_wait(self, X: torch.Tensor, dY: torch.Tensor, m: torch.Tensor,
                                v: torch.Tensor, wait_limit_ns: int) -> None:
        """adama_debug_wgrad_expire_wait (test hook: a device-side wait that runs out and a
        kernel that returns all the same).  Dense 2-D tensors as for linear_wgrad_fold."""
        tokens, d_in = X.shape
        d_out = dY.shape[1]
        self._check(self._L.adama_debug_wgrad_expire_wait(
            self._h, _dev_ptr(X, torch.bfloat16, "X"), _dev_ptr(dY, torch.bfloat16, "dY"),
            tokens, d_in, d_out, X.stride(0), dY.stride(0), _dev_ptr(m, torch.float32, "m"),
            _dev_ptr(v, torch.float32, "v"), m.stride(0), int(wait_limit_ns),
            _stream_ptr(self.device)))

    def debug_set_wgrad_variant(self, epilogue: int = 0, epi_warps: int = 0, box_loads: int = 0,
                                no_pdl: int = 0) -> None:
        """adama_debug_set_wgrad_variant (test hook: pins the fused kernel's instance)."""
        self._check(self._L.adama_debug_set_wgrad_variant(self._h, epilogue, epi_warps, box_loads,
                                                          no_pdl))

    @property
    def launch_count(self) -> int:
        return int(self._L.adama_launch_count(self._h))


def linear_wgrad_fold_noalloc(X: torch.Tensor, dY: torch.Tensor, m: torch.Tensor, v: torch.Tensor,
                              n_micro: int, beta1=0.9, beta2=0.999, status_out=None,
                              grads_prescaled=False) -> None:
    """adama_linear_wgrad_fold_noalloc: the fused weight-gradient fold for callers that may
    not allocate device memory.  Needs no AdamA context; the kernel's status block is a
    fixed array inside the library.  `status_out`, if given, is a pinned CPU int32/uint32
    tensor of >= 4 elements that receives {code, wait, tile, 0} when the stream gets there."""
    L = load_library()
    tokens, d_in = X.shape
    d_out = dY.shape[1]
    dev = X.device.index if X.device.index is not None else torch.cuda.current_device()
    cfg = _Config(beta1, beta2, 0.0, dev, GRADS_PRESCALED if grads_prescaled else 0)
    err = ctypes.create_string_buffer(256)
    ldx = X.stride(0) if tokens > 1 else max(d_in, X.stride(0))
    ldy = dY.stride(0) if tokens > 1 else max(d_out, dY.stride(0))
    ldmv = m.stride(0) if d_in > 1 else max(d_out, m.stride(0))
    sp = None
    if status_out is not None:
        if status_out.is_cuda or status_out.numel() < 4 or status_out.element_size() != 4:
            raise TypeError("status_out must be a CPU tensor of >= 4 32-bit elements")
        sp = status_out.data_ptr()
    st = L.adama_linear_wgrad_fold_noalloc(
        ctypes.byref(cfg), int(n_micro), _dev_ptr(X, torch.bfloat16, "X"),
        _dev_ptr(dY, torch.bfloat16, "dY"), tokens, d_in, d_out, ldx, ldy,
        _dev_ptr(m, torch.float32, "m"), _dev_ptr(v, torch.float32, "v"), ldmv, sp, err, 256,
        _stream_ptr(torch.device("cuda", dev)))
    if st != 0:
        raise AdamAError(st, err.value.decode())


def debug_setup_state(device: int) -> int:
    """adama_debug_setup_state: bit 0 = tensor-map encoder resolved, bit 1 = kernel attributes
    set on `device` (no GPU needed)."""
    return int(load_library().adama_debug_setup_state(int(device)))


def version() -> str:
    return load_library().adama_version().decode()
