"""CPU-side checks of the boundary: the shared library loads without a GPU, exports every
symbol the header declares, and derives its fp32 constants in double (Algorithm 2's
(1-beta)/N scalings and bias corrections)."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import paper_2305_19982_b200 as adama
from paper_2305_19982_b200 import build as adama_build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    adama_build.build()
    return adama.load_library()


def _declared_symbols():
    text = (ROOT / "include" / "adama.h").read_text()
    return sorted(set(re.findall(r"ADAMA_API[^;(]*?\b(adama_\w+)\s*\(", text)))


def test_header_symbols_all_exported(lib):
    declared = _declared_symbols()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in adama.h but not exported"
    assert sorted(adama.EXPORTED_SYMBOLS) == declared


def test_version(lib):
    assert re.fullmatch(r"\d+\.\d+\.\d+", lib.adama_version().decode())


@pytest.mark.parametrize("N,t,lr", [(1, 1, 1e-3), (8, 3, 1e-3), (16, 1000, 3e-4), (4, 100000, 1.0)])
def test_host_constants_are_formed_in_double(N, t, lr):
    b1, b2, eps = 0.9, 0.999, 1e-8
    c = adama.host_constants(b1, b2, eps, N, t, lr)
    f32 = lambda x: float(np.float32(x))
    assert c[0] == f32((1 - b1) / N)
    assert c[1] == f32((1 - b2) / (N * N))
    assert c[2] == f32(lr / (1 - b1 ** t))
    assert c[3] == f32(1 / (1 - b2 ** t))
    assert c[4] == f32(eps)
    # hi + lo reproduces the double beta far below fp32 resolution
    assert abs((c[5] + c[6]) - b1) < 1e-14
    assert abs((c[7] + c[8]) - b2) < 1e-14
    # the naive fp32 route (1 - float(beta2)) would be off by ~1e-5 relative; ours is not
    naive = float(np.float32(1) - np.float32(b2)) / (N * N)
    assert abs(c[1] - (1 - b2) / (N * N)) / ((1 - b2) / (N * N)) < 1e-7
    assert abs(naive - (1 - b2) / (N * N)) / ((1 - b2) / (N * N)) > 1e-6


def test_host_constants_prescaled_flag():
    c = adama.host_constants(0.9, 0.999, 1e-8, 8, 1, 1e-3, flags=1)
    assert c[0] == float(np.float32(1 - 0.9))
    assert c[1] == float(np.float32(1 - 0.999))


def test_host_constants_reject_bad_arguments():
    for args in [(1.0, 0.999, 1e-8, 1, 1, 1e-3), (0.9, -0.1, 1e-8, 1, 1, 1e-3),
                 (0.9, 0.999, -1.0, 1, 1, 1e-3), (0.9, 0.999, 1e-8, 0, 1, 1e-3),
                 (0.9, 0.999, 1e-8, 1, 0, 1e-3)]:
        with pytest.raises(adama.AdamAError) as e:
            adama.host_constants(*args)
        assert e.value.status == adama.Status.ERR_INVALID_ARG


def test_null_context_calls_do_not_crash(lib):
    assert lib.adama_begin_minibatch(None, 4) == adama.Status.ERR_INVALID_ARG
    assert lib.adama_fold(None, None, 0, None, None, 0, None) == adama.Status.ERR_INVALID_ARG
    assert lib.adama_apply(None, None, None, None, 0, 1e-3, None) == adama.Status.ERR_INVALID_ARG
    assert lib.adama_destroy(None) == adama.Status.OK
    assert lib.adama_get_step(None) == -1


def test_init_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(adama.AdamAError):
        adama.AdamA()


def test_setup_bookkeeping_is_per_device_and_starts_empty():
    """The fused kernel's attributes are per device: the table that remembers them answers
    "not set up" for every device no launch has run on, and for ordinals outside the table
    (those are set up on every call).  No GPU needed: nothing has been launched here."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("another test in this process may already have launched on device 0")
    for dev in (0, 1, 7, 63, 64, 1000, -1):
        assert adama.debug_setup_state(dev) & 2 == 0


def test_config_flags_known_and_unknown():
    """The three configuration flags are accepted, any other bit is refused (host-only check)."""
    for flags in (0, 1, 2, 4, 7):
        adama.host_constants(0.9, 0.999, 1e-8, 4, 1, 1e-3, flags=flags)
    for flags in (8, 16, 1 << 31):
        with pytest.raises(adama.AdamAError) as e:
            adama.host_constants(0.9, 0.999, 1e-8, 4, 1, 1e-3, flags=flags)
        assert e.value.status == adama.Status.ERR_INVALID_ARG
