"""Call-order, argument and alignment errors of the C ABI on a GPU machine (all rejected on
the host; nothing here launches a faulty kernel)."""
import pytest
import torch

import paper_2305_19982_b200 as adama
from paper_2305_19982_b200 import Status

pytestmark = pytest.mark.gpu


def _err(fn, *a):
    with pytest.raises(adama.AdamAError) as e:
        fn(*a)
    return e.value.status


def test_call_order():
    opt = adama.AdamA()
    x = torch.zeros(16, device="cuda")
    assert _err(opt.fold, x, x.clone(), x.clone()) == Status.ERR_BAD_STATE
    assert _err(opt.apply, x, x.clone(), x.clone(), 1e-3) == Status.ERR_BAD_STATE
    X = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    mm = torch.zeros(64, 64, device="cuda")
    assert _err(opt.linear_wgrad_fold, X, X, mm, mm.clone()) == Status.ERR_BAD_STATE
    assert _err(opt.begin_minibatch, 0) == Status.ERR_INVALID_ARG
    assert opt.step == 0
    opt.begin_minibatch(3)
    assert opt.step == 1 and opt.n_micro == 3
    opt.close()


def test_bad_hyperparameters():
    for kw in (dict(beta1=1.0), dict(beta2=-0.5), dict(eps=-1.0)):
        with pytest.raises(adama.AdamAError) as e:
            adama.AdamA(**kw)
        assert e.value.status == Status.ERR_INVALID_ARG


def test_wgrad_alignment_and_shape_errors():
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    bf = dict(dtype=torch.bfloat16, device="cuda")
    X = torch.zeros(64, 72, **bf)
    dY = torch.zeros(64, 80, **bf)
    m = torch.zeros(72, 80, device="cuda")
    v = torch.zeros(72, 80, device="cuda")
    opt.linear_wgrad_fold(X, dY, m, v)  # fine
    # row pitch not a multiple of 8 elements
    assert _err(opt.linear_wgrad_fold, torch.zeros(64, 70, **bf), dY,
                torch.zeros(70, 80, device="cuda"), torch.zeros(70, 80, device="cuda")) == Status.ERR_MISALIGNED
    # m pitch not a multiple of 4
    assert _err(opt.linear_wgrad_fold, X, torch.zeros(64, 82, **bf)[:, :82],
                torch.zeros(72, 82, device="cuda"), torch.zeros(72, 82, device="cuda")) == Status.ERR_MISALIGNED
    # base pointer not 16-byte aligned
    Xo = torch.zeros(64 * 72 + 8, **bf)[1:1 + 64 * 72].view(64, 72)
    assert _err(opt.linear_wgrad_fold, Xo, dY, m, v) == Status.ERR_MISALIGNED
    opt.sync_status()
    opt.close()


def test_set_step_round_trip():
    opt = adama.AdamA()
    opt.set_step(41)
    opt.begin_minibatch(2)
    assert opt.step == 42
    assert _err(opt.set_step, -1) == Status.ERR_INVALID_ARG
    opt.close()


def test_host_staging_checks():
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    g = torch.zeros(1024, dtype=torch.bfloat16).pin_memory()
    m = torch.zeros(1024, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert _err(opt.fold_host, g, m, m.clone(), small) == Status.ERR_INVALID_ARG
    opt.close()
