"""GPU parity of the two additions beside Algorithm 2: SGD with momentum on the same pipeline
(adama_sgdm_fold / adama_sgdm_apply) and the coefficient statistics of Section 4.1
(adama_coefficient_stats), each against the fp64 oracle."""
import numpy as np
import pytest
import torch

import adama_workloads as wl
import oracle
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle, SGDMOracle
from parity import Guarded, f64, rel_l2

pytestmark = pytest.mark.gpu
TOL = 1e-6


# ----- SGD with momentum -----------------------------------------------------------------------

def _run_sgdm(n, dtype, N, steps, mu=0.9, lr=0.05, offset=0, g_offset=0):
    opt = adama.AdamA()
    w0 = wl.normal((n,), 0.02, torch.float32, wl.seed_for(6, 99))
    orc = SGDMOracle(f64(w0), momentum=mu)
    w = Guarded(n, offset=offset).fill(w0.cuda())
    buf = Guarded(n, offset=offset).zero()
    g = Guarded(n, dtype=dtype, offset=g_offset)
    for step in range(steps):
        opt.begin_minibatch(N)
        orc.begin_minibatch(N)
        for i in range(N):
            grad = wl.normal((n,), 1e-2, dtype, wl.seed_for(6, step, i))
            g.fill(grad.cuda())
            opt.sgdm_fold(g.view, buf.view)
            orc.fold(f64(grad))
        assert rel_l2(f64(buf.view), orc.buf) <= TOL
        opt.sgdm_apply(w.view, buf.view, lr, mu)
        orc.update(lr)
        assert rel_l2(f64(w.view), orc.theta) <= TOL
        assert rel_l2(f64(buf.view), mu * orc.buf) <= TOL   # decayed for the next mini-batch
    for b in (w, buf, g):
        b.check()
    assert opt.launch_count == steps * (N + 1)
    opt.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n", [1, 3, 1025, 1_000_003, 1 << 21])
def test_sgdm_matches_oracle(n, dtype):
    _run_sgdm(n, dtype, N=4, steps=3)


@pytest.mark.parametrize("offset,g_offset", [(1, 0), (0, 1), (3, 2)])
def test_sgdm_misaligned_pointers(offset, g_offset):
    _run_sgdm(10_007, torch.bfloat16, N=2, steps=2, offset=offset, g_offset=g_offset)


def test_sgdm_argument_errors():
    opt = adama.AdamA()
    w = torch.zeros(8, device="cuda")
    buf = torch.zeros(8, device="cuda")
    with pytest.raises(adama.AdamAError) as e:
        opt.sgdm_fold(w, buf)
    assert e.value.status == adama.Status.ERR_BAD_STATE
    with pytest.raises(adama.AdamAError) as e:
        opt.sgdm_apply(w, buf, 0.1, 0.9)
    assert e.value.status == adama.Status.ERR_BAD_STATE
    opt.begin_minibatch(2)
    for bad in (1.0, -0.1, float("nan")):
        with pytest.raises(adama.AdamAError) as e:
            opt.sgdm_apply(w, buf, 0.1, bad)
        assert e.value.status == adama.Status.ERR_INVALID_ARG
    with pytest.raises(adama.AdamAError) as e:
        opt.sgdm_apply(w, buf, float("inf"), 0.9)
    assert e.value.status == adama.Status.ERR_INVALID_ARG
    e0 = torch.empty(0, device="cuda")
    opt.sgdm_fold(e0, e0.clone())
    opt.sgdm_apply(e0.clone(), e0.clone(), 0.1, 0.9)
    assert opt.launch_count == 0
    opt.close()


# ----- coefficient statistics ------------------------------------------------------------------

def _stats(t):
    s = t.cpu().numpy()
    cnt = int(s[3])
    return {"sum": s[0], "min": s[1], "max": s[2], "count": cnt,
            "mean": s[0] / cnt if cnt else float("nan")}


def _run_coef(n, N, steps, grads_fn, beta1=wl.BETA1, beta2=wl.BETA2, offset=0, check=None):
    """Runs `steps` mini-batches on the GPU (states in fp32, Adam's v' derived from the change of
    m) and in the oracle (Adam's v' from the materialised gradients, Algorithm 1's first bracket
    term); yields both statistics per step to `check`."""
    opt = adama.AdamA(beta1, beta2, wl.EPS)
    orc = AdamAOracle(np.zeros(n), beta1, beta2, wl.EPS)
    m_adam, v_adam_o = np.zeros(n), np.zeros(n)
    w = torch.zeros(n, device="cuda")
    m = Guarded(n, offset=offset).zero()
    v = Guarded(n, offset=offset).zero()
    va = Guarded(n, offset=offset).zero()
    m_begin = Guarded(n, offset=offset).zero()
    stats = torch.full((4,), -1.0, dtype=torch.float64, device="cuda")
    for step in range(steps):
        opt.begin_minibatch(N)
        orc.begin_minibatch(N)
        m_begin.view.copy_(m.view)
        grads = [grads_fn(step, i) for i in range(N)]
        for grad in grads:
            opt.fold(grad.cuda(), m.view, v.view)
            orc.fold(f64(grad))
        opt.coefficient_stats(m.view, None if step == 0 else m_begin.view, v.view, va.view, stats)
        m_adam, v_adam_o = oracle.closed_form_moments(m_adam, v_adam_o,
                                                      np.stack([f64(g) for g in grads]), beta1,
                                                      beta2, adam_variant=True)
        want = oracle.coefficient_stats(orc.v, v_adam_o, orc.t, beta2)
        check(step, _stats(stats), want, f64(va.view), beta2 * v_adam_o)
        opt.apply(w, m.view, v.view, wl.LR)
        orc.update(wl.LR)
    for b in (m, v, va, m_begin):
        b.check()
    opt.close()


@pytest.mark.parametrize("n", [5, 4099, 1 << 20])
def test_coefficient_exact_arithmetic_case(n):
    """beta1 = 0.5, beta2 = 0.75, N = 4 and small integer gradients: every fp32 operation of the
    folds, of m - m_begin and of Adam's v' is exact, so only the fp32 rounding of the division
    and root (and of the stored beta2*v') is left between the GPU and the oracle."""
    def grads(step, i):
        return wl.small_integers((n,), 6, torch.float32, wl.seed_for(7, step, i))

    def check(step, got, want, va_gpu, va_want):
        assert got["count"] == want["count"]
        for key in ("mean", "min", "max"):
            assert got[key] == pytest.approx(want[key], rel=3e-7)
        assert rel_l2(va_gpu, va_want) <= 1e-7

    _run_coef(n, 4, 3, grads, beta1=0.5, beta2=0.75, check=check)


@pytest.mark.parametrize("N", [1, 2, 8])
def test_coefficient_identical_micro_gradients(N):
    """Identical micro-batch gradients: the coefficient is 1/sqrt(N) at every element and step."""
    n = 300_001
    base = {}

    def grads(step, i):
        if step not in base:
            base[step] = wl.normal((n,), 1e-2, torch.float32, wl.seed_for(7, step, 50))
        return base[step]

    def check(step, got, want, va_gpu, va_want):
        assert got["count"] == want["count"] == n
        for key in ("mean", "min", "max"):
            assert want[key] == pytest.approx(1 / np.sqrt(N), rel=1e-10)   # serial fp64 sum of n
            # fp32 states: each of v, v' carries ~N roundings of 6e-8; the root halves them
            assert got[key] == pytest.approx(1 / np.sqrt(N), rel=2e-6)

    _run_coef(n, N, 3, grads, check=check)


@pytest.mark.parametrize("offset", [0, 1])
def test_coefficient_random_gradients_with_history(offset):
    """bf16 normal gradients (the flat workload's distribution), N = 8.  Adam's v' is recovered
    from d = m - m_begin in fp32: |err(d)| ~ sqrt(N) * 2^-24 * |m|, so an element's v'
    increment k*d^2 carries a relative error ~ 4e-7 * |m|/|d|.  From the second mini-batch on v'
    has history and the statistics are well conditioned: mean and min to 1e-5; max sits at the
    elements whose v' is smallest, |d| ~ 1e-3 of typical over 1 M elements: 5e-3.  At t = 1
    c = sqrt(v)/|d|*const has no finite mean for continuous data, so nothing but the
    stored v' is compared there.  The stored v' itself: relative L2 5e-6."""
    n = 1 << 20

    def grads(step, i):
        g = wl.normal((n,), 1e-3, torch.bfloat16, wl.seed_for(7, step, i))
        g[:17] = 0          # elements that never see a gradient are not counted
        return g

    def check(step, got, want, va_gpu, va_want):
        assert rel_l2(va_gpu, va_want) <= 5e-6
        if step == 0:
            # bf16 gradients sit on a grid, so some exact sums are 0 (no coefficient) where the
            # fp32 accumulation leaves a tiny residue (a huge one): the counts differ slightly
            assert got["count"] <= n - 17 and abs(got["count"] - want["count"]) <= n // 1000
        else:
            assert got["count"] == want["count"] == n - 17
            assert got["mean"] == pytest.approx(want["mean"], rel=1e-5)
            assert got["min"] == pytest.approx(want["min"], rel=1e-5)
            assert got["max"] == pytest.approx(want["max"], rel=5e-3)
            assert got["min"] >= 1 / np.sqrt(8) * (1 - 1e-5)      # Cauchy-Schwarz floor

    _run_coef(n, 8, 4, grads, offset=offset, check=check)


def test_coefficient_empty_and_errors():
    opt = adama.AdamA()
    stats = torch.full((4,), -1.0, dtype=torch.float64, device="cuda")
    e0 = torch.empty(0, device="cuda")
    with pytest.raises(adama.AdamAError) as e:
        opt.coefficient_stats(e0, None, e0, e0, stats)
    assert e.value.status == adama.Status.ERR_BAD_STATE
    opt.begin_minibatch(1)
    opt.coefficient_stats(e0, None, e0.clone(), e0.clone(), stats)
    s = stats.cpu().numpy()
    assert s[0] == 0 and s[1] == np.inf and s[2] == 0 and s[3] == 0
    # all-zero states: nothing counted
    z = torch.zeros(1000, device="cuda")
    opt.coefficient_stats(z, None, z.clone(), z.clone(), stats)
    assert _stats(stats)["count"] == 0
    with pytest.raises(ValueError):
        opt.coefficient_stats(z, None, z, z, torch.zeros(3, dtype=torch.float64, device="cuda"))
    opt.close()
