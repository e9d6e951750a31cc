"""GPU parity of the streaming kernels (adama_fold, adama_apply) against the fp64 oracle.

Tolerance (stated by the workload definition): relative L2 error <= 1e-6 on m, v and w.
Comparison points: m_t, v_t after the last fold of a mini-batch; w_t after apply; and after
apply the buffers hold beta1*m_t, beta2*v_t (the decay of the next Algorithm-2 iteration).
"""
import numpy as np
import pytest
import torch

import adama_workloads as wl
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from parity import Guarded, assert_close, f64, rel_l2

pytestmark = pytest.mark.gpu
TOL = 1e-6


def _run_flat(cfg: wl.FlatConfig, n: int, steps: int, offset=0, g_offset=0):
    """Runs cfg's flow on n elements on the GPU and in the oracle; asserts parity each step."""
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS)
    w0 = wl.normal((n,), cfg.w_std, torch.float32, wl.seed_for(cfg.config, 99))
    orc = AdamAOracle(f64(w0), wl.BETA1, wl.BETA2, wl.EPS)
    w = Guarded(n, offset=offset).fill(w0.cuda())
    m = Guarded(n, offset=offset).zero()
    v = Guarded(n, offset=offset).zero()
    g = Guarded(n, dtype=cfg.grad_dtype, offset=g_offset)
    for step in range(steps):
        opt.begin_minibatch(cfg.n_micro)
        orc.begin_minibatch(cfg.n_micro)
        for i in range(cfg.n_micro):
            grad = wl.normal((n,), cfg.grad_std, cfg.grad_dtype, wl.seed_for(cfg.config, step, i))
            g.fill(grad.cuda())
            opt.fold(g.view, m.view, v.view)
            orc.fold(f64(grad))
        assert_close(f64(m.view), orc.m, TOL, "m_t")
        assert_close(f64(v.view), orc.v, TOL, "v_t")
        opt.apply(w.view, m.view, v.view, wl.LR)
        orc.update(wl.LR)
        assert_close(f64(w.view), orc.theta, TOL, "w")
        assert_close(f64(m.view), wl.BETA1 * orc.m, TOL, "beta1*m")
        assert_close(f64(v.view), wl.BETA2 * orc.v, TOL, "beta2*v")
        assert opt.step == orc.t == step + 1
    for b in (w, m, v, g):
        b.check()
    opt.sync_status()
    assert opt.launch_count == steps * (cfg.n_micro + 1)
    opt.close()


def test_config1_full():
    """1024x1024 fp32 tensor, fp32 gradients, N=4, 3 steps, every element compared."""
    _run_flat(wl.CONFIG1, wl.CONFIG1.n, wl.CONFIG1.steps)


@pytest.mark.parametrize("n", [1 << 20, (1 << 20) + 1, 1_000_003, 1 << 22])
def test_config2_bf16_gradients(n):
    """bf16 gradients, N=8, 5 steps; sizes span many CTAs and include ragged tails."""
    _run_flat(wl.CONFIG2, n, wl.CONFIG2.steps)


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 7, 1023, 1025, 4099])
@pytest.mark.parametrize("dtype_cfg", [wl.CONFIG1, wl.CONFIG2])
def test_tiny_and_ragged_sizes(n, dtype_cfg):
    _run_flat(dtype_cfg, n, 2)


@pytest.mark.parametrize("offset,g_offset", [(1, 0), (0, 1), (3, 3), (2, 1)])
@pytest.mark.parametrize("dtype_cfg", [wl.CONFIG1, wl.CONFIG2])
def test_misaligned_pointers_take_the_scalar_path(offset, g_offset, dtype_cfg):
    _run_flat(dtype_cfg, 10_007, 2, offset=offset, g_offset=g_offset)


def test_empty_tensor_is_a_noop():
    opt = adama.AdamA()
    opt.begin_minibatch(2)
    e = torch.empty(0, device="cuda")
    opt.fold(e, e.clone(), e.clone())
    opt.apply(e.clone(), e.clone(), e.clone(), 1e-3)
    assert opt.launch_count == 0
    opt.close()


def test_n1_on_gpu_matches_oracle_adam():
    """N=1: the GPU path is standard Adam (Algorithm 1, both bracket terms coincide)."""
    cfg = wl.FlatConfig(config=7, n=50_000, n_micro=1, steps=4, grad_dtype=torch.float32,
                        grad_std=1e-2)
    _run_flat(cfg, cfg.n, cfg.steps)


def test_prescaled_gradients_flag():
    n, N = 4096, 4
    opt = adama.AdamA(grads_prescaled=True)
    orc = AdamAOracle(np.zeros(n))
    m = torch.zeros(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    opt.begin_minibatch(N)
    orc.begin_minibatch(N)
    for i in range(N):
        grad = wl.normal((n,), 1e-2, torch.float32, 500 + i)
        opt.fold((grad / N).cuda(), m, v)       # caller already divided by N
        orc.fold(f64(grad / N) * N)             # oracle divides by N itself
    assert rel_l2(f64(m), orc.m) <= TOL
    assert rel_l2(f64(v), orc.v) <= TOL
    opt.close()


def test_many_steps_decay_has_no_drift():
    """200 mini-batches.  Every fp32 rounding of the state (2 folds + a two-rounding decay
    per step = 800 per element) adds an independent error of about 2^-24/sqrt(3) * 1.4
    relative, so a random walk of ~sqrt(800) * 4.8e-8 = 1.4e-6 is what fp32 state must show;
    the bound is twice that.  What must NOT appear is a bias: a plain fp32 beta2 (relative
    error 1.3e-8) would shift every element of v by about -1.3e-6 after 200 steps, which the
    mean signed error (noise 1.4e-6/sqrt(n)) exposes.
    The first moment forgets: with beta1 = 0.9 a rounding made k steps ago survives with weight
    beta1^k, so its error is the geometric sum sqrt(4/(1-beta1^2)) = 4.6 roundings' worth,
    2.2e-7 relative to the size of m, however many steps are run; the bound is twice that, and
    a bias in its decay would show in w (below) long before it showed in m."""
    n, N, steps = 4096, 2, 200
    opt = adama.AdamA()
    w0 = wl.normal((n,), 0.02, torch.float32, 1)
    orc = AdamAOracle(f64(w0))
    w, m, v = w0.cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    for step in range(steps):
        opt.begin_minibatch(N)
        orc.begin_minibatch(N)
        for i in range(N):
            grad = wl.normal((n,), 1e-2, torch.float32, 9000 + 10 * step + i)
            opt.fold(grad.cuda(), m, v)
            orc.fold(f64(grad))
        opt.apply(w, m, v, wl.LR)
        orc.update(wl.LR)
    random_walk = np.sqrt(4 * steps) * 2.0 ** -24 / np.sqrt(3) * 1.4
    want_v = wl.BETA2 * orc.v
    assert rel_l2(f64(v), want_v) <= 2 * random_walk
    bias = float(np.mean((f64(v) - want_v) / want_v))
    assert abs(bias) <= 2e-7, bias
    forgetful_walk = np.sqrt(4 / (1 - wl.BETA1 ** 2)) * 2.0 ** -24 / np.sqrt(3) * 1.4
    assert rel_l2(f64(m), wl.BETA1 * orc.m) <= 2 * forgetful_walk
    assert rel_l2(f64(w), orc.theta) <= TOL
    opt.close()


def test_full_size_config2_sampled():
    """335M-element buffer, bf16 gradients, N=8, one mini-batch in the benchmark's launch
    configuration; a strided sample plus head and tail are checked element by element
    (elementwise op: any subset is a valid check)."""
    n = wl.CONFIG2_FULL_N
    cfg = wl.CONFIG2
    idx = torch.cat([torch.arange(0, 4096), torch.arange(n - 4099, n),
                     torch.arange(0, n, 331)]).unique()
    idx_d = idx.cuda()
    opt = adama.AdamA()
    w = wl.normal((n,), cfg.w_std, torch.float32, wl.seed_for(2, 99), device="cuda")
    m = torch.zeros(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    orc = AdamAOracle(f64(w[idx_d]))
    opt.begin_minibatch(cfg.n_micro)
    orc.begin_minibatch(cfg.n_micro)
    for i in range(cfg.n_micro):
        g = wl.normal((n,), cfg.grad_std, torch.bfloat16, wl.seed_for(2, 0, i), device="cuda")
        opt.fold(g, m, v)
        orc.fold(f64(g[idx_d]))
        del g
    assert rel_l2(f64(m[idx_d]), orc.m) <= TOL
    assert rel_l2(f64(v[idx_d]), orc.v) <= TOL
    opt.apply(w, m, v, wl.LR)
    orc.update(wl.LR)
    assert rel_l2(f64(w[idx_d]), orc.theta) <= TOL
    assert rel_l2(f64(m[idx_d]), wl.BETA1 * orc.m) <= TOL
    assert rel_l2(f64(v[idx_d]), wl.BETA2 * orc.v) <= TOL
    # properties that hold at any size: v >= 0 everywhere, nothing non-finite
    assert bool((v >= 0).all()) and bool(torch.isfinite(w).all()) and bool(torch.isfinite(m).all())
    opt.sync_status()
    opt.close()


def test_more_than_2_to_32_elements_sampled():
    """n = 2^32 + 7: element indices and byte offsets beyond 32 bits (the largest size the
    workloads reach is 335 M; this is the index-arithmetic edge).  One mini-batch with N = 2;
    head, tail and windows around 2^31 and 2^32 are checked element by element."""
    n = (1 << 32) + 7
    win = torch.arange(-2050, 2050)
    idx = torch.cat([torch.arange(0, 4096), (1 << 31) + win, (1 << 32) + win[win < 7],
                     torch.arange(0, n, 1_000_003)]).unique()
    idx = idx[(idx >= 0) & (idx < n)]
    idx_d = idx.cuda()
    opt = adama.AdamA()
    w = wl.normal((n,), 0.02, torch.float32, wl.seed_for(9, 99), device="cuda")
    m = torch.zeros(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    orc = AdamAOracle(f64(w[idx_d]))
    opt.begin_minibatch(2)
    orc.begin_minibatch(2)
    for i in range(2):
        g = wl.normal((n,), 1e-3, torch.bfloat16, wl.seed_for(9, 0, i), device="cuda")
        opt.fold(g, m, v)
        orc.fold(f64(g[idx_d]))
        del g
    assert rel_l2(f64(m[idx_d]), orc.m) <= TOL
    assert rel_l2(f64(v[idx_d]), orc.v) <= TOL
    opt.apply(w, m, v, wl.LR)
    orc.update(wl.LR)
    assert rel_l2(f64(w[idx_d]), orc.theta) <= TOL
    assert rel_l2(f64(m[idx_d]), wl.BETA1 * orc.m) <= TOL
    assert rel_l2(f64(v[idx_d]), wl.BETA2 * orc.v) <= TOL
    # every element was visited exactly once: with two N(0, 1e-3) gradients v > 0 almost surely,
    # and a second visit would show as a second decay
    assert int((v == 0).sum()) < 1000
    opt.sync_status()
    opt.close()
    del w, m, v
    torch.cuda.empty_cache()


def test_decoupled_weight_decay_extension():
    """adama_set_weight_decay (AdamW-style, beyond the paper's algorithms) against the oracle's
    pinned decoupled-decay update; and lambda = 0 stays bit-identical to the plain update."""
    n, N, wd = 70_001, 2, 0.1
    w0 = wl.normal((n,), 0.5, torch.float32, 12)
    orc = AdamAOracle(f64(w0))
    opt = adama.AdamA()
    opt.set_weight_decay(wd)
    plain, zero = adama.AdamA(), adama.AdamA()
    zero.set_weight_decay(0.0)
    w, m, v = w0.cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    wp, mp, vp = w0.cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    wz, mz, vz = w0.cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    for step in range(3):
        for o in (opt, plain, zero):
            o.begin_minibatch(N)
        orc.begin_minibatch(N)
        for i in range(N):
            g = wl.normal((n,), 1e-2, torch.float32, 300 + 10 * step + i)
            opt.fold(g.cuda(), m, v)
            plain.fold(g.cuda(), mp, vp)
            zero.fold(g.cuda(), mz, vz)
            orc.fold(f64(g))
        opt.apply(w, m, v, wl.LR)
        plain.apply(wp, mp, vp, wl.LR)
        zero.apply(wz, mz, vz, wl.LR)
        orc.update(wl.LR, weight_decay=wd)
        assert rel_l2(f64(w), orc.theta) <= TOL
        assert torch.equal(wp, wz)
    assert not torch.equal(w, wp)
    with pytest.raises(adama.AdamAError):
        opt.set_weight_decay(-1.0)
    for o in (opt, plain, zero):
        o.close()


@pytest.mark.parametrize("n,offset", [(1_000_003, 0), (4099, 0), (10_007, 1), (5, 0)])
def test_apply_with_bf16_copy(n, offset):
    """The bf16 copy is the round-to-nearest-even of the fp32 result, and w, m, v are the same
    bits as plain apply gives (vector and scalar paths)."""
    g = wl.normal((n,), 1e-2, torch.float32, 77).cuda()
    res = []
    for copy in (False, True):
        opt = adama.AdamA()
        opt.begin_minibatch(1)
        w = Guarded(n, offset=offset).fill(wl.normal((n,), 0.02, torch.float32, 78).cuda())
        m, v = Guarded(n, offset=offset).zero(), Guarded(n, offset=offset).zero()
        wb = Guarded(n, dtype=torch.bfloat16, offset=offset)
        opt.fold(g, m.view, v.view)
        if copy:
            opt.apply_bf16_copy(w.view, m.view, v.view, wb.view, wl.LR)
            assert torch.equal(wb.view, w.view.to(torch.bfloat16))
        else:
            opt.apply(w.view, m.view, v.view, wl.LR)
        for b in (w, m, v, wb):
            b.check()
        res.append((w.view.clone(), m.view.clone(), v.view.clone()))
        opt.close()
    assert all(torch.equal(a, b) for a, b in zip(*res))
