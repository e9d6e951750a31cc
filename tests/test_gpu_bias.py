"""adama_bias_grad_fold against the oracle: the bias gradient of a linear layer is the column
sum of dY, which the oracle forms as linear_wgrad(ones[T,1], dY) (naive loop, fp64)."""
import numpy as np
import pytest
import torch

import adama_workloads as wl
import oracle
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from parity import SENTINEL, f64, rel_l2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d_out,integer", [(4096, 4096, False), (100, 328, True), (7, 8, True),
                                             (1000, 1603, True), (4096, 1600, False), (1, 130, True)])
def test_bias_grad_fold(T, d_out, integer):
    N, steps = 2, 2
    opt = adama.AdamA()
    orc = AdamAOracle(np.zeros(d_out))
    ldy = (d_out + 7) // 8 * 8 + 8
    buf_m = torch.full((d_out + 16,), SENTINEL, device="cuda")
    buf_v = torch.full((d_out + 16,), SENTINEL, device="cuda")
    m, v = buf_m[8:8 + d_out], buf_v[8:8 + d_out]
    m.zero_()
    v.zero_()
    w = torch.zeros(d_out, device="cuda")
    for step in range(steps):
        opt.begin_minibatch(N)
        orc.begin_minibatch(N)
        for i in range(N):
            if integer:
                dY = wl.small_integers((T, d_out), 3, torch.bfloat16, 40 + 10 * step + i)
            else:
                dY = wl.normal((T, d_out), 1e-2, torch.bfloat16, 40 + 10 * step + i)
            Yb = torch.full((T, ldy), 5.0, dtype=torch.bfloat16, device="cuda")
            Yb[:, :d_out] = dY.cuda()
            opt.bias_grad_fold(Yb[:, :d_out], m, v)
            orc.fold(oracle.linear_wgrad(np.ones((T, 1)), f64(dY))[0])
        tol = 1e-6 if integer else 2e-3
        assert rel_l2(f64(m), orc.m) <= tol
        assert rel_l2(f64(v), orc.v) <= tol
        mc, vc = m.contiguous(), v.contiguous()
        opt.apply(w, mc, vc, wl.LR)
        m.copy_(mc)
        v.copy_(vc)
        orc.update(wl.LR)
        assert rel_l2(f64(w), orc.theta) <= tol
    assert bool((buf_m[:8] == SENTINEL).all()) and bool((buf_m[8 + d_out:] == SENTINEL).all())
    assert bool((buf_v[:8] == SENTINEL).all()) and bool((buf_v[8 + d_out:] == SENTINEL).all())
    opt.sync_status()
    opt.close()


def test_bias_grad_deterministic_and_noop():
    dY = wl.normal((512, 1600), 1e-2, torch.bfloat16, 9).cuda()
    outs = []
    for _ in range(2):
        opt = adama.AdamA()
        opt.begin_minibatch(1)
        m, v = torch.zeros(1600, device="cuda"), torch.zeros(1600, device="cuda")
        opt.bias_grad_fold(dY, m, v)
        opt.bias_grad_fold(dY[:0], m, v)       # zero tokens: nothing happens
        assert opt.launch_count == 1
        outs.append((m.clone(), v.clone()))
        opt.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("T,d_in,d_out,integer", [(4096, 512, 4096, False), (100, 200, 328, True),
                                                  (7, 8, 8, True), (1000, 130, 1603, True),
                                                  (2048, 1600, 1600, False), (1, 3, 130, True),
                                                  (777, 300, 11008, True)])
def test_fused_bias_in_the_weight_gradient_launch(T, d_in, d_out, integer):
    """adama_linear_wgrad_bias_fold: the bias moments against the oracle (column sums of dY by
    the naive loop), the weight moments bit-identical to the plain fused call, guard bands
    around the bias moments untouched; d_out spans ragged 32-column slabs and more slabs than
    CTAs."""
    N = 2
    opt, ref = adama.AdamA(), adama.AdamA()
    orc = AdamAOracle(np.zeros(d_out))
    buf_m = torch.full((d_out + 16,), SENTINEL, device="cuda")
    buf_v = torch.full((d_out + 16,), SENTINEL, device="cuda")
    mb, vb = buf_m[8:8 + d_out], buf_v[8:8 + d_out]
    mb.zero_()
    vb.zero_()
    up = lambda x, k: (x + k - 1) // k * k
    ldx, ldy, ldmv = up(d_in, 8) + 8, up(d_out, 8) + 8, up(d_out, 4) + 4   # padded row pitches
    m = torch.zeros(d_in, ldmv, device="cuda")[:, :d_out]
    v = torch.zeros(d_in, ldmv, device="cuda")[:, :d_out]
    m_ref = torch.zeros(d_in, ldmv, device="cuda")[:, :d_out]
    v_ref = torch.zeros(d_in, ldmv, device="cuda")[:, :d_out]
    for step in range(2):
        opt.begin_minibatch(N)
        ref.begin_minibatch(N)
        orc.begin_minibatch(N)
        for i in range(N):
            seed = 60 + 10 * step + i
            if integer:
                X = wl.small_integers((T, d_in), 3, torch.bfloat16, seed)
                dY = wl.small_integers((T, d_out), 3, torch.bfloat16, seed + 100)
            else:
                X = wl.normal((T, d_in), 1.0, torch.bfloat16, seed)
                dY = wl.normal((T, d_out), 1e-2, torch.bfloat16, seed + 100)
            Xd = torch.full((T, ldx), 7.0, dtype=torch.bfloat16, device="cuda")[:, :d_in]
            Yd = torch.full((T, ldy), 7.0, dtype=torch.bfloat16, device="cuda")[:, :d_out]
            Xd.copy_(X)
            Yd.copy_(dY)
            opt.linear_wgrad_fold(Xd, Yd, m, v, mb, vb)
            ref.linear_wgrad_fold(Xd, Yd, m_ref, v_ref)
            orc.fold(oracle.linear_wgrad(np.ones((T, 1)), f64(dY))[0])
        tol = 1e-6 if integer else 2e-3
        assert rel_l2(f64(mb), orc.m) <= tol
        assert rel_l2(f64(vb), orc.v) <= tol
        assert torch.equal(m, m_ref) and torch.equal(v, v_ref)
        # between mini-batches the library's buffers hold the decayed moments (what an apply
        # leaves behind); the oracle decays in its own begin_minibatch
        mb.copy_(torch.from_numpy(wl.BETA1 * orc.m).float())
        vb.copy_(torch.from_numpy(wl.BETA2 * orc.v).float())
        orc.m = mb.cpu().double().numpy() / wl.BETA1
        orc.v = vb.cpu().double().numpy() / wl.BETA2
        m.mul_(wl.BETA1)
        v.mul_(wl.BETA2)
        m_ref.mul_(wl.BETA1)
        v_ref.mul_(wl.BETA2)
    assert bool((buf_m[:8] == SENTINEL).all()) and bool((buf_m[8 + d_out:] == SENTINEL).all())
    assert bool((buf_v[:8] == SENTINEL).all()) and bool((buf_v[8 + d_out:] == SENTINEL).all())
    opt.sync_status()
    ref.sync_status()
    assert opt.launch_count == 4      # one launch per call: no separate bias kernel
    opt.close()
    ref.close()


def test_fused_bias_is_deterministic_and_checks_arguments():
    X = wl.normal((512, 256), 1.0, torch.bfloat16, 3).cuda()
    dY = wl.normal((512, 1600), 1e-2, torch.bfloat16, 4).cuda()
    outs = []
    for _ in range(2):
        opt = adama.AdamA()
        opt.begin_minibatch(1)
        m, v = torch.zeros(256, 1600, device="cuda"), torch.zeros(256, 1600, device="cuda")
        mb, vb = torch.zeros(1600, device="cuda"), torch.zeros(1600, device="cuda")
        opt.linear_wgrad_fold(X, dY, m, v, mb, vb)
        outs.append((mb.clone(), vb.clone()))
        with pytest.raises(ValueError):
            opt.linear_wgrad_fold(X, dY, m, v, mb, None)
        with pytest.raises(ValueError):
            opt.linear_wgrad_fold(X, dY, m, v, mb[:100], vb[:100])
        opt.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
