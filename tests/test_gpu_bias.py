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
