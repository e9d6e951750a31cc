"""adama_apply_allreduced on one GPU: R data-parallel ranks are emulated one after the other
with separate state buffers (no kernels waiting on each other), their m and v are summed with
a torch add standing in for the all-reduce, and every rank applies.  Section 3.3, Eqs. 4-7:
the result must equal single-device AdamA with N*R micro-batches (fp64 oracle)."""
import pytest
import torch

import adama_workloads as wl
import paper_2305_19982_b200 as adama
from oracle import AdamADDPOracle, AdamAOracle
from parity import f64, rel_l2

pytestmark = pytest.mark.gpu
TOL = 1e-6


@pytest.mark.parametrize("R,N", [(2, 3), (4, 2), (8, 1)])
def test_allreduced_apply_equals_single_device(R, N):
    n, steps = 100_003, 3
    w0 = wl.normal((n,), 0.02, torch.float32, 1)
    single = AdamAOracle(f64(w0))
    ddp_orc = AdamADDPOracle(f64(w0), R)
    opts = [adama.AdamA() for _ in range(R)]
    w = [w0.cuda() for _ in range(R)]
    m = [torch.zeros(n, device="cuda") for _ in range(R)]
    v = [torch.zeros(n, device="cuda") for _ in range(R)]
    for step in range(steps):
        single.begin_minibatch(N * R)
        ddp_orc.begin_minibatch(N)
        for r in range(R):
            opts[r].begin_minibatch(N)
            for i in range(N):
                g = wl.normal((n,), 1e-2, torch.float32, 1000 * step + 10 * r + i + 7)
                opts[r].fold(g.cuda(), m[r], v[r])
                single.fold(f64(g))
                ddp_orc.fold(r, f64(g))
        m_sum = torch.stack(m).sum(0)          # stands in for all-reduce(SUM)
        v_sum = torch.stack(v).sum(0)
        for r in range(R):
            m[r].copy_(m_sum)
            v[r].copy_(v_sum)
            opts[r].apply_allreduced(w[r], m[r], v[r], wl.LR, R)
        single.update(wl.LR)
        ddp_orc.allreduce_and_update(wl.LR)
        for r in range(R):
            assert rel_l2(f64(w[r]), single.theta) <= TOL
            assert rel_l2(f64(w[r]), ddp_orc.theta) <= TOL
            assert rel_l2(f64(m[r]), wl.BETA1 * single.m) <= TOL
            assert rel_l2(f64(v[r]), R * wl.BETA2 * single.v) <= TOL
        assert all(torch.equal(w[0], w[r]) for r in range(1, R))
    for o in opts:
        o.close()


def test_world_size_one_is_plain_apply():
    n = 4099
    g = wl.normal((n,), 1e-2, torch.float32, 3).cuda()
    res = []
    for ddp in (False, True):
        opt = adama.AdamA()
        opt.begin_minibatch(1)
        w = wl.normal((n,), 0.02, torch.float32, 4).cuda()
        m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        opt.fold(g, m, v)
        if ddp:
            opt.apply_allreduced(w, m, v, wl.LR, 1)
        else:
            opt.apply(w, m, v, wl.LR)
        res.append((w.clone(), m.clone(), v.clone()))
        opt.close()
    assert all(torch.equal(a, b) for a, b in zip(*res))


def test_world_size_must_be_positive():
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    x = torch.zeros(8, device="cuda")
    with pytest.raises(adama.AdamAError) as e:
        opt.apply_allreduced(x, x.clone(), x.clone(), 1e-3, 0)
    assert e.value.status == adama.Status.ERR_INVALID_ARG
    opt.close()


@pytest.mark.parametrize("R,N", [(2, 2), (4, 1)])
def test_sharded_apply_equals_single_device(R, N):
    """adama_apply_sharded with R ranks emulated in turn: full-size local accumulators, summed
    shard by shard (standing in for reduce-scatter), owner-only update, foreign shards zeroed,
    weights gathered."""
    n, steps = 8 * 4099, 3
    k = n // R
    w0 = wl.normal((n,), 0.02, torch.float32, 11)
    single = AdamAOracle(f64(w0))
    opts = [adama.AdamA() for _ in range(R)]
    w = w0.cuda()                                     # identical on all ranks after the gather
    m = [torch.zeros(n, device="cuda") for _ in range(R)]
    v = [torch.zeros(n, device="cuda") for _ in range(R)]
    for step in range(steps):
        single.begin_minibatch(N * R)
        for r in range(R):
            opts[r].begin_minibatch(N)
            for i in range(N):
                g = wl.normal((n,), 1e-2, torch.float32, 2000 * step + 10 * r + i + 3)
                opts[r].fold(g.cuda(), m[r], v[r])
                single.fold(f64(g))
        m_sum = torch.stack(m).sum(0)
        v_sum = torch.stack(v).sum(0)
        for r in range(R):
            lo, hi = r * k, (r + 1) * k
            m[r].zero_()
            v[r].zero_()
            m[r][lo:hi] = m_sum[lo:hi]
            v[r][lo:hi] = v_sum[lo:hi]
            opts[r].apply_sharded(w[lo:hi], m[r][lo:hi], v[r][lo:hi], wl.LR, R)
        single.update(wl.LR)
        assert rel_l2(f64(w), single.theta) <= TOL
        for r in range(R):
            lo, hi = r * k, (r + 1) * k
            assert rel_l2(f64(m[r][lo:hi]), R * wl.BETA1 * single.m[lo:hi]) <= TOL
            assert rel_l2(f64(v[r][lo:hi]), R * R * wl.BETA2 * single.v[lo:hi]) <= TOL
    for o in opts:
        o.close()


@pytest.mark.parametrize("R,N", [(2, 2), (4, 1), (8, 1)])
def test_fused_peer_exchange_apply_equals_single_device(R, N):
    """adama_apply_sharded_peers: reduce-scatter + update + all-gather in one kernel over
    peer-mapped buffers.  The R ranks' buffers all live on this one GPU and the R launches run
    one after the other (the kernel never waits for a peer, so this is a faithful emulation):
    every rank must end with the single-device weights for N*R micro-batches, keep the
    un-normalised sums for its own shard only, and hold zeros elsewhere."""
    n, steps = 4 * R * 1031, 3
    k = n // R
    w0 = wl.normal((n,), 0.02, torch.float32, 21)
    single = AdamAOracle(f64(w0))
    opts = [adama.AdamA() for _ in range(R)]
    w = [w0.cuda() for _ in range(R)]
    m = [torch.zeros(n, device="cuda") for _ in range(R)]
    v = [torch.zeros(n, device="cuda") for _ in range(R)]
    ptrs = lambda ts: [t.data_ptr() for t in ts]
    for step in range(steps):
        single.begin_minibatch(N * R)
        for r in range(R):
            opts[r].begin_minibatch(N)
            for i in range(N):
                g = wl.normal((n,), 1e-2, torch.float32, 3000 * step + 10 * r + i + 5)
                opts[r].fold(g.cuda(), m[r], v[r])
                single.fold(f64(g))
        torch.cuda.synchronize()                       # "all ranks have finished folding"
        for r in range(R):
            opts[r].apply_sharded_peers(ptrs(w), ptrs(m), ptrs(v), r, n, wl.LR)
        torch.cuda.synchronize()                       # "all exchanges have finished"
        single.update(wl.LR)
        for r in range(R):
            lo, hi = r * k, (r + 1) * k
            assert rel_l2(f64(w[r]), single.theta) <= TOL
            assert torch.equal(w[r], w[0])
            assert rel_l2(f64(m[r][lo:hi]), R * wl.BETA1 * single.m[lo:hi]) <= TOL
            assert rel_l2(f64(v[r][lo:hi]), R * R * wl.BETA2 * single.v[lo:hi]) <= TOL
            mask = torch.ones(n, dtype=torch.bool, device="cuda")
            mask[lo:hi] = False
            assert not bool(m[r][mask].any()) and not bool(v[r][mask].any())
    with pytest.raises(adama.AdamAError) as e:
        opts[0].apply_sharded_peers(ptrs(w), ptrs(m), ptrs(v), 0, n - 4, wl.LR)
    assert e.value.status == adama.Status.ERR_UNSUPPORTED
    for o in opts:
        o.close()
