"""Call-order, argument and alignment errors of the C ABI on a GPU machine (all rejected on
the host; nothing here launches a faulty kernel)."""
import pytest
import torch

import adama_workloads as wl
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


def test_timeout_report_path_without_a_waiting_kernel():
    """The host side of the bounded-wait design: a status block that says "a wait expired" is
    reported once as ERR_TIMEOUT with the wait and tile in the message, cleared, and the
    context keeps working.  The record is planted by the test hook; no kernel is made to wait."""
    import adama_workloads as wl
    opt = adama.AdamA()
    opt.sync_status()                                   # clean
    opt.debug_set_status(1, wait=3, tile=17)
    with pytest.raises(adama.AdamAError) as e:
        opt.sync_status()
    assert e.value.status == Status.ERR_TIMEOUT and "wait 3" in str(e.value) and "tile 17" in str(e.value)
    opt.sync_status()                                   # cleared by the report
    opt.begin_minibatch(1)
    X = wl.small_integers((64, 128), 2, torch.bfloat16, 1).cuda()
    dY = wl.small_integers((64, 256), 2, torch.bfloat16, 2).cuda()
    m = torch.zeros(128, 256, device="cuda")
    v = torch.zeros(128, 256, device="cuda")
    opt.linear_wgrad_fold(X, dY, m, v)                  # the context is still usable
    opt.sync_status()
    assert torch.allclose(m, (1 - 0.9) * (X.float().t() @ dY.float()), rtol=1e-6)
    opt.close()


@pytest.mark.parametrize("tokens,epilogue", [(256, 0), (2304, 0), (256, 1), (2304, 2)])
def test_device_side_wait_runs_out_and_the_kernel_returns(tokens, epilogue):
    """A wait inside the fused kernel that really expires, in the non-hanging form: the test
    entry launches the normal kernel with a 1 ms limit on every wait and a producer that
    never loads the last stage of the last tile.  The kernel must come back by itself (the
    synchronise below returns), report a time-out with the wait and the tile, leave the
    other tiles folded and the withheld tile untouched, and the same context must then pass
    a normal call.  Both epilogue forms (256 tokens: staged, 2304: direct; and each forced the
    other way)."""
    import time
    import adama_workloads as wl
    d_in, d_out = 512, 768                      # 2 x 3 tiles; the withheld one is the last
    opt = adama.AdamA()
    opt.debug_set_wgrad_variant(epilogue=epilogue)
    opt.begin_minibatch(1)
    X = wl.small_integers((tokens, d_in), 2, torch.bfloat16, 1).cuda()
    dY = wl.small_integers((tokens, d_out), 2, torch.bfloat16, 2).cuda()
    m = torch.zeros(d_in, d_out, device="cuda")
    v = torch.zeros(d_in, d_out, device="cuda")
    t0 = time.perf_counter()
    opt.debug_wgrad_expire_wait(X, dY, m, v, wait_limit_ns=1_000_000)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0       # limits of 1 ms (+20 ms of draining), not 2 s
    with pytest.raises(adama.AdamAError) as e:
        opt.sync_status()
    assert e.value.status == Status.ERR_TIMEOUT
    assert "wait" in str(e.value) and "tile" in str(e.value)
    G = X.float().t() @ dY.float()              # small integers: exact in fp32
    want = (1 - 0.9) * G
    # the withheld work item is the launch's last: the bottom-right tile, or its right half
    # when the launch issues its tiles as column halves
    missing = (m == 0) & (G != 0)
    rows = missing.any(dim=1).nonzero().flatten()
    cols = missing.any(dim=0).nonzero().flatten()
    assert int(rows.min()) >= 256 and int(cols.min()) in (512, 640)
    done = torch.ones(d_in, d_out, dtype=torch.bool, device="cuda")
    done[256:, int(cols.min()):] = False
    assert torch.allclose(m[done], want[done], rtol=1e-6)
    assert bool((m[~done] == 0).all()) and bool((v[~done] == 0).all())
    opt.sync_status()                           # cleared by the report
    m.zero_()
    v.zero_()
    opt.linear_wgrad_fold(X, dY, m, v)          # the context (and the GPU) are still usable
    opt.sync_status()
    assert torch.allclose(m, want, rtol=1e-6)
    assert torch.allclose(v, (1 - 0.999) * G * G, rtol=1e-6)
    opt.close()


def test_expire_wait_entry_rejects_limits_out_of_range():
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    X = torch.zeros(64, 128, dtype=torch.bfloat16, device="cuda")
    dY = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(128, 256, device="cuda")
    for limit in (0, 999, 2_000_000_000):
        with pytest.raises(adama.AdamAError) as e:
            opt.debug_wgrad_expire_wait(X, dY, m, m.clone(), wait_limit_ns=limit)
        assert e.value.status == Status.ERR_INVALID_ARG
    assert opt.launch_count == 0
    opt.close()


def test_setup_state_after_a_launch_on_device_0():
    """Kernel attributes are remembered per device: after a fused launch on device 0 the
    table says so for device 0 and for no other device."""
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    X = torch.zeros(64, 128, dtype=torch.bfloat16, device="cuda")
    dY = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(128, 256, device="cuda")
    opt.linear_wgrad_fold(X, dY, m, m.clone())
    opt.sync_status()
    assert adama.debug_setup_state(0) == 3
    assert adama.debug_setup_state(1) & 2 == 0 and adama.debug_setup_state(64) & 2 == 0
    opt.close()


def test_checkpoint_resume_is_bit_identical():
    """State = w, m, v (stored decayed after apply) + the step counter: a new context restored
    with set_step continues exactly as the uninterrupted run."""
    import adama_workloads as wl
    n, N = 50_000, 2

    def run(total_steps, resume_after=None):
        opt = adama.AdamA()
        w = wl.normal((n,), 0.02, torch.float32, 5).cuda()
        m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        for step in range(total_steps):
            if resume_after is not None and step == resume_after:
                saved = (w.clone(), m.clone(), v.clone(), opt.step)
                opt.close()
                opt = adama.AdamA()                     # "new process": fresh context
                w, m, v = saved[0], saved[1], saved[2]
                opt.set_step(saved[3])
            opt.begin_minibatch(N)
            for i in range(N):
                opt.fold(wl.normal((n,), 1e-2, torch.bfloat16, 100 * step + i).cuda(), m, v)
            opt.apply(w, m, v, 1e-3)
        opt.close()
        return w, m, v

    a = run(4)
    b = run(4, resume_after=2)
    assert all(torch.equal(x, y) for x, y in zip(a, b))


def test_async_copyback_gives_the_same_weights_and_is_ordered_before_the_next_update():
    """ADAMA_ASYNC_COPYBACK: the device-to-host copy of apply_to_host runs on the context's own
    stream.  Three mini-batches without any host synchronisation in between: every copy-back
    must hold the weights of ITS step (the next update has to wait for the copy that is still
    reading w), and the final state equals the stream-ordered form bit for bit."""
    n = 8_000_003            # 32 MB: long enough copies for an ordering mistake to show
    g = [wl.normal((n,), 1e-3, torch.bfloat16, 70 + i).cuda() for i in range(2)]
    res = {}
    for mode in (False, True):
        opt = adama.AdamA(async_copyback=mode)
        w = wl.normal((n,), 0.02, torch.float32, 71).cuda()
        m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        hosts = [torch.zeros(n, dtype=torch.float32).pin_memory() for _ in range(3)]
        snaps = []
        for step in range(3):
            opt.begin_minibatch(2)
            for i in range(2):
                opt.fold(g[i], m, v)
            opt.apply_to_host(w, m, v, wl.LR, hosts[step])
            if not mode:
                snaps.append(w.clone())     # stream-ordered: what w holds after this step
        opt.sync_status()
        torch.cuda.synchronize()
        res[mode] = (w.cpu(), [h.clone() for h in hosts], [s.cpu() for s in snaps])
        opt.close()
    w_sync, hosts_sync, snaps = res[False]
    w_async, hosts_async, _ = res[True]
    assert torch.equal(w_sync, w_async)
    for step in range(3):
        assert torch.equal(hosts_sync[step], snaps[step])
        assert torch.equal(hosts_async[step], snaps[step])
