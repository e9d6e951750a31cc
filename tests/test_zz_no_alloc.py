"""The allocation-free entry point against the regular one and against the oracle.

Some users of this library cannot take device memory from CUDA while they call it: their
GPU memory belongs to a framework's pool, or they run at a point where the allocator must
not be touched.  adama_linear_wgrad_fold_noalloc serves them: no context, and the
kernel's status block is a fixed array inside the library.  It must give what
adama_linear_wgrad_fold gives (the same kernel on the same inputs: bit for bit), on a first
call and again on a second call that finds the first call's leftovers in the shared block,
and it must leave the device's free memory where it found it.  This file is collected last
on purpose.
"""
import subprocess
import sys
import textwrap
from pathlib import Path

import pytest
import torch

import adama_workloads as wl
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from parity import assert_close, f64

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-3   # the tolerance of the bf16-input fused path in the other tests
ROOT = Path(__file__).resolve().parent.parent


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


def test_noalloc_entry_point_matches_regular_entry_point_twice():
    T, d_in, d_out, N = 320, 200, 328, 4           # ragged tiles, 5 k-blocks
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS)
    opt.begin_minibatch(N)
    orc = AdamAOracle(f64(torch.zeros(d_in, d_out)), wl.BETA1, wl.BETA2, wl.EPS)
    orc.begin_minibatch(N)
    m_ref = torch.zeros(d_in, d_out, device="cuda")
    v_ref = torch.zeros(d_in, d_out, device="cuda")
    m = torch.zeros(d_in, d_out, device="cuda")
    v = torch.zeros(d_in, d_out, device="cuda")
    status = torch.full((4,), 77, dtype=torch.int32).pin_memory()
    for call in range(2):                          # two calls in a row share the static block
        Xh = wl.normal((T, d_in), 1.0, torch.bfloat16, 600 + call)
        dYh = wl.normal((T, d_out), 1e-2, torch.bfloat16, 700 + call)
        X, dY = Xh.cuda(), dYh.cuda()
        opt.linear_wgrad_fold(X, dY, m_ref, v_ref)
        orc.fold_linear(f64(Xh), f64(dYh))
        torch.cuda.synchronize()
        # what the driver itself reports as free: sees a cudaMalloc made by anyone in the process
        free_before, _ = torch.cuda.mem_get_info()
        adama.linear_wgrad_fold_noalloc(X, dY, m, v, N, wl.BETA1, wl.BETA2, status_out=status)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call == 1:   # the first call on a device may load the kernel image; later ones take nothing
            assert free_after == free_before
        assert status.tolist() == [0, 0, 0, 0]
        assert _rel(m, m_ref) <= TOL_BF16 and _rel(v, v_ref) <= TOL_BF16
        assert torch.equal(m, m_ref) and torch.equal(v, v_ref)      # same kernel, same inputs
        assert_close(f64(m), orc.m, TOL_BF16, f"m after call {call}")  # and the oracle's fold
        assert_close(f64(v), orc.v, TOL_BF16, f"v after call {call}")
        status.fill_(77)
    opt.sync_status()
    opt.close()


_FIRST_USE = textwrap.dedent("""
    import sys
    sys.path.insert(0, {root!r})
    import torch
    import adama_workloads as wl
    import paper_2305_19982_b200 as adama
    T, d_in, d_out, N = 320, 200, 328, 4
    X = [wl.normal((T, d_in), 1.0, torch.bfloat16, 600 + c).cuda() for c in range(2)]
    dY = [wl.normal((T, d_out), 1e-2, torch.bfloat16, 700 + c).cuda() for c in range(2)]
    m = torch.zeros(d_in, d_out, device="cuda"); v = torch.zeros_like(m)
    m_ref = torch.zeros_like(m); v_ref = torch.zeros_like(m)
    status = torch.full((4,), 77, dtype=torch.int32).pin_memory()
    torch.cuda.synchronize()
    # no context of the library exists yet: this call does the per-device set-up itself
    adama.linear_wgrad_fold_noalloc(X[0], dY[0], m, v, N, wl.BETA1, wl.BETA2, status_out=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 0, 0, 0], status.tolist()
    free_before, _ = torch.cuda.mem_get_info()
    adama.linear_wgrad_fold_noalloc(X[1], dY[1], m, v, N, wl.BETA1, wl.BETA2, status_out=status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert status.tolist() == [0, 0, 0, 0], status.tolist()
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS)      # only now: the regular entry point
    opt.begin_minibatch(N)
    for c in range(2):
        opt.linear_wgrad_fold(X[c], dY[c], m_ref, v_ref)
    opt.sync_status()
    assert torch.equal(m, m_ref) and torch.equal(v, v_ref)
    assert float(v.max()) > 0
    print("first-use ok")
""")


def test_noalloc_entry_point_as_the_first_use_of_the_library_in_a_process():
    """A fresh process that never created a context: the entry point's own first call sets the
    device up (scratch address, kernel attributes), its second call leaves the device's free
    memory untouched, and both give what the regular entry point gives afterwards."""
    res = subprocess.run([sys.executable, "-c", _FIRST_USE.format(root=str(ROOT))],
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "first-use ok" in res.stdout


def test_noalloc_entry_point_rejects_bad_arguments_with_a_message():
    X = torch.zeros(64, 72, dtype=torch.bfloat16, device="cuda")
    dY = torch.zeros(64, 80, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(72, 80, device="cuda")
    with pytest.raises(adama.AdamAError) as e:
        adama.linear_wgrad_fold_noalloc(X, dY, m, m.clone(), 0)
    assert e.value.status == adama.Status.ERR_INVALID_ARG and "n_micro" in str(e.value)
    Xo = torch.zeros(64 * 72 + 8, dtype=torch.bfloat16, device="cuda")[1:1 + 64 * 72].view(64, 72)
    with pytest.raises(adama.AdamAError) as e:
        adama.linear_wgrad_fold_noalloc(Xo, dY, m, m.clone(), 1)
    assert e.value.status == adama.Status.ERR_MISALIGNED and "aligned" in str(e.value)
