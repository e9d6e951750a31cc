"""The allocation-free entry point against the regular one.

Some users of this library cannot take device memory from CUDA while they call it: their
GPU memory belongs to a framework's pool, or they run at a point where the allocator must
not be touched.  adama_linear_wgrad_fold_noalloc serves them: no context, and the
kernel's status block is a fixed array inside the library.  It must give what
adama_linear_wgrad_fold gives, on a first call and again on a second call that finds the
first call's leftovers in the shared block.  This file is collected last on purpose.
"""
import pytest
import torch

import adama_workloads as wl
import paper_2305_19982_b200 as adama

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-3   # the tolerance of the bf16-input fused path in the other tests


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


def test_noalloc_entry_point_matches_regular_entry_point_twice():
    T, d_in, d_out, N = 320, 200, 328, 4           # ragged tiles, 5 k-blocks
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS)
    opt.begin_minibatch(N)
    m_ref = torch.zeros(d_in, d_out, device="cuda")
    v_ref = torch.zeros(d_in, d_out, device="cuda")
    m = torch.zeros(d_in, d_out, device="cuda")
    v = torch.zeros(d_in, d_out, device="cuda")
    status = torch.full((4,), 77, dtype=torch.int32).pin_memory()
    for call in range(2):                          # two calls in a row share the static block
        X = wl.normal((T, d_in), 1.0, torch.bfloat16, 600 + call).cuda()
        dY = wl.normal((T, d_out), 1e-2, torch.bfloat16, 700 + call).cuda()
        opt.linear_wgrad_fold(X, dY, m_ref, v_ref)
        before = torch.cuda.memory_allocated()
        adama.linear_wgrad_fold_noalloc(X, dY, m, v, N, wl.BETA1, wl.BETA2, status_out=status)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert status.tolist() == [0, 0, 0, 0]
        assert _rel(m, m_ref) <= TOL_BF16
        assert _rel(v, v_ref) <= TOL_BF16
        status.fill_(77)
    opt.sync_status()
    opt.close()


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
