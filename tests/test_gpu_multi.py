"""Multi-tensor fold / apply: many small tensors in one launch must give, bit for bit, what
one adama_fold / adama_apply call per tensor gives, and match the fp64 oracle."""
import numpy as np
import pytest
import torch

import adama_workloads as wl
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from parity import f64, rel_l2

pytestmark = pytest.mark.gpu
TOL = 1e-6


def _sizes(count, seed):
    rng = np.random.default_rng(seed)
    sizes = [int(x) for x in rng.integers(1, 20_000, count)]
    sizes[3], sizes[7], sizes[11] = 1, 4096, 4097
    sizes[5] = (1 << 22) + 3            # long enough for the single-tensor kernel
    return sizes


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_multi_equals_per_tensor_and_oracle(gdtype):
    count, N = 150, 2                   # 150 tensors: three launches of <= 64
    sizes = _sizes(count, 1)

    def carve(offset_by):               # views with mixed alignment (offset 0..3 elements)
        return [torch.zeros(n + 8, device="cuda")[(i * offset_by) % 4:(i * offset_by) % 4 + n]
                for i, n in enumerate(sizes)]

    w_a, m_a, v_a = carve(1), carve(2), carve(3)
    w0 = [wl.normal((n,), 0.02, torch.float32, 100 + i) for i, n in enumerate(sizes)]
    for wa, x in zip(w_a, w0):
        wa.copy_(x)
    w_b = [x.clone() for x in w_a]
    m_b = [x.clone() for x in m_a]
    v_b = [x.clone() for x in v_a]
    orcs = [AdamAOracle(f64(x)) for x in w0]
    multi, single = adama.AdamA(), adama.AdamA()
    for step in range(2):
        multi.begin_minibatch(N)
        single.begin_minibatch(N)
        for o in orcs:
            o.begin_minibatch(N)
        for i in range(N):
            grads = [wl.normal((n,), 1e-2, gdtype, 7000 + 1000 * step + 200 * i + k).cuda()
                     for k, n in enumerate(sizes)]
            multi.fold_multi(grads, m_a, v_a)
            for g, m, v, o in zip(grads, m_b, v_b, orcs):
                single.fold(g, m, v)
                o.fold(f64(g))
        multi.apply_multi(w_a, m_a, v_a, wl.LR)
        for w, m, v, o in zip(w_b, m_b, v_b, orcs):
            single.apply(w, m, v, wl.LR)
            o.update(wl.LR)
        for k in range(count):
            assert torch.equal(w_a[k], w_b[k]) and torch.equal(m_a[k], m_b[k]) and torch.equal(v_a[k], v_b[k]), k
        for k in (0, 3, 5, 7, 11, 64, 149):
            if sizes[k] > 8:
                assert rel_l2(f64(w_a[k]), orcs[k].theta) <= TOL
                assert rel_l2(f64(v_a[k]), wl.BETA2 * orcs[k].v) <= TOL
    # 149 small tensors in 3 grouped launches + 1 long tensor alone, per fold / apply
    assert multi.launch_count == 2 * (N + 1) * 4
    assert single.launch_count == 2 * (N + 1) * count
    multi.close()
    single.close()


def test_multi_empty_and_errors():
    opt = adama.AdamA()
    opt.fold_multi([], [], [])          # nothing to do, no state needed
    x = torch.zeros(8, device="cuda")
    with pytest.raises(adama.AdamAError) as e:
        opt.fold_multi([x], [x.clone()], [x.clone()])
    assert e.value.status == adama.Status.ERR_BAD_STATE
    opt.begin_minibatch(1)
    opt.fold_multi([x, torch.zeros(0, device="cuda")], [x.clone(), torch.zeros(0, device="cuda")],
                   [x.clone(), torch.zeros(0, device="cuda")])
    assert opt.launch_count == 1
    opt.close()
