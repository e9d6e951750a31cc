"""Layer stacks (the GPT-2-XL- and Llama-7B-shaped workloads) through the stack driver:
back-to-front layer order, immediate release of (X, dY), one apply per mini-batch.  Large
stacks are checked on sampled entries: for a sample (p, q) of a layer the oracle needs
only column p of X and column q of dY, which are gathered on the GPU and widened on the
host (data movement only)."""
import numpy as np
import pytest
import torch

import adama_workloads as wl
import oracle
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from paper_2305_19982_b200.stack import LayerSpec, LinearStack, gpt2xl_stack, llama7b_stack
from parity import f64, rel_l2

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-3


@pytest.mark.parametrize("biases,materialise", [(False, "none"), (True, "none"), (True, "layer")])
def test_small_stack_full_parity(biases, materialise):
    layers = [LayerSpec("a", 200, 328), LayerSpec("b", 328, 136), LayerSpec("c", 136, 8)]
    T, N, steps = 192, 2, 2
    stack = LinearStack(layers, biases=biases)
    stack.w.normal_(0, 0.02, generator=torch.Generator(device="cuda").manual_seed(5))
    orcs = [AdamAOracle(f64(stack.view(stack.w, j))) for j in range(len(layers))]
    borcs = [AdamAOracle(f64(stack.bias_view(stack.w, j))) for j in range(len(layers))] if biases else []
    opt = adama.AdamA()
    order = []
    for step in range(steps):
        def inputs(i, j, spec):
            order.append((i, j))
            X = wl.normal((T, spec.d_in), 1.0, torch.bfloat16, wl.seed_for(4, step, i, j))
            dY = wl.normal((T, spec.d_out), 1e-2, torch.bfloat16, wl.seed_for(4, step, i, j) + 50)
            if i == 0:
                orcs[j].begin_minibatch(N)
                if biases:
                    borcs[j].begin_minibatch(N)
            orcs[j].fold_linear(f64(X), f64(dY))
            if biases:      # bias gradient = column sums of dY (naive loop in the oracle)
                borcs[j].fold(oracle.linear_wgrad(np.ones((T, 1)), f64(dY))[0])
            return X.cuda(), dY.cuda()
        stack.minibatch(opt, N, wl.LR, inputs, materialise=materialise)
        opt.sync_status()
        for j in range(len(layers)):
            if biases:
                borcs[j].update(wl.LR)
                assert rel_l2(f64(stack.bias_view(stack.w, j)), borcs[j].theta) <= TOL_BF16
                assert rel_l2(f64(stack.bias_view(stack.m, j)), wl.BETA1 * borcs[j].m) <= TOL_BF16
                assert rel_l2(f64(stack.bias_view(stack.v, j)), wl.BETA2 * borcs[j].v) <= TOL_BF16
            orcs[j].update(wl.LR)
            assert rel_l2(f64(stack.view(stack.w, j)), orcs[j].theta) <= TOL_BF16
            assert rel_l2(f64(stack.view(stack.m, j)), wl.BETA1 * orcs[j].m) <= TOL_BF16
            assert rel_l2(f64(stack.view(stack.v, j)), wl.BETA2 * orcs[j].v) <= TOL_BF16
    # layers are visited from the last to the first inside every micro-batch
    assert order[:3] == [(0, 2), (0, 1), (0, 0)]
    opt.close()


def _sampled_stack(stack: LinearStack, tokens: int, n_micro: int, config: int, per_layer: int):
    rng = np.random.default_rng(config)
    gen = torch.Generator(device="cuda").manual_seed(config)
    stack.w.normal_(0, 0.02, generator=gen)
    samples, flat_idx = [], []
    for j, L in enumerate(stack.layers):
        p = np.concatenate([rng.integers(0, L.d_in, per_layer), [0, L.d_in - 1]])
        q = np.concatenate([rng.integers(0, L.d_out, per_layer), [L.d_out - 1, L.d_out - 1]])
        samples.append((torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda()))
        flat_idx.append(stack.offsets[j] + p * L.d_out + q)
    flat = torch.from_numpy(np.concatenate(flat_idx)).cuda()
    S = per_layer + 2
    orc = AdamAOracle(f64(stack.w[flat]))
    opt = adama.AdamA()
    orc.begin_minibatch(n_micro)
    ar = np.arange(S)

    def inputs(i, j, spec):
        X = wl.normal((tokens, spec.d_in), 1.0, torch.bfloat16, wl.seed_for(config, 0, i, j),
                      device="cuda")
        dY = wl.normal((tokens, spec.d_out), 1e-2, torch.bfloat16,
                       wl.seed_for(config, 0, i, j) + 50, device="cuda")
        p, q = samples[j]
        G = oracle.linear_wgrad_entries(f64(X[:, p]), f64(dY[:, q]), ar, ar)
        orc.fold(G, lo=j * S)
        return X, dY

    stack.minibatch(opt, n_micro, wl.LR, inputs)
    opt.sync_status()
    orc.update(wl.LR)
    assert rel_l2(f64(stack.w[flat]), orc.theta) <= TOL_BF16
    assert rel_l2(f64(stack.m[flat]), wl.BETA1 * orc.m) <= TOL_BF16
    assert rel_l2(f64(stack.v[flat]), wl.BETA2 * orc.v) <= TOL_BF16
    assert bool((stack.v >= 0).all()) and bool(torch.isfinite(stack.w).all())
    opt.close()


def test_gpt2xl_full_stack_sampled():
    """All 48 blocks x 4 linears (1.475 B parameters, 17.7 GB of state), 4096 tokens,
    2 micro-batches, 40 sampled entries per layer."""
    stack = gpt2xl_stack(wl.CONFIG4_BLOCKS)
    assert stack.n_params == 48 * (1600 * 4800 + 1600 * 1600 + 2 * 1600 * 6400)
    _sampled_stack(stack, wl.CONFIG4_TOKENS, 2, 4, 40)


def test_llama7b_two_blocks_sampled():
    stack = llama7b_stack(2)
    _sampled_stack(stack, wl.CONFIG5_TOKENS, 1, 5, 40)


def test_llama7b_full_stack_sampled():
    """All 32 blocks x 7 linears (6.476 B parameters, 77.7 GB of fp32 state), 4096 tokens, one
    micro-batch, 10 sampled entries per layer, in the launch configuration the bench times."""
    free, _ = torch.cuda.mem_get_info()
    if free < 100 * (1 << 30):
        pytest.skip("needs ~90 GB of free device memory")
    torch.cuda.empty_cache()
    stack = llama7b_stack(wl.CONFIG5_BLOCKS)
    assert stack.n_params == 32 * (4 * 4096 * 4096 + 3 * 4096 * 11008)
    _sampled_stack(stack, wl.CONFIG5_TOKENS, 1, 5, 10)
    del stack
    torch.cuda.empty_cache()
