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
from parity import assert_close, f64

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-3


@pytest.mark.parametrize("biases,per_launch", [(False, 1), (True, 1), (False, 2), (True, 3)])
def test_small_stack_full_parity(biases, per_launch):
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
        stack.fold_micro_batches(opt, N, inputs, layers_per_launch=per_launch)
        opt.sync_status()
        for j in range(len(layers)):   # m_t, v_t after the last fold of the mini-batch
            assert_close(f64(stack.view(stack.m, j)), orcs[j].m, TOL_BF16, f"m_t layer {j}")
            assert_close(f64(stack.view(stack.v, j)), orcs[j].v, TOL_BF16, f"v_t layer {j}")
        stack.apply(opt, wl.LR)
        opt.sync_status()
        for j in range(len(layers)):
            if biases:
                borcs[j].update(wl.LR)
                assert_close(f64(stack.bias_view(stack.w, j)), borcs[j].theta, TOL_BF16, "bias w")
                assert_close(f64(stack.bias_view(stack.m, j)), wl.BETA1 * borcs[j].m, TOL_BF16, "bias m")
                assert_close(f64(stack.bias_view(stack.v, j)), wl.BETA2 * borcs[j].v, TOL_BF16, "bias v")
            orcs[j].update(wl.LR)
            assert_close(f64(stack.view(stack.w, j)), orcs[j].theta, TOL_BF16, f"w layer {j}")
            assert_close(f64(stack.view(stack.m, j)), wl.BETA1 * orcs[j].m, TOL_BF16, f"m layer {j}")
            assert_close(f64(stack.view(stack.v, j)), wl.BETA2 * orcs[j].v, TOL_BF16, f"v layer {j}")
    # layers are visited from the last to the first inside every micro-batch
    assert order[:3] == [(0, 2), (0, 1), (0, 0)]
    opt.close()


def _sampled_stack(stack: LinearStack, tokens: int, n_micro: int, steps: int, config: int,
                   per_layer: int, layers_per_launch: int = 1):
    """`steps` mini-batches of `n_micro` micro-batches over every layer of the stack, in the
    launch configuration the benchmark times.  Per layer a fixed sample of entries (random ones
    plus the first and the last row / column) is followed through the whole recurrence by the
    oracle: each G entry is a `tokens`-term dot product of one column of X and one of dY.
    Compared: m_t, v_t after the last fold of every mini-batch, then w, beta1*m_t, beta2*v_t
    after every apply."""
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
    ar = np.arange(S)
    for step in range(steps):
        orc.begin_minibatch(n_micro)

        def inputs(i, j, spec):
            X = wl.normal((tokens, spec.d_in), 1.0, torch.bfloat16, wl.seed_for(config, step, i, j),
                          device="cuda")
            dY = wl.normal((tokens, spec.d_out), 1e-2, torch.bfloat16,
                           wl.seed_for(config, step, i, j) + 50, device="cuda")
            p, q = samples[j]
            G = oracle.linear_wgrad_entries(f64(X[:, p]), f64(dY[:, q]), ar, ar)
            orc.fold(G, lo=j * S)
            return X, dY

        stack.fold_micro_batches(opt, n_micro, inputs, layers_per_launch)
        opt.sync_status()
        assert_close(f64(stack.m[flat]), orc.m, TOL_BF16, f"m_t step {step}")
        assert_close(f64(stack.v[flat]), orc.v, TOL_BF16, f"v_t step {step}")
        stack.apply(opt, wl.LR)
        opt.sync_status()
        orc.update(wl.LR)
        assert_close(f64(stack.w[flat]), orc.theta, TOL_BF16, f"w step {step}")
        assert_close(f64(stack.m[flat]), wl.BETA1 * orc.m, TOL_BF16, f"beta1*m step {step}")
        assert_close(f64(stack.v[flat]), wl.BETA2 * orc.v, TOL_BF16, f"beta2*v step {step}")
    assert bool((stack.v >= 0).all()) and bool(torch.isfinite(stack.w).all())
    assert opt.step == steps and opt.n_micro == n_micro
    opt.close()


def test_gpt2xl_full_stack_sampled():
    """All 48 blocks x 4 linears (1.475 B parameters, 17.7 GB of state), 4096 tokens per
    micro-batch, N = 8 micro-batches as the workload states, 2 mini-batches (the second starts
    from the decayed state), 24 sampled entries per layer."""
    stack = gpt2xl_stack(wl.CONFIG4_BLOCKS)
    assert stack.n_params == 48 * (1600 * 4800 + 1600 * 1600 + 2 * 1600 * 6400)
    _sampled_stack(stack, wl.CONFIG4_TOKENS, wl.CONFIG4_N_MICRO, 2, 4, 24)


def test_gpt2xl_full_stack_one_launch_per_block_sampled():
    """The same stack with the four linears of a block folded by one grouped launch
    (adama_linear_wgrad_fold_multi), N = 8, 2 mini-batches."""
    stack = gpt2xl_stack(wl.CONFIG4_BLOCKS)
    _sampled_stack(stack, wl.CONFIG4_TOKENS, wl.CONFIG4_N_MICRO, 2, 4, 24, layers_per_launch=4)


def test_llama7b_two_blocks_sampled():
    stack = llama7b_stack(2)
    _sampled_stack(stack, wl.CONFIG5_TOKENS, 2, 1, 5, 40)


def test_llama7b_full_stack_sampled():
    """All 32 blocks x 7 linears (6.476 B parameters, 77.7 GB of fp32 state), 4096 tokens,
    N = 16 micro-batches and 2 mini-batches as the workload states, 8 sampled entries per
    layer, in the launch configuration the benchmark times."""
    free, _ = torch.cuda.mem_get_info()
    if free < 100 * (1 << 30):
        pytest.skip("needs ~90 GB of free device memory")
    torch.cuda.empty_cache()
    stack = llama7b_stack(wl.CONFIG5_BLOCKS)
    assert stack.n_params == 32 * (4 * 4096 * 4096 + 3 * 4096 * 11008)
    _sampled_stack(stack, wl.CONFIG5_TOKENS, wl.CONFIG5_N_MICRO, wl.CONFIG5_STEPS, 5, 8)
    del stack
    torch.cuda.empty_cache()
