"""GPU parity of the fused weight-gradient + fold kernel against the fp64 oracle.

The oracle forms G = X^T.dY by the naive triple loop (or entry by entry for sampled
checks) and folds it as Algorithm 2 states.  Tolerance for the bf16-input path: relative
L2 error <= 2e-3 on m, v and w; with small-integer inputs the fp32 accumulation is exact
and the fp32 fold tolerance (1e-6) applies.
"""
import numpy as np
import pytest
import torch

import adama_workloads as wl
import oracle
import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from parity import SENTINEL, assert_close, f64

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-3
TOL_EXACT = 1e-6


def _draw(T, d_in, d_out, seed, integer=False):
    if integer:
        X = wl.small_integers((T, d_in), 4, torch.bfloat16, seed)
        dY = wl.small_integers((T, d_out), 4, torch.bfloat16, seed + 1)
    else:
        X = wl.normal((T, d_in), 1.0, torch.bfloat16, seed)
        dY = wl.normal((T, d_out), 1e-2, torch.bfloat16, seed + 1)
    return X, dY


def _full_parity(T, d_in, d_out, n_micro=2, steps=1, integer=False, pad=0, tol=None, variant=None):
    """Whole-matrix comparison; `pad` > 0 embeds X, dY, m, v in wider buffers (row pitch >
    row length) whose extra columns hold a sentinel that must survive.  `variant` pins the
    kernel instance (adama_debug_set_wgrad_variant) instead of the automatic choice."""
    tol = tol if tol is not None else (TOL_EXACT if integer else TOL_BF16)
    opt = adama.AdamA()
    if variant:
        opt.debug_set_wgrad_variant(**variant)
    w0 = wl.normal((d_in, d_out), 0.02, torch.float32, 77)
    orc = AdamAOracle(f64(w0))
    up = lambda x, k: (x + k - 1) // k * k
    ldmv = up(d_out + pad, 4) if pad else d_out
    ldx = up(d_in + pad, 8) if pad else d_in
    ldy = up(d_out + pad, 8) if pad else d_out
    mbuf = torch.full((d_in, ldmv), SENTINEL, device="cuda")
    vbuf = torch.full((d_in, ldmv), SENTINEL, device="cuda")
    m, v = mbuf[:, :d_out], vbuf[:, :d_out]
    m.zero_()
    v.zero_()
    w = w0.cuda()
    for step in range(steps):
        opt.begin_minibatch(n_micro)
        orc.begin_minibatch(n_micro)
        for i in range(n_micro):
            X, dY = _draw(T, d_in, d_out, 1000 * step + 10 * i + d_in, integer)
            Xb = torch.full((T, ldx), 7.0, dtype=torch.bfloat16, device="cuda")
            Yb = torch.full((T, ldy), 7.0, dtype=torch.bfloat16, device="cuda")
            Xb[:, :d_in] = X.cuda()
            Yb[:, :d_out] = dY.cuda()
            opt.linear_wgrad_fold(Xb[:, :d_in], Yb[:, :d_out], m, v)
            orc.fold_linear(f64(X), f64(dY))
        opt.sync_status()
        assert_close(f64(m), orc.m, tol, "m_t")
        assert_close(f64(v), orc.v, tol, "v_t")
        # apply works on contiguous buffers: use dense copies of the views
        mc, vc = m.contiguous(), v.contiguous()
        opt.apply(w, mc, vc, wl.LR)
        orc.update(wl.LR)
        m.copy_(mc)
        v.copy_(vc)
        assert_close(f64(w), orc.theta, tol, "w", elementwise=integer or n_micro > 1 or step > 0)
    if pad:
        assert bool((mbuf[:, d_out:] == SENTINEL).all()) and bool((vbuf[:, d_out:] == SENTINEL).all())
    opt.close()


def test_single_tile_integer_inputs_exact():
    _full_parity(64, 128, 256, integer=True)


def test_single_tile_partial_k():
    """tokens not a multiple of the 64-token stage nor of the 16-token MMA."""
    _full_parity(100, 128, 256, integer=True)
    _full_parity(7, 128, 256, integer=True)


def test_operand_roles_not_swapped():
    """d_in != d_out and one-hot activations: G is a scatter-add of dY rows, so a swapped or
    transposed operand cannot pass."""
    T, d_in, d_out = 96, 136, 264
    idx = torch.randint(0, d_in, (T,), generator=torch.Generator().manual_seed(3))
    X = torch.zeros(T, d_in, dtype=torch.bfloat16)
    X[torch.arange(T), idx] = 1.0
    dY = wl.small_integers((T, d_out), 8, torch.bfloat16, 5)
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    m = torch.zeros(d_in, d_out, device="cuda")
    v = torch.zeros(d_in, d_out, device="cuda")
    opt.linear_wgrad_fold(X.cuda(), dY.cuda(), m, v)
    opt.sync_status()
    G = np.zeros((d_in, d_out))
    for tau in range(T):
        G[idx[tau]] += f64(dY[tau])
    np.testing.assert_allclose(f64(m), (1 - wl.BETA1) * G, rtol=1e-6, atol=1e-12)
    np.testing.assert_allclose(f64(v), (1 - wl.BETA2) * G * G, rtol=1e-6, atol=1e-12)
    opt.close()


@pytest.mark.parametrize("T,d_in,d_out", [(100, 200, 328), (64, 8, 8), (130, 136, 520),
                                          (33, 1, 8), (64, 129, 263), (1, 3, 1)])
def test_ragged_shapes(T, d_in, d_out):
    """Shapes that are no multiple of the 128x256 tile, the 64-feature TMA box or the
    32x32 reduce box, in padded buffers (row pitch > row length) whose padding must stay
    untouched; integer inputs make the contraction exact."""
    _full_parity(T, d_in, d_out, integer=True, pad=5)


@pytest.mark.parametrize("T", [1100, 2048, 2100, 2500])
@pytest.mark.parametrize("d_in,d_out", [(200, 328), (129, 263), (136, 520), (300, 1000)])
def test_ragged_shapes_on_both_sides_of_the_short_call_limit(T, d_in, d_out):
    """Calls of up to 2048 tokens take the staged epilogue (accumulator -> shared memory ->
    streaming fold), longer ones the direct epilogue; the same ragged shapes and padded buffers
    on both sides of the limit.  Integer inputs: exact contraction, fp32 fold tolerance."""
    _full_parity(T, d_in, d_out, integer=True, pad=5)


def test_multi_tile_normal_inputs_two_steps():
    _full_parity(512, 384, 768, n_micro=2, steps=2)


def test_more_tiles_than_sms():
    """16 x 16 = 256 tiles on 148 SMs: persistent CTAs take a second tile and both
    accumulator stages, with phase wrap-around of the 4-stage ring (T=640: 10 k-blocks)."""
    _full_parity(640, 2048, 4096, n_micro=1, integer=False)


@pytest.mark.parametrize("T,d_in,d_out,why", [
    (640, 2048, 4096, "128 full tiles on 74 CTA pairs: second accumulator stage, ring phase wrap"),
    (128, 5120, 1024, "20 x 4 tiles: row index slowest, 6 left-over tiles issued as column halves"),
    (192, 1024, 5120, "4 x 20 tiles: column index slowest, same split tail"),
    (320, 1600, 1600, "layer of the GPT-2-XL-shaped stack: ragged last row and column tiles"),
    (2112, 1600, 4800, "the same beyond the short-call limit, several k-blocks per ring wrap"),
    (1100, 1664, 832, "short-call (staged) instance over more than one round of tiles"),
])
def test_whole_matrix_exact_beyond_one_round_of_tiles(T, d_in, d_out, why):
    """Shapes that need more than one tile per CTA group, a split tail or either tile
    numbering, with small-integer inputs (|x| <= 4: every product and every partial sum over
    at most 2112 tokens is below 2^24, hence exact in fp32).  The whole matrix is compared
    with the oracle at the fp32 fold tolerance, in the L2 norm and element by element, so one
    wrong chunk, tile or accumulator stage cannot hide."""
    _full_parity(T, d_in, d_out, n_micro=2, integer=True)


@pytest.mark.parametrize("variant", [
    dict(epilogue=1, epi_warps=4), dict(epilogue=1, epi_warps=8), dict(epilogue=2),
    dict(box_loads=1), dict(no_pdl=1), dict(epilogue=2, box_loads=1, no_pdl=1)],
    ids=lambda v: ",".join(f"{k}={x}" for k, x in v.items()))
@pytest.mark.parametrize("T,d_in,d_out,pad", [(320, 300, 1000, 5), (2240, 512, 768, 0),
                                              (192, 2560, 2048, 0)])
def test_every_kernel_instance_on_every_kind_of_shape(variant, T, d_in, d_out, pad):
    """The launch picks an epilogue form, a warp count and a load form from the shape; here each
    is pinned in turn, on a ragged shape in padded buffers, on a shape that allows grouped
    loads (both sides of the short-call limit) and on one with more tiles than CTA pairs, so
    that no instance is only ever reached by the shapes that happen to select it.  Integer
    inputs: exact contraction, fp32 fold tolerance."""
    _full_parity(T, d_in, d_out, integer=True, pad=pad, variant=variant)


def test_variant_entry_rejects_values_out_of_range():
    opt = adama.AdamA()
    for bad in (dict(epilogue=3), dict(epi_warps=6), dict(box_loads=2), dict(no_pdl=-1)):
        with pytest.raises(adama.AdamAError) as e:
            opt.debug_set_wgrad_variant(**bad)
        assert e.value.status == adama.Status.ERR_INVALID_ARG
    opt.close()


def test_multi_layer_launch_equals_per_layer_calls_and_the_oracle():
    """adama_linear_wgrad_fold_multi: ten layers of assorted shapes (ragged, more tiles than CTA
    pairs, a single tile, token counts on both sides of the short-call limit, two with bias
    moments) in one call -- two launches, since a launch takes at most eight.  Every layer must
    come out bit for bit as from its own adama_linear_wgrad_fold / _bias_fold call, and (integer
    inputs: exact contraction) match the oracle at the fp32 fold tolerance, element by element."""
    specs = [(192, 200, 328, False), (320, 512, 768, True), (64, 136, 8, False), (192, 2560, 2048, False),
             (2240, 304, 1000, False), (100, 128, 256, True), (640, 1600, 1600, False), (7, 136, 264, False),
             (256, 768, 512, False), (2112, 640, 1280, False)]
    N = 3
    single, multi = adama.AdamA(), adama.AdamA()
    single.begin_minibatch(N)
    multi.begin_minibatch(N)
    layers_s, layers_m, orcs, borcs = [], [], [], []
    for k, (T, d_in, d_out, bias) in enumerate(specs):
        z = lambda *shape: torch.zeros(*shape, device="cuda")
        layers_s.append([z(d_in, d_out), z(d_in, d_out)] + ([z(d_out), z(d_out)] if bias else []))
        layers_m.append([z(d_in, d_out), z(d_in, d_out)] + ([z(d_out), z(d_out)] if bias else []))
        o = AdamAOracle(np.zeros((d_in, d_out)))
        o.begin_minibatch(N)
        orcs.append(o)
        bo = AdamAOracle(np.zeros(d_out))
        bo.begin_minibatch(N)
        borcs.append(bo)
    for i in range(N):
        items = []
        for k, (T, d_in, d_out, bias) in enumerate(specs):
            X, dY = _draw(T, d_in, d_out, 5000 + 100 * i + k, integer=True)
            orcs[k].fold_linear(f64(X), f64(dY))
            if bias:
                borcs[k].fold(oracle.linear_wgrad(np.ones((T, 1)), f64(dY))[0])
            X, dY = X.cuda(), dY.cuda()
            single.linear_wgrad_fold(X, dY, *layers_s[k])
            items.append((X, dY, *layers_m[k]))
        before = multi.launch_count
        multi.linear_wgrad_fold_multi(items)
        assert multi.launch_count - before == 2
    single.sync_status()
    multi.sync_status()
    for k, (T, d_in, d_out, bias) in enumerate(specs):
        for a, b in zip(layers_s[k], layers_m[k]):
            assert torch.equal(a, b), f"layer {k}: grouped launch differs from the per-layer call"
        assert_close(f64(layers_m[k][0]), orcs[k].m, TOL_EXACT, f"m layer {k}")
        assert_close(f64(layers_m[k][1]), orcs[k].v, TOL_EXACT, f"v layer {k}")
        if bias:
            assert_close(f64(layers_m[k][2]), borcs[k].m, TOL_EXACT, f"bias m layer {k}")
            assert_close(f64(layers_m[k][3]), borcs[k].v, TOL_EXACT, f"bias v layer {k}")
    single.close()
    multi.close()


def test_multi_layer_call_checks_every_item_before_launching():
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    X = torch.zeros(64, 128, dtype=torch.bfloat16, device="cuda")
    dY = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(128, 256, device="cuda")
    bad = torch.zeros(64 * 128 + 8, dtype=torch.bfloat16, device="cuda")[1:1 + 64 * 128].view(64, 128)
    with pytest.raises(adama.AdamAError) as e:
        opt.linear_wgrad_fold_multi([(X, dY, m, m.clone()), (bad, dY, m.clone(), m.clone())])
    assert e.value.status == adama.Status.ERR_MISALIGNED and opt.launch_count == 0
    opt.linear_wgrad_fold_multi([])                      # nothing to do
    e0 = torch.empty(0, 128, dtype=torch.bfloat16, device="cuda")
    opt.linear_wgrad_fold_multi([(e0, torch.empty(0, 256, dtype=torch.bfloat16, device="cuda"), m, m.clone())])
    assert opt.launch_count == 0                         # zero tokens: skipped
    opt.close()


def test_long_contraction_phase_wraps():
    _full_parity(4096 + 48, 256, 512, n_micro=1)


def _sampled_entries(d_in, d_out, count, seed):
    rng = np.random.default_rng(seed)
    p = rng.integers(0, d_in, count)
    q = rng.integers(0, d_out, count)
    # corners and the last rows / columns (ragged tiles) are always included
    edge_p = [0, 0, d_in - 1, d_in - 1, d_in - 1, d_in // 2]
    edge_q = [0, d_out - 1, 0, d_out - 1, d_out // 2, d_out - 1]
    return np.concatenate([p, edge_p]), np.concatenate([q, edge_q])


def _sampled_parity(T, d_in, d_out, n_micro, steps, config, count=3000):
    """Benchmark-sized layers: sampled entries (each a T-term dot product in the oracle)
    plus one whole 128x256 tile at the bottom-right corner."""
    opt = adama.AdamA()
    p, q = _sampled_entries(d_in, d_out, count, config)
    r0, c0 = max(0, d_in - 128), max(0, d_out - 256)
    tp, tq = np.meshgrid(np.arange(r0, d_in), np.arange(c0, d_out), indexing="ij")
    p = np.concatenate([p, tp.reshape(-1)])
    q = np.concatenate([q, tq.reshape(-1)])
    flat = torch.from_numpy(p * d_out + q).cuda()
    w = wl.normal((d_in, d_out), 0.02, torch.float32, wl.seed_for(config, 99), device="cuda")
    m = torch.zeros(d_in, d_out, device="cuda")
    v = torch.zeros(d_in, d_out, device="cuda")
    orc = AdamAOracle(f64(w.view(-1)[flat]))
    for step in range(steps):
        opt.begin_minibatch(n_micro)
        orc.begin_minibatch(n_micro)
        for i in range(n_micro):
            X = wl.normal((T, d_in), 1.0, torch.bfloat16, wl.seed_for(config, step, i), device="cuda")
            dY = wl.normal((T, d_out), 1e-2, torch.bfloat16, wl.seed_for(config, step, i) + 50,
                           device="cuda")
            opt.linear_wgrad_fold(X, dY, m, v)
            orc.fold(oracle.linear_wgrad_entries(f64(X), f64(dY), p, q))
        opt.sync_status()
        assert_close(f64(m.view(-1)[flat]), orc.m, TOL_BF16, "m_t")
        assert_close(f64(v.view(-1)[flat]), orc.v, TOL_BF16, "v_t")
        opt.apply(w, m, v, wl.LR)
        orc.update(wl.LR)
        assert_close(f64(w.view(-1)[flat]), orc.theta, TOL_BF16, "w", elementwise=n_micro > 1 or step > 0)
        assert_close(f64(m.view(-1)[flat]), wl.BETA1 * orc.m, TOL_BF16, "beta1*m")
        assert_close(f64(v.view(-1)[flat]), wl.BETA2 * orc.v, TOL_BF16, "beta2*v")
    assert bool((v >= 0).all()) and bool(torch.isfinite(m).all()) and bool(torch.isfinite(w).all())
    opt.close()


def test_config3_sampled():
    """d_in = d_out = 4096, 4096 tokens, N=4, 3 steps (the benchmark's linear layer)."""
    c = wl.CONFIG3
    _sampled_parity(c.tokens, c.d_in, c.d_out, c.n_micro, c.steps, 3)


@pytest.mark.parametrize("name,d_in,d_out", wl.gpt2xl_block_linears())
def test_config4_layer_shapes_sampled(name, d_in, d_out):
    """GPT-2-XL-shaped linears (1600 = 12.5 tiles of 128, 4800 = 18.75 tiles of 256)."""
    _sampled_parity(wl.CONFIG4_TOKENS, d_in, d_out, 2, 1, 4, count=1500)


@pytest.mark.parametrize("name,d_in,d_out", [x for x in wl.llama7b_block_linears()
                                              if x[0] in ("gate", "down")])
def test_config5_layer_shapes_sampled(name, d_in, d_out):
    _sampled_parity(wl.CONFIG5_TOKENS, d_in, d_out, 1, 1, 5, count=1500)


def test_weight_matrix_beyond_2_to_31_elements_sampled():
    """49152 x 49152 weights (2.4 G elements: element offsets into m, v beyond 31 bits, byte
    offsets beyond 33), 64 tokens: sampled entries plus the bottom-right tile."""
    _sampled_parity(64, 49152, 49152, 1, 1, 10, count=4000)
    torch.cuda.empty_cache()


def test_zero_tokens_is_a_noop():
    opt = adama.AdamA()
    opt.begin_minibatch(1)
    m = torch.ones(64, 64, device="cuda")
    v = torch.ones(64, 64, device="cuda")
    e = torch.empty(0, 64, dtype=torch.bfloat16, device="cuda")
    before = opt.launch_count
    opt.linear_wgrad_fold(e, e.clone(), m, v)
    assert opt.launch_count == before and bool((m == 1).all())
    opt.close()


def test_run_twice_is_deterministic():
    T, d_in, d_out = 256, 384, 512
    X, dY = _draw(T, d_in, d_out, 11)
    outs = []
    for _ in range(2):
        opt = adama.AdamA()
        opt.begin_minibatch(3)
        m = torch.zeros(d_in, d_out, device="cuda")
        v = torch.zeros(d_in, d_out, device="cuda")
        for _ in range(3):
            opt.linear_wgrad_fold(X.cuda(), dY.cuda(), m, v)
        opt.sync_status()
        outs.append((m.clone(), v.clone()))
        opt.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_host_buffer_variants_match_device_variants():
    T, d_in, d_out, n = 128, 256, 512, 256 * 512
    X, dY = _draw(T, d_in, d_out, 21)
    g = wl.normal((n,), 1e-3, torch.bfloat16, 22)
    res = []
    for host in (False, True):
        opt = adama.AdamA()
        opt.begin_minibatch(2)
        w = wl.normal((d_in, d_out), 0.02, torch.float32, 23).cuda()
        m = torch.zeros(d_in, d_out, device="cuda")
        v = torch.zeros(d_in, d_out, device="cuda")
        if host:
            staging = torch.empty(4 << 20, dtype=torch.uint8, device="cuda")
            w_host = torch.empty(n, dtype=torch.float32).pin_memory()
            opt.linear_wgrad_fold_host(X.pin_memory(), dY.pin_memory(), m, v, staging)
            opt.fold_host(g.pin_memory(), m.view(-1), v.view(-1), staging)
            opt.apply_to_host(w, m, v, wl.LR, w_host)
            opt.sync_status()
            assert torch.equal(w_host, w.cpu().view(-1))
        else:
            opt.linear_wgrad_fold(X.cuda(), dY.cuda(), m, v)
            opt.fold(g.cuda(), m.view(-1), v.view(-1))
            opt.apply(w, m, v, wl.LR)
            opt.sync_status()
        res.append((w.cpu(), m.cpu(), v.cpu()))
        opt.close()
    for a, b in zip(*res):
        assert torch.equal(a, b)


@pytest.mark.parametrize("T", [512, 4096])
def test_inputs_written_just_before_the_call_and_overwritten_just_after(T):
    """The fused kernel is launched so that its set-up may overlap the end of the kernel before
    it in the stream.  Here that kernel is the one that WRITES dY (and X), and the next one
    overwrites them again at once, 30 times over without any synchronisation: the result must be
    bit-identical to the same sequence with a device synchronisation after every operation."""
    d_in, d_out, rounds = 512, 768, 30
    Xs = [wl.normal((T, d_in), 1.0, torch.bfloat16, 900 + i, device="cuda") for i in range(3)]
    Ys = [wl.normal((T, d_out), 1e-2, torch.bfloat16, 950 + i, device="cuda") for i in range(3)]
    outs = []
    for sync in (True, False):
        opt = adama.AdamA()
        opt.begin_minibatch(rounds)
        X = torch.zeros(T, d_in, dtype=torch.bfloat16, device="cuda")
        dY = torch.zeros(T, d_out, dtype=torch.bfloat16, device="cuda")
        m = torch.zeros(d_in, d_out, device="cuda")
        v = torch.zeros(d_in, d_out, device="cuda")
        for i in range(rounds):
            X.copy_(Xs[i % 3])
            dY.copy_(Ys[(i + 1) % 3])
            if sync:
                torch.cuda.synchronize()
            opt.linear_wgrad_fold(X, dY, m, v)
            if sync:
                torch.cuda.synchronize()
        opt.sync_status()
        outs.append((m.clone(), v.clone()))
        opt.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert float(outs[0][1].max()) > 0


def test_inputs_settled_flag_gives_the_same_results_back_to_back():
    """ADAMA_INPUTS_SETTLED: the operand loads of a call do not wait for the kernel before it, so
    the first tiles of a call run beside the last round of the previous one.  A run of calls back
    to back -- the same layer four times in a row (its m, v carry from call to call, which the
    epilogue's own wait must keep in order), layers with one tile and with more tiles than CTA
    pairs, both epilogue forms, single and grouped launches -- must come out bit for bit as from
    a context without the flag, and the repeated layer must match the oracle (integer inputs: exact).
    All inputs are complete before the first call, which is what the flag promises."""
    N = 4
    specs = [(640, 1600, 1600), (192, 2560, 2048), (2304, 512, 768), (64, 136, 264), (2112, 640, 1280)]
    data = []
    for k, (T, d_in, d_out) in enumerate(specs):
        Xs = [wl.small_integers((T, d_in), 3, torch.bfloat16, 900 + 10 * k + i) for i in range(N)]
        Ys = [wl.small_integers((T, d_out), 3, torch.bfloat16, 950 + 10 * k + i) for i in range(N)]
        data.append((Xs, Ys, [x.cuda() for x in Xs], [y.cuda() for y in Ys]))
    torch.cuda.synchronize()
    results = []
    for settled in (False, True):
        opt = adama.AdamA(inputs_settled=settled)
        opt.begin_minibatch(N)
        states = [(torch.zeros(d_in, d_out, device="cuda"), torch.zeros(d_in, d_out, device="cuda"))
                  for (_, d_in, d_out) in specs]
        for rep in range(2):
            for i in range(N):                       # the same layer, call after call
                opt.linear_wgrad_fold(data[0][2][i], data[0][3][i], *states[0])
            for k in range(1, len(specs)):           # other layers, one launch each
                opt.linear_wgrad_fold(data[k][2][rep], data[k][3][rep], *states[k])
            opt.linear_wgrad_fold_multi([(data[k][2][2 + rep], data[k][3][2 + rep], *states[k])
                                         for k in range(1, len(specs))])   # and grouped
        opt.sync_status()
        results.append(states)
        opt.close()
    for (m0, v0), (m1, v1) in zip(*results):
        assert torch.equal(m0, m1) and torch.equal(v0, v1)
    T, d_in, d_out = specs[0]
    orc = AdamAOracle(np.zeros((d_in, d_out)))
    orc.begin_minibatch(N)
    for rep in range(2):
        for i in range(N):
            orc.fold_linear(f64(data[0][0][i]), f64(data[0][1][i]))
    assert_close(f64(results[1][0][0]), orc.m, TOL_EXACT, "m, settled inputs", elementwise=True)
    assert_close(f64(results[1][0][1]), orc.v, TOL_EXACT, "v, settled inputs", elementwise=True)
