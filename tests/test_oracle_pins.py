"""Pins for the fp64 CPU oracle: checks against things other than itself.

  * hand-worked updates derived from Algorithm 2 (tests/golden/worked_examples.txt);
  * N=1  ==> AdamA is standard Adam (Algorithm 1: both bracket terms coincide),
    checked against torch.optim.Adam in float64;
  * the first moment equals Adam's on the mini-batch mean gradient for any N
    (Algorithm 1, m_t line; Section 3.2 "same updating direction");
  * second moment: identical micro-gradients give exactly Adam's v divided by N;
    Cauchy-Schwarz bound v_AdamA >= v_Adam / N; v >= 0; order of micro-batches
    does not matter;
  * exact rational evaluation of the fully unrolled recurrence on <=16 elements;
  * Algorithm 1's closed form against Algorithm 2's incremental form;
  * the weight gradient against numpy's matmul and structured inputs with
    known answers;
  * Section 3.3, Eqs. 4-7: R devices x N micro-batches == one device x N*R;
  * Section 4.1's coefficient sqrt(v_hat)/sqrt(v_hat'): hand-worked values, the 1/sqrt(N)
    closed form for identical micro-gradients, numpy statistics, the Cauchy-Schwarz floor;
  * the SGD-momentum extension: a hand-worked example and torch.optim.SGD in float64.
"""
from decimal import Decimal, getcontext
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from oracle import AdamADDPOracle, AdamAOracle

GOLDEN = Path(__file__).resolve().parent / "golden" / "worked_examples.txt"
B1, B2, EPS, LR = 0.9, 0.999, 1e-8, 1e-3


def _rows():
    rows = []
    for line in GOLDEN.read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        case, step, N, grads, w0, m, v, w1 = line.split()
        rows.append((case, int(step), int(N), [float(x) for x in grads.split(",")],
                     float(w0), float(m), float(v), float(w1)))
    return rows


def test_worked_examples_adama():
    """Algorithm 2 by hand, examples A (two steps, N=2) and B (identical grads, N=4)."""
    for case in ("A", "B"):
        rows = [r for r in _rows() if r[0] == case]
        orc = AdamAOracle([rows[0][4]], B1, B2, EPS)
        for _, step, N, grads, w0, m, v, w1 in rows:
            assert orc.theta[0] == pytest.approx(w0, rel=1e-15)
            orc.begin_minibatch(N)
            assert orc.t == step
            for g in grads:
                orc.fold([g])
            assert orc.m[0] == pytest.approx(m, rel=1e-13)
            assert orc.v[0] == pytest.approx(v, rel=1e-13)
            orc.update(LR)
            assert orc.theta[0] == pytest.approx(w1, rel=1e-15)


def test_worked_example_adam_variant_differs():
    """The same data under standard Adam (first bracket term of Algorithm 1) gives the
    golden ADAM rows, which differ from AdamA's: the closed-form routine must tell the
    two second moments apart."""
    rows = [r for r in _rows() if r[0] == "ADAM"]
    m = np.zeros(1)
    v = np.zeros(1)
    for _, step, N, grads, w0, m_gold, v_gold, w1 in rows:
        m, v = oracle.closed_form_moments(m, v, np.array(grads).reshape(N, 1), B1, B2, True)
        assert m[0] == pytest.approx(m_gold, rel=1e-13)
        assert v[0] == pytest.approx(v_gold, rel=1e-13)
    a_rows = [r for r in _rows() if r[0] == "A"]
    assert a_rows[-1][6] != pytest.approx(rows[-1][6], rel=1e-3)


def _torch_adam(theta0, eps=EPS, lr=LR):
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.Adam([p], lr=lr, betas=(B1, B2), eps=eps, weight_decay=0.0,
                           amsgrad=False, foreach=False, fused=False)
    return p, opt


@pytest.mark.parametrize("eps", [1e-8, 1e-3])
def test_n1_is_standard_adam(eps):
    """N=1: AdamA == Adam (library implementation, fp64), w, m and v, over 6 steps.
    eps=1e-3 makes the placement of eps (outside the root, after bias correction)
    visible far above rounding."""
    rng = np.random.default_rng(11)
    n = 64
    theta0 = rng.normal(0, 0.02, n)
    orc = AdamAOracle(theta0, B1, B2, eps)
    p, opt = _torch_adam(theta0, eps)
    for step in range(6):
        g = rng.normal(0, 1e-2, n)
        orc.begin_minibatch(1)
        orc.fold(g)
        orc.update(LR)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        st = opt.state[p]
        np.testing.assert_allclose(orc.m, st["exp_avg"].numpy(), rtol=1e-13, atol=0)
        np.testing.assert_allclose(orc.v, st["exp_avg_sq"].numpy(), rtol=1e-13, atol=0)
        np.testing.assert_allclose(orc.theta, p.detach().numpy(), rtol=1e-13, atol=0)


def test_n1_with_decoupled_decay_is_torch_adamw():
    """The weight-decay extension: N=1 equals torch.optim.AdamW (fp64) step by step."""
    rng = np.random.default_rng(31)
    n, wd = 40, 0.05
    theta0 = rng.normal(0, 0.5, n)
    orc = AdamAOracle(theta0, B1, B2, EPS)
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=LR, betas=(B1, B2), eps=EPS, weight_decay=wd, amsgrad=False,
                            foreach=False, fused=False)
    for step in range(5):
        g = rng.normal(0, 1e-2, n)
        orc.begin_minibatch(1)
        orc.fold(g)
        orc.update(LR, weight_decay=wd)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(orc.theta, p.detach().numpy(), rtol=1e-13, atol=0)
    plain = AdamAOracle(theta0, B1, B2, EPS)
    plain.begin_minibatch(1)
    plain.fold(g)
    plain.update(LR)
    assert not np.allclose(plain.theta, theta0 * (1 - LR * wd), rtol=1e-9)


@pytest.mark.parametrize("N", [2, 4, 8])
def test_first_moment_is_adams_on_mean_gradient(N):
    rng = np.random.default_rng(5 + N)
    n = 48
    theta0 = rng.normal(0, 0.02, n)
    orc = AdamAOracle(theta0)
    p, opt = _torch_adam(theta0)
    for step in range(4):
        grads = rng.normal(0, 1e-2, (N, n))
        orc.begin_minibatch(N)
        for i in range(N):
            orc.fold(grads[i])
        orc.update(LR)
        p.grad = torch.tensor(grads.mean(axis=0), dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(orc.m, opt.state[p]["exp_avg"].numpy(), rtol=1e-12, atol=1e-18)


@pytest.mark.parametrize("N", [2, 3, 8])
def test_identical_micro_gradients_give_adam_v_over_n(N):
    """grad_i = G for all i: v increment is (1-beta2) G^2 / N, so v == v_Adam / N for all t."""
    rng = np.random.default_rng(77)
    n = 32
    theta0 = rng.normal(0, 0.02, n)
    orc = AdamAOracle(theta0)
    p, opt = _torch_adam(theta0)
    for step in range(5):
        G = rng.normal(0, 1e-2, n)
        orc.begin_minibatch(N)
        for _ in range(N):
            orc.fold(G)
        orc.update(LR)
        p.grad = torch.tensor(G, dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(orc.v * N, opt.state[p]["exp_avg_sq"].numpy(), rtol=1e-12)
        np.testing.assert_allclose(orc.m, opt.state[p]["exp_avg"].numpy(), rtol=1e-12, atol=1e-18)


def test_cauchy_schwarz_bound_and_sign():
    """(sum g_i)^2 <= N sum g_i^2  ==>  v_AdamA >= v_Adam / N elementwise, and v >= 0."""
    rng = np.random.default_rng(3)
    n, N = 200, 4
    orc = AdamAOracle(np.zeros(n))
    p, opt = _torch_adam(np.zeros(n))
    for step in range(5):
        grads = rng.normal(0, 1.0, (N, n))
        orc.begin_minibatch(N)
        for i in range(N):
            orc.fold(grads[i])
        orc.update(LR)
        p.grad = torch.tensor(grads.mean(axis=0), dtype=torch.float64)
        opt.step()
        v_adam = opt.state[p]["exp_avg_sq"].numpy()
        assert np.all(orc.v >= 0)
        assert np.all(orc.v >= v_adam / N * (1 - 1e-12))
        # and strictly larger somewhere: the micro-gradients are not identical
        assert np.any(orc.v > v_adam / N * 1.01)


def test_micro_batch_order_does_not_matter():
    rng = np.random.default_rng(9)
    n, N = 40, 5
    grads = rng.normal(0, 1e-2, (N, n))
    a = AdamAOracle(np.ones(n))
    b = AdamAOracle(np.ones(n))
    a.begin_minibatch(N)
    b.begin_minibatch(N)
    for i in range(N):
        a.fold(grads[i])
    for i in reversed(range(N)):
        b.fold(grads[i])
    np.testing.assert_allclose(a.m, b.m, rtol=1e-13, atol=1e-20)
    np.testing.assert_allclose(a.v, b.v, rtol=1e-13)


def test_closed_form_matches_incremental():
    """Algorithm 1's per-mini-batch lines against Algorithm 2's decay + folds."""
    rng = np.random.default_rng(21)
    n, N = 100, 4
    orc = AdamAOracle(np.zeros(n))
    m = np.zeros(n)
    v = np.zeros(n)
    for step in range(4):
        grads = rng.normal(0, 1e-2, (N, n))
        orc.begin_minibatch(N)
        for i in range(N):
            orc.fold(grads[i])
        m, v = oracle.closed_form_moments(m, v, grads, B1, B2, adam_variant=False)
        np.testing.assert_allclose(orc.m, m, rtol=1e-12, atol=1e-20)
        np.testing.assert_allclose(orc.v, v, rtol=1e-12)


def test_exact_rational_bruteforce():
    """<=16 elements, N<=4, 3 steps: m_t and v_t are polynomials in the inputs, evaluated
    here in exact rationals from the fully unrolled sums
        m_t = (1-b1) sum_s b1^(t-s) sum_i G_si / N,
        v_t = (1-b2) sum_s b2^(t-s) sum_i (G_si / N)^2,
    and theta with 50-digit decimals."""
    getcontext().prec = 50
    rng = np.random.default_rng(1234)
    n, steps = 16, 3
    Ns = [4, 1, 3]
    theta0 = rng.normal(0, 0.02, n)
    grads = [rng.normal(0, 1e-2, (Ns[s], n)) for s in range(steps)]
    orc = AdamAOracle(theta0, B1, B2, EPS)
    b1, b2 = Fraction(B1), Fraction(B2)            # the doubles, exactly
    theta = [Decimal(float(x)) for x in theta0]

    def dec(fr):
        return Decimal(fr.numerator) / Decimal(fr.denominator)

    for t in range(1, steps + 1):
        orc.begin_minibatch(Ns[t - 1])
        for i in range(Ns[t - 1]):
            orc.fold(grads[t - 1][i])
        orc.update(LR)
        for k in range(n):
            m = Fraction(0)
            v = Fraction(0)
            for s in range(1, t + 1):
                N = Ns[s - 1]
                sg = sum(Fraction(float(grads[s - 1][i, k])) for i in range(N)) / N
                sg2 = sum(Fraction(float(grads[s - 1][i, k])) ** 2 for i in range(N)) / (N * N)
                m += (1 - b1) * b1 ** (t - s) * sg
                v += (1 - b2) * b2 ** (t - s) * sg2
            assert orc.m[k] == pytest.approx(float(m), rel=1e-12, abs=1e-22)
            assert orc.v[k] == pytest.approx(float(v), rel=1e-12)
            m_hat = dec(m / (1 - b1 ** t))
            v_hat = dec(v / (1 - b2 ** t))
            theta[k] = theta[k] - Decimal(LR) * m_hat / (v_hat.sqrt() + Decimal(EPS))
            assert orc.theta[k] == pytest.approx(float(theta[k]), rel=1e-13)


# ---- weight gradient -----------------------------------------------------------------

def test_wgrad_matches_numpy_matmul():
    rng = np.random.default_rng(2)
    T, d_in, d_out = 37, 13, 29                    # all different: a transposed operand fails
    X = rng.normal(0, 1, (T, d_in))
    dY = rng.normal(0, 1e-2, (T, d_out))
    G = oracle.linear_wgrad(X, dY)
    assert G.shape == (d_in, d_out)
    np.testing.assert_allclose(G, X.T @ dY, rtol=1e-12, atol=1e-15)
    p = np.array([0, 12, 5, 7])
    q = np.array([28, 0, 5, 11])
    np.testing.assert_allclose(oracle.linear_wgrad_entries(X, dY, p, q), (X.T @ dY)[p, q],
                               rtol=1e-12, atol=1e-15)


def test_wgrad_structured_inputs():
    rng = np.random.default_rng(4)
    T, d_in, d_out = 12, 5, 7
    dY = rng.normal(0, 1, (T, d_out))
    # all-ones activations: every row of G is the column sum of dY
    G = oracle.linear_wgrad(np.ones((T, d_in)), dY)
    for p in range(d_in):
        np.testing.assert_allclose(G[p], dY.sum(axis=0), rtol=1e-13)
    # one-hot activations: token tau activates feature idx[tau]; G is a scatter-add of dY rows
    idx = rng.integers(0, d_in, T)
    X = np.zeros((T, d_in))
    X[np.arange(T), idx] = 1.0
    G = oracle.linear_wgrad(X, dY)
    want = np.zeros((d_in, d_out))
    for tau in range(T):
        want[idx[tau]] += dY[tau]
    np.testing.assert_allclose(G, want, rtol=1e-13, atol=1e-15)


def test_wgrad_tiny_by_hand():
    X = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]])          # T=3, d_in=2
    dY = np.array([[1.0, 0.0, -1.0], [2.0, 1.0, 0.0], [0.0, -2.0, 1.0]])   # d_out=3
    # G[0] = 1*[1,0,-1] + 3*[2,1,0] + 5*[0,-2,1] = [7,-7,4]
    # G[1] = 2*[1,0,-1] + 4*[2,1,0] + 6*[0,-2,1] = [10,-8,4]
    np.testing.assert_array_equal(oracle.linear_wgrad(X, dY), [[7, -7, 4], [10, -8, 4]])


def test_fold_linear_places_layer_in_flat_state():
    rng = np.random.default_rng(8)
    T, d_in, d_out, N = 9, 3, 4, 2
    orc = AdamAOracle(np.zeros(5 + d_in * d_out))
    orc.begin_minibatch(N)
    X = rng.normal(0, 1, (T, d_in))
    dY = rng.normal(0, 1, (T, d_out))
    orc.fold_linear(X, dY, lo=5)
    G = (X.T @ dY).reshape(-1)
    assert np.all(orc.m[:5] == 0) and np.all(orc.v[:5] == 0)
    np.testing.assert_allclose(orc.m[5:], (1 - B1) * G / N, rtol=1e-12)
    np.testing.assert_allclose(orc.v[5:], (1 - B2) * (G / N) ** 2, rtol=1e-12)


# ---- data-parallel variant -------------------------------------------------------------

@pytest.mark.parametrize("R,N", [(2, 3), (4, 2)])
def test_ddp_state_allreduce_equals_single_device_with_NR_micro_batches(R, N):
    """Eqs. 6-7: after the all-reduce the states equal single-device AdamA with N*R
    micro-batches, every step, so the weights agree too."""
    rng = np.random.default_rng(100 + R)
    n = 24
    theta0 = rng.normal(0, 0.02, n)
    single = AdamAOracle(theta0)
    ddp = AdamADDPOracle(theta0, R)
    for step in range(4):
        grads = rng.normal(0, 1e-2, (R, N, n))
        single.begin_minibatch(N * R)
        ddp.begin_minibatch(N)
        for r in range(R):
            for i in range(N):
                # Section 3.3: on each device g = grad / N (its local micro-batch count)
                ddp.fold(r, grads[r, i])
                single.fold(grads[r, i])
        single.update(LR)
        ddp.allreduce_and_update(LR)
        for r in range(R):
            np.testing.assert_allclose(ddp.m[r], single.m, rtol=1e-12, atol=1e-20)
            np.testing.assert_allclose(ddp.v[r], single.v, rtol=1e-12)
        np.testing.assert_allclose(ddp.theta, single.theta, rtol=1e-13)


# ----- Section 4.1 coefficient statistics and the SGD-momentum extension -----

EXT_GOLDEN = Path(__file__).resolve().parent / "golden" / "extension_examples.txt"


def _ext_rows(kind):
    return [line.split()[1:] for line in EXT_GOLDEN.read_text().splitlines()
            if line.startswith(kind + " ")]


def test_coefficient_worked_example():
    """Section 4.1's coefficient on example A, from the hand-worked v (AdamA) and v' (Adam); the
    oracle's own two second moments on that data must give the same number."""
    rows = [r for r in _rows() if r[0] == "A"]
    adama = AdamAOracle([rows[0][4]], B1, B2, EPS)
    m_adam, v_adam = np.zeros(1), np.zeros(1)
    for (step, va, vb, c), (_, _, N, grads, *_rest) in zip(_ext_rows("COEF"), rows):
        st = oracle.coefficient_stats([float(va)], [float(vb)], int(step), B2)
        assert st["count"] == 1
        for key in ("mean", "min", "max"):
            assert st[key] == pytest.approx(float(c), rel=1e-15)
        adama.begin_minibatch(N)
        for g in grads:
            adama.fold([g])
        m_adam, v_adam = oracle.closed_form_moments(m_adam, v_adam, np.array(grads)[:, None],
                                                    B1, B2, adam_variant=True)
        st = oracle.coefficient_stats(adama.v, v_adam, int(step), B2)
        assert st["mean"] == pytest.approx(float(c), rel=1e-13)
        adama.update(LR)


@pytest.mark.parametrize("N", [1, 2, 5])
def test_coefficient_for_identical_micro_gradients_is_rsqrt_n(N):
    """Identical micro-batch gradients in every mini-batch: v = v'/N at every element and step
    (Algorithm 1's two bracket terms differ by exactly the factor N), so the coefficient is
    1/sqrt(N) everywhere: mean = min = max; N = 1 gives exactly 1 (AdamA is Adam)."""
    rng = np.random.default_rng(5)
    n = 37
    adama = AdamAOracle(np.zeros(n), B1, B2, EPS)
    m_adam, v_adam = np.zeros(n), np.zeros(n)
    for step in range(1, 5):
        G = rng.normal(0, 1e-2, n)
        adama.begin_minibatch(N)
        for _ in range(N):
            adama.fold(G)
        m_adam, v_adam = oracle.closed_form_moments(m_adam, v_adam, np.tile(G, (N, 1)), B1, B2,
                                                    adam_variant=True)
        st = oracle.coefficient_stats(adama.v, v_adam, step, B2)
        assert st["count"] == n
        for key in ("mean", "min", "max"):
            assert st[key] == pytest.approx(1.0 / np.sqrt(N), rel=1e-13)
        adama.update(LR)


def test_coefficient_stats_bruteforce_and_bounds():
    """mean / min / max against numpy on independently formed arrays; zero v' elements are left
    out; Cauchy-Schwarz keeps every coefficient at or above 1/sqrt(N)."""
    rng = np.random.default_rng(6)
    n, N = 50, 4
    adama = AdamAOracle(np.zeros(n), B1, B2, EPS)
    v_adam = np.zeros(n)
    for step in range(1, 4):
        grads = rng.normal(0, 1e-2, (N, n))
        grads[:, :3] = 0.0                       # three elements never see a gradient
        adama.begin_minibatch(N)
        for g in grads:
            adama.fold(g)
        v_adam = B2 * v_adam + (1 - B2) * (grads / N).sum(0) ** 2
        st = oracle.coefficient_stats(adama.v, v_adam, step, B2)
        c = np.sqrt(adama.v[3:] / v_adam[3:])
        assert st["count"] == n - 3
        assert st["mean"] == pytest.approx(c.mean(), rel=1e-13)
        assert st["min"] == pytest.approx(c.min(), rel=1e-13)
        assert st["max"] == pytest.approx(c.max(), rel=1e-13)
        assert st["min"] >= 1 / np.sqrt(N) * (1 - 1e-12)
        assert st["max"] > 1.0 > st["min"] or N == 1
        adama.update(LR)
    empty = oracle.coefficient_stats(np.ones(4), np.zeros(4), 1, B2)
    assert empty["count"] == 0 and empty["min"] == np.inf and empty["max"] == 0.0


def test_sgdm_worked_example():
    rows = _ext_rows("SGDM")
    orc = oracle.SGDMOracle([float(rows[0][3])], momentum=0.9)
    for step, N, grads, w0, buf, w1 in rows:
        assert orc.theta[0] == pytest.approx(float(w0), rel=1e-15)
        orc.begin_minibatch(int(N))
        for g in grads.split(","):
            orc.fold([float(g)])
        assert orc.buf[0] == pytest.approx(float(buf), rel=1e-14)
        orc.update(0.1)
        assert orc.theta[0] == pytest.approx(float(w1), rel=1e-15)


@pytest.mark.parametrize("N", [1, 4])
def test_sgdm_is_torch_sgd_on_the_mean_gradient(N):
    """The folded momentum buffer equals torch.optim.SGD's (fp64, momentum, no dampening) fed
    with the mini-batch mean gradient, step by step."""
    rng = np.random.default_rng(8)
    n, mu, lr = 33, 0.8, 0.05
    theta0 = rng.normal(0, 0.5, n)
    orc = oracle.SGDMOracle(theta0, momentum=mu)
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=lr, momentum=mu, dampening=0.0, nesterov=False, foreach=False)
    for step in range(5):
        grads = rng.normal(0, 1e-1, (N, n))
        orc.begin_minibatch(N)
        for g in grads:
            orc.fold(g)
        orc.update(lr)
        p.grad = torch.tensor(grads.mean(0), dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(orc.buf, opt.state[p]["momentum_buffer"].numpy(), rtol=1e-12)
        np.testing.assert_allclose(orc.theta, p.detach().numpy(), rtol=1e-13)
