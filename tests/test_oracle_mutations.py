"""The pins must be sharp: a plausible mistake planted in a copy of the oracle's C
source (on the CPU, in a temporary directory) has to make at least one pin fail."""
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

MUTATIONS = {
    "square dropped": ("(1.0 - beta2) * (g * g)", "(1.0 - beta2) * g"),
    "missing 1/N": ("double g = grad[k] / (double)N;", "double g = grad[k];"),
    "square taken before the 1/N": ("(1.0 - beta2) * (g * g)",
                                    "(1.0 - beta2) * (grad[k] * grad[k] / (double)N)"),
    "eps inside the root": ("(sqrt(v_hat) + eps)", "sqrt(v_hat + eps)"),
    "update sign": ("theta[k] - alpha * m_hat", "theta[k] + alpha * m_hat"),
    "no bias correction of v": ("double v_hat = v[k] / c2;", "double v_hat = v[k];"),
    "bias corrections swapped": ("double m_hat = m[k] / c1;", "double m_hat = m[k] / c2;"),
    "v decayed by beta1": ("v[k] = beta2 * v[k];\n    }\n}\n\n/* Algorithm 2, inner",
                           "v[k] = beta1 * v[k];\n    }\n}\n\n/* Algorithm 2, inner"),
    "m folded with beta2": ("m[k] = m[k] + (1.0 - beta1) * g;", "m[k] = m[k] + (1.0 - beta2) * g;"),
    "ddp v divided by R only": ("sv / ((double)devices * (double)devices)", "sv / (double)devices"),
    "ddp v not pre-scaled": ("v[k] = (double)devices * beta2 * v[k];", "v[k] = beta2 * v[k];"),
    "closed form: adam/adama swapped": ("adam_variant ? sum_g * sum_g : sum_g2",
                                        "adam_variant ? sum_g2 : sum_g * sum_g"),
    "weight decay coupled into the gradient term": (
        "theta[k] - alpha * lambda * theta[k] - alpha * m_hat / (sqrt(v_hat) + eps)",
        "theta[k] - alpha * (m_hat + lambda * theta[k]) / (sqrt(v_hat) + eps)"),
    "coefficient inverted": ("double c = sqrt(v_hat) / sqrt(v_hat_adam);",
                             "double c = sqrt(v_hat_adam) / sqrt(v_hat);"),
    "coefficient without the roots": ("double c = sqrt(v_hat) / sqrt(v_hat_adam);",
                                      "double c = v_hat / v_hat_adam;"),
    "coefficient counts zero v'": ("if (!(v_adam[k] > 0.0)) continue;", ""),
    "sgdm missing 1/N": ("double g = grad[k] / (double)N;\n        buf[k]",
                         "double g = grad[k];\n        buf[k]"),
    "sgdm decay dropped": ("buf[k] = mu * buf[k];", "buf[k] = buf[k];"),
    "sgdm update sign": ("theta[k] - alpha * buf[k]", "theta[k] + alpha * buf[k]"),
    "wgrad accumulates |x|": ("acc += X[(size_t)tau * ldx + (size_t)p] * dY",
                              "acc += fabs(X[(size_t)tau * ldx + (size_t)p]) * dY"),
}


def _run_all_pins():
    pins.test_worked_examples_adama()
    pins.test_worked_example_adam_variant_differs()
    for eps in (1e-8, 1e-3):
        pins.test_n1_is_standard_adam(eps)
    pins.test_n1_with_decoupled_decay_is_torch_adamw()
    pins.test_first_moment_is_adams_on_mean_gradient(4)
    pins.test_identical_micro_gradients_give_adam_v_over_n(3)
    pins.test_cauchy_schwarz_bound_and_sign()
    pins.test_closed_form_matches_incremental()
    pins.test_exact_rational_bruteforce()
    pins.test_wgrad_matches_numpy_matmul()
    pins.test_wgrad_structured_inputs()
    pins.test_ddp_state_allreduce_equals_single_device_with_NR_micro_batches(2, 3)
    pins.test_coefficient_worked_example()
    pins.test_coefficient_for_identical_micro_gradients_is_rsqrt_n(5)
    pins.test_coefficient_stats_bruteforce_and_bounds()
    pins.test_sgdm_worked_example()
    pins.test_sgdm_is_torch_sgd_on_the_mean_gradient(4)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    src = (oracle._SRC).read_text()
    assert src.count(old) >= 1, f"mutation target not found: {old!r}"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new, 1))
    so = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(so),
                    str(mutated), "-lm"], check=True)
    monkeypatch.setattr(oracle, "_lib", oracle.load(so))
    with pytest.raises(AssertionError):
        _run_all_pins()


def test_unmutated_oracle_passes_the_same_list():
    _run_all_pins()
