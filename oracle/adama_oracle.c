/*
 * AdamA reference arithmetic, fp64, plain C.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct CPU
 * statement of what the GPU library computes.  It shares no code, header,
 * constant or helper with the CUDA path and must never be reached from the
 * product path; only the test-suite, the smoke check and the CPU-baseline leg
 * of the benchmark may load it.
 *
 * Every function follows one passage of the AdamA paper (arXiv 2305.19982):
 *   - Algorithm 2  : the training pipeline (decay, per-micro-batch per-layer
 *                    accumulation into m and v, bias-corrected update);
 *   - Algorithm 1  : the per-mini-batch closed form of the same moments, with
 *                    standard Adam's second moment printed beside AdamA's;
 *   - Section 3.3, Eqs. 4-7 : the data-parallel variant that all-reduces the
 *                    optimizer states instead of the gradients;
 *   - Section 4.1, the figure of the coefficient sqrt(v_hat)/sqrt(v_hat'): the
 *                    statistic that compares AdamA's adaptive scaling with Adam's;
 *   - Discussion   : the same accumulation applied to another momentum optimizer
 *                    (SGD with momentum).
 * Nothing is blocked, fused or reordered beyond what those passages state.
 * Loops carry an OpenMP "parallel for" over independent elements only (no
 * reduction is ever split), so results do not depend on the thread count.
 *
 * Pin status: every function below is pinned by tests that do not re-type its
 * formula (torch.optim.Adam in fp64, exact rational evaluation of the
 * unrolled recurrence, closed forms for structured inputs, library matmul).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#if defined(__GNUC__)
#define ORACLE_API __attribute__((visibility("default")))
#else
#define ORACLE_API
#endif

/* Number of threads an "omp parallel for" in this file will use. */
ORACLE_API int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Limits the threads of the loops below (timing with 1 thread and with all cores); no
 * effect on results, since no reduction is split across threads. */
ORACLE_API void oracle_set_num_threads(int threads) {
#ifdef _OPENMP
    if (threads >= 1) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
}

/* Algorithm 2, first line of the while-body: m_t <- beta1*m_{t-1},
 * v_t <- beta2*v_{t-1}.  (The step counter t <- t+1 is kept by the caller.) */
ORACLE_API void oracle_decay(double *m, double *v, size_t n, double beta1, double beta2) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        m[k] = beta1 * m[k];
        v[k] = beta2 * v[k];
    }
}

/* Algorithm 2, inner loop body for one (micro-batch i, layer j):
 *     g   <- (1/N) * grad                      (grad = raw micro-batch gradient)
 *     m_j <- m_j + (1-beta1) * g
 *     v_j <- v_j + (1-beta2) * g^2
 * The square is taken after the 1/N scaling, as Eq. 5 prints it. */
ORACLE_API void oracle_fold(double *m, double *v, const double *grad, size_t n,
                            int N, double beta1, double beta2) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        double g = grad[k] / (double)N;
        m[k] = m[k] + (1.0 - beta1) * g;
        v[k] = v[k] + (1.0 - beta2) * (g * g);
    }
}

/* Algorithm 2 (and Algorithm 1), "Update":
 *     m_hat <- m/(1-beta1^t),  v_hat <- v/(1-beta2^t),
 *     theta <- theta - alpha*m_hat/(sqrt(v_hat)+eps)
 * eps sits outside the square root and is added after the bias correction. */
ORACLE_API void oracle_update(double *theta, const double *m, const double *v, size_t n,
                              long t, double alpha, double beta1, double beta2, double eps) {
    double c1 = 1.0 - pow(beta1, (double)t);
    double c2 = 1.0 - pow(beta2, (double)t);
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        double m_hat = m[k] / c1;
        double v_hat = v[k] / c2;
        theta[k] = theta[k] - alpha * m_hat / (sqrt(v_hat) + eps);
    }
}

/* Extension outside the paper's algorithms (its Discussion only remarks that other
 * momentum optimizers can take the same accumulation): the update above with decoupled
 * weight decay as in AdamW (Loshchilov & Hutter, "Decoupled Weight Decay Regularization",
 * Algorithm 2):  theta <- theta - alpha*lambda*theta - alpha*m_hat/(sqrt(v_hat)+eps).
 * lambda = 0 is oracle_update. */
ORACLE_API void oracle_update_decoupled_decay(double *theta, const double *m, const double *v,
                                              size_t n, long t, double alpha, double beta1,
                                              double beta2, double eps, double lambda) {
    double c1 = 1.0 - pow(beta1, (double)t);
    double c2 = 1.0 - pow(beta2, (double)t);
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        double m_hat = m[k] / c1;
        double v_hat = v[k] / c2;
        theta[k] = theta[k] - alpha * lambda * theta[k] - alpha * m_hat / (sqrt(v_hat) + eps);
    }
}

/* Algorithm 1, the two moment lines, evaluated per mini-batch from the stored
 * list of raw micro-batch gradients grads[i*n + k], i < N:
 *     g_i = grads_i / N
 *     m_t = beta1*m + (1-beta1) * sum_i g_i
 *     v_t = beta2*v + (1-beta2) * [ (sum_i g_i)^2   if adam_variant   (Adam)
 *                                   sum_i (g_i^2)   otherwise ]       (AdamA)
 * Written independently of oracle_decay/oracle_fold so the two routes to the
 * AdamA moments can be checked against one another. */
ORACLE_API void oracle_closed_form_moments(double *m, double *v, const double *grads, size_t n,
                                           int N, double beta1, double beta2, int adam_variant) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        double sum_g = 0.0, sum_g2 = 0.0;
        for (int i = 0; i < N; ++i) {
            double g = grads[(size_t)i * n + (size_t)k] / (double)N;
            sum_g += g;
            sum_g2 += g * g;
        }
        double second = adam_variant ? sum_g * sum_g : sum_g2;
        m[k] = beta1 * m[k] + (1.0 - beta1) * sum_g;
        v[k] = beta2 * v[k] + (1.0 - beta2) * second;
    }
}

/* Raw weight gradient of a linear layer y = x.W with W laid out [d_in, d_out]:
 *     G[p,q] = sum_{tau<T} X[tau,p] * dY[tau,q]
 * (the "gradients of a layer" that Algorithm 2 accumulates; the paper leaves
 * their production to the framework).  Naive triple loop; X is [T, ldx],
 * dY is [T, ldy], G is [d_in, d_out] dense. */
ORACLE_API void oracle_linear_wgrad(const double *X, const double *dY, int T, int d_in, int d_out,
                                    size_t ldx, size_t ldy, double *G) {
#pragma omp parallel for schedule(static)
    for (int p = 0; p < d_in; ++p) {
        for (int q = 0; q < d_out; ++q) {
            double acc = 0.0;
            for (int tau = 0; tau < T; ++tau) {
                acc += X[(size_t)tau * ldx + (size_t)p] * dY[(size_t)tau * ldy + (size_t)q];
            }
            G[(size_t)p * (size_t)d_out + (size_t)q] = acc;
        }
    }
}

/* Same definition, for a list of sampled entries (p[s], q[s]) only, so that
 * layers too large for the full triple loop can still be checked entry by
 * entry. */
ORACLE_API void oracle_linear_wgrad_entries(const double *X, const double *dY, int T,
                                            size_t ldx, size_t ldy, const int64_t *p,
                                            const int64_t *q, size_t count, double *out) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t s = 0; s < (ptrdiff_t)count; ++s) {
        double acc = 0.0;
        for (int tau = 0; tau < T; ++tau) {
            acc += X[(size_t)tau * ldx + (size_t)p[s]] * dY[(size_t)tau * ldy + (size_t)q[s]];
        }
        out[s] = acc;
    }
}

/* Section 3.3, data-parallel variant, start of a mini-batch on one device:
 * v_{t-1} is scaled by devices*beta2 where the single-device algorithm scales it
 * by beta2; m is decayed by beta1 as before (Eqs. 4-5). */
ORACLE_API void oracle_ddp_decay(double *m, double *v, size_t n, int devices,
                                 double beta1, double beta2) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        m[k] = beta1 * m[k];
        v[k] = (double)devices * beta2 * v[k];
    }
}

/* Section 3.3, the state all-reduce at the end of a mini-batch: the devices'
 * m are summed and divided by M; the devices' v are summed and divided by M^2
 * (giving Eqs. 6-7).  m_ranks / v_ranks hold `devices` arrays of n back to
 * back; every device ends with the same reduced state, written to m_out/v_out. */
ORACLE_API void oracle_ddp_allreduce(const double *m_ranks, const double *v_ranks, size_t n,
                                     int devices, double *m_out, double *v_out) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        double sm = 0.0, sv = 0.0;
        for (int r = 0; r < devices; ++r) {
            sm += m_ranks[(size_t)r * n + (size_t)k];
            sv += v_ranks[(size_t)r * n + (size_t)k];
        }
        m_out[k] = sm / (double)devices;
        v_out[k] = sv / ((double)devices * (double)devices);
    }
}

/* Section 4.1, the coefficient between AdamA's and standard Adam's adaptive scaling at
 * step t:  c = sqrt(v_hat) / sqrt(v_hat'),  v_hat = v/(1-beta2^t) AdamA's bias-corrected
 * second moment and v_hat' = v'/(1-beta2^t) Adam's, both tracked over the same gradients.
 * The paper plots, per training step, the mean of c over the elements and its range.
 * out[0] = sum of c, out[1] = min, out[2] = max, out[3] = number of elements counted.
 * Elements whose v' is zero have no coefficient and are left out (the paper does not say;
 * with out[3] == 0, min is +infinity and max is 0).  Serial: one fixed summation order. */
ORACLE_API void oracle_coefficient_stats(const double *v_adama, const double *v_adam, size_t n,
                                         long t, double beta2, double *out) {
    double c2 = 1.0 - pow(beta2, (double)t);
    double sum = 0.0, lo = INFINITY, hi = 0.0, count = 0.0;
    for (size_t k = 0; k < n; ++k) {
        if (!(v_adam[k] > 0.0)) continue;
        double v_hat = v_adama[k] / c2;
        double v_hat_adam = v_adam[k] / c2;
        double c = sqrt(v_hat) / sqrt(v_hat_adam);
        sum += c;
        if (c < lo) lo = c;
        if (c > hi) hi = c;
        count += 1.0;
    }
    out[0] = sum;
    out[1] = lo;
    out[2] = hi;
    out[3] = count;
}

/* Extension outside the paper's algorithms (its Discussion says that other momentum
 * optimizers can take the same accumulation): SGD with momentum mu and no dampening,
 *     buf_t = mu*buf_{t-1} + g_t,   theta_t = theta_{t-1} - alpha*buf_t,
 * with g_t = sum_i grad_i/N folded into buf one micro-batch at a time, as Algorithm 2
 * folds into m.  Three steps in Algorithm 2's order: decay, fold, update. */
ORACLE_API void oracle_sgdm_decay(double *buf, size_t n, double mu) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        buf[k] = mu * buf[k];
    }
}

ORACLE_API void oracle_sgdm_fold(double *buf, const double *grad, size_t n, int N) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        double g = grad[k] / (double)N;
        buf[k] = buf[k] + g;
    }
}

ORACLE_API void oracle_sgdm_update(double *theta, const double *buf, size_t n, double alpha) {
#pragma omp parallel for schedule(static)
    for (ptrdiff_t k = 0; k < (ptrdiff_t)n; ++k) {
        theta[k] = theta[k] - alpha * buf[k];
    }
}
