// Reference ("oracle") implementation of the parameter-server update of Gap-Aware
// asynchronous SGD (arXiv 1909.10802), with Staleness-Aware and plain momentum-ASGD
// as variants.
//
// THIS IS TEST INFRASTRUCTURE. It is a plain, single-threaded, obviously-correct CPU
// program that follows the paper's algorithms step by step. Only the tests, the smoke
// check and the CPU-baseline leg of the benchmark may use it. It shares no code with
// the CUDA library and neither includes the other.
//
// What follows which passage of the paper:
//   push, variant ASGD : Algorithm "Momentum-ASGD: master" (Section 4)
//   push, variant SA   : Algorithm "Staleness-Aware: master" (Section 4.1)
//   push, variant GA   : Algorithm "Gap-Aware: master" (Section 5) with the
//                        parameter-wise Gap of Section 5.3 (|theta_k - theta_{k-tau}|/C + 1)
//   C                  : Algorithm "C Coefficient Calculation" (Appendix, C Coefficient)
//   pull               : the closing send step (for GA: save, then send) of the three master
//                        algorithms; the saved copy is
//                        the theta^i = theta_{k-tau_k} of the appendix's remark
//   push, ADAM*        : Algorithms "Adam: master", "Adam-Staleness-Aware: master" and
//                        "Adam-Gap-Aware: master" (appendix): the penalty (1/tau or 1/G) enters
//                        the first moment only
//   push, GA_LAYER     : Section 5.3, the layer-wise Gap G_p = ||theta_p - theta^i_p|| / C_p + 1
//                        (one layer = the global Gap of Definition 1); the gradient of layer
//                        p is multiplied by 1/G_p, then the momentum step of "Gap-Aware: master"
//   momentum           : Section 3, the variant without dampening: v <- gamma v + g
//   push, SA_GRAD      : Algorithm "Staleness-Aware-Gradient: master" (appendix): g / tau
//   push/pull, DANA*   : Algorithms "DANA: master", "DANA-Staleness-Aware: master" and
//                        "DANA-Gap-Aware: master" (appendix): one momentum vector v^i per
//                        worker, theta <- theta - eta v^i, and the worker is sent (and, for
//                        the Gap, the master saves) the estimate theta - eta gamma sum_j v^j
//
// Readings taken where the paper leaves a choice (all also listed in the design notes):
//   * Order of C and Gap (option c_order). 0 = "lagged": the Gap at arrival k uses the C
//     that stands after arrival k-1; after the step, the second moment m is refreshed with
//     the update vector actually applied (the master's new v). 1 = "Adam order": first
//     u = gamma v + g with the raw gradient (the printed line of the C algorithm),
//     m <- beta m + (1-beta) u^2, C from the new m, then Gap, penalised gradient, v, theta.
//   * The C algorithm starts from C = 0: before any refresh, C = eta_max * eps (the last line of the C
//     algorithm at m_hat = 0), so the first Gap is 0/C + 1 = 1, not 0/0.
//   * The exponent of the bias correction is the number of refreshes of m so far.
//   * eps = 1e-8 is added after the square root, inside the eta_max product.
//   * eta_max is the learning rate given at creation.
//   * delay tau_k = k - iter[i], k counting arrivals from 1, iter[] starting at 0;
//     a pull records the number of pushes applied so far.
//   * The penalised gradient is formed as the algorithm prints it, (1/G_k) (.) g: the
//     reciprocal of the Gap, rounded, then an elementwise product.
//   * DANA's sum over the workers' momentum vectors (option dana_sum): 1 = kept as a running
//     sum, S <- (S - v^i_old) + v^i_new at each arrival (what a master would do; default);
//     0 = the printed sum_{j=1..N} v^j evaluated afresh, in order, at every send. The two are
//     equal in exact arithmetic and are pinned against each other.
//   * Adam-GA's C: the C algorithm is written for a momentum update step gamma v + g, and Adam has no momentum
//     coefficient, so it is run with gamma = 0: m is the running second moment of the raw
//     gradient with the constant beta given at creation (its own state, separate from Adam's
//     v); c_order decides as before whether the Gap sees m before or after this arrival's refresh.
//   * Adam's bias corrections use k = the arrival index; m_hat = m * (1/(1-beta1^k)) with the
//     reciprocal formed in double and rounded once, as for C.
//   * Layer-wise / global C: the C algorithm run once per layer: m_p is the running average
//     of the squared NORM of layer p's update vector, C_p = eta_max (sqrt(m_p / (1 - beta^k))
//     + eps). Squared norms are accumulated in fp64 and rounded once to the working precision
//     (a sum of millions of fp32 terms has no meaningful fp32 order). Lagged order only.
//   * Arithmetic: every line below is one IEEE operation per symbol, in the order
//     written, with v <- gamma*v + g_hat and theta <- theta - eta*v each a single fused
//     multiply-add. Build with -ffp-contract=off so nothing else is fused.
//
// Parity pins (tests/test_oracle_pins.py): Gap >= 1 and Gap == 1 where the saved copy
// equals the master; one worker reduces to heavy-ball SGD (closed form); the SA two-step
// expansion of Section 4.1; gamma = 0; constant |v| gives C = eta_max (c + eps) at every k;
// same-direction steps give Gap = tau; round-robin delays; an exact-rational brute force.
// "parity unpinned": the choice between the two c_order readings and the value of C
// before the first refresh -- nothing the paper prints separates them.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

// The parity reference is this file built single-threaded. Built a second time with
// -fopenmp -DGAO_OPENMP, the loops over parameters (independent per parameter) are split across
// threads; that build exists only so that the benchmark can time the same program on all host
// cores, and a test holds it to the single-threaded build bit for bit (the statistics' fp64 sum
// changes its order, nothing else does).
#ifdef GAO_OPENMP
#define GAO_PARALLEL _Pragma("omp parallel for schedule(static)")
#define GAO_PARALLEL_STATS _Pragma("omp parallel for schedule(static) reduction(+ : sum_gap) reduction(max : max_gap)")
#else
#define GAO_PARALLEL
#define GAO_PARALLEL_STATS
#endif

namespace {

enum Variant { ASGD = 0, SA = 1, GA = 2, SA_GRAD = 3, DANA = 4, DANA_SA = 5, DANA_GA = 6,
               ADAM = 7, ADAM_SA = 8, ADAM_GA = 9, GA_LAYER = 10 };

template <typename T>
struct Master {
    int64_t d = 0;
    int n_workers = 0;
    T eta = 0;        // learning rate eta_k (constant here)
    T eta_max = 0;    // eta_max of the C algorithm
    T gamma = 0;      // momentum
    T beta = 0;       // beta_1 of the C algorithm
    T eps = (T)1e-8;  // epsilon of the C algorithm
    int variant = GA;
    int c_order = 0;  // 0 lagged, 1 Adam order
    std::vector<T> theta, v, m;
    std::vector<T> saved;       // N x d, row i = theta^i, the parameters last sent to worker i
    std::vector<T> vw;          // DANA: N x d, row i = v^i, worker i's momentum
    std::vector<T> vsum;        // DANA: sum_j v^j
    int dana_sum = 1;           // 1 running sum, 0 summed afresh at every send
    std::vector<int64_t> layer_off;   // GA_LAYER: layer p = elements [layer_off[p], layer_off[p+1])
    std::vector<T> m_layer;           // GA_LAYER: m_p of the C algorithm, one scalar per layer
    std::vector<double> last_layer_gap;
    std::vector<T> v2;          // Adam: second moment (the first moment lives in v; gamma is beta_1)
    T wd = 0;                   // weight decay lambda
    int nesterov = 0;           // 1: Nesterov form of the momentum step
    T beta2 = (T)0.999f;        // Adam: beta_2
    T adam_eps = (T)1e-8f;      // Adam: epsilon
    std::vector<int64_t> iter;  // iteration array of the SA algorithm
    int64_t k_done = 0;         // arrivals applied so far
    int64_t k_c = 0;            // refreshes of m so far
    double last_sum_gap = 0.0, last_max_gap = 0.0;

    // The gradient the master works with. Appendix "Weight Decay": under GA the decay term
    // belongs to the gradient and is penalised by the Gap with it; the master forms it from its
    // current parameters, g + lambda * theta_k (one FMA).
    T gw(const float* grad, int64_t j) const {
        return wd == (T)0 ? (T)grad[j] : std::fma(wd, theta[j], (T)grad[j]);
    }

    // The parameter step of the one-momentum-vector masters. Printed form: theta - eta v_{k+1}.
    // Nesterov form (Section 6 says the runs used Nesterov momentum but no master algorithm is printed that way;
    // this is the form of the common framework optimisers): theta - eta (g_hat + gamma v_{k+1}).
    T step(T th, T v_new, T g_pen, T e) const {
        if (!nesterov) return std::fma(-e, v_new, th);
        return std::fma(-e, std::fma(gamma, v_new, g_pen), th);
    }

    // 1 / (1 - beta^k) of the bias correction, k = refreshes of m so far (k >= 1).
    T inv_bias() const { return (T)(1.0 / (1.0 - std::pow((double)beta, (double)k_c))); }

    // C from the second moment as it stands (C algorithm, last two lines).
    T coeff(T m_j, T inv_bias_k) const {
        if (k_c == 0) return eta_max * eps;
        const T m_hat = m_j * inv_bias_k;
        return eta_max * (std::sqrt(m_hat) + eps);
    }

    void set_params(const float* theta0) {
        for (int64_t j = 0; j < d; ++j) {
            theta[j] = (T)theta0[j];
            v[j] = 0;
            m[j] = 0;
        }
        for (int i = 0; i < n_workers; ++i)
            for (int64_t j = 0; j < d; ++j) saved[(size_t)i * d + j] = theta[j];
        for (int i = 0; i < n_workers; ++i) iter[i] = 0;
        k_done = 0;
        k_c = 0;
        std::fill(v2.begin(), v2.end(), (T)0);
        std::fill(m_layer.begin(), m_layer.end(), (T)0);
        std::fill(vw.begin(), vw.end(), (T)0);
        std::fill(vsum.begin(), vsum.end(), (T)0);
    }

    bool is_dana() const { return variant == DANA || variant == DANA_SA || variant == DANA_GA; }
    bool has_gap() const { return variant == GA || variant == DANA_GA || variant == ADAM_GA; }
    // One arrival with the layer-wise Gap.
    void push_layers(int i, const float* grad) {
        const T* s = &saved[(size_t)i * d];
        const T one_minus_beta = (T)(1.0 - (double)beta);
        const T ib = k_c > 0 ? inv_bias() : (T)0;
        const size_t P = m_layer.size();
        for (size_t p = 0; p < P; ++p) {
            const int64_t lo = layer_off[p], hi = layer_off[p + 1];
            double dist2 = 0.0;                                   // ||theta_p - theta^i_p||^2
            for (int64_t j = lo; j < hi; ++j) {
                const T diff = theta[j] - s[j];
                dist2 += (double)diff * (double)diff;
            }
            const T dist = (T)std::sqrt(dist2);
            const T C = coeff(m_layer[p], ib);
            const T G = dist / C + (T)1;
            const T inv_gap = (T)1 / G;
            last_layer_gap[p] = (double)G;
            double norm2 = 0.0;                                   // ||v_{k+1,p}||^2
            for (int64_t j = lo; j < hi; ++j) {
                const T g_hat = inv_gap * gw(grad, j);
                v[j] = std::fma(gamma, v[j], g_hat);
                theta[j] = step(theta[j], v[j], g_hat, eta);
                norm2 += (double)v[j] * (double)v[j];
            }
            m_layer[p] = std::fma(beta, m_layer[p], one_minus_beta * (T)norm2);
        }
        k_c += 1;
    }

    void set_layers(const int64_t* off, int n) {
        layer_off.assign(off, off + n + 1);
        m_layer.assign(n, 0);
        last_layer_gap.assign(n, 1.0);
    }

    bool is_adam() const { return variant == ADAM || variant == ADAM_SA || variant == ADAM_GA; }

    // One arrival of the three Adam masters. v holds the first moment, gamma is beta_1.
    void push_adam(int i, const float* grad, int64_t k, int64_t tau) {
        const T* s = &saved[(size_t)i * d];
        const T beta1 = gamma;
        const T one_minus_beta1 = (T)(1.0 - (double)beta1);
        const T one_minus_beta2 = (T)(1.0 - (double)beta2);
        const T one_minus_beta = (T)(1.0 - (double)beta);
        const T inv_bias1 = (T)(1.0 / (1.0 - std::pow((double)beta1, (double)k)));
        const T inv_bias2 = (T)(1.0 / (1.0 - std::pow((double)beta2, (double)k)));
        double sum_gap = 0.0, max_gap = 0.0;
        if (variant == ADAM_GA && c_order == 1) {
            GAO_PARALLEL
            for (int64_t j = 0; j < d; ++j) {
                const T g = gw(grad, j);
                m[j] = std::fma(beta, m[j], one_minus_beta * (g * g));
            }
            k_c += 1;
        }
        const T ib = k_c > 0 ? inv_bias() : (T)0;
        GAO_PARALLEL_STATS
        for (int64_t j = 0; j < d; ++j) {
            const T g = gw(grad, j);
            T first;                                         // what is added to beta_1 m
            if (variant == ADAM) {
                first = one_minus_beta1 * g;
            } else if (variant == ADAM_SA) {
                first = one_minus_beta1 * (g / (T)tau);      // (1 - beta_1) g / tau
            } else {
                const T C = coeff(m[j], ib);
                const T dist = std::fabs(theta[j] - s[j]);
                const T G = dist / C + (T)1;
                first = (one_minus_beta1 / G) * g;           // ((1 - beta_1) / G) (.) g
                sum_gap += (double)G;
                if ((double)G > max_gap) max_gap = (double)G;
            }
            v[j] = std::fma(beta1, v[j], first);
            v2[j] = std::fma(beta2, v2[j], one_minus_beta2 * (g * g));
            const T m_hat = v[j] * inv_bias1;
            const T v_hat = v2[j] * inv_bias2;
            theta[j] = theta[j] - (eta * m_hat) / (std::sqrt(v_hat) + adam_eps);
            if (variant == ADAM_GA && c_order == 0)          // lagged: C's state sees g after the Gap used it
                m[j] = std::fma(beta, m[j], one_minus_beta * (g * g));
        }
        if (variant == ADAM_GA && c_order == 0) k_c += 1;
        last_sum_gap = sum_gap;
        last_max_gap = max_gap;
    }

    void pull(int i) {
        if (is_dana()) { pull_dana(i); return; }
        GAO_PARALLEL
        for (int64_t j = 0; j < d; ++j) saved[(size_t)i * d + j] = theta[j];
        iter[i] = k_done;
    }

    // DANA's send step: the worker gets the estimate theta - eta gamma sum_j v^j, which is also saved.
    void pull_dana(int i) {
        const T eta_gamma = eta * gamma;
        GAO_PARALLEL
        for (int64_t j = 0; j < d; ++j) {
            T total = vsum[j];
            if (dana_sum == 0) {
                total = 0;
                for (int w = 0; w < n_workers; ++w) total = total + vw[(size_t)w * d + j];
            }
            saved[(size_t)i * d + j] = std::fma(-eta_gamma, total, theta[j]);
        }
        iter[i] = k_done;
    }

    // One arrival of the three DANA masters.
    void push_dana(int i, const float* grad, int64_t tau) {
        T* vi = &vw[(size_t)i * d];
        const T* s = &saved[(size_t)i * d];
        const T one_minus_beta = (T)(1.0 - (double)beta);
        double sum_gap = 0.0, max_gap = 0.0;
        if (variant == DANA_GA && c_order == 1) {
            GAO_PARALLEL
            for (int64_t j = 0; j < d; ++j) {
                const T u = std::fma(gamma, vi[j], gw(grad, j));
                m[j] = std::fma(beta, m[j], one_minus_beta * (u * u));
            }
            k_c += 1;
        }
        const T ib = k_c > 0 ? inv_bias() : (T)0;
        GAO_PARALLEL_STATS
        for (int64_t j = 0; j < d; ++j) {
            const T g = gw(grad, j);
            T g_pen = g;                                   // DANA: the gradient as it is
            if (variant == DANA_SA) {
                g_pen = g / (T)tau;                        // DANA-SA: g / tau
            } else if (variant == DANA_GA) {
                const T C = coeff(m[j], ib);
                const T dist = std::fabs(theta[j] - s[j]); // s = the estimate saved when sent
                const T G = dist / C + (T)1;
                const T inv_gap = (T)1 / G;
                g_pen = inv_gap * g;
                sum_gap += (double)G;
                if ((double)G > max_gap) max_gap = (double)G;
            }
            const T v_old = vi[j];
            const T v_new = std::fma(gamma, v_old, g_pen); // worker's momentum v^i
            vi[j] = v_new;
            theta[j] = std::fma(-eta, v_new, theta[j]);    // master's weights
            vsum[j] = (vsum[j] - v_old) + v_new;           // running sum_j v^j
        }
        if (variant == DANA_GA && c_order == 0) {
            GAO_PARALLEL
            for (int64_t j = 0; j < d; ++j)
                m[j] = std::fma(beta, m[j], one_minus_beta * (vi[j] * vi[j]));
            k_c += 1;
        }
        last_sum_gap = sum_gap;
        last_max_gap = max_gap;
    }

    int64_t push(int i, const float* grad) {
        const int64_t k = k_done + 1;
        const int64_t tau = k - iter[i];
        const T* s = &saved[(size_t)i * d];
        if (is_dana()) {
            push_dana(i, grad, tau);
        } else if (is_adam()) {
            push_adam(i, grad, k, tau);
        } else if (variant == GA_LAYER) {
            push_layers(i, grad);
        } else if (variant == SA_GRAD) {
            GAO_PARALLEL
            for (int64_t j = 0; j < d; ++j) {
                const T g_tau = gw(grad, j) / (T)tau;
                v[j] = std::fma(gamma, v[j], g_tau);
                theta[j] = step(theta[j], v[j], g_tau, eta);
            }
        } else if (variant == ASGD) {
            GAO_PARALLEL
            for (int64_t j = 0; j < d; ++j) {
                const T g = gw(grad, j);
                v[j] = std::fma(gamma, v[j], g);
                theta[j] = step(theta[j], v[j], g, eta);
            }
        } else if (variant == SA) {
            const T eta_tau = eta / (T)tau;
            GAO_PARALLEL
            for (int64_t j = 0; j < d; ++j) {
                const T g = gw(grad, j);
                v[j] = std::fma(gamma, v[j], g);
                theta[j] = step(theta[j], v[j], g, eta_tau);
            }
        } else {
            const T one_minus_beta = (T)(1.0 - (double)beta);
            double sum_gap = 0.0, max_gap = 0.0;
            if (c_order == 1) {
                // Adam order: refresh m from u = gamma v + g (raw gradient) first.
                GAO_PARALLEL
                for (int64_t j = 0; j < d; ++j) {
                    const T u = std::fma(gamma, v[j], gw(grad, j));
                    m[j] = std::fma(beta, m[j], one_minus_beta * (u * u));
                }
                k_c += 1;
            }
            const T ib = k_c > 0 ? inv_bias() : (T)0;
            GAO_PARALLEL_STATS
            for (int64_t j = 0; j < d; ++j) {
                const T g = gw(grad, j);
                const T C = coeff(m[j], ib);
                const T dist = std::fabs(theta[j] - s[j]);
                const T G = dist / C + (T)1;
                const T inv_gap = (T)1 / G;       // the printed form: (1/G_k) (.) g
                const T g_hat = inv_gap * g;
                v[j] = std::fma(gamma, v[j], g_hat);
                theta[j] = step(theta[j], v[j], g_hat, eta);
                sum_gap += (double)G;
                if ((double)G > max_gap) max_gap = (double)G;
            }
            if (c_order == 0) {
                GAO_PARALLEL
                for (int64_t j = 0; j < d; ++j)
                    m[j] = std::fma(beta, m[j], one_minus_beta * (v[j] * v[j]));
                k_c += 1;
            }
            last_sum_gap = sum_gap;
            last_max_gap = max_gap;
        }
        k_done = k;
        return tau;
    }

    // Overwrite the whole state (used by tests that start both precisions from one state).
    void set_state(const double* th, const double* vv, const double* mm, const double* sv,
                   const int64_t* it, int64_t kd, int64_t kc, const double* vworkers) {
        for (int64_t j = 0; j < d; ++j) { theta[j] = (T)th[j]; v[j] = (T)vv[j]; m[j] = (T)mm[j]; }
        if (is_adam()) {      // vworkers carries Adam's second moment (one row)
            for (int64_t j = 0; j < d; ++j) v2[j] = (T)vworkers[j];
        }
        if (is_dana()) {      // vv carries sum_j v^j, vworkers the N rows
            for (int64_t j = 0; j < d; ++j) vsum[j] = (T)vv[j];
            for (size_t q = 0; q < (size_t)n_workers * d; ++q) vw[q] = (T)vworkers[q];
        }
        for (size_t q = 0; q < (size_t)n_workers * d; ++q) saved[q] = (T)sv[q];
        for (int i = 0; i < n_workers; ++i) iter[i] = it[i];
        k_done = kd;
        k_c = kc;
    }

    // Gap of worker i against the master as it stands; changes nothing.
    void gap(int i, double* out) const {
        const T* s = &saved[(size_t)i * d];
        const T ib = k_c > 0 ? inv_bias() : (T)0;
        for (int64_t j = 0; j < d; ++j) {
            const T C = coeff(m[j], ib);
            const T dist = std::fabs(theta[j] - s[j]);
            out[j] = (double)(dist / C + (T)1);
        }
    }
};

struct Handle {
    int precision;  // 32 or 64
    Master<float>* f;
    Master<double>* g;
};

template <typename T>
Master<T>* make(int64_t d, int n, double lr, double momentum, double beta, int variant) {
    auto* M = new Master<T>();
    M->d = d;
    M->n_workers = n;
    // Hyper-parameters arrive as fp32 values (the library's interface takes floats).
    M->eta = (T)(float)lr;
    M->eta_max = (T)(float)lr;
    M->gamma = (T)(float)momentum;
    M->beta = (T)(float)beta;
    M->variant = variant;
    M->theta.assign(d, 0);
    M->v.assign(d, 0);
    M->m.assign(d, 0);
    M->saved.assign((size_t)n * d, 0);
    M->iter.assign(n, 0);
    if (M->is_adam()) M->v2.assign(d, 0);
    if (variant == GA_LAYER) { const int64_t whole[2] = {0, d}; M->set_layers(whole, 1); }
    if (M->is_dana()) {
        M->vw.assign((size_t)n * d, 0);
        M->vsum.assign(d, 0);
    }
    return M;
}

}  // namespace

#define DISPATCH(h, call) ((h)->precision == 32 ? (h)->f->call : (h)->g->call)

extern "C" {

void* gao_create(int64_t d, int n_workers, double lr, double momentum, double beta, int variant,
                 int precision) {
    if (d <= 0 || n_workers <= 0 || (precision != 32 && precision != 64)) return nullptr;
    if (variant < 0 || variant > 10) return nullptr;
    auto* h = new (std::nothrow) Handle{precision, nullptr, nullptr};
    if (!h) return nullptr;
    try {
        if (precision == 32) h->f = make<float>(d, n_workers, lr, momentum, beta, variant);
        else h->g = make<double>(d, n_workers, lr, momentum, beta, variant);
    } catch (...) {
        delete h;
        return nullptr;
    }
    return h;
}

void gao_destroy(void* p) {
    auto* h = (Handle*)p;
    if (!h) return;
    delete h->f;
    delete h->g;
    delete h;
}

void gao_set_c_order(void* p, int c_order) {
    auto* h = (Handle*)p;
    if (h->precision == 32) h->f->c_order = c_order; else h->g->c_order = c_order;
}

// Learning rate eta_k of the coming arrivals; eta_max of the C algorithm stays as created
// (the C algorithm takes the maximal rate as an input of its own, normally the first rate).
void gao_set_lr(void* p, double lr) {
    auto* h = (Handle*)p;
    if (h->precision == 32) h->f->eta = (float)lr; else h->g->eta = (double)(float)lr;
}

void gao_set_nesterov(void* p, int on) {
    auto* h = (Handle*)p;
    if (h->precision == 32) h->f->nesterov = on; else h->g->nesterov = on;
}

void gao_set_weight_decay(void* p, double wd) {
    auto* h = (Handle*)p;
    if (h->precision == 32) h->f->wd = (float)wd; else h->g->wd = (double)(float)wd;
}

void gao_set_eps(void* p, double eps) {
    auto* h = (Handle*)p;
    if (h->precision == 32) h->f->eps = (float)eps; else h->g->eps = eps;
}

void gao_set_params(void* p, const float* theta0) { auto* h = (Handle*)p; DISPATCH(h, set_params(theta0)); }
void gao_pull(void* p, int worker) { auto* h = (Handle*)p; DISPATCH(h, pull(worker)); }
int64_t gao_push(void* p, int worker, const float* grad) { auto* h = (Handle*)p; return DISPATCH(h, push(worker, grad)); }
void gao_gap(void* p, int worker, double* out) { auto* h = (Handle*)p; DISPATCH(h, gap(worker, out)); }
int64_t gao_k_done(void* p) { auto* h = (Handle*)p; return h->precision == 32 ? h->f->k_done : h->g->k_done; }
int64_t gao_iter(void* p, int worker) { auto* h = (Handle*)p; return h->precision == 32 ? h->f->iter[worker] : h->g->iter[worker]; }

void gao_set_state(void* p, const double* th, const double* v, const double* m, const double* saved,
                   const int64_t* iter, int64_t k_done, int64_t k_c, const double* v_workers) {
    auto* h = (Handle*)p;
    DISPATCH(h, set_state(th, v, m, saved, iter, k_done, k_c, v_workers));
}
// Layers of the layer-wise Gap: offsets[0] = 0 < ... < offsets[n] = d. Resets m_p.
int gao_set_layers(void* p, const int64_t* offsets, int n) {
    auto* h = (Handle*)p;
    const int64_t d = h->precision == 32 ? h->f->d : h->g->d;
    if (n < 1 || offsets[0] != 0 || offsets[n] != d) return -1;
    for (int q = 0; q < n; ++q) if (offsets[q + 1] <= offsets[q]) return -1;
    DISPATCH(h, set_layers(offsets, n));
    return 0;
}
// Gap and m_p of every layer at the last arrival.
void gao_layer_state(void* p, double* gaps, double* m_layer) {
    auto* h = (Handle*)p;
    auto copy = [&](auto* M) {
        for (size_t q = 0; q < M->m_layer.size(); ++q) { gaps[q] = M->last_layer_gap[q]; m_layer[q] = (double)M->m_layer[q]; }
    };
    if (h->precision == 32) copy(h->f); else copy(h->g);
}
void gao_set_adam(void* p, double beta2, double adam_eps) {
    auto* h = (Handle*)p;
    if (h->precision == 32) { h->f->beta2 = (float)beta2; h->f->adam_eps = (float)adam_eps; }
    else { h->g->beta2 = (double)(float)beta2; h->g->adam_eps = (double)(float)adam_eps; }
}
void gao_set_dana_sum(void* p, int mode) {
    auto* h = (Handle*)p;
    if (h->precision == 32) h->f->dana_sum = mode; else h->g->dana_sum = mode;
}
int64_t gao_k_c(void* p) { auto* h = (Handle*)p; return h->precision == 32 ? h->f->k_c : h->g->k_c; }

void gao_stats(void* p, double* sum_gap, double* max_gap) {
    auto* h = (Handle*)p;
    *sum_gap = h->precision == 32 ? h->f->last_sum_gap : h->g->last_sum_gap;
    *max_gap = h->precision == 32 ? h->f->last_max_gap : h->g->last_max_gap;
}

// which: 0 theta, 1 v (DANA: sum_j v^j), 2 m, 3 C (derived from m), 4+i saved copy of worker i,
// 100000+i worker i's momentum v^i (DANA), 200000 Adam's second moment (its first is 1).
// Output in double.
int gao_get(void* p, int which, double* out) {
    auto* h = (Handle*)p;
    auto copy = [&](auto* M) -> int {
        const int64_t d = M->d;
        if (which == 0) for (int64_t j = 0; j < d; ++j) out[j] = (double)M->theta[j];
        else if (which == 1 && M->is_dana()) for (int64_t j = 0; j < d; ++j) out[j] = (double)M->vsum[j];
        else if (which >= 100000 && which < 100000 + M->n_workers && M->is_dana())
            for (int64_t j = 0; j < d; ++j) out[j] = (double)M->vw[(size_t)(which - 100000) * d + j];
        else if (which == 200000 && M->is_adam()) for (int64_t j = 0; j < d; ++j) out[j] = (double)M->v2[j];
        else if (which == 1) for (int64_t j = 0; j < d; ++j) out[j] = (double)M->v[j];
        else if (which == 2) for (int64_t j = 0; j < d; ++j) out[j] = (double)M->m[j];
        else if (which == 3) {
            const auto ib = M->k_c > 0 ? M->inv_bias() : 0;
            for (int64_t j = 0; j < d; ++j) out[j] = (double)M->coeff(M->m[j], ib);
        }
        else if (which >= 4 && which < 4 + M->n_workers)
            for (int64_t j = 0; j < d; ++j) out[j] = (double)M->saved[(size_t)(which - 4) * d + j];
        else return -1;
        return 0;
    };
    return h->precision == 32 ? copy(h->f) : copy(h->g);
}

// The saved copy of one worker rounded to fp32: what is "sent" to the worker.
void gao_sent_f32(void* p, int worker, float* out) {
    auto* h = (Handle*)p;
    if (h->precision == 32) {
        std::memcpy(out, &h->f->saved[(size_t)worker * h->f->d], sizeof(float) * h->f->d);
    } else {
        const double* s = &h->g->saved[(size_t)worker * h->g->d];
        for (int64_t j = 0; j < h->g->d; ++j) out[j] = (float)s[j];
    }
}

}  // extern "C"
