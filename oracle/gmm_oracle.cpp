// gmm_oracle.cpp -- float64 CPU oracle for one EM iteration of a diagonal-covariance Gaussian mixture.
//
// TEST INFRASTRUCTURE ONLY.  Nothing on the product path may include, link or call this file; it shares no code,
// header, table or helper with the CUDA library.  Only the tests, the smoke check and the benchmark's cpu_baseline /
// reference legs use it.
//
// Every function is the plain definition written out, in the order and notation of the paper:
//   density and log-likelihood ........ Section 2 (mixture density, log p(X|Theta))
//   responsibilities .................. Section 2 (z_ik = pi_k N_ik, r_ik = z_ik / sum_j z_ij), log-sum-exp remark
//   N_k, pi_k, mu_k, sigma_k^2 ........ Eq. 1, the pi_k = N_k / N line, Eq. 2, Eq. 3
//   per-tile accumulators ............. Section 3.1 / Algorithm 1 (N_k(t), M_k(t)); here one "tile" per thread
// The paper's model is isotropic (sigma_k^2 I).  This oracle is the diagonal generalisation: sigma^2 is K x D and
// Eq. 3 is taken per dimension (no 1/D average).  With sigma^2_kd constant over d it reduces to the paper's density,
// and the mean over d of the per-dimension update is Eq. 3 (both are pinned by tests).
//
// Readings where the paper is silent or inconsistent:
//   * variance uses the NEW mean (Eq. 3 read as standard EM), not the old mean that Algorithm 1's Q_k would imply;
//   * pi_k = N_k / N (Section 2), not N_k / sum N_k' (Algorithm 1's last line) -- equal when sum_k N_k = N;
//   * variance floor: sigma^2 = max(estimate, floor);
//   * a component with N_k < 1e-12 keeps its mu and sigma^2, pi_k = N_k / N;
//   * log-likelihood is the TOTAL sum_i log sum_k z_ik under the parameters that enter the step, with the
//     -(D/2) log(2 pi) constant included.
//
// No blocking, fusion or reordering beyond "threads split the points into contiguous ranges and their partial sums
// are added in thread order".  All arithmetic is double.  X is float32 storage (the values the GPU sees), widened.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

const double LOG_2PI = 1.8378770664093454835606594728112;

int clamp_threads(int nthreads) {
#ifdef _OPENMP
    int mx = omp_get_max_threads();
    if (nthreads <= 0 || nthreads > mx) nthreads = mx;
    return nthreads < 1 ? 1 : nthreads;
#else
    (void)nthreads;
    return 1;
#endif
}

// Per-component constants of the log-density, computed once per call (they do not depend on the point):
//   log pi_k, sum_d log var_kd, and 1/var_kd.
struct Prepared {
    std::vector<double> log_pi, log_det, inv_var;
    Prepared(int D, int K, const double* pi, const double* var) : log_pi(K), log_det(K), inv_var((size_t)K * D) {
        for (int k = 0; k < K; ++k) {
            log_pi[k] = (pi[k] > 0.0) ? std::log(pi[k]) : -std::numeric_limits<double>::infinity();
            double s = 0.0;
            for (int d = 0; d < D; ++d) {
                s += std::log(var[(size_t)k * D + d]);
                inv_var[(size_t)k * D + d] = 1.0 / var[(size_t)k * D + d];
            }
            log_det[k] = s;
        }
    }
};

// log z_ik = log pi_k + log N(x_i | mu_k, diag(var_k))          (Section 2, density; direct quadratic form)
//          = log pi_k - 1/2 [ sum_d (x_id - mu_kd)^2 / var_kd + sum_d log var_kd + D log(2 pi) ]
inline double log_joint(const float* x, int D, int k, const Prepared& pre, const double* mu_k) {
    const double* iv = pre.inv_var.data() + (size_t)k * D;
    double q = 0.0;
    for (int d = 0; d < D; ++d) {
        double diff = (double)x[d] - mu_k[d];
        q += diff * diff * iv[d];
    }
    return pre.log_pi[k] - 0.5 * (q + pre.log_det[k] + D * LOG_2PI);
}

// Responsibilities of one point (Section 2, log-space with the log-sum-exp shift).  Returns log Z_i.
double point_responsibilities(const float* x, int D, int K, const Prepared& pre, const double* mu,
                              double* ell /*K scratch*/, double* r /*K out*/) {
    double m = -std::numeric_limits<double>::infinity();
    for (int k = 0; k < K; ++k) {
        ell[k] = log_joint(x, D, k, pre, mu + (size_t)k * D);
        if (ell[k] > m) m = ell[k];
    }
    double s = 0.0;
    for (int k = 0; k < K; ++k) s += std::exp(ell[k] - m);     // exp(-inf) = 0 for pi_k = 0
    double logZ = m + std::log(s);
    for (int k = 0; k < K; ++k) r[k] = std::exp(ell[k] - logZ);
    return logZ;
}

}  // namespace

extern "C" {

int oracle_num_threads(void) { return clamp_threads(0); }

// ell[i*K + k] = log z_ik.  Small inputs only (N*K doubles).
int oracle_log_joint(const float* X, int64_t N, int D, int K, const double* pi, const double* mu, const double* var,
                     double* ell) {
    const Prepared pre(D, K, pi, var);
    for (int64_t i = 0; i < N; ++i)
        for (int k = 0; k < K; ++k) ell[i * K + k] = log_joint(X + i * D, D, k, pre, mu + (size_t)k * D);
    return 0;
}

// R[i*K + k] = r_ik, logZ[i] = log sum_k z_ik.  Small inputs only.
int oracle_responsibilities(const float* X, int64_t N, int D, int K, const double* pi, const double* mu,
                            const double* var, double* R, double* logZ) {
    const Prepared pre(D, K, pi, var);
    std::vector<double> ell(K);
    for (int64_t i = 0; i < N; ++i) {
        double lz = point_responsibilities(X + i * D, D, K, pre, mu, ell.data(), R + i * K);
        if (logZ) logZ[i] = lz;
    }
    return 0;
}

// "Dumbest possible" evaluator for tiny inputs: linear-space product of D univariate normal pdfs, plain
// normalisation, no logarithms of sums, no shift.  R[i*K+k] and p[i] = sum_k z_ik (the mixture density).
int oracle_brute_force(const float* X, int64_t N, int D, int K, const double* pi, const double* mu,
                       const double* var, double* R, double* p) {
    const double PI = 3.14159265358979323846264338327950288;
    for (int64_t i = 0; i < N; ++i) {
        double tot = 0.0;
        for (int k = 0; k < K; ++k) {
            double z = pi[k];
            for (int d = 0; d < D; ++d) {
                double v = var[(size_t)k * D + d];
                double diff = (double)X[i * D + d] - mu[(size_t)k * D + d];
                z *= std::exp(-diff * diff / (2.0 * v)) / std::sqrt(2.0 * PI * v);
            }
            R[i * K + k] = z;
            tot += z;
        }
        for (int k = 0; k < K; ++k) R[i * K + k] /= tot;
        if (p) p[i] = tot;
    }
    return 0;
}

// E-step + sufficient statistics under the INPUT parameters:
//   N_k = sum_i r_ik (Eq. 1), S1_kd = sum_i r_ik x_id (numerator of Eq. 2), S2_kd = sum_i r_ik x_id^2,
//   loglik = sum_i log Z_i (Section 2).
int oracle_em_step(const float* X, int64_t N, int D, int K, const double* pi, const double* mu, const double* var,
                   double* Nk, double* S1, double* S2, double* loglik, int nthreads) {
    if (!X || !pi || !mu || !var || !Nk || !S1 || !S2 || !loglik || N < 1 || D < 1 || K < 1) return -1;
    const int T = clamp_threads(nthreads);
    const size_t KD = (size_t)K * D;
    const Prepared pre(D, K, pi, var);
    std::vector<std::vector<double>> pNk(T), pS1(T), pS2(T);
    std::vector<double> pL(T, 0.0);
#pragma omp parallel num_threads(T)
    {
#ifdef _OPENMP
        const int t = omp_get_thread_num();
#else
        const int t = 0;
#endif
        pNk[t].assign(K, 0.0);
        pS1[t].assign(KD, 0.0);
        pS2[t].assign(KD, 0.0);
        std::vector<double> ell(K), r(K);
        const int64_t lo = N * t / T, hi = N * (t + 1) / T;
        double L = 0.0;
        for (int64_t i = lo; i < hi; ++i) {
            const float* x = X + i * D;
            L += point_responsibilities(x, D, K, pre, mu, ell.data(), r.data());
            for (int k = 0; k < K; ++k) {
                const double rk = r[k];
                if (rk == 0.0) continue;           // adds exact zeros only
                pNk[t][k] += rk;
                double* s1 = pS1[t].data() + (size_t)k * D;
                double* s2 = pS2[t].data() + (size_t)k * D;
                for (int d = 0; d < D; ++d) {
                    const double xd = (double)x[d];
                    s1[d] += rk * xd;
                    s2[d] += rk * xd * xd;
                }
            }
        }
        pL[t] = L;
    }
    std::fill(Nk, Nk + K, 0.0);
    std::fill(S1, S1 + KD, 0.0);
    std::fill(S2, S2 + KD, 0.0);
    double L = 0.0;
    for (int t = 0; t < T; ++t) {                   // fixed thread order
        for (int k = 0; k < K; ++k) Nk[k] += pNk[t][k];
        for (size_t j = 0; j < KD; ++j) { S1[j] += pS1[t][j]; S2[j] += pS2[t][j]; }
        L += pL[t];
    }
    *loglik = L;
    return 0;
}

// Parameter update from the moments:  pi_k = N_k/N, mu = S1/N_k, var = max(S2/N_k - mu^2, floor).
// Algebraically equal to Eq. 3 per dimension with the new mean; used to cross-check the centred form below and as
// the finalize definition when only statistics are available.  mu/var are in/out (kept for empty components).
int oracle_finalize_moments(int64_t N, int D, int K, const double* Nk, const double* S1, const double* S2,
                            double var_floor, double* pi, double* mu, double* var) {
    for (int k = 0; k < K; ++k) {
        pi[k] = Nk[k] / (double)N;
        if (Nk[k] < 1e-12) continue;
        for (int d = 0; d < D; ++d) {
            const size_t j = (size_t)k * D + d;
            const double m = S1[j] / Nk[k];
            mu[j] = m;
            var[j] = std::max(S2[j] / Nk[k] - m * m, var_floor);
        }
    }
    return 0;
}

// One full EM iteration, written as the definition: E-step, then Eq. 1, pi_k = N_k/N, Eq. 2, and Eq. 3 per
// dimension in its centred form sum_i r_ik (x_id - mu_kd^new)^2 / N_k (a second pass over the data with the
// responsibilities recomputed from the OLD parameters).  pi/mu/var are in (old) / out (new).  Optional outputs
// Nk, S1 (may be null).  loglik is under the OLD parameters.
int oracle_em_iteration(const float* X, int64_t N, int D, int K, double* pi, double* mu, double* var,
                        double var_floor, double* loglik, double* Nk_out, double* S1_out, int nthreads) {
    if (!X || !pi || !mu || !var || !loglik || N < 1 || D < 1 || K < 1) return -1;
    const size_t KD = (size_t)K * D;
    std::vector<double> Nk(K), S1(KD), S2(KD);
    int rc = oracle_em_step(X, N, D, K, pi, mu, var, Nk.data(), S1.data(), S2.data(), loglik, nthreads);
    if (rc) return rc;
    std::vector<double> mu_new(mu, mu + KD);
    for (int k = 0; k < K; ++k) {
        if (Nk[k] < 1e-12) continue;
        for (int d = 0; d < D; ++d) mu_new[(size_t)k * D + d] = S1[(size_t)k * D + d] / Nk[k];      // Eq. 2
    }
    // second pass: Q_kd = sum_i r_ik (x_id - mu_new_kd)^2 with r from the old parameters
    const int T = clamp_threads(nthreads);
    const Prepared pre(D, K, pi, var);          // OLD parameters: pi and var are not modified until the end
    std::vector<std::vector<double>> pQ(T);
#pragma omp parallel num_threads(T)
    {
#ifdef _OPENMP
        const int t = omp_get_thread_num();
#else
        const int t = 0;
#endif
        pQ[t].assign(KD, 0.0);
        std::vector<double> ell(K), r(K);
        const int64_t lo = N * t / T, hi = N * (t + 1) / T;
        for (int64_t i = lo; i < hi; ++i) {
            const float* x = X + i * D;
            point_responsibilities(x, D, K, pre, mu, ell.data(), r.data());
            for (int k = 0; k < K; ++k) {
                const double rk = r[k];
                if (rk == 0.0) continue;
                double* q = pQ[t].data() + (size_t)k * D;
                const double* m = mu_new.data() + (size_t)k * D;
                for (int d = 0; d < D; ++d) {
                    const double diff = (double)x[d] - m[d];
                    q[d] += rk * diff * diff;
                }
            }
        }
    }
    std::vector<double> Q(KD, 0.0);
    for (int t = 0; t < T; ++t)
        for (size_t j = 0; j < KD; ++j) Q[j] += pQ[t][j];
    for (int k = 0; k < K; ++k) {
        pi[k] = Nk[k] / (double)N;                                                                 // pi_k = N_k / N
        if (Nk[k] < 1e-12) continue;                                                               // frozen component
        for (int d = 0; d < D; ++d) {
            const size_t j = (size_t)k * D + d;
            mu[j] = mu_new[j];
            var[j] = std::max(Q[j] / Nk[k], var_floor);                                            // Eq. 3 per dim
        }
    }
    if (Nk_out) std::memcpy(Nk_out, Nk.data(), K * sizeof(double));
    if (S1_out) std::memcpy(S1_out, S1.data(), KD * sizeof(double));
    return 0;
}

// The paper's own model: isotropic covariance sigma_k^2 I.  One EM iteration exactly as Section 2 states it: E-step,
// Eq. 1, pi_k = N_k / N, Eq. 2, and Eq. 3  sigma_k^2 = (1 / (D N_k)) sum_i r_ik ||x_i - mu_k^new||^2  (new mean; second pass
// with the responsibilities recomputed from the OLD parameters).  var holds one value per component replicated over d
// (so the same E-step code evaluates N(x | mu_k, sigma_k^2 I)); it is in (old) / out (new).
int oracle_em_iteration_isotropic(const float* X, int64_t N, int D, int K, double* pi, double* mu, double* var,
                                  double var_floor, double* loglik, int nthreads) {
    if (!X || !pi || !mu || !var || !loglik || N < 1 || D < 1 || K < 1) return -1;
    const size_t KD = (size_t)K * D;
    std::vector<double> Nk(K), S1(KD), S2(KD);
    int rc = oracle_em_step(X, N, D, K, pi, mu, var, Nk.data(), S1.data(), S2.data(), loglik, nthreads);
    if (rc) return rc;
    std::vector<double> mu_new(mu, mu + KD);
    for (int k = 0; k < K; ++k) {
        if (Nk[k] < 1e-12) continue;
        for (int d = 0; d < D; ++d) mu_new[(size_t)k * D + d] = S1[(size_t)k * D + d] / Nk[k];      // Eq. 2
    }
    const int T = clamp_threads(nthreads);
    const Prepared pre(D, K, pi, var);
    std::vector<std::vector<double>> pQ(T);
#pragma omp parallel num_threads(T)
    {
#ifdef _OPENMP
        const int t = omp_get_thread_num();
#else
        const int t = 0;
#endif
        pQ[t].assign(K, 0.0);
        std::vector<double> ell(K), r(K);
        const int64_t lo = N * t / T, hi = N * (t + 1) / T;
        for (int64_t i = lo; i < hi; ++i) {
            const float* x = X + i * D;
            point_responsibilities(x, D, K, pre, mu, ell.data(), r.data());
            for (int k = 0; k < K; ++k) {
                if (r[k] == 0.0) continue;
                const double* m = mu_new.data() + (size_t)k * D;
                double sq = 0.0;
                for (int d = 0; d < D; ++d) {
                    const double diff = (double)x[d] - m[d];
                    sq += diff * diff;
                }
                pQ[t][k] += r[k] * sq;                                                              // r_ik ||x_i - mu_k||^2
            }
        }
    }
    for (int k = 0; k < K; ++k) {
        pi[k] = Nk[k] / (double)N;
        if (Nk[k] < 1e-12) continue;
        double Q = 0.0;
        for (int t = 0; t < T; ++t) Q += pQ[t][k];
        const double v = std::max(Q / ((double)D * Nk[k]), var_floor);                              // Eq. 3
        for (int d = 0; d < D; ++d) {
            mu[(size_t)k * D + d] = mu_new[(size_t)k * D + d];
            var[(size_t)k * D + d] = v;
        }
    }
    return 0;
}

// EM driver: iters iterations from the given parameters (in/out).  trace[t] = log-likelihood under the
// parameters ENTERING iteration t.  If params_trace is non-null it receives the parameters entering each
// iteration, laid out [iters+1][K + 2*K*D] as (pi, mu, var), the last block being the final parameters.
// tol > 0: stop after iteration t when |L_t - L_{t-1}| <= tol * |L_t| (Section 2's stopping rule).
int oracle_fit(const float* X, int64_t N, int D, int K, double* pi, double* mu, double* var, int iters,
               double var_floor, double tol, double* trace, int* iters_done, double* params_trace, int nthreads) {
    const size_t KD = (size_t)K * D, P = (size_t)K + 2 * KD;
    int t = 0;
    for (; t < iters; ++t) {
        if (params_trace) {
            double* p = params_trace + (size_t)t * P;
            std::memcpy(p, pi, K * sizeof(double));
            std::memcpy(p + K, mu, KD * sizeof(double));
            std::memcpy(p + K + KD, var, KD * sizeof(double));
        }
        int rc = oracle_em_iteration(X, N, D, K, pi, mu, var, var_floor, trace + t, nullptr, nullptr, nthreads);
        if (rc) return rc;
        if (tol > 0.0 && t > 0 && std::fabs(trace[t] - trace[t - 1]) <= tol * std::fabs(trace[t])) { ++t; break; }
    }
    if (params_trace) {
        double* p = params_trace + (size_t)t * P;
        std::memcpy(p, pi, K * sizeof(double));
        std::memcpy(p + K, mu, KD * sizeof(double));
        std::memcpy(p + K + KD, var, KD * sizeof(double));
    }
    if (iters_done) *iters_done = t;
    return 0;
}

// Top-m components by responsibility for every point (Section 4.2: argmax; Section 4.3: the clusters with the
// largest responsibilities).  idx[i*m + j], resp[i*m + j], descending, ties -> smaller k.  Plain selection:
// repeat m times "take the largest not yet taken".  Also returns the full r row's (m+1)-th value in
// next_resp[i] (0 if m == K) so a caller can tell when the m-th choice is a near-tie.
int oracle_topm(const float* X, int64_t N, int D, int K, const double* pi, const double* mu, const double* var,
                int m, int32_t* idx, double* resp, double* next_resp, int nthreads) {
    if (m < 1 || m > K) return -1;
    const int T = clamp_threads(nthreads);
    const Prepared pre(D, K, pi, var);
#pragma omp parallel num_threads(T)
    {
        std::vector<double> ell(K), r(K);
        std::vector<char> taken(K);
#pragma omp for schedule(static)
        for (int64_t i = 0; i < N; ++i) {
            point_responsibilities(X + i * D, D, K, pre, mu, ell.data(), r.data());
            std::fill(taken.begin(), taken.end(), 0);
            for (int j = 0; j <= m; ++j) {
                int best = -1;
                for (int k = 0; k < K; ++k)
                    if (!taken[k] && (best < 0 || r[k] > r[best])) best = k;
                if (j < m) {
                    taken[best] = 1;
                    idx[i * m + j] = best;
                    resp[i * m + j] = r[best];
                } else if (next_resp) {
                    next_resp[i] = (best >= 0) ? r[best] : 0.0;
                }
            }
        }
    }
    return 0;
}

}  // extern "C"
