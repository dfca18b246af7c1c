// Fisher-vector encoding from the sufficient statistics of one group of points (paper Section 6, Discussion: the fused
// log-sum-exp + responsibility-weighted statistics pattern applied per group instead of once globally).  The tile
// kernels of the EM step produce (N_k, S1 = r^T X, S2 = r^T X^2) of the group; the gradient of the group's mean
// log-likelihood, scaled coordinate-wise by the inverse square root of the diagonal Fisher information, is then
//
//   G_mu[k, d]    = (S1_kd - mu_kd N_k) / (T sigma_kd sqrt(pi_k))
//   G_sigma[k, d] = (S2_kd - 2 mu_kd S1_kd + (mu_kd^2 - sigma_kd^2) N_k) / (T sigma_kd^2 sqrt(2 pi_k))
//
// evaluated in float64 (the differences cancel when the data lie far from the origin in units of sigma).
#include "internal.cuh"

namespace fg {

namespace {

__global__ void fisher_kernel(int64_t T, int D, int K, const double* __restrict__ Nk, const double* __restrict__ S1,
                              const double* __restrict__ S2, const float* __restrict__ pi, const float* __restrict__ mu,
                              const float* __restrict__ var, float* __restrict__ out) {
    const size_t KD = (size_t)K * D;
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    const int k = (int)(e / D);
    const double p = (double)pi[k];
    float gm = 0.f, gs = 0.f;
    if (p > 0.0 && T > 0) {                                   // a component of weight 0 has r = 0 everywhere
        const double nk = Nk[k], m = (double)mu[e], v = (double)var[e];
        const double s1 = S1[e], s2 = S2[e];
        const double t = (double)T;
        gm = (float)((s1 - m * nk) / (t * sqrt(v) * sqrt(p)));
        gs = (float)(((s2 - 2.0 * m * s1) + (m * m - v) * nk) / (t * v * sqrt(2.0 * p)));
    }
    out[e] = gm;
    out[KD + e] = gs;
}

}  // namespace

cudaError_t launch_fisher(cudaStream_t s, int64_t T, int D, int K, const double* Nk, const double* S1, const double* S2,
                          const float* pi, const float* mu, const float* var, float* out) {
    const size_t n = (size_t)K * D;
    fisher_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(T, D, K, Nk, S1, S2, pi, mu, var, out);
    return cudaGetLastError();
}

}  // namespace fg
