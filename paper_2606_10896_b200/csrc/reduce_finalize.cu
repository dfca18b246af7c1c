// Deterministic cross-CTA reduction of the per-CTA partial statistics, log-likelihood reduction, and the parameter
// update (paper Algorithm 1: the atomic accumulation of the per-tile statistics at the end of its Step 2 is replaced by
// per-CTA partials summed in a fixed order in float64; its last line is the finalize kernel, with Eq. 3 taken per
// dimension).
#include "internal.cuh"

namespace fg {

namespace {

// Partials hold N_k and the sums of r (x - g), r (x - g)^2 about the per-dimension centre g (NULL = 0); with
// S1c, S2c their totals over the splits,  S1 = S1c + g N_k,  S2 = S2c + 2 g S1c + g^2 N_k  (float64).
template <typename T>
__global__ void reduce_partials_kernel(int D, int K, int splits, const T* __restrict__ partials,
                                       const float* __restrict__ g, double* __restrict__ Nk, double* __restrict__ S1,
                                       double* __restrict__ S2, int accumulate, const int* __restrict__ run_if) {
    if (run_if && *run_if == 0) return;                  // (the kernel that fills the partials did not run either)
    const size_t KD = (size_t)K * D, per = (size_t)K + 2 * KD;
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= per) return;
    double s = 0.0;
    for (int p = 0; p < splits; ++p) s += (double)partials[(size_t)p * per + e];      // fixed order
    double* dst = (e < (size_t)K) ? (Nk + e) : (e < K + KD) ? (S1 + (e - K)) : (S2 + (e - K - KD));
    if (g && e >= (size_t)K) {
        const size_t j = (e < K + KD) ? (e - K) : (e - K - KD);
        const size_t k = j / D;
        const double gd = (double)g[j % D];
        double nk = 0.0;
        for (int p = 0; p < splits; ++p) nk += (double)partials[(size_t)p * per + k];
        if (e < K + KD) {
            s += gd * nk;
        } else {
            double s1c = 0.0;
            for (int p = 0; p < splits; ++p) s1c += (double)partials[(size_t)p * per + K + j];
            s += 2.0 * gd * s1c + gd * gd * nk;
        }
    }
    *dst = accumulate ? (*dst + s) : s;
}

// One block; thread t sums elements t, t + 256, ... in order, then a fixed-shape tree adds the 256 partials.
__global__ void reduce_ll_kernel(const double* __restrict__ llpart, int64_t n, double* __restrict__ ll,
                                 int accumulate) {
    __shared__ double red[256];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < n; i += 256) s += llpart[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *ll = accumulate ? (*ll + red[0]) : red[0];
}

__global__ void finalize_kernel(int64_t N, int D, int K, const double* __restrict__ Nk, const double* __restrict__ S1,
                                const double* __restrict__ S2, float var_floor, float* __restrict__ pi,
                                float* __restrict__ mu, float* __restrict__ var, int* __restrict__ counts,
                                const int* __restrict__ skip_status, const double* __restrict__ skip_ll) {
    if ((skip_status && *skip_status != 0) || (skip_ll && !isfinite(*skip_ll))) return;      // the step failed: keep the parameters
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (size_t)K * D) return;
    const int k = (int)(e / D);
    const double nk = Nk[k];
    if (e % D == 0) pi[k] = (float)(nk / (double)N);                      // pi_k = N_k / N
    if (nk < 1e-12) {                                                     // empty component keeps mu, var
        if (counts && e % D == 0) atomicAdd(counts + 1, 1);
        return;
    }
    const double m = S1[e] / nk;                                          // Eq. 2
    double v = S2[e] / nk - m * m;                                        // Eq. 3 per dimension, new mean
    const double fl = (double)var_floor;
    if (!(v > fl)) {
        v = fl;
        if (counts) atomicAdd(counts, 1);
    }
    mu[e] = (float)m;
    var[e] = (float)v;
}

// The paper's isotropic model: sigma_k^2 = (1 / (D N_k)) sum_i r_ik ||x_i - mu_k^new||^2 (Eq. 3), which in terms of the
// statistics is (1 / (D N_k)) sum_d (S2_kd - N_k mu_kd^2).  One block per component; the value is written to all D
// entries of var so that every other entry point sees an ordinary diagonal model.
__global__ void finalize_isotropic_kernel(int64_t N, int D, int K, const double* __restrict__ Nk,
                                          const double* __restrict__ S1, const double* __restrict__ S2,
                                          float var_floor, float* __restrict__ pi, float* __restrict__ mu,
                                          float* __restrict__ var, int* __restrict__ counts,
                                          const int* __restrict__ skip_status, const double* __restrict__ skip_ll) {
    if ((skip_status && *skip_status != 0) || (skip_ll && !isfinite(*skip_ll))) return;      // the step failed: keep the parameters
    const int k = blockIdx.x;
    __shared__ double red[128];
    const double nk = Nk[k];
    if (threadIdx.x == 0) pi[k] = (float)(nk / (double)N);
    if (nk < 1e-12) {
        if (counts && threadIdx.x == 0) atomicAdd(counts + 1, 1);
        return;
    }
    double q = 0.0;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        const double m = S1[(size_t)k * D + d] / nk;
        q += S2[(size_t)k * D + d] - nk * m * m;
        mu[(size_t)k * D + d] = (float)m;
    }
    red[threadIdx.x] = q;
    __syncthreads();
    for (int o = blockDim.x / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    double v = red[0] / ((double)D * nk);
    const double fl = (double)var_floor;
    if (!(v > fl)) {
        v = fl;
        if (counts && threadIdx.x == 0) atomicAdd(counts, D);      // all D replicated entries sit at the floor
    }
    for (int d = threadIdx.x; d < D; d += blockDim.x) var[(size_t)k * D + d] = (float)v;
}

}  // namespace

cudaError_t launch_finalize_isotropic(cudaStream_t s, int64_t N, int D, int K, const double* Nk, const double* S1,
                                      const double* S2, float var_floor, float* pi, float* mu, float* var, int* counts,
                                      const int* skip_status, const double* skip_ll) {
    finalize_isotropic_kernel<<<K, 128, 0, s>>>(N, D, K, Nk, S1, S2, var_floor, pi, mu, var, counts, skip_status, skip_ll);
    return cudaGetLastError();
}

cudaError_t launch_reduce_partials(cudaStream_t s, int D, int K, int splits, const float* partials, const float* g,
                                   double* Nk, double* S1, double* S2, bool accumulate, const int* run_if) {
    const size_t per = (size_t)K + 2 * (size_t)K * D;
    const unsigned blocks = (unsigned)((per + 255) / 256);
    if (fp32_plan(D, K).wide)
        reduce_partials_kernel<double><<<blocks, 256, 0, s>>>(D, K, splits, reinterpret_cast<const double*>(partials), g, Nk, S1, S2,
                                                              accumulate ? 1 : 0, run_if);
    else
        reduce_partials_kernel<float><<<blocks, 256, 0, s>>>(D, K, splits, partials, g, Nk, S1, S2, accumulate ? 1 : 0, run_if);
    return cudaGetLastError();
}

cudaError_t launch_reduce_ll(cudaStream_t s, const double* llpart, int64_t n, double* ll, bool accumulate) {
    reduce_ll_kernel<<<1, 256, 0, s>>>(llpart, n, ll, accumulate ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_finalize(cudaStream_t s, int64_t N, int D, int K, const double* Nk, const double* S1,
                            const double* S2, float var_floor, float* pi, float* mu, float* var, int* counts,
                            const int* skip_status, const double* skip_ll) {
    const size_t n = (size_t)K * D;
    finalize_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(N, D, K, Nk, S1, S2, var_floor, pi, mu, var, counts, skip_status, skip_ll);
    return cudaGetLastError();
}

}  // namespace fg
