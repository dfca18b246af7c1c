// One Lloyd (k-means) iteration: the warm start the paper runs before its EM iterations (Section 4.4, experimental setup, and the warm-start appendix:
// 10 iterations of k-means, then Flash-GMM).
//
// Assignment: the nearest centroid of a point is the top-1 "component" of a mixture with unit variances and equal
// weights (log z = const - sum_d (x - c)^2), so the direct-difference tile kernel of the FP32 path does the search, ties
// to the smaller index.  Update: the posting lists of that assignment (ascending point indices, built without atomics)
// give every cluster its points in a fixed order; a CTA sums the rows of one segment of one list in float64, a second
// kernel adds the segments in order.  No atomics anywhere: the step is reproducible bit for bit.
#include "internal.cuh"

namespace fg {

namespace {

constexpr int KM_THREADS = 128;

__global__ void km_unit_params_kernel(size_t KD, int K, float* __restrict__ w2, double* __restrict__ c2d) {
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < KD) w2[e] = 1.0f;                     // log2 z = 0 - sum_d 1 * (x - c)^2: the largest is the nearest
    if (e < (size_t)K) c2d[e] = 0.0;
}

// grid (K, S): cluster k, segment s of its list.  psum [K][S][D], psq [K][S].
__global__ void __launch_bounds__(KM_THREADS)
km_update_kernel(const float* __restrict__ X, int D, const float* __restrict__ cent, const int64_t* __restrict__ offsets,
                 const int32_t* __restrict__ items, int S, double* __restrict__ psum, double* __restrict__ psq) {
    __shared__ double red[KM_THREADS];
    const int k = blockIdx.x, s = blockIdx.y, tid = threadIdx.x;
    const int64_t lo = offsets[k], cnt = offsets[k + 1] - lo;
    const int64_t seg = (cnt + S - 1) / S;
    const int64_t a = lo + (int64_t)s * seg;
    int64_t b = a + seg;
    if (b > lo + cnt) b = lo + cnt;
    double sq_total = 0.0;
    for (int d0 = 0; d0 < D; d0 += KM_THREADS) {
        const int d = d0 + tid;
        double acc = 0.0, sq = 0.0;
        if (d < D) {
            const double c = (double)__ldg(cent + (size_t)k * D + d);
            for (int64_t it = a; it < b; ++it) {                      // ascending point index: a fixed order
                const double x = (double)__ldg(X + (size_t)__ldg(items + it) * D + d);
                acc += x;
                sq += (x - c) * (x - c);
            }
            psum[((size_t)k * S + s) * D + d] = acc;
        }
        sq_total += sq;
    }
    red[tid] = sq_total;
    __syncthreads();
    for (int o = KM_THREADS / 2; o > 0; o >>= 1) {                    // fixed tree
        if (tid < o) red[tid] += red[tid + o];
        __syncthreads();
    }
    if (tid == 0) psq[(size_t)k * S + s] = red[0];
}

__global__ void __launch_bounds__(KM_THREADS)
km_finish_kernel(int D, int S, const float* __restrict__ cent_in, const int64_t* __restrict__ offsets,
                 const double* __restrict__ psum, const double* __restrict__ psq, float* __restrict__ cent_out,
                 int64_t* __restrict__ counts, double* __restrict__ inertia_k) {
    const int k = blockIdx.x, tid = threadIdx.x;
    const int64_t cnt = offsets[k + 1] - offsets[k];
    for (int d = tid; d < D; d += KM_THREADS) {
        double sum = 0.0;
        for (int s = 0; s < S; ++s) sum += psum[((size_t)k * S + s) * D + d];
        const float old = cent_in[(size_t)k * D + d];
        cent_out[(size_t)k * D + d] = (cnt > 0) ? (float)(sum / (double)cnt) : old;     // an empty cluster stays
    }
    if (tid == 0) {
        double q = 0.0;
        for (int s = 0; s < S; ++s) q += psq[(size_t)k * S + s];
        inertia_k[k] = q;
        if (counts) counts[k] = cnt;
    }
}

}  // namespace

int km_segments(int K) {
    int S = (4 * 148 + K - 1) / K;
    if (S < 1) S = 1;
    if (S > 64) S = 64;
    return S;
}

size_t km_scratch_bytes(int D, int K) {
    const int S = km_segments(K);
    return ((size_t)K * S * D + (size_t)K * S + (size_t)K) * sizeof(double) + (size_t)(K + 1) * sizeof(int64_t);
}

namespace {
__global__ void km_unit_mixture_kernel(size_t KD, int K, float* __restrict__ pi, float* __restrict__ var) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < KD) var[i] = 1.f;
    if (i < (size_t)K) pi[i] = 1.f / (float)K;
}
}  // namespace

namespace {
// Spread of the centroids: vd[d] = variance of centroid coordinate d over the K centroids (float64 sums, fixed order).
__global__ void __launch_bounds__(128) km_spread_kernel(int D, int K, const float* __restrict__ cent, float* __restrict__ vd) {
    __shared__ double r1[128], r2[128];
    const int d = blockIdx.x, t = threadIdx.x;
    double a = 0.0, b = 0.0;
    for (int k = t; k < K; k += 128) {
        const double c = (double)cent[(size_t)k * D + d];
        a += c;
        b += c * c;
    }
    r1[t] = a; r2[t] = b;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (t < o) { r1[t] += r1[t + o]; r2[t] += r2[t + o]; }
        __syncthreads();
    }
    if (t == 0) {
        const double m = r1[0] / K;
        vd[d] = (float)fmax(r2[0] / K - m * m, 0.0);
    }
}
// pi = 1 / K, var = the mean of vd over the dimensions (1 if that is zero or not finite), everywhere.
__global__ void km_scaled_mixture_kernel(size_t KD, int D, int K, const float* __restrict__ vd, float* __restrict__ pi,
                                         float* __restrict__ var) {
    __shared__ float v_s;
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += (double)vd[d];
        const float v = (float)(s / D);
        v_s = (v > 1e-30f && v < 1e30f) ? v : 1.f;
    }
    __syncthreads();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < KD) var[i] = v_s;
    if (i < (size_t)K) pi[i] = 1.f / (float)K;
}
}  // namespace

cudaError_t launch_kmeans_scaled_mixture(cudaStream_t s, int D, int K, const float* centroids, float* pi, float* var, float* vd) {
    km_spread_kernel<<<(unsigned)D, 128, 0, s>>>(D, K, centroids, vd);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t KD = (size_t)K * D;
    km_scaled_mixture_kernel<<<(unsigned)((KD + 255) / 256), 256, 0, s>>>(KD, D, K, vd, pi, var);
    return cudaGetLastError();
}

cudaError_t launch_kmeans_unit_mixture(cudaStream_t s, int D, int K, float* pi, float* var) {
    const size_t KD = (size_t)K * D;
    km_unit_mixture_kernel<<<(unsigned)((KD + 255) / 256), 256, 0, s>>>(KD, K, pi, var);
    return cudaGetLastError();
}

cudaError_t launch_kmeans_unit_params(cudaStream_t s, int D, int K, float* w2, double* c2d) {
    const size_t KD = (size_t)K * D;
    km_unit_params_kernel<<<(unsigned)((KD + 255) / 256), 256, 0, s>>>(KD, K, w2, c2d);
    return cudaGetLastError();
}

// scratch layout: offsets int64 [K + 1] | psum [K][S][D] | psq [K][S] | inertia_k [K]
int64_t* km_offsets(void* scratch) { return static_cast<int64_t*>(scratch); }
double* km_inertia_k(void* scratch, int D, int K) {
    const int S = km_segments(K);
    return reinterpret_cast<double*>(static_cast<unsigned char*>(scratch) + (size_t)(K + 1) * sizeof(int64_t)) + (size_t)K * S * D + (size_t)K * S;
}

cudaError_t launch_kmeans_update(cudaStream_t s, const float* X, int D, int K, const float* cent_in, const int32_t* items,
                                 void* scratch, float* cent_out, int64_t* counts) {
    const int S = km_segments(K);
    const int64_t* offsets = km_offsets(scratch);
    double* psum = reinterpret_cast<double*>(static_cast<unsigned char*>(scratch) + (size_t)(K + 1) * sizeof(int64_t));
    double* psq = psum + (size_t)K * S * D;
    double* ik = psq + (size_t)K * S;
    km_update_kernel<<<dim3((unsigned)K, (unsigned)S), KM_THREADS, 0, s>>>(X, D, cent_in, offsets, items, S, psum, psq);
    km_finish_kernel<<<K, KM_THREADS, 0, s>>>(D, S, cent_in, offsets, psum, psq, cent_out, counts, ik);
    return cudaGetLastError();
}

}  // namespace fg
