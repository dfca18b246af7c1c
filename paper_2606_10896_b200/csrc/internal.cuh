// Internal declarations of libflashgmm (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/flashgmm.h"

namespace fg {

// Points per super-tile of the two-phase FP32 path: log Z_i of one super-tile lives in a fixed-size scratch buffer,
// so scratch memory is independent of N.
constexpr int64_t SUPER_TILE = 1 << 20;
constexpr int FP32_TILE_P = 64;    // points per CTA tile
constexpr int FP32_TILE_C = 64;    // components per CTA tile
constexpr int FP32_MSTEP_DC = 128; // dimensions per M-step CTA
constexpr int FP32_TARGET_CTAS = 296;
constexpr int LL_SLOTS = 64;       // device slots for log-likelihood values (gmm_fit keeps one per iteration in a ring)

// Status word bits written by device code, read by the host after a synchronising call.
enum : int { ST_BAD_VAR = 1, ST_BAD_PI = 2, ST_NONFINITE = 4, ST_TIMEOUT = 8, ST_ILLCOND = 16, ST_BAD_X = 32 };

struct Fp32Plan {
    int comp_blocks, d_chunks, splits;
    bool wide;      // D > 128: one CTA sweeps all slices of D; partials are float64
};
Fp32Plan fp32_plan(int D, int K);
size_t fp32_partial_floats(int D, int K);   // floats in the per-CTA partial buffer

// ---- FP32 (CUDA-core) path -----------------------------------------------------------------------------------
// g [D] (may be NULL): receives the per-dimension centre of the means (launch_center_fp32), which the kernels below take
cudaError_t launch_prepare_fp32(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                                float* w2, float* c2, double* c2d, float* g, int* status);
cudaError_t launch_center_fp32(cudaStream_t s, int D, int K, const float* mu, float* g);
// log2-domain log Z of n points -> logZ2[n]; per-block float64 partial log-likelihoods -> llpart[ceil(n/64)]
// c2d: the per-component constants in float64; logZ2: float64 (the kernels carry logits in float64 when D > 128)
// g: the per-dimension centre subtracted from points and means before the products are formed (NULL = none; any value
// gives the same mathematics, a centre near the data keeps the fp32 rounding small)
// lower2 (may be NULL; honoured for D > 128 only): per point a lower bound of its final log2 Z known from elsewhere;
// tiles whose terms all lie 2^-40 below it are not evaluated to the end (their terms count as zero).
cudaError_t launch_lse_fp32(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                            const float* w2, const double* c2d, const float* g, double* logZ2, double* llpart,
                            const double* lower2 = nullptr, const int* run_if = nullptr);
// out[i] = ln 2 * logZ2[i]: the per-point log-density in natural units, fp32
cudaError_t launch_logz_out_fp32(cudaStream_t s, const double* logZ2, int64_t n, float* out);
cudaError_t launch_mstep_fp32(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                              const float* w2, const double* c2d, const float* g, const double* logZ2, float* partials,
                              const Fp32Plan& plan, bool early = false, const int* run_if = nullptr);
// early (D > 128 only): skip the tiles in which no responsibility can reach 2^-40 (sub-mixtures of collapsed components)
// run_if (launch_lse_fp32, and launch_mstep_fp32 for D > 128): NULL, or a device flag: the kernel does nothing unless
// run_if[0] != 0 (the partials of a gated-off M-step stay zero).
// run_if: NULL, or a device flag: the kernel does nothing unless run_if[0] != 0.
// gather: NULL, or device row indices: the points are X[gather[0 .. min(n, *gather_count))], and the outputs go to those
// rows of idx / resp (n then bounds the number of gathered points, and sizes the grid).
cudaError_t launch_topm_fp32(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                             const float* w2, const double* c2d, const float* g, int m, int32_t* idx, float* resp,
                             const int* run_if = nullptr, const int32_t* gather = nullptr, const int* gather_count = nullptr);

// ---- shared by all paths -------------------------------------------------------------------------------------
// stats (+)= sum over `splits` partial blocks, fixed order, float64.  Partial layout: [splits][K + 2*K*D] floats,
// each block being (N_k [K], sums of r (x - g) [K*D], sums of r (x - g)^2 [K*D]); float64 instead when
// fp32_plan(D, K).wide.  g [D]: the centre launch_mstep_fp32 was given (NULL = 0); the shift back to S1, S2 is exact.
cudaError_t launch_reduce_partials(cudaStream_t s, int D, int K, int splits, const float* partials, const float* g,
                                   double* Nk, double* S1, double* S2, bool accumulate, const int* run_if = nullptr);
// *ll (+)= sum of llpart[0..n) in a fixed order
cudaError_t launch_reduce_ll(cudaStream_t s, const double* llpart, int64_t n, double* ll, bool accumulate);
// counts (may be NULL): counts[0] += variance entries raised to the floor, counts[1] += components left unchanged
// because N_k < 1e-12 (integer atomics).  skip_status / skip_ll (may be NULL): the kernel writes nothing when
// *skip_status != 0 or *skip_ll is not finite (the step that produced the statistics failed).
cudaError_t launch_finalize(cudaStream_t s, int64_t N, int D, int K, const double* Nk, const double* S1,
                            const double* S2, float var_floor, float* pi, float* mu, float* var, int* counts,
                            const int* skip_status, const double* skip_ll);

cudaError_t launch_finalize_isotropic(cudaStream_t s, int64_t N, int D, int K, const double* Nk, const double* S1,
                                      const double* S2, float var_floor, float* pi, float* mu, float* var, int* counts,
                                      const int* skip_status, const double* skip_ll);

// ---- Fisher vector of one group from its statistics (paper Section 6) ----------------------------------------------
// out[2 * K * D] (device): the means part [K x D], then the standard-deviations part [K x D]
cudaError_t launch_fisher(cudaStream_t s, int64_t T, int D, int K, const double* Nk, const double* S1, const double* S2,
                          const float* pi, const float* mu, const float* var, float* out);

// ---- IVF posting lists from the top-m assignment (paper Sections 4.2-4.3) ---------------------------------------
constexpr int PL_MAX_BLOCKS = 1024;       // the vectors are cut into at most this many contiguous ranges
constexpr int PL_MAX_K = 8192;            // one 32-bit cursor per cluster in shared memory
size_t pl_scratch_bytes(int K);
// offsets[K + 1] (device), items[>= n * max_lists] (device); scratch of pl_scratch_bytes(K) bytes
cudaError_t launch_posting_lists(cudaStream_t s, const int32_t* idx, const float* resp, int64_t n, int m, int K, float tau,
                                 int max_lists, void* scratch, int64_t* offsets, int32_t* items);

// ---- one Lloyd (k-means) iteration: the paper's warm start (Section 4.4 and the warm-start appendix) -----------------------------------------------
size_t km_scratch_bytes(int D, int K);
int64_t* km_offsets(void* scratch);                     // [K + 1] inside the scratch: the posting-list offsets go here
double* km_inertia_k(void* scratch, int D, int K);      // [K] per-cluster inertia, written by launch_kmeans_update
cudaError_t launch_kmeans_unit_params(cudaStream_t s, int D, int K, float* w2, double* c2d);
// pi [K] = 1 / K, var [K x D] = 1: the mixture whose top-1 component is the nearest centroid
cudaError_t launch_kmeans_unit_mixture(cudaStream_t s, int D, int K, float* pi, float* var);
// The same arg-max from a mixture with pi = 1 / K and ONE variance everywhere, the mean spread of the centroids per dimension
// (vd [D]: scratch): the nearest centroid does not depend on that variance, but with it the posteriors are as sharp as
// the clusters are separate, which is what the screening route of the wide tensor path needs.
cudaError_t launch_kmeans_scaled_mixture(cudaStream_t s, int D, int K, const float* centroids, float* pi, float* var, float* vd);
cudaError_t launch_kmeans_update(cudaStream_t s, const float* X, int D, int K, const float* cent_in, const int32_t* items,
                                 void* scratch, float* cent_out, int64_t* counts);

}  // namespace fg
