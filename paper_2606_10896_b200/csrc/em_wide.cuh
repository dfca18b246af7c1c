// Declarations of the tensor-core path for wide data (128 < D <= 1024), internal.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

namespace fg {

constexpr int WIDE_MAX_D = 1024;
constexpr int WIDE_MAX_K = 4096;
constexpr int64_t WIDE_PIECE = 1 << 17;      // points per pair of launches: capacity of the fp16 planes of Y in scratch
constexpr int WIDE_BATCH = 256;              // points per batch of the second sweep
constexpr int WIDE_TILE = 128;               // points per tile of the first sweep
constexpr int WIDE_MAX_ILL = 2048;           // ill-conditioned components the FP32 kernels evaluate as a sub-mixture
constexpr int WIDE_LL_BLOCKS = 64;           // per-block partial sums of the log-likelihood

struct WidePlan {
    int n_slices;   // ceil(D / 128): slices of 128 dimensions = 256 columns of the planes
    int Dpad;       // n_slices * 128
    int CL;         // ceil(K / 128) component slices
    int Kpad;       // CL * 128
    int R;          // point ranges of the second sweep: its grid is CL * R CTAs
    int pcols;      // columns of a partial block: 2 * Dpad statistics columns + 2 columns of N_k
};

struct WideBuffers {
    float* sd;      // [Dpad] power-of-two scale of a dimension
    float* kap;     // [Dpad] constant added to the squares
    float* gd;      // [Dpad] centre subtracted from points and means
    unsigned char* p_hi;   // [Kpad][2 Dpad] fp16: high parts of the scaled coefficients, k-step interleaved columns
    unsigned char* p_lo;   // the low parts
    float* tk;      // [Kpad] row scale t_k
    float* tkck;    // [Kpad] pairs (t_k, c_k - c_ref); c = -inf for padded, zero-weight and ill-conditioned components
    double* ckd;    // [Kpad] c_k in float64
    double* cref;   // [1] reference constant: the largest finite c_k
    float* illb;    // [Kpad] > 0 for an ill-conditioned component
    int* flags;     // [8]: [0] any ill-conditioned component, [4] how many, [2] slots of the list, [5] slots of its first kind
    int* ill_list;  // [WIDE_MAX_ILL] ascending indices of the ill-conditioned components
    float* mu_c;    // [WIDE_MAX_ILL][D] their means, packed: the sub-mixture the FP32 kernels evaluate exactly
    float* w2_c;    // [WIDE_MAX_ILL][D] their weights (log2 e / 2) / var
    double* c2d_c;  // [WIDE_MAX_ILL] their constants
    double* stats_c;   // [n_ill + 2 n_ill D] their statistics (N_k, S1, S2), accumulated over the pieces of a step
    unsigned char* y_hi;   // [WIDE_PIECE][2 Dpad] fp16
    unsigned char* y_lo;
    double* logz;   // [WIDE_PIECE] log2 Z of the piece's points as sweep 1 finds it (consistent with sweep 2's logits)
    double* logz_x; // [WIDE_PIECE] the same with the two leading terms of every point replaced by their exact values
    float* top;     // [WIDE_PIECE][4] per point: its two largest approximate log2 z - c_ref and their components
    float* partial; // [R * CL][pcols][128] per-CTA partial statistics of the second sweep
    double* llpart; // [WIDE_LL_BLOCKS] partial sums of log Z
};

bool wide_supports(int D, int K);
WidePlan wide_plan(int D, int K, int num_sms);
// flags are cleared, then: scales, coefficient planes, constants; components whose error estimate exceeds cond_limit or
// whose weight pi_k is below min_weight are flagged (flags[4] counts them) and excluded from the tensor passes (c = -inf).
cudaError_t launch_prepare_wide(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                                const WideBuffers& wb, float cond_limit, float min_weight);
// n <= WIDE_PIECE points: X -> the fp16 planes of Y (rows up to the next multiple of 256 are written as zeros).
cudaError_t launch_transform_wide(cudaStream_t s, const float* X, int64_t n, int D, const WideBuffers& wb, int* status);
// The components flagged by launch_prepare_wide: their list (flags[2] = how many), then their rows of the FP32 path's
// derived parameters packed into wb.mu_c / w2_c / c2d_c.
cudaError_t launch_ill_list_wide(cudaStream_t s, int D, int K, const WideBuffers& wb);
cudaError_t launch_ill_gather_wide(cudaStream_t s, int D, int n_ill, const WideBuffers& wb, const float* mu, const float* w2,
                                   const double* c2d);
// wb.logz_x = wb.logz corrected by the exact values of every point's two leading terms (mu, w2, c2d: the FP32 path's
// parameters): the normaliser of the exactly evaluated components and of the log-likelihood.
cudaError_t launch_refine_wide(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                               const double* c2d, const WideBuffers& wb);
// Both wb.logz and wb.logz_x take in the sub-mixture's log2(sum): log2(2^a + 2^logz_ill[i]) (logz_ill may be NULL), and
// wb.llpart += block sums of the exact log Z.
cudaError_t launch_merge_ll_wide(cudaStream_t s, int64_t n, const WideBuffers& wb, const double* logz_ill);
// stats rows of the listed components += wb.stats_c.
cudaError_t launch_ill_scatter_wide(cudaStream_t s, int D, int K, int n_ill, const WideBuffers& wb, double* Nk, double* S1,
                                    double* S2);
// First sweep over the n points whose planes were written: log2 Z per point (over the well-conditioned components) -> wb.logz.
cudaError_t launch_lse_wide(cudaStream_t s, int64_t n, int D, int K, const WideBuffers& wb, int num_sms, int* status);
// Second sweep: responsibilities from wb.logz, statistics accumulated into wb.partial (+=).
cudaError_t launch_em_wide(cudaStream_t s, int64_t n, int D, int K, const WideBuffers& wb, int num_sms, int* status);
// stats += the partial blocks (fixed order, float64, scale / centre / column order undone).
cudaError_t launch_reduce_wide(cudaStream_t s, int D, int K, const WideBuffers& wb, int num_sms, double* Nk, double* S1,
                               double* S2);

}  // namespace fg
