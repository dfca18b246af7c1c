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
    int* flags;     // [8]: [0] any ill-conditioned component, [4] how many
    unsigned char* y_hi;   // [WIDE_PIECE][2 Dpad] fp16
    unsigned char* y_lo;
    double* logz;   // [WIDE_PIECE] log2 Z of the piece's points
    float* partial; // [R * CL][pcols][128] per-CTA partial statistics of the second sweep
    double* llpart; // [grid of the first sweep] per-CTA sums of log2 Z
};

bool wide_supports(int D, int K);
WidePlan wide_plan(int D, int K, int num_sms);
// flags are cleared, then: scales, coefficient planes, constants; components whose error estimate exceeds cond_limit
// are flagged (flags[4] counts them) and excluded from the tensor passes (c = -inf).
cudaError_t launch_prepare_wide(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                                const WideBuffers& wb, float cond_limit);
// n <= WIDE_PIECE points: X -> the fp16 planes of Y (rows up to the next multiple of 256 are written as zeros).
cudaError_t launch_transform_wide(cudaStream_t s, const float* X, int64_t n, int D, const WideBuffers& wb, int* status);
// First sweep over the n points whose planes were written: log2 Z per point -> wb.logz, per-CTA sums -> wb.llpart (+=).
cudaError_t launch_lse_wide(cudaStream_t s, int64_t n, int D, int K, const WideBuffers& wb, int num_sms, int* status);
// Second sweep: responsibilities from wb.logz, statistics accumulated into wb.partial (+=).
cudaError_t launch_em_wide(cudaStream_t s, int64_t n, int D, int K, const WideBuffers& wb, int num_sms, int* status);
// stats += the partial blocks (fixed order, float64, scale / centre / column order undone).
cudaError_t launch_reduce_wide(cudaStream_t s, int D, int K, const WideBuffers& wb, int num_sms, double* Nk, double* S1,
                               double* S2);

}  // namespace fg
