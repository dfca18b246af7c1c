// Declarations of the tensor-core path (internal).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

namespace fg {

constexpr int TC_BN = 64;            // points per tile
constexpr int TC_FLUSH = 64;         // tiles between flushes of the TMEM accumulators into float64 partials (even)
constexpr float TC_RSCALE = 4096.f;  // responsibilities are scaled by this power of two before the fp16 split
constexpr int TC_PCOLS = 258;        // columns of a partial row: 256 statistics columns + N_k of each softmax group
constexpr int TC_MAX_K = 4096;         // the E+M tile kernel: a group of ceil(K / 128) <= 32 CTAs covers the components
constexpr int TC_ASSIGN_MAX_K = 4096;  // the tensor-core assignment takes up to this many components
constexpr int TC_MAX_ILL = 256;       // ill-conditioned components the tensor-core assignment evaluates exactly for every point
constexpr int64_t TC_YPOINTS = 1 << 19;   // points per launch of the tile kernel: capacity of the fp16 planes of Y in scratch
constexpr size_t TC_YPLANE_BYTES = (size_t)TC_YPOINTS * 512;   // one plane: 256 fp16 values per point

// What the assignment kernels keep of every ill-conditioned component for a cheap first test: its 8 dimensions of largest
// weight (log2 e / (2 var), descending), the mean and the weight there, and its constant.  [dimension slot][component]
struct TcIllCache {
    float mu[8][TC_MAX_ILL], w[8][TC_MAX_ILL], c[TC_MAX_ILL];
    int dim[8][TC_MAX_ILL];
    int k[TC_MAX_ILL];
};

struct TcPlan {
    int CL;     // CTAs per group = ceil(K / 128)
    int Kpad;   // CL * 128
    int Q;      // groups (of CL CTAs) in the persistent grid
    int n_ks;   // k-steps of 8 dimensions
};

struct TcBuffers {
    uint32_t* phi_img;
    unsigned char* plo_img;
    float* tk;
    float* ck;
    float* sd;
    float* kap;
    float* gd;      // [128] per-dimension centre subtracted from points and means (0 for padded dimensions)
    float* illb;
    int* flags;
    double* partial;
    double* llpart;
    void* xg;   // exchange slots of the log-sum-exp, [Q][4][CL][64] x 16 bytes
    void* xl;   // exchange slots of the lower-bound pass
    unsigned char* y_hi;   // [TC_YPOINTS][256] fp16: high parts of Y = [s x | (s x)^2 + kap], k-step interleaved
    unsigned char* y_lo;   // the low parts
    unsigned char* p_hi_rm;   // [Kpad][256] fp16: high parts of the scaled coefficients P / t_k, row-major, same column order as Y
    unsigned char* p_lo_rm;   // the low parts
    float* tkck;              // [Kpad] pairs (t_k, c_k); c_k = -inf for ill-conditioned components
    int* ill_list;            // [Kpad] ascending indices of the ill-conditioned components (flags[2] of them)
    TcIllCache* ill_cache;    // filled by launch_ill_cache_tc
    int* dec_dim;             // [Kpad][8] per ill-conditioned component: its 8 dimensions of largest weight,
    float* dec_w;             // [Kpad][8] the weights there (units of the scaled data)
    float* dec_mu;            // [Kpad][8] and the scaled means
};

bool tc_supports(int D, int K);          // the E+M tile kernel
bool tc_assign_supports(int D, int K);   // the assignment kernels (a superset)
void tc_set_order(int o);   // MMA issue order: 0 = pairs E E M M, 1 = interleaved M(i) E(i+2), 2 = whichever of E(i+2), M(i+1) is ready first (default)
// Time-out test: CTA `silent_rank` of group 0 never publishes its exchange slot for tile 0 (-1: off), and every device-side
// wait gives up after wait_limit_ns (0: the default 2 s).  Process-wide, like tc_set_order.
void tc_set_test_hooks(int silent_rank, unsigned long long wait_limit_ns);
TcPlan tc_plan(int D, int K, int num_sms);
cudaError_t tc_max_clusters(int D, int K, int* out);
cudaError_t launch_prepare_tc(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                              const TcBuffers& tb, float cond_limit, int* status, bool ill_list = false);
// One pass over at most TC_YPOINTS points: X -> the two fp16 planes of Y in scratch (read by the tile kernel through TMA).
// A non-finite value in X raises ST_BAD_X in *status (the planes themselves are clamped to a finite range).
cudaError_t launch_transform_tc(cudaStream_t s, const float* X, int64_t n, int D, const TcBuffers& tb, int* status);
// n <= TC_YPOINTS points whose planes launch_transform_tc has written.
// mu, w2, c2: the FP32 path's derived parameters (launch_prepare_fp32), used to recompute ill-conditioned logits exactly.
// tight: use the filter meant for launches in which many components are ill-conditioned (tb.flags[4] counts them).
cudaError_t launch_em_tc(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                         const float* c2, const TcBuffers& tb, int Q, int flush_tiles, bool tight, int* status,
                         const int* tile_valid = nullptr, const int64_t* tile_src = nullptr);
// Grouped launches: CTA group b of a launch with Q = `groups` takes the tiles b, b + Q, b + 2 Q, ... of the planes, so a
// plane layout in which those tiles hold the points of one group of the caller (an image's descriptors, say) leaves that
// group's statistics in partial[b].  tile_valid[t] (0 .. TC_BN) = points of tile t, tile_src[t] = their first row in X
// (device arrays, rows / TC_BN entries); launch_em_tc then gets n = rows and the same two arrays.
cudaError_t launch_transform_grouped_tc(cudaStream_t s, const float* X, int64_t rows, int D, const int* tile_valid,
                                        const int64_t* tile_src, const TcBuffers& tb, int* status);
// After a grouped launch_em_tc: Fisher vector of group b (its T = group_points[b]) into fv[out_index[b]][2][K][D].
cudaError_t launch_fisher_tc(cudaStream_t s, int D, int K, int groups, const TcBuffers& tb, const float* pi, const float* mu,
                             const float* var, const int* out_index, const int64_t* group_points, float* fv);
// After launch_prepare_tc(..., ill_list = true): fills tb.ill_cache for the first min(flags[2], TC_MAX_ILL) listed components.
// w2, c2: the FP32 path's derived parameters (launch_prepare_fp32).
cudaError_t launch_ill_cache_tc(cudaStream_t s, int D, const float* mu, const float* w2, const float* c2, const TcBuffers& tb);
// Tensor map of a plane [rows][256 halves] (Y or P): boxes of (one 128-byte atom row, box_rows rows, box_atoms atoms).
cudaError_t tc_make_plane_map(CUtensorMap* tm, void* base, int64_t rows, int box_rows, int box_atoms);
// Top-m assignment of n <= TC_YPOINTS points whose planes launch_transform_tc has written (tensor-core selection of
// candidates + exact refinement).  rec: n * assign_tc_record_bytes(m) bytes of device scratch.  Needs launch_prepare_tc
// with ill_list = true.  Both kernels return at once when tb.flags[3] != 0 (more than TC_MAX_ILL ill-conditioned
// components): the caller then runs the FP32 kernels, gated the other way.
size_t assign_tc_record_bytes(int m);
// unc_rows / unc_count [1]: the rows whose result is not certain (not written to idx / resp) are appended as row +
// row_offset at position (*unc_count)++ (the caller zeroes the count and may let several pieces share one list): the
// caller runs launch_topm_fp32 over them (gather mode).
cudaError_t launch_assign_tc(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                             const float* c2, const TcBuffers& tb, float* rec, int32_t* unc_rows, int* unc_count, int row_offset,
                             int m, int32_t* idx, float* resp, int* status, bool index_only = false);
// index_only (with m = 1): the caller uses idx alone; resp is then only approximate.
cudaError_t launch_reduce_tc(cudaStream_t s, int D, int K, int Q, const TcBuffers& tb, double* Nk, double* S1,
                             double* S2, bool accumulate);

}  // namespace fg
