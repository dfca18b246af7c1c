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
constexpr int WIDE_PAIR_VALS = 32 * (int)WIDE_PIECE; // exact values kept from the pairs' evaluation for their statistics (more marked
                                                // pairs in a piece: the statistics kernel evaluates its pairs again)
constexpr int WIDE_REC = 128;                   // marks of a point whose upper bounds sweep 1 records for the filter (more: they stay)
static_assert(WIDE_MAX_K + 64 <= 8192, "a recorded mark keeps its slot in 13 bits");
constexpr int WIDE_MAX_ILL = WIDE_MAX_K + 64; // slots of the list of components evaluated exactly (all of them may be; + the gap)
constexpr int WIDE_LL_BLOCKS = 64;           // per-block partial sums of the log-likelihood
constexpr int WIDE_MAX_TOP = 10;             // candidates per point sweep 1 can report (the top-m assignment asks for m + 2)
constexpr int WIDE_HEAVY_SLOTS = 128, WIDE_HEAVY_SEG = 16;    // see wide_cand_mstep_kernel
constexpr int WIDE_CAND_WORDS = (WIDE_MAX_ILL + 31) / 32;   // 32-bit words of a point's row of the candidate bitmap, at most
constexpr int WIDE_CANDT_WORDS = (int)(WIDE_PIECE / 32);    // words of a slot's row of the transposed bitmap

struct WidePlan {
    int n_slices;   // ceil(D / 128): slices of 128 dimensions = 256 columns of the planes
    int Dpad;       // n_slices * 128
    int CL;         // ceil(K / 128) component slices
    int Kpad;       // CL * 128
    int rows;       // Kpad + 256: rows of the coefficient planes and of the per-position arrays (the listed components sit
                    // behind the evaluated ones, from the next multiple of 256 on)
    int R;          // point ranges of the second sweep: its grid is CL * R CTAs
    int pcols;      // columns of a partial block: 2 * Dpad statistics columns + 2 columns of N_k
};

struct WideBuffers {
    float* sd;      // [Dpad] power-of-two scale of a dimension
    float* kap;     // [Dpad] constant added to the squares
    float* gd;      // [Dpad] centre subtracted from points and means
    // Arrays "by position": the tensor passes see the components in the order comp_of gives (evaluated ones first).
    unsigned char* p_hi;   // [rows][2 Dpad] fp16: high parts of the scaled coefficients, k-step interleaved columns
    unsigned char* p_lo;   // the low parts
    float* tk;      // [rows] row scale t
    float* tkck;    // [rows] pairs (t, c - c_ref); c = -inf for empty positions, zero-weight and listed components
    double* ckd;    // [rows] c in float64
    double* cref;   // [1] reference constant: the largest finite c of the evaluated components
    int* comp_of;   // [rows] component at a position, -1 for none
    float* illb;    // [Kpad] by component: > 0 for an ill-conditioned one
    float* scra;    // [Kpad] by component: bound of the error of its approximate log2 z at the centre ...
    float* scrw;    // [Kpad] ... and per unit of |x - g|^2
    float* scra_hi; // [Kpad] the same two for the leading product alone (low halves of the operands dropped)
    float* scrw_hi;
    int* flags;     // [8]: [0] any ill-conditioned component, [4] how many, [2] slots of the list, [5] slots of its first
                    //      kind, [6] evaluated components (positions [0, flags[6])); [1], [3], [7]: see launch_cand_count_wide
    int* ill_list;  // [WIDE_MAX_ILL] ascending indices of the ill-conditioned components
    float* mu_c;    // [WIDE_MAX_ILL][D] their means, packed: the sub-mixture the FP32 kernels evaluate exactly
    float* w2_c;    // [WIDE_MAX_ILL][D] their weights (log2 e / 2) / var
    double* c2d_c;  // [WIDE_MAX_ILL] their constants
    double* stats_c;   // [n_ill + 2 n_ill D] their statistics (N_k, S1, S2), accumulated over the pieces of a step
    unsigned char* y_hi;   // [WIDE_PIECE][2 Dpad] fp16
    unsigned char* y_lo;
    double* logz;   // [WIDE_PIECE] log2 Z of the piece's points as sweep 1 finds it (consistent with sweep 2's logits)
    double* logz_x; // [WIDE_PIECE] the same with the two leading terms of every point replaced by their exact values
    float* top;     // [WIDE_PIECE][2 WIDE_MAX_TOP] per point: its largest approximate log2 z - c_ref, then their positions
                    // (rows of 2 ntop floats for the ntop of the launch)
    float* partial; // [R * CL][pcols][128] per-CTA partial statistics of the second sweep
    double* llpart; // [WIDE_LL_BLOCKS] partial sums of log Z
    // Screening of the (point, ill-conditioned component) pairs by sweep 1 and their exact evaluation pair by pair:
    float* scr;     // [rows] pairs.  Listed components: (c - c_ref + error allowance, allowance per unit of |x - g|^2);
                    // evaluated components: (error allowance, allowance per unit of |x - g|^2); (-inf, 0) elsewhere
    float* scr_e;   // [rows] listed components: the error allowance alone (what scr's first entry adds to c - c_ref)
    int* slot_of;   // [rows] slot in the list of the component at a position, -1 if it is not listed
    int* scr_mask;  // [rows / 32] nonzero where a chunk of 32 positions holds a listed component
    float* n2;      // [WIDE_PIECE] |x_i - g|^2
    unsigned* cand; // [WIDE_PIECE][words] bit (i, slot): the pair may matter (set by sweep 1)
    unsigned* candT;// [WIDE_MAX_ILL][WIDE_CANDT_WORDS] bit (slot, i): the pair matters (set by the exact evaluation)
    int* slot_cnt;  // [slots] pairs kept per slot in the current piece
    int* heavy_of;  // [slots] index of a slot's partial sums when its points are split over several blocks, else -1
    int* heavy_slot;// [WIDE_HEAVY_SLOTS] the slot of each set of partial sums, -1 if unused
    double* heavy_part;    // [WIDE_HEAVY_SLOTS][WIDE_HEAVY_SEG][1 + 2 D] partial (N_k, S1, S2) of the split slots' segments
    unsigned* rec;     // [WIDE_PIECE][WIDE_REC] sweep 1's marks of a point: upper bound (rounded up to 19 bits) | slot (13 bits)
    int* rec_cnt;      // [WIDE_PIECE][2] how many in each half of a point's record (one half per softmax warpgroup; a count may
                       // exceed the half's WIDE_REC / 2 entries: the rest was not recorded)
    float* rec_thr;    // [WIDE_PIECE] the point's final screening threshold (before the 2^-40 margin)
    float* pair_val;   // [WIDE_PAIR_VALS] exact log2 z of a piece's kept pairs relative to the point's best value, a point's
                       // marked pairs consecutive and in slot order (positions from a counter: ctl[4])
    int* pair_off;     // [WIDE_PIECE] where a point's values start
    double* pair_best; // [WIDE_PIECE] the point's best value (the reference of its pair_val entries)
    unsigned short* pair_key8; // [WIDE_PIECE][8] the slots of a point's first eight marked pairs (0xFFFF: not kept), and
    float* pair_val8;          // [WIDE_PIECE][8] their values: what the statistics kernel finds in one read
    int* ctl;       // [8]: [0] pairs sweep 1 let through (less what the filter took out again), [1] nonzero: too many, the
                    //      FP32 kernels evaluate the sub-mixture densely, [2] nonzero: the pairs are evaluated one by one,
                    //      [4] entries of pair_val handed out, [5] nonzero: pair_val ran out (the statistics kernel evaluates
                    //      its pairs itself)
};

bool wide_supports(int D, int K);
WidePlan wide_plan(int D, int K, int num_sms);
// flags are cleared, then: scales; components whose error estimate exceeds cond_limit or whose weight pi_k is below
// min_weight are flagged (flags[4] counts them), listed (flags[2], flags[5]) and placed behind the others (flags[6] =
// how many the tensor passes evaluate); coefficient planes and constants by position.
cudaError_t launch_prepare_wide(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                                const WideBuffers& wb, float cond_limit, float min_weight, int hi_mode = 0);
// hi_mode 1 (only with every component listed): the groups of 256 positions behind the first kind of listed components
// get the allowances of the leading product alone; launch_lse_wide must then be given hi_first_slots = flags[5].
// hi_mode 2 (the assignment): the evaluated components get them; launch_lse_wide (ntop > 2) is given hi_first_slots = 0
// and launch_assign_refine_wide hi = true.
// n <= WIDE_PIECE points: X -> the fp16 planes of Y (rows up to the next multiple of 256 are written as zeros).
cudaError_t launch_transform_wide(cudaStream_t s, const float* X, int64_t n, int D, const WideBuffers& wb, int* status,
                                  bool hi_only = false, bool with_norm = false);
// hi_only: the lo plane is not written (a sweep of leading products follows); with_norm: wb.n2[i] = |x_i - g|^2 of the piece's
// points as well (what a screening sweep's bounds need; a warp per point, fixed order of additions).
// The listed components' rows of the FP32 path's derived parameters packed into wb.mu_c / w2_c / c2d_c.
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
// wb.flags[1] += wb.ctl[0] (pairs marked), wb.flags[3] += the sum of wb.slot_cnt (pairs kept), wb.flags[7] += 1 if the piece went through
// the dense kernels: totals of a step, for diagnostics.
cudaError_t launch_cand_count_wide(cudaStream_t s, int n_slots, const WideBuffers& wb);
// First sweep over the n points whose planes were written: log2 Z per point over the Kg evaluated components -> wb.logz.
// n_listed > 0 (listed components, n_slots slots of the list): the sweep also marks in wb.cand every pair of a point and a
// listed component whose approximate log2 z, raised by its error bound, comes within 2^-40 of the point's maximum, and
// counts the marks in wb.ctl[0]; wb.n2, wb.cand (zeroed) and wb.ctl (zeroed) must have been prepared for the piece.
// ntop (2, 6 or WIDE_MAX_TOP): how many of a point's largest approximate values go to wb.top.
// hi_first_slots >= 0 (with parameters prepared in hi_mode): the slots of the list's first kind (flags[5]); the groups of
// 256 positions behind them are screened by the leading product alone.
cudaError_t launch_lse_wide(cudaStream_t s, int64_t n, int D, int K, int Kg, int n_listed, int n_slots, const WideBuffers& wb,
                            int num_sms, int* status, int ntop = 2, int hi_first_slots = -1, bool pre_pass = false,
                            bool record = false, bool listed_only = false, int topm = 0);
// topm > 0 (ntop = 6 or 10, listed_only, hi_first_slots = 0; the top-m assignment by screening): wb.top[i] also reports the
// ntop blocks of 32 listed components with the largest upper bounds at point i (the bound, and the position of the block's
// best component).
// Top-m assignment of the n points of a piece from what launch_lse_wide (ntop >= m + 2; screened: it also marked the listed
// pairs) and launch_transform_wide (with_norm) left in wb: idx [n][m], resp [n][m] (may be NULL); rows whose answer is not certain are appended to unc_rows
// (unc_count += 1 each) and left unwritten.  mu, w2, c2d: the FP32 path's derived parameters.
cudaError_t launch_assign_refine_wide(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                                      const double* c2d, int n_slots, bool screened, const WideBuffers& wb, int ntop, int m,
                                      int32_t* idx, float* resp, int32_t* unc_rows, int* unc_count, bool index_only,
                                      bool hi = false);
// wb.n2[i] = |x_i - g|^2 for the n points of a piece.
// Clears wb.ctl, the n rows of wb.cand and the n_slots rows of wb.candT before a piece's first sweep.
cudaError_t launch_cand_clear_wide(cudaStream_t s, int64_t n, int n_slots, const WideBuffers& wb);
// After a screening sweep 1 with record = true: the marks whose recorded upper bound lies below the point's final threshold
// are taken out of wb.cand again and off wb.ctl[0].  (The sweep marks against the threshold as it stands when it meets a
// pair - the largest lower bound so far - which for most of a point's pairs is far from final.)
cudaError_t launch_cand_filter_wide(cudaStream_t s, int64_t n, int n_slots, const WideBuffers& wb);
// After sweep 1: wb.ctl[1] = (wb.ctl[0] > max_pairs), wb.ctl[2] = !wb.ctl[1].
cudaError_t launch_cand_gate_wide(cudaStream_t s, const WideBuffers& wb, long long max_pairs);
// The marked pairs evaluated exactly, one warp per point (no-op when wb.ctl[1] is set): logz_ill[i] = log2 of the sum of
// the listed components' exact densities at point i over the pairs that reach 2^-40 of wb.logz[i] (-inf if none); those
// pairs are marked in wb.candT.  best_out != NULL (the hard assignment, after a sweep with listed_only): instead, best_out[i]
// = the component of the point's largest exact value (of equal values the smaller component); logz_ill is not written.
cudaError_t launch_cand_lse_wide(cudaStream_t s, const float* X, int64_t n, int D, int n_slots, const WideBuffers& wb,
                                 double* logz_ill, int32_t* best_out = nullptr);
// The top-m assignment from the marked pairs (after a sweep with topm = m and ntop candidates, and the filter): idx [n][m],
// resp [n][m] (may be NULL) from the exact values of the point's marked pairs, largest first, of equal values the smaller
// component.  The marked pairs hold every component within 2^-40 of the point's best; ranks beyond them (responsibility
// 0) are filled from the sweep's candidates in the order of their upper bounds.  A point that still has fewer than m
// components is appended to unc_rows (unc_count += 1) and left unwritten.
cudaError_t launch_cand_topm_wide(cudaStream_t s, const float* X, int64_t n, int D, int n_slots, const WideBuffers& wb, int m,
                                  int32_t* idx, float* resp, int32_t* unc_rows, int* unc_count, int ntop);
// wb.stats_c += the statistics of the pairs marked in wb.candT with r = 2^(exact log2 z - wb.logz_x[i]); one block per
// slot, points in ascending order (no-op when wb.ctl[1] is set).
cudaError_t launch_cand_mstep_wide(cudaStream_t s, const float* X, int64_t n, int D, int n_slots, const WideBuffers& wb);
// Second sweep: responsibilities from wb.logz, statistics accumulated into wb.partial (+=).
cudaError_t launch_em_wide(cudaStream_t s, int64_t n, int D, int K, int Kg, const WideBuffers& wb, int num_sms, int* status);
// stats += the partial blocks (fixed order, float64, scale / centre / column order undone).
cudaError_t launch_reduce_wide(cudaStream_t s, int D, int K, int Kg, const WideBuffers& wb, int num_sms, double* Nk,
                               double* S1, double* S2);

}  // namespace fg
