/* flashgmm.h -- C ABI of libflashgmm: fused EM iteration of a diagonal-covariance Gaussian mixture on one
 * NVIDIA B200 (sm_100a).
 *
 * Model (paper Section 2, generalised from sigma_k^2 I to a per-dimension variance):
 *     p(x) = sum_k pi_k N(x | mu_k, diag(var_k)),   log z_ik = log pi_k + log N(x_i | mu_k, diag(var_k)),
 *     r_ik = z_ik / sum_j z_ij  (evaluated in log space with a log-sum-exp shift).
 * One EM iteration (paper Eq. 1-3 and Algorithm 1) is computed without ever storing the N x K responsibility
 * matrix: only the sufficient statistics
 *     N_k = sum_i r_ik,   S1_kd = sum_i r_ik x_id,   S2_kd = sum_i r_ik x_id^2,   loglik = sum_i log sum_k z_ik
 * leave the chip (Algorithm 1's M_k is S1; its scalar Q_k is replaced by S2 so that the variance can use the NEW
 * mean as Eq. 3 requires).  Device memory used beyond the caller's arrays is gmm_scratch_bytes(D, K): it does not
 * grow with N (paper Section 3.2, "Peak memory use").
 *
 * Conventions
 *   - "device" pointers are CUDA device pointers on the context's device; "host" pointers are ordinary host memory.
 *   - Layout: X is row-major [N x D] float32; mu, var, S1, S2 are row-major [K x D]; pi, Nk are [K].
 *   - Ownership: the caller owns every array it passes.  The library owns only the context's scratch, which it
 *     allocates at gmm_create / first use of a larger (D, K) and frees in gmm_destroy.
 *   - Every function returns GMM_OK (0) or a negative error code and never throws or aborts.  After a failure
 *     gmm_last_error(ctx) gives a human-readable message.  Output arrays are unspecified after a failure.
 *   - Work is enqueued on the context's stream; a call that has a host output synchronises that stream before it
 *     returns, calls without host outputs (gmm_finalize, gmm_assign_topm) return with the work still in flight.
 *     What device code finds wrong (invalid parameters, an expired wait) is recorded in a status word that stays set
 *     until the host has reported it: for an asynchronous call that is the next synchronising call on the context, or
 *     gmm_sync_status.
 *   - Results are deterministic: the same inputs give the same bits on every call (no floating-point atomics;
 *     per-CTA partial sums are added in a fixed order in float64).
 *   - A context is not thread-safe; use one per host thread.
 */
#ifndef FLASHGMM_H
#define FLASHGMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GMM_OK        0
#define GMM_EINVAL   -1   /* null pointer, N/D/K/m/iters out of range, negative floor */
#define GMM_EALIGN   -2   /* a pointer is not aligned for its element type */
#define GMM_ENOMEM   -3   /* scratch allocation failed */
#define GMM_ECUDA    -4   /* a CUDA call failed; message in gmm_last_error */
#define GMM_ENUMERIC -5   /* var <= 0, pi < 0, non-finite parameter, non-finite value in X, or non-finite log-likelihood */
#define GMM_ETIMEOUT -6   /* a bounded device-side wait expired; results invalid */
#define GMM_EUNSUPPORTED -7 /* the requested kernel path cannot run this shape */

/* Kernel paths (gmm_set_path).  AUTO picks the tensor-core path when the shape allows it. */
#define GMM_PATH_AUTO   0
#define GMM_PATH_FP32   1  /* CUDA-core float32 kernels with direct differences (x - mu)^2 / var; any shape */
#define GMM_PATH_TENSOR 2  /* tcgen05 tensor-core kernels on the expanded quadratic form; restricted shapes */

/* Covariance model used by the parameter update of gmm_fit (gmm_set_covariance). */
#define GMM_COV_DIAG      0  /* per-dimension variances (default) */
#define GMM_COV_ISOTROPIC 1  /* the paper's sigma_k^2 I: one variance per component, stored replicated over d */

#define GMM_MAX_TOPM 8

typedef struct gmm_ctx gmm_ctx;

/* Create a context on CUDA device `device`.  `cuda_stream` is a cudaStream_t (NULL = the legacy default stream) on
 * which all work of this context is enqueued; the caller keeps ownership of the stream. */
int gmm_create(gmm_ctx** out, int device, void* cuda_stream);
int gmm_destroy(gmm_ctx* ctx);

/* Select the kernel path for later calls (default GMM_PATH_AUTO).  GMM_EUNSUPPORTED is reported by the compute
 * call, not here, if a forced path cannot run the shape. */
int gmm_set_path(gmm_ctx* ctx, int path);
/* 1 if a tensor-core path can run shape (D, K) (D <= 1024 and K <= 4096; one kernel design for D <= 128, another for
 * wider data), else 0.  Components too ill-conditioned for the expanded quadratic form (sum_d mu^2 / var beyond what a
 * 22-bit split resolves, e.g. a component collapsed onto one point) are evaluated exactly in fp32 where they matter. */
int gmm_tensor_path_supports(int D, int K);
/* The path GMM_PATH_AUTO picks for shape (D, K): the tensor-core path when it is supported and the shape fills at
 * least half of a 128-component MMA tile (K >= 64, and D >= 8); otherwise the FP32 path, which is both faster and more
 * accurate for small mixtures.  On wide data (D > 128) a step may still run on the FP32 kernels when the parameters
 * or the data make that the better choice (more than half of the components ill-conditioned; fewer than 128 points per
 * component and posteriors too broad for the screening mode): gmm_last_path tells. */
int gmm_auto_path(int D, int K);
/* The path (GMM_PATH_FP32 or GMM_PATH_TENSOR) the most recent compute call actually ran. */
int gmm_last_path(const gmm_ctx* ctx);
/* How many components the most recent tensor-path step treated as ill-conditioned, i.e. evaluated (where they matter)
 * exactly in fp32 instead of through the expanded quadratic form; 0 after a step on the FP32 path.  On wide data
 * (D > 128), whenever a sample of the points shows that few pairs per point matter, the tensor path only screens the
 * (point, component) pairs and evaluates all that can matter exactly: the count is then the number of components with a
 * positive weight. */
int gmm_last_exact_count(const gmm_ctx* ctx);
/* For the most recent tensor-path step on wide data (D > 128) that had such components: how their (point, component)
 * pairs were evaluated.  *marked: pairs the screening sweep and its filter could not rule out; *kept: pairs whose exact density came
 * within 2^-40 of the point's total and entered the statistics (both summed over the pieces of the step that went pair
 * by pair, saturating at 2^31 - 1); *dense_pieces: pieces of the step whose marked pairs were too many (more than one in
 * 64; one in 16 when every component is screened), for which the FP32 kernels evaluated the whole sub-mixture instead.  All zero after any other step.  Reads a few
 * bytes back from the device (synchronises the context's stream).  Errors: GMM_EINVAL (NULL argument), GMM_ECUDA. */
int gmm_last_exact_pairs(gmm_ctx* ctx, int64_t* marked, int64_t* kept, int* dense_pieces);

/* E-step and sufficient statistics under the INPUT parameters (paper Section 2 responsibilities; Eq. 1; the
 * numerators of Eq. 2 and Eq. 3; Algorithm 1 without its last line).
 *   X [N x D] device; pi [K], mu [K x D], var [K x D] device float32, var > 0, pi >= 0.
 *   Nk [K], S1 [K x D], S2 [K x D] device float64 outputs (overwritten).
 *   loglik: host output, total log-likelihood sum_i log sum_k z_ik under the input parameters (natural log,
 *           including the -(D/2) log(2 pi) constant).
 * Synchronises the stream.  1 <= N, 1 <= D, 1 <= K. */
int gmm_em_step(gmm_ctx* ctx, const float* X, int64_t N, int D, int K,
                const float* pi, const float* mu, const float* var,
                double* Nk, double* S1, double* S2, double* loglik);

/* The same statistics with X in HOST memory (pageable or pinned): the library streams X through two device
 * staging buffers, overlapping the copy of one chunk with the kernels of the previous one, and accumulates every
 * chunk into the same O(K D) statistics (the chunked scheme the paper's Limitations section describes).  A staging
 * buffer holds 128 MiB of rows - on wide data (D > 128) where the tensor path applies, one piece of that path (2^17 rows:
 * 403 MB at D = 768) - and is allocated by the first call that needs it, outside gmm_scratch_bytes; on wide data the
 * automatic choice of the mode looks at the first rows of the first chunk.
 * All other arrays are host pointers too.  Synchronises the stream. */
int gmm_em_step_host(gmm_ctx* ctx, const float* X_host, int64_t N, int D, int K,
                     const float* pi_host, const float* mu_host, const float* var_host,
                     double* Nk_host, double* S1_host, double* S2_host, double* loglik);

/* Parameter update from the statistics (paper Section 2: pi_k = N_k / N; Eq. 2; Eq. 3 taken per dimension with the
 * new mean, i.e. var_kd = max(S2_kd / N_k - mu_kd^2, var_floor); Algorithm 1's last line).
 *   Nk, S1, S2 device float64 inputs; pi, mu, var device float32, in/out: a component with N_k < 1e-12 keeps its
 *   mu and var (its pi becomes N_k / N).  Asynchronous on the stream. */
int gmm_finalize(gmm_ctx* ctx, int64_t N, int D, int K,
                 const double* Nk, const double* S1, const double* S2,
                 float var_floor, float* pi, float* mu, float* var);

/* The paper's own update (Section 2, Eq. 3; Algorithm 1's last line) for the isotropic model sigma_k^2 I:
 *   sigma_k^2 = (1 / (D N_k)) sum_i r_ik ||x_i - mu_k^new||^2 = (1 / (D N_k)) sum_d (S2_kd - N_k mu_kd^2),
 * floored at var_floor and written to all D entries of var[k, :], so that gmm_em_step / gmm_assign_topm evaluate
 * N(x | mu_k, sigma_k^2 I) with the same kernels.  Same arguments and rules as gmm_finalize. */
int gmm_finalize_isotropic(gmm_ctx* ctx, int64_t N, int D, int K,
                           const double* Nk, const double* S1, const double* S2,
                           float var_floor, float* pi, float* mu, float* var);
/* Selects which update gmm_fit applies: GMM_COV_DIAG (default) or GMM_COV_ISOTROPIC. */
int gmm_set_covariance(gmm_ctx* ctx, int covariance);

/* EM driver: `iters` iterations of gmm_em_step + gmm_finalize (paper Section 2, last paragraph; Algorithm 1 run
 * repeatedly).  pi/mu/var: device, in = initial parameters, out = fitted.  loglik_trace: host [iters];
 * trace[t] is the log-likelihood under the parameters ENTERING iteration t.  tol > 0 stops after iteration t >= 1
 * when |L_t - L_{t-1}| <= tol * |L_t|; tol = 0 runs all iterations.  iters_done (host, may be NULL) receives the
 * number of iterations run.  If an iteration fails (GMM_ENUMERIC: invalid parameters or non-finite data; GMM_ETIMEOUT),
 * its parameter update is not applied: pi, mu, var hold the parameters that entered the failed iteration.
 * Synchronises the stream. */
int gmm_fit(gmm_ctx* ctx, const float* X, int64_t N, int D, int K,
            float* pi, float* mu, float* var,
            int iters, float var_floor, double tol,
            double* loglik_trace, int* iters_done);

/* Top-m components by responsibility for every point (paper Section 4.2: the arg-max assignment; Section 4.3: the
 * clusters with the largest responsibilities, which the caller thresholds with tau = 1/K).
 *   idx [N x m] int32 and resp [N x m] float32, device outputs; per point descending by responsibility, ties to the
 *   smaller component index.  1 <= m <= min(K, GMM_MAX_TOPM).  Asynchronous on the stream.
 *   resp may be NULL: the indices alone are computed (the hard assignment of Section 4.2 with m = 1); the tensor-core
 *   path then needs no accurate log-sum-exp and, for m = 1, keeps half as many candidates per point.
 * Where the tensor-core path applies (the rule of gmm_em_step) the logits of all components come from the tensor cores
 * as a selection pass and the best few per point are recomputed exactly in fp32, so indices and values are those of the
 * FP32 kernels; a point whose selection is not certain within the error bound of the selection pass is evaluated
 * against all K components exactly; components whose responsibility for a point is below 4.8e-7 keep the order and
 * the values of the selection pass (inside the 1e-6 tie width).  On wide data (D > 128), whenever a sample of the points
 * shows that few (point, component) pairs matter, one tensor sweep screens all pairs instead, every component within
 * 2^-40 of a point's best is evaluated exactly (indices and responsibilities from those values), and ranks beyond them
 * are reported with responsibility 0 in the order of the sweep's upper bounds.  Parameters with more than 256 ill-conditioned
 * components run on the FP32 kernels (decided on the device; gmm_last_path then still reports the tensor path).  The
 * first call allocates a work buffer outside gmm_scratch_bytes: 128 or 192 bytes (m <= 4, m > 4) per point of one piece
 * of at most 2^19 points plus 4 bytes per point of eight pieces (84 MB or 118 MB at most, independent of N). */
int gmm_assign_topm(gmm_ctx* ctx, const float* X, int64_t N, int D, int K,
                    const float* pi, const float* mu, const float* var, int m,
                    int32_t* idx, float* resp);

/* IVF posting lists from the top-m assignment (paper Section 4.2: every vector is stored with the cluster of its highest
 * responsibility; Section 4.3, multi-assignment: with at most two clusters, the top clusters whose responsibility
 * exceeds tau = 1/K).  The rule implemented: choice 0 of a vector is always taken; choices 1 .. max_lists-1 are taken
 * in order while resp > tau (strictly); a negative index ends a vector's list.
 *   idx [N x m] int32, resp [N x m] float32: device, as written by gmm_assign_topm (descending responsibility).
 *   tau: threshold; <= 0 selects the paper's 1/K.   max_lists: 1 (hard assignment) .. m (the paper uses 2).
 *   offsets [K + 1] int64, device out: list k holds items[offsets[k] .. offsets[k+1]).
 *   items  int32, device out, capacity >= N * max_lists entries: vector indices, ascending inside every list.
 *   total (host out, may be NULL): offsets[K];  mean_lists (host out, may be NULL): total / N, the paper's average
 *   number of posting lists per vector (Section 4.6, multi-assignment analysis).
 * Deterministic (no atomics on the output); scratch O(K), independent of N.  Limits: N < 2^31, K <= 8192 (otherwise
 * GMM_EUNSUPPORTED).  Synchronises the stream. */
int gmm_build_posting_lists(gmm_ctx* ctx, const int32_t* idx, const float* resp, int64_t N, int m, int K,
                            float tau, int max_lists, int64_t* offsets, int32_t* items,
                            int64_t* total, double* mean_lists);

/* One Lloyd (k-means) iteration, the warm start the paper runs before its EM iterations (Section 4.4, experimental setup, and the warm-start appendix:
 * 10 iterations of k-means, then Flash-GMM).  Assignment: every point goes to the centroid at the smallest squared
 * Euclidean distance (direct differences in fp32; ties to the smaller index).  Update: a centroid becomes the mean of its
 * points (float64 sums in a fixed order); a centroid without points keeps its position.
 *   X [N x D], centroids [K x D]: device, row-major fp32.
 *   assign [N] int32, device out: the index of each point's nearest centroid.
 *   work [2 N] int32, device scratch owned by the caller (the library holds no O(N) memory).
 *   centroids_out [K x D] fp32, device out (may be the same array as centroids).
 *   counts [K] int64, device out, may be NULL: points per centroid.
 *   inertia (host out, may be NULL): sum over the points of the squared distance to their (input) centroid.
 * Deterministic (no atomics).  Limits: N < 2^31, K <= 8192 (otherwise GMM_EUNSUPPORTED).  Synchronises the stream. */
int gmm_kmeans_step(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* centroids,
                    int32_t* assign, int32_t* work, float* centroids_out, int64_t* counts, double* inertia);

/* Per-point log-density under the mixture, log p(x_i) = log sum_k pi_k N(x_i | mu_k, diag var_k) (Section 2; the
 * stable log-sum-exp of Section 3.2, whose per-point value Algorithm 1 keeps on chip): the quantity a kernel density
 * estimate evaluates, which the paper's Discussion (Section 6) names as another user of the fused pattern.
 *   X [N x D], pi [K], mu [K x D], var [K x D]: device fp32, as for gmm_em_step.
 *   logp [N] fp32, device out (natural logarithm);  loglik (host out, may be NULL): their sum in float64.
 * Every value comes from exact direct-difference logits in fp32 (a per-point value has no averaging over points to absorb
 * approximate logits): the log-sum-exp kernel of the FP32 path, or, on wide data (D > 128, K >= 64, path not forced to
 * FP32) whenever a sample of the points shows that few (point, component) pairs matter, one tensor sweep that screens the
 * pairs followed by the exact evaluation of those it cannot rule out (every component within 2^-40 of a point's best);
 * gmm_last_path tells which.  Errors as gmm_em_step.  Synchronises the stream. */
int gmm_score_samples(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* pi, const float* mu,
                      const float* var, float* logp, double* loglik);

/* Fisher-vector encoding of G groups of points under a fixed mixture: the per-group use of the fused pattern (log-sum-exp
 * over the K weighted Gaussian terms, then responsibility-weighted statistics) that the paper's Discussion (Section 6)
 * names.  The paper prints no formula; the standard definition is used.  For a group of T points with responsibilities
 * r_tk (Section 2),
 *   G_mu[k, d]    = 1 / (T sqrt(pi_k))   * sum_t r_tk (x_td - mu_kd) / sigma_kd
 *   G_sigma[k, d] = 1 / (T sqrt(2 pi_k)) * sum_t r_tk ((x_td - mu_kd)^2 / sigma_kd^2 - 1),   sigma_kd = sqrt(var_kd),
 * i.e. the gradient of the group's mean log-likelihood in (mu, sigma), each coordinate divided by the square root of
 * its diagonal Fisher information.  Each group's (N_k, S1, S2) come from the tile kernels of gmm_em_step (nothing of
 * size T x K is written to memory) and are turned into the two parts in float64.
 *   X [N x D]: device, row-major fp32; group g is rows offsets[g] .. offsets[g + 1] - 1.
 *   offsets [G + 1] int64, HOST: non-decreasing, offsets[0] >= 0, offsets[G] <= N; an empty group gets zeros.
 *   pi [K], mu [K x D], var [K x D]: device fp32, as for gmm_em_step; a component with pi_k = 0 gets zeros.
 *   fv [G x 2 x K x D] fp32, device out: per group the means part [K x D], then the standard-deviations part [K x D].
 *   No power or L2 normalisation is applied.
 *   loglik (host out, may be NULL): the total log-likelihood of all the groups' points.
 * On the tensor-core path several groups share a launch (each group of CTAs accumulates one of them); groups too large
 * for that are accumulated one at a time.
 * Accuracy: a coordinate is a difference of the raw moments (N_k, S1, S2), which carry about 4e-6 relative error, so
 * with A_k = N_k / (T sqrt(pi_k)) (at most about 1 for a group that resembles the mixture, up to 1 / sqrt(pi_k) for a
 * group that sits on one light component) the error is about 2e-5 (1 + max|G|) + A_k (1e-3 + 4e-5 (1 + mu^2 / var));
 * data far from the origin in units of sigma should be centred first.
 * Errors as gmm_em_step; GMM_EINVAL for offsets out of order or out of range.  Synchronises the stream. */
int gmm_fisher_vectors(gmm_ctx* ctx, const float* X, int64_t N, const int64_t* offsets, int G, int D, int K,
                       const float* pi, const float* mu, const float* var, float* fv, double* loglik);

/* The statistics of gmm_em_step for callers that cannot allocate device memory.  (The paper has no counterpart of
 * this entry point; it exists for the library's users.)
 *
 * Who needs it: a host that must not call cudaMalloc/cudaFree where it takes an EM step -- a plugin running inside
 * a service whose device memory is budgeted and owned by another allocator, code called between a framework's own
 * allocations where a driver allocation would stall the device, or a latency-bound loop that may not block on the
 * driver's allocator.  This function needs no context and allocates nothing: all scratch of the FP32 kernel chain
 * lives in a 6 MiB array that is part of the library's device image (every GPU that loads the library holds those
 * 6 MiB until the process exits).  It calls no cudaMalloc, no cudaFree and no allocating library routine.
 *
 *   device, cuda_stream: the device to run on and a cudaStream_t on it (NULL = legacy default stream).
 *   X, pi, mu, var, Nk, S1, S2: device arrays exactly as for gmm_em_step; loglik: host output.
 *   Limits: K <= 1024 and K * D <= 32768; larger shapes return GMM_EUNSUPPORTED and launch nothing.
 *   Always the FP32 path.  Results equal gmm_em_step's up to float32 summation order (the per-CTA partials are
 *   grouped differently), i.e. well inside the tolerances of the parity tests; they are still deterministic.
 *   The first call on each device looks up the array's device address (cudaGetSymbolAddress): make that first call
 *   before starting any stream capture.  The CUDA runtime also loads a kernel's code into the device the first time
 *   that kernel is launched, which may allocate and synchronise inside the driver: a caller that must not allocate
 *   from some point on makes one warm-up call per device and per kernel variant before that point -- the variants
 *   are D <= 128 (float logits) and D > 128 (float64 logits, another M-step kernel).  The looked-up address is cached
 *   per device for the life of the process; it does not survive cudaDeviceReset.
 *   Every call on a device shares the one array and the array keeps the previous call's contents; the function
 *   clears what it accumulates into, but two calls that overlap on the same GPU (different streams or threads)
 *   race on it -- serialise them.  Synchronises the stream before returning. */
int gmm_em_step_static(int device, void* cuda_stream, const float* X, int64_t N, int D, int K,
                       const float* pi, const float* mu, const float* var,
                       double* Nk, double* S1, double* S2, double* loglik);

/* Waits for the context's stream and reports what device code recorded since the last report: GMM_OK, or the error of
 * an earlier asynchronous call (GMM_ENUMERIC for var <= 0, pi < 0 or non-finite parameters given to gmm_assign_topm;
 * GMM_ETIMEOUT).  The outputs of that call are then invalid.  Reporting clears the record. */
int gmm_sync_status(gmm_ctx* ctx);

/* Diagnostics of the most recent parameter update on this context (gmm_finalize, gmm_finalize_isotropic, or the last
 * iteration of gmm_fit): how many variance entries were raised to var_floor, and how many components were left
 * unchanged because N_k < 1e-12.  (The paper has neither rule; both can break the monotone growth of the
 * log-likelihood, so a caller watching the trace wants to know.)  Either output may be NULL.  Synchronises the stream. */
int gmm_update_counts(gmm_ctx* ctx, int64_t* floored_variances, int64_t* empty_components);

/* Bytes of device scratch a context in GMM_PATH_AUTO holds for shape (D, K); independent of N.  Where the tensor
 * path runs (see gmm_auto_path) this includes 512 MiB for the fp16 planes of one launch-sized piece of the data;
 * forcing GMM_PATH_TENSOR on a shape AUTO sends to the FP32 path adds the same 512 MiB. */
size_t gmm_scratch_bytes(int D, int K);

/* Instrumentation.  Kernel launches enqueued by this context since creation (or the last reset). */
int64_t gmm_launch_count(const gmm_ctx* ctx);
/* With profiling on, the dominant kernel of each compute call (the E/M tile kernel) is bracketed by CUDA events on
 * the context's stream.  gmm_kernel_time synchronises the stream and returns the summed event time in
 * milliseconds and the number of bracketed launches since the last gmm_reset_counters. */
int gmm_set_profiling(gmm_ctx* ctx, int on);
int gmm_kernel_time(gmm_ctx* ctx, double* total_ms, int64_t* launches);
int gmm_reset_counters(gmm_ctx* ctx);

/* Measures, on the given device, the two rates the secondary roofs of an EM iteration are quoted against: dependent
 * fp32 fused multiply-adds at full occupancy (in flop/s, 2 per FMA: the roof of the FP32 path) and ex2.approx.ftz.f32
 * results per second (the special-function unit: the roof of the N K exponentials).  Two launches of a few milliseconds
 * each on the default stream; allocates and frees 256 bytes.  Host outputs. */
int gmm_probe_rates(int device, double* fp32_fma_flops, double* ex2_per_s);

const char* gmm_strerror(int code);
const char* gmm_last_error(const gmm_ctx* ctx);
const char* gmm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FLASHGMM_H */
