// Host side of libflashgmm: context, argument checking, scratch management, path dispatch, the EM driver and the
// host-streaming variant.  Every step of the numerical path runs in the CUDA kernels of the other files.
#include "internal.cuh"
#include "em_tc.cuh"
#include "em_wide.cuh"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

using namespace fg;

namespace {

struct DevResult {
    double ll[LL_SLOTS];
    int status;     // sticky: device code ORs bits in; the host clears it only after it has reported them
    int n_ill;      // ill-conditioned components found by the tensor path's last preparation
    int counts[2];  // the last parameter update: variance entries raised to the floor, components left unchanged as empty
};

constexpr size_t STAGE_BYTES = (size_t)128 << 20;   // per staging buffer of the host-streaming path
constexpr int EVENT_POOL = 128;

inline size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

struct ScratchLayout {
    size_t w2, c2, c2d, center, partials, logZ2, llpart, result, stats, total;
    size_t tc_phi, tc_plo, tc_tk, tc_ck, tc_sd, tc_kap, tc_gd, tc_illb, tc_flags, tc_xg, tc_xl, tc_partial, tc_llpart, tc_partial_bytes, tc_yhi, tc_ylo, tc_phirm, tc_plorm, tc_tkck, tc_illlist, tc_illcache, tc_decdim, tc_decw, tc_decmu;
    bool tc;
    // the tensor-core path for D > 128
    size_t w_sd, w_kap, w_gd, w_phi, w_plo, w_tk, w_tkck, w_ckd, w_cref, w_illb, w_flags, w_yhi, w_ylo, w_logz, w_partial, w_llpart, w_illlist, w_muc, w_w2c, w_c2dc, w_statsc, w_top, w_logzx, w_compof, w_scra, w_scrw, w_scr, w_slotof, w_scrmask, w_n2, w_cand, w_candT, w_ctl, w_scre, w_slotcnt, w_heavyof, w_heavyslot, w_heavypart, w_scrahi, w_scrwhi, w_pairval, w_pairoff, w_pairbest, w_pairkey8, w_pairval8, w_rec, w_reccnt, w_recthr;
    size_t w_partial_bytes;
    bool wide;
};

// planes: include the fp16 planes of Y (tensor path only; 2 x TC_YPLANE_BYTES, placed last so that no other offset moves)
ScratchLayout scratch_layout(int D, int K, bool planes) {
    ScratchLayout L;
    const size_t KD = (size_t)K * D;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
    L.w2 = take(KD * 4);
    L.c2 = take((size_t)K * 4);
    L.c2d = take((size_t)K * 8);
    L.center = take((size_t)D * 4);
    L.partials = take(fp32_partial_floats(D, K) * 4);
    L.logZ2 = take((size_t)SUPER_TILE * 8);
    L.llpart = take((size_t)(SUPER_TILE / FP32_TILE_P) * 8);
    L.result = take(sizeof(DevResult));
    L.stats = take(((size_t)K + 2 * KD) * 8);
    L.tc = tc_assign_supports(D, K);           // the assignment kernels' shapes include the E+M tile kernel's
    L.tc_phi = L.tc_plo = L.tc_tk = L.tc_ck = L.tc_sd = L.tc_kap = L.tc_gd = L.tc_illb = L.tc_flags = L.tc_xg = L.tc_xl = L.tc_partial = L.tc_llpart = L.tc_yhi = L.tc_ylo = L.tc_phirm = L.tc_plorm = L.tc_tkck = L.tc_illlist = L.tc_illcache = L.tc_decdim = L.tc_decw = L.tc_decmu = 0;
    L.tc_partial_bytes = 0;
    if (L.tc) {
        const TcPlan pl = tc_plan(D, K, 160);       // an upper bound on the number of clusters
        L.tc_phi = take((size_t)pl.CL * 128 * 128 * 4);
        L.tc_plo = take((size_t)pl.CL * 65536);
        L.tc_tk = take((size_t)pl.Kpad * 4);
        L.tc_ck = take((size_t)pl.Kpad * 4);
        L.tc_sd = take(128 * 4);
        L.tc_kap = take(128 * 4);
        L.tc_gd = take(128 * 4);
        L.tc_illb = take((size_t)pl.Kpad * 4);
        L.tc_flags = take(32);
        if (tc_supports(D, K)) {                // what only the E+M tile kernel needs
            L.tc_xg = take((size_t)pl.Q * 4 * pl.CL * 64 * 16);
            L.tc_xl = take((size_t)pl.Q * 4 * pl.CL * 256 * 16);
            L.tc_partial_bytes = (size_t)pl.Q * pl.Kpad * TC_PCOLS * 8;
            L.tc_partial = take(L.tc_partial_bytes);
            L.tc_llpart = take((size_t)pl.Q * 16);
        }
        L.tc_phirm = take((size_t)pl.Kpad * 512);
        L.tc_plorm = take((size_t)pl.Kpad * 512);
        L.tc_tkck = take((size_t)pl.Kpad * 8);
        L.tc_illlist = take((size_t)pl.Kpad * 4);
        L.tc_illcache = take(sizeof(TcIllCache));
        L.tc_decdim = take((size_t)pl.Kpad * 8 * 4);
        L.tc_decw = take((size_t)pl.Kpad * 8 * 4);
        L.tc_decmu = take((size_t)pl.Kpad * 8 * 4);
    }
    if (L.tc && planes) {
        L.tc_yhi = take(TC_YPLANE_BYTES);
        L.tc_ylo = take(TC_YPLANE_BYTES);
    }
    L.w_sd = L.w_kap = L.w_gd = L.w_phi = L.w_plo = L.w_tk = L.w_tkck = L.w_ckd = L.w_cref = L.w_illb = L.w_flags = L.w_yhi = L.w_ylo = L.w_logz = L.w_partial = L.w_llpart = L.w_illlist = L.w_muc = L.w_w2c = L.w_c2dc = L.w_statsc = L.w_top = L.w_logzx = 0;
    L.w_compof = L.w_scra = L.w_scrw = L.w_scr = L.w_slotof = L.w_scrmask = L.w_n2 = L.w_cand = L.w_candT = L.w_ctl = L.w_scre = L.w_slotcnt = L.w_heavyof = L.w_heavyslot = L.w_heavypart = L.w_scrahi = L.w_scrwhi = L.w_pairval = L.w_pairoff = L.w_pairbest = L.w_pairkey8 = L.w_pairval8 = L.w_rec = L.w_reccnt = L.w_recthr = 0;
    L.w_partial_bytes = 0;
    L.wide = wide_supports(D, K) && planes;
    if (L.wide) {
        const WidePlan wp = wide_plan(D, K, 160);
        L.w_sd = take((size_t)wp.Dpad * 4);
        L.w_kap = take((size_t)wp.Dpad * 4);
        L.w_gd = take((size_t)wp.Dpad * 4);
        L.w_phi = take((size_t)wp.rows * wp.Dpad * 4);
        L.w_plo = take((size_t)wp.rows * wp.Dpad * 4);
        L.w_tk = take((size_t)wp.rows * 4);
        L.w_tkck = take((size_t)wp.rows * 8);
        L.w_ckd = take((size_t)wp.rows * 8);
        L.w_cref = take(8);
        L.w_illb = take((size_t)wp.Kpad * 4);
        L.w_flags = take(32);
        L.w_compof = take((size_t)wp.rows * 4);
        L.w_scra = take((size_t)wp.Kpad * 4);
        L.w_scrw = take((size_t)wp.Kpad * 4);
        L.w_scr = take((size_t)wp.rows * 8);
        L.w_slotof = take((size_t)wp.rows * 4);
        L.w_scrmask = take((size_t)wp.rows / 32 * 4);
        L.w_n2 = take((size_t)WIDE_PIECE * 4);
        const size_t slots = (size_t)(K + 64 < WIDE_MAX_ILL ? K + 64 : WIDE_MAX_ILL);     // the list is never longer
        L.w_cand = take((size_t)WIDE_PIECE * ((slots + 31) / 32) * 4);
        L.w_candT = take(slots * WIDE_CANDT_WORDS * 4);
        L.w_ctl = take(32);
        L.w_scre = take((size_t)wp.rows * 4);
        L.w_scrahi = take((size_t)wp.Kpad * 4);
        L.w_scrwhi = take((size_t)wp.Kpad * 4);
        L.w_slotcnt = take(slots * 4);
        L.w_heavyof = take(slots * 4);
        L.w_heavyslot = take((size_t)WIDE_HEAVY_SLOTS * 4);
        L.w_heavypart = take((size_t)WIDE_HEAVY_SLOTS * WIDE_HEAVY_SEG * (1 + 2 * (size_t)D) * 8);
        L.w_pairval = take((size_t)WIDE_PAIR_VALS * 4);
        L.w_pairoff = take((size_t)WIDE_PIECE * 4);
        L.w_pairbest = take((size_t)WIDE_PIECE * 8);
        L.w_pairkey8 = take((size_t)WIDE_PIECE * 8 * 2);
        L.w_pairval8 = take((size_t)WIDE_PIECE * 8 * 4);
        L.w_rec = take((size_t)WIDE_PIECE * WIDE_REC * 4);
        L.w_reccnt = take((size_t)WIDE_PIECE * 8);
        L.w_recthr = take((size_t)WIDE_PIECE * 4);
        L.w_logz = take((size_t)WIDE_PIECE * 8);
        L.w_top = take((size_t)WIDE_PIECE * 2 * WIDE_MAX_TOP * 4);
        L.w_logzx = take((size_t)WIDE_PIECE * 8);
        L.w_partial_bytes = (size_t)wp.R * wp.CL * wp.pcols * 128 * 4;
        L.w_partial = take(L.w_partial_bytes);
        L.w_llpart = take(256 * 8);
        L.w_illlist = take((size_t)WIDE_MAX_ILL * 4);
        L.w_muc = take(slots * D * 4);
        L.w_w2c = take(slots * D * 4);
        L.w_c2dc = take(slots * 8);
        L.w_statsc = take((slots + 2 * slots * D) * 8);
        L.w_yhi = take((size_t)WIDE_PIECE * wp.Dpad * 4);
        L.w_ylo = take((size_t)WIDE_PIECE * wp.Dpad * 4);
    }
    L.total = off;
    return L;
}

}  // namespace

struct gmm_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int path = GMM_PATH_AUTO;
    int last_path = 0;
    int covariance = GMM_COV_DIAG;
    // scratch
    unsigned char* scratch = nullptr;
    size_t scratch_bytes = 0;
    int capD = 0, capK = 0;
    void* pl_scratch = nullptr;      // posting-list builder: counters per (range of vectors, cluster)
    void* km_scratch = nullptr;      // k-means step: list offsets, per-segment float64 sums
    void* at_scratch = nullptr;      // tensor-core assignment: candidate records of one piece of points
    size_t at_scratch_bytes = 0;
    void* fv_scratch = nullptr;      // Fisher vectors, grouped launches: tile and group tables
    size_t fv_scratch_bytes = 0;
    void* km_unit = nullptr;         // k-means step on the tensor path: var = 1 [K x D], pi = 1 / K [K]
    size_t km_unit_bytes = 0;
    size_t km_scratch_bytes = 0;
    size_t pl_scratch_bytes = 0;
    bool capPlanes = false;    // the scratch layout in force includes the tensor path's planes of Y
    ScratchLayout lay{};
    int tc_Q = 0;              // resident clusters of the tensor-path kernel for (capD, capK)
    float tc_cond_limit = -1.f;      // < 0: automatic, tc_cond_scale * sqrt(N / K)
    float tc_cond_scale = 1.5e-4f;
    int tc_flush = TC_FLUSH;
    int64_t tc_piece = TC_YPOINTS;   // points per launch of the tile kernel (<= capacity of the Y planes)
    int64_t wide_piece = WIDE_PIECE; // points per pair of sweeps of the D > 128 tensor path
    int sms = 148;                   // multiprocessors of the device
    double wide_min_points = 64.0;   // components expected to hold fewer points (pi_k N) are evaluated exactly
    bool wide_refine = true;         // correct log2 Z by the exact values of each point's two leading terms
    int wide_n_first = 0;            // of which the first kind (flagged by the error estimate: mostly collapsed components)
    int wide_n_list = 0;             // slots of the packed sub-mixture (the ill-conditioned components plus padding)
    int wide_n_ill = 0;              // ill-conditioned components of the current step on the D > 128 tensor path
    int wide_n_good = 0;             // components the tensor passes evaluate in the current step (the others are listed)
    int wide_mode = 0;               // GMM_WIDE_MODE: 0 = automatic, 1 = "sweeps" (two tensor sweeps, few components exact),
                                     // 2 = "screen" (one tensor sweep screens every pair, every component evaluated exactly)
    double wide_probe_limit = 0.0;   // automatic mode: "screen" while a sample of the points has at most this many marked pairs per
                                     // point (0: from the measured costs, see wide_pair_limit)
    bool wide_screen_all = false;    // the current step runs in "screen" mode
    bool wide_pre = false;           // GMM_WIDE_PRE=1: a first pass over the leading product for the screening threshold (instead
                                     // of leaving the marks made against an immature threshold to the filter alone)
    int wide_hi = 2;                 // GMM_WIDE_HI: which listed components the screening mode screens by the leading product alone:
                                     // 0 = none (all three products for every component), 1 = those behind the first kind of the list
                                     // (the components flagged by the rounding estimate keep all three products), 2 = all
    int wide_sparse = 1;             // GMM_WIDE_SPARSE: 0 = the listed components always go through the dense FP32 kernels,
                                     // 1 = pair by pair unless sweep 1 marks too many pairs, 2 = always pair by pair (tests)
    int tc_n_ill = 0;                // ill-conditioned components at the last result that was read back (picks the filter)
    int tc_force_filter = -1;        // GMM_TC_FILTER=plain / tight: 0 / 1 (tests); -1: automatic
    int sticky_status = 0;           // status bits read off the device but not yet reported (see ensure_scratch)
    // host-streaming path
    cudaStream_t copy_stream = nullptr;
    float* xstage[2] = {nullptr, nullptr};
    size_t xstage_bytes = 0;         // size of each staging buffer
    cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr};
    float* hparams = nullptr;      // device copies of pi, mu, var for the host path
    size_t hparams_floats = 0;
    // instrumentation
    int64_t launches = 0;
    bool profiling = false;
    cudaEvent_t ev_a[EVENT_POOL], ev_b[EVENT_POOL];
    int ev_used = 0;
    bool ev_created = false;
    double prof_ms = 0.0;
    int64_t prof_launches = 0;
    char err[512] = {0};

    float* w2() const { return reinterpret_cast<float*>(scratch + lay.w2); }
    float* c2() const { return reinterpret_cast<float*>(scratch + lay.c2); }
    double* c2d() const { return reinterpret_cast<double*>(scratch + lay.c2d); }
    float* center() const { return reinterpret_cast<float*>(scratch + lay.center); }     // per-dimension centre of the means
    float* partials() const { return reinterpret_cast<float*>(scratch + lay.partials); }
    double* logZ2() const { return reinterpret_cast<double*>(scratch + lay.logZ2); }
    double* llpart() const { return reinterpret_cast<double*>(scratch + lay.llpart); }
    DevResult* result() const { return reinterpret_cast<DevResult*>(scratch + lay.result); }
    double* stats() const { return reinterpret_cast<double*>(scratch + lay.stats); }
    TcBuffers tc() const {
        TcBuffers b;
        b.phi_img = reinterpret_cast<uint32_t*>(scratch + lay.tc_phi);
        b.plo_img = scratch + lay.tc_plo;
        b.tk = reinterpret_cast<float*>(scratch + lay.tc_tk);
        b.ck = reinterpret_cast<float*>(scratch + lay.tc_ck);
        b.sd = reinterpret_cast<float*>(scratch + lay.tc_sd);
        b.kap = reinterpret_cast<float*>(scratch + lay.tc_kap);
        b.gd = reinterpret_cast<float*>(scratch + lay.tc_gd);
        b.illb = reinterpret_cast<float*>(scratch + lay.tc_illb);
        b.flags = reinterpret_cast<int*>(scratch + lay.tc_flags);
        b.xg = scratch + lay.tc_xg;
        b.xl = scratch + lay.tc_xl;
        b.partial = reinterpret_cast<double*>(scratch + lay.tc_partial);
        b.llpart = reinterpret_cast<double*>(scratch + lay.tc_llpart);
        b.y_hi = scratch + lay.tc_yhi;
        b.y_lo = scratch + lay.tc_ylo;
        b.p_hi_rm = scratch + lay.tc_phirm;
        b.p_lo_rm = scratch + lay.tc_plorm;
        b.tkck = reinterpret_cast<float*>(scratch + lay.tc_tkck);
        b.ill_list = reinterpret_cast<int*>(scratch + lay.tc_illlist);
        b.ill_cache = reinterpret_cast<TcIllCache*>(scratch + lay.tc_illcache);
        b.dec_dim = reinterpret_cast<int*>(scratch + lay.tc_decdim);
        b.dec_w = reinterpret_cast<float*>(scratch + lay.tc_decw);
        b.dec_mu = reinterpret_cast<float*>(scratch + lay.tc_decmu);
        return b;
    }
    WideBuffers wide() const {
        WideBuffers b;
        b.sd = reinterpret_cast<float*>(scratch + lay.w_sd);
        b.kap = reinterpret_cast<float*>(scratch + lay.w_kap);
        b.gd = reinterpret_cast<float*>(scratch + lay.w_gd);
        b.p_hi = scratch + lay.w_phi;
        b.p_lo = scratch + lay.w_plo;
        b.tk = reinterpret_cast<float*>(scratch + lay.w_tk);
        b.tkck = reinterpret_cast<float*>(scratch + lay.w_tkck);
        b.ckd = reinterpret_cast<double*>(scratch + lay.w_ckd);
        b.cref = reinterpret_cast<double*>(scratch + lay.w_cref);
        b.illb = reinterpret_cast<float*>(scratch + lay.w_illb);
        b.flags = reinterpret_cast<int*>(scratch + lay.w_flags);
        b.y_hi = scratch + lay.w_yhi;
        b.y_lo = scratch + lay.w_ylo;
        b.logz = reinterpret_cast<double*>(scratch + lay.w_logz);
        b.top = reinterpret_cast<float*>(scratch + lay.w_top);
        b.logz_x = reinterpret_cast<double*>(scratch + lay.w_logzx);
        b.partial = reinterpret_cast<float*>(scratch + lay.w_partial);
        b.llpart = reinterpret_cast<double*>(scratch + lay.w_llpart);
        b.ill_list = reinterpret_cast<int*>(scratch + lay.w_illlist);
        b.mu_c = reinterpret_cast<float*>(scratch + lay.w_muc);
        b.w2_c = reinterpret_cast<float*>(scratch + lay.w_w2c);
        b.c2d_c = reinterpret_cast<double*>(scratch + lay.w_c2dc);
        b.stats_c = reinterpret_cast<double*>(scratch + lay.w_statsc);
        b.comp_of = reinterpret_cast<int*>(scratch + lay.w_compof);
        b.scra = reinterpret_cast<float*>(scratch + lay.w_scra);
        b.scrw = reinterpret_cast<float*>(scratch + lay.w_scrw);
        b.scr = reinterpret_cast<float*>(scratch + lay.w_scr);
        b.slot_of = reinterpret_cast<int*>(scratch + lay.w_slotof);
        b.scr_mask = reinterpret_cast<int*>(scratch + lay.w_scrmask);
        b.n2 = reinterpret_cast<float*>(scratch + lay.w_n2);
        b.cand = reinterpret_cast<unsigned*>(scratch + lay.w_cand);
        b.candT = reinterpret_cast<unsigned*>(scratch + lay.w_candT);
        b.ctl = reinterpret_cast<int*>(scratch + lay.w_ctl);
        b.scr_e = reinterpret_cast<float*>(scratch + lay.w_scre);
        b.scra_hi = reinterpret_cast<float*>(scratch + lay.w_scrahi);
        b.scrw_hi = reinterpret_cast<float*>(scratch + lay.w_scrwhi);
        b.slot_cnt = reinterpret_cast<int*>(scratch + lay.w_slotcnt);
        b.heavy_of = reinterpret_cast<int*>(scratch + lay.w_heavyof);
        b.heavy_slot = reinterpret_cast<int*>(scratch + lay.w_heavyslot);
        b.heavy_part = reinterpret_cast<double*>(scratch + lay.w_heavypart);
        b.pair_val = reinterpret_cast<float*>(scratch + lay.w_pairval);
        b.pair_off = reinterpret_cast<int*>(scratch + lay.w_pairoff);
        b.pair_best = reinterpret_cast<double*>(scratch + lay.w_pairbest);
        b.pair_key8 = reinterpret_cast<unsigned short*>(scratch + lay.w_pairkey8);
        b.pair_val8 = reinterpret_cast<float*>(scratch + lay.w_pairval8);
        b.rec = reinterpret_cast<unsigned*>(scratch + lay.w_rec);
        b.rec_cnt = reinterpret_cast<int*>(scratch + lay.w_reccnt);
        b.rec_thr = reinterpret_cast<float*>(scratch + lay.w_recthr);
        return b;
    }
};

namespace {

int fail(gmm_ctx* ctx, int code, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

#define CU(call)                                                                                      \
    do {                                                                                              \
        cudaError_t e_ = (call);                                                                      \
        if (e_ != cudaSuccess)                                                                        \
            return fail(ctx, GMM_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
    } while (0)

#define KL(call)                                                                                      \
    do {                                                                                              \
        cudaError_t e_ = (call);                                                                      \
        if (e_ != cudaSuccess)                                                                        \
            return fail(ctx, GMM_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
        ctx->launches++;                                                                              \
    } while (0)

// The tensor path runs when it is forced or when AUTO picks it for the shape: only then are the planes of Y needed.
bool auto_is_tensor(int D, int K) { return tc_supports(D, K) && K >= 64 && D >= 8; }
// AUTO also uses the tensor-core assignment for the larger K that only the assignment kernels take: planes are needed then
// (and for D > 128 the two-sweep tensor path, which needs its own planes)
bool auto_wants_planes(int D, int K) { return (tc_assign_supports(D, K) && K >= 64 && D >= 8) || (wide_supports(D, K) && K >= 64); }
// Points per component from which AUTO takes the tensor path for D > 128.  Its logits carry an error of a few 1e-4 in the
// log2 domain (fp32 accumulators of magnitude ~100, truncated at every step), which the averaging over a component's
// points must absorb; components expected to hold fewer than wide_min_points (64) points are evaluated exactly, and
// with fewer than about twice that per component on average most components would be.
constexpr int64_t WIDE_AUTO_MIN_POINTS_PER_COMPONENT = 128;

int ensure_scratch(gmm_ctx* ctx, int D, int K) {
    const bool planes = (tc_assign_supports(D, K) || wide_supports(D, K)) &&
                        (ctx->path == GMM_PATH_TENSOR || (ctx->path == GMM_PATH_AUTO && auto_wants_planes(D, K)));
    if (ctx->scratch && D == ctx->capD && K == ctx->capK && planes == ctx->capPlanes) return GMM_OK;
    const ScratchLayout L = scratch_layout(D, K, planes);
    if (ctx->scratch) {
        // The status word moves with the layout: what asynchronous calls may have left in it is kept on the host.
        int st = 0;
        CU(cudaMemcpyAsync(&st, &ctx->result()->status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
        ctx->sticky_status |= st;
    }
    if (L.total > ctx->scratch_bytes) {
        if (ctx->scratch) {
            CU(cudaFree(ctx->scratch));
            ctx->scratch = nullptr;
            ctx->scratch_bytes = 0;
        }
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, L.total);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(ctx, GMM_ENOMEM, "cannot allocate %zu bytes of scratch: %s", L.total, cudaGetErrorString(e));
        }
        ctx->scratch = static_cast<unsigned char*>(p);
        ctx->scratch_bytes = L.total;
    }
    ctx->lay = L;
    ctx->capD = D;
    ctx->capK = K;
    ctx->capPlanes = planes;
    CU(cudaMemsetAsync(ctx->result(), 0, sizeof(DevResult), ctx->stream));
    ctx->tc_Q = 0;
    CU(cudaDeviceGetAttribute(&ctx->sms, cudaDevAttrMultiProcessorCount, ctx->device));
    if (L.tc && tc_supports(D, K)) {
        int q = 0;
        CU(tc_max_clusters(D, K, &q));
        const TcPlan pl = tc_plan(D, K, 160);
        if (q > pl.Q) q = pl.Q;
        ctx->tc_Q = q;
    }
    return GMM_OK;
}

int check_shape(gmm_ctx* ctx, int64_t N, int D, int K) {
    if (!ctx) return GMM_EINVAL;
    if (N < 1 || D < 1 || K < 1) return fail(ctx, GMM_EINVAL, "N, D and K must be >= 1 (got N=%lld D=%d K=%d)", (long long)N, D, K);
    if ((int64_t)K * D > ((int64_t)1 << 28)) return fail(ctx, GMM_EINVAL, "K*D too large (%lld)", (long long)K * D);
    return GMM_OK;
}

int check_ptr(gmm_ctx* ctx, const void* p, size_t align, const char* name) {
    if (!p) return fail(ctx, GMM_EINVAL, "%s is NULL", name);
    if (reinterpret_cast<uintptr_t>(p) % align) return fail(ctx, GMM_EALIGN, "%s is not %zu-byte aligned", name, align);
    return GMM_OK;
}

#define CHECK(expr)            \
    do {                       \
        int rc_ = (expr);      \
        if (rc_ != GMM_OK) return rc_; \
    } while (0)

int prof_begin(gmm_ctx* ctx) {
    if (!ctx->profiling) return GMM_OK;
    if (!ctx->ev_created) {
        for (int i = 0; i < EVENT_POOL; ++i) {
            CU(cudaEventCreate(&ctx->ev_a[i]));
            CU(cudaEventCreate(&ctx->ev_b[i]));
        }
        ctx->ev_created = true;
    }
    if (ctx->ev_used == EVENT_POOL) {
        CU(cudaStreamSynchronize(ctx->stream));
        for (int i = 0; i < ctx->ev_used; ++i) {
            float ms = 0.f;
            CU(cudaEventElapsedTime(&ms, ctx->ev_a[i], ctx->ev_b[i]));
            ctx->prof_ms += ms;
        }
        ctx->ev_used = 0;
    }
    CU(cudaEventRecord(ctx->ev_a[ctx->ev_used], ctx->stream));
    return GMM_OK;
}

int prof_end(gmm_ctx* ctx) {
    if (!ctx->profiling) return GMM_OK;
    CU(cudaEventRecord(ctx->ev_b[ctx->ev_used], ctx->stream));
    ctx->ev_used++;
    ctx->prof_launches++;
    return GMM_OK;
}

// Derived per-component constants for both paths; validates the parameters into the status word.  Then picks the
// path: the tensor-core path whenever the shape allows it (ill-conditioned components are handled inside its kernel).
// Marked pairs per point up to which the screening mode is the cheaper way through a step on wide data (see the comment in
// prepare_and_choose): against the two tensor sweeps, or (dense = true) against the FP32 kernels over all listed components.
double wide_pair_limit(int n_list, int D, bool dense) {
    const double kd = (double)n_list * D;
    const double saved = (dense ? 5.0e-4 : 3.3e-5) * kd - 3.6e-6 * kd - 5.0;
    return saved > 0.0 ? saved / (1.0 + 3.4e-3 * D) : 0.0;
}

int prepare_and_choose(gmm_ctx* ctx, int64_t N, int D, int K, const float* pi, const float* mu, const float* var,
                       int* path, const float* Xprobe = nullptr, int64_t n_probe = 0) {
    KL(launch_prepare_fp32(ctx->stream, D, K, pi, mu, var, ctx->w2(), ctx->c2(), ctx->c2d(), ctx->center(), &ctx->result()->status));
    if ((size_t)K * D > ((size_t)1 << 12)) ctx->launches++;      // but for tiny problems, the centre of the means is a launch of its own
    if (wide_supports(D, K)) {
        // D > 128, K >= 64 (or forced): the tensor path for wide data, in one of two modes.
        //   "screen"  one tensor sweep over all components only SCREENS the (point, component) pairs - it marks those whose
        //             approximate log2 z, with its error bound, can come within 2^-40 of the point's best - and every marked
        //             pair is evaluated exactly in fp32.  On wide data posteriors are sparse (a few pairs per point), so
        //             this is both the faster and the more accurate mode.  Xprobe (device rows of this step's data, may be
        //             NULL) lets the automatic choice try it on a sample first.
        //   "sweeps"  the two sweeps of Algorithm 1 on the tensor cores, with only the ill-conditioned and light components
        //             evaluated exactly: for data whose posteriors are broad (many marked pairs per point).  Needs 128
        //             points per component under AUTO (with fewer, most components would be "light").
        // Parameter sets with too many ill-conditioned components for "sweeps" go to the FP32 kernels.  The flags come
        // back through small synchronisations (two or three per step, against a second of compute at these shapes).
        const bool want = ctx->lay.wide && (ctx->path == GMM_PATH_TENSOR || (ctx->path == GMM_PATH_AUTO && K >= 64));
        *path = GMM_PATH_FP32;
        ctx->wide_screen_all = false;
        if (!want) return GMM_OK;
        float limit = ctx->tc_cond_limit;
        if (limit < 0.f) limit = ctx->tc_cond_scale * std::sqrt((float)((double)N / (double)K));
        const WideBuffers wb = ctx->wide();
        int fl[8];
        const bool can_probe = Xprobe != nullptr && n_probe >= 1;
        // Automatic choice, step by step: the screening sweep and its filter are tried on the first 8192 rows, and "screen" is
        // taken if they mark few enough pairs per point.  Costs per point, measured at config 5's shape and checked at
        // five others (K 64-4096, D 200-1024): "screen" 5 ns + 3.6e-6 K D ns (norm, filter, the pair kernels' fixed part;
        // the leading-product sweep) + (1 + 3.4e-3 D) ns per marked pair (nearly every marked pair is kept: its exact value
        // and its statistics); "sweeps" 3.3e-5 K D ns; the FP32 kernels 5e-4 K D ns.  From 128 points per component on the
        // alternative is "sweeps" (limit 24 marked pairs per point at config 5, whose iterations from a data-row
        // initialisation mark 12, 30, 11, 4.5, 3.3, 2.9; none at K D below 170,000, where "sweeps" costs less than the pair
        // kernels' fixed part); below, where "sweeps" would list most components as light, the FP32 kernels.
        const bool few_points = N < WIDE_AUTO_MIN_POINTS_PER_COMPONENT * K;
        if (ctx->wide_mode == 2 || (ctx->wide_mode == 0 && can_probe)) {
            KL(launch_prepare_wide(ctx->stream, D, K, pi, mu, var, wb, limit, INFINITY, ctx->wide_hi == 2 ? 3 : ctx->wide_hi ? 1 : 0));      // every component is listed
            ctx->launches += 4;
            CU(cudaMemcpyAsync(fl, wb.flags, sizeof(fl), cudaMemcpyDeviceToHost, ctx->stream));
            CU(cudaStreamSynchronize(ctx->stream));
            const int n_list = fl[2];
            bool ok = n_list >= 1 && fl[4] + 64 <= WIDE_MAX_ILL;
            if (ok) KL(launch_ill_gather_wide(ctx->stream, D, n_list, wb, mu, ctx->w2(), ctx->c2d()));
            if (ok && ctx->wide_mode == 0) {
                // the first rows of the data through the screening sweep: how many pairs per point does it mark?
                const int64_t np = n_probe < 8192 ? n_probe : 8192;
                CU(launch_cand_clear_wide(ctx->stream, np, n_list, wb));
                KL(launch_transform_wide(ctx->stream, Xprobe, np, D, wb, &ctx->result()->status, ctx->wide_hi == 2, true));
                KL(launch_lse_wide(ctx->stream, np, D, K, fl[6], fl[4], n_list, wb, ctx->sms, &ctx->result()->status, 2, ctx->wide_hi == 2 ? 0 : ctx->wide_hi ? fl[5] : -1, ctx->wide_pre, true, true));
                KL(launch_cand_filter_wide(ctx->stream, np, n_list, wb));
                int marks = 0;
                CU(cudaMemcpyAsync(&marks, wb.ctl, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
                CU(cudaStreamSynchronize(ctx->stream));
                const double auto_limit = wide_pair_limit(n_list, D, few_points);
                ok = (double)marks <= (ctx->wide_probe_limit > 0.0 ? ctx->wide_probe_limit : auto_limit) * (double)np;
            }
            if (ok) {
                ctx->wide_n_ill = fl[4];
                ctx->wide_n_good = fl[6];
                ctx->wide_n_list = n_list;
                ctx->wide_n_first = fl[5] < n_list ? fl[5] : n_list;
                ctx->wide_screen_all = true;
                *path = GMM_PATH_TENSOR;
                return GMM_OK;
            }
        }
        if (!(ctx->path == GMM_PATH_TENSOR || N >= WIDE_AUTO_MIN_POINTS_PER_COMPONENT * K)) return GMM_OK;
        KL(launch_prepare_wide(ctx->stream, D, K, pi, mu, var, wb, limit, (float)((double)ctx->wide_min_points / (double)N)));
        ctx->launches += 4;
        // how many components were flagged, the length of their list and how many are left to the tensor passes
        CU(cudaMemcpyAsync(fl, wb.flags, sizeof(fl), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
        const int n_ill = fl[4];
        ctx->wide_n_ill = n_ill;
        ctx->wide_n_good = fl[6];
        if (n_ill + 64 > WIDE_MAX_ILL || 2 * n_ill > K || fl[6] < 1) return GMM_OK;     // too many: the FP32 kernels take the whole step
        if (n_ill > 0) {
            // The flagged components take no part in the tensor passes: they are evaluated exactly as a packed sub-mixture,
            // pair by pair where sweep 1 finds that a pair can matter, or densely by the FP32 kernels (a collapsed component
            // is hopeless for every point but its own, which those kernels notice after the first 32 dimensions of a tile).
            // (the list has a gap of empty slots between its two kinds of components)
            const int n_list = fl[2];
            ctx->wide_n_list = n_list;
            ctx->wide_n_first = fl[5] < n_list ? fl[5] : n_list;
            KL(launch_ill_gather_wide(ctx->stream, D, n_list, wb, mu, ctx->w2(), ctx->c2d()));
        }
        *path = GMM_PATH_TENSOR;
        return GMM_OK;
    }
    const bool tc_ok = ctx->lay.tc && ctx->tc_Q >= 1;
    const bool tc_auto = tc_ok && gmm_auto_path(D, K) == GMM_PATH_TENSOR;
    if (ctx->path == GMM_PATH_TENSOR && !tc_ok)
        return fail(ctx, GMM_EUNSUPPORTED, "the tensor-core path needs D <= %d and K <= 4096 (got D=%d K=%d)", WIDE_MAX_D, D, K);
    if (ctx->path == GMM_PATH_FP32 || !tc_ok || (ctx->path == GMM_PATH_AUTO && !tc_auto)) {
        *path = GMM_PATH_FP32;
        return GMM_OK;
    }
    // Components whose estimated logit error exceeds the limit get their competitive logits recomputed exactly.  The
    // error a responsibility may carry shrinks with the number of points that average it out, so the limit follows
    // sqrt(points per component): parameter errors stay below 1e-4 of the data scale at any N / K.
    float limit = ctx->tc_cond_limit;
    if (limit < 0.f) limit = ctx->tc_cond_scale * std::sqrt((float)((double)N / (double)K));
    // The log-likelihood sums a component's error over its points instead of averaging it out.  The points' log2 Z are
    // about 0.72 D in size, so for small D (where little else is large) the limit is capped at 4e-5 D, which keeps the
    // log-likelihood within 1e-5 relative; at D >= 32 typical estimates (1e-3) are 1e-5 of log2 Z without a cap.
    if (ctx->tc_cond_limit < 0.f && D < 32) limit = std::fmin(limit, 4e-5f * (float)D);
    KL(launch_prepare_tc(ctx->stream, D, K, pi, mu, var, ctx->tc(), limit, &ctx->result()->status));
    ctx->launches += 2;   // launch_prepare_tc enqueues three kernels
    // the number of ill-conditioned components travels back with the result: the next step picks its filter by it
    CU(cudaMemcpyAsync(&ctx->result()->n_ill, ctx->tc().flags + 4, sizeof(int), cudaMemcpyDeviceToDevice, ctx->stream));
    *path = GMM_PATH_TENSOR;
    return GMM_OK;
}

// Adds the statistics of n device-resident points to (Nk, S1, S2) and their log-likelihood to result()->ll[slot].
int accumulate_points(gmm_ctx* ctx, int path, const float* X, int64_t n, int D, int K, const float* mu, double* Nk,
                      double* S1, double* S2, int slot) {
    if (path == GMM_PATH_TENSOR && wide_supports(D, K)) {
        // Two sweeps per piece of at most 2^17 points (the capacity of the planes of Y and of the log2 Z buffer): planes,
        // log-sum-exp, responsibilities + statistics into per-CTA fp32 partials, which are folded into the float64
        // statistics piece by piece (no fp32 chain longer than a piece's batches).
        const WideBuffers wb = ctx->wide();
        const int n_ill = ctx->wide_n_ill > 0 ? ctx->wide_n_list : 0;      // slots of the packed sub-mixture
        // The sub-mixture's M-step runs as two launches, one per kind of component: tiles of collapsed components leave after
        // their first chunk of dimensions, so a grid shared with the broad ones would leave most of its CTAs idle.  Each
        // launch has its own plan; their float64 partials share the FP32 path's partial buffer (sized for all K components).
        const int n_a = n_ill > 0 ? ctx->wide_n_first : 0, n_b = n_ill - n_a;
        Fp32Plan plan_a = fp32_plan(D, n_a > 0 ? n_a : 1), plan_b = fp32_plan(D, n_b > 0 ? n_b : 1);
        if (n_ill > 0) {
            const size_t cap = fp32_partial_floats(D, K) * sizeof(float);
            auto fit = [&](Fp32Plan& pl, int kk) {
                const size_t per_split = ((size_t)kk + 2 * (size_t)kk * D) * sizeof(double);
                while (pl.splits > 1 && (size_t)pl.splits * per_split > cap) --pl.splits;
            };
            if (n_a > 0) fit(plan_a, n_a);
            if (n_b > 0) fit(plan_b, n_b);
            CU(cudaMemsetAsync(wb.stats_c, 0, ((size_t)n_ill + 2 * (size_t)n_ill * D) * sizeof(double), ctx->stream));
        }
        CU(cudaMemsetAsync(wb.llpart, 0, 256 * 8, ctx->stream));
        const int Kg = ctx->wide_n_good;
        const int n_listed = n_ill > 0 ? ctx->wide_n_ill : 0;
        const bool all = ctx->wide_screen_all;                              // "screen" mode: no component is left to sweep 2
        const bool screen = n_ill > 0 && (ctx->wide_sparse != 0 || all);
        const int* dense_if = screen ? wb.ctl + 1 : nullptr;             // the dense kernels run when the gate says so
        for (int64_t off = 0; off < n; off += ctx->wide_piece) {
            const int64_t cnt = (n - off < ctx->wide_piece) ? (n - off) : ctx->wide_piece;
            const float* Xs = X + off * D;
            if (!all) CU(cudaMemsetAsync(wb.partial, 0, ctx->lay.w_partial_bytes, ctx->stream));
            if (screen) CU(launch_cand_clear_wide(ctx->stream, cnt, n_ill, wb));
            CHECK(prof_begin(ctx));
            KL(launch_transform_wide(ctx->stream, Xs, cnt, D, wb, &ctx->result()->status, all && ctx->wide_hi == 2, screen));
            KL(launch_lse_wide(ctx->stream, cnt, D, K, Kg, screen ? n_listed : 0, n_ill, wb, ctx->sms, &ctx->result()->status, 2,
                               !(all && ctx->wide_hi) ? -1 : ctx->wide_hi == 2 ? 0 : ctx->wide_n_first, ctx->wide_pre, true, all));
            if (screen) KL(launch_cand_filter_wide(ctx->stream, cnt, n_ill, wb));
            if (ctx->wide_refine && !all) KL(launch_refine_wide(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), wb));
            else CU(cudaMemcpyAsync(wb.logz_x, wb.logz, (size_t)cnt * 8, cudaMemcpyDeviceToDevice, ctx->stream));
            if (n_ill > 0) {
                if (screen) {
                    // more than one pair in 64 marked (or the pair-by-pair route switched off): the dense kernels are cheaper
                    // ("screen" mode: the dense alternative evaluates every component, so the pair route pays for longer)
                    const long long max_pairs = ctx->wide_sparse >= 2 ? ((long long)1 << 62)
                                              : all ? (long long)((double)cnt * wide_pair_limit(n_ill, D, true)) : (long long)cnt * n_ill / 64;
                    KL(launch_cand_gate_wide(ctx->stream, wb, max_pairs));
                    KL(launch_cand_lse_wide(ctx->stream, Xs, cnt, D, n_ill, wb, ctx->logZ2()));
                }
                KL(launch_lse_fp32(ctx->stream, Xs, cnt, D, n_ill, wb.mu_c, wb.w2_c, wb.c2d_c, ctx->center(), ctx->logZ2(), nullptr, wb.logz, dense_if));
            }
            KL(launch_merge_ll_wide(ctx->stream, cnt, wb, n_ill > 0 ? ctx->logZ2() : nullptr));
            if (!all) KL(launch_em_wide(ctx->stream, cnt, D, K, Kg, wb, ctx->sms, &ctx->result()->status));
            if (!all) KL(launch_reduce_wide(ctx->stream, D, K, Kg, wb, ctx->sms, Nk, S1, S2));
            if (n_ill > 0) {
                double* Nk_c = wb.stats_c;
                double* S1_c = Nk_c + n_ill;
                double* S2_c = S1_c + (size_t)n_ill * D;
                if (screen) {
                    KL(launch_cand_mstep_wide(ctx->stream, Xs, cnt, D, n_ill, wb));
                    ctx->launches += 2;
                }
                if (n_a > 0) {
                    KL(launch_mstep_fp32(ctx->stream, Xs, cnt, D, n_a, wb.mu_c, wb.w2_c, wb.c2d_c, ctx->center(), wb.logz_x, ctx->partials(), plan_a, true, dense_if));
                    KL(launch_reduce_partials(ctx->stream, D, n_a, plan_a.splits, ctx->partials(), ctx->center(), Nk_c, S1_c, S2_c, true, dense_if));
                }
                if (n_b > 0) {
                    const size_t o = (size_t)n_a * D;
                    KL(launch_mstep_fp32(ctx->stream, Xs, cnt, D, n_b, wb.mu_c + o, wb.w2_c + o, wb.c2d_c + n_a, ctx->center(), wb.logz_x, ctx->partials(), plan_b, true, dense_if));
                    KL(launch_reduce_partials(ctx->stream, D, n_b, plan_b.splits, ctx->partials(), ctx->center(), Nk_c + n_a, S1_c + o, S2_c + o, true, dense_if));
                }
                if (screen) KL(launch_cand_count_wide(ctx->stream, n_ill, wb));
            }
            CHECK(prof_end(ctx));                             // (the bracket holds every kernel of the piece)
        }
        if (n_ill > 0) KL(launch_ill_scatter_wide(ctx->stream, D, K, n_ill, wb, Nk, S1, S2));
        KL(launch_reduce_ll(ctx->stream, wb.llpart, WIDE_LL_BLOCKS, &ctx->result()->ll[slot], true));
        return GMM_OK;
    }
    if (path == GMM_PATH_TENSOR) {
        const TcBuffers tb = ctx->tc();
        const TcPlan pl = tc_plan(D, K, 160);
        const int Q = ctx->tc_Q;
        // Which filter the tile kernel applies to ill-conditioned components (both are correct on any input).  With few
        // points per component the flagged components are mostly narrow in a few dimensions, the test on their error
        // bound passes nearly every pair and the exact test on their decisive dimensions pays; with many points per
        // component they are collapsed singletons that the error-bound test already discards.  Decided from the count of
        // the last preparation whose result was read back (none yet: the plain filter).
        bool tight = ctx->tc_n_ill > 0 && (n < (int64_t)512 * K || (int64_t)ctx->tc_n_ill * 8 > K);
        if (ctx->tc_force_filter >= 0) tight = ctx->tc_force_filter == 1;
        CU(cudaMemsetAsync(tb.partial, 0, (size_t)Q * pl.Kpad * TC_PCOLS * 8, ctx->stream));
        CU(cudaMemsetAsync(tb.llpart, 0, (size_t)Q * 16, ctx->stream));
        // The fp16 planes of Y are built once per launch-sized piece of X (not once per CTA of a group), so the tile kernel
        // is launched per piece; its float64 partials and log-likelihood partials accumulate across the launches.
        for (int64_t off = 0; off < n; off += ctx->tc_piece) {
            const int64_t cnt = (n - off < ctx->tc_piece) ? (n - off) : ctx->tc_piece;
            const float* Xs = X + off * D;
            CHECK(prof_begin(ctx));
            KL(launch_transform_tc(ctx->stream, Xs, cnt, D, tb, &ctx->result()->status));
            KL(launch_em_tc(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2(), tb, Q, ctx->tc_flush, tight, &ctx->result()->status));
            CHECK(prof_end(ctx));
        }
        KL(launch_reduce_ll(ctx->stream, tb.llpart, 2 * Q, &ctx->result()->ll[slot], true));
        KL(launch_reduce_tc(ctx->stream, D, K, Q, tb, Nk, S1, S2, true));
        return GMM_OK;
    }
    const Fp32Plan plan = fp32_plan(D, K);
    for (int64_t off = 0; off < n; off += SUPER_TILE) {
        const int64_t cnt = (n - off < SUPER_TILE) ? (n - off) : SUPER_TILE;
        const float* Xs = X + off * D;
        CHECK(prof_begin(ctx));
        KL(launch_lse_fp32(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), ctx->logZ2(), ctx->llpart()));
        KL(launch_mstep_fp32(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), ctx->logZ2(), ctx->partials(), plan));
        CHECK(prof_end(ctx));
        KL(launch_reduce_ll(ctx->stream, ctx->llpart(), (cnt + FP32_TILE_P - 1) / FP32_TILE_P, &ctx->result()->ll[slot], true));
        KL(launch_reduce_partials(ctx->stream, D, K, plan.splits, ctx->partials(), ctx->center(), Nk, S1, S2, true));
    }
    return GMM_OK;
}

int zero_stats(gmm_ctx* ctx, int D, int K, double* Nk, double* S1, double* S2, int slot) {
    const size_t KD = (size_t)K * D;
    CU(cudaMemsetAsync(Nk, 0, (size_t)K * 8, ctx->stream));
    CU(cudaMemsetAsync(S1, 0, KD * 8, ctx->stream));
    CU(cudaMemsetAsync(S2, 0, KD * 8, ctx->stream));
    CU(cudaMemsetAsync(&ctx->result()->ll[slot], 0, 8, ctx->stream));
    return GMM_OK;
}

// The status word is sticky: device code ORs error bits into it and nothing clears it until the host has reported
// them, so an error raised by an asynchronous call (gmm_assign_topm, gmm_finalize) surfaces at the next synchronising
// call or at gmm_sync_status.  Called with the stream synchronised and `status` = the word as read from the device.
int report_status(gmm_ctx* ctx, int status) {
    status |= ctx->sticky_status;
    if (status == 0) return GMM_OK;
    ctx->sticky_status = 0;
    CU(cudaMemsetAsync(&ctx->result()->status, 0, sizeof(int), ctx->stream));
    if (status & ST_TIMEOUT) return fail(ctx, GMM_ETIMEOUT, "a bounded device-side wait expired (in this call or an earlier asynchronous one)");
    if (status & ST_BAD_VAR) return fail(ctx, GMM_ENUMERIC, "var must be finite and > 0 (in this call or an earlier asynchronous one)");
    if (status & ST_BAD_PI) return fail(ctx, GMM_ENUMERIC, "pi must be finite and >= 0 (in this call or an earlier asynchronous one)");
    if (status & ST_BAD_X) return fail(ctx, GMM_ENUMERIC, "X holds a non-finite value (in this call or an earlier asynchronous one)");
    return fail(ctx, GMM_ENUMERIC, "non-finite parameter (in this call or an earlier asynchronous one)");
}

// Synchronising read of the log-likelihood slot and the status word.
int read_result(gmm_ctx* ctx, int slot, double* loglik) {
    DevResult r;
    CU(cudaMemcpyAsync(&r, ctx->result(), sizeof(DevResult), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    CHECK(report_status(ctx, r.status));
    ctx->tc_n_ill = r.n_ill;
    *loglik = r.ll[slot];
    if (!std::isfinite(*loglik)) return fail(ctx, GMM_ENUMERIC, "log-likelihood is not finite (%g): non-finite values in X?", *loglik);
    return GMM_OK;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" {

int gmm_create(gmm_ctx** out, int device, void* cuda_stream) {
    if (!out) return GMM_EINVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return GMM_ECUDA;
    }
    gmm_ctx* ctx = new (std::nothrow) gmm_ctx();
    if (!ctx) return GMM_ENOMEM;
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    if (const char* e = std::getenv("GMM_TC_COND_LIMIT")) ctx->tc_cond_limit = (float)std::atof(e);
    if (const char* e = std::getenv("GMM_TC_FILTER")) ctx->tc_force_filter = (e[0] == 't') ? 1 : (e[0] == 'p' ? 0 : -1);
    if (const char* e = std::getenv("GMM_TC_FLUSH")) ctx->tc_flush = std::atoi(e);
    if (const char* e = std::getenv("GMM_WIDE_MIN_POINTS")) ctx->wide_min_points = std::atof(e);
    if (const char* e = std::getenv("GMM_WIDE_REFINE")) ctx->wide_refine = std::atoi(e) != 0;
    if (const char* e = std::getenv("GMM_WIDE_SPARSE")) ctx->wide_sparse = std::atoi(e);
    if (const char* e = std::getenv("GMM_WIDE_HI")) ctx->wide_hi = std::atoi(e);
    if (const char* e = std::getenv("GMM_WIDE_PRE")) ctx->wide_pre = std::atoi(e) != 0;
    if (const char* e = std::getenv("GMM_WIDE_MODE")) ctx->wide_mode = !std::strcmp(e, "sweeps") ? 1 : !std::strcmp(e, "screen") ? 2 : 0;
    if (const char* e = std::getenv("GMM_WIDE_PROBE_LIMIT")) ctx->wide_probe_limit = std::atof(e);
    if (const char* e = std::getenv("GMM_WIDE_PIECE")) {
        const long long v = std::atoll(e);
        if (v >= 256 && v <= WIDE_PIECE) ctx->wide_piece = v / 256 * 256;
    }
    if (const char* e = std::getenv("GMM_TC_PIECE")) {
        const long long v = std::atoll(e);
        if (v >= 64 && v <= TC_YPOINTS) ctx->tc_piece = v / 64 * 64;
    }
    {   // test hooks of the bounded-wait path, process-wide and set at every create like the issue order
        const char* r = std::getenv("GMM_TC_TEST_SILENT_RANK");
        const char* w = std::getenv("GMM_TC_TEST_WAIT_MS");
        tc_set_test_hooks(r ? std::atoi(r) : -1, w ? (unsigned long long)std::atoll(w) * 1000000ull : 0ull);
    }
    {   // the issue order is process-wide: every create sets it, so a context never inherits an earlier context's choice
        const char* e = std::getenv("GMM_TC_ORDER");
        tc_set_order(e ? std::atoi(e) : 2);
    }
    *out = ctx;
    return GMM_OK;
}

int gmm_destroy(gmm_ctx* ctx) {
    if (!ctx) return GMM_EINVAL;
    DeviceGuard g(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    if (ctx->scratch) cudaFree(ctx->scratch);
    for (int b = 0; b < 2; ++b) {
        if (ctx->xstage[b]) cudaFree(ctx->xstage[b]);
        if (ctx->ev_copied[b]) cudaEventDestroy(ctx->ev_copied[b]);
        if (ctx->ev_done[b]) cudaEventDestroy(ctx->ev_done[b]);
    }
    if (ctx->hparams) cudaFree(ctx->hparams);
    if (ctx->pl_scratch) cudaFree(ctx->pl_scratch);
    if (ctx->km_scratch) cudaFree(ctx->km_scratch);
    if (ctx->at_scratch) cudaFree(ctx->at_scratch);
    if (ctx->fv_scratch) cudaFree(ctx->fv_scratch);
    if (ctx->km_unit) cudaFree(ctx->km_unit);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->ev_created)
        for (int i = 0; i < EVENT_POOL; ++i) {
            cudaEventDestroy(ctx->ev_a[i]);
            cudaEventDestroy(ctx->ev_b[i]);
        }
    cudaGetLastError();
    delete ctx;
    return GMM_OK;
}

int gmm_set_path(gmm_ctx* ctx, int path) {
    if (!ctx) return GMM_EINVAL;
    if (path != GMM_PATH_AUTO && path != GMM_PATH_FP32 && path != GMM_PATH_TENSOR)
        return fail(ctx, GMM_EINVAL, "unknown path %d", path);
    ctx->path = path;
    return GMM_OK;
}

int gmm_last_path(const gmm_ctx* ctx) { return ctx ? ctx->last_path : GMM_EINVAL; }

int gmm_last_exact_count(const gmm_ctx* ctx) {
    if (!ctx) return GMM_EINVAL;
    if (ctx->last_path != GMM_PATH_TENSOR) return 0;
    return wide_supports(ctx->capD, ctx->capK) ? ctx->wide_n_ill : ctx->tc_n_ill;
}

int gmm_last_exact_pairs(gmm_ctx* ctx, int64_t* marked, int64_t* kept, int* dense_pieces) {
    if (!ctx || !marked || !kept || !dense_pieces) return GMM_EINVAL;
    *marked = *kept = 0;
    *dense_pieces = 0;
    if (ctx->last_path != GMM_PATH_TENSOR || !wide_supports(ctx->capD, ctx->capK) || !ctx->lay.wide || ctx->wide_n_ill <= 0) return GMM_OK;
    int fl[8];
    CU(cudaMemcpyAsync(fl, ctx->wide().flags, sizeof(fl), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    *marked = fl[1];
    *kept = fl[3];
    *dense_pieces = fl[7];
    return GMM_OK;
}

int gmm_em_step(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* pi, const float* mu,
                const float* var, double* Nk, double* S1, double* S2, double* loglik) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X, 4, "X"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    CHECK(check_ptr(ctx, Nk, 8, "Nk"));
    CHECK(check_ptr(ctx, S1, 8, "S1"));
    CHECK(check_ptr(ctx, S2, 8, "S2"));
    if (!loglik) return fail(ctx, GMM_EINVAL, "loglik is NULL");
    DeviceGuard g(ctx->device);
    int path;
    CHECK(ensure_scratch(ctx, D, K));
    CHECK(prepare_and_choose(ctx, N, D, K, pi, mu, var, &path, X, N));
    CHECK(zero_stats(ctx, D, K, Nk, S1, S2, 0));
    CHECK(accumulate_points(ctx, path, X, N, D, K, mu, Nk, S1, S2, 0));
    ctx->last_path = path;
    return read_result(ctx, 0, loglik);
}

int gmm_finalize(gmm_ctx* ctx, int64_t N, int D, int K, const double* Nk, const double* S1, const double* S2,
                 float var_floor, float* pi, float* mu, float* var) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, Nk, 8, "Nk"));
    CHECK(check_ptr(ctx, S1, 8, "S1"));
    CHECK(check_ptr(ctx, S2, 8, "S2"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    if (!(var_floor >= 0.f)) return fail(ctx, GMM_EINVAL, "var_floor must be >= 0");
    DeviceGuard g(ctx->device);
    int* counts = ctx->scratch ? ctx->result()->counts : nullptr;
    if (counts) CU(cudaMemsetAsync(counts, 0, 2 * sizeof(int), ctx->stream));
    KL(launch_finalize(ctx->stream, N, D, K, Nk, S1, S2, var_floor, pi, mu, var, counts, nullptr, nullptr));
    return GMM_OK;
}

int gmm_set_covariance(gmm_ctx* ctx, int covariance) {
    if (!ctx) return GMM_EINVAL;
    if (covariance != GMM_COV_DIAG && covariance != GMM_COV_ISOTROPIC) return fail(ctx, GMM_EINVAL, "unknown covariance type %d", covariance);
    ctx->covariance = covariance;
    return GMM_OK;
}

int gmm_finalize_isotropic(gmm_ctx* ctx, int64_t N, int D, int K, const double* Nk, const double* S1, const double* S2,
                           float var_floor, float* pi, float* mu, float* var) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, Nk, 8, "Nk"));
    CHECK(check_ptr(ctx, S1, 8, "S1"));
    CHECK(check_ptr(ctx, S2, 8, "S2"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    if (!(var_floor >= 0.f)) return fail(ctx, GMM_EINVAL, "var_floor must be >= 0");
    DeviceGuard g(ctx->device);
    int* counts = ctx->scratch ? ctx->result()->counts : nullptr;
    if (counts) CU(cudaMemsetAsync(counts, 0, 2 * sizeof(int), ctx->stream));
    KL(launch_finalize_isotropic(ctx->stream, N, D, K, Nk, S1, S2, var_floor, pi, mu, var, counts, nullptr, nullptr));
    return GMM_OK;
}

int gmm_fit(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, float* pi, float* mu, float* var, int iters,
            float var_floor, double tol, double* loglik_trace, int* iters_done) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X, 4, "X"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    if (!loglik_trace) return fail(ctx, GMM_EINVAL, "loglik_trace is NULL");
    if (iters < 1) return fail(ctx, GMM_EINVAL, "iters must be >= 1");
    if (!(var_floor >= 0.f)) return fail(ctx, GMM_EINVAL, "var_floor must be >= 0");
    if (!(tol >= 0.0)) return fail(ctx, GMM_EINVAL, "tol must be >= 0");
    DeviceGuard g(ctx->device);
    int path;
    CHECK(ensure_scratch(ctx, D, K));
    const size_t KD = (size_t)K * D;
    double* Nk = ctx->stats();
    double* S1 = Nk + K;
    double* S2 = S1 + KD;
    int t = 0;
    for (; t < iters; ++t) {
        const int slot = t % LL_SLOTS;
        CHECK(prepare_and_choose(ctx, N, D, K, pi, mu, var, &path, X, N));
        CHECK(zero_stats(ctx, D, K, Nk, S1, S2, slot));
        CHECK(accumulate_points(ctx, path, X, N, D, K, mu, Nk, S1, S2, slot));
        // The update is skipped on the device when the step raised a status bit or left a non-finite log-likelihood
        // (invalid parameters, a time-out, non-finite data): the caller then keeps the last good parameters.
        CU(cudaMemsetAsync(ctx->result()->counts, 0, 2 * sizeof(int), ctx->stream));
        if (ctx->covariance == GMM_COV_ISOTROPIC)
            KL(launch_finalize_isotropic(ctx->stream, N, D, K, Nk, S1, S2, var_floor, pi, mu, var, ctx->result()->counts,
                                         &ctx->result()->status, &ctx->result()->ll[slot]));
        else
            KL(launch_finalize(ctx->stream, N, D, K, Nk, S1, S2, var_floor, pi, mu, var, ctx->result()->counts,
                               &ctx->result()->status, &ctx->result()->ll[slot]));
        ctx->last_path = path;
        int rc = read_result(ctx, slot, &loglik_trace[t]);
        if (rc != GMM_OK) {
            if (iters_done) *iters_done = t;
            return rc;
        }
        if (tol > 0.0 && t > 0 &&
            std::fabs(loglik_trace[t] - loglik_trace[t - 1]) <= tol * std::fabs(loglik_trace[t])) {
            ++t;
            break;
        }
    }
    if (iters_done) *iters_done = t;
    return GMM_OK;
}

int gmm_em_step_host(gmm_ctx* ctx, const float* X_host, int64_t N, int D, int K, const float* pi_host,
                     const float* mu_host, const float* var_host, double* Nk_host, double* S1_host, double* S2_host,
                     double* loglik) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X_host, 4, "X_host"));
    CHECK(check_ptr(ctx, pi_host, 4, "pi_host"));
    CHECK(check_ptr(ctx, mu_host, 4, "mu_host"));
    CHECK(check_ptr(ctx, var_host, 4, "var_host"));
    CHECK(check_ptr(ctx, Nk_host, 8, "Nk_host"));
    CHECK(check_ptr(ctx, S1_host, 8, "S1_host"));
    CHECK(check_ptr(ctx, S2_host, 8, "S2_host"));
    if (!loglik) return fail(ctx, GMM_EINVAL, "loglik is NULL");
    DeviceGuard g(ctx->device);
    int path;
    CHECK(ensure_scratch(ctx, D, K));
    const size_t KD = (size_t)K * D;
    // one-time resources of the host path.  A staging buffer holds 128 MiB of rows; on wide data a whole piece of the
    // tensor path (2^17 rows: 403 MB at D = 768), whose kernels lose a third of their speed on pieces a third the size.
    if (!ctx->copy_stream) {
        CU(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
        for (int b = 0; b < 2; ++b) {
            CU(cudaEventCreateWithFlags(&ctx->ev_copied[b], cudaEventDisableTiming));
            CU(cudaEventCreateWithFlags(&ctx->ev_done[b], cudaEventDisableTiming));
        }
    }
    size_t stage_bytes = STAGE_BYTES;
    if (ctx->lay.wide && ctx->capPlanes && ctx->path != GMM_PATH_FP32) {
        const size_t piece_bytes = align256((size_t)ctx->wide_piece * D * 4);
        if (piece_bytes > stage_bytes) stage_bytes = piece_bytes;
    }
    if (ctx->xstage_bytes < stage_bytes) {
        CU(cudaStreamSynchronize(ctx->stream));
        CU(cudaStreamSynchronize(ctx->copy_stream));
        for (int b = 0; b < 2; ++b) {
            if (ctx->xstage[b]) CU(cudaFree(ctx->xstage[b]));
            ctx->xstage[b] = nullptr;
        }
        ctx->xstage_bytes = 0;
        for (int b = 0; b < 2; ++b) {
            void* p = nullptr;
            if (cudaMalloc(&p, stage_bytes) != cudaSuccess) {
                cudaGetLastError();
                return fail(ctx, GMM_ENOMEM, "cannot allocate a %zu-byte staging buffer", stage_bytes);
            }
            ctx->xstage[b] = static_cast<float*>(p);
        }
        ctx->xstage_bytes = stage_bytes;
    }
    const size_t pfloats = (size_t)K + 2 * KD;
    if (pfloats > ctx->hparams_floats) {
        if (ctx->hparams) {
            CU(cudaStreamSynchronize(ctx->stream));
            CU(cudaFree(ctx->hparams));
            ctx->hparams = nullptr;
        }
        void* p = nullptr;
        if (cudaMalloc(&p, pfloats * 4) != cudaSuccess) {
            cudaGetLastError();
            return fail(ctx, GMM_ENOMEM, "cannot allocate the parameter copies");
        }
        ctx->hparams = static_cast<float*>(p);
        ctx->hparams_floats = pfloats;
    }
    float* pi = ctx->hparams;
    float* mu = pi + K;
    float* var = mu + KD;
    CU(cudaMemcpyAsync(pi, pi_host, (size_t)K * 4, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(mu, mu_host, KD * 4, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(var, var_host, KD * 4, cudaMemcpyHostToDevice, ctx->stream));
    double* Nk = ctx->stats();
    double* S1 = Nk + K;
    double* S2 = S1 + KD;
    const int64_t rows_per_chunk = (int64_t)(ctx->xstage_bytes / ((size_t)D * 4));
    if (rows_per_chunk < 1) return fail(ctx, GMM_EINVAL, "D too large for the staging buffer");
    // The first chunk is on its way before the parameters are prepared: on wide data the automatic choice of the mode
    // looks at its first rows.  (The copy stream must not overtake work of an earlier call that still reads the buffer.)
    CU(cudaEventRecord(ctx->ev_done[0], ctx->stream));
    CU(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[0], 0));
    const int64_t cnt0 = N < rows_per_chunk ? N : rows_per_chunk;
    CU(cudaMemcpyAsync(ctx->xstage[0], X_host, (size_t)cnt0 * D * 4, cudaMemcpyHostToDevice, ctx->copy_stream));
    CU(cudaEventRecord(ctx->ev_copied[0], ctx->copy_stream));
    CU(cudaStreamWaitEvent(ctx->stream, ctx->ev_copied[0], 0));
    CHECK(prepare_and_choose(ctx, N, D, K, pi, mu, var, &path, ctx->xstage[0], cnt0));
    CHECK(zero_stats(ctx, D, K, Nk, S1, S2, 0));
    int c = 0;
    for (int64_t off = 0; off < N; off += rows_per_chunk, ++c) {
        const int b = c & 1;
        const int64_t cnt = (N - off < rows_per_chunk) ? (N - off) : rows_per_chunk;
        if (c > 0) {
            if (c >= 2) CU(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[b], 0));
            CU(cudaMemcpyAsync(ctx->xstage[b], X_host + off * D, (size_t)cnt * D * 4, cudaMemcpyHostToDevice, ctx->copy_stream));
            CU(cudaEventRecord(ctx->ev_copied[b], ctx->copy_stream));
            CU(cudaStreamWaitEvent(ctx->stream, ctx->ev_copied[b], 0));
        }
        CHECK(accumulate_points(ctx, path, ctx->xstage[b], cnt, D, K, mu, Nk, S1, S2, 0));
        CU(cudaEventRecord(ctx->ev_done[b], ctx->stream));
    }
    CU(cudaMemcpyAsync(Nk_host, Nk, (size_t)K * 8, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaMemcpyAsync(S1_host, S1, KD * 8, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaMemcpyAsync(S2_host, S2, KD * 8, cudaMemcpyDeviceToHost, ctx->stream));
    ctx->last_path = path;
    return read_result(ctx, 0, loglik);
}

namespace {
int grow_buffer(gmm_ctx* ctx, void** buf, size_t* have, size_t need, const char* what);
}

namespace {
int assign_topm_impl(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* pi, const float* mu,
                     const float* var, int m, int32_t* idx, float* resp, bool index_only = false);
}

int gmm_assign_topm(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* pi, const float* mu,
                    const float* var, int m, int32_t* idx, float* resp) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X, 4, "X"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    CHECK(check_ptr(ctx, idx, 4, "idx"));
    if (resp) CHECK(check_ptr(ctx, resp, 4, "resp"));
    if (m < 1 || m > K || m > GMM_MAX_TOPM) return fail(ctx, GMM_EINVAL, "m must be in [1, min(K, %d)] (got %d)", GMM_MAX_TOPM, m);
    DeviceGuard g(ctx->device);
    CHECK(ensure_scratch(ctx, D, K));
    return assign_topm_impl(ctx, X, N, D, K, pi, mu, var, m, idx, resp, resp == nullptr);
}

namespace {
// The assignment pass proper (arguments checked, scratch in place); also the nearest-centroid search of the k-means step.
int assign_topm_impl(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* pi, const float* mu,
                     const float* var, int m, int32_t* idx, float* resp, bool index_only) {
    KL(launch_prepare_fp32(ctx->stream, D, K, pi, mu, var, ctx->w2(), ctx->c2(), ctx->c2d(), ctx->center(), &ctx->result()->status));
    if ((size_t)K * D > ((size_t)1 << 12)) ctx->launches++;      // but for tiny problems, the centre of the means is a launch of its own
    // Tensor-core assignment where the E+M step would take the tensor path too.  Ill-conditioned components are evaluated
    // exactly for every point; parameters with more than TC_MAX_ILL of them (a flag written on the device by the
    // preparation kernels) go through the FP32 kernels instead: both sets of kernels are enqueued and each checks the
    // flag, so the call stays asynchronous.
    if (wide_supports(D, K)) {
        // Wide data: the first sweep of the two-sweep tensor path reports every point's m + 2 largest approximate values and
        // marks the listed (ill-conditioned) components that can matter; a warp per point then evaluates those exactly.  Rows
        // whose answer is not certain, pieces with too many marked pairs, and parameter sets with too many listed components
        // go through the FP32 kernels.
        const bool want = ctx->capPlanes && ctx->lay.wide && ctx->path != GMM_PATH_FP32 && K >= 64 && m + 2 <= WIDE_MAX_TOP;
        bool tensor_w = false;
        // The hard assignment (m = 1, indices only) by the EM step's screening machinery: every component listed, one sweep
        // over the leading product marks the pairs that can come within 2^-40 of a point's best, the filter drops those
        // that the final threshold rules out, and a warp per point evaluates the rest exactly and takes the largest.  No
        // row is left uncertain.  Taken when the first 8192 rows mark few pairs (half the EM step's limit: a pair costs 2 ns, the
        // route below 30 ns per point at config 5's shape); the same limit, per piece, sends a piece to the FP32 kernels.
        // The general top-m goes the same way: the marked pairs hold every component within 2^-40 of the point's best, their
        // exact values give the leading ranks and the responsibilities; ranks beyond them (responsibility 0) are filled from
        // the candidates the sweep reports (the blocks of 32 components with the largest upper bounds).
        if (want && ctx->wide_hi == 2 && ctx->wide_mode != 1) {
            const bool argmax = index_only && m == 1;
            const WideBuffers wb = ctx->wide();
            float limit = ctx->tc_cond_limit;
            if (limit < 0.f) limit = ctx->tc_cond_scale * std::sqrt((float)((double)N / (double)K));
            KL(launch_prepare_wide(ctx->stream, D, K, pi, mu, var, wb, limit, INFINITY, 3));
            ctx->launches += 4;
            int fl[8];
            CU(cudaMemcpyAsync(fl, wb.flags, sizeof(fl), cudaMemcpyDeviceToHost, ctx->stream));
            CU(cudaStreamSynchronize(ctx->stream));
            const int n_list = fl[2], n_ill = fl[4], Kg = fl[6];
            bool ok = n_list >= 1 && n_ill + 64 <= WIDE_MAX_ILL;
            if (ok) {
                KL(launch_ill_gather_wide(ctx->stream, D, n_list, wb, mu, ctx->w2(), ctx->c2d()));
                const int ntop = argmax ? 2 : (m + 2 <= 6) ? 6 : WIDE_MAX_TOP;
                auto screen_piece = [&](const float* Xs, int64_t cnt) -> int {
                    CU(launch_cand_clear_wide(ctx->stream, cnt, n_list, wb));
                    KL(launch_transform_wide(ctx->stream, Xs, cnt, D, wb, &ctx->result()->status, true, true));
                    KL(launch_lse_wide(ctx->stream, cnt, D, K, Kg, n_ill, n_list, wb, ctx->sms, &ctx->result()->status, ntop, 0, false, true, true,
                                       argmax ? 0 : m));
                    KL(launch_cand_filter_wide(ctx->stream, cnt, n_list, wb));
                    return GMM_OK;
                };
                // (a pair costs 2 ns, the route below 30-60 ns per point at config 5's shape)
                const double per_point = ctx->wide_probe_limit > 0.0 ? ctx->wide_probe_limit : 0.5 * wide_pair_limit(n_list, D, false);
                int32_t* unc_rows = nullptr;
                int* unc_count = nullptr;
                if (!argmax) {
                    const int64_t cap = N < ctx->wide_piece ? N : ctx->wide_piece;
                    const size_t need = align256((size_t)cap * sizeof(int32_t)) + 256;       // rows with fewer than m finite values, their count
                    CHECK(grow_buffer(ctx, &ctx->at_scratch, &ctx->at_scratch_bytes, need, "the assignment's list of uncertain rows"));
                    unsigned char* base = static_cast<unsigned char*>(ctx->at_scratch);
                    unc_rows = reinterpret_cast<int32_t*>(base);
                    unc_count = reinterpret_cast<int*>(base + need - 256);
                }
                if (ctx->wide_mode != 2) {
                    const int64_t np = N < 8192 ? N : 8192;
                    CHECK(screen_piece(X, np));
                    int marks = 0;
                    CU(cudaMemcpyAsync(&marks, wb.ctl, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
                    CU(cudaStreamSynchronize(ctx->stream));
                    ok = (double)marks <= per_point * (double)np;
                }
                if (ok) {
                    const int64_t piece = ctx->wide_piece;
                    for (int64_t off = 0; off < N; off += piece) {
                        const int64_t cnt = (N - off < piece) ? (N - off) : piece;
                        const float* Xs = X + off * D;
                        CHECK(prof_begin(ctx));
                        CHECK(screen_piece(Xs, cnt));
                        KL(launch_cand_gate_wide(ctx->stream, wb, ctx->wide_sparse >= 2 ? ((long long)1 << 62) : (long long)((double)cnt * per_point)));
                        int32_t* idx_p = idx + off * m;
                        float* resp_p = resp ? resp + off * m : nullptr;
                        if (argmax) {
                            KL(launch_cand_lse_wide(ctx->stream, Xs, cnt, D, n_list, wb, ctx->logZ2(), idx_p));
                        } else {
                            CU(cudaMemsetAsync(unc_count, 0, sizeof(int), ctx->stream));
                            KL(launch_cand_topm_wide(ctx->stream, Xs, cnt, D, n_list, wb, m, idx_p, resp_p, unc_rows, unc_count, ntop));
                            KL(launch_topm_fp32(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m, idx_p, resp_p, nullptr, unc_rows, unc_count));
                        }
                        KL(launch_topm_fp32(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m, idx_p, resp_p, wb.ctl + 1));
                        CHECK(prof_end(ctx));
                    }
                    ctx->last_path = GMM_PATH_TENSOR;
                    return GMM_OK;
                }
            }
        }
        if (want) {
            const WideBuffers wb = ctx->wide();
            const float limit = ctx->tc_cond_limit >= 0.f ? ctx->tc_cond_limit : 0.01f;
            // (indices only: the sweep forms the leading fp16 product alone for the evaluated components - a third of the tensor
            // work - and ranks by correspondingly wider bounds; with responsibilities asked for, the approximate log Z has to
            // be good and all three products are formed)
            const bool hi = index_only && ctx->wide_hi != 0;
            KL(launch_prepare_wide(ctx->stream, D, K, pi, mu, var, wb, limit, 0.f, hi ? 2 : 0));
            ctx->launches += 4;
            int fl[8];
            CU(cudaMemcpyAsync(fl, wb.flags, sizeof(fl), cudaMemcpyDeviceToHost, ctx->stream));
            CU(cudaStreamSynchronize(ctx->stream));
            const int n_ill = fl[4], Kg = fl[6], n_list = fl[2];
            if (n_ill + 64 <= WIDE_MAX_ILL && 2 * n_ill <= K && Kg >= 1) {
                tensor_w = true;
                if (n_ill > 0) KL(launch_ill_gather_wide(ctx->stream, D, n_list, wb, mu, ctx->w2(), ctx->c2d()));
                // (ten reported candidates instead of six for m <= 4 leave no fewer rows to the FP32 kernels: the rows that
                // go there have broad posteriors, with more than ten components above 1e-3 of Z between them)
                const int ntop = (m + 2 <= 6) ? 6 : WIDE_MAX_TOP;
                const bool screen = n_ill > 0;
                const int64_t piece = ctx->wide_piece;
                const int64_t cap = N < piece ? N : piece;
                const size_t need = align256((size_t)cap * sizeof(int32_t)) + 256;       // uncertain rows of a piece, their count
                CHECK(grow_buffer(ctx, &ctx->at_scratch, &ctx->at_scratch_bytes, need, "the assignment's list of uncertain rows"));
                unsigned char* base = static_cast<unsigned char*>(ctx->at_scratch);
                int32_t* unc_rows = reinterpret_cast<int32_t*>(base);
                int* unc_count = reinterpret_cast<int*>(base + need - 256);
                for (int64_t off = 0; off < N; off += piece) {
                    const int64_t cnt = (N - off < piece) ? (N - off) : piece;
                    const float* Xs = X + off * D;
                    int32_t* idx_p = idx + off * m;
                    float* resp_p = resp ? resp + off * m : nullptr;
                    CU(cudaMemsetAsync(unc_count, 0, sizeof(int), ctx->stream));
                    if (screen) CU(launch_cand_clear_wide(ctx->stream, cnt, n_list, wb));
                    CHECK(prof_begin(ctx));
                    KL(launch_transform_wide(ctx->stream, Xs, cnt, D, wb, &ctx->result()->status, false, true));
                    KL(launch_lse_wide(ctx->stream, cnt, D, K, Kg, screen ? n_ill : 0, n_list, wb, ctx->sms, &ctx->result()->status, ntop, hi ? 0 : -1));
                    if (screen) KL(launch_cand_gate_wide(ctx->stream, wb, ctx->wide_sparse >= 2 ? ((long long)1 << 62) : (long long)cnt * n_list / 64));
                    KL(launch_assign_refine_wide(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), n_list, screen, wb, ntop, m, idx_p, resp_p,
                                                 unc_rows, unc_count, index_only, hi));
                    // the rows left uncertain, against all K components; and the whole piece if its marked pairs were too many
                    KL(launch_topm_fp32(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m, idx_p, resp_p, nullptr, unc_rows, unc_count));
                    if (screen) KL(launch_topm_fp32(ctx->stream, Xs, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m, idx_p, resp_p, wb.ctl + 1));
                    CHECK(prof_end(ctx));
                }
            }
        }
        if (!tensor_w)
            for (int64_t off = 0; off < N; off += SUPER_TILE) {
                const int64_t cnt = (N - off < SUPER_TILE) ? (N - off) : SUPER_TILE;
                KL(launch_topm_fp32(ctx->stream, X + off * D, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m, idx + off * m, resp ? resp + off * m : nullptr, nullptr));
            }
        ctx->last_path = tensor_w ? GMM_PATH_TENSOR : GMM_PATH_FP32;
        return GMM_OK;
    }
    const bool tensor = ctx->capPlanes && ctx->lay.tc && ctx->path != GMM_PATH_FP32;
    const int* run_fp32_if = nullptr;
    if (tensor) {
        const TcBuffers tb = ctx->tc();
        const float limit = ctx->tc_cond_limit >= 0.f ? ctx->tc_cond_limit : 0.01f;
        KL(launch_prepare_tc(ctx->stream, D, K, pi, mu, var, tb, limit, &ctx->result()->status, true));
        ctx->launches += 3;
        KL(launch_ill_cache_tc(ctx->stream, D, mu, ctx->w2(), ctx->c2(), tb));
        const int64_t piece = ctx->tc_piece;
        const int64_t cap = N < piece ? N : piece;
        constexpr int WINDOW = 8;            // pieces that share one list of uncertain rows (and one exact pass over it)
        const int64_t win_cap = (N < WINDOW * piece) ? N : WINDOW * piece;
        const size_t rec_bytes = align256((size_t)cap * assign_tc_record_bytes(m));
        const size_t need = rec_bytes + align256((size_t)win_cap * sizeof(int32_t)) + 256;   // records, uncertain rows, their count
        CHECK(grow_buffer(ctx, &ctx->at_scratch, &ctx->at_scratch_bytes, need, "the assignment records"));
        unsigned char* base = static_cast<unsigned char*>(ctx->at_scratch);
        int32_t* unc_rows = reinterpret_cast<int32_t*>(base + rec_bytes);
        int* unc_count = reinterpret_cast<int*>(base + need - 256);
        int in_window = 0;
        int64_t win_start = 0;
        for (int64_t off = 0; off < N; off += piece) {
            const int64_t cnt = (N - off < piece) ? (N - off) : piece;
            if (in_window == 0) {
                win_start = off;
                CU(cudaMemsetAsync(unc_count, 0, sizeof(int), ctx->stream));
            }
            CHECK(prof_begin(ctx));
            KL(launch_transform_tc(ctx->stream, X + off * D, cnt, D, tb, &ctx->result()->status));
            KL(launch_assign_tc(ctx->stream, X + off * D, cnt, D, K, mu, ctx->w2(), ctx->c2(), tb, reinterpret_cast<float*>(base),
                                unc_rows, unc_count, (int)(off - win_start), m, idx + off * m, resp ? resp + off * m : nullptr, &ctx->result()->status,
                                index_only));
            ctx->launches++;
            ++in_window;
            if (in_window == WINDOW || off + piece >= N) {
                // The rows the refinement was not certain about, of the whole window: all K components exactly, by the FP32
                // tile kernel.  (One launch per window: with a few hundred rows per piece a launch per piece is all latency.)
                const int64_t win_rows = off + cnt - win_start;
                KL(launch_topm_fp32(ctx->stream, X + win_start * D, win_rows, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m,
                                    idx + win_start * m, resp ? resp + win_start * m : nullptr, nullptr, unc_rows, unc_count));
                in_window = 0;
            }
            CHECK(prof_end(ctx));
        }
        run_fp32_if = tb.flags + 3;
    }
    for (int64_t off = 0; off < N; off += SUPER_TILE) {
        const int64_t cnt = (N - off < SUPER_TILE) ? (N - off) : SUPER_TILE;
        KL(launch_topm_fp32(ctx->stream, X + off * D, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), m, idx + off * m, resp ? resp + off * m : nullptr, run_fp32_if));
    }
    ctx->last_path = tensor ? GMM_PATH_TENSOR : GMM_PATH_FP32;
    return GMM_OK;
}
}  // namespace

int gmm_tensor_path_supports(int D, int K) { return (tc_supports(D, K) || wide_supports(D, K)) ? 1 : 0; }

int gmm_auto_path(int D, int K) {
    return (auto_is_tensor(D, K) || (wide_supports(D, K) && K >= 64)) ? GMM_PATH_TENSOR : GMM_PATH_FP32;
}

size_t gmm_scratch_bytes(int D, int K) {
    if (D < 1 || K < 1) return 0;
    return scratch_layout(D, K, auto_wants_planes(D, K)).total;      // what a context in GMM_PATH_AUTO allocates
}

int64_t gmm_launch_count(const gmm_ctx* ctx) { return ctx ? ctx->launches : 0; }

int gmm_set_profiling(gmm_ctx* ctx, int on) {
    if (!ctx) return GMM_EINVAL;
    ctx->profiling = on != 0;
    return GMM_OK;
}

int gmm_kernel_time(gmm_ctx* ctx, double* total_ms, int64_t* launches) {
    if (!ctx || !total_ms || !launches) return GMM_EINVAL;
    DeviceGuard g(ctx->device);
    CU(cudaStreamSynchronize(ctx->stream));
    for (int i = 0; i < ctx->ev_used; ++i) {
        float ms = 0.f;
        CU(cudaEventElapsedTime(&ms, ctx->ev_a[i], ctx->ev_b[i]));
        ctx->prof_ms += ms;
    }
    ctx->ev_used = 0;
    *total_ms = ctx->prof_ms;
    *launches = ctx->prof_launches;
    return GMM_OK;
}

int gmm_reset_counters(gmm_ctx* ctx) {
    if (!ctx) return GMM_EINVAL;
    ctx->launches = 0;
    ctx->prof_ms = 0.0;
    ctx->prof_launches = 0;
    ctx->ev_used = 0;
    return GMM_OK;
}

namespace {
// grows *buf to at least `need` bytes (contents are not kept)
int grow_buffer(gmm_ctx* ctx, void** buf, size_t* have, size_t need, const char* what) {
    if (need <= *have) return GMM_OK;
    if (*buf) {
        CU(cudaStreamSynchronize(ctx->stream));
        CU(cudaFree(*buf));
        *buf = nullptr;
        *have = 0;
    }
    cudaError_t e = cudaMalloc(buf, need);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ctx, GMM_ENOMEM, "cannot allocate %zu bytes for %s: %s", need, what, cudaGetErrorString(e));
    }
    *have = need;
    return GMM_OK;
}
}  // namespace

int gmm_build_posting_lists(gmm_ctx* ctx, const int32_t* idx, const float* resp, int64_t N, int m, int K, float tau,
                            int max_lists, int64_t* offsets, int32_t* items, int64_t* total, double* mean_lists) {
    if (!ctx) return GMM_EINVAL;
    DeviceGuard g(ctx->device);
    if (!idx || !resp || !offsets || !items) return fail(ctx, GMM_EINVAL, "null pointer argument");
    if (N < 1 || K < 1) return fail(ctx, GMM_EINVAL, "N and K must be >= 1 (got N=%lld K=%d)", (long long)N, K);
    if (m < 1 || m > GMM_MAX_TOPM) return fail(ctx, GMM_EINVAL, "m must be in [1, %d] (got %d)", GMM_MAX_TOPM, m);
    if (max_lists < 1 || max_lists > m) return fail(ctx, GMM_EINVAL, "max_lists must be in [1, m] (got %d, m=%d)", max_lists, m);
    if (N >= ((int64_t)1 << 31)) return fail(ctx, GMM_EUNSUPPORTED, "N must be below 2^31 (vector indices are int32)");
    if (K > PL_MAX_K) return fail(ctx, GMM_EUNSUPPORTED, "K must be <= %d for the posting-list builder (got %d)", PL_MAX_K, K);
    if (!(tau > 0.f)) tau = 1.0f / (float)K;                 // also for NaN
    CHECK(grow_buffer(ctx, &ctx->pl_scratch, &ctx->pl_scratch_bytes, pl_scratch_bytes(K), "the posting-list counters"));
    KL(launch_posting_lists(ctx->stream, idx, resp, N, m, K, tau, max_lists, ctx->pl_scratch, offsets, items));
    ctx->launches += 4;        // launch_posting_lists enqueues five kernels
    int64_t tot = 0;
    CU(cudaMemcpyAsync(&tot, offsets + K, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    if (total) *total = tot;
    if (mean_lists) *mean_lists = (double)tot / (double)N;
    return GMM_OK;
}

int gmm_kmeans_step(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* centroids, int32_t* assign,
                    int32_t* work, float* centroids_out, int64_t* counts, double* inertia) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X, 4, "X"));
    CHECK(check_ptr(ctx, centroids, 4, "centroids"));
    CHECK(check_ptr(ctx, assign, 4, "assign"));
    CHECK(check_ptr(ctx, work, 4, "work"));
    CHECK(check_ptr(ctx, centroids_out, 4, "centroids_out"));
    if (N >= ((int64_t)1 << 31)) return fail(ctx, GMM_EUNSUPPORTED, "N must be below 2^31 (point indices are int32)");
    if (K > PL_MAX_K) return fail(ctx, GMM_EUNSUPPORTED, "K must be <= %d for the k-means step (got %d)", PL_MAX_K, K);
    DeviceGuard g(ctx->device);
    CHECK(ensure_scratch(ctx, D, K));
    CHECK(grow_buffer(ctx, &ctx->pl_scratch, &ctx->pl_scratch_bytes, pl_scratch_bytes(K), "the posting-list counters"));
    CHECK(grow_buffer(ctx, &ctx->km_scratch, &ctx->km_scratch_bytes, km_scratch_bytes(D, K), "the k-means partial sums"));
    // nearest centroid = top-1 component of a unit-variance, equal-weight mixture
    float* resp = reinterpret_cast<float*>(work);                 // [N], not used afterwards except as the builder's input
    int32_t* items = work + N;                                    // [N]
    bool tensor = ctx->capPlanes && ctx->lay.tc && ctx->path != GMM_PATH_FP32;
    const bool tensor_wide = ctx->capPlanes && ctx->lay.wide && ctx->path != GMM_PATH_FP32 && K >= 64;
    if (tensor_wide) {
        // wide data: the hard assignment of the wide tensor path (screening, or six candidates per point), under a mixture
        // whose one variance is the spread of the centroids
        const size_t KD = (size_t)K * D;
        CHECK(grow_buffer(ctx, &ctx->km_unit, &ctx->km_unit_bytes, (KD + (size_t)K + (size_t)D) * sizeof(float), "the mixture of the k-means step"));
        float* var_u = static_cast<float*>(ctx->km_unit);
        float* pi_u = var_u + KD;
        KL(launch_kmeans_scaled_mixture(ctx->stream, D, K, centroids, pi_u, var_u, pi_u + K));
        ctx->launches++;
        CHECK(assign_topm_impl(ctx, X, N, D, K, pi_u, centroids, var_u, 1, assign, nullptr, true));
        tensor = ctx->last_path == GMM_PATH_TENSOR;
    } else if (tensor) {
        // through the assignment pass of the tensor path, with that mixture written out: pi = 1 / K, var = 1
        const size_t KD = (size_t)K * D;
        CHECK(grow_buffer(ctx, &ctx->km_unit, &ctx->km_unit_bytes, (KD + (size_t)K) * sizeof(float), "the unit mixture of the k-means step"));
        float* var_u = static_cast<float*>(ctx->km_unit);
        float* pi_u = var_u + KD;
        KL(launch_kmeans_unit_mixture(ctx->stream, D, K, pi_u, var_u));
        CHECK(assign_topm_impl(ctx, X, N, D, K, pi_u, centroids, var_u, 1, assign, resp, true));       // the indices alone are used
    } else {
        KL(launch_kmeans_unit_params(ctx->stream, D, K, ctx->w2(), ctx->c2d()));
        KL(launch_center_fp32(ctx->stream, D, K, centroids, ctx->center()));
        for (int64_t off = 0; off < N; off += SUPER_TILE) {
            const int64_t cnt = (N - off < SUPER_TILE) ? (N - off) : SUPER_TILE;
            KL(launch_topm_fp32(ctx->stream, X + off * D, cnt, D, K, centroids, ctx->w2(), ctx->c2d(), ctx->center(), 1, assign + off, resp + off));
        }
    }
    // the points of every cluster in ascending order, then fixed-order float64 sums
    KL(launch_posting_lists(ctx->stream, assign, resp, N, 1, K, 1.0f, 1, ctx->pl_scratch, km_offsets(ctx->km_scratch), items));
    KL(launch_kmeans_update(ctx->stream, X, D, K, centroids, items, ctx->km_scratch, centroids_out, counts));
    ctx->launches += 5;
    const int slot = 0;
    CU(cudaMemsetAsync(&ctx->result()->ll[slot], 0, 8, ctx->stream));
    KL(launch_reduce_ll(ctx->stream, km_inertia_k(ctx->km_scratch, D, K), K, &ctx->result()->ll[slot], false));
    double v = 0.0;
    CU(cudaMemcpyAsync(&v, &ctx->result()->ll[slot], sizeof(double), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    if (inertia) *inertia = v;
    ctx->last_path = tensor ? GMM_PATH_TENSOR : GMM_PATH_FP32;
    return GMM_OK;
}

int gmm_score_samples(gmm_ctx* ctx, const float* X, int64_t N, int D, int K, const float* pi, const float* mu,
                      const float* var, float* logp, double* loglik) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X, 4, "X"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    CHECK(check_ptr(ctx, logp, 4, "logp"));
    DeviceGuard guard(ctx->device);
    CHECK(ensure_scratch(ctx, D, K));
    KL(launch_prepare_fp32(ctx->stream, D, K, pi, mu, var, ctx->w2(), ctx->c2(), ctx->c2d(), ctx->center(), &ctx->result()->status));
    if ((size_t)K * D > ((size_t)1 << 12)) ctx->launches++;
    CU(cudaMemsetAsync(&ctx->result()->ll[0], 0, 8, ctx->stream));
    // Wide data with sparse posteriors: the EM step's screening route without its statistics.  Every component with a weight
    // is listed, one sweep over the leading fp16 product marks the pairs that can come within 2^-40 of a point's best, the
    // filter drops those that the final threshold rules out, and a warp per point evaluates the rest exactly: their
    // log-sum-exp is the point's log-density to 2^-40.  Taken when the first 8192 rows mark few pairs per point (a pair costs
    // 0.5 + 1.8e-3 D ns, the FP32 kernel 1.4e-4 K D ns per point); a piece that marks too many goes through the FP32 kernel.
    if (wide_supports(D, K) && ctx->capPlanes && ctx->lay.wide && ctx->path != GMM_PATH_FP32 && K >= 64 && ctx->wide_hi == 2 &&
        ctx->wide_mode != 1) {
        const WideBuffers wb = ctx->wide();
        float limit = ctx->tc_cond_limit;
        if (limit < 0.f) limit = ctx->tc_cond_scale * std::sqrt((float)((double)N / (double)K));
        KL(launch_prepare_wide(ctx->stream, D, K, pi, mu, var, wb, limit, INFINITY, 3));
        ctx->launches += 4;
        int fl[8];
        CU(cudaMemcpyAsync(fl, wb.flags, sizeof(fl), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
        const int n_list = fl[2], n_ill = fl[4], Kg = fl[6];
        bool ok = n_list >= 1 && n_ill + 64 <= WIDE_MAX_ILL;
        if (ok) {
            KL(launch_ill_gather_wide(ctx->stream, D, n_list, wb, mu, ctx->w2(), ctx->c2d()));
            auto screen_piece = [&](const float* Xs, int64_t cnt) -> int {
                CU(launch_cand_clear_wide(ctx->stream, cnt, n_list, wb));
                KL(launch_transform_wide(ctx->stream, Xs, cnt, D, wb, &ctx->result()->status, true, true));
                KL(launch_lse_wide(ctx->stream, cnt, D, K, Kg, n_ill, n_list, wb, ctx->sms, &ctx->result()->status, 2, 0, false, true, true));
                KL(launch_cand_filter_wide(ctx->stream, cnt, n_list, wb));
                return GMM_OK;
            };
            const double kd = (double)n_list * D;
            const double saved = (1.4e-4 - 3.6e-6) * kd - 5.0;
            const double per_point = ctx->wide_probe_limit > 0.0 ? ctx->wide_probe_limit : (saved > 0.0 ? saved / (0.5 + 1.8e-3 * D) : 0.0);
            if (ctx->wide_mode != 2) {
                const int64_t np = N < 8192 ? N : 8192;
                CHECK(screen_piece(X, np));
                int marks = 0;
                CU(cudaMemcpyAsync(&marks, wb.ctl, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
                CU(cudaStreamSynchronize(ctx->stream));
                ok = (double)marks <= per_point * (double)np;
            }
            if (ok) {
                CU(cudaMemsetAsync(wb.llpart, 0, 256 * 8, ctx->stream));
                const int64_t piece = ctx->wide_piece;
                for (int64_t off = 0; off < N; off += piece) {
                    const int64_t cnt = (N - off < piece) ? (N - off) : piece;
                    const float* Xs = X + off * D;
                    CHECK(prof_begin(ctx));
                    CHECK(screen_piece(Xs, cnt));
                    KL(launch_cand_gate_wide(ctx->stream, wb, ctx->wide_sparse >= 2 ? ((long long)1 << 62) : (long long)((double)cnt * per_point)));
                    CU(cudaMemcpyAsync(wb.logz_x, wb.logz, (size_t)cnt * 8, cudaMemcpyDeviceToDevice, ctx->stream));     // (-inf: no unlisted component has a weight)
                    KL(launch_cand_lse_wide(ctx->stream, Xs, cnt, D, n_list, wb, ctx->logZ2()));
                    KL(launch_lse_fp32(ctx->stream, Xs, cnt, D, n_list, wb.mu_c, wb.w2_c, wb.c2d_c, ctx->center(), ctx->logZ2(), nullptr, wb.logz, wb.ctl + 1));
                    KL(launch_merge_ll_wide(ctx->stream, cnt, wb, ctx->logZ2()));
                    CHECK(prof_end(ctx));
                    KL(launch_logz_out_fp32(ctx->stream, wb.logz_x, cnt, logp + off));
                }
                KL(launch_reduce_ll(ctx->stream, wb.llpart, WIDE_LL_BLOCKS, &ctx->result()->ll[0], true));
                ctx->last_path = GMM_PATH_TENSOR;
                double total = 0.0;
                const int rc = read_result(ctx, 0, &total);
                if (rc != GMM_OK) return rc;
                if (loglik) *loglik = total;
                return GMM_OK;
            }
        }
    }
    // the log-sum-exp kernel of the FP32 path, one super-tile at a time; its per-point values go out instead of into an M-step
    for (int64_t off = 0; off < N; off += SUPER_TILE) {
        const int64_t cnt = (N - off < SUPER_TILE) ? (N - off) : SUPER_TILE;
        CHECK(prof_begin(ctx));
        KL(launch_lse_fp32(ctx->stream, X + off * D, cnt, D, K, mu, ctx->w2(), ctx->c2d(), ctx->center(), ctx->logZ2(), ctx->llpart()));
        CHECK(prof_end(ctx));
        KL(launch_logz_out_fp32(ctx->stream, ctx->logZ2(), cnt, logp + off));
        KL(launch_reduce_ll(ctx->stream, ctx->llpart(), (cnt + FP32_TILE_P - 1) / FP32_TILE_P, &ctx->result()->ll[0], true));
    }
    ctx->last_path = GMM_PATH_FP32;
    double total = 0.0;
    const int rc = read_result(ctx, 0, &total);
    if (rc != GMM_OK) return rc;
    if (loglik) *loglik = total;
    return GMM_OK;
}

int gmm_fisher_vectors(gmm_ctx* ctx, const float* X, int64_t N, const int64_t* offsets, int G, int D, int K,
                       const float* pi, const float* mu, const float* var, float* fv, double* loglik) {
    CHECK(check_shape(ctx, N, D, K));
    CHECK(check_ptr(ctx, X, 4, "X"));
    CHECK(check_ptr(ctx, pi, 4, "pi"));
    CHECK(check_ptr(ctx, mu, 4, "mu"));
    CHECK(check_ptr(ctx, var, 4, "var"));
    CHECK(check_ptr(ctx, fv, 4, "fv"));
    if (!offsets) return fail(ctx, GMM_EINVAL, "offsets is NULL");
    if (G < 1) return fail(ctx, GMM_EINVAL, "G must be >= 1 (got %d)", G);
    int64_t smallest = 0;                       // size of the smallest group that has points
    for (int g = 0; g < G; ++g) {
        if (offsets[g] < 0 || offsets[g + 1] < offsets[g] || offsets[g + 1] > N)
            return fail(ctx, GMM_EINVAL, "offsets[%d..%d] = %lld, %lld: must be non-decreasing inside [0, N]", g, g + 1,
                        (long long)offsets[g], (long long)offsets[g + 1]);
        const int64_t T = offsets[g + 1] - offsets[g];
        if (T > 0 && (smallest == 0 || T < smallest)) smallest = T;
    }
    DeviceGuard guard(ctx->device);
    CHECK(ensure_scratch(ctx, D, K));
    const size_t KD = (size_t)K * D;
    double* Nk = ctx->stats();
    double* S1 = Nk + K;
    double* S2 = S1 + KD;
    // One preparation for all groups.  The conditioning limit of the tensor path is the one an EM step over all the
    // groups' points would use: what bounds the accuracy of a Fisher coordinate is the cancellation between the raw
    // moments (N_k, S1, S2), about 4e-6 (1 + mu^2 / var) N_k / (T sqrt(pi_k)), which the stricter limit of the smallest
    // group alone would not improve (measured: the same errors with and without any exact recomputation).
    int path;
    int64_t total_points = 0;
    for (int g = 0; g < G; ++g) total_points += offsets[g + 1] - offsets[g];
    CHECK(prepare_and_choose(ctx, total_points > 0 ? total_points : 1, D, K, pi, mu, var, &path, X, N));     // (wide data: the first rows of X tell the mode)
    if (path == GMM_PATH_TENSOR && ctx->path == GMM_PATH_AUTO && !wide_supports(D, K)) {
        // Once the limit flags nearly all the components the tile kernel has no well-conditioned logits left to bound
        // a point's maximum with, tests every pair exactly, and the FP32 kernels are the faster exact path.
        int n_ill = 0;
        CU(cudaMemcpyAsync(&n_ill, ctx->tc().flags + 4, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
        ctx->tc_n_ill = n_ill;
        if ((int64_t)n_ill * 50 > (int64_t)K * 49) path = GMM_PATH_FP32;
    }
    CU(cudaMemsetAsync(&ctx->result()->ll[0], 0, 8, ctx->stream));
    // Tensor path: groups small enough that one launch can hold a tile column for each of its CTA groups are processed
    // several at a time, CTA group b of a launch accumulating the statistics of one of them (its tiles are laid out at
    // b, b + Q, ... in the planes); their vectors come straight from the per-CTA-group partials.  Groups are taken in
    // order of size so that the groups of a launch finish together.  Larger groups go one at a time through the step's
    // own accumulation below.
    std::vector<char> batched((size_t)G, 0);
    if (path == GMM_PATH_TENSOR && !wide_supports(D, K)) {      // (D > 128: every group goes through the step's own two sweeps below)
        const TcBuffers tb = ctx->tc();
        const TcPlan pl = tc_plan(D, K, 160);
        const int Qmax = ctx->tc_Q;
        const int64_t cap_tiles = ctx->tc_piece / TC_BN;                        // tiles that the planes of one launch hold
        std::vector<int> order;
        for (int g = 0; g < G; ++g) {
            const int64_t T = offsets[g + 1] - offsets[g];
            if (T > 0 && 2 * ((T + TC_BN - 1) / TC_BN) <= cap_tiles) order.push_back(g);      // at least two per launch
        }
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
            return offsets[a + 1] - offsets[a] > offsets[b + 1] - offsets[b];
        });
        struct Batch { size_t tile0, group0; int Q; int64_t tiles_each; };
        std::vector<Batch> batches;
        std::vector<int> h_valid, h_index;
        std::vector<int64_t> h_src, h_points;
        for (size_t a = 0; a < order.size();) {
            const int64_t T0 = offsets[order[a] + 1] - offsets[order[a]];          // the largest of the batch
            const int64_t tiles_each = (T0 + TC_BN - 1) / TC_BN;
            const int Qb = (int)std::min<int64_t>(std::min<int64_t>(Qmax, cap_tiles / tiles_each), (int64_t)(order.size() - a));
            // A launch of Qb < Qmax groups leaves CTA groups idle; a group on its own uses them all but pays about 30
            // tile times of launches and reductions.  Per group: tiles / Qb against tiles / Qmax + 30.
            if (Qb < 2 || tiles_each * (Qmax - Qb) > (int64_t)30 * Qb * Qmax) { ++a; continue; }      // left to the loop over single groups
            batches.push_back({h_valid.size(), h_index.size(), Qb, tiles_each});
            for (int64_t i = 0; i < tiles_each; ++i)
                for (int b = 0; b < Qb; ++b) {                                     // tile b + i Qb of the planes
                    const int g = order[a + b];
                    const int64_t T = offsets[g + 1] - offsets[g];
                    const int64_t left = T - i * TC_BN;
                    h_valid.push_back(left <= 0 ? 0 : (int)std::min<int64_t>(left, TC_BN));
                    h_src.push_back(left <= 0 ? offsets[g] : offsets[g] + i * TC_BN);
                }
            for (int b = 0; b < Qb; ++b) {
                const int g = order[a + b];
                h_index.push_back(g);
                h_points.push_back(offsets[g + 1] - offsets[g]);
                batched[g] = 1;
            }
            a += (size_t)Qb;
        }
        if (!batches.empty()) {
            const size_t nt = h_valid.size(), ng = h_index.size();
            const size_t o_src = 0, o_points = o_src + align256(nt * 8), o_valid = o_points + align256(ng * 8),
                         o_index = o_valid + align256(nt * 4), total_bytes = o_index + align256(ng * 4);
            CHECK(grow_buffer(ctx, &ctx->fv_scratch, &ctx->fv_scratch_bytes, total_bytes, "the tile tables of the grouped launches"));
            unsigned char* base = static_cast<unsigned char*>(ctx->fv_scratch);
            // (pageable sources: each copy has left the host array when the call returns)
            CU(cudaMemcpyAsync(base + o_src, h_src.data(), nt * 8, cudaMemcpyHostToDevice, ctx->stream));
            CU(cudaMemcpyAsync(base + o_points, h_points.data(), ng * 8, cudaMemcpyHostToDevice, ctx->stream));
            CU(cudaMemcpyAsync(base + o_valid, h_valid.data(), nt * 4, cudaMemcpyHostToDevice, ctx->stream));
            CU(cudaMemcpyAsync(base + o_index, h_index.data(), ng * 4, cudaMemcpyHostToDevice, ctx->stream));
            const int64_t* d_src = reinterpret_cast<const int64_t*>(base + o_src);
            const int64_t* d_points = reinterpret_cast<const int64_t*>(base + o_points);
            const int* d_valid = reinterpret_cast<const int*>(base + o_valid);
            const int* d_index = reinterpret_cast<const int*>(base + o_index);
            bool tight = ctx->tc_n_ill > 0 && (smallest < (int64_t)512 * K || (int64_t)ctx->tc_n_ill * 8 > K);
            if (ctx->tc_force_filter >= 0) tight = ctx->tc_force_filter == 1;
            for (const Batch& bt : batches) {
                const int64_t rows = bt.tiles_each * bt.Q * TC_BN;
                CU(cudaMemsetAsync(tb.partial, 0, (size_t)bt.Q * pl.Kpad * TC_PCOLS * 8, ctx->stream));
                CU(cudaMemsetAsync(tb.llpart, 0, (size_t)bt.Q * 16, ctx->stream));
                CHECK(prof_begin(ctx));
                KL(launch_transform_grouped_tc(ctx->stream, X, rows, D, d_valid + bt.tile0, d_src + bt.tile0, tb, &ctx->result()->status));
                KL(launch_em_tc(ctx->stream, X, rows, D, K, mu, ctx->w2(), ctx->c2(), tb, bt.Q, ctx->tc_flush, tight,
                                &ctx->result()->status, d_valid + bt.tile0, d_src + bt.tile0));
                CHECK(prof_end(ctx));
                KL(launch_reduce_ll(ctx->stream, tb.llpart, 2 * bt.Q, &ctx->result()->ll[0], true));
                KL(launch_fisher_tc(ctx->stream, D, K, bt.Q, tb, pi, mu, var, d_index + bt.group0, d_points + bt.group0, fv));
                ctx->launches += 2;
            }
        }
    }
    for (int g = 0; g < G; ++g) {
        if (batched[g]) continue;
        const int64_t T = offsets[g + 1] - offsets[g];
        float* out = fv + (size_t)g * 2 * KD;
        if (T == 0) {
            CU(cudaMemsetAsync(out, 0, 2 * KD * sizeof(float), ctx->stream));
            continue;
        }
        CU(cudaMemsetAsync(Nk, 0, ((size_t)K + 2 * KD) * 8, ctx->stream));
        CHECK(accumulate_points(ctx, path, X + offsets[g] * D, T, D, K, mu, Nk, S1, S2, 0));
        KL(launch_fisher(ctx->stream, T, D, K, Nk, S1, S2, pi, mu, var, out));
    }
    ctx->last_path = path;
    double total = 0.0;
    if (smallest == 0) {                        // no points at all: nothing was accumulated, only the parameters were checked
        DevResult r;
        CU(cudaMemcpyAsync(&r, ctx->result(), sizeof(DevResult), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
        CHECK(report_status(ctx, r.status));
        if (loglik) *loglik = 0.0;
        return GMM_OK;
    }
    const int rc = read_result(ctx, 0, &total);
    if (rc != GMM_OK) return rc;
    if (loglik) *loglik = total;
    return GMM_OK;
}

int gmm_sync_status(gmm_ctx* ctx) {
    if (!ctx) return GMM_EINVAL;
    DeviceGuard g(ctx->device);
    CU(cudaStreamSynchronize(ctx->stream));
    int st = 0;
    if (ctx->scratch) {
        CU(cudaMemcpyAsync(&st, &ctx->result()->status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
    }
    if (st == 0 && ctx->sticky_status == 0) return GMM_OK;
    return report_status(ctx, st);
}

int gmm_update_counts(gmm_ctx* ctx, int64_t* floored_variances, int64_t* empty_components) {
    if (!ctx) return GMM_EINVAL;
    DeviceGuard g(ctx->device);
    int c[2] = {0, 0};
    if (ctx->scratch) {
        CU(cudaMemcpyAsync(c, ctx->result()->counts, sizeof(c), cudaMemcpyDeviceToHost, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
    }
    if (floored_variances) *floored_variances = c[0];
    if (empty_components) *empty_components = c[1];
    return GMM_OK;
}

const char* gmm_strerror(int code) {
    switch (code) {
        case GMM_OK: return "ok";
        case GMM_EINVAL: return "invalid argument";
        case GMM_EALIGN: return "misaligned pointer";
        case GMM_ENOMEM: return "out of device memory";
        case GMM_ECUDA: return "CUDA error";
        case GMM_ENUMERIC: return "numerical error (invalid parameters or non-finite log-likelihood)";
        case GMM_ETIMEOUT: return "device-side wait timed out";
        case GMM_EUNSUPPORTED: return "kernel path does not support this shape";
        default: return "unknown error";
    }
}

const char* gmm_last_error(const gmm_ctx* ctx) { return ctx ? ctx->err : "null context"; }

const char* gmm_version(void) { return "flashgmm 0.1 (sm_100a)"; }

}  // extern "C"
