// Tensor-core path for wide data (128 < D <= 1024; sm_100a, tcgen05 + TMEM): the EM iteration in the two sweeps of the
// paper's Algorithm 1, each a streamed contraction on the expanded quadratic form.
//
// Why two sweeps here and one for D <= 128: the M-step result of 128 components is 128 x 2D fp32 values, which for
// D > 128 no longer fits the 512 TMEM columns of an SM next to the logits, and the coefficient slice of 128 components
// (128 x 2D x 2 fp16 planes) no longer fits shared memory, so neither can stay on chip for the life of a CTA.
//
//   sweep 1  (lse_wide_kernel, TMEM lanes = POINTS)   Algorithm 1, Step 1.  A CTA takes tiles of 128 points and walks the
//            components in groups of 256 (256 TMEM columns for the main product, 256 for the two small cross products:
//            the same split, and the same order of accumulation, as in sweep 2, so that both sweeps see the same logits
//            and the responsibilities of a point sum to one; a group that is only screened forms the leading product
//            alone, in one half of the columns, while the softmax warps read the other half); for every 64-column atom
//            of the contraction it streams one stage per plane - the tile's Y atom and the group's two coefficient atoms -
//            through a ring in shared memory.
//            A softmax thread owns one point: running (max, sum) over all K, log2 Z_i to a scratch buffer of one piece
//            (2^17 points; no O(N) memory), sum of log2 Z for the log-likelihood.
//   sweep 2  (em_wide_kernel, TMEM lanes = COMPONENTS)   Algorithm 1, Step 2.  A CTA owns 128 components and takes
//            batches of 256 points: E-step again (main product and the two small cross products in separate TMEM
//            accumulators), r = 2^(log2 z - log2 Z_i) written over the logits as fp16 hi + lo (the A operand of the
//            M-step), then for each half-slice of 64 dimensions S[128 x 128] = r^T [Y | Y^2] over the batch in one of two
//            alternating TMEM accumulators, which the softmax warps add to the CTA's own fp32 partial block in global
//            memory while the next half-slice accumulates.  No exchange between CTAs and no cooperative launch: Z_i is
//            known from sweep 1.
// Precision as on the D <= 128 path (every operand split into two fp16 values; three products per contraction), with
// kap_d chosen so that a component's own points give terms of zero mean in every dimension: the accumulators then stay
// small (tens, not D / 2), and with them the truncation error of the tensor core's fp32 accumulation.
//
// Components the expanded form cannot carry (collapsed or narrow ones, and ones that hold few points) are "listed": they
// sit behind the others in the order the sweeps see the components, sweep 2 leaves them out, and sweep 1 only SCREENS
// them - it marks, in a bitmap, the (point, component) pairs whose approximate log2 z plus a rigorous error bound can
// come within 2^-40 of the point's best (as far as the sweep knows it when it meets the pair; wide_cand_filter_kernel
// then drops the marks that the point's final threshold rules out).  The marked pairs are then evaluated exactly in fp32,
// pair by pair (wide_cand_lse_kernel, wide_cand_mstep_kernel), or, when they are too many, densely by the FP32 kernels.
// In the "screen" mode EVERY component is listed: one tensor sweep over the leading fp16 product decides which pairs are
// looked at, all statistics come from exact evaluations.  The same screening, with the candidates ranked by upper
// bounds, gives the top-m assignment (wide_assign_refine_kernel).
#include "internal.cuh"
#include "em_tc.cuh"
#include "em_wide.cuh"

#include <cuda.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#define TC_WAIT_LIMIT_NS 2000000000ull
#include "tc_prims.cuh"

namespace fg {

namespace {

constexpr int WT_THREADS = 320;            // 8 softmax warps, producer warp, MMA warp
constexpr int WT_PRODUCER = 8, WT_MMA = 9;
constexpr int SLOT = 32768;                // ring slot: [hi 16 KB | lo 16 KB] or one 32 KB atom of 256 rows
constexpr float RSCALE = TC_RSCALE;

// ------------------------------------------------------------------------------------------------------------------
// Sweep 1
// The ring holds four stages of 48 KB: one plane's atoms of a contraction step, [Y atom | coefficient atoms of the group's
// two chunks] (the two chunks adjacent: one operand of 256 rows).  A step of a group that forms all three products takes
// two stages (hi planes, lo planes), a step of a leading-product group one.  One barrier pair and one commit per stage:
// with a barrier pair per atom the two single-lane loops (loads, MMAs) took 2000 cycles per step of 516 cycles of MMAs.
constexpr int HSLOT = 16384;
constexpr int L_STAGE = 3 * HSLOT;
constexpr int L_SLOTS = 4;
constexpr int L_BAR = L_SLOTS * L_STAGE;
constexpr int L_MERGE = L_BAR + 256;                // 128 x 8 bytes: (max, sum) pairs of warpgroup 1, later the log-likelihood terms
constexpr int L_SMEM = L_MERGE + 1024 + 1024;
// LB_LFULL, LB_LEMPTY: one pair per half of the accumulator columns.  A group that forms all three products fills both
// halves (main products in [0, 256), cross products in [256, 512)); a leading-product group fills one, so that the next
// group's products run while the softmax warps read this one's.
enum { LB_FULL = 0, LB_EMPTY = L_SLOTS, LB_LFULL = 2 * L_SLOTS, LB_LEMPTY = 2 * L_SLOTS + 2, LB_FINAL = 2 * L_SLOTS + 4, LB_COUNT };
static_assert(LB_COUNT * 8 <= 256, "barriers");

struct LseParams {
    int64_t n;
    int NC;              // chunks of 128 components
    int NZ;              // atoms of 64 columns in the contraction (4 per slice of 128 dimensions)
    const float2* tkck;  // [NC * 128]
    const double* cref;
    double* logz;
    double* llpart;
    float* top;          // [n][2 NTOP] per point: its NTOP largest approximate log2 z (relative to c_ref), then their positions
    int* status;
    // screening of the listed (ill-conditioned) components, all NULL / 0 when there are none
    bool screen;         // listed components follow the evaluated ones and are screened
    const float2* scr;   // [NC * 128] listed components: (c - c_ref + error allowance, allowance per unit of |x - g|^2);
                         // evaluated components: (error allowance, allowance per unit of |x - g|^2)
    const float* scr_e;  // [NC * 128] listed components: the error allowance alone
    const int* scr_mask; // [NC * 4] nonzero where a chunk of 32 components holds a listed one
    const int* slot_of;  // [NC * 128]
    const float* n2;     // [n]
    unsigned* cand;      // [n][cand_words]
    int cand_words;
    int scr_group;       // first group of 256 columns that holds listed components (they hold nothing else from there on)
    int hi_group;        // groups [hi_group, hi_end): only the leading product (Y_hi P_hi) is formed, with wider allowances
    int hi_end;
    unsigned* rec;       // NULL, or [n][WIDE_REC]: the marks' upper bounds, for the filter that follows
    int* rec_cnt;        // [n]
    float* rec_thr;      // [n] the point's final threshold
    int g0;              // the sweep starts at this group (the "screen" mode: behind the unlisted components, which have no weight)
    int topm;            // > 0 (NTOP > 2; the assignment by screening): the sweep also reports, per point, the NTOP blocks of 32
                         // listed components with the largest upper bounds (the bound and the component's position)
    int pre_pass;        // 1: before a tile's sweep proper, the groups from hi_group on are swept once for their lower bounds only
    int* ctl;
};

// NTOP: how many of a point's largest approximate log2 z the sweep reports (2 for the EM step's exact normaliser, m + 2 for
// the top-m assignment).
template <int NTOP>
struct WideTop {
    float a[NTOP];
    int i[NTOP];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int j = 0; j < NTOP; ++j) { a[j] = -CUDART_INF_F; i[j] = -1; }
    }
    __device__ __forceinline__ void insert(float val, int id) {      // descending; a later equal value stays behind
        if (!(val > a[NTOP - 1])) return;
        a[NTOP - 1] = val; i[NTOP - 1] = id;
#pragma unroll
        for (int j = NTOP - 1; j > 0; --j) {
            if (a[j] > a[j - 1]) {
                const float fv = a[j]; a[j] = a[j - 1]; a[j - 1] = fv;
                const int fi = i[j]; i[j] = i[j - 1]; i[j - 1] = fi;
            }
        }
    }
};

template <int NTOP>
__global__ void __launch_bounds__(WT_THREADS, 1)
lse_wide_kernel(const LseParams p, const __grid_constant__ CUtensorMap tm_yhi, const __grid_constant__ CUtensorMap tm_ylo,
                const __grid_constant__ CUtensorMap tm_phi, const __grid_constant__ CUtensorMap tm_plo) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, drain_s;
    volatile int* abort_flag = &abort_s;
    volatile int* drain_flag = &drain_s;
    float2* merge_s = reinterpret_cast<float2*>(smem + L_MERGE);
    double* ll_s = reinterpret_cast<double*>(smem + L_MERGE);      // after the last tile
    __shared__ float top_s[128][2 * NTOP + 1];
    __shared__ float xm_s[256];
    // Per-component constants of the group at hand, one copy per warpgroup and two buffers (a warpgroup fills one while its
    // slower warps may still read the other): (t, c, screening offset, screening slope), the allowance alone, the slot, the chunk masks.
    // Read from global memory inside the loops over the accumulators they cost a trip to L2 per pair of components (the
    // shared-memory ring leaves almost no L1).
    __shared__ float4 tab_s[2][2][128];
    __shared__ float tabe_s[2][2][128];
    __shared__ int tabs_s[2][2][128];                    // (the slot of a listed component)
    __shared__ int tabm_s[2][2][4];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t ntiles = (p.n + WIDE_TILE - 1) / WIDE_TILE;
    const int64_t ntl = ((int64_t)blockIdx.x < ntiles) ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int NC = p.NC, NZ = p.NZ;
    const int NG = (NC + 1) >> 1;                        // groups of two chunks
    // A tile's steps, the same for every role: with pre_pass the groups from hi_group on once for their lower bounds (so that
    // the threshold is final before anything is marked), then every group.
    const int npre = (p.pre_pass && p.hi_group < NG) ? NG - p.hi_group : 0;
    const int nsteps = npre + NG - p.g0;
    auto step_group = [&](int t) { return t < npre ? p.hi_group + t : p.g0 + t - npre; };
    auto leading_only = [&](int g) { return g >= p.hi_group && g < p.hi_end; };

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L_BAR);
    auto BAR = [&](int i) { return smem_u32(&bars[i]); };
    if (tid == 0) {
        abort_s = 0;
        drain_s = 0;
        for (int s = 0; s < L_SLOTS; ++s) { bar_init(BAR(LB_FULL + s), 1); bar_init(BAR(LB_EMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) { bar_init(BAR(LB_LFULL + b), 1); bar_init(BAR(LB_LEMPTY + b), 256); }
        bar_init(BAR(LB_FINAL), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == WT_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = tmem_base_s;

    if (warp < 8) {
        // =========================== softmax warps: thread = TMEM lane = point ===========================
        // Warpgroup g reads chunk g of every group of two chunks (main product in columns [128 g, 128 g + 128), cross products
        // in [256 + 128 g, ...)); the two running (max, sum) pairs of a point are merged at the end of its tile.
        const int grp = warp >> 2, wq = warp & 3;
        const uint32_t lane_addr = ((uint32_t)(wq * 32)) << 16;
        const int pt = wq * 32 + lane;                       // point within the tile
        const double cref = *p.cref;
        uint32_t ub0 = 0, ub1 = 0, tcount = 0;               // uses of the two accumulator halves; tables staged so far
        int nb = 0;                                          // the half the next leading-product group takes
        double ll_acc = 0.0;
        float2 n_tk = make_float2(0.f, 0.f), n_sc = make_float2(0.f, 0.f);
        float n_se = 0.f;
        int n_mask = 0, n_slot = -1;
        int nhit = 0;                                        // pairs this thread has marked (all tiles)
        auto table_load = [&](int g) {                       // this thread's component of the warpgroup's chunk of group g
            if (2 * g + grp < NC) {
                const int col = (2 * g + grp) * 128 + pt;
                n_tk = __ldg(p.tkck + col);
                if (p.screen || NTOP > 2) n_sc = __ldg(p.scr + col);
                if (p.screen) {
                    n_se = __ldg(p.scr_e + col);
                    n_slot = __ldg(p.slot_of + col);
                    if (pt < 4) n_mask = __ldg(p.scr_mask + (col >> 5) + pt);
                }
            }
        };
        auto table_store = [&](int tb) {
            tab_s[tb][grp][pt] = make_float4(n_tk.x, n_tk.y, n_sc.x, n_sc.y);
            tabe_s[tb][grp][pt] = n_se;
            tabs_s[tb][grp][pt] = n_slot;
            if (pt < 4) tabm_s[tb][grp][pt] = n_mask;
        };
        for (int64_t i = 0; i < ntl; ++i) {
            const int64_t row = (blockIdx.x + i * gridDim.x) * WIDE_TILE + pt;
            float m_run = -1e30f, s_run = 0.f;               // finite start: blocks of -inf logits must not make NaN
            const float nrm = ((p.screen || NTOP > 2) && row < p.n) ? __ldg(p.n2 + row) : 0.f;
            float thr_base = -1e30f;
            WideTop<NTOP> tl;                                // the largest logits of this thread's chunks, and where
            tl.init();
            // A pair that can matter: its bit in the map, and (for the filter that follows the sweep) its upper bound, rounded
            // up to the 19 bits that share a word with the slot.
            // (each warpgroup has its own half of the point's record)
            int nrec = 0;
            auto mark = [&](float u, int sl) {
                if (sl < 0) return;
                atomicOr(p.cand + row * p.cand_words + (sl >> 5), 1u << (sl & 31));
                ++nhit;
                if (p.rec) {
                    if (nrec < WIDE_REC / 2)
                        p.rec[row * WIDE_REC + grp * (WIDE_REC / 2) + nrec] = (__float_as_uint(u + fabsf(u) * 0.001953125f) & ~0x1FFFu) | (unsigned)sl;
                    ++nrec;
                }
            };
            table_load(step_group(0));
            table_store((int)(tcount & 1u));
            for (int t = 0; t < nsteps; ++t) {
                const int ph = t < npre ? 0 : 1;             // 0: lower bounds only
                const int g = step_group(t);
                const int nch = (NC - 2 * g < 2) ? (NC - 2 * g) : 2;
                const bool screening = p.screen && g >= p.scr_group;
                const bool hi_grp = leading_only(g);
                const int tb = (int)(tcount & 1u);
                ++tcount;
                named_bar_sync(4 + grp, 128);                // the group's table is in place (and the other buffer free)
                const float4* tab = tab_s[tb][grp];
                if (t == 0 && npre > 0) {                    // the tile's first use of the exchange slots
                    xm_s[grp * 128 + pt] = thr_base;
                    named_bar_sync(3, 256);
                }
                if (screening) {
                    // What a pair is screened against: the point's maximum over the evaluated components (final by now; the
                    // two warpgroups merge theirs at the first screening group) and the largest LOWER bound among the listed
                    // components seen so far (each warpgroup publishes its own after every group and picks up the other's:
                    // a value that is a little old is still a valid bound).
                    if (ph == 1 && g == p.scr_group) {
                        const float mine = fmaxf(m_run, thr_base);
                        named_bar_sync(3, 256);               // (nobody still reads the slots of an earlier phase)
                        xm_s[grp * 128 + pt] = mine;
                        named_bar_sync(3, 256);
                        thr_base = fmaxf(mine, xm_s[(grp ^ 1) * 128 + pt]);
                        named_bar_sync(3, 256);
                        xm_s[grp * 128 + pt] = thr_base;
                    } else {
                        xm_s[grp * 128 + pt] = thr_base;
                        thr_base = fmaxf(thr_base, xm_s[(grp ^ 1) * 128 + pt]);
                    }
                }
                int half = 0;
                bool got;
                if (hi_grp) {
                    half = nb;
                    nb ^= 1;
                    got = bar_wait(BAR(LB_LFULL + half), (half ? ub1 : ub0) & 1u, abort_flag, p.status, false);
                    if (half) ++ub1; else ++ub0;
                } else {
                    got = bar_wait(BAR(LB_LFULL), ub0 & 1u, abort_flag, p.status, false);
                    got = bar_wait(BAR(LB_LFULL + 1), ub1 & 1u, abort_flag, p.status, false) && got;
                    ++ub0;
                    ++ub1;
                }
                const bool ok = __all_sync(0xffffffffu, got);
                fence_after();
                if (t + 1 < nsteps) table_load(step_group(t + 1));    // (in flight during this group's pass)
                const uint32_t acc = tmem + (uint32_t)(half * 256);
                if (ok) {
                    {
                        const int c = grp;
                        if (c < nch) {                       // uniform over the warpgroup
#pragma unroll 1
                        for (int sub = 0; sub < 4; ++sub) {
                            uint32_t v[32], vc[32];
                            tmem_ld32(acc + c * 128 + sub * 32 + lane_addr, v);
                            if (!hi_grp) tmem_ld32(tmem + 256 + c * 128 + sub * 32 + lane_addr, vc);
                            tmem_wait_ld();
                            const int col0 = (2 * g + c) * 128 + sub * 32;
                            const float4* tb4 = tab + sub * 32;
                            if (screening) {
                                // Columns of listed components (they take no part in the sums): their approximate values,
                                // raised by what they can be wrong by, tell which pairs can matter at all.  The point's
                                // maximum over the evaluated components is final by now.  (!(a < b): a NaN passes.)
                                if (tabm_s[tb][grp][sub] != 0 && row < p.n) {
                                    const float2* se2 = reinterpret_cast<const float2*>(&tabe_s[tb][grp][sub * 32]);
                                    // (topm: the block's largest upper bound and where - one candidate per block of 32
                                    // components for the ranks that no marked pair fills; an insertion per component
                                    // made the sweep four times slower, the insertions of 32 points diverge)
                                    float bub = -CUDART_INF_F;
                                    int bcol = col0;
#pragma unroll
                                    for (int j = 0; j < 32; j += 2) {
                                        const float4 t0 = tb4[j], t1 = tb4[j + 1];
                                        const float4 q = make_float4(t0.x, t0.y, t1.x, t1.y);
                                        const float4 sq = make_float4(t0.z, t0.w, t1.z, t1.w);
                                        const float2 se = se2[j >> 1];
                                        const float a0 = hi_grp ? __uint_as_float(v[j]) : __uint_as_float(v[j]) + __uint_as_float(vc[j]);
                                        const float a1 = hi_grp ? __uint_as_float(v[j + 1]) : __uint_as_float(v[j + 1]) + __uint_as_float(vc[j + 1]);
                                        const float u0 = fmaf(a0, q.x, fmaf(sq.y, nrm, sq.x));
                                        const float u1 = fmaf(a1, q.z, fmaf(sq.w, nrm, sq.z));
                                        // lower bounds: the upper bound minus twice the allowance (fmaxf drops a NaN)
                                        const float lb0 = u0 - 2.f * fmaf(sq.y, nrm, se.x), lb1 = u1 - 2.f * fmaf(sq.w, nrm, se.y);
                                        thr_base = fmaxf(thr_base, fmaxf(lb0, lb1));
                                        const float thr = thr_base - 40.f;
                                        if (NTOP > 2 && p.topm > 0) {
                                            if (u0 > bub && sq.x > -CUDART_INF_F) { bub = u0; bcol = col0 + j; }
                                            if (u1 > bub && sq.z > -CUDART_INF_F) { bub = u1; bcol = col0 + j + 1; }
                                        }
                                        if (ph == 0) continue;                          // (lower bounds only)
                                        if (!(u0 < thr) && sq.x > -CUDART_INF_F) mark(u0, tabs_s[tb][grp][sub * 32 + j]);
                                        if (!(u1 < thr) && sq.z > -CUDART_INF_F) mark(u1, tabs_s[tb][grp][sub * 32 + j + 1]);
                                    }
                                    if (NTOP > 2 && p.topm > 0 && ph == 1) tl.insert(bub, bcol);
                                }
                                continue;
                            }
                            float l[32];
                            float bmax = -CUDART_INF_F;
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                const float4 t0 = tb4[j], t1 = tb4[j + 1];       // same address in every lane
                                const float4 q = make_float4(t0.x, t0.y, t1.x, t1.y);
                                l[j] = fmaf(hi_grp ? __uint_as_float(v[j]) : __uint_as_float(v[j]) + __uint_as_float(vc[j]), q.x, q.y);
                                l[j + 1] = fmaf(hi_grp ? __uint_as_float(v[j + 1]) : __uint_as_float(v[j + 1]) + __uint_as_float(vc[j + 1]), q.z, q.w);
                                bmax = fmaxf(bmax, fmaxf(l[j], l[j + 1]));
                            }
                            if (bmax > m_run) {
                                s_run *= fast_ex2(m_run - bmax);
                                m_run = bmax;
                            }
                            if (NTOP == 2) {
                                if (bmax > tl.a[NTOP - 1]) { // (rare after the first chunks)
#pragma unroll
                                    for (int j = 0; j < 32; ++j) tl.insert(l[j], col0 + j);
                                }
                            } else {
                                // the assignment ranks by an UPPER bound of the exact value (approximate value + what it can be
                                // wrong by for this point): what is not reported then lies below the last reported bound
                                float bub = -CUDART_INF_F;
#pragma unroll
                                for (int j = 0; j < 32; j += 2) {
                                    const float4 t0 = tb4[j], t1 = tb4[j + 1];
                                    const float4 sq = make_float4(t0.z, t0.w, t1.z, t1.w);
                                    bub = fmaxf(bub, fmaxf(l[j] + fmaf(sq.y, nrm, sq.x), l[j + 1] + fmaf(sq.w, nrm, sq.z)));
                                }
                                if (bub > tl.a[NTOP - 1]) {
#pragma unroll
                                    for (int j = 0; j < 32; j += 2) {
                                        const float4 t0 = tb4[j], t1 = tb4[j + 1];
                                        const float4 sq = make_float4(t0.z, t0.w, t1.z, t1.w);
                                        tl.insert(l[j] + fmaf(sq.y, nrm, sq.x), col0 + j);
                                        tl.insert(l[j + 1] + fmaf(sq.w, nrm, sq.z), col0 + j + 1);
                                    }
                                }
                            }
                            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                acc0 += fast_ex2(l[j] - m_run);
                                acc1 += fast_ex2(l[j + 1] - m_run);
                            }
                            s_run += acc0 + acc1;
                        }
                        }
                    }
                }
                fence_before();
                if (hi_grp) bar_arrive(BAR(LB_LEMPTY + half));
                else { bar_arrive(BAR(LB_LEMPTY)); bar_arrive(BAR(LB_LEMPTY + 1)); }
                if (t + 1 < nsteps) table_store((int)(tcount & 1u));
            }
            // merge the two warpgroups' pairs; warpgroup 0 writes log2 Z and the two leading candidates
            if (p.rec) {
                xm_s[grp * 128 + pt] = thr_base;             // (each warpgroup's own slot; read after the barrier below)
                if (row < p.n) p.rec_cnt[2 * row + grp] = nrec;
            }
            if (grp == 1) {
                merge_s[pt] = make_float2(m_run, s_run);
#pragma unroll
                for (int j = 0; j < NTOP; ++j) { top_s[pt][j] = tl.a[j]; top_s[pt][NTOP + j] = __int_as_float(tl.i[j]); }
            }
            named_bar_sync(1, 256);
            if (grp == 0) {
                const float2 o = merge_s[pt];
                const float m = fmaxf(m_run, o.x);
                const float s = s_run * fast_ex2(m_run - m) + o.y * fast_ex2(o.x - m);
#pragma unroll
                for (int j = 0; j < NTOP; ++j) tl.insert(top_s[pt][j], __float_as_int(top_s[pt][NTOP + j]));
                if (row < p.n && !*abort_flag) {
                    const double lz = cref + (double)m + (double)log2f(s);
                    p.logz[row] = lz;
                    float* tp = p.top + row * (2 * NTOP);
#pragma unroll
                    for (int j = 0; j < NTOP; ++j) { tp[j] = tl.a[j]; tp[NTOP + j] = __int_as_float(tl.i[j]); }
                    ll_acc += lz;
                    if (p.rec) p.rec_thr[row] = fmaxf(thr_base, xm_s[128 + pt]);
                }
            }
            named_bar_sync(2, 256);                          // merge_s is rewritten by the next tile
        }
        // (one addition per warp: an addition per thread and tile, all to one address, kept an L2 slice busy for a third
        // of the sweep's time)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) nhit += __shfl_xor_sync(0xffffffffu, nhit, o);
        if (lane == 0 && nhit > 0) atomicAdd(p.ctl, nhit);
        if (grp == 0) ll_s[pt] = ll_acc;
        named_bar_sync(1, 256);
        if (tid == 0 && p.llpart) {
            double s = 0.0;
            for (int j = 0; j < 128; ++j) s += ll_s[j];
            p.llpart[blockIdx.x] += s * 0.69314718055994530942;       // one owner per slot: launches add up
        }
    } else if (warp == WT_PRODUCER) {
        // =========================== producer warp (TMA) ===========================
        // Stage order = order of use: per (tile, step of the tile, atom z) the hi planes' stage, then (unless the group forms
        // the leading product only) the lo planes' stage.
        int64_t g = 0;
        bool ok = true;
        // Both streams are kept in L2 with priority: the coefficient atoms are read by every CTA for every tile, the tile's
        // own atoms once per step of the tile.  (Marked evict-first, the tile's atoms missed L2 on nearly every re-read -
        // a third of the sweep's sectors came from DRAM, 17 % of its time: L2 is full of older lines of normal priority,
        // e.g. the planes as the transform wrote them, which such lines do not displace.)
        const uint64_t pol_keep = l2_policy_evict_last();
        auto stage = [&](const CUtensorMap* my, const CUtensorMap* mp, int32_t yrow, int32_t prow, int nch, int32_t z) -> bool {
            const int slot = (int)(g % L_SLOTS);
            const int64_t use = g / L_SLOTS;
            if (use > 0) {
                uint32_t w = 1;
                if (lane == 0) w = bar_wait(BAR(LB_EMPTY + slot), (uint32_t)((use - 1) & 1), abort_flag, p.status, false) ? 1u : 0u;
                if (!__shfl_sync(0xffffffffu, w, 0)) return false;
            }
            if (elect_one()) {
                const uint32_t dst = smem_u32(smem + slot * L_STAGE);
                bar_expect_tx(BAR(LB_FULL + slot), (uint32_t)((1 + nch) * HSLOT));
                tma_load_3d_hint(dst, my, 0, yrow, z, BAR(LB_FULL + slot), pol_keep);
                for (int c = 0; c < nch; ++c)
                    tma_load_3d_hint(dst + (uint32_t)((1 + c) * HSLOT), mp, 0, prow + c * 128, z, BAR(LB_FULL + slot), pol_keep);
            }
            __syncwarp();
            ++g;
            return true;
        };
        for (int64_t i = 0; i < ntl && ok; ++i) {
            const int32_t row0 = (int32_t)((blockIdx.x + i * gridDim.x) * WIDE_TILE);
            for (int t = 0; t < nsteps && ok; ++t) {
                const int gq = step_group(t);
                const int nch = (NC - 2 * gq < 2) ? (NC - 2 * gq) : 2;
                const bool hi_only = leading_only(gq);
                for (int z = 0; z < NZ && ok; ++z) {
                    ok = stage(&tm_yhi, &tm_phi, row0, 2 * gq * 128, nch, z);
                    if (ok && !hi_only) ok = stage(&tm_ylo, &tm_plo, row0, 2 * gq * 128, nch, z);
                }
            }
        }
        // the loads in flight must have landed before the CTA may exit, also after an abort
        if (!ok || *abort_flag) {
            for (int64_t h = (g > L_SLOTS ? g - L_SLOTS : 0); h < g; ++h) {
                if (lane == 0) bar_wait(BAR(LB_FULL + (int)(h % L_SLOTS)), (uint32_t)((h / L_SLOTS) & 1), drain_flag, p.status, false);
                __syncwarp();
            }
        }
    } else {
        // =========================== MMA warp ===========================
        const uint32_t idesc1 = make_idesc(WIDE_TILE, 128, 0), idesc2 = make_idesc(WIDE_TILE, 256, 0);
        const uint64_t d0 = make_desc(smem_u32(smem), 16, 1024);
        bool alive = true;
        auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
            uint32_t ok = 1;
            if (lane == 0) ok = bar_wait(bar, parity, abort_flag, p.status, false) ? 1u : 0u;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            fence_after();
            return ok != 0u;
        };
        int64_t g = 0;
        uint32_t ub0 = 0, ub1 = 0;                           // uses of the two accumulator halves
        int nb = 0;
        auto take = [&](int& slot) -> bool {                 // the next stage of the ring, once it has landed
            slot = (int)(g % L_SLOTS);
            const bool ok = wait_all(BAR(LB_FULL + slot), (uint32_t)((g / L_SLOTS) & 1));
            ++g;
            return ok;
        };
        for (int64_t i = 0; i < ntl && alive; ++i) {
            for (int t = 0; t < nsteps && alive; ++t) {
                const int gq = step_group(t);
                const int nch = (NC - 2 * gq < 2) ? (NC - 2 * gq) : 2;
                const bool hi_only = leading_only(gq);
                const uint32_t idesc = nch == 2 ? idesc2 : idesc1;       // both chunks of the group as one operand of 256 rows
                // the softmax warps must be done with the accumulator columns this group writes
                int half = 0;
                if (hi_only) {
                    half = nb;
                    nb ^= 1;
                    const uint32_t u = half ? ub1 : ub0;
                    if (u > 0 && !wait_all(BAR(LB_LEMPTY + half), (u - 1) & 1u)) { alive = false; break; }
                } else {
                    if (ub0 > 0 && !wait_all(BAR(LB_LEMPTY), (ub0 - 1) & 1u)) { alive = false; break; }
                    if (ub1 > 0 && !wait_all(BAR(LB_LEMPTY + 1), (ub1 - 1) & 1u)) { alive = false; break; }
                }
                const uint32_t d = tmem + half * 256, dc = tmem + 256;
                for (int z = 0; z < NZ && alive; ++z) {
                    int sh = 0, sl = 0;
                    if (!take(sh)) { alive = false; break; }
                    if (!hi_only && !take(sl)) { alive = false; break; }
                    if (elect_one()) {
                        const uint64_t ah = d0 + ((sh * L_STAGE) >> 4), bh = ah + (HSLOT >> 4);
                        // the two small cross products into their own accumulator, the leading product into the main one:
                        // the same three chains, in the same order, as the E-step of sweep 2
                        if (!hi_only) {
                            const uint64_t al = d0 + ((sl * L_STAGE) >> 4), bl = al + (HSLOT >> 4);
#pragma unroll
                            for (int j = 0; j < 4; ++j) mma_ss(dc, ah + ((j * 32) >> 4), bl + ((j * 32) >> 4), idesc, (z > 0 || j > 0) ? 1u : 0u);
#pragma unroll
                            for (int j = 0; j < 4; ++j) mma_ss(dc, al + ((j * 32) >> 4), bh + ((j * 32) >> 4), idesc, 1u);
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) mma_ss(d, ah + ((j * 32) >> 4), bh + ((j * 32) >> 4), idesc, (z > 0 || j > 0) ? 1u : 0u);
                        mma_commit(BAR(LB_EMPTY + sh));
                        if (!hi_only) mma_commit(BAR(LB_EMPTY + sl));
                        if (z == NZ - 1) {
                            if (hi_only) mma_commit(BAR(LB_LFULL + half));
                            else { mma_commit(BAR(LB_LFULL)); mma_commit(BAR(LB_LFULL + 1)); }
                        }
                    }
                    __syncwarp();
                }
                if (hi_only) { if (half) ++ub1; else ++ub0; }
                else { ++ub0; ++ub1; }
            }
        }
        if (elect_one()) mma_commit(BAR(LB_FINAL));
        __syncwarp();
        if (lane == 0) bar_wait(BAR(LB_FINAL), 0, drain_flag, p.status, false);
        __syncwarp();
        fence_after();
    }

    fence_before();
    __syncthreads();
    if (warp == WT_MMA) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------------------------
// Sweep 2
constexpr int E_SLOTS = 6;
constexpr int E_BAR = E_SLOTS * SLOT;
constexpr int E_LZ = E_BAR + 256;                  // 2 x 256 doubles: log2 Z of the batch's points
constexpr int E_SMEM = E_LZ + 4096 + 1024;
enum { EB_FULL = 0, EB_EMPTY = E_SLOTS, EB_LFULL = 2 * E_SLOTS, EB_RREADY, EB_ACCFULL0, EB_ACCFULL1, EB_ACCFREE0,
       EB_ACCFREE1, EB_FINAL, EB_COUNT };

struct EmWideParams {
    int64_t n;
    int CL, R, NZ, pcols;
    const float2* tkck;
    const double* ckd;
    const double* logz;
    float* partial;      // [R * CL][pcols][128]
    int* status;
};

__global__ void __launch_bounds__(WT_THREADS, 1)
em_wide_kernel(const EmWideParams p, const __grid_constant__ CUtensorMap tm_phi, const __grid_constant__ CUtensorMap tm_plo,
               const __grid_constant__ CUtensorMap tm_ye_hi, const __grid_constant__ CUtensorMap tm_ye_lo,
               const __grid_constant__ CUtensorMap tm_ym_hi, const __grid_constant__ CUtensorMap tm_ym_lo) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, drain_s;
    volatile int* abort_flag = &abort_s;
    volatile int* drain_flag = &drain_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slice = blockIdx.x % p.CL;                 // 128 components
    const int range = blockIdx.x / p.CL;                 // takes batches range, range + R, ...
    const int64_t nbatches = (p.n + WIDE_BATCH - 1) / WIDE_BATCH;
    const int64_t nbl = (range < nbatches) ? (nbatches - range + p.R - 1) / p.R : 0;
    const int NZ = p.NZ, NH = NZ >> 1;                   // atoms; half-slices of 64 dimensions (2 atoms = 128 columns)

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + E_BAR);
    auto BAR = [&](int i) { return smem_u32(&bars[i]); };
    if (tid == 0) {
        abort_s = 0;
        drain_s = 0;
        for (int s = 0; s < E_SLOTS; ++s) { bar_init(BAR(EB_FULL + s), 1); bar_init(BAR(EB_EMPTY + s), 1); }
        bar_init(BAR(EB_LFULL), 1);
        bar_init(BAR(EB_RREADY), 256);
        bar_init(BAR(EB_ACCFULL0), 1);  bar_init(BAR(EB_ACCFULL1), 1);
        bar_init(BAR(EB_ACCFREE0), 256); bar_init(BAR(EB_ACCFREE1), 256);
        bar_init(BAR(EB_FINAL), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == WT_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = tmem_base_s;
    // TMEM columns: [0,128) / [128,256) the two alternating M-step accumulators (during the E-step: the accumulator of the
    // two small cross products, points 0-255), [256,512) the main E-step product of the batch's 256 points, overwritten
    // in place by the responsibilities: 32 points -> [r_hi 16 columns | r_lo 16 columns]
    const uint32_t T_MAIN = tmem + 256;

    if (warp < 8) {
        // =========================== softmax / flush warps: thread = TMEM lane = component ===========================
        const int grp = warp >> 2, wq = warp & 3;
        const uint32_t lane_addr = ((uint32_t)(wq * 32)) << 16;
        const int kloc = wq * 32 + lane;
        const float2 tc = __ldg(p.tkck + slice * 128 + kloc);
        // c_k - log2 Z_i is formed in float64 (both are in the thousands, their difference is what the exponent needs)
        const double ckd = (tc.y == -CUDART_INF_F) ? -CUDART_INF : __ldg(p.ckd + slice * 128 + kloc);
        double* lz_s = reinterpret_cast<double*>(smem + E_LZ);            // [2][256]
        float* pblk = p.partial + (size_t)blockIdx.x * p.pcols * 128 + kloc;      // [column][component]: one owner per address
        uint32_t acc_uses[2] = {0u, 0u};
        for (int64_t b = 0; b < nbl; ++b) {
            const int64_t row0 = (range + b * p.R) * WIDE_BATCH;
            double* lz = lz_s + (b & 1) * 256;
            {   // log2 Z of the batch's points (+inf beyond n: those points get r = 0)
                const int64_t row = row0 + (tid & 255);
                lz[tid & 255] = (row < p.n) ? p.logz[row] : CUDART_INF;
            }
            named_bar_sync(1, 256);
            const bool got = bar_wait(BAR(EB_LFULL), (uint32_t)(b & 1), abort_flag, p.status, false);
            const bool ok = __all_sync(0xffffffffu, got);
            fence_after();
            float nsum = 0.f;
            if (ok) {
#pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    const int p0 = 128 * grp + 32 * ch;                   // this thread's 32 points of the batch
                    uint32_t vm[32], vc[32];
                    tmem_ld32(T_MAIN + p0 + lane_addr, vm);
                    tmem_ld32(tmem + p0 + lane_addr, vc);
                    tmem_wait_ld();
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const double2 za = *reinterpret_cast<const double2*>(lz + p0 + j);
                        const double2 zb = *reinterpret_cast<const double2*>(lz + p0 + j + 2);
                        float r[4];
                        const double zz[4] = {za.x, za.y, zb.x, zb.y};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float acc = __uint_as_float(vm[j + q]) + __uint_as_float(vc[j + q]);
                            r[q] = fast_ex2(fmaf(acc, tc.x, (float)(ckd - zz[q]))) * RSCALE;
                        }
                        const __half2 h01 = __floats2half2_rn(r[0], r[1]), h23 = __floats2half2_rn(r[2], r[3]);
                        const float2 b01 = __half22float2(h01), b23 = __half22float2(h23);
                        const __half2 g01 = __floats2half2_rn(r[0] - b01.x, r[1] - b01.y), g23 = __floats2half2_rn(r[2] - b23.x, r[3] - b23.y);
                        const float2 c01 = __half22float2(g01), c23 = __half22float2(g23);
                        // N_k is the sum of exactly the weights the M-step uses (hi + lo)
                        nsum += ((b01.x + c01.x) + (b01.y + c01.y)) + ((b23.x + c23.x) + (b23.y + c23.y));
                        hi[j / 2] = *reinterpret_cast<const uint32_t*>(&h01);
                        hi[j / 2 + 1] = *reinterpret_cast<const uint32_t*>(&h23);
                        lo[j / 2] = *reinterpret_cast<const uint32_t*>(&g01);
                        lo[j / 2 + 1] = *reinterpret_cast<const uint32_t*>(&g23);
                    }
                    tmem_st16(T_MAIN + p0 + lane_addr, hi);
                    tmem_st16(T_MAIN + p0 + 16 + lane_addr, lo);
                }
                tmem_wait_st();
            }
            fence_before();
            bar_arrive(BAR(EB_RREADY));
            if (ok) atomicAdd(pblk + (size_t)(p.pcols - 2 + grp) * 128, nsum);         // N_k column of this warpgroup
            // flush the M-step accumulators, half-slice by half-slice, as the MMA warp hands them over: warpgroup g takes
            // columns [64 g, 64 g + 64) of the 128
            for (int h = 0; h < NH; ++h) {
                const int buf = h & 1;
                const bool gotf = bar_wait(BAR(EB_ACCFULL0 + buf), acc_uses[buf] & 1u, abort_flag, p.status, false);
                const bool okf = __all_sync(0xffffffffu, gotf);
                ++acc_uses[buf];
                fence_after();
                if (okf) {
#pragma unroll 1
                    for (int c0 = 0; c0 < 64; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(tmem + buf * 128 + grp * 64 + c0 + lane_addr, v);
                        tmem_wait_ld();
                        float* dst = pblk + (size_t)(h * 128 + grp * 64 + c0) * 128;
#pragma unroll
                        for (int j = 0; j < 32; ++j) atomicAdd(dst + (size_t)j * 128, __uint_as_float(v[j]));
                    }
                }
                fence_before();
                bar_arrive(BAR(EB_ACCFREE0 + buf));
            }
        }
    } else if (warp == WT_PRODUCER) {
        // =========================== producer warp (TMA) ===========================
        // Items in order of use.  E-step, per atom z: the slice's coefficient atom (hi, lo: 2 x 16 KB in one slot), the batch's
        // Y atom hi (256 points x 128 bytes: one slot), the same of the lo plane.  M-step, per half-slice and quarter of the
        // batch: 64 points x 2 atoms of both planes (2 x 16 KB in one slot).
        int64_t g = 0;
        bool ok = true;
        const uint64_t pol_keep = l2_policy_evict_last();     // the slice's coefficient atoms come back with every batch
        auto acquire = [&]() -> int {
            const int slot = (int)(g % E_SLOTS);
            const int64_t use = g / E_SLOTS;
            if (use > 0) {
                uint32_t w = 1;
                if (lane == 0) w = bar_wait(BAR(EB_EMPTY + slot), (uint32_t)((use - 1) & 1), abort_flag, p.status, false) ? 1u : 0u;
                if (!__shfl_sync(0xffffffffu, w, 0)) return -1;
            }
            return slot;
        };
        for (int64_t b = 0; b < nbl && ok; ++b) {
            const int32_t row0 = (int32_t)((range + b * p.R) * WIDE_BATCH);
            for (int z = 0; z < NZ && ok; ++z) {
                int slot = acquire();
                if (slot < 0) { ok = false; break; }
                if (elect_one()) {
                    const uint32_t dst = smem_u32(smem + slot * SLOT);
                    bar_expect_tx(BAR(EB_FULL + slot), SLOT);
                    tma_load_3d_hint(dst, &tm_phi, 0, slice * 128, z, BAR(EB_FULL + slot), pol_keep);
                    tma_load_3d_hint(dst + SLOT / 2, &tm_plo, 0, slice * 128, z, BAR(EB_FULL + slot), pol_keep);
                }
                __syncwarp();
                ++g;
                for (int pl = 0; pl < 2 && ok; ++pl) {
                    slot = acquire();
                    if (slot < 0) { ok = false; break; }
                    if (elect_one()) {
                        bar_expect_tx(BAR(EB_FULL + slot), SLOT);
                        tma_load_3d(smem_u32(smem + slot * SLOT), pl ? &tm_ye_lo : &tm_ye_hi, 0, row0, z, BAR(EB_FULL + slot));
                    }
                    __syncwarp();
                    ++g;
                }
            }
            for (int h = 0; h < NH && ok; ++h) {
                for (int q4 = 0; q4 < 4 && ok; ++q4) {
                    const int slot = acquire();
                    if (slot < 0) { ok = false; break; }
                    if (elect_one()) {
                        const uint32_t dst = smem_u32(smem + slot * SLOT);
                        bar_expect_tx(BAR(EB_FULL + slot), SLOT);
                        tma_load_3d(dst, &tm_ym_hi, 0, row0 + 64 * q4, 2 * h, BAR(EB_FULL + slot));
                        tma_load_3d(dst + SLOT / 2, &tm_ym_lo, 0, row0 + 64 * q4, 2 * h, BAR(EB_FULL + slot));
                    }
                    __syncwarp();
                    ++g;
                }
            }
        }
        if (!ok || *abort_flag) {
            for (int64_t h = (g > E_SLOTS ? g - E_SLOTS : 0); h < g; ++h) {
                if (lane == 0) bar_wait(BAR(EB_FULL + (int)(h % E_SLOTS)), (uint32_t)((h / E_SLOTS) & 1), drain_flag, p.status, false);
                __syncwarp();
            }
        }
    } else {
        // =========================== MMA warp ===========================
        const uint32_t id_e = make_idesc(128, WIDE_BATCH, 0);       // E-step: M = 128 components, N = 256 points, both K-major
        const uint32_t id_m = make_idesc(128, 128, 1);              // M-step: N = 128 statistics columns, B MN-major
        const uint64_t dk = make_desc(smem_u32(smem), 16, 1024);    // K-major view of the ring
        const uint64_t dm = make_desc(smem_u32(smem), 8192, 1024);  // MN-major view: 64-column atoms of 64 points, 8192 bytes apart
        bool alive = true;
        auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
            uint32_t ok = 1;
            if (lane == 0) ok = bar_wait(bar, parity, abort_flag, p.status, false) ? 1u : 0u;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            fence_after();
            return ok != 0u;
        };
        int64_t g = 0;
        uint32_t full_cnt[2] = {0u, 0u}, freed_cnt[2] = {0u, 0u};
        // an accumulator may be written again only when every earlier hand-over of it has been flushed
        auto ensure_free = [&](int buf) -> bool {
            while (freed_cnt[buf] < full_cnt[buf]) {
                if (!wait_all(BAR(EB_ACCFREE0 + buf), freed_cnt[buf] & 1u)) return false;
                ++freed_cnt[buf];
            }
            return true;
        };
        for (int64_t b = 0; b < nbl && alive; ++b) {
            // ---- E-step: the cross products use columns [0, 256), i.e. both M-step accumulators
            if (!ensure_free(0) || !ensure_free(1)) { alive = false; break; }
            for (int z = 0; z < NZ && alive; ++z) {
                int sl[3];
                for (int q = 0; q < 3; ++q) {
                    sl[q] = (int)(g % E_SLOTS);
                    if (!wait_all(BAR(EB_FULL + sl[q]), (uint32_t)((g / E_SLOTS) & 1))) { alive = false; break; }
                    ++g;
                }
                if (!alive) break;
                if (elect_one()) {
                    const uint64_t ph = dk + ((sl[0] * SLOT) >> 4), plo = ph + ((SLOT / 2) >> 4);
                    const uint64_t yh = dk + ((sl[1] * SLOT) >> 4), yl = dk + ((sl[2] * SLOT) >> 4);
#pragma unroll
                    for (int j = 0; j < 4; ++j) mma_ss(tmem, plo + ((j * 32) >> 4), yh + ((j * 32) >> 4), id_e, (z > 0 || j > 0) ? 1u : 0u);
#pragma unroll
                    for (int j = 0; j < 4; ++j) mma_ss(tmem, ph + ((j * 32) >> 4), yl + ((j * 32) >> 4), id_e, 1u);
#pragma unroll
                    for (int j = 0; j < 4; ++j) mma_ss(T_MAIN, ph + ((j * 32) >> 4), yh + ((j * 32) >> 4), id_e, (z > 0 || j > 0) ? 1u : 0u);
                    mma_commit(BAR(EB_EMPTY + sl[0]));
                    mma_commit(BAR(EB_EMPTY + sl[1]));
                    mma_commit(BAR(EB_EMPTY + sl[2]));
                    if (z == NZ - 1) mma_commit(BAR(EB_LFULL));
                }
                __syncwarp();
            }
            if (!alive) break;
            // ---- M-step
            if (!wait_all(BAR(EB_RREADY), (uint32_t)(b & 1))) { alive = false; break; }
            for (int h = 0; h < NH && alive; ++h) {
                const int buf = h & 1;
                if (!ensure_free(buf)) { alive = false; break; }
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int s = (int)(g % E_SLOTS);
                    if (!wait_all(BAR(EB_FULL + s), (uint32_t)((g / E_SLOTS) & 1))) { alive = false; break; }
                    ++g;
                    if (elect_one()) {
                        const uint64_t yh = dm + ((s * SLOT) >> 4), yl = yh + ((SLOT / 2) >> 4);
                        const uint32_t d = tmem + buf * 128;
                        // A operand: 16 points per k-step; points 32 c .. 32 c + 31 sit in columns [32 c, 32 c + 16) (r_hi) and
                        // [32 c + 16, 32 c + 32) (r_lo) of the main buffer
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const int kg = 4 * q4 + ks;
                            mma_ts(d, T_MAIN + (kg >> 1) * 32 + (kg & 1) * 8, yh + ((ks * 2048) >> 4), id_m, (q4 > 0 || ks > 0) ? 1u : 0u);
                        }
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const int kg = 4 * q4 + ks;
                            mma_ts(d, T_MAIN + (kg >> 1) * 32 + (kg & 1) * 8, yl + ((ks * 2048) >> 4), id_m, 1u);
                        }
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const int kg = 4 * q4 + ks;
                            mma_ts(d, T_MAIN + (kg >> 1) * 32 + (kg & 1) * 8 + 16, yh + ((ks * 2048) >> 4), id_m, 1u);
                        }
                        mma_commit(BAR(EB_EMPTY + s));
                        if (q4 == 3) mma_commit(BAR(EB_ACCFULL0 + buf));
                    }
                    __syncwarp();
                }
                if (alive) ++full_cnt[buf];
            }
        }
        if (elect_one()) mma_commit(BAR(EB_FINAL));
        __syncwarp();
        if (lane == 0) bar_wait(BAR(EB_FINAL), 0, drain_flag, p.status, false);
        __syncwarp();
        fence_after();
    }

    fence_before();
    __syncthreads();
    if (warp == WT_MMA) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------------------------
// X -> the two fp16 planes of Y = [u | u^2 + kap], u = s_d (x - g_d).  A point has 2 Dpad halves per plane: k-step ks (8
// dimensions) occupies halves [16 ks, 16 ks + 8) = u and [16 ks + 8, 16 ks + 16) = u^2 + kap.  A plane is stored atom by
// atom (an atom = 64 halves = 4 k-steps of every point: [atom][point][128 bytes]), so that the tiles the sweeps load -
// some rows of one atom - are contiguous in memory.  One thread converts one (point, k-step) unit and writes 32
// contiguous bytes per plane.  Rows n .. rows_padded - 1 are written as zeros.
__global__ void __launch_bounds__(256) wide_transform_kernel(const float* __restrict__ X, int64_t n, int64_t rows_padded, int D,
                                                             int Dpad, const float* __restrict__ sd, const float* __restrict__ kap,
                                                             const float* __restrict__ gd, unsigned char* __restrict__ yhi,
                                                             unsigned char* __restrict__ ylo, float* __restrict__ n2,
                                                             int* __restrict__ status) {
    // A warp per row (its units lane, lane + 32, ...), so that |x - g|^2 of the row (n2, may be NULL: what the screening
    // bounds need) comes out of the same pass in a fixed order of additions.
    const int upr = Dpad >> 3;                           // units per row
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const bool vec_ok = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15) == 0);
    bool bad = false;
    for (int64_t row = warp0; row < rows_padded; row += nwarps) {
        const bool valid = row < n;
        float nrm = 0.f;
        for (int ks = lane; ks < upr; ks += 32) {
            const int d0 = ks * 8;
            float x[8];
            if (valid && vec_ok && d0 + 8 <= D) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(X + row * D + d0));
                const float4 b = __ldg(reinterpret_cast<const float4*>(X + row * D + d0 + 4));
                x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) x[j] = (valid && d0 + j < D) ? __ldg(X + row * D + d0 + j) : 0.f;
            }
            // (the per-dimension constants in 16-byte loads: the arrays hold Dpad entries and start on 256-byte boundaries;
            // one load per element kept the load/store unit's queue full and the kernel at a third of the DRAM bandwidth)
            float gv[8], sv[8], kv[8];
            {
                const float4 g0 = __ldg(reinterpret_cast<const float4*>(gd + d0)), g1 = __ldg(reinterpret_cast<const float4*>(gd + d0) + 1);
                const float4 s0 = __ldg(reinterpret_cast<const float4*>(sd + d0)), s1 = __ldg(reinterpret_cast<const float4*>(sd + d0) + 1);
                const float4 k0 = __ldg(reinterpret_cast<const float4*>(kap + d0)), k1 = __ldg(reinterpret_cast<const float4*>(kap + d0) + 1);
                gv[0] = g0.x; gv[1] = g0.y; gv[2] = g0.z; gv[3] = g0.w; gv[4] = g1.x; gv[5] = g1.y; gv[6] = g1.z; gv[7] = g1.w;
                sv[0] = s0.x; sv[1] = s0.y; sv[2] = s0.z; sv[3] = s0.w; sv[4] = s1.x; sv[5] = s1.y; sv[6] = s1.z; sv[7] = s1.w;
                kv[0] = k0.x; kv[1] = k0.y; kv[2] = k0.z; kv[3] = k0.w; kv[4] = k1.x; kv[5] = k1.y; kv[6] = k1.z; kv[7] = k1.w;
            }
            uint32_t xh[4], xl[4], qh[4], ql[4];
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                bad |= !(fabsf(x[j]) <= 3.0e38f) || !(fabsf(x[j + 1]) <= 3.0e38f);
                const bool in0 = valid && d0 + j < D, in1 = valid && d0 + j + 1 < D;
                const float c0 = in0 ? x[j] - gv[j] : 0.f, c1 = in1 ? x[j + 1] - gv[j + 1] : 0.f;
                nrm = fmaf(c0, c0, fmaf(c1, c1, nrm));
                float u0 = c0 * sv[j];
                float u1 = c1 * sv[j + 1];
                u0 = fminf(fmaxf(u0, -240.f), 240.f);
                u1 = fminf(fmaxf(u1, -240.f), 240.f);
                const float q0 = in0 ? fmaf(u0, u0, kv[j]) : 0.f;
                const float q1 = in1 ? fmaf(u1, u1, kv[j + 1]) : 0.f;
                const __half2 h = __floats2half2_rn(u0, u1);
                const float2 hf = __half22float2(h);
                const __half2 g2 = __floats2half2_rn(u0 - hf.x, u1 - hf.y);
                const __half2 sq = __floats2half2_rn(q0, q1);
                const float2 sf = __half22float2(sq);
                const __half2 t2 = __floats2half2_rn(q0 - sf.x, q1 - sf.y);
                xh[j / 2] = *reinterpret_cast<const uint32_t*>(&h);
                xl[j / 2] = *reinterpret_cast<const uint32_t*>(&g2);
                qh[j / 2] = *reinterpret_cast<const uint32_t*>(&sq);
                ql[j / 2] = *reinterpret_cast<const uint32_t*>(&t2);
            }
            const size_t o = ((size_t)(ks >> 2) * rows_padded + row) * 128 + (ks & 3) * 32;      // [atom][row][128 bytes]
            uint4* oh = reinterpret_cast<uint4*>(yhi + o);
            oh[0] = make_uint4(xh[0], xh[1], xh[2], xh[3]);
            oh[1] = make_uint4(qh[0], qh[1], qh[2], qh[3]);
            if (ylo) {                                           // (NULL: the sweep that follows forms leading products only)
                uint4* ol = reinterpret_cast<uint4*>(ylo + o);
                ol[0] = make_uint4(xl[0], xl[1], xl[2], xl[3]);
                ol[1] = make_uint4(ql[0], ql[1], ql[2], ql[3]);
            }
        }
        if (n2) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, o);
            if (lane == 0 && valid) n2[row] = (nrm <= 3e38f) ? nrm : 3e38f;     // (a NaN or an infinity in X is reported below)
        }
    }
    if (bad) atomicOr(status, ST_BAD_X);
}

// ------------------------------------------------------------------------------------------------------------------
// Parameter preparation (float64 arithmetic on K * D elements).
// One block per dimension: centre g_d = sum_k pi_k mu_kd / sum_k pi_k, scale s_d = 2^-round(log2 rms_d) with
// rms_d^2 = sum_k pi_k ((mu_kd - g_d)^2 + var_kd), and the constant kap_d added to the squares.
// kap_d: a point of component k (x = mu + sigma z) adds a u + b (u^2 + kap) = w2 ((mu'^2 - kap') - (x' - mu')^2) to the
// accumulator in dimension d (w2 = log2 e / (2 var), primes: centred, unscaled), on average w2 (mu'^2 - var - kap').
// kap'_d is chosen so that this average vanishes over the mixture, each component weighted by pi_k w2_kd:
//     kap'_d = sum_k pi_k w2_kd (mu'_kd^2 - var_kd) / sum_k pi_k w2_kd
// (the weight w2 matters: with variances that differ between components, E[var] E[1 / var] > 1, and the plain average
// leaves every component a drift of hundreds of log2 units at D = 768).  The contraction's partial sums are then a
// zero-mean walk over the dimensions, tens in size instead of D / 2, and the truncation error of the tensor core's fp32
// accumulation shrinks with them.  A component much narrower than the rest (one collapsed onto a point, say) has its
// weight capped at 16 times that of the average variance, so that it cannot pull kap_d toward itself.
__global__ void __launch_bounds__(128) wide_scale_kernel(int D, int K, const float* __restrict__ pi, const float* __restrict__ mu,
                                                         const float* __restrict__ var, float* __restrict__ sd,
                                                         float* __restrict__ kap, float* __restrict__ gd) {
    const int d = blockIdx.x, t = threadIdx.x;
    __shared__ double r_a[128], r_b[128], r_w[128];
    __shared__ double g_s, v_s;
    double a = 0.0, w = 0.0, v0 = 0.0;
    if (d < D)
        for (int k = t; k < K; k += 128) {
            const double pk = (double)pi[k];
            a += pk * (double)mu[(size_t)k * D + d];
            v0 += pk * (double)var[(size_t)k * D + d];
            w += pk;
        }
    r_a[t] = a; r_b[t] = v0; r_w[t] = w;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (t < o) { r_a[t] += r_a[t + o]; r_b[t] += r_b[t + o]; r_w[t] += r_w[t + o]; }
        __syncthreads();
    }
    if (t == 0) {
        const float gf = (r_w[0] > 0.0) ? (float)(r_a[0] / r_w[0]) : 0.f;
        g_s = (d < D && isfinite(gf)) ? (double)gf : 0.0;
        v_s = (r_w[0] > 0.0) ? r_b[0] / r_w[0] : 0.0;          // the mixture's average variance in this dimension
    }
    __syncthreads();
    const double g = g_s, vbar = v_s;
    const double wcap = (vbar > 0.0 && isfinite(vbar)) ? 16.0 / vbar : 0.0;
    double m2 = 0.0, num = 0.0, den = 0.0;
    w = 0.0;
    if (d < D)
        for (int k = t; k < K; k += 128) {
            const double pk = (double)pi[k];
            const double m = (double)mu[(size_t)k * D + d] - g;
            const double v = (double)var[(size_t)k * D + d];
            m2 += pk * m * m;
            w += pk;
            if (v > 0.0) {
                const double wk = pk * fmin(1.0 / v, wcap);
                num += wk * (m * m - v);
                den += wk;
            }
        }
    __syncthreads();
    r_a[t] = m2; r_w[t] = w;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (t < o) { r_a[t] += r_a[t + o]; r_w[t] += r_w[t + o]; }
        __syncthreads();
    }
    const double mm_tot = r_a[0], w_tot = r_w[0];
    __syncthreads();
    r_a[t] = num; r_b[t] = den;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (t < o) { r_a[t] += r_a[t + o]; r_b[t] += r_b[t + o]; }
        __syncthreads();
    }
    if (t == 0) {
        float s = 1.f, kp = 0.f;
        const double mm = w_tot > 0.0 ? mm_tot / w_tot : 0.0;
        const double ms = mm + vbar;
        if (d < D && ms > 0.0 && isfinite(ms)) {
            const double e = rint(0.5 * log2(ms));
            s = (float)exp2(-fmin(fmax(e, -60.0), 60.0));
            const double kq = (r_b[0] > 0.0) ? r_a[0] / r_b[0] : (mm - vbar);
            kp = isfinite(kq) ? (float)(kq * (double)s * (double)s) : 0.f;
        }
        sd[d] = s;
        kap[d] = kp;
        gd[d] = (float)g;
    }
}

// One block per component: the error estimate of its approximate logits, and whether the tensor passes may take it.
// Error estimate of the approximate log2 z of the pairs that matter (points of the component itself).
// (i) operand rounding at 2^-22 of every term, terms of independent sign.  (ii) The tensor core truncates its fp32
// accumulator at each of the Dpad / 8 steps of the main product, by half an ulp (2^-24 relative) on average and
// always toward zero: with the accumulator climbing to A = |mean drift of the component| + 2 standard deviations
// of the walk (each dimension adds (log2 e / 2)(z^2 - 1), standard deviation 1.02), that is about
// (Dpad / 16) 2^-23 A.  The drift is what kap_d cannot remove: kap_d centres the mixture's average component,
// a component whose sum_d (mu'^2 - var) / var is far from that average keeps the difference.
// A component that holds few points (pi_k N below a threshold) is evaluated exactly as well: its parameters are
// averages over few responsibilities, which for a component far from most of its points are formed from large
// accumulators (|log2 z - c_k| in the thousands) whose truncation error nothing averages out.
// Output: illb[k] > 0 for a flagged component (two kinds, kept apart by the list kernel.  Flagged by the rounding estimate:
// narrow in some or all dimensions, hopeless for most points -- the mark is 8 x that estimate.  Flagged for its drift or its
// weight alone: broad -- a tiny positive mark); scra[k], scrw[k]: what the approximate log2 z of ANY point can be wrong by
// is at most scra + scrw |x - g|^2.  (Every term a u + b (u^2 + kap) is formed from operands kept to 2^-22 and added
// into an accumulator that loses up to 2^-23 of its size at each of at most 128 steps, so the error is below 2^-15 times
// the sum of the terms' sizes, and sum_d w (|mu' x'| + (x'^2 + |kap'|) / 2) <= sum_d w (mu'^2 + |kap'|) / 2 + max_d w |x'|^2.)
__global__ void __launch_bounds__(256) wide_flag_kernel(int D, int Dpad, int K, const float* __restrict__ pi,
                                                        const float* __restrict__ mu, const float* __restrict__ var,
                                                        const float* __restrict__ sd, const float* __restrict__ kap,
                                                        const float* __restrict__ gd, float* __restrict__ illb,
                                                        float* __restrict__ scra, float* __restrict__ scrw,
                                                        float* __restrict__ scra_hi, float* __restrict__ scrw_hi,
                                                        float cond_limit, float min_weight, int* __restrict__ flags) {
    __shared__ double red[4][256];
    const int k = blockIdx.x, t = threadIdx.x;
    double cond2 = 0.0, ramp = 0.0, asum = 0.0, wmax = 0.0;
    if (k < K)
        for (int d = t; d < D; d += 256) {
            const double v = (double)var[(size_t)k * D + d], m = (double)mu[(size_t)k * D + d] - (double)gd[d], s = (double)sd[d];
            const double w = 1.4426950408889634074 / v;
            const double kp = (double)kap[d] / (s * s);
            const double tau = 0.5 * w * 3.0 * (m * m + 9.0 * v);       // size of the dimension's terms at 3 sigma
            cond2 += tau * tau;
            // what a point of this component adds to the accumulator in this dimension, on average (log2 units)
            ramp += 0.5 * w * (m * m - v - kp);
            asum += 0.5 * w * (m * m + fabs(kp));
            wmax = fmax(wmax, w);
        }
    red[0][t] = cond2; red[1][t] = ramp; red[2][t] = asum; red[3][t] = wmax;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (t < o) {
            red[0][t] += red[0][t + o];
            red[1][t] += red[1][t + o];
            red[2][t] += red[2][t + o];
            red[3][t] = fmax(red[3][t], red[3][t + o]);
        }
        __syncthreads();
    }
    if (t == 0) {
        const double est_round = 4.0 * 2.384185791015625e-07 * sqrt(red[0][0]);
        const double est_trunc = (double)Dpad / 16.0 * 1.1920928955078125e-07 * (fabs(red[1][0]) + 2.04 * sqrt((double)D));
        const double est = fmax(est_round, est_trunc);
        float margin = 0.f;
        if (k < K && pi[k] > 0.f && (!(est <= (double)cond_limit) || pi[k] < min_weight)) {
            margin = !(est_round <= (double)cond_limit) ? (float)fmin(fmax(8.0 * est_round, 1e-10), 1e30) : 1e-30f;
            if (!(margin > 0.f)) margin = 1e30f;
            atomicOr(flags, 1);
            atomicAdd(flags + 4, 1);
        }
        illb[k] = margin;
        const double eps = 3.0517578125e-05;                 // 2^-15
        const double a = 8.0 * est + eps * red[2][0] + 0.0625, w = eps * red[3][0];
        scra[k] = (float)fmin(isfinite(a) ? a : 1e30, 1e30);
        scrw[k] = (float)fmin(isfinite(w) ? w : 1e30, 1e30);
        // with the leading product alone (the low halves of both operands dropped: 2^-11 of every term, twice)
        const double eps_hi = 9.765625e-04;                  // 2^-10
        const double ah = a + eps_hi * red[2][0], wh = w + eps_hi * red[3][0];
        scra_hi[k] = (float)fmin(isfinite(ah) ? ah : 1e30, 1e30);
        scrw_hi[k] = (float)fmin(isfinite(wh) ? wh : 1e30, 1e30);
    }
}

// Where each component sits in the tensor passes, and the list of the flagged ones.  One block of 1024 threads.
// Positions [0, Kg): the components the tensor passes evaluate, in ascending order (flags[6] = Kg); [Kg, Kgp = the next
// multiple of 256): empty; from Kgp on: the flagged components in the order of the list, which sweep 1 only screens (its
// groups of 256 columns then hold either kind, never both, and every point's running maximum is final when the
// screening starts).  comp_of[pos] = component or -1; slot_of[pos] = slot in the list or -1; scr_mask[pos / 32].
// The list (at most WIDE_MAX_ILL slots; flags[2] = its length): first, in ascending order, the components flagged by
// their error estimate (mostly collapsed onto a point), then, from the next multiple of 64 on (flags[5]; the gap is
// filled with -1 = empty slots), those flagged for their drift or weight alone (broad): the FP32 kernels that evaluate the
// list densely when the pairs are too many leave a tile of 64 collapsed components after its first chunk of dimensions.
__global__ void __launch_bounds__(1024) wide_ill_list_kernel(int K, int rows, const float* __restrict__ illb, int* __restrict__ list,
                                                             int* __restrict__ comp_of, int* __restrict__ slot_of,
                                                             int* __restrict__ scr_mask, int* __restrict__ flags) {
    __shared__ int wcount[32];
    __shared__ int kgp_s;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int j = threadIdx.x; j < rows; j += 1024) { comp_of[j] = -1; slot_of[j] = -1; }
    __syncthreads();
    int done = 0;        // list slots used so far (kinds 0, 1) / positions used so far (kind 2 = the others)
    int nflag = 0;       // flagged components placed so far
    for (int kind = 2; kind >= 0; kind = (kind == 2 ? 0 : (kind == 0 ? 1 : -1))) {
        if (kind == 0) done = 0;
        for (int base = 0; base < K; base += 1024) {
            const int k = base + threadIdx.x;
            const float e = k < K ? illb[k] : -1.f;
            const bool is = kind == 2 ? (e == 0.f) : (kind == 0 ? (e > 1e-20f) : (e > 0.f && e <= 1e-20f));
            const unsigned b = __ballot_sync(0xffffffffu, is);
            __syncthreads();
            if (lane == 0) wcount[w] = __popc(b);
            __syncthreads();
            int before = 0, total = 0;
            for (int j = 0; j < 32; ++j) {
                if (j < w) before += wcount[j];
                total += wcount[j];
            }
            const int rank = before + __popc(b & ((1u << lane) - 1u));
            if (is) {
                if (kind == 2) {
                    comp_of[done + rank] = k;
                } else if (done + rank < WIDE_MAX_ILL) {
                    list[done + rank] = k;
                    const int pos = kgp_s + nflag + rank;
                    if (pos < rows) { comp_of[pos] = k; slot_of[pos] = done + rank; }
                }
            }
            done += total;
            if (kind != 2) nflag += total;
        }
        if (kind == 2) {
            if (threadIdx.x == 0) { flags[6] = done; kgp_s = (done + 255) & ~255; }
            __syncthreads();
        }
        if (kind == 0) {
            const int padded = (done + 63) & ~63;
            for (int j = done + threadIdx.x; j < padded && j < WIDE_MAX_ILL; j += 1024) list[j] = -1;
            done = padded < WIDE_MAX_ILL ? padded : done;
            if (threadIdx.x == 0) flags[5] = done;            // where the second kind starts
            __syncthreads();
        }
    }
    if (threadIdx.x == 0) flags[2] = done < WIDE_MAX_ILL ? done : WIDE_MAX_ILL;
    __syncthreads();
    for (int c = threadIdx.x; c < rows / 32; c += 1024) {
        int any = 0;
        for (int j = 0; j < 32; ++j) any |= (slot_of[32 * c + j] >= 0) ? 1 : 0;
        scr_mask[c] = any;
    }
}

// One block per position of the tensor passes: coefficient planes, t, c (float64) of the component that sits there
// (zero planes and c = -inf for an empty position).
__global__ void __launch_bounds__(256) wide_prepare_kernel(int D, int Dpad, int rows, const int* __restrict__ comp_of, const float* __restrict__ pi,
                                                           const float* __restrict__ mu, const float* __restrict__ var,
                                                           const float* __restrict__ sd, const float* __restrict__ kap,
                                                           const float* __restrict__ gd, __half* __restrict__ p_hi,
                                                           __half* __restrict__ p_lo, float* __restrict__ tk,
                                                           double* __restrict__ ckd) {
    extern __shared__ double ab_s[];                     // [2][Dpad]: a, b of this component
    __shared__ double red[3][256];
    const int pos = blockIdx.x, t = threadIdx.x;
    const int k = comp_of[pos];
    double mx = 0.0, csum = 0.0;
    for (int d = t; d < Dpad; d += 256) {
        double a = 0.0, b = 0.0;
        if (k >= 0 && d < D) {
            const double v = (double)var[(size_t)k * D + d], m = (double)mu[(size_t)k * D + d] - (double)gd[d], s = (double)sd[d];
            const double w = 1.4426950408889634074 / v;
            a = w * m / s;
            b = -0.5 * w / (s * s);
            csum += m * m / v + log(6.283185307179586476925286766559 * v);
            mx = fmax(mx, fmax(fabs(a), fabs(b)));
        }
        ab_s[d] = a;
        ab_s[Dpad + d] = b;
    }
    red[0][t] = mx; red[1][t] = csum;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (t < o) {
            red[0][t] = fmax(red[0][t], red[0][t + o]);
            red[1][t] += red[1][t + o];
        }
        __syncthreads();
    }
    mx = red[0][0];
    double tt = 1.0;
    if (mx > 0.0 && isfinite(mx)) tt = exp2(floor(log2(mx)) - 9.0);      // max |P / t| in [512, 1024)
    double ksum = 0.0;
    // planes stored atom by atom: [atom of 64 columns][position][64 halves]
    auto at = [&](int cx) { return ((size_t)(cx >> 6) * rows + pos) * 64 + (cx & 63); };
    for (int d = t; d < Dpad; d += 256) {
        const double as = ab_s[d] / tt, bs = ab_s[Dpad + d] / tt;
        const __half ah = __double2half(as), bh = __double2half(bs);
        const __half al = __double2half(as - (double)__half2float(ah)), bl = __double2half(bs - (double)__half2float(bh));
        const int cx = 16 * (d >> 3) + (d & 7);          // k-step interleaved column order, slices of 128 dimensions in sequence
        p_hi[at(cx)] = ah; p_hi[at(cx + 8)] = bh; p_lo[at(cx)] = al; p_lo[at(cx + 8)] = bl;
        // what the contraction adds through the shifted squares is taken out of c_k; so is what the rounding of the
        // coefficients (22 bits of the row's largest entry: the same error for every point) makes it miss at the
        // component's own mean u = s (mu - g), which leaves an error proportional to a point's distance from that mean
        const double bq = (double)__half2float(bh) + (double)__half2float(bl);
        const double ra = as - ((double)__half2float(ah) + (double)__half2float(al)), rb = bs - bq;
        double um = 0.0;
        if (k >= 0 && d < D) um = ((double)mu[(size_t)k * D + d] - (double)gd[d]) * (double)sd[d];
        ksum += tt * (bq * (double)kap[d] - (ra * um + rb * (um * um + (double)kap[d])));
    }
    __syncthreads();
    red[2][t] = ksum;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (t < o) red[2][t] += red[2][t + o];
        __syncthreads();
    }
    if (t == 0) {
        double c = -CUDART_INF;
        if (k >= 0) {
            const float pk = pi[k];
            if (pk > 0.f) c = 1.4426950408889634074 * (log((double)pk) - 0.5 * red[1][0]) - red[2][0];
        }
        tk[pos] = (float)tt;
        ckd[pos] = c;
    }
}

// c_ref = the largest finite c among the positions the tensor passes evaluate; tkck[pos] = (t, c - c_ref) in fp32 (-inf
// where the position takes no part); scr[pos] = (c - c_ref + scra, scrw) for a listed component, (scra, scrw) for an
// evaluated one, (-inf, 0) elsewhere.
__global__ void __launch_bounds__(1024) wide_cref_kernel(int rows, const int* __restrict__ flags, const float* __restrict__ tk,
                                                         const double* __restrict__ ckd, const int* __restrict__ comp_of,
                                                         const int* __restrict__ slot_of, const float* __restrict__ scra,
                                                         const float* __restrict__ scrw, const float* __restrict__ scra_hi,
                                                         const float* __restrict__ scrw_hi, int hi_mode, double* __restrict__ cref,
                                                         float2* __restrict__ tkck, float2* __restrict__ scr,
                                                         float* __restrict__ scr_e) {
    __shared__ double red[1024];
    const int Kg = flags[6];
    double m = -CUDART_INF;
    for (int k = threadIdx.x; k < Kg; k += 1024)
        if (isfinite(ckd[k])) m = fmax(m, ckd[k]);
    red[threadIdx.x] = m;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] = fmax(red[threadIdx.x], red[threadIdx.x + o]);
        __syncthreads();
    }
    const double r = isfinite(red[0]) ? red[0] : 0.0;
    if (threadIdx.x == 0) *cref = r;
    const int hi_start = ((((Kg + 255) & ~255) + flags[5]) + 255) & ~255;
    for (int k = threadIdx.x; k < rows; k += 1024) {
        const bool in = k < Kg && isfinite(ckd[k]);
        tkck[k] = make_float2(tk[k], in ? (float)(ckd[k] - r) : -CUDART_INF_F);
        const int c = comp_of[k];
        const bool listed = slot_of[k] >= 0 && c >= 0 && isfinite(ckd[k]);
        // (hi_mode: the groups of 256 positions behind the first kind of listed components are screened by the leading
        // product alone, with the allowances that go with it)
        const bool hi = (hi_mode == 1 && k >= hi_start) || (hi_mode == 3 && k >= ((Kg + 255) & ~255));      // (3: every listed component)
        const float ea = listed ? (hi ? scra_hi[c] : scra[c]) : 0.f, ew = listed ? (hi ? scrw_hi[c] : scrw[c]) : 0.f;
        scr[k] = listed ? make_float2((float)fmin(ckd[k] - r + (double)ea, 3e38), ew)
                        : (in && c >= 0) ? (hi_mode == 2 ? make_float2(scra_hi[c], scrw_hi[c]) : make_float2(scra[c], scrw[c]))
                                         : make_float2(-CUDART_INF_F, 0.f);
        scr_e[k] = ea;
    }
}

// stats += sum over the R partial blocks of a component slice (fixed order, float64), undoing the responsibility scale,
// the per-dimension scale and centre, and the column order; the partial blocks are left as they are (the caller clears them).
__global__ void wide_reduce_kernel(int D, int Kg, int CL, int R, int pcols, const float* __restrict__ partial,
                                   const int* __restrict__ comp_of, const float* __restrict__ sd, const float* __restrict__ kap,
                                   const float* __restrict__ gd, double* __restrict__ Nk, double* __restrict__ S1,
                                   double* __restrict__ S2) {
    // Kg: the positions the sweep evaluated; position p holds component comp_of[p]
    const size_t KD = (size_t)Kg * D, per = (size_t)Kg + 2 * KD;
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= per) return;
    const double unscale = 1.0 / (double)TC_RSCALE;
    auto column = [&](int col, int pos) {
        double s = 0.0;
        const int sl = pos >> 7, kl = pos & 127;
        for (int q = 0; q < R; ++q) s += (double)partial[((size_t)(q * CL + sl) * pcols + col) * 128 + kl];
        return s;
    };
    if (e < (size_t)Kg) {
        const int pos = (int)e, k = comp_of[pos];
        if (k >= 0) Nk[k] += (column(pcols - 2, pos) + column(pcols - 1, pos)) * unscale;
        return;
    }
    const bool second = e >= Kg + KD;
    const size_t j = second ? (e - Kg - KD) : (e - Kg);
    const int pos = (int)(j / D), d = (int)(j % D);
    const int k = comp_of[pos];
    if (k < 0) return;
    const size_t o = (size_t)k * D + d;
    const int col = 16 * (d >> 3) + (d & 7);
    const double s_d = (double)sd[d], g = (double)gd[d];
    const double nk_raw = column(pcols - 2, pos) + column(pcols - 1, pos);
    const double nk = nk_raw * unscale;
    const double s1c = column(col, pos) * unscale / s_d;
    if (!second) {
        S1[o] += s1c + g * nk;
    } else {
        const double s2c = (column(col + 8, pos) - (double)kap[d] * nk_raw) * unscale / (s_d * s_d);
        S2[o] += s2c + 2.0 * g * s1c + g * g * nk;
    }
}

// Exact log2 Z.  The approximate logits carry an error of up to about 1e-3 (the tensor core truncates its fp32 accumulator
// at every step; the loss grows with the accumulator's magnitude), most of it common to the components that matter for
// a point, and log2 Z_i from sweep 1 carries the same error: in r = 2^(log2 z - log2 Z) of sweep 2 it cancels, which is why
// sweep 2 must use the log2 Z of sweep 1 as it is.  The components evaluated EXACTLY (the sub-mixture of the FP32
// kernels) need an exact normaliser instead, and so does the log-likelihood: the two leading terms of every point are
// recomputed exactly (fp32 direct differences, chunk sums added in float64: the arithmetic of the FP32 kernels) and a
// second array gets Z' = Z + sum_c (2^exact_c - 2^approx_c).  One warp per point.
__global__ void __launch_bounds__(256) wide_refine_kernel(const float* __restrict__ X, int64_t n, int D, int K,
                                                          const float* __restrict__ mu, const float* __restrict__ w2,
                                                          const double* __restrict__ c2d, const double* __restrict__ cref,
                                                          const float4* __restrict__ top, const int* __restrict__ comp_of,
                                                          const double* __restrict__ logz, double* __restrict__ logz_x) {
    const int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (i >= n) return;
    const float4 t = top[i];
    const double lz = logz[i], cr = *cref;
    const float av[2] = {t.x, t.y};
    const int ak[2] = {__float_as_int(t.z), __float_as_int(t.w)};
    const float* xr = X + i * D;
    double corr = 0.0;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const int k = (ak[c] >= 0) ? __ldg(comp_of + ak[c]) : -1;     // the sweep reports positions
        if (k < 0 || k >= K) continue;                       // warp-uniform
        const float* mr = mu + (size_t)k * D;
        const float* wr = w2 + (size_t)k * D;
        double q = 0.0;
        for (int d0 = 0; d0 < D; d0 += 128) {                // a lane sums 4 dimensions of each 128 in fp32
            float part = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int d = d0 + lane + 32 * j;
                if (d < D) {
                    const float diff = __ldg(xr + d) - __ldg(mr + d);
                    part = fmaf(diff * diff, __ldg(wr + d), part);
                }
            }
            q += (double)part;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
        const double exact = __ldg(c2d + k) - q, approx = cr + (double)av[c];
        corr += exp2(exact - lz) - exp2(approx - lz);
    }
    if (lane == 0) {
        const double f = 1.0 + corr;
        logz_x[i] = lz + log2(f > 1e-6 ? f : 1e-6);
    }
}

// ---- ill-conditioned components: evaluated exactly, as a packed sub-mixture -------------------------------------------
// The listed components' rows of mu, w2 and their constants, packed: the sub-mixture the FP32 kernels evaluate.
__global__ void wide_ill_gather_kernel(int D, int n_ill, const int* __restrict__ list, const float* __restrict__ mu,
                                       const float* __restrict__ w2, const double* __restrict__ c2d, float* __restrict__ mu_c,
                                       float* __restrict__ w2_c, double* __restrict__ c2d_c) {
    const int j = blockIdx.x;
    if (j >= n_ill) return;
    const int k = list[j];
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        mu_c[(size_t)j * D + d] = k >= 0 ? mu[(size_t)k * D + d] : 0.f;
        w2_c[(size_t)j * D + d] = k >= 0 ? w2[(size_t)k * D + d] : 0.f;
    }
    if (threadIdx.x == 0) c2d_c[j] = k >= 0 ? c2d[k] : -CUDART_INF;       // an empty slot: log2 z = -inf for every point
}

// Both log2 Z arrays (the one consistent with the tensor passes' logits, the exact one) take in the sub-mixture's
// log-sum-exp b: log2(2^a + 2^b) (b may be NULL); per-block sums of the exact log Z (natural log) for the
// log-likelihood: fixed grid, fixed order inside a block -> deterministic.
__global__ void __launch_bounds__(256) wide_merge_ll_kernel(int64_t n, double* __restrict__ logz, double* __restrict__ logz_x,
                                                            const double* __restrict__ logz_ill, double* __restrict__ llpart) {
    __shared__ double red[256];
    const int64_t per = (n + gridDim.x - 1) / gridDim.x;
    const int64_t lo = (int64_t)blockIdx.x * per, hi = (lo + per < n) ? (lo + per) : n;
    double s = 0.0;
    for (int64_t i = lo + threadIdx.x; i < hi; i += 256) {
        double a = logz[i], x = logz_x[i];
        if (logz_ill) {
            const double b = logz_ill[i];
            double m = fmax(a, b);
            if (m > -CUDART_INF) a = m + log2(exp2(a - m) + exp2(b - m));
            m = fmax(x, b);
            if (m > -CUDART_INF) x = m + log2(exp2(x - m) + exp2(b - m));
            logz[i] = a;
            logz_x[i] = x;
        }
        s += x;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) llpart[blockIdx.x] += red[0] * 0.69314718055994530942;
}

// ---- the listed components evaluated pair by pair ---------------------------------------------------------------------
// Sweep 1 marks the (point, listed component) pairs that can matter; at the paper's IVF sizes those are a few thousand
// of the 10^8 pairs of a piece (a component collapsed onto a point matters for that point only), so evaluating them one
// by one costs nothing next to the dense evaluation of the whole sub-mixture by the FP32 kernels, which stays as the
// route for parameter sets in which the marked pairs are many (ctl[1]).

// One warp per point: the marks sweep 1 recorded for it, against the point's final threshold.
__global__ void __launch_bounds__(256) wide_cand_filter_kernel(int64_t n, int words, unsigned* __restrict__ cand,
                                                               const unsigned* __restrict__ rec, const int* __restrict__ rec_cnt,
                                                               const float* __restrict__ rec_thr, int* __restrict__ ctl) {
    __shared__ int drop_s[8];
    const int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const bool in = i < n;
    const int c0 = in ? min(rec_cnt[2 * i], WIDE_REC / 2) : 0, c1 = in ? min(rec_cnt[2 * i + 1], WIDE_REC / 2) : 0;     // the two halves of the record
    const float thr = in ? rec_thr[i] - 40.f : 0.f;
    int dropped = 0;
    for (int r = lane; in && r < WIDE_REC / 2 + c1; r += 32) {
        if (r >= c0 && r < WIDE_REC / 2) continue;
        const unsigned v = rec[i * WIDE_REC + r];
        const int sl = (int)(v & 0x1FFFu);
        if (__uint_as_float(v & ~0x1FFFu) < thr) {           // (a NaN stays)
            atomicAnd(cand + i * words + (sl >> 5), ~(1u << (sl & 31)));
            ++dropped;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dropped += __shfl_xor_sync(0xffffffffu, dropped, o);
    if (lane == 0) drop_s[threadIdx.x >> 5] = dropped;
    __syncthreads();
    if (threadIdx.x == 0) {                                  // (one subtraction per block: they all go to one address)
        int t = 0;
        for (int w = 0; w < 8; ++w) t += drop_s[w];
        if (t > 0) atomicSub(ctl, t);
    }
}

__global__ void wide_cand_gate_kernel(int* __restrict__ ctl, long long max_pairs) {
    const int dense = ((long long)ctl[0] > max_pairs) ? 1 : 0;
    ctl[1] = dense;
    ctl[2] = 1 - dense;
}

// Per-step totals for diagnostics: flags[1] += pairs marked, flags[3] += pairs kept, flags[7] += 1 for a piece that went
// through the dense kernels (saturating).
__global__ void __launch_bounds__(256) wide_cand_count_kernel(const int* __restrict__ ctl, int* __restrict__ flags,
                                                              const int* __restrict__ slot_cnt, int n_slots) {
    __shared__ long long red[256];
    long long k = 0;                                         // pairs kept: the slots' counts
    for (int j = threadIdx.x; j < n_slots; j += 256) k += slot_cnt[j];
    red[threadIdx.x] = k;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x != 0) return;
    auto add = [](int a, long long b) { const long long t = (long long)a + b; return t > 2147483647LL ? 2147483647 : (int)t; };
    flags[1] = add(flags[1], ctl[0]);
    flags[3] = add(flags[3], ctl[1] ? 0 : red[0]);
    flags[7] = add(flags[7], ctl[1] ? 1 : 0);
}

// Exact log2 z of one pair by a whole warp: direct differences in fp32, a lane sums 4 dimensions of each 128 in fp32 and
// adds the chunk sums in float64 (the arithmetic of the FP32 kernels and of wide_refine_kernel), fixed butterfly: every
// lane returns the same bits.  The quadratic form only grows: once c - q (tracked in fp32, with a margin of 1) falls below
// `stop` the rest cannot matter and -inf is returned.
__device__ __forceinline__ double wide_pair_log2z(const float* __restrict__ xr, const float* __restrict__ mr,
                                                  const float* __restrict__ wr, double c, int D, int lane, double stop) {
    double q = 0.0;
    float run = 0.f;
    const float room = (stop > -CUDART_INF) ? (float)fmin(fmax(c - stop + 1.0, -3e38), 3e38) : CUDART_INF_F;
    for (int d0 = 0; d0 < D; d0 += 128) {
        float part = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int d = d0 + lane + 32 * j;
            if (d < D) {
                const float diff = __ldg(xr + d) - __ldg(mr + d);
                part = fmaf(diff * diff, __ldg(wr + d), part);
            }
        }
        q += (double)part;
        float tot = part;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        run += tot;
        if (run > room) return -CUDART_INF;                  // warp-uniform: tot is the same in every lane
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    return c - q;
}

// One warp per point: its marked pairs in ascending slot order, evaluated exactly.  First round: every pair's exact log2 z,
// each abandoned as soon as it cannot come within 2^-40 of the largest value so far (the point's log2 Z over the evaluated
// components to begin with: logz); the first 128 values are kept in shared memory.  Second round: the pairs within 2^-40
// of the final maximum are kept: log-sum-exp into out[i], bit (slot, i) of the transposed map.
constexpr int CAND_WORDS_PER_LANE = (WIDE_CAND_WORDS + 31) / 32;
constexpr int CAND_KEEP = 256;          // exact values of a point's first pairs kept between the two rounds
constexpr int CAND_LIST = 256;          // marked slots of a point listed in shared memory (more: the row is scanned instead)
constexpr int CAND_G = 4;               // marked pairs of a point taken together (their loads overlap)
template <int TOPM>
__global__ void __launch_bounds__(256, 3) wide_cand_lse_kernel(const float* __restrict__ X, int64_t n, int D, int words,
                                                            const unsigned* __restrict__ cand, unsigned* __restrict__ candT,
                                                            const float* __restrict__ mu_c, const float* __restrict__ w2_c,
                                                            const double* __restrict__ c2d_c, const double* __restrict__ logz,
                                                            double* __restrict__ out, int* __restrict__ ctl,
                                                            int* __restrict__ slot_cnt, float* __restrict__ pair_val,
                                                            int* __restrict__ pair_off, double* __restrict__ pair_best,
                                                            const int* __restrict__ list, int32_t* __restrict__ best_out,
                                                            int m_top, int32_t* __restrict__ top_idx, float* __restrict__ top_resp,
                                                            int32_t* __restrict__ unc_rows, int* __restrict__ unc_count,
                                                            const float* __restrict__ swp_top, int swp_ntop,
                                                            const int* __restrict__ comp_of,
                                                            unsigned short* __restrict__ pair_key8, float* __restrict__ pair_val8) {
    // TOPM > 0 (the top-m assignment, m_top <= TOPM): only the first round runs; it keeps the m_top largest exact values
    // (a pair is abandoned once it can reach neither the m_top-th of them nor 2^-40 of the largest) and the sum of all.
    // Ranks that no marked pair fills (every component there lies 2^-40 below the point's best: responsibility 0) are
    // taken from the sweep's candidates, in the order of their upper bounds.
    // best_out != NULL (the hard assignment): only the first round runs, and the component (list[slot]) of the point's
    // largest exact value goes to best_out[i]; of equal values the smaller component.
    if (ctl[1] != 0) return;
    __shared__ double lbuf[8][CAND_KEEP];
    __shared__ unsigned short slist[8][CAND_LIST];
    __shared__ int tot_s[8];
    __shared__ int base_s;
    const int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned bits[CAND_WORDS_PER_LANE];
    int nmarked = 0;
#pragma unroll
    for (int q = 0; q < CAND_WORDS_PER_LANE; ++q) {
        bits[q] = (i < n && lane + 32 * q < words) ? cand[i * words + lane + 32 * q] : 0u;
        nmarked += __popc(bits[q]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) nmarked += __shfl_xor_sync(0xffffffffu, nmarked, o);
    // Room for the exact values of the block's pairs (the statistics kernel reads them back instead of evaluating its pairs
    // again): one request per block - they all go to one counter.  Where the room starts depends on timing, what is stored
    // there does not.  No room left: ctl[5] tells the statistics kernel to evaluate every pair of the piece itself.
    const bool assign_mode = TOPM > 0 || best_out != nullptr;      // (block-uniform: no values are kept for a statistics kernel)
    if (!assign_mode) {
        if (lane == 0) tot_s[w] = nmarked;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = 0;
            for (int j = 0; j < 8; ++j) t += tot_s[j];
            int b = t > 0 ? atomicAdd(ctl + 4, t) : 0;
            if (b < 0 || b > WIDE_PAIR_VALS - t) { b = -1; ctl[5] = 1; }
            base_s = b;
        }
        __syncthreads();
    }
    if (i >= n) return;
    if (nmarked == 0) {
        if (lane == 0) {
            if (TOPM > 0) unc_rows[atomicAdd(unc_count, 1)] = (int32_t)i;
            else if (best_out) best_out[i] = 0;
            else out[i] = -CUDART_INF;
        }
        return;
    }
    int off = assign_mode ? -1 : base_s;
    for (int j = 0; j < w && !assign_mode; ++j) off += (off >= 0) ? tot_s[j] : 0;
    // The assignment of a point with ONE marked pair needs no evaluation: that component is the point's best, and every other
    // lies 2^-40 below it (responsibility 1 and 0).
    const bool single = assign_mode && nmarked == 1;
    if (single && best_out) {
        int slot = -1;
#pragma unroll
        for (int q = 0; q < CAND_WORDS_PER_LANE; ++q)
            if (bits[q]) slot = (lane + 32 * q) * 32 + __ffs(bits[q]) - 1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) slot = max(slot, __shfl_xor_sync(0xffffffffu, slot, o));
        if (lane == 0) best_out[i] = __ldg(list + slot);
        return;
    }
    const float* xr = X + i * D;
    auto word_at = [&](int wi) {
        unsigned v = bits[0];
#pragma unroll
        for (int q = 1; q < CAND_WORDS_PER_LANE; ++q)
            if ((wi >> 5) == q) v = bits[q];
        return __shfl_sync(0xffffffffu, v, wi & 31);
    };
    // exact log2 z of one pair by the whole warp, abandoned once it cannot reach `stop`
    // (With rows of whole 16-byte groups the point stays in registers, a lane holding dimensions 4 l .. 4 l + 3 of every
    // 128, and a component's row comes in 16-byte loads: a quarter of the instructions of the general routine.  A lane
    // sums its 4 dimensions of each 128 in fp32, the chunk sums are added in float64, fixed butterfly at the end; the
    // running total is looked at after the first 128 dimensions and then after every 256.)
    const bool vec = (D % 4 == 0) && (((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(mu_c) | reinterpret_cast<uintptr_t>(w2_c)) & 15) == 0);
    float4 xq[8];
    if (vec && !single) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            xq[j] = (128 * j + 4 * lane < D) ? __ldg(reinterpret_cast<const float4*>(xr + 128 * j) + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    auto full = [&](int slot, double stop) -> double {
        const double c = __ldg(c2d_c + slot);
        if (!vec) return wide_pair_log2z(xr, mu_c + (size_t)slot * D, w2_c + (size_t)slot * D, c, D, lane, stop);
        const float4* mr = reinterpret_cast<const float4*>(mu_c + (size_t)slot * D) + lane;
        const float4* wr = reinterpret_cast<const float4*>(w2_c + (size_t)slot * D) + lane;
        const float room = (stop > -CUDART_INF) ? (float)fmin(fmax(c - stop + 1.0, -3e38), 3e38) : CUDART_INF_F;
        double q = 0.0;
        float run = 0.f;
        // (four chunks of 128 dimensions at a time: their loads are in flight together, and the running total is looked at
        // after each four - with a final threshold nearly every pair that gets here is kept, and a look after every chunk
        // or two made the evaluation a chain of five trips to L2)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (512 * h < D) {                               // warp-uniform
                float4 m4[4], w4[4];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 4 * h + jj;
                    const bool in = 128 * j + 4 * lane < D;
                    m4[jj] = in ? __ldg(mr + 32 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
                    w4[jj] = in ? __ldg(wr + 32 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 4 * h + jj;
                    float part = 0.f;
                    float dd = xq[j].x - m4[jj].x;  part = fmaf(dd * dd, w4[jj].x, part);
                    dd = xq[j].y - m4[jj].y;        part = fmaf(dd * dd, w4[jj].y, part);
                    dd = xq[j].z - m4[jj].z;        part = fmaf(dd * dd, w4[jj].z, part);
                    dd = xq[j].w - m4[jj].w;        part = fmaf(dd * dd, w4[jj].w, part);
                    q += (double)part;
                    run += part;
                }
                float tot = run;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
                if (tot > room) return -CUDART_INF;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
        return c - q;
    };
    // Most marked pairs are ruled out by their first 128 dimensions.  Those are taken four pairs at a time, one per group
    // of eight lanes: a lane holds 16 consecutive dimensions of the point (registers) and loads the same 16 of its pair's
    // component (four 16-byte loads per array), three shuffles sum the group.  (D > 128 on this path.)
    const int gid = lane >> 3, sub = lane & 7;
    // (the point's first 128 dimensions, regrouped by shuffles from the registers that hold the whole point - lane 4 sub + t
    // holds dimensions 16 sub + 4 t .. + 3 - or, for rows that are not whole 16-byte groups, read again: a copy of its own
    // cost 16 registers and a block per SM)
    auto first_chunks = [&](const int (&sl)[CAND_G], int cnt, double stop, bool (&alive)[CAND_G]) {
        const int mine = (gid == 0) ? sl[0] : (gid == 1) ? sl[1] : (gid == 2) ? sl[2] : sl[3];
        float part = 0.f;
        float4 fm[4], fw[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) { fm[t] = make_float4(0.f, 0.f, 0.f, 0.f); fw[t] = fm[t]; }
        if (gid < cnt) {
            const float* mr = mu_c + (size_t)mine * D + 16 * sub;
            const float* wr = w2_c + (size_t)mine * D + 16 * sub;
            if (vec) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float4 m4 = __ldg(reinterpret_cast<const float4*>(mr) + t);
                    const float4 w4 = __ldg(reinterpret_cast<const float4*>(wr) + t);
                    fm[t] = m4; fw[t] = w4;
                }
            } else {
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    const float dd = __ldg(xr + 16 * sub + t) - __ldg(mr + t);
                    part = fmaf(dd * dd, __ldg(wr + t), part);
                }
            }
        }
        if (vec) {                                           // (all lanes take part in the shuffles)
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int src = 4 * sub + t;
                const float x0 = __shfl_sync(0xffffffffu, xq[0].x, src), x1 = __shfl_sync(0xffffffffu, xq[0].y, src);
                const float x2 = __shfl_sync(0xffffffffu, xq[0].z, src), x3 = __shfl_sync(0xffffffffu, xq[0].w, src);
                if (gid < cnt) {
                    float dd = x0 - fm[t].x;     part = fmaf(dd * dd, fw[t].x, part);
                    dd = x1 - fm[t].y;           part = fmaf(dd * dd, fw[t].y, part);
                    dd = x2 - fm[t].z;           part = fmaf(dd * dd, fw[t].z, part);
                    dd = x3 - fm[t].w;           part = fmaf(dd * dd, fw[t].w, part);
                }
            }
        }
        part += __shfl_xor_sync(0xffffffffu, part, 1);
        part += __shfl_xor_sync(0xffffffffu, part, 2);
        part += __shfl_xor_sync(0xffffffffu, part, 4);
        bool dead = true;
        if (gid < cnt) {
            const double c = __ldg(c2d_c + mine);
            // (the sum of 128 dimensions in another order than the exact evaluation's: a margin of 2 instead of 1)
            const float room = (stop > -CUDART_INF) ? (float)fmin(fmax(c - stop + 2.0, -3e38), 3e38) : CUDART_INF_F;
            dead = part > room;
        }
        const unsigned am = __ballot_sync(0xffffffffu, !dead && sub == 0);
#pragma unroll
        for (int g = 0; g < CAND_G; ++g) alive[g] = ((am >> (8 * g)) & 1u) != 0u;
    };
    // The point's marked slots, in ascending order, as a list in shared memory (scanning the 130 words of the row twice
    // cost more than evaluating the pairs): word lane + 32 q belongs to lane `lane`, so the order is (q, lane, bit).
    int total = 0;
    {
        int base = 0;
#pragma unroll
        for (int q = 0; q < CAND_WORDS_PER_LANE; ++q) {
            const int c = __popc(bits[q]);
            int incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            int at = base + incl - c;
            unsigned word = bits[q];
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                if (at < CAND_LIST) slist[w][at] = (unsigned short)((lane + 32 * q) * 32 + b);
                ++at;
            }
            base += __shfl_sync(0xffffffffu, incl, 31);
        }
        total = base;
    }
    __syncwarp();
    const bool listed = total <= CAND_LIST;                   // (else: the row is scanned word by word, as a fallback)
    double best = logz[i];
    int best_comp = 0x7fffffff;                               // (tracked for best_out only)
    constexpr int TM = TOPM > 0 ? TOPM : 1;
    double topv[TM];                                         // (TOPM > 0) the largest exact values so far, descending ...
    int topc[TM];                                            // ... and their components; every lane holds the same
    double zm = -CUDART_INF, zs = 0.0;                       // running log-sum-exp of all exact values
#pragma unroll
    for (int r = 0; r < TM; ++r) { topv[r] = -CUDART_INF; topc[r] = -1; }
    int idx = 0;
    {
        int sl[CAND_G], cnt = 0;
        auto flush = [&]() {
            bool alive[CAND_G];
            double stop = best - 40.0;
            if (TOPM > 0) {
#pragma unroll
                for (int r = 0; r < TM; ++r)
                    if (r == m_top - 1) stop = fmin(stop, topv[r]);
            }
            if (single || total == 1) alive[0] = true;       // (a point's only pair is its best: nothing to rule out)
            else first_chunks(sl, cnt, stop, alive);
#pragma unroll
            for (int g = 0; g < CAND_G; ++g) {
                if (g < cnt) {
                    if (TOPM > 0) {
                        stop = best - 40.0;
#pragma unroll
                        for (int r = 0; r < TM; ++r)
                            if (r == m_top - 1) stop = fmin(stop, topv[r]);
                    }
                    const double l = single ? 0.0 : alive[g] ? full(sl[g], TOPM > 0 ? stop : best - 40.0) : -CUDART_INF;
                    if (TOPM > 0 && l > -CUDART_INF) {
                        if (l > zm) { zs = zs * exp2(zm - l) + 1.0; zm = l; }
                        else zs += exp2(l - zm);
                        // insertion by (value descending, component ascending)
                        double v = l;
                        int c = __ldg(list + sl[g]);
#pragma unroll
                        for (int r = 0; r < TM; ++r) {
                            if (r < m_top && (v > topv[r] || (v == topv[r] && topc[r] >= 0 && c < topc[r]) || topc[r] < 0)) {
                                const double tv = topv[r]; const int tc = topc[r];
                                topv[r] = v; topc[r] = c;
                                v = tv; c = tc;
                                if (c < 0) break;
                            }
                        }
                    }
                    if (idx < CAND_KEEP && lane == 0) lbuf[w][idx] = l;
                    ++idx;
                    if (best_out && l >= best && l > -CUDART_INF) {
                        const int comp = __ldg(list + sl[g]);
                        if (l > best || comp < best_comp) best_comp = comp;
                    }
                    if (l > best) best = l;
                }
            }
            cnt = 0;
        };
        if (listed) {
            for (int e = 0; e < total; e += CAND_G) {
                cnt = (total - e < CAND_G) ? (total - e) : CAND_G;
#pragma unroll
                for (int g = 0; g < CAND_G; ++g) sl[g] = (g < cnt) ? (int)slist[w][e + g] : 0;
                flush();
            }
        } else {
            for (int wi = 0; wi < words; ++wi) {
                unsigned word = word_at(wi);
                while (word) {
                    const int b = __ffs(word) - 1;
                    word &= word - 1;
#pragma unroll
                    for (int g = 0; g < CAND_G; ++g)
                        if (g == cnt) sl[g] = wi * 32 + b;
                    if (++cnt == CAND_G) flush();
                }
            }
            if (cnt > 0) flush();
        }
    }
    __syncwarp();
    if (TOPM > 0) {
        if (lane == 0) {
            const double lzf = zm + log2(zs);
            int have = 0;
#pragma unroll
            for (int r = 0; r < TM; ++r)
                if (r < m_top && topc[r] >= 0) ++have;
            for (int q = 0; q < swp_ntop && have > 0 && have < m_top; ++q) {
                const int pos = __float_as_int(swp_top[i * 2 * swp_ntop + swp_ntop + q]);
                const int c = pos >= 0 ? __ldg(comp_of + pos) : -1;
                bool dup = c < 0;
#pragma unroll
                for (int r = 0; r < TM; ++r)
                    if (r < m_top && topc[r] == c) dup = true;
                if (dup) continue;
#pragma unroll
                for (int r = 0; r < TM; ++r)
                    if (r == have) { topc[r] = c; topv[r] = -CUDART_INF; }
                ++have;
            }
            bool full_row = have == m_top;
            if (!full_row) {
                unc_rows[atomicAdd(unc_count, 1)] = (int32_t)i;
            } else {
#pragma unroll
                for (int r = 0; r < TM; ++r) {
                    if (r < m_top) {
                        top_idx[i * m_top + r] = topc[r];
                        if (top_resp) top_resp[i * m_top + r] = (float)exp2(topv[r] - lzf);
                    }
                }
            }
        }
        return;
    }
    if (best_out) {
        if (lane == 0) best_out[i] = best_comp != 0x7fffffff ? best_comp : 0;
        return;
    }
    const double lim = best - 40.0;
    double m = -CUDART_INF, ssum = 0.0;
    int kept = 0;
    // (lane j < 8 holds the j-th marked pair's slot and value for the table of first pairs: what the statistics kernel
    // looks at before it counts the marked bits below a slot)
    unsigned short key8 = 0xFFFFu;
    float val8 = 0.f;
    auto second = [&](int slot, int at) {
        double l;
        if (at < CAND_KEEP) l = lbuf[w][at];
        else l = full(slot, lim);
        if (l >= lim && l > -CUDART_INF) {                   // warp-uniform
            if (l > m) { ssum = ssum * exp2(m - l) + 1.0; m = l; }
            else ssum += exp2(l - m);
            if (lane == 0) {
                atomicOr(candT + (size_t)slot * WIDE_CANDT_WORDS + (i >> 5), 1u << (i & 31));
                atomicAdd(slot_cnt + slot, 1);
                if (off >= 0) pair_val[off + at] = (float)(l - best);       // in [-40, 0]
            }
            if (lane == at) {
                key8 = (unsigned short)slot;
                val8 = (float)(l - best);
            }
            ++kept;
        }
    };
    if (listed) {
        for (int e = 0; e < total; ++e) second((int)slist[w][e], e);
    } else {
        idx = 0;
        for (int wi = 0; wi < words; ++wi) {
            unsigned word = word_at(wi);
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                second(wi * 32 + b, idx);
                ++idx;
            }
        }
    }
    if (lane == 0) {
        out[i] = kept ? m + log2(ssum) : -CUDART_INF;
        pair_off[i] = off;
        pair_best[i] = best;
    }
    if (lane < 8) {
        pair_key8[i * 8 + lane] = key8;
        pair_val8[i * 8 + lane] = val8;
    }
}

// One block per slot: the points marked for it in the transposed map, in ascending order (the order of the additions is
// fixed: same bits in every run).  The block lists its points in shared memory (up to MS_CAP per pass over the map), then
// looks up each pair's exact log2 z as wide_cand_lse_kernel left it (the pair's rank among the point's marked pairs = bits
// below the slot in the point's row of the map) and takes the points eight at a time: every thread loads its 3-4
// dimensions of the eight rows (all loads in flight together) and adds r (x - g), r (x - g)^2, r = 2^(log2 z - log2 Z),
// for its dimensions in float64.  Without the stored values (a piece with more marked pairs than there is room for) the
// eight quadratic forms are evaluated again and reduced over the block (fp32 per thread, float64 from there).  The sums
// are shifted back to the origin and added to the slot's statistics.
constexpr int MS_CAP = 1024, MS_B = 8;
constexpr int MS_SEG = WIDE_HEAVY_SEG;     // a component kept for many points of a piece is split over this many blocks ...
constexpr int MS_SPLIT_MIN = 512;         // ... from this many pairs on
constexpr int MS_HEAVY = WIDE_HEAVY_SLOTS; // at most this many components are split per piece (the others take one block each)

// Which slots are split: heavy_of[slot] = index of the slot's partial sums or -1, heavy_slot[index] = slot or -1; in slot
// order, so that nothing depends on timing.  One block of 1024 threads.
__global__ void __launch_bounds__(1024) wide_heavy_kernel(int n_slots, const int* __restrict__ slot_cnt, int* __restrict__ heavy_of,
                                                          int* __restrict__ heavy_slot, const int* __restrict__ ctl) {
    if (ctl[1] != 0) return;
    __shared__ int wcount[32];
    __shared__ int level[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int h = threadIdx.x; h < MS_HEAVY; h += 1024) heavy_slot[h] = -1;
    if (threadIdx.x < 8) level[threadIdx.x] = 0;
    __syncthreads();
    // Where more than MS_HEAVY slots reach MS_SPLIT_MIN pairs (broad posteriors: the first iterations of a fit), the sets of
    // partial sums go to the heaviest: the limit doubles until at most MS_HEAVY slots reach it (counts are exact integers:
    // nothing depends on timing).
    for (int sl = threadIdx.x; sl < n_slots; sl += 1024) {
        const int c = slot_cnt[sl];
#pragma unroll
        for (int l = 0; l < 8; ++l)
            if (c >= (MS_SPLIT_MIN << l)) atomicAdd(&level[l], 1);
    }
    __syncthreads();
    int split_min = MS_SPLIT_MIN;
#pragma unroll
    for (int l = 0; l < 8; ++l)
        if (level[l] > MS_HEAVY) split_min = MS_SPLIT_MIN << (l + 1);
    int done = 0;
    for (int base = 0; base < n_slots; base += 1024) {
        const int sl = base + threadIdx.x;
        const bool is = sl < n_slots && slot_cnt[sl] >= split_min;
        const unsigned b = __ballot_sync(0xffffffffu, is);
        __syncthreads();
        if (lane == 0) wcount[w] = __popc(b);
        __syncthreads();
        int before = 0, total = 0;
        for (int j = 0; j < 32; ++j) {
            if (j < w) before += wcount[j];
            total += wcount[j];
        }
        const int h = done + before + __popc(b & ((1u << lane) - 1u));
        if (sl < n_slots) heavy_of[sl] = (is && h < MS_HEAVY) ? h : -1;
        if (is && h < MS_HEAVY) heavy_slot[h] = sl;
        done += total;
    }
}

template <bool STORED>      // (two instances, each a no-op unless ctl[5] says it is its turn: the stored-value loop alone needs fewer registers)
__global__ void __launch_bounds__(256, STORED ? 3 : 2) wide_cand_mstep_kernel(const float* __restrict__ X, int64_t n, int D, const int* __restrict__ list,
                                                              const unsigned* __restrict__ candT, const float* __restrict__ mu_c,
                                                              const float* __restrict__ w2_c, const double* __restrict__ c2d_c,
                                                              const float* __restrict__ gd, const double* __restrict__ logz_x,
                                                              double* __restrict__ Nk_c, double* __restrict__ S1_c,
                                                              double* __restrict__ S2_c, const int* __restrict__ ctl,
                                                              const int* __restrict__ heavy_of, double* __restrict__ heavy_part,
                                                              const unsigned* __restrict__ cand, int cand_words,
                                                              const float* __restrict__ pair_val, const int* __restrict__ pair_off,
                                                              const double* __restrict__ pair_best, int n_slots,
                                                              const int* __restrict__ heavy_slot,
                                                              const unsigned short* __restrict__ pair_key8,
                                                              const float* __restrict__ pair_val8) {
    if (ctl[1] != 0) return;
    if ((ctl[5] == 0) != STORED) return;                     // (ctl[5] == 0: the pairs' exact values are there)
    constexpr bool stored = STORED;
    // Blocks [0, n_slots): one per slot (all of an ordinary slot's points, or segment 0 of a split one); behind them
    // MS_SEG - 1 blocks for each of the MS_HEAVY sets of partial sums: segments 1 .. MS_SEG - 1 of the slot that owns the set.
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int slot = blockIdx.x, seg = 0;
    if ((int)blockIdx.x >= n_slots) {
        const int e = (int)blockIdx.x - n_slots;
        slot = heavy_slot[e / (MS_SEG - 1)];
        seg = 1 + e % (MS_SEG - 1);
        if (slot < 0) return;
    }
    const unsigned* bits = candT + (size_t)slot * WIDE_CANDT_WORDS;
    const int words = (int)((n + 31) >> 5);
    // the block's words of the slot's row: all 4096 (16 per thread) or the segment's 256 (one per thread); thread t owns
    // consecutive words, so the rows ascend across the block.  The 16 words of the ordinary case are requested before the
    // slot's kind is known (the row has them whatever its kind), so that the three reads share one round trip.
    unsigned mine[16];
    {
        const uint4* b4 = reinterpret_cast<const uint4*>(bits + 16 * tid);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint4 v = __ldg(b4 + j);
            mine[4 * j] = v.x;
            mine[4 * j + 1] = v.y;
            mine[4 * j + 2] = v.z;
            mine[4 * j + 3] = v.w;
        }
    }
    const int listed = list[slot];
    const int hv = heavy_of[slot];
    if (listed < 0) return;
    if (hv < 0 && seg > 0) return;                           // (cannot happen: only split slots own a set)
    const int wpt = hv < 0 ? 16 : 16 / MS_SEG;
    const int w0 = (hv < 0 ? 0 : seg * (WIDE_CANDT_WORDS / MS_SEG)) + wpt * tid;
    if (hv >= 0) {
#pragma unroll
        for (int j = 0; j < 16; ++j) mine[j] = (j < wpt && w0 + j < words) ? bits[w0 + j] : 0u;
    }
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        if (hv < 0 && w0 + j >= words) mine[j] = 0u;         // (words past the piece's points)
        cnt += __popc(mine[j]);
    }
    __shared__ int rows_s[MS_CAP];
    __shared__ double r_s[MS_CAP];
    __shared__ int wtot[8];
    __shared__ double red_s[8][MS_B];
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    int before = incl - cnt, total = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (j < warp) before += wtot[j];
        total += wtot[j];
    }
    if (total == 0 && hv < 0) return;                        // block-uniform (a segment still writes its zeros)
    const double c = c2d_c[slot];
    float mu_r[4], w2_r[4], g_r[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int d = tid + 256 * q;
        mu_r[q] = (d < D) ? mu_c[(size_t)slot * D + d] : 0.f;
        w2_r[q] = (d < D) ? w2_c[(size_t)slot * D + d] : 0.f;
        g_r[q] = (d < D) ? gd[d] : 0.f;
    }
    double s1[4] = {0.0, 0.0, 0.0, 0.0}, s2[4] = {0.0, 0.0, 0.0, 0.0}, nk = 0.0;
    for (int base = 0; base < total; base += MS_CAP) {
        // this pass's window of the list
        {
            int at = before;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                unsigned word = mine[j];
                while (word) {
                    const int b = __ffs(word) - 1;
                    word &= word - 1;
                    if (at >= base && at < base + MS_CAP) rows_s[at - base] = (w0 + j) * 32 + b;
                    ++at;
                }
            }
        }
        __syncthreads();
        const int here = (total - base < MS_CAP) ? (total - base) : MS_CAP;
        if constexpr (stored) {
            for (int e = tid; e < here; e += 256) {
                const int row = rows_s[e];
                // the pair's value: among the point's first eight marked pairs (one read), else at its rank among all of them
                const uint4 k8 = __ldg(reinterpret_cast<const uint4*>(pair_key8 + (size_t)row * 8));
                const float4 va = __ldg(reinterpret_cast<const float4*>(pair_val8 + (size_t)row * 8));
                const float4 vb = __ldg(reinterpret_cast<const float4*>(pair_val8 + (size_t)row * 8) + 1);
                const double shift = pair_best[row] - logz_x[row];
                const unsigned ks = (unsigned)slot;
                float val = 0.f;
                bool hit = true;
                if ((k8.x & 0xffffu) == ks) val = va.x;
                else if ((k8.x >> 16) == ks) val = va.y;
                else if ((k8.y & 0xffffu) == ks) val = va.z;
                else if ((k8.y >> 16) == ks) val = va.w;
                else if ((k8.z & 0xffffu) == ks) val = vb.x;
                else if ((k8.z >> 16) == ks) val = vb.y;
                else if ((k8.w & 0xffffu) == ks) val = vb.z;
                else if ((k8.w >> 16) == ks) val = vb.w;
                else hit = false;
                if (!hit) {
                    const unsigned* cr = cand + (size_t)row * cand_words;
                    int rank = 0;
                    for (int w = 0; w < (slot >> 5); ++w) rank += __popc(__ldg(cr + w));
                    rank += __popc(__ldg(cr + (slot >> 5)) & ((1u << (slot & 31)) - 1u));
                    val = pair_val[pair_off[row] + rank];
                }
                r_s[e] = exp2((double)val + shift);
            }
            __syncthreads();
            for (int e0 = 0; e0 < here; e0 += MS_B) {
                float xv[MS_B][4];
#pragma unroll
                for (int b = 0; b < MS_B; ++b) {
                    const bool in = e0 + b < here;
                    const float* xr = X + (size_t)(in ? rows_s[e0 + b] : rows_s[e0]) * D;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int d = tid + 256 * q;
                        xv[b][q] = (d < D) ? __ldg(xr + d) : 0.f;
                    }
                }
#pragma unroll
                for (int b = 0; b < MS_B; ++b) {
                    if (e0 + b < here) {                     // block-uniform
                        const double r = r_s[e0 + b];
                        nk += r;
#pragma unroll
                        for (int qq = 0; qq < 4; ++qq) {
                            const double xd = (double)(xv[b][qq] - g_r[qq]);
                            s1[qq] += r * xd;
                            s2[qq] += r * xd * xd;
                        }
                    }
                }
            }
            __syncthreads();                                 // rows_s, r_s are rewritten by the next pass
        } else {
        for (int e0 = 0; e0 < here; e0 += MS_B) {
            float xv[MS_B][4];
            float part[MS_B];
#pragma unroll
            for (int b = 0; b < MS_B; ++b) {
                const bool in = e0 + b < here;
                const float* xr = X + (size_t)(in ? rows_s[e0 + b] : rows_s[e0]) * D;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int d = tid + 256 * q;
                    xv[b][q] = (d < D) ? __ldg(xr + d) : 0.f;
                }
            }
#pragma unroll
            for (int b = 0; b < MS_B; ++b) {
                float p = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float diff = xv[b][q] - mu_r[q];
                    p = fmaf(diff * diff, w2_r[q], p);
                }
                part[b] = p;
            }
            // the block's sums of the eight quadratic forms: fixed butterfly, then the eight warps in order
#pragma unroll
            for (int b = 0; b < MS_B; ++b) {
                double v = (double)part[b];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) red_s[warp][b] = v;
            }
            __syncthreads();
#pragma unroll
            for (int b = 0; b < MS_B; ++b) {
                if (e0 + b < here) {                         // block-uniform
                    double q = 0.0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) q += red_s[j][b];
                    const double r = exp2(c - q - logz_x[rows_s[e0 + b]]);
                    nk += r;
#pragma unroll
                    for (int qq = 0; qq < 4; ++qq) {
                        const double xd = (double)(xv[b][qq] - g_r[qq]);
                        s1[qq] += r * xd;
                        s2[qq] += r * xd * xd;
                    }
                }
            }
            __syncthreads();                                 // red_s is rewritten by the next batch
        }
        __syncthreads();                                     // rows_s is rewritten by the next pass
        }
    }
    // sums about the origin: into the slot's statistics, or into the segment's partial sums of a split slot
    double* oN = hv < 0 ? Nk_c + slot : heavy_part + ((size_t)hv * MS_SEG + seg) * (1 + 2 * (size_t)D);
    double* o1 = hv < 0 ? S1_c + (size_t)slot * D : oN + 1;
    double* o2 = hv < 0 ? S2_c + (size_t)slot * D : oN + 1 + D;
    // An ordinary slot's sums are ADDED to its statistics: one addition per address and launch, by the address's only owner,
    // so the order of the additions is the order of the launches; issued as a reduction, which returns nothing, the addition
    // does not keep the block waiting for the old value.
    if (tid == 0) {
        if (hv < 0) atomicAdd(oN, nk);
        else *oN = nk;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int d = tid + 256 * q;
        if (d < D) {
            const double g = (double)g_r[q];
            const double a1 = s1[q] + g * nk, a2 = s2[q] + 2.0 * g * s1[q] + g * g * nk;
            if (hv < 0) {
                atomicAdd(o1 + d, a1);
                atomicAdd(o2 + d, a2);
            } else {
                o1[d] = a1;
                o2[d] = a2;
            }
        }
    }
}

// The split slots' statistics: their segments' partial sums in order.
__global__ void __launch_bounds__(256) wide_heavy_combine_kernel(int D, const int* __restrict__ heavy_slot, const double* __restrict__ heavy_part,
                                                                 double* __restrict__ Nk_c, double* __restrict__ S1_c,
                                                                 double* __restrict__ S2_c, const int* __restrict__ ctl) {
    if (ctl[1] != 0) return;
    const int slot = heavy_slot[blockIdx.x];
    if (slot < 0) return;
    const double* p = heavy_part + (size_t)blockIdx.x * MS_SEG * (1 + 2 * (size_t)D);
    for (int e = threadIdx.x; e < 1 + 2 * D; e += 256) {
        double s = 0.0;
        for (int g = 0; g < MS_SEG; ++g) s += p[(size_t)g * (1 + 2 * (size_t)D) + e];
        if (e == 0) Nk_c[slot] += s;
        else if (e <= D) S1_c[(size_t)slot * D + (e - 1)] += s;
        else S2_c[(size_t)slot * D + (e - 1 - D)] += s;
    }
}

// ---- top-m assignment on wide data (paper Sections 4.2-4.3) -----------------------------------------------------------
// Sweep 1 reports a point's NTOP evaluated components of largest UPPER BOUND (approximate log2 z plus what it can be wrong
// by for that point; what is not reported lies below the last reported bound), its approximate log2 Z, and marks the listed
// components that can matter for it.  One warp per point then evaluates exactly (a) the marked listed pairs, (b) the
// reported candidates, in the order of their bounds, for as long as a bound reaches 2^-21 of the best exact value so far,
// orders the exact values by (value, component) and writes the first m with r = 2^(log2 z - log2 Z'), Z' = Z with the
// evaluated terms replaced by their exact values; places left over are filled from the reported candidates that were not
// evaluated (their responsibilities are below 5e-7).  A point is left to the FP32 kernels (its row joins unc_rows) when
// the answer is not certain: every reported candidate had to be evaluated and the m-th exact value does not clear the last
// reported bound; fewer than m candidates exist; or (unless only indices are wanted) the terms that stay approximate make
// up more than 1e-3 of Z'.
struct WideAssignArgs {
    const float* X; int64_t n; int D, K;
    const float* mu; const float* w2; const double* c2d;      // the FP32 path's derived parameters, by component
    const int* comp_of; const float* top; const double* logz; const double* cref; const float* n2;
    const float* scra; const float* scrw;                     // error allowances by component
    const unsigned* cand; int cand_words; const int* list; const float* mu_c; const float* w2_c; const double* c2d_c;
    const int* ctl;
    int m; int32_t* idx; float* resp; int32_t* unc_rows; int* unc_count; bool index_only;
};

template <int NTOP>
__global__ void __launch_bounds__(256) wide_assign_refine_kernel(const WideAssignArgs g) {
    if (g.ctl != nullptr && g.ctl[1] != 0) return;            // the piece went to the dense kernels as a whole
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= g.n) return;
    const int D = g.D, m = g.m;
    const float* tp = g.top + row * (2 * NTOP);
    float ub[NTOP];
    int ap[NTOP];
    int nvalid = 0;
#pragma unroll
    for (int j = 0; j < NTOP; ++j) {
        ub[j] = __ldg(tp + j);
        ap[j] = __float_as_int(__ldg(tp + NTOP + j));
        if (ap[j] >= 0) ++nvalid;
    }
    const double lz = g.logz[row], cr = *g.cref;
    const float nrm = __ldg(g.n2 + row);
    const float* xr = g.X + row * D;
    // exact values, the largest kept in order (value descending, component ascending)
    double tv[GMM_MAX_TOPM];
    int tk[GMM_MAX_TOPM];
#pragma unroll
    for (int j = 0; j < GMM_MAX_TOPM; ++j) { tv[j] = -CUDART_INF; tk[j] = -1; }
    int n_exact = 0;
    auto insert = [&](double val, int k) {
        ++n_exact;
        constexpr int L = GMM_MAX_TOPM - 1;
        if (!(tk[L] < 0 || val > tv[L] || (val == tv[L] && k < tk[L]))) return;
        tv[L] = val; tk[L] = k;
#pragma unroll
        for (int j = L; j > 0; --j) {
            if (tk[j - 1] < 0 || tv[j] > tv[j - 1] || (tv[j] == tv[j - 1] && tk[j] < tk[j - 1])) {
                const double fv = tv[j]; tv[j] = tv[j - 1]; tv[j - 1] = fv;
                const int fi = tk[j]; tk[j] = tk[j - 1]; tk[j - 1] = fi;
            }
        }
    };
    // log2 Z' as a running (reference, sum): starts as Z itself; exact_part: the share of the exactly evaluated terms
    double Mr = lz, Ss = (lz > -CUDART_INF) ? 1.0 : 0.0, exact_part = 0.0;
    auto add_term = [&](double t) {
        if (t > Mr) { const double f = exp2(Mr - t); Ss = Ss * f + 1.0; exact_part = exact_part * f + 1.0; Mr = t; }
        else { const double e = exp2(t - Mr); Ss += e; exact_part += e; }
    };
    if (g.cand != nullptr) {
        const double lim = lz - 40.0;
        const int words = g.cand_words;
        unsigned bits[CAND_WORDS_PER_LANE];
        unsigned any = 0u;
#pragma unroll
        for (int q = 0; q < CAND_WORDS_PER_LANE; ++q) {
            bits[q] = (lane + 32 * q < words) ? g.cand[row * words + lane + 32 * q] : 0u;
            any |= bits[q];
        }
        if (__any_sync(0xffffffffu, any != 0u)) {
            for (int wi = 0; wi < words; ++wi) {
                unsigned bv = bits[0];
#pragma unroll
                for (int q = 1; q < CAND_WORDS_PER_LANE; ++q)
                    if ((wi >> 5) == q) bv = bits[q];
                unsigned word = __shfl_sync(0xffffffffu, bv, wi & 31);
                while (word) {
                    const int b = __ffs(word) - 1;
                    word &= word - 1;
                    const int slot = wi * 32 + b;
                    const int k = __ldg(g.list + slot);
                    if (k < 0) continue;
                    const double l = wide_pair_log2z(xr, g.mu_c + (size_t)slot * D, g.w2_c + (size_t)slot * D, __ldg(g.c2d_c + slot), D, lane, lim);
                    if (l >= lim && l > -CUDART_INF) { add_term(l); insert(l, k); }
                }
            }
        }
    }
    int p = 0;                                                // reported candidates evaluated (a prefix)
#pragma unroll
    for (int j = 0; j < NTOP; ++j) {
        // warp-uniform: the bounds descend, so the first that cannot matter ends the evaluation
        if (j == p && ap[j] >= 0 && !(cr + (double)ub[j] < tv[0] - 21.0)) {
            const int k = __ldg(g.comp_of + ap[j]);
            if (k >= 0 && k < g.K) {
                const double approx = cr + (double)(ub[j] - fmaf(__ldg(g.scrw + k), nrm, __ldg(g.scra + k)));
                const double l = wide_pair_log2z(xr, g.mu + (size_t)k * D, g.w2 + (size_t)k * D, __ldg(g.c2d + k), D, lane, -CUDART_INF);
                Ss -= exp2(approx - Mr);                      // its approximate term leaves the sum (Mr >= lz >= that term)
                if (l > -CUDART_INF) { add_term(l); insert(l, k); }
            }
            ++p;
        }
    }
    const int n_top = n_exact < GMM_MAX_TOPM ? n_exact : GMM_MAX_TOPM;
    const int rest = nvalid - p;                              // reported candidates that were not evaluated (they do not matter)
    bool certain = (n_top + rest >= m) && (Ss > 0.0) && (Ss < CUDART_INF);
    if (certain && p == NTOP) {
        // every reported candidate had to be evaluated: unreported components (all below the last bound) may matter too
        double vm = tv[0];
#pragma unroll
        for (int j = 1; j < GMM_MAX_TOPM; ++j)
            if (j == m - 1) vm = tv[j];
        certain = n_top >= m && vm > cr + (double)ub[NTOP - 1];
    }
    if (certain && !g.index_only && !(Ss - exact_part <= 1e-3 * Ss)) certain = false;
    if (!certain) {
        if (lane == 0) g.unc_rows[atomicAdd(g.unc_count, 1)] = (int32_t)row;
        return;
    }
    const double lzp = Mr + log2(Ss);
    if (lane < m) {
        double v;
        int k;
        if (lane < n_top) {
            v = tv[0]; k = tk[0];
#pragma unroll
            for (int j = 1; j < GMM_MAX_TOPM; ++j)
                if (lane == j) { v = tv[j]; k = tk[j]; }
        } else {
            const int q = p + (lane - n_top);                 // unevaluated candidates in the order of their bounds
            float a = ub[0];
            int pos = ap[0];
#pragma unroll
            for (int j = 1; j < NTOP; ++j)
                if (q == j) { a = ub[j]; pos = ap[j]; }
            k = __ldg(g.comp_of + pos);
            v = cr + (double)(a - fmaf(__ldg(g.scrw + k), nrm, __ldg(g.scra + k)));
        }
        g.idx[row * m + lane] = k;
        if (g.resp) g.resp[row * m + lane] = (float)exp2(v - lzp);
    }
}

// The sub-mixture's statistics go to the rows of its components (which the tensor passes left at zero).
__global__ void wide_ill_scatter_kernel(int D, int K, int n_ill, const int* __restrict__ list, const double* __restrict__ Nk_c,
                                        const double* __restrict__ S1_c, const double* __restrict__ S2_c, double* __restrict__ Nk,
                                        double* __restrict__ S1, double* __restrict__ S2) {
    const int j = blockIdx.x;
    if (j >= n_ill) return;
    const int k = list[j];
    if (k < 0) return;
    if (threadIdx.x == 0) Nk[k] += Nk_c[j];
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        S1[(size_t)k * D + d] += S1_c[(size_t)j * D + d];
        S2[(size_t)k * D + d] += S2_c[(size_t)j * D + d];
    }
}

// A plane [atoms][rows][128 bytes] seen as a 3-D tensor (x = 64 halves of an atom's row, y = row, z = atom): a box of
// (64, box_rows, box_atoms) is box_atoms contiguous blocks of box_rows x 128 bytes in memory and lands in shared memory as
// [atom][row][128 bytes], each 128-byte row swizzled.
cudaError_t wide_make_map(CUtensorMap* tm, void* base, int64_t rows, int atoms, int box_rows, int box_atoms) {
    const cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)atoms};
    const cuuint64_t strides[2] = {128, (cuuint64_t)rows * 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_atoms};
    const cuuint32_t estr[3] = {1, 1, 1};
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return e;
        if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        encode = reinterpret_cast<encode_fn>(fn);
    }
    const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

inline int64_t rows_padded_of(int64_t n) { return (n + WIDE_BATCH - 1) / WIDE_BATCH * WIDE_BATCH; }

}  // namespace

bool wide_supports(int D, int K) { return D > 128 && D <= WIDE_MAX_D && K >= 1 && K <= WIDE_MAX_K; }

WidePlan wide_plan(int D, int K, int num_sms) {
    WidePlan pl;
    pl.n_slices = (D + 127) / 128;
    pl.Dpad = pl.n_slices * 128;
    pl.CL = (K + 127) / 128;
    pl.Kpad = pl.CL * 128;
    pl.rows = pl.Kpad + 256;
    pl.R = num_sms / pl.CL;
    if (pl.R < 1) pl.R = 1;
    pl.pcols = 2 * pl.Dpad + 2;
    return pl;
}

cudaError_t launch_prepare_wide(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                                const WideBuffers& wb, float cond_limit, float min_weight, int hi_mode) {
    const WidePlan pl = wide_plan(D, K, 148);
    cudaError_t e = cudaMemsetAsync(wb.flags, 0, 8 * sizeof(int), s);
    if (e != cudaSuccess) return e;
    wide_scale_kernel<<<pl.Dpad, 128, 0, s>>>(D, K, pi, mu, var, wb.sd, wb.kap, wb.gd);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    wide_flag_kernel<<<K, 256, 0, s>>>(D, pl.Dpad, K, pi, mu, var, wb.sd, wb.kap, wb.gd, wb.illb, wb.scra, wb.scrw, wb.scra_hi, wb.scrw_hi, cond_limit,
                                       min_weight, wb.flags);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    wide_ill_list_kernel<<<1, 1024, 0, s>>>(K, pl.rows, wb.illb, wb.ill_list, wb.comp_of, wb.slot_of, wb.scr_mask, wb.flags);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    wide_prepare_kernel<<<pl.rows, 256, (size_t)2 * pl.Dpad * sizeof(double), s>>>(
        D, pl.Dpad, pl.rows, wb.comp_of, pi, mu, var, wb.sd, wb.kap, wb.gd, reinterpret_cast<__half*>(wb.p_hi),
        reinterpret_cast<__half*>(wb.p_lo), wb.tk, wb.ckd);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    wide_cref_kernel<<<1, 1024, 0, s>>>(pl.rows, wb.flags, wb.tk, wb.ckd, wb.comp_of, wb.slot_of, wb.scra, wb.scrw, wb.scra_hi, wb.scrw_hi, hi_mode, wb.cref,
                                        reinterpret_cast<float2*>(wb.tkck), reinterpret_cast<float2*>(wb.scr), wb.scr_e);
    return cudaGetLastError();
}

cudaError_t launch_ill_gather_wide(cudaStream_t s, int D, int n_ill, const WideBuffers& wb, const float* mu, const float* w2,
                                   const double* c2d) {
    wide_ill_gather_kernel<<<(unsigned)n_ill, 256, 0, s>>>(D, n_ill, wb.ill_list, mu, w2, c2d, wb.mu_c, wb.w2_c, wb.c2d_c);
    return cudaGetLastError();
}

cudaError_t launch_refine_wide(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                               const double* c2d, const WideBuffers& wb) {
    wide_refine_kernel<<<(unsigned)((n + 7) / 8), 256, 0, s>>>(X, n, D, K, mu, w2, c2d, wb.cref, reinterpret_cast<const float4*>(wb.top),
                                                               wb.comp_of, wb.logz, wb.logz_x);
    return cudaGetLastError();
}

cudaError_t launch_merge_ll_wide(cudaStream_t s, int64_t n, const WideBuffers& wb, const double* logz_ill) {
    wide_merge_ll_kernel<<<WIDE_LL_BLOCKS, 256, 0, s>>>(n, wb.logz, wb.logz_x, logz_ill, wb.llpart);
    return cudaGetLastError();
}

cudaError_t launch_ill_scatter_wide(cudaStream_t s, int D, int K, int n_ill, const WideBuffers& wb, double* Nk, double* S1,
                                    double* S2) {
    const size_t KD = (size_t)n_ill * D;
    wide_ill_scatter_kernel<<<(unsigned)n_ill, 256, 0, s>>>(D, K, n_ill, wb.ill_list, wb.stats_c, wb.stats_c + n_ill,
                                                            wb.stats_c + n_ill + KD, Nk, S1, S2);
    return cudaGetLastError();
}

cudaError_t launch_cand_clear_wide(cudaStream_t s, int64_t n, int n_slots, const WideBuffers& wb) {
    const int words = (n_slots + 31) / 32;
    cudaError_t e = cudaMemsetAsync(wb.ctl, 0, 8 * sizeof(int), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(wb.cand, 0, (size_t)n * words * sizeof(unsigned), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(wb.candT, 0, (size_t)n_slots * WIDE_CANDT_WORDS * sizeof(unsigned), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(wb.slot_cnt, 0, (size_t)n_slots * sizeof(int), s);
    return e;
}

cudaError_t launch_cand_filter_wide(cudaStream_t s, int64_t n, int n_slots, const WideBuffers& wb) {
    wide_cand_filter_kernel<<<(unsigned)((n + 7) / 8), 256, 0, s>>>(n, (n_slots + 31) / 32, wb.cand, wb.rec, wb.rec_cnt, wb.rec_thr, wb.ctl);
    return cudaGetLastError();
}

cudaError_t launch_cand_gate_wide(cudaStream_t s, const WideBuffers& wb, long long max_pairs) {
    wide_cand_gate_kernel<<<1, 1, 0, s>>>(wb.ctl, max_pairs);
    return cudaGetLastError();
}

cudaError_t launch_cand_count_wide(cudaStream_t s, int n_slots, const WideBuffers& wb) {
    wide_cand_count_kernel<<<1, 256, 0, s>>>(wb.ctl, wb.flags, wb.slot_cnt, n_slots);
    return cudaGetLastError();
}

cudaError_t launch_cand_lse_wide(cudaStream_t s, const float* X, int64_t n, int D, int n_slots, const WideBuffers& wb,
                                 double* logz_ill, int32_t* best_out) {
    const int words = (n_slots + 31) / 32;
    wide_cand_lse_kernel<0><<<(unsigned)((n + 7) / 8), 256, 0, s>>>(X, n, D, words, wb.cand, wb.candT, wb.mu_c, wb.w2_c, wb.c2d_c, wb.logz,
                                                                    logz_ill, wb.ctl, wb.slot_cnt, wb.pair_val, wb.pair_off, wb.pair_best, wb.ill_list, best_out,
                                                                    0, nullptr, nullptr, nullptr, nullptr, nullptr, 0, nullptr, wb.pair_key8, wb.pair_val8);
    return cudaGetLastError();
}

cudaError_t launch_cand_topm_wide(cudaStream_t s, const float* X, int64_t n, int D, int n_slots, const WideBuffers& wb, int m,
                                  int32_t* idx, float* resp, int32_t* unc_rows, int* unc_count, int ntop) {
    if (m < 1 || m > GMM_MAX_TOPM || (ntop != 6 && ntop != WIDE_MAX_TOP)) return cudaErrorInvalidValue;
    const int words = (n_slots + 31) / 32;
    wide_cand_lse_kernel<GMM_MAX_TOPM><<<(unsigned)((n + 7) / 8), 256, 0, s>>>(X, n, D, words, wb.cand, wb.candT, wb.mu_c, wb.w2_c, wb.c2d_c, wb.logz,
                                                                               nullptr, wb.ctl, wb.slot_cnt, wb.pair_val, wb.pair_off, wb.pair_best,
                                                                               wb.ill_list, nullptr, m, idx, resp, unc_rows, unc_count,
                                                                               wb.top, ntop, wb.comp_of, wb.pair_key8, wb.pair_val8);
    return cudaGetLastError();
}

cudaError_t launch_cand_mstep_wide(cudaStream_t s, const float* X, int64_t n, int D, int n_slots, const WideBuffers& wb) {
    double* Nk_c = wb.stats_c;
    double* S1_c = Nk_c + n_slots;
    double* S2_c = S1_c + (size_t)n_slots * D;
    wide_heavy_kernel<<<1, 1024, 0, s>>>(n_slots, wb.slot_cnt, wb.heavy_of, wb.heavy_slot, wb.ctl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const unsigned blocks = (unsigned)(n_slots + MS_HEAVY * (MS_SEG - 1));
    wide_cand_mstep_kernel<true><<<blocks, 256, 0, s>>>(X, n, D, wb.ill_list, wb.candT, wb.mu_c, wb.w2_c, wb.c2d_c, wb.gd, wb.logz_x, Nk_c, S1_c,
                                                        S2_c, wb.ctl, wb.heavy_of, wb.heavy_part, wb.cand, (n_slots + 31) / 32, wb.pair_val,
                                                        wb.pair_off, wb.pair_best, n_slots, wb.heavy_slot, wb.pair_key8, wb.pair_val8);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    wide_cand_mstep_kernel<false><<<blocks, 256, 0, s>>>(X, n, D, wb.ill_list, wb.candT, wb.mu_c, wb.w2_c, wb.c2d_c, wb.gd, wb.logz_x, Nk_c, S1_c,
                                                         S2_c, wb.ctl, wb.heavy_of, wb.heavy_part, wb.cand, (n_slots + 31) / 32, wb.pair_val,
                                                         wb.pair_off, wb.pair_best, n_slots, wb.heavy_slot, wb.pair_key8, wb.pair_val8);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    wide_heavy_combine_kernel<<<MS_HEAVY, 256, 0, s>>>(D, wb.heavy_slot, wb.heavy_part, Nk_c, S1_c, S2_c, wb.ctl);
    return cudaGetLastError();
}

cudaError_t launch_assign_refine_wide(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                                      const double* c2d, int n_slots, bool screened, const WideBuffers& wb, int ntop, int m,
                                      int32_t* idx, float* resp, int32_t* unc_rows, int* unc_count, bool index_only, bool hi) {
    if (m < 1 || m > GMM_MAX_TOPM || m > ntop) return cudaErrorInvalidValue;
    WideAssignArgs g;
    g.X = X; g.n = n; g.D = D; g.K = K; g.mu = mu; g.w2 = w2; g.c2d = c2d;
    g.comp_of = wb.comp_of; g.top = wb.top; g.logz = wb.logz; g.cref = wb.cref; g.n2 = wb.n2; g.scra = hi ? wb.scra_hi : wb.scra; g.scrw = hi ? wb.scrw_hi : wb.scrw;
    g.cand = screened ? wb.cand : nullptr; g.cand_words = (n_slots + 31) / 32; g.list = wb.ill_list;
    g.mu_c = wb.mu_c; g.w2_c = wb.w2_c; g.c2d_c = wb.c2d_c; g.ctl = screened ? wb.ctl : nullptr;
    g.m = m; g.idx = idx; g.resp = resp; g.unc_rows = unc_rows; g.unc_count = unc_count; g.index_only = index_only;
    const unsigned grid = (unsigned)((n + 7) / 8);
    if (ntop == 6) wide_assign_refine_kernel<6><<<grid, 256, 0, s>>>(g);
    else if (ntop == WIDE_MAX_TOP) wide_assign_refine_kernel<WIDE_MAX_TOP><<<grid, 256, 0, s>>>(g);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

cudaError_t launch_transform_wide(cudaStream_t s, const float* X, int64_t n, int D, const WideBuffers& wb, int* status, bool hi_only,
                                  bool with_norm) {
    if (n < 1 || n > WIDE_PIECE) return cudaErrorInvalidValue;
    const WidePlan pl = wide_plan(D, 1, 148);
    const int64_t rp = rows_padded_of(n);
    int64_t blocks = (rp + 7) / 8;                       // a warp per row
    if (blocks > 148 * 16) blocks = 148 * 16;
    wide_transform_kernel<<<(unsigned)blocks, 256, 0, s>>>(X, n, rp, D, pl.Dpad, wb.sd, wb.kap, wb.gd, wb.y_hi, hi_only ? nullptr : wb.y_lo,
                                                           with_norm ? wb.n2 : nullptr, status);
    return cudaGetLastError();
}

cudaError_t launch_lse_wide(cudaStream_t s, int64_t n, int D, int K, int Kg, int n_listed, int n_slots, const WideBuffers& wb,
                            int num_sms, int* status, int ntop, int hi_first_slots, bool pre_pass, bool record, bool listed_only,
                            int topm) {
    if (n < 1 || n > WIDE_PIECE || Kg < 0 || Kg > K || (Kg < 1 && n_listed < 1)) return cudaErrorInvalidValue;
    const WidePlan pl = wide_plan(D, K, num_sms);
    const int64_t rp = rows_padded_of(n);
    const int atoms = 4 * pl.n_slices;
    CUtensorMap tm_yhi, tm_ylo, tm_phi, tm_plo;
    cudaError_t e = wide_make_map(&tm_yhi, wb.y_hi, rp, atoms, WIDE_TILE, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_ylo, wb.y_lo, rp, atoms, WIDE_TILE, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_phi, wb.p_hi, pl.rows, atoms, 128, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_plo, wb.p_lo, pl.rows, atoms, 128, 1);
    if (ntop != 2 && ntop != 6 && ntop != WIDE_MAX_TOP) return cudaErrorInvalidValue;
    if (e == cudaSuccess)
        e = ntop == 2 ? cudaFuncSetAttribute(lse_wide_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, L_SMEM)
          : ntop == 6 ? cudaFuncSetAttribute(lse_wide_kernel<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, L_SMEM)
                      : cudaFuncSetAttribute(lse_wide_kernel<WIDE_MAX_TOP>, cudaFuncAttributeMaxDynamicSharedMemorySize, L_SMEM);
    if (e != cudaSuccess) return e;
    const int Kgp = (Kg + 255) & ~255;                   // where the listed components start
    const bool screen = n_listed > 0 && n_slots > 0;
    const int cols = screen ? (Kgp + n_listed) : Kg;
    if (cols > pl.rows) return cudaErrorInvalidValue;
    LseParams p;
    p.n = n; p.NC = (cols + 127) / 128; p.NZ = atoms;
    p.tkck = reinterpret_cast<const float2*>(wb.tkck); p.cref = wb.cref; p.logz = wb.logz; p.llpart = nullptr; p.status = status;
    p.top = wb.top;
    p.screen = screen;
    p.scr = reinterpret_cast<const float2*>(wb.scr);
    p.scr_e = wb.scr_e; p.scr_mask = wb.scr_mask; p.slot_of = wb.slot_of; p.n2 = wb.n2; p.cand = wb.cand;
    p.cand_words = (n_slots + 31) / 32; p.scr_group = Kgp / 256; p.ctl = wb.ctl;
    p.hi_group = 0x7fffffff; p.hi_end = 0x7fffffff; p.pre_pass = 0;
    p.topm = 0;
    if (topm > 0) {                                          // the assignment by screening: as the EM step's screening mode
        if (ntop == 2 || topm > ntop || !screen || !listed_only || hi_first_slots != 0) return cudaErrorInvalidValue;
        p.topm = topm;
        p.hi_group = Kgp / 256; p.hi_end = 0x7fffffff;
    }
    const bool em_like = ntop == 2 || topm > 0;
    p.g0 = (listed_only && screen && em_like) ? Kgp / 256 : 0;
    p.rec = (record && screen && em_like) ? wb.rec : nullptr; p.rec_cnt = wb.rec_cnt; p.rec_thr = wb.rec_thr;
    if (ntop == 2 && screen && hi_first_slots >= 0) {                                                      // the EM step's screening mode
        p.hi_group = (Kgp + hi_first_slots + 255) / 256;
        p.pre_pass = pre_pass ? 1 : 0;
    }
    if (ntop != 2 && hi_first_slots >= 0 && topm <= 0) { p.hi_group = 0; p.hi_end = Kgp / 256; }             // the assignment's evaluated groups
    const int64_t ntiles = (n + WIDE_TILE - 1) / WIDE_TILE;
    const unsigned grid = (unsigned)(ntiles < num_sms ? ntiles : num_sms);
    if (ntop == 2) lse_wide_kernel<2><<<grid, WT_THREADS, L_SMEM, s>>>(p, tm_yhi, tm_ylo, tm_phi, tm_plo);
    else if (ntop == 6) lse_wide_kernel<6><<<grid, WT_THREADS, L_SMEM, s>>>(p, tm_yhi, tm_ylo, tm_phi, tm_plo);
    else lse_wide_kernel<WIDE_MAX_TOP><<<grid, WT_THREADS, L_SMEM, s>>>(p, tm_yhi, tm_ylo, tm_phi, tm_plo);
    return cudaGetLastError();
}

cudaError_t launch_em_wide(cudaStream_t s, int64_t n, int D, int K, int Kg, const WideBuffers& wb, int num_sms, int* status) {
    if (n < 1 || n > WIDE_PIECE || Kg < 1 || Kg > K) return cudaErrorInvalidValue;
    const WidePlan pk = wide_plan(D, K, num_sms);
    const WidePlan pl = wide_plan(D, Kg, num_sms);       // the sweep covers the evaluated positions only
    const int64_t rp = rows_padded_of(n);
    const int atoms = 4 * pl.n_slices;
    CUtensorMap tm_phi, tm_plo, tm_ye_hi, tm_ye_lo, tm_ym_hi, tm_ym_lo;
    cudaError_t e = wide_make_map(&tm_phi, wb.p_hi, pk.rows, atoms, 128, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_plo, wb.p_lo, pk.rows, atoms, 128, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_ye_hi, wb.y_hi, rp, atoms, WIDE_BATCH, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_ye_lo, wb.y_lo, rp, atoms, WIDE_BATCH, 1);
    if (e == cudaSuccess) e = wide_make_map(&tm_ym_hi, wb.y_hi, rp, atoms, 64, 2);
    if (e == cudaSuccess) e = wide_make_map(&tm_ym_lo, wb.y_lo, rp, atoms, 64, 2);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(em_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, E_SMEM);
    if (e != cudaSuccess) return e;
    EmWideParams p;
    p.n = n; p.CL = pl.CL; p.R = pl.R; p.NZ = atoms; p.pcols = pl.pcols;
    p.tkck = reinterpret_cast<const float2*>(wb.tkck); p.ckd = wb.ckd; p.logz = wb.logz; p.partial = wb.partial; p.status = status;
    em_wide_kernel<<<(unsigned)(pl.CL * pl.R), WT_THREADS, E_SMEM, s>>>(p, tm_phi, tm_plo, tm_ye_hi, tm_ye_lo, tm_ym_hi, tm_ym_lo);
    return cudaGetLastError();
}

cudaError_t launch_reduce_wide(cudaStream_t s, int D, int K, int Kg, const WideBuffers& wb, int num_sms, double* Nk, double* S1,
                               double* S2) {
    if (Kg < 1 || Kg > K) return cudaErrorInvalidValue;
    const WidePlan pl = wide_plan(D, Kg, num_sms);       // the plan of the sweep that wrote the partial blocks
    const size_t per = (size_t)Kg + 2 * (size_t)Kg * D;
    wide_reduce_kernel<<<(unsigned)((per + 255) / 256), 256, 0, s>>>(D, Kg, pl.CL, pl.R, pl.pcols, wb.partial, wb.comp_of, wb.sd,
                                                                     wb.kap, wb.gd, Nk, S1, S2);
    return cudaGetLastError();
}

}  // namespace fg
