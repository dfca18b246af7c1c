// Top-m assignment on the tensor cores (sm_100a, tcgen05 + TMEM): paper Sections 4.2-4.3 (hard assignment and
// multi-assignment read the largest responsibilities of every vector), computed from the same expanded quadratic form
// as the E-step of Algorithm 1.
//
// Two kernels per piece of at most TC_YPOINTS points, after tc_transform_kernel has written the fp16 planes of Y:
//
//   assign_tc_kernel   lanes of TMEM = POINTS (the E+M tile kernel has lanes = components because its M-step needs that;
//                      selection wants the opposite: one thread owns one point and walks over the components, so neither
//                      the log-sum-exp nor the selection needs a single cross-lane operation or an exchange between CTAs).
//                      A persistent CTA takes tiles of 128 points: the tile's two planes of Y stay in shared memory (A operand,
//                      128 KB) while the coefficient planes P_hi, P_lo of all K components stream through a ring of
//                      32 KB stages (B operand: 128 components x 64 columns x 2 planes, from L2 by TMA).  Per chunk of 128
//                      components: logits (approximate, 22-bit operands) = Y_hi P_lo + Y_lo P_hi + Y_hi P_hi in a 128-column TMEM
//                      buffer; two such buffers, one per softmax warpgroup, alternate.  A softmax thread keeps for its point
//                      the running (max, sum) of the log-sum-exp and the LIST largest logits with their indices, and
//                      writes one record per tile.
//   assign_refine_kernel  first one thread per point: it merges the records of the two warpgroups, and where a single
//                      component matters (all others below 2^-21 of it) it writes the answer from the approximate values.
//                      The other points are taken by a whole warp each: the candidates that matter (at most LIST - 1)
//                      are recomputed EXACTLY (fp32 direct differences, the arithmetic of the FP32 path), the
//                      log-sum-exp is corrected by the difference between exact and approximate candidate terms, the
//                      exact values are ordered (ties to the smaller index) and the top m written.  That result is
//                      certain when the m-th exact value clears the best value left outside by more than the error
//                      bound of the approximation, and accurate when the terms that stayed approximate are a small part
//                      of the log-sum-exp; otherwise (near ties, exact ties, fewer than m finite candidates, broad
//                      posteriors) the row is put on a list, and the FP32 tile kernel evaluates the listed rows against
//                      all K components afterwards.  Ill-conditioned components take no part in the selection and are
//                      evaluated exactly where a test on their 8 dimensions of largest weight does not rule them out.
#include "internal.cuh"
#include "em_tc.cuh"

#define TC_WAIT_LIMIT_NS 2000000000ull
#include "tc_prims.cuh"

namespace fg {

namespace {

constexpr int AT_POINTS = 128;               // points per tile = TMEM lanes
constexpr int AT_COMPS = 128;                // components per chunk = MMA N
constexpr int AT_THREADS = 320;              // 8 softmax warps, producer warp, MMA warp
constexpr int AT_PRODUCER = 8, AT_MMA = 9;
constexpr int AT_STAGES = 3;
constexpr int AT_ATOM = 16384;               // 128 rows x 128 bytes
constexpr int ASM_A = 0;                     // [plane][atom]: 2 x 4 x 16384
constexpr int ASM_ALO = 4 * AT_ATOM;
constexpr int ASM_B = 8 * AT_ATOM;           // stages x [plane]: 3 x 2 x 16384
constexpr int ASM_BAR = ASM_B + AT_STAGES * 2 * AT_ATOM;
constexpr int ASM_BYTES = ASM_BAR + 256 + 1024;      // barriers, alignment slack

enum { AB_AFULL = 0, AB_AEMPTY = 4, AB_BFULL = 8, AB_BEMPTY = 8 + AT_STAGES, AB_LFULL = 8 + 2 * AT_STAGES,
       AB_LEMPTY = AB_LFULL + 2, AB_FINAL = AB_LEMPTY + 2, AB_COUNT };

struct AssignParams {
    int64_t n;                 // points of this piece
    int n_chunks, n_ks;
    const float2* tkck;        // [n_chunks * 128] (t_k, c_k): log2 z = t_k * contraction + c_k
    float* rec;                // [n][2][RECW] records (see assign_recw)
    int* status;
    const int* gate;           // the launch does nothing when gate[0] != 0 (too many ill-conditioned components: the FP32 kernels run instead)
};

constexpr int assign_recw(int LIST) { return (2 + 2 * LIST + 3) & ~3; }      // words per record: m, s, LIST values, LIST indices

template <int LIST>
__global__ void __launch_bounds__(AT_THREADS, 1)
assign_tc_kernel(const AssignParams p, const __grid_constant__ CUtensorMap tm_yhi, const __grid_constant__ CUtensorMap tm_ylo,
                 const __grid_constant__ CUtensorMap tm_phi, const __grid_constant__ CUtensorMap tm_plo) {
    extern __shared__ unsigned char smem_raw[];
    if (p.gate[0] != 0) return;                                     // uniform over the grid, before anything is allocated
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, drain_s;
    volatile int* abort_flag = &abort_s;
    volatile int* drain_flag = &drain_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t ntiles = (p.n + AT_POINTS - 1) / AT_POINTS;
    const int64_t ntl = ((int64_t)blockIdx.x < ntiles) ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int NC = p.n_chunks;
    const int n_atoms = (p.n_ks + 3) >> 2;

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ASM_BAR);
    auto BAR = [&](int i) { return smem_u32(&bars[i]); };

    if (tid == 0) {
        abort_s = 0;
        drain_s = 0;
        for (int a = 0; a < 4; ++a) { bar_init(BAR(AB_AFULL + a), 1); bar_init(BAR(AB_AEMPTY + a), 1); }
        for (int s = 0; s < AT_STAGES; ++s) { bar_init(BAR(AB_BFULL + s), 1); bar_init(BAR(AB_BEMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) { bar_init(BAR(AB_LFULL + b), 1); bar_init(BAR(AB_LEMPTY + b), 128); }
        bar_init(BAR(AB_FINAL), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == AT_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = tmem_base_s;

    if (warp < 8) {
        // =========================== softmax / selection warps ===========================
        // Warpgroup g takes the chunks c with c mod 2 = g (logits buffer g).  Thread = TMEM lane = point.
        const int grp = warp >> 2, wq = warp & 3;
        const uint32_t lane_addr = ((uint32_t)(wq * 32)) << 16;
        const uint32_t tbuf = tmem + grp * AT_COMPS + lane_addr;
        constexpr int RECW = assign_recw(LIST);
        uint32_t uses = 0;                       // completed uses of this group's buffer
        bool alive = true;
        for (int64_t i = 0; i < ntl && alive; ++i) {
            const int64_t row = (blockIdx.x + i * gridDim.x) * AT_POINTS + wq * 32 + lane;
            float m_run = -1e30f, s_run = 0.f;          // finite start: a first block of -inf logits must not make NaN
            float tv[LIST];
            int ti[LIST];
#pragma unroll
            for (int j = 0; j < LIST; ++j) { tv[j] = -CUDART_INF_F; ti[j] = -1; }
            for (int c = grp; c < NC; c += 2) {
                // every lane waits itself, and the warp leaves together: the TMEM loads below are warp-wide instructions
                const bool got = bar_wait(BAR(AB_LFULL + grp), uses & 1u, abort_flag, p.status, false);
                if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
                fence_after();
                ++uses;
#pragma unroll 1
                for (int sub = 0; sub < 4; ++sub) {
                    uint32_t v[32];
                    tmem_ld32(tbuf + sub * 32, v);
                    tmem_wait_ld();
                    if (sub == 3) {                     // the buffer's last columns are in registers: hand it back
                        fence_before();
                        bar_arrive(BAR(AB_LEMPTY + grp));
                    }
                    const int col0 = c * AT_COMPS + sub * 32;
                    const float4* tc4 = reinterpret_cast<const float4*>(p.tkck + col0);
                    float l[32];
                    float bmax = -CUDART_INF_F;
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float4 q = __ldg(tc4 + (j >> 1));          // (t, c) of two components; same address in every lane
                        l[j] = fmaf(__uint_as_float(v[j]), q.x, q.y);
                        l[j + 1] = fmaf(__uint_as_float(v[j + 1]), q.z, q.w);
                        bmax = fmaxf(bmax, fmaxf(l[j], l[j + 1]));
                    }
                    if (bmax > m_run) {
                        s_run *= fast_ex2(m_run - bmax);
                        m_run = bmax;
                    }
                    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        acc0 += fast_ex2(l[j] - m_run);
                        acc1 += fast_ex2(l[j + 1] - m_run);
                    }
                    s_run += acc0 + acc1;
                    // the LIST largest: most blocks hold nothing that beats any lane's current LIST-th value
                    if (__any_sync(0xffffffffu, bmax > tv[LIST - 1])) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (l[j] > tv[LIST - 1]) {              // strict: of equal values the smaller index stays
                                tv[LIST - 1] = l[j];
                                ti[LIST - 1] = col0 + j;
#pragma unroll
                                for (int q = LIST - 1; q > 0; --q) {
                                    if (tv[q] > tv[q - 1]) {
                                        const float fv = tv[q]; tv[q] = tv[q - 1]; tv[q - 1] = fv;
                                        const int fi = ti[q]; ti[q] = ti[q - 1]; ti[q - 1] = fi;
                                    }
                                }
                            }
                        }
                    }
                }
            }
            if (alive && row < p.n) {
                float w[RECW];
                w[0] = m_run;
                w[1] = s_run;
#pragma unroll
                for (int j = 0; j < LIST; ++j) { w[2 + j] = tv[j]; w[2 + LIST + j] = __int_as_float(ti[j]); }
#pragma unroll
                for (int j = 2 + 2 * LIST; j < RECW; ++j) w[j] = 0.f;
                float4* dst = reinterpret_cast<float4*>(p.rec + ((size_t)row * 2 + grp) * RECW);
#pragma unroll
                for (int j = 0; j < RECW; j += 4) dst[j >> 2] = make_float4(w[j], w[j + 1], w[j + 2], w[j + 3]);
            }
        }
    } else if (warp == AT_PRODUCER) {
        // =========================== producer warp (TMA) ===========================
        // Order of the loads = order of use: the tile's A atoms are interleaved with the B stages of its first chunk.  An A
        // atom of the next tile is loaded as soon as the last chunk's MMAs over that atom have completed, i.e. while the
        // rest of that chunk still runs.
        int64_t g = 0;                               // B steps issued
        int64_t a_tile[4] = {-1, -1, -1, -1};        // last tile whose atom was requested
        bool ok = true;
        auto wait0 = [&](uint32_t bar, uint32_t parity) -> bool {
            uint32_t w = 1;
            if (lane == 0) w = bar_wait(bar, parity, abort_flag, p.status, false) ? 1u : 0u;
            return __shfl_sync(0xffffffffu, w, 0) != 0u;
        };
        for (int64_t i = 0; i < ntl && ok; ++i) {
            const int32_t row0 = (int32_t)((blockIdx.x + i * gridDim.x) * AT_POINTS);
            for (int c = 0; c < NC && ok; ++c) {
                for (int a = 0; a < n_atoms && ok; ++a) {
                    if (c == 0) {
                        if (i > 0 && !wait0(BAR(AB_AEMPTY + a), (uint32_t)((i - 1) & 1))) { ok = false; break; }
                        if (elect_one()) {
                            bar_expect_tx(BAR(AB_AFULL + a), 2 * AT_ATOM);
                            tma_load_3d(smem_u32(smem + ASM_A + a * AT_ATOM), &tm_yhi, 0, row0, a, BAR(AB_AFULL + a));
                            tma_load_3d(smem_u32(smem + ASM_ALO + a * AT_ATOM), &tm_ylo, 0, row0, a, BAR(AB_AFULL + a));
                            if (i + 1 < ntl) {       // the planes come from HBM: ask for the next tile's atom now
                                const int32_t rown = (int32_t)((blockIdx.x + (i + 1) * gridDim.x) * AT_POINTS);
                                tma_prefetch_3d(&tm_yhi, 0, rown, a);
                                tma_prefetch_3d(&tm_ylo, 0, rown, a);
                            }
                        }
                        __syncwarp();
                        a_tile[a] = i;
                    }
                    const int st = (int)(g % AT_STAGES);
                    const int64_t use = g / AT_STAGES;
                    if (use > 0 && !wait0(BAR(AB_BEMPTY + st), (uint32_t)((use - 1) & 1))) { ok = false; break; }
                    if (elect_one()) {
                        const uint32_t dst = smem_u32(smem + ASM_B + st * 2 * AT_ATOM);
                        bar_expect_tx(BAR(AB_BFULL + st), 2 * AT_ATOM);
                        tma_load_3d(dst, &tm_phi, 0, c * AT_COMPS, a, BAR(AB_BFULL + st));
                        tma_load_3d(dst + AT_ATOM, &tm_plo, 0, c * AT_COMPS, a, BAR(AB_BFULL + st));
                    }
                    __syncwarp();
                    ++g;
                }
            }
        }
        // After an abort nobody may be waiting for the last loads, yet they must have landed before the CTA exits.
        if (!ok || *abort_flag) {
            for (int a = 0; a < 4; ++a) {
                if (a_tile[a] >= 0 && lane == 0) bar_wait(BAR(AB_AFULL + a), (uint32_t)(a_tile[a] & 1), drain_flag, p.status, false);
                __syncwarp();
            }
            for (int64_t h = (g > AT_STAGES ? g - AT_STAGES : 0); h < g; ++h) {
                if (lane == 0) bar_wait(BAR(AB_BFULL + (int)(h % AT_STAGES)), (uint32_t)((h / AT_STAGES) & 1), drain_flag, p.status, false);
                __syncwarp();
            }
        }
    } else {
        // =========================== MMA warp ===========================
        // The whole warp runs the loop convergently: lane 0 waits and broadcasts, one elected lane issues and commits.
        const uint32_t idesc = make_idesc(AT_POINTS, AT_COMPS, 0);
        const uint64_t d_ahi = make_desc(smem_u32(smem + ASM_A), 16, 1024);
        const uint64_t d_alo = make_desc(smem_u32(smem + ASM_ALO), 16, 1024);
        const uint64_t d_b = make_desc(smem_u32(smem + ASM_B), 16, 1024);
        bool alive = true;
        auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
            uint32_t ok = 1;
            if (lane == 0) ok = bar_wait(bar, parity, abort_flag, p.status, false) ? 1u : 0u;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            fence_after();
            return ok != 0u;
        };
        int64_t g = 0;
        uint32_t cnt[2] = {0u, 0u};
        for (int64_t i = 0; i < ntl && alive; ++i) {
            for (int c = 0; c < NC && alive; ++c) {
                const int b = c & 1;
                if (cnt[b] > 0 && !wait_all(BAR(AB_LEMPTY + b), (cnt[b] - 1) & 1u)) { alive = false; break; }
                ++cnt[b];
                const uint32_t d = tmem + b * AT_COMPS;
                for (int a = 0; a < n_atoms; ++a) {
                    if (c == 0 && !wait_all(BAR(AB_AFULL + a), (uint32_t)(i & 1))) { alive = false; break; }
                    const int st = (int)(g % AT_STAGES);
                    if (!wait_all(BAR(AB_BFULL + st), (uint32_t)((g / AT_STAGES) & 1))) { alive = false; break; }
                    if (elect_one()) {
                        const int kk = (p.n_ks - 4 * a < 4) ? (p.n_ks - 4 * a) : 4;          // k-steps of this atom
                        const uint64_t ah = d_ahi + ((a * AT_ATOM) >> 4), al = d_alo + ((a * AT_ATOM) >> 4);
                        const uint64_t bh = d_b + ((st * 2 * AT_ATOM) >> 4), bl = bh + (AT_ATOM >> 4);
                        // the two small cross products first, then the leading one (as in the E-step of the tile kernel)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < kk) mma_ss(d, ah + ((j * 32) >> 4), bl + ((j * 32) >> 4), idesc, (a > 0 || j > 0) ? 1u : 0u);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < kk) mma_ss(d, al + ((j * 32) >> 4), bh + ((j * 32) >> 4), idesc, 1u);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < kk) mma_ss(d, ah + ((j * 32) >> 4), bh + ((j * 32) >> 4), idesc, 1u);
                        mma_commit(BAR(AB_BEMPTY + st));
                        if (c == NC - 1) mma_commit(BAR(AB_AEMPTY + a));
                        if (a == n_atoms - 1) mma_commit(BAR(AB_LFULL + b));
                    }
                    __syncwarp();
                    ++g;
                }
            }
        }
        // drain: every MMA issued by this warp has completed before TMEM is released
        if (elect_one()) mma_commit(BAR(AB_FINAL));
        __syncwarp();
        if (lane == 0) bar_wait(BAR(AB_FINAL), 0, drain_flag, p.status, false);
        __syncwarp();
        fence_after();
    }

    fence_before();
    __syncthreads();
    if (warp == AT_MMA) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------------
// Exact log2 z of (point, component) pairs by direct differences in fp32, one warp per point.  Lane l holds the
// dimensions 4 l .. 4 l + 3 of the point (16-byte loads; D a multiple of 4 and 16-byte aligned rows), else the
// dimensions l, l + 32, l + 64, l + 96.
struct PointRow {
    float x[4];
    bool vec;
    __device__ __forceinline__ void load(const float* __restrict__ xr, int D, int lane) {
        vec = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(xr) & 15) == 0);
        if (vec) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (4 * lane < D) v = __ldg(reinterpret_cast<const float4*>(xr) + lane);
            x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) x[j] = (lane + 32 * j < D) ? __ldg(xr + lane + 32 * j) : 0.f;
        }
    }
    // this lane's share of sum_d w (x - mu)^2 and, with MAG, of sum_d w (|x| + |mu|)^2 (the size of the terms the
    // expanded form adds up); mr, wr: rows of a [K][D] array whose base is 16-byte aligned
    template <bool MAG>
    __device__ __forceinline__ float partial(const float* __restrict__ mr, const float* __restrict__ wr, int D, int lane, float& mag) const {
        float q = 0.f, t = 0.f;
        if (vec) {
            if (4 * lane < D) {
                const float4 m4 = __ldg(reinterpret_cast<const float4*>(mr) + lane);
                const float4 w4 = __ldg(reinterpret_cast<const float4*>(wr) + lane);
                const float mm[4] = {m4.x, m4.y, m4.z, m4.w}, ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float diff = x[j] - mm[j];
                    q = fmaf(diff * diff, ww[j], q);
                    if (MAG) { const float a = fabsf(x[j]) + fabsf(mm[j]); t = fmaf(a * a, ww[j], t); }
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int d = lane + 32 * j;
                if (d < D) {
                    const float mu = __ldg(mr + d), w = __ldg(wr + d);
                    const float diff = x[j] - mu;
                    q = fmaf(diff * diff, w, q);
                    if (MAG) { const float a = fabsf(x[j]) + fabsf(mu); t = fmaf(a * a, w, t); }
                }
            }
        }
        mag = t;
        return q;
    }
    template <bool MAG>
    __device__ __forceinline__ float quad(const float* __restrict__ mr, const float* __restrict__ wr, int D, int lane, float& mag) const {
        float t;
        float q = partial<MAG>(mr, wr, D, lane, t);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            q += __shfl_xor_sync(0xffffffffu, q, o);
            if (MAG) t += __shfl_xor_sync(0xffffffffu, t, o);
        }
        mag = t;
        return q;
    }
};


// Warp-uniform list (every lane holds the same copy) of the MAXM largest exact values seen so far: descending, equal
// values in ascending component order, whatever the order of insertion.
template <int MAXM>
struct ExactTop {
    float v[MAXM];
    int k[MAXM];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int j = 0; j < MAXM; ++j) { v[j] = -CUDART_INF_F; k[j] = -1; }
    }
    __device__ __forceinline__ void insert(float e, int kk) {
        constexpr int L = MAXM - 1;
        if (!(k[L] < 0 || e > v[L] || (e == v[L] && kk < k[L]))) return;
        v[L] = e; k[L] = kk;
#pragma unroll
        for (int j = L; j > 0; --j) {
            if (k[j - 1] < 0 || v[j] > v[j - 1] || (v[j] == v[j - 1] && k[j] < k[j - 1])) {
                const float fv = v[j]; v[j] = v[j - 1]; v[j - 1] = fv;
                const int fk = k[j]; k[j] = k[j - 1]; k[j - 1] = fk;
            }
        }
    }
    __device__ __forceinline__ float value_at(int pos) const {
        float r = -CUDART_INF_F;
#pragma unroll
        for (int j = 0; j < MAXM; ++j) if (j == pos) r = v[j];
        return r;
    }
    __device__ __forceinline__ int index_at(int pos) const {
        int r = -1;
#pragma unroll
        for (int j = 0; j < MAXM; ++j) if (j == pos) r = k[j];
        return r;
    }
};

// Per-thread sorted list of approximate values (descending, equal values in ascending component order).
template <int LIST>
struct ApproxList {
    float a[LIST];
    int i[LIST];
    __device__ __forceinline__ void insert(float val, int id) {
        constexpr int L = LIST - 1;
        if (!(i[L] < 0 || val > a[L] || (val == a[L] && id < i[L]))) return;
        a[L] = val; i[L] = id;
#pragma unroll
        for (int j = L; j > 0; --j) {
            if (i[j - 1] < 0 || a[j] > a[j - 1] || (a[j] == a[j - 1] && i[j] < i[j - 1])) {
                const float fv = a[j]; a[j] = a[j - 1]; a[j - 1] = fv;
                const int fi = i[j]; i[j] = i[j - 1]; i[j - 1] = fi;
            }
        }
    }
};

struct RefineArgs {
    const float* X; int64_t n; int D, K;
    const float* mu; const float* w2; const float* c2;
    int m; int32_t* idx_out; float* resp_out;
    float e_launch; int n_ill;
    int32_t* unc_rows; int* unc_count;      // rows left to the exact kernel (row + row_offset), and their number
    int row_offset;                         // position of this piece inside the window of pieces that share the list
    bool index_only;                        // the caller uses the indices alone: no demand on the accuracy of the log-sum-exp
};

// One point, the whole warp: exact evaluation of what matters (see assign_refine_kernel).  Lane q < LIST holds the q-th
// best approximate value sv and its component si of the point (-inf / -1 where there is none).
template <int LIST, int MAXM>
__device__ __forceinline__ void refine_point(const RefineArgs& g, const TcIllCache& ill, int64_t row, int lane, float sv, int si,
                                             float m0, float s0, float m1, float s1) {
    constexpr int C = LIST - 1;                                  // candidates that may be recomputed exactly
    const float NEG = -CUDART_INF_F;
    const int m = g.m, D = g.D;
    const float e_launch = g.e_launch;
    const int nvalid = __popc(__ballot_sync(0xffffffffu, si >= 0));
    const int nc = nvalid < C ? nvalid : C;
    // A component matters when its responsibility may exceed 2^-21 (4.8e-7): those are evaluated exactly.  Among the rest,
    // order and values are those of the approximate pass (differences below the 1e-6 tie width of the assignment).
    const float a0 = __shfl_sync(0xffffffffu, sv, 0);
    const float matter = a0 - e_launch - 21.f;
    const int p = __popc(__ballot_sync(0xffffffffu, lane < nc && sv >= matter));      // a prefix: the values descend
    PointRow pr;
    pr.load(g.X + row * D, D, lane);
    ExactTop<MAXM> top;
    top.init();
    int n_exact = 0;                                              // exact values inserted into `top`

    // Ill-conditioned components are evaluated exactly, unless their 8 dimensions of largest weight (kept in shared
    // memory, one component per lane) already show that the component can neither reach the top m (its value stays below
    // a lower bound of the m-th largest) nor weigh in the log-sum-exp (2^-40 of the largest term): a component that has
    // collapsed in some dimensions is hopeless for every point but its own.  Their terms of the log-sum-exp are summed
    // on line: (Mi, Si).
    float Mi = NEG, Si = 0.f;
    if (g.n_ill > 0) {
        const float a_m = __shfl_sync(0xffffffffu, sv, m - 1);
        const float skip_below = fminf(a_m - (e_launch + 1.f), fmaxf(m0, m1) - e_launch - 40.f);
        const float* xr = g.X + row * D;
        for (int base = 0; base < g.n_ill; base += 32) {
            const int t = base + lane;
            float part = 0.f, cc = NEG;
            if (t < g.n_ill) {
                cc = ill.c[t];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float diff = __ldg(xr + ill.dim[j][t]) - ill.mu[j][t];          // (the row sits in L1 by now)
                    part = fmaf(diff * diff, ill.w[j][t], part);
                }
            }
            // cc - part is an upper bound of the value: the other dimensions only lower it
            unsigned alive_set = __ballot_sync(0xffffffffu, t < g.n_ill && !(cc - part < skip_below));
            while (alive_set) {
                const int k = ill.k[base + __ffs(alive_set) - 1];
                alive_set &= alive_set - 1;
                float mag;
                const float e = __ldg(g.c2 + k) - pr.quad<false>(g.mu + (size_t)k * D, g.w2 + (size_t)k * D, D, lane, mag);
                if (e > NEG) {
                    top.insert(e, k);
                    ++n_exact;
                    if (e > Mi) { Si = Si * fast_ex2(Mi - e) + 1.f; Mi = e; }
                    else Si += fast_ex2(e - Mi);
                }
            }
        }
    }

    // Candidates that matter, exactly, all of them at once (their loads and reductions overlap).  A point with a single
    // component that matters needs none: its responsibility is 1 - (what the approximate pass summed for the others).
    // Error bound of an approximate logit: from the parameters (8 x the estimate, over the components of the approximate
    // pass) plus from this point (8 x 2^-22 x the summed magnitude of the terms of the best candidate, doubled for the
    // others).
    float ev = NEG, ea = NEG, tmax = 0.f;
    int evaluated = 0;
    if (p >= 2 || (p == 1 && n_exact > 0)) {
        float qv[C];
        int kv[C];
        float mag0 = 0.f;
#pragma unroll
        for (int r = 0; r < C; ++r) {
            kv[r] = __shfl_sync(0xffffffffu, si, r);
            qv[r] = 0.f;
            if (r < p) {
                float mg;
                if (r == 0) { qv[r] = pr.partial<true>(g.mu + (size_t)kv[r] * D, g.w2 + (size_t)kv[r] * D, D, lane, mg); mag0 = mg; }
                else qv[r] = pr.partial<false>(g.mu + (size_t)kv[r] * D, g.w2 + (size_t)kv[r] * D, D, lane, mg);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mag0 += __shfl_xor_sync(0xffffffffu, mag0, o);
#pragma unroll
            for (int r = 0; r < C; ++r)
                if (r < p) qv[r] += __shfl_xor_sync(0xffffffffu, qv[r], o);
        }
        tmax = 2.f * mag0;
#pragma unroll
        for (int r = 0; r < C; ++r) {
            if (r < p) {
                const float e = __ldg(g.c2 + kv[r]) - qv[r];
                if (lane == r) { ev = e; ea = sv; }
                if (e > NEG) { top.insert(e, kv[r]); ++n_exact; }
            }
        }
        evaluated = p;
    }
    const int n_top = n_exact < MAXM ? n_exact : MAXM;            // what the list holds
    const float ebound = e_launch + 1.9073486e-06f * tmax;
    const float next_a = __shfl_sync(0xffffffffu, sv, evaluated);      // best approximate value among what was not evaluated (lane LIST - 1 at most)
    // The first m come from the exact list, then from the unevaluated candidates in approximate order.
    bool certain = n_top + (nvalid - evaluated) >= m && (n_top >= m || nvalid <= C || next_a < matter || evaluated == 0);
    if (certain && n_top >= m)
        certain = next_a == NEG || next_a < matter || top.value_at(m - 1) > next_a + ebound;
    float M = fmaxf(m0, m1), S = 0.f;
    if (certain) {
        if (n_top > 0) M = fmaxf(M, top.v[0]);
        // log-sum-exp: the approximate total with the evaluated candidates' approximate terms replaced by the exact ones,
        // plus the ill-conditioned components.  The terms that stay approximate carry a relative error of a few 1e-4
        // each: where components were evaluated, the result is kept only if the others make up less than a tenth of the
        // total.
        float ex = (ev > NEG) ? fast_ex2(ev - M) : 0.f;
        float ap = (ea > NEG) ? fast_ex2(ea - M) : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ex += __shfl_xor_sync(0xffffffffu, ex, o);
            ap += __shfl_xor_sync(0xffffffffu, ap, o);
        }
        if (Si > 0.f) ex += Si * fast_ex2(Mi - M);
        S = (s0 * fast_ex2(m0 - M) + s1 * fast_ex2(m1 - M) - ap) + ex;
        if (!(S > 0.f) || !(S < CUDART_INF_F)) certain = false;
        else if (!g.index_only && evaluated > 0 && !(S - ex <= 0.1f * S)) certain = false;
    }
    if (certain) {
        // lane j writes output j: from the exact list, then from the unevaluated candidates
        int q = evaluated + lane - n_top;
        q = q < 0 ? 0 : (q > 31 ? 31 : q);
        const float va = __shfl_sync(0xffffffffu, sv, q);
        const int ka = __shfl_sync(0xffffffffu, si, q);
        const bool from_top = lane < n_top;
        const float v = from_top ? top.value_at(lane) : va;
        const int k = from_top ? top.index_at(lane) : ka;
        if (lane < m) {
            g.idx_out[row * m + lane] = k;
            if (g.resp_out) g.resp_out[row * m + lane] = __fdividef(fast_ex2(v - M), S);
        }
        return;
    }
    // Not certain (near ties, exact ties, too few finite candidates, broad posteriors): the point joins the list of rows
    // that the FP32 tile kernel evaluates against all K components afterwards.  (The order of the list varies from run to
    // run; the result of a row does not depend on it.)
    if (lane == 0) g.unc_rows[atomicAdd(g.unc_count, 1)] = (int32_t)row + g.row_offset;
}

// A warp takes 32 consecutive points.  First every lane looks at one point on its own: it merges the records of the two
// warpgroups and, if only one component matters for the point (the second best approximate value lies 21 + the error
// bound below the best, and no ill-conditioned component passes the test on its 8 decisive dimensions), writes the answer straight from
// the approximate values: the best responsibility is 1 - (the rest), the others are below 6e-8.  The points that are
// left are then taken one after the other by the whole warp (refine_point).
template <int LIST, int MAXM>
__global__ void __launch_bounds__(256)
assign_refine_kernel(const float* __restrict__ rec, const float* __restrict__ X, int64_t n, int D, int K,
                     const float* __restrict__ mu, const float* __restrict__ w2, const float* __restrict__ c2,
                     const int* __restrict__ flags, const TcIllCache* __restrict__ ill_cache, int m, int32_t* __restrict__ idx_out,
                     float* __restrict__ resp_out, int32_t* __restrict__ unc_rows, int* __restrict__ unc_count, int row_offset,
                     int index_only) {
    if (flags[3] != 0) return;
    constexpr int RECW = assign_recw(LIST);
    RefineArgs g;
    g.unc_rows = unc_rows; g.unc_count = unc_count; g.row_offset = row_offset; g.index_only = index_only != 0;
    g.X = X; g.n = n; g.D = D; g.K = K; g.mu = mu; g.w2 = w2; g.c2 = c2; g.m = m; g.idx_out = idx_out; g.resp_out = resp_out;
    g.e_launch = __int_as_float(flags[1]);          // error bound of the approximate logits from the parameters
    g.n_ill = flags[2];                             // ill-conditioned components (<= TC_MAX_ILL): left out of the approximate pass
    const int lane = threadIdx.x & 31;
    __shared__ TcIllCache ill;
    if (g.n_ill > 0) {
        const int* src = reinterpret_cast<const int*>(ill_cache);
        int* dst = reinterpret_cast<int*>(&ill);
        for (int i = threadIdx.x; i < (int)(sizeof(TcIllCache) / 4); i += blockDim.x) dst[i] = __ldg(src + i);
    }
    __syncthreads();
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const float NEG = -CUDART_INF_F;
    for (int64_t base = warp0 * 32; base < n; base += nwarps * 32) {
        const int64_t row = base + lane;
        const bool valid = row < n;
        ApproxList<LIST> al;
        float m0 = -1e30f, s0 = 0.f, m1 = -1e30f, s1 = 0.f;
#pragma unroll
        for (int j = 0; j < LIST; ++j) { al.a[j] = NEG; al.i[j] = -1; }
        if (valid) {
            const float4* r4 = reinterpret_cast<const float4*>(rec + (size_t)row * 2 * RECW);
            float w[2 * RECW];
#pragma unroll
            for (int j = 0; j < 2 * RECW / 4; ++j) {
                const float4 q = __ldg(r4 + j);
                w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
            }
            m0 = w[0]; s0 = w[1]; m1 = w[RECW]; s1 = w[RECW + 1];
#pragma unroll
            for (int j = 0; j < LIST; ++j) { al.a[j] = w[2 + j]; al.i[j] = __float_as_int(w[2 + LIST + j]); }      // sorted already
#pragma unroll
            for (int j = 0; j < LIST; ++j) {
                const int id = __float_as_int(w[RECW + 2 + LIST + j]);
                if (id >= 0) al.insert(w[RECW + 2 + j], id);
            }
        }
        int nv = 0;
#pragma unroll
        for (int j = 0; j < LIST; ++j) nv += (al.i[j] >= 0) ? 1 : 0;
        bool sharp = valid && nv >= m && al.a[1] < al.a[0] - g.e_launch - 21.f;
        if (sharp && g.n_ill > 0) {
            float a_m = NEG;
#pragma unroll
            for (int j = 0; j < LIST; ++j) if (j == m - 1) a_m = al.a[j];
            const float skip_below = fminf(a_m - (g.e_launch + 1.f), fmaxf(m0, m1) - g.e_launch - 40.f);
            const float* xr = X + row * D;
            for (int t = 0; t < g.n_ill && sharp; ++t) {
                // upper bound of the component's value from its dimensions of largest weight, the largest first: most
                // components are out after one
                float ub = ill.c[t];
                bool out = false;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (!out) {
                        const float diff = __ldg(xr + ill.dim[j][t]) - ill.mu[j][t];
                        ub -= diff * diff * ill.w[j][t];
                        out = ub < skip_below;
                    }
                }
                if (!out) sharp = false;
            }
        }
        if (sharp) {
            const float M = fmaxf(m0, m1);
            const float S = s0 * fast_ex2(m0 - M) + s1 * fast_ex2(m1 - M);
#pragma unroll
            for (int j = 0; j < LIST; ++j) {
                if (j < m) {
                    idx_out[row * m + j] = al.i[j];
                    if (resp_out) resp_out[row * m + j] = __fdividef(fast_ex2(al.a[j] - M), S);
                }
            }
        }
        unsigned todo = __ballot_sync(0xffffffffu, valid && !sharp);
        while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            float sv = NEG;
            int si = -1;
#pragma unroll
            for (int q = 0; q < LIST; ++q) {
                const float v = __shfl_sync(0xffffffffu, al.a[q], src);
                const int i = __shfl_sync(0xffffffffu, al.i[q], src);
                if (lane == q) { sv = v; si = i; }
            }
            refine_point<LIST, MAXM>(g, ill, base + src, lane, sv, si, __shfl_sync(0xffffffffu, m0, src),
                                     __shfl_sync(0xffffffffu, s0, src), __shfl_sync(0xffffffffu, m1, src),
                                     __shfl_sync(0xffffffffu, s1, src));
        }
    }
}

template <int LIST>
cudaError_t launch_assign_t(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                            const float* c2, const TcBuffers& tb, float* rec, int32_t* unc_rows, int* unc_count, int row_offset, int m,
                            int32_t* idx, float* resp, int* status, bool index_only) {
    const TcPlan pl = tc_plan(D, K, 148);
    AssignParams p;
    p.n = n; p.n_chunks = pl.CL; p.n_ks = pl.n_ks;
    p.tkck = reinterpret_cast<const float2*>(tb.tkck);
    p.rec = rec; p.status = status; p.gate = tb.flags + 3;
    const int64_t rows_padded = (n + TC_BN - 1) / TC_BN * TC_BN;       // what launch_transform_tc wrote
    CUtensorMap tm_yhi, tm_ylo, tm_phi, tm_plo;
    cudaError_t e = tc_make_plane_map(&tm_yhi, tb.y_hi, rows_padded, AT_POINTS, 1);
    if (e != cudaSuccess) return e;
    e = tc_make_plane_map(&tm_ylo, tb.y_lo, rows_padded, AT_POINTS, 1);
    if (e != cudaSuccess) return e;
    e = tc_make_plane_map(&tm_phi, tb.p_hi_rm, pl.Kpad, AT_COMPS, 1);
    if (e != cudaSuccess) return e;
    e = tc_make_plane_map(&tm_plo, tb.p_lo_rm, pl.Kpad, AT_COMPS, 1);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(assign_tc_kernel<LIST>, cudaFuncAttributeMaxDynamicSharedMemorySize, ASM_BYTES);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int64_t ntiles = (n + AT_POINTS - 1) / AT_POINTS;
    const unsigned grid = (unsigned)(ntiles < sms ? ntiles : sms);          // persistent: one CTA per SM
    assign_tc_kernel<LIST><<<grid, AT_THREADS, ASM_BYTES, s>>>(p, tm_yhi, tm_ylo, tm_phi, tm_plo);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t batches = (n + 31) / 32;                                         // a warp takes 32 points at a time
    const int64_t warps_wanted = batches < (int64_t)sms * 64 ? batches : (int64_t)sms * 64;
    const unsigned rgrid = (unsigned)((warps_wanted + 7) / 8);
    assign_refine_kernel<LIST, (LIST <= 6 ? 4 : GMM_MAX_TOPM)><<<rgrid, 256, 0, s>>>(rec, X, n, D, K, mu, w2, c2, tb.flags, tb.ill_cache, m, idx,
                                                                               resp, unc_rows, unc_count, row_offset, index_only ? 1 : 0);
    return cudaGetLastError();
}

}  // namespace


// LIST = 6 (m <= 4) or 10: the m wanted, at least one spare candidate, and the best value left outside (for the certainty
// test).  Small m keeps 5 candidates too: the responsibilities are only as accurate as the share of the log-sum-exp that
// the exactly evaluated components hold.
size_t assign_tc_record_bytes(int m) { return (size_t)2 * assign_recw(m <= 4 ? 6 : 10) * sizeof(float); }

cudaError_t launch_assign_tc(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                             const float* c2, const TcBuffers& tb, float* rec, int32_t* unc_rows, int* unc_count, int row_offset, int m,
                             int32_t* idx, float* resp, int* status, bool index_only) {
    if (n < 1 || n > TC_YPOINTS || m < 1 || m > GMM_MAX_TOPM) return cudaErrorInvalidValue;
    // A caller that wants the nearest component alone (the k-means step) needs two candidates and the best value left
    // outside, and no accurate log-sum-exp: the selection keeps 3 values per thread instead of 6.
    if (index_only && m == 1)
        return launch_assign_t<3>(s, X, n, D, K, mu, w2, c2, tb, rec, unc_rows, unc_count, row_offset, m, idx, resp, status, true);
    if (m <= 4) return launch_assign_t<6>(s, X, n, D, K, mu, w2, c2, tb, rec, unc_rows, unc_count, row_offset, m, idx, resp, status, false);
    return launch_assign_t<10>(s, X, n, D, K, mu, w2, c2, tb, rec, unc_rows, unc_count, row_offset, m, idx, resp, status, false);
}

}  // namespace fg
