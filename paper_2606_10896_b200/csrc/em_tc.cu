// Tensor-core path (sm_100a, tcgen05 + TMEM): the fused E+M tile kernel on the expanded quadratic form.
//
// What one launch computes (paper Algorithm 1, both sweeps, for every tile of 64 points):
//   E-step   L[k, i] = sum_c P[k, c] * Y[i, c]         P = per-component coefficients (a = log2e mu/var, b = -log2e/(2 var)),
//                                                      Y = [x | x^2], contraction length 2 * 128 padded dimensions
//   log2 z_ik = t_k * L[k, i] + c_k                     (row scale t_k, constant c_k = log2e (log pi_k - 1/2 sum_d (mu^2/var + log 2 pi var)))
//   log-sum-exp over ALL K components of a point        (warp butterflies, then one (max, sum) exchange per tile between the ceil(K/128) CTAs of a
//                                                        group through tagged slots in global memory (L2): each CTA owns 128 components)
//   r_ik = 2^(log2 z_ik - log2 Z_i)                     on chip only: written back into TMEM as the A operand of the M-step
//   M-step   S[k, c] += sum_i r_ik * Y[i, c]            accumulators stationary in TMEM for the CTA's whole life
// Precision: every operand is split into two fp16 values (hi + lo, 22 bits).  E-step = P_hi Y_hi + P_hi Y_lo + P_lo Y_hi,
// M-step = r_hi Y_hi + r_hi Y_lo + r_lo Y_hi, fp32 accumulation in TMEM.  Columns of P / Y are interleaved so that one
// k-step of 16 holds [8 dims of x | the same 8 dims of x^2], which keeps partial sums small.  N_k is summed from the same
// rounded r (hi + lo) that feeds the M-step.  Accumulators are flushed to float64 partials every TC_FLUSH tiles so that
// no fp32 accumulation chain is longer than that.
//
// Layout: lanes of TMEM = components.  TMEM columns: [0,256) statistics accumulator, [256,384) P_hi (fp16 pairs),
// [384,448) / [448,512) logits of the two tiles in flight (overwritten in place by r_hi | r_lo).
// Shared memory: P_lo (64 KB, SW128 K-major), two stages of Y (hi and lo planes, written by TMA with the 128-byte swizzle;
// read K-major by the E-step and MN-major by the M-step), exchange buffers, barriers.
//
// Warp roles (10 warps): warps 0-7 softmax (two warpgroups, each taking 32 of a tile's 64 points; warp w owns TMEM lanes
// 32 (w mod 4) ...), warp 8 produces the Y stages (TMA loads of the fp16 planes that tc_transform_kernel wrote once for
// all CTAs, one 3-D box per plane, L2 prefetch two tiles ahead), warp 9 issues the MMAs: the whole warp runs the issue loop
// convergently, lane 0 does the waits and broadcasts their outcome, one elected lane issues (descriptors = hoisted base +
// immediate offset, loops unrolled) and commits.  Three issue orders exist (pairs, interleaved, whichever-is-ready =
// default); all give identical results.  Every wait is bounded by a wall-clock limit;
// on expiry the CTA sets ST_TIMEOUT, all roles leave their loops, TMEM is freed and the kernel returns.
#include "internal.cuh"
#include "em_tc.cuh"

#include <cuda.h>
#include <cuda_fp16.h>
#include <math_constants.h>

namespace fg {
namespace {
// Wall-clock limit of every device-side wait, in ns (2 s; a test of the time-out path shortens it).
__constant__ unsigned long long c_wait_limit_ns = 2000000000ull;
}  // namespace
}  // namespace fg
#define TC_WAIT_LIMIT_NS c_wait_limit_ns
#include "tc_prims.cuh"

namespace fg {

namespace {

constexpr int BN = TC_BN;                 // points per tile
constexpr int NTHREADS = 320;          // 8 softmax warps, 1 producer warp, 1 MMA warp (10 warps: up to 200 registers each)
constexpr int MMA_WARP = 9;
constexpr int PRODUCER_WARP = 8;
constexpr float RSCALE = TC_RSCALE;
#define WAIT_LIMIT_NS TC_WAIT_LIMIT_NS
constexpr float ILL_MARGIN = 40.f;     // log2 units: a logit more than this below the best one is negligible (2^-40)

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int SM_PLO = 0;                       // 65536
constexpr int SM_Y = 65536;                     // 2 stages x (hi 32768 + lo 32768)
constexpr int SM_YSTAGE = 65536;
constexpr int SM_YLO = 32768;
constexpr int SM_MISC = SM_Y + 2 * SM_YSTAGE;   // 196608
constexpr int SM_GATHER = SM_MISC;              // 2 groups x 4 warps x 64 floats    2048
constexpr int SM_WS = SM_GATHER + 2048;         // 2 groups x 4 warps x 64 float2    4096
constexpr int SM_FAC = SM_WS + 4096;            // 2 groups x 4 warps x 64 floats    2048
constexpr int SM_LL = SM_FAC + 2048;            // 2 x 64 doubles                1024
constexpr int SM_BAR = SM_LL + 1024;             // barriers                       256
constexpr int SM_END = SM_BAR + 256;
constexpr int SMEM_BYTES = SM_END + 1024;       // + alignment slack

enum { B_YFULL0 = 0, B_YFULL1, B_YEMPTY0, B_YEMPTY1, B_LFULL0, B_LFULL1, B_RREADY0, B_RREADY1, B_ACCFULL,
       B_ACCFREE, B_FINAL, B_COUNT };


// ---- exchange between the CTAs of a group through global memory (L2).  A slot is two 64-bit words {value, tag}: each
//      word is written and read as one unit, so a reader that sees the expected tag in both words has both values.
//      Slots form a ring of 4 per (group, source CTA): a CTA writes tile i+4 only after it has finished tile i+2, which
//      needed every peer's tile-(i+2) slot, which that peer wrote after it had read all slots of tile i.
struct __align__(16) XSlot { float a; uint32_t ta; float b; uint32_t tb; };
__device__ __forceinline__ void xslot_write(XSlot* q, float a, float b, uint32_t tag) {
    asm volatile("st.relaxed.gpu.global.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"l"(q), "r"(__float_as_uint(a)), "r"(tag), "r"(__float_as_uint(b)), "r"(tag) : "memory");
}
__device__ __forceinline__ void xslot_load(const XSlot* q, uint32_t (&v)[4]) {
    asm volatile("ld.relaxed.gpu.global.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "l"(q) : "memory");
}

// Bounded poll of the CL slots of one point (stride 64 slots between source CTAs): all outstanding loads are issued
// together, so one round costs one L2 round trip.  Called by a whole warp, one point per lane; the warp leaves the loop
// TOGETHER (when every lane has all its slots): lanes that left at different rounds would run the code that follows
// once per group of lanes, which cost more than the wait itself.
__device__ __forceinline__ bool xslot_wait_all(const XSlot* q, int CL, uint32_t tag, float2 (&e)[8], volatile int* abort_flag,
                                               int* status) {
    uint32_t pending = (CL >= 32) ? 0xffffffffu : ((1u << CL) - 1u);
#pragma unroll
    for (int c = 0; c < 8; ++c) e[c] = make_float2(-CUDART_INF_F, 0.f);
    unsigned long long t0 = 0;
    for (int it = 0;; ++it) {
        uint32_t v[8][4];
#pragma unroll
        for (int c = 0; c < 8; ++c)
            if (pending & (1u << c)) xslot_load(q + c * 64, v[c]);
#pragma unroll
        for (int c = 0; c < 8; ++c)
            if ((pending & (1u << c)) && v[c][1] == tag && v[c][3] == tag) {
                e[c] = make_float2(__uint_as_float(v[c][0]), __uint_as_float(v[c][2]));
                pending &= ~(1u << c);
            }
        if (__all_sync(0xffffffffu, pending == 0u)) return true;
        bool give_up = *abort_flag != 0;
        if ((it & 15) == 15) {
            const unsigned long long now = gtime();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                atomicOr(status, ST_TIMEOUT);
                give_up = true;
            }
        }
        if (__any_sync(0xffffffffu, give_up)) return false;
    }
}


// Groups of more than 8 CTAs (K > 1024), used by the BIG instantiation of the kernel only (the common instantiation
// contains none of this, so its register allocation is not touched).
// The (max, sum) pairs of the CL source CTAs are collected 8 at a time and merged as they come: mi = max, Z = sum of
// s 2^(m - mi).
__device__ __forceinline__ bool xslot_collect_many(const XSlot* ring, int CL, uint32_t tag, float& mi_out, float& Z_out,
                                                volatile int* abort_flag, int* status) {
    float mi = -CUDART_INF_F, Z = 0.f;
    bool all = true;
    for (int cb = 0; cb < CL; cb += 8) {
        float2 e[8];
        const int nc = (CL - cb < 8) ? (CL - cb) : 8;
        if (!xslot_wait_all(ring + cb * 64, nc, tag, e, abort_flag, status)) all = false;
        float m8 = mi;
#pragma unroll
        for (int c = 0; c < 8; ++c) m8 = fmaxf(m8, e[c].x);
        const float m8_safe = (m8 == -CUDART_INF_F) ? 0.f : m8;
        Z = (mi == -CUDART_INF_F) ? 0.f : Z * fast_ex2(mi - m8_safe);
#pragma unroll
        for (int c = 0; c < 8; ++c) Z += (e[c].x == -CUDART_INF_F) ? 0.f : e[c].y * fast_ex2(e[c].x - m8_safe);
        mi = m8;
    }
    mi_out = mi;
    Z_out = Z;
    return all;
}
// The lower-bound slots beyond the first 32 of a point (slot s at q + 64 s): lane l takes slots 32 + l, 64 + l, ...; lb
// becomes the maximum with what it already holds.  Returns false if a slot does not carry the tag yet.
__device__ __forceinline__ bool xslot_more_bounds(const XSlot* q, int nslots, uint32_t tag, int lane, float& lb) {
    bool ok = true;
    for (int sb = 32 + lane; sb < nslots; sb += 32) {
        uint32_t v[4];
        xslot_load(q + sb * 64, v);
        if (v[1] == tag && v[3] == tag) lb = fmaxf(lb, __uint_as_float(v[0]));
        else ok = false;
    }
    return ok;
}

// ---- warp reduce-scatter butterflies over 64 per-thread values: afterwards lane l holds the reduction (over the
//      32 lanes) for points 2l and 2l+1.  62 shuffles instead of 64 x 5.
template <int HALF, bool IS_MAX>
__device__ __forceinline__ void bfly_round(const float (&v)[2 * HALF], float (&out)[HALF], bool upper, int mask) {
#pragma unroll
    for (int j = 0; j < HALF; ++j) {
        const float mine = upper ? v[HALF + j] : v[j];
        const float other = upper ? v[j] : v[HALF + j];
        const float recv = __shfl_xor_sync(0xffffffffu, other, mask);
        out[j] = IS_MAX ? fmaxf(mine, recv) : (mine + recv);
    }
}
template <bool IS_MAX>
__device__ __forceinline__ void warp_reduce_scatter(const float (&v)[64], float (&out)[2], int lane) {
    float a[32], b[16], c[8], d[4];
    bfly_round<32, IS_MAX>(v, a, lane & 16, 16);
    bfly_round<16, IS_MAX>(a, b, lane & 8, 8);
    bfly_round<8, IS_MAX>(b, c, lane & 4, 4);
    bfly_round<4, IS_MAX>(c, d, lane & 2, 2);
    bfly_round<2, IS_MAX>(d, out, lane & 1, 1);
}

// 32-value variant: afterwards lane l holds the reduction for point l.
template <bool IS_MAX>
__device__ __forceinline__ void warp_reduce_scatter32(const float (&v)[32], float& out, int lane) {
    float a[16], b[8], c[4], d[2], e[1];
    bfly_round<16, IS_MAX>(v, a, lane & 16, 16);
    bfly_round<8, IS_MAX>(a, b, lane & 8, 8);
    bfly_round<4, IS_MAX>(b, c, lane & 4, 4);
    bfly_round<2, IS_MAX>(c, d, lane & 2, 2);
    bfly_round<1, IS_MAX>(d, e, lane & 1, 1);
    out = e[0];
}


// s_d x of point r (0..63) of the tile held in a Y stage (the two fp16 planes, 128-byte swizzle as TMA wrote them)
__device__ __forceinline__ float y_scaled_x(const unsigned char* stage, int r, int d) {
    const int cx = 16 * (d >> 3) + (d & 7);              // column of dimension d (k-step interleaved order)
    const int atom = cx >> 6, cc = cx & 63;
    const uint32_t off = (uint32_t)(atom * 8192 + r * 128 + ((((cc >> 3) ^ (r & 7)) << 4) | ((cc & 7) << 1)));
    const __half hi = *reinterpret_cast<const __half*>(stage + off);
    const __half lo = *reinterpret_cast<const __half*>(stage + SM_YLO + off);
    return __half2float(hi) + __half2float(lo);
}

struct TcKernelParams {
    const float* X;
    int64_t n;
    int D, K, CL, Q, n_ks, flush, order;
    int test_silent_rank;          // >= 0: that CTA of group 0 never publishes its exchange slot for tile 0 (time-out test)
    const uint32_t* phi_img;       // [CL][128 lanes][128] packed fp16 pairs
    const unsigned char* plo_img;  // [CL][65536] shared-memory image (SW128, K-major)
    const float* tk;               // [CL*128]
    const float* ck;               // [CL*128]
    const float* illb;             // [CL*128] 0, or for an ill-conditioned component a bound E_k on the error of its approximate log2 z
    const int* flags;              // [0] != 0 when some component is ill-conditioned (kernel-uniform protocol switch)
    const float* mu;               // [K][D] means (exact recomputation)
    const float* w2;               // [K][D] (log2 e / 2) / var
    const float* c2;               // [K] log2 e (log pi - 1/2 sum log(2 pi var))
    const int* dec_dim;            // [CL*128][8] ill-conditioned components: their 8 dimensions of largest weight (descending),
    const float* dec_w;            // [CL*128][8] the weight there in units of the scaled data: (log2 e / 2) / (var s_d^2),
    const float* dec_mu;           // [CL*128][8] and the scaled mean s_d mu
    double* partial;               // [Q][TC_PCOLS][CL*128]  (+=)
    double* llpart;                // [2 Q]
    XSlot* xg;                     // [Q][4][CL][64] exchange slots (zeroed before every launch)
    XSlot* xl;                     // [Q][4][CL][4][64] lower-bound slots, one per warp and point
    int* status;
    // Grouped launches (one group of points per CTA group, e.g. Fisher vectors): tile t of the planes holds tile_valid[t]
    // points (0 .. BN; the rest of its rows are zeros) taken from rows tile_src[t] .. of X.  Both NULL otherwise.
    const int* tile_valid;
    const int64_t* tile_src;
};

// BIG: groups of more than 8 CTAs (1024 < K <= 4096).  TIGHT: the filter for launches in which many components are
// ill-conditioned (see `tight` below); the host picks it from the count the previous preparation reported.
template <bool BIG, bool TIGHT>
__global__ void __launch_bounds__(NTHREADS, 1) em_tc_kernel(const TcKernelParams p, const __grid_constant__ CUtensorMap tm_hi,
                                                            const __grid_constant__ CUtensorMap tm_lo) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int drain_s;          // never raised: drain waits end on completion or on the time limit, not on an abort
    __shared__ int decision_s[2];
    volatile int* abort_flag = &abort_s;
    volatile int* drain_flag = &drain_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = blockIdx.x % p.CL;          // slice of 128 components within the group
    const int cluster_id = blockIdx.x / p.CL;          // group index: a group of CL CTAs covers all K components of its tiles
    const int64_t ntiles = (p.n + BN - 1) / BN;
    const int64_t ntl = (cluster_id < ntiles) ? (ntiles - cluster_id + p.Q - 1) / p.Q : 0;   // tiles of this cluster

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM_BAR);
    auto BAR = [&](int i) { return smem_u32(&bars[i]); };

    if (tid == 0) {
        abort_s = 0;
        drain_s = 0;
        decision_s[0] = 0;
        decision_s[1] = 0;
        bar_init(BAR(B_YFULL0), 1);    bar_init(BAR(B_YFULL1), 1);      // one arrive.expect_tx by the producer + the TMA bytes
        bar_init(BAR(B_YEMPTY0), 1);   bar_init(BAR(B_YEMPTY1), 1);
        bar_init(BAR(B_LFULL0), 1);    bar_init(BAR(B_LFULL1), 1);
        bar_init(BAR(B_RREADY0), 256); bar_init(BAR(B_RREADY1), 256);
        bar_init(BAR(B_ACCFULL), 1);   bar_init(BAR(B_ACCFREE), 128);
        bar_init(BAR(B_FINAL), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // P_lo image -> shared memory (plain 16-byte copies; the image is already swizzled)
    {
        const uint4* src = reinterpret_cast<const uint4*>(p.plo_img + (size_t)rank * 65536);
        uint4* dst = reinterpret_cast<uint4*>(smem + SM_PLO);
        for (int i = tid; i < 65536 / 16; i += NTHREADS) dst[i] = __ldg(src + i);
    }
    fence_async_smem();
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = tmem_base_s;
    const uint32_t T_ACC = tmem, T_PHI = tmem + 256, T_LOG = tmem + 384;

    if (warp < 4) {
        // P_hi -> TMEM (thread = lane = component of this CTA's slice)
        const uint32_t* src = p.phi_img + ((size_t)rank * 128 + tid) * 128;
        const uint32_t lane_addr = ((uint32_t)(warp * 32)) << 16;
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t v[32];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(src + c0 + j));
                v[j] = q.x; v[j + 1] = q.y; v[j + 2] = q.z; v[j + 3] = q.w;
            }
            tmem_st32(T_PHI + lane_addr + c0, v);
        }
        tmem_wait_st();
    }
    fence_before();
    __syncthreads();
    fence_after();

    if (warp < 8) {
        // =========================== softmax warps ===========================
        // Two warpgroups share every tile: group g (warps 4g..4g+3) takes points 32g..32g+31, so the latency between the
        // E-step and the M-step of a tile is that of a 32-point softmax (latency, not throughput, is what the tensor
        // pipe waits for).
        const int grp = warp >> 2, wq = warp & 3, gtid = tid & 127;
        const int p0 = 32 * grp;                                // first point of this group within the tile
        const uint32_t lane_addr = ((uint32_t)(wq * 32)) << 16;
        const int kloc = gtid;                                  // component within the slice
        const float tk = p.tk[rank * 128 + kloc];
        const float ck = p.ck[rank * 128 + kloc];
        const float illb = p.illb[rank * 128 + kloc];
        const bool any_ill = p.flags[0] != 0;
        // Two filters for flagged components.  With few of them (large N / K: a few percent, truly collapsed ones) the test
        // on the error bound alone discards nearly every pair, and anything more only adds instructions to every tile.
        // With many (small N / K: half of the components narrow in a few dimensions) that test passes almost everything
        // and the exact test on the decisive dimensions takes over (TIGHT; both give correct results on any input).
        const bool tight = TIGHT && any_ill;
        float emax_w = illb;                                    // largest error bound among this warp's components
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) emax_w = fmaxf(emax_w, __shfl_xor_sync(0xffffffffu, emax_w, o));
        float* gather = reinterpret_cast<float*>(smem + SM_GATHER) + warp * 32;    // [8 warps][32]
        float2* ws = reinterpret_cast<float2*>(smem + SM_WS) + grp * 128;          // [4][32] per group
        float* fac = reinterpret_cast<float*>(smem + SM_FAC) + grp * 128;          // [4][32] per group
        XSlot* xg = p.xg + (size_t)cluster_id * 4 * p.CL * 64;             // [4][CL][64] ring of exchange slots
        XSlot* xl = p.xl + (size_t)cluster_id * 4 * p.CL * 256;            // [4][CL][4 warps][64]: lower bounds (ill-conditioned mode)
        float nk_acc = 0.f;
        // log2 Z of this lane's points (rank 0, first warp of the group): a compensated fp32 sum, formed AFTER the tile's
        // responsibilities were handed over, so that neither float64 arithmetic nor the logarithm sits on the path that
        // the whole group of CTAs waits on
        float ll_s = 0.f, ll_c = 0.f, ll_m = 0.f, ll_z = 1.f;
        bool ll_have = false;
        // partial layout [group][column][component]: the 32 lanes of a warp touch 32 consecutive doubles; every address
        // belongs to exactly one thread of the grid, so the reductions below are deterministic
        const size_t pstride = (size_t)p.CL * 128;
        double* prow = p.partial + (size_t)cluster_id * TC_PCOLS * pstride + rank * 128 + kloc;
        bool alive = true;

        // Softmax threads leave the loop only at the uniform decision point after named barrier 2: a thread that
        // left earlier would strand the others in a hardware barrier.
        for (int64_t i = 0; i < ntl; ++i) {
            const int s = (int)(i & 1);
            const uint32_t ph = (uint32_t)((i >> 1) & 1);
            const int64_t tile = cluster_id + i * p.Q;
            const int64_t row0 = tile * BN;
            const int tile_points = p.tile_valid ? __ldg(p.tile_valid + tile) : (int)((p.n - row0 < BN) ? (p.n - row0) : BN);
            const int nvalid = tile_points - p0;                                      // valid points of this group's half
            const int64_t xrow0 = p.tile_src ? __ldg(p.tile_src + tile) : row0;       // where the tile's points sit in X

            if (!bar_wait(BAR(B_LFULL0 + s), ph, abort_flag, p.status, false)) alive = false;
            fence_after();
            float l[32];
            {
                uint32_t v0[32];
                tmem_ld32(T_LOG + s * 64 + p0 + lane_addr, v0);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) l[j] = fmaf(__uint_as_float(v0[j]), tk, ck);
            }
            float red;
            // Ill-conditioned components (sum_d mu^2 / var too large for the 22-bit expanded form, e.g. a component
            // collapsed onto one point at the variance floor): their approximate logits carry an error of up to E_k.
            // A (component, point) pair can only matter if its upper bound l + E_k reaches the best LOWER bound
            // max_k' (l - E_k') over ALL K components minus the 2^-40 margin.  In launches that have such components
            // every warp publishes a lower bound of its per-point maximum (a store, no wait, no barrier).  A warp first tests its
            // flagged lanes against the warp's own bound (a weaker, local bound that already discards
            // almost everything: a collapsed component is hopeless for every point but its own); the rare survivors
            // are checked against the group-wide bound read from the published slots and, if they pass, recomputed
            // exactly with direct differences in fp32, the whole warp working on one pair at a time.
            // warp-level max per point (lane j ends up with point j).  In a warp that has flagged components the maximum is
            // taken over the well-conditioned ones only: that is a valid lower bound of the point's best log2 z (E = 0), a
            // tight one, and it is also the maximum of everything that stays in play: a flagged pair either fails the
            // tests below (its value lies 2^-40 below this bound or is removed) or is recomputed exactly, after which the
            // maxima are formed again.
            if (tight && emax_w > 0.f) {
                float lt[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) lt[j] = (illb > 0.f) ? -CUDART_INF_F : l[j];
                warp_reduce_scatter32<true>(lt, red, lane);
            } else {
                warp_reduce_scatter32<true>(l, red, lane);
            }
            if (any_ill) {
                // max_k (l_k - E_k) >= max_k l_k - max_k E_k: the warp maximum minus the warp's largest error bound is a
                // valid lower bound (and for a warp without flagged lanes it is the maximum itself)
                const uint32_t tag = (uint32_t)(i + 1);
                XSlot* ring = xl + (size_t)(i & 3) * p.CL * 256 + p0;
                // this warp's lower bound for point `lane`: see above, or max_k (l_k - E_k) >= max_k l_k - max_k E_k
                const float lb_own = tight ? red : red - emax_w;
                uint32_t mlo = 0;
                if (emax_w > 0.f) {
                    // Local filter, by shuffles (no shared memory, no warp barrier: a barrier here would also wait for
                    // global stores in flight): bit j of mlo = point j of this lane's component may matter.
                    // (only flagged lanes: in the tight mode a warp without a well-conditioned component has the bound -inf,
                    // which every value reaches, also the -inf of a padded component)
                    const bool flagged = illb > 0.f;
                    const float reach = illb + ILL_MARGIN;
                    // Cheapest first: a value that does not reach the LOWEST of the 32 bounds reaches none (5 shuffles and
                    // no per-point shuffle; collapsed components, hopeless for all points of most tiles, end here).
                    float lbmin = lb_own;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) lbmin = fminf(lbmin, __shfl_xor_sync(0xffffffffu, lbmin, o));
                    bool maybe = false;
                    if (flagged) {
                        const float cut = lbmin - reach;
#pragma unroll
                        for (int j = 0; j < 32; ++j) maybe |= l[j] >= cut;
                    }
                    if (__any_sync(0xffffffffu, maybe)) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float lbj = __shfl_sync(0xffffffffu, lb_own, j);
                            if (flagged && j < nvalid && l[j] + reach >= lbj) mlo |= 1u << j;
                        }
                    }
                    // For a component that is narrow in a few dimensions only, E is in the thousands and almost every pair
                    // passes that test.  Such pairs are then tested exactly: c_k minus the terms of the component's 8
                    // dimensions of largest weight is an upper bound of its log2 z, whatever the other dimensions add.  The
                    // warp takes one flagged component at a time, lane j testing point j; the coordinates are read from
                    // the tile's fp16 planes in shared memory.
                    unsigned fl = tight ? __ballot_sync(0xffffffffu, mlo != 0u) : 0u;
                    if (fl) {
                        // (the planes were written by TMA: observing the stage's barrier makes them visible to these loads)
                        bar_wait(BAR(B_YFULL0 + s), ph, abort_flag, p.status, false);
                        const unsigned char* ystage = smem + SM_Y + s * SM_YSTAGE;
                        while (fl) {
                            const int f = __ffs(fl) - 1;
                            fl &= fl - 1;
                            const int kf = (int)rank * 128 + wq * 32 + f;
                            const unsigned maskf = __shfl_sync(0xffffffffu, mlo, f);
                            float ub = __ldg(p.c2 + kf);
#pragma unroll
                            for (int q8 = 0; q8 < 8; ++q8) {
                                const int d = __ldg(p.dec_dim + kf * 8 + q8);
                                const float x = y_scaled_x(ystage, p0 + lane, d);
                                // (coordinates are clamped to +-240 when the planes are built: such a one proves nothing)
                                const float w = (fabsf(x) < 239.f) ? __ldg(p.dec_w + kf * 8 + q8) : 0.f;
                                const float diff = x - __ldg(p.dec_mu + kf * 8 + q8);
                                ub -= w * diff * diff;
                            }
                            // 8: rounding of the 22-bit coordinates
                            const bool keep = ((maskf >> lane) & 1u) && !(ub < lb_own - ILL_MARGIN - 8.f);
                            const unsigned km = __ballot_sync(0xffffffffu, keep);
                            if (lane == f) mlo = km;
                        }
                    }
                }
                // publish AFTER the filter: peers read these slots only for the rare pairs that survive their own filter,
                // and a global store in flight makes the next warp-level barrier wait for it
                xslot_write(ring + (rank * 4 + wq) * 64 + lane, lb_own, 0.f, tag);
                if (emax_w > 0.f) {
                    const int kglob = (int)rank * 128 + kloc;
                    bool fixed_any = false;
                    uint32_t exact_mask = 0;                                 // points of this lane's component recomputed exactly
                    // Second filter, against the GROUP-wide lower bound of each point (the maximum of the bounds that all
                    // 4 CL warps of the group published).  That bound depends on the point only, so it is fetched once per
                    // point that has candidates - four points per L2 round trip, lane c reading the slot of
                    // (CTA c / 4, warp c % 4) - and not once per candidate pair: with half of the components flagged
                    // (small N / K) two thousand pairs per tile pass the warp-local filter and a handful survive this one.
                    // (at large N / K almost no tile has a candidate at all: one ballot decides, and the rest is skipped)
                    const bool have_cand = __ballot_sync(0xffffffffu, mlo != 0u) != 0u;
                    uint32_t pm = have_cand ? __reduce_or_sync(0xffffffffu, mlo) : 0u;       // points with at least one candidate
                    float lb_keep = CUDART_INF_F;                            // lane j keeps the group bound of point j
                    while (pm != 0u && alive) {
                        int jb[4];
                        uint32_t rest = pm;
#pragma unroll
                        for (int b8 = 0; b8 < 4; ++b8) {
                            jb[b8] = rest ? (__ffs(rest) - 1) : -1;
                            if (rest) rest &= rest - 1;
                        }
                        float lbv[4];
                        unsigned long long t0 = 0;
                        for (int it = 0;; ++it) {
                            bool ok = true;
#pragma unroll
                            for (int b8 = 0; b8 < 4; ++b8) {
                                lbv[b8] = -CUDART_INF_F;
                                if (jb[b8] >= 0 && lane < 4 * p.CL) {
                                    uint32_t v[4];
                                    xslot_load(ring + lane * 64 + jb[b8], v);
                                    if (v[1] == tag && v[3] == tag) lbv[b8] = __uint_as_float(v[0]);
                                    else ok = false;
                                }
                                if (BIG && jb[b8] >= 0) ok = xslot_more_bounds(ring + jb[b8], 4 * p.CL, tag, lane, lbv[b8]) && ok;
                            }
                            if (__all_sync(0xffffffffu, ok)) break;
                            bool give_up = *abort_flag != 0;
                            if ((it & 15) == 15) {
                                const unsigned long long now = gtime();
                                if (t0 == 0) t0 = now;
                                else if (now - t0 > WAIT_LIMIT_NS) {
                                    *abort_flag = 1;
                                    atomicOr(p.status, ST_TIMEOUT);
                                    give_up = true;
                                }
                            }
                            if (__any_sync(0xffffffffu, give_up)) { alive = false; break; }
                        }
                        if (!alive) break;
#pragma unroll
                        for (int b8 = 0; b8 < 4; ++b8) {
                            if (jb[b8] < 0) continue;                       // uniform: jb is the same in every lane
                            float m = lbv[b8];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                            if (lane == jb[b8]) lb_keep = m;
                        }
                        pm = rest;
                    }
                    if (have_cand && alive) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float lbj = __shfl_sync(0xffffffffu, lb_keep, j);
                            if (((mlo >> j) & 1u) && !(l[j] + illb >= lbj - ILL_MARGIN)) mlo &= ~(1u << j);
                        }
                    } else {
                        mlo = 0u;
                    }
                    // The survivors are recomputed exactly with direct differences in fp32, the whole warp on one pair.
                    while (have_cand) {
                        const uint32_t ballot = __ballot_sync(0xffffffffu, mlo != 0u);
                        if (ballot == 0u) break;
                        const int src = __ffs(ballot) - 1;
                        int j = __ffs(mlo) - 1;
                        j = __shfl_sync(0xffffffffu, j, src);
                        const int kk = __shfl_sync(0xffffffffu, kglob, src);
                        const float* xr = p.X + (xrow0 + p0 + j) * p.D;
                        const float* mr = p.mu + (size_t)kk * p.D;
                        const float* wr = p.w2 + (size_t)kk * p.D;
                        float q = 0.f;
                        for (int d = lane; d < p.D; d += 32) {
                            const float diff = __ldg(xr + d) - __ldg(mr + d);
                            q = fmaf(diff * diff, __ldg(wr + d), q);
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
                        const float val = __ldg(p.c2 + kk) - q;
                        if (lane == src) {
#pragma unroll
                            for (int jj = 0; jj < 32; ++jj)
                                if (jj == j) l[jj] = val;
                            mlo &= ~(1u << j);
                            exact_mask |= 1u << j;
                        }
                        fixed_any = true;
                    }
                    // Tight mode: the approximate value of a flagged component is never used: a pair that was not recomputed has been
                    // shown to lie 2^-40 below the point's best value (and its approximation may be off by thousands, in
                    // either direction), so it takes no further part.
                    if (tight && illb > 0.f) {
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj)
                            if (!((exact_mask >> jj) & 1u)) l[jj] = -CUDART_INF_F;
                    }
                    __syncwarp();
                    if (fixed_any) warp_reduce_scatter32<true>(l, red, lane);      // maxima with the corrected logits
                }
            }
            // all-gather the warp maxima through shared memory
            gather[lane] = red;
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                const float4 m4 = *reinterpret_cast<const float4*>(gather + j);
                const float m0 = (m4.x == -CUDART_INF_F) ? 0.f : m4.x;
                const float m1 = (m4.y == -CUDART_INF_F) ? 0.f : m4.y;
                const float m2 = (m4.z == -CUDART_INF_F) ? 0.f : m4.z;
                const float m3 = (m4.w == -CUDART_INF_F) ? 0.f : m4.w;
                l[j] = fast_ex2(l[j] - m0);
                l[j + 1] = fast_ex2(l[j + 1] - m1);
                l[j + 2] = fast_ex2(l[j + 2] - m2);
                l[j + 3] = fast_ex2(l[j + 3] - m3);
            }
            __syncwarp();
            float sred;
            warp_reduce_scatter32<false>(l, sred, lane);
            ws[wq * 32 + lane] = make_float2(red, sred);
            named_bar_sync(1 + 2 * grp, 128);
            if (gtid < 32) {
                const int pt = gtid;
                float2 w4[4];
#pragma unroll
                for (int w = 0; w < 4; ++w) w4[w] = ws[w * 32 + pt];
                float mc = fmaxf(fmaxf(w4[0].x, w4[1].x), fmaxf(w4[2].x, w4[3].x));
                const float mc_safe = (mc == -CUDART_INF_F) ? 0.f : mc;
                float sc = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w)       // a warp whose lanes are all padded / zero-weight has m_w = -inf: skip it
                    sc += (w4[w].x == -CUDART_INF_F) ? 0.f : w4[w].y * fast_ex2(w4[w].x - mc_safe);
                // publish (m, s) of this CTA's 128 components, then collect the group's
                const uint32_t tag = (uint32_t)(i + 1);
                XSlot* ring = xg + (size_t)(i & 3) * p.CL * 64 + p0 + pt;
                // (test hook: one CTA stays silent for the first tile, so that its peers' bounded waits run out)
                if (!(p.test_silent_rank == (int)rank && cluster_id == 0 && i == 0)) xslot_write(ring + rank * 64, mc, sc, tag);
                float mi = -CUDART_INF_F, mi_safe = 0.f, Z = 0.f;
                if (!BIG) {
                    float2 e[8];
                    if (!xslot_wait_all(ring, p.CL, tag, e, abort_flag, p.status)) alive = false;
#pragma unroll
                    for (int c = 0; c < 8; ++c) mi = fmaxf(mi, e[c].x);
                    mi_safe = (mi == -CUDART_INF_F) ? 0.f : mi;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        Z += (e[c].x == -CUDART_INF_F) ? 0.f : e[c].y * fast_ex2(e[c].x - mi_safe);
                } else {
                    if (!xslot_collect_many(ring, p.CL, tag, mi, Z, abort_flag, p.status)) alive = false;
                    mi_safe = (mi == -CUDART_INF_F) ? 0.f : mi;
                }
                const bool valid = pt < nvalid;
                const float inv = (valid && Z > 0.f) ? __fdividef(RSCALE, Z) : 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w)
                    fac[w * 32 + pt] = (w4[w].x == -CUDART_INF_F) ? 0.f : fast_ex2(w4[w].x - mi_safe) * inv;
                ll_have = rank == 0 && valid;
                ll_m = mi; ll_z = Z;
            }
            if (gtid == 0) decision_s[grp] = *abort_flag;
            named_bar_sync(2 + 2 * grp, 128);
            if (decision_s[grp]) break;
            // responsibilities: r = p * fac, split into fp16 hi + lo, written over the logits as the M-step A operand
            {
                uint32_t hi[16], lo[16];
                const float* fw = fac + wq * 32;
                float nsum = 0.f;
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 f4 = *reinterpret_cast<const float4*>(fw + j);
                    const float r0 = l[j] * f4.x, r1 = l[j + 1] * f4.y, r2 = l[j + 2] * f4.z, r3 = l[j + 3] * f4.w;
                    const __half2 h01 = __floats2half2_rn(r0, r1), h23 = __floats2half2_rn(r2, r3);
                    const float2 b01 = __half22float2(h01), b23 = __half22float2(h23);
                    const __half2 g01 = __floats2half2_rn(r0 - b01.x, r1 - b01.y), g23 = __floats2half2_rn(r2 - b23.x, r3 - b23.y);
                    const float2 c01 = __half22float2(g01), c23 = __half22float2(g23);
                    // N_k must be the sum of exactly the weights the M-step uses (hi + lo): responsibilities too small for
                    // fp16 vanish from S1 and S2, and a dying component whose N_k still counted them would get mu = S1 / N_k
                    // pulled toward zero instead of staying a weighted mean
                    nsum += ((b01.x + c01.x) + (b01.y + c01.y)) + ((b23.x + c23.x) + (b23.y + c23.y));
                    hi[j / 2] = *reinterpret_cast<const uint32_t*>(&h01);
                    hi[j / 2 + 1] = *reinterpret_cast<const uint32_t*>(&h23);
                    lo[j / 2] = *reinterpret_cast<const uint32_t*>(&g01);
                    lo[j / 2 + 1] = *reinterpret_cast<const uint32_t*>(&g23);
                }
                nk_acc += nsum;
                // each group overwrites only the 32 columns its own logits came from: [r_hi (16) | r_lo (16)]
                tmem_st16(T_LOG + s * 64 + p0 + lane_addr, hi);
                tmem_st16(T_LOG + s * 64 + p0 + 16 + lane_addr, lo);
                tmem_wait_st();
            }
            fence_before();
            bar_arrive(BAR(B_RREADY0 + s));
            if (gtid < 32 && ll_have) {              // two-sum: (ll_s, ll_c) += log2 Z_i exactly to fp32 pair precision
                const float v = ll_m + log2f(ll_z);
                const float t = ll_s + v;
                const float bp = t - ll_s;
                ll_c += (ll_s - (t - bp)) + (v - bp);
                ll_s = t;
            }

            // periodic flush of the TMEM accumulators into float64 partials, by group 1, after the second tile of a pair
            // (or the last tile); the flush index (hence the barrier parity) follows from the tile index alone
            const bool pair_end = (i & 1) || (i + 1 == ntl);
            const int64_t pair_next = (i | 1) + 1;
            if (grp == 1 && pair_end && ((pair_next % p.flush) == 0 || pair_next >= ntl)) {
                const uint32_t fpar = (uint32_t)(((pair_next - 1) / p.flush) & 1);
                if (!bar_wait(BAR(B_ACCFULL), fpar, abort_flag, p.status, false)) alive = false;
                fence_after();
#pragma unroll 1
                for (int c0 = 0; c0 < 256; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(T_ACC + lane_addr + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) atomicAdd(prow + (size_t)(c0 + j) * pstride, (double)__uint_as_float(v[j]));
                }
                fence_before();
                bar_arrive(BAR(B_ACCFREE));
            }
            // N_k of this group's points has its own column
            if (((i + 1) % 64) == 0 || i + 1 >= ntl) {
                atomicAdd(prow + (size_t)(256 + grp) * pstride, (double)nk_acc);
                nk_acc = 0.f;
            }
        }
        if (rank == 0) {
            double* lls = reinterpret_cast<double*>(smem + SM_LL) + grp * 32;
            if (gtid < 32) lls[gtid] = (double)ll_s + (double)ll_c;
            named_bar_sync(5 + grp, 128);
            if (gtid == 0) {
                double sum = 0.0;
                for (int j = 0; j < 32; ++j) sum += lls[j];
                p.llpart[cluster_id * 2 + grp] += sum * 0.69314718055994530942;      // one owner per slot: launches add up
            }
        }
    } else if (warp == PRODUCER_WARP) {
        // =========================== producer warp: Y planes -> shared memory by TMA ===========================
        // The fp16 planes of Y = [s x | (s x)^2 + kap] were written once for all CTAs by tc_transform_kernel; a stage is
        // 2 planes x 4 atoms of (64 points x 128 bytes): one 3-D box per plane, and TMA's 128-byte swizzle produces exactly
        // the K-major layout the MMA descriptors describe.  The whole warp runs the loop; lane 0 waits, one elected lane issues.
        const int n_atoms = (p.n_ks + 3) >> 2;
        const uint32_t stage_bytes = (uint32_t)n_atoms * 2u * 8192u;
        int64_t issued = 0;
        bool ok = true;
        for (int64_t i = 0; i < ntl && ok; ++i) {
            const int s = (int)(i & 1);
            const uint32_t ph = (uint32_t)((i >> 1) & 1);
            const int32_t row0 = (int32_t)((cluster_id + i * p.Q) * BN);
            if (i >= 2) {
                uint32_t w = 1;
                if (lane == 0) w = bar_wait(BAR(B_YEMPTY0 + s), ph ^ 1, abort_flag, p.status, false) ? 1u : 0u;
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w) { ok = false; break; }
            }
            if (elect_one()) {
                const uint32_t bar = BAR(B_YFULL0 + s);
                const uint32_t dst = smem_u32(smem + SM_Y + s * SM_YSTAGE);
                bar_expect_tx(bar, stage_bytes);
                tma_load_3d(dst, &tm_hi, 0, row0, 0, bar);                 // box = (128 bytes, 64 points, n_atoms atoms)
                tma_load_3d(dst + SM_YLO, &tm_lo, 0, row0, 0, bar);
                // The planes were written by another kernel and are larger than L2: ask for the tile this CTA will load
                // two steps from now (the next one is already in flight for the other stage); one CTA of the group asks
                // for all, in turn.
                if (i + 2 < ntl && (int)(i % p.CL) == (int)rank) {
                    const int32_t rown = (int32_t)((cluster_id + (i + 2) * p.Q) * BN);
                    tma_prefetch_3d(&tm_hi, 0, rown, 0);
                    tma_prefetch_3d(&tm_lo, 0, rown, 0);
                }
            }
            __syncwarp();
            issued = i + 1;
        }
        // On an abort the consumer may never wait for the last loads: they must have landed before the CTA may exit.
        if (!ok || *abort_flag) {
            for (int64_t i = (issued > 2 ? issued - 2 : 0); i < issued; ++i) {
                if (lane == 0) bar_wait(BAR(B_YFULL0 + (int)(i & 1)), (uint32_t)((i >> 1) & 1), drain_flag, p.status, false);
                __syncwarp();
            }
        }
    } else {
        // =========================== MMA warp ===========================
        // The whole warp runs this loop convergently; lane 0 does the (bounded) waits and broadcasts their outcome, one
        // elected lane issues the MMAs and commits, and the warp meets again after every batch.
        const uint32_t id_e = make_idesc(128, BN, 0);
        const uint32_t id_m = make_idesc(128, p.n_ks * 16, 1);
        const int n_ks = p.n_ks;
        // Descriptors are hoisted bases plus compile-time offsets (address field, 16-byte units): the issuing thread must
        // spend only a few instructions per MMA or it, not the tensor pipe, sets the pace.
        const uint64_t d_plo = make_desc(smem_u32(smem + SM_PLO), 16, 1024);
        const uint32_t y0 = smem_u32(smem + SM_Y);
        bool acc_valid = false;
        uint32_t accfree_parity = 0;
        bool alive = true;
        auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
            uint32_t ok = 1;
            if (lane == 0) ok = bar_wait(bar, parity, abort_flag, p.status, false) ? 1u : 0u;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            fence_after();
            return ok != 0u;
        };
        auto issue_E = [&](int64_t i, bool seen = false) -> bool {
            const int s = (int)(i & 1);
            const uint32_t ph = (uint32_t)((i >> 1) & 1);
            if (!seen && !wait_all(BAR(B_YFULL0 + s), ph)) return false;
            if (elect_one()) {
                const uint32_t d = T_LOG + s * 64;
                const uint64_t dyh = make_desc(y0 + s * SM_YSTAGE, 16, 1024);            // K-major views of the stage
                const uint64_t dyl = make_desc(y0 + s * SM_YSTAGE + SM_YLO, 16, 1024);
                // The two small cross products go first: the accumulator truncates (toward zero) at every add, by up to
                // one ulp of its CURRENT magnitude, so they are added while it is still small.
#pragma unroll
                for (int ks = 0; ks < 16; ++ks)
                    if (ks < n_ks) mma_ss(d, d_plo + (((ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                                          dyh + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), id_e, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 16; ++ks)
                    if (ks < n_ks) mma_ts(d, T_PHI + ks * 8, dyl + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), id_e, 1);
#pragma unroll
                for (int ks = 0; ks < 16; ++ks)
                    if (ks < n_ks) mma_ts(d, T_PHI + ks * 8, dyh + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), id_e, 1);
                mma_commit(BAR(B_LFULL0 + s));
            }
            __syncwarp();
            return true;
        };
        auto issue_M = [&](int64_t i, bool seen = false) -> bool {
            const int s = (int)(i & 1);
            const uint32_t ph = (uint32_t)((i >> 1) & 1);
            if (!seen && !wait_all(BAR(B_RREADY0 + s), ph)) return false;
            if (elect_one()) {
                // A operand layout in the logits buffer: points 0-31 -> columns [0,16) r_hi, [16,32) r_lo; points 32-63 -> +32
                const uint32_t rbase = T_LOG + s * 64;
                const uint64_t dyh = make_desc(y0 + s * SM_YSTAGE, 8192, 1024);          // MN-major views of the stage
                const uint64_t dyl = make_desc(y0 + s * SM_YSTAGE + SM_YLO, 8192, 1024);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks)
                    mma_ts(T_ACC, rbase + (ks >> 1) * 32 + (ks & 1) * 8, dyh + ((ks * 2048) >> 4), id_m, (acc_valid || ks > 0) ? 1u : 0u);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks)
                    mma_ts(T_ACC, rbase + (ks >> 1) * 32 + (ks & 1) * 8, dyl + ((ks * 2048) >> 4), id_m, 1);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks)
                    mma_ts(T_ACC, rbase + (ks >> 1) * 32 + (ks & 1) * 8 + 16, dyh + ((ks * 2048) >> 4), id_m, 1);
                mma_commit(BAR(B_YEMPTY0 + s));
            }
            __syncwarp();
            acc_valid = true;
            return true;
        };
        // Hands the TMEM accumulators to the flushing softmax group and waits until they are free again.
        auto flush_acc = [&]() -> bool {
            if (elect_one()) mma_commit(BAR(B_ACCFULL));
            __syncwarp();
            if (!wait_all(BAR(B_ACCFREE), accfree_parity)) return false;
            accfree_parity ^= 1;
            acc_valid = false;
            return true;
        };
        if ((p.order & 3) == 2) {
            // Dynamic order: E(j) needs its Y stage (and M(j-2) issued, which frees that stage and logits buffer), M(i)
            // needs the responsibilities of tile i; the two are independent, so whichever is ready first is issued.
            // With a fixed order the warp sat in the wait for the refill of E(i+2)'s stage while M(i+1) was ready.
            int64_t next_e = 0, next_m = 0;
            unsigned long long t0 = 0;
            int spins = 0;
            while (next_m < ntl && alive) {
                uint32_t act = 0;                                   // 1: E(next_e)   2: M(next_m)   3: give up
                if (lane == 0) {
                    if (next_e < ntl && next_e < next_m + 2 &&
                        bar_test(BAR(B_YFULL0 + (int)(next_e & 1)), (uint32_t)((next_e >> 1) & 1))) act = 1;
                    else if (next_m < next_e && bar_test(BAR(B_RREADY0 + (int)(next_m & 1)), (uint32_t)((next_m >> 1) & 1))) act = 2;
                    else if (*abort_flag) act = 3;
                    else if ((++spins & 63) == 0) {
                        const unsigned long long now = gtime();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > WAIT_LIMIT_NS) {
                            *abort_flag = 1;
                            atomicOr(p.status, ST_TIMEOUT);
                            act = 3;
                        }
                    }
                }
                act = __shfl_sync(0xffffffffu, act, 0);
                if (act == 0) continue;
                if (act == 3) { alive = false; break; }
                t0 = 0; spins = 0;
                fence_after();
                if (act == 1) {
                    alive = issue_E(next_e, true);
                    ++next_e;
                } else {
                    const int64_t i = next_m;
                    alive = issue_M(i, true);
                    ++next_m;
                    const bool pair_end = (i & 1) || (i + 1 == ntl);
                    const int64_t pair_next = (i | 1) + 1;
                    if (alive && pair_end && ((pair_next % p.flush) == 0 || pair_next >= ntl)) alive = flush_acc();
                }
            }
        } else if ((p.order & 1) == 0) {
            // Issue order per pair of tiles: E(a) E(b) M(a) M(b).
            for (int64_t i = 0; i < ntl && alive; i += 2) {
                const bool has2 = i + 1 < ntl;
                alive = issue_E(i);
                if (alive && has2) alive = issue_E(i + 1);
                if (alive) alive = issue_M(i);
                if (alive && has2) alive = issue_M(i + 1);
                if (!alive) break;
                const int64_t pair_next = i + 2;
                if ((pair_next % p.flush) == 0 || pair_next >= ntl) alive = flush_acc();
            }
        } else {
            // Interleaved order E(0) E(1) | M(0) E(2) | M(1) E(3) | ...: M(i) must precede E(i+2) (two logits buffers, two
            // Y stages); the softmax of tile i+1 overlaps E(i+2).
            if (ntl > 0) alive = issue_E(0);
            if (alive && ntl > 1) alive = issue_E(1);
            for (int64_t i = 0; i < ntl && alive; ++i) {
                alive = issue_M(i);
                if (!alive) break;
                const bool pair_end = (i & 1) || (i + 1 == ntl);
                const int64_t pair_next = (i | 1) + 1;
                if (pair_end && ((pair_next % p.flush) == 0 || pair_next >= ntl)) {
                    alive = flush_acc();
                    if (!alive) break;
                }
                if (i + 2 < ntl) alive = issue_E(i + 2);
            }
        }
        // drain: every MMA issued by this warp has completed before TMEM is released
        if (elect_one()) mma_commit(BAR(B_FINAL));
        __syncwarp();
        if (lane == 0) bar_wait(BAR(B_FINAL), 0, drain_flag, p.status, false);      // also after an abort
        __syncwarp();
        fence_after();
    }

    // teardown: everybody meets, peers are done with this CTA's shared memory, TMEM is released
    fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------------
// X -> the two fp16 planes of Y, once per launch of the tile kernel (the CTAs of a group all read the same tiles, so
// converting inside the tile kernel repeated this work in every CTA and took issue slots from the softmax warps).
// Row i of a plane holds 256 halves: k-step ks (8 dimensions) occupies halves [16 ks, 16 ks + 8) = s x and
// [16 ks + 8, 16 ks + 16) = (s x)^2 + kap, i.e. the column order of the E-step contraction.  One thread converts one
// (point, k-step) unit and writes 32 contiguous bytes per plane; 16 consecutive threads write one 512-byte row.
// Rows n .. rows_padded - 1 are written as zeros so that the last tile's loads need no out-of-bounds handling.
__device__ __forceinline__ void tc_load_unit(const float* __restrict__ X, int64_t n, int D, bool vec_ok, int64_t u, int64_t units,
                                             float (&x)[8]) {
    const int64_t row = u >> 4;
    const int d0 = (int)(u & 15) * 8;
    if (u < units && row < n && vec_ok && d0 + 8 <= D) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(X + row * D + d0));
        const float4 b = __ldg(reinterpret_cast<const float4*>(X + row * D + d0 + 4));
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = (u < units && row < n && d0 + j < D) ? __ldg(X + row * D + d0 + j) : 0.f;
    }
}

__device__ __forceinline__ void tc_store_unit(const float (&x)[8], bool valid, const float* __restrict__ sd,
                                              const float* __restrict__ kap, const float* __restrict__ gd, int64_t u,
                                              unsigned char* __restrict__ yhi, unsigned char* __restrict__ ylo) {
    const int64_t row = u >> 4;
    const int ks = (int)(u & 15), d0 = ks * 8;
    // (the per-dimension constants in 16-byte loads: the arrays hold 128 entries and start on 256-byte boundaries)
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
        // centred and scaled: u = s_d (x - g_d)  (padded dimensions: s = 1, g = 0, x = 0)
        float u0 = (x[j] - gv[j]) * sv[j], u1 = (x[j + 1] - gv[j + 1]) * sv[j + 1];
        if (!valid) { u0 = 0.f; u1 = 0.f; }
        u0 = fminf(fmaxf(u0, -240.f), 240.f);
        u1 = fminf(fmaxf(u1, -240.f), 240.f);
        float q0 = fmaf(u0, u0, kv[j]), q1 = fmaf(u1, u1, kv[j + 1]);
        if (!valid) { q0 = 0.f; q1 = 0.f; }
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
    uint4* oh = reinterpret_cast<uint4*>(yhi + row * 512 + ks * 32);
    uint4* ol = reinterpret_cast<uint4*>(ylo + row * 512 + ks * 32);
    oh[0] = make_uint4(xh[0], xh[1], xh[2], xh[3]);
    oh[1] = make_uint4(qh[0], qh[1], qh[2], qh[3]);
    ol[0] = make_uint4(xl[0], xl[1], xl[2], xl[3]);
    ol[1] = make_uint4(ql[0], ql[1], ql[2], ql[3]);
}

__global__ void __launch_bounds__(256) tc_transform_kernel(const float* __restrict__ X, int64_t n, int64_t rows_padded, int D,
                                                           const float* __restrict__ sd, const float* __restrict__ kap,
                                                           const float* __restrict__ gd,
                                                           unsigned char* __restrict__ yhi, unsigned char* __restrict__ ylo,
                                                           int* __restrict__ status) {
    const bool vec_ok = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15) == 0);
    const int64_t units = rows_padded * 16;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool bad = false;
    // two units per step, both loads issued before the first store: twice the bytes in flight per thread
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += 2 * stride) {
        float xa[8], xb[8];
        tc_load_unit(X, n, D, vec_ok, u, units, xa);
        tc_load_unit(X, n, D, vec_ok, u + stride, units, xb);
        // (the planes clamp every coordinate to a finite range, so a NaN or an infinity in X has to be caught here)
#pragma unroll
        for (int j = 0; j < 8; ++j) bad |= !(fabsf(xa[j]) <= 3.0e38f) || !(fabsf(xb[j]) <= 3.0e38f);
        tc_store_unit(xa, (u >> 4) < n, sd, kap, gd, u, yhi, ylo);
        if (u + stride < units) tc_store_unit(xb, ((u + stride) >> 4) < n, sd, kap, gd, u + stride, yhi, ylo);
    }
    if (bad) atomicOr(status, ST_BAD_X);
}

// The same planes for a grouped launch: row r of the planes belongs to tile t = r / BN and holds point
// tile_src[t] + (r mod BN) of X if (r mod BN) < tile_valid[t], zeros otherwise.
__global__ void __launch_bounds__(256) tc_transform_grouped_kernel(const float* __restrict__ X, int64_t rows, int D,
                                                                   const int* __restrict__ tile_valid,
                                                                   const int64_t* __restrict__ tile_src,
                                                                   const float* __restrict__ sd, const float* __restrict__ kap,
                                                                   const float* __restrict__ gd,
                                                                   unsigned char* __restrict__ yhi, unsigned char* __restrict__ ylo,
                                                                   int* __restrict__ status) {
    const int64_t units = rows * 16;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += stride) {
        const int64_t row = u >> 4;
        const int64_t t = row / BN;
        const int j = (int)(row - t * BN);
        const bool valid = j < __ldg(tile_valid + t);
        const float* xr = X + (valid ? (__ldg(tile_src + t) + j) * D : 0);
        const int d0 = (int)(u & 15) * 8;
        float x[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            x[q] = (valid && d0 + q < D) ? __ldg(xr + d0 + q) : 0.f;
            bad |= !(fabsf(x[q]) <= 3.0e38f);
        }
        tc_store_unit(x, valid, sd, kap, gd, u, yhi, ylo);
    }
    if (bad) atomicOr(status, ST_BAD_X);
}

// ---------------------------------------------------------------------------------------------------------------
// Parameter preparation for the tensor path (float64 arithmetic, K*D elements: negligible)

// (All means below are taken about the per-dimension centre g_d, see the kernel.)
// s_d = 2^-round(log2 rms_d) with rms_d^2 = sum_k pi_k (mu_kd^2 + var_kd): brings every dimension to O(1) so that the
// fp16 splits keep their precision whatever the data's units.  kap_d = s_d^2 sum_k pi_k mu_kd^2: the squares enter the
// contraction as (s x)^2 + kap_d, which turns the monotonically growing partial sums sum_d w (mu x - x^2 / 2) ~ sum_d w mu^2 / 2
// into a zero-mean walk sum_d w (mu^2 - kap) / 2 (several times smaller), and with it the error of the fp32 accumulation
// in the tensor core.  The constant is given back exactly through c_k (E-step) and kap_d N_k (M-step).
__global__ void __launch_bounds__(128) tc_scale_kernel(int D, int K, const float* __restrict__ pi, const float* __restrict__ mu,
                                                       const float* __restrict__ var, float* __restrict__ sd,
                                                       float* __restrict__ kap, float* __restrict__ gd) {
    // one block per dimension (padded to 128); threads stride over the components, fixed-shape tree reductions.
    // First the centre g_d = sum_k pi_k mu_kd / sum_k pi_k: points and means enter every product as x - g, mu - g, so that
    // data far from the origin (in units of its spread) costs the fp16 splits and the fp32 accumulators no precision; the
    // statistics are shifted back in float64 by the reduction.
    const int d = blockIdx.x, t = threadIdx.x;
    __shared__ double r_acc[128], r_m[128], r_w[128];
    __shared__ double g_s;
    double accg = 0.0, wsum = 0.0;
    if (d < D) {
        for (int k = t; k < K; k += 128) {
            const double w = (double)pi[k];
            accg += w * (double)mu[(size_t)k * D + d];
            wsum += w;
        }
    }
    r_acc[t] = accg; r_w[t] = wsum;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (t < o) { r_acc[t] += r_acc[t + o]; r_w[t] += r_w[t + o]; }
        __syncthreads();
    }
    if (t == 0) {
        double g = (r_w[0] > 0.0) ? r_acc[0] / r_w[0] : 0.0;
        const float gf = (float)g;                       // the kernels subtract the fp32 value: use exactly that one
        g_s = (d < D && isfinite(gf)) ? (double)gf : 0.0;
    }
    __syncthreads();
    const double g = g_s;
    double acc = 0.0, accm = 0.0;
    wsum = 0.0;
    if (d < D) {
        for (int k = t; k < K; k += 128) {
            const double w = (double)pi[k];
            const double m = (double)mu[(size_t)k * D + d] - g;
            acc += w * (m * m + (double)var[(size_t)k * D + d]);
            accm += w * m * m;
            wsum += w;
        }
    }
    __syncthreads();
    r_acc[t] = acc; r_m[t] = accm; r_w[t] = wsum;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (t < o) { r_acc[t] += r_acc[t + o]; r_m[t] += r_m[t + o]; r_w[t] += r_w[t + o]; }
        __syncthreads();
    }
    if (t == 0) {
        float s = 1.f, kp = 0.f;
        acc = r_acc[0]; accm = r_m[0]; wsum = r_w[0];
        if (wsum > 0.0) { acc /= wsum; accm /= wsum; }
        if (d < D && acc > 0.0 && isfinite(acc)) {
            const double e = rint(0.5 * log2(acc));
            s = (float)exp2(-fmin(fmax(e, -60.0), 60.0));
            kp = (float)(accm * (double)s * (double)s);      // mean of (mu - g)^2 in scaled units
        }
        sd[d] = s;
        kap[d] = kp;
        gd[d] = (float)g;
    }
}

// One block (128 threads) per padded component: builds the P_hi TMEM image, the P_lo shared-memory image, t_k, c_k,
// and flags ill-conditioned components.
__global__ void __launch_bounds__(128) tc_prepare_kernel(int D, int K, const float* __restrict__ pi,
                                                         const float* __restrict__ mu, const float* __restrict__ var,
                                                         const float* __restrict__ sd, const float* __restrict__ kap,
                                                         const float* __restrict__ gd, uint32_t* __restrict__ phi_img,
                                                         unsigned char* __restrict__ plo_img, float* __restrict__ tk,
                                                         float* __restrict__ ck, float* __restrict__ illb, float cond_limit,
                                                         int* __restrict__ flags, uint32_t* __restrict__ phi_rm,
                                                         uint32_t* __restrict__ plo_rm, float2* __restrict__ tkck) {
    const int k = blockIdx.x, d = threadIdx.x;
    const int slice = k >> 7, row = k & 127;
    __shared__ double red_max[128], red_c[128], red_cond[128], red_k[128];
    __shared__ __half hi_s[256], lo_s[256];
    double a = 0.0, b = 0.0, cterm = 0.0, cond = 0.0;
    const bool live = (k < K) && (d < D);
    if (live) {
        const double v = (double)var[(size_t)k * D + d], m = (double)mu[(size_t)k * D + d] - (double)gd[d], s = (double)sd[d];
        const double w = 1.4426950408889634074 / v;
        a = w * m / s;
        b = -0.5 * w / (s * s);
        cterm = m * m / v + log(6.283185307179586476925286766559 * v);
        cond = 0.5 * w * 3.0 * (m * m + 9.0 * v);
    }
    red_max[d] = fmax(fabs(a), fabs(b));
    red_c[d] = cterm;
    red_cond[d] = cond;
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (d < o) {
            red_max[d] = fmax(red_max[d], red_max[d + o]);
            red_c[d] += red_c[d + o];
            red_cond[d] += red_cond[d + o];
        }
        __syncthreads();
    }
    const double mx = red_max[0];
    double t = 1.0;
    if (mx > 0.0 && isfinite(mx)) t = exp2(floor(log2(mx)) - 9.0);      // max |P / t| in [512, 1024)
    const double as = a / t, bs = b / t;
    const __half ah = __double2half(as), bh = __double2half(bs);
    const __half al = __double2half(as - (double)__half2float(ah)), bl = __double2half(bs - (double)__half2float(bh));
    // interleaved column order: k-step ks = d / 8 holds [x(8 dims) | x^2(8 dims)]
    const int cx = 16 * (d >> 3) + (d & 7), cq = cx + 8;
    hi_s[cx] = ah; hi_s[cq] = bh; lo_s[cx] = al; lo_s[cq] = bl;
    // what the contraction adds through the shifted squares: t * (b_hi + b_lo) * kap, summed over d, is taken out of c_k.
    // So is the effect of the coefficients' own rounding (a, b are kept to 22 bits of the row's largest entry: an error
    // that is the same for every point, so nothing averages it out) AT THE COMPONENT'S MEAN: with ra, rb the residuals of
    // the split, the contraction misses t (ra u + rb (u^2 + kap)); its value at u = s (mu - g) goes into c_k, and what is
    // left is proportional to a point's distance from the mean, i.e. smaller by the component's |mu - g| / sigma.
    {
        const double bq = (double)__half2float(bh) + (double)__half2float(bl);
        const double ra = as - ((double)__half2float(ah) + (double)__half2float(al)), rb = bs - bq;
        double um = 0.0;
        if (live) um = ((double)mu[(size_t)k * D + d] - (double)gd[d]) * (double)sd[d];
        red_k[d] = live ? t * (bq * (double)kap[d] - (ra * um + rb * (um * um + (double)kap[d]))) : 0.0;
    }
    __syncthreads();
    for (int o = 64; o > 0; o >>= 1) {
        if (d < o) red_k[d] += red_k[d + o];
        __syncthreads();
    }
    // P_hi image: [slice][row][128] packed pairs (even column in the low half)
    phi_img[((size_t)slice * 128 + row) * 128 + d] =
        (uint32_t)__half_as_ushort(hi_s[2 * d]) | ((uint32_t)__half_as_ushort(hi_s[2 * d + 1]) << 16);
    // The same coefficients as two plain row-major planes [component][256 halves] (the B operand of the assignment kernel,
    // fetched by TMA, which applies the swizzle itself)
    phi_rm[(size_t)k * 128 + d] = (uint32_t)__half_as_ushort(hi_s[2 * d]) | ((uint32_t)__half_as_ushort(hi_s[2 * d + 1]) << 16);
    plo_rm[(size_t)k * 128 + d] = (uint32_t)__half_as_ushort(lo_s[2 * d]) | ((uint32_t)__half_as_ushort(lo_s[2 * d + 1]) << 16);
    // P_lo image: SW128 K-major, atoms of 64 columns, 128 rows
    for (int c = d; c < 256; c += 128) {
        const int atom = c >> 6, cc = c & 63;
        const size_t off = (size_t)slice * 65536 + atom * 16384 + row * 128 + ((((cc >> 3) ^ (row & 7)) << 4) | ((cc & 7) << 1));
        *reinterpret_cast<__half*>(plo_img + off) = lo_s[c];
    }
    if (d == 0) {
        float c = -CUDART_INF_F;
        if (k < K) {
            const float pk = pi[k];
            if (pk > 0.f) c = (float)(1.4426950408889634074 * (log((double)pk) - 0.5 * red_c[0]) - red_k[0]);
        }
        tk[k] = (float)t;
        ck[k] = c;

        // conditioning estimate of the expanded form: 2^-22 sum_d w2 * 3 (mu^2 + 9 var) ~ absolute log2 error bound
        const double cond = red_cond[0] * 2.384185791015625e-07;
        float margin = 0.f;
        if (k < K && cond > (double)cond_limit) {
            margin = (float)fmin(8.0 * cond, 1e30);       // E_k: error bound of the approximate log2 z (8 x the estimate)
            atomicOr(flags, 1);
            atomicAdd(flags + 4, 1);                      // how many: the tile kernel picks its filter by their share
        }
        illb[k] = margin;
        // For the assignment kernels: an ill-conditioned component takes no part in the approximate selection (constant
        // -inf; it is evaluated exactly for every point instead), and flags[1] = the largest error bound (8 x the estimate)
        // over the other components, as the bits of a non-negative float (their integer order is the order of the floats).
        tkck[k] = make_float2((float)t, margin > 0.f ? -CUDART_INF_F : c);
        if (k < K && margin == 0.f) {
            const float eb = (float)fmin(8.0 * cond, 1e30);
            if (eb > 0.f) atomicMax(flags + 1, __float_as_int(eb));
        }
    }
}

// One warp per ill-conditioned component (illb > 0): its 8 dimensions of largest weight, in descending order of the weight,
// in units of the centred, scaled data (the tile kernel reads s_d (x - g_d) from the fp16 planes): weight
// (log2 e / 2) / (var s_d^2), mean s_d (mu - g_d).  The tile kernel uses them for an exact upper bound of log2 z that costs a few shared-memory reads.
__global__ void __launch_bounds__(256) tc_decisive_kernel(int D, int K, const float* __restrict__ mu, const float* __restrict__ var,
                                                          const float* __restrict__ sd, const float* __restrict__ gd,
                                                          const float* __restrict__ illb, int* __restrict__ dec_dim, float* __restrict__ dec_w,
                                                          float* __restrict__ dec_mu) {
    const int k = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (k >= K || !(illb[k] > 0.f)) return;          // warp-uniform
    float wv[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int d = lane + 32 * j;
        wv[j] = -1.f;
        if (d < D) {
            const float sdd = sd[d];
            wv[j] = (0.72134752044448170368f / var[(size_t)k * D + d]) / (sdd * sdd);
            if (!(wv[j] >= 0.f) || !isfinite(wv[j])) wv[j] = 0.f;
        }
    }
    for (int r = 0; r < 8; ++r) {
        float bv = wv[0];
        int bd = lane;
#pragma unroll
        for (int j = 1; j < 4; ++j)
            if (wv[j] > bv) { bv = wv[j]; bd = lane + 32 * j; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int od = __shfl_xor_sync(0xffffffffu, bd, o);
            if (ov > bv || (ov == bv && od < bd)) { bv = ov; bd = od; }
        }
        if ((bd & 31) == lane) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (lane + 32 * j == bd) wv[j] = -1.f;          // taken
        }
        if (lane == 0) {
            const bool have = bv >= 0.f;
            dec_dim[k * 8 + r] = have ? bd : 0;
            dec_w[k * 8 + r] = have ? bv : 0.f;
            dec_mu[k * 8 + r] = have ? sd[bd] * (mu[(size_t)k * D + bd] - gd[bd]) : 0.f;
        }
    }
}

// Ascending list of the ill-conditioned components (illb > 0): flags[2] = their number, flags[3] = 1 when there are more
// than TC_MAX_ILL of them (the assignment then runs on the FP32 kernels).  One block of 1024 threads takes the components
// 1024 at a time.
__global__ void __launch_bounds__(1024) tc_ill_list_kernel(int Kpad, const float* __restrict__ illb, int* __restrict__ ill_list,
                                                           int* __restrict__ flags) {
    __shared__ int wcount[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int done = 0;                                    // listed so far (the same in every thread)
    for (int base = 0; base < Kpad; base += 1024) {
        const int k = base + threadIdx.x;
        const bool is = k < Kpad && illb[k] > 0.f;
        const unsigned b = __ballot_sync(0xffffffffu, is);
        __syncthreads();                             // the previous round's counts have been read
        if (lane == 0) wcount[w] = __popc(b);
        __syncthreads();
        int before = 0, total = 0;
        for (int j = 0; j < 32; ++j) {
            if (j < w) before += wcount[j];
            total += wcount[j];
        }
        if (is) ill_list[done + before + __popc(b & ((1u << lane) - 1u))] = k;
        done += total;
    }
    if (threadIdx.x == 0) { flags[2] = done; flags[3] = done > TC_MAX_ILL ? 1 : 0; }
}

// One thread per listed ill-conditioned component: its 8 dimensions of largest weight, in descending order of the weight.
__global__ void __launch_bounds__(TC_MAX_ILL) tc_ill_cache_kernel(int D, const float* __restrict__ mu, const float* __restrict__ w2,
                                                                  const float* __restrict__ c2, const int* __restrict__ ill_list,
                                                                  const int* __restrict__ flags, TcIllCache* __restrict__ out) {
    const int t = threadIdx.x;
    const int n_ill = flags[2] < TC_MAX_ILL ? flags[2] : TC_MAX_ILL;
    if (t >= n_ill) return;
    const int k = ill_list[t];
    float bw[8];
    int bd[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { bw[j] = -1.f; bd[j] = 0; }
    for (int d = 0; d < D; ++d) {
        const float w = w2[(size_t)k * D + d];
        if (w > bw[7]) {
            bw[7] = w; bd[7] = d;
#pragma unroll
            for (int j = 7; j > 0; --j) {
                if (bw[j] > bw[j - 1]) {
                    const float fw = bw[j]; bw[j] = bw[j - 1]; bw[j - 1] = fw;
                    const int fd = bd[j]; bd[j] = bd[j - 1]; bd[j - 1] = fd;
                }
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const bool have = bw[j] >= 0.f;                 // fewer than 8 dimensions: the slot weighs nothing
        out->dim[j][t] = bd[j];
        out->w[j][t] = have ? bw[j] : 0.f;
        out->mu[j][t] = have ? mu[(size_t)k * D + bd[j]] : 0.f;
    }
    out->c[t] = c2[k];
    out->k[t] = k;
}

// stats (+)= sum over Q cluster partials (float64, fixed order), undoing the responsibility scale, the per-dimension
// data scale and centre, and the interleaved column order.
__global__ void tc_reduce_kernel(int D, int K, int Kpad, int Q, const double* __restrict__ partial,
                                 const float* __restrict__ sd, const float* __restrict__ kap, const float* __restrict__ gd,
                                 double* __restrict__ Nk, double* __restrict__ S1, double* __restrict__ S2, int accumulate) {
    const size_t KD = (size_t)K * D, per = (size_t)K + 2 * KD;
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= per) return;
    const double unscale = 1.0 / (double)TC_RSCALE;
    auto column = [&](int col, int k) {                      // fixed order over the CTA groups
        double s = 0.0;
        for (int q = 0; q < Q; ++q) s += partial[((size_t)q * TC_PCOLS + col) * Kpad + k];
        return s;
    };
    if (e < (size_t)K) {
        const int k = (int)e;
        const double s = (column(256, k) + column(257, k)) * unscale;      // N_k of the two softmax groups
        Nk[e] = accumulate ? (Nk[e] + s) : s;
        return;
    }
    // The planes hold u = s_d (x - g_d) and u^2 + kap_d: the sums come back as S1c = sum r (x - g), S2c = sum r (x - g)^2,
    // then  S1 = S1c + g N_k,  S2 = S2c + 2 g S1c + g^2 N_k.
    const bool second = e >= K + KD;
    const size_t j = second ? (e - K - KD) : (e - K);
    const int k = (int)(j / D), d = (int)(j % D);
    const int col = 16 * (d >> 3) + (d & 7);
    const double s_d = (double)sd[d], g = (double)gd[d];
    const double nk_raw = column(256, k) + column(257, k);
    const double nk = nk_raw * unscale;
    const double s1c = column(col, k) * unscale / s_d;
    double out;
    if (!second) {
        out = s1c + g * nk;
    } else {
        const double s2c = (column(col + 8, k) - (double)kap[d] * nk_raw) * unscale / (s_d * s_d);
        out = s2c + 2.0 * g * s1c + g * g * nk;
    }
    double* dst = second ? (S2 + j) : (S1 + j);
    *dst = accumulate ? (*dst + out) : out;
}

// Fisher vectors of the groups of a grouped launch, straight from the per-CTA-group partials (group b of the launch =
// CTA group b): the statistics are unscaled as in tc_reduce_kernel, then
//   G_mu = (S1 - mu N_k) / (T sigma sqrt(pi)),  G_sigma = (S2 - 2 mu S1 + (mu^2 - var) N_k) / (T var sqrt(2 pi))
// in float64.  out_index[b] = which of the caller's groups it is, group_points[b] = its T.
__global__ void __launch_bounds__(256) tc_fisher_kernel(int D, int K, int Kpad, const double* __restrict__ partial,
                                                        const float* __restrict__ sd, const float* __restrict__ kap,
                                                        const float* __restrict__ gd,
                                                        const float* __restrict__ pi, const float* __restrict__ mu,
                                                        const float* __restrict__ var, const int* __restrict__ out_index,
                                                        const int64_t* __restrict__ group_points, float* __restrict__ fv) {
    // A block takes 32 components x 32 dimensions of one group.  The partials are [column][component] (component
    // fastest), the output is [component][dimension]: the 64 columns of the 32 dimensions (x and x^2 parts) and the two
    // N_k columns pass through shared memory, so that both the reads and the writes are contiguous per warp.
    __shared__ double tile[64][33];
    __shared__ double nk_s[32];
    const int k0 = blockIdx.x * 32, d0 = blockIdx.y * 32, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const double* pb = partial + (size_t)b * TC_PCOLS * Kpad;
    const bool kin = k0 + lane < Kpad;
    for (int c = warp; c < 64; c += 8) {
        const int d = d0 + (c & 31);                                   // c < 32: the x part, else the x^2 part
        const int col = 16 * (d >> 3) + (d & 7) + ((c >> 5) << 3);
        tile[c][lane] = (kin && d < 128) ? pb[(size_t)col * Kpad + k0 + lane] : 0.0;
    }
    if (warp == 0) nk_s[lane] = kin ? pb[(size_t)256 * Kpad + k0 + lane] + pb[(size_t)257 * Kpad + k0 + lane] : 0.0;
    __syncthreads();
    const int d = d0 + lane;
    if (d >= D) return;
    const size_t KD = (size_t)K * D;
    // The differences cancel and are formed in float64; the positive scale factors (1 / (T sigma sqrt(pi)) and
    // 1 / (T var sqrt(2 pi))) are formed in fp32, whose 1e-7 relative error goes straight into the result (float64
    // divisions and square roots per element would make this kernel arithmetic-bound).
    const double unscale = 1.0 / (double)TC_RSCALE;
    const double u1 = unscale / (double)sd[d], u2 = u1 / (double)sd[d], kp = (double)kap[d];
    const float inv_t = 1.0f / (float)group_points[b];
    float* out = fv + (size_t)out_index[b] * 2 * KD;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int kk = warp + 8 * j, k = k0 + kk;
        if (k >= K) continue;
        const double nk_raw = nk_s[kk];
        const double nk = nk_raw * unscale;
        const double s1 = tile[lane][kk] * u1;
        const double s2 = (tile[32 + lane][kk] - kp * nk_raw) * u2;
        const size_t e = (size_t)k * D + d;
        const float w = pi[k];
        float gm = 0.f, gs = 0.f;
        if (w > 0.f) {
            const float vf = var[e];
            // s1, s2 are moments of x - g: the vector depends on x - mu only, so the centred mean is used with them
            const double m = (double)mu[e] - (double)gd[d], v = (double)vf;
            gm = (float)(s1 - m * nk) * (inv_t * rsqrtf(vf) * rsqrtf(w));
            gs = (float)((s2 - 2.0 * m * s1) + (m * m - v) * nk) * (inv_t * rsqrtf(2.0f * w) / vf);
        }
        out[e] = gm;
        out[KD + e] = gs;
    }
}

}  // namespace

cudaError_t launch_fisher_tc(cudaStream_t s, int D, int K, int groups, const TcBuffers& tb, const float* pi, const float* mu,
                             const float* var, const int* out_index, const int64_t* group_points, float* fv) {
    const TcPlan pl = tc_plan(D, K, 148);
    tc_fisher_kernel<<<dim3((unsigned)((K + 31) / 32), (unsigned)((D + 31) / 32), (unsigned)groups), 256, 0, s>>>(
        D, K, pl.Kpad, tb.partial, tb.sd, tb.kap, tb.gd, pi, mu, var, out_index, group_points, fv);
    return cudaGetLastError();
}

cudaError_t launch_transform_grouped_tc(cudaStream_t s, const float* X, int64_t rows, int D, const int* tile_valid,
                                        const int64_t* tile_src, const TcBuffers& tb, int* status) {
    if (rows < 1 || rows > TC_YPOINTS || rows % TC_BN != 0) return cudaErrorInvalidValue;
    int64_t blocks = (rows * 16 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    tc_transform_grouped_kernel<<<(unsigned)blocks, 256, 0, s>>>(X, rows, D, tile_valid, tile_src, tb.sd, tb.kap, tb.gd, tb.y_hi, tb.y_lo, status);
    return cudaGetLastError();
}


int g_tc_order = 2;
// test hooks of the time-out path (see tc_set_test_hooks)
int g_tc_test_silent_rank = -1;
unsigned long long g_tc_wait_limit_ns = 2000000000ull, g_tc_wait_limit_set = 2000000000ull;
void tc_set_test_hooks(int silent_rank, unsigned long long wait_limit_ns) {
    g_tc_test_silent_rank = silent_rank;
    g_tc_wait_limit_ns = wait_limit_ns ? wait_limit_ns : 2000000000ull;
}
void tc_set_order(int o) { g_tc_order = o; }

bool tc_supports(int D, int K) { return D >= 1 && D <= 128 && K >= 1 && K <= TC_MAX_K; }
// The assignment kernels walk over the components in chunks of 128 inside one CTA: no group of CTAs, so K may be larger.
bool tc_assign_supports(int D, int K) { return D >= 1 && D <= 128 && K >= 1 && K <= TC_ASSIGN_MAX_K; }

TcPlan tc_plan(int D, int K, int num_sms) {
    TcPlan pl;
    pl.CL = (K + 127) / 128;
    pl.Kpad = pl.CL * 128;
    pl.Q = num_sms / pl.CL;
    if (pl.Q < 1) pl.Q = 1;
    pl.n_ks = (D + 7) / 8;
    return pl;
}

cudaError_t launch_prepare_tc(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                              const TcBuffers& tb, float cond_limit, int* status, bool ill_list) {
    const TcPlan pl = tc_plan(D, K, 148);
    (void)status;
    cudaError_t e0 = cudaMemsetAsync(tb.flags, 0, 8 * sizeof(int), s);
    if (e0 != cudaSuccess) return e0;
    tc_scale_kernel<<<128, 128, 0, s>>>(D, K, pi, mu, var, tb.sd, tb.kap, tb.gd);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tc_prepare_kernel<<<pl.Kpad, 128, 0, s>>>(D, K, pi, mu, var, tb.sd, tb.kap, tb.gd, tb.phi_img, tb.plo_img, tb.tk, tb.ck, tb.illb, cond_limit, tb.flags,
                                                  reinterpret_cast<uint32_t*>(tb.p_hi_rm), reinterpret_cast<uint32_t*>(tb.p_lo_rm),
                                                  reinterpret_cast<float2*>(tb.tkck));
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tc_decisive_kernel<<<(unsigned)((K + 7) / 8), 256, 0, s>>>(D, K, mu, var, tb.sd, tb.gd, tb.illb, tb.dec_dim, tb.dec_w, tb.dec_mu);
    e = cudaGetLastError();
    if (e != cudaSuccess || !ill_list) return e;
    tc_ill_list_kernel<<<1, 1024, 0, s>>>(pl.Kpad, tb.illb, tb.ill_list, tb.flags);
    return cudaGetLastError();
}

cudaError_t launch_ill_cache_tc(cudaStream_t s, int D, const float* mu, const float* w2, const float* c2, const TcBuffers& tb) {
    tc_ill_cache_kernel<<<1, TC_MAX_ILL, 0, s>>>(D, mu, w2, c2, tb.ill_list, tb.flags, tb.ill_cache);
    return cudaGetLastError();
}

cudaError_t launch_transform_tc(cudaStream_t s, const float* X, int64_t n, int D, const TcBuffers& tb, int* status) {
    if (n < 1 || n > TC_YPOINTS) return cudaErrorInvalidValue;
    const int64_t rows_padded = (n + TC_BN - 1) / TC_BN * TC_BN;
    const int64_t units = rows_padded * 16;
    int64_t blocks = (units + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    tc_transform_kernel<<<(unsigned)blocks, 256, 0, s>>>(X, n, rows_padded, D, tb.sd, tb.kap, tb.gd, tb.y_hi, tb.y_lo, status);
    return cudaGetLastError();
}

// A plane [rows][256 halves] seen as a 3-D tensor (x = 64 halves of an atom's row, y = row, z = atom): a box of
// (64, box_rows, box_atoms) lands in shared memory as [atom][row][128 bytes], each 128-byte row swizzled.
cudaError_t tc_make_plane_map(CUtensorMap* tm, void* base, int64_t rows, int box_rows, int box_atoms) {
    const cuuint64_t dims[3] = {64, (cuuint64_t)rows, 4};
    const cuuint64_t strides[2] = {512, 128};                 // bytes between rows, between atoms
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_atoms};
    const cuuint32_t estr[3] = {1, 1, 1};
    // The encoder lives in the driver library; it is looked up at run time so that this library has no load-time
    // dependency on the driver (it must load, e.g. for symbol checks, on a machine without one).
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

namespace {
cudaError_t set_smem_attr(bool big, bool tight) {
    if (big) return tight ? cudaFuncSetAttribute(em_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)
                          : cudaFuncSetAttribute(em_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    return tight ? cudaFuncSetAttribute(em_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)
                 : cudaFuncSetAttribute(em_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}
}  // namespace

cudaError_t launch_em_tc(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu, const float* w2,
                         const float* c2, const TcBuffers& tb, int Q, int flush_tiles, bool tight, int* status,
                         const int* tile_valid, const int64_t* tile_src) {
    const TcPlan pl = tc_plan(D, K, 148);
    const bool big = pl.CL > 8;
    TcKernelParams p;
    p.tile_valid = tile_valid; p.tile_src = tile_src;
    p.X = X; p.n = n; p.D = D; p.K = K; p.CL = pl.CL; p.Q = Q; p.n_ks = pl.n_ks;
    p.flush = (flush_tiles < 2) ? 2 : (flush_tiles & ~1);
    p.order = g_tc_order;
    p.test_silent_rank = g_tc_test_silent_rank;
    if (g_tc_wait_limit_ns != g_tc_wait_limit_set) {
        const cudaError_t ew = cudaMemcpyToSymbolAsync(c_wait_limit_ns, &g_tc_wait_limit_ns, sizeof(unsigned long long), 0,
                                                       cudaMemcpyHostToDevice, s);
        if (ew != cudaSuccess) return ew;
        g_tc_wait_limit_set = g_tc_wait_limit_ns;
    }
    p.phi_img = tb.phi_img; p.plo_img = tb.plo_img; p.tk = tb.tk; p.ck = tb.ck;
    p.illb = tb.illb; p.flags = tb.flags; p.mu = mu; p.w2 = w2; p.c2 = c2;
    p.dec_dim = tb.dec_dim; p.dec_w = tb.dec_w; p.dec_mu = tb.dec_mu;
    p.partial = tb.partial; p.llpart = tb.llpart; p.status = status;
    p.xg = static_cast<XSlot*>(tb.xg); p.xl = static_cast<XSlot*>(tb.xl);
    cudaError_t e = set_smem_attr(big, tight);
    if (e != cudaSuccess) return e;
    // exchange slots carry the tile number as their tag: clear what the previous launch left behind
    const size_t xbytes = (size_t)Q * 4 * pl.CL * 64 * sizeof(XSlot);
    e = cudaMemsetAsync(tb.xg, 0, xbytes, s);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(tb.xl, 0, 4 * xbytes, s);
    if (e != cudaSuccess) return e;
    // The CTAs of a group wait for one another, so all of them must be resident at once: a cooperative launch either
    // guarantees that or fails.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(Q * pl.CL));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (n < 1 || n > TC_YPOINTS) return cudaErrorInvalidValue;
    const int64_t rows_padded = (n + TC_BN - 1) / TC_BN * TC_BN;       // launch_transform_tc wrote zeros beyond n
    CUtensorMap tm_hi, tm_lo;
    const int n_atoms = (pl.n_ks + 3) / 4;
    e = tc_make_plane_map(&tm_hi, tb.y_hi, rows_padded, TC_BN, n_atoms);
    if (e != cudaSuccess) return e;
    e = tc_make_plane_map(&tm_lo, tb.y_lo, rows_padded, TC_BN, n_atoms);
    if (e != cudaSuccess) return e;
    if (big) return tight ? cudaLaunchKernelEx(&cfg, em_tc_kernel<true, true>, p, tm_hi, tm_lo) : cudaLaunchKernelEx(&cfg, em_tc_kernel<true, false>, p, tm_hi, tm_lo);
    return tight ? cudaLaunchKernelEx(&cfg, em_tc_kernel<false, true>, p, tm_hi, tm_lo) : cudaLaunchKernelEx(&cfg, em_tc_kernel<false, false>, p, tm_hi, tm_lo);
}

// Number of groups (of ceil(K/128) CTAs, one CTA per SM) that can be resident at once: the persistent grid size.
cudaError_t tc_max_clusters(int D, int K, int* out) {
    const TcPlan pl = tc_plan(D, K, 148);
    const bool big = pl.CL > 8;
    cudaError_t e = set_smem_attr(big, true);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0, per_sm = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    // (the same for every instantiation: one CTA per SM, by shared memory)
    e = big ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, em_tc_kernel<true, true>, NTHREADS, SMEM_BYTES)
            : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, em_tc_kernel<false, true>, NTHREADS, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    *out = (sms * per_sm) / pl.CL;
    return cudaSuccess;
}

cudaError_t launch_reduce_tc(cudaStream_t s, int D, int K, int Q, const TcBuffers& tb, double* Nk, double* S1,
                             double* S2, bool accumulate) {
    const TcPlan pl = tc_plan(D, K, 148);
    const size_t per = (size_t)K + 2 * (size_t)K * D;
    tc_reduce_kernel<<<(unsigned)((per + 255) / 256), 256, 0, s>>>(D, K, pl.Kpad, Q, tb.partial, tb.sd, tb.kap, tb.gd, Nk, S1, S2, accumulate ? 1 : 0);
    return cudaGetLastError();
}

}  // namespace fg
