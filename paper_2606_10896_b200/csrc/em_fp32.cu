// FP32 CUDA-core path: direct differences (x - mu)^2 / var, two phases per super-tile of points.
//
// Phase 1 (lse_kernel): for a tile of 64 points sweep all K components in blocks of 64, keep the running
//   (max, sum) of the online log-sum-exp per point on chip, write log Z_i (paper Algorithm 1, Step 1).
// Phase 2 (mstep_kernel): a CTA owns 64 components (and a 128-wide slice of D); for each of its point tiles it
//   recomputes log z_ik, forms r_ik = exp(log z_ik - log Z_i) in shared memory and accumulates N_k and the CENTRED
//   sums of r (x - g), r (x - g)^2 in registers across ALL its tiles (Algorithm 1, Step 2) -- the accumulators leave
//   the SM once, as a per-CTA partial; there are no atomics.  The reduction shifts them back to S1, S2 in float64.
// The arithmetic is in the log2 domain: w2 = (log2 e / 2) / var, c2 = log2 e * (log pi - 1/2 sum_d log(2 pi var)),
// log2 z = c2 - sum_d w2 (x - mu)^2, so the exponential is a bare ex2.  A term w2 (x - mu)^2 is formed as t^2 with
// t = (x - g) sqrt(w2) - (mu - g) sqrt(w2): one FMA for t (the second product is prepared when the tile is staged) and
// one for the sum, instead of a subtraction, a product and an FMA.  g is a per-dimension centre (the mean of the
// component means): with it both products are of the size of the data's spread, not of its distance from the origin, so
// the rounding of the prepared product stays as harmless as that of the direct difference.
#include "internal.cuh"
#include <math_constants.h>
#include <stdint.h>

namespace fg {

namespace {

constexpr int TP = FP32_TILE_P;
constexpr int TC = FP32_TILE_C;
constexpr int DCH = 32;       // dimensions staged per step
constexpr int LDT = 68;       // shared-memory row stride in floats (16-byte aligned rows, fewer store conflicts)
constexpr int NTHREADS = 256;

struct TileSmem {
    float xs[DCH][LDT];
    float ms[DCH][LDT];
    float ws[DCH][LDT];
};

__device__ __forceinline__ float fast_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// q[a][b] = sum_d w2[k0 + 4 tx + b][d] * (X[row0 + 4 ty + a][d] - mu[k0 + 4 tx + b][d])^2
// Rows >= n and components >= K are staged as zeros (w2 = 0 -> contributes nothing).  g: per-dimension centre (may be NULL = 0).
// ACC = float: one fp32 accumulation chain over D (D <= 128: a few 1e-6 of error).  ACC = double: each 32-dimension
// chunk is summed in fp32 and the chunk sums are added in float64, which keeps long chains (D = 768: |q| ~ 1000 in the
// log2 domain) from drowning the responsibilities in rounding noise.
// EARLY: cv[b] = constant of this thread's component b, fl[a] = a value below which log2 z of this thread's point a is
// negligible (a lower bound of the point's log2 Z minus 40).  The quadratic forms only grow with every chunk of
// dimensions, so once cv - q < fl for every pair of the tile the rest of the chunks cannot matter: the block leaves the
// loop together and the caller sees q = +inf (log2 z = -inf).  This is what makes a sub-mixture of collapsed components
// (hopeless for every point but their own) cost one chunk per tile instead of D / 32.
template <typename ACC, bool EARLY = false>
__device__ __forceinline__ void tile_quadratic(TileSmem& sm, const float* __restrict__ X, int64_t row0, int64_t n,
                                               int D, const float* __restrict__ mu, const float* __restrict__ w2,
                                               int k0, int K, ACC (&q)[4][4], const float* __restrict__ g,
                                               const int32_t* __restrict__ gather = nullptr, const ACC* cv = nullptr,
                                               const ACC* fl = nullptr) {
    constexpr bool HP = sizeof(ACC) == 8;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) q[a][b] = (ACC)0;
    // Staging: the tile's next 32 dimensions are fetched into registers (16-byte loads: eight consecutive threads read
    // 128 bytes of one row) while the current 32 are being computed from shared memory, so the load latency is hidden
    // behind the arithmetic instead of being exposed at every stage.
    const bool vec = (D % 4 == 0) && (((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(mu) |
                                        reinterpret_cast<uintptr_t>(w2) | reinterpret_cast<uintptr_t>(g)) & 15) == 0);
    float4 px[2], pm[2], pw[2], pg[2];
    auto fetch = [&](int d0) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int e4 = tid + j * NTHREADS, r = e4 >> 3, d = d0 + (e4 & 7) * 4;
            const int64_t slot = row0 + r;
            const int64_t row = (gather && slot < n) ? (int64_t)__ldg(gather + slot) : slot;     // gather: the tile's rows are X[gather[slot]], slot < n
            const int k = k0 + r;
            px[j] = pm[j] = pw[j] = pg[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (vec && d + 4 <= D) {
                if (g) pg[j] = __ldg(reinterpret_cast<const float4*>(g + d));
                if (slot < n) px[j] = __ldg(reinterpret_cast<const float4*>(X + row * D + d));
                if (k < K) {
                    pm[j] = __ldg(reinterpret_cast<const float4*>(mu + (size_t)k * D + d));
                    pw[j] = __ldg(reinterpret_cast<const float4*>(w2 + (size_t)k * D + d));
                }
            } else {
                float xv[4] = {0.f, 0.f, 0.f, 0.f}, mv[4] = {0.f, 0.f, 0.f, 0.f}, wv[4] = {0.f, 0.f, 0.f, 0.f};
                float gv[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    if (d + t < D) {
                        if (g) gv[t] = __ldg(g + d + t);
                        if (slot < n) xv[t] = __ldg(X + row * D + d + t);
                        if (k < K) {
                            mv[t] = __ldg(mu + (size_t)k * D + d + t);
                            wv[t] = __ldg(w2 + (size_t)k * D + d + t);
                        }
                    }
                px[j] = make_float4(xv[0], xv[1], xv[2], xv[3]);
                pm[j] = make_float4(mv[0], mv[1], mv[2], mv[3]);
                pw[j] = make_float4(wv[0], wv[1], wv[2], wv[3]);
                pg[j] = make_float4(gv[0], gv[1], gv[2], gv[3]);
            }
        }
    };
    fetch(0);
    for (int d0 = 0; d0 < D; d0 += DCH) {
        __syncthreads();
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int e4 = tid + j * NTHREADS, r = e4 >> 3, c = (e4 & 7) * 4;
            // staged: x - g, -(mu - g) sqrt(w), sqrt(w)   (zero weight for padded components: t = 0)
            const float sx = sqrtf(pw[j].x), sy = sqrtf(pw[j].y), sz = sqrtf(pw[j].z), sq = sqrtf(pw[j].w);
            sm.xs[c][r] = px[j].x - pg[j].x; sm.xs[c + 1][r] = px[j].y - pg[j].y;
            sm.xs[c + 2][r] = px[j].z - pg[j].z; sm.xs[c + 3][r] = px[j].w - pg[j].w;
            sm.ms[c][r] = (pg[j].x - pm[j].x) * sx; sm.ms[c + 1][r] = (pg[j].y - pm[j].y) * sy;
            sm.ms[c + 2][r] = (pg[j].z - pm[j].z) * sz; sm.ms[c + 3][r] = (pg[j].w - pm[j].w) * sq;
            sm.ws[c][r] = sx; sm.ws[c + 1][r] = sy; sm.ws[c + 2][r] = sz; sm.ws[c + 3][r] = sq;
        }
        __syncthreads();
        if (d0 + DCH < D) fetch(d0 + DCH);
        float part[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) part[a][b] = HP ? 0.f : (float)q[a][b];
#pragma unroll 8
        for (int c = 0; c < DCH; ++c) {
            const float4 xv = *reinterpret_cast<const float4*>(&sm.xs[c][4 * ty]);
            const float4 mv = *reinterpret_cast<const float4*>(&sm.ms[c][4 * tx]);
            const float4 wv = *reinterpret_cast<const float4*>(&sm.ws[c][4 * tx]);
            const float xa[4] = {xv.x, xv.y, xv.z, xv.w};
            const float mb[4] = {mv.x, mv.y, mv.z, mv.w};
            const float wb[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const float t = fmaf(xa[a], wb[b], mb[b]);
                    part[a][b] = fmaf(t, t, part[a][b]);
                }
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) q[a][b] = HP ? (ACC)(q[a][b] + (ACC)part[a][b]) : (ACC)part[a][b];
        if (EARLY && d0 + DCH < D) {
            bool live = false;
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) live |= (cv[b] - q[a][b] >= fl[a]);
            if (!__syncthreads_or(live ? 1 : 0)) {
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) q[a][b] = (ACC)CUDART_INF_F;
                return;
            }
        }
    }
}

template <int M, typename ACC>
struct TopList {
    ACC v[M];
    int i[M];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int j = 0; j < M; ++j) { v[j] = (ACC)(-CUDART_INF_F); i[j] = -1; }
    }
    // insert keeping descending order; equal values keep the earlier (smaller) index first
    __device__ __forceinline__ void insert(ACC val, int id) {
        if (i[M - 1] >= 0 && !(val > v[M - 1])) return;
        v[M - 1] = val; i[M - 1] = id;
#pragma unroll
        for (int j = M - 1; j > 0; --j) {
            const bool up = (i[j - 1] < 0) || (v[j] > v[j - 1]);
            if (up) {
                const ACC tv = v[j]; v[j] = v[j - 1]; v[j - 1] = tv;
                const int ti = i[j]; i[j] = i[j - 1]; i[j - 1] = ti;
            }
        }
    }
};

// M == 0: log-sum-exp only.  M > 0: also the top-M components per point.
// ACC is the type the logits are carried in: float for D <= 128, double beyond (see tile_quadratic).  The exponentials
// always take a float argument formed AFTER the subtraction of the reference, so large common offsets cancel exactly.
// One tile of TP points (tile number blk) of the log-sum-exp / top-m pass: see lse_kernel.
template <int M, typename ACC>
__device__ __forceinline__ void lse_tile(unsigned char* smem_raw, int64_t blk, const float* __restrict__ X, int64_t n, int D, int K,
                                         const float* __restrict__ mu, const float* __restrict__ w2, const double* __restrict__ c2,
                                         const float* __restrict__ g, double* __restrict__ logZ2, double* __restrict__ llpart,
                                         int m_out, int32_t* __restrict__ idx_out, float* __restrict__ resp_out,
                                         const int32_t* __restrict__ gather, const double* __restrict__ lower2 = nullptr) {
    TileSmem& sm = *reinterpret_cast<TileSmem*>(smem_raw);
    __shared__ double ll_s[TP];
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t row0 = blk * TP;
    const ACC NEG_INF = (ACC)(-CUDART_INF_F);

    ACC m_run[4];
    float s_run[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) { m_run[a] = NEG_INF; s_run[a] = 0.f; }
    TopList<(M > 0 ? M : 1), ACC> top[4];
    if (M > 0) {
#pragma unroll
        for (int a = 0; a < 4; ++a) top[a].init();
    }

    // lower2 (only with EARLY instantiations: M == 0, ACC = double): a lower bound of every point's final log2 Z, known
    // from elsewhere (the other components' log-sum-exp); terms more than 2^-40 below it are not evaluated to the end
    constexpr bool EARLY = (M == 0) && (sizeof(ACC) == 8);
    ACC fl[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int64_t row = row0 + 4 * ty + a;
        fl[a] = (EARLY && lower2) ? ((row < n) ? (ACC)(__ldg(lower2 + row) - 40.0) : (ACC)CUDART_INF_F) : NEG_INF;
    }
    for (int k0 = 0; k0 < K; k0 += TC) {
        ACC q[4][4];
        ACC cv[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int k = k0 + 4 * tx + b;
            cv[b] = (k < K) ? (ACC)__ldg(c2 + k) : NEG_INF;
        }
        if (EARLY && lower2) tile_quadratic<ACC, EARLY>(sm, X, row0, n, D, mu, w2, k0, K, q, g, gather, cv, fl);
        else tile_quadratic<ACC>(sm, X, row0, n, D, mu, w2, k0, K, q, g, gather);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            ACC l[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) l[b] = cv[b] - q[a][b];
            if (M > 0) {
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (k0 + 4 * tx + b < K) top[a].insert(l[b], k0 + 4 * tx + b);
            }
            ACC mloc = l[0] > l[1] ? l[0] : l[1];
            mloc = l[2] > mloc ? l[2] : mloc;
            mloc = l[3] > mloc ? l[3] : mloc;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) {
                const ACC other = __shfl_xor_sync(0xffffffffu, mloc, o);
                mloc = other > mloc ? other : mloc;
            }
            const ACC m_new = m_run[a] > mloc ? m_run[a] : mloc;
            const ACC m_safe = (m_new == NEG_INF) ? (ACC)0 : m_new;
            float sloc = fast_ex2((float)(l[0] - m_safe)) + fast_ex2((float)(l[1] - m_safe)) +
                         fast_ex2((float)(l[2] - m_safe)) + fast_ex2((float)(l[3] - m_safe));
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) sloc += __shfl_xor_sync(0xffffffffu, sloc, o);
            s_run[a] = s_run[a] * fast_ex2((float)(m_run[a] - m_safe)) + sloc;
            m_run[a] = m_new;
        }
    }

    double lz[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) lz[a] = (double)m_run[a] + (double)log2f(s_run[a]);
    if (tx == 0) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int64_t row = row0 + 4 * ty + a;
            const bool ok = row < n;
            if (ok && logZ2) logZ2[row] = lz[a];
            ll_s[4 * ty + a] = ok ? lz[a] * 0.69314718055994530942 : 0.0;
        }
    }
    if (M > 0) {
        // merge the 16 per-thread lists of each point through shared memory (reuses the staging area)
        __syncthreads();
        ACC* cand_v = reinterpret_cast<ACC*>(smem_raw);
        int* cand_i = reinterpret_cast<int*>(cand_v + TP * 16 * M);
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int j = 0; j < M; ++j) {
                const int slot = (4 * ty + a) * 16 * M + tx * M + j;
                cand_v[slot] = top[a].v[j];
                cand_i[slot] = top[a].i[j];
            }
        __shared__ double lz_s[TP];
        if (tx == 0) {
#pragma unroll
            for (int a = 0; a < 4; ++a) lz_s[4 * ty + a] = lz[a];
        }
        __syncthreads();
        if (tid < TP && row0 + tid < n) {
            ACC* cv = cand_v + tid * 16 * M;
            int* ci = cand_i + tid * 16 * M;
            const double lzp = lz_s[tid];
            const int64_t out_row = gather ? (int64_t)__ldg(gather + row0 + tid) : row0 + tid;
            for (int j = 0; j < m_out; ++j) {
                int best = -1;
                for (int s = 0; s < 16 * M; ++s) {
                    if (ci[s] < 0) continue;
                    if (best < 0 || cv[s] > cv[best] || (cv[s] == cv[best] && ci[s] < ci[best])) best = s;
                }
                int id = 0;
                float r = 0.f;
                if (best >= 0) {
                    id = ci[best];
                    r = fast_ex2((float)((double)cv[best] - lzp));
                    ci[best] = -1;
                }
                idx_out[out_row * m_out + j] = id;
                if (resp_out) resp_out[out_row * m_out + j] = r;
            }
        }
    }
    if (llpart) {
        __syncthreads();
        if (tid == 0) {
            double s = 0.0;
            for (int i = 0; i < TP; ++i) s += ll_s[i];
            llpart[blk] = s;
        }
    }
}

template <int M, typename ACC>
__global__ void __launch_bounds__(NTHREADS)
lse_kernel(const float* __restrict__ X, int64_t n, int D, int K, const float* __restrict__ mu,
           const float* __restrict__ w2, const double* __restrict__ c2, const float* __restrict__ g,
           double* __restrict__ logZ2, double* __restrict__ llpart, int m_out, int32_t* __restrict__ idx_out,
           float* __restrict__ resp_out, const int* __restrict__ run_if, const int32_t* __restrict__ gather,
           const int* __restrict__ gather_count, const double* __restrict__ lower2 = nullptr) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // run_if: the launch does nothing unless run_if[0] != 0 (the tensor-core assignment covers the other case)
    if (run_if && run_if[0] == 0) return;
    if (!gather) {                                   // one CTA per tile
        lse_tile<M, ACC>(smem_raw, blockIdx.x, X, n, D, K, mu, w2, c2, g, logZ2, llpart, m_out, idx_out, resp_out, nullptr, lower2);
        return;
    }
    // gather: the points are X[gather[0 .. *gather_count)] (top-m outputs go to those rows).  The count is only known on
    // the device, so the grid is fixed and small and its CTAs stride over the tiles of the list.
    const int64_t cnt = *gather_count;
    n = cnt < n ? cnt : n;
    for (int64_t blk = blockIdx.x; blk * TP < n; blk += gridDim.x) {
        lse_tile<M, ACC>(smem_raw, blk, X, n, D, K, mu, w2, c2, g, logZ2, llpart, m_out, idx_out, resp_out, gather);
        __syncthreads();                             // the next tile reuses the shared memory
    }
}

constexpr int LDR = TC + 4;                 // r tile row stride
constexpr int LDX = FP32_MSTEP_DC + 4;      // X tile row stride
constexpr size_t MSTEP_SMEM = sizeof(TileSmem) + (size_t)TP * LDR * 4 + (size_t)TP * LDX * 4;

template <typename ACC>
__global__ void __launch_bounds__(NTHREADS, sizeof(ACC) == 4 ? 2 : 1)      // float logits: two CTAs per SM
mstep_kernel(const float* __restrict__ X, int64_t n, int D, int K, const float* __restrict__ mu,
             const float* __restrict__ w2, const double* __restrict__ c2, const float* __restrict__ g,
             const double* __restrict__ logZ2, float* __restrict__ partials) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TileSmem& sm = *reinterpret_cast<TileSmem*>(smem_raw);
    float* r_s = reinterpret_cast<float*>(smem_raw + sizeof(TileSmem));     // [TP][LDR]
    float* xm = r_s + TP * LDR;                                              // [TP][LDX]
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int kq = tid >> 5, dq = tid & 31;
    const int k0 = blockIdx.x * TC;
    const int split = blockIdx.y, nsplits = gridDim.y;
    const int dz0 = blockIdx.z * FP32_MSTEP_DC;
    const int64_t ntiles = (n + TP - 1) / TP;

    float acc1[8][4], acc2[8][4];
#pragma unroll
    for (int c = 0; c < 8; ++c)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc1[c][j] = 0.f; acc2[c][j] = 0.f; }
    float nacc = 0.f;
    ACC cv[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int k = k0 + 4 * tx + b;
        cv[b] = (k < K) ? (ACC)__ldg(c2 + k) : (ACC)(-CUDART_INF_F);
    }

    for (int64_t t = split; t < ntiles; t += nsplits) {
        const int64_t row0 = t * TP;
        ACC q[4][4];
        tile_quadratic<ACC>(sm, X, row0, n, D, mu, w2, k0, K, q, g);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int64_t row = row0 + 4 * ty + a;
            const ACC lz = (row < n) ? (ACC)__ldg(logZ2 + row) : (ACC)CUDART_INF_F;    // +inf -> r = 0 for padded rows
            float4 rv;
            rv.x = fast_ex2((float)(cv[0] - q[a][0] - lz));
            rv.y = fast_ex2((float)(cv[1] - q[a][1] - lz));
            rv.z = fast_ex2((float)(cv[2] - q[a][2] - lz));
            rv.w = fast_ex2((float)(cv[3] - q[a][3] - lz));
            *reinterpret_cast<float4*>(&r_s[(4 * ty + a) * LDR + 4 * tx]) = rv;
        }
        // stage this CTA's D-slice of the X tile, row-major
#pragma unroll 4
        for (int j = 0; j < (TP * FP32_MSTEP_DC) / NTHREADS; ++j) {
            const int e = tid + j * NTHREADS, r = e >> 7, c = e & 127;
            const int64_t row = row0 + r;
            const int d = dz0 + c;
            // centred: the sums are taken of x - g and (x - g)^2 (the reduction shifts them back in float64), so that
            // fp32 accumulation errors scale with the data's spread, not with its distance from the origin
            xm[r * LDX + c] = (row < n && d < D) ? __ldg(X + row * D + d) - (g ? __ldg(g + d) : 0.f) : 0.f;
        }
        __syncthreads();
        if (tid < TC) {
            float s = 0.f;
#pragma unroll 8
            for (int i = 0; i < TP; ++i) s += r_s[i * LDR + tid];
            nacc += s;
        }
#pragma unroll 2
        for (int i = 0; i < TP; ++i) {
            const float4 xv = *reinterpret_cast<const float4*>(&xm[i * LDX + 4 * dq]);
            const float4 ra = *reinterpret_cast<const float4*>(&r_s[i * LDR + 8 * kq]);
            const float4 rb = *reinterpret_cast<const float4*>(&r_s[i * LDR + 8 * kq + 4]);
            const float x1[4] = {xv.x, xv.y, xv.z, xv.w};
            const float x2[4] = {xv.x * xv.x, xv.y * xv.y, xv.z * xv.z, xv.w * xv.w};
            const float rr[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
            for (int c = 0; c < 8; ++c)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc1[c][j] = fmaf(rr[c], x1[j], acc1[c][j]);
                    acc2[c][j] = fmaf(rr[c], x2[j], acc2[c][j]);
                }
        }
        // the next tile_quadratic starts with __syncthreads(), which also protects r_s / xm
    }

    const size_t KD = (size_t)K * D;
    float* pN = partials + (size_t)split * (K + 2 * KD);
    float* pS1 = pN + K;
    float* pS2 = pS1 + KD;
    if (blockIdx.z == 0 && tid < TC && k0 + tid < K) pN[k0 + tid] = nacc;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const int k = k0 + 8 * kq + c;
        if (k >= K) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int d = dz0 + 4 * dq + j;
            if (d < D) {
                pS1[(size_t)k * D + d] = acc1[c][j];
                pS2[(size_t)k * D + d] = acc2[c][j];
            }
        }
    }
}

// M-step for D > 128.  A CTA owns 64 components and ALL of D: it forms the responsibilities of a batch of WT point
// tiles once (full-D quadratic forms, float64 logits) and keeps them in shared memory, then sweeps the 128-wide slices
// of D, accumulating each slice over the whole batch in registers and adding it to this CTA's own rows of a float64
// partial in global memory (no other CTA touches them: deterministic, no atomics).  The E-step is thus recomputed once
// per point and component, not once per slice of D.
constexpr int WT = 3;
constexpr size_t MSTEP_WIDE_SMEM = sizeof(TileSmem) + (size_t)WT * TP * LDR * 4 + (size_t)TP * LDX * 4;

// EARLY: tiles none of whose (point, component) pairs can reach 2^-40 of the point's Z leave the quadratic form after the
// first chunks (see tile_quadratic); batches in which every responsibility is zero skip the sweep over D as well.
template <bool EARLY>
__global__ void __launch_bounds__(NTHREADS, 2)
mstep_wide_kernel(const float* __restrict__ X, int64_t n, int D, int K, const float* __restrict__ mu,
                  const float* __restrict__ w2, const double* __restrict__ c2, const float* __restrict__ g,
                  const double* __restrict__ logZ2, double* __restrict__ partials, const int* __restrict__ run_if) {
    if (run_if && run_if[0] == 0) return;          // gated launch: see lse_kernel
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TileSmem& sm = *reinterpret_cast<TileSmem*>(smem_raw);
    float* r_all = reinterpret_cast<float*>(smem_raw + sizeof(TileSmem));   // [WT][TP][LDR]
    float* xm = r_all + WT * TP * LDR;                                       // [TP][LDX]
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int kq = tid >> 5, dq = tid & 31;
    const int k0 = blockIdx.x * TC;
    const int split = blockIdx.y, nsplits = gridDim.y;
    const int64_t ntiles = (n + TP - 1) / TP;
    const int d_chunks = (D + FP32_MSTEP_DC - 1) / FP32_MSTEP_DC;
    const size_t KD = (size_t)K * D;
    double* pN = partials + (size_t)split * (K + 2 * KD);
    double* pS1 = pN + K;
    double* pS2 = pS1 + KD;

    double cv[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int k = k0 + 4 * tx + b;
        cv[b] = (k < K) ? __ldg(c2 + k) : (double)(-CUDART_INF_F);
    }
    double nacc = 0.0;

    for (int64_t t0 = split; t0 < ntiles; t0 += (int64_t)nsplits * WT) {
        // ---- responsibilities of the batch (tiles t0, t0 + nsplits, ...) ----
        int nb = 0;
        bool any_r = false;
        for (int w = 0; w < WT; ++w) {
            const int64_t t = t0 + (int64_t)w * nsplits;
            if (t >= ntiles) break;
            ++nb;
            const int64_t row0 = t * TP;
            double q[4][4];
            if (EARLY) {
                double fl[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const int64_t row = row0 + 4 * ty + a;
                    fl[a] = (row < n) ? __ldg(logZ2 + row) - 40.0 : (double)CUDART_INF_F;
                }
                tile_quadratic<double, true>(sm, X, row0, n, D, mu, w2, k0, K, q, g, nullptr, cv, fl);
            } else {
                tile_quadratic<double>(sm, X, row0, n, D, mu, w2, k0, K, q, g);
            }
            float* r_s = r_all + w * TP * LDR;
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int64_t row = row0 + 4 * ty + a;
                const double lz = (row < n) ? __ldg(logZ2 + row) : (double)CUDART_INF_F;
                float4 rv;
                rv.x = fast_ex2((float)(cv[0] - q[a][0] - lz));
                rv.y = fast_ex2((float)(cv[1] - q[a][1] - lz));
                rv.z = fast_ex2((float)(cv[2] - q[a][2] - lz));
                rv.w = fast_ex2((float)(cv[3] - q[a][3] - lz));
                any_r |= (rv.x > 0.f) || (rv.y > 0.f) || (rv.z > 0.f) || (rv.w > 0.f);
                *reinterpret_cast<float4*>(&r_s[(4 * ty + a) * LDR + 4 * tx]) = rv;
            }
        }
        if (EARLY) {
            if (!__syncthreads_or(any_r ? 1 : 0)) continue;          // nothing to accumulate from this batch
        } else {
            __syncthreads();
        }
        if (tid < TC) {
            float s = 0.f;
            for (int w = 0; w < nb; ++w)
                for (int i = 0; i < TP; ++i) s += r_all[(w * TP + i) * LDR + tid];
            nacc += (double)s;
        }
        // ---- sweep the slices of D ----
        for (int dz = 0; dz < d_chunks; ++dz) {
            const int dz0 = dz * FP32_MSTEP_DC;
            float acc1[8][4], acc2[8][4];
#pragma unroll
            for (int c = 0; c < 8; ++c)
#pragma unroll
                for (int j = 0; j < 4; ++j) { acc1[c][j] = 0.f; acc2[c][j] = 0.f; }
            for (int w = 0; w < nb; ++w) {
                const int64_t row0 = (t0 + (int64_t)w * nsplits) * TP;
                __syncthreads();
#pragma unroll 4
                for (int j = 0; j < (TP * FP32_MSTEP_DC) / NTHREADS; ++j) {
                    const int e = tid + j * NTHREADS, r = e >> 7, c = e & 127;
                    const int64_t row = row0 + r;
                    const int d = dz0 + c;
                    xm[r * LDX + c] = (row < n && d < D) ? __ldg(X + row * D + d) - (g ? __ldg(g + d) : 0.f) : 0.f;      // centred
                }
                __syncthreads();
                const float* r_s = r_all + w * TP * LDR;
#pragma unroll 2
                for (int i = 0; i < TP; ++i) {
                    const float4 xv = *reinterpret_cast<const float4*>(&xm[i * LDX + 4 * dq]);
                    const float4 ra = *reinterpret_cast<const float4*>(&r_s[i * LDR + 8 * kq]);
                    const float4 rb = *reinterpret_cast<const float4*>(&r_s[i * LDR + 8 * kq + 4]);
                    const float x1[4] = {xv.x, xv.y, xv.z, xv.w};
                    const float x2[4] = {xv.x * xv.x, xv.y * xv.y, xv.z * xv.z, xv.w * xv.w};
                    const float rr[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
                    for (int c = 0; c < 8; ++c)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            acc1[c][j] = fmaf(rr[c], x1[j], acc1[c][j]);
                            acc2[c][j] = fmaf(rr[c], x2[j], acc2[c][j]);
                        }
                }
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int k = k0 + 8 * kq + c;
                if (k >= K) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int d = dz0 + 4 * dq + j;
                    if (d < D) {
                        pS1[(size_t)k * D + d] += (double)acc1[c][j];
                        pS2[(size_t)k * D + d] += (double)acc2[c][j];
                    }
                }
            }
        }
        __syncthreads();      // r_all is rewritten by the next batch
    }
    if (tid < TC && k0 + tid < K) pN[k0 + tid] = nacc;
}

// One block per component: w2 = (log2 e / 2) / var, c2 = log2 e (log pi - 1/2 sum_d log(2 pi var)), in float64.
__global__ void prepare_fp32_kernel(int D, int K, const float* __restrict__ pi, const float* __restrict__ mu,
                                    const float* __restrict__ var, float* __restrict__ w2, float* __restrict__ c2,
                                    double* __restrict__ c2d, int* __restrict__ status, float* __restrict__ g_small) {
    const int k = blockIdx.x;
    // small problems (launch-bound): block 0 also forms the centre of the means, which saves a launch
    if (g_small && k == 0) {
        for (int d = threadIdx.x; d < D; d += blockDim.x) {
            double s = 0.0;
            for (int kk = 0; kk < K; ++kk) s += (double)mu[(size_t)kk * D + d];
            const float c = (float)(s / (double)K);
            g_small[d] = isfinite(c) ? c : 0.f;
        }
    }
    __shared__ double red[128];
    double s = 0.0;
    int bad = 0;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        const float v = var[(size_t)k * D + d];
        const float m = mu[(size_t)k * D + d];
        if (!(v > 0.f) || !isfinite(v)) bad |= ST_BAD_VAR;
        if (!isfinite(m)) bad |= ST_NONFINITE;
        const double vd = (double)v;
        s += log(6.283185307179586476925286766559 * vd);
        w2[(size_t)k * D + d] = (float)(0.72134752044448170368 / vd);
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = blockDim.x / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float p = pi[k];
        if (!(p >= 0.f) || !isfinite(p)) bad |= ST_BAD_PI;
        const double lp = (p > 0.f) ? log((double)p) : -CUDART_INF;
        const double cd = 1.4426950408889634074 * (lp - 0.5 * red[0]);
        c2[k] = (float)cd;
        c2d[k] = cd;
    }
    if (bad) atomicOr(status, bad);
}

// g[d] = mean over the components of mu[k][d]: the centre the tile routine subtracts from points and means.  A block takes
// 32 dimensions; its 32 warps sum every 32nd component in float64 and the 32 partial sums are added in a fixed order.  A
// non-finite mean (reported through the status word by prepare_fp32_kernel) gives centre 0.
__global__ void __launch_bounds__(1024) center_fp32_kernel(int D, int K, const float* __restrict__ mu, float* __restrict__ g) {
    __shared__ double part[32][33];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int d = blockIdx.x * 32 + lane;
    double s = 0.0;
    if (d < D)
        for (int k = w; k < K; k += 32) s += (double)mu[(size_t)k * D + d];
    part[w][lane] = s;
    __syncthreads();
    if (w == 0 && d < D) {
        double t = 0.0;
        for (int j = 0; j < 32; ++j) t += part[j][lane];
        const float c = (float)(t / (double)K);
        g[d] = isfinite(c) ? c : 0.f;
    }
}

}  // namespace

Fp32Plan fp32_plan(int D, int K) {
    Fp32Plan p;
    p.comp_blocks = (K + TC - 1) / TC;
    p.d_chunks = (D + FP32_MSTEP_DC - 1) / FP32_MSTEP_DC;
    p.wide = D > FP32_MSTEP_DC;
    // wide shapes: one CTA loops over the D slices itself (one resident CTA per SM: float64 logits are register-hungry)
    if (p.wide) {
        // Two resident CTAs per SM: pick the number of point splits whose grid fills whole waves of 296 CTAs best (a
        // grid of 1.3 waves leaves most SMs idle through the second one), among those whose float64 partials stay
        // within 256 MB.
        const size_t per_split = ((size_t)K + 2 * (size_t)K * D) * sizeof(double);
        int max_sp = (int)(((size_t)256 << 20) / per_split);
        if (max_sp < 1) max_sp = 1;
        if (max_sp > 296) max_sp = 296;
        int best = 1;
        double best_eff = 0.0;
        for (int sp = 1; sp <= max_sp; ++sp) {
            const int ctas = p.comp_blocks * sp;
            const int waves = (ctas + 295) / 296;
            const double eff = (double)ctas / (296.0 * waves);
            if (eff > best_eff + 1e-9) { best_eff = eff; best = sp; }
        }
        p.splits = best;
        return p;
    }
    const int per = p.comp_blocks * p.d_chunks;
    p.splits = (FP32_TARGET_CTAS + per - 1) / per;
    if (p.splits < 1) p.splits = 1;
    return p;
}

size_t fp32_partial_floats(int D, int K) {
    const Fp32Plan p = fp32_plan(D, K);
    // wide shapes keep float64 partials (they are accumulated into across batches of tiles)
    return (size_t)p.splits * ((size_t)K + 2 * (size_t)K * D) * (p.wide ? 2 : 1);
}

cudaError_t launch_center_fp32(cudaStream_t s, int D, int K, const float* mu, float* g) {
    center_fp32_kernel<<<(unsigned)((D + 31) / 32), 1024, 0, s>>>(D, K, mu, g);
    return cudaGetLastError();
}

cudaError_t launch_prepare_fp32(cudaStream_t s, int D, int K, const float* pi, const float* mu, const float* var,
                                float* w2, float* c2, double* c2d, float* g, int* status) {
    const bool small = g && (size_t)K * D <= ((size_t)1 << 12);
    prepare_fp32_kernel<<<K, 128, 0, s>>>(D, K, pi, mu, var, w2, c2, c2d, status, small ? g : nullptr);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || !g || small) return e;
    return launch_center_fp32(s, D, K, mu, g);
}

// Logits are carried in float64 when the accumulation over D is long.
static inline bool fp32_high_precision(int D) { return D > 128; }

cudaError_t launch_lse_fp32(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                            const float* w2, const double* c2d, const float* g, double* logZ2, double* llpart,
                            const double* lower2, const int* run_if) {
    const unsigned blocks = (unsigned)((n + TP - 1) / TP);
    if (fp32_high_precision(D))
        lse_kernel<0, double><<<blocks, NTHREADS, sizeof(TileSmem), s>>>(X, n, D, K, mu, w2, c2d, g, logZ2, llpart, 0, nullptr, nullptr, run_if, nullptr, nullptr, lower2);
    else
        lse_kernel<0, float><<<blocks, NTHREADS, sizeof(TileSmem), s>>>(X, n, D, K, mu, w2, c2d, g, logZ2, llpart, 0, nullptr, nullptr, run_if, nullptr, nullptr);
    return cudaGetLastError();
}

// Per-point log-density output of gmm_score_samples: log Z (natural log) from the base-2 values lse_kernel left.
static __global__ void logz_out_kernel(const double* __restrict__ logZ2, int64_t n, float* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = (float)(logZ2[i] * 0.69314718055994530942);
}

cudaError_t launch_logz_out_fp32(cudaStream_t s, const double* logZ2, int64_t n, float* out) {
    logz_out_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(logZ2, n, out);
    return cudaGetLastError();
}

template <int M, typename ACC>
static cudaError_t launch_topm_t(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                                 const float* w2, const double* c2d, const float* g, int m, int32_t* idx, float* resp,
                                 const int* run_if, const int32_t* gather, const int* gather_count) {
    size_t smem = sizeof(TileSmem);
    const size_t need = (size_t)TP * 16 * M * (sizeof(ACC) + 4);
    if (need > smem) smem = need;
    cudaError_t e = cudaFuncSetAttribute(lse_kernel<M, ACC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    unsigned blocks = (unsigned)((n + TP - 1) / TP);
    if (gather && blocks > 592) blocks = 592;          // the listed rows are few: at most 4 CTAs per SM stride over them
    lse_kernel<M, ACC><<<blocks, NTHREADS, smem, s>>>(X, n, D, K, mu, w2, c2d, g, nullptr, nullptr, m, idx, resp, run_if, gather, gather_count);
    return cudaGetLastError();
}

cudaError_t launch_topm_fp32(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                             const float* w2, const double* c2d, const float* g, int m, int32_t* idx, float* resp,
                             const int* run_if, const int32_t* gather, const int* gather_count) {
    if (fp32_high_precision(D)) {
        if (m <= 1) return launch_topm_t<1, double>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
        if (m <= 2) return launch_topm_t<2, double>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
        if (m <= 4) return launch_topm_t<4, double>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
        return launch_topm_t<8, double>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
    }
    if (m <= 1) return launch_topm_t<1, float>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
    if (m <= 2) return launch_topm_t<2, float>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
    if (m <= 4) return launch_topm_t<4, float>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
    return launch_topm_t<8, float>(s, X, n, D, K, mu, w2, c2d, g, m, idx, resp, run_if, gather, gather_count);
}

cudaError_t launch_mstep_fp32(cudaStream_t s, const float* X, int64_t n, int D, int K, const float* mu,
                              const float* w2, const double* c2d, const float* g, const double* logZ2, float* partials,
                              const Fp32Plan& plan, bool early, const int* run_if) {
    if (plan.wide) {
        cudaError_t e = early ? cudaFuncSetAttribute(mstep_wide_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MSTEP_WIDE_SMEM)
                              : cudaFuncSetAttribute(mstep_wide_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MSTEP_WIDE_SMEM);
        if (e != cudaSuccess) return e;
        const size_t bytes = (size_t)plan.splits * ((size_t)K + 2 * (size_t)K * D) * sizeof(double);
        e = cudaMemsetAsync(partials, 0, bytes, s);          // the kernel accumulates into its partials
        if (e != cudaSuccess) return e;
        dim3 wgrid(plan.comp_blocks, plan.splits, 1);
        if (early) mstep_wide_kernel<true><<<wgrid, NTHREADS, MSTEP_WIDE_SMEM, s>>>(X, n, D, K, mu, w2, c2d, g, logZ2, reinterpret_cast<double*>(partials), run_if);
        else mstep_wide_kernel<false><<<wgrid, NTHREADS, MSTEP_WIDE_SMEM, s>>>(X, n, D, K, mu, w2, c2d, g, logZ2, reinterpret_cast<double*>(partials), run_if);
        return cudaGetLastError();
    }
    dim3 grid(plan.comp_blocks, plan.splits, plan.d_chunks);
    if (fp32_high_precision(D)) {
        cudaError_t e = cudaFuncSetAttribute(mstep_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MSTEP_SMEM);
        if (e != cudaSuccess) return e;
        mstep_kernel<double><<<grid, NTHREADS, MSTEP_SMEM, s>>>(X, n, D, K, mu, w2, c2d, g, logZ2, partials);
    } else {
        cudaError_t e = cudaFuncSetAttribute(mstep_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MSTEP_SMEM);
        if (e != cudaSuccess) return e;
        mstep_kernel<float><<<grid, NTHREADS, MSTEP_SMEM, s>>>(X, n, D, K, mu, w2, c2d, g, logZ2, partials);
    }
    return cudaGetLastError();
}

}  // namespace fg
