// IVF posting lists from the top-m assignment (paper Sections 4.2 and 4.3).
//
// Rule: a vector is stored with its best cluster (Section 4.2) and with further clusters of its top-m list, up to
// max_lists in all (the paper uses two), while their responsibility is strictly greater than tau (tau = 1 / K in the
// paper: a cluster is taken only if seeing the vector raised its posterior above the uniform prior, Section 4.3).
// Output: CSR lists, offsets[K + 1] and the vectors of each list in ascending order.  Integer work, deterministic.
//
// The N vectors are cut into at most PL_MAX_BLOCKS contiguous ranges, one CTA each, so that the scratch (one counter per
// range and cluster) does not grow with N:
//   1. pl_count_kernel: entries per (range, cluster), counted in shared memory;
//   2. pl_totals_kernel / pl_scan_kernel / pl_block_offsets_kernel: list lengths, their exclusive prefix sum (= offsets)
//      and, per cluster, the running start of every range inside the list;
//   3. pl_fill_kernel: every CTA walks its range again IN ORDER, 256 vectors at a time, the eight warps of a step one
//      after the other; inside a warp every entry counts the entries of the same list that lower lanes hold, so every
//      list comes out ascending without a sort and without atomics.
#include "internal.cuh"

namespace fg {

namespace {

constexpr int PL_THREADS = 256;
constexpr int PL_MAX_LISTS = GMM_MAX_TOPM;      // at most this many lists per vector

__device__ __forceinline__ bool pl_take(int j, float r, float tau) { return j == 0 || r > tau; }

__global__ void __launch_bounds__(PL_THREADS)
pl_count_kernel(const int32_t* __restrict__ idx, const float* __restrict__ resp, int64_t n, int m, int K, float tau,
                int max_lists, int64_t range, int32_t* __restrict__ counts /* [blocks][K] */) {
    extern __shared__ int32_t hist[];
    for (int k = threadIdx.x; k < K; k += PL_THREADS) hist[k] = 0;
    __syncthreads();
    const int64_t i0 = (int64_t)blockIdx.x * range;
    const int64_t i1 = (i0 + range < n) ? (i0 + range) : n;
    for (int64_t i = i0 + threadIdx.x; i < i1; i += PL_THREADS) {
        for (int j = 0; j < max_lists; ++j) {
            const int32_t k = __ldg(idx + i * m + j);
            if (k < 0 || k >= K || !pl_take(j, __ldg(resp + i * m + j), tau)) break;
            atomicAdd(&hist[k], 1);                 // integer counts: the order of the additions does not matter
        }
    }
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += PL_THREADS) counts[(size_t)blockIdx.x * K + k] = hist[k];
}

__global__ void pl_totals_kernel(const int32_t* __restrict__ counts, int blocks, int K, int64_t* __restrict__ totals) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    int64_t s = 0;
    for (int b = 0; b < blocks; ++b) s += counts[(size_t)b * K + k];
    totals[k] = s;
}

// offsets = exclusive prefix sum of totals (one CTA, Hillis-Steele over chunks of 1024 with a running carry)
__global__ void __launch_bounds__(1024) pl_scan_kernel(const int64_t* __restrict__ totals, int K, int64_t* __restrict__ offsets) {
    __shared__ int64_t buf[1024];
    __shared__ int64_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < K; base += 1024) {
        const int k = base + threadIdx.x;
        const int64_t v = (k < K) ? totals[k] : 0;
        buf[threadIdx.x] = v;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            const int64_t add = (threadIdx.x >= o) ? buf[threadIdx.x - o] : 0;
            __syncthreads();
            buf[threadIdx.x] += add;
            __syncthreads();
        }
        if (k < K) offsets[k] = carry + buf[threadIdx.x] - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry += buf[1023];
        __syncthreads();
    }
    if (threadIdx.x == 0) offsets[K] = carry;
}

// counts[b][k] -> where range b starts inside list k (in place; int32 is enough: a list holds fewer than 2^31 vectors)
__global__ void pl_block_offsets_kernel(int32_t* __restrict__ counts, int blocks, int K) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    int32_t run = 0;
    for (int b = 0; b < blocks; ++b) {
        const int32_t c = counts[(size_t)b * K + k];
        counts[(size_t)b * K + k] = run;
        run += c;
    }
}

__global__ void __launch_bounds__(PL_THREADS)
pl_fill_kernel(const int32_t* __restrict__ idx, const float* __restrict__ resp, int64_t n, int m, int K, float tau,
               int max_lists, int64_t range, const int32_t* __restrict__ starts /* [blocks][K] */,
               const int64_t* __restrict__ offsets, int32_t* __restrict__ items) {
    extern __shared__ int32_t cursor[];                // next free position of this range inside every list
    for (int k = threadIdx.x; k < K; k += PL_THREADS) cursor[k] = starts[(size_t)blockIdx.x * K + k];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t i0 = (int64_t)blockIdx.x * range;
    const int64_t i1 = (i0 + range < n) ? (i0 + range) : n;
    for (int64_t base = i0; base < i1; base += PL_THREADS) {
        const int64_t i = base + threadIdx.x;
        // the warps take their 32 vectors one warp after the other, so that positions grow with the vector index
        for (int w = 0; w < PL_THREADS / 32; ++w) {
            if (warp == w) {
                // this lane's entries (clusters of its vector that pass the rule), -1 where there is none
                int32_t kk[PL_MAX_LISTS];
                bool more = i < i1;
#pragma unroll
                for (int j = 0; j < PL_MAX_LISTS; ++j) {
                    kk[j] = -1;
                    if (more && j < max_lists) {
                        const int32_t k = __ldg(idx + i * m + j);
                        if (k < 0 || k >= K || !pl_take(j, __ldg(resp + i * m + j), tau)) more = false;
                        else kk[j] = k;
                    }
                }
                // An entry's place inside its list: after the entries of the same list from LOWER lanes, whichever of
                // their choices it is (a first choice of vector i + 5 must not land before a second choice of i + 3).
                int rank[PL_MAX_LISTS], cnt[PL_MAX_LISTS];
#pragma unroll
                for (int j = 0; j < PL_MAX_LISTS; ++j) { rank[j] = 0; cnt[j] = 0; }
                for (int src = 0; src < 32; ++src) {
#pragma unroll
                    for (int j2 = 0; j2 < PL_MAX_LISTS; ++j2) {
                        if (j2 >= max_lists) break;                                 // uniform
                        const int32_t v = __shfl_sync(0xffffffffu, kk[j2], src);
                        if (v < 0) continue;                                        // uniform
#pragma unroll
                        for (int j = 0; j < PL_MAX_LISTS; ++j)
                            if (kk[j] == v) { ++cnt[j]; if (src < lane) ++rank[j]; }
                    }
                }
                // all entries of a list read its cursor, then the first of them moves it past the whole warp's entries
                int32_t pos[PL_MAX_LISTS];
#pragma unroll
                for (int j = 0; j < PL_MAX_LISTS; ++j) pos[j] = (kk[j] >= 0) ? cursor[kk[j]] : 0;
                __syncwarp();
#pragma unroll
                for (int j = 0; j < PL_MAX_LISTS; ++j)
                    if (kk[j] >= 0) {
                        items[offsets[kk[j]] + pos[j] + rank[j]] = (int32_t)i;
                        if (rank[j] == 0) cursor[kk[j]] = pos[j] + cnt[j];
                    }
                __syncwarp();
            }
            __syncthreads();
        }
    }
}

}  // namespace

int pl_blocks(int64_t n, int64_t* range_out) {
    int64_t range = (n + PL_MAX_BLOCKS - 1) / PL_MAX_BLOCKS;
    range = (range + PL_THREADS - 1) / PL_THREADS * PL_THREADS;        // whole steps of 256 vectors
    if (range < PL_THREADS) range = PL_THREADS;
    *range_out = range;
    return (int)((n + range - 1) / range);
}

size_t pl_scratch_bytes(int K) { return (size_t)PL_MAX_BLOCKS * K * sizeof(int32_t) + (size_t)(K + 1) * sizeof(int64_t); }

cudaError_t launch_posting_lists(cudaStream_t s, const int32_t* idx, const float* resp, int64_t n, int m, int K, float tau,
                                 int max_lists, void* scratch, int64_t* offsets, int32_t* items) {
    int64_t range = 0;
    const int blocks = pl_blocks(n, &range);
    int32_t* counts = static_cast<int32_t*>(scratch);
    int64_t* totals = reinterpret_cast<int64_t*>(static_cast<unsigned char*>(scratch) + (size_t)PL_MAX_BLOCKS * K * sizeof(int32_t));
    const size_t smem = (size_t)K * sizeof(int32_t);
    cudaError_t e = cudaFuncSetAttribute(pl_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(pl_fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    pl_count_kernel<<<blocks, PL_THREADS, smem, s>>>(idx, resp, n, m, K, tau, max_lists, range, counts);
    pl_totals_kernel<<<(K + 255) / 256, 256, 0, s>>>(counts, blocks, K, totals);
    pl_scan_kernel<<<1, 1024, 0, s>>>(totals, K, offsets);
    pl_block_offsets_kernel<<<(K + 255) / 256, 256, 0, s>>>(counts, blocks, K);
    pl_fill_kernel<<<blocks, PL_THREADS, smem, s>>>(idx, resp, n, m, K, tau, max_lists, range, counts, offsets, items);
    return cudaGetLastError();
}

}  // namespace fg
