// gmm_em_step_static: the E-step + sufficient statistics of gmm_em_step for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need an EM step: code running inside
// a memory-budgeted service whose device heap is owned by another allocator, a plugin invoked between a framework's
// own allocations where a driver allocation would synchronise the device, or a real-time loop that forbids any call
// that can block on the driver's allocator.  For them this file keeps ALL scratch of the FP32 kernel chain in one
// file-scope device array that is part of the loaded module: this file and the launch routines it calls make no
// allocation call.  (What the CUDA runtime itself does on the FIRST launch of a kernel -- loading its code into the
// device -- is outside this library's control: a warm-up call per device and per kernel variant, D <= 128 and
// D > 128, puts that behind the caller.  The cached device address of the array does not survive cudaDeviceReset.)
#include "internal.cuh"

#include <cmath>
#include <mutex>

using namespace fg;

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = (size_t)6 << 20;     // 6 MiB, held by every GPU that loads the library
constexpr int STATIC_MAX_K = 1024;
constexpr int64_t STATIC_MAX_KD = 32768;
constexpr int STATIC_MAX_SPLITS = 16;
constexpr int64_t STATIC_TILE = 1 << 16;                     // points per pass (log Z_i of one pass lives in scratch)
constexpr int MAX_DEVICES = 64;

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

struct StaticResult {
    double ll;
    int status;
    int pad;
};

struct StaticLayout {
    size_t w2, c2, c2d, center, logZ2, llpart, result, partials, total;
    int splits;
};

inline size_t al(size_t b) { return (b + 255) & ~(size_t)255; }

StaticLayout static_layout(int D, int K) {
    StaticLayout L;
    const size_t KD = (size_t)K * D;
    Fp32Plan plan = fp32_plan(D, K);
    const int max_splits = plan.wide ? STATIC_MAX_SPLITS / 2 : STATIC_MAX_SPLITS;   // float64 partials when wide
    L.splits = plan.splits < max_splits ? plan.splits : max_splits;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += al(bytes); return o; };
    L.w2 = take(KD * 4);
    L.c2 = take((size_t)K * 4);
    L.c2d = take((size_t)K * 8);
    L.center = take((size_t)D * 4);
    L.logZ2 = take((size_t)STATIC_TILE * 8);
    L.llpart = take((size_t)(STATIC_TILE / FP32_TILE_P) * 8);
    L.result = take(sizeof(StaticResult));
    L.partials = take((size_t)L.splits * ((size_t)K + 2 * KD) * (plan.wide ? 8 : 4));
    L.total = off;
    return L;
}

// Device address of g_static_scratch per device.  In host code the array's name is only a handle for the symbol,
// not a device address, so it is resolved once per device with cudaGetSymbolAddress while that device is current.
std::mutex g_mu;
unsigned char* g_base[MAX_DEVICES] = {nullptr};

cudaError_t scratch_base(int device, unsigned char** out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_base[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_base[device] = static_cast<unsigned char*>(p);
    }
    *out = g_base[device];
    return cudaSuccess;
}

}  // namespace

extern "C" int gmm_em_step_static(int device, void* cuda_stream, const float* X, int64_t N, int D, int K,
                                  const float* pi, const float* mu, const float* var, double* Nk, double* S1,
                                  double* S2, double* loglik) {
    if (!X || !pi || !mu || !var || !Nk || !S1 || !S2 || !loglik) return GMM_EINVAL;
    if (N < 1 || D < 1 || K < 1) return GMM_EINVAL;
    if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(pi) | reinterpret_cast<uintptr_t>(mu) |
         reinterpret_cast<uintptr_t>(var)) % 4)
        return GMM_EALIGN;
    if ((reinterpret_cast<uintptr_t>(Nk) | reinterpret_cast<uintptr_t>(S1) | reinterpret_cast<uintptr_t>(S2)) % 8)
        return GMM_EALIGN;
    if (K > STATIC_MAX_K || (int64_t)K * D > STATIC_MAX_KD) return GMM_EUNSUPPORTED;
    if (device < 0 || device >= MAX_DEVICES) return GMM_EINVAL;
    const StaticLayout L = static_layout(D, K);
    if (L.total > STATIC_SCRATCH_BYTES) return GMM_EUNSUPPORTED;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return GMM_ECUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return GMM_ECUDA;
    struct Restore {
        int prev, device;
        ~Restore() { if (prev != device) cudaSetDevice(prev); }
    } restore{prev, device};

    unsigned char* base = nullptr;
    if (scratch_base(device, &base) != cudaSuccess) return GMM_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    float* w2 = reinterpret_cast<float*>(base + L.w2);
    float* c2 = reinterpret_cast<float*>(base + L.c2);
    double* c2d = reinterpret_cast<double*>(base + L.c2d);
    float* center = reinterpret_cast<float*>(base + L.center);
    double* logZ2 = reinterpret_cast<double*>(base + L.logZ2);
    double* llpart = reinterpret_cast<double*>(base + L.llpart);
    StaticResult* res = reinterpret_cast<StaticResult*>(base + L.result);
    float* partials = reinterpret_cast<float*>(base + L.partials);
    Fp32Plan plan = fp32_plan(D, K);
    plan.splits = L.splits;

#define SCU(call) do { if ((call) != cudaSuccess) { cudaGetLastError(); return GMM_ECUDA; } } while (0)
    // The array keeps whatever the previous call left in it: clear everything that is accumulated into.
    const size_t KD = (size_t)K * D;
    SCU(cudaMemsetAsync(res, 0, sizeof(StaticResult), s));
    SCU(cudaMemsetAsync(Nk, 0, (size_t)K * 8, s));
    SCU(cudaMemsetAsync(S1, 0, KD * 8, s));
    SCU(cudaMemsetAsync(S2, 0, KD * 8, s));
    SCU(launch_prepare_fp32(s, D, K, pi, mu, var, w2, c2, c2d, center, &res->status));
    for (int64_t off = 0; off < N; off += STATIC_TILE) {
        const int64_t cnt = (N - off < STATIC_TILE) ? (N - off) : STATIC_TILE;
        const float* Xs = X + off * D;
        SCU(launch_lse_fp32(s, Xs, cnt, D, K, mu, w2, c2d, center, logZ2, llpart));
        SCU(launch_mstep_fp32(s, Xs, cnt, D, K, mu, w2, c2d, center, logZ2, partials, plan));
        SCU(launch_reduce_ll(s, llpart, (cnt + FP32_TILE_P - 1) / FP32_TILE_P, &res->ll, true));
        SCU(launch_reduce_partials(s, D, K, plan.splits, partials, center, Nk, S1, S2, true));
    }
    StaticResult h;
    SCU(cudaMemcpyAsync(&h, res, sizeof(StaticResult), cudaMemcpyDeviceToHost, s));
    SCU(cudaStreamSynchronize(s));
#undef SCU
    if (h.status & (ST_BAD_VAR | ST_BAD_PI | ST_NONFINITE)) return GMM_ENUMERIC;
    *loglik = h.ll;
    if (!std::isfinite(h.ll)) return GMM_ENUMERIC;
    return GMM_OK;
}
