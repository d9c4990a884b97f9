// co3_moments_static: the pooled moments of a = g + gamma m (the statistics the GenNorm fit is
// made from) computed without allocating anything.
//
// Who needs this.  Some callers of this library are not allowed to allocate device memory at the
// moment they need the statistics: code that runs inside a host application whose device memory is
// owned entirely by that application's own pool (a raw cudaMalloc there can fail, fragment the
// pool or be forbidden by policy), and latency-sensitive loops that cannot afford the
// device-wide synchronisation a cudaMalloc/cudaFree implies.  co3_plan_create allocates tens of
// megabytes of tables and scratch, so such callers cannot make a plan just to look at the moments
// of a gradient.  This entry point gives them the numbers with the inputs and outputs they
// already own.
//
// How.  The per-chunk partial sums that the regular path keeps in plan-owned scratch live here in
// a file-scope device array of fixed size (CO3_STATIC_MAX_ELEMENTS / 4096 slots of 24 bytes =
// 3 MiB; every GPU on which this library is loaded holds that much until the process exits).
// In host code the array's name is only a host-side handle, not a device address, so the address
// is asked from the runtime once per device with cudaGetSymbolAddress and passed to the kernels.
//
// Consequences the caller must know:
//  * The first call on each device performs that address look-up; make that first call before
//    any stream capture is started.
//  * All calls share the one array and it keeps whatever the previous call left in it.  Nothing in
//    it has to start at zero: each call writes every slot it later reads.  But two calls whose
//    kernels overlap on the GPU (different streams, or different host threads) race on the array;
//    serialise them.
//  * n above CO3_STATIC_MAX_ELEMENTS is refused with CO3_ELIMIT; nothing is launched.
#include <mutex>

#include "co3_internal.h"

namespace {

constexpr int STATIC_CHUNK = 4096;                       // elements per partial-sum slot
constexpr long long STATIC_SLOTS = CO3_STATIC_MAX_ELEMENTS / STATIC_CHUNK;
constexpr int STATIC_THREADS = 256;
constexpr int MAX_DEVICES = 64;

struct Partial {
    double s1, s2;
    unsigned long long nonfinite;
};

static __device__ __align__(256) Partial g_static_partials[STATIC_SLOTS];

// One block per chunk of 4096 elements: sum |a| and a^2 over the finite a = g + gamma m.
__global__ void __launch_bounds__(STATIC_THREADS)
static_partial_kernel(const float* __restrict__ g, const float* __restrict__ m, long long n, float gamma,
                      Partial* __restrict__ partials) {
    __shared__ double s_a[STATIC_THREADS / 32], s_b[STATIC_THREADS / 32];
    __shared__ unsigned long long s_n[STATIC_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long base = (long long)blockIdx.x * STATIC_CHUNK;
    double s1 = 0.0, s2 = 0.0;
    unsigned long long nf = 0;
#pragma unroll
    for (int r = 0; r < STATIC_CHUNK / (4 * STATIC_THREADS); ++r) {
        const long long e0 = base + 4LL * (tid + STATIC_THREADS * r);
        float gv[4] = {0.f, 0.f, 0.f, 0.f}, mv[4] = {0.f, 0.f, 0.f, 0.f};
        int cnt = 0;
        if (e0 + 4 <= n) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(g + e0));
            const float4 b = __ldg(reinterpret_cast<const float4*>(m + e0));
            gv[0] = a.x; gv[1] = a.y; gv[2] = a.z; gv[3] = a.w;
            mv[0] = b.x; mv[1] = b.y; mv[2] = b.z; mv[3] = b.w;
            cnt = 4;
        } else if (e0 < n) {                              // ragged tail of the array
            cnt = (int)(n - e0);
            for (int e = 0; e < cnt; ++e) { gv[e] = g[e0 + e]; mv[e] = m[e0 + e]; }
        }
        for (int e = 0; e < cnt; ++e) {
            const float a = __fadd_rn(gv[e], __fmul_rn(gamma, mv[e]));
            if ((__float_as_uint(a) & 0x7F800000u) == 0x7F800000u) { ++nf; continue; }
            const double ad = (double)fabsf(a);
            s1 += ad;
            s2 = __fma_rn(ad, ad, s2);                    // ad * ad is exact in double
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_down_sync(0xffffffffu, s1, o);
        s2 += __shfl_down_sync(0xffffffffu, s2, o);
        nf += __shfl_down_sync(0xffffffffu, nf, o);
    }
    if (lane == 0) { s_a[warp] = s1; s_b[warp] = s2; s_n[warp] = nf; }
    __syncthreads();
    if (tid == 0) {
        Partial p;
        p.s1 = 0.0; p.s2 = 0.0; p.nonfinite = 0;
        for (int w = 0; w < STATIC_THREADS / 32; ++w) { p.s1 += s_a[w]; p.s2 += s_b[w]; p.nonfinite += s_n[w]; }
        partials[blockIdx.x] = p;                         // every slot that is read later is written here
    }
}

// One block: add the chunk partials in a fixed order and write N, S1, S2, non-finite count.
__global__ void __launch_bounds__(1024)
static_final_kernel(const Partial* __restrict__ partials, long long n_slots, long long n, double* __restrict__ out) {
    __shared__ double s_a[1024], s_b[1024];
    __shared__ unsigned long long s_n[1024];
    const int tid = threadIdx.x;
    double s1 = 0.0, s2 = 0.0;
    unsigned long long nf = 0;
    for (long long k = tid; k < n_slots; k += 1024) {
        const Partial p = partials[k];
        s1 += p.s1; s2 += p.s2; nf += p.nonfinite;
    }
    s_a[tid] = s1; s_b[tid] = s2; s_n[tid] = nf;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (tid < o) { s_a[tid] += s_a[tid + o]; s_b[tid] += s_b[tid + o]; s_n[tid] += s_n[tid + o]; }
        __syncthreads();
    }
    if (tid == 0) {
        out[0] = (double)((unsigned long long)n - s_n[0]);
        out[1] = s_a[0];
        out[2] = s_b[0];
        out[3] = (double)s_n[0];
    }
}

std::mutex g_static_mu;
Partial* g_static_addr[MAX_DEVICES];                      // device address of the array, per device

// Device address of g_static_partials on the current device (looked up once per device).
int static_scratch(Partial** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { (void)cudaGetLastError(); return CO3_ECUDA; }
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_addr[dev]) {
        Partial* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_static_partials) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return CO3_ECUDA;
        }
        g_static_addr[dev] = ptr;
    }
    *out = g_static_addr[dev];
    return CO3_OK;
}

}  // namespace

extern "C" int co3_moments_static(const float* grad, const float* residual, int64_t n, float gamma,
                                  double* moments, void* cuda_stream) {
    if (!grad || !residual || !moments || n < 1) return CO3_EINVAL;
    if (((uintptr_t)grad | (uintptr_t)residual) & 15) return CO3_EINVAL;
    if (n > CO3_STATIC_MAX_ELEMENTS) return CO3_ELIMIT;   // would not fit the fixed scratch array
    Partial* scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc != CO3_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const long long n_slots = (n + STATIC_CHUNK - 1) / STATIC_CHUNK;
    static_partial_kernel<<<(unsigned)n_slots, STATIC_THREADS, 0, st>>>(grad, residual, (long long)n, gamma, scratch);
    if (cudaGetLastError() != cudaSuccess) return CO3_ECUDA;
    static_final_kernel<<<1, 1024, 0, st>>>(scratch, n_slots, (long long)n, moments);
    if (cudaGetLastError() != cudaSuccess) return CO3_ECUDA;
    return CO3_OK;
}
