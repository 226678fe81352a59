// Consensus distance sum_i ||xbar - x_i||^2 (sum of the Q_{k,i} of Eq. 10; M_k of Eq. 13 is
// this divided by n) and the node average xbar (output of Algorithm 1).
//
// One pass over X (4 bytes per replica-parameter).  Per column the rows are shifted by row 0,
// d_i = x_i - x_0, and sum_i (d_i - dbar)^2 = sum d_i^2 - (sum d_i)^2 / n is accumulated in
// fp64, so no cancellation against |x| occurs.  Columns are combined by warp shuffles, one
// fp64 partial per CTA, and a second single-CTA kernel adds the partials in a fixed order:
// the result is bit-reproducible (no floating-point atomics).
#include <mutex>

#include "ctx.h"

namespace dpsgd {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double block_sum(double v, double* smem) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (warp == 0) {
        r = lane < (blockDim.x >> 5) ? smem[lane] : 0.0;
        r = warp_sum(r);
    }
    return r;  // valid in thread 0
}

template <int U>
__global__ void __launch_bounds__(kThreads)
consensus_partial_kernel(const float4* __restrict__ X, int n, int64_t ld4, double* __restrict__ partials) {
    __shared__ double red[kThreads / 32];
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    double acc = 0.0;
    if (c < ld4) {
        const float4* x = X + c;
        const float4 x0 = __ldcs(x);
        double s1[4] = {0, 0, 0, 0}, s2[4] = {0, 0, 0, 0};
        int i = 1;
        for (; i + U <= n; i += U) {
            float4 v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) v[u] = __ldcs(x + (int64_t)(i + u) * ld4);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const double d0 = (double)(v[u].x - x0.x), d1 = (double)(v[u].y - x0.y);
                const double d2 = (double)(v[u].z - x0.z), d3 = (double)(v[u].w - x0.w);
                s1[0] += d0; s1[1] += d1; s1[2] += d2; s1[3] += d3;
                s2[0] = fma(d0, d0, s2[0]); s2[1] = fma(d1, d1, s2[1]);
                s2[2] = fma(d2, d2, s2[2]); s2[3] = fma(d3, d3, s2[3]);
            }
        }
        for (; i < n; ++i) {
            const float4 v = __ldcs(x + (int64_t)i * ld4);
            const double d0 = (double)(v.x - x0.x), d1 = (double)(v.y - x0.y);
            const double d2 = (double)(v.z - x0.z), d3 = (double)(v.w - x0.w);
            s1[0] += d0; s1[1] += d1; s1[2] += d2; s1[3] += d3;
            s2[0] = fma(d0, d0, s2[0]); s2[1] = fma(d1, d1, s2[1]);
            s2[2] = fma(d2, d2, s2[2]); s2[3] = fma(d3, d3, s2[3]);
        }
        const double inv_n = 1.0 / (double)n;
#pragma unroll
        for (int t = 0; t < 4; ++t) acc += s2[t] - s1[t] * s1[t] * inv_n;
    }
    const double r = block_sum(acc, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = r;
}

__global__ void __launch_bounds__(kThreads)
consensus_final_kernel(const double* __restrict__ partials, int count, double* __restrict__ out) {
    __shared__ double red[kThreads / 32];
    double acc = 0.0;
    for (int t = threadIdx.x; t < count; t += kThreads) acc += partials[t];
    const double r = block_sum(acc, red);
    if (threadIdx.x == 0) *out = r > 0.0 ? r : 0.0;
}

__global__ void __launch_bounds__(kThreads)
average_kernel(const float4* __restrict__ X, int n, int64_t ld4, float4* __restrict__ xbar) {
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= ld4) return;
    double s[4] = {0, 0, 0, 0};
    for (int i = 0; i < n; ++i) {
        const float4 v = __ldg(X + (int64_t)i * ld4 + c);
        s[0] += v.x; s[1] += v.y; s[2] += v.z; s[3] += v.w;
    }
    const double inv_n = 1.0 / (double)n;
    xbar[c] = make_float4((float)(s[0] * inv_n), (float)(s[1] * inv_n), (float)(s[2] * inv_n),
                          (float)(s[3] * inv_n));
}

}  // namespace

// Grows the per-CTA partial-sum buffer of the context to at least `count` doubles.
cudaError_t ensure_partials(dpsgd_ctx* c, int count) {
    if (count <= c->partials_cap) return cudaSuccess;
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return e;
    cudaFree(c->d_partials);
    c->d_partials = nullptr; c->partials_cap = 0;
    e = cudaMalloc(&c->d_partials, sizeof(double) * (size_t)count);
    if (e != cudaSuccess) return e;
    c->partials_cap = count;
    return cudaSuccess;
}

// Adds the first `count` partials of the context in a fixed order into *result_dev.
cudaError_t launch_consensus_final(dpsgd_ctx* c, int count, double* result_dev) {
    consensus_final_kernel<<<1, kThreads, 0, c->stream>>>(c->d_partials, count, result_dev);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_consensus(dpsgd_ctx* c, const float* X, double* result_dev) {
    const int64_t ld4 = c->ld / 4;
    const int grid = (int)((ld4 + kThreads - 1) / kThreads);
    {
        cudaError_t e = ensure_partials(c, grid);
        if (e != cudaSuccess) return e;
    }
    consensus_partial_kernel<8><<<grid, kThreads, 0, c->stream>>>(
        reinterpret_cast<const float4*>(X), c->n, ld4, c->d_partials);
    consensus_final_kernel<<<1, kThreads, 0, c->stream>>>(c->d_partials, grid, result_dev);
    c->launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_average(dpsgd_ctx* c, const float* X, float* xbar) {
    const int64_t ld4 = c->ld / 4;
    const unsigned grid = (unsigned)((ld4 + kThreads - 1) / kThreads);
    average_kernel<<<grid, kThreads, 0, c->stream>>>(reinterpret_cast<const float4*>(X), c->n, ld4,
                                                     reinterpret_cast<float4*>(xbar));
    c->launches++;
    return cudaGetLastError();
}

}  // namespace dpsgd

// ---------------------------------------------------------------------------------------------
// Consensus distance without any allocation.
//
// Some callers cannot let this library allocate: a process that handed its whole device-memory
// budget to its own pool at start-up (a later cudaMalloc would fail or eat into someone else's
// share), a latency-critical loop that must not hit the device-wide synchronisation an
// allocation implies, or code that holds only a raw device pointer and has no dpsgd context (a
// context allocates its scratch when it is created and grown).  For them the per-CTA partial
// sums live in a fixed array inside the library image instead of a cudaMalloc'ed buffer.
//
// The array's name is only a host-side handle in host code; the kernels need its device
// address, fetched once per device with cudaGetSymbolAddress while that device is current.
// ---------------------------------------------------------------------------------------------
namespace dpsgd {
void set_thread_error(const std::string& msg);   // api.cu: message returned by dpsgd_last_error(NULL)
namespace {

constexpr int kNoAllocMaxCtas = 65536;                                   // 512 KB of partials per GPU
constexpr int64_t kNoAllocMaxLd = (int64_t)kNoAllocMaxCtas * kThreads * 4;  // 67,108,864 columns
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) double g_noalloc_partials[kNoAllocMaxCtas];

std::mutex g_noalloc_mutex;
double* g_noalloc_ptr[kNoAllocMaxDevices] = {nullptr};

// Device address of the partials array on the current device (set up on the first call there).
cudaError_t noalloc_scratch(double** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_partials);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = static_cast<double*>(p);
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

dpsgd_status noalloc_fail(dpsgd_status s, const std::string& msg) {
    set_thread_error(msg);
    return s;
}

}  // namespace
}  // namespace dpsgd

extern "C" DPSGD_API dpsgd_status dpsgd_consensus_dist_noalloc(const float* X_dev, int32_t n, int64_t N,
                                                               int64_t ld, void* cuda_stream,
                                                               double* out_dev) {
    using namespace dpsgd;
    if (!X_dev || !out_dev) return noalloc_fail(DPSGD_ERR_ARG, "X_dev or out_dev is NULL");
    if (n < 1 || n > 65535 || N < 1 || ld < N) return noalloc_fail(DPSGD_ERR_ARG, "need 1 <= n <= 65535 and 1 <= N <= ld");
    if (ld % 32 != 0 || reinterpret_cast<uintptr_t>(X_dev) % 128 != 0 || reinterpret_cast<uintptr_t>(out_dev) % 8 != 0)
        return noalloc_fail(DPSGD_ERR_ALIGN, "X_dev must be 128-byte aligned, ld a multiple of 32 floats, out_dev 8-byte aligned");
    if (ld > kNoAllocMaxLd) {
        char buf[160];
        snprintf(buf, sizeof buf, "ld = %lld exceeds the %lld columns the built-in scratch array covers; "
                 "use a context and dpsgd_consensus_dist instead", (long long)ld, (long long)kNoAllocMaxLd);
        return noalloc_fail(DPSGD_ERR_UNSUPPORTED, buf);
    }
    // Both pointers must be memory of the CURRENT device: the scratch address below belongs to it, and
    // a kernel handed another GPU's pointer would fault.  The query allocates nothing.
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return noalloc_fail(DPSGD_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    const void* ptrs[2] = {X_dev, out_dev};
    for (const void* p : ptrs) {
        cudaPointerAttributes attr;
        e = cudaPointerGetAttributes(&attr, p);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return noalloc_fail(DPSGD_ERR_ARG, std::string("X_dev / out_dev is not a CUDA pointer: ") + cudaGetErrorString(e));
        }
        if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)
            return noalloc_fail(DPSGD_ERR_ARG, "X_dev and out_dev must be device memory");
        if (attr.type == cudaMemoryTypeDevice && attr.device != dev)
            return noalloc_fail(DPSGD_ERR_ARG, "X_dev and out_dev must belong to the current device");
    }
    double* partials = nullptr;
    e = noalloc_scratch(&partials);
    if (e != cudaSuccess) return noalloc_fail(DPSGD_ERR_CUDA, std::string("scratch set-up: ") + cudaGetErrorString(e));
    cudaGetLastError();   // an error left by an earlier launch on this thread is not this call's
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int64_t ld4 = ld / 4;
    const int grid = (int)((ld4 + kThreads - 1) / kThreads);
    // every partial in [0, grid) is overwritten by the first kernel before the second reads it, so
    // whatever an earlier call left in the array is never seen
    consensus_partial_kernel<8><<<grid, kThreads, 0, stream>>>(reinterpret_cast<const float4*>(X_dev), n, ld4,
                                                               partials);
    consensus_final_kernel<<<1, kThreads, 0, stream>>>(partials, grid, out_dev);
    e = cudaGetLastError();
    if (e != cudaSuccess) return noalloc_fail(DPSGD_ERR_CUDA, std::string("consensus kernels: ") + cudaGetErrorString(e));
    return DPSGD_OK;
}
