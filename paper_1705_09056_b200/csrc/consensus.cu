// Consensus distance sum_i ||xbar - x_i||^2 (sum of the Q_{k,i} of Eq. 10; M_k of Eq. 13 is
// this divided by n) and the node average xbar (output of Algorithm 1).
//
// One pass over X (4 bytes per replica-parameter).  Per column the rows are shifted by row 0,
// d_i = x_i - x_0, and sum_i (d_i - dbar)^2 = sum d_i^2 - (sum d_i)^2 / n is accumulated in
// fp64, so no cancellation against |x| occurs.  Columns are combined by warp shuffles, one
// fp64 partial per CTA, and a second single-CTA kernel adds the partials in a fixed order:
// the result is bit-reproducible (no floating-point atomics).
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

cudaError_t launch_consensus(dpsgd_ctx* c, const float* X, double* result_dev) {
    const int64_t ld4 = c->ld / 4;
    const int grid = (int)((ld4 + kThreads - 1) / kThreads);
    if (grid > c->partials_cap) {
        cudaError_t e = cudaStreamSynchronize(c->stream);
        if (e != cudaSuccess) return e;
        cudaFree(c->d_partials);
        c->d_partials = nullptr; c->partials_cap = 0;
        e = cudaMalloc(&c->d_partials, sizeof(double) * (size_t)grid);
        if (e != cudaSuccess) return e;
        c->partials_cap = grid;
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
