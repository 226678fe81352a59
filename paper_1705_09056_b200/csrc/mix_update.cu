// Fused gossip step of D-PSGD (Algorithm 1 steps 4-5; global form of Section 3):
//     X_next[i][c] = sum_j W_ij X[j][c] - gamma G[i][c]
// One pass over HBM: every element of X and G is read once, X_next written once
// (12 bytes per replica-parameter), whatever the topology.
//
// All kernels here give one thread a group of 4 adjacent columns (one 128-bit access per row)
// and let it walk down the n rows; a warp therefore touches 512 contiguous bytes of one row
// per access.  The stacked matrices are far larger than L2 on the bandwidth-bound shapes, so
// once-only traffic uses streaming (evict-first) loads and stores.
#include <algorithm>

#include "ctx.h"

namespace dpsgd {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

__device__ __forceinline__ float4 mix3(float wl, float4 a, float ws, float4 b, float wr, float4 c,
                                       float ngamma, float4 g) {
    float4 r;
    r.x = fmaf(ngamma, g.x, fmaf(wr, c.x, fmaf(ws, b.x, wl * a.x)));
    r.y = fmaf(ngamma, g.y, fmaf(wr, c.y, fmaf(ws, b.y, wl * a.y)));
    r.z = fmaf(ngamma, g.z, fmaf(wr, c.z, fmaf(ws, b.z, wl * a.z)));
    r.w = fmaf(ngamma, g.w, fmaf(wr, c.w, fmaf(ws, b.w, wl * a.w)));
    return r;
}

// Ring (Theorem 3): row i mixes rows i-1, i, i+1 (mod n).  A rolling register window
// (prev, cur, next) walks down the column; rows 0 and n-1 are kept for the wrap-around, so
// each X element is loaded exactly once.  The row loop is unrolled U times so that the 2U
// independent 128-bit loads of an unrolled body are in flight together.
template <int U>
__global__ void __launch_bounds__(kThreads)
mix_ring_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                const float* __restrict__ band, int n, int64_t ld4, float ngamma) {
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= ld4) return;
    const float4* x = X + c;
    const float4* g = G + c;
    float4* o = Xn + c;

    const float4 first = ld_stream(x);
    const float4 last = ld_stream(x + (int64_t)(n - 1) * ld4);
    float4 prev = last, cur = first;

    int i = 0;
    // rows whose lower neighbour i+1 <= n-2 comes from memory
    for (; i + U <= n - 2; i += U) {
        float4 xn[U], gv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            xn[u] = ld_stream(x + (int64_t)(i + u + 1) * ld4);
            gv[u] = ld_stream(g + (int64_t)(i + u) * ld4);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float wl = __ldg(band + 3 * (i + u));
            const float ws = __ldg(band + 3 * (i + u) + 1);
            const float wr = __ldg(band + 3 * (i + u) + 2);
            st_stream(o + (int64_t)(i + u) * ld4, mix3(wl, prev, ws, cur, wr, xn[u], ngamma, gv[u]));
            prev = cur;
            cur = xn[u];
        }
    }
    for (; i < n; ++i) {
        float4 nx;
        if (i + 1 == n) nx = first;
        else if (i + 1 == n - 1) nx = last;
        else nx = ld_stream(x + (int64_t)(i + 1) * ld4);
        const float4 gv = ld_stream(g + (int64_t)i * ld4);
        const float wl = __ldg(band + 3 * i), ws = __ldg(band + 3 * i + 1), wr = __ldg(band + 3 * i + 2);
        st_stream(o + (int64_t)i * ld4, mix3(wl, prev, ws, cur, wr, nx, ngamma, gv));
        prev = cur;
        cur = nx;
    }
}

// W = w 1 1^T (all entries equal; w = 1/n is the averaging step of centralized PSGD):
// every row mixes to the same vector w * (column sum), computed once per column.
template <int U>
__global__ void __launch_bounds__(kThreads)
mix_uniform_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                   int n, int64_t ld4, float w, float ngamma) {
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= ld4) return;
    const float4* x = X + c;
    const float4* g = G + c;
    float4* o = Xn + c;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    int i = 0;
    for (; i + U <= n; i += U) {
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) v[u] = ld_stream(x + (int64_t)(i + u) * ld4);
#pragma unroll
        for (int u = 0; u < U; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
    }
    for (; i < n; ++i) {
        const float4 v = ld_stream(x + (int64_t)i * ld4);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    s.x *= w; s.y *= w; s.z *= w; s.w *= w;
    i = 0;
    for (; i + U <= n; i += U) {
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) v[u] = ld_stream(g + (int64_t)(i + u) * ld4);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float4 r;
            r.x = fmaf(ngamma, v[u].x, s.x); r.y = fmaf(ngamma, v[u].y, s.y);
            r.z = fmaf(ngamma, v[u].z, s.z); r.w = fmaf(ngamma, v[u].w, s.w);
            st_stream(o + (int64_t)(i + u) * ld4, r);
        }
    }
    for (; i < n; ++i) {
        const float4 v = ld_stream(g + (int64_t)i * ld4);
        float4 r;
        r.x = fmaf(ngamma, v.x, s.x); r.y = fmaf(ngamma, v.y, s.y);
        r.z = fmaf(ngamma, v.z, s.z); r.w = fmaf(ngamma, v.w, s.w);
        st_stream(o + (int64_t)i * ld4, r);
    }
}

// Any W in CSR: neighbour rows are gathered with cached loads.  A CTA owns a column strip of
// all n rows, so the repeated reads of a neighbour row are served by L1/L2 after its first
// touch.  Correct for every valid W; the tiled kernel is the fast path for sparse W.
__global__ void __launch_bounds__(128)
mix_gather_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                  const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                  const float* __restrict__ val, int n, int64_t ld4, float ngamma) {
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (c >= ld4) return;
    const float4* x = X + c;
    for (int i = 0; i < n; ++i) {
        const float4 gv = ld_stream(G + (int64_t)i * ld4 + c);
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        const int pe = __ldg(row_ptr + i + 1);
        for (int p = __ldg(row_ptr + i); p < pe; ++p) {
            const float w = __ldg(val + p);
            const float4 v = __ldg(x + (int64_t)__ldg(col + p) * ld4);
            a.x = fmaf(w, v.x, a.x); a.y = fmaf(w, v.y, a.y);
            a.z = fmaf(w, v.z, a.z); a.w = fmaf(w, v.w, a.w);
        }
        a.x = fmaf(ngamma, gv.x, a.x); a.y = fmaf(ngamma, gv.y, a.y);
        a.z = fmaf(ngamma, gv.z, a.z); a.w = fmaf(ngamma, gv.w, a.w);
        st_stream(Xn + (int64_t)i * ld4 + c, a);
    }
}

// Small problems (X fits L2 many times over): one thread per OUTPUT group of 4 columns instead of
// one per column walking all rows, so the step is a single load-compute-store latency deep.  The
// neighbour rows are re-read through L1/L2, which costs nothing at this size.
__global__ void __launch_bounds__(128)
mix_rowpar_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                  const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                  const float* __restrict__ val, int n, int64_t ld4, float ngamma, int swapped) {
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    const int i = blockIdx.y;
    if (c >= ld4) return;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    const int pe = __ldg(row_ptr + i + 1);
    for (int p = __ldg(row_ptr + i); p < pe; ++p) {
        const float w = __ldg(val + p);
        const int64_t j = __ldg(col + p);
        float4 v = __ldg(X + j * ld4 + c);
        if (swapped) {
            const float4 g = __ldg(G + j * ld4 + c);
            v.x = fmaf(ngamma, g.x, v.x); v.y = fmaf(ngamma, g.y, v.y);
            v.z = fmaf(ngamma, g.z, v.z); v.w = fmaf(ngamma, g.w, v.w);
        }
        a.x = fmaf(w, v.x, a.x); a.y = fmaf(w, v.y, a.y);
        a.z = fmaf(w, v.z, a.z); a.w = fmaf(w, v.w, a.w);
    }
    if (!swapped) {
        const float4 g = __ldg(G + (int64_t)i * ld4 + c);
        a.x = fmaf(ngamma, g.x, a.x); a.y = fmaf(ngamma, g.y, a.y);
        a.z = fmaf(ngamma, g.z, a.z); a.w = fmaf(ngamma, g.w, a.w);
    }
    Xn[(int64_t)i * ld4 + c] = a;
}

// Gossip step on a few column ranges of the stacked matrices (the columns a fused gradient kernel
// has not already written): one thread per output group of 4 columns, as in the kernel above.
struct ColRanges {
    int count;
    int64_t begin4[kMaxLayers + 1];   // first float4 column of each range
    int64_t start4[kMaxLayers + 2];   // running total of the range lengths, start4[count] = all
};

__global__ void __launch_bounds__(128)
mix_ranges_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                  const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                  const float* __restrict__ val, int64_t src_ld4, int64_t ld4, float ngamma, ColRanges rg) {
    const int64_t t = (int64_t)blockIdx.x * 128 + threadIdx.x;
    const int i = blockIdx.y;
    if (t >= rg.start4[rg.count]) return;
    int r = 0;
    while (r + 1 < rg.count && t >= rg.start4[r + 1]) ++r;
    const int64_t c = rg.begin4[r] + (t - rg.start4[r]);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    const int pe = __ldg(row_ptr + i + 1);
    for (int p = __ldg(row_ptr + i); p < pe; ++p) {
        const float w = __ldg(val + p);
        const float4 v = __ldg(X + (int64_t)__ldg(col + p) * src_ld4 + c);
        a.x = fmaf(w, v.x, a.x); a.y = fmaf(w, v.y, a.y);
        a.z = fmaf(w, v.z, a.z); a.w = fmaf(w, v.w, a.w);
    }
    const float4 g = __ldg(G + (int64_t)i * ld4 + c);
    a.x = fmaf(ngamma, g.x, a.x); a.y = fmaf(ngamma, g.y, a.y);
    a.z = fmaf(ngamma, g.z, a.z); a.w = fmaf(ngamma, g.w, a.w);
    Xn[(int64_t)i * ld4 + c] = a;
}

}  // namespace

cudaError_t launch_mix_rest(dpsgd_ctx* c, const float* X, const float* G, float* Xn) {
    // complement of the fused blocks inside [0, ld); block bounds are multiples of 4 columns
    std::vector<std::pair<int64_t, int64_t>> blocks = c->fused_blocks;
    std::sort(blocks.begin(), blocks.end());
    ColRanges rg{};
    int64_t at = 0, total = 0;
    auto add = [&](int64_t b, int64_t e) {
        if (e <= b) return true;
        if (rg.count >= kMaxLayers + 1) return false;
        rg.begin4[rg.count] = b / 4;
        rg.start4[rg.count] = total;
        total += (e - b) / 4;
        rg.count++;
        return true;
    };
    for (const auto& b : blocks) {
        if (b.first % 4 != 0 || b.second % 4 != 0 || b.first < at || b.second > c->ld) return cudaErrorInvalidValue;
        if (!add(at, b.first)) return cudaErrorInvalidValue;
        at = b.second;
    }
    if (!add(at, c->ld)) return cudaErrorInvalidValue;
    rg.start4[rg.count] = total;
    if (total == 0) return cudaSuccess;
    if (c->n > 65535) return cudaErrorInvalidValue;
    dim3 grid((unsigned)((total + 127) / 128), (unsigned)c->n);
    const bool mean = c->fsrc_X != nullptr;      // W = w 1 1^T: gather from the column mean (a one-row matrix)
    mix_ranges_kernel<<<grid, 128, 0, c->stream>>>(
        reinterpret_cast<const float4*>(mean ? c->fsrc_X : X), reinterpret_cast<const float4*>(G),
        reinterpret_cast<float4*>(Xn), mean ? c->fsrc_row_ptr : c->W.row_ptr, mean ? c->fsrc_col : c->W.col,
        mean ? c->fsrc_val : c->W.val, mean ? c->fsrc_ld / 4 : c->ld / 4, c->ld / 4, -c->gamma, rg);
    c->launches++;
    return cudaGetLastError();
}

bool mix_is_small(const dpsgd_ctx* c) {
    return (int64_t)c->n * c->ld * (int64_t)sizeof(float) <= (int64_t(8) << 20) && c->n <= 65535 &&
           (int64_t)c->W.nnz <= (int64_t)c->n * 32;
}

cudaError_t launch_mix_rowpar(dpsgd_ctx* c, const float* X, const float* G, float* Xn) {
    const int64_t ld4 = c->ld / 4;
    dim3 grid((unsigned)((ld4 + 127) / 128), (unsigned)c->n);
    mix_rowpar_kernel<<<grid, 128, 0, c->stream>>>(
        reinterpret_cast<const float4*>(X), reinterpret_cast<const float4*>(G), reinterpret_cast<float4*>(Xn),
        c->W.row_ptr, c->W.col, c->W.val, c->n, ld4, -c->gamma, c->swapped ? 1 : 0);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_mix_ring(dpsgd_ctx* c, const float* X, const float* G, float* Xn) {
    const int64_t ld4 = c->ld / 4;
    const unsigned grid = (unsigned)((ld4 + kThreads - 1) / kThreads);
    mix_ring_kernel<4><<<grid, kThreads, 0, c->stream>>>(
        reinterpret_cast<const float4*>(X), reinterpret_cast<const float4*>(G),
        reinterpret_cast<float4*>(Xn), c->W.band, c->n, ld4, -c->gamma);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_mix_uniform(dpsgd_ctx* c, const float* X, const float* G, float* Xn) {
    const int64_t ld4 = c->ld / 4;
    const unsigned grid = (unsigned)((ld4 + kThreads - 1) / kThreads);
    mix_uniform_kernel<8><<<grid, kThreads, 0, c->stream>>>(
        reinterpret_cast<const float4*>(X), reinterpret_cast<const float4*>(G),
        reinterpret_cast<float4*>(Xn), c->n, ld4, c->W.uniform, -c->gamma);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_mix_gather(dpsgd_ctx* c, const float* X, const float* G, float* Xn) {
    const int64_t ld4 = c->ld / 4;
    const unsigned grid = (unsigned)((ld4 + 127) / 128);
    mix_gather_kernel<<<grid, 128, 0, c->stream>>>(
        reinterpret_cast<const float4*>(X), reinterpret_cast<const float4*>(G),
        reinterpret_cast<float4*>(Xn), c->W.row_ptr, c->W.col, c->W.val, c->n, ld4, -c->gamma);
    c->launches++;
    return cudaGetLastError();
}

}  // namespace dpsgd
