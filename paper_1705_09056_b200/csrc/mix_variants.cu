// Variants of the gossip step (Algorithm 1 steps 4-5) beside the plain kernels of mix_update.cu:
//
//   SWAPPED  footnote c of Algorithm 1: update locally first, then average,
//                X_next[i] = sum_j W_ij (X[j] - gamma G[j]),
//            which with W = 1 1^T / n is exactly centralized minibatch SGD on every row.
//   STATS    the consensus distance sum_i ||xbar - x_i||^2 (Eq. 10 / Eq. 13) of X_next, accumulated
//            while the column is in registers, so that logging it every step costs no second pass
//            over HBM.  Per column the new rows are shifted by the first one and sum d, sum d^2 are
//            kept in fp64; per-CTA partials are added in a fixed order by consensus_final.
//
//   MOM      the momentum buffers of the Section 5.3 runs, updated in the same pass: where row j of G is
//            loaded, d_j = beta V[j] + G[j] is formed, written back to V[j] and used in place of G[j]
//            (20 bytes per replica-parameter instead of 24 with a separate momentum pass).
//
// Same traffic as the plain kernels otherwise: X and G read once, X_next written once.
#include "ctx.h"

namespace dpsgd {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

__device__ __forceinline__ float4 axpy4(float a, float4 x, float4 y) {   // a*x + y
    return make_float4(fmaf(a, x.x, y.x), fmaf(a, x.y, y.y), fmaf(a, x.z, y.z), fmaf(a, x.w, y.w));
}
__device__ __forceinline__ float4 mix3(float wl, float4 a, float ws, float4 b, float wr, float4 c) {
    return make_float4(fmaf(wr, c.x, fmaf(ws, b.x, wl * a.x)), fmaf(wr, c.y, fmaf(ws, b.y, wl * a.y)),
                       fmaf(wr, c.z, fmaf(ws, b.z, wl * a.z)), fmaf(wr, c.w, fmaf(ws, b.w, wl * a.w)));
}

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

// Running sum d and sum d^2 of the new rows of four columns, d = row - first new row.
struct ColumnStats {
    float4 ref;
    double s1[4], s2[4];
    bool have;
    __device__ __forceinline__ void init() {
        have = false;
#pragma unroll
        for (int t = 0; t < 4; ++t) { s1[t] = 0.0; s2[t] = 0.0; }
    }
    __device__ __forceinline__ void add(float4 v) {
        if (!have) { ref = v; have = true; return; }
        const double d0 = (double)(v.x - ref.x), d1 = (double)(v.y - ref.y);
        const double d2 = (double)(v.z - ref.z), d3 = (double)(v.w - ref.w);
        s1[0] += d0; s1[1] += d1; s1[2] += d2; s1[3] += d3;
        s2[0] = fma(d0, d0, s2[0]); s2[1] = fma(d1, d1, s2[1]);
        s2[2] = fma(d2, d2, s2[2]); s2[3] = fma(d3, d3, s2[3]);
    }
    __device__ __forceinline__ double total(int n) const {
        const double inv_n = 1.0 / (double)n;
        double acc = 0.0;
#pragma unroll
        for (int t = 0; t < 4; ++t) acc += s2[t] - s1[t] * s1[t] * inv_n;
        return acc;
    }
};

// Ring (Theorem 3).  v_j = X[j] (Algorithm 1 order) or X[j] - gamma G[j] (footnote c); a rolling
// register window (prev, cur, next) over v walks down the column, rows 0 and n-1 kept for the wrap.
template <bool SWAPPED, bool STATS, bool MOM>
__global__ void __launch_bounds__(kThreads)
mix_ring_x_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                  float4* __restrict__ V, float beta, const float* __restrict__ band, int n, int64_t ld4,
                  float ngamma, double* __restrict__ partials) {
    __shared__ double red[kThreads / 32];
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    ColumnStats st;
    st.init();
    if (c < ld4) {
        const float4* x = X + c;
        const float4* g = G + c;
        float4* o = Xn + c;
        float4* vb = MOM ? V + c : nullptr;
        auto direction = [&](int j) {            // row j of G, or of the updated momentum buffers
            const float4 gv = ld_stream(g + (int64_t)j * ld4);
            if (!MOM) return gv;
            const float4 d = axpy4(beta, ld_stream(vb + (int64_t)j * ld4), gv);
            st_stream(vb + (int64_t)j * ld4, d);
            return d;
        };
        auto row_value = [&](int j) {            // v_j
            const float4 xv = ld_stream(x + (int64_t)j * ld4);
            return SWAPPED ? axpy4(ngamma, direction(j), xv) : xv;
        };
        const float4 first = row_value(0);
        const float4 last = n > 1 ? row_value(n - 1) : first;   // each row's direction is formed once
        float4 prev = last, cur = first;
        constexpr int U = 4;
        int i = 0;
        for (; i + U <= n - 2; i += U) {          // rows whose lower neighbour i+1 <= n-2 comes from memory
            float4 xn[U], gv[U], mv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t gr = (int64_t)(i + u + (SWAPPED ? 1 : 0)) * ld4;
                xn[u] = ld_stream(x + (int64_t)(i + u + 1) * ld4);
                gv[u] = ld_stream(g + gr);
                if (MOM) mv[u] = ld_stream(vb + gr);
            }
            if (MOM) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    gv[u] = axpy4(beta, mv[u], gv[u]);
                    st_stream(vb + (int64_t)(i + u + (SWAPPED ? 1 : 0)) * ld4, gv[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float* w = band + 3 * (i + u);
                const float4 nx = SWAPPED ? axpy4(ngamma, gv[u], xn[u]) : xn[u];
                float4 r = mix3(__ldg(w), prev, __ldg(w + 1), cur, __ldg(w + 2), nx);
                if (!SWAPPED) r = axpy4(ngamma, gv[u], r);
                st_stream(o + (int64_t)(i + u) * ld4, r);
                if (STATS) st.add(r);
                prev = cur;
                cur = nx;
            }
        }
        for (; i < n; ++i) {
            float4 nx;
            if (i + 1 == n) nx = first;
            else if (i + 1 == n - 1) nx = last;
            else nx = row_value(i + 1);
            const float* w = band + 3 * i;
            float4 r = mix3(__ldg(w), prev, __ldg(w + 1), cur, __ldg(w + 2), nx);
            if (!SWAPPED) r = axpy4(ngamma, direction(i), r);
            st_stream(o + (int64_t)i * ld4, r);
            if (STATS) st.add(r);
            prev = cur;
            cur = nx;
        }
    }
    if (STATS) {
        const double r = block_sum(st.total(n), red);
        if (threadIdx.x == 0) partials[blockIdx.x] = r;
    }
}

// W = w 1 1^T.  Algorithm 1 order: x'_i = w sum_j x_j - gamma g_i.  Footnote c: every row becomes
// w sum_j (x_j - gamma g_j), i.e. one centralized SGD step when w = 1/n.
template <bool SWAPPED, bool STATS, bool MOM>
__global__ void __launch_bounds__(kThreads)
mix_uniform_x_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                     float4* __restrict__ V, float beta, int n, int64_t ld4, float w, float ngamma,
                     double* __restrict__ partials) {
    __shared__ double red[kThreads / 32];
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    ColumnStats st;
    st.init();
    if (c < ld4) {
        const float4* x = X + c;
        const float4* g = G + c;
        float4* o = Xn + c;
        float4* vb = MOM ? V + c : nullptr;
        auto direction = [&](int j) {            // row j of G, or of the updated momentum buffers
            const float4 gv = ld_stream(g + (int64_t)j * ld4);
            if (!MOM) return gv;
            const float4 d = axpy4(beta, ld_stream(vb + (int64_t)j * ld4), gv);
            st_stream(vb + (int64_t)j * ld4, d);
            return d;
        };
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        constexpr int U = MOM ? 4 : 8;
        int i = 0;
        for (; i + U <= n; i += U) {
            float4 v[U], gv[U], mv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                v[u] = ld_stream(x + (int64_t)(i + u) * ld4);
                if (SWAPPED) gv[u] = ld_stream(g + (int64_t)(i + u) * ld4);
                if (SWAPPED && MOM) mv[u] = ld_stream(vb + (int64_t)(i + u) * ld4);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (SWAPPED && MOM) {
                    gv[u] = axpy4(beta, mv[u], gv[u]);
                    st_stream(vb + (int64_t)(i + u) * ld4, gv[u]);
                }
                const float4 t = SWAPPED ? axpy4(ngamma, gv[u], v[u]) : v[u];
                s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
            }
        }
        for (; i < n; ++i) {
            float4 t = ld_stream(x + (int64_t)i * ld4);
            if (SWAPPED) t = axpy4(ngamma, direction(i), t);
            s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
        }
        s.x *= w; s.y *= w; s.z *= w; s.w *= w;
        if (SWAPPED) {
            for (i = 0; i < n; ++i) st_stream(o + (int64_t)i * ld4, s);
            // all rows equal: the consensus distance is exactly zero
        } else {
            i = 0;
            for (; i + U <= n; i += U) {
                float4 gv[U], mv[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    gv[u] = ld_stream(g + (int64_t)(i + u) * ld4);
                    if (MOM) mv[u] = ld_stream(vb + (int64_t)(i + u) * ld4);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (MOM) {
                        gv[u] = axpy4(beta, mv[u], gv[u]);
                        st_stream(vb + (int64_t)(i + u) * ld4, gv[u]);
                    }
                    const float4 r = axpy4(ngamma, gv[u], s);
                    st_stream(o + (int64_t)(i + u) * ld4, r);
                    if (STATS) st.add(r);
                }
            }
            for (; i < n; ++i) {
                const float4 r = axpy4(ngamma, direction(i), s);
                st_stream(o + (int64_t)i * ld4, r);
                if (STATS) st.add(r);
            }
        }
    }
    if (STATS) {
        const double r = block_sum(st.total(n), red);
        if (threadIdx.x == 0) partials[blockIdx.x] = r;
    }
}

// Footnote c for any W in CSR, neighbour rows of X and G through the caches.
__global__ void __launch_bounds__(128)
mix_gather_swapped_kernel(const float4* __restrict__ X, const float4* __restrict__ G, float4* __restrict__ Xn,
                          const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                          const float* __restrict__ val, int n, int64_t ld4, float ngamma) {
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (c >= ld4) return;
    for (int i = 0; i < n; ++i) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        const int pe = __ldg(row_ptr + i + 1);
        for (int p = __ldg(row_ptr + i); p < pe; ++p) {
            const float w = __ldg(val + p);
            const int64_t j = __ldg(col + p);
            const float4 y = axpy4(ngamma, __ldg(G + j * ld4 + c), __ldg(X + j * ld4 + c));
            a.x = fmaf(w, y.x, a.x); a.y = fmaf(w, y.y, a.y);
            a.z = fmaf(w, y.z, a.z); a.w = fmaf(w, y.w, a.w);
        }
        st_stream(Xn + (int64_t)i * ld4 + c, a);
    }
}

// Momentum buffer of the Torch experiments (Section 5.3): V <- beta V + G, in place.  blockIdx.y is
// the node; a node whose entry of `active` is zero keeps its buffer.
__global__ void __launch_bounds__(kThreads)
momentum_kernel(float4* __restrict__ V, const float4* __restrict__ G, int64_t ld4, float beta,
                const int32_t* __restrict__ active) {
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= ld4 || (active && __ldg(active + blockIdx.y) == 0)) return;
    const int64_t t = (int64_t)blockIdx.y * ld4 + c;
    st_stream(V + t, axpy4(beta, ld_stream(V + t), ld_stream(G + t)));
}

// Local SGD step without communication: X <- X - gamma D, in place (W = I), for the active nodes.
__global__ void __launch_bounds__(kThreads)
local_update_kernel(float4* __restrict__ X, const float4* __restrict__ D, int64_t ld4, float ngamma,
                    const int32_t* __restrict__ active) {
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= ld4 || (active && __ldg(active + blockIdx.y) == 0)) return;
    const int64_t t = (int64_t)blockIdx.y * ld4 + c;
    st_stream(X + t, axpy4(ngamma, ld_stream(D + t), ld_stream(X + t)));
}

}  // namespace

// Grids of (column blocks, node): gridDim.y <= 65535 bounds n here.
cudaError_t launch_local_update(dpsgd_ctx* c, float* X, const float* D, const int32_t* active) {
    if (c->n > 65535) return cudaErrorInvalidConfiguration;
    const int64_t ld4 = c->ld / 4;
    const dim3 grid((unsigned)((ld4 + kThreads - 1) / kThreads), (unsigned)c->n);
    local_update_kernel<<<grid, kThreads, 0, c->stream>>>(
        reinterpret_cast<float4*>(X), reinterpret_cast<const float4*>(D), ld4, -c->gamma, active);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_momentum(dpsgd_ctx* c, float* V, const float* G, const int32_t* active) {
    if (c->n > 65535) return cudaErrorInvalidConfiguration;
    const int64_t ld4 = c->ld / 4;
    const dim3 grid((unsigned)((ld4 + kThreads - 1) / kThreads), (unsigned)c->n);
    momentum_kernel<<<grid, kThreads, 0, c->stream>>>(
        reinterpret_cast<float4*>(V), reinterpret_cast<const float4*>(G), ld4, c->beta, active);
    c->launches++;
    return cudaGetLastError();
}

// stats_out != nullptr: also leave the consensus distance of X_next in *stats_out (device).
// V != nullptr (ring and uniform W only): G holds the gradients, and the momentum buffers V are
// updated in the same pass and used as the step direction.
// Returns cudaErrorNotSupported when this W has no kernel for what is asked (the caller then runs
// the separate passes).
namespace {

template <bool SWAPPED, bool STATS, bool MOM>
void launch_ring_x(dpsgd_ctx* c, int grid, const float4* x4, const float4* g4, float4* o4, float4* v4) {
    mix_ring_x_kernel<SWAPPED, STATS, MOM><<<grid, kThreads, 0, c->stream>>>(
        x4, g4, o4, v4, c->beta, c->W.band, c->n, c->ld / 4, -c->gamma, c->d_partials);
}
template <bool SWAPPED, bool STATS, bool MOM>
void launch_uniform_x(dpsgd_ctx* c, int grid, const float4* x4, const float4* g4, float4* o4, float4* v4) {
    mix_uniform_x_kernel<SWAPPED, STATS, MOM><<<grid, kThreads, 0, c->stream>>>(
        x4, g4, o4, v4, c->beta, c->n, c->ld / 4, c->W.uniform, -c->gamma, c->d_partials);
}

#define DPSGD_X_DISPATCH(fn, sw, st, mo, ...)                                   \
    do {                                                                        \
        const int key = ((sw) ? 4 : 0) | ((st) ? 2 : 0) | ((mo) ? 1 : 0);       \
        switch (key) {                                                          \
            case 0: fn<false, false, false>(__VA_ARGS__); break;                \
            case 1: fn<false, false, true>(__VA_ARGS__); break;                 \
            case 2: fn<false, true, false>(__VA_ARGS__); break;                 \
            case 3: fn<false, true, true>(__VA_ARGS__); break;                  \
            case 4: fn<true, false, false>(__VA_ARGS__); break;                 \
            case 5: fn<true, false, true>(__VA_ARGS__); break;                  \
            case 6: fn<true, true, false>(__VA_ARGS__); break;                  \
            default: fn<true, true, true>(__VA_ARGS__); break;                  \
        }                                                                       \
    } while (0)

}  // namespace

cudaError_t launch_mix_variant(dpsgd_ctx* c, const float* X, const float* G, float* Xn, bool swapped,
                               double* stats_out, float* V) {
    const int64_t ld4 = c->ld / 4;
    const int grid = (int)((ld4 + kThreads - 1) / kThreads);
    const float4* x4 = reinterpret_cast<const float4*>(X);
    const float4* g4 = reinterpret_cast<const float4*>(G);
    float4* o4 = reinterpret_cast<float4*>(Xn);
    float4* v4 = reinterpret_cast<float4*>(V);
    const bool ring = c->mix_kind == DPSGD_MIX_RING, uniform = c->mix_kind == DPSGD_MIX_UNIFORM_DENSE;
    if ((stats_out || V) && !(ring || uniform)) return cudaErrorNotSupported;
    if (stats_out) {
        cudaError_t e = ensure_partials(c, grid);
        if (e != cudaSuccess) return e;
    }
    if (ring) {
        DPSGD_X_DISPATCH(launch_ring_x, swapped, stats_out != nullptr, V != nullptr, c, grid, x4, g4, o4, v4);
    } else if (uniform) {
        DPSGD_X_DISPATCH(launch_uniform_x, swapped, stats_out != nullptr, V != nullptr, c, grid, x4, g4, o4, v4);
    } else {
        mix_gather_swapped_kernel<<<(unsigned)((ld4 + 127) / 128), 128, 0, c->stream>>>(
            x4, g4, o4, c->W.row_ptr, c->W.col, c->W.val, c->n, ld4, -c->gamma);
    }
    c->launches++;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && stats_out) e = launch_consensus_final(c, grid, stats_out);
    return e;
}

}  // namespace dpsgd
