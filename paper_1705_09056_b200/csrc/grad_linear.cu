// Algorithm 1 steps 2-3 for the two linear models: every node's minibatch gradient at its own
// row x_{k,i} (the columns of dF(X_k; xi_k), Section 3), as the mean over B samples.
//
//   least squares : F = 1/2 (a.x - y)^2             g = (1/B) sum_b (a_b.x - y_b) a_b
//   logistic      : F = log(1 + exp(-y (a.w + c)))  g_w = (1/B) sum_b -y_b s_b a_b + l2 w,
//                   x = [w | c]                     g_c = (1/B) sum_b -y_b s_b,  s_b = sigma(-y_b z_b)
//
// Two kernels: a batched GEMV "forward" (one CTA per (node, sample): draw the index, dot the
// gathered data row with the node's parameters by warp shuffles, turn it into the per-sample
// coefficient) and a rank-B "backward" (G_i = sum_b coef_b a_b, eight interleaved slices of the minibatch added in a fixed order).  All reductions run in a
// fixed order, so results are bit-reproducible.
#include "ctx.h"
#include "philox.cuh"

namespace dpsgd {
namespace {

constexpr int kFwdThreads = 256;

__device__ __forceinline__ float warp_allsum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One CTA per (node, sample): all loads of the 16 KB data row are in flight at once (four 128-bit
// loads per thread at d = 4096), then a shuffle + shared-memory reduction in a fixed order.
template <int VEC>
__global__ void __launch_bounds__(kFwdThreads)
glm_forward_kernel(const float* __restrict__ X, int64_t ld, const float* __restrict__ A,
                   const float* __restrict__ y, int64_t m, int d, int B, int n, uint64_t seed,
                   uint64_t k, const uint64_t* __restrict__ k_ptr, int model, int32_t* __restrict__ idx,
                   float* __restrict__ coef, const int32_t* __restrict__ node_batch) {
    __shared__ float part[kFwdThreads / 32];
    const int w = blockIdx.x;
    const int node = w / B, b = w - node * B;
    if (k_ptr) k = *k_ptr;        // iteration counter kept on the device (graph replay)
    const int32_t j = sample_index(seed, k, (uint32_t)node, (uint32_t)b, (uint32_t)m);
    const int Bi = node_batch ? __ldg(node_batch + node) : B;   // this node's minibatch size
    if (b >= Bi) {                // draw beyond this node's minibatch: recorded, not used
        if (threadIdx.x == 0) { idx[w] = j; coef[w] = 0.f; }
        return;
    }
    const float* row = A + ((int64_t)node * m + j) * d;
    const float* x = X + (int64_t)node * ld;
    float acc = 0.f;
    if (VEC == 4) {
        const float4* r4 = reinterpret_cast<const float4*>(row);
        const float4* x4 = reinterpret_cast<const float4*>(x);
        const int d4 = d / 4;
        int c = threadIdx.x;
        for (; c + 3 * kFwdThreads < d4; c += 4 * kFwdThreads) {
            float4 a[4], v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { a[u] = __ldg(r4 + c + u * kFwdThreads); v[u] = __ldg(x4 + c + u * kFwdThreads); }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc = fmaf(a[u].x, v[u].x, acc); acc = fmaf(a[u].y, v[u].y, acc);
                acc = fmaf(a[u].z, v[u].z, acc); acc = fmaf(a[u].w, v[u].w, acc);
            }
        }
        for (; c < d4; c += kFwdThreads) {
            const float4 a = __ldg(r4 + c), v = __ldg(x4 + c);
            acc = fmaf(a.x, v.x, acc); acc = fmaf(a.y, v.y, acc);
            acc = fmaf(a.z, v.z, acc); acc = fmaf(a.w, v.w, acc);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += kFwdThreads) acc = fmaf(__ldg(row + c), __ldg(x + c), acc);
    }
    acc = warp_allsum(acc);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float dot = 0.f;
#pragma unroll
        for (int t = 0; t < kFwdThreads / 32; ++t) dot += part[t];
        const float yv = __ldg(y + (int64_t)node * m + j);
        float cf;
        if (model == DPSGD_MODEL_LSQ) {
            cf = (dot - yv) / (float)Bi;
        } else {
            const float z = dot + __ldg(x + d);
            const float s = 1.f / (1.f + expf(yv * z));
            cf = -yv * s / (float)Bi;
        }
        idx[w] = j;
        coef[w] = cf;
    }
}

// blockDim = (32, 8): 32 column groups x 8 interleaved slices of the minibatch.
template <int VEC>
__global__ void __launch_bounds__(256)
glm_backward_kernel(const float* __restrict__ X, float* __restrict__ G, int64_t ld,
                    const float* __restrict__ A, int64_t m, int d, int B, int model, float l2,
                    const int32_t* __restrict__ idx, const float* __restrict__ coef,
                    const int32_t* __restrict__ node_batch) {
    __shared__ float red[8][32][VEC];
    const int node = blockIdx.y;
    const int Bi = node_batch ? __ldg(node_batch + node) : B;
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int col = (blockIdx.x * 32 + tx) * VEC;       // first of VEC columns
    const bool live = col < d;
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    const int32_t* ix = idx + (int64_t)node * B;
    const float* cf = coef + (int64_t)node * B;
    if (live) {
        const float* base = A + (int64_t)node * m * d + col;
#pragma unroll 8
        for (int b = ty; b < Bi; b += 8) {
            const float w = __ldg(cf + b);
            const float* row = base + (int64_t)__ldg(ix + b) * d;
            if (VEC == 4) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(row));
                acc[0] = fmaf(w, a.x, acc[0]); acc[1 % VEC] = fmaf(w, a.y, acc[1 % VEC]);
                acc[2 % VEC] = fmaf(w, a.z, acc[2 % VEC]); acc[3 % VEC] = fmaf(w, a.w, acc[3 % VEC]);
            } else {
                acc[0] = fmaf(w, __ldg(row), acc[0]);
            }
        }
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) red[ty][tx][v] = acc[v];
    __syncthreads();
    if (ty == 0 && live) {
        float* g = G + (int64_t)node * ld + col;
        const float* x = X + (int64_t)node * ld + col;
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            float s = red[0][tx][v];
#pragma unroll
            for (int t = 1; t < 8; ++t) s += red[t][tx][v];
            if (model == DPSGD_MODEL_LOGISTIC) s = fmaf(l2, __ldg(x + v), s);
            g[v] = s;
        }
    }
    // bias gradient (logistic) and zero padding: columns [d, ld)
    if (blockIdx.x == 0 && ty == 1) {
        for (int64_t c = d + tx; c < ld; c += 32) {
            float s = 0.f;
            if (model == DPSGD_MODEL_LOGISTIC && c == d)
                for (int b = 0; b < Bi; ++b) s += __ldg(cf + b);
            G[(int64_t)node * ld + c] = s;
        }
    }
}

// ---- rows kept in registers: forward and backward from ONE read of the sampled rows ----
//
// A CTA owns kRowsS consecutive draws of a node.  Thread t holds the 16-byte columns t, t + 256, ... of
// each of their data rows (d <= 4096: at most four per row), so the dot products (shuffles, then a
// fixed-order sum over the warps), the coefficients and the CTA's share sum_s coef_s a_s of the gradient
// all come from that one read.  The shares go to a scratch [node][group][ld] and a second, small kernel
// adds them in group order (bit-reproducible), applies the L2 term and writes the padding.
constexpr int kRowsS = 4;
constexpr int kRowsThreads = 256;
constexpr int kRowsMaxR = 4;             // 16-byte columns per thread and row: d <= 4 * 4 * 256

__global__ void __launch_bounds__(kRowsThreads)
glm_rows_kernel(const float* __restrict__ X, int64_t ld, const float* __restrict__ A, const float* __restrict__ y,
                int64_t m, int d, int B, uint64_t seed, uint64_t k, const uint64_t* __restrict__ k_ptr, int model,
                int32_t* __restrict__ idx, float* __restrict__ part, int groups,
                const int32_t* __restrict__ node_batch) {
    __shared__ float red[kRowsThreads / 32][kRowsS];
    __shared__ float coef[kRowsS];
    const int node = blockIdx.y, grp = blockIdx.x, tid = threadIdx.x;
    if (k_ptr) k = *k_ptr;        // iteration counter kept on the device (graph replay)
    const int Bi = node_batch ? __ldg(node_batch + node) : B;
    const int d4 = d / 4;
    const float4* x4 = reinterpret_cast<const float4*>(X + (int64_t)node * ld);
    float4 row[kRowsS][kRowsMaxR], xv[kRowsMaxR];
    int32_t jdx[kRowsS];
#pragma unroll
    for (int s = 0; s < kRowsS; ++s) {
        const int b = grp * kRowsS + s;
        jdx[s] = b < B ? sample_index(seed, k, (uint32_t)node, (uint32_t)b, (uint32_t)m) : 0;
        if (tid == 0 && b < B) idx[node * B + b] = jdx[s];
        const float4* r4 = reinterpret_cast<const float4*>(A + ((int64_t)node * m + jdx[s]) * d);
#pragma unroll
        for (int r = 0; r < kRowsMaxR; ++r) {
            const int c = tid + r * kRowsThreads;
            row[s][r] = (b < Bi && c < d4) ? __ldg(r4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
#pragma unroll
    for (int r = 0; r < kRowsMaxR; ++r) {
        const int c = tid + r * kRowsThreads;
        xv[r] = c < d4 ? __ldg(x4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int s = 0; s < kRowsS; ++s) {
        float acc = 0.f;
#pragma unroll
        for (int r = 0; r < kRowsMaxR; ++r) {
            acc = fmaf(row[s][r].x, xv[r].x, acc); acc = fmaf(row[s][r].y, xv[r].y, acc);
            acc = fmaf(row[s][r].z, xv[r].z, acc); acc = fmaf(row[s][r].w, xv[r].w, acc);
        }
        acc = warp_allsum(acc);
        if ((tid & 31) == 0) red[tid >> 5][s] = acc;
    }
    __syncthreads();
    if (tid < kRowsS) {
        const int b = grp * kRowsS + tid;
        float cf = 0.f;
        if (b < Bi) {
            float dot = 0.f;
#pragma unroll
            for (int t = 0; t < kRowsThreads / 32; ++t) dot += red[t][tid];
            const float yv = __ldg(y + (int64_t)node * m + jdx[tid]);
            if (model == DPSGD_MODEL_LSQ) {
                cf = (dot - yv) / (float)Bi;
            } else {
                const float z = dot + __ldg(X + (int64_t)node * ld + d);
                cf = -yv * (1.f / (1.f + expf(yv * z))) / (float)Bi;
            }
        }
        coef[tid] = cf;
    }
    __syncthreads();
    float* out = part + ((int64_t)node * groups + grp) * ld;
#pragma unroll
    for (int r = 0; r < kRowsMaxR; ++r) {
        const int c = tid + r * kRowsThreads;
        if (c < d4) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int s = 0; s < kRowsS; ++s) {
                const float w = coef[s];
                a.x = fmaf(w, row[s][r].x, a.x); a.y = fmaf(w, row[s][r].y, a.y);
                a.z = fmaf(w, row[s][r].z, a.z); a.w = fmaf(w, row[s][r].w, a.w);
            }
            reinterpret_cast<float4*>(out)[c] = a;
        }
    }
    if (tid == 0 && model == DPSGD_MODEL_LOGISTIC) {   // the bias column's share: sum of the coefficients
        float sb = 0.f;
#pragma unroll
        for (int s = 0; s < kRowsS; ++s) sb += coef[s];
        out[d] = sb;
    }
}

// G[node][c] = sum over the groups, in order; + l2 x for the logistic weights; zero beyond the parameters.
__global__ void __launch_bounds__(128)
glm_rows_reduce_kernel(const float* __restrict__ X, float* __restrict__ G, int64_t ld, const float* __restrict__ part,
                       int groups, int d, int model, float l2) {
    const int node = blockIdx.y;
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (c >= ld) return;
    const int last = model == DPSGD_MODEL_LOGISTIC ? d : d - 1;      // last parameter column
    float s = 0.f;
    if (c <= last) {
        const float* p = part + (int64_t)node * groups * ld + c;
        int g = 0;
        for (; g + 8 <= groups; g += 8) {          // eight loads in flight, added in group order
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = __ldg(p + (int64_t)(g + u) * ld);
#pragma unroll
            for (int u = 0; u < 8; ++u) s += v[u];
        }
        for (; g < groups; ++g) s += __ldg(p + (int64_t)g * ld);
        if (model == DPSGD_MODEL_LOGISTIC && c < d) s = fmaf(l2, __ldg(X + (int64_t)node * ld + c), s);
    }
    G[(int64_t)node * ld + c] = s;
}

// The same reduction followed at once by the gossip step of Algorithm 1 (steps 4-5) for its four columns:
// G = sum of the shares (+ l2 x), X_next = sum_j W_ij X_j - gamma G.  For matrices small enough to sit in
// L2, where a separate mixing launch costs more than its work.
__global__ void __launch_bounds__(128)
glm_rows_reduce_mix_kernel(const float4* __restrict__ X, float4* __restrict__ G, float4* __restrict__ Xn, int64_t ld4,
                           const float4* __restrict__ part, int groups, int d, int model, float l2,
                           const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                           const float* __restrict__ val, float ngamma) {
    const int node = blockIdx.y;
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (c >= ld4) return;
    const int last = model == DPSGD_MODEL_LOGISTIC ? d : d - 1;      // last parameter column
    const float4 x = __ldg(X + (int64_t)node * ld4 + c);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (4 * c <= last) {
        const float4* p = part + (int64_t)node * groups * ld4 + c;
        int g = 0;
        for (; g + 8 <= groups; g += 8) {          // eight loads in flight, added in group order
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = __ldg(p + (int64_t)(g + u) * ld4);
#pragma unroll
            for (int u = 0; u < 8; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
        }
        for (; g < groups; ++g) {
            const float4 v = __ldg(p + (int64_t)g * ld4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        const int64_t c0 = 4 * c;
        if (model == DPSGD_MODEL_LOGISTIC) {
            if (c0 < d) s.x = fmaf(l2, x.x, s.x);
            if (c0 + 1 < d) s.y = fmaf(l2, x.y, s.y);
            if (c0 + 2 < d) s.z = fmaf(l2, x.z, s.z);
            if (c0 + 3 < d) s.w = fmaf(l2, x.w, s.w);
        }
        // shares never written beyond the parameters hold stale scratch: zero them
        if (c0 + 1 > last) s.y = 0.f;
        if (c0 + 2 > last) s.z = 0.f;
        if (c0 + 3 > last) s.w = 0.f;
    }
    G[(int64_t)node * ld4 + c] = s;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    const int pe = __ldg(row_ptr + node + 1);
    for (int p = __ldg(row_ptr + node); p < pe; ++p) {
        const float w = __ldg(val + p);
        const float4 v = __ldg(X + (int64_t)__ldg(col + p) * ld4 + c);
        a.x = fmaf(w, v.x, a.x); a.y = fmaf(w, v.y, a.y);
        a.z = fmaf(w, v.z, a.z); a.w = fmaf(w, v.w, a.w);
    }
    a.x = fmaf(ngamma, s.x, a.x); a.y = fmaf(ngamma, s.y, a.y);
    a.z = fmaf(ngamma, s.z, a.z); a.w = fmaf(ngamma, s.w, a.w);
    Xn[(int64_t)node * ld4 + c] = a;
}

// ---- one launch per iteration for small linear models ----
//
// One CTA per node does the node's whole iteration of Algorithm 1: draws the B indices (step 2), stages the
// sampled rows and the node's own x in shared memory, forms the B dot products and coefficients and the
// gradient row (step 3), writes it to G, and applies the gossip step X_next[i] = sum_j W_ij X[j] - gamma g_i
// (steps 4-5).  The update is out of place (neighbours are read from X_k, results go to X_{k+1}), so no CTA
// waits for another.  Every reduction runs in the order of glm_forward_kernel / glm_backward_kernel /
// mix_rowpar_kernel (lanes of a 32-wide xor tree, warps in order, eight interleaved slices of the minibatch
// in order), so the result is bit-identical to the three-launch path.
// Replayed graphs: with k_next != NULL the kernel reads the iteration number from *k_ptr and leaves k + 2 there
// for the launch after next (two slots used alternately by consecutive launches, so no counter kernel runs in
// between and a launch never reads a slot its predecessor writes).  That, and the fact that everything before
// griddepcontrol.wait reads only the dataset (never written by this library), lets consecutive launches of a
// captured chain be programmatic dependents: launch t + 1 draws its indices and gathers its rows while launch
// t is still computing, and touches X, G and the index buffer only after launch t has completed.
constexpr int kNodeThreads = 256;

__global__ void __launch_bounds__(kNodeThreads)
glm_node_step_kernel(const float4* __restrict__ X, float4* __restrict__ G, float4* __restrict__ Xn, int64_t ld,
                     const float* __restrict__ A, const float* __restrict__ y, int64_t m, int d, int B, uint64_t seed,
                     uint64_t k, const uint64_t* __restrict__ k_ptr, uint64_t* __restrict__ k_next, int model, float l2,
                     int32_t* __restrict__ idx, float* __restrict__ coef_out, const int32_t* __restrict__ node_batch,
                     const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                     const float* __restrict__ val, float ngamma) {
    extern __shared__ __align__(16) unsigned char node_smem[];
    const int node = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d4 = d / 4;
    const int64_t ld4 = ld / 4;
    float4* rows = reinterpret_cast<float4*>(node_smem);                   // [B][d4]
    float4* xs = rows + (size_t)B * d4;                                    // [ld4] the node's own row
    float4* gs = xs + ld4;                                                 // [ld4] its gradient row
    float4* ms = gs + ld4;                                                 // [ld4] sum_j W_ij X[j], formed while the rows load
    float4* red = ms + ld4;                                                // [8][32]
    float* scoef = reinterpret_cast<float*>(red + 8 * 32);                 // [B]
    int32_t* sj = reinterpret_cast<int32_t*>(scoef + B);                   // [B]
    float* sy = reinterpret_cast<float*>(sj + B);                          // [B] targets / labels of the draws
    if (k_ptr) k = *k_ptr;                 // written two launches ago: complete before this launch could start
    const int Bi = node_batch ? __ldg(node_batch + node) : B;
    for (int b = tid; b < B; b += kNodeThreads) sj[b] = sample_index(seed, k, (uint32_t)node, (uint32_t)b, (uint32_t)m);
    __syncthreads();
    for (int e = tid; e < B * d4; e += kNodeThreads) {
        const int b = e / d4, c = e - b * d4;
        rows[e] = b < Bi ? __ldg(reinterpret_cast<const float4*>(A + ((int64_t)node * m + sj[b]) * d) + c)
                         : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int b = tid; b < B; b += kNodeThreads) sy[b] = __ldg(y + (int64_t)node * m + sj[b]);   // with the rows, not after the dots
    // ---- everything above read the dataset only; from here on X, G and the scratch of the previous launch ----
    asm volatile("griddepcontrol.wait;" ::: "memory");              // no-op unless launched as a programmatic dependent
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); // the next launch may begin its own gathers
    if (k_next && node == 0 && tid == 0) *k_next = k + 2;
    for (int b = tid; b < B; b += kNodeThreads) idx[node * B + b] = sj[b];
    const int p0 = __ldg(row_ptr + node), pe = __ldg(row_ptr + node + 1);
    for (int64_t c = tid; c < ld4; c += kNodeThreads) {
        xs[c] = __ldg(X + (int64_t)node * ld4 + c);
        // the mixing half of the gossip step needs X_k only: its loads overlap the gathers of the sampled rows
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int p = p0; p < pe; ++p) {
            const float w = __ldg(val + p);
            const float4 v = __ldg(X + (int64_t)__ldg(col + p) * ld4 + c);
            a.x = fmaf(w, v.x, a.x); a.y = fmaf(w, v.y, a.y);
            a.z = fmaf(w, v.z, a.z); a.w = fmaf(w, v.w, a.w);
        }
        ms[c] = a;
    }
    __syncthreads();
    // forward: a warp per draw; lane l of pass w stands for thread 32 w + l of the per-sample CTA
    for (int b = warp; b < B; b += kNodeThreads / 32) {
        float cf = 0.f;
        if (b < Bi) {
            float dot = 0.f;
            // passes beyond the row's last 16-byte column would add 0.0f to dot, which changes nothing: skipped
#pragma unroll 1
            for (int w = 0; w * 32 < d4; ++w) {
                const int c = w * 32 + lane;
                float acc = 0.f;
                if (c < d4) {
                    const float4 a = rows[b * d4 + c], v = xs[c];
                    acc = fmaf(a.x, v.x, acc); acc = fmaf(a.y, v.y, acc);
                    acc = fmaf(a.z, v.z, acc); acc = fmaf(a.w, v.w, acc);
                }
                dot += warp_allsum(acc);
            }
            const float yv = sy[b];
            if (model == DPSGD_MODEL_LSQ) {
                cf = (dot - yv) / (float)Bi;
            } else {
                const float z = dot + reinterpret_cast<const float*>(xs)[d];
                const float s = 1.f / (1.f + expf(yv * z));
                cf = -yv * s / (float)Bi;
            }
        }
        if (lane == 0) { scoef[b] = cf; coef_out[node * B + b] = cf; }
    }
    __syncthreads();
    // backward: 32 column groups x 8 interleaved slices of the minibatch, slices added in order
    const int tx = lane, ty = warp;
    for (int c0 = 0; c0 < d4; c0 += 32) {
        const int cg = c0 + tx;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (cg < d4) {
            for (int b = ty; b < Bi; b += 8) {
                const float w = scoef[b];
                const float4 a = rows[b * d4 + cg];
                acc.x = fmaf(w, a.x, acc.x); acc.y = fmaf(w, a.y, acc.y);
                acc.z = fmaf(w, a.z, acc.z); acc.w = fmaf(w, a.w, acc.w);
            }
        }
        red[ty * 32 + tx] = acc;
        __syncthreads();
        if (ty == 0 && cg < d4) {
            float4 s = red[tx];
#pragma unroll
            for (int t = 1; t < 8; ++t) {
                const float4 r = red[t * 32 + tx];
                s.x += r.x; s.y += r.y; s.z += r.z; s.w += r.w;
            }
            if (model == DPSGD_MODEL_LOGISTIC) {
                const float4 x = xs[cg];
                s.x = fmaf(l2, x.x, s.x); s.y = fmaf(l2, x.y, s.y); s.z = fmaf(l2, x.z, s.z); s.w = fmaf(l2, x.w, s.w);
            }
            gs[cg] = s;
        }
        __syncthreads();
    }
    if (ty == 1) {          // bias gradient (logistic) and zero padding: columns [d, ld)
        for (int64_t c = d + tx; c < ld; c += 32) {
            float s = 0.f;
            if (model == DPSGD_MODEL_LOGISTIC && c == d)
                for (int b = 0; b < Bi; ++b) s += scoef[b];
            reinterpret_cast<float*>(gs)[c] = s;
        }
    }
    __syncthreads();
    // gradient row out, then the update half of the gossip step on this node's row
    for (int64_t c = tid; c < ld4; c += kNodeThreads) {
        const float4 g = gs[c];
        G[(int64_t)node * ld4 + c] = g;
        float4 a = ms[c];
        a.x = fmaf(ngamma, g.x, a.x); a.y = fmaf(ngamma, g.y, a.y);
        a.z = fmaf(ngamma, g.z, a.z); a.w = fmaf(ngamma, g.w, a.w);
        Xn[(int64_t)node * ld4 + c] = a;
    }
}

size_t node_step_smem(const dpsgd_ctx* c) {
    return sizeof(float) * ((size_t)c->batch * c->d + 3 * (size_t)c->ld + 8 * 32 * 4 + 3 * (size_t)c->batch);
}

bool rows_path(const dpsgd_ctx* c) {
    return c->d % 4 == 0 && c->d >= 1024 && c->d <= 16 * kRowsThreads * kRowsMaxR / 4 && c->n <= 65535;
}

// First half of the rows-in-registers gradient: the shares of every group of four draws.
cudaError_t launch_rows(dpsgd_ctx* c, uint64_t k, const float* X, int* groups_out) {
    const int n = c->n, B = c->batch;
    const int groups = (B + kRowsS - 1) / kRowsS;
    const size_t need = (size_t)n * groups * c->ld;
    if (c->glm_part_floats < need) {
        cudaFree(c->d_glm_part);
        c->d_glm_part = nullptr; c->glm_part_floats = 0;
        cudaError_t e = cudaMalloc(&c->d_glm_part, need * sizeof(float));
        if (e != cudaSuccess) return e;
        c->glm_part_floats = need;
    }
    glm_rows_kernel<<<dim3(groups, n), kRowsThreads, 0, c->stream>>>(
        X, c->ld, c->A, static_cast<const float*>(c->y), c->m, c->d, B, c->seed, k, c->k_dev_active, c->model,
        c->d_idx, c->d_glm_part, groups, c->d_node_batch);
    c->launches++;
    *groups_out = groups;
    return cudaGetLastError();
}

}  // namespace

// Narrow rows on a small matrix: the whole iteration in ONE launch (a CTA per node).
bool linear_node_step_fuses(const dpsgd_ctx* c) {
    return c->model != DPSGD_MODEL_MLP && !rows_path(c) && c->d % 4 == 0 && c->d < 1024 && c->batch <= 1024 &&
           (int64_t)c->batch * c->d <= 8192 && c->ld <= 2048 && !c->kind_forced && mix_is_small(c) && !c->swapped &&
           c->V == nullptr && c->n <= 65535;
}

// Whole iteration of a linear model in one launch (narrow rows) or two (wide rows: shares of the gradient,
// then their reduction and the gossip step together).  False when the shapes or the options call for the
// separate stages.
bool linear_step_fuses(const dpsgd_ctx* c) {
    if (linear_node_step_fuses(c)) return true;
    return c->model != DPSGD_MODEL_MLP && rows_path(c) && !c->kind_forced && mix_is_small(c) && !c->swapped &&
           c->V == nullptr;
}

cudaError_t launch_linear_step(dpsgd_ctx* c, uint64_t k, const float* X, float* G, float* Xn) {
    if (linear_node_step_fuses(c)) {
        const size_t smem = node_step_smem(c);
        cudaError_t e = cudaFuncSetAttribute(glm_node_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        // inside a captured chain (k_dev_next set) every launch after the first is a programmatic dependent of the one before
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)c->n); cfg.blockDim = dim3(kNodeThreads); cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = (c->k_dev_next && c->chain_pos > 0) ? 1 : 0;
        e = cudaLaunchKernelEx(&cfg, glm_node_step_kernel, reinterpret_cast<const float4*>(X), reinterpret_cast<float4*>(G),
                               reinterpret_cast<float4*>(Xn), c->ld, c->A, static_cast<const float*>(c->y), c->m, c->d,
                               c->batch, c->seed, k, c->k_dev_active, c->k_dev_next, c->model, c->l2, c->d_idx, c->d_coef,
                               (const int32_t*)c->d_node_batch, c->W.row_ptr, c->W.col, c->W.val, -c->gamma);
        c->launches++;
        return e != cudaSuccess ? e : cudaGetLastError();
    }
    int groups = 0;
    cudaError_t e = launch_rows(c, k, X, &groups);
    if (e != cudaSuccess) return e;
    const int64_t ld4 = c->ld / 4;
    glm_rows_reduce_mix_kernel<<<dim3((unsigned)((ld4 + 127) / 128), c->n), 128, 0, c->stream>>>(
        reinterpret_cast<const float4*>(X), reinterpret_cast<float4*>(G), reinterpret_cast<float4*>(Xn), ld4,
        reinterpret_cast<const float4*>(c->d_glm_part), groups, c->d, c->model, c->l2, c->W.row_ptr, c->W.col,
        c->W.val, -c->gamma);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_grad_linear(dpsgd_ctx* c, uint64_t k, const float* X, float* G) {
    const int n = c->n, B = c->batch, d = c->d;
    const float* y = static_cast<const float*>(c->y);
    const bool vec = (d % 4 == 0);
    if (rows_path(c)) {
        // one read of the sampled rows: they stay in registers between the forward and the backward part
        // (rows of a few hundred bytes leave most of such a CTA idle: they keep the two kernels below)
        int groups = 0;
        cudaError_t e = launch_rows(c, k, X, &groups);
        if (e != cudaSuccess) return e;
        glm_rows_reduce_kernel<<<dim3((unsigned)((c->ld + 127) / 128), n), 128, 0, c->stream>>>(
            X, G, c->ld, c->d_glm_part, groups, d, c->model, c->l2);
        c->launches++;
        return cudaGetLastError();
    }
    const int fwd_grid = n * B;
    if (vec)
        glm_forward_kernel<4><<<fwd_grid, kFwdThreads, 0, c->stream>>>(
            X, c->ld, c->A, y, c->m, d, B, n, c->seed, k, c->k_dev_active, c->model, c->d_idx, c->d_coef,
            c->d_node_batch);
    else
        glm_forward_kernel<1><<<fwd_grid, kFwdThreads, 0, c->stream>>>(
            X, c->ld, c->A, y, c->m, d, B, n, c->seed, k, c->k_dev_active, c->model, c->d_idx, c->d_coef,
            c->d_node_batch);
    const int vw = vec ? 4 : 1;
    dim3 grid((d + 32 * vw - 1) / (32 * vw), n), block(32, 8);
    if (vec)
        glm_backward_kernel<4><<<grid, block, 0, c->stream>>>(X, G, c->ld, c->A, c->m, d, B, c->model,
                                                              c->l2, c->d_idx, c->d_coef, c->d_node_batch);
    else
        glm_backward_kernel<1><<<grid, block, 0, c->stream>>>(X, G, c->ld, c->A, c->m, d, B, c->model,
                                                              c->l2, c->d_idx, c->d_coef, c->d_node_batch);
    c->launches += 2;
    return cudaGetLastError();
}

}  // namespace dpsgd
