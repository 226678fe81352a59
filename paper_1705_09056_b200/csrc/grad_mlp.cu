// Algorithm 1 steps 2-3 for the MLP: every node's minibatch gradient of the softmax
// cross-entropy of a ReLU network at its own parameters x_{k,i} (one column of dF(X_k; xi_k),
// Section 3), as the mean over the B sampled examples (footnote a).
//
// Parameter row layout: [W_1 (d_1 x d_0, row-major) | b_1 | W_2 | b_2 | ...].
// Per node i, with h_0 the gathered inputs [B][d_0]:
//     h_l     = relu(h_{l-1} W_l^T + b_l)        l = 1..L-1,   h_L = h_{L-1} W_L^T + b_L (logits)
//     delta_L = (softmax(h_L) - onehot(y)) / B
//     gW_l    = delta_l^T h_{l-1},   gb_l = sum_b delta_l[b],
//     delta_{l-1} = (delta_l W_l) * [h_{l-1} > 0]                      (ReLU'(0) = 0)
// All three products are batched GEMMs over the n nodes with per-node operands.  They run on the
// tensor cores (tcgen05 TF32 MMAs, three per product for fp32-faithful results) when the minibatch
// fits a 128-column tile: forward and input gradient on the weight-streaming kernel of tc_stream.cuh,
// the weight gradient on tc_wgrad.cuh (both TMA-fed, weight-side operand in tensor memory), the
// classifier layer's backward on the fp32 kernel of grad_mlp_narrow.cuh, and shapes TMA cannot
// address (rows not 16-byte aligned) on the register-staged kernel of tc_gemm.cuh.  Otherwise - or
// when asked - everything runs on the fp32 FMA kernel below (exact fp32 products, fp32 accumulation
// in a fixed order).
#include <algorithm>

#include "ctx.h"
#include "philox.cuh"
#include "grad_mlp_narrow.cuh"
#include "tc_gemm.cuh"
#include "tc_stream.cuh"
#include "tc_wgrad.cuh"
#include "tma_host.h"

namespace dpsgd {
namespace {

// activations: h_l of every node, l = 0..L, stored [l][node][B][d_l]
struct MlpPlan {
    int L;
    int B;
    int n;
    size_t act_off[kMaxLayers + 2];
    size_t delta_off[kMaxLayers + 1];   // delta_l for l = 1..L, stored [l][node][B][pitch_l]
    int delta_pitch[kMaxLayers + 1];    // d_l; the output layer's rounded up to 4 floats (16-byte rows for TMA)
};

int delta_row_floats(const dpsgd_ctx* c, int l) {
    const int d = c->mlp.dims[l];
    return l == c->mlp.nlayers ? (d + 3) & ~3 : d;
}

MlpPlan make_plan(const dpsgd_ctx* c) {
    MlpPlan p{};
    p.L = c->mlp.nlayers; p.B = c->batch; p.n = c->n;
    size_t a = 0, d = 0;
    for (int l = 0; l <= p.L; ++l) {
        p.act_off[l] = a;
        a += (size_t)c->n * c->batch * c->mlp.dims[l];
        p.delta_off[l] = d;
        p.delta_pitch[l] = delta_row_floats(c, l);
        if (l >= 1) d += (size_t)c->n * c->batch * p.delta_pitch[l];
    }
    return p;
}

// h_0[node][b][:] = A[node][idx][:] with idx drawn for (iteration k, node, b).
__global__ void __launch_bounds__(128)
mlp_gather_kernel(const float* __restrict__ A, int64_t m, int d, int B, uint64_t seed, uint64_t k,
                  const uint64_t* __restrict__ k_ptr, int32_t* __restrict__ idx, float* __restrict__ h0) {
    if (k_ptr) k = *k_ptr;        // iteration counter kept on the device (graph replay)
    const int node = blockIdx.y, b = blockIdx.x;
    const int32_t j = sample_index(seed, k, (uint32_t)node, (uint32_t)b, (uint32_t)m);
    if (threadIdx.x == 0) idx[node * B + b] = j;
    const float* src = A + ((int64_t)node * m + j) * d;
    float* dst = h0 + ((int64_t)node * B + b) * d;
    if ((d & 3) == 0) {
        for (int c = threadIdx.x; c < d / 4; c += 128)
            reinterpret_cast<float4*>(dst)[c] = __ldg(reinterpret_cast<const float4*>(src) + c);
    } else {
        for (int c = threadIdx.x; c < d; c += 128) dst[c] = __ldg(src + c);
    }
}

enum { EPI_BIAS_RELU = 0, EPI_BIAS = 1, EPI_STORE = 2, EPI_MASK = 3 };

struct GemmArgs {
    const float* A; int64_t a_node, a_m, a_k;   // element strides: per node, along m, along k
    const float* Bm; int64_t b_node, b_n, b_k;
    float* C; int64_t c_node, c_m;              // C[m][n], n contiguous
    const float* aux; int64_t aux_node, aux_m;  // bias[n] (aux_m = 0) or mask source [m][n]
    int M, N, K;
};

// C[m][n] = sum_k A(m,k) * B(n,k) per node, 64x64x16 tiles, 256 threads, 4x4 outputs per thread.
// A_K / B_K say whether the operand is contiguous along k (else along m / n).
template <bool A_K, bool B_K, int EPI>
__global__ void __launch_bounds__(256)
bgemm_kernel(GemmArgs g) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int node = blockIdx.z;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const float* A = g.A + (int64_t)node * g.a_node;
    const float* Bp = g.Bm + (int64_t)node * g.b_node;
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < g.K; k0 += BK) {
        // 64 x 16 elements per operand, 4 per thread
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int e = tid + t * 256;
            int mm, kk;
            if (A_K) { kk = e % BK; mm = e / BK; } else { mm = e % BM; kk = e / BM; }
            const int gm = m0 + mm, gk = k0 + kk;
            As[kk][mm] = (gm < g.M && gk < g.K) ? __ldg(A + (int64_t)gm * g.a_m + (int64_t)gk * g.a_k) : 0.f;
            int nn, kb;
            if (B_K) { kb = e % BK; nn = e / BK; } else { nn = e % BN; kb = e / BN; }
            const int gn = n0 + nn, gkb = k0 + kb;
            Bs[kb][nn] = (gn < g.N && gkb < g.K) ? __ldg(Bp + (int64_t)gn * g.b_n + (int64_t)gkb * g.b_k) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* C = g.C + (int64_t)node * g.c_node;
    const float* aux = g.aux ? g.aux + (int64_t)node * g.aux_node : nullptr;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= g.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= g.N) continue;
            float v = acc[i][j];
            if (EPI == EPI_BIAS_RELU) { v += __ldg(aux + gn); v = v > 0.f ? v : 0.f; }
            if (EPI == EPI_BIAS) v += __ldg(aux + gn);
            if (EPI == EPI_MASK) v = __ldg(aux + (int64_t)gm * g.aux_m + gn) > 0.f ? v : 0.f;
            C[(int64_t)gm * g.c_m + gn] = v;
        }
    }
}

// delta_L[b][:] = (softmax(logits[b]) - onehot(y[idx[b]])) / B_i; one warp per (node, sample).
// Columns b >= B_i (a node with a smaller minibatch) get delta = 0 and so drop out of every
// product of the backward pass.
__global__ void __launch_bounds__(128)
softmax_ce_delta_kernel(const float* __restrict__ logits, const int32_t* __restrict__ y, int64_t m,
                        const int32_t* __restrict__ idx, int n, int B, int C, float* __restrict__ delta,
                        int dpitch, const int32_t* __restrict__ node_batch) {
    const int w = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (w >= n * B) return;
    const int node = w / B;
    const int Bi = node_batch ? __ldg(node_batch + node) : B;
    if (w - node * B >= Bi) {
        for (int c = lane; c < C; c += 32) delta[(int64_t)w * dpitch + c] = 0.f;
        return;
    }
    const float* z = logits + (int64_t)w * C;
    float mx = -INFINITY;
    for (int c = lane; c < C; c += 32) mx = fmaxf(mx, z[c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float s = 0.f;
    for (int c = lane; c < C; c += 32) s += expf(z[c] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const int label = __ldg(y + (int64_t)node * m + __ldg(idx + w));
    const float inv = 1.f / s, invB = 1.f / (float)Bi;
    for (int c = lane; c < C; c += 32)
        delta[(int64_t)w * dpitch + c] = (expf(z[c] - mx) * inv - (c == label ? 1.f : 0.f)) * invB;
}

// gb[o] = sum_b delta[b][o], written into the gradient row; fixed order over b.
__global__ void __launch_bounds__(128)
bias_grad_kernel(const float* __restrict__ delta, int B, int D, int dpitch, float* __restrict__ G, int64_t ld,
                 int64_t b_off) {
    const int node = blockIdx.y;
    const int o = blockIdx.x * 128 + threadIdx.x;
    if (o >= D) return;
    const float* d = delta + (int64_t)node * B * dpitch + o;
    float s = 0.f;
    for (int b = 0; b < B; ++b) s += d[(int64_t)b * dpitch];
    G[(int64_t)node * ld + b_off + o] = s;
}

__global__ void zero_pad_kernel(float* __restrict__ G, int64_t ld, int64_t N, int n) {
    const int64_t width = ld - N;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= width * n) return;
    G[(t / width) * ld + N + (t % width)] = 0.f;
}

template <bool A_K, bool B_K, int EPI>
void run_gemm(dpsgd_ctx* c, const GemmArgs& g) {
    dim3 grid((g.N + 63) / 64, (g.M + 63) / 64, c->n);
    bgemm_kernel<A_K, B_K, EPI><<<grid, 256, 0, c->stream>>>(g);
    c->launches++;
}

template <int NT, bool A_K, bool B_K, bool VEC, bool PRECISE>
cudaError_t launch_tc_inst(dpsgd_ctx* c, const tc::Args& a, int n_tiles, int problems) {
    auto kernel = tc::tc_gemm_kernel<NT, A_K, B_K, VEC, PRECISE>;
    constexpr size_t smem = tc::smem_bytes<NT, A_K, B_K, PRECISE>();
    // per device and cheap: set on every launch rather than remembered in a process-wide flag
    cudaError_t ea = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (ea != cudaSuccess) return ea;
    dim3 grid((a.M + tc::kTileM - 1) / tc::kTileM, (n_tiles + a.n_per_cta - 1) / a.n_per_cta, problems);
    kernel<<<grid, tc::kThreads, smem, c->stream>>>(a);
    c->launches++;
    return cudaGetLastError();
}

template <int NT, bool VEC>
cudaError_t launch_tc_nt(dpsgd_ctx* c, const tc::Args& a, int n_tiles, int problems) {
    if (a.precise) {
        if (a.a_kcontig && a.b_kcontig) return launch_tc_inst<NT, true, true, VEC, true>(c, a, n_tiles, problems);
        if (!a.a_kcontig && a.b_kcontig) return launch_tc_inst<NT, false, true, VEC, true>(c, a, n_tiles, problems);
        if (!a.a_kcontig && !a.b_kcontig) return launch_tc_inst<NT, false, false, VEC, true>(c, a, n_tiles, problems);
    } else {
        if (a.a_kcontig && a.b_kcontig) return launch_tc_inst<NT, true, true, VEC, false>(c, a, n_tiles, problems);
        if (!a.a_kcontig && a.b_kcontig) return launch_tc_inst<NT, false, true, VEC, false>(c, a, n_tiles, problems);
        if (!a.a_kcontig && !a.b_kcontig) return launch_tc_inst<NT, false, false, VEC, false>(c, a, n_tiles, problems);
    }
    return cudaErrorInvalidValue;
}

// 128-bit loads need 16-byte aligned rows and whole chunks inside the matrix: the extent of the
// operand's contiguous direction (which equals its pitch here) must be a multiple of 4.
bool vec_ok(const float* p, int64_t pitch, int64_t node_stride, int contig_extent) {
    return (reinterpret_cast<uintptr_t>(p) % 16 == 0) && (pitch % 4 == 0) && (node_stride % 4 == 0) &&
           (contig_extent % 4 == 0);
}

// C[n][m] = epi(sum_k A(m,k) B(n,k)); max_tile = widest column tile (multiple of 16, <= 128).
// problems: independent problems in the launch (blockIdx.z), one per node unless given; force_precise: three
// MMAs per product whatever the model's precision setting.
cudaError_t run_tc(dpsgd_ctx* c, tc::Args a, int max_tile, int problems = -1, bool force_precise = false) {
    if (problems < 0) problems = c->n;
    const bool vec = vec_ok(a.A, a.a_pitch, a.a_node, a.a_kcontig ? a.K : a.M) &&
                     vec_ok(a.B, a.b_pitch, a.b_node, a.b_kcontig ? a.K : a.N);
    a.a_vec = a.b_vec = vec;
    a.precise = force_precise || c->mlp_precision == 0;
    a.status = &c->d_result->status;
    const int want = a.N < max_tile ? a.N : max_tile;
    {   // column tiles per CTA: up to 8 (keeps the A tile staged), but never so many that the grid
        // falls under about four CTAs per CTA slot of the device
        const int tile = want <= 16 ? 16 : (want <= 32 ? 32 : (want <= 64 ? 64 : 128));
        const long long tiles = (long long)((a.M + tc::kTileM - 1) / tc::kTileM) * ((a.N + tile - 1) / tile) * problems;
        const long long per = tiles / (4LL * 2 * 148);
        a.n_per_cta = (int)(per < 1 ? 1 : (per > 8 ? 8 : per));
    }
    if (vec) {
        if (want <= 16) return launch_tc_nt<1, true>(c, a, (a.N + 15) / 16, problems);
        if (want <= 32) return launch_tc_nt<2, true>(c, a, (a.N + 31) / 32, problems);
        if (want <= 64) return launch_tc_nt<4, true>(c, a, (a.N + 63) / 64, problems);
        return launch_tc_nt<8, true>(c, a, (a.N + 127) / 128, problems);
    }
    if (want <= 16) return launch_tc_nt<1, false>(c, a, (a.N + 15) / 16, problems);
    if (want <= 32) return launch_tc_nt<2, false>(c, a, (a.N + 31) / 32, problems);
    if (want <= 64) return launch_tc_nt<4, false>(c, a, (a.N + 63) / 64, problems);
    return launch_tc_nt<8, false>(c, a, (a.N + 127) / 128, problems);
}

// ---- weight-streaming kernel (tc_stream.cuh): forward and input-gradient products ----

template <int NT, bool A_K, bool PRECISE>
cudaError_t launch_tcs_inst(dpsgd_ctx* c, const CUtensorMap& mapA, const CUtensorMap& mapB, tcs::Args a) {
    auto kernel = tcs::tc_stream_kernel<NT, A_K, PRECISE>;
    constexpr size_t smem = tcs::smem_bytes<NT, PRECISE>();
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                  cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
    int sms = 0, dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int per_sm = NT <= 4 ? 2 : 1;                          // what the kernel's shared memory allows
    const int grid = std::min(a.total_tiles, sms * per_sm);      // persistent CTAs
    // the tiles left over after the rounds that fill every CTA are cut by k-blocks and finished by stream_fixup_kernel
    const int left_tiles = a.total_tiles % grid;
    const bool cut = left_tiles != 0;
    if (cut && (!c->d_stream_parts || (size_t)grid * 2 * 16 * NT * tcs::kTileM > c->stream_parts_floats)) return cudaErrorNotSupported;
    a.partial = c->d_stream_parts;
    kernel<<<grid, tcs::kThreads, smem, c->stream>>>(mapA, mapB, a);
    c->launches++;
    if ((e = cudaGetLastError()) != cudaSuccess || !cut) return e;
    tcs::stream_fixup_kernel<<<dim3(left_tiles, a.N), tcs::kTileM, 0, c->stream>>>(a, 16 * NT, grid);
    c->launches++;
    return cudaGetLastError();
}

template <int NT>
cudaError_t launch_tcs_nt(dpsgd_ctx* c, const CUtensorMap& mapA, const CUtensorMap& mapB, const tcs::Args& a,
                          bool a_kcontig, bool precise) {
    if (a_kcontig) return precise ? launch_tcs_inst<NT, true, true>(c, mapA, mapB, a)
                                  : launch_tcs_inst<NT, true, false>(c, mapA, mapB, a);
    return precise ? launch_tcs_inst<NT, false, true>(c, mapA, mapB, a)
                   : launch_tcs_inst<NT, false, false>(c, mapA, mapB, a);
}

// The TMA loads need 16-byte aligned bases and strides, B contiguous along k and one column tile
// for the whole minibatch.
bool stream_ok(const tc::Args& a) {
    auto al = [](const float* p, int64_t pitch, int64_t node) {
        return reinterpret_cast<uintptr_t>(p) % 16 == 0 && pitch % 4 == 0 && node % 4 == 0;
    };
    return a.b_kcontig && a.N <= 128 && al(a.A, a.a_pitch, a.a_node) && al(a.B, a.b_pitch, a.b_node);
}

// Returns cudaErrorNotSupported when the tensor maps cannot be built (the caller falls back).
cudaError_t run_tcs(dpsgd_ctx* c, const tc::Args& t) {
    const int rows_b = t.N <= 16 ? 16 : (t.N <= 32 ? 32 : (t.N <= 64 ? 64 : 128));
    CUtensorMap mapA, mapB;
    const uint64_t nodes = (uint64_t)c->n;
    bool ok;
    if (t.a_kcontig)     // A(m,k) at m*pitch + k
        ok = make_map_3d(&mapA, t.A, (uint64_t)t.K, (uint64_t)t.M, nodes, (uint64_t)t.a_pitch * 4,
                         (uint64_t)t.a_node * 4, tcs::kBK, tcs::kTileM, true);
    else                 // A(m,k) at k*pitch + m
        ok = make_map_3d(&mapA, t.A, (uint64_t)t.M, (uint64_t)t.K, nodes, (uint64_t)t.a_pitch * 4,
                         (uint64_t)t.a_node * 4, tcs::kTileM, tcs::kBK, false);
    ok = ok && make_map_3d(&mapB, t.B, (uint64_t)t.K, (uint64_t)t.N, nodes, (uint64_t)t.b_pitch * 4,
                           (uint64_t)t.b_node * 4, tcs::kBK, (uint32_t)rows_b, true);
    if (!ok) return cudaErrorNotSupported;
    tcs::Args a{};
    a.C = t.C; a.c_node = t.c_node; a.c_pitch = t.c_pitch;
    a.aux = t.aux; a.aux_node = t.aux_node; a.aux_pitch = t.aux_pitch;
    a.M = t.M; a.N = t.N; a.K = t.K;
    a.m_tiles = (t.M + tcs::kTileM - 1) / tcs::kTileM;
    a.total_tiles = a.m_tiles * c->n;
    a.epi = t.epi;
    a.status = &c->d_result->status;
    const bool precise = c->mlp_precision == 0;
    switch (rows_b) {
        case 16: return launch_tcs_nt<1>(c, mapA, mapB, a, t.a_kcontig != 0, precise);
        case 32: return launch_tcs_nt<2>(c, mapA, mapB, a, t.a_kcontig != 0, precise);
        case 64: return launch_tcs_nt<4>(c, mapA, mapB, a, t.a_kcontig != 0, precise);
        default: return launch_tcs_nt<8>(c, mapA, mapB, a, t.a_kcontig != 0, precise);
    }
}

// ---- weight-gradient kernel (tc_wgrad.cuh) ----

template <int NT, bool PRECISE>
cudaError_t launch_tcw_inst(dpsgd_ctx* c, const CUtensorMap& mapA, const CUtensorMap& mapB, const CUtensorMap& mapC,
                            tcw::Args a) {
    auto kernel = tcw::tc_wgrad_kernel<NT, PRECISE>;
    constexpr size_t smem = tcw::smem_bytes<NT, PRECISE>();
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int sms = 0, dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    // items = (node, 128-row block, run of column tiles): enough of them to balance the persistent CTAs
    const long long blocks = (long long)c->n * a.m_tiles;
    int chunks = (int)std::min<long long>(a.n_tiles, std::max<long long>(1, (12LL * sms + blocks - 1) / blocks));
    a.chunk = (a.n_tiles + chunks - 1) / chunks;
    a.chunks = (a.n_tiles + a.chunk - 1) / a.chunk;
    a.nodes = c->n; a.splits = c->n; a.split_len = 1;            // node-major order
    a.total_seqs = (int)(blocks * a.chunks);
    const int grid = std::min(a.total_seqs, sms);                // one persistent CTA per SM
    kernel<<<grid, tcw::kThreads, smem, c->stream>>>(mapA, mapB, mapC, a);
    c->launches++;
    return cudaGetLastError();
}

// gW[o][k'] = sum_b delta[b][o] h[b][k'] for every node.  Returns cudaErrorNotSupported when the
// shapes or alignments rule the TMA path out (the caller falls back).
cudaError_t run_tcw(dpsgd_ctx* c, const float* h, int din, const float* delta, int dout, int dpitch, float* gW) {
    const int B = c->batch;
    auto al = [](const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; };
    if (B > tcw::kMaxK || din % 4 != 0 || dpitch % 4 != 0 || !al(h) || !al(delta) || !al(gW) || c->ld % 4 != 0)
        return cudaErrorNotSupported;
    const int rows_b = dout <= 16 ? 16 : (dout <= 32 ? 32 : 64);
    const uint64_t nodes = (uint64_t)c->n;
    CUtensorMap mapA, mapB, mapC;
    bool ok = make_map_3d(&mapA, h, (uint64_t)din, (uint64_t)B, nodes, (uint64_t)din * 4, (uint64_t)B * din * 4,
                          tcw::kTileM, tcw::kMaxK, false);
    ok = ok && make_map_3d(&mapB, delta, (uint64_t)dout, (uint64_t)B, nodes, (uint64_t)dpitch * 4,
                           (uint64_t)B * dpitch * 4, (uint32_t)rows_b, tcw::kMaxK, false);
    ok = ok && make_map_3d(&mapC, gW, (uint64_t)din, (uint64_t)dout, nodes, (uint64_t)din * 4, (uint64_t)c->ld * 4,
                           tcw::kTileM, (uint32_t)rows_b, false);
    if (!ok) return cudaErrorNotSupported;
    tcw::Args a{};
    a.M = din; a.N = dout; a.K = B;
    a.m_tiles = (din + tcw::kTileM - 1) / tcw::kTileM;
    a.n_tiles = (dout + rows_b - 1) / rows_b;
    a.status = &c->d_result->status;
    const bool precise = c->mlp_precision == 0;
    switch (rows_b) {
        case 16: return precise ? launch_tcw_inst<1, true>(c, mapA, mapB, mapC, a) : launch_tcw_inst<1, false>(c, mapA, mapB, mapC, a);
        case 32: return precise ? launch_tcw_inst<2, true>(c, mapA, mapB, mapC, a) : launch_tcw_inst<2, false>(c, mapA, mapB, mapC, a);
        default: return precise ? launch_tcw_inst<4, true>(c, mapA, mapB, mapC, a) : launch_tcw_inst<4, false>(c, mapA, mapB, mapC, a);
    }
}

// Forward / input-gradient product: the streaming kernel when its loads are legal, else the
// register-staged one.
cudaError_t run_tc_weights(dpsgd_ctx* c, const tc::Args& a) {
    if (stream_ok(a)) {
        const cudaError_t e = run_tcs(c, a);
        if (e != cudaErrorNotSupported) return e;
    }
    return run_tc(c, a, 128);
}

}  // namespace

// Batched GEMM with both operands contiguous along k, for callers outside this file:
//     C[p][nn * c_pitch + m] = sum_k A[p][m * a_pitch + k] * B[p][nn * b_pitch + k],   p < problems,
// on the register-staged tensor-core kernel (tc_gemm.cuh), three TF32 MMAs per product.
cudaError_t launch_tc_gemm_kmajor(dpsgd_ctx* c, const float* A, int64_t a_problem, int64_t a_pitch, const float* B,
                                  int64_t b_problem, int64_t b_pitch, float* C, int64_t c_problem, int64_t c_pitch,
                                  int M, int N, int K, int problems) {
    tc::Args a{};
    a.A = A; a.a_node = a_problem; a.a_pitch = a_pitch; a.a_kcontig = 1;
    a.B = B; a.b_node = b_problem; a.b_pitch = b_pitch; a.b_kcontig = 1;
    a.C = C; a.c_node = c_problem; a.c_pitch = c_pitch;
    a.aux = nullptr; a.aux_node = 0; a.aux_pitch = 0;
    a.M = M; a.N = N; a.K = K;
    a.epi = tc::EPI_STORE;
    return run_tc(c, a, 128, problems, true);
}

size_t mlp_act_floats(const dpsgd_ctx* c) {
    size_t a = 0;
    for (int l = 0; l <= c->mlp.nlayers; ++l) a += (size_t)c->n * c->batch * c->mlp.dims[l];
    return a;
}

// Scratch of the weight-streaming kernel: two 128 x 128 accumulator tiles per persistent CTA (two CTAs per SM).
size_t mlp_stream_parts_floats(int sms) { return (size_t)sms * 2 * 2 * 128 * tcs::kTileM; }

size_t mlp_delta_floats(const dpsgd_ctx* c) {
    size_t a = 0;
    for (int l = 1; l <= c->mlp.nlayers; ++l) a += (size_t)c->n * c->batch * delta_row_floats(c, l);
    return a;
}

cudaError_t launch_grad_mlp(dpsgd_ctx* c, uint64_t k, const float* X, float* G, float* Xn) {
    const MlpPlan p = make_plan(c);
    c->fused_blocks.clear();
    const MlpShape& s = c->mlp;
    const int n = c->n, B = c->batch, L = s.nlayers;
    const int32_t* y = static_cast<const int32_t*>(c->y);
    const bool use_tc = c->mlp_precision != 2 && B <= 128;   // precision 2 = fp32 FMA kernel

    mlp_gather_kernel<<<dim3(B, n), 128, 0, c->stream>>>(c->A, c->m, s.dims[0], B, c->seed, k, c->k_dev_active, c->d_idx,
                                                         c->d_act + p.act_off[0]);
    c->launches++;

    // forward
    for (int l = 1; l <= L; ++l) {
        const int din = s.dims[l - 1], dout = s.dims[l];
        GemmArgs g{};
        g.A = c->d_act + p.act_off[l - 1]; g.a_node = (int64_t)B * din; g.a_m = din; g.a_k = 1;
        g.Bm = X + s.w_off[l - 1]; g.b_node = c->ld; g.b_n = din; g.b_k = 1;
        g.C = c->d_act + p.act_off[l]; g.c_node = (int64_t)B * dout; g.c_m = dout;
        g.aux = X + s.b_off[l - 1]; g.aux_node = c->ld; g.aux_m = 0;
        g.M = B; g.N = dout; g.K = din;
        if (use_tc && l == L && dout <= narrow::kMaxOut && din % 4 == 0 && s.w_off[l - 1] % 4 == 0 &&
            reinterpret_cast<uintptr_t>(X) % 16 == 0 && reinterpret_cast<uintptr_t>(g.A) % 16 == 0) {
            // classifier layer: a CTA per (node, four samples) on the fp32 pipes
            narrow::narrow_forward_kernel<<<dim3((B + narrow::kFwdSamples - 1) / narrow::kFwdSamples, n),
                                            narrow::kFwdThreads, 0, c->stream>>>(
                X, c->ld, s.w_off[l - 1], s.b_off[l - 1], g.A, g.C, B, din, dout);
            c->launches++;
        } else if (use_tc) {   // m = output unit, n = sample: h_l[b][o]
            tc::Args a{};
            a.A = g.Bm; a.a_node = g.b_node; a.a_pitch = din; a.a_kcontig = 1;
            a.B = g.A; a.b_node = g.a_node; a.b_pitch = din; a.b_kcontig = 1;
            a.C = g.C; a.c_node = g.c_node; a.c_pitch = dout;
            a.aux = g.aux; a.aux_node = g.aux_node; a.aux_pitch = 0;
            a.M = dout; a.N = B; a.K = din; a.epi = l < L ? tc::EPI_BIAS_RELU : tc::EPI_BIAS;
            cudaError_t e = run_tc_weights(c, a);
            if (e != cudaSuccess) return e;
        } else if (l < L) run_gemm<true, true, EPI_BIAS_RELU>(c, g);
        else run_gemm<true, true, EPI_BIAS>(c, g);
    }

    softmax_ce_delta_kernel<<<(n * B + 3) / 4, 128, 0, c->stream>>>(
        c->d_act + p.act_off[L], y, c->m, c->d_idx, n, B, s.dims[L], c->d_delta + p.delta_off[L],
        p.delta_pitch[L], c->d_node_batch);
    c->launches++;

    // backward
    for (int l = L; l >= 1; --l) {
        const int din = s.dims[l - 1], dout = s.dims[l];
        const float* delta = c->d_delta + p.delta_off[l];
        const int dp = p.delta_pitch[l];      // floats per sample in delta_l
        if (use_tc && l == L && dout <= narrow::kMaxOut && (size_t)B * narrow::kMaxOut * sizeof(float) <= 32 * 1024) {
            // classifier layer: weight gradient and the error passed on, in one pass over h_{l-1}
            auto a16 = [](const void* q) { return reinterpret_cast<uintptr_t>(q) % 16 == 0; };
            const float* hprev = c->d_act + p.act_off[l - 1];
            float* dprev = l > 1 ? c->d_delta + p.delta_off[l - 1] : nullptr;
            const size_t smem = (size_t)B * narrow::kMaxOut * sizeof(float);
            const bool vec = din % 4 == 0 && s.w_off[l - 1] % 4 == 0 && a16(X) && a16(G) && a16(hprev) &&
                             (!dprev || a16(dprev));
            if (vec)
                narrow::narrow_backward_kernel<4><<<dim3((din + 4 * narrow::kBwdThreads - 1) / (4 * narrow::kBwdThreads), n),
                                                    narrow::kBwdThreads, smem, c->stream>>>(
                    X, G, c->ld, s.w_off[l - 1], hprev, delta, dp, dprev, B, din, dout);
            else
                narrow::narrow_backward_kernel<1><<<dim3((din + narrow::kBwdThreads - 1) / narrow::kBwdThreads, n),
                                                    narrow::kBwdThreads, smem, c->stream>>>(
                    X, G, c->ld, s.w_off[l - 1], hprev, delta, dp, dprev, B, din, dout);
            c->launches++;
            bias_grad_kernel<<<dim3((dout + 127) / 128, n), 128, 0, c->stream>>>(delta, B, dout, dp, G, c->ld,
                                                                                   s.b_off[l - 1]);
            c->launches++;
            continue;
        }
        {   // gW_l[o][k] = sum_b delta[b][o] h_{l-1}[b][k]
            GemmArgs g{};
            g.A = delta; g.a_node = (int64_t)B * dp; g.a_m = 1; g.a_k = dp;
            g.Bm = c->d_act + p.act_off[l - 1]; g.b_node = (int64_t)B * din; g.b_n = 1; g.b_k = din;
            g.C = G + s.w_off[l - 1]; g.c_node = c->ld; g.c_m = din;
            g.M = dout; g.N = din; g.K = B;
            if (use_tc) {   // m = input unit k', n = output unit o: gW[o][k']
                tc::Args a{};
                a.A = g.Bm; a.a_node = g.b_node; a.a_pitch = din; a.a_kcontig = 0;
                a.B = delta; a.b_node = (int64_t)B * dp; a.b_pitch = dp; a.b_kcontig = 0;
                a.C = g.C; a.c_node = c->ld; a.c_pitch = din;
                a.M = din; a.N = dout; a.K = B; a.epi = tc::EPI_STORE;
                cudaError_t e = cudaErrorNotSupported;
                if (Xn && (c->fuse_step >= 2 || fused_step_pays(c, din, dout))) {   // gossip step applied in the product's epilogue: this block goes straight to X_next
                    if (c->fuse_step != 3) e = run_tcw_ring(c, g.Bm, din, delta, dout, dp, s.w_off[l - 1], X, Xn);
                    if (e == cudaErrorNotSupported) e = run_tcw_fused(c, g.Bm, din, delta, dout, dp, s.w_off[l - 1], X, Xn);
                    if (e == cudaSuccess) c->fused_blocks.emplace_back(s.w_off[l - 1], s.w_off[l - 1] + (int64_t)dout * din);
                }
                if (e == cudaErrorNotSupported) e = run_tcw(c, g.Bm, din, delta, dout, dp, g.C);
                if (e == cudaErrorNotSupported) e = run_tc(c, a, 64);
                if (e != cudaSuccess) return e;
            } else run_gemm<false, false, EPI_STORE>(c, g);
        }
        bias_grad_kernel<<<dim3((dout + 127) / 128, n), 128, 0, c->stream>>>(delta, B, dout, dp, G, c->ld,
                                                                               s.b_off[l - 1]);
        c->launches++;
        if (l > 1) {   // delta_{l-1}[b][k] = (sum_o delta[b][o] W_l[o][k]) * [h_{l-1}[b][k] > 0]
            GemmArgs g{};
            g.A = delta; g.a_node = (int64_t)B * dp; g.a_m = dp; g.a_k = 1;
            g.Bm = X + s.w_off[l - 1]; g.b_node = c->ld; g.b_n = 1; g.b_k = din;
            g.C = c->d_delta + p.delta_off[l - 1]; g.c_node = (int64_t)B * din; g.c_m = din;
            g.aux = c->d_act + p.act_off[l - 1]; g.aux_node = (int64_t)B * din; g.aux_m = din;
            g.M = B; g.N = din; g.K = dout;
            if (use_tc) {   // m = input unit k', n = sample: delta_{l-1}[b][k']
                tc::Args a{};
                a.A = g.Bm; a.a_node = c->ld; a.a_pitch = din; a.a_kcontig = 0;
                a.B = delta; a.b_node = (int64_t)B * dp; a.b_pitch = dp; a.b_kcontig = 1;
                a.C = g.C; a.c_node = g.c_node; a.c_pitch = din;
                a.aux = g.aux; a.aux_node = g.aux_node; a.aux_pitch = din;
                a.M = din; a.N = B; a.K = dout; a.epi = tc::EPI_MASK;
                cudaError_t e = run_tc_weights(c, a);
                if (e != cudaSuccess) return e;
            } else run_gemm<true, false, EPI_MASK>(c, g);
        }
    }
    if (c->ld > c->N) {
        const int64_t total = (c->ld - c->N) * n;
        zero_pad_kernel<<<(unsigned)((total + 127) / 128), 128, 0, c->stream>>>(G, c->ld, c->N, n);
        c->launches++;
    }
    return cudaGetLastError();
}

}  // namespace dpsgd
