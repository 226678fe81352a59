// Weight-gradient product of the MLP with the gossip step of Algorithm 1 (steps 4-5) applied in its
// epilogue: for one weight block of every node,
//
//     X_next[i][block] = sum_j W_ij X[j][block] - gamma * (delta_i^T h_i)
//
// so this block of the stochastic gradient dF(X_k; xi_k) (Section 3) is consumed on chip and never
// written to HBM.  The kernels are tc_wgrad_kernel<..., kGather> and <..., kRing> of tc_wgrad.cuh; this
// file holds their host side: shape checks, tensor maps, the division of the work into node ranges.
#include <algorithm>

#include "ctx.h"
#include "tc_wgrad.cuh"
#include "tma_host.h"

namespace dpsgd {
namespace {

constexpr int kFusedChunk = 2;       // column tiles per item of the fused kernel

// Node ranges for the kernels that walk consecutive nodes at one tile position: whole waves of CTAs,
// each range re-reading the tiles just outside its ends (weighted as one node step).
void choose_ranges(tcw::Args& a, int n, int sms) {
    const long long positions = (long long)a.m_tiles * a.chunks;
    double best = 0.0;
    a.splits = 1; a.split_len = n;
    for (int s = 1; s <= std::min(n, 256); ++s) {
        const int len = (n + s - 1) / s;
        if ((n + len - 1) / len != s) continue;                  // ranges that would hold no node
        const long long waves = (positions * s + sms - 1) / sms;
        const double cost = (double)waves * (len + 1.0);
        if (s == 1 || cost < best) { best = cost; a.splits = s; a.split_len = len; }
    }
    a.total_seqs = (int)(positions * a.splits);
}

template <int NT, bool PRECISE, int DEG>
cudaError_t launch(dpsgd_ctx* c, const CUtensorMap& mapA, const CUtensorMap& mapB, const CUtensorMap& mapC, tcw::Args a) {
    auto kernel = tcw::tc_wgrad_kernel<NT, PRECISE, tcw::kGather, DEG>;
    constexpr size_t smem = tcw::smem_bytes<NT, PRECISE>();
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int sms = 0, dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    // An item is (node, 128-row block, run of `chunk` column tiles); a CTA walks a range of consecutive
    // nodes at one position, so that the tiles of X it gathers for node i (its neighbours in W) are the
    // ones it fetched for nodes i-1 and i-2: they come from L2 as long as the data all CTAs touch during
    // two node steps fits there.  Short runs keep that window small; the price is one h tile converted
    // per node and run.
    a.nodes = c->n;
    a.chunk = std::min(a.n_tiles, kFusedChunk);
    a.chunks = (a.n_tiles + a.chunk - 1) / a.chunk;
    choose_ranges(a, c->n, sms);
    const int grid = std::min(a.total_seqs, sms);                // one persistent CTA per SM
    kernel<<<grid, tcw::kThreadsFused, smem, c->stream>>>(mapA, mapB, mapC, a);
    c->launches++;
    return cudaGetLastError();
}

template <bool PRECISE>
cudaError_t launch_ring(dpsgd_ctx* c, const CUtensorMap& mapA, const CUtensorMap& mapB, const CUtensorMap& mapX, tcw::Args a) {
    auto kernel = tcw::tc_wgrad_kernel<4, PRECISE, tcw::kRing, 0>;
    constexpr size_t smem = tcw::smem_bytes<4, PRECISE, false>();
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int sms = 0, dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    a.nodes = c->n;
    a.chunk = 1;                                                 // the X window in tensor memory holds one tile position
    a.chunks = a.n_tiles;
    choose_ranges(a, c->n, sms);
    const int grid = std::min(a.total_seqs, sms);                // one persistent CTA per SM
    kernel<<<grid, tcw::kThreadsRing, smem, c->stream>>>(mapA, mapB, mapX, a);
    c->launches++;
    return cudaGetLastError();
}

template <int NT, bool PRECISE>
cudaError_t launch_deg(dpsgd_ctx* c, const CUtensorMap& mapA, const CUtensorMap& mapB, const CUtensorMap& mapC,
                       const tcw::Args& a, int deg) {
    switch (deg) {            // common row degree: the column mean 1, ring 3, torus 5
        case 1: return launch<NT, PRECISE, 1>(c, mapA, mapB, mapC, a);
        case 3: return launch<NT, PRECISE, 3>(c, mapA, mapB, mapC, a);
        case 5: return launch<NT, PRECISE, 5>(c, mapA, mapB, mapC, a);
        default: return launch<NT, PRECISE, 0>(c, mapA, mapB, mapC, a);
    }
}

}  // namespace

bool fused_step_supported(const dpsgd_ctx* c) {
    return c->model == DPSGD_MODEL_MLP && !c->swapped && c->V == nullptr && c->mlp_precision != 2 &&
           c->batch <= tcw::kMaxK && c->W.max_deg >= 1 && (c->W.max_deg <= kFusedMaxDegree || c->can_uniform);
}

// Where a fused kernel is faster than the two stages (measured on B200).  Ring W: the kernel with the
// X window on chip reads X once and wins as soon as the stacked weight block is no longer small
// against L2 (n = 112, 2048 x 2048: 2.7 against 3.3 ms per iteration; n = 32, 784 x 1024: level).
// Other W: the gathering kernel pays only when rows of W are as short as a ring's and the block is far
// beyond L2, so that the separate gossip pass would stream it from HBM.
bool fused_step_pays(const dpsgd_ctx* c, int din, int dout) {
    const double block_bytes = (double)c->n * din * dout * sizeof(float);
    if (c->can_ring && c->n >= 3) return block_bytes >= 64.0 * 1024 * 1024;
    const bool short_rows = c->W.max_deg <= 3 || (c->can_uniform && c->W.max_deg > kFusedMaxDegree);   // the mean counts as one row
    return short_rows && block_bytes >= 512.0 * 1024 * 1024;
}

// Ring W (Theorem 3's band): the kernel that keeps the X tiles of nodes i-1 and i in tensor memory
// while it walks the nodes, so every element of X is read once.  Same contract as run_tcw_fused.
cudaError_t run_tcw_ring(dpsgd_ctx* c, const float* h, int din, const float* delta, int dout, int dpitch,
                         int64_t w_off, const float* X, float* Xn) {
    const int B = c->batch;
    auto al = [](const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; };
    // w_off and din multiples of 4: the columns left to the mixing kernel are then whole groups of four
    if (!c->can_ring || !c->W.band || c->n < 3 || B > tcw::kMaxK || din % 4 != 0 || dpitch % 4 != 0 || w_off % 4 != 0 ||
        !al(h) || !al(delta) || !al(X + w_off) || c->ld % 4 != 0)
        return cudaErrorNotSupported;
    const uint64_t nodes = (uint64_t)c->n;
    CUtensorMap mapA, mapB, mapX;
    bool ok = make_map_3d(&mapA, h, (uint64_t)din, (uint64_t)B, nodes, (uint64_t)din * 4, (uint64_t)B * din * 4,
                          tcw::kTileM, tcw::kMaxK, false);
    ok = ok && make_map_3d(&mapB, delta, (uint64_t)dout, (uint64_t)B, nodes, (uint64_t)dpitch * 4,
                           (uint64_t)B * dpitch * 4, 64u, tcw::kMaxK, false);
    // this weight block of X as (input unit, output unit, node): the tile of X_{i+1} of every node step
    ok = ok && make_map_3d(&mapX, X + w_off, (uint64_t)din, (uint64_t)dout, nodes, (uint64_t)din * 4, (uint64_t)c->ld * 4,
                           tcw::kTileM, 64u, false);
    if (!ok) return cudaErrorNotSupported;
    tcw::Args a{};
    a.M = din; a.N = dout; a.K = B;
    a.m_tiles = (din + tcw::kTileM - 1) / tcw::kTileM;
    a.n_tiles = (dout + 63) / 64;
    a.status = &c->d_result->status;
    a.mix.X = X; a.mix.Xn = Xn; a.mix.ld = c->ld; a.mix.ld_out = c->ld; a.mix.w_off = w_off;
    a.mix.row_ptr = c->W.row_ptr; a.mix.col = c->W.col; a.mix.val = c->W.val; a.mix.band = c->W.band;
    a.mix.ngamma = -c->gamma;
    return c->mlp_precision == 0 ? launch_ring<true>(c, mapA, mapB, mapX, a) : launch_ring<false>(c, mapA, mapB, mapX, a);
}

// Returns cudaErrorNotSupported when the shapes or alignments rule the kernel out (the caller then
// writes this block of G and leaves it to the mixing kernel).
cudaError_t run_tcw_fused(dpsgd_ctx* c, const float* h, int din, const float* delta, int dout, int dpitch,
                          int64_t w_off, const float* X, float* Xn) {
    const int B = c->batch;
    auto al = [](const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; };
    if (B > tcw::kMaxK || din % 4 != 0 || dpitch % 4 != 0 || w_off % 4 != 0 || c->ld % 4 != 0 || !al(h) || !al(delta) ||
        !al(X) || !al(Xn))
        return cudaErrorNotSupported;
    const int rows_b = dout <= 16 ? 16 : (dout <= 32 ? 32 : 64);
    const uint64_t nodes = (uint64_t)c->n;
    CUtensorMap mapA, mapB, mapC;
    bool ok = make_map_3d(&mapA, h, (uint64_t)din, (uint64_t)B, nodes, (uint64_t)din * 4, (uint64_t)B * din * 4,
                          tcw::kTileM, tcw::kMaxK, false);
    ok = ok && make_map_3d(&mapB, delta, (uint64_t)dout, (uint64_t)B, nodes, (uint64_t)dpitch * 4,
                           (uint64_t)B * dpitch * 4, (uint32_t)rows_b, tcw::kMaxK, false);
    mapC = mapA;              // the fused kernel issues no TMA store; the parameter only keeps the signature
    if (!ok) return cudaErrorNotSupported;
    tcw::Args a{};
    a.M = din; a.N = dout; a.K = B;
    a.m_tiles = (din + tcw::kTileM - 1) / tcw::kTileM;
    a.n_tiles = (dout + rows_b - 1) / rows_b;
    a.status = &c->d_result->status;
    // gathered from X through W, or (W = w 1 1^T) from the column mean through a one-entry-per-row matrix
    a.mix.X = c->fsrc_X ? c->fsrc_X : X; a.mix.Xn = Xn; a.mix.ld = c->fsrc_X ? c->fsrc_ld : c->ld; a.mix.ld_out = c->ld; a.mix.w_off = w_off;
    a.mix.row_ptr = c->fsrc_X ? c->fsrc_row_ptr : c->W.row_ptr; a.mix.col = c->fsrc_X ? c->fsrc_col : c->W.col;
    a.mix.val = c->fsrc_X ? c->fsrc_val : c->W.val; a.mix.band = c->W.band;
    a.mix.ngamma = -c->gamma;
    const int deg = c->fsrc_X ? 1 : c->W.uniform_deg;
    const bool precise = c->mlp_precision == 0;
    switch (rows_b) {
        case 16: return precise ? launch_deg<1, true>(c, mapA, mapB, mapC, a, deg) : launch_deg<1, false>(c, mapA, mapB, mapC, a, deg);
        case 32: return precise ? launch_deg<2, true>(c, mapA, mapB, mapC, a, deg) : launch_deg<2, false>(c, mapA, mapB, mapC, a, deg);
        default: return precise ? launch_deg<4, true>(c, mapA, mapB, mapC, a, deg) : launch_deg<4, false>(c, mapA, mapB, mapC, a, deg);
    }
}

}  // namespace dpsgd
