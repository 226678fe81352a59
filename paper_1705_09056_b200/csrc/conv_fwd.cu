// 3x3 convolution forward (padding 1, stride 1 or 2), batched over the nodes, each node with the filters
// of its OWN parameter row: the layer family of the paper's image workloads (Section 5.1: ResNet-20 on
// CIFAR-10; Section 5.3: a 32-layer residual network), whose gradient is Algorithm 1 step 3 for them.
//
//     y[node][b][o][i][j] = act( bias[o] + sum_{c,kh,kw} w[o][c][kh][kw] * x[node][b][c][s i + kh - 1][s j + kw - 1] )
//
// Implicit GEMM on the tensor cores with no unfolded matrix in memory: per node
//     C[p][o] = sum_k A(p, k) B(o, k),   p = output position (b, i, j),  k = (c, kh, kw),  K = 9 C_in
// A tile is 128 consecutive output positions (whole output rows of one image, or whole small images), which
// sit on the 128 lanes of tensor memory; the C_out <= 64 output channels are the accumulator's columns.
//
//   TMA warp        one thread fetches, per tile, the input patch the 128 positions read: a 5-D box
//                   (W_in, rows, C_in, images, node) of the NCHW input with one halo row above and below.
//                   Rows outside the image are zero-filled by the TMA unit (the box starts at row -1);
//                   the box always starts at column 0, so the copy is 16-byte aligned whatever the tap.
//   converter warps (8) two threads own an output position, 16 of a block's 32 k each.  Per block a thread gathers its part of the row of the
//                   unfolded matrix from the patch in shared memory (a table gives, for every k, the offset
//                   of tap (c, kh, kw) inside the patch; the left / right zero border is a predicate),
//                   splits each value into its TF32 head and remainder and writes both to its TENSOR
//                   MEMORY lane (tcgen05.st): A never exists in memory.  When the CTA moves to another
//                   node the same warps convert that node's filters, once, into the K-major no-swizzle
//                   shared-memory layout of the MMA descriptors (heads and remainders), for all of K.
//   MMA warp        one thread issues, per block of 32 k, three TF32 MMAs per 8 k (lo*hi + hi*lo + hi*hi,
//                   fp32 accumulation in tensor memory), A from tensor memory, B through descriptors.
//   epilogue        the converter warps read a finished accumulator (tcgen05.ld), add the bias, apply the
//                   ReLU and store with the positions contiguous across lanes (NCHW: 128-byte lines).  There are
//                   two accumulators and the epilogue of a tile runs after the NEXT tile's blocks have been
//                   converted, so the tensor core never waits for it.
//
// CTAs are persistent and take CONTIGUOUS ranges of (node, tile), so a node's filters are converted once
// per CTA that touches the node.  Every mbarrier wait is bounded; a wait that runs out raises the status
// word, the TMA thread waits (bounded) for its copies in flight and the CTA frees its tensor memory before
// it returns.  No cluster multicast: every CTA fetches its own patch, from this GPU's memory.
#include <algorithm>

#include "ctx.h"
#include "tc_stream.cuh"
#include "tma_host.h"

namespace dpsgd {
namespace conv {

using tc::mbar_arrive;
using tc::mbar_init;
using tc::mbar_wait;
using tc::smem_u32;
using tcs::lds32;
using tcs::mbar_expect_tx;

constexpr int kThreads = 320;        // 8 converter / epilogue warps, MMA warp, TMA warp
constexpr int kConvThreads = 256;    // two threads per output position: 16 of a block's 32 k each
constexpr int kMmaWarp = 8, kTmaWarp = 9;
constexpr int kMaxPatchStages = 4;   // input patches in flight: a TMA copy takes longer than a small tile's work
constexpr int kTileP = 128;          // output positions per tile
constexpr int kBK = 32;              // k per converted block
constexpr uint32_t kACols = 2 * kBK; // heads, then remainders
constexpr uint32_t kAccCols = 64;    // per accumulator; two of them, so that a tile's epilogue runs under the next tile's MMAs
constexpr uint32_t kTmemCols = 256;  // two accumulators + two converted blocks

struct Args {
    const float* W;          // first filter of node 0 (inside its parameter row); node stride ld_w
    const float* bias;       // first bias of node 0; same stride (NULL: no bias)
    int64_t ld_w;
    float* Y;                // [n][B][C_out_total][Ho][Wo]
    int n, B, C_in, C_out_total, o0;   // this launch computes channels [o0, o0 + ROWS_B)
    int H_in, W_in, Ho, Wo, stride, relu;
    int K, KB;               // 9 C_in, ceil(K / 32)
    int imgs_per_tile, rows_per_tile, rows_patch, tiles_per_node, total_tiles;
    uint32_t patch_bytes, patch_stride, patch_stages;   // box bytes; stage stride (box rounded up to 128 bytes)
    int log2_wo, log2_img;   // Wo and (positions per image inside a tile) are powers of two
    int* status;
};

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ uint32_t lds32u(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// Shared memory: [patch stages][B heads | B remainders][tap table][barriers].
__host__ __device__ inline uint32_t b_copy_bytes(int kb, int rows) { return (uint32_t)kb * (kBK / 4) * rows * 16; }

// TAPMAJOR (C_in a multiple of 16): the contraction index runs tap-major, k = (kh, kw) C_in + c, so that the 16
// values a thread gathers per block share one tap: one border predicate, addresses one channel plane apart, no
// table.  Otherwise k = c 9 + (kh, kw) as the filters lie in memory, through the tap table.
template <int NT, bool TAPMAJOR>
__global__ void __launch_bounds__(kThreads, 2)
conv3x3_fwd_kernel(const __grid_constant__ CUtensorMap mapX, Args g) {
    constexpr int ROWS_B = 16 * NT;                       // output channels of this launch
    constexpr uint32_t B_LBO = (uint32_t)ROWS_B * 16, SBO = 128;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t S = g.patch_stages;
    const uint32_t B_COPY = b_copy_bytes(g.KB, ROWS_B);
    const uint32_t patch0 = base;
    const uint32_t b_hi = patch0 + S * g.patch_stride, b_lo = b_hi + B_COPY;
    const uint32_t table = b_lo + B_COPY;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + S * g.patch_stride + 2 * B_COPY + (uint32_t)g.KB * kBK * 4);
    uint64_t* patch_full = bars;                 // [kMaxPatchStages]
    uint64_t* patch_empty = bars + kMaxPatchStages;
    uint64_t* conv_full = bars + 2 * kMaxPatchStages;            // [2]
    uint64_t* conv_empty = conv_full + 2;        // [2]
    uint64_t* acc_full = conv_full + 4;          // [2] one per accumulator
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(conv_full + 6);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kMaxPatchStages; ++s) { mbar_init(patch_full + s, 1); mbar_init(patch_empty + s, kConvThreads); }
        for (int s = 0; s < 2; ++s) { mbar_init(conv_full + s, kConvThreads); mbar_init(conv_empty + s, 1); }
        mbar_init(acc_full, 1); mbar_init(acc_full + 1, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // tap table: for k = (c, kh, kw): ((offset of the tap inside the patch, + 1) << 2) | kw; kw = 3 marks k >= K
    for (int k = tid; k < g.KB * kBK; k += kThreads) {
        uint32_t e = 3u;
        if (k < g.K) {
            const int c = k / 9, r = k - 9 * c, kh = r / 3, kw = r - 3 * kh;
            e = ((uint32_t)((c * g.rows_patch + kh) * g.W_in + kw) << 2) | (uint32_t)kw;     // (offset + 1, kw)
        }
        reinterpret_cast<uint32_t*>(base_ptr + S * g.patch_stride + 2 * B_COPY)[k] = e;
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // contiguous range of (node, tile) for this CTA
    const int per = (g.total_tiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int t_begin = min(g.total_tiles, (int)blockIdx.x * per), t_end = min(g.total_tiles, t_begin + per);
    const int pos_per_img = g.Ho * g.Wo;
    const int total_pos = g.B * pos_per_img;              // per node

    if (warp < 8) {
        // ------------------------------ converters, then epilogue ------------------------------
        // thread = (output position p, half): lane quarter warp % 4 of tensor memory, columns 16 half .. of a block
        const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t half = (uint32_t)warp >> 2;
        bool ok = true;
        uint32_t q = 0, done = 0;
        int cur_node = -1;
        // position of this thread inside a tile: image, output row, output column (all local to the tile)
        const int p = tid & 127;
        const int img_l = p >> g.log2_img, pin = p & ((1 << g.log2_img) - 1);
        const int i_l = pin >> g.log2_wo, j = pin & (g.Wo - 1);
        const int jj0 = g.stride * j - 1;                                   // input column under tap kw = 0
        const uint32_t base_p = (uint32_t)(((img_l * g.C_in) * g.rows_patch + g.stride * i_l) * g.W_in + g.stride * j);

        // Epilogue of the tile whose MMAs went into accumulator `slot`: bias, ReLU, NCHW store (positions contiguous
        // across lanes).  It is run one tile late, after the next tile's blocks have been converted, so that the MMAs
        // it waits for have had that long to finish and the tensor core works on the next tile meanwhile.
        auto epilogue = [&](int t_done, uint32_t idx) -> bool {
            const uint32_t slot = idx & 1u;
            bool fine = mbar_wait(acc_full + slot, (idx >> 1) & 1u);
            fine = __all_sync(0xffffffffu, fine);                            // tcgen05.ld needs the whole warp
            if (!fine) return false;
            tc::tc_fence_after();
            const int node = t_done / g.tiles_per_node, tile = t_done - node * g.tiles_per_node;
            const int pg = tile * kTileP + p;                                // position inside the node
            const bool live = pg < total_pos;
            const int img = pg / pos_per_img, pin_g = pg - img * pos_per_img;
            float* yb = g.Y + (((int64_t)node * g.B + img) * g.C_out_total + g.o0) * pos_per_img + pin_g;
            const float* bn = g.bias ? g.bias + (int64_t)node * g.ld_w + g.o0 : nullptr;
#pragma unroll 1
            for (int c0 = 16 * (int)half; c0 < ROWS_B; c0 += 32) {
                float v[16];
                tc::tmem_ld16(lane_base + slot * kAccCols + (uint32_t)c0, v);
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    float x = bn ? v[u] + __ldg(bn + c0 + u) : v[u];
                    if (g.relu && !(x > 0.f)) x = 0.f;
                    if (live) yb[(int64_t)(c0 + u) * pos_per_img] = x;
                }
            }
            tc::tc_fence_before();          // these accumulator reads precede the MMAs of the tile after next
            return true;
        };

        int pending = -1;                                                    // tile whose epilogue is still owed
        for (int t = t_begin; t < t_end && ok; ++t, ++done) {
            const int node = t / g.tiles_per_node;
            if (node != cur_node) {
                // this node's filters for channels [o0, o0 + ROWS_B): the buffers are free once every MMA of the
                // previous tile has completed, i.e. once its accumulator is full
                if (pending >= 0) { ok = epilogue(pending, done - 1); pending = -1; if (!ok) break; }
                const float* wn = g.W + (int64_t)node * g.ld_w + (int64_t)g.o0 * g.K;
                const bool vec = (g.K & 3) == 0 && (reinterpret_cast<uintptr_t>(wn) & 15) == 0;
                if (TAPMAJOR) {
                    // read the filters as they lie in memory (o, c, tap: coalesced, all loads of a thread in flight)
                    // and scatter every value to its tap-major place k = tap C_in + c of the MMA layout
                    const int quads = g.K >> 2;                              // K = 9 C_in is a multiple of 16
                    for (int idx = tid; idx < quads * ROWS_B; idx += kConvThreads) {
                        const int o = idx / quads, m0 = 4 * (idx - o * quads);
                        const float* src = wn + (int64_t)o * g.K + m0;
                        float v[4];
                        if (vec) {
                            const float4 t = __ldg(reinterpret_cast<const float4*>(src));
                            v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
                        } else {
                            v[0] = __ldg(src); v[1] = __ldg(src + 1); v[2] = __ldg(src + 2); v[3] = __ldg(src + 3);
                        }
                        const uint32_t row = (uint32_t)(o >> 3) * SBO + (uint32_t)(o & 7) * 16;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int m = m0 + e, ch = m / 9, tap = m - 9 * ch;
                            const uint32_t k = (uint32_t)(tap * g.C_in + ch);
                            const uint32_t off = (k >> 2) * B_LBO + row + (k & 3u) * 4;
                            uint32_t hi, lo;
                            tcs::split(v[e], hi, lo);
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(b_hi + off), "r"(hi) : "memory");
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(b_lo + off), "r"(lo) : "memory");
                        }
                    }
                } else {
                    const int chunks = g.KB * (kBK / 4);
                    for (int idx = tid; idx < chunks * ROWS_B; idx += kConvThreads) {
                        const int o = idx % ROWS_B, c = idx / ROWS_B;        // lanes run along o: conflict-free stores
                        const int k = 4 * c;
                        const float* src = wn + (int64_t)o * g.K + k;
                        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (vec) {
                            if (k < g.K) v = __ldg(reinterpret_cast<const float4*>(src));
                        } else {
                            if (k < g.K) v.x = __ldg(src);
                            if (k + 1 < g.K) v.y = __ldg(src + 1);
                            if (k + 2 < g.K) v.z = __ldg(src + 2);
                            if (k + 3 < g.K) v.w = __ldg(src + 3);
                        }
                        tcs::put<true>(b_hi, b_lo, (uint32_t)c * B_LBO + (uint32_t)(o >> 3) * SBO + (uint32_t)(o & 7) * 16, v);
                    }
                }
                cur_node = node;
            }
            const uint32_t ps = done % S;
            if (!__all_sync(0xffffffffu, mbar_wait(patch_full + ps, (done / S) & 1u))) { ok = false; break; }
            const uint32_t patch = patch0 + ps * g.patch_stride + base_p * 4;
            for (int kb = 0; kb < g.KB; ++kb, ++q) {
                const uint32_t buf = q & 1u;
                if (!__all_sync(0xffffffffu, mbar_wait(conv_empty + buf, ((q >> 1) & 1u) ^ 1u))) { ok = false; break; }
                tc::tc_fence_after();
                const uint32_t a_cols = lane_base + 2 * kAccCols + buf * kACols;
                uint32_t hi[16], lo[16];
                if (TAPMAJOR) {
                    const int k0 = kb * kBK + (int)half * 16;            // 16 consecutive channels of one tap
                    const int tap = k0 / g.C_in, ch = k0 - tap * g.C_in;
                    const int kh = (tap * 11) >> 5, kw = tap - 3 * kh;   // tap / 3 for tap < 9
                    const int jj = jj0 + kw;
                    const bool in = k0 < g.K && jj >= 0 && jj < g.W_in;
                    const uint32_t plane = (uint32_t)(g.rows_patch * g.W_in) * 4;
                    const uint32_t src = patch + (uint32_t)((ch * g.rows_patch + kh) * g.W_in + kw) * 4 - 4;
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        const float v = in ? lds32(src + (uint32_t)u * plane) : 0.f;
                        tcs::split(v, hi[u], lo[u]);
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        const uint32_t e = lds32u(table + (uint32_t)(kb * kBK + half * 16 + u) * 4);
                        const int kw = (int)(e & 3u);
                        const int jj = jj0 + kw;                             // input column under this tap
                        const bool in = kw != 3 && jj >= 0 && jj < g.W_in;   // left / right zero border
                        // e >> 2 = offset of the tap from this position's patch base, plus one
                        const float v = in ? lds32(patch + (e >> 2) * 4 - 4) : 0.f;
                        tcs::split(v, hi[u], lo[u]);
                    }
                }
                tcs::tmem_st16(a_cols + 16 * half, hi);
                tcs::tmem_st16(a_cols + kBK + 16 * half, lo);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc::tc_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the filters written above, first block
                mbar_arrive(conv_full + buf);
            }
            if (!ok) break;
            mbar_arrive(patch_empty + ps);                                   // the patch has been read
            if (pending >= 0) ok = epilogue(pending, done - 1);              // the tile before this one
            pending = t;
        }
        if (ok && pending >= 0) ok = epilogue(pending, done - 1);
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    } else if (warp == kMmaWarp) {
        if (lane == 0) {
            // ------------------------------ MMA issuer ------------------------------
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ROWS_B >> 3) << 17) |
                                   ((uint32_t)(kTileP >> 4) << 24);
            bool ok = true;
            uint32_t q = 0, done = 0;
            for (int t = t_begin; t < t_end && ok; ++t, ++done) {
                uint32_t acc = 0;
                // accumulator done & 1: its previous contents (tile done - 2) were read before the converters wrote
                // the first block of this tile
                const uint32_t d_acc = tmem_base + (done & 1u) * kAccCols;
                for (int kb = 0; kb < g.KB; ++kb, ++q) {
                    const uint32_t buf = q & 1u;
                    if (!mbar_wait(conv_full + buf, (q >> 1) & 1u)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t a_hi = tmem_base + 2 * kAccCols + buf * kACols, a_lo = a_hi + kBK;
#pragma unroll
                    for (uint32_t kk = 0; kk < kBK / 8; ++kk) {
                        if ((int)(kb * kBK + kk * 8) >= g.K) break;          // zero padding only from here on
                        const uint32_t boff = (uint32_t)(kb * (kBK / 8) + kk) * 2 * B_LBO;
                        const uint64_t dbh = tc::smem_desc(b_hi + boff, B_LBO, SBO);
                        const uint64_t dbl = tc::smem_desc(b_lo + boff, B_LBO, SBO);
                        tcs::mma_tf32_ts(d_acc, a_lo + kk * 8, dbh, idesc, acc); acc = 1;
                        tcs::mma_tf32_ts(d_acc, a_hi + kk * 8, dbl, idesc, acc);
                        tcs::mma_tf32_ts(d_acc, a_hi + kk * 8, dbh, idesc, acc);
                    }
                    tc::mma_commit(conv_empty + buf);
                }
                if (ok) tc::mma_commit(acc_full + (done & 1u));
            }
            if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
        }
    } else if (warp == kTmaWarp && lane == 0) {
        // ------------------------------ TMA: input patches ------------------------------
        bool ok = true;
        uint32_t done = 0;
        for (int t = t_begin; t < t_end && ok; ++t, ++done) {
            const int node = t / g.tiles_per_node, tile = t - node * g.tiles_per_node;
            const uint32_t ps = done % S;
            if (!mbar_wait(patch_empty + ps, ((done / S) & 1u) ^ 1u)) { ok = false; break; }
            // first image and first output row of the tile
            int img0, row0;
            if (g.imgs_per_tile > 1) { img0 = tile * g.imgs_per_tile; row0 = 0; }
            else {
                const int tiles_per_img = g.Ho / g.rows_per_tile;
                img0 = tile / tiles_per_img;
                row0 = (tile - img0 * tiles_per_img) * g.rows_per_tile;
            }
            mbar_expect_tx(patch_full + ps, g.patch_bytes);
            tma_load_5d(patch0 + ps * g.patch_stride, &mapX, 0, g.stride * row0 - 1, 0, img0, node, patch_full + ps);
        }
        for (uint32_t jx = 0; jx < S && jx < done; ++jx) {      // copies in flight when somebody gave up
            const uint32_t dd = done - 1 - jx;
            mbar_wait(patch_full + dd % S, (dd / S) & 1u);
        }
        if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <int NT>
cudaError_t launch_nt(dpsgd_ctx* c, const CUtensorMap& map, const Args& a, size_t smem);

int ilog2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

template <int NT, bool TAPMAJOR>
cudaError_t launch_nt_k(dpsgd_ctx* c, const CUtensorMap& map, const Args& a, size_t smem) {
    auto kernel = conv3x3_fwd_kernel<NT, TAPMAJOR>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int sms = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device)) != cudaSuccess) return e;
    const int per_sm = smem <= 110 * 1024 ? 2 : 1;              // tensor memory: 256 columns per CTA
    const int grid = std::min(a.total_tiles, sms * per_sm);     // persistent CTAs over contiguous tile ranges
    kernel<<<grid, kThreads, smem, c->stream>>>(map, a);
    c->launches++;
    return cudaGetLastError();
}

template <int NT>
cudaError_t launch_nt(dpsgd_ctx* c, const CUtensorMap& map, const Args& a, size_t smem) {
    return a.C_in % 16 == 0 ? launch_nt_k<NT, true>(c, map, a, smem) : launch_nt_k<NT, false>(c, map, a, smem);
}

}  // namespace conv

// Shapes the kernel takes: W_in and the output width powers of two with 4 <= W_in <= 256, output positions
// of an image either a multiple of 128 or a divisor of it, C_out a multiple of 16.
const char* conv3x3_forward_unsupported(int batch, int c_in, int h, int w, int c_out, int stride) {
    if (batch < 1 || c_in < 1 || h < 1 || w < 1 || c_out < 1) return "sizes must be positive";
    if (stride != 1 && stride != 2) return "stride must be 1 or 2";
    if (c_out % 16 != 0) return "C_out must be a multiple of 16";
    if (w < 4 || w > 256 || (w & (w - 1)) != 0) return "W must be a power of two in [4, 256]";
    const int ho = (h - 1) / stride + 1, wo = (w - 1) / stride + 1;
    if ((wo & (wo - 1)) != 0 || wo > 128) return "output width must be a power of two of at most 128";
    const int pos = ho * wo;
    if (pos >= 128 ? (pos % 128 != 0 || 128 % wo != 0) : (128 % pos != 0)) return "output positions per image must be a multiple or a divisor of 128";
    if (c_in > 256) return "C_in must be at most 256";
    return nullptr;
}

cudaError_t launch_conv3x3_forward(dpsgd_ctx* c, const float* x, int batch, int c_in, int h, int w, int c_out, int stride,
                                   int64_t w_off, int64_t b_off, int relu, float* y, const char** why) {
    return launch_conv3x3_forward_on(c, x, batch, c_in, h, w, c_out, stride, c->X[c->cur] + w_off, c->X[c->cur] + b_off,
                                     c->ld, relu, y, why);
}

cudaError_t launch_conv3x3_forward_on(dpsgd_ctx* c, const float* x, int batch, int c_in, int h, int w, int c_out,
                                      int stride, const float* W, const float* bias, int64_t ld_w, int relu, float* y,
                                      const char** why) {
    using namespace conv;
    *why = nullptr;
    Args a{};
    a.n = c->n; a.B = batch; a.C_in = c_in; a.C_out_total = c_out; a.H_in = h; a.W_in = w; a.stride = stride; a.relu = relu;
    a.Ho = (h - 1) / stride + 1; a.Wo = (w - 1) / stride + 1;
    a.K = 9 * c_in; a.KB = (a.K + kBK - 1) / kBK;
    const int pos = a.Ho * a.Wo;
    if (pos >= kTileP) { a.imgs_per_tile = 1; a.rows_per_tile = kTileP / a.Wo; }
    else { a.imgs_per_tile = kTileP / pos; a.rows_per_tile = a.Ho; }
    a.rows_patch = stride * (a.rows_per_tile - 1) + 3;
    a.tiles_per_node = (batch * pos + kTileP - 1) / kTileP;
    a.total_tiles = a.tiles_per_node * c->n;
    a.patch_bytes = (uint32_t)(a.imgs_per_tile * c_in * a.rows_patch * w) * 4u;   // = the TMA box (a multiple of 16)
    a.patch_stride = (a.patch_bytes + 127u) & ~127u;
    a.log2_wo = ilog2(a.Wo);
    a.log2_img = ilog2(std::min(pos, kTileP));
    a.W = W; a.bias = bias; a.ld_w = ld_w;
    a.Y = y;
    a.status = &c->d_result->status;
    if (a.rows_patch > 256) { *why = "the input patch of a tile is taller than a TMA box"; return cudaErrorNotSupported; }

    // input as (W, H, C, image, node); the box is one tile's patch: every column, rows_patch rows starting
    // one row above the first output row's window (rows outside the image read as zero), every channel
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) { *why = "the driver's tensor-map encoder is not available"; return cudaErrorNotSupported; }
    CUtensorMap map;
    const cuuint64_t dims[5] = {(cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)c_in, (cuuint64_t)batch, (cuuint64_t)c->n};
    const cuuint64_t strides[4] = {(cuuint64_t)w * 4, (cuuint64_t)w * h * 4, (cuuint64_t)w * h * c_in * 4,
                                   (cuuint64_t)w * h * c_in * batch * 4};
    const cuuint32_t box[5] = {(cuuint32_t)w, (cuuint32_t)a.rows_patch, (cuuint32_t)c_in, (cuuint32_t)a.imgs_per_tile, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
        *why = "the tensor map of the input could not be encoded";
        return cudaErrorNotSupported;
    }

    // Output channels per launch: heads and remainders of the filters for all of K sit in shared memory
    // beside one or two patches; a layer too wide for that takes several launches over channel ranges.
    const size_t budget = 227 * 1024 - 1024;
    cudaError_t e = cudaSuccess;
    for (int o0 = 0; o0 < c_out && e == cudaSuccess;) {
        int rows = (c_out - o0) >= 64 ? 64 : ((c_out - o0) >= 32 ? 32 : 16);
        size_t need = 0;
        uint32_t stages = 2;
        for (;;) {
            const size_t fixed = 2 * (size_t)b_copy_bytes(a.KB, rows) + (size_t)a.KB * kBK * 4 + 128 + 256;
            // as many patches in flight (up to four) as leave room for two CTAs per SM when one patch does;
            // otherwise as many as fit beside the filters with one CTA per SM
            const size_t two_ctas = (size_t)110 * 1024;
            const size_t limit = fixed + (size_t)a.patch_stride <= two_ctas ? two_ctas : budget;
            bool fits = false;
            for (uint32_t st = kMaxPatchStages; st >= 1 && !fits; --st) {
                need = fixed + st * (size_t)a.patch_stride;
                if (need <= limit) { stages = st; fits = true; }
            }
            if (fits) break;
            if (rows == 16) { *why = "a tile's input patch and the filters do not fit shared memory"; return cudaErrorNotSupported; }
            rows /= 2;
        }
        Args al = a;
        al.o0 = o0;
        al.patch_stages = stages;
        switch (rows) {
            case 64: e = launch_nt<4>(c, map, al, need); break;
            case 32: e = launch_nt<2>(c, map, al, need); break;
            default: e = launch_nt<1>(c, map, al, need); break;
        }
        o0 += rows;
    }
    return e;
}

}  // namespace dpsgd
