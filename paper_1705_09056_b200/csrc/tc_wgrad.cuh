// Weight-gradient product of the MLP (Algorithm 1 step 3), batched over the nodes:
//
//     gW[o][k'] = sum_b delta[b][o] * h[b][k']          K = minibatch <= 64, output din x dout per node
//
// i.e. C[n][m] = sum_k A(m,k) B(n,k) with m = k' (input unit), n = o (output unit), k = b, both
// operands contiguous along their row index in memory (h is [b][k'], delta is [b][o]).  The product
// is bound by WRITING the gradient (one pass over G), so the kernel is built around the output:
//
//   TMA warp        loads the raw h tile of a work item ([k][128 m], once per item) and, per column
//                   tile, the raw delta tile ([k][N]) into a ring of stages.
//   converter warps (4) split values into TF32 head and remainder (three MMAs per product, as in
//                   tc_gemm.cuh).  The h tile goes to TENSOR MEMORY once per item (thread t owns row
//                   t: column t of the raw tile, which transposes it) and serves every column tile
//                   of the item; delta tiles go to shared memory in the K-major no-swizzle layout
//                   (element (r,k) at (k/4)*LBO + (r/8)*128 + (r%8)*16 + (k%4)*4), double-buffered.
//   MMA warp        one thread issues the MMAs of a column tile into one of two accumulators.
//   epilogue warps  (4) read a finished accumulator with tcgen05.ld, lay it out in shared memory as
//                   [n][128 m] and hand it to a TMA store (cp.async.bulk.tensor, shared -> global),
//                   which writes whole lines asynchronously and clips at the matrix edge; two
//                   staging buffers, so the store of one tile overlaps the next.
//
// That is MODE kStore.  In the two other modes the gossip step of Algorithm 1 (steps 4-5) is applied to
// the tile while it is on chip and the kernel writes
//     X_next[node] = sum_j W_ij X[j] - gamma * gW
// so that this block of the gradient never reaches HBM: 8 bytes per parameter (read X, write X_next)
// instead of 16 (write G; read X, read G, write X_next).  A CTA then walks a range of consecutive nodes
// at one tile position, so that the neighbours' tiles of X it needs for node i are the ones it touched
// for nodes i-1 and i-2.
//
//   kGather (any W with few entries per row, or the column mean as a one-row matrix): no TMA store;
//           sixteen more warps (the mixers; a gather is bound by the bytes its threads keep in flight)
//           take a staged tile, read the same tile of X from the node's neighbours with 128-bit loads
//           (all but the first read of an element come from L2; the next node's tiles are prefetched
//           into L2 one item ahead) and write X_next.  Two column tiles per item.
//   kRing   (Theorem 3's ring): no epilogue warps and no staging of the output; sixteen mixer warps read
//           the accumulator in its own layout and keep the tiles of X_{i-1} and X_i in tensor memory, so
//           X is read from memory once: the tile of X_{i+1}, which the TMA thread fetches one to two
//           nodes ahead into two shared-memory stages (no mixer thread waits on HBM, no registers
//           hold loads in flight).  One column tile per item (the window holds one position), hence
//           one h tile AND one delta tile to convert per item: four converter warps alone were the
//           slowest stage (one warp per SM partition, ~500 dependent instructions per item), and the
//           mixers' chain of dependent steps per item is the next slowest, so the delta tiles are split
//           by four warps of their own (26 warps, 72 registers).
//
// One persistent CTA per SM; a work item is (node, 128-row block of m, run of column tiles).  Every
// mbarrier wait is bounded; a wait that runs out raises the status word, the TMA thread waits
// (bounded) for its loads in flight, outstanding stores are drained, and the CTA frees its TMEM
// columns before it returns.
#pragma once
#include "tc_stream.cuh"

namespace dpsgd {
namespace tcw {

using tc::mbar_arrive;
using tc::mbar_init;
using tc::mbar_wait;
using tc::smem_u32;
using tcs::lds32;
using tcs::mbar_expect_tx;
using tcs::tma_load_3d;

constexpr int kThreads = 320;        // 4 epilogue warps, 4 converter warps, MMA warp, TMA warp
constexpr int kMixWarps = 16;        // kGather: warps 10..25 apply the gossip step to staged tiles
constexpr int kThreadsFused = kThreads + 32 * kMixWarps;
constexpr int kThreadsRing = 832;    // kRing: converters (h), MMA, TMA as above; warps 0-3 and 10-21 mix; warps 22-25 split delta
enum { kStore = 0, kGather = 1, kRing = 2 };
constexpr int kTileM = 128;
constexpr int kMaxK = 64;            // minibatch rows a raw tile holds
constexpr int kStagesB = 3;
constexpr int kStagesBRing = 2;      // kRing: one delta tile per item, and shared memory also holds two tiles of X
constexpr uint32_t kAccStride = 64;  // TMEM columns per accumulator
constexpr uint32_t kACols = 2 * kMaxK;   // heads, then remainders
constexpr uint32_t A_COL0_ = 2 * kAccStride;   // first tensor-memory column of the converted h tiles

// What the fused gossip epilogue needs: the stacked X of this iteration, the buffer of the next one,
// where this weight block starts inside a parameter row, W in CSR and -gamma.
struct Mix {
    const float* X;
    float* Xn;
    int64_t ld, ld_out, w_off;       // row strides of X (0 when every row gathers from one shared row) and of Xn
    const int32_t* row_ptr;
    const int32_t* col;
    const float* val;
    const float* band;               // kRing: [n][3] = (W_{i,i-1}, W_ii, W_{i,i+1})
    float ngamma;
};

// Work decomposition.  A work item is (node, 128-row block of m, run of `chunk` column tiles); the h
// tile of the item is converted once and serves its column tiles.  Items are grouped into sequences of
// `split_len` consecutive nodes at one (row block, run) position; a CTA takes whole sequences
// (blockIdx.x, blockIdx.x + gridDim.x, ...), ordered run-fastest, then row block, then node range.
// split_len = 1 gives plain node-major order.  The fused kernel walks longer node ranges so that the
// neighbours' tiles of X it gathers for node i were fetched by the same CTA for nodes i-1 and i-2.
struct Args {
    int M, N, K;                     // din, dout, minibatch
    int nodes;
    int m_tiles, n_tiles, chunk, chunks;   // column tiles per item, items per (node, m block)
    int splits, split_len;           // node ranges, nodes per range
    int total_seqs;                  // m_tiles * chunks * splits
    int* status;
    Mix mix;                         // kGather, kRing
};

__host__ __device__ constexpr uint32_t a_raw_bytes() { return kMaxK * kTileM * 4; }
__host__ __device__ constexpr uint32_t b_raw_bytes(int rows) { return (uint32_t)kMaxK * rows * 4; }
__host__ __device__ constexpr uint32_t b_lbo(int rows) { return (uint32_t)rows * 16; }
__host__ __device__ constexpr uint32_t b_conv_bytes(int rows) { return (kMaxK / 4) * b_lbo(rows); }
__host__ __device__ constexpr uint32_t stage_bytes(int rows) { return (uint32_t)rows * kTileM * 4; }

// STAGED: two staging buffers for the output tile and one raw h tile; otherwise (kRing) two raw h
// tiles and two stages for the tile of X_{i+1}.
template <int NT, bool PRECISE, bool STAGED = true>
constexpr size_t smem_bytes() {
    return 1024 + (STAGED ? 1 : 2) * a_raw_bytes() + (STAGED ? kStagesB : kStagesBRing) * b_raw_bytes(16 * NT) +
           2 * (PRECISE ? 2 : 1) * b_conv_bytes(16 * NT) + 2 * stage_bytes(16 * NT) + 256;
}

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
__device__ __forceinline__ void sts32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// Gossip step on ROWS rows (output units) of a staged gradient tile: warp `warp` of the kMixWarps
// mixer warps takes rows warp, warp + kMixWarps, ...; its lanes cover the 128 input units of a row, four each.
// `off` = offset of (first row of the tile, this lane's first column) inside a parameter row; rows at
// or beyond `rows` and lanes with !col_ok lie outside the weight matrix.  DEG > 0: every row of W has
// DEG entries (loads of four rows x DEG neighbours in flight); DEG == 0: any degree.
template <int DEG, int ROWS>
__device__ __forceinline__ void mix_rows(const Mix& mx, int node, uint32_t st, int64_t off, int din, int rows,
                                         bool col_ok, int warp, int lane) {
    constexpr int U = 4;
    const int p0 = __ldg(mx.row_ptr + node);
    const int deg = DEG > 0 ? DEG : __ldg(mx.row_ptr + node + 1) - p0;
    float* out = mx.Xn + (int64_t)node * mx.ld_out + off;
#pragma unroll 1
    for (int r0 = warp; r0 < ROWS; r0 += kMixWarps * U) {
        float4 acc[U];
#pragma unroll
        for (int u = 0; u < U; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (DEG > 0) {
            float4 v[DEG > 0 ? DEG : 1][U];
#pragma unroll
            for (int p = 0; p < DEG; ++p) {
                const float* xr = mx.X + (int64_t)__ldg(mx.col + p0 + p) * mx.ld + off;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = r0 + kMixWarps * u;
                    v[p][u] = (col_ok && r < rows) ? __ldcg(reinterpret_cast<const float4*>(xr + (int64_t)r * din))
                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int p = 0; p < DEG; ++p) {
                const float w = __ldg(mx.val + p0 + p);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    acc[u].x = fmaf(w, v[p][u].x, acc[u].x); acc[u].y = fmaf(w, v[p][u].y, acc[u].y);
                    acc[u].z = fmaf(w, v[p][u].z, acc[u].z); acc[u].w = fmaf(w, v[p][u].w, acc[u].w);
                }
            }
        } else {
#pragma unroll 1
            for (int p = 0; p < deg; ++p) {
                const float* xr = mx.X + (int64_t)__ldg(mx.col + p0 + p) * mx.ld + off;
                const float w = __ldg(mx.val + p0 + p);
                float4 v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = r0 + kMixWarps * u;
                    v[u] = (col_ok && r < rows) ? __ldcg(reinterpret_cast<const float4*>(xr + (int64_t)r * din))
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    acc[u].x = fmaf(w, v[u].x, acc[u].x); acc[u].y = fmaf(w, v[u].y, acc[u].y);
                    acc[u].z = fmaf(w, v[u].z, acc[u].z); acc[u].w = fmaf(w, v[u].w, acc[u].w);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int r = r0 + kMixWarps * u;
            if (col_ok && r < rows) {
                const float4 g = tcs::lds128(st + (uint32_t)r * (kTileM * 4) + (uint32_t)lane * 16);
                float4 o;
                o.x = fmaf(mx.ngamma, g.x, acc[u].x); o.y = fmaf(mx.ngamma, g.y, acc[u].y);
                o.z = fmaf(mx.ngamma, g.z, acc[u].z); o.w = fmaf(mx.ngamma, g.w, acc[u].w);
                __stcs(reinterpret_cast<float4*>(out + (int64_t)r * din), o);
            }
        }
    }
}

// The work items of this CTA in order.  The position (row block, run of column tiles, node range) is decoded
// once per node range; inside a range the walk only counts nodes up, so that the per-item cost on the threads
// that sit on the critical path (TMA, converters, MMA issuer) is an increment, not a chain of integer divisions.
struct Walk {
    int node, n1, m0, t0, t1;        // the current item: node, first row, column tiles [t0, t1)
    int rd, rounds;
    __device__ __forceinline__ explicit Walk(const Args& g) : node(0), n1(0), m0(0), t0(0), t1(0), rd(-1) {
        const int b = (int)blockIdx.x, grid = (int)gridDim.x;
        rounds = b < g.total_seqs ? (g.total_seqs - b + grid - 1) / grid : 0;
    }
    // Advances to the next item; false after the last one.
    __device__ __forceinline__ bool next(const Args& g) {
        if (++node < n1) return true;
        while (++rd < rounds) {
            const int seq = (int)blockIdx.x + rd * (int)gridDim.x;
            const int per_split = g.m_tiles * g.chunks;
            const int sp = seq / per_split, rem = seq - sp * per_split;
            const int mt = rem / g.chunks, ch = rem - mt * g.chunks;
            node = sp * g.split_len;
            n1 = min(g.nodes, node + g.split_len);
            m0 = mt * kTileM;
            t0 = ch * g.chunk;
            t1 = min(g.n_tiles, t0 + g.chunk);
            if (node < n1) return true;
        }
        return false;
    }
    // The node of the next item when it belongs to the same range, else -1.
    __device__ __forceinline__ int next_in_range() const { return node + 1 < n1 ? node + 1 : -1; }
};

// NT = column tile / 16 (16, 32 or 64 output units per tile); PRECISE: three split MMAs per product.
// mapA: h as (m, k, node), box 128 x 64.  mapB: delta as (n, k, node), box 16 NT x 64.  mapC: as
// (m, n, node) with box 128 x 16 NT, the gradient block (kStore, written) or this weight block of X
// (kRing, read).
//
// Tensor memory columns: [0, 128) two accumulators, then two converted h tiles of 64 heads +
// 64 remainders each.
// MODE: kStore, kGather or kRing (see the head of this file); DEG is the common row degree of W for
// kGather (0 = read it per node).
template <int NT, bool PRECISE, int MODE = kStore, int DEG = 0>
__global__ void __launch_bounds__(MODE == kGather ? kThreadsFused : (MODE == kRing ? kThreadsRing : kThreads), 1)
tc_wgrad_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                const __grid_constant__ CUtensorMap mapC, Args g) {
    constexpr int ROWS_B = 16 * NT;
    constexpr uint32_t A_RAW = a_raw_bytes(), B_RAW = b_raw_bytes(ROWS_B);
    constexpr uint32_t B_CONV = b_conv_bytes(ROWS_B), B_LBO = b_lbo(ROWS_B), SBO = 128;
    constexpr uint32_t NCOPY = PRECISE ? 2 : 1;
    constexpr uint32_t CONV_BUF = NCOPY * B_CONV;
    constexpr bool FUSE = MODE == kGather;            // staged tiles go to the mixer warps instead of a TMA store
    constexpr uint32_t STAGE = stage_bytes(ROWS_B);     // kStore, kGather: output staging; kRing: the tile of X_{i+1}
    constexpr int SB = MODE == kRing ? kStagesBRing : kStagesB;
    constexpr uint32_t WIN_COL0 = A_COL0_ + 2 * kACols;      // kRing: two 64-column slots of the X window
    constexpr uint32_t A_COL0 = A_COL0_;
    constexpr uint32_t TMEM_COLS = 512;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    // threads that split the delta tiles: the converter warps, or in kRing the sixteen mixer warps (the converters
    // of a CTA with one h tile per column tile are the slowest stage otherwise)
    constexpr uint32_t B_CONVERTERS = 128u;
    constexpr uint32_t A_BUFS = MODE == kRing ? 2u : 1u;     // raw h tiles in flight (a new one every column tile in kRing)
    const uint32_t a_raw = base;
    const uint32_t b_raw = a_raw + A_BUFS * A_RAW;
    const uint32_t b_conv = b_raw + SB * B_RAW;
    const uint32_t stage = b_conv + 2 * CONV_BUF;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + A_BUFS * A_RAW + SB * B_RAW + 2 * CONV_BUF + 2 * STAGE);
    uint64_t* a_raw_full = bars;                 // [A_BUFS]
    uint64_t* a_raw_empty = bars + 2;            // [A_BUFS]
    uint64_t* a_conv_full = bars + 4;            // [2]
    uint64_t* a_conv_empty = bars + 6;           // [2]
    uint64_t* b_raw_full = bars + 8;             // [kStagesB]
    uint64_t* b_raw_empty = b_raw_full + kStagesB;
    uint64_t* b_conv_full = b_raw_empty + kStagesB;   // [2]
    uint64_t* b_conv_empty = b_conv_full + 2;    // [2]
    uint64_t* acc_full = b_conv_empty + 2;       // [2]
    uint64_t* acc_empty = acc_full + 2;          // [2]
    uint64_t* stage_free = acc_empty + 2;        // [2] the TMA store that last read the buffer is done reading (kRing: the mixers are)
    uint64_t* stage_ready = stage_free + 2;      // [2] all epilogue threads have written the buffer (kRing: the tile of X has landed)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(stage_ready + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int KS = (g.K + 7) / 8;                // MMAs (k = 8) per product and column tile

    if (tid == 0) {
        for (uint32_t b = 0; b < A_BUFS; ++b) { mbar_init(a_raw_full + b, 1); mbar_init(a_raw_empty + b, 128); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(a_conv_full + b, 128); mbar_init(a_conv_empty + b, 1);
            mbar_init(b_conv_full + b, B_CONVERTERS); mbar_init(b_conv_empty + b, 1);
            mbar_init(acc_full + b, 1); mbar_init(acc_empty + b, MODE == kRing ? 16 : 128);
            mbar_init(stage_free + b, MODE == kStore ? 1 : 32 * kMixWarps); mbar_init(stage_ready + b, MODE == kRing ? 1 : 128);
        }
        for (int s = 0; s < SB; ++s) { mbar_init(b_raw_full + s, 1); mbar_init(b_raw_empty + s, B_CONVERTERS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;

    if (MODE != kRing && warp < 4) {
        // ------------------------------ epilogue: TMEM -> shared memory -> TMA store ------------------------------
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        uint32_t q = 0;
        for (Walk w(g); ok && w.next(g);) {
            for (int t = w.t0; t < w.t1; ++t, ++q) {
                const uint32_t ab = q & 1u, ph = (q >> 1) & 1u;
                const uint32_t st = stage + ab * STAGE;
                if (!FUSE && tid == 0) {     // the store issued two tiles ago has finished reading this staging buffer
                    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    mbar_arrive(stage_free + ab);
                }
                // FUSE: the mixers arrive once they have consumed the tile staged here two tiles ago
                const bool go = mbar_wait(acc_full + ab, ph) && mbar_wait(stage_free + ab, FUSE ? ph ^ 1u : ph);
                if (!__all_sync(0xffffffffu, go)) { ok = false; break; }     // tcgen05.ld needs the whole warp
                tc::tc_fence_after();
#pragma unroll 1
                for (int c0 = 0; c0 < ROWS_B; c0 += 16) {
                    float v[16];
                    tc::tmem_ld16(lane_base + ab * kAccStride + (uint32_t)c0, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) sts32(st + (uint32_t)(c0 + j) * (kTileM * 4) + (uint32_t)tid * 4, v[j]);
                }
                tc::tc_fence_before();
                mbar_arrive(acc_empty + ab);                                 // the accumulator may be overwritten
                if (FUSE) {
                    mbar_arrive(stage_ready + ab);                           // handed to the mixer warps
                    continue;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(stage_ready + ab);
                if (tid == 0) {
                    if (mbar_wait(stage_ready + ab, ph)) {
                        tma_store_3d(&mapC, st, w.m0, t * ROWS_B, w.node);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    } else {
                        atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);     // tile not stored; the others run into their own limits
                    }
                }
            }
        }
        if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores complete before exit
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------ converters ------------------------------
        const uint32_t ct = (uint32_t)tid - 128u, cw = (uint32_t)warp - 4u;
        const uint32_t lane_base = tmem_base + ((cw * 32u) << 16);
        uint32_t q = 0, it = 0;
        for (Walk w(g); ok && w.next(g);) {
            const uint32_t abuf = it & 1u;
            {   // h tile -> tensor memory: row ct of A is column ct of the raw [k][m] tile
                const uint32_t rbuf = it % A_BUFS, a_tile = a_raw + rbuf * A_RAW;
                const bool go = mbar_wait(a_raw_full + rbuf, (it / A_BUFS) & 1u) &&
                                mbar_wait(a_conv_empty + abuf, ((it >> 1) & 1u) ^ 1u);
                if (!__all_sync(0xffffffffu, go)) { ok = false; break; }     // tcgen05.st needs the whole warp
                tc::tc_fence_after();
                const uint32_t a_cols = lane_base + A_COL0 + abuf * kACols;
#pragma unroll 1
                for (int k0 = 0; k0 < g.K; k0 += 16) {
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const float v = lds32(a_tile + (uint32_t)(k0 + k) * (kTileM * 4) + ct * 4);
                        if (PRECISE) tcs::split(v, hi[k], lo[k]);
                        else hi[k] = __float_as_uint(v);
                    }
                    tcs::tmem_st16(a_cols + (uint32_t)k0, hi);
                    if (PRECISE) tcs::tmem_st16(a_cols + kMaxK + (uint32_t)k0, lo);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc::tc_fence_before();
                mbar_arrive(a_conv_full + abuf);
                mbar_arrive(a_raw_empty + rbuf);
            }
            for (int t = w.t0; MODE != kRing && t < w.t1; ++t, ++q) {
                const uint32_t s = q % SB, bb = q & 1u;
                if (!mbar_wait(b_raw_full + s, (q / SB) & 1u) || !mbar_wait(b_conv_empty + bb, ((q >> 1) & 1u) ^ 1u)) {
                    ok = false;
                    break;
                }
                const uint32_t rb = b_raw + s * B_RAW;
                const uint32_t b_hi = b_conv + bb * CONV_BUF, b_lo = b_hi + B_CONV;
#pragma unroll
                for (uint32_t j = 0; j < (uint32_t)(ROWS_B * (kMaxK / 4)) / 128u; ++j) {
                    const uint32_t idx = ct + j * 128u;
                    const uint32_t n = idx % ROWS_B, c = idx / ROWS_B;      // output unit, 16-byte chunk (four k)
                    const uint32_t src = rb + (4 * c) * (ROWS_B * 4) + n * 4;
                    const float4 v = make_float4(lds32(src), lds32(src + ROWS_B * 4), lds32(src + 2 * ROWS_B * 4),
                                                 lds32(src + 3 * ROWS_B * 4));
                    tcs::put<PRECISE>(b_hi, b_lo, c * B_LBO + (n >> 3) * SBO + (n & 7) * 16, v);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(b_conv_full + bb);
                mbar_arrive(b_raw_empty + s);
            }
            ++it;
        }
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    else if (MODE == kRing && warp >= 22) {
        // ------------------------------ kRing: delta converters ------------------------------
        // With one h tile AND one delta tile per item the four converter warps are the slowest stage, and the
        // mixers' chain per item is the next slowest, so the delta tiles get four warps of their own.
        const uint32_t ct = (uint32_t)tid - 704u;
        uint32_t q = 0;
        for (Walk w(g); ok && w.next(g); ++q) {
            const uint32_t s = q % SB, bb = q & 1u;
            if (!mbar_wait(b_raw_full + s, (q / SB) & 1u) || !mbar_wait(b_conv_empty + bb, ((q >> 1) & 1u) ^ 1u)) {
                ok = false;
                break;
            }
            const uint32_t rb = b_raw + s * B_RAW;
            const uint32_t b_hi = b_conv + bb * CONV_BUF, b_lo = b_hi + B_CONV;
#pragma unroll
            for (uint32_t j = 0; j < (uint32_t)(ROWS_B * (kMaxK / 4)) / 128u; ++j) {
                const uint32_t idx = ct + j * 128u;
                const uint32_t n = idx % ROWS_B, c = idx / ROWS_B;      // output unit, 16-byte chunk (four k)
                const uint32_t src = rb + (4 * c) * (ROWS_B * 4) + n * 4;
                const float4 v = make_float4(lds32(src), lds32(src + ROWS_B * 4), lds32(src + 2 * ROWS_B * 4),
                                             lds32(src + 3 * ROWS_B * 4));
                tcs::put<PRECISE>(b_hi, b_lo, c * B_LBO + (n >> 3) * SBO + (n & 7) * 16, v);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(b_conv_full + bb);
            mbar_arrive(b_raw_empty + s);
        }
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    else if (warp == 8) {
        if (lane == 0) {
            // ------------------------------ MMA issuer ------------------------------
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ROWS_B >> 3) << 17) |
                                   ((uint32_t)(kTileM >> 4) << 24);
            uint32_t q = 0, it = 0;
            for (Walk w(g); ok && w.next(g);) {
                const uint32_t abuf = it & 1u;
                if (!mbar_wait(a_conv_full + abuf, (it >> 1) & 1u)) { ok = false; break; }
                const uint32_t a_hi = tmem_base + A_COL0 + abuf * kACols, a_lo = a_hi + kMaxK;
                for (int t = w.t0; t < w.t1; ++t, ++q) {
                    const uint32_t bb = q & 1u, ph = (q >> 1) & 1u;
                    if (!mbar_wait(b_conv_full + bb, ph) || !mbar_wait(acc_empty + bb, ph ^ 1u)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t d = tmem_base + bb * kAccStride;
                    const uint32_t b_hi = b_conv + bb * CONV_BUF, b_lo = b_hi + B_CONV;
                    uint32_t acc = 0;
                    for (int ks = 0; ks < KS; ++ks) {
                        const uint64_t dbh = tc::smem_desc(b_hi + (uint32_t)ks * 2 * B_LBO, B_LBO, SBO);
                        if (PRECISE) {
                            const uint64_t dbl = tc::smem_desc(b_lo + (uint32_t)ks * 2 * B_LBO, B_LBO, SBO);
                            tcs::mma_tf32_ts(d, a_lo + (uint32_t)ks * 8, dbh, idesc, acc); acc = 1;
                            tcs::mma_tf32_ts(d, a_hi + (uint32_t)ks * 8, dbl, idesc, acc);
                        }
                        tcs::mma_tf32_ts(d, a_hi + (uint32_t)ks * 8, dbh, idesc, acc); acc = 1;
                    }
                    tc::mma_commit(b_conv_empty + bb);
                    tc::mma_commit(acc_full + bb);
                }
                if (ok) tc::mma_commit(a_conv_empty + abuf);     // every MMA that reads this h tile has been issued
                ++it;
            }
            if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
        }
    } else if (warp == 9 && lane == 0) {
        // ------------------------------ TMA loads ------------------------------
        uint32_t q = 0, it = 0, xq = 0;          // delta tiles, h tiles and tiles of X issued so far
        for (Walk w(g); ok && w.next(g);) {
            const uint32_t rbuf = it % A_BUFS;
            if (!mbar_wait(a_raw_empty + rbuf, ((it / A_BUFS) & 1u) ^ 1u)) { ok = false; break; }
            mbar_expect_tx(a_raw_full + rbuf, A_RAW);
            tma_load_3d(a_raw + rbuf * A_RAW, &mapA, w.m0, 0, w.node, a_raw_full + rbuf);
            ++it;
            for (int t = w.t0; t < w.t1; ++t, ++q) {
                const uint32_t s = q % SB;
                if (!mbar_wait(b_raw_empty + s, ((q / SB) & 1u) ^ 1u)) { ok = false; break; }
                mbar_expect_tx(b_raw_full + s, B_RAW);
                tma_load_3d(b_raw + s * B_RAW, &mapB, t * ROWS_B, 0, w.node, b_raw_full + s);
            }
            if (MODE == kRing) {
                // the tile of X_{node+1}: the one tile of X this node step reads from memory; after the loads the
                // converters wait for, so that its gate (the mixers, two nodes back) never holds those up
                const uint32_t xs = xq & 1u;
                if (!ok || !mbar_wait(stage_free + xs, ((xq >> 1) & 1u) ^ 1u)) { ok = false; break; }
                mbar_expect_tx(stage_ready + xs, STAGE);
                tma_load_3d(stage + xs * STAGE, &mapC, w.m0, w.t0 * ROWS_B, w.node + 1 == g.nodes ? 0 : w.node + 1,
                            stage_ready + xs);
                ++xq;
            }
        }
        // loads still in flight (only when somebody gave up): let them land before the CTA leaves
        for (uint32_t j = 0; j < A_BUFS && j < it; ++j) {
            const uint32_t ii = it - 1 - j;
            mbar_wait(a_raw_full + ii % A_BUFS, (ii / A_BUFS) & 1u);
        }
        for (uint32_t j = 0; j < (uint32_t)SB && j < q; ++j) {
            const uint32_t qq = q - 1 - j;
            mbar_wait(b_raw_full + qq % SB, (qq / SB) & 1u);
        }
        for (uint32_t j = 0; MODE == kRing && j < 2u && j < xq; ++j) {
            const uint32_t qq = xq - 1 - j;
            mbar_wait(stage_ready + (qq & 1u), (qq >> 1) & 1u);
        }
        if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    if (MODE == kRing && (warp < 4 || (warp >= 10 && warp < 22))) {
        // ------------------------------ ring mixers: X window in tensor memory ------------------------------
        // Thread = (row m of the tile, 16 of its 64 columns): the accumulator's own layout, so a tile needs
        // no staging.  The CTA walks consecutive nodes i at one tile position; the tiles of X_{i-1} and X_i
        // are kept in two 64-column slots of tensor memory (each thread's own lane and columns: no
        // synchronisation), so only X_{i+1} is read from memory - one read of X per element - from the
        // shared-memory stage that the TMA thread filled one to two nodes ahead.
        // sixteen warps: lane quarter warp % 4 (the lanes a warp may address), column group by warp:
        // 0-3 -> 0, 12-15 -> 1, 16-19 -> 2, {20, 21, 10, 11} -> 3
        const int quarter = warp & 3, cg = warp < 4 ? 0 : (warp < 12 || warp >= 20 ? 3 : ((warp - 12) >> 2) + 1);
        const int m = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t win[2] = {lane_addr + WIN_COL0 + (uint32_t)cg * 16, lane_addr + WIN_COL0 + 64 + (uint32_t)cg * 16};
        const int64_t cstride = g.M;                         // one output unit further = din elements further
        const uint32_t xt_off = (uint32_t)(cg * 16) * (kTileM * 4) + (uint32_t)m * 4;   // this thread's corner of a staged tile of X
        auto load16 = [&](const float* p, int ncols, float (&v)[16]) {
            if (ncols == 16) {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = __ldcg(p + j * cstride);
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = j < ncols ? __ldcg(p + j * cstride) : 0.f;
            }
        };
        const int b = (int)blockIdx.x, grid = (int)gridDim.x;
        const int rounds = b < g.total_seqs ? (g.total_seqs - b + grid - 1) / grid : 0;
        const int per_split = g.m_tiles * g.chunks;
        uint32_t q = 0;
        for (int rd = 0; rd < rounds && ok; ++rd) {
            // one node range at one tile position (decoded as in Walk; chunk == 1: one column tile)
            const int seq = b + rd * grid;
            const int sp = seq / per_split, rem = seq - sp * per_split;
            const int mt = rem / g.chunks, t = rem - mt * g.chunks;
            const int n0 = sp * g.split_len, n1 = min(g.nodes, n0 + g.split_len);
            const int m0 = mt * kTileM, c0 = t * ROWS_B + cg * 16;
            const int ncols = m0 + m < g.M ? max(0, min(16, g.N - c0)) : 0;
            const int64_t pos = g.mix.w_off + (int64_t)c0 * g.M + m0 + m;
            const float* xpos = g.mix.X + pos;
            float* opos = g.mix.Xn + pos;
            for (int node = n0; node < n1; ++node, ++q) {
                const bool cold = node == n0;                // first node of the range: nothing kept yet
                const float wl = __ldg(g.mix.band + 3 * node), ws = __ldg(g.mix.band + 3 * node + 1),
                            wr = __ldg(g.mix.band + 3 * node + 2);
                float xr[16], tmp[16];
                uint32_t bits[16];
                const uint32_t jj = (uint32_t)(node - n0);
                // X_{i+1}: the one tile read from memory, staged by the TMA thread (zero outside the block)
                {
                    const uint32_t xs = q & 1u;
                    const bool landed = mbar_wait(stage_ready + xs, (q >> 1) & 1u);
                    if (!__all_sync(0xffffffffu, landed)) { ok = false; break; }
                    const uint32_t xt = stage + xs * STAGE + xt_off;
#pragma unroll
                    for (int j = 0; j < 16; ++j) xr[j] = lds32(xt + (uint32_t)j * (kTileM * 4));
                }
                if (cold) load16(xpos + (int64_t)(node == 0 ? g.nodes - 1 : node - 1) * g.mix.ld, ncols, tmp);
                else tc::tmem_ld16(win[(jj - 1) & 1u], tmp);                     // X_{i-1}
#pragma unroll
                for (int j = 0; j < 16; ++j) bits[j] = __float_as_uint(xr[j]);
                mbar_arrive(stage_free + (q & 1u));                              // this thread's part of the stage is in registers
                tcs::tmem_st16(cold ? win[1] : win[(jj - 1) & 1u], bits);        // X_{i+1} takes its place
#pragma unroll
                for (int j = 0; j < 16; ++j) xr[j] = fmaf(wr, xr[j], wl * tmp[j]);   // accumulated in place
                if (cold) {
                    load16(xpos + (int64_t)node * g.mix.ld, ncols, tmp);         // X_i
#pragma unroll
                    for (int j = 0; j < 16; ++j) bits[j] = __float_as_uint(tmp[j]);
                    tcs::tmem_st16(win[0], bits);                                // the next node's left neighbour
                } else {
                    tc::tmem_ld16(win[jj & 1u], tmp);                            // X_i
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) xr[j] = fmaf(ws, tmp[j], xr[j]);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                const uint32_t ab = q & 1u, ph = (q >> 1) & 1u;
                const bool go = mbar_wait(acc_full + ab, ph);
                if (!__all_sync(0xffffffffu, go)) { ok = false; break; }     // tcgen05.ld needs the whole warp
                tc::tc_fence_after();
                tc::tmem_ld16(lane_addr + ab * kAccStride + (uint32_t)cg * 16, tmp);
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty + ab);                  // the accumulator may be overwritten
                float* out = opos + (int64_t)node * g.mix.ld;
                if (ncols == 16) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) __stcs(out + j * cstride, fmaf(g.mix.ngamma, tmp[j], xr[j]));
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (j < ncols) __stcs(out + j * cstride, fmaf(g.mix.ngamma, tmp[j], xr[j]));
                }
            }
        }
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    if (FUSE && warp >= 10) {
        // ------------------------------ mixers: gossip step on staged tiles ------------------------------
        const int mw = warp - 10;
        uint32_t q = 0;
        for (Walk w(g); ok && w.next(g);) {
            // the next item of this CTA, when it is the next node of the same range
            const int next_node = w.next_in_range();
            for (int t = w.t0; t < w.t1; ++t, ++q) {
                const uint32_t ab = q & 1u, ph = (q >> 1) & 1u;
                if (!mbar_wait(stage_ready + ab, ph)) { ok = false; break; }
                if (next_node >= 0) {
                    // The same tile position of the next node's neighbours, one 128-byte line per thread and
                    // neighbour: whatever is not in L2 yet (for a ring, one tile of three) is on its way
                    // before the gather of the next item asks for it.
                    const int line = mw * 32 + lane, row = line >> 2, seg = line & 3;
                    if (row < min(ROWS_B, g.N - t * ROWS_B) && w.m0 + seg * 32 < g.M) {
                        const int64_t o = g.mix.w_off + (int64_t)(t * ROWS_B + row) * g.M + w.m0 + seg * 32;
                        const int pe = __ldg(g.mix.row_ptr + next_node + 1);
                        for (int p = __ldg(g.mix.row_ptr + next_node); p < pe; ++p)
                            prefetch_l2(g.mix.X + (int64_t)__ldg(g.mix.col + p) * g.mix.ld + o);
                    }
                }
                const int64_t off = g.mix.w_off + (int64_t)(t * ROWS_B) * g.M + w.m0 + lane * 4;
                mix_rows<DEG, ROWS_B>(g.mix, w.node, stage + ab * STAGE, off, g.M, g.N - t * ROWS_B,
                                      w.m0 + lane * 4 < g.M, mw, lane);
                mbar_arrive(stage_free + ab);
            }
        }
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace tcw
}  // namespace dpsgd
