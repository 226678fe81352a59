// Weight-streaming batched GEMM for the MLP forward and input-gradient products (Algorithm 1 step 3):
//
//     C[n][m] = epilogue( sum_k A(m,k) * B(n,k) )      one problem per node,  N = minibatch <= 128
//
// A is a weight matrix inside the node's parameter row (the long stream: every element is used
// once), B the node's activations or back-propagated errors (small, k-contiguous).  Same tcgen05
// TF32 arithmetic as tc_gemm.cuh (three MMAs on split operands, fp32 accumulation in TMEM).  With a
// minibatch of 64 columns an MMA that takes A from shared memory is bound by that fetch (4 KB of A
// per 128x64x8 MMA), and the split copies double it; so here A is handed to the tensor core in
// TENSOR MEMORY (row m on lane m, element k in column k), which takes the weights off the
// shared-memory pipe after their one staging pass:
//
//   TMA warp        one thread walks the CTA's tiles and k-blocks ahead of everyone else and issues
//                   cp.async.bulk.tensor loads of the raw fp32 tiles (A: 128 x 32 k, B: N x 32 k)
//                   into a ring of stages; no registers, no thread waits on HBM.
//   converter warps (4) read a landed stage from shared memory and split each value into its TF32
//                   head and remainder.  Thread t owns row t of the A tile: it writes the 32 heads
//                   and 32 remainders of its row to its TMEM lane with tcgen05.st.  B is written to
//                   shared memory in the no-swizzle K-major layout of the MMA descriptors, element
//                   (r,k) at (k/4)*LBO + (r/8)*128 + (r%8)*16 + (k%4)*4.  A k-contiguous tile is
//                   loaded with the 128-byte TMA swizzle (16-byte chunk index xor row%8) so that
//                   these reads are conflict-free; an m-contiguous tile (the transposed weight of
//                   the input gradient) is loaded plain as [k][m] and read by lanes that run along
//                   m, which transposes it on the way.  Converted operands are double-buffered.
//   MMA warp        one thread issues the MMAs of a converted k-block (A from TMEM, B through a
//                   descriptor); tcgen05.commit hands the buffers back to the converters.
//   epilogue        the converter warps read the accumulator of a finished tile with tcgen05.ld and
//                   store with m contiguous across lanes.
//
// CTAs are persistent: tile = blockIdx.x + i * gridDim.x over nodes x ceil(M/128) for the rounds that fill
// every CTA; the tiles left over after those rounds (1792 tiles on 296 CTAs: 16, which would cost a seventh
// round for 0.05 rounds of work) are cut by k-blocks instead: their (tile, k-block) pairs form one sequence,
// every CTA takes an equal part of it, writes the raw accumulator of each part to a scratch buffer, and
// stream_fixup_kernel adds the parts of a tile in k order and applies the epilogue.  The loads of the next tile are in flight while
// the current one is converted and drained; two CTAs share an SM and cover each other's serial sections.  Out-of-range rows, columns and k are zero-filled by the
// TMA unit.  Every mbarrier wait is bounded; a wait that runs out raises the status word, the TMA
// thread waits (bounded) for its loads in flight, and the CTA frees its TMEM columns before it
// returns.
#pragma once
#include <cuda.h>
#include "tc_gemm.cuh"

namespace dpsgd {
namespace tcs {

using tc::mbar_arrive;
using tc::mbar_init;
using tc::mbar_wait;
using tc::smem_u32;

constexpr int kConvThreads = 128;
constexpr int kThreads = 192;        // 4 converter/epilogue warps + MMA warp + TMA warp
constexpr int kTileM = 128;
constexpr int kBK = 32;              // fp32 elements along k per stage: one 128-byte swizzle row
constexpr int kChunks = kBK / 4;

struct Args {
    float* C; int64_t c_node; int64_t c_pitch;                      // C[n*c_pitch + m]
    const float* aux; int64_t aux_node; int64_t aux_pitch;          // bias[m] or mask[n*aux_pitch + m]
    int M, N, K;
    int m_tiles, total_tiles;                                       // ceil(M/128), nodes * m_tiles
    int epi;
    int* status;
    float* partial;          // [gridDim.x][2][16 NT][128]: accumulators of the tiles a CTA shares with a neighbour
};

// The work of a CTA, segment by segment: segment = (tile, k-blocks [kb0, kb1)).  First whole tiles, strided
// (tile = cta + i * ctas for the rounds that fill every CTA: CTAs that run side by side then work on
// neighbouring tiles of the same nodes and share their activations in L2); then the tiles left over
// (fewer than ctas), whose k-blocks are dealt out evenly as one sequence, every CTA one contiguous range.
struct Seg { int tile, kb0, kb1, slot; };     // slot: scratch slot of a left-over segment (0: first tile of the range, 1: a later one)
struct SegWalk {
    int i, rounds, KB, cta, ctas, first_left;
    int u, u1, t_first;      // this CTA's range of the left-over k-blocks, the left-over tile it starts in
    __device__ __forceinline__ SegWalk(int total_tiles, int KB_, unsigned cta_, unsigned ctas_)
        : i(0), KB(KB_), cta((int)cta_), ctas((int)ctas_) {
        rounds = total_tiles / ctas;
        first_left = rounds * ctas;
        const long long left = (long long)(total_tiles - first_left) * KB;
        u = (int)(cta * left / ctas);
        u1 = (int)((cta + 1) * left / ctas);
        t_first = u / KB;
    }
    __device__ __forceinline__ bool next(Seg& s) {
        if (i < rounds) {
            s.tile = cta + i * ctas; s.kb0 = 0; s.kb1 = KB; s.slot = 0;
            ++i;
            return true;
        }
        if (u >= u1) return false;
        const int t = u / KB, t0 = t * KB, end = min(t0 + KB, u1);
        s.tile = first_left + t; s.kb0 = u - t0; s.kb1 = end - t0; s.slot = t == t_first ? 0 : 1;
        u = end;
        return true;
    }
};

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}

__host__ __device__ constexpr uint32_t conv_lbo(int rows) { return (uint32_t)rows * 16; }
__host__ __device__ constexpr uint32_t conv_tile(int rows) { return kChunks * conv_lbo(rows); }
__host__ __device__ constexpr uint32_t raw_tile(int rows) { return (uint32_t)rows * kBK * 4; }
__host__ __device__ constexpr int stages(int nt) { return nt <= 4 ? 3 : 4; }
constexpr int kConvBufs = 2;         // converted operands: one being multiplied, one being written

template <int NT, bool PRECISE>
constexpr size_t smem_bytes() {
    return 1024 + (size_t)stages(NT) * (raw_tile(kTileM) + raw_tile(16 * NT)) +
           (size_t)kConvBufs * (PRECISE ? 2 : 1) * conv_tile(16 * NT) + 128;
}

template <bool PRECISE>
__device__ __forceinline__ void put(uint32_t hi, uint32_t lo, uint32_t off, float4 v) {
    if (PRECISE) {
        float4 h, l;
        h.x = tc::tf32_head(v.x); l.x = v.x - h.x;
        h.y = tc::tf32_head(v.y); l.y = v.y - h.y;
        h.z = tc::tf32_head(v.z); l.z = v.z - h.z;
        h.w = tc::tf32_head(v.w); l.w = v.w - h.w;
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(hi + off), "f"(h.x), "f"(h.y), "f"(h.z), "f"(h.w) : "memory");
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(lo + off), "f"(l.x), "f"(l.y), "f"(l.z), "f"(l.w) : "memory");
    } else {
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(hi + off), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
    }
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float lds32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// TF32 head and remainder of one value.
__device__ __forceinline__ void split(float v, uint32_t& hi, uint32_t& lo) {
    const float h = tc::tf32_head(v);
    hi = __float_as_uint(h);
    lo = __float_as_uint(v - h);
}

// 16 consecutive columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// A from tensor memory (row m on lane m, element k in column k), B through a shared-memory descriptor.
__device__ __forceinline__ void mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// NT = column tile / 16 (rows of B per tile, >= N); A_K: A contiguous along k in memory (forward)
// or along m (input gradient); PRECISE: three split MMAs per product.
//
// Tensor memory columns of a CTA: [0, 16 NT) accumulator, then per converted buffer 32 columns of
// heads and (PRECISE) 32 of remainders.
template <int NT, bool A_K, bool PRECISE>
__global__ void __launch_bounds__(kThreads, NT <= 4 ? 2 : 1)
tc_stream_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, Args g) {
    constexpr int ROWS_B = 16 * NT;
    constexpr int S = stages(NT);
    constexpr uint32_t A_RAW = raw_tile(kTileM), B_RAW = raw_tile(ROWS_B), RAW = A_RAW + B_RAW;
    constexpr uint32_t B_CONV = conv_tile(ROWS_B), B_LBO = conv_lbo(ROWS_B), SBO = 128;
    constexpr uint32_t NCOPY = PRECISE ? 2 : 1;
    constexpr uint32_t CONV_BUF = NCOPY * B_CONV;                     // B hi | B lo of one buffer
    constexpr uint32_t ACC_COLS = ROWS_B < 32 ? 32 : ROWS_B;
    constexpr uint32_t A_COLS = NCOPY * kBK;                          // per buffer
    constexpr uint32_t USED_COLS = ACC_COLS + kConvBufs * A_COLS;
    constexpr uint32_t TMEM_COLS = USED_COLS <= 64 ? 64 : (USED_COLS <= 128 ? 128 : 256);
    static_assert(USED_COLS <= 256, "two CTAs share the 512 columns of an SM");
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // swizzled tiles want 1024-byte alignment
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t conv = base + S * RAW;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + S * RAW + kConvBufs * CONV_BUF);
    uint64_t* raw_full = bars;                        // [S] TMA bytes landed
    uint64_t* raw_empty = bars + S;                   // [S] converters are done reading the stage
    uint64_t* conv_full = bars + 2 * S;               // [2] converted k-block written
    uint64_t* conv_empty = conv_full + kConvBufs;     // [2] MMAs that read it have completed
    uint64_t* acc_full = conv_empty + kConvBufs;      // accumulator of a tile complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int KB = (g.K + kBK - 1) / kBK;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(raw_full + s, 1); mbar_init(raw_empty + s, kConvThreads); }
        for (int b = 0; b < kConvBufs; ++b) { mbar_init(conv_full + b, kConvThreads); mbar_init(conv_empty + b, 1); }
        mbar_init(acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        // ------------------------------ converters, then epilogue ------------------------------
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        uint32_t q = 0, done_tiles = 0;
        SegWalk walk(g.total_tiles, KB, blockIdx.x, gridDim.x);
        Seg sg;
        for (; ok && walk.next(sg); ++done_tiles) {
            const int tile = sg.tile;
            const int node = tile / g.m_tiles;
            const int m0 = (tile - node * g.m_tiles) * kTileM;
            for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++q) {
                const uint32_t s = q % S, buf = q & 1u;
                const bool landed = mbar_wait(raw_full + s, (q / S) & 1u) &&
                                    mbar_wait(conv_empty + buf, ((q >> 1) & 1u) ^ 1u);
                if (!__all_sync(0xffffffffu, landed)) { ok = false; break; }   // tcgen05.st needs the whole warp
                tc::tc_fence_after();
                const uint32_t ra = base + s * RAW, rb = ra + A_RAW;
                const uint32_t a_cols = lane_base + ACC_COLS + buf * A_COLS;       // heads, then remainders
                // row tid of the A tile, 16 k at a time, into this thread's TMEM lane
#pragma unroll
                for (uint32_t half = 0; half < 2; ++half) {
                    float v[16];
                    if (A_K) {  // raw A: 128 rows of 128 bytes, 16-byte chunk c of row r at chunk c ^ (r % 8)
                        const uint32_t r = tid;
#pragma unroll
                        for (uint32_t c = 0; c < 4; ++c) {
                            const float4 t = lds128(ra + r * 128 + (((4 * half + c) ^ (r & 7)) << 4));
                            v[4 * c] = t.x; v[4 * c + 1] = t.y; v[4 * c + 2] = t.z; v[4 * c + 3] = t.w;
                        }
                    } else {    // raw A: 32 k-rows of 128 m: column tid, which transposes the tile
#pragma unroll
                        for (uint32_t k = 0; k < 16; ++k) v[k] = lds32(ra + (16 * half + k) * (kTileM * 4) + tid * 4);
                    }
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        if (PRECISE) split(v[k], hi[k], lo[k]);
                        else hi[k] = __float_as_uint(v[k]);
                    }
                    tmem_st16(a_cols + 16 * half, hi);
                    if (PRECISE) tmem_st16(a_cols + kBK + 16 * half, lo);
                }
                const uint32_t b_hi = conv + buf * CONV_BUF, b_lo = b_hi + B_CONV;
#pragma unroll
                for (uint32_t j = 0; j < (uint32_t)(ROWS_B * kChunks) / kConvThreads; ++j) {
                    const uint32_t idx = tid + j * kConvThreads;
                    const uint32_t r = idx % ROWS_B, c = idx / ROWS_B;
                    put<PRECISE>(b_hi, b_lo, c * B_LBO + (r >> 3) * SBO + (r & 7) * 16,
                                 lds128(rb + r * 128 + ((c ^ (r & 7)) << 4)));
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc::tc_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(conv_full + buf);
                mbar_arrive(raw_empty + s);
            }
            if (ok && !mbar_wait(acc_full, done_tiles & 1u)) ok = false;
            ok = __all_sync(0xffffffffu, ok);                   // tcgen05.ld below needs the whole warp
            if (!ok) break;
            tc::tc_fence_after();
            if (sg.kb0 != 0 || sg.kb1 != KB) {
                // part of a left-over tile: the raw accumulator goes to one of this CTA's two scratch slots
                float* part = g.partial + ((int64_t)blockIdx.x * 2 + sg.slot) * (ROWS_B * kTileM) + tid;
#pragma unroll 1
                for (int c0 = 0; c0 < ROWS_B; c0 += 16) {
                    if (c0 >= g.N) break;
                    float v[16];
                    tc::tmem_ld16(lane_base + (uint32_t)c0, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) part[(c0 + j) * kTileM] = v[j];
                }
                tc::tc_fence_before();
                continue;
            }
            const int m = m0 + warp * 32 + lane;
            float* C = g.C + (int64_t)node * g.c_node;
            const float* aux = g.aux ? g.aux + (int64_t)node * g.aux_node : nullptr;
            const float bias = (g.epi <= tc::EPI_BIAS && m < g.M) ? __ldg(aux + m) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < ROWS_B; c0 += 16) {
                if (c0 >= g.N) break;
                float v[16];
                tc::tmem_ld16(lane_base + (uint32_t)c0, v);
                const int cnt = m < g.M ? min(16, g.N - c0) : 0;
                float* out = C + (int64_t)c0 * g.c_pitch + m;
                if (g.epi == tc::EPI_MASK) {
                    const float* mk = aux + (int64_t)c0 * g.aux_pitch + m;
                    float gate[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) gate[j] = j < cnt ? __ldg(mk + (int64_t)j * g.aux_pitch) : 0.f;
#pragma unroll
                    for (int j = 0; j < 16; ++j) if (j < cnt) out[(int64_t)j * g.c_pitch] = gate[j] > 0.f ? v[j] : 0.f;
                } else {
                    const bool relu = g.epi == tc::EPI_BIAS_RELU;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float x = v[j] + bias;
                        if (j < cnt) out[(int64_t)j * g.c_pitch] = (relu && x < 0.f) ? 0.f : x;
                    }
                }
            }
            tc::tc_fence_before();      // the accumulator reads above precede the next tile's first MMA
        }
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    } else if (warp == 4) {
        if (lane == 0) {
            // ------------------------------ MMA issuer ------------------------------
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ROWS_B >> 3) << 17) |
                                   ((uint32_t)(kTileM >> 4) << 24);
            bool ok = true;
            uint32_t q = 0;
            SegWalk walk(g.total_tiles, KB, blockIdx.x, gridDim.x);
            Seg sg;
            while (ok && walk.next(sg)) {
                uint32_t acc = 0;                               // the first MMA of a segment overwrites the accumulator
                for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++q) {
                    const uint32_t buf = q & 1u;
                    if (!mbar_wait(conv_full + buf, (q >> 1) & 1u)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t a_hi = tmem_base + ACC_COLS + buf * A_COLS, a_lo = a_hi + kBK;
                    const uint32_t b_hi = conv + buf * CONV_BUF, b_lo = b_hi + B_CONV;
#pragma unroll
                    for (uint32_t kk = 0; kk < kBK / 8; ++kk) {  // one MMA consumes k = 8: 8 columns of A, two chunk columns of B
                        if ((int)(kb * kBK + kk * 8) >= g.K) break;   // nothing but zero fill from here on
                        const uint64_t dbh = tc::smem_desc(b_hi + kk * 2 * B_LBO, B_LBO, SBO);
                        if (PRECISE) {
                            const uint64_t dbl = tc::smem_desc(b_lo + kk * 2 * B_LBO, B_LBO, SBO);
                            mma_tf32_ts(tmem_base, a_lo + kk * 8, dbh, idesc, acc); acc = 1;
                            mma_tf32_ts(tmem_base, a_hi + kk * 8, dbl, idesc, acc);
                        }
                        mma_tf32_ts(tmem_base, a_hi + kk * 8, dbh, idesc, acc); acc = 1;
                    }
                    tc::mma_commit(conv_empty + buf);           // frees the buffer once these MMAs have read it
                }
                if (ok) tc::mma_commit(acc_full);
            }
            if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
        }
    } else if (lane == 0) {
        // ------------------------------ TMA issuer ------------------------------
        bool ok = true;
        uint32_t q = 0;
        SegWalk walk(g.total_tiles, KB, blockIdx.x, gridDim.x);
        Seg sg;
        while (ok && walk.next(sg)) {
            const int node = sg.tile / g.m_tiles;
            const int m0 = (sg.tile - node * g.m_tiles) * kTileM;
            for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++q) {
                const uint32_t s = q % S;
                if (!mbar_wait(raw_empty + s, ((q / S) & 1u) ^ 1u)) { ok = false; break; }
                const uint32_t ra = base + s * RAW;
                mbar_expect_tx(raw_full + s, RAW);
                if (A_K) tma_load_3d(ra, &mapA, kb * kBK, m0, node, raw_full + s);
                else tma_load_3d(ra, &mapA, m0, kb * kBK, node, raw_full + s);
                tma_load_3d(ra + A_RAW, &mapB, kb * kBK, 0, node, raw_full + s);
            }
        }
        // loads still in flight (only when somebody gave up): let them land before the CTA leaves
        for (uint32_t j = 0; j < (uint32_t)S && j < q; ++j) {
            const uint32_t qq = q - 1 - j;
            mbar_wait(raw_full + qq % S, (qq / S) & 1u);
        }
        if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// Adds the parts of every left-over tile (in k order) and applies the epilogue.  One CTA per (left-over tile,
// sample), thread = row of the tile.  rows = 16 NT of the stream kernel, ctas = its grid.
static __global__ void __launch_bounds__(kTileM)
stream_fixup_kernel(Args g, int rows, int ctas) {
    const int KB = (g.K + kBK - 1) / kBK;
    const int first_left = (g.total_tiles / ctas) * ctas;
    const long long left = (long long)(g.total_tiles - first_left) * KB;
    const int t = (int)blockIdx.x, tile = first_left + t;
    const int t0 = t * KB, t1 = t0 + KB;
    auto start = [&](int bb) { return (int)(bb * left / ctas); };     // first left-over k-block of stream CTA bb
    int bb0 = (int)((long long)t0 * ctas / left);                     // the CTA whose range holds k-block t0
    while (bb0 > 0 && start(bb0) > t0) --bb0;
    while (bb0 + 1 < ctas && start(bb0 + 1) <= t0) ++bb0;
    if (start(bb0) <= t0 && start(bb0 + 1) >= t1) return;             // one CTA ran the whole tile and finished it
    const int node = tile / g.m_tiles;
    const int m = (tile - node * g.m_tiles) * kTileM + (int)threadIdx.x;
    if (m >= g.M) return;
    float* C = g.C + (int64_t)node * g.c_node + m;
    const float* aux = g.aux ? g.aux + (int64_t)node * g.aux_node : nullptr;
    const int n = (int)blockIdx.y;                                    // one sample (column of the tile) per CTA
    const float* part = g.partial + n * kTileM + threadIdx.x;
    const int64_t pstride = (int64_t)2 * rows * kTileM;               // from one CTA's slot 0 to the next CTA's
    float s;
    if (left >= ctas) {
        // no range is empty: the parts are those of CTAs bb0 .. bb1 - 1, all but possibly the first in slot 0,
        // and their loads do not depend on one another
        int bb1 = (int)(((long long)t1 * ctas + left - 1) / left);   // first CTA whose range starts at or after t1
        while (bb1 > bb0 + 1 && start(bb1 - 1) >= t1) --bb1;
        while (bb1 < ctas && start(bb1) < t1) ++bb1;
        s = __ldcg(part + bb0 * pstride + (start(bb0) >= t0 ? 0 : rows * kTileM));
#pragma unroll 8
        for (int bb = bb0 + 1; bb < bb1; ++bb) s += __ldcg(part + bb * pstride);
    } else {
        // start(bb + 1) from start(bb) without a division: floor(bb * left / ctas) grows by 0 or 1
        const int r = (int)left;
        int u0 = start(bb0), err = (int)((long long)bb0 * left % ctas);
        s = 0.f;
        for (int bb = bb0; bb < ctas && u0 < t1; ++bb) {              // the CTAs whose ranges meet this tile, in k order
            int u1 = u0;
            err += r;
            if (err >= ctas) { err -= ctas; ++u1; }
            if (u1 > u0 && u1 > t0) s += __ldcg(part + bb * pstride + (u0 >= t0 ? 0 : rows * kTileM));
            u0 = u1;
        }
    }
    if (g.epi == tc::EPI_MASK) {
        C[(int64_t)n * g.c_pitch] = __ldg(aux + (int64_t)n * g.aux_pitch + m) > 0.f ? s : 0.f;
    } else {
        const float x = s + (g.epi <= tc::EPI_BIAS ? __ldg(aux + m) : 0.f);
        C[(int64_t)n * g.c_pitch] = (g.epi == tc::EPI_BIAS_RELU && x < 0.f) ? 0.f : x;
    }
}

}  // namespace tcs
}  // namespace dpsgd
