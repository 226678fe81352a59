// Batched skinny GEMM on the 5th-generation tensor cores for the MLP gradients (Algorithm 1 step 3).
//
//     C[n][m] = epilogue( sum_k A(m,k) * B(n,k) )         one problem per node (blockIdx.z)
//
// The long (weight) dimension m sits on the 128 TMEM lanes, the short one (batch, or a 16..128 wide
// slice) on the TMEM columns.  tcgen05.mma kind::tf32 multiplies 10-bit-mantissa operands, so an
// fp32-faithful product is built from three MMAs on split operands (a = a_hi + a_lo):
//     a*b ~= a_hi*b_hi + a_lo*b_hi + a_hi*b_lo        (fp32 accumulation in TMEM)
// The operands are fp32 in HBM.  Four loader warps read them with 128-bit loads, 64 k at a time,
// shaped so that one warp instruction covers 256 contiguous bytes of a row (k-contiguous operand)
// or 128 bytes of each of four k-rows (operand contiguous along m / n): measured on B200, 64-byte
// pieces reach 2.5 TB/s, full 128-byte lines 3.5 and 256-byte runs 5.1.  The values are split in
// registers and written as hi / lo copies to shared memory directly in the no-swizzle K-major
// layout the MMA descriptors describe: element (r,k) at (k/4)*LBO + (r/8)*SBO + (r%8)*16 + (k%4)*4.
// The descriptor arithmetic is linear in its two strides, so they carry 16 bytes of padding that
// spreads the loaders' 128-bit stores over the banks.  An operand that is contiguous along m / n is
// transposed on the way, 4x4 blocks at a time in registers.  (tcgen05 has no no-swizzle MN-major
// mode for 32-bit operands.)  One thread of a fifth warp
// issues the MMAs; tcgen05.commit releases a stage back to the loaders; the loader warps then
// read the accumulator with tcgen05.ld and apply the epilogue with coalesced stores (m contiguous).
// Every mbarrier wait is bounded; a wait that runs out raises the status word, and the CTA still
// frees its TMEM columns before it returns.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dpsgd {
namespace tc {

constexpr int kLoaderThreads = 128;
constexpr int kThreads = 160;          // 4 loader/epilogue warps + 1 MMA warp
constexpr int kTileM = 128;
constexpr int kBlockK = 64;            // fp32 elements per pipeline stage along k (8 MMAs of K = 8)
constexpr int kChunks = kBlockK / 4;   // 16-byte chunk columns per stage
constexpr int kStages = 1;            // one stage per CTA: four CTAs share an SM and overlap each other
constexpr uint32_t kWaitSpins = 1u << 20;

enum { EPI_BIAS_RELU = 0, EPI_BIAS = 1, EPI_STORE = 2, EPI_MASK = 3 };

struct Args {
    const float* A; int64_t a_node; int64_t a_pitch; int a_kcontig; int a_vec;   // A(m,k)
    const float* B; int64_t b_node; int64_t b_pitch; int b_kcontig; int b_vec;   // B(n,k)
    float* C; int64_t c_node; int64_t c_pitch;                                   // C[n*c_pitch + m]
    const float* aux; int64_t aux_node; int64_t aux_pitch;                       // bias[m] or mask[n*aux_pitch + m]
    int M, N, K;
    int n_per_cta;     // column tiles one CTA walks through (the A tile is kept when K fits one k-block)
    int epi;
    int precise;       // 1: three split MMAs per product, 0: one TF32 MMA
    int* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One poll of a phase.  The suspend-time hint lets the hardware park the thread until the phase completes (it is
// woken then) or the hint runs out, instead of returning after its short default slice.  Measured on the fused
// weight-gradient kernel (two dozen warps, most of them waiting at any time): 4 % shorter per work item than tight polling,
// which competes with the converting warps for their SM partition's issue slots and shared-memory queue.
constexpr uint32_t kSuspendNs = 2000;
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendNs) : "memory");
    return ok != 0;
}
// Bounded wait: kWaitSpins polls of at most kSuspendNs each (about two seconds), then false.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t spin = 0; spin < kWaitSpins; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// Shared-memory matrix descriptor, no swizzle: start address, leading / stride byte offsets in
// 16-byte units, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// TF32 head of v: v with its low 13 mantissa bits cleared (truncation), so that the remainder v - head is
// exact in fp32 and has the sign of v.  Rounding the head to nearest instead halves the remainder, but the
// extra integer add per element cost 4 % of the fused iteration on B200 (the converter warps are the
// critical stage) and made no difference to the outcome of the parity tests against the fp64 oracle.
__device__ __forceinline__ float tf32_head(float v) {
    return __uint_as_float(__float_as_uint(v) & 0xFFFFE000u);
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}

// Shared-memory layout of a ROWS-row operand tile: element (r,k) at
//     (k/4)*LBO + (r/8)*SBO + (r%8)*16 + (k%4)*4.
// The descriptor arithmetic is linear, so both strides can carry padding that spreads the loader's
// 128-bit stores over the banks: a k-contiguous operand is stored by lanes that run along k (pad LBO
// by 16 bytes), a transposed one by lanes that run along rows, four rows apart (pad SBO by 16 bytes).
__host__ __device__ constexpr uint32_t tile_sbo(bool kc) { return kc ? 128u : 144u; }
__host__ __device__ constexpr uint32_t tile_lbo(int rows, bool kc) {
    return kc ? (uint32_t)rows * 16 + 16 : (uint32_t)(rows / 8) * 144;
}
__host__ __device__ constexpr uint32_t tile_bytes(int rows, bool kc) { return kChunks * tile_lbo(rows, kc); }

// One loader thread's share of an operand tile (ROWS x 64 k) as 16-byte chunks, i.e. four
// consecutive elements along the operand's contiguous direction.
//   KC  : the operand is contiguous along k in memory (element (r,k) at r*pitch + k).  Lanes 0-15
//         cover the 16 chunks (256 bytes) of one row, lanes 16-31 the next row; a chunk is stored
//         as it is (four k of one row).
//   !KC : it is contiguous along its row index (element (r,k) at k*pitch + r) and is transposed on
//         the way to shared memory.  ROWS/4 lanes cover all rows of one k (512 bytes for 128 rows);
//         a thread loads the same four rows at four consecutive k, transposes the 4x4 block in
//         registers (free) and stores four chunks, one per row.
//   VEC : 128-bit loads are legal (16-byte aligned rows, extent of the contiguous direction a
//         multiple of 4); otherwise the four elements are loaded and bounds-checked one by one.
// Loads are predicated, never branched around, so that all of a thread's loads are in flight together.
template <int ROWS, bool KC, bool VEC>
struct OperandLoader {
    static constexpr int LPR = ROWS / 4;                       // !KC: lanes per k-row
    static constexpr int G = 32 / LPR;                         // !KC: chunk columns per warp instruction
    static constexpr int ROUNDS = (kChunks + 4 * G - 1) / (4 * G);
    static constexpr int T = KC ? ROWS / 8 : 4 * ROUNDS;
    static constexpr uint32_t LBO = tile_lbo(ROWS, KC), SBO = tile_sbo(KC);
    const float* src;
    int64_t pitch;
    int row_base, rows, K, warp, lane;

    __device__ __forceinline__ void init(const float* src_, int64_t pitch_, int warp_, int lane_, int row_base_,
                                         int rows_, int K_) {
        src = src_; pitch = pitch_; warp = warp_; lane = lane_; row_base = row_base_; rows = rows_; K = K_;
    }
    // KC: tile-local row of chunk t (its 16-byte chunk column is lane & 15)
    __device__ __forceinline__ int krow(int t) const { return (t * 4 + warp) * 2 + (lane >> 4); }
    // !KC: chunk column of round u (rows are (lane % LPR) * 4 .. +3)
    __device__ __forceinline__ int tcol(int u) const { return (u * 4 + warp) * G + lane / LPR; }

    __device__ __forceinline__ void fetch(int kb, float4 (&r)[T]) const {
#pragma unroll
        for (int t = 0; t < T; ++t) {
            int row, k;
            bool tile_ok = true;
            if (KC) { row = row_base + krow(t); k = kb * kBlockK + (lane & 15) * 4; }
            else {
                const int c = tcol(t >> 2);
                tile_ok = c < kChunks;
                row = row_base + (lane % LPR) * 4; k = kb * kBlockK + c * 4 + (t & 3);
            }
            const float* q = KC ? src + (int64_t)row * pitch + k : src + (int64_t)k * pitch + row;
            if (VEC) {
                const bool in = tile_ok && (k < K) && (row < rows);
                r[t] = in ? __ldg(reinterpret_cast<const float4*>(q)) : make_float4(0.f, 0.f, 0.f, 0.f);
            } else if (KC) {
                const bool in = row < rows;
                r[t].x = (in && k < K) ? __ldg(q) : 0.f;
                r[t].y = (in && k + 1 < K) ? __ldg(q + 1) : 0.f;
                r[t].z = (in && k + 2 < K) ? __ldg(q + 2) : 0.f;
                r[t].w = (in && k + 3 < K) ? __ldg(q + 3) : 0.f;
            } else {
                const bool in = tile_ok && k < K;
                r[t].x = (in && row < rows) ? __ldg(q) : 0.f;
                r[t].y = (in && row + 1 < rows) ? __ldg(q + 1) : 0.f;
                r[t].z = (in && row + 2 < rows) ? __ldg(q + 2) : 0.f;
                r[t].w = (in && row + 3 < rows) ? __ldg(q + 3) : 0.f;
            }
        }
    }

    template <bool PRECISE>
    static __device__ __forceinline__ void put(unsigned char* hi, unsigned char* lo, uint32_t off, float4 v) {
        if (PRECISE) {
            float4 h, l;
            h.x = tf32_head(v.x); l.x = v.x - h.x;
            h.y = tf32_head(v.y); l.y = v.y - h.y;
            h.z = tf32_head(v.z); l.z = v.z - h.z;
            h.w = tf32_head(v.w); l.w = v.w - h.w;
            *reinterpret_cast<float4*>(hi + off) = h;
            *reinterpret_cast<float4*>(lo + off) = l;
        } else {
            *reinterpret_cast<float4*>(hi + off) = v;
        }
    }

    // Split each value into its TF32 head and the remainder and write both tiles (only the raw
    // value when !PRECISE).
    template <bool PRECISE>
    __device__ __forceinline__ void store(unsigned char* hi, unsigned char* lo, const float4 (&r)[T]) const {
        if (KC) {
#pragma unroll
            for (int t = 0; t < T; ++t)
                put<PRECISE>(hi, lo, (uint32_t)(lane & 15) * LBO + (uint32_t)krow(t) * 16, r[t]);
        } else {
            // rows rl .. rl+3 lie inside one 8-row group; lanes are 4 rows (64 + 8 pad bytes) apart
            const int rl = (lane % LPR) * 4;
            const uint32_t roff = (uint32_t)(rl >> 3) * SBO + (uint32_t)(rl & 7) * 16;
#pragma unroll
            for (int u = 0; u < ROUNDS; ++u) {
                const int c = tcol(u);
                if (c < kChunks) {
                    const float4 k0 = r[4 * u], k1 = r[4 * u + 1], k2 = r[4 * u + 2], k3 = r[4 * u + 3];
                    const uint32_t off = (uint32_t)c * LBO + roff;      // 4x4 transpose in registers
                    put<PRECISE>(hi, lo, off, make_float4(k0.x, k1.x, k2.x, k3.x));
                    put<PRECISE>(hi, lo, off + 16, make_float4(k0.y, k1.y, k2.y, k3.y));
                    put<PRECISE>(hi, lo, off + 32, make_float4(k0.z, k1.z, k2.z, k3.z));
                    put<PRECISE>(hi, lo, off + 48, make_float4(k0.w, k1.w, k2.w, k3.w));
                }
            }
        }
    }
};

// NT = column tile / 16 (B operand rows per CTA = 16 * NT <= 128); A_K / B_K: operand contiguous
// along k in memory; VEC: both operands allow 128-bit loads; PRECISE: three split MMAs per product.
// Grid: (ceil(M/128), ceil(N/(16 NT * n_per_cta)), nodes).
template <int NT, bool A_K, bool B_K, bool VEC, bool PRECISE>
__global__ void __launch_bounds__(kThreads, (PRECISE || NT > 4) ? 2 : 3)
tc_gemm_kernel(Args g) {
    constexpr int ROWS_A = kTileM, ROWS_B = 16 * NT;
    constexpr uint32_t A_BYTES = tile_bytes(ROWS_A, A_K), B_BYTES = tile_bytes(ROWS_B, B_K);
    constexpr uint32_t A_LBO = tile_lbo(ROWS_A, A_K), B_LBO = tile_lbo(ROWS_B, B_K);
    constexpr uint32_t A_SBO = tile_sbo(A_K), B_SBO = tile_sbo(B_K);
    constexpr uint32_t TMEM_COLS = ROWS_B <= 32 ? 32 : (ROWS_B <= 64 ? 64 : 128);
    extern __shared__ __align__(1024) unsigned char smem[];
    // stage: A hi | A lo | B hi | B lo   (the lo tiles only when PRECISE)
    constexpr uint32_t NCOPY = PRECISE ? 2 : 1;
    constexpr uint32_t STAGE = NCOPY * (A_BYTES + B_BYTES);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGE);      // one stage per CTA
    uint64_t* empty = full + 1;
    uint64_t* accum = empty + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int node = blockIdx.z;
    const int m0 = blockIdx.x * kTileM;
    const int tile0 = blockIdx.y * g.n_per_cta;
    const int n_tiles = min(g.n_per_cta, (g.N + ROWS_B - 1) / ROWS_B - tile0);
    const int KB = (g.K + kBlockK - 1) / kBlockK;

    if (tid == 0) {
        mbar_init(full, kLoaderThreads); mbar_init(empty, 1);
        mbar_init(accum, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        // ------------------------------ loaders ------------------------------
        using LoaderA = OperandLoader<ROWS_A, A_K, VEC>;
        using LoaderB = OperandLoader<ROWS_B, B_K, VEC>;
        LoaderA la;
        LoaderB lb;
        la.init(g.A + (int64_t)node * g.a_node, g.a_pitch, warp, lane, m0, g.M, g.K);
        // One k-block per thread in flight: the proxy fence below also waits for the thread's
        // outstanding global loads, so deeper register prefetch would not overlap anything.  Memory
        // parallelism comes from the CTAs that share the SM.
        float4 ra[LoaderA::T], rb[LoaderB::T];
        const int m = m0 + warp * 32 + lane;
        float* C = g.C + (int64_t)node * g.c_node;
        const float* aux = g.aux ? g.aux + (int64_t)node * g.aux_node : nullptr;
        const float bias = (g.epi <= EPI_BIAS && m < g.M) ? __ldg(aux + m) : 0.f;
        bool ok = true;
        uint32_t q = 0;                                     // k-blocks pushed so far (stage phase)
        lb.init(g.B + (int64_t)node * g.b_node, g.b_pitch, warp, lane, tile0 * ROWS_B, g.N, g.K);
        la.fetch(0, ra); lb.fetch(0, rb);
        for (int it = 0; it < n_tiles && ok; ++it) {
            const int n0 = (tile0 + it) * ROWS_B;
            const bool keep_a = (KB == 1 && it > 0);        // the A tile of the only k-block is already staged
            for (int kb = 0; kb < KB; ++kb, ++q) {
                if (!mbar_wait(empty, (q & 1u) ^ 1u)) { ok = false; break; }
                if (!keep_a) la.template store<PRECISE>(smem, smem + A_BYTES, ra);
                lb.template store<PRECISE>(smem + NCOPY * A_BYTES, smem + NCOPY * A_BYTES + B_BYTES, rb);
                tc_fence_before();                          // orders this thread's earlier tcgen05.ld (previous tile)
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(full);
                if (kb + 1 < KB) { la.fetch(kb + 1, ra); lb.fetch(kb + 1, rb); }
                else if (it + 1 < n_tiles) {                // first k-block of the next column tile
                    lb.row_base = n0 + ROWS_B;
                    if (KB > 1) la.fetch(0, ra);
                    lb.fetch(0, rb);
                }
            }
            // ------------------------------ epilogue of this column tile ------------------------------
            if (ok && !mbar_wait(accum, (uint32_t)it & 1u)) ok = false;
            ok = __all_sync(0xffffffffu, ok);               // tcgen05.ld below needs the whole warp
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < ROWS_B; c0 += 16) {
                float v[16];
                tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                const int nb = n0 + c0;
                const int cnt = m < g.M ? min(16, g.N - nb) : 0;      // columns of this group inside the matrix
                float* out = C + (int64_t)nb * g.c_pitch + m;
                if (g.epi == EPI_STORE) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) if (j < cnt) out[(int64_t)j * g.c_pitch] = v[j];
                } else if (g.epi == EPI_MASK) {
                    const float* mk = aux + (int64_t)nb * g.aux_pitch + m;
                    float gate[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) gate[j] = j < cnt ? __ldg(mk + (int64_t)j * g.aux_pitch) : 0.f;
#pragma unroll
                    for (int j = 0; j < 16; ++j) if (j < cnt) out[(int64_t)j * g.c_pitch] = gate[j] > 0.f ? v[j] : 0.f;
                } else {
                    const bool relu = g.epi == EPI_BIAS_RELU;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float x = v[j] + bias;
                        if (j < cnt) out[(int64_t)j * g.c_pitch] = (relu && x < 0.f) ? 0.f : x;
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    } else if (lane == 0) {
        // ------------------------------ MMA issuer ------------------------------
        // instruction descriptor: fp32 accumulate, TF32 x TF32, both operands K-major, N, M
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ROWS_B >> 3) << 17) |
                               ((uint32_t)(kTileM >> 4) << 24);
        bool ok = true;
        uint32_t q = 0;
        for (int it = 0; it < n_tiles && ok; ++it) {
            uint32_t acc = 0;                               // the first MMA of a column tile overwrites the accumulator
            for (int kb = 0; kb < KB; ++kb, ++q) {
                if (!mbar_wait(full, q & 1u)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_hi = smem_u32(smem), a_lo = a_hi + A_BYTES;
                const uint32_t b_hi = a_hi + NCOPY * A_BYTES, b_lo = b_hi + B_BYTES;
#pragma unroll
                for (int kk = 0; kk < kBlockK / 8; ++kk) {       // one MMA consumes k = 8 = two chunk columns
                    const uint64_t dah = smem_desc(a_hi + kk * 2 * A_LBO, A_LBO, A_SBO);
                    const uint64_t dbh = smem_desc(b_hi + kk * 2 * B_LBO, B_LBO, B_SBO);
                    if (PRECISE) {
                        const uint64_t dal = smem_desc(a_lo + kk * 2 * A_LBO, A_LBO, A_SBO);
                        const uint64_t dbl = smem_desc(b_lo + kk * 2 * B_LBO, B_LBO, B_SBO);
                        mma_tf32(tmem_base, dal, dbh, idesc, acc); acc = 1;
                        mma_tf32(tmem_base, dah, dbl, idesc, acc);
                    }
                    mma_tf32(tmem_base, dah, dbh, idesc, acc); acc = 1;
                }
                mma_commit(empty);      // frees the stage once these MMAs have read it
            }
            if (ok) mma_commit(accum);  // accumulator of this column tile complete
        }
        if (!ok) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int NT, bool A_K, bool B_K, bool PRECISE>
constexpr size_t smem_bytes() {
    return (size_t)(PRECISE ? 2 : 1) * (tile_bytes(kTileM, A_K) + tile_bytes(16 * NT, B_K)) + 3 * 8 + 16;
}

}  // namespace tc
}  // namespace dpsgd
