// Batched skinny GEMM on the 5th-generation tensor cores for the MLP gradients (Algorithm 1 step 3).
//
//     C[n][m] = epilogue( sum_k A(m,k) * B(n,k) )         one problem per node (blockIdx.z)
//
// The long (weight) dimension m sits on the 128 TMEM lanes, the short one (batch, or a 16..128 wide
// slice) on the TMEM columns.  tcgen05.mma kind::tf32 multiplies 10-bit-mantissa operands, so an
// fp32-faithful product is built from three MMAs on split operands (a = a_hi + a_lo):
//     a*b ~= a_hi*b_hi + a_lo*b_hi + a_hi*b_lo        (fp32 accumulation in TMEM)
// The operands are fp32 in HBM.  Four loader warps read them with 128-bit loads (64-byte segments
// per row), split them in registers and write hi / lo copies to shared memory directly in the
// no-swizzle K-major canonical layout the MMA descriptors describe (core matrix = 8 rows x 16 B,
// element (r,k) at (k/4)*LBO + r*16 + (k%4)*4).  An operand that is contiguous along m / n in
// memory is transposed on the way: each lane scatters the four elements of its 128-bit load to
// four rows, rotated per lane so that a warp's 32 stores hit 32 different banks.  (tcgen05 has
// no no-swizzle MN-major mode for 32-bit operands.)  One thread of a fifth warp
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
constexpr int kBlockK = 32;            // fp32 elements per pipeline stage along k (4 MMAs of K = 8)
constexpr int kStages = 1;            // one stage per CTA: four CTAs share an SM and overlap each other
constexpr uint32_t kWaitSpins = 1u << 21;

enum { EPI_BIAS_RELU = 0, EPI_BIAS = 1, EPI_STORE = 2, EPI_MASK = 3 };

struct Args {
    const float* A; int64_t a_node; int64_t a_pitch; int a_kcontig; int a_vec;   // A(m,k)
    const float* B; int64_t b_node; int64_t b_pitch; int b_kcontig; int b_vec;   // B(n,k)
    float* C; int64_t c_node; int64_t c_pitch;                                   // C[n*c_pitch + m]
    const float* aux; int64_t aux_node; int64_t aux_pitch;                       // bias[m] or mask[n*aux_pitch + m]
    int M, N, K;
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
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    // try_wait itself blocks for a short hardware-defined slice, so plain polling is cheap; back
    // off with nanosleep (coarse: it can cost a microsecond) only once the wait is clearly long
    for (uint32_t spin = 0; spin < kWaitSpins; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (spin > 4096) __nanosleep(128);
    }
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

__device__ __forceinline__ float pick(float4 v, int e) {
    return e == 0 ? v.x : (e == 1 ? v.y : (e == 2 ? v.z : v.w));
}

// One loader thread's share of an operand tile (ROWS x 32 k): ROWS/16 chunks of 16 bytes, i.e.
// four consecutive elements along the operand's contiguous direction.
//   KC  : the operand is contiguous along k in memory (element (r,k) at r*pitch + k)
//   !KC : it is contiguous along its row index (element (r,k) at k*pitch + r) and is transposed
//         on the way to shared memory
//   VEC : 128-bit loads are legal (16-byte aligned rows, extent of the contiguous direction a
//         multiple of 4); otherwise the four elements are loaded and bounds-checked one by one.
// Lane mapping: 8 lanes along the slow direction x 4 lanes along the contiguous one, so a warp
// reads 8 segments of 64 bytes; successive chunks of a thread are 16 rows apart.  Loads are
// predicated, never branched around, so that all of a thread's loads are in flight together.
template <int ROWS, bool KC, bool VEC>
struct OperandLoader {
    static constexpr int T = ROWS / 16;
    const float* ptr0;
    int64_t tstride, kstride;
    int row0, kfix, rows, K;
    uint32_t soff0;      // shared-memory byte offset of chunk 0 inside the hi (or lo) tile
    int rot;

    __device__ __forceinline__ void init(const float* src, int64_t pitch, int warp, int lane, int row_base,
                                         int rows_, int K_) {
        rows = rows_; K = K_;
        if (KC) {
            const int rl = (warp >> 1) * 8 + (lane & 7);
            kfix = ((warp & 1) * 4 + (lane >> 3)) * 4;
            row0 = row_base + rl;
            ptr0 = src + (int64_t)row0 * pitch + kfix;
            tstride = 16 * pitch; kstride = kBlockK;
            soff0 = (uint32_t)(kfix >> 2) * (ROWS * 16) + (uint32_t)rl * 16;
            rot = 0;
        } else {
            const int rl = (lane >> 3) * 4;
            kfix = warp * 8 + (lane & 7);
            row0 = row_base + rl;
            ptr0 = src + (int64_t)kfix * pitch + row0;
            tstride = 16; kstride = (int64_t)kBlockK * pitch;
            soff0 = (uint32_t)(kfix >> 2) * (ROWS * 16) + (uint32_t)rl * 16 + (uint32_t)(kfix & 3) * 4;
            rot = ((lane >> 2) & 1) + 2 * (lane >> 4);
        }
    }

    __device__ __forceinline__ void fetch(int kb, float4 (&r)[T]) const {
        const int k = kb * kBlockK + kfix;
        const float* p = ptr0 + (int64_t)kb * kstride;
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const int row = row0 + 16 * t;
            const float* q = p + (int64_t)t * tstride;
            if (VEC) {
                const bool in = (k < K) && (row < rows);
                r[t] = in ? __ldg(reinterpret_cast<const float4*>(q)) : make_float4(0.f, 0.f, 0.f, 0.f);
            } else if (KC) {
                const bool in = row < rows;
                r[t].x = (in && k < K) ? __ldg(q) : 0.f;
                r[t].y = (in && k + 1 < K) ? __ldg(q + 1) : 0.f;
                r[t].z = (in && k + 2 < K) ? __ldg(q + 2) : 0.f;
                r[t].w = (in && k + 3 < K) ? __ldg(q + 3) : 0.f;
            } else {
                const bool in = k < K;
                r[t].x = (in && row < rows) ? __ldg(q) : 0.f;
                r[t].y = (in && row + 1 < rows) ? __ldg(q + 1) : 0.f;
                r[t].z = (in && row + 2 < rows) ? __ldg(q + 2) : 0.f;
                r[t].w = (in && row + 3 < rows) ? __ldg(q + 3) : 0.f;
            }
        }
    }

    // Split each value into its TF32 head and the remainder and write both tiles (only the raw
    // value when precise == 0).  K-major canonical layout: (r,k) at (k/4)*ROWS*16 + r*16 + (k%4)*4.
    __device__ __forceinline__ void store(unsigned char* hi, unsigned char* lo, const float4 (&r)[T], int precise) const {
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const uint32_t off = soff0 + (uint32_t)t * 256;       // 16 rows further
            const float4 v = r[t];
            if (KC) {
                if (precise) {
                    float4 h, l;
                    h.x = __uint_as_float(__float_as_uint(v.x) & 0xFFFFE000u); l.x = v.x - h.x;
                    h.y = __uint_as_float(__float_as_uint(v.y) & 0xFFFFE000u); l.y = v.y - h.y;
                    h.z = __uint_as_float(__float_as_uint(v.z) & 0xFFFFE000u); l.z = v.z - h.z;
                    h.w = __uint_as_float(__float_as_uint(v.w) & 0xFFFFE000u); l.w = v.w - h.w;
                    *reinterpret_cast<float4*>(hi + off) = h;
                    *reinterpret_cast<float4*>(lo + off) = l;
                } else {
                    *reinterpret_cast<float4*>(hi + off) = v;
                }
            } else {
                // the four elements go to four rows; the order is rotated per lane so that the 32
                // scalar stores of a warp fall into 32 different banks
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int e = (j + rot) & 3;
                    const float x = pick(v, e);
                    const uint32_t o = off + (uint32_t)e * 16;
                    if (precise) {
                        const float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
                        *reinterpret_cast<float*>(hi + o) = h;
                        *reinterpret_cast<float*>(lo + o) = x - h;
                    } else {
                        *reinterpret_cast<float*>(hi + o) = x;
                    }
                }
            }
        }
    }
};

// NT = column tile / 16 (B operand rows per CTA = 16 * NT <= 128); A_K / B_K: operand contiguous
// along k in memory; VEC: both operands allow 128-bit loads.
// Grid: (ceil(M/128), ceil(N/(16 NT)), nodes).
template <int NT, bool A_K, bool B_K, bool VEC>
__global__ void __launch_bounds__(kThreads, NT <= 4 ? 4 : 2)
tc_gemm_kernel(Args g) {
    constexpr int ROWS_A = kTileM, ROWS_B = 16 * NT;
    constexpr uint32_t A_BYTES = ROWS_A * kBlockK * 4, B_BYTES = ROWS_B * kBlockK * 4;
    constexpr int TA = ROWS_A / 16, TB = ROWS_B / 16;          // 16-byte chunks per loader thread
    constexpr uint32_t TMEM_COLS = ROWS_B <= 32 ? 32 : (ROWS_B <= 64 ? 64 : 128);
    extern __shared__ __align__(1024) unsigned char smem[];
    // per stage: A hi | A lo | B hi | B lo
    constexpr uint32_t STAGE = 2 * A_BYTES + 2 * B_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * STAGE);
    uint64_t* empty = full + kStages;
    uint64_t* accum = empty + kStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int node = blockIdx.z;
    const int m0 = blockIdx.x * kTileM, n0 = blockIdx.y * ROWS_B;
    const int KB = (g.K + kBlockK - 1) / kBlockK;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full + s, kLoaderThreads); mbar_init(empty + s, 1); }
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
        OperandLoader<ROWS_A, A_K, VEC> la;
        OperandLoader<ROWS_B, B_K, VEC> lb;
        la.init(g.A + (int64_t)node * g.a_node, g.a_pitch, warp, lane, m0, g.M, g.K);
        lb.init(g.B + (int64_t)node * g.b_node, g.b_pitch, warp, lane, n0, g.N, g.K);
        // One k-block per thread in flight: the proxy fence below also waits for the thread's
        // outstanding global loads, so deeper register prefetch would not overlap anything.  Memory
        // parallelism comes from the CTAs that share the SM.
        float4 ra[TA], rb[TB];
        bool ok = true;
        la.fetch(0, ra); lb.fetch(0, rb);
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % kStages;
            const uint32_t fill = (uint32_t)(kb / kStages);
            if (!mbar_wait(empty + s, (fill & 1u) ^ 1u)) { ok = false; break; }
            unsigned char* base = smem + s * STAGE;
            la.store(base, base + A_BYTES, ra, g.precise);
            lb.store(base + 2 * A_BYTES, base + 2 * A_BYTES + B_BYTES, rb, g.precise);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(full + s);
            if (kb + 1 < KB) { la.fetch(kb + 1, ra); lb.fetch(kb + 1, rb); }
        }
        // ------------------------------ epilogue ------------------------------
        if (ok && !mbar_wait(accum, 0)) ok = false;
        ok = __all_sync(0xffffffffu, ok);      // tcgen05.ld below needs the whole warp
        if (!ok) {
            if (lane == 0) atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
        } else {
            tc_fence_after();
            const int m = m0 + warp * 32 + lane;
            float* C = g.C + (int64_t)node * g.c_node;
            const float* aux = g.aux ? g.aux + (int64_t)node * g.aux_node : nullptr;
            const float bias = (g.epi <= EPI_BIAS && m < g.M) ? __ldg(aux + m) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < ROWS_B; c0 += 16) {
                float v[16];
                tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                if (m < g.M) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = n0 + c0 + j;
                        if (n < g.N) {
                            float x = v[j];
                            if (g.epi == EPI_BIAS_RELU) { x += bias; x = x > 0.f ? x : 0.f; }
                            else if (g.epi == EPI_BIAS) x += bias;
                            else if (g.epi == EPI_MASK) x = __ldg(aux + (int64_t)n * g.aux_pitch + m) > 0.f ? x : 0.f;
                            C[(int64_t)n * g.c_pitch + m] = x;
                        }
                    }
                }
            }
        }
    } else if (lane == 0) {
        // ------------------------------ MMA issuer ------------------------------
        // instruction descriptor: fp32 accumulate, TF32 x TF32, both operands K-major, N, M
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ROWS_B >> 3) << 17) |
                               ((uint32_t)(kTileM >> 4) << 24);
        const uint32_t a_lbo = ROWS_A * 16, b_lbo = ROWS_B * 16;      // next 4 k: one 16-byte chunk column further
        const uint32_t a_step = 2 * a_lbo, b_step = 2 * b_lbo;        // one MMA consumes k = 8 = two chunks
        bool ok = true;
        uint32_t acc = 0;
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % kStages;
            const uint32_t fill = (uint32_t)(kb / kStages);
            if (!mbar_wait(full + s, fill & 1u)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_hi = smem_u32(smem + s * STAGE), a_lo = a_hi + A_BYTES;
            const uint32_t b_hi = a_hi + 2 * A_BYTES, b_lo = b_hi + B_BYTES;
#pragma unroll
            for (int kk = 0; kk < kBlockK / 8; ++kk) {
                const uint64_t dah = smem_desc(a_hi + kk * a_step, a_lbo, 128), dbh = smem_desc(b_hi + kk * b_step, b_lbo, 128);
                if (g.precise) {
                    const uint64_t dal = smem_desc(a_lo + kk * a_step, a_lbo, 128), dbl = smem_desc(b_lo + kk * b_step, b_lbo, 128);
                    mma_tf32(tmem_base, dal, dbh, idesc, acc); acc = 1;
                    mma_tf32(tmem_base, dah, dbl, idesc, acc);
                }
                mma_tf32(tmem_base, dah, dbh, idesc, acc); acc = 1;
            }
            mma_commit(empty + s);      // frees the stage once these MMAs have read it
        }
        if (ok) mma_commit(accum);      // accumulator complete
        else atomicExch(g.status, (int)DPSGD_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int NT>
constexpr size_t smem_bytes() {
    return (size_t)kStages * (2 * kTileM * kBlockK * 4 + 2 * 16 * NT * kBlockK * 4) + (2 * kStages + 1) * 8 + 16;
}

}  // namespace tc
}  // namespace dpsgd
