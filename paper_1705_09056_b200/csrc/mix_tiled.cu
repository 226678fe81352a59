// Gossip step for an arbitrary sparse W (Algorithm 1 steps 4-5):
//     X_next[i][c] = sum_{j in row i of W} W_ij X[j][c] - gamma G[i][c]
//
// Persistent CTAs walk over column tiles.  For each tile the full n x T slab of X is brought
// into shared memory by one TMA box load (cp.async.bulk.tensor) and the matching slab of G by
// per-thread 16-byte async copies, both signalling one mbarrier per stage, two tiles deep.  Every
// element of X and G therefore crosses HBM exactly once no matter how many neighbours re-use a
// row; the CSR gather reads shared memory only.  Tiles are kept small (about 16-32 KB per array)
// and two or more CTAs share an SM, so that one CTA's gather overlaps another's waiting: measured
// on B200 this beats wider tiles or deeper pipelines in a single CTA.  No cluster multicast is
// used: each CTA fetches its own tiles.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets the context's status word and
// the CTA leaves without touching the tile.
#include <cuda.h>

#include <algorithm>
#include <cstring>
#include <vector>

#include "ctx.h"
#include "tma_host.h"

namespace dpsgd {
namespace {

constexpr int kThreads = 512;
constexpr int kMaxRows = 256;                    // TMA box height limit
constexpr size_t kSmemPerSm = 227 * 1024;        // usable shared memory of one SM
constexpr size_t kSmemPerCtaReserve = 1024;      // driver-reserved bytes per resident CTA
constexpr uint32_t kWaitSpins = 1u << 22;        // x ~100 ns backoff each: well under a second

// One nonzero of W as the gather loop wants it: the byte offset of the neighbour's row inside a
// staged tile and the weight.
struct __align__(8) PackedNz {
    uint32_t row_bytes;   // col * T * sizeof(float)
    float w;
};

struct TiledState {
    CUtensorMap mapX[2];
    int T = 0;
    int stages = 0;
    int ctas_per_sm = 1;
    size_t smem = 0;
    int grid = 0;
    int csr_in_smem = 0;
    int x_tma = 1;
    int swapped = 0;
    int stats = 0;        // this launch also accumulates the consensus statistics
    int last_grid = 0;    // CTAs of the last launch (= partials written)
    int* d_status = nullptr;
    PackedNz* d_nz = nullptr;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the spin budget.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t spin = 0; spin < kWaitSpins; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (spin > 4096) __nanosleep(128);    // try_wait already blocks briefly; sleep only on long waits
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void cp_async_16(void* dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(src_bytes)
                 : "memory");
}
// Arrive on `bar` (without raising its pending count) once all of this thread's earlier cp.async landed.
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Shared memory: S x { X tile [n][T] | G tile [n][T] }, S mbarriers, two scratch buffers for the consensus
// statistics, then (when it fits) a copy of row_ptr and of the packed nonzeros so that the gather loop
// never leaves the SM.
// X arrives by TMA (one box per tile) or, with X_TMA = false, by per-thread 16-byte async copies
// like G always does; each stage's mbarrier counts the TMA transaction plus one arrival per thread.
// SWAPPED (footnote c of Algorithm 1): X_next[i] = sum_j W_ij (X[j] - gamma G[j]); every neighbour's term
// is formed on the fly from the two staged tiles (no rewrite of the X tile, no extra barrier).
// STATS (Theorem 4, Eq. 10): also accumulates sum_i ||xbar - x_i||^2 of the NEW rows while they are in
// registers.  Per column the new values are shifted by the staged old X[0][c] (any common shift cancels),
// d_i = x'_i - X[0][c]; the rows of a column sit in different threads, so per-thread sums of d and d^2 are
// combined by shuffles inside a warp and through shared memory across warps (in a fixed order), the
// column's sum d^2 - (sum d)^2 / n is formed in fp64, and every CTA leaves one fp64 partial.
constexpr int kWarps = kThreads / 32;
__host__ __device__ constexpr size_t stats_scratch_bytes(int T) { return (size_t)2 * 2 * kWarps * T * sizeof(float); }

template <int T, int S, bool X_TMA, bool SWAPPED, bool STATS>
__global__ void __launch_bounds__(kThreads)
mix_tiled_kernel(const __grid_constant__ CUtensorMap mapX, const float4* __restrict__ X,
                 const float4* __restrict__ G, float4* __restrict__ Xn, const int32_t* row_ptr,
                 const PackedNz* nz, int n, int64_t ld4, int64_t tiles, float ngamma, int csr_in_smem,
                 int* __restrict__ status, double* __restrict__ partials) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr int kGroups = T / 4;                 // float4 column groups per tile
    constexpr int kRowStep = kThreads / kGroups;   // rows processed concurrently by the CTA
    constexpr int kGW = kGroups < 32 ? kGroups : 32;   // column groups one warp covers
    const uint32_t tile_bytes = (uint32_t)n * T * sizeof(float);
    const uint32_t stage_bytes = 2 * tile_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + (size_t)S * stage_bytes);
    // statistics scratch: [2 buffers][sum d | sum d^2][warp][column group of the warp] float4
    float4* scratch = reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(full) + 16 * ((S * 8 + 15) / 16));

    const int tid = threadIdx.x;
    if (csr_in_smem) {
        const int nnz = __ldg(row_ptr + n);
        PackedNz* s_nz = reinterpret_cast<PackedNz*>(reinterpret_cast<unsigned char*>(scratch) + stats_scratch_bytes(T));
        int32_t* s_rp = reinterpret_cast<int32_t*>(s_nz + nnz);
        for (int t = tid; t <= n; t += kThreads) s_rp[t] = __ldg(row_ptr + t);
        for (int t = tid; t < nnz; t += kThreads) s_nz[t] = nz[t];
        row_ptr = s_rp; nz = s_nz;
    }
    if (tid == 0) {
        for (int s = 0; s < S; ++s) mbar_init(full + s, kThreads + (X_TMA ? 1 : 0));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int64_t first = blockIdx.x;
    const int64_t step = gridDim.x;
    const int64_t my_tiles = first < tiles ? (tiles - first + step - 1) / step : 0;
    const int cg = tid % kGroups;
    const int r0 = tid / kGroups;
    double col_acc = 0.0;                          // STATS: threads tid < T, one column of the tile each

    // every thread takes part: rows r0, r0 + kRowStep, ... of its own column group
    auto issue = [&](int64_t it, int s) {
        unsigned char* xs = smem_raw + (size_t)s * stage_bytes;
        const int64_t tile = first + it * step;
        if (X_TMA && tid == 0) {
            mbar_expect_tx(full + s, tile_bytes);
            tma_load_2d(xs, &mapX, (int)(tile * T), 0, full + s);
        }
        const int64_t c4 = tile * kGroups + cg;
        const bool inside = c4 < ld4;
        const int64_t c4s = inside ? c4 : 0;
        const uint32_t nbytes = inside ? 16u : 0u;          // out-of-range columns are zero-filled
        for (int i = r0; i < n; i += kRowStep) {
            const uint32_t off = ((uint32_t)i * kGroups + cg) * 16u;
            if (!X_TMA) cp_async_16(xs + off, X + (int64_t)i * ld4 + c4s, nbytes);
            cp_async_16(xs + tile_bytes + off, G + (int64_t)i * ld4 + c4s, nbytes);
        }
        cp_async_arrive(full + s);
    };
    for (int it = 0; it < my_tiles && it < S; ++it) issue(it, it);

    int s = 0;
    uint32_t parity = 0;
    for (int64_t it = 0; it < my_tiles; ++it) {
        if (!mbar_wait(full + s, parity)) {
            if (tid == 0) atomicExch(status, (int)DPSGD_ERR_TIMEOUT);
            // give copies already in flight a bounded chance to land before the CTA exits
            for (int j = 1; j < S; ++j) {
                const int sj = (s + j) % S;
                if (it + j < my_tiles) mbar_wait(full + sj, sj > s ? parity : parity ^ 1u);
            }
            // the result is void (the status word says so); leave a defined partial and go, as threads that
            // have exited do not hold up the CTA's barriers
            if (STATS) partials[blockIdx.x] = 0.0;
            return;
        }
        unsigned char* xs = smem_raw + (size_t)s * stage_bytes + cg * 16;   // this thread's column group
        const unsigned char* gs = xs + tile_bytes;
        const int64_t c4 = (first + it * step) * kGroups + cg;
        float4 s1 = make_float4(0.f, 0.f, 0.f, 0.f), s2 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c4 < ld4) {
            float4* out = Xn + c4;
            const float4 sh = STATS ? *reinterpret_cast<const float4*>(xs) : make_float4(0.f, 0.f, 0.f, 0.f);
            for (int i = r0; i < n; i += kRowStep) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                const int pe = row_ptr[i + 1];
                for (int p = row_ptr[i]; p < pe; ++p) {
                    const PackedNz e = nz[p];
                    float4 v = *reinterpret_cast<const float4*>(xs + e.row_bytes);
                    if (SWAPPED) {
                        const float4 g = *reinterpret_cast<const float4*>(gs + e.row_bytes);
                        v.x = fmaf(ngamma, g.x, v.x); v.y = fmaf(ngamma, g.y, v.y);
                        v.z = fmaf(ngamma, g.z, v.z); v.w = fmaf(ngamma, g.w, v.w);
                    }
                    a.x = fmaf(e.w, v.x, a.x); a.y = fmaf(e.w, v.y, a.y);
                    a.z = fmaf(e.w, v.z, a.z); a.w = fmaf(e.w, v.w, a.w);
                }
                if (!SWAPPED) {
                    const float4 g = *reinterpret_cast<const float4*>(gs + (uint32_t)i * (T * 4u));
                    a.x = fmaf(ngamma, g.x, a.x); a.y = fmaf(ngamma, g.y, a.y);
                    a.z = fmaf(ngamma, g.z, a.z); a.w = fmaf(ngamma, g.w, a.w);
                }
                __stcs(out + (int64_t)i * ld4, a);
                if (STATS) {
                    const float dx = a.x - sh.x, dy = a.y - sh.y, dz = a.z - sh.z, dw = a.w - sh.w;
                    s1.x += dx; s1.y += dy; s1.z += dz; s1.w += dw;
                    s2.x = fmaf(dx, dx, s2.x); s2.y = fmaf(dy, dy, s2.y);
                    s2.z = fmaf(dz, dz, s2.z); s2.w = fmaf(dw, dw, s2.w);
                }
            }
        }
        float4* sc = scratch + (size_t)(it & 1) * (2 * kWarps * kGW);
        if (STATS) {
            // lanes of a warp that share a column group (kGroups < 32: rows r0 differ), then one entry per warp
#pragma unroll
            for (int o = kGW; o < 32; o <<= 1) {
                s1.x += __shfl_xor_sync(0xffffffffu, s1.x, o); s1.y += __shfl_xor_sync(0xffffffffu, s1.y, o);
                s1.z += __shfl_xor_sync(0xffffffffu, s1.z, o); s1.w += __shfl_xor_sync(0xffffffffu, s1.w, o);
                s2.x += __shfl_xor_sync(0xffffffffu, s2.x, o); s2.y += __shfl_xor_sync(0xffffffffu, s2.y, o);
                s2.z += __shfl_xor_sync(0xffffffffu, s2.z, o); s2.w += __shfl_xor_sync(0xffffffffu, s2.w, o);
            }
            const int lane = tid & 31, warp = tid >> 5;
            if (lane < kGW) {
                sc[warp * kGW + lane] = s1;
                sc[(kWarps + warp) * kGW + lane] = s2;
            }
        }
        __syncthreads();                       // everyone is done reading stage s (and has left its statistics)
        if (it + S < my_tiles) issue(it + S, s);
        if (STATS && tid < T) {
            // column tid of the tile: its group is covered by the warps w with (w * 32 / kGroups ...) - for
            // kGroups >= 32 a warp covers groups [32 (w % (kGroups / 32)), +32); otherwise every warp covers all
            const int grp = tid >> 2, comp = tid & 3;
            double a1 = 0.0, a2 = 0.0;
            for (int w = 0; w < kWarps; ++w) {
                if (kGroups > 32 && (w % (kGroups / 32)) != grp / 32) continue;
                const float* e1 = reinterpret_cast<const float*>(sc + w * kGW + (grp % kGW));
                const float* e2 = reinterpret_cast<const float*>(sc + (kWarps + w) * kGW + (grp % kGW));
                a1 += (double)e1[comp];
                a2 += (double)e2[comp];
            }
            col_acc += a2 - a1 * a1 / (double)n;
        }
        if (++s == S) { s = 0; parity ^= 1u; }
    }
    if (STATS) {
        // one fp64 partial per CTA, added in thread order
        double* red = reinterpret_cast<double*>(scratch);
        __syncthreads();
        if (tid < T) red[tid] = col_acc;
        __syncthreads();
        if (tid == 0) {
            double r = 0.0;
            for (int t = 0; t < T; ++t) r += red[t];
            partials[blockIdx.x] = r;
        }
    }
}

// The give-up path of the bounded waits, on its own: one mbarrier that expects an arrival nobody makes.
// After max_polls unsuccessful polls the CTA raises the status word, exactly as mix_tiled_kernel does, and
// returns; it holds nothing else (no copy in flight, no tensor memory).
__global__ void wait_probe_kernel(uint32_t max_polls, int* __restrict__ status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool done = false;
    for (uint32_t spin = 0; spin < max_polls && !done; ++spin) done = mbar_try_wait(&bar, 0);
    if (!done && threadIdx.x == 0) atomicExch(status, (int)DPSGD_ERR_TIMEOUT);
}

bool make_map(CUtensorMap* map, const float* base, int n, int64_t ld, int T) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)ld, (cuuint64_t)n};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)T, (cuuint32_t)n};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t smem_need(int n, int nnz, int T, int S, bool with_csr) {
    size_t b = (size_t)S * 2 * n * T * sizeof(float) + 16 * ((S * sizeof(uint64_t) + 15) / 16) + stats_scratch_bytes(T);
    if (with_csr) b += sizeof(PackedNz) * (size_t)nnz + sizeof(int32_t) * (n + 1);
    return b;
}

// Two stages; 64-column tiles (256-byte row segments; 128 columns for n <= 32, 32 only when
// nothing wider fits); as many CTAs per SM as keep about 128 KB staged per SM (at most 4).
bool pick_shape(int n, int nnz, int* T_out, int* S_out, int* ctas_out) {
    const int prefer[3] = {n <= 32 ? 128 : 64, n <= 32 ? 64 : 32, 32};
    for (int T : prefer) {
        const size_t need = smem_need(n, nnz, T, 2, false);
        if (need + kSmemPerCtaReserve > kSmemPerSm) continue;
        *T_out = T; *S_out = 2;
        const size_t per = smem_need(n, nnz, T, 2, true) + kSmemPerCtaReserve;
        const size_t fit = std::max<size_t>(1, kSmemPerSm / per);
        const size_t want = std::max<size_t>(1, (128 * 1024 + need / 2) / need);
        *ctas_out = (int)std::min<size_t>(std::min<size_t>(fit, want), 2048 / kThreads);
        return true;
    }
    return false;
}

template <int T, int S, bool X_TMA, bool SWAPPED, bool STATS>
cudaError_t launch_tsx(dpsgd_ctx* c, TiledState* st, int which, const float* G, float* Xn) {
    // per device and cheap: set on every launch rather than remembered in a process-wide flag
    cudaError_t ea = cudaFuncSetAttribute(mix_tiled_kernel<T, S, X_TMA, SWAPPED, STATS>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)(kSmemPerSm - kSmemPerCtaReserve));
    if (ea != cudaSuccess) return ea;
    const int64_t ld4 = c->ld / 4;
    const int64_t tiles = (c->ld + T - 1) / T;
    const int grid = (int)std::min<int64_t>(tiles, st->grid);
    mix_tiled_kernel<T, S, X_TMA, SWAPPED, STATS><<<grid, kThreads, st->smem, c->stream>>>(
        st->mapX[which], reinterpret_cast<const float4*>(c->X[which]), reinterpret_cast<const float4*>(G),
        reinterpret_cast<float4*>(Xn), c->W.row_ptr, st->d_nz, c->n, ld4, tiles, -c->gamma, st->csr_in_smem,
        st->d_status, c->d_partials);
    st->last_grid = grid;
    return cudaGetLastError();
}

template <int T, int S>
cudaError_t launch_ts(dpsgd_ctx* c, TiledState* st, int which, const float* G, float* Xn) {
#define DPSGD_TILED_PICK(XT, SW) \
    (st->stats ? launch_tsx<T, S, XT, SW, true>(c, st, which, G, Xn) : launch_tsx<T, S, XT, SW, false>(c, st, which, G, Xn))
    if (st->swapped) return st->x_tma ? DPSGD_TILED_PICK(true, true) : DPSGD_TILED_PICK(false, true);
    return st->x_tma ? DPSGD_TILED_PICK(true, false) : DPSGD_TILED_PICK(false, false);
#undef DPSGD_TILED_PICK
}

template <int T>
cudaError_t launch_t(dpsgd_ctx* c, TiledState* st, int which, const float* G, float* Xn) {
    switch (st->stages) {
        case 2: return launch_ts<T, 2>(c, st, which, G, Xn);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool mix_tiled_supported(const dpsgd_ctx* c) {
    int T, S, ctas;
    return c->n <= kMaxRows && pick_shape(c->n, c->W.nnz, &T, &S, &ctas);
}

void mix_tiled_release(dpsgd_ctx* c) {
    if (!c->tma_state) return;
    TiledState* st = static_cast<TiledState*>(c->tma_state);
    cudaFree(st->d_nz);
    delete st;
    c->tma_state = nullptr;
}

cudaError_t launch_wait_probe(dpsgd_ctx* c, uint32_t max_polls) {
    wait_probe_kernel<<<1, 32, 0, c->stream>>>(max_polls, &c->d_result->status);
    c->launches++;
    return cudaGetLastError();
}

// stats_out != NULL: the kernel also accumulates the consensus distance of X_next, and a fixed-order
// reduction of the per-CTA partials leaves it in *stats_out (device).
cudaError_t launch_mix_tiled(dpsgd_ctx* c, const float* X, const float* G, float* Xn, double* stats_out) {
    TiledState* st = static_cast<TiledState*>(c->tma_state);
    if (!st) {
        st = new TiledState();
        if (!pick_shape(c->n, c->W.nnz, &st->T, &st->stages, &st->ctas_per_sm)) { delete st; return cudaErrorInvalidValue; }
        st->smem = smem_need(c->n, c->W.nnz, st->T, st->stages, false);
        const size_t with_csr = smem_need(c->n, c->W.nnz, st->T, st->stages, true);
        if ((with_csr + kSmemPerCtaReserve) * st->ctas_per_sm <= kSmemPerSm) { st->smem = with_csr; st->csr_in_smem = 1; }
        std::vector<PackedNz> packed(c->W.nnz);
        for (int p = 0; p < c->W.nnz; ++p) {
            packed[p].row_bytes = (uint32_t)c->h_col[p] * (uint32_t)st->T * (uint32_t)sizeof(float);
            packed[p].w = c->h_val[p];
        }
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
        if (e != cudaSuccess) { delete st; return e; }
        st->grid = sms * st->ctas_per_sm;
        st->d_status = &c->d_result->status;
        if (c->ld >= (int64_t(1) << 31)) {
            st->x_tma = 0;                      // TMA coordinates are 32-bit: X goes the way G does
            memset(st->mapX, 0, sizeof(st->mapX));
        } else if (!make_map(&st->mapX[0], c->X[0], c->n, c->ld, st->T) ||
                   !make_map(&st->mapX[1], c->X[1], c->n, c->ld, st->T)) {
            delete st;
            return cudaErrorInvalidValue;
        }
        e = cudaMalloc(&st->d_nz, sizeof(PackedNz) * std::max<size_t>(1, packed.size()));
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(st->d_nz, packed.data(), sizeof(PackedNz) * packed.size(), cudaMemcpyHostToDevice,
                                c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // packed[] is a local
        if (e != cudaSuccess) { cudaFree(st->d_nz); delete st; return e; }
        c->tma_state = st;
    }
    const int which = (X == c->X[0]) ? 0 : 1;
    st->swapped = c->swapped ? 1 : 0;
    st->stats = stats_out ? 1 : 0;
    cudaError_t e;
    if (stats_out && (e = ensure_partials(c, st->grid)) != cudaSuccess) return e;
    switch (st->T) {
        case 128: e = launch_t<128>(c, st, which, G, Xn); break;
        case 64: e = launch_t<64>(c, st, which, G, Xn); break;
        default: e = launch_t<32>(c, st, which, G, Xn); break;
    }
    c->launches++;
    if (e == cudaSuccess && stats_out) e = launch_consensus_final(c, st->last_grid, stats_out);
    return e;
}

}  // namespace dpsgd
