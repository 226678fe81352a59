// Backward products of a NARROW MLP layer (at most 16 output units: the classifier layer), Algorithm 1
// step 3.  A 128-row tensor-core tile would be 90 % padding there and the two tensor-core launches it
// replaces are bound by latency, so this runs on the fp32 pipes with exact FMA products and fixed
// summation orders, one pass over h for both results:
//
//     gW[o][k']    = sum_b delta[b][o] h[b][k']
//     dprev[b][k'] = [h[b][k'] > 0] sum_o delta[b][o] W[o][k']
//
// A thread owns one k' (or four); the node's delta sits in shared memory, zero-padded to 16 output
// units so that the inner loops carry no branch and the loads of h stay in flight together.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dpsgd {
namespace narrow {

constexpr int kMaxOut = 16;
constexpr int kBwdThreads = 128;

// grid (ceil(din / (128 VEC)), nodes), block 128, dynamic shared memory B * 16 floats (the node's
// delta).  dprev == nullptr: first layer, no error to pass on.
template <int VEC>
__global__ void __launch_bounds__(kBwdThreads)
narrow_backward_kernel(const float* __restrict__ X, float* __restrict__ G, int64_t ld, int64_t w_off,
                       const float* __restrict__ h, const float* __restrict__ delta, int dpitch,
                       float* __restrict__ dprev, int B, int din, int dout) {
    extern __shared__ float ds[];                 // [B][16], zero beyond dout: the loops below need no branch
    const int node = blockIdx.y;
    const float* dn = delta + (int64_t)node * B * dpitch;
    for (int i = threadIdx.x; i < B * kMaxOut; i += kBwdThreads) {
        const int b = i / kMaxOut, o = i % kMaxOut;
        ds[i] = o < dout ? __ldg(dn + (int64_t)b * dpitch + o) : 0.f;
    }
    __syncthreads();
    const int k0 = (blockIdx.x * kBwdThreads + threadIdx.x) * VEC;
    if (k0 >= din) return;
    const float* W = X + (int64_t)node * ld + w_off + k0;
    float* gW = G + (int64_t)node * ld + w_off + k0;
    const float* hn = h + (int64_t)node * B * din + k0;
    float* dp = dprev ? dprev + (int64_t)node * B * din + k0 : nullptr;
    float w[kMaxOut][VEC], acc[kMaxOut][VEC];
#pragma unroll
    for (int o = 0; o < kMaxOut; ++o)
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            acc[o][v] = 0.f;
            w[o][v] = (dprev && o < dout) ? __ldg(W + (int64_t)o * din + v) : 0.f;     // a zero row meets a zero delta
        }
#pragma unroll 8
    for (int b = 0; b < B; ++b) {
        float hv[VEC], s[VEC];
        if (VEC == 4) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(hn + (int64_t)b * din));
            hv[0] = t.x; hv[1 % VEC] = t.y; hv[2 % VEC] = t.z; hv[3 % VEC] = t.w;
        } else {
            hv[0] = __ldg(hn + (int64_t)b * din);
        }
#pragma unroll
        for (int v = 0; v < VEC; ++v) s[v] = 0.f;
#pragma unroll
        for (int o = 0; o < kMaxOut; ++o) {
            const float d = ds[b * kMaxOut + o];
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                acc[o][v] = fmaf(d, hv[v], acc[o][v]);
                s[v] = fmaf(d, w[o][v], s[v]);
            }
        }
        if (dp) {
            if (VEC == 4) {
                *reinterpret_cast<float4*>(dp + (int64_t)b * din) =
                    make_float4(hv[0] > 0.f ? s[0] : 0.f, hv[1 % VEC] > 0.f ? s[1 % VEC] : 0.f,
                                hv[2 % VEC] > 0.f ? s[2 % VEC] : 0.f, hv[3 % VEC] > 0.f ? s[3 % VEC] : 0.f);
            } else {
                dp[(int64_t)b * din] = hv[0] > 0.f ? s[0] : 0.f;
            }
        }
    }
#pragma unroll
    for (int o = 0; o < kMaxOut; ++o) {
        if (o < dout) {
            if (VEC == 4) *reinterpret_cast<float4*>(gW + (int64_t)o * din) =
                make_float4(acc[o][0], acc[o][1 % VEC], acc[o][2 % VEC], acc[o][3 % VEC]);
            else gW[(int64_t)o * din] = acc[o][0];
        }
    }
}

}  // namespace narrow
}  // namespace dpsgd
