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

// Forward product of the same layer: out[b][o] = b_o + sum_k h[b][k] W[o][k] (logits: no ReLU).  On the
// tensor-core kernel one CTA per node walks all of k alone (one 128-row tile, 90 % padding): latency,
// not bandwidth.  Here a CTA owns four samples of a node: thread t takes the 16-byte columns t, t + 128, ...
// of k, loads the up to 16 weight rows there once and uses them for the four samples (all loads of an
// iteration in flight together), then the 64 partial sums are reduced by shuffles and across the four
// warps in a fixed order.  Exact fp32 FMA products.
constexpr int kFwdThreads = 128;
constexpr int kFwdSamples = 4;

// grid (ceil(B / 4), nodes), block 128.  din % 4 == 0, rows 16-byte aligned.
__global__ void __launch_bounds__(kFwdThreads)
narrow_forward_kernel(const float* __restrict__ X, int64_t ld, int64_t w_off, int64_t b_off,
                      const float* __restrict__ h, float* __restrict__ out, int B, int din, int dout) {
    __shared__ float part[kFwdThreads / 32][kFwdSamples * kMaxOut];
    const int node = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b0 = blockIdx.x * kFwdSamples;
    const int nb = min(kFwdSamples, B - b0);
    const int d4 = din / 4;
    const float4* W = reinterpret_cast<const float4*>(X + (int64_t)node * ld + w_off);
    const float4* hv = reinterpret_cast<const float4*>(h + ((int64_t)node * B + b0) * din);
    float acc[kFwdSamples][kMaxOut];
#pragma unroll
    for (int s = 0; s < kFwdSamples; ++s)
#pragma unroll
        for (int o = 0; o < kMaxOut; ++o) acc[s][o] = 0.f;
    for (int c = tid; c < d4; c += kFwdThreads) {
        float4 w[kMaxOut], x[kFwdSamples];
#pragma unroll
        for (int o = 0; o < kMaxOut; ++o)
            w[o] = o < dout ? __ldg(W + (int64_t)o * d4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < kFwdSamples; ++s)
            x[s] = s < nb ? __ldg(hv + (int64_t)s * d4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < kFwdSamples; ++s)
#pragma unroll
            for (int o = 0; o < kMaxOut; ++o) {
                acc[s][o] = fmaf(x[s].x, w[o].x, acc[s][o]); acc[s][o] = fmaf(x[s].y, w[o].y, acc[s][o]);
                acc[s][o] = fmaf(x[s].z, w[o].z, acc[s][o]); acc[s][o] = fmaf(x[s].w, w[o].w, acc[s][o]);
            }
    }
#pragma unroll
    for (int s = 0; s < kFwdSamples; ++s)
#pragma unroll
        for (int o = 0; o < kMaxOut; ++o) {
            float v = acc[s][o];
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sh);
            if (lane == 0) part[warp][s * kMaxOut + o] = v;
        }
    __syncthreads();
    if (tid < kFwdSamples * kMaxOut) {
        const int s = tid / kMaxOut, o = tid % kMaxOut;
        if (s < nb && o < dout) {
            float v = part[0][tid];
#pragma unroll
            for (int wv = 1; wv < kFwdThreads / 32; ++wv) v += part[wv][tid];
            out[((int64_t)node * B + b0 + s) * dout + o] = v + __ldg(X + (int64_t)node * ld + b_off + o);
        }
    }
}

}  // namespace narrow
}  // namespace dpsgd
