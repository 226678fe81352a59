// Backward of the 3x3 convolution layer of conv_fwd.cu (the gradient half of Algorithm 1 step 3 for the paper's
// image workloads, Sections 5.1 / 5.3), for all nodes at once, every node with its own filters:
//
//     dym = dy * [y > 0]                                   (ReLU layers; ReLU'(0) = 0)
//     db[o]            = sum_{b,i,j} dym[b][o][i][j]
//     dw[o][c][kh][kw] = sum_{b,i,j} dym[b][o][i][j] * x[b][c][s i + kh - 1][s j + kw - 1]
//     dx[b][c][h][w]   = sum_{o,kh,kw} w[o][c][kh][kw] * dym[b][o][i][j]   over s i + kh - 1 = h, s j + kw - 1 = w
//
// The two contractions run on the tensor-core kernels that exist already, fed by small streaming kernels:
//   filter gradient  the input of every image is unfolded (U[k = (c,kh,kw)][p = (i,j)], p contiguous) and the
//                    batched GEMM of tc_gemm.cuh (tcgen05, three TF32 MMAs per product) contracts it with dym
//                    over the positions, one problem per (node, image); the per-image results are then added
//                    in image order (bit-reproducible) into the gradient matrix G at the filters' columns.
//   input gradient   is itself a stride-1 3x3 convolution: of dym (for a stride-2 layer: of dym spread out
//                    with zeros between its elements) with the filters flipped in both directions and
//                    transposed in (o, c); it runs on conv3x3_fwd_kernel with those filters.
// Scratch (masked gradient, unfolded input, per-image filter gradients, flipped filters, spread gradient) is
// one library-owned buffer that grows to the largest layer seen and lives until dpsgd_destroy.
#include <algorithm>

#include "ctx.h"

namespace dpsgd {
namespace {

// dym = dy * [y > 0] (or dy); for a stride-2 layer also D[2i][2j] = dym[i][j] into a zeroed H x W image.
__global__ void __launch_bounds__(256)
conv_mask_kernel(const float* __restrict__ dy, const float* __restrict__ y, float* __restrict__ dym,
                 float* __restrict__ spread, int64_t total, int pos, int wo, int h, int w) {
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= total) return;
    float v = __ldg(dy + t);
    if (y && !(__ldg(y + t) > 0.f)) v = 0.f;
    dym[t] = v;
    if (spread) {
        const int64_t img = t / pos;
        const int q = (int)(t - img * pos), i = q / wo, j = q - i * wo;
        spread[img * (int64_t)h * w + (int64_t)(2 * i) * w + 2 * j] = v;
    }
}

// db[node][o] = sum over images and positions, thread-strided partial sums combined in a fixed order.
__global__ void __launch_bounds__(256)
conv_bias_grad_kernel(const float* __restrict__ dym, float* __restrict__ G, int64_t ld, int64_t b_off, int batch,
                      int c_out, int pos) {
    __shared__ float red[256];
    const int o = blockIdx.x, node = blockIdx.y, tid = threadIdx.x;
    float acc = 0.f;
    for (int b = 0; b < batch; ++b) {
        const float* p = dym + (((int64_t)node * batch + b) * c_out + o) * pos;
        for (int q = tid; q < pos; q += 256) acc += __ldg(p + q);
    }
    red[tid] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (tid < s) red[tid] += red[tid + s];
        __syncthreads();
    }
    if (tid == 0) G[(int64_t)node * ld + b_off + o] = red[0];
}

// U[img][k = (c,kh,kw)][p = (i,j)] = x[img][c][s i + kh - 1][s j + kw - 1], zero outside the image.
// Block (px, 256 / px): threadIdx.x walks the positions, VEC consecutive ones of an output row per thread (VEC = 4
// when the output width is a multiple of 4: one 16-byte store), threadIdx.y the taps; grid (position chunks, tap
// groups, images).
template <int VEC>
__global__ void __launch_bounds__(256)
conv_unfold_kernel(const float* __restrict__ x, float* __restrict__ U, int c_in, int h, int w, int ho, int wo, int stride) {
    const int pos = ho * wo;
    const int q = (blockIdx.x * blockDim.x + threadIdx.x) * VEC;
    const int k = blockIdx.y * blockDim.y + threadIdx.y;
    if (q >= pos || k >= 9 * c_in) return;
    const int c = k / 9, tap = k - 9 * c, kh = tap / 3, kw = tap - 3 * kh;
    const int64_t img = blockIdx.z;
    const int i = q / wo, j = q - i * wo;
    const int hh = stride * i + kh - 1;
    const float* row = x + ((img * c_in + c) * (int64_t)h + hh) * w;
    float v[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) {
        const int ww = stride * (j + u) + kw - 1;
        v[u] = (hh >= 0 && hh < h && ww >= 0 && ww < w) ? __ldg(row + ww) : 0.f;
    }
    float* dst = U + (img * (9 * c_in) + k) * (int64_t)pos + q;
    if (VEC == 4) *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1 % VEC], v[2 % VEC], v[3 % VEC]);
    else dst[0] = v[0];
}

// G[node][w_off + e] = sum_b P[node][b][e], images added in order.
__global__ void __launch_bounds__(256)
conv_sum_images_kernel(const float* __restrict__ P, float* __restrict__ G, int64_t ld, int64_t w_off, int batch,
                       int64_t elems) {
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int node = blockIdx.y;
    if (e >= elems) return;
    const float* p = P + (int64_t)node * batch * elems + e;
    float s = 0.f;
    for (int b = 0; b < batch; ++b) s += __ldg(p + (int64_t)b * elems);
    G[(int64_t)node * ld + w_off + e] = s;
}

// Wt[node][c][o][kh][kw] = w[node][o][c][2 - kh][2 - kw]: the filters of the input gradient's convolution.
__global__ void __launch_bounds__(256)
conv_flip_filters_kernel(const float* __restrict__ X, int64_t ld, int64_t w_off, float* __restrict__ Wt, int c_in,
                         int c_out) {
    const int64_t per = (int64_t)c_in * c_out * 9;
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int node = blockIdx.y;
    if (t >= per) return;
    const int c = (int)(t / (c_out * 9)), r = (int)(t - (int64_t)c * c_out * 9);
    const int o = r / 9, tap = r - 9 * o, kh = tap / 3, kw = tap - 3 * kh;
    Wt[node * per + t] = __ldg(X + (int64_t)node * ld + w_off + ((int64_t)(o * c_in + c) * 3 + (2 - kh)) * 3 + (2 - kw));
}

size_t round64(size_t v) { return (v + 63) / 64 * 64; }
unsigned blocks(int64_t total) { return (unsigned)((total + 255) / 256); }

}  // namespace

cudaError_t launch_conv3x3_backward(dpsgd_ctx* c, const float* x, const float* y, const float* dy, int batch, int c_in,
                                    int h, int w, int c_out, int stride, int64_t w_off, int64_t b_off, int relu,
                                    float* dx, const char** why) {
    *why = nullptr;
    const int n = c->n;
    const int ho = (h - 1) / stride + 1, wo = (w - 1) / stride + 1, pos = ho * wo, kc = 9 * c_in;
    const int64_t imgs = (int64_t)n * batch;
    if (imgs > 65535) { *why = "nodes x images must be at most 65535"; return cudaErrorNotSupported; }
    if (dx) {
        if (const char* u = conv3x3_forward_unsupported(batch, c_out, stride == 2 ? h : ho, stride == 2 ? w : wo, c_in, 1)) {
            *why = u;       // the input gradient runs on the forward kernel with the roles of the channels swapped
            return cudaErrorNotSupported;
        }
    }
    const size_t f_dym = round64((size_t)imgs * c_out * pos), f_unf = round64((size_t)imgs * kc * pos);
    const size_t f_par = round64((size_t)imgs * c_out * kc), f_flip = dx ? round64((size_t)n * c_in * c_out * 9) : 0;
    const size_t f_spread = (dx && stride == 2) ? round64((size_t)imgs * c_out * h * w) : 0;
    const size_t need = f_dym + f_unf + f_par + f_flip + f_spread;
    if (c->conv_ws_floats < need) {
        cudaError_t e = cudaStreamSynchronize(c->stream);      // kernels in flight may still use the old buffer
        if (e != cudaSuccess) return e;
        cudaFree(c->d_conv_ws);
        c->d_conv_ws = nullptr; c->conv_ws_floats = 0;
        if ((e = cudaMalloc(&c->d_conv_ws, need * sizeof(float))) != cudaSuccess) return e;
        c->conv_ws_floats = need;
    }
    float* dym = c->d_conv_ws;
    float* unf = dym + f_dym;
    float* par = unf + f_unf;
    float* flip = par + f_par;
    float* spread = f_spread ? flip + f_flip : nullptr;

    cudaError_t e = cudaSuccess;
    if (spread) e = cudaMemsetAsync(spread, 0, f_spread * sizeof(float), c->stream);
    if (e != cudaSuccess) return e;
    const int64_t total = imgs * c_out * pos;
    conv_mask_kernel<<<blocks(total), 256, 0, c->stream>>>(dy, relu ? y : nullptr, dym, spread, total, pos, wo, h, w);
    conv_bias_grad_kernel<<<dim3(c_out, n), 256, 0, c->stream>>>(dym, c->G, c->ld, b_off, batch, c_out, pos);
    {
        const int vec = wo % 4 == 0 ? 4 : 1;                 // then pos % 4 == 0 too and every store is 16-byte aligned
        const int chunks = (pos + vec - 1) / vec;
        int px = 1;
        while (px < chunks && px < 256) px *= 2;
        const dim3 block((unsigned)px, (unsigned)(256 / px));
        const dim3 grid((unsigned)((chunks + px - 1) / px), (unsigned)((kc + block.y - 1) / block.y), (unsigned)imgs);
        if (vec == 4) conv_unfold_kernel<4><<<grid, block, 0, c->stream>>>(x, unf, c_in, h, w, ho, wo, stride);
        else conv_unfold_kernel<1><<<grid, block, 0, c->stream>>>(x, unf, c_in, h, w, ho, wo, stride);
    }
    c->launches += 3;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // per image: par[o][k] = sum_p unf[k][p] * dym[o][p]
    e = launch_tc_gemm_kmajor(c, unf, (int64_t)kc * pos, pos, dym, (int64_t)c_out * pos, pos, par, (int64_t)c_out * kc, kc,
                              kc, c_out, pos, (int)imgs);
    if (e != cudaSuccess) return e;
    const int64_t elems = (int64_t)c_out * kc;
    conv_sum_images_kernel<<<dim3(blocks(elems), n), 256, 0, c->stream>>>(par, c->G, c->ld, w_off, batch, elems);
    c->launches++;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (dx) {
        const int64_t per = (int64_t)c_in * c_out * 9;
        conv_flip_filters_kernel<<<dim3(blocks(per), n), 256, 0, c->stream>>>(c->X[c->cur], c->ld, w_off, flip, c_in, c_out);
        c->launches++;
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        e = launch_conv3x3_forward_on(c, spread ? spread : dym, batch, c_out, spread ? h : ho, spread ? w : wo, c_in, 1,
                                      flip, nullptr, per, 0, dx, why);
    }
    return e;
}

}  // namespace dpsgd
