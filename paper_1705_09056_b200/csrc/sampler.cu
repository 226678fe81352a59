// Algorithm 1 step 2 as a stand-alone kernel: the minibatch indices of every node.
#include "ctx.h"
#include "philox.cuh"

namespace dpsgd {
namespace {

__global__ void sample_kernel(uint64_t seed, uint64_t k, int n, int B, uint32_t m, int32_t* __restrict__ idx) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n * B) return;
    const int node = t / B, b = t - node * B;
    idx[t] = sample_index(seed, k, (uint32_t)node, (uint32_t)b, m);
}

__global__ void set_k_kernel(uint64_t* k, uint64_t v) { k[0] = v; k[1] = v + 1; }   // the two slots of a replayed chain
__global__ void advance_k_kernel(uint64_t* k) { *k += 1; }

}  // namespace

cudaError_t launch_set_k(dpsgd_ctx* c, uint64_t v) {
    set_k_kernel<<<1, 1, 0, c->stream>>>(c->d_k, v);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_advance_k(dpsgd_ctx* c) {
    advance_k_kernel<<<1, 1, 0, c->stream>>>(c->d_k);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_sample(dpsgd_ctx* c, uint64_t k, int32_t* idx) {
    const int total = c->n * c->batch;
    sample_kernel<<<(total + 127) / 128, 128, 0, c->stream>>>(c->seed, k, c->n, c->batch, (uint32_t)c->m, idx);
    c->launches++;
    return cudaGetLastError();
}

}  // namespace dpsgd
