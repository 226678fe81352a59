// Internal state of a D-PSGD context and the kernel launchers the C ABI dispatches to.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <utility>
#include <vector>

#include "../../include/dpsgd.h"

namespace dpsgd {

constexpr int kMaxLayers = 8;
constexpr int kFusedMaxDegree = 8;   // widest row of W the gradient kernel's gossip epilogue gathers

// Mixing matrix W on the device, as the kernels consume it.
struct MixW {
    int n = 0;
    int nnz = 0;
    int max_deg = 0;
    int uniform_deg = 0;               // the common number of entries per row, 0 when rows differ
    const int32_t* row_ptr = nullptr;  // [n+1]
    const int32_t* col = nullptr;      // [nnz]
    const float* val = nullptr;        // [nnz]
    const float* band = nullptr;       // ring only: [n][3] = (W_{i,i-1}, W_ii, W_{i,i+1})
    float uniform = 0.f;               // uniform dense only: the common entry
};

// Written by the device, read back by the synchronising calls.
struct ResultBlock {
    double value;   // consensus distance
    int status;     // 0, or a dpsgd_status set by a kernel whose bounded wait ran out
    int pad;
};

struct MlpShape {
    int nlayers = 0;                 // number of weight layers L
    int dims[kMaxLayers + 1] = {0};  // d_0 .. d_L
    int64_t w_off[kMaxLayers] = {0}; // offset of W_l inside a parameter row
    int64_t b_off[kMaxLayers] = {0}; // offset of b_l
};

}  // namespace dpsgd

struct dpsgd_ctx {
    int n = 0;
    int64_t N = 0;
    float gamma = 0.f;
    uint64_t seed = 0;
    int device = 0;

    // W
    std::vector<int32_t> h_row_ptr, h_col;
    std::vector<float> h_val;
    dpsgd::MixW W;
    void* d_w_blob = nullptr;  // one allocation holding row_ptr | col | val | band
    int mix_kind = DPSGD_MIX_GATHER_CSR;
    bool swapped = false;      // footnote c of Algorithm 1: update locally, then average
    float beta = 0.f;          // momentum coefficient
    float* V = nullptr;        // momentum buffers [n][ld] (caller-owned), NULL = plain SGD
    bool can_ring = false, can_uniform = false, can_tiled = false;
    bool kind_forced = false;  // dpsgd_mix_kind(force) was used: no automatic small-problem kernel

    // bound buffers
    float* X[2] = {nullptr, nullptr};
    float* G = nullptr;
    int cur = 0;
    int64_t ld = 0;
    cudaStream_t stream = nullptr;
    bool bound = false;

    // model + data
    int model = -1;
    int d = 0;  // input width
    int batch = 0;
    float l2 = 0.f;
    int mlp_precision = 0;
    dpsgd::MlpShape mlp;
    const float* A = nullptr;
    const void* y = nullptr;
    int64_t m = 0;
    bool have_data = false;

    // scratch (library-owned)
    int32_t* d_idx = nullptr;    // [n][B]
    float* d_coef = nullptr;     // [n][B] per-sample backward coefficients (linear models)
    float* d_glm_part = nullptr; // [n][ceil(B / 4)][ld] shares of the gradient, one per group of four draws
    size_t glm_part_floats = 0;
    int32_t* d_node_batch = nullptr;  // [n] per-node minibatch sizes B_i <= B; NULL: every node uses B
    int32_t* d_active = nullptr;      // [n] nodes that take part in a masked local step
    float* d_act = nullptr;      // MLP activations h_0..h_L  (see grad_mlp.cu for the layout)
    float* d_delta = nullptr;    // MLP back-propagated errors
    size_t act_floats = 0, delta_floats = 0;
    float* d_stream_parts = nullptr;   // MLP forward / input gradient: accumulators of tiles shared by two CTAs
    size_t stream_parts_floats = 0;
    double* d_partials = nullptr;  // consensus partial sums, one per CTA
    int partials_cap = 0;
    dpsgd::ResultBlock* d_result = nullptr;  // final scalar + device status word
    dpsgd::ResultBlock* h_result = nullptr;  // pinned
    void* tma_state = nullptr;     // tensor maps for the tiled mixing kernel

    // graph replay of pairs of iterations (small, launch-bound problems)
    uint64_t* d_k = nullptr;                 // device iteration counter (two slots, see capture_pair)
    const uint64_t* k_dev_active = nullptr;  // non-NULL only while a graph is captured
    uint64_t* k_dev_next = nullptr;          // capture of a self-advancing step kernel: the slot it leaves k + 2 in
    int chain_pos = 0;                       // position of the iteration being captured inside its chain
    cudaGraphExec_t graph_exec = nullptr;
    cudaStream_t capture_stream = nullptr;   // private stream the pair is recorded on
    int graph_cur = 0;                       // value of `cur` the graph was captured at
    int64_t graph_launches = 0;              // kernels in one replay

    // gossip step fused into the MLP weight-gradient kernels (dpsgd_set_fused_step)
    // W = w 1 1^T in the fused iteration: every row mixes to the column mean, so the kernels gather from
    // a one-row matrix (the mean, recomputed each iteration) through a CSR with one entry per row
    void* d_mean_blob = nullptr;           // mean [ld] | row_ptr [n+1] | col [n] | val [n]
    int64_t mean_ld = 0;
    const float* fsrc_X = nullptr;         // what the fused kernels gather from during this iteration
    int64_t fsrc_ld = 0;
    const int32_t* fsrc_row_ptr = nullptr;
    const int32_t* fsrc_col = nullptr;
    const float* fsrc_val = nullptr;
    int fuse_step = 1;         // 0 off, 1 where it pays (default), 2 wherever a fused kernel applies, 3 as 2 without the ring kernel
    std::vector<std::pair<int64_t, int64_t>> fused_blocks;   // [begin, end) columns already written to X_next

    // convolution backward: masked output gradient, unfolded input, per-image filter gradients, flipped filters
    float* d_conv_ws = nullptr;
    size_t conv_ws_floats = 0;

    int64_t launches = 0;
    std::string err;
};

namespace dpsgd {

// Each launcher enqueues on ctx->stream, bumps ctx->launches and returns cudaGetLastError().
cudaError_t launch_mix_ring(dpsgd_ctx* c, const float* X, const float* G, float* Xn);
cudaError_t launch_mix_uniform(dpsgd_ctx* c, const float* X, const float* G, float* Xn);
cudaError_t launch_mix_gather(dpsgd_ctx* c, const float* X, const float* G, float* Xn);
cudaError_t launch_mix_rowpar(dpsgd_ctx* c, const float* X, const float* G, float* Xn);
bool mix_is_small(const dpsgd_ctx* c);
cudaError_t launch_mix_tiled(dpsgd_ctx* c, const float* X, const float* G, float* Xn, double* stats_out = nullptr);
bool mix_tiled_supported(const dpsgd_ctx* c);
// One CTA that waits, with the kernels' bounded wait cut to max_polls polls, on an mbarrier nothing arrives at.
cudaError_t launch_wait_probe(dpsgd_ctx* c, uint32_t max_polls);
void mix_tiled_release(dpsgd_ctx* c);

cudaError_t launch_consensus(dpsgd_ctx* c, const float* X, double* result_dev);
cudaError_t ensure_partials(dpsgd_ctx* c, int count);
cudaError_t launch_consensus_final(dpsgd_ctx* c, int count, double* result_dev);
// active: device [n], rows with 0 are left untouched; NULL: every row.
cudaError_t launch_momentum(dpsgd_ctx* c, float* V, const float* G, const int32_t* active);
cudaError_t launch_local_update(dpsgd_ctx* c, float* X, const float* D, const int32_t* active);
cudaError_t launch_mix_variant(dpsgd_ctx* c, const float* X, const float* G, float* Xn, bool swapped,
                               double* stats_out, float* V);
cudaError_t launch_average(dpsgd_ctx* c, const float* X, float* xbar);

cudaError_t launch_sample(dpsgd_ctx* c, uint64_t k, int32_t* idx);
cudaError_t launch_set_k(dpsgd_ctx* c, uint64_t v);
cudaError_t launch_advance_k(dpsgd_ctx* c);
cudaError_t launch_grad_linear(dpsgd_ctx* c, uint64_t k, const float* X, float* G);
bool linear_step_fuses(const dpsgd_ctx* c);
bool linear_node_step_fuses(const dpsgd_ctx* c);   // the one-launch variant (its kernel advances the replay counter itself)
cudaError_t launch_linear_step(dpsgd_ctx* c, uint64_t k, const float* X, float* G, float* Xn);
// Xn != NULL: weight blocks whose product runs on the fused kernel are written to Xn after the gossip
// step instead of to G, and listed in c->fused_blocks.
cudaError_t launch_grad_mlp(dpsgd_ctx* c, uint64_t k, const float* X, float* G, float* Xn = nullptr);
bool fused_step_supported(const dpsgd_ctx* c);
bool fused_step_pays(const dpsgd_ctx* c, int din, int dout);
cudaError_t run_tcw_ring(dpsgd_ctx* c, const float* h, int din, const float* delta, int dout, int dpitch,
                         int64_t w_off, const float* X, float* Xn);
cudaError_t run_tcw_fused(dpsgd_ctx* c, const float* h, int din, const float* delta, int dout, int dpitch,
                          int64_t w_off, const float* X, float* Xn);
// Gossip step on the columns of [0, ld) outside c->fused_blocks.
cudaError_t launch_mix_rest(dpsgd_ctx* c, const float* X, const float* G, float* Xn);
// 3x3 convolution forward with every node's own filters (conv_fwd.cu).  *why names what is unsupported
// when the result is cudaErrorNotSupported.
const char* conv3x3_forward_unsupported(int batch, int c_in, int h, int w, int c_out, int stride);
cudaError_t launch_conv3x3_forward(dpsgd_ctx* c, const float* x, int batch, int c_in, int h, int w, int c_out, int stride,
                                   int64_t w_off, int64_t b_off, int relu, float* y, const char** why);
// Backward of the same layer (conv_bwd.cu): filter and bias gradients into G, optionally the input gradient.
cudaError_t launch_conv3x3_backward(dpsgd_ctx* c, const float* x, const float* y, const float* dy, int batch, int c_in,
                                    int h, int w, int c_out, int stride, int64_t w_off, int64_t b_off, int relu,
                                    float* dx, const char** why);
// Forward kernel on filters outside the parameter matrix (W: first filter of node 0, rows ld_w apart; bias may be
// NULL = none): what the input gradient runs on.
cudaError_t launch_conv3x3_forward_on(dpsgd_ctx* c, const float* x, int batch, int c_in, int h, int w, int c_out,
                                      int stride, const float* W, const float* bias, int64_t ld_w, int relu, float* y,
                                      const char** why);
cudaError_t launch_tc_gemm_kmajor(dpsgd_ctx* c, const float* A, int64_t a_problem, int64_t a_pitch, const float* B,
                                  int64_t b_problem, int64_t b_pitch, float* C, int64_t c_problem, int64_t c_pitch,
                                  int M, int N, int K, int problems);
size_t mlp_act_floats(const dpsgd_ctx* c);
size_t mlp_delta_floats(const dpsgd_ctx* c);
size_t mlp_stream_parts_floats(int sms);

}  // namespace dpsgd
