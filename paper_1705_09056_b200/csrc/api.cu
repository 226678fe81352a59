// C ABI of libdpsgd: argument checking, validation of W, context state and dispatch.
// No arithmetic of the method lives here; every step runs in the kernels of the other files.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "ctx.h"

using namespace dpsgd;

namespace {

thread_local std::string g_create_error = "";

dpsgd_status fail(dpsgd_ctx* c, dpsgd_status s, const std::string& msg) {
    if (c) c->err = msg; else g_create_error = msg;
    return s;
}

dpsgd_status cuda_fail(dpsgd_ctx* c, cudaError_t e, const char* what) {
    return fail(c, DPSGD_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

// Section 3: W symmetric, doubly stochastic, entries in [0,1]; CSR rows sorted and unique.
bool validate_w(int n, const int32_t* rp, const int32_t* col, const float* val, std::string* why) {
    char buf[160];
    if (rp[0] != 0) { *why = "row_ptr[0] != 0"; return false; }
    for (int i = 0; i < n; ++i) {
        if (rp[i + 1] < rp[i]) { *why = "row_ptr not non-decreasing"; return false; }
        if (rp[i + 1] - rp[i] > n) { *why = "row with more than n entries"; return false; }
    }
    for (int i = 0; i < n; ++i) {
        double sum = 0.0;
        for (int p = rp[i]; p < rp[i + 1]; ++p) {
            const int j = col[p];
            if (j < 0 || j >= n) {
                snprintf(buf, sizeof buf, "row %d: column %d out of range", i, j);
                *why = buf; return false;
            }
            if (p > rp[i] && col[p - 1] >= j) {
                snprintf(buf, sizeof buf, "row %d: columns not strictly increasing", i);
                *why = buf; return false;
            }
            const float v = val[p];
            if (!(v >= 0.f && v <= 1.f)) {
                snprintf(buf, sizeof buf, "W[%d][%d] = %g outside [0,1]", i, j, (double)v);
                *why = buf; return false;
            }
            sum += (double)v;
        }
        if (std::fabs(sum - 1.0) > 1e-6) {
            snprintf(buf, sizeof buf, "row %d sums to %.9g, not 1", i, sum);
            *why = buf; return false;
        }
    }
    for (int i = 0; i < n; ++i) {
        for (int p = rp[i]; p < rp[i + 1]; ++p) {
            const int j = col[p];
            const int32_t* b = col + rp[j];
            const int32_t* e = col + rp[j + 1];
            const int32_t* it = std::lower_bound(b, e, i);
            const float mirror = (it != e && *it == i) ? val[it - col] : 0.f;
            if (mirror != val[p]) {
                snprintf(buf, sizeof buf, "W[%d][%d] = %g but W[%d][%d] = %g (not symmetric)", i, j,
                         (double)val[p], j, i, (double)mirror);
                *why = buf; return false;
            }
        }
    }
    return true;
}

void classify_w(dpsgd_ctx* c) {
    const int n = c->n;
    const auto& rp = c->h_row_ptr;
    const auto& col = c->h_col;
    const auto& val = c->h_val;
    int max_deg = 0;
    for (int i = 0; i < n; ++i) max_deg = std::max(max_deg, rp[i + 1] - rp[i]);
    c->W.max_deg = max_deg;
    bool same_deg = true;
    for (int i = 0; i < n; ++i) same_deg = same_deg && rp[i + 1] - rp[i] == max_deg;
    c->W.uniform_deg = same_deg ? max_deg : 0;

    bool uniform = (int64_t)rp[n] == (int64_t)n * n;
    if (uniform)
        for (size_t p = 1; p < val.size() && uniform; ++p)
            uniform = (memcmp(&val[p], &val[0], sizeof(float)) == 0);
    c->can_uniform = uniform;
    if (uniform) c->W.uniform = val[0];

    bool ringlike = n >= 3;
    for (int i = 0; i < n && ringlike; ++i) {
        if (rp[i + 1] - rp[i] != 3) { ringlike = false; break; }
        int want[3] = {(i + n - 1) % n, i, (i + 1) % n};
        std::sort(want, want + 3);
        for (int t = 0; t < 3; ++t)
            if (col[rp[i] + t] != want[t]) ringlike = false;
    }
    c->can_ring = ringlike;
    c->can_tiled = mix_tiled_supported(c);

    if (uniform && n != 3) c->mix_kind = DPSGD_MIX_UNIFORM_DENSE;
    else if (ringlike) c->mix_kind = DPSGD_MIX_RING;
    else if (uniform) c->mix_kind = DPSGD_MIX_UNIFORM_DENSE;
    else if (c->can_tiled) c->mix_kind = DPSGD_MIX_TILED_CSR;
    else c->mix_kind = DPSGD_MIX_GATHER_CSR;
}

// Anything baked into a captured graph changed: drop it.
void drop_graph(dpsgd_ctx* c) {
    if (c->graph_exec) { cudaGraphExecDestroy(c->graph_exec); c->graph_exec = nullptr; }
}

float band_entry(const dpsgd_ctx* c, int i, int j) {
    for (int p = c->h_row_ptr[i]; p < c->h_row_ptr[i + 1]; ++p)
        if (c->h_col[p] == j) return c->h_val[p];
    return 0.f;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

void release(dpsgd_ctx* c) {
    if (!c) return;
    mix_tiled_release(c);
    drop_graph(c);
    if (c->capture_stream) cudaStreamDestroy(c->capture_stream);
    cudaFree(c->d_k);
    cudaFree(c->d_w_blob);
    cudaFree(c->d_mean_blob);
    cudaFree(c->d_idx);
    cudaFree(c->d_coef);
    cudaFree(c->d_glm_part);
    cudaFree(c->d_node_batch);
    cudaFree(c->d_active);
    cudaFree(c->d_act);
    cudaFree(c->d_delta);
    cudaFree(c->d_stream_parts);
    cudaFree(c->d_partials);
    cudaFree(c->d_conv_ws);
    cudaFree(c->d_result);
    if (c->h_result) cudaFreeHost(c->h_result);
    delete c;
}

// Copies the device status word back, waits for the stream and clears the word when a kernel set it.
// DPSGD_ERR_TIMEOUT when a bounded device-side wait ran out since the last check.
dpsgd_status collect_device_status(dpsgd_ctx* c) {
    if (!c->d_result || !c->h_result) return DPSGD_OK;
    cudaError_t e = cudaMemcpyAsync(&c->h_result->status, &c->d_result->status, sizeof(int), cudaMemcpyDeviceToHost,
                                    c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "stream synchronisation");
    if (c->h_result->status != 0) {
        c->h_result->status = 0;
        e = cudaMemsetAsync(&c->d_result->status, 0, sizeof(int), c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        return fail(c, DPSGD_ERR_TIMEOUT,
                    "a kernel gave up waiting for a tile copy since the last synchronising call; X is not valid");
    }
    return DPSGD_OK;
}

dpsgd_status need_bound(dpsgd_ctx* c) {
    if (!c) return DPSGD_ERR_ARG;
    if (!c->bound) return fail(c, DPSGD_ERR_STATE, "no buffers bound: call dpsgd_bind first");
    return DPSGD_OK;
}

dpsgd_status need_model(dpsgd_ctx* c) {
    if (c->model < 0) return fail(c, DPSGD_ERR_STATE, "no model: call dpsgd_set_model first");
    if (!c->have_data) return fail(c, DPSGD_ERR_STATE, "no data: call dpsgd_set_data first");
    return DPSGD_OK;
}

// The buffer the gossip step subtracts: the gradients, or the momentum buffers after their update.
cudaError_t step_direction(dpsgd_ctx* c, const float** dir, const int32_t* active = nullptr) {
    *dir = c->G;
    if (!c->V) return cudaSuccess;
    *dir = c->V;
    return launch_momentum(c, c->V, c->G, active);
}

// Ring and uniform W have kernels that update the momentum buffers inside the gossip pass.
bool momentum_fuses(const dpsgd_ctx* c) {
    return c->V && (c->mix_kind == DPSGD_MIX_RING || c->mix_kind == DPSGD_MIX_UNIFORM_DENSE);
}

cudaError_t run_mix(dpsgd_ctx* c) {
    const float* X = c->X[c->cur];
    float* Xn = c->X[c->cur ^ 1];
    const bool small = !c->kind_forced && mix_is_small(c);
    if (!small && momentum_fuses(c)) return launch_mix_variant(c, X, c->G, Xn, c->swapped, nullptr, c->V);
    const float* D = nullptr;
    cudaError_t e = step_direction(c, &D);
    if (e != cudaSuccess) return e;
    if (small) return launch_mix_rowpar(c, X, D, Xn);   // latency-bound sizes
    if (c->swapped && c->mix_kind != DPSGD_MIX_TILED_CSR) return launch_mix_variant(c, X, D, Xn, true, nullptr, nullptr);
    switch (c->mix_kind) {
        case DPSGD_MIX_RING: return launch_mix_ring(c, X, D, Xn);
        case DPSGD_MIX_UNIFORM_DENSE: return launch_mix_uniform(c, X, D, Xn);
        case DPSGD_MIX_TILED_CSR: return launch_mix_tiled(c, X, D, Xn);
        default: return launch_mix_gather(c, X, D, Xn);
    }
}

cudaError_t run_grad(dpsgd_ctx* c, uint64_t k) {
    if (c->model == DPSGD_MODEL_MLP) return launch_grad_mlp(c, k, c->X[c->cur], c->G);
    return launch_grad_linear(c, k, c->X[c->cur], c->G);
}

}  // namespace

namespace dpsgd {
// Lets entry points that take no context leave a message for dpsgd_last_error(NULL).
void set_thread_error(const std::string& msg) { g_create_error = msg; }
}  // namespace dpsgd

namespace {
cudaError_t prepare_fused_source(dpsgd_ctx* c, const float* X);   // defined beside dpsgd_set_fused_step
}

extern "C" {

DPSGD_API dpsgd_status dpsgd_create(dpsgd_ctx** out, int32_t n, int64_t N, const int32_t* row_ptr,
                          const int32_t* col_idx, const float* val, float gamma, uint64_t seed) {
    if (!out) return fail(nullptr, DPSGD_ERR_ARG, "out is NULL");
    *out = nullptr;
    if (n < 1 || n > 65535) return fail(nullptr, DPSGD_ERR_ARG, "n must be in [1, 65535]");
    if (N < 1 || N >= (int64_t(1) << 40)) return fail(nullptr, DPSGD_ERR_ARG, "N must be in [1, 2^40)");
    if (!row_ptr || !col_idx || !val) return fail(nullptr, DPSGD_ERR_ARG, "CSR pointer is NULL");
    if (!(gamma == gamma)) return fail(nullptr, DPSGD_ERR_ARG, "gamma is NaN");
    std::string why;
    if (!validate_w(n, row_ptr, col_idx, val, &why)) return fail(nullptr, DPSGD_ERR_W_INVALID, why);

    dpsgd_ctx* c = new (std::nothrow) dpsgd_ctx();
    if (!c) return fail(nullptr, DPSGD_ERR_ARG, "out of host memory");
    c->n = n; c->N = N; c->gamma = gamma; c->seed = seed;
    const int nnz = row_ptr[n];
    c->h_row_ptr.assign(row_ptr, row_ptr + n + 1);
    c->h_col.assign(col_idx, col_idx + nnz);
    c->h_val.assign(val, val + nnz);
    c->W.n = n; c->W.nnz = nnz;

    cudaError_t e = cudaGetDevice(&c->device);
    if (e != cudaSuccess) { auto s = cuda_fail(nullptr, e, "cudaGetDevice"); release(c); return s; }
    classify_w(c);

    // one blob: row_ptr | col | val | band
    const size_t o_rp = 0;
    const size_t o_col = (o_rp + sizeof(int32_t) * (n + 1) + 255) / 256 * 256;
    const size_t o_val = (o_col + sizeof(int32_t) * nnz + 255) / 256 * 256;
    const size_t o_band = (o_val + sizeof(float) * nnz + 255) / 256 * 256;
    const size_t total = o_band + sizeof(float) * 3 * n;
    std::vector<char> blob(total, 0);
    memcpy(blob.data() + o_rp, row_ptr, sizeof(int32_t) * (n + 1));
    memcpy(blob.data() + o_col, col_idx, sizeof(int32_t) * nnz);
    memcpy(blob.data() + o_val, val, sizeof(float) * nnz);
    if (c->can_ring) {
        float* band = reinterpret_cast<float*>(blob.data() + o_band);
        for (int i = 0; i < n; ++i) {
            band[3 * i + 0] = band_entry(c, i, (i + n - 1) % n);
            band[3 * i + 1] = band_entry(c, i, i);
            band[3 * i + 2] = band_entry(c, i, (i + 1) % n);
        }
    }
    e = cudaMalloc(&c->d_w_blob, total);
    if (e == cudaSuccess) e = cudaMemcpy(c->d_w_blob, blob.data(), total, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_result, sizeof(ResultBlock));
    if (e == cudaSuccess) e = cudaMemset(c->d_result, 0, sizeof(ResultBlock));
    if (e == cudaSuccess) e = cudaMallocHost(&c->h_result, sizeof(ResultBlock));
    if (e != cudaSuccess) { auto s = cuda_fail(nullptr, e, "dpsgd_create allocation"); release(c); return s; }
    char* base = static_cast<char*>(c->d_w_blob);
    c->W.row_ptr = reinterpret_cast<int32_t*>(base + o_rp);
    c->W.col = reinterpret_cast<int32_t*>(base + o_col);
    c->W.val = reinterpret_cast<float*>(base + o_val);
    c->W.band = reinterpret_cast<float*>(base + o_band);
    *out = c;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_destroy(dpsgd_ctx* c) {
    if (!c) return DPSGD_ERR_ARG;
    const dpsgd_status s = c->bound ? collect_device_status(c) : DPSGD_OK;
    release(c);
    return s == DPSGD_ERR_TIMEOUT ? s : DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_bind(dpsgd_ctx* c, float* X0, float* X1, float* G, int64_t ld, void* stream) {
    if (!c) return DPSGD_ERR_ARG;
    if (!X0 || !X1 || !G) return fail(c, DPSGD_ERR_ARG, "buffer pointer is NULL");
    if (ld < c->N) return fail(c, DPSGD_ERR_ARG, "ld < N");
    if (ld % 32 != 0) return fail(c, DPSGD_ERR_ALIGN, "ld must be a multiple of 32 floats");
    if (!aligned(X0, 128) || !aligned(X1, 128) || !aligned(G, 128))
        return fail(c, DPSGD_ERR_ALIGN, "X0, X1 and G must be 128-byte aligned");
    const uintptr_t bytes = (uintptr_t)c->n * (uintptr_t)ld * sizeof(float);
    const uintptr_t p[3] = {(uintptr_t)X0, (uintptr_t)X1, (uintptr_t)G};
    for (int a = 0; a < 3; ++a)
        for (int b = a + 1; b < 3; ++b)
            if (p[a] < p[b] + bytes && p[b] < p[a] + bytes)
                return fail(c, DPSGD_ERR_ARG, "X0, X1 and G must not overlap");
    c->X[0] = X0; c->X[1] = X1; c->G = G; c->cur = 0; c->ld = ld;
    c->stream = static_cast<cudaStream_t>(stream);
    drop_graph(c);
    c->bound = true;
    c->V = nullptr; c->beta = 0.f;    // momentum buffers belong to the previous binding
    mix_tiled_release(c);  // tensor maps depend on the bound pointers
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_set_model(dpsgd_ctx* c, int32_t kind, const int32_t* dims, int32_t ndims,
                             float l2_lambda, int32_t batch, int32_t mlp_precision) {
    if (!c) return DPSGD_ERR_ARG;
    if (!dims || ndims < 1) return fail(c, DPSGD_ERR_ARG, "dims missing");
    if (batch < 1 || batch > 4096) return fail(c, DPSGD_ERR_ARG, "batch must be in [1, 4096]");
    for (int t = 0; t < ndims; ++t)
        if (dims[t] < 1) return fail(c, DPSGD_ERR_ARG, "non-positive layer width");
    int64_t want = 0;
    MlpShape shape;
    if (kind == DPSGD_MODEL_LSQ) {
        if (ndims != 1) return fail(c, DPSGD_ERR_ARG, "least squares takes dims = {d}");
        want = dims[0];
    } else if (kind == DPSGD_MODEL_LOGISTIC) {
        if (ndims != 1) return fail(c, DPSGD_ERR_ARG, "logistic regression takes dims = {d}");
        want = (int64_t)dims[0] + 1;
    } else if (kind == DPSGD_MODEL_MLP) {
        if (ndims < 2 || ndims - 1 > kMaxLayers)
            return fail(c, DPSGD_ERR_UNSUPPORTED, "MLP needs 1..8 weight layers");
        shape.nlayers = ndims - 1;
        for (int t = 0; t < ndims; ++t) shape.dims[t] = dims[t];
        for (int l = 0; l < shape.nlayers; ++l) {
            shape.w_off[l] = want; want += (int64_t)dims[l + 1] * dims[l];
            shape.b_off[l] = want; want += dims[l + 1];
        }
    } else {
        return fail(c, DPSGD_ERR_ARG, "unknown model kind");
    }
    if (want != c->N) {
        char buf[128];
        snprintf(buf, sizeof buf, "model has %lld parameters but the context was created with N = %lld",
                 (long long)want, (long long)c->N);
        return fail(c, DPSGD_ERR_ARG, buf);
    }
    const dpsgd_status pending = c->bound ? collect_device_status(c) : DPSGD_OK;
    if (pending != DPSGD_OK) return pending;
    drop_graph(c);
    cudaFree(c->d_idx); cudaFree(c->d_coef); cudaFree(c->d_act); cudaFree(c->d_delta); cudaFree(c->d_stream_parts);
    cudaFree(c->d_node_batch);
    c->d_idx = nullptr; c->d_coef = nullptr; c->d_act = nullptr; c->d_delta = nullptr; c->d_stream_parts = nullptr;
    c->d_node_batch = nullptr;             // per-node sizes belong to the model they were set for
    c->model = kind; c->d = dims[0]; c->batch = batch; c->l2 = l2_lambda; c->mlp = shape;
    c->mlp_precision = mlp_precision;
    cudaError_t e = cudaMalloc(&c->d_idx, sizeof(int32_t) * (size_t)c->n * batch);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_coef, sizeof(float) * (size_t)c->n * batch);
    if (e == cudaSuccess && kind == DPSGD_MODEL_MLP) {
        c->act_floats = mlp_act_floats(c);
        c->delta_floats = mlp_delta_floats(c);
        e = cudaMalloc(&c->d_act, sizeof(float) * c->act_floats);
        if (e == cudaSuccess) e = cudaMalloc(&c->d_delta, sizeof(float) * c->delta_floats);
        int sms = 0;
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
        c->stream_parts_floats = mlp_stream_parts_floats(sms);
        if (e == cudaSuccess) e = cudaMalloc(&c->d_stream_parts, sizeof(float) * c->stream_parts_floats);
    }
    if (e != cudaSuccess) { c->model = -1; return cuda_fail(c, e, "dpsgd_set_model allocation"); }
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_set_data(dpsgd_ctx* c, const float* A, const void* y, int64_t m, int32_t d) {
    if (!c) return DPSGD_ERR_ARG;
    if (c->model < 0) return fail(c, DPSGD_ERR_STATE, "call dpsgd_set_model before dpsgd_set_data");
    if (!A || !y) return fail(c, DPSGD_ERR_ARG, "data pointer is NULL");
    if (m < 1 || m >= (int64_t(1) << 31)) return fail(c, DPSGD_ERR_ARG, "m_per_node must be in [1, 2^31)");
    if (d != c->d) return fail(c, DPSGD_ERR_ARG, "d does not match the model's input width");
    if (!aligned(A, 16) || !aligned(y, 16)) return fail(c, DPSGD_ERR_ALIGN, "A and y must be 16-byte aligned");
    drop_graph(c);
    c->A = A; c->y = y; c->m = m; c->have_data = true;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_sample(dpsgd_ctx* c, uint64_t k, int32_t* idx) {
    if (!c) return DPSGD_ERR_ARG;
    if (!idx) return fail(c, DPSGD_ERR_ARG, "idx is NULL");
    if (c->model < 0 || !c->have_data) return fail(c, DPSGD_ERR_STATE, "model and data must be set");
    cudaError_t e = launch_sample(c, k, idx);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "sample kernel");
}

DPSGD_API dpsgd_status dpsgd_grad(dpsgd_ctx* c, uint64_t k) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if ((s = need_model(c)) != DPSGD_OK) return s;
    cudaError_t e = run_grad(c, k);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "gradient kernels");
}

DPSGD_API dpsgd_status dpsgd_mix_update(dpsgd_ctx* c) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    cudaError_t e = run_mix(c);
    if (e != cudaSuccess) return cuda_fail(c, e, "mix_update kernel");
    c->cur ^= 1;
    return DPSGD_OK;
}

// Gossip step that also leaves the consensus distance of the new X in *out_dev.
dpsgd_status mix_with_consensus(dpsgd_ctx* c, double* out_dev) {
    const float* X = c->X[c->cur];
    float* Xn = c->X[c->cur ^ 1];
    const bool fused = c->mix_kind == DPSGD_MIX_RING || c->mix_kind == DPSGD_MIX_UNIFORM_DENSE;
    const bool small = !c->kind_forced && mix_is_small(c);
    cudaError_t e;
    if (fused) {
        e = launch_mix_variant(c, X, c->G, Xn, c->swapped, out_dev, c->V);   // V, when set, updated in the pass
    } else if (c->mix_kind == DPSGD_MIX_TILED_CSR && !small) {
        // any sparse W on the tile-staging kernel: the statistics come from the rows it has in registers
        const float* D = nullptr;
        e = step_direction(c, &D);
        if (e == cudaSuccess) e = launch_mix_tiled(c, X, D, Xn, out_dev);
    } else {                                // no fused kernel for this W: mix, then one pass over the new X
        e = run_mix(c);
        if (e == cudaSuccess) e = launch_consensus(c, Xn, out_dev);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "mix_update with consensus");
    c->cur ^= 1;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_set_order(dpsgd_ctx* c, int32_t update_then_mix) {
    if (!c) return DPSGD_ERR_ARG;
    drop_graph(c);
    c->swapped = update_then_mix != 0;
    return DPSGD_OK;
}

namespace {
dpsgd_status local_step(dpsgd_ctx* c, uint64_t k, const int32_t* active_dev) {
    cudaError_t e = run_grad(c, k);
    const float* D = nullptr;
    if (e == cudaSuccess) e = step_direction(c, &D, active_dev);
    if (e == cudaSuccess) e = launch_local_update(c, c->X[c->cur], D, active_dev);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "local step");
}
}  // namespace

DPSGD_API dpsgd_status dpsgd_local_step(dpsgd_ctx* c, uint64_t k) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if ((s = need_model(c)) != DPSGD_OK) return s;
    return local_step(c, k, nullptr);
}

DPSGD_API dpsgd_status dpsgd_local_step_nodes(dpsgd_ctx* c, uint64_t k, const int32_t* active_host) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if ((s = need_model(c)) != DPSGD_OK) return s;
    if (!active_host) return fail(c, DPSGD_ERR_ARG, "active_host is NULL");
    if (c->n > 65535) return fail(c, DPSGD_ERR_UNSUPPORTED, "masked local steps need n <= 65535");
    cudaError_t e = cudaSuccess;
    if (!c->d_active) e = cudaMalloc(&c->d_active, sizeof(int32_t) * (size_t)c->n);
    // pageable source: the copy is staged before the call returns, so the caller's array is free at once
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(c->d_active, active_host, sizeof(int32_t) * (size_t)c->n, cudaMemcpyHostToDevice,
                            c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "dpsgd_local_step_nodes mask copy");
    return local_step(c, k, c->d_active);
}

DPSGD_API dpsgd_status dpsgd_set_node_batches(dpsgd_ctx* c, const int32_t* batch_host) {
    if (!c) return DPSGD_ERR_ARG;
    if (c->model < 0) return fail(c, DPSGD_ERR_STATE, "call dpsgd_set_model before dpsgd_set_node_batches");
    drop_graph(c);
    cudaError_t e = cudaSuccess;
    const dpsgd_status pending = collect_device_status(c);   // waits: kernels in flight may still read the old sizes
    if (pending != DPSGD_OK) return pending;
    if (!batch_host) {
        cudaFree(c->d_node_batch);
        c->d_node_batch = nullptr;
        return DPSGD_OK;
    }
    for (int i = 0; i < c->n; ++i)
        if (batch_host[i] < 1 || batch_host[i] > c->batch)
            return fail(c, DPSGD_ERR_ARG, "every per-node minibatch size must be in [1, batch]");
    if (!c->d_node_batch) e = cudaMalloc(&c->d_node_batch, sizeof(int32_t) * (size_t)c->n);
    if (e == cudaSuccess)
        e = cudaMemcpy(c->d_node_batch, batch_host, sizeof(int32_t) * (size_t)c->n, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(c->d_node_batch);
        c->d_node_batch = nullptr;
        return cuda_fail(c, e, "dpsgd_set_node_batches");
    }
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_set_momentum(dpsgd_ctx* c, float beta, float* V_dev) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    drop_graph(c);
    if (!V_dev) { c->V = nullptr; c->beta = 0.f; return DPSGD_OK; }
    if (!(beta >= 0.f && beta < 1.f)) return fail(c, DPSGD_ERR_ARG, "momentum must be in [0, 1)");
    if (!aligned(V_dev, 128)) return fail(c, DPSGD_ERR_ALIGN, "V_dev must be 128-byte aligned");
    const uintptr_t bytes = (uintptr_t)c->n * (uintptr_t)c->ld * sizeof(float);
    const uintptr_t v = (uintptr_t)V_dev, p[3] = {(uintptr_t)c->X[0], (uintptr_t)c->X[1], (uintptr_t)c->G};
    for (int a = 0; a < 3; ++a)
        if (v < p[a] + bytes && p[a] < v + bytes) return fail(c, DPSGD_ERR_ARG, "V_dev overlaps a bound buffer");
    c->V = V_dev; c->beta = beta;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_mix_update_consensus(dpsgd_ctx* c, double* out_dev) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!out_dev) return fail(c, DPSGD_ERR_ARG, "consensus_out_dev is NULL");
    if (!aligned(out_dev, 8)) return fail(c, DPSGD_ERR_ALIGN, "consensus_out_dev must be 8-byte aligned");
    return mix_with_consensus(c, out_dev);
}

DPSGD_API dpsgd_status dpsgd_step_consensus(dpsgd_ctx* c, uint64_t k, double* out_dev) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if ((s = need_model(c)) != DPSGD_OK) return s;
    if (!out_dev) return fail(c, DPSGD_ERR_ARG, "consensus_out_dev is NULL");
    if (!aligned(out_dev, 8)) return fail(c, DPSGD_ERR_ALIGN, "consensus_out_dev must be 8-byte aligned");
    if (c->fuse_step && fused_step_supported(c)) {
        // the iteration with the gossip step inside the gradient kernels, then one pass over the new X:
        // cheaper than writing G for the mixing kernel that accumulates the distance on the way
        const float* X = c->X[c->cur];
        float* Xn = c->X[c->cur ^ 1];
        cudaError_t e = prepare_fused_source(c, X);
        if (e == cudaSuccess) e = launch_grad_mlp(c, k, X, c->G, Xn);
        if (e != cudaSuccess) { c->fsrc_X = nullptr; return cuda_fail(c, e, "gradient kernels"); }
        if (c->fused_blocks.empty()) { c->fsrc_X = nullptr; return mix_with_consensus(c, out_dev); }
        e = launch_mix_rest(c, X, c->G, Xn);
        c->fsrc_X = nullptr;
        if (e == cudaSuccess) e = launch_consensus(c, Xn, out_dev);
        if (e != cudaSuccess) return cuda_fail(c, e, "mix_update with consensus");
        c->cur ^= 1;
        return DPSGD_OK;
    }
    cudaError_t e = run_grad(c, k);
    if (e != cudaSuccess) return cuda_fail(c, e, "gradient kernels");
    return mix_with_consensus(c, out_dev);
}

}  // extern "C"

namespace {
// Fused iteration with W = w 1 1^T (more entries per row than the kernels gather): the column mean is
// formed once (one pass over X) and the kernels gather from it as from a one-row matrix.  Sets or
// clears the source the fused kernels read; allocates the small buffer on first use.
cudaError_t prepare_fused_source(dpsgd_ctx* c, const float* X) {
    c->fsrc_X = nullptr;
    if (!(c->can_uniform && c->W.max_deg > kFusedMaxDegree)) return cudaSuccess;
    const size_t mean_bytes = sizeof(float) * (size_t)c->ld;
    if (!c->d_mean_blob || c->mean_ld != c->ld) {
        cudaFree(c->d_mean_blob);
        c->d_mean_blob = nullptr;
        const size_t total = mean_bytes + sizeof(int32_t) * (2 * (size_t)c->n + 1) + sizeof(float) * (size_t)c->n;
        cudaError_t e = cudaMalloc(&c->d_mean_blob, total);
        if (e != cudaSuccess) return e;
        std::vector<int32_t> rp((size_t)c->n + 1), col((size_t)c->n, 0);
        std::vector<float> one((size_t)c->n, 1.f);
        for (int i = 0; i <= c->n; ++i) rp[i] = i;
        char* b = static_cast<char*>(c->d_mean_blob) + mean_bytes;
        e = cudaMemcpy(b, rp.data(), sizeof(int32_t) * rp.size(), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(b + sizeof(int32_t) * rp.size(), col.data(), sizeof(int32_t) * col.size(), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(b + sizeof(int32_t) * (rp.size() + col.size()), one.data(), sizeof(float) * one.size(), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { cudaFree(c->d_mean_blob); c->d_mean_blob = nullptr; return e; }
        c->mean_ld = c->ld;
    }
    float* mean = static_cast<float*>(c->d_mean_blob);
    cudaError_t e = launch_average(c, X, mean);
    if (e != cudaSuccess) return e;
    char* b = static_cast<char*>(c->d_mean_blob) + mean_bytes;
    c->fsrc_X = mean; c->fsrc_ld = 0;
    c->fsrc_row_ptr = reinterpret_cast<const int32_t*>(b);
    c->fsrc_col = c->fsrc_row_ptr + c->n + 1;
    c->fsrc_val = reinterpret_cast<const float*>(c->fsrc_col + c->n);
    return cudaSuccess;
}
}  // namespace

extern "C" {

DPSGD_API dpsgd_status dpsgd_set_fused_step(dpsgd_ctx* c, int32_t on) {
    if (!c) return DPSGD_ERR_ARG;
    drop_graph(c);
    if (on < 0 || on > 3) return fail(c, DPSGD_ERR_ARG, "mode must be 0, 1, 2 or 3");
    c->fuse_step = on;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_step(dpsgd_ctx* c, uint64_t k) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if ((s = need_model(c)) != DPSGD_OK) return s;
    if (c->fuse_step && fused_step_supported(c)) {
        // the weight-gradient kernels write their blocks of X_next themselves; the remaining columns
        // (biases, blocks on other kernels, padding) take the gossip step from G afterwards
        const float* X = c->X[c->cur];
        float* Xn = c->X[c->cur ^ 1];
        cudaError_t e = prepare_fused_source(c, X);
        if (e == cudaSuccess) e = launch_grad_mlp(c, k, X, c->G, Xn);
        if (e != cudaSuccess) { c->fsrc_X = nullptr; return cuda_fail(c, e, "gradient kernels"); }
        e = c->fused_blocks.empty() ? run_mix(c) : launch_mix_rest(c, X, c->G, Xn);
        c->fsrc_X = nullptr;
        if (e != cudaSuccess) return cuda_fail(c, e, "mix_update kernel");
        c->cur ^= 1;
        return DPSGD_OK;
    }
    if (c->fuse_step && linear_step_fuses(c)) {
        // linear model with wide rows on a small matrix: the reduction of the gradient shares and the
        // gossip step in one launch (G is written as well)
        cudaError_t e = launch_linear_step(c, k, c->X[c->cur], c->G, c->X[c->cur ^ 1]);
        if (e != cudaSuccess) return cuda_fail(c, e, "gradient and mix_update kernels");
        c->cur ^= 1;
        return DPSGD_OK;
    }
    cudaError_t e = run_grad(c, k);
    if (e != cudaSuccess) return cuda_fail(c, e, "gradient kernels");
    e = run_mix(c);
    if (e != cudaSuccess) return cuda_fail(c, e, "mix_update kernel");
    c->cur ^= 1;
    return DPSGD_OK;
}

// Captures kGraphChain iterations (an even number: the X buffers swap back) that read the iteration number from
// device memory and advance it, so that one graph can be replayed for any k.  A longer chain means fewer graph
// launches, whose boundaries cost more than the dependency between two kernels inside a graph.
constexpr int kGraphChain = 16;
dpsgd_status capture_pair(dpsgd_ctx* c) {
    cudaError_t e = cudaSuccess;
    if (!c->d_k) e = cudaMalloc(&c->d_k, 2 * sizeof(uint64_t));
    if (e != cudaSuccess) return cuda_fail(c, e, "iteration counter");
    // record on a private stream (the bound one may be the legacy default stream, which cannot
    // capture); the instantiated graph is launched on the bound stream
    if (!c->capture_stream) e = cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) return cuda_fail(c, e, "capture stream");
    const int cur0 = c->cur;
    const int64_t launches0 = c->launches;
    cudaStream_t bound_stream = c->stream;
    e = cudaStreamBeginCapture(c->capture_stream, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return cuda_fail(c, e, "begin capture");
    c->stream = c->capture_stream;
    // The one-launch step kernel reads the iteration number from its slot and leaves k + 2 there for the launch
    // after next; consecutive iterations alternate between the two slots (set to k and k + 1 before the replay),
    // need no counter kernel and can be programmatic dependents of one another.  Every other path reads slot 0
    // and a one-thread kernel advances it.
    const bool self = c->fuse_step && linear_node_step_fuses(c);
    dpsgd_status s = DPSGD_OK;
    for (int t = 0; t < kGraphChain && s == DPSGD_OK; ++t) {
        c->k_dev_active = c->d_k + (self ? (t & 1) : 0);
        c->k_dev_next = self ? c->d_k + (t & 1) : nullptr;
        c->chain_pos = t;
        s = dpsgd_step(c, 0);
        if (!self && s == DPSGD_OK && launch_advance_k(c) != cudaSuccess) s = DPSGD_ERR_CUDA;
    }
    c->k_dev_active = nullptr;
    c->k_dev_next = nullptr;
    c->chain_pos = 0;
    c->stream = bound_stream;
    cudaGraph_t graph = nullptr;
    e = cudaStreamEndCapture(c->capture_stream, &graph);
    c->cur = cur0;                                // nothing ran: the capture only recorded
    c->graph_launches = c->launches - launches0;
    c->launches = launches0;
    if (s != DPSGD_OK || e != cudaSuccess || !graph) {
        if (graph) cudaGraphDestroy(graph);
        return s != DPSGD_OK ? s : cuda_fail(c, e, "end capture");
    }
    e = cudaGraphInstantiate(&c->graph_exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) { c->graph_exec = nullptr; return cuda_fail(c, e, "graph instantiate"); }
    c->graph_cur = cur0;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_run(dpsgd_ctx* c, uint64_t k_first, int64_t iterations) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if ((s = need_model(c)) != DPSGD_OK) return s;
    if (iterations < 0) return fail(c, DPSGD_ERR_ARG, "iterations must be >= 0");
    int64_t t = 0;
    // Launch-bound sizes only: replay a captured chain of iterations.  The first two iterations always
    // run directly, which also completes any first-use set-up before a capture starts.
    // (rows of 4 KB and more make the gradient kernels long enough to hide the launches: replay measured
    // slower there, 29 against 24 us per iteration on the 4096-feature logistic configuration)
    const bool small = mix_is_small(c) && c->model != DPSGD_MODEL_MLP && c->d < 1024 && iterations >= 2 * kGraphChain;
    if (small) {
        for (; t < 2; ++t)
            if ((s = dpsgd_step(c, k_first + (uint64_t)t)) != DPSGD_OK) return s;
        if (!c->graph_exec && capture_pair(c) != DPSGD_OK) drop_graph(c);
        if (c->graph_exec) {
            if (c->cur != c->graph_cur) {           // bring the buffer parity to the captured one
                if ((s = dpsgd_step(c, k_first + (uint64_t)t)) != DPSGD_OK) return s;
                ++t;
            }
            cudaError_t e = launch_set_k(c, k_first + (uint64_t)t);
            for (; e == cudaSuccess && t + kGraphChain <= iterations; t += kGraphChain) {
                e = cudaGraphLaunch(c->graph_exec, c->stream);
                c->launches += c->graph_launches;
            }
            if (e != cudaSuccess) return cuda_fail(c, e, "graph replay");
        }
    }
    for (; t < iterations; ++t)
        if ((s = dpsgd_step(c, k_first + (uint64_t)t)) != DPSGD_OK) return s;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_consensus_dist(dpsgd_ctx* c, double* out) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!out) return fail(c, DPSGD_ERR_ARG, "out_host is NULL");
    cudaError_t e = launch_consensus(c, c->X[c->cur], &c->d_result->value);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(c->h_result, c->d_result, sizeof(ResultBlock), cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "consensus distance");
    *out = c->h_result->value;
    if (c->h_result->status != 0) {
        c->h_result->status = 0;
        cudaMemsetAsync(&c->d_result->status, 0, sizeof(int), c->stream);
        return fail(c, DPSGD_ERR_TIMEOUT,
                    "a kernel gave up waiting for a tile copy since the last synchronising call; X is not valid");
    }
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_sync(dpsgd_ctx* c) {
    if (!c) return DPSGD_ERR_ARG;
    return collect_device_status(c);
}

DPSGD_API dpsgd_status dpsgd_selftest_wait(dpsgd_ctx* c, uint32_t max_polls) {
    if (!c) return DPSGD_ERR_ARG;
    if (max_polls < 1 || max_polls > (1u << 20)) return fail(c, DPSGD_ERR_ARG, "max_polls must be in [1, 2^20]");
    cudaError_t e = launch_wait_probe(c, max_polls);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "wait probe kernel");
}

DPSGD_API dpsgd_status dpsgd_conv3x3_forward(dpsgd_ctx* c, const float* in_dev, int32_t batch, int32_t c_in, int32_t h,
                                             int32_t w, int32_t c_out, int32_t stride, int64_t w_off, int64_t b_off,
                                             int32_t relu, float* out_dev) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!in_dev || !out_dev) return fail(c, DPSGD_ERR_ARG, "in_dev or out_dev is NULL");
    if (!aligned(in_dev, 16) || !aligned(out_dev, 16)) return fail(c, DPSGD_ERR_ALIGN, "in_dev and out_dev must be 16-byte aligned");
    if (const char* why = conv3x3_forward_unsupported(batch, c_in, h, w, c_out, stride)) return fail(c, DPSGD_ERR_UNSUPPORTED, why);
    const int64_t wsz = (int64_t)c_out * c_in * 9;
    if (w_off < 0 || b_off < 0 || w_off + wsz > c->N || b_off + c_out > c->N)
        return fail(c, DPSGD_ERR_ARG, "filter or bias block lies outside the parameter row");
    const char* why = nullptr;
    cudaError_t e = launch_conv3x3_forward(c, in_dev, batch, c_in, h, w, c_out, stride, w_off, b_off, relu, out_dev, &why);
    if (e == cudaErrorNotSupported && why) return fail(c, DPSGD_ERR_UNSUPPORTED, why);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "convolution kernel");
}

DPSGD_API dpsgd_status dpsgd_conv3x3_backward(dpsgd_ctx* c, const float* in_dev, const float* out_dev,
                                              const float* dout_dev, int32_t batch, int32_t c_in, int32_t h, int32_t w,
                                              int32_t c_out, int32_t stride, int64_t w_off, int64_t b_off, int32_t relu,
                                              float* din_dev) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!in_dev || !dout_dev || (relu && !out_dev)) return fail(c, DPSGD_ERR_ARG, "in_dev, dout_dev (and out_dev of a ReLU layer) must not be NULL");
    if (!aligned(in_dev, 16) || !aligned(dout_dev, 16) || !aligned(out_dev, 16) || !aligned(din_dev, 16))
        return fail(c, DPSGD_ERR_ALIGN, "activation and gradient buffers must be 16-byte aligned");
    if (batch < 1 || c_in < 1 || h < 1 || w < 1 || c_out < 1) return fail(c, DPSGD_ERR_ARG, "sizes must be positive");
    if (stride != 1 && stride != 2) return fail(c, DPSGD_ERR_UNSUPPORTED, "stride must be 1 or 2");
    const int64_t wsz = (int64_t)c_out * c_in * 9;
    if (w_off < 0 || b_off < 0 || w_off + wsz > c->N || b_off + c_out > c->N)
        return fail(c, DPSGD_ERR_ARG, "filter or bias block lies outside the parameter row");
    const char* why = nullptr;
    cudaError_t e = launch_conv3x3_backward(c, in_dev, out_dev, dout_dev, batch, c_in, h, w, c_out, stride, w_off, b_off,
                                            relu, din_dev, &why);
    if (e == cudaErrorNotSupported && why) return fail(c, DPSGD_ERR_UNSUPPORTED, why);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "convolution backward kernels");
}

DPSGD_API dpsgd_status dpsgd_average(dpsgd_ctx* c, float* xbar) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!xbar) return fail(c, DPSGD_ERR_ARG, "xbar_dev is NULL");
    if (!aligned(xbar, 16)) return fail(c, DPSGD_ERR_ALIGN, "xbar_dev must be 16-byte aligned");
    cudaError_t e = launch_average(c, c->X[c->cur], xbar);
    return e == cudaSuccess ? DPSGD_OK : cuda_fail(c, e, "average kernel");
}

DPSGD_API dpsgd_status dpsgd_mix_update_host(dpsgd_ctx* c, const float* G_host, int64_t ld_host, double* out) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!G_host || !out) return fail(c, DPSGD_ERR_ARG, "G_host or consensus_out_host is NULL");
    if (ld_host < c->N) return fail(c, DPSGD_ERR_ARG, "ld_host < N");
    cudaError_t e = cudaMemcpy2DAsync(c->G, sizeof(float) * c->ld, G_host, sizeof(float) * ld_host,
                                      sizeof(float) * c->N, c->n, cudaMemcpyHostToDevice, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "copy of G to the device");
    if ((s = dpsgd_mix_update(c)) != DPSGD_OK) return s;
    return dpsgd_consensus_dist(c, out);
}

DPSGD_API dpsgd_status dpsgd_current(dpsgd_ctx* c, float** X_cur) {
    dpsgd_status s = need_bound(c);
    if (s != DPSGD_OK) return s;
    if (!X_cur) return fail(c, DPSGD_ERR_ARG, "X_cur_dev is NULL");
    *X_cur = c->X[c->cur];
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_set_gamma(dpsgd_ctx* c, float gamma) {
    if (!c) return DPSGD_ERR_ARG;
    if (!(gamma == gamma)) return fail(c, DPSGD_ERR_ARG, "gamma is NaN");
    drop_graph(c);
    c->gamma = gamma;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_mix_kind(dpsgd_ctx* c, int32_t force, int32_t* kind_out) {
    if (!c) return DPSGD_ERR_ARG;
    if (force >= 0) {
        const bool ok = (force == DPSGD_MIX_RING && c->can_ring) ||
                        (force == DPSGD_MIX_UNIFORM_DENSE && c->can_uniform) ||
                        (force == DPSGD_MIX_TILED_CSR && c->can_tiled) ||
                        force == DPSGD_MIX_GATHER_CSR;
        if (!ok) return fail(c, DPSGD_ERR_UNSUPPORTED, "this W cannot use the requested mixing kernel");
        drop_graph(c);
        c->mix_kind = force;
        c->kind_forced = true;
    }
    if (kind_out) *kind_out = c->mix_kind;
    return DPSGD_OK;
}

DPSGD_API dpsgd_status dpsgd_launch_count(dpsgd_ctx* c, int64_t* count_out) {
    if (!c || !count_out) return DPSGD_ERR_ARG;
    *count_out = c->launches;
    return DPSGD_OK;
}

DPSGD_API const char* dpsgd_last_error(dpsgd_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

}  // extern "C"
