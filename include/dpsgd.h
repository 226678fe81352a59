/*
 * dpsgd.h - C ABI of the B200 D-PSGD library (libdpsgd.so).
 *
 * D-PSGD (Lian et al., "Can Decentralized Algorithms Outperform Centralized Algorithms?",
 * arXiv 1705.09056) simulated for n nodes on ONE GPU.  The n local models x_{k,i} are the
 * rows of an n x ld fp32 matrix X (the paper's X_k in R^{N x n} of Section 3, stored
 * transposed; W is symmetric, so X_k W becomes W X).  One iteration k of Algorithm 1 is
 *
 *     xi_{k,i}  <- minibatch of B indices into node i's local data        (step 2)
 *     g_i       <- (1/B) sum_b grad F(x_{k,i}; sample_b)                   (step 3, footnote a)
 *     x_{k+1,i} <- sum_j W_ij x_{k,j} - gamma g_i                          (steps 4-5)
 *
 * i.e. the global form X_{k+1} = X_k W - gamma dF(X_k; xi_k) of Section 3.
 *
 * Conventions
 *  - Every function returns a dpsgd_status; nothing throws, aborts or traps.
 *    dpsgd_last_error() gives a human-readable message for the last failure on a context.
 *  - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global memory of the
 *    current device.  Big buffers (X, G, the dataset) are owned by the CALLER and must stay
 *    alive while bound; the library owns only small internals (CSR copy, index and activation
 *    scratch, reduction partials), released by dpsgd_destroy().
 *  - All work is enqueued on the stream given to dpsgd_bind(); calls return without waiting
 *    unless stated otherwise.  Calls on one context must not overlap in time.
 *  - There is no CPU fallback: without a CUDA device every compute call fails with
 *    DPSGD_ERR_CUDA.
 *  - Device code never traps.  The kernels that wait for tile copies (the tiled gossip kernel, the
 *    tensor-core gradient kernels) bound every wait; a wait that runs out raises a status word in
 *    device memory, the CTA skips its tile and returns, and the NEXT call that waits for the
 *    stream reports DPSGD_ERR_TIMEOUT once and clears the word: dpsgd_sync, dpsgd_consensus_dist,
 *    dpsgd_mix_update_host, dpsgd_set_model, dpsgd_set_node_batches, dpsgd_destroy.  X is not
 *    valid after such a report.  The asynchronous calls (dpsgd_step, dpsgd_mix_update, ...)
 *    cannot see it; end a run with dpsgd_sync before trusting X.
 *
 * Stacked layout: row i of X / G starts at element i*ld; ld >= N, ld a multiple of 32 floats
 * (128 bytes), base pointers 128-byte aligned.  Padding columns [N, ld) must be zero in X and
 * G on entry; they stay zero (rows of W sum to one, applied to zeros).
 */
#ifndef DPSGD_H_
#define DPSGD_H_

#include <stdint.h>

#if defined(__GNUC__)
#define DPSGD_API __attribute__((visibility("default")))
#else
#define DPSGD_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dpsgd_ctx dpsgd_ctx; /* opaque, library-owned */

typedef enum dpsgd_status {
    DPSGD_OK = 0,
    DPSGD_ERR_ARG = 1,         /* null pointer, non-positive size, value out of range           */
    DPSGD_ERR_W_INVALID = 2,   /* W is not a symmetric doubly stochastic matrix in sorted CSR    */
    DPSGD_ERR_ALIGN = 3,       /* pointer or leading dimension not aligned as required           */
    DPSGD_ERR_STATE = 4,       /* call made before the buffers / model / data it needs were set  */
    DPSGD_ERR_UNSUPPORTED = 5, /* shape outside what the kernels handle                          */
    DPSGD_ERR_CUDA = 6,        /* a CUDA runtime call or kernel launch failed                    */
    DPSGD_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up (status word set by kernel) */
} dpsgd_status;

enum { DPSGD_MODEL_LSQ = 0, DPSGD_MODEL_LOGISTIC = 1, DPSGD_MODEL_MLP = 2 };

/* Mixing kernel chosen from the structure of W (reported by dpsgd_mix_kind). */
enum {
    DPSGD_MIX_RING = 0,          /* circulant tridiagonal band (Theorem 3's ring)               */
    DPSGD_MIX_UNIFORM_DENSE = 1, /* all n*n entries equal (W = 1 1^T / n, the C-PSGD average)   */
    DPSGD_MIX_TILED_CSR = 2,     /* any sparse W: column tiles of all n rows staged on chip      */
    DPSGD_MIX_GATHER_CSR = 3     /* any W: neighbour rows gathered through the caches            */
};

/*
 * Inputs of Algorithm 1 (its step length gamma and weight matrix W): creates a context
 * for n nodes with N parameters each.  W comes as host CSR (row_ptr[n+1], col_idx[nnz],
 * val[nnz]); it is validated against Section 3's definition and copied:
 *   square; column indices in range, strictly increasing inside a row; 0 <= W_ij <= 1;
 *   W_ij == W_ji exactly; |sum_j W_ij - 1| <= 1e-6 for every row.
 * Otherwise DPSGD_ERR_W_INVALID and *out = NULL (nothing is left allocated).
 * seed keys the minibatch sampler.  Limits: 1 <= n <= 65535, 1 <= N < 2^40.
 */
DPSGD_API dpsgd_status dpsgd_create(dpsgd_ctx** out, int32_t n, int64_t N, const int32_t* row_ptr_host,
                          const int32_t* col_idx_host, const float* val_host, float gamma,
                          uint64_t seed);

/* Releases the context and its internal device memory.  Caller-owned buffers are untouched. */
DPSGD_API dpsgd_status dpsgd_destroy(dpsgd_ctx* ctx);

/*
 * Binds the caller's device buffers: X0 holds X_k now, X1 receives X_{k+1} (they swap roles
 * each mix_update), G holds the stochastic gradients dF(X_k; xi_k) (Section 3).  All three are
 * n x ld fp32, 128-byte aligned, distinct and non-overlapping.  cuda_stream is a cudaStream_t
 * (NULL = legacy default stream).  May be called again to rebind.
 */
DPSGD_API dpsgd_status dpsgd_bind(dpsgd_ctx* ctx, float* X0_dev, float* X1_dev, float* G_dev, int64_t ld,
                        void* cuda_stream);

/*
 * Chooses F of Eq. (1)/(2).  dims/ndims:
 *   DPSGD_MODEL_LSQ      dims = {d}: F = 1/2 (a.x - y)^2,                       N = d
 *   DPSGD_MODEL_LOGISTIC dims = {d}: F = log(1+exp(-y(a.w+b))) + l2/2 |w|^2,    N = d+1, x=[w|b]
 *   DPSGD_MODEL_MLP      dims = {d_0,...,d_L}: ReLU layers, softmax cross-entropy,
 *                        x = [W_1 (d_1 x d_0 row-major) | b_1 | W_2 | b_2 ...], N = sum
 * batch = minibatch size B per node (footnote a of Algorithm 1; gradients are the MEAN over
 * the minibatch).  N must match the context's N.  Allocates the activation scratch.
 * mlp_precision (MLP only): 0 = fp32-faithful on the tensor cores (each product as three TF32
 * MMAs on split operands; minibatches above 128 use the fp32 FMA kernel), 1 = one TF32 MMA per
 * product (faster, about 1e-3 relative on G), 2 = fp32 FMA kernel always.
 */
DPSGD_API dpsgd_status dpsgd_set_model(dpsgd_ctx* ctx, int32_t kind, const int32_t* dims_host,
                             int32_t ndims, float l2_lambda, int32_t batch,
                             int32_t mlp_precision);

/*
 * Local data of the n nodes (Section 3, Strategy 1/2): A_dev is fp32 [n][m_per_node][d],
 * y_dev is fp32 [n][m_per_node] (targets, or labels +-1) for the linear models and int32
 * [n][m_per_node] class ids for the MLP.  Caller-owned, 16-byte aligned, d = dims[0].
 */
DPSGD_API dpsgd_status dpsgd_set_data(dpsgd_ctx* ctx, const float* A_dev, const void* y_dev,
                            int64_t m_per_node, int32_t d);

/*
 * Algorithm 1 step 2 on its own (test hook): writes the indices xi_{k,i} of iteration k,
 * int32 [n][B] on the device.  Draw b of node i is word (b mod 4) of Philox4x32-10 with
 * counter (b div 4, i, k_lo, k_hi) and key (seed_lo, seed_hi), mapped to
 * floor(u * m_per_node / 2^32): i.i.d. uniform with replacement.
 */
DPSGD_API dpsgd_status dpsgd_sample(dpsgd_ctx* ctx, uint64_t k, int32_t* idx_dev);

/* Algorithm 1 steps 2-3 for all nodes: G <- dF(X_k; xi_k), gradients at the nodes' own rows. */
DPSGD_API dpsgd_status dpsgd_grad(dpsgd_ctx* ctx, uint64_t k);

/*
 * Algorithm 1 steps 4-5 fused, one pass over HBM: X_next <- W X_cur - gamma G, then the two X
 * buffers swap roles.  Reads X and G once and writes X_next once (12 bytes per
 * replica-parameter).
 */
DPSGD_API dpsgd_status dpsgd_mix_update(dpsgd_ctx* ctx);

/*
 * Footnote c of Algorithm 1: with update_then_mix != 0 every later gossip step first applies the
 * local gradient and then averages, X_next <- W (X_cur - gamma G); 0 restores the printed order.
 * With W = 1 1^T / n the swapped order is exactly centralized minibatch SGD on every row.
 */
DPSGD_API dpsgd_status dpsgd_set_order(dpsgd_ctx* ctx, int32_t update_then_mix);

/*
 * Algorithm 1 steps 3-5 in one pass for the MLP: with mode != 0, dpsgd_step() applies the gossip step
 * X_next <- W X_cur - gamma dF(X_cur; xi) (Section 3) inside the kernels that form the weight
 * gradients, tile by tile while the gradient is on chip.  Those blocks of the gradient are never
 * written: per parameter the iteration moves 8 bytes through HBM (read X, write X_next) instead of 16
 * (write G, then read X and G and write X_next).  After such a step the fused weight blocks of G hold
 * old values; biases, and blocks whose product runs on another kernel, are still written to G and
 * take the gossip step from there.  The result equals dpsgd_grad + dpsgd_mix_update up to fp32
 * rounding order.
 *   mode 0  off: two stages.
 *   mode 1  (default) fused for the weight blocks where it is faster on B200: a ring W (Theorem 3)
 *           and a stacked block of at least 64 MB, or rows of W with at most 3 entries and a stacked
 *           block of at least 512 MB (far beyond L2); other blocks in two stages.
 *   mode 2  fused for every block a fused kernel can take.  A ring W takes the kernel that keeps the
 *           tiles of X_{i-1} and X_i on chip while it walks the nodes (X is read once); any other W
 *           the kernel that gathers the neighbours' tiles through L2.
 *   mode 3  as mode 2, but the gathering kernel for a ring W too (for comparison).
 * The kernel applies when the model is the MLP on the tensor-core path (minibatch <= 64, layer input
 * widths multiples of 4), the printed order of Algorithm 1 is in force, no momentum is set and either no
 * row of W has more than 8 entries or W is the averaging matrix 1 1^T / n (its rows all mix to the column
 * mean, formed once per iteration); otherwise dpsgd_step() runs the two stages whatever the mode.
 * dpsgd_grad, dpsgd_mix_update and the other entry points are not affected.
 * The linear models have a small counterpart under any mode but 0: with data rows of 4 to 16 KB and
 * a stacked matrix of at most 8 MB, dpsgd_step() adds up the gradient's per-group shares and applies
 * the gossip step in one launch (G is still written in full there).
 */
DPSGD_API dpsgd_status dpsgd_set_fused_step(dpsgd_ctx* ctx, int32_t mode);

/*
 * A local iteration without communication (Section 5.3, last paragraph: a node may run more than
 * one minibatch before it synchronises): samples xi_{k,i}, computes g_i at x_{k,i} and updates
 * x_i <- x_i - gamma g_i in place (the gossip step with W = I), momentum included when set.  Call it
 * tau - 1 times with distinct k between two dpsgd_step() calls for tau local steps per exchange.
 */
DPSGD_API dpsgd_status dpsgd_local_step(dpsgd_ctx* ctx, uint64_t k);

/*
 * The same local iteration for some nodes only (Section 5.3, last paragraph: with machines of
 * different speed, the faster ones may run more than one minibatch before the synchronisation).
 * active_host: host, int32 [n]; node i takes the step when active_host[i] != 0, and otherwise its
 * row of X (and of the momentum buffers) is left as it is.  The array is copied before the call
 * returns.  n <= 65535.  Errors: DPSGD_ERR_ARG (NULL), DPSGD_ERR_STATE, DPSGD_ERR_UNSUPPORTED.
 */
DPSGD_API dpsgd_status dpsgd_local_step_nodes(dpsgd_ctx* ctx, uint64_t k, const int32_t* active_host);

/*
 * Per-node minibatch sizes (Section 5.3, last paragraph: different minibatch sizes compensate for
 * machines of different speed).  batch_host: host, int32 [n], 1 <= B_i <= batch of dpsgd_set_model;
 * node i then averages its gradient over its first B_i draws of the iteration (dpsgd_sample still
 * returns all `batch` draws per node).  NULL restores the common size.  Synchronises the bound
 * stream; a later dpsgd_set_model resets the sizes.  Errors: DPSGD_ERR_ARG (a size out of range),
 * DPSGD_ERR_STATE (no model).
 */
DPSGD_API dpsgd_status dpsgd_set_node_batches(dpsgd_ctx* ctx, const int32_t* batch_host);

/*
 * Momentum as used for both algorithms in the Torch experiments (Section 5.3: learning rate 0.1,
 * momentum 0.9).  The paper prints no formula; the reading is the heavy-ball update of the
 * framework it used, kept per node: v_i <- beta v_i + g_i, then the gossip step with v_i in place
 * of g_i.  V_dev: device, fp32 [n][ld], 128-byte aligned, caller-owned, zero before the first
 * step, distinct from X0/X1/G; 0 <= beta < 1.  V_dev = NULL switches momentum off.  Call after
 * dpsgd_bind (rebinding switches it off).
 */
DPSGD_API dpsgd_status dpsgd_set_momentum(dpsgd_ctx* ctx, float beta, float* V_dev);

/*
 * dpsgd_mix_update() that also writes sum_i ||xbar - x_i||^2 of the NEW X (Theorem 4, Eq. 10) to
 * one double in device memory, asynchronously on the stream.  For ring and uniform-dense W the
 * sum is accumulated inside the gossip kernel (no second pass over HBM); otherwise a consensus
 * pass over the new X follows.  consensus_out_dev: device, 8-byte aligned, caller-owned.
 */
DPSGD_API dpsgd_status dpsgd_mix_update_consensus(dpsgd_ctx* ctx, double* consensus_out_dev);

/* dpsgd_grad(k) followed by dpsgd_mix_update_consensus(): an iteration that logs its consensus
 * distance (as the 112-node experiments of Section 5 would, per step). */
DPSGD_API dpsgd_status dpsgd_step_consensus(dpsgd_ctx* ctx, uint64_t k, double* consensus_out_dev);

/* One full iteration k of Algorithm 1: the result of dpsgd_grad(k) followed by dpsgd_mix_update().  For
 * the MLP the two stages may run as one (see dpsgd_set_fused_step: mode 1 is the default); G then does
 * not hold the whole gradient afterwards.  Call dpsgd_grad() when G itself is wanted. */
DPSGD_API dpsgd_status dpsgd_step(dpsgd_ctx* ctx, uint64_t k);

/* The loop of Algorithm 1: iterations k_first, k_first + 1, ... (dpsgd_step each), enqueued in one
 * call.  For launch-bound sizes (linear models, matrices of at most 8 MB, at least 32 iterations) a
 * chain of 16 iterations is captured once into a CUDA graph that reads the iteration number from
 * device memory, and replayed; results are identical to repeated dpsgd_step calls.  The bound
 * stream must not be used by other threads during the call. */
DPSGD_API dpsgd_status dpsgd_run(dpsgd_ctx* ctx, uint64_t k_first, int64_t iterations);

/*
 * sum_i || xbar - x_i ||^2 over the current X (sum_i Q_{k,i} of Eq. 10; divide by n for M_k
 * of Eq. 13), accumulated in fp64.  Waits for the stream and writes one double to host memory.
 */
DPSGD_API dpsgd_status dpsgd_consensus_dist(dpsgd_ctx* ctx, double* out_host);

/*
 * Waits for everything enqueued on the bound stream and reports what the device recorded meanwhile:
 * DPSGD_ERR_TIMEOUT if a kernel's bounded wait ran out since the last synchronising call (the word is
 * cleared, so the next report concerns later work), DPSGD_ERR_CUDA if the stream failed, else
 * DPSGD_OK.  The barrier of Algorithm 1 between iterations needs no such call: kernel boundaries on
 * the stream are that barrier.  Call it before reading X on another stream or trusting a run.
 */
DPSGD_API dpsgd_status dpsgd_sync(dpsgd_ctx* ctx);

/*
 * Self-test of the give-up path (no counterpart in the paper): enqueues one small CTA that waits on a
 * barrier at which nothing ever arrives, with the kernels' bounded wait cut to max_polls polls
 * (1 .. 2^20; a poll takes well under a microsecond).  The CTA then raises the status word and
 * returns; it faults nothing and holds nothing.  The next synchronising call returns
 * DPSGD_ERR_TIMEOUT, and the context stays usable.  X, G and the iteration state are not touched.
 */
DPSGD_API dpsgd_status dpsgd_selftest_wait(dpsgd_ctx* ctx, uint32_t max_polls);

/*
 * A layer of the paper's image workloads (Section 5.1: ResNet-20 on CIFAR-10; Section 5.3: a 32-layer
 * residual network): 3x3 convolution, zero padding 1, stride 1 or 2, for all nodes at once, each node with
 * the filters of its OWN current parameter row x_{k,i} (forward half of Algorithm 1 step 3 for such a model):
 *   out[i][b][o][p][q] = act( bias_i[o] + sum_{c,kh,kw} w_i[o][c][kh][kw] * in[i][b][c][stride p + kh - 1][stride q + kw - 1] )
 * with the input read as zero outside the image, act = ReLU when relu != 0, else the identity.
 *   in_dev   device, fp32 [n][batch][c_in][h][w] (NCHW per node), 16-byte aligned, caller-owned
 *   out_dev  device, fp32 [n][batch][c_out][h'][w'], h' = (h - 1) / stride + 1, w' likewise, 16-byte aligned
 *   w_off    column of the first filter weight inside a parameter row; the c_out x c_in x 3 x 3 block is
 *            row-major in (o, c, kh, kw); b_off: column of the c_out biases.  Both blocks inside [0, N).
 * Products are fp32-faithful on the tensor cores (three TF32 MMAs on split operands).  Asynchronous on the
 * bound stream.  Shapes taken: w and w' powers of two, 4 <= w <= 256, w' <= 128, h' * w' a multiple or a
 * divisor of 128, c_out a multiple of 16, c_in <= 256; otherwise DPSGD_ERR_UNSUPPORTED.
 */
DPSGD_API dpsgd_status dpsgd_conv3x3_forward(dpsgd_ctx* ctx, const float* in_dev, int32_t batch, int32_t c_in, int32_t h,
                                             int32_t w, int32_t c_out, int32_t stride, int64_t w_off, int64_t b_off,
                                             int32_t relu, float* out_dev);

/*
 * Backward of dpsgd_conv3x3_forward for the same layer, all nodes at once (gradient half of Algorithm 1 step 3
 * for the image workloads of Sections 5.1 / 5.3).  With dym = dout * [out > 0] for a ReLU layer (ReLU'(0) = 0),
 * dym = dout otherwise:
 *   G[i][b_off + o]                      <- sum_{b,p,q} dym[i][b][o][p][q]
 *   G[i][w_off + ((o c_in + c) 3 + kh) 3 + kw] <- sum_{b,p,q} dym[i][b][o][p][q] * in[i][b][c][stride p + kh - 1][stride q + kw - 1]
 *   din[i][b][c][y][x] <- sum_{o,kh,kw} w_i[o][c][kh][kw] * dym[i][b][o][p][q] over stride p + kh - 1 = y, stride q + kw - 1 = x
 * i.e. the filter and bias blocks of node i's row of the bound gradient matrix G receive SUMS over the minibatch
 * (the caller's dout carries the 1/B of a mean loss), and din (optional, NULL = not wanted) receives the
 * gradient at the layer's input.  Filters are read from the current X.
 *   in_dev / out_dev   the layer's input and its output as dpsgd_conv3x3_forward wrote it (out_dev only read for
 *                      relu != 0); dout_dev: gradient at the output, same shape as out_dev; all fp32, device,
 *                      16-byte aligned, caller-owned.
 * The contractions run on the tensor-core kernels (three TF32 MMAs per product); the library keeps a scratch
 * buffer of about (9 c_in + c_out) x the size of dout (allocated on the first call, grown when a larger layer
 * comes, released by dpsgd_destroy).  Asynchronous on the bound stream; results are bit-reproducible.
 * din needs c_in to be a multiple of 16 and the shape limits of dpsgd_conv3x3_forward on the input's size;
 * n * batch <= 65535.  Errors: DPSGD_ERR_ARG, DPSGD_ERR_ALIGN, DPSGD_ERR_UNSUPPORTED, DPSGD_ERR_CUDA.
 */
DPSGD_API dpsgd_status dpsgd_conv3x3_backward(dpsgd_ctx* ctx, const float* in_dev, const float* out_dev,
                                              const float* dout_dev, int32_t batch, int32_t c_in, int32_t h, int32_t w,
                                              int32_t c_out, int32_t stride, int64_t w_off, int64_t b_off, int32_t relu,
                                              float* din_dev);

/* Output of Algorithm 1: xbar = (1/n) sum_i x_i into xbar_dev (fp32 [ld], 16-byte aligned). */
DPSGD_API dpsgd_status dpsgd_average(dpsgd_ctx* ctx, float* xbar_dev);

/*
 * Host-buffer variant of the gossip step, for callers whose gradients live in CPU memory:
 * copies G_host (n rows of N floats, row stride ld_host >= N elements; pinned memory makes the
 * copy asynchronous) into the bound G, runs dpsgd_mix_update(), evaluates the consensus
 * distance of the new X, waits, and writes it to *consensus_out_host.
 */
DPSGD_API dpsgd_status dpsgd_mix_update_host(dpsgd_ctx* ctx, const float* G_host, int64_t ld_host,
                                   double* consensus_out_host);

/*
 * (The paper has no counterpart: this is a packaging variant of dpsgd_consensus_dist.)
 * Consensus distance for callers that must not trigger an allocation: a process whose device
 * memory was handed to its own pool up front, a loop that cannot afford the device-wide
 * synchronisation an allocation implies, or code that has a raw device pointer and no context
 * (contexts allocate scratch).  It calls no cudaMalloc/cudaFree and no allocating library
 * routine; the per-CTA partial sums live in a fixed 512 KB array inside the library image, which
 * every GPU that loads the library keeps until the process exits.
 *   X_dev   device, fp32 [n][ld], 128-byte aligned, ld a multiple of 32, columns [N, ld) zero
 *   out_dev device, one double (8-byte aligned), written asynchronously on cuda_stream:
 *           sum_i ||xbar - x_i||^2, the same value dpsgd_consensus_dist returns
 * Limit: ld <= DPSGD_NOALLOC_MAX_LD (67,108,864 columns); larger inputs are refused with
 * DPSGD_ERR_UNSUPPORTED and a message in dpsgd_last_error(NULL).  1 <= n <= 65535.
 * The first call on each device looks up the array's device address (with that device current,
 * which must be the device that owns X_dev); make that first call outside any stream capture.
 * All calls in the process share the one array: it keeps the previous call's partial sums, each
 * call overwrites the entries it reads before reading them, and two calls whose kernels overlap
 * on the GPU (different streams) race on it - serialise them.
 */
#define DPSGD_NOALLOC_MAX_LD 67108864LL
DPSGD_API dpsgd_status dpsgd_consensus_dist_noalloc(const float* X_dev, int32_t n, int64_t N, int64_t ld,
                                                    void* cuda_stream, double* out_dev);

/* Device pointer of the buffer that currently holds X_k (one of the two bound buffers). */
DPSGD_API dpsgd_status dpsgd_current(dpsgd_ctx* ctx, float** X_cur_dev);

/* Step length gamma of Algorithm 1; may change between iterations (schedules). */
DPSGD_API dpsgd_status dpsgd_set_gamma(dpsgd_ctx* ctx, float gamma);

/* Which DPSGD_MIX_* kernel the structure of W selected; force >= 0 overrides it when the
 * requested kernel can handle W (else DPSGD_ERR_UNSUPPORTED).  Pass force = -1 to query.
 * Unless a kernel was forced, problems of at most 8 MB per matrix (latency-bound) take a
 * one-thread-per-output kernel instead, whatever the structure of W. */
DPSGD_API dpsgd_status dpsgd_mix_kind(dpsgd_ctx* ctx, int32_t force, int32_t* kind_out);

/* Number of kernels this context has launched so far (for launch accounting). */
DPSGD_API dpsgd_status dpsgd_launch_count(dpsgd_ctx* ctx, int64_t* count_out);

/* Message for the last non-OK status on ctx (never NULL; valid until the next call on ctx).
 * With ctx == NULL, the message of the last failed dpsgd_create() on this thread. */
DPSGD_API const char* dpsgd_last_error(dpsgd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* DPSGD_H_ */
