// MLP gradients (placeholder until the batched GEMM kernels land).
#include "ctx.h"

namespace dpsgd {
size_t mlp_act_floats(const dpsgd_ctx*) { return 1; }
size_t mlp_delta_floats(const dpsgd_ctx*) { return 1; }
cudaError_t launch_grad_mlp(dpsgd_ctx*, uint64_t, const float*, float*) { return cudaErrorNotSupported; }
}  // namespace dpsgd
