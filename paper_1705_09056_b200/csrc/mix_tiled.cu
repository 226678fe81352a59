// Tiled CSR mixing kernel (placeholder).
#include "ctx.h"

namespace dpsgd {
bool mix_tiled_supported(const dpsgd_ctx*) { return false; }
void mix_tiled_release(dpsgd_ctx*) {}
cudaError_t launch_mix_tiled(dpsgd_ctx*, const float*, const float*, float*) { return cudaErrorNotSupported; }
}  // namespace dpsgd
