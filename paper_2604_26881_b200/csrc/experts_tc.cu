// Tensor-core (tcgen05 / TMEM / TMA) grouped expert GEMMs.  Placeholder until the kernel lands.
#include "internal.h"

namespace faasmoe {

struct TensorMaps { int unused; };

bool tc_supported(const moe_ctx*) { return false; }
int tc_setup_layer(moe_ctx*, int) { return MOE_ERR_UNSUPPORTED; }
void tc_destroy(moe_ctx*) {}

cudaError_t launch_experts_tc(moe_ctx*, int, const bf16*, const bf16*, int, float*, float*, const int32_t*, cudaStream_t)
{
    return cudaErrorNotSupported;
}

}  // namespace faasmoe
