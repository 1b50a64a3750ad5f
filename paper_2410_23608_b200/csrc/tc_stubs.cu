// Placeholders for tensor-core kernels that are not built yet: they report "unsupported" so the
// dispatcher keeps those operations on the fp32-FMA kernels.
#include "spa_tc.cuh"

namespace spa {

size_t tc_attention_workspace_bytes(const spa_params&) { return 0; }
bool tc_attention_bwd_supported(const spa_params&) { return false; }
int launch_attention_bwd_tc(const spa_params&, const void*, const void*, const float*, const void*, const int32_t*,
                            int, void*, void*, int32_t*, cudaStream_t) { return SPA_ERR_UNSUPPORTED; }

}  // namespace spa
