// Tensor-core (tcgen05 / TMEM / TMA) kernels for bf16 problems: entry points used by the dispatcher.
#pragma once

#include "spa_common.cuh"

namespace spa {

size_t tc_linear_workspace_bytes(const spa_params& p);
size_t tc_attention_workspace_bytes(const spa_params& p);

bool tc_linear_supported(int n_in, int n_out);
// row_map (optional): output row i is written to row row_map[i] of `out`, added to its contents if `accumulate`.
int launch_linear_fwd_tc(const spa_params& p, const void* a, const void* W, const void* bias, int n_in, int n_out,
                         const int32_t* cu, void* out, int32_t* d_status, cudaStream_t st,
                         const int32_t* row_map = nullptr, bool accumulate = false);
int launch_linear_bwd_tc(const spa_params& p, const void* a, const void* W, const void* dout, int n_in, int n_out,
                         const int32_t* cu, void* da, float* dW, float* db, void* workspace, int32_t* d_status,
                         cudaStream_t st, const int32_t* row_map = nullptr, bool accumulate = false);

// CTA-pair variants (cta_group::2, 256 x 256 tiles) of the forward product and the input gradient
bool tc_pair_linear_supported(const spa_params& p, int n_in, int n_out);
int launch_linear_fwd_pair(const spa_params& p, const void* a, const void* W, const void* bias, int n_in, int n_out,
                           const int32_t* cu, void* out, int32_t* d_status, cudaStream_t st, const int32_t* row_map,
                           bool accumulate);
int launch_linear_dgrad_pair(const spa_params& p, const void* W, const void* dout, int n_in, int n_out, const int32_t* cu,
                             void* da, int32_t* d_status, cudaStream_t st, const int32_t* row_map, bool accumulate);

bool tc_attention_fwd_supported(const spa_params& p);
int launch_attention_fwd_tc(const spa_params& p, const void* qkv, const int32_t* seg, int n_seg, void* ao, float* lse,
                            int32_t* d_status, cudaStream_t st);
bool tc_attention_bwd_supported(const spa_params& p);
int launch_attention_bwd_tc(const spa_params& p, const void* qkv, const void* ao, const float* lse, const void* dao,
                            const int32_t* seg, int n_seg, void* dqkv, void* workspace, int32_t* d_status,
                            cudaStream_t st);
// Device address, on the current device, of the SPA_STATIC_SCRATCH_BYTES array built into the library.
int static_attention_scratch(void** out);

}  // namespace spa
