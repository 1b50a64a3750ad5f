// C boundary: argument validation and dispatch to the kernels.  Nothing here computes.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <new>

#include "spa_common.cuh"
#include "spa_tc.cuh"

namespace spa {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
}

bool pdl_enabled() {
  static const bool on = []() { const char* e = getenv("SPA_PDL"); return !(e != nullptr && e[0] == '0'); }();
  return on;
}

static std::atomic<unsigned long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_params(const spa_params* p) {
  if (p == nullptr) return SPA_ERR_INVALID_ARG;
  if (p->B < 0 || p->N <= 0 || p->C <= 0 || p->H <= 0) return SPA_ERR_INVALID_ARG;
  if ((long long)p->B * p->N > (1LL << 20)) return SPA_ERR_UNSUPPORTED;
  if (p->capacity < 1 || (long long)p->capacity > (long long)(p->B > 0 ? p->B : 1) * p->N) return SPA_ERR_INVALID_ARG;
  if (p->dtype != SPA_F32 && p->dtype != SPA_BF16) return SPA_ERR_UNSUPPORTED;
  if (p->C % p->H != 0) return SPA_ERR_INVALID_ARG;
  const int es = p->dtype == SPA_F32 ? 4 : 2;
  if ((p->C * es) % 16 != 0 || p->C > 8192) return SPA_ERR_UNSUPPORTED;
  // the kernels take row maxima before scaling, which needs a scale that is positive (0 selects 1/sqrt(d))
  if (!(p->softmax_scale >= 0.f) || !(p->softmax_scale <= 3.0e38f)) return SPA_ERR_INVALID_ARG;
  return SPA_OK;
}

int check_heads(const spa_params* p) {
  const int d = p->C / p->H;
  return (d == 32 || d == 64) ? SPA_OK : SPA_ERR_UNSUPPORTED;
}

// bf16 problems run on the tensor-core kernels unless the caller asks for the fp32-FMA ones
inline bool use_tc(const spa_params* p) { return p->dtype == SPA_BF16 && !(p->flags & SPA_FLAG_SIMT_ONLY); }

#define SPA_REQUIRE(cond, code) do { if (!(cond)) return (code); } while (0)
#define SPA_PTR(ptr) SPA_REQUIRE((ptr) != nullptr && aligned16(ptr), SPA_ERR_INVALID_ARG)
#define SPA_OPT_PTR(ptr) SPA_REQUIRE((ptr) == nullptr || aligned16(ptr), SPA_ERR_INVALID_ARG)

}  // namespace
}  // namespace spa

using namespace spa;

extern "C" {

size_t spa_workspace_bytes(const spa_params* p) {
  if (check_params(p) != SPA_OK) return 0;
  const size_t a = tc_linear_workspace_bytes(*p), b = tc_attention_workspace_bytes(*p);
  return a > b ? a : b;
}

int spa_gate(const spa_params* p, const void* x, const void* w_g, float b_g, const float* s_up, float* scores,
             uint8_t* mask, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(w_g); SPA_PTR(scores); SPA_PTR(mask); SPA_OPT_PTR(s_up);
  return launch_gate(*p, x, w_g, b_g, s_up, scores, mask, nullptr, (cudaStream_t)stream);
}

int spa_gate_prefill(const spa_params* p, const void* x, const void* w_g, float b_g, const float* s_up, float* scores,
                     uint8_t* mask, void* y, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(w_g); SPA_PTR(scores); SPA_PTR(mask); SPA_PTR(y); SPA_OPT_PTR(s_up);
  return launch_gate(*p, x, w_g, b_g, s_up, scores, mask, y == x ? nullptr : y, (cudaStream_t)stream);
}

int spa_select_pack(const spa_params* p, const void* x, const uint8_t* mask, const float* scores, void* x_packed,
                    int32_t* idx, int32_t* inv, int32_t* cu_seqlens, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(mask); SPA_PTR(x_packed); SPA_PTR(idx); SPA_PTR(cu_seqlens); SPA_OPT_PTR(inv);
  if (p->flags & SPA_FLAG_GATE_SCALE) SPA_PTR(scores);
  if (p->B == 0) {
    cudaError_t e = cudaMemsetAsync(cu_seqlens, 0, sizeof(int32_t), (cudaStream_t)stream);
    if (e != cudaSuccess) { set_cuda_error(e, "spa_select_pack"); return SPA_ERR_CUDA; }
    return SPA_OK;
  }
  return launch_select_pack(*p, x, mask, scores, nullptr, x_packed, idx, inv, cu_seqlens, d_status, (cudaStream_t)stream);
}

size_t spa_pack_state_bytes(const spa_params* p) {
  if (check_params(p) != SPA_OK) return 0;
  return gate_pack_state_bytes(*p);
}

int spa_gate_select_pack_supported(const spa_params* p) {
  return (check_params(p) == SPA_OK && gate_pack_supported(*p)) ? 1 : 0;
}

int spa_gate_select_pack(const spa_params* p, const void* x, const void* w_g, float b_g, const float* s_up,
                         float* scores, uint8_t* mask, void* y, void* x_packed, int32_t* idx, int32_t* inv,
                         int32_t* cu_seqlens, void* pack_state, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(w_g); SPA_PTR(scores); SPA_PTR(mask); SPA_PTR(x_packed); SPA_PTR(idx); SPA_PTR(cu_seqlens);
  SPA_PTR(pack_state); SPA_OPT_PTR(s_up); SPA_OPT_PTR(inv); SPA_OPT_PTR(y);
  if (!gate_pack_supported(*p)) return SPA_ERR_UNSUPPORTED;
  if (p->B == 0) {
    cudaError_t e = cudaMemsetAsync(cu_seqlens, 0, sizeof(int32_t), (cudaStream_t)stream);
    if (e != cudaSuccess) { set_cuda_error(e, "spa_gate_select_pack"); return SPA_ERR_CUDA; }
    return SPA_OK;
  }
  return launch_gate_pack(*p, x, w_g, b_g, s_up, scores, mask, y == x ? nullptr : y, x_packed, idx, inv, cu_seqlens,
                          pack_state, d_status, (cudaStream_t)stream);
}

int spa_select_pack_ordered(const spa_params* p, const void* x, const uint8_t* mask, const float* scores,
                            const int32_t* order, void* x_packed, int32_t* idx, int32_t* inv, int32_t* cu_seqlens,
                            int32_t* d_status, void* stream) {
  if (order == nullptr) return SPA_ERR_INVALID_ARG;
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(mask); SPA_PTR(x_packed); SPA_PTR(idx); SPA_PTR(cu_seqlens); SPA_OPT_PTR(inv);
  if (p->flags & SPA_FLAG_GATE_SCALE) SPA_PTR(scores);
  if (p->B == 0) {
    cudaError_t e = cudaMemsetAsync(cu_seqlens, 0, sizeof(int32_t), (cudaStream_t)stream);
    if (e != cudaSuccess) { set_cuda_error(e, "spa_select_pack_ordered"); return SPA_ERR_CUDA; }
    return SPA_OK;
  }
  return launch_select_pack(*p, x, mask, scores, order, x_packed, idx, inv, cu_seqlens, d_status, (cudaStream_t)stream);
}

int32_t spa_container_max_segments(const spa_params* p, int32_t L) {
  if (check_params(p) != SPA_OK || L < 1) return 0;
  return p->B + p->capacity / L;
}

int spa_container_offsets(const spa_params* p, const int32_t* cu_seqlens, int32_t L, int32_t* seg_offsets,
                          void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  if (cu_seqlens == nullptr || seg_offsets == nullptr || L < 1) return SPA_ERR_INVALID_ARG;
  return launch_container_offsets(*p, cu_seqlens, L, spa_container_max_segments(p, L), seg_offsets, (cudaStream_t)stream);
}

int spa_packed_qkv(const spa_params* p, const void* x_packed, const void* W_qkv, const void* b_qkv,
                   const int32_t* cu_seqlens, void* qkv, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x_packed); SPA_PTR(W_qkv); SPA_PTR(cu_seqlens); SPA_PTR(qkv); SPA_OPT_PTR(b_qkv);
  if (use_tc(p) && tc_linear_supported(p->C, 3 * p->C)) {
    rc = launch_linear_fwd_tc(*p, x_packed, W_qkv, b_qkv, p->C, 3 * p->C, cu_seqlens, qkv, d_status,
                              (cudaStream_t)stream);
    if (rc != SPA_ERR_UNSUPPORTED) return rc;  // geometry the TMA path cannot describe: fp32-FMA kernels
  }
  return launch_linear_fwd_simt(*p, x_packed, W_qkv, b_qkv, p->C, 3 * p->C, cu_seqlens, qkv, (cudaStream_t)stream);
}

int spa_packed_proj(const spa_params* p, const void* a, const void* W_o, const void* b_o, const int32_t* cu_seqlens,
                    void* z, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(a); SPA_PTR(W_o); SPA_PTR(cu_seqlens); SPA_PTR(z); SPA_OPT_PTR(b_o);
  if (use_tc(p) && tc_linear_supported(p->C, p->C)) {
    rc = launch_linear_fwd_tc(*p, a, W_o, b_o, p->C, p->C, cu_seqlens, z, d_status, (cudaStream_t)stream);
    if (rc != SPA_ERR_UNSUPPORTED) return rc;
  }
  return launch_linear_fwd_simt(*p, a, W_o, b_o, p->C, p->C, cu_seqlens, z, (cudaStream_t)stream);
}

int spa_packed_attention_fwd(const spa_params* p, const void* qkv, const int32_t* seg_offsets, int32_t n_seg,
                             void* attn_out, float* lse, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  rc = check_heads(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(qkv); SPA_PTR(seg_offsets); SPA_PTR(attn_out); SPA_PTR(lse);
  SPA_REQUIRE(n_seg >= 0, SPA_ERR_INVALID_ARG);
  if (use_tc(p) && tc_attention_fwd_supported(*p)) {
    rc = launch_attention_fwd_tc(*p, qkv, seg_offsets, n_seg, attn_out, lse, d_status, (cudaStream_t)stream);
    if (rc != SPA_ERR_UNSUPPORTED) return rc;
  }
  return launch_attention_fwd_simt(*p, qkv, seg_offsets, n_seg, attn_out, lse, (cudaStream_t)stream);
}

int spa_packed_attention_bwd(const spa_params* p, const void* qkv, const void* attn_out, const float* lse,
                             const void* d_attn_out, const int32_t* seg_offsets, int32_t n_seg, void* dqkv,
                             void* workspace, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  rc = check_heads(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(qkv); SPA_PTR(attn_out); SPA_PTR(lse); SPA_PTR(d_attn_out); SPA_PTR(seg_offsets); SPA_PTR(dqkv);
  SPA_OPT_PTR(workspace);
  SPA_REQUIRE(n_seg >= 0, SPA_ERR_INVALID_ARG);
  if (use_tc(p) && tc_attention_bwd_supported(*p) && workspace != nullptr) {
    rc = launch_attention_bwd_tc(*p, qkv, attn_out, lse, d_attn_out, seg_offsets, n_seg, dqkv, workspace, d_status,
                                 (cudaStream_t)stream);
    if (rc != SPA_ERR_UNSUPPORTED) return rc;
  }
  return launch_attention_bwd_simt(*p, qkv, attn_out, lse, d_attn_out, seg_offsets, n_seg, dqkv,
                                   (cudaStream_t)stream);
}

int spa_packed_attention_bwd_static(const spa_params* p, const void* qkv, const void* attn_out, const float* lse,
                                    const void* d_attn_out, const int32_t* seg_offsets, int32_t n_seg, void* dqkv,
                                    int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  rc = check_heads(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(qkv); SPA_PTR(attn_out); SPA_PTR(lse); SPA_PTR(d_attn_out); SPA_PTR(seg_offsets); SPA_PTR(dqkv);
  SPA_REQUIRE(n_seg >= 0, SPA_ERR_INVALID_ARG);
  if (!use_tc(p) || !tc_attention_bwd_supported(*p)) return SPA_ERR_UNSUPPORTED;
  if ((unsigned long long)p->H * (unsigned long long)p->capacity * sizeof(float) > SPA_STATIC_SCRATCH_BYTES)
    return SPA_ERR_SCRATCH;
  void* scratch = nullptr;  // the array inside the library image: nothing is allocated here
  rc = static_attention_scratch(&scratch);
  if (rc != SPA_OK) return rc;
  return launch_attention_bwd_tc(*p, qkv, attn_out, lse, d_attn_out, seg_offsets, n_seg, dqkv, scratch, d_status,
                                 (cudaStream_t)stream);
}

int spa_unpack_scatter(const spa_params* p, const void* z_packed, const void* x, const int32_t* idx,
                       const int32_t* inv, const int32_t* cu_seqlens, void* y, int32_t* d_status, void* stream) {
  (void)d_status;
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(z_packed); SPA_PTR(cu_seqlens); SPA_PTR(y);
  if (p->flags & SPA_FLAG_INPLACE) {
    SPA_PTR(idx);
    SPA_REQUIRE(x == nullptr || x == y, SPA_ERR_INVALID_ARG);
    x = y;
  } else {
    SPA_PTR(x); SPA_PTR(inv);
    SPA_REQUIRE(x != y, SPA_ERR_INVALID_ARG);
  }
  if (p->B == 0) return SPA_OK;
  return launch_unpack_scatter(*p, z_packed, x, idx, inv, cu_seqlens, y, (cudaStream_t)stream);
}

int spa_unpack_scatter_bwd(const spa_params* p, const void* dY, const int32_t* idx, const int32_t* inv,
                           const int32_t* cu_seqlens, void* dz_packed, void* dX, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dY); SPA_PTR(inv); SPA_PTR(cu_seqlens); SPA_PTR(dz_packed); SPA_OPT_PTR(dX);
  if (p->B == 0) return SPA_OK;
  return launch_unpack_scatter_bwd(*p, dY, idx, inv, cu_seqlens, dz_packed, dX, (cudaStream_t)stream);
}

int spa_select_pack_bwd(const spa_params* p, const void* dx_packed, const void* dY, const int32_t* idx,
                        const int32_t* cu_seqlens, void* dX, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dx_packed); SPA_PTR(idx); SPA_PTR(cu_seqlens); SPA_PTR(dX);
  if (p->flags & SPA_FLAG_RESIDUAL) SPA_PTR(dY);
  if (p->B == 0) return SPA_OK;
  return launch_select_pack_bwd(*p, dx_packed, dY, idx, cu_seqlens, dX, (cudaStream_t)stream);
}

int spa_packed_linear_bwd(const spa_params* p, const void* a, const void* W, const void* dout, int32_t n_in,
                          int32_t n_out, const int32_t* cu_seqlens, void* da, float* dW, float* db, void* workspace,
                          int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dout); SPA_PTR(cu_seqlens);
  SPA_OPT_PTR(da); SPA_OPT_PTR(dW); SPA_OPT_PTR(db); SPA_OPT_PTR(workspace);
  if (da != nullptr) SPA_PTR(W);
  if (dW != nullptr) SPA_PTR(a);
  SPA_REQUIRE(n_in > 0 && n_out > 0, SPA_ERR_INVALID_ARG);
  const int es = p->dtype == SPA_F32 ? 4 : 2;
  SPA_REQUIRE((n_in * es) % 16 == 0 && (n_out * es) % 16 == 0, SPA_ERR_UNSUPPORTED);
  if (use_tc(p) && tc_linear_supported(n_in, n_out) && workspace != nullptr) {
    rc = launch_linear_bwd_tc(*p, a, W, dout, n_in, n_out, cu_seqlens, da, dW, db, workspace, d_status,
                              (cudaStream_t)stream);
    if (rc != SPA_ERR_UNSUPPORTED) return rc;
  }
  return launch_linear_bwd_simt(*p, a, W, dout, n_in, n_out, cu_seqlens, da, dW, db, (cudaStream_t)stream);
}

int spa_fused_scatter_supported(const spa_params* p) {
  if (check_params(p) != SPA_OK) return 0;
  return (use_tc(p) && tc_linear_supported(p->C, p->C) && tc_linear_supported(p->C, 3 * p->C)) ? 1 : 0;
}

int spa_unpack_prefill(const spa_params* p, const void* src, void* dst, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(src); SPA_PTR(dst);
  if (src == dst || p->B == 0) return SPA_OK;
  return launch_copy_tokens(*p, src, dst, (cudaStream_t)stream);
}

int spa_packed_proj_scatter(const spa_params* p, const void* a, const void* W_o, const void* b_o, const int32_t* idx,
                            const int32_t* cu_seqlens, void* y, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(a); SPA_PTR(W_o); SPA_PTR(idx); SPA_PTR(cu_seqlens); SPA_PTR(y); SPA_OPT_PTR(b_o);
  if (!spa_fused_scatter_supported(p)) return SPA_ERR_UNSUPPORTED;
  return launch_linear_fwd_tc(*p, a, W_o, b_o, p->C, p->C, cu_seqlens, y, d_status, (cudaStream_t)stream, idx,
                              (p->flags & SPA_FLAG_RESIDUAL) != 0);
}

int spa_packed_linear_bwd_scatter(const spa_params* p, const void* a, const void* W, const void* dout, int32_t n_in,
                                  int32_t n_out, const int32_t* idx, const int32_t* cu_seqlens, void* dX, float* dW,
                                  float* db, void* workspace, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dout); SPA_PTR(W); SPA_PTR(idx); SPA_PTR(cu_seqlens); SPA_PTR(dX);
  SPA_OPT_PTR(dW); SPA_OPT_PTR(db); SPA_OPT_PTR(workspace);
  if (dW != nullptr) SPA_PTR(a);
  SPA_REQUIRE(n_in == p->C && n_out > 0, SPA_ERR_INVALID_ARG);  // rows of dX are C wide
  SPA_REQUIRE(n_out % 8 == 0, SPA_ERR_UNSUPPORTED);
  if (!spa_fused_scatter_supported(p) || !tc_linear_supported(n_in, n_out)) return SPA_ERR_UNSUPPORTED;
  if ((dW != nullptr || db != nullptr) && workspace == nullptr) return SPA_ERR_INVALID_ARG;
  return launch_linear_bwd_tc(*p, a, W, dout, n_in, n_out, cu_seqlens, dX, dW, db, workspace, d_status,
                              (cudaStream_t)stream, idx, (p->flags & SPA_FLAG_RESIDUAL) != 0);
}

size_t spa_train_workspace_bytes(const spa_params* p) {
  if (check_params(p) != SPA_OK) return 0;
  return train_workspace_bytes(*p);
}

int spa_score_pool(const float* scores_prev, int32_t B, int32_t rows, int32_t cols, float* s_up, void* stream) {
  if (B < 0 || rows <= 0 || cols <= 0 || (long long)B * rows * cols > (1LL << 28)) return SPA_ERR_INVALID_ARG;
  if (scores_prev == nullptr || s_up == nullptr) return SPA_ERR_INVALID_ARG;
  return launch_score_pool(scores_prev, B, rows, cols, s_up, (cudaStream_t)stream);
}

int spa_select_loss(const spa_params* p, const float* scores, const uint8_t* labels, float alpha, float* ds,
                    float* loss, void* workspace, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  if (scores == nullptr || ds == nullptr || workspace == nullptr) return SPA_ERR_INVALID_ARG;
  return launch_select_loss(*p, scores, labels, alpha, ds, loss, workspace, (cudaStream_t)stream);
}

int spa_select_pack_bwd_gated(const spa_params* p, const void* dx_packed, const void* x, const float* scores,
                              const void* dY, const int32_t* idx, const int32_t* cu_seqlens, void* dX, float* ds,
                              void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dx_packed); SPA_PTR(x); SPA_PTR(idx); SPA_PTR(cu_seqlens); SPA_PTR(dX);
  if (scores == nullptr || ds == nullptr) return SPA_ERR_INVALID_ARG;
  if (p->flags & SPA_FLAG_RESIDUAL) SPA_PTR(dY);
  if (p->B == 0) return SPA_OK;
  return launch_pack_bwd_gated(*p, dx_packed, x, scores, dY, idx, cu_seqlens, dX, ds, (cudaStream_t)stream);
}

int spa_gate_bwd(const spa_params* p, const void* x, const void* w_g, const float* scores, const float* s_up,
                 const float* ds, void* dX, float* dw_g, float* db_g, float* ds_up, void* workspace, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(w_g); SPA_PTR(dX);
  if (scores == nullptr || ds == nullptr || dw_g == nullptr || workspace == nullptr) return SPA_ERR_INVALID_ARG;
  return launch_gate_bwd(*p, x, w_g, scores, s_up, ds, dX, dw_g, db_g, ds_up, workspace, (cudaStream_t)stream);
}

int spa_packed_linear(const spa_params* p, const void* a, const void* W, const void* b, int32_t n_in, int32_t n_out,
                      const int32_t* cu_seqlens, void* out, int32_t accumulate, int32_t* d_status, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(a); SPA_PTR(W); SPA_PTR(cu_seqlens); SPA_PTR(out); SPA_OPT_PTR(b);
  SPA_REQUIRE(n_in > 0 && n_out > 0, SPA_ERR_INVALID_ARG);
  const int es = p->dtype == SPA_F32 ? 4 : 2;
  SPA_REQUIRE((n_in * es) % 16 == 0 && (n_out * es) % 16 == 0, SPA_ERR_UNSUPPORTED);
  if (use_tc(p) && tc_linear_supported(n_in, n_out)) {
    rc = launch_linear_fwd_tc(*p, a, W, b, n_in, n_out, cu_seqlens, out, d_status, (cudaStream_t)stream, nullptr,
                              accumulate != 0);
    if (rc != SPA_ERR_UNSUPPORTED) return rc;
  }
  return launch_linear_fwd_simt(*p, a, W, b, n_in, n_out, cu_seqlens, out, (cudaStream_t)stream, accumulate != 0);
}

int spa_layer_norm(const spa_params* p, const void* x, const void* gamma, const void* beta, float eps, void* y,
                   float* mean, float* rstd, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(x); SPA_PTR(gamma); SPA_PTR(beta); SPA_PTR(y);
  if (mean == nullptr || rstd == nullptr || !(eps > 0.f)) return SPA_ERR_INVALID_ARG;
  return launch_layer_norm(*p, x, gamma, beta, eps, y, mean, rstd, (cudaStream_t)stream);
}

int spa_layer_norm_bwd(const spa_params* p, const void* dy, const void* x, const void* gamma, const float* mean,
                       const float* rstd, const void* add, void* dx, float* dgamma, float* dbeta, void* workspace,
                       void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dy); SPA_PTR(x); SPA_PTR(gamma); SPA_PTR(dx); SPA_OPT_PTR(add);
  if (mean == nullptr || rstd == nullptr || dgamma == nullptr || dbeta == nullptr || workspace == nullptr)
    return SPA_ERR_INVALID_ARG;
  return launch_layer_norm_bwd(*p, dy, x, gamma, mean, rstd, add, dx, dgamma, dbeta, workspace, (cudaStream_t)stream);
}

int spa_gelu(const spa_params* p, const void* u, int32_t n_cols, void* h, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(u); SPA_PTR(h);
  SPA_REQUIRE(n_cols > 0 && (n_cols * (p->dtype == SPA_F32 ? 4 : 2)) % 16 == 0, SPA_ERR_INVALID_ARG);
  return launch_gelu(*p, u, nullptr, n_cols, h, (cudaStream_t)stream);
}

int spa_gelu_bwd(const spa_params* p, const void* dh, const void* u, int32_t n_cols, void* du, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  SPA_PTR(dh); SPA_PTR(u); SPA_PTR(du);
  SPA_REQUIRE(n_cols > 0 && (n_cols * (p->dtype == SPA_F32 ? 4 : 2)) % 16 == 0, SPA_ERR_INVALID_ARG);
  return launch_gelu(*p, u, dh, n_cols, du, (cudaStream_t)stream);
}

// ---- the block as one unit: sequencing only ------------------------------------------------------------------
struct spa_overlap {
  cudaStream_t side;
  cudaEvent_t fork, join;
};

int spa_overlap_create(spa_overlap** out) {
  if (out == nullptr) return SPA_ERR_INVALID_ARG;
  spa_overlap* ov = new (std::nothrow) spa_overlap{nullptr, nullptr, nullptr};
  if (ov == nullptr) return SPA_ERR_INVALID_ARG;
  cudaError_t e = cudaStreamCreateWithFlags(&ov->side, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ov->fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ov->join, cudaEventDisableTiming);
  if (e != cudaSuccess) {
    set_cuda_error(e, "spa_overlap_create");
    spa_overlap_destroy(ov);
    return SPA_ERR_CUDA;
  }
  *out = ov;
  return SPA_OK;
}

int spa_overlap_destroy(spa_overlap* ov) {
  if (ov == nullptr) return SPA_OK;
  if (ov->join != nullptr) cudaEventDestroy(ov->join);
  if (ov->fork != nullptr) cudaEventDestroy(ov->fork);
  if (ov->side != nullptr) cudaStreamDestroy(ov->side);
  delete ov;
  return SPA_OK;
}

namespace {
inline bool block_fused(const spa_params* p) {
  return !(p->flags & SPA_FLAG_UNFUSED) && spa_fused_scatter_supported(p) != 0;
}
// the second stream starts after everything enqueued on the main stream so far
inline int fork_side(const spa_overlap* ov, cudaStream_t main) {
  cudaError_t e = cudaEventRecord(ov->fork, main);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ov->side, ov->fork, 0);
  if (e != cudaSuccess) { set_cuda_error(e, "spa_block_bwd: fork"); return SPA_ERR_CUDA; }
  return SPA_OK;
}
inline int join_side(const spa_overlap* ov, cudaStream_t main) {
  cudaError_t e = cudaEventRecord(ov->join, ov->side);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(main, ov->join, 0);
  if (e != cudaSuccess) { set_cuda_error(e, "spa_block_bwd: join"); return SPA_ERR_CUDA; }
  return SPA_OK;
}
#define SPA_STEP(call) do { rc = (call); if (rc != SPA_OK) return rc; } while (0)
}  // namespace

int spa_block_fwd(const spa_params* p, const spa_block_buffers* b, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  if (b == nullptr) return SPA_ERR_INVALID_ARG;
  const bool inplace = (p->flags & SPA_FLAG_INPLACE) != 0;
  const bool fused = block_fused(p);
  void* y = inplace ? const_cast<void*>(b->x) : b->y;
  SPA_REQUIRE(!inplace || b->y == nullptr || b->y == b->x, SPA_ERR_INVALID_ARG);
  // gate (Eq. 4) and hard selection; on the fused path it also writes the pass-through rows y = x
  const bool one_pass = b->pack_state != nullptr && b->order == nullptr && gate_pack_supported(*p);
  if (one_pass)  // gate, selection and packing read x once
    SPA_STEP(spa_gate_select_pack(p, b->x, b->w_g, b->b_g, b->s_up, b->scores, b->mask, (fused && !inplace) ? y : nullptr,
                                  b->x_packed, b->idx, b->inv, b->cu_seqlens, b->pack_state, b->d_status, stream));
  else if (fused && !inplace) SPA_STEP(spa_gate_prefill(p, b->x, b->w_g, b->b_g, b->s_up, b->scores, b->mask, y, stream));
  else SPA_STEP(spa_gate(p, b->x, b->w_g, b->b_g, b->s_up, b->scores, b->mask, stream));
  // token packing
  if (one_pass) {
  } else if (b->order == nullptr)
    SPA_STEP(spa_select_pack(p, b->x, b->mask, b->scores, b->x_packed, b->idx, b->inv, b->cu_seqlens, b->d_status, stream));
  else
    SPA_STEP(spa_select_pack_ordered(p, b->x, b->mask, b->scores, b->order, b->x_packed, b->idx, b->inv, b->cu_seqlens,
                                     b->d_status, stream));
  if (b->container_len > 0) {  // the paper's containers: cuts built on the device from the selection just packed
    SPA_REQUIRE(b->seg_offsets != nullptr, SPA_ERR_INVALID_ARG);
    SPA_STEP(spa_container_offsets(p, b->cu_seqlens, b->container_len, const_cast<int32_t*>(b->seg_offsets), stream));
  }
  SPA_STEP(spa_packed_qkv(p, b->x_packed, b->W_qkv, b->b_qkv, b->cu_seqlens, b->qkv, b->d_status, stream));
  const int32_t* seg = b->seg_offsets != nullptr ? b->seg_offsets : b->cu_seqlens;
  const int32_t n_seg = b->container_len > 0 ? spa_container_max_segments(p, b->container_len)
                                             : (b->seg_offsets != nullptr ? b->n_seg : p->B);
  SPA_STEP(spa_packed_attention_fwd(p, b->qkv, seg, n_seg, b->attn_out, b->lse, b->d_status, stream));
  if (fused) return spa_packed_proj_scatter(p, b->attn_out, b->W_o, b->b_o, b->idx, b->cu_seqlens, y, b->d_status, stream);
  SPA_STEP(spa_packed_proj(p, b->attn_out, b->W_o, b->b_o, b->cu_seqlens, b->z, b->d_status, stream));
  return spa_unpack_scatter(p, b->z, inplace ? nullptr : b->x, b->idx, b->inv, b->cu_seqlens, y, b->d_status, stream);
}

int spa_block_bwd(const spa_params* p, const spa_block_buffers* b, void* stream) {
  int rc = check_params(p);
  if (rc != SPA_OK) return rc;
  if (b == nullptr) return SPA_ERR_INVALID_ARG;
  const int C = p->C;
  cudaStream_t main = (cudaStream_t)stream;
  // the weight gradients feed nothing downstream: with `overlap` they run on the second stream, with a scratch
  // area of their own, beside the attention backward and the input gradients.  The trainable path keeps one stream.
  const spa_overlap* ov = b->trainable ? nullptr : b->overlap;
  SPA_REQUIRE(ov == nullptr || b->workspace_side != nullptr || spa_workspace_bytes(p) == 0, SPA_ERR_INVALID_ARG);
  const bool fused = block_fused(p) && !b->trainable;
  const int32_t* seg = b->seg_offsets != nullptr ? b->seg_offsets : b->cu_seqlens;
  const int32_t n_seg = (b->container_len > 0 && b->seg_offsets != nullptr)
                            ? spa_container_max_segments(p, b->container_len)
                            : (b->seg_offsets != nullptr ? b->n_seg : p->B);
  void* side = ov != nullptr ? (void*)ov->side : nullptr;

  if (b->trainable)
    SPA_STEP(spa_select_loss(p, b->scores, b->labels, b->alpha, b->ds, b->loss, b->train_workspace, stream));
  // dz = rows of dY at the selected tokens; dX = dY on the tokens that passed through
  SPA_STEP(spa_unpack_scatter_bwd(p, b->dY, b->idx, b->inv, b->cu_seqlens, b->dz, b->dX, stream));
  bool forked = false;
  int rc_side = SPA_OK;
  if (ov == nullptr) {
    SPA_STEP(spa_packed_linear_bwd(p, b->attn_out, b->W_o, b->dz, C, C, b->cu_seqlens, b->d_attn_out, b->dW_o, b->db_o,
                                   b->workspace, b->d_status, stream));
  } else {
    SPA_STEP(fork_side(ov, main));
    forked = true;
    rc_side = spa_packed_linear_bwd(p, b->attn_out, b->W_o, b->dz, C, C, b->cu_seqlens, nullptr, b->dW_o, b->db_o,
                                    b->workspace_side, b->d_status, side);
    rc = spa_packed_linear_bwd(p, b->attn_out, b->W_o, b->dz, C, C, b->cu_seqlens, b->d_attn_out, nullptr, nullptr,
                               b->workspace, b->d_status, stream);
  }
  if (rc == SPA_OK && rc_side == SPA_OK)
    rc = spa_packed_attention_bwd(p, b->qkv, b->attn_out, b->lse, b->d_attn_out, seg, n_seg, b->dqkv, b->workspace,
                                  b->d_status, stream);
  if (rc == SPA_OK && rc_side == SPA_OK) {
    if (ov != nullptr) {
      // the second stream's next call reads dqkv: it waits for the attention backward
      rc_side = fork_side(ov, main);
      if (rc_side == SPA_OK)
        rc_side = spa_packed_linear_bwd(p, b->x_packed, b->W_qkv, b->dqkv, C, 3 * C, b->cu_seqlens, nullptr, b->dW_qkv,
                                        b->db_qkv, b->workspace_side, b->d_status, side);
    }
    float* dW = ov != nullptr ? nullptr : b->dW_qkv;
    float* db = ov != nullptr ? nullptr : b->db_qkv;
    void* ws = ov != nullptr ? nullptr : b->workspace;
    if (fused) {
      // the input gradient scatters its rows to the selected tokens itself: no packed dx, no scatter kernel
      rc = spa_packed_linear_bwd_scatter(p, b->x_packed, b->W_qkv, b->dqkv, C, 3 * C, b->idx, b->cu_seqlens, b->dX, dW,
                                         db, ws, b->d_status, stream);
    } else {
      rc = spa_packed_linear_bwd(p, b->x_packed, b->W_qkv, b->dqkv, C, 3 * C, b->cu_seqlens, b->dx_packed, dW, db,
                                 ov != nullptr ? b->workspace : ws, b->d_status, stream);
      if (rc == SPA_OK) {
        if (b->trainable && (p->flags & SPA_FLAG_GATE_SCALE))
          rc = spa_select_pack_bwd_gated(p, b->dx_packed, b->x, b->scores, b->dY, b->idx, b->cu_seqlens, b->dX, b->ds,
                                         stream);
        else
          rc = spa_select_pack_bwd(p, b->dx_packed, b->dY, b->idx, b->cu_seqlens, b->dX, stream);
      }
    }
  }
  if (forked) {  // joined on every path, so that a recording stream is never left forked
    const int rj = join_side(ov, main);
    if (rc == SPA_OK) rc = rc_side != SPA_OK ? rc_side : rj;
  }
  if (rc != SPA_OK) return rc;
  if (b->trainable)
    SPA_STEP(spa_gate_bwd(p, b->x, b->w_g, b->scores, b->s_up, b->ds, b->dX, b->dw_g, b->db_g, b->ds_up,
                          b->train_workspace, stream));
  return SPA_OK;
}
#undef SPA_STEP

int spa_read_status(const int32_t* d_status, void* stream) {
  if (d_status == nullptr) return SPA_ERR_INVALID_ARG;
  int32_t v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, d_status, sizeof(v), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e, "spa_read_status"); return SPA_ERR_CUDA; }
  return v;
}

const char* spa_status_string(int status) {
  switch (status) {
    case SPA_OK: return "ok";
    case SPA_ERR_INVALID_ARG: return "invalid argument";
    case SPA_ERR_UNSUPPORTED: return "unsupported dtype, head dimension or size";
    case SPA_ERR_CAPACITY: return "more selected tokens than the packed capacity";
    case SPA_ERR_CUDA: return "CUDA runtime error";
    case SPA_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case SPA_ERR_SCRATCH: return "the problem needs more scratch than the built-in array holds";
    default: return "unknown status";
  }
}

const char* spa_last_cuda_error(void) { return g_cuda_error; }

unsigned long long spa_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
