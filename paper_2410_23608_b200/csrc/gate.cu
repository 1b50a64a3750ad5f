// Gate GEMV fused with the hard threshold (Sec. 3.2, Eq. 4 and the deterministic form of Eq. 6).
//
// HBM-bound: every element of x is read exactly once with 16-byte streaming loads; the only
// writes are 4 B (score) + 1 B (mask) per token - plus, on request, the copy y = x that the fused
// unpack needs for the tokens that pass through, which costs no second read of x.  One warp owns kGateRows token rows at a time so
// that several independent 16-byte loads per lane are in flight; w_g sits in shared memory as fp32.
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kGateThreads = 256;
constexpr int kGateRows = 2;  // rows per warp per iteration

template <typename T>
__global__ void __launch_bounds__(kGateThreads)
gate_kernel(const T* __restrict__ x, const T* __restrict__ w_g, float b_g, const float* __restrict__ s_up,
            float tau, int rows, int C, float* __restrict__ scores, uint8_t* __restrict__ mask, uint4* __restrict__ y16) {
  pdl_entry();
  constexpr int E = Vec16<T>::kElems;
  extern __shared__ float w_s[];
  for (int c = threadIdx.x; c < C; c += blockDim.x) w_s[c] = to_f32<T>(w_g[c]);
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  const int warp = blockIdx.x * warps_per_cta + (threadIdx.x >> 5);
  const int n_warps = gridDim.x * warps_per_cta;
  const int Q = C / E;  // 16-byte chunks per row
  const uint4* x16 = reinterpret_cast<const uint4*>(x);

  for (int r0 = warp * kGateRows; r0 < rows; r0 += n_warps * kGateRows) {
    float acc[kGateRows];
#pragma unroll
    for (int k = 0; k < kGateRows; ++k) acc[k] = 0.f;
    for (int q = lane; q < Q; q += 32) {
      uint4 v[kGateRows];
#pragma unroll
      for (int k = 0; k < kGateRows; ++k)
        if (r0 + k < rows) v[k] = ld_nc16(x16 + (size_t)(r0 + k) * Q + q);
      if (y16 != nullptr) {  // pass-through copy y = x rides on the one read of x
#pragma unroll
        for (int k = 0; k < kGateRows; ++k)
          if (r0 + k < rows) y16[(size_t)(r0 + k) * Q + q] = v[k];
      }
      const float4* wq = reinterpret_cast<const float4*>(w_s + q * E);
      float w[E];
#pragma unroll
      for (int e = 0; e < E / 4; ++e) {
        float4 t = wq[e];
        w[4 * e] = t.x; w[4 * e + 1] = t.y; w[4 * e + 2] = t.z; w[4 * e + 3] = t.w;
      }
#pragma unroll
      for (int k = 0; k < kGateRows; ++k) {
        if (r0 + k < rows) {
          float f[E];
          Vec16<T>::to_float(v[k], f);
#pragma unroll
          for (int e = 0; e < E; ++e) acc[k] = fmaf(f[e], w[e], acc[k]);
        }
      }
    }
#pragma unroll
    for (int k = 0; k < kGateRows; ++k) {
      float s = warp_sum(acc[k]) + b_g;
      const int r = r0 + k;
      if (lane == 0 && r < rows) {
        if (s_up != nullptr) s = fmaxf(s, s_up[r]);
        scores[r] = s;
        mask[r] = s > tau ? 1 : 0;
      }
    }
  }
}

}  // namespace

int launch_gate(const spa_params& p, const void* x, const void* w_g, float b_g, const float* s_up,
                float* scores, uint8_t* mask, void* y, cudaStream_t st) {
  const int rows = p.B * p.N;
  if (rows == 0) return SPA_OK;
  const int warps = kGateThreads / 32;
  int grid = (rows + warps * kGateRows - 1) / (warps * kGateRows);
  if (grid > kNumSMs * 8) grid = kNumSMs * 8;
  const size_t smem = (size_t)p.C * sizeof(float);
  if (p.dtype == SPA_F32)
    launch_pdl(gate_kernel<float>, grid, kGateThreads, smem, st, (const float*)x, (const float*)w_g, b_g, s_up, p.tau,
                                                         rows, p.C, scores, mask, (uint4*)y);
  else
    launch_pdl(gate_kernel<__nv_bfloat16>, grid, kGateThreads, smem, st, (const __nv_bfloat16*)x, (const __nv_bfloat16*)w_g,
                                                                 b_g, s_up, p.tau, rows, p.C, scores, mask, (uint4*)y);
  SPA_CUDA_CHECK_LAUNCH("gate_kernel");
  return SPA_OK;
}

}  // namespace spa
