// The rest of the pre-norm transformer block around SPA (Sec. 3.2: selected tokens go through attention, the
// others straight to the feed-forward network): LayerNorm over the channels and the exact GELU, forward and
// backward.  The two feed-forward products are the library's linear layers run over all B*N tokens.
// Row-wise streaming kernels: one warp per token row, 16-byte accesses, fp32 arithmetic; the per-channel sums
// of the LayerNorm backward are taken per CTA in a fixed order and combined by the shared reduction kernel.
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kRestThreads = 256;
constexpr int kLnChunks = 4;  // 16-byte chunks of a row per lane: C <= 128 chunks (1024 bf16 / 512 fp32 channels)

template <typename T>
__global__ void __launch_bounds__(kRestThreads)
layer_norm_kernel(const uint4* __restrict__ x16, const T* __restrict__ gamma, const T* __restrict__ beta, float eps,
                  int rows, int C, uint4* __restrict__ y16, float* __restrict__ mean, float* __restrict__ rstd) {
  pdl_entry();
  constexpr int E = Vec16<T>::kElems;
  const int lane = threadIdx.x & 31, Q = C / E;
  const int warps = gridDim.x * (kRestThreads / 32);
  for (int t = blockIdx.x * (kRestThreads / 32) + (threadIdx.x >> 5); t < rows; t += warps) {
    float v[kLnChunks][E];
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kLnChunks; ++k) {
      const int q = lane + 32 * k;
      if (q < Q) {
        Vec16<T>::to_float(ld_nc16(x16 + (long long)t * Q + q), v[k]);
#pragma unroll
        for (int e = 0; e < E; ++e) s += v[k][e];
      }
    }
    const float mu = warp_sum(s) / C;
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < kLnChunks; ++k)
      if (lane + 32 * k < Q) {
#pragma unroll
        for (int e = 0; e < E; ++e) { const float d = v[k][e] - mu; ss = fmaf(d, d, ss); }
      }
    const float rs = rsqrtf(warp_sum(ss) / C + eps);
    if (lane == 0) { mean[t] = mu; rstd[t] = rs; }
#pragma unroll
    for (int k = 0; k < kLnChunks; ++k) {
      const int q = lane + 32 * k;
      if (q < Q) {
        float o[E];
#pragma unroll
        for (int e = 0; e < E; ++e)
          o[e] = (v[k][e] - mu) * rs * to_f32<T>(gamma[q * E + e]) + to_f32<T>(beta[q * E + e]);
        y16[(long long)t * Q + q] = Vec16<T>::from_float(o);
      }
    }
  }
}

// dx = rstd (g - mean(g) - xh mean(g xh)), g = dy gamma, xh = (x - mean) rstd; optionally + add (the residual
// branch's gradient).  Per-CTA sums of dy xh (dgamma) and dy (dbeta) go to part[blockIdx][2C].
// kCh = 16-byte chunks of a row per lane (ceil(C / (32 chunks))): sized exactly, so that narrow rows do not
// carry the registers of wide ones and several CTAs share an SM.
template <typename T, int kCh>
__global__ void __launch_bounds__(kRestThreads)
layer_norm_bwd_kernel(const uint4* __restrict__ dy16, const uint4* __restrict__ x16, const T* __restrict__ gamma,
                      const float* __restrict__ mean, const float* __restrict__ rstd, const uint4* add16, int rows,
                      int C, uint4* dx16, float* __restrict__ part) {
  pdl_entry();
  constexpr int E = Vec16<T>::kElems;
  extern __shared__ float acc_s[];  // [8 warps][2C]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, Q = C / E;
  float ag[kCh][E], ab[kCh][E];
#pragma unroll
  for (int k = 0; k < kCh; ++k)
#pragma unroll
    for (int e = 0; e < E; ++e) { ag[k][e] = 0.f; ab[k][e] = 0.f; }
  const int warps = gridDim.x * (kRestThreads / 32);
  for (int t = blockIdx.x * (kRestThreads / 32) + warp; t < rows; t += warps) {
    const float mu = mean[t], rs = rstd[t];
    float g[kCh][E], xh[kCh][E];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int k = 0; k < kCh; ++k) {
      const int q = lane + 32 * k;
      if (q < Q) {
        float dy[E], xv[E];
        Vec16<T>::to_float(ld_nc16(dy16 + (long long)t * Q + q), dy);
        Vec16<T>::to_float(ld_nc16(x16 + (long long)t * Q + q), xv);
#pragma unroll
        for (int e = 0; e < E; ++e) {
          xh[k][e] = (xv[e] - mu) * rs;
          g[k][e] = dy[e] * to_f32<T>(gamma[q * E + e]);
          s1 += g[k][e];
          s2 = fmaf(g[k][e], xh[k][e], s2);
          ag[k][e] = fmaf(dy[e], xh[k][e], ag[k][e]);
          ab[k][e] += dy[e];
        }
      }
    }
    const float m1 = warp_sum(s1) / C, m2 = warp_sum(s2) / C;
#pragma unroll
    for (int k = 0; k < kCh; ++k) {
      const int q = lane + 32 * k;
      if (q < Q) {
        float o[E];
#pragma unroll
        for (int e = 0; e < E; ++e) o[e] = (g[k][e] - m1 - xh[k][e] * m2) * rs;
        if (add16 != nullptr) {
          float a[E];
          Vec16<T>::to_float(add16[(long long)t * Q + q], a);
#pragma unroll
          for (int e = 0; e < E; ++e) o[e] += a[e];
        }
        dx16[(long long)t * Q + q] = Vec16<T>::from_float(o);
      }
    }
  }
  float* mine = acc_s + warp * 2 * C;
#pragma unroll
  for (int k = 0; k < kCh; ++k) {
    const int q = lane + 32 * k;
    if (q < Q) {
#pragma unroll
      for (int e = 0; e < E; ++e) { mine[q * E + e] = ag[k][e]; mine[C + q * E + e] = ab[k][e]; }
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < 2 * C; c += kRestThreads) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kRestThreads / 32; ++w) s += acc_s[w * 2 * C + c];
    part[(long long)blockIdx.x * 2 * C + c] = s;
  }
}

__device__ __forceinline__ float gelu_f(float u) { return 0.5f * u * (1.f + erff(u * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_grad_f(float u) {
  return 0.5f * (1.f + erff(u * 0.70710678118654752f)) + u * 0.3989422804014327f * __expf(-0.5f * u * u);
}

// out = gelu(u) (kBwd = false) or out = dh * gelu'(u) (kBwd = true), over `total` 16-byte chunks
template <typename T, bool kBwd>
__global__ void __launch_bounds__(kRestThreads)
gelu_kernel(const uint4* __restrict__ u16, const uint4* dh16, long long total, uint4* out16) {
  pdl_entry();
  constexpr int E = Vec16<T>::kElems;
  for (long long k = (long long)blockIdx.x * kRestThreads + threadIdx.x; k < total; k += (long long)gridDim.x * kRestThreads) {
    float u[E], o[E];
    Vec16<T>::to_float(ld_nc16(u16 + k), u);
    if (kBwd) {
      float d[E];
      Vec16<T>::to_float(dh16[k], d);
#pragma unroll
      for (int e = 0; e < E; ++e) o[e] = d[e] * gelu_grad_f(u[e]);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) o[e] = gelu_f(u[e]);
    }
    out16[k] = Vec16<T>::from_float(o);
  }
}

// Both kernels are bound by the latency of a row rather than by bandwidth: the forward takes two rows per
// warp; the backward four, because every extra CTA is another line of partial sums to combine (measured).
int ln_grid(int rows) {
  int g = (rows + 15) / 16;
  if (g > kNumSMs * 6) g = kNumSMs * 6;
  return g < 1 ? 1 : g;
}
int ln_bwd_grid(int rows) {
  int g = (rows + 31) / 32;
  if (g > kNumSMs * 4) g = kNumSMs * 4;
  return g < 1 ? 1 : g;
}

}  // namespace

size_t layer_norm_workspace_bytes(const spa_params& p) { return (size_t)ln_bwd_grid(p.B * p.N) * 2 * p.C * sizeof(float) + 256; }

bool layer_norm_supported(const spa_params& p) { return p.C / (p.dtype == SPA_F32 ? 4 : 8) <= 32 * kLnChunks; }

int launch_layer_norm(const spa_params& p, const void* x, const void* gamma, const void* beta, float eps, void* y,
                      float* mean, float* rstd, cudaStream_t st) {
  const int rows = p.B * p.N;
  if (rows == 0) return SPA_OK;
  if (!layer_norm_supported(p)) return SPA_ERR_UNSUPPORTED;
  if (p.dtype == SPA_F32)
    launch_pdl(layer_norm_kernel<float>, ln_grid(rows), kRestThreads, 0, st, (const uint4*)x, (const float*)gamma,
               (const float*)beta, eps, rows, p.C, (uint4*)y, mean, rstd);
  else
    launch_pdl(layer_norm_kernel<__nv_bfloat16>, ln_grid(rows), kRestThreads, 0, st, (const uint4*)x,
               (const __nv_bfloat16*)gamma, (const __nv_bfloat16*)beta, eps, rows, p.C, (uint4*)y, mean, rstd);
  SPA_CUDA_CHECK_LAUNCH("layer_norm_kernel");
  return SPA_OK;
}

int launch_layer_norm_bwd(const spa_params& p, const void* dy, const void* x, const void* gamma, const float* mean,
                          const float* rstd, const void* add, void* dx, float* dgamma, float* dbeta, void* workspace,
                          cudaStream_t st) {
  const int rows = p.B * p.N;
  if (rows == 0) return SPA_OK;
  if (!layer_norm_supported(p)) return SPA_ERR_UNSUPPORTED;
  const int grid = ln_bwd_grid(rows);
  const size_t smem = (size_t)(kRestThreads / 32) * 2 * p.C * sizeof(float);
  float* part = reinterpret_cast<float*>(workspace);
  const int chunks = (p.C / (p.dtype == SPA_F32 ? 4 : 8) + 31) / 32;  // 1..4 (layer_norm_supported)
  cudaError_t e = cudaSuccess;
#define SPA_LN_BWD(T, CH)                                                                                             \
  do {                                                                                                                \
    auto kern = layer_norm_bwd_kernel<T, CH>;                                                                         \
    static DeviceOnce attr;                                                                                           \
    e = attr.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024); }); \
    if (e == cudaSuccess)                                                                                             \
      launch_pdl(kern, grid, kRestThreads, smem, st, (const uint4*)dy, (const uint4*)x, (const T*)gamma, mean, rstd, \
                 (const uint4*)add, rows, p.C, (uint4*)dx, part);                                                     \
  } while (0)
#define SPA_LN_BWD_T(T)                                                                                               \
  do {                                                                                                                \
    if (chunks <= 1) SPA_LN_BWD(T, 1); else if (chunks == 2) SPA_LN_BWD(T, 2); else if (chunks == 3) SPA_LN_BWD(T, 3); \
    else SPA_LN_BWD(T, 4);                                                                                            \
  } while (0)
  if (p.dtype == SPA_F32) SPA_LN_BWD_T(float); else SPA_LN_BWD_T(__nv_bfloat16);
#undef SPA_LN_BWD_T
#undef SPA_LN_BWD
  if (e != cudaSuccess) { set_cuda_error(e, "layer_norm_bwd_kernel"); return SPA_ERR_CUDA; }
  SPA_CUDA_CHECK_LAUNCH("layer_norm_bwd_kernel");
  // dgamma = columns [0, C) of the per-CTA sums, dbeta = columns [C, 2C): one reduction launch for both
  return launch_partial_sum(part, grid, 2 * p.C, p.C, dgamma, p.C, dbeta, st);
}

int launch_gelu(const spa_params& p, const void* u, const void* dh, int n_cols, void* out, cudaStream_t st) {
  const int E = p.dtype == SPA_F32 ? 4 : 8;
  const long long total = (long long)p.B * p.N * n_cols / E;
  if (total == 0) return SPA_OK;
  long long g = (total + kRestThreads * 4 - 1) / (kRestThreads * 4);
  if (g > kNumSMs * 8) g = kNumSMs * 8;
  const int grid = g < 1 ? 1 : (int)g;
  if (p.dtype == SPA_F32) {
    if (dh) launch_pdl(gelu_kernel<float, true>, grid, kRestThreads, 0, st, (const uint4*)u, (const uint4*)dh, total, (uint4*)out);
    else launch_pdl(gelu_kernel<float, false>, grid, kRestThreads, 0, st, (const uint4*)u, (const uint4*)dh, total, (uint4*)out);
  } else {
    if (dh) launch_pdl(gelu_kernel<__nv_bfloat16, true>, grid, kRestThreads, 0, st, (const uint4*)u, (const uint4*)dh, total, (uint4*)out);
    else launch_pdl(gelu_kernel<__nv_bfloat16, false>, grid, kRestThreads, 0, st, (const uint4*)u, (const uint4*)dh, total, (uint4*)out);
  }
  SPA_CUDA_CHECK_LAUNCH("gelu_kernel");
  return SPA_OK;
}

}  // namespace spa
