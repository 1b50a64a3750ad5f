// Trainable selection: the pieces that let a gradient reach the gate (Sec. 3.2 Eq. 4-5, Sec. 3.3 Eq. 10).
//   score_pool_kernel      up-scale scores max-pooled 2x2 to this stage's grid (multi-scale selection)
//   select_loss_kernel     binary cross-entropy of Sigmoid(s) against the select labels, and its gradient
//   pack_bwd_gated_kernel  transpose of the pack gather when rows were scaled by Sigmoid(s) (Eq. 5)
//   gate_bwd_kernel        backward of s = Max(w_g . x + b_g, s_up)
// All of it is element-wise or row-wise streaming work: 16-byte loads, fp32 arithmetic, sums over tokens
// taken per CTA in a fixed order and combined by a second kernel, so results are bitwise reproducible.
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kTrainThreads = 256;

__device__ __forceinline__ float sigmoid_f(float s) { return 1.f / (1.f + __expf(-s)); }
// ln(1 + e^s) without overflow
__device__ __forceinline__ float softplus_f(float s) { return fmaxf(s, 0.f) + log1pf(__expf(-fabsf(s))); }

__global__ void __launch_bounds__(kTrainThreads)
score_pool_kernel(const float* __restrict__ prev, int B, int rows, int cols, float* __restrict__ s_up) {
  pdl_entry();
  const long long total = (long long)B * rows * cols;
  for (long long t = (long long)blockIdx.x * kTrainThreads + threadIdx.x; t < total;
       t += (long long)gridDim.x * kTrainThreads) {
    const int j = (int)(t % cols);
    const long long r = t / cols;
    const int i = (int)(r % rows);
    const long long b = r / rows;
    const float* src = prev + (b * 2 * rows + 2 * i) * (2LL * cols) + 2 * j;
    s_up[t] = fmaxf(fmaxf(src[0], src[1]), fmaxf(src[2 * cols], src[2 * cols + 1]));
  }
}

// ds[t] = alpha (Sigmoid(s_t) - y_t); part[blockIdx] = this CTA's share of the loss (tokens in a fixed
// grid-stride order, tree reduction of fixed shape).  labels == nullptr: ds = 0, loss = 0.
__global__ void __launch_bounds__(kTrainThreads)
select_loss_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ labels, float alpha, long long total,
                   float* __restrict__ ds, float* __restrict__ part) {
  pdl_entry();
  float acc = 0.f;
  for (long long t = (long long)blockIdx.x * kTrainThreads + threadIdx.x; t < total;
       t += (long long)gridDim.x * kTrainThreads) {
    float g = 0.f;
    if (labels != nullptr) {
      const float s = scores[t];
      const float y = labels[t] ? 1.f : 0.f;
      g = alpha * (sigmoid_f(s) - y);
      acc += y != 0.f ? softplus_f(-s) : softplus_f(s);  // -log p  |  -log(1 - p)
    }
    ds[t] = g;
  }
  __shared__ float red[kTrainThreads / 32];
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int w = 0; w < kTrainThreads / 32; ++w) s += red[w];
    part[blockIdx.x] = s;
  }
}

// out[j] = sum over blocks of part[block * stride + j] for j < n_out; columns n_out .. n_out + n_out2 - 1 go to out2.
// One warp per column: lane l adds blocks l, l + 32, ... in order, then the lanes combine in a fixed tree.
__global__ void __launch_bounds__(kTrainThreads)
partial_sum_kernel(const float* __restrict__ part, int n_blocks, int stride, int n_out, float* __restrict__ out, int n_out2,
                   float* __restrict__ out2) {
  pdl_entry();
  const int j = blockIdx.x * (kTrainThreads / 32) + (threadIdx.x >> 5);
  if (j >= n_out + n_out2) return;
  float s = 0.f;
  for (int b = threadIdx.x & 31; b < n_blocks; b += 32) s += part[(long long)b * stride + j];
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) {
    if (j < n_out) out[j] = s; else out2[j - n_out] = s;
  }
}

// One warp per packed row i (token t = idx[i]):  dX_t = Sigmoid(s_t) dxp_i (+ dY_t with the residual),
// ds_t += Sigmoid'(s_t) (dxp_i . x_t).
template <typename T, bool kResidual>
__global__ void __launch_bounds__(kTrainThreads)
pack_bwd_gated_kernel(const uint4* __restrict__ dxp16, const uint4* __restrict__ x16, const float* __restrict__ scores,
                      const uint4* dY16, const int32_t* __restrict__ idx, const int32_t* __restrict__ cu, int B,
                      int capacity, int Q, uint4* dX16, float* __restrict__ ds) {
  pdl_entry();
  constexpr int E = Vec16<T>::kElems;
  const int Np = packed_rows(cu, B, capacity);
  const int lane = threadIdx.x & 31;
  const int warps = gridDim.x * (kTrainThreads / 32);
  for (int i = blockIdx.x * (kTrainThreads / 32) + (threadIdx.x >> 5); i < Np; i += warps) {
    const long long t = __ldg(idx + i);
    const float p = sigmoid_f(scores[t]);
    float dot = 0.f;
    for (int q = lane; q < Q; q += 32) {
      const uint4 g = ld_nc16(dxp16 + (long long)i * Q + q);
      const uint4 xv = ld_nc16(x16 + t * Q + q);
      float fg[E], fx[E];
      Vec16<T>::to_float(g, fg);
      Vec16<T>::to_float(xv, fx);
#pragma unroll
      for (int e = 0; e < E; ++e) {
        dot = fmaf(fg[e], fx[e], dot);
        fg[e] *= p;
      }
      if (kResidual) {
        float fy[E];
        Vec16<T>::to_float(dY16[t * Q + q], fy);
#pragma unroll
        for (int e = 0; e < E; ++e) fg[e] += fy[e];
      }
      dX16[t * Q + q] = Vec16<T>::from_float(fg);
    }
    dot = warp_sum(dot);
    if (lane == 0) ds[t] += p * (1.f - p) * dot;
  }
}

// Backward of the gate.  A warp walks rows t, two at a time; where the linear layer supplied the maximum
// (g = ds_t) it adds g w_g to dX_t and g x_t to its running dw_g (registers: a lane owns the same columns of
// every row), g to its db_g; elsewhere ds_t goes to ds_up.  Per CTA the eight warps' sums are combined in
// warp order into part[blockIdx][C + 1].
constexpr int kGbRows = 2;     // rows in flight per warp
constexpr int kGbChunks = 4;   // 16-byte chunks of a row per lane: C <= 128 chunks

template <typename T>
__global__ void __launch_bounds__(kTrainThreads)
gate_bwd_kernel(const uint4* __restrict__ x16, const T* __restrict__ w_g, const float* __restrict__ scores,
                const float* __restrict__ s_up, const float* __restrict__ ds, int rows, int C, uint4* dX16,
                float* __restrict__ ds_up, float* __restrict__ part) {
  pdl_entry();
  constexpr int E = Vec16<T>::kElems;
  extern __shared__ float sm[];           // w_g as fp32 [C], then per-warp sums [8][C + 1]
  float* w_s = sm;
  float* acc_s = sm + C;
  for (int c = threadIdx.x; c < C; c += kTrainThreads) w_s[c] = to_f32<T>(w_g[c]);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int Q = C / E;
  float acc[kGbChunks][E];
#pragma unroll
  for (int k = 0; k < kGbChunks; ++k)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[k][e] = 0.f;
  float db = 0.f;
  const int warps = gridDim.x * (kTrainThreads / 32);
  for (int t0 = (blockIdx.x * (kTrainThreads / 32) + warp) * kGbRows; t0 < rows; t0 += warps * kGbRows) {
    float d[kGbRows];
#pragma unroll
    for (int r = 0; r < kGbRows; ++r) {
      const int t = t0 + r;
      d[r] = 0.f;
      if (t < rows) {
        const float dv = ds[t];
        const bool lin = s_up == nullptr || scores[t] > s_up[t];
        if (ds_up != nullptr && lane == 0) ds_up[t] = lin ? 0.f : dv;
        d[r] = lin ? dv : 0.f;
        db += d[r];
      }
    }
#pragma unroll
    for (int k = 0; k < kGbChunks; ++k) {
      const int q = lane + 32 * k;
      if (q >= Q) break;
      uint4 xv[kGbRows], gv[kGbRows];
#pragma unroll
      for (int r = 0; r < kGbRows; ++r)
        if (d[r] != 0.f) {  // warp-uniform
          xv[r] = ld_nc16(x16 + (long long)(t0 + r) * Q + q);
          gv[r] = dX16[(long long)(t0 + r) * Q + q];
        }
#pragma unroll
      for (int r = 0; r < kGbRows; ++r)
        if (d[r] != 0.f) {
          float fx[E], fd[E];
          Vec16<T>::to_float(xv[r], fx);
          Vec16<T>::to_float(gv[r], fd);
#pragma unroll
          for (int e = 0; e < E; ++e) {
            acc[k][e] = fmaf(d[r], fx[e], acc[k][e]);
            fd[e] = fmaf(d[r], w_s[q * E + e], fd[e]);
          }
          dX16[(long long)(t0 + r) * Q + q] = Vec16<T>::from_float(fd);
        }
    }
  }
  float* my_acc = acc_s + warp * (C + 1);
#pragma unroll
  for (int k = 0; k < kGbChunks; ++k) {
    const int q = lane + 32 * k;
    if (q < Q) {
#pragma unroll
      for (int e = 0; e < E; ++e) my_acc[q * E + e] = acc[k][e];
    }
  }
  if (lane == 0) my_acc[C] = db;
  __syncthreads();
  for (int c = threadIdx.x; c <= C; c += kTrainThreads) {
    float s2 = 0.f;
#pragma unroll
    for (int w = 0; w < kTrainThreads / 32; ++w) s2 += acc_s[w * (C + 1) + c];
    part[(long long)blockIdx.x * (C + 1) + c] = s2;
  }
}

int loss_grid(long long total) {
  long long g = (total + kTrainThreads - 1) / kTrainThreads;
  if (g > kNumSMs * 4) g = kNumSMs * 4;
  return g < 1 ? 1 : (int)g;
}
int gate_bwd_grid(int rows) {
  int g = (rows + 31) / 32;  // at least four rows per warp
  if (g > kNumSMs * 4) g = kNumSMs * 4;
  return g < 1 ? 1 : g;
}

}  // namespace

int launch_partial_sum(const float* part, int n_blocks, int stride, int n_out, float* out, int n_out2, float* out2,
                       cudaStream_t st) {
  if (out2 == nullptr) n_out2 = 0;
  const int cols = n_out + n_out2;
  launch_pdl(partial_sum_kernel, (cols + kTrainThreads / 32 - 1) / (kTrainThreads / 32), kTrainThreads, 0, st, part, n_blocks,
             stride, n_out, out, n_out2, out2);
  SPA_CUDA_CHECK_LAUNCH("partial_sum_kernel");
  return SPA_OK;
}

size_t train_workspace_bytes(const spa_params& p) {
  const size_t a = (size_t)gate_bwd_grid(p.B * p.N) * (p.C + 1) * sizeof(float);
  const size_t b = (size_t)loss_grid((long long)p.B * p.N) * sizeof(float);
  const size_t c = layer_norm_workspace_bytes(p);
  const size_t m = a > b ? (a > c ? a : c) : (b > c ? b : c);
  return (m + 255) & ~(size_t)255;
}

int launch_score_pool(const float* prev, int B, int rows, int cols, float* s_up, cudaStream_t st) {
  const long long total = (long long)B * rows * cols;
  if (total == 0) return SPA_OK;
  launch_pdl(score_pool_kernel, loss_grid(total), kTrainThreads, 0, st, prev, B, rows, cols, s_up);
  SPA_CUDA_CHECK_LAUNCH("score_pool_kernel");
  return SPA_OK;
}

int launch_select_loss(const spa_params& p, const float* scores, const uint8_t* labels, float alpha, float* ds,
                       float* loss, void* workspace, cudaStream_t st) {
  const long long total = (long long)p.B * p.N;
  if (total == 0) return SPA_OK;
  const int grid = loss_grid(total);
  float* part = reinterpret_cast<float*>(workspace);
  launch_pdl(select_loss_kernel, grid, kTrainThreads, 0, st, scores, labels, alpha, total, ds, part);
  SPA_CUDA_CHECK_LAUNCH("select_loss_kernel");
  if (loss != nullptr) {
    const int rc = launch_partial_sum(part, grid, 1, 1, loss, 0, nullptr, st);
    if (rc != SPA_OK) return rc;
  }
  return SPA_OK;
}

int launch_pack_bwd_gated(const spa_params& p, const void* dxp, const void* x, const float* scores, const void* dY,
                          const int32_t* idx, const int32_t* cu, void* dX, float* ds, cudaStream_t st) {
  const bool res = (p.flags & SPA_FLAG_RESIDUAL) != 0;
  int grid = (p.capacity + 7) / 8;
  if (grid > kNumSMs * 8) grid = kNumSMs * 8;
#define SPA_GATED(T, R)                                                                                           \
  launch_pdl(pack_bwd_gated_kernel<T, R>, grid, kTrainThreads, 0, st, (const uint4*)dxp, (const uint4*)x, scores, \
             (const uint4*)dY, idx, cu, p.B, p.capacity, p.C / Vec16<T>::kElems, (uint4*)dX, ds)
  if (p.dtype == SPA_F32) { if (res) SPA_GATED(float, true); else SPA_GATED(float, false); }
  else { if (res) SPA_GATED(__nv_bfloat16, true); else SPA_GATED(__nv_bfloat16, false); }
#undef SPA_GATED
  SPA_CUDA_CHECK_LAUNCH("pack_bwd_gated_kernel");
  return SPA_OK;
}

int launch_gate_bwd(const spa_params& p, const void* x, const void* w_g, const float* scores, const float* s_up,
                    const float* ds, void* dX, float* dw_g, float* db_g, float* ds_up, void* workspace,
                    cudaStream_t st) {
  const int rows = p.B * p.N;
  if (rows == 0) return SPA_OK;
  const int grid = gate_bwd_grid(rows);
  float* part = reinterpret_cast<float*>(workspace);
  const size_t smem = ((size_t)p.C + (kTrainThreads / 32) * (p.C + 1)) * sizeof(float);
  if (smem > 48 * 1024 || p.C / (p.dtype == SPA_F32 ? 4 : 8) > 32 * kGbChunks) return SPA_ERR_UNSUPPORTED;
  if (p.dtype == SPA_F32)
    launch_pdl(gate_bwd_kernel<float>, grid, kTrainThreads, smem, st, (const uint4*)x, (const float*)w_g, scores, s_up, ds,
               rows, p.C, (uint4*)dX, ds_up, part);
  else
    launch_pdl(gate_bwd_kernel<__nv_bfloat16>, grid, kTrainThreads, smem, st, (const uint4*)x, (const __nv_bfloat16*)w_g,
               scores, s_up, ds, rows, p.C, (uint4*)dX, ds_up, part);
  SPA_CUDA_CHECK_LAUNCH("gate_bwd_kernel");
  // dw_g[0..C) and db_g (column C of the partials) in one pass over the per-CTA sums
  const int rc = launch_partial_sum(part, grid, p.C + 1, p.C, dw_g, 1, db_g, st);
  if (rc != SPA_OK) return rc;
  return SPA_OK;
}

}  // namespace spa
