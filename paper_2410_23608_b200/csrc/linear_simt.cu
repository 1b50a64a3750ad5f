// fp32-FMA linear layers on the packed tokens (QKV / output projection and their gradients; the
// 3LC^2 and NC^2 terms of Eq. 9).  This is the path of the fp32 workload, whose 1e-4 tolerance a
// single-pass reduced-precision tensor-core product cannot meet, and the reference path the
// tensor-core kernels are brought up against.  One generic tiled kernel covers all three products
// by taking element strides:  out[m][n] = sum_k A(m,k) * B(n,k).
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kTile = 64;   // output tile is kTile x kTile
constexpr int kBK = 16;
constexpr int kThreads = 256;

// dyn_which: 0 = sizes as given, 1 = M is the device-side packed row count, 2 = K is.
template <typename T, typename TO>
__global__ void __launch_bounds__(kThreads)
gemm_simt_kernel(const T* __restrict__ A, long long sAm, long long sAk, const T* __restrict__ Bm, long long sBn,
                 long long sBk, const T* __restrict__ bias, TO* __restrict__ out, long long ldo, int M, int N, int K,
                 const int32_t* __restrict__ cu, int n_seg, int capacity, int dyn_which, int accumulate) {
  pdl_entry();
  if (dyn_which != 0) {
    const int rows = packed_rows(cu, n_seg, capacity);
    if (dyn_which == 1) M = rows; else K = rows;
  }
  const int m0 = blockIdx.y * kTile, n0 = blockIdx.x * kTile;
  if (m0 >= M || n0 >= N) return;

  __shared__ __align__(16) float As[kBK][kTile + 4];
  __shared__ __align__(16) float Bs[kBK][kTile + 4];
  const int tid = threadIdx.x;
  const int ty = tid / 16, tx = tid % 16;  // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4] = {};

  for (int k0 = 0; k0 < K; k0 += kBK) {
#pragma unroll
    for (int u = 0; u < (kTile * kBK) / kThreads; ++u) {
      const int e = tid + u * kThreads;
      int m, k;
      if (sAk == 1) { m = e / kBK; k = e % kBK; } else { k = e / kTile; m = e % kTile; }
      float v = 0.f;
      if (m0 + m < M && k0 + k < K) v = to_f32<T>(A[(long long)(m0 + m) * sAm + (long long)(k0 + k) * sAk]);
      As[k][m] = v;
      int n, kk;
      if (sBk == 1) { n = e / kBK; kk = e % kBK; } else { kk = e / kTile; n = e % kTile; }
      float w = 0.f;
      if (n0 + n < N && k0 + kk < K) w = to_f32<T>(Bm[(long long)(n0 + n) * sBn + (long long)(k0 + kk) * sBk]);
      Bs[kk][n] = w;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kBK; ++k) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w};
      const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j];
      if (bias != nullptr) v += to_f32<T>(bias[n]);
      if (accumulate) v += to_f32<TO>(out[(long long)m * ldo + n]);  // residual: the product joins what the row holds
      out[(long long)m * ldo + n] = from_f32<TO>(v);
    }
  }
}

// db[j] = sum over packed rows of dout[i][j], rows added in a fixed order.
template <typename T>
__global__ void __launch_bounds__(kThreads)
colsum_kernel(const T* __restrict__ dout, int n_out, const int32_t* __restrict__ cu, int n_seg, int capacity,
              float* __restrict__ db) {
  pdl_entry();
  const int rows = packed_rows(cu, n_seg, capacity);
  __shared__ float part[4][64];
  const int c = threadIdx.x % 64, g = threadIdx.x / 64;
  const int col = blockIdx.x * 64 + c;
  float s = 0.f;
  if (col < n_out)
    for (int i = g; i < rows; i += 4) s += to_f32<T>(dout[(long long)i * n_out + col]);
  part[g][c] = s;
  __syncthreads();
  if (g == 0 && col < n_out) db[col] = (part[0][c] + part[1][c]) + (part[2][c] + part[3][c]);
}

template <typename T, typename TO>
void launch_gemm(const T* A, long long sAm, long long sAk, const T* Bm, long long sBn, long long sBk, const T* bias,
                 TO* out, long long ldo, int M, int N, int K, const int32_t* cu, int n_seg, int capacity,
                 int dyn_which, cudaStream_t st, int accumulate = 0) {
  dim3 grid((N + kTile - 1) / kTile, (M + kTile - 1) / kTile);
  launch_pdl(gemm_simt_kernel<T, TO>, grid, kThreads, 0, st, A, sAm, sAk, Bm, sBn, sBk, bias, out, ldo, M, N, K, cu, n_seg,
                                                    capacity, dyn_which, accumulate);
}

template <typename T>
int linear_fwd(const spa_params& p, const void* a, const void* W, const void* bias, int n_in, int n_out,
               const int32_t* cu, void* out, cudaStream_t st, bool accumulate) {
  launch_gemm<T, T>((const T*)a, n_in, 1, (const T*)W, n_in, 1, (const T*)bias, (T*)out, n_out, p.capacity, n_out,
                    n_in, cu, p.B, p.capacity, 1, st, accumulate ? 1 : 0);
  SPA_CUDA_CHECK_LAUNCH("gemm_simt_kernel(fwd)");
  return SPA_OK;
}

template <typename T>
int linear_bwd(const spa_params& p, const void* a, const void* W, const void* dout, int n_in, int n_out,
               const int32_t* cu, void* da, float* dW, float* db, cudaStream_t st) {
  if (da != nullptr) {  // da[m][j] = sum_o dout[m][o] W[o][j]
    launch_gemm<T, T>((const T*)dout, n_out, 1, (const T*)W, 1, n_in, nullptr, (T*)da, n_in, p.capacity, n_in, n_out,
                      cu, p.B, p.capacity, 1, st);
    SPA_CUDA_CHECK_LAUNCH("gemm_simt_kernel(dgrad)");
  }
  if (dW != nullptr) {  // dW[o][j] = sum_i dout[i][o] a[i][j]
    launch_gemm<T, float>((const T*)dout, 1, n_out, (const T*)a, 1, n_in, nullptr, dW, n_in, n_out, n_in, p.capacity,
                          cu, p.B, p.capacity, 2, st);
    SPA_CUDA_CHECK_LAUNCH("gemm_simt_kernel(wgrad)");
  }
  if (db != nullptr) {
    launch_pdl(colsum_kernel<T>, (n_out + 63) / 64, kThreads, 0, st, (const T*)dout, n_out, cu, p.B, p.capacity, db);
    SPA_CUDA_CHECK_LAUNCH("colsum_kernel");
  }
  return SPA_OK;
}

}  // namespace

int launch_linear_fwd_simt(const spa_params& p, const void* a, const void* W, const void* bias, int n_in, int n_out,
                           const int32_t* cu, void* out, cudaStream_t st, bool accumulate) {
  return p.dtype == SPA_F32 ? linear_fwd<float>(p, a, W, bias, n_in, n_out, cu, out, st, accumulate)
                            : linear_fwd<__nv_bfloat16>(p, a, W, bias, n_in, n_out, cu, out, st, accumulate);
}

int launch_linear_bwd_simt(const spa_params& p, const void* a, const void* W, const void* dout, int n_in, int n_out,
                           const int32_t* cu, void* da, float* dW, float* db, cudaStream_t st) {
  return p.dtype == SPA_F32 ? linear_bwd<float>(p, a, W, dout, n_in, n_out, cu, da, dW, db, st)
                            : linear_bwd<__nv_bfloat16>(p, a, W, dout, n_in, n_out, cu, da, dW, db, st);
}

}  // namespace spa
