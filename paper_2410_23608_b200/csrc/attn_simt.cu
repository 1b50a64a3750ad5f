// fp32-FMA segment-masked attention, forward and backward, on the packed tokens (Sec. 3.2: packed
// tokens attend only to tokens of the same image; the 2L^2C term of Eq. 9).  The path of the fp32
// workload and the bring-up reference of the tensor-core kernels.
//
// Work split: a CTA owns 64 consecutive packed rows and one head, wherever segment boundaries fall;
// it walks the key range spanned by the segments of its rows in tiles of 64 staged in shared memory
// as fp32, and each thread masks the keys outside its own row's segment.  A row is owned by
// kSplit = d/32 adjacent lanes, each holding 32 of the d head dimensions in registers; dot products
// are completed with one shuffle.  No padding token is ever computed, nothing is atomically
// accumulated, and every sum runs in a fixed order.
#include <math_constants.h>

#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kRows = 64;   // packed rows per CTA and rows per staged tile
constexpr int kPart = 32;   // head dimensions held by one thread

// Stage rows [row0, row0 + kRows) of one head's slice (column offset col0 of a [*, ld] matrix) as fp32.
template <typename T, int D>
__device__ __forceinline__ void stage_rows(float (*dst)[D], const T* __restrict__ src, long long ld, int col0, int row0,
                                           int row_end, int tid, int nthreads) {
  constexpr int E = Vec16<T>::kElems;
  constexpr int CPR = D / E;
  for (int c = tid; c < kRows * CPR; c += nthreads) {
    const int r = c / CPR, cc = c % CPR;
    float f[E];
    if (row0 + r < row_end) {
      const uint4 v = *reinterpret_cast<const uint4*>(src + (long long)(row0 + r) * ld + col0 + cc * E);
      Vec16<T>::to_float(v, f);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) f[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < E; ++e) dst[r][cc * E + e] = f[e];
  }
}

template <typename T>
__device__ __forceinline__ void load_part(float* dst, const T* __restrict__ src) {  // kPart contiguous elements
  constexpr int E = Vec16<T>::kElems;
#pragma unroll
  for (int c = 0; c < kPart / E; ++c) Vec16<T>::to_float(*reinterpret_cast<const uint4*>(src + c * E), dst + c * E);
}

template <typename T>
__device__ __forceinline__ void store_part(T* dst, const float* src) {
  constexpr int E = Vec16<T>::kElems;
#pragma unroll
  for (int c = 0; c < kPart / E; ++c) *reinterpret_cast<uint4*>(dst + c * E) = Vec16<T>::from_float(src + c * E);
}

template <int kSplit>
__device__ __forceinline__ float split_sum(float v) {
  if (kSplit >= 2) v += __shfl_xor_sync(0xffffffffu, v, 1);
  if (kSplit >= 4) v += __shfl_xor_sync(0xffffffffu, v, 2);
  return v;
}

__device__ __forceinline__ float dot_part(const float* a, const float* __restrict__ b_smem) {
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < kPart; e += 4) {
    const float4 b = *reinterpret_cast<const float4*>(b_smem + e);
    s = fmaf(a[e], b.x, s); s = fmaf(a[e + 1], b.y, s); s = fmaf(a[e + 2], b.z, s); s = fmaf(a[e + 3], b.w, s);
  }
  return s;
}

__device__ __forceinline__ void axpy_part(float* acc, float w, const float* __restrict__ b_smem) {
#pragma unroll
  for (int e = 0; e < kPart; e += 4) {
    const float4 b = *reinterpret_cast<const float4*>(b_smem + e);
    acc[e] = fmaf(w, b.x, acc[e]); acc[e + 1] = fmaf(w, b.y, acc[e + 1]);
    acc[e + 2] = fmaf(w, b.z, acc[e + 2]); acc[e + 3] = fmaf(w, b.w, acc[e + 3]);
  }
}

// CTA-wide range of "other side" rows: from the segment start of the first row to the segment end
// of the last valid row of this CTA.
__device__ __forceinline__ void cta_range(const RowSeg& mine, int i, int i0, int Np, bool leader, int* range_smem) {
  const int last = (i0 + kRows - 1 < Np - 1) ? i0 + kRows - 1 : Np - 1;
  if (leader && i == i0) range_smem[0] = mine.lo;
  if (leader && i == last) range_smem[1] = mine.hi;
  __syncthreads();
}

// ------------------------------------------------------------------------------------ forward
template <typename T, int D>
__global__ void __launch_bounds__(kRows * (D / kPart))
attn_fwd_simt_kernel(const T* __restrict__ qkv, const int32_t* __restrict__ seg, int n_seg, int capacity, int C,
                     float scale, T* __restrict__ ao, float* __restrict__ lse) {
  pdl_entry();
  constexpr int kSplit = D / kPart;
  constexpr int kThreads = kRows * kSplit;
  __shared__ __align__(16) float Ks[kRows][D];
  __shared__ __align__(16) float Vs[kRows][D];
  __shared__ int range[2];
  const int Np = packed_rows(seg, n_seg, capacity);
  const int i0 = blockIdx.x * kRows;
  if (i0 >= Np) return;
  const int tid = threadIdx.x, r = tid / kSplit, part = tid % kSplit, h = blockIdx.y;
  const int i = i0 + r;
  const long long ld = 3LL * C;
  const RowSeg mine = row_segment(seg, n_seg, Np, i);
  cta_range(mine, i, i0, Np, part == 0, range);
  const int kv_lo = range[0], kv_hi = range[1];

  float q[kPart], o[kPart];
#pragma unroll
  for (int e = 0; e < kPart; ++e) { q[e] = 0.f; o[e] = 0.f; }
  if (i < Np) {
    load_part<T>(q, qkv + (long long)i * ld + h * D + part * kPart);
#pragma unroll
    for (int e = 0; e < kPart; ++e) q[e] *= scale;
  }
  float m = -CUDART_INF_F, l = 0.f;

  for (int kv0 = kv_lo; kv0 < kv_hi; kv0 += kRows) {
    __syncthreads();
    stage_rows<T, D>(Ks, qkv, ld, C + h * D, kv0, kv_hi, tid, kThreads);
    stage_rows<T, D>(Vs, qkv, ld, 2 * C + h * D, kv0, kv_hi, tid, kThreads);
    __syncthreads();
    const int jmax = kv_hi - kv0 < kRows ? kv_hi - kv0 : kRows;
    for (int j0 = 0; j0 < jmax; j0 += 8) {
      float s[8];
      float cm = -CUDART_INF_F;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = j0 + u;  // rows >= jmax are zero-filled and masked below
        float v = split_sum<kSplit>(dot_part(q, &Ks[j][part * kPart]));
        const int ja = kv0 + j;
        s[u] = (j < jmax && ja >= mine.lo && ja < mine.hi) ? v : -CUDART_INF_F;
        cm = fmaxf(cm, s[u]);
      }
      if (cm > -CUDART_INF_F) {
        const float m_new = fmaxf(m, cm);
        const float alpha = expf(m - m_new);
        l *= alpha;
#pragma unroll
        for (int e = 0; e < kPart; ++e) o[e] *= alpha;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float pj = expf(s[u] - m_new);
          l += pj;
          axpy_part(o, pj, &Vs[j0 + u][part * kPart]);
        }
        m = m_new;
      }
    }
  }
  if (i < Np) {
    const float inv_l = 1.f / l;
#pragma unroll
    for (int e = 0; e < kPart; ++e) o[e] *= inv_l;
    store_part<T>(ao + (long long)i * C + h * D + part * kPart, o);
    if (part == 0) lse[(long long)h * capacity + i] = m + logf(l);
  }
}

// ------------------------------------------------------------------------------------ backward, dQ
template <typename T, int D>
__global__ void __launch_bounds__(kRows * (D / kPart))
attn_bwd_dq_simt_kernel(const T* __restrict__ qkv, const T* __restrict__ ao, const float* __restrict__ lse,
                        const T* __restrict__ dao, const int32_t* __restrict__ seg, int n_seg, int capacity, int C,
                        float scale, T* __restrict__ dqkv) {
  pdl_entry();
  constexpr int kSplit = D / kPart;
  constexpr int kThreads = kRows * kSplit;
  __shared__ __align__(16) float Ks[kRows][D];
  __shared__ __align__(16) float Vs[kRows][D];
  __shared__ int range[2];
  const int Np = packed_rows(seg, n_seg, capacity);
  const int i0 = blockIdx.x * kRows;
  if (i0 >= Np) return;
  const int tid = threadIdx.x, r = tid / kSplit, part = tid % kSplit, h = blockIdx.y;
  const int i = i0 + r;
  const long long ld = 3LL * C;
  const RowSeg mine = row_segment(seg, n_seg, Np, i);
  cta_range(mine, i, i0, Np, part == 0, range);
  const int kv_lo = range[0], kv_hi = range[1];

  float q[kPart], dO[kPart], dq[kPart];
  float Di = 0.f, lse_i = 0.f;
#pragma unroll
  for (int e = 0; e < kPart; ++e) { q[e] = 0.f; dO[e] = 0.f; dq[e] = 0.f; }
  if (i < Np) {
    load_part<T>(q, qkv + (long long)i * ld + h * D + part * kPart);
    load_part<T>(dO, dao + (long long)i * C + h * D + part * kPart);
    float ov[kPart];
    load_part<T>(ov, ao + (long long)i * C + h * D + part * kPart);
#pragma unroll
    for (int e = 0; e < kPart; ++e) Di = fmaf(dO[e], ov[e], Di);
    lse_i = lse[(long long)h * capacity + i];
  }
  Di = split_sum<kSplit>(Di);

  for (int kv0 = kv_lo; kv0 < kv_hi; kv0 += kRows) {
    __syncthreads();
    stage_rows<T, D>(Ks, qkv, ld, C + h * D, kv0, kv_hi, tid, kThreads);
    stage_rows<T, D>(Vs, qkv, ld, 2 * C + h * D, kv0, kv_hi, tid, kThreads);
    __syncthreads();
    const int jmax = kv_hi - kv0 < kRows ? kv_hi - kv0 : kRows;
    for (int j = 0; j < jmax; ++j) {
      const float s = scale * split_sum<kSplit>(dot_part(q, &Ks[j][part * kPart]));
      const float dp = split_sum<kSplit>(dot_part(dO, &Vs[j][part * kPart]));
      const int ja = kv0 + j;
      const bool ok = ja >= mine.lo && ja < mine.hi;
      const float pj = ok ? expf(s - lse_i) : 0.f;
      axpy_part(dq, pj * (dp - Di), &Ks[j][part * kPart]);
    }
  }
  if (i < Np) {
#pragma unroll
    for (int e = 0; e < kPart; ++e) dq[e] *= scale;
    store_part<T>(dqkv + (long long)i * ld + h * D + part * kPart, dq);
  }
}

// ------------------------------------------------------------------------------------ backward, dK and dV
template <typename T, int D>
__global__ void __launch_bounds__(kRows * (D / kPart))
attn_bwd_dkv_simt_kernel(const T* __restrict__ qkv, const T* __restrict__ ao, const float* __restrict__ lse,
                         const T* __restrict__ dao, const int32_t* __restrict__ seg, int n_seg, int capacity, int C,
                         float scale, T* __restrict__ dqkv) {
  pdl_entry();
  constexpr int kSplit = D / kPart;
  constexpr int kThreads = kRows * kSplit;
  constexpr int E = Vec16<T>::kElems;
  __shared__ __align__(16) float Qs[kRows][D];
  __shared__ __align__(16) float dOs[kRows][D];
  __shared__ float lse_s[kRows], D_s[kRows];
  __shared__ int range[2];
  const int Np = packed_rows(seg, n_seg, capacity);
  const int j0 = blockIdx.x * kRows;
  if (j0 >= Np) return;
  const int tid = threadIdx.x, r = tid / kSplit, part = tid % kSplit, h = blockIdx.y;
  const int j = j0 + r;
  const long long ld = 3LL * C;
  const RowSeg mine = row_segment(seg, n_seg, Np, j);
  cta_range(mine, j, j0, Np, part == 0, range);
  const int q_lo = range[0], q_hi = range[1];

  float k[kPart], v[kPart], dk[kPart], dv[kPart];
#pragma unroll
  for (int e = 0; e < kPart; ++e) { k[e] = 0.f; v[e] = 0.f; dk[e] = 0.f; dv[e] = 0.f; }
  if (j < Np) {
    load_part<T>(k, qkv + (long long)j * ld + C + h * D + part * kPart);
    load_part<T>(v, qkv + (long long)j * ld + 2 * C + h * D + part * kPart);
  }

  for (int q0 = q_lo; q0 < q_hi; q0 += kRows) {
    __syncthreads();
    stage_rows<T, D>(Qs, qkv, ld, h * D, q0, q_hi, tid, kThreads);
    stage_rows<T, D>(dOs, dao, (long long)C, h * D, q0, q_hi, tid, kThreads);
    if (tid < kRows) {  // D_i = dO_i . O_i and lse_i of the staged query rows
      const int i = q0 + tid;
      float Di = 0.f, li = 0.f;
      if (i < q_hi) {
        const T* orow = ao + (long long)i * C + h * D;
        const T* grow = dao + (long long)i * C + h * D;
#pragma unroll
        for (int c = 0; c < D / E; ++c) {
          float a[E], b[E];
          Vec16<T>::to_float(*reinterpret_cast<const uint4*>(orow + c * E), a);
          Vec16<T>::to_float(*reinterpret_cast<const uint4*>(grow + c * E), b);
#pragma unroll
          for (int e = 0; e < E; ++e) Di = fmaf(a[e], b[e], Di);
        }
        li = lse[(long long)h * capacity + i];
      }
      D_s[tid] = Di;
      lse_s[tid] = li;
    }
    __syncthreads();
    const int imax = q_hi - q0 < kRows ? q_hi - q0 : kRows;
    for (int ii = 0; ii < imax; ++ii) {
      const float s = scale * split_sum<kSplit>(dot_part(k, &Qs[ii][part * kPart]));
      const float dp = split_sum<kSplit>(dot_part(v, &dOs[ii][part * kPart]));
      const int ia = q0 + ii;
      const bool ok = ia >= mine.lo && ia < mine.hi;
      const float pij = ok ? expf(s - lse_s[ii]) : 0.f;
      axpy_part(dv, pij, &dOs[ii][part * kPart]);
      axpy_part(dk, pij * (dp - D_s[ii]), &Qs[ii][part * kPart]);
    }
  }
  if (j < Np) {
#pragma unroll
    for (int e = 0; e < kPart; ++e) dk[e] *= scale;
    store_part<T>(dqkv + (long long)j * ld + C + h * D + part * kPart, dk);
    store_part<T>(dqkv + (long long)j * ld + 2 * C + h * D + part * kPart, dv);
  }
}

template <typename T, int D>
int fwd_launch(const spa_params& p, const void* qkv, const int32_t* seg, int n_seg, void* ao, float* lse,
               cudaStream_t st) {
  dim3 grid((p.capacity + kRows - 1) / kRows, p.H);
  launch_pdl(attn_fwd_simt_kernel<T, D>, grid, kRows * (D / kPart), 0, st, (const T*)qkv, seg, n_seg, p.capacity, p.C,
                                                                  softmax_scale_of(p), (T*)ao, lse);
  SPA_CUDA_CHECK_LAUNCH("attn_fwd_simt_kernel");
  return SPA_OK;
}

template <typename T, int D>
int bwd_launch(const spa_params& p, const void* qkv, const void* ao, const float* lse, const void* dao,
               const int32_t* seg, int n_seg, void* dqkv, cudaStream_t st) {
  dim3 grid((p.capacity + kRows - 1) / kRows, p.H);
  const float scale = softmax_scale_of(p);
  launch_pdl(attn_bwd_dq_simt_kernel<T, D>, grid, kRows * (D / kPart), 0, st, (const T*)qkv, (const T*)ao, lse, (const T*)dao,
                                                                     seg, n_seg, p.capacity, p.C, scale, (T*)dqkv);
  SPA_CUDA_CHECK_LAUNCH("attn_bwd_dq_simt_kernel");
  launch_pdl(attn_bwd_dkv_simt_kernel<T, D>, grid, kRows * (D / kPart), 0, st, (const T*)qkv, (const T*)ao, lse,
                                                                      (const T*)dao, seg, n_seg, p.capacity, p.C,
                                                                      scale, (T*)dqkv);
  SPA_CUDA_CHECK_LAUNCH("attn_bwd_dkv_simt_kernel");
  return SPA_OK;
}

}  // namespace

int launch_attention_fwd_simt(const spa_params& p, const void* qkv, const int32_t* seg, int n_seg, void* ao,
                              float* lse, cudaStream_t st) {
  const int d = p.C / p.H;
  if (p.dtype == SPA_F32)
    return d == 32 ? fwd_launch<float, 32>(p, qkv, seg, n_seg, ao, lse, st)
                   : fwd_launch<float, 64>(p, qkv, seg, n_seg, ao, lse, st);
  return d == 32 ? fwd_launch<__nv_bfloat16, 32>(p, qkv, seg, n_seg, ao, lse, st)
                 : fwd_launch<__nv_bfloat16, 64>(p, qkv, seg, n_seg, ao, lse, st);
}

int launch_attention_bwd_simt(const spa_params& p, const void* qkv, const void* ao, const float* lse,
                              const void* dao, const int32_t* seg, int n_seg, void* dqkv, cudaStream_t st) {
  const int d = p.C / p.H;
  if (p.dtype == SPA_F32)
    return d == 32 ? bwd_launch<float, 32>(p, qkv, ao, lse, dao, seg, n_seg, dqkv, st)
                   : bwd_launch<float, 64>(p, qkv, ao, lse, dao, seg, n_seg, dqkv, st);
  return d == 32 ? bwd_launch<__nv_bfloat16, 32>(p, qkv, ao, lse, dao, seg, n_seg, dqkv, st)
                 : bwd_launch<__nv_bfloat16, 64>(p, qkv, ao, lse, dao, seg, n_seg, dqkv, st);
}

}  // namespace spa
