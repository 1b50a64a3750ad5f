// Shared device/host helpers of the SPA kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "spa.h"

namespace spa {

constexpr int kNumSMs = 148;  // B200: two dies of 74 SMs

// Number of valid packed rows: the device-resident total, clamped to the allocated rows.
__device__ __forceinline__ int packed_rows(const int32_t* __restrict__ offsets, int n_seg, int capacity) {
  int n = __ldg(offsets + n_seg);
  return n < capacity ? n : capacity;
}

__device__ __forceinline__ void record_status(int32_t* d_status, int code) {
  if (d_status != nullptr) atomicCAS(d_status, 0, code);
}

// Programmatic dependent launch: every kernel lets its successor in the stream start being scheduled at
// once, and itself waits for its predecessor's results before touching global memory.  Launch
// latency and CTA ramp-up of the next kernel overlap the tail of this one.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_entry() { pdl_launch_dependents(); pdl_wait(); }

// ---- 16-byte vector access, converted to fp32 ------------------------------------------------
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int kElems = 4;
  __device__ static __forceinline__ void to_float(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ uint4 from_float(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static __forceinline__ void to_float(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // a bf16 is the high half of an fp32
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ uint4 from_float(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ uint4 ld_nc16(const void* p) {  // streaming 16-byte load
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Segment containing packed row i: the s with offsets[s] <= i < offsets[s+1] (empty segments are skipped).
__device__ __forceinline__ int find_segment(const int32_t* __restrict__ offsets, int n_seg, int i) {
  int lo = 0, hi = n_seg;  // invariant: offsets[lo] <= i < offsets[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(offsets + mid) <= i) lo = mid; else hi = mid;
  }
  return lo;
}

struct RowSeg { int lo, hi; };

// Segment bounds of packed row i (hi clamped to the valid rows); rows >= Np get an empty range.
__device__ __forceinline__ RowSeg row_segment(const int32_t* __restrict__ seg, int n_seg, int Np, int i) {
  RowSeg r{0, 0};
  if (i < Np) {
    const int s = find_segment(seg, n_seg, i);
    r.lo = __ldg(seg + s);
    const int hi = __ldg(seg + s + 1);
    r.hi = hi < Np ? hi : Np;
  }
  return r;
}

// ---- host side -------------------------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char* where);
void count_launch();  // one more kernel of this library was enqueued (host-side tally)
#define SPA_CUDA_CHECK_LAUNCH(where)                                   \
  do {                                                                 \
    cudaError_t e__ = cudaGetLastError();                              \
    if (e__ != cudaSuccess) { ::spa::set_cuda_error(e__, where); return SPA_ERR_CUDA; } \
    ::spa::count_launch();                                             \
  } while (0)

// Set-up that a kernel needs once on every device that runs it (the opt-in to more than 48 KB of dynamic shared
// memory is a per-device attribute of the function).  run(fn) calls fn with the current device the first time that
// device is seen and never again once fn has returned cudaSuccess; safe to call from several host threads.
class DeviceOnce {
 public:
  template <typename F> cudaError_t run(F&& fn) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (done_.load(std::memory_order_acquire) & bit) return cudaSuccess;
    e = fn();
    if (e == cudaSuccess) done_.fetch_or(bit, std::memory_order_release);
    return e;
  }
 private:
  std::atomic<unsigned long long> done_{0};
};

bool pdl_enabled();  // programmatic dependent launch is on unless the environment sets SPA_PDL=0

// Launch `kern` on `st`, allowing it to overlap the tail of the previous kernel of the stream.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// launchers implemented per .cu file; every one enqueues on `st` and returns a spa_status
int launch_gate(const spa_params& p, const void* x, const void* w_g, float b_g, const float* s_up,
                float* scores, uint8_t* mask, void* y, cudaStream_t st);
int launch_select_pack(const spa_params& p, const void* x, const uint8_t* mask, const float* scores,
                       const int32_t* order, void* xp, int32_t* idx, int32_t* inv, int32_t* cu, int32_t* d_status,
                       cudaStream_t st);
// gate + selection + packing in one kernel (gate_pack.cu); y may be NULL (no pass-through copy)
bool gate_pack_supported(const spa_params& p);
size_t gate_pack_state_bytes(const spa_params& p);
int launch_gate_pack(const spa_params& p, const void* x, const void* w_g, float b_g, const float* s_up, float* scores,
                     uint8_t* mask, void* y, void* xp, int32_t* idx, int32_t* inv, int32_t* cu, void* state,
                     int32_t* d_status, cudaStream_t st);
int launch_container_offsets(const spa_params& p, const int32_t* cu, int L, int n_max, int32_t* out, cudaStream_t st);
int launch_unpack_scatter(const spa_params& p, const void* z, const void* x, const int32_t* idx,
                          const int32_t* inv, const int32_t* cu, void* y, cudaStream_t st);
int launch_unpack_scatter_bwd(const spa_params& p, const void* dY, const int32_t* idx, const int32_t* inv,
                              const int32_t* cu, void* dz, void* dX, cudaStream_t st);
int launch_select_pack_bwd(const spa_params& p, const void* dxp, const void* dY, const int32_t* idx,
                           const int32_t* cu, void* dX, cudaStream_t st);
// trainable selection (select_train.cu)
size_t train_workspace_bytes(const spa_params& p);
int launch_score_pool(const float* prev, int B, int rows, int cols, float* s_up, cudaStream_t st);
int launch_select_loss(const spa_params& p, const float* scores, const uint8_t* labels, float alpha, float* ds,
                       float* loss, void* workspace, cudaStream_t st);
int launch_pack_bwd_gated(const spa_params& p, const void* dxp, const void* x, const float* scores, const void* dY,
                          const int32_t* idx, const int32_t* cu, void* dX, float* ds, cudaStream_t st);
int launch_gate_bwd(const spa_params& p, const void* x, const void* w_g, const float* scores, const float* s_up,
                    const float* ds, void* dX, float* dw_g, float* db_g, float* ds_up, void* workspace,
                    cudaStream_t st);
// out[j] = sum over blocks (fixed order) of part[block * stride + j], j < n_out; the next n_out2 columns go to out2
int launch_partial_sum(const float* part, int n_blocks, int stride, int n_out, float* out, int n_out2, float* out2,
                       cudaStream_t st);
// the rest of the transformer block (block_rest.cu)
size_t layer_norm_workspace_bytes(const spa_params& p);
bool layer_norm_supported(const spa_params& p);
int launch_layer_norm(const spa_params& p, const void* x, const void* gamma, const void* beta, float eps, void* y,
                      float* mean, float* rstd, cudaStream_t st);
int launch_layer_norm_bwd(const spa_params& p, const void* dy, const void* x, const void* gamma, const float* mean,
                          const float* rstd, const void* add, void* dx, float* dgamma, float* dbeta, void* workspace,
                          cudaStream_t st);
int launch_gelu(const spa_params& p, const void* u, const void* dh, int n_cols, void* out, cudaStream_t st);
int launch_copy_tokens(const spa_params& p, const void* src, void* dst, cudaStream_t st);  // dst[B*N][C] = src

// out[M][n_out] = a[M][n_in] W[n_out][n_in]^T + bias, M = packed rows (device)
int launch_linear_fwd_simt(const spa_params& p, const void* a, const void* W, const void* bias, int n_in,
                           int n_out, const int32_t* cu, void* out, cudaStream_t st, bool accumulate = false);
int launch_linear_bwd_simt(const spa_params& p, const void* a, const void* W, const void* dout, int n_in,
                           int n_out, const int32_t* cu, void* da, float* dW, float* db, cudaStream_t st);
int launch_attention_fwd_simt(const spa_params& p, const void* qkv, const int32_t* seg, int n_seg, void* ao,
                              float* lse, cudaStream_t st);
int launch_attention_bwd_simt(const spa_params& p, const void* qkv, const void* ao, const float* lse,
                              const void* dao, const int32_t* seg, int n_seg, void* dqkv, cudaStream_t st);

inline float softmax_scale_of(const spa_params& p) {
  return p.softmax_scale != 0.f ? p.softmax_scale : 1.0f / sqrtf((float)(p.C / p.H));
}

}  // namespace spa
