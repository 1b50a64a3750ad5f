// Two small diagnostic kernels behind the C boundary: the exponential-unit throughput that bounds attention at small
// head dimensions, and a bounded wait that is made to run out so that the error path can be tested.
#include "sm100_ptx.cuh"
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kProbeThreads = 512;
constexpr int kProbeChains = 8;  // independent exponentials in flight per thread

// Every thread evaluates iters x kProbeChains base-2 exponentials (ex2.approx, the instruction of the softmax
// kernels), each feeding the next one of its chain through one add so that nothing can be hoisted.
__global__ void __launch_bounds__(kProbeThreads) exp2_probe_kernel(int iters, float* __restrict__ sink) {
  float v[kProbeChains];
#pragma unroll
  for (int c = 0; c < kProbeChains; ++c) v[c] = -1.0f - 0.001f * (float)(threadIdx.x + c);
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) v[c] = ptx::ex2_approx(v[c]) - 1.5f;  // stays in (-1.5, -0.5)
  }
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < kProbeChains; ++c) s += v[c];
  if (s == 123.456f) sink[blockIdx.x] = s;  // never true: keeps the loop alive without a store per thread
}

// One warp waits on an mbarrier that nobody arrives at.  The wait gives up after `limit` polls, the kernel records
// SPA_ERR_TIMEOUT in the status word and returns like any other kernel.
__global__ void wait_expiry_kernel(uint32_t limit, int32_t* d_status, int32_t* polls_done) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = ptx::smem_u32(&bar);
  if (threadIdx.x == 0) {
    ptx::mbar_init(b, 1);
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const bool ok = ptx::mbar_wait(b, 0, limit);
  if (threadIdx.x == 0) {
    if (!ok) record_status(d_status, SPA_ERR_TIMEOUT);
    if (polls_done != nullptr) *polls_done = ok ? 0 : (int32_t)limit;
  }
}

}  // namespace
}  // namespace spa

using namespace spa;

extern "C" int spa_probe_exp2(int32_t n_ctas, int32_t iters, float* sink, unsigned long long* n_exp, void* stream) {
  if (n_ctas <= 0 || n_ctas > 65535 || iters <= 0 || sink == nullptr) return SPA_ERR_INVALID_ARG;
  exp2_probe_kernel<<<n_ctas, kProbeThreads, 0, (cudaStream_t)stream>>>(iters, sink);
  SPA_CUDA_CHECK_LAUNCH("exp2_probe_kernel");
  if (n_exp != nullptr) *n_exp = (unsigned long long)n_ctas * kProbeThreads * kProbeChains * (unsigned long long)iters;
  return SPA_OK;
}

extern "C" int spa_probe_wait_expiry(int32_t limit, int32_t* d_status, int32_t* polls_done, void* stream) {
  if (limit <= 0 || limit > (1 << 20) || d_status == nullptr) return SPA_ERR_INVALID_ARG;
  wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((uint32_t)limit, d_status, polls_done);
  SPA_CUDA_CHECK_LAUNCH("wait_expiry_kernel");
  return SPA_OK;
}
