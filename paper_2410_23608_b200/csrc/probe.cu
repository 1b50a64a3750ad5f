// Small diagnostic kernels behind the C boundary: the exponential-unit throughput that bounds attention at small
// head dimensions, a bounded wait that is made to run out so that the error path can be tested, and the cost of
// issuing tensor-core products of the shapes the attention kernels use.
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

// 32 back-to-back tcgen05.mma (M = 128, K = 16, bf16, operands all zero) into one accumulator, issued either by lane 0
// alone or by one elected lane of a warp whose lanes all run the loop; 20 repetitions, the fastest is reported:
// cycles[0] = from the first product to the commit (the issuing thread's time), cycles[1] = until the commit's
// barrier completes.  VAR: 0 = both operands in shared memory, N = 64; 1 = A in TMEM, N = 64; 2 / 3 = shared memory,
// N = 128 / 256.  One CTA; it holds all 512 TMEM columns while it runs.
constexpr int kMmaProbeOps = 32;
template <int VAR, bool kElect>
__global__ void __launch_bounds__(128, 1) mma_issue_probe_kernel(uint32_t* __restrict__ cycles, int32_t* d_status) {
  extern __shared__ uint8_t raw[];
  const uint32_t base = (ptx::smem_u32(raw) + 1023u) & ~1023u;
  uint8_t* al = raw + (base - ptx::smem_u32(raw));
  const uint32_t a_s = base, b_s = base + 16384;  // A: 128 x 64 bf16; B: up to 256 x 64 bf16
  const uint32_t bar = base + 49152;
  volatile uint32_t* slot = reinterpret_cast<volatile uint32_t*>(al + 49152 + 64);
  for (int i = threadIdx.x; i < 49152 / 4; i += 128) reinterpret_cast<uint32_t*>(al)[i] = 0;
  ptx::fence_proxy_async_smem();
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);
    ptx::fence_mbar_init();
  }
  if (threadIdx.x < 32) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(slot)), 512);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *slot;
  constexpr int N = VAR == 2 ? 128 : (VAR == 3 ? 256 : 64);
  constexpr uint32_t kIdesc = ptx::idesc_bf16_f32(128, N, false, VAR == 1);
  if (kElect ? (threadIdx.x < 32) : (threadIdx.x == 0)) {
    const uint64_t ad0 = ptx::smem_desc_sw128(a_s, 16, 1024), bd0 = ptx::smem_desc_sw128(b_s, 16, 1024);
    uint32_t phase = 0, best_issue = 0xffffffffu, best_total = 0xffffffffu;
    bool ok = true;
    for (int r = 0; r < 20 && ok; ++r) {
      const uint32_t t0 = (uint32_t)clock();
      if (!kElect || ptx::elect_one()) {
#pragma unroll
        for (int i = 0; i < kMmaProbeOps; ++i) {
          const int k = i & 3;
          if (VAR == 1) ptx::mma_bf16_ts(tmem, tmem + 448 + k * 8, bd0 + (uint64_t)(k * 128), kIdesc, 1u);  // B MN-major
          else ptx::mma_bf16(tmem, ad0 + (uint64_t)(k * 2), bd0 + (uint64_t)(k * 2), kIdesc, 1u);
        }
        ptx::mma_commit(bar);
      }
      if (kElect) __syncwarp();  // the whole warp is here only in that mode
      const uint32_t t1 = (uint32_t)clock();
      ok = ptx::mbar_wait(bar, phase);
      const uint32_t t2 = (uint32_t)clock();
      phase ^= 1u;
      ptx::tc_fence_after_sync();
      if (t1 - t0 < best_issue) best_issue = t1 - t0;
      if (t2 - t0 < best_total) best_total = t2 - t0;
    }
    if (threadIdx.x == 0) {
      if (!ok) record_status(d_status, SPA_ERR_TIMEOUT);
      cycles[0] = best_issue;
      cycles[1] = best_total;
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x < 32) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem, 512);
  }
}
constexpr int kMmaProbeSmem = 49152 + 1024 + 256;

template <int VAR, bool kElect> int launch_mma_probe(uint32_t* cycles, int32_t* d_status, cudaStream_t st) {
  auto kern = mma_issue_probe_kernel<VAR, kElect>;
  static DeviceOnce attr;
  cudaError_t e = attr.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMmaProbeSmem); });
  if (e != cudaSuccess) { set_cuda_error(e, "mma_issue_probe_kernel"); return SPA_ERR_CUDA; }
  kern<<<1, 128, kMmaProbeSmem, st>>>(cycles, d_status);
  SPA_CUDA_CHECK_LAUNCH("mma_issue_probe_kernel");
  return SPA_OK;
}

}  // namespace
}  // namespace spa

using namespace spa;

extern "C" int spa_probe_mma_issue(int32_t variant, int32_t elected, uint32_t* cycles, int32_t* d_status, void* stream) {
  if (variant < 0 || variant > 3 || cycles == nullptr || d_status == nullptr) return SPA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  switch (variant * 2 + (elected ? 1 : 0)) {
    case 0: return launch_mma_probe<0, false>(cycles, d_status, st);
    case 1: return launch_mma_probe<0, true>(cycles, d_status, st);
    case 2: return launch_mma_probe<1, false>(cycles, d_status, st);
    case 3: return launch_mma_probe<1, true>(cycles, d_status, st);
    case 4: return launch_mma_probe<2, false>(cycles, d_status, st);
    case 5: return launch_mma_probe<2, true>(cycles, d_status, st);
    case 6: return launch_mma_probe<3, false>(cycles, d_status, st);
    default: return launch_mma_probe<3, true>(cycles, d_status, st);
  }
}

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
