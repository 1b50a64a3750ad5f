// bf16 linear layers on CTA pairs: the forward product and the input gradient of the wide layers
// (the 3LC^2 and NC^2 terms of Eq. 9 at C >= 512) with one tcgen05.mma spanning two SMs.
//
// A 128 x 128 tile per CTA needs 32 KB of operands for every 2 x 128 x 128 x 64 flops and is bound by the
// L2-to-SM operand feed at about half of the tensor pipe.  Here two CTAs of a cluster share one
// 256 x 256 tile: CTA r holds rows [128 r, 128 r + 128) of A and of the accumulator, and one half
// (128 of the 256 N positions) of B; the pair's MMA (cta_group::2, M = 256, N = 256) reads both
// halves of B from the two CTAs' shared memory.  Per CTA that is the same 32 KB per k-block for
// twice the flops.  Operand stages are filled by each CTA's own TMA loads (no multicast); all
// transaction bytes are counted on the leader CTA's barrier, whose MMA warp issues for the pair;
// tcgen05.commit releases the stage in both CTAs.  Two 256-column accumulators per CTA (all 512 TMEM
// columns) let the epilogue of one tile run under the main loop of the next.
//
// Barriers (s = stage, a = accumulator):
//   full[s]        leader only, 2 arrivals (one expect_tx per CTA) + the bytes of both CTAs' loads
//   empty[s]       both CTAs, 1 arrival: commit of the MMAs that read stage s (multicast to the pair)
//   tmem_full[a]   both CTAs, 1 arrival: commit after the last k-block of a tile (multicast)
//   tmem_empty[a]  leader only, 16 arrivals: the eight epilogue warps of each CTA
// Every wait is bounded; the two cluster-wide barriers (after set-up, before exit) are reached by every
// thread on every path, so a CTA never leaves while its peer may still touch its shared memory.
#include "sm100_ptx.cuh"
#include "spa_tc.cuh"

namespace spa {
namespace {

namespace ptx2 {
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive (and add expected bytes) on a barrier that may live in the peer CTA
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// tiled load into this CTA's shared memory, completion counted on a barrier of the pair (leader's)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t cluster_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(cluster_bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem, both CTAs] (+)= A * B with A, B in the shared memory of both CTAs; issued by one thread of the leader
__device__ __forceinline__ void mma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                              uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(z) : "memory");
}
// arrive on the barrier at this offset in both CTAs once every MMA issued so far has completed
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
}  // namespace ptx2

constexpr int PM = 128;            // rows of A and of the accumulator per CTA
constexpr int PN = 256;            // N of the pair's tile; each CTA stages PN / 2 positions of B
constexpr int PK = 64;             // k-block
constexpr int kPairStages = 5;
constexpr int kPairEpiWarps = 8;   // two per TMEM lane quarter: they split the 32-column groups of a tile
constexpr int kPairThreads = 64 + 32 * kPairEpiWarps;  // warp 0: TMA, warp 1: MMA (leader) + TMEM owner, then the epilogue warps
constexpr int kPairStage = PM * PK * 2 + (PN / 2) * PK * 2;  // 32 KB
constexpr int kPairSmem = kPairStages * kPairStage + 1024 + 256 + kPairEpiWarps * 2048;  // ring, alignment slack, barriers, transposition

// kBMn: B = W is MN-major (input gradient: K = n_out rows of W, N = n_in contiguous); otherwise K-major
// (forward: N = n_out rows of W, K = n_in contiguous).  A is always K-major, the output bf16.
// M is the device-side packed row count.  row_map / accumulate as in the single-CTA kernel.
template <bool kBMn>
__global__ void __launch_bounds__(kPairThreads)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ out, long long ldo, int N, int K,
                 const int32_t* __restrict__ cu, int n_seg, int capacity, const int32_t* __restrict__ row_map,
                 int accumulate, int32_t* d_status) {
  constexpr uint32_t kIdesc = ptx::idesc_bf16_f32(2 * PM, PN, false, kBMn);
  pdl_launch_dependents();

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kPairStages * kPairStage;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kPairStages + s); };
  auto tmem_full_bar = [&](int a) { return bar_base + 8u * (2 * kPairStages + a); };
  auto tmem_empty_bar = [&](int a) { return bar_base + 8u * (2 * kPairStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_al + kPairStages * kPairStage + 192);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_al + kPairStages * kPairStage + 196);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx2::cluster_ctarank();   // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    for (int s = 0; s < kPairStages; ++s) {
      ptx::mbar_init(full_bar(s), 2);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(tmem_full_bar(a), 1); ptx::mbar_init(tmem_empty_bar(a), 2 * kPairEpiWarps); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) ptx2::tmem_alloc_pair(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), 2 * PN);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx2::cluster_sync();  // both CTAs' barriers exist before either signals the other
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  pdl_wait();  // everything above touched no global memory
  const int M = packed_rows(cu, n_seg, capacity);
  const int tiles_n = (N + PN - 1) / PN;
  const int tiles_m = (M + 2 * PM - 1) / (2 * PM);
  const int total = tiles_m * tiles_n;
  const int k_blocks = (K + PK - 1) / PK;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one per CTA)
    if (lane == 0) {
      int it = 0;
      for (int tile = pair; tile < total && !*abort_flag; tile += n_pairs) {
        const int m0 = (tile / tiles_n) * 2 * PM + (int)rank * PM;
        const int n0 = (tile % tiles_n) * PN + (int)rank * (PN / 2);
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % kPairStages;
          if (it >= kPairStages && !ptx::mbar_wait(empty_bar(s), ((it / kPairStages) - 1) & 1)) {
            record_status(d_status, SPA_ERR_TIMEOUT);
            *abort_flag = 1;
          }
          if (*abort_flag) break;
          const uint32_t a_dst = smem_base + s * kPairStage, b_dst = a_dst + PM * PK * 2;
          const uint32_t lead_full = ptx2::map_to_cta(full_bar(s), 0);
          ptx2::mbar_expect_tx_cluster(lead_full, kPairStage);
          const int k0 = kb * PK;
          ptx2::tma_load_2d_pair(a_dst, &tmA, lead_full, k0, m0);
          if (!kBMn) {
            ptx2::tma_load_2d_pair(b_dst, &tmB, lead_full, k0, n0);
          } else {
#pragma unroll
            for (int j = 0; j < PN / 2 / 64; ++j)
              ptx2::tma_load_2d_pair(b_dst + j * (PK * 128), &tmB, lead_full, n0 + 64 * j, k0);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the leader's, for the pair
    if (rank == 0) {
      int it = 0, tl = 0;
      bool dead = false;
      for (int tile = pair; tile < total && !dead; tile += n_pairs, ++tl) {
        if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
        const int acc = tl & 1;
        if (tl >= 2 && !__all_sync(0xffffffffu, ptx::mbar_wait(tmem_empty_bar(acc), ((tl >> 1) - 1) & 1))) {
          if (lane == 0) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_flag = 1; }
          break;
        }
        ptx::tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + acc * PN;
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const int s = it % kPairStages;
          if (__any_sync(0xffffffffu, *abort_flag != 0)) { dead = true; break; }
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(full_bar(s), (it / kPairStages) & 1))) {
            if (lane == 0) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_flag = 1; }
            dead = true;
            break;
          }
          ptx::tc_fence_after_sync();
          const uint32_t a_src = smem_base + s * kPairStage, b_src = a_src + PM * PK * 2;
          if (lane == 0) {
#pragma unroll
            for (int k = 0; k < PK / 16; ++k) {
              const uint64_t adesc = ptx::smem_desc_sw128(a_src + k * 32, 16, 1024);
              const uint64_t bdesc = kBMn ? ptx::smem_desc_sw128(b_src + k * 2048, PK * 128, 1024)
                                          : ptx::smem_desc_sw128(b_src + k * 32, 16, 1024);
              ptx2::mma_bf16_pair(tmem_d, adesc, bdesc, kIdesc, (kb == 0 && k == 0) ? 0u : 1u);
            }
            ptx2::mma_commit_pair(empty_bar(s));
          }
          __syncwarp();
        }
        if (lane == 0 && !dead && k_blocks > 0) ptx2::mma_commit_pair(tmem_full_bar(acc));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;  // which of the two warps of that quarter: even or odd 32-column groups
    uint8_t* stage = smem_al + kPairStages * kPairStage + 256 + (warp - 2) * 2048;  // this warp's transposition buffer
    const uint32_t lead_empty[2] = {ptx2::map_to_cta(tmem_empty_bar(0), 0), ptx2::map_to_cta(tmem_empty_bar(1), 0)};
    const int my_chunk = lane & 3, my_row = lane >> 2;
    int tl = 0;
    for (int tile = pair; tile < total; tile += n_pairs, ++tl) {
      if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
      const int m0 = (tile / tiles_n) * 2 * PM + (int)rank * PM;
      const int n0 = (tile % tiles_n) * PN;
      const int acc = tl & 1;
      const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(tmem_full_bar(acc), (tl >> 1) & 1) && !*abort_flag);
      if (!ok) {
        if (lane == 0) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_flag = 1; }
        break;
      }
      ptx::tc_fence_after_sync();
      long long orow[4];  // destination rows of the four rows this lane stores
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int grow = m0 + q * 32 + my_row + 8 * j;
        orow[j] = (row_map != nullptr && grow < M) ? (long long)__ldg(row_map + grow) : (long long)grow;
      }
#pragma unroll 1
      for (int cc = half; cc < PN / 32; cc += 2) {
        if (n0 + cc * 32 >= N) break;  // warp-uniform: columns past the layer's width
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * PN + cc * 32, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // 16-byte chunk i of this row's 64-byte segment
          float v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[i * 8 + e]);
          const int col = n0 + cc * 32 + i * 8;
          if (bias != nullptr && col < N) {
            float b[8];
            Vec16<__nv_bfloat16>::to_float(__ldg(reinterpret_cast<const uint4*>(bias + col)), b);
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] += b[e];
          }
          *reinterpret_cast<uint4*>(stage + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)) = Vec16<__nv_bfloat16>::from_float(v);
        }
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int rr = my_row + 8 * j;
          const uint4 v4 = *reinterpret_cast<const uint4*>(stage + rr * 64 + ((my_chunk ^ ((rr >> 1) & 3)) << 4));
          const int grow = m0 + q * 32 + rr;
          const int gcol = n0 + cc * 32 + my_chunk * 8;
          if (grow < M && gcol < N) {
            uint4* dst = reinterpret_cast<uint4*>(out + orow[j] * ldo + gcol);
            if (accumulate) {
              float fa[8], fb[8];
              Vec16<__nv_bfloat16>::to_float(*dst, fa);
              Vec16<__nv_bfloat16>::to_float(v4, fb);
#pragma unroll
              for (int e = 0; e < 8; ++e) fa[e] += fb[e];
              *dst = Vec16<__nv_bfloat16>::from_float(fa);
            } else {
              *dst = v4;
            }
          }
        }
        __syncwarp();
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx2::mbar_arrive_cluster(lead_empty[acc]);  // this warp has drained its quarter of the accumulator
    }
  }
  // nobody leaves while the peer may still read this CTA's operands or signal its barriers
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx2::cluster_sync();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx2::tmem_dealloc_pair(tmem_base, 2 * PN);
  }
}

constexpr int kMaxPairs = kNumSMs / 2;

template <bool kBMn>
int launch_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const __nv_bfloat16* bias, __nv_bfloat16* out, long long ldo,
                int N, int K, const int32_t* cu, int n_seg, int capacity, const int32_t* row_map, int accumulate,
                int32_t* d_status, cudaStream_t st, const char* what) {
  auto kern = gemm_pair_kernel<kBMn>;
  static DeviceOnce smem_attr;  // per instantiation and device
  cudaError_t ea = smem_attr.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem); });
  if (ea != cudaSuccess) { set_cuda_error(ea, what); return SPA_ERR_CUDA; }
  const long long tiles = (long long)((N + PN - 1) / PN) * ((capacity + 2 * PM - 1) / (2 * PM));
  const int pairs = (int)(tiles < kMaxPairs ? (tiles < 1 ? 1 : tiles) : kMaxPairs);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = kPairSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, bias, out, ldo, N, K, cu, n_seg, capacity, row_map, accumulate,
                                     d_status);
  if (e != cudaSuccess) { set_cuda_error(e, what); return SPA_ERR_CUDA; }
  SPA_CUDA_CHECK_LAUNCH(what);
  return SPA_OK;
}

}  // namespace

// The pair kernels pay off where the 128 x 128 tiles are operand-feed bound: wide layers with enough
// rows for several 256 x 256 tiles per pair.
bool tc_pair_linear_supported(const spa_params& p, int n_in, int n_out) {
  if (p.flags & SPA_FLAG_NO_CTA_PAIRS) return false;
  return n_in % 8 == 0 && n_out % 8 == 0 && n_in >= 512 && n_out >= 512 && p.capacity >= 4096 && tensor_maps_available();
}

int launch_linear_fwd_pair(const spa_params& p, const void* a, const void* W, const void* bias, int n_in, int n_out,
                           const int32_t* cu, void* out, int32_t* d_status, cudaStream_t st, const int32_t* row_map,
                           bool accumulate) {
  CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, a, n_in, p.capacity, (uint64_t)n_in * 2, PK, PM) ||
      !make_tmap_bf16_2d(&tmB, W, n_in, n_out, (uint64_t)n_in * 2, PK, PN / 2))
    return SPA_ERR_UNSUPPORTED;
  return launch_pair<false>(tmA, tmB, (const __nv_bfloat16*)bias, (__nv_bfloat16*)out, n_out, n_out, n_in, cu, p.B, p.capacity,
                            row_map, accumulate ? 1 : 0, d_status, st, "gemm_pair_kernel(fwd)");
}

// da[M][n_in] = dout[M][n_out] W[n_out][n_in]
int launch_linear_dgrad_pair(const spa_params& p, const void* W, const void* dout, int n_in, int n_out, const int32_t* cu,
                             void* da, int32_t* d_status, cudaStream_t st, const int32_t* row_map, bool accumulate) {
  CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, dout, n_out, p.capacity, (uint64_t)n_out * 2, PK, PM) ||
      !make_tmap_bf16_2d(&tmB, W, n_in, n_out, (uint64_t)n_in * 2, 64, PK))
    return SPA_ERR_UNSUPPORTED;
  return launch_pair<true>(tmA, tmB, nullptr, (__nv_bfloat16*)da, n_in, n_in, n_out, cu, p.B, p.capacity, row_map,
                           accumulate ? 1 : 0, d_status, st, "gemm_pair_kernel(dgrad)");
}

}  // namespace spa
