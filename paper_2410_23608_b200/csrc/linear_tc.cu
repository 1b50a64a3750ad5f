// bf16 linear layers on the packed tokens as tcgen05 GEMMs: QKV / output projection (the 3LC^2 and
// NC^2 terms of Eq. 9), their input gradients and their weight gradients.
//
// One kernel, three operand arrangements.  D[128 x BN] tiles accumulate in TMEM (fp32); operands
// are staged by TMA into 128-byte-swizzled shared memory through a ring of kStages buffers; one
// thread issues tcgen05.mma, one thread issues TMA, four warps drain TMEM and store.
//   forward   out = a W^T      A = a    (K-major),  B = W   (K-major),  M = packed rows (device)
//   dgrad     da  = dout W     A = dout (K-major),  B = W   (MN-major), M = packed rows (device)
//   wgrad     dW  = dout^T a   A = dout (MN-major), B = a   (MN-major), K = packed rows (device)
// The packed row count N_p lives on the device: grids are sized for `capacity` rows and CTAs
// beyond N_p exit at once.  wgrad splits K = N_p across CTAs; each split writes an fp32 partial to
// the workspace and a second kernel adds the partials in a fixed order (no float atomics, bitwise
// reproducible).  Rows of the last K block that lie beyond N_p are zeroed in shared memory before
// the MMA reads them, so unspecified rows of the packed buffers never reach a sum.
#include <mutex>
#include <string>
#include <unordered_map>

#include "sm100_ptx.cuh"
#include "spa_tc.cuh"

namespace spa {

// ------------------------------------------------------------------------------ tensor maps
namespace {
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = []() -> EncodeFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeFn>(p);
  }();
  return fn;
}

std::mutex g_tm_mutex;
std::unordered_map<std::string, CUtensorMap> g_tm_cache;
}  // namespace

bool tensor_maps_available() { return encode_fn() != nullptr; }

bool make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t rows, uint64_t row_stride_bytes,
                       uint32_t box_inner, uint32_t box_rows, int swizzle_bytes) {
  struct Key { const void* b; uint64_t i, r, s; uint32_t bi, br; int sw; int pad; } key{base, inner, rows, row_stride_bytes,
                                                                                     box_inner, box_rows, swizzle_bytes, 0};
  std::string k(reinterpret_cast<const char*>(&key), sizeof(key));
  std::lock_guard<std::mutex> lock(g_tm_mutex);
  auto it = g_tm_cache.find(k);
  if (it != g_tm_cache.end()) { *out = it->second; return true; }
  EncodeFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (g_tm_cache.size() > 4096) g_tm_cache.clear();
  g_tm_cache.emplace(std::move(k), *out);
  return true;
}

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kStages = 3;
constexpr int kGemmThreads = 192;  // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int kABytes = BM * BK * 2;

template <int BN> __host__ __device__ constexpr int stage_bytes() { return kABytes + BN * BK * 2; }
// operand ring, alignment slack, barriers, 2 KB per epilogue warp for the output transposition
template <int BN> __host__ __device__ constexpr int gemm_smem_bytes() { return kStages * stage_bytes<BN>() + 1024 + 128 + 4 * 2048; }

// Tile bookkeeping shared by the three roles of the persistent kernel.
struct TileCoord { int m0, n0, z, n_t; };

// dyn_which: 1 = M is the device-side packed row count, 2 = K is.
// Persistent: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... of the (m, n, split) space
// that the device-side row count leaves; two accumulator stages in TMEM let the epilogue of one tile
// overlap the main loop of the next, and the TMA ring runs ahead across tile boundaries.
// row_map (optional): output row i goes to row row_map[i] of `out` (the unpack scatter fused into the
// epilogue); with `accumulate` the bf16 result is added to what that row holds.
template <int BN, bool kAMn, bool kBMn, typename OutT>
__global__ void __launch_bounds__(kGemmThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __nv_bfloat16* __restrict__ bias, OutT* __restrict__ out, long long ldo,
               long long split_stride, int M, int N, int K, const int32_t* __restrict__ cu, int n_seg, int capacity,
               int dyn_which, int k_per_split, int k_interleave, const int32_t* __restrict__ row_map,
               int accumulate, int32_t* d_status) {
  constexpr int kStage = stage_bytes<BN>();
  constexpr uint32_t kIdesc = ptx::idesc_bf16_f32(BM, BN, kAMn, kBMn);
  pdl_launch_dependents();

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStage;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tmem_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tmem_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_al + kStages * kStage + 96);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_al + kStages * kStage + 100);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(tmem_full_bar(a), 1); ptx::mbar_init(tmem_empty_bar(a), 4); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), 2 * BN);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  pdl_wait();  // everything above touched no global memory; the predecessor's results are needed from here on
  {
    const int rows = packed_rows(cu, n_seg, capacity);
    if (dyn_which == 1) M = rows; else if (dyn_which == 2) K = rows;
  }
  const int tiles_n = (N + BN - 1) / BN;
  const int tiles_m = (M + BM - 1) / BM;
  // Split-K: contiguous spans of k_per_split, or (k_interleave > 0) that many splits dealt the BK-blocks of K in
  // turn - split z takes blocks z, z + splits, ... - so that the splits get equal work whatever K turns out to be.
  const int k_blocks = (K + BK - 1) / BK;
  const int n_splits = k_interleave > 0 ? (k_blocks < k_interleave ? k_blocks : k_interleave)
                                        : (K > 0 ? (K + k_per_split - 1) / k_per_split : 0);
  const int total = tiles_m * tiles_n * n_splits;
  auto coord = [&](int tile) {
    TileCoord c;
    c.n_t = tile % tiles_n;
    const int rest = tile / tiles_n;
    c.m0 = (rest % tiles_m) * BM;
    c.z = rest / tiles_m;
    c.n0 = c.n_t * BN;
    return c;
  };
  auto k_range = [&](int z, int& k_begin, int& k_end, int& k_step) {
    if (k_interleave > 0) {
      k_begin = z * BK;
      k_end = K;
      k_step = n_splits * BK;
    } else {
      k_begin = z * k_per_split;
      k_end = k_begin + k_per_split;
      if (k_end > K) k_end = K;
      k_step = BK;
    }
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int it = 0;  // k-block counter over all tiles of this CTA: ring position and phase
      for (int tile = blockIdx.x; tile < total && !*abort_flag; tile += gridDim.x) {
        const TileCoord c = coord(tile);
        int k_begin, k_end, k_step;
        k_range(c.z, k_begin, k_end, k_step);
        for (int k0 = k_begin; k0 < k_end; k0 += k_step, ++it) {
          const int s = it % kStages;
          if (it >= kStages && !ptx::mbar_wait(empty_bar(s), ((it / kStages) - 1) & 1)) {
            record_status(d_status, SPA_ERR_TIMEOUT);
            *abort_flag = 1;
          }
          if (*abort_flag) break;
          const uint32_t a_dst = smem_base + s * kStage, b_dst = a_dst + kABytes;
          ptx::mbar_expect_tx(full_bar(s), kStage);
          if (!kAMn) {
            ptx::tma_load_2d(a_dst, &tmA, full_bar(s), k0, c.m0);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j)
              ptx::tma_load_2d(a_dst + j * (BK * 128), &tmA, full_bar(s), c.m0 + 64 * j, k0);
          }
          if (!kBMn) {
            ptx::tma_load_2d(b_dst, &tmB, full_bar(s), k0, c.n0);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)
              ptx::tma_load_2d(b_dst + j * (BK * 128), &tmB, full_bar(s), c.n0 + 64 * j, k0);
          }
        }
      }
      if (*abort_flag) {  // let our own copies land before the CTA's shared memory goes away
        for (int j = it > kStages ? it - kStages : 0; j < it; ++j)
          ptx::mbar_wait(full_bar(j % kStages), (j / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    int it = 0, tl = 0;  // k-block counter, tile counter of this CTA
    bool dead = false;   // warp-uniform: a wait of this warp ran out, or another role gave up
    for (int tile = blockIdx.x; tile < total && !dead; tile += gridDim.x, ++tl) {
      if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
      const TileCoord c = coord(tile);
      int k_begin, k_end, k_step;
      k_range(c.z, k_begin, k_end, k_step);
      const int acc = tl & 1;
      if (tl >= 2 && !__all_sync(0xffffffffu, ptx::mbar_wait(tmem_empty_bar(acc), ((tl >> 1) - 1) & 1))) {
        if (lane == 0) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_flag = 1; }
        break;
      }
      ptx::tc_fence_after_sync();
      const uint32_t tmem_d = tmem_base + acc * BN;
      bool first = true;
      for (int k0 = k_begin; k0 < k_end; k0 += k_step, ++it) {
        const int s = it % kStages;
        if (__any_sync(0xffffffffu, *abort_flag != 0)) { dead = true; break; }
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(full_bar(s), (it / kStages) & 1))) {
          if (lane == 0) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_flag = 1; }
          dead = true;
          break;
        }
        const uint32_t a_src = smem_base + s * kStage, b_src = a_src + kABytes;
        const int k_valid = k_end - k0;
        if ((kAMn || kBMn) && k_valid < BK) {
          // K rows beyond the end of the reduction: zero them (a K row is one 128-byte line per 64-wide box)
          const int n_lines = BK - k_valid;
          if (kAMn)
            for (int j = 0; j < BM / 64; ++j)
              for (int q = lane; q < n_lines * 8; q += 32)
                *reinterpret_cast<uint4*>(smem_al + s * kStage + j * (BK * 128) + (k_valid + q / 8) * 128 + (q % 8) * 16) =
                    make_uint4(0, 0, 0, 0);
          if (kBMn)
            for (int j = 0; j < BN / 64; ++j)
              for (int q = lane; q < n_lines * 8; q += 32)
                *reinterpret_cast<uint4*>(smem_al + s * kStage + kABytes + j * (BK * 128) + (k_valid + q / 8) * 128 +
                                          (q % 8) * 16) = make_uint4(0, 0, 0, 0);
          ptx::fence_proxy_async_smem();
          __syncwarp();
        }
        ptx::tc_fence_after_sync();
        if (ptx::elect_one()) {  // one lane of the converged warp issues: the descriptors stay in uniform registers
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t adesc = kAMn ? ptx::smem_desc_sw128(a_src + k * 2048, BK * 128, 1024)
                                        : ptx::smem_desc_sw128(a_src + k * 32, 16, 1024);
            const uint64_t bdesc = kBMn ? ptx::smem_desc_sw128(b_src + k * 2048, BK * 128, 1024)
                                        : ptx::smem_desc_sw128(b_src + k * 32, 16, 1024);
            ptx::mma_bf16(tmem_d, adesc, bdesc, kIdesc, (first && k == 0) ? 0u : 1u);
          }
          ptx::mma_commit(empty_bar(s));
        }
        first = false;
        __syncwarp();
      }
      if (!first && ptx::elect_one()) ptx::mma_commit(tmem_full_bar(acc));  // the same lane as above: it covers its products
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;          // TMEM lane quarter this warp may read
    uint8_t* stage = smem_al + kStages * kStage + 128 + (warp - 2) * 2048;  // this warp's transposition buffer
    int tl = 0;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++tl) {
      if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
      const TileCoord c = coord(tile);
      const int acc = tl & 1;
      const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(tmem_full_bar(acc), (tl >> 1) & 1) && !*abort_flag);
      if (!ok) {
        if (lane == 0) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_flag = 1; }
        break;
      }
      ptx::tc_fence_after_sync();
      // Thread `lane` receives row (q*32 + lane) of the accumulator.  Written straight from there, every
      // store instruction would touch 32 rows with 16 bytes each; instead the warp turns 64-byte row
      // segments around in its private 2 KB of shared memory, so that a store instruction covers 8 rows
      // with 64 contiguous bytes each (whole 32-byte sectors only).
      OutT* obase = out + (long long)c.z * split_stride;
      constexpr int kPasses = sizeof(OutT) == 2 ? 1 : 2;        // 64-byte segments per 32 accumulator columns
      constexpr int kSegCols = 64 / (int)sizeof(OutT);          // output columns per segment
      const int my_chunk = lane & 3, my_row = lane >> 2;        // role of this lane on the store side
      long long orow[4];                                        // destination rows of the four rows this lane stores
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int grow = c.m0 + q * 32 + my_row + 8 * j;
        orow[j] = (row_map != nullptr && grow < M) ? (long long)__ldg(row_map + grow) : (long long)grow;
      }
#pragma unroll 1
      for (int cc = 0; cc < BN / 32; ++cc) {
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + cc * 32, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {  // 16-byte chunk i of this row's segment
            uint4 packed;
            if (sizeof(OutT) == 2) {
              float v[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[i * 8 + e]);
              const int col = c.n0 + cc * 32 + i * 8;
              if (bias != nullptr && col < N) {
                float b[8];
                Vec16<__nv_bfloat16>::to_float(__ldg(reinterpret_cast<const uint4*>(bias + col)), b);
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] += b[e];
              }
              packed = Vec16<__nv_bfloat16>::from_float(v);
            } else {
              packed = make_uint4(r[ps * 16 + i * 4], r[ps * 16 + i * 4 + 1], r[ps * 16 + i * 4 + 2], r[ps * 16 + i * 4 + 3]);
            }
            *reinterpret_cast<uint4*>(stage + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)) = packed;
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int rr = my_row + 8 * j;
            const uint4 v4 = *reinterpret_cast<const uint4*>(stage + rr * 64 + ((my_chunk ^ ((rr >> 1) & 3)) << 4));
            const int grow = c.m0 + q * 32 + rr;
            const int gcol = c.n0 + cc * 32 + ps * kSegCols + my_chunk * (16 / (int)sizeof(OutT));
            if (grow < M && gcol < N) {
              uint4* dst = reinterpret_cast<uint4*>(obase + orow[j] * ldo + gcol);
              if (sizeof(OutT) == 2 && accumulate) {
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
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tmem_empty_bar(acc));  // this warp has drained its quarter of the accumulator
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ---- wgrad helpers --------------------------------------------------------------------------------
// Partial column sums of dout over one chunk of rows: part[chunk][col].  A streaming reduction: CTA (x, y) owns 64
// columns and the rows of chunk y, eight threads across the columns (16 bytes each) and 32 down the rows with four
// loads in flight per thread; the 32 row lanes are added up in shared memory in a fixed order.
constexpr int kColsumChunks = 64;  // row chunks over the allocated rows (rows per chunk: a multiple of 8)
inline int colsum_rows_per_chunk(int capacity) { return (((capacity + kColsumChunks - 1) / kColsumChunks) + 7) & ~7; }

__global__ void __launch_bounds__(256)
colsum_partial_kernel(const __nv_bfloat16* __restrict__ dout, int n_out, const int32_t* __restrict__ cu, int n_seg,
                      int capacity, int rows_per_chunk, float* __restrict__ part) {
  pdl_entry();
  const int rows = packed_rows(cu, n_seg, capacity);
  const int r_begin = blockIdx.y * rows_per_chunk;
  if (r_begin >= rows) return;  // chunks past the valid rows are not read by the reduction
  int r_end = r_begin + rows_per_chunk;
  if (r_end > rows) r_end = rows;
  __shared__ float red[32][65];
  const int cg = threadIdx.x & 7, rl = threadIdx.x >> 3;  // 8 column groups of 8, 32 row lanes
  const int col = blockIdx.x * 64 + cg * 8;
  float acc[8] = {};
  if (col < n_out) {
    for (int i0 = r_begin + rl; i0 < r_end; i0 += 128) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i0 + 32 * u < r_end) v[u] = ld_nc16(dout + (long long)(i0 + 32 * u) * n_out + col);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (i0 + 32 * u < r_end) {
          float f[8];
          Vec16<__nv_bfloat16>::to_float(v[u], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] += f[e];
        }
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) red[rl][cg * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < 64) {
    const int c = blockIdx.x * 64 + threadIdx.x;
    if (c < n_out) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < 32; ++r) s += red[r][threadIdx.x];
      part[(long long)blockIdx.y * n_out + c] = s;
    }
  }
}

// out[e] = sum over the splits that hold rows (in split order) of part[s][e]; zero if there are none.
// Two arrays in one launch: the weight-gradient partials (a few splits: a thread adds them in split order) and,
// optionally, the bias-gradient partials, which have row chunks of their own - up to hundreds of them for a few
// thousand outputs, so there a warp owns four outputs: lane l adds chunks l, l + 32, ... in order and a fixed shuffle
// tree adds the lanes.  The first ceil(n2 / 32) blocks take the second array.
__global__ void __launch_bounds__(256)
split_reduce_kernel(const float* __restrict__ part, long long n, const float* __restrict__ part2, long long n2,
                    int splits, int rows_per_chunk2, const int32_t* __restrict__ cu, int n_seg, int capacity,
                    float* __restrict__ out, float* __restrict__ out2) {
  pdl_entry();
  const int rows = packed_rows(cu, n_seg, capacity);
  const int k_blocks = (rows + BK - 1) / BK;  // the splits were dealt the BK-blocks of the rows in turn
  const int valid1 = k_blocks < splits ? k_blocks : splits;
  const long long n4 = n >> 2, m4 = n2 >> 2;
  const int nb2 = (int)((m4 + 7) / 8);
  if ((int)blockIdx.x < nb2) {
    const int valid2 = (rows + rows_per_chunk2 - 1) / rows_per_chunk2;
    const long long j = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (j >= m4) return;
    const int lane = threadIdx.x & 31;
    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int z = lane; z < valid2; z += 32) {
      const float4 v = __ldcs(reinterpret_cast<const float4*>(part2 + (long long)z * n2) + j);
      s4.x += v.x; s4.y += v.y; s4.z += v.z; s4.w += v.w;
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      s4.x += __shfl_xor_sync(0xffffffffu, s4.x, off);
      s4.y += __shfl_xor_sync(0xffffffffu, s4.y, off);
      s4.z += __shfl_xor_sync(0xffffffffu, s4.z, off);
      s4.w += __shfl_xor_sync(0xffffffffu, s4.w, off);
    }
    if (lane == 0) reinterpret_cast<float4*>(out2)[j] = s4;
    return;
  }
  const long long first = (long long)(blockIdx.x - nb2) * blockDim.x + threadIdx.x;
  for (long long j = first; j < n4; j += (long long)(gridDim.x - nb2) * blockDim.x) {
    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // four splits' loads in flight at a time; the additions stay in split order
    auto add = [&](const float4& v) { s4.x += v.x; s4.y += v.y; s4.z += v.z; s4.w += v.w; };
    auto at = [&](int z) { return __ldcs(reinterpret_cast<const float4*>(part + (long long)z * n) + j); };
    int z = 0;
    for (; z + 4 <= valid1; z += 4) {
      const float4 v0 = at(z), v1 = at(z + 1), v2 = at(z + 2), v3 = at(z + 3);
      add(v0); add(v1); add(v2); add(v3);
    }
    for (; z < valid1; ++z) add(at(z));
    reinterpret_cast<float4*>(out)[j] = s4;
  }
}

struct SplitPlan { int splits, k_per_split; };

// The BK-blocks of K = packed rows are dealt to the splits in turn, so every split is in use whatever the row count;
// as many splits as keep tiles x splits within the CTAs that are resident at once (a second tile for some of the CTAs
// would double the longest path).
SplitPlan plan_splits(int capacity, int n_in, int n_out) {
  const int tiles = ((n_out + BM - 1) / BM) * ((n_in + 127) / 128);
  int splits = (2 * kNumSMs) / tiles;
  const int max_by_rows = (capacity + BK - 1) / BK;
  if (splits > max_by_rows) splits = max_by_rows;
  if (splits > 32) splits = 32;
  if (splits < 1) splits = 1;
  int kps = (capacity + splits - 1) / splits;
  kps = ((kps + BK - 1) / BK) * BK;
  splits = (capacity + kps - 1) / kps;
  return {splits, kps};
}

size_t wgrad_workspace_bytes(int capacity, int n_in, int n_out) {
  const SplitPlan sp = plan_splits(capacity, n_in, n_out);
  size_t w = (size_t)sp.splits * n_out * n_in * sizeof(float);
  w = (w + 255) & ~(size_t)255;
  return w + (size_t)kColsumChunks * n_out * sizeof(float) + 256;
}

template <int BN, bool kAMn, bool kBMn, typename OutT>
int launch_gemm(const CUtensorMap& tmA, const CUtensorMap& tmB, const __nv_bfloat16* bias, OutT* out, long long ldo,
                long long split_stride, int M, int N, int K, const int32_t* cu, int n_seg, int capacity, int dyn_which,
                int k_per_split, int splits, int k_interleave, const int32_t* row_map, int accumulate,
                int32_t* d_status, cudaStream_t st, const char* what) {
  auto kern = gemm_tc_kernel<BN, kAMn, kBMn, OutT>;
  static DeviceOnce attr;  // per instantiation and device
  cudaError_t ea = attr.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes<BN>()); });
  if (ea != cudaSuccess) { set_cuda_error(ea, what); return SPA_ERR_CUDA; }
  // persistent grid: two CTAs per SM (99 KB of shared memory and 256 TMEM columns each), never more
  // CTAs than there are tiles when every allocated row is in use
  long long tiles = (long long)((N + BN - 1) / BN) * ((M + BM - 1) / BM) * splits;
  const int grid = (int)(tiles < 2 * kNumSMs ? (tiles < 1 ? 1 : tiles) : 2 * kNumSMs);
  launch_pdl(kern, grid, kGemmThreads, gemm_smem_bytes<BN>(), st, tmA, tmB, bias, out, ldo, split_stride, M, N, K, cu,
             n_seg, capacity, dyn_which, k_per_split, k_interleave, row_map, accumulate, d_status);
  SPA_CUDA_CHECK_LAUNCH(what);
  return SPA_OK;
}

}  // namespace

bool tc_linear_supported(int n_in, int n_out) {
  return n_in % 8 == 0 && n_out % 8 == 0 && n_in >= 64 && n_out >= 64 && encode_fn() != nullptr;
}

size_t tc_linear_workspace_bytes(const spa_params& p) {
  if (p.dtype != SPA_BF16 || !tc_linear_supported(p.C, 3 * p.C)) return 0;
  const size_t a = wgrad_workspace_bytes(p.capacity, p.C, 3 * p.C);
  const size_t b = wgrad_workspace_bytes(p.capacity, p.C, p.C);
  return a > b ? a : b;
}

int launch_linear_fwd_tc(const spa_params& p, const void* a, const void* W, const void* bias, int n_in, int n_out,
                         const int32_t* cu, void* out, int32_t* d_status, cudaStream_t st, const int32_t* row_map,
                         bool accumulate) {
  if (tc_pair_linear_supported(p, n_in, n_out))
    return launch_linear_fwd_pair(p, a, W, bias, n_in, n_out, cu, out, d_status, st, row_map, accumulate);
  CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, a, n_in, p.capacity, (uint64_t)n_in * 2, BK, BM) ||
      !make_tmap_bf16_2d(&tmB, W, n_in, n_out, (uint64_t)n_in * 2, BK, 128))
    return SPA_ERR_UNSUPPORTED;
  return launch_gemm<128, false, false, __nv_bfloat16>(tmA, tmB, (const __nv_bfloat16*)bias,
                                                              (__nv_bfloat16*)out, n_out, 0, p.capacity, n_out, n_in,
                                                              cu, p.B, p.capacity, 1, n_in, 1, 0, row_map,
                                                              accumulate ? 1 : 0, d_status, st, "gemm_tc_kernel(fwd)");
}

int launch_linear_bwd_tc(const spa_params& p, const void* a, const void* W, const void* dout, int n_in, int n_out,
                         const int32_t* cu, void* da, float* dW, float* db, void* workspace, int32_t* d_status,
                         cudaStream_t st, const int32_t* row_map, bool accumulate) {
  CUtensorMap tmA, tmB, tmA2, tmB2;
  if (da != nullptr && (!make_tmap_bf16_2d(&tmA, dout, n_out, p.capacity, (uint64_t)n_out * 2, BK, BM) ||
                        !make_tmap_bf16_2d(&tmB, W, n_in, n_out, (uint64_t)n_in * 2, 64, BK)))
    return SPA_ERR_UNSUPPORTED;
  if (dW != nullptr && (!make_tmap_bf16_2d(&tmA2, dout, n_out, p.capacity, (uint64_t)n_out * 2, 64, BK) ||
                        !make_tmap_bf16_2d(&tmB2, a, n_in, p.capacity, (uint64_t)n_in * 2, 64, BK)))
    return SPA_ERR_UNSUPPORTED;
  // A pair CTA owns its SM (all 512 TMEM columns, 175 KB of shared memory).  A call that asks for da alone is
  // the pattern of a caller that runs the weight gradients beside it on another stream: there the one-CTA
  // kernel, which shares an SM with them, gives the shorter step; a call that computes everything in
  // sequence takes the pair kernel for da.
  const bool pair_dgrad = da != nullptr && (dW != nullptr || db != nullptr) && tc_pair_linear_supported(p, n_in, n_out);
  if (pair_dgrad) {
    int rc = launch_linear_dgrad_pair(p, W, dout, n_in, n_out, cu, da, d_status, st, row_map, accumulate);
    if (rc != SPA_OK) return rc;
  } else if (da != nullptr) {  // da[M][n_in] = dout[M][n_out] W[n_out][n_in]
    int rc = launch_gemm<128, false, true, __nv_bfloat16>(tmA, tmB, nullptr, (__nv_bfloat16*)da, n_in, 0,
                                                                 p.capacity, n_in, n_out, cu, p.B, p.capacity, 1, n_out,
                                                                 1, 0, row_map, accumulate ? 1 : 0, d_status, st,
                                                                 "gemm_tc_kernel(dgrad)");
    if (rc != SPA_OK) return rc;
  }
  if (dW == nullptr && db == nullptr) return SPA_OK;
  const SplitPlan sp = plan_splits(p.capacity, n_in, n_out);
  float* part_w = reinterpret_cast<float*>(workspace);
  size_t off = ((size_t)sp.splits * n_out * n_in * sizeof(float) + 255) & ~(size_t)255;
  float* part_b = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace) + off);
  const long long n_w = (long long)n_out * n_in;
  const int rpc = colsum_rows_per_chunk(p.capacity);
  if (db != nullptr) {  // db[j] = sum_i dout[i][j]: partial sums per row chunk, added up by the reduction below
    dim3 grid((n_out + 63) / 64, (p.capacity + rpc - 1) / rpc);
    launch_pdl(colsum_partial_kernel, grid, 256, 0, st, (const __nv_bfloat16*)dout, n_out, cu, p.B, p.capacity, rpc, part_b);
    SPA_CUDA_CHECK_LAUNCH("colsum_partial_kernel");
  }
  if (dW != nullptr) {  // dW[n_out][n_in] = sum_i dout[i][:]^T a[i][:]
    int rc = launch_gemm<128, true, true, float>(tmA2, tmB2, nullptr, part_w, n_in, n_w, n_out, n_in, p.capacity,
                                                        cu, p.B, p.capacity, 2, sp.k_per_split, sp.splits, sp.splits,
                                                        nullptr, 0, d_status, st, "gemm_tc_kernel(wgrad)");
    if (rc != SPA_OK) return rc;
    const long long n_b = db != nullptr ? n_out : 0;
    int grid = (int)((n_w / 4 + 255) / 256);
    if (grid > kNumSMs * 8) grid = kNumSMs * 8;
    grid += (int)((n_b / 4 + 7) / 8);  // the blocks of the bias gradient come first
    launch_pdl(split_reduce_kernel, grid, 256, 0, st, part_w, n_w, part_b, n_b, sp.splits, rpc, cu, p.B, p.capacity, dW,
               db);
    SPA_CUDA_CHECK_LAUNCH("split_reduce_kernel");
  } else {  // db alone
    launch_pdl(split_reduce_kernel, (n_out / 4 + 7) / 8, 256, 0, st, (const float*)nullptr, 0LL, (const float*)part_b,
               (long long)n_out, 0, rpc, cu, p.B, p.capacity, (float*)nullptr, db);
    SPA_CUDA_CHECK_LAUNCH("split_reduce_kernel(db)");
  }
  return SPA_OK;
}

}  // namespace spa
