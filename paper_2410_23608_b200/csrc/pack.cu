// Token packing and its inverse / transposes (Sec. 3.2 "Token Packing"; unselected tokens pass
// through unchanged).  All four kernels are pure row movers: 16-byte coalesced loads and stores,
// several independent loads in flight per thread, no shared-memory staging of the rows.
//
// Stable compaction: packing the whole batch in (image, raster) order is a stream compaction over
// the flat token index, so cu_seqlens[b] is simply the exclusive mask prefix at token b*N.  Each
// CTA owns one tile of tokens; it obtains the prefix at its tile start by counting the mask bytes
// before it (16-byte loads + SIMD popcount; the mask is at most 1 MiB and lives in L2), so there
// is no inter-CTA dependency, no scratch memory and the result is deterministic.
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kPackThreads = 256;
constexpr int kBatch = 4;  // independent 16-byte loads in flight per thread

__device__ __forceinline__ int count_nonzero_bytes(uint4 m) {
  return __popc(__vcmpne4(m.x, 0u) & 0x01010101u) + __popc(__vcmpne4(m.y, 0u) & 0x01010101u) +
         __popc(__vcmpne4(m.z, 0u) & 0x01010101u) + __popc(__vcmpne4(m.w, 0u) & 0x01010101u);
}

template <typename T>
__device__ __forceinline__ uint4 scale16(uint4 v, float s) {
  float f[Vec16<T>::kElems];
  Vec16<T>::to_float(v, f);
#pragma unroll
  for (int e = 0; e < Vec16<T>::kElems; ++e) f[e] *= s;
  return Vec16<T>::from_float(f);
}

template <typename T>
__device__ __forceinline__ uint4 add16(uint4 a, uint4 b) {
  float fa[Vec16<T>::kElems], fb[Vec16<T>::kElems];
  Vec16<T>::to_float(a, fa);
  Vec16<T>::to_float(b, fb);
#pragma unroll
  for (int e = 0; e < Vec16<T>::kElems; ++e) fa[e] += fb[e];
  return Vec16<T>::from_float(fa);
}

// ------------------------------------------------------------------------------ select + pack
// kOrdered: the tokens of every image are visited in the order order[0], order[1], ... (a cyclically shifted
// feature map) instead of raster order.  Flat position t = b*N + j of the visiting order then stands for
// token b*N + order[j]; mask, scores, idx and inv stay indexed by the original token.
template <typename T, bool kGateScale, bool kOrdered>
__global__ void __launch_bounds__(kPackThreads)
select_pack_kernel(const uint4* __restrict__ x16, const uint8_t* __restrict__ mask, const float* __restrict__ scores,
                   const int32_t* __restrict__ order, int rows, int N, int B, int Q, int tile, int capacity,
                   uint4* __restrict__ xp16,
                   int32_t* __restrict__ idx, int32_t* __restrict__ inv, int32_t* __restrict__ cu,
                   int32_t* d_status) {
  pdl_entry();
  __shared__ int warp_cnt[kPackThreads / 32];
  __shared__ int warp_sel[kPackThreads / 32];
  __shared__ int sel_tok[kPackThreads];   // flat indices of the tile's selected tokens, in order
  __shared__ float sel_scale[kPackThreads];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int tile_start = blockIdx.x * tile;  // multiple of 16

  // 1. number of selected tokens before this tile
  int cnt = 0;
  const uint4* mask16 = reinterpret_cast<const uint4*>(mask);
  if (!kOrdered) {
    for (int k = tid; k < (tile_start >> 4); k += kPackThreads) cnt += count_nonzero_bytes(__ldg(mask16 + k));
  } else {
    // whole images before the tile's first image: any order visits the same bytes; then the positions of
    // that image which the given order visits before the tile
    const int img0 = (tile_start / N) * N;
    for (int k = tid; k < (img0 >> 4); k += kPackThreads) cnt += count_nonzero_bytes(__ldg(mask16 + k));
    for (int k = (img0 & ~15) + tid; k < img0; k += kPackThreads) cnt += mask[k] != 0;
    for (int j = tid; j < tile_start - img0; j += kPackThreads) cnt += mask[img0 + __ldg(order + j)] != 0;
  }
  cnt = (int)__reduce_add_sync(0xffffffffu, (unsigned)cnt);
  if (lane == 0) warp_cnt[wid] = cnt;

  // 2. ranks inside the tile
  const int t = tile_start + tid;
  const bool in_tile = tid < tile && t < rows;
  int tok = t;  // the token that position t of the visiting order stands for
  if (kOrdered && in_tile) tok = (t / N) * N + __ldg(order + t % N);
  const bool sel = in_tile && mask[tok] != 0;
  const unsigned ballot = __ballot_sync(0xffffffffu, sel);
  if (lane == 0) warp_sel[wid] = __popc(ballot);
  __syncthreads();
  int base = 0, before = 0, tile_total = 0;
#pragma unroll
  for (int w = 0; w < kPackThreads / 32; ++w) {
    base += warp_cnt[w];
    before += w < wid ? warp_sel[w] : 0;
    tile_total += warp_sel[w];
  }
  const int local = before + __popc(ballot & ((1u << lane) - 1u));  // exclusive rank in the tile
  const int dst = base + local;
  if (in_tile) {
    if (t % N == 0) cu[t / N] = dst;  // exclusive prefix at an image's first token
    if (inv != nullptr) inv[tok] = (sel && dst < capacity) ? dst : -1;
  }
  if (sel) {
    if (dst < capacity) {
      idx[dst] = tok;
      sel_tok[local] = tok;
      if (kGateScale) sel_scale[local] = 1.f / (1.f + __expf(-scores[tok]));
    } else {
      record_status(d_status, SPA_ERR_CAPACITY);
    }
  }
  if (tid == 0 && tile_start + tile >= rows) cu[B] = base + tile_total;
  __syncthreads();

  // 3. gather the selected rows: chunk k of the tile is (row k / Q, 16-byte column k % Q)
  int n_ok = capacity - base;
  n_ok = n_ok < 0 ? 0 : (n_ok < tile_total ? n_ok : tile_total);
  const int total = n_ok * Q;
  for (int k0 = tid; k0 < total; k0 += kPackThreads * kBatch) {
    uint4 v[kBatch];
    int r[kBatch], q[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int k = k0 + u * kPackThreads;
      if (k < total) {
        r[u] = k / Q;
        q[u] = k - r[u] * Q;
        v[u] = ld_nc16(x16 + (size_t)sel_tok[r[u]] * Q + q[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int k = k0 + u * kPackThreads;
      if (k < total) {
        if (kGateScale) v[u] = scale16<T>(v[u], sel_scale[r[u]]);
        xp16[(size_t)(base + r[u]) * Q + q[u]] = v[u];
      }
    }
  }
}

// ------------------------------------------------------------------------------ unpack
// Out of place: every row of y is written, from z (selected) or x (pass-through).
template <typename T, bool kResidual>
__global__ void __launch_bounds__(kPackThreads)
unpack_scatter_kernel(const uint4* __restrict__ z16, const uint4* __restrict__ x16, const int32_t* __restrict__ inv,
                      const int32_t* __restrict__ cu, int B, int capacity, long long total, int Q,
                      uint4* __restrict__ y16) {
  pdl_entry();
  const int Np = packed_rows(cu, B, capacity);
  const long long stride = (long long)gridDim.x * kPackThreads;
  for (long long k0 = (long long)blockIdx.x * kPackThreads + threadIdx.x; k0 < total; k0 += stride * kBatch) {
    uint4 v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const long long k = k0 + u * stride;
      if (k < total) {
        const long long t = k / Q;
        const int q = (int)(k - t * Q);
        const int i = __ldg(inv + t);
        if (i >= 0 && i < Np) {
          v[u] = ld_nc16(z16 + (size_t)i * Q + q);
          if (kResidual) v[u] = add16<T>(v[u], ld_nc16(x16 + k));
        } else {
          v[u] = ld_nc16(x16 + k);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const long long k = k0 + u * stride;
      if (k < total) y16[k] = v[u];
    }
  }
}

// Row scatter over the packed rows: dst[idx[i]] = src[i] (+ add[idx[i]]).  Serves the in-place
// unpack (dst = y = x, add = x under the residual flag) and the transpose of the pack gather
// (dst = dX, add = dY under the residual flag).  `add` may alias `dst`.
template <typename T, bool kAdd>
__global__ void __launch_bounds__(kPackThreads)
row_scatter_kernel(const uint4* __restrict__ src16, const uint4* addp, const int32_t* __restrict__ idx,
                   const int32_t* __restrict__ cu, int B, int capacity, int Q, uint4* dst16) {
  pdl_entry();
  const long long total = (long long)packed_rows(cu, B, capacity) * Q;
  const long long stride = (long long)gridDim.x * kPackThreads;
  for (long long k0 = (long long)blockIdx.x * kPackThreads + threadIdx.x; k0 < total; k0 += stride * kBatch) {
    uint4 v[kBatch];
    size_t o[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const long long k = k0 + u * stride;
      if (k < total) {
        const long long i = k / Q;
        const int q = (int)(k - i * Q);
        o[u] = (size_t)__ldg(idx + i) * Q + q;
        v[u] = ld_nc16(src16 + k);
        if (kAdd) v[u] = add16<T>(v[u], addp[o[u]]);
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const long long k = k0 + u * stride;
      if (k < total) dst16[o[u]] = v[u];
    }
  }
}

// Transpose of the unpack: one pass over dY; selected rows go to dz, the others to dX.
__global__ void __launch_bounds__(kPackThreads)
unpack_scatter_bwd_kernel(const uint4* __restrict__ dY16, const int32_t* __restrict__ inv,
                          const int32_t* __restrict__ cu, int B, int capacity, long long total, int Q,
                          uint4* __restrict__ dz16, uint4* dX16, bool copy_pass_through, bool copy_selected) {
  pdl_entry();
  const int Np = packed_rows(cu, B, capacity);
  const long long stride = (long long)gridDim.x * kPackThreads;
  for (long long k0 = (long long)blockIdx.x * kPackThreads + threadIdx.x; k0 < total; k0 += stride * kBatch) {
    uint4 v[kBatch];
    long long o[kBatch];  // >= 0: chunk of dz; -1: pass-through; -2: nothing to do
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const long long k = k0 + u * stride;
      o[u] = -2;
      if (k < total) {
        const long long t = k / Q;
        const int q = (int)(k - t * Q);
        const int i = __ldg(inv + t);
        if (i >= 0 && i < Np) o[u] = (long long)i * Q + q;
        else if (copy_pass_through) o[u] = -1;
        if (o[u] != -2) v[u] = ld_nc16(dY16 + k);
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const long long k = k0 + u * stride;
      if (o[u] >= 0) {
        dz16[o[u]] = v[u];
        if (copy_selected) dX16[k] = v[u];
      } else if (o[u] == -1) {
        dX16[k] = v[u];
      }
    }
  }
}

int stream_grid(long long total_chunks) {
  long long g = (total_chunks + (long long)kPackThreads * kBatch - 1) / ((long long)kPackThreads * kBatch);
  const long long cap = (long long)kNumSMs * 16;
  if (g > cap) g = cap;
  return g < 1 ? 1 : (int)g;
}

// dst = src over `total` 16-byte chunks: the pass-through rows of the unpack step written ahead of
// time, so that the projection (or the input-gradient product) only has to scatter the selected rows.
__global__ void __launch_bounds__(kPackThreads)
copy_chunks_kernel(const uint4* __restrict__ src16, uint4* __restrict__ dst16, long long total) {
  pdl_entry();
  const long long stride = (long long)gridDim.x * kPackThreads;
  for (long long k0 = (long long)blockIdx.x * kPackThreads + threadIdx.x; k0 < total; k0 += stride * kBatch) {
    uint4 v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      if (k0 + u * stride < total) v[u] = ld_nc16(src16 + k0 + u * stride);
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      if (k0 + u * stride < total) dst16[k0 + u * stride] = v[u];
  }
}

template <typename T> int chunks_per_row(int C) { return C / Vec16<T>::kElems; }


// ------------------------------------------------------------------------------ container cuts
// Attention segments of the paper's fixed-length containers (Sec. 3.2 "Token Packing": the packed tokens fill
// containers of L tokens, and the mask keeps a token from attending to other images): the packed buffer is cut at
// every multiple of L and at every image boundary.  out receives the distinct cut positions in ascending order,
// 0 first and N_p last, followed by copies of N_p up to n_max + 1 entries (empty segments, which the attention
// kernels skip), so that the caller can pass the upper bound n_max as the segment count without reading anything back.
// A cut position's rank is the number of multiples of L below it plus the number of distinct image boundaries below
// it that are not multiples of L; one CTA computes the latter as a prefix sum over the B + 1 offsets.
constexpr int kCutThreads = 1024;
constexpr int kCutMaxOffsets = 4096;  // B + 1 offsets and their prefix counts are held in shared memory

__global__ void __launch_bounds__(kCutThreads)
container_offsets_kernel(const int32_t* __restrict__ cu, int B, int L, int n_max, int32_t* __restrict__ out) {
  pdl_entry();
  __shared__ int32_t cu_s[kCutMaxOffsets];
  __shared__ int32_t pre_s[kCutMaxOffsets + 1];  // pre_s[b] = distinct non-multiple offsets among cu[0..b)
  __shared__ int warp_tot[kCutThreads / 32];
  __shared__ int carry_s;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int n = B + 1;
  for (int i = tid; i < n; i += kCutThreads) cu_s[i] = __ldg(cu + i);
  if (tid == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n; base += kCutThreads) {
    const int b = base + tid;
    const int c = b < n ? cu_s[b] : 0;
    const int flag = (b < n && c % L != 0 && (b == 0 || c != cu_s[b - 1])) ? 1 : 0;
    int incl = flag;  // inclusive scan inside the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    int before = carry_s;
    for (int w = 0; w < wid; ++w) before += warp_tot[w];
    if (b < n) pre_s[b] = before + incl - flag;
    __syncthreads();
    if (tid == kCutThreads - 1) carry_s = before + incl;
    __syncthreads();
  }
  if (tid == 0) pre_s[n] = carry_s;
  __syncthreads();
  const int Np = cu_s[B];
  const int K = Np / L;                 // multiples 0, L, ..., K L
  const int total = K + 1 + pre_s[n];   // distinct cut positions
  for (int b = tid; b < n; b += kCutThreads) {
    const int c = cu_s[b];
    if (c % L != 0 && (b == 0 || c != cu_s[b - 1])) out[(c + L - 1) / L + pre_s[b]] = c;
  }
  for (int k = tid; k <= K; k += kCutThreads) {
    const int v = k * L;
    int lo = 0, hi = n;  // first index with cu_s[index] >= v
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (cu_s[mid] < v) lo = mid + 1; else hi = mid;
    }
    out[k + pre_s[lo]] = v;
  }
  for (int j = total + tid; j <= n_max; j += kCutThreads) out[j] = Np;
}

}  // namespace

int launch_container_offsets(const spa_params& p, const int32_t* cu, int L, int n_max, int32_t* out, cudaStream_t st) {
  if (p.B + 1 > kCutMaxOffsets) return SPA_ERR_UNSUPPORTED;
  launch_pdl(container_offsets_kernel, 1, kCutThreads, 0, st, cu, p.B, L, n_max, out);
  SPA_CUDA_CHECK_LAUNCH("container_offsets_kernel");
  return SPA_OK;
}

int launch_select_pack(const spa_params& p, const void* x, const uint8_t* mask, const float* scores,
                       const int32_t* order, void* xp, int32_t* idx, int32_t* inv, int32_t* cu, int32_t* d_status,
                       cudaStream_t st) {
  const int rows = p.B * p.N;
  int tile = 256;
  while (tile > 32 && (rows + tile - 1) / tile < 2 * kNumSMs) tile >>= 1;
  const int grid = (rows + tile - 1) / tile;
  const bool gs = (p.flags & SPA_FLAG_GATE_SCALE) != 0;
#define SPA_PACK_LAUNCH(T, GS, ORD)                                                                              \
  launch_pdl(select_pack_kernel<T, GS, ORD>, grid, kPackThreads, 0, st, (const uint4*)x, mask, scores, order, rows, p.N, \
             p.B, chunks_per_row<T>(p.C), tile, p.capacity, (uint4*)xp, idx, inv, cu, d_status)
#define SPA_PACK_ORD(T, GS) do { if (order != nullptr) SPA_PACK_LAUNCH(T, GS, true); else SPA_PACK_LAUNCH(T, GS, false); } while (0)
  if (p.dtype == SPA_F32) { if (gs) SPA_PACK_ORD(float, true); else SPA_PACK_ORD(float, false); }
  else { if (gs) SPA_PACK_ORD(__nv_bfloat16, true); else SPA_PACK_ORD(__nv_bfloat16, false); }
#undef SPA_PACK_ORD
#undef SPA_PACK_LAUNCH
  SPA_CUDA_CHECK_LAUNCH("select_pack_kernel");
  return SPA_OK;
}

#define SPA_SCATTER(T, ADD, SRC, ADDP, DST) \
  launch_pdl(row_scatter_kernel<T, ADD>, grid, kPackThreads, 0, st, (const uint4*)(SRC), (const uint4*)(ADDP), idx, cu, p.B, p.capacity, Q, (uint4*)(DST))

int launch_unpack_scatter(const spa_params& p, const void* z, const void* x, const int32_t* idx,
                          const int32_t* inv, const int32_t* cu, void* y, cudaStream_t st) {
  const bool res = (p.flags & SPA_FLAG_RESIDUAL) != 0;
  const bool f32 = p.dtype == SPA_F32;
  const int Q = f32 ? chunks_per_row<float>(p.C) : chunks_per_row<__nv_bfloat16>(p.C);
  if (p.flags & SPA_FLAG_INPLACE) {
    const int grid = stream_grid((long long)p.capacity * Q);
    if (f32) { if (res) SPA_SCATTER(float, true, z, x, y); else SPA_SCATTER(float, false, z, x, y); }
    else { if (res) SPA_SCATTER(__nv_bfloat16, true, z, x, y); else SPA_SCATTER(__nv_bfloat16, false, z, x, y); }
    SPA_CUDA_CHECK_LAUNCH("row_scatter_kernel");
    return SPA_OK;
  }
  const long long total = (long long)p.B * p.N * Q;
  const int grid = stream_grid(total);
#define SPA_UNPACK(T, RES) \
  launch_pdl(unpack_scatter_kernel<T, RES>, grid, kPackThreads, 0, st, (const uint4*)z, (const uint4*)x, inv, cu, p.B, p.capacity, total, Q, (uint4*)y)
  if (f32) { if (res) SPA_UNPACK(float, true); else SPA_UNPACK(float, false); }
  else { if (res) SPA_UNPACK(__nv_bfloat16, true); else SPA_UNPACK(__nv_bfloat16, false); }
#undef SPA_UNPACK
  SPA_CUDA_CHECK_LAUNCH("unpack_scatter_kernel");
  return SPA_OK;
}

int launch_unpack_scatter_bwd(const spa_params& p, const void* dY, const int32_t* idx, const int32_t* inv,
                              const int32_t* cu, void* dz, void* dX, cudaStream_t st) {
  (void)idx;
  const int Q = p.dtype == SPA_F32 ? chunks_per_row<float>(p.C) : chunks_per_row<__nv_bfloat16>(p.C);
  const long long total = (long long)p.B * p.N * Q;
  const bool copy = dX != nullptr && dX != dY;
  launch_pdl(unpack_scatter_bwd_kernel, stream_grid(total), kPackThreads, 0, st, (const uint4*)dY, inv, cu, p.B, p.capacity,
                                                                        total, Q, (uint4*)dz, (uint4*)dX, copy,
                                                                        copy && (p.flags & SPA_FLAG_RESIDUAL) != 0);
  SPA_CUDA_CHECK_LAUNCH("unpack_scatter_bwd_kernel");
  return SPA_OK;
}

int launch_select_pack_bwd(const spa_params& p, const void* dxp, const void* dY, const int32_t* idx,
                           const int32_t* cu, void* dX, cudaStream_t st) {
  const bool res = (p.flags & SPA_FLAG_RESIDUAL) != 0;
  const bool f32 = p.dtype == SPA_F32;
  const int Q = f32 ? chunks_per_row<float>(p.C) : chunks_per_row<__nv_bfloat16>(p.C);
  const int grid = stream_grid((long long)p.capacity * Q);
  if (f32) { if (res) SPA_SCATTER(float, true, dxp, dY, dX); else SPA_SCATTER(float, false, dxp, dY, dX); }
  else { if (res) SPA_SCATTER(__nv_bfloat16, true, dxp, dY, dX); else SPA_SCATTER(__nv_bfloat16, false, dxp, dY, dX); }
  SPA_CUDA_CHECK_LAUNCH("row_scatter_kernel");
  return SPA_OK;
}
#undef SPA_SCATTER

int launch_copy_tokens(const spa_params& p, const void* src, void* dst, cudaStream_t st) {
  const int Q = p.dtype == SPA_F32 ? chunks_per_row<float>(p.C) : chunks_per_row<__nv_bfloat16>(p.C);
  const long long total = (long long)p.B * p.N * Q;
  launch_pdl(copy_chunks_kernel, stream_grid(total), kPackThreads, 0, st, (const uint4*)src, (uint4*)dst, total);
  SPA_CUDA_CHECK_LAUNCH("copy_chunks_kernel");
  return SPA_OK;
}

}  // namespace spa
