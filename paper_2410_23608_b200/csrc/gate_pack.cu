// Gate, hard selection and token packing in one pass over x (Sec. 3.2: Eq. 4, the thresholded form of Eq. 6 and
// "Token Packing").
//
// A CTA owns a tile of consecutive tokens.  Each warp pulls its rows of x into registers with 16-byte streaming loads
// (and, on request, writes the pass-through copy y = x from them), forms the gate logits, thresholds them, and the CTA
// counts its selected tokens.  Where the tile's rows land in the packed buffer depends on the number of selected tokens
// in all earlier tiles: every tile publishes its count in a small state array as soon as it knows it, and obtains its
// exclusive prefix by reading the counts of up to kWindow predecessors at once, all threads of the CTA polling in
// parallel (one round trip to L2 when the others are ready), plus the published inclusive prefix of the tile before
// that window.  The selected rows then go from the registers straight to x_packed: x is read from memory exactly once.
//
// A CTA waits only for CTAs with smaller block indices, which the hardware dispatches first, so whatever it waits for
// is running or done.  Every poll loop is bounded all the same: when one runs out the kernel records SPA_ERR_TIMEOUT
// and returns without writing packed rows.  The state array must be zero when the kernel starts; the CTA that
// finishes last puts it back to zero.
#include "sm100_ptx.cuh"
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kGpThreads = 256;
constexpr int kGpWarps = kGpThreads / 32;
constexpr uint32_t kValid = 1u << 31;  // set in a published word; the low bits hold the count
constexpr int kWindow = 4 * kGpThreads;   // predecessors whose counts a tile sums directly
constexpr int kStateHeader = 4;           // words: finished counter, three spare; then counts[tiles], prefixes[tiles]

__device__ __forceinline__ uint32_t ld_volatile(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_volatile(uint32_t* p, uint32_t v) {
  asm volatile("st.volatile.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <typename T>
__device__ __forceinline__ uint4 scaled16(uint4 v, float s) {
  float f[Vec16<T>::kElems];
  Vec16<T>::to_float(v, f);
#pragma unroll
  for (int e = 0; e < Vec16<T>::kElems; ++e) f[e] *= s;
  return Vec16<T>::from_float(f);
}

// kChunks: 16-byte chunks of a row held by one lane (row = up to 32 * kChunks chunks); kRows: rows per warp.
template <typename T, int kChunks, int kRows, bool kGateScale>
__global__ void __launch_bounds__(kGpThreads)
gate_pack_kernel(const uint4* __restrict__ x16, const T* __restrict__ w_g, float b_g, const float* __restrict__ s_up,
                 float tau, int rows, int N, int B, int Q, int capacity, float* __restrict__ scores,
                 uint8_t* __restrict__ mask, uint4* __restrict__ y16, uint4* __restrict__ xp16,
                 int32_t* __restrict__ idx, int32_t* __restrict__ inv, int32_t* __restrict__ cu, uint32_t* state,
                 int n_tiles, int max_tiles, int32_t* d_status) {
  constexpr int E = Vec16<T>::kElems;
  constexpr int kTile = kGpWarps * kRows;
  __shared__ __align__(16) float w_s[32 * kChunks * E];
  __shared__ int s_last;
  __shared__ int warp_sel[kGpWarps], warp_part[kGpWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = blockIdx.x;
  const int row0 = tile * kTile + warp * kRows;
  pdl_entry();

  // ---- this warp's rows into registers (and out again as the pass-through copy)
  uint4 v[kRows][kChunks];
#pragma unroll
  for (int k = 0; k < kRows; ++k) {
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      const int q = lane + 32 * c;
      v[k][c] = make_uint4(0u, 0u, 0u, 0u);
      if (row0 + k < rows && q < Q) v[k][c] = ld_nc16(x16 + (size_t)(row0 + k) * Q + q);
    }
  }
  if (y16 != nullptr) {
#pragma unroll
    for (int k = 0; k < kRows; ++k) {
#pragma unroll
      for (int c = 0; c < kChunks; ++c) {
        const int q = lane + 32 * c;
        if (row0 + k < rows && q < Q) y16[(size_t)(row0 + k) * Q + q] = v[k][c];
      }
    }
  }
  for (int c = tid; c < 32 * kChunks * E; c += kGpThreads) w_s[c] = c < Q * E ? to_f32<T>(w_g[c]) : 0.f;
  __syncthreads();
  // ---- gate logits (Eq. 4) and the selection
  float acc[kRows];
#pragma unroll
  for (int k = 0; k < kRows; ++k) acc[k] = 0.f;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    float w[E];
    const float4* wq = reinterpret_cast<const float4*>(w_s + (lane + 32 * c) * E);
#pragma unroll
    for (int e = 0; e < E / 4; ++e) {
      const float4 t = wq[e];
      w[4 * e] = t.x; w[4 * e + 1] = t.y; w[4 * e + 2] = t.z; w[4 * e + 3] = t.w;
    }
#pragma unroll
    for (int k = 0; k < kRows; ++k) {
      float f[E];
      Vec16<T>::to_float(v[k][c], f);
#pragma unroll
      for (int e = 0; e < E; ++e) acc[k] = fmaf(f[e], w[e], acc[k]);
    }
  }
  unsigned sel_bits = 0;  // bit k: row k of this warp is selected (the same in every lane)
  float s_row[kRows];
#pragma unroll
  for (int k = 0; k < kRows; ++k) {
    float s = warp_sum(acc[k]) + b_g;
    const int r = row0 + k;
    if (r < rows) {
      if (s_up != nullptr) s = fmaxf(s, __ldg(s_up + r));
      if (s > tau) sel_bits |= 1u << k;
      if (lane == 0) {
        scores[r] = s;
        mask[r] = s > tau ? 1 : 0;
      }
    }
    s_row[k] = s;
  }
  if (lane == 0) warp_sel[warp] = __popc(sel_bits);
  __syncthreads();
  int before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kGpWarps; ++w) {
    before += w < warp ? warp_sel[w] : 0;
    total += warp_sel[w];
  }

  // ---- exclusive prefix of this tile: publish the tile's count, then sum the predecessors' counts
  uint32_t* counts = state + kStateHeader;
  uint32_t* prefixes = counts + max_tiles;
  if (tid == 0) st_volatile(counts + tile, kValid | (uint32_t)total);
  const int lo = tile > kWindow ? tile - kWindow : 0;
  int part = 0;
  bool ok = true;
  for (int t = lo + tid; t < tile; t += kGpThreads) {
    uint32_t wv = 0u;
    for (uint32_t i = 0; i < ptx::kWaitLimit && !(wv & kValid); ++i) wv = ld_volatile(counts + t);
    ok = ok && (wv & kValid);
    part += (int)(wv & ~kValid);
  }
  if (lo > 0 && tid == kGpThreads - 1) {  // everything before the window: the inclusive prefix of tile lo - 1
    uint32_t wv = 0u;
    for (uint32_t i = 0; i < ptx::kWaitLimit && !(wv & kValid); ++i) wv = ld_volatile(prefixes + lo - 1);
    ok = ok && (wv & kValid);
    part += (int)(wv & ~kValid);
  }
  part = (int)__reduce_add_sync(0xffffffffu, (unsigned)part);
  if (lane == 0) warp_part[warp] = part;
  const bool all_ok = __syncthreads_and(ok ? 1 : 0) != 0;
  int excl = 0;
#pragma unroll
  for (int w = 0; w < kGpWarps; ++w) excl += warp_part[w];
  if (tid == 0) {
    if (all_ok) st_volatile(prefixes + tile, kValid | (uint32_t)(excl + total));
    else record_status(d_status, SPA_ERR_TIMEOUT);
  }

  // ---- indices, offsets and the packed rows
  if (all_ok) {
    const int base = excl + before;
#pragma unroll
    for (int k = 0; k < kRows; ++k) {
      const int r = row0 + k;
      if (r >= rows) break;
      const int dst = base + __popc(sel_bits & ((1u << k) - 1u));
      const bool sel = (sel_bits >> k) & 1u;
      if (lane == 0) {
        if (r % N == 0) cu[r / N] = dst;  // exclusive prefix at an image's first token
        if (inv != nullptr) inv[r] = (sel && dst < capacity) ? dst : -1;
      }
      if (sel) {
        if (dst < capacity) {
          if (lane == 0) idx[dst] = r;
          const float g = kGateScale ? 1.f / (1.f + __expf(-s_row[k])) : 1.f;
#pragma unroll
          for (int c = 0; c < kChunks; ++c) {
            const int q = lane + 32 * c;
            if (q < Q) xp16[(size_t)dst * Q + q] = kGateScale ? scaled16<T>(v[k][c], g) : v[k][c];
          }
        } else if (lane == 0) {
          record_status(d_status, SPA_ERR_CAPACITY);
        }
      }
    }
    if (tid == 0 && tile == n_tiles - 1) cu[B] = excl + total;
  }

  // ---- the CTA that finishes last leaves the state array zeroed for the next call
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&state[0], 1u) == (uint32_t)(n_tiles - 1) ? 1 : 0;
  __syncthreads();
  if (s_last) {
    for (int i = tid; i < n_tiles; i += kGpThreads) { counts[i] = 0u; prefixes[i] = 0u; }
    if (tid == 0) state[0] = 0u;
  }
}

template <int kChunks> constexpr int rows_per_warp() { return kChunks == 1 ? 8 : 4; }

inline int chunks_per_lane(const spa_params& p) {
  const int Q = p.C * (p.dtype == SPA_F32 ? 4 : 2) / 16;
  return (Q + 31) / 32;
}

// tiles of the smallest tile size (32 tokens): the length of each of the two arrays in the state
inline int max_tiles_of(const spa_params& p) { return (int)(((long long)p.B * p.N + 31) / 32); }

template <typename T, int kChunks>
int launch_one(const spa_params& p, const void* x, const void* w_g, float b_g, const float* s_up, float* scores,
               uint8_t* mask, void* y, void* xp, int32_t* idx, int32_t* inv, int32_t* cu, void* state,
               int32_t* d_status, cudaStream_t st) {
  constexpr int kRows = rows_per_warp<kChunks>();
  const int rows = p.B * p.N;
  const int n_tiles = (rows + kGpWarps * kRows - 1) / (kGpWarps * kRows);
  const int Q = p.C * (int)sizeof(T) / 16;
  if (p.flags & SPA_FLAG_GATE_SCALE)
    launch_pdl(gate_pack_kernel<T, kChunks, kRows, true>, n_tiles, kGpThreads, 0, st, (const uint4*)x, (const T*)w_g, b_g,
               s_up, p.tau, rows, p.N, p.B, Q, p.capacity, scores, mask, (uint4*)y, (uint4*)xp, idx, inv, cu,
               (uint32_t*)state, n_tiles, max_tiles_of(p), d_status);
  else
    launch_pdl(gate_pack_kernel<T, kChunks, kRows, false>, n_tiles, kGpThreads, 0, st, (const uint4*)x, (const T*)w_g, b_g,
               s_up, p.tau, rows, p.N, p.B, Q, p.capacity, scores, mask, (uint4*)y, (uint4*)xp, idx, inv, cu,
               (uint32_t*)state, n_tiles, max_tiles_of(p), d_status);
  SPA_CUDA_CHECK_LAUNCH("gate_pack_kernel");
  return SPA_OK;
}

template <typename T>
int launch_typed(const spa_params& p, const void* x, const void* w_g, float b_g, const float* s_up, float* scores,
                 uint8_t* mask, void* y, void* xp, int32_t* idx, int32_t* inv, int32_t* cu, void* state,
                 int32_t* d_status, cudaStream_t st) {
  switch (chunks_per_lane(p)) {
    case 1: return launch_one<T, 1>(p, x, w_g, b_g, s_up, scores, mask, y, xp, idx, inv, cu, state, d_status, st);
    case 2: return launch_one<T, 2>(p, x, w_g, b_g, s_up, scores, mask, y, xp, idx, inv, cu, state, d_status, st);
    case 3: return launch_one<T, 3>(p, x, w_g, b_g, s_up, scores, mask, y, xp, idx, inv, cu, state, d_status, st);
    case 4: return launch_one<T, 4>(p, x, w_g, b_g, s_up, scores, mask, y, xp, idx, inv, cu, state, d_status, st);
    default: return SPA_ERR_UNSUPPORTED;
  }
}

}  // namespace

bool gate_pack_supported(const spa_params& p) { return chunks_per_lane(p) <= 4; }

// state words: header, then a count and an inclusive prefix per tile
size_t gate_pack_state_bytes(const spa_params& p) {
  return ((kStateHeader + 2 * (size_t)max_tiles_of(p)) * sizeof(uint32_t) + 255) & ~(size_t)255;
}

int launch_gate_pack(const spa_params& p, const void* x, const void* w_g, float b_g, const float* s_up, float* scores,
                     uint8_t* mask, void* y, void* xp, int32_t* idx, int32_t* inv, int32_t* cu, void* state,
                     int32_t* d_status, cudaStream_t st) {
  if (p.dtype == SPA_F32)
    return launch_typed<float>(p, x, w_g, b_g, s_up, scores, mask, y, xp, idx, inv, cu, state, d_status, st);
  return launch_typed<__nv_bfloat16>(p, x, w_g, b_g, s_up, scores, mask, y, xp, idx, inv, cu, state, d_status, st);
}

}  // namespace spa
