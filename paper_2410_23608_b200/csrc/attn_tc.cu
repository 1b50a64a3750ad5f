// Segment-masked attention, forward and backward, on the packed tokens with tcgen05 tensor cores (Sec. 3.2: packed
// tokens attend only to tokens of the same image; the 2L^2C term of Eq. 9).
//
// A CTA owns 128 consecutive packed query rows of one head, wherever image boundaries fall, and
// walks the key range spanned by the segments of those rows in tiles of 128 keys; cu_seqlens alone
// decides the range, so no padding token is ever loaded or multiplied.  Per key tile:
//   S = Q K^T        tcgen05.mma, Q and K tiles staged by TMA (K two tiles ahead, V one), S in TMEM (fp32)
//   P = exp2(S - m)  two threads per query row pull their halves of the S row into registers in one TMEM pass, mask
//                    keys outside the row's own segment, update the running sum, write P back to TMEM as bf16
//   O += P V         tcgen05.mma with P read from TMEM and V from shared memory; O accumulates in TMEM over all tiles
// m is the maximum that the stored P and O refer to.  It is raised - and O rescaled, TMEM -> registers -> TMEM - only
// when a row's true maximum has outgrown it by more than 2^8, so most tiles cost no pass over O; sums and outputs are
// exact for any reference value.  One elected lane of a ninth warp issues every copy and every product: the next tile's
// S product is issued as soon as every softmax warp holds the current S row, so the tensor core works under the
// softmax.  K/V rows past the last valid packed row are unspecified memory: K columns are masked after the
// product and V lines are zeroed in shared memory before the product.
#include <math_constants.h>

#include <mutex>

#include "sm100_ptx.cuh"
#include "spa_tc.cuh"

namespace spa {
namespace {

constexpr int kQ = 128;        // query rows per CTA = TMEM lanes
constexpr int kKV = 128;       // keys per tile
constexpr int kSoftmaxThreads = 256;  // two threads per query row: each owns half of the key columns and half of d
constexpr int kFwdThreads = kSoftmaxThreads + 32;  // and one warp, one lane of which issues every copy and product
constexpr float kRescaleGap = 8.f;  // log2 units by which a row's maximum may outgrow the one its P and O refer to
constexpr uint32_t kTmemCols = 256;  // S: 128 fp32 columns, P: 64 (bf16 pairs), O tile: up to 64
constexpr uint32_t kColS = 0, kColP = 128, kColO = 192;

template <int D> struct HeadTile {
  static constexpr int kRowBytes = D * 2;          // 128 (d = 64) or 64 (d = 32): also the swizzle span
  static constexpr int kTileBytes = 128 * kRowBytes;
  static constexpr int kSbo = 8 * kRowBytes;
  // K-major operand (Q or K rows, head dimension contiguous), k-th group of 16 head dimensions
  __device__ static __forceinline__ uint64_t kmajor(uint32_t addr, int k) {
    return D == 64 ? ptx::smem_desc_sw128(addr + k * 32, 16, kSbo) : ptx::smem_desc_sw64(addr + k * 32, 16, kSbo);
  }
  // MN-major operand (V: key rows are the K dimension, head dimension contiguous), k-th group of 16 keys
  __device__ static __forceinline__ uint64_t mnmajor(uint32_t addr, int k) {
    return D == 64 ? ptx::smem_desc_sw128(addr + k * 16 * kRowBytes, 16, kSbo)
                   : ptx::smem_desc_sw64(addr + k * 16 * kRowBytes, 16, kSbo);
  }
};

constexpr int kSegStage = 512;  // segment offsets are searched in shared memory when there are at most this many

// Segment bounds of packed row i (hi clamped to the valid rows) from offsets held in shared memory.
__device__ __forceinline__ RowSeg row_segment_staged(const int32_t* s_off, int n_seg, int Np, int i) {
  RowSeg r{0, 0};
  if (i < Np) {
    int lo = 0, hi = n_seg;  // invariant: s_off[lo] <= i < s_off[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_off[mid] <= i) lo = mid; else hi = mid;
    }
    r.lo = s_off[lo];
    const int h2 = s_off[lo + 1];
    r.hi = h2 < Np ? h2 : Np;
  }
  return r;
}

constexpr int kShortMax = 128;  // segments of at most this many rows are taken by the one-pass backward kernel

// Does the tile of packed rows [r0, r0 + 128) hold a row of a segment longer than kShortMax?  Such a segment covers
// the tile's first or its last valid row (one that lies strictly inside the tile has fewer rows than the tile), so two
// searches decide.  Every thread of a CTA gets the same answer.
__device__ __forceinline__ bool tile_has_long_rows(const int32_t* s_off, const int32_t* g_off, bool staged, int n_seg, int Np,
                                                   int r0) {
  const int last = r0 + 127 < Np - 1 ? r0 + 127 : Np - 1;
  const RowSeg a = staged ? row_segment_staged(s_off, n_seg, Np, r0) : row_segment(g_off, n_seg, Np, r0);
  if (a.hi - a.lo > kShortMax) return true;
  const RowSeg b = staged ? row_segment_staged(s_off, n_seg, Np, last) : row_segment(g_off, n_seg, Np, last);
  return b.hi - b.lo > kShortMax;
}

// Rotation of the 16-byte chunks of row r of a [128][D] bf16 tile in shared memory that makes the
// accesses of 8 neighbouring rows to one chunk index fall into different banks.
template <int D> __device__ __forceinline__ int chunk_rot(int r) { return D == 64 ? (r & 7) : ((r >> 1) & 3); }

// Copy a [128][D] bf16 tile that the threads wrote to shared memory (chunk c of row r at position
// c ^ chunk_rot(r)) to rows r0.. of a matrix with `ld` elements per row: a warp covers whole rows, so the
// stores are full 64- or 128-byte lines.  Rows from Np on are not written.
template <int D, int kThreads>
__device__ __forceinline__ void copy_tile_out(const uint8_t* tile, __nv_bfloat16* dst, long long ld, int r0, int Np, int tid,
                                              const volatile uint8_t* row_ok = nullptr) {
  constexpr int kChunks = D * 2 / 16;
#pragma unroll
  for (int i = tid; i < 128 * kChunks; i += kThreads) {
    const int r = i / kChunks, c = i % kChunks;
    if (r0 + r < Np && (row_ok == nullptr || row_ok[r]))
      *reinterpret_cast<uint4*>(dst + (long long)(r0 + r) * ld + c * 8) =
          *reinterpret_cast<const uint4*>(tile + r * (D * 2) + ((c ^ chunk_rot<D>(r)) << 4));
  }
}

template <int D> __host__ __device__ constexpr int fwd_smem_bytes() {
  // Q + 2 x (K, V), alignment slack, barriers, row-max exchange, segment offsets
  return 5 * 128 * D * 2 + 1024 + 128 + 2048 + kSegStage * 4 + 64;
}

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tm, const int32_t* __restrict__ seg, int n_seg, int capacity,
                   int C, int H, float scale_log2e, __nv_bfloat16* __restrict__ ao, float* __restrict__ lse,
                   int32_t* d_status) {
  using HT = HeadTile<D>;
  constexpr int kTile = HT::kTileBytes;
  // A CTA takes the work items blockIdx.x, blockIdx.x + gridDim.x, ... of the (tile, head) pairs that the device-side
  // row count leaves (heads fastest, so that CTAs running side by side share their K / V tiles in L2): no CTA is
  // launched for rows that do not exist, and TMEM and the staged segment offsets are set up once per CTA.
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool is_softmax = warp < kSoftmaxThreads / 32;  // warps 0-7; warp 8 issues the copies and the products
  // warps w and w + 4 may touch the same quarter of the TMEM lanes: they share 32 query rows and split
  // the work of each row (key columns of S and P, head dimensions of O) in two halves
  const int quarter = warp & 3, half = (warp >> 2) & 1, rl = quarter * 32 + lane;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t q_s = smem_base;
  auto k_s = [&](int st) { return smem_base + kTile * (1 + 2 * st); };
  auto v_s = [&](int st) { return smem_base + kTile * (2 + 2 * st); };
  const uint32_t bar_base = smem_base + 5 * kTile;
  const uint32_t bar_q = bar_base, bar_s = bar_base + 40, bar_o = bar_base + 48;
  const uint32_t bar_sfree = bar_base + 56;   // 8 arrivals: every softmax warp holds its part of S_t in registers
  const uint32_t bar_pready = bar_base + 64;  // 8 arrivals: every softmax warp has written its part of P_t
  auto bar_k = [&](int st) { return bar_base + 8 + 8 * st; };
  auto bar_v = [&](int st) { return bar_base + 24 + 8 * st; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_al + 5 * kTile + 72);
  volatile int* abort_any = reinterpret_cast<volatile int*>(smem_al + 5 * kTile + 76);
  volatile int* range = reinterpret_cast<volatile int*>(smem_al + 5 * kTile + 80);
  // [2 tile parities][4 quarters]: written by the two warps of a quarter before their barrier, read after it
  volatile int* abort_pair = reinterpret_cast<volatile int*>(smem_al + 5 * kTile + 88);
  float* xch = reinterpret_cast<float*>(smem_al + 5 * kTile + 128);  // [2 tile parities][2 halves][128 rows]
  int32_t* seg_s = reinterpret_cast<int32_t*>(smem_al + 5 * kTile + 128 + 2048);  // [kSegStage + 1]

  // The thread that sets the barriers up is the one that later issues the copies counted on them (program order: no
  // copy can meet a barrier that is not initialised yet).
  auto init_barriers = [&]() {
    ptx::mbar_init(bar_q, 1);
    for (int s = 0; s < 2; ++s) { ptx::mbar_init(bar_k(s), 1); ptx::mbar_init(bar_v(s), 1); }
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_o, 1);
    ptx::mbar_init(bar_sfree, kSoftmaxThreads / 32);
    ptx::mbar_init(bar_pready, kSoftmaxThreads / 32);
    *abort_any = 0;
    for (int i = 0; i < 8; ++i) abort_pair[i] = 0;
    ptx::fence_mbar_init();
  };
  // everything up to the wait touches no global memory, so it runs under the previous kernel's tail
  if (tid == kSoftmaxThreads) {
    ptx::prefetch_tensormap(&tm);
    init_barriers();
  }
  pdl_entry();
  const bool staged = n_seg < kSegStage;
  if (staged)
    for (int i = tid; i <= n_seg; i += kFwdThreads) seg_s[i] = __ldg(seg + i);
  const int Np = packed_rows(seg, n_seg, capacity);
  const int n_items = ((Np + kQ - 1) / kQ) * H;
  if ((int)blockIdx.x >= n_items) return;
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  bool cta_failed = false;
  for (int item = blockIdx.x; item < n_items && !cta_failed; item += gridDim.x) {
  const int h = item % H, q0 = (item / H) * kQ;
  if (tid == kSoftmaxThreads) {
    if (item != (int)blockIdx.x) {  // every phase of the previous item has completed: the barriers start over
      ptx::mbar_inval(bar_q);
      for (int s = 0; s < 2; ++s) { ptx::mbar_inval(bar_k(s)); ptx::mbar_inval(bar_v(s)); }
      ptx::mbar_inval(bar_s);
      ptx::mbar_inval(bar_o);
      ptx::mbar_inval(bar_sfree);
      ptx::mbar_inval(bar_pready);
      init_barriers();
    }
    // the Q tile depends only on q0: fetch it under the segment search
    ptx::mbar_expect_tx(bar_q, kTile);
    ptx::tma_load_2d(q_s, &tm, bar_q, h * D, q0);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // barriers, TMEM address and staged offsets are visible
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  const int row = q0 + rl;
  RowSeg mine{0, 0};
  if (is_softmax) {
    mine = staged ? row_segment_staged(seg_s, n_seg, Np, row) : row_segment(seg, n_seg, Np, row);
    if (half == 0) {
      const int last = (q0 + kQ - 1 < Np - 1) ? q0 + kQ - 1 : Np - 1;
      if (row == q0) range[0] = mine.lo;
      if (row == last) range[1] = mine.hi;
    }
  }
  __syncthreads();
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;  // TMEM lanes this warp may touch
  float lse_m = 0.f;
  constexpr int kCols = kKV / 2;  // key columns of each tile owned by this thread
  constexpr int kDh = D / 2;      // head dimensions of O owned by this thread
  const int col0 = half * kCols;
  const int kv_lo = range[0], kv_hi = range[1];
  const int n_tiles = (kv_hi - kv_lo + kKV - 1) / kKV;

  constexpr uint32_t kIdescS = ptx::idesc_bf16_f32(kQ, kKV, false, false);
  constexpr uint32_t kIdescO = ptx::idesc_bf16_f32(kQ, D, false, true);

  // Bounded wait that also gives up as soon as any thread of the CTA has reported a failure.
  auto wait = [&](uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < ptx::kWaitLimit; ++i) {
      if (ptx::mbar_try_wait(bar, parity)) return true;
      if ((i & 255u) == 255u && *abort_any) return false;
    }
    return false;
  };

  // every lane polls (measured faster than one lane polling for the warp); the warp takes one answer
  auto wait_w = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, wait(bar, parity)) != 0; };
  if (!is_softmax) {
    // ---------------------------------------------------------------- copies and products: one warp, whose lanes
    // all follow the tiles and take every wait together; one elected lane issues (see ptx::elect_one)
    auto load_k = [&](int t) {
      if (ptx::elect_one()) {
        ptx::mbar_expect_tx(bar_k(t & 1), kTile);
        ptx::tma_load_2d(k_s(t & 1), &tm, bar_k(t & 1), C + h * D, kv_lo + t * kKV);
      }
      __syncwarp();
    };
    auto load_v = [&](int t) {
      if (ptx::elect_one()) {
        ptx::mbar_expect_tx(bar_v(t & 1), kTile);
        ptx::tma_load_2d(v_s(t & 1), &tm, bar_v(t & 1), 2 * C + h * D, kv_lo + t * kKV);
      }
      __syncwarp();
    };
    auto issue_qk = [&](int t) {  // S = Q K_t^T into TMEM; bar_s completes when it is done
      if (!wait_w(bar_k(t & 1), (t >> 1) & 1)) return false;
      ptx::tc_fence_after_sync();
      const uint32_t ka = k_s(t & 1);
      if (ptx::elect_one()) {
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          ptx::mma_bf16(tmem + kColS, HT::kmajor(q_s, k), HT::kmajor(ka, k), kIdescS, k != 0 ? 1u : 0u);
        ptx::mma_commit(bar_s);
      }
      __syncwarp();
      return true;
    };
    int loads_k = 0, loads_v = 0;  // tiles whose loads have been issued
    bool ok = true;
    if (n_tiles > 0) {
      load_k(0);
      load_v(0);
      loads_k = loads_v = 1;
      if (n_tiles > 1) { load_k(1); loads_k = 2; }
      ok = wait_w(bar_q, 0) && issue_qk(0);
    }
    for (int t = 0; ok && t < n_tiles; ++t) {
      // every softmax thread holds its S_t columns: the S columns and K stage t & 1 are free
      if (!(ok = wait_w(bar_sfree, t & 1))) break;
      if (t + 1 < n_tiles) {
        if (!(ok = issue_qk(t + 1))) break;  // runs on the tensor core under the softmax of tile t
        if (t + 2 < n_tiles) { load_k(t + 2); loads_k = t + 3; }
      }
      // P_t is in TMEM, O has been rescaled where needed, and the previous P V product has completed
      if (!(ok = wait_w(bar_pready, t & 1))) break;
      if (!(ok = wait_w(bar_v(t & 1), (t >> 1) & 1))) break;
      ptx::tc_fence_after_sync();
      const uint32_t va = v_s(t & 1);
      if (ptx::elect_one()) {
#pragma unroll
        for (int k = 0; k < kKV / 16; ++k)
          ptx::mma_bf16_ts(tmem + kColO, tmem + kColP + k * 8, HT::mnmajor(va, k), kIdescO, (k != 0 || t > 0) ? 1u : 0u);
        ptx::mma_commit(bar_o);
      }
      __syncwarp();
      if (t + 1 < n_tiles) { load_v(t + 1); loads_v = t + 2; }  // its stage held V of tile t - 1
    }
    if (!ok && lane == 0) {
      record_status(d_status, SPA_ERR_TIMEOUT);
      *abort_any = 1;
      // let outstanding loads land before shared memory is released
      for (int t = loads_k > 2 ? loads_k - 2 : 0; t < loads_k; ++t) ptx::mbar_wait(bar_k(t & 1), (t >> 1) & 1);
      for (int t = loads_v > 2 ? loads_v - 2 : 0; t < loads_v; ++t) ptx::mbar_wait(bar_v(t & 1), (t >> 1) & 1);
      ptx::mbar_wait(bar_q, 0);
    }
  } else {
    // ---------------------------------------------------------------- online softmax: two threads per query row
    float m = -CUDART_INF_F, l = 0.f;  // m: the maximum the stored P and O refer to (may lag the true one by kRescaleGap)
    const unsigned span = (unsigned)(mine.hi - mine.lo);
    auto fail = [&](int slot) {
      record_status(d_status, SPA_ERR_TIMEOUT);
      abort_pair[slot * 4 + quarter] = 1;
      *abort_any = 1;
    };
    for (int t = 0; t < n_tiles; ++t) {
      const int st = t & 1;
      const int kv0 = kv_lo + t * kKV;
      // ---- S_t into registers: TMEM loads in flight together, one wait
      if (!wait_w(bar_s, t & 1)) fail(t & 1);
      ptx::tc_fence_after_sync();
      uint32_t s[kCols];
#pragma unroll
      for (int c = 0; c < kCols / 32; ++c) ptx::tmem_ld_32x32(tmem + lane_base + kColS + col0 + c * 32, s + c * 32);
      ptx::tmem_ld_wait();
      // Which of this thread's groups of 32 key columns meet its row's segment at all (the others take no
      // arithmetic: their P is zero); the mask is applied only where a boundary of the segment crosses a group.
      // This half's row maximum is handed to the partner thread through shared memory.
      const int kc0 = kv0 + col0;
      bool need[kCols / 32];
#pragma unroll
      for (int c = 0; c < kCols / 32; ++c) {
        const int g0 = kc0 + c * 32;
        need[c] = g0 < mine.hi && g0 + 32 > mine.lo;
        if (need[c] && !(g0 >= mine.lo && g0 + 32 <= mine.hi)) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if ((unsigned)(g0 + j - mine.lo) >= span) s[c * 32 + j] = 0xff800000u;  // -inf
        }
      }
      float mx[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int c = 0; c < kCols / 32; ++c) {
        if (need[c]) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) mx[u] = fmaxf(mx[u], __uint_as_float(s[c * 32 + j + u]));
          }
        }
      }
      float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      xch[((t & 1) * 2 + half) * 128 + rl] = mt;
      ptx::tc_fence_before_sync();
      ptx::named_barrier(1 + quarter, 64);  // the two warps that share these 32 rows
      if (abort_pair[(t & 1) * 4 + quarter]) break;
      if (lane == 0) ptx::mbar_arrive(bar_sfree);

      // ---- this half row's P (exp2 domain): one fma, one ex2 and one add per key.  The maximum that P and O
      // refer to is raised only when the true one has grown by more than kRescaleGap, so O (accumulated in
      // TMEM over all tiles) is rescaled rarely; sums and outputs are exact for any such reference value.
      mt = fmaxf(mt, xch[((t & 1) * 2 + (half ^ 1)) * 128 + rl]);
      const float m_cand = fmaxf(m, mt * scale_log2e);  // the scale is positive: max commutes with it
      const bool raise = m_cand > m + kRescaleGap;      // also the first tile that has a key of this row
      const float m_new = raise ? m_cand : m;
      const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
      const float alpha = raise ? ptx::ex2_approx(m - m_use) : 1.f;
      float rs0 = 0.f, rs1 = 0.f;
      uint32_t pk[kCols / 2];
#pragma unroll
      for (int c = 0; c < kCols / 32; ++c) {
        if (need[c]) {
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float p0 = ptx::ex2_approx(fmaf(__uint_as_float(s[c * 32 + j]), scale_log2e, -m_use));  // -inf -> 0
            const float p1 = ptx::ex2_approx(fmaf(__uint_as_float(s[c * 32 + j + 1]), scale_log2e, -m_use));
            rs0 += p0;
            rs1 += p1;
            __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);  // low half = even key
            pk[c * 16 + (j >> 1)] = *reinterpret_cast<uint32_t*>(&b);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) pk[c * 16 + j] = 0u;
        }
      }
      // ---- the previous P V product must have completed before P is overwritten or O rescaled
      if (t > 0) {
        if (!wait_w(bar_o, (t - 1) & 1)) fail((t + 1) & 1);
        ptx::tc_fence_after_sync();
        if (__any_sync(0xffffffffu, raise)) {
          uint32_t r[kDh];
          if (kDh == 32) ptx::tmem_ld_32x32(tmem + lane_base + kColO + half * kDh, r);
          else ptx::tmem_ld_32x16(tmem + lane_base + kColO + half * kDh, r);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < kDh; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
          if (kDh == 32) ptx::tmem_st_32x32(tmem + lane_base + kColO + half * kDh, r);
          else ptx::tmem_st_32x16(tmem + lane_base + kColO + half * kDh, r);
        }
      }
#pragma unroll
      for (int c = 0; c < kCols / 32; ++c)
        ptx::tmem_st_32x16(tmem + lane_base + kColP + (col0 >> 1) + c * 16, pk + c * 16);
      ptx::tmem_st_wait();
      l = l * alpha + (rs0 + rs1);
      m = m_new;
      // ---- V lines past the last valid packed row must not reach the product
      if (kv0 + kKV > Np) {
        if (!wait(bar_v(st), (t >> 1) & 1)) fail((t + 1) & 1);
        const int first = Np - kv0;  // >= 1
        constexpr int kChunks = HT::kRowBytes / 16;
        for (int c = tid; c < (kKV - first) * kChunks; c += kSoftmaxThreads)
          *reinterpret_cast<uint4*>(smem_al + kTile * (2 + 2 * st) + (first + c / kChunks) * HT::kRowBytes +
                                    (c % kChunks) * 16) = make_uint4(0, 0, 0, 0);
        ptx::fence_proxy_async_smem();
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_pready);
    }
    // the last product completes O
    const bool gave_up = __shfl_sync(0xffffffffu, *abort_any, 0) != 0;  // one answer per warp
    if (n_tiles > 0 && !gave_up && !wait_w(bar_o, (n_tiles - 1) & 1)) fail(0);
    xch[half * 128 + rl] = l;  // the two halves of a row share the reference maximum but kept separate sums
    lse_m = m;
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // nobody reports a failure from here on: the branches below are taken by all threads or by none
  ptx::tc_fence_after_sync();
  const bool failed = *abort_any != 0;
  if (!failed && is_softmax) {
    // normalised rows go to the Q tile's shared memory (idle now: every product has completed) as bf16 and
    // leave from there as whole lines
    uint32_t r[kDh];
    if (n_tiles > 0) {
      if (kDh == 32) ptx::tmem_ld_32x32(tmem + lane_base + kColO + half * kDh, r);
      else ptx::tmem_ld_32x16(tmem + lane_base + kColO + half * kDh, r);
      ptx::tmem_ld_wait();
    } else {
#pragma unroll
      for (int e = 0; e < kDh; ++e) r[e] = 0u;
    }
    const float l_row = xch[half * 128 + rl] + xch[(half ^ 1) * 128 + rl];
    const float inv_l = row < Np ? 1.f / l_row : 0.f;
    const int rot = chunk_rot<D>(rl);
#pragma unroll
    for (int c = 0; c < kDh / 8; ++c) {
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = row < Np ? __uint_as_float(r[c * 8 + e]) * inv_l : 0.f;
      *reinterpret_cast<uint4*>(smem_al + rl * HT::kRowBytes + (((half * (kDh / 8) + c) ^ rot) << 4)) =
          Vec16<__nv_bfloat16>::from_float(v);
    }
    if (half == 0 && row < Np) lse[(long long)h * capacity + row] = (lse_m + log2f(l_row)) * 0.6931471805599453f;
  }
  __syncthreads();
  if (!failed) copy_tile_out<D, kFwdThreads>(smem_al, ao + h * D, C, q0, Np, tid);
  cta_failed = failed;
  ptx::tc_fence_before_sync();
  __syncthreads();  // the tile's memory and the barriers are free for the next item
  }
  if (warp == 0) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(*tmem_slot, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Backward.
// Two passes over the same tile machinery, each accumulating its outputs in TMEM over its whole loop, so
// that no sum is split across CTAs (no float atomics, bitwise reproducible):
//   kDQ = true : a CTA owns 128 query rows i; per streamed tile of 64 keys   S = Q K^T, dP = dO V^T,
//                dS = P (dP - D_i) written to TMEM as bf16,   dQ += dS K.   Also stores D_i = dO_i . O_i.
//   kDQ = false: a CTA owns 128 key rows j; per streamed tile of 64 queries  S^T = K Q^T, dP^T = V dO^T,
//                P^T and dS^T written to TMEM as bf16,        dV += P^T dO,  dK += dS^T Q.
// The footprint is kept to 256 TMEM columns and about 80 KB of shared memory so that two CTAs share an
// SM.  Warps 0-7 do the arithmetic (two threads per row, 32 of the 64 streamed columns each); the first
// lane of warp 8 issues every copy and product and is told through mbarriers when the others hold a tile's
// fp32 values in registers and when its bf16 operands are in TMEM.
// The bf16 operands have TMEM columns of their own, so the next tile's fp32 products are issued as soon as
// the current ones are in registers and run under the arithmetic.  That needs room in TMEM: this kernel serves
// the dQ pass and the dK/dV pass at d = 32; the dK/dV pass at d = 64 is attn_bwd_kv_split_kernel below.
constexpr int kBwdMath = 256;      // arithmetic threads: two per TMEM lane (row)
constexpr int kBwdThreads = kBwdMath + 32;
constexpr int kBwdY = 64;          // rows of a streamed tile
constexpr uint32_t kBwdTmemCols = 256;
constexpr uint32_t kColS1 = 0, kColS2 = 64, kColAcc1 = 128, kColAcc2 = 192;
constexpr int kBwdStatBytes = 3 * 2 * kBwdY * 4;  // three tiles' worth of lse_i and D_i of the streamed queries

// Streamed tiles in shared memory.  In the dQ pass the first of them is the memory of the O tile, which is only
// needed for D_i before the loop starts.  A stage is as large as an own tile (two 64-row tiles).
template <int D, bool kDQ> __host__ __device__ constexpr int bwd_stages() { return D == 32 ? 6 : (kDQ ? 4 : 3); }
template <int D, bool kDQ> __host__ __device__ constexpr int bwd_smem_bytes() {
  // two own tiles, streamed stages, alignment slack, statistics, barriers, segment offsets, row flags
  return (2 + bwd_stages<D, kDQ>()) * 128 * D * 2 + 1024 + kBwdStatBytes + 128 + kSegStage * 4 + 64 + 128;
}

template <int D, bool kDQ, bool kLoop>
__global__ void __launch_bounds__(kBwdThreads, 2)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap tm_qkv, const __grid_constant__ CUtensorMap tm_do,
                   const __grid_constant__ CUtensorMap tm_qkv_y, const __grid_constant__ CUtensorMap tm_do_y,
                   const __grid_constant__ CUtensorMap tm_o,
                   const float* __restrict__ lse, float* __restrict__ delta, const int32_t* __restrict__ seg, int n_seg,
                   int capacity, int C, int H, float scale, __nv_bfloat16* __restrict__ dqkv, int skip_short, int32_t* d_status) {
  using HT = HeadTile<D>;
  constexpr int kTile = HT::kTileBytes;             // own tiles: 128 rows
  constexpr int kYTile = kBwdY * HT::kRowBytes;     // streamed tiles: 64 rows
  constexpr int kStages = bwd_stages<D, kDQ>();     // streamed stages; in the dQ pass stage 0 first holds the O tile
  constexpr int kShift = kDQ ? 1 : 0;               // tile t lives in stage (t + kShift) mod kStages
  static_assert(2 * kYTile == kTile, "a stage is as large as an own tile");
  constexpr float kLog2e = 1.4426950408889634f;
  // the bf16 operands have TMEM columns of their own, so the next fp32 products need not wait for the accumulating ones
  static_assert(kDQ || D == 32, "the dK / dV pass at d = 64 fills TMEM: attn_bwd_kv_split_kernel");
  constexpr uint32_t kColOpP = 160u;                // P^T (dK/dV pass only)
  constexpr uint32_t kColOpDS = kDQ ? 192u : 224u;  // dS or dS^T
  // dQ pass: the last 32 columns hold the Q tile (d = 64) or the Q and the dO tile (d = 32, 16 columns each) as bf16
  // operands, so that S = Q K^T (and dP = dO V^T) reads only the streamed tile from shared memory (a product with both
  // operands there is bound by the operand read: 52 clocks against 36)
  constexpr bool kQTmem = kDQ;
  constexpr bool kDoTmem = kDQ && D == 32;
  constexpr uint32_t kColQ = 224u, kColDO = 240u;
  // A CTA takes the work items blockIdx.x, blockIdx.x + gridDim.x, ... of the (tile, head) pairs that the device-side
  // row count leaves (heads fastest); TMEM and the staged segment offsets are set up once per CTA.
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool is_math = warp < kBwdMath / 32;
  // warps w and w + 4 may touch the same quarter of the TMEM lanes: they share 32 rows and split the columns
  const int quarter = warp & 3, half = (warp >> 2) & 1, rl = quarter * 32 + lane;
  const float scale_log2e = scale * kLog2e;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t x1_s = smem_base, x2_s = smem_base + kTile, x3_s = smem_base + 2 * kTile;
  constexpr int kYBase = 2 * kTile;
  auto y1_off = [&](int st) { return kYBase + kYTile * (2 * st); };
  auto y2_off = [&](int st) { return kYBase + kYTile * (2 * st + 1); };
  auto stage_of = [&](int t_) { return (t_ + kShift) % kStages; };
  auto use_of = [&](int t_) { return (uint32_t)(((t_ + kShift) / kStages) & 1); };  // parity of that stage's barrier
  constexpr int kStatBase = kYBase + kStages * 2 * kYTile;
  float* stat_lse = reinterpret_cast<float*>(smem_al + kStatBase);  // [3][64] lse_i * log2e of the staged query tile
  float* stat_D = stat_lse + 3 * kBwdY;                              // [3][64] D_i
  constexpr int kBarBase = kStatBase + kBwdStatBytes;
  const uint32_t bar_base = smem_base + kBarBase;
  const uint32_t bar_x = bar_base, bar_s = bar_base + 56, bar_acc = bar_base + 64;
  const uint32_t bar_sfree = bar_base + 72;    // 8 arrivals: every arithmetic warp holds the fp32 values of tile t
  const uint32_t bar_opready = bar_base + 80;  // 8 arrivals: every arithmetic warp has written the operands of tile t
  auto bar_y = [&](int st) { return bar_base + 8 + 8 * st; };  // up to six stages
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_al + kBarBase + 88);
  volatile int* abort_any = reinterpret_cast<volatile int*>(smem_al + kBarBase + 92);
  volatile int* range = reinterpret_cast<volatile int*>(smem_al + kBarBase + 96);
  int32_t* seg_s = reinterpret_cast<int32_t*>(smem_al + kBarBase + 128);  // [kSegStage + 1]
  // rows of this tile whose results this kernel writes (all valid rows, or those of the long segments only)
  volatile uint8_t* row_ok = reinterpret_cast<volatile uint8_t*>(smem_al + kBarBase + 128 + kSegStage * 4 + 64);

  // The thread that sets the barriers up is the one that later issues the copies counted on them.
  auto init_barriers = [&]() {
    range[0] = 0x7fffffff;
    range[1] = 0;
    ptx::mbar_init(bar_x, 1);
    for (int s3 = 0; s3 < kStages; ++s3) ptx::mbar_init(bar_y(s3), 1);
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_acc, 1);
    ptx::mbar_init(bar_sfree, kBwdMath / 32);
    ptx::mbar_init(bar_opready, kBwdMath / 32);
    *abort_any = 0;
    ptx::fence_mbar_init();
  };
  // everything up to the wait touches no global memory, so it runs under the previous kernel's tail
  if (tid == kBwdMath) {
    ptx::prefetch_tensormap(&tm_qkv);
    ptx::prefetch_tensormap(&tm_do);
    ptx::prefetch_tensormap(&tm_qkv_y);
    ptx::prefetch_tensormap(&tm_do_y);
    if (kDQ) ptx::prefetch_tensormap(&tm_o);
    init_barriers();
  }
  pdl_entry();
  const bool staged = n_seg < kSegStage;
  if (staged)
    for (int i = tid; i <= n_seg; i += kBwdThreads) seg_s[i] = __ldg(seg + i);
  const int Np = packed_rows(seg, n_seg, capacity);
  const int n_items = ((Np + 127) / 128) * H;
  if ((int)blockIdx.x >= n_items) return;
  if (skip_short) __syncthreads();  // the staged offsets are visible to the tile test
  bool cta_failed = false, first_item = true;
  int item = blockIdx.x;
  do {  // kLoop: this CTA strides over the items; otherwise the grid holds one CTA per item and this is no loop
  const int h = item % H, r0 = (item / H) * 128;
  // tiles whose rows all belong to the one-pass kernel are passed over before anything is fetched
  if (skip_short && !tile_has_long_rows(seg_s, seg, staged, n_seg, Np, r0)) continue;
  const int x1_col = (kDQ ? 0 : C) + h * D;           // own operand inside qkv: Q | K
  if (tid == kBwdMath) {
    if (!first_item) {  // every phase of the previous item has completed: the barriers start over
      ptx::mbar_inval(bar_x);
      for (int s3 = 0; s3 < kStages; ++s3) ptx::mbar_inval(bar_y(s3));
      ptx::mbar_inval(bar_s);
      ptx::mbar_inval(bar_acc);
      ptx::mbar_inval(bar_sfree);
      ptx::mbar_inval(bar_opready);
      init_barriers();
    }
    // the own tiles depend only on r0: fetch them under the segment search
    ptx::mbar_expect_tx(bar_x, 2 * kTile);
    ptx::tma_load_2d(x1_s, &tm_qkv, bar_x, x1_col, r0);
    if (kDQ) {
      ptx::tma_load_2d(x2_s, &tm_do, bar_x, h * D, r0);                  // dO
      ptx::mbar_expect_tx(bar_y(0), kTile);                              // first use of stage 0:
      ptx::tma_load_2d(x3_s, &tm_o, bar_y(0), h * D, r0);                // O, for D_i = dO_i . O_i
    } else {
      ptx::tma_load_2d(x2_s, &tm_qkv, bar_x, 2 * C + h * D, r0);         // V
    }
  }
  if (first_item && warp == 0) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), kBwdTmemCols);
  first_item = false;
  ptx::tc_fence_before_sync();
  __syncthreads();  // barriers, (first item) the TMEM address and the staged offsets are visible
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;

  const int row = r0 + rl;
  RowSeg mine{0, 0};
  if (is_math) {
    mine = staged ? row_segment_staged(seg_s, n_seg, Np, row) : row_segment(seg, n_seg, Np, row);
    // segments that fit one tile belong to the one-pass kernel: their rows are no rows of this one
    if (skip_short && mine.hi - mine.lo <= kShortMax) mine = RowSeg{0, 0};
    if (half == 0) {
      row_ok[rl] = mine.hi > mine.lo ? 1 : 0;
      if (mine.hi > mine.lo) {  // the rows of the other side to visit: the union of the segments of this tile's rows
        atomicMin(const_cast<int*>(range), mine.lo);
        atomicMax(const_cast<int*>(range) + 1, mine.hi);
      }
    }
  }
  __syncthreads();
  const bool any_row = range[1] > range[0];  // false: every row of the tile belongs to the one-pass kernel
  const int o_lo = any_row ? range[0] : 0, o_hi = any_row ? range[1] : 0;
  const int n_tiles = (o_hi - o_lo + kBwdY - 1) / kBwdY;

  const int y1_col = (kDQ ? C : 0) + h * D;           // streamed operand inside qkv: K | Q
  auto load_other = [&](int t_) {  // streamed tile t_ into its stage
    const int st = stage_of(t_), y0 = o_lo + t_ * kBwdY;
    ptx::mbar_expect_tx(bar_y(st), 2 * kYTile);
    ptx::tma_load_2d(smem_base + y1_off(st), &tm_qkv_y, bar_y(st), y1_col, y0);
    if (kDQ) ptx::tma_load_2d(smem_base + y2_off(st), &tm_qkv_y, bar_y(st), 2 * C + h * D, y0);   // V
    else ptx::tma_load_2d(smem_base + y2_off(st), &tm_do_y, bar_y(st), h * D, y0);                // dO
  };
  int issued = 0;  // streamed tiles whose loads have been issued (kept by the issuing thread)
  if (tid == kBwdMath) {
    for (int t_ = 0; t_ < n_tiles && t_ < kStages - 1; ++t_) load_other(t_);  // the stages that are free at the start
    issued = n_tiles < kStages - 1 ? n_tiles : kStages - 1;
  }

  // Bounded wait that also gives up as soon as any thread of the CTA has reported a failure.
  auto wait = [&](uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < ptx::kWaitLimit; ++i) {
      if (ptx::mbar_try_wait(bar, parity)) return true;
      if ((i & 255u) == 255u && *abort_any) return false;
    }
    return false;
  };
  // every lane polls; the warp takes one answer, so that a whole warp gives up or none of it
  auto wait_w = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, wait(bar, parity)) != 0; };

  // per-row statistics of the query side
  float my_lse = 0.f, my_D = 0.f;   // kDQ: this thread's query row
  float nxt_lse = 0.f, nxt_D = 0.f; // !kDQ: prefetched values of the next streamed query tile, row rl < 64
  if (is_math) {
    if (kDQ) {
      if (mine.hi > mine.lo) my_lse = lse[(long long)h * capacity + row] * kLog2e;
    } else if (half == 0 && rl < kBwdY) {
      const int i = o_lo + rl;
      if (i < o_hi) { nxt_lse = lse[(long long)h * capacity + i] * kLog2e; nxt_D = delta[(long long)h * capacity + i]; }
    }
  }

  constexpr uint32_t kIdescS = ptx::idesc_bf16_f32(128, kBwdY, false, false);
  constexpr uint32_t kIdescAcc = ptx::idesc_bf16_f32(128, D, false, true);
  const unsigned span = (unsigned)(mine.hi - mine.lo);

  // Make streamed tile t_ ready for the products (arithmetic warps): its load has landed, lines past the last
  // valid packed row are zeroed (they are unspecified memory and would be summed over), its query statistics
  // are staged.  Returns false when the wait for the load gave up.
  auto prep = [&](int t_) {
    const int st = stage_of(t_);
    bool ok = true;
    const int y0 = o_lo + t_ * kBwdY;
    // the issuing thread waits for the load itself; the arithmetic warps need it only where they touch the tile
    if (t_ == 0) {
      ok = wait_w(bar_y(st), use_of(t_));
      ok = wait_w(bar_x, 0) && ok;
      if (kDQ) ok = wait_w(bar_y(0), 0) && ok;  // the O tile
    } else if (y0 + kBwdY > Np) {
      ok = wait_w(bar_y(st), use_of(t_));
    }
    if (y0 + kBwdY > Np) {
      const int first = Np - y0;
      constexpr int kChunks = HT::kRowBytes / 16;
      for (int c = tid; c < (kBwdY - first) * kChunks; c += kBwdMath) {
        const int off = (first + c / kChunks) * HT::kRowBytes + (c % kChunks) * 16;
        *reinterpret_cast<uint4*>(smem_al + y1_off(st) + off) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(smem_al + y2_off(st) + off) = make_uint4(0, 0, 0, 0);
      }
      ptx::fence_proxy_async_smem();
    }
    if (!kDQ && half == 0 && rl < kBwdY) {
      stat_lse[(t_ % 3) * kBwdY + rl] = nxt_lse;
      stat_D[(t_ % 3) * kBwdY + rl] = nxt_D;
      const int i = y0 + kBwdY + rl;
      nxt_lse = 0.f; nxt_D = 0.f;
      if (i < o_hi) { nxt_lse = lse[(long long)h * capacity + i] * kLog2e; nxt_D = delta[(long long)h * capacity + i]; }
    }
    return ok;
  };

  if (is_math && n_tiles > 0 && !prep(0)) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_any = 1; }
  if (kQTmem && is_math && n_tiles > 0) {
    // the own tiles have landed (prep(0) waited for them).  d = 64: each of a row's two threads moves its half of the
    // Q row; d = 32: one moves the Q row, the other the dO row (16 columns either way).
    uint32_t q[16];
    const uint8_t* src = smem_al + (D == 32 && half == 1 ? kTile : 0) + rl * HT::kRowBytes;
    const int c0 = D == 64 ? half * 4 : 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint4 v = *reinterpret_cast<const uint4*>(src + (((c0 + c) ^ chunk_rot<D>(rl)) << 4));
      q[4 * c] = v.x; q[4 * c + 1] = v.y; q[4 * c + 2] = v.z; q[4 * c + 3] = v.w;
    }
    ptx::tmem_st_32x16(tmem + lane_base + (D == 64 ? kColQ + half * 16 : (half == 0 ? kColQ : kColDO)), q);
    ptx::tmem_st_wait();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // tile 0 is ready; a failure so far is seen by all threads or by none
  const bool failed_early = *abort_any != 0 || n_tiles == 0;

  if (!is_math) {
    // ---------------------------------------------------------------- copies and products: one warp, whose lanes
    // all follow the tiles and take every wait together; one elected lane issues (see ptx::elect_one)
    if (!failed_early) {
      auto issue_s = [&](int t_) {  // the two fp32 tiles of streamed tile t_ (S and dP, or their transposes)
        const int st = stage_of(t_);
        const uint32_t y1a = smem_base + y1_off(st), y2a = smem_base + y2_off(st);
        if (ptx::elect_one()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            if (kQTmem) ptx::mma_bf16_ts(tmem + kColS1, tmem + kColQ + k * 8, HT::kmajor(y1a, k), kIdescS, k != 0 ? 1u : 0u);
            else ptx::mma_bf16(tmem + kColS1, HT::kmajor(x1_s, k), HT::kmajor(y1a, k), kIdescS, k != 0 ? 1u : 0u);
          }
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            if (kDoTmem) ptx::mma_bf16_ts(tmem + kColS2, tmem + kColDO + k * 8, HT::kmajor(y2a, k), kIdescS, k != 0 ? 1u : 0u);
            else ptx::mma_bf16(tmem + kColS2, HT::kmajor(x2_s, k), HT::kmajor(y2a, k), kIdescS, k != 0 ? 1u : 0u);
          }
          ptx::mma_commit(bar_s);
        }
        __syncwarp();
      };
      bool ok = true;
      ptx::tc_fence_after_sync();
      if (n_tiles > 0) issue_s(0);
      for (int t = 0; ok && t < n_tiles; ++t) {
        const int st = stage_of(t);
        if (t + 1 < n_tiles) {
          // the fp32 values of tile t are in registers and tile t + 1 is ready: its products run under the arithmetic
          if (!(ok = wait_w(bar_sfree, t & 1))) break;
          if (!(ok = wait_w(bar_y(stage_of(t + 1)), use_of(t + 1)))) break;
          ptx::tc_fence_after_sync();
          issue_s(t + 1);
        }
        // the stage of tile t - 1 is free once its accumulating products have completed; at t = 0 the stage that
        // is filled is the last one, or in the dQ pass the O tile's memory, which the arithmetic warps have finished
        // with before they announce tile 0 (waited for above: a tile to prefetch implies a tile t + 1)
        if (t + kStages - 1 < n_tiles) {
          if (t > 0 && !(ok = wait_w(bar_acc, (t - 1) & 1))) break;
          if (ptx::elect_one()) load_other(t + kStages - 1);
          __syncwarp();
          issued = t + kStages;
        }
        if (!(ok = wait_w(bar_opready, t & 1))) break;
        ptx::tc_fence_after_sync();
        const uint32_t acc = (t != 0) ? 1u : 0u;
        const uint32_t y1a = smem_base + y1_off(st), y2a = smem_base + y2_off(st);
        if (ptx::elect_one()) {
          if (kDQ) {
#pragma unroll
            for (int k = 0; k < kBwdY / 16; ++k)   // dQ += dS K
              ptx::mma_bf16_ts(tmem + kColAcc1, tmem + kColOpDS + k * 8, HT::mnmajor(y1a, k), kIdescAcc, acc | (k != 0));
          } else {
#pragma unroll
            for (int k = 0; k < kBwdY / 16; ++k)   // dV += P^T dO
              ptx::mma_bf16_ts(tmem + kColAcc1, tmem + kColOpP + k * 8, HT::mnmajor(y2a, k), kIdescAcc, acc | (k != 0));
#pragma unroll
            for (int k = 0; k < kBwdY / 16; ++k)   // dK += dS^T Q
              ptx::mma_bf16_ts(tmem + kColAcc2, tmem + kColOpDS + k * 8, HT::mnmajor(y1a, k), kIdescAcc, acc | (k != 0));
          }
          ptx::mma_commit(bar_acc);
        }
        __syncwarp();
      }
      if (!ok && lane == 0) {
        record_status(d_status, SPA_ERR_TIMEOUT);
        *abort_any = 1;
      }
    }
  } else if (!failed_early) {
    // ---------------------------------------------------------------- arithmetic: two threads per row
    if (kDQ && mine.hi > mine.lo) {
      // D_i = dO_i . O_i from the two staged tiles (their load has completed: prep(0) waited for it).  Both
      // carry the same swizzle, so equal positions hold equal columns and the order of the chunks is free:
      // each row starts at a different chunk to keep 8 neighbouring rows off one bank.
      constexpr int kChunks = HT::kRowBytes / 16;
      const uint8_t* po = smem_al + 2 * kTile + rl * HT::kRowBytes;
      const uint8_t* pg = smem_al + kTile + rl * HT::kRowBytes;
      const int rot = chunk_rot<D>(rl);
#pragma unroll
      for (int c = 0; c < kChunks; ++c) {
        float a[8], b[8];
        Vec16<__nv_bfloat16>::to_float(*reinterpret_cast<const uint4*>(po + ((c ^ rot) << 4)), a);
        Vec16<__nv_bfloat16>::to_float(*reinterpret_cast<const uint4*>(pg + ((c ^ rot) << 4)), b);
#pragma unroll
        for (int e = 0; e < 8; ++e) my_D = fmaf(a[e], b[e], my_D);
      }
      if (half == 0) delta[(long long)h * capacity + row] = my_D;
    }

    constexpr int kPc = kBwdY / 2;  // fp32 columns of each tile owned by this thread
    const int col0 = half * kPc;
    // no barrier joins the arithmetic warps inside the loop, so a warp whose wait gave up may leave it alone: the
    // others see the flag in their own waits
    auto fail = [&]() {
      record_status(d_status, SPA_ERR_TIMEOUT);
      *abort_any = 1;
    };
    for (int t = 0; t < n_tiles; ++t) {
      const int y0 = o_lo + t * kBwdY;
      // ---- this thread's columns of both fp32 tiles into registers
      bool ok = wait_w(bar_s, t & 1);
      ptx::tc_fence_after_sync();
      uint32_t rs[kPc], rp[kPc];
      ptx::tmem_ld_32x32(tmem + lane_base + kColS1 + col0, rs);
      ptx::tmem_ld_32x32(tmem + lane_base + kColS2 + col0, rp);
      ptx::tmem_ld_wait();
      if (ok && t + 1 < n_tiles) ok = prep(t + 1);
      // the statistics of tile t were staged by other warps before they announced tile t - 1 (that phase has
      // completed; it is waited for, before this warp's own arrival for tile t, to order the reads below)
      if (ok && !kDQ && t > 0) ok = wait_w(bar_sfree, (t - 1) & 1);
      if (!ok) { fail(); break; }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_sfree);

      // ---- P = 2^(S - lse), dS = P (dP - D).  A thread whose 32 columns lie wholly outside its row's segment
      // writes zeros without doing the arithmetic; the mask costs something only where a boundary crosses.
      const int yc0 = y0 + col0;
      uint32_t pk_p[kPc / 2], pk_ds[kPc / 2];
      if (yc0 < mine.hi && yc0 + kPc > mine.lo) {
        if (!(yc0 >= mine.lo && yc0 + kPc <= mine.hi)) {
#pragma unroll
          for (int j = 0; j < kPc; ++j)
            if ((unsigned)(yc0 + j - mine.lo) >= span) { rs[j] = 0xff800000u; rp[j] = 0u; }  // p = 2^-inf = 0, dP = 0
        }
        const float* sl = stat_lse + (t % 3) * kBwdY + col0;
        const float* sd = stat_D + (t % 3) * kBwdY + col0;
#pragma unroll
        for (int j = 0; j < kPc; j += 2) {
          float pv[2], dsv[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const float l2 = kDQ ? my_lse : sl[j + u];
            const float Dv = kDQ ? my_D : sd[j + u];
            pv[u] = ptx::ex2_approx(fmaf(__uint_as_float(rs[j + u]), scale_log2e, -l2));
            dsv[u] = pv[u] * (__uint_as_float(rp[j + u]) - Dv);
          }
          __nv_bfloat162 bds = __floats2bfloat162_rn(dsv[0], dsv[1]);
          pk_ds[j >> 1] = *reinterpret_cast<uint32_t*>(&bds);
          __nv_bfloat162 bp = __floats2bfloat162_rn(pv[0], pv[1]);
          pk_p[j >> 1] = *reinterpret_cast<uint32_t*>(&bp);
        }
      } else {
#pragma unroll
        for (int j = 0; j < kPc / 2; ++j) { pk_p[j] = 0u; pk_ds[j] = 0u; }
      }
      // The accumulating products of tile t - 1 must have read the operand columns.  (Two operand copies in the dQ
      // pass, written without this wait on the grounds that the fp32 products of tile t were committed after the
      // accumulating products of tile t - 2, gave sporadic non-finite dQ at d = 32: the wait stays.)
      if (t > 0) {
        if (!wait_w(bar_acc, (t - 1) & 1)) { fail(); break; }
        ptx::tc_fence_after_sync();
      }
      if (!kDQ) ptx::tmem_st_32x16(tmem + lane_base + kColOpP + (col0 >> 1), pk_p);
      ptx::tmem_st_32x16(tmem + lane_base + kColOpDS + (col0 >> 1), pk_ds);
      ptx::tmem_st_wait();
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_opready);
    }
    // the last accumulating products complete the outputs
    const bool gave_up = __shfl_sync(0xffffffffu, *abort_any, 0) != 0;  // one answer per warp
    if (n_tiles > 0 && !gave_up && !wait_w(bar_acc, (n_tiles - 1) & 1)) fail();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // nobody reports a failure from here on: the branches below are taken by all threads or by none
  ptx::tc_fence_after_sync();
  const bool failed = *abort_any != 0;

  if (!failed && n_tiles > 0) {
    // Each thread drains d/2 columns of its row of the accumulators into the own tiles' shared memory (idle
    // now: every product has completed), from where whole rows go out as full lines.
    constexpr int kDh = D / 2;
    auto stage_acc = [&](uint32_t acc_col, uint8_t* tile, float mul) {
      uint32_t r[kDh];
      if (kDh == 32) ptx::tmem_ld_32x32(tmem + lane_base + acc_col + half * kDh, r);
      else ptx::tmem_ld_32x16(tmem + lane_base + acc_col + half * kDh, r);
      ptx::tmem_ld_wait();
      const int rot = chunk_rot<D>(rl);
#pragma unroll
      for (int g = 0; g < kDh / 8; ++g) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[g * 8 + e]) * mul;
        *reinterpret_cast<uint4*>(tile + rl * HT::kRowBytes + (((half * (kDh / 8) + g) ^ rot) << 4)) =
            Vec16<__nv_bfloat16>::from_float(v);
      }
    };
    const long long ld = 3LL * C;
    if (kDQ) {
      if (is_math) stage_acc(kColAcc1, smem_al, scale);
      __syncthreads();
      copy_tile_out<D, kBwdThreads>(smem_al, dqkv + h * D, ld, r0, Np, tid, row_ok);
    } else {
      if (is_math) {
        stage_acc(kColAcc1, smem_al, 1.f);             // dV
        stage_acc(kColAcc2, smem_al + kTile, scale);   // dK
      }
      __syncthreads();
      copy_tile_out<D, kBwdThreads>(smem_al, dqkv + 2 * C + h * D, ld, r0, Np, tid, row_ok);
      copy_tile_out<D, kBwdThreads>(smem_al + kTile, dqkv + C + h * D, ld, r0, Np, tid, row_ok);
    }
  }
  if ((failed || n_tiles == 0) && tid == kBwdMath) {  // let outstanding loads land before shared memory is released
    for (int t = issued > kStages ? issued - kStages : 0; t < issued; ++t) ptx::mbar_wait(bar_y(stage_of(t)), use_of(t));
    if (kDQ && issued < kStages) ptx::mbar_wait(bar_y(0), 0);  // the O tile, if no streamed tile followed it there
    ptx::mbar_wait(bar_x, 0);
  }
  cta_failed = failed;
  ptx::tc_fence_before_sync();
  __syncthreads();  // the tiles' memory and the barriers are free for the next item
  } while (kLoop && (item += gridDim.x) < n_items && !cta_failed);
  if (!first_item && warp == 0) {  // TMEM was taken with the first item that this CTA worked on
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(*tmem_slot, kBwdTmemCols);
  }
}

// The dK / dV pass at d = 64 with the products running under the arithmetic.  S^T, dP^T, dV and dK fill the 256 TMEM
// columns of a CTA, so the bf16 operands live elsewhere: P^T in shared memory (the A operand of dV += P^T dO, K-major,
// written by the threads that computed it) and dS^T over the dP^T columns it was computed from.  The arithmetic of a
// tile splits the same way: P^T = 2^(S^T - lse) needs S^T only - it holds the exponentials, the expensive part - and
// runs while dP^T of the same tile is still being computed; dS^T = P^T (dP^T - D) follows.  Per tile the issuing warp
// queues S^T(t+1) (once every arithmetic warp holds S^T(t) in registers), dV(t) (P^T(t) written), dK(t) (dS^T(t)
// stored) and dP^T(t+1), the last behind dK(t), which reads the columns it overwrites.
constexpr int kSplitStages = 3;  // streamed stages of a 64-row Q tile and a 64-row dO tile
template <int D> __host__ __device__ constexpr int split_smem_bytes() {
  // own K and V, streamed stages, P^T, alignment slack, statistics, barriers, segment offsets, row flags
  return (2 + kSplitStages) * 128 * D * 2 + 128 * kBwdY * 2 + 1024 + kBwdStatBytes + 128 + kSegStage * 4 + 64 + 128;
}

template <int D, bool kLoop>
__global__ void __launch_bounds__(kBwdThreads, 2)
attn_bwd_kv_split_kernel(const __grid_constant__ CUtensorMap tm_qkv, const __grid_constant__ CUtensorMap tm_do,
                   const __grid_constant__ CUtensorMap tm_qkv_y, const __grid_constant__ CUtensorMap tm_do_y,
                   const __grid_constant__ CUtensorMap tm_o,
                   const float* __restrict__ lse, float* __restrict__ delta, const int32_t* __restrict__ seg, int n_seg,
                   int capacity, int C, int H, float scale, __nv_bfloat16* __restrict__ dqkv, int skip_short, int32_t* d_status) {
  using HT = HeadTile<D>;
  constexpr int kTile = HT::kTileBytes;             // own tiles: 128 rows
  constexpr int kYTile = kBwdY * HT::kRowBytes;     // streamed tiles: 64 rows
  constexpr int kStages = kSplitStages;             // streamed stages (a Q and a dO tile each): tile t lives in stage t mod kStages
  constexpr int kShift = 0;
  static_assert(2 * kYTile == kTile, "a stage is as large as an own tile");
  constexpr float kLog2e = 1.4426950408889634f;
  static_assert(D == 64, "d = 32 leaves TMEM columns for the operands: attn_bwd_tc_kernel");
  // A CTA takes the work items blockIdx.x, blockIdx.x + gridDim.x, ... of the (tile, head) pairs that the device-side
  // row count leaves (heads fastest); TMEM and the staged segment offsets are set up once per CTA.
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool is_math = warp < kBwdMath / 32;
  // warps w and w + 4 may touch the same quarter of the TMEM lanes: they share 32 rows and split the columns
  const int quarter = warp & 3, half = (warp >> 2) & 1, rl = quarter * 32 + lane;
  const float scale_log2e = scale * kLog2e;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t x1_s = smem_base, x2_s = smem_base + kTile;
  constexpr int kYBase = 2 * kTile;
  auto y1_off = [&](int st) { return kYBase + kYTile * (2 * st); };
  auto y2_off = [&](int st) { return kYBase + kYTile * (2 * st + 1); };
  auto stage_of = [&](int t_) { return (t_ + kShift) % kStages; };
  auto use_of = [&](int t_) { return (uint32_t)(((t_ + kShift) / kStages) & 1); };  // parity of that stage's barrier
  constexpr int kPBase = kYBase + kStages * 2 * kYTile;   // P^T of the current tile: [128 keys][64 queries] bf16, K-major
  const uint32_t p_s = smem_base + kPBase;
  constexpr int kStatBase = kPBase + kTile;
  float* stat_lse = reinterpret_cast<float*>(smem_al + kStatBase);  // [3][64] lse_i * log2e of the staged query tile
  float* stat_D = stat_lse + 3 * kBwdY;                              // [3][64] D_i
  constexpr int kBarBase = kStatBase + kBwdStatBytes;
  const uint32_t bar_base = smem_base + kBarBase;
  const uint32_t bar_x = bar_base, bar_s = bar_base + 32, bar_dp = bar_base + 40, bar_acc = bar_base + 48;
  const uint32_t bar_sfree = bar_base + 56;    // 8 arrivals: every arithmetic warp holds S^T of tile t in registers
  const uint32_t bar_pready = bar_base + 64;   // 8 arrivals: every arithmetic warp has written its part of P^T of tile t
  const uint32_t bar_dsready = bar_base + 72;  // 8 arrivals: every arithmetic warp has stored its part of dS^T of tile t
  auto bar_y = [&](int st) { return bar_base + 8 + 8 * st; };  // three stages
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_al + kBarBase + 88);
  volatile int* abort_any = reinterpret_cast<volatile int*>(smem_al + kBarBase + 92);
  volatile int* range = reinterpret_cast<volatile int*>(smem_al + kBarBase + 96);
  int32_t* seg_s = reinterpret_cast<int32_t*>(smem_al + kBarBase + 128);  // [kSegStage + 1]
  // rows of this tile whose results this kernel writes (all valid rows, or those of the long segments only)
  volatile uint8_t* row_ok = reinterpret_cast<volatile uint8_t*>(smem_al + kBarBase + 128 + kSegStage * 4 + 64);

  // The thread that sets the barriers up is the one that later issues the copies counted on them.
  auto init_barriers = [&]() {
    range[0] = 0x7fffffff;
    range[1] = 0;
    ptx::mbar_init(bar_x, 1);
    for (int s3 = 0; s3 < kStages; ++s3) ptx::mbar_init(bar_y(s3), 1);
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_dp, 1);
    ptx::mbar_init(bar_acc, 1);
    ptx::mbar_init(bar_sfree, kBwdMath / 32);
    ptx::mbar_init(bar_pready, kBwdMath / 32);
    ptx::mbar_init(bar_dsready, kBwdMath / 32);
    *abort_any = 0;
    ptx::fence_mbar_init();
  };
  // everything up to the wait touches no global memory, so it runs under the previous kernel's tail
  if (tid == kBwdMath) {
    ptx::prefetch_tensormap(&tm_qkv);
    ptx::prefetch_tensormap(&tm_do);
    ptx::prefetch_tensormap(&tm_qkv_y);
    ptx::prefetch_tensormap(&tm_do_y);
    init_barriers();
  }
  pdl_entry();
  const bool staged = n_seg < kSegStage;
  if (staged)
    for (int i = tid; i <= n_seg; i += kBwdThreads) seg_s[i] = __ldg(seg + i);
  const int Np = packed_rows(seg, n_seg, capacity);
  const int n_items = ((Np + 127) / 128) * H;
  if ((int)blockIdx.x >= n_items) return;
  if (skip_short) __syncthreads();  // the staged offsets are visible to the tile test
  bool cta_failed = false, first_item = true;
  int item = blockIdx.x;
  do {  // kLoop: this CTA strides over the items; otherwise the grid holds one CTA per item and this is no loop
  const int h = item % H, r0 = (item / H) * 128;
  // tiles whose rows all belong to the one-pass kernel are passed over before anything is fetched
  if (skip_short && !tile_has_long_rows(seg_s, seg, staged, n_seg, Np, r0)) continue;
  const int x1_col = C + h * D;                       // own operand inside qkv: K
  if (tid == kBwdMath) {
    if (!first_item) {  // every phase of the previous item has completed: the barriers start over
      ptx::mbar_inval(bar_x);
      for (int s3 = 0; s3 < kStages; ++s3) ptx::mbar_inval(bar_y(s3));
      ptx::mbar_inval(bar_s);
      ptx::mbar_inval(bar_dp);
      ptx::mbar_inval(bar_acc);
      ptx::mbar_inval(bar_sfree);
      ptx::mbar_inval(bar_pready);
      ptx::mbar_inval(bar_dsready);
      init_barriers();
    }
    // the own tiles depend only on r0: fetch them under the segment search
    ptx::mbar_expect_tx(bar_x, 2 * kTile);
    ptx::tma_load_2d(x1_s, &tm_qkv, bar_x, x1_col, r0);
    ptx::tma_load_2d(x2_s, &tm_qkv, bar_x, 2 * C + h * D, r0);           // V
  }
  if (first_item && warp == 0) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), kBwdTmemCols);
  first_item = false;
  ptx::tc_fence_before_sync();
  __syncthreads();  // barriers, (first item) the TMEM address and the staged offsets are visible
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;

  const int row = r0 + rl;
  RowSeg mine{0, 0};
  if (is_math) {
    mine = staged ? row_segment_staged(seg_s, n_seg, Np, row) : row_segment(seg, n_seg, Np, row);
    // segments that fit one tile belong to the one-pass kernel: their rows are no rows of this one
    if (skip_short && mine.hi - mine.lo <= kShortMax) mine = RowSeg{0, 0};
    if (half == 0) {
      row_ok[rl] = mine.hi > mine.lo ? 1 : 0;
      if (mine.hi > mine.lo) {  // the rows of the other side to visit: the union of the segments of this tile's rows
        atomicMin(const_cast<int*>(range), mine.lo);
        atomicMax(const_cast<int*>(range) + 1, mine.hi);
      }
    }
  }
  __syncthreads();
  const bool any_row = range[1] > range[0];  // false: every row of the tile belongs to the one-pass kernel
  const int o_lo = any_row ? range[0] : 0, o_hi = any_row ? range[1] : 0;
  const int n_tiles = (o_hi - o_lo + kBwdY - 1) / kBwdY;

  const int y1_col = h * D;                           // streamed operand inside qkv: Q
  auto load_other = [&](int t_) {  // streamed tile t_ into its stage
    const int st = stage_of(t_), y0 = o_lo + t_ * kBwdY;
    ptx::mbar_expect_tx(bar_y(st), 2 * kYTile);
    ptx::tma_load_2d(smem_base + y1_off(st), &tm_qkv_y, bar_y(st), y1_col, y0);
    ptx::tma_load_2d(smem_base + y2_off(st), &tm_do_y, bar_y(st), h * D, y0);                     // dO
  };
  int issued = 0;  // streamed tiles whose loads have been issued (kept by the issuing thread)
  if (tid == kBwdMath) {
    for (int t_ = 0; t_ < n_tiles && t_ < kStages; ++t_) load_other(t_);  // every stage is free at the start
    issued = n_tiles < kStages ? n_tiles : kStages;
  }

  // Bounded wait that also gives up as soon as any thread of the CTA has reported a failure.
  auto wait = [&](uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < ptx::kWaitLimit; ++i) {
      if (ptx::mbar_try_wait(bar, parity)) return true;
      if ((i & 255u) == 255u && *abort_any) return false;
    }
    return false;
  };
  // every lane polls; the warp takes one answer, so that a whole warp gives up or none of it
  auto wait_w = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, wait(bar, parity)) != 0; };

  // per-row statistics of the query side
  float nxt_lse = 0.f, nxt_D = 0.f;  // prefetched values of the next streamed query tile, row rl < 64
  if (is_math && half == 0 && rl < kBwdY) {
    const int i = o_lo + rl;
    if (i < o_hi) { nxt_lse = lse[(long long)h * capacity + i] * kLog2e; nxt_D = delta[(long long)h * capacity + i]; }
  }

  constexpr uint32_t kIdescS = ptx::idesc_bf16_f32(128, kBwdY, false, false);
  const unsigned span = (unsigned)(mine.hi - mine.lo);

  // Make streamed tile t_ ready for the products (arithmetic warps): its load has landed, lines past the last
  // valid packed row are zeroed (they are unspecified memory and would be summed over), its query statistics
  // are staged.  Returns false when the wait for the load gave up.
  auto prep = [&](int t_) {
    const int st = stage_of(t_);
    bool ok = true;
    const int y0 = o_lo + t_ * kBwdY;
    // the issuing thread waits for the load itself; the arithmetic warps need it only where they touch the tile
    if (t_ == 0) {
      ok = wait_w(bar_y(st), use_of(t_));
      ok = wait_w(bar_x, 0) && ok;
    } else if (y0 + kBwdY > Np) {
      ok = wait_w(bar_y(st), use_of(t_));
    }
    if (y0 + kBwdY > Np) {
      const int first = Np - y0;
      constexpr int kChunks = HT::kRowBytes / 16;
      for (int c = tid; c < (kBwdY - first) * kChunks; c += kBwdMath) {
        const int off = (first + c / kChunks) * HT::kRowBytes + (c % kChunks) * 16;
        *reinterpret_cast<uint4*>(smem_al + y1_off(st) + off) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(smem_al + y2_off(st) + off) = make_uint4(0, 0, 0, 0);
      }
      ptx::fence_proxy_async_smem();
    }
    if (half == 0 && rl < kBwdY) {
      stat_lse[(t_ % 3) * kBwdY + rl] = nxt_lse;
      stat_D[(t_ % 3) * kBwdY + rl] = nxt_D;
      const int i = y0 + kBwdY + rl;
      nxt_lse = 0.f; nxt_D = 0.f;
      if (i < o_hi) { nxt_lse = lse[(long long)h * capacity + i] * kLog2e; nxt_D = delta[(long long)h * capacity + i]; }
    }
    return ok;
  };

  if (is_math && n_tiles > 0 && !prep(0)) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_any = 1; }
  ptx::tc_fence_before_sync();
  __syncthreads();  // tile 0 is ready; a failure so far is seen by all threads or by none
  const bool failed_early = *abort_any != 0 || n_tiles == 0;

  if (!is_math) {
    // ---------------------------------------------------------------- copies and products: one warp, whose lanes
    // all follow the tiles and take every wait together; one elected lane issues (the same one each time, so its
    // commits cover all its products)
    if (!failed_early) {
      constexpr uint32_t kIdescV = ptx::idesc_bf16_f32(128, D, false, true);  // A K-major (P^T in shared memory or dS^T in TMEM)
      auto issue_st = [&](int t_) {  // S^T of streamed tile t_
        const uint32_t y1a = smem_base + y1_off(stage_of(t_));
        if (ptx::elect_one()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k)
            ptx::mma_bf16(tmem + kColS1, HT::kmajor(x1_s, k), HT::kmajor(y1a, k), kIdescS, k != 0 ? 1u : 0u);
          ptx::mma_commit(bar_s);
        }
        __syncwarp();
      };
      auto issue_dpt = [&](int t_) {  // dP^T of streamed tile t_
        const uint32_t y2a = smem_base + y2_off(stage_of(t_));
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          ptx::mma_bf16(tmem + kColS2, HT::kmajor(x2_s, k), HT::kmajor(y2a, k), kIdescS, k != 0 ? 1u : 0u);
        ptx::mma_commit(bar_dp);
      };
      bool ok = true;
      ptx::tc_fence_after_sync();
      issue_st(0);
      if (ptx::elect_one()) issue_dpt(0);
      __syncwarp();
      for (int t = 0; ok && t < n_tiles; ++t) {
        const int st = stage_of(t);
        if (t + 1 < n_tiles) {
          // S^T of tile t is in registers and tile t + 1 has landed: its S^T runs under the arithmetic of tile t
          if (!(ok = wait_w(bar_sfree, t & 1))) break;
          if (!(ok = wait_w(bar_y(stage_of(t + 1)), use_of(t + 1)))) break;
          ptx::tc_fence_after_sync();
          issue_st(t + 1);
        }
        // the stage of tile t - 1 is free once its accumulating products have completed
        if (t > 0 && t - 1 + kStages < n_tiles) {
          if (!(ok = wait_w(bar_acc, (t - 1) & 1))) break;
          if (ptx::elect_one()) load_other(t - 1 + kStages);
          __syncwarp();
          issued = t + kStages;
        }
        const uint32_t acc = (t != 0) ? 1u : 0u;
        const uint32_t y1a = smem_base + y1_off(st), y2a = smem_base + y2_off(st);
        if (!(ok = wait_w(bar_pready, t & 1))) break;     // P^T of tile t is in shared memory
        ptx::tc_fence_after_sync();
        if (ptx::elect_one()) {
#pragma unroll
          for (int k = 0; k < kBwdY / 16; ++k)   // dV += P^T dO
            ptx::mma_bf16(tmem + kColAcc1, HT::kmajor(p_s, k), HT::mnmajor(y2a, k), kIdescV, acc | (k != 0));
        }
        __syncwarp();
        if (!(ok = wait_w(bar_dsready, t & 1))) break;    // dS^T of tile t is in TMEM, over the dP^T columns
        ptx::tc_fence_after_sync();
        if (ptx::elect_one()) {
#pragma unroll
          for (int k = 0; k < kBwdY / 16; ++k)   // dK += dS^T Q: queries 16k.. of the tile, stored by the warps of half k / 2
            ptx::mma_bf16_ts(tmem + kColAcc2, tmem + kColS2 + (k >> 1) * 32 + (k & 1) * 8, HT::mnmajor(y1a, k), kIdescV,
                             acc | (k != 0));
          ptx::mma_commit(bar_acc);
          // queued behind dK, which reads the columns that it overwrites (products of one thread execute in issue order)
          if (t + 1 < n_tiles) issue_dpt(t + 1);
        }
        __syncwarp();
      }
      if (!ok && lane == 0) {
        record_status(d_status, SPA_ERR_TIMEOUT);
        *abort_any = 1;
      }
    }
  } else if (!failed_early) {
    // ---------------------------------------------------------------- arithmetic: two threads per key row
    constexpr int kPc = kBwdY / 2;  // fp32 columns of each tile owned by this thread
    const int col0 = half * kPc;
    // no barrier joins the arithmetic warps inside the loop, so a warp whose wait gave up may leave it alone: the
    // others see the flag in their own waits
    auto fail = [&]() {
      record_status(d_status, SPA_ERR_TIMEOUT);
      *abort_any = 1;
    };
    // this thread's 64 bytes of its row of P^T: chunks 4 * half .. of a 128-byte line, under the 128-byte swizzle
    uint8_t* p_row = smem_al + kPBase + rl * 128;
    const int p_rot = rl & 7;
    for (int t = 0; t < n_tiles; ++t) {
      const int y0 = o_lo + t * kBwdY;
      // ---- S^T: this thread's columns into registers
      bool ok = wait_w(bar_s, t & 1);
      ptx::tc_fence_after_sync();
      uint32_t rs[kPc];
      ptx::tmem_ld_32x32(tmem + lane_base + kColS1 + col0, rs);
      ptx::tmem_ld_wait();
      if (ok && t + 1 < n_tiles) ok = prep(t + 1);
      // the statistics of tile t were staged by other warps before they announced tile t - 1 (that phase has
      // completed; it is waited for, before this warp's own arrival for tile t, to order the reads below)
      if (ok && t > 0) ok = wait_w(bar_sfree, (t - 1) & 1);
      if (!ok) { fail(); break; }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_sfree);

      // ---- P^T = 2^(S^T - lse): needs S^T only, and holds the exponentials.  A thread whose 32 columns lie wholly
      // outside its row's segment writes zeros without doing the arithmetic; the mask costs something only where a
      // boundary crosses.
      const int yc0 = y0 + col0;
      const bool some = yc0 < mine.hi && yc0 + kPc > mine.lo;
      const bool partial = some && !(yc0 >= mine.lo && yc0 + kPc <= mine.hi);
      uint32_t pk[kPc / 2];
      if (some) {
        if (partial) {
#pragma unroll
          for (int j = 0; j < kPc; ++j)
            if ((unsigned)(yc0 + j - mine.lo) >= span) rs[j] = 0xff800000u;  // p = 2^-inf = 0
        }
        const float* sl = stat_lse + (t % 3) * kBwdY + col0;
#pragma unroll
        for (int j = 0; j < kPc; j += 2) {
          const float p0 = ptx::ex2_approx(fmaf(__uint_as_float(rs[j]), scale_log2e, -sl[j]));
          const float p1 = ptx::ex2_approx(fmaf(__uint_as_float(rs[j + 1]), scale_log2e, -sl[j + 1]));
          rs[j] = __float_as_uint(p0);
          rs[j + 1] = __float_as_uint(p1);
          __nv_bfloat162 bp = __floats2bfloat162_rn(p0, p1);
          pk[j >> 1] = *reinterpret_cast<uint32_t*>(&bp);
        }
      } else {
#pragma unroll
        for (int j = 0; j < kPc / 2; ++j) pk[j] = 0u;
      }
      // dV of tile t - 1 must have read P^T (its completion is announced together with dK's)
      if (t > 0) {
        if (!wait_w(bar_acc, (t - 1) & 1)) { fail(); break; }
      }
#pragma unroll
      for (int c = 0; c < 4; ++c)
        *reinterpret_cast<uint4*>(p_row + (((half * 4 + c) ^ p_rot) << 4)) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_pready);

      // ---- dS^T = P^T (dP^T - D), stored over this thread's own dP^T columns (the first 16 of its 32)
      if (!wait_w(bar_dp, t & 1)) { fail(); break; }
      ptx::tc_fence_after_sync();
      uint32_t rp[kPc];
      ptx::tmem_ld_32x32(tmem + lane_base + kColS2 + col0, rp);  // by the whole warp: the load is a collective
      ptx::tmem_ld_wait();
      if (some) {
        const float* sd = stat_D + (t % 3) * kBwdY + col0;
#pragma unroll
        for (int j = 0; j < kPc; j += 2) {
          // a masked column has p = 0 exactly and a finite dP^T (rows past the last valid one are zeroed): dS^T = 0
          const float d0 = __uint_as_float(rs[j]) * (__uint_as_float(rp[j]) - sd[j]);
          const float d1 = __uint_as_float(rs[j + 1]) * (__uint_as_float(rp[j + 1]) - sd[j + 1]);
          __nv_bfloat162 bds = __floats2bfloat162_rn(d0, d1);
          pk[j >> 1] = *reinterpret_cast<uint32_t*>(&bds);
        }
      }
      ptx::tmem_st_32x16(tmem + lane_base + kColS2 + col0, pk);
      ptx::tmem_st_wait();
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_dsready);
    }
    // the last accumulating products complete the outputs
    const bool gave_up = __shfl_sync(0xffffffffu, *abort_any, 0) != 0;  // one answer per warp
    if (n_tiles > 0 && !gave_up && !wait_w(bar_acc, (n_tiles - 1) & 1)) fail();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // nobody reports a failure from here on: the branches below are taken by all threads or by none
  ptx::tc_fence_after_sync();
  const bool failed = *abort_any != 0;

  if (!failed && n_tiles > 0) {
    // Each thread drains d/2 columns of its row of the accumulators into the own tiles' shared memory (idle
    // now: every product has completed), from where whole rows go out as full lines.
    constexpr int kDh = D / 2;
    auto stage_acc = [&](uint32_t acc_col, uint8_t* tile, float mul) {
      uint32_t r[kDh];
      if (kDh == 32) ptx::tmem_ld_32x32(tmem + lane_base + acc_col + half * kDh, r);
      else ptx::tmem_ld_32x16(tmem + lane_base + acc_col + half * kDh, r);
      ptx::tmem_ld_wait();
      const int rot = chunk_rot<D>(rl);
#pragma unroll
      for (int g = 0; g < kDh / 8; ++g) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[g * 8 + e]) * mul;
        *reinterpret_cast<uint4*>(tile + rl * HT::kRowBytes + (((half * (kDh / 8) + g) ^ rot) << 4)) =
            Vec16<__nv_bfloat16>::from_float(v);
      }
    };
    const long long ld = 3LL * C;
    if (is_math) {
      stage_acc(kColAcc1, smem_al, 1.f);             // dV
      stage_acc(kColAcc2, smem_al + kTile, scale);   // dK
    }
    __syncthreads();
    copy_tile_out<D, kBwdThreads>(smem_al, dqkv + 2 * C + h * D, ld, r0, Np, tid, row_ok);
    copy_tile_out<D, kBwdThreads>(smem_al + kTile, dqkv + C + h * D, ld, r0, Np, tid, row_ok);
  }
  if ((failed || n_tiles == 0) && tid == kBwdMath) {  // let outstanding loads land before shared memory is released
    for (int t = issued > kStages ? issued - kStages : 0; t < issued; ++t) ptx::mbar_wait(bar_y(stage_of(t)), use_of(t));
    ptx::mbar_wait(bar_x, 0);
  }
  cta_failed = failed;
  ptx::tc_fence_before_sync();
  __syncthreads();  // the tiles' memory and the barriers are free for the next item
  } while (kLoop && (item += gridDim.x) < n_items && !cta_failed);
  if (!first_item && warp == 0) {  // TMEM was taken with the first item that this CTA worked on
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(*tmem_slot, kBwdTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Backward for segments of at most 128 rows, in one pass: a CTA owns one segment and one head, holds its queries
// and its keys at once, and evaluates S, P, dP and dS exactly once.
//   loads    Q, K, V, dO, O rows of the segment (one TMA tile each, 128 rows from the segment's first row)
//   MMA      S = Q K^T and dP = dO V^T, 128 x 128 fp32 each, TMEM columns [0,128) and [128,256)
//   threads  two per query row: D_i = dO_i . O_i, P = 2^(S - lse), dS = P (dP - D); P and dS go to shared memory
//            as bf16 in one layout that the tensor core can read both ways (rows = queries of 128 bytes per 64 keys,
//            16-byte chunks XOR-swizzled by the row): K-major for dQ = dS K, MN-major for dV = P^T dO, dK = dS^T Q
//   MMA      dV, dK, dQ into TMEM columns [0, 3d), over the fp32 tiles that the threads have taken into registers
//   stores   the three tiles leave through shared memory as whole lines, rows of the segment only.
// Nothing is recomputed and q, k, v, dO are read once.  Rows of the tiles beyond the segment belong to other
// segments (finite data, multiplied by zeros) or lie past the last valid packed row (unspecified memory: zeroed in
// shared memory before any product sums over them).  256 TMEM columns and under 113 KB: two CTAs per SM.
constexpr int kShortThreads = 256;
template <int D> __host__ __device__ constexpr int short_smem_bytes() {
  // Q, K, dO tiles; P buffer (V tile first lives there); dS buffer (O tile first lives there); barriers.  No slack
  // for aligning the base: with it two CTAs would not fit an SM at d = 64; the kernel checks the alignment instead.
  return 3 * 128 * D * 2 + 2 * 128 * 128 * 2 + 64;
}

template <int D>
__global__ void __launch_bounds__(kShortThreads, 2)
attn_bwd_short_kernel(const __grid_constant__ CUtensorMap tm_qkv, const __grid_constant__ CUtensorMap tm_do,
                      const __grid_constant__ CUtensorMap tm_o, const float* __restrict__ lse,
                      const int32_t* __restrict__ seg, int n_seg, int capacity, int C, float scale,
                      __nv_bfloat16* __restrict__ dqkv, int32_t* d_status) {
  using HT = HeadTile<D>;
  constexpr int kTile = HT::kTileBytes;
  constexpr int kOp = 128 * 128 * 2;  // a P or dS buffer: two panels of 64 keys, 128 query rows of 128 bytes each
  constexpr float kLog2e = 1.4426950408889634f;
  const int h = blockIdx.x, s_idx = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int quarter = warp & 3, half = warp >> 2, rl = quarter * 32 + lane;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = ptx::smem_u32(smem_raw);
  uint8_t* smem_al = smem_raw;
  if ((smem_base & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base: refuse rather than misread
    if (threadIdx.x == 0) record_status(d_status, SPA_ERR_UNSUPPORTED);
    return;
  }
  const uint32_t q_s = smem_base, k_s = smem_base + kTile, do_s = smem_base + 2 * kTile;
  const uint32_t p_s = smem_base + 3 * kTile, ds_s = p_s + kOp;
  const uint32_t v_s = p_s, o_s = ds_s;  // needed only until the first products / D_i are done
  constexpr int kBarOff = 3 * kTile + 2 * kOp;
  const uint32_t bar_ld = smem_base + kBarOff, bar_s = bar_ld + 8, bar_acc = bar_ld + 16;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_al + kBarOff + 24);
  volatile int* abort_any = reinterpret_cast<volatile int*>(smem_al + kBarOff + 28);

  if (tid == 0) {
    ptx::prefetch_tensormap(&tm_qkv);
    ptx::prefetch_tensormap(&tm_do);
    ptx::prefetch_tensormap(&tm_o);
    ptx::mbar_init(bar_ld, 1);
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_acc, 1);
    *abort_any = 0;
    ptx::fence_mbar_init();
  }
  pdl_entry();
  const int Np = packed_rows(seg, n_seg, capacity);
  const int lo = __ldg(seg + s_idx);
  int hi = __ldg(seg + s_idx + 1);
  hi = hi < Np ? hi : Np;
  const int n = hi - lo;  // rows of this segment
  if (n <= 0 || n > kShortMax) return;  // empty, or one for the two-pass kernels
  if (tid == 0) {
    ptx::mbar_expect_tx(bar_ld, 5 * kTile);
    ptx::tma_load_2d(q_s, &tm_qkv, bar_ld, h * D, lo);
    ptx::tma_load_2d(k_s, &tm_qkv, bar_ld, C + h * D, lo);
    ptx::tma_load_2d(v_s, &tm_qkv, bar_ld, 2 * C + h * D, lo);
    ptx::tma_load_2d(do_s, &tm_do, bar_ld, h * D, lo);
    ptx::tma_load_2d(o_s, &tm_o, bar_ld, h * D, lo);
  }
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), 256);
  const bool valid = rl < n;
  const float my_lse = valid ? lse[(long long)h * capacity + lo + rl] * kLog2e : 0.f;
  ptx::tc_fence_before_sync();
  __syncthreads();  // barriers and the TMEM address are visible
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
  const float scale_log2e = scale * kLog2e;

  bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_ld, 0)) != 0;
  // D_i = dO_i . O_i (both tiles carry the same swizzle: equal positions hold equal columns)
  float my_D = 0.f;
  if (valid) {
    constexpr int kChunks = HT::kRowBytes / 16;
    const uint8_t* po = smem_al + (o_s - smem_base) + rl * HT::kRowBytes;
    const uint8_t* pg = smem_al + 2 * kTile + rl * HT::kRowBytes;
    const int rot = chunk_rot<D>(rl);
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      float a[8], b[8];
      Vec16<__nv_bfloat16>::to_float(*reinterpret_cast<const uint4*>(po + ((c ^ rot) << 4)), a);
      Vec16<__nv_bfloat16>::to_float(*reinterpret_cast<const uint4*>(pg + ((c ^ rot) << 4)), b);
#pragma unroll
      for (int e = 0; e < 8; ++e) my_D = fmaf(a[e], b[e], my_D);
    }
  }
  // lines past the last valid packed row are unspecified memory: the second products sum over the rows of Q, K and dO
  if (lo + 128 > Np) {
    const int first = Np - lo;  // >= n >= 1
    constexpr int kChunks = HT::kRowBytes / 16;
    for (int c = tid; c < (128 - first) * kChunks; c += kShortThreads) {
      const int off = (first + c / kChunks) * HT::kRowBytes + (c % kChunks) * 16;
      *reinterpret_cast<uint4*>(smem_al + off) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(smem_al + kTile + off) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(smem_al + 2 * kTile + off) = make_uint4(0, 0, 0, 0);
    }
    ptx::fence_proxy_async_smem();
  }
  if (!ok) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_any = 1; }
  ptx::tc_fence_before_sync();
  __syncthreads();  // tiles are ready (and everybody has read the O tile, whose memory becomes the dS buffer)
  if (tid == 0 && !*abort_any) {
    ptx::tc_fence_after_sync();
    constexpr uint32_t kIdescS = ptx::idesc_bf16_f32(128, 128, false, false);
#pragma unroll
    for (int k = 0; k < D / 16; ++k)
      ptx::mma_bf16(tmem, HT::kmajor(q_s, k), HT::kmajor(k_s, k), kIdescS, k != 0 ? 1u : 0u);          // S = Q K^T
#pragma unroll
    for (int k = 0; k < D / 16; ++k)
      ptx::mma_bf16(tmem + 128, HT::kmajor(do_s, k), HT::kmajor(v_s, k), kIdescS, k != 0 ? 1u : 0u);   // dP = dO V^T
    ptx::mma_commit(bar_s);
  }
  if (!*abort_any) {
    ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_s, 0)) != 0;
    if (!ok) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_any = 1; }
  }
  ptx::tc_fence_after_sync();
  // ---- P and dS of this thread's 64 key columns, 32 at a time, into the operand buffers (the V tile has been read:
  // the products above have completed)
  if (ok) {
    uint8_t* prow = smem_al + (p_s - smem_base) + half * (kOp / 2) + rl * 128;
    uint8_t* dsrow = prow + kOp;
    const int rsw = rl & 7;
#pragma unroll
    for (int part = 0; part < 2; ++part) {
      const int col0 = half * 64 + part * 32;  // first key column of this group
      uint32_t rs[32], rp[32];
      ptx::tmem_ld_32x32(tmem + lane_base + col0, rs);
      ptx::tmem_ld_32x32(tmem + lane_base + 128 + col0, rp);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int c = 0; c < 4; ++c) {  // 16-byte chunk: 8 keys
        uint32_t wp[4], wd[4];
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
          float pv[2], dsv[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int col = col0 + c * 8 + j + u;
            const bool in = valid && col < n;
            const float pe = ptx::ex2_approx(fmaf(__uint_as_float(rs[c * 8 + j + u]), scale_log2e, -my_lse));
            pv[u] = in ? pe : 0.f;
            dsv[u] = in ? pe * (__uint_as_float(rp[c * 8 + j + u]) - my_D) : 0.f;
          }
          __nv_bfloat162 bp = __floats2bfloat162_rn(pv[0], pv[1]);
          __nv_bfloat162 bd = __floats2bfloat162_rn(dsv[0], dsv[1]);
          wp[j >> 1] = *reinterpret_cast<uint32_t*>(&bp);
          wd[j >> 1] = *reinterpret_cast<uint32_t*>(&bd);
        }
        const int chunk = (part * 4 + c) ^ rsw;
        *reinterpret_cast<uint4*>(prow + (chunk << 4)) = make_uint4(wp[0], wp[1], wp[2], wp[3]);
        *reinterpret_cast<uint4*>(dsrow + (chunk << 4)) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
      }
    }
    ptx::fence_proxy_async_smem();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // operands complete; every thread holds its fp32 values: their TMEM columns take the results
  if (tid == 0 && !*abort_any) {
    ptx::tc_fence_after_sync();
    constexpr uint32_t kIdescT = ptx::idesc_bf16_f32(128, D, true, true);    // A = P^T or dS^T (MN-major), B MN-major
    constexpr uint32_t kIdescQ = ptx::idesc_bf16_f32(128, D, false, true);   // A = dS (K-major), B = K (MN-major)
#pragma unroll
    for (int k = 0; k < 8; ++k)   // dV = P^T dO: 16 query rows per step
      ptx::mma_bf16(tmem, ptx::smem_desc_sw128(p_s + k * 2048, kOp / 2, 1024), HT::mnmajor(do_s, k), kIdescT, k != 0 ? 1u : 0u);
#pragma unroll
    for (int k = 0; k < 8; ++k)   // dK = dS^T Q
      ptx::mma_bf16(tmem + D, ptx::smem_desc_sw128(ds_s + k * 2048, kOp / 2, 1024), HT::mnmajor(q_s, k), kIdescT, k != 0 ? 1u : 0u);
#pragma unroll
    for (int k = 0; k < 8; ++k)   // dQ = dS K: 16 keys per step, 64 keys per panel
      ptx::mma_bf16(tmem + 2 * D, ptx::smem_desc_sw128(ds_s + (k >> 2) * (kOp / 2) + (k & 3) * 32, 16, 1024),
                    HT::mnmajor(k_s, k), kIdescQ, k != 0 ? 1u : 0u);
    ptx::mma_commit(bar_acc);
  }
  if (!*abort_any) {
    ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_acc, 0)) != 0;
    if (!ok) { record_status(d_status, SPA_ERR_TIMEOUT); *abort_any = 1; }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();  // nobody reports a failure from here on
  ptx::tc_fence_after_sync();
  if (!*abort_any) {
    // dV, dK, dQ rows as bf16 into the Q, K, dO tiles' memory (idle now), from where whole lines go out
    constexpr int kDh = D / 2;
    const float mul[3] = {1.f, scale, scale};
#pragma unroll
    for (int a = 0; a < 3; ++a) {
      uint32_t r[kDh];
      if (kDh == 32) ptx::tmem_ld_32x32(tmem + lane_base + a * D + half * kDh, r);
      else ptx::tmem_ld_32x16(tmem + lane_base + a * D + half * kDh, r);
      ptx::tmem_ld_wait();
      const int rot = chunk_rot<D>(rl);
#pragma unroll
      for (int g = 0; g < kDh / 8; ++g) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[g * 8 + e]) * mul[a];
        *reinterpret_cast<uint4*>(smem_al + a * kTile + rl * HT::kRowBytes + (((half * (kDh / 8) + g) ^ rot) << 4)) =
            Vec16<__nv_bfloat16>::from_float(v);
      }
    }
    __syncthreads();
    const long long ld = 3LL * C;
    copy_tile_out<D, kShortThreads>(smem_al, dqkv + 2 * C + h * D, ld, lo, hi, tid);               // dV
    copy_tile_out<D, kShortThreads>(smem_al + kTile, dqkv + C + h * D, ld, lo, hi, tid);           // dK
    copy_tile_out<D, kShortThreads>(smem_al + 2 * kTile, dqkv + h * D, ld, lo, hi, tid);           // dQ
  } else if (tid == 0) {
    ptx::mbar_wait(bar_ld, 0);  // let the loads land before shared memory is released
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem, 256);
  }
}

// Which kernel runs the dK / dV pass for head dimension D.
template <int D> struct kv_pass {
  static constexpr int kThreads = kBwdThreads;
  static constexpr int kSmem = bwd_smem_bytes<D, false>();
  template <bool kLoop> static auto kernel() { return attn_bwd_tc_kernel<D, false, kLoop>; }
};
template <> struct kv_pass<64> {
  static constexpr int kThreads = kBwdThreads;
  static constexpr int kSmem = split_smem_bytes<64>();
  template <bool kLoop> static auto kernel() { return attn_bwd_kv_split_kernel<64, kLoop>; }
};

template <int D>
int bwd_launch(const spa_params& p, const void* qkv, const void* ao, const float* lse, const void* dao,
               const int32_t* seg, int n_seg, void* dqkv, void* workspace, int32_t* d_status, cudaStream_t st) {
  CUtensorMap tm_qkv, tm_do, tm_qkv_y, tm_do_y, tm_o;  // own tiles: 128-row boxes; streamed tiles: 64-row boxes
  if (!make_tmap_bf16_2d(&tm_qkv, qkv, 3ull * p.C, p.capacity, 6ull * p.C, D, 128, D * 2) ||
      !make_tmap_bf16_2d(&tm_do, dao, (uint64_t)p.C, p.capacity, 2ull * p.C, D, 128, D * 2) ||
      !make_tmap_bf16_2d(&tm_qkv_y, qkv, 3ull * p.C, p.capacity, 6ull * p.C, D, kBwdY, D * 2) ||
      !make_tmap_bf16_2d(&tm_do_y, dao, (uint64_t)p.C, p.capacity, 2ull * p.C, D, kBwdY, D * 2) ||
      !make_tmap_bf16_2d(&tm_o, ao, (uint64_t)p.C, p.capacity, 2ull * p.C, D, 128, D * 2))
    return SPA_ERR_UNSUPPORTED;
  static DeviceOnce attr;
  cudaError_t ea = attr.run([&] {
    const auto smem_attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = cudaFuncSetAttribute(attn_bwd_tc_kernel<D, true, false>, smem_attr, bwd_smem_bytes<D, true>());
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_tc_kernel<D, true, true>, smem_attr, bwd_smem_bytes<D, true>());
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_short_kernel<D>, smem_attr, short_smem_bytes<D>());
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kv_pass<D>::template kernel<false>(), smem_attr, kv_pass<D>::kSmem);
    return e != cudaSuccess ? e : cudaFuncSetAttribute(kv_pass<D>::template kernel<true>(), smem_attr, kv_pass<D>::kSmem);
  });
  if (ea != cudaSuccess) { set_cuda_error(ea, "attn_bwd_tc_kernel"); return SPA_ERR_CUDA; }
  float* delta = reinterpret_cast<float*>(workspace);  // [H][capacity]
  // One CTA per (tile, head) item, or a persistent grid of two CTAs per SM that strides over the items.  The stride
  // is a static assignment: it pays (one prologue per CTA instead of one per item) where the items cost about the
  // same, i.e. short segments that span a key tile or two, and where a CTA gets several of them; with long segments
  // the key ranges differ widely from item to item and the hardware's own block scheduling balances them better.
  // The host knows the item slots of the capacity, not the rows that the selection kept (typically about half):
  // three grids' worth of slots stands for one and a half items per CTA or more.
  const long long items = (long long)p.H * ((p.capacity + 127) / 128);
  const bool even_items = (long long)p.capacity <= 256ll * (n_seg > 0 ? n_seg : 1);
  const bool loop = even_items && items >= 3ll * 2 * kNumSMs;
  const int grid = (int)(loop ? 2 * kNumSMs : items);
  auto kq = loop ? attn_bwd_tc_kernel<D, true, true> : attn_bwd_tc_kernel<D, true, false>;
  auto kkv = loop ? kv_pass<D>::template kernel<true>() : kv_pass<D>::template kernel<false>();
  const float scale = softmax_scale_of(p);
  // Under SPA_FLAG_ONE_PASS_BWD segments of at most 128 rows go to the one-pass kernel (one CTA per segment and
  // head) and the two passes take the longer ones; otherwise, or with more segments than a grid dimension holds, the
  // two passes take everything.
  const int skip_short = ((p.flags & SPA_FLAG_ONE_PASS_BWD) && n_seg >= 1 && n_seg <= 65535) ? 1 : 0;
  if (skip_short) {
    launch_pdl(attn_bwd_short_kernel<D>, dim3(p.H, n_seg), kShortThreads, short_smem_bytes<D>(), st, tm_qkv, tm_do, tm_o, lse,
               seg, n_seg, p.capacity, p.C, scale, (__nv_bfloat16*)dqkv, d_status);
    SPA_CUDA_CHECK_LAUNCH("attn_bwd_short_kernel");
  }
  launch_pdl(kq, grid, kBwdThreads, bwd_smem_bytes<D, true>(), st, tm_qkv, tm_do, tm_qkv_y, tm_do_y, tm_o, lse, delta, seg,
             n_seg, p.capacity, p.C, p.H, scale, (__nv_bfloat16*)dqkv, skip_short, d_status);
  SPA_CUDA_CHECK_LAUNCH("attn_bwd_tc_kernel(dQ)");
  launch_pdl(kkv, grid, kv_pass<D>::kThreads, kv_pass<D>::kSmem, st, tm_qkv, tm_do, tm_qkv_y, tm_do_y, tm_o, lse, delta, seg,
             n_seg, p.capacity, p.C, p.H, scale, (__nv_bfloat16*)dqkv, skip_short, d_status);
  SPA_CUDA_CHECK_LAUNCH("attn_bwd_tc_kernel(dKV)");
  return SPA_OK;
}

template <int D>
int fwd_launch(const spa_params& p, const void* qkv, const int32_t* seg, int n_seg, void* ao, float* lse,
               int32_t* d_status, cudaStream_t st) {
  CUtensorMap tm;
  if (!make_tmap_bf16_2d(&tm, qkv, 3ull * p.C, p.capacity, 6ull * p.C, D, 128, D * 2)) return SPA_ERR_UNSUPPORTED;
  auto kern = attn_fwd_tc_kernel<D>;
  static DeviceOnce attr;
  cudaError_t ea = attr.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, fwd_smem_bytes<D>()); });
  if (ea != cudaSuccess) { set_cuda_error(ea, "attn_fwd_tc_kernel"); return SPA_ERR_CUDA; }
  // a persistent grid: two CTAs per SM (87 KB of shared memory, 256 TMEM columns each), never more than work items
  const long long items = (long long)p.H * ((p.capacity + kQ - 1) / kQ);
  const int grid = (int)(items < 2 * kNumSMs ? items : 2 * kNumSMs);
  launch_pdl(kern, grid, kFwdThreads, fwd_smem_bytes<D>(), st, tm, seg, n_seg, p.capacity, p.C, p.H,
                                                      softmax_scale_of(p) * 1.4426950408889634f,
                                                      (__nv_bfloat16*)ao, lse, d_status);
  SPA_CUDA_CHECK_LAUNCH("attn_fwd_tc_kernel");
  return SPA_OK;
}

}  // namespace

bool tc_attention_fwd_supported(const spa_params& p) {
  const int d = p.C / p.H;
  return p.dtype == SPA_BF16 && (d == 32 || d == 64) && tensor_maps_available();
}

bool tc_attention_bwd_supported(const spa_params& p) { return tc_attention_fwd_supported(p); }

size_t tc_attention_workspace_bytes(const spa_params& p) {
  if (!tc_attention_fwd_supported(p)) return 0;
  return ((size_t)p.H * p.capacity * sizeof(float) + 255) & ~(size_t)255;
}

int launch_attention_bwd_tc(const spa_params& p, const void* qkv, const void* ao, const float* lse, const void* dao,
                            const int32_t* seg, int n_seg, void* dqkv, void* workspace, int32_t* d_status,
                            cudaStream_t st) {
  return p.C / p.H == 64 ? bwd_launch<64>(p, qkv, ao, lse, dao, seg, n_seg, dqkv, workspace, d_status, st)
                         : bwd_launch<32>(p, qkv, ao, lse, dao, seg, n_seg, dqkv, workspace, d_status, st);
}

int launch_attention_fwd_tc(const spa_params& p, const void* qkv, const int32_t* seg, int n_seg, void* ao, float* lse,
                            int32_t* d_status, cudaStream_t st) {
  return p.C / p.H == 64 ? fwd_launch<64>(p, qkv, seg, n_seg, ao, lse, d_status, st)
                         : fwd_launch<32>(p, qkv, seg, n_seg, ao, lse, d_status, st);
}

}  // namespace spa

// ------------------------------------------------------------------------------------------------
// Scratch of spa_packed_attention_bwd_static, the attention backward for callers that cannot allocate.
// The D_i values (one float per head and packed row) that the dQ pass hands to the dK/dV pass live in
// this array, which is part of the library image.  Host code must not pass the symbol itself to a
// kernel - on the host it only stands for the array - so the device address is looked up once per
// device, with that device current, and cached.
static __device__ __align__(256) unsigned char g_static_scratch[SPA_STATIC_SCRATCH_BYTES];

namespace spa {
namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};
}  // namespace

// Device address of g_static_scratch on the current device (looked up on first use).
int static_attention_scratch(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { set_cuda_error(e, "spa_packed_attention_bwd_static: cudaGetDevice"); return SPA_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return SPA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || ptr == nullptr) {
      set_cuda_error(e, "spa_packed_attention_bwd_static: cudaGetSymbolAddress");
      return SPA_ERR_CUDA;
    }
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return SPA_OK;
}

}  // namespace spa
