// Row tiles for the attention kernels that follow the segment boundaries (Sec. 3.2: attention stays inside an image,
// or inside a container of an image).
//
// The kernels work on tiles of up to 128 packed query (or key) rows.  Laid over the packed buffer at fixed multiples
// of 128, a tile straddles the boundaries of short segments, and its key range - the union of the segments of its rows -
// grows to two or three tiles where one would do.  The map built here cuts the rows along the segments instead:
//   - a segment longer than 128 rows gets tiles of its own, 128 rows each from its first row on;
//   - consecutive shorter segments are grouped greedily (a group takes the next segment while its rows still fit
//     into 128), so that a tile holds whole segments only and its key range is its own rows.
// Every valid packed row lies in exactly one tile.  Layout of the map (int32): [0] number of tiles, [1] unused,
// then (first row, end row) per tile; tiles of long segments come first (they take the longest).
// One CTA: each thread finds, for its segments, where a group that starts there would end (a binary search in the
// staged offsets); one thread then follows that chain from segment 0.
#include "spa_common.cuh"

namespace spa {
namespace {

constexpr int kMapThreads = 1024;
constexpr int kMapMaxSeg = 4096;  // offsets and group ends are held in shared memory
constexpr int kTileRows = 128;

__global__ void __launch_bounds__(kMapThreads)
attention_tile_map_kernel(const int32_t* __restrict__ seg, int n_seg, int capacity, int max_tiles,
                          int32_t* __restrict__ tiles) {
  pdl_entry();
  __shared__ int32_t off_s[kMapMaxSeg + 1];
  __shared__ int32_t end_s[kMapMaxSeg];  // end_s[s] = t: a group starting at segment s holds segments s .. t-1; t == s: long
  const int tid = threadIdx.x;
  const int Np = packed_rows(seg, n_seg, capacity);
  for (int i = tid; i <= n_seg; i += kMapThreads) {
    const int v = __ldg(seg + i);
    off_s[i] = v < Np ? v : Np;
  }
  __syncthreads();
  for (int s = tid; s < n_seg; s += kMapThreads) {
    const int limit = off_s[s] + kTileRows;
    int lo = s, hi = n_seg + 1;  // last index t in [s, n_seg] with off_s[t] <= limit
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (off_s[mid] <= limit) lo = mid; else hi = mid;
    }
    end_s[s] = lo;
  }
  __syncthreads();
  if (tid == 0) {
    int n = 0;
    for (int s = 0; s < n_seg;) {  // tiles of the long segments
      const int t = end_s[s];
      if (t == s) {
        for (int r = off_s[s]; r < off_s[s + 1] && n < max_tiles; r += kTileRows) {
          tiles[2 + 2 * n] = r;
          tiles[3 + 2 * n] = r + kTileRows < off_s[s + 1] ? r + kTileRows : off_s[s + 1];
          ++n;
        }
        s += 1;
      } else {
        s = t;
      }
    }
    for (int s = 0; s < n_seg;) {  // groups of whole shorter segments
      const int t = end_s[s];
      if (t == s) {
        s += 1;
      } else {
        if (off_s[t] > off_s[s] && n < max_tiles) {
          tiles[2 + 2 * n] = off_s[s];
          tiles[3 + 2 * n] = off_s[t];
          ++n;
        }
        s = t;
      }
    }
    tiles[0] = n;
    tiles[1] = 0;
  }
}

}  // namespace

// Upper bound on the number of tiles for any segmentation of `capacity` rows into n_seg segments: a segment alone
// needs at most len / 128 + 1 tiles, and grouping only lowers the count; independently of n_seg, three tiles per 128
// rows are never exceeded (alternating segments of 129 rows and 1 row).
int attention_max_tiles(const spa_params& p, int n_seg) {
  const long long nw = (p.capacity + kTileRows - 1) / kTileRows;
  const long long a = 3 * nw + 1, b = nw + n_seg;
  return (int)(a < b ? a : b);
}

bool attention_tiles_supported(const spa_params& p, int n_seg) { return n_seg >= 1 && n_seg <= kMapMaxSeg; }

size_t attention_tiles_bytes(const spa_params& p, int n_seg) {
  if (!attention_tiles_supported(p, n_seg)) return 0;
  return ((size_t)(2 + 2 * attention_max_tiles(p, n_seg)) * sizeof(int32_t) + 255) & ~(size_t)255;
}

int launch_attention_tile_map(const spa_params& p, const int32_t* seg, int n_seg, int32_t* tiles, cudaStream_t st) {
  if (!attention_tiles_supported(p, n_seg)) return SPA_ERR_UNSUPPORTED;
  launch_pdl(attention_tile_map_kernel, 1, kMapThreads, 0, st, seg, n_seg, p.capacity, attention_max_tiles(p, n_seg), tiles);
  SPA_CUDA_CHECK_LAUNCH("attention_tile_map_kernel");
  return SPA_OK;
}

}  // namespace spa
