// Stable LSD radix sort of (uint32 key, uint32 value) pairs and the distinct-key pass that
// follows it.  Used to group the lookups of a batch by row (backward: the aggregation of
// Section 5.9; cache: the grouping of requests in Section 5.5.1).  Stability is what makes
// the backward deterministic: equal keys keep their input order.
//
// One pass = three kernels over G blocks, block b owning a contiguous range of tiles:
//   digit_histogram  : hist[d][b] = occurrences of digit d in block b's range
//   scan_histogram   : per digit, exclusive prefix over blocks (+ digit totals)
//   scatter_by_digit : per tile, stable in-block ranking (match_any within a warp, prefix
//                      over warps), reorder through shared memory so that each digit's
//                      run is written with consecutive threads on consecutive addresses.
// No block waits on another block inside a kernel; ordering comes from kernel boundaries.
#include <algorithm>

#include "common.cuh"

namespace mts {

constexpr int SORT_THREADS = 256;
constexpr int SORT_WARPS = SORT_THREADS / 32;
#ifndef MTS_SORT_ITEMS
#define MTS_SORT_ITEMS 16
#endif
constexpr int SORT_ITEMS = MTS_SORT_ITEMS;
constexpr int SORT_TILE = SORT_THREADS * SORT_ITEMS;   // 4096 pairs
constexpr int SORT_BINS = 256;
constexpr int SORT_MAX_BLOCKS = 1024;

// Element count of a launch: the host bound, or the smaller device-resident count when the
// caller only knows an upper bound on the host (no host synchronisation).
__device__ __forceinline__ int64_t effective_n(int64_t n_max, const uint32_t* n_dev) {
  if (n_dev == nullptr) return n_max;
  const int64_t n = (int64_t)*n_dev;
  return n < n_max ? n : n_max;
}

__device__ __forceinline__ int64_t tiles_per_block_of(int64_t n, int G) {
  const int64_t ntiles = (n + SORT_TILE - 1) / SORT_TILE;
  return (ntiles + G - 1) / G;
}

size_t sort_hist_words() { return (size_t)SORT_BINS * SORT_MAX_BLOCKS + SORT_BINS; }

// Segmented sort: the input is a sequence of T segments (the lookups of a batch arrive grouped by
// table) and each segment is sorted on its own, on the digits of key - base[t].  Keys of different
// tables never have to be compared, so only the bits of the largest table's row index are sorted
// (20 instead of 25 bits for 26 tables of a million rows: 3 passes instead of 4).
#ifndef MTS_SORT_SEG_TILES
#define MTS_SORT_SEG_TILES 4
#endif
int sort_segment_blocks(int64_t n, int T) {
  const int64_t avg_tiles = (n / (T > 0 ? T : 1) + SORT_TILE - 1) / SORT_TILE;
  int64_t g = 1;
  while (g * MTS_SORT_SEG_TILES < 2 * avg_tiles) g <<= 1;   // about MTS_SORT_SEG_TILES / 2 .. MTS_SORT_SEG_TILES tiles per block for an average table
  const int64_t cap = std::max<int64_t>(64, SORT_MAX_BLOCKS / (T > 0 ? T : 1));
  return (int)std::min<int64_t>(std::min<int64_t>(g, cap), SORT_MAX_BLOCKS);
}
size_t sort_hist_words_segmented(int64_t n, int T) {
  return (size_t)T * SORT_BINS * sort_segment_blocks(n, T) + (size_t)T * SORT_BINS;
}

// Bounds and key base of the segment a block works on (the whole input when SEG is false).
template <bool SEG>
__device__ __forceinline__ void segment_of_block(const SortSegments& seg, int64_t n_max, const uint32_t* n_dev,
                                                 int64_t* seg_begin, int64_t* n, uint32_t* base) {
  if (SEG) {
    const int t = blockIdx.y;
    *seg_begin = seg.offsets[(int64_t)t * seg.stride];
    *n = seg.offsets[(int64_t)(t + 1) * seg.stride] - *seg_begin;
    *base = (uint32_t)seg.meta[t].row_offset;
  } else {
    *seg_begin = 0;
    *n = effective_n(n_max, n_dev);
    *base = 0u;
  }
}
size_t scan_scratch_words() { return SORT_MAX_BLOCKS + 8; }

// Exclusive scan of one value per thread over a 256-thread block; returns the exclusive
// prefix, *total receives the block sum.  `sh` is 9 words of shared memory.
__device__ __forceinline__ uint32_t block_exclusive_scan_256(uint32_t v, uint32_t* sh, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) sh[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = lane < SORT_WARPS ? sh[lane] : 0u;
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < SORT_WARPS; o <<= 1) {
      uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    if (lane < SORT_WARPS) sh[lane] = winc - w;
    if (lane == SORT_WARPS - 1) sh[SORT_WARPS] = winc;
  }
  __syncthreads();
  uint32_t res = sh[warp] + inc - v;
  *total = sh[SORT_WARPS];
  __syncthreads();
  return res;
}

template <bool SEG>
__global__ void __launch_bounds__(SORT_THREADS)
digit_histogram(const uint32_t* __restrict__ keys, int64_t n_max, const uint32_t* __restrict__ n_dev,
                int shift, uint32_t mask, uint32_t* __restrict__ hist, int G, SortSegments seg) {
  __shared__ uint32_t h[SORT_BINS];
  h[threadIdx.x] = 0;
  __syncthreads();
  int64_t seg_begin, n;
  uint32_t base;
  segment_of_block<SEG>(seg, n_max, n_dev, &seg_begin, &n, &base);
  const int64_t tiles_per_block = tiles_per_block_of(n, G);
  const int64_t begin = (int64_t)blockIdx.x * tiles_per_block * SORT_TILE;
  const int64_t end = min(n, begin + tiles_per_block * SORT_TILE);
  for (int64_t i = begin + threadIdx.x; i < end; i += SORT_THREADS)
    atomicAdd(&h[((keys[seg_begin + i] - base) >> shift) & mask], 1u);
  __syncthreads();
  hist[((size_t)blockIdx.y * SORT_BINS + threadIdx.x) * G + blockIdx.x] = h[threadIdx.x];
}

// Block (d, segment): exclusive prefix over the G per-block counts of digit d, in place; totals = sum.
__global__ void __launch_bounds__(SORT_THREADS)
scan_histogram(uint32_t* __restrict__ hist, uint32_t* __restrict__ totals, int G) {
  __shared__ uint32_t sh[SORT_WARPS + 1];
  uint32_t* row = hist + ((size_t)blockIdx.y * SORT_BINS + blockIdx.x) * G;
  const int per = (G + SORT_THREADS - 1) / SORT_THREADS;      // <= 4
  const int j0 = threadIdx.x * per;
  uint32_t v[SORT_MAX_BLOCKS / SORT_THREADS];
  uint32_t s = 0;
#pragma unroll
  for (int k = 0; k < SORT_MAX_BLOCKS / SORT_THREADS; ++k) {
    v[k] = (k < per && j0 + k < G) ? row[j0 + k] : 0u;
    s += v[k];
  }
  uint32_t total;
  uint32_t ex = block_exclusive_scan_256(s, sh, &total);
#pragma unroll
  for (int k = 0; k < SORT_MAX_BLOCKS / SORT_THREADS; ++k) {
    if (k < per && j0 + k < G) row[j0 + k] = ex;
    ex += v[k];
  }
  if (threadIdx.x == 0) totals[blockIdx.y * SORT_BINS + blockIdx.x] = total;
}

// The same scan for short rows (segmented sort: few blocks per segment): one warp per (digit, segment).
__global__ void __launch_bounds__(SORT_THREADS)
scan_histogram_rows(uint32_t* __restrict__ hist, uint32_t* __restrict__ totals, int G, int n_rows) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * SORT_WARPS + (threadIdx.x >> 5);     // r = segment * SORT_BINS + digit
  if (r >= n_rows) return;
  uint32_t* row = hist + (size_t)r * G;
  uint32_t carry = 0;
  for (int j0 = 0; j0 < G; j0 += 32) {
    const int j = j0 + lane;
    const uint32_t v = j < G ? row[j] : 0u;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (j < G) row[j] = carry + inc - v;
    carry += __shfl_sync(0xffffffffu, inc, 31);
  }
  if (lane == 0) totals[r] = carry;
}

#ifndef MTS_SORT_MINBLK
#define MTS_SORT_MINBLK 3
#endif
template <bool SEG>
__global__ void __launch_bounds__(SORT_THREADS, MTS_SORT_MINBLK)
scatter_by_digit(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                 uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out, int64_t n_max,
                 const uint32_t* __restrict__ n_dev, int shift, uint32_t mask,
                 const uint32_t* __restrict__ hist, const uint32_t* __restrict__ totals, int G, SortSegments seg) {
  __shared__ uint32_t s_key[SORT_TILE];
  __shared__ uint32_t s_val[SORT_TILE];
  __shared__ uint32_t warp_cnt[SORT_WARPS][SORT_BINS];
  __shared__ uint32_t s_off[SORT_BINS];     // first shared-memory position of a digit in the tile
  __shared__ uint32_t s_goff[SORT_BINS];    // global position of this block's next element of a digit
  __shared__ uint32_t sh[SORT_WARPS + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  int64_t seg_begin, n;
  uint32_t base;
  segment_of_block<SEG>(seg, n_max, n_dev, &seg_begin, &n, &base);
  const int64_t tiles_per_block = tiles_per_block_of(n, G);
  keys_in += seg_begin; vals_in += seg_begin; keys_out += seg_begin; vals_out += seg_begin;

  // where this block's elements of digit `tid` start in the (segment's) output
  uint32_t dummy;
  uint32_t digit_base = block_exclusive_scan_256(totals[blockIdx.y * SORT_BINS + tid], sh, &dummy);
  uint32_t goff = digit_base + hist[((size_t)blockIdx.y * SORT_BINS + tid) * G + blockIdx.x];

  const int64_t begin = (int64_t)blockIdx.x * tiles_per_block * SORT_TILE;
  const int64_t end = min(n, begin + tiles_per_block * SORT_TILE);
  for (int64_t tile = begin; tile < end; tile += SORT_TILE) {
    const int tile_n = (int)min((int64_t)SORT_TILE, end - tile);
    uint32_t key[SORT_ITEMS], val[SORT_ITEMS];
    uint16_t rank[SORT_ITEMS];
#pragma unroll
    for (int j = 0; j < SORT_ITEMS; ++j) {
      const int li = warp * (32 * SORT_ITEMS) + j * 32 + lane;
      const bool valid = li < tile_n;
      key[j] = valid ? keys_in[tile + li] : 0xffffffffu;
      val[j] = valid ? vals_in[tile + li] : 0u;
    }
    // padding takes the largest digit; it comes last in the tile, so it gets the last ranks of that digit
    auto digit_of = [&](int j) -> uint32_t {
      const int li = warp * (32 * SORT_ITEMS) + j * 32 + lane;
      return li < tile_n ? ((key[j] - base) >> shift) & mask : mask;
    };
#pragma unroll
    for (int k = 0; k < SORT_BINS / 32; ++k) warp_cnt[warp][lane + 32 * k] = 0;
    s_goff[tid] = goff;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < SORT_ITEMS; ++j) {
      const uint32_t d = digit_of(j);
      const uint32_t peers = __match_any_sync(0xffffffffu, d);
      const int leader = __ffs(peers) - 1;
      uint32_t basec = 0;
      if (lane == leader) {
        basec = warp_cnt[warp][d];
        warp_cnt[warp][d] = basec + __popc(peers);
      }
      basec = __shfl_sync(0xffffffffu, basec, leader);
      rank[j] = (uint16_t)(basec + __popc(peers & lt_mask));
      __syncwarp();
    }
    __syncthreads();
    // digit `tid`: prefix over warps, then over digits
    uint32_t run = 0;
#pragma unroll
    for (int w = 0; w < SORT_WARPS; ++w) {
      uint32_t c = warp_cnt[w][tid];
      warp_cnt[w][tid] = run;
      run += c;
    }
    uint32_t tot;
    uint32_t off = block_exclusive_scan_256(run, sh, &tot);
    s_off[tid] = off;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < SORT_ITEMS; ++j) {
      const uint32_t d = digit_of(j);
      const uint32_t p = s_off[d] + warp_cnt[warp][d] + rank[j];
      s_key[p] = key[j];
      s_val[p] = val[j];
    }
    __syncthreads();
    // padding has the largest digit and the last ranks, so it sits at positions >= tile_n
    for (int i = tid; i < tile_n; i += SORT_THREADS) {
      const uint32_t k = s_key[i];
      const uint32_t d = ((k - base) >> shift) & mask;
      const uint32_t g = s_goff[d] + (uint32_t)i - s_off[d];
      keys_out[g] = k;
      vals_out[g] = s_val[i];
    }
    uint32_t mine = run;
    if ((uint32_t)tid == mask) mine -= (uint32_t)(SORT_TILE - tile_n);
    goff += mine;
    __syncthreads();
  }
}

int radix_sort_pairs(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b,
                     int64_t n_max, const uint32_t* n_dev, int key_bits, uint32_t* hist,
                     uint32_t** keys_out, uint32_t** vals_out, cudaStream_t stream) {
  *keys_out = keys_a;
  *vals_out = vals_a;
  if (n_max <= 1 || key_bits <= 0) return MTS_OK;
  const int64_t ntiles = ceil_div(n_max, SORT_TILE);
  const int G = (int)std::min<int64_t>(ntiles, SORT_MAX_BLOCKS);
  uint32_t* totals = hist + (size_t)SORT_BINS * SORT_MAX_BLOCKS;
  const int passes = (key_bits + 7) / 8;
  uint32_t *ki = keys_a, *vi = vals_a, *ko = keys_b, *vo = vals_b;
  for (int p = 0; p < passes; ++p) {
    const int shift = 8 * p;
    const int bits = min(8, key_bits - shift);
    const uint32_t mask = (1u << bits) - 1u;
    const SortSegments none{nullptr, 0, nullptr};
    {
      LaunchScope scope(K_SORT_HISTOGRAM, stream);
      digit_histogram<false><<<G, SORT_THREADS, 0, stream>>>(ki, n_max, n_dev, shift, mask, hist, G, none);
    }
    {
      LaunchScope scope(K_SORT_SCAN, stream);
      scan_histogram<<<SORT_BINS, SORT_THREADS, 0, stream>>>(hist, totals, G);
    }
    {
      LaunchScope scope(K_SORT_SCATTER, stream);
      scatter_by_digit<false><<<G, SORT_THREADS, 0, stream>>>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist, totals, G,
                                                               none);
    }
    uint32_t* t;
    t = ki; ki = ko; ko = t;
    t = vi; vi = vo; vo = t;
  }
  *keys_out = ki;
  *vals_out = vi;
  return check_launch("radix_sort_pairs");
}

int radix_sort_pairs_segmented(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b, int64_t n,
                               int T, const SortSegments& seg, int key_bits, uint32_t* hist, uint32_t** keys_out,
                               uint32_t** vals_out, cudaStream_t stream) {
  *keys_out = keys_a;
  *vals_out = vals_a;
  if (n <= 1 || key_bits <= 0 || T <= 0) return MTS_OK;
  const int G = sort_segment_blocks(n, T);
  uint32_t* totals = hist + (size_t)T * SORT_BINS * G;
  const int passes = (key_bits + 7) / 8;
  const dim3 grid((unsigned)G, (unsigned)T);
  uint32_t *ki = keys_a, *vi = vals_a, *ko = keys_b, *vo = vals_b;
  for (int p = 0; p < passes; ++p) {
    const int shift = 8 * p;
    const int bits = min(8, key_bits - shift);
    const uint32_t mask = (1u << bits) - 1u;
    {
      LaunchScope scope(K_SORT_HISTOGRAM, stream);
      digit_histogram<true><<<grid, SORT_THREADS, 0, stream>>>(ki, n, nullptr, shift, mask, hist, G, seg);
    }
    {
      LaunchScope scope(K_SORT_SCAN, stream);
      const int n_rows = T * SORT_BINS;
      scan_histogram_rows<<<(unsigned)ceil_div(n_rows, SORT_WARPS), SORT_THREADS, 0, stream>>>(hist, totals, G, n_rows);
    }
    {
      LaunchScope scope(K_SORT_SCATTER, stream);
      scatter_by_digit<true><<<grid, SORT_THREADS, 0, stream>>>(ki, vi, ko, vo, n, nullptr, shift, mask, hist, totals, G,
                                                               seg);
    }
    uint32_t* t;
    t = ki; ki = ko; ko = t;
    t = vi; vi = vo; vo = t;
  }
  *keys_out = ki;
  *vals_out = vi;
  return check_launch("radix_sort_pairs_segmented");
}

// ------------------------------------------------------------------------------------ distinct keys

constexpr int UNIQ_THREADS = 256;

__device__ __forceinline__ int64_t per_block_of(int64_t n, int G) {
  const int64_t per = (n + G - 1) / G;
  return (per + UNIQ_THREADS - 1) / UNIQ_THREADS * UNIQ_THREADS;
}

__global__ void __launch_bounds__(UNIQ_THREADS)
count_heads(const uint32_t* __restrict__ keys, int64_t n_max, const uint32_t* __restrict__ n_dev,
            uint32_t* __restrict__ cnt) {
  __shared__ uint32_t sh[SORT_WARPS + 1];
  const int64_t n = effective_n(n_max, n_dev);
  const int64_t per_block = per_block_of(n, gridDim.x);
  const int64_t begin = (int64_t)blockIdx.x * per_block;
  const int64_t end = min(n, begin + per_block);
  uint32_t c = 0;
  for (int64_t i = begin + threadIdx.x; i < end; i += UNIQ_THREADS)
    c += (i == 0 || keys[i] != keys[i - 1]) ? 1u : 0u;
  uint32_t total;
  block_exclusive_scan_256(c, sh, &total);
  if (threadIdx.x == 0) cnt[blockIdx.x] = total;
}

__global__ void __launch_bounds__(UNIQ_THREADS)
scan_block_counts(uint32_t* __restrict__ cnt, int G, uint32_t* __restrict__ n_unique,
                  uint32_t* __restrict__ seg_start, int64_t n_max, const uint32_t* __restrict__ n_dev) {
  __shared__ uint32_t sh[SORT_WARPS + 1];
  const int64_t n = effective_n(n_max, n_dev);
  const int per = (G + UNIQ_THREADS - 1) / UNIQ_THREADS;
  const int j0 = threadIdx.x * per;
  uint32_t v[SORT_MAX_BLOCKS / UNIQ_THREADS];
  uint32_t s = 0;
#pragma unroll
  for (int k = 0; k < SORT_MAX_BLOCKS / UNIQ_THREADS; ++k) {
    v[k] = (k < per && j0 + k < G) ? cnt[j0 + k] : 0u;
    s += v[k];
  }
  uint32_t total;
  uint32_t ex = block_exclusive_scan_256(s, sh, &total);
#pragma unroll
  for (int k = 0; k < SORT_MAX_BLOCKS / UNIQ_THREADS; ++k) {
    if (k < per && j0 + k < G) cnt[j0 + k] = ex;
    ex += v[k];
  }
  if (threadIdx.x == 0) {
    *n_unique = total;
    seg_start[total] = (uint32_t)n;
  }
}

__global__ void __launch_bounds__(UNIQ_THREADS)
write_heads(const uint32_t* __restrict__ keys, int64_t n_max, const uint32_t* __restrict__ n_dev,
            const uint32_t* __restrict__ base_of_block, uint32_t* __restrict__ seg_start,
            uint32_t* __restrict__ uniq_idx) {
  __shared__ uint32_t sh[SORT_WARPS + 1];
  const int64_t n = effective_n(n_max, n_dev);
  const int64_t per_block = per_block_of(n, gridDim.x);
  const int64_t begin = (int64_t)blockIdx.x * per_block;
  const int64_t end = min(n, begin + per_block);
  uint32_t base = base_of_block[blockIdx.x];
  for (int64_t t0 = begin; t0 < end; t0 += UNIQ_THREADS) {
    const int64_t i = t0 + threadIdx.x;
    const bool valid = i < end;
    const uint32_t head = (valid && (i == 0 || keys[i] != keys[i - 1])) ? 1u : 0u;
    uint32_t total;
    uint32_t ex = block_exclusive_scan_256(head, sh, &total);
    if (head) seg_start[base + ex] = (uint32_t)i;
    if (valid && uniq_idx) uniq_idx[i] = base + ex + head - 1u;
    base += total;
  }
}

int unique_segments(const uint32_t* sorted_keys, int64_t n_max, const uint32_t* n_dev, uint32_t* seg_start,
                    uint32_t* uniq_idx, uint32_t* n_unique, uint32_t* scratch, cudaStream_t stream) {
  if (n_max <= 0) {
    int rc = check_cuda(cudaMemsetAsync(n_unique, 0, sizeof(uint32_t), stream), "memset(n_unique)");
    if (rc != MTS_OK) return rc;
    return check_cuda(cudaMemsetAsync(seg_start, 0, sizeof(uint32_t), stream), "memset(seg_start)");
  }
  const int64_t nchunks = ceil_div(n_max, UNIQ_THREADS * 8);
  const int G = (int)std::min<int64_t>(nchunks, SORT_MAX_BLOCKS);
  {
    LaunchScope scope(K_UNIQUE, stream);
    count_heads<<<G, UNIQ_THREADS, 0, stream>>>(sorted_keys, n_max, n_dev, scratch);
  }
  {
    LaunchScope scope(K_UNIQUE, stream);
    scan_block_counts<<<1, UNIQ_THREADS, 0, stream>>>(scratch, G, n_unique, seg_start, n_max, n_dev);
  }
  {
    LaunchScope scope(K_UNIQUE, stream);
    write_heads<<<G, UNIQ_THREADS, 0, stream>>>(sorted_keys, n_max, n_dev, scratch, seg_start, uniq_idx);
  }
  return check_launch("unique_segments");
}

}  // namespace mts
