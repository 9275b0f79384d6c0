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
constexpr int SORT_ITEMS = 16;
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

__global__ void __launch_bounds__(SORT_THREADS)
digit_histogram(const uint32_t* __restrict__ keys, int64_t n_max, const uint32_t* __restrict__ n_dev,
                int shift, uint32_t mask, uint32_t* __restrict__ hist, int G) {
  __shared__ uint32_t h[SORT_BINS];
  h[threadIdx.x] = 0;
  __syncthreads();
  const int64_t n = effective_n(n_max, n_dev);
  const int64_t tiles_per_block = tiles_per_block_of(n, G);
  const int64_t begin = (int64_t)blockIdx.x * tiles_per_block * SORT_TILE;
  const int64_t end = min(n, begin + tiles_per_block * SORT_TILE);
  for (int64_t i = begin + threadIdx.x; i < end; i += SORT_THREADS)
    atomicAdd(&h[(keys[i] >> shift) & mask], 1u);
  __syncthreads();
  hist[(size_t)threadIdx.x * G + blockIdx.x] = h[threadIdx.x];
}

// Block d: exclusive prefix over the G per-block counts of digit d, in place; totals[d] = sum.
__global__ void __launch_bounds__(SORT_THREADS)
scan_histogram(uint32_t* __restrict__ hist, uint32_t* __restrict__ totals, int G) {
  __shared__ uint32_t sh[SORT_WARPS + 1];
  uint32_t* row = hist + (size_t)blockIdx.x * G;
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
  if (threadIdx.x == 0) totals[blockIdx.x] = total;
}

#ifndef MTS_SORT_MINBLK
#define MTS_SORT_MINBLK 3
#endif
__global__ void __launch_bounds__(SORT_THREADS, MTS_SORT_MINBLK)
scatter_by_digit(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                 uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out, int64_t n_max,
                 const uint32_t* __restrict__ n_dev, int shift, uint32_t mask,
                 const uint32_t* __restrict__ hist, const uint32_t* __restrict__ totals, int G) {
  __shared__ uint32_t s_key[SORT_TILE];
  __shared__ uint32_t s_val[SORT_TILE];
  __shared__ uint32_t warp_cnt[SORT_WARPS][SORT_BINS];
  __shared__ uint32_t s_off[SORT_BINS];     // first shared-memory position of a digit in the tile
  __shared__ uint32_t s_goff[SORT_BINS];    // global position of this block's next element of a digit
  __shared__ uint32_t sh[SORT_WARPS + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const int64_t n = effective_n(n_max, n_dev);
  const int64_t tiles_per_block = tiles_per_block_of(n, G);

  // where this block's elements of digit `tid` start in the output
  uint32_t dummy;
  uint32_t digit_base = block_exclusive_scan_256(totals[tid], sh, &dummy);
  uint32_t goff = digit_base + hist[(size_t)tid * G + blockIdx.x];

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
#pragma unroll
    for (int k = 0; k < SORT_BINS / 32; ++k) warp_cnt[warp][lane + 32 * k] = 0;
    s_goff[tid] = goff;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < SORT_ITEMS; ++j) {
      const uint32_t d = (key[j] >> shift) & mask;
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
      const uint32_t d = (key[j] >> shift) & mask;
      const uint32_t p = s_off[d] + warp_cnt[warp][d] + rank[j];
      s_key[p] = key[j];
      s_val[p] = val[j];
    }
    __syncthreads();
    // padding keys are all ones: largest digit, last ranks, so they sit at positions >= tile_n
    for (int i = tid; i < tile_n; i += SORT_THREADS) {
      const uint32_t k = s_key[i];
      const uint32_t d = (k >> shift) & mask;
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
    {
      LaunchScope scope(K_SORT_HISTOGRAM, stream);
      digit_histogram<<<G, SORT_THREADS, 0, stream>>>(ki, n_max, n_dev, shift, mask, hist, G);
    }
    {
      LaunchScope scope(K_SORT_SCAN, stream);
      scan_histogram<<<SORT_BINS, SORT_THREADS, 0, stream>>>(hist, totals, G);
    }
    {
      LaunchScope scope(K_SORT_SCATTER, stream);
      scatter_by_digit<<<G, SORT_THREADS, 0, stream>>>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist, totals, G);
    }
    uint32_t* t;
    t = ki; ki = ko; ko = t;
    t = vi; vi = vo; vo = t;
  }
  *keys_out = ki;
  *vals_out = vi;
  return check_launch("radix_sort_pairs");
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
