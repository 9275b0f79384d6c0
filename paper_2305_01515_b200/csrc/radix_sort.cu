// Stable LSD radix sort of (uint32 key, uint32 value) pairs and the distinct-key pass that
// follows it.  Used to group the lookups of a batch by row (backward: the aggregation of
// Section 5.9; cache: the grouping of requests in Section 5.5.1).  Stability is what makes
// the backward deterministic: equal keys keep their input order.
//
// Digits are 8 to 11 bits wide: the key bits are split evenly over the fewest passes of at most 11
// bits (20 bits: two passes of 10; 24: three of 8; 27: three of 9).
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

static int sort_bins(int key_bits) { return 1 << std::max(8, sort_digit_bits(key_bits)); }
size_t sort_hist_words(int64_t n, int key_bits) {
  const int64_t G = std::min<int64_t>(std::max<int64_t>(ceil_div(n, SORT_TILE), 1), SORT_MAX_BLOCKS);
  return (size_t)sort_bins(key_bits) * (size_t)(G + 1);
}

// Segmented sort: the input is a sequence of T segments (the lookups of a batch arrive grouped by
// table) and each segment is sorted on its own, on the digits of key - base[t].  Keys of different
// tables never have to be compared, so only the bits of the largest table's row index are sorted
// (20 instead of 25 bits for 26 tables of a million rows), and a table whose row index has no bit
// left in a pass is only copied in that pass.
constexpr int SORT_SEG_TILES = 4;
int sort_segment_blocks(int64_t n, int T) {
  const int64_t avg_tiles = (n / (T > 0 ? T : 1) + SORT_TILE - 1) / SORT_TILE;
  int64_t g = 1;
  while (g * SORT_SEG_TILES < 2 * avg_tiles) g <<= 1;   // about SORT_SEG_TILES / 2 .. SORT_SEG_TILES tiles per block for an average table
  const int64_t cap = std::max<int64_t>(64, SORT_MAX_BLOCKS / (T > 0 ? T : 1));
  return (int)std::min<int64_t>(std::min<int64_t>(g, cap), SORT_MAX_BLOCKS);
}
size_t sort_hist_words_segmented(int64_t n, int T, int key_bits) {
  return (size_t)T * sort_bins(key_bits) * (size_t)(sort_segment_blocks(n, T) + 1);
}

// Bounds and key base of the segment a block works on (the whole input when SEG is false), and
// whether every digit of the segment is zero from bit `shift` on (then the pass only copies it).
template <bool SEG>
__device__ __forceinline__ void segment_of_block(const SortSegments& seg, int64_t n_max, const uint32_t* n_dev,
                                                 int shift, int64_t* seg_begin, int64_t* n, uint32_t* base,
                                                 bool* exhausted) {
  if (SEG) {
    const int t = blockIdx.y;
    *seg_begin = seg.offsets[(int64_t)t * seg.stride];
    *n = seg.offsets[(int64_t)(t + 1) * seg.stride] - *seg_begin;
    *base = (uint32_t)seg.meta[t].row_offset;
    *exhausted = ((uint64_t)(seg.meta[t].rows - 1) >> shift) == 0;
  } else {
    *seg_begin = 0;
    *n = effective_n(n_max, n_dev);
    *base = seg.base;
    *exhausted = false;
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

// hist[(segment * BINS + digit) * G + block]
template <int BITS, bool SEG>
__global__ void __launch_bounds__(SORT_THREADS)
digit_histogram(const uint32_t* __restrict__ keys, int64_t n_max, const uint32_t* __restrict__ n_dev,
                int shift, uint32_t mask, uint32_t* __restrict__ hist, int G, SortSegments seg) {
  constexpr int BINS = 1 << BITS;
  __shared__ uint32_t h[BINS];
  int64_t seg_begin, n;
  uint32_t base;
  bool exhausted;
  segment_of_block<SEG>(seg, n_max, n_dev, shift, &seg_begin, &n, &base, &exhausted);
  const int64_t tiles_per_block = tiles_per_block_of(n, G);
  const int64_t begin = (int64_t)blockIdx.x * tiles_per_block * SORT_TILE;
  const int64_t end = min(n, begin + tiles_per_block * SORT_TILE);
  if (exhausted) {
    // every digit is zero: the count of digit 0 is the size of the block's range
    for (int d = threadIdx.x; d < BINS; d += SORT_THREADS)
      hist[((size_t)blockIdx.y * BINS + d) * G + blockIdx.x] = d == 0 ? (uint32_t)max((int64_t)0, end - begin) : 0u;
    return;
  }
  for (int d = threadIdx.x; d < BINS; d += SORT_THREADS) h[d] = 0;
  __syncthreads();
  for (int64_t i = begin + threadIdx.x; i < end; i += SORT_THREADS)
    atomicAdd(&h[((keys[seg_begin + i] - base) >> shift) & mask], 1u);
  __syncthreads();
  for (int d = threadIdx.x; d < BINS; d += SORT_THREADS)
    hist[((size_t)blockIdx.y * BINS + d) * G + blockIdx.x] = h[d];
}

// Block (d, segment): exclusive prefix over the G per-block counts of digit d, in place; totals = sum.
__global__ void __launch_bounds__(SORT_THREADS)
scan_histogram(uint32_t* __restrict__ hist, uint32_t* __restrict__ totals, int G) {
  __shared__ uint32_t sh[SORT_WARPS + 1];
  uint32_t* row = hist + ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * G;
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
  if (threadIdx.x == 0) totals[blockIdx.y * gridDim.x + blockIdx.x] = total;
}

// The same scan for short rows (segmented sort: few blocks per segment): one warp per (digit, segment).
__global__ void __launch_bounds__(SORT_THREADS)
scan_histogram_rows(uint32_t* __restrict__ hist, uint32_t* __restrict__ totals, int G, int n_rows) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * SORT_WARPS + (threadIdx.x >> 5);     // r = segment * BINS + digit
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

// Shared memory of scatter_by_digit<BITS>: the tile (keys, values), per-warp digit counts (16 bits: a
// warp holds 512 elements), the digit offsets inside the tile and in the output.
template <int BITS>
constexpr size_t scatter_smem_bytes() {
  return (size_t)SORT_TILE * 8 + (size_t)SORT_WARPS * (1 << BITS) * 2 + (size_t)(1 << BITS) * 8 + 64;
}

template <int BITS, bool SEG>
__global__ void __launch_bounds__(SORT_THREADS, 3)
scatter_by_digit(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                 uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out, int64_t n_max,
                 const uint32_t* __restrict__ n_dev, int shift, uint32_t mask,
                 const uint32_t* __restrict__ hist, const uint32_t* __restrict__ totals, int G, SortSegments seg) {
  constexpr int BINS = 1 << BITS;
  constexpr int DPT = BINS / SORT_THREADS;      // digits per thread: thread tid owns digits tid*DPT .. tid*DPT + DPT-1
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* s_key = reinterpret_cast<uint32_t*>(smem_raw);
  uint32_t* s_val = s_key + SORT_TILE;
  uint32_t* s_off = s_val + SORT_TILE;          // first shared-memory position of a digit in the tile
  uint32_t* s_goff = s_off + BINS;              // global position of this block's next element of a digit
  uint32_t* sh = s_goff + BINS;                 // 9 words (+ padding to 16)
  uint16_t* warp_cnt = reinterpret_cast<uint16_t*>(sh + 16);    // [SORT_WARPS][BINS]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  int64_t seg_begin, n;
  uint32_t base;
  bool exhausted;
  segment_of_block<SEG>(seg, n_max, n_dev, shift, &seg_begin, &n, &base, &exhausted);
  const int64_t tiles_per_block = tiles_per_block_of(n, G);
  keys_in += seg_begin; vals_in += seg_begin; keys_out += seg_begin; vals_out += seg_begin;
  const int64_t begin = (int64_t)blockIdx.x * tiles_per_block * SORT_TILE;
  const int64_t end = min(n, begin + tiles_per_block * SORT_TILE);
  if (exhausted) {
    // no bit of this segment's keys is left: the pass keeps the order, copy the block's range
    for (int64_t i = begin + tid; i < end; i += SORT_THREADS) {
      keys_out[i] = keys_in[i];
      vals_out[i] = vals_in[i];
    }
    return;
  }

  // where this block's elements of the thread's digits start in the (segment's) output
  uint32_t goff[DPT];
  {
    uint32_t tot[DPT], sum = 0;
#pragma unroll
    for (int k = 0; k < DPT; ++k) { tot[k] = totals[blockIdx.y * BINS + tid * DPT + k]; sum += tot[k]; }
    uint32_t dummy;
    uint32_t digit_base = block_exclusive_scan_256(sum, sh, &dummy);
#pragma unroll
    for (int k = 0; k < DPT; ++k) {
      goff[k] = digit_base + hist[((size_t)blockIdx.y * BINS + tid * DPT + k) * G + blockIdx.x];
      digit_base += tot[k];
    }
  }

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
    {
      uint32_t* wc32 = reinterpret_cast<uint32_t*>(warp_cnt + warp * BINS);
#pragma unroll
      for (int k = 0; k < BINS / 64; ++k) wc32[lane + 32 * k] = 0u;
    }
#pragma unroll
    for (int k = 0; k < DPT; ++k) s_goff[tid * DPT + k] = goff[k];
    __syncwarp();
#pragma unroll
    for (int j = 0; j < SORT_ITEMS; ++j) {
      const uint32_t d = digit_of(j);
      const uint32_t peers = __match_any_sync(0xffffffffu, d);
      const int leader = __ffs(peers) - 1;
      uint32_t basec = 0;
      if (lane == leader) {
        basec = warp_cnt[warp * BINS + d];
        warp_cnt[warp * BINS + d] = (uint16_t)(basec + __popc(peers));
      }
      basec = __shfl_sync(0xffffffffu, basec, leader);
      rank[j] = (uint16_t)(basec + __popc(peers & lt_mask));
      __syncwarp();
    }
    __syncthreads();
    // the thread's digits: prefix over warps, then over digits
    uint32_t run[DPT], sum = 0;
#pragma unroll
    for (int k = 0; k < DPT; ++k) {
      const int d = tid * DPT + k;
      uint32_t r = 0;
#pragma unroll
      for (int w = 0; w < SORT_WARPS; ++w) {
        const uint32_t c = warp_cnt[w * BINS + d];
        warp_cnt[w * BINS + d] = (uint16_t)r;
        r += c;
      }
      run[k] = r;
      sum += r;
    }
    uint32_t tot;
    uint32_t off = block_exclusive_scan_256(sum, sh, &tot);
#pragma unroll
    for (int k = 0; k < DPT; ++k) { s_off[tid * DPT + k] = off; off += run[k]; }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < SORT_ITEMS; ++j) {
      const uint32_t d = digit_of(j);
      const uint32_t p = s_off[d] + warp_cnt[warp * BINS + d] + rank[j];
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
#pragma unroll
    for (int k = 0; k < DPT; ++k) {
      uint32_t mine = run[k];
      if ((uint32_t)(tid * DPT + k) == mask) mine -= (uint32_t)(SORT_TILE - tile_n);
      goff[k] += mine;
    }
    __syncthreads();
  }
}

namespace {

template <int BITS, bool SEG>
int launch_pass(const uint32_t* ki, const uint32_t* vi, uint32_t* ko, uint32_t* vo, int64_t n_max,
                const uint32_t* n_dev, int shift, uint32_t mask, uint32_t* hist, uint32_t* totals, int G, int T,
                const SortSegments& seg, cudaStream_t stream) {
  constexpr int BINS = 1 << BITS;
  constexpr size_t SMEM = scatter_smem_bytes<BITS>();
  static bool attr_set[64] = {};                         // per device: the opt-in for more than 48 KB
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return set_error(MTS_ERR_CUDA, "sort: cudaGetDevice");
  if (!attr_set[dev]) {
    int rc = check_cuda(cudaFuncSetAttribute(scatter_by_digit<BITS, SEG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)SMEM), "cudaFuncSetAttribute(scatter_by_digit)");
    if (rc != MTS_OK) return rc;
    attr_set[dev] = true;
  }
  const dim3 grid((unsigned)G, SEG ? (unsigned)T : 1u);
  {
    LaunchScope scope(K_SORT_HISTOGRAM, stream);
    digit_histogram<BITS, SEG><<<grid, SORT_THREADS, 0, stream>>>(ki, n_max, n_dev, shift, mask, hist, G, seg);
  }
  {
    LaunchScope scope(K_SORT_SCAN, stream);
    const int n_rows = (SEG ? T : 1) * BINS;
    if (G <= 64)
      scan_histogram_rows<<<(unsigned)ceil_div(n_rows, SORT_WARPS), SORT_THREADS, 0, stream>>>(hist, totals, G, n_rows);
    else
      scan_histogram<<<dim3(BINS, SEG ? (unsigned)T : 1u), SORT_THREADS, 0, stream>>>(hist, totals, G);
  }
  {
    LaunchScope scope(K_SORT_SCATTER, stream);
    scatter_by_digit<BITS, SEG><<<grid, SORT_THREADS, SMEM, stream>>>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist,
                                                                     totals, G, seg);
  }
  return MTS_OK;
}

template <bool SEG>
int run_passes(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b, int64_t n_max,
               const uint32_t* n_dev, int key_bits, uint32_t* hist, int G, int T, const SortSegments& seg,
               uint32_t** keys_out, uint32_t** vals_out, cudaStream_t stream) {
  const int passes = sort_passes(key_bits), width = sort_digit_bits(key_bits);
  const int bins_bits = width <= 8 ? 8 : width;          // the kernels exist for 8 to SORT_MAX_DIGIT_BITS bits
  uint32_t* totals = hist + (size_t)(SEG ? T : 1) * (1u << bins_bits) * G;
  uint32_t *ki = keys_a, *vi = vals_a, *ko = keys_b, *vo = vals_b;
  for (int p = 0; p < passes; ++p) {
    const int shift = width * p;
    const int bits = std::min(width, key_bits - shift);
    const uint32_t mask = (1u << bits) - 1u;
    int rc;
    switch (bins_bits) {
      case 8: rc = launch_pass<8, SEG>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist, totals, G, T, seg, stream); break;
      case 9: rc = launch_pass<9, SEG>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist, totals, G, T, seg, stream); break;
      case 10: rc = launch_pass<10, SEG>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist, totals, G, T, seg, stream); break;
      default: rc = launch_pass<11, SEG>(ki, vi, ko, vo, n_max, n_dev, shift, mask, hist, totals, G, T, seg, stream); break;
    }
    if (rc != MTS_OK) return rc;
    uint32_t* t;
    t = ki; ki = ko; ko = t;
    t = vi; vi = vo; vo = t;
  }
  *keys_out = ki;
  *vals_out = vi;
  return check_launch("radix sort passes");
}

}  // namespace

int radix_sort_pairs(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b,
                     int64_t n_max, const uint32_t* n_dev, int key_bits, uint32_t key_base, uint32_t* hist,
                     uint32_t** keys_out, uint32_t** vals_out, cudaStream_t stream) {
  *keys_out = keys_a;
  *vals_out = vals_a;
  if (n_max <= 1 || key_bits <= 0) return MTS_OK;
  const int64_t ntiles = ceil_div(n_max, SORT_TILE);
  // a device-resident count is usually far below its host bound (the keys that missed, the victims): fewer
  // blocks then, so that the histogram and its scan are not sized for the bound
  const int G = (int)std::min<int64_t>(ntiles, n_dev != nullptr ? 256 : SORT_MAX_BLOCKS);
  const SortSegments none{nullptr, 0, nullptr, key_base};
  return run_passes<false>(keys_a, vals_a, keys_b, vals_b, n_max, n_dev, key_bits, hist, G, 1, none, keys_out, vals_out,
                           stream);
}

int radix_sort_pairs_segmented(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b, int64_t n,
                               int T, const SortSegments& seg, int key_bits, uint32_t* hist, uint32_t** keys_out,
                               uint32_t** vals_out, cudaStream_t stream) {
  *keys_out = keys_a;
  *vals_out = vals_a;
  if (n <= 1 || key_bits <= 0 || T <= 0) return MTS_OK;
  const int G = sort_segment_blocks(n, T);
  return run_passes<true>(keys_a, vals_a, keys_b, vals_b, n, nullptr, key_bits, hist, G, T, seg, keys_out, vals_out,
                          stream);
}

// ------------------------------------------------------------------------------------ distinct keys

constexpr int UNIQ_THREADS = 256;
constexpr int UNIQ_ITEMS = 4;                       // consecutive keys per thread and round: one block scan per 1024 keys

__device__ __forceinline__ int64_t per_block_of(int64_t n, int G) {
  const int64_t per = (n + G - 1) / G;
  constexpr int64_t ROUND = UNIQ_THREADS * UNIQ_ITEMS;
  return (per + ROUND - 1) / ROUND * ROUND;
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
  for (int64_t t0 = begin; t0 < end; t0 += UNIQ_THREADS * UNIQ_ITEMS) {
    // a thread looks at UNIQ_ITEMS consecutive keys
    const int64_t i0 = t0 + (int64_t)threadIdx.x * UNIQ_ITEMS;
    uint32_t k[UNIQ_ITEMS + 1];
    k[0] = (i0 > 0 && i0 < end) ? keys[i0 - 1] : 0u;
#pragma unroll
    for (int j = 0; j < UNIQ_ITEMS; ++j) k[j + 1] = i0 + j < end ? keys[i0 + j] : 0u;
    uint32_t head[UNIQ_ITEMS], mine = 0;
#pragma unroll
    for (int j = 0; j < UNIQ_ITEMS; ++j) {
      head[j] = (i0 + j < end && (i0 + j == 0 || k[j + 1] != k[j])) ? 1u : 0u;
      mine += head[j];
    }
    uint32_t total;
    uint32_t at = base + block_exclusive_scan_256(mine, sh, &total);
#pragma unroll
    for (int j = 0; j < UNIQ_ITEMS; ++j) {
      if (head[j]) seg_start[at] = (uint32_t)(i0 + j);
      at += head[j];
      if (i0 + j < end && uniq_idx) uniq_idx[i0 + j] = at - 1u;
    }
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
