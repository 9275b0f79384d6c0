// Shared declarations of the mtrains_b200 library: handle layouts, error reporting, small
// device helpers.  Internal to the library; the public surface is include/mtrains_b200.h.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "mtrains_b200.h"

namespace mts {

// ----------------------------------------------------------------------------- errors
int set_error(int code, const char* fmt, ...);
int check_cuda(cudaError_t e, const char* what);
inline int check_launch(const char* what) { return check_cuda(cudaGetLastError(), what); }

// ----------------------------------------------------------------------------- instrumentation
// Every kernel launch of the library sits inside a LaunchScope: it counts the launch and, when
// tracing is on, brackets it with CUDA events on the launching stream.
enum KernelId {
  K_FORWARD = 0, K_LINEARIZE, K_SORT_HISTOGRAM, K_SORT_SCAN, K_SORT_SCATTER, K_UNIQUE, K_REDUCE_CHUNKS,
  K_COMBINE_PARTIALS, K_CACHE_PREPARE, K_CACHE_DESCRIBE, K_CACHE_PROBE_REPLACE, K_CACHE_LISTS, K_CACHE_SCATTER_SLOTS,
  K_CACHE_SAVE_VICTIMS, K_CACHE_FETCH_MISSES, K_CACHE_WRITE_VICTIMS, K_CACHE_FLUSH, K_OTHER, K_COUNT
};

struct LaunchScope {
  LaunchScope(int kernel_id, cudaStream_t stream);
  ~LaunchScope();
  int slot;
  cudaStream_t stream;
};

// ----------------------------------------------------------------------------- tables
// Per-table metadata as the kernels see it (device array of T entries).
struct TableMeta {
  int64_t rows;
  int64_t row_offset;      // linear row id of row 0
  int64_t weight_offset;   // element offset inside the backing buffer
  int32_t dim;
  int32_t out_offset;      // first output column
  int32_t cache_id;        // -1: HBM resident; >= 0: host tier behind this cache
  int32_t vec16;           // 16-byte chunks per row
};

// Row storage of each cache, passed to kernels by value.
struct CachePtrs {
  void* data[MTS_MAX_CACHES];
  uint8_t* dirty[MTS_MAX_CACHES];
};

}  // namespace mts

struct mts_tables {
  int32_t T = 0;
  int32_t dtype = 0;
  int32_t elem_bytes = 4;
  int32_t max_dim = 0;
  int32_t total_dim = 0;
  int32_t any_cached = 0;
  int32_t n_cache_ids = 0;
  int64_t total_rows = 0;
  std::vector<mts::TableMeta> h_meta;
  mts::TableMeta* d_meta = nullptr;
  void* dev_weights = nullptr;
  void* host_weights = nullptr;
  float* momentum = nullptr;
  int32_t* d_status = nullptr;       // sticky status bits
  int32_t sm_count = 148;
};

namespace mts {

constexpr int STATUS_INDEX_CLAMPED = 1;

// ----------------------------------------------------------------------------- device helpers
__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

__device__ __forceinline__ uint4 ld_nc_16(const void* p) {
  return __ldg(reinterpret_cast<const uint4*>(p));
}

// acc0 += lo half of v, acc1 += hi half of v, in fp32.  The mixed-precision add of sm_100 takes the
// fp16 operand as it is (same result as converting first: the conversion is exact), which halves
// the instructions of an fp16 accumulation.
__device__ __forceinline__ void add_half2(float& acc0, float& acc1, uint32_t v) {
  asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\t"
      "add.rn.f32.f16 %0, lo, %0;\n\tadd.rn.f32.f16 %1, hi, %1;\n\t}"
      : "+f"(acc0), "+f"(acc1) : "r"(v));
}

// 8 halves packed in a uint4 -> 8 floats added into acc.
__device__ __forceinline__ void add_half8(float* acc, const uint4& v) {
  add_half2(acc[0], acc[1], v.x);
  add_half2(acc[2], acc[3], v.y);
  add_half2(acc[4], acc[5], v.z);
  add_half2(acc[6], acc[7], v.w);
}

__device__ __forceinline__ void add_float4(float* acc, const uint4& v) {
  acc[0] += __uint_as_float(v.x);
  acc[1] += __uint_as_float(v.y);
  acc[2] += __uint_as_float(v.z);
  acc[3] += __uint_as_float(v.w);
}

// Clamp a row id into [0, rows) and raise the sticky status bit when it was outside.
__device__ __forceinline__ int64_t clamp_index(int64_t idx, int64_t rows, int32_t* status) {
  if (idx < 0 || idx >= rows) {
    atomicOr(status, STATUS_INDEX_CLAMPED);
    idx = idx < 0 ? 0 : rows - 1;
  }
  return idx;
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ----------------------------------------------------------------------------- sorting (radix_sort.cu)
// Stable LSD radix sort of (key, value) pairs on the low `key_bits` bits of key - key_base.
// keys_a/vals_a hold the input; *_b are same-sized scratch.  The sorted result ends in
// (*keys_out, *vals_out), which point at either the a or the b buffers.
// hist: scratch of sort_hist_words(n_max, key_bits) uint32.
size_t sort_hist_words(int64_t n_max, int key_bits);
// Pass plan of the sort: the fewest passes of at most SORT_MAX_DIGIT_BITS bits, the key bits split
// evenly over them.
constexpr int SORT_MAX_DIGIT_BITS = 11;
inline int sort_passes(int key_bits) { return key_bits <= 8 ? 1 : (key_bits + SORT_MAX_DIGIT_BITS - 1) / SORT_MAX_DIGIT_BITS; }
inline int sort_digit_bits(int key_bits) { const int p = sort_passes(key_bits); return (key_bits + p - 1) / p; }
// Segments of a segmented sort: segment t = positions [offsets[t*stride], offsets[(t+1)*stride]),
// digits taken from key - meta[t].row_offset.  An unsegmented sort takes its digits from key - base.
struct SortSegments {
  const int64_t* offsets;    // device
  int32_t stride;
  const TableMeta* meta;     // device
  uint32_t base;
};
size_t sort_hist_words_segmented(int64_t n, int T, int key_bits);
// Sorts every segment on its own by the low key_bits of (key - base of its segment); same buffers and
// result convention as radix_sort_pairs, hist: sort_hist_words_segmented(n, T, key_bits) uint32.
int radix_sort_pairs_segmented(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b, int64_t n,
                               int T, const SortSegments& seg, int key_bits, uint32_t* hist, uint32_t** keys_out,
                               uint32_t** vals_out, cudaStream_t stream);
// n_max is the host-known element count or an upper bound of it; when n_dev is not null the
// kernels use min(*n_dev, n_max) (a device-resident count) instead.
int radix_sort_pairs(uint32_t* keys_a, uint32_t* vals_a, uint32_t* keys_b, uint32_t* vals_b,
                     int64_t n_max, const uint32_t* n_dev, int key_bits, uint32_t key_base, uint32_t* hist,
                     uint32_t** keys_out, uint32_t** vals_out, cudaStream_t stream);

// Distinct keys of an ascending key array.  Writes seg_start[u] = first position of the u-th
// distinct key (u < U), seg_start[U] = n, and *n_unique = U (device).  uniq_idx (nullable,
// [n]) receives for every position the index u of its key.  scratch: scan_scratch_words() uint32.
size_t scan_scratch_words();
int unique_segments(const uint32_t* sorted_keys, int64_t n_max, const uint32_t* n_dev, uint32_t* seg_start,
                    uint32_t* uniq_idx, uint32_t* n_unique, uint32_t* scratch, cudaStream_t stream);

// Cache row storage as kernels take it; validates the caller's pointer arrays.
int fill_cache_ptrs(const mts_tables* h, void* const* host_cache_data, uint8_t* const* host_cache_dirty,
                    int32_t n_caches, const int32_t* slot_of_lookup, CachePtrs* out);

}  // namespace mts
