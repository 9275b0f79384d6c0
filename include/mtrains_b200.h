/*
 * mtrains_b200 — C ABI of the sparse-embedding step of MTrainS-style DLRM training on one
 * NVIDIA B200 (sm_100a): pooled multi-table embedding lookup, backward fused with row-wise
 * Adagrad on the touched rows, and a software-managed set-associative row cache in HBM in
 * front of pinned host memory.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the name starts with host_ or the comment says
 *     "host".  The caller owns every buffer it passes; the library allocates device memory
 *     only inside mts_tables_create and mts_cache_create and frees it in the matching
 *     destroy call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued asynchronously; no entry point synchronises the device except where stated.
 *   - Return value: MTS_OK (0) or a negative MTS_ERR_* code.  Nothing throws, exits, aborts or
 *     traps on the device.  mts_last_error_string() describes the calling thread's last error.
 *   - Layouts: weights of table t are a row-major [rows[t], dim[t]] array of the storage type
 *     (fp32 or IEEE binary16) starting at element weight_offset[t] of its backing buffer;
 *     dim[t] * sizeof(element) must be a multiple of 16 bytes and every base pointer 16-byte
 *     aligned.  Pooled outputs and their gradients are fp32 [B, out_stride] row-major, table t
 *     occupying columns [out_offset[t], out_offset[t] + dim[t]) with out_offset the prefix sum
 *     of dim.  Sparse input is CSR: `indices` int64 [N] and `offsets` int64 [T*B + 1] over bag
 *     id t*B + b (table-major), offsets[T*B] == N.
 */
#ifndef MTRAINS_B200_H_
#define MTRAINS_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MTS_OK 0
#define MTS_ERR_INVALID_ARG (-1)
#define MTS_ERR_ALIGNMENT (-2)
#define MTS_ERR_WORKSPACE (-3)
#define MTS_ERR_CAPACITY (-4)
#define MTS_ERR_CUDA (-5)
#define MTS_ERR_TIMEOUT (-6)
#define MTS_ERR_UNSUPPORTED (-7)

#define MTS_DTYPE_FP32 0
#define MTS_DTYPE_FP16 1

#define MTS_POOL_SUM 0
#define MTS_POOL_MEAN 1
#define MTS_POOL_MAX 2          /* forward only */

#define MTS_POLICY_LRU 0
#define MTS_POLICY_LFU 1

#define MTS_MAX_CACHES 8
#define MTS_CACHE_WAYS 32
#define MTS_NUM_COUNTERS 10

/* Indices into the counter block written by mts_cache_lookup_insert. */
enum {
  MTS_CNT_LOOKUPS = 0,       /* N */
  MTS_CNT_UNIQUE = 1,        /* distinct keys in the call */
  MTS_CNT_HIT_LOOKUPS = 2,   /* lookups whose key was resident before the call */
  MTS_CNT_MISS_LOOKUPS = 3,
  MTS_CNT_UNIQUE_HITS = 4,
  MTS_CNT_UNIQUE_MISSES = 5,
  MTS_CNT_INSERTED = 6,      /* length of the miss list */
  MTS_CNT_EVICTED = 7,       /* length of the evict list */
  MTS_CNT_EVICTED_DIRTY = 8,
  MTS_CNT_OVERFLOW = 9       /* distinct missing keys that found no evictable way */
};

/* Counter block of the two-level cache (mts_cache2_lookup_insert): entries 0..9 are the counters above
 * for the first level, then: */
#define MTS_NUM_COUNTERS2 20
enum {
  MTS_CNT2_L2_HIT_LOOKUPS = 10,   /* lookups that missed the first level and hit the second */
  MTS_CNT2_L2_UNIQUE_HITS = 11,
  MTS_CNT2_PROMOTED = 12,         /* second-level hits inserted into the first level */
  MTS_CNT2_DEMOTED = 13,          /* first-level victims inserted into the second level */
  MTS_CNT2_L2_EVICTED = 14,       /* length of the second-level evict list */
  MTS_CNT2_L2_EVICTED_DIRTY = 15,
  MTS_CNT2_L2_BYPASS = 16,        /* first-level victims that found no second-level way (go to the store) */
  MTS_CNT2_L2_BYPASS_DIRTY = 17,
  MTS_CNT2_L2_DROPPED = 18,       /* second-level hits that found no first-level way (length of the drop list) */
  MTS_CNT2_L2_DROPPED_DIRTY = 19
};

const char* mts_last_error_string(void);

/* ---------------------------------------------------------------------------------------
 * Instrumentation (the paper has no counterpart; it reports external tools only).
 * mts_launch_count: kernels this library has launched in this process so far.
 * mts_trace_enable(1) makes every later launch record a CUDA event before and after itself on
 * its stream (a few microseconds of host time per launch); mts_trace_enable(0) stops it; both
 * drop unreported records.  mts_trace_report waits for the recorded launches and returns, per
 * kernel id in [0, mts_trace_kernel_count()), the summed device time in milliseconds and the
 * number of launches since the last enable/report (host arrays of n >= kernel count entries).
 * Do not enable tracing while a stream is being captured into a CUDA graph. */
int64_t mts_launch_count(void);
int mts_trace_enable(int32_t enable);
int32_t mts_trace_kernel_count(void);
const char* mts_trace_kernel_name(int32_t kernel);
int mts_trace_report(double* host_total_ms, int64_t* host_launches, int32_t n);

/* ---------------------------------------------------------------------------------------
 * Tables.  The paper's model: T embedding tables, table t a 2-D tensor of H_t rows and D
 * columns of p bytes (Section 2.1.2, Eq. 1), the same structure in every memory that holds
 * it (Section 5.2), plus per-table metadata that says which memory serves it (Section 5.8).
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int32_t T;                      /* number of tables (>= 1) */
  int32_t dtype;                  /* MTS_DTYPE_*: storage type of all weights */
  const int64_t* host_rows;       /* host [T]  rows per table (>= 1) */
  const int32_t* host_dim;        /* host [T]  columns per table */
  const int64_t* host_weight_offset; /* host [T]  element offset of table t in its buffer */
  const int32_t* host_cache_id;   /* host [T] or NULL.  -1: rows live in dev_weights.
                                     c >= 0: rows live in the host tier (host_weights_mapped)
                                     and are served through cache c (see mts_cache_*). */
  void* dev_weights;              /* device buffer of the HBM-resident tables (may be NULL
                                     when every table is cached) */
  void* host_weights_mapped;      /* device-visible address of the pinned, mapped host buffer
                                     holding the host-tier tables (NULL when none) */
  float* momentum;                /* device fp32 [sum rows]: one Adagrad state per row, indexed
                                     by linear row id row_offset[t] + r (prefix sum of rows).
                                     Optimizer state stays in HBM (Section 5.6). */
} mts_table_desc;

typedef struct mts_tables mts_tables;

/* Validates the description, copies the per-table metadata to the device (one small
 * allocation) and returns a handle.  Synchronous.  Errors: INVALID_ARG (null, T < 1,
 * rows < 1, cache id out of range), UNSUPPORTED (sum rows >= 2^32, dim > 1024), ALIGNMENT
 * (row bytes or a base pointer not a multiple of 16), CUDA. */
int mts_tables_create(const mts_table_desc* desc, mts_tables** out);
int mts_tables_destroy(mts_tables* tables);

/* Reads and clears the handle's sticky device status word.  Synchronises `stream`.
 * *host_status receives a bit mask: bit 0 = an index outside [0, rows[t]) was seen (the
 * lookup was clamped to a valid row, never read out of bounds). */
int mts_tables_status(mts_tables* tables, int32_t* host_status, void* stream);

/* ---------------------------------------------------------------------------------------
 * Forward: pooled lookup (Section 2.1.1: an embedding operator selects rows of a table and
 * pools them by sum, mean or max).
 *   out[b, out_offset[t] + d] = sum over the lookups i of bag (t, b) of W_t[indices[i], d]
 * accumulated in fp32; MTS_POOL_MEAN divides by the bag length; MTS_POOL_MAX takes the largest of
 * the bag's values in every column instead of their sum (forward only: the backward entry points
 * take sum and mean); an empty bag gives 0 in every mode; an id that occurs twice in a bag counts
 * twice.
 * slot_of_lookup (int32 [N], may be NULL when no table is cached): for a lookup of a cached
 * table, the cache slot holding its row, or -1 = read the row from the host tier directly.
 * A lookup that has a slot may be served without its index being read (the slot names the row);
 * the index-range check of mts_tables_status then covers the lookups of HBM tables and those without
 * a slot, and the cache's lookup reports keys outside its key space (mts_cache_status).
 * host_cache_data: host array [n_caches] of device pointers to each cache's row storage.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA (launch failure). */
int mts_tbe_forward(const mts_tables* tables, int32_t B, const int64_t* indices,
                    const int64_t* offsets, int64_t N, int32_t pooling_mode,
                    const int32_t* slot_of_lookup, void* const* host_cache_data, int32_t n_caches,
                    float* out, int64_t out_stride, void* stream);

/* ---------------------------------------------------------------------------------------
 * Backward fused with row-wise Adagrad on the touched rows (Section 2.1.2: an Adagrad-type
 * optimizer with few states per row; Section 5.9: the backward pass aggregates gradients,
 * runs the optimizer and writes the rows back to whichever memory holds them).  For every
 * distinct row r of table t in the batch:
 *   g_r[d]  = sum over all occurrences i of r of s_i * grad_out[b(i), out_offset[t] + d]
 *             (s_i = 1, or 1 / bag length for mean pooling)
 *   m_r    += (1 / D_t) * sum_d g_r[d]^2
 *   W[r,d] -= lr * g_r[d] / (sqrt(m_r) + eps)      with the new m_r
 * One step per row per batch; other rows and states keep their bits.  fp32 arithmetic, fp16
 * rows stored with round-to-nearest-even.  The result is deterministic: occurrences are
 * summed in a fixed order that depends only on the batch.
 * Cached rows are updated in their slot and host_cache_dirty[c][slot] is set to 1; rows with
 * slot -1 are updated in the host tier directly.
 * workspace: device scratch of at least mts_tbe_backward_workspace_bytes(...) bytes, 256-byte
 * aligned, contents undefined on entry and exit.
 * uniq_rows_out / n_unique_out (both or neither; nullable, device int64 [N] / [1]): ascending
 * distinct linear row ids of the batch and their count.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE (too small), CUDA. */
size_t mts_tbe_backward_workspace_bytes(const mts_tables* tables, int32_t B, int64_t N);
int mts_tbe_backward_rowwise_adagrad(const mts_tables* tables, int32_t B, const int64_t* indices,
                                     const int64_t* offsets, int64_t N, int32_t pooling_mode,
                                     const float* grad_out, int64_t grad_stride, float lr, float eps,
                                     const int32_t* slot_of_lookup, void* const* host_cache_data,
                                     uint8_t* const* host_cache_dirty, int32_t n_caches,
                                     void* workspace, size_t workspace_bytes,
                                     int64_t* uniq_rows_out, int64_t* n_unique_out, void* stream);

/* The same backward in two calls, for callers that schedule the two halves themselves.
 * mts_tbe_backward_sort needs only the batch's indices: it writes into the workspace the lookups
 * ordered by row (and, if asked, the distinct rows), so it can run before the gradient exists,
 * for instance on another stream while the forward pass of the same batch runs (the paper's
 * pipeline likewise works on a batch's indices ahead of its training step, Section 5.7).
 * mts_tbe_backward_apply sums the gradients per row and applies the optimizer (Section 5.9); it
 * must be ordered after the matching mts_tbe_backward_sort (same stream, or an event), with the
 * same tables, B, offsets, N and workspace, whose contents nothing else may touch in between.
 * mts_tbe_backward_rowwise_adagrad is exactly sort followed by apply on one stream; arguments
 * and errors are the same as there. */
int mts_tbe_backward_sort(const mts_tables* tables, int32_t B, const int64_t* indices,
                          const int64_t* offsets, int64_t N, void* workspace, size_t workspace_bytes,
                          int64_t* uniq_rows_out, int64_t* n_unique_out, void* stream);
int mts_tbe_backward_apply(const mts_tables* tables, int32_t B, const int64_t* offsets, int64_t N,
                           int32_t pooling_mode, const float* grad_out, int64_t grad_stride, float lr,
                           float eps, const int32_t* slot_of_lookup, void* const* host_cache_data,
                           uint8_t* const* host_cache_dirty, int32_t n_caches, void* workspace,
                           size_t workspace_bytes, void* stream);

/* The same forward and gradient half of the backward with fp16 tensors on the dense side (the
 * paper's operators pool rows into an output that the dense network consumes, Section 2.1.1; it
 * does not fix that output's type).  out_f16 / grad_out_f16: device, IEEE binary16, [B, out_stride]
 * and [B, grad_stride] in elements, 16-byte aligned, strides multiples of 4.  The pooled sum is
 * accumulated in fp32 and rounded to nearest even once; the gradient is converted exactly to fp32
 * and everything after that is the arithmetic of the fp32 entry points.  Halves the bytes of the
 * output and, in the backward, of the gradient slices read once per lookup.  Other arguments,
 * ordering rules (mts_tbe_backward_sort first) and errors as for the fp32 entry points. */
int mts_tbe_forward_f16(const mts_tables* tables, int32_t B, const int64_t* indices,
                        const int64_t* offsets, int64_t N, int32_t pooling_mode,
                        const int32_t* slot_of_lookup, void* const* host_cache_data, int32_t n_caches,
                        void* out_f16, int64_t out_stride, void* stream);
/* The forward with a bfloat16 output (round to nearest even once, from the fp32 pooled value); layout and
 * alignment rules as for mts_tbe_forward_f16. */
int mts_tbe_forward_bf16(const mts_tables* tables, int32_t B, const int64_t* indices,
                         const int64_t* offsets, int64_t N, int32_t pooling_mode,
                         const int32_t* slot_of_lookup, void* const* host_cache_data, int32_t n_caches,
                         void* out_bf16, int64_t out_stride, void* stream);
int mts_tbe_backward_apply_f16(const mts_tables* tables, int32_t B, const int64_t* offsets, int64_t N,
                               int32_t pooling_mode, const void* grad_out_f16, int64_t grad_stride,
                               float lr, float eps, const int32_t* slot_of_lookup,
                               void* const* host_cache_data, uint8_t* const* host_cache_dirty,
                               int32_t n_caches, void* workspace, size_t workspace_bytes, void* stream);

/* The gradient half of the backward on lookups that are already ordered by row (Section 5.9; the
 * cache's tag lookup, Section 5.5.1, orders a batch's requests by row for its own purposes, and the
 * backward of the same batch can reuse that order instead of sorting again).
 *   sorted_rows[p] : linear row id (row_offset[t] + index) of the p-th lookup in ascending row order,
 *                    equal rows in ascending position in the batch,
 *   sorted_bag[p]  : that lookup's bag id t*B + b,
 *   sorted_slot[p] : its cache slot, or -1 = the row is updated in the host tier (ignored for tables that
 *                    live in HBM),
 * all device arrays of N entries covering every lookup of the batch — as written by
 * mts_cache_lookup_insert_tables calls that together cover all tables (every table cached).  The
 * arrays are trusted: rows outside the tables or an order that is not ascending give undefined
 * results.  grad_dtype: MTS_DTYPE_FP32 (float) or MTS_DTYPE_FP16 (binary16) gradient.  The
 * workspace is the one of mts_tbe_backward_workspace_bytes; mts_tbe_backward_sort is not needed.
 * Same arithmetic, summation order and errors as mts_tbe_backward_apply. */
int mts_tbe_backward_apply_presorted(const mts_tables* tables, int32_t B, const int64_t* offsets, int64_t N,
                                     int32_t pooling_mode, const void* grad_out, int32_t grad_dtype,
                                     int64_t grad_stride, float lr, float eps, const uint32_t* sorted_rows,
                                     const uint32_t* sorted_bag, const int32_t* sorted_slot,
                                     void* const* host_cache_data, uint8_t* const* host_cache_dirty,
                                     int32_t n_caches, void* workspace, size_t workspace_bytes, void* stream);

/* Backward without a workspace argument and without any allocation (the paper has no
 * counterpart; this exists for callers of this library that cannot allocate device memory).
 * Such callers are, for example, a training or serving loop embedded in a framework that
 * has reserved the whole device for its own pool, so that cudaMalloc fails or is forbidden by
 * policy; a step function that must not trigger the device-wide synchronisation an allocation
 * can imply; or plain C code that has no allocator to size the workspace with.
 * Same computation, arguments and errors as mts_tbe_backward_rowwise_adagrad, except that the
 * scratch memory is a fixed array of MTS_STATIC_SCRATCH_BYTES bytes inside the library image
 * (every GPU that loads the library holds that much until the process exits).
 *   - Limit: the batch must satisfy mts_tbe_backward_workspace_bytes(tables, B, N) <=
 *     MTS_STATIC_SCRATCH_BYTES (about 83,000 lookups at dim <= 1024, about 229,000 at dim <= 128);
 *     larger batches are rejected with MTS_ERR_CAPACITY before anything is launched.
 *   - The first call on each device looks up the array's device address (no allocation).  Make
 *     that first call outside of any stream capture.
 *   - The call itself calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls share the one array and it keeps the previous call's contents; the kernels
 *     write every scratch word before reading it, so nothing needs clearing, but two calls whose
 *     kernels overlap on the GPU (different streams, or different host threads) race on it.
 *     Issue these calls on one stream, or order them with events. */
#define MTS_STATIC_SCRATCH_BYTES (8u << 20)
int mts_tbe_backward_rowwise_adagrad_static(const mts_tables* tables, int32_t B, const int64_t* indices,
                                            const int64_t* offsets, int64_t N, int32_t pooling_mode,
                                            const float* grad_out, int64_t grad_stride, float lr, float eps,
                                            const int32_t* slot_of_lookup, void* const* host_cache_data,
                                            uint8_t* const* host_cache_dirty, int32_t n_caches,
                                            int64_t* uniq_rows_out, int64_t* n_unique_out, void* stream);

/* ---------------------------------------------------------------------------------------
 * Row cache (Section 5.3.1 cache class: row-granular cache memory, tags, per-entry timestamp
 * states; Section 5.5 GPU-managed cache kernels).  One level: HBM in front of pinned host
 * memory.  32-way set associative; set of a key = floor(((key * 0x9E3779B97F4A7C15) mod 2^64)
 * * num_sets / 2^64).  Keys are row ids relative to the cache's table group (tables of one
 * dim, contiguous in the host buffer): row `key` starts at element key * dim of
 * host_rows_mapped.
 * ------------------------------------------------------------------------------------- */
typedef struct mts_cache mts_cache;

/* Allocates tags, states, dirty bytes and num_sets*32 rows of `dim` elements in HBM.
 * key_space: number of rows of the table group the cache serves; keys are in [0, key_space).
 * lock_depth: a way stamped at step >= step - lock_depth is not evictable (Section 5.7: a
 * prefetched row is not evicted before its batch has trained).  Synchronous.
 * Errors: INVALID_ARG (num_sets < 1 or num_sets*32 >= 2^31, key_space >= 2^32 - 1, ways != 32),
 * UNSUPPORTED (dim > 1024), ALIGNMENT, CUDA. */
int mts_cache_create(mts_cache** out, int64_t num_sets, int64_t key_space, int32_t ways, int32_t dim,
                     int32_t dtype, int32_t policy, int32_t lock_depth);
int mts_cache_destroy(mts_cache* cache);
/* Reads and clears the cache's sticky device status word; synchronises `stream`.  Bit 0: a
 * bounded wait for a bulk copy of missed rows ran out (the kernel gave up instead of hanging; the
 * rows of that call are incomplete) — also reported as MTS_ERR_TIMEOUT.  Bit 1: a key outside
 * [0, key_space) was passed to mts_cache_lookup_insert; it was clamped into the range (the call
 * stays memory-safe, its result for that lookup is the clamped key's).  Bit 2: a miss list was
 * full and later missing keys were not inserted (see mts_cache_lookup_insert). */
int mts_cache_status(mts_cache* cache, int32_t* host_status, void* stream);
void* mts_cache_data(mts_cache* cache);        /* device [num_sets*32, dim] */
uint8_t* mts_cache_dirty(mts_cache* cache);    /* device [num_sets*32] */

/* Row keys of the lookups of tables [t_begin, t_end) relative to that group:
 * keys_out[i - lookup_begin] = row_offset[t] - row_offset[t_begin] + indices[i] for the n
 * lookups i in [lookup_begin, lookup_begin + n) = [offsets[t_begin*B], offsets[t_end*B]).
 * (The metadata consulted on every lookup, Section 5.8.) */
int mts_linearize_keys(const mts_tables* tables, int32_t t_begin, int32_t t_end, int32_t B,
                       const int64_t* indices, const int64_t* offsets, int64_t lookup_begin,
                       int64_t n, int64_t* keys_out, void* stream);

/* Tag/state lookup and replacement for one batch at time `step` (Sections 5.5.1, 5.5.2):
 *  1. every distinct key is probed in its set; a lookup is a hit iff its key was resident
 *     before the call;
 *  2. all hits are refreshed (timestamp = step);
 *  3. per set, the missing keys in ascending order take the set's evictable ways (free ways,
 *     then ways with timestamp < step - lock_depth) in (timestamp, way) order [LFU: (count, timestamp,
 *     way)]; a victim with a valid tag is appended to the evict list with its dirty byte, which
 *     is cleared; missing keys beyond the evictable ways are not inserted (slot -1, counted as
 *     overflow);
 *  4. slot = set * 32 + way; slot_of_lookup[i] = slot of keys[i].
 * miss list {key, slot} is ordered by (set, key); evict list {old key, slot, dirty} by (set,
 * order of the misses that displaced them).  list_capacity >= number of distinct keys is always
 * enough.  When the miss list is full, every further missing key is treated like one without an
 * evictable way: it is not inserted (slot -1), its victim keeps its way, and it is counted in
 * MTS_CNT_OVERFLOW and listed in overflow_keys; bit 2 of mts_cache_status records that this
 * happened.  MTS_CNT_INSERTED and MTS_CNT_EVICTED are the lengths of the lists.
 * overflow_keys (nullable, device int64 [list_capacity]): the keys counted in MTS_CNT_OVERFLOW, in no
 * particular order (see mts_cache_refetch_overflowed).
 * counters: device int64 [MTS_NUM_COUNTERS], overwritten.  `step` must not decrease between calls.
 * workspace: at least mts_cache_workspace_bytes(cache, N) bytes, 256-byte aligned.
 * Errors: INVALID_ARG, WORKSPACE, CUDA. */
size_t mts_cache_workspace_bytes(const mts_cache* cache, int64_t N);
int mts_cache_lookup_insert(mts_cache* cache, const int64_t* keys, int64_t N, int64_t step,
                            int32_t* slot_of_lookup, int64_t* miss_keys, int32_t* miss_slots,
                            int64_t* evict_keys, int32_t* evict_slots, uint8_t* evict_dirty,
                            int64_t* overflow_keys, int64_t list_capacity, int64_t* counters,
                            void* workspace, size_t workspace_bytes, void* stream);

/* The same tag/state lookup and replacement, fed from a batch's sparse input instead of a key
 * array (Sections 5.5.1, 5.5.2 and the per-table metadata of Section 5.8): the lookups of tables
 * [t_begin, t_end) — one cache's table group, whose rows must add up to the cache's key_space — are
 * positions [lookup_begin, lookup_begin + n) = [offsets[t_begin*B], offsets[t_end*B]) of `indices`;
 * the key of a lookup is its row id relative to the group.  Differences from mts_cache_lookup_insert:
 *   - slot_of_lookup is the batch-wide array (int32 [>= lookup_begin + n]); the call writes the
 *     entries of its own lookups, slot_of_lookup[i] for position i;
 *   - the overflow list has a capacity of its own (overflow_capacity; n is always enough);
 *   - sorted_rows_out, sorted_bag_out, sorted_slot_out (all NULL or all three; batch-wide device arrays):
 *     entries [lookup_begin, lookup_begin + n) receive the group's lookups ordered by row — linear row id
 *     row_offset[t] + index ascending, equal rows in ascending position — with the bag id t*B + b and the
 *     cache slot (or -1) of each.  Calls for all groups of a batch fill the arrays
 *     mts_tbe_backward_apply_presorted consumes.
 * An index outside [0, rows[t]) is clamped and raises bit 0 of mts_tables_status. */
int mts_cache_lookup_insert_tables(mts_cache* cache, const mts_tables* tables, int32_t t_begin, int32_t t_end,
                                   int32_t B, const int64_t* indices, const int64_t* offsets,
                                   int64_t lookup_begin, int64_t n, int64_t step, int32_t* slot_of_lookup,
                                   int64_t* miss_keys, int32_t* miss_slots, int64_t* evict_keys,
                                   int32_t* evict_slots, uint8_t* evict_dirty, int64_t list_capacity,
                                   int64_t* overflow_keys, int64_t overflow_capacity, int64_t* counters,
                                   uint32_t* sorted_rows_out, uint32_t* sorted_bag_out,
                                   int32_t* sorted_slot_out, void* workspace, size_t workspace_bytes,
                                   void* stream);

/* ---------------------------------------------------------------------------------------
 * Two cache levels, exclusive (Section 5.3.2: the faster memory is the first level, the larger one the
 * second, a row is in at most one of them; Section 5.5.4: both levels are looked up; first-level
 * misses that hit the second level and rows fetched from the lowest tier are promoted to the first
 * level; first-level LRU rows are evicted to the second level, second-level LRU rows to the lowest
 * tier).  Here the first level is a cache in HBM (mts_cache_create), the second level keeps its rows in
 * pinned host memory and its tags and states in HBM (mts_cache_create_host_level), and the lowest tier
 * ("store") is a device-visible host buffer of all rows, row `key` at element key * dim.
 * ------------------------------------------------------------------------------------- */

/* A cache level whose rows live in caller-owned pinned, mapped host memory: host_rows_mapped is the
 * device-visible address of [num_sets*32, dim] elements, 16-byte aligned; it must outlive the handle.
 * Other arguments and errors as for mts_cache_create. */
int mts_cache_create_host_level(mts_cache** out, int64_t num_sets, int64_t key_space, int32_t ways, int32_t dim,
                                int32_t dtype, int32_t policy, int32_t lock_depth, void* host_rows_mapped);

/* Tag/state lookup and replacement of both levels for one batch at time `step`:
 *  1. every distinct key is probed in both levels (state before the call);
 *  2. the first level is handled exactly as by mts_cache_lookup_insert (hits refreshed, missing keys take
 *     the evictable ways of their set, victims go to the first-level evict list, keys beyond the evictable
 *     ways get slot -1 and are served from the store); whether a key that misses the first level sits in
 *     the second level only says where its row comes from: fetch_src[k] = its second-level slot, or -1 =
 *     the store, for entry k of the fetch list {fetch_keys, fetch_slots} (the miss list of the first
 *     level); a promoted row keeps the dirty byte it had in the second level;
 *  3. every second-level hit leaves the second level: promoted, or — when it found no first-level way —
 *     listed in the drop list {key, second-level slot, dirty} (no particular order) so that the data
 *     movement writes a dirty row to the store before the batch reads it there;
 *  4. the first-level victims are inserted into the second level: per second-level set in ascending key
 *     order they take the set's evictable ways (free ways, then ways with timestamp < step - lock_depth of
 *     the second level, in (timestamp, way) order [LFU: (count, timestamp, way)]) and keep the timestamp,
 *     use count and dirty byte they had in the first level; ev1_dst[k] = second-level slot of entry k of
 *     the first-level evict list {ev1_keys, ev1_slots, ev1_dirty}, or -1 = no way left, the row goes to the
 *     store; displaced second-level rows form the second-level evict list {ev2_keys, ev2_slots, ev2_dirty}
 *     in (second-level set, key of the displacing row) order.
 * All lists are device arrays of list_capacity entries (the number of distinct keys is always enough);
 * counters2: device int64 [MTS_NUM_COUNTERS2].  The two levels must have the same dim, dtype and
 * key_space.  workspace: mts_cache2_workspace_bytes(l1, l2, N, list_capacity) bytes, 256-byte aligned.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, CUDA. */
size_t mts_cache2_workspace_bytes(const mts_cache* l1, const mts_cache* l2, int64_t N, int64_t list_capacity);
int mts_cache2_lookup_insert(mts_cache* l1, mts_cache* l2, const int64_t* keys, int64_t N, int64_t step,
                             int32_t* slot_of_lookup, int64_t* fetch_keys, int32_t* fetch_slots, int32_t* fetch_src,
                             int64_t* ev1_keys, int32_t* ev1_slots, uint8_t* ev1_dirty, int32_t* ev1_dst,
                             int64_t* ev2_keys, int32_t* ev2_slots, uint8_t* ev2_dirty, int64_t* drop_keys,
                             int32_t* drop_slots, uint8_t* drop_dirty, int64_t list_capacity, int64_t* counters2,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Data movement for one mts_cache2_lookup_insert result (Section 5.5.4), in an order that never reads a slot
 * after it was overwritten: dirty rows of the second-level evict list and of the drop list go to the store;
 * the rows of the fetch list are collected in fetch_staging (device, [list_capacity, dim]) from their
 * second-level slot or from the store; the first-level victims move to their second-level slot, or to the
 * store when they have none and are dirty; the collected rows enter their first-level slots.  All on
 * `stream`; list lengths are read from counters2 on the device.  mts_cache_flush on each level writes the
 * dirty rows of that level to the store. */
int mts_cache2_move(mts_cache* l1, mts_cache* l2, void* host_store_mapped, const int64_t* fetch_keys,
                    const int32_t* fetch_slots, const int32_t* fetch_src, const int64_t* ev1_keys,
                    const int32_t* ev1_slots, const uint8_t* ev1_dirty, const int32_t* ev1_dst,
                    const int64_t* ev2_keys, const int32_t* ev2_slots, const uint8_t* ev2_dirty,
                    const int64_t* drop_keys, const int32_t* drop_slots, const uint8_t* drop_dirty,
                    int64_t list_capacity, const int64_t* counters2, void* fetch_staging, void* stream);

/* Data movement for one lookup_insert result (Sections 5.5.3, 5.5.4): first the rows of dirty
 * victims are saved, slot -> evict_staging[k] (k = position in the evict list), then every
 * missed row is pulled from the host tier into its slot.  List lengths are read on the device
 * from `counters`.  evict_staging: device [list_capacity, dim]. */
int mts_cache_prefetch_misses(mts_cache* cache, const void* host_rows_mapped, const int64_t* miss_keys,
                              const int32_t* miss_slots, const int32_t* evict_slots,
                              const uint8_t* evict_dirty, int64_t list_capacity,
                              const int64_t* counters, void* evict_staging, void* stream);

/* The same data movement with the missed rows arriving through the copy engine instead of being read
 * from host memory by the kernels (Sections 5.5.3, 5.5.4; the paper's own lower tier is read by host
 * threads as well).  Rows read by SMs over the host link are slow (small requests) and slow down every
 * kernel that shares the GPU with them; a contiguous copy is neither.  Three steps, the middle one the
 * caller's: (1) mts_host_gather_rows, on the host: host_out[k] = host_rows[host_keys[k]] for k < n, with
 * `threads` host threads (plain memory, no GPU call; host_keys is a HOST copy of the first n entries of
 * the miss list; blocks until done; the rows must not be written meanwhile); (2) one contiguous copy of
 * host_out to a device buffer `fetched`; (3) mts_cache_place_fetched, on `stream` after that copy: saves
 * the dirty victims like mts_cache_prefetch_misses, then fetched[k] -> slot miss_slots[k] for every k
 * below min(MTS_CNT_INSERTED, list_capacity).  fetched: device [>= that many rows, dim], 16-byte aligned.
 * evict_staging NULL: the victims were saved already (mts_cache_save_victims), only place.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA. */
int mts_host_gather_rows(const void* host_rows, const int64_t* host_keys, int64_t n, int64_t row_bytes,
                         void* host_out, int32_t threads);
/* The write-back the same way (Section 5.5.4: evicted rows go back to the lower tier): after
 * mts_cache_place_fetched the dirty victims sit in evict_staging in list order; the caller copies the first
 * MTS_CNT_EVICTED rows of it, with evict_keys and evict_dirty, to host buffers (one contiguous copy each) and
 * calls this on the host: host_rows[host_keys[k]] = host_in[k] for every k < n with host_mask[k] != 0
 * (host_mask NULL = all), with `threads` host threads.  Plain memory, no GPU call; blocks until done. */
int mts_host_scatter_rows(void* host_rows, const int64_t* host_keys, const uint8_t* host_mask, int64_t n,
                          int64_t row_bytes, const void* host_in, int32_t threads);
int mts_cache_place_fetched(mts_cache* cache, const void* fetched, const int32_t* miss_slots,
                            const int32_t* evict_slots, const uint8_t* evict_dirty, int64_t list_capacity,
                            const int64_t* counters, void* evict_staging, void* stream);
/* The first half of mts_cache_place_fetched alone (Section 5.5.4): the rows of the dirty victims, slot ->
 * evict_staging[k].  A victim's row is final once the lookup that chose it has run (no batch in flight may
 * use it), so the caller can save and copy the victims out on a second stream while the host still gathers
 * the missed rows; mts_cache_place_fetched with evict_staging = NULL then only places (the caller orders it
 * after this call, e.g. with an event).  Errors: INVALID_ARG, ALIGNMENT, CUDA. */
int mts_cache_save_victims(mts_cache* cache, const int32_t* evict_slots, const uint8_t* evict_dirty,
                           int64_t list_capacity, const int64_t* counters, void* evict_staging, void* stream);

/* The copy-engine data movement of one cache run by a host thread of the library (Sections 5.5.3, 5.5.4: rows
 * between the cache and the lower tier; Section 5.7: ahead of the training of their batch).  A mover owns one
 * thread, pinned host buffers for `n_contexts` batches in flight (keys and rows, both directions; they start at
 * first_buffer_bytes per list and grow up to max_buffer_bytes when a batch's lists are longer) and one device
 * buffer.  Per submitted batch, in submission order, the thread: waits for the event `tag_done` (recorded by
 * the caller after the batch's mts_cache_lookup_insert* AND after a copy of its `counters` to the pinned
 * `host_counters`); starts the miss keys on their way to the host on `copy_stream`; saves the victims
 * (mts_cache_save_victims) and copies them, their keys and dirty bytes out on `save_stream`; puts the previous
 * batch's victims into their host rows (mts_host_scatter_rows: a row evicted by one batch may be missed by the
 * next); gathers the missed rows (mts_host_gather_rows); enqueues their copy and mts_cache_place_fetched on
 * `move_stream`; records the batch's "moved" event there.  It does not wait for the copy of the rows.  Lists
 * longer than the buffers may grow to are moved by mts_cache_prefetch_misses / mts_cache_writeback_evicted
 * on `move_stream` instead (the thread then waits for them).
 * host_rows: base of the cache's keys in the host tier (pinned, device-visible; row k at k * row_bytes).
 * The job's device pointers are the arguments and results of the batch's mts_cache_lookup_insert*; they and
 * evict_staging must stay untouched until the batch has moved; one evict_staging may serve all batches of a
 * mover.  The three streams must not be the legacy default stream's aliases of one another's work in a way
 * that makes them wait for the caller's later work (the thread enqueues on them while the caller runs).
 * mts_mover_submit returns at once.  mts_mover_stream_wait_moved blocks the calling host thread until the
 * batch's "moved" event has been recorded (not until it has completed) and makes `stream` wait for it.
 * mts_mover_drain waits until every submitted batch has been enqueued and puts the last victims into their
 * rows (call it with the streams still alive; afterwards the host tier is current once move_stream and
 * save_stream are idle).  mts_mover_stats: seconds gathering, bytes gathered, seconds scattering, bytes
 * scattered, batches moved by kernels.  A failure in the thread is returned by every later call.
 * Errors: INVALID_ARG, CUDA. */
typedef struct mts_mover mts_mover;
typedef struct {
  const int64_t* miss_keys;      /* device lists of the batch (mts_cache_lookup_insert*) */
  const int32_t* miss_slots;
  const int64_t* evict_keys;
  const int32_t* evict_slots;
  const uint8_t* evict_dirty;
  int64_t list_capacity;
  const int64_t* counters;       /* device [MTS_NUM_COUNTERS] */
  const int64_t* host_counters;  /* pinned copy of `counters`, complete when tag_done is */
  void* evict_staging;           /* device [list_capacity, dim] */
  void* tag_done;                /* cudaEvent_t */
  void* move_stream;             /* cudaStream_t: copy of the gathered rows, placing kernel, "moved" event */
  void* save_stream;             /* cudaStream_t: victims saved and copied out */
  void* copy_stream;             /* cudaStream_t: miss keys to the host */
} mts_move_job;
int mts_mover_create(mts_mover** out, mts_cache* cache, void* host_rows, int64_t row_bytes, int32_t threads,
                     int32_t n_contexts, int64_t first_buffer_bytes, int64_t max_buffer_bytes);
int mts_mover_submit(mts_mover* mover, const mts_move_job* job);
int mts_mover_stream_wait_moved(mts_mover* mover, int64_t job_index, void* stream);
int mts_mover_drain(mts_mover* mover);
int mts_mover_stats(mts_mover* mover, double* out5);
int mts_mover_destroy(mts_mover* mover);

/* Evicted dirty rows go back to the host tier: evict_staging[k] -> host row evict_keys[k]. */
int mts_cache_writeback_evicted(mts_cache* cache, void* host_rows_mapped, const int64_t* evict_keys,
                                const uint8_t* evict_dirty, int64_t list_capacity,
                                const int64_t* counters, const void* evict_staging, void* stream);

/* Support for running the data movement of a batch while earlier batches still train (Section 5.7).
 * A key that overflowed in batch u is read and updated in the host tier by batch u's forward and
 * backward; if a later batch t inserts that key and its data movement runs before batch u's backward,
 * the copy it takes of the host row is stale.  Call this after batch u's backward and batch t's data
 * movement with batch u's overflow list and counters: every listed key whose row was inserted by the
 * lookup_insert call with step `placed_step` (batch t's; -1 = whichever call inserted it) gets its row
 * copied from the host tier again.  The cache remembers the step at which each resident row was inserted,
 * apart from its timestamp, so the call leaves alone both a row inserted earlier (it has been updated in
 * its slot since, the host copy is the older one) and a key that a tag step running further ahead has
 * inserted meanwhile (that slot still holds its victim's row until that batch's data movement).
 * list_capacity: capacity of the overflow list.  A no-op when the steps run one after the other. */
int mts_cache_refetch_overflowed(mts_cache* cache, const void* host_rows_mapped, const int64_t* overflow_keys,
                                 int64_t list_capacity, const int64_t* counters, int64_t placed_step,
                                 void* stream);

/* Writes every dirty resident row to the host tier and clears its dirty byte. */
int mts_cache_flush(mts_cache* cache, void* host_rows_mapped, void* stream);

/* Copies tags (int64 [sets*32], -1 = free), timestamps (int64, -1 = free), use counts (int64)
 * and dirty bytes to caller buffers (device); any pointer may be NULL. */
int mts_cache_export_state(mts_cache* cache, int64_t* tags, int64_t* timestamps, int64_t* counts,
                           uint8_t* dirty, void* stream);

/* ---------------------------------------------------------------------------------------
 * Table placement (Section 5.6, Eq. 6).  Chooses for every table the memory that holds it — HBM
 * (placement 0, cache id -1 in mts_table_desc) or the host tier behind a cache (placement 1) — so that
 * each table is in one memory, the HBM tables fit hbm_budget_bytes, and the lookup time per sample
 *   sum over tables of host_bytes_per_sample[t] / (bw_hbm or bw_host),  bytes_per_sample = D * L * p,
 * is minimal (Eq. 6 for one GPU).  Exact (branch and bound) unless the search meets its node limit, in
 * which case the best placement found is returned and *optimal_out is 0.  All pointers are HOST pointers;
 * time_out and optimal_out may be NULL; bandwidths in bytes per second.  No GPU call.
 * Errors: INVALID_ARG. */
int mts_place_tables(int32_t T, const int64_t* host_size_bytes, const double* host_bytes_per_sample,
                     int64_t hbm_budget_bytes, double bw_hbm, double bw_host, int32_t* host_placement_out,
                     double* time_out, int32_t* optimal_out);

/* The inverse of mts_cache_export_state, for resuming a run (the paper keeps the cache's tags and states in
 * HBM, Section 5.6, and has no checkpoint format of its own): sets tags (-1 = free way), timestamps, use
 * counts and dirty bytes from device arrays of num_sets*32 entries and fills the slot of every resident tag
 * with its row from the host tier.  The rows themselves are not part of the exported state, so export after
 * mts_cache_flush: then every row of the host tier is current and every dirty byte 0.  The step of the next
 * mts_cache_lookup_insert must be larger than every imported timestamp.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA. */
int mts_cache_import_state(mts_cache* cache, const int64_t* tags, const int64_t* timestamps, const int64_t* counts,
                           const uint8_t* dirty, const void* host_rows_mapped, void* stream);

/* How many times mts_cache_prefetch_misses polls for a tile of missed rows before it gives up (default and
 * maximum 2^22; the paper has no counterpart).  When the polls run out the kernel raises bit 0 of
 * mts_cache_status, waits (bounded by the maximum) until its copies in flight have landed and returns; the
 * rows of that call are incomplete, the call can simply be repeated.  0 makes every call give up at once:
 * for testing the error path without hanging anything. */
int mts_cache_set_fetch_wait_limit(mts_cache* cache, int64_t polls);

#ifdef __cplusplus
}
#endif
#endif /* MTRAINS_B200_H_ */
