// Software-managed row cache in HBM in front of pinned host memory: the cache class of
// Section 5.3.1 (row-granular data, tags, per-entry timestamp states) and the GPU cache
// kernels of Section 5.5 (tag/state lookup, LRU/LFU replacement, data lookup/update, data
// movement), one level deep.
//
// lookup_insert, all on the caller's stream and without host synchronisation:
//   keys -> stable sort by key -> distinct keys (U, on the device) -> set index of each
//   distinct key -> stable sort of the distinct keys by set (keeps ascending key inside a
//   set) -> one warp per touched set: probe (lane = way), refresh hits, order the evictable
//   ways, hand them to the set's misses -> ordered compaction of the miss and evict lists
//   (prefix sums, no atomics on list positions) -> slot of every lookup.
// Every decision is a pure function of the cache state and the batch, so the slots, lists and
// counters are reproducible bit for bit.
#include <algorithm>
#include <cstring>
#include <thread>
#include <atomic>
#include <condition_variable>
#include <functional>
#include <mutex>
#include <vector>
#if defined(__SSE2__)
#include <emmintrin.h>
#endif

#include "common.cuh"

struct mts_cache {
  int64_t S = 0;
  int64_t key_space = 0;
  int32_t ways = MTS_CACHE_WAYS;
  int32_t dim = 0, dtype = 0, elem_bytes = 4, policy = 0, lock_depth = 0;
  int32_t row_bytes = 0;
  int32_t sm_count = 148;
  uint32_t* tags = nullptr;      // [S*32]  0xffffffff = free
  int32_t* ts = nullptr;         // [S*32]  -1 = free
  int32_t* placed = nullptr;     // [S*32]  step at which the way's current row was inserted (-1 = free)
  uint32_t* freq = nullptr;      // [S*32]
  uint8_t* dirty = nullptr;      // [S*32]
  char* data = nullptr;          // [S*32, row_bytes]  HBM, or pinned host memory of the caller (a second level)
  bool owns_data = true;
  uint32_t fetch_wait_limit = 1u << 22;   // polls the bulk-copy fetch waits for a tile before it gives up
  int32_t* d_status = nullptr;   // sticky status bits (bit 0: a bounded wait on a bulk copy ran out)
};

namespace mts {

constexpr uint32_t FREE_TAG = 0xffffffffu;
constexpr int CACHE_THREADS = 256;
constexpr int CACHE_STATUS_FETCH_TIMEOUT = 1;   // a bounded wait on a bulk copy ran out
constexpr int CACHE_STATUS_KEY_RANGE = 2;       // a key outside [0, key_space) was clamped
constexpr int CACHE_STATUS_LIST_CUT = 4;        // more placements than list_capacity: the surplus was not inserted

__device__ __forceinline__ uint32_t set_of_key(uint32_t key, uint64_t S) {
  const uint64_t x = (uint64_t)key * 0x9E3779B97F4A7C15ull;
  return (uint32_t)__umul64hi(x, S);
}

__global__ void cache_init_state(uint32_t* tags, int32_t* ts, int32_t* placed, uint32_t* freq, uint8_t* dirty, int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    tags[i] = FREE_TAG; ts[i] = -1; placed[i] = -1; freq[i] = 0; dirty[i] = 0;
  }
}

// A key outside [0, key_space) is clamped into the range (never sorted or probed as it is: the
// sort only looks at the bits of key_space) and raises status bit 1.
__global__ void cache_prepare_keys(const int64_t* __restrict__ keys, int64_t n, const uint32_t* __restrict__ n_dev,
                                   int64_t key_space,
                                   uint32_t* __restrict__ k32, uint32_t* __restrict__ pos,
                                   int64_t* __restrict__ counters, uint32_t* __restrict__ overflow_cursor,
                                   int32_t* __restrict__ status) {
  if (n_dev != nullptr) n = min(n, (int64_t)*n_dev);      // the number of keys is only known on the device
  const int64_t i0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i0 < MTS_NUM_COUNTERS) counters[i0] = i0 == MTS_CNT_LOOKUPS ? n : 0;
  if (i0 == 0) *overflow_cursor = 0u;
  for (int64_t i = i0; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t k = keys[i];
    if (k < 0 || k >= key_space) {
      atomicOr(status, CACHE_STATUS_KEY_RANGE);
      k = k < 0 ? 0 : key_space - 1;
    }
    k32[i] = (uint32_t)k;
    pos[i] = (uint32_t)i;
  }
}

// The same preparation straight from a batch's sparse input, for the lookups of the tables
// [t_begin, t_end) (8 lanes per bag): the sort key is the linear row id row_offset[t] + index, the
// value the lookup's position in the batch; bag_of_lookup (nullable, indexed by position - lookup_begin)
// receives every lookup's bag id.
__global__ void cache_prepare_from_indices(const TableMeta* __restrict__ meta, int32_t t_begin, int64_t n_bags,
                                           int32_t B, const int64_t* __restrict__ indices,
                                           const int64_t* __restrict__ offsets, int64_t lookup_begin, int64_t n,
                                           uint32_t* __restrict__ k32, uint32_t* __restrict__ pos,
                                           uint32_t* __restrict__ bag_of_lookup, int64_t* __restrict__ counters,
                                           uint32_t* __restrict__ overflow_cursor, int32_t* __restrict__ status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid < MTS_NUM_COUNTERS) counters[gid] = gid == MTS_CNT_LOOKUPS ? n : 0;
  if (gid == 0) *overflow_cursor = 0u;
  const int64_t gb = gid / 8;
  if (gb >= n_bags) return;
  const int sub = (int)(gid % 8);
  const int64_t bag = (int64_t)t_begin * B + gb;
  const int32_t t = (int32_t)(bag / B);
  const int64_t rows = meta[t].rows;
  const int64_t roff = meta[t].row_offset;
  const int64_t i1 = offsets[bag + 1];
  for (int64_t i = offsets[bag] + sub; i < i1; i += 8) {
    const int64_t o = i - lookup_begin;
    if (o >= 0 && o < n) {
      k32[o] = (uint32_t)(roff + clamp_index(indices[i], rows, status));
      pos[o] = (uint32_t)i;
      if (bag_of_lookup != nullptr) bag_of_lookup[o] = (uint32_t)bag;
    }
  }
}

// Exclusive scan of one value per thread over a 256-thread block (`sh`: 9 words of shared memory).
__device__ __forceinline__ uint32_t block_scan_256(uint32_t v, uint32_t* sh, uint32_t* total) {
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
    uint32_t w = lane < 8 ? sh[lane] : 0u;
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    if (lane < 8) sh[lane] = winc - w;
    if (lane == 7) sh[8] = winc;
  }
  __syncthreads();
  const uint32_t res = sh[warp] + inc - v;
  *total = sh[8];
  __syncthreads();
  return res;
}

// Rows that are inserted with a history instead of as fresh rows (first-level victims entering a second
// level): timestamp, use count and dirty byte per entry of the source list; all null = fresh rows.
struct InsertAttrs {
  const int32_t* ts = nullptr;
  const uint32_t* freq = nullptr;
  const uint8_t* dirty = nullptr;
};

// The second level as the first level's tag step sees it.
struct SecondLevel {
  uint32_t* tags = nullptr;
  int32_t* ts = nullptr;
  int32_t* placed = nullptr;
  uint32_t* freq = nullptr;
  uint8_t* dirty = nullptr;
  uint64_t S = 0;
};

// Probe of every distinct key against the state before the call, 32 keys per warp at a time: each lane
// describes one key (value, multiplicity, set), then the warp walks the 32 keys and compares the 32 tags of
// each key's set (lane = way).  A hit is refreshed here (timestamp, use count) and gets its slot; a key
// that misses is only flagged.  Block b owns a contiguous range of keys and counts its misses, so that
// the misses can be compacted in key order afterwards.  Entries u >= U are not touched.
constexpr int PROBE_BLOCKS = 1024;

__device__ __forceinline__ int64_t probe_per_block(int64_t n, int G) {
  const int64_t per = (n + G - 1) / G;
  return (per + CACHE_THREADS - 1) / CACHE_THREADS * CACHE_THREADS;
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_probe_hits(const uint32_t* __restrict__ sorted_keys, uint32_t key_base,
                 const uint32_t* __restrict__ seg_start, const uint32_t* __restrict__ n_unique, uint64_t S,
                 const uint32_t* __restrict__ tags, int32_t* __restrict__ ts, uint32_t* __restrict__ freq,
                 int32_t step, uint32_t* __restrict__ ukey, uint32_t* __restrict__ mult,
                 int32_t* __restrict__ slot_of_uniq, uint8_t* __restrict__ missed,
                 uint32_t* __restrict__ cnt_missed, unsigned long long* __restrict__ counters,
                 const uint32_t* __restrict__ sorted_pos, InsertAttrs attrs, int32_t* __restrict__ ins_ts,
                 uint8_t* __restrict__ ins_dirty) {
  __shared__ uint32_t sh[9];
  const int lane = threadIdx.x & 31;
  const int64_t U = *n_unique;
  const int64_t per = probe_per_block(U, gridDim.x);
  const int64_t begin = (int64_t)blockIdx.x * per, end = min(U, begin + per);
  unsigned long long c_hit_lookups = 0, c_uhits = 0;
  uint32_t my_missed = 0;
  for (int64_t base = begin + (threadIdx.x & ~31); base < end; base += CACHE_THREADS) {
    const int64_t u = base + lane;
    const bool valid = u < end;
    uint32_t k = 0, mu = 0, set = 0;
    if (valid) {
      const uint32_t s0 = seg_start[u];
      k = sorted_keys[s0] - key_base;
      mu = seg_start[u + 1] - s0;
      set = set_of_key(k, S);
      if (attrs.ts != nullptr) {
        // a row that arrives with a history: the entry it came from (position in the source list)
        const uint32_t e = sorted_pos[s0];
        mu = attrs.freq[e];
        ins_ts[u] = attrs.ts[e];
        ins_dirty[u] = attrs.dirty[e];
      }
      ukey[u] = k;
      mult[u] = mu;
    }
    const int m = (int)min((int64_t)32, end - base);
    int32_t my_slot = -1;
#pragma unroll 8
    for (int q = 0; q < 32; ++q) {
      if (q < m) {
        const uint32_t kq = __shfl_sync(0xffffffffu, k, q);
        const uint32_t sq = __shfl_sync(0xffffffffu, set, q);
        const uint32_t tag = tags[(int64_t)sq * 32 + lane];
        const uint32_t hit = __ballot_sync(0xffffffffu, tag == kq);      // a free way holds no valid key
        if (hit && lane == q) my_slot = (int32_t)((int64_t)sq * 32 + __ffs(hit) - 1);
      }
    }
    if (valid) {
      if (my_slot >= 0) {
        ts[my_slot] = step;
        freq[my_slot] += mu;
        c_hit_lookups += mu;
        c_uhits += 1;
        slot_of_uniq[u] = my_slot;
        missed[u] = 0;
      } else {
        missed[u] = 1;
        my_missed += 1;
      }
    }
  }
  uint32_t total;
  block_scan_256(my_missed, sh, &total);
  if (threadIdx.x == 0) cnt_missed[blockIdx.x] = total;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    c_hit_lookups += __shfl_xor_sync(0xffffffffu, c_hit_lookups, o);
    c_uhits += __shfl_xor_sync(0xffffffffu, c_uhits, o);
  }
  if (lane == 0) {
    if (c_hit_lookups) atomicAdd(&counters[MTS_CNT_HIT_LOOKUPS], c_hit_lookups);
    if (c_uhits) atomicAdd(&counters[MTS_CNT_UNIQUE_HITS], c_uhits);
  }
}

// Exclusive prefix over the blocks' miss counts (in place); *n_missed = their sum.
__global__ void __launch_bounds__(CACHE_THREADS)
cache_scan_missed(uint32_t* __restrict__ cnt_missed, int G, uint32_t* __restrict__ n_missed) {
  __shared__ uint32_t sh[9];
  constexpr int PER = PROBE_BLOCKS / CACHE_THREADS;
  const int j0 = threadIdx.x * PER;
  uint32_t v[PER];
  uint32_t s = 0;
#pragma unroll
  for (int k = 0; k < PER; ++k) { v[k] = j0 + k < G ? cnt_missed[j0 + k] : 0u; s += v[k]; }
  uint32_t total;
  uint32_t ex = block_scan_256(s, sh, &total);
#pragma unroll
  for (int k = 0; k < PER; ++k) { if (j0 + k < G) cnt_missed[j0 + k] = ex; ex += v[k]; }
  if (threadIdx.x == 0) *n_missed = total;
}

// The missing keys in ascending key order: (set, index among the distinct keys), the input of the sort by set.
__global__ void __launch_bounds__(CACHE_THREADS)
cache_compact_missed(const uint8_t* __restrict__ missed, const uint32_t* __restrict__ ukey,
                     const uint32_t* __restrict__ n_unique, uint64_t S, const uint32_t* __restrict__ base_missed,
                     uint32_t* __restrict__ set_keys, uint32_t* __restrict__ set_vals) {
  __shared__ uint32_t sh[9];
  const int64_t U = *n_unique;
  const int64_t per = probe_per_block(U, gridDim.x);
  const int64_t begin = (int64_t)blockIdx.x * per, end = min(U, begin + per);
  uint32_t at = base_missed[blockIdx.x];
  for (int64_t t0 = begin; t0 < end; t0 += CACHE_THREADS) {
    const int64_t u = t0 + threadIdx.x;
    const bool miss = u < end && missed[u] != 0;
    uint32_t total;
    const uint32_t p = block_scan_256(miss ? 1u : 0u, sh, &total);
    if (miss) {
      set_keys[at + p] = set_of_key(ukey[u], S);
      set_vals[at + p] = (uint32_t)u;
    }
    at += total;
  }
}

// Second level: where does every key that missed the first level sit there (slot, or -1)?  Read only; 32 of
// the compacted misses per warp at a time, lane = way in the walk.
__global__ void __launch_bounds__(CACHE_THREADS)
cache_probe_second_level(const uint32_t* __restrict__ miss_uidx, const uint32_t* __restrict__ n_missed,
                         const uint32_t* __restrict__ ukey, const uint32_t* __restrict__ mult, SecondLevel l2,
                         int32_t* __restrict__ l2slot_of_uniq, unsigned long long* __restrict__ counters2) {
  const int lane = threadIdx.x & 31;
  const int64_t M = *n_missed;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  unsigned long long c_lookups = 0, c_keys = 0;
  for (int64_t base = warp0 * 32; base < M; base += nwarps * 32) {
    const int64_t j = base + lane;
    uint32_t u = 0, k = 0, set = 0;
    if (j < M) { u = miss_uidx[j]; k = ukey[u]; set = set_of_key(k, l2.S); }
    const int m = (int)min((int64_t)32, M - base);
    int32_t my_slot = -1;
#pragma unroll 8
    for (int q = 0; q < 32; ++q) {
      if (q < m) {
        const uint32_t kq = __shfl_sync(0xffffffffu, k, q);
        const uint32_t sq = __shfl_sync(0xffffffffu, set, q);
        const uint32_t hit = __ballot_sync(0xffffffffu, l2.tags[(int64_t)sq * 32 + lane] == kq);
        if (hit && lane == q) my_slot = (int32_t)((int64_t)sq * 32 + __ffs(hit) - 1);
      }
    }
    if (j < M) {
      l2slot_of_uniq[u] = my_slot;
      if (my_slot >= 0) { c_lookups += mult[u]; c_keys += 1; }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    c_lookups += __shfl_xor_sync(0xffffffffu, c_lookups, o);
    c_keys += __shfl_xor_sync(0xffffffffu, c_keys, o);
  }
  if (lane == 0) {
    if (c_lookups) atomicAdd(&counters2[MTS_CNT2_L2_HIT_LOOKUPS], c_lookups);
    if (c_keys) atomicAdd(&counters2[MTS_CNT2_L2_UNIQUE_HITS], c_keys);
  }
}

// One warp per touched set; lane = way.  The walk is a chain of dependent loads per set, so the kernel lives
// on resident warps: the register allocation is bounded for four blocks per SM.
__global__ void __launch_bounds__(CACHE_THREADS, 4)
cache_probe_replace(const uint32_t* __restrict__ set_sorted,      // set of member j (ascending)
                    const uint32_t* __restrict__ member_uidx,     // distinct-key index of member j
                    const uint32_t* __restrict__ sseg_start, const uint32_t* __restrict__ n_sets,
                    const uint32_t* __restrict__ ukey, const uint32_t* __restrict__ mult,
                    uint32_t* __restrict__ tags, int32_t* __restrict__ ts, int32_t* __restrict__ placed_at,
                    uint32_t* __restrict__ freq,
                    uint8_t* __restrict__ dirty, int32_t step, int32_t lock_depth, int32_t policy,
                    int32_t* __restrict__ slot_of_uniq, uint8_t* __restrict__ member_flag,
                    uint32_t* __restrict__ member_old_key, uint8_t* __restrict__ member_old_dirty,
                    int32_t* __restrict__ member_old_ts, uint32_t* __restrict__ member_old_freq,
                    int32_t* __restrict__ member_old_placed,
                    int32_t* __restrict__ member_slot, unsigned long long* __restrict__ counters,
                    const int32_t* __restrict__ ins_ts, const uint8_t* __restrict__ ins_dirty,
                    unsigned long long* __restrict__ overflow_dirty_count) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const uint32_t NS = *n_sets;
  unsigned long long c_hit_lookups = 0, c_uhits = 0, c_dirty = 0, c_overflow = 0, c_overflow_dirty = 0;
  // The state of the warp's next set is requested before the current set is worked on (the sets of one warp
  // are different sets, so nothing written below is read here): the chain set bounds -> set -> state of
  // one set overlaps the work on the one before it.
  uint32_t n_j0 = 0, n_j1 = 0, n_set = 0, n_tag = 0, n_cnt = 0;
  int32_t n_stamp = 0, n_plc = 0;
  auto request = [&](int64_t s_i) {
    if (s_i < NS) {
      n_j0 = sseg_start[s_i]; n_j1 = sseg_start[s_i + 1];
      n_set = set_sorted[n_j0];
      const int64_t at = (int64_t)n_set * 32 + lane;
      n_tag = tags[at]; n_stamp = ts[at]; n_cnt = freq[at]; n_plc = placed_at[at];
    }
  };
  request(warp0);
  for (int64_t si = warp0; si < NS; si += nwarps) {
    const uint32_t j0 = n_j0, j1 = n_j1;
    const uint32_t set = n_set;
    const int64_t slot0 = (int64_t)set * 32;
    uint32_t tag = n_tag;
    int32_t stamp = n_stamp;
    uint32_t cnt = n_cnt;
    int32_t plc = n_plc;
    request(si + nwarps);
    bool touched = false;
    // pass 1: probe every member against the state before the call, refresh the hits
    for (uint32_t jb = j0; jb < j1; jb += 32) {
      const uint32_t j = jb + lane;
      uint32_t u = 0, k = 0, mu = 0;
      if (j < j1) { u = member_uidx[j]; k = ukey[u]; mu = mult[u]; }
      const int m = (int)min(32u, j1 - jb);
      uint8_t my_flag = 0;
      int32_t my_slot = -1;
      for (int q = 0; q < m; ++q) {
        const uint32_t kq = __shfl_sync(0xffffffffu, k, q);
        const uint32_t mq = __shfl_sync(0xffffffffu, mu, q);
        const uint32_t hit = __ballot_sync(0xffffffffu, tag == kq && tag != FREE_TAG);
        if (hit) {
          const int way = __ffs(hit) - 1;
          if (lane == way) { stamp = step; cnt += mq; touched = true; }
          if (lane == q) { my_flag = 3; my_slot = (int32_t)(slot0 + way); }
          c_hit_lookups += mq;
          c_uhits += 1;
        }
      }
      if (j < j1) {
        member_flag[j] = my_flag;          // 3 = hit, rewritten below for misses
        member_slot[j] = my_slot;
      }
    }
    // candidates after the refresh: ways outside the lock window, free ways first by their -1 stamp
    const bool cand = tag == FREE_TAG || stamp < step - lock_depth;
    const uint32_t cand_mask = __ballot_sync(0xffffffffu, cand);
    const int ncand = __popc(cand_mask);
    int rank = 0;
    for (int q = 0; q < 32; ++q) {
      const int32_t sq = __shfl_sync(0xffffffffu, stamp, q);
      const uint32_t fq = __shfl_sync(0xffffffffu, cnt, q);
      if ((cand_mask >> q) & 1u) {
        bool before;
        if (policy == MTS_POLICY_LFU && fq != cnt) before = fq < cnt;
        else if (sq != stamp) before = sq < stamp;
        else before = q < lane;
        rank += before ? 1 : 0;
      }
    }
    // pass 2: the k-th missing key (ascending) takes the k-th candidate
    int placed = 0;
    uint8_t dirty_reg = 0;
    bool dirty_loaded = false;
    for (uint32_t jb = j0; jb < j1; jb += 32) {
      const uint32_t j = jb + lane;
      uint32_t u = 0, k = 0, mu = 0;
      uint8_t fl = 3;
      int32_t its = step;              // state a placed row starts with: fresh, or the history it arrives with
      uint32_t idr = 0;
      if (j < j1) {
        u = member_uidx[j]; k = ukey[u]; mu = mult[u]; fl = member_flag[j];
        if (ins_ts != nullptr) { its = ins_ts[u]; idr = ins_dirty[u]; }
      }
      const int m = (int)min(32u, j1 - jb);
      const uint32_t miss_mask = __ballot_sync(0xffffffffu, j < j1 && fl == 0);
      uint8_t my_flag = fl;
      int32_t my_slot = -1;
      uint32_t my_old = FREE_TAG;
      uint8_t my_old_dirty = 0;
      int32_t my_old_ts = -1, my_old_placed = -1;
      uint32_t my_old_freq = 0;
      for (int q = 0; q < m; ++q) {
        if (!((miss_mask >> q) & 1u)) continue;
        const uint32_t kq = __shfl_sync(0xffffffffu, k, q);
        const uint32_t mq = __shfl_sync(0xffffffffu, mu, q);
        const int32_t tsq = __shfl_sync(0xffffffffu, its, q);
        const uint32_t drq = __shfl_sync(0xffffffffu, idr, q);
        if (placed < ncand) {
          const uint32_t sel = __ballot_sync(0xffffffffu, cand && rank == placed);
          const int way = __ffs(sel) - 1;
          uint32_t old_tag = 0;
          uint8_t old_dirty = 0;
          int32_t old_ts = -1, old_placed = -1;
          uint32_t old_freq = 0;
          if (lane == way) {
            old_tag = tag; old_ts = stamp; old_freq = cnt; old_placed = plc;
            if (!dirty_loaded) { dirty_reg = dirty[slot0 + lane]; dirty_loaded = true; }
            old_dirty = tag != FREE_TAG ? dirty_reg : 0;
            tag = kq; stamp = tsq; cnt = mq; plc = step; dirty_reg = (uint8_t)drq; touched = true;
          }
          old_tag = __shfl_sync(0xffffffffu, old_tag, way);
          old_placed = __shfl_sync(0xffffffffu, old_placed, way);
          old_dirty = (uint8_t)__shfl_sync(0xffffffffu, (uint32_t)old_dirty, way);
          old_ts = __shfl_sync(0xffffffffu, old_ts, way);
          old_freq = __shfl_sync(0xffffffffu, old_freq, way);
          if (lane == q) {
            my_flag = 1; my_slot = (int32_t)(slot0 + way); my_old = old_tag; my_old_dirty = old_dirty;
            my_old_ts = old_ts; my_old_freq = old_freq; my_old_placed = old_placed;
          }
          if (old_tag != FREE_TAG && old_dirty) c_dirty += 1;
          ++placed;
        } else {
          if (lane == q) { my_flag = 2; my_slot = -1; }
          c_overflow += 1;
          c_overflow_dirty += drq ? 1 : 0;
        }
      }
      if (j < j1 && fl == 0) {
        member_flag[j] = my_flag;          // 1 = placed, 2 = overflow
        member_slot[j] = my_slot;
        member_old_key[j] = my_old;
        member_old_dirty[j] = my_old_dirty;
        member_old_ts[j] = my_old_ts;
        member_old_freq[j] = my_old_freq;
        member_old_placed[j] = my_old_placed;
      }
      if (j < j1) slot_of_uniq[u] = (fl == 0) ? my_slot : member_slot[j];
    }
    if (touched) {
      tags[slot0 + lane] = tag;
      ts[slot0 + lane] = stamp;
      placed_at[slot0 + lane] = plc;
      freq[slot0 + lane] = cnt;
      if (dirty_loaded) dirty[slot0 + lane] = dirty_reg;
    }
  }
  if (lane == 0) {
    if (c_hit_lookups) atomicAdd(&counters[MTS_CNT_HIT_LOOKUPS], c_hit_lookups);
    if (c_uhits) atomicAdd(&counters[MTS_CNT_UNIQUE_HITS], c_uhits);
    if (c_dirty) atomicAdd(&counters[MTS_CNT_EVICTED_DIRTY], c_dirty);
    if (c_overflow) atomicAdd(&counters[MTS_CNT_OVERFLOW], c_overflow);
    if (c_overflow_dirty && overflow_dirty_count != nullptr) atomicAdd(overflow_dirty_count, c_overflow_dirty);
  }
}

// Ordered compaction of the members flagged "placed" (miss list) and of those whose victim
// held a row (evict list): count per block, scan the block counts, write.
constexpr int LIST_BLOCKS = 1024;

__device__ __forceinline__ int64_t list_per_block(int64_t n, int G) {
  const int64_t per = (n + G - 1) / G;
  return (per + CACHE_THREADS - 1) / CACHE_THREADS * CACHE_THREADS;
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_count_lists(const uint8_t* __restrict__ member_flag, const uint32_t* __restrict__ member_old_key,
                  const uint32_t* __restrict__ n_unique, uint32_t* __restrict__ cnt_miss,
                  uint32_t* __restrict__ cnt_evict) {
  __shared__ uint32_t sh[9];
  const int64_t n = *n_unique;
  const int64_t per = list_per_block(n, gridDim.x);
  const int64_t begin = (int64_t)blockIdx.x * per, end = min(n, begin + per);
  uint32_t a = 0, b = 0;
  for (int64_t j = begin + threadIdx.x; j < end; j += CACHE_THREADS) {
    if (member_flag[j] == 1) { a += 1; b += member_old_key[j] != FREE_TAG ? 1u : 0u; }
  }
  uint32_t ta, tb;
  block_scan_256(a, sh, &ta);
  block_scan_256(b, sh, &tb);
  if (threadIdx.x == 0) { cnt_miss[blockIdx.x] = ta; cnt_evict[blockIdx.x] = tb; }
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_scan_lists(uint32_t* __restrict__ cnt_miss, uint32_t* __restrict__ cnt_evict, int G,
                 const uint32_t* __restrict__ n_unique, int64_t n_lookups, int64_t capacity,
                 int64_t* __restrict__ counters, int32_t* __restrict__ status) {
  __shared__ uint32_t sh[9];
  constexpr int PER = LIST_BLOCKS / CACHE_THREADS;
  const int j0 = threadIdx.x * PER;
  for (int which = 0; which < 2; ++which) {
    uint32_t* cnt = which == 0 ? cnt_miss : cnt_evict;
    uint32_t v[PER];
    uint32_t s = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) { v[k] = j0 + k < G ? cnt[j0 + k] : 0u; s += v[k]; }
    uint32_t total;
    uint32_t ex = block_scan_256(s, sh, &total);
#pragma unroll
    for (int k = 0; k < PER; ++k) { if (j0 + k < G) cnt[j0 + k] = ex; ex += v[k]; }
    // more placements than list entries: the surplus is undone by cache_write_lists, which also sets
    // the number of evictions that remain
    if (threadIdx.x == 0) {
      if (which == 0) {
        counters[MTS_CNT_INSERTED] = min((int64_t)total, capacity);
        if ((int64_t)total > capacity) atomicOr(status, CACHE_STATUS_LIST_CUT);
      } else {
        counters[MTS_CNT_EVICTED] = capacity > 0 ? (int64_t)total : 0;
      }
    }
  }
  if (threadIdx.x == 0) {
    const int64_t U = *n_unique;
    counters[MTS_CNT_UNIQUE] = U;
    counters[MTS_CNT_MISS_LOOKUPS] = n_lookups - counters[MTS_CNT_HIT_LOOKUPS];
    counters[MTS_CNT_UNIQUE_MISSES] = U - counters[MTS_CNT_UNIQUE_HITS];
  }
}

// What the first level's list pass does for a second level behind it (all null when there is none).
struct TwoLevelLists {
  const int32_t* l2slot_of_uniq = nullptr;     // second-level slot of every key that missed the first level, or -1
  SecondLevel l2;
  int32_t* fetch_src = nullptr;                // per miss-list entry: second-level slot of the row, or -1 = store
  int64_t* drop_keys = nullptr;
  int32_t* drop_slots = nullptr;
  uint8_t* drop_dirty = nullptr;
  uint32_t* drop_cursor = nullptr;
  int32_t* ev1_ts = nullptr;                   // per evict-list entry: timestamp and use count of the victim
  uint32_t* ev1_freq = nullptr;
  unsigned long long* counters2 = nullptr;
};

// Writes the lists.  A placement whose list position is beyond the capacity cannot be carried out by the
// data movement, so it is undone here: the way gets its old tag, timestamp, count and dirty byte back,
// the key is not inserted (slot -1) and joins the overflow list.  Inside a set the surplus placements are
// the last ones, so the earlier ones stand as they are.
__global__ void __launch_bounds__(CACHE_THREADS)
cache_write_lists(uint8_t* __restrict__ member_flag, const uint32_t* __restrict__ member_old_key,
                  const uint8_t* __restrict__ member_old_dirty, const int32_t* __restrict__ member_old_ts,
                  const uint32_t* __restrict__ member_old_freq, const int32_t* __restrict__ member_old_placed,
                  const int32_t* __restrict__ member_slot,
                  const uint32_t* __restrict__ member_uidx, const uint32_t* __restrict__ ukey,
                  const uint32_t* __restrict__ n_unique, const uint32_t* __restrict__ base_miss,
                  const uint32_t* __restrict__ base_evict, int64_t capacity,
                  int64_t* __restrict__ miss_keys, int32_t* __restrict__ miss_slots,
                  int64_t* __restrict__ evict_keys, int32_t* __restrict__ evict_slots,
                  uint8_t* __restrict__ evict_dirty, int64_t* __restrict__ overflow_keys,
                  int64_t overflow_capacity, uint32_t* __restrict__ overflow_cursor,
                  uint32_t* __restrict__ tags, int32_t* __restrict__ ts, int32_t* __restrict__ placed_at,
                  uint32_t* __restrict__ freq, uint8_t* __restrict__ dirty, int32_t* __restrict__ slot_of_uniq,
                  unsigned long long* __restrict__ counters, TwoLevelLists two) {
  __shared__ uint32_t sh[9];
  const int64_t n = *n_unique;
  const int64_t per = list_per_block(n, gridDim.x);
  const int64_t begin = (int64_t)blockIdx.x * per, end = min(n, begin + per);
  uint32_t bm = base_miss[blockIdx.x], be = base_evict[blockIdx.x];
  for (int64_t t0 = begin; t0 < end; t0 += CACHE_THREADS) {
    const int64_t j = t0 + threadIdx.x;
    bool overflowed = j < end && member_flag[j] == 2;
    const bool placed = j < end && member_flag[j] == 1;
    const bool ev = placed && member_old_key[j] != FREE_TAG;
    uint32_t ta, tb;
    const uint32_t pa = block_scan_256(placed ? 1u : 0u, sh, &ta);
    const uint32_t pb = block_scan_256(ev ? 1u : 0u, sh, &tb);
    if (placed) {
      const int64_t at = (int64_t)bm + pa;
      if (at < capacity) {
        miss_keys[at] = (int64_t)ukey[member_uidx[j]];
        miss_slots[at] = member_slot[j];
        if (ev) {                                  // its position is at most `at`: inside the capacity too
          evict_keys[be + pb] = (int64_t)member_old_key[j];
          evict_slots[be + pb] = member_slot[j];
          evict_dirty[be + pb] = member_old_dirty[j];
          if (two.ev1_ts != nullptr) {             // the history the victim takes along to the second level
            two.ev1_ts[be + pb] = member_old_ts[j];
            two.ev1_freq[be + pb] = member_old_freq[j];
          }
        }
        if (two.l2slot_of_uniq != nullptr) {
          // where the row comes from: its second-level slot (the row is promoted: it leaves the second level
          // and keeps its dirty byte), or -1 = the backing store
          const int32_t s2 = two.l2slot_of_uniq[member_uidx[j]];
          two.fetch_src[at] = s2;
          if (s2 >= 0) {
            dirty[member_slot[j]] = two.l2.dirty[s2];
            two.l2.tags[s2] = FREE_TAG; two.l2.ts[s2] = -1; two.l2.placed[s2] = -1; two.l2.freq[s2] = 0; two.l2.dirty[s2] = 0;
            atomicAdd(&two.counters2[MTS_CNT2_PROMOTED], 1ull);
          }
        }
        // the last placement that fits fixes the length of the evict list
        if (at == capacity - 1) counters[MTS_CNT_EVICTED] = (unsigned long long)(be + pb + (ev ? 1u : 0u));
      } else {
        const int32_t slot = member_slot[j];
        tags[slot] = member_old_key[j];
        ts[slot] = member_old_ts[j];
        placed_at[slot] = member_old_placed[j];
        freq[slot] = member_old_freq[j];
        dirty[slot] = member_old_dirty[j];
        slot_of_uniq[member_uidx[j]] = -1;
        member_flag[j] = 2;
        overflowed = true;
        atomicAdd(&counters[MTS_CNT_OVERFLOW], 1ull);
        if (ev && member_old_dirty[j]) atomicAdd(&counters[MTS_CNT_EVICTED_DIRTY], ~0ull);     // minus one
      }
    }
    if (overflow_keys != nullptr && overflowed) {
      // the overflow list is a set: its order is not specified
      const uint32_t at = atomicAdd(overflow_cursor, 1u);
      if ((int64_t)at < overflow_capacity) overflow_keys[at] = (int64_t)ukey[member_uidx[j]];
    }
    if (two.l2slot_of_uniq != nullptr && overflowed) {
      // a second-level hit without a first-level way is served from the backing store in this batch: it
      // leaves the second level (dirty rows are written to the store by the data movement: drop list)
      const int32_t s2 = two.l2slot_of_uniq[member_uidx[j]];
      if (s2 >= 0) {
        const uint32_t at = atomicAdd(two.drop_cursor, 1u);
        const uint8_t d = two.l2.dirty[s2];
        if ((int64_t)at < capacity) {
          two.drop_keys[at] = (int64_t)ukey[member_uidx[j]];
          two.drop_slots[at] = s2;
          two.drop_dirty[at] = d;
        }
        two.l2.tags[s2] = FREE_TAG; two.l2.ts[s2] = -1; two.l2.placed[s2] = -1; two.l2.freq[s2] = 0; two.l2.dirty[s2] = 0;
        atomicAdd(&two.counters2[MTS_CNT2_L2_DROPPED], 1ull);
        if (d) atomicAdd(&two.counters2[MTS_CNT2_L2_DROPPED_DIRTY], 1ull);
      }
    }
    bm += ta;
    be += tb;
  }
}

__global__ void cache_scatter_slots(const uint32_t* __restrict__ sorted_pos, const uint32_t* __restrict__ uniq_idx,
                                    const int32_t* __restrict__ slot_of_uniq, int64_t n,
                                    const uint32_t* __restrict__ n_dev, int32_t* __restrict__ slot_of_lookup,
                                    const uint32_t* __restrict__ bag_of_lookup, int64_t pos_base,
                                    uint32_t* __restrict__ sorted_bag, int32_t* __restrict__ sorted_slot) {
  if (n_dev != nullptr) n = min(n, (int64_t)*n_dev);
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < n; p += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t ps = sorted_pos[p];
    const int32_t slot = slot_of_uniq[uniq_idx[p]];
    slot_of_lookup[ps] = slot;
    if (sorted_bag != nullptr) {
      // for the backward of the same batch: bag and slot of every lookup in the order of the sorted rows
      sorted_bag[p] = bag_of_lookup[ps - pos_base];
      sorted_slot[p] = slot;
    }
  }
}

// ------------------------------------------------------------------------------------ data movement
// Row copies in 16-byte pieces; thread i of the flattened (row, piece) space moves one piece,
// UNROLL independent pieces per thread are in flight before the first store.

#ifndef MTS_COPY_UNROLL
#define MTS_COPY_UNROLL 4
#endif
#ifndef MTS_COPY_BLOCKS_PER_SM
#define MTS_COPY_BLOCKS_PER_SM 8
#endif
constexpr int COPY_UNROLL = MTS_COPY_UNROLL;

template <typename SrcOf, typename DstOf>
__device__ __forceinline__ void copy_rows(int64_t n_rows, int vec16, SrcOf src_of, DstOf dst_of) {
  const int64_t total = n_rows * vec16;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride * COPY_UNROLL) {
    uint4 v[COPY_UNROLL];
    char* dst[COPY_UNROLL];
#pragma unroll
    for (int u = 0; u < COPY_UNROLL; ++u) {
      const int64_t e = i + u * stride;
      dst[u] = nullptr;
      if (e < total) {
        const int64_t r = e / vec16;
        const int c = (int)(e - r * vec16);
        const char* s = src_of(r);
        dst[u] = dst_of(r);
        if (s != nullptr && dst[u] != nullptr) {
          v[u] = *reinterpret_cast<const uint4*>(s + (int64_t)c * 16);
          dst[u] += (int64_t)c * 16;
        } else {
          dst[u] = nullptr;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < COPY_UNROLL; ++u)
      if (dst[u] != nullptr) *reinterpret_cast<uint4*>(dst[u]) = v[u];
  }
}

__device__ __forceinline__ int64_t list_len(const int64_t* counters, int which, int64_t capacity) {
  const int64_t n = counters[which];
  return n < capacity ? n : capacity;
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_save_victims(const char* __restrict__ data, int row_bytes, const int32_t* __restrict__ evict_slots,
                   const uint8_t* __restrict__ evict_dirty, const int64_t* __restrict__ counters,
                   int64_t capacity, char* __restrict__ staging) {
  const int64_t n = list_len(counters, MTS_CNT_EVICTED, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return evict_dirty[k] ? data + (int64_t)evict_slots[k] * row_bytes : nullptr; },
            [&](int64_t k) { return staging + k * row_bytes; });
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_fetch_misses(char* __restrict__ data, int row_bytes, const char* __restrict__ host_rows,
                   const int64_t* __restrict__ miss_keys, const int32_t* __restrict__ miss_slots,
                   const int64_t* __restrict__ counters, int64_t capacity) {
  const int64_t n = list_len(counters, MTS_CNT_INSERTED, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return host_rows + miss_keys[k] * row_bytes; },
            [&](int64_t k) { return data + (int64_t)miss_slots[k] * row_bytes; });
}

// Missed rows that arrived in list order through a contiguous copy: fetched[k] -> slot miss_slots[k].
__global__ void __launch_bounds__(CACHE_THREADS)
cache_place_fetched(char* __restrict__ data, int row_bytes, const char* __restrict__ fetched,
                    const int32_t* __restrict__ miss_slots, const int64_t* __restrict__ counters, int64_t capacity) {
  const int64_t n = list_len(counters, MTS_CNT_INSERTED, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return fetched + k * row_bytes; },
            [&](int64_t k) { return data + (int64_t)miss_slots[k] * row_bytes; });
}

// ---- missed rows through the bulk-copy engine (TMA, non-tensor form) ------------------------
// Plain 16-byte loads from mapped host memory top out far below the host link's bandwidth (the
// requests that reach the link are small).  Here one warp per block asks the bulk-copy engine for
// whole rows (host memory -> shared memory, completion counted in bytes on an mbarrier); the block
// then stores the tile to the rows' cache slots.  The wait on the mbarrier is bounded: if it ever
// ran out, the block raises the cache's status bit, waits once more (bounded) for its copies in
// flight and leaves, so the kernel cannot hang.
#ifndef MTS_FETCH_BLOCKS
#define MTS_FETCH_BLOCKS 32      // blocks of the bulk-copy fetch: the host link needs few copies in flight
#endif
constexpr int FETCH_THREADS = 128;
constexpr int FETCH_TILE_BYTES = 16384;
constexpr uint32_t FETCH_WAIT_LIMIT = 1u << 22;

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

__global__ void __launch_bounds__(FETCH_THREADS)
cache_fetch_misses_bulk(char* __restrict__ data, int row_bytes, const char* __restrict__ host_rows,
                        const int64_t* __restrict__ miss_keys, const int32_t* __restrict__ miss_slots,
                        const int64_t* __restrict__ counters, int64_t capacity, int32_t* status,
                        uint32_t wait_limit) {
  __shared__ __align__(128) unsigned char tile[FETCH_TILE_BYTES];
  __shared__ __align__(8) unsigned long long bar_storage;
  const int64_t n = list_len(counters, MTS_CNT_INSERTED, capacity);
  const int rows_per_tile = FETCH_TILE_BYTES / row_bytes;
  const int64_t n_tiles = (n + rows_per_tile - 1) / rows_per_tile;
  const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&bar_storage);
  const uint32_t tile_s = (uint32_t)__cvta_generic_to_shared(tile);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  uint32_t parity = 0;
  const int vec = row_bytes / 16;
  for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const int64_t r0 = t * rows_per_tile;
    const int nr = (int)min((int64_t)rows_per_tile, n - r0);
    if (threadIdx.x < 32) {
      // writes of the engine into the tile must be ordered after the block's reads of the last tile
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      if (threadIdx.x == 0)
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(nr * row_bytes))
                     : "memory");
      __syncwarp();
      for (int k = threadIdx.x; k < nr; k += 32) {
        const char* src = host_rows + miss_keys[r0 + k] * (int64_t)row_bytes;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(tile_s + (uint32_t)(k * row_bytes)), "l"(src), "r"((uint32_t)row_bytes), "r"(bar)
                     : "memory");
      }
    }
    bool ok = mbar_wait_bounded(bar, parity, wait_limit);
    if (!__syncthreads_and(ok)) {
      // give up on this call: say so, but leave only when the copies in flight have landed (bounded as
      // well), so that nothing writes into this block's shared memory after it is gone
      if (threadIdx.x == 0) atomicOr(status, CACHE_STATUS_FETCH_TIMEOUT);
      mbar_wait_bounded(bar, parity, FETCH_WAIT_LIMIT);
      return;
    }
    parity ^= 1u;
    const int total = nr * vec;
    for (int e = threadIdx.x; e < total; e += FETCH_THREADS) {
      const int k = e / vec, c = e - k * vec;
      *reinterpret_cast<uint4*>(data + (int64_t)miss_slots[r0 + k] * row_bytes + c * 16) =
          *reinterpret_cast<const uint4*>(tile + k * row_bytes + c * 16);
    }
    __syncthreads();
  }
}

// One warp per key of an overflow list: if the key is resident now, copy its host row into its
// slot again (the copy made when it was placed may predate an update applied to the host row).
__global__ void __launch_bounds__(CACHE_THREADS)
cache_refetch_resident(char* __restrict__ data, int row_bytes, const char* __restrict__ host_rows,
                       const int64_t* __restrict__ keys, const int64_t* __restrict__ counters, int64_t capacity,
                       const uint32_t* __restrict__ tags, const int32_t* __restrict__ placed_at, int64_t placed_step,
                       uint64_t S) {
  const int64_t n = list_len(counters, MTS_CNT_OVERFLOW, capacity);
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t k = warp0; k < n; k += nwarps) {
    const uint32_t key = (uint32_t)keys[k];
    const int64_t slot0 = (int64_t)set_of_key(key, S) * 32;
    // only a row inserted by the batch named in placed_step.  A row inserted earlier has been updated in
    // its slot since (the host copy is the stale one); a later tag step may have inserted the key meanwhile,
    // in a slot whose victim has not been saved yet and whose own fetch is still to come.  The step of the
    // insertion is kept apart from the timestamp, which later hits refresh.
    const uint32_t hit = __ballot_sync(0xffffffffu, tags[slot0 + lane] == key &&
                                                        (placed_step < 0 || (int64_t)placed_at[slot0 + lane] == placed_step));
    if (hit) {
      const char* src = host_rows + (int64_t)key * row_bytes;
      char* dst = data + (slot0 + __ffs(hit) - 1) * row_bytes;
      for (int c = lane * 16; c < row_bytes; c += 32 * 16)
        *reinterpret_cast<uint4*>(dst + c) = *reinterpret_cast<const uint4*>(src + c);
    }
  }
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_write_victims(char* __restrict__ host_rows, int row_bytes, const int64_t* __restrict__ evict_keys,
                    const uint8_t* __restrict__ evict_dirty, const int64_t* __restrict__ counters,
                    int64_t capacity, const char* __restrict__ staging) {
  const int64_t n = list_len(counters, MTS_CNT_EVICTED, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return evict_dirty[k] ? staging + k * row_bytes : nullptr; },
            [&](int64_t k) { return host_rows + evict_keys[k] * row_bytes; });
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_flush_rows(const char* __restrict__ data, int row_bytes, const uint32_t* __restrict__ tags,
                 const uint8_t* __restrict__ dirty, int64_t n_slots, char* __restrict__ host_rows) {
  copy_rows(n_slots, row_bytes / 16,
            [&](int64_t s) { return (tags[s] != FREE_TAG && dirty[s]) ? data + s * row_bytes : nullptr; },
            [&](int64_t s) { return host_rows + (int64_t)tags[s] * row_bytes; });
}

__global__ void cache_clear_dirty(uint8_t* dirty, int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    dirty[i] = 0;
}

__global__ void cache_export(const uint32_t* __restrict__ tags, const int32_t* __restrict__ ts,
                             const uint32_t* __restrict__ freq, const uint8_t* __restrict__ dirty, int64_t n,
                             int64_t* o_tags, int64_t* o_ts, int64_t* o_freq, uint8_t* o_dirty) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    if (o_tags) o_tags[i] = tags[i] == FREE_TAG ? -1 : (int64_t)tags[i];
    if (o_ts) o_ts[i] = (int64_t)ts[i];
    if (o_freq) o_freq[i] = (int64_t)freq[i];
    if (o_dirty) o_dirty[i] = dirty[i];
  }
}

struct CacheLayout {
  size_t keys_a, keys_b, vals_a, vals_b, uniq_idx, seg_start, ukey, mult, set_a, set_b, sval_a, sval_b,
      sseg_start, slot_of_uniq, member_flag, member_old_key, member_old_dirty, member_old_ts, member_old_freq,
      member_old_placed, member_slot, hist, scan, cnt_miss,
      cnt_evict, n_unique, n_sets, ovf_cursor, missed, cnt_missed, n_missed, ins_ts, ins_dirty, l2slot_of_uniq,
      drop_cursor, bag_of_lookup, total;
};

static int bits_of(int64_t values) {
  int bits = 1;
  while (bits < 32 && (1ll << bits) < values) ++bits;
  return bits;
}

static CacheLayout cache_layout(const mts_cache* c, int64_t N) {
  CacheLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t n = (size_t)(N > 0 ? N : 1);
  L.keys_a = take(n * 4); L.keys_b = take(n * 4); L.vals_a = take(n * 4); L.vals_b = take(n * 4);
  L.uniq_idx = take(n * 4); L.seg_start = take((n + 1) * 4);
  L.ukey = take(n * 4); L.mult = take(n * 4);
  L.set_a = take(n * 4); L.set_b = take(n * 4); L.sval_a = take(n * 4); L.sval_b = take(n * 4);
  L.sseg_start = take((n + 1) * 4);
  L.slot_of_uniq = take(n * 4);
  L.member_flag = take(n); L.member_old_key = take(n * 4); L.member_old_dirty = take(n); L.member_slot = take(n * 4);
  L.member_old_ts = take(n * 4); L.member_old_freq = take(n * 4); L.member_old_placed = take(n * 4);
  L.hist = take(std::max(sort_hist_words((int64_t)n, bits_of(c->key_space)), sort_hist_words((int64_t)n, bits_of(c->S))) * 4);
  L.scan = take(scan_scratch_words() * 4);
  L.cnt_miss = take(LIST_BLOCKS * 4); L.cnt_evict = take(LIST_BLOCKS * 4);
  L.n_unique = take(256); L.n_sets = take(256); L.ovf_cursor = take(256);
  L.missed = take(n); L.cnt_missed = take(PROBE_BLOCKS * 4); L.n_missed = take(256);
  L.ins_ts = take(n * 4); L.ins_dirty = take(n); L.l2slot_of_uniq = take(n * 4); L.drop_cursor = take(256);
  L.bag_of_lookup = take(n * 4);
  L.total = off;
  return L;
}

}  // namespace mts

using namespace mts;

extern "C" int mts_cache_destroy(mts_cache* c);

static int cache_create_impl(mts_cache** out, int64_t num_sets, int64_t key_space, int32_t ways, int32_t dim,
                             int32_t dtype, int32_t policy, int32_t lock_depth, void* external_rows) {
  if (!out) return set_error(MTS_ERR_INVALID_ARG, "cache_create: null out");
  *out = nullptr;
  if (ways != MTS_CACHE_WAYS) return set_error(MTS_ERR_INVALID_ARG, "cache_create: ways must be %d", MTS_CACHE_WAYS);
  if (num_sets < 1 || num_sets * MTS_CACHE_WAYS >= (1ll << 31))
    return set_error(MTS_ERR_INVALID_ARG, "cache_create: num_sets %lld out of range", (long long)num_sets);
  if (key_space < 1 || key_space >= (1ll << 32) - 1)
    return set_error(MTS_ERR_INVALID_ARG, "cache_create: key_space %lld out of range", (long long)key_space);
  if (dtype != MTS_DTYPE_FP32 && dtype != MTS_DTYPE_FP16) return set_error(MTS_ERR_INVALID_ARG, "cache_create: dtype");
  if (policy != MTS_POLICY_LRU && policy != MTS_POLICY_LFU) return set_error(MTS_ERR_INVALID_ARG, "cache_create: policy");
  if (lock_depth < 0 || dim < 1) return set_error(MTS_ERR_INVALID_ARG, "cache_create: lock_depth / dim");
  if (dim > 1024) return set_error(MTS_ERR_UNSUPPORTED, "cache_create: dim %d above 1024", dim);
  const int eb = dtype == MTS_DTYPE_FP32 ? 4 : 2;
  if ((dim * eb) % 16) return set_error(MTS_ERR_ALIGNMENT, "cache_create: row bytes %d not a multiple of 16", dim * eb);
  mts_cache* c = new mts_cache();
  c->S = num_sets; c->key_space = key_space; c->dim = dim; c->dtype = dtype; c->elem_bytes = eb;
  c->policy = policy; c->lock_depth = lock_depth; c->row_bytes = dim * eb;
  const int64_t n = num_sets * MTS_CACHE_WAYS;
  int dev = 0, sms = 0;
  int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc == MTS_OK) rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "sm count");
  if (rc == MTS_OK && sms > 0) c->sm_count = sms;
  if (rc == MTS_OK) rc = check_cuda(cudaMalloc(&c->tags, n * 4), "cudaMalloc(tags)");
  if (rc == MTS_OK) rc = check_cuda(cudaMalloc(&c->ts, n * 4), "cudaMalloc(timestamps)");
  if (rc == MTS_OK) rc = check_cuda(cudaMalloc(&c->placed, n * 4), "cudaMalloc(insertion steps)");
  if (rc == MTS_OK) rc = check_cuda(cudaMalloc(&c->freq, n * 4), "cudaMalloc(counts)");
  if (rc == MTS_OK) rc = check_cuda(cudaMalloc(&c->dirty, n), "cudaMalloc(dirty)");
  if (external_rows != nullptr) {
    c->data = static_cast<char*>(external_rows);
    c->owns_data = false;
  } else if (rc == MTS_OK) {
    rc = check_cuda(cudaMalloc(&c->data, (size_t)n * c->row_bytes), "cudaMalloc(cache rows)");
  }
  if (rc == MTS_OK) rc = check_cuda(cudaMalloc(&c->d_status, 256), "cudaMalloc(cache status)");
  if (rc == MTS_OK) rc = check_cuda(cudaMemset(c->d_status, 0, 256), "cudaMemset(cache status)");
  if (rc == MTS_OK) {
    {
      LaunchScope scope(K_OTHER, nullptr);
      cache_init_state<<<c->sm_count * 4, 256>>>(c->tags, c->ts, c->placed, c->freq, c->dirty, n);
    }
    rc = check_launch("cache_init_state");
  }
  if (rc == MTS_OK && c->owns_data) rc = check_cuda(cudaMemset(c->data, 0, (size_t)n * c->row_bytes), "cudaMemset(cache rows)");
  if (rc == MTS_OK) rc = check_cuda(cudaDeviceSynchronize(), "cache_create sync");
  if (rc != MTS_OK) { mts_cache_destroy(c); return rc; }
  *out = c;
  return MTS_OK;
}

extern "C" int mts_cache_create(mts_cache** out, int64_t num_sets, int64_t key_space, int32_t ways, int32_t dim,
                                int32_t dtype, int32_t policy, int32_t lock_depth) {
  return cache_create_impl(out, num_sets, key_space, ways, dim, dtype, policy, lock_depth, nullptr);
}

extern "C" int mts_cache_create_host_level(mts_cache** out, int64_t num_sets, int64_t key_space, int32_t ways,
                                           int32_t dim, int32_t dtype, int32_t policy, int32_t lock_depth,
                                           void* host_rows_mapped) {
  if (!host_rows_mapped) return set_error(MTS_ERR_INVALID_ARG, "cache_create_host_level: null row storage");
  if ((uintptr_t)host_rows_mapped & 15) return set_error(MTS_ERR_ALIGNMENT, "cache_create_host_level: row storage must be 16-byte aligned");
  return cache_create_impl(out, num_sets, key_space, ways, dim, dtype, policy, lock_depth, host_rows_mapped);
}

extern "C" int mts_cache_destroy(mts_cache* c) {
  if (!c) return MTS_OK;
  cudaFree(c->tags); cudaFree(c->ts); cudaFree(c->placed); cudaFree(c->freq); cudaFree(c->dirty);
  if (c->owns_data) cudaFree(c->data);
  cudaFree(c->d_status);
  delete c;
  return MTS_OK;
}

extern "C" int mts_cache_status(mts_cache* c, int32_t* host_status, void* stream) {
  if (!c || !host_status) return set_error(MTS_ERR_INVALID_ARG, "cache_status: null argument");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = check_cuda(cudaMemcpyAsync(host_status, c->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, s),
                      "cudaMemcpyAsync(cache status)");
  if (rc == MTS_OK) rc = check_cuda(cudaMemsetAsync(c->d_status, 0, sizeof(int32_t), s), "cudaMemsetAsync(cache status)");
  if (rc == MTS_OK) rc = check_cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize(cache status)");
  if (rc == MTS_OK && (*host_status & 1)) return set_error(MTS_ERR_TIMEOUT, "cache: a bounded wait on a bulk copy ran out");
  return rc;
}

extern "C" void* mts_cache_data(mts_cache* c) { return c ? c->data : nullptr; }
extern "C" uint8_t* mts_cache_dirty(mts_cache* c) { return c ? c->dirty : nullptr; }

__global__ void linearize_group_keys(const TableMeta* __restrict__ meta, int32_t t_begin, int64_t n_bags, int32_t B,
                                     const int64_t* __restrict__ indices, const int64_t* __restrict__ offsets,
                                     int64_t lookup_begin, int64_t n, int64_t* __restrict__ keys_out,
                                     int32_t* status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t gb = gid / 8;
  if (gb >= n_bags) return;
  const int sub = (int)(gid % 8);
  const int64_t bag = (int64_t)t_begin * B + gb;
  const int32_t t = (int32_t)(bag / B);
  const int64_t rows = meta[t].rows;
  const int64_t roff = meta[t].row_offset - meta[t_begin].row_offset;
  const int64_t i1 = offsets[bag + 1];
  for (int64_t i = offsets[bag] + sub; i < i1; i += 8) {
    const int64_t o = i - lookup_begin;
    if (o >= 0 && o < n) keys_out[o] = roff + clamp_index(indices[i], rows, status);
  }
}

extern "C" int mts_linearize_keys(const mts_tables* h, int32_t t_begin, int32_t t_end, int32_t B,
                                  const int64_t* indices, const int64_t* offsets, int64_t lookup_begin, int64_t n,
                                  int64_t* keys_out, void* stream) {
  if (!h || !offsets || B < 1 || t_begin < 0 || t_end > h->T || t_begin >= t_end || n < 0 || lookup_begin < 0 ||
      (n > 0 && (!indices || !keys_out)))
    return set_error(MTS_ERR_INVALID_ARG, "linearize_keys: bad argument");
  if (n == 0) return MTS_OK;
  const int64_t n_bags = (int64_t)(t_end - t_begin) * B;
  {
    LaunchScope scope(K_LINEARIZE, static_cast<cudaStream_t>(stream));
    linearize_group_keys<<<(unsigned)ceil_div(n_bags * 8, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        h->d_meta, t_begin, n_bags, B, indices, offsets, lookup_begin, n, keys_out, h->d_status);
  }
  return check_launch("linearize_group_keys");
}

extern "C" size_t mts_cache_workspace_bytes(const mts_cache* c, int64_t N) {
  if (!c || N < 0) return 0;
  return cache_layout(c, N).total;
}

namespace {

// Where the keys of a lookup_insert call come from: an array of keys relative to the cache's table
// group, or the sparse input of a batch (tables [t_begin, t_end) of `tables`).
struct KeySource {
  const int64_t* keys = nullptr;
  const mts_tables* tables = nullptr;
  int32_t t_begin = 0, t_end = 0, B = 0;
  const int64_t* indices = nullptr;
  const int64_t* offsets = nullptr;
  int64_t lookup_begin = 0;
  uint32_t* sorted_rows_out = nullptr;     // batch-wide arrays; this call fills [lookup_begin, lookup_begin + N)
  uint32_t* sorted_bag_out = nullptr;
  int32_t* sorted_slot_out = nullptr;
};

// n_dev (nullable): device-resident number of keys, N is then its upper bound.  attrs: the keys are rows that
// arrive with a history (see InsertAttrs; indexed by position in `src.keys`).  two (nullable): a second level
// behind this cache; its l2slot_of_uniq and drop_cursor are taken from the workspace here.
int lookup_insert_impl(mts_cache* c, const KeySource& src, int64_t N, int64_t step, int32_t* slot_of_lookup,
                       int64_t* miss_keys, int32_t* miss_slots, int64_t* evict_keys, int32_t* evict_slots,
                       uint8_t* evict_dirty, int64_t* overflow_keys, int64_t list_capacity, int64_t overflow_capacity,
                       int64_t* counters, void* workspace, size_t workspace_bytes, void* stream,
                       const uint32_t* n_dev = nullptr, InsertAttrs attrs = InsertAttrs(),
                       TwoLevelLists* two = nullptr, unsigned long long* overflow_dirty_count = nullptr) {
  if (!c || !counters || N < 0 || list_capacity < 0 || overflow_capacity < 0 || step < 0 || step >= (1ll << 31) - 1)
    return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert: bad argument");
  if (N > 0 && !slot_of_lookup) return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert: null slot_of_lookup");
  if (list_capacity > 0 && (!miss_keys || !miss_slots || !evict_keys || !evict_slots || !evict_dirty))
    return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert: null list buffer");
  if (N >= (1ll << 32) - 1) return set_error(MTS_ERR_UNSUPPORTED, "cache_lookup_insert: N must fit 32 bits");
  const CacheLayout L = cache_layout(c, N);
  if (!workspace || ((uintptr_t)workspace & 255))
    return set_error(MTS_ERR_ALIGNMENT, "cache_lookup_insert: workspace must be non-null and 256-byte aligned");
  if (workspace_bytes < L.total)
    return set_error(MTS_ERR_WORKSPACE, "cache_lookup_insert: workspace of %zu bytes, %zu needed", workspace_bytes, L.total);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  auto U32 = [&](size_t off) { return reinterpret_cast<uint32_t*>(ws + off); };
  const int grid = c->sm_count * 8;
  const int key_bits = bits_of(c->key_space);
  // The sort alternates between two buffer pairs.  When the caller wants the sorted lookups, its
  // arrays are the pair the last pass writes into, so that exporting them costs nothing.
  uint32_t *keys_a = U32(L.keys_a), *vals_a = U32(L.vals_a), *keys_b = U32(L.keys_b), *vals_b = U32(L.vals_b);
  uint32_t key_base = 0u;
  if (src.tables != nullptr) {
    key_base = (uint32_t)src.tables->h_meta[src.t_begin].row_offset;
    if (src.sorted_rows_out != nullptr) {
      const bool result_in_a = N <= 1 || (sort_passes(key_bits) & 1) == 0;
      (result_in_a ? keys_a : keys_b) = src.sorted_rows_out + src.lookup_begin;
    }
  }
  int rc;
  if (src.tables == nullptr) {
    if (N > 0 && !src.keys) return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert: null keys");
    {
      LaunchScope scope(K_CACHE_PREPARE, s);
      cache_prepare_keys<<<grid, 256, 0, s>>>(src.keys, N, n_dev, c->key_space, keys_a, vals_a, counters,
                                              U32(L.ovf_cursor), c->d_status);
    }
    rc = check_launch("cache_prepare_keys");
  } else {
    const int64_t n_bags = (int64_t)(src.t_end - src.t_begin) * src.B;
    {
      LaunchScope scope(K_CACHE_PREPARE, s);
      cache_prepare_from_indices<<<(unsigned)ceil_div(std::max<int64_t>(n_bags * 8, MTS_NUM_COUNTERS), 256), 256, 0, s>>>(
          src.tables->d_meta, src.t_begin, n_bags, src.B, src.indices, src.offsets, src.lookup_begin, N, keys_a, vals_a,
          src.sorted_rows_out != nullptr ? U32(L.bag_of_lookup) : nullptr, counters, U32(L.ovf_cursor),
          src.tables->d_status);
    }
    rc = check_launch("cache_prepare_from_indices");
  }
  if (rc != MTS_OK) return rc;
  uint32_t* n_unique = U32(L.n_unique);
  uint32_t* n_sets = U32(L.n_sets);
  if (N == 0) {
    return MTS_OK;   // counters already written: all zero
  }
  uint32_t *sk = nullptr, *sp = nullptr;
  rc = radix_sort_pairs(keys_a, vals_a, keys_b, vals_b, N, n_dev, key_bits, key_base, U32(L.hist), &sk, &sp, s);
  if (rc != MTS_OK) return rc;
  rc = unique_segments(sk, N, n_dev, U32(L.seg_start), U32(L.uniq_idx), n_unique, U32(L.scan), s);
  if (rc != MTS_OK) return rc;
  // hits are found and refreshed key by key; only the missing keys are grouped by set for the replacement
  int32_t* slot_of_uniq = reinterpret_cast<int32_t*>(ws + L.slot_of_uniq);
  uint8_t* missed = reinterpret_cast<uint8_t*>(ws + L.missed);
  uint32_t* n_missed = U32(L.n_missed);
  const int PG = (int)std::min<int64_t>((int64_t)PROBE_BLOCKS, ceil_div(N, CACHE_THREADS * 4));
  {
    LaunchScope scope(K_CACHE_DESCRIBE, s);
    cache_probe_hits<<<PG, CACHE_THREADS, 0, s>>>(sk, key_base, U32(L.seg_start), n_unique, (uint64_t)c->S, c->tags, c->ts,
                                                  c->freq, (int32_t)step, U32(L.ukey), U32(L.mult), slot_of_uniq, missed,
                                                  U32(L.cnt_missed), reinterpret_cast<unsigned long long*>(counters), sp,
                                                  attrs, reinterpret_cast<int32_t*>(ws + L.ins_ts),
                                                  reinterpret_cast<uint8_t*>(ws + L.ins_dirty));
  }
  {
    LaunchScope scope(K_CACHE_DESCRIBE, s);
    cache_scan_missed<<<1, CACHE_THREADS, 0, s>>>(U32(L.cnt_missed), PG, n_missed);
  }
  {
    LaunchScope scope(K_CACHE_DESCRIBE, s);
    cache_compact_missed<<<PG, CACHE_THREADS, 0, s>>>(missed, U32(L.ukey), n_unique, (uint64_t)c->S, U32(L.cnt_missed),
                                                      U32(L.set_a), U32(L.sval_a));
  }
  TwoLevelLists lists2;
  if (two != nullptr) {
    // where the keys that missed this level sit in the second one (before the sort by set reuses the buffers)
    two->l2slot_of_uniq = reinterpret_cast<int32_t*>(ws + L.l2slot_of_uniq);
    two->drop_cursor = U32(L.drop_cursor);
    if (cudaMemsetAsync(two->drop_cursor, 0, sizeof(uint32_t), s) != cudaSuccess) return check_launch("memset(drop cursor)");
    {
      LaunchScope scope(K_CACHE_DESCRIBE, s);
      cache_probe_second_level<<<grid, CACHE_THREADS, 0, s>>>(U32(L.sval_a), n_missed, U32(L.ukey), U32(L.mult), two->l2,
                                                              reinterpret_cast<int32_t*>(ws + L.l2slot_of_uniq),
                                                              two->counters2);
    }
    lists2 = *two;
  }
  rc = check_launch("cache_probe_hits / cache_compact_missed");
  if (rc != MTS_OK) return rc;
  const int set_bits = c->S > 1 ? bits_of(c->S) : 0;
  uint32_t *ss = nullptr, *su = nullptr;
  rc = radix_sort_pairs(U32(L.set_a), U32(L.sval_a), U32(L.set_b), U32(L.sval_b), N, n_missed, set_bits, 0u,
                        U32(L.hist), &ss, &su, s);
  if (rc != MTS_OK) return rc;
  rc = unique_segments(ss, N, n_missed, U32(L.sseg_start), nullptr, n_sets, U32(L.scan), s);
  if (rc != MTS_OK) return rc;
  uint8_t* member_flag = reinterpret_cast<uint8_t*>(ws + L.member_flag);
  uint8_t* member_old_dirty = reinterpret_cast<uint8_t*>(ws + L.member_old_dirty);
  int32_t* member_slot = reinterpret_cast<int32_t*>(ws + L.member_slot);
  {
    LaunchScope scope(K_CACHE_PROBE_REPLACE, s);
    cache_probe_replace<<<grid, CACHE_THREADS, 0, s>>>(
        ss, su, U32(L.sseg_start), n_sets, U32(L.ukey), U32(L.mult), c->tags, c->ts, c->placed, c->freq, c->dirty, (int32_t)step,
        c->lock_depth, c->policy, slot_of_uniq, member_flag, U32(L.member_old_key), member_old_dirty,
        reinterpret_cast<int32_t*>(ws + L.member_old_ts), U32(L.member_old_freq),
        reinterpret_cast<int32_t*>(ws + L.member_old_placed), member_slot,
        reinterpret_cast<unsigned long long*>(counters),
        attrs.ts != nullptr ? reinterpret_cast<const int32_t*>(ws + L.ins_ts) : nullptr,
        attrs.ts != nullptr ? reinterpret_cast<const uint8_t*>(ws + L.ins_dirty) : nullptr, overflow_dirty_count);
  }
  rc = check_launch("cache_probe_replace");
  if (rc != MTS_OK) return rc;
  const int G = (int)std::min<int64_t>((int64_t)LIST_BLOCKS, ceil_div(N, CACHE_THREADS * 4));
  {
    LaunchScope scope(K_CACHE_LISTS, s);
    cache_count_lists<<<G, CACHE_THREADS, 0, s>>>(member_flag, U32(L.member_old_key), n_missed, U32(L.cnt_miss),
                                                  U32(L.cnt_evict));
  }
  {
    LaunchScope scope(K_CACHE_LISTS, s);
    cache_scan_lists<<<1, CACHE_THREADS, 0, s>>>(U32(L.cnt_miss), U32(L.cnt_evict), G, n_unique, N, list_capacity,
                                                 counters, c->d_status);
  }
  {
    LaunchScope scope(K_CACHE_LISTS, s);
    cache_write_lists<<<G, CACHE_THREADS, 0, s>>>(
        member_flag, U32(L.member_old_key), member_old_dirty, reinterpret_cast<int32_t*>(ws + L.member_old_ts),
        U32(L.member_old_freq), reinterpret_cast<int32_t*>(ws + L.member_old_placed), member_slot, su, U32(L.ukey), n_missed, U32(L.cnt_miss), U32(L.cnt_evict), list_capacity,
        miss_keys, miss_slots, evict_keys, evict_slots, evict_dirty, overflow_keys, overflow_capacity, U32(L.ovf_cursor),
        c->tags, c->ts, c->placed, c->freq, c->dirty, slot_of_uniq, reinterpret_cast<unsigned long long*>(counters), lists2);
  }
  {
    // positions are relative to the key array, or batch positions when the keys came from a batch's
    // sparse input (slot_of_lookup is then the batch-wide array)
    LaunchScope scope(K_CACHE_SCATTER_SLOTS, s);
    const bool exp = src.sorted_rows_out != nullptr;
    cache_scatter_slots<<<grid, 256, 0, s>>>(sp, U32(L.uniq_idx), slot_of_uniq, N, n_dev, slot_of_lookup,
                                             exp ? U32(L.bag_of_lookup) : nullptr, src.lookup_begin,
                                             exp ? src.sorted_bag_out + src.lookup_begin : nullptr,
                                             exp ? src.sorted_slot_out + src.lookup_begin : nullptr);
  }
  return check_launch("cache lists / scatter");
}

}  // namespace

extern "C" int mts_cache_lookup_insert(mts_cache* c, const int64_t* keys, int64_t N, int64_t step,
                                       int32_t* slot_of_lookup, int64_t* miss_keys, int32_t* miss_slots,
                                       int64_t* evict_keys, int32_t* evict_slots, uint8_t* evict_dirty,
                                       int64_t* overflow_keys, int64_t list_capacity, int64_t* counters,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  KeySource src;
  src.keys = keys;
  return lookup_insert_impl(c, src, N, step, slot_of_lookup, miss_keys, miss_slots, evict_keys, evict_slots, evict_dirty,
                            overflow_keys, list_capacity, list_capacity, counters, workspace, workspace_bytes, stream);
}

extern "C" int mts_cache_lookup_insert_tables(mts_cache* c, const mts_tables* h, int32_t t_begin, int32_t t_end,
                                              int32_t B, const int64_t* indices, const int64_t* offsets,
                                              int64_t lookup_begin, int64_t n, int64_t step, int32_t* slot_of_lookup,
                                              int64_t* miss_keys, int32_t* miss_slots, int64_t* evict_keys,
                                              int32_t* evict_slots, uint8_t* evict_dirty, int64_t list_capacity,
                                              int64_t* overflow_keys, int64_t overflow_capacity, int64_t* counters,
                                              uint32_t* sorted_rows_out, uint32_t* sorted_bag_out,
                                              int32_t* sorted_slot_out, void* workspace, size_t workspace_bytes,
                                              void* stream) {
  if (!c || !h || !offsets || B < 1 || t_begin < 0 || t_end > h->T || t_begin >= t_end || n < 0 || lookup_begin < 0 ||
      (n > 0 && !indices))
    return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert_tables: bad argument");
  if (h->h_meta[t_end - 1].row_offset + h->h_meta[t_end - 1].rows - h->h_meta[t_begin].row_offset != c->key_space)
    return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert_tables: tables [%d, %d) hold %lld rows, the cache was created for %lld",
                     t_begin, t_end,
                     (long long)(h->h_meta[t_end - 1].row_offset + h->h_meta[t_end - 1].rows - h->h_meta[t_begin].row_offset),
                     (long long)c->key_space);
  if ((sorted_rows_out == nullptr) != (sorted_bag_out == nullptr) || (sorted_rows_out == nullptr) != (sorted_slot_out == nullptr))
    return set_error(MTS_ERR_INVALID_ARG, "cache_lookup_insert_tables: pass sorted_rows_out, sorted_bag_out and sorted_slot_out together");
  if (lookup_begin + n >= (1ll << 32) - 1 || (int64_t)h->T * B >= (1ll << 32))
    return set_error(MTS_ERR_UNSUPPORTED, "cache_lookup_insert_tables: lookup positions and bag ids must fit 32 bits");
  KeySource src;
  src.tables = h; src.t_begin = t_begin; src.t_end = t_end; src.B = B;
  src.indices = indices; src.offsets = offsets; src.lookup_begin = lookup_begin;
  src.sorted_rows_out = sorted_rows_out; src.sorted_bag_out = sorted_bag_out; src.sorted_slot_out = sorted_slot_out;
  return lookup_insert_impl(c, src, n, step, slot_of_lookup, miss_keys, miss_slots, evict_keys, evict_slots, evict_dirty,
                            overflow_keys, list_capacity, overflow_capacity, counters, workspace, workspace_bytes, stream);
}

// ------------------------------------------------------------------------------------ two cache levels
namespace mts {

// counters2[0..9] come from the first level's pass; the second level's pass counted into a scratch block.
__global__ void cache2_finish_counters(const int64_t* __restrict__ l2_counters,
                                       const unsigned long long* __restrict__ bypass_dirty,
                                       int64_t* __restrict__ counters2) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    counters2[MTS_CNT2_DEMOTED] = l2_counters[MTS_CNT_INSERTED];
    counters2[MTS_CNT2_L2_EVICTED] = l2_counters[MTS_CNT_EVICTED];
    counters2[MTS_CNT2_L2_EVICTED_DIRTY] = l2_counters[MTS_CNT_EVICTED_DIRTY];
    counters2[MTS_CNT2_L2_BYPASS] = l2_counters[MTS_CNT_OVERFLOW];
    counters2[MTS_CNT2_L2_BYPASS_DIRTY] = (int64_t)*bypass_dirty;
  }
}

__global__ void cache2_begin(int64_t* __restrict__ counters2, unsigned long long* __restrict__ bypass_dirty) {
  if (blockIdx.x == 0 && threadIdx.x < MTS_NUM_COUNTERS2 - MTS_NUM_COUNTERS) counters2[MTS_NUM_COUNTERS + threadIdx.x] = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) *bypass_dirty = 0ull;
}

// number of first-level victims as the 32-bit device count the second level's pass takes
__global__ void cache2_victim_count(const int64_t* __restrict__ counters, int64_t capacity, uint32_t* __restrict__ n_out) {
  if (blockIdx.x == 0 && threadIdx.x == 0) *n_out = (uint32_t)list_len(counters, MTS_CNT_EVICTED, capacity);
}

// rows that leave the second level for the store (its victims, and hits that found no first-level way)
__global__ void __launch_bounds__(CACHE_THREADS)
cache2_rows_to_store(const char* __restrict__ l2_rows, int row_bytes, const int64_t* __restrict__ keys,
                     const int32_t* __restrict__ slots, const uint8_t* __restrict__ dirty,
                     const int64_t* __restrict__ counters2, int which, int64_t capacity, char* __restrict__ store) {
  const int64_t n = list_len(counters2, which, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return dirty[k] ? l2_rows + (int64_t)slots[k] * row_bytes : nullptr; },
            [&](int64_t k) { return store + keys[k] * row_bytes; });
}

// the rows to be inserted into the first level, from their second-level slot or from the store, in list order
__global__ void __launch_bounds__(CACHE_THREADS)
cache2_gather_fetch(const char* __restrict__ l2_rows, const char* __restrict__ store, int row_bytes,
                    const int64_t* __restrict__ fetch_keys, const int32_t* __restrict__ fetch_src,
                    const int64_t* __restrict__ counters2, int64_t capacity, char* __restrict__ fetched) {
  const int64_t n = list_len(counters2, MTS_CNT_INSERTED, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return fetch_src[k] >= 0 ? l2_rows + (int64_t)fetch_src[k] * row_bytes : store + fetch_keys[k] * row_bytes; },
            [&](int64_t k) { return fetched + k * row_bytes; });
}

// first-level victims to their second-level slot, or to the store when they have none and are dirty
__global__ void __launch_bounds__(CACHE_THREADS)
cache2_demote(const char* __restrict__ l1_rows, int row_bytes, const int64_t* __restrict__ ev1_keys,
              const int32_t* __restrict__ ev1_slots, const uint8_t* __restrict__ ev1_dirty,
              const int32_t* __restrict__ ev1_dst, const int64_t* __restrict__ counters2, int64_t capacity,
              char* __restrict__ l2_rows, char* __restrict__ store) {
  const int64_t n = list_len(counters2, MTS_CNT_EVICTED, capacity);
  copy_rows(n, row_bytes / 16,
            [&](int64_t k) { return l1_rows + (int64_t)ev1_slots[k] * row_bytes; },
            [&](int64_t k) -> char* {
              if (ev1_dst[k] >= 0) return l2_rows + (int64_t)ev1_dst[k] * row_bytes;
              return ev1_dirty[k] ? store + ev1_keys[k] * row_bytes : nullptr;
            });
}

struct Cache2Layout { size_t first, second, ev1_ts, ev1_freq, miss2_keys, miss2_slots, l2_counters, n_victims, bypass_dirty, total; };

static Cache2Layout cache2_layout(const mts_cache* l1, const mts_cache* l2, int64_t N, int64_t list_capacity) {
  Cache2Layout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t cap = (size_t)(list_capacity > 0 ? list_capacity : 1);
  L.first = take(cache_layout(l1, N).total);
  L.second = take(cache_layout(l2, list_capacity).total);
  L.ev1_ts = take(cap * 4); L.ev1_freq = take(cap * 4);
  L.miss2_keys = take(cap * 8); L.miss2_slots = take(cap * 4);
  L.l2_counters = take(MTS_NUM_COUNTERS * 8); L.n_victims = take(256); L.bypass_dirty = take(256);
  L.total = off;
  return L;
}

}  // namespace mts

extern "C" size_t mts_cache2_workspace_bytes(const mts_cache* l1, const mts_cache* l2, int64_t N, int64_t list_capacity) {
  if (!l1 || !l2 || N < 0 || list_capacity < 0) return 0;
  return cache2_layout(l1, l2, N, list_capacity).total;
}

extern "C" int mts_cache2_lookup_insert(mts_cache* l1, mts_cache* l2, const int64_t* keys, int64_t N, int64_t step,
                                        int32_t* slot_of_lookup, int64_t* fetch_keys, int32_t* fetch_slots,
                                        int32_t* fetch_src, int64_t* ev1_keys, int32_t* ev1_slots, uint8_t* ev1_dirty,
                                        int32_t* ev1_dst, int64_t* ev2_keys, int32_t* ev2_slots, uint8_t* ev2_dirty,
                                        int64_t* drop_keys, int32_t* drop_slots, uint8_t* drop_dirty,
                                        int64_t list_capacity, int64_t* counters2, void* workspace,
                                        size_t workspace_bytes, void* stream) {
  if (!l1 || !l2 || !counters2 || N < 0 || list_capacity < 1)
    return set_error(MTS_ERR_INVALID_ARG, "cache2_lookup_insert: bad argument");
  if (l1->row_bytes != l2->row_bytes || l1->key_space != l2->key_space || l1->dtype != l2->dtype)
    return set_error(MTS_ERR_INVALID_ARG, "cache2_lookup_insert: the two levels must hold the same rows (dim, dtype, key_space)");
  if (!fetch_src || !ev1_dst || !ev2_keys || !ev2_slots || !ev2_dirty || !drop_keys || !drop_slots || !drop_dirty)
    return set_error(MTS_ERR_INVALID_ARG, "cache2_lookup_insert: null list buffer");
  const Cache2Layout L = cache2_layout(l1, l2, N, list_capacity);
  if (!workspace || ((uintptr_t)workspace & 255))
    return set_error(MTS_ERR_ALIGNMENT, "cache2_lookup_insert: workspace must be non-null and 256-byte aligned");
  if (workspace_bytes < L.total)
    return set_error(MTS_ERR_WORKSPACE, "cache2_lookup_insert: workspace of %zu bytes, %zu needed", workspace_bytes, L.total);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  unsigned long long* bypass_dirty = reinterpret_cast<unsigned long long*>(ws + L.bypass_dirty);
  int64_t* l2_counters = reinterpret_cast<int64_t*>(ws + L.l2_counters);
  uint32_t* n_victims = reinterpret_cast<uint32_t*>(ws + L.n_victims);
  {
    LaunchScope scope(K_CACHE_PREPARE, s);
    cache2_begin<<<1, 32, 0, s>>>(counters2, bypass_dirty);
  }
  // first level: exactly the one-level pass; its list pass also resolves the second-level hits
  TwoLevelLists two;
  two.l2.tags = l2->tags; two.l2.ts = l2->ts; two.l2.placed = l2->placed; two.l2.freq = l2->freq; two.l2.dirty = l2->dirty;
  two.l2.S = (uint64_t)l2->S;
  two.fetch_src = fetch_src;
  two.drop_keys = drop_keys; two.drop_slots = drop_slots; two.drop_dirty = drop_dirty;
  two.ev1_ts = reinterpret_cast<int32_t*>(ws + L.ev1_ts);
  two.ev1_freq = reinterpret_cast<uint32_t*>(ws + L.ev1_freq);
  two.counters2 = reinterpret_cast<unsigned long long*>(counters2);
  KeySource src;
  src.keys = keys;
  int rc = lookup_insert_impl(l1, src, N, step, slot_of_lookup, fetch_keys, fetch_slots, ev1_keys, ev1_slots, ev1_dirty,
                              nullptr, list_capacity, 0, counters2, ws + L.first, cache_layout(l1, N).total, stream, nullptr,
                              InsertAttrs(), &two);
  if (rc != MTS_OK) return rc;
  if (N == 0) {
    return check_cuda(cudaMemsetAsync(counters2 + MTS_NUM_COUNTERS, 0, (MTS_NUM_COUNTERS2 - MTS_NUM_COUNTERS) * sizeof(int64_t), s),
                      "memset(counters2)");
  }
  // second level: the first level's victims enter with their timestamp, use count and dirty byte
  {
    LaunchScope scope(K_CACHE_PREPARE, s);
    cache2_victim_count<<<1, 32, 0, s>>>(counters2, list_capacity, n_victims);
  }
  InsertAttrs attrs;
  attrs.ts = two.ev1_ts; attrs.freq = two.ev1_freq; attrs.dirty = ev1_dirty;
  KeySource victims;
  victims.keys = ev1_keys;
  rc = lookup_insert_impl(l2, victims, list_capacity, step, ev1_dst, reinterpret_cast<int64_t*>(ws + L.miss2_keys),
                          reinterpret_cast<int32_t*>(ws + L.miss2_slots), ev2_keys, ev2_slots, ev2_dirty, nullptr,
                          list_capacity, 0, l2_counters, ws + L.second, cache_layout(l2, list_capacity).total, stream,
                          n_victims, attrs, nullptr, bypass_dirty);
  if (rc != MTS_OK) return rc;
  {
    LaunchScope scope(K_CACHE_LISTS, s);
    cache2_finish_counters<<<1, 32, 0, s>>>(l2_counters, bypass_dirty, counters2);
  }
  return check_launch("cache2_lookup_insert");
}

extern "C" int mts_cache2_move(mts_cache* l1, mts_cache* l2, void* host_store_mapped, const int64_t* fetch_keys,
                               const int32_t* fetch_slots, const int32_t* fetch_src, const int64_t* ev1_keys,
                               const int32_t* ev1_slots, const uint8_t* ev1_dirty, const int32_t* ev1_dst,
                               const int64_t* ev2_keys, const int32_t* ev2_slots, const uint8_t* ev2_dirty,
                               const int64_t* drop_keys, const int32_t* drop_slots, const uint8_t* drop_dirty,
                               int64_t list_capacity, const int64_t* counters2, void* fetch_staging, void* stream) {
  if (!l1 || !l2 || !host_store_mapped || !counters2 || list_capacity < 1 || !fetch_staging || !fetch_keys || !fetch_slots ||
      !fetch_src || !ev1_keys || !ev1_slots || !ev1_dirty || !ev1_dst || !ev2_keys || !ev2_slots || !ev2_dirty || !drop_keys ||
      !drop_slots || !drop_dirty)
    return set_error(MTS_ERR_INVALID_ARG, "cache2_move: null argument");
  if (((uintptr_t)host_store_mapped | (uintptr_t)fetch_staging) & 15)
    return set_error(MTS_ERR_ALIGNMENT, "cache2_move: buffers must be 16-byte aligned");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int grid = l1->sm_count * 8;
  const int rb = l1->row_bytes;
  char* store = static_cast<char*>(host_store_mapped);
  {
    LaunchScope scope(K_CACHE_WRITE_VICTIMS, s);
    cache2_rows_to_store<<<grid, CACHE_THREADS, 0, s>>>(l2->data, rb, ev2_keys, ev2_slots, ev2_dirty, counters2,
                                                        MTS_CNT2_L2_EVICTED, list_capacity, store);
  }
  {
    LaunchScope scope(K_CACHE_WRITE_VICTIMS, s);
    cache2_rows_to_store<<<grid, CACHE_THREADS, 0, s>>>(l2->data, rb, drop_keys, drop_slots, drop_dirty, counters2,
                                                        MTS_CNT2_L2_DROPPED, list_capacity, store);
  }
  {
    LaunchScope scope(K_CACHE_FETCH_MISSES, s);
    cache2_gather_fetch<<<grid, CACHE_THREADS, 0, s>>>(l2->data, store, rb, fetch_keys, fetch_src, counters2, list_capacity,
                                                       static_cast<char*>(fetch_staging));
  }
  {
    LaunchScope scope(K_CACHE_SAVE_VICTIMS, s);
    cache2_demote<<<grid, CACHE_THREADS, 0, s>>>(l1->data, rb, ev1_keys, ev1_slots, ev1_dirty, ev1_dst, counters2,
                                                 list_capacity, l2->data, store);
  }
  {
    LaunchScope scope(K_CACHE_FETCH_MISSES, s);
    cache_place_fetched<<<grid, CACHE_THREADS, 0, s>>>(l1->data, rb, static_cast<const char*>(fetch_staging), fetch_slots,
                                                       counters2, list_capacity);
  }
  return check_launch("cache2_move");
}

extern "C" int mts_cache_prefetch_misses(mts_cache* c, const void* host_rows_mapped, const int64_t* miss_keys,
                                         const int32_t* miss_slots, const int32_t* evict_slots,
                                         const uint8_t* evict_dirty, int64_t list_capacity, const int64_t* counters,
                                         void* evict_staging, void* stream) {
  if (!c || !host_rows_mapped || !counters || list_capacity < 0 ||
      (list_capacity > 0 && (!miss_keys || !miss_slots || !evict_slots || !evict_dirty || !evict_staging)))
    return set_error(MTS_ERR_INVALID_ARG, "cache_prefetch_misses: null argument");
  if (((uintptr_t)host_rows_mapped | (uintptr_t)evict_staging) & 15)
    return set_error(MTS_ERR_ALIGNMENT, "cache_prefetch_misses: buffers must be 16-byte aligned");
  if (list_capacity == 0) return MTS_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int grid = c->sm_count * 8;
  {
    LaunchScope scope(K_CACHE_SAVE_VICTIMS, s);
    cache_save_victims<<<grid, CACHE_THREADS, 0, s>>>(c->data, c->row_bytes, evict_slots, evict_dirty, counters,
                                                      list_capacity, static_cast<char*>(evict_staging));
  }
  {
    LaunchScope scope(K_CACHE_FETCH_MISSES, s);
#ifdef MTS_FETCH_PLAIN_LOADS
    cache_fetch_misses<<<grid, CACHE_THREADS, 0, s>>>(c->data, c->row_bytes, static_cast<const char*>(host_rows_mapped),
                                                      miss_keys, miss_slots, counters, list_capacity);
#else
    cache_fetch_misses_bulk<<<MTS_FETCH_BLOCKS, FETCH_THREADS, 0, s>>>(
        c->data, c->row_bytes, static_cast<const char*>(host_rows_mapped), miss_keys, miss_slots, counters,
        list_capacity, c->d_status, c->fetch_wait_limit);
#endif
  }
  return check_launch("cache_save_victims / cache_fetch_misses");
}

// Host-side row copy whose destination is not read again by this core: non-temporal 16-byte stores where the
// CPU has them and both sides are 16-byte multiples, so that the rows go to memory instead of filling the
// cores' caches (the copy engine, which reads the gathered rows next, would have to pull them out of there).
static inline void host_copy_row_streaming(char* dst, const char* src, size_t bytes) {
#if defined(__SSE2__)
  if ((((uintptr_t)dst | bytes) & 15) == 0) {
    for (size_t b = 0; b < bytes; b += 16)
      _mm_stream_si128(reinterpret_cast<__m128i*>(dst + b), _mm_loadu_si128(reinterpret_cast<const __m128i*>(src + b)));
    return;
  }
#endif
  memcpy(dst, src, bytes);
}

static inline void host_copy_fence() {
#if defined(__SSE2__)
  _mm_sfence();
#endif
}

// Host threads for the row copies, kept between calls (a gather of a few hundred thousand rows takes about a
// millisecond: starting sixteen threads for it would cost a good part of that).  One job at a time; the
// pieces of a job are handed out through a counter, so a thread that is held up costs one piece, not its share.
namespace {
class HostPool {
 public:
  static HostPool& get() { static HostPool p; return p; }
  // fn(k0, k1) over [0, n) in pieces of `grain`, on up to `threads` threads (the caller is one of them)
  template <class F>
  void run(int64_t n, int64_t grain, int threads, const F& fn) {
    const int64_t pieces = (n + grain - 1) / grain;
    const int helpers = (int)std::max<int64_t>(0, std::min<int64_t>(threads - 1, pieces - 1));
    if (helpers == 0) { fn(0, n); return; }
    std::lock_guard<std::mutex> job(job_mu_);
    auto body = [&](void) {
      for (;;) {
        const int64_t k0 = next_.fetch_add(grain, std::memory_order_relaxed);
        if (k0 >= n) break;
        fn(k0, std::min(n, k0 + grain));
      }
    };
    std::function<void(void)> erased = body;
    {
      std::unique_lock<std::mutex> lk(mu_);
      while ((int)workers_.size() < helpers) {
        const int id = (int)workers_.size();
        workers_.emplace_back([this, id] { worker(id); });
      }
      next_.store(0, std::memory_order_relaxed);
      body_ = &erased;
      helpers_ = helpers;
      pending_ = helpers;
      ++epoch_;
    }
    cv_work_.notify_all();
    body();
    std::unique_lock<std::mutex> lk(mu_);
    cv_done_.wait(lk, [this] { return pending_ == 0; });
    body_ = nullptr;
  }
  ~HostPool() {
    {
      std::lock_guard<std::mutex> lk(mu_);
      stop_ = true;
    }
    cv_work_.notify_all();
    for (auto& t : workers_) t.join();
  }

 private:
  void worker(int id) {
    uint64_t seen = 0;
    for (;;) {
      const std::function<void(void)>* body = nullptr;
      {
        std::unique_lock<std::mutex> lk(mu_);
        cv_work_.wait(lk, [&] { return stop_ || epoch_ != seen; });
        if (stop_) return;
        seen = epoch_;
        if (id >= helpers_) continue;          // this job uses fewer threads
        body = body_;
      }
      (*body)();
      {
        std::lock_guard<std::mutex> lk(mu_);
        --pending_;
      }
      cv_done_.notify_one();
    }
  }
  std::mutex job_mu_, mu_;
  std::condition_variable cv_work_, cv_done_;
  std::vector<std::thread> workers_;
  const std::function<void(void)>* body_ = nullptr;
  std::atomic<int64_t> next_{0};
  int helpers_ = 0, pending_ = 0;
  uint64_t epoch_ = 0;
  bool stop_ = false;
};
constexpr int64_t HOST_COPY_GRAIN = 512;      // rows per piece
// rows requested ahead of the copy and the cache level asked for (__builtin_prefetch locality): 32 rows into
// the outer levels gave the highest and steadiest rates on rows of 128 to 512 bytes (16 cores)
#ifndef MTS_HOST_PREFETCH_AHEAD
#define MTS_HOST_PREFETCH_AHEAD 32
#endif
#ifndef MTS_HOST_PREFETCH_LOCALITY
#define MTS_HOST_PREFETCH_LOCALITY 1
#endif
}  // namespace

extern "C" int mts_host_gather_rows(const void* host_rows, const int64_t* host_keys, int64_t n, int64_t row_bytes,
                                    void* host_out, int32_t threads) {
  if (n < 0 || row_bytes < 1 || (n > 0 && (!host_rows || !host_keys || !host_out)))
    return set_error(MTS_ERR_INVALID_ARG, "host_gather_rows: null argument or bad size");
  if (n == 0) return MTS_OK;
  const char* src = static_cast<const char*>(host_rows);
  char* dst = static_cast<char*>(host_out);
  const size_t rb = (size_t)row_bytes;
  auto work = [=](int64_t k0, int64_t k1) {
    constexpr int64_t AHEAD = MTS_HOST_PREFETCH_AHEAD;   // rows requested ahead of the copy: the reads are random DRAM accesses
    for (int64_t k = k0; k < k1; ++k) {
      if (k + AHEAD < n) {
        const char* ahead = src + (size_t)host_keys[k + AHEAD] * rb;
        for (size_t b = 0; b < rb; b += 64) __builtin_prefetch(ahead + b, 0, MTS_HOST_PREFETCH_LOCALITY);
      }
      host_copy_row_streaming(dst + (size_t)k * rb, src + (size_t)host_keys[k] * rb, rb);
    }
    host_copy_fence();
  };
  HostPool::get().run(n, HOST_COPY_GRAIN, threads, work);
  return MTS_OK;
}

extern "C" int mts_host_scatter_rows(void* host_rows, const int64_t* host_keys, const uint8_t* host_mask, int64_t n,
                                     int64_t row_bytes, const void* host_in, int32_t threads) {
  if (n < 0 || row_bytes < 1 || (n > 0 && (!host_rows || !host_keys || !host_in)))
    return set_error(MTS_ERR_INVALID_ARG, "host_scatter_rows: null argument or bad size");
  if (n == 0) return MTS_OK;
  char* dst = static_cast<char*>(host_rows);
  const char* src = static_cast<const char*>(host_in);
  const size_t rb = (size_t)row_bytes;
  auto work = [=](int64_t k0, int64_t k1) {
    for (int64_t k = k0; k < k1; ++k)
      if (host_mask == nullptr || host_mask[k]) host_copy_row_streaming(dst + (size_t)host_keys[k] * rb, src + (size_t)k * rb, rb);
    host_copy_fence();
  };
  HostPool::get().run(n, HOST_COPY_GRAIN, threads, work);
  return MTS_OK;
}

extern "C" int mts_cache_save_victims(mts_cache* c, const int32_t* evict_slots, const uint8_t* evict_dirty,
                                      int64_t list_capacity, const int64_t* counters, void* evict_staging,
                                      void* stream) {
  if (!c || !counters || list_capacity < 0 || (list_capacity > 0 && (!evict_slots || !evict_dirty || !evict_staging)))
    return set_error(MTS_ERR_INVALID_ARG, "cache_save_victims: null argument");
  if ((uintptr_t)evict_staging & 15)
    return set_error(MTS_ERR_ALIGNMENT, "cache_save_victims: the staging buffer must be 16-byte aligned");
  if (list_capacity == 0) return MTS_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    LaunchScope scope(K_CACHE_SAVE_VICTIMS, s);
    cache_save_victims<<<c->sm_count * 8, CACHE_THREADS, 0, s>>>(c->data, c->row_bytes, evict_slots, evict_dirty, counters,
                                                                 list_capacity, static_cast<char*>(evict_staging));
  }
  return check_launch("cache_save_victims");
}

extern "C" int mts_cache_place_fetched(mts_cache* c, const void* fetched, const int32_t* miss_slots,
                                       const int32_t* evict_slots, const uint8_t* evict_dirty, int64_t list_capacity,
                                       const int64_t* counters, void* evict_staging, void* stream) {
  if (!c || !counters || list_capacity < 0 || (list_capacity > 0 && (!fetched || !miss_slots)))
    return set_error(MTS_ERR_INVALID_ARG, "cache_place_fetched: null argument");
  if ((uintptr_t)fetched & 15)
    return set_error(MTS_ERR_ALIGNMENT, "cache_place_fetched: buffers must be 16-byte aligned");
  if (list_capacity == 0) return MTS_OK;
  if (evict_staging != nullptr) {
    const int rc = mts_cache_save_victims(c, evict_slots, evict_dirty, list_capacity, counters, evict_staging, stream);
    if (rc != MTS_OK) return rc;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    LaunchScope scope(K_CACHE_FETCH_MISSES, s);
    cache_place_fetched<<<c->sm_count * 8, CACHE_THREADS, 0, s>>>(c->data, c->row_bytes, static_cast<const char*>(fetched),
                                                                  miss_slots, counters, list_capacity);
  }
  return check_launch("cache_place_fetched");
}

extern "C" int mts_cache_writeback_evicted(mts_cache* c, void* host_rows_mapped, const int64_t* evict_keys,
                                           const uint8_t* evict_dirty, int64_t list_capacity,
                                           const int64_t* counters, const void* evict_staging, void* stream) {
  if (!c || !host_rows_mapped || !counters || list_capacity < 0 ||
      (list_capacity > 0 && (!evict_keys || !evict_dirty || !evict_staging)))
    return set_error(MTS_ERR_INVALID_ARG, "cache_writeback_evicted: null argument");
  if (((uintptr_t)host_rows_mapped | (uintptr_t)evict_staging) & 15)
    return set_error(MTS_ERR_ALIGNMENT, "cache_writeback_evicted: buffers must be 16-byte aligned");
  if (list_capacity == 0) return MTS_OK;
  {
    LaunchScope scope(K_CACHE_WRITE_VICTIMS, static_cast<cudaStream_t>(stream));
    cache_write_victims<<<c->sm_count * 8, CACHE_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<char*>(host_rows_mapped), c->row_bytes, evict_keys, evict_dirty, counters, list_capacity,
        static_cast<const char*>(evict_staging));
  }
  return check_launch("cache_write_victims");
}

extern "C" int mts_cache_refetch_overflowed(mts_cache* c, const void* host_rows_mapped, const int64_t* overflow_keys,
                                            int64_t list_capacity, const int64_t* counters, int64_t placed_step,
                                            void* stream) {
  if (!c || !host_rows_mapped || !counters || list_capacity < 0 || (list_capacity > 0 && !overflow_keys))
    return set_error(MTS_ERR_INVALID_ARG, "cache_refetch_overflowed: null argument");
  if ((uintptr_t)host_rows_mapped & 15) return set_error(MTS_ERR_ALIGNMENT, "cache_refetch_overflowed: host buffer alignment");
  if (list_capacity == 0) return MTS_OK;
  {
    LaunchScope scope(K_CACHE_FETCH_MISSES, static_cast<cudaStream_t>(stream));
    cache_refetch_resident<<<c->sm_count, CACHE_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
        c->data, c->row_bytes, static_cast<const char*>(host_rows_mapped), overflow_keys, counters, list_capacity,
        c->tags, c->placed, placed_step, (uint64_t)c->S);
  }
  return check_launch("cache_refetch_resident");
}

extern "C" int mts_cache_flush(mts_cache* c, void* host_rows_mapped, void* stream) {
  if (!c || !host_rows_mapped) return set_error(MTS_ERR_INVALID_ARG, "cache_flush: null argument");
  if ((uintptr_t)host_rows_mapped & 15) return set_error(MTS_ERR_ALIGNMENT, "cache_flush: host buffer alignment");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t n = c->S * MTS_CACHE_WAYS;
  {
    LaunchScope scope(K_CACHE_FLUSH, s);
    cache_flush_rows<<<c->sm_count * 8, CACHE_THREADS, 0, s>>>(c->data, c->row_bytes, c->tags, c->dirty, n,
                                                               static_cast<char*>(host_rows_mapped));
  }
  {
    LaunchScope scope(K_CACHE_FLUSH, s);
    cache_clear_dirty<<<c->sm_count * 4, 256, 0, s>>>(c->dirty, n);
  }
  return check_launch("cache_flush");
}

namespace mts {
__global__ void cache_import(const int64_t* __restrict__ i_tags, const int64_t* __restrict__ i_ts,
                             const int64_t* __restrict__ i_freq, const uint8_t* __restrict__ i_dirty, int64_t n,
                             uint32_t* tags, int32_t* ts, int32_t* placed, uint32_t* freq, uint8_t* dirty) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const bool free_way = i_tags[i] < 0;
    tags[i] = free_way ? FREE_TAG : (uint32_t)i_tags[i];
    ts[i] = free_way ? -1 : (int32_t)i_ts[i];
    placed[i] = ts[i];            // inserted no later than its last use: never equal to a later call's step
    freq[i] = free_way ? 0u : (uint32_t)i_freq[i];
    dirty[i] = free_way ? 0 : i_dirty[i];
  }
}

__global__ void __launch_bounds__(CACHE_THREADS)
cache_refill_rows(char* __restrict__ data, int row_bytes, const uint32_t* __restrict__ tags, int64_t n_slots,
                  const char* __restrict__ host_rows) {
  copy_rows(n_slots, row_bytes / 16,
            [&](int64_t s) { return tags[s] != FREE_TAG ? host_rows + (int64_t)tags[s] * row_bytes : nullptr; },
            [&](int64_t s) { return data + s * row_bytes; });
}
}  // namespace mts

extern "C" int mts_cache_import_state(mts_cache* c, const int64_t* tags, const int64_t* timestamps, const int64_t* counts,
                                      const uint8_t* dirty, const void* host_rows_mapped, void* stream) {
  if (!c || !tags || !timestamps || !counts || !dirty || !host_rows_mapped)
    return set_error(MTS_ERR_INVALID_ARG, "cache_import_state: null argument");
  if ((uintptr_t)host_rows_mapped & 15) return set_error(MTS_ERR_ALIGNMENT, "cache_import_state: host buffer alignment");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t n = c->S * MTS_CACHE_WAYS;
  {
    LaunchScope scope(K_OTHER, s);
    cache_import<<<c->sm_count * 4, 256, 0, s>>>(tags, timestamps, counts, dirty, n, c->tags, c->ts, c->placed, c->freq,
                                                 c->dirty);
  }
  {
    LaunchScope scope(K_CACHE_FETCH_MISSES, s);
    cache_refill_rows<<<c->sm_count * 8, CACHE_THREADS, 0, s>>>(c->data, c->row_bytes, c->tags, n,
                                                                static_cast<const char*>(host_rows_mapped));
  }
  return check_launch("cache_import_state");
}

extern "C" int mts_cache_set_fetch_wait_limit(mts_cache* c, int64_t polls) {
  if (!c || polls < 0 || polls > (1ll << 22)) return set_error(MTS_ERR_INVALID_ARG, "cache_set_fetch_wait_limit: 0 .. 2^22 polls");
  c->fetch_wait_limit = (uint32_t)polls;
  return MTS_OK;
}

extern "C" int mts_cache_export_state(mts_cache* c, int64_t* tags, int64_t* timestamps, int64_t* counts,
                                      uint8_t* dirty, void* stream) {
  if (!c) return set_error(MTS_ERR_INVALID_ARG, "cache_export_state: null cache");
  {
    LaunchScope scope(K_OTHER, static_cast<cudaStream_t>(stream));
    cache_export<<<c->sm_count * 4, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        c->tags, c->ts, c->freq, c->dirty, c->S * MTS_CACHE_WAYS, tags, timestamps, counts, dirty);
  }
  return check_launch("cache_export");
}
