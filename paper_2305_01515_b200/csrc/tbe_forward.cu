// Pooled multi-table embedding lookup (Section 2.1.1 of the paper: an embedding operator
// selects rows of a table and pools them).  One warp per bag (table t, sample b) at a time; a row of
// vec16 16-byte chunks is read by a group of G = pow2(vec16) lanes, so 32 / G rows are in
// flight per load instruction and UNROLL of those instructions are issued back to back.
// Accumulation in fp32 registers, one 16-byte store per lane group member at the end.
#include <type_traits>

#include <cuda_bf16.h>

#include "common.cuh"

namespace mts {

#ifndef MTS_FWD_UNROLL
#define MTS_FWD_UNROLL 4         // load instructions issued back to back per lane
#endif
#ifndef MTS_FWD_MINBLK
#define MTS_FWD_MINBLK 8         // resident blocks per SM the register allocation is bounded for
#endif
#ifndef MTS_FWD_BAGS
#define MTS_FWD_BAGS 4           // consecutive bags one warp walks through
#endif
#ifndef MTS_FWD_WARPS
#define MTS_FWD_WARPS 4
#endif
constexpr int FWD_WARPS = MTS_FWD_WARPS;
constexpr int FWD_UNROLL = MTS_FWD_UNROLL;
constexpr int FWD_BAGS = MTS_FWD_BAGS;
static_assert(FWD_BAGS >= 1 && FWD_BAGS <= 30, "a warp keeps the offsets of its bags in its lanes");

// Pooled values leave as fp32, IEEE binary16 or bfloat16 (round to nearest even).
enum OutKind { OUT_F32 = 0, OUT_F16 = 1, OUT_BF16 = 2 };

// One lane's EPC consecutive pooled values (already scaled) to element offset `o` of `out`.
template <int EPC>
__device__ __forceinline__ void store_pooled(void* __restrict__ out, int out_kind, int64_t o, const float (&v)[EPC]) {
  if (out_kind == OUT_F32) {
    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(out) + o);
    dst[0] = make_float4(v[0], v[1], v[2], v[3]);
    if (EPC == 8) dst[1] = make_float4(v[4], v[5], v[6], v[7]);
    return;
  }
  uint32_t w[EPC / 2];
#pragma unroll
  for (int e = 0; e < EPC / 2; ++e) {
    if (out_kind == OUT_F16) {
      __half2 h = __floats2half2_rn(v[2 * e], v[2 * e + 1]);
      w[e] = *reinterpret_cast<uint32_t*>(&h);
    } else {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
      w[e] = *reinterpret_cast<uint32_t*>(&h);
    }
  }
  uint16_t* dst = static_cast<uint16_t*>(out) + o;
  *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
  if (EPC == 8) *reinterpret_cast<uint2*>(dst + 4) = make_uint2(w[2], w[3]);
}

// max pooling: acc = max(acc, value) per column; a piece that is not loaded is filled with -infinity
__device__ __forceinline__ void max_half8(float* acc, const uint4& v) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 f = __half22float2(h[e]);
    acc[2 * e] = fmaxf(acc[2 * e], f.x);
    acc[2 * e + 1] = fmaxf(acc[2 * e + 1], f.y);
  }
}
__device__ __forceinline__ void max_float4(float* acc, const uint4& v) {
  acc[0] = fmaxf(acc[0], __uint_as_float(v.x));
  acc[1] = fmaxf(acc[1], __uint_as_float(v.y));
  acc[2] = fmaxf(acc[2], __uint_as_float(v.z));
  acc[3] = fmaxf(acc[3], __uint_as_float(v.w));
}

// A warp walks FWD_BAGS consecutive bags.  Their offsets are read with one load, and the first 32
// indices of the next bag are requested before the rows of the current bag, so that a bag costs
// about one memory round trip (its rows) instead of three (offsets, indices, rows).
template <bool FP16, int NV, bool MAXP>
__global__ void __launch_bounds__(FWD_WARPS * 32, (NV == 1 ? MTS_FWD_MINBLK : 1))
tbe_forward_kernel(const TableMeta* __restrict__ meta, int64_t n_bags, int32_t B,
                   const int64_t* __restrict__ indices, const int64_t* __restrict__ offsets,
                   const int32_t* __restrict__ slot_of_lookup, const __grid_constant__ CachePtrs caches,
                   const char* __restrict__ dev_w, const char* __restrict__ host_w,
                   int32_t pooling_mode, void* __restrict__ out, int out_kind, int64_t out_stride,
                   int32_t* status) {
  constexpr int EPC = FP16 ? 8 : 4;       // elements per 16-byte chunk
  constexpr int EB = FP16 ? 2 : 4;
  // what an accumulator starts from and a piece that is not loaded holds: 0, or -infinity for max pooling
  const float acc0 = MAXP ? __uint_as_float(0xff800000u) : 0.f;
  const uint32_t pad = MAXP ? (FP16 ? 0xfc00fc00u : 0xff800000u) : 0u;
  const int lane = threadIdx.x & 31;
  const int64_t bag0 = ((int64_t)blockIdx.x * FWD_WARPS + (threadIdx.x >> 5)) * FWD_BAGS;
  if (bag0 >= n_bags) return;
  const int nb = (int)min((int64_t)FWD_BAGS, n_bags - bag0);
  // lane k holds the start of bag k of this warp, lane nb the end of the last one
  const int64_t my_off = offsets[bag0 + min(lane, nb)];
  int64_t i1 = __shfl_sync(0xffffffffu, my_off, 0);
  // table and sample of the warp's first bag; the following bags step from there (no division per bag)
  int32_t t = (int32_t)(bag0 / B);
  int32_t b = (int32_t)(bag0 - (int64_t)t * B);
  // per-table values, refreshed only when the walk crosses into the next table
  TableMeta m = meta[t];
  // first indices (and cache slots) of the first bag
  int64_t pf_idx = 0;
  int32_t pf_slot = -1;
  {
    const int64_t e = __shfl_sync(0xffffffffu, my_off, 1);
    if (i1 + lane < e) {
      pf_idx = indices[i1 + lane];
      if (m.cache_id >= 0) pf_slot = slot_of_lookup[i1 + lane];
    }
  }

  int32_t t_cur = -1;
  int vec16 = 0, logG = 0, G = 1, R = 32, sub = 0, cl = 0;
  int64_t row_bytes = 0;
  const char* table_base = nullptr;
  const char* cache_base = nullptr;
  for (int k = 0; k < nb; ++k, ++b) {
    if (b == B) { b = 0; ++t; }
    if (t != t_cur) {
      t_cur = t;
      m = meta[t];
      vec16 = m.vec16;
      // lanes per row: smallest power of two >= vec16, at most 32
      logG = 0;
      while ((1 << logG) < vec16 && logG < 5) ++logG;
      G = 1 << logG;
      R = 32 >> logG;               // rows per load instruction
      sub = lane >> logG;
      cl = lane & (G - 1);
      row_bytes = (int64_t)m.dim * EB;
      table_base = (m.cache_id < 0 ? dev_w : host_w) + m.weight_offset * EB;
      cache_base = m.cache_id >= 0 ? static_cast<const char*>(caches.data[m.cache_id]) : nullptr;
    }
    const int64_t i0 = i1;
    i1 = __shfl_sync(0xffffffffu, my_off, k + 1);
    const int64_t cur_idx = pf_idx;
    const int32_t cur_slot = pf_slot;
    if (k + 1 < nb) {
      const int64_t e = __shfl_sync(0xffffffffu, my_off, k + 2);
      pf_slot = -1;
      if (i1 + lane < e) {
        pf_idx = indices[i1 + lane];
        const int32_t next_cache = b + 1 == B ? meta[t + 1].cache_id : m.cache_id;
        if (next_cache >= 0) pf_slot = slot_of_lookup[i1 + lane];
      }
    }

    float acc[NV][EPC];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
      for (int e = 0; e < EPC; ++e) acc[v][e] = acc0;

    for (int64_t base = i0; base < i1; base += 32) {
      const int cnt = (int)min((int64_t)32, i1 - base);
      const char* my_ptr = table_base;
      if (lane < cnt) {
        const bool first = base == i0;
        const int64_t idx = clamp_index(first ? cur_idx : indices[base + lane], m.rows, status);
        my_ptr = table_base + idx * row_bytes;
        if (cache_base != nullptr) {
          const int32_t s = first ? cur_slot : slot_of_lookup[base + lane];
          if (s >= 0) my_ptr = cache_base + (int64_t)s * row_bytes;
        }
      }
      // `whole` = the row is exactly G pieces wide (a power of two, at most 32): every lane of a
      // group has a piece, no column test
      auto rows = [&](auto whole) {
        constexpr bool WHOLE = decltype(whole)::value;
        for (int r = 0; r < cnt; r += R * FWD_UNROLL) {
          uint4 v[FWD_UNROLL][NV];
#pragma unroll
          for (int u = 0; u < FWD_UNROLL; ++u) {
            const int j = r + u * R + sub;
            const unsigned long long p =
                __shfl_sync(0xffffffffu, (unsigned long long)(uintptr_t)my_ptr, j & 31);
            const bool valid = j < cnt;
#pragma unroll
            for (int q = 0; q < (WHOLE ? 1 : NV); ++q) {
              const int c = cl + q * 32;
              if (valid && (WHOLE || c < vec16)) v[u][q] = ld_nc_16(reinterpret_cast<const char*>(p) + (int64_t)c * 16);
              else v[u][q] = make_uint4(pad, pad, pad, pad);
            }
          }
#pragma unroll
          for (int u = 0; u < FWD_UNROLL; ++u)
#pragma unroll
            for (int q = 0; q < (WHOLE ? 1 : NV); ++q) {
              if (MAXP) {
                if (FP16) max_half8(acc[q], v[u][q]);
                else max_float4(acc[q], v[u][q]);
              } else {
                if (FP16) add_half8(acc[q], v[u][q]);
                else add_float4(acc[q], v[u][q]);
              }
            }
        }
      };
      if (vec16 == G) rows(std::true_type{});
      else rows(std::false_type{});
    }
    // fold the row groups of the warp together
    for (int o = G; o < 32; o <<= 1) {
#pragma unroll
      for (int q = 0; q < NV; ++q)
#pragma unroll
        for (int e = 0; e < EPC; ++e) {
          const float other = __shfl_xor_sync(0xffffffffu, acc[q][e], o);
          acc[q][e] = MAXP ? fmaxf(acc[q][e], other) : acc[q][e] + other;
        }
    }
    if (sub == 0) {
      float scale = 1.f;
      if (pooling_mode == MTS_POOL_MEAN && i1 > i0) scale = 1.f / (float)(i1 - i0);
      const int64_t o = (int64_t)b * out_stride + m.out_offset;     // element offset of the bag's slice
#pragma unroll
      for (int q = 0; q < NV; ++q) {
        const int c = cl + q * 32;
        if (c < vec16) {
          float r[EPC];
#pragma unroll
          for (int e = 0; e < EPC; ++e) r[e] = MAXP ? (i1 > i0 ? acc[q][e] : 0.f) : acc[q][e] * scale;
          store_pooled<EPC>(out, out_kind, o + c * EPC, r);
        }
      }
    }
  }
}

template <bool FP16, int NV>
static int launch_forward(const mts_tables* h, int32_t B, const int64_t* indices, const int64_t* offsets,
                          int32_t pooling_mode, const int32_t* slot_of_lookup, const CachePtrs& caches,
                          void* out, int out_kind, int64_t out_stride, cudaStream_t stream) {
  const int64_t n_bags = (int64_t)h->T * B;
  const int64_t grid = ceil_div(n_bags, (int64_t)FWD_WARPS * FWD_BAGS);
  {
    LaunchScope scope(K_FORWARD, stream);
    if (pooling_mode == MTS_POOL_MAX)
      tbe_forward_kernel<FP16, NV, true><<<(unsigned)grid, FWD_WARPS * 32, 0, stream>>>(
          h->d_meta, n_bags, B, indices, offsets, slot_of_lookup, caches,
          static_cast<const char*>(h->dev_weights), static_cast<const char*>(h->host_weights), pooling_mode,
          out, out_kind, out_stride, h->d_status);
    else
      tbe_forward_kernel<FP16, NV, false><<<(unsigned)grid, FWD_WARPS * 32, 0, stream>>>(
          h->d_meta, n_bags, B, indices, offsets, slot_of_lookup, caches,
          static_cast<const char*>(h->dev_weights), static_cast<const char*>(h->host_weights), pooling_mode,
          out, out_kind, out_stride, h->d_status);
  }
  return check_launch("tbe_forward_kernel");
}

// ---- tbe_forward_lean: the same walk when a row is at most 32 16-byte pieces.  The walk is bound by latency
// and instruction issue, not by bytes in flight, so this form trades loads in flight per warp for resident
// warps: positions and row numbers are 32-bit and the register allocation is bounded for MTS_FWD_LEAN_MINBLK
// blocks per SM.  Same summation order and arithmetic as tbe_forward_kernel (bit-identical results).
// CACHED: tables may sit behind a cache.  A lookup of such a table reads its cache slot instead of its index
// (the row is cache_data[slot]); only a lookup without a slot (slot < 0: the row is read from the host tier)
// reads the index too, and a batch of 32 lookups that has one takes a slower form of the inner loop.  An
// out-of-range index of a cached table is reported by the cache's lookup, not here.
#ifndef MTS_FWD_LEAN
#define MTS_FWD_LEAN 1
#endif
#ifndef MTS_FWD_LEAN_MINBLK
#define MTS_FWD_LEAN_MINBLK 16    // 64 warps per SM: 32 registers a thread
#endif
#ifndef MTS_FWD_LEAN_UNROLL
#define MTS_FWD_LEAN_UNROLL 1    // load instructions issued back to back per lane
#endif
constexpr int LEAN_UNROLL = MTS_FWD_LEAN_UNROLL;

template <bool FP16, bool CACHED>
__global__ void __launch_bounds__(FWD_WARPS * 32, MTS_FWD_LEAN_MINBLK)
tbe_forward_lean(const TableMeta* __restrict__ meta, int32_t n_bags, int32_t B,
                 const int64_t* __restrict__ indices, const int64_t* __restrict__ offsets,
                 const int32_t* __restrict__ slot_of_lookup, const __grid_constant__ CachePtrs caches,
                 const char* __restrict__ dev_w, const char* __restrict__ host_w, int32_t pooling_mode,
                 void* __restrict__ out, int out_kind, int64_t out_stride, int32_t* status) {
  constexpr int EPC = FP16 ? 8 : 4;       // elements per 16-byte chunk
  constexpr int EB = FP16 ? 2 : 4;
  const int lane = threadIdx.x & 31;
  const int32_t bag0 = (int32_t)((blockIdx.x * FWD_WARPS + (threadIdx.x >> 5)) * FWD_BAGS);
  if (bag0 >= n_bags) return;
  const int nb = min(FWD_BAGS, n_bags - bag0);
  // lane k holds the start of bag k of this warp, lane nb the end of the last one
  const uint32_t my_off = (uint32_t)offsets[bag0 + min(lane, nb)];
  uint32_t i1 = __shfl_sync(0xffffffffu, my_off, 0);
  int32_t t = (int32_t)((uint32_t)bag0 / (uint32_t)B);
  int32_t b = bag0 - t * B;
  // what a lookup's row is found by: its cache slot (cached table) or its index
  auto reference = [&](uint32_t i, bool cached) -> int64_t {
    return (CACHED && cached) ? (int64_t)slot_of_lookup[i] : indices[i];
  };
  // first references of the first bag
  int64_t pf_ref = 0;
  {
    const uint32_t e = __shfl_sync(0xffffffffu, my_off, 1);
    if (i1 + lane < e) pf_ref = reference(i1 + lane, CACHED && meta[t].cache_id >= 0);
  }
  // per-table values, refreshed only when the walk crosses into the next table
  int32_t t_cur = -1;
  int vec16 = 0, logG = 0, row_bytes = 0, out_offset = 0;
  uint32_t rows = 0;
  bool cached = false;
  const char* lane_base = nullptr;        // the lane's 16-byte piece of row 0 (of the table, or of the cache's slot 0)
  for (int k = 0; k < nb; ++k, ++b) {
    if (b == B) { b = 0; ++t; }
    if (t != t_cur) {
      t_cur = t;
      const TableMeta m = meta[t];
      vec16 = m.vec16;
      logG = 0;
      while ((1 << logG) < vec16) ++logG;   // lanes per row: smallest power of two >= vec16 (vec16 <= 32 here)
      row_bytes = m.dim * EB;
      rows = (uint32_t)m.rows;
      out_offset = m.out_offset;
      cached = CACHED && m.cache_id >= 0;
      lane_base = (cached ? static_cast<const char*>(caches.data[m.cache_id]) : dev_w + m.weight_offset * EB) +
                  (lane & ((1 << logG) - 1)) * 16;
    }
    const int R = 32 >> logG;               // rows per load instruction
    const int sub = lane >> logG;
    const int cl = lane & ((1 << logG) - 1);
    const uint32_t i0 = i1;
    i1 = __shfl_sync(0xffffffffu, my_off, k + 1);
    const int64_t cur_ref = pf_ref;
    if (k + 1 < nb) {
      const uint32_t e = __shfl_sync(0xffffffffu, my_off, k + 2);
      if (i1 + lane < e) {
        bool next_cached = cached;
        if (CACHED && b + 1 == B) next_cached = meta[t + 1].cache_id >= 0;
        pf_ref = reference(i1 + lane, next_cached);
      }
    }

    float acc[EPC];
#pragma unroll
    for (int e = 0; e < EPC; ++e) acc[e] = 0.f;

    for (uint32_t base = i0; base < i1; base += 32) {
      const int cnt = (int)min(32u, i1 - base);
      uint32_t my_row = 0;
      bool no_slot = false;                 // cached table, lookup without a slot: my_row is a row of the host tier
      if (lane < cnt) {
        int64_t ref = base == i0 ? cur_ref : reference(base + lane, cached);
        if (CACHED && cached) {
          no_slot = ref < 0;
          if (no_slot) ref = indices[base + lane];
        }
        if (!(CACHED && cached) || no_slot) {
          if (ref < 0 || ref >= (int64_t)rows) {
            atomicOr(status, STATUS_INDEX_CLAMPED);
            ref = ref < 0 ? 0 : (int64_t)rows - 1;
          }
        }
        my_row = (uint32_t)ref;
      }
      const uint32_t no_slot_mask = CACHED ? __ballot_sync(0xffffffffu, no_slot) : 0u;
      auto walk = [&](auto whole, auto mixed) {
        constexpr bool WHOLE = decltype(whole)::value;
        constexpr bool MIXED = decltype(mixed)::value;      // some lookups of the batch read the host tier
        const char* host_base = nullptr;
        if (MIXED) host_base = host_w + meta[t].weight_offset * EB + cl * 16;
        for (int r = 0; r < cnt; r += R * LEAN_UNROLL) {
          uint4 v[LEAN_UNROLL];
#pragma unroll
          for (int u = 0; u < LEAN_UNROLL; ++u) {
            const int j = r + u * R + sub;
            const uint32_t row = __shfl_sync(0xffffffffu, my_row, j & 31);
            const char* from = (MIXED && ((no_slot_mask >> (j & 31)) & 1u)) ? host_base : lane_base;
            if (j < cnt && (WHOLE || cl < vec16)) v[u] = ld_nc_16(from + (int64_t)row * row_bytes);
            else v[u] = make_uint4(0u, 0u, 0u, 0u);
          }
#pragma unroll
          for (int u = 0; u < LEAN_UNROLL; ++u) {
            if (FP16) add_half8(acc, v[u]);
            else add_float4(acc, v[u]);
          }
        }
      };
      if (CACHED && no_slot_mask != 0u) {
        if (vec16 == (1 << logG)) walk(std::true_type{}, std::true_type{});
        else walk(std::false_type{}, std::true_type{});
      } else {
        if (vec16 == (1 << logG)) walk(std::true_type{}, std::false_type{});
        else walk(std::false_type{}, std::false_type{});
      }
    }
    // fold the row groups of the warp together
    for (int o = 1 << logG; o < 32; o <<= 1) {
#pragma unroll
      for (int e = 0; e < EPC; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    }
    if (sub == 0 && cl < vec16) {
      float scale = 1.f;
      if (pooling_mode == MTS_POOL_MEAN && i1 > i0) scale = 1.f / (float)(i1 - i0);
      const int64_t o = (int64_t)b * out_stride + out_offset + cl * EPC;     // first element of the lane's piece
      float r[EPC];
#pragma unroll
      for (int e = 0; e < EPC; ++e) r[e] = acc[e] * scale;
      store_pooled<EPC>(out, out_kind, o, r);
    }
  }
}

template <bool FP16>
static int launch_forward_lean(const mts_tables* h, int32_t B, const int64_t* indices, const int64_t* offsets,
                               int32_t pooling_mode, const int32_t* slot_of_lookup, const CachePtrs& caches,
                               void* out, int out_kind, int64_t out_stride, cudaStream_t stream) {
  const int64_t n_bags = (int64_t)h->T * B;
  const int64_t grid = ceil_div(n_bags, (int64_t)FWD_WARPS * FWD_BAGS);
  {
    LaunchScope scope(K_FORWARD, stream);
    if (h->any_cached)
      tbe_forward_lean<FP16, true><<<(unsigned)grid, FWD_WARPS * 32, 0, stream>>>(
          h->d_meta, (int32_t)n_bags, B, indices, offsets, slot_of_lookup, caches, static_cast<const char*>(h->dev_weights),
          static_cast<const char*>(h->host_weights), pooling_mode, out, out_kind, out_stride, h->d_status);
    else
      tbe_forward_lean<FP16, false><<<(unsigned)grid, FWD_WARPS * 32, 0, stream>>>(
          h->d_meta, (int32_t)n_bags, B, indices, offsets, slot_of_lookup, caches, static_cast<const char*>(h->dev_weights),
          static_cast<const char*>(h->host_weights), pooling_mode, out, out_kind, out_stride, h->d_status);
  }
  return check_launch("tbe_forward_lean");
}

int fill_cache_ptrs(const mts_tables* h, void* const* host_cache_data, uint8_t* const* host_cache_dirty,
                    int32_t n_caches, const int32_t* slot_of_lookup, CachePtrs* out) {
  for (int c = 0; c < MTS_MAX_CACHES; ++c) { out->data[c] = nullptr; out->dirty[c] = nullptr; }
  if (!h->any_cached) return MTS_OK;
  if (!slot_of_lookup || !host_cache_data || n_caches < h->n_cache_ids || n_caches > MTS_MAX_CACHES)
    return set_error(MTS_ERR_INVALID_ARG,
                     "cached tables need slot_of_lookup and %d cache data pointers (got %d)",
                     h->n_cache_ids, n_caches);
  for (int c = 0; c < n_caches; ++c) {
    if (!host_cache_data[c] || ((uintptr_t)host_cache_data[c] & 15))
      return set_error(MTS_ERR_ALIGNMENT, "cache %d: data pointer null or not 16-byte aligned", c);
    out->data[c] = host_cache_data[c];
    out->dirty[c] = host_cache_dirty ? host_cache_dirty[c] : nullptr;
  }
  return MTS_OK;
}

}  // namespace mts

using namespace mts;

namespace {
int forward_any(const mts_tables* h, int32_t B, const int64_t* indices, const int64_t* offsets, int64_t N,
                int32_t pooling_mode, const int32_t* slot_of_lookup, void* const* host_cache_data, int32_t n_caches,
                void* out, int out_kind, int64_t out_stride, void* stream) {
  if (!h || !offsets || !out || B < 1 || N < 0 || (N > 0 && !indices))
    return set_error(MTS_ERR_INVALID_ARG, "tbe_forward: null argument or bad size");
  if (pooling_mode != MTS_POOL_SUM && pooling_mode != MTS_POOL_MEAN && pooling_mode != MTS_POOL_MAX)
    return set_error(MTS_ERR_INVALID_ARG, "tbe_forward: pooling mode %d", pooling_mode);
  if (out_stride < h->total_dim || (out_stride & 3) || ((uintptr_t)out & 15))
    return set_error(MTS_ERR_ALIGNMENT, "tbe_forward: out must be 16-byte aligned, out_stride >= %d and a multiple of 4",
                     h->total_dim);
  if ((int64_t)h->T * B >= (1ll << 31) * FWD_WARPS)
    return set_error(MTS_ERR_UNSUPPORTED, "tbe_forward: too many bags");
  CachePtrs caches;
  int rc = fill_cache_ptrs(h, host_cache_data, nullptr, n_caches, slot_of_lookup, &caches);
  if (rc != MTS_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int max_vec = h->max_dim * h->elem_bytes / 16;
  const int nv = max_vec <= 32 ? 1 : max_vec <= 64 ? 2 : max_vec <= 128 ? 4 : 8;
  const bool fp16 = h->dtype == MTS_DTYPE_FP16;
#if MTS_FWD_LEAN
  // positions and bag numbers fit 32 bits (row numbers always do), rows of at most 32 pieces
  if (nv == 1 && pooling_mode != MTS_POOL_MAX && N < (1ll << 31) &&
      (int64_t)h->T * B < (1ll << 31) - FWD_WARPS * FWD_BAGS) {
    if (fp16) return launch_forward_lean<true>(h, B, indices, offsets, pooling_mode, slot_of_lookup, caches, out, out_kind, out_stride, s);
    return launch_forward_lean<false>(h, B, indices, offsets, pooling_mode, slot_of_lookup, caches, out, out_kind, out_stride, s);
  }
#endif
#define MTS_FWD(F, V) return launch_forward<F, V>(h, B, indices, offsets, pooling_mode, slot_of_lookup, caches, out, out_kind, out_stride, s)
  if (fp16) {
    if (nv == 1) MTS_FWD(true, 1);
    if (nv == 2) MTS_FWD(true, 2);
    MTS_FWD(true, 4);
  } else {
    if (nv == 1) MTS_FWD(false, 1);
    if (nv == 2) MTS_FWD(false, 2);
    if (nv == 4) MTS_FWD(false, 4);
    MTS_FWD(false, 8);
  }
#undef MTS_FWD
}
}  // namespace

extern "C" int mts_tbe_forward(const mts_tables* h, int32_t B, const int64_t* indices,
                               const int64_t* offsets, int64_t N, int32_t pooling_mode,
                               const int32_t* slot_of_lookup, void* const* host_cache_data,
                               int32_t n_caches, float* out, int64_t out_stride, void* stream) {
  return forward_any(h, B, indices, offsets, N, pooling_mode, slot_of_lookup, host_cache_data, n_caches, out, OUT_F32,
                     out_stride, stream);
}

extern "C" int mts_tbe_forward_f16(const mts_tables* h, int32_t B, const int64_t* indices,
                                   const int64_t* offsets, int64_t N, int32_t pooling_mode,
                                   const int32_t* slot_of_lookup, void* const* host_cache_data,
                                   int32_t n_caches, void* out_f16, int64_t out_stride, void* stream) {
  return forward_any(h, B, indices, offsets, N, pooling_mode, slot_of_lookup, host_cache_data, n_caches, out_f16, OUT_F16,
                     out_stride, stream);
}

extern "C" int mts_tbe_forward_bf16(const mts_tables* h, int32_t B, const int64_t* indices,
                                    const int64_t* offsets, int64_t N, int32_t pooling_mode,
                                    const int32_t* slot_of_lookup, void* const* host_cache_data,
                                    int32_t n_caches, void* out_bf16, int64_t out_stride, void* stream) {
  return forward_any(h, B, indices, offsets, N, pooling_mode, slot_of_lookup, host_cache_data, n_caches, out_bf16, OUT_BF16,
                     out_stride, stream);
}
