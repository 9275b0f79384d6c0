// Backward of the pooled lookup fused with row-wise Adagrad on the touched rows (Section 2.1.2:
// optimizer with few states per row; Section 5.9: aggregate, optimize, write rows back).
//
// Steps, all on the caller's stream, no host synchronisation:
//   1. linearize_lookups : key = linear row id of every lookup, value = its position and
//                          bag_of_pos[position] = bag id (value = bag id when no table is cached)
//   2. radix_sort_pairs  : stable sort by key; equal rows keep ascending position
//   3. reduce_chunks     : one warp per CHUNK consecutive sorted lookups.  Gradients of a row
//                          are summed in sorted order; a row whose lookups lie inside the
//                          chunk is updated at once (Adagrad fused); the piece of a row that
//                          continues over a chunk border is written as a partial sum
//   4. combine_partials  : the chunk in which such a row starts adds the partial sums in
//                          chunk order and applies the update
// The summation tree depends only on the sorted order and CHUNK, so two runs give the same
// bits.  No thread ever writes a word another thread of the same launch writes.
#include <algorithm>
#include <mutex>
#include <type_traits>

#include "common.cuh"

namespace mts {

#ifndef MTS_BWD_CHUNK
#define MTS_BWD_CHUNK 128
#endif
#ifndef MTS_BWD_GROUP1
#define MTS_BWD_GROUP1 4        // lookups whose loads are issued together when a row fits one warp pass
#endif
#ifndef MTS_BWD_USE_LEAN
#define MTS_BWD_USE_LEAN 1      // rows of up to 128 columns take reduce_chunks_lean
#endif
#ifndef MTS_BWD_LEAN_WARPS
#define MTS_BWD_LEAN_WARPS 4
#endif
#ifndef MTS_BWD_LEAN_RUN
#define MTS_BWD_LEAN_RUN 4      // gradient loads issued together inside a run of lookups of one row
#endif
#ifndef MTS_BWD_LEAN_MINBLK
#define MTS_BWD_LEAN_MINBLK 16  // resident blocks per SM reduce_chunks_lean is bounded for (32 registers)
#endif
#ifndef MTS_BWD_LEAN_MINBLK2
#define MTS_BWD_LEAN_MINBLK2 12 // the same for its two-piece form (rows of 129..256 columns)
#endif
#ifndef MTS_BWD_LEAN_RUN2
#define MTS_BWD_LEAN_RUN2 2     // MTS_BWD_LEAN_RUN of the two-piece form
#endif
#ifndef MTS_BWD_GROUP2
#define MTS_BWD_GROUP2 1        // the same for rows of 129..256 columns
#endif
#ifndef MTS_BWD_MINBLK2
#define MTS_BWD_MINBLK2 10      // resident blocks per SM for those rows
#endif
#ifndef MTS_BWD_MINBLK
#define MTS_BWD_MINBLK 8        // resident blocks per SM the register allocation is bounded for
#endif
constexpr int BWD_CHUNK = MTS_BWD_CHUNK;
constexpr int BWD_WARPS = 4;
constexpr int LEAN_RUN = MTS_BWD_LEAN_RUN;
constexpr int LEAN_WARPS = MTS_BWD_LEAN_WARPS;   // warps per block of reduce_chunks_lean
constexpr int LIN_GROUP = 8;     // lanes per bag in linearize_lookups

__global__ void __launch_bounds__(256)
linearize_lookups(const TableMeta* __restrict__ meta, int64_t n_bags, int32_t B,
                  const int64_t* __restrict__ indices, const int64_t* __restrict__ offsets,
                  uint32_t* __restrict__ keys, uint32_t* __restrict__ vals,
                  uint32_t* __restrict__ bag_of_pos, int32_t* status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t bag = gid / LIN_GROUP;
  if (bag >= n_bags) return;
  const int sub = (int)(gid % LIN_GROUP);
  const int32_t t = (int32_t)(bag / B);
  const int64_t rows = meta[t].rows;
  const int64_t roff = meta[t].row_offset;
  const int64_t i1 = offsets[bag + 1];
  for (int64_t i = offsets[bag] + sub; i < i1; i += LIN_GROUP) {
    const int64_t idx = clamp_index(indices[i], rows, status);
    keys[i] = (uint32_t)(roff + idx);
    if (bag_of_pos != nullptr) {
      vals[i] = (uint32_t)i;
      bag_of_pos[i] = (uint32_t)bag;
    } else {
      vals[i] = (uint32_t)bag;       // no cached table: nothing needs the position, the bag id travels with the key
    }
  }
}

// Table that owns a linear row id (largest t with row_offset[t] <= key).
__device__ __forceinline__ int table_of_key(const TableMeta* __restrict__ meta, int T, int64_t key) {
  int lo = 0, hi = T - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (meta[mid].row_offset <= key) lo = mid; else hi = mid - 1;
  }
  return lo;
}

#ifndef MTS_BWD_PREFETCH_ROWS
#define MTS_BWD_PREFETCH_ROWS 1   // rows and states that a batch of 32 lookups will update are requested into L2 while it is staged
#endif
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

struct RowTarget {
  char* w;            // row storage (HBM table, cache slot, or host tier)
  uint8_t* dirty;     // dirty byte to set, or nullptr
};

// Cache slot of the lookup at sorted position p (batch position ps): from the array ordered like the sorted
// lookups when the caller has one, else through the lookup's position.
__device__ __forceinline__ int32_t slot_at(const TableMeta& m, const int32_t* __restrict__ sorted_slot, int64_t p,
                                           const int32_t* __restrict__ slot_of_lookup, uint32_t ps) {
  if (m.cache_id < 0) return -1;
  return sorted_slot != nullptr ? sorted_slot[p] : slot_of_lookup[ps];
}

__device__ __forceinline__ RowTarget row_target(const TableMeta& m, int64_t key, int32_t s, int eb,
                                                const CachePtrs& caches, char* dev_w, char* host_w) {
  RowTarget r;
  const int64_t row_bytes = (int64_t)m.dim * eb;
  const int64_t idx = key - m.row_offset;
  r.dirty = nullptr;
  if (m.cache_id < 0) {
    r.w = dev_w + m.weight_offset * eb + idx * row_bytes;
  } else {
    if (s >= 0) {
      r.w = static_cast<char*>(caches.data[m.cache_id]) + (int64_t)s * row_bytes;
      r.dirty = caches.dirty[m.cache_id] ? caches.dirty[m.cache_id] + s : nullptr;
    } else {
      r.w = host_w + m.weight_offset * eb + idx * row_bytes;
    }
  }
  return r;
}

// Four consecutive values of the upstream gradient starting at element `elem` (fp32, or fp16 when GH).
template <bool GH>
__device__ __forceinline__ float4 load_grad4(const void* __restrict__ grad, int64_t elem) {
  if (GH) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(static_cast<const __half*>(grad) + elem));
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
  return __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(grad) + elem));
}

// A lane's four gradient values as loaded: fp32, or fp16 left packed so that the sum can use the
// mixed-precision add (no conversion instructions).
template <bool GH>
struct GradPiece {
  float4 f;
  uint2 h;
};
template <bool GH>
__device__ __forceinline__ GradPiece<GH> load_piece(const void* __restrict__ grad, int64_t elem, bool valid) {
  GradPiece<GH> p;
  if (GH) {
    p.h = make_uint2(0u, 0u);
    if (valid) p.h = __ldg(reinterpret_cast<const uint2*>(static_cast<const __half*>(grad) + elem));
  } else {
    p.f = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid) p.f = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(grad) + elem));
  }
  return p;
}
template <bool GH>
__device__ __forceinline__ void add_piece(float4& acc, const GradPiece<GH>& p) {
  if (GH) {
    add_half2(acc.x, acc.y, p.h.x);
    add_half2(acc.z, acc.w, p.h.y);
  } else {
    acc.x += p.f.x; acc.y += p.f.y; acc.z += p.f.z; acc.w += p.f.w;
  }
}
template <bool GH>
__device__ __forceinline__ void fma_piece(float4& acc, float sc, const GradPiece<GH>& p) {
  float4 g = p.f;
  if (GH) {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&p.h.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&p.h.y));
    g = make_float4(a.x, a.y, b.x, b.y);
  }
  acc.x = fmaf(sc, g.x, acc.x); acc.y = fmaf(sc, g.y, acc.y);
  acc.z = fmaf(sc, g.z, acc.z); acc.w = fmaf(sc, g.w, acc.w);
}

// Row-wise Adagrad on one row held across the warp: lane owns columns (q*32 + lane)*4 .. +3.
// m += mean(g^2); W -= lr * g / (sqrt(m) + eps).  inv_dim = __frcp_rn(dim), hoisted by the callers.
template <bool FP16, int NV>
__device__ __forceinline__ void adagrad_row(const float4 (&g)[NV], const uint4 (&wraw)[NV], float m_old,
                                            int dim, float inv_dim, float lr, float eps, char* wptr,
                                            float* mom_ptr, uint8_t* dirty) {
  const int lane = threadIdx.x & 31;
  float sq = 0.f;
#pragma unroll
  for (int q = 0; q < NV; ++q) sq += g[q].x * g[q].x + g[q].y * g[q].y + g[q].z * g[q].z + g[q].w * g[q].w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float m_new = m_old + sq * inv_dim;
  // approximate square root and division: their relative error (a few 2^-23) only scales the
  // step, far inside the tolerance of the update; the state m itself is exact fp32 arithmetic
  float root;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root) : "f"(m_new));
  const float step = __fdividef(lr, root + eps);
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    const int d = (q * 32 + lane) * 4;
    if (d < dim) {
      if (FP16) {
        const __half2* h = reinterpret_cast<const __half2*>(&wraw[q]);
        float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
        a.x -= step * g[q].x; a.y -= step * g[q].y; b.x -= step * g[q].z; b.y -= step * g[q].w;
        uint2 o;
        __half2 ha = __floats2half2_rn(a.x, a.y), hb = __floats2half2_rn(b.x, b.y);
        o.x = *reinterpret_cast<uint32_t*>(&ha);
        o.y = *reinterpret_cast<uint32_t*>(&hb);
        *reinterpret_cast<uint2*>(wptr + (int64_t)d * 2) = o;
      } else {
        float4 w = *reinterpret_cast<const float4*>(&wraw[q]);
        w.x -= step * g[q].x; w.y -= step * g[q].y; w.z -= step * g[q].z; w.w -= step * g[q].w;
        *reinterpret_cast<float4*>(wptr + (int64_t)d * 4) = w;
      }
    }
  }
  if (lane == 0) {
    *mom_ptr = m_new;
    if (dirty) *dirty = 1;
  }
}

template <bool FP16, int NV>
__device__ __forceinline__ void load_row(uint4 (&wraw)[NV], const char* wptr, int dim) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    const int d = (q * 32 + lane) * 4;
    wraw[q] = make_uint4(0u, 0u, 0u, 0u);
    if (d < dim) {
      if (FP16) {
        const uint2 v = *reinterpret_cast<const uint2*>(wptr + (int64_t)d * 2);
        wraw[q].x = v.x; wraw[q].y = v.y;
      } else {
        wraw[q] = *reinterpret_cast<const uint4*>(wptr + (int64_t)d * 4);
      }
    }
  }
}

// reduce_chunks: one warp per CHUNK consecutive sorted lookups, 32 at a time.  Each lane first
// resolves one lookup (gradient slice, row address, "last lookup of its row") and stages the
// result in shared memory; then the warp walks the 32 lookups in order, GROUP at a time: the
// loads of a whole group (gradient slices, and row + Adagrad state where a row ends) are issued
// before the first one is used.
template <bool FP16, int NV, int GROUP, bool MEAN, bool GH>
__global__ void __launch_bounds__(BWD_WARPS * 32, (NV == 1 ? MTS_BWD_MINBLK : NV == 2 ? MTS_BWD_MINBLK2 : 1))
reduce_chunks(const TableMeta* __restrict__ meta, int T, int32_t B,
              const uint32_t* __restrict__ keys, const uint32_t* __restrict__ pos,
              const uint32_t* __restrict__ bag_of_pos, int64_t n,
              const int64_t* __restrict__ offsets,
              const void* __restrict__ grad, int64_t grad_stride, float lr, float eps,
              const int32_t* __restrict__ slot_of_lookup, const int32_t* __restrict__ sorted_slot,
              const __grid_constant__ CachePtrs caches, char* dev_w, char* host_w,
              float* __restrict__ momentum, float* __restrict__ partial_head,
              float* __restrict__ partial_tail, uint32_t* __restrict__ next_chunk) {
  constexpr int EB = FP16 ? 2 : 4;
  constexpr int PSTRIDE = NV * 128;
  __shared__ uint4 s_desc[BWD_WARPS][32];      // {gradient float offset, key, row address lo, hi}
  __shared__ uint2 s_aux[BWD_WARPS][32];       // {dim, mean-pooling scale bits}
  __shared__ uint8_t* s_dirty[BWD_WARPS][32];
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  // a warp takes its next chunk from a counter: chunk costs differ a lot (see reduce_chunks_lean)
  for (;;) {
  uint32_t taken = 0;
  if (lane == 0) taken = atomicAdd(next_chunk, 1u);
  const int64_t chunk = (int64_t)__shfl_sync(0xffffffffu, taken, 0);
  const int64_t p0 = chunk * BWD_CHUNK;
  if (p0 >= n) return;
  const int64_t p1 = min(n, p0 + BWD_CHUNK);
  const bool first_open = p0 > 0 && keys[p0 - 1] == keys[p0];
  bool seen_end = false;
  float4 acc[NV];
#pragma unroll
  for (int q = 0; q < NV; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
  bool last_is_end = true;

  for (int64_t base = p0; base < p1; base += 32) {
    const int cnt = (int)min((int64_t)32, p1 - base);
    bool my_end = false;
    bool my_dirty = false;
    int my_dim = 0;
    if (lane < cnt) {
      const int64_t p = base + lane;
      const uint32_t key = keys[p];
      my_end = (p + 1 >= n) || keys[p + 1] != key;
      const uint32_t ps = pos[p];
      const uint32_t bag = bag_of_pos != nullptr ? bag_of_pos[ps] : ps;
      const int t = (int)(bag / (uint32_t)B);
      const int b = (int)(bag - (uint32_t)t * (uint32_t)B);
      const TableMeta m = meta[t];
      my_dim = m.dim;
      uint4 d;
      d.x = (uint32_t)((int64_t)b * grad_stride + m.out_offset);
      d.y = key;
      d.z = 0u; d.w = 0u;
      uint8_t* dirty = nullptr;
      if (my_end) {
        const RowTarget rt = row_target(m, (int64_t)key, slot_at(m, sorted_slot, p, slot_of_lookup, ps), EB, caches, dev_w, host_w);
        d.z = (uint32_t)(uintptr_t)rt.w;
        d.w = (uint32_t)((uintptr_t)rt.w >> 32);
        dirty = rt.dirty;
      }
      uint2 a;
      a.x = (uint32_t)m.dim;
      a.y = MEAN ? __float_as_uint(1.f / (float)(offsets[bag + 1] - offsets[bag])) : 0u;
      s_desc[wib][lane] = d;
      s_aux[wib][lane] = a;
      s_dirty[wib][lane] = dirty;
      my_dirty = dirty != nullptr;
    }
    __syncwarp();                                                  // staged descriptions visible to the warp
    const uint32_t ends = __ballot_sync(0xffffffffu, my_end);
    const bool any_dirty = __any_sync(0xffffffffu, my_dirty);
    // one dim for the whole batch unless it straddles tables of different width
    const int dim0 = __shfl_sync(0xffffffffu, my_dim, 0);
    const bool uniform = __all_sync(0xffffffffu, lane >= cnt || my_dim == dim0);
    if (base + 32 >= p1) last_is_end = (ends >> (cnt - 1)) & 1u;

    for (int r = 0; r < cnt; r += GROUP) {
      float4 g[GROUP][NV];
      uint4 w[GROUP][NV];
      float mo[GROUP];
#pragma unroll
      for (int u = 0; u < GROUP; ++u) {
        const int j = r + u;
        if (j < cnt) {
          const uint4 d = s_desc[wib][j];
          const int dim = uniform ? dim0 : (int)s_aux[wib][j].x;
          const int64_t gp = d.x;
#pragma unroll
          for (int q = 0; q < NV; ++q) {
            const int c = (q * 32 + lane) * 4;
            g[u][q] = c < dim ? load_grad4<GH>(grad, gp + c) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
          if ((ends >> j) & 1u) {
            const char* wp = reinterpret_cast<const char*>((uintptr_t)d.z | ((uintptr_t)d.w << 32));
            load_row<FP16, NV>(w[u], wp, dim);
            mo[u] = momentum[d.y];
          }
        }
      }
#pragma unroll
      for (int u = 0; u < GROUP; ++u) {
        const int j = r + u;
        if (j < cnt) {
          if (MEAN) {
            const float sc = __uint_as_float(s_aux[wib][j].y);
#pragma unroll
            for (int q = 0; q < NV; ++q) {
              acc[q].x = fmaf(sc, g[u][q].x, acc[q].x); acc[q].y = fmaf(sc, g[u][q].y, acc[q].y);
              acc[q].z = fmaf(sc, g[u][q].z, acc[q].z); acc[q].w = fmaf(sc, g[u][q].w, acc[q].w);
            }
          } else {
#pragma unroll
            for (int q = 0; q < NV; ++q) {
              acc[q].x += g[u][q].x; acc[q].y += g[u][q].y; acc[q].z += g[u][q].z; acc[q].w += g[u][q].w;
            }
          }
          if ((ends >> j) & 1u) {
            if (first_open && !seen_end) {
              // the row started in an earlier chunk: leave its piece for combine_partials
#pragma unroll
              for (int q = 0; q < NV; ++q)
                *reinterpret_cast<float4*>(partial_head + chunk * PSTRIDE + (q * 32 + lane) * 4) = acc[q];
            } else {
              const uint4 d = s_desc[wib][j];
              const int dim = uniform ? dim0 : (int)s_aux[wib][j].x;
              char* wp = reinterpret_cast<char*>((uintptr_t)d.z | ((uintptr_t)d.w << 32));
              adagrad_row<FP16, NV>(acc, w[u], mo[u], dim, __frcp_rn((float)dim), lr, eps, wp, momentum + d.y,
                                    any_dirty ? s_dirty[wib][j] : nullptr);
            }
            seen_end = true;
#pragma unroll
            for (int q = 0; q < NV; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
      }
    }
    __syncwarp();      // the next batch overwrites the staged descriptions
  }
  if (!last_is_end) {
    float* dst = (first_open && !seen_end) ? partial_head : partial_tail;
#pragma unroll
    for (int q = 0; q < NV; ++q)
      *reinterpret_cast<float4*>(dst + chunk * PSTRIDE + (q * 32 + lane) * 4) = acc[q];
  }
  }
}

// ---- reduce_chunks_lean: the same walk for rows of up to NVL x 128 columns (NVL 16-byte gradient pieces
// per lane, NVL = 1 or 2).  The walk is bound by instruction issue and by the latency of dependent
// instructions, not by bytes in flight, so this form keeps one lookup in flight per warp, fits 32 registers
// (NVL = 1: 64 warps per SM) and issues a row's loads (gradient slice, and row + state where the row
// ends) together.  Same summation order and arithmetic as reduce_chunks.  PNV = pieces per lane of a stored
// partial sum (the layout combine_partials reads), >= NVL.
// `klass` splits the chunks of a model with narrow (<= 128 columns) and wide tables between two launches:
// 0 = every chunk, 1 = only chunks that touch no wide table, 2 = only the others.  The sorted lookups are
// ordered by table, so the tables of a chunk are those from its first lookup's to its last one's.
template <bool FP16, int NVL, int PNV, bool MEAN, bool GH>
__global__ void __launch_bounds__(LEAN_WARPS * 32, (NVL == 1 ? MTS_BWD_LEAN_MINBLK : MTS_BWD_LEAN_MINBLK2))
reduce_chunks_lean(const TableMeta* __restrict__ meta, int T, int32_t B,
                   const uint32_t* __restrict__ keys, const uint32_t* __restrict__ pos,
                   const uint32_t* __restrict__ bag_of_pos, int64_t n,
                   const int64_t* __restrict__ offsets,
                   const void* __restrict__ grad, int64_t grad_stride, float lr, float eps,
                   const int32_t* __restrict__ slot_of_lookup, const int32_t* __restrict__ sorted_slot,
                   const __grid_constant__ CachePtrs caches, char* dev_w, char* host_w,
                   float* __restrict__ momentum, float* __restrict__ partial_head,
                   float* __restrict__ partial_tail, uint32_t* __restrict__ next_chunk, int klass) {
  static_assert(NVL >= 1 && NVL <= 2 && PNV >= NVL, "piece counts");
  constexpr int EB = FP16 ? 2 : 4;
  constexpr int PSTRIDE = PNV * 128;
  __shared__ uint4 s_desc[LEAN_WARPS][32];      // {gradient float offset, key, row address lo, hi}
  __shared__ uint2 s_aux[LEAN_WARPS][32];       // {dim, mean-pooling scale bits}
  __shared__ uint8_t* s_dirty[LEAN_WARPS][32];
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  const int64_t lane_elem = lane * 4;
  auto store_partial = [&](float* dst, int64_t chunk, const float4 (&acc)[NVL]) {
#pragma unroll
    for (int q = 0; q < PNV; ++q)
      *reinterpret_cast<float4*>(dst + chunk * PSTRIDE + (q * 32 + lane) * 4) =
          q < NVL ? acc[q < NVL ? q : 0] : make_float4(0.f, 0.f, 0.f, 0.f);
  };
  // Chunks differ a lot in cost (a chunk inside one hot row is a plain sum, a chunk of rows seen
  // once is 128 updates), so a warp takes its next chunk from a counter instead of a fixed share.
  for (;;) {
  uint32_t taken = 0;
  if (lane == 0) taken = atomicAdd(next_chunk, 1u);
  const int64_t chunk = (int64_t)__shfl_sync(0xffffffffu, taken, 0);
  const int64_t p0 = chunk * BWD_CHUNK;
  if (p0 >= n) return;
  const int len = (int)min((int64_t)BWD_CHUNK, n - p0);
  if (klass != 0) {
    uint32_t bag_a = pos[p0], bag_b = pos[p0 + len - 1];
    if (bag_of_pos != nullptr) { bag_a = bag_of_pos[bag_a]; bag_b = bag_of_pos[bag_b]; }
    const int t_a = (int)(bag_a / (uint32_t)B), t_b = (int)(bag_b / (uint32_t)B);
    bool wide = false;
    for (int t = t_a + lane; t <= t_b; t += 32) wide |= meta[t].dim > 128;
    wide = __any_sync(0xffffffffu, wide);
    if (wide != (klass == 2)) continue;
  }
  // a row that started in an earlier chunk: its piece here goes to combine_partials
  bool open_head = p0 > 0 && keys[p0 - 1] == keys[p0];
  float4 acc[NVL];
#pragma unroll
  for (int q = 0; q < NVL; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
  bool last_is_end = true;

  for (int k0 = 0; k0 < len; k0 += 32) {
    const int cnt = min(32, len - k0);
    bool my_end = false;
    bool my_dirty = false;
    int my_dim = 0;
    if (lane < cnt) {
      const int64_t p = p0 + k0 + lane;
      const uint32_t key = keys[p];
      my_end = (p + 1 >= n) || keys[p + 1] != key;
      const uint32_t ps = pos[p];
      const uint32_t bag = bag_of_pos != nullptr ? bag_of_pos[ps] : ps;
      const int t = (int)(bag / (uint32_t)B);
      const int b = (int)(bag - (uint32_t)t * (uint32_t)B);
      const TableMeta m = meta[t];
      my_dim = m.dim;
      uint4 d;
      d.x = (uint32_t)((int64_t)b * grad_stride + m.out_offset);
      d.y = key;
      d.z = 0u; d.w = 0u;
      uint8_t* dirty = nullptr;
      if (my_end) {
        const int32_t slot = slot_at(m, sorted_slot, p, slot_of_lookup, ps);
        const RowTarget rt = row_target(m, (int64_t)key, slot, EB, caches, dev_w, host_w);
        d.z = (uint32_t)(uintptr_t)rt.w;
        d.w = (uint32_t)((uintptr_t)rt.w >> 32);
        dirty = rt.dirty;
        // the walk reaches this row up to 31 lookups from now: ask for it (device memory only) and its state
        if (MTS_BWD_PREFETCH_ROWS && (m.cache_id < 0 || slot >= 0)) {
          const int row_bytes = m.dim * EB;
          for (int o = 0; o < row_bytes; o += 128) prefetch_l2(rt.w + o);
          prefetch_l2(rt.w + row_bytes - 1);
          prefetch_l2(momentum + key);
        }
      }
      s_desc[wib][lane] = d;
      if (MEAN) {
        uint2 a;
        a.x = (uint32_t)m.dim;
        a.y = __float_as_uint(1.f / (float)(offsets[bag + 1] - offsets[bag]));
        s_aux[wib][lane] = a;
      } else {
        s_aux[wib][lane].x = (uint32_t)m.dim;
      }
      s_dirty[wib][lane] = dirty;
      my_dirty = dirty != nullptr;
    }
    __syncwarp();                                                  // staged descriptions visible to the warp
    const uint32_t ends = __ballot_sync(0xffffffffu, my_end);
    const bool any_dirty = __any_sync(0xffffffffu, my_dirty);
    // one dim for the whole batch unless it straddles tables of different width
    const int dim0 = __shfl_sync(0xffffffffu, my_dim, 0);
    const bool uniform = __all_sync(0xffffffffu, lane >= cnt || my_dim == dim0);
    if (k0 + 32 >= len) last_is_end = (ends >> (cnt - 1)) & 1u;
    const float inv_dim0 = __frcp_rn((float)dim0);

    // walk the 32 lookups run by run: the lookups before the next "last of its row" are only
    // summed (no test per lookup), then that lookup closes its row.  WIDTH = 128 or 256: every row of
    // the batch has that many columns (all lanes take part, the width is a constant); 0 = any widths.
    auto walk = [&](auto width) {
    constexpr int WIDTH = decltype(width)::value;
    constexpr int NP = WIDTH == 128 ? 1 : NVL;                     // pieces a lane loads per lookup
    constexpr int RUN = NP == 1 ? LEAN_RUN : MTS_BWD_LEAN_RUN2;
    struct Pieces { GradPiece<GH> q[NP]; };
    auto add_scaled = [&](const Pieces& g, int jj) {
      if (MEAN) {
        const float sc = __uint_as_float(s_aux[wib][jj].y);
#pragma unroll
        for (int q = 0; q < NP; ++q) fma_piece<GH>(acc[q], sc, g.q[q]);
      } else {
#pragma unroll
        for (int q = 0; q < NP; ++q) add_piece<GH>(acc[q], g.q[q]);
      }
    };
    auto load_at = [&](uint32_t goff, int dim) {
      Pieces g;
#pragma unroll
      for (int q = 0; q < NP; ++q)
        g.q[q] = load_piece<GH>(grad, lane_elem + q * 128 + goff, WIDTH != 0 || (q * 32 + lane) * 4 < dim);
      return g;
    };
    auto dim_of = [&](int jj) { return WIDTH != 0 ? WIDTH : uniform ? dim0 : (int)s_aux[wib][jj].x; };
    auto load_grad = [&](int jj) { return load_at(s_desc[wib][jj].x, dim_of(jj)); };
    int j = 0;
    while (j < cnt) {
      const uint32_t rest = ends >> j;
      const int e = rest ? j + __ffs(rest) - 1 : cnt;              // next lookup that ends a row (or none)
      for (; j + RUN <= e; j += RUN) {
        Pieces g[RUN];
#pragma unroll
        for (int u = 0; u < RUN; ++u) g[u] = load_grad(j + u);
#pragma unroll
        for (int u = 0; u < RUN; ++u) add_scaled(g[u], j + u);
      }
      for (; j < e; ++j) add_scaled(load_grad(j), j);
      if (e < cnt) {
        const uint4 d = s_desc[wib][e];
        const int dim = dim_of(e);
        const Pieces g = load_at(d.x, dim);
        if (open_head) {
          add_scaled(g, e);
          store_partial(partial_head, chunk, acc);
          open_head = false;
        } else {
          uint4 w[NP];
          char* wp = reinterpret_cast<char*>((uintptr_t)d.z | ((uintptr_t)d.w << 32));
          load_row<FP16, NP>(w, wp, dim);
          const float m_old = momentum[d.y];
          add_scaled(g, e);
          float4 a[NP];
#pragma unroll
          for (int q = 0; q < NP; ++q) a[q] = acc[q];
          adagrad_row<FP16, NP>(a, w, m_old, dim,
                                WIDTH == 128 ? 0.0078125f : WIDTH == 256 ? 0.00390625f : uniform ? inv_dim0 : __frcp_rn((float)dim),
                                lr, eps, wp, momentum + d.y, any_dirty ? s_dirty[wib][e] : nullptr);
        }
#pragma unroll
        for (int q = 0; q < NVL; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        j = e + 1;
      }
    }
    };
    if (uniform && dim0 == 128) walk(std::integral_constant<int, 128>{});
    else if (NVL == 2 && uniform && dim0 == 256) walk(std::integral_constant<int, (NVL == 2 ? 256 : 0)>{});
    else walk(std::integral_constant<int, 0>{});
    __syncwarp();      // the next batch overwrites the staged descriptions
  }
  if (!last_is_end) {
    // open_head still set: the whole chunk lies inside a row that started earlier
    store_partial(open_head ? partial_head : partial_tail, chunk, acc);
  }
  }
}

// Rows with very many lookups span hundreds of chunks.  One warp per aligned group of
// COMBINE_GROUP consecutive chunks: when every chunk of the group starts inside one row that began
// before the group, the group's head partials are added up (in chunk order) into one partial, so
// that the owner of the row adds one vector per group instead of COMBINE_GROUP.
constexpr int COMBINE_GROUP = 32;

template <int NV>
__global__ void __launch_bounds__(BWD_WARPS * 32)
combine_groups(const uint32_t* __restrict__ keys, int64_t n, const float* __restrict__ partial_head,
               float* __restrict__ partial_group) {
  constexpr int PSTRIDE = NV * 128;
  const int lane = threadIdx.x & 31;
  const int64_t grp = (int64_t)blockIdx.x * BWD_WARPS + (threadIdx.x >> 5);
  const int64_t c0 = grp * COMBINE_GROUP;
  const int64_t p0 = c0 * BWD_CHUNK;
  if (p0 == 0 || p0 + (int64_t)(COMBINE_GROUP - 1) * BWD_CHUNK >= n) return;
  const uint32_t key = keys[p0 - 1];
  // the last chunk of the group still starts inside the row <=> all of them do (keys ascend)
  if (keys[p0 + (int64_t)(COMBINE_GROUP - 1) * BWD_CHUNK] != key) return;
  float4 acc[NV];
#pragma unroll
  for (int q = 0; q < NV; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
  constexpr int U = 4;
  for (int c = 0; c < COMBINE_GROUP; c += U) {
    float4 v[U][NV];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int q = 0; q < NV; ++q)
        v[u][q] = *reinterpret_cast<const float4*>(partial_head + (c0 + c + u) * PSTRIDE + (q * 32 + lane) * 4);
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int q = 0; q < NV; ++q) {
        acc[q].x += v[u][q].x; acc[q].y += v[u][q].y; acc[q].z += v[u][q].z; acc[q].w += v[u][q].w;
      }
  }
#pragma unroll
  for (int q = 0; q < NV; ++q)
    *reinterpret_cast<float4*>(partial_group + grp * PSTRIDE + (q * 32 + lane) * 4) = acc[q];
}

// One warp per chunk.  The chunk owns a row iff the row's lookups start in it and run past
// its end; the owner adds tail[c] + head[c+1] + ... in chunk order and applies the update.
template <bool FP16, int NV>
__global__ void __launch_bounds__(BWD_WARPS * 32)
combine_partials(const TableMeta* __restrict__ meta, int T, const uint32_t* __restrict__ keys,
                 const uint32_t* __restrict__ pos, int64_t n, float lr, float eps,
                 const int32_t* __restrict__ slot_of_lookup, const int32_t* __restrict__ sorted_slot,
                 const __grid_constant__ CachePtrs caches, char* dev_w, char* host_w,
                 float* __restrict__ momentum, const float* __restrict__ partial_head,
                 const float* __restrict__ partial_tail, const float* __restrict__ partial_group) {
  constexpr int EB = FP16 ? 2 : 4;
  constexpr int PSTRIDE = NV * 128;
  const int lane = threadIdx.x & 31;
  const int64_t chunk = (int64_t)blockIdx.x * BWD_WARPS + (threadIdx.x >> 5);
  const int64_t p0 = chunk * BWD_CHUNK;
  const int64_t pe = p0 + BWD_CHUNK;           // first position of the next chunk
  if (pe >= n) return;                         // no later chunk: nothing can continue
  const uint32_t key = keys[pe - 1];
  if (keys[pe] != key) return;                 // last row of the chunk ends here
  if (p0 > 0 && keys[p0 - 1] == key) return;   // started earlier: an earlier chunk owns it
  // number of later chunks the row reaches into
  int64_t nc = 0;
  for (;;) {
    const int64_t start = pe + (nc + lane) * (int64_t)BWD_CHUNK;
    const bool in = start < n && keys[start] == key;
    const uint32_t bal = __ballot_sync(0xffffffffu, in);
    const int lead = __ffs(~bal) - 1;          // leading run of chunks that continue the row
    if (bal == 0xffffffffu) { nc += 32; continue; }
    nc += lead;
    break;
  }
  float4 acc[NV];
#pragma unroll
  for (int q = 0; q < NV; ++q)
    acc[q] = *reinterpret_cast<const float4*>(partial_tail + chunk * PSTRIDE + (q * 32 + lane) * 4);
  // chunks chunk+1 .. chunk+nc carry the row's pieces; whole aligned groups of them were added up
  // by combine_groups.  The order (single chunks up to the first group border, groups, single
  // chunks again) depends only on the chunk numbers.
  constexpr int U = 4;
  int64_t c = chunk + 1;
  const int64_t c_end = chunk + nc;            // inclusive
  while (c <= c_end) {
    if ((c % COMBINE_GROUP) == 0 && c + COMBINE_GROUP - 1 <= c_end) {
      const int64_t grp = c / COMBINE_GROUP;
#pragma unroll
      for (int q = 0; q < NV; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(partial_group + grp * PSTRIDE + (q * 32 + lane) * 4);
        acc[q].x += v.x; acc[q].y += v.y; acc[q].z += v.z; acc[q].w += v.w;
      }
      c += COMBINE_GROUP;
      continue;
    }
    // single chunks up to the next group border (or the end), U loads in flight
    const int64_t stop = min(c_end, (c / COMBINE_GROUP + 1) * COMBINE_GROUP - 1);
    for (; c <= stop; c += U) {
      float4 v[U][NV];
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int q = 0; q < NV; ++q)
          v[u][q] = (c + u <= stop)
                        ? *reinterpret_cast<const float4*>(partial_head + (c + u) * PSTRIDE + (q * 32 + lane) * 4)
                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (c + u <= stop) {
#pragma unroll
          for (int q = 0; q < NV; ++q) {
            acc[q].x += v[u][q].x; acc[q].y += v[u][q].y; acc[q].z += v[u][q].z; acc[q].w += v[u][q].w;
          }
        }
    }
    c = stop + 1;
  }
  const int t = table_of_key(meta, T, (int64_t)key);
  const TableMeta m = meta[t];
  const RowTarget rt = row_target(m, (int64_t)key, slot_at(m, sorted_slot, pe - 1, slot_of_lookup, pos[pe - 1]), EB, caches,
                                  dev_w, host_w);
  uint4 w[NV];
  load_row<FP16, NV>(w, rt.w, m.dim);
  adagrad_row<FP16, NV>(acc, w, momentum[key], m.dim, __frcp_rn((float)m.dim), lr, eps, rt.w, momentum + key, rt.dirty);
}

__global__ void export_unique(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ seg_start,
                              const uint32_t* __restrict__ n_unique, int64_t* __restrict__ uniq_rows_out,
                              int64_t* __restrict__ n_unique_out) {
  const uint32_t U = *n_unique;
  for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < U; u += (int64_t)gridDim.x * blockDim.x)
    uniq_rows_out[u] = (int64_t)keys[seg_start[u]];
  if (blockIdx.x == 0 && threadIdx.x == 0) *n_unique_out = (int64_t)U;
}

namespace {

int bits_for(int64_t values) {
  int bits = 1;
  while (bits < 32 && (1ll << bits) < values) ++bits;
  return bits;
}

// How the lookups are sorted by row.  They arrive grouped by table, so each table's lookups can be
// sorted on their own on the bits of the row index inside the table; that is used when it saves a
// pass over sorting the linear row ids of all tables together.
struct SortPlan {
  bool segmented;
  int key_bits;
  int passes() const { return sort_passes(key_bits); }
};

SortPlan sort_plan(const mts_tables* h) {
  int64_t max_rows = 1;
  for (const auto& m : h->h_meta) max_rows = std::max<int64_t>(max_rows, m.rows);
  int64_t min_rows = max_rows;
  for (const auto& m : h->h_meta) min_rows = std::min<int64_t>(min_rows, m.rows);
  const int all_bits = bits_for(h->total_rows), table_bits = bits_for(max_rows);
  if (h->T > 1) {
    if (sort_passes(table_bits) < sort_passes(all_bits)) return {true, table_bits};
    // as many passes, but the smaller tables have no bit left in the last one and are only copied there
    if (sort_passes(table_bits) == sort_passes(all_bits) && sort_passes(table_bits) > 1 &&
        bits_for(min_rows) <= sort_digit_bits(table_bits) * (sort_passes(table_bits) - 1))
      return {true, table_bits};
  }
  return {false, all_bits};
}

// which of the two buffer pairs holds the sorted lookups after the sort
bool sorted_in_b(const mts_tables* h, int64_t N) {
  return N > 1 && (sort_plan(h).passes() & 1) != 0;
}

}  // namespace

struct BwdLayout {
  size_t keys_a, keys_b, vals_a, vals_b, bag_of_pos, hist, scan, seg_start, n_unique, next_chunk, head, tail, group, total;
};

static BwdLayout bwd_layout(const mts_tables* h, int64_t N) {
  BwdLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t n = (size_t)(N > 0 ? N : 1);
  L.keys_a = take(n * 4); L.keys_b = take(n * 4); L.vals_a = take(n * 4); L.vals_b = take(n * 4);
  L.bag_of_pos = take(n * 4);
  const SortPlan plan = sort_plan(h);
  L.hist = take((plan.segmented ? sort_hist_words_segmented((int64_t)n, h->T, plan.key_bits)
                                : sort_hist_words((int64_t)n, plan.key_bits)) * 4);
  L.scan = take(scan_scratch_words() * 4);
  L.seg_start = take((n + 1) * 4);
  L.n_unique = take(256);
  L.next_chunk = take(256);
  const int nv = (h->max_dim + 127) / 128;
  const int nvp = nv <= 1 ? 1 : nv <= 2 ? 2 : nv <= 4 ? 4 : 8;
  const size_t chunks = (size_t)ceil_div((int64_t)n, BWD_CHUNK);
  L.head = take(chunks * nvp * 128 * 4);
  L.tail = take(chunks * nvp * 128 * 4);
  L.group = take((chunks / COMBINE_GROUP + 1) * nvp * 128 * 4);
  L.total = off;
  return L;
}

template <bool FP16, int NV, int GROUP>
static int launch_backward(const mts_tables* h, int32_t B, const uint32_t* keys, const uint32_t* pos,
                           const uint32_t* bag_of_pos, int64_t N, const int64_t* offsets, int32_t pooling_mode,
                           const void* grad, bool grad_half, int64_t grad_stride, float lr, float eps,
                           const int32_t* slot_of_lookup, const int32_t* sorted_slot, const CachePtrs& caches,
                           float* head, float* tail, float* group, uint32_t* next_chunk, cudaStream_t s) {
  const int64_t chunks = ceil_div(N, BWD_CHUNK);
  const unsigned grid = (unsigned)ceil_div(chunks, BWD_WARPS);
  // the reduce kernels exist for fp32 and for fp16 upstream gradients
#define COMMA ,
#define MTS_LAUNCH_GH(KERNEL, TARGS, GRID, THREADS)                                                                  \
  do {                                                                                                               \
    if (grad_half)                                                                                                   \
      KERNEL<TARGS, true><<<GRID, THREADS, 0, s>>>(h->d_meta, h->T, B, keys, pos, bag_of_pos, N, offsets, grad,     \
                                                    grad_stride, lr, eps, slot_of_lookup, sorted_slot, caches,       \
                                                    static_cast<char*>(h->dev_weights),                              \
                                                    static_cast<char*>(h->host_weights), h->momentum, head, tail,    \
                                                    next_chunk);                                                     \
    else                                                                                                             \
      KERNEL<TARGS, false><<<GRID, THREADS, 0, s>>>(h->d_meta, h->T, B, keys, pos, bag_of_pos, N, offsets, grad,    \
                                                     grad_stride, lr, eps, slot_of_lookup, sorted_slot, caches,      \
                                                     static_cast<char*>(h->dev_weights),                             \
                                                     static_cast<char*>(h->host_weights), h->momentum, head, tail,   \
                                                     next_chunk);                                                    \
  } while (0)
  if constexpr (NV <= 2 && MTS_BWD_USE_LEAN) {
    LaunchScope scope(K_REDUCE_CHUNKS, s);
    // as many blocks as fit on the device at once (or fewer); the warps share out the chunks.  (With cached
    // tables too: a grid that covers all chunks, so that blocks retire and the kernels of the cache's other
    // streams get warp slots during this kernel, measured slower for the step as a whole.)
    auto lean_grid = [&](int resident) {
      return (unsigned)std::min<int64_t>(ceil_div(chunks, LEAN_WARPS), (int64_t)h->sm_count * resident);
    };
    // NVL pieces per lane over the chunks of class `klass`
    auto launch_lean = [&](auto nvl, int klass) -> bool {
      constexpr int NVL = decltype(nvl)::value;
      if (cudaMemsetAsync(next_chunk, 0, sizeof(uint32_t), s) != cudaSuccess) return false;
      const unsigned g = lean_grid(NVL == 1 ? MTS_BWD_LEAN_MINBLK : MTS_BWD_LEAN_MINBLK2);
      const bool mean = pooling_mode == MTS_POOL_MEAN;
#define MTS_LEAN(M, G)                                                                                              \
      reduce_chunks_lean<FP16, NVL, NV, M, G><<<g, LEAN_WARPS * 32, 0, s>>>(                                        \
          h->d_meta, h->T, B, keys, pos, bag_of_pos, N, offsets, grad, grad_stride, lr, eps, slot_of_lookup,        \
          sorted_slot, caches, static_cast<char*>(h->dev_weights), static_cast<char*>(h->host_weights), h->momentum, \
          head, tail, next_chunk, klass)
      if (mean) { if (grad_half) MTS_LEAN(true, true); else MTS_LEAN(true, false); }
      else      { if (grad_half) MTS_LEAN(false, true); else MTS_LEAN(false, false); }
#undef MTS_LEAN
      return true;
    };
    bool ok = true;
    if constexpr (NV == 1) {
      ok = launch_lean(std::integral_constant<int, 1>{}, 0);
    } else {
      int min_dim = h->max_dim;
      for (const auto& m : h->h_meta) min_dim = std::min<int>(min_dim, m.dim);
      if (min_dim > 128) {
        ok = launch_lean(std::integral_constant<int, 2>{}, 0);
      } else {
        // narrow and wide tables: the chunks of the narrow ones keep the one-piece walk and its occupancy
        ok = launch_lean(std::integral_constant<int, 1>{}, 1) && launch_lean(std::integral_constant<int, 2>{}, 2);
      }
    }
    if (!ok) return check_launch("memset(next_chunk)");
  } else {
    LaunchScope scope(K_REDUCE_CHUNKS, s);
    constexpr int resident = NV == 1 ? MTS_BWD_MINBLK : NV == 2 ? MTS_BWD_MINBLK2 : 2;
    const unsigned dyn_grid = (unsigned)std::min<int64_t>(grid, (int64_t)h->sm_count * resident);
    if (cudaMemsetAsync(next_chunk, 0, sizeof(uint32_t), s) != cudaSuccess) return check_launch("memset(next_chunk)");
    if (pooling_mode == MTS_POOL_MEAN)
      MTS_LAUNCH_GH(reduce_chunks, FP16 COMMA NV COMMA GROUP COMMA true, dyn_grid, BWD_WARPS * 32);
    else
      MTS_LAUNCH_GH(reduce_chunks, FP16 COMMA NV COMMA GROUP COMMA false, dyn_grid, BWD_WARPS * 32);
  }
  if (chunks >= 2 * COMBINE_GROUP) {
    LaunchScope scope(K_COMBINE_PARTIALS, s);
    combine_groups<NV><<<(unsigned)ceil_div(ceil_div(chunks, COMBINE_GROUP), BWD_WARPS), BWD_WARPS * 32, 0, s>>>(
        keys, N, head, group);
  }
  {
    LaunchScope scope(K_COMBINE_PARTIALS, s);
    combine_partials<FP16, NV><<<grid, BWD_WARPS * 32, 0, s>>>(
        h->d_meta, h->T, keys, pos, N, lr, eps, slot_of_lookup, sorted_slot, caches, static_cast<char*>(h->dev_weights),
        static_cast<char*>(h->host_weights), h->momentum, head, tail, group);
  }
#undef MTS_LAUNCH_GH
#undef COMMA
  return check_launch("reduce_chunks / combine_partials");
}

}  // namespace mts

using namespace mts;

extern "C" size_t mts_tbe_backward_workspace_bytes(const mts_tables* h, int32_t B, int64_t N) {
  (void)B;
  if (!h || N < 0) return 0;
  return bwd_layout(h, N).total;
}

namespace {

int check_backward_common(const mts_tables* h, int32_t B, const int64_t* offsets, int64_t N, void* workspace,
                          size_t workspace_bytes, const BwdLayout& L, const char* who) {
  if (!h || !offsets || B < 1 || N < 0) return set_error(MTS_ERR_INVALID_ARG, "%s: null argument or bad size", who);
  if (N >= (1ll << 32) - BWD_CHUNK || (int64_t)h->T * B >= (1ll << 32))
    return set_error(MTS_ERR_UNSUPPORTED, "%s: lookup positions and bag ids must fit 32 bits", who);
  if (!workspace || ((uintptr_t)workspace & 255))
    return set_error(MTS_ERR_ALIGNMENT, "%s: workspace must be non-null and 256-byte aligned", who);
  if (workspace_bytes < L.total)
    return set_error(MTS_ERR_WORKSPACE, "%s: workspace of %zu bytes, %zu needed", who, workspace_bytes, L.total);
  return MTS_OK;
}

}  // namespace

extern "C" int mts_tbe_backward_sort(const mts_tables* h, int32_t B, const int64_t* indices, const int64_t* offsets,
                                     int64_t N, void* workspace, size_t workspace_bytes, int64_t* uniq_rows_out,
                                     int64_t* n_unique_out, void* stream) {
  if (!h) return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_sort: null tables");
  const BwdLayout L = bwd_layout(h, N > 0 ? N : 0);
  int rc = check_backward_common(h, B, offsets, N, workspace, workspace_bytes, L, "tbe_backward_sort");
  if (rc != MTS_OK) return rc;
  if (N > 0 && !indices) return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_sort: null indices");
  if ((uniq_rows_out == nullptr) != (n_unique_out == nullptr))
    return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_sort: pass both uniq_rows_out and n_unique_out or neither");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  if (N == 0) {
    if (n_unique_out) return check_cuda(cudaMemsetAsync(n_unique_out, 0, sizeof(int64_t), s), "memset(n_unique_out)");
    return MTS_OK;
  }
  uint32_t* keys_a = reinterpret_cast<uint32_t*>(ws + L.keys_a);
  uint32_t* keys_b = reinterpret_cast<uint32_t*>(ws + L.keys_b);
  uint32_t* vals_a = reinterpret_cast<uint32_t*>(ws + L.vals_a);
  uint32_t* vals_b = reinterpret_cast<uint32_t*>(ws + L.vals_b);
  // positions are only needed to find a lookup's cache slot; without cached tables the sorted value is the bag id
  uint32_t* bag_of_pos = h->any_cached ? reinterpret_cast<uint32_t*>(ws + L.bag_of_pos) : nullptr;
  const int64_t n_bags = (int64_t)h->T * B;
  {
    const int64_t threads = n_bags * LIN_GROUP;
    {
      LaunchScope scope(K_LINEARIZE, s);
      linearize_lookups<<<(unsigned)ceil_div(threads, 256), 256, 0, s>>>(h->d_meta, n_bags, B, indices, offsets, keys_a,
                                                                         vals_a, bag_of_pos, h->d_status);
    }
    rc = check_launch("linearize_lookups");
    if (rc != MTS_OK) return rc;
  }
  uint32_t *keys = nullptr, *pos = nullptr;
  const SortPlan plan = sort_plan(h);
  if (plan.segmented) {
    const SortSegments seg{offsets, B, h->d_meta, 0u};
    rc = radix_sort_pairs_segmented(keys_a, vals_a, keys_b, vals_b, N, h->T, seg, plan.key_bits,
                                    reinterpret_cast<uint32_t*>(ws + L.hist), &keys, &pos, s);
  } else {
    rc = radix_sort_pairs(keys_a, vals_a, keys_b, vals_b, N, nullptr, plan.key_bits, 0u,
                          reinterpret_cast<uint32_t*>(ws + L.hist), &keys, &pos, s);
  }
  if (rc != MTS_OK) return rc;
  if ((keys == keys_b) != sorted_in_b(h, N)) return set_error(MTS_ERR_CUDA, "tbe_backward_sort: unexpected result buffer");
  if (uniq_rows_out) {
    uint32_t* seg_start = reinterpret_cast<uint32_t*>(ws + L.seg_start);
    uint32_t* n_unique = reinterpret_cast<uint32_t*>(ws + L.n_unique);
    rc = unique_segments(keys, N, nullptr, seg_start, nullptr, n_unique, reinterpret_cast<uint32_t*>(ws + L.scan), s);
    if (rc != MTS_OK) return rc;
    {
      LaunchScope scope(K_UNIQUE, s);
      export_unique<<<h->sm_count * 4, 256, 0, s>>>(keys, seg_start, n_unique, uniq_rows_out, n_unique_out);
    }
    rc = check_launch("export_unique");
    if (rc != MTS_OK) return rc;
  }
  return MTS_OK;
}

namespace {
// sorted_rows / sorted_bag / sorted_slot: null = the arrays mts_tbe_backward_sort left in the workspace (and
// the slots through slot_of_lookup)
int backward_apply(const mts_tables* h, int32_t B, const int64_t* offsets, int64_t N, int32_t pooling_mode,
                   const void* grad_out, bool grad_half, int64_t grad_stride, float lr, float eps,
                   const int32_t* slot_of_lookup, void* const* host_cache_data, uint8_t* const* host_cache_dirty,
                   int32_t n_caches, void* workspace, size_t workspace_bytes, void* stream,
                   const uint32_t* sorted_rows = nullptr, const uint32_t* sorted_bag = nullptr,
                   const int32_t* sorted_slot = nullptr) {
  if (!h) return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_apply: null tables");
  const BwdLayout L = bwd_layout(h, N > 0 ? N : 0);
  int rc = check_backward_common(h, B, offsets, N, workspace, workspace_bytes, L, "tbe_backward_apply");
  if (rc != MTS_OK) return rc;
  if (!grad_out) return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_apply: null grad_out");
  if (pooling_mode != MTS_POOL_SUM && pooling_mode != MTS_POOL_MEAN)
    return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_apply: pooling mode %d", pooling_mode);
  if (grad_stride < h->total_dim || (grad_stride & 3) || ((uintptr_t)grad_out & 15))
    return set_error(MTS_ERR_ALIGNMENT,
                     "tbe_backward_apply: grad_out must be 16-byte aligned, grad_stride >= %d and a multiple of 4", h->total_dim);
  if ((int64_t)B * grad_stride >= (1ll << 32))
    return set_error(MTS_ERR_UNSUPPORTED, "tbe_backward_apply: grad_out element offsets must fit 32 bits");
  CachePtrs caches;
  rc = fill_cache_ptrs(h, host_cache_data, host_cache_dirty, n_caches, slot_of_lookup, &caches);
  if (rc != MTS_OK) return rc;
  if (N == 0) return MTS_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  const bool in_b = sorted_in_b(h, N);
  const uint32_t* keys = reinterpret_cast<const uint32_t*>(ws + (in_b ? L.keys_b : L.keys_a));
  const uint32_t* pos = reinterpret_cast<const uint32_t*>(ws + (in_b ? L.vals_b : L.vals_a));
  const uint32_t* bag_of_pos = h->any_cached ? reinterpret_cast<const uint32_t*>(ws + L.bag_of_pos) : nullptr;
  if (sorted_rows != nullptr) {
    keys = sorted_rows;
    pos = sorted_bag;            // the value that travels with a key is its bag id: no position -> bag lookup
    bag_of_pos = nullptr;
  }
  float* head = reinterpret_cast<float*>(ws + L.head);
  float* tail = reinterpret_cast<float*>(ws + L.tail);
  float* group = reinterpret_cast<float*>(ws + L.group);
  const int nv = (h->max_dim + 127) / 128;
  const bool fp16 = h->dtype == MTS_DTYPE_FP16;
#define MTS_BWD(F, V, G) return launch_backward<F, V, G>(h, B, keys, pos, bag_of_pos, N, offsets, pooling_mode, grad_out, grad_half, grad_stride, lr, eps, slot_of_lookup, sorted_slot, caches, head, tail, group, reinterpret_cast<uint32_t*>(ws + L.next_chunk), s)
  if (fp16) {
    if (nv <= 1) MTS_BWD(true, 1, MTS_BWD_GROUP1);
    if (nv <= 2) MTS_BWD(true, 2, MTS_BWD_GROUP2);
    if (nv <= 4) MTS_BWD(true, 4, 2);
    MTS_BWD(true, 8, 1);
  } else {
    if (nv <= 1) MTS_BWD(false, 1, MTS_BWD_GROUP1);
    if (nv <= 2) MTS_BWD(false, 2, MTS_BWD_GROUP2);
    if (nv <= 4) MTS_BWD(false, 4, 2);
    MTS_BWD(false, 8, 1);
  }
#undef MTS_BWD
}
}  // namespace

extern "C" int mts_tbe_backward_apply(const mts_tables* h, int32_t B, const int64_t* offsets, int64_t N,
                                      int32_t pooling_mode, const float* grad_out, int64_t grad_stride, float lr,
                                      float eps, const int32_t* slot_of_lookup, void* const* host_cache_data,
                                      uint8_t* const* host_cache_dirty, int32_t n_caches, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  return backward_apply(h, B, offsets, N, pooling_mode, grad_out, false, grad_stride, lr, eps, slot_of_lookup,
                        host_cache_data, host_cache_dirty, n_caches, workspace, workspace_bytes, stream);
}

extern "C" int mts_tbe_backward_apply_f16(const mts_tables* h, int32_t B, const int64_t* offsets, int64_t N,
                                          int32_t pooling_mode, const void* grad_out_f16, int64_t grad_stride,
                                          float lr, float eps, const int32_t* slot_of_lookup,
                                          void* const* host_cache_data, uint8_t* const* host_cache_dirty,
                                          int32_t n_caches, void* workspace, size_t workspace_bytes, void* stream) {
  return backward_apply(h, B, offsets, N, pooling_mode, grad_out_f16, true, grad_stride, lr, eps, slot_of_lookup,
                        host_cache_data, host_cache_dirty, n_caches, workspace, workspace_bytes, stream);
}

extern "C" int mts_tbe_backward_apply_presorted(const mts_tables* h, int32_t B, const int64_t* offsets, int64_t N,
                                                int32_t pooling_mode, const void* grad_out, int32_t grad_dtype,
                                                int64_t grad_stride, float lr, float eps,
                                                const uint32_t* sorted_rows, const uint32_t* sorted_bag,
                                                const int32_t* sorted_slot, void* const* host_cache_data,
                                                uint8_t* const* host_cache_dirty, int32_t n_caches,
                                                void* workspace, size_t workspace_bytes, void* stream) {
  if (grad_dtype != MTS_DTYPE_FP32 && grad_dtype != MTS_DTYPE_FP16)
    return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_apply_presorted: grad_dtype %d", grad_dtype);
  if (N > 0 && (!sorted_rows || !sorted_bag || !sorted_slot))
    return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_apply_presorted: null sorted_rows / sorted_bag / sorted_slot");
  return backward_apply(h, B, offsets, N, pooling_mode, grad_out, grad_dtype == MTS_DTYPE_FP16, grad_stride, lr, eps,
                        sorted_slot, host_cache_data, host_cache_dirty, n_caches, workspace, workspace_bytes, stream,
                        sorted_rows, sorted_bag, sorted_slot);
}

extern "C" int mts_tbe_backward_rowwise_adagrad(
    const mts_tables* h, int32_t B, const int64_t* indices, const int64_t* offsets, int64_t N,
    int32_t pooling_mode, const float* grad_out, int64_t grad_stride, float lr, float eps,
    const int32_t* slot_of_lookup, void* const* host_cache_data, uint8_t* const* host_cache_dirty,
    int32_t n_caches, void* workspace, size_t workspace_bytes, int64_t* uniq_rows_out,
    int64_t* n_unique_out, void* stream) {
  // every argument is checked before the first launch
  if (!h || !offsets || !grad_out || B < 1 || N < 0 || (N > 0 && !indices))
    return set_error(MTS_ERR_INVALID_ARG, "tbe_backward: null argument or bad size");
  if (pooling_mode != MTS_POOL_SUM && pooling_mode != MTS_POOL_MEAN)
    return set_error(MTS_ERR_INVALID_ARG, "tbe_backward: pooling mode %d", pooling_mode);
  if (grad_stride < h->total_dim || (grad_stride & 3) || ((uintptr_t)grad_out & 15))
    return set_error(MTS_ERR_ALIGNMENT, "tbe_backward: grad_out must be 16-byte aligned, grad_stride >= %d and a multiple of 4",
                     h->total_dim);
  if ((int64_t)B * grad_stride >= (1ll << 32))
    return set_error(MTS_ERR_UNSUPPORTED, "tbe_backward: grad_out element offsets must fit 32 bits");
  {
    CachePtrs caches;
    int rc = fill_cache_ptrs(h, host_cache_data, host_cache_dirty, n_caches, slot_of_lookup, &caches);
    if (rc != MTS_OK) return rc;
  }
  int rc = mts_tbe_backward_sort(h, B, indices, offsets, N, workspace, workspace_bytes, uniq_rows_out, n_unique_out, stream);
  if (rc != MTS_OK) return rc;
  return mts_tbe_backward_apply(h, B, offsets, N, pooling_mode, grad_out, grad_stride, lr, eps, slot_of_lookup,
                                host_cache_data, host_cache_dirty, n_caches, workspace, workspace_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
// Backward without a caller-provided workspace: the scratch lives in a fixed array that is part
// of the library image.
static __device__ __align__(256) unsigned char g_static_scratch[MTS_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};      // device address of g_static_scratch, per device
}  // namespace

extern "C" int mts_tbe_backward_rowwise_adagrad_static(
    const mts_tables* h, int32_t B, const int64_t* indices, const int64_t* offsets, int64_t N,
    int32_t pooling_mode, const float* grad_out, int64_t grad_stride, float lr, float eps,
    const int32_t* slot_of_lookup, void* const* host_cache_data, uint8_t* const* host_cache_dirty,
    int32_t n_caches, int64_t* uniq_rows_out, int64_t* n_unique_out, void* stream) {
  if (!h || N < 0) return set_error(MTS_ERR_INVALID_ARG, "tbe_backward_static: null tables or negative N");
  const size_t need = mts_tbe_backward_workspace_bytes(h, B, N);
  if (need > (size_t)MTS_STATIC_SCRATCH_BYTES)
    return set_error(MTS_ERR_CAPACITY,
                     "tbe_backward_static: %lld lookups need %zu bytes of scratch, the built-in array holds %zu; "
                     "use mts_tbe_backward_rowwise_adagrad with a workspace of your own",
                     (long long)N, need, (size_t)MTS_STATIC_SCRATCH_BYTES);
  int dev = 0;
  int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != MTS_OK) return rc;
  if (dev < 0 || dev >= kMaxDevices) return set_error(MTS_ERR_UNSUPPORTED, "tbe_backward_static: device %d", dev);
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (g_static_ptr[dev] == nullptr) {
      // In host code the array's name is only a handle; its device address has to be asked for,
      // once per device, with that device current.
      void* p = nullptr;
      rc = check_cuda(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)");
      if (rc != MTS_OK) return rc;
      g_static_ptr[dev] = p;
    }
    scratch = g_static_ptr[dev];
  }
  // Every scratch word the kernels read is written earlier in the same call, so nothing has to
  // be cleared even though the array still holds the previous call's contents.
  return mts_tbe_backward_rowwise_adagrad(h, B, indices, offsets, N, pooling_mode, grad_out, grad_stride, lr, eps,
                                          slot_of_lookup, host_cache_data, host_cache_dirty, n_caches, scratch,
                                          (size_t)MTS_STATIC_SCRATCH_BYTES, uniq_rows_out, n_unique_out, stream);
}
