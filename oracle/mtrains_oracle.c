/*
 * CPU oracle for the sparse-embedding step of MTrainS-style DLRM training.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the step
 * computes; it exists to check the GPU library and to be timed as a CPU baseline.  It
 * shares no code, header, table or constant generator with the CUDA path, and the
 * product never calls it.
 *
 * What is defined here, and where the paper defines it:
 *   - pooled embedding lookup (sum / mean over the rows a sample selects)   Section 2.1.1
 *     (embedding table operators: select rows of a table, pool them)
 *   - backward: aggregate the gradients of every row a batch touched, run a
 *     row-wise Adagrad step with one state per row, write the row back      Section 2.1.2
 *     (optimizer with few states per row), Section 5.9 (aggregations and
 *     optimizers, then update the weights in their memories)
 *   - row cache with tags and per-entry timestamps, LRU in three steps       Section 5.3.1,
 *     (refresh hits, place misses, evict when no free entry), insert of     Section 5.5.1-5.5.4
 *     fetched rows and eviction of LRU rows back to the lower tier
 *   - prefetch invariant (a prefetched row is not evicted before its batch  Section 5.7
 *     trained), expressed as a lock window on timestamps
 *   - table placement over two memories by the lookup-time objective        Section 5.6, Eq. 6
 *   - two cache levels, exclusive, over a backing store: promotion of       Section 5.3.2,
 *     second-level hits and fetched rows, demotion of first-level LRU rows,  Section 5.5.4
 *     eviction of second-level LRU rows to the store
 *
 * Floating point: all sums and the optimizer step are evaluated in double precision and
 * rounded once to the storage type (fp32, or IEEE binary16 with round-to-nearest-even).
 *
 * Parity pins (tests/, CPU only): brute-force per-bag loops, torch embedding_bag, a
 * hand-worked Adagrad step, torch.optim.Adagrad for D = 1, a list-based LRU simulation,
 * cache invariants and cached-vs-uncached transparency; the two-level cache against the
 * one-level cache (its first level decides identically), a list simulation of the second
 * level, the exclusivity invariant and transparency.  The paper prints no worked
 * numeric example for this path, so no pin comes from a printed value:
 * parity unpinned against paper-printed values; pinned against definitions only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_FP32 0
#define ORC_FP16 1

/* ------------------------------------------------------------------ threads */

static int orc_threads = 1;

void orc_set_threads(int n) {
    orc_threads = n < 1 ? 1 : n;
#ifdef _OPENMP
    omp_set_num_threads(orc_threads);
#endif
}

int orc_get_threads(void) { return orc_threads; }

int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ binary16 */

/* IEEE 754 binary16 -> double (exact). */
double orc_half_to_double(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0) v = ldexp((double)f, -24);                 /* zero and subnormals */
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp((double)(1024 + f), e - 25);
    return sign ? -v : v;
}

/* double -> IEEE 754 binary16, round to nearest, ties to even. */
uint16_t orc_double_to_half(double x) {
    uint16_t sign = signbit(x) ? 0x8000u : 0u;
    double a = fabs(x);
    if (isnan(x)) return (uint16_t)(sign | 0x7e00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);   /* rounds to infinity */
    if (a == 0.0) return sign;
    int ex;
    (void)frexp(a, &ex);                                   /* a = m * 2^ex, m in [0.5, 1) */
    int e = ex - 1;                                        /* a in [2^e, 2^(e+1)) */
    if (e < -14) {                                         /* subnormal spacing 2^-24 */
        double q = nearbyint(ldexp(a, 24));                /* 0 .. 1024 */
        return (uint16_t)(sign | (uint16_t)q);
    }
    double q = nearbyint(ldexp(a, 10 - e));                /* 1024 .. 2048 */
    if (q >= 2048.0) { q = 1024.0; e += 1; }
    if (e > 15) return (uint16_t)(sign | 0x7c00u);
    return (uint16_t)(sign | ((uint16_t)(e + 15) << 10) | ((uint16_t)q - 1024u));
}

static inline double load_elem(const void* base, int dtype, int64_t i) {
    if (dtype == ORC_FP32) return (double)((const float*)base)[i];
    return orc_half_to_double(((const uint16_t*)base)[i]);
}

static inline void store_elem(void* base, int dtype, int64_t i, double v) {
    if (dtype == ORC_FP32) ((float*)base)[i] = (float)v;
    else ((uint16_t*)base)[i] = orc_double_to_half(v);
}

/* ------------------------------------------------------------------ set hash */

/* Set index of a row key: x = key * 0x9E3779B97F4A7C15 mod 2^64 (the odd integer nearest
 * 2^64 / golden ratio), set = floor(x * S / 2^64).  Works for any S >= 1. */
int64_t orc_cache_set_of(int64_t key, int64_t S) {
    uint64_t x = (uint64_t)key * 0x9E3779B97F4A7C15ull;
    return (int64_t)(((unsigned __int128)x * (unsigned __int128)(uint64_t)S) >> 64);
}

/* ------------------------------------------------------------------ row addressing */

/* Where lookup i of table t reads/writes its row.  A table without cache (cache_data[t]
 * NULL, or no cache_data at all) uses the flat weight buffer.  A cached table uses the
 * cache slot slot_of_lookup[i] when it is >= 0, and the flat (host-tier) buffer when the
 * lookup overflowed the cache (slot -1). */
static inline void row_location(int t, int64_t i, int64_t idx, const int32_t* dim,
                                const int64_t* weight_offset, void* weights,
                                const int32_t* slot_of_lookup, void* const* cache_data,
                                void** base, int64_t* elem0, int64_t* slot_out) {
    int64_t D = dim[t];
    if (cache_data && cache_data[t] && slot_of_lookup && slot_of_lookup[i] >= 0) {
        *base = cache_data[t];
        *elem0 = (int64_t)slot_of_lookup[i] * D;
        *slot_out = slot_of_lookup[i];
    } else {
        *base = weights;
        *elem0 = weight_offset[t] + idx * D;
        *slot_out = -1;
    }
}

/* ------------------------------------------------------------------ forward */

/* Pooled lookup.  For every table t and sample b:
 *   out[b, out_offset[t] + d] = sum over the bag's lookups i of W_t[indices[i], d]
 * (pooling_mode 0; mode 1, mean pooling, divides by the bag length; mode 2, max pooling, takes
 * the largest of the bag's values in every column instead of their sum; an empty bag gives 0 in
 * every mode).  A row id that occurs twice in a bag counts twice.  offsets is CSR over bag id
 * t*B + b.  mag (nullable, same layout as out, double) receives sum |W| (max pooling: the
 * largest |W|) for error bounds. */
void orc_tbe_forward(int32_t T, int32_t dtype, const int32_t* dim, const int32_t* out_offset,
                     const int64_t* weight_offset, const void* weights, int32_t B,
                     const int64_t* indices, const int64_t* offsets, int32_t pooling_mode,
                     const int32_t* slot_of_lookup, void* const* cache_data,
                     float* out, int64_t out_stride, double* mag) {
#pragma omp parallel for collapse(2) schedule(dynamic, 64)
    for (int32_t t = 0; t < T; ++t) {
        for (int32_t b = 0; b < B; ++b) {
            int64_t bag = (int64_t)t * B + b;
            int64_t i0 = offsets[bag], i1 = offsets[bag + 1];
            int32_t D = dim[t];
            for (int32_t d = 0; d < D; ++d) {
                double acc = 0.0, am = 0.0;
                for (int64_t i = i0; i < i1; ++i) {
                    void* base; int64_t e0, slot;
                    row_location(t, i, indices[i], dim, weight_offset, (void*)weights,
                                 slot_of_lookup, cache_data, &base, &e0, &slot);
                    double w = load_elem(base, dtype, e0 + d);
                    if (pooling_mode == 2) {
                        if (i == i0 || w > acc) acc = w;
                        if (fabs(w) > am) am = fabs(w);
                    } else {
                        acc += w;
                        am += fabs(w);
                    }
                }
                if (pooling_mode == 1 && i1 > i0) { acc /= (double)(i1 - i0); am /= (double)(i1 - i0); }
                out[(int64_t)b * out_stride + out_offset[t] + d] = (float)acc;
                if (mag) mag[(int64_t)b * out_stride + out_offset[t] + d] = am;
            }
        }
    }
}

/* ------------------------------------------------------------------ backward */

typedef struct { int64_t key; int64_t pos; } orc_pair;

static int pair_cmp(const void* a, const void* b) {
    const orc_pair* x = (const orc_pair*)a; const orc_pair* y = (const orc_pair*)b;
    if (x->key != y->key) return x->key < y->key ? -1 : 1;
    if (x->pos != y->pos) return x->pos < y->pos ? -1 : 1;
    return 0;
}

/* Backward of the pooled lookup fused with row-wise Adagrad, on touched rows only.
 * For every distinct row r of table t that occurs in the batch:
 *   g_r[d]  = sum over all occurrences i of r of s_i * grad_out[b(i), out_offset[t] + d]
 *             (s_i = 1 for sum pooling, 1 / bag length for mean pooling)
 *   m_r    += (1 / D_t) * sum_d g_r[d]^2          (one fp32 state per row, starts at 0)
 *   W[r,d] -= lr * g_r[d] / (sqrt(m_r) + eps)     (eps outside the root, new m_r)
 * One optimizer step per row per batch.  Rows not in the batch keep their bits.
 * momentum is indexed by the linear row id row_offset[t] + r.  Cached rows are updated in
 * their cache slot and the slot's dirty byte is set; overflowed rows in the flat buffer.
 * uniq_out (nullable, capacity N) receives the ascending distinct linear row ids;
 * returns their count U.
 * step_mag (nullable, double, indexed like the flat weight buffer: weight_offset[t] + r*D + d,
 * wherever the row lives) receives lr * sum_i |s_i * grad_i[d]| / (sqrt(m_r) + eps): the size
 * of the step had no two gradient terms cancelled, which bounds what a single-precision
 * summation of the same terms may lose. */
int64_t orc_tbe_backward_rowwise_adagrad(
        int32_t T, int32_t dtype, const int32_t* dim, const int32_t* out_offset,
        const int64_t* weight_offset, const int64_t* row_offset, void* weights, float* momentum,
        int32_t B, const int64_t* indices, const int64_t* offsets, int32_t pooling_mode,
        const float* grad_out, int64_t grad_stride, float lr, float eps,
        const int32_t* slot_of_lookup, void* const* cache_data, uint8_t* const* cache_dirty,
        int64_t* uniq_out, double* step_mag) {
    int64_t N = offsets[(int64_t)T * B];
    if (N == 0) return 0;
    orc_pair* pairs = (orc_pair*)malloc((size_t)N * sizeof(orc_pair));
    int32_t* tab_of = (int32_t*)malloc((size_t)N * sizeof(int32_t));
    int32_t* smp_of = (int32_t*)malloc((size_t)N * sizeof(int32_t));
    double* scale_of = (double*)malloc((size_t)N * sizeof(double));
    for (int32_t t = 0; t < T; ++t)
        for (int32_t b = 0; b < B; ++b) {
            int64_t bag = (int64_t)t * B + b;
            int64_t len = offsets[bag + 1] - offsets[bag];
            for (int64_t i = offsets[bag]; i < offsets[bag + 1]; ++i) {
                pairs[i].key = row_offset[t] + indices[i];
                pairs[i].pos = i;
                tab_of[i] = t; smp_of[i] = b;
                scale_of[i] = pooling_mode == 1 ? 1.0 / (double)len : 1.0;
            }
        }
    qsort(pairs, (size_t)N, sizeof(orc_pair), pair_cmp);
    int64_t* seg = (int64_t*)malloc((size_t)(N + 1) * sizeof(int64_t));
    int64_t U = 0;
    for (int64_t i = 0; i < N; ++i)
        if (i == 0 || pairs[i].key != pairs[i - 1].key) seg[U++] = i;
    seg[U] = N;
    double dlr = (double)lr, deps = (double)eps;
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t u = 0; u < U; ++u) {
        int64_t p0 = pairs[seg[u]].pos;
        int32_t t = tab_of[p0];
        int32_t D = dim[t];
        double* g = (double*)calloc((size_t)D, sizeof(double));
        double* gabs = (double*)calloc((size_t)D, sizeof(double));
        for (int64_t j = seg[u]; j < seg[u + 1]; ++j) {
            int64_t i = pairs[j].pos;
            const float* go = grad_out + (int64_t)smp_of[i] * grad_stride + out_offset[t];
            for (int32_t d = 0; d < D; ++d) {
                g[d] += scale_of[i] * (double)go[d];
                gabs[d] += fabs(scale_of[i] * (double)go[d]);
            }
        }
        double sq = 0.0;
        for (int32_t d = 0; d < D; ++d) sq += g[d] * g[d];
        int64_t key = pairs[seg[u]].key;
        double m = (double)momentum[key] + sq / (double)D;
        momentum[key] = (float)m;
        double denom = sqrt(m) + deps;
        void* base; int64_t e0, slot;
        row_location(t, p0, indices[p0], dim, weight_offset, weights, slot_of_lookup,
                     cache_data, &base, &e0, &slot);
        for (int32_t d = 0; d < D; ++d) {
            double w = load_elem(base, dtype, e0 + d);
            store_elem(base, dtype, e0 + d, w - dlr * g[d] / denom);
        }
        if (slot >= 0 && cache_dirty && cache_dirty[t]) cache_dirty[t][slot] = 1;
        if (step_mag)
            for (int32_t d = 0; d < D; ++d)
                step_mag[weight_offset[t] + indices[p0] * D + d] = dlr * gabs[d] / denom;
        if (uniq_out) uniq_out[u] = key;
        free(gabs);
        free(g);
    }
    free(seg); free(scale_of); free(smp_of); free(tab_of); free(pairs);
    return U;
}

/* ------------------------------------------------------------------ cache */

/* One cache level: row-granular data, tags (which row id sits in an entry; -1 = free)
 * and states (per-entry timestamp; -1 = free), plus a dirty byte per entry.
 * policy 0 = LRU (state = step of last use).  policy 1 = LFU (state = use count). */
typedef struct {
    int64_t S;
    int32_t ways, dim, dtype, policy, lock_depth;
    int64_t* tag;     /* [S * ways] */
    int64_t* ts;      /* [S * ways]  last-use step (both policies; also the lock window) */
    int64_t* freq;    /* [S * ways]  use count (LFU order) */
    uint8_t* dirty;   /* [S * ways] */
    void* data;       /* [S * ways, dim] storage dtype, NULL for a tag-only simulation */
} orc_cache;

orc_cache* orc_cache_create(int64_t S, int32_t ways, int32_t dim, int32_t dtype, int32_t policy,
                            int32_t lock_depth, int32_t with_data) {
    orc_cache* c = (orc_cache*)calloc(1, sizeof(orc_cache));
    int64_t n = S * ways;
    c->S = S; c->ways = ways; c->dim = dim; c->dtype = dtype; c->policy = policy;
    c->lock_depth = lock_depth;
    c->tag = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    c->ts = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    c->freq = (int64_t*)calloc((size_t)n, sizeof(int64_t));
    c->dirty = (uint8_t*)calloc((size_t)n, 1);
    for (int64_t i = 0; i < n; ++i) { c->tag[i] = -1; c->ts[i] = -1; }
    c->data = with_data ? calloc((size_t)n * dim, dtype == ORC_FP32 ? 4 : 2) : NULL;
    return c;
}

void orc_cache_destroy(orc_cache* c) {
    if (!c) return;
    free(c->tag); free(c->ts); free(c->freq); free(c->dirty); free(c->data); free(c);
}

int64_t* orc_cache_tags(orc_cache* c) { return c->tag; }
int64_t* orc_cache_ts(orc_cache* c) { return c->ts; }
int64_t* orc_cache_freq(orc_cache* c) { return c->freq; }
uint8_t* orc_cache_dirty(orc_cache* c) { return c->dirty; }
void* orc_cache_data(orc_cache* c) { return c->data; }

static int i64_cmp(const void* a, const void* b) {
    int64_t x = *(const int64_t*)a, y = *(const int64_t*)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

typedef struct { int64_t set; int64_t key; int64_t u; } orc_setkey;   /* u: index among distinct keys */

static int setkey_cmp(const void* a, const void* b) {
    const orc_setkey* x = (const orc_setkey*)a; const orc_setkey* y = (const orc_setkey*)b;
    if (x->set != y->set) return x->set < y->set ? -1 : 1;
    return x->key < y->key ? -1 : (x->key > y->key ? 1 : 0);
}

static int64_t find_way(const orc_cache* c, int64_t set, int64_t key) {
    for (int32_t w = 0; w < c->ways; ++w)
        if (c->tag[set * c->ways + w] == key) return w;
    return -1;
}

/* counters: 0 lookups, 1 unique, 2 hit_lookups, 3 miss_lookups, 4 unique_hits,
 * 5 unique_misses, 6 inserted, 7 evicted, 8 evicted_dirty, 9 overflow */
#define ORC_NCOUNTERS 10

/* Tag/state lookup + replacement for one batch of row keys at time `step`.
 *  1. Every distinct key is probed in its set; a lookup is a hit iff its key was resident
 *     before this call.
 *  2. All hits are refreshed first (ts = step; LFU: count += occurrences in the batch).
 *  3. Then, set by set (ascending), the set's missing keys in ascending order are paired
 *     with the set's evictable ways.  A way is evictable iff it is free or its ts <
 *     step - lock_depth (free ways have ts = -1, so they are taken first).  Candidates are ordered by (ts, way) for LRU and by
 *     (count, ts, way) for LFU; the k-th missing key takes the k-th candidate.  A victim
 *     with a valid tag is appended to the evict list with its dirty byte, which is then
 *     cleared.  Misses beyond the candidates are not inserted: slot -1 (overflow).  The miss
 *     list holds at most list_capacity entries: once it is full, every further missing key is
 *     treated like one without a candidate (not inserted, slot -1, counted as overflow).
 *  4. slot = set * ways + way.  miss list order: (set, key).
 * slot_of_lookup[i] receives the slot of keys[i] (or -1).  The lists hold list_capacity entries
 * (the number of distinct keys is always enough).  Returns the number of distinct keys. */
int64_t orc_cache_lookup_insert(orc_cache* c, const int64_t* keys, int64_t N, int64_t step,
                                int32_t* slot_of_lookup, int64_t* miss_keys, int32_t* miss_slots,
                                int64_t* evict_keys, int32_t* evict_slots, uint8_t* evict_dirty,
                                int64_t list_capacity, int64_t* counters) {
    for (int k = 0; k < ORC_NCOUNTERS; ++k) counters[k] = 0;
    counters[0] = N;
    if (N == 0) return 0;
    int64_t* sorted = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    memcpy(sorted, keys, (size_t)N * sizeof(int64_t));
    qsort(sorted, (size_t)N, sizeof(int64_t), i64_cmp);
    orc_setkey* uq = (orc_setkey*)malloc((size_t)N * sizeof(orc_setkey));
    int64_t* mult = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    int64_t U = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (i == 0 || sorted[i] != sorted[i - 1]) {
            uq[U].key = sorted[i]; uq[U].set = orc_cache_set_of(sorted[i], c->S); uq[U].u = U;
            mult[U] = 0; ++U;
        }
        ++mult[U - 1];
    }
    counters[1] = U;
    /* steps 1 + 2: probe everything against the state before the call, refresh hits */
    int64_t* slot_of_uniq = (int64_t*)malloc((size_t)U * sizeof(int64_t));
    for (int64_t u = 0; u < U; ++u) {
        int64_t w = find_way(c, uq[u].set, uq[u].key);
        if (w >= 0) {
            slot_of_uniq[u] = uq[u].set * c->ways + w;
            counters[2] += mult[u]; counters[4] += 1;
        } else {
            slot_of_uniq[u] = -2;       /* to be placed */
            counters[3] += mult[u]; counters[5] += 1;
        }
    }
    for (int64_t u = 0; u < U; ++u)
        if (slot_of_uniq[u] >= 0) {
            c->ts[slot_of_uniq[u]] = step;
            c->freq[slot_of_uniq[u]] += mult[u];
        }
    /* step 3: misses grouped by set, ascending key inside a set */
    orc_setkey* ms = (orc_setkey*)malloc((size_t)U * sizeof(orc_setkey));
    int64_t M = 0;
    for (int64_t u = 0; u < U; ++u) if (slot_of_uniq[u] == -2) ms[M++] = uq[u];
    qsort(ms, (size_t)M, sizeof(orc_setkey), setkey_cmp);
    int64_t n_miss = 0, n_evict = 0;
    int32_t* cand = (int32_t*)malloc((size_t)c->ways * sizeof(int32_t));
    for (int64_t a = 0; a < M;) {
        int64_t z = a;
        while (z < M && ms[z].set == ms[a].set) ++z;
        int64_t set = ms[a].set;
        int32_t nc = 0;
        for (int32_t w = 0; w < c->ways; ++w)
            if (c->tag[set * c->ways + w] == -1 || c->ts[set * c->ways + w] < step - c->lock_depth) cand[nc++] = w;
        /* order candidates; insertion sort keeps it plain */
        for (int32_t x = 1; x < nc; ++x) {
            int32_t w = cand[x]; int32_t y = x - 1;
            while (y >= 0) {
                int64_t sa = set * c->ways + cand[y], sb = set * c->ways + w;
                int before;     /* does cand[y] come before w ? */
                if (c->policy == 1 && c->freq[sa] != c->freq[sb]) before = c->freq[sa] < c->freq[sb];
                else if (c->ts[sa] != c->ts[sb]) before = c->ts[sa] < c->ts[sb];
                else before = cand[y] < w;
                if (before) break;
                cand[y + 1] = cand[y]; --y;
            }
            cand[y + 1] = w;
        }
        for (int64_t k = a; k < z; ++k) {
            int64_t key = ms[k].key;
            int64_t slot = -1;
            if (k - a < nc && n_miss < list_capacity) {
                slot = set * c->ways + cand[k - a];
                if (c->tag[slot] != -1) {
                    evict_keys[n_evict] = c->tag[slot];
                    evict_slots[n_evict] = (int32_t)slot;
                    evict_dirty[n_evict] = c->dirty[slot];
                    counters[7] += 1; counters[8] += c->dirty[slot] ? 1 : 0;
                    ++n_evict;
                }
                c->dirty[slot] = 0;
                c->tag[slot] = key; c->ts[slot] = step;
                miss_keys[n_miss] = key; miss_slots[n_miss] = (int32_t)slot; ++n_miss;
                counters[6] += 1;
            } else {
                counters[9] += 1;
            }
            slot_of_uniq[ms[k].u] = slot;
            if (slot >= 0) c->freq[slot] = mult[ms[k].u];   /* LFU: count starts at this batch's uses */
        }
        a = z;
    }
    /* step 4: slot of every lookup */
    for (int64_t i = 0; i < N; ++i) {
        int64_t lo = 0, hi = U;
        while (lo < hi) { int64_t mid = (lo + hi) / 2; if (uq[mid].key < keys[i]) lo = mid + 1; else hi = mid; }
        slot_of_lookup[i] = (int32_t)slot_of_uniq[lo];
    }
    free(cand); free(ms); free(slot_of_uniq); free(mult); free(uq); free(sorted);
    return U;
}

/* Data movement for one lookup_insert result (Section 5.5.3-5.5.4):
 * first the rows of dirty victims are saved (slot -> staging[k]), then every missed row is
 * fetched from the lower tier into its slot (host[key] -> data[slot]).
 * host is the lower-tier buffer of this cache's table group: row `key` starts at
 * element key * dim. */
void orc_cache_prefetch_misses(orc_cache* c, const void* host, const int64_t* miss_keys,
                               const int32_t* miss_slots, int64_t n_miss,
                               const int32_t* evict_slots, const uint8_t* evict_dirty,
                               int64_t n_evict, void* staging) {
    size_t rb = (size_t)c->dim * (c->dtype == ORC_FP32 ? 4 : 2);
    for (int64_t k = 0; k < n_evict; ++k)
        if (evict_dirty[k])
            memcpy((char*)staging + (size_t)k * rb, (char*)c->data + (size_t)evict_slots[k] * rb, rb);
    for (int64_t k = 0; k < n_miss; ++k)
        memcpy((char*)c->data + (size_t)miss_slots[k] * rb, (const char*)host + (size_t)miss_keys[k] * rb, rb);
}

/* Evicted dirty rows go back to the lower tier: staging[k] -> host[evict_keys[k]]. */
void orc_cache_writeback_evicted(orc_cache* c, void* host, const int64_t* evict_keys,
                                 const uint8_t* evict_dirty, int64_t n_evict, const void* staging) {
    size_t rb = (size_t)c->dim * (c->dtype == ORC_FP32 ? 4 : 2);
    for (int64_t k = 0; k < n_evict; ++k)
        if (evict_dirty[k])
            memcpy((char*)host + (size_t)evict_keys[k] * rb, (const char*)staging + (size_t)k * rb, rb);
}

/* Write every dirty resident row back and clear its dirty byte; residency is unchanged. */
int64_t orc_cache_flush(orc_cache* c, void* host) {
    size_t rb = (size_t)c->dim * (c->dtype == ORC_FP32 ? 4 : 2);
    int64_t n = 0;
    for (int64_t s = 0; s < c->S * c->ways; ++s)
        if (c->tag[s] != -1 && c->dirty[s]) {
            memcpy((char*)host + (size_t)c->tag[s] * rb, (char*)c->data + (size_t)s * rb, rb);
            c->dirty[s] = 0; ++n;
        }
    return n;
}

/* ------------------------------------------------------------------ two-level exclusive cache */

/* Two cache levels over a backing store (Section 5.3.2: a two-level exclusive cache, the faster
 * memory as the first level; Section 5.5.4: both levels are looked up, first-level misses that
 * hit the second level and rows fetched from the lowest tier are promoted to the first level,
 * first-level LRU rows are evicted to the second level, second-level LRU rows back to the
 * lowest tier).  Exclusive: a row is in at most one level.  Both levels are orc_cache objects.
 *
 * lookup_insert2(keys, step):
 *  1. Every distinct key is probed in both levels (state before the call).
 *  2. + 3. The first level is handled exactly like a one-level cache (orc_cache_lookup_insert):
 *     hits are refreshed, the missing keys of a set take its evictable ways, victims go to the
 *     first-level evict list, keys beyond the evictable ways are not inserted (slot -1, served
 *     from the backing store).  Whether a key that misses the first level sits in the second
 *     level makes no difference to these decisions; it only says where its row comes from:
 *     fetch_src = its second-level slot, or -1 = the backing store.  A promoted row keeps the
 *     dirty byte it had in the second level.
 *  4. Every second-level hit leaves the second level (its way becomes free): it was promoted, or
 *     it found no first-level way and is served from the backing store in this batch, in which
 *     case it is listed in the drop list {key, slot, dirty} so that a dirty row is written to
 *     the store first.
 *  5. The first-level victims are inserted into the second level: grouped by second-level set
 *     (ascending), ascending key inside a set, the k-th takes the set's k-th evictable way (free
 *     ways, then ways with ts < step - lock_depth of the second level, ordered like first-level
 *     candidates).  The inserted entry keeps the timestamp, use count and dirty byte it had in
 *     the first level.  A second-level victim with a valid tag goes to the second-level evict list
 *     {key, slot, dirty}.  ev1_dst = the second-level slot, or -1 when the set had no evictable
 *     way left: that victim goes to the backing store directly.
 * Lists: fetch {key, first-level slot, src} in (first-level set, key) order; ev1 {key, slot,
 * dirty, dst} in the order of the one-level evict list; ev2 in (second-level set, key of the
 * displacing row) order; drop in (first-level set, key) order.
 * counters[0..9] as for one level (hits and misses of the first level), then
 * 10 l2_hit_lookups, 11 l2_unique_hits, 12 promoted, 13 demoted, 14 l2_evicted,
 * 15 l2_evicted_dirty, 16 l2_bypass, 17 l2_bypass_dirty, 18 l2_dropped, 19 l2_dropped_dirty. */
#define ORC_NCOUNTERS2 20

typedef struct { int64_t set; int64_t key; int64_t idx; } orc_demote;

static int demote_cmp(const void* a, const void* b) {
    const orc_demote* x = (const orc_demote*)a; const orc_demote* y = (const orc_demote*)b;
    if (x->set != y->set) return x->set < y->set ? -1 : 1;
    return x->key < y->key ? -1 : (x->key > y->key ? 1 : 0);
}

/* candidate ways of one set in eviction order; returns their number */
static int32_t ordered_candidates(const orc_cache* c, int64_t set, int64_t step, int32_t* cand) {
    int32_t nc = 0;
    for (int32_t w = 0; w < c->ways; ++w)
        if (c->tag[set * c->ways + w] == -1 || c->ts[set * c->ways + w] < step - c->lock_depth) cand[nc++] = w;
    for (int32_t x = 1; x < nc; ++x) {
        int32_t w = cand[x]; int32_t y = x - 1;
        while (y >= 0) {
            int64_t sa = set * c->ways + cand[y], sb = set * c->ways + w;
            int before;
            if (c->policy == 1 && c->freq[sa] != c->freq[sb]) before = c->freq[sa] < c->freq[sb];
            else if (c->ts[sa] != c->ts[sb]) before = c->ts[sa] < c->ts[sb];
            else before = cand[y] < w;
            if (before) break;
            cand[y + 1] = cand[y]; --y;
        }
        cand[y + 1] = w;
    }
    return nc;
}

int64_t orc_cache2_lookup_insert(orc_cache* l1, orc_cache* l2, const int64_t* keys, int64_t N, int64_t step,
                                 int32_t* slot_of_lookup,
                                 int64_t* fetch_keys, int32_t* fetch_slots, int32_t* fetch_src,
                                 int64_t* ev1_keys, int32_t* ev1_slots, uint8_t* ev1_dirty, int32_t* ev1_dst,
                                 int64_t* ev2_keys, int32_t* ev2_slots, uint8_t* ev2_dirty,
                                 int64_t* drop_keys, int32_t* drop_slots, uint8_t* drop_dirty,
                                 int64_t* counters) {
    for (int k = 0; k < ORC_NCOUNTERS2; ++k) counters[k] = 0;
    counters[0] = N;
    if (N == 0) return 0;
    int64_t* sorted = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    memcpy(sorted, keys, (size_t)N * sizeof(int64_t));
    qsort(sorted, (size_t)N, sizeof(int64_t), i64_cmp);
    orc_setkey* uq = (orc_setkey*)malloc((size_t)N * sizeof(orc_setkey));
    int64_t* mult = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    int64_t U = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (i == 0 || sorted[i] != sorted[i - 1]) {
            uq[U].key = sorted[i]; uq[U].set = orc_cache_set_of(sorted[i], l1->S); uq[U].u = U;
            mult[U] = 0; ++U;
        }
        ++mult[U - 1];
    }
    counters[1] = U;
    /* step 1: probe both levels against the state before the call */
    int64_t* slot_of_uniq = (int64_t*)malloc((size_t)U * sizeof(int64_t));
    int64_t* l2slot_of_uniq = (int64_t*)malloc((size_t)U * sizeof(int64_t));
    for (int64_t u = 0; u < U; ++u) {
        int64_t w = find_way(l1, uq[u].set, uq[u].key);
        l2slot_of_uniq[u] = -1;
        if (w >= 0) {
            slot_of_uniq[u] = uq[u].set * l1->ways + w;
            counters[2] += mult[u]; counters[4] += 1;
        } else {
            slot_of_uniq[u] = -2;
            counters[3] += mult[u]; counters[5] += 1;
            int64_t set2 = orc_cache_set_of(uq[u].key, l2->S);
            int64_t w2 = find_way(l2, set2, uq[u].key);
            if (w2 >= 0) {
                l2slot_of_uniq[u] = set2 * l2->ways + w2;
                counters[10] += mult[u]; counters[11] += 1;
            }
        }
    }
    /* step 2: refresh first-level hits */
    for (int64_t u = 0; u < U; ++u)
        if (slot_of_uniq[u] >= 0) {
            l1->ts[slot_of_uniq[u]] = step;
            l1->freq[slot_of_uniq[u]] += mult[u];
        }
    /* step 3: first-level placement, set by set */
    orc_setkey* ms = (orc_setkey*)malloc((size_t)U * sizeof(orc_setkey));
    int64_t M = 0;
    for (int64_t u = 0; u < U; ++u) if (slot_of_uniq[u] == -2) ms[M++] = uq[u];
    qsort(ms, (size_t)M, sizeof(orc_setkey), setkey_cmp);
    int64_t n_fetch = 0, n_ev1 = 0, n_ev2 = 0, n_drop = 0;
    int64_t* ev1_ts = (int64_t*)malloc((size_t)(U + 1) * sizeof(int64_t));
    int64_t* ev1_freq = (int64_t*)malloc((size_t)(U + 1) * sizeof(int64_t));
    int32_t* cand = (int32_t*)malloc((size_t)(l1->ways > l2->ways ? l1->ways : l2->ways) * sizeof(int32_t));
    for (int64_t a = 0; a < M;) {
        int64_t z = a;
        while (z < M && ms[z].set == ms[a].set) ++z;
        int64_t set = ms[a].set;
        int32_t nc = ordered_candidates(l1, set, step, cand);
        for (int64_t k = a; k < z; ++k) {
            int64_t key = ms[k].key, u = ms[k].u;
            int64_t slot = -1;
            if (k - a < nc) {
                slot = set * l1->ways + cand[k - a];
                if (l1->tag[slot] != -1) {
                    ev1_keys[n_ev1] = l1->tag[slot]; ev1_slots[n_ev1] = (int32_t)slot;
                    ev1_dirty[n_ev1] = l1->dirty[slot];
                    ev1_ts[n_ev1] = l1->ts[slot]; ev1_freq[n_ev1] = l1->freq[slot];
                    counters[7] += 1; counters[8] += l1->dirty[slot] ? 1 : 0;
                    ++n_ev1;
                }
                l1->tag[slot] = key; l1->ts[slot] = step; l1->freq[slot] = mult[u];
                l1->dirty[slot] = l2slot_of_uniq[u] >= 0 ? l2->dirty[l2slot_of_uniq[u]] : 0;
                fetch_keys[n_fetch] = key; fetch_slots[n_fetch] = (int32_t)slot;
                fetch_src[n_fetch] = (int32_t)l2slot_of_uniq[u]; ++n_fetch;
                counters[6] += 1;
                if (l2slot_of_uniq[u] >= 0) counters[12] += 1;
            } else {
                counters[9] += 1;
                if (l2slot_of_uniq[u] >= 0) {
                    drop_keys[n_drop] = key; drop_slots[n_drop] = (int32_t)l2slot_of_uniq[u];
                    drop_dirty[n_drop] = l2->dirty[l2slot_of_uniq[u]];
                    counters[18] += 1; counters[19] += l2->dirty[l2slot_of_uniq[u]] ? 1 : 0;
                    ++n_drop;
                }
            }
            slot_of_uniq[u] = slot;
        }
        a = z;
    }
    /* step 4: every second-level hit leaves the second level */
    for (int64_t u = 0; u < U; ++u)
        if (l2slot_of_uniq[u] >= 0) {
            int64_t s2 = l2slot_of_uniq[u];
            l2->tag[s2] = -1; l2->ts[s2] = -1; l2->freq[s2] = 0; l2->dirty[s2] = 0;
        }
    /* step 5: first-level victims into the second level */
    orc_demote* dm = (orc_demote*)malloc((size_t)(n_ev1 + 1) * sizeof(orc_demote));
    for (int64_t k = 0; k < n_ev1; ++k) {
        dm[k].key = ev1_keys[k]; dm[k].set = orc_cache_set_of(ev1_keys[k], l2->S); dm[k].idx = k;
    }
    qsort(dm, (size_t)n_ev1, sizeof(orc_demote), demote_cmp);
    for (int64_t a = 0; a < n_ev1;) {
        int64_t z = a;
        while (z < n_ev1 && dm[z].set == dm[a].set) ++z;
        int64_t set = dm[a].set;
        int32_t nc = ordered_candidates(l2, set, step, cand);
        for (int64_t k = a; k < z; ++k) {
            int64_t e = dm[k].idx;
            if (k - a < nc) {
                int64_t s2 = set * l2->ways + cand[k - a];
                if (l2->tag[s2] != -1) {
                    ev2_keys[n_ev2] = l2->tag[s2]; ev2_slots[n_ev2] = (int32_t)s2; ev2_dirty[n_ev2] = l2->dirty[s2];
                    counters[14] += 1; counters[15] += l2->dirty[s2] ? 1 : 0;
                    ++n_ev2;
                }
                l2->tag[s2] = dm[k].key; l2->ts[s2] = ev1_ts[e]; l2->freq[s2] = ev1_freq[e];
                l2->dirty[s2] = ev1_dirty[e];
                ev1_dst[e] = (int32_t)s2;
                counters[13] += 1;
            } else {
                ev1_dst[e] = -1;
                counters[16] += 1; counters[17] += ev1_dirty[e] ? 1 : 0;
            }
        }
        a = z;
    }
    for (int64_t i = 0; i < N; ++i) {
        int64_t lo = 0, hi = U;
        while (lo < hi) { int64_t mid = (lo + hi) / 2; if (uq[mid].key < keys[i]) lo = mid + 1; else hi = mid; }
        slot_of_lookup[i] = (int32_t)slot_of_uniq[lo];
    }
    free(dm); free(cand); free(ev1_freq); free(ev1_ts); free(ms); free(l2slot_of_uniq); free(slot_of_uniq);
    free(mult); free(uq); free(sorted);
    return U;
}

/* Data movement for one lookup_insert2 result (Section 5.5.4), in an order that never reads a
 * slot after it was overwritten: second-level rows that leave for the store (victims and dropped
 * hits, when dirty); the rows to be fetched are read (from their second-level slot or from the
 * store); first-level victims move to their second-level slot, or to the store when they have
 * none and are dirty; the fetched rows enter their first-level slots. */
void orc_cache2_move(orc_cache* l1, orc_cache* l2, void* store,
                     const int64_t* fetch_keys, const int32_t* fetch_slots, const int32_t* fetch_src, int64_t n_fetch,
                     const int64_t* ev1_keys, const int32_t* ev1_slots, const uint8_t* ev1_dirty,
                     const int32_t* ev1_dst, int64_t n_ev1,
                     const int64_t* ev2_keys, const int32_t* ev2_slots, const uint8_t* ev2_dirty, int64_t n_ev2,
                     const int64_t* drop_keys, const int32_t* drop_slots, const uint8_t* drop_dirty, int64_t n_drop) {
    size_t rb = (size_t)l1->dim * (l1->dtype == ORC_FP32 ? 4 : 2);
    char* d1 = (char*)l1->data; char* d2 = (char*)l2->data; char* st = (char*)store;
    for (int64_t k = 0; k < n_ev2; ++k)
        if (ev2_dirty[k]) memcpy(st + (size_t)ev2_keys[k] * rb, d2 + (size_t)ev2_slots[k] * rb, rb);
    for (int64_t k = 0; k < n_drop; ++k)
        if (drop_dirty[k]) memcpy(st + (size_t)drop_keys[k] * rb, d2 + (size_t)drop_slots[k] * rb, rb);
    char* tmp = (char*)malloc((size_t)(n_fetch > 0 ? n_fetch : 1) * rb);
    for (int64_t k = 0; k < n_fetch; ++k)
        memcpy(tmp + (size_t)k * rb,
               fetch_src[k] >= 0 ? d2 + (size_t)fetch_src[k] * rb : st + (size_t)fetch_keys[k] * rb, rb);
    for (int64_t k = 0; k < n_ev1; ++k) {
        if (ev1_dst[k] >= 0) memcpy(d2 + (size_t)ev1_dst[k] * rb, d1 + (size_t)ev1_slots[k] * rb, rb);
        else if (ev1_dirty[k]) memcpy(st + (size_t)ev1_keys[k] * rb, d1 + (size_t)ev1_slots[k] * rb, rb);
    }
    for (int64_t k = 0; k < n_fetch; ++k)
        memcpy(d1 + (size_t)fetch_slots[k] * rb, tmp + (size_t)k * rb, rb);
    free(tmp);
}

/* ------------------------------------------------------------------ table placement */

/* Table placement over two memories of one GPU (Section 5.6, Eq. 6): each table goes to exactly one
 * memory, the tables of the fast memory must fit its capacity, and the lookup time
 *   time = sum over tables of (D * L * p) / BW of the table's memory
 * is minimal (Eq. 6 with one GPU, where the maximum over GPUs is the single term).  bytes_per_sample[t]
 * = D_t * L_t * p.  Brute force over all 2^T assignments (T <= 24).  placement[t] = 0 fast memory, 1 slow
 * memory.  Returns the minimal time per sample (seconds when the bandwidths are bytes per second). */
double orc_place_tables(int32_t T, const int64_t* size_bytes, const double* bytes_per_sample,
                        int64_t fast_capacity_bytes, double bw_fast, double bw_slow, int32_t* placement) {
    double best = -1.0;
    uint32_t best_mask = 0;
    for (uint32_t mask = 0; mask < (1u << T); ++mask) {       /* bit t set = table t in the fast memory */
        int64_t used = 0;
        double time = 0.0;
        for (int32_t t = 0; t < T; ++t) {
            if ((mask >> t) & 1u) { used += size_bytes[t]; time += bytes_per_sample[t] / bw_fast; }
            else time += bytes_per_sample[t] / bw_slow;
        }
        if (used > fast_capacity_bytes) continue;
        if (best < 0.0 || time < best) { best = time; best_mask = mask; }
    }
    for (int32_t t = 0; t < T; ++t) placement[t] = ((best_mask >> t) & 1u) ? 0 : 1;
    return best;
}

/* ------------------------------------------------------------------ analytical models */

/* Eq. 3: embedding bandwidth demand = QPS * T * D * p * L * 2 (bytes/s). */
double orc_eq3_bandwidth(double qps, double T, double D, double p, double L) {
    return qps * T * D * p * L * 2.0;
}

/* Eq. 4: lower-tier request rate = QPS * T_B * L_B * alpha, alpha = fraction that misses. */
double orc_eq4_iops(double qps, double TB, double LB, double alpha) {
    return qps * TB * LB * alpha;
}
