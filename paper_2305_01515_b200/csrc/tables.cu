// Table handle: validation of the caller's description and the per-table metadata block
// that every lookup consults (which memory serves a table, Section 5.8 of the paper).
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace mts {

static thread_local char g_err[512] = "no error";

int set_error(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return MTS_OK;
  return set_error(MTS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// ------------------------------------------------------------------------------- instrumentation
static const char* const kKernelNames[K_COUNT] = {
    "tbe_forward_kernel", "linearize_lookups", "digit_histogram", "scan_histogram", "scatter_by_digit",
    "unique_segments", "reduce_chunks", "combine_partials", "cache_prepare_keys", "cache_describe_unique",
    "cache_probe_replace", "cache_lists", "cache_scatter_slots", "cache_save_victims", "cache_fetch_misses",
    "cache_write_victims", "cache_flush", "other"};

struct TraceRecord { int kernel; cudaEvent_t start, stop; };

static std::mutex g_trace_mu;
static std::atomic<long long> g_launches{0};
static std::atomic<int> g_trace_on{0};
static std::vector<TraceRecord> g_records;      // events are reused across enable/report cycles
static size_t g_used = 0;

LaunchScope::LaunchScope(int kernel_id, cudaStream_t s) : slot(-1), stream(s) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (!g_trace_on.load(std::memory_order_relaxed)) return;
  std::lock_guard<std::mutex> lk(g_trace_mu);
  if (g_used == g_records.size()) {
    TraceRecord r;
    r.kernel = kernel_id;
    if (cudaEventCreate(&r.start) != cudaSuccess) return;
    if (cudaEventCreate(&r.stop) != cudaSuccess) { cudaEventDestroy(r.start); return; }
    g_records.push_back(r);
  }
  g_records[g_used].kernel = kernel_id;
  slot = (int)g_used++;
  cudaEventRecord(g_records[slot].start, stream);
}

LaunchScope::~LaunchScope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lk(g_trace_mu);
  cudaEventRecord(g_records[slot].stop, stream);
}

}  // namespace mts

using namespace mts;

extern "C" const char* mts_last_error_string(void) { return g_err; }

extern "C" int64_t mts_launch_count(void) { return (int64_t)g_launches.load(); }

extern "C" int mts_trace_enable(int32_t enable) {
  std::lock_guard<std::mutex> lk(g_trace_mu);
  g_used = 0;
  g_trace_on.store(enable ? 1 : 0);
  return MTS_OK;
}

extern "C" int32_t mts_trace_kernel_count(void) { return K_COUNT; }

extern "C" const char* mts_trace_kernel_name(int32_t kernel) {
  return (kernel >= 0 && kernel < K_COUNT) ? kKernelNames[kernel] : "";
}

extern "C" int mts_trace_report(double* host_total_ms, int64_t* host_launches, int32_t n) {
  if (!host_total_ms || !host_launches || n < K_COUNT)
    return set_error(MTS_ERR_INVALID_ARG, "trace_report: need %d entries", (int)K_COUNT);
  std::lock_guard<std::mutex> lk(g_trace_mu);
  for (int k = 0; k < n; ++k) { host_total_ms[k] = 0.0; host_launches[k] = 0; }
  for (size_t i = 0; i < g_used; ++i) {
    int rc = check_cuda(cudaEventSynchronize(g_records[i].stop), "cudaEventSynchronize(trace)");
    if (rc != MTS_OK) return rc;
    float ms = 0.f;
    rc = check_cuda(cudaEventElapsedTime(&ms, g_records[i].start, g_records[i].stop), "cudaEventElapsedTime(trace)");
    if (rc != MTS_OK) return rc;
    host_total_ms[g_records[i].kernel] += ms;
    host_launches[g_records[i].kernel] += 1;
  }
  g_used = 0;
  return MTS_OK;
}

extern "C" int mts_tables_create(const mts_table_desc* desc, mts_tables** out) {
  if (!desc || !out) return set_error(MTS_ERR_INVALID_ARG, "tables_create: null argument");
  *out = nullptr;
  if (desc->T < 1) return set_error(MTS_ERR_INVALID_ARG, "tables_create: T = %d", desc->T);
  if (desc->dtype != MTS_DTYPE_FP32 && desc->dtype != MTS_DTYPE_FP16)
    return set_error(MTS_ERR_INVALID_ARG, "tables_create: dtype = %d", desc->dtype);
  if (!desc->host_rows || !desc->host_dim || !desc->host_weight_offset || !desc->momentum)
    return set_error(MTS_ERR_INVALID_ARG, "tables_create: null rows/dim/weight_offset/momentum");
  const int eb = desc->dtype == MTS_DTYPE_FP32 ? 4 : 2;
  mts_tables* h = new mts_tables();
  h->T = desc->T;
  h->dtype = desc->dtype;
  h->elem_bytes = eb;
  h->dev_weights = desc->dev_weights;
  h->host_weights = desc->host_weights_mapped;
  h->momentum = desc->momentum;
  h->h_meta.resize(desc->T);
  int64_t row_off = 0;
  int32_t out_off = 0;
  int rc = MTS_OK;
  for (int t = 0; t < desc->T && rc == MTS_OK; ++t) {
    TableMeta& m = h->h_meta[t];
    m.rows = desc->host_rows[t];
    m.dim = desc->host_dim[t];
    m.weight_offset = desc->host_weight_offset[t];
    m.cache_id = desc->host_cache_id ? desc->host_cache_id[t] : -1;
    m.row_offset = row_off;
    m.out_offset = out_off;
    if (m.rows < 1 || m.dim < 1 || m.weight_offset < 0)
      rc = set_error(MTS_ERR_INVALID_ARG, "tables_create: table %d rows %lld dim %d offset %lld", t,
                     (long long)m.rows, m.dim, (long long)m.weight_offset);
    else if (m.dim > 1024)
      rc = set_error(MTS_ERR_UNSUPPORTED, "tables_create: table %d dim %d > 1024", t, m.dim);
    else if (((int64_t)m.dim * eb) % 16 != 0 || (m.weight_offset * eb) % 16 != 0)
      rc = set_error(MTS_ERR_ALIGNMENT, "tables_create: table %d row bytes %lld / offset not 16-byte multiples",
                     t, (long long)m.dim * eb);
    else if (m.cache_id < -1 || m.cache_id >= MTS_MAX_CACHES)
      rc = set_error(MTS_ERR_INVALID_ARG, "tables_create: table %d cache id %d", t, m.cache_id);
    else if (m.cache_id >= 0 && !desc->host_weights_mapped)
      rc = set_error(MTS_ERR_INVALID_ARG, "tables_create: table %d is cached but host_weights_mapped is null", t);
    else if (m.cache_id < 0 && !desc->dev_weights)
      rc = set_error(MTS_ERR_INVALID_ARG, "tables_create: table %d is HBM resident but dev_weights is null", t);
    m.vec16 = (int32_t)((int64_t)m.dim * eb / 16);
    if (m.cache_id >= 0) {
      h->any_cached = 1;
      if (m.cache_id + 1 > h->n_cache_ids) h->n_cache_ids = m.cache_id + 1;
    }
    if (m.dim > h->max_dim) h->max_dim = m.dim;
    row_off += m.rows;
    out_off += m.dim;
  }
  if (rc == MTS_OK && row_off >= (1ll << 32))
    rc = set_error(MTS_ERR_UNSUPPORTED, "tables_create: %lld rows in total; linear row ids must fit 32 bits",
                   (long long)row_off);
  if (rc == MTS_OK && (((uintptr_t)desc->dev_weights | (uintptr_t)desc->host_weights_mapped) & 15))
    rc = set_error(MTS_ERR_ALIGNMENT, "tables_create: weight buffers must be 16-byte aligned");
  h->total_rows = row_off;
  h->total_dim = out_off;
  if (rc == MTS_OK) {
    int dev = 0;
    rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
    if (rc == MTS_OK) {
      int sms = 0;
      rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "sm count");
      if (rc == MTS_OK && sms > 0) h->sm_count = sms;
    }
  }
  if (rc == MTS_OK) {
    size_t bytes = sizeof(TableMeta) * (size_t)desc->T + 256;
    char* blk = nullptr;
    rc = check_cuda(cudaMalloc(&blk, bytes), "cudaMalloc(table metadata)");
    if (rc == MTS_OK) {
      h->d_status = reinterpret_cast<int32_t*>(blk);
      h->d_meta = reinterpret_cast<TableMeta*>(blk + 256);
      rc = check_cuda(cudaMemset(blk, 0, 256), "cudaMemset(status)");
      if (rc == MTS_OK)
        rc = check_cuda(cudaMemcpy(h->d_meta, h->h_meta.data(), sizeof(TableMeta) * (size_t)desc->T,
                                   cudaMemcpyHostToDevice), "cudaMemcpy(table metadata)");
    }
  }
  if (rc != MTS_OK) {
    if (h->d_status) cudaFree(h->d_status);
    delete h;
    return rc;
  }
  *out = h;
  return MTS_OK;
}

extern "C" int mts_tables_destroy(mts_tables* h) {
  if (!h) return MTS_OK;
  int rc = MTS_OK;
  if (h->d_status) rc = check_cuda(cudaFree(h->d_status), "cudaFree(table metadata)");
  delete h;
  return rc;
}

extern "C" int mts_tables_status(mts_tables* h, int32_t* host_status, void* stream) {
  if (!h || !host_status) return set_error(MTS_ERR_INVALID_ARG, "tables_status: null argument");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = check_cuda(cudaMemcpyAsync(host_status, h->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, s),
                      "cudaMemcpyAsync(status)");
  if (rc != MTS_OK) return rc;
  rc = check_cuda(cudaMemsetAsync(h->d_status, 0, sizeof(int32_t), s), "cudaMemsetAsync(status)");
  if (rc != MTS_OK) return rc;
  return check_cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize(status)");
}
