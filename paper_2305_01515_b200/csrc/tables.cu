// Table handle: validation of the caller's description and the per-table metadata block
// that every lookup consults (which memory serves a table, Section 5.8 of the paper).
#include <cstdarg>
#include <cstdio>
#include <cstring>

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

}  // namespace mts

using namespace mts;

extern "C" const char* mts_last_error_string(void) { return g_err; }

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
