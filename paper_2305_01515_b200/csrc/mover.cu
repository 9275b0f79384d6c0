// mts_mover: the data movement of one cache, batch after batch, on a host thread of the library's own
// (Section 5.5.4: rows between the cache and the lower tier; Section 5.7: ahead of the training of their
// batch).  It is the copy-engine path of the header (mts_host_gather_rows / mts_cache_save_victims /
// mts_cache_place_fetched / mts_host_scatter_rows) driven without an interpreter in the loop: per batch the
// thread waits for the tag step's event, reads the list lengths from the pinned copy of the counters,
// starts the victims on their way out, puts the previous batch's victims into their host rows, gathers the
// missed rows and enqueues their copy and the placing kernel, then records the batch's "moved" event.
// Every wait is on a CUDA event or stream that the caller's own work completes; nothing spins.
#include <condition_variable>
#include <deque>
#include <mutex>
#include <thread>
#include <vector>

#include "common.cuh"

using namespace mts;

namespace {
constexpr int MOVED_RING = 64;       // "moved" events kept; far more than batches in flight
}

struct mts_mover {
  mts_cache* cache = nullptr;
  char* host_rows = nullptr;         // the cache's table group in the host tier (pinned, device-visible)
  int64_t row_bytes = 0;
  int32_t threads = 1;
  int32_t n_ctx = 1;
  int device = 0;
  size_t first_bytes = 0, max_bytes = 0;

  // buffers owned by the mover: per batch context pinned keys / rows in / victims out, one device buffer
  struct Ctx {
    int64_t* miss_keys = nullptr; char* rows_in = nullptr;
    int64_t* evict_keys = nullptr; uint8_t* evict_dirty = nullptr; char* rows_out = nullptr;
    cudaEvent_t copied = nullptr;    // victims of the batch in this context are in rows_out
  };
  std::vector<Ctx> ctx;
  char* fetch_dev = nullptr;
  int64_t buf_rows = 0;
  cudaEvent_t saved = nullptr;
  cudaEvent_t moved[MOVED_RING] = {};

  // pending write-back: the batch whose victims still have to go into their host rows
  bool has_pending = false;
  int pending_ctx = 0;
  int64_t pending_evict = 0;

  std::thread worker;
  std::mutex mu;
  std::condition_variable cv_job, cv_done;
  std::deque<std::pair<int64_t, mts_move_job>> jobs;
  int64_t submitted = 0, recorded = 0;   // jobs handed in / jobs whose moved event has been recorded
  bool stop = false;
  int error = MTS_OK;
  double stats[5] = {0, 0, 0, 0, 0};     // gather s, gather bytes, scatter s, scatter bytes, jobs through kernels
};

namespace {

double now_s() {
  timespec ts;
  clock_gettime(CLOCK_MONOTONIC, &ts);
  return (double)ts.tv_sec + 1e-9 * (double)ts.tv_nsec;
}

void free_buffers(mts_mover* m) {
  for (auto& c : m->ctx) {
    if (c.miss_keys) cudaFreeHost(c.miss_keys);
    if (c.rows_in) cudaFreeHost(c.rows_in);
    if (c.evict_keys) cudaFreeHost(c.evict_keys);
    if (c.evict_dirty) cudaFreeHost(c.evict_dirty);
    if (c.rows_out) cudaFreeHost(c.rows_out);
    c.miss_keys = nullptr; c.rows_in = nullptr; c.evict_keys = nullptr; c.evict_dirty = nullptr; c.rows_out = nullptr;
  }
  if (m->fetch_dev) cudaFree(m->fetch_dev);
  m->fetch_dev = nullptr;
  m->buf_rows = 0;
}

// buffers for lists of up to `rows` rows; nothing of this mover may be in flight
int size_buffers(mts_mover* m, int64_t rows) {
  free_buffers(m);
  const size_t rb = (size_t)m->row_bytes;
  for (auto& c : m->ctx) {
    if (cudaHostAlloc(&c.miss_keys, (size_t)rows * 8, cudaHostAllocDefault) != cudaSuccess ||
        cudaHostAlloc(&c.rows_in, (size_t)rows * rb, cudaHostAllocDefault) != cudaSuccess ||
        cudaHostAlloc(&c.evict_keys, (size_t)rows * 8, cudaHostAllocDefault) != cudaSuccess ||
        cudaHostAlloc(&c.evict_dirty, (size_t)rows, cudaHostAllocDefault) != cudaSuccess ||
        cudaHostAlloc(&c.rows_out, (size_t)rows * rb, cudaHostAllocDefault) != cudaSuccess)
      return check_cuda(cudaGetLastError(), "mover: pinned buffers");
  }
  if (cudaMalloc(&m->fetch_dev, (size_t)rows * rb) != cudaSuccess) return check_cuda(cudaGetLastError(), "mover: device buffer");
  m->buf_rows = rows;
  return MTS_OK;
}

int finish_writeback(mts_mover* m) {
  if (!m->has_pending) return MTS_OK;
  mts_mover::Ctx& c = m->ctx[m->pending_ctx];
  int rc = check_cuda(cudaEventSynchronize(c.copied), "mover: victims' copy");
  if (rc != MTS_OK) return rc;
  const double t0 = now_s();
  rc = mts_host_scatter_rows(m->host_rows, c.evict_keys, c.evict_dirty, m->pending_evict, m->row_bytes, c.rows_out, m->threads);
  m->stats[2] += now_s() - t0;
  m->stats[3] += (double)m->pending_evict * (double)m->row_bytes;
  m->has_pending = false;
  return rc;
}

#define MV_CUDA(call, what)                              \
  do {                                                   \
    const int rc_ = check_cuda((call), what);            \
    if (rc_ != MTS_OK) return rc_;                       \
  } while (0)
#define MV_RC(call)                                      \
  do {                                                   \
    const int rc_ = (call);                              \
    if (rc_ != MTS_OK) return rc_;                       \
  } while (0)

int run_job(mts_mover* m, int64_t index, const mts_move_job& j) {
  cudaStream_t s_move = static_cast<cudaStream_t>(j.move_stream);
  cudaStream_t s_save = static_cast<cudaStream_t>(j.save_stream);
  cudaStream_t s_copy = static_cast<cudaStream_t>(j.copy_stream);
  cudaEvent_t tag_done = static_cast<cudaEvent_t>(j.tag_done);
  cudaEvent_t moved = m->moved[index % MOVED_RING];
  MV_CUDA(cudaEventSynchronize(tag_done), "mover: tag step");
  const int64_t n_miss = j.host_counters[MTS_CNT_INSERTED], n_evict = j.host_counters[MTS_CNT_EVICTED];
  const int64_t need = std::max(n_miss, n_evict);
  const size_t rb = (size_t)m->row_bytes;
  if (need > m->buf_rows && need <= j.list_capacity && (size_t)need * rb <= m->max_bytes) {
    // longer lists than any before: larger buffers, once nothing of this cache is in flight
    MV_RC(finish_writeback(m));
    MV_CUDA(cudaStreamSynchronize(s_copy), "mover: sync");
    MV_CUDA(cudaStreamSynchronize(s_save), "mover: sync");
    MV_CUDA(cudaStreamSynchronize(s_move), "mover: sync");
    const int64_t want = std::min<int64_t>(std::min<int64_t>(need * 5 / 4, j.list_capacity), (int64_t)(m->max_bytes / rb));
    MV_RC(size_buffers(m, std::max<int64_t>(want, need)));
  }
  MV_CUDA(cudaStreamWaitEvent(s_move, tag_done, 0), "mover: wait");
  if (need <= m->buf_rows) {
    const int ci = (int)(index % m->n_ctx);
    mts_mover::Ctx& c = m->ctx[ci];
    // the miss keys first: the same copy engine serves the victims, and the gather waits for the keys only
    if (n_miss > 0) MV_CUDA(cudaMemcpyAsync(c.miss_keys, j.miss_keys, (size_t)n_miss * 8, cudaMemcpyDeviceToHost, s_copy), "mover: keys");
    MV_CUDA(cudaStreamWaitEvent(s_save, tag_done, 0), "mover: wait");
    MV_RC(mts_cache_save_victims(m->cache, j.evict_slots, j.evict_dirty, j.list_capacity, j.counters, j.evict_staging, s_save));
    MV_CUDA(cudaEventRecord(m->saved, s_save), "mover: record");
    if (n_evict > 0) {
      MV_CUDA(cudaMemcpyAsync(c.evict_keys, j.evict_keys, (size_t)n_evict * 8, cudaMemcpyDeviceToHost, s_save), "mover: victims");
      MV_CUDA(cudaMemcpyAsync(c.evict_dirty, j.evict_dirty, (size_t)n_evict, cudaMemcpyDeviceToHost, s_save), "mover: victims");
      MV_CUDA(cudaMemcpyAsync(c.rows_out, j.evict_staging, (size_t)n_evict * rb, cudaMemcpyDeviceToHost, s_save), "mover: victims");
    }
    MV_CUDA(cudaEventRecord(c.copied, s_save), "mover: record");
    // this cache's write-backs of earlier batches reach host memory before the gather reads it
    MV_RC(finish_writeback(m));
    m->has_pending = true;
    m->pending_ctx = ci;
    m->pending_evict = n_evict;
    if (n_miss > 0) {
      MV_CUDA(cudaStreamSynchronize(s_copy), "mover: keys");
      const double t0 = now_s();
      MV_RC(mts_host_gather_rows(m->host_rows, c.miss_keys, n_miss, m->row_bytes, c.rows_in, m->threads));
      m->stats[0] += now_s() - t0;
      m->stats[1] += (double)n_miss * (double)rb;
      MV_CUDA(cudaMemcpyAsync(m->fetch_dev, c.rows_in, (size_t)n_miss * rb, cudaMemcpyHostToDevice, s_move), "mover: rows");
    }
    MV_CUDA(cudaStreamWaitEvent(s_move, m->saved, 0), "mover: wait");
    MV_RC(mts_cache_place_fetched(m->cache, m->fetch_dev, j.miss_slots, nullptr, nullptr, j.list_capacity, j.counters, nullptr, s_move));
    MV_CUDA(cudaEventRecord(moved, s_move), "mover: record");
  } else {
    // lists that the buffers may not grow to (a cold cache's first batches, a cut list): the kernels move the rows
    MV_RC(finish_writeback(m));
    MV_RC(mts_cache_prefetch_misses(m->cache, m->host_rows, j.miss_keys, j.miss_slots, j.evict_slots, j.evict_dirty,
                                    j.list_capacity, j.counters, j.evict_staging, s_move));
    MV_RC(mts_cache_writeback_evicted(m->cache, m->host_rows, j.evict_keys, j.evict_dirty, j.list_capacity, j.counters,
                                      j.evict_staging, s_move));
    MV_CUDA(cudaEventRecord(moved, s_move), "mover: record");
    MV_CUDA(cudaEventSynchronize(moved), "mover: kernels' write-back");   // in host memory before the next gather
    m->stats[4] += 1.0;
  }
  return MTS_OK;
}

void mover_loop(mts_mover* m) {
  cudaSetDevice(m->device);
  for (;;) {
    std::pair<int64_t, mts_move_job> job;
    {
      std::unique_lock<std::mutex> lk(m->mu);
      m->cv_job.wait(lk, [m] { return m->stop || !m->jobs.empty(); });
      if (m->jobs.empty()) return;            // stop, and nothing left to do
      job = m->jobs.front();
      m->jobs.pop_front();
    }
    int rc = MTS_OK;
    {
      std::unique_lock<std::mutex> lk(m->mu);
      rc = m->error;
    }
    if (rc == MTS_OK) rc = run_job(m, job.first, job.second);
    {
      std::lock_guard<std::mutex> lk(m->mu);
      if (rc != MTS_OK && m->error == MTS_OK) m->error = rc;
      m->recorded = job.first + 1;
    }
    m->cv_done.notify_all();
  }
}

}  // namespace

extern "C" int mts_mover_create(mts_mover** out, mts_cache* cache, void* host_rows, int64_t row_bytes, int32_t threads,
                                int32_t n_contexts, int64_t first_buffer_bytes, int64_t max_buffer_bytes) {
  if (!out || !cache || !host_rows || row_bytes < 16 || (row_bytes & 15) || threads < 1 || n_contexts < 1 ||
      n_contexts > MOVED_RING / 2 || first_buffer_bytes < row_bytes || max_buffer_bytes < first_buffer_bytes)
    return set_error(MTS_ERR_INVALID_ARG, "mover_create: bad argument");
  mts_mover* m = new mts_mover;
  m->cache = cache;
  m->host_rows = static_cast<char*>(host_rows);
  m->row_bytes = row_bytes;
  m->threads = threads;
  m->n_ctx = n_contexts;
  m->first_bytes = (size_t)first_buffer_bytes;
  m->max_bytes = (size_t)max_buffer_bytes;
  m->ctx.resize(n_contexts);
  int rc = check_cuda(cudaGetDevice(&m->device), "cudaGetDevice");
  if (rc == MTS_OK) rc = check_cuda(cudaEventCreateWithFlags(&m->saved, cudaEventDisableTiming), "cudaEventCreate");
  for (int i = 0; rc == MTS_OK && i < MOVED_RING; ++i)
    rc = check_cuda(cudaEventCreateWithFlags(&m->moved[i], cudaEventDisableTiming), "cudaEventCreate");
  for (auto& c : m->ctx)
    if (rc == MTS_OK) rc = check_cuda(cudaEventCreateWithFlags(&c.copied, cudaEventDisableTiming), "cudaEventCreate");
  if (rc == MTS_OK) rc = size_buffers(m, std::max<int64_t>(1, first_buffer_bytes / row_bytes));
  if (rc != MTS_OK) {
    free_buffers(m);
    delete m;
    return rc;
  }
  m->worker = std::thread(mover_loop, m);
  *out = m;
  return MTS_OK;
}

extern "C" int mts_mover_submit(mts_mover* m, const mts_move_job* job) {
  if (!m || !job || !job->counters || !job->host_counters || !job->tag_done || job->list_capacity < 0)
    return set_error(MTS_ERR_INVALID_ARG, "mover_submit: null argument");
  {
    std::lock_guard<std::mutex> lk(m->mu);
    if (m->error != MTS_OK) return m->error;
    m->jobs.emplace_back(m->submitted++, *job);
  }
  m->cv_job.notify_one();
  return MTS_OK;
}

extern "C" int mts_mover_stream_wait_moved(mts_mover* m, int64_t job_index, void* stream) {
  if (!m || job_index < 0) return set_error(MTS_ERR_INVALID_ARG, "mover_stream_wait_moved: bad argument");
  {
    std::unique_lock<std::mutex> lk(m->mu);
    if (job_index >= m->submitted) return set_error(MTS_ERR_INVALID_ARG, "mover_stream_wait_moved: job %lld not submitted", (long long)job_index);
    if (job_index + MOVED_RING <= m->submitted) return set_error(MTS_ERR_INVALID_ARG, "mover_stream_wait_moved: job %lld is too old", (long long)job_index);
    m->cv_done.wait(lk, [&] { return m->recorded > job_index; });
    if (m->error != MTS_OK) return m->error;
  }
  return check_cuda(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), m->moved[job_index % MOVED_RING], 0),
                    "mover_stream_wait_moved");
}

extern "C" int mts_mover_drain(mts_mover* m) {
  if (!m) return set_error(MTS_ERR_INVALID_ARG, "mover_drain: null mover");
  std::unique_lock<std::mutex> lk(m->mu);
  m->cv_done.wait(lk, [m] { return m->recorded == m->submitted; });
  // the worker is idle now (it only touches the pending write-back inside a job)
  const int rc = finish_writeback(m);
  if (rc != MTS_OK && m->error == MTS_OK) m->error = rc;
  return m->error;
}

extern "C" int mts_mover_stats(mts_mover* m, double* out5) {
  if (!m || !out5) return set_error(MTS_ERR_INVALID_ARG, "mover_stats: null argument");
  std::lock_guard<std::mutex> lk(m->mu);
  for (int i = 0; i < 5; ++i) out5[i] = m->stats[i];
  return MTS_OK;
}

extern "C" int mts_mover_destroy(mts_mover* m) {
  if (!m) return MTS_OK;
  {
    std::lock_guard<std::mutex> lk(m->mu);
    m->stop = true;
  }
  m->cv_job.notify_all();
  if (m->worker.joinable()) m->worker.join();
  cudaSetDevice(m->device);
  if (m->has_pending) finish_writeback(m);
  free_buffers(m);
  if (m->saved) cudaEventDestroy(m->saved);
  for (auto& e : m->moved)
    if (e) cudaEventDestroy(e);
  for (auto& c : m->ctx)
    if (c.copied) cudaEventDestroy(c.copied);
  delete m;
  return MTS_OK;
}
