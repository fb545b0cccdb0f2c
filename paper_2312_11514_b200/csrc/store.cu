// Bundle store in a file: the storage tier of the paper (Section 2.2 "Read Throughput",
// Section 4.1 "Implementation Details", Appendix C "Caching Considerations for Data Loading
// from Flash Memory").  The paper reads the row-column bundles of the newly needed neurons from
// flash with many threads (32), in reads of one bundle each (32 KiB and more in fp32), and
// without the operating system's cache, and manages the loads on the CPU.  This file does
// exactly that on the host: a pool of reader threads, one positional read per bundle, direct
// I/O where the file system allows it, into a pinned staging buffer from which a copy kernel
// moves the rows to their places in the cache.  Nothing here is on the fast path of the
// pinned-memory store; it exists so that the same layer can be fed from a block device.
#include <fcntl.h>
#include <unistd.h>

#include <atomic>
#include <chrono>
#include <condition_variable>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "lif_internal.cuh"

struct lif_store {
  int fd = -1;
  int direct = 0;                 // the file is open with O_DIRECT
  int64_t n_bundles = 0, bundle_bytes = 0;
  int n_threads = 0;
  // one batch of reads at a time
  const int32_t* ids = nullptr;
  unsigned char* dst = nullptr;
  int n = 0;
  std::atomic<int> next{0}, failed{0};
  int generation = 0, running = 0;
  bool stop = false;
  std::mutex m;
  std::condition_variable cv_start, cv_done;
  std::vector<std::thread> workers;
  // host copies of a step's counts and load list (pinned, owned by the store)
  int32_t* host_counts = nullptr;   // [LIF_CNT_LEN]
  int32_t* host_ids = nullptr;      // [n_bundles]
  // statistics
  std::atomic<uint64_t> reads{0}, bytes_read{0};
  uint64_t bytes_requested = 0;
  double seconds_reading = 0.0;
};

namespace lif {
namespace {

constexpr size_t kBlock = 4096;     // alignment direct I/O asks of offsets, sizes and buffers

// Read bundle `id` into `out`.  `bounce`: this thread's aligned buffer for reads that direct
// I/O cannot place directly (bundle size or destination not block-aligned).
bool read_bundle(lif_store* s, int id, unsigned char* out, unsigned char* bounce) {
  if (id < 0 || id >= s->n_bundles) return false;
  const size_t len = (size_t)s->bundle_bytes;
  const off_t off = (off_t)id * (off_t)len;
  const bool direct_ok = !s->direct || (len % kBlock == 0 && (uintptr_t)out % kBlock == 0);
  unsigned char* buf = direct_ok ? out : bounce;
  const off_t a0 = direct_ok ? off : (off / (off_t)kBlock) * (off_t)kBlock;
  const size_t span = direct_ok ? len : (((size_t)(off - a0) + len + kBlock - 1) / kBlock) * kBlock;
  size_t got = 0;
  while (got < (direct_ok ? len : (size_t)(off - a0) + len)) {
    const ssize_t r = pread(s->fd, buf + got, span - got, a0 + (off_t)got);
    if (r <= 0) return false;       // error, or the file is shorter than the store it stands for
    got += (size_t)r;
    s->reads.fetch_add(1, std::memory_order_relaxed);
    s->bytes_read.fetch_add((uint64_t)r, std::memory_order_relaxed);
  }
  if (!direct_ok) memcpy(out, bounce + (off - a0), len);
  return true;
}

void worker(lif_store* s) {
  unsigned char* bounce = nullptr;
  if (posix_memalign((void**)&bounce, kBlock, ((size_t)s->bundle_bytes / kBlock + 3) * kBlock) != 0)
    bounce = nullptr;
  int seen = 0;
  for (;;) {
    {
      std::unique_lock<std::mutex> lk(s->m);
      s->cv_start.wait(lk, [&] { return s->stop || s->generation != seen; });
      if (s->stop) break;
      seen = s->generation;
    }
    for (;;) {
      const int j = s->next.fetch_add(1, std::memory_order_relaxed);
      if (j >= s->n) break;
      if (!bounce || !read_bundle(s, s->ids[j], s->dst + (size_t)j * s->bundle_bytes, bounce))
        s->failed.store(1, std::memory_order_relaxed);
    }
    std::lock_guard<std::mutex> lk(s->m);
    if (--s->running == 0) s->cv_done.notify_one();
  }
  free(bounce);
}

// Read bundles ids[0..n) into dst[j * bundle_bytes] with the store's threads; blocks.
bool read_batch(lif_store* s, const int32_t* ids, int n, void* dst) {
  if (n <= 0) return true;
  const auto t0 = std::chrono::steady_clock::now();
  {
    std::lock_guard<std::mutex> lk(s->m);
    s->ids = ids;
    s->dst = (unsigned char*)dst;
    s->n = n;
    s->next.store(0);
    s->failed.store(0);
    s->running = s->n_threads;
    ++s->generation;
  }
  s->cv_start.notify_all();
  {
    std::unique_lock<std::mutex> lk(s->m);
    s->cv_done.wait(lk, [&] { return s->running == 0; });
  }
  s->bytes_requested += (uint64_t)n * (uint64_t)s->bundle_bytes;
  s->seconds_reading += std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
  return s->failed.load() == 0;
}

}  // namespace
}  // namespace lif

using namespace lif;

extern "C" {

lif_status lif_store_open(const char* path, int64_t n_bundles, int64_t bundle_bytes,
                          int32_t n_threads, int32_t direct_io, lif_store** out) {
  if (!out) return LIF_ERR_INVALID_ARG;
  *out = nullptr;
  if (!path || n_bundles < 1 || n_bundles >= (1 << 21) || bundle_bytes < 16 || bundle_bytes % 16 ||
      n_threads < 1 || n_threads > 256)
    return LIF_ERR_INVALID_ARG;
  int fd = -1, direct = 0;
  if (direct_io) {
    fd = open(path, O_RDONLY | O_DIRECT);
    direct = fd >= 0;
  }
  if (fd < 0) fd = open(path, O_RDONLY);       // file systems without direct I/O (tmpfs)
  if (fd < 0) return LIF_ERR_INVALID_ARG;
  const off_t size = lseek(fd, 0, SEEK_END);
  if (size < (off_t)(n_bundles * bundle_bytes)) {
    close(fd);
    return LIF_ERR_INVALID_ARG;
  }
  lif_store* s = new (std::nothrow) lif_store();
  if (!s) {
    close(fd);
    return LIF_ERR_STATE;
  }
  s->fd = fd;
  s->direct = direct;
  s->n_bundles = n_bundles;
  s->bundle_bytes = bundle_bytes;
  s->n_threads = n_threads;
  if (cudaHostAlloc((void**)&s->host_counts, LIF_CNT_LEN * 4, cudaHostAllocDefault) != cudaSuccess ||
      cudaHostAlloc((void**)&s->host_ids, (size_t)n_bundles * 4, cudaHostAllocDefault) != cudaSuccess) {
    // no device: plain memory serves lif_store_read; lif_decode_step_store needs a device anyway
    cudaGetLastError();
    if (s->host_counts) cudaFreeHost(s->host_counts);
    s->host_counts = nullptr;
    s->host_ids = nullptr;
  }
  for (int i = 0; i < n_threads; ++i) s->workers.emplace_back(worker, s);
  *out = s;
  return LIF_OK;
}

lif_status lif_store_close(lif_store* s) {
  if (!s) return LIF_ERR_INVALID_ARG;
  {
    std::lock_guard<std::mutex> lk(s->m);
    s->stop = true;
  }
  s->cv_start.notify_all();
  for (auto& t : s->workers) t.join();
  if (s->host_counts) cudaFreeHost(s->host_counts);
  if (s->host_ids) cudaFreeHost(s->host_ids);
  close(s->fd);
  delete s;
  return LIF_OK;
}

lif_status lif_store_read(lif_store* s, const int32_t* host_ids, int32_t n, void* host_dst) {
  if (!s || n < 0 || (n > 0 && (!host_ids || !host_dst))) return LIF_ERR_INVALID_ARG;
  for (int j = 0; j < n; ++j)
    if (host_ids[j] < 0 || host_ids[j] >= s->n_bundles) return LIF_ERR_INVALID_ARG;
  return read_batch(s, host_ids, n, host_dst) ? LIF_OK : LIF_ERR_STATE;
}

lif_status lif_store_get_stats(lif_store* s, lif_store_stats* o) {
  if (!s || !o) return LIF_ERR_INVALID_ARG;
  o->reads = s->reads.load();
  o->bytes_read = s->bytes_read.load();
  o->bytes_requested = s->bytes_requested;
  o->seconds_reading = s->seconds_reading;
  o->direct_io = s->direct;
  o->n_threads = s->n_threads;
  return LIF_OK;
}

lif_status lif_decode_step_store(lif_layer* L, lif_store* s, const void* dev_x, float* dev_y,
                                 void* stream) {
  if (!L || !s || !dev_x || !dev_y || !s->host_counts) return LIF_ERR_INVALID_ARG;
  if (((uintptr_t)dev_x % 16) || ((uintptr_t)dev_y % 16)) return LIF_ERR_ALIGNMENT;
  const lif_layer_desc& D = L->desc;
  if (D.staging_rows == 0) return LIF_ERR_STATE;      // host_bundles is a whole store, not a staging buffer
  if (s->bundle_bytes != 2 * (int64_t)row_elems(D) || s->n_bundles != D.d_ff) return LIF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const __half* x = (const __half*)dev_x;
  // predict and update the window exactly as lif_decode_step does on one stream
  bool ok;
  if (L->fused_plan) {
    ok = launch_predict(L, x, nullptr, L->active_idx, L->n_tmp, st, nullptr, 0) == cudaSuccess;
    ok = ok && launch_window_plan(L, st, nullptr, true) == cudaSuccess;
  } else {
    ok = launch_predict(L, x, nullptr, L->active_idx, L->n_tmp, st, nullptr) == cudaSuccess;
    ok = ok && launch_window(L, L->active_idx, L->n_tmp, st, nullptr, true) == cudaSuccess;
  }
  // the load list comes to the host: the loads are managed there, as in the paper
  ok = ok && cudaMemcpyAsync(s->host_counts, L->counts, LIF_CNT_LEN * 4, cudaMemcpyDeviceToHost, st) ==
                 cudaSuccess;
  ok = ok && cudaMemcpyAsync(s->host_ids, L->load_ids, (size_t)D.capacity * 4, cudaMemcpyDeviceToHost,
                             st) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return LIF_ERR_CUDA;
  }
  const int n_load = s->host_counts[LIF_CNT_N_LOAD];
  if (n_load < 0 || n_load > D.capacity) return LIF_ERR_STATE;
  for (int j = 0; j < n_load; ++j)
    if (s->host_ids[j] < 0 || s->host_ids[j] >= D.d_ff) return LIF_ERR_STATE;
  // bundle load_ids[j] -> row j of the staging buffer (the layer's host_bundles)
  if (!read_batch(s, s->host_ids, n_load, const_cast<void*>(D.host_bundles))) return LIF_ERR_STATE;
  // staging row j -> cache row load_slots[j], then the FFN
  ok = launch_fetch_staged(L, st) == cudaSuccess;
  if (D.ffn_mode == 0)
    ok = ok && launch_ffn(L, x, L->active_slots, L->counts + LIF_CNT_N_ACTIVE, nullptr, dev_y, false,
                          st) == cudaSuccess;
  else
    ok = ok && launch_ffn(L, x, nullptr, L->counts + LIF_CNT_NUM_USED, nullptr, dev_y, false, st) ==
                   cudaSuccess;
  // the staging rows are rewritten by the next step's reads: the copy must have finished
  ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
  if (!ok) cudaGetLastError();
  return ok ? LIF_OK : LIF_ERR_CUDA;
}

}  // extern "C"
