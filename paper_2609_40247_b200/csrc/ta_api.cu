// C-ABI entry points (include/ta.h): argument checks, the handle, memory
// through the caller's allocator, call-order bookkeeping.  All arithmetic lives
// in the kernels of the other translation units.
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>

#include "ta_internal.cuh"

// Without caller callbacks memory comes from a private stream-ordered pool per device that
// keeps what it has been given (release threshold = everything): the default pool hands its
// memory back at every synchronisation, which makes each call pay for fresh gigabytes.
static cudaMemPool_t own_pool(int device) {
  static cudaMemPool_t pools[64] = {};
  static std::mutex guard;  // handles on different threads may arrive here together
  if (device < 0 || device >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(guard);
  if (!pools[device]) {
    cudaMemPoolProps props;
    memset(&props, 0, sizeof(props));
    props.allocType = cudaMemAllocationTypePinned;
    props.handleTypes = cudaMemHandleTypeNone;
    props.location.type = cudaMemLocationTypeDevice;
    props.location.id = device;
    cudaMemPool_t pool = nullptr;
    if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    unsigned long long keep = ~0ull;
    cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
    pools[device] = pool;
  }
  return pools[device];
}

// Blocks the library's own pool handed out are kept by exact size when they are released and
// given out again to a request of the same device, stream and size: successive windows ask for
// the same sizes in the same order, and the CUDA pool took 0.1 ms and more to carve a block of
// a new size out of what it holds (2.8 ms per 66.8 M record window).  A block is reused on the
// stream it was released on only, so stream order protects work still queued on it.  Blocks
// that no request has taken during the lifetime of the last two handles go back to the pool.
struct CachedBlock {
  void *p;
  size_t bytes;
  int device;
  cudaStream_t stream;
  unsigned long long gen;
};
static std::mutex g_cache_guard;
static std::vector<CachedBlock> g_cache;
static unsigned long long g_cache_gen = 0;

static void *cache_take(int device, cudaStream_t stream, size_t bytes) {
  std::lock_guard<std::mutex> lock(g_cache_guard);
  for (size_t i = 0; i < g_cache.size(); i++)
    if (g_cache[i].bytes == bytes && g_cache[i].device == device && g_cache[i].stream == stream) {
      void *p = g_cache[i].p;
      g_cache[i] = g_cache.back();
      g_cache.pop_back();
      return p;
    }
  return nullptr;
}
static void cache_put(int device, cudaStream_t stream, void *p, size_t bytes) {
  std::lock_guard<std::mutex> lock(g_cache_guard);
  g_cache.push_back(CachedBlock{p, bytes, device, stream, g_cache_gen});
}
// Called when a handle goes away, after its stream has been synchronised.  Invariant: a block
// enters the cache only once the stream it was used on is idle (ta_dfree and ta_free are only
// reached behind a synchronisation), so handing it back to the pool below cannot race with work
// still queued on that stream - cudaFree itself does not wait for a stream-ordered allocation.
static void cache_age() {
  std::vector<void *> out;
  {
    std::lock_guard<std::mutex> lock(g_cache_guard);
    g_cache_gen++;
    for (size_t i = 0; i < g_cache.size();) {
      if (g_cache[i].gen + 2 < g_cache_gen) {
        out.push_back(g_cache[i].p);
        g_cache[i] = g_cache.back();
        g_cache.pop_back();
      } else {
        i++;
      }
    }
  }
  for (void *p : out) cudaFree(p);  // the stream the block was used on may no longer exist
}

void *ta_dalloc(ta_window *h, size_t bytes) {
  if (bytes == 0) bytes = 256;
  void *p = nullptr;
  if (h->env.alloc) {
    p = h->env.alloc(bytes, h->env.ctx);
  } else if (!(p = cache_take(h->device, h->stream, bytes))) {
    cudaMemPool_t pool = own_pool(h->device);
    cudaError_t e = pool ? cudaMallocFromPoolAsync(&p, bytes, pool, h->stream)
                         : cudaMallocAsync(&p, bytes, h->stream);
    if (e != cudaSuccess) {
      cudaGetLastError();
      p = nullptr;
    }
  }
  if (p) {
    h->allocs.push_back(p);
    h->alloc_bytes.push_back(bytes);
  }
  return p;
}

static void release_one(ta_window *h, void *p, size_t bytes) {
  if (h->env.alloc) {
    if (h->env.release) h->env.release(p, h->env.ctx);
  } else {
    cache_put(h->device, h->stream, p, bytes);
  }
}

void ta_dfree(ta_window *h, void *p) {
  if (!p) return;
  for (size_t i = 0; i < h->allocs.size(); i++)
    if (h->allocs[i] == p) {
      const size_t bytes = h->alloc_bytes[i];
      h->allocs[i] = h->allocs.back();
      h->allocs.pop_back();
      h->alloc_bytes[i] = h->alloc_bytes.back();
      h->alloc_bytes.pop_back();
      release_one(h, p, bytes);
      return;
    }
}

// Page-locked staging blocks are expensive to create (a system call and a page-table update
// each), so they are kept for the life of the process and handed from handle to handle.
#define TA_PIN_BYTES (512u << 10)
static std::mutex g_pin_guard;
static std::vector<unsigned char *> g_pin_free;
static unsigned char *pin_take() {
  {
    std::lock_guard<std::mutex> lock(g_pin_guard);
    if (!g_pin_free.empty()) {
      unsigned char *p = g_pin_free.back();
      g_pin_free.pop_back();
      return p;
    }
  }
  void *p = nullptr;
  if (cudaHostAlloc(&p, TA_PIN_BYTES, cudaHostAllocPortable | cudaHostAllocMapped) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;  // the copies then go straight to their (pageable) destinations
  }
  return (unsigned char *)p;
}
static void pin_put(unsigned char *p) {
  if (!p) return;
  std::lock_guard<std::mutex> lock(g_pin_guard);
  g_pin_free.push_back(p);
}

// Writes up to TA_FETCH_MAX small device regions into the mapped staging block: one launch in
// place of one copy each (a copy costs some six microseconds of stream time, however small).
#define TA_FETCH_MAX 8
#define TA_FETCH_BYTES (16u << 10)
struct FetchList {
  const void *src[TA_FETCH_MAX];
  unsigned off[TA_FETCH_MAX], bytes[TA_FETCH_MAX];
};
__global__ void __launch_bounds__(256) k_collect(FetchList f, unsigned char *pin_dev) {
  const unsigned char *s = (const unsigned char *)f.src[blockIdx.x];
  unsigned char *d = pin_dev + f.off[blockIdx.x];
  const unsigned b = f.bytes[blockIdx.x];
  if ((((uintptr_t)s | (uintptr_t)b) & 7u) == 0) {
    for (unsigned i = threadIdx.x; i < b / 8; i += blockDim.x)
      reinterpret_cast<u64 *>(d)[i] = reinterpret_cast<const u64 *>(s)[i];
  } else {
    for (unsigned i = threadIdx.x; i < b; i += blockDim.x) d[i] = s[i];
  }
}
static ta_status flush_fetch(ta_window *h) {
  if (h->fetch.empty()) return TA_OK;
  FetchList f;
  memset(&f, 0, sizeof(f));
  const unsigned m = (unsigned)h->fetch.size();
  for (unsigned i = 0; i < m; i++) { f.src[i] = h->fetch[i].src; f.off[i] = h->fetch[i].off; f.bytes[i] = h->fetch[i].bytes; }
  h->fetch.clear();
  k_collect<<<TA_N m, 256, 0, h->stream>>>(f, h->pin_dev);
  TA_CHECK_CUDA(h, cudaGetLastError());
  return TA_OK;
}

ta_status ta_queue_d2h(ta_window *h, void *dst, const void *dev_src, size_t bytes) {
  if (bytes == 0) return TA_OK;
  const size_t need = (bytes + 15) & ~(size_t)15;
  if (h->pin_dev && bytes <= TA_FETCH_BYTES && h->pin_used + need <= h->pin_bytes) {
    if (h->fetch.size() == TA_FETCH_MAX) TA_TRY(flush_fetch(h));
    h->fetch.push_back(ta_window::Fetch{dev_src, (unsigned)h->pin_used, (unsigned)bytes});
    h->pending.push_back(ta_window::Pending{dst, h->pin_used, bytes});
    h->pin_used += need;
  } else if (h->pin && h->pin_used + need <= h->pin_bytes) {
    TA_CHECK_CUDA(h, cudaMemcpyAsync(h->pin + h->pin_used, dev_src, bytes, cudaMemcpyDeviceToHost, h->stream));
    h->pending.push_back(ta_window::Pending{dst, h->pin_used, bytes});
    h->pin_used += need;
  } else {
    TA_CHECK_CUDA(h, cudaMemcpyAsync(dst, dev_src, bytes, cudaMemcpyDeviceToHost, h->stream));
  }
  return TA_OK;
}

static void release_one(ta_window *h, void *p, size_t bytes);

ta_status ta_sync_fetch(ta_window *h) {
  const ta_status fs = flush_fetch(h);
  if (fs != TA_OK) { h->pending.clear(); h->pin_used = 0; return fs; }
  const cudaError_t e = cudaStreamSynchronize(h->stream);
  if (e == cudaSuccess)
    for (const ta_window::Pending &q : h->pending) memcpy(q.dst, h->pin + q.off, q.bytes);
  h->pending.clear();
  h->pin_used = 0;
  if (e != cudaSuccess) {
    h->last_cuda = e;
    return TA_ERR_CUDA;
  }
  for (void *p : h->deferred) ta_dfree(h, p);
  h->deferred.clear();
  return TA_OK;
}

ta_status ta_read_status(ta_window *h, int32_t *w) {
  TA_TRY(ta_queue_d2h(h, w, h->d_status, ST_WORDS * sizeof(int32_t)));
  return ta_sync_fetch(h);
}

void ta_dfree_later(ta_window *h, void *p) {
  if (p) h->deferred.push_back(p);
}

// Start of every entry point: copies an earlier call queued and never collected (it returned
// early with an error) must not be delivered to destinations that no longer exist.
// Also makes the handle's device current (it stays current when the call returns).
static ta_status begin_call(ta_window *h) {
  h->pending.clear();
  h->fetch.clear();
  h->pin_used = 0;
  if (cudaSetDevice(h->device) != cudaSuccess) {
    h->last_cuda = cudaGetLastError();
    return TA_ERR_CUDA;
  }
  return TA_OK;
}

// ---- test hooks: the poll limit of device-side waits, and a wait that nothing ends ----
static std::atomic<int> g_ta_spin_limit{0};  // 0 = TA_SPIN_LIMIT; copied into each new handle's status word

// One warp looks back from tile 1 at a tile-0 descriptor that nothing publishes.
__global__ void k_selftest_wait(u64 *state, int32_t *status) {
  bool failed;
  tile_lookback<OpAdd>(state, 1, 1ull, OpAdd(), status, &failed);
  if (threadIdx.x == 0) status[ST_LONG_RUN] = failed ? 1 : 0;
}

// ---- instrumentation: launch counter and event pairs around the radix passes ----
std::atomic<long long> g_ta_launches{0};
int g_ta_profile = 0;
static std::vector<cudaEvent_t> g_prof_events;  // begin, end, begin, end, ...
static size_t g_prof_used = 0;
static double g_prof_bytes = 0;  // algorithmic bytes of the timed passes

void ta_profile_mark(cudaStream_t st, int begin, double bytes) {
  if (begin) g_prof_bytes += bytes;
  if (g_prof_used == g_prof_events.size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    g_prof_events.push_back(e);
  }
  cudaEventRecord(g_prof_events[g_prof_used++], st);
}

extern "C" {

// Instrumentation helpers (they carry no work).  ta_profile_enable(1) makes the
// library record a CUDA event pair around every radix-sort pass and forgets the
// pairs recorded so far; ta_profile_radix reads them back (synchronises the
// events): number of passes timed and their summed duration in milliseconds.
void ta_profile_enable(int32_t on) {
  g_ta_profile = on;
  g_prof_used = 0;
  g_prof_bytes = 0;
}
int32_t ta_profile_radix(int64_t *n_passes, double *total_ms, double *total_bytes) {
  int64_t n = 0;
  double ms = 0;
  for (size_t i = 0; i + 1 < g_prof_used; i += 2) {
    if (cudaEventSynchronize(g_prof_events[i + 1]) != cudaSuccess) return -1;
    float t = 0;
    if (cudaEventElapsedTime(&t, g_prof_events[i], g_prof_events[i + 1]) != cudaSuccess) return -1;
    ms += t;
    n++;
  }
  if (n_passes) *n_passes = n;
  if (total_ms) *total_ms = ms;
  if (total_bytes) *total_bytes = g_prof_bytes;
  return 0;
}
int64_t ta_launch_count(void) { return g_ta_launches.load(); }

void ta_set_spin_limit(int32_t polls) { g_ta_spin_limit.store(polls > 0 ? polls : 0); }

ta_status ta_inject_device_error(ta_window *h, ta_status code) {
  if (!h || !h->d_status || code <= TA_OK || code > TA_ERR_BAD_NESTING) return TA_ERR_INVALID_ARG;
  if (cudaSetDevice(h->device) != cudaSuccess) return TA_ERR_CUDA;
  const int32_t c = (int32_t)code;
  TA_CHECK_CUDA(h, cudaMemcpyAsync(h->d_status + ST_ERR, &c, sizeof(c), cudaMemcpyHostToDevice, h->stream));
  TA_CHECK_CUDA(h, cudaStreamSynchronize(h->stream));
  return TA_OK;
}

ta_status ta_selftest_wait_timeout(void *cuda_stream, int32_t polls) {
  if (polls < 1 || polls > (1 << 20)) return TA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned char *buf = nullptr;
  if (cudaMallocAsync((void **)&buf, 512, st) != cudaSuccess) {
    cudaGetLastError();
    return TA_ERR_OOM;
  }
  u64 *state = (u64 *)buf;                    // two descriptors, both EMPTY
  int32_t *status = (int32_t *)(buf + 256);   // ST_WORDS words
  int32_t words[ST_WORDS];
  memset(words, 0, sizeof(words));
  words[ST_SPIN] = polls;
  cudaError_t e = cudaMemsetAsync(buf, 0, 512, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(status, words, sizeof(words), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) {
    k_selftest_wait<<<TA_N 1, 32, 0, st>>>(state, status);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(words, status, sizeof(words), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFreeAsync(buf, st);
  if (e != cudaSuccess) return TA_ERR_CUDA;
  // the kernel must have come back by itself, with the error recorded and nothing published
  if (words[ST_LONG_RUN] != 1) return TA_ERR_CUDA;
  return (ta_status)words[ST_ERR];
}

const char *ta_strerror(ta_status s) {
  switch (s) {
    case TA_OK: return "ok";
    case TA_ERR_INVALID_ARG: return "invalid argument";
    case TA_ERR_OOM: return "device allocation failed";
    case TA_ERR_CUDA: return "CUDA runtime error";
    case TA_ERR_ORDER: return "entry point called before its prerequisites";
    case TA_ERR_TOO_LARGE: return "size limit exceeded";
    case TA_ERR_OVERFLOW: return "internal table overflow";
    case TA_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case TA_ERR_DEPTH: return "operator nesting deeper than TA_MAX_DEPTH";
    case TA_ERR_BAD_NESTING: return "partially overlapping ranges on one host thread";
  }
  return "unknown status";
}

int32_t ta_version(void) { return 1; }

static ta_status load_impl(ta_window *h, const ta_event *events, int32_t on_device,
                           ta_load_summary *out_summary) {
  const int64_t n = h->n;
  const int W = h->W;
  cudaStream_t st = h->stream;
  // one device block: [off | t0 | t1 | misc] filled by one copy, [status | load summaries |
  // digit histograms] zeroed by one fill, [triple table | communicator table] emptied (all
  // ones) by one fill
  const size_t up_words = (size_t)(W + 1) + 2 * (size_t)W + 16;
  size_t bytes = Carver::pad(up_words * 8) + Carver::pad(ST_WORDS * 4) +
                 Carver::pad(sizeof(TripleTable)) + Carver::pad(sizeof(CommTable)) +
                 Carver::pad(W * sizeof(ta_load_summary)) + Carver::pad(10 * 256 * 4) +
                 Carver::pad(TA_TRIPLE_SLOTS * 4) + 256;
  void *b = ta_dalloc(h, bytes);
  if (!b) return TA_ERR_OOM;
  Carver c(b);
  int64_t *up = c.take<int64_t>(up_words);
  h->d_off = up;
  h->d_t0 = up + (W + 1);
  h->d_t1 = h->d_t0 + W;
  h->d_misc = h->d_t1 + W;
  char *zero_begin = c.base + c.off;
  h->d_status = c.take<int32_t>(ST_WORDS);
  h->d_load_sum = c.take<ta_load_summary>(W);
  h->d_hist = c.take<u32>(10 * 256);
  h->d_slot_cnt = c.take<u32>(TA_TRIPLE_SLOTS);
  char *zero_end = c.base + c.off;
  h->d_triples = c.take<TripleTable>(1);
  h->d_comms = c.take<CommTable>(1);
  char *ones_end = c.base + c.off;
  h->d_keys = (u64 *)ta_dalloc(h, (size_t)(n > 0 ? n : 1) * 8);
  if (!h->d_keys) return TA_ERR_OOM;

  if (!on_device) {
    h->events_copy = ta_dalloc(h, (size_t)(n > 0 ? n : 1) * sizeof(ta_event));
    if (!h->events_copy) return TA_ERR_OOM;
    if (n > 0)
      TA_CHECK_CUDA(h, cudaMemcpyAsync(h->events_copy, events, (size_t)n * sizeof(ta_event),
                                       cudaMemcpyHostToDevice, st));
    h->events = (const ta_event *)h->events_copy;
  } else {
    h->events = events;
  }
  {
    std::vector<int64_t> host(up_words, 0);
    memcpy(host.data(), h->h_off.data(), (size_t)(W + 1) * 8);
    memcpy(host.data() + (W + 1), h->h_t0.data(), (size_t)W * 8);
    memcpy(host.data() + (W + 1) + W, h->h_t1.data(), (size_t)W * 8);
    int64_t *misc_init = host.data() + (W + 1) + 2 * (size_t)W;
    misc_init[0] = INT64_MAX;  // min name
    misc_init[1] = INT64_MIN;  // max name
    misc_init[3] = INT64_MAX;  // min seq
    misc_init[4] = INT64_MIN;  // max seq
    // a pageable source is staged by the runtime before the call returns
    TA_CHECK_CUDA(h, cudaMemcpyAsync(up, host.data(), up_words * 8, cudaMemcpyHostToDevice, st));
  }
  TA_CHECK_CUDA(h, cudaMemsetAsync(zero_begin, 0, zero_end - zero_begin, st));
  TA_CHECK_CUDA(h, cudaMemsetAsync(zero_end, 0xFF, ones_end - zero_end, st));
  const int32_t spin = g_ta_spin_limit.load();
  if (spin > 0)
    TA_CHECK_CUDA(h, cudaMemcpyAsync(h->d_status + ST_SPIN, &spin, sizeof(spin), cudaMemcpyHostToDevice, st));

  TA_TRY(ta_launch_discover(h));

  int32_t words[ST_WORDS];
  int64_t misc[16];
  std::vector<ta_load_summary> sums(W);
  h->h_comm_sorted.assign(TA_MAX_COMMS, 0);
  TA_TRY(ta_queue_d2h(h, misc, h->d_misc, sizeof(misc)));
  TA_TRY(ta_queue_d2h(h, sums.data(), h->d_load_sum, W * sizeof(ta_load_summary)));
  TA_TRY(ta_queue_d2h(h, h->h_comm_sorted.data(), h->d_comms->sorted_id, TA_MAX_COMMS * sizeof(u64)));
  TA_TRY(ta_read_status(h, words));
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  h->n_triples = words[ST_N_TRIPLES];
  h->n_pids = words[ST_N_PIDS];
  h->min_name = misc[0];
  h->max_name = misc[1];
  h->max_dur = misc[2];
  h->min_seq = misc[3];
  h->max_seq = misc[4];
  h->n_coll = misc[5];
  if (h->tkeep < 0) h->tkeep = (int)misc[6];
  h->n_comms = words[ST_N_COMMS];
  h->h_comm_sorted.resize((size_t)h->n_comms);
  h->n_valid = 0;
  for (int w = 0; w < W; w++) {
    ta_load_summary &s = sums[w];
    s.n_events = h->h_off[w + 1] - h->h_off[w];
    s.n_valid = s.n_events - s.n_bad_kind - s.n_bad_interval - s.n_out_of_window;
    h->n_valid += s.n_valid;
    if (out_summary) out_summary[w] = s;
  }
  h->has_dropped = h->n_valid < n ? 1 : 0;
  TA_TRY(ta_launch_load(h, true));
  h->stage |= 1;
  return TA_OK;
}

ta_status ta_load_window(const ta_env *env, const ta_event *events, int64_t n,
                         int32_t events_on_device, const int64_t *win_off, const int64_t *win_t0,
                         const int64_t *win_t1, int32_t W, ta_load_summary *out_summary,
                         ta_window **handle) {
  if (!handle) return TA_ERR_INVALID_ARG;
  *handle = nullptr;
  if (!env || n < 0 || W < 1 || !win_off || !win_t0 || !win_t1 || (n > 0 && !events))
    return TA_ERR_INVALID_ARG;
  if (n >= (1ll << 31)) return TA_ERR_TOO_LARGE;
  if ((env->alloc == nullptr) != (env->release == nullptr)) return TA_ERR_INVALID_ARG;
  if (win_off[0] != 0 || win_off[W] != n) return TA_ERR_INVALID_ARG;
  for (int w = 0; w < W; w++) {
    if (win_off[w + 1] < win_off[w]) return TA_ERR_INVALID_ARG;
    if (win_t0[w] >= win_t1[w]) return TA_ERR_INVALID_ARG;
    if ((uint64_t)win_t1[w] - (uint64_t)win_t0[w] >= (1ull << 40)) return TA_ERR_TOO_LARGE;
  }
  ta_window *h = new (std::nothrow) ta_window();
  if (!h) return TA_ERR_OOM;
  h->env = *env;
  h->stream = (cudaStream_t)env->cuda_stream;
  h->device = env->device;
  h->last_cuda = cudaSuccess;
  h->n = n;
  h->W = W;
  h->stage = 0;
  h->events = nullptr;
  h->events_copy = nullptr;
  h->d_keys = nullptr;
  h->prekeys = 0;
  h->attr_status = 0;
  h->d_op_gap_ns = nullptr;
  h->d_on_path = nullptr;
  h->d_status = nullptr;
  h->pin = pin_take();
  h->pin_bytes = h->pin ? TA_PIN_BYTES : 0;
  h->pin_dev = nullptr;
  if (h->pin) {
    void *dp = nullptr;
    if (cudaHostGetDevicePointer(&dp, h->pin, 0) == cudaSuccess) h->pin_dev = (unsigned char *)dp;
    else cudaGetLastError();
  }
  h->pin_used = 0;
  h->h_off.assign(win_off, win_off + W + 1);
  h->h_t0.assign(win_t0, win_t0 + W);
  h->h_t1.assign(win_t1, win_t1 + W);
  *handle = h;
  TA_TRY(begin_call(h));
  return load_impl(h, events, events_on_device, out_summary);
}

ta_status ta_sort_timeline(ta_window *h, ta_sort_result *out) {
  if (!h || !out) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 1) || (h->stage & 2)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  TA_TRY(ta_run_sort_timeline(h));
  h->stage |= 2;
  *out = h->sorted;
  return TA_OK;
}

ta_status ta_correlate_launches(ta_window *h, ta_join_result *out, ta_join_summary *out_summary) {
  if (!h || !out) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 2) || (h->stage & 4)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  TA_TRY(ta_run_correlate(h, out_summary));
  h->stage |= 4;
  *out = h->join;
  return TA_OK;
}

ta_status ta_attribute_operators(ta_window *h, ta_attr_result *out, ta_attr_summary *out_summary) {
  if (!h || !out) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 4) || (h->stage & 8)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  ta_status s = ta_run_attribute(h, out_summary);
  if (s != TA_OK && s != TA_ERR_DEPTH && s != TA_ERR_BAD_NESTING) return s;
  h->stage |= 8;
  h->attr_status = (int)s;
  *out = h->attr;
  return s;
}

ta_status ta_stream_gaps(ta_window *h, int64_t min_gap_ns, ta_gap_result *out) {
  if (!h || !out) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 2)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_gaps(h, min_gap_ns, out);
}

ta_status ta_aggregate_ops(ta_window *h, uint32_t kind_mask, int32_t value_sel, ta_agg_result *out) {
  if (!h || !out) return TA_ERR_INVALID_ARG;
  if (value_sel < 0 || value_sel > 3) return TA_ERR_INVALID_ARG;
  if ((value_sel == 1 || value_sel == 2) && kind_mask != (1u << TA_KIND_OP)) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 2)) return TA_ERR_ORDER;
  if (value_sel == 1 && (!(h->stage & 8) || h->attr_status != 0)) return TA_ERR_ORDER;
  if (value_sel == 2 && !h->d_op_gap_ns) return TA_ERR_ORDER;
  if (value_sel == 3 && !h->d_on_path) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_aggregate(h, kind_mask, value_sel, out);
}

ta_status ta_match_collectives(ta_window *h, const ta_comm_size *sizes, int32_t n_comms,
                               ta_coll_result *out) {
  if (!h || !out || n_comms < 0 || (n_comms > 0 && !sizes)) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 2)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_collectives(h, sizes, n_comms, out);
}

ta_status ta_rollup_operators(ta_window *h, ta_rollup_result *out, ta_rollup_summary *out_summary) {
  if (!h || !out || !out_summary) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 8) || h->attr_status != 0) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_rollup(h, out, out_summary);
}

ta_status ta_operator_sol(ta_window *h, const double *flops, const double *bytes,
                          int32_t counts_on_device, double peak_flops, double peak_bw,
                          ta_sol_result *out, ta_sol_summary *out_summary) {
  if (!h || !out || !out_summary || (h->n > 0 && (!flops || !bytes))) return TA_ERR_INVALID_ARG;
  if (!(peak_flops > 0.0) || !(peak_bw > 0.0)) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 8) || h->attr_status != 0) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_sol(h, flops, bytes, counts_on_device, peak_flops, peak_bw, out, out_summary);
}

ta_status ta_blame_gaps(ta_window *h, const ta_gap_result *gaps, ta_blame_result *out,
                        ta_blame_summary *out_summary) {
  if (!h || !gaps || !out || !out_summary) return TA_ERR_INVALID_ARG;
  if (gaps->n_long_gaps < 0 || (gaps->n_long_gaps > 0 && !gaps->long_gaps)) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 4)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_blame(h, gaps, out, out_summary);
}

ta_status ta_critical_path(ta_window *h, ta_critpath_result *out, ta_critpath_summary *out_summary) {
  if (!h || !out || !out_summary) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 4)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_critpath(h, out, out_summary);
}

ta_status ta_device_overlap(ta_window *h, ta_overlap_result *out) {
  if (!h || !out) return TA_ERR_INVALID_ARG;
  if (!(h->stage & 2)) return TA_ERR_ORDER;
  TA_TRY(begin_call(h));
  return ta_run_overlap(h, out);
}

void ta_free(ta_window *h) {
  if (!h) return;
  cudaSetDevice(h->device);
  cudaStreamSynchronize(h->stream);
  for (size_t i = 0; i < h->allocs.size(); i++) release_one(h, h->allocs[i], h->alloc_bytes[i]);
  h->allocs.clear();
  h->alloc_bytes.clear();
  pin_put(h->pin);
  const bool own = !h->env.alloc;
  delete h;
  if (own) cache_age();
}

}  // extern "C"
