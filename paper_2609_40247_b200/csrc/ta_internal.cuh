// Internal declarations of the trace-window analyzer CUDA library (sm_100a).
// Host-side handle, memory helpers, and the device primitives every step
// shares: relaxed loads/stores for tile descriptors, a bounded decoupled
// look-back, warp/block scans.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "../../include/ta.h"

typedef unsigned long long u64;
typedef long long i64;
typedef unsigned int u32;

// ---------------------------------------------------------------- limits
#define TA_MAX_TRIPLES 4096       // distinct (pid, domain, stream)
#define TA_TRIPLE_SLOTS 8192      // open-addressing slots for them
#define TA_MAX_COMMS 1024         // distinct communicator ids
#define TA_COMM_SLOTS 2048
#define TA_SPIN_LIMIT (1 << 22)   // polls of a tile descriptor before giving up
#define TA_TIE_RUN_MAX 48         // equal-key runs up to this length are fixed in place
#define TA_PACK_MAX_DROP 12        // low time bits a packed key may give up
#define TA_AGG_DENSE_LIMIT (1ll << 27)

// device status word indices (h->d_status)
// ST_SPIN: polls a device-side wait may make before it gives up (0 = TA_SPIN_LIMIT)
enum { ST_ERR = 0, ST_LONG_RUN = 1, ST_N_TRIPLES = 2, ST_N_PIDS = 3, ST_N_COMMS = 4, ST_SPIN = 5,
       ST_WORDS = 16 };

struct TripleTable {       // device-resident, filled by the discovery kernel
  u64 slots[TA_TRIPLE_SLOTS];          // biased code or EMPTY
  int32_t rank_of_slot[TA_TRIPLE_SLOTS];
  u64 sorted_code[TA_MAX_TRIPLES];     // ascending
  int32_t pid_rank[TA_MAX_TRIPLES];    // per triple rank
  int32_t pid_value[TA_MAX_TRIPLES];   // per pid rank
};

struct CommTable {         // communicator ids seen on COLL records (biased; all-ones = empty)
  u64 slots[TA_COMM_SLOTS];
  int32_t rank_of_slot[TA_COMM_SLOTS];
  u64 sorted_id[TA_MAX_COMMS];         // ascending (biased)
};

struct SortPlan {
  int n_pass;
  int shift[10];
  int bits[10];
};
// Passes over key bits [lo_bit, hi_bit): as few digits of at most 8 bits as cover them, the
// bits spread evenly.  Host and device build the same plan from the same two numbers.
#ifdef __CUDACC__
__host__ __device__
#endif
static inline SortPlan ta_plan_bits(int lo_bit, int hi_bit) {
  SortPlan p;
  int total = hi_bit - lo_bit;
  if (total < 1) total = 1;
  p.n_pass = (total + 7) / 8;
  int b = lo_bit;
  for (int i = 0; i < 10; i++) { p.shift[i] = 0; p.bits[i] = 0; }
  for (int i = 0; i < p.n_pass; i++) {
    const int w = (total - (b - lo_bit) + (p.n_pass - i) - 1) / (p.n_pass - i);
    p.shift[i] = b;
    p.bits[i] = w;
    b += w;
  }
  return p;
}

// --------------------------------------------------------------- handle
struct ta_window {
  ta_env env;
  cudaStream_t stream;
  int device;
  cudaError_t last_cuda;
  int64_t n;
  int32_t W;
  int stage;  // bit flags: 1 loaded, 2 sorted, 4 correlated, 8 attributed

  const ta_event *events;  // device, borrowed (or events_copy)
  void *events_copy;
  std::vector<int64_t> h_off, h_t0, h_t1;
  int64_t *d_off, *d_t0, *d_t1;

  std::vector<void *> allocs;  // everything obtained from env.alloc (or the library's own pool)
  std::vector<size_t> alloc_bytes;  // their sizes, same order
  std::vector<void *> deferred;  // temporaries to release after the next synchronisation

  // device -> host results of the call in progress: copies are queued into one page-locked
  // staging block (truly asynchronous, unlike a copy into pageable memory, which blocks until
  // it is done) and handed to their destinations after the call's one synchronisation
  unsigned char *pin;
  size_t pin_bytes, pin_used;
  struct Pending { void *dst; size_t off, bytes; };
  std::vector<Pending> pending;
  // small results (status words, per-window summaries) are not copied one by one: one kernel
  // at the end of the call writes them all into the staging block through its device alias
  unsigned char *pin_dev;  // device address of `pin`, null when the block is not mapped
  struct Fetch { const void *src; unsigned off, bytes; };
  std::vector<Fetch> fetch;

  // load products
  int32_t *d_status;
  TripleTable *d_triples;
  int64_t *d_misc;           // [0]=min name,[1]=max name,[2]=max duration,[3]=min seq,[4]=max seq,
                             // [5]=kept COLL records
  CommTable *d_comms;
  int n_comms;
  std::vector<u64> h_comm_sorted;  // host copy of the ranked communicator ids (biased)
  int64_t min_seq, max_seq, n_coll;
  ta_load_summary *d_load_sum;
  u64 *d_keys;
  int prekeys;               // d_keys holds the words of the discovery pass, not keys yet
  u32 *d_hist;               // [pass][256]
  int64_t n_valid;
  int n_triples, n_pids;
  int sbits, tbits, wbits, has_dropped;
  int packed, dshift, ibits;   // packed keys: low ibits = index inside the window, dshift low time bits dropped
  int tkeep;                   // time bits the planning kernel decided to keep (0 = it did not run)
  int fast_keys;               // the first radix pass builds the keys from the discovery words itself
  u32 *d_slot_cnt;             // kept records per triple slot (one window only), or null
  int64_t min_name, max_name, max_dur;
  SortPlan plan;

  // sort products
  ta_sort_result sorted;
  int32_t *d_lane_code;      // per lane: window << tbits | triple rank
  int32_t *d_lane_slot;      // per lane: window * n_pids + pid rank
  int32_t *d_lane_dom_end;   // per lane: first position behind the run of lanes of the same domain
  int32_t *d_lane_dev_base;  // per device lane: number of device records in earlier lanes
  int32_t *d_lane_dom_next;  // per lane: index of the first later lane of the other domain
  int64_t n_device;          // kept device records
  i64 *d_slot_min, *d_slot_max;               // per slot: corr_id range of its LAUNCH records
  std::vector<int64_t> h_slot_min, h_slot_max;  // host copies (INT64_MAX / INT64_MIN when none)

  // join / attribution products
  ta_join_result join;
  ta_attr_result attr;
  const int64_t *d_op_gap_ns;  // per sorted position, set by the gap blame (null before)
  const uint8_t *d_on_path;    // per sorted position, set by the critical path (null before)
  int attr_status;
};

// number of bits needed to write v (0 for 0)
static inline int ta_bit_len(uint64_t v) {
  int b = 0;
  while (v) { b++; v >>= 1; }
  return b;
}

// -------------------------------------------------------------- memory
void *ta_dalloc(ta_window *h, size_t bytes);            // NULL on failure
void ta_dfree(ta_window *h, void *p);                   // early release of one allocation
// carve sub-buffers out of one allocation
struct Carver {
  char *base;
  size_t off;
  explicit Carver(void *b = nullptr) : base((char *)b), off(0) {}
  static size_t pad(size_t b) { return (b + 255) & ~(size_t)255; }
  template <class T>
  T *take(size_t count) {
    T *p = (T *)(base + off);
    off += pad(count * sizeof(T));
    return p;
  }
};

#define TA_CHECK_CUDA(h, x)                                  \
  do {                                                       \
    cudaError_t e__ = (x);                                   \
    if (e__ != cudaSuccess) {                                \
      (h)->last_cuda = e__;                                  \
      return TA_ERR_CUDA;                                    \
    }                                                        \
  } while (0)
#define TA_TRY(x)                      \
  do {                                 \
    ta_status s__ = (x);               \
    if (s__ != TA_OK) return s__;      \
  } while (0)

// ----------------------------------------------- launchers (one per .cu)
// sort.cu
size_t ta_sort_temp_bytes(int64_t n);
ta_status ta_radix_sort_pairs(ta_window *h, const u64 *keys_in, const u32 *vals_in,
                              u64 *keys_scratch, u32 *vals_scratch, u64 *keys_final,
                              u32 *vals_final, int64_t n, const SortPlan &plan,
                              const u32 *hist /*nullable*/, void *temp);
// How the first pass of the timeline sort turns a discovery word into a key on the fly.
struct PrekeyInfo {
  const int64_t *off;          // window offsets (device), W + 1
  int W;
  const int32_t *rank_of_slot; // triple slot -> rank
  int tbits, wbits, tsb, dshift, ibits;  // tsb = time bits kept
};
ta_status ta_radix_sort_keys(ta_window *h, const u64 *keys_in, u64 *keys_scratch, u64 *keys_final,
                             int64_t n, const SortPlan &plan, const u32 *hist /*nullable*/,
                             void *temp,
                             bool first_pass_unstable, const PrekeyInfo *prekey = nullptr);
SortPlan ta_make_plan(int lo_bit, int hi_bit);
// load.cu
ta_status ta_launch_discover(ta_window *h);
ta_status ta_launch_rank_triples(ta_window *h);
ta_status ta_launch_load(ta_window *h, bool allow_packed);
// timeline.cu
ta_status ta_run_sort_timeline(ta_window *h);
// join.cu
ta_status ta_run_correlate(ta_window *h, ta_join_summary *out_summary);
// attr.cu
ta_status ta_run_attribute(ta_window *h, ta_attr_summary *out_summary);
// gaps.cu
ta_status ta_run_gaps(ta_window *h, int64_t min_gap, ta_gap_result *out);
// agg.cu
ta_status ta_run_aggregate(ta_window *h, uint32_t kind_mask, int value_sel, ta_agg_result *out);
// coll.cu
ta_status ta_run_collectives(ta_window *h, const ta_comm_size *sizes, int32_t n_comms,
                             ta_coll_result *out);

// overlap.cu
ta_status ta_run_overlap(ta_window *h, ta_overlap_result *out);
// rollup.cu
ta_status ta_run_rollup(ta_window *h, ta_rollup_result *out, ta_rollup_summary *out_summary);
// sol.cu
ta_status ta_run_sol(ta_window *h, const double *flops, const double *bytes, int on_device,
                     double peak_flops, double peak_bw, ta_sol_result *out, ta_sol_summary *out_summary);
// blame.cu
ta_status ta_run_blame(ta_window *h, const ta_gap_result *gaps, ta_blame_result *out,
                       ta_blame_summary *out_summary);

// critpath.cu
ta_status ta_run_critpath(ta_window *h, ta_critpath_result *out, ta_critpath_summary *out_summary);

// Queues a device -> host copy of the call in progress; *dst is valid after the next
// ta_read_status / ta_sync_fetch.
ta_status ta_queue_d2h(ta_window *h, void *dst, const void *dev_src, size_t bytes);
// One stream synchronisation: delivers the queued copies and releases deferred temporaries.
ta_status ta_sync_fetch(ta_window *h);
// The same, with the device status words.
ta_status ta_read_status(ta_window *h, int32_t *host_words /*ST_WORDS*/);
// Releases a temporary that queued work may still use: after the next synchronisation.
void ta_dfree_later(ta_window *h, void *p);


// ---- instrumentation (no work: a launch counter and optional event pairs) ----
extern std::atomic<long long> g_ta_launches;  // kernels launched by this library since load
extern int g_ta_profile;          // 1 = record a CUDA event pair around each radix pass
static inline unsigned ta_one() { ++g_ta_launches; return 1u; }
#define TA_N ta_one() *           // used as kernel<<<TA_N grid, ...>>>: counts the launch
void ta_profile_mark(cudaStream_t st, int begin, double bytes);  // called around k_radix_pass when profiling

// =================================================================== device
#ifdef __CUDACC__

__device__ __forceinline__ u64 ld_relaxed(const u64 *p) {
  u64 v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(u64 *p, u64 v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ int32_t ld_relaxed_i32(const int32_t *p) {
  int32_t v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ void ta_set_err(int32_t *status, int code) {
  atomicCAS(&status[ST_ERR], 0, code);
}
// Failure rule of the library: once the status word holds an error other than the data error
// TA_ERR_DEPTH (a bounded wait gave up, a bounded table filled), intermediate buffers may be
// incomplete, so every kernel launched afterwards returns before it indexes with anything an
// earlier kernel produced.  ta_peek_err issues the load (kernels call it first and test the
// value after their first position-only loads, so that the load costs no latency of its own).
__device__ __forceinline__ int ta_peek_err(const int32_t *status) { return __ldcg(&status[ST_ERR]); }
__device__ __forceinline__ bool ta_is_failure(int err) { return err != 0 && err != TA_ERR_DEPTH; }
__device__ __forceinline__ bool ta_failed(const int32_t *status) { return ta_is_failure(ta_peek_err(status)); }

// Tile descriptor: bits 63..62 = flag, low 62 bits = value.
#define TD_EMPTY 0ull
#define TD_AGG 1ull
#define TD_PREFIX 2ull
#define TD_MASK ((1ull << 62) - 1)
__device__ __forceinline__ u64 td_pack(u64 flag, u64 v) { return (flag << 62) | (v & TD_MASK); }

// Polls a descriptor until it is published; gives up after status[ST_SPIN] polls (TA_SPIN_LIMIT
// when that word is 0), or as soon as another wait has given up: sets *timed_out, records
// TA_ERR_TIMEOUT and returns a PREFIX of 0 so that the caller's loop terminates.  A caller whose
// wait timed out publishes no inclusive prefix and writes no output.
__device__ __forceinline__ u64 td_wait(const u64 *p, int32_t *status, bool *timed_out) {
  u64 w = ld_relaxed(p);
  int spins = 0, limit = 0;
  while ((w >> 62) == TD_EMPTY) {
    if (limit == 0) {
      limit = ld_relaxed_i32(&status[ST_SPIN]);
      if (limit <= 0) limit = TA_SPIN_LIMIT;
    }
    if (++spins > limit || ta_is_failure(ld_relaxed_i32(&status[ST_ERR]))) {
      *timed_out = true;
      ta_set_err(status, TA_ERR_TIMEOUT);
      return td_pack(TD_PREFIX, 0);
    }
    __nanosleep(40);
    w = ld_relaxed(p);
  }
  return w;
}

struct OpAdd {
  __device__ __forceinline__ u64 operator()(u64 a, u64 b) const { return a + b; }
  __device__ __forceinline__ u64 identity() const { return 0; }
};
struct OpMax {
  __device__ __forceinline__ u64 operator()(u64 a, u64 b) const { return a > b ? a : b; }
  __device__ __forceinline__ u64 identity() const { return 0; }
};

template <class Op>
__device__ __forceinline__ u64 warp_reduce(u64 v, Op op) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = op(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Maximum over the warp in two hardware reductions (high words, then the low words of the lanes
// that hold the largest high word) instead of five shuffle rounds on 64-bit values.
__device__ __forceinline__ u64 warp_reduce(u64 v, OpMax) {
  const u32 hi = (u32)(v >> 32);
  const u32 mh = __reduce_max_sync(0xffffffffu, hi);
  const u32 ml = __reduce_max_sync(0xffffffffu, hi == mh ? (u32)v : 0u);
  return ((u64)mh << 32) | ml;
}
// Sum over the warp (mod 2^64) in three hardware reductions: limbs of 22 bits, so that 32 of
// them cannot overflow a 32-bit sum.
__device__ __forceinline__ u64 warp_reduce(u64 v, OpAdd) {
  const u32 s0 = __reduce_add_sync(0xffffffffu, (u32)v & 0x3FFFFFu);
  const u32 s1 = __reduce_add_sync(0xffffffffu, (u32)(v >> 22) & 0x3FFFFFu);
  const u32 s2 = __reduce_add_sync(0xffffffffu, (u32)(v >> 44));
  return (u64)s0 + ((u64)s1 << 22) + ((u64)s2 << 44);
}
template <class Op>
__device__ __forceinline__ u64 warp_scan_inclusive(u64 v, Op op) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    u64 t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v = op(t, v);
  }
  return v;
}

// Decoupled look-back for one value per tile; called by all 32 lanes of ONE
// warp.  Publishes this tile's aggregate, combines the predecessors' values
// (commutative op) and publishes the inclusive prefix.  Returns the exclusive
// prefix in every lane.  *failed (the same in every lane) is set when a wait
// gave up: the prefix is then incomplete, nothing more is published (tiles
// behind this one run into the same unpublished descriptor, or into the error
// word, and fail too) and the caller must not write any output.
template <class Op>
__device__ __forceinline__ u64 tile_lookback(u64 *state, int tile, u64 aggregate, Op op,
                                             int32_t *status, bool *failed) {
  const int lane = threadIdx.x & 31;
  *failed = false;
  if (tile == 0) {
    if (lane == 0) st_relaxed(&state[0], td_pack(TD_PREFIX, aggregate));
    return op.identity();
  }
  if (lane == 0) st_relaxed(&state[tile], td_pack(TD_AGG, aggregate));
  u64 excl = op.identity();
  bool timed_out = false;
  for (int base = tile - 1;; base -= 32) {
    int idx = base - lane;
    u64 w = idx >= 0 ? td_wait(&state[idx], status, &timed_out) : td_pack(TD_PREFIX, op.identity());
    u32 pm = __ballot_sync(0xffffffffu, (w >> 62) == TD_PREFIX);
    int first = pm ? (__ffs(pm) - 1) : 31;
    u64 c = lane <= first ? (w & TD_MASK) : op.identity();
    c = warp_reduce(c, op);
    excl = op(c, excl);
    if (__any_sync(0xffffffffu, timed_out)) {
      *failed = true;
      return excl;
    }
    if (pm) break;
  }
  if (lane == 0) st_relaxed(&state[tile], td_pack(TD_PREFIX, op(excl, aggregate)));
  return excl;
}

// Block-wide exclusive scan of one value per thread (blockDim.x multiple of 32,
// <= 1024).  `smem` needs 33 u64.  Returns the exclusive prefix; *total gets the
// block aggregate in every thread.
template <class Op>
__device__ __forceinline__ u64 block_scan_exclusive(u64 v, Op op, u64 *smem, u64 *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  u64 inc = warp_scan_inclusive(v, op);
  if (lane == 31) smem[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    u64 w = lane < nw ? smem[lane] : op.identity();
    u64 wi = warp_scan_inclusive(w, op);
    if (lane < nw) smem[lane] = wi;
    if (lane == nw - 1) smem[32] = wi;
  }
  __syncthreads();
  u64 prev_lane = __shfl_up_sync(0xffffffffu, inc, 1);
  u64 ex = lane == 0 ? op.identity() : prev_lane;
  if (warp > 0) ex = op(smem[warp - 1], ex);
  *total = smem[32];
  __syncthreads();
  return ex;
}

// True when no record of [p, p_end) lies in a lane of domain `want`; l = lane of p.
__device__ __forceinline__ bool span_outside_domain(const int16_t *lane_domain,
                                                    const int32_t *lane_dom_end, int l,
                                                    int64_t p_end, int want) {
  return lane_domain[l] != want && (int64_t)lane_dom_end[l] >= p_end;
}
// Lane of a sorted position: binary search in lane_off (n_lanes + 1 entries).
__device__ __forceinline__ int lane_of_pos(const int32_t *lane_off, int n_lanes, int64_t p) {
  int lo = 0, hi = n_lanes - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if ((int64_t)lane_off[mid] <= p) lo = mid;
    else hi = mid - 1;
  }
  return lo;
}

// Hash of a triple code or a biased communicator id: 32-bit mixing of the two halves (the
// tables it indexes hold a few dozen entries; a 64-bit multiply per record is not worth it).
__device__ __forceinline__ u32 hash_code(u64 c) {
  u32 h = (u32)c * 0x9E3779B1u ^ (u32)(c >> 32) * 0x85EBCA77u;
  h ^= h >> 15;
  h *= 0x2C1B3C6Du;
  h ^= h >> 13;
  return h;
}

__device__ __forceinline__ int log2_bin(int64_t v) {
  if (v <= 1) return 0;
  int b = 63 - __clzll(v);
  return b > TA_NBINS - 1 ? TA_NBINS - 1 : b;
}

#endif  // __CUDACC__
