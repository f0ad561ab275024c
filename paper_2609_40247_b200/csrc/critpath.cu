// ta_critical_path: per (window, process) the chain of binding dependencies that ends
// at the last record to finish.  Three kinds of dependency are followed (a kernel on
// its launch, a record on its predecessor in the same stream or thread, a waiting call
// on the device record that released it); a delay the trace explains by none of them
// is reported as unresolved (Sec. 6.1, "Execution progress and state"; Fig. "Critical path").
//
// Nodes are the API / LAUNCH records of the host lanes and the records of the device
// lanes; each has a START and an END point.  The path is the backward walk from the END
// of the sink that always steps to the dependency released last (include/ta.h states the
// rules).  Walking record by record would be one long pointer chase, so the step is
// reshaped around the two kinds of edge:
//   - edges that stay in a lane (stream order, program order) link NEIGHBOURS, so a lane
//     falls into runs, and the run of any record is found by a max-scan of "last position
//     where a run starts";
//   - edges that change lane (submission: device -> host; synchronisation: host -> device)
//     are the only ones the walk itself has to follow.
// Kernels:
//   (in-order streams end their records in ascending order: then "the device record of the
//   process that finished last before t" - needed per API record and for the sink - is one
//   binary search per stream lane; k_cp_classify checks the order on the way, and only if some
//   record ends before the one in front of it the step starts over with)
//   k_cp_keys      (slot, ts_end) keys of the device records and a stable radix sort, after
//                  which the same question is one binary search in the sorted keys;
//   k_cp_classify  device records: which dependency binds (stream order / submission /
//                  none); API records: the record whose end released the wait; per slot the
//                  latest end among host nodes;
//   k_cp_runs      two chained max-scans over the sorted positions: the host node before
//                  each host node, then the head of every run (device: last record whose
//                  binding edge leaves the lane; host: last wait that was released by the
//                  device and is entered from its END);
//                  the waits that head a host run go to a list (they are few);
//   k_cp_succ      per listed wait, the next wait down the path: wait -> the record that
//                  released it -> head of that device run -> its launch -> head of that host run;
//   k_cp_start     one thread per slot: the sink, and the hops from it to the first listed wait;
//   k_cp_double    pointer doubling over the list: a wait reached from a marked wait is marked,
//                  successors are squared; after log2(list) rounds exactly the waits on a path
//                  are marked, whatever the length of the chain;
//   k_cp_enter     every marked wait records where the walk enters the two runs that follow it;
//   k_cp_mark      every record decides from its run's entry whether it is on the path and
//                  adds its share of the eight time classes (folded per warp);
//   a scan         compacts the slots that have a path into rows.
// HBM traffic: three passes over the columns (plus the sort, 8 B + 8 B per device record and
// pass, when it is needed); the chain of lane changes costs a few short kernels over the list of waits.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define CP_THREADS 256
#define CP_ITEMS 8
#define CP_TILE (CP_THREADS * CP_ITEMS)
#define CP_ACC 12  // per slot: nodes, eight classes, begin, reason, sink + 1

enum { CP_LINK_END = 0, CP_LINK_STREAM = 1, CP_LINK_SUBMIT = 2 };

struct CpArgs {
  int64_t n, n_valid, m;  // m = device records
  int n_lanes, n_pids;
  int64_t n_slots;
  const int16_t *kind;
  const int64_t *ts, *te;
  const int32_t *launch_of;
  const int64_t *latency;  // ts_start - ts_start of the launch, for records with a launch
  const int32_t *lane_off, *lane_slot, *lane_window, *lane_dom_end, *lane_dev_base, *lane_dom_next;
  const int16_t *lane_domain;
  const int64_t *t0;
  int tsbits, idxbits;
  int use_sort;         // 0: every device lane is taken to end in ascending order (checked), no sort
  u32 *not_ascending;   // set when some device record ends before the one in front of it in its lane
  u64 *keys;            // [device record index] ((slot << tsbits) | ts_end - t0) << idxbits | index
  u32 *pos;             // [device record index] sorted position
  const u64 *skeys;     // sorted keys
  const u32 *spos;      // pairs: sorted position of element i; packed keys: = pos
  uint8_t *link;        // device records: CP_LINK_*
  int32_t *cross;       // API records: device record whose end released the wait, or -1
  int32_t *prev_node;   // host nodes: the node before it in its lane, or -1
  int32_t *head;        // nodes: head of the run (host: -1 = the run reaches the lane start)
  int32_t *entry;       // [position of a run head] where the walk entered that run, or -1
  int32_t *entry_lane;  // [lane] the same for host runs that reach the lane start
  u64 *slot_host_te;    // per slot: latest end among host nodes (order-preserving code, 0 = none)
  int32_t *slot_host_pos;  // per slot: highest position among the host nodes that end then
  u64 *st_a, *st_b;     // tile descriptors of the two scans
  u32 *counter;
  u32 *n_eff;           // length of the list below
  u32 *eff_pos;         // positions of the waits that head a host run, in no particular order
  int32_t *id_of;       // [position] index in that list, or -1
  int32_t *jump_in, *jump_out;  // per listed wait: the wait 2^round steps down the path, or -1
  uint8_t *mark;        // per listed wait: on a path
  int64_t n_list;
  u64 *acc;             // [slot][CP_ACC]
  uint8_t *on_path;
  int32_t *status;
};

__device__ __forceinline__ u64 cp_code(i64 v) { return (u64)v ^ (1ull << 63); }
__device__ __forceinline__ bool cp_host_node(int k) { return k == TA_KIND_API || k == TA_KIND_LAUNCH; }
__device__ __forceinline__ bool cp_device(int k) { return k >= TA_KIND_KERNEL; }

// sorted position of the element at index i of the sorted key array
__device__ __forceinline__ int32_t cp_pos_of(const CpArgs &a, int64_t i) {
  if (a.idxbits) return (int32_t)a.pos[a.skeys[i] & ((1ull << a.idxbits) - 1)];
  return (int32_t)a.spos[i];
}

// Device lanes of one (window, process) are neighbours in the lane table.  When the ends of every
// lane ascend, the record of the process that ended last before `limit` (or at all, limit =
// INT64_MAX and `inclusive`) is the best of one binary search per lane: greatest ts_end, then
// the highest position.
__device__ __forceinline__ int32_t cp_last_ended(const CpArgs &a, int first_dev_lane, int slot, i64 limit,
                                                 bool inclusive) {
  int32_t best = -1;
  i64 best_e = 0;
  for (int dl = first_dev_lane; dl >= 0 && dl < a.n_lanes && a.lane_slot[dl] == slot && a.lane_domain[dl] == 1; dl++) {
    int64_t lo = a.lane_off[dl], hi = a.lane_off[dl + 1];  // first position of the lane that ends at / after the limit
    const int64_t begin = lo;
    while (lo < hi) {
      const int64_t mid = (lo + hi) >> 1;
      const i64 e = a.te[mid];
      if (inclusive ? e <= limit : e < limit) lo = mid + 1;
      else hi = mid;
    }
    if (lo > begin) {
      const i64 e = a.te[lo - 1];
      if (best < 0 || e >= best_e) { best = (int32_t)(lo - 1); best_e = e; }
    }
  }
  return best;
}

// lane bookkeeping of a thread that visits ascending positions
struct CpLane {
  const CpArgs &a;
  int l;
  int64_t cur_off, next_off;
  __device__ __forceinline__ CpLane(const CpArgs &args, int lane0) : a(args), l(lane0) {
    cur_off = a.lane_off[l];
    next_off = a.lane_off[l + 1];
  }
  __device__ __forceinline__ void to(int64_t p) {
    while (p >= next_off) {
      l++;
      cur_off = next_off;
      next_off = a.lane_off[l + 1];
    }
  }
};

__device__ __forceinline__ int cp_tile_lane(const CpArgs &a, int64_t tile_start, int *s_lane0) {
  if (threadIdx.x < 32) {
    const int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (threadIdx.x == 0) *s_lane0 = l;
  }
  __syncthreads();
  return *s_lane0;
}

// ---- keys of the device records ------------------------------------------------------
__global__ void __launch_bounds__(CP_THREADS) k_cp_keys(CpArgs a) {
  if (ta_failed(a.status)) return;
  __shared__ int s_lane0;
  const int64_t tile_start = (int64_t)blockIdx.x * CP_TILE;
  if (tile_start >= a.n_valid) return;
  const int l0 = cp_tile_lane(a, tile_start, &s_lane0);
  const int64_t tile_end = min(tile_start + CP_TILE, a.n_valid);
  if (span_outside_domain(a.lane_domain, a.lane_dom_end, l0, tile_end, 1)) return;
  const int64_t p0 = tile_start + (int64_t)threadIdx.x * CP_ITEMS;
  if (p0 >= tile_end) return;
  i64 e[CP_ITEMS];
  load8_i64(a.te, p0, a.n, e);
  CpLane ln(a, l0);
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++) {
    const int64_t p = p0 + j;
    if (p >= tile_end) break;
    ln.to(p);
    if (a.lane_domain[ln.l] != 1) continue;
    const int64_t c = a.lane_dev_base[ln.l] + (p - ln.cur_off);
    const u64 rel = (u64)(e[j] - a.t0[a.lane_window[ln.l]]);
    a.keys[c] = ((((u64)a.lane_slot[ln.l] << a.tsbits) | rel) << a.idxbits) | (a.idxbits ? (u64)c : 0ull);
    a.pos[c] = (u32)p;
  }
}

// ---- binding dependency of device records, waits of API records ------------------------
__global__ void __launch_bounds__(CP_THREADS, 3) k_cp_classify(CpArgs a) {
  if (ta_failed(a.status)) return;
  __shared__ int s_lane0;
  const int64_t tile_start = (int64_t)blockIdx.x * CP_TILE;
  if (tile_start >= a.n_valid) return;
  const int l0 = cp_tile_lane(a, tile_start, &s_lane0);
  const int64_t tile_end = min(tile_start + CP_TILE, a.n_valid);
  const int64_t p0 = tile_start + (int64_t)threadIdx.x * CP_ITEMS;
  if (p0 >= tile_end) return;
  int16_t kd[CP_ITEMS];
  i64 s[CP_ITEMS], e[CP_ITEMS];
  load8_i16(a.kind, p0, a.n, -1, kd);
  load8_i64(a.ts, p0, a.n, s);
  load8_i64(a.te, p0, a.n, e);
  const i64 e_before = p0 > 0 ? a.te[p0 - 1] : 0;
  // start of the launch = own start - launch latency: two sequential columns, no gather
  int32_t lo[CP_ITEMS];
  i64 sl[CP_ITEMS];
  bool any_dev = false;
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++) {
    lo[j] = -1;
    sl[j] = 0;
    any_dev |= p0 + j < tile_end && (kd[j] == TA_KIND_KERNEL || kd[j] == TA_KIND_MEMCPY);
  }
  if (any_dev) {
    if (p0 + CP_ITEMS <= a.n) {
      const int4 x = *reinterpret_cast<const int4 *>(a.launch_of + p0), y = *reinterpret_cast<const int4 *>(a.launch_of + p0 + 4);
      lo[0] = x.x; lo[1] = x.y; lo[2] = x.z; lo[3] = x.w;
      lo[4] = y.x; lo[5] = y.y; lo[6] = y.z; lo[7] = y.w;
    } else {
#pragma unroll
      for (int j = 0; j < CP_ITEMS; j++)
        if (p0 + j < a.n) lo[j] = a.launch_of[p0 + j];
    }
    load8_i64(a.latency, p0, a.n, sl);
#pragma unroll
    for (int j = 0; j < CP_ITEMS; j++) {
      if (!(kd[j] == TA_KIND_KERNEL || kd[j] == TA_KIND_MEMCPY)) lo[j] = -1;
      sl[j] = s[j] - sl[j];
    }
  }

  CpLane ln(a, l0);
  const int sh = a.tsbits + a.idxbits;
  u64 links = 0;
  int run_slot = -1;
  u64 run_max = 0;
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++) {
    const int64_t p = p0 + j;
    if (p >= tile_end) break;
    ln.to(p);
    if (cp_device(kd[j])) {
      const i64 eq = j ? e[j - 1] : e_before;
      if (!a.use_sort && p > ln.cur_off && e[j] < eq) *a.not_ascending = 1u;
      const bool q_ok = p > ln.cur_off && eq <= s[j];
      const bool l_ok = lo[j] >= 0 && sl[j] <= s[j];
      const u64 lk = (q_ok && (!l_ok || eq > sl[j])) ? CP_LINK_STREAM : (l_ok ? CP_LINK_SUBMIT : CP_LINK_END);
      links |= lk << (8 * j);
    } else if (cp_host_node(kd[j])) {
      const int slot = a.lane_slot[ln.l];
      if (slot != run_slot) {
        if (run_slot >= 0) atomicMax(&a.slot_host_te[run_slot], run_max);
        run_slot = slot;
        run_max = 0;
      }
      run_max = max(run_max, cp_code(e[j]));
      if (kd[j] == TA_KIND_API) {
        // last element of the sorted (slot, ts_end) keys below (slot, this call's ts_end)
        int32_t d = -1;
        if (!a.use_sort) {
          d = cp_last_ended(a, a.lane_dom_next[ln.l], slot, e[j], false);
          if (d >= 0 && a.te[d] < s[j]) d = -1;
        } else if (a.m > 0) {
          const u64 want = ((u64)slot << a.tsbits) | (u64)(e[j] - a.t0[a.lane_window[ln.l]]);
          int64_t lo_i = 0, hi_i = a.m;
          while (lo_i < hi_i) {
            const int64_t mid = (lo_i + hi_i) >> 1;
            if ((a.skeys[mid] >> a.idxbits) < want) lo_i = mid + 1;
            else hi_i = mid;
          }
          if (lo_i > 0 && (int)(a.skeys[lo_i - 1] >> sh) == slot) {
            d = cp_pos_of(a, lo_i - 1);
            if (a.te[d] < s[j]) d = -1;  // finished before the call began: the call did not wait for it
          }
        }
        a.cross[p] = d;
      }
    }
  }
  if (p0 + CP_ITEMS <= a.n) *reinterpret_cast<u64 *>(a.link + p0) = links;
  else
    for (int j = 0; j < CP_ITEMS && p0 + j < a.n; j++) a.link[p0 + j] = (uint8_t)(links >> (8 * j));
  // the thread's last slot: one atomic per warp when the whole warp is here and sits in that slot
  const u32 act = __activemask();
  const u32 has = __ballot_sync(act, run_slot >= 0);
  if (!has) return;
  const int s0 = __shfl_sync(act, run_slot, __ffs(has) - 1);
  if (act == 0xffffffffu && __all_sync(act, run_slot < 0 || run_slot == s0)) {
    const u64 v = warp_reduce(run_slot >= 0 ? run_max : 0ull, OpMax());
    if ((threadIdx.x & 31) == 0) atomicMax(&a.slot_host_te[s0], v);
  } else if (run_slot >= 0) {
    atomicMax(&a.slot_host_te[run_slot], run_max);
  }
}

// ---- runs: previous host node, then run heads ------------------------------------------
__global__ void __launch_bounds__(CP_THREADS) k_cp_runs(CpArgs a) {
  __shared__ u64 tmp[33];
  __shared__ u64 s_excl;
  __shared__ int s_tile, s_lane0, s_fail;
  const int tid = threadIdx.x;
  if (tid == 0) {
    s_tile = (int)atomicAdd(a.counter, 1u);
    s_fail = ta_failed(a.status) ? 1 : 0;
  }
  __syncthreads();
  if (s_fail) return;
  const int tile = s_tile;
  const int64_t tile_start = (int64_t)tile * CP_TILE;
  const int64_t tile_end = min(tile_start + CP_TILE, a.n_valid);
  const int l0 = cp_tile_lane(a, tile_start, &s_lane0);
  const int64_t p0 = tile_start + (int64_t)tid * CP_ITEMS;
  int16_t kd[CP_ITEMS];
  load8_i16(a.kind, p0, a.n, -1, kd);
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++)
    if (p0 + j >= tile_end) kd[j] = -1;

  // scan A: position + 1 of the last host node before each position.  A tile without host
  // lanes has nothing to add and nobody after it in its lanes to tell: it publishes an empty
  // prefix (values of earlier lanes are ignored anyway) and leaves prev_node untouched.
  const bool no_host = span_outside_domain(a.lane_domain, a.lane_dom_end, l0, tile_end, 0);
  u64 run = 0, total, pre;
  int32_t prev[CP_ITEMS];
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++) prev[j] = -1;
  if (no_host) {
    if (tid == 0) st_relaxed(&a.st_a[tile], td_pack(TD_PREFIX, 0));
  } else {
#pragma unroll
    for (int j = 0; j < CP_ITEMS; j++)
      if (cp_host_node(kd[j])) run = (u64)(p0 + j + 1);
    pre = block_scan_exclusive<OpMax>(run, OpMax(), tmp, &total);
    if (tid < 32) {
      bool failed;
      const u64 ex = tile_lookback<OpMax>(a.st_a, tile, total, OpMax(), a.status, &failed);
      if (tid == 0) { s_excl = ex; s_fail = failed ? 1 : 0; }
    }
    __syncthreads();
    if (s_fail) return;
    pre = max(pre, s_excl);
    CpLane ln(a, l0);
#pragma unroll
    for (int j = 0; j < CP_ITEMS; j++) {
      if (kd[j] < 0) continue;
      if (!cp_host_node(kd[j])) continue;
      const int64_t p = p0 + j;
      ln.to(p);
      if ((int64_t)pre - 1 >= ln.cur_off) prev[j] = (int32_t)(pre - 1);
      pre = (u64)(p + 1);
      // the sink among host nodes: the highest position among those that end last
      const int slot = a.lane_slot[ln.l];
      if (cp_code(a.te[p]) == a.slot_host_te[slot]) atomicMax(&a.slot_host_pos[slot], (int32_t)p);
    }
    store8_i32(a.prev_node, p0, a.n, prev);
    __syncthreads();  // s_excl is written again below
  }

  // scan B: position + 1 of the last run head at or before each position
  i64 s[CP_ITEMS];
  uint8_t lk[CP_ITEMS];
  u64 cand[CP_ITEMS];
  bool any_node = false;
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++) any_node |= kd[j] > 0;
  if (any_node) {
    load8_i64(a.ts, p0, a.n, s);
    if (p0 + CP_ITEMS <= a.n) {
      const u64 w = *reinterpret_cast<const u64 *>(a.link + p0);
#pragma unroll
      for (int j = 0; j < CP_ITEMS; j++) lk[j] = (uint8_t)(w >> (8 * j));
    } else {
#pragma unroll
      for (int j = 0; j < CP_ITEMS; j++) lk[j] = p0 + j < a.n ? a.link[p0 + j] : 0;
    }
  }
  run = 0;
#pragma unroll
  for (int j = 0; j < CP_ITEMS; j++) {
    cand[j] = 0;
    if (kd[j] <= 0) continue;
    if (cp_device(kd[j])) {
      if (lk[j] != CP_LINK_STREAM) cand[j] = (u64)(p0 + j + 1);
    } else if (prev[j] >= 0) {
      const int32_t u = prev[j];
      // a wait that the device released, entered from its END (it ended before this node began)
      if (a.kind[u] == TA_KIND_API && a.cross[u] >= 0 && a.te[u] <= s[j]) {
        cand[j] = (u64)(u + 1);
        const u32 id = atomicAdd(a.n_eff, 1u);  // each such wait is found once, by the node after it
        a.eff_pos[id] = (u32)u;
        a.id_of[u] = (int32_t)id;
      }
    }
    run = max(run, cand[j]);
  }
  pre = block_scan_exclusive<OpMax>(run, OpMax(), tmp, &total);
  if (tid < 32) {
    bool failed;
    const u64 ex = tile_lookback<OpMax>(a.st_b, tile, total, OpMax(), a.status, &failed);
    if (tid == 0) { s_excl = ex; s_fail = failed ? 1 : 0; }
  }
  __syncthreads();
  if (s_fail) return;
  pre = max(pre, s_excl);
  int32_t hd[CP_ITEMS];
  {
    CpLane ln(a, l0);
#pragma unroll
    for (int j = 0; j < CP_ITEMS; j++) {
      hd[j] = -1;
      if (kd[j] < 0) continue;
      pre = max(pre, cand[j]);
      if (kd[j] == 0) continue;
      ln.to(p0 + j);
      if ((int64_t)pre - 1 >= ln.cur_off) hd[j] = (int32_t)(pre - 1);
    }
  }
  store8_i32(a.head, p0, a.n, hd);
}

// ---- the chain of lane changes ---------------------------------------------------------------
// From the END of device record d: records where the walk enters d's run and, if the head of
// that run was bound by its submission, the host run of its launch.  Returns the list index of
// the wait that heads that host run, or -1 when the path ends first.
__device__ __forceinline__ int32_t cp_follow(const CpArgs &a, int32_t d, bool record) {
  const int32_t h = a.head[d];
  if (h < 0) return -1;  // cannot happen: the first record of a device lane always heads a run
  if (record) a.entry[h] = d;
  if (a.link[h] != CP_LINK_SUBMIT) return -1;  // unresolved: the head records where the path begins
  const int32_t l = a.launch_of[h];
  const int32_t e = a.head[l];
  if (e < 0) {
    if (record) a.entry_lane[lane_of_pos(a.lane_off, a.n_lanes, l)] = l;
    return -1;
  }
  if (record) a.entry[e] = l;
  return a.id_of[e];
}

__global__ void __launch_bounds__(256) k_cp_succ(CpArgs a) {
  if (ta_failed(a.status)) return;
  const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= a.n_list) return;
  a.jump_in[id] = cp_follow(a, a.cross[a.eff_pos[id]], false);
}

// one thread per (window, process): the sink and the hops from it to the first listed wait
__global__ void __launch_bounds__(64) k_cp_start(CpArgs a) {
  if (ta_failed(a.status)) return;
  const int64_t slot = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (slot >= a.n_slots) return;
  const int sh = a.tsbits + a.idxbits;
  // last device record of the slot in (ts_end, position) order
  int32_t dsink = -1;
  if (!a.use_sort) {
    int lo = 0, hi = a.n_lanes;  // first lane of the slot (lane_slot ascends with the lane index)
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if ((int64_t)a.lane_slot[mid] < slot) lo = mid + 1;
      else hi = mid;
    }
    while (lo < a.n_lanes && (int64_t)a.lane_slot[lo] == slot && a.lane_domain[lo] != 1) lo++;
    dsink = cp_last_ended(a, lo, (int)slot, LLONG_MAX, true);
  } else if (a.m > 0) {
    int64_t lo = 0, hi = a.m;
    while (lo < hi) {
      const int64_t mid = (lo + hi) >> 1;
      if ((int64_t)(a.skeys[mid] >> sh) <= slot) lo = mid + 1;
      else hi = mid;
    }
    if (lo > 0 && (int64_t)(a.skeys[lo - 1] >> sh) == slot) dsink = cp_pos_of(a, lo - 1);
  }
  const int32_t hsink = a.slot_host_te[slot] ? a.slot_host_pos[slot] : -1;
  int32_t sink;
  if (dsink < 0 && hsink < 0) return;
  if (dsink >= 0 && hsink >= 0) sink = a.te[dsink] >= a.te[hsink] ? dsink : hsink;  // device positions are the higher ones
  else sink = dsink >= 0 ? dsink : hsink;
  u64 *acc = a.acc + (size_t)slot * CP_ACC;
  acc[11] = (u64)(sink + 1);

  int32_t first = -1;  // list index of the first wait on the path
  if (cp_device(a.kind[sink])) {
    first = cp_follow(a, sink, true);
  } else {
    const int32_t d = a.kind[sink] == TA_KIND_API ? a.cross[sink] : -1;
    if (d >= 0) {  // the sink is a wait: its tail is on the path, then the record that released it
      atomicAdd(&acc[8], (u64)(a.te[sink] - a.te[d]));
      a.entry[sink] = sink;
      first = cp_follow(a, d, true);
    } else {       // the sink ran: the walk enters its host run at its START
      atomicAdd(&acc[6], (u64)(a.te[sink] - a.ts[sink]));
      const int32_t e = a.head[sink];
      if (e < 0) a.entry_lane[lane_of_pos(a.lane_off, a.n_lanes, sink)] = sink;
      else {
        a.entry[e] = sink;
        first = a.id_of[e];
      }
    }
  }
  if (first >= 0) a.mark[first] = 1;
}

// one round: what a marked wait reaches is marked (a wait marked during the round may pass its
// mark on at once - everything it reaches is on the path as well), successors are squared
__global__ void __launch_bounds__(256) k_cp_double(CpArgs a) {
  if (ta_failed(a.status)) return;
  const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= a.n_list) return;
  const int32_t j = a.jump_in[id];
  if (j < 0) {
    a.jump_out[id] = -1;
    return;
  }
  if (a.mark[id]) a.mark[j] = 1;
  a.jump_out[id] = a.jump_in[j];
}

__global__ void __launch_bounds__(256) k_cp_enter(CpArgs a) {
  if (ta_failed(a.status)) return;
  const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= a.n_list || !a.mark[id]) return;
  cp_follow(a, a.cross[a.eff_pos[id]], true);
}

// ---- membership and time classes ---------------------------------------------------------
__global__ void __launch_bounds__(CP_THREADS) k_cp_mark(CpArgs a) {
  if (ta_failed(a.status)) return;
  __shared__ int s_lane0;
  const int lane = threadIdx.x & 31;
  const int64_t tile_start = (int64_t)blockIdx.x * CP_TILE;
  if (tile_start >= a.n_valid) return;
  const int l0 = cp_tile_lane(a, tile_start, &s_lane0);
  const int64_t tile_end = min(tile_start + CP_TILE, a.n_valid);
  const int64_t p0 = tile_start + (int64_t)threadIdx.x * CP_ITEMS;
  int16_t kd[CP_ITEMS];
  int32_t hd[CP_ITEMS];
  u64 flags = 0;
  u64 sum[10];
#pragma unroll
  for (int c = 0; c < 10; c++) sum[c] = 0;
  int first = -1;
  if (p0 < tile_end) {
    load8_i16(a.kind, p0, a.n, -1, kd);
    if (p0 + CP_ITEMS <= a.n) {
      const int4 x = *reinterpret_cast<const int4 *>(a.head + p0), y = *reinterpret_cast<const int4 *>(a.head + p0 + 4);
      hd[0] = x.x; hd[1] = x.y; hd[2] = x.z; hd[3] = x.w;
      hd[4] = y.x; hd[5] = y.y; hd[6] = y.z; hd[7] = y.w;
    } else {
#pragma unroll
      for (int j = 0; j < CP_ITEMS; j++) hd[j] = p0 + j < a.n ? a.head[p0 + j] : -1;
    }
    CpLane ln(a, l0);
#pragma unroll
    for (int j = 0; j < CP_ITEMS; j++) {
      const int64_t p = p0 + j;
      if (p >= tile_end || kd[j] <= 0) continue;
      ln.to(p);
      bool on;
      if (cp_device(kd[j])) on = hd[j] >= 0 && a.entry[hd[j]] >= p;
      else on = (hd[j] >= 0 ? a.entry[hd[j]] : a.entry_lane[ln.l]) >= p;
      const bool as_head = !cp_device(kd[j]) && a.entry[p] >= 0;  // a wait the walk left through its END
      if (!on && !as_head) continue;
      flags |= 1ull << (8 * j);
      const int slot = a.lane_slot[ln.l];
      u64 add[10];
#pragma unroll
      for (int c = 0; c < 10; c++) add[c] = 0;
      add[0] = 1;
      u64 *acc = a.acc + (size_t)slot * CP_ACC;
      if (on) {
        const i64 s = a.ts[p];
        if (cp_device(kd[j])) {
          const u64 dur = (u64)(a.te[p] - s);
          add[1] = kd[j] == TA_KIND_KERNEL ? dur : 0;
          add[2] = kd[j] == TA_KIND_MEMCPY ? dur : 0;
          add[3] = kd[j] == TA_KIND_COLL ? dur : 0;
          const int lk = a.link[p];
          if (lk == CP_LINK_STREAM) add[5] = (u64)(s - a.te[p - 1]);
          else if (lk == CP_LINK_SUBMIT) add[4] = (u64)a.latency[p];
          else { acc[9] = (u64)s; acc[10] = 1; }
        } else {
          const int32_t u = a.prev_node[p];
          if (u < 0) { acc[9] = (u64)s; acc[10] = 0; }
          else {
            const i64 ue = a.te[u];
            if (ue <= s) {
              add[7] = (u64)(s - ue);
              if (u == hd[j]) add[8] = (u64)(ue - a.te[a.cross[u]]);  // the wait at the head of this run
              else add[6] = (u64)(ue - a.ts[u]);
            } else {
              add[6] = (u64)(s - a.ts[u]);
            }
          }
        }
      }
      if (first < 0) first = slot;
      if (slot == first) {
#pragma unroll
        for (int c = 0; c < 10; c++) sum[c] += add[c];
      } else {
#pragma unroll
        for (int c = 0; c < 10; c++)
          if (add[c]) atomicAdd(&acc[c], add[c]);
      }
    }
    if (p0 + CP_ITEMS <= a.n) *reinterpret_cast<u64 *>(a.on_path + p0) = flags;
    else
      for (int j = 0; j < CP_ITEMS && p0 + j < a.n; j++) a.on_path[p0 + j] = (uint8_t)(flags >> (8 * j));
  }
  // fold per warp when all its records on a path belong to one process
  const u32 has = __ballot_sync(0xffffffffu, first >= 0);
  if (!has) return;
  const int wfirst = __shfl_sync(0xffffffffu, first, __ffs(has) - 1);
  if (__all_sync(0xffffffffu, first < 0 || first == wfirst)) {
#pragma unroll
    for (int c = 0; c < 10; c++) {
      const u64 t = warp_reduce(sum[c], OpAdd());
      if (lane == 0 && t) atomicAdd(&a.acc[(size_t)wfirst * CP_ACC + c], t);
    }
  } else if (first >= 0) {
#pragma unroll
    for (int c = 0; c < 10; c++)
      if (sum[c]) atomicAdd(&a.acc[(size_t)first * CP_ACC + c], sum[c]);
  }
}

// ---- rows: the slots that have a path, in slot order -----------------------------------------
struct CpRowIn {
  const u64 *acc;
  __device__ u64 operator()(int64_t s) const { return acc[(size_t)s * CP_ACC + 11] ? 1ull : 0ull; }
};
struct CpRowOut {
  const u64 *acc;
  const TripleTable *tt;
  const int64_t *te;
  int n_pids;
  int32_t *p_window, *p_pid, *p_sink, *p_n_nodes, *p_reason;
  int64_t *p_begin, *p_end, *p_ns;
  __device__ void operator()(int64_t s, u64 row, u64 v) const {
    if (!v) return;
    const u64 *r = acc + (size_t)s * CP_ACC;
    const int32_t sink = (int32_t)(r[11] - 1);
    p_window[row] = (int32_t)(s / n_pids);
    p_pid[row] = tt->pid_value[s % n_pids];
    p_sink[row] = sink;
    p_n_nodes[row] = (int32_t)r[0];
    p_reason[row] = (int32_t)r[10];
    p_begin[row] = (i64)r[9];
    p_end[row] = te[sink];
    for (int c = 0; c < 8; c++) p_ns[row * 8 + c] = (i64)r[1 + c];
  }
};

ta_status ta_run_critpath(ta_window *h, ta_critpath_result *out, ta_critpath_summary *out_summary) {
  cudaStream_t st = h->stream;
  memset(out, 0, sizeof(*out));
  const int W = h->W;
  for (int w = 0; w < W; w++) memset(&out_summary[w], 0, sizeof(ta_critpath_summary));
  const int n_pids = h->n_pids > 0 ? h->n_pids : 1;
  const int64_t n_slots = (int64_t)W * n_pids;
  const int64_t n = h->n, nn = n > 0 ? n : 1, m = h->n_device;
  const int n_lanes = h->sorted.n_lanes;

  // key layout: ts_end - t0 is below (longest window + longest record)
  int64_t max_span = 1;
  for (int w = 0; w < W; w++) max_span = h->h_t1[w] - h->h_t0[w] > max_span ? h->h_t1[w] - h->h_t0[w] : max_span;
  const int64_t max_dur = h->max_dur > 0 ? h->max_dur : 0;
  if (max_span >= (1ll << 40) || max_dur >= (1ll << 40)) return TA_ERR_TOO_LARGE;
  const int tsbits = ta_bit_len((uint64_t)(max_span + max_dur));
  int slot_bits = ta_bit_len((uint64_t)(n_slots - 1));
  if (slot_bits < 1) slot_bits = 1;
  if (tsbits + slot_bits > 63 || n_slots >= (1ll << 22)) return TA_ERR_TOO_LARGE;
  int idxbits = ta_bit_len((uint64_t)(m > 0 ? m - 1 : 0));
  if (idxbits < 1) idxbits = 1;
  if (tsbits + slot_bits + idxbits > 64) idxbits = 0;

  // results (kept)
  size_t kb = Carver::pad((size_t)nn) + 5 * Carver::pad((size_t)n_slots * 4) + 2 * Carver::pad((size_t)n_slots * 8) +
              Carver::pad((size_t)n_slots * 64) + 256;
  void *keep = ta_dalloc(h, kb);
  if (!keep) return TA_ERR_OOM;
  Carver ck(keep);
  CpRowOut ro;
  uint8_t *on_path = ck.take<uint8_t>(nn);
  ro.p_window = ck.take<int32_t>(n_slots); ro.p_pid = ck.take<int32_t>(n_slots);
  ro.p_sink = ck.take<int32_t>(n_slots); ro.p_n_nodes = ck.take<int32_t>(n_slots);
  ro.p_reason = ck.take<int32_t>(n_slots);
  ro.p_begin = ck.take<int64_t>(n_slots); ro.p_end = ck.take<int64_t>(n_slots);
  ro.p_ns = ck.take<int64_t>(n_slots * 8);
  TA_CHECK_CUDA(h, cudaMemsetAsync(on_path, 0, (size_t)nn, st));
  out->on_path = on_path;
  if (h->n_valid <= 0) {
    h->d_on_path = on_path;
    return TA_OK;
  }

  const int64_t tiles = (h->n_valid + CP_TILE - 1) / CP_TILE;
  const int64_t mm = m > 0 ? m : 1;
  size_t tb = Carver::pad((size_t)nn) + 6 * Carver::pad((size_t)nn * 4) + Carver::pad((size_t)(n_lanes + 1) * 4) +
              2 * Carver::pad((size_t)tiles * 8) + Carver::pad(64) + Carver::pad((size_t)n_slots * 8) +
              Carver::pad((size_t)n_slots * 4) + Carver::pad((size_t)n_slots * CP_ACC * 8) +
              scan_temp_bytes(n_slots) + 1024;
  void *tmpb = ta_dalloc(h, tb);
  if (!tmpb) return TA_ERR_OOM;
  Carver ct(tmpb);
  CpArgs a;
  memset(&a, 0, sizeof(a));
  a.link = ct.take<uint8_t>(nn);
  a.cross = ct.take<int32_t>(nn);
  a.prev_node = ct.take<int32_t>(nn);
  a.head = ct.take<int32_t>(nn);
  a.eff_pos = ct.take<u32>(nn);
  // zeroed block
  char *zb = ct.base + ct.off;
  a.st_a = ct.take<u64>(tiles); a.st_b = ct.take<u64>(tiles);
  a.counter = (u32 *)ct.take<u64>(8);
  a.n_eff = a.counter + 2;
  a.not_ascending = a.counter + 3;
  a.slot_host_te = ct.take<u64>(n_slots);
  a.acc = ct.take<u64>(n_slots * CP_ACC);
  const size_t zbytes = (ct.base + ct.off) - zb;
  // block filled with -1
  char *fb = ct.base + ct.off;
  a.entry = ct.take<int32_t>(nn);
  a.id_of = ct.take<int32_t>(nn);
  a.entry_lane = ct.take<int32_t>(n_lanes + 1);
  a.slot_host_pos = ct.take<int32_t>(n_slots);
  const size_t fbytes = (ct.base + ct.off) - fb;
  void *scan_mem = ct.base + ct.off;

  a.n = n; a.n_valid = h->n_valid; a.m = m; a.n_lanes = n_lanes; a.n_pids = n_pids; a.n_slots = n_slots;
  a.kind = h->sorted.kind; a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end;
  a.launch_of = h->join.launch_of; a.latency = h->join.launch_latency;
  a.lane_off = h->sorted.lane_off; a.lane_slot = h->d_lane_slot; a.lane_window = h->sorted.lane_window;
  a.lane_dom_end = h->d_lane_dom_end; a.lane_dev_base = h->d_lane_dev_base;
  a.lane_dom_next = h->d_lane_dom_next;
  a.lane_domain = h->sorted.lane_domain; a.t0 = h->d_t0;
  a.tsbits = tsbits; a.idxbits = idxbits;
  a.on_path = on_path; a.status = h->d_status;

  // In-order streams end their records in ascending order; then "the record of the process that
  // ended last before t" is a binary search per device lane and nothing has to be sorted.  The
  // first attempt assumes that and checks it; if some record ends before its predecessor, the
  // second attempt sorts the device records by (process slot, ts_end) and searches there.
  void *sortb = nullptr;
  u32 n_list = 0;
  for (int attempt = 0; attempt < 2; attempt++) {
    a.use_sort = attempt;
    TA_CHECK_CUDA(h, cudaMemsetAsync(zb, 0, zbytes, st));
    TA_CHECK_CUDA(h, cudaMemsetAsync(fb, 0xff, fbytes, st));
    if (a.use_sort && m > 0) {
      sortb = ta_dalloc(h, 3 * Carver::pad((size_t)mm * 8) + 3 * Carver::pad((size_t)mm * 4) + ta_sort_temp_bytes(mm) + 256);
      if (!sortb) return TA_ERR_OOM;
      Carver cs(sortb);
      u64 *k_in = cs.take<u64>(mm), *k_scr = cs.take<u64>(mm), *k_fin = cs.take<u64>(mm);
      u32 *v_in = cs.take<u32>(mm), *v_scr = cs.take<u32>(mm), *v_fin = cs.take<u32>(mm);
      void *sort_tmp = cs.base + cs.off;
      a.keys = k_in; a.pos = v_in;
      k_cp_keys<<<TA_N (unsigned)tiles, CP_THREADS, 0, st>>>(a);
      TA_CHECK_CUDA(h, cudaGetLastError());
      if (idxbits) {
        TA_TRY(ta_radix_sort_keys(h, k_in, k_scr, k_fin, m, ta_make_plan(idxbits, idxbits + tsbits + slot_bits),
                                  nullptr, sort_tmp, false));
        a.spos = v_in;
      } else {
        TA_TRY(ta_radix_sort_pairs(h, k_in, v_in, k_scr, v_scr, k_fin, v_fin, m,
                                   ta_make_plan(0, tsbits + slot_bits), nullptr, sort_tmp));
        a.spos = v_fin;
      }
      a.skeys = k_fin;
    }
    k_cp_classify<<<TA_N (unsigned)tiles, CP_THREADS, 0, st>>>(a);
    k_cp_runs<<<TA_N (unsigned)tiles, CP_THREADS, 0, st>>>(a);
    TA_CHECK_CUDA(h, cudaGetLastError());
    // the waits that head a host run: a list whose length decides the number of doubling rounds
    u32 words2[2] = {0, 0};
    TA_TRY(ta_queue_d2h(h, words2, a.n_eff, 8));
    TA_TRY(ta_sync_fetch(h));
    n_list = words2[0];
    if (!a.use_sort && words2[1]) continue;
    break;
  }
  a.n_list = (int64_t)n_list;
  const int64_t nl = n_list > 0 ? n_list : 1;
  void *lb = ta_dalloc(h, 2 * Carver::pad((size_t)nl * 4) + Carver::pad((size_t)nl) + 256);
  if (!lb) return TA_ERR_OOM;
  Carver cl(lb);
  a.jump_in = cl.take<int32_t>(nl);
  a.jump_out = cl.take<int32_t>(nl);
  a.mark = cl.take<uint8_t>(nl);
  TA_CHECK_CUDA(h, cudaMemsetAsync(a.mark, 0, (size_t)nl, st));
  const unsigned lblocks = (unsigned)((nl + 255) / 256);
  if (n_list) k_cp_succ<<<TA_N lblocks, 256, 0, st>>>(a);
  k_cp_start<<<TA_N (unsigned)((n_slots + 63) / 64), 64, 0, st>>>(a);
  if (n_list) {
    for (int r = ta_bit_len((uint64_t)n_list); r > 0; r--) {
      k_cp_double<<<TA_N lblocks, 256, 0, st>>>(a);
      int32_t *t = a.jump_in; a.jump_in = a.jump_out; a.jump_out = t;
    }
    k_cp_enter<<<TA_N lblocks, 256, 0, st>>>(a);
  }
  k_cp_mark<<<TA_N (unsigned)tiles, CP_THREADS, 0, st>>>(a);
  TA_CHECK_CUDA(h, cudaGetLastError());

  ro.acc = a.acc; ro.tt = h->d_triples; ro.te = a.te; ro.n_pids = n_pids;
  ScanTemp s3;
  TA_TRY(scan_temp_init(h, scan_mem, n_slots, &s3));
  CpRowIn ri{a.acc};
  TA_TRY((launch_scan<OpAdd, CpRowIn, CpRowOut>(h, n_slots, ri, ro, OpAdd(), s3)));
  u64 rows = 0;
  std::vector<u64> hacc((size_t)n_slots * CP_ACC);
  TA_TRY(ta_queue_d2h(h, &rows, s3.total, 8));
  TA_TRY(ta_queue_d2h(h, hacc.data(), a.acc, hacc.size() * 8));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  ta_dfree(h, lb);
  if (sortb) ta_dfree(h, sortb);
  ta_dfree(h, tmpb);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  for (int64_t s = 0; s < n_slots; s++) {
    const u64 *r = &hacc[(size_t)s * CP_ACC];
    if (!r[11]) continue;
    ta_critpath_summary *ws = &out_summary[s / n_pids];
    ws->n_paths++;
    ws->n_nodes += (int64_t)r[0];
    for (int c = 0; c < 8; c++) ws->ns[c] += (int64_t)r[1 + c];
  }
  out->n_rows = (int64_t)rows;
  h->d_on_path = on_path;
  out->p_window = ro.p_window; out->p_pid = ro.p_pid; out->p_sink = ro.p_sink;
  out->p_n_nodes = ro.p_n_nodes; out->p_reason = ro.p_reason;
  out->p_begin = ro.p_begin; out->p_end = ro.p_end; out->p_ns = ro.p_ns;
  return TA_OK;
}
