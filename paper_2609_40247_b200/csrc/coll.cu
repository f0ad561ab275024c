// ta_match_collectives: records of different processes that name the same collective
// are linked, and every rank's wait for the last arrival is measured (cross-process
// links: Sec. 6.1 "Execution progress and state"; ranks held up by a late one: Sec. 9.2).  Group key (window, comm_id, seq).
//
//   1. compact the COLL records (a few percent of the window), in sorted-
//      position order, which is pid-major;
//   2. stable pair sort by (window | communicator rank | seq - min seq): the
//      members of a group become adjacent and stay ordered by pid;
//   3. group heads by comparing neighbours, group ids by a scan;
//   4. one thread per group: arrival range, skew, straggler, flags;
//   5. one thread per member in pid-major order: wait, and per-(window, pid)
//      totals folded per CTA before they touch global memory.
#include <algorithm>
#include <climits>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"


struct CollCtx {
  int64_t m;
  const u32 *posc;      // compacted index -> sorted position
  const int64_t *corr, *ts, *te;
  const int32_t *seq, *pid;
  const int32_t *lane_off, *lane_slot, *lane_window;
  int n_lanes, n_pids;
  const CommTable *cm;
  int64_t min_seq;
  int qbits, cbits;
};

__global__ void __launch_bounds__(256) k_coll_keys(CollCtx c, u64 *keys, int32_t *slot_of, int32_t *status) {
  __shared__ int s_lane0;
  if (ta_failed(status)) return;
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // the compacted positions ascend: the lane of the CTA's first record is searched once, the
  // others walk on from it (a few lanes at most as a rule; a full search after eight steps)
  if (threadIdx.x == 0) s_lane0 = lane_of_pos(c.lane_off, c.n_lanes, c.posc[min(j, c.m - 1)]);
  __syncthreads();
  if (j >= c.m) return;
  u32 p = c.posc[j];
  int lane = s_lane0;
  for (int step = 0; lane + 1 < c.n_lanes && (int64_t)c.lane_off[lane + 1] <= (int64_t)p; step++) {
    if (step == 8) { lane = lane_of_pos(c.lane_off, c.n_lanes, p); break; }
    lane++;
  }
  u64 cc = (u64)c.corr[p] ^ (1ull << 63);
  // every communicator id was inserted while the records were loaded: a bounded probe all the same
  u32 s = hash_code(cc) & (TA_COMM_SLOTS - 1);
  int probes = 0;
  while (c.cm->slots[s] != cc && ++probes < TA_COMM_SLOTS) s = (s + 1) & (TA_COMM_SLOTS - 1);
  u64 rank = 0;
  if (probes < TA_COMM_SLOTS) rank = (u64)c.cm->rank_of_slot[s];
  else ta_set_err(status, TA_ERR_OVERFLOW);
  u64 w = (u64)c.lane_window[lane];
  keys[j] = (w << (c.cbits + c.qbits)) | (rank << c.qbits) | (u64)((int64_t)c.seq[p] - c.min_seq);
  slot_of[j] = c.lane_slot[lane];
}

struct CollHeadIn {
  const u64 *ks;
  __device__ u64 operator()(int64_t j) const { return (j == 0 || ks[j] != ks[j - 1]) ? 1ull : 0ull; }
};
struct CollHeadOut {
  const u32 *cs;     // sorted rank -> compacted index
  int32_t *gid_of_c; // per compacted index
  int32_t *gstart;   // per group
  __device__ void operator()(int64_t j, u64 excl, u64 v) const {
    int32_t g = (int32_t)(excl + v) - 1;
    gid_of_c[cs[j]] = g;
    if (v) gstart[g] = (int32_t)j;
  }
};

struct CollGroupArgs {
  CollCtx c;
  int64_t n_groups;          // rows allocated; the number of groups unless n_groups_dev is set
  const u64 *n_groups_dev;   // device: the number of groups (the total of the head scan), or null
  const u64 *ks;
  const u32 *cs;
  const int32_t *gstart;
  const int32_t *slot_of;        // per compacted index
  const int32_t *expected;       // per communicator rank, -1 = not given
  int32_t *g_window, *g_seq, *g_n, *g_strag, *g_flags;
  int64_t *g_comm, *g_min, *g_max, *g_skew, *g_end;
  u64 *r_nstrag;                 // per (window, pid) slot
  const int32_t *status;
};

__global__ void __launch_bounds__(256) k_coll_groups(CollGroupArgs a) {
  if (ta_failed(a.status)) return;
  int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n_groups = a.n_groups_dev ? (int64_t)*a.n_groups_dev : a.n_groups;
  if (g >= n_groups) return;
  const int64_t b = a.gstart[g], e = g + 1 < n_groups ? (int64_t)a.gstart[g + 1] : a.c.m;
  i64 mn = INT64_MAX, mx = INT64_MIN, me = INT64_MIN;
  int32_t strag = 0, strag_slot = 0, prev_pid = 0;
  int flags = 0;
  // members four at a time: each is reached through two index levels (sorted rank -> compacted
  // index -> sorted position), and one member after the other would make the group a chain of
  // forty-odd dependent loads; the order of the updates stays the members' order
  for (int64_t j0 = b; j0 < e; j0 += 4) {
    u32 ci[4], p[4];
    i64 s[4], en[4];
    int32_t pd[4], sl[4];
#pragma unroll
    for (int k = 0; k < 4; k++) ci[k] = j0 + k < e ? a.cs[j0 + k] : 0u;
#pragma unroll
    for (int k = 0; k < 4; k++) p[k] = j0 + k < e ? a.c.posc[ci[k]] : 0u;
#pragma unroll
    for (int k = 0; k < 4; k++) {
      s[k] = en[k] = 0;
      pd[k] = sl[k] = 0;
      if (j0 + k < e) { s[k] = a.c.ts[p[k]]; en[k] = a.c.te[p[k]]; pd[k] = a.c.pid[p[k]]; sl[k] = a.slot_of[ci[k]]; }
    }
#pragma unroll
    for (int k = 0; k < 4; k++) {
      if (j0 + k >= e) break;
      mn = min(mn, s[k]);
      me = max(me, en[k]);
      if (s[k] > mx || (s[k] == mx && pd[k] < strag)) { mx = s[k]; strag = pd[k]; strag_slot = sl[k]; }
      if (j0 + k > b && pd[k] == prev_pid) flags |= TA_COLL_DUP_PID;
      prev_pid = pd[k];
    }
  }
  const u64 key = a.ks[b];
  const int rank = (int)((key >> a.c.qbits) & ((1ull << a.c.cbits) - 1));
  const int32_t ex = a.expected[rank];
  const int64_t nm = e - b;
  if (ex >= 0) { if (nm != ex) flags |= TA_COLL_INCOMPLETE; }
  else if (nm < 2) flags |= TA_COLL_INCOMPLETE;
  a.g_window[g] = (int32_t)(key >> (a.c.cbits + a.c.qbits));
  a.g_comm[g] = (int64_t)(a.c.cm->sorted_id[rank] ^ (1ull << 63));
  a.g_seq[g] = (int32_t)((int64_t)(key & ((1ull << a.c.qbits) - 1)) + a.c.min_seq);
  a.g_n[g] = (int32_t)nm;
  a.g_min[g] = mn;
  a.g_max[g] = mx;
  a.g_skew[g] = mx - mn;
  a.g_end[g] = me;
  a.g_strag[g] = strag;
  a.g_flags[g] = flags;
  if (flags == 0) atomicAdd(&a.r_nstrag[strag_slot], 1ull);
}

struct CollMemberArgs {
  CollCtx c;
  const int32_t *gid_of_c, *slot_of;
  const int64_t *g_max;
  const int32_t *g_flags;
  int64_t *wait_ns;
  u64 *r_seen, *r_ncoll, *r_sum, *r_maxw;  // per (window, pid) slot
  const int32_t *status;
};

// members in compacted (= pid-major) order: a CTA almost always sees one slot
__global__ void __launch_bounds__(256) k_coll_members(CollMemberArgs a) {
  __shared__ int s_same;
  __shared__ u64 red[4][8];
  if (ta_failed(a.status)) return;
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const bool in = j < a.c.m;
  int slot = -1;
  u64 ok = 0, wait = 0;
  if (in) {
    u32 p = a.c.posc[j];
    int g = a.gid_of_c[j];
    i64 w = a.g_max[g] - a.c.ts[p];
    a.wait_ns[p] = w;
    slot = a.slot_of[j];
    if (a.g_flags[g] == 0) { ok = 1; wait = (u64)w; }
  }
  if (threadIdx.x == 0) s_same = 1;
  __syncthreads();
  const int block_first = a.slot_of[min((int64_t)blockIdx.x * blockDim.x, a.c.m - 1)];
  if (in && slot != block_first) s_same = 0;
  __syncthreads();
  if (s_same) {
    u64 seen = in ? 1 : 0;
    u64 v0 = warp_reduce(seen, OpAdd()), v1 = warp_reduce(ok, OpAdd()), v2 = warp_reduce(wait, OpAdd()),
        v3 = warp_reduce(wait, OpMax());
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red[0][warp] = v0; red[1][warp] = v1; red[2][warp] = v2; red[3][warp] = v3; }
    __syncthreads();
    if (threadIdx.x == 0) {
      u64 t0 = 0, t1 = 0, t2 = 0, t3 = 0;
      for (int w = 0; w < 8; w++) { t0 += red[0][w]; t1 += red[1][w]; t2 += red[2][w]; t3 = max(t3, red[3][w]); }
      atomicAdd(&a.r_seen[block_first], t0);
      if (t1) {
        atomicAdd(&a.r_ncoll[block_first], t1);
        atomicAdd(&a.r_sum[block_first], t2);
        atomicMax(&a.r_maxw[block_first], t3);
      }
    }
  } else if (in) {
    atomicAdd(&a.r_seen[slot], 1ull);
    if (ok) {
      atomicAdd(&a.r_ncoll[slot], 1ull);
      atomicAdd(&a.r_sum[slot], wait);
      atomicMax(&a.r_maxw[slot], wait);
    }
  }
}

struct RankRowIn {
  const u64 *seen;
  __device__ u64 operator()(int64_t s) const { return seen[s] ? 1ull : 0ull; }
};
struct RankRowOut {
  const u64 *ncoll, *sum, *maxw, *nstrag;
  const TripleTable *tt;
  int n_pids;
  int32_t *r_window, *r_pid;
  int64_t *r_n_coll, *r_sum_wait, *r_max_wait, *r_n_straggler;
  __device__ void operator()(int64_t s, u64 row, u64 v) const {
    if (!v) return;
    r_window[row] = (int32_t)(s / n_pids);
    r_pid[row] = tt->pid_value[s % n_pids];
    r_n_coll[row] = (int64_t)ncoll[s];
    r_sum_wait[row] = (int64_t)sum[s];
    r_max_wait[row] = (int64_t)maxw[s];
    r_n_straggler[row] = (int64_t)nstrag[s];
  }
};

ta_status ta_run_collectives(ta_window *h, const ta_comm_size *sizes, int32_t n_comms_given,
                             ta_coll_result *out) {
  const int64_t n = h->n, nn = n > 0 ? n : 1;
  cudaStream_t st = h->stream;
  const int n_pids = h->n_pids > 0 ? h->n_pids : 1;
  const int64_t n_slots = (int64_t)h->W * n_pids;
  memset(out, 0, sizeof(*out));

  // kept: wait_ns; everything else is sized once the counts are known
  int64_t *wait_ns = (int64_t *)ta_dalloc(h, (size_t)nn * 8);
  if (!wait_ns) return TA_ERR_OOM;
  out->wait_ns = wait_ns;
  const int64_t m = h->n_coll;  // kept COLL records, counted while the records were loaded
  if (h->n_valid == 0 || h->n_comms == 0 || m == 0) {
    TA_CHECK_CUDA(h, cudaMemsetAsync(wait_ns, 0, (size_t)nn * 8, st));
    return TA_OK;
  }

  // 1. compaction
  size_t t1b = Carver::pad((size_t)m * 4) + scan_temp_bytes(n) + 256;
  void *t1 = ta_dalloc(h, t1b);
  if (!t1) return TA_ERR_OOM;
  Carver c1(t1);
  u32 *pos_all = c1.take<u32>(m);
  ScanTemp s1;
  TA_TRY(scan_temp_init(h, c1.base + c1.off, n, &s1));
  // the compaction pass clears the wait column on its way (one 0.5 GB memset less on c3)
  TA_TRY(launch_compact_kind(h, h->sorted.kind, h->n_valid, 1u << TA_KIND_COLL, pos_all, s1, reinterpret_cast<i64 *>(wait_ns), nn));
  const std::vector<u64> &comm_sorted = h->h_comm_sorted;

  // expected communicator sizes by rank
  std::vector<int32_t> expected(h->n_comms, -1);
  for (int i = 0; i < n_comms_given; i++) {
    u64 b = (u64)sizes[i].comm_id ^ (1ull << 63);
    auto it = std::lower_bound(comm_sorted.begin(), comm_sorted.end(), b);
    if (it != comm_sorted.end() && *it == b) expected[it - comm_sorted.begin()] = sizes[i].n_ranks;
  }

  CollCtx cx;
  cx.m = m; cx.posc = pos_all;
  cx.corr = h->sorted.corr_id; cx.ts = h->sorted.ts_start; cx.te = h->sorted.ts_end;
  cx.seq = h->sorted.seq; cx.pid = h->sorted.pid;
  cx.lane_off = h->sorted.lane_off; cx.lane_slot = h->d_lane_slot; cx.lane_window = h->sorted.lane_window;
  cx.n_lanes = h->sorted.n_lanes; cx.n_pids = n_pids; cx.cm = h->d_comms; cx.min_seq = h->min_seq;
  cx.qbits = ta_bit_len((uint64_t)(h->max_seq - h->min_seq));
  cx.cbits = ta_bit_len((uint64_t)(h->n_comms - 1));
  const int wbits = ta_bit_len((uint64_t)(h->W - 1));
  if (cx.qbits < 1) cx.qbits = 1;
  if (cx.qbits + cx.cbits + wbits > 62) return TA_ERR_TOO_LARGE;

  // 2. keys + sort; 3. heads
  size_t t2b = 3 * Carver::pad((size_t)m * 8) + 4 * Carver::pad((size_t)m * 4) + Carver::pad((size_t)(m + 1) * 4) +
               Carver::pad((size_t)h->n_comms * 4) + 5 * Carver::pad((size_t)n_slots * 8) +
               ta_sort_temp_bytes(m) + scan_temp_bytes(m) + scan_temp_bytes(n_slots) + 512;
  void *t2 = ta_dalloc(h, t2b);
  if (!t2) return TA_ERR_OOM;
  Carver c2(t2);
  u64 *k_in = c2.take<u64>(m), *k_s = c2.take<u64>(m), *ks = c2.take<u64>(m);
  u32 *v_s = c2.take<u32>(m), *cs = c2.take<u32>(m);
  int32_t *slot_of = c2.take<int32_t>(m), *gid_of_c = c2.take<int32_t>(m);
  int32_t *gstart = c2.take<int32_t>(m + 1);
  int32_t *d_expected = c2.take<int32_t>(h->n_comms);
  char *zb = c2.base + c2.off;
  u64 *r_seen = c2.take<u64>(n_slots), *r_ncoll = c2.take<u64>(n_slots), *r_sum = c2.take<u64>(n_slots);
  u64 *r_maxw = c2.take<u64>(n_slots), *r_nstrag = c2.take<u64>(n_slots);
  TA_CHECK_CUDA(h, cudaMemsetAsync(zb, 0, (c2.base + c2.off) - zb, st));
  void *sort_tmp = c2.base + c2.off; c2.off += ta_sort_temp_bytes(m);
  void *scan2 = c2.base + c2.off; c2.off += scan_temp_bytes(m);
  void *scan3 = c2.base + c2.off;
  TA_CHECK_CUDA(h, cudaMemcpyAsync(d_expected, expected.data(), h->n_comms * 4, cudaMemcpyHostToDevice, st));

  const int gb = (int)((m + 255) / 256);
  k_coll_keys<<<TA_N gb, 256, 0, st>>>(cx, k_in, slot_of, h->d_status);
  TA_TRY(ta_radix_sort_pairs(h, k_in, nullptr, k_s, v_s, ks, cs, m,
                             ta_make_plan(0, cx.qbits + cx.cbits + wbits), nullptr, sort_tmp));
  ScanTemp s2;
  TA_TRY(scan_temp_init(h, scan2, m, &s2));
  CollHeadIn hin{ks};
  CollHeadOut hout{cs, gid_of_c, gstart};
  TA_TRY((launch_scan<OpAdd, CollHeadIn, CollHeadOut>(h, m, hin, hout, OpAdd(), s2)));
  // The group tables are sized by the number of groups when that is worth a round trip; while
  // the bound "one group per COLL record" keeps them under 1 GiB they are sized by the bound
  // and the count comes back with the call's one synchronisation.
  u64 ng64 = 0;
  const bool bounded = (u64)m * 60 <= (1ull << 30);
  if (!bounded) {
    TA_TRY(ta_queue_d2h(h, &ng64, s2.total, 8));
    TA_TRY(ta_sync_fetch(h));
  }
  const int64_t ng = bounded ? m : (int64_t)ng64;  // rows allocated (an upper bound when bounded)

  // 4. groups
  size_t ob = 5 * Carver::pad((size_t)ng * 4) + 5 * Carver::pad((size_t)ng * 8) + 256;
  void *outb = ta_dalloc(h, ob);
  if (!outb) return TA_ERR_OOM;
  Carver co(outb);
  CollGroupArgs ga;
  ga.c = cx; ga.n_groups = ng; ga.n_groups_dev = bounded ? s2.total : nullptr; ga.ks = ks; ga.cs = cs; ga.gstart = gstart; ga.slot_of = slot_of;
  ga.expected = d_expected;
  ga.g_window = co.take<int32_t>(ng); ga.g_seq = co.take<int32_t>(ng); ga.g_n = co.take<int32_t>(ng);
  ga.g_strag = co.take<int32_t>(ng); ga.g_flags = co.take<int32_t>(ng);
  ga.g_comm = co.take<int64_t>(ng); ga.g_min = co.take<int64_t>(ng); ga.g_max = co.take<int64_t>(ng);
  ga.g_skew = co.take<int64_t>(ng); ga.g_end = co.take<int64_t>(ng);
  ga.r_nstrag = r_nstrag; ga.status = h->d_status;
  k_coll_groups<<<TA_N (unsigned)((ng + 255) / 256), 256, 0, st>>>(ga);

  // 5. members
  CollMemberArgs ma;
  ma.c = cx; ma.gid_of_c = gid_of_c; ma.slot_of = slot_of; ma.g_max = ga.g_max; ma.g_flags = ga.g_flags;
  ma.status = h->d_status;
  ma.wait_ns = wait_ns; ma.r_seen = r_seen; ma.r_ncoll = r_ncoll; ma.r_sum = r_sum; ma.r_maxw = r_maxw;
  k_coll_members<<<TA_N gb, 256, 0, st>>>(ma);
  TA_CHECK_CUDA(h, cudaGetLastError());

  // rank table: compact the (window, pid) slots that saw a COLL record
  size_t rb = 2 * Carver::pad((size_t)n_slots * 4) + 4 * Carver::pad((size_t)n_slots * 8) + 256;
  void *rankb = ta_dalloc(h, rb);
  if (!rankb) return TA_ERR_OOM;
  Carver cr(rankb);
  RankRowOut ro;
  ro.ncoll = r_ncoll; ro.sum = r_sum; ro.maxw = r_maxw; ro.nstrag = r_nstrag;
  ro.tt = h->d_triples; ro.n_pids = n_pids;
  ro.r_window = cr.take<int32_t>(n_slots); ro.r_pid = cr.take<int32_t>(n_slots);
  ro.r_n_coll = cr.take<int64_t>(n_slots); ro.r_sum_wait = cr.take<int64_t>(n_slots);
  ro.r_max_wait = cr.take<int64_t>(n_slots); ro.r_n_straggler = cr.take<int64_t>(n_slots);
  ScanTemp s3;
  TA_TRY(scan_temp_init(h, scan3, n_slots, &s3));
  RankRowIn ri{r_seen};
  TA_TRY((launch_scan<OpAdd, RankRowIn, RankRowOut>(h, n_slots, ri, ro, OpAdd(), s3)));
  u64 nr64 = 0;
  TA_TRY(ta_queue_d2h(h, &nr64, s3.total, 8));
  if (bounded) TA_TRY(ta_queue_d2h(h, &ng64, s2.total, 8));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  ta_dfree(h, t1);
  ta_dfree(h, t2);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];

  out->n_groups = (int64_t)ng64;
  out->n_ranks = (int64_t)nr64;
  out->g_window = ga.g_window; out->g_comm = ga.g_comm; out->g_seq = ga.g_seq; out->g_n_members = ga.g_n;
  out->g_min_start = ga.g_min; out->g_max_start = ga.g_max; out->g_skew = ga.g_skew;
  out->g_max_end = ga.g_end; out->g_straggler_pid = ga.g_strag; out->g_flags = ga.g_flags;
  out->r_window = ro.r_window; out->r_pid = ro.r_pid; out->r_n_coll = ro.r_n_coll;
  out->r_sum_wait = ro.r_sum_wait; out->r_max_wait = ro.r_max_wait; out->r_n_straggler = ro.r_n_straggler;
  return TA_OK;
}
