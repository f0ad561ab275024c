// ta_blame_gaps: why was a device stream idle, and which host calls did the idle
// time overlap.  A gap counts against the host when the work that ended it was
// submitted only after the stream had gone idle (the late-dispatch test of Sec. 6.2);
// idle time is charged to the operators that were running meanwhile (Sec. 9.1).
//
// Input: the long-gap list of ta_stream_gaps (ordered by lane, then time) and the
// launch of every device record (ta_correlate_launches).
//   k_blame_classify  per long gap: TAIL / NO_LAUNCH / SUBMISSION (the launch of the
//                     record that ends the gap started at or after the gap began) /
//                     QUEUED, folded per warp into per-window counts and lengths;
//   a scan            running total of the gap lengths along the list;
//   k_blame_lanes     the list range of every lane (binary search);
//   k_blame_ops       per OP record: for each device stream of its process the total
//                     long-gap length before a time t is (running total at the last
//                     gap that starts before t) + min(t - its start, its length); the
//                     operator is charged C(ts_end) - C(ts_start), summed over streams.
// The gap list is small (it stays in L2), the OP pass reads 18 B per host record.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define BL_THREADS 256
#define BL_ITEMS 8
#define BL_TILE (BL_THREADS * BL_ITEMS)

struct BlameArgs {
  int64_t n, n_valid, m;  // m = long gaps
  int n_lanes, W;
  const ta_long_gap *list;
  const int32_t *launch_of;
  const int64_t *ts, *te;
  const int16_t *kind;
  const int32_t *lane_off, *lane_window, *lane_slot, *lane_dom_end, *lane_dom_next;
  const int16_t *lane_domain;
  int32_t *g_class, *g_launch;
  u64 *win_count, *win_ns;  // [W][4]
  u64 *pre;                 // exclusive running total of gap_len along the list
  int32_t *lane_first;      // [n_lanes + 1] first list entry of every lane
  int64_t *op_gap_ns;
  const int32_t *status;
};

__global__ void __launch_bounds__(256) k_blame_classify(BlameArgs a) {
  if (ta_failed(a.status)) return;
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  int cls = -1, w = -1;
  u64 len = 0;
  if (k < a.m) {
    const ta_long_gap g = a.list[k];
    int32_t l = -1;
    if (g.next_event < 0) cls = TA_BLAME_TAIL;
    else {
      l = a.launch_of[g.next_event];
      cls = l < 0 ? TA_BLAME_NO_LAUNCH : (a.ts[l] >= g.gap_start ? TA_BLAME_SUBMISSION : TA_BLAME_QUEUED);
    }
    a.g_class[k] = cls;
    a.g_launch[k] = l;
    w = a.lane_window[g.lane];
    len = (u64)g.gap_len;
  }
  // per class and warp: one pair of atomics when the warp sits in one window
  const u32 act = __ballot_sync(0xffffffffu, cls >= 0);
  if (!act) return;
  const int w0 = __shfl_sync(0xffffffffu, w, __ffs(act) - 1);
  if (__all_sync(0xffffffffu, cls < 0 || w == w0)) {
#pragma unroll
    for (int c = 0; c < 4; c++) {
      const u32 mine = __ballot_sync(0xffffffffu, cls == c);
      const u64 t = warp_reduce(cls == c ? len : 0ull, OpAdd());
      if (lane == 0 && mine) {
        atomicAdd(&a.win_count[(size_t)w0 * 4 + c], (u64)__popc(mine));
        atomicAdd(&a.win_ns[(size_t)w0 * 4 + c], t);
      }
    }
  } else if (cls >= 0) {
    atomicAdd(&a.win_count[(size_t)w * 4 + cls], 1ull);
    atomicAdd(&a.win_ns[(size_t)w * 4 + cls], len);
  }
}

struct GapLenIn {
  const ta_long_gap *list;
  __device__ u64 operator()(int64_t k) const { return (u64)list[k].gap_len; }
};
struct GapLenOut {
  u64 *pre;
  __device__ void operator()(int64_t k, u64 excl, u64) const { pre[k] = excl; }
};

// lane_first[l] = number of list entries whose lane is < l
__global__ void __launch_bounds__(256) k_blame_lanes(BlameArgs a) {
  if (ta_failed(a.status)) return;
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l > a.n_lanes) return;
  int64_t lo = 0, hi = a.m;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (a.list[mid].lane < l) lo = mid + 1;
    else hi = mid;
  }
  a.lane_first[l] = (int32_t)lo;
}

// number of gaps of list range [first, last) that start before time t
__device__ __forceinline__ int64_t gaps_started_before(const BlameArgs &a, int64_t first, int64_t last,
                                                       i64 t) {
  int64_t lo = first, hi = last;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (a.list[mid].gap_start < t) lo = mid + 1;
    else hi = mid;
  }
  return lo;
}
// total long-gap length of the range that lies before time t, given i = gaps_started_before(t)
__device__ __forceinline__ i64 gap_time_before(const BlameArgs &a, int64_t first, int64_t i, i64 t) {
  if (i == first) return 0;
  const int64_t k = i - 1;
  const i64 part = t - a.list[k].gap_start, len = a.list[k].gap_len;
  return (i64)(a.pre[k] - a.pre[first]) + (part < len ? part : len);
}
// length of [s, e) that lies inside the gaps of the range
__device__ __forceinline__ i64 gap_time_within(const BlameArgs &a, int64_t first, int64_t last, i64 s,
                                               i64 e) {
  const int64_t ie = gaps_started_before(a, first, last, e);
  if (ie == first) return 0;  // every gap starts at or after e
  const ta_long_gap g = a.list[ie - 1];
  if (g.gap_start < s && g.gap_start + g.gap_len <= s) return 0;  // the last gap before e ends before s
  const int64_t is = g.gap_start < s ? ie : gaps_started_before(a, first, ie, s);
  return gap_time_before(a, first, ie, e) - gap_time_before(a, first, is, s);
}

__global__ void __launch_bounds__(BL_THREADS) k_blame_ops(BlameArgs a) {
  __shared__ int s_lane0;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x;
  const int64_t tile_start = (int64_t)blockIdx.x * BL_TILE;
  if (tile_start >= a.n_valid) return;
  if (tid < 32) {
    const int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (tid == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  const int64_t tile_end = min(tile_start + BL_TILE, a.n_valid);
  if (span_outside_domain(a.lane_domain, a.lane_dom_end, l0, tile_end, 0)) return;
  const int64_t p0 = tile_start + (int64_t)tid * BL_ITEMS;
  if (p0 >= tile_end) return;
  int16_t kd[BL_ITEMS];
  load8_i16(a.kind, p0, a.n, 9, kd);
  unsigned ops = 0;
#pragma unroll
  for (int j = 0; j < BL_ITEMS; j++)
    if (p0 + j < tile_end && kd[j] == TA_KIND_OP) ops |= 1u << j;
  if (!ops) return;
  i64 s[BL_ITEMS], e[BL_ITEMS];
  load8_i64(a.ts, p0, a.n, s);
  load8_i64(a.te, p0, a.n, e);
  int l = l0;
  int64_t next_off = a.lane_off[l + 1];
  int dlo = -1, dhi = -1;  // device lanes of the record's (window, process)
  int cur = -1;
#pragma unroll
  for (int j = 0; j < BL_ITEMS; j++) {
    if (!(ops & (1u << j))) continue;
    const int64_t p = p0 + j;
    while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; }
    if (l != cur) {
      cur = l;
      dlo = a.lane_dom_next[l];
      dhi = dlo;
      const int slot = a.lane_slot[l];
      while (dhi < a.n_lanes && a.lane_domain[dhi] == 1 && a.lane_slot[dhi] == slot) dhi++;
    }
    i64 sum = 0;
    for (int d = dlo; d < dhi; d++) {
      const int64_t first = a.lane_first[d], last = a.lane_first[d + 1];
      if (first == last) continue;
      sum += gap_time_within(a, first, last, s[j], e[j]);
    }
    if (sum) a.op_gap_ns[p] = sum;
  }
}

ta_status ta_run_blame(ta_window *h, const ta_gap_result *gaps, ta_blame_result *out,
                       ta_blame_summary *out_summary) {
  cudaStream_t st = h->stream;
  memset(out, 0, sizeof(*out));
  const int W = h->W;
  const int64_t n = h->n, nn = n > 0 ? n : 1, m = gaps->n_long_gaps, mm = m > 0 ? m : 1;
  const int L = h->sorted.n_lanes;
  for (int w = 0; w < W && out_summary; w++) memset(&out_summary[w], 0, sizeof(ta_blame_summary));

  size_t kb = Carver::pad((size_t)nn * 8) + 2 * Carver::pad((size_t)mm * 4) + 256;
  void *keep = ta_dalloc(h, kb);
  if (!keep) return TA_ERR_OOM;
  Carver ck(keep);
  int64_t *op_gap = ck.take<int64_t>(nn);
  int32_t *g_class = ck.take<int32_t>(mm), *g_launch = ck.take<int32_t>(mm);
  TA_CHECK_CUDA(h, cudaMemsetAsync(op_gap, 0, (size_t)nn * 8, st));
  out->n_long_gaps = m;
  out->g_class = g_class; out->g_launch = g_launch; out->op_gap_ns = op_gap;
  h->d_op_gap_ns = op_gap;
  if (m == 0 || h->n_valid == 0) return TA_OK;

  size_t tb = 2 * Carver::pad((size_t)W * 4 * 8) + Carver::pad((size_t)mm * 8) +
              Carver::pad((size_t)(L + 2) * 4) + scan_temp_bytes(m) + 256;
  void *tmpb = ta_dalloc(h, tb);
  if (!tmpb) return TA_ERR_OOM;
  Carver ct(tmpb);
  BlameArgs a;
  memset(&a, 0, sizeof(a));
  a.win_count = ct.take<u64>((size_t)W * 4);
  a.win_ns = ct.take<u64>((size_t)W * 4);
  TA_CHECK_CUDA(h, cudaMemsetAsync(tmpb, 0, ct.off, st));
  a.pre = ct.take<u64>(mm);
  a.lane_first = ct.take<int32_t>(L + 2);
  void *scan_mem = ct.base + ct.off;
  a.n = n; a.n_valid = h->n_valid; a.m = m; a.n_lanes = L; a.W = W;
  a.list = gaps->long_gaps; a.launch_of = h->join.launch_of;
  a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end; a.kind = h->sorted.kind;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window; a.lane_slot = h->d_lane_slot;
  a.lane_dom_end = h->d_lane_dom_end; a.lane_dom_next = h->d_lane_dom_next;
  a.lane_domain = h->sorted.lane_domain;
  a.g_class = g_class; a.g_launch = g_launch; a.op_gap_ns = op_gap; a.status = h->d_status;

  k_blame_classify<<<TA_N (unsigned)((m + 255) / 256), 256, 0, st>>>(a);
  ScanTemp s1;
  TA_TRY(scan_temp_init(h, scan_mem, m, &s1));
  GapLenIn gi{a.list};
  GapLenOut go{a.pre};
  TA_TRY((launch_scan<OpAdd, GapLenIn, GapLenOut>(h, m, gi, go, OpAdd(), s1)));
  k_blame_lanes<<<TA_N (unsigned)((L + 1 + 255) / 256), 256, 0, st>>>(a);
  const int64_t tiles = (h->n_valid + BL_TILE - 1) / BL_TILE;
  k_blame_ops<<<TA_N (unsigned)tiles, BL_THREADS, 0, st>>>(a);
  TA_CHECK_CUDA(h, cudaGetLastError());

  std::vector<u64> hc((size_t)W * 4), hn((size_t)W * 4);
  TA_TRY(ta_queue_d2h(h, hc.data(), a.win_count, (size_t)W * 32));
  TA_TRY(ta_queue_d2h(h, hn.data(), a.win_ns, (size_t)W * 32));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  ta_dfree(h, tmpb);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  for (int w = 0; w < W && out_summary; w++)
    for (int c = 0; c < 4; c++) {
      out_summary[w].count[c] = (int64_t)hc[(size_t)w * 4 + c];
      out_summary[w].ns[c] = (int64_t)hn[(size_t)w * 4 + c];
    }
  return TA_OK;
}
