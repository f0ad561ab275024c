// ta_stream_gaps: per device lane, the running maximum of the clipped end times
// (an exclusive max-scan in canonical order) gives the gap before every record,
// the busy union, idle time, a log2 gap histogram and the list of long gaps.
// Device activity records reveal idle intervals (Sec. 9.1).
//
// One pass over the sorted ts_start / ts_end / kind columns.  The scan is made
// lane-aware without segment flags: the scanned value is (lane + 1) << 40 |
// (clipped end - window start), which grows from lane to lane, so a prefix
// that belongs to an earlier lane is recognised by its upper bits.  Two chained
// tile scans run in the same kernel: the maximum, then the number of long-gap
// list entries (so the list is written in order, without a sort).
// HBM-bound: 18 B read + 8 B written per device record.
#include <climits>

#include "ta_internal.cuh"

#define GP_THREADS 512
#define GP_ITEMS 4
#define GP_TILE (GP_THREADS * GP_ITEMS)
#define GP_LOW ((1ull << 40) - 1)

struct GapArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int64_t *ts, *te;
  const int16_t *kind;
  const int32_t *lane_off, *lane_window;
  const int16_t *lane_domain;
  const int64_t *t0, *t1;
  i64 min_gap;
  int list_only;  // second run: only (re)write the long-gap list
  int64_t *gap_before;
  ta_lane_gaps *lane_gaps;
  u32 *lane_hist, *win_hist;
  ta_long_gap *long_gaps;
  i64 list_cap;
  u64 *st_max, *st_cnt;
  u32 *counter;
  int32_t *status;
  u64 *n_long_out;
};

__device__ __forceinline__ u64 block_reduce(u64 v, bool is_max, u64 *smem) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = is_max ? warp_reduce(v, OpMax()) : warp_reduce(v, OpAdd());
  __syncthreads();
  if (lane == 0) smem[warp] = v;
  __syncthreads();
  if (warp == 0) {
    u64 w = lane < (int)(blockDim.x >> 5) ? smem[lane] : 0;
    w = is_max ? warp_reduce(w, OpMax()) : warp_reduce(w, OpAdd());
    if (lane == 0) smem[32] = w;
  }
  __syncthreads();
  return smem[32];
}

__global__ void __launch_bounds__(GP_THREADS) k_gaps(GapArgs a) {
  __shared__ u64 tmp[33];
  __shared__ u64 s_excl_max, s_excl_cnt;
  __shared__ u32 s_hist[TA_NBINS];
  __shared__ int s_tile;
  const int tid = threadIdx.x;
  if (tid == 0) s_tile = (int)atomicAdd(a.counter, 1u);
  __syncthreads();
  const int tile = s_tile;
  const int64_t p0 = (int64_t)tile * GP_TILE + (int64_t)tid * GP_ITEMS;

  // lane of the first item, then walk
  int lane_id = -1;
  if (p0 < a.n_valid && a.n_lanes > 0) lane_id = lane_of_pos(a.lane_off, a.n_lanes, p0);
  i64 s[GP_ITEMS], ce[GP_ITEMS], W0[GP_ITEMS], W1[GP_ITEMS];
  int ln[GP_ITEMS];
  bool dev[GP_ITEMS];
  u64 v[GP_ITEMS];
  u64 run = 0;
#pragma unroll
  for (int j = 0; j < GP_ITEMS; j++) {
    int64_t p = p0 + j;
    dev[j] = false;
    ln[j] = -1;
    v[j] = 0;
    s[j] = ce[j] = W0[j] = W1[j] = 0;
    if (p < a.n_valid) {
      while (lane_id + 1 < a.n_lanes && (int64_t)a.lane_off[lane_id + 1] <= p) lane_id++;
      if (a.kind[p] >= 3) {
        dev[j] = true;
        ln[j] = lane_id;
        int w = a.lane_window[lane_id];
        W0[j] = a.t0[w];
        W1[j] = a.t1[w];
        s[j] = a.ts[p];
        i64 e = a.te[p];
        ce[j] = e < W1[j] ? e : W1[j];
        v[j] = ((u64)(lane_id + 1) << 40) | (u64)(ce[j] - W0[j]);
      }
    }
    run = run > v[j] ? run : v[j];
  }
  u64 tile_max;
  u64 thread_excl = block_scan_exclusive<OpMax>(run, OpMax(), tmp, &tile_max);
  if (tid < 32) {
    u64 e = tile_lookback<OpMax>(a.st_max, tile, tile_max, OpMax(), a.status);
    if (tid == 0) s_excl_max = e;
  }
  __syncthreads();
  u64 pre = s_excl_max > thread_excl ? s_excl_max : thread_excl;

  // gaps, busy, list flags
  i64 gap[GP_ITEMS], P[GP_ITEMS], tail[GP_ITEMS];
  i64 busy[GP_ITEMS];
  bool last[GP_ITEMS];
  int cnt = 0;
#pragma unroll
  for (int j = 0; j < GP_ITEMS; j++) {
    int64_t p = p0 + j;
    gap[j] = 0; busy[j] = 0; tail[j] = 0; last[j] = false; P[j] = 0;
    if (dev[j]) {
      i64 Pi = ((pre >> 40) == (u64)(ln[j] + 1)) ? W0[j] + (i64)(pre & GP_LOW) : W0[j];
      P[j] = Pi;
      gap[j] = s[j] > Pi ? s[j] - Pi : 0;
      i64 from = s[j] > Pi ? s[j] : Pi;
      busy[j] = ce[j] > from ? ce[j] - from : 0;
      last[j] = (p + 1 == (int64_t)a.lane_off[ln[j] + 1]);
      if (last[j]) {
        i64 Pm = Pi > ce[j] ? Pi : ce[j];
        tail[j] = W1[j] - Pm;
      }
      if (gap[j] > 0 && gap[j] >= a.min_gap) cnt++;
      if (last[j] && tail[j] > 0 && tail[j] >= a.min_gap) cnt++;
      pre = pre > v[j] ? pre : v[j];
    }
    if (p < a.n && !a.list_only) a.gap_before[p] = gap[j];
  }
  // ordered long-gap list
  u64 tile_cnt;
  u64 cnt_excl = block_scan_exclusive<OpAdd>((u64)cnt, OpAdd(), tmp, &tile_cnt);
  if (tid < 32) {
    u64 e = tile_lookback<OpAdd>(a.st_cnt, tile, tile_cnt, OpAdd(), a.status);
    if (tid == 0) {
      s_excl_cnt = e;
      if ((int64_t)(tile + 1) * GP_TILE >= a.n) *a.n_long_out = e + tile_cnt;  // last tile
    }
  }
  __syncthreads();
  if (cnt) {
    i64 o = (i64)(s_excl_cnt + cnt_excl);
#pragma unroll
    for (int j = 0; j < GP_ITEMS; j++) {
      if (!dev[j]) continue;
      if (gap[j] > 0 && gap[j] >= a.min_gap) {
        if (o < a.list_cap) a.long_gaps[o] = ta_long_gap{ln[j], (int32_t)(p0 + j), P[j], gap[j]};
        o++;
      }
      if (last[j] && tail[j] > 0 && tail[j] >= a.min_gap) {
        if (o < a.list_cap) a.long_gaps[o] = ta_long_gap{ln[j], -1, W1[j] - tail[j], tail[j]};
        o++;
      }
    }
  }
  if (a.list_only) return;

  // per-lane statistics: one masked block reduction per lane that meets the tile
  __shared__ int s_l0, s_l1;
  if (tid == 0) { s_l0 = INT_MAX; s_l1 = -1; }
  __syncthreads();
  int my_lo = INT_MAX, my_hi = -1;
#pragma unroll
  for (int j = 0; j < GP_ITEMS; j++)
    if (dev[j]) { my_lo = min(my_lo, ln[j]); my_hi = max(my_hi, ln[j]); }
  if (my_hi >= 0) { atomicMin(&s_l0, my_lo); atomicMax(&s_l1, my_hi); }
  __syncthreads();
  const int l0 = s_l0, l1 = s_l1;
  for (int l = l0; l <= l1; l++) {
    if (a.lane_domain[l] != 1) continue;  // uniform over the CTA
    if (tid < TA_NBINS) s_hist[tid] = 0;
    __syncthreads();
    u64 sb = 0, si = 0, ng = 0, mg = 0;
#pragma unroll
    for (int j = 0; j < GP_ITEMS; j++) {
      if (!dev[j] || ln[j] != l) continue;
      sb += (u64)busy[j];
      si += (u64)gap[j];
      if (gap[j] > 0) { ng++; mg = max(mg, (u64)gap[j]); atomicAdd(&s_hist[log2_bin(gap[j])], 1u); }
      if (last[j]) {
        si += (u64)tail[j];
        if (tail[j] > 0) { ng++; mg = max(mg, (u64)tail[j]); atomicAdd(&s_hist[log2_bin(tail[j])], 1u); }
        a.lane_gaps[l].last_end = W1[j] - tail[j];
        a.lane_gaps[l].n_events = (i64)a.lane_off[l + 1] - (i64)a.lane_off[l];
      }
      if (p0 + j == (int64_t)a.lane_off[l]) a.lane_gaps[l].first_start = s[j];
    }
    sb = block_reduce(sb, false, tmp);
    si = block_reduce(si, false, tmp);
    ng = block_reduce(ng, false, tmp);
    mg = block_reduce(mg, true, tmp);
    if (tid == 0) {
      if (sb) atomicAdd((u64 *)&a.lane_gaps[l].busy, sb);
      if (si) atomicAdd((u64 *)&a.lane_gaps[l].idle, si);
      if (ng) atomicAdd((u64 *)&a.lane_gaps[l].n_gaps, ng);
      if (mg) atomicMax((i64 *)&a.lane_gaps[l].max_gap, (i64)mg);
    }
    if (tid < TA_NBINS && s_hist[tid]) {
      atomicAdd(&a.lane_hist[(size_t)l * TA_NBINS + tid], s_hist[tid]);
      atomicAdd(&a.win_hist[(size_t)a.lane_window[l] * TA_NBINS + tid], s_hist[tid]);
    }
    __syncthreads();
  }
}

ta_status ta_run_gaps(ta_window *h, int64_t min_gap, ta_gap_result *out) {
  const int64_t n = h->n;
  const int L = h->sorted.n_lanes;
  const int W = h->W;
  cudaStream_t st = h->stream;
  if (L >= (1 << 22) - 1) return TA_ERR_TOO_LARGE;
  const int64_t tiles = (n + GP_TILE - 1) / GP_TILE;
  int64_t cap = n / 8 > 65536 ? n / 8 : 65536;
  size_t bytes = Carver::pad((size_t)(n > 0 ? n : 1) * 8) + Carver::pad((size_t)(L + 1) * sizeof(ta_lane_gaps)) +
                 Carver::pad((size_t)(L + 1) * TA_NBINS * 4) + Carver::pad((size_t)W * TA_NBINS * 4) +
                 Carver::pad((size_t)cap * sizeof(ta_long_gap)) + 2 * Carver::pad((size_t)(tiles + 1) * 8) +
                 Carver::pad(64) + 512;
  void *b = ta_dalloc(h, bytes);
  if (!b) return TA_ERR_OOM;
  Carver c(b);
  int64_t *gap_before = c.take<int64_t>(n > 0 ? n : 1);
  // everything that must start at zero sits in one contiguous range
  char *zero_begin = c.base + c.off;
  ta_lane_gaps *lane_gaps = c.take<ta_lane_gaps>(L + 1);
  u32 *lane_hist = c.take<u32>((size_t)(L + 1) * TA_NBINS);
  u32 *win_hist = c.take<u32>((size_t)W * TA_NBINS);
  u64 *st_max = c.take<u64>(tiles + 1), *st_cnt = c.take<u64>(tiles + 1);
  u64 *scal = c.take<u64>(8);  // [0] n_long, [1] tile counter
  char *zero_end = c.base + c.off;
  ta_long_gap *list = c.take<ta_long_gap>(cap);
  TA_CHECK_CUDA(h, cudaMemsetAsync(zero_begin, 0, zero_end - zero_begin, st));

  GapArgs a;
  a.n = n; a.n_valid = h->n_valid; a.n_lanes = L;
  a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end; a.kind = h->sorted.kind;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window;
  a.lane_domain = h->sorted.lane_domain; a.t0 = h->d_t0; a.t1 = h->d_t1;
  a.min_gap = min_gap; a.list_only = 0;
  a.gap_before = gap_before; a.lane_gaps = lane_gaps; a.lane_hist = lane_hist; a.win_hist = win_hist;
  a.long_gaps = list; a.list_cap = cap; a.st_max = st_max; a.st_cnt = st_cnt;
  a.counter = (u32 *)(scal + 1); a.status = h->d_status; a.n_long_out = scal;
  if (tiles > 0) k_gaps<<<TA_N (unsigned)tiles, GP_THREADS, 0, st>>>(a);
  TA_CHECK_CUDA(h, cudaGetLastError());
  u64 n_long = 0;
  int32_t words[ST_WORDS];
  TA_CHECK_CUDA(h, cudaMemcpyAsync(&n_long, scal, 8, cudaMemcpyDeviceToHost, st));
  TA_TRY(ta_read_status(h, words));
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  if ((int64_t)n_long > cap) {
    // rare: a tiny min_gap made the list longer than the first guess; rebuild it
    void *b2 = ta_dalloc(h, (size_t)n_long * sizeof(ta_long_gap));
    if (!b2) return TA_ERR_OOM;
    TA_CHECK_CUDA(h, cudaMemsetAsync(st_max, 0, (char *)zero_end - (char *)st_max, st));
    a.long_gaps = (ta_long_gap *)b2; a.list_cap = (i64)n_long; a.list_only = 1;
    k_gaps<<<TA_N (unsigned)tiles, GP_THREADS, 0, st>>>(a);
    TA_CHECK_CUDA(h, cudaGetLastError());
    TA_TRY(ta_read_status(h, words));
    if (words[ST_ERR]) return (ta_status)words[ST_ERR];
    list = (ta_long_gap *)b2;
  }
  out->gap_before = gap_before;
  out->lane_gaps = lane_gaps;
  out->lane_hist = lane_hist;
  out->win_hist = win_hist;
  out->long_gaps = list;
  out->n_long_gaps = (int64_t)n_long;
  return TA_OK;
}
