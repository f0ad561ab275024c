// ta_stream_gaps: per device lane, the running maximum of the clipped end times
// (an exclusive max-scan in canonical order) gives the gap before every record,
// the busy union, idle time, a log2 gap histogram and the list of long gaps.
// Idle time of a stream = what none of its activity records covers (Sec. 9.1).
//
// One pass over the sorted ts_start / ts_end / kind columns.  The scan is made
// lane-aware without segment flags: the scanned value is (lane + 1) << 40 |
// (clipped end - window start), which grows from lane to lane, so a prefix
// that belongs to an earlier lane is recognised by its upper bits.  Long gaps
// are rare: they are appended to a list with an atomic cursor and the list is
// put in (lane, time) order afterwards with the pair sorter.
// HBM-bound: 18 B read + 8 B written per device record.
#include <climits>

#include "scan.cuh"
#include "ta_internal.cuh"

#define GP_THREADS 256
#ifndef GP_ITEMS
#define GP_ITEMS 8
#endif
#ifndef GP_MINB
#define GP_MINB 4
#endif
#define GP_TILE (GP_THREADS * GP_ITEMS)
#define GP_LOW ((1ull << 40) - 1)

struct GapArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int64_t *ts, *te;
  const int16_t *kind;
  const int32_t *lane_off, *lane_window;
  const int16_t *lane_domain;
  const int32_t *lane_dom_end;
  const int64_t *t0, *t1;
  i64 min_gap;
  int list_only;  // second run: only (re)write the long-gap list
  int local;      // 1: take the end of the record in front as the running maximum (and check that it is)
  u32 *not_ascending;  // set in local mode when some lane does not end its records in ascending order
  int64_t *gap_before;
  ta_lane_gaps *lane_gaps;
  u32 *lane_hist, *win_hist;
  ta_long_gap *list;  // unordered
  u64 *list_key;      // lane << 32 | next_event (0xFFFFFFFF for a tail gap)
  i64 list_cap;
  u64 *st_max;
  u32 *counter;
  int32_t *status;
  u64 *n_long;        // append cursor
};


__global__ void __launch_bounds__(GP_THREADS, GP_MINB) k_gaps(GapArgs a) {
  __shared__ u64 tmp[33];
  __shared__ u64 red[4][GP_THREADS / 32];
  __shared__ u64 s_excl_max;
  __shared__ u32 s_hist[2][TA_NBINS];  // the tile's first two lanes; further lanes go straight to global
  __shared__ int s_tile, s_lane0, s_lane1, s_fail;
  const int tid = threadIdx.x;
  if (tid == 0) {
    s_tile = (int)atomicAdd(a.counter, 1u);
    s_lane1 = -1;
    s_fail = ta_failed(a.status) ? 1 : 0;
  }
  if (tid < 2 * TA_NBINS) (&s_hist[0][0])[tid] = 0;
  __syncthreads();
  if (s_fail) return;
  const int tile = s_tile;
  const int64_t tile_start = (int64_t)tile * GP_TILE;
  const int64_t p0 = tile_start + (int64_t)tid * GP_ITEMS;
  if (tid < 32) {
    int l = -1;
    if (tile_start < a.n_valid && a.n_lanes > 0) l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (tid == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  const bool full = p0 + GP_ITEMS <= a.n;
  if (l0 >= 0 && span_outside_domain(a.lane_domain, a.lane_dom_end, l0,
                                     min(tile_start + GP_TILE, a.n_valid), 1)) {
    // host lanes only: no gaps here, and no later device lane can use anything scanned so far
    if (tid == 0) st_relaxed(&a.st_max[tile], td_pack(TD_PREFIX, 0));
    if (a.list_only) return;
    if (full) {
      longlong2 *pg = reinterpret_cast<longlong2 *>(a.gap_before + p0);
#pragma unroll
      for (int j = 0; j < GP_ITEMS / 2; j++) pg[j] = make_longlong2(0, 0);
    } else {
      for (int j = 0; j < GP_ITEMS; j++)
        if (p0 + j < a.n) a.gap_before[p0 + j] = 0;
    }
    return;
  }
  // kinds, start and end times of the thread's records and, for the scan-free mode, the end of
  // the record in front of the thread's first one: all requested together (the tile holds a
  // device lane, so nearly every record needs its times anyway)
  int16_t kd[GP_ITEMS];
  loadn_i16<GP_ITEMS>(a.kind, p0, a.n, 0, kd);
  i64 s[GP_ITEMS], ce[GP_ITEMS];  // ce: ts_end, clipped below
#pragma unroll
  for (int j = 0; j < GP_ITEMS; j++) s[j] = ce[j] = 0;
  if (full) {
    const longlong2 *ps = reinterpret_cast<const longlong2 *>(a.ts + p0);
    const longlong2 *pe = reinterpret_cast<const longlong2 *>(a.te + p0);
#pragma unroll
    for (int j = 0; j < GP_ITEMS / 2; j++) {
      longlong2 x = ps[j], y = pe[j];
      s[2 * j] = x.x; s[2 * j + 1] = x.y;
      ce[2 * j] = y.x; ce[2 * j + 1] = y.y;
    }
  } else {
#pragma unroll
    for (int j = 0; j < GP_ITEMS; j++)
      if (p0 + j < a.n) { s[j] = a.ts[p0 + j]; ce[j] = a.te[p0 + j]; }
  }
  const i64 e_before = (a.local && p0 > 0 && p0 <= a.n) ? a.te[p0 - 1] : 0;
#pragma unroll
  for (int j = 0; j < GP_ITEMS; j++)
    if (p0 + j >= a.n_valid) kd[j] = 0;
  // lanes of the items: walk forward from the tile's first lane
  int ln[GP_ITEMS];
  u64 run = 0;
  unsigned lastmask = 0, firstmask = 0;  // items that end / begin their lane
  {
    int l = l0;
    int64_t next_off = l >= 0 ? (int64_t)a.lane_off[l + 1] : LLONG_MAX;
    int64_t cur_off = l >= 0 ? (int64_t)a.lane_off[l] : 0;
    i64 w0 = 0, w1 = 0;
    int wl = -1;
#pragma unroll
    for (int j = 0; j < GP_ITEMS; j++) {
      const int64_t p = p0 + j;
      ln[j] = -1;
      if (kd[j] >= 3) {
        while (p >= next_off) { l++; cur_off = next_off; next_off = a.lane_off[l + 1]; }
        if (wl != l) { int w = a.lane_window[l]; w0 = a.t0[w]; w1 = a.t1[w]; wl = l; }
        ln[j] = l;
        if (p + 1 == next_off) lastmask |= 1u << j;
        if (p == cur_off) firstmask |= 1u << j;
        ce[j] = ce[j] < w1 ? ce[j] : w1;
        u64 v = ((u64)(l + 1) << 40) | (u64)(ce[j] - w0);
        run = run > v ? run : v;
      }
    }
    const int64_t plast = min(tile_start + GP_TILE, a.n_valid) - 1;
    if (plast >= p0 && plast < p0 + GP_ITEMS) {  // this thread owns the tile's last kept record
      while (plast >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      s_lane1 = l;
    }
  }
  u64 pre = 0;
  if (a.local) {
    // in-order streams end their records in ascending order: the running maximum in front of a
    // record is the (clipped) end of its neighbour, no scan and no look-back; the loop below
    // checks the order and reports the first lane that breaks it
    const int l = ln[0];
    if (l >= 0 && p0 > (int64_t)a.lane_off[l]) {
      const int w = a.lane_window[l];
      const i64 w0 = a.t0[w], w1 = a.t1[w], e = e_before;
      pre = ((u64)(l + 1) << 40) | (u64)((e < w1 ? e : w1) - w0);
    }
    __syncthreads();  // s_lane1 and the zeroed histograms are read below
  } else {
    u64 tile_max;
    u64 thread_excl = block_scan_exclusive<OpMax>(run, OpMax(), tmp, &tile_max);
    if (tid < 32) {
      bool failed;
      u64 ex = tile_lookback<OpMax>(a.st_max, tile, tile_max, OpMax(), a.status, &failed);
      if (tid == 0) { s_excl_max = ex; s_fail = failed ? 1 : 0; }
    }
    __syncthreads();
    if (s_fail) return;
    pre = s_excl_max > thread_excl ? s_excl_max : thread_excl;
  }

  // gaps; statistics of the thread's first lane stay in registers, anything else is rare
  i64 gap[GP_ITEMS];
  u64 sb = 0, si = 0, ng = 0, mg = 0;
  int lm = -1;
  {
    i64 w0 = 0, w1 = 0;
    int wl = -1;
#pragma unroll
    for (int j = 0; j < GP_ITEMS; j++) {
      gap[j] = 0;
      const int l = ln[j];
      i64 Pi = 0, g = 0, bz = 0, tl = 0;
      bool last = false, lg = false, lt = false;
      if (l >= 0) {
        if (wl != l) { int w = a.lane_window[l]; w0 = a.t0[w]; w1 = a.t1[w]; wl = l; }
        Pi = ((pre >> 40) == (u64)(l + 1)) ? w0 + (i64)(pre & GP_LOW) : w0;
        if (a.local && (pre >> 40) == (u64)(l + 1) && ce[j] < Pi) *a.not_ascending = 1u;
        g = s[j] > Pi ? s[j] - Pi : 0;
        const i64 from = s[j] > Pi ? s[j] : Pi;
        bz = ce[j] > from ? ce[j] - from : 0;
        last = (lastmask >> j) & 1u;
        if (last) tl = w1 - (Pi > ce[j] ? Pi : ce[j]);
        gap[j] = g;
        pre = max(pre, ((u64)(l + 1) << 40) | (u64)(ce[j] - w0));
        lg = g > 0 && g >= a.min_gap;
        lt = last && tl > 0 && tl >= a.min_gap;
      }
      // long-gap list: the warp reserves its entries with one add on the cursor (the order of
      // the list does not matter, it is sorted afterwards)
      if (__any_sync(0xffffffffu, lg || lt)) {  // rare: one vote decides for the warp
        const u32 m_g = __ballot_sync(0xffffffffu, lg), m_t = __ballot_sync(0xffffffffu, lt);
        {
          const int wlane = threadIdx.x & 31;
          const u32 below = (1u << wlane) - 1u;
          u64 base = 0;
          if (wlane == 0) base = atomicAdd(a.n_long, (u64)(__popc(m_g) + __popc(m_t)));
          base = __shfl_sync(0xffffffffu, base, 0);
          if (lg) {
            const i64 o = (i64)base + __popc(m_g & below);
            if (o < a.list_cap) {
              a.list[o] = ta_long_gap{l, (int32_t)(p0 + j), Pi, g};
              a.list_key[o] = ((u64)l << 32) | (u64)(u32)(p0 + j);
            }
          }
          if (lt) {
            const i64 o = (i64)base + __popc(m_g) + __popc(m_t & below);
            if (o < a.list_cap) {
              a.list[o] = ta_long_gap{l, -1, w1 - tl, tl};
              a.list_key[o] = ((u64)l << 32) | 0xFFFFFFFFull;
            }
          }
        }
      }
      if (l < 0) continue;
      if (a.list_only) continue;
      if (lm < 0) lm = l;
      const int li = l - l0;
      if (l == lm && li <= 1) {
        sb += (u64)bz;
        si += (u64)(g + tl);
        if (g > 0) { ng++; mg = max(mg, (u64)g); atomicAdd(&s_hist[li][log2_bin(g)], 1u); }
        if (tl > 0) { ng++; mg = max(mg, (u64)tl); atomicAdd(&s_hist[li][log2_bin(tl)], 1u); }
      } else {  // a thread that straddles a lane boundary, or a third lane in the tile
        ta_lane_gaps *gl = &a.lane_gaps[l];
        const int w = a.lane_window[l];
        if (bz) atomicAdd((u64 *)&gl->busy, (u64)bz);
        if (g + tl) atomicAdd((u64 *)&gl->idle, (u64)(g + tl));
        if (g > 0) {
          atomicAdd((u64 *)&gl->n_gaps, 1ull);
          atomicMax((i64 *)&gl->max_gap, g);
          atomicAdd(&a.lane_hist[(size_t)l * TA_NBINS + log2_bin(g)], 1u);
          atomicAdd(&a.win_hist[(size_t)w * TA_NBINS + log2_bin(g)], 1u);
        }
        if (tl > 0) {
          atomicAdd((u64 *)&gl->n_gaps, 1ull);
          atomicMax((i64 *)&gl->max_gap, tl);
          atomicAdd(&a.lane_hist[(size_t)l * TA_NBINS + log2_bin(tl)], 1u);
          atomicAdd(&a.win_hist[(size_t)w * TA_NBINS + log2_bin(tl)], 1u);
        }
      }
      if (last) {
        a.lane_gaps[l].last_end = w1 - tl;
        a.lane_gaps[l].n_events = (i64)a.lane_off[l + 1] - (i64)a.lane_off[l];
      }
      if ((firstmask >> j) & 1u) a.lane_gaps[l].first_start = s[j];
    }
  }
  if (a.list_only) return;
  if (full) {
    longlong2 *pg = reinterpret_cast<longlong2 *>(a.gap_before + p0);
#pragma unroll
    for (int j = 0; j < GP_ITEMS / 2; j++) pg[j] = make_longlong2(gap[2 * j], gap[2 * j + 1]);
  } else {
#pragma unroll
    for (int j = 0; j < GP_ITEMS; j++)
      if (p0 + j < a.n) a.gap_before[p0 + j] = gap[j];
  }
  // fold the register statistics of the tile's first two lanes
  const int l1 = s_lane1;
  for (int li = 0; li < 2; li++) {
    const int l = l0 + li;
    if (l0 < 0 || l > l1) break;
    if (a.lane_domain[l] != 1) continue;  // uniform over the CTA
    const bool mine = lm == l;
    u64 r0 = warp_reduce(mine ? sb : 0, OpAdd());
    u64 r1 = warp_reduce(mine ? si : 0, OpAdd());
    u64 r2 = warp_reduce(mine ? ng : 0, OpAdd());
    u64 r3 = warp_reduce(mine ? mg : 0, OpMax());
    __syncthreads();
    if ((tid & 31) == 0) { red[0][tid >> 5] = r0; red[1][tid >> 5] = r1; red[2][tid >> 5] = r2; red[3][tid >> 5] = r3; }
    __syncthreads();
    if (tid < 4) {
      u64 t = 0;
      for (int w = 0; w < GP_THREADS / 32; w++) t = tid == 3 ? max(t, red[3][w]) : t + red[tid][w];
      if (t) {
        ta_lane_gaps *gl = &a.lane_gaps[l];
        if (tid == 0) atomicAdd((u64 *)&gl->busy, t);
        else if (tid == 1) atomicAdd((u64 *)&gl->idle, t);
        else if (tid == 2) atomicAdd((u64 *)&gl->n_gaps, t);
        else atomicMax((i64 *)&gl->max_gap, (i64)t);
      }
    }
    if (tid < TA_NBINS && s_hist[li][tid]) {
      atomicAdd(&a.lane_hist[(size_t)l * TA_NBINS + tid], s_hist[li][tid]);
      atomicAdd(&a.win_hist[(size_t)a.lane_window[l] * TA_NBINS + tid], s_hist[li][tid]);
    }
  }
}

__global__ void __launch_bounds__(256) k_gap_list_gather(const ta_long_gap *src, const u32 *order,
                                                         int64_t m, ta_long_gap *dst,
                                                         const int32_t *status) {
  if (ta_failed(status)) return;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < m) dst[i] = src[order[i]];
}

ta_status ta_run_gaps(ta_window *h, int64_t min_gap, ta_gap_result *out) {
  const int64_t n = h->n;
  const int L = h->sorted.n_lanes;
  const int W = h->W;
  cudaStream_t st = h->stream;
  if (L >= (1 << 22) - 1) return TA_ERR_TOO_LARGE;
  const int64_t tiles = (n + GP_TILE - 1) / GP_TILE;
  int64_t cap = n / 8 > 65536 ? n / 8 : 65536;  // first guess; a longer list is rebuilt below
  size_t bytes = Carver::pad((size_t)(n > 0 ? n : 1) * 8) + Carver::pad((size_t)(L + 1) * sizeof(ta_lane_gaps)) +
                 Carver::pad((size_t)(L + 1) * TA_NBINS * 4) + Carver::pad((size_t)W * TA_NBINS * 4) +
                 Carver::pad((size_t)(tiles + 1) * 8) + Carver::pad(64) + 512;
  void *b = ta_dalloc(h, bytes);
  if (!b) return TA_ERR_OOM;
  Carver c(b);
  int64_t *gap_before = c.take<int64_t>(n > 0 ? n : 1);
  // everything that must start at zero sits in one contiguous range
  char *zero_begin = c.base + c.off;
  ta_lane_gaps *lane_gaps = c.take<ta_lane_gaps>(L + 1);
  u32 *lane_hist = c.take<u32>((size_t)(L + 1) * TA_NBINS);
  u32 *win_hist = c.take<u32>((size_t)W * TA_NBINS);
  u64 *st_max = c.take<u64>(tiles + 1);
  u64 *scal = c.take<u64>(8);  // [0] list cursor, [1] tile counter
  char *zero_end = c.base + c.off;
  TA_CHECK_CUDA(h, cudaMemsetAsync(zero_begin, 0, zero_end - zero_begin, st));
  // unordered list + keys (temporary)
  void *lt = ta_dalloc(h, Carver::pad((size_t)cap * sizeof(ta_long_gap)) + Carver::pad((size_t)cap * 8) + 256);
  if (!lt) return TA_ERR_OOM;
  Carver cl(lt);
  ta_long_gap *ulist = cl.take<ta_long_gap>(cap);
  u64 *ukeys = cl.take<u64>(cap);

  GapArgs a;
  a.n = n; a.n_valid = h->n_valid; a.n_lanes = L;
  a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end; a.kind = h->sorted.kind;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window;
  a.lane_domain = h->sorted.lane_domain; a.lane_dom_end = h->d_lane_dom_end; a.t0 = h->d_t0; a.t1 = h->d_t1;
  a.min_gap = min_gap; a.list_only = 0;
  a.gap_before = gap_before; a.lane_gaps = lane_gaps; a.lane_hist = lane_hist; a.win_hist = win_hist;
  a.list = ulist; a.list_key = ukeys; a.list_cap = cap; a.st_max = st_max;
  a.counter = (u32 *)(scal + 1); a.status = h->d_status; a.n_long = scal;
  a.not_ascending = (u32 *)(scal + 2);
  u64 n_long = 0;
  int32_t words[ST_WORDS];
  // first without the scan (every lane is taken to end its records in ascending order, which the
  // kernel checks); if a lane does not, once more with the chained maximum scan
  for (a.local = 1; a.local >= 0; a.local--) {
    if (tiles > 0) k_gaps<<<TA_N (unsigned)tiles, GP_THREADS, 0, st>>>(a);
    TA_CHECK_CUDA(h, cudaGetLastError());
    u64 two[3] = {0, 0, 0};
    TA_TRY(ta_queue_d2h(h, two, scal, 24));
    TA_TRY(ta_read_status(h, words));
    if (words[ST_ERR]) return (ta_status)words[ST_ERR];
    n_long = two[0];
    if (!a.local || !(u32)two[2]) break;
    TA_CHECK_CUDA(h, cudaMemsetAsync(zero_begin, 0, zero_end - zero_begin, st));
  }
  if ((int64_t)n_long > cap) {
    // rare: a tiny min_gap made the list longer than the first guess; rebuild it
    ta_dfree(h, lt);
    cap = (int64_t)n_long;
    lt = ta_dalloc(h, Carver::pad((size_t)cap * sizeof(ta_long_gap)) + Carver::pad((size_t)cap * 8) + 256);
    if (!lt) return TA_ERR_OOM;
    Carver cl2(lt);
    ulist = cl2.take<ta_long_gap>(cap);
    ukeys = cl2.take<u64>(cap);
    TA_CHECK_CUDA(h, cudaMemsetAsync(st_max, 0, (char *)zero_end - (char *)st_max, st));
    a.list = ulist; a.list_key = ukeys; a.list_cap = cap; a.list_only = 1;
    k_gaps<<<TA_N (unsigned)tiles, GP_THREADS, 0, st>>>(a);
    TA_CHECK_CUDA(h, cudaGetLastError());
    TA_TRY(ta_read_status(h, words));
    if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  }
  // order the list by (lane, position; tail last)
  ta_long_gap *list = nullptr;
  const int64_t m = (int64_t)n_long;
  if (m > 0) {
    list = (ta_long_gap *)ta_dalloc(h, (size_t)m * sizeof(ta_long_gap));
    if (!list) return TA_ERR_OOM;
    void *stb = ta_dalloc(h, 2 * Carver::pad((size_t)m * 8) + 2 * Carver::pad((size_t)m * 4) +
                                 ta_sort_temp_bytes(m) + 256);
    if (!stb) return TA_ERR_OOM;
    Carver cs(stb);
    u64 *ks = cs.take<u64>(m), *kf = cs.take<u64>(m);
    u32 *vs = cs.take<u32>(m), *order = cs.take<u32>(m);
    TA_TRY(ta_radix_sort_pairs(h, ukeys, nullptr, ks, vs, kf, order, m,
                               ta_make_plan(0, 32 + ta_bit_len((uint64_t)(L > 1 ? L - 1 : 1))), nullptr,
                               cs.base + cs.off));
    k_gap_list_gather<<<TA_N (unsigned)((m + 255) / 256), 256, 0, st>>>(ulist, order, m, list, h->d_status);
    TA_CHECK_CUDA(h, cudaGetLastError());
    // the sort and the gather are still queued: their temporaries go back after the handle's
    // next synchronisation (the list itself is used in stream order like every other result)
    ta_dfree_later(h, stb);
    ta_dfree_later(h, lt);
    lt = nullptr;
  }
  if (lt) ta_dfree(h, lt);
  out->gap_before = gap_before;
  out->lane_gaps = lane_gaps;
  out->lane_hist = lane_hist;
  out->win_hist = win_hist;
  out->long_gaps = list;
  out->n_long_gaps = m;
  return TA_OK;
}
