// ta_sort_timeline: canonical order of the timeline.
//
// Packed keys (the usual case): the key carries the record's index in its low bits and the
// start time at a coarser resolution, so four keys-only radix passes settle the order down
// to (lane, coarse time); k_gather, which brings every 40-byte record into registers once to
// write the eight sorted columns, ranks the members of a run of equal coarse keys by
// (ts_start, -ts_end, input index) on the way, and records the lane boundaries and the
// correlation-id range of every (window, pid) for the join.
// Fallback (a run longer than TA_TIE_RUN_MAX, or keys that do not fit): stable radix sort of
// (key, input index) pairs at full time resolution; runs of equal keys are reordered by
// ts_end descending in place (k_fix_ties), and if even such a run is too long the sort is
// redone with the duration as a least-significant key.
// Dropped records (the tail) are ordered by the full tuple with a chain of stable sorts.
#include <climits>

#include "records.cuh"
#include "ta_internal.cuh"

// ---- pair path: equal-key runs -------------------------------------------
__global__ void __launch_bounds__(256) k_fix_ties(const u64 *keys, u32 *perm, int64_t n_valid,
                                                  const ta_event *ev, int32_t *status) {
  if (ta_failed(status)) return;
  int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n_valid || p + 1 >= n_valid) return;
  u64 k = keys[p];
  if (keys[p + 1] != k) return;
  if (p > 0 && keys[p - 1] == k) return;
  int len = 2;
  while (p + len < n_valid && len <= TA_TIE_RUN_MAX && keys[p + len] == k) len++;
  if (len > TA_TIE_RUN_MAX) {
    status[ST_LONG_RUN] = 1;
    return;
  }
  u32 idx[TA_TIE_RUN_MAX];
  i64 end[TA_TIE_RUN_MAX];
  for (int i = 0; i < len; i++) {
    idx[i] = perm[p + i];
    end[i] = reinterpret_cast<const i64 *>(ev)[(int64_t)idx[i] * 5 + 1];
  }
  for (int i = 1; i < len; i++) {  // stable insertion sort, ts_end descending
    u32 xi = idx[i];
    i64 xe = end[i];
    int j = i - 1;
    while (j >= 0 && end[j] < xe) {
      idx[j + 1] = idx[j];
      end[j + 1] = end[j];
      j--;
    }
    idx[j + 1] = xi;
    end[j + 1] = xe;
  }
  for (int i = 0; i < len; i++) perm[p + i] = idx[i];
}

// ---- fallback: duration as a least-significant key ------------------------
__global__ void __launch_bounds__(256) k_duration_key(const ta_event *ev, int64_t n, const u64 *keys,
                                                      u64 dropped_bit, i64 max_dur, u64 *out) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  if (keys[i] & dropped_bit) { out[i] = 0; return; }
  const i64 *p = reinterpret_cast<const i64 *>(ev) + i * 5;
  out[i] = (u64)(max_dur - (p[1] - p[0]));  // longer first
}
__global__ void __launch_bounds__(256) k_gather_u64(const u64 *src, const u32 *idx, int64_t n, u64 *dst,
                                                    const int32_t *status) {
  if (ta_failed(status)) return;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[idx[i]];
}

// ---- step 3: full-tuple keys for the dropped tail -------------------------
// stage 0: ~ts_end, 1: ts_start, 2: (pid, domain, stream), 3: window
__global__ void __launch_bounds__(256) k_tail_key(const ta_event *ev, const u32 *idx, int64_t m,
                                                  int stage, const int64_t *off, int W, u64 *out,
                                                  const int32_t *status) {
  if (ta_failed(status)) return;
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  Rec r = load_rec(ev, idx[j]);
  u64 k;
  if (stage == 0) k = ~((u64)r.ts_end ^ (1ull << 63));
  else if (stage == 1) k = (u64)r.ts_start ^ (1ull << 63);
  else if (stage == 2) k = triple_code(r.pid, r.kind, r.stream);
  else k = (u64)window_of(off, W, idx[j]);
  out[j] = k;
}

// ---- step 4: gather records into sorted columns + lane heads ---------------
struct GatherArgs {
  const ta_event *ev;
  u32 *perm;          // pairs: input; packed keys: written here for the kept records
  const u64 *keys;
  int64_t n, n_valid;
  int sbits;          // key bits below the lane code (time bits kept [+ index bits])
  int packed, ibits, wshift, wbits;
  const int64_t *off;
  // corr_id range of the LAUNCH records per (window, pid) slot, for the join
  const TripleTable *tt;
  int tbits, n_pids;
  i64 *slot_min, *slot_max;
  i64 *ts_start, *ts_end, *corr;
  int32_t *pid, *name, *seq;
  int16_t *stream, *kind;
  int32_t *lane_start;  // per lane code, -1 = empty
  int32_t *status;
};
__device__ __forceinline__ u32 gather_index(u64 k, const GatherArgs &a) {
  const int w = a.wbits ? (int)((k >> a.wshift) & ((1ull << a.wbits) - 1)) : 0;
  return (u32)(a.off[w] + (int64_t)(k & ((1ull << a.ibits) - 1)));
}

// eight CTAs per SM (32 registers): the kernel lives on occupancy, 42 or 51 registers measured slower
#ifndef GT_MINB
#define GT_MINB 8
#endif
__global__ void __launch_bounds__(256, GT_MINB) k_gather(GatherArgs a) {
  __shared__ int s_slot[8];
  __shared__ u64 s_mx[8], s_mn[8];
  if (ta_failed(a.status)) return;  // the sort gave up: the keys name no records
  // positions fit 32 bits (n < 2^31): 32-bit indices keep the address arithmetic of the nine
  // column stores and of the neighbour reads short
  const u32 p = blockIdx.x * blockDim.x + threadIdx.x;
  const u32 n = (u32)a.n, nv = (u32)a.n_valid;
  int slot = -1;
  u64 mx = 0, mn_inv = 0;
  if (p < n) {
  u32 idx;
  u32 dst = p;  // where the record goes: p, or its place inside a run of equal coarse keys
  int before = 0, after = 0;
  // the record's key and the key in front of it: both are needed twice below
  u64 k = 0, kprev = 0;
  if (p < nv) {
    k = a.keys[p];
    if (p > 0) kprev = a.keys[p - 1];
  }
  if (a.packed && p < nv) {
    idx = gather_index(k, a);
    // packed keys order the records down to a coarse time only: members of a run of equal
    // (lane, coarse time) sit in no particular order (the first radix pass is not stable) and
    // are ranked here by (ts_start, -ts_end, input index)
    const u64 hk = k >> a.ibits;
    if (p > 0 && (kprev >> a.ibits) == hk) {
      before = 1;
      while (before <= TA_TIE_RUN_MAX && p - before > 0 && (a.keys[p - before - 1] >> a.ibits) == hk)
        before++;
    }
    while (after <= TA_TIE_RUN_MAX && p + after + 1 < nv && (a.keys[p + after + 1] >> a.ibits) == hk)
      after++;
    if (before + after + 1 > TA_TIE_RUN_MAX) {
      a.status[ST_LONG_RUN] = 1;  // the caller starts over with full-resolution keys
      before = after = 0;
    }
  } else {
    idx = a.perm[p];
  }
  Rec r = load_rec(a.ev, idx);
  if (before + after > 0) {
    int rank = 0;
    for (int q = -before; q <= after; q++) {
      if (q == 0) continue;
      const u32 oi = gather_index(a.keys[p + q], a);
      const i64 *o = reinterpret_cast<const i64 *>(a.ev) + (u64)oi * 5;
      const i64 os = o[0], oe = o[1];
      const bool first = os < r.ts_start || (os == r.ts_start && (oe > r.ts_end || (oe == r.ts_end && oi < idx)));
      rank += first ? 1 : 0;
    }
    dst = p - before + rank;
  }
  if (a.packed && p < nv) a.perm[dst] = idx;
  a.ts_start[dst] = r.ts_start;
  a.ts_end[dst] = r.ts_end;
  a.corr[dst] = r.corr;
  a.pid[dst] = r.pid;
  a.name[dst] = r.name;
  a.seq[dst] = r.seq;
  a.stream[dst] = r.stream;
  a.kind[dst] = r.kind;
  if (p < nv) {
    const u64 code = k >> a.sbits;
    if (p == 0 || (kprev >> a.sbits) != code) a.lane_start[code] = (int32_t)p;
    if (r.kind == TA_KIND_LAUNCH) {
      slot = (int)(code >> a.tbits) * a.n_pids + a.tt->pid_rank[code & ((1ull << a.tbits) - 1)];
      mx = (u64)r.corr ^ (1ull << 63);
      mn_inv = ~mx;
    }
  }
  }  // p < n
  // fold the range per CTA (a CTA almost always sits inside one lane)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const u32 has = __ballot_sync(0xffffffffu, slot >= 0);
  int wslot = -1;
  if (has) {
    wslot = __shfl_sync(0xffffffffu, slot, __ffs(has) - 1);
    if (__all_sync(0xffffffffu, slot < 0 || slot == wslot)) {
      mx = warp_reduce(mx, OpMax());
      mn_inv = warp_reduce(mn_inv, OpMax());
    } else {  // mixed warp (lane boundary): every thread for itself
      if (slot >= 0) {
        atomicMax(&a.slot_max[slot], (i64)(mx ^ (1ull << 63)));
        atomicMin(&a.slot_min[slot], (i64)((~mn_inv) ^ (1ull << 63)));
      }
      wslot = -1;
    }
  }
  if (lane == 0) { s_slot[warp] = wslot; s_mx[warp] = mx; s_mn[warp] = mn_inv; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int cur = -1;
    u64 cmx = 0, cmn = 0;
    for (int w = 0; w <= 8; w++) {
      const int sl = w < 8 ? s_slot[w] : -2;
      if (sl == -1) continue;
      if (sl != cur) {
        if (cur >= 0) {
          const i64 hi = (i64)(cmx ^ (1ull << 63)), lo = (i64)((~cmn) ^ (1ull << 63));
          if (hi > a.slot_max[cur]) atomicMax(&a.slot_max[cur], hi);
          if (lo < a.slot_min[cur]) atomicMin(&a.slot_min[cur], lo);
        }
        cur = sl;
        cmx = 0;
        cmn = 0;
      }
      if (w < 8) { cmx = max(cmx, s_mx[w]); cmn = max(cmn, s_mn[w]); }
    }
  }
}

// One CTA: compacts the non-empty lane codes into the lane table (code order is
// canonical order).
__global__ void __launch_bounds__(1024) k_lane_table(const int32_t *lane_start, int64_t n_codes,
                                                     int tbits, int n_pids, const TripleTable *tt,
                                                     int64_t n_valid, int32_t *lane_window,
                                                     int32_t *lane_pid, int16_t *lane_stream,
                                                     int16_t *lane_domain, int32_t *lane_off,
                                                     int32_t *lane_code, int32_t *lane_slot,
                                                     int32_t *lane_dom_end, int32_t *lane_dom_next,
                                                     int32_t *lane_dev_base, int32_t *n_lanes_out,
                                                     int64_t cap, const int32_t *status) {
  __shared__ u64 tmp[33];
  __shared__ u64 base;
  if (ta_failed(status)) {  // no lanes: every later call then finds nothing to index
    if (threadIdx.x == 0) { n_lanes_out[0] = 0; n_lanes_out[1] = 0; }
    return;
  }
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int64_t c0 = 0; c0 < n_codes; c0 += blockDim.x) {
    int64_t c = c0 + threadIdx.x;
    int32_t st = c < n_codes ? lane_start[c] : -1;
    u64 total;
    u64 ex = block_scan_exclusive<OpAdd>(st >= 0 ? 1ull : 0ull, OpAdd(), tmp, &total);
    if (st >= 0) {
      int64_t l = (int64_t)(base + ex);
      if (l < cap) {
        int w = (int)(c >> tbits), t = (int)(c & ((1ll << tbits) - 1));
        u64 code = tt->sorted_code[t];
        lane_window[l] = w;
        lane_pid[l] = code_pid(code);
        lane_stream[l] = code_stream(code);
        lane_domain[l] = code_domain(code);
        lane_off[l] = st;
        lane_code[l] = (int32_t)c;
        lane_slot[l] = w * n_pids + tt->pid_rank[t];
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) base += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    int64_t L = (int64_t)base;
    if (L < cap + 1) lane_off[L] = (int32_t)n_valid;
    *n_lanes_out = (int32_t)L;
  }
  __syncthreads();
  // per lane: the first later lane of the other domain, and the position where it begins (host
  // and device lanes alternate per (window, pid), so the runs are a few lanes long - but a batch
  // of device-only windows is one long run, hence a scan and no walk).  Going backwards over
  // the lanes, the nearest boundary at or behind lane l is a running maximum of
  // L - (index of the lane behind a boundary); chunks of blockDim.x lanes, carried in `base`.
  const int64_t L = (int64_t)base < cap ? (int64_t)base : cap;
  __syncthreads();  // every thread has read the lane count before `base` is reused
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int64_t r0 = 0; r0 < L; r0 += blockDim.x) {
    const int64_t r = r0 + threadIdx.x;  // reversed lane index
    const int64_t l = L - 1 - r;
    u64 v = 0;
    if (r < L && l + 1 < L && lane_domain[l + 1] != lane_domain[l]) v = (u64)(L - (l + 1));
    u64 total;
    const u64 ex = block_scan_exclusive<OpMax>(v, OpMax(), tmp, &total);
    if (r < L) {
      u64 best = ex > v ? ex : v;
      best = best > base ? best : base;
      const int64_t m = best ? L - (int64_t)best : L;
      lane_dom_end[l] = m < L ? lane_off[m] : (int32_t)n_valid;
      lane_dom_next[l] = (int32_t)m;  // index of the first later lane of the other domain (L if none)
    }
    __syncthreads();
    if (threadIdx.x == 0) base = base > total ? base : total;
    __syncthreads();
  }
  // per device lane: how many device records sit in earlier lanes (their index once the device
  // records are taken out in order); n_lanes_out[1] = the number of device records
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int64_t l0 = 0; l0 < L; l0 += blockDim.x) {
    const int64_t l = l0 + threadIdx.x;
    u64 sz = 0;
    if (l < L && lane_domain[l] == 1) sz = (u64)((l + 1 < L ? lane_off[l + 1] : (int32_t)n_valid) - lane_off[l]);
    u64 total;
    const u64 ex = block_scan_exclusive<OpAdd>(sz, OpAdd(), tmp, &total);
    if (l < L) lane_dev_base[l] = (int32_t)(base + ex);
    __syncthreads();
    if (threadIdx.x == 0) base += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) n_lanes_out[1] = (int32_t)base;
}

// ---- packed keys: index of the record a key stands for -------------------------
struct PackInfo {
  int ibits, wshift, wbits;
  const int64_t *off;
};
__device__ __forceinline__ u32 packed_index(u64 k, const PackInfo &pi) {
  const int w = pi.wbits ? (int)((k >> pi.wshift) & ((1ull << pi.wbits) - 1)) : 0;
  return (u32)(pi.off[w] + (int64_t)(k & ((1ull << pi.ibits) - 1)));
}
__global__ void __launch_bounds__(256) k_unpack_tail(const u64 *keys, int64_t n_valid, int64_t n,
                                                     PackInfo pi, u32 *perm, const int32_t *status) {
  if (ta_failed(status)) return;
  int64_t p = n_valid + (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p < n) perm[p] = packed_index(keys[p], pi);
}

static inline int nblk(int64_t n, int t) { return (int)((n + t - 1) / t); }

ta_status ta_run_sort_timeline(ta_window *h) {
  const int64_t n = h->n;
  cudaStream_t st = h->stream;
  const int64_t n_codes = (int64_t)h->W << h->tbits;  // lane code = window << tbits | triple rank
  const int64_t lane_cap = (n_codes < n ? n_codes : n) + 1;  // lanes <= min(codes, records)
  const int64_t n_slots = (int64_t)h->W * (h->n_pids > 0 ? h->n_pids : 1);

  // result buffers (kept until ta_free)
  size_t keep = Carver::pad(n * 4) + 3 * Carver::pad(n * 8) + 3 * Carver::pad(n * 4) +
                2 * Carver::pad(n * 2) + 7 * Carver::pad(lane_cap * 4) + 2 * Carver::pad(lane_cap * 2) +
                Carver::pad((lane_cap + 1) * 4) + Carver::pad((size_t)n_slots * 16) + 512;
  void *kb = ta_dalloc(h, keep);
  if (!kb) return TA_ERR_OOM;
  Carver ck(kb);
  u32 *perm = ck.take<u32>(n);
  i64 *c_ts = ck.take<i64>(n), *c_te = ck.take<i64>(n), *c_corr = ck.take<i64>(n);
  int32_t *c_pid = ck.take<int32_t>(n), *c_name = ck.take<int32_t>(n), *c_seq = ck.take<int32_t>(n);
  int16_t *c_stream = ck.take<int16_t>(n), *c_kind = ck.take<int16_t>(n);
  int32_t *lane_window = ck.take<int32_t>(lane_cap), *lane_pid = ck.take<int32_t>(lane_cap);
  int32_t *lane_code = ck.take<int32_t>(lane_cap), *lane_slot = ck.take<int32_t>(lane_cap);
  int16_t *lane_stream = ck.take<int16_t>(lane_cap), *lane_domain = ck.take<int16_t>(lane_cap);
  int32_t *lane_off = ck.take<int32_t>(lane_cap + 1);
  int32_t *lane_dom_end = ck.take<int32_t>(lane_cap);
  int32_t *lane_dev_base = ck.take<int32_t>(lane_cap);
  int32_t *lane_dom_next = ck.take<int32_t>(lane_cap);
  int32_t *n_lanes_dev = ck.take<int32_t>(2);  // [0] lanes, [1] device records
  h->d_slot_min = ck.take<i64>(2 * n_slots);  // minima, then maxima, contiguous
  h->d_slot_max = h->d_slot_min + n_slots;

  // temporaries (released at the end of the call)
  size_t tmp_bytes = 2 * Carver::pad(n * 8) + Carver::pad(n * 4) + ta_sort_temp_bytes(n) +
                     Carver::pad(n_codes * 4) + 512;
  void *tb = ta_dalloc(h, tmp_bytes);
  if (!tb) return TA_ERR_OOM;
  Carver ct(tb);
  u64 *kscr = ct.take<u64>(n), *skeys = ct.take<u64>(n);
  u32 *vscr = ct.take<u32>(n);
  int32_t *lane_start = ct.take<int32_t>(n_codes);
  void *sort_tmp = ct.base + ct.off;

  int32_t n_lanes_host[2] = {0, 0};
  // Packed keys settle the order down to a coarse time; the gather ranks the members of a run
  // of equal coarse keys itself.  A run too long for that is reported at the end, and the
  // second attempt sorts (key, index) pairs at full time resolution.
  for (int attempt = 0; attempt < 2; attempt++) {
    int32_t words[ST_WORDS];
    h->h_slot_min.assign((size_t)n_slots, INT64_MAX);
    h->h_slot_max.assign((size_t)n_slots, INT64_MIN);
    {  // the two ranges sit side by side on the device: one copy
      std::vector<int64_t> init(h->h_slot_min);
      init.insert(init.end(), h->h_slot_max.begin(), h->h_slot_max.end());
      TA_CHECK_CUDA(h, cudaMemcpyAsync(h->d_slot_min, init.data(), 2 * n_slots * 8, cudaMemcpyHostToDevice, st));
    }
    TA_CHECK_CUDA(h, cudaMemsetAsync(lane_start, 0xFF, n_codes * sizeof(int32_t), st));
    if (n > 0) {
      if (h->packed) {
        // keys carry the index: 8-byte elements, fewer bytes per pass
        PackInfo pi{h->ibits, h->ibits + h->tbits + (h->sbits - h->dshift), h->wbits, h->d_off};
        PrekeyInfo pre{h->d_off, h->W, h->d_triples->rank_of_slot, h->tbits, h->wbits,
                       h->sbits - h->dshift, h->dshift, h->ibits};
        TA_TRY(ta_radix_sort_keys(h, h->d_keys, kscr, skeys, n, h->plan, h->d_hist, sort_tmp, true,
                                  h->fast_keys ? &pre : nullptr));
        if (n > h->n_valid)
          k_unpack_tail<<<TA_N nblk(n - h->n_valid, 256), 256, 0, st>>>(skeys, h->n_valid, n, pi, perm,
                                                                            h->d_status);
      }
      if (!h->packed) {
        // step 1: (key, input index) pairs; the last pass writes (skeys, perm)
        TA_TRY(ta_radix_sort_pairs(h, h->d_keys, nullptr, kscr, vscr, skeys, perm, n, h->plan,
                                   h->d_hist, sort_tmp));
        // step 2: equal-key runs
        if (h->n_valid > 1)
          k_fix_ties<<<TA_N nblk(h->n_valid, 256), 256, 0, st>>>(skeys, perm, h->n_valid, h->events,
                                                            h->d_status);
        TA_TRY(ta_read_status(h, words));
        if (words[ST_ERR]) return (ta_status)words[ST_ERR];
        if (words[ST_LONG_RUN]) {
          TA_CHECK_CUDA(h, cudaMemsetAsync(h->d_status + ST_LONG_RUN, 0, sizeof(int32_t), st));
          // redo with the duration as a least-significant key: first a stable sort by
          // (max_dur - duration), then the timeline key on top of that order
          void *xb = ta_dalloc(h, Carver::pad(n * 8) + Carver::pad(n * 4));
          if (!xb) return TA_ERR_OOM;
          Carver cx(xb);
          u64 *dkeys = cx.take<u64>(n);
          u32 *dorder = cx.take<u32>(n);
          const u64 dropped_bit = h->has_dropped ? 1ull << (h->sbits + h->tbits + h->wbits) : 0ull;
          k_duration_key<<<TA_N nblk(n, 256), 256, 0, st>>>(h->events, n, h->d_keys, dropped_bit,
                                                       h->max_dur, dkeys);
          int dbits = 1;
          while (dbits < 63 && (h->max_dur >> dbits) != 0) dbits++;
          SortPlan dplan = ta_make_plan(0, dbits);
          TA_TRY(ta_radix_sort_pairs(h, dkeys, nullptr, kscr, vscr, skeys, dorder, n, dplan, nullptr,
                                     sort_tmp));
          k_gather_u64<<<TA_N nblk(n, 256), 256, 0, st>>>(h->d_keys, dorder, n, dkeys, h->d_status);
          TA_TRY(ta_radix_sort_pairs(h, dkeys, dorder, kscr, vscr, skeys, perm, n, h->plan, nullptr,
                                     sort_tmp));
          TA_TRY(ta_sync_fetch(h));
          ta_dfree(h, xb);
        }
      }
      // step 3: dropped tail, chain of stable sorts over the full tuple (least
      // significant field first); perm[n_valid..n) holds the tail in input order
      const int64_t m = n - h->n_valid;
      if (m > 1) {
        void *xb = ta_dalloc(h, 2 * Carver::pad(m * 8) + Carver::pad(m * 4));
        if (!xb) return TA_ERR_OOM;
        Carver cx(xb);
        u64 *tk = cx.take<u64>(m), *tk2 = cx.take<u64>(m);
        u32 *alt = cx.take<u32>(m);
        u32 *cur = perm + h->n_valid, *nxt = alt;
        // packed keys: the first radix pass does not keep equal keys in input order, and all
        // dropped records of a window share one key, so the tail is put in input order first
        for (int stage = h->packed ? -1 : 0; stage < 4; stage++) {
          if (stage == 3 && h->W == 1) break;
          k_tail_key<<<TA_N nblk(m, 256), 256, 0, st>>>(h->events, cur, m, stage, h->d_off, h->W, tk,
                                                        h->d_status);
          int bits = stage == 2 ? 49 : stage == 3 ? (h->wbits > 0 ? h->wbits : 1) : stage < 0 ? 32 : 64;
          SortPlan tp = ta_make_plan(0, bits);
          TA_TRY(ta_radix_sort_pairs(h, tk, cur, kscr, vscr, tk2, nxt, m, tp, nullptr, sort_tmp));
          u32 *t = cur; cur = nxt; nxt = t;
        }
        if (cur != perm + h->n_valid)
          TA_CHECK_CUDA(h, cudaMemcpyAsync(perm + h->n_valid, cur, m * sizeof(u32),
                                           cudaMemcpyDeviceToDevice, st));
        TA_TRY(ta_sync_fetch(h));
        ta_dfree(h, xb);
      }
      // step 4
      GatherArgs g;
      g.ev = h->events; g.perm = perm; g.keys = skeys; g.n = n; g.n_valid = h->n_valid;
      g.packed = h->packed; g.ibits = h->ibits; g.wbits = h->wbits; g.off = h->d_off;
      g.wshift = h->ibits + h->tbits + (h->sbits - h->dshift);
      g.sbits = h->packed ? h->ibits + (h->sbits - h->dshift) : h->sbits;
      g.ts_start = c_ts; g.ts_end = c_te; g.corr = c_corr; g.pid = c_pid; g.name = c_name; g.seq = c_seq;
      g.stream = c_stream; g.kind = c_kind; g.lane_start = lane_start;
      g.tt = h->d_triples; g.tbits = h->tbits; g.n_pids = h->n_pids > 0 ? h->n_pids : 1;
      g.slot_min = h->d_slot_min; g.slot_max = h->d_slot_max; g.status = h->d_status;
      k_gather<<<TA_N nblk(n, 256), 256, 0, st>>>(g);
    }
    k_lane_table<<<TA_N 1, 1024, 0, st>>>(lane_start, n_codes, h->tbits,
                                     h->n_pids > 0 ? h->n_pids : 1, h->d_triples, h->n_valid,
                                     lane_window, lane_pid, lane_stream, lane_domain, lane_off,
                                     lane_code, lane_slot, lane_dom_end, lane_dom_next, lane_dev_base, n_lanes_dev,
                                     lane_cap, h->d_status);
    TA_CHECK_CUDA(h, cudaGetLastError());
    TA_TRY(ta_queue_d2h(h, n_lanes_host, n_lanes_dev, 2 * sizeof(int32_t)));
    TA_TRY(ta_queue_d2h(h, h->h_slot_min.data(), h->d_slot_min, n_slots * 8));
    TA_TRY(ta_queue_d2h(h, h->h_slot_max.data(), h->d_slot_max, n_slots * 8));
    TA_TRY(ta_read_status(h, words));
    if (words[ST_ERR]) return (ta_status)words[ST_ERR];
    if (!words[ST_LONG_RUN]) break;
    if (!h->packed) return TA_ERR_OVERFLOW;  // cannot happen: the pair path resolves long runs itself
    TA_CHECK_CUDA(h, cudaMemsetAsync(h->d_status + ST_LONG_RUN, 0, sizeof(int32_t), st));
    TA_TRY(ta_launch_load(h, false));
  }
  ta_dfree(h, tb);
  ta_dfree(h, h->d_keys);
  h->d_keys = nullptr;

  const int32_t n_lanes = n_lanes_host[0];
  h->n_device = n_lanes_host[1];
  ta_sort_result &r = h->sorted;
  r.n = n; r.n_valid = h->n_valid; r.n_lanes = n_lanes; r.n_windows = h->W;
  r.perm = (const int32_t *)perm;
  r.ts_start = (const int64_t *)c_ts; r.ts_end = (const int64_t *)c_te;
  r.corr_id = (const int64_t *)c_corr;
  r.pid = c_pid; r.name_id = c_name; r.seq = c_seq; r.stream = c_stream; r.kind = c_kind;
  r.lane_window = lane_window; r.lane_pid = lane_pid; r.lane_stream = lane_stream;
  r.lane_domain = lane_domain; r.lane_off = lane_off;
  h->d_lane_code = lane_code;
  h->d_lane_slot = lane_slot;
  h->d_lane_dom_end = lane_dom_end;
  h->d_lane_dev_base = lane_dev_base;
  h->d_lane_dom_next = lane_dom_next;
  return TA_OK;
}
