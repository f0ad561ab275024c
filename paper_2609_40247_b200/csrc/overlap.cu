// ta_device_overlap: per (window, process), over ALL device streams, the time the
// device was busy, the time covered by computation (KERNEL) and by communication /
// IO (MEMCPY, COLL), how much of the communication was hidden under computation and
// how much stayed exposed, all as measures of unions of intervals (Sec. 6.1, "Execution
// progress and state"; Fig. "Overlap and exposed work").
//
// The measure of a union of intervals taken in start order is
//   sum_i max(0, e_i - max(s_i, P_i)),   P_i = max of the ends seen before i,
// the same recurrence as the per-stream gap scan, so the step is: take the device
// records of every process out of their stream lanes, sort them by (window, process,
// ts_start) - keys that carry the record's index in their low bits when (process slot, time,
// index) fit 64 bits, (key, index) pairs otherwise - and run ONE chained max-scan with three channels
// (all records, computation, communication).  The measure of the intersection follows
// from the three unions: |A n B| = |A| + |B| - |A u B|.  Scanned values are tagged with
// the (window, process) slot in their upper bits, as in the gap scan, so a prefix that
// belongs to an earlier process is recognised and ignored.
// HBM-bound on the sort: 8 B + 8 B (keys) or 12 B + 12 B (pairs) per device record and pass.
#include <climits>
#include <cstring>

#include "scan.cuh"
#include "ta_internal.cuh"

#define OV_THREADS 256
#define OV_ITEMS 8
#define OV_TILE (OV_THREADS * OV_ITEMS)
#define OV_LOW ((1ull << 40) - 1)

struct OvKeyArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int64_t *ts;
  const int32_t *lane_off, *lane_slot, *lane_window, *lane_dom_end, *lane_dev_base;
  const int16_t *lane_domain;
  const int64_t *t0;
  int tsbits, idxbits;
  u64 *keys;  // [device record index] ((slot << tsbits) | (ts_start - t0)) << idxbits | index
  u32 *pos;   // [device record index] sorted position
  const int32_t *status;
};

// one tile of 2048 sorted positions per CTA; tiles that hold host lanes only leave at once
__global__ void __launch_bounds__(OV_THREADS) k_ov_keys(OvKeyArgs a) {
  __shared__ int s_lane0;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x;
  const int64_t tile_start = (int64_t)blockIdx.x * OV_TILE;
  if (tile_start >= a.n_valid) return;
  if (tid < 32) {
    const int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (tid == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  const int64_t tile_end = min(tile_start + OV_TILE, a.n_valid);
  if (span_outside_domain(a.lane_domain, a.lane_dom_end, l0, tile_end, 1)) return;
  const int64_t p0 = tile_start + (int64_t)tid * OV_ITEMS;
  if (p0 >= tile_end) return;
  i64 s[OV_ITEMS];
  load8_i64(a.ts, p0, a.n, s);
  int l = l0;
  int64_t cur_off = a.lane_off[l], next_off = a.lane_off[l + 1];
  bool dev = a.lane_domain[l] == 1;
  int slot = a.lane_slot[l];
  i64 w0 = a.t0[a.lane_window[l]];
  int64_t cbase = a.lane_dev_base[l];
#pragma unroll
  for (int j = 0; j < OV_ITEMS; j++) {
    const int64_t p = p0 + j;
    if (p >= tile_end) break;
    while (p >= next_off) {
      l++;
      cur_off = next_off;
      next_off = a.lane_off[l + 1];
      dev = a.lane_domain[l] == 1;
      slot = a.lane_slot[l];
      w0 = a.t0[a.lane_window[l]];
      cbase = a.lane_dev_base[l];
    }
    if (!dev) continue;
    const int64_t c = cbase + (p - cur_off);
    a.keys[c] = ((((u64)slot << a.tsbits) | (u64)(s[j] - w0)) << a.idxbits) |
                (a.idxbits ? (u64)c : 0ull);
    a.pos[c] = (u32)p;
  }
}

struct OvScanArgs {
  int64_t m;          // device records
  const u64 *keys;    // sorted
  const u32 *pos;     // sorted position: of element i (pairs), or of device record index c (packed keys)
  int idxbits;        // packed keys: low bits hold the device record index; 0 = pairs
  const int64_t *te;
  const int16_t *kind;
  const int64_t *t0, *t1;
  int tsbits, n_pids;
  u64 *st[3];         // tile descriptors of the three channels
  u32 *counter;
  u64 *acc;           // [slot][4]: records, busy, compute, communication
  int32_t *status;
};

__global__ void __launch_bounds__(OV_THREADS, 3) k_ov_scan(OvScanArgs a) {
  __shared__ u64 tmp[3][33];
  __shared__ u64 s_excl[3];
  __shared__ int s_tile, s_fail;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_tile = (int)atomicAdd(a.counter, 1u);
    s_fail = ta_failed(a.status) ? 1 : 0;
  }
  __syncthreads();
  if (s_fail) return;  // the sort gave up: the keys name no records
  const int tile = s_tile;
  const int64_t i0 = (int64_t)tile * OV_TILE + (int64_t)tid * OV_ITEMS;
  // keys and positions of the thread's eight records, then the gathers, all issued together
  u64 key[OV_ITEMS];
  u32 pp[OV_ITEMS];
  i64 en[OV_ITEMS];
  int16_t kd[OV_ITEMS];
#pragma unroll
  for (int j = 0; j < OV_ITEMS; j++) {
    const bool in = i0 + j < a.m;
    key[j] = in ? a.keys[i0 + j] : ~0ull;
    if (a.idxbits) {
      pp[j] = in ? a.pos[key[j] & ((1ull << a.idxbits) - 1)] : 0u;
      key[j] >>= a.idxbits;
    } else {
      pp[j] = in ? a.pos[i0 + j] : 0u;
    }
  }
#pragma unroll
  for (int j = 0; j < OV_ITEMS; j++) {
    const bool in = i0 + j < a.m;
    en[j] = in ? a.te[pp[j]] : 0;
    kd[j] = in ? a.kind[pp[j]] : (int16_t)-1;
  }
  const u64 tsmask = (1ull << a.tsbits) - 1;
  u64 val[OV_ITEMS];   // (slot + 1) << 40 | clipped end - window start
  i64 srel[OV_ITEMS];  // ts_start - window start
  int slot_of[OV_ITEMS];
  u64 run[3] = {0, 0, 0};
  {
    int wl = -1;
    i64 w0 = 0, w1 = 0;
#pragma unroll
    for (int j = 0; j < OV_ITEMS; j++) {
      val[j] = 0;
      srel[j] = 0;
      slot_of[j] = -1;
      if (kd[j] < 0) continue;
      const int slot = (int)(key[j] >> a.tsbits);
      const int w = slot / a.n_pids;
      if (w != wl) { w0 = a.t0[w]; w1 = a.t1[w]; wl = w; }
      const i64 ce = (en[j] < w1 ? en[j] : w1) - w0;
      slot_of[j] = slot;
      srel[j] = (i64)(key[j] & tsmask);
      val[j] = ((u64)(slot + 1) << 40) | (u64)ce;
      run[0] = max(run[0], val[j]);
      const int ch = kd[j] == TA_KIND_KERNEL ? 1 : 2;
      run[ch] = max(run[ch], val[j]);
    }
  }
  u64 pre[3];
#pragma unroll
  for (int ch = 0; ch < 3; ch++) {
    u64 total;
    pre[ch] = block_scan_exclusive<OpMax>(run[ch], OpMax(), tmp[ch], &total);
    if (warp == ch) {  // three warps look back at the same time, one channel each
      bool failed;
      const u64 ex = tile_lookback<OpMax>(a.st[ch], tile, total, OpMax(), a.status, &failed);
      if (lane == 0) s_excl[ch] = ex;
      if (lane == 0 && failed) s_fail = 1;
    }
  }
  __syncthreads();
  if (s_fail) return;
#pragma unroll
  for (int ch = 0; ch < 3; ch++) pre[ch] = max(pre[ch], s_excl[ch]);

  // coverage added by each record; sums of the thread's first slot stay in registers
  u64 sum[4] = {0, 0, 0, 0};
  int first = -1;
#pragma unroll
  for (int j = 0; j < OV_ITEMS; j++) {
    const int slot = slot_of[j];
    if (slot < 0) continue;
    const i64 ce = (i64)(val[j] & OV_LOW);
    const int ch = kd[j] == TA_KIND_KERNEL ? 1 : 2;
    u64 add[4] = {1, 0, 0, 0};
#pragma unroll
    for (int c = 0; c < 3; c++) {
      if (c != 0 && c != ch) continue;
      const i64 P = ((pre[c] >> 40) == (u64)(slot + 1)) ? (i64)(pre[c] & OV_LOW) : 0;
      const i64 from = srel[j] > P ? srel[j] : P;
      add[1 + c] = ce > from ? (u64)(ce - from) : 0ull;
      pre[c] = max(pre[c], val[j]);
    }
    if (first < 0) first = slot;
    if (slot == first) {
#pragma unroll
      for (int c = 0; c < 4; c++) sum[c] += add[c];
    } else {  // the thread straddles two processes
#pragma unroll
      for (int c = 0; c < 4; c++)
        if (add[c]) atomicAdd(&a.acc[(size_t)slot * 4 + c], add[c]);
    }
  }
  // fold per warp when the warp sits inside one process (almost always)
  const u32 has = __ballot_sync(0xffffffffu, first >= 0);
  if (!has) return;
  const int wfirst = __shfl_sync(0xffffffffu, first, __ffs(has) - 1);
  if (__all_sync(0xffffffffu, first < 0 || first == wfirst)) {
#pragma unroll
    for (int c = 0; c < 4; c++) {
      const u64 t = warp_reduce(sum[c], OpAdd());
      if (lane == 0 && t) atomicAdd(&a.acc[(size_t)wfirst * 4 + c], t);
    }
  } else if (first >= 0) {
#pragma unroll
    for (int c = 0; c < 4; c++)
      if (sum[c]) atomicAdd(&a.acc[(size_t)first * 4 + c], sum[c]);
  }
}

// compaction of the (window, process) slots that have device records, in slot order
struct OvRowIn {
  const u64 *acc;
  __device__ u64 operator()(int64_t s) const { return acc[(size_t)s * 4] ? 1ull : 0ull; }
};
struct OvRowOut {
  const u64 *acc;
  const TripleTable *tt;
  const int64_t *t0, *t1;
  int n_pids;
  int32_t *d_window, *d_pid;
  int64_t *d_n_events, *d_busy, *d_idle, *d_compute, *d_comm, *d_overlap, *d_exposed;
  __device__ void operator()(int64_t s, u64 row, u64 v) const {
    if (!v) return;
    const int w = (int)(s / n_pids);
    const i64 all = (i64)acc[(size_t)s * 4 + 1], comp = (i64)acc[(size_t)s * 4 + 2],
              comm = (i64)acc[(size_t)s * 4 + 3];
    d_window[row] = w;
    d_pid[row] = tt->pid_value[s % n_pids];
    d_n_events[row] = (i64)acc[(size_t)s * 4];
    d_busy[row] = all;
    d_idle[row] = (t1[w] - t0[w]) - all;
    d_compute[row] = comp;
    d_comm[row] = comm;
    d_overlap[row] = comp + comm - all;
    d_exposed[row] = all - comp;
  }
};

ta_status ta_run_overlap(ta_window *h, ta_overlap_result *out) {
  cudaStream_t st = h->stream;
  memset(out, 0, sizeof(*out));
  const int n_pids = h->n_pids > 0 ? h->n_pids : 1;
  const int64_t n_slots = (int64_t)h->W * n_pids;
  const int64_t m = h->n_device;
  if (m <= 0 || h->n_valid <= 0) return TA_OK;
  int64_t max_span = 1;
  for (int w = 0; w < h->W; w++) max_span = h->h_t1[w] - h->h_t0[w] > max_span ? h->h_t1[w] - h->h_t0[w] : max_span;
  const int tsbits = ta_bit_len((uint64_t)max_span);
  const int slot_bits = ta_bit_len((uint64_t)(n_slots - 1));
  if (tsbits > 40 || tsbits + slot_bits > 63 || n_slots >= (1ll << 22)) return TA_ERR_TOO_LARGE;
  // when (slot, time, index) fit one 64-bit word the index travels inside the key and the
  // passes move keys only (8 B + 8 B per record instead of 12 B + 12 B)
  int idxbits = ta_bit_len((uint64_t)(m - 1));
  if (idxbits < 1) idxbits = 1;
  if (tsbits + slot_bits + idxbits > 64) idxbits = 0;

  // results (kept): at most one row per slot
  size_t kb = 2 * Carver::pad((size_t)n_slots * 4) + 7 * Carver::pad((size_t)n_slots * 8) + 256;
  void *keep = ta_dalloc(h, kb);
  if (!keep) return TA_ERR_OOM;
  Carver ck(keep);
  OvRowOut ro;
  ro.d_window = ck.take<int32_t>(n_slots); ro.d_pid = ck.take<int32_t>(n_slots);
  ro.d_n_events = ck.take<int64_t>(n_slots); ro.d_busy = ck.take<int64_t>(n_slots);
  ro.d_idle = ck.take<int64_t>(n_slots); ro.d_compute = ck.take<int64_t>(n_slots);
  ro.d_comm = ck.take<int64_t>(n_slots); ro.d_overlap = ck.take<int64_t>(n_slots);
  ro.d_exposed = ck.take<int64_t>(n_slots);

  const int64_t tiles = (m + OV_TILE - 1) / OV_TILE;
  size_t tb = 3 * Carver::pad((size_t)m * 8) + 3 * Carver::pad((size_t)m * 4) + ta_sort_temp_bytes(m) +
              3 * Carver::pad((size_t)tiles * 8) + Carver::pad(64) + Carver::pad((size_t)n_slots * 32) +
              scan_temp_bytes(n_slots) + 512;
  void *tmpb = ta_dalloc(h, tb);
  if (!tmpb) return TA_ERR_OOM;
  Carver ct(tmpb);
  u64 *k_in = ct.take<u64>(m), *k_scr = ct.take<u64>(m), *k_fin = ct.take<u64>(m);
  u32 *v_in = ct.take<u32>(m), *v_scr = ct.take<u32>(m), *v_fin = ct.take<u32>(m);
  char *zb = ct.base + ct.off;
  OvScanArgs sa;
  for (int c = 0; c < 3; c++) sa.st[c] = ct.take<u64>(tiles);
  sa.counter = (u32 *)ct.take<u64>(8);
  sa.acc = ct.take<u64>(n_slots * 4);
  TA_CHECK_CUDA(h, cudaMemsetAsync(zb, 0, (ct.base + ct.off) - zb, st));
  void *sort_tmp = ct.base + ct.off; ct.off += ta_sort_temp_bytes(m);
  void *scan_mem = ct.base + ct.off;

  OvKeyArgs ka;
  ka.n = h->n; ka.n_valid = h->n_valid; ka.n_lanes = h->sorted.n_lanes;
  ka.ts = h->sorted.ts_start;
  ka.lane_off = h->sorted.lane_off; ka.lane_slot = h->d_lane_slot; ka.lane_window = h->sorted.lane_window;
  ka.lane_dom_end = h->d_lane_dom_end; ka.lane_dev_base = h->d_lane_dev_base;
  ka.lane_domain = h->sorted.lane_domain; ka.t0 = h->d_t0; ka.tsbits = tsbits; ka.idxbits = idxbits;
  ka.keys = k_in; ka.pos = v_in; ka.status = h->d_status;
  const int64_t key_tiles = (h->n_valid + OV_TILE - 1) / OV_TILE;
  k_ov_keys<<<TA_N (unsigned)key_tiles, OV_THREADS, 0, st>>>(ka);
  TA_CHECK_CUDA(h, cudaGetLastError());
  if (idxbits) {
    TA_TRY(ta_radix_sort_keys(h, k_in, k_scr, k_fin, m,
                              ta_make_plan(idxbits, idxbits + tsbits + slot_bits), nullptr, sort_tmp,
                              true));  // coverage sums do not depend on the order of equal starts
    sa.pos = v_in;
  } else {
    TA_TRY(ta_radix_sort_pairs(h, k_in, v_in, k_scr, v_scr, k_fin, v_fin, m,
                               ta_make_plan(0, tsbits + slot_bits), nullptr, sort_tmp));
    sa.pos = v_fin;
  }
  sa.m = m; sa.keys = k_fin; sa.idxbits = idxbits;
  sa.te = h->sorted.ts_end; sa.kind = h->sorted.kind; sa.t0 = h->d_t0; sa.t1 = h->d_t1;
  sa.tsbits = tsbits; sa.n_pids = n_pids; sa.status = h->d_status;
  k_ov_scan<<<TA_N (unsigned)tiles, OV_THREADS, 0, st>>>(sa);
  TA_CHECK_CUDA(h, cudaGetLastError());

  ro.acc = sa.acc; ro.tt = h->d_triples; ro.t0 = h->d_t0; ro.t1 = h->d_t1; ro.n_pids = n_pids;
  ScanTemp s3;
  TA_TRY(scan_temp_init(h, scan_mem, n_slots, &s3));
  OvRowIn ri{sa.acc};
  TA_TRY((launch_scan<OpAdd, OvRowIn, OvRowOut>(h, n_slots, ri, ro, OpAdd(), s3)));
  u64 rows = 0;
  TA_TRY(ta_queue_d2h(h, &rows, s3.total, 8));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  ta_dfree(h, tmpb);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  out->n_rows = (int64_t)rows;
  out->d_window = ro.d_window; out->d_pid = ro.d_pid; out->d_n_events = ro.d_n_events;
  out->d_busy = ro.d_busy; out->d_idle = ro.d_idle; out->d_compute = ro.d_compute;
  out->d_comm = ro.d_comm; out->d_overlap = ro.d_overlap; out->d_exposed = ro.d_exposed;
  return TA_OK;
}
