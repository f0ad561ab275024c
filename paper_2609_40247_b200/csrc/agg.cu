// ta_aggregate_ops: per (window, pid, name_id) count / sum / min / max and a log2
// histogram of a value column (own duration, T_op of operators with kernels, or the
// idle time charged to an operator by the gap blame).
// Per-symbol counts and duration statistics are what Sec. 8.1 compares.
//
// Symbol popularity is heavy-tailed (a few names carry most records), so global
// atomics alone would serialise on the hot rows.  Each CTA takes 16384
// consecutive sorted positions (one process, mostly; CTAs whose lanes cannot
// hold a selected kind return at once) and folds its records into a
// shared-memory hash table first; the table is flushed to a dense global table
// indexed by (window, pid rank, name_id - min name) with one atomic per field.
// A scan then compacts the non-empty rows in key order.  Symbol ids spread too wide
// for a dense table take the sort-based path at the end of this file instead.
// HBM-bound on the column reads: 2 B (kind) for every record, 24 B more for the
// selected ones.
#include <climits>
#include <cstring>
#include <vector>

#include "records.cuh"
#include "scan.cuh"
#include "ta_internal.cuh"

#define AG_THREADS 256
#define AG_ITEMS 4
#define AG_STEP (AG_THREADS * AG_ITEMS)
#define AG_SLOTS 256
#define AG_ITEM (16 * AG_STEP)   // positions per CTA
#define AG_FLUSH_EVERY 32768  // records per CTA between flushes (keeps 16-bit bins safe)

struct AggArgs {
  int64_t n_valid;
  int n_lanes;
  const int16_t *kind;
  const int32_t *name;
  const int64_t *ts, *te;
  const int32_t *lane_off, *lane_slot;
  const int32_t *op_n;
  const int64_t *op_first, *op_last;
  const int64_t *op_gap;  // value_sel 2
  const uint8_t *on_path; // value_sel 3
  uint32_t kind_mask;
  int value_sel;
  int64_t min_name, R;
  const int16_t *lane_domain;
  const int32_t *lane_dom_end;
  int want_domain;  // 0 / 1: the selected kinds all live in lanes of this domain; -1: both
  int64_t chunk;    // positions per CTA, a multiple of AG_STEP
  unsigned n_items, spread, per;
  // dense table (all zero-initialised; min is kept as the complement of the biased value)
  u64 *d_cnt, *d_sum, *d_minc, *d_maxb;
  u32 *d_hist;
  u64 *n_groups;
  const int32_t *status;
};

struct AggSmem {
  int32_t key[AG_SLOTS];
  u32 cnt[AG_SLOTS];
  u32 sum16[3][AG_SLOTS];  // the sum in 16-bit limbs: native 32-bit shared-memory atomics only
  u64 minc[AG_SLOTS];
  u64 maxb[AG_SLOTS];
  uint16_t hist[AG_SLOTS][TA_NBINS];
};

__device__ __forceinline__ void agg_global_add(const AggArgs &a, int64_t g, u64 cnt, u64 sum, u64 minc,
                                               u64 maxb) {
  // none of the results is used: the adds go out without the thread waiting for them
  atomicAdd(&a.d_cnt[g], cnt);
  atomicAdd(&a.d_sum[g], sum);
  atomicMax(&a.d_minc[g], minc);
  atomicMax(&a.d_maxb[g], maxb);
}

__device__ __forceinline__ void agg_clear(AggSmem &s) {
  for (int i = threadIdx.x; i < AG_SLOTS; i += AG_THREADS) {
    s.key[i] = -1;
    s.cnt[i] = 0;
    s.sum16[0][i] = s.sum16[1][i] = s.sum16[2][i] = 0;
    s.minc[i] = 0;
    s.maxb[i] = 0;
  }
  u32 *hw = reinterpret_cast<u32 *>(&s.hist[0][0]);
  for (int i = threadIdx.x; i < AG_SLOTS * TA_NBINS / 2; i += AG_THREADS) hw[i] = 0;
}

__device__ __forceinline__ void agg_flush(const AggArgs &a, AggSmem &s) {
  __syncthreads();
  for (int i = threadIdx.x; i < AG_SLOTS; i += AG_THREADS) {
    int32_t k = s.key[i];
    if (k >= 0)
      agg_global_add(a, k, s.cnt[i],
                     (u64)s.sum16[0][i] + ((u64)s.sum16[1][i] << 16) + ((u64)s.sum16[2][i] << 32),
                     s.minc[i], s.maxb[i]);
  }
  // histogram bins: one thread per (slot, bin)
  for (int i = threadIdx.x; i < AG_SLOTS * TA_NBINS; i += AG_THREADS) {
    const int sl = i / TA_NBINS, b = i - sl * TA_NBINS;
    const u32 c = s.hist[sl][b];
    if (c) atomicAdd(&a.d_hist[(size_t)s.key[sl] * TA_NBINS + b], c);
  }
  __syncthreads();
  agg_clear(s);
  __syncthreads();
}

__global__ void __launch_bounds__(AG_THREADS, 6) k_agg(AggArgs a) {
  __shared__ AggSmem s;
  if (ta_failed(a.status)) return;
  int since_flush = 0;
  LaneWalker lw(a.lane_off, a.n_lanes, a.n_valid, a.n_valid);
  {
    // CTA b -> chunk (b mod G) * S + b / G: CTAs that run together work far apart in the
    // timeline (different processes), so their flushes rarely meet on the same global rows;
    // chunks whose lanes cannot hold a selected kind return at once and make room
    const unsigned item = (blockIdx.x % a.spread) * a.per + blockIdx.x / a.spread;
    if (item >= a.n_items) return;
    const int64_t begin = (int64_t)item * a.chunk;
    const int64_t end = min(begin + a.chunk, a.n_valid);
    int bl = lane_of_pos(a.lane_off, a.n_lanes, begin);  // lane of `base`, the same in every thread
    if (a.want_domain >= 0 &&
        span_outside_domain(a.lane_domain, a.lane_dom_end, bl, end, a.want_domain))
      return;
    agg_clear(s);
    __syncthreads();
    for (int64_t base = begin; base < end; base += AG_STEP) {
      while (bl + 1 < a.n_lanes && (int64_t)a.lane_off[bl + 1] <= base) bl++;
      if (a.want_domain >= 0 && span_outside_domain(a.lane_domain, a.lane_dom_end, bl,
                                                    min(base + AG_STEP, end), a.want_domain))
        continue;
      lw.lane = bl;
      const int64_t p0 = base + (int64_t)threadIdx.x * AG_ITEMS;
      // all loads of the thread's four records are issued before any of them is used; for the
      // plain duration the times and names are requested with the kinds, not after them (the
      // step holds lanes of the wanted domain, so most records are selected anyway)
      int16_t kd[AG_ITEMS];
      i64 pre_v[AG_ITEMS];
      int32_t pre_nm[AG_ITEMS];
#pragma unroll
      for (int j = 0; j < AG_ITEMS; j++) { pre_v[j] = 0; pre_nm[j] = 0; }
      if (p0 + AG_ITEMS <= end) {
        uint2 q = *reinterpret_cast<const uint2 *>(a.kind + p0);
        if (a.value_sel == 0) {
          const longlong2 *ps = reinterpret_cast<const longlong2 *>(a.ts + p0);
          const longlong2 *pe = reinterpret_cast<const longlong2 *>(a.te + p0);
          const int4 nq = *reinterpret_cast<const int4 *>(a.name + p0);
#pragma unroll
          for (int h2 = 0; h2 < AG_ITEMS / 2; h2++) {
            const longlong2 x = ps[h2], y = pe[h2];
            pre_v[2 * h2] = y.x - x.x;
            pre_v[2 * h2 + 1] = y.y - x.y;
          }
          pre_nm[0] = nq.x; pre_nm[1] = nq.y; pre_nm[2] = nq.z; pre_nm[3] = nq.w;
        } else if (a.value_sel == 1) {  // the kernel counts with the kinds (pre_nm holds them)
          const int4 cq = *reinterpret_cast<const int4 *>(a.op_n + p0);
          pre_nm[0] = cq.x; pre_nm[1] = cq.y; pre_nm[2] = cq.z; pre_nm[3] = cq.w;
        }
        const int16_t *hq = reinterpret_cast<const int16_t *>(&q);
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++) kd[j] = hq[j];
      } else {
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++) {
          kd[j] = p0 + j < end ? a.kind[p0 + j] : (int16_t)-1;
          if (a.value_sel == 0 && p0 + j < end) { pre_v[j] = a.te[p0 + j] - a.ts[p0 + j]; pre_nm[j] = a.name[p0 + j]; }
          if (a.value_sel == 1 && p0 + j < end) pre_nm[j] = a.op_n[p0 + j];
        }
      }
      bool sel[AG_ITEMS];
      i64 v[AG_ITEMS];
      int32_t nm[AG_ITEMS];
#pragma unroll
      for (int j = 0; j < AG_ITEMS; j++) {
        sel[j] = kd[j] >= 0 && ((a.kind_mask >> kd[j]) & 1u);
        v[j] = 0;
        nm[j] = 0;
      }
      if (a.value_sel == 0) {
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) { v[j] = pre_v[j]; nm[j] = pre_nm[j]; }
      } else if (a.value_sel == 1) {
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) sel[j] = pre_nm[j] > 0;
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) { v[j] = a.op_last[p0 + j] - a.op_first[p0 + j]; nm[j] = a.name[p0 + j]; }
      } else if (a.value_sel == 2) {
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) { v[j] = a.op_gap[p0 + j]; sel[j] = v[j] > 0; }
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) nm[j] = a.name[p0 + j];
      } else {
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) sel[j] = a.on_path[p0 + j] != 0;
#pragma unroll
        for (int j = 0; j < AG_ITEMS; j++)
          if (sel[j]) { v[j] = a.te[p0 + j] - a.ts[p0 + j]; nm[j] = a.name[p0 + j]; }
      }
#pragma unroll
      for (int j = 0; j < AG_ITEMS; j++) {
        if (!sel[j]) continue;
        const int lane = lw.at(p0 + j);
        const int64_t g = (int64_t)a.lane_slot[lane] * a.R + ((int64_t)nm[j] - a.min_name);
        const u64 vb = (u64)v[j] ^ (1ull << 63);
        const int bin = log2_bin(v[j]);
        u32 hsh = (u32)g * 2654435761u;
        int slot = (int)(hsh >> 24) & (AG_SLOTS - 1);
        bool placed = false;
        for (int probe = 0; probe < 8; probe++) {
          int32_t cur = s.key[slot];
          if (cur == (int32_t)g) { placed = true; break; }
          if (cur == -1) {
            int32_t old = atomicCAS(&s.key[slot], -1, (int32_t)g);
            if (old == -1 || old == (int32_t)g) { placed = true; break; }
          }
          slot = (slot + 1) & (AG_SLOTS - 1);
        }
        if (placed) {
          atomicAdd(&s.cnt[slot], 1u);
          {  // values are durations (>= 0): 16 + 16 + 32 bit limbs, at most 32768 adds per flush
            const u64 uv = (u64)v[j];
            atomicAdd(&s.sum16[0][slot], (u32)(uv & 0xFFFF));
            if (uv >> 16) atomicAdd(&s.sum16[1][slot], (u32)((uv >> 16) & 0xFFFF));
            if (uv >> 32) atomicAdd(&s.sum16[2][slot], (u32)(uv >> 32));
          }
          // 64-bit min/max in shared memory are compare-and-swap loops: skip them unless the
          // value would actually move the extreme (rare once a slot has seen a few records)
          if (~vb > s.minc[slot]) atomicMax(&s.minc[slot], ~vb);
          if (vb > s.maxb[slot]) atomicMax(&s.maxb[slot], vb);
          // 16-bit bins packed two per word
          u32 *hw = reinterpret_cast<u32 *>(&s.hist[slot][0]) + (bin >> 1);
          atomicAdd(hw, (bin & 1) ? 0x10000u : 1u);
        } else {
          agg_global_add(a, g, 1, (u64)v[j], ~vb, vb);
          atomicAdd(&a.d_hist[(size_t)g * TA_NBINS + bin], 1u);
        }
      }
      since_flush += AG_STEP;
      if (since_flush >= AG_FLUSH_EVERY) {
        agg_flush(a, s);
        since_flush = 0;
      }
    }
  }
  agg_flush(a, s);
}

// number of non-empty rows (only needed up front when the output cannot be sized by a bound)
__global__ void __launch_bounds__(256) k_agg_count_rows(const u64 *cnt, int64_t G, u64 *n_rows) {
  u64 c = 0;
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < G; g += (int64_t)gridDim.x * blockDim.x)
    c += cnt[g] ? 1ull : 0ull;
  c = warp_reduce(c, OpAdd());
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(n_rows, c);
}

// compaction of the non-empty rows in dense (= key) order
struct AggRowIn {
  const u64 *cnt;
  __device__ u64 operator()(int64_t g) const { return cnt[g] ? 1ull : 0ull; }
};
struct AggRowOut {
  const u64 *cnt, *sum, *minc, *maxb;
  const u32 *hist;
  const TripleTable *tt;
  int n_pids;
  int64_t R, min_name;
  int32_t *g_window, *g_pid, *g_name;
  int64_t *g_count, *g_sum, *g_min, *g_max;
  u32 *g_hist;
  __device__ void operator()(int64_t g, u64 row, u64 v) const {
    if (!v) return;
    int64_t slot = g / R;
    g_window[row] = (int32_t)(slot / n_pids);
    g_pid[row] = tt->pid_value[slot % n_pids];
    g_name[row] = (int32_t)(min_name + g % R);
    g_count[row] = (int64_t)cnt[g];
    g_sum[row] = (int64_t)sum[g];
    g_min[row] = (int64_t)((~minc[g]) ^ (1ull << 63));
    g_max[row] = (int64_t)(maxb[g] ^ (1ull << 63));
    // the 40 bins as ten 16-byte loads issued together, then ten stores (rows are 160 B apart,
    // both tables 16-byte aligned)
    const uint4 *src = reinterpret_cast<const uint4 *>(hist + (size_t)g * TA_NBINS);
    uint4 *dst = reinterpret_cast<uint4 *>(g_hist + row * TA_NBINS);
    uint4 q[TA_NBINS / 4];
#pragma unroll
    for (int b = 0; b < TA_NBINS / 4; b++) q[b] = src[b];
#pragma unroll
    for (int b = 0; b < TA_NBINS / 4; b++) dst[b] = q[b];
  }
};

// ---- symbol ids too spread out for the dense table: aggregate by sorting ---------------
// The selected records are compacted to (key, position) pairs with key = (window, pid) slot
// << 32 | name_id (order-preserving code), sorted with the pair sorter, cut into groups where
// the key changes, and reduced with atomics on the group rows - one per run of equal keys
// inside a thread's eight consecutive elements, so a popular symbol costs an eighth of its
// records in atomics.  Rows come out in key order, as from the dense path.
struct AggSortCtx {
  int64_t n_valid;
  int n_lanes, n_pids;
  uint32_t kind_mask;
  int value_sel;
  const int16_t *kind;
  const int32_t *name;
  const int64_t *ts, *te;
  const int32_t *op_n;
  const int64_t *op_first, *op_last, *op_gap;
  const uint8_t *on_path;
  const int32_t *lane_off, *lane_slot;
  const TripleTable *tt;
  const int32_t *status;
};
__device__ __forceinline__ bool agg_selected(const AggSortCtx &c, int64_t p, i64 *v) {
  const int k = c.kind[p];
  if (k < 0 || k > 5 || !((c.kind_mask >> k) & 1u)) return false;
  if (c.value_sel == 0) { *v = c.te[p] - c.ts[p]; return true; }
  if (c.value_sel == 1) {
    if (c.op_n[p] <= 0) return false;
    *v = c.op_last[p] - c.op_first[p];
    return true;
  }
  if (c.value_sel == 2) {
    *v = c.op_gap[p];
    return *v > 0;
  }
  if (!c.on_path[p]) return false;
  *v = c.te[p] - c.ts[p];
  return true;
}
struct AggSelIn {
  AggSortCtx c;
  __device__ u64 operator()(int64_t p) const {
    i64 v;
    return agg_selected(c, p, &v) ? 1ull : 0ull;
  }
};
struct AggSelOut {
  AggSortCtx c;
  u64 *keys;
  u32 *pos;
  __device__ void operator()(int64_t p, u64 excl, u64 v) const {
    if (!v) return;
    const int lane = lane_of_pos(c.lane_off, c.n_lanes, p);
    keys[excl] = ((u64)c.lane_slot[lane] << 32) | (u64)((u32)c.name[p] ^ 0x80000000u);
    pos[excl] = (u32)p;
  }
};
struct AggHeadIn {
  const u64 *ks;
  __device__ u64 operator()(int64_t j) const { return (j == 0 || ks[j] != ks[j - 1]) ? 1ull : 0ull; }
};
struct AggHeadOut {
  int32_t *gid;     // per sorted element
  int32_t *gstart;  // per group
  __device__ void operator()(int64_t j, u64 excl, u64 v) const {
    const int32_t g = (int32_t)(excl + v) - 1;
    gid[j] = g;
    if (v) gstart[g] = (int32_t)j;
  }
};
struct AggSortedOut {
  int32_t *g_window, *g_pid, *g_name;
  int64_t *g_count, *g_sum, *g_min, *g_max;
  u32 *g_hist;
};
__global__ void __launch_bounds__(256) k_agg_sorted_rows(AggSortCtx c, const u64 *ks, const int32_t *gstart,
                                                        int64_t ng, AggSortedOut o) {
  if (ta_failed(c.status)) return;
  const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= ng) return;
  const u64 key = ks[gstart[g]];
  const int64_t slot = (int64_t)(key >> 32);
  o.g_window[g] = (int32_t)(slot / c.n_pids);
  o.g_pid[g] = c.tt->pid_value[slot % c.n_pids];
  o.g_name[g] = (int32_t)((u32)key ^ 0x80000000u);
  o.g_min[g] = INT64_MAX;
  o.g_max[g] = INT64_MIN;
}
__global__ void __launch_bounds__(256) k_agg_sorted_reduce(AggSortCtx c, const u32 *pos, const int32_t *gid,
                                                          int64_t m, AggSortedOut o) {
  if (ta_failed(c.status)) return;
  const int64_t j0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (j0 >= m) return;
  int32_t cur = -1;
  u64 cnt = 0, sum = 0;
  i64 mn = INT64_MAX, mx = INT64_MIN;
  for (int k = 0; k < 8 && j0 + k < m; k++) {
    const int32_t g = gid[j0 + k];
    i64 v = 0;
    agg_selected(c, pos[j0 + k], &v);
    if (g != cur) {
      if (cur >= 0) {
        atomicAdd((u64 *)&o.g_count[cur], cnt);
        atomicAdd((u64 *)&o.g_sum[cur], sum);
        atomicMin((i64 *)&o.g_min[cur], mn);
        atomicMax((i64 *)&o.g_max[cur], mx);
      }
      cur = g; cnt = 0; sum = 0; mn = INT64_MAX; mx = INT64_MIN;
    }
    cnt++;
    sum += (u64)v;
    mn = v < mn ? v : mn;
    mx = v > mx ? v : mx;
    atomicAdd(&o.g_hist[(size_t)g * TA_NBINS + log2_bin(v)], 1u);
  }
  if (cur >= 0) {
    atomicAdd((u64 *)&o.g_count[cur], cnt);
    atomicAdd((u64 *)&o.g_sum[cur], sum);
    atomicMin((i64 *)&o.g_min[cur], mn);
    atomicMax((i64 *)&o.g_max[cur], mx);
  }
}

static ta_status ta_run_aggregate_sorted(ta_window *h, uint32_t kind_mask, int value_sel,
                                         ta_agg_result *out) {
  cudaStream_t st = h->stream;
  const int n_pids = h->n_pids > 0 ? h->n_pids : 1;
  const int64_t nv = h->n_valid;
  AggSortCtx c;
  memset(&c, 0, sizeof(c));
  c.n_valid = nv; c.n_lanes = h->sorted.n_lanes; c.n_pids = n_pids;
  c.kind_mask = kind_mask & 63u; c.value_sel = value_sel;
  c.kind = h->sorted.kind; c.name = h->sorted.name_id; c.ts = h->sorted.ts_start; c.te = h->sorted.ts_end;
  c.op_n = h->attr.op_n_kernels; c.op_first = h->attr.op_first_start; c.op_last = h->attr.op_last_end;
  c.op_gap = h->d_op_gap_ns; c.on_path = h->d_on_path; c.lane_off = h->sorted.lane_off; c.lane_slot = h->d_lane_slot;
  c.tt = h->d_triples; c.status = h->d_status;

  // 1. selection
  size_t t1b = Carver::pad((size_t)nv * 8) + Carver::pad((size_t)nv * 4) + scan_temp_bytes(nv) + 256;
  void *t1 = ta_dalloc(h, t1b);
  if (!t1) return TA_ERR_OOM;
  Carver c1(t1);
  u64 *k_in = c1.take<u64>(nv);
  u32 *v_in = c1.take<u32>(nv);
  ScanTemp s1;
  TA_TRY(scan_temp_init(h, c1.base + c1.off, nv, &s1));
  AggSelIn si{c};
  AggSelOut so{c, k_in, v_in};
  TA_TRY((launch_scan<OpAdd, AggSelIn, AggSelOut>(h, nv, si, so, OpAdd(), s1)));
  u64 m64 = 0;
  TA_TRY(ta_queue_d2h(h, &m64, s1.total, 8));
  TA_TRY(ta_sync_fetch(h));
  const int64_t m = (int64_t)m64;
  if (m == 0) { ta_dfree(h, t1); return TA_OK; }

  // 2. sort, 3. groups
  int slot_bits = 1;
  while (slot_bits < 31 && ((int64_t)h->W * n_pids - 1) >> slot_bits) slot_bits++;
  size_t t2b = 2 * Carver::pad((size_t)m * 8) + 2 * Carver::pad((size_t)m * 4) + 2 * Carver::pad((size_t)(m + 1) * 4) +
               ta_sort_temp_bytes(m) + scan_temp_bytes(m) + 256;
  void *t2 = ta_dalloc(h, t2b);
  if (!t2) return TA_ERR_OOM;
  Carver c2(t2);
  u64 *k_scr = c2.take<u64>(m), *ks = c2.take<u64>(m);
  u32 *v_scr = c2.take<u32>(m), *vs = c2.take<u32>(m);
  int32_t *gid = c2.take<int32_t>(m + 1), *gstart = c2.take<int32_t>(m + 1);
  void *sort_tmp = c2.base + c2.off; c2.off += ta_sort_temp_bytes(m);
  void *scan2 = c2.base + c2.off;
  TA_TRY(ta_radix_sort_pairs(h, k_in, v_in, k_scr, v_scr, ks, vs, m, ta_make_plan(0, 32 + slot_bits), nullptr,
                             sort_tmp));
  ScanTemp s2;
  TA_TRY(scan_temp_init(h, scan2, m, &s2));
  AggHeadIn hi{ks};
  AggHeadOut ho{gid, gstart};
  TA_TRY((launch_scan<OpAdd, AggHeadIn, AggHeadOut>(h, m, hi, ho, OpAdd(), s2)));
  u64 ng64 = 0;
  TA_TRY(ta_queue_d2h(h, &ng64, s2.total, 8));
  TA_TRY(ta_sync_fetch(h));
  const int64_t ng = (int64_t)ng64;

  // 4. rows
  size_t ob = 3 * Carver::pad((size_t)ng * 4) + 4 * Carver::pad((size_t)ng * 8) +
              Carver::pad((size_t)ng * TA_NBINS * 4) + 256;
  void *outb = ta_dalloc(h, ob);
  if (!outb) return TA_ERR_OOM;
  TA_CHECK_CUDA(h, cudaMemsetAsync(outb, 0, ob, st));
  Carver co(outb);
  AggSortedOut o;
  o.g_window = co.take<int32_t>(ng); o.g_pid = co.take<int32_t>(ng); o.g_name = co.take<int32_t>(ng);
  o.g_count = co.take<int64_t>(ng); o.g_sum = co.take<int64_t>(ng);
  o.g_min = co.take<int64_t>(ng); o.g_max = co.take<int64_t>(ng);
  o.g_hist = co.take<u32>((size_t)ng * TA_NBINS);
  k_agg_sorted_rows<<<TA_N (unsigned)((ng + 255) / 256), 256, 0, st>>>(c, ks, gstart, ng, o);
  k_agg_sorted_reduce<<<TA_N (unsigned)((m + 2047) / 2048), 256, 0, st>>>(c, vs, gid, m, o);
  TA_CHECK_CUDA(h, cudaGetLastError());
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  ta_dfree(h, t1);
  ta_dfree(h, t2);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  out->n_groups = ng;
  out->g_window = o.g_window; out->g_pid = o.g_pid; out->g_name = o.g_name;
  out->g_count = o.g_count; out->g_sum = o.g_sum; out->g_min = o.g_min; out->g_max = o.g_max;
  out->g_hist = o.g_hist;
  return TA_OK;
}

ta_status ta_run_aggregate(ta_window *h, uint32_t kind_mask, int value_sel, ta_agg_result *out) {
  cudaStream_t st = h->stream;
  const int n_pids = h->n_pids > 0 ? h->n_pids : 1;
  memset(out, 0, sizeof(*out));
  if (h->n_valid == 0 || (kind_mask & 63u) == 0) return TA_OK;
  const unsigned __int128 R128 = (unsigned __int128)((uint64_t)h->max_name - (uint64_t)h->min_name) + 1;
  const unsigned __int128 G128 = R128 * (unsigned __int128)((uint64_t)h->W * (uint64_t)n_pids);
  if (G128 > (unsigned __int128)TA_AGG_DENSE_LIMIT) return ta_run_aggregate_sorted(h, kind_mask, value_sel, out);
  const int64_t R = (int64_t)R128, G = (int64_t)G128;

  size_t tb = 4 * Carver::pad((size_t)G * 8) + Carver::pad((size_t)G * TA_NBINS * 4) + Carver::pad(64) +
              scan_temp_bytes(G) + 256;
  void *tmpb = ta_dalloc(h, tb);
  if (!tmpb) return TA_ERR_OOM;
  Carver ct(tmpb);
  AggArgs a;
  memset(&a, 0, sizeof(a));
  a.d_cnt = ct.take<u64>(G);
  a.d_sum = ct.take<u64>(G);
  a.d_minc = ct.take<u64>(G);
  a.d_maxb = ct.take<u64>(G);
  a.d_hist = ct.take<u32>((size_t)G * TA_NBINS);
  a.n_groups = ct.take<u64>(8);
  TA_CHECK_CUDA(h, cudaMemsetAsync(tmpb, 0, ct.off, st));
  void *scan_mem = ct.base + ct.off;

  a.n_valid = h->n_valid; a.n_lanes = h->sorted.n_lanes;
  a.kind = h->sorted.kind; a.name = h->sorted.name_id; a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end;
  a.lane_off = h->sorted.lane_off; a.lane_slot = h->d_lane_slot;
  a.op_n = h->attr.op_n_kernels; a.op_first = h->attr.op_first_start; a.op_last = h->attr.op_last_end;
  a.op_gap = h->d_op_gap_ns; a.on_path = h->d_on_path;
  a.kind_mask = kind_mask & 63u; a.value_sel = value_sel; a.min_name = h->min_name; a.R = R;
  a.lane_domain = h->sorted.lane_domain; a.lane_dom_end = h->d_lane_dom_end; a.status = h->d_status;
  const bool host_kinds = (a.kind_mask & 7u) != 0, dev_kinds = (a.kind_mask & 56u) != 0;
  a.want_domain = host_kinds && dev_kinds ? -1 : (dev_kinds ? 1 : 0);
  a.chunk = AG_ITEM;
  a.n_items = (unsigned)((h->n_valid + a.chunk - 1) / a.chunk);
  a.spread = a.n_items < 148u * 6u ? a.n_items : 148u * 6u;
  a.per = (a.n_items + a.spread - 1) / a.spread;
  const int64_t blocks = (int64_t)a.spread * a.per;
  k_agg<<<TA_N (unsigned)blocks, AG_THREADS, 0, st>>>(a);
  TA_CHECK_CUDA(h, cudaGetLastError());
  // Rows are compacted without waiting for their count when a bound on it (dense rows, selected
  // records) keeps the output small; otherwise the count is fetched first.
  u64 ng = 0;
  u64 cap = (u64)G < (u64)h->n_valid ? (u64)G : (u64)h->n_valid;
  const bool bounded = cap * (28 + 32 + TA_NBINS * 4) <= (256ull << 20);
  if (!bounded) {
    const int64_t want = (G + 255) / 256;
    k_agg_count_rows<<<TA_N (unsigned)(want < 148 * 8 ? want : 148 * 8), 256, 0, st>>>(a.d_cnt, G, a.n_groups);
    TA_TRY(ta_queue_d2h(h, &ng, a.n_groups, 8));
    TA_TRY(ta_sync_fetch(h));
    cap = ng;
  }
  u64 *scan_total = nullptr;
  if (cap > 0) {
    size_t ob = 3 * Carver::pad(cap * 4) + 4 * Carver::pad(cap * 8) + Carver::pad(cap * TA_NBINS * 4) + 256;
    void *outb = ta_dalloc(h, ob);
    if (!outb) return TA_ERR_OOM;
    Carver co(outb);
    AggRowOut ro;
    ro.cnt = a.d_cnt; ro.sum = a.d_sum; ro.minc = a.d_minc; ro.maxb = a.d_maxb; ro.hist = a.d_hist;
    ro.tt = h->d_triples; ro.n_pids = n_pids; ro.R = R; ro.min_name = h->min_name;
    ro.g_window = co.take<int32_t>(cap); ro.g_pid = co.take<int32_t>(cap); ro.g_name = co.take<int32_t>(cap);
    ro.g_count = co.take<int64_t>(cap); ro.g_sum = co.take<int64_t>(cap);
    ro.g_min = co.take<int64_t>(cap); ro.g_max = co.take<int64_t>(cap);
    ro.g_hist = co.take<u32>(cap * TA_NBINS);
    ScanTemp t;
    TA_TRY(scan_temp_init(h, scan_mem, G, &t));
    AggRowIn ri{a.d_cnt};
    TA_TRY((launch_scan<OpAdd, AggRowIn, AggRowOut>(h, G, ri, ro, OpAdd(), t)));
    scan_total = t.total;
    out->g_window = ro.g_window; out->g_pid = ro.g_pid; out->g_name = ro.g_name;
    out->g_count = ro.g_count; out->g_sum = ro.g_sum; out->g_min = ro.g_min; out->g_max = ro.g_max;
    out->g_hist = ro.g_hist;
  }
  if (bounded && scan_total)  // the scan's total is the number of rows
    TA_TRY(ta_queue_d2h(h, &ng, scan_total, 8));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  out->n_groups = (int64_t)ng;
  ta_dfree(h, tmpb);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  return TA_OK;
}
