// ta_correlate_launches: every device record is joined to the host call that
// submitted it through the correlation id both carry (Sec. 5.2; Fig. "Key
// performance observations" (a)).  Key =
// (window, pid, corr_id); the smallest sorted position among equal LAUNCH keys
// wins.
//
// Two paths, same results:
//   direct   when the correlation ids of each (window, pid) span a compact
//            range (they count up per process in real traces): a table of
//            sorted positions indexed by corr_id - min, filled with atomicMin.
//            Launches and kernels are time-ordered, so the table is touched
//            nearly sequentially.
//   general  any 64-bit ids: launches and probes are compacted, stably sorted
//            by (slot, corr_id) with the pair sorter, and each probe takes the
//            head of its run if that head is a LAUNCH.
// HBM-bound: streams kind/corr/ts columns, writes three outputs per record.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define JN_THREADS 512
#define JN_ITEMS 4
#define JN_TILE (JN_THREADS * JN_ITEMS)
#define EMPTY_U32 0xFFFFFFFFu

struct JoinArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int16_t *kind;
  const int64_t *corr, *ts, *te;
  const int32_t *lane_off, *lane_slot, *lane_window, *lane_dom_end;
  const int16_t *lane_domain;
  // per slot (window * n_pids + pid rank)
  i64 *slot_min, *slot_max;       // corr range of LAUNCH records
  const i64 *slot_base;           // direct path: table offset of the slot, -1 = no launches
  u32 *table;                     // direct path
  const int32_t *found;           // general path: winner launch per launch/probe position
  int32_t *launch_of, *kol;
  int64_t *latency, *qdelay;
  ta_join_summary *sum;           // device, per window
  const int32_t *status;
};

__device__ __forceinline__ u64 bias64(i64 v) { return (u64)v ^ (1ull << 63); }
__device__ __forceinline__ i64 unbias64(u64 v) { return (i64)(v ^ (1ull << 63)); }

// block-wide reduction helper (all threads call); smem >= 33 u64
__device__ __forceinline__ u64 blk_reduce(u64 v, bool is_max, u64 *smem) {
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

// lanes touched by the CTA's selected items -> [l0, l1] (l1 < l0 if none)
__device__ __forceinline__ void tile_lane_range(int my_lo, int my_hi, int *s_lo, int *s_hi, int *l0,
                                                int *l1) {
  if (threadIdx.x == 0) { *s_lo = INT_MAX; *s_hi = -1; }
  __syncthreads();
  if (my_hi >= 0) { atomicMin(s_lo, my_lo); atomicMax(s_hi, my_hi); }
  __syncthreads();
  *l0 = *s_lo;
  *l1 = *s_hi;
  __syncthreads();
}


// ---- direct path: fill the table -------------------------------------------
__global__ void __launch_bounds__(JN_THREADS) k_join_build(JoinArgs a) {
  __shared__ int s_lane0;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x;
  const int64_t tile_start = (int64_t)blockIdx.x * JN_TILE;
  if (tile_start >= a.n_valid) return;
  if (tid < 32) {
    const int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (tid == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  // launches live in host lanes: a tile of device lanes has none
  if (span_outside_domain(a.lane_domain, a.lane_dom_end, l0, min(tile_start + JN_TILE, a.n_valid), 0)) return;
  const int64_t p0 = tile_start + (int64_t)tid * JN_ITEMS;
  int16_t kd[JN_ITEMS];
  i64 c[JN_ITEMS];
  loadn_i16<JN_ITEMS>(a.kind, p0, a.n, 9, kd);
  loadn_i64<JN_ITEMS>(a.corr, p0, a.n, c);
  int l = l0;
  int64_t next_off = a.lane_off[l + 1];
  int slot = a.lane_slot[l];
#pragma unroll
  for (int j = 0; j < JN_ITEMS; j++) {
    const int64_t p = p0 + j;
    if (p < a.n_valid && kd[j] == TA_KIND_LAUNCH) {
      while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; slot = a.lane_slot[l]; }
      const i64 idx = a.slot_base[slot] + (c[j] - a.slot_min[slot]);
      atomicMin(&a.table[idx], (u32)p);
    }
  }
}

template <bool DIRECT>
__device__ __forceinline__ int32_t winner_of(const JoinArgs &a, int64_t p, int slot) {
  if (!DIRECT) return a.found[p];
  i64 base = a.slot_base[slot];
  if (base < 0) return -1;
  i64 c = a.corr[p];
  if (c < a.slot_min[slot] || c > a.slot_max[slot]) return -1;
  u32 v = a.table[base + (c - a.slot_min[slot])];
  return v == EMPTY_U32 ? -1 : (int32_t)v;
}

// ---- pass 2: probes ----------------------------------------------------------
// 256 threads x JP_ITEMS consecutive positions; every output column is written once.
#define JP_THREADS 256
#ifndef JP_MINB
#define JP_MINB 3
#endif
#ifndef JP_ITEMS
#define JP_ITEMS 8
#endif
#define JP_TILE (JP_THREADS * JP_ITEMS)

template <bool DIRECT>
__global__ void __launch_bounds__(JP_THREADS, JP_MINB) k_join_probe(JoinArgs a) {
  __shared__ u64 red[7][JP_THREADS / 32];
  __shared__ int s_lane0, s_lane1;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t tile_start = (int64_t)blockIdx.x * JP_TILE;
  constexpr int IT = JP_ITEMS;
  const int64_t p0 = tile_start + (int64_t)tid * IT;
  if (tid == 0) { s_lane0 = -1; s_lane1 = -1; }
  __syncthreads();
  if (tid < 32 && tile_start < a.n_valid && a.n_lanes > 0) {
    int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (lane == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  // A tile of host lanes holds no probe: nothing to read, the three outputs are -1 / 0 / 0.
  if (l0 >= 0 && span_outside_domain(a.lane_domain, a.lane_dom_end, l0, min(tile_start + JP_TILE, a.n_valid), 1)) {
    int32_t lo0[IT];
    i64 z[IT];
#pragma unroll
    for (int j = 0; j < IT; j++) { lo0[j] = -1; z[j] = 0; }
    storen_i32<IT>(a.launch_of, p0, a.n, lo0);
    storen_i64<IT>(a.latency, p0, a.n, z);
    storen_i64<IT>(a.qdelay, p0, a.n, z);
    return;
  }
  // kinds, correlation ids and start times are requested together: one round of memory
  // latency less than loading the ids only where the kinds ask for them
  int16_t kd[IT];
  i64 c[IT], s[IT];
  loadn_i16<IT>(a.kind, p0, a.n, 0, kd);
  loadn_i64<IT>(a.corr, p0, a.n, c);
  loadn_i64<IT>(a.ts, p0, a.n, s);
  unsigned pm = 0;  // probes among the thread's records
#pragma unroll
  for (int j = 0; j < IT; j++)
    if (p0 + j < a.n_valid && (kd[j] == TA_KIND_KERNEL || kd[j] == TA_KIND_MEMCPY)) pm |= 1u << j;
  int32_t lo[IT];
  int ln[IT];
  {
    int l = l0;
    int64_t next_off = l >= 0 ? (int64_t)a.lane_off[l + 1] : LLONG_MAX;
    int slot = l >= 0 ? a.lane_slot[l] : 0;
#pragma unroll
    for (int j = 0; j < IT; j++) {
      lo[j] = -1;
      ln[j] = -1;
      if (pm & (1u << j)) {
        const int64_t p = p0 + j;
        while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; slot = a.lane_slot[l]; }
        ln[j] = l;
        if (DIRECT) {
          const i64 base = a.slot_base[slot];
          if (base >= 0 && c[j] >= a.slot_min[slot] && c[j] <= a.slot_max[slot]) {
            const u32 v = a.table[base + (c[j] - a.slot_min[slot])];
            lo[j] = v == EMPTY_U32 ? -1 : (int32_t)v;
          }
        } else {
          lo[j] = a.found[p];
        }
      }
    }
    const int64_t plast = min(tile_start + JP_TILE, a.n_valid) - 1;
    if (plast >= p0 && plast < p0 + IT) {
      while (plast >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      s_lane1 = l;
    }
  }
  // launch times of the matched probes (independent gathers, issued together)
  i64 ls[IT], le[IT];
#pragma unroll
  for (int j = 0; j < IT; j++) {
    ls[j] = le[j] = 0;
    if (lo[j] >= 0) { ls[j] = a.ts[lo[j]]; le[j] = a.te[lo[j]]; }
  }
  i64 lat[IT], q[IT];
  u64 np = 0, nm = 0, sl = 0, sq = 0, mxl = 0, mnl_inv = 0, mxq = 0;
  int lm = -1;
#pragma unroll
  for (int j = 0; j < IT; j++) {
    lat[j] = q[j] = 0;
    if (!(pm & (1u << j))) continue;
    const bool matched = lo[j] >= 0;
    if (matched) {
      lat[j] = s[j] - ls[j];
      const i64 d = s[j] - le[j];
      q[j] = d > 0 ? d : 0;
      atomicAdd(&a.kol[lo[j]], 1);
    }
    if (lm < 0) lm = ln[j];
    if (ln[j] == lm && ln[j] - l0 <= 1) {
      np++;
      if (matched) {
        nm++;
        sl += (u64)lat[j];
        sq += (u64)q[j];
        mxl = max(mxl, bias64(lat[j]));
        mnl_inv = max(mnl_inv, ~bias64(lat[j]));
        mxq = max(mxq, (u64)q[j]);
      }
    } else {  // a thread that straddles a lane boundary, or a third lane in the tile
      ta_join_summary *sm = &a.sum[a.lane_window[ln[j]]];
      atomicAdd((u64 *)&sm->n_probe, 1ull);
      if (matched) {
        atomicAdd((u64 *)&sm->n_matched, 1ull);
        atomicAdd((u64 *)&sm->sum_latency, (u64)lat[j]);
        atomicAdd((u64 *)&sm->sum_queue, (u64)q[j]);
        atomicMax((i64 *)&sm->max_latency, lat[j]);
        atomicMin((i64 *)&sm->min_latency, lat[j]);
        atomicMax((i64 *)&sm->max_queue, q[j]);
      }
    }
  }
  storen_i32<IT>(a.launch_of, p0, a.n, lo);
  storen_i64<IT>(a.latency, p0, a.n, lat);
  storen_i64<IT>(a.qdelay, p0, a.n, q);
  __syncthreads();
  const int l1 = s_lane1;
  for (int li = 0; li < 2; li++) {
    const int l = l0 + li;
    if (l0 < 0 || l > l1) break;
    if (a.lane_domain[l] != 1) continue;  // uniform over the CTA
    const bool mine = lm == l;
    u64 r[7] = {mine ? np : 0, mine ? nm : 0, mine ? sl : 0, mine ? sq : 0,
                mine ? mxl : 0, mine ? mnl_inv : 0, mine ? mxq : 0};
#pragma unroll
    for (int k = 0; k < 4; k++) r[k] = warp_reduce(r[k], OpAdd());
#pragma unroll
    for (int k = 4; k < 7; k++) r[k] = warp_reduce(r[k], OpMax());
    __syncthreads();
    if (lane == 0)
#pragma unroll
      for (int k = 0; k < 7; k++) red[k][tid >> 5] = r[k];
    __syncthreads();
    if (tid == 0) {
      u64 t[7] = {0, 0, 0, 0, 0, 0, 0};
      for (int w = 0; w < JP_THREADS / 32; w++) {
        for (int k = 0; k < 4; k++) t[k] += red[k][w];
        for (int k = 4; k < 7; k++) t[k] = max(t[k], red[k][w]);
      }
      if (t[0]) {
        ta_join_summary *sm = &a.sum[a.lane_window[l]];
        atomicAdd((u64 *)&sm->n_probe, t[0]);
        if (t[1]) {
          atomicAdd((u64 *)&sm->n_matched, t[1]);
          atomicAdd((u64 *)&sm->sum_latency, t[2]);
          atomicAdd((u64 *)&sm->sum_queue, t[3]);
          atomicMax((i64 *)&sm->max_latency, unbias64(t[4]));
          atomicMin((i64 *)&sm->min_latency, unbias64(~t[5]));
          atomicMax((i64 *)&sm->max_queue, (i64)t[6]);
        }
      }
    }
  }
}

// ---- pass 3: launch statistics (duplicates, orphans) ---------------------------
#define JS_TILE (JP_THREADS * 8)
template <bool DIRECT>
__global__ void __launch_bounds__(JP_THREADS) k_join_launch_stats(JoinArgs a) {
  __shared__ u64 red[JP_THREADS / 32];
  __shared__ int s_lane0, s_lane1;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t tile_start = (int64_t)blockIdx.x * JS_TILE;
  const int64_t p0 = tile_start + (int64_t)tid * 8;
  if (tid == 0) { s_lane0 = -1; s_lane1 = -1; }
  __syncthreads();
  if (tid < 32 && tile_start < a.n_valid && a.n_lanes > 0) {
    int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (lane == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  // launches live in host lanes: a tile of device lanes has none
  if (l0 < 0 || span_outside_domain(a.lane_domain, a.lane_dom_end, l0, min(tile_start + JS_TILE, a.n_valid), 0))
    return;
  // kinds, correlation ids and kernel counts of the thread's records together, then the table
  // entries of its launches together: two rounds of memory latency
  int16_t kd[8];
  i64 cr[8];
  int32_t nk[8];
  load8_i16(a.kind, p0, a.n, 0, kd);
  load8_i64(a.corr, p0, a.n, cr);
  if (p0 + 8 <= a.n) {
    const int4 x = *reinterpret_cast<const int4 *>(a.kol + p0), y = *reinterpret_cast<const int4 *>(a.kol + p0 + 4);
    nk[0] = x.x; nk[1] = x.y; nk[2] = x.z; nk[3] = x.w; nk[4] = y.x; nk[5] = y.y; nk[6] = y.z; nk[7] = y.w;
  } else {
#pragma unroll
    for (int j = 0; j < 8; j++) nk[j] = p0 + j < a.n ? a.kol[p0 + j] : 0;
  }
  unsigned lmask = 0;
#pragma unroll
  for (int j = 0; j < 8; j++)
    if (p0 + j < a.n_valid && kd[j] == TA_KIND_LAUNCH) lmask |= 1u << j;
  u64 packed = 0;  // n_launch | n_dup << 20 | n_orphan << 40 for the thread's first lane
  int lm = -1;
  {
    int l = l0;
    int64_t next_off = l >= 0 ? (int64_t)a.lane_off[l + 1] : LLONG_MAX;
    int ln[8];
    int32_t win[8];
#pragma unroll
    for (int j = 0; j < 8; j++) {
      ln[j] = -1;
      win[j] = -1;
      if (!(lmask & (1u << j))) continue;
      const int64_t p = p0 + j;
      while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      ln[j] = l;
      if (DIRECT) {
        const int slot = a.lane_slot[l];
        const i64 base = a.slot_base[slot];
        if (base >= 0 && cr[j] >= a.slot_min[slot] && cr[j] <= a.slot_max[slot]) {
          const u32 v = a.table[base + (cr[j] - a.slot_min[slot])];
          win[j] = v == EMPTY_U32 ? -1 : (int32_t)v;
        }
      } else {
        win[j] = a.found[p];
      }
    }
    const int l_end = l;
    int64_t next_end = next_off;
#pragma unroll
    for (int j = 0; j < 8; j++) {
      if (!(lmask & (1u << j))) continue;
      const int64_t p = p0 + j;
      const int l = ln[j];
      const bool dup = win[j] != (int32_t)p;
      const bool orphan = !dup && nk[j] == 0;
      if (lm < 0) lm = l;
      if (l == lm && l - l0 <= 1) {
        packed += 1ull + ((u64)dup << 20) + ((u64)orphan << 40);
      } else {
        ta_join_summary *sm = &a.sum[a.lane_window[l]];
        atomicAdd((u64 *)&sm->n_launch, 1ull);
        if (dup) atomicAdd((u64 *)&sm->n_dup_launch, 1ull);
        if (orphan) atomicAdd((u64 *)&sm->n_orphan_launch, 1ull);
      }
    }
    const int64_t plast = min(tile_start + JS_TILE, a.n_valid) - 1;
    if (plast >= p0 && plast < p0 + 8) {
      int le = l_end;
      while (plast >= next_end) { le++; next_end = a.lane_off[le + 1]; }
      s_lane1 = le;
    }
  }
  __syncthreads();
  const int l1 = s_lane1;
  for (int li = 0; li < 2; li++) {
    const int l = l0 + li;
    if (l0 < 0 || l > l1) break;
    if (a.lane_domain[l] != 0) continue;
    u64 v = warp_reduce(lm == l ? packed : 0, OpAdd());
    __syncthreads();
    if (lane == 0) red[tid >> 5] = v;
    __syncthreads();
    if (tid == 0) {
      u64 t = 0;
      for (int w = 0; w < JP_THREADS / 32; w++) t += red[w];
      const u64 m = (1ull << 20) - 1;
      ta_join_summary *sm = &a.sum[a.lane_window[l]];
      if (t & m) atomicAdd((u64 *)&sm->n_launch, t & m);
      if ((t >> 20) & m) atomicAdd((u64 *)&sm->n_dup_launch, (t >> 20) & m);
      if ((t >> 40) & m) atomicAdd((u64 *)&sm->n_orphan_launch, (t >> 40) & m);
    }
  }
}

// ---- general path helpers -----------------------------------------------------
__global__ void __launch_bounds__(256) k_join_key_corr(const u32 *pos, int64_t m, const int64_t *corr,
                                                       u64 *out, const int32_t *status) {
  if (ta_failed(status)) return;
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j < m) out[j] = bias64(corr[pos[j]]);
}
__global__ void __launch_bounds__(256) k_join_key_slot(const u32 *pos, int64_t m,
                                                       const int32_t *lane_off, int n_lanes,
                                                       const int32_t *lane_slot, u64 *out,
                                                       const int32_t *status) {
  if (ta_failed(status)) return;
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j < m) out[j] = (u64)lane_slot[lane_of_pos(lane_off, n_lanes, pos[j])];
}
struct JoinHeadIn {
  const u64 *slot_key;
  const u32 *pos;
  const int64_t *corr;
  __device__ u64 operator()(int64_t j) const {
    bool head = j == 0 || slot_key[j] != slot_key[j - 1] || corr[pos[j]] != corr[pos[j - 1]];
    return head ? (u64)(j + 1) : 0ull;
  }
};
struct JoinHeadOut {
  const u32 *pos;
  const int16_t *kind;
  int32_t *found;
  __device__ void operator()(int64_t j, u64 excl, u64 v) const {
    u64 hd = (excl > v ? excl : v) - 1;  // index of the head of j's run
    u32 hp = pos[hd];
    found[pos[j]] = kind[hp] == TA_KIND_LAUNCH ? (int32_t)hp : -1;
  }
};

static int bit_length64(uint64_t v) {
  int b = 0;
  while (v) { b++; v >>= 1; }
  return b;
}

ta_status ta_run_correlate(ta_window *h, ta_join_summary *out_summary) {
  const int64_t n = h->n;
  const int W = h->W;
  const int n_slots = W * (h->n_pids > 0 ? h->n_pids : 1);
  cudaStream_t st = h->stream;
  const int64_t nn = n > 0 ? n : 1;
  size_t keep = 2 * Carver::pad(nn * 4) + 2 * Carver::pad(nn * 8) + Carver::pad((size_t)n_slots * 8) +
                Carver::pad((size_t)W * sizeof(ta_join_summary)) + 256;
  void *kb = ta_dalloc(h, keep);
  if (!kb) return TA_ERR_OOM;
  Carver ck(kb);
  int32_t *launch_of = ck.take<int32_t>(nn), *kol = ck.take<int32_t>(nn);
  int64_t *latency = ck.take<int64_t>(nn), *qdelay = ck.take<int64_t>(nn);
  i64 *slot_min = h->d_slot_min, *slot_max = h->d_slot_max;  // filled while the records were gathered
  i64 *slot_base = ck.take<i64>(n_slots);
  ta_join_summary *d_sum = ck.take<ta_join_summary>(W);

  std::vector<ta_join_summary> hs(W);
  for (auto &s : hs) {
    memset(&s, 0, sizeof(s));
    s.min_latency = INT64_MAX;
    s.max_latency = INT64_MIN;
  }
  std::vector<i64> hmin(h->h_slot_min.begin(), h->h_slot_min.end());
  std::vector<i64> hmax(h->h_slot_max.begin(), h->h_slot_max.end()), hbase(n_slots, -1);
  TA_CHECK_CUDA(h, cudaMemcpyAsync(d_sum, hs.data(), W * sizeof(ta_join_summary), cudaMemcpyHostToDevice, st));
  TA_CHECK_CUDA(h, cudaMemsetAsync(kol, 0, nn * 4, st));

  JoinArgs a;
  memset(&a, 0, sizeof(a));
  a.n = n; a.n_valid = h->n_valid; a.n_lanes = h->sorted.n_lanes;
  a.kind = h->sorted.kind; a.corr = h->sorted.corr_id; a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end;
  a.lane_off = h->sorted.lane_off; a.lane_slot = h->d_lane_slot; a.lane_window = h->sorted.lane_window;
  a.lane_domain = h->sorted.lane_domain; a.lane_dom_end = h->d_lane_dom_end;
  a.slot_min = slot_min; a.slot_max = slot_max; a.slot_base = slot_base;
  a.launch_of = launch_of; a.kol = kol; a.latency = latency; a.qdelay = qdelay; a.sum = d_sum;
  a.status = h->d_status;
  const unsigned grid = (unsigned)((n + JN_TILE - 1) / JN_TILE);
  const unsigned grid8 = (unsigned)((n + JS_TILE - 1) / JS_TILE);
  const unsigned grid_probe = (unsigned)((n + JP_TILE - 1) / JP_TILE);
  void *tmp_alloc = nullptr;
  bool direct = true;
  if (n > 0) {
    // table size if every slot is addressed directly
    unsigned __int128 total = 0;
    for (int s = 0; s < n_slots; s++)
      if (hmin[s] <= hmax[s]) {
        hbase[s] = (i64)total;
        total += (unsigned __int128)((uint64_t)hmax[s] - (uint64_t)hmin[s]) + 1;
      }
    const uint64_t limit = (uint64_t)4 * (uint64_t)n + 65536;
    direct = total <= limit;
    if (direct) {
      uint64_t M = (uint64_t)total;
      tmp_alloc = ta_dalloc(h, (size_t)(M > 0 ? M : 1) * 4);
      if (!tmp_alloc) return TA_ERR_OOM;
      a.table = (u32 *)tmp_alloc;
      TA_CHECK_CUDA(h, cudaMemsetAsync(a.table, 0xFF, (size_t)(M > 0 ? M : 1) * 4, st));
      TA_CHECK_CUDA(h, cudaMemcpyAsync(slot_base, hbase.data(), n_slots * 8, cudaMemcpyHostToDevice, st));
      k_join_build<<<TA_N grid, JN_THREADS, 0, st>>>(a);
      k_join_probe<true><<<TA_N grid_probe, JP_THREADS, 0, st>>>(a);
      k_join_launch_stats<true><<<TA_N grid8, JP_THREADS, 0, st>>>(a);
    } else {
      // general path: compact, sort by (slot, corr) with sorted position as the stable tie-break
      size_t tb = Carver::pad(nn * 4) * 3 + Carver::pad(nn * 8) * 3 + scan_temp_bytes(n) * 2 +
                  ta_sort_temp_bytes(n) + 512;
      tmp_alloc = ta_dalloc(h, tb);
      if (!tmp_alloc) return TA_ERR_OOM;
      Carver ct(tmp_alloc);
      u32 *pos = ct.take<u32>(nn), *pos_s = ct.take<u32>(nn);
      int32_t *found = ct.take<int32_t>(nn);
      u64 *k_in = ct.take<u64>(nn), *k_s = ct.take<u64>(nn), *k_f = ct.take<u64>(nn);
      void *scan_mem1 = ct.base + ct.off; ct.off += scan_temp_bytes(n);
      void *scan_mem2 = ct.base + ct.off; ct.off += scan_temp_bytes(n);
      void *sort_tmp = ct.base + ct.off;
      ScanTemp t1;
      TA_TRY(scan_temp_init(h, scan_mem1, n, &t1));
      TA_TRY(launch_compact_kind(h, a.kind, h->n_valid,
                                 (1u << TA_KIND_LAUNCH) | (1u << TA_KIND_KERNEL) | (1u << TA_KIND_MEMCPY),
                                 pos, t1));
      u64 m64 = 0;
      TA_TRY(ta_queue_d2h(h, &m64, t1.total, 8));
      TA_TRY(ta_sync_fetch(h));
      const int64_t m = (int64_t)m64;
      TA_CHECK_CUDA(h, cudaMemsetAsync(found, 0xFF, nn * 4, st));
      if (m > 0) {
        const int gb = (int)((m + 255) / 256);
        u32 *vscr = (u32 *)found;  // found is not needed before the sorts are done
        k_join_key_corr<<<TA_N gb, 256, 0, st>>>(pos, m, a.corr, k_in, h->d_status);
        TA_TRY(ta_radix_sort_pairs(h, k_in, pos, k_s, vscr, k_f, pos_s, m, ta_make_plan(0, 64), nullptr,
                                   sort_tmp));
        k_join_key_slot<<<TA_N gb, 256, 0, st>>>(pos_s, m, a.lane_off, a.n_lanes, a.lane_slot, k_in,
                                                 h->d_status);
        int sb = bit_length64((uint64_t)(n_slots > 1 ? n_slots - 1 : 1));
        TA_TRY(ta_radix_sort_pairs(h, k_in, pos_s, k_s, vscr, k_f, pos, m, ta_make_plan(0, sb), nullptr,
                                   sort_tmp));
        TA_CHECK_CUDA(h, cudaMemsetAsync(found, 0xFF, nn * 4, st));
        ScanTemp t2;
        TA_TRY(scan_temp_init(h, scan_mem2, m, &t2));
        JoinHeadIn hin{k_f, pos, a.corr};
        JoinHeadOut hout{pos, a.kind, found};
        TA_TRY((launch_scan<OpMax, JoinHeadIn, JoinHeadOut>(h, m, hin, hout, OpMax(), t2)));
      }
      a.found = found;
      k_join_probe<false><<<TA_N grid_probe, JP_THREADS, 0, st>>>(a);
      k_join_launch_stats<false><<<TA_N grid8, JP_THREADS, 0, st>>>(a);
    }
    TA_CHECK_CUDA(h, cudaGetLastError());
  }
  TA_TRY(ta_queue_d2h(h, hs.data(), d_sum, W * sizeof(ta_join_summary)));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  if (tmp_alloc) ta_dfree(h, tmp_alloc);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  for (int w = 0; w < W; w++) {
    ta_join_summary &s = hs[w];
    s.n_unmatched = s.n_probe - s.n_matched;
    if (s.n_matched == 0) { s.min_latency = 0; s.max_latency = 0; }
    if (out_summary) out_summary[w] = s;
  }
  h->join.launch_of = launch_of;
  h->join.launch_latency = latency;
  h->join.queue_delay = qdelay;
  h->join.kernels_of_launch = kol;
  if (n == 0) {
    // nothing was launched: outputs are single dummy entries
  }
  return TA_OK;
}
