// ta_attribute_operators: thread id plus call intervals link host API calls to
// the enclosing calls (Sec. 9.1); device records inherit the operator of their
// launch; T_op spans the first kernel start to the last completion (Sec. 6.1).
//
// In canonical order (ts_start ascending, ts_end descending) a properly nested
// host lane has a simple structure: the innermost encloser of record i is the
// nearest earlier OP that is still running when i starts.  That is answered
//   - inside a tile of 2048 records (256 threads x 8 consecutive records) by a
//     backward look over the thread's own records and, failing that, one descent
//     of a max-tree over the threads' largest OP end times in shared memory;
//   - across tiles by carrying the stack of still-open OPs (at most
//     TA_MAX_DEPTH + 1 entries when nesting is legal) through a bounded
//     decoupled look-back that one warp performs with one stack entry per lane.
//     Combining a carried stack with a tile's stack is associative: entries that
//     end no later than the tile's outermost surviving OP can never be chosen
//     again and are dropped.
// Partial overlap is detected on the way: that nearest running OP must also
// cover i's end.
// HBM-bound: 18 B read per host record + 5 B written per record, plus the
// per-operator atomics of the device records.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define AT_THREADS 256
#define AT_ITEMS 8
#define AT_TILE (AT_THREADS * AT_ITEMS)
#define AT_CAP 16
#define AT_NONE (-1)
#define AT_UNRESOLVED (-2)

struct AttrArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int16_t *kind;
  const int64_t *ts, *te;
  const int32_t *lane_off, *lane_window;
  const int16_t *lane_domain;
  int32_t *parent;
  uint8_t *depth;
  ta_attr_summary *sum;
  // tile descriptors
  u64 *flag;
  int32_t *agg_meta, *pre_meta;  // count | reset << 8
  i64 *agg_e, *pre_e;            // [tile][AT_CAP]
  int32_t *agg_pos, *pre_pos;
  u32 *counter;
  int32_t *status;
  // second kernel
  const int32_t *launch_of;
  int32_t *op_of, *op_n;
  u64 *op_first, *op_last;
  int64_t *op_ns;
};

struct AttrSmem {
  i64 leaf[AT_TILE];              // OP end time, INT64_MIN elsewhere
  i64 T[2 * AT_THREADS];          // max-tree over the threads' maxima, leaves at [AT_THREADS, 2*AT_THREADS)
  int16_t parent_local[AT_TILE];
  uint8_t kcarry[AT_TILE];
  i64 agg_e[AT_CAP], carry_e[AT_CAP];
  int32_t agg_pos[AT_CAP], carry_pos[AT_CAP];
  int agg_raw, carry_cnt;
  int tile, lane0, lane1, dmax;
};

// A stack of open operators, one entry per lane of a warp (bottom = lane 0).
struct WStack {
  int cnt, reset;
  i64 e;
  int32_t pos;
};

// acc <- earlier (+) acc, all 32 lanes
__device__ __forceinline__ void wstack_combine(const WStack &ear, WStack &acc, bool *overflow) {
  if (acc.reset) return;
  const int lane = threadIdx.x & 31;
  int keep = ear.cnt;
  if (acc.cnt > 0) {
    const i64 e0 = __shfl_sync(0xffffffffu, acc.e, 0);
    keep = __popc(__ballot_sync(0xffffffffu, lane < ear.cnt && ear.e > e0));
  }
  if (keep + acc.cnt > AT_CAP) {
    *overflow = true;
    keep = AT_CAP - acc.cnt;
  }
  const int src = lane - keep < 0 ? 0 : lane - keep;
  const i64 se = __shfl_sync(0xffffffffu, acc.e, src);
  const int32_t sp = __shfl_sync(0xffffffffu, acc.pos, src);
  acc.e = lane < keep ? ear.e : se;
  acc.pos = lane < keep ? ear.pos : sp;
  acc.cnt += keep;
  acc.reset = ear.reset;
}

__device__ __forceinline__ int warp_lane_search_a(const int32_t *lane_off, int n_lanes, int64_t p) {
  const int lane = threadIdx.x & 31;
  int lo = 0, hi = n_lanes;
  while (hi - lo > 1) {
    int step = (hi - lo + 31) >> 5;
    int idx = lo + lane * step;
    bool ok = idx < hi && (int64_t)lane_off[idx] <= p;
    u32 m = __ballot_sync(0xffffffffu, ok);
    int k = 31 - __clz((int)m);
    lo = lo + k * step;
    hi = min(hi, lo + step);
  }
  return lo;
}

__device__ __forceinline__ void publish_stack(i64 *pe, int32_t *pp, int32_t *pmeta, u64 *flag, int tile,
                                              const WStack &s, u64 kind) {
  const int lane = threadIdx.x & 31;
  if (lane < s.cnt) {
    pe[(size_t)tile * AT_CAP + lane] = s.e;
    pp[(size_t)tile * AT_CAP + lane] = s.pos;
  }
  if (lane == 0) pmeta[tile] = s.cnt | (s.reset << 8);
  __threadfence();
  __syncwarp();
  if (lane == 0) st_relaxed(&flag[tile], td_pack(kind, 0));
}

__global__ void __launch_bounds__(AT_THREADS, 3) k_attr(AttrArgs a) {
  __shared__ AttrSmem s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s.tile = (int)atomicAdd(a.counter, 1u);
    s.lane1 = -1;
    s.agg_raw = 0;
    s.dmax = 0;
    s.lane0 = -1;
  }
  __syncthreads();
  const int tile = s.tile;
  const int64_t tile_start = (int64_t)tile * AT_TILE;
  const int x0 = tid * AT_ITEMS;
  const int64_t p0 = tile_start + x0;
  const bool full = p0 + AT_ITEMS <= a.n;
  if (warp == 0 && tile_start < a.n_valid && a.n_lanes > 0) {
    int l = warp_lane_search_a(a.lane_off, a.n_lanes, tile_start);
    if (lane == 0) s.lane0 = l;
  }
  int16_t kd[AT_ITEMS];
  if (full) {
    uint4 q = *reinterpret_cast<const uint4 *>(a.kind + p0);
    const int16_t *hq = reinterpret_cast<const int16_t *>(&q);
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++) kd[j] = hq[j];
  } else {
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++) kd[j] = p0 + j < a.n ? a.kind[p0 + j] : (int16_t)9;
  }
  unsigned hostmask = 0;
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++)
    if (p0 + j < a.n_valid && kd[j] <= TA_KIND_LAUNCH) hostmask |= 1u << j;
  const int any_host = __syncthreads_or(hostmask != 0);
  if (!any_host) {
    // no host record here: the tile ends in a device lane (or beyond the kept records)
    if (tid == 0) {
      a.pre_meta[tile] = 1 << 8;
      __threadfence();
      st_relaxed(&a.flag[tile], td_pack(TD_PREFIX, 0));
    }
    if (full) {
      *reinterpret_cast<int4 *>(a.parent + p0) = make_int4(-1, -1, -1, -1);
      *reinterpret_cast<int4 *>(a.parent + p0 + 4) = make_int4(-1, -1, -1, -1);
      *reinterpret_cast<uint2 *>(a.depth + p0) = make_uint2(0, 0);
    } else {
      for (int j = 0; j < AT_ITEMS; j++)
        if (p0 + j < a.n) { a.parent[p0 + j] = -1; a.depth[p0 + j] = 0; }
    }
    return;
  }
  i64 st[AT_ITEMS], en[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) st[j] = en[j] = 0;
  if (hostmask) {
    if (full) {
      const longlong2 *ps = reinterpret_cast<const longlong2 *>(a.ts + p0);
      const longlong2 *pe = reinterpret_cast<const longlong2 *>(a.te + p0);
#pragma unroll
      for (int j = 0; j < AT_ITEMS / 2; j++) {
        longlong2 x = ps[j], y = pe[j];
        st[2 * j] = x.x; st[2 * j + 1] = x.y;
        en[2 * j] = y.x; en[2 * j + 1] = y.y;
      }
    } else {
#pragma unroll
      for (int j = 0; j < AT_ITEMS; j++)
        if (p0 + j < a.n) { st[j] = a.ts[p0 + j]; en[j] = a.te[p0 + j]; }
    }
  }
  // lanes, leaves, the thread's maximum
  const int l0 = s.lane0;
  int ln[AT_ITEMS];
  int lo_local[AT_ITEMS];  // first tile-local index of the record's lane (-1: the lane began earlier)
  i64 m8 = INT64_MIN;
  {
    int l = l0;
    int64_t next_off = l >= 0 ? (int64_t)a.lane_off[l + 1] : LLONG_MAX;
    int64_t cur_off = l >= 0 ? (int64_t)a.lane_off[l] : 0;
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++) {
      const int64_t p = p0 + j;
      ln[j] = -1;
      lo_local[j] = 0;
      i64 leaf = INT64_MIN;
      if (hostmask & (1u << j)) {
        while (p >= next_off) { l++; cur_off = next_off; next_off = a.lane_off[l + 1]; }
        ln[j] = l;
        lo_local[j] = cur_off < tile_start ? -1 : (int)(cur_off - tile_start);
        if (kd[j] == TA_KIND_OP) leaf = en[j];
      }
      s.leaf[x0 + j] = leaf;
      m8 = leaf > m8 ? leaf : m8;
    }
    const int64_t plast = min(tile_start + AT_TILE, a.n_valid) - 1;
    if (plast >= p0 && plast < p0 + AT_ITEMS) {
      while (plast >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      s.lane1 = l;
    }
  }
  s.T[AT_THREADS + tid] = m8;
  __syncwarp();
  // tree levels inside the warp's subtree: 16, 8, 4, 2, 1 nodes
#pragma unroll
  for (int lv = 4; lv >= 0; lv--) {
    const int cntl = 1 << lv;
    const int base = (AT_THREADS >> (5 - lv)) + warp * cntl;  // first node of this warp on the level
    if (lane < cntl) {
      const int i = base + lane;
      i64 x = s.T[2 * i], y = s.T[2 * i + 1];
      s.T[i] = x > y ? x : y;
    }
    __syncwarp();
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int lv = 2; lv >= 0; lv--) {
      const int cntl = 1 << lv;
      if (lane < cntl) {
        const int i = cntl + lane;
        i64 x = s.T[2 * i], y = s.T[2 * i + 1];
        s.T[i] = x > y ? x : y;
      }
      __syncwarp();
    }
  }
  __syncthreads();

  // nearest earlier OP of the tile that is still running when the record starts
  unsigned bad = 0;
  i64 thr[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    const int x = x0 + j;
    int pl = AT_NONE;
    thr[j] = 0;
    if (hostmask & (1u << j)) {
      const i64 t = en[j] > st[j] ? st[j] + 1 : en[j];
      thr[j] = t;
      int y = -1;
      for (int k = x - 1; k >= x0; k--)
        if (s.leaf[k] >= t) { y = k; break; }
      if (y < 0) {
        int pos = AT_THREADS + tid;
        while (pos > 1) {
          if ((pos & 1) && s.T[pos - 1] >= t) {
            pos = pos - 1;
            while (pos < AT_THREADS) pos = s.T[2 * pos + 1] >= t ? 2 * pos + 1 : 2 * pos;
            const int tb = (pos - AT_THREADS) * AT_ITEMS;
            for (int k = tb + AT_ITEMS - 1; k >= tb; k--)
              if (s.leaf[k] >= t) { y = k; break; }
            break;
          }
          pos >>= 1;
        }
      }
      const int lo = lo_local[j];
      if (y >= 0 && y >= lo) {
        pl = y;
        if (s.leaf[y] < en[j]) bad |= 1u << j;
      } else {
        pl = lo >= 0 ? AT_NONE : AT_UNRESOLVED;
      }
    }
    s.parent_local[x] = (int16_t)pl;
  }

  // stack of the tile's last lane segment: OPs that no later OP of the tile dominates
  const int lane_last = s.lane1;
  const bool last_is_host = lane_last >= 0 && a.lane_domain[lane_last] == 0;
  if (last_is_host) {
    i64 sfx = INT64_MIN;
    int l = tid + 1 + AT_THREADS, r = 2 * AT_THREADS;
    while (l < r) {
      if (l & 1) { sfx = sfx > s.T[l] ? sfx : s.T[l]; l++; }
      if (r & 1) { --r; sfx = sfx > s.T[r] ? sfx : s.T[r]; }
      l >>= 1;
      r >>= 1;
    }
#pragma unroll
    for (int j = AT_ITEMS - 1; j >= 0; j--) {
      if ((hostmask & (1u << j)) && kd[j] == TA_KIND_OP) {
        if (ln[j] == lane_last && en[j] > sfx) {
          int o = atomicAdd(&s.agg_raw, 1);
          if (o < AT_CAP) { s.agg_e[o] = en[j]; s.agg_pos[o] = (int32_t)(p0 + j); }
        }
        sfx = sfx > en[j] ? sfx : en[j];
      }
    }
  }
  __syncthreads();

  if (warp == 0) {
    bool overflow = s.agg_raw > AT_CAP;
    WStack agg;
    agg.cnt = overflow ? AT_CAP : s.agg_raw;
    agg.reset = (!last_is_host || (int64_t)a.lane_off[lane_last] >= tile_start) ? 1 : 0;
    // order the surviving OPs by position (they were appended in arbitrary order)
    {
      const i64 me = lane < agg.cnt ? s.agg_e[lane] : 0;
      const int32_t mp = lane < agg.cnt ? s.agg_pos[lane] : INT_MAX;
      int rank = 0;
      for (int k = 0; k < agg.cnt; k++) rank += __shfl_sync(0xffffffffu, mp, k) < mp ? 1 : 0;
      __syncwarp();
      if (lane < agg.cnt) { s.agg_e[rank] = me; s.agg_pos[rank] = mp; }
      __syncwarp();
      agg.e = lane < agg.cnt ? s.agg_e[lane] : 0;
      agg.pos = lane < agg.cnt ? s.agg_pos[lane] : 0;
    }
    bool need_carry = false;
    if (tile > 0 && l0 >= 0) need_carry = a.lane_domain[l0] == 0 && (int64_t)a.lane_off[l0] < tile_start;
    if (agg.reset) publish_stack(a.pre_e, a.pre_pos, a.pre_meta, a.flag, tile, agg, TD_PREFIX);
    else publish_stack(a.agg_e, a.agg_pos, a.agg_meta, a.flag, tile, agg, TD_AGG);
    WStack acc;
    acc.cnt = 0; acc.reset = 0; acc.e = 0; acc.pos = 0;
    if (need_carry) {
      for (int t = tile - 1; t >= 0; --t) {
        u64 w = 0;
        int to = 0;
        if (lane == 0) {
          bool timed_out = false;
          w = td_wait(&a.flag[t], a.status, &timed_out);
          to = timed_out ? 1 : 0;
        }
        w = __shfl_sync(0xffffffffu, w, 0);
        to = __shfl_sync(0xffffffffu, to, 0);
        if (to) break;
        __threadfence();
        const bool is_prefix = (w >> 62) == TD_PREFIX;
        const int32_t meta = ld_relaxed_i32(is_prefix ? &a.pre_meta[t] : &a.agg_meta[t]);
        WStack ear;
        ear.cnt = meta & 0xFF;
        ear.reset = (meta >> 8) & 1;
        ear.e = 0; ear.pos = 0;
        if (lane < ear.cnt) {
          const i64 *pe = (is_prefix ? a.pre_e : a.agg_e) + (size_t)t * AT_CAP;
          const int32_t *pp = (is_prefix ? a.pre_pos : a.agg_pos) + (size_t)t * AT_CAP;
          ear.e = (i64)ld_relaxed((const u64 *)&pe[lane]);
          ear.pos = ld_relaxed_i32(&pp[lane]);
        }
        wstack_combine(ear, acc, &overflow);
        if (is_prefix || ear.reset) break;
      }
    }
    if (lane < acc.cnt) { s.carry_e[lane] = acc.e; s.carry_pos[lane] = acc.pos; }
    if (lane == 0) s.carry_cnt = acc.cnt;
    if (!agg.reset) {
      WStack incl = agg;
      wstack_combine(acc, incl, &overflow);
      publish_stack(a.pre_e, a.pre_pos, a.pre_meta, a.flag, tile, incl, TD_PREFIX);
    }
    if (overflow && lane == 0) ta_set_err(a.status, TA_ERR_DEPTH);
  }
  __syncthreads();

  // records whose encloser lies before the tile: look it up in the carried stack
  int32_t par_abs[AT_ITEMS];
  const int ccnt = s.carry_cnt;
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    const int x = x0 + j;
    par_abs[j] = -1;
    if (!(hostmask & (1u << j))) continue;
    const int pl = s.parent_local[x];
    if (pl >= 0) par_abs[j] = (int32_t)(tile_start + pl);
    else if (pl == AT_UNRESOLVED) {
      int k = 0;
      while (k < ccnt && s.carry_e[k] >= thr[j]) k++;
      s.kcarry[x] = (uint8_t)k;
      if (k > 0) {
        par_abs[j] = s.carry_pos[k - 1];
        if (s.carry_e[k - 1] < en[j]) bad |= 1u << j;
      }
    }
  }
  __syncthreads();
  int dmax = 0;
  uint8_t dep[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    int d = 0;
    if (hostmask & (1u << j)) {
      int c = x0 + j;
      for (int it = 0; it < 300; it++) {
        const int pl = s.parent_local[c];
        if (pl == AT_NONE) break;
        if (pl == AT_UNRESOLVED) { d += s.kcarry[c]; break; }
        d++;
        c = pl;
      }
      if (d > 255) d = 255;
      dmax = max(dmax, d);
      if (bad & (1u << j)) atomicOr(&a.sum[a.lane_window[ln[j]]].bad_nesting, 1);
    }
    dep[j] = (uint8_t)d;
  }
  if (full) {
    *reinterpret_cast<int4 *>(a.parent + p0) = make_int4(par_abs[0], par_abs[1], par_abs[2], par_abs[3]);
    *reinterpret_cast<int4 *>(a.parent + p0 + 4) = make_int4(par_abs[4], par_abs[5], par_abs[6], par_abs[7]);
    uint2 dq;
    dq.x = dep[0] | (dep[1] << 8) | (dep[2] << 16) | ((u32)dep[3] << 24);
    dq.y = dep[4] | (dep[5] << 8) | (dep[6] << 16) | ((u32)dep[7] << 24);
    *reinterpret_cast<uint2 *>(a.depth + p0) = dq;
  } else {
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++)
      if (p0 + j < a.n) { a.parent[p0 + j] = par_abs[j]; a.depth[p0 + j] = dep[j]; }
  }
  // per-window maximum depth (a tile rarely meets more than one window)
  const int w_first = l0 >= 0 ? a.lane_window[l0] : 0;
  const int w_last = lane_last >= 0 ? a.lane_window[lane_last] : w_first;
  if (w_first == w_last) {
    dmax = (int)warp_reduce((u64)dmax, OpMax());
    if (lane == 0 && dmax > 0) atomicMax(&s.dmax, dmax);
    __syncthreads();
    if (tid == 0 && s.dmax > 0) atomicMax(&a.sum[w_first].max_depth, s.dmax);
  } else {
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++)
      if ((hostmask & (1u << j)) && dep[j]) atomicMax(&a.sum[a.lane_window[ln[j]]].max_depth, (int)dep[j]);
  }
}

// ---- device records inherit the operator of their launch ------------------------
__global__ void __launch_bounds__(512) k_attr_ops(AttrArgs a) {
  __shared__ u64 tmp[33];
  __shared__ int s_lo, s_hi;
  const int64_t p0 = ((int64_t)blockIdx.x * 512 + threadIdx.x) * 4;
  LaneWalker lw(a.lane_off, a.n_lanes, p0, a.n_valid);
  int ln[4];
  int cls[4];  // 0 none, 1 attributed, 2 no launch, 3 no op
  int my_lo = INT_MAX, my_hi = -1;
#pragma unroll
  for (int j = 0; j < 4; j++) {
    int64_t p = p0 + j;
    ln[j] = -1;
    cls[j] = 0;
    if (p >= a.n) continue;
    int32_t op = -1;
    if (p < a.n_valid) {
      int k = a.kind[p];
      if (k == TA_KIND_KERNEL || k == TA_KIND_MEMCPY) {
        ln[j] = lw.at(p);
        my_lo = min(my_lo, ln[j]);
        my_hi = max(my_hi, ln[j]);
        int32_t l = a.launch_of[p];
        if (l < 0) cls[j] = 2;
        else {
          op = a.parent[l];
          if (op < 0) cls[j] = 3;
          else {
            cls[j] = 1;
            i64 s = a.ts[p], e = a.te[p];
            atomicAdd(&a.op_n[op], 1);
            atomicAdd((u64 *)&a.op_ns[op], (u64)(e - s));
            atomicMax(&a.op_first[op], ~((u64)s ^ (1ull << 63)));
            atomicMax(&a.op_last[op], (u64)e ^ (1ull << 63));
          }
        }
      }
    }
    a.op_of[p] = op;
  }
  if (threadIdx.x == 0) { s_lo = INT_MAX; s_hi = -1; }
  __syncthreads();
  if (my_hi >= 0) { atomicMin(&s_lo, my_lo); atomicMax(&s_hi, my_hi); }
  __syncthreads();
  const int l0 = s_lo, l1 = s_hi;
  for (int l = l0; l <= l1; l++) {
    if (a.lane_domain[l] != 1) continue;
    u64 c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
    for (int j = 0; j < 4; j++)
      if (ln[j] == l) { c1 += cls[j] == 1; c2 += cls[j] == 2; c3 += cls[j] == 3; }
    u64 packed = c1 | (c2 << 20) | (c3 << 40);  // each < 2^20 per tile
    u64 v = warp_reduce(packed, OpAdd());
    __syncthreads();
    if ((threadIdx.x & 31) == 0) tmp[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
      u64 t = 0;
      for (int w = 0; w < 16; w++) t += tmp[w];
      ta_attr_summary *s = &a.sum[a.lane_window[l]];
      u64 m = (1ull << 20) - 1;
      if (t & m) atomicAdd((u64 *)&s->n_attributed, t & m);
      if ((t >> 20) & m) atomicAdd((u64 *)&s->n_no_launch, (t >> 20) & m);
      if ((t >> 40) & m) atomicAdd((u64 *)&s->n_no_op, (t >> 40) & m);
    }
    __syncthreads();
  }
}

// first/last were accumulated in an order-preserving unsigned encoding (0 = untouched)
__global__ void __launch_bounds__(256) k_attr_finalize(AttrArgs a) {
  int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= a.n_valid || a.kind[p] != TA_KIND_OP) return;
  if (a.op_n[p] > 0) {
    a.op_first[p] = (~a.op_first[p]) ^ (1ull << 63);
    a.op_last[p] = a.op_last[p] ^ (1ull << 63);
  }
}

ta_status ta_run_attribute(ta_window *h, ta_attr_summary *out_summary) {
  const int64_t n = h->n, nn = n > 0 ? n : 1;
  const int W = h->W;
  cudaStream_t st = h->stream;
  const int64_t tiles = (n + AT_TILE - 1) / AT_TILE;
  size_t keep = 3 * Carver::pad(nn * 4) + Carver::pad(nn) + 3 * Carver::pad(nn * 8) +
                Carver::pad((size_t)W * sizeof(ta_attr_summary)) + 256;
  void *kb = ta_dalloc(h, keep);
  if (!kb) return TA_ERR_OOM;
  Carver ck(kb);
  int32_t *parent = ck.take<int32_t>(nn), *op_of = ck.take<int32_t>(nn);
  uint8_t *depth = ck.take<uint8_t>(nn);
  char *zero_begin = ck.base + ck.off;
  int32_t *op_n = ck.take<int32_t>(nn);
  u64 *op_first = ck.take<u64>(nn), *op_last = ck.take<u64>(nn);
  int64_t *op_ns = ck.take<int64_t>(nn);
  ta_attr_summary *d_sum = ck.take<ta_attr_summary>(W);
  char *zero_end = ck.base + ck.off;
  TA_CHECK_CUDA(h, cudaMemsetAsync(zero_begin, 0, zero_end - zero_begin, st));

  const int64_t tt = tiles > 0 ? tiles : 1;
  size_t tb = Carver::pad(tt * 8) + 2 * Carver::pad(tt * 4) + 2 * Carver::pad(tt * AT_CAP * 8) +
              2 * Carver::pad(tt * AT_CAP * 4) + Carver::pad(64) + 256;
  void *tmpb = ta_dalloc(h, tb);
  if (!tmpb) return TA_ERR_OOM;
  Carver ct(tmpb);
  AttrArgs a;
  memset(&a, 0, sizeof(a));
  a.flag = ct.take<u64>(tt);
  a.agg_meta = ct.take<int32_t>(tt);
  a.pre_meta = ct.take<int32_t>(tt);
  a.counter = ct.take<u32>(16);
  const size_t zero_bytes = ct.off;  // flags, metas and the counter start at zero; payloads need not
  a.agg_e = ct.take<i64>(tt * AT_CAP);
  a.pre_e = ct.take<i64>(tt * AT_CAP);
  a.agg_pos = ct.take<int32_t>(tt * AT_CAP);
  a.pre_pos = ct.take<int32_t>(tt * AT_CAP);
  TA_CHECK_CUDA(h, cudaMemsetAsync(tmpb, 0, zero_bytes, st));

  a.n = n; a.n_valid = h->n_valid; a.n_lanes = h->sorted.n_lanes;
  a.kind = h->sorted.kind; a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window;
  a.lane_domain = h->sorted.lane_domain;
  a.parent = parent; a.depth = depth; a.sum = d_sum; a.status = h->d_status;
  a.launch_of = h->join.launch_of; a.op_of = op_of; a.op_n = op_n; a.op_first = op_first;
  a.op_last = op_last; a.op_ns = op_ns;
  if (n > 0) {
    k_attr<<<TA_N (unsigned)tiles, AT_THREADS, 0, st>>>(a);
    k_attr_ops<<<TA_N (unsigned)((n + 2047) / 2048), 512, 0, st>>>(a);
    const int64_t fb = (h->n_valid + 255) / 256;
    k_attr_finalize<<<TA_N (unsigned)(fb > 0 ? fb : 1), 256, 0, st>>>(a);
    TA_CHECK_CUDA(h, cudaGetLastError());
  }
  std::vector<ta_attr_summary> hs(W);
  TA_CHECK_CUDA(h, cudaMemcpyAsync(hs.data(), d_sum, W * sizeof(ta_attr_summary), cudaMemcpyDeviceToHost, st));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  ta_dfree(h, tmpb);
  bool any_bad = false, any_deep = words[ST_ERR] == TA_ERR_DEPTH;
  if (words[ST_ERR] && words[ST_ERR] != TA_ERR_DEPTH) return (ta_status)words[ST_ERR];
  if (any_deep)  // a data error of this call only: later calls start with a clean status word
    TA_CHECK_CUDA(h, cudaMemsetAsync(h->d_status, 0, sizeof(int32_t), st));
  for (int w = 0; w < W; w++) {
    if (hs[w].bad_nesting) any_bad = true;
    if (hs[w].max_depth > TA_MAX_DEPTH) any_deep = true;
    if (out_summary) out_summary[w] = hs[w];
  }
  h->attr.parent = parent;
  h->attr.depth = depth;
  h->attr.op_of = op_of;
  h->attr.op_first_start = (const int64_t *)op_first;
  h->attr.op_last_end = (const int64_t *)op_last;
  h->attr.op_kernel_ns = op_ns;
  h->attr.op_n_kernels = op_n;
  if (any_bad) return TA_ERR_BAD_NESTING;
  if (any_deep) return TA_ERR_DEPTH;
  return TA_OK;
}
