// ta_attribute_operators: every host record gets the operator range of its own
// thread that contains it (same thread, nested intervals: the linkage of Sec. 9.1);
// device records inherit the operator of their launch; per operator, T_op runs from
// the start of its first kernel to the end of its last (Sec. 6.1).
//
// In canonical order (ts_start ascending, ts_end descending) a properly nested
// host lane has a simple structure: the innermost encloser of record i is the
// nearest earlier OP that is still running when i starts.  Tiles of 2048
// records (256 threads x 8 consecutive records), three kernels, no kernel ever
// waits for another CTA:
//   k_attr_agg     per tile, the stack of OPs that are still undominated at the
//                  tile's end (at most TA_MAX_DEPTH + 1 entries when nesting is
//                  legal);
//   k_attr_fold_*  an exclusive scan of those stacks under the stack monoid (one
//                  stack entry per warp lane; entries that end no later than a
//                  later tile's outermost surviving OP are dropped; a tile whose
//                  last lane starts inside it cuts off what came before), as a
//                  fan-out-32 tree, leaves every tile the stack open at its start;
//   k_attr_resolve per record: a backward look over the thread's own records,
//                  else one descent of a max-tree over the threads' largest OP
//                  end times in shared memory, else the carried stack.
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
// 4 or 8 records per thread in the stack and resolve kernels: with four the resolve kernel fits
// 64 registers and 16 KB of shared memory, four CTAs per SM (eight and three: 0.12 ms slower)
#ifndef AT_ITEMS
#define AT_ITEMS 4
#endif
#define AT_TILE (AT_THREADS * AT_ITEMS)
#define AT_CAP 16
#ifndef AT_RES_MINB
#define AT_RES_MINB 4
#endif
// k_attr_ops: four records per thread keep it at 64 registers, four CTAs per SM (eight records and
// three CTAs measured 0.12 ms slower on the 66.8 M record window: the kernel waits on gathers)
#ifndef AT_OPS_MINB
#define AT_OPS_MINB 4
#endif
#define AT_NONE (-1)
#define AT_UNRESOLVED (-2)

struct AttrArgs {
  int64_t n, n_valid;
  int n_lanes;
  int64_t n_tiles;
  const int16_t *kind;
  const int64_t *ts, *te;
  const int32_t *lane_off, *lane_window, *lane_dom_end;
  const int16_t *lane_domain;
  int32_t *parent;
  uint8_t *depth;
  ta_attr_summary *sum;
  // per tile: stack at the tile's end (agg) and stack open at its start (carry)
  int32_t *agg_meta, *carry_cnt;  // agg_meta = count | reset << 8
  i64 *agg_e, *carry_e;           // [tile][AT_CAP]
  int32_t *agg_pos, *carry_pos;
  int32_t *status;
  const int32_t *kol;  // kernels of each launch (from the join)
  // k_attr_ops
  const int32_t *launch_of;
  int32_t *op_of, *op_n;
  u64 *op_first, *op_last;
  int64_t *op_ns;
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
    // an earlier OP that ends exactly when the outermost later one does still encloses it
    keep = __popc(__ballot_sync(0xffffffffu, lane < ear.cnt && ear.e >= e0));
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



// ---- kernel 1: the stack each tile leaves behind --------------------------------
__global__ void __launch_bounds__(AT_THREADS) k_attr_agg(AttrArgs a) {
  __shared__ i64 wmax[AT_THREADS / 32];
  __shared__ i64 s_e[AT_CAP];
  __shared__ int32_t s_pos[AT_CAP];
  __shared__ int s_raw, s_lane1;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = blockIdx.x;
  const int64_t tile_start = (int64_t)tile * AT_TILE;
  const int64_t p0 = tile_start + (int64_t)tid * AT_ITEMS;
  const int64_t plast = min(tile_start + AT_TILE, a.n_valid) - 1;
  if (tid == 0) s_raw = 0;
  if (warp == 0) {
    int l = -1;
    if (plast >= tile_start) l = tile_lane_search(a.lane_off, a.n_lanes, plast);
    if (lane == 0) s_lane1 = l;
  }
  int16_t kd[AT_ITEMS];
  loadn_i16<AT_ITEMS>(a.kind, p0, a.n, 9, kd);
  __syncthreads();
  const int lane1 = s_lane1;
  if (lane1 < 0 || a.lane_domain[lane1] != 0) {
    if (tid == 0) a.agg_meta[tile] = 1 << 8;  // nothing carried past a device lane
    return;
  }
  const int64_t seg_begin = a.lane_off[lane1];  // first record of the tile's last lane
  unsigned opmask = 0;
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++)
    if (kd[j] == TA_KIND_OP && p0 + j <= plast && p0 + j >= seg_begin) opmask |= 1u << j;
  i64 en[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) en[j] = INT64_MIN;
  i64 m8 = INT64_MIN;
  if (opmask) {
    i64 t[AT_ITEMS];
    loadn_i64<AT_ITEMS>(a.te, p0, a.n, t);
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++)
      if (opmask & (1u << j)) { en[j] = t[j]; m8 = m8 > t[j] ? m8 : t[j]; }
  }
  // largest OP end among the threads after this one
  i64 after = INT64_MIN;
  {
    i64 v = m8;  // inclusive suffix max inside the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      i64 t = __shfl_down_sync(0xffffffffu, v, o);
      if (lane + o < 32) v = v > t ? v : t;
    }
    if (lane == 0) wmax[warp] = v;
    i64 nxt = __shfl_down_sync(0xffffffffu, v, 1);
    after = lane < 31 ? nxt : INT64_MIN;
    __syncthreads();
    for (int w = warp + 1; w < AT_THREADS / 32; w++) after = after > wmax[w] ? after : wmax[w];
  }
  i64 sfx = after;
#pragma unroll
  for (int j = AT_ITEMS - 1; j >= 0; j--) {
    if (opmask & (1u << j)) {
      if (en[j] >= sfx) {  // equal ends nest: the earlier OP encloses the later one
        int o = atomicAdd(&s_raw, 1);
        if (o < AT_CAP) { s_e[o] = en[j]; s_pos[o] = (int32_t)(p0 + j); }
      }
      sfx = sfx > en[j] ? sfx : en[j];
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int raw = s_raw;
    const int cnt = raw > AT_CAP ? AT_CAP : raw;
    if (raw > AT_CAP && lane == 0) ta_set_err(a.status, TA_ERR_DEPTH);
    // survivors were appended in arbitrary order: rank them by position
    const i64 me = lane < cnt ? s_e[lane] : 0;
    const int32_t mp = lane < cnt ? s_pos[lane] : INT_MAX;
    int rank = 0;
    for (int k = 0; k < cnt; k++) rank += __shfl_sync(0xffffffffu, mp, k) < mp ? 1 : 0;
    if (lane < cnt) {
      a.agg_e[(size_t)tile * AT_CAP + rank] = me;
      a.agg_pos[(size_t)tile * AT_CAP + rank] = mp;
    }
    if (lane == 0) a.agg_meta[tile] = cnt | ((seg_begin >= tile_start ? 1 : 0) << 8);
  }
}

// ---- kernel 2: the stack open at the start of every tile --------------------------
// An exclusive scan of the tile stacks under the stack monoid (wstack_combine; a stack whose
// reset flag is set cuts off everything before it, which is how lanes stay apart).  One fold
// over all tiles would be a serial chain as long as the longest host lane, so it is done as a
// tree with fan-out 32: fold groups of 32 stacks upwards until at most 32 remain, scan those
// with one warp, then unfold downwards.  Every step is one warp working through 32 staged
// stacks; no kernel waits for another.
struct StackArr {
  int32_t *meta;  // count | reset << 8
  i64 *e;
  int32_t *pos;
};
#define AT_FAN 32
struct StackStage {
  i64 e[4][AT_FAN][AT_CAP];
  int32_t pos[4][AT_FAN][AT_CAP];
  int meta[4][AT_FAN];
};
// lane i of the warp copies stack first + i into the stage (count 0 beyond n)
__device__ __forceinline__ void stack_stage(const StackArr &src, int64_t first, int64_t n, StackStage &st,
                                            int warp, int lane) {
  const int64_t t = first + lane;
  int m = 0;
  if (t < n) {
    m = src.meta[t];
    const int c = m & 0xFF;
#pragma unroll
    for (int k = 0; k < AT_CAP; k++)
      if (k < c) {
        st.e[warp][lane][k] = src.e[(size_t)t * AT_CAP + k];
        st.pos[warp][lane][k] = src.pos[(size_t)t * AT_CAP + k];
      }
  }
  st.meta[warp][lane] = m;
  __syncwarp();
}
__device__ __forceinline__ WStack stack_staged(const StackStage &st, int warp, int i, int lane) {
  WStack x;
  const int m = st.meta[warp][i];
  x.cnt = m & 0xFF;
  x.reset = (m >> 8) & 1;
  x.e = lane < x.cnt ? st.e[warp][i][lane] : 0;
  x.pos = lane < x.cnt ? st.pos[warp][i][lane] : 0;
  return x;
}
__device__ __forceinline__ WStack stack_load(const StackArr &src, int64_t t, int lane) {
  WStack x;
  const int m = src.meta[t];
  x.cnt = m & 0xFF;
  x.reset = (m >> 8) & 1;
  x.e = lane < x.cnt ? src.e[(size_t)t * AT_CAP + lane] : 0;
  x.pos = lane < x.cnt ? src.pos[(size_t)t * AT_CAP + lane] : 0;
  return x;
}
__device__ __forceinline__ void stack_store(const StackArr &dst, int64_t t, const WStack &x, int lane,
                                            bool count_only) {
  if (lane < x.cnt) {
    dst.e[(size_t)t * AT_CAP + lane] = x.e;
    dst.pos[(size_t)t * AT_CAP + lane] = x.pos;
  }
  if (lane == 0) dst.meta[t] = count_only ? x.cnt : (x.cnt | (x.reset << 8));
}

// parent[j] = child[32j] (+) ... (+) child[32j + 31]
__global__ void __launch_bounds__(128) k_attr_fold_up(StackArr child, int64_t n_child, StackArr parent,
                                                      int64_t n_parent, int32_t *status) {
  __shared__ StackStage st;
  if (ta_failed(status)) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t j = (int64_t)blockIdx.x * 4 + warp;
  if (j >= n_parent) return;
  stack_stage(child, j * AT_FAN, n_child, st, warp, lane);
  bool overflow = false;
  WStack acc;
  acc.cnt = 0; acc.reset = 0; acc.e = 0; acc.pos = 0;
  const int cnt = (int)min((int64_t)AT_FAN, n_child - j * AT_FAN);
  for (int i = 0; i < cnt; i++) {
    WStack nxt = stack_staged(st, warp, i, lane);
    wstack_combine(acc, nxt, &overflow);
    acc = nxt;
  }
  stack_store(parent, j, acc, lane, false);
  if (overflow && lane == 0) ta_set_err(status, TA_ERR_DEPTH);
}

// one warp: start[i] = node[0] (+) ... (+) node[i - 1] for the few nodes of the top level
__global__ void __launch_bounds__(32) k_attr_fold_top(StackArr node, int64_t n, StackArr start,
                                                      int leaf, int32_t *status) {
  if (ta_failed(status)) return;
  const int lane = threadIdx.x & 31;
  bool overflow = false;
  WStack acc;
  acc.cnt = 0; acc.reset = 0; acc.e = 0; acc.pos = 0;
  for (int64_t i = 0; i < n; i++) {
    stack_store(start, i, acc, lane, leaf != 0);
    WStack nxt = stack_load(node, i, lane);
    wstack_combine(acc, nxt, &overflow);
    acc = nxt;
  }
  if (overflow && lane == 0) ta_set_err(status, TA_ERR_DEPTH);
}

// child_start[32j + i] = parent_start[j] (+) child[32j] (+) ... (+) child[32j + i - 1]
__global__ void __launch_bounds__(128) k_attr_fold_down(StackArr child, int64_t n_child,
                                                        StackArr parent_start, int64_t n_parent,
                                                        StackArr child_start, int leaf, int32_t *status) {
  __shared__ StackStage st;
  if (ta_failed(status)) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t j = (int64_t)blockIdx.x * 4 + warp;
  if (j >= n_parent) return;
  stack_stage(child, j * AT_FAN, n_child, st, warp, lane);
  bool overflow = false;
  WStack acc = stack_load(parent_start, j, lane);
  const int cnt = (int)min((int64_t)AT_FAN, n_child - j * AT_FAN);
  for (int i = 0; i < cnt; i++) {
    stack_store(child_start, j * AT_FAN + i, acc, lane, leaf != 0);
    WStack nxt = stack_staged(st, warp, i, lane);
    wstack_combine(acc, nxt, &overflow);
    acc = nxt;
  }
  if (overflow && lane == 0) ta_set_err(status, TA_ERR_DEPTH);
}

// ---- kernel 3: parent and depth of every host record -----------------------------
// a thread's eight leaves are followed by one pad entry: the threads of a warp then touch
// distinct banks when each walks its own records
#define AT_LX(x) ((x) + ((x) >> 3))
struct __align__(16) AttrSmem {
  i64 leaf[AT_TILE + AT_TILE / 8];  // OP end time, INT64_MIN elsewhere; index through AT_LX
  i64 T[2 * AT_THREADS];          // max-tree over the threads' maxima, leaves at [AT_THREADS, 2*AT_THREADS)
  int16_t parent_local[AT_TILE];
  uint8_t kcarry[AT_TILE];
  i64 carry_e[AT_CAP];
  int32_t carry_pos[AT_CAP];
  int lane0, lane1, dmax;
};

__global__ void __launch_bounds__(AT_THREADS, AT_RES_MINB) k_attr_resolve(AttrArgs a) {
  __shared__ AttrSmem s;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = blockIdx.x;
  const int64_t tile_start = (int64_t)tile * AT_TILE;
  const int x0 = tid * AT_ITEMS;
  const int64_t p0 = tile_start + x0;
  const bool full = p0 + AT_ITEMS <= a.n;
  if (tid == 0) { s.lane1 = -1; s.dmax = 0; s.lane0 = -1; }
  __syncthreads();
  if (warp == 0 && tile_start < a.n_valid && a.n_lanes > 0) {
    int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (lane == 0) s.lane0 = l;
  }
  const int ccnt = a.carry_cnt[tile];
  if (tid < ccnt) {
    s.carry_e[tid] = a.carry_e[(size_t)tile * AT_CAP + tid];
    s.carry_pos[tid] = a.carry_pos[(size_t)tile * AT_CAP + tid];
  }
  __syncthreads();
  const int l0 = s.lane0;
  // A tile of device lanes holds no host record: parent -1, depth 0 throughout, nothing read.
  if (l0 < 0 || span_outside_domain(a.lane_domain, a.lane_dom_end, l0, min(tile_start + AT_TILE, a.n_valid), 0)) {
    if (full) {
#pragma unroll
      for (int q = 0; q < AT_ITEMS / 4; q++) {
        *reinterpret_cast<int4 *>(a.parent + p0 + 4 * q) = make_int4(-1, -1, -1, -1);
        *reinterpret_cast<u32 *>(a.depth + p0 + 4 * q) = 0u;
      }
    } else {
      for (int j = 0; j < AT_ITEMS; j++)
        if (p0 + j < a.n) { a.parent[p0 + j] = -1; a.depth[p0 + j] = 0; }
    }
    return;
  }
  // kinds and both times of the thread's records are requested together (the tile holds a host
  // lane, so nearly every record needs its times)
  int16_t kd[AT_ITEMS];
  i64 st[AT_ITEMS], en[AT_ITEMS];
  loadn_i16<AT_ITEMS>(a.kind, p0, a.n, 9, kd);
  loadn_i64<AT_ITEMS>(a.ts, p0, a.n, st);
  loadn_i64<AT_ITEMS>(a.te, p0, a.n, en);
  int32_t nk[AT_ITEMS];  // kernels of the thread's launches (0 elsewhere)
  if (full) {
#pragma unroll
    for (int q = 0; q < AT_ITEMS / 4; q++) {
      const int4 x = *reinterpret_cast<const int4 *>(a.kol + p0 + 4 * q);
      nk[4 * q] = x.x; nk[4 * q + 1] = x.y; nk[4 * q + 2] = x.z; nk[4 * q + 3] = x.w;
    }
  } else {
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++) nk[j] = p0 + j < a.n ? a.kol[p0 + j] : 0;
  }
  unsigned hostmask = 0;
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++)
    if (p0 + j < a.n_valid && kd[j] <= TA_KIND_LAUNCH) hostmask |= 1u << j;
  // lanes, leaves, the thread's maximum
  int ln[AT_ITEMS];
  int lo_local[AT_ITEMS];  // first tile-local index of the record's lane (-1: the lane began earlier)
  i64 m8 = INT64_MIN;
  unsigned opmask = 0;  // the thread's own OP records (its leaves are their en[])
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
        if (kd[j] == TA_KIND_OP) { leaf = en[j]; opmask |= 1u << j; }
      }
      s.leaf[AT_LX(x0 + j)] = leaf;
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

  // nearest earlier OP that is still running when the record starts.  Consecutive records
  // mostly share it: when the threshold t did not go down since the previous record, nothing
  // between the previous answer and that record can qualify, so the previous answer (or the
  // fact that the tile holds none) is reused and the tree is only walked when it has ended.
  unsigned bad = 0;
  int32_t par_abs[AT_ITEMS];
  int16_t plv[AT_ITEMS];
  uint8_t kc[AT_ITEMS];
  bool have = false;  // (tq, yq, yeq): threshold and answer of the previous search outside the thread
  i64 tq = 0, yeq = 0;
  int yq = -1;
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    const int x = x0 + j;
    int pl = AT_NONE;
    par_abs[j] = -1;
    kc[j] = 0;
    if (hostmask & (1u << j)) {
      const i64 t = en[j] > st[j] ? st[j] + 1 : en[j];
      int y = -1;
      i64 ye = 0;  // end time of y
#pragma unroll
      for (int jj = AT_ITEMS - 1; jj >= 0; jj--)
        if (jj < j && y < 0 && (opmask & (1u << jj)) && en[jj] >= t) { y = x0 + jj; ye = en[jj]; }
      if (y < 0) {
        if (have && t >= tq && (yq < 0 || yeq >= t)) {
          y = yq;
          ye = yeq;
        } else {
          int pos = AT_THREADS + tid;
          while (pos > 1) {
            if ((pos & 1) && s.T[pos - 1] >= t) {
              pos = pos - 1;
              while (pos < AT_THREADS) pos = s.T[2 * pos + 1] >= t ? 2 * pos + 1 : 2 * pos;
              const int tb = (pos - AT_THREADS) * AT_ITEMS;
              for (int k = tb + AT_ITEMS - 1; k >= tb; k--) {
                ye = s.leaf[AT_LX(k)];
                if (ye >= t) { y = k; break; }
              }
              break;
            }
            pos >>= 1;
          }
          have = true;
          yq = y;
          yeq = ye;
        }
        tq = t;
      }
      const int lo = lo_local[j];
      if (y >= 0 && y >= lo) {
        pl = y;
        par_abs[j] = (int32_t)(tile_start + y);
        if (ye < en[j]) bad |= 1u << j;
      } else if (lo >= 0) {
        pl = AT_NONE;
      } else {  // the encloser, if any, lies before the tile: the carried stack has it
        pl = AT_UNRESOLVED;
        int k = 0;
        while (k < ccnt && s.carry_e[k] >= t) k++;
        s.kcarry[x] = (uint8_t)k;
        kc[j] = (uint8_t)k;
        if (k > 0) {
          par_abs[j] = s.carry_pos[k - 1];
          if (s.carry_e[k - 1] < en[j]) bad |= 1u << j;
        }
      }
    }
    plv[j] = (int16_t)pl;
  }
  // Kernels per operator: an operator owns the kernels of the launches directly inside it, and
  // the join has counted the kernels of every launch, so the counts are added up here, from
  // the launch side - consecutive launches mostly share their operator, and one add serves a
  // run of them - instead of one atomic per kernel from the device side.
  {
    int32_t run_par = -1, run_cnt = 0;
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++) {
      if (!(hostmask & (1u << j)) || kd[j] != TA_KIND_LAUNCH || par_abs[j] < 0 || nk[j] <= 0) continue;
      if (par_abs[j] != run_par) {
        if (run_cnt) atomicAdd(&a.op_n[run_par], run_cnt);
        run_par = par_abs[j];
        run_cnt = 0;
      }
      run_cnt += nk[j];
    }
    if (run_cnt) atomicAdd(&a.op_n[run_par], run_cnt);
  }
#pragma unroll
  for (int q = 0; q < AT_ITEMS / 2; q++)
    *reinterpret_cast<u32 *>(&s.parent_local[x0 + 2 * q]) =
        (u32)(uint16_t)plv[2 * q] | ((u32)(uint16_t)plv[2 * q + 1] << 16);
  __syncthreads();
  // depth = level in the parent forest; the chain is only followed through shared memory when
  // the parent is another thread's record and differs from the previous record's parent
  int dmax = 0;
  uint8_t dep[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    int d = 0;
    if (hostmask & (1u << j)) {
      const int pl = plv[j];
      if (pl == AT_UNRESOLVED) {
        d = kc[j];
      } else if (pl >= x0) {  // one of the thread's own earlier records
#pragma unroll
        for (int jj = 0; jj < AT_ITEMS; jj++)
          if (jj < j && pl == x0 + jj) d = dep[jj] + 1;
      } else if (pl >= 0) {
        if (j > 0 && (hostmask & (1u << (j > 0 ? j - 1 : 0))) && plv[j > 0 ? j - 1 : 0] == pl) {
          d = dep[j > 0 ? j - 1 : 0];
        } else {
          d = 1;
          int c = pl;
          for (int it = 0; it < 300; it++) {
            const int q = s.parent_local[c];
            if (q == AT_NONE) break;
            if (q == AT_UNRESOLVED) { d += s.kcarry[c]; break; }
            d++;
            c = q;
          }
        }
      }
      if (d > 255) d = 255;
      dmax = max(dmax, d);
      if (bad & (1u << j)) atomicOr(&a.sum[a.lane_window[ln[j]]].bad_nesting, 1);
    }
    dep[j] = (uint8_t)d;
  }
  if (full) {
#pragma unroll
    for (int q = 0; q < AT_ITEMS / 4; q++) {
      *reinterpret_cast<int4 *>(a.parent + p0 + 4 * q) =
          make_int4(par_abs[4 * q], par_abs[4 * q + 1], par_abs[4 * q + 2], par_abs[4 * q + 3]);
      *reinterpret_cast<u32 *>(a.depth + p0 + 4 * q) =
          dep[4 * q] | (dep[4 * q + 1] << 8) | (dep[4 * q + 2] << 16) | ((u32)dep[4 * q + 3] << 24);
    }
  } else {
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++)
      if (p0 + j < a.n) { a.parent[p0 + j] = par_abs[j]; a.depth[p0 + j] = dep[j]; }
  }
  // per-window maximum depth (a tile rarely meets more than one window)
  const int lane_last = s.lane1;
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
#ifndef AT_OPS_ITEMS
#define AT_OPS_ITEMS 4
#endif
#define AT_OPS_TILE (AT_THREADS * AT_OPS_ITEMS)
__global__ void __launch_bounds__(AT_THREADS, AT_OPS_MINB) k_attr_ops(AttrArgs a) {
  constexpr int IT = AT_OPS_ITEMS;
  __shared__ u64 red[AT_THREADS / 32];
  __shared__ int s_lane0, s_lane1;
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t tile_start = (int64_t)blockIdx.x * AT_OPS_TILE;
  const int64_t p0 = tile_start + (int64_t)tid * IT;
  if (tid == 0) { s_lane0 = -1; s_lane1 = -1; }
  __syncthreads();
  if (tid < 32 && tile_start < a.n_valid && a.n_lanes > 0) {
    int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (lane == 0) s_lane0 = l;
  }
  __syncthreads();
  const int l0 = s_lane0;
  // A tile of host lanes holds no device record: nothing to read, op_of = -1 throughout.
  if (l0 >= 0 && span_outside_domain(a.lane_domain, a.lane_dom_end, l0,
                                     min(tile_start + AT_OPS_TILE, a.n_valid), 1)) {
    if (p0 + IT <= a.n) {
#pragma unroll
      for (int q = 0; q < IT / 4; q++) *reinterpret_cast<int4 *>(a.op_of + p0 + 4 * q) = make_int4(-1, -1, -1, -1);
    } else {
      for (int j = 0; j < IT; j++)
        if (p0 + j < a.n) a.op_of[p0 + j] = -1;
    }
    return;
  }
  // kinds, launches and times of the thread's records are requested together (launch_of is -1
  // wherever the record is no matched kernel or copy, so the gather below needs no kind), then
  // the parents of the launches: two rounds of memory latency instead of three
  int16_t kd[IT];
  loadn_i16<IT>(a.kind, p0, a.n, 0, kd);
  int32_t lo[IT], op[IT];
  i64 st[IT], en[IT];
#pragma unroll
  for (int j = 0; j < IT; j++) { lo[j] = -1; op[j] = -1; st[j] = en[j] = 0; }
  if (p0 + IT <= a.n) {
#pragma unroll
    for (int q = 0; q < IT / 4; q++) {
      const int4 x = *reinterpret_cast<const int4 *>(a.launch_of + p0 + 4 * q);
      lo[4 * q] = x.x; lo[4 * q + 1] = x.y; lo[4 * q + 2] = x.z; lo[4 * q + 3] = x.w;
    }
    const longlong2 *ps = reinterpret_cast<const longlong2 *>(a.ts + p0);
    const longlong2 *pe = reinterpret_cast<const longlong2 *>(a.te + p0);
#pragma unroll
    for (int q = 0; q < IT / 2; q++) {
      const longlong2 x = ps[q], y = pe[q];
      st[2 * q] = x.x; st[2 * q + 1] = x.y;
      en[2 * q] = y.x; en[2 * q + 1] = y.y;
    }
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++)
      if (p0 + j < a.n) { lo[j] = a.launch_of[p0 + j]; st[j] = a.ts[p0 + j]; en[j] = a.te[p0 + j]; }
  }
#pragma unroll
  for (int j = 0; j < IT; j++)
    if (lo[j] >= 0) op[j] = a.parent[lo[j]];
  unsigned pm = 0;
#pragma unroll
  for (int j = 0; j < IT; j++)
    if (p0 + j < a.n_valid && (kd[j] == TA_KIND_KERNEL || kd[j] == TA_KIND_MEMCPY)) pm |= 1u << j;
  u64 packed = 0;  // attributed | no launch << 20 | no op << 40, for the thread's first lane
  int lm = -1;
  {
    int l = l0;
    int64_t next_off = l >= 0 ? (int64_t)a.lane_off[l + 1] : LLONG_MAX;
#pragma unroll
    for (int j = 0; j < IT; j++) {
      if (!(pm & (1u << j))) { op[j] = -1; continue; }
      const int64_t p = p0 + j;
      while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      u64 add;
      if (lo[j] < 0) add = 1ull << 20;
      else if (op[j] < 0) add = 1ull << 40;
      else {
        add = 1ull;
        const int32_t r = op[j];
        // (the kernel count of the operator is accumulated from the launch side, in k_attr_resolve)
        atomicAdd((u64 *)&a.op_ns[r], (u64)(en[j] - st[j]));
        atomicMax(&a.op_first[r], ~((u64)st[j] ^ (1ull << 63)));
        atomicMax(&a.op_last[r], (u64)en[j] ^ (1ull << 63));
      }
      if (lm < 0) lm = l;
      if (l == lm && l - l0 <= 1) packed += add;
      else {
        ta_attr_summary *sm = &a.sum[a.lane_window[l]];
        if (add == 1ull) atomicAdd((u64 *)&sm->n_attributed, 1ull);
        else if (add == (1ull << 20)) atomicAdd((u64 *)&sm->n_no_launch, 1ull);
        else atomicAdd((u64 *)&sm->n_no_op, 1ull);
      }
    }
    const int64_t plast = min(tile_start + AT_OPS_TILE, a.n_valid) - 1;
    if (plast >= p0 && plast < p0 + IT) {
      while (plast >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      s_lane1 = l;
    }
  }
  if (p0 + IT <= a.n) {
#pragma unroll
    for (int q = 0; q < IT / 4; q++)
      *reinterpret_cast<int4 *>(a.op_of + p0 + 4 * q) = make_int4(op[4 * q], op[4 * q + 1], op[4 * q + 2], op[4 * q + 3]);
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++)
      if (p0 + j < a.n) a.op_of[p0 + j] = op[j];
  }
  __syncthreads();
  const int l1 = s_lane1;
  for (int li = 0; li < 2; li++) {
    const int l = l0 + li;
    if (l0 < 0 || l > l1) break;
    if (a.lane_domain[l] != 1) continue;
    u64 v = warp_reduce(lm == l ? packed : 0, OpAdd());
    __syncthreads();
    if (lane == 0) red[tid >> 5] = v;
    __syncthreads();
    if (tid == 0) {
      u64 t = 0;
      for (int w = 0; w < AT_THREADS / 32; w++) t += red[w];
      const u64 m = (1ull << 20) - 1;
      ta_attr_summary *sm = &a.sum[a.lane_window[l]];
      if (t & m) atomicAdd((u64 *)&sm->n_attributed, t & m);
      if ((t >> 20) & m) atomicAdd((u64 *)&sm->n_no_launch, (t >> 20) & m);
      if ((t >> 40) & m) atomicAdd((u64 *)&sm->n_no_op, (t >> 40) & m);
    }
  }
}

// first/last were accumulated in an order-preserving unsigned encoding (0 = untouched)
#ifndef AT_FIN_ITEMS
#define AT_FIN_ITEMS 4
#endif
__global__ void __launch_bounds__(256) k_attr_finalize(AttrArgs a) {
  constexpr int IT = AT_FIN_ITEMS;
  const int err = ta_peek_err(a.status);
  const int64_t p0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * IT;
  if (p0 >= a.n_valid) return;
  // A kernel count above zero only ever sits at the position of an operator that owns kernels
  // (the counts are accumulated on operator rows alone), so the kinds need not be read: the
  // counts of all the thread's positions in vector loads, then both times of those operators -
  // two rounds of memory latency, the thread's misses overlapping
  int32_t cnt[IT];
  if (p0 + IT <= a.n) {
#pragma unroll
    for (int q = 0; q < IT / 4; q++) {
      const int4 x = *reinterpret_cast<const int4 *>(a.op_n + p0 + 4 * q);
      cnt[4 * q] = x.x; cnt[4 * q + 1] = x.y; cnt[4 * q + 2] = x.z; cnt[4 * q + 3] = x.w;
    }
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++) cnt[j] = p0 + j < a.n ? a.op_n[p0 + j] : 0;
  }
  if (ta_is_failure(err)) return;
  unsigned m = 0;
#pragma unroll
  for (int j = 0; j < IT; j++)
    if (p0 + j < a.n_valid && cnt[j] > 0) m |= 1u << j;
  if (!m) return;
  u64 f[IT], l[IT];
#pragma unroll
  for (int j = 0; j < IT; j++)
    if (m & (1u << j)) { f[j] = a.op_first[p0 + j]; l[j] = a.op_last[p0 + j]; }
#pragma unroll
  for (int j = 0; j < IT; j++)
    if (m & (1u << j)) {
      a.op_first[p0 + j] = (~f[j]) ^ (1ull << 63);
      a.op_last[p0 + j] = l[j] ^ (1ull << 63);
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
  char *zero_end = ck.base + ck.off;
  ta_attr_summary *d_sum = ck.take<ta_attr_summary>(W);
  TA_CHECK_CUDA(h, cudaMemsetAsync(zero_begin, 0, zero_end - zero_begin, st));
  TA_CHECK_CUDA(h, cudaMemsetAsync(d_sum, 0, (size_t)W * sizeof(ta_attr_summary), st));

  const int64_t tt = tiles > 0 ? tiles : 1;
  size_t tb = 2 * Carver::pad(tt * 4) + 2 * Carver::pad(tt * AT_CAP * 8) + 2 * Carver::pad(tt * AT_CAP * 4) + 256;
  // upper levels of the stack scan: node and start stacks per level
  std::vector<int64_t> level_n(1, tt);
  while (level_n.back() > AT_FAN) level_n.push_back((level_n.back() + AT_FAN - 1) / AT_FAN);
  for (size_t k = 1; k < level_n.size(); k++)
    tb += 2 * (Carver::pad(level_n[k] * 4) + Carver::pad(level_n[k] * AT_CAP * 8) +
               Carver::pad(level_n[k] * AT_CAP * 4));
  void *tmpb = ta_dalloc(h, tb);
  if (!tmpb) return TA_ERR_OOM;
  Carver ct(tmpb);
  AttrArgs a;
  memset(&a, 0, sizeof(a));
  a.agg_meta = ct.take<int32_t>(tt);
  a.carry_cnt = ct.take<int32_t>(tt);
  const size_t zero_bytes = ct.off;  // metas and carry counts start at zero; payloads need not
  a.agg_e = ct.take<i64>(tt * AT_CAP);
  a.carry_e = ct.take<i64>(tt * AT_CAP);
  a.agg_pos = ct.take<int32_t>(tt * AT_CAP);
  a.carry_pos = ct.take<int32_t>(tt * AT_CAP);
  TA_CHECK_CUDA(h, cudaMemsetAsync(tmpb, 0, zero_bytes, st));

  a.n = n; a.n_valid = h->n_valid; a.n_lanes = h->sorted.n_lanes; a.n_tiles = tiles;
  a.kind = h->sorted.kind; a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window;
  a.lane_domain = h->sorted.lane_domain; a.lane_dom_end = h->d_lane_dom_end;
  a.parent = parent; a.depth = depth; a.sum = d_sum; a.status = h->d_status;
  a.launch_of = h->join.launch_of; a.kol = h->join.kernels_of_launch; a.op_of = op_of; a.op_n = op_n; a.op_first = op_first;
  a.op_last = op_last; a.op_ns = op_ns;
  if (n > 0) {
    k_attr_agg<<<TA_N (unsigned)tiles, AT_THREADS, 0, st>>>(a);
    {
      // level 0 = tiles; fold upwards until at most AT_FAN stacks remain, scan those, unfold
      std::vector<StackArr> node(level_n.size()), start(level_n.size());
      node[0] = StackArr{a.agg_meta, a.agg_e, a.agg_pos};
      start[0] = StackArr{a.carry_cnt, a.carry_e, a.carry_pos};
      for (size_t k = 1; k < level_n.size(); k++) {
        const int64_t c = level_n[k];
        node[k] = StackArr{ct.take<int32_t>(c), ct.take<i64>(c * AT_CAP), ct.take<int32_t>(c * AT_CAP)};
        start[k] = StackArr{ct.take<int32_t>(c), ct.take<i64>(c * AT_CAP), ct.take<int32_t>(c * AT_CAP)};
      }
      const size_t top = level_n.size() - 1;
      for (size_t k = 1; k <= top; k++)
        k_attr_fold_up<<<TA_N (unsigned)((level_n[k] + 3) / 4), 128, 0, st>>>(
            node[k - 1], level_n[k - 1], node[k], level_n[k], h->d_status);
      k_attr_fold_top<<<TA_N 1, 32, 0, st>>>(node[top], level_n[top], start[top], top == 0 ? 1 : 0,
                                            h->d_status);
      for (size_t k = top; k >= 1; k--)
        k_attr_fold_down<<<TA_N (unsigned)((level_n[k] + 3) / 4), 128, 0, st>>>(
            node[k - 1], level_n[k - 1], start[k], level_n[k], start[k - 1], k == 1 ? 1 : 0,
            h->d_status);
    }
    k_attr_resolve<<<TA_N (unsigned)tiles, AT_THREADS, 0, st>>>(a);
    k_attr_ops<<<TA_N (unsigned)((n + AT_OPS_TILE - 1) / AT_OPS_TILE), AT_THREADS, 0, st>>>(a);
    const int64_t fb = (h->n_valid + 256 * AT_FIN_ITEMS - 1) / (256 * AT_FIN_ITEMS);
    k_attr_finalize<<<TA_N (unsigned)(fb > 0 ? fb : 1), 256, 0, st>>>(a);
    TA_CHECK_CUDA(h, cudaGetLastError());
  }
  std::vector<ta_attr_summary> hs(W);
  TA_TRY(ta_queue_d2h(h, hs.data(), d_sum, W * sizeof(ta_attr_summary)));
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
