// ta_attribute_operators: thread id plus call intervals link host API calls to
// the enclosing calls (Sec. 9.1); device records inherit the operator of their
// launch; T_op spans the first kernel start to the last completion (Sec. 6.1).
//
// In canonical order (ts_start ascending, ts_end descending) a properly nested
// host lane has a simple structure: the innermost encloser of record i is the
// nearest earlier OP whose end is still ahead of i.  That is answered
//   - inside a tile of 2048 records by a max-tree over OP end times in shared
//     memory (one descent per record), and
//   - across tiles by carrying the stack of still-open OPs (at most
//     TA_MAX_DEPTH + 1 entries when nesting is legal) through a bounded
//     decoupled look-back.  Combining a carried stack with a tile's stack is
//     associative: entries that end no later than the tile's outermost
//     surviving OP can never be chosen again and are dropped.
// Partial overlap is detected on the way: the nearest earlier OP that is still
// running when i starts must also cover i's end.
// HBM-bound: 18 B read + 5 B written per host record, plus the per-operator
// atomics of the device records.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define AT_THREADS 512
#define AT_ITEMS 4
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

struct Stack {
  int cnt;
  int reset;
  i64 e[AT_CAP];
  int32_t pos[AT_CAP];
};

// earlier (+) later
__device__ __forceinline__ void stack_combine(const Stack &earlier, Stack &later, bool *overflow) {
  if (later.reset) return;
  int keep = earlier.cnt;
  if (later.cnt > 0) {
    keep = 0;
    while (keep < earlier.cnt && earlier.e[keep] > later.e[0]) keep++;
  }
  if (keep + later.cnt > AT_CAP) {
    *overflow = true;
    keep = AT_CAP - later.cnt;
  }
  for (int i = later.cnt - 1; i >= 0; i--) {
    later.e[keep + i] = later.e[i];
    later.pos[keep + i] = later.pos[i];
  }
  for (int i = 0; i < keep; i++) {
    later.e[i] = earlier.e[i];
    later.pos[i] = earlier.pos[i];
  }
  later.cnt += keep;
  later.reset = earlier.reset;
}

__device__ __forceinline__ u64 blk_reduce_max(u64 v, u64 *smem) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_reduce(v, OpMax());
  __syncthreads();
  if (lane == 0) smem[warp] = v;
  __syncthreads();
  if (warp == 0) {
    u64 w = lane < (int)(blockDim.x >> 5) ? smem[lane] : 0;
    w = warp_reduce(w, OpMax());
    if (lane == 0) smem[32] = w;
  }
  __syncthreads();
  return smem[32];
}

__global__ void __launch_bounds__(AT_THREADS) k_attr(AttrArgs a) {
  __shared__ i64 node[2 * AT_TILE];
  __shared__ int16_t parent_local[AT_TILE];
  __shared__ uint8_t kcarry[AT_TILE];
  __shared__ Stack s_agg, s_carry;
  __shared__ u64 tmp[33];
  __shared__ int s_tile, s_lane_last, s_lo, s_hi;
  const int tid = threadIdx.x;
  if (tid == 0) s_tile = (int)atomicAdd(a.counter, 1u);
  __syncthreads();
  const int tile = s_tile;
  const int64_t tile_start = (int64_t)tile * AT_TILE;
  const int x0 = tid * AT_ITEMS;
  const int64_t p0 = tile_start + x0;

  LaneWalker lw(a.lane_off, a.n_lanes, p0, a.n_valid);
  bool host[AT_ITEMS];
  int ln[AT_ITEMS];
  i64 s[AT_ITEMS], e[AT_ITEMS];
  int64_t lb[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    int64_t p = p0 + j;
    host[j] = false;
    ln[j] = -1;
    s[j] = e[j] = 0;
    lb[j] = 0;
    i64 leaf = INT64_MIN;
    if (p < a.n_valid) {
      int k = a.kind[p];
      if (k <= TA_KIND_LAUNCH) {
        host[j] = true;
        ln[j] = lw.at(p);
        lb[j] = a.lane_off[ln[j]];
        s[j] = a.ts[p];
        e[j] = a.te[p];
        if (k == TA_KIND_OP) leaf = e[j];
      }
    }
    node[AT_TILE + x0 + j] = leaf;
  }
  if (tid == 0) {
    int64_t plast = min(tile_start + AT_TILE, a.n_valid) - 1;
    s_lane_last = plast >= tile_start ? lane_of_pos(a.lane_off, a.n_lanes, plast) : -1;
  }
  __syncthreads();
  for (int w = AT_TILE >> 1; w >= 1; w >>= 1) {
    for (int i = tid; i < w; i += AT_THREADS) {
      i64 l = node[2 * (w + i)], r = node[2 * (w + i) + 1];
      node[w + i] = l > r ? l : r;
    }
    __syncthreads();
  }

  // nearest earlier OP of the tile that is still running when the record starts
  unsigned bad = 0;  // bit j: item j overlaps an earlier OP partially
  i64 thr[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    const int x = x0 + j;
    int16_t pl = AT_NONE;
    thr[j] = 0;
    if (host[j]) {
      thr[j] = e[j] > s[j] ? s[j] + 1 : e[j];
      int y = -1;
      int pos = x + AT_TILE;
      while (pos > 1) {
        if ((pos & 1) && node[pos - 1] >= thr[j]) {
          pos = pos - 1;
          while (pos < AT_TILE) pos = node[2 * pos + 1] >= thr[j] ? 2 * pos + 1 : 2 * pos;
          y = pos - AT_TILE;
          break;
        }
        pos >>= 1;
      }
      int64_t lo_local = lb[j] - tile_start;
      if (y >= 0 && (int64_t)y >= lo_local) {
        pl = (int16_t)y;
        if (node[AT_TILE + y] < e[j]) bad |= 1u << j;
      } else {
        pl = lb[j] >= tile_start ? AT_NONE : AT_UNRESOLVED;
      }
    }
    parent_local[x] = pl;
  }

  // stack of the tile's last lane segment: OPs that no later OP of the tile dominates
  const int lane_last = s_lane_last;
  const bool last_is_host = lane_last >= 0 && a.lane_domain[lane_last] == 0;
  int surv = 0;
  bool is_surv[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    is_surv[j] = false;
    if (last_is_host && host[j] && ln[j] == lane_last) {
      const int x = x0 + j;
      i64 mine = node[AT_TILE + x];
      if (mine != INT64_MIN) {
        i64 mx = INT64_MIN;
        int l = x + 1 + AT_TILE, r = 2 * AT_TILE;
        while (l < r) {
          if (l & 1) { mx = mx > node[l] ? mx : node[l]; l++; }
          if (r & 1) { --r; mx = mx > node[r] ? mx : node[r]; }
          l >>= 1;
          r >>= 1;
        }
        if (mx < mine) { is_surv[j] = true; surv++; }
      }
    }
  }
  u64 n_surv;
  u64 surv_ex = block_scan_exclusive<OpAdd>((u64)surv, OpAdd(), tmp, &n_surv);
  {
    int o = (int)surv_ex;
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++)
      if (is_surv[j]) {
        if (o < AT_CAP) { s_agg.e[o] = e[j]; s_agg.pos[o] = (int32_t)(p0 + j); }
        o++;
      }
  }
  __syncthreads();

  if (tid == 0) {
    bool overflow = n_surv > AT_CAP;
    s_agg.cnt = overflow ? AT_CAP : (int)n_surv;
    s_agg.reset = (!last_is_host || (int64_t)a.lane_off[lane_last] >= tile_start) ? 1 : 0;
    // does the first record continue a host lane that began in an earlier tile?
    bool need_carry = false;
    if (tile_start < a.n_valid && tile > 0) {
      int l0 = lane_of_pos(a.lane_off, a.n_lanes, tile_start);
      need_carry = a.lane_domain[l0] == 0 && (int64_t)a.lane_off[l0] < tile_start;
    }
    const size_t tb = (size_t)tile * AT_CAP;
    if (s_agg.reset) {
      for (int i = 0; i < s_agg.cnt; i++) { a.pre_e[tb + i] = s_agg.e[i]; a.pre_pos[tb + i] = s_agg.pos[i]; }
      a.pre_meta[tile] = s_agg.cnt | (1 << 8);
      __threadfence();
      st_relaxed(&a.flag[tile], td_pack(TD_PREFIX, 0));
    } else {
      for (int i = 0; i < s_agg.cnt; i++) { a.agg_e[tb + i] = s_agg.e[i]; a.agg_pos[tb + i] = s_agg.pos[i]; }
      a.agg_meta[tile] = s_agg.cnt;
      __threadfence();
      st_relaxed(&a.flag[tile], td_pack(TD_AGG, 0));
    }
    Stack acc;
    acc.cnt = 0;
    acc.reset = 0;
    if (need_carry) {
      bool timed_out = false;
      for (int t = tile - 1; t >= 0; --t) {
        u64 w = td_wait(&a.flag[t], a.status, &timed_out);
        if (timed_out) break;
        __threadfence();
        const bool is_prefix = (w >> 62) == TD_PREFIX;
        const int32_t meta = ld_relaxed_i32(is_prefix ? &a.pre_meta[t] : &a.agg_meta[t]);
        Stack ear;
        ear.cnt = meta & 0xFF;
        ear.reset = (meta >> 8) & 1;
        const i64 *pe = (is_prefix ? a.pre_e : a.agg_e) + (size_t)t * AT_CAP;
        const int32_t *pp = (is_prefix ? a.pre_pos : a.agg_pos) + (size_t)t * AT_CAP;
        for (int i = 0; i < ear.cnt; i++) {
          ear.e[i] = (i64)ld_relaxed((const u64 *)&pe[i]);
          ear.pos[i] = ld_relaxed_i32(&pp[i]);
        }
        stack_combine(ear, acc, &overflow);
        if (is_prefix || ear.reset) break;
      }
    }
    s_carry = acc;
    if (!s_agg.reset) {
      Stack incl = s_agg;
      stack_combine(acc, incl, &overflow);
      for (int i = 0; i < incl.cnt; i++) { a.pre_e[tb + i] = incl.e[i]; a.pre_pos[tb + i] = incl.pos[i]; }
      a.pre_meta[tile] = incl.cnt | (incl.reset << 8);
      __threadfence();
      st_relaxed(&a.flag[tile], td_pack(TD_PREFIX, 0));
    }
    if (overflow) ta_set_err(a.status, TA_ERR_DEPTH);
  }
  __syncthreads();

  // records whose encloser lies before the tile: look it up in the carried stack
  int32_t par_abs[AT_ITEMS];
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    const int x = x0 + j;
    par_abs[j] = -1;
    if (!host[j]) continue;
    int16_t pl = parent_local[x];
    if (pl >= 0) par_abs[j] = (int32_t)(tile_start + pl);
    else if (pl == AT_UNRESOLVED) {
      int k = 0;
      while (k < s_carry.cnt && s_carry.e[k] >= thr[j]) k++;
      kcarry[x] = (uint8_t)k;
      if (k > 0) {
        par_abs[j] = s_carry.pos[k - 1];
        if (s_carry.e[k - 1] < e[j]) bad |= 1u << j;
      }
    }
  }
  __syncthreads();
  int dmax = 0;
  int my_lo = INT_MAX, my_hi = -1;
#pragma unroll
  for (int j = 0; j < AT_ITEMS; j++) {
    int64_t p = p0 + j;
    if (p >= a.n) continue;
    int d = 0;
    if (host[j]) {
      int c = x0 + j;
      for (int it = 0; it < 300; it++) {
        int pl = parent_local[c];
        if (pl == AT_NONE) break;
        if (pl == AT_UNRESOLVED) { d += kcarry[c]; break; }
        d++;
        c = pl;
      }
      if (d > 255) d = 255;
      dmax = max(dmax, d);
      my_lo = min(my_lo, ln[j]);
      my_hi = max(my_hi, ln[j]);
      if (bad & (1u << j)) atomicOr(&a.sum[a.lane_window[ln[j]]].bad_nesting, 1);
    }
    a.parent[p] = par_abs[j];
    a.depth[p] = (uint8_t)d;
  }
  // per-window maximum depth (a tile rarely meets more than one lane)
  if (tid == 0) { s_lo = INT_MAX; s_hi = -1; }
  __syncthreads();
  if (my_hi >= 0) { atomicMin(&s_lo, my_lo); atomicMax(&s_hi, my_hi); }
  __syncthreads();
  const int l0 = s_lo, l1 = s_hi;
  if (l1 < 0) return;
  const int w0 = a.lane_window[l0], w1 = a.lane_window[l1];
  if (w0 == w1) {
    u64 m = blk_reduce_max((u64)dmax, tmp);
    if (tid == 0 && m > 0) atomicMax(&a.sum[w0].max_depth, (int)m);
  } else {
#pragma unroll
    for (int j = 0; j < AT_ITEMS; j++)
      if (host[j] && p0 + j < a.n) atomicMax(&a.sum[a.lane_window[ln[j]]].max_depth, (int)a.depth[p0 + j]);
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
  a.agg_e = ct.take<i64>(tt * AT_CAP);
  a.pre_e = ct.take<i64>(tt * AT_CAP);
  a.agg_pos = ct.take<int32_t>(tt * AT_CAP);
  a.pre_pos = ct.take<int32_t>(tt * AT_CAP);
  a.counter = ct.take<u32>(16);
  TA_CHECK_CUDA(h, cudaMemsetAsync(tmpb, 0, ct.off, st));

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
    k_attr_finalize<<<TA_N (unsigned)((h->n_valid + 255) / 256 > 0 ? (h->n_valid + 255) / 256 : 1), 256, 0, st>>>(a);
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
