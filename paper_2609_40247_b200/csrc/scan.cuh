// Generic single-pass device-wide exclusive scan over u64 values with a
// commutative operator (sum or max), built on the bounded decoupled look-back
// of ta_internal.cuh.  `In` supplies element i, `Out` consumes (i, exclusive
// prefix, value).  Used for stream compaction and for segment-head tracking.
#pragma once
#include "ta_internal.cuh"

#define SC_THREADS 512
#define SC_ITEMS 4
#define SC_TILE (SC_THREADS * SC_ITEMS)

struct ScanTemp {
  u64 *state;    // tiles + 1 descriptors, zeroed
  u32 *counter;  // zeroed
  u64 *total;    // receives the reduction of all elements
};

static inline size_t scan_temp_bytes(int64_t n) {
  int64_t tiles = (n + SC_TILE - 1) / SC_TILE + 1;
  return Carver::pad((size_t)tiles * 8) + Carver::pad(64);
}
// carves and zeroes the temp (one memset)
static inline ta_status scan_temp_init(ta_window *h, void *mem, int64_t n, ScanTemp *t) {
  int64_t tiles = (n + SC_TILE - 1) / SC_TILE + 1;
  Carver c(mem);
  t->state = c.take<u64>(tiles);
  u64 *sc = c.take<u64>(8);
  t->counter = (u32 *)(sc + 1);
  t->total = sc;
  TA_CHECK_CUDA(h, cudaMemsetAsync(mem, 0, c.off, h->stream));
  return TA_OK;
}

#ifdef __CUDACC__
template <class Op, class In, class Out>
__global__ void __launch_bounds__(SC_THREADS) k_scan(int64_t n, In in, Out out, Op op, ScanTemp t,
                                                     int32_t *status) {
  __shared__ u64 tmp[33];
  __shared__ u64 s_excl;
  __shared__ int s_tile, s_fail;
  const int tid = threadIdx.x;
  if (tid == 0) {
    s_tile = (int)atomicAdd(t.counter, 1u);
    s_fail = ta_failed(status) ? 1 : 0;
  }
  __syncthreads();
  if (s_fail) return;
  const int tile = s_tile;
  const int64_t i0 = (int64_t)tile * SC_TILE + (int64_t)tid * SC_ITEMS;
  u64 v[SC_ITEMS];
  u64 run = op.identity();
#pragma unroll
  for (int j = 0; j < SC_ITEMS; j++) {
    v[j] = (i0 + j < n) ? in(i0 + j) : op.identity();
    run = op(run, v[j]);
  }
  u64 tile_total;
  u64 ex = block_scan_exclusive<Op>(run, op, tmp, &tile_total);
  if (tid < 32) {
    bool failed;
    u64 e = tile_lookback<Op>(t.state, tile, tile_total, op, status, &failed);
    if (tid == 0) {
      s_excl = e;
      s_fail = failed ? 1 : 0;
      if (!failed && (int64_t)(tile + 1) * SC_TILE >= n) *t.total = op(e, tile_total);
    }
  }
  __syncthreads();
  if (s_fail) return;
  u64 pre = op(s_excl, ex);
#pragma unroll
  for (int j = 0; j < SC_ITEMS; j++) {
    if (i0 + j < n) out(i0 + j, pre, v[j]);
    pre = op(pre, v[j]);
  }
}

template <class Op, class In, class Out>
static inline ta_status launch_scan(ta_window *h, int64_t n, In in, Out out, Op op, ScanTemp t) {
  if (n <= 0) return TA_OK;
  int64_t tiles = (n + SC_TILE - 1) / SC_TILE;
  k_scan<Op, In, Out><<<TA_N (unsigned)tiles, SC_THREADS, 0, h->stream>>>(n, in, out, op, t, h->d_status);
  TA_CHECK_CUDA(h, cudaGetLastError());
  return TA_OK;
}

// ---- helpers for kernels that give every thread eight consecutive sorted positions ----
// largest l with lane_off[l] <= p, found by the 32 lanes of one warp together
__device__ __forceinline__ int tile_lane_search(const int32_t *lane_off, int n_lanes, int64_t p) {
  const int lane = threadIdx.x & 31;
  int lo = 0, hi = n_lanes;
  while (hi - lo > 1) {
    int step = (hi - lo + 31) >> 5;
    int idx = lo + lane * step;
    bool ok = idx < hi && (int64_t)lane_off[idx] <= p;
    u32 m = __ballot_sync(0xffffffffu, ok);
    int k = 31 - __clz((int)m);  // lane 0 always qualifies
    lo = lo + k * step;
    hi = min(hi, lo + step);
  }
  return lo;
}
__device__ __forceinline__ void load8_i16(const int16_t *col, int64_t p0, int64_t n, int16_t fill,
                                          int16_t *v) {
  if (p0 + 8 <= n) {
    uint4 q = *reinterpret_cast<const uint4 *>(col + p0);
    const int16_t *hq = reinterpret_cast<const int16_t *>(&q);
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] = hq[j];
  } else {
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] = p0 + j < n ? col[p0 + j] : fill;
  }
}
__device__ __forceinline__ void load8_i64(const int64_t *col, int64_t p0, int64_t n, i64 *v) {
  if (p0 + 8 <= n) {
    const longlong2 *ps = reinterpret_cast<const longlong2 *>(col + p0);
#pragma unroll
    for (int j = 0; j < 4; j++) {
      longlong2 x = ps[j];
      v[2 * j] = x.x;
      v[2 * j + 1] = x.y;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] = p0 + j < n ? col[p0 + j] : 0;
  }
}
__device__ __forceinline__ void store8_i64(int64_t *col, int64_t p0, int64_t n, const i64 *v) {
  if (p0 + 8 <= n) {
    longlong2 *ps = reinterpret_cast<longlong2 *>(col + p0);
#pragma unroll
    for (int j = 0; j < 4; j++) ps[j] = make_longlong2(v[2 * j], v[2 * j + 1]);
  } else {
#pragma unroll
    for (int j = 0; j < 8; j++)
      if (p0 + j < n) col[p0 + j] = v[j];
  }
}
__device__ __forceinline__ void store8_i32(int32_t *col, int64_t p0, int64_t n, const int32_t *v) {
  if (p0 + 8 <= n) {
    int4 *ps = reinterpret_cast<int4 *>(col + p0);
    ps[0] = make_int4(v[0], v[1], v[2], v[3]);
    ps[1] = make_int4(v[4], v[5], v[6], v[7]);
  } else {
#pragma unroll
    for (int j = 0; j < 8; j++)
      if (p0 + j < n) col[p0 + j] = v[j];
  }
}

// the same for IT = 4 or 8 consecutive positions (p0 a multiple of IT)
template <int IT>
__device__ __forceinline__ void loadn_i16(const int16_t *col, int64_t p0, int64_t n, int16_t fill, int16_t *v) {
  if (IT == 8) { load8_i16(col, p0, n, fill, v); return; }
  if (p0 + IT <= n) {
    const uint2 q = *reinterpret_cast<const uint2 *>(col + p0);
    const int16_t *hq = reinterpret_cast<const int16_t *>(&q);
#pragma unroll
    for (int j = 0; j < IT; j++) v[j] = hq[j];
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++) v[j] = p0 + j < n ? col[p0 + j] : fill;
  }
}
template <int IT>
__device__ __forceinline__ void loadn_i64(const int64_t *col, int64_t p0, int64_t n, i64 *v) {
  if (p0 + IT <= n) {
    const longlong2 *ps = reinterpret_cast<const longlong2 *>(col + p0);
#pragma unroll
    for (int j = 0; j < IT / 2; j++) {
      const longlong2 x = ps[j];
      v[2 * j] = x.x;
      v[2 * j + 1] = x.y;
    }
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++) v[j] = p0 + j < n ? col[p0 + j] : 0;
  }
}
template <int IT>
__device__ __forceinline__ void storen_i64(int64_t *col, int64_t p0, int64_t n, const i64 *v) {
  if (p0 + IT <= n) {
    longlong2 *ps = reinterpret_cast<longlong2 *>(col + p0);
#pragma unroll
    for (int j = 0; j < IT / 2; j++) ps[j] = make_longlong2(v[2 * j], v[2 * j + 1]);
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++)
      if (p0 + j < n) col[p0 + j] = v[j];
  }
}
template <int IT>
__device__ __forceinline__ void storen_i32(int32_t *col, int64_t p0, int64_t n, const int32_t *v) {
  if (p0 + IT <= n) {
    int4 *ps = reinterpret_cast<int4 *>(col + p0);
#pragma unroll
    for (int j = 0; j < IT / 4; j++) ps[j] = make_int4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
  } else {
#pragma unroll
    for (int j = 0; j < IT; j++)
      if (p0 + j < n) col[p0 + j] = v[j];
  }
}

// Ordered compaction of the sorted positions whose kind is in `kind_mask`: 256 threads x 16
// positions per tile, vector loads of the kind column, one tile scan.
#define CK_THREADS 256
#define CK_ITEMS 16
#define CK_TILE (CK_THREADS * CK_ITEMS)
// zero_col (may be null): an n-sized 64-bit column the caller needs cleared; the kernel reads two
// bytes per record and has the bandwidth to write it on the way (positions below zero_n that its
// tiles cover; the caller clears the rest).
static __global__ void __launch_bounds__(CK_THREADS) k_compact_kind(const int16_t *kind, int64_t n_valid,
                                                             u32 kind_mask, u32 *pos_out, ScanTemp t,
                                                             int32_t *status, i64 *zero_col,
                                                             int64_t zero_n) {
  __shared__ u64 tmp[33];
  __shared__ u64 s_excl;
  __shared__ int s_tile, s_fail;
  const int tid = threadIdx.x;
  if (tid == 0) {
    s_tile = (int)atomicAdd(t.counter, 1u);
    s_fail = ta_failed(status) ? 1 : 0;
  }
  __syncthreads();
  if (s_fail) return;
  const int tile = s_tile;
  const int64_t p0 = (int64_t)tile * CK_TILE + (int64_t)tid * CK_ITEMS;
  if (zero_col) {
#pragma unroll
    for (int k = 0; k < CK_ITEMS / 2; k++) {
      const int64_t z = (int64_t)tile * CK_TILE + (int64_t)k * (2 * CK_THREADS) + 2 * tid;
      if (z + 2 <= zero_n) *reinterpret_cast<longlong2 *>(zero_col + z) = make_longlong2(0, 0);
      else if (z < zero_n) zero_col[z] = 0;
    }
  }
  int16_t kd[CK_ITEMS];
  load8_i16(kind, p0, n_valid, -1, kd);
  load8_i16(kind, p0 + 8, n_valid, -1, kd + 8);
  u32 sel = 0;
#pragma unroll
  for (int j = 0; j < CK_ITEMS; j++)
    if (kd[j] >= 0 && ((kind_mask >> kd[j]) & 1u)) sel |= 1u << j;
  u64 total;
  u64 ex = block_scan_exclusive<OpAdd>((u64)__popc(sel), OpAdd(), tmp, &total);
  if (tid < 32) {
    bool failed;
    u64 e = tile_lookback<OpAdd>(t.state, tile, total, OpAdd(), status, &failed);
    if (tid == 0) {
      s_excl = e;
      s_fail = failed ? 1 : 0;
      if (!failed && (int64_t)(tile + 1) * CK_TILE >= n_valid) *t.total = e + total;
    }
  }
  __syncthreads();
  if (s_fail) return;
  u64 o = s_excl + ex;
#pragma unroll
  for (int j = 0; j < CK_ITEMS; j++)
    if (sel & (1u << j)) pos_out[o++] = (u32)(p0 + j);
}
static inline ta_status launch_compact_kind(ta_window *h, const int16_t *kind, int64_t n_valid,
                                            u32 kind_mask, u32 *pos_out, ScanTemp t,
                                            i64 *zero_col = nullptr, int64_t zero_n = 0) {
  int64_t tiles = n_valid > 0 ? (n_valid + CK_TILE - 1) / CK_TILE : 0;
  if (zero_col && tiles * CK_TILE < zero_n)  // what the tiles do not reach (the dropped tail)
    TA_CHECK_CUDA(h, cudaMemsetAsync(zero_col + tiles * CK_TILE, 0, (size_t)(zero_n - tiles * CK_TILE) * 8,
                                     h->stream));
  if (n_valid <= 0) return TA_OK;
  k_compact_kind<<<TA_N (unsigned)tiles, CK_THREADS, 0, h->stream>>>(kind, n_valid, kind_mask, pos_out, t,
                                                                   h->d_status, zero_col, zero_n);
  TA_CHECK_CUDA(h, cudaGetLastError());
  return TA_OK;
}

// Walks the lane table along ascending sorted positions.
struct LaneWalker {
  const int32_t *lane_off;
  int n_lanes;
  int lane;
  __device__ __forceinline__ LaneWalker(const int32_t *off, int nl, int64_t p0, int64_t n_valid)
      : lane_off(off), n_lanes(nl), lane(-1) {
    if (p0 < n_valid && nl > 0) lane = lane_of_pos(off, nl, p0);
  }
  __device__ __forceinline__ int at(int64_t p) {
    while (lane + 1 < n_lanes && (int64_t)lane_off[lane + 1] <= p) lane++;
    return lane;
  }
};
#endif
