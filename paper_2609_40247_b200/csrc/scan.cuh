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
  __shared__ int s_tile;
  const int tid = threadIdx.x;
  if (tid == 0) s_tile = (int)atomicAdd(t.counter, 1u);
  __syncthreads();
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
    u64 e = tile_lookback<Op>(t.state, tile, tile_total, op, status);
    if (tid == 0) {
      s_excl = e;
      if ((int64_t)(tile + 1) * SC_TILE >= n) *t.total = op(e, tile_total);
    }
  }
  __syncthreads();
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
