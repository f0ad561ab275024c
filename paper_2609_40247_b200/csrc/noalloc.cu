// ta_lane_gaps_noalloc: the stream-gap scan of ONE device lane for callers that
// must not allocate device memory (see include/ta.h).  Same arithmetic as the
// per-lane part of ta_stream_gaps; the tile descriptors of the chained max-scan,
// the tile counter and the status word live in a fixed file-scope device array
// instead of memory obtained from an allocator.
#include "ta_internal.cuh"

#define NA_THREADS 256
#define NA_ITEMS 8
#define NA_TILE (NA_THREADS * NA_ITEMS)
#define NA_MAX_RECORDS TA_NOALLOC_MAX_RECORDS
#define NA_MAX_TILES (NA_MAX_RECORDS / NA_TILE)

struct NaScratch {
  u64 state[NA_MAX_TILES + 1];  // tile descriptors of the max-scan
  int32_t status[ST_WORDS];
  u32 counter;
  u32 pad[3];
};

// Every device that loads the library holds this array until the process exits.
// In host code `g_na_scratch` is only a stand-in for the symbol, not a device
// address: the address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_na_scratch[sizeof(NaScratch)];

__global__ void __launch_bounds__(NA_THREADS) k_lane_gaps_noalloc(const int64_t *ts, const int64_t *te,
                                                                   int64_t n, i64 W0, i64 W1,
                                                                   int64_t *gap_before,
                                                                   ta_lane_gaps *out, NaScratch *sc) {
  __shared__ u64 tmp[33];
  __shared__ u64 red[5][8];
  __shared__ u64 s_excl;
  __shared__ int s_tile, s_fail;
  const int tid = threadIdx.x;
  if (tid == 0) s_tile = (int)atomicAdd(&sc->counter, 1u);
  __syncthreads();
  const int tile = s_tile;
  const int64_t p0 = (int64_t)tile * NA_TILE + (int64_t)tid * NA_ITEMS;
  i64 s[NA_ITEMS], ce[NA_ITEMS];
  u64 v[NA_ITEMS];
  u64 run = 0;
#pragma unroll
  for (int j = 0; j < NA_ITEMS; j++) {
    int64_t p = p0 + j;
    s[j] = ce[j] = 0;
    v[j] = 0;
    if (p < n) {
      s[j] = ts[p];
      i64 e = te[p];
      ce[j] = e < W1 ? e : W1;
      i64 rel = ce[j] - W0;
      v[j] = (u64)(rel > 0 ? rel : 0) + 1;  // 0 is reserved for "nothing before"
    }
    run = run > v[j] ? run : v[j];
  }
  u64 tile_max;
  u64 thread_excl = block_scan_exclusive<OpMax>(run, OpMax(), tmp, &tile_max);
  if (tid < 32) {
    bool failed;
    u64 e = tile_lookback<OpMax>(sc->state, tile, tile_max, OpMax(), sc->status, &failed);
    if (tid == 0) { s_excl = e; s_fail = failed ? 1 : 0; }
  }
  __syncthreads();
  if (s_fail) return;  // a bounded wait gave up: the status word says so, nothing is written
  u64 pre = s_excl > thread_excl ? s_excl : thread_excl;
  u64 sb = 0, si = 0, ng = 0, mg = 0;
#pragma unroll
  for (int j = 0; j < NA_ITEMS; j++) {
    int64_t p = p0 + j;
    if (p >= n) break;
    i64 P = pre ? W0 + (i64)(pre - 1) : W0;
    i64 gap = s[j] > P ? s[j] - P : 0;
    i64 from = s[j] > P ? s[j] : P;
    i64 busy = ce[j] > from ? ce[j] - from : 0;
    gap_before[p] = gap;
    sb += (u64)busy;
    si += (u64)gap;
    if (gap > 0) { ng++; mg = mg > (u64)gap ? mg : (u64)gap; }
    if (p == 0) out->first_start = s[j];
    if (p == n - 1) {
      i64 Pm = P > ce[j] ? P : ce[j];
      i64 tail = W1 - Pm;
      si += (u64)tail;
      if (tail > 0) { ng++; mg = mg > (u64)tail ? mg : (u64)tail; }
      out->last_end = Pm;
      out->n_events = n;
    }
    pre = pre > v[j] ? pre : v[j];
  }
  sb = warp_reduce(sb, OpAdd());
  si = warp_reduce(si, OpAdd());
  ng = warp_reduce(ng, OpAdd());
  mg = warp_reduce(mg, OpMax());
  if ((tid & 31) == 0) { red[0][tid >> 5] = sb; red[1][tid >> 5] = si; red[2][tid >> 5] = ng; red[3][tid >> 5] = mg; }
  __syncthreads();
  if (tid == 0) {
    u64 a = 0, b = 0, c = 0, d = 0;
    for (int w = 0; w < NA_THREADS / 32; w++) { a += red[0][w]; b += red[1][w]; c += red[2][w]; d = d > red[3][w] ? d : red[3][w]; }
    if (a) atomicAdd((u64 *)&out->busy, a);
    if (b) atomicAdd((u64 *)&out->idle, b);
    if (c) atomicAdd((u64 *)&out->n_gaps, c);
    if (d) atomicMax((i64 *)&out->max_gap, (i64)d);
  }
}

extern "C" ta_status ta_lane_gaps_noalloc(const int64_t *ts_start, const int64_t *ts_end, int64_t n,
                                          int64_t win_t0, int64_t win_t1, int64_t *gap_before,
                                          ta_lane_gaps *lane_out, void *cuda_stream) {
  if (n < 0 || win_t0 >= win_t1 || !lane_out || (n > 0 && (!ts_start || !ts_end || !gap_before)))
    return TA_ERR_INVALID_ARG;
  if (n > NA_MAX_RECORDS) return TA_ERR_TOO_LARGE;  // the fixed scratch array covers no more
  if ((uint64_t)win_t1 - (uint64_t)win_t0 >= (1ull << 40)) return TA_ERR_TOO_LARGE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // set-up, once per device, with that device current: the address of the scratch array
  static NaScratch *scratch_of[64] = {nullptr};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TA_ERR_CUDA;
  if (!scratch_of[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_na_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return TA_ERR_CUDA;
    }
    scratch_of[dev] = (NaScratch *)p;
  }
  NaScratch *sc = scratch_of[dev];
  // the array keeps the previous call's contents: clear what must start at zero
  if (cudaMemsetAsync(sc, 0, sizeof(NaScratch), st) != cudaSuccess) return TA_ERR_CUDA;
  if (cudaMemsetAsync(lane_out, 0, sizeof(ta_lane_gaps), st) != cudaSuccess) return TA_ERR_CUDA;
  if (n == 0) {
    ta_lane_gaps empty = {0, win_t1 - win_t0, 0, 1, win_t1 - win_t0, 0, win_t0};
    if (cudaMemcpyAsync(lane_out, &empty, sizeof(empty), cudaMemcpyHostToDevice, st) != cudaSuccess)
      return TA_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? TA_OK : TA_ERR_CUDA;
  }
  const unsigned tiles = (unsigned)((n + NA_TILE - 1) / NA_TILE);
  k_lane_gaps_noalloc<<<TA_N tiles, NA_THREADS, 0, st>>>(ts_start, ts_end, n, win_t0, win_t1,
                                                        gap_before, lane_out, sc);
  if (cudaGetLastError() != cudaSuccess) return TA_ERR_CUDA;
  int32_t err = 0;
  if (cudaMemcpyAsync(&err, &sc->status[ST_ERR], sizeof(err), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return TA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TA_ERR_CUDA;
  return (ta_status)err;
}
