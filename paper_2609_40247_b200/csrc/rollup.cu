// ta_rollup_operators: inclusive per-operator kernel figures and graph replays.
// An invocation's kernel composition comes from the call-to-kernel links and T_op
// spans the first kernel start to the last completion; CUDA Graph replay hides the
// operator calls, and launch correlations separate the replays (Sec. 6.1, "Operator
// execution and efficiency").
//
//   k_roll_ops       every OP that owns kernels adds its direct figures to itself and
//                    to each OP on its parent chain (at most TA_MAX_DEPTH hops once the
//                    attribution has passed): count and nanoseconds by atomic add, first
//                    start / last end by atomic max on order-preserving codes;
//   k_roll_replays   every device record whose launch owns two or more adds itself to
//                    that launch's row in the same way;
//   k_roll_finalize  decodes the rows that were touched and folds the per-window counts.
// Host-lane tiles and device-lane tiles each skip the kernel that is not theirs.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define RO_THREADS 256
#define RO_ITEMS 8
#define RO_TILE (RO_THREADS * RO_ITEMS)

struct RollArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int16_t *kind;
  const int64_t *ts, *te;
  const int32_t *parent, *op_n, *launch_of, *kol;
  const int64_t *op_first, *op_last, *op_ns;
  const int32_t *lane_off, *lane_window, *lane_dom_end;
  const int16_t *lane_domain;
  int32_t *incl_n;
  u64 *incl_first, *incl_last, *replay_first, *replay_last;  // coded until the finalize kernel
  int64_t *incl_ns, *replay_ns;
  u64 *win_sum;  // [window][3]
  const int32_t *status;
};

__device__ __forceinline__ u64 roll_code(i64 v) { return (u64)v ^ (1ull << 63); }

// lane of the tile's first position; false if the tile holds no lane of `domain`
__device__ __forceinline__ bool roll_tile(const RollArgs &a, int domain, int64_t *p0, int64_t *tile_end) {
  __shared__ int s_lane0;
  if (ta_failed(a.status)) return false;
  const int64_t tile_start = (int64_t)blockIdx.x * RO_TILE;
  if (tile_start >= a.n_valid) return false;
  if (threadIdx.x < 32) {
    const int l = tile_lane_search(a.lane_off, a.n_lanes, tile_start);
    if (threadIdx.x == 0) s_lane0 = l;
  }
  __syncthreads();
  *tile_end = min(tile_start + RO_TILE, a.n_valid);
  *p0 = tile_start + (int64_t)threadIdx.x * RO_ITEMS;
  return !span_outside_domain(a.lane_domain, a.lane_dom_end, s_lane0, *tile_end, domain) && *p0 < *tile_end;
}

__global__ void __launch_bounds__(RO_THREADS) k_roll_ops(RollArgs a) {
  int64_t p0, tile_end;
  if (!roll_tile(a, 0, &p0, &tile_end)) return;
  int16_t kd[RO_ITEMS];
  load8_i16(a.kind, p0, a.n, 9, kd);
  int32_t cnt[RO_ITEMS];
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++)
    cnt[j] = (p0 + j < tile_end && kd[j] == TA_KIND_OP) ? a.op_n[p0 + j] : 0;
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) {
    if (cnt[j] <= 0) continue;
    const int64_t p = p0 + j;
    const u64 ns = (u64)a.op_ns[p], fc = ~roll_code(a.op_first[p]), lc = roll_code(a.op_last[p]);
    int32_t q = (int32_t)p;
    for (int hop = 0; hop < 300 && q >= 0; hop++) {
      atomicAdd(&a.incl_n[q], cnt[j]);
      atomicAdd((u64 *)&a.incl_ns[q], ns);
      atomicMax(&a.incl_first[q], fc);
      atomicMax(&a.incl_last[q], lc);
      q = a.parent[q];
    }
  }
}

__global__ void __launch_bounds__(RO_THREADS) k_roll_replays(RollArgs a) {
  int64_t p0, tile_end;
  if (!roll_tile(a, 1, &p0, &tile_end)) return;
  int16_t kd[RO_ITEMS];
  load8_i16(a.kind, p0, a.n, 9, kd);
  int32_t lo[RO_ITEMS];
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++)
    lo[j] = (p0 + j < tile_end && (kd[j] == TA_KIND_KERNEL || kd[j] == TA_KIND_MEMCPY)) ? a.launch_of[p0 + j] : -1;
  int32_t many[RO_ITEMS];
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) many[j] = lo[j] >= 0 ? a.kol[lo[j]] : 0;
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) {
    if (many[j] < 2) continue;
    const i64 s = a.ts[p0 + j], e = a.te[p0 + j];
    atomicMax(&a.replay_first[lo[j]], ~roll_code(s));
    atomicMax(&a.replay_last[lo[j]], roll_code(e));
    atomicAdd((u64 *)&a.replay_ns[lo[j]], (u64)(e - s));
  }
}

__global__ void __launch_bounds__(RO_THREADS) k_roll_finalize(RollArgs a) {
  int64_t p0, tile_end;
  if (!roll_tile(a, 0, &p0, &tile_end)) return;
  int16_t kd[RO_ITEMS];
  load8_i16(a.kind, p0, a.n, 9, kd);
  // counts first (inclusive kernels of the OPs, kernels of the launches), then the coded times
  // of the rows that were touched, all of a thread's loads of one kind issued together
  int32_t cnt[RO_ITEMS];
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) {
    cnt[j] = 0;
    if (p0 + j >= tile_end) continue;
    if (kd[j] == TA_KIND_OP) cnt[j] = a.incl_n[p0 + j];
    else if (kd[j] == TA_KIND_LAUNCH) cnt[j] = a.kol[p0 + j];
  }
  unsigned ops = 0, reps = 0;
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) {
    if (kd[j] == TA_KIND_OP && cnt[j] > 0) ops |= 1u << j;
    if (kd[j] == TA_KIND_LAUNCH && cnt[j] >= 2) reps |= 1u << j;
  }
  if (!(ops | reps)) return;
  u64 f[RO_ITEMS], l[RO_ITEMS];
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) {
    if (ops & (1u << j)) { f[j] = a.incl_first[p0 + j]; l[j] = a.incl_last[p0 + j]; }
    else if (reps & (1u << j)) { f[j] = a.replay_first[p0 + j]; l[j] = a.replay_last[p0 + j]; }
  }
#pragma unroll
  for (int j = 0; j < RO_ITEMS; j++) {
    const int64_t p = p0 + j;
    if (ops & (1u << j)) {
      a.incl_first[p] = (~f[j]) ^ (1ull << 63);
      a.incl_last[p] = l[j] ^ (1ull << 63);
    } else if (reps & (1u << j)) {
      a.replay_first[p] = (~f[j]) ^ (1ull << 63);
      a.replay_last[p] = l[j] ^ (1ull << 63);
      const int w = a.lane_window[lane_of_pos(a.lane_off, a.n_lanes, p)];
      atomicAdd(&a.win_sum[(size_t)w * 3], 1ull);
      atomicAdd(&a.win_sum[(size_t)w * 3 + 1], (u64)cnt[j]);
      atomicMax(&a.win_sum[(size_t)w * 3 + 2], (u64)cnt[j]);
    }
  }
}

ta_status ta_run_rollup(ta_window *h, ta_rollup_result *out, ta_rollup_summary *out_summary) {
  cudaStream_t st = h->stream;
  memset(out, 0, sizeof(*out));
  const int W = h->W;
  const int64_t n = h->n, nn = n > 0 ? n : 1;
  for (int w = 0; w < W; w++) memset(&out_summary[w], 0, sizeof(ta_rollup_summary));
  size_t kb = Carver::pad((size_t)nn * 4) + 6 * Carver::pad((size_t)nn * 8) + Carver::pad((size_t)W * 24) + 256;
  void *keep = ta_dalloc(h, kb);
  if (!keep) return TA_ERR_OOM;
  Carver ck(keep);
  RollArgs a;
  memset(&a, 0, sizeof(a));
  a.incl_n = ck.take<int32_t>(nn);
  a.incl_ns = ck.take<int64_t>(nn);
  a.incl_first = ck.take<u64>(nn); a.incl_last = ck.take<u64>(nn);
  a.replay_first = ck.take<u64>(nn); a.replay_last = ck.take<u64>(nn);
  a.replay_ns = ck.take<int64_t>(nn);
  a.win_sum = ck.take<u64>((size_t)W * 3);
  TA_CHECK_CUDA(h, cudaMemsetAsync(keep, 0, ck.off, st));
  out->incl_n_kernels = a.incl_n; out->incl_kernel_ns = a.incl_ns;
  out->incl_first_start = (const int64_t *)a.incl_first; out->incl_last_end = (const int64_t *)a.incl_last;
  out->replay_first_start = (const int64_t *)a.replay_first;
  out->replay_last_end = (const int64_t *)a.replay_last; out->replay_kernel_ns = a.replay_ns;
  if (h->n_valid == 0) return TA_OK;

  a.n = n; a.n_valid = h->n_valid; a.n_lanes = h->sorted.n_lanes;
  a.kind = h->sorted.kind; a.ts = h->sorted.ts_start; a.te = h->sorted.ts_end;
  a.parent = h->attr.parent; a.op_n = h->attr.op_n_kernels; a.launch_of = h->join.launch_of;
  a.kol = h->join.kernels_of_launch;
  a.op_first = h->attr.op_first_start; a.op_last = h->attr.op_last_end; a.op_ns = h->attr.op_kernel_ns;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window;
  a.lane_dom_end = h->d_lane_dom_end; a.lane_domain = h->sorted.lane_domain; a.status = h->d_status;
  const unsigned tiles = (unsigned)((h->n_valid + RO_TILE - 1) / RO_TILE);
  k_roll_ops<<<TA_N tiles, RO_THREADS, 0, st>>>(a);
  k_roll_replays<<<TA_N tiles, RO_THREADS, 0, st>>>(a);
  k_roll_finalize<<<TA_N tiles, RO_THREADS, 0, st>>>(a);
  TA_CHECK_CUDA(h, cudaGetLastError());
  std::vector<u64> hs((size_t)W * 3);
  TA_TRY(ta_queue_d2h(h, hs.data(), a.win_sum, (size_t)W * 24));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  for (int w = 0; w < W; w++) {
    out_summary[w].n_graph_launches = (int64_t)hs[(size_t)w * 3];
    out_summary[w].n_graph_kernels = (int64_t)hs[(size_t)w * 3 + 1];
    out_summary[w].max_kernels_per_launch = (int64_t)hs[(size_t)w * 3 + 2];
  }
  return TA_OK;
}
