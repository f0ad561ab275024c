// ta_operator_sol: model FLOPs utilisation, model bandwidth utilisation and speed-of-light
// attainment of every operator invocation (Sec. 6.1, "Operator execution and efficiency"):
// the invocation's theoretical operation count and logical data volume, each divided by T_op
// and by the device peak; SOL_op is the larger of the two.  The counts are the caller's (they
// come from shapes, data types and sharding, which no trace record carries): one pair of
// doubles per INPUT record, gathered through perm for the OP records only.
// One streaming pass: 2 B (kind) per record, 24 B + two 8-byte gathers per OP record, 25 B
// written per record.  The only floating-point kernel of the library.
#include <climits>
#include <cstring>
#include <vector>

#include "scan.cuh"
#include "ta_internal.cuh"

#define SO_THREADS 256
#define SO_ITEMS 4
#define SO_TILE (SO_THREADS * SO_ITEMS)

struct SolArgs {
  int64_t n, n_valid;
  int n_lanes;
  const int16_t *kind;
  const int32_t *perm, *op_n;
  const int64_t *op_first, *op_last;
  const double *flops, *bytes;  // per input record
  double peak_flops, peak_bw;
  const int32_t *lane_off, *lane_window, *lane_dom_end;
  const int16_t *lane_domain;
  double *mfu, *mbu, *sol;
  uint8_t *state;
  ta_sol_summary *sum;  // device, per window
  const int32_t *status;
};

__device__ __forceinline__ void sol_add(ta_sol_summary *s, u64 n1, u64 n2, u64 n3, u64 top, double f,
                                        double b, double mx) {
  if (n1) {
    atomicAdd((u64 *)&s->n_resolved, n1);
    atomicAdd((u64 *)&s->sum_top_ns, top);
    atomicAdd(&s->sum_flops, f);
    atomicAdd(&s->sum_bytes, b);
    // non-negative doubles order like their bit patterns
    atomicMax((u64 *)&s->max_sol, (u64)__double_as_longlong(mx));
  }
  if (n2) atomicAdd((u64 *)&s->n_no_kernels, n2);
  if (n3) atomicAdd((u64 *)&s->n_no_counts, n3);
}

__device__ __forceinline__ void sol_store_zero(const SolArgs &a, int64_t p0) {
  if (p0 + SO_ITEMS <= a.n) {
    double2 *pm = reinterpret_cast<double2 *>(a.mfu + p0), *pb = reinterpret_cast<double2 *>(a.mbu + p0);
    double2 *ps = reinterpret_cast<double2 *>(a.sol + p0);
#pragma unroll
    for (int q = 0; q < SO_ITEMS / 2; q++) pm[q] = pb[q] = ps[q] = make_double2(0.0, 0.0);
    *reinterpret_cast<u32 *>(a.state + p0) = 0u;
  } else {
    for (int j = 0; j < SO_ITEMS; j++)
      if (p0 + j < a.n) { a.mfu[p0 + j] = a.mbu[p0 + j] = a.sol[p0 + j] = 0.0; a.state[p0 + j] = 0; }
  }
}

// Per-window sums of one CTA: every thread keeps its share in registers while the CTA stays inside
// one window; the CTA folds and adds them to the window's row when it moves on (a row takes seven
// atomics on the same addresses, so adding per warp would serialise the whole grid on them).
struct SolAcc {
  u64 n1, n2, n3, top;
  double f, b, mx;
  __device__ __forceinline__ void clear() { n1 = n2 = n3 = top = 0; f = b = mx = 0.0; }
};

__device__ __forceinline__ void sol_flush(SolAcc &acc, ta_sol_summary *row, u64 (*red)[SO_THREADS / 32]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const u64 n1 = warp_reduce(acc.n1, OpAdd()), n2 = warp_reduce(acc.n2, OpAdd());
  const u64 n3 = warp_reduce(acc.n3, OpAdd()), top = warp_reduce(acc.top, OpAdd());
  double f = acc.f, b = acc.b, mx = acc.mx;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    f += __shfl_xor_sync(0xffffffffu, f, o);
    b += __shfl_xor_sync(0xffffffffu, b, o);
    const double t = __shfl_xor_sync(0xffffffffu, mx, o);
    mx = t > mx ? t : mx;
  }
  __syncthreads();  // red may still be read by the flush before
  if (lane == 0) {
    red[0][warp] = n1; red[1][warp] = n2; red[2][warp] = n3; red[3][warp] = top;
    red[4][warp] = (u64)__double_as_longlong(f); red[5][warp] = (u64)__double_as_longlong(b);
    red[6][warp] = (u64)__double_as_longlong(mx);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    u64 t1 = 0, t2 = 0, t3 = 0, tt = 0;
    double tf = 0.0, tb = 0.0, tm = 0.0;
    for (int w = 0; w < SO_THREADS / 32; w++) {
      t1 += red[0][w]; t2 += red[1][w]; t3 += red[2][w]; tt += red[3][w];
      tf += __longlong_as_double((i64)red[4][w]);
      tb += __longlong_as_double((i64)red[5][w]);
      const double m = __longlong_as_double((i64)red[6][w]);
      tm = m > tm ? m : tm;
    }
    sol_add(row, t1, t2, t3, tt, tf, tb, tm);
  }
  acc.clear();
}

// Persistent CTAs, each over a contiguous range of tiles.
__global__ void __launch_bounds__(SO_THREADS) k_operator_sol(SolArgs a, int64_t n_tiles, int64_t tiles_per_cta) {
  __shared__ int s_lane0, s_lane1;
  __shared__ u64 red[7][SO_THREADS / 32];
  if (ta_failed(a.status)) return;
  const int tid = threadIdx.x;
  SolAcc acc;
  acc.clear();
  int cw = -1;  // window the registers hold sums of (the same in every thread)
  const int64_t t_begin = (int64_t)blockIdx.x * tiles_per_cta;
  const int64_t t_end = min(t_begin + tiles_per_cta, n_tiles);
  for (int64_t tile = t_begin; tile < t_end; tile++) {
    const int64_t tile_start = tile * SO_TILE;
    const int64_t p0 = tile_start + (int64_t)tid * SO_ITEMS;
    const int64_t valid_end = min(tile_start + SO_TILE, a.n_valid);
    __syncthreads();  // the lanes of the tile before have been read
    if (tid < 64) {
      // warp 0: lane of the tile's first record; warp 1: lane of its last kept record
      int l = -1;
      if (tile_start < a.n_valid && a.n_lanes > 0)
        l = tile_lane_search(a.lane_off, a.n_lanes, tid < 32 ? tile_start : valid_end - 1);
      if (tid == 0) s_lane0 = l;
      if (tid == 32) s_lane1 = l;
    }
    __syncthreads();
    const int l0 = s_lane0, l1 = s_lane1;
    // Operators sit in host lanes: a tile of device lanes (or of dropped records) is all zeros
    // and reads nothing.
    if (l0 < 0 || span_outside_domain(a.lane_domain, a.lane_dom_end, l0, valid_end, 0)) {
      sol_store_zero(a, p0);
      continue;
    }
    // one window per tile, almost always: its sums stay in registers.  A tile that spans windows
    // (at most one per window boundary) adds record by record.
    const int w_first = a.lane_window[l0];
    const bool one_window = w_first == a.lane_window[l1];
    if (cw >= 0 && (!one_window || w_first != cw)) { sol_flush(acc, &a.sum[cw], red); cw = -1; }
    if (one_window) cw = w_first;
    int16_t kd[SO_ITEMS];
    loadn_i16<SO_ITEMS>(a.kind, p0, a.n, 9, kd);
    unsigned ops = 0;
#pragma unroll
    for (int j = 0; j < SO_ITEMS; j++)
      if (p0 + j < a.n_valid && kd[j] == TA_KIND_OP) ops |= 1u << j;
    if (!ops) {
      sol_store_zero(a, p0);
      continue;
    }
    // counts and times of the thread's OP records first, then the two gathers of those that
    // own kernels, so that the misses overlap
    i64 top[SO_ITEMS];
    int32_t src[SO_ITEMS];
#pragma unroll
    for (int j = 0; j < SO_ITEMS; j++) {
      top[j] = 0;
      src[j] = -1;
      if (!(ops & (1u << j))) continue;
      const int64_t p = p0 + j;
      if (a.op_n[p] > 0) top[j] = a.op_last[p] - a.op_first[p];
      if (top[j] > 0) src[j] = a.perm[p];
    }
    double f[SO_ITEMS], b[SO_ITEMS];
#pragma unroll
    for (int j = 0; j < SO_ITEMS; j++) {
      f[j] = b[j] = -1.0;
      if (src[j] >= 0) { f[j] = a.flops[src[j]]; b[j] = a.bytes[src[j]]; }
    }
    int l = l0;
    int64_t next_off = a.lane_off[l + 1];
    u32 st_word = 0;
    const bool whole = p0 + SO_ITEMS <= a.n;
#pragma unroll
    for (int q = 0; q < SO_ITEMS / 2; q++) {
      double mfu[2] = {0.0, 0.0}, mbu[2] = {0.0, 0.0}, sol[2] = {0.0, 0.0};
#pragma unroll
      for (int h = 0; h < 2; h++) {
        const int j = 2 * q + h;
        if (!(ops & (1u << j))) continue;
        u64 c1 = 0, c2 = 0, c3 = 0;
        u32 st = 0;
        if (top[j] <= 0) { st = 2; c2 = 1; }
        else if (!(f[j] >= 0.0) || !(b[j] >= 0.0)) { st = 3; c3 = 1; }
        else {
          // the same operations in the same order as the definition: no sum, so nothing fuses
          const double seconds = (double)top[j] * 1e-9;
          mfu[h] = f[j] / (seconds * a.peak_flops);
          mbu[h] = b[j] / (seconds * a.peak_bw);
          sol[h] = mfu[h] > mbu[h] ? mfu[h] : mbu[h];
          st = 1;
          c1 = 1;
        }
        st_word |= st << (8 * j);
        if (one_window) {
          acc.n1 += c1; acc.n2 += c2; acc.n3 += c3;
          if (c1) { acc.top += (u64)top[j]; acc.f += f[j]; acc.b += b[j]; acc.mx = sol[h] > acc.mx ? sol[h] : acc.mx; }
        } else {
          const int64_t p = p0 + j;
          while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; }
          sol_add(&a.sum[a.lane_window[l]], c1, c2, c3, c1 ? (u64)top[j] : 0, c1 ? f[j] : 0.0,
                  c1 ? b[j] : 0.0, sol[h]);
        }
      }
      if (whole) {
        reinterpret_cast<double2 *>(a.mfu + p0)[q] = make_double2(mfu[0], mfu[1]);
        reinterpret_cast<double2 *>(a.mbu + p0)[q] = make_double2(mbu[0], mbu[1]);
        reinterpret_cast<double2 *>(a.sol + p0)[q] = make_double2(sol[0], sol[1]);
      } else {
#pragma unroll
        for (int h = 0; h < 2; h++)
          if (p0 + 2 * q + h < a.n) {
            a.mfu[p0 + 2 * q + h] = mfu[h]; a.mbu[p0 + 2 * q + h] = mbu[h]; a.sol[p0 + 2 * q + h] = sol[h];
          }
      }
    }
    if (whole) *reinterpret_cast<u32 *>(a.state + p0) = st_word;
    else
      for (int j = 0; j < SO_ITEMS; j++)
        if (p0 + j < a.n) a.state[p0 + j] = (uint8_t)(st_word >> (8 * j));
  }
  if (cw >= 0) sol_flush(acc, &a.sum[cw], red);
}

ta_status ta_run_sol(ta_window *h, const double *flops, const double *bytes, int on_device,
                     double peak_flops, double peak_bw, ta_sol_result *out, ta_sol_summary *out_summary) {
  const int64_t n = h->n, nn = n > 0 ? n : 1;
  const int W = h->W;
  cudaStream_t st = h->stream;
  size_t keep = 3 * Carver::pad((size_t)nn * 8) + Carver::pad((size_t)nn) +
                Carver::pad((size_t)W * sizeof(ta_sol_summary)) + 256;
  void *kb = ta_dalloc(h, keep);
  if (!kb) return TA_ERR_OOM;
  Carver ck(kb);
  SolArgs a;
  memset(&a, 0, sizeof(a));
  a.mfu = ck.take<double>(nn); a.mbu = ck.take<double>(nn); a.sol = ck.take<double>(nn);
  a.state = ck.take<uint8_t>(nn);
  a.sum = ck.take<ta_sol_summary>(W);
  TA_CHECK_CUDA(h, cudaMemsetAsync(a.sum, 0, (size_t)W * sizeof(ta_sol_summary), st));
  void *tmp = nullptr;
  if (!on_device && n > 0) {
    tmp = ta_dalloc(h, 2 * Carver::pad((size_t)n * 8));
    if (!tmp) return TA_ERR_OOM;
    Carver ct(tmp);
    double *df = ct.take<double>(n), *db = ct.take<double>(n);
    TA_CHECK_CUDA(h, cudaMemcpyAsync(df, flops, (size_t)n * 8, cudaMemcpyHostToDevice, st));
    TA_CHECK_CUDA(h, cudaMemcpyAsync(db, bytes, (size_t)n * 8, cudaMemcpyHostToDevice, st));
    flops = df;
    bytes = db;
  }
  a.n = n; a.n_valid = h->n_valid; a.n_lanes = h->sorted.n_lanes;
  a.kind = h->sorted.kind; a.perm = h->sorted.perm; a.op_n = h->attr.op_n_kernels;
  a.op_first = h->attr.op_first_start; a.op_last = h->attr.op_last_end;
  a.flops = flops; a.bytes = bytes; a.peak_flops = peak_flops; a.peak_bw = peak_bw;
  a.lane_off = h->sorted.lane_off; a.lane_window = h->sorted.lane_window; a.status = h->d_status;
  a.lane_domain = h->sorted.lane_domain; a.lane_dom_end = h->d_lane_dom_end;
  if (n > 0) {
    const int64_t n_tiles = (n + SO_TILE - 1) / SO_TILE;
    const int64_t ctas = n_tiles < 148 * 8 ? n_tiles : 148 * 8;
    const int64_t per = (n_tiles + ctas - 1) / ctas;
    k_operator_sol<<<TA_N (unsigned)((n_tiles + per - 1) / per), SO_THREADS, 0, st>>>(a, n_tiles, per);
    TA_CHECK_CUDA(h, cudaGetLastError());
  }
  std::vector<ta_sol_summary> hs(W);
  TA_TRY(ta_queue_d2h(h, hs.data(), a.sum, (size_t)W * sizeof(ta_sol_summary)));
  int32_t words[ST_WORDS];
  TA_TRY(ta_read_status(h, words));
  if (tmp) ta_dfree(h, tmp);
  if (words[ST_ERR]) return (ta_status)words[ST_ERR];
  for (int w = 0; w < W; w++) out_summary[w] = hs[w];
  out->mfu = a.mfu; out->mbu = a.mbu; out->sol = a.sol; out->state = a.state;
  return TA_OK;
}
