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
  const int32_t *lane_off, *lane_window;
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

__global__ void __launch_bounds__(SO_THREADS) k_operator_sol(SolArgs a) {
  const int err = ta_peek_err(a.status);
  const int64_t p0 = ((int64_t)blockIdx.x * SO_THREADS + threadIdx.x) * SO_ITEMS;
  int16_t kd[SO_ITEMS];
  loadn_i16<SO_ITEMS>(a.kind, p0, a.n, 9, kd);
  if (ta_is_failure(err)) return;
  unsigned ops = 0;
#pragma unroll
  for (int j = 0; j < SO_ITEMS; j++)
    if (p0 + j < a.n_valid && kd[j] == TA_KIND_OP) ops |= 1u << j;
  double mfu[SO_ITEMS], mbu[SO_ITEMS], sol[SO_ITEMS];
  uint8_t st[SO_ITEMS];
#pragma unroll
  for (int j = 0; j < SO_ITEMS; j++) { mfu[j] = mbu[j] = sol[j] = 0.0; st[j] = 0; }
  u64 n1 = 0, n2 = 0, n3 = 0, top_sum = 0;
  double fs = 0.0, bs = 0.0, mx = 0.0;
  int win = -1;
  if (ops) {
    int l = lane_of_pos(a.lane_off, a.n_lanes, p0);
    int64_t next_off = a.lane_off[l + 1];
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
#pragma unroll
    for (int j = 0; j < SO_ITEMS; j++) {
      if (!(ops & (1u << j))) continue;
      const int64_t p = p0 + j;
      while (p >= next_off) { l++; next_off = a.lane_off[l + 1]; }
      const int w = a.lane_window[l];
      u64 c1 = 0, c2 = 0, c3 = 0;
      if (top[j] <= 0) { st[j] = 2; c2 = 1; }
      else if (!(f[j] >= 0.0) || !(b[j] >= 0.0)) { st[j] = 3; c3 = 1; }
      else {
        // the same operations in the same order as the definition: no sum, so nothing fuses
        const double seconds = (double)top[j] * 1e-9;
        mfu[j] = f[j] / (seconds * a.peak_flops);
        mbu[j] = b[j] / (seconds * a.peak_bw);
        sol[j] = mfu[j] > mbu[j] ? mfu[j] : mbu[j];
        st[j] = 1;
        c1 = 1;
      }
      if (win < 0) win = w;
      if (w == win) {
        n1 += c1; n2 += c2; n3 += c3;
        if (c1) { top_sum += (u64)top[j]; fs += f[j]; bs += b[j]; mx = sol[j] > mx ? sol[j] : mx; }
      } else {  // a thread that straddles two windows
        sol_add(&a.sum[w], c1, c2, c3, c1 ? (u64)top[j] : 0, c1 ? f[j] : 0.0, c1 ? b[j] : 0.0, sol[j]);
      }
    }
  }
  if (p0 + SO_ITEMS <= a.n) {
    double2 *pm = reinterpret_cast<double2 *>(a.mfu + p0), *pb = reinterpret_cast<double2 *>(a.mbu + p0);
    double2 *ps = reinterpret_cast<double2 *>(a.sol + p0);
#pragma unroll
    for (int q = 0; q < SO_ITEMS / 2; q++) {
      pm[q] = make_double2(mfu[2 * q], mfu[2 * q + 1]);
      pb[q] = make_double2(mbu[2 * q], mbu[2 * q + 1]);
      ps[q] = make_double2(sol[2 * q], sol[2 * q + 1]);
    }
    *reinterpret_cast<u32 *>(a.state + p0) = st[0] | (st[1] << 8) | (st[2] << 16) | ((u32)st[3] << 24);
  } else {
#pragma unroll
    for (int j = 0; j < SO_ITEMS; j++)
      if (p0 + j < a.n) { a.mfu[p0 + j] = mfu[j]; a.mbu[p0 + j] = mbu[j]; a.sol[p0 + j] = sol[j]; a.state[p0 + j] = st[j]; }
  }
  // fold per warp when the warp sits in one window (almost always)
  const int lane = threadIdx.x & 31;
  const u32 has = __ballot_sync(0xffffffffu, win >= 0);
  if (!has) return;
  const int w0 = __shfl_sync(0xffffffffu, win, __ffs(has) - 1);
  if (__all_sync(0xffffffffu, win < 0 || win == w0)) {
    n1 = warp_reduce(n1, OpAdd()); n2 = warp_reduce(n2, OpAdd()); n3 = warp_reduce(n3, OpAdd());
    top_sum = warp_reduce(top_sum, OpAdd());
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      fs += __shfl_xor_sync(0xffffffffu, fs, o);
      bs += __shfl_xor_sync(0xffffffffu, bs, o);
      const double t = __shfl_xor_sync(0xffffffffu, mx, o);
      mx = t > mx ? t : mx;
    }
    if (lane == 0) sol_add(&a.sum[w0], n1, n2, n3, top_sum, fs, bs, mx);
  } else if (win >= 0) {
    sol_add(&a.sum[win], n1, n2, n3, top_sum, fs, bs, mx);
  }
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
  if (n > 0) {
    k_operator_sol<<<TA_N (unsigned)((n + SO_TILE - 1) / SO_TILE), SO_THREADS, 0, st>>>(a);
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
