// Stable LSD radix sort of 64-bit keys, with or without a 32-bit value: one
// scatter pass per digit with a chained scan over tiles ("one sweep"), so each
// pass reads and writes every element exactly once.  Digits are at most 8 bits
// wide; the digit histograms of all passes are taken up front (by the load kernel
// for the timeline sort, by k_radix_hist otherwise).
//
// Tile layout: THREADS x ITEMS elements per CTA, keys staged through shared
// memory so that both the global loads (warp-striped) and the scattered stores
// (runs of equal digits) are coalesced.  HBM-bound: per element and pass 8 B read
// + 8 B written (keys only) or 12 B + 12 B (pairs).
#include "ta_internal.cuh"

#define RS_BINS 256

struct RadixArgs {
  const u64 *keys_in;
  u64 *keys_out;
  const u32 *vals_in;  // may be null: value = global index
  u32 *vals_out;
  int64_t n;
  int shift, bits;
  const u32 *bin_offset;  // exclusive global digit offsets of this pass
  u64 *tile_state;        // [tile][RS_BINS]
  u32 *tile_counter;
  int32_t *status;
};

template <int THREADS, int ITEMS>
struct RadixSmem {
  u64 keys[THREADS * ITEMS];  // aliased by u32 values after the keys are written out
  u32 warp_hist[THREADS / 32][RS_BINS];
  u32 bin_start[RS_BINS];
  i64 adj[RS_BINS];
  u64 scan_tmp[33];
  int tile;
  int fail;
};

template <int THREADS, int ITEMS, bool VALS>
__global__ void __launch_bounds__(THREADS) k_radix_pass(RadixArgs a) {
  constexpr int TILE = THREADS * ITEMS;
  constexpr int WARPS = THREADS / 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  RadixSmem<THREADS, ITEMS> &s = *reinterpret_cast<RadixSmem<THREADS, ITEMS> *>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s.tile = (int)atomicAdd(a.tile_counter, 1u);
    s.fail = 0;
  }
  for (int i = tid; i < WARPS * RS_BINS; i += THREADS) (&s.warp_hist[0][0])[i] = 0;
  __syncthreads();
  const int tile = s.tile;
  const int64_t base = (int64_t)tile * TILE;
  const int count = (int)min((int64_t)TILE, a.n - base);
  const u32 mask = (1u << a.bits) - 1u;

  u64 key[ITEMS];
  int lrank[ITEMS];
  const int wbase = warp * 32 * ITEMS;
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    int li = wbase + j * 32 + lane;
    key[j] = li < count ? a.keys_in[base + li] : ~0ull;
  }
  // rank inside the warp, item row by item row (stable: row-major, then lane)
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    int li = wbase + j * 32 + lane;
    bool valid = li < count;
    u32 d = valid ? ((u32)(key[j] >> a.shift) & mask) : 0xFFFFFFFFu;
#ifdef RS_USE_MATCH
    u32 m = __match_any_sync(0xffffffffu, d);
#else
    // lanes with the same digit: one ballot per digit bit (cheaper than match.any here)
    u32 m = __ballot_sync(0xffffffffu, valid);
    if (!valid) m = ~m;
#pragma unroll
    for (int b = 0; b < 8; b++) {
      if (b < a.bits) {
        const u32 bal = __ballot_sync(0xffffffffu, (d >> b) & 1u);
        m &= ((d >> b) & 1u) ? bal : ~bal;
      }
    }
#endif
    // one population count per key (they run on the slow special-function pipe): the number of
    // peers at or above the lane.  The lowest peer adds the group size to the warp's digit
    // counter; every peer then reads the counter back and steps down from its new value.
    const u32 above1 = (u32)__popc(m >> lane);
    if (valid && (m & ((1u << lane) - 1u)) == 0) atomicAdd(&s.warp_hist[warp][d], above1);
    __syncwarp();
    const u32 after = valid ? s.warp_hist[warp][d] : 0u;
    lrank[j] = (int)(after - above1);
    __syncwarp();
  }
  __syncthreads();
  // per digit: exclusive offsets of the warps, then the CTA's digit count
  u32 cnt = 0;
  if (tid < RS_BINS) {
    u32 run = 0;
#pragma unroll
    for (int w = 0; w < WARPS; w++) {
      u32 t = s.warp_hist[w][tid];
      s.warp_hist[w][tid] = run;
      run += t;
    }
    cnt = run;
  }
  u64 total;
  u64 ex = block_scan_exclusive<OpAdd>((u64)cnt, OpAdd(), s.scan_tmp, &total);
  if (tid < RS_BINS) s.bin_start[tid] = (u32)ex;
  // chained scan over tiles, one digit per thread
  if (tid < (1 << a.bits)) {
    u64 *st = a.tile_state + (size_t)tile * RS_BINS + tid;
    u64 excl;
    if (tile == 0) {
      excl = a.bin_offset[tid];
      st_relaxed(st, td_pack(TD_PREFIX, excl + cnt));
    } else {
      st_relaxed(st, td_pack(TD_AGG, cnt));
      excl = 0;
      bool timed_out = false;
      for (int t = tile - 1;; --t) {
        u64 w = td_wait(a.tile_state + (size_t)t * RS_BINS + tid, a.status, &timed_out);
        excl += w & TD_MASK;
        if ((w >> 62) == TD_PREFIX) break;
      }
      st_relaxed(st, td_pack(TD_PREFIX, excl + cnt));
      if (timed_out) s.fail = 1;
    }
    s.adj[tid] = (i64)excl - (i64)ex;
  }
  __syncthreads();
  if (s.fail) return;
  // stage keys in shared memory in digit order
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    int li = wbase + j * 32 + lane;
    if (li < count) {
      u32 d = (u32)(key[j] >> a.shift) & mask;
      lrank[j] += (int)(s.bin_start[d] + s.warp_hist[warp][d]);
      s.keys[lrank[j]] = key[j];
    }
  }
  __syncthreads();
  u32 gpos[VALS ? ITEMS : 1];
#pragma unroll
  for (int k = 0; k < ITEMS; k++) {
    int sl = tid + k * THREADS;
    if (VALS) gpos[k] = 0xFFFFFFFFu;
    if (sl < count) {
      u64 kk = s.keys[sl];
      u32 d = (u32)(kk >> a.shift) & mask;
      i64 p = s.adj[d] + sl;
      if (VALS) gpos[k] = (u32)p;
      a.keys_out[p] = kk;
    }
  }
  if (!VALS) return;
  __syncthreads();
  u32 *svals = reinterpret_cast<u32 *>(s.keys);
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    int li = wbase + j * 32 + lane;
    if (li < count) svals[lrank[j]] = a.vals_in ? a.vals_in[base + li] : (u32)(base + li);
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < ITEMS; k++) {
    int sl = tid + k * THREADS;
    if (sl < count) a.vals_out[gpos[VALS ? k : 0]] = svals[sl];
  }
}

// tile shapes
#define RSP_THREADS 384  // pairs
#define RSP_ITEMS 12
#ifndef RSK_THREADS
#define RSK_THREADS 384  // keys only
#endif
#ifndef RSK_ITEMS
#define RSK_ITEMS 16
#endif

// digit histograms of every pass (used when the caller has none)
__global__ void __launch_bounds__(256) k_radix_hist(const u64 *keys, int64_t n, SortPlan plan,
                                                    u32 *hist) {
  __shared__ u32 sh[10 * RS_BINS];
  for (int i = threadIdx.x; i < plan.n_pass * RS_BINS; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    u64 k = keys[i];
    for (int p = 0; p < plan.n_pass; p++)
      atomicAdd(&sh[p * RS_BINS + ((u32)(k >> plan.shift[p]) & ((1u << plan.bits[p]) - 1u))], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < plan.n_pass * RS_BINS; i += blockDim.x)
    if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// exclusive scan of each pass's histogram: one CTA of 256 threads per pass
__global__ void __launch_bounds__(256) k_radix_scan_hist(const u32 *hist, u32 *bin_offset) {
  __shared__ u64 tmp[33];
  u64 total;
  u32 v = hist[blockIdx.x * RS_BINS + threadIdx.x];
  u64 ex = block_scan_exclusive<OpAdd>((u64)v, OpAdd(), tmp, &total);
  bin_offset[blockIdx.x * RS_BINS + threadIdx.x] = (u32)ex;
}

SortPlan ta_make_plan(int lo_bit, int hi_bit) {
  SortPlan p;
  int total = hi_bit - lo_bit;
  if (total < 1) total = 1;
  p.n_pass = (total + 7) / 8;
  int b = lo_bit;
  for (int i = 0; i < p.n_pass; i++) {
    int w = (total - (b - lo_bit) + (p.n_pass - i) - 1) / (p.n_pass - i);  // spread bits evenly
    p.shift[i] = b;
    p.bits[i] = w;
    b += w;
  }
  return p;
}

static size_t min_tile() {
  size_t a = (size_t)RSP_THREADS * RSP_ITEMS, b = (size_t)RSK_THREADS * RSK_ITEMS;
  return a < b ? a : b;
}

size_t ta_sort_temp_bytes(int64_t n) {
  size_t tiles = (size_t)((n + (int64_t)min_tile() - 1) / (int64_t)min_tile());
  if (tiles == 0) tiles = 1;
  return Carver::pad(tiles * RS_BINS * sizeof(u64)) + Carver::pad(16 * sizeof(u32)) +
         2 * Carver::pad(10 * RS_BINS * sizeof(u32));
}

// Sorts n keys (vals: pairs) by the key bits the plan covers.  Pass outputs
// alternate between the scratch and the final buffers such that the last pass
// writes the final ones; keys_in / vals_in are only read (pairs with vals_in null:
// the value of element i is i).  keys_in must not alias scratch or final.
// `hist` = precomputed [pass][256] digit histograms, or null.
template <bool VALS>
static ta_status radix_sort(ta_window *h, const u64 *keys_in, const u32 *vals_in, u64 *keys_scratch,
                            u32 *vals_scratch, u64 *keys_final, u32 *vals_final, int64_t n,
                            const SortPlan &plan, const u32 *hist, void *temp) {
  if (n <= 0) return TA_OK;
  constexpr int THREADS = VALS ? RSP_THREADS : RSK_THREADS;
  constexpr int ITEMS = VALS ? RSP_ITEMS : RSK_ITEMS;
  constexpr int TILE = THREADS * ITEMS;
  typedef RadixSmem<THREADS, ITEMS> Smem;
  auto kern = k_radix_pass<THREADS, ITEMS, VALS>;
  TA_CHECK_CUDA(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)sizeof(Smem)));
  size_t tiles = (size_t)((n + TILE - 1) / TILE);
  Carver c(temp);
  size_t max_tiles = (size_t)((n + (int64_t)min_tile() - 1) / (int64_t)min_tile());
  u64 *state = c.take<u64>(max_tiles * RS_BINS);
  u32 *counter = c.take<u32>(16);
  u32 *bin_offset = c.take<u32>(10 * RS_BINS);
  u32 *own_hist = c.take<u32>(10 * RS_BINS);
  cudaStream_t st = h->stream;
  if (!hist) {
    TA_CHECK_CUDA(h, cudaMemsetAsync(own_hist, 0, 10 * RS_BINS * sizeof(u32), st));
    int64_t want = (n + 255) / 256;
    int grid = (int)(want < 148 * 8 ? want : 148 * 8);
    k_radix_hist<<<TA_N grid, 256, 0, st>>>(keys_in, n, plan, own_hist);
    hist = own_hist;
  }
  k_radix_scan_hist<<<TA_N plan.n_pass, 256, 0, st>>>(hist, bin_offset);
  const u64 *kin = keys_in;
  const u32 *vin = vals_in;
  for (int p = 0; p < plan.n_pass; p++) {
    bool to_final = ((plan.n_pass - 1 - p) & 1) == 0;
    TA_CHECK_CUDA(h, cudaMemsetAsync(state, 0, tiles * RS_BINS * sizeof(u64), st));
    TA_CHECK_CUDA(h, cudaMemsetAsync(counter, 0, sizeof(u32), st));
    RadixArgs a;
    a.keys_in = kin; a.keys_out = to_final ? keys_final : keys_scratch;
    a.vals_in = vin; a.vals_out = to_final ? vals_final : vals_scratch;
    a.n = n; a.shift = plan.shift[p]; a.bits = plan.bits[p];
    a.bin_offset = bin_offset + p * RS_BINS;
    a.tile_state = state; a.tile_counter = counter; a.status = h->d_status;
    const bool timed = g_ta_profile && n == h->n;  // only the timeline sort (all records)
    if (timed) ta_profile_mark(st, 1, (VALS ? 24.0 : 16.0) * (double)n);
    kern<<<TA_N (unsigned)tiles, THREADS, sizeof(Smem), st>>>(a);
    if (timed) ta_profile_mark(st, 0, 0.0);
    kin = a.keys_out;
    vin = a.vals_out;
  }
  TA_CHECK_CUDA(h, cudaGetLastError());
  return TA_OK;
}

ta_status ta_radix_sort_pairs(ta_window *h, const u64 *keys_in, const u32 *vals_in,
                              u64 *keys_scratch, u32 *vals_scratch, u64 *keys_final,
                              u32 *vals_final, int64_t n, const SortPlan &plan, const u32 *hist,
                              void *temp) {
  return radix_sort<true>(h, keys_in, vals_in, keys_scratch, vals_scratch, keys_final, vals_final, n,
                          plan, hist, temp);
}

ta_status ta_radix_sort_keys(ta_window *h, const u64 *keys_in, u64 *keys_scratch, u64 *keys_final,
                             int64_t n, const SortPlan &plan, const u32 *hist, void *temp) {
  return radix_sort<false>(h, keys_in, nullptr, keys_scratch, nullptr, keys_final, nullptr, n, plan,
                           hist, temp);
}
