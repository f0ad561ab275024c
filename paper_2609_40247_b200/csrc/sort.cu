// Stable LSD radix sort of 64-bit keys, with or without a 32-bit value: one
// scatter pass per digit with a chained scan over tiles ("one sweep"), so each
// pass reads and writes every element exactly once.  Digits are at most 8 bits
// wide; the digit histograms of all passes are taken up front (by the load kernel
// for the timeline sort, by k_radix_hist otherwise).
//
// Tile layout: THREADS x ITEMS elements per CTA, keys staged through shared
// memory so that both the global loads (warp-striped) and the scattered stores
// (runs of equal digits) are coalesced.  HBM-bound by design (per element and
// pass 8 B read + 8 B written for keys, 12 B + 12 B for pairs); in practice the
// pass is instruction-bound on B200, so the kernel is specialised on the digit
// width and on full tiles, and every key costs one population count, one
// shared-memory atomic and as many warp votes as the digit has bits.
#include "ta_internal.cuh"

#define RS_BINS 256
// descriptors of earlier tiles fetched together in the look back (1 = one at a time)
#ifndef RS_LOOKBACK_BATCH
#define RS_LOOKBACK_BATCH 4
#endif

// resident CTAs per SM the register allocation is sized for (pairs, keys only)
#ifndef RSP_MINB
#define RSP_MINB 2
#endif
#ifndef RSK_MINB
#define RSK_MINB 4
#endif

struct RadixArgs {
  const u64 *keys_in;
  u64 *keys_out;
  const u32 *vals_in;  // may be null: value = global index
  u32 *vals_out;
  int64_t n;
  int shift;
  const u32 *bin_offset;  // exclusive global digit offsets of this pass
  u64 *tile_state;        // [tile][RS_BINS]
  u32 *tile_counter;
  int32_t *status;
  u32 gen;                // 1 + pass index: tags this pass's tile descriptors
  PrekeyInfo pk;          // PREKEY passes only
};

// Discovery word of input record i ([dropped][triple slot, 13 bits][ts_start - t0, 40 bits]) ->
// packed key [dropped][window][triple rank][(ts_start - t0) >> dshift][index inside the window].
#define RS_PRE_DROPPED (1ull << 63)
#define RS_PRE_TS_BITS 40
__device__ __forceinline__ u64 prekey_to_key(const PrekeyInfo &k, u64 w64, int w, int64_t i) {
  u64 hi;
  if (w64 & RS_PRE_DROPPED) {
    hi = (1ull << (k.wbits + k.tbits + k.tsb)) | ((u64)w << (k.tbits + k.tsb));
  } else {
    const u32 slot = (u32)(w64 >> RS_PRE_TS_BITS) & (TA_TRIPLE_SLOTS - 1);
    const u64 rank = (u64)__ldg(&k.rank_of_slot[slot]);
    hi = ((u64)w << (k.tbits + k.tsb)) | (rank << k.tsb) |
         ((w64 & ((1ull << RS_PRE_TS_BITS) - 1)) >> k.dshift);
  }
  return (hi << k.ibits) | (u64)(i - k.off[w]);
}

// Tile descriptors of the pair passes (the small sorts: long-gap list, collective keys) carry the
// pass they belong to, so that one clearing of the descriptor array serves every pass of a sort:
// [status, 2 bits][pass tag, 6 bits][count, 56 bits]; a descriptor whose tag is not the running
// pass's is as good as empty.  The keys-only passes (the timeline sort: 16 k tiles) keep plain
// descriptors and a clearing per pass: the tag test cost them 11 us per pass, more than the
// clearings it saves.
#define RS_GEN_SHIFT 56
#define RS_VMASK ((1ull << RS_GEN_SHIFT) - 1)
template <bool GEN>
__device__ __forceinline__ u64 rs_pack(u64 flag, u32 gen, u64 v) {
  return GEN ? (flag << 62) | ((u64)gen << RS_GEN_SHIFT) | (v & RS_VMASK) : td_pack(flag, v);
}
template <bool GEN>
__device__ __forceinline__ bool rs_ready(u64 x, u32 gen) {
  return GEN ? (u32)(x >> RS_GEN_SHIFT & 0x3Fu) == gen : (x >> 62) != TD_EMPTY;
}
// bounded wait for a descriptor of this pass, as td_wait
template <bool GEN>
__device__ __forceinline__ u64 rs_wait(const u64 *p, u32 gen, int32_t *status, bool *timed_out) {
  u64 w = ld_relaxed(p);
  int spins = 0, limit = 0;
  while (!rs_ready<GEN>(w, gen)) {
    if (limit == 0) {
      limit = ld_relaxed_i32(&status[ST_SPIN]);
      if (limit <= 0) limit = TA_SPIN_LIMIT;
    }
    if (++spins > limit || ta_is_failure(ld_relaxed_i32(&status[ST_ERR]))) {
      *timed_out = true;
      ta_set_err(status, TA_ERR_TIMEOUT);
      return rs_pack<GEN>(TD_PREFIX, gen, 0);
    }
    __nanosleep(40);
    w = ld_relaxed(p);
  }
  return w;
}

template <int THREADS, int ITEMS>
struct RadixSmem {
  u64 keys[THREADS * ITEMS];  // aliased by u32 values after the keys are written out
  u32 warp_hist[THREADS / 32][RS_BINS];  // per warp: digit counts, later tile-local start of the warp's run
  u32 adj[RS_BINS];           // global position of a digit's run minus its tile-local start (mod 2^32)
  u32 pcnt[RS_BINS];          // keys-only passes: the digit counts, for the thread that publishes two digits
  u64 scan_tmp[33];
  int tile;
  int fail;
  int win0;  // PREKEY passes: window of the tile's first record
};

// STABLE = false: equal digits may leave the pass in any order (one shared-memory atomic per
// key instead of the vote ranking).  Only legal for the FIRST pass of a sort whose caller
// does not rely on the input order of keys that are equal in all sorted bits.
template <int THREADS, int ITEMS, bool VALS, int BITS, bool FULL, bool STABLE, bool PREKEY>
__device__ __forceinline__ void radix_tile(const RadixArgs &a, RadixSmem<THREADS, ITEMS> &s, int tile,
                                           int count) {
  constexpr int TILE = THREADS * ITEMS;
  constexpr int WARPS = THREADS / 32;
  constexpr u32 MASK = (1u << BITS) - 1u;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t base = (int64_t)tile * TILE;
  const u32 lt = (1u << lane) - 1u;

  u64 key[ITEMS];
  int rd[ITEMS];  // (tile-local rank << 8) | digit
  const int wbase = warp * 32 * ITEMS;
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    const int li = wbase + j * 32 + lane;
    key[j] = (FULL || li < count) ? a.keys_in[base + li] : ~0ull;
  }
  if (PREKEY) {
    // the words are in input order: the tile's window range is short (usually one window); the
    // window of the tile's first record comes from one search per CTA, each thread walks on
    int w = s.win0;
    int64_t next = a.pk.off[w + 1];
#pragma unroll
    for (int j = 0; j < ITEMS; j++) {
      const int li = wbase + j * 32 + lane;  // grows with j: the walk only moves forward
      if (FULL || li < count) {
        const int64_t i = base + li;
        while (i >= next) {  // also steps over empty windows; off[W] = n > i
          w++;
          next = a.pk.off[w + 1];
        }
        key[j] = prekey_to_key(a.pk, key[j], w, i);
      }
    }
  }
  // rank inside the warp, item row by item row (stable: row-major, then lane)
  u32 *wh = s.warp_hist[warp];
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    const bool valid = FULL || (wbase + j * 32 + lane) < count;
    const u32 d = (u32)(key[j] >> a.shift) & MASK;
    if (!STABLE) {
      const u32 old = valid ? atomicAdd(&wh[d], 1u) : 0u;
      rd[j] = (int)((old << 8) | d);
      continue;
    }
    u32 m = FULL ? 0xffffffffu : __ballot_sync(0xffffffffu, valid);
    if (!FULL && !valid) m = ~m;
    // lanes with the same digit: one vote per digit bit.  Written out as the four instructions it
    // takes (test, vote, select, combine); the compiler's own sequence for the same expression was
    // six per bit, and the pass is bound by instruction issue (-16 % instructions, -5 % time).
    const u32 dv = (FULL || valid) ? d : 0u;  // a lane without a key never votes "set"
#pragma unroll
    for (int b = 0; b < BITS; b++) {
      asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 t, bal;\n\t"
          "and.b32 t, %1, %2;\n\tsetp.ne.u32 p, t, 0;\n\t"
          "vote.sync.ballot.b32 bal, p, 0xffffffff;\n\t"
          "selp.b32 t, 0, 0xffffffff, p;\n\t"   // bit set: keep bal; bit clear: keep ~bal
          "lop3.b32 %0, %0, bal, t, 0x60;\n\t}"  // m & (bal ^ t)
          : "+r"(m)
          : "r"(dv), "r"(1u << b));
    }
    if (!FULL && !valid) m = 0;
#ifndef RS_RANK_READBACK
    // The lowest peer adds the group size to the warp's digit counter and hands the counter's
    // old value to its peers by a shuffle; a peer's rank is that value plus the number of peers
    // below it.  No read-back of the counter and no warp barrier: the rows of a thread are
    // independent up to the order of the warp's own atomics on one address, which is program
    // order, so the votes of later rows overlap the atomics of earlier ones.
    const int leader = __ffs((int)m) - 1;  // -1 for an invalid lane (m = 0)
    u32 old = 0;
    if (valid && lane == leader) old = atomicAdd(&wh[d], (u32)__popc(m));
    old = __shfl_sync(0xffffffffu, old, leader < 0 ? lane : leader);
    rd[j] = (int)(((old + (u32)__popc(m & lt)) << 8) | d);
  }
#else
    // one population count per key: the number of peers at or above the lane.  The lowest
    // peer adds the group size to the warp's digit counter; every peer then reads the counter
    // back and steps down from its new value.
    const u32 above1 = (u32)__popc(m >> lane);
    if (valid && (m & lt) == 0) atomicAdd(&wh[d], above1);
    __syncwarp();
    const u32 after = valid ? wh[d] : 0u;
    rd[j] = (int)(((after - above1) << 8) | d);
    __syncwarp();
  }
#endif
  __syncthreads();
  // per digit: the CTA's count, exclusive starts of the digits, and per warp the tile-local
  // start of its run (so the scatter needs one shared load per key)
  u32 cnt = 0;
  if (tid < RS_BINS) {
#pragma unroll
    for (int w = 0; w < WARPS; w++) cnt += s.warp_hist[w][tid];
  }
  if (!VALS && tid < RS_BINS) s.pcnt[tid] = cnt;  // visible after the scan's barriers
  u64 total;
  const u64 ex = block_scan_exclusive<OpAdd>((u64)cnt, OpAdd(), s.scan_tmp, &total);
  if (tid < RS_BINS) {
    if (!VALS) s.adj[tid] = (u32)ex;  // read by the digit's publisher after the next barrier
    u32 run = (u32)ex;
#pragma unroll
    for (int w = 0; w < WARPS; w++) {
      const u32 t = s.warp_hist[w][tid];
      s.warp_hist[w][tid] = run;
      run += t;
    }
  }
  // chained scan over tiles: the tile's own counts are published first, the keys are staged in
  // shared memory in digit order (which needs tile-local offsets only), and the look back over
  // the earlier tiles comes last, when they have had time to publish.
  // Pair passes: one digit per thread and descriptor.  Keys-only passes: TWO digits per thread
  // and descriptor, [status, 2 bits][digit d + NB/2, 31 bits][digit d, 31 bits] - counts and
  // prefixes stay below 2^31 (n < 2^31), so one 64-bit add sums both without a carry between
  // them, and half as many threads walk half as many descriptors.
  constexpr int NB = 1 << BITS, HB = NB / 2;
  constexpr int PER_TILE = VALS ? RS_BINS : RS_BINS / 2;
  constexpr int WALKERS = VALS ? NB : HB;
  u64 *st = a.tile_state + (size_t)tile * PER_TILE + tid;
  u32 cnt_hi = 0;  // keys-only: count of digit tid + HB
  if (tid < WALKERS) {
    if (VALS) {
      if (tile == 0) st_relaxed(st, rs_pack<VALS>(TD_PREFIX, a.gen, (u64)a.bin_offset[tid] + cnt));
      else st_relaxed(st, rs_pack<VALS>(TD_AGG, a.gen, cnt));
    } else {
      cnt_hi = s.pcnt[tid + HB];
      if (tile == 0)
        st_relaxed(st, td_pack(TD_PREFIX, ((u64)(a.bin_offset[tid + HB] + cnt_hi) << 31) | (a.bin_offset[tid] + cnt)));
      else
        st_relaxed(st, td_pack(TD_AGG, ((u64)cnt_hi << 31) | cnt));
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    if (FULL || (wbase + j * 32 + lane) < count) {
      const u32 d = (u32)rd[j] & 0xFFu;
      const int r = (rd[j] >> 8) + (int)wh[d];
      rd[j] = r;
      s.keys[r] = key[j];
    }
  }
  if (tid < WALKERS) {
    u64 sum = 0;  // pair passes: the exclusive prefix; keys-only passes: both of them, packed
    if (tile == 0) {
      sum = VALS ? (u64)a.bin_offset[tid] : ((u64)a.bin_offset[tid + HB] << 31) | a.bin_offset[tid];
    } else {
      bool timed_out = false;
      // The walk over earlier tiles is a chain of dependent L2 reads (each some hundred
      // cycles): the descriptors of the next few tiles back are fetched together and consumed
      // in order, which divides the latency of a long walk by the batch size.  An unpublished
      // descriptor among them is waited for with the bounded wait.  An index below tile 0 is
      // clamped to tile 0, whose descriptor is an inclusive prefix from the start and ends the
      // walk before it is met twice.
      const u64 *sp = a.tile_state + tid;
      for (int lb_t = tile - 1;; lb_t -= RS_LOOKBACK_BATCH) {
        u64 lb[RS_LOOKBACK_BATCH];
#pragma unroll
        for (int i = 0; i < RS_LOOKBACK_BATCH; i++)
          lb[i] = ld_relaxed(sp + (size_t)max(lb_t - i, 0) * PER_TILE);
        bool done = false;
#pragma unroll
        for (int i = 0; i < RS_LOOKBACK_BATCH; i++) {
          if (done) continue;
          u64 x = lb[i];
          if (!rs_ready<VALS>(x, a.gen))
            x = rs_wait<VALS>(sp + (size_t)max(lb_t - i, 0) * PER_TILE, a.gen, a.status, &timed_out);
          sum += x & (VALS ? RS_VMASK : TD_MASK);
          done = (x >> 62) == TD_PREFIX;
        }
        if (done) break;
      }
      // a wait that gave up leaves the descriptor at its aggregate: the tiles behind this one
      // look past it, meet the same unpublished tile (or the error word) and give up as well
      if (timed_out) s.fail = 1;
      else if (VALS) st_relaxed(st, rs_pack<VALS>(TD_PREFIX, a.gen, sum + cnt));
      else st_relaxed(st, td_pack(TD_PREFIX, sum + (((u64)cnt_hi << 31) | cnt)));
    }
    if (VALS) {
      s.adj[tid] = (u32)sum - (u32)ex;
    } else {
      const u32 ex_hi = s.adj[tid + HB];
      s.adj[tid] = ((u32)sum & 0x7FFFFFFFu) - (u32)ex;
      s.adj[tid + HB] = ((u32)(sum >> 31) & 0x7FFFFFFFu) - ex_hi;
    }
  }
  __syncthreads();
  if (s.fail) return;
  u32 gpos[VALS ? ITEMS : 1];
#pragma unroll
  for (int k = 0; k < ITEMS; k++) {
    const int sl = tid + k * THREADS;
    if (VALS) gpos[k] = 0xFFFFFFFFu;
    if (FULL || sl < count) {
      const u64 kk = s.keys[sl];
      const u32 p = s.adj[(u32)(kk >> a.shift) & MASK] + (u32)sl;
      if (VALS) gpos[k] = p;
      a.keys_out[p] = kk;
    }
  }
  if (!VALS) return;
  __syncthreads();
  u32 *svals = reinterpret_cast<u32 *>(s.keys);
#pragma unroll
  for (int j = 0; j < ITEMS; j++) {
    const int li = wbase + j * 32 + lane;
    if (FULL || li < count) svals[rd[j]] = a.vals_in ? a.vals_in[base + li] : (u32)(base + li);
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < ITEMS; k++) {
    const int sl = tid + k * THREADS;
    if (FULL || sl < count) a.vals_out[gpos[VALS ? k : 0]] = svals[sl];
  }
}

template <int THREADS, int ITEMS, bool VALS, int BITS, bool STABLE, bool PREKEY>
__global__ void __launch_bounds__(THREADS, VALS ? RSP_MINB : RSK_MINB) k_radix_pass(RadixArgs a) {
  constexpr int TILE = THREADS * ITEMS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  RadixSmem<THREADS, ITEMS> &s = *reinterpret_cast<RadixSmem<THREADS, ITEMS> *>(smem_raw);
  const int tid = threadIdx.x;
  if (tid == 0) {
    s.tile = (int)atomicAdd(a.tile_counter, 1u);
    s.fail = ta_failed(a.status) ? 1 : 0;
  }
  for (int i = tid; i < (THREADS / 32) * RS_BINS; i += THREADS) (&s.warp_hist[0][0])[i] = 0;
  __syncthreads();
  if (s.fail) return;  // an earlier kernel failed: the keys may be incomplete
  const int tile = s.tile;
  if (PREKEY) {
    if (tid == 0) {
      const int64_t first = (int64_t)tile * TILE;
      int lo = 0, hi = a.pk.W - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (a.pk.off[mid] <= first) lo = mid;
        else hi = mid - 1;
      }
      s.win0 = lo;
    }
    __syncthreads();
  }
  const int count = (int)min((int64_t)TILE, a.n - (int64_t)tile * TILE);
  if (count == TILE) radix_tile<THREADS, ITEMS, VALS, BITS, true, STABLE, PREKEY>(a, s, tile, count);
  else radix_tile<THREADS, ITEMS, VALS, BITS, false, STABLE, PREKEY>(a, s, tile, count);
}

// tile shapes
#define RSP_THREADS 384  // pairs
#define RSP_ITEMS 12
#ifndef RSK_THREADS
#define RSK_THREADS 256  // keys only
#endif
#ifndef RSK_ITEMS
#define RSK_ITEMS 16
#endif

// digit histograms of every pass (used when the caller has none)
__global__ void __launch_bounds__(256) k_radix_hist(const u64 *keys, int64_t n, SortPlan plan,
                                                    u32 *hist) {
  // no failure check: reads keys by position only, and the passes that use the histogram check
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

SortPlan ta_make_plan(int lo_bit, int hi_bit) { return ta_plan_bits(lo_bit, hi_bit); }

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

template <int THREADS, int ITEMS, bool VALS, bool STABLE, bool PREKEY = false>
static cudaError_t launch_pass(const RadixArgs &a, int bits, unsigned tiles, cudaStream_t st) {
  typedef RadixSmem<THREADS, ITEMS> Smem;
#define RS_CASE(B)                                                                                  \
  case B: {                                                                                         \
    auto kern = k_radix_pass<THREADS, ITEMS, VALS, B, STABLE, PREKEY>;                                     \
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,         \
                                         (int)sizeof(Smem));                                        \
    if (e != cudaSuccess) return e;                                                                 \
    kern<<<TA_N tiles, THREADS, sizeof(Smem), st>>>(a);                                             \
    return cudaGetLastError();                                                                      \
  }
  switch (bits) {
    RS_CASE(1) RS_CASE(2) RS_CASE(3) RS_CASE(4) RS_CASE(5) RS_CASE(6) RS_CASE(7) RS_CASE(8)
  }
#undef RS_CASE
  return cudaErrorInvalidValue;
}

// Sorts n keys (vals: pairs) by the key bits the plan covers.  Pass outputs
// alternate between the scratch and the final buffers such that the last pass
// writes the final ones; keys_in / vals_in are only read (pairs with vals_in null:
// the value of element i is i).  keys_in must not alias scratch or final.
// `hist` = precomputed [pass][256] digit histograms, or null.
template <bool VALS>
static ta_status radix_sort(ta_window *h, const u64 *keys_in, const u32 *vals_in, u64 *keys_scratch,
                            u32 *vals_scratch, u64 *keys_final, u32 *vals_final, int64_t n,
                            const SortPlan &plan, const u32 *hist, void *temp,
                            bool first_pass_unstable, const PrekeyInfo *prekey) {
  if (n <= 0) return TA_OK;
  constexpr int THREADS = VALS ? RSP_THREADS : RSK_THREADS;
  constexpr int ITEMS = VALS ? RSP_ITEMS : RSK_ITEMS;
  constexpr int TILE = THREADS * ITEMS;
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
  // one clearing for all passes of a pair sort (descriptors tagged with their pass); every pass
  // draws its tile tickets from a counter of its own (state and counters are neighbours)
  TA_CHECK_CUDA(h, cudaMemsetAsync(state, 0, (size_t)((char *)(counter + 16) - (char *)state), st));
  const u64 *kin = keys_in;
  const u32 *vin = vals_in;
  for (int p = 0; p < plan.n_pass; p++) {
    bool to_final = ((plan.n_pass - 1 - p) & 1) == 0;
    RadixArgs a = RadixArgs();
    a.keys_in = kin; a.keys_out = to_final ? keys_final : keys_scratch;
    a.vals_in = vin; a.vals_out = to_final ? vals_final : vals_scratch;
    a.n = n; a.shift = plan.shift[p];
    a.bin_offset = bin_offset + p * RS_BINS;
    if (!VALS && p > 0)  // untagged descriptors: cleared in front of every pass
      TA_CHECK_CUDA(h, cudaMemsetAsync(state, 0, tiles * (RS_BINS / 2) * sizeof(u64), st));
    a.tile_state = state; a.tile_counter = counter + p; a.status = h->d_status;
    a.gen = VALS ? (u32)(p + 1) : 0u;
    const bool timed = g_ta_profile && n == h->n;  // only the timeline sort (all records)
    if (timed) ta_profile_mark(st, 1, (VALS ? 24.0 : 16.0) * (double)n);
    bool launched = false;
    if constexpr (!VALS) {
      if (p == 0 && first_pass_unstable) {
        if (prekey) {
          a.pk = *prekey;
          TA_CHECK_CUDA(h, (launch_pass<THREADS, ITEMS, false, false, true>(a, plan.bits[p], (unsigned)tiles, st)));
        } else {
          TA_CHECK_CUDA(h, (launch_pass<THREADS, ITEMS, false, false>(a, plan.bits[p], (unsigned)tiles, st)));
        }
        launched = true;
      }
    }
    if (!launched)
      TA_CHECK_CUDA(h, (launch_pass<THREADS, ITEMS, VALS, true>(a, plan.bits[p], (unsigned)tiles, st)));
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
                          plan, hist, temp, false, nullptr);
}

ta_status ta_radix_sort_keys(ta_window *h, const u64 *keys_in, u64 *keys_scratch, u64 *keys_final,
                             int64_t n, const SortPlan &plan, const u32 *hist, void *temp,
                             bool first_pass_unstable, const PrekeyInfo *prekey) {
  return radix_sort<false>(h, keys_in, nullptr, keys_scratch, nullptr, keys_final, nullptr, n, plan,
                           hist, temp, first_pass_unstable, prekey);
}
