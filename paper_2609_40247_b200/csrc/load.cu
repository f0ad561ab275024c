// ta_load_window kernels: validity (a record belongs to the window in which it
// starts, Sec. 5.2), discovery and dense ranking of the (pid, domain, stream) triples
// that name a lane, and the 64-bit sort key together with the digit histograms
// of every radix pass.
//   k_plan          one CTA samples the records and decides how many time bits the packed
//                   sort key keeps (before anything is known about the lanes);
//   k_discover      one pass over the 40-byte records: defect counters, the triple and
//                   communicator sets, value ranges, and one 64-bit word per record
//                   (dropped flag | triple slot | ts_start - t0);
//   k_discover_staged  the same for 16-byte aligned input, tiles of records brought to shared
//                   memory by bulk asynchronous copies (two tiles in flight per CTA); it also
//                   takes the digit histograms of the radix passes over the time bits and
//                   counts the records of every triple, so that the first radix pass can build
//                   the keys itself and no separate key pass is needed;
//   k_top_hist*     digit histograms of the passes over the (window, lane) bits, from the
//                   per-triple counts (one window) or from the words (several);
//   k_rank_*        one CTA each: sort and rank the few triples / communicator ids;
//   k_load_pre      turns those words into keys in place - [dropped][window][triple
//                   rank][(ts_start - t0) >> dshift]{[index in window]} - and takes the
//                   histograms; k_load does the same from the records when the sort
//                   falls back to full-resolution (key, index) pairs.
// The records are streamed once here and gathered once by the sort.
#include "ta_internal.cuh"
#include "records.cuh"

#define TRIPLE_EMPTY (~0ull)

__device__ __forceinline__ i64 warp_min_i64(i64 v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = min(v, (i64)__shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ i64 warp_max_i64(i64 v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, (i64)__shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Pass 1 over the records: defect counters, the set of lane triples, the range
// of name ids and the longest duration.  It also leaves one 64-bit word per record with
// all the key pass needs - bit 63 for a dropped record, else the triple's slot in the hash
// table (13 bits) and ts_start - t0 (40 bits) - so that the 40-byte records are read once.
#define PRE_DROPPED (1ull << 63)
#define PRE_TS_BITS 40
__global__ void __launch_bounds__(256) k_discover(const ta_event *ev, int64_t n, const int64_t *off,
                                                  const int64_t *t0, const int64_t *t1, int W,
                                                  TripleTable *tt, CommTable *cm,
                                                  ta_load_summary *sum, int64_t *misc,
                                                  int32_t *status, u64 *prekey) {
  __shared__ u64 cache[256];  // (triple code << 13) | slot: one word, so a racing reader sees a pair
  __shared__ u64 ccache[64];
  cache[threadIdx.x] = TRIPLE_EMPTY;
  if (threadIdx.x < 64) ccache[threadIdx.x] = TRIPLE_EMPTY;
  __syncthreads();
  i64 mn = INT64_MAX, mx = INT64_MIN, md = 0, qmn = INT64_MAX, qmx = INT64_MIN;
  u64 n_coll = 0;  // kept COLL records: sizes the collective matching without a count round trip
  WindowWalker ww(off, W);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    Rec r = load_rec(ev, i);
    int w = ww.at(i);
    int def = defect_of(r, t0[w], t1[w]);
    if (def) {
      int64_t *f = def == 1 ? &sum[w].n_bad_kind
                            : def == 2 ? &sum[w].n_bad_interval : &sum[w].n_out_of_window;
      atomicAdd((u64 *)f, 1ull);
      prekey[i] = PRE_DROPPED;
      continue;
    }
    mn = min(mn, (i64)r.name);
    mx = max(mx, (i64)r.name);
    md = max(md, r.ts_end - r.ts_start);
    if (r.kind == TA_KIND_COLL) {  // communicator set and sequence range
      n_coll++;
      qmn = min(qmn, (i64)r.seq);
      qmx = max(qmx, (i64)r.seq);
      u64 cc = (u64)r.corr ^ (1ull << 63);
      u32 ch = hash_code(cc);
      if (cc == TRIPLE_EMPTY) ta_set_err(status, TA_ERR_INVALID_ARG);  // reserved id
      else if (ccache[ch & 63] != cc) {
        u32 slot = ch & (TA_COMM_SLOTS - 1);
        bool ok = false;
        for (int probe = 0; probe < TA_COMM_SLOTS; probe++) {
          u64 cur = ld_relaxed(&cm->slots[slot]);
          if (cur == cc) { ok = true; break; }
          if (cur == TRIPLE_EMPTY) {
            u64 old = atomicCAS(&cm->slots[slot], TRIPLE_EMPTY, cc);
            if (old == TRIPLE_EMPTY || old == cc) { ok = true; break; }
          }
          slot = (slot + 1) & (TA_COMM_SLOTS - 1);
        }
        if (!ok) ta_set_err(status, TA_ERR_TOO_LARGE);
        ccache[ch & 63] = cc;
      }
    }
    u64 code = triple_code(r.pid, r.kind, r.stream);
    u32 hsh = hash_code(code);
    const u64 ts_rel = (u64)(r.ts_start - t0[w]);
    const u64 hit = cache[hsh & 255];
    if ((hit >> 13) == code) {  // a stale miss only costs a probe
      prekey[i] = ((hit & (TA_TRIPLE_SLOTS - 1)) << PRE_TS_BITS) | ts_rel;
      continue;
    }
    u32 slot = hsh & (TA_TRIPLE_SLOTS - 1);
    bool done = false;
    for (int probe = 0; probe < TA_TRIPLE_SLOTS; probe++) {
      u64 cur = ld_relaxed(&tt->slots[slot]);
      if (cur == code) { done = true; break; }
      if (cur == TRIPLE_EMPTY) {
        u64 old = atomicCAS(&tt->slots[slot], TRIPLE_EMPTY, code);
        if (old == TRIPLE_EMPTY || old == code) { done = true; break; }
      }
      slot = (slot + 1) & (TA_TRIPLE_SLOTS - 1);
    }
    if (!done) ta_set_err(status, TA_ERR_TOO_LARGE);
    cache[hsh & 255] = (code << 13) | slot;
    prekey[i] = ((u64)slot << PRE_TS_BITS) | ts_rel;
  }
  mn = warp_min_i64(mn);
  mx = warp_max_i64(mx);
  md = warp_max_i64(md);
  qmn = warp_min_i64(qmn);
  qmx = warp_max_i64(qmx);
  n_coll = warp_reduce(n_coll, OpAdd());
  if ((threadIdx.x & 31) == 0 && qmn != INT64_MAX) {
    atomicMin((i64 *)&misc[3], qmn);
    atomicMax((i64 *)&misc[4], qmx);
    atomicAdd((u64 *)&misc[5], n_coll);
  }
  if ((threadIdx.x & 31) == 0) {
    if (mn != INT64_MAX) {
      atomicMin((i64 *)&misc[0], mn);
      atomicMax((i64 *)&misc[1], mx);
    }
    if (md > 0) atomicMax((i64 *)&misc[2], md);
  }
}

// ---- planning: how many time bits the packed key keeps -----------------------------------
// The sort settles the order down to cells of 2^d ns; records of one lane that share a cell
// are ranked afterwards, which stays cheap while cells rarely hold more than one record.  One
// CTA samples up to 4096 records spread over the input, estimates the size of the largest
// lane and keeps the smallest number of whole radix passes over time bits for which the
// expected occupancy of a cell (largest lane x cell / span) stays at or below 1/4.  Any answer
// is correct (long runs fall back to full resolution); the estimate only steers the cost.
// misc[6] <- time bits kept, misc[7] <- estimated size of the largest lane.
#define PL_THREADS 1024
#define PL_PER_THREAD 4
#define PL_SLOTS 2048
__global__ void __launch_bounds__(PL_THREADS) k_plan(const ta_event *ev, int64_t n, const int64_t *off,
                                                     const int64_t *t0, const int64_t *t1, int W,
                                                     int sbits, int64_t max_span, int64_t max_win,
                                                     int64_t *misc) {
  __shared__ u64 code[PL_SLOTS];
  __shared__ u32 cnt[PL_SLOTS];
  __shared__ u32 s_max, s_valid;
  for (int i = threadIdx.x; i < PL_SLOTS; i += PL_THREADS) { code[i] = TRIPLE_EMPTY; cnt[i] = 0; }
  if (threadIdx.x == 0) { s_max = 0; s_valid = 0; }
  __syncthreads();
  const int64_t S = n < (int64_t)PL_THREADS * PL_PER_THREAD ? n : (int64_t)PL_THREADS * PL_PER_THREAD;
  for (int j = 0; j < PL_PER_THREAD; j++) {
    const int64_t k = (int64_t)j * PL_THREADS + threadIdx.x;
    if (k >= S) break;
    const int64_t i = k * (n / S);  // S <= n: evenly spread, in range
    const Rec r = load_rec(ev, i);
    const int w = window_of(off, W, i);
    if (defect_of(r, t0[w], t1[w])) continue;
    atomicAdd(&s_valid, 1u);
    // lanes are per window: the window is part of the sampled code
    const u64 c = triple_code(r.pid, r.kind, r.stream) ^ ((u64)w * 0x9E3779B97F4A7C15ull);
    u32 slot = hash_code(c) & (PL_SLOTS - 1);
    for (int probe = 0; probe < 64; probe++) {  // a table that fills up only loses samples
      const u64 cur = code[slot];
      if (cur == c) { atomicAdd(&cnt[slot], 1u); break; }
      if (cur == TRIPLE_EMPTY) {
        const u64 old = atomicCAS(&code[slot], TRIPLE_EMPTY, c);
        if (old == TRIPLE_EMPTY || old == c) { atomicAdd(&cnt[slot], 1u); break; }
      }
      slot = (slot + 1) & (PL_SLOTS - 1);
    }
  }
  __syncthreads();
  u32 m = 0;
  for (int i = threadIdx.x; i < PL_SLOTS; i += PL_THREADS) m = max(m, cnt[i]);
  m = (u32)warp_reduce((u64)m, OpMax());
  if ((threadIdx.x & 31) == 0) atomicMax(&s_max, m);
  __syncthreads();
  if (threadIdx.x == 0) {
    // few samples in the fullest lane say little: take at least 32 of them for granted
    const double per_sample = S > 0 ? (double)n / (double)S : 1.0;
    double est = (double)(s_max < 32u ? 32u : s_max) * per_sample;
    if (est > (double)max_win) est = (double)max_win;
    if (est < 1.0) est = 1.0;
    int keep = sbits;
    for (int passes = 1; passes * 8 < sbits; passes++) {
      const int d = sbits - passes * 8;
      if (est * (double)(1ull << d) / (double)max_span <= 0.25) { keep = passes * 8; break; }
    }
    misc[6] = keep;
    misc[7] = (int64_t)est;
  }
}

// ---- discovery with staged tiles -----------------------------------------------------------
#ifndef DS_THREADS
#define DS_THREADS 256
#endif
#ifndef DS_RPT
#define DS_RPT 2                          // records per thread and tile
#endif
#define DS_TILE (DS_THREADS * DS_RPT)     // 512 records = 20480 bytes
#define DS_TILE_BYTES (DS_TILE * 40)
#define DS_WAIT_POLLS (1 << 18)  // a tile arrives within microseconds; each poll may itself wait a little

__device__ __forceinline__ u32 smem_addr(const void *p) { return (u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(u64 *bar, u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
// one tile of whole records from this GPU's memory into shared memory: a 1-D bulk copy (no
// tensor map; the copy goes to this CTA alone) that reports its bytes to the barrier
__device__ __forceinline__ void bulk_load(void *dst, const void *src, u32 bytes, u64 *bar) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_addr(dst)),
      "l"(src), "r"(bytes), "r"(smem_addr(bar))
      : "memory");
}
// bounded wait for the phase with the given parity; false = gave up
__device__ __forceinline__ bool mbar_wait(u64 *bar, u32 parity) {
  for (int polls = 0; polls < DS_WAIT_POLLS; polls++) {
    u32 done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

struct DiscoverArgs {
  const ta_event *ev;
  int64_t n;
  const int64_t *off, *t0, *t1;
  int W;
  TripleTable *tt;
  CommTable *cm;
  ta_load_summary *sum;
  int64_t *misc;
  int32_t *status;
  u64 *prekey;
  u32 *hist;      // [pass][256]: digit histograms of the passes over time bits
  u32 *slot_cnt;  // [TA_TRIPLE_SLOTS] kept records per triple slot, or null (several windows)
  int sbits, ibits;
};

struct __align__(128) DiscoverSmem {
  unsigned char buf[2][DS_TILE_BYTES];
  u64 bar[2];
  u64 cache[256];
  u64 ccache[64];
  u32 hist[5][256];
  int fail;
};

__global__ void __launch_bounds__(DS_THREADS) k_discover_staged(DiscoverArgs a) {
  extern __shared__ __align__(128) unsigned char ds_raw[];
  DiscoverSmem &s = *reinterpret_cast<DiscoverSmem *>(ds_raw);
  const int tid = threadIdx.x, lane = tid & 31;
  for (int i = tid; i < 256; i += DS_THREADS) s.cache[i] = TRIPLE_EMPTY;
  if (tid < 64) s.ccache[tid] = TRIPLE_EMPTY;
  for (int i = tid; i < 5 * 256; i += DS_THREADS) (&s.hist[0][0])[i] = 0;
  if (tid == 0) {
    mbar_init(&s.bar[0], 1);
    mbar_init(&s.bar[1], 1);
    s.fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // passes over the time bits kept (decided by k_plan): digit p = (ts_rel >> sh[p]) & mk[p]
  const int keep = (int)a.misc[6];
  const int dshift = a.sbits - keep;
  const SortPlan tp = ta_plan_bits(0, keep);
  const int n_tp = tp.n_pass <= 5 ? tp.n_pass : 0;  // more than five time passes: no histograms here
  int sh[5];
  u32 mk[5];
#pragma unroll
  for (int p = 0; p < 5; p++) {
    sh[p] = dshift + tp.shift[p];
    mk[p] = (1u << tp.bits[p]) - 1u;
  }
  const int64_t n_tiles = (a.n + DS_TILE - 1) / DS_TILE;
  // name and sequence ranges in 32 bits (the fields are int32), folded to 64 at the end
  int32_t mn = INT32_MAX, mx = INT32_MIN, qmn = INT32_MAX, qmx = INT32_MIN;
  i64 md = 0;
  u32 n_coll = 0;
  WindowWalker ww(a.off, a.W);
  int cw = -1;  // window whose bounds are in registers
  i64 ct0 = 0, ct1 = 0;
  int64_t tile = blockIdx.x;
  auto tile_bytes = [&](int64_t t) -> u32 {
    const int64_t cntr = min((int64_t)DS_TILE, a.n - t * DS_TILE);
    return (u32)(cntr * 40);
  };
  // a tile whose size is no multiple of 16 bytes (an odd number of records, the last tile only)
  // is copied with plain loads instead
  if (tid == 0 && tile < n_tiles && (tile_bytes(tile) & 15u) == 0)
    bulk_load(s.buf[0], reinterpret_cast<const unsigned char *>(a.ev) + tile * DS_TILE_BYTES, tile_bytes(tile),
              &s.bar[0]);
  for (int it = 0; tile < n_tiles; tile += gridDim.x, it++) {
    const int cur = it & 1;
    const int64_t nxt = tile + gridDim.x;
    if (tid == 0 && nxt < n_tiles && (tile_bytes(nxt) & 15u) == 0)
      bulk_load(s.buf[cur ^ 1], reinterpret_cast<const unsigned char *>(a.ev) + nxt * DS_TILE_BYTES,
                tile_bytes(nxt), &s.bar[cur ^ 1]);
    const u32 bytes = tile_bytes(tile);
    const int count = (int)(bytes / 40);
    if ((bytes & 15u) == 0) {
      // one thread polls the barrier; the others sleep at the block barrier below instead of
      // spending issue slots on polls
      if (tid == 0 && !mbar_wait(&s.bar[cur], (u32)((it >> 1) & 1))) s.fail = 1;
    } else {
      const u64 *src = reinterpret_cast<const u64 *>(a.ev) + tile * (DS_TILE * 5);
      u64 *dst = reinterpret_cast<u64 *>(s.buf[cur]);
      for (int k = tid; k < count * 5; k += DS_THREADS) dst[k] = __ldg(src + k);
    }
    __syncthreads();
    if (s.fail) {  // the copy never arrived: report and leave (nothing this CTA holds is pending use)
      if (tid == 0) ta_set_err(a.status, TA_ERR_TIMEOUT);
      return;
    }
#pragma unroll
    for (int j = 0; j < DS_RPT; j++) {
      const int rl = j * DS_THREADS + tid;
      const bool in = rl < count;
      const int64_t i = tile * DS_TILE + rl;
      int slot_mine = -1;  // triple slot of a kept record
      u64 trel = 0;
      if (in) {
        const u64 *q = reinterpret_cast<const u64 *>(s.buf[cur] + (size_t)rl * 40);
        Rec r;
        r.ts_start = (i64)q[0];
        r.ts_end = (i64)q[1];
        r.corr = (i64)q[2];
        const u64 x = q[3], y = q[4];
        r.pid = (int32_t)(u32)x;
        r.name = (int32_t)(u32)(x >> 32);
        r.seq = (int32_t)(u32)y;
        r.stream = (int16_t)(uint16_t)(y >> 32);
        r.kind = (int16_t)(uint16_t)(y >> 48);
        const int w = ww.at(i);
        if (w != cw) { cw = w; ct0 = a.t0[w]; ct1 = a.t1[w]; }
        const int def = defect_of(r, ct0, ct1);
        if (def) {
          int64_t *f = def == 1 ? &a.sum[w].n_bad_kind
                                : def == 2 ? &a.sum[w].n_bad_interval : &a.sum[w].n_out_of_window;
          atomicAdd((u64 *)f, 1ull);
          a.prekey[i] = PRE_DROPPED;
        } else {
          mn = min(mn, r.name);
          mx = max(mx, r.name);
          md = max(md, r.ts_end - r.ts_start);
          if (r.kind == TA_KIND_COLL) {  // communicator set and sequence range
            n_coll++;
            qmn = min(qmn, r.seq);
            qmx = max(qmx, r.seq);
            const u64 cc = (u64)r.corr ^ (1ull << 63);
            const u32 ch = hash_code(cc);
            if (cc == TRIPLE_EMPTY) ta_set_err(a.status, TA_ERR_INVALID_ARG);  // reserved id
            else if (s.ccache[ch & 63] != cc) {
              u32 slot = ch & (TA_COMM_SLOTS - 1);
              bool ok = false;
              for (int probe = 0; probe < TA_COMM_SLOTS; probe++) {
                const u64 c2 = ld_relaxed(&a.cm->slots[slot]);
                if (c2 == cc) { ok = true; break; }
                if (c2 == TRIPLE_EMPTY) {
                  const u64 old = atomicCAS(&a.cm->slots[slot], TRIPLE_EMPTY, cc);
                  if (old == TRIPLE_EMPTY || old == cc) { ok = true; break; }
                }
                slot = (slot + 1) & (TA_COMM_SLOTS - 1);
              }
              if (!ok) ta_set_err(a.status, TA_ERR_TOO_LARGE);
              s.ccache[ch & 63] = cc;
            }
          }
          const u64 code = triple_code(r.pid, r.kind, r.stream);
          const u32 hsh = hash_code(code);
          trel = (u64)(r.ts_start - ct0);
          const u64 hit = s.cache[hsh & 255];
          if ((hit >> 13) == code) {  // a stale miss only costs a probe
            slot_mine = (int)(hit & (TA_TRIPLE_SLOTS - 1));
          } else {
            u32 slot = hsh & (TA_TRIPLE_SLOTS - 1);
            bool done = false;
            for (int probe = 0; probe < TA_TRIPLE_SLOTS; probe++) {
              const u64 c2 = ld_relaxed(&a.tt->slots[slot]);
              if (c2 == code) { done = true; break; }
              if (c2 == TRIPLE_EMPTY) {
                const u64 old = atomicCAS(&a.tt->slots[slot], TRIPLE_EMPTY, code);
                if (old == TRIPLE_EMPTY || old == code) { done = true; break; }
              }
              slot = (slot + 1) & (TA_TRIPLE_SLOTS - 1);
            }
            if (!done) ta_set_err(a.status, TA_ERR_TOO_LARGE);
            s.cache[hsh & 255] = (code << 13) | slot;
            slot_mine = (int)slot;
          }
          a.prekey[i] = ((u64)slot_mine << PRE_TS_BITS) | trel;
        }
      }
      // digit histograms of the time passes (dropped records count in digit 0 later, from the
      // defect counters).  The upper digits are the same for a whole warp most of the time
      // (neighbouring records are close in time): one vote, one add.
      const u32 kept = __ballot_sync(0xffffffffu, slot_mine >= 0);
      if (kept) {
        const int leader = __ffs(kept) - 1;
#pragma unroll
        for (int p = 0; p < 5; p++) {
          if (p >= n_tp) break;
          const u32 d = (u32)(trel >> sh[p]) & mk[p];
          if (p >= 1) {
            const u32 d0 = __shfl_sync(0xffffffffu, d, leader);
            if (__all_sync(0xffffffffu, slot_mine < 0 || d == d0)) {
              if (lane == leader) atomicAdd(&s.hist[p][d0], (u32)__popc(kept));
              continue;
            }
          }
          if (slot_mine >= 0) atomicAdd(&s.hist[p][d], 1u);
        }
        // records per triple slot: one add per distinct slot of the warp
        if (a.slot_cnt) {
          u32 left = kept;
          while (left) {
            const int ld = __ffs(left) - 1;
            const int sv = __shfl_sync(0xffffffffu, slot_mine, ld);
            const u32 same = __ballot_sync(0xffffffffu, slot_mine == sv) & left;
            if (lane == ld) atomicAdd(&a.slot_cnt[sv], (u32)__popc(same));
            left &= ~same;
          }
        }
      }
    }
    __syncthreads();  // every thread is done with buf[cur] before the next copy into it is issued
  }
  for (int i = tid; i < n_tp * 256; i += DS_THREADS) {
    const u32 c = (&s.hist[0][0])[i];
    if (c) atomicAdd(&a.hist[i], c);
  }
  mn = __reduce_min_sync(0xffffffffu, mn);
  mx = __reduce_max_sync(0xffffffffu, mx);
  qmn = __reduce_min_sync(0xffffffffu, qmn);
  qmx = __reduce_max_sync(0xffffffffu, qmx);
  n_coll = __reduce_add_sync(0xffffffffu, n_coll);
  md = warp_max_i64(md);
  if (lane == 0 && n_coll) {
    atomicMin((i64 *)&a.misc[3], (i64)qmn);
    atomicMax((i64 *)&a.misc[4], (i64)qmx);
    atomicAdd((u64 *)&a.misc[5], (u64)n_coll);
  }
  if (lane == 0) {
    if (mn <= mx) {
      atomicMin((i64 *)&a.misc[0], (i64)mn);
      atomicMax((i64 *)&a.misc[1], (i64)mx);
    }
    if (md > 0) atomicMax((i64 *)&a.misc[2], md);
  }
}

// ---- histograms of the passes over the (dropped, window, triple rank) bits ------------------
struct TopHistArgs {
  SortPlan plan;        // the whole plan; passes [n_time, n_pass) are the top passes
  int n_time;
  int top_lo;           // key bit where the top bits begin (index bits + time bits kept)
  int tbits, wbits;
  int64_t n_dropped;
  const TripleTable *tt;
  const u32 *slot_cnt;
  u32 *hist;            // [pass][256]
  // several windows: from the words
  const u64 *prekey;
  int64_t n;
  const int64_t *off;
  int W;
};
__device__ __forceinline__ void top_hist_add(const TopHistArgs &a, u32 *hist, u64 c, u32 count) {
  for (int p = a.n_time; p < a.plan.n_pass; p++) {
    const u32 d = (u32)(c >> (a.plan.shift[p] - a.top_lo)) & ((1u << a.plan.bits[p]) - 1u);
    atomicAdd(&hist[p * 256 + d], count);
  }
}
// one window: the lane sizes are the per-triple counts
__global__ void __launch_bounds__(1024) k_top_hist(TopHistArgs a) {
  for (int sl = threadIdx.x; sl < TA_TRIPLE_SLOTS; sl += blockDim.x) {
    const u32 c = a.slot_cnt[sl];
    if (c) top_hist_add(a, a.hist, (u64)a.tt->rank_of_slot[sl], c);
  }
  if (threadIdx.x == 0) {
    if (a.n_dropped > 0) {
      top_hist_add(a, a.hist, 1ull << (a.wbits + a.tbits), (u32)a.n_dropped);
      for (int p = 0; p < a.n_time; p++) atomicAdd(&a.hist[p * 256], (u32)a.n_dropped);  // time digits 0
    }
  }
}
// several windows: one pass over the words (8 bytes per record)
__global__ void __launch_bounds__(256) k_top_hist_words(TopHistArgs a) {
  __shared__ u32 sh[10 * 256];
  for (int i = threadIdx.x; i < a.plan.n_pass * 256; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  WindowWalker ww(a.off, a.W);
  const int64_t n_round = ((a.n + 31) / 32) * 32;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_round;
       i += (int64_t)gridDim.x * blockDim.x) {
    const bool in = i < a.n;
    u64 c = 0;
    bool dropped = false;
    if (in) {
      const u64 pk = a.prekey[i];
      const int w = ww.at(i);
      dropped = (pk & PRE_DROPPED) != 0;
      if (dropped) c = (1ull << (a.wbits + a.tbits)) | ((u64)w << a.tbits);
      else c = ((u64)w << a.tbits) |
               (u64)__ldg(&a.tt->rank_of_slot[(u32)(pk >> PRE_TS_BITS) & (TA_TRIPLE_SLOTS - 1)]);
    }
    // neighbouring records mostly share window and lane: one vote, one add per pass
    const u32 act = __ballot_sync(0xffffffffu, in);
    if (!act) continue;
    const int leader = __ffs(act) - 1;
    const u64 c0 = __shfl_sync(0xffffffffu, c, leader);
    const bool same = __all_sync(0xffffffffu, !in || c == c0);
    const u32 nd = __popc(__ballot_sync(0xffffffffu, in && dropped));
    if (same) {
      if ((threadIdx.x & 31) == leader) top_hist_add(a, sh, c0, (u32)__popc(act));
    } else if (in) {
      top_hist_add(a, sh, c, 1u);
    }
    if ((threadIdx.x & 31) == leader && nd)
      for (int p = 0; p < a.n_time; p++) atomicAdd(&sh[p * 256], nd);  // time digits 0
  }
  __syncthreads();
  for (int i = threadIdx.x; i < a.plan.n_pass * 256; i += blockDim.x)
    if (sh[i]) atomicAdd(&a.hist[i], sh[i]);
}

// One CTA: sorts the discovered triples, ranks them and the pids they contain.
__device__ __forceinline__ void rank_triples(TripleTable *tt, int32_t *status, u64 *buf /* TA_TRIPLE_SLOTS */) {
  __shared__ u64 tmp[33];
  __shared__ int n_tr;
  const int tid = threadIdx.x;
  // the occupied slots, packed to the front (a window has tens of triples, not thousands)
  if (tid == 0) n_tr = 0;
  __syncthreads();
  for (int c0 = 0; c0 < TA_TRIPLE_SLOTS; c0 += blockDim.x) {
    const u64 v = tt->slots[c0 + tid];
    u64 total;
    const u64 ex = block_scan_exclusive<OpAdd>(v != TRIPLE_EMPTY ? 1ull : 0ull, OpAdd(), tmp, &total);
    if (v != TRIPLE_EMPTY) buf[n_tr + (int)ex] = v;
    __syncthreads();
    if (tid == 0) n_tr += (int)total;
    __syncthreads();
  }
  int padded = 32;
  while (padded < n_tr) padded <<= 1;
  for (int i = n_tr + tid; i < padded; i += blockDim.x) buf[i] = TRIPLE_EMPTY;  // sorts last
  __syncthreads();
  for (int k = 2; k <= padded; k <<= 1)
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = tid; i < padded; i += blockDim.x) {
        int ixj = i ^ j;
        if (ixj > i) {
          u64 a = buf[i], b = buf[ixj];
          bool up = (i & k) == 0;
          if ((a > b) == up) { buf[i] = b; buf[ixj] = a; }
        }
      }
      __syncthreads();
    }
  int n = n_tr;
  if (n > TA_MAX_TRIPLES) {
    if (tid == 0) ta_set_err(status, TA_ERR_TOO_LARGE);
    n = TA_MAX_TRIPLES;
  }
  for (int i = tid; i < n; i += blockDim.x) tt->sorted_code[i] = buf[i];
  if (tid == 0) {
    int pr = -1;
    u64 prev = ~0ull;
    for (int i = 0; i < n; i++) {
      u64 pidb = buf[i] >> 17;
      if (pidb != prev) { pr++; prev = pidb; tt->pid_value[pr] = (int32_t)((u32)pidb ^ 0x80000000u); }
      tt->pid_rank[i] = pr;
    }
    status[ST_N_TRIPLES] = n;
    status[ST_N_PIDS] = pr + 1;
  }
  for (int s = tid; s < TA_TRIPLE_SLOTS; s += blockDim.x) {
    u64 c = tt->slots[s];
    int r = -1;
    if (c != TRIPLE_EMPTY) {
      int lo = 0, hi = n - 1;
      while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (buf[mid] < c) lo = mid + 1;
        else hi = mid;
      }
      r = lo;
    }
    tt->rank_of_slot[s] = r;
  }
}

// One CTA: sorts and ranks the communicator ids.
__device__ __forceinline__ void rank_comms(CommTable *cm, int32_t *status, u64 *buf /* TA_COMM_SLOTS */) {
  __shared__ int n_c;
  const int tid = threadIdx.x;
  for (int i = tid; i < TA_COMM_SLOTS; i += blockDim.x) buf[i] = cm->slots[i];
  if (tid == 0) n_c = 0;
  __syncthreads();
  for (int k = 2; k <= TA_COMM_SLOTS; k <<= 1)
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = tid; i < TA_COMM_SLOTS; i += blockDim.x) {
        int ixj = i ^ j;
        if (ixj > i) {
          u64 a = buf[i], b = buf[ixj];
          bool up = (i & k) == 0;
          if ((a > b) == up) { buf[i] = b; buf[ixj] = a; }
        }
      }
      __syncthreads();
    }
  for (int i = tid; i < TA_COMM_SLOTS; i += blockDim.x)
    if (buf[i] != TRIPLE_EMPTY && (i + 1 == TA_COMM_SLOTS || buf[i + 1] == TRIPLE_EMPTY)) n_c = i + 1;
  __syncthreads();
  int n = n_c;
  if (n > TA_MAX_COMMS) {
    if (tid == 0) ta_set_err(status, TA_ERR_TOO_LARGE);
    n = TA_MAX_COMMS;
  }
  for (int i = tid; i < n; i += blockDim.x) cm->sorted_id[i] = buf[i];
  if (tid == 0) status[ST_N_COMMS] = n;
  for (int s = tid; s < TA_COMM_SLOTS; s += blockDim.x) {
    u64 c = cm->slots[s];
    int r = -1;
    if (c != TRIPLE_EMPTY) {
      int lo = 0, hi = n - 1;
      while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (buf[mid] < c) lo = mid + 1;
        else hi = mid;
      }
      r = lo;
    }
    cm->rank_of_slot[s] = r;
  }
}

// Both rankings in one launch: CTA 0 the triples, CTA 1 the communicator ids (they are
// independent, and two single-CTA kernels one after the other cost a launch latency more).
__global__ void __launch_bounds__(1024) k_rank(TripleTable *tt, CommTable *cm, int32_t *status) {
  extern __shared__ u64 rank_buf[];  // TA_TRIPLE_SLOTS
  if (blockIdx.x == 0) rank_triples(tt, status, rank_buf);
  else rank_comms(cm, status, rank_buf);
}

struct LoadArgs {
  const ta_event *ev;
  int64_t n;
  const int64_t *off, *t0, *t1;
  int W;
  const TripleTable *tt;
  u64 *keys;
  u32 *hist;
  int sbits, tbits, wbits;
  int packed, dshift, ibits;  // packed: key also carries the index inside the window (low ibits)
  SortPlan plan;
  int32_t *status;
};

// Pass 2 over the records: sort key and the digit histograms of all passes.
__global__ void __launch_bounds__(256) k_load(LoadArgs a) {
  __shared__ u32 sh[10 * 256];
  for (int i = threadIdx.x; i < a.plan.n_pass * 256; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const int tsb = a.sbits - a.dshift;  // time bits kept in the key
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t n_round = ((a.n + 31) / 32) * 32;  // keep warps converged for the votes
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_round; i += stride) {
    bool in = i < a.n;
    u64 key = 0;
    if (in) {
      Rec r = load_rec(a.ev, i);
      int w = window_of(a.off, a.W, i);
      u64 hi;  // [dropped][window][triple rank][time]
      if (defect_of(r, a.t0[w], a.t1[w])) {
        hi = (1ull << (a.wbits + a.tbits + tsb)) | ((u64)w << (a.tbits + tsb));
        if (!a.packed) hi = 1ull << (a.wbits + a.tbits + tsb);
      } else {
        u64 code = triple_code(r.pid, r.kind, r.stream);
        // the discovery pass inserted every triple; a record that is not found was changed
        // behind the library's back (the records are borrowed): bounded probe, error, rank 0
        u32 slot = hash_code(code) & (TA_TRIPLE_SLOTS - 1);
        int probes = 0;
        while (__ldg(&a.tt->slots[slot]) != code && ++probes < TA_TRIPLE_SLOTS)
          slot = (slot + 1) & (TA_TRIPLE_SLOTS - 1);
        u64 rank = 0;
        if (probes < TA_TRIPLE_SLOTS) rank = (u64)__ldg(&a.tt->rank_of_slot[slot]);
        else ta_set_err(a.status, TA_ERR_OVERFLOW);
        hi = ((u64)w << (a.tbits + tsb)) | (rank << tsb) | ((u64)(r.ts_start - a.t0[w]) >> a.dshift);
      }
      key = a.packed ? (hi << a.ibits) | (u64)(i - a.off[w]) : hi;
      a.keys[i] = key;
    }
    u32 active = __ballot_sync(0xffffffffu, in);
    if (!in) continue;
    const int lane = threadIdx.x & 31;
    const int leader = __ffs(active) - 1;
    for (int p = 0; p < a.plan.n_pass; p++) {
      // high digits are the same across a warp most of the time: one vote, one add
      u32 d = (u32)(key >> a.plan.shift[p]) & ((1u << a.plan.bits[p]) - 1u);
      u32 d0 = __shfl_sync(active, d, leader);
      if (__all_sync(active, d == d0)) {
        if (lane == leader) atomicAdd(&sh[p * 256 + d0], (u32)__popc(active));
      } else {
        atomicAdd(&sh[p * 256 + d], 1u);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < a.plan.n_pass * 256; i += blockDim.x)
    if (sh[i]) atomicAdd(&a.hist[i], sh[i]);
}

// The same from the words k_discover left in a.keys (rewritten in place): 8 B read + 8 B
// written per record instead of another pass over the 40-byte records.
__global__ void __launch_bounds__(256) k_load_pre(LoadArgs a) {
  __shared__ u32 sh[10 * 256];
  for (int i = threadIdx.x; i < a.plan.n_pass * 256; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const int tsb = a.sbits - a.dshift;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t n_round = ((a.n + 31) / 32) * 32;
  WindowWalker ww(a.off, a.W);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_round; i += stride) {
    bool in = i < a.n;
    u64 key = 0;
    if (in) {
      const u64 pk = a.keys[i];
      int w = ww.at(i);
      u64 hi;
      if (pk & PRE_DROPPED) {
        hi = (1ull << (a.wbits + a.tbits + tsb)) | ((u64)w << (a.tbits + tsb));
        if (!a.packed) hi = 1ull << (a.wbits + a.tbits + tsb);
      } else {
        const u32 slot = (u32)(pk >> PRE_TS_BITS) & (TA_TRIPLE_SLOTS - 1);
        const u64 rank = (u64)__ldg(&a.tt->rank_of_slot[slot]);
        hi = ((u64)w << (a.tbits + tsb)) | (rank << tsb) | ((pk & ((1ull << PRE_TS_BITS) - 1)) >> a.dshift);
      }
      key = a.packed ? (hi << a.ibits) | (u64)(i - a.off[w]) : hi;
      a.keys[i] = key;
    }
    u32 active = __ballot_sync(0xffffffffu, in);
    if (!in) continue;
    const int lane = threadIdx.x & 31;
    const int leader = __ffs(active) - 1;
    for (int p = 0; p < a.plan.n_pass; p++) {
      u32 d = (u32)(key >> a.plan.shift[p]) & ((1u << a.plan.bits[p]) - 1u);
      // only the two most significant digits (window, lane, top time bits) are ever the same for
      // a whole warp: the test is not worth its instructions on the others
      if (p >= a.plan.n_pass - 2) {
        u32 d0 = __shfl_sync(active, d, leader);
        if (__all_sync(active, d == d0)) {
          if (lane == leader) atomicAdd(&sh[p * 256 + d0], (u32)__popc(active));
          continue;
        }
      }
      atomicAdd(&sh[p * 256 + d], 1u);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < a.plan.n_pass * 256; i += blockDim.x)
    if (sh[i]) atomicAdd(&a.hist[i], sh[i]);
}

// ------------------------------------------------------------------ host
static int grid_for(int64_t n, int threads, int per_sm) {
  int64_t g = (n + threads - 1) / threads;
  int64_t cap = 148ll * per_sm;
  return (int)(g < 1 ? 1 : (g > cap ? cap : g));
}

ta_status ta_launch_discover(ta_window *h) {
  h->tkeep = 0;
  h->fast_keys = 0;
  if (h->n > 0) {
    if (((uintptr_t)h->events & 15u) == 0) {
      // 16-byte aligned records: plan the time resolution, then the staged pass that also takes
      // the histograms of the time passes and the per-triple counts
      int64_t max_span = 1, max_win = 1;
      for (int w = 0; w < h->W; w++) {
        max_span = max_span > h->h_t1[w] - h->h_t0[w] ? max_span : h->h_t1[w] - h->h_t0[w];
        max_win = max_win > h->h_off[w + 1] - h->h_off[w] ? max_win : h->h_off[w + 1] - h->h_off[w];
      }
      const int sbits = ta_bit_len((uint64_t)(max_span - 1));
      k_plan<<<TA_N 1, PL_THREADS, 0, h->stream>>>(h->events, h->n, h->d_off, h->d_t0, h->d_t1, h->W, sbits,
                                                  max_span, max_win, h->d_misc);
      DiscoverArgs a;
      a.ev = h->events; a.n = h->n; a.off = h->d_off; a.t0 = h->d_t0; a.t1 = h->d_t1; a.W = h->W;
      a.tt = h->d_triples; a.cm = h->d_comms; a.sum = h->d_load_sum; a.misc = h->d_misc;
      a.status = h->d_status; a.prekey = h->d_keys; a.hist = h->d_hist;
      a.slot_cnt = h->W == 1 ? h->d_slot_cnt : nullptr;
      a.sbits = sbits; a.ibits = 0;
      TA_CHECK_CUDA(h, cudaFuncSetAttribute(k_discover_staged, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)sizeof(DiscoverSmem)));
      const int64_t tiles = (h->n + DS_TILE - 1) / DS_TILE;
#ifndef DS_CTAS_PER_SM
#define DS_CTAS_PER_SM 4
#endif
      const int grid = (int)(tiles < 148 * DS_CTAS_PER_SM ? tiles : 148 * DS_CTAS_PER_SM);
      k_discover_staged<<<TA_N grid, DS_THREADS, sizeof(DiscoverSmem), h->stream>>>(a);
      h->tkeep = -1;  // read back with the other results of the pass
    } else {
      k_discover<<<TA_N grid_for(h->n, 256, 8), 256, 0, h->stream>>>(
          h->events, h->n, h->d_off, h->d_t0, h->d_t1, h->W, h->d_triples, h->d_comms, h->d_load_sum,
          h->d_misc, h->d_status, h->d_keys);
    }
    h->prekeys = 1;
  }
  TA_CHECK_CUDA(h, cudaFuncSetAttribute(k_rank, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        TA_TRIPLE_SLOTS * (int)sizeof(u64)));
  k_rank<<<TA_N 2, 1024, TA_TRIPLE_SLOTS * sizeof(u64), h->stream>>>(h->d_triples, h->d_comms, h->d_status);
  TA_CHECK_CUDA(h, cudaGetLastError());
  return TA_OK;
}

// Chooses the key layout and launches k_load.  allow_packed: try the layout that also
// carries the record's index inside its window in the low bits, so that the sort
// moves 8-byte keys only; it needs (window + triple + time + index) bits to fit 64
// after giving up at most TA_PACK_MAX_DROP low time bits (records that collide in
// the coarser time are put right by the equal-key fix-up).
ta_status ta_launch_load(ta_window *h, bool allow_packed) {
  // key layout: [dropped][window][triple rank][(ts_start - t0) >> dshift]{[index in window]}
  int64_t max_span = 1, max_win = 1;
  for (int w = 0; w < h->W; w++) {
    max_span = max_span > h->h_t1[w] - h->h_t0[w] ? max_span : h->h_t1[w] - h->h_t0[w];
    max_win = max_win > h->h_off[w + 1] - h->h_off[w] ? max_win : h->h_off[w + 1] - h->h_off[w];
  }
  h->sbits = ta_bit_len((uint64_t)(max_span - 1));
  h->tbits = ta_bit_len((uint64_t)(h->n_triples > 0 ? h->n_triples - 1 : 0));
  h->wbits = ta_bit_len((uint64_t)(h->W - 1));
  const int hd = h->has_dropped ? 1 : 0;
  int total = h->sbits + h->tbits + h->wbits + hd;
  if (total > 63) return TA_ERR_TOO_LARGE;
  if (((int64_t)h->W << h->tbits) > (1ll << 24)) return TA_ERR_TOO_LARGE;
  h->ibits = ta_bit_len((uint64_t)(max_win - 1));
  if (h->ibits < 1) h->ibits = 1;
  h->fast_keys = 0;
  if (allow_packed && h->prekeys && h->tkeep > 0 && h->tkeep <= h->sbits) {
    // The staged discovery pass took the histograms of the passes over the time bits kept, and
    // the lane sizes give those of the passes above them: the first radix pass can build the
    // keys from the discovery words, no key pass is needed.  Passes over time bits and passes
    // over (dropped, window, triple rank) bits never share a digit.
    const int T = h->tkeep, L = hd + h->wbits + h->tbits;
    const SortPlan tp = ta_plan_bits(h->ibits, h->ibits + T);
    const SortPlan lp = ta_plan_bits(h->ibits + T, h->ibits + T + L);
    const int n_top = L > 0 ? lp.n_pass : 0;
    if (T + L + h->ibits <= 64 && tp.n_pass <= 5 && tp.n_pass + n_top <= 10) {
      h->packed = 1;
      h->dshift = h->sbits - T;
      h->plan = tp;
      for (int q = 0; q < n_top; q++) {
        h->plan.shift[tp.n_pass + q] = lp.shift[q];
        h->plan.bits[tp.n_pass + q] = lp.bits[q];
      }
      h->plan.n_pass = tp.n_pass + n_top;
      h->fast_keys = 1;
      if (h->n == 0) return TA_OK;
      TopHistArgs a;
      memset(&a, 0, sizeof(a));
      a.plan = h->plan; a.n_time = tp.n_pass; a.top_lo = h->ibits + T;
      a.tbits = h->tbits; a.wbits = h->wbits; a.n_dropped = h->n - h->n_valid;
      a.tt = h->d_triples; a.slot_cnt = h->d_slot_cnt; a.hist = h->d_hist;
      a.prekey = h->d_keys; a.n = h->n; a.off = h->d_off; a.W = h->W;
      if (h->W == 1) k_top_hist<<<TA_N 1, 1024, 0, h->stream>>>(a);
      else k_top_hist_words<<<TA_N grid_for(h->n, 256, 8), 256, 0, h->stream>>>(a);
      TA_CHECK_CUDA(h, cudaGetLastError());
      return TA_OK;  // the words stay in d_keys (h->prekeys stays set): a retry can still use them
    }
  }
  int drop = total + h->ibits - 64;
  if (drop < 0) drop = 0;
  h->packed = allow_packed && drop <= TA_PACK_MAX_DROP && drop < h->sbits;
  if (h->packed) {
    // Coarser time saves whole passes as long as records of one lane rarely share a time
    // bucket (the equal-key fix-up restores the exact order).  Allow a coarsening whose
    // expected bucket occupancy stays below 1/4, assuming lanes up to 4x the average size.
    const double per_lane = 4.0 * (double)(h->n_valid > 0 ? h->n_valid : 1) /
                            ((double)h->W * (double)(h->n_triples > 0 ? h->n_triples : 1));
    int best = drop, best_pass = (total - drop + 7) / 8;
    for (int d = drop + 1; d <= TA_PACK_MAX_DROP && d < h->sbits; d++) {
      if (per_lane * (double)(1ull << d) / (double)max_span > 0.25) break;
      const int np = (total - d + 7) / 8;
      if (np < best_pass) { best = d; best_pass = np; }
    }
    drop = best;
  }
  h->dshift = h->packed ? drop : 0;
  if (h->packed) h->plan = ta_make_plan(h->ibits, h->ibits + total - h->dshift);
  else h->plan = ta_make_plan(0, total);
  if (h->n == 0) return TA_OK;
  TA_CHECK_CUDA(h, cudaMemsetAsync(h->d_hist, 0, 10 * 256 * 4, h->stream));
  LoadArgs a;
  a.ev = h->events; a.n = h->n; a.off = h->d_off; a.t0 = h->d_t0; a.t1 = h->d_t1; a.W = h->W;
  a.tt = h->d_triples; a.keys = h->d_keys; a.hist = h->d_hist;
  a.sbits = h->sbits; a.tbits = h->tbits; a.wbits = h->wbits; a.plan = h->plan;
  a.packed = h->packed; a.dshift = h->dshift; a.ibits = h->ibits; a.status = h->d_status;
  // the words of the discovery pass are there once; a later call (the fall back to full
  // resolution keys) goes back to the records
  if (h->prekeys) k_load_pre<<<TA_N grid_for(h->n, 256, 8), 256, 0, h->stream>>>(a);
  else k_load<<<TA_N grid_for(h->n, 256, 8), 256, 0, h->stream>>>(a);
  h->prekeys = 0;
  TA_CHECK_CUDA(h, cudaGetLastError());
  return TA_OK;
}
