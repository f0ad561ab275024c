// ta_load_window kernels: validity (start-time filtering separates windows,
// Sec. 5.2), discovery and dense ranking of the (pid, domain, stream) triples
// that name a lane, and the 64-bit sort key together with the digit histograms
// of every radix pass.
//   k_discover      one pass over the 40-byte records: defect counters, the triple and
//                   communicator sets, value ranges, and one 64-bit word per record
//                   (dropped flag | triple slot | ts_start - t0);
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

// One CTA: sorts the discovered triples, ranks them and the pids they contain.
__global__ void __launch_bounds__(1024) k_rank_triples(TripleTable *tt, int32_t *status) {
  extern __shared__ u64 buf[];  // TA_TRIPLE_SLOTS
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
__global__ void __launch_bounds__(1024) k_rank_comms(CommTable *cm, int32_t *status) {
  __shared__ u64 buf[TA_COMM_SLOTS];
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
  if (h->n > 0) {
    k_discover<<<TA_N grid_for(h->n, 256, 8), 256, 0, h->stream>>>(
        h->events, h->n, h->d_off, h->d_t0, h->d_t1, h->W, h->d_triples, h->d_comms, h->d_load_sum,
        h->d_misc, h->d_status, h->d_keys);
    h->prekeys = 1;
  }
  k_rank_comms<<<TA_N 1, 1024, 0, h->stream>>>(h->d_comms, h->d_status);
  TA_CHECK_CUDA(h, cudaFuncSetAttribute(k_rank_triples, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        TA_TRIPLE_SLOTS * (int)sizeof(u64)));
  k_rank_triples<<<TA_N 1, 1024, TA_TRIPLE_SLOTS * sizeof(u64), h->stream>>>(h->d_triples, h->d_status);
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
