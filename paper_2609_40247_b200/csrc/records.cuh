// Device helpers for reading 40-byte trace records (layout of ta_event) and
// naming lanes.  Shared by the load, sort and gather kernels.
#pragma once
#include "ta_internal.cuh"

struct Rec {
  i64 ts_start, ts_end, corr;
  int32_t pid, name, seq;
  int16_t stream, kind;
};

// A record is five aligned 8-byte words.
__device__ __forceinline__ Rec load_rec(const ta_event *ev, int64_t i) {
  const i64 *p = reinterpret_cast<const i64 *>(ev) + i * 5;
  Rec r;
  r.ts_start = __ldg(p);
  r.ts_end = __ldg(p + 1);
  r.corr = __ldg(p + 2);
  u64 a = (u64)__ldg(p + 3), b = (u64)__ldg(p + 4);
  r.pid = (int32_t)(u32)a;
  r.name = (int32_t)(u32)(a >> 32);
  r.seq = (int32_t)(u32)b;
  r.stream = (int16_t)(uint16_t)(b >> 32);
  r.kind = (int16_t)(uint16_t)(b >> 48);
  return r;
}

// Order-preserving unsigned code of (pid, domain, stream): pid and stream are
// biased so that unsigned order equals signed order.
__device__ __forceinline__ u64 triple_code(int32_t pid, int16_t kind, int16_t stream) {
  u64 dom = kind >= 3 ? 1ull : 0ull;
  return ((u64)((u32)pid ^ 0x80000000u) << 17) | (dom << 16) | (u64)((uint16_t)stream ^ 0x8000u);
}
__device__ __forceinline__ int32_t code_pid(u64 c) { return (int32_t)((u32)(c >> 17) ^ 0x80000000u); }
__device__ __forceinline__ int16_t code_domain(u64 c) { return (int16_t)((c >> 16) & 1); }
__device__ __forceinline__ int16_t code_stream(u64 c) { return (int16_t)((uint16_t)(c & 0xFFFF) ^ 0x8000u); }

__device__ __forceinline__ int window_of(const int64_t *off, int W, int64_t i) {
  if (W == 1) return 0;
  int lo = 0, hi = W - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (off[mid] <= i) lo = mid;
    else hi = mid - 1;
  }
  return lo;
}

// Window of an input index for a thread whose indices only grow (grid-stride loops): one
// binary search, then a forward walk over the window offsets.
struct WindowWalker {
  const int64_t *off;
  int W, w;
  int64_t hi;  // off[w + 1]
  __device__ __forceinline__ WindowWalker(const int64_t *o, int nw) : off(o), W(nw), w(-1), hi(0) {}
  __device__ __forceinline__ int at(int64_t i) {
    if (w < 0) {
      w = window_of(off, W, i);
      hi = off[w + 1];
    }
    while (i >= hi) {  // also steps over empty windows
      w++;
      hi = off[w + 1];
    }
    return w;
  }
};

// 0 = kept, 1 bad kind, 2 bad interval, 3 start outside the window
__device__ __forceinline__ int defect_of(const Rec &r, i64 t0, i64 t1) {
  if (r.kind < 0 || r.kind > 5) return 1;
  if (r.ts_end < r.ts_start) return 2;
  if (r.ts_start < t0 || r.ts_start >= t1) return 3;
  return 0;
}
