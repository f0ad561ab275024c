// CPU oracle of the trace-window analyzer.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded C++17 restatement of what the analyzer's
// seven steps compute, written from the paper's statement of the problem
// (Sec. 5.2 record model; Sec. 6.1 operator executions and T_op; Sec. 9.1
// thread id + call intervals, idle intervals from device activity; Sec. 9.2
// ranks meeting in collectives) and, where the paper is silent, from the
// readings stated beside each function.  Every step has an exact definition,
// so each function is that definition written out with std::stable_sort,
// std::unordered_map and std::map; there is no blocking, fusion or reordering.
//
// It shares no code with the CUDA library, is imported only by tests/, by the
// smoke check and by the benchmark's CPU-baseline leg, and must never sit on
// the product path.
//
// Pins (tests/test_oracle_*.py): hand-worked windows under tests/golden/,
// O(n^2) / bitmap brute force written independently in Python, telescoping
// invariants (busy + idle == window length), and the generator's ground truth.
// Every function below has at least one such pin; none is "parity unpinned".
//
// Build: g++ -O2 -std=c++17 -shared -fPIC ta_oracle.cpp -o libta_oracle.so
#include <algorithm>
#include <climits>
#include <cstdint>
#include <cstring>
#include <map>
#include <string>
#include <tuple>
#include <unordered_map>
#include <vector>

namespace {

struct Event {
  int64_t ts_start, ts_end, corr_id;
  int32_t pid, name_id, seq;
  int16_t stream, kind;
};
static_assert(sizeof(Event) == 40, "record must be 40 bytes");

enum { OP = 0, API = 1, LAUNCH = 2, KERNEL = 3, MEMCPY = 4, COLL = 5 };
constexpr int NBINS = 40;
constexpr int MAX_DEPTH = 8;

struct LoadSummary { int64_t n_events, n_valid, n_bad_kind, n_bad_interval, n_out_of_window; };
struct JoinSummary {
  int64_t n_probe, n_matched, n_unmatched, n_launch, n_dup_launch, n_orphan_launch;
  int64_t sum_latency, min_latency, max_latency, sum_queue, max_queue;
};
struct AttrSummary { int64_t n_attributed, n_no_launch, n_no_op; int32_t max_depth, bad_nesting; };
struct LaneGaps { int64_t busy, idle, n_events, n_gaps, max_gap, first_start, last_end; };
struct LongGap { int32_t lane, next_event; int64_t gap_start, gap_len; };
struct CommSize { int64_t comm_id; int32_t n_ranks, reserved; };

// floor(log2 v) clamped to the last bin; values <= 1 land in bin 0.
int log2_bin(int64_t v) {
  if (v <= 1) return 0;
  int b = 0;
  while (b < NBINS - 1 && (v >> (b + 1)) != 0) b++;
  return b;
}

struct Oracle {
  // inputs
  std::vector<Event> in;
  std::vector<int64_t> win_off, t0, t1;
  int32_t W = 0;
  int64_t n = 0;

  // load
  std::vector<int32_t> win_of;      // per input record
  std::vector<uint8_t> dropped;     // per input record
  std::vector<LoadSummary> load_sum;

  // sort
  int64_t n_valid = 0;
  std::vector<int32_t> perm;
  std::vector<int64_t> ts_start, ts_end, corr_id;
  std::vector<int32_t> pid, name_id, seq;
  std::vector<int16_t> stream, kind;
  std::vector<int32_t> win_sorted;  // window of each sorted position
  std::vector<int32_t> lane_window, lane_pid, lane_off;
  std::vector<int16_t> lane_stream, lane_domain;

  // join
  std::vector<int32_t> launch_of, kernels_of_launch;
  std::vector<int64_t> launch_latency, queue_delay;
  std::vector<JoinSummary> join_sum;

  // attribution
  std::vector<int32_t> parent, op_of, op_n_kernels;
  std::vector<uint8_t> depth;
  std::vector<int64_t> op_first_start, op_last_end, op_kernel_ns;
  std::vector<AttrSummary> attr_sum;

  // gaps
  std::vector<int64_t> gap_before;
  std::vector<LaneGaps> lane_gaps;
  std::vector<uint32_t> lane_hist, win_hist;
  std::vector<LongGap> long_gaps;

  // aggregates (last call)
  std::vector<int32_t> g_window, g_pid, g_name;
  std::vector<int64_t> g_count, g_sum, g_min, g_max;
  std::vector<uint32_t> g_hist;

  // collectives
  std::vector<int32_t> c_window, c_seq, c_n_members, c_straggler_pid, c_flags;
  std::vector<int64_t> c_comm, c_min_start, c_max_start, c_skew, c_max_end;
  std::vector<int64_t> wait_ns;
  std::vector<int32_t> r_window, r_pid;
  std::vector<int64_t> r_n_coll, r_sum_wait, r_max_wait, r_n_straggler;

  // inclusive roll-up and graph replays
  std::vector<int32_t> incl_n_kernels;
  std::vector<int64_t> incl_first_start, incl_last_end, incl_kernel_ns;
  std::vector<int64_t> replay_first_start, replay_last_end, replay_kernel_ns;
  std::vector<int64_t> roll_sum;  // [window][3]: graph launches, their kernels, most kernels of one launch

  // gap blame
  std::vector<int32_t> b_class, b_launch;      // per long gap
  std::vector<int64_t> b_win_count, b_win_ns;  // [window][class]
  std::vector<int64_t> op_gap_ns;              // per sorted position

  // device-level coverage
  std::vector<int32_t> d_window, d_pid;
  std::vector<int64_t> d_n_events, d_busy, d_idle, d_compute, d_comm, d_overlap, d_exposed;

  // critical path
  std::vector<uint8_t> on_path;                 // per sorted position
  std::vector<int32_t> cp_window, cp_pid, cp_sink, cp_n_nodes, cp_reason;
  std::vector<int64_t> cp_begin, cp_end, cp_ns;  // cp_ns: [row][8]
  std::vector<int64_t> cp_sum;                  // [window][10]: paths, nodes, the eight classes

  bool is_kept(int64_t p) const { return p < n_valid; }

  // ---- step 1: validity.  A record belongs to the window in which it starts
  // (Sec. 5.2).  Reading: the first failing rule counts; ts_end > t1 is legal.
  void load() {
    win_of.assign(n, 0);
    dropped.assign(n, 0);
    load_sum.assign(W, LoadSummary{0, 0, 0, 0, 0});
    for (int32_t w = 0; w < W; w++) {
      for (int64_t k = win_off[w]; k < win_off[w + 1]; k++) {
        const Event& e = in[k];
        win_of[k] = w;
        LoadSummary& s = load_sum[w];
        s.n_events++;
        if (e.kind < 0 || e.kind > 5) { dropped[k] = 1; s.n_bad_kind++; }
        else if (e.ts_end < e.ts_start) { dropped[k] = 1; s.n_bad_interval++; }
        else if (e.ts_start < t0[w] || e.ts_start >= t1[w]) { dropped[k] = 1; s.n_out_of_window++; }
        else s.n_valid++;
      }
    }
  }

  // ---- step 2: canonical order.  Device and stream identifiers locate device
  // work, thread identifiers locate calls (Sec. 5.2).  Reading: stable order by
  // (dropped, window, pid, domain, stream, ts_start asc, ts_end desc, input index).
  void sort() {
    perm.resize(n);
    for (int64_t i = 0; i < n; i++) perm[i] = (int32_t)i;
    auto domain = [&](const Event& e) { return e.kind >= 3 ? 1 : 0; };
    std::stable_sort(perm.begin(), perm.end(), [&](int32_t a, int32_t b) {
      const Event &x = in[a], &y = in[b];
      if (dropped[a] != dropped[b]) return dropped[a] < dropped[b];
      if (win_of[a] != win_of[b]) return win_of[a] < win_of[b];
      if (x.pid != y.pid) return x.pid < y.pid;
      int dx = domain(x), dy = domain(y);
      if (dx != dy) return dx < dy;
      if (x.stream != y.stream) return x.stream < y.stream;
      if (x.ts_start != y.ts_start) return x.ts_start < y.ts_start;
      if (x.ts_end != y.ts_end) return x.ts_end > y.ts_end;
      return false;
    });
    n_valid = 0;
    for (int64_t i = 0; i < n; i++) n_valid += dropped[i] ? 0 : 1;
    ts_start.resize(n); ts_end.resize(n); corr_id.resize(n);
    pid.resize(n); name_id.resize(n); seq.resize(n);
    stream.resize(n); kind.resize(n); win_sorted.resize(n);
    for (int64_t p = 0; p < n; p++) {
      const Event& e = in[perm[p]];
      ts_start[p] = e.ts_start; ts_end[p] = e.ts_end; corr_id[p] = e.corr_id;
      pid[p] = e.pid; name_id[p] = e.name_id; seq[p] = e.seq;
      stream[p] = e.stream; kind[p] = e.kind; win_sorted[p] = win_of[perm[p]];
    }
    lane_window.clear(); lane_pid.clear(); lane_stream.clear(); lane_domain.clear(); lane_off.clear();
    for (int64_t p = 0; p < n_valid; p++) {
      int16_t d = kind[p] >= 3 ? 1 : 0;
      bool head = p == 0 || win_sorted[p] != win_sorted[p - 1] || pid[p] != pid[p - 1] ||
                  d != (kind[p - 1] >= 3 ? 1 : 0) || stream[p] != stream[p - 1];
      if (head) {
        lane_window.push_back(win_sorted[p]); lane_pid.push_back(pid[p]);
        lane_stream.push_back(stream[p]); lane_domain.push_back(d);
        lane_off.push_back((int32_t)p);
      }
    }
    lane_off.push_back((int32_t)n_valid);
  }

  // ---- step 3: a device record and the host call that submitted it carry the same
  // correlation id (Sec. 5.2; Fig. "Key performance observations" (a)).  Readings: the key is
  // (window, pid, corr_id); the first LAUNCH in canonical order wins a key;
  // latency = kernel start - launch start; queue delay = the part of it after
  // the launch call returned; COLL records do not join.
  struct JKey {
    int32_t w, pid; int64_t corr;
    bool operator==(const JKey& o) const { return w == o.w && pid == o.pid && corr == o.corr; }
  };
  struct JHash {
    size_t operator()(const JKey& k) const {
      uint64_t h = (uint64_t)k.corr * 0x9E3779B97F4A7C15ull;
      h ^= ((uint64_t)(uint32_t)k.pid << 32 | (uint32_t)k.w) + 0x7F4A7C15u + (h << 6) + (h >> 2);
      return (size_t)h;
    }
  };
  void correlate() {
    launch_of.assign(n, -1); kernels_of_launch.assign(n, 0);
    launch_latency.assign(n, 0); queue_delay.assign(n, 0);
    join_sum.assign(W, JoinSummary{0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0});
    std::unordered_map<JKey, int32_t, JHash> first_launch;
    std::vector<uint8_t> is_dup(n, 0);
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != LAUNCH) continue;
      JoinSummary& s = join_sum[win_sorted[p]];
      s.n_launch++;
      JKey k{win_sorted[p], pid[p], corr_id[p]};
      auto it = first_launch.find(k);
      if (it == first_launch.end()) first_launch.emplace(k, (int32_t)p);
      else { is_dup[p] = 1; s.n_dup_launch++; }
    }
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != KERNEL && kind[p] != MEMCPY) continue;
      JoinSummary& s = join_sum[win_sorted[p]];
      s.n_probe++;
      auto it = first_launch.find(JKey{win_sorted[p], pid[p], corr_id[p]});
      if (it == first_launch.end()) { s.n_unmatched++; continue; }
      int32_t l = it->second;
      launch_of[p] = l;
      kernels_of_launch[l]++;
      int64_t lat = ts_start[p] - ts_start[l];
      int64_t q = ts_start[p] - ts_end[l];
      if (q < 0) q = 0;
      launch_latency[p] = lat; queue_delay[p] = q;
      if (s.n_matched == 0) { s.min_latency = lat; s.max_latency = lat; }
      else { s.min_latency = std::min(s.min_latency, lat); s.max_latency = std::max(s.max_latency, lat); }
      s.n_matched++;
      s.sum_latency += lat; s.sum_queue += q; s.max_queue = std::max(s.max_queue, q);
    }
    for (int64_t p = 0; p < n_valid; p++)
      if (kind[p] == LAUNCH && !is_dup[p] && kernels_of_launch[p] == 0)
        join_sum[win_sorted[p]].n_orphan_launch++;
  }

  // ---- step 4: a host record lies in the operator ranges of its own thread whose
  // intervals contain it (Sec. 9.1); T_op runs from the start of an operator's first
  // kernel to the end of its last (Sec. 6.1); a kernel may outlive the call (Sec.
  // 5.2) so containment is tested on the launch interval.  The definition is
  // evaluated against every earlier OP of the lane that has not ended before
  // the record starts (an OP that ended earlier can enclose nothing later).
  int attribute() {
    parent.assign(n, -1); depth.assign(n, 0); op_of.assign(n, -1);
    op_n_kernels.assign(n, 0);
    op_first_start.assign(n, 0); op_last_end.assign(n, 0); op_kernel_ns.assign(n, 0);
    attr_sum.assign(W, AttrSummary{0, 0, 0, 0, 0});
    bool any_bad = false, any_deep = false;
    const int64_t L = (int64_t)lane_window.size();
    for (int64_t l = 0; l < L; l++) {
      if (lane_domain[l] != 0) continue;
      AttrSummary& s = attr_sum[lane_window[l]];
      std::vector<int32_t> open;  // earlier OPs with ts_end >= current ts_start
      for (int32_t i = lane_off[l]; i < lane_off[l + 1]; i++) {
        std::vector<int32_t> keep;
        for (int32_t j : open)
          if (ts_end[j] >= ts_start[i]) keep.push_back(j);
        open.swap(keep);
        int32_t best = -1;
        int d = 0;
        for (int32_t j : open) {
          // j precedes i in canonical order, so ts_start[j] <= ts_start[i] and the
          // identical-interval rule is satisfied
          if (ts_end[i] <= ts_end[j]) {
            d++;
            if (best < 0 || ts_start[j] > ts_start[best] ||
                (ts_start[j] == ts_start[best] &&
                 (ts_end[j] < ts_end[best] || (ts_end[j] == ts_end[best] && j > best))))
              best = j;
          } else if (ts_start[j] < ts_start[i] && ts_start[i] < ts_end[j]) {
            s.bad_nesting = 1; any_bad = true;  // ts_end[j] < ts_end[i]: partial overlap
          }
        }
        parent[i] = best;
        // depth = level in the forest that `parent` defines (the parent precedes the child
        // in canonical order, so its depth is known); saturates at 255 (uint8).  It equals
        // the encloser count d except for a zero-length record that sits exactly on the end
        // of an earlier sibling range: closed intervals put such a record inside both.
        (void)d;
        int lvl = best < 0 ? 0 : std::min(255, (int)depth[best] + 1);
        depth[i] = (uint8_t)lvl;
        if (lvl > s.max_depth) s.max_depth = lvl;
        if (lvl > MAX_DEPTH) any_deep = true;
        if (kind[i] == OP) open.push_back(i);
      }
    }
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != KERNEL && kind[p] != MEMCPY) continue;
      AttrSummary& s = attr_sum[win_sorted[p]];
      int32_t l = launch_of[p];
      if (l < 0) { s.n_no_launch++; continue; }
      int32_t r = parent[l];
      if (r < 0) { s.n_no_op++; continue; }
      op_of[p] = r;
      s.n_attributed++;
      if (op_n_kernels[r] == 0) { op_first_start[r] = ts_start[p]; op_last_end[r] = ts_end[p]; }
      else {
        op_first_start[r] = std::min(op_first_start[r], ts_start[p]);
        op_last_end[r] = std::max(op_last_end[r], ts_end[p]);
      }
      op_n_kernels[r]++;
      op_kernel_ns[r] += ts_end[p] - ts_start[p];
    }
    if (any_bad) return 9;
    if (any_deep) return 8;
    return 0;
  }

  // ---- step 5: a stream is idle where none of its activity records covers (Sec. 9.1).
  // Readings: all three device kinds occupy the stream; ends are clipped to the
  // window; head and tail gaps are idle time and enter the histogram.
  void gaps(int64_t min_gap) {
    const int64_t L = (int64_t)lane_window.size();
    gap_before.assign(n, 0);
    lane_gaps.assign(L, LaneGaps{0, 0, 0, 0, 0, 0, 0});
    lane_hist.assign(L * NBINS, 0);
    win_hist.assign((int64_t)W * NBINS, 0);
    long_gaps.clear();
    for (int64_t l = 0; l < L; l++) {
      if (lane_domain[l] != 1) continue;
      const int32_t w = lane_window[l];
      const int64_t W0 = t0[w], W1 = t1[w];
      LaneGaps& g = lane_gaps[l];
      int64_t P = W0;
      auto note_gap = [&](int64_t len, int64_t start, int32_t next) {
        if (len <= 0) return;
        g.n_gaps++;
        g.max_gap = std::max(g.max_gap, len);
        int b = log2_bin(len);
        lane_hist[l * NBINS + b]++;
        win_hist[(int64_t)w * NBINS + b]++;
        if (len >= min_gap) long_gaps.push_back(LongGap{(int32_t)l, next, start, len});
      };
      g.first_start = ts_start[lane_off[l]];
      for (int32_t i = lane_off[l]; i < lane_off[l + 1]; i++) {
        int64_t ce = std::min(ts_end[i], W1);
        int64_t gap = std::max<int64_t>(0, ts_start[i] - P);
        int64_t busy = std::max<int64_t>(0, ce - std::max(ts_start[i], P));
        gap_before[i] = gap;
        g.idle += gap; g.busy += busy; g.n_events++;
        note_gap(gap, P, i);
        P = std::max(P, ce);
      }
      int64_t tail = W1 - P;
      g.idle += tail;
      note_gap(tail, P, -1);
      g.last_end = P;
    }
  }

  // ---- step 6: per-symbol counts and duration statistics (Sec. 8.1 compares
  // per-symbol call counts and kernel durations).
  int aggregate(uint32_t kind_mask, int value_sel) {
    if (value_sel < 0 || value_sel > 3) return 1;
    if ((value_sel == 1 || value_sel == 2) && kind_mask != (1u << OP)) return 1;
    struct Row { int64_t count, sum, mn, mx; uint32_t hist[NBINS]; };
    std::map<std::tuple<int32_t, int32_t, int32_t>, Row> rows;
    for (int64_t p = 0; p < n_valid; p++) {
      if (!((1u << kind[p]) & kind_mask)) continue;
      int64_t v;
      if (value_sel == 0) v = ts_end[p] - ts_start[p];
      else if (value_sel == 1) {
        if (op_n_kernels[p] <= 0) continue;
        v = op_last_end[p] - op_first_start[p];
      } else if (value_sel == 2) {  // idle time of the process's device streams that coincides with the operator
        if (op_gap_ns[p] <= 0) continue;
        v = op_gap_ns[p];
      } else {  // records a critical path passes through, by their own duration
        if (!on_path[p]) continue;
        v = ts_end[p] - ts_start[p];
      }
      auto key = std::make_tuple(win_sorted[p], pid[p], name_id[p]);
      auto it = rows.find(key);
      if (it == rows.end()) {
        Row r; r.count = 0; r.sum = 0; r.mn = v; r.mx = v; std::memset(r.hist, 0, sizeof(r.hist));
        it = rows.emplace(key, r).first;
      }
      Row& r = it->second;
      r.count++; r.sum += v; r.mn = std::min(r.mn, v); r.mx = std::max(r.mx, v);
      r.hist[log2_bin(v)]++;
    }
    g_window.clear(); g_pid.clear(); g_name.clear();
    g_count.clear(); g_sum.clear(); g_min.clear(); g_max.clear(); g_hist.clear();
    for (auto& kv : rows) {
      g_window.push_back(std::get<0>(kv.first)); g_pid.push_back(std::get<1>(kv.first));
      g_name.push_back(std::get<2>(kv.first));
      g_count.push_back(kv.second.count); g_sum.push_back(kv.second.sum);
      g_min.push_back(kv.second.mn); g_max.push_back(kv.second.mx);
      for (int b = 0; b < NBINS; b++) g_hist.push_back(kv.second.hist[b]);
    }
    return 0;
  }

  // ---- step 7: records of different processes that name the same collective are
  // linked; each rank waits for the last one to arrive (Sec. 6.1, Sec. 9.2).
  // Readings: arrival = the rank's ts_start; wait = time until the last arrival;
  // all pids share one clock; corr_id carries the communicator id.
  void collectives(const CommSize* sizes, int32_t n_comms) {
    std::map<int64_t, int32_t> expected;
    for (int32_t i = 0; i < n_comms; i++) expected[sizes[i].comm_id] = sizes[i].n_ranks;
    std::map<std::tuple<int32_t, int64_t, int32_t>, std::vector<int32_t>> groups;
    for (int64_t p = 0; p < n_valid; p++)
      if (kind[p] == COLL) groups[std::make_tuple(win_sorted[p], corr_id[p], seq[p])].push_back((int32_t)p);
    wait_ns.assign(n, 0);
    c_window.clear(); c_comm.clear(); c_seq.clear(); c_n_members.clear();
    c_min_start.clear(); c_max_start.clear(); c_skew.clear(); c_max_end.clear();
    c_straggler_pid.clear(); c_flags.clear();
    struct Rank { int64_t n_coll, sum_wait, max_wait, n_straggler; };
    std::map<std::pair<int32_t, int32_t>, Rank> ranks;
    for (auto& kv : groups) {
      const std::vector<int32_t>& m = kv.second;
      int64_t mn = ts_start[m[0]], mx = ts_start[m[0]], me = ts_end[m[0]];
      int32_t strag = pid[m[0]];
      for (int32_t p : m) {
        mn = std::min(mn, ts_start[p]); me = std::max(me, ts_end[p]);
        if (ts_start[p] > mx || (ts_start[p] == mx && pid[p] < strag)) { mx = ts_start[p]; strag = pid[p]; }
      }
      int32_t flags = 0;
      auto ex = expected.find(std::get<1>(kv.first));
      if (ex != expected.end()) { if ((int64_t)m.size() != ex->second) flags |= 1; }
      else if (m.size() < 2) flags |= 1;
      for (size_t a = 0; a < m.size(); a++)
        for (size_t b = a + 1; b < m.size(); b++)
          if (pid[m[a]] == pid[m[b]]) flags |= 2;
      for (int32_t p : m) {
        wait_ns[p] = mx - ts_start[p];
        Rank& r = ranks[std::make_pair(std::get<0>(kv.first), pid[p])];  // row exists for every rank seen
        if (flags == 0) {
          r.n_coll++; r.sum_wait += wait_ns[p]; r.max_wait = std::max(r.max_wait, wait_ns[p]);
        }
      }
      if (flags == 0) ranks[std::make_pair(std::get<0>(kv.first), strag)].n_straggler++;
      c_window.push_back(std::get<0>(kv.first)); c_comm.push_back(std::get<1>(kv.first));
      c_seq.push_back(std::get<2>(kv.first)); c_n_members.push_back((int32_t)m.size());
      c_min_start.push_back(mn); c_max_start.push_back(mx); c_skew.push_back(mx - mn);
      c_max_end.push_back(me); c_straggler_pid.push_back(strag); c_flags.push_back(flags);
    }
    r_window.clear(); r_pid.clear(); r_n_coll.clear(); r_sum_wait.clear(); r_max_wait.clear();
    r_n_straggler.clear();
    for (auto& kv : ranks) {
      r_window.push_back(kv.first.first); r_pid.push_back(kv.first.second);
      r_n_coll.push_back(kv.second.n_coll); r_sum_wait.push_back(kv.second.sum_wait);
      r_max_wait.push_back(kv.second.max_wait); r_n_straggler.push_back(kv.second.n_straggler);
    }
  }

  // ---- inclusive operator figures and graph replays (needs attribute() without error).
  // An invocation's kernel composition comes from the call-to-kernel links, and T_op spans the
  // first kernel start to the last completion (Sec. 6.1, "Operator execution and efficiency").
  // Readings: the inclusive figures of an OP are those of the OP itself plus those of every OP
  // below it in the parent forest (count and nanoseconds add; first start is the minimum and
  // last end the maximum over the OPs that own kernels; all zero when the subtree owns none).
  // Under CUDA Graph replay no operator call is recorded; the launch they share tells the
  // kernels of one replay apart (Sec. 6.1):
  // a LAUNCH that owns two or more device records is one replay, spanning the first start to
  // the last end of those records, with the sum of their durations; all zero for other launches.
  void rollup() {
    incl_n_kernels.assign(n, 0); incl_kernel_ns.assign(n, 0);
    incl_first_start.assign(n, 0); incl_last_end.assign(n, 0);
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != OP || op_n_kernels[p] <= 0) continue;
      incl_n_kernels[p] = op_n_kernels[p]; incl_kernel_ns[p] = op_kernel_ns[p];
      incl_first_start[p] = op_first_start[p]; incl_last_end[p] = op_last_end[p];
    }
    // a child always follows its parent in canonical order: going backwards, every OP is
    // complete before it is added to its parent
    for (int64_t p = n_valid - 1; p >= 0; p--) {
      if (kind[p] != OP || incl_n_kernels[p] <= 0 || parent[p] < 0) continue;
      const int32_t q = parent[p];
      if (incl_n_kernels[q] == 0) { incl_first_start[q] = incl_first_start[p]; incl_last_end[q] = incl_last_end[p]; }
      else {
        incl_first_start[q] = std::min(incl_first_start[q], incl_first_start[p]);
        incl_last_end[q] = std::max(incl_last_end[q], incl_last_end[p]);
      }
      incl_n_kernels[q] += incl_n_kernels[p]; incl_kernel_ns[q] += incl_kernel_ns[p];
    }
    replay_first_start.assign(n, 0); replay_last_end.assign(n, 0); replay_kernel_ns.assign(n, 0);
    roll_sum.assign((size_t)W * 3, 0);
    std::vector<uint8_t> seen(n, 0);
    for (int64_t p = 0; p < n_valid; p++) {
      const int32_t l = (kind[p] == KERNEL || kind[p] == MEMCPY) ? launch_of[p] : -1;
      if (l < 0 || kernels_of_launch[l] < 2) continue;
      if (!seen[l]) { seen[l] = 1; replay_first_start[l] = ts_start[p]; replay_last_end[l] = ts_end[p]; }
      else {
        replay_first_start[l] = std::min(replay_first_start[l], ts_start[p]);
        replay_last_end[l] = std::max(replay_last_end[l], ts_end[p]);
      }
      replay_kernel_ns[l] += ts_end[p] - ts_start[p];
    }
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != LAUNCH || kernels_of_launch[p] < 2) continue;
      int64_t* r = &roll_sum[(size_t)win_sorted[p] * 3];
      r[0]++; r[1] += kernels_of_launch[p]; r[2] = std::max<int64_t>(r[2], kernels_of_launch[p]);
    }
  }

  // ---- operator efficiency (needs attribute() == 0).  An invocation's theoretical operation
  // count and logical data volume, normalised by T_op and the device peaks, give model FLOPs
  // utilisation and model bandwidth utilisation; speed-of-light attainment is the larger of
  // the two (Sec. 6.1, "Operator execution and efficiency").  The counts come from outside
  // the trace (shapes, data types, sharding): one pair of doubles per INPUT record, read for
  // OP records only; a negative or NaN count means "not known".  Missing composition or
  // inputs leave the measurement unresolved:
  //   state 0  not a kept OP record            state 2  no kernels, or T_op == 0
  //   state 1  resolved                        state 3  kernels, but a count is missing
  //   MFU = flops / (T_op * 1e-9 s * peak_flops),  MBU = bytes / (T_op * 1e-9 s * peak_bw),
  //   SOL_op = max(MFU, MBU); all three 0 unless resolved.
  // Per window: the three state counts, the sums of flops, bytes and T_op over resolved
  // invocations, and the largest SOL_op.  The only floating-point step of the analyzer.
  struct SolSummary { int64_t n_resolved, n_no_kernels, n_no_counts, sum_top_ns; double sum_flops, sum_bytes, max_sol; };
  std::vector<double> sol_mfu, sol_mbu, sol_op;
  std::vector<uint8_t> sol_state;
  std::vector<SolSummary> sol_sum;
  void sol(const double* flops, const double* bytes, double peak_flops, double peak_bw) {
    sol_mfu.assign(n, 0.0); sol_mbu.assign(n, 0.0); sol_op.assign(n, 0.0);
    sol_state.assign(n, 0);
    sol_sum.assign(W, SolSummary{0, 0, 0, 0, 0.0, 0.0, 0.0});
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != OP) continue;
      SolSummary& s = sol_sum[win_sorted[p]];
      const int64_t top = op_last_end[p] - op_first_start[p];
      if (op_n_kernels[p] <= 0 || top <= 0) { sol_state[p] = 2; s.n_no_kernels++; continue; }
      const double f = flops[perm[p]], b = bytes[perm[p]];
      if (!(f >= 0.0) || !(b >= 0.0)) { sol_state[p] = 3; s.n_no_counts++; continue; }
      const double seconds = (double)top * 1e-9;
      sol_mfu[p] = f / (seconds * peak_flops);
      sol_mbu[p] = b / (seconds * peak_bw);
      sol_op[p] = std::max(sol_mfu[p], sol_mbu[p]);
      sol_state[p] = 1;
      s.n_resolved++; s.sum_top_ns += top; s.sum_flops += f; s.sum_bytes += b;
      s.max_sol = std::max(s.max_sol, sol_op[p]);
    }
  }

  // ---- gap blame (needs correlate() and gaps()).  A gap counts against the host when the
  // work that ended it was submitted only after the stream had gone idle (the late-dispatch
  // test of Sec. 6.2, engine patterns; "submission gaps", Sec. 8.2), and idle time is charged
  // to the host calls that were running meanwhile (Sec. 9.1: one waiting call overlaps 13.8 s of
  // GPU idle).  Readings, per long gap of the list gaps() made:
  //   class 3 TAIL        the gap runs to the end of the window (no next record);
  //   class 0 NO_LAUNCH   the next record has no launch (a COLL record, or launch_of = -1);
  //   class 1 SUBMISSION  its launch started at or after the gap began (the stream was already
  //                       idle when the host submitted the work);
  //   class 2 QUEUED      its launch started before the gap began (submitted in time, started late).
  // And per OP record: op_gap_ns = sum over the long gaps of ALL device streams of the OP's
  // (window, process) of the length of [gap_start, gap_start + gap_len) n [ts_start, ts_end).
  void blame() {
    const size_t G = long_gaps.size();
    b_class.assign(G, 0); b_launch.assign(G, -1);
    b_win_count.assign((size_t)W * 4, 0); b_win_ns.assign((size_t)W * 4, 0);
    for (size_t k = 0; k < G; k++) {
      const LongGap& g = long_gaps[k];
      int cls;
      if (g.next_event < 0) cls = 3;
      else {
        const int32_t l = launch_of[g.next_event];
        b_launch[k] = l;
        if (l < 0) cls = 0;
        else cls = ts_start[l] >= g.gap_start ? 1 : 2;
      }
      b_class[k] = cls;
      const int32_t w = lane_window[g.lane];
      b_win_count[(size_t)w * 4 + cls]++;
      b_win_ns[(size_t)w * 4 + cls] += g.gap_len;
    }
    // the long gaps of each (window, process), all device streams together
    std::map<std::pair<int32_t, int32_t>, std::vector<std::pair<int64_t, int64_t>>> idle;
    for (const LongGap& g : long_gaps)
      idle[std::make_pair(lane_window[g.lane], lane_pid[g.lane])].push_back(
          std::make_pair(g.gap_start, g.gap_start + g.gap_len));
    op_gap_ns.assign(n, 0);
    for (int64_t p = 0; p < n_valid; p++) {
      if (kind[p] != OP) continue;
      auto it = idle.find(std::make_pair(win_sorted[p], pid[p]));
      if (it == idle.end()) continue;
      int64_t sum = 0;
      for (const auto& iv : it->second) {
        const int64_t lo = std::max(iv.first, ts_start[p]), hi = std::min(iv.second, ts_end[p]);
        if (hi > lo) sum += hi - lo;
      }
      op_gap_ns[p] = sum;
    }
  }

  // ---- critical path (needs correlate()).  Three kinds of dependency are followed (a kernel on
  // its launch, a record on its predecessor in stream or thread, a waiting call on the device
  // record that released it); a delay that none of them explains is reported as unresolved
  // (Sec. 6.1, "Execution progress and state"; Fig. "Critical path":
  // host work, the API call that submits kernel k1, k1, the end of the host's wait, host work
  // again - kernel k2 of another stream and the wait itself are off the path).
  // Readings.  One path per (window, process).  Nodes are the valid API and LAUNCH records
  // (host) and the KERNEL, MEMCPY and COLL records (device); OP records are context.  A node
  // has a START point (ts_start) and an END point (ts_end).  The walk starts at the END of the
  // sink - the node with the greatest ts_end, the highest canonical position among equals -
  // and always steps back to the dependency that was released last:
  //   END(v), v an API record that waited: to END(d), where d is the device record of the
  //     process with the greatest ts_end < ts_end(v) (highest position among equals) and
  //     v waited iff ts_end(d) >= ts_start(v)                        [synchronisation edge]
  //   END(v) otherwise: to START(v)                                  [v ran]
  //   START(k), k a device record: stream order offers END(q), q the record just before k
  //     in its lane, if ts_end(q) <= ts_start(k); submission offers START(l), l = launch_of[k],
  //     if l >= 0 and ts_start(l) <= ts_start(k).  With both on offer stream order binds iff
  //     ts_end(q) > ts_start(l) (the comparison of the gap blame); with neither the path
  //     ends here, unresolved (reason 1).
  //   START(h), h a host node: to the node u just before h in its lane (program order) -
  //     END(u) if ts_end(u) <= ts_start(h), else START(u) (h ran inside u); without u the
  //     path ends at the start of the thread (reason 0).
  // Time never increases along the walk and strictly decreases on a synchronisation edge, and
  // every cycle would need one, so the walk ends.  The time between the path's begin and the
  // sink's end splits into eight classes that add up exactly:
  //   0 KERNEL, 1 MEMCPY, 2 COLL execution; 3 launch latency (submission edges); 4 delay on a
  //   stream-order edge (unresolved); 5 inside host API / LAUNCH calls; 6 host time between
  //   calls; 7 tail of a wait after the device finished (synchronisation edges).
  void critical_path() {
    on_path.assign(n, 0);
    cp_window.clear(); cp_pid.clear(); cp_sink.clear(); cp_n_nodes.clear(); cp_reason.clear();
    cp_begin.clear(); cp_end.clear(); cp_ns.clear();
    cp_sum.assign((size_t)W * 10, 0);
    const int n_lanes = (int)lane_window.size();
    std::vector<int32_t> lane_of(n, -1);
    for (int l = 0; l < n_lanes; l++)
      for (int64_t p = lane_off[l]; p < lane_off[l + 1]; p++) lane_of[p] = l;
    auto is_host_node = [&](int64_t p) { return kind[p] == API || kind[p] == LAUNCH; };
    auto is_node = [&](int64_t p) { return kind[p] != OP; };
    // nodes of each (window, process); device records by (ts_end, position)
    std::map<std::pair<int32_t, int32_t>, std::vector<int32_t>> nodes;
    std::map<std::pair<int32_t, int32_t>, std::vector<std::pair<int64_t, int32_t>>> dev_by_end;
    for (int64_t p = 0; p < n_valid; p++) {
      if (!is_node(p)) continue;
      const auto key = std::make_pair(win_sorted[p], pid[p]);
      nodes[key].push_back((int32_t)p);
      if (kind[p] >= KERNEL) dev_by_end[key].push_back(std::make_pair(ts_end[p], (int32_t)p));
    }
    for (auto& kv : dev_by_end) std::sort(kv.second.begin(), kv.second.end());
    for (auto& kv : nodes) {
      const auto& dv = dev_by_end[kv.first];
      int32_t sink = -1;
      for (int32_t p : kv.second)
        if (sink < 0 || ts_end[p] >= ts_end[sink]) sink = p;  // positions ascend: the last equal wins
      int64_t ns[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      int32_t n_nodes = 0, reason = 0;
      int64_t begin = 0;
      auto visit = [&](int32_t v) { if (!on_path[v]) { on_path[v] = 1; n_nodes++; } };
      int32_t v = sink;
      bool at_end = true;
      for (int64_t guard = 0; guard <= 2 * n_valid + 2; guard++) {
        visit(v);
        if (at_end) {
          if (kind[v] == API) {
            // the device record that finished last before the call returned
            auto it = std::lower_bound(dv.begin(), dv.end(), std::make_pair(ts_end[v], (int32_t)-1));
            if (it != dv.begin()) {
              const int32_t d = (it - 1)->second;
              if (ts_end[d] >= ts_start[v]) {
                ns[7] += ts_end[v] - ts_end[d];
                v = d;
                continue;  // at END(d)
              }
            }
          }
          ns[kind[v] >= KERNEL ? kind[v] - KERNEL : 5] += ts_end[v] - ts_start[v];
          at_end = false;
          continue;
        }
        if (kind[v] >= KERNEL) {
          const int32_t q = v > lane_off[lane_of[v]] ? v - 1 : -1;
          const bool q_ok = q >= 0 && ts_end[q] <= ts_start[v];
          const int32_t l = (kind[v] == KERNEL || kind[v] == MEMCPY) ? launch_of[v] : -1;
          const bool l_ok = l >= 0 && ts_start[l] <= ts_start[v];
          if (q_ok && (!l_ok || ts_end[q] > ts_start[l])) {
            ns[4] += ts_start[v] - ts_end[q];
            v = q; at_end = true;
          } else if (l_ok) {
            ns[3] += ts_start[v] - ts_start[l];
            v = l;  // at START(l)
          } else {
            begin = ts_start[v]; reason = 1;
            break;
          }
        } else {
          int32_t u = -1;
          for (int64_t p = (int64_t)v - 1; p >= lane_off[lane_of[v]]; p--)
            if (is_host_node(p)) { u = (int32_t)p; break; }
          if (u < 0) { begin = ts_start[v]; reason = 0; break; }
          if (ts_end[u] <= ts_start[v]) { ns[6] += ts_start[v] - ts_end[u]; v = u; at_end = true; }
          else { ns[5] += ts_start[v] - ts_start[u]; v = u; }
        }
      }
      cp_window.push_back(kv.first.first); cp_pid.push_back(kv.first.second);
      cp_sink.push_back(sink); cp_n_nodes.push_back(n_nodes); cp_reason.push_back(reason);
      cp_begin.push_back(begin); cp_end.push_back(ts_end[sink]);
      int64_t* ws = &cp_sum[(size_t)kv.first.first * 10];
      ws[0]++; ws[1] += n_nodes;
      for (int c = 0; c < 8; c++) { cp_ns.push_back(ns[c]); ws[2 + c] += ns[c]; }
    }
  }

  // ---- device-level coverage: how much communication time ran while kernels ran too and
  // how much was left uncovered, as measures of unions of intervals (Sec. 6.1, "Execution
  // progress and state"; Fig. "Overlap and exposed work": a compute lane, a communication / IO
  // lane, their overlap, the exposed remainder).  Readings: per (window, process), over all
  // device streams; compute = KERNEL records, communication / IO = MEMCPY and COLL records;
  // every interval is [ts_start, min(ts_end, t1)); busy = measure of the union of all of them,
  // compute / comm = measure of each class's union, overlap = measure of the intersection of
  // the two unions, exposed = comm - overlap, idle = window length - busy.
  // Written out as a sweep over interval boundaries with one open-interval counter per class.
  void device_overlap() {
    d_window.clear(); d_pid.clear(); d_n_events.clear(); d_busy.clear(); d_idle.clear();
    d_compute.clear(); d_comm.clear(); d_overlap.clear(); d_exposed.clear();
    std::map<std::pair<int32_t, int32_t>, std::vector<int32_t>> groups;
    for (int64_t p = 0; p < n_valid; p++)
      if (kind[p] >= KERNEL) groups[std::make_pair(win_sorted[p], pid[p])].push_back((int32_t)p);
    for (auto& kv : groups) {
      const int32_t w = kv.first.first;
      struct Edge { int64_t t; int cls; int delta; };
      std::vector<Edge> edges;
      for (int32_t p : kv.second) {
        const int64_t s = ts_start[p], e = std::min(ts_end[p], t1[w]);
        if (e <= s) continue;  // an empty interval covers nothing
        const int cls = kind[p] == KERNEL ? 0 : 1;
        edges.push_back(Edge{s, cls, +1});
        edges.push_back(Edge{e, cls, -1});
      }
      std::sort(edges.begin(), edges.end(), [](const Edge& a, const Edge& b) { return a.t < b.t; });
      int64_t open[2] = {0, 0}, busy = 0, comp = 0, comm = 0, both = 0;
      for (size_t i = 0; i < edges.size();) {
        size_t j = i;
        while (j < edges.size() && edges[j].t == edges[i].t) { open[edges[j].cls] += edges[j].delta; j++; }
        if (j < edges.size()) {
          const int64_t dt = edges[j].t - edges[i].t;
          if (open[0] > 0 || open[1] > 0) busy += dt;
          if (open[0] > 0) comp += dt;
          if (open[1] > 0) comm += dt;
          if (open[0] > 0 && open[1] > 0) both += dt;
        }
        i = j;
      }
      d_window.push_back(w); d_pid.push_back(kv.first.second);
      d_n_events.push_back((int64_t)kv.second.size());
      d_busy.push_back(busy); d_idle.push_back((t1[w] - t0[w]) - busy);
      d_compute.push_back(comp); d_comm.push_back(comm); d_overlap.push_back(both);
      d_exposed.push_back(comm - both);
    }
  }
};

template <class T>
int give(const std::vector<T>& v, const void** ptr, int64_t* count, int32_t* elem) {
  *ptr = v.data(); *count = (int64_t)v.size(); *elem = (int32_t)sizeof(T);
  return 0;
}

}  // namespace

extern "C" {

void* orc_create(const void* events, int64_t n, const int64_t* win_off, const int64_t* t0,
                 const int64_t* t1, int32_t W) {
  Oracle* o = new Oracle();
  o->n = n; o->W = W;
  o->in.assign((const Event*)events, (const Event*)events + n);
  o->win_off.assign(win_off, win_off + W + 1);
  o->t0.assign(t0, t0 + W);
  o->t1.assign(t1, t1 + W);
  return o;
}
void orc_destroy(void* h) { delete (Oracle*)h; }
void orc_load(void* h) { ((Oracle*)h)->load(); }
void orc_sort(void* h) { ((Oracle*)h)->sort(); }
void orc_correlate(void* h) { ((Oracle*)h)->correlate(); }
int32_t orc_attribute(void* h) { return ((Oracle*)h)->attribute(); }
void orc_gaps(void* h, int64_t min_gap) { ((Oracle*)h)->gaps(min_gap); }
int32_t orc_aggregate(void* h, uint32_t mask, int32_t sel) { return ((Oracle*)h)->aggregate(mask, sel); }
void orc_collectives(void* h, const void* sizes, int32_t n_comms) {
  ((Oracle*)h)->collectives((const CommSize*)sizes, n_comms);
}
void orc_device_overlap(void* h) { ((Oracle*)h)->device_overlap(); }
void orc_blame(void* h) { ((Oracle*)h)->blame(); }
void orc_rollup(void* h) { ((Oracle*)h)->rollup(); }
void orc_critical_path(void* h) { ((Oracle*)h)->critical_path(); }
void orc_sol(void* h, const double* flops, const double* bytes, double peak_flops, double peak_bw) {
  ((Oracle*)h)->sol(flops, bytes, peak_flops, peak_bw);
}
int64_t orc_n_valid(void* h) { return ((Oracle*)h)->n_valid; }

// Exposes a result array by name: pointer into the oracle's storage, element
// count and element size.  Returns 0, or -1 for an unknown name.
int32_t orc_get(void* h, const char* name, const void** ptr, int64_t* count, int32_t* elem) {
  Oracle* o = (Oracle*)h;
  std::string s(name);
#define G(field) if (s == #field) return give(o->field, ptr, count, elem);
  G(load_sum) G(dropped) G(win_of)
  G(perm) G(ts_start) G(ts_end) G(corr_id) G(pid) G(name_id) G(seq) G(stream) G(kind) G(win_sorted)
  G(lane_window) G(lane_pid) G(lane_stream) G(lane_domain) G(lane_off)
  G(launch_of) G(kernels_of_launch) G(launch_latency) G(queue_delay) G(join_sum)
  G(parent) G(depth) G(op_of) G(op_n_kernels) G(op_first_start) G(op_last_end) G(op_kernel_ns) G(attr_sum)
  G(gap_before) G(lane_gaps) G(lane_hist) G(win_hist) G(long_gaps)
  G(g_window) G(g_pid) G(g_name) G(g_count) G(g_sum) G(g_min) G(g_max) G(g_hist)
  G(c_window) G(c_comm) G(c_seq) G(c_n_members) G(c_min_start) G(c_max_start) G(c_skew) G(c_max_end)
  G(c_straggler_pid) G(c_flags) G(wait_ns)
  G(r_window) G(r_pid) G(r_n_coll) G(r_sum_wait) G(r_max_wait) G(r_n_straggler)
  G(incl_n_kernels) G(incl_first_start) G(incl_last_end) G(incl_kernel_ns)
  G(replay_first_start) G(replay_last_end) G(replay_kernel_ns) G(roll_sum)
  G(b_class) G(b_launch) G(b_win_count) G(b_win_ns) G(op_gap_ns)
  G(on_path) G(cp_window) G(cp_pid) G(cp_sink) G(cp_n_nodes) G(cp_reason) G(cp_begin) G(cp_end) G(cp_ns) G(cp_sum)
  G(sol_mfu) G(sol_mbu) G(sol_op) G(sol_state) G(sol_sum)
  G(d_window) G(d_pid) G(d_n_events) G(d_busy) G(d_idle) G(d_compute) G(d_comm) G(d_overlap) G(d_exposed)
#undef G
  return -1;
}

}  // extern "C"
