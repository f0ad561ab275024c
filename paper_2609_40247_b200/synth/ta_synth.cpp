// Seeded synthetic profiling-window generator.
//
// Produces 40-byte trace records (layout of ta_event in include/ta.h) that
// stand in for the private production traces the paper analyses, plus a
// ground-truth sidecar that records what the simulation did.  This file holds
// no analysis arithmetic: it simulates host threads, in-order device streams
// and lock-step collectives, and writes down what happened.
//
// Shapes and magnitudes follow the paper's reported ranges: kernel durations
// from half a microsecond to several milliseconds (Sec. 8.1), tens to
// hundreds of inference steps per 30 s window (Sec. 5.3), ranks that meet in
// collectives, where the other ranks wait for the last one to arrive (Sec. 9.2).
//
// Build: g++ -O2 -std=c++17 -shared -fPIC ta_synth.cpp -o libta_synth.so
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

struct Event {
  int64_t ts_start, ts_end, corr_id;
  int32_t pid, name_id, seq;
  int16_t stream, kind;
};
static_assert(sizeof(Event) == 40, "record must be 40 bytes");

enum { K_OP = 0, K_API = 1, K_LAUNCH = 2, K_KERNEL = 3, K_MEMCPY = 4, K_COLL = 5 };

struct Rng {
  uint64_t s;
  explicit Rng(uint64_t seed) : s(seed) {}
  uint64_t next() {
    uint64_t z = (s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  }
  double uniform() { return ((next() >> 11) + 0.5) * (1.0 / 9007199254740992.0); }
  double normal() {
    double u1 = uniform(), u2 = uniform();
    return std::sqrt(-2.0 * std::log(u1)) * std::cos(6.283185307179586 * u2);
  }
  double expo(double mean) { return -mean * std::log(uniform()); }
  int64_t lognormal_ns(double median, double sigma, int64_t lo) {
    double v = median * std::exp(sigma * normal());
    int64_t r = (int64_t)std::llround(v);
    return r < lo ? lo : r;
  }
  uint64_t below(uint64_t n) { return next() % n; }
};

}  // namespace

extern "C" {

// Plain-data configuration; mirrored field by field in synth/__init__.py.
struct tasynth_config {
  int32_t mode;        // 0 = random operator tree per step, 1 = layered lock-step ranks
  int32_t n_pid;
  int32_t n_threads;   // host threads per pid (mode 1 uses thread 0 only)
  int32_t n_streams;   // device streams per pid
  int32_t pid_base;    // pids are pid_base .. pid_base + n_pid - 1
  int32_t n_steps;     // steps per host thread
  // mode 0
  int32_t ops_per_step, launches_per_step, max_depth;
  // mode 1
  int32_t layers_per_step, ops_per_layer, kernels_per_layer, colls_per_layer;
  int32_t sync_api;    // 1 = emit an API record that waits for the streams at step end
  int32_t n_names;
  int32_t name_mode;   // 0 uniform, 1 Zipf(zipf_s), 2 pattern by (layer mod 21, slot)
  int32_t shuffle_mode;  // 0 = 4096-record buffers in shuffled order, 1 = full shuffle, 2 = generation order
  int32_t comm_offset;   // collective communicator ids are 0x5EED0000 + comm_offset + stream
  uint64_t seed;
  int64_t span_ns;     // window length; 0 = generated extent rounded up to a whole second
  double zipf_s;
  double k_med1_ns, k_sigma1, k_frac2, k_med2_ns, k_sigma2;  // kernel duration mixture
  double launch_delay_mean_ns;                               // launch start -> kernel ready
  double coll_skew_sigma_ns;
  double stall_prob, stall_min_ns, stall_max_ns;
  double memcpy_frac;
  double delete_launch_frac;
  double tie_prob;
  double step_gap_mean_ns;
};

// Upper bound on the number of records one call of tasynth_generate emits.
int64_t tasynth_max_events(const tasynth_config* c) {
  int64_t per_step;
  if (c->mode == 0)
    per_step = (int64_t)c->ops_per_step + 2ll * c->launches_per_step + (c->sync_api ? 1 : 0);
  else
    per_step = 1 + (c->sync_api ? 1 : 0) +
               (int64_t)c->layers_per_step *
                   (c->ops_per_layer + 2ll * c->kernels_per_layer + c->colls_per_layer);
  int64_t threads = (c->mode == 0) ? c->n_threads : 1;
  return per_step * c->n_steps * c->n_pid * threads;
}

// Generates one window starting at t0.
//   out        records (capacity cap >= tasynth_max_events)
//   truth_link per record, index (within this call's output) of: the innermost
//              open OP when a host record was emitted; the LAUNCH of a
//              KERNEL/MEMCPY (-1 when that LAUNCH record was deleted); -1 otherwise
//   truth_val  per record: device records: idle time on the stream right before
//              the record (start - max(previous end on that stream, t0));
//              host records: number of OPs open when it was emitted
//   truth_wait per record: COLL: latest arrival in its collective - own arrival; else 0
//   n_out, t1_out, n_deleted_out: record count, window end, deleted LAUNCH count
// Returns 0, or 1 if cap is too small, 2 if a fixed span was exceeded, 3 bad config.
int32_t tasynth_generate(const tasynth_config* c, int64_t t0, void* out_v, int64_t cap,
                         int32_t* truth_link, int64_t* truth_val, int64_t* truth_wait,
                         int64_t* n_out, int64_t* t1_out, int64_t* n_deleted_out) {
  if (!c || c->n_pid < 1 || c->n_streams < 1 || c->n_threads < 1 || c->n_names < 1) return 3;
  if (c->mode == 0 && (c->ops_per_step < 1 || c->max_depth < 1)) return 3;
  if (c->mode == 1 && (c->ops_per_layer < 1 || c->layers_per_step < 1 ||
                       c->kernels_per_layer < std::max(1, c->ops_per_layer - 1) ||
                       c->colls_per_layer > c->kernels_per_layer))
    return 3;
  Event* out = (Event*)out_v;
  Rng rng(c->seed * 0x2545F4914F6CDD1Dull + 0x1234567ull);

  const int P = c->n_pid, S = c->n_streams;
  const int T = (c->mode == 0) ? c->n_threads : 1;

  // Zipf table
  std::vector<double> zcdf;
  if (c->name_mode == 1) {
    zcdf.resize(c->n_names);
    double acc = 0;
    for (int i = 0; i < c->n_names; i++) {
      acc += 1.0 / std::pow((double)(i + 1), c->zipf_s);
      zcdf[i] = acc;
    }
    for (auto& v : zcdf) v /= acc;
  }
  auto draw_name = [&](int layer, int slot) -> int32_t {
    if (c->name_mode == 1) {
      double u = rng.uniform();
      int idx = (int)(std::lower_bound(zcdf.begin(), zcdf.end(), u) - zcdf.begin());
      return idx >= c->n_names ? c->n_names - 1 : idx;
    }
    if (c->name_mode == 2) return (int32_t)(((layer % 21) * 12 + slot) % c->n_names);
    return (int32_t)rng.below((uint64_t)c->n_names);
  };

  // generation-order storage
  std::vector<Event> ev;
  std::vector<int32_t> link;
  std::vector<int64_t> val, wait;
  int64_t est = tasynth_max_events(c);
  ev.reserve(est); link.reserve(est); val.reserve(est); wait.reserve(est);
  std::vector<int8_t> cls;  // shuffle class: 0 OP, 1 API/LAUNCH, 2 device
  cls.reserve(est);

  struct Thread {
    int64_t h;                    // host clock
    std::vector<int32_t> stack;   // generation indices of open OPs
  };
  std::vector<Thread> th(P * T);
  std::vector<int64_t> f(P * S, t0);  // stream free time
  std::vector<int64_t> corr(P, 0);
  std::vector<int32_t> comm_seq(S, 0);
  int64_t n_deleted = 0;
  for (auto& t : th) t.h = t0 + 1000 + (int64_t)rng.expo(2000.0);

  auto emit = [&](const Event& e, int32_t l, int64_t v, int64_t w, int8_t k) -> int32_t {
    ev.push_back(e); link.push_back(l); val.push_back(v); wait.push_back(w); cls.push_back(k);
    return (int32_t)ev.size() - 1;
  };
  auto step_small = [&](double mean) -> int64_t {
    if (rng.uniform() < c->tie_prob) return 0;
    return 1 + (int64_t)rng.expo(mean);
  };
  auto kernel_dur = [&]() -> int64_t {
    if (c->k_frac2 > 0 && rng.uniform() < c->k_frac2)
      return rng.lognormal_ns(c->k_med2_ns, c->k_sigma2, 500);
    return rng.lognormal_ns(c->k_med1_ns, c->k_sigma1, 500);
  };
  auto open_op = [&](int p, int t, int32_t name) {
    Thread& x = th[p * T + t];
    Event e{};
    e.ts_start = x.h; e.ts_end = x.h; e.pid = c->pid_base + p; e.name_id = name;
    e.stream = (int16_t)t; e.kind = K_OP;
    int32_t par = x.stack.empty() ? -1 : x.stack.back();
    int32_t gi = emit(e, par, (int64_t)x.stack.size(), 0, 0);
    x.stack.push_back(gi);
    x.h += step_small(300.0);
  };
  auto close_op = [&](int p, int t) {
    Thread& x = th[p * T + t];
    int64_t d = step_small(300.0);
    x.h += d < 1 ? 1 : d;  // ends strictly increase while the stack unwinds
    ev[x.stack.back()].ts_end = x.h;
    x.stack.pop_back();
    x.h += step_small(300.0);
  };
  auto launch = [&](int p, int t, int s, int32_t name) {
    Thread& x = th[p * T + t];
    if (c->stall_prob > 0 && rng.uniform() < c->stall_prob)
      x.h += (int64_t)(c->stall_min_ns + rng.uniform() * (c->stall_max_ns - c->stall_min_ns));
    bool is_copy = c->memcpy_frac > 0 && rng.uniform() < c->memcpy_frac;
    int64_t ldur = rng.lognormal_ns(4000.0, 0.5, 200);
    int64_t cid = ++corr[p];
    Event l{};
    l.ts_start = x.h; l.ts_end = x.h + ldur; l.corr_id = cid; l.pid = c->pid_base + p;
    l.name_id = name; l.stream = (int16_t)t; l.kind = K_LAUNCH;
    bool deleted = c->delete_launch_frac > 0 && rng.uniform() < c->delete_launch_frac;
    int32_t lgi = -1;
    if (!deleted) {
      int32_t par = x.stack.empty() ? -1 : x.stack.back();
      lgi = emit(l, par, (int64_t)x.stack.size(), 0, 1);
    } else {
      n_deleted++;
    }
    int64_t ready = l.ts_start + 1 + (int64_t)rng.expo(c->launch_delay_mean_ns);
    int64_t& fs = f[p * S + s];
    int64_t ks = std::max(ready, fs);
    int64_t kd = is_copy ? rng.lognormal_ns(50000.0, 1.0, 500) : kernel_dur();
    Event k{};
    k.ts_start = ks; k.ts_end = ks + kd; k.corr_id = cid; k.pid = c->pid_base + p;
    k.name_id = name; k.stream = (int16_t)s; k.kind = is_copy ? K_MEMCPY : K_KERNEL;
    emit(k, lgi, ks - std::max(fs, t0), 0, 2);
    fs = k.ts_end;
    x.h = l.ts_end + step_small(500.0);
  };
  auto sync_step = [&](int p, int t) {
    Thread& x = th[p * T + t];
    int64_t drain = x.h;
    for (int s = 0; s < S; s++)
      if (c->mode == 1 || s % T == t) drain = std::max(drain, f[p * S + s]);
    int64_t end = std::max(x.h + 500, drain + 1 + (int64_t)rng.expo(2000.0));
    if (c->sync_api) {
      Event a{};
      a.ts_start = x.h; a.ts_end = end; a.pid = c->pid_base + p;
      a.name_id = (int32_t)(c->n_names - 1); a.stream = (int16_t)t; a.kind = K_API;
      int32_t par = x.stack.empty() ? -1 : x.stack.back();
      emit(a, par, (int64_t)x.stack.size(), 0, 1);
    }
    x.h = end;
  };

  if (c->mode == 0) {
    // every (pid, thread) runs n_steps random operator trees; thread t owns streams s with s % T == t
    for (int step = 0; step < c->n_steps; step++) {
      for (int p = 0; p < P; p++)
        for (int t = 0; t < T; t++) {
          Thread& x = th[p * T + t];
          if (c->step_gap_mean_ns > 0) x.h += (int64_t)rng.expo(c->step_gap_mean_ns);
          int rem_ops = c->ops_per_step - 1, rem_l = c->launches_per_step;
          open_op(p, t, draw_name(step, 0));
          int own = 0;
          std::vector<int> owned;
          for (int s = 0; s < S; s++)
            if (s % T == t) owned.push_back(s);
          if (owned.empty()) owned.push_back(t % S);
          while (rem_ops + rem_l > 0) {
            double u = rng.uniform();
            int depth = (int)x.stack.size();
            if (depth > 1 && u < 0.25) { close_op(p, t); continue; }
            double po = (double)rem_ops / (double)(rem_ops + rem_l);
            if (rem_ops > 0 && rng.uniform() < po) {
              if (depth >= c->max_depth) { close_op(p, t); continue; }
              open_op(p, t, draw_name(step, rem_ops));
              rem_ops--;
            } else if (rem_l > 0) {
              launch(p, t, owned[own++ % owned.size()], draw_name(step, rem_l));
              rem_l--;
            }
          }
          while (x.stack.size() > 1) close_op(p, t);
          sync_step(p, t);
          close_op(p, t);
        }
    }
  } else {
    const int L = c->layers_per_step, OPL = c->ops_per_layer, KPL = c->kernels_per_layer,
              CPL = c->colls_per_layer;
    const int n_child = OPL - 1;
    std::vector<int64_t> arrive(P);
    for (int step = 0; step < c->n_steps; step++) {
      for (int p = 0; p < P; p++) {
        if (c->step_gap_mean_ns > 0) th[p * T].h += (int64_t)rng.expo(c->step_gap_mean_ns);
        open_op(p, 0, draw_name(step, 0));
      }
      for (int layer = 0; layer < L; layer++) {
        for (int p = 0; p < P; p++) open_op(p, 0, draw_name(layer, 1));
        int coll_done = 0;
        for (int k = 0; k < KPL; k++) {
          // child operator boundaries: child j covers kernels [j*KPL/n_child, (j+1)*KPL/n_child)
          for (int p = 0; p < P; p++) {
            if (n_child > 0) {
              for (int j = 0; j < n_child; j++)
                if (k == (int)((int64_t)j * KPL / n_child)) open_op(p, 0, draw_name(layer, 2 + j));
            }
            launch(p, 0, k % S, draw_name(layer, k));
            if (n_child > 0) {
              for (int j = 0; j < n_child; j++)
                if (k + 1 == (int)((int64_t)(j + 1) * KPL / n_child)) close_op(p, 0);
            }
          }
          // collectives are spread evenly after kernel slots
          while (coll_done < CPL && k + 1 == (int)((int64_t)(coll_done + 1) * KPL / CPL)) {
            int sc = coll_done % S;
            int64_t latest = INT64_MIN;
            for (int p = 0; p < P; p++) {
              int64_t ready = std::max(f[p * S + sc], th[p * T].h);
              arrive[p] = ready + (int64_t)std::fabs(rng.normal() * c->coll_skew_sigma_ns);
              latest = std::max(latest, arrive[p]);
            }
            int64_t end = latest + rng.lognormal_ns(12000.0, 0.3, 500);
            int32_t sq = comm_seq[sc]++;
            for (int p = 0; p < P; p++) {
              Event e{};
              e.ts_start = arrive[p]; e.ts_end = end; e.corr_id = 0x5EED0000ll + c->comm_offset + sc;
              e.pid = c->pid_base + p; e.name_id = draw_name(layer, 11); e.seq = sq;
              e.stream = (int16_t)sc; e.kind = K_COLL;
              int64_t& fs = f[p * S + sc];
              emit(e, -1, arrive[p] - std::max(fs, t0), latest - arrive[p], 2);
              fs = end;
            }
            coll_done++;
          }
        }
        for (int p = 0; p < P; p++) close_op(p, 0);
      }
      for (int p = 0; p < P; p++) {
        sync_step(p, 0);
        close_op(p, 0);
      }
    }
  }

  const int64_t n = (int64_t)ev.size();
  if (n > cap) return 1;
  int64_t extent = t0;
  for (const auto& e : ev) extent = std::max(extent, e.ts_start);
  int64_t t1;
  if (c->span_ns > 0) {
    t1 = t0 + c->span_ns;
    if (extent >= t1) return 2;
  } else {
    int64_t sec = 1000000000ll;
    t1 = t0 + ((extent - t0) / sec + 1) * sec;
  }

  // delivery order: per-(pid, class) buffers of 4096 records, buffer order shuffled
  std::vector<int32_t> order(n);
  if (c->shuffle_mode == 2) {
    for (int64_t i = 0; i < n; i++) order[i] = (int32_t)i;
  } else if (c->shuffle_mode == 1) {
    for (int64_t i = 0; i < n; i++) order[i] = (int32_t)i;
    for (int64_t i = n - 1; i > 0; i--) std::swap(order[i], order[rng.below((uint64_t)i + 1)]);
  } else {
    std::vector<std::vector<int32_t>> by(P * 3);
    for (int64_t i = 0; i < n; i++)
      by[(ev[i].pid - c->pid_base) * 3 + cls[i]].push_back((int32_t)i);
    struct Buf { int32_t grp; int32_t begin, end; };
    std::vector<Buf> bufs;
    for (int g = 0; g < P * 3; g++)
      for (size_t b = 0; b < by[g].size(); b += 4096)
        bufs.push_back({g, (int32_t)b, (int32_t)std::min(by[g].size(), b + 4096)});
    for (int64_t i = (int64_t)bufs.size() - 1; i > 0; i--)
      std::swap(bufs[i], bufs[rng.below((uint64_t)i + 1)]);
    int64_t o = 0;
    for (const auto& b : bufs)
      for (int32_t j = b.begin; j < b.end; j++) order[o++] = by[b.grp][j];
  }
  std::vector<int32_t> where(n);
  for (int64_t o = 0; o < n; o++) where[order[o]] = (int32_t)o;
  for (int64_t o = 0; o < n; o++) {
    int32_t g = order[o];
    out[o] = ev[g];
    if (truth_link) truth_link[o] = link[g] < 0 ? -1 : where[link[g]];
    if (truth_val) truth_val[o] = val[g];
    if (truth_wait) truth_wait[o] = wait[g];
  }
  if (n_out) *n_out = n;
  if (t1_out) *t1_out = t1;
  if (n_deleted_out) *n_deleted_out = n_deleted;
  return 0;
}

}  // extern "C"
