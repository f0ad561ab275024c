/*
 * ta.h - C ABI of the trace-window analyzer (single NVIDIA B200, sm_100a).
 *
 * The library rebuilds operator executions and cross-process dependencies from
 * one or more bounded profiling windows of host-operator, host-API, launch,
 * kernel, memcpy and collective events.  It implements the reconstruction
 * stage of the paper's Analyzer (Sec. 6.1 "Deriving Performance Observations",
 * Fig. "Key performance observations" (a) and (e)), fed by the record model of
 * Sec. 5.2 "Cross-Layer Profiling Collection".  The paper states the problem;
 * it gives no algorithm, so every rule below that is not followed by a
 * citation is this library's own reading and is stated in full.
 *
 * General conventions
 *   - All times are int64 nanoseconds, all ids are integers; nothing on the
 *     path is floating point.
 *   - Every entry point returns a ta_status; nothing throws, aborts or traps.
 *     After any error the handle stays valid for ta_free().
 *   - "device" pointers live in the memory of env.device, "host" pointers are
 *     ordinary host memory.  Result structs are filled with device pointers
 *     OWNED BY THE HANDLE (valid until ta_free) and host scalars.  Host-side
 *     per-window summary arrays are CALLER-OWNED, W entries, and are filled
 *     after one stream synchronisation at the end of the call.
 *   - Every kernel is enqueued on env.cuda_stream.  Every call that takes a
 *     handle (and ta_load_window) makes env.device the current device of the
 *     calling thread and leaves it current when it returns.
 *   - "Sorted position" p in [0, n) always means a position in the canonical
 *     order produced by ta_sort_timeline; every per-event output of the later
 *     calls is indexed by sorted position.
 *   - Call order: load -> sort -> { correlate -> attribute ; gaps ;
 *     aggregate(value_sel 0) ; collectives }.  aggregate(value_sel 1) needs
 *     attribute.  A call made too early returns TA_ERR_ORDER.
 *   - Threads: a handle is used by one thread at a time; different handles may
 *     be used from different threads and on different streams at the same time
 *     (the library keeps no state outside the handle except its memory pool, the
 *     launch counter and the benchmark instrumentation at the end of this file).
 */
#ifndef TA_H
#define TA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- record model (Sec. 5.2: call function / thread / entry+return times;
 * host API intervals; device activity; correlation id; device and stream ids)
 * 40-byte little-endian record.                                             */
typedef struct ta_event {
  int64_t ts_start; /* entry / start time, ns                                */
  int64_t ts_end;   /* return / completion time, ns, >= ts_start             */
  int64_t corr_id;  /* LAUNCH,KERNEL,MEMCPY: correlation id (per process);
                       COLL: communicator id; otherwise ignored              */
  int32_t pid;      /* process id (signed compare)                           */
  int32_t name_id;  /* symbol id of the function / kernel                    */
  int32_t seq;      /* COLL: sequence number inside the communicator         */
  int16_t stream;   /* host kinds: host thread index; device kinds: stream   */
  int16_t kind;     /* TA_KIND_*                                             */
} ta_event;

enum {
  TA_KIND_OP = 0,     /* host: operator / Python call range                  */
  TA_KIND_API = 1,    /* host: accelerator API call other than a launch      */
  TA_KIND_LAUNCH = 2, /* host: submission API call                           */
  TA_KIND_KERNEL = 3, /* device: kernel execution                            */
  TA_KIND_MEMCPY = 4, /* device: memory operation                            */
  TA_KIND_COLL = 5    /* device: collective                                  */
};
#define TA_N_KINDS 6
#define TA_NBINS 40     /* log2 histogram bins; bin 39 collects >= 2^39 ns   */
#define TA_MAX_DEPTH 8  /* deepest legal nesting of OP ranges                */

typedef enum ta_status {
  TA_OK = 0,
  TA_ERR_INVALID_ARG = 1,
  TA_ERR_OOM = 2,        /* env.alloc returned NULL                          */
  TA_ERR_CUDA = 3,       /* a CUDA runtime call failed                       */
  TA_ERR_ORDER = 4,      /* entry point called before its prerequisites      */
  TA_ERR_TOO_LARGE = 5,  /* a documented size limit was exceeded             */
  TA_ERR_OVERFLOW = 6,   /* an internal bounded table filled up              */
  TA_ERR_TIMEOUT = 7,    /* a bounded device-side wait gave up               */
  TA_ERR_DEPTH = 8,      /* some host record's depth (its level in the parent
                            forest, see ta_attribute_operators) exceeds
                            TA_MAX_DEPTH                                     */
  TA_ERR_BAD_NESTING = 9 /* two ranges of one host thread overlap partially  */
} ta_status;

/* Caller-supplied device memory and stream.  alloc returns device memory on
 * `device` aligned to at least 256 bytes, or NULL; release takes it back.  If
 * alloc is NULL the library allocates stream-ordered from a pool of its own (one
 * per device, created on first use) that keeps freed memory for later calls
 * until the process ends; released blocks are handed out again to requests of
 * the same size on the same stream, and those that no handle has asked for
 * during the lifetime of the last two handles return to the pool. */
typedef struct ta_env {
  void *(*alloc)(size_t bytes, void *ctx);
  void (*release)(void *ptr, void *ctx);
  void *ctx;
  void *cuda_stream; /* cudaStream_t */
  int32_t device;
} ta_env;

typedef struct ta_window ta_window; /* opaque handle; owns every result buffer */

/* ------------------------------------------------------------------------
 * ta_load_window - ingest and validate.  A record belongs to a window by the time
 * it starts (the rule the collection side uses when one recording session
 * follows another, Sec. 5.2 "Session transitions").
 *
 * events   n records, device memory if events_on_device else host memory
 *          (then copied to the device first).  BORROWED: must stay alive and
 *          unmodified until ta_sort_timeline has returned; never freed here.
 * win_off  host, W+1 ascending offsets, win_off[0]=0, win_off[W]=n.  Record k
 *          belongs to window w iff win_off[w] <= k < win_off[w+1].
 * win_t0/1 host, W entries, t0 < t1, t1 - t0 < 2^40.
 * A record is DROPPED by the first rule that applies:
 *   kind outside [0,5]            -> n_bad_kind
 *   ts_end < ts_start             -> n_bad_interval
 *   ts_start < t0 or >= t1        -> n_out_of_window
 * (ts_end > t1 is legal.)  Dropped records take part in nothing but `perm`.
 * Limits: n < 2^31; at most 4096 distinct (pid, domain, stream) triples; the
 * sort key (window, triple, ts_start - t0) must fit 63 bits; W x 2^ceil(log2(number of
 * triples)) <= 2^24.
 * out_summary: host, W entries, caller-owned.
 * Errors: INVALID_ARG (null pointers, bad offsets, t0 >= t1), TOO_LARGE, OOM, CUDA.
 */
typedef struct ta_load_summary {
  int64_t n_events, n_valid, n_bad_kind, n_bad_interval, n_out_of_window;
} ta_load_summary;

ta_status ta_load_window(const ta_env *env, const ta_event *events, int64_t n,
                         int32_t events_on_device, const int64_t *win_off,
                         const int64_t *win_t0, const int64_t *win_t1, int32_t W,
                         ta_load_summary *out_summary, ta_window **handle);

/* ------------------------------------------------------------------------
 * ta_sort_timeline - canonical order (device and stream identifiers locate
 * device work, thread identifiers locate calls: Sec. 5.2).
 *
 * domain d = 0 for kinds 0..2 (host), 1 for kinds 3..5 (device).
 * Canonical order = ascending by the tuple
 *   (dropped, window, pid, d, stream, ts_start, -ts_end, input index),
 * pid and stream compared as signed integers.  For a dropped record
 * d = (kind >= 3).  perm[p] = input index of the record at sorted position p;
 * kept records occupy [0, n_valid), dropped ones [n_valid, n).
 * A LANE is a maximal run of kept records with equal (window, pid, d, stream);
 * lanes are listed in sorted order, lane l covers [lane_off[l], lane_off[l+1]).
 * The eight columns hold the records in sorted order (all n of them).
 */
typedef struct ta_sort_result {
  int64_t n, n_valid;
  int32_t n_lanes;
  int32_t n_windows;
  const int32_t *perm;                         /* device, n                  */
  const int64_t *ts_start, *ts_end, *corr_id;  /* device, n each             */
  const int32_t *pid, *name_id, *seq;          /* device, n each             */
  const int16_t *stream, *kind;                /* device, n each             */
  const int32_t *lane_window, *lane_pid;       /* device, n_lanes each       */
  const int16_t *lane_stream, *lane_domain;    /* device, n_lanes each       */
  const int32_t *lane_off;                     /* device, n_lanes + 1        */
} ta_sort_result;

ta_status ta_sort_timeline(ta_window *h, ta_sort_result *out);

/* ------------------------------------------------------------------------
 * ta_correlate_launches - joins every device record to the host call that
 * submitted it, through the correlation id both carry (Sec. 5.2; Fig. "Key
 * performance observations" (a)).
 *
 * Build side: kept LAUNCH records.  Probe side: kept KERNEL and MEMCPY
 * records.  Key = (window, pid, corr_id), all 64 bits of corr_id significant.
 * For a probe at sorted position i, launch_of[i] = the SMALLEST sorted
 * position of a LAUNCH with an equal key, or -1.  If matched to l:
 *   launch_latency[i] = ts_start[i] - ts_start[l]          (signed)
 *   queue_delay[i]    = max(0, ts_start[i] - ts_end[l])
 * Elsewhere launch_of = -1 and both times are 0.  kernels_of_launch[l] = number
 * of probes with launch_of == l (0 at non-launch positions); several probes
 * per launch are legal (graph replay, Sec. 6.1).
 * Per-window summary: n_dup_launch counts LAUNCH records whose key already
 * belongs to a smaller sorted position; n_orphan_launch counts LAUNCH records
 * that are not such duplicates and have no probe; min/max are 0 when
 * n_matched == 0.
 */
typedef struct ta_join_summary {
  int64_t n_probe, n_matched, n_unmatched, n_launch, n_dup_launch, n_orphan_launch;
  int64_t sum_latency, min_latency, max_latency, sum_queue, max_queue;
} ta_join_summary;

typedef struct ta_join_result {
  const int32_t *launch_of;         /* device, n */
  const int64_t *launch_latency;    /* device, n */
  const int64_t *queue_delay;       /* device, n */
  const int32_t *kernels_of_launch; /* device, n */
} ta_join_result;

ta_status ta_correlate_launches(ta_window *h, ta_join_result *out,
                                ta_join_summary *out_summary);

/* ------------------------------------------------------------------------
 * ta_attribute_operators - finds, for every host record, the operator range of
 * the same thread that contains it (the linkage of Sec. 9.1: same thread,
 * nested intervals) and gives every device record the operator of its launch;
 * per operator, T_op runs from the start of its first kernel to the end of its
 * last (Sec. 6.1).  A kernel may still run after the call that launched it has
 * returned (Sec. 5.2), so containment is tested on the LAUNCH interval.
 *
 * Inside one host lane, OP j ENCLOSES host record i (i != j) iff
 * ts_start[j] <= ts_start[i] and ts_end[i] <= ts_end[j] and, when both
 * intervals are identical, j precedes i in canonical order.
 *   parent[i] = the encloser with the largest ts_start, then the smallest
 *               ts_end, then the largest sorted position; -1 if none.
 *   depth[i]  = 0 if parent[i] == -1, else depth[parent[i]] + 1, saturating at
 *               255.  In a properly nested lane this is the number of enclosers
 *               of every record of non-zero length.
 * Device records: op_of[i] = parent[launch_of[i]] for KERNEL/MEMCPY with a
 * launch, else -1.  For every OP r, over device records with op_of == r:
 *   op_n_kernels[r], op_first_start[r] = min ts_start, op_last_end[r] =
 *   max ts_end, op_kernel_ns[r] = sum of durations;
 *   T_op[r] = op_last_end[r] - op_first_start[r].
 * All four are 0 when op_n_kernels[r] == 0 and at non-OP positions.
 * Returns TA_ERR_BAD_NESTING if some OP j and host record i of one lane have
 * ts_start[j] < ts_start[i] < ts_end[j] < ts_end[i], else TA_ERR_DEPTH if some
 * depth exceeds TA_MAX_DEPTH; in both cases the summaries' max_depth /
 * bad_nesting fields are filled and the other outputs are unspecified.
 */
typedef struct ta_attr_summary {
  int64_t n_attributed, n_no_launch, n_no_op;
  int32_t max_depth, bad_nesting;
} ta_attr_summary;

typedef struct ta_attr_result {
  const int32_t *parent;         /* device, n */
  const uint8_t *depth;          /* device, n */
  const int32_t *op_of;          /* device, n */
  const int64_t *op_first_start; /* device, n */
  const int64_t *op_last_end;    /* device, n */
  const int64_t *op_kernel_ns;   /* device, n */
  const int32_t *op_n_kernels;   /* device, n */
} ta_attr_result;

ta_status ta_attribute_operators(ta_window *h, ta_attr_result *out,
                                 ta_attr_summary *out_summary);

/* ------------------------------------------------------------------------
 * ta_stream_gaps - where each device stream sat idle: the time not covered by
 * any of its activity records (the idle-time observation of Sec. 9.1).
 *
 * For a device lane of a window [W0, W1) with records 0..m-1 in canonical
 * order and clipped ends c_i = min(ts_end_i, W1):
 *   P_0 = W0, P_{i+1} = max(P_i, c_i)
 *   gap_before[i] = max(0, ts_start_i - P_i)
 *   busy_i        = max(0, c_i - max(ts_start_i, P_i))
 *   tail_gap      = W1 - P_m
 * so that busy + idle == W1 - W0 for every lane.  Each positive gap g (head,
 * interior, tail) adds one to histogram bin min(39, floor(log2 g)).
 * lane_gaps / lane_hist have one row per lane of the lane table; rows of host
 * lanes are zero.  win_hist[w] sums the window's lanes.  The long-gap list
 * holds every gap with g > 0 and g >= min_gap_ns, ordered by lane, then time,
 * a lane's tail gap last.
 * Limits: fewer than 2^22 - 1 lanes (TA_ERR_TOO_LARGE).
 */
typedef struct ta_lane_gaps {
  int64_t busy, idle, n_events, n_gaps, max_gap, first_start, last_end;
} ta_lane_gaps;

typedef struct ta_long_gap {
  int32_t lane;       /* index into the lane table                           */
  int32_t next_event; /* sorted position of the record after the gap, -1 = tail */
  int64_t gap_start;  /* = P_i                                               */
  int64_t gap_len;
} ta_long_gap;

typedef struct ta_gap_result {
  const int64_t *gap_before;      /* device, n (0 at host and dropped positions) */
  const ta_lane_gaps *lane_gaps;  /* device, n_lanes                         */
  const uint32_t *lane_hist;      /* device, n_lanes x TA_NBINS              */
  const uint32_t *win_hist;       /* device, n_windows x TA_NBINS            */
  const ta_long_gap *long_gaps;   /* device, n_long_gaps                     */
  int64_t n_long_gaps;
} ta_gap_result;

ta_status ta_stream_gaps(ta_window *h, int64_t min_gap_ns, ta_gap_result *out);

/* ------------------------------------------------------------------------
 * ta_aggregate_ops - per-symbol call counts and duration statistics (the
 * fidelity measures of Sec. 8.1 are per-symbol counts and kernel durations).
 *
 * Population: kept records with (1 << kind) & kind_mask.  value_sel 0: value =
 * ts_end - ts_start.  value_sel 1: kind_mask must be exactly 1 << TA_KIND_OP
 * (else INVALID_ARG); the population is further restricted to OPs with
 * op_n_kernels > 0 and value = T_op.  value_sel 2 (after ta_blame_gaps, else
 * TA_ERR_ORDER; kind_mask again exactly 1 << TA_KIND_OP): OPs with
 * op_gap_ns > 0, value = op_gap_ns.  value_sel 3 (after ta_critical_path, else
 * TA_ERR_ORDER; any kind_mask): records with on_path = 1, value = ts_end -
 * ts_start - which symbols the critical paths run through, and for how long.
 * Group key (window, pid, name_id); one
 * output row per non-empty group in ascending signed key order with count,
 * sum, min, max and a histogram whose bin is min(39, floor(log2 v)) for
 * v >= 1 and 0 for v <= 0.
 * While (#windows x #pids x (max name_id - min name_id + 1)) <= 2^27 the rows are
 * accumulated in a dense table; symbol ids spread wider than that are grouped
 * by sorting instead (slower, same result).  The result buffers of an earlier
 * ta_aggregate_ops call on the same handle stay valid.
 */
typedef struct ta_agg_result {
  int64_t n_groups;
  const int32_t *g_window, *g_pid, *g_name;       /* device, n_groups each   */
  const int64_t *g_count, *g_sum, *g_min, *g_max; /* device, n_groups each   */
  const uint32_t *g_hist;                         /* device, n_groups x TA_NBINS */
} ta_agg_result;

ta_status ta_aggregate_ops(ta_window *h, uint32_t kind_mask, int32_t value_sel,
                           ta_agg_result *out);

/* ------------------------------------------------------------------------
 * ta_match_collectives - links the records of different processes that name the
 * same collective (same communicator, same sequence number) and measures how
 * long each rank waited for the last one to arrive (cross-process links:
 * Sec. 6.1 "Execution progress and state"; ranks held up by a late one: Sec. 9.2).
 *
 * Population: kept COLL records; comm_id = corr_id.  Group key
 * (window, comm_id, seq), groups output in ascending signed key order.
 * Per group: n_members, min_start, max_start, skew = max_start - min_start,
 * max_end, straggler_pid = pid of the member with the largest ts_start (ties:
 * smallest pid), flags bit0 INCOMPLETE (n_members != the size given for that
 * comm_id in `sizes`; for a comm_id not listed: n_members < 2), bit1 DUP_PID
 * (some pid occurs twice).  wait_ns[i] = max_start - ts_start[i] for every
 * member of every group, 0 at non-COLL positions.  Rank table: one row per
 * (window, pid) that has COLL records, ascending; its four counters cover only
 * members of groups with flags == 0 (n_coll = number of such members,
 * n_straggler = number of those groups whose straggler_pid is this pid).
 * sizes: host, n_comms entries (may be NULL when n_comms == 0).
 */
typedef struct ta_comm_size {
  int64_t comm_id;
  int32_t n_ranks;
  int32_t reserved;
} ta_comm_size;

#define TA_COLL_INCOMPLETE 1
#define TA_COLL_DUP_PID 2

typedef struct ta_coll_result {
  int64_t n_groups, n_ranks;
  const int32_t *g_window;      /* device, n_groups */
  const int64_t *g_comm;        /* device, n_groups */
  const int32_t *g_seq;         /* device, n_groups */
  const int32_t *g_n_members;   /* device, n_groups */
  const int64_t *g_min_start, *g_max_start, *g_skew, *g_max_end; /* device, n_groups */
  const int32_t *g_straggler_pid, *g_flags;                      /* device, n_groups */
  const int64_t *wait_ns;       /* device, n */
  const int32_t *r_window, *r_pid;                               /* device, n_ranks */
  const int64_t *r_n_coll, *r_sum_wait, *r_max_wait, *r_n_straggler; /* device, n_ranks */
} ta_coll_result;

ta_status ta_match_collectives(ta_window *h, const ta_comm_size *sizes,
                               int32_t n_comms, ta_coll_result *out);

/* ------------------------------------------------------------------------
 * ta_device_overlap - device-level coverage per (window, process): how much of
 * the communication time ran while kernels were running too, and how much was
 * left uncovered, both as measures of unions of intervals (Sec. 6.1, "Execution
 * progress and state"; Fig. "Overlap and exposed work").  Beyond the seven calls above:
 * the first of the analyses that build on them.  Needs ta_sort_timeline only.
 *
 * For every (window, pid) that has at least one kept device record, over ALL of
 * its device streams, with every record's interval taken as
 * [ts_start, min(ts_end, t1)) (an empty interval covers nothing):
 *   d_n_events  number of kept device records
 *   d_busy      measure of the union of all intervals; d_idle = (t1 - t0) - d_busy
 *   d_compute   measure of the union of the KERNEL intervals
 *   d_comm      measure of the union of the MEMCPY and COLL intervals
 *   d_overlap   measure of the intersection of those two unions
 *   d_exposed   d_comm - d_overlap
 * Rows are ordered by (window, pid ascending).  Readings (the paper names the
 * two lanes "Compute" and "Comm. / IO" and gives no rule): memory copies count
 * as communication / IO; ends are clipped to the window as in ta_stream_gaps.
 * All arrays are device memory owned by the handle, n_rows entries each.
 * Limits: as ta_load_window, and windows x pids < 2^22 (TA_ERR_TOO_LARGE).
 * Errors: TA_ERR_ORDER before ta_sort_timeline; TA_ERR_OOM; TA_ERR_CUDA;
 * TA_ERR_TIMEOUT.  One stream synchronisation at the end. */
typedef struct ta_overlap_result {
  int64_t n_rows;
  const int32_t *d_window, *d_pid;
  const int64_t *d_n_events, *d_busy, *d_idle, *d_compute, *d_comm, *d_overlap, *d_exposed;
} ta_overlap_result;

ta_status ta_device_overlap(ta_window *h, ta_overlap_result *out);

/* ------------------------------------------------------------------------
 * ta_rollup_operators - inclusive per-operator kernel figures and graph
 * replays.  Which kernels make up an operator invocation follows from the join
 * and the attribution above; under CUDA Graph replay no operator call is
 * recorded and the kernels of one replay are told apart only by the launch they
 * share (Sec. 6.1, "Operator execution and efficiency").  Beyond the seven
 * calls above.  Needs ta_attribute_operators to have returned TA_OK.
 *
 * Readings.  For an OP at sorted position r, over r itself and every OP below it
 * in the forest `parent` defines:
 *   incl_n_kernels[r] = sum of op_n_kernels, incl_kernel_ns[r] = sum of op_kernel_ns,
 *   incl_first_start[r] = min of op_first_start, incl_last_end[r] = max of
 *   op_last_end over those of them that own kernels; all four 0 when none does.
 * For a LAUNCH at position l with kernels_of_launch[l] >= 2 (one graph replay):
 *   replay_first_start[l] / replay_last_end[l] = min ts_start / max ts_end
 *   (unclipped) of the device records with launch_of == l, replay_kernel_ns[l] =
 *   sum of their durations; 0 for every other position.
 * out_summary[w]: number of such launches in window w, the device records they
 * own, and the most owned by one launch.
 * MFU, MBU and SOL_op of the same section need per-invocation operation counts
 * and device peaks that a 40-byte record does not carry: see ta_operator_sol.
 * All arrays are device memory owned by the handle, n entries each.
 * Errors: TA_ERR_ORDER unless ta_attribute_operators returned TA_OK;
 * TA_ERR_OOM; TA_ERR_CUDA.  One stream synchronisation at the end. */
typedef struct ta_rollup_summary {
  int64_t n_graph_launches, n_graph_kernels, max_kernels_per_launch;
} ta_rollup_summary;

typedef struct ta_rollup_result {
  const int32_t *incl_n_kernels;
  const int64_t *incl_first_start, *incl_last_end, *incl_kernel_ns;
  const int64_t *replay_first_start, *replay_last_end, *replay_kernel_ns;
} ta_rollup_result;

ta_status ta_rollup_operators(ta_window *h, ta_rollup_result *out,
                              ta_rollup_summary *out_summary /* host, n_windows entries */);

/* ------------------------------------------------------------------------
 * ta_operator_sol - efficiency of every operator invocation (Sec. 6.1, "Operator
 * execution and efficiency"): its theoretical operation count and its logical
 * data volume, each normalised by T_op and by the device peak, are the model
 * FLOPs utilisation and the model bandwidth utilisation; speed-of-light
 * attainment is SOL_op = max(MFU, MBU).  Beyond the seven calls above.  Needs
 * ta_attribute_operators to have returned TA_OK.  The only floating-point step
 * of the library.
 *
 * The counts are the caller's: they follow from shapes, data types and sharding,
 * which no trace record carries.  flops / bytes: n float64 each, indexed by INPUT
 * record index (the order of `events`), in device memory if counts_on_device else
 * in host memory (then copied first); read for OP records only; a negative value
 * or a NaN means "not known".  Borrowed for the duration of the call.
 * peak_flops in FLOP/s, peak_bw in bytes/s, both > 0 (else TA_ERR_INVALID_ARG).
 * Per kept OP record at sorted position r with T_op = op_last_end - op_first_start:
 *   state[r] = 2  op_n_kernels[r] == 0 or T_op == 0: no kernel composition, unresolved
 *              3  kernels, but flops or bytes of the record is not known: unresolved
 *              1  resolved:  mfu[r] = flops / (T_op * 1e-9 * peak_flops)
 *                            mbu[r] = bytes / (T_op * 1e-9 * peak_bw)
 *                            sol[r] = max(mfu[r], mbu[r])
 * state = 0 at every other position; mfu = mbu = sol = 0 unless state = 1.
 * out_summary[w]: the three state counts of window w; over its resolved
 * invocations the sums of T_op (exact), flops and bytes, and the largest sol.
 * Precision: IEEE double, the operations exactly as written above (two
 * multiplications and one division per figure), so the per-record figures equal
 * a plain CPU evaluation bit for bit; sum_flops and sum_bytes are accumulated in
 * no particular order and agree with a sequential sum to a relative 1e-9 (the
 * worst case of adding 10^7 positive doubles in another order).
 * All arrays are device memory owned by the handle, n entries each.
 * Errors: TA_ERR_ORDER unless ta_attribute_operators returned TA_OK;
 * TA_ERR_INVALID_ARG; TA_ERR_OOM; TA_ERR_CUDA.  One stream synchronisation. */
typedef struct ta_sol_summary {
  int64_t n_resolved, n_no_kernels, n_no_counts, sum_top_ns;
  double sum_flops, sum_bytes, max_sol;
} ta_sol_summary;

typedef struct ta_sol_result {
  const double *mfu, *mbu, *sol; /* device, n each */
  const uint8_t *state;          /* device, n      */
} ta_sol_result;

ta_status ta_operator_sol(ta_window *h, const double *flops, const double *bytes,
                          int32_t counts_on_device, double peak_flops, double peak_bw,
                          ta_sol_result *out, ta_sol_summary *out_summary /* host, n_windows entries */);

/* ------------------------------------------------------------------------
 * ta_blame_gaps - why a device stream sat idle, and which host calls were
 * running meanwhile.  A gap is laid at the door of the host when the work that
 * ended it had not even been submitted while the stream was already idle (the
 * late-dispatch test of Sec. 6.2, engine patterns; "submission gaps", Sec. 8.2);
 * idle time is charged to the operators it overlaps (the case of Sec. 9.1, where
 * one waiting call accounts for most of the idle time).  Beyond the seven calls above.
 * Needs ta_correlate_launches and the result of a ta_stream_gaps call on the
 * same handle (`gaps`, borrowed for the duration of the call).
 *
 * Readings (the paper gives no rule).  Per long gap k of gaps->long_gaps:
 *   g_class[k] = TA_BLAME_TAIL        the gap runs to the window end (next_event = -1)
 *                TA_BLAME_NO_LAUNCH   the record that ends it has launch_of = -1
 *                                     (COLL records, kernels whose launch is missing)
 *                TA_BLAME_SUBMISSION  ts_start[launch] >= gap_start: the stream was
 *                                     already idle when the host submitted the work
 *                TA_BLAME_QUEUED      ts_start[launch] <  gap_start: submitted in
 *                                     time, started late (queue, dependency)
 *   g_launch[k] = that launch's sorted position, or -1.
 * out_summary[w].count[c] / .ns[c]: number and total length of the long gaps of
 * window w per class c.
 * Per OP record r: op_gap_ns[r] = sum, over the long gaps of ALL device streams
 * of r's (window, pid), of the length of [gap_start, gap_start + gap_len) n
 * [ts_start[r], ts_end[r]); 0 at every other position.  With one stream per
 * device this is the GPU idle time that coincides with the call; with several
 * streams it is stream-idle time (each stream counts).  The per-symbol table is
 * ta_aggregate_ops(h, 1 << TA_KIND_OP, 2, ...): operators with op_gap_ns > 0.
 * All arrays are device memory owned by the handle.
 * Errors: TA_ERR_ORDER before ta_correlate_launches; TA_ERR_INVALID_ARG;
 * TA_ERR_OOM; TA_ERR_CUDA; TA_ERR_TIMEOUT.  One stream synchronisation. */
enum { TA_BLAME_NO_LAUNCH = 0, TA_BLAME_SUBMISSION = 1, TA_BLAME_QUEUED = 2, TA_BLAME_TAIL = 3 };

typedef struct ta_blame_summary {
  int64_t count[4], ns[4]; /* indexed by TA_BLAME_* */
} ta_blame_summary;

typedef struct ta_blame_result {
  int64_t n_long_gaps;
  const int32_t *g_class, *g_launch; /* device, n_long_gaps */
  const int64_t *op_gap_ns;          /* device, n           */
} ta_blame_result;

ta_status ta_blame_gaps(ta_window *h, const ta_gap_result *gaps, ta_blame_result *out,
                        ta_blame_summary *out_summary /* host, n_windows entries */);

/* ta_free - releases every buffer of the handle through env.release.
 * NULL-safe.  Synchronises the handle's stream first. */
void ta_free(ta_window *h);

/* ------------------------------------------------------------------------
 * ta_critical_path - per (window, process), the chain of binding dependencies
 * that ends at the last record to finish.  Three kinds of dependency are
 * followed - a kernel on its launch, a record on the one before it in its
 * stream or thread, a waiting host call on the device record that released it -
 * and a delay for which the trace holds no such dependency is reported as
 * unresolved rather than guessed (Sec. 6.1, "Execution
 * progress and state"; Fig. "Critical path": host work, the call that submits
 * k1, k1, the end of the host's wait, host work again - a kernel of another
 * stream and the wait itself stay off the path).  Beyond the seven calls above.
 * Needs ta_correlate_launches.
 *
 * Readings.  Nodes are the valid API and LAUNCH records (host) and the KERNEL,
 * MEMCPY and COLL records (device); OP records are context, not nodes.  A node
 * has a START point (ts_start) and an END point (ts_end).  The walk starts at the
 * END of the sink - the node of the (window, process) with the greatest ts_end,
 * the highest sorted position among equals - and always steps back to the
 * dependency that was released last:
 *   END(v), v an API record that waited: to END(d), d = the device record of the
 *     process with the greatest ts_end < ts_end(v) (highest position among
 *     equals); v waited iff ts_end(d) >= ts_start(v).        [synchronisation]
 *   END(v) otherwise: to START(v).                            [v ran]
 *   START(k), k a device record: stream order offers END(q), q the record just
 *     before k in its lane, if ts_end(q) <= ts_start(k); submission offers
 *     START(l), l = launch_of[k], if l >= 0 and ts_start(l) <= ts_start(k).  With
 *     both on offer stream order binds iff ts_end(q) > ts_start(l) (the test of
 *     ta_blame_gaps); with neither the path ends here, unresolved (reason 1).
 *   START(h), h a host node: to the node u just before h in its lane (program
 *     order): END(u) if ts_end(u) <= ts_start(h), else START(u) (h ran inside u);
 *     without u the path ends at the start of the thread (reason 0).
 * Time never increases along the walk and strictly decreases on a
 * synchronisation edge, which every cycle would need, so the walk ends.
 * The time between the path's begin and the sink's end splits into eight
 * classes that add up exactly (p_ns, TA_CP_*): execution of KERNEL, MEMCPY and
 * COLL records on the path; launch latency (ts_start(k) - ts_start(l) on
 * submission edges); delay on stream-order edges (unresolved); time inside host
 * calls; host time between calls; the tail of a wait after the device finished
 * (ts_end(v) - ts_end(d) on synchronisation edges - the wait itself is context,
 * not another copy of the device's time).
 *
 * Outputs (device memory owned by the handle): on_path[n], 1 for every node the
 * walk passes through; one row per (window, process) that has a node, ordered by
 * (window, pid): p_sink (sorted position), p_begin / p_end (time where the walk
 * ended / ts_end of the sink), p_n_nodes, p_reason, p_ns[row * 8 + class].
 * out_summary[w]: rows, nodes and class totals of window w.
 * Limits: window span and the longest record < 2^40 ns each, windows x pids <
 * 2^22 (TA_ERR_TOO_LARGE).
 * Errors: TA_ERR_ORDER before ta_correlate_launches; TA_ERR_OOM; TA_ERR_CUDA;
 * TA_ERR_TIMEOUT.  Two stream synchronisations (three when some stream lane
 * does not end its records in ascending order and the device records have to
 * be sorted by end time). */
enum {
  TA_CP_KERNEL = 0, TA_CP_MEMCPY = 1, TA_CP_COLL = 2, TA_CP_LAUNCH_LATENCY = 3,
  TA_CP_STREAM_DELAY = 4, TA_CP_IN_CALL = 5, TA_CP_BETWEEN_CALLS = 6, TA_CP_WAIT_TAIL = 7
};
typedef struct ta_critpath_summary {
  int64_t n_paths, n_nodes, ns[8];
} ta_critpath_summary;

typedef struct ta_critpath_result {
  int64_t n_rows;
  const uint8_t *on_path;
  const int32_t *p_window, *p_pid, *p_sink, *p_n_nodes, *p_reason;
  const int64_t *p_begin, *p_end, *p_ns;
} ta_critpath_result;

ta_status ta_critical_path(ta_window *h, ta_critpath_result *out,
                           ta_critpath_summary *out_summary /* host, n_windows entries */);

/* ------------------------------------------------------------------------
 * ta_lane_gaps_noalloc - the stream-gap scan of ONE device lane, for callers
 * that cannot allocate device memory.  (The paper has no counterpart for this
 * entry point; it exists for integration reasons only.)
 *
 * Who needs it: a monitoring agent that lives inside a serving process whose
 * device heap is fully reserved at start-up, a plug-in whose host forbids
 * cudaMalloc / cudaFree inside its callbacks, or a latency-critical loop that
 * cannot afford the device-wide synchronisation an allocation or a free may
 * imply.  Every other entry point obtains its buffers through ta_env; this one
 * obtains nothing: it calls no cudaMalloc, cudaFree or any allocating routine.
 * Its scratch (tile descriptors of the scan, a counter, a status word: about
 * 16 KB) is a fixed array inside the library image, which every GPU that loads
 * the library holds until the process exits.
 *
 * Input: the records of one device lane of one window [win_t0, win_t1), already
 * in canonical order (ts_start ascending), as two device columns of n entries;
 * every ts_start lies in the window.  Output, both caller-owned device memory:
 * gap_before[n] and one ta_lane_gaps row, with exactly the values ta_stream_gaps
 * gives for that lane (gap_before, busy, idle, n_events, n_gaps, max_gap,
 * first_start, last_end).  No histogram and no long-gap list.
 *
 * Limits and rules: n <= TA_NOALLOC_MAX_RECORDS, else TA_ERR_TOO_LARGE (the
 * fixed scratch covers no more).  gap_before and lane_out must be 8-byte aligned
 * (lane_out receives 64-bit atomic updates).  The first call on a device looks
 * up the address of the scratch array (with that device current) and should
 * therefore be made before any stream capture begins; it is also the call at
 * which the CUDA runtime may load the library's code and the scratch array onto
 * the device (lazy module loading), which does take device memory: make it once
 * at start-up, before the heap is reserved, not at the first moment of need.  All calls on a device share the
 * one scratch array, which keeps the previous call's contents; each call clears
 * it first, so two calls that overlap on the GPU (different streams or threads)
 * race and must be serialised by the caller.  The call enqueues its work on
 * cuda_stream, waits for it and returns TA_OK, TA_ERR_INVALID_ARG,
 * TA_ERR_TOO_LARGE, TA_ERR_CUDA or TA_ERR_TIMEOUT.
 */
#define TA_NOALLOC_MAX_RECORDS (1 << 22)
ta_status ta_lane_gaps_noalloc(const int64_t *ts_start, const int64_t *ts_end, int64_t n,
                               int64_t win_t0, int64_t win_t1, int64_t *gap_before,
                               ta_lane_gaps *lane_out, void *cuda_stream);

/* Helpers that carry no work. */
const char *ta_strerror(ta_status s);
int32_t ta_version(void);

/* Instrumentation (process-wide, not thread-safe; meant for benchmarks).
 * ta_launch_count: number of kernels this library has launched since it was
 * loaded.  ta_profile_enable(1): from now on record a CUDA event pair around
 * every radix-sort pass (the dominant kernel) on the launching stream, and
 * forget the pairs recorded so far; ta_profile_enable(0) stops recording.
 * ta_profile_radix: synchronises the recorded events and returns the number of
 * passes timed, the sum of their durations in milliseconds and the algorithmic
 * bytes they moved (16 B per record and pass when the sort key carries the
 * record index, 24 B when (key, index) pairs are sorted); 0 on success, -1 on a
 * CUDA error. */
int64_t ta_launch_count(void);
void ta_profile_enable(int32_t on);
int32_t ta_profile_radix(int64_t *n_passes, double *total_ms, double *total_bytes);

/* Test hooks for the failure path (process-wide; meant for tests).
 * Kernels that wait for another thread block (the chained scans, the radix
 * passes) poll a descriptor a bounded number of times - 2^22 unless changed
 * here - and then record TA_ERR_TIMEOUT in the handle's device status word and
 * finish without writing output; every kernel launched on the handle afterwards
 * sees the word and returns at once, and the entry point returns TA_ERR_TIMEOUT
 * (as does every later call on that handle except ta_free).
 * ta_set_spin_limit: poll limit of handles created from now on (<= 0 restores
 * the default).  ta_selftest_wait_timeout: launches one warp on cuda_stream that
 * waits, with a limit of `polls` polls (1 .. 2^20), for a descriptor that nothing
 * ever publishes, waits for the kernel and returns what the wait recorded:
 * TA_ERR_TIMEOUT when the bounded wait works as intended.  Uses 512 bytes from
 * cudaMallocAsync.  Other returns: TA_ERR_INVALID_ARG, TA_ERR_OOM, TA_ERR_CUDA. */
void ta_set_spin_limit(int32_t polls);
ta_status ta_selftest_wait_timeout(void *cuda_stream, int32_t polls);
/* ta_inject_device_error: writes `code` (an error status) into the handle's
 * device status word from the host, as a device-side wait that gave up would,
 * so that a test can check what follows such a failure without causing one:
 * every later call on the handle except ta_free returns `code`, and its kernels
 * return without touching their inputs.  Returns TA_OK, TA_ERR_INVALID_ARG or
 * TA_ERR_CUDA. */
ta_status ta_inject_device_error(ta_window *h, ta_status code);

#ifdef __cplusplus
}
#endif
#endif /* TA_H */
