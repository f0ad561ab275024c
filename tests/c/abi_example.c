/* A C program that uses the analyzer through include/ta.h alone (no Python, no
 * allocator callbacks: the library's own stream-ordered pool serves the memory).
 * It analyses the hand-worked gap window H1 (six kernels on one stream, window
 * [0, 1000)) and checks the figures worked out by hand in tests/golden/H1_gaps.txt.
 * Exit code 0 = all checks passed.  Built and run by tests/test_c_abi.py. */
#include <cuda_runtime_api.h>
#include <stdio.h>
#include <string.h>

#include "ta.h"

#define CHECK(cond)                                                        \
  do {                                                                     \
    if (!(cond)) {                                                         \
      fprintf(stderr, "check failed at line %d: %s\n", __LINE__, #cond);   \
      return 1;                                                            \
    }                                                                      \
  } while (0)

int main(void) {
  const int64_t starts[6] = {100, 150, 300, 500, 520, 900};
  const int64_t ends[6] = {200, 300, 350, 600, 540, 1200};
  ta_event ev[6];
  memset(ev, 0, sizeof(ev));
  for (int i = 0; i < 6; i++) {
    ev[i].ts_start = starts[i];
    ev[i].ts_end = ends[i];
    ev[i].pid = 1;
    ev[i].stream = 7;
    ev[i].kind = TA_KIND_KERNEL;
  }
  CHECK(cudaSetDevice(0) == cudaSuccess);
  ta_env env;
  memset(&env, 0, sizeof(env));  /* no callbacks, default stream, device 0 */
  const int64_t off[2] = {0, 6}, t0[1] = {0}, t1[1] = {1000};
  ta_load_summary ls;
  ta_window *h = NULL;
  CHECK(ta_load_window(&env, ev, 6, 0 /* host records */, off, t0, t1, 1, &ls, &h) == TA_OK);
  CHECK(ls.n_events == 6 && ls.n_valid == 6);

  ta_gap_result gaps;
  CHECK(ta_stream_gaps(h, 120, &gaps) == TA_ERR_ORDER); /* the sort comes first */
  ta_sort_result sorted;
  CHECK(ta_sort_timeline(h, &sorted) == TA_OK);
  CHECK(sorted.n_valid == 6 && sorted.n_lanes == 1);
  CHECK(ta_stream_gaps(h, 120, &gaps) == TA_OK);
  CHECK(gaps.n_long_gaps == 2);

  int64_t gap_before[6];
  ta_lane_gaps lane;
  ta_long_gap list[2];
  CHECK(cudaMemcpy(gap_before, gaps.gap_before, sizeof(gap_before), cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(&lane, gaps.lane_gaps, sizeof(lane), cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(list, gaps.long_gaps, sizeof(list), cudaMemcpyDeviceToHost) == cudaSuccess);
  const int64_t want[6] = {100, 0, 0, 150, 0, 300};
  for (int i = 0; i < 6; i++) CHECK(gap_before[i] == want[i]);
  CHECK(lane.busy == 450 && lane.idle == 550 && lane.n_gaps == 3 && lane.max_gap == 300);
  CHECK(lane.first_start == 100 && lane.last_end == 1000 && lane.n_events == 6);
  CHECK(list[0].next_event == 3 && list[0].gap_start == 350 && list[0].gap_len == 150);
  CHECK(list[1].next_event == 5 && list[1].gap_start == 600 && list[1].gap_len == 300);

  ta_overlap_result ov;
  CHECK(ta_device_overlap(h, &ov) == TA_OK && ov.n_rows == 1);
  int64_t busy = 0, comm = -1;
  CHECK(cudaMemcpy(&busy, ov.d_busy, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(&comm, ov.d_comm, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(busy == 450 && comm == 0);

  /* the critical path of a stream without launches: from the kernel that ends last (1200) back
   * along the stream - [520,540) ended before it began, a delay of 360 - and unresolved at 520,
   * because the kernel before that one was still running when it began */
  ta_critpath_result cp;
  ta_critpath_summary cps;
  CHECK(ta_critical_path(h, &cp, &cps) == TA_ERR_ORDER); /* the join comes first */
  ta_join_result join;
  ta_join_summary js;
  CHECK(ta_correlate_launches(h, &join, &js) == TA_OK);
  CHECK(ta_critical_path(h, &cp, &cps) == TA_OK && cp.n_rows == 1);
  CHECK(cps.n_paths == 1 && cps.n_nodes == 2);
  CHECK(cps.ns[TA_CP_KERNEL] == 320 && cps.ns[TA_CP_STREAM_DELAY] == 360);
  int64_t begin = 0, end = 0;
  int32_t reason = -1;
  CHECK(cudaMemcpy(&begin, cp.p_begin, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(&end, cp.p_end, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(&reason, cp.p_reason, 4, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(begin == 520 && end == 1200 && reason == 1);

  ta_free(h);
  ta_free(NULL);
  printf("c abi ok (library version %d, %lld kernel launches)\n", (int)ta_version(), (long long)ta_launch_count());
  return 0;
}
