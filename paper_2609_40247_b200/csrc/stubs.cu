// Temporary placeholders for steps that are not implemented yet.
#include "ta_internal.cuh"
ta_status ta_run_correlate(ta_window *, ta_join_summary *) { return TA_ERR_ORDER; }
ta_status ta_run_attribute(ta_window *, ta_attr_summary *) { return TA_ERR_ORDER; }
ta_status ta_run_aggregate(ta_window *, uint32_t, int, ta_agg_result *) { return TA_ERR_ORDER; }
ta_status ta_run_collectives(ta_window *, const ta_comm_size *, int32_t, ta_coll_result *) { return TA_ERR_ORDER; }
