// Placeholder until the tcgen05 engine lands: no node is selected for the tensor cores.
#include "sr_tc.h"

void sr_tc_select_nodes(sr_graph*) {}
sr_status sr_tc_plan(sr_graph*, size_t&) { return SR_OK; }
sr_status sr_tc_bind(sr_graph*) { return SR_OK; }
sr_status sr_tc_set_weights(sr_graph*, int, const float*) { return SR_ERR_UNSUPPORTED; }
int sr_tc_stage_inputs(sr_graph*, int, cudaStream_t) { return 0; }
int sr_tc_launch_group(sr_graph*, int, int, cudaStream_t) { return 0; }
int sr_tc_after_state_change(sr_graph*, cudaStream_t) { return 0; }
void sr_tc_destroy(sr_graph*) {}
