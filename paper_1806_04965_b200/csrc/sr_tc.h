// Tensor-core engine (tcgen05 implicit GEMM) as the API layer sees it.
#pragma once
#include <cuda_runtime.h>

#include "sr_internal.h"

void sr_tc_select_nodes(sr_graph* g);                         // sets SrHostNode::use_tc
sr_status sr_tc_plan(sr_graph* g, size_t& offset);            // reserves workspace regions
sr_status sr_tc_bind(sr_graph* g);                            // uploads tile tables and tensor maps
sr_status sr_tc_set_weights(sr_graph* g, int edge, const float* w_eff /* [C_out][k][k][C_in], host */);
int sr_tc_stage_inputs(sr_graph* g, int t_off, cudaStream_t s);          // returns launches queued
int sr_tc_launch_group(sr_graph* g, int group, int t_off, cudaStream_t s);
bool sr_tc_group_has_work(const sr_graph* g, int group);
sr_status sr_tc_timing(sr_graph* g, double* ms, long long* launches);
int sr_tc_after_state_change(sr_graph* g, cudaStream_t s);    // re-stage frame-t inputs after reset / set_state
void sr_tc_destroy(sr_graph* g);
