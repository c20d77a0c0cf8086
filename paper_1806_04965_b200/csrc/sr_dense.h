// Dense resident engine: the frame update of small all-dense fp32 networks with weights and states kept in the
// shared memory of one thread-block cluster.
#pragma once
#include <cuda_runtime.h>

#include "sr_internal.h"

sr_status sr_dn_plan(sr_graph* g, size_t& offset);            // decides eligibility, reserves workspace regions
sr_status sr_dn_bind(sr_graph* g);
sr_status sr_dn_set_weights(sr_graph* g, int edge, const float* w /* host, [C_out][K] */);
bool sr_dn_available(const sr_graph* g);
// Queues ONE kernel that performs the T frame updates described by `init` and leaves the frame control block and
// the state buffers in global memory as T single-frame updates would.
sr_status sr_dn_launch(sr_graph* g, int T, const SrFrameCtl& init, cudaStream_t s);
void sr_dn_describe(const sr_graph* g, int* cluster_size, int* smem_bytes);
sr_status sr_dn_timing(sr_graph* g, double* ms, long long* launches);
void sr_dn_destroy(sr_graph* g);
