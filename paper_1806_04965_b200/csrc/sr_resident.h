// Resident engine: the frame update of small networks with every node state kept in shared memory.
#pragma once
#include <cuda_runtime.h>

#include "sr_internal.h"

sr_status sr_rs_plan(sr_graph* g, size_t& offset);            // decides eligibility, reserves workspace regions
sr_status sr_rs_bind(sr_graph* g);                            // uploads the per-rank tables
sr_status sr_rs_set_weights(sr_graph* g, int edge, const float* w_eff /* host; conv [C_out][k][k][C_in], dense [C_out][K] */);
bool sr_rs_available(const sr_graph* g);
// Queues ONE kernel that performs the T frame updates described by `init` and leaves the frame control block in
// global memory as T single-frame updates would (frame counters advanced by T).
sr_status sr_rs_launch(sr_graph* g, int T, const SrFrameCtl& init, cudaStream_t s);
void sr_rs_describe(const sr_graph* g, int* cluster_size, int* warps, int* smem_bytes, int* heads_on_chip);
sr_status sr_rs_timing(sr_graph* g, double* ms, long long* launches);   // event-timed resident launches since the last call
void sr_rs_destroy(sr_graph* g);
