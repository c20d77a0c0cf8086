// Launch wrappers shared between the API layer and the kernel files.
#pragma once
#include <cuda_runtime.h>

#include "sr_internal.h"

void sr_launch_direct_group(const sr_graph* g, int group, int t_off, cudaStream_t s);
void sr_launch_input(const sr_graph* g, const int* input_nodes_dev, int t_off, cudaStream_t s);
void sr_launch_set_ctl(const sr_graph* g, const SrFrameCtl& v, cudaStream_t s);
void sr_launch_advance(const sr_graph* g, int n, cudaStream_t s);
int sr_direct_conv_pixels_per_block();
int sr_direct_dense_outputs_per_block();
int sr_direct_dense_samples_per_block();
int sr_direct_head_outputs_per_block();
int sr_direct_head_max_channels();
