// Host-side launch interface between the C-ABI layer and the kernels.
#pragma once

#include <cuda_runtime.h>

#include "bv_device.cuh"

namespace bv {

// Most clusters of `cluster` CTAs of the streaming kernel that can be resident at once
// on the current device (0 if that cluster size cannot be scheduled).
int stream_max_clusters(int algo, int dtype, bool vec, int cluster);

// Enqueue the streaming kernel: `nclusters` clusters of `cluster` CTAs each.
cudaError_t launch_stream(const Params& prm, int algo, int dtype, bool vec, int cluster,
                          int nclusters, cudaStream_t stream);

}  // namespace bv
