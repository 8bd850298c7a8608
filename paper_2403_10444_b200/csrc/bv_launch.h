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

// Cluster kernel for 16-byte aligned rows (both algorithms): several clusters per SM,
// rows re-read from L2 for the residual sweep.
int cluster_max_clusters(int algo, int dtype, int cluster);
cudaError_t launch_cluster(const Params& prm, int algo, int dtype, int cluster, int nclusters, cudaStream_t stream);

// Resident kernel (Block Verification only, 128-bit path): a thread holds up to `nk`
// vectors per row, nk in {2, 4, 8}.
int resident_vectors_per_cta(int nk);
int resident_max_clusters(int dtype, int nk, int cluster);
cudaError_t launch_resident(const Params& prm, int dtype, int nk, int cluster, int nclusters,
                            cudaStream_t stream);

}  // namespace bv
