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

// Flow kernel (Block Verification, 128-bit path): independent work items with dependency
// counters in a scratch area of flow_scratch_bytes(); its first *zero_bytes must be zero
// when the kernel starts.
struct RowZ { double MP, ZP, MQ, ZQ; };   // row (or chunk) references and sums of 2^{z k - M}
struct FlowScratch {
    unsigned* counters;   // ticket counter of the sweep-1 items, rows queued for their second sweep, pieces of
                          // queued rows handed out, blocks finished (one 128-byte line each)
    unsigned* row_cnt;    // [B (gamma+1)] sweep-1 chunks finished per row
    unsigned* row_done;   // [B (gamma+1)] row normalisers published
    unsigned* s2_cnt;     // [B (gamma+1)] sweep-2 chunks finished per position
    unsigned* cand_cnt;   // [B] positions with a candidate
    unsigned* chain;      // [B] rows folded into the recursion
    unsigned* lock;       // [B]
    unsigned* bad;        // [B] data fault seen
    unsigned* rel;        // [B (gamma+1)] row folded into the recursion, and what becomes of its second sweep
    unsigned* s2q;        // [B (gamma+1)] queue of rows whose second sweep has been started (row index + 1)
    unsigned* lq;         // [B] queue of last target rows whose first sweep has been asked for (row index + 1)
    RowZ* part;           // [B (gamma+1) nch]
    RowZ* rowZ;           // [B (gamma+1)]
    double* pchain;       // [B (gamma+2)]
    float* cscale;        // [B (gamma+1)] p_r Z_Q / Z_P
    double* ratio;        // [B (gamma+1)] P_r(X_{r+1}) / Q_r(X_{r+1})
    double* zratio;       // [B (gamma+1)] Z_Q / Z_P
    float* seg_tot;       // [B (gamma+1) segs]
    double* S;            // [B (gamma+1)]
    int* cand;            // [B (gamma+1)]
    int nch;              // chunks per row in the first sweep (1 .. kFlowMaxChunks)
    int np;               // pieces per row in the second sweep (1 .. kFlowMaxChunks)
    int depth;            // flow kernel: descriptors a CTA may have published and not yet post-processed (2 or 3)
    int segs;             // residual totals kept per row
};
constexpr int kFlowMaxChunks = 32;
size_t flow_scratch_bytes(int B, int gamma, int nch, int np, size_t* zero_bytes);
void flow_scratch_layout(void* base, int B, int gamma, int nch, int np, FlowScratch* fl);
int flow_pick_pieces(long long units);
int flow_max_ctas_per_sm(int dtype);
int flow_pick_chunks(long long units, int B, int gamma, long long nctas);
cudaError_t launch_flow(const Params& prm, const FlowScratch& fl, int dtype, int nctas, cudaStream_t stream);


// Resident kernel (Block Verification only, 128-bit path): a thread holds up to `nk`
// vectors per row, nk in {2, 4, 8}.
int resident_vectors_per_cta(int nk);
int resident_max_clusters(int dtype, int nk, int cluster);
cudaError_t launch_resident(const Params& prm, int dtype, int nk, int cluster, int nclusters,
                            cudaStream_t stream);

}  // namespace bv
