// Host-side launch interface between the C-ABI layer and the kernels.
#pragma once

#include <cuda_runtime.h>

#include "bv_device.cuh"

namespace bv {

// Shared by the files that hold entry points: argument checks of the verification calls, the
// thread's record of the last failing CUDA call (returns BV_ERR_CUDA) and of the launches of its last call.
int check_verify_args(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                      int V, int dtype, float T, const int32_t* ot, const int32_t* ol);
int note_cuda_error(cudaError_t e);
void note_launches(int n);

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
// when the kernel starts, and the kernel leaves them zero when it ends.
struct RowZ { double MP, ZP, MQ, ZQ; };   // row (or chunk) references and sums of 2^{z k - M}
struct FlowScratch {
    unsigned* counters;   // ticket counter of the sweep-1 items, rows queued for their second sweep, pieces of
                          // queued rows handed out, blocks finished (one 128-byte line each)
    unsigned* row_cnt;    // [B (gamma+1)] sweep-1 chunks finished per row
    unsigned* s2_cnt;     // [B (gamma+1)] sweep-2 chunks finished per position
    unsigned* cand_cnt;   // [B] positions with a candidate
    unsigned* rows_in;    // [B] rows 0 .. gamma-1 whose normalisers are published
    unsigned* bad;        // [B] data fault seen (Token Verification: in the last target row)
    // Token Verification (Algorithm 1): bit r of tv_done = the acceptance test that row r feeds has been made, of
    // tv_acc = it passed, of tv_badrows = row r holds a data fault; tv_front = rows beyond the first tv_spec
    // whose first sweep has been asked for; tv_decided = tau is known; tv_tau = tau
    unsigned long long* tv_acc;
    unsigned long long* tv_done;
    unsigned long long* tv_badrows;
    unsigned* tv_front;
    unsigned* tv_decided;
    int* tv_tau;
    int tv;               // the launch runs Algorithm 1
    int tv_spec;          // rows 0 .. tv_spec-1 of every block are swept from the start, the others once all before them passed
    int tv_ahead;         // rows asked for beyond the last test that passed (1: none is read in vain)
    unsigned* rel;        // [B (gamma+1)] what becomes of the position's second sweep (0 until the block is folded)
    unsigned* s2q;        // [B (gamma+1)] queue of rows whose second sweep has been started (row index + 1)
    unsigned* lq;         // [B] queue of last target rows whose first sweep has been asked for (row index + 1)
    RowZ* part;           // [B (gamma+1) part_stride]
    RowZ* rowZ;           // [B (gamma+1)]
    double* pchain;       // [B (gamma+2)]
    float* cscale;        // [B (gamma+1)] p_r Z_Q / Z_P
    double* ratio;        // [B (gamma+1)] P_r(X_{r+1}) / Q_r(X_{r+1})
    double* zratio;       // [B (gamma+1)] Z_Q / Z_P
    double* seg_tot;      // [B (gamma+1) segs] per-segment sums, in double: they decide sampled tokens
    double* S;            // [B (gamma+1)]
    int* cand;            // [B (gamma+1)]
    int nch;              // chunks per row in the first sweep of rows 0 .. gamma-1 (1 .. kFlowMaxChunks)
    int part_stride;      // chunk results kept per row: max(nch, nch_late)
    int nch_late;         // chunks of a last target row, whose first sweep is asked for on demand
    int fine_from;        // Block Verification: rows 0 .. gamma-1 of the blocks from this one on are cut into nch_late chunks (B: none)
    int np;               // pieces per row in the second sweep (1 .. kFlowMaxChunks)
    unsigned total_s1;    // first-sweep tickets: fine_from gamma nch + (B - fine_from) gamma nch_late
    unsigned zero_words;  // 32-bit words at the start of the scratch area (from `counters` on) that start and end at zero
    int depth;            // flow kernel: descriptors a CTA may have handed to its workers and not yet seen swept
    int segs;             // residual totals kept per row
    int tail_mode;        // 0: a block's candidates are started all at once when the first-sweep tickets have run out;
                          // 1: always (a launch without first sweeps that would not fill the GPU); 2: never
    int keep_l2;          // tuning switch: first-sweep loads leave their lines at normal priority in L2 (default: evicted first)
};
constexpr int kFlowMaxChunks = 32;
// How a launch is cut into work items (flow_plan): chunks per row in the first sweep, chunks of a
// last target row (swept on demand), pieces per row in the second sweep.
struct FlowPlan {
    int nch, nch_late, np;
    int tv_spec;          // Token Verification: rows of every block swept from the start (0: Block Verification)
    int tv_ahead;         // Token Verification: rows asked for beyond the last test that passed
    bool probs;           // the rows hold probabilities: no first sweep
    int tail_mode;        // see FlowScratch
    int fine_from;        // see FlowScratch
    int part_stride() const { return nch > nch_late ? nch : nch_late; }
};
// units: 16-byte vectors per row; pair_items: false when the first sweep streams one row per item
// (supplied draft normalisers); chunks / pieces > 0 force the chunk count / the piece count.
FlowPlan flow_plan(long long units, int B, int gamma, long long nctas, bool pair_items, int chunks, int pieces, bool token_verify = false, bool probs = false);
size_t flow_scratch_bytes(int B, int gamma, const FlowPlan& plan, size_t* zero_bytes);
void flow_scratch_layout(void* base, int B, int gamma, const FlowPlan& plan, FlowScratch* fl);
int flow_max_ctas_per_sm(int dtype);
cudaError_t launch_flow(const Params& prm, const FlowScratch& fl, int dtype, int nctas, cudaStream_t stream);

// Small-batch kernel (bv_small.cu): a cooperative launch of one CTA per SM with two grid-wide barriers.
constexpr int kSmallMaxB = 32;        // sequences
constexpr int kSmallMaxChunks = 32;   // chunks per row in its first phase
struct SmallScratch {
    unsigned* barrier;    // [0]: arrivals at the grid barriers, [16]: CTAs that have left; both zero between launches
    double2* part;        // [B (2 gamma + 1)][nch] {reference, sum} of every chunk
    double* seg;          // [B (gamma + 1)][np * 16] per-segment sums of the residual terms
    int nch, np;
};
struct SmallPlan { int nch, np; };
bool small_fits(int B, int gamma);
SmallPlan small_plan(long long units, int B, int gamma, int nctas);
size_t small_scratch_bytes(int B, int gamma, const SmallPlan& pl);
void small_scratch_layout(void* base, unsigned* barrier, int B, int gamma, const SmallPlan& pl, SmallScratch* sc);
int small_max_ctas(int dtype, int sm_count);
cudaError_t launch_small(const Params& prm, const SmallScratch& sc, int dtype, int nctas, cudaStream_t stream);

}  // namespace bv
