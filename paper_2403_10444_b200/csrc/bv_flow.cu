// Block Verification (Algorithm 2; also Algorithm 4, Algorithm 1 and the variants with supplied
// draft normalisers or with probabilities as inputs) as a dependency-driven flow of independent work items.
//
// Persistent CTAs of 14 worker warps that only stream, one publisher warp that finds the next items
// and hands their descriptors to the workers, and three post warps that do what follows the sweep
// of an item.  Items come from three sources, in this order of preference:
//
//   sweep-2 piece (b, r, piece)  a piece of a row pair whose second sweep has been asked for:
//       leaves sum max(p_r P_r(x) - Q_r(x), 0) per warp segment (Eq. "pacc_block").  The warp
//       that completes a position adds the segments to S_r, locates u * S_r, rescans that one
//       segment in index order for the candidate Y_r (Eq. "pres-block"), and then either finds
//       the position selected or asks for the next lower candidate; the warp that completes the
//       block forms h_i, selects tau and emits X^tau, Y_tau.
//   late sweep-1 chunk  of a row whose first sweep is asked for on demand: a last target row
//       P_gamma, which is read only if position gamma can be the selected one (its sample is drawn
//       from that one sweep); under Algorithm 1 a row whose tests before it have all passed.
//   sweep-1 item (b, r < gamma, chunk)  by ticket: streams the chunk of both rows from HBM and
//       leaves the chunk's {reference, sum 2^{z k - M}} pair for each row in scratch.  The warp
//       that completes a row combines the chunks into the row normalisers; the warp that
//       completes the last row of a block folds it: the prefix recursion
//       p_{r+1} = min(p_r P_r(X)/Q_r(X), 1) (Eq. "def_as") and which positions are candidates.
//
// A second sweep runs only where the outcome can depend on it: S_r <= p_r gives h_r <= p_r, so
// a position with eta_r > p_r can never be selected; the others are swept from the top down
// until one passes its test (bv_flow_common.cuh).  With diagnostic outputs every position is
// swept.
//
// Every hand-over is a counter in global memory whose last increment elects the warp that goes on
// (no locks).  No CTA ever waits for another one while it holds work that others need: sweep-1
// items have no prerequisites, and a CTA polls (bounded) only when nothing is left to start.  So
// CTAs need not be co-resident.
#include "bv_flow_common.cuh"

namespace bv {

constexpr int kFThreads = 448;
constexpr int kFWarps = kFThreads / 32;

// vectors [u0, u1) of `units` that part `ch` out of `nparts` covers
__device__ __forceinline__ void item_range(int units, int nparts, int ch, int& u0, int& u1) {
    u0 = static_cast<int>(static_cast<long long>(units) * ch / nparts);
    u1 = static_cast<int>(static_cast<long long>(units) * (ch + 1) / nparts);
}
// Vectors [w0, w1) of the part [u0, u1) that worker `warp` takes (a part is far below 2^27 vectors).
// The shares are cut to the vector, not to whole ring steps of 32 vectors: with every warp's stream
// aligned to 512 bytes the kernel was measured 9 % slower (the streams of a CTA then advance through
// the same memory channels together), which costs more than the short last step of each share.
__device__ __forceinline__ void warp_range(int u0, int u1, int warp, int& w0, int& w1) {
    const unsigned n = static_cast<unsigned>(u1 - u0);
    w0 = u0 + static_cast<int>(n * static_cast<unsigned>(warp) / kFWarps);
    w1 = u0 + static_cast<int>(n * static_cast<unsigned>(warp + 1) / kFWarps);
}
__device__ __forceinline__ void chunk_range(const FlowCtx& cx, int nparts, int ch, int warp, int& w0, int& w1) {
    int u0, u1;
    item_range(cx.units, nparts, ch, u0, u1);
    warp_range(u0, u1, warp, w0, w1);
}


// Ring of a worker thread: kFSlots steps of lookahead, each of two 16-byte cells (A, B).  A step of
// an item with a draft row holds one vector of P and the same vector of Q; without a draft row it
// holds two consecutive vectors of P.  The ring is not drained between items: while a warp works
// through the last steps of one item the loads of the next one are already in flight.
constexpr int kFSlots = 3;
constexpr int kFDepth = 2 * kFSlots;
constexpr int kFDesc = 8;      // descriptors a CTA can hold: being swept, queued behind, or waiting for their post warp
constexpr int kFPost = 3;      // post warps: what follows the sweep of item n is done by post warp n mod kFPost
constexpr int kFAllThreads = kFThreads + 32 * (1 + kFPost);   // worker warps + the publisher + the post warps

// One work item as the publisher hands it to the workers.
struct FlowDesc {
    int kind;                   // kExit, kSweep1, kSweep2
    int ri, ch;                 // row index b (gamma+1) + r, chunk
    int u0, u1;                 // the chunk's vectors [u0, u1) of the row
    int have_q;
    const char* rowP;
    const char* rowQ;
    float cp, nMP, nMQ;         // sweep 2: p_r Z_Q / Z_P and minus the row references
};


struct FlowShared {
    FlowDesc desc[kFDesc];
    unsigned long long full[kFDesc];    // the publisher has filled desc[i]
    unsigned long long done[kFDesc];    // all worker warps have left their partials of desc[i]
    float part_M[kFDesc][2][kFWarps];   // sweep 1: references of P and Q per worker warp
    float part_s[kFDesc][kFWarps];      // sweep 1: sums of the draft row
    double part_d[kFDesc][kFWarps];     // sweep 1: sums of the target row; sweep 2: the residual totals (they decide sampled
                                        // tokens, so a last target row and every second sweep accumulate them in double)
    // a finished item is moved here by its post warp, so that its descriptor slot is free again
    // before anything is asked of global memory
    unsigned long long freeb[kFDesc];   // the post warp has moved the item of desc[i] out
    FlowDesc sdesc[kFPost];
    float stage_M[kFPost][2][kFWarps];
    float stage_s[kFPost][kFWarps];
    double stage_d[kFPost][kFWarps];
    unsigned posted;                    // items whose post-processing is complete
};

// ---- post warp: Y ~ P_gamma from the first sweep of the last target row ----
// The sample needs the row's normaliser and a second look at one segment only: the segment
// {reference, sum} pairs of all chunks are in scratch, so u * Z is located among their prefix sums
// (fp32, index order) and that one segment is rescanned.  No second sweep of the row.
template <int DT>
__device__ void f_draw_from_sweep1(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int ri, int lane) {
    const int g = cx.g, b = ri / (g + 1);
    const int nseg = fl.nch_late * kFWarps;                  // <= 128: four per lane
    const double* pairs = fl.seg_tot + static_cast<size_t>(ri) * fl.segs;
    float m[4];
    double w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i = 4 * lane + j;
        m[j] = i < nseg ? static_cast<float>(__ldcg(&pairs[2 * i])) : kNoRef;
        w[j] = i < nseg ? __ldcg(&pairs[2 * i + 1]) : 0.0;
    }
    const float Mrow = warp_max(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])));
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] *= static_cast<double>(ref_scale(m[j], Mrow));
    // (fp64 sums of the segment totals, as for the residual samples)
    const double d1 = w[0], d2 = d1 + w[1], d3 = d2 + w[2], d4 = d3 + w[3];
    double inc = d4;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double o = shfl_up_d(inc, off);
        if (lane >= off) inc += o;
    }
    const double total = shfl_d(inc, 31);
    int found = -1;
    if (Mrow > kNoRef && Mrow < INFINITY && total > 0.0 && total < static_cast<double>(INFINITY)) {
        const double t = static_cast<double>(prm.uni[static_cast<size_t>(b) * (g + 2) + g + 1]) * total;
        double exc = shfl_up_d(inc, 1);
        if (lane == 0) exc = 0.0;
        const double p0 = exc, p1 = exc + d1, p2 = exc + d2, p3 = exc + d3, p4 = exc + d4;
        // first non-empty segment whose inclusive prefix exceeds t, else the last non-empty one
        const bool h1 = p1 > t && w[0] > 0.0, h2 = p2 > t && w[1] > 0.0;
        const bool h3 = p3 > t && w[2] > 0.0, h4 = p4 > t && w[3] > 0.0;
        const unsigned hit = __ballot_sync(0xffffffffu, h1 || h2 || h3 || h4);
        const unsigned nz = __ballot_sync(0xffffffffu, d4 > 0.0);
        int e = 3; double bef = p3; int src;
        if (hit) {
            src = __ffs(hit) - 1;
            if (h1) { e = 0; bef = p0; } else if (h2) { e = 1; bef = p1; } else if (h3) { e = 2; bef = p2; }
        } else {
            src = 31 - __clz(nz);
            e = 0; bef = p0;
            if (w[3] > 0.0) { e = 3; bef = p3; } else if (w[2] > 0.0) { e = 2; bef = p2; }
            else if (w[1] > 0.0) { e = 1; bef = p1; }
        }
        const int sel = __shfl_sync(0xffffffffu, 4 * lane + e, src);
        const double before = shfl_d(bef, src);
        int s0, s1;
        chunk_range(cx, fl.nch_late, sel / kFWarps, sel % kFWarps, s0, s1);
        const char* rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
        found = f_rescan<DT>(rowP, nullptr, s0, s1, lane, cx.kf, 1.f, -Mrow, 0.f, t - before);
    }
    if (lane == 0) {
        fl.cand[ri] = found;
        __threadfence();
    }
    __syncwarp();
}

// ---- post warp: what follows the sweep of an item, in three steps:
//   store     the item's result goes to scratch;
//   (one __threadfence, then one atomic on the counter of the item's row or position)
//   complete  for the item that was the last of its row or position. ----
template <int DT>
__device__ void f_store_sweep1(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, FlowShared& sh, int j,
                               int ri, int ch, int lane) {
    // combine the worker warps of this chunk in fp64
    const float mP = lane < kFWarps ? sh.stage_M[j][0][lane] : kNoRef;
    const float mQ = lane < kFWarps ? sh.stage_M[j][1][lane] : kNoRef;
    const float MPc = warp_max(mP), MQc = warp_max(mQ);
    double zP = lane < kFWarps ? sh.stage_d[j][lane] * ref_scale(mP, MPc) : 0.0;
    double zQ = lane < kFWarps ? static_cast<double>(sh.stage_s[j][lane]) * ref_scale(mQ, MQc) : 0.0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { zP += shfl_xor_d(zP, off); zQ += shfl_xor_d(zQ, off); }
    // A last target row is swept for one purpose only: the sample from P_gamma.  Its warps' pairs
    // {reference, sum} are kept, so that the token can be drawn from this one sweep.
    if (ri % (cx.g + 1) == cx.g && f_draws_in_sweep1(prm, fl.nch_late)) {
        double* pairs = fl.seg_tot + static_cast<size_t>(ri) * fl.segs + static_cast<size_t>(ch) * kFWarps * 2;
        if (lane < kFWarps) { pairs[2 * lane] = mP; pairs[2 * lane + 1] = sh.stage_d[j][lane]; }
    }
    if (lane == 0) {
        RowZ z; z.MP = MPc; z.ZP = zP; z.MQ = MQc; z.ZQ = zQ;
        fl.part[static_cast<size_t>(ri) * fl.part_stride + ch] = z;
    }
}
template <int DT>
__device__ void f_complete_sweep1(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int ri, int lane) {
    __threadfence();
    const int g = cx.g, b = ri / (g + 1), r = ri % (g + 1);
    f_row_complete<DT>(prm, fl, cx, b, r, lane);
    if (fl.tv) {
        if (r < g) { f_tv_row_done<DT>(prm, fl, cx, b, r, lane); return; }
        // the last target row of a block whose tests have all passed: Y ~ P_gamma
        if (f_draws_in_sweep1(prm, fl.nch_late)) {
            f_draw_from_sweep1<DT>(prm, fl, cx, ri, lane);
            f_tv_finalize(prm, fl, b, g, lane);
        } else {
            if (lane == 0) {
                const unsigned slot = atomicAdd(&fl.counters[kCtrQueued], 1u);
                atomicExch(&fl.s2q[slot], static_cast<unsigned>(ri) + 1u);
            }
            __syncwarp();
        }
        return;
    }
    if (r < g) {
        // the warp that publishes the last of a block's rows 0 .. gamma-1 folds the block
        unsigned n = 0;
        if (lane == 0) n = atomicAdd(&fl.rows_in[b], 1u);
        n = __shfl_sync(0xffffffffu, n, 0);
        if (n == static_cast<unsigned>(g) - 1u) f_fold_block<DT>(prm, fl, cx, b, lane);
    } else if (f_draws_in_sweep1(prm, fl.nch_late)) {
        // The last target row was swept because position gamma can be selected, and its token is
        // drawn from that very sweep: the position is complete.  It is the highest candidate, so
        // either it is the selected one (lower candidates are dropped) or the next lower one is started.
        f_draw_from_sweep1<DT>(prm, fl, cx, ri, lane);
        f_position_done(prm, fl, b, g, lane);
    } else {
        // with diagnostics the sample from P_gamma comes from a second sweep of the row, like any other
        if (lane == 0) {
            atomicExch(&fl.rel[ri], kRelSweep);
            __threadfence();
            const unsigned slot = atomicAdd(&fl.counters[kCtrQueued], 1u);
            atomicExch(&fl.s2q[slot], static_cast<unsigned>(ri) + 1u);
        }
        __syncwarp();
    }
}

__device__ __forceinline__ void f_store_sweep2(const FlowScratch& fl, FlowShared& sh, int j, int ri, int ch, int lane) {
    double* segs = fl.seg_tot + static_cast<size_t>(ri) * fl.segs;
    if (lane < kFWarps) segs[ch * kFWarps + lane] = sh.stage_d[j][lane];
}
template <int DT, bool PROBS>
__device__ void f_complete_sweep2(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, const FlowDesc& d, int lane) {
    const int np = fl.np;
    const double* segs = fl.seg_tot + static_cast<size_t>(d.ri) * fl.segs;
    f_position_complete<DT, PROBS>(prm, fl, cx, d.ri, d.have_q != 0, d.rowP, d.rowQ, d.cp, d.nMP, d.nMQ, np * kFWarps, segs, lane,
                            [&](int sel, int& s0, int& s1) { chunk_range(cx, np, sel / kFWarps, sel % kFWarps, s0, s1); });
}

// ---- worker warps: the arithmetic of one ring step ----
// First sweep, one vector of each row: running sums of 2^{z k - M} against the warp's integer
// references, which are raised when a vector's terms show a logit above them.
template <int EPV>
__device__ __forceinline__ void f_step_sweep1_pair(const float (&vp)[EPV], const float (&vq)[EPV], float kf,
                                                   float& MPw, float& sP, float& MQw, float& sQ) {
    float vsP = f_exp_sum<EPV>(vp, kf, -MPw);
    float vsQ = f_exp_sum<EPV>(vq, kf, -MQw);
    if (__any_sync(0xffffffffu, fmaxf(vsP, vsQ) > kRaiseBound)) {   // a logit above a reference
        if (__any_sync(0xffffffffu, vsP > kRaiseBound)) {
            const float y = rintf(warp_max(vec_max<EPV>(vp)) * kf);
            if (y > MPw) { sP *= ref_scale(MPw, y); MPw = y; }
            vsP = f_exp_sum<EPV>(vp, kf, -MPw);
        }
        if (__any_sync(0xffffffffu, vsQ > kRaiseBound)) {
            const float y = rintf(warp_max(vec_max<EPV>(vq)) * kf);
            if (y > MQw) { sQ *= ref_scale(MQw, y); MQw = y; }
            vsQ = f_exp_sum<EPV>(vq, kf, -MQw);
        }
    }
    sP += vsP;
    sQ += vsQ;
}
// First sweep, two consecutive vectors of one row; the running sum in double.
template <int EPV>
__device__ __forceinline__ void f_step_sweep1_single(const float (&va)[EPV], const float (&vb)[EPV], float kf,
                                                     float& MPw, double& sP) {
    float vsA = f_exp_sum<EPV>(va, kf, -MPw);
    float vsB = f_exp_sum<EPV>(vb, kf, -MPw);
    if (__any_sync(0xffffffffu, fmaxf(vsA, vsB) > kRaiseBound)) {
        const float y = rintf(warp_max(fmaxf(vec_max<EPV>(va), vec_max<EPV>(vb))) * kf);
        if (y > MPw) { sP *= static_cast<double>(ref_scale(MPw, y)); MPw = y; }
        vsA = f_exp_sum<EPV>(va, kf, -MPw);
        vsB = f_exp_sum<EPV>(vb, kf, -MPw);
    }
    sP += static_cast<double>(vsA);
    sP += static_cast<double>(vsB);
}

// PROBS: the rows hold probabilities (used as stored) instead of logits: no row has a first sweep,
// the blocks are folded by the post warps when the launch starts, and the residual terms are formed
// from the stored numbers.
template <int DT, bool PROBS>
__global__ void __launch_bounds__(kFAllThreads, 2) verify_flow_kernel(const Params prm, const FlowScratch fl) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ FlowShared sh;
    // Each worker thread streams its own vectors through a private ring of 16-byte cells filled
    // by cp.async, so loads run kFSlots steps ahead of the arithmetic without costing registers.
    extern __shared__ __align__(16) unsigned char dyn[];

    // polls after which a bounded wait gives up
    const uint32_t lim_spin = prm.wait_limit ? prm.wait_limit : (1u << 24);
    const uint32_t lim_nap = prm.wait_limit ? prm.wait_limit : (1u << 22);
    FlowCtx cx;
    cx.g = prm.gamma; cx.V = prm.V; cx.B = prm.B; cx.units = prm.V / EPV;
    cx.row_bytes = static_cast<size_t>(prm.V) * ESZ; cx.kf = prm.kf; cx.kd = prm.kd;
    const int g = cx.g;
    const float kf = cx.kf;

    if (tid == 0) {
        for (int i = 0; i < kFDesc; ++i) {
            sh.desc[i].kind = kExit;      // what a wait that gives up would find
            mbar_init(smem_u32(&sh.full[i]), 1);
            mbar_init(smem_u32(&sh.done[i]), kFWarps);
            mbar_init(smem_u32(&sh.freeb[i]), 1);
        }
        sh.posted = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp > kFWarps) {
        // =============================== post warps ===============================
        // What follows the sweep of item n is done by post warp n mod kFPost: the item's partials and
        // descriptor are moved to the warp's staging area (the slot is free again), the result goes
        // to scratch, and the row's or position's counter tells whether this item was its last one.
        // Every step here is a round trip to global memory of a few microseconds on a busy GPU; three
        // warps working on different items keep up with items of a few microseconds each.
        const int k = warp - kFWarps - 1;
        if (PROBS) {
            // every block's ratios are read off its rows and the block is folded (Algorithm 1: decided)
            for (int b = static_cast<int>(blockIdx.x) * kFPost + k; b < cx.B; b += static_cast<int>(gridDim.x) * kFPost)
                f_probs_start<DT>(prm, fl, cx, b, lane);
        }
        for (int n = k;; n += kFPost) {
            const int slot = n % kFDesc;
            const uint32_t par = static_cast<uint32_t>(n / kFDesc) & 1u;
            if (!mbar_wait_relaxed(smem_u32(&sh.full[slot]), par, prm.status, 200, lim_nap)) break;
            if (sh.desc[slot].kind == kExit) break;
            if (!mbar_wait_relaxed(smem_u32(&sh.done[slot]), par, prm.status, 200, lim_nap)) break;
            if (lane == 0) sh.sdesc[k] = sh.desc[slot];
            if (lane < kFWarps) {
                sh.stage_M[k][0][lane] = sh.part_M[slot][0][lane]; sh.stage_M[k][1][lane] = sh.part_M[slot][1][lane];
                sh.stage_s[k][lane] = sh.part_s[slot][lane]; sh.stage_d[k][lane] = sh.part_d[slot][lane];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.freeb[slot]));
            const FlowDesc d = sh.sdesc[k];
            if (!PROBS && d.kind == kSweep1) f_store_sweep1<DT>(prm, fl, cx, sh, k, d.ri, d.ch, lane);
            else f_store_sweep2(fl, sh, k, d.ri, d.ch, lane);
            __threadfence();
            __syncwarp();
            int last = 0;
            if (lane == 0) {
                if (!PROBS && d.kind == kSweep1) last = atomicAdd(&fl.row_cnt[d.ri], 1u) == static_cast<unsigned>(f_nch_row(fl, d.ri / (g + 1), d.ri % (g + 1), g)) - 1u;
                else last = atomicAdd(&fl.s2_cnt[d.ri], 1u) == static_cast<unsigned>(fl.np) - 1u;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                if (!PROBS && d.kind == kSweep1) f_complete_sweep1<DT>(prm, fl, cx, d.ri, lane);
                else f_complete_sweep2<DT, PROBS>(prm, fl, cx, d, lane);
            }
            __syncwarp();
            if (lane == 0) atomicAdd(&sh.posted, 1u);
        }
        return;
    }
    if (warp == kFWarps) {
        // =============================== publisher ===============================
        // takes tickets, waits for what a sweep-2 item needs and hands descriptors to the workers.
        // What it asks of global memory is arranged so that the round trips overlap: the four queue
        // counters are read after every descriptor for the next one, and tickets of first-sweep items
        // are drawn ahead of their use.
        // tickets cover the rows that every block needs: target and draft rows 0 .. gamma-1
        const unsigned total_s1 = fl.total_s1;
        // Tickets are drawn several at a time (one atomic) and ahead of their use, so that the round
        // trip is over by the time a descriptor slot is free.
        unsigned tk_raw = 0, tk_lo = 0;   // (lane 0) answer of the last draw; next ticket on hand (all lanes)
        int tk_cnt = 0;                   // tickets on hand
        bool tk_pending = false;          // tk_raw has not been looked at yet
        auto draw_tickets = [&](int k) {
            if (lane == 0) tk_raw = atomicAdd(&fl.counters[kCtrTicket], static_cast<unsigned>(k));
            tk_cnt = k;
            tk_pending = true;
        };
        auto next_ticket = [&]() -> unsigned {
            if (tk_pending) { tk_lo = __shfl_sync(0xffffffffu, tk_raw, 0); tk_pending = false; }
            --tk_cnt;
            return tk_lo++;
        };
        // the first-sweep item of ticket t
        auto sweep1_desc = [&](unsigned t, FlowDesc& d) {
            // (the blocks from fine_from on are cut into nch_late chunks per row: Block Verification only)
            const unsigned t_coarse = static_cast<unsigned>(fl.fine_from) * g * fl.nch;
            const bool fine = !fl.tv && t >= t_coarse;
            const int nch = fine ? fl.nch_late : fl.nch;
            const unsigned tt = fine ? t - t_coarse : t;
            const int ch = static_cast<int>(tt % nch);
            // Block Verification goes block by block (a block's rows are wanted together); Algorithm 1
            // row by row over all blocks (a block's next row matters only if the one before passed)
            const int r = fl.tv ? static_cast<int>(tt / nch) / cx.B : static_cast<int>(tt / nch) % g;
            const int b = fl.tv ? static_cast<int>(tt / nch) % cx.B : (fine ? fl.fine_from : 0) + static_cast<int>(tt / nch) / g;
            const int ri = b * (g + 1) + r;
            // (with supplied draft normalisers the first sweep has nothing to learn from the draft row)
            d.kind = kSweep1; d.ri = ri; d.ch = ch; d.have_q = prm.lse_d == nullptr;
            item_range(cx.units, nch, ch, d.u0, d.u1);
            d.rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
            d.rowQ = d.have_q ? static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes
                              : nullptr;
            d.cp = 1.f; d.nMP = 0.f; d.nMQ = 0.f;
        };
        // Rows whose second sweep has been started stand in a queue, each cut into np pieces.  A
        // piece is claimed by a ticket from the queue's head counter, drawn only while the head is
        // seen behind the tail; a ticket that still runs ahead of the tail (several CTAs drew at
        // once, or the counters were read a while ago) is kept until its row arrives.  -1: no piece
        // right now.  Last target rows whose first sweep has been asked for stand in a queue of their
        // own, cut into chunks.
        unsigned seen_rows = 0, seen_pieces = 0, seen_late = 0, seen_chunks = 0;   // (lane 0) the counters as last read
        auto poll = [&]() {
            if (lane == 0) {
                seen_rows = ld_volatile(&fl.counters[kCtrQueued]);
                seen_pieces = ld_volatile(&fl.counters[kCtrPieces]);
                seen_late = ld_volatile(&fl.counters[kCtrLateQueued]);
                seen_chunks = ld_volatile(&fl.counters[kCtrLateChunks]);
            }
        };
        int held = -1, held_late = -1;    // (lane 0) tickets drawn and not yet used
        auto claim = [&](unsigned rows, unsigned taken_seen, int taken, int per_row, int& hold) -> int {
            int t = -1;
            if (lane == 0) {
                const unsigned avail = rows * static_cast<unsigned>(per_row);
                if (hold < 0 && taken_seen < avail) hold = static_cast<int>(atomicAdd(&fl.counters[taken], 1u));
                if (hold >= 0 && static_cast<unsigned>(hold) < avail) { t = hold; hold = -1; }
            }
            return __shfl_sync(0xffffffffu, t, 0);
        };
        auto late_desc = [&](int t, FlowDesc& d) -> bool {
            unsigned e = 0;
            for (unsigned spins = 0; (e = ld_volatile(&fl.lq[t / fl.nch_late])) == 0u; ++spins)
                if (spins > lim_nap) { if (prm.status) atomicExch(prm.status, 1); return false; }
            const int ri = static_cast<int>(e - 1u);
            const int r = ri % (g + 1), b = ri / (g + 1);
            // (a last target row, or a row pair that Algorithm 1 asks for once the tests before it have passed)
            d.kind = kSweep1; d.ri = ri; d.ch = t % fl.nch_late; d.have_q = r < g && prm.lse_d == nullptr;
            item_range(cx.units, fl.nch_late, d.ch, d.u0, d.u1);
            d.rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
            d.rowQ = d.have_q ? static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes : nullptr;
            d.cp = 1.f; d.nMP = 0.f; d.nMQ = 0.f;
            return true;
        };
        auto piece_desc = [&](int t, FlowDesc& d) -> bool {
            unsigned e = 0;
            for (unsigned spins = 0; (e = ld_volatile(&fl.s2q[t / fl.np])) == 0u; ++spins)   // the entry follows the tail at once
                if (spins > lim_nap) { if (prm.status) atomicExch(prm.status, 1); return false; }
            const int ri = static_cast<int>(e - 1u);
            const int r = ri % (g + 1), b = ri / (g + 1);
            d.kind = kSweep2; d.ri = ri; d.ch = t % fl.np; d.have_q = r < g;
            item_range(cx.units, fl.np, d.ch, d.u0, d.u1);
            d.rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
            d.rowQ = r < g ? static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes
                           : nullptr;
            d.cp = 1.f;
            __threadfence();
            if (d.have_q) d.cp = __ldcg(&fl.cscale[ri]);
            d.nMP = -static_cast<float>(__ldcg(&fl.rowZ[ri].MP));
            d.nMQ = -static_cast<float>(__ldcg(&fl.rowZ[ri].MQ));
            return true;
        };
        auto publish = [&](const FlowDesc& d, int q) {
            if (lane == 0) { sh.desc[q % kFDesc] = d; mbar_arrive(smem_u32(&sh.full[q % kFDesc])); }
            __syncwarp();
        };
        int q = 0;                        // items published
        bool tail = false;                // the tickets are about to run out
        bool exhausted = false;           // the ticket counter has run past the last item
        bool failed = false;
        int depth = fl.depth;             // descriptors published and not yet swept, at most
        unsigned idle = 0;
        draw_tickets(1);
        poll();
        for (;;) {
            // the slot must be free (its previous item moved out by its post warp), and at most `depth`
            // published items may still be with the workers
            if (q >= kFDesc && !mbar_wait_relaxed(smem_u32(&sh.freeb[q % kFDesc]), static_cast<uint32_t>(q / kFDesc - 1) & 1u, prm.status, 100, lim_nap)) { failed = true; break; }
            if (q >= depth && !mbar_wait_relaxed(smem_u32(&sh.done[(q - depth) % kFDesc]), static_cast<uint32_t>((q - depth) / kFDesc) & 1u, prm.status, 100, lim_nap)) { failed = true; break; }
            FlowDesc d;
            d.kind = kExit;
            // (a) a piece of a row that waits for its second sweep: they are few and others wait for them;
            // (b) a chunk of a row whose first sweep turned out to be wanted (a last target row, or the
            // next rows of Algorithm 1 after a test has passed).  Algorithm 1 looks at (b) first: there a
            // second sweep ends its block and nothing waits for it, while the next row of a block that
            // keeps accepting is what the launch waits for in the end.
            int t = -1;
            bool is_piece = false;
            if (fl.tv) {
                t = claim(seen_late, seen_chunks, kCtrLateChunks, fl.nch_late, held_late);
                if (t < 0) { t = claim(seen_rows, seen_pieces, kCtrPieces, fl.np, held); is_piece = t >= 0; }
            } else {
                t = claim(seen_rows, seen_pieces, kCtrPieces, fl.np, held);
                is_piece = t >= 0;
                if (t < 0) t = claim(seen_late, seen_chunks, kCtrLateChunks, fl.nch_late, held_late);
            }
            if (t >= 0 && is_piece) {
                if (!piece_desc(t, d)) { failed = true; break; }
                if (lane == 0) ++seen_pieces;
            } else if (t >= 0) {
                if (!late_desc(t, d)) { failed = true; break; }
                if (lane == 0) ++seen_chunks;
            } else if (!exhausted) {
                // (c) a new first-sweep chunk, by the ticket drawn ahead
                if (tk_cnt == 0) draw_tickets(1);
                const unsigned t1 = next_ticket();
                if (t1 >= total_s1) { exhausted = true; tk_cnt = 0; continue; }
                sweep1_desc(t1, d);
                // Towards the end of the tickets a CTA no longer claims a chunk ahead of its needs:
                // a CTA that has run dry could start it at once.
                tail = t1 + gridDim.x >= total_s1;
                if (!tail) draw_tickets(1);
            }
            if (d.kind != kExit) {
                publish(d, q);
                ++q;
                poll();                   // (answers arrive while the workers sweep)
                idle = 0;
                continue;
            }
            // (d) nothing to start: leave once every block is finished and every item post-processed
            if (*reinterpret_cast<volatile unsigned*>(&sh.posted) == static_cast<unsigned>(q) &&
                ld_volatile(&fl.counters[kCtrBlocks]) >= static_cast<unsigned>(cx.B)) break;
            // the next item waits for a row that another CTA completes (all idle CTAs look at the same
            // counters: wait long enough not to crowd those who work)
            __nanosleep(exhausted || idle < 4 ? 500 : 2000);
            poll();
            if (++idle > (lim_nap >> 1)) { if (prm.status) atomicExch(prm.status, 1); failed = true; break; }
        }
        // release the workers and the post warps: one exit descriptor for each post warp to find
        // (on the regular way out every slot is free; after a wait that gave up nothing is relied on)
        for (int j = 0; j < kFPost; ++j) {
            FlowDesc d; d.kind = kExit;
            publish(d, q + j);
        }
        // The counters and flags must be zero when the next launch starts.  Every block is finished,
        // so nobody needs the flags any more: each CTA clears its share of them on its way out.  The
        // global counters are still read by CTAs that have yet to see that all blocks are finished;
        // the last CTA to leave clears those (and everything, if a wait gave up somewhere and the
        // others may have written after their shares were cleared).
        {
            unsigned* z = fl.counters;
            const unsigned words = fl.zero_words - kCounterWords;
            const unsigned per = (words + gridDim.x - 1) / gridDim.x;
            const unsigned w0 = kCounterWords + blockIdx.x * per;
            const unsigned w1 = min(w0 + per, fl.zero_words);
            for (unsigned i = w0 + lane; i < w1; i += 32) z[i] = 0u;
            __threadfence();
            __syncwarp();
            unsigned left = 0;
            if (lane == 0) left = atomicAdd(&fl.counters[kCtrExited], 1u);
            left = __shfl_sync(0xffffffffu, left, 0);
            if (left == gridDim.x - 1) {
                __threadfence();
                if (prm.status && *reinterpret_cast<volatile int*>(prm.status) != 0)
                    for (unsigned i = kCounterWords + lane; i < fl.zero_words; i += 32) z[i] = 0u;
                for (unsigned i = lane; i < kCounterWords; i += 32) z[i] = 0u;
            }
        }
        return;
    }

    // =============================== worker warps ===============================
    // A warp sees the CTA's items as one stream of ring steps.  The consume side does the arithmetic
    // of the oldest step in flight and then refills that very ring slot from the issue cursor, which
    // runs kFSlots steps ahead and moves on to the next item as soon as it has asked for the last
    // vector of the current one, provided the next descriptor is already there.  So the ring is not
    // drained between items; it is only when the issue cursor finds no descriptor (or the exit
    // descriptor) that it stops for good, and the consume side restarts it with a fresh prologue once
    // it reaches an item whose loads have not been started.  Every ring step commits exactly one
    // copy group (an empty one when nothing was asked for), so "all but the kFSlots - 1 newest groups
    // are complete" always means that the slot about to be consumed has landed.
    constexpr uint32_t kCell = kFThreads * 16;               // bytes between consecutive ring cells of a thread
    constexpr uint32_t kPad = PROBS ? 0u : R::kNegInf;       // what a lane beyond the end of a segment finds: no weight
    const uint32_t sb = smem_u32(dyn) + static_cast<uint32_t>(tid) * 16u;   // this thread's ring cell 0
    const uint32_t ring_end = sb + kFDepth * kCell;
    // Every load streams past L2 (its lines are the first to be evicted).  Leaving the first sweep's
    // lines at normal priority, so that a second sweep that follows soon finds them in L2, is a
    // tuning switch: measured 2 to 5 % slower on every shape tried, Algorithm 1 included.
    const uint64_t pol_stream = l2_policy_evict_first();
    const uint64_t pol_keep = fl.keep_l2 ? l2_policy_evict_normal() : pol_stream;
    uint64_t pol = pol_stream;
    const char* iA = nullptr;         // issue cursor: this lane's next vector for cell A and for cell B
    const char* iB = nullptr;
    int i_rem = 0;                    // vectors of the current segment not yet asked for
    int i_adv = 32;                   // vectors a step covers: 32 of each row, or 64 of the one row
    uint32_t i_adv16 = 512;           // the same in bytes
    int n_i = 0;                      // items the issue cursor has started
    bool i_stalled = false;
    uint32_t rp = sb;                 // ring slot to consume next, and to refill right afterwards

    auto issue_load = [&](int slot) {
        int w0, w1;
        warp_range(sh.desc[slot].u0, sh.desc[slot].u1, warp, w0, w1);
        const bool single = sh.desc[slot].have_q == 0;
        pol = sh.desc[slot].kind == kSweep1 ? pol_keep : pol_stream;
        i_rem = w1 - w0;
        i_adv = single ? 64 : 32;
        i_adv16 = single ? 1024u : 512u;
        iA = sh.desc[slot].rowP + static_cast<size_t>(w0 + lane) * 16;
        iB = single ? iA + 512 : sh.desc[slot].rowQ + static_cast<size_t>(w0 + lane) * 16;
    };
    // one ring step of the issue cursor into the slot at `slot_addr`
    auto issue_step = [&](uint32_t slot_addr) {
        if (i_rem >= i_adv) {                                // a full step: every lane has its two vectors
            cp_async16_hint(slot_addr, iA, pol);
            cp_async16_hint(slot_addr + kCell, iB, pol);
            cp_async_commit();
            i_rem -= i_adv;
            iA += i_adv16;
            iB += i_adv16;
            return;
        }
        if (i_rem <= 0 && !i_stalled) {
            for (;;) {                                       // the next item with something for this warp
                const int slot = n_i % kFDesc;
                if (!mbar_try_wait_now(smem_u32(&sh.full[slot]), static_cast<uint32_t>(n_i / kFDesc) & 1u) ||
                    sh.desc[slot].kind == kExit) { i_stalled = true; break; }
                issue_load(slot);
                ++n_i;
                if (i_rem > 0) break;
            }
        }
        if (i_rem >= i_adv) {
            cp_async16_hint(slot_addr, iA, pol);
            cp_async16_hint(slot_addr + kCell, iB, pol);
        } else if (i_rem > 0) {                              // the short last step of a segment
            ring_fetch_hint(slot_addr, iA, lane < i_rem, kPad, pol);
            ring_fetch_hint(slot_addr + kCell, iB, lane + (i_adv - 32) < i_rem, kPad, pol);
        }
        if (i_rem > 0) {
            i_rem -= i_adv;
            iA += i_adv16;
            iB += i_adv16;
        }
        cp_async_commit();
    };
    for (int n_c = 0;; ++n_c) {
        const int slot = n_c % kFDesc;
        if (n_i == n_c) {
            // the loads of this item have not been started: the ring is empty
            if (!mbar_wait_now(smem_u32(&sh.full[slot]), static_cast<uint32_t>(n_c / kFDesc) & 1u, prm.status, lim_spin)) break;
            if (sh.desc[slot].kind == kExit) break;
            i_stalled = false;
            issue_load(slot);
            n_i = n_c + 1;
            uint32_t a = rp;
#pragma unroll
            for (int j = 0; j < kFSlots; ++j) {
                issue_step(a);
                a += 2 * kCell;
                if (a == ring_end) a = sb;
            }
        }
        const int kind = sh.desc[slot].kind;
        const bool have_q = sh.desc[slot].have_q != 0;
        int w0, w1;
        warp_range(sh.desc[slot].u0, sh.desc[slot].u1, warp, w0, w1);
        int c_left = have_q ? (w1 - w0 + 31) >> 5 : (w1 - w0 + 63) >> 6;
        float MPw = kNoRef, sP = 0.f, MQw = kNoRef, sQ = 0.f;
        // the steps of this item; the oldest step in flight is always the next one of this item
        auto run_steps = [&](auto&& body) {
            for (; c_left > 0; --c_left) {
                cp_async_wait<kFSlots - 1>();
                float va[EPV], vb[EPV];
                R::unpack(lds128(rp), va);
                R::unpack(lds128(rp + kCell), vb);
                body(va, vb);
                issue_step(rp);
                rp += 2 * kCell;
                if (rp == ring_end) rp = sb;
            }
        };
        if (!PROBS && kind == kSweep1) {
            if (c_left > 0) {                                // references from the first vector of every lane
                cp_async_wait<kFSlots - 1>();
                float va[EPV], vb[EPV];
                R::unpack(lds128(rp), va);
                R::unpack(lds128(rp + kCell), vb);
                if (have_q) {
                    MPw = fmaxf(rintf(warp_max(vec_max<EPV>(va)) * kf), kNoRef);
                    MQw = fmaxf(rintf(warp_max(vec_max<EPV>(vb)) * kf), kNoRef);
                } else {
                    MPw = fmaxf(rintf(warp_max(fmaxf(vec_max<EPV>(va), vec_max<EPV>(vb))) * kf), kNoRef);
                }
            }
            double tPd;
            if (have_q) {
                run_steps([&](const float (&va)[EPV], const float (&vb)[EPV]) {
                    f_step_sweep1_pair<EPV>(va, vb, kf, MPw, sP, MQw, sQ);
                });
                tPd = static_cast<double>(warp_sum(sP));
            } else {
                // (a row swept alone is a last target row, from whose sums a token may be drawn: in double)
                double sPd = 0.0;
                run_steps([&](const float (&va)[EPV], const float (&vb)[EPV]) {
                    f_step_sweep1_single<EPV>(va, vb, kf, MPw, sPd);
                });
                tPd = warp_sum_d(sPd);
            }
            const float tQ = have_q ? warp_sum(sQ) : 0.f;
            if (lane == 0) {
                sh.part_M[slot][0][warp] = MPw; sh.part_d[slot][warp] = tPd;
                sh.part_M[slot][1][warp] = MQw; sh.part_s[slot][warp] = tQ;
            }
        } else {
            const float cp = sh.desc[slot].cp, nMP = sh.desc[slot].nMP, nMQ = sh.desc[slot].nMQ;
            double acc = 0.0;
            if (have_q) {
                run_steps([&](const float (&va)[EPV], const float (&vb)[EPV]) {
                    float t[EPV];
                    acc += static_cast<double>(f_pair_sum<EPV, true, PROBS>(va, vb, kf, cp, nMP, nMQ, t));
                });
            } else {
                run_steps([&](const float (&va)[EPV], const float (&vb)[EPV]) {
                    float t[EPV];
                    acc += static_cast<double>(f_pair_sum<EPV, false, PROBS>(va, va, kf, cp, nMP, nMQ, t));
                    acc += static_cast<double>(f_pair_sum<EPV, false, PROBS>(vb, vb, kf, cp, nMP, nMQ, t));
                });
            }
            const double tP = warp_sum_d(acc);
            if (lane == 0) sh.part_d[slot][warp] = tP;
        }
        if (lane == 0 && !prm.never_signal) mbar_arrive(smem_u32(&sh.done[slot]));   // releases this warp's partials and the descriptor
        __syncwarp();
    }
    cp_async_wait<0>();
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static size_t up256(size_t x) { return (x + 255) / 256 * 256; }
// floats of seg_tot per row: the sweep-2 totals (np pieces of kFWarps segments) or, for a last
// target row, the sweep-1 {reference, sum} pairs (nch_late chunks of kFWarps segments)
static size_t flow_seg_stride(const FlowPlan& plan) {
    const size_t a = static_cast<size_t>(plan.np) * kFWarps, b = static_cast<size_t>(plan.nch_late) * kFWarps * 2;
    return a > b ? a : b;
}

size_t flow_scratch_bytes(int B, int gamma, const FlowPlan& plan, size_t* zero_bytes) {
    const size_t rows = static_cast<size_t>(B) * (gamma + 1);
    const size_t segs = flow_seg_stride(plan);
    size_t z = 0;
    z += up256(kCounterWords * sizeof(unsigned));   // counters
    z += 2 * up256(rows * sizeof(unsigned));        // row_cnt, s2_cnt
    z += 3 * up256(static_cast<size_t>(B) * sizeof(unsigned));   // cand_cnt, rows_in, bad
    z += 2 * up256(rows * sizeof(unsigned));        // rel, s2q
    z += up256(rows * sizeof(unsigned));            // lq
    if (plan.tv_spec > 0) {
        z += 3 * up256(static_cast<size_t>(B) * sizeof(unsigned long long));   // tv_acc, tv_done, tv_badrows
        z += 2 * up256(static_cast<size_t>(B) * sizeof(unsigned));             // tv_front, tv_decided
    }
    if (zero_bytes) *zero_bytes = z;
    size_t n = z;
    n += up256(rows * plan.part_stride() * sizeof(RowZ));   // part
    n += up256(rows * sizeof(RowZ));                // rowZ
    n += up256(static_cast<size_t>(B) * (gamma + 2) * sizeof(double));   // pchain
    n += up256(rows * sizeof(float));               // cscale
    n += 2 * up256(rows * sizeof(double));          // ratio, zratio
    n += up256(rows * segs * sizeof(double));       // seg_tot
    n += up256(rows * sizeof(double));              // S
    n += up256(rows * sizeof(int));                 // cand
    n += up256(static_cast<size_t>(B) * sizeof(int));   // tv_tau
    return n;
}

void flow_scratch_layout(void* base, int B, int gamma, const FlowPlan& plan, FlowScratch* fl) {
    const size_t rows = static_cast<size_t>(B) * (gamma + 1);
    const size_t segs = flow_seg_stride(plan);
    char* p = static_cast<char*>(base);
    auto take = [&](size_t bytes) { char* q = p; p += up256(bytes); return q; };
    fl->counters = reinterpret_cast<unsigned*>(take(kCounterWords * sizeof(unsigned)));
    fl->row_cnt = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->s2_cnt = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->cand_cnt = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->rows_in = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->bad = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->rel = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->s2q = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->lq = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->tv = plan.tv_spec > 0;
    fl->tv_spec = plan.tv_spec;
    fl->tv_ahead = plan.tv_ahead;
    fl->tv_acc = fl->tv_done = fl->tv_badrows = nullptr;
    fl->tv_front = fl->tv_decided = nullptr;
    if (plan.tv_spec > 0) {
        fl->tv_acc = reinterpret_cast<unsigned long long*>(take(static_cast<size_t>(B) * sizeof(unsigned long long)));
        fl->tv_done = reinterpret_cast<unsigned long long*>(take(static_cast<size_t>(B) * sizeof(unsigned long long)));
        fl->tv_badrows = reinterpret_cast<unsigned long long*>(take(static_cast<size_t>(B) * sizeof(unsigned long long)));
        fl->tv_front = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
        fl->tv_decided = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    }
    fl->part = reinterpret_cast<RowZ*>(take(rows * plan.part_stride() * sizeof(RowZ)));
    fl->rowZ = reinterpret_cast<RowZ*>(take(rows * sizeof(RowZ)));
    fl->pchain = reinterpret_cast<double*>(take(static_cast<size_t>(B) * (gamma + 2) * sizeof(double)));
    fl->cscale = reinterpret_cast<float*>(take(rows * sizeof(float)));
    fl->ratio = reinterpret_cast<double*>(take(rows * sizeof(double)));
    fl->zratio = reinterpret_cast<double*>(take(rows * sizeof(double)));
    fl->seg_tot = reinterpret_cast<double*>(take(rows * segs * sizeof(double)));
    fl->S = reinterpret_cast<double*>(take(rows * sizeof(double)));
    fl->cand = reinterpret_cast<int*>(take(rows * sizeof(int)));
    fl->tv_tau = reinterpret_cast<int*>(take(static_cast<size_t>(B) * sizeof(int)));
    fl->nch = plan.nch;
    fl->keep_l2 = 0;
    fl->part_stride = plan.part_stride();
    fl->fine_from = plan.fine_from;
    fl->total_s1 = plan.probs ? 0u
                 : plan.tv_spec > 0 ? static_cast<unsigned>(B) * plan.tv_spec * plan.nch
                 : static_cast<unsigned>(plan.fine_from) * gamma * plan.nch + static_cast<unsigned>(B - plan.fine_from) * gamma * plan.nch_late;
    fl->tail_mode = plan.tail_mode;
    fl->nch_late = plan.nch_late;
    fl->np = plan.np;
    // descriptors a CTA hands to its workers ahead of the sweep: two keep the ring from draining between items;
    // a third only delays the second-sweep pieces and late rows a CTA claims (Block Verification: 1 to 8 %
    // where many tokens are accepted), while Algorithm 1, whose items are shorter, measured better with three
    fl->depth = plan.tv_spec > 0 ? 3 : 2;
    size_t zb = 0;
    flow_scratch_bytes(B, gamma, plan, &zb);
    fl->zero_words = static_cast<unsigned>(zb / sizeof(unsigned));
    fl->segs = static_cast<int>(segs);
}

// How a launch is cut into work items.
//   First sweep: an item should be large next to what it costs to hand it out and account for it
//   (about a microsecond, and half a ring step per warp at its end), so rows are cut into chunks of
//   about 16000 vectors (256 KB per row), finer while the batch alone cannot give every CTA a few
//   items.  A chunk keeps at least 2048 vectors.
//   Second sweep, and the first sweep of a last target row that turns out to be wanted: only few rows
//   are concerned and a block's candidates are swept one after the other, so these rows are cut into
//   pieces of about 4000 vectors that many CTAs share.
FlowPlan flow_plan(long long units, int B, int gamma, long long nctas, bool pair_items, int chunks, int pieces, bool token_verify, bool probs) {
    FlowPlan pl{};
    pl.probs = probs;
    long long np = units / 3500;
    if (np < 1) np = 1;
    if (np > 128 / kFWarps) np = 128 / kFWarps;             // (a position's segment totals are looked at four per lane)
    pl.np = pieces > 0 ? pieces : static_cast<int>(np);
    pl.nch_late = static_cast<int>(np > 8 ? 8 : np);
    const long long row_units = pair_items ? units : units / 2;   // (a single-row item streams half as much)
    long long nch = (row_units + 8000) / 16000;
    if (nch < 1) nch = 1;
    if (nch > 8) nch = 8;
    // (Algorithm 1 starts with one row of every block, or a few: that is what has to fill the GPU)
    const long long rows = static_cast<long long>(B) * (token_verify ? 1 : gamma);
    while (nch < 8 && rows * nch < 4 * nctas && row_units / (nch + 1) >= 2048) ++nch;
    pl.nch = chunks > 0 ? chunks : static_cast<int>(nch);
    if (chunks > pl.nch_late && chunks <= 8) pl.nch_late = chunks;
    // Algorithm 1.  Where one row pair of every block is more than about 100 MB (17 us of streaming, what a
    // dependent row costs in latency), rows are read strictly on demand: one row of every block from the
    // start, the next only when the test before it has passed, so nothing beyond the first rejection is
    // read.  Smaller batches leave the GPU idle while a block waits for its next row: there, as many rows
    // from the start as it takes to give every CTA an item (at least two), and once all of those have
    // passed, which marks a draft that is mostly accepted, all the remaining rows at once.
    // Given probabilities nothing is swept before a block's candidates are known.  A batch whose
    // highest candidates alone give every CTA a few pieces sweeps them from the top down, one at a
    // time (the fewest bytes); a smaller one starts all of a block's candidates at once.
    pl.tail_mode = 0;
    if (probs) pl.tail_mode = static_cast<long long>(B) * pl.np >= 2 * nctas ? 2 : 1;
    pl.fine_from = B;
    pl.tv_spec = 0;
    pl.tv_ahead = 1;
    if (token_verify) {
        pl.tv_spec = 1;
        const long long pair_bytes = units * 32;
        if (static_cast<long long>(B) * pair_bytes <= 100000000LL) {
            long long k = (nctas + static_cast<long long>(B) * pl.nch - 1) / (static_cast<long long>(B) * pl.nch);
            if (k < 2) k = 2;
            pl.tv_spec = static_cast<int>(k > gamma ? gamma : k);
            pl.tv_ahead = gamma;
        }
    }
    return pl;
}

using FKernelFn = void (*)(const Params, const FlowScratch);
static FKernelFn pick_flow(int dtype, bool probs) {
    if (probs) return dtype == kF32 ? verify_flow_kernel<kF32, true> : verify_flow_kernel<kBF16, true>;
    return dtype == kF32 ? verify_flow_kernel<kF32, false> : verify_flow_kernel<kBF16, false>;
}

static constexpr size_t kFlowSmem = sizeof(uint4) * kFDepth * kFThreads;

int flow_threads() { return kFAllThreads; }

int flow_max_ctas_per_sm(int dtype) {
    int n = 0;
    for (int probs = 0; probs < 2; ++probs) {
        if (cudaFuncSetAttribute(reinterpret_cast<const void*>(pick_flow(dtype, probs != 0)),
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kFlowSmem)) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
    }
    // (the variant on logits is the larger program: its occupancy serves both)
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pick_flow(dtype, false), kFAllThreads, kFlowSmem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t launch_flow(const Params& prm, const FlowScratch& fl_in, int dtype, int nctas, cudaStream_t stream) {
    const FlowScratch& fl = fl_in;
    pick_flow(dtype, prm.probs != 0)<<<nctas, kFAllThreads, kFlowSmem, stream>>>(prm, fl);
    return cudaGetLastError();
}

}  // namespace bv
