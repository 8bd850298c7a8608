// Block Verification (Algorithm 2) as a dependency-driven flow of independent work items.
//
// Persistent CTAs (16 worker warps that only stream, one service warp that does everything
// else) pull items from three sources, in this order of preference:
//
//   sweep-2 piece (b, r, piece)  a piece of a row pair whose second sweep has been started:
//       leaves sum max(p_r P_r(x) - Q_r(x), 0) per warp segment (Eq. "pacc_block").  The CTA
//       that completes a position adds the segments to S_r, locates u * S_r, rescans that one
//       segment in index order for the candidate Y_r (Eq. "pres-block"), and then either finds
//       the position selected or starts the next lower candidate; the CTA that completes the
//       block forms h_i, selects tau and emits X^tau, Y_tau.
//   late sweep-1 chunk  of a last target row P_gamma, which is read only if position gamma can
//       be the selected one; its sample is drawn from that one sweep.
//   sweep-1 item (b, r < gamma, chunk)  by ticket, in row order: streams the chunk of both
//       rows from HBM and leaves the chunk's {reference, sum 2^{z k - M}} pair for each row in
//       scratch.  The CTA that completes a row combines the chunks into the row normalisers
//       and, holding the block's lock, advances the prefix recursion
//       p_{r+1} = min(p_r P_r(X)/Q_r(X), 1) (Eq. "def_as") over every row that is complete.
//
// A second sweep runs only where the outcome can depend on it: S_r <= p_r gives h_r <= p_r, so
// a position with eta_r > p_r can never be selected; the others are swept from the top down
// until one passes its test (bv_flow_common.cuh).  With diagnostic outputs every position is
// swept.
//
// No CTA ever waits for another one while it holds work that others need: sweep-1 items
// have no prerequisites, the lock is only held over a few scalar operations, and a CTA
// polls (bounded) only when nothing is left to start.  So CTAs need not be co-resident.
#include "bv_flow_common.cuh"

namespace bv {

constexpr int kFThreads = 512;
constexpr int kFWarps = kFThreads / 32;

// vectors [w0, w1) of a row that worker `warp` takes of part `ch` out of `nparts`
__device__ __forceinline__ void chunk_range(const FlowCtx& cx, int nparts, int ch, int warp, int& w0, int& w1) {
    const int u0 = static_cast<int>(static_cast<long long>(cx.units) * ch / nparts);
    const int u1 = static_cast<int>(static_cast<long long>(cx.units) * (ch + 1) / nparts);
    w0 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * warp / kFWarps);
    w1 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * (warp + 1) / kFWarps);
}


// ring slots per worker thread: three (P, Q) steps of lookahead.  Measured at B = 256, gamma = 8,
// V = 256000 bf16: 4 slots 0.485 ms, 6 slots 0.471 ms, 8 slots 0.482 ms, 12 slots 0.505 ms; with 32
// streaming warps per SM the latency is hidden by the other warps, and more bytes in flight only
// crowd the memory system.
constexpr int kFDepth = 6;
constexpr int kFAhead = kFDepth / 2;
constexpr int kFDesc = 3;      // items in flight per CTA: one being swept, two queued behind it
constexpr int kFAllThreads = kFThreads + 32;   // 16 worker warps + 1 service warp

// One work item as the service warp hands it to the workers.
struct FlowDesc {
    int kind;                   // kExit, kSweep1, kSweep2
    int ri, ch;                 // row index b (gamma+1) + r, chunk
    int have_q;
    const char* rowP;
    const char* rowQ;
    float cp, nMP, nMQ;         // sweep 2: p_r Z_Q / Z_P and minus the row references
};


struct FlowShared {
    FlowDesc desc[kFDesc];
    unsigned long long full[kFDesc];    // the service warp has filled desc[i]
    unsigned long long done[kFDesc];    // all 16 worker warps have left their partials of desc[i]
    float part_M[kFDesc][2][kFWarps];   // sweep 1: references of P and Q per worker warp
    float part_s[kFDesc][2][kFWarps];   // sweep 1: sums; sweep 2: [0] holds the residual totals
};

// ---- service warp: Y ~ P_gamma from the first sweep of the last target row ----
// The sample needs the row's normaliser and a second look at one segment only: the segment
// {reference, sum} pairs of all chunks are in scratch, so u * Z is located among their prefix sums
// (fp32, index order) and that one segment is rescanned.  No second sweep of the row.
template <int DT>
__device__ void f_draw_from_sweep1(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int ri, int lane) {
    const int g = cx.g, b = ri / (g + 1);
    const int nseg = cx.nch * kFWarps;                       // <= 128: four per lane
    const float* pairs = fl.seg_tot + static_cast<size_t>(ri) * fl.segs;
    float m[4], w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i = 4 * lane + j;
        m[j] = i < nseg ? __ldcg(&pairs[2 * i]) : kNoRef;
        w[j] = i < nseg ? __ldcg(&pairs[2 * i + 1]) : 0.f;
    }
    const float Mrow = warp_max(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])));
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] *= ref_scale(m[j], Mrow);
    const float l1 = w[0], l2 = l1 + w[1], l3 = l2 + w[2], l4 = l3 + w[3];
    float inc = l4;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float o = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += o;
    }
    const float total = __shfl_sync(0xffffffffu, inc, 31);
    int found = -1;
    if (Mrow > kNoRef && Mrow < INFINITY && total > 0.f && total < INFINITY) {
        const float t = prm.uni[static_cast<size_t>(b) * (g + 2) + g + 1] * total;
        float exc = __shfl_up_sync(0xffffffffu, inc, 1);
        if (lane == 0) exc = 0.f;
        const float p0 = exc, p1 = exc + l1, p2 = exc + l2, p3 = exc + l3, p4 = exc + l4;
        // first non-empty segment whose inclusive prefix exceeds t, else the last non-empty one
        const bool h1 = p1 > t && w[0] > 0.f, h2 = p2 > t && w[1] > 0.f;
        const bool h3 = p3 > t && w[2] > 0.f, h4 = p4 > t && w[3] > 0.f;
        const unsigned hit = __ballot_sync(0xffffffffu, h1 || h2 || h3 || h4);
        const unsigned nz = __ballot_sync(0xffffffffu, l4 > 0.f);
        int e = 3; float bef = p3; int src;
        if (hit) {
            src = __ffs(hit) - 1;
            if (h1) { e = 0; bef = p0; } else if (h2) { e = 1; bef = p1; } else if (h3) { e = 2; bef = p2; }
        } else {
            src = 31 - __clz(nz);
            e = 0; bef = p0;
            if (w[3] > 0.f) { e = 3; bef = p3; } else if (w[2] > 0.f) { e = 2; bef = p2; }
            else if (w[1] > 0.f) { e = 1; bef = p1; }
        }
        const int sel = __shfl_sync(0xffffffffu, 4 * lane + e, src);
        const float before = __shfl_sync(0xffffffffu, bef, src);
        int s0, s1;
        chunk_range(cx, cx.nch, sel / kFWarps, sel % kFWarps, s0, s1);
        const char* rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
        found = f_rescan<DT>(rowP, nullptr, s0, s1, lane, cx.kf, 1.f, -Mrow, 0.f, t - before);
    }
    if (lane == 0) {
        fl.cand[ri] = found;
        __threadfence();
    }
    __syncwarp();
}

// ---- service warp: what follows the sweep of one item ----
template <int DT>
__device__ void f_after_sweep1(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, FlowShared& sh, int slot,
                               int ri, int ch, int lane) {
    // combine the 16 worker warps of this chunk in fp64
    const float mP = lane < kFWarps ? sh.part_M[slot][0][lane] : kNoRef;
    const float mQ = lane < kFWarps ? sh.part_M[slot][1][lane] : kNoRef;
    const float MPc = warp_max(mP), MQc = warp_max(mQ);
    double zP = lane < kFWarps ? static_cast<double>(sh.part_s[slot][0][lane]) * ref_scale(mP, MPc) : 0.0;
    double zQ = lane < kFWarps ? static_cast<double>(sh.part_s[slot][1][lane]) * ref_scale(mQ, MQc) : 0.0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { zP += shfl_xor_d(zP, off); zQ += shfl_xor_d(zQ, off); }
    // A last target row is swept for one purpose only: the sample from P_gamma.  Its warps' pairs
    // {reference, sum} are kept, so that the token can be drawn from this one sweep (below).
    const bool draw = ri % (cx.g + 1) == cx.g && f_draws_in_sweep1(prm, cx.nch);
    if (draw) {
        float* pairs = fl.seg_tot + static_cast<size_t>(ri) * fl.segs + static_cast<size_t>(ch) * kFWarps * 2;
        if (lane < kFWarps) { pairs[2 * lane] = mP; pairs[2 * lane + 1] = sh.part_s[slot][0][lane]; }
        __threadfence();
        __syncwarp();
    }
    int last = 0;
    if (lane == 0) {
        RowZ z; z.MP = MPc; z.ZP = zP; z.MQ = MQc; z.ZQ = zQ;
        fl.part[static_cast<size_t>(ri) * cx.nch + ch] = z;
        __threadfence();
        last = atomicAdd(&fl.row_cnt[ri], 1u) == static_cast<unsigned>(cx.nch) - 1u;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;
    __threadfence();
    if (draw) f_draw_from_sweep1<DT>(prm, fl, cx, ri, lane);
    if (lane == 0) f_row_complete<DT>(prm, fl, cx, ri / (cx.g + 1), ri % (cx.g + 1));
    __syncwarp();
}

template <int DT>
__device__ void f_after_sweep2(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, FlowShared& sh, int slot,
                               const FlowDesc& d, int lane) {
    const int ri = d.ri;
    const int np = fl.np;
    const int nseg = np * kFWarps;
    float* segs = fl.seg_tot + static_cast<size_t>(ri) * fl.segs;
    if (lane < kFWarps) segs[d.ch * kFWarps + lane] = sh.part_s[slot][0][lane];
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) last = atomicAdd(&fl.s2_cnt[ri], 1u) == static_cast<unsigned>(np) - 1u;
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;

    f_position_complete<DT>(prm, fl, cx, ri, d.have_q != 0, d.rowP, d.rowQ, d.cp, d.nMP, d.nMQ, nseg, segs, lane,
                            [&](int sel, int& s0, int& s1) { chunk_range(cx, np, sel / kFWarps, sel % kFWarps, s0, s1); });
}

// ---- worker warps: one warp's segment of one item ----
// The segment's vectors go through the thread's private ring, kFAhead steps ahead of the
// arithmetic.  A step is one vector per lane of each row; the last step may be partial, and
// lanes past the end then find -inf logits in their slots.
template <int DT, bool HAVEQ, int KIND>
__device__ __forceinline__ void f_sweep_segment(uint32_t sb, const char* rowP, const char* rowQ, int w0, int w1,
                                                int lane, float kf, float cp, float nMP, float nMQ,
                                                float& oMP, float& osP, float& oMQ, float& osQ) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr uint32_t kSlot = kFThreads * 16;               // bytes between consecutive ring cells
    // a step takes two of the thread's ring cells, or one when there is no draft row: then the
    // loads run twice as many steps ahead, so that as many bytes are in flight
    constexpr int kA = HAVEQ ? kFAhead : kFDepth;
    constexpr int kC = HAVEQ ? 2 : 1;
    const int nv = w1 - w0;
    const int nsteps = (nv + 31) >> 5;
    const int nlast = nv - 32 * (nsteps - 1);                // lanes that take part in the last step
    const char* gP = rowP + static_cast<size_t>(w0 + lane) * 16;
    const char* gQ = HAVEQ ? rowQ + static_cast<size_t>(w0 + lane) * 16 : gP;
    // sweep 1 asks L2 to keep the rows (they are read again soon); sweep 2 marks them as done with
    // no row is needed again soon (the few second sweeps come long after the first): stream past L2
    const uint64_t pol = l2_policy_evict_first();
    auto fetch_step = [&](int k, int j) {                    // step k goes to cells kC j (, + 1), j = k mod kA
        if (k < nsteps) {
            const bool ok = (k + 1 < nsteps) || lane < nlast;
            ring_fetch_hint(sb + (kC * j) * kSlot, gP + static_cast<size_t>(k) * 512, ok, R::kNegInf, pol);
            if (HAVEQ) ring_fetch_hint(sb + (kC * j + 1) * kSlot, gQ + static_cast<size_t>(k) * 512, ok, R::kNegInf, pol);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int j = 0; j < kA; ++j) fetch_step(j, j);

    float MPw = kNoRef, sP = 0.f, MQw = kNoRef, sQ = 0.f, acc = 0.f;
    for (int kb = 0; kb < nsteps; kb += kA) {
#pragma unroll
        for (int j = 0; j < kA; ++j) {
            const int k = kb + j;
            if (k < nsteps) {
                cp_async_wait<kA - 1>();                     // step k has landed
                float vp[EPV], vq[EPV];
                R::unpack(lds128(sb + (kC * j) * kSlot), vp);
                if (HAVEQ) R::unpack(lds128(sb + (kC * j + 1) * kSlot), vq);
                if (KIND == kSweep1) {
                    if (j == 0 && kb == 0) {                 // references from the first vector of every lane
                        MPw = fmaxf(rintf(warp_max(vec_max<EPV>(vp)) * kf), kNoRef);
                        if (HAVEQ) MQw = fmaxf(rintf(warp_max(vec_max<EPV>(vq)) * kf), kNoRef);
                    }
                    float vsP = f_exp_sum<EPV>(vp, kf, -MPw);
                    float vsQ = HAVEQ ? f_exp_sum<EPV>(vq, kf, -MQw) : 0.f;
                    if (__any_sync(0xffffffffu, fmaxf(vsP, vsQ) > kRaiseBound)) {   // a logit above a reference
                        if (__any_sync(0xffffffffu, vsP > kRaiseBound)) {
                            const float y = rintf(warp_max(vec_max<EPV>(vp)) * kf);
                            if (y > MPw) { sP *= ref_scale(MPw, y); MPw = y; }
                            vsP = f_exp_sum<EPV>(vp, kf, -MPw);
                        }
                        if (HAVEQ && __any_sync(0xffffffffu, vsQ > kRaiseBound)) {
                            const float y = rintf(warp_max(vec_max<EPV>(vq)) * kf);
                            if (y > MQw) { sQ *= ref_scale(MQw, y); MQw = y; }
                            vsQ = f_exp_sum<EPV>(vq, kf, -MQw);
                        }
                    }
                    sP += vsP;
                    sQ += vsQ;
                } else {
                    float t[EPV];
                    acc += f_pair_sum<EPV, HAVEQ>(vp, vq, kf, cp, nMP, nMQ, t);
                }
                fetch_step(k + kA, j);
            }
        }
    }
    cp_async_wait<0>();
    if (KIND == kSweep1) {
        oMP = MPw; osP = warp_sum(sP);
        oMQ = MQw; osQ = HAVEQ ? warp_sum(sQ) : 0.f;
    } else {
        osP = warp_sum(acc);
    }
}

template <int DT>
__global__ void __launch_bounds__(kFAllThreads, 2) verify_flow_kernel(const Params prm, const FlowScratch fl) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ FlowShared sh;
    // Each worker thread streams its own vectors through a private ring of 16-byte cells filled
    // by cp.async, so loads run kFAhead steps ahead of the arithmetic without costing registers.
    extern __shared__ __align__(16) unsigned char dyn[];

    FlowCtx cx;
    cx.g = prm.gamma; cx.V = prm.V; cx.B = prm.B; cx.nch = fl.nch; cx.units = prm.V / EPV;
    cx.row_bytes = static_cast<size_t>(prm.V) * ESZ; cx.kf = prm.kf; cx.kd = prm.kd;
    const int g = cx.g;
    const float kf = cx.kf;

    if (tid == 0) {
        for (int i = 0; i < kFDesc; ++i) {
            mbar_init(smem_u32(&sh.full[i]), 1);
            mbar_init(smem_u32(&sh.done[i]), kFWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kFWarps) {
        // =============================== service warp ===============================
        // takes tickets, waits for what a sweep-2 item needs, hands descriptors to the workers,
        // and does everything that follows a sweep, so that the workers never stop streaming
        // tickets cover the rows that every block needs: target and draft rows 0 .. gamma-1
        const unsigned total_s1 = static_cast<unsigned>(cx.B) * g * cx.nch;
        // the next sweep-1 item, or kExit when all have been handed out; never blocks
        auto take = [&](FlowDesc& d) {
            unsigned t = 0;
            if (lane == 0) t = atomicAdd(&fl.counters[kCtrTicket], 1u);
            t = __shfl_sync(0xffffffffu, t, 0);
            if (t >= total_s1) { d.kind = kExit; return; }
            const int ch = static_cast<int>(t % cx.nch);
            const int r = static_cast<int>(t / cx.nch) % g, b = static_cast<int>(t / cx.nch) / g;
            const int ri = b * (g + 1) + r;
            // (with supplied draft normalisers the first sweep has nothing to learn from the draft row)
            d.kind = kSweep1; d.ri = ri; d.ch = ch; d.have_q = prm.lse_d == nullptr;
            d.rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
            d.rowQ = d.have_q ? static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes
                              : nullptr;
            d.cp = 1.f; d.nMP = 0.f; d.nMQ = 0.f;
        };
        // Rows whose second sweep has been started stand in a queue, each cut into np pieces.  A
        // piece is claimed by a ticket from the queue's head counter, drawn only while the head is
        // seen behind the tail; a ticket that still runs ahead of the tail (several CTAs drew at
        // once) is kept until its row arrives.  -1: no piece right now.
        int held = -1, held_late = -1;    // (lane 0) tickets drawn and not yet used
        auto claim = [&](int queued, int taken, int per_row, int& hold) -> int {
            int t = -1;
            if (lane == 0) {
                const unsigned avail = ld_volatile(&fl.counters[queued]) * static_cast<unsigned>(per_row);
                if (hold < 0 && ld_volatile(&fl.counters[taken]) < avail)
                    hold = static_cast<int>(atomicAdd(&fl.counters[taken], 1u));
                if (hold >= 0 && static_cast<unsigned>(hold) < avail) { t = hold; hold = -1; }
            }
            return __shfl_sync(0xffffffffu, t, 0);
        };
        auto take_piece = [&]() -> int { return claim(kCtrQueued, kCtrPieces, fl.np, held); };
        // likewise the chunks of last target rows whose first sweep has been asked for
        auto late_desc = [&](FlowDesc& d) -> bool {
            const int t = claim(kCtrLateQueued, kCtrLateChunks, cx.nch, held_late);
            if (t < 0) return false;
            unsigned e = 0;
            for (unsigned spins = 0; (e = ld_volatile(&fl.lq[t / cx.nch])) == 0u; ++spins)
                if (spins > (1u << 22)) { if (prm.status) atomicExch(prm.status, 1); return false; }
            const int ri = static_cast<int>(e - 1u);
            d.kind = kSweep1; d.ri = ri; d.ch = t % cx.nch; d.have_q = 0;
            d.rowP = static_cast<const char*>(prm.tgt) + static_cast<size_t>(ri) * cx.row_bytes;
            d.rowQ = nullptr;
            d.cp = 1.f; d.nMP = 0.f; d.nMQ = 0.f;
            return true;
        };
        auto piece_desc = [&](int t, FlowDesc& d) -> bool {
            unsigned e = 0;
            for (unsigned spins = 0; (e = ld_volatile(&fl.s2q[t / fl.np])) == 0u; ++spins)   // the entry follows the tail at once
                if (spins > (1u << 22)) { if (prm.status) atomicExch(prm.status, 1); return false; }
            const int ri = static_cast<int>(e - 1u);
            const int r = ri % (g + 1), b = ri / (g + 1);
            d.kind = kSweep2; d.ri = ri; d.ch = t % fl.np; d.have_q = r < g;
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
        int q = 0, n = 0, qexit = -1;     // items published / post-processed; index of the exit descriptor
        bool exhausted = false;           // the ticket counter has run past the last item
        unsigned idle = 0;
        for (;;) {
            // 1. publish what can be published (a slot is free once its previous item is post-processed)
            while (qexit < 0 && q - n < fl.depth) {
                FlowDesc d;
                // (a) a piece of a row that waits for its second sweep: they are few and others wait for them
                const int t = take_piece();
                if (t >= 0) {
                    if (!piece_desc(t, d)) { exhausted = true; break; }
                    publish(d, q);
                    ++q;
                    continue;
                }
                // (b) a chunk of a last target row that turned out to be wanted
                if (late_desc(d)) {
                    publish(d, q);
                    ++q;
                    continue;
                }
                // (c) a new sweep-1 item
                if (!exhausted) {
                    take(d);
                    if (d.kind == kExit) { exhausted = true; continue; }
                    publish(d, q);
                    ++q;
                    continue;
                }
                // (d) nothing to start: leave once every block is finished
                if (q == n && ld_volatile(&fl.counters[kCtrBlocks]) >= static_cast<unsigned>(cx.B)) {
                    d.kind = kExit; publish(d, q); qexit = q; ++q;
                }
                break;
            }
            // 2. the oldest item in flight: wait for the workers, then do what follows its sweep
            const int in_flight_end = qexit >= 0 ? qexit : q;
            if (n < in_flight_end) {
                const int slot = n % kFDesc;
                const FlowDesc d = sh.desc[slot];
                mbar_wait_now(smem_u32(&sh.done[slot]), static_cast<uint32_t>(n / kFDesc) & 1u, prm.status);
                if (d.kind == kSweep1) {
                    f_after_sweep1<DT>(prm, fl, cx, sh, slot, d.ri, d.ch, lane);
                } else {
                    f_after_sweep2<DT>(prm, fl, cx, sh, slot, d, lane);
                }
                ++n;
                idle = 0;
                continue;
            }
            if (qexit >= 0) break;
            // 3. nothing in flight and the next item waits for a row that another CTA completes
            // (all idle CTAs look at the same counters: wait long enough not to crowd those who work)
            __nanosleep(idle < 4 ? 500 : 2000);
            if (++idle > (1u << 21)) { if (prm.status) atomicExch(prm.status, 1); break; }
        }
        if (qexit < 0) {      // gave up: release the workers
            FlowDesc d; d.kind = kExit;
            publish(d, q);
        }
        return;
    }

    // =============================== worker warps ===============================
    const uint32_t sb = smem_u32(dyn) + static_cast<uint32_t>(tid) * 16u;   // this thread's ring slot 0
    for (int n = 0;; ++n) {
        const int slot = n % kFDesc;
        const uint32_t parity = static_cast<uint32_t>(n / kFDesc) & 1u;
        mbar_wait_now(smem_u32(&sh.full[slot]), parity, prm.status);
        const int kind = sh.desc[slot].kind;
        if (kind == kExit) break;
        const bool have_q = sh.desc[slot].have_q != 0;
        const char* rowP = sh.desc[slot].rowP;
        const char* rowQ = sh.desc[slot].rowQ;
        int w0, w1;
        chunk_range(cx, kind == kSweep1 ? cx.nch : fl.np, sh.desc[slot].ch, warp, w0, w1);
        float MPw = kNoRef, sP = 0.f, MQw = kNoRef, sQ = 0.f;
        if (kind == kSweep1) {
            if (have_q) f_sweep_segment<DT, true, kSweep1>(sb, rowP, rowQ, w0, w1, lane, kf, 1.f, 0.f, 0.f, MPw, sP, MQw, sQ);
            else        f_sweep_segment<DT, false, kSweep1>(sb, rowP, rowQ, w0, w1, lane, kf, 1.f, 0.f, 0.f, MPw, sP, MQw, sQ);
            if (lane == 0) {
                sh.part_M[slot][0][warp] = MPw; sh.part_s[slot][0][warp] = sP;
                sh.part_M[slot][1][warp] = MQw; sh.part_s[slot][1][warp] = sQ;
            }
        } else {
            const float cp = sh.desc[slot].cp, nMP = sh.desc[slot].nMP, nMQ = sh.desc[slot].nMQ;
            if (have_q) f_sweep_segment<DT, true, kSweep2>(sb, rowP, rowQ, w0, w1, lane, kf, cp, nMP, nMQ, MPw, sP, MQw, sQ);
            else        f_sweep_segment<DT, false, kSweep2>(sb, rowP, rowQ, w0, w1, lane, kf, cp, nMP, nMQ, MPw, sP, MQw, sQ);
            if (lane == 0) sh.part_s[slot][0][warp] = sP;
        }
        if (lane == 0) mbar_arrive(smem_u32(&sh.done[slot]));   // releases this warp's partials and the descriptor
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static size_t up256(size_t x) { return (x + 255) / 256 * 256; }
// floats of seg_tot per row: the sweep-2 totals (np pieces of kFWarps segments) or, for a last
// target row, the sweep-1 {reference, sum} pairs (nch chunks of kFWarps segments)
static size_t flow_seg_stride(int nch, int np) {
    const size_t a = static_cast<size_t>(np) * kFWarps, b = static_cast<size_t>(nch) * kFWarps * 2;
    return a > b ? a : b;
}

size_t flow_scratch_bytes(int B, int gamma, int nch, int np, size_t* zero_bytes) {
    const size_t rows = static_cast<size_t>(B) * (gamma + 1);
    const size_t segs = flow_seg_stride(nch, np);
    size_t z = 0;
    z += up256(kCounterWords * sizeof(unsigned));   // counters
    z += 3 * up256(rows * sizeof(unsigned));        // row_cnt, row_done, s2_cnt
    z += 4 * up256(static_cast<size_t>(B) * sizeof(unsigned));   // cand_cnt, chain, lock, bad
    z += 2 * up256(rows * sizeof(unsigned));        // rel, s2q
    z += up256(static_cast<size_t>(B) * sizeof(unsigned));       // lq
    if (zero_bytes) *zero_bytes = z;
    size_t n = z;
    n += up256(rows * nch * sizeof(RowZ));          // part
    n += up256(rows * sizeof(RowZ));                // rowZ
    n += up256(static_cast<size_t>(B) * (gamma + 2) * sizeof(double));   // pchain
    n += up256(rows * sizeof(float));               // cscale
    n += 2 * up256(rows * sizeof(double));          // ratio, zratio
    n += up256(rows * segs * sizeof(float));        // seg_tot
    n += up256(rows * sizeof(double));              // S
    n += up256(rows * sizeof(int));                 // cand
    return n;
}

void flow_scratch_layout(void* base, int B, int gamma, int nch, int np, FlowScratch* fl) {
    const size_t rows = static_cast<size_t>(B) * (gamma + 1);
    const size_t segs = flow_seg_stride(nch, np);
    char* p = static_cast<char*>(base);
    auto take = [&](size_t bytes) { char* q = p; p += up256(bytes); return q; };
    fl->counters = reinterpret_cast<unsigned*>(take(kCounterWords * sizeof(unsigned)));
    fl->row_cnt = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->row_done = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->s2_cnt = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->cand_cnt = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->chain = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->lock = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->bad = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->rel = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->s2q = reinterpret_cast<unsigned*>(take(rows * sizeof(unsigned)));
    fl->lq = reinterpret_cast<unsigned*>(take(static_cast<size_t>(B) * sizeof(unsigned)));
    fl->part = reinterpret_cast<RowZ*>(take(rows * nch * sizeof(RowZ)));
    fl->rowZ = reinterpret_cast<RowZ*>(take(rows * sizeof(RowZ)));
    fl->pchain = reinterpret_cast<double*>(take(static_cast<size_t>(B) * (gamma + 2) * sizeof(double)));
    fl->cscale = reinterpret_cast<float*>(take(rows * sizeof(float)));
    fl->ratio = reinterpret_cast<double*>(take(rows * sizeof(double)));
    fl->zratio = reinterpret_cast<double*>(take(rows * sizeof(double)));
    fl->seg_tot = reinterpret_cast<float*>(take(rows * segs * sizeof(float)));
    fl->S = reinterpret_cast<double*>(take(rows * sizeof(double)));
    fl->cand = reinterpret_cast<int*>(take(rows * sizeof(int)));
    fl->nch = nch;
    fl->np = np;
    fl->depth = kFDesc;
    fl->segs = static_cast<int>(segs);
}

// Pieces per row in the second sweep.  Only the few rows that may hold the selected position are
// swept again, and the candidates of a block are swept one after the other, so their rows are cut
// finer than in the first sweep: more CTAs share a row and the chain of a block gets shorter.  A
// piece keeps at least 2048 vectors.
int flow_pick_pieces(long long units) {
    long long np = units / 4000;
    if (np < 1) np = 1;
    if (np > 8) np = 8;
    return static_cast<int>(np);
}

// Chunks per row.  An item should be large next to what it costs to hand it out (about
// 16000 vectors, 256 KB, per row), yet there should be a few items per CTA to balance the
// load, as long as a chunk keeps at least 2048 vectors.
int flow_pick_chunks(long long units, int B, int gamma, long long nctas) {
    long long nch = (units + 8000) / 16000;
    if (nch < 1) nch = 1;
    if (nch > 8) nch = 8;
    const long long rows = static_cast<long long>(B) * (gamma + 1);
    while (nch < 8 && rows * nch < 4 * nctas && units / (nch + 1) >= 2048) ++nch;
    return static_cast<int>(nch);
}

using FKernelFn = void (*)(const Params, const FlowScratch);
static FKernelFn pick_flow(int dtype) {
    return dtype == kF32 ? verify_flow_kernel<kF32> : verify_flow_kernel<kBF16>;
}

static constexpr size_t kFlowSmem = sizeof(uint4) * kFDepth * kFThreads;

int flow_threads() { return kFAllThreads; }

int flow_max_ctas_per_sm(int dtype) {
    int n = 0;
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(pick_flow(dtype)),
                             cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kFlowSmem)) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pick_flow(dtype), kFAllThreads, kFlowSmem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t launch_flow(const Params& prm, const FlowScratch& fl_in, int dtype, int nctas, cudaStream_t stream) {
    const FlowScratch& fl = fl_in;
    pick_flow(dtype)<<<nctas, kFAllThreads, kFlowSmem, stream>>>(prm, fl);
    return cudaGetLastError();
}

}  // namespace bv
