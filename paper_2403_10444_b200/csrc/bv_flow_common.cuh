// Pieces shared by the kernels that run Block Verification (Algorithm 2) as a flow of work
// items (bv_flow.cu and the entry point without allocations): per-vector arithmetic, the rescan that turns a sampled mass
// into a token, the end of a row (normalisers, prefix recursion of Eq. "def_as"), the end of a
// position (S_r of Eq. "pacc_block" and the candidate of Eq. "pres-block") and the end of a
// block (h_i, tau, output).
#pragma once
#include "bv_device.cuh"
#include "bv_launch.h"

namespace bv {



enum : int { kExit = 0, kSweep1 = 1, kSweep2 = 2 };
// Global counters, one per 128-byte line so that polling one does not slow the others down:
// the sweep-1 ticket counter, rows queued for their second sweep, pieces of queued rows handed
// out, blocks finished, last target rows queued for their first sweep, chunks of those handed out.
// (and the number of CTAs that have left, by which the last one knows itself)
constexpr int kCounterWords = 224;
enum : int { kCtrTicket = 0, kCtrQueued = 32, kCtrPieces = 64, kCtrBlocks = 96, kCtrLateQueued = 128, kCtrLateChunks = 160, kCtrExited = 192 };
// rel[row]: 0 = not folded yet, then whether the row's second sweep is wanted
enum : unsigned { kRelSweep = 1u, kRelSkip = 2u, kRelHold = 3u, kRelLate = 4u };   // hold: wanted only if every higher
// candidate is rejected; late: the last target row, whose first sweep has only now been asked for

__device__ __forceinline__ unsigned ld_volatile(const unsigned* p) {
    return *reinterpret_cast<const volatile unsigned*>(p);
}

// ---- per-vector arithmetic; multiply-adds and additions are issued two lanes at a time
// (fma.rn.f32x2 / add.rn.f32x2), which halves their share of the instruction stream ----
__device__ __forceinline__ float2 f2(float x, float y) { return make_float2(x, y); }

// a_e = 2^{v_e k - M}
template <int EPV> __device__ __forceinline__ void f_exps(const float (&v)[EPV], float kf, float nM, float (&a)[EPV]) {
    const float2 kk = f2(kf, kf), mm = f2(nM, nM);
#pragma unroll
    for (int e = 0; e < EPV; e += 2) {
        const float2 x = __ffma2_rn(f2(v[e], v[e + 1]), kk, mm);
        a[e] = ex2(x.x);
        a[e + 1] = ex2(x.y);
    }
}
template <int EPV> __device__ __forceinline__ float f_sum(const float (&a)[EPV]) {
    float2 s = __fadd2_rn(f2(a[0], a[1]), f2(a[2], a[3]));
    if (EPV == 8) s = __fadd2_rn(s, __fadd2_rn(f2(a[4], a[5]), f2(a[6], a[7])));
    return s.x + s.y;
}
template <int EPV> __device__ __forceinline__ float f_exp_sum(const float (&v)[EPV], float kf, float nM) {
    float a[EPV];
    f_exps<EPV>(v, kf, nM, a);
    return f_sum<EPV>(a);
}
template <int EPV> __device__ __forceinline__ void f_accumulate(const float (&v)[EPV], float kf, float& M, float& s) {
    float vs = f_exp_sum<EPV>(v, kf, -M);
    if (__any_sync(0xffffffffu, vs > kRaiseBound)) {      // some logit lies above the reference
        const float y = rintf(warp_max(vec_max<EPV>(v)) * kf);
        if (y > M) { s *= ref_scale(M, y); M = y; }
        vs = f_exp_sum<EPV>(v, kf, -M);
    }
    s += vs;
}
// residual terms t_e = max(cp 2^{zP k - MP} - 2^{zQ k - MQ}, 0) and their sum; HAVEQ = false: t_e = cp 2^{zP k - MP}.
// PROBS: the rows hold probabilities, t_e = max(cp P_e - Q_e, 0) resp. cp P_e.
template <int EPV, bool HAVEQ, bool PROBS = false>
__device__ __forceinline__ float f_pair_sum(const float (&vp)[EPV], const float (&vq)[EPV], float kf, float cp,
                                            float nMP, float nMQ, float (&t)[EPV]) {
    float a[EPV], q[EPV];
    if (PROBS) {
#pragma unroll
        for (int e = 0; e < EPV; ++e) { a[e] = vp[e]; q[e] = vq[e]; }
    } else {
        f_exps<EPV>(vp, kf, nMP, a);
        if (HAVEQ) f_exps<EPV>(vq, kf, nMQ, q);
    }
    const float2 cc = f2(cp, cp), ncc = f2(-cp, -cp);
#pragma unroll
    for (int e = 0; e < EPV; e += 2) {
        if (HAVEQ) {
            // q - cp a in one packed multiply-add; the sign flips for free inside the max
            const float2 d = __ffma2_rn(ncc, f2(a[e], a[e + 1]), f2(q[e], q[e + 1]));
            t[e] = fmaxf(-d.x, 0.f);
            t[e + 1] = fmaxf(-d.y, 0.f);
        } else {
            const float2 d = __fmul2_rn(cc, f2(a[e], a[e + 1]));
            t[e] = d.x;
            t[e + 1] = d.y;
        }
    }
    return f_sum<EPV>(t);
}
template <int DT> __device__ __forceinline__ void f_load(const char* row, int i, float (&v)[Raw<DT>::EPV]) {
    Raw<DT>::unpack(ld_stream_v4(row + static_cast<size_t>(i) * 16), v);
}
template <int DT>
__device__ __forceinline__ void f_load_tail(const char* row, int i, int end, float (&v)[Raw<DT>::EPV]) {
    if (row != nullptr && i < end) {
        f_load<DT>(row, i, v);
    } else {
#pragma unroll
        for (int e = 0; e < Raw<DT>::EPV; ++e) v[e] = -INFINITY;
    }
}

// scratch written by other CTAs is always read through L2
__device__ __forceinline__ RowZ load_rowz(const RowZ* p) {
    RowZ z;
    z.MP = __ldcg(&p->MP); z.ZP = __ldcg(&p->ZP); z.MQ = __ldcg(&p->MQ); z.ZQ = __ldcg(&p->ZQ);
    return z;
}

// chunks of row r of a block in its first sweep
// (rows whose first sweep is asked for on demand - a last target row, a row of Algorithm 1 beyond the
// ones swept from the start - are cut into nch_late chunks)
// (and so are all rows of the blocks from fine_from on, the last ones to be started: the launch ends
// a chunk's sweep after its last ticket, so the last chunks are short ones)
__device__ __forceinline__ int f_nch_row(const FlowScratch& fl, int b, int r, int g) {
    return (r == g || b >= fl.fine_from || (fl.tv && r >= fl.tv_spec)) ? fl.nch_late : fl.nch;
}

struct FlowCtx {
    int g, V, B, units;
    size_t row_bytes;
    float kf;
    double kd;
};

// One warp walks segment [w0, w1) of a row pair in index order and returns the first element
// whose running residual mass exceeds tw (else the last element with positive mass, else -1).
template <int DT, bool PROBS = false, int kAhead = 4>      // kAhead: runs of 32 vectors whose loads are in flight together
__device__ int f_rescan(const char* rowP, const char* rowQ, int w0, int w1, int lane, float kf, float cp,
                        float nMP, float nMQ, double tw) {
    constexpr int EPV = Raw<DT>::EPV;
    constexpr uint32_t kPad = PROBS ? 0u : Raw<DT>::kNegInf;   // an element beyond the segment weighs nothing
    // The terms are the fp32 values of the sweeps; their running sum, which decides the token, is
    // kept in fp64 (a cell of the distribution can be far narrower than fp32 resolves next to the
    // mass before it).
    double run = 0.0;
    int found = -1, last_pos = -1;
    for (int base0 = w0; base0 < w1 && found < 0; base0 += 32 * kAhead) {
        // the loads of kAhead runs are issued before the first is looked at: the walk is a chain of
        // dependent steps, and a load's latency is what each step would otherwise wait for
        uint4 rp[kAhead], rq[kAhead];
#pragma unroll
        for (int a = 0; a < kAhead; ++a) {
            const int i = base0 + 32 * a + lane;
            const bool ok = i < w1;
            rp[a] = ok ? ld_stream_v4(rowP + static_cast<size_t>(i) * 16) : make_uint4(kPad, kPad, kPad, kPad);
            rq[a] = (ok && rowQ) ? ld_stream_v4(rowQ + static_cast<size_t>(i) * 16) : make_uint4(kPad, kPad, kPad, kPad);
        }
#pragma unroll
        for (int a = 0; a < kAhead; ++a) {
            const int base = base0 + 32 * a;
            if (base >= w1 || found >= 0) break;
            const int i = base + lane;
            float vp[EPV], vq[EPV], tt[EPV];
            Raw<DT>::unpack(rp[a], vp);
            Raw<DT>::unpack(rq[a], vq);
            if (rowQ) f_pair_sum<EPV, true, PROBS>(vp, vq, kf, cp, nMP, nMQ, tt);
            else f_pair_sum<EPV, false, PROBS>(vp, vq, kf, cp, nMP, nMQ, tt);
            double ls = 0.0;
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                ls += static_cast<double>(tt[e]);
                if (tt[e] > 0.f) last_pos = i * EPV + e;
            }
            double incw = ls;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const double o = shfl_up_d(incw, off);
                if (lane >= off) incw += o;
            }
            const unsigned bal = __ballot_sync(0xffffffffu, run + incw > tw && ls > 0.0);
            if (bal) {
                const int src = __ffs(bal) - 1;
                int f = -1;
                if (lane == src) {
                    double cum = run + incw - ls;
                    int lp = -1;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        cum += static_cast<double>(tt[e]);
                        if (tt[e] > 0.f) lp = i * EPV + e;
                        if (f < 0 && cum > tw && tt[e] > 0.f) f = i * EPV + e;
                    }
                    if (f < 0) f = lp;
                }
                found = __shfl_sync(0xffffffffu, f, src);
            }
            run += shfl_d(incw, 31);
        }
    }
    if (found < 0) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, off));
        found = last_pos;
    }
    return found;
}

// Acceptance weight of position 0 < i < gamma from p_i and S_i: Eq. "pacc_block",
// h_i = S_i / (S_i + 1 - p_i), and 0 for an empty residual.  Algorithm 4 prints its h_i as
// sum_x max(pt_i P_i - Q_i, 0) / sum_x max(Q_i - pt_i P_i, 0); both rows sum to one, so the second
// sum is the first plus 1 - pt_i and the same expression serves, with the unclipped product pt_i:
// for pt_i >= 1 the denominator is at most S_i (the test passes whatever the uniform), and a
// denominator that is not positive gives +inf.
__device__ __forceinline__ double f_weight(double pi, double Si) {
    if (!(Si > 0.0)) return 0.0;
    const double den = Si + 1.0 - pi;
    return den > 0.0 ? Si / den : INFINITY;
}

// With diagnostic outputs every position is computed in full.
__device__ __forceinline__ bool f_all_positions(const Params& prm) {
    return prm.out_p || prm.out_S || prm.out_h || prm.out_lse_t || prm.out_lse_d;
}

// ---- the end of a block (one warp; lanes i and i + 32 speak for positions i and i + 32, position
// gamma is handled by every lane alike): Eq. "pacc_block", selection of tau, output ----
static __device__ void f_finalize_block(const Params& prm, const FlowScratch& fl, int b, int lane) {
    const int g = prm.gamma;
    __threadfence();
    int32_t* ot = prm.out_tokens + static_cast<size_t>(b) * (g + 1);
    const int32_t* X = prm.tok + static_cast<size_t>(b) * g;
    const float* u = prm.uni + static_cast<size_t>(b) * (g + 2);
    const double* p = fl.pchain + static_cast<size_t>(b) * (g + 2);
    const double* S = fl.S + static_cast<size_t>(b) * (g + 1);
    const int* cand = fl.cand + static_cast<size_t>(b) * (g + 1);
    // everything asked for in one go
    double pi[2], Si[2];
    float eta[2];
    int cd[2], xi[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int i = lane + 32 * h;
        const bool in = i < g;
        pi[h] = in ? __ldcg(&p[i]) : 0.0;
        Si[h] = in ? __ldcg(&S[i]) : 0.0;
        cd[h] = in ? __ldcg(&cand[i]) : -1;
        eta[h] = (in && i >= 1) ? u[i - 1] : 2.f;
        xi[h] = in ? X[i] : -1;
    }
    const double p_g = __ldcg(&p[g]);
    const int cand_g = __ldcg(&cand[g]);
    const float eta_g = u[g - 1];
    const bool bad = ld_volatile(&fl.bad[b]) != 0;
    // h_gamma = p_gamma; h_i = S_i / (S_i + 1 - p_i); tau = max{i >= 1 : h_i > 0 and eta_i <= h_i}, else 0
    double hw[2];
    bool pass[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int i = lane + 32 * h;
        hw[h] = i == 0 ? 1.0 : f_weight(pi[h], Si[h]);
        pass[h] = i >= 1 && i < g && hw[h] > 0.0 && static_cast<double>(eta[h]) <= hw[h];
    }
    const unsigned m_lo = __ballot_sync(0xffffffffu, pass[0]), m_hi = __ballot_sync(0xffffffffu, pass[1]);
    int tau = 0;
    if (p_g > 0.0 && static_cast<double>(eta_g) <= p_g) tau = g;
    else if (m_hi) tau = 32 + 31 - __clz(m_hi);
    else if (m_lo) tau = 31 - __clz(m_lo);
    if (bad) tau = -1;
    int y = cand_g;                       // the candidate of position tau
    if (tau >= 0 && tau < g) y = __shfl_sync(0xffffffffu, tau < 32 ? cd[0] : cd[1], tau & 31);
    // Nothing to sample from at the selected position (an empty residual, which the algorithm cannot
    // select: P_tau == Q_tau makes position tau + 1 pass its test): a domain error of the block
    if (tau >= 0 && y < 0) tau = -1;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int i = lane + 32 * h;
        if (i < g) ot[i] = i < tau ? xi[h] : (i == tau ? y : -1);
    }
    if (lane == 0) {
        ot[g] = tau == g ? y : -1;
        prm.out_len[b] = tau >= 0 ? tau + 1 : -1;
    }
    if (f_all_positions(prm)) {
        const double ln2 = 0.693147180559945309417232;
        for (int i = lane; i <= g; i += 32) {
            const size_t o1 = static_cast<size_t>(b) * (g + 1) + i, o0 = static_cast<size_t>(b) * g + i;
            const double pv = i == g ? p_g : (i < 32 ? pi[0] : pi[1]);
            const double Sv = i == g ? 0.0 : (i < 32 ? Si[0] : Si[1]);
            const double h = (i == 0) ? 1.0 : (i == g ? pv : f_weight(pv, Sv));
            const RowZ z = load_rowz(&fl.rowZ[static_cast<size_t>(b) * (g + 1) + i]);
            if (prm.out_p) prm.out_p[o1] = static_cast<float>(pv);
            if (prm.out_h) prm.out_h[o1] = static_cast<float>(h);
            if (prm.out_lse_t) prm.out_lse_t[o1] = static_cast<float>((static_cast<double>(z.MP) + log2(z.ZP)) * ln2);
            if (i < g && prm.out_S) prm.out_S[o0] = static_cast<float>(Sv);
            if (i < g && prm.out_lse_d) prm.out_lse_d[o0] = static_cast<float>((static_cast<double>(z.MQ) + log2(z.ZQ)) * ln2);
        }
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(&fl.counters[kCtrBlocks], 1u);      // (CTAs leave when every block is finished)
}

// Is the GPU emptying, so that a block's candidates are all started at once?  It is when the
// first-sweep tickets have run out and little is left in the two queues as well (fewer pieces than a
// quarter of the CTAs).  With a good draft nearly every position is a candidate and the second
// sweeps are half of the launch: there the queues stay full long after the last ticket, and
// sweeping all candidates of every block would double the traffic for nothing (measured: 13 % of
// the time at B = 256, gamma = 8 with a draft that is accepted 7 times in 8).
// A launch on probabilities has no first sweep; it says which way it wants it.
__device__ __forceinline__ bool f_tail(const FlowScratch& fl) {
    if (fl.tail_mode) return fl.tail_mode == 1;
    if (ld_volatile(&fl.counters[kCtrTicket]) < fl.total_s1) return false;
    const unsigned q = ld_volatile(&fl.counters[kCtrQueued]), p = ld_volatile(&fl.counters[kCtrPieces]);
    const unsigned lq = ld_volatile(&fl.counters[kCtrLateQueued]), lc = ld_volatile(&fl.counters[kCtrLateChunks]);
    // (the heads may run ahead of the tails by tickets drawn early: a negative backlog is an empty queue)
    const long long backlog = (static_cast<long long>(q) * fl.np - p) + (static_cast<long long>(lq) * fl.nch_late - lc);
    return backlog < static_cast<long long>(gridDim.x / 4);
}

// Is the token of position gamma drawn from the first sweep of the last target row (bv_flow.cu)?
__device__ __forceinline__ bool f_draws_in_sweep1(const Params& prm, int nch_late) {
    return !f_all_positions(prm) && nch_late <= 8;
}

// ---- second sweeps that start together: the positions in `mask` (bit c = position c; mask_hi:
// position c + 32) take consecutive places in the queue from which every CTA draws pieces (one warp) ----
static __device__ void f_queue_rows(const FlowScratch& fl, int b, int g, unsigned mask, unsigned mask_hi, int lane) {
    const int n_lo = __popc(mask), n = n_lo + __popc(mask_hi);
    if (n == 0) return;
    unsigned slot = 0;
    if (lane == 0) slot = atomicAdd(&fl.counters[kCtrQueued], static_cast<unsigned>(n));
    slot = __shfl_sync(0xffffffffu, slot, 0);
    // the entry itself says when it is written (the queue starts at zero)
    if (mask >> lane & 1u)
        atomicExch(&fl.s2q[slot + __popc(mask & ((1u << lane) - 1u))], static_cast<unsigned>(b * (g + 1) + lane) + 1u);
    if (mask_hi >> lane & 1u)
        atomicExch(&fl.s2q[slot + n_lo + __popc(mask_hi & ((1u << lane) - 1u))], static_cast<unsigned>(b * (g + 1) + lane + 32) + 1u);
}

// Which of the candidates on hold (bit c = position c < 32, hold_hi: c + 32) are swept next.  The
// selected position is the highest candidate that passes its test, so the candidates are swept from
// the top, one at a time; position 0, what remains when no other is selected, last.  Once the
// GPU is emptying (f_tail) a block's chain of candidates, one after
// the other, would only prolong the launch: then all of them are started at once, position 0
// included (one that turns out not to be needed costs bandwidth nobody else wants).
__device__ __forceinline__ void f_pick_next(unsigned hold_lo, unsigned hold_hi, bool tail, unsigned& s_lo, unsigned& s_hi) {
    s_lo = 0; s_hi = 0;
    const unsigned c_lo = hold_lo & ~1u;                     // candidates other than position 0
    if (tail || (c_lo | hold_hi) == 0u) { s_lo = hold_lo; s_hi = hold_hi; }
    else if (hold_hi) s_hi = 1u << (31 - __clz(hold_hi));
    else s_lo = 1u << (31 - __clz(c_lo));
}

// ---- position i of a block is complete: S_i and its candidate token are in scratch (one warp).
// Without diagnostics: if it passes its test, tau >= i whatever the higher candidates do, and no lower
// position is wanted; if not, the next lower candidate is started.  A position on hold changes
// state exactly once, whoever gets there first (positions of one block may complete side by side
// once several candidates are swept at a time).  The warp that completes a block's last position
// ends the block. ----
static __device__ void f_position_done(const Params& prm, const FlowScratch& fl, int b, int i, int lane) {
    const int g = prm.gamma;
    const size_t row0 = static_cast<size_t>(b) * (g + 1);
    unsigned done = 1;
    if (!f_all_positions(prm)) {
        __threadfence();
        // everything asked for in one go
        unsigned rl[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = lane + 32 * h;
            rl[h] = c < i && c < g ? ld_volatile(&fl.rel[row0 + c]) : 0u;
        }
        const double p_i = __ldcg(&fl.pchain[static_cast<size_t>(b) * (g + 2) + i]);
        const double S_i = i < g ? __ldcg(&fl.S[row0 + i]) : 0.0;
        const float eta_i = i >= 1 ? prm.uni[static_cast<size_t>(b) * (g + 2) + i - 1] : 0.f;
        const bool tail = f_tail(fl);
        const double hw = i == g ? p_i : f_weight(p_i, S_i);
        const bool selected = i == 0 || (hw > 0.0 && static_cast<double>(eta_i) <= hw);
        const unsigned hold_lo = __ballot_sync(0xffffffffu, rl[0] == kRelHold), hold_hi = __ballot_sync(0xffffffffu, rl[1] == kRelHold);
        unsigned s_lo = hold_lo, s_hi = hold_hi;             // selected: every lower candidate is dropped
        if (!selected) f_pick_next(hold_lo, hold_hi, tail, s_lo, s_hi);
        bool won[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = lane + 32 * h;
            won[h] = ((h ? s_hi : s_lo) >> lane & 1u) && atomicCAS(&fl.rel[row0 + c], kRelHold, selected ? kRelSkip : kRelSweep) == kRelHold;
            if (won[h] && selected) { fl.S[row0 + c] = 0.0; fl.cand[row0 + c] = -1; }
        }
        const unsigned w_lo = __ballot_sync(0xffffffffu, won[0]), w_hi = __ballot_sync(0xffffffffu, won[1]);
        if (selected) done += static_cast<unsigned>(__popc(w_lo) + __popc(w_hi));
        else { __threadfence(); f_queue_rows(fl, b, g, w_lo, w_hi, lane); }
    }
    __threadfence();
    unsigned n = 0;
    if (lane == 0) n = atomicAdd(&fl.cand_cnt[b], done);
    n = __shfl_sync(0xffffffffu, n, 0);
    if (n + done == static_cast<unsigned>(g) + 1u) f_finalize_block(prm, fl, b, lane);
}

// ================= Token Verification (Algorithm 1) on the same work items =================
// Row r feeds one acceptance test, eta_{r+1} <= min(P_r(X_{r+1}) / Q_r(X_{r+1}), 1), which needs that
// row's normalisers only; tau is the number of tests that pass before the first one that fails, and
// Y is drawn from Eq. "pres-token" at position tau (one second sweep of that row pair with p = 1), or
// from P_gamma.  Rows 0 .. tv_spec-1 of every block are swept from the start; a further row is
// asked for when every test before it has passed, so no row beyond the first rejection is read
// unless it was among the first ones.

// ---- the end of a block of Algorithm 1 (one warp): X_1 .. X_tau, Y, diagnostics ----
static __device__ void f_tv_finalize(const Params& prm, const FlowScratch& fl, int b, int tau, int lane) {
    const int g = prm.gamma;
    __threadfence();
    const size_t row0 = static_cast<size_t>(b) * (g + 1);
    int32_t* ot = prm.out_tokens + static_cast<size_t>(b) * (g + 1);
    const int32_t* X = prm.tok + static_cast<size_t>(b) * g;
    const int y = __ldcg(&fl.cand[row0 + tau]);
    const unsigned long long badrows = *reinterpret_cast<const volatile unsigned long long*>(&fl.tv_badrows[b]);
    const int last_pair = tau < g ? tau : g - 1;             // row pairs 0 .. last_pair were needed
    bool bad = (badrows & (last_pair >= 63 ? ~0ull : ((2ull << last_pair) - 1ull))) != 0ull;
    if (tau == g && ld_volatile(&fl.bad[b]) != 0u) bad = true;
    if (y < 0) bad = true;                // (nothing to sample from: Algorithm 1 cannot stop where P_tau == Q_tau)
    for (int i = lane; i <= g; i += 32) ot[i] = bad ? -1 : (i < tau ? X[i] : (i == tau ? y : -1));
    if (lane == 0) prm.out_len[b] = bad ? -1 : tau + 1;
    if (f_all_positions(prm)) {
        const double ln2 = 0.693147180559945309417232;
        const float nanf_ = __int_as_float(0x7fc00000);
        for (int i = lane; i <= g; i += 32) {
            const size_t o1 = row0 + i, o0 = static_cast<size_t>(b) * g + i;
            const bool read_t = i <= tau, read_d = i <= last_pair;
            const RowZ z = load_rowz(&fl.rowZ[row0 + i]);
            // h_i = min(ratio_i, 1) for the tests made: i = 1 .. min(tau + 1, gamma)
            float h = nanf_;
            if (i == 0) h = 1.f;
            else if (i <= tau + 1 && i <= g) h = static_cast<float>(fmin(__ldcg(&fl.ratio[row0 + i - 1]), 1.0));
            if (prm.out_p) prm.out_p[o1] = nanf_;
            if (prm.out_h) prm.out_h[o1] = h;
            if (prm.out_lse_t) prm.out_lse_t[o1] = read_t ? static_cast<float>((static_cast<double>(z.MP) + log2(z.ZP)) * ln2) : nanf_;
            if (i < g && prm.out_S) prm.out_S[o0] = i == tau ? static_cast<float>(__ldcg(&fl.S[row0 + i])) : nanf_;
            if (i < g && prm.out_lse_d) prm.out_lse_d[o0] = read_d ? static_cast<float>((static_cast<double>(z.MQ) + log2(z.ZQ)) * ln2) : nanf_;
        }
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(&fl.counters[kCtrBlocks], 1u);
}

// ---- row r of a block of Algorithm 1 is complete, its normalisers and ratio published (one warp) ----
template <int DT>
__device__ void f_tv_row_done(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int b, int r, int lane) {
    const int g = cx.g;
    const size_t row0 = static_cast<size_t>(b) * (g + 1);
    if (lane == 0 && r < g) {
        const double ratio = __ldcg(&fl.ratio[row0 + r]);     // 0 for a row with a data fault: the test fails
        const double h = fmin(ratio, 1.0);
        const bool pass = h > 0.0 && static_cast<double>(prm.uni[static_cast<size_t>(b) * (g + 2) + r]) <= h;
        // the decision first, then the fact that it is in: whoever sees the second sees the first
        if (pass) atomicOr(&fl.tv_acc[b], 1ull << r);
        __threadfence();
        atomicOr(&fl.tv_done[b], 1ull << r);
        __threadfence();
        const unsigned long long a = *reinterpret_cast<const volatile unsigned long long*>(&fl.tv_acc[b]);
        const unsigned long long dn = *reinterpret_cast<const volatile unsigned long long*>(&fl.tv_done[b]);
        int f = a == ~0ull ? 64 : __ffsll(static_cast<long long>(~a)) - 1;   // tests 1 .. f have passed
        if (f > g) f = g;
        if (f == g || (dn >> f & 1ull)) {
            // tau = f: every test has passed, or test f + 1 has been made and failed.  The warp whose
            // update completes the picture sees it; several may, one acts.
            if (atomicCAS(&fl.tv_decided[b], 0u, 1u) == 0u) {
                fl.tv_tau[b] = f;
                if (f == g) {             // Y ~ P_gamma: the last target row is asked for
                    const unsigned slot = atomicAdd(&fl.counters[kCtrLateQueued], 1u);
                    atomicExch(&fl.lq[slot], static_cast<unsigned>(row0 + g) + 1u);
                } else {                  // Y from Eq. "pres-token": one second sweep of row pair f with p = 1
                    fl.cscale[row0 + f] = static_cast<float>(__ldcg(&fl.zratio[row0 + f]));
                    __threadfence();
                    const unsigned slot = atomicAdd(&fl.counters[kCtrQueued], 1u);
                    atomicExch(&fl.s2q[slot], static_cast<unsigned>(row0 + f) + 1u);
                }
            }
        } else {
            // Every test before row f has passed.  Once that includes all the rows swept from the start,
            // rows up to f + tv_ahead - 1 are asked for, those of them that have not been yet (tv_ahead
            // is 1 when one row of every block fills the GPU, so that nothing beyond the first rejection
            // is read; all the rest for small batches, whose chain of dependent rows would otherwise
            // leave most of the GPU idle).
            // (a block that has passed two tests or more is likely to pass more, and such blocks are few
            // unless the draft is good: it asks for as many rows again as it has passed, which halves
            // the chain of its dependent rows at the price of at most as many rows read in vain)
            const int ahead = fl.tv_ahead > f ? fl.tv_ahead : (f >= 2 ? f : 1);
            int want = f >= fl.tv_spec ? f + ahead : 0;       // (rows from the start that are still out: nothing yet)
            if (want > g) want = g;
            want -= fl.tv_spec;
            for (int tries = 0; tries < 64 && want > 0; ++tries) {
                const unsigned have = ld_volatile(&fl.tv_front[b]);
                if (have >= static_cast<unsigned>(want)) break;
                if (atomicCAS(&fl.tv_front[b], have, static_cast<unsigned>(want)) != have) continue;
                const unsigned n = static_cast<unsigned>(want) - have;
                const unsigned slot = atomicAdd(&fl.counters[kCtrLateQueued], n);
                for (unsigned j = 0; j < n; ++j)
                    atomicExch(&fl.lq[slot + j], static_cast<unsigned>(row0 + fl.tv_spec + have + j) + 1u);
                break;
            }
        }
    }
    __syncwarp();
}

// ---- all rows 0 .. gamma-1 of a block have their normalisers: the prefix recursion
// p_{c+1} = min(p_c ratio_c, 1) (Eq. "def_as"; Algorithm 4 does not clip), what becomes of every
// position's second sweep, and the start of the first ones (one warp; lanes c and c + 32 speak for
// positions c and c + 32) ----
template <int DT>
__device__ void f_fold_block(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int b, int lane) {
    const int g = cx.g;
    const bool all_positions = f_all_positions(prm);
    __threadfence();
    const size_t row0 = static_cast<size_t>(b) * (g + 1);
    const float* u = prm.uni + static_cast<size_t>(b) * (g + 2);
    // everything this warp needs from global memory, asked for in one go
    double rat[2], zr[2];
    float eta[2];                         // the uniform that position c is tested with: eta_c = uniforms[c - 1]
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        rat[h] = c < g ? __ldcg(&fl.ratio[row0 + c]) : 1.0;
        zr[h] = c < g ? __ldcg(&fl.zratio[row0 + c]) : 1.0;
        eta[h] = (c >= 1 && c < g) ? u[c - 1] : 0.f;
    }
    const float eta_g = u[g - 1];
    const bool tail = f_tail(fl);
    // the recursion, by every lane alike; a lane keeps the p of its own positions
    double pc = 1.0, mine[2] = {1.0, 1.0};
    for (int c = 0; c < g; ++c) {
        if ((c & 31) == lane) mine[c >> 5] = pc;
        const double r = shfl_d(c < 32 ? rat[0] : rat[1], c & 31);
        const double next = pc * r;
        pc = prm.greedy ? next : fmin(next, 1.0);
    }
    const double p_g = pc;
    // Does anything depend on a position's second sweep?  S_c <= p_c (the residual mass of
    // Eq. "pacc_block" is at most p_c sum_x P_c(x)), hence h_c <= p_c: a position whose uniform
    // lies above p_c can never be the selected one, and nobody will ask for its S_c or its
    // candidate.  Position gamma is selected iff eta_gamma <= h_gamma = p_gamma, and only then is the
    // last target row read and the sample from P_gamma drawn.  Position 0 is what remains when no other
    // is selected.  (The margin keeps a uniform within rounding of p_c on the long path; with
    // diagnostic outputs every position is computed.)  The unclipped product of Algorithm 4 obeys
    // the same bound while it is at most one; above one the position passes its test whatever the
    // uniform, and the comparison below makes it a candidate.
    double* p = fl.pchain + static_cast<size_t>(b) * (g + 2);
    bool need[2] = {false, false};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        if (c < g) {
            const size_t ci = row0 + c;
            p[c] = mine[h];
            need[h] = all_positions || c == 0 || static_cast<double>(eta[h]) <= mine[h] * (1.0 + 1e-6);
            fl.cscale[ci] = static_cast<float>(mine[h] * zr[h]);
            if (!need[h]) { fl.S[ci] = 0.0; fl.cand[ci] = -1; }
        }
    }
    const bool last_row_wanted = all_positions || static_cast<double>(eta_g) <= p_g * (1.0 + 1e-6);
    if (lane == 0) {
        p[g] = p_g;
        if (!last_row_wanted) fl.cand[row0 + g] = -1;
    }
    const unsigned m_lo = __ballot_sync(0xffffffffu, need[0]), m_hi = __ballot_sync(0xffffffffu, need[1]);
    // Which second sweeps start now.  With diagnostics: all of them.  Otherwise the selected position
    // is the highest candidate that passes its test, so the candidates are swept from the top, one
    // at a time: position gamma first if it is one (its row joins the queue of last target rows),
    // else the highest candidate below; position 0 only when it is alone.  Once the GPU is
    // emptying (f_tail) a block's chain of candidates, one after the
    // other, would only prolong the launch: then all of them are started at once (a lower one that
    // turns out not to be needed costs bandwidth nobody else wants).
    unsigned s_lo = 0, s_hi = 0;
    if (all_positions) { s_lo = m_lo; s_hi = m_hi; }
    else if (tail || !last_row_wanted) f_pick_next(m_lo, m_hi, tail, s_lo, s_hi);   // (emptying GPU: alongside the last target row)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        if (c < g) {
            const bool started = ((h ? s_hi : s_lo) >> lane & 1u) != 0u;
            fl.rel[row0 + c] = started ? kRelSweep : (need[h] ? kRelHold : kRelSkip);
        }
    }
    if (lane == 0) fl.rel[row0 + g] = last_row_wanted ? (prm.probs ? kRelSweep : kRelLate) : kRelSkip;
    __threadfence();
    __syncwarp();
    f_queue_rows(fl, b, g, s_lo, s_hi, lane);
    if (lane == 0) {
        if (last_row_wanted && prm.probs) {
            // (given probabilities there is no normaliser to learn: P_gamma is swept once, as a position like the others)
            const unsigned slot = atomicAdd(&fl.counters[kCtrQueued], 1u);
            atomicExch(&fl.s2q[slot], static_cast<unsigned>(row0 + g) + 1u);
        } else if (last_row_wanted) {     // the last target row joins the queue of its kind
            const unsigned slot = atomicAdd(&fl.counters[kCtrLateQueued], 1u);
            atomicExch(&fl.lq[slot], static_cast<unsigned>(row0 + g) + 1u);
        }
        // skipped positions count as complete (position 0 never is, so the block cannot end here)
        const unsigned nskip = static_cast<unsigned>(g - __popc(m_lo) - __popc(m_hi)) + (last_row_wanted ? 0u : 1u);
        if (nskip > 0) atomicAdd(&fl.cand_cnt[b], nskip);
    }
    __syncwarp();
}

// ---- a row is complete (one warp): its chunks are combined (fp64) and its normalisers
// published, for r < gamma with the ratio P_r(X_{r+1}) / Q_r(X_{r+1}) of the drafted token ----
template <int DT>
__device__ void f_row_complete(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int b, int r, int lane) {
    const int g = cx.g;
    const size_t rowi = static_cast<size_t>(b) * (g + 1) + r;
    const int nch = f_nch_row(fl, b, r, g);
    const bool have_q = r < g;
    // loads in flight together: the chunks' sums, the drafted token
    RowZ z; z.MP = kNoRef; z.ZP = 0.0; z.MQ = kNoRef; z.ZQ = 0.0;
    if (lane < nch) z = load_rowz(&fl.part[rowi * fl.part_stride + lane]);
    int x = (lane == 31 && have_q) ? prm.tok[static_cast<size_t>(b) * g + r] : 0;
    x = __shfl_sync(0xffffffffu, x, 31);
    const bool xok = have_q && x >= 0 && x < cx.V;
    const char* rowP = static_cast<const char*>(prm.tgt) + rowi * cx.row_bytes;
    const char* rowQ = static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + (have_q ? r : 0)) * cx.row_bytes;
    double zl = 0.0;                      // the two logits of the drafted token (lanes 0 and 1)
    if (xok && lane < 2) zl = load_logit<DT>(lane == 0 ? rowP : rowQ, x);
    // row reference = max of the chunk references (integers, exact as floats), then the scaled sums
    const float MPf = warp_max(static_cast<float>(z.MP)), MQf = warp_max(static_cast<float>(z.MQ));
    double ZP = z.ZP * static_cast<double>(ref_scale(static_cast<float>(z.MP), MPf));
    double ZQ = z.ZQ * static_cast<double>(ref_scale(static_cast<float>(z.MQ), MQf));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { ZP += shfl_xor_d(ZP, off); ZQ += shfl_xor_d(ZQ, off); }
    const double zp = shfl_d(zl, 0), zq = shfl_d(zl, 1);
    if (lane == 0) {
        double MP = MPf, MQ = MQf;
        if (prm.lse_d != nullptr && have_q) {
            // the draft row's normaliser is supplied: as an integer reference at or above every scaled
            // logit of the row plus a sum in [2^-1/2, 2^1/2]; a value that is not finite leaves the
            // row without a reference, which marks the block as faulty below
            const double L2 = static_cast<double>(prm.lse_d[static_cast<size_t>(b) * g + r]) * 1.4426950408889634073599246810019;
            const bool fin = L2 > -1e300 && L2 < 1e300;
            MQ = fin ? rint(L2) : static_cast<double>(kNoRef);
            ZQ = fin ? exp2(L2 - MQ) : 0.0;
        }
        RowZ out; out.MP = MP; out.ZP = ZP; out.MQ = MQ; out.ZQ = ZQ;
        fl.rowZ[rowi] = out;
        // the row's maximum is finite iff its reference is; Z is NaN / inf iff the row holds a NaN / overflowed
        bool bad = !(MP > kNoRef && MP < INFINITY) || !(ZP < INFINITY);
        if (have_q) {
            bad = bad || !(MQ > kNoRef && MQ < INFINITY) || !(ZQ < INFINITY) || !xok || zq == -INFINITY;
            // ratio = P_r(X_{r+1}) / Q_r(X_{r+1}) from the two logits of the drafted token
            fl.ratio[rowi] = bad ? 0.0 : exp2((zp - zq) * cx.kd - (MP - MQ)) * (ZQ / ZP);
            fl.zratio[rowi] = ZQ / ZP;
        }
        if (bad) {
            // (Algorithm 1 reads rows 0 .. tau only: a fault counts if its row is among them)
            if (fl.tv && have_q) atomicOr(&fl.tv_badrows[b], 1ull << r);
            else atomicOr(&fl.bad[b], 1u);
        }
    }
    __threadfence();
    __syncwarp();
}

// ---- a launch on given probabilities (one warp per block, at the start of the launch): the ratios
// P_r(X_{r+1}) / Q_r(X_{r+1}) are read off the rows, no row needs a first sweep.  Algorithm 2: the block is
// folded at once.  Algorithm 1: tau is known at once, and the one position to sample from is queued. ----
template <int DT>
__device__ void f_probs_start(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int b, int lane) {
    const int g = cx.g;
    const size_t row0 = static_cast<size_t>(b) * (g + 1);
    bool okrow[2] = {true, true};
    double rat[2] = {0.0, 0.0};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = lane + 32 * h;
        if (r < g) {
            const int x = prm.tok[static_cast<size_t>(b) * g + r];
            bool ok = x >= 0 && x < cx.V;
            double P = 0.0, Q = 1.0;
            if (ok) {
                P = load_logit<DT>(static_cast<const char*>(prm.tgt) + (row0 + r) * cx.row_bytes, x);
                Q = load_logit<DT>(static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes, x);
                ok = Q > 0.0 && Q < static_cast<double>(INFINITY) && P >= 0.0 && P < static_cast<double>(INFINITY);
            }
            okrow[h] = ok;
            rat[h] = ok ? P / Q : 0.0;
            fl.ratio[row0 + r] = rat[h];
            fl.zratio[row0 + r] = 1.0;
        }
        if (r <= g) { RowZ z; z.MP = 0.0; z.ZP = 1.0; z.MQ = 0.0; z.ZQ = 1.0; fl.rowZ[row0 + r] = z; }
    }
    const unsigned bad_lo = __ballot_sync(0xffffffffu, !okrow[0]), bad_hi = __ballot_sync(0xffffffffu, !okrow[1]);
    if (!fl.tv) {
        if (lane == 0 && (bad_lo | bad_hi)) atomicOr(&fl.bad[b], 1u);
        __threadfence();
        __syncwarp();
        f_fold_block<DT>(prm, fl, cx, b, lane);
        return;
    }
    // Algorithm 1: tests 1 .. gamma in order, test r + 1 on row r; tau = the number passed before the first failure
    bool pass[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = lane + 32 * h;
        const double hw = fmin(rat[h], 1.0);
        pass[h] = r >= g || (hw > 0.0 && static_cast<double>(prm.uni[static_cast<size_t>(b) * (g + 2) + r]) <= hw);
    }
    const unsigned f_lo = __ballot_sync(0xffffffffu, !pass[0]), f_hi = __ballot_sync(0xffffffffu, !pass[1]);
    const int tau = f_lo ? __ffs(f_lo) - 1 : (f_hi ? 32 + __ffs(f_hi) - 1 : g);
    if (lane == 0) {
        // (a fault counts if its row is among the ones Algorithm 1 reads: rows 0 .. min(tau, gamma - 1))
        const unsigned long long badrows = static_cast<unsigned long long>(bad_lo) | (static_cast<unsigned long long>(bad_hi) << 32);
        if (badrows) atomicOr(&fl.tv_badrows[b], badrows);
        fl.tv_tau[b] = tau;
        fl.cscale[row0 + tau] = 1.f;
        __threadfence();
        const unsigned slot = atomicAdd(&fl.counters[kCtrQueued], 1u);
        atomicExch(&fl.s2q[slot], static_cast<unsigned>(row0 + tau) + 1u);
    }
    __syncwarp();
}

// ---- a position is complete (one warp): S_r from the segment totals, and the candidate Y_r.
// `segs` holds the nseg <= 128 totals of the row's segments in index order (four per lane);
// range(s, v0, v1) gives the vectors [v0, v1) of segment s. ----
template <int DT, bool PROBS = false, class RangeFn>
__device__ void f_position_complete(const Params& prm, const FlowScratch& fl, const FlowCtx& cx, int ri, bool have_q,
                                    const char* rowP, const char* rowQ, float cp, float nMP, float nMQ,
                                    int nseg, const double* segs, int lane, RangeFn range) {
    const int g = cx.g, r = ri % (g + 1), b = ri / (g + 1);
    __threadfence();
    // everything asked for in one go: the uniform, the segment totals, the draft row's normaliser
    const float uf = prm.uni[static_cast<size_t>(b) * (g + 2) + (have_q ? g : g + 1)];
    double w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i = 4 * lane + j;
        w[j] = i < nseg ? __ldcg(&segs[i]) : 0.0;
    }
    const double ZQ = have_q ? __ldcg(&fl.rowZ[ri].ZQ) : 1.0;
    // S_r, and the segment that holds the sample, by fp64 sums of the segment totals in index order
    const double d1 = w[0], d2 = d1 + w[1], d3 = d2 + w[2], d4 = d3 + w[3];
    double inc = d4;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double o = shfl_up_d(inc, off);
        if (lane >= off) inc += o;
    }
    const double total = shfl_d(inc, 31);
    if (lane == 0 && have_q) fl.S[ri] = total / ZQ;
    int found = -1;
    if (total > 0.0 && total < static_cast<double>(INFINITY)) {
        const double t = static_cast<double>(uf) * total;
        double exc = shfl_up_d(inc, 1);
        if (lane == 0) exc = 0.0;
        const double p0 = exc, p1 = exc + d1, p2 = exc + d2, p3 = exc + d3, p4 = exc + d4;
        // first non-empty segment whose inclusive prefix exceeds t, else the last non-empty one
        const bool h1 = p1 > t && w[0] > 0.0, h2 = p2 > t && w[1] > 0.0;
        const bool h3 = p3 > t && w[2] > 0.0, h4 = p4 > t && w[3] > 0.0;
        const unsigned hit = __ballot_sync(0xffffffffu, h1 || h2 || h3 || h4);
        const unsigned nz = __ballot_sync(0xffffffffu, d4 > 0.0);
        int e = 3, src;
        double bef = p3;
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
        range(sel, s0, s1);
        found = f_rescan<DT, PROBS>(rowP, rowQ, s0, s1, lane, cx.kf, cp, nMP, nMQ, t - before);
    }
    // (an empty residual leaves no candidate: the position cannot be the selected one, see the end of a block)
    if (lane == 0) fl.cand[ri] = found;
    __syncwarp();
    if (fl.tv) f_tv_finalize(prm, fl, b, r, lane);
    else f_position_done(prm, fl, b, r, lane);
}

}  // namespace bv
