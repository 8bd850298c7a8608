// Block Verification (Algorithm 2, also with supplied draft normalisers), Greedy Block Verification
// (Algorithm 4) and Token Verification (Algorithm 1) for batches so small that a launch is a matter
// of latency, not of bandwidth (a few sequences: the whole input fits in L2).
//
// The flow kernel hands work from CTA to CTA through queues and counters in global memory, and a
// sequence goes through a dozen such hand-overs of a microsecond or more each.  Here all CTAs of a
// cooperative launch walk through three phases separated by two grid-wide barriers:
//   1. every row (all 2 gamma + 1 of every sequence, whether the algorithm will want them or not:
//      the bytes are few) is cut into chunks and every CTA reduces its chunks to {reference, sum};
//   2. every CTA combines all chunks (fp64) and runs the scalar part for every sequence itself -
//      normalisers, ratios of the drafted tokens, the recursion of Eq. "def_as" or the tests of
//      Algorithm 1, and which positions can be the selected one - so that all CTAs know the same
//      list of (position, piece) items without talking to each other; each takes its share and
//      leaves per-segment sums of the residual terms max(p_i P_i - Q_i, 0) (rows now come from L2);
//   3. one CTA per sequence: S_i and h_i (Eq. "pacc_block") of the candidates from the top down, tau,
//      and the token by inverse CDF over the segment sums and a rescan of one segment.
// Arithmetic, sampling convention and outputs are those of the flow kernel.
#include <cooperative_groups.h>

#include "bv_flow_common.cuh"

namespace bv {

constexpr int kSmThreads = 512;       // streaming threads; one more warp fetches the scalars while they stream
constexpr int kSmWarps = kSmThreads / 32;
constexpr int kSmAllThreads = kSmThreads + 32;
constexpr int kSmMaxRows = 1056;      // rows B (2 gamma + 1) whose normalisers a CTA keeps in shared memory
constexpr int kSmMaxPos = 560;        // positions B (gamma + 1)
constexpr int kSmInFlight = 8;        // 16-byte loads a thread has in flight in the first phase
constexpr int kSmPairsInFlight = 5;   // pairs of them in the second
constexpr int kSmMaxUni = kSmMaxPos + kSmallMaxB;   // uniforms B (gamma + 2)

struct SmallShared {
    float rowM[kSmMaxRows];
    double rowZ[kSmMaxRows];
    double pch[kSmMaxPos];            // p_i of every position (Algorithm 1: unused)
    float csc[kSmMaxPos];             // p_i Z_Q / Z_P: the scale of the target terms against the draft terms
    double ratio[kSmMaxPos];          // P_i(X_{i+1}) / Q_i(X_{i+1})
    unsigned mask_lo[kSmallMaxB], mask_hi[kSmallMaxB];   // candidate positions 0 .. 63 of a sequence
    int last_wanted[kSmallMaxB];      // position gamma is a candidate
    int bad[kSmallMaxB];
    int tv_tau[kSmallMaxB];
    int item0[kSmallMaxB + 1];        // first item of every sequence in the second phase
    float wM[kSmWarps];
    float wS[kSmWarps];
    double cS[kSmMaxPos];             // third phase: S_i of this CTA's sequence
    // fetched by the extra warp during the first phase: the logits of the drafted tokens, the uniforms
    float zp[kSmMaxPos], zq[kSmMaxPos];
    unsigned char xok[kSmMaxPos];
    float u[kSmMaxUni];
};

// the grid-wide barrier: arrivals are counted up through the launch; the wait is bounded
// (absent: a test switch; the CTA does not arrive, so that every CTA's wait runs out)
__device__ __forceinline__ bool small_grid_barrier(unsigned* counter, unsigned target, int* status, unsigned limit, bool absent) {
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) {
        __threadfence();
        if (!absent) atomicAdd(counter, 1u);
        unsigned spins = 0;
        while (ld_volatile(counter) < target) {
            if (++spins > limit) { if (status) atomicExch(status, 1); ok = false; break; }
        }
        __threadfence();
    }
    return __syncthreads_and(ok ? 1 : 0) != 0;
}

// vectors [s0, s1) of segment `seg` (piece * kSmWarps + warp) of a row cut into nseg segments
__device__ __forceinline__ void small_seg_range(int units, int nseg, int seg, int& s0, int& s1) {
    s0 = static_cast<int>(static_cast<long long>(units) * seg / nseg);
    s1 = static_cast<int>(static_cast<long long>(units) * (seg + 1) / nseg);
}

// row index -> pointer: rows 0 .. gamma of a sequence are its target rows, gamma+1 .. 2 gamma its draft rows
__device__ __forceinline__ const char* small_row(const Params& prm, size_t row_bytes, int b, int j) {
    const int g = prm.gamma;
    return j <= g ? static_cast<const char*>(prm.tgt) + (static_cast<size_t>(b) * (g + 1) + j) * row_bytes
                  : static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + (j - g - 1)) * row_bytes;
}

// PROBS: the rows hold probabilities, used as stored: there is no first phase (and no first barrier).
template <int DT, bool PROBS>
__global__ void __launch_bounds__(kSmAllThreads, 1) verify_small_kernel(const Params prm, const SmallScratch sc) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr uint32_t kPad = PROBS ? 0u : R::kNegInf;       // what a lane beyond the end of a segment finds: no weight
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    __shared__ SmallShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = prm.gamma, B = prm.B, units = prm.V / EPV;
    const size_t row_bytes = static_cast<size_t>(prm.V) * ESZ;
    const float kf = prm.kf;
    const int rpb = 2 * g + 1, nrows = B * rpb;
    const unsigned limit = prm.wait_limit ? prm.wait_limit : (1u << 22);
    const bool tv = prm.algo == kTokenVerify;
    const bool all_positions = f_all_positions(prm);
    bool alive = true;

    // ---------------- phase 1: {reference, sum 2^{z k - M}} of every chunk of every row ----------------
    const int nch = sc.nch;
    if (warp == kSmWarps) {
        // nothing here depends on the first phase: the two dependent round trips (token, then its two
        // logits) and the uniforms are over before the streaming warps are
        for (int i = lane; i < B * g; i += 32) {
            const int b = i / g, c = i % g;
            const int x = prm.tok[i];
            const bool xok = x >= 0 && x < prm.V;
            sh.xok[b * (g + 1) + c] = xok;
            sh.zp[b * (g + 1) + c] = xok ? static_cast<float>(load_logit<DT>(small_row(prm, row_bytes, b, c), x)) : 0.f;
            sh.zq[b * (g + 1) + c] = xok ? static_cast<float>(load_logit<DT>(small_row(prm, row_bytes, b, g + 1 + c), x)) : 0.f;
        }
        for (int i = lane; i < B * (g + 2); i += 32) sh.u[i] = prm.uni[i];
    }
    for (int item = blockIdx.x; !PROBS && item < nrows * nch; item += gridDim.x) {
        const int rid = item / nch, ch = item % nch;
        if (prm.lse_d != nullptr && rid % rpb > g) continue;      // (a draft row whose normaliser is supplied: nothing to learn)
        const char* row = small_row(prm, row_bytes, rid / rpb, rid % rpb);
        int u0, u1;
        small_seg_range(units, nch, ch, u0, u1);
        float M = kNoRef, s = 0.f;
        const uint4 ninf = make_uint4(R::kNegInf, R::kNegInf, R::kNegInf, R::kNegInf);
        for (int base = u0; warp < kSmWarps && base < u1; base += kSmThreads * kSmInFlight) {
            uint4 raw[kSmInFlight];
#pragma unroll
            for (int j = 0; j < kSmInFlight; ++j) {
                const int i = base + j * kSmThreads + tid;
                raw[j] = i < u1 ? ld_stream_v4(row + static_cast<size_t>(i) * 16) : ninf;
            }
#pragma unroll
            for (int j = 0; j < kSmInFlight; ++j) {
                if (base + j * kSmThreads + (warp << 5) < u1) {          // (warp-uniform)
                    float v[EPV];
                    R::unpack(raw[j], v);
                    f_accumulate<EPV>(v, kf, M, s);
                }
            }
        }
        s = warp_sum(s);
        if (lane == 0 && warp < kSmWarps) { sh.wM[warp] = M; sh.wS[warp] = s; }
        __syncthreads();
        if (warp == 0) {
            const float m = lane < kSmWarps ? sh.wM[lane] : kNoRef;
            const float Mc = warp_max(m);
            double z = lane < kSmWarps ? static_cast<double>(sh.wS[lane]) * static_cast<double>(ref_scale(m, Mc)) : 0.0;
            z = warp_sum_d(z);
            if (lane == 0) sc.part[static_cast<size_t>(rid) * nch + ch] = make_double2(static_cast<double>(Mc), z);
        }
        __syncthreads();
    }
    if (PROBS) __syncthreads();
    else alive = small_grid_barrier(sc.barrier, gridDim.x, prm.status, limit, prm.never_signal && blockIdx.x == 0);

    // ---------------- phase 2a: normalisers of every row, the scalar part of every sequence ----------------
    if (alive) {
        for (int rid = tid; rid < nrows; rid += kSmAllThreads) {
            if (PROBS) { sh.rowM[rid] = 0.f; sh.rowZ[rid] = 1.0; continue; }
            if (prm.lse_d != nullptr && rid % rpb > g) {
                // the supplied normaliser as an integer reference at or above every scaled logit of the row
                // plus a sum in [2^-1/2, 2^1/2]; a value that is not finite leaves the row without a reference
                const double L2 = static_cast<double>(prm.lse_d[static_cast<size_t>(rid / rpb) * g + (rid % rpb - g - 1)]) * 1.4426950408889634073599246810019;
                const bool fin = L2 > -1e300 && L2 < 1e300;
                sh.rowM[rid] = fin ? static_cast<float>(rint(L2)) : kNoRef;
                sh.rowZ[rid] = fin ? exp2(L2 - rint(L2)) : 0.0;
                continue;
            }
            float M = kNoRef;
            double z[kSmallMaxChunks];
            float m[kSmallMaxChunks];
#pragma unroll 4
            for (int c = 0; c < nch; ++c) {
                const double2 p = __ldcg(&sc.part[static_cast<size_t>(rid) * nch + c]);
                m[c] = static_cast<float>(p.x); z[c] = p.y;
                M = fmaxf(M, m[c]);
            }
            double Z = 0.0;
            for (int c = 0; c < nch; ++c) Z += z[c] * static_cast<double>(ref_scale(m[c], M));
            sh.rowM[rid] = M;
            sh.rowZ[rid] = Z;
        }
    }
    __syncthreads();
    if (alive) {
        for (int b = warp; warp < kSmWarps && b < B; b += kSmWarps) {
            // lanes c and c + 32 speak for rows / positions c and c + 32
            double rat[2] = {1.0, 1.0};
            bool badrow[2] = {false, false};
            float eta[2] = {0.f, 0.f};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = lane + 32 * h;
                if (c < g) {
                    const float MP = sh.rowM[b * rpb + c], MQ = sh.rowM[b * rpb + g + 1 + c];
                    const double ZP = sh.rowZ[b * rpb + c], ZQ = sh.rowZ[b * rpb + g + 1 + c];
                    const bool xok = sh.xok[b * (g + 1) + c] != 0;
                    const double zp = sh.zp[b * (g + 1) + c], zq = sh.zq[b * (g + 1) + c];
                    bool bad;
                    if (PROBS) {
                        // the stored numbers themselves: Q must be a positive finite number, P a non-negative finite one
                        bad = !xok || !(zq > 0.0 && zq < static_cast<double>(INFINITY)) || !(zp >= 0.0 && zp < static_cast<double>(INFINITY));
                        rat[h] = bad ? 0.0 : zp / zq;
                    } else {
                        bad = !(MP > kNoRef && MP < INFINITY) || !(ZP < static_cast<double>(INFINITY)) ||
                              !(MQ > kNoRef && MQ < INFINITY) || !(ZQ < static_cast<double>(INFINITY)) || !xok || zq == -INFINITY;
                        rat[h] = bad ? 0.0 : exp2((zp - zq) * prm.kd - (static_cast<double>(MP) - static_cast<double>(MQ))) * (ZQ / ZP);
                    }
                    badrow[h] = bad;
                    sh.ratio[b * (g + 1) + c] = rat[h];
                    // the uniform that decides about this lane's row / position
                    eta[h] = tv ? sh.u[b * (g + 2) + c] : (c >= 1 ? sh.u[b * (g + 2) + c - 1] : 0.f);
                }
            }
            const float MPg = sh.rowM[b * rpb + g];
            const double ZPg = sh.rowZ[b * rpb + g];
            const bool bad_last = !PROBS && (!(MPg > kNoRef && MPg < INFINITY) || !(ZPg < static_cast<double>(INFINITY)));
            const unsigned bad_lo = __ballot_sync(0xffffffffu, badrow[0]), bad_hi = __ballot_sync(0xffffffffu, badrow[1]);
            unsigned m_lo = 0, m_hi = 0;
            int lastw = 0, bad = 0, tau_tv = 0;
            if (tv) {
                // Algorithm 1: test c + 1 on row c; tau = the tests passed before the first failure
                bool pass[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c = lane + 32 * h;
                    const double hw = fmin(rat[h], 1.0);
                    pass[h] = c >= g || (hw > 0.0 && static_cast<double>(eta[h]) <= hw);
                }
                const unsigned f_lo = __ballot_sync(0xffffffffu, !pass[0]), f_hi = __ballot_sync(0xffffffffu, !pass[1]);
                tau_tv = f_lo ? __ffs(f_lo) - 1 : (f_hi ? 32 + __ffs(f_hi) - 1 : g);
                // (a fault counts if its row is among rows 0 .. min(tau, gamma - 1), or in the last target row when tau = gamma)
                const int last_pair = tau_tv < g ? tau_tv : g - 1;
                const unsigned long long badrows = static_cast<unsigned long long>(bad_lo) | (static_cast<unsigned long long>(bad_hi) << 32);
                bad = (badrows & (last_pair >= 63 ? ~0ull : ((2ull << last_pair) - 1ull))) != 0ull || (tau_tv == g && bad_last);
                if (all_positions) bad = bad;     // (diagnostics never widen what counts as a fault)
                if (tau_tv == g) lastw = 1;
                else if (tau_tv < 32) m_lo = 1u << tau_tv;
                else m_hi = 1u << (tau_tv - 32);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c = lane + 32 * h;
                    if (c < g) sh.csc[b * (g + 1) + c] = static_cast<float>(sh.rowZ[b * rpb + g + 1 + c] / sh.rowZ[b * rpb + c]);
                }
            } else {
                double pc = 1.0, mine[2] = {1.0, 1.0};
                for (int c = 0; c < g; ++c) {
                    if ((c & 31) == lane) mine[c >> 5] = pc;
                    const double r = shfl_d(c < 32 ? rat[0] : rat[1], c & 31);
                    const double next = pc * r;
                    pc = prm.greedy ? next : fmin(next, 1.0);
                }
                const double p_g = pc;
                bool need[2] = {false, false};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c = lane + 32 * h;
                    if (c < g) {
                        // h_c <= p_c: a position whose uniform lies above p_c cannot be the selected one
                        need[h] = all_positions || c == 0 || static_cast<double>(eta[h]) <= mine[h] * (1.0 + 1e-6);
                        sh.pch[b * (g + 1) + c] = mine[h];
                        sh.csc[b * (g + 1) + c] = static_cast<float>(mine[h] * (sh.rowZ[b * rpb + g + 1 + c] / sh.rowZ[b * rpb + c]));
                    }
                }
                m_lo = __ballot_sync(0xffffffffu, need[0]);
                m_hi = __ballot_sync(0xffffffffu, need[1]);
                const float eta_g = sh.u[b * (g + 2) + g - 1];
                lastw = all_positions || static_cast<double>(eta_g) <= p_g * (1.0 + 1e-6);
                bad = (bad_lo | bad_hi) != 0u || bad_last;
                if (lane == 0) sh.pch[b * (g + 1) + g] = p_g;
            }
            if (lane == 0) {
                sh.mask_lo[b] = m_lo; sh.mask_hi[b] = m_hi; sh.last_wanted[b] = lastw;
                sh.bad[b] = bad; sh.tv_tau[b] = tau_tv;
                sh.csc[b * (g + 1) + g] = 1.f;
            }
        }
    }
    __syncthreads();
    const int np = sc.np, nseg = np * kSmWarps;
    if (tid == 0) {
        int acc = 0;
        for (int b = 0; b < B; ++b) {
            sh.item0[b] = acc;
            acc += (__popc(sh.mask_lo[b]) + __popc(sh.mask_hi[b]) + sh.last_wanted[b]) * np;
        }
        sh.item0[B] = acc;
    }
    __syncthreads();

    // ---------------- phase 2b: per-segment sums of the residual terms of every candidate position ----------------
    if (alive) {
        const int total = sh.item0[B];
        for (int item = blockIdx.x; item < total; item += gridDim.x) {
            int b = 0;
            while (item >= sh.item0[b + 1]) ++b;
            const int k = (item - sh.item0[b]) / np, piece = (item - sh.item0[b]) % np;
            // the k-th candidate of the sequence, from position 0 up; position gamma last
            const int n_lo = __popc(sh.mask_lo[b]), n_hi = __popc(sh.mask_hi[b]);
            int i;
            if (k < n_lo) i = __fns(sh.mask_lo[b], 0, k + 1);
            else if (k < n_lo + n_hi) i = 32 + __fns(sh.mask_hi[b], 0, k - n_lo + 1);
            else i = g;
            const bool have_q = i < g;
            const char* rowP = small_row(prm, row_bytes, b, i);
            const char* rowQ = have_q ? small_row(prm, row_bytes, b, g + 1 + i) : nullptr;
            const float cp = sh.csc[b * (g + 1) + i];
            const float nMP = -sh.rowM[b * rpb + i], nMQ = have_q ? -sh.rowM[b * rpb + g + 1 + i] : 0.f;
            int s0, s1;
            small_seg_range(units, nseg, piece * kSmWarps + (warp < kSmWarps ? warp : 0), s0, s1);
            double acc = 0.0;
            for (int base = s0; warp < kSmWarps && base < s1; base += 32 * kSmPairsInFlight) {
                uint4 rp[kSmPairsInFlight], rq[kSmPairsInFlight];
                const uint4 ninf = make_uint4(kPad, kPad, kPad, kPad);
#pragma unroll
                for (int j = 0; j < kSmPairsInFlight; ++j) {
                    const int v = base + 32 * j + lane;
                    rp[j] = v < s1 ? ld_stream_v4(rowP + static_cast<size_t>(v) * 16) : ninf;
                    rq[j] = (v < s1 && have_q) ? ld_stream_v4(rowQ + static_cast<size_t>(v) * 16) : ninf;
                }
#pragma unroll
                for (int j = 0; j < kSmPairsInFlight; ++j) {
                    float vp[EPV], vq[EPV], t[EPV];
                    R::unpack(rp[j], vp);
                    R::unpack(rq[j], vq);
                    if (have_q) acc += static_cast<double>(f_pair_sum<EPV, true, PROBS>(vp, vq, kf, cp, nMP, nMQ, t));
                    else acc += static_cast<double>(f_pair_sum<EPV, false, PROBS>(vp, vq, kf, cp, nMP, nMQ, t));
                }
            }
            acc = warp_sum_d(acc);
            if (lane == 0 && warp < kSmWarps) sc.seg[(static_cast<size_t>(b) * (g + 1) + i) * nseg + piece * kSmWarps + warp] = acc;
        }
    }
    // (arrivals are counted up through the launch: the second barrier of a launch on logits, the only one otherwise)
    if (alive) alive = small_grid_barrier(sc.barrier, (PROBS ? 1u : 2u) * gridDim.x, prm.status, limit,
                                          PROBS && prm.never_signal && blockIdx.x == 0);

    // ---------------- phase 3: one CTA per sequence ----------------
    for (int b = blockIdx.x; alive && b < B; b += gridDim.x) {
        // S_i of every candidate (a warp per position at a time)
        const unsigned m_lo = sh.mask_lo[b], m_hi = sh.mask_hi[b];
        for (int i = warp; i < g; i += kSmAllThreads / 32) {
            const bool cand = (i < 32 ? m_lo >> i : m_hi >> (i - 32)) & 1u;
            double tot = 0.0;
            if (cand) {
                const double* segs = sc.seg + (static_cast<size_t>(b) * (g + 1) + i) * nseg;
                for (int s = lane; s < nseg; s += 32) tot += __ldcg(&segs[s]);
                tot = warp_sum_d(tot) / sh.rowZ[b * rpb + g + 1 + i];
            }
            if (lane == 0) sh.cS[i] = tot;
        }
        __syncthreads();
        if (warp == 0) {
            const float* u = sh.u + b * (g + 2);
            int tau;
            if (tv) {
                tau = sh.tv_tau[b];
            } else {
                // tau = max{i >= 1 : h_i > 0 and eta_i <= h_i}, else 0; h_gamma = p_gamma, h_i = S_i / (S_i + 1 - p_i)
                bool pass[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int i = lane + 32 * h;
                    const bool cand = i >= 1 && i < g && ((i < 32 ? m_lo >> i : m_hi >> (i - 32)) & 1u);
                    const double hw = cand ? f_weight(sh.pch[b * (g + 1) + i], sh.cS[i]) : 0.0;
                    pass[h] = cand && hw > 0.0 && static_cast<double>(u[i - 1]) <= hw;
                }
                const unsigned p_lo = __ballot_sync(0xffffffffu, pass[0]), p_hi = __ballot_sync(0xffffffffu, pass[1]);
                const double p_g = sh.pch[b * (g + 1) + g];
                tau = 0;
                if (sh.last_wanted[b] && p_g > 0.0 && static_cast<double>(u[g - 1]) <= p_g) tau = g;
                else if (p_hi) tau = 32 + 31 - __clz(p_hi);
                else if (p_lo) tau = 31 - __clz(p_lo);
            }
            // Y by inverse CDF in index order over the segment sums of position tau, then within one segment
            const bool have_q = tau < g;
            const double* segs = sc.seg + (static_cast<size_t>(b) * (g + 1) + tau) * nseg;
            double w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) w[j] = 4 * lane + j < nseg ? __ldcg(&segs[4 * lane + j]) : 0.0;
            const double d1 = w[0], d2 = d1 + w[1], d3 = d2 + w[2], d4 = d3 + w[3];
            double inc = d4;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const double o = shfl_up_d(inc, off);
                if (lane >= off) inc += o;
            }
            const double total = shfl_d(inc, 31);
            int found = -1;
            if (total > 0.0 && total < static_cast<double>(INFINITY)) {
                const double t = static_cast<double>(u[have_q ? g : g + 1]) * total;
                double exc = shfl_up_d(inc, 1);
                if (lane == 0) exc = 0.0;
                const double p0 = exc, p1 = exc + d1, p2 = exc + d2, p3 = exc + d3, p4 = exc + d4;
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
                small_seg_range(units, nseg, sel, s0, s1);
                found = f_rescan<DT, PROBS, 5>(small_row(prm, row_bytes, b, tau), have_q ? small_row(prm, row_bytes, b, g + 1 + tau) : nullptr,
                                     s0, s1, lane, kf, sh.csc[b * (g + 1) + tau], -sh.rowM[b * rpb + tau],
                                     have_q ? -sh.rowM[b * rpb + g + 1 + tau] : 0.f, t - before);
            }
            const bool bad = sh.bad[b] != 0 || found < 0;      // (an empty residual where the algorithm must sample: a domain error)
            int32_t* ot = prm.out_tokens + static_cast<size_t>(b) * (g + 1);
            const int32_t* X = prm.tok + static_cast<size_t>(b) * g;
            for (int i = lane; i <= g; i += 32) ot[i] = bad ? -1 : (i < tau ? X[i] : (i == tau ? found : -1));
            if (lane == 0) prm.out_len[b] = bad ? -1 : tau + 1;
            if (all_positions) {
                const double ln2 = 0.693147180559945309417232;
                const float nanf_ = __int_as_float(0x7fc00000);
                for (int i = lane; i <= g; i += 32) {
                    const size_t o1 = static_cast<size_t>(b) * (g + 1) + i, o0 = static_cast<size_t>(b) * g + i;
                    float pv, hv, Sv = nanf_;
                    if (tv) {
                        pv = nanf_;
                        hv = i == 0 ? 1.f : static_cast<float>(fmin(sh.ratio[b * (g + 1) + i - 1], 1.0));
                        if (i == tau && i < g) Sv = static_cast<float>(sh.cS[i]);
                    } else {
                        const double p = sh.pch[b * (g + 1) + i];
                        pv = static_cast<float>(p);
                        hv = static_cast<float>(i == 0 ? 1.0 : (i == g ? p : f_weight(p, sh.cS[i])));
                        if (i < g) Sv = static_cast<float>(sh.cS[i]);
                    }
                    if (prm.out_p) prm.out_p[o1] = pv;
                    if (prm.out_h) prm.out_h[o1] = hv;
                    if (prm.out_lse_t) prm.out_lse_t[o1] = static_cast<float>((static_cast<double>(sh.rowM[b * rpb + i]) + log2(sh.rowZ[b * rpb + i])) * ln2);
                    if (i < g && prm.out_S) prm.out_S[o0] = Sv;
                    if (i < g && prm.out_lse_d) prm.out_lse_d[o0] = static_cast<float>((static_cast<double>(sh.rowM[b * rpb + g + 1 + i]) + log2(sh.rowZ[b * rpb + g + 1 + i])) * ln2);
                }
            }
        }
        __syncthreads();
    }

    // the barrier word is zero again when the last CTA leaves (whatever became of the waits)
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(sc.barrier + 16, 1u) == gridDim.x - 1) {
            atomicExch(sc.barrier, 0u);
            atomicExch(sc.barrier + 16, 0u);
        }
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static size_t up256s(size_t x) { return (x + 255) / 256 * 256; }

bool small_fits(int B, int gamma) {
    return B >= 1 && B <= kSmallMaxB && static_cast<long long>(B) * (2 * gamma + 1) <= kSmMaxRows &&
           static_cast<long long>(B) * (gamma + 1) <= kSmMaxPos;
}

// Chunks per row in the first phase and pieces per position in the second.  A CTA goes through its
// items one after the other, each costing its share of the row plus a fixed part (the reduction
// across the CTA and its barriers: about as long as streaming 2500 vectors), so the count is the
// one that minimises rounds x (vectors per item + 2500); no chunk below 512 vectors.
static int small_best_split(long long units, long long rows, int nctas, int most) {
    int best = 1;
    long long best_cost = -1;
    for (int n = 1; n <= most && units / n >= 512; ++n) {
        const long long rounds = (rows * n + nctas - 1) / nctas;
        const long long cost = rounds * (units / n + 2500);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = n; }
    }
    return best;
}

SmallPlan small_plan(long long units, int B, int gamma, int nctas) {
    SmallPlan pl{};
    pl.nch = small_best_split(units, static_cast<long long>(B) * (2 * gamma + 1), nctas, kSmallMaxChunks);
    // (about two candidate positions per sequence and the odd last target row: 5 rows for every 2 sequences)
    pl.np = small_best_split(units, (5LL * B + 1) / 2, nctas, 8);
    return pl;
}

size_t small_scratch_bytes(int B, int gamma, const SmallPlan& pl) {
    const size_t rows = static_cast<size_t>(B) * (2 * gamma + 1), pos = static_cast<size_t>(B) * (gamma + 1);
    return up256s(rows * pl.nch * sizeof(double2)) + up256s(pos * pl.np * kSmWarps * sizeof(double));
}

// barrier: two words 64 bytes apart that are zero between launches (the kernel leaves them so)
void small_scratch_layout(void* base, unsigned* barrier, int B, int gamma, const SmallPlan& pl, SmallScratch* sc) {
    char* p = static_cast<char*>(base);
    const size_t rows = static_cast<size_t>(B) * (2 * gamma + 1);
    sc->barrier = barrier;
    sc->part = reinterpret_cast<double2*>(p);
    sc->seg = reinterpret_cast<double*>(p + up256s(rows * pl.nch * sizeof(double2)));
    sc->nch = pl.nch;
    sc->np = pl.np;
}

using SKernelFn = void (*)(const Params, const SmallScratch);
static SKernelFn pick_small(int dtype, bool probs) {
    if (probs) return dtype == kF32 ? verify_small_kernel<kF32, true> : verify_small_kernel<kBF16, true>;
    return dtype == kF32 ? verify_small_kernel<kF32, false> : verify_small_kernel<kBF16, false>;
}

int small_max_ctas(int dtype, int sm_count) {
    int n = 0;
    // (the variant on logits is the larger program)
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pick_small(dtype, false), kSmAllThreads, 0) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n > 0 ? sm_count : 0;          // one CTA per SM: all of them resident at once, as the barriers need
}

cudaError_t launch_small(const Params& prm, const SmallScratch& sc, int dtype, int nctas, cudaStream_t stream) {
    Params p = prm;
    SmallScratch s = sc;
    void* args[] = {&p, &s};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(pick_small(dtype, prm.probs != 0)), dim3(nctas), dim3(kSmAllThreads), args, 0, stream);
}

}  // namespace bv
