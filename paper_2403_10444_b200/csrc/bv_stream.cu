// General ("streaming") verification kernel: one thread-block cluster walks one
// drafted block position by position.
//
// For position r = 0..gamma the cluster
//   sweep 1: streams P_r (and Q_r) once from HBM and forms the softmax
//            normalisers (row reference M, Z = sum 2^{z k - M});
//   scalars: reads the two logits of the drafted token X_{r+1}, extends the
//            prefix recursion p_{r+1} = min(p_r P_r(X)/Q_r(X), 1)  (Eq. "def_as")
//            or takes Algorithm 1's accept/reject decision;
//   sweep 2: re-reads the pair (an L2 hit while the cluster's working set is
//            resident) and forms S_r = sum_x max(p_r P_r(x) - Q_r(x), 0)
//            (Eq. "pacc_block") with one partial total per warp segment;
//   sample : picks the candidate Y_r by inverse CDF in index order from the
//            segment totals, rescanning only the one segment that holds u * S_r.
// After the last position rank 0 forms h_i, selects tau and emits X^tau, Y_tau.
//
// A row is split into contiguous slices per CTA and, inside a CTA, contiguous
// segments per warp, so that segment totals are in vocabulary order.
#include "bv_device.cuh"
#include "bv_launch.h"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace bv {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;

struct StreamShared {
    float red_M[2][kWarps];          // sweep 1, per warp: [P/Q][warp]
    double red_s[2][kWarps];
    float x_M[2][kMaxCluster];       // sweep 1, per CTA, written by every peer: [P/Q][rank]
    double x_s[2][kMaxCluster];
    double segtot[kWarps];           // sweep 2, per warp segment
    double x_tot[kMaxCluster];       // sweep 2, per CTA, written by every peer
    double p[kMaxGamma + 1];         // per-sequence scalars (thread 0 writes)
    double S[kMaxGamma + 1];
    double h[kMaxGamma + 1];
    double lse_t[kMaxGamma + 1];
    double lse_d[kMaxGamma + 1];
    int cand[kMaxGamma + 1];         // candidate Y_r; rank 0's copy is the one read
    int b;                           // sequence this cluster works on (-1: none left)
    int bad;                         // data fault seen in this sequence
    int tau;                         // Algorithm 1: accepted length so far
    int do_sweep2;                   // control for the current position
    int last_row;                    // Algorithm 1: stop after this position
    float c;                         // sweep 2: p_r * Z_Q / Z_P
    float negMP, negMQ;              // sweep 2: minus the row references
    double invZQ;                    // sweep 2: 1 / Z_Q (1 / Z_P when there is no draft row)
};

template <class U, bool HAVEQ>
__device__ __forceinline__ void sweep1(const void* rowP, const void* rowQ, int w0, int w1, int lane,
                                       float kf, MaxSum& aP, MaxSum& aQ) {
    constexpr int EPV = U::EPV;
    constexpr int UNR = 4;
    int i = w0 + lane;
    for (; i + 32 * (UNR - 1) < w1; i += 32 * UNR) {
        float vp[UNR][EPV], vq[UNR][EPV];
#pragma unroll
        for (int k = 0; k < UNR; ++k) {
            U::load(rowP, i + 32 * k, vp[k]);
            if (HAVEQ) U::load(rowQ, i + 32 * k, vq[k]);
        }
#pragma unroll
        for (int k = 0; k < UNR; ++k) {
            aP.add(vp[k], kf);
            if (HAVEQ) aQ.add(vq[k], kf);
        }
    }
    for (; i < w1; i += 32) {
        float vp[EPV], vq[EPV];
        U::load(rowP, i, vp);
        if (HAVEQ) U::load(rowQ, i, vq);
        aP.add(vp, kf);
        if (HAVEQ) aQ.add(vq, kf);
    }
}

// terms t_e = max(c * 2^{zP k - MP} - 2^{zQ k - MQ}, 0), or 2^{zP k - MP} without a draft row
template <int EPV, bool HAVEQ>
__device__ __forceinline__ void terms(const float (&vp)[EPV], const float (&vq)[EPV], float kf,
                                      float c, float negMP, float negMQ, float (&t)[EPV]) {
#pragma unroll
    for (int e = 0; e < EPV; ++e) {
        float a = ex2(fmaf(vp[e], kf, negMP));
        if (HAVEQ) {
            float q = ex2(fmaf(vq[e], kf, negMQ));
            t[e] = fmaxf(fmaf(c, a, -q), 0.f);
        } else {
            t[e] = a;
        }
    }
}

template <class U, bool HAVEQ>
__device__ __forceinline__ float sweep2(const void* rowP, const void* rowQ, int w0, int w1, int lane,
                                        float kf, float c, float negMP, float negMQ) {
    constexpr int EPV = U::EPV;
    constexpr int UNR = 4;
    float acc = 0.f;
    int i = w0 + lane;
    for (; i + 32 * (UNR - 1) < w1; i += 32 * UNR) {
        float vp[UNR][EPV], vq[UNR][EPV];
#pragma unroll
        for (int k = 0; k < UNR; ++k) {
            U::load(rowP, i + 32 * k, vp[k]);
            if (HAVEQ) U::load(rowQ, i + 32 * k, vq[k]);
        }
#pragma unroll
        for (int k = 0; k < UNR; ++k) {
            float t[EPV];
            terms<EPV, HAVEQ>(vp[k], vq[k], kf, c, negMP, negMQ, t);
            float v = t[0];
#pragma unroll
            for (int e = 1; e < EPV; ++e) v += t[e];
            acc += v;
        }
    }
    for (; i < w1; i += 32) {
        float vp[EPV], vq[EPV], t[EPV];
        U::load(rowP, i, vp);
        if (HAVEQ) U::load(rowQ, i, vq);
        terms<EPV, HAVEQ>(vp, vq, kf, c, negMP, negMQ, t);
        float v = t[0];
#pragma unroll
        for (int e = 1; e < EPV; ++e) v += t[e];
        acc += v;
    }
    return acc;
}

// One warp walks its segment [w0, w1) in index order and returns the first
// element whose running sum exceeds tw (else the last element with a positive
// term, else -1).  Result valid in every lane.
template <class U, bool HAVEQ>
__device__ int rescan_segment(const void* rowP, const void* rowQ, int w0, int w1, int lane,
                              float kf, float c, float negMP, float negMQ, double tw) {
    constexpr int EPV = U::EPV;
    double run = 0.0;
    int last_pos = -1;
    for (int base = w0; base < w1; base += 32) {
        const int i = base + lane;
        float t[EPV];
        float ls = 0.f;
        if (i < w1) {
            float vp[EPV], vq[EPV];
            U::load(rowP, i, vp);
            if (HAVEQ) U::load(rowQ, i, vq);
            terms<EPV, HAVEQ>(vp, vq, kf, c, negMP, negMQ, t);
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                ls += t[e];
                if (t[e] > 0.f) last_pos = i * EPV + e;
            }
        } else {
#pragma unroll
            for (int e = 0; e < EPV; ++e) t[e] = 0.f;
        }
        double inc = static_cast<double>(ls);
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            double o = shfl_up_d(inc, off);
            if (lane >= off) inc += o;
        }
        const bool hit = (i < w1) && (run + inc > tw);
        const unsigned bal = __ballot_sync(0xffffffffu, hit);
        if (bal) {
            const int src = __ffs(bal) - 1;
            int found = -1;
            if (lane == src) {
                double cum = run + inc - static_cast<double>(ls);
                int lp = -1;
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    cum += static_cast<double>(t[e]);
                    if (t[e] > 0.f) lp = i * EPV + e;
                    if (found < 0 && cum > tw && t[e] > 0.f) found = i * EPV + e;
                }
                if (found < 0) found = lp;
            }
            found = __shfl_sync(0xffffffffu, found, src);
            if (found >= 0) return found;
        }
        run += shfl_d(inc, 31);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, off));
    return last_pos;
}

template <int ALGO>
__device__ void finalize_sequence(StreamShared& sh, const Params& prm) {
    const int g = prm.gamma;
    const int b = sh.b;
    int32_t* ot = prm.out_tokens + static_cast<size_t>(b) * (g + 1);
    const int32_t* X = prm.tok + static_cast<size_t>(b) * g;
    const float* u = prm.uni + static_cast<size_t>(b) * (g + 2);
    int tau = -1;
    if (!sh.bad) {
        if (ALGO == kBlockVerify) {
            // h_gamma = p_gamma; h_i = S_i / (S_i + 1 - p_i); tau = max{i : eta_i <= h_i}
            sh.h[0] = 1.0;
            for (int i = 1; i < g; ++i)
                sh.h[i] = sh.S[i] > 0.0 ? sh.S[i] / (sh.S[i] + 1.0 - sh.p[i]) : 0.0;
            sh.h[g] = sh.p[g];
            tau = 0;
            for (int i = g; i >= 1; --i)
                if (sh.h[i] > 0.0 && static_cast<double>(u[i - 1]) <= sh.h[i]) { tau = i; break; }
        } else {
            sh.h[0] = 1.0;
            tau = sh.tau;
        }
    }
    for (int i = 0; i <= g; ++i) ot[i] = -1;
    if (tau >= 0 && sh.cand[tau] < 0) tau = -1;      // (nothing to sample from at the selected position: a domain error)
    if (tau >= 0) {
        for (int i = 0; i < tau; ++i) ot[i] = X[i];
        ot[tau] = sh.cand[tau];
        prm.out_len[b] = tau + 1;
    } else {
        prm.out_len[b] = -1;
    }
    for (int i = 0; i <= g; ++i) {
        const size_t o1 = static_cast<size_t>(b) * (g + 1) + i, o0 = static_cast<size_t>(b) * g + i;
        if (prm.out_p) prm.out_p[o1] = static_cast<float>(sh.p[i]);
        if (prm.out_h) prm.out_h[o1] = static_cast<float>(sh.h[i]);
        if (prm.out_lse_t) prm.out_lse_t[o1] = static_cast<float>(sh.lse_t[i]);
        if (i < g && prm.out_S) prm.out_S[o0] = static_cast<float>(sh.S[i]);
        if (i < g && prm.out_lse_d) prm.out_lse_d[o0] = static_cast<float>(sh.lse_d[i]);
    }
}

template <int DT, bool VEC, int ALGO>
__global__ void __launch_bounds__(kThreads, 1) verify_stream_kernel(const Params prm) {
    using U = Unit<DT, VEC>;
    constexpr int EPV = U::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ StreamShared sh;

    const int g = prm.gamma, V = prm.V;
    const float kf = prm.kf;
    const double kd = prm.kd;
    const int units = V / EPV;
    // contiguous slice of this CTA, contiguous segment of this warp
    const int u0 = static_cast<int>(static_cast<long long>(units) * rank / C);
    const int u1 = static_cast<int>(static_cast<long long>(units) * (rank + 1) / C);
    const int w0 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * warp / kWarps);
    const int w1 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * (warp + 1) / kWarps);

    bool first = true;
    for (;;) {
        cluster.sync();  // candidates of the finished sequence are visible at rank 0
        if (rank == 0 && tid == 0) {
            if (!first) finalize_sequence<ALGO>(sh, prm);
            const unsigned t = atomicAdd(&prm.ticket[0], 1u);
            const int nb = t < static_cast<unsigned>(prm.B) ? static_cast<int>(t) : -1;
            for (int c = 0; c < C; ++c) *cluster.map_shared_rank(&sh.b, c) = nb;
        }
        first = false;
        cluster.sync();
        const int b = sh.b;
        if (b < 0) break;

        if (tid <= g) {
            const double nan = __longlong_as_double(0x7ff8000000000000LL);
            sh.p[tid] = nan; sh.S[tid] = nan; sh.h[tid] = nan;
            sh.lse_t[tid] = nan; sh.lse_d[tid] = nan; sh.cand[tid] = -1;
        }
        if (tid == 0) { sh.bad = 0; sh.tau = 0; }
        __syncthreads();
        if (tid == 0 && ALGO == kBlockVerify) sh.p[0] = 1.0;

        const char* tgt_b = static_cast<const char*>(prm.tgt) + static_cast<size_t>(b) * (g + 1) * V * ESZ;
        const char* drf_b = static_cast<const char*>(prm.drf) + static_cast<size_t>(b) * g * V * ESZ;

        for (int r = 0; r <= g; ++r) {
            const bool have_q = r < g;
            const void* rowP = tgt_b + static_cast<size_t>(r) * V * ESZ;
            const void* rowQ = drf_b + static_cast<size_t>(r) * V * ESZ;

            // ---------------- sweep 1: normalisers ----------------
            MaxSum aP, aQ;
            aP.init(); aQ.init();
            if (have_q) sweep1<U, true>(rowP, rowQ, w0, w1, lane, kf, aP, aQ);
            else        sweep1<U, false>(rowP, rowQ, w0, w1, lane, kf, aP, aQ);
            warp_combine(aP.M, aP.s);
            warp_combine(aQ.M, aQ.s);
            if (lane == 0) {
                sh.red_M[0][warp] = aP.M; sh.red_s[0][warp] = static_cast<double>(aP.s);
                sh.red_M[1][warp] = aQ.M; sh.red_s[1][warp] = static_cast<double>(aQ.s);
            }
            __syncthreads();
            if (warp == 0) {
#pragma unroll
                for (int row = 0; row < 2; ++row) {
                    float M = lane < kWarps ? sh.red_M[row][lane] : -INFINITY;
                    double s = lane < kWarps ? sh.red_s[row][lane] : 0.0;
                    float Mc = M;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) Mc = fmaxf(Mc, __shfl_xor_sync(0xffffffffu, Mc, off));
                    s = (s != s) ? s : s * static_cast<double>(pow2_nonpos(M - Mc));
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) s += shfl_xor_d(s, off);
                    if (lane < C) {
                        *cluster.map_shared_rank(&sh.x_M[row][rank], lane) = Mc;
                        *cluster.map_shared_rank(&sh.x_s[row][rank], lane) = s;
                    }
                }
            }
            cluster.sync();

            // ---------------- scalars: combine ranks, recursion / decision ----------------
            if (warp == 0) {
                // lanes 0..7 hold the target row's per-CTA partials, lanes 8..15 the draft row's
                const int row = (lane >> 3) & 1, rk = lane & 7;
                const bool live = lane < 16 && rk < C;
                float M = live ? sh.x_M[row][rk] : -INFINITY;
                double s = live ? sh.x_s[row][rk] : 0.0;
                float Mr = M;
#pragma unroll
                for (int off = 4; off > 0; off >>= 1) Mr = fmaxf(Mr, __shfl_xor_sync(0xffffffffu, Mr, off));
                s = (s != s) ? s : s * static_cast<double>(pow2_nonpos(M - Mr));
#pragma unroll
                for (int off = 4; off > 0; off >>= 1) s += shfl_xor_d(s, off);
                const float MQ = __shfl_sync(0xffffffffu, Mr, 8);
                const double ZQ = shfl_d(s, 8);
                if (lane == 0) {
                    const float MP = Mr;
                    const double ZP = s;
                    const double ln2 = 0.693147180559945309417232;
                    int bad = sh.bad;
                    // M is finite iff the row's maximum is; Z is NaN iff the row holds a NaN
                    if (!(fabsf(MP) < INFINITY) || !(ZP == ZP)) bad = 1;
                    if (have_q && (!(fabsf(MQ) < INFINITY) || !(ZQ == ZQ))) bad = 1;
                    const double lse2P = static_cast<double>(MP) + log2(ZP);
                    const double lse2Q = static_cast<double>(MQ) + log2(ZQ);
                    sh.lse_t[r] = lse2P * ln2;
                    if (have_q) sh.lse_d[r] = lse2Q * ln2;

                    double ratio = 0.0;
                    if (have_q && !bad) {
                        const int x = prm.tok[static_cast<size_t>(b) * g + r];
                        if (x < 0 || x >= V) {
                            bad = 1;
                        } else {
                            const double zq = load_logit<DT>(rowQ, x), zp = load_logit<DT>(rowP, x);
                            if (zq == -INFINITY) bad = 1;
                            else ratio = exp2((zp * kd - lse2P) - (zq * kd - lse2Q));
                        }
                    }
                    double p_r = 1.0;       // multiplier of P_r in the residual at this position
                    int do2 = 1, last = 0;
                    if (ALGO == kBlockVerify) {
                        p_r = sh.p[r];
                        if (have_q) sh.p[r + 1] = fmin(p_r * ratio, 1.0);
                    } else if (have_q) {
                        const double h = fmin(ratio, 1.0);
                        sh.h[r + 1] = h;
                        const double eta = static_cast<double>(prm.uni[static_cast<size_t>(b) * (g + 2) + r]);
                        if (!bad && h > 0.0 && eta <= h) { sh.tau = r + 1; do2 = 0; }
                        else last = 1;
                    }
                    if (bad) { do2 = 0; last = 1; }
                    sh.bad = bad;
                    sh.do_sweep2 = do2;
                    sh.last_row = last;
                    sh.c = have_q ? static_cast<float>(p_r * ZQ / ZP) : 1.f;
                    sh.negMP = -MP;
                    sh.negMQ = -MQ;
                    sh.invZQ = have_q ? 1.0 / ZQ : 1.0 / ZP;
                }
            }
            __syncthreads();
            const bool last_row = sh.last_row != 0;
            if (sh.do_sweep2) {
                const float c = sh.c, negMP = sh.negMP, negMQ = sh.negMQ;
                // (an empty residual leaves no candidate; a block that selects such a position, which the
                // algorithms cannot do, ends as a domain error)
                bool use_q = have_q;
                for (int attempt = 0; attempt < 2; ++attempt) {
                    // ---------------- sweep 2: residual mass per warp segment ----------------
                    float acc = use_q ? sweep2<U, true>(rowP, rowQ, w0, w1, lane, kf, c, negMP, negMQ)
                                      : sweep2<U, false>(rowP, rowQ, w0, w1, lane, kf, c, negMP, negMQ);
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                    if (lane == 0) sh.segtot[warp] = static_cast<double>(acc);
                    __syncthreads();
                    if (warp == 0) {
                        double v = lane < kWarps ? sh.segtot[lane] : 0.0;
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) v += shfl_xor_d(v, off);
                        if (lane < C) *cluster.map_shared_rank(&sh.x_tot[rank], lane) = v;
                    }
                    cluster.sync();

                    // ---------------- candidate sample Y_r ----------------
                    double total = 0.0, before = 0.0;
                    for (int k = 0; k < C; ++k) {
                        if (k == rank) before = total;
                        total += sh.x_tot[k];
                    }
                    if (attempt == 0 && use_q && tid == 0) sh.S[r] = total * sh.invZQ;
                    const bool empty = !(total > 0.0);
                    if (!empty) {
                        const float uf = prm.uni[static_cast<size_t>(b) * (g + 2) + (have_q ? g : g + 1)];
                        const double t = static_cast<double>(uf) * total;
                        // first CTA whose inclusive prefix exceeds t, else the last non-empty one
                        int sel = -1, lastnz = -1;
                        double run = 0.0, sel_before = 0.0, nz_before = 0.0;
                        for (int k = 0; k < C; ++k) {
                            const double v = sh.x_tot[k];
                            if (v > 0.0) { lastnz = k; nz_before = run; }
                            if (sel < 0 && run + v > t) { sel = k; sel_before = run; }
                            run += v;
                        }
                        if (sel < 0) { sel = lastnz; sel_before = nz_before; }
                        (void)before;
                        if (sel == rank) {
                            const double tc = t - sel_before;
                            int wsel = -1, wlast = -1;
                            double wrun = 0.0, wsel_before = 0.0, wnz_before = 0.0;
                            for (int k = 0; k < kWarps; ++k) {
                                const double v = sh.segtot[k];
                                if (v > 0.0) { wlast = k; wnz_before = wrun; }
                                if (wsel < 0 && wrun + v > tc) { wsel = k; wsel_before = wrun; }
                                wrun += v;
                            }
                            if (wsel < 0) { wsel = wlast; wsel_before = wnz_before; }
                            if (warp == wsel) {
                                const double tw = tc - wsel_before;
                                const int y = use_q
                                    ? rescan_segment<U, true>(rowP, rowQ, w0, w1, lane, kf, c, negMP, negMQ, tw)
                                    : rescan_segment<U, false>(rowP, rowQ, w0, w1, lane, kf, c, negMP, negMQ, tw);
                                if (lane == 0) *cluster.map_shared_rank(&sh.cand[r], 0) = y;
                            }
                        }
                    }
                    break;
                }
            }
            if (last_row) break;
        }
    }

    // the last cluster to leave re-arms the ticket for the next launch
    if (rank == 0 && tid == 0) {
        const unsigned d = atomicAdd(&prm.ticket[1], 1u);
        if (d == static_cast<unsigned>(prm.nclusters) - 1u) {
            prm.ticket[0] = 0u;
            prm.ticket[1] = 0u;
            __threadfence();
        }
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
using KernelFn = void (*)(const Params);

static KernelFn pick_kernel(int algo, int dtype, bool vec) {
    if (algo == kBlockVerify) {
        if (dtype == kF32) return vec ? verify_stream_kernel<kF32, true, kBlockVerify>
                                      : verify_stream_kernel<kF32, false, kBlockVerify>;
        return vec ? verify_stream_kernel<kBF16, true, kBlockVerify>
                   : verify_stream_kernel<kBF16, false, kBlockVerify>;
    }
    if (dtype == kF32) return vec ? verify_stream_kernel<kF32, true, kTokenVerify>
                                  : verify_stream_kernel<kF32, false, kTokenVerify>;
    return vec ? verify_stream_kernel<kBF16, true, kTokenVerify>
               : verify_stream_kernel<kBF16, false, kTokenVerify>;
}

static void fill_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int cluster, int nclusters,
                        cudaStream_t stream) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(static_cast<unsigned>(cluster * nclusters), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

int stream_max_clusters(int algo, int dtype, bool vec, int cluster) {
    KernelFn fn = pick_kernel(algo, dtype, vec);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_config(cfg, attr, cluster, 1, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, reinterpret_cast<const void*>(fn), &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t launch_stream(const Params& prm, int algo, int dtype, bool vec, int cluster,
                          int nclusters, cudaStream_t stream) {
    KernelFn fn = pick_kernel(algo, dtype, vec);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_config(cfg, attr, cluster, nclusters, stream);
    return cudaLaunchKernelEx(&cfg, fn, prm);
}

}  // namespace bv
