// Verification kernel for 16-byte aligned rows: one thread-block cluster walks one
// drafted block position by position; several clusters share every SM, so that
// while one of them waits for an exchange the others keep the pipes busy.
//
// For position r = 0..gamma the cluster
//   sweep 1  streams P_r and Q_r from HBM with 128-bit loads and forms, per warp
//            segment, sum 2^{z k - M} against a warp-uniform integer reference M;
//   exchange every warp sends {M_P, s_P, M_Q, s_Q} to every CTA of the cluster
//            (st.async into distributed shared memory, counted by a transaction
//            barrier); warp 0 of each CTA combines them into the row normalisers;
//   scalars  Algorithm 2: p_{r+1} = min(p_r P_r(X)/Q_r(X), 1)  (Eq. "def_as");
//            Algorithm 1: h = min(ratio, 1), accept or stop;
//   sweep 2  re-reads the pair (served by L2: the cluster's working set is one row
//            pair) and forms S_r = sum max(p_r P_r(x) - Q_r(x), 0) per warp segment
//            (Eq. "pacc_block"; p_r = 1 for Algorithm 1, Eq. "pres-token");
//   sample   every warp locates u * S_r among the segment totals; the one warp
//            that holds it rescans its segment in index order and sends the
//            candidate Y_r to rank 0.
// After the last position rank 0 forms h_i, selects tau and emits X^tau, Y_tau.
#include "bv_device.cuh"
#include "bv_launch.h"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace bv {

constexpr int kCThreads = 512;
constexpr int kCWarps = kCThreads / 32;
constexpr int kCSegs = kMaxCluster * kCWarps;   // warp segments of a row, in vocabulary order

struct ClusterShared {
    float4 x_ms[kCSegs];     // {ref P, sum P, ref Q, sum Q} of every warp of every CTA
    float x_seg[kCSegs];     // sweep-2 totals of every warp of every CTA
    unsigned long long bar_ms, bar_seg, bar_cand, bar_b;
    double p[kMaxGamma + 1];
    double S[kMaxGamma + 1];
    double h[kMaxGamma + 1];
    double lse_t[kMaxGamma + 1];
    double lse_d[kMaxGamma + 1];
    int cand[kMaxGamma + 1];
    int b_next;              // block this cluster works on next (-1: none left)
    int bad, tau, do_sweep2, last_row;
    float c, MP, MQ;
};

// sum_e 2^{v_e k - M}
template <int EPV> __device__ __forceinline__ float exp_sum(const float (&v)[EPV], float kf, float nM) {
    float a[EPV];
#pragma unroll
    for (int e = 0; e < EPV; ++e) a[e] = ex2(fmaf(v[e], kf, nM));
    float s0 = a[0] + a[1], s1 = a[2] + a[3];
    if (EPV == 8) { s0 += a[4] + a[5]; s1 += a[6] + a[7]; }
    return s0 + s1;
}

// Add one vector per lane to the warp's running (reference, sum).
template <int EPV> __device__ __forceinline__ void accumulate(const float (&v)[EPV], float kf, float& M, float& s) {
    float vs = exp_sum<EPV>(v, kf, -M);
    if (__any_sync(0xffffffffu, vs > kRaiseBound)) {      // some logit lies above the reference
        const float y = rintf(warp_max(vec_max<EPV>(v)) * kf);
        if (y > M) { s *= ref_scale(M, y); M = y; }
        vs = exp_sum<EPV>(v, kf, -M);
    }
    s += vs;
}

// residual terms of one vector pair: max(cp 2^{zP k - MP} - cq 2^{zQ k - MQ}, 0)
template <int EPV>
__device__ __forceinline__ void pair_terms(const float (&vp)[EPV], const float (&vq)[EPV], float kf, float cp,
                                           float cq, float nMP, float nMQ, float (&t)[EPV]) {
#pragma unroll
    for (int e = 0; e < EPV; ++e) {
        const float a = ex2(fmaf(vp[e], kf, nMP));
        const float q = ex2(fmaf(vq[e], kf, nMQ));
        t[e] = fmaxf(fmaf(cp, a, -(cq * q)), 0.f);
    }
}
template <int EPV> __device__ __forceinline__ float sum_terms(const float (&t)[EPV]) {
    float s0 = t[0] + t[1], s1 = t[2] + t[3];
    if (EPV == 8) { s0 += t[4] + t[5]; s1 += t[6] + t[7]; }
    return s0 + s1;
}

template <int DT> __device__ __forceinline__ void load_vec(const char* row, int i, float (&v)[Raw<DT>::EPV]) {
    Raw<DT>::unpack(ld_stream_v4(row + static_cast<size_t>(i) * 16), v);
}
// tail: lanes past the end of the segment see -inf logits
template <int DT>
__device__ __forceinline__ void load_vec_tail(const char* row, int i, int w1, float (&v)[Raw<DT>::EPV]) {
    if (i < w1) {
        load_vec<DT>(row, i, v);
    } else {
#pragma unroll
        for (int e = 0; e < Raw<DT>::EPV; ++e) v[e] = -INFINITY;
    }
}

template <int DT, int ALGO>
__global__ void __launch_bounds__(kCThreads, 2) verify_cluster_kernel(const Params prm) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;

    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int myseg = rank * kCWarps + warp;
    __shared__ ClusterShared sh;

    const int g = prm.gamma, V = prm.V, B = prm.B;
    const float kf = prm.kf;
    const double kd = prm.kd;
    const int units = V / EPV;
    const int u0 = static_cast<int>(static_cast<long long>(units) * rank / C);
    const int u1 = static_cast<int>(static_cast<long long>(units) * (rank + 1) / C);
    const int w0 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * warp / kCWarps);
    const int w1 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * (warp + 1) / kCWarps);
    const int wfull = w0 + ((w1 - w0) & ~31);      // end of the part every lane takes part in
    const size_t row_bytes = static_cast<size_t>(V) * ESZ;
    int* const status = prm.status;

    if (tid < kCSegs) {
        sh.x_ms[tid] = make_float4(kNoRef, 0.f, kNoRef, 0.f);   // ranks >= C stay neutral
        sh.x_seg[tid] = 0.f;
    }
    if (tid == 0) {
        mbar_init(smem_u32(&sh.bar_ms), 1);
        mbar_init(smem_u32(&sh.bar_seg), 1);
        mbar_init(smem_u32(&sh.bar_cand), 1);
        mbar_init(smem_u32(&sh.bar_b), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int peer = lane < C ? lane : 0;
    const uint32_t r_ms = map_to_rank(smem_u32(&sh.x_ms[myseg]), peer);
    const uint32_t r_seg = map_to_rank(smem_u32(&sh.x_seg[myseg]), peer);
    const uint32_t r_bar_ms = map_to_rank(smem_u32(&sh.bar_ms), peer);
    const uint32_t r_bar_seg = map_to_rank(smem_u32(&sh.bar_seg), peer);
    const uint32_t r_bar_cand = map_to_rank(smem_u32(&sh.bar_cand), 0);
    const uint32_t bytes_ms = static_cast<uint32_t>(C) * kCWarps * 16u;
    const uint32_t bytes_seg = static_cast<uint32_t>(C) * kCWarps * 4u;
    uint32_t ph_ms = 0, ph_seg = 0, ph_cand = 0, ph_b = 0;
    if (tid == 0) sh.b_next = -1;
    cluster.sync();   // barriers and exchange arrays are ready everywhere before any message

    for (;;) {
        // ---------------- next block: rank 0 draws a ticket and tells every CTA ----------------
        if (tid == 0) mbar_arrive_expect(smem_u32(&sh.bar_b), 4u);
        if (rank == 0 && tid == 0) {
            const unsigned t = atomicAdd(&prm.ticket[0], 1u);
            const uint32_t nb = t < static_cast<unsigned>(B) ? t : 0xffffffffu;
            for (int c = 0; c < C; ++c)
                send_b32(map_to_rank(smem_u32(&sh.b_next), c), map_to_rank(smem_u32(&sh.bar_b), c), nb);
        }
        // (a wait that gives up leaves sh.b_next at -1: the CTA goes to the final barrier without
        // ever using a block index that nobody sent)
        const bool told = mbar_wait(smem_u32(&sh.bar_b), ph_b, status);
        ph_b ^= 1u;
        const int b = told ? sh.b_next : -1;
        if (b < 0) break;

        if (tid <= g) {
            const double nan = __longlong_as_double(0x7ff8000000000000LL);
            sh.p[tid] = nan; sh.S[tid] = nan; sh.h[tid] = nan; sh.lse_t[tid] = nan; sh.lse_d[tid] = nan;
        }
        __syncthreads();
        if (tid == 0) {
            sh.bad = 0; sh.tau = 0;
            if (ALGO == kBlockVerify) sh.p[0] = 1.0;
            if (rank == 0)
                mbar_arrive_expect(smem_u32(&sh.bar_cand), ALGO == kBlockVerify ? 4u * static_cast<uint32_t>(g + 1) : 4u);
        }
        const char* tgt_b = static_cast<const char*>(prm.tgt) + static_cast<size_t>(b) * (g + 1) * row_bytes;
        const char* drf_b = static_cast<const char*>(prm.drf) + static_cast<size_t>(b) * g * row_bytes;

        for (int r = 0; r <= g; ++r) {
            const bool have_q = r < g;
            const char* rowP = tgt_b + static_cast<size_t>(r) * row_bytes;
            const char* rowQ = drf_b + static_cast<size_t>(r) * row_bytes;
            if (tid == 0) mbar_arrive_expect(smem_u32(&sh.bar_ms), bytes_ms);

            // thread 0: the drafted token's logits and this position's uniforms, fetched early
            double zp_x = 0.0, zq_x = 0.0;
            int x_ok = 1;
            float eta = 0.f;
            if (tid == 0 && have_q) {
                const int x = prm.tok[static_cast<size_t>(b) * g + r];
                x_ok = (x >= 0 && x < V);
                if (x_ok) { zp_x = load_logit<DT>(rowP, x); zq_x = load_logit<DT>(rowQ, x); }
                eta = prm.uni[static_cast<size_t>(b) * (g + 2) + r];
            }
            const float uf = prm.uni[static_cast<size_t>(b) * (g + 2) + (have_q ? g : g + 1)];

            // ---------------- sweep 1 ----------------
            float MPw = kNoRef, sP = 0.f, MQw = kNoRef, sQ = 0.f;
            {
                int i = w0 + lane;
                if (w0 < w1) {   // references from the first vector of every lane
                    float vp[EPV], vq[EPV];
                    load_vec_tail<DT>(rowP, i, w1, vp);
                    if (have_q) load_vec_tail<DT>(rowQ, i, w1, vq);
                    MPw = fmaxf(rintf(warp_max(vec_max<EPV>(vp)) * kf), kNoRef);
                    accumulate<EPV>(vp, kf, MPw, sP);
                    if (have_q) {
                        MQw = fmaxf(rintf(warp_max(vec_max<EPV>(vq)) * kf), kNoRef);
                        accumulate<EPV>(vq, kf, MQw, sQ);
                    }
                    i += 32;
                }
                int base = i - lane;          // warp-uniform start of the next step
                if (have_q) {
                    for (; base + 64 <= wfull; base += 64) {      // two steps in which every lane has a vector
                        float vp0[EPV], vq0[EPV], vp1[EPV], vq1[EPV];
                        load_vec<DT>(rowP, base + lane, vp0); load_vec<DT>(rowQ, base + lane, vq0);
                        load_vec<DT>(rowP, base + 32 + lane, vp1); load_vec<DT>(rowQ, base + 32 + lane, vq1);
                        accumulate<EPV>(vp0, kf, MPw, sP); accumulate<EPV>(vq0, kf, MQw, sQ);
                        accumulate<EPV>(vp1, kf, MPw, sP); accumulate<EPV>(vq1, kf, MQw, sQ);
                    }
                    for (; base < w1; base += 32) {
                        float vp[EPV], vq[EPV];
                        load_vec_tail<DT>(rowP, base + lane, w1, vp); load_vec_tail<DT>(rowQ, base + lane, w1, vq);
                        accumulate<EPV>(vp, kf, MPw, sP); accumulate<EPV>(vq, kf, MQw, sQ);
                    }
                } else {
                    for (; base < w1; base += 32) {
                        float vp[EPV];
                        load_vec_tail<DT>(rowP, base + lane, w1, vp);
                        accumulate<EPV>(vp, kf, MPw, sP);
                    }
                }
            }
            sP = warp_sum(sP);
            sQ = warp_sum(sQ);
            if (lane < C) send_v4(r_ms, r_bar_ms, MPw, sP, MQw, sQ);

            // ---------------- row normalisers, recursion / decision (warp 0) ----------------
            if (warp == 0) {
                mbar_wait(smem_u32(&sh.bar_ms), ph_ms, status);
                const float4 e0 = sh.x_ms[4 * lane], e1 = sh.x_ms[4 * lane + 1];
                const float4 e2 = sh.x_ms[4 * lane + 2], e3 = sh.x_ms[4 * lane + 3];
                const float MPr = warp_max(fmaxf(fmaxf(e0.x, e1.x), fmaxf(e2.x, e3.x)));
                const float MQr = warp_max(fmaxf(fmaxf(e0.z, e1.z), fmaxf(e2.z, e3.z)));
                double ZP = static_cast<double>(e0.y) * ref_scale(e0.x, MPr) + static_cast<double>(e1.y) * ref_scale(e1.x, MPr) +
                            static_cast<double>(e2.y) * ref_scale(e2.x, MPr) + static_cast<double>(e3.y) * ref_scale(e3.x, MPr);
                double ZQ = static_cast<double>(e0.w) * ref_scale(e0.z, MQr) + static_cast<double>(e1.w) * ref_scale(e1.z, MQr) +
                            static_cast<double>(e2.w) * ref_scale(e2.z, MQr) + static_cast<double>(e3.w) * ref_scale(e3.z, MQr);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) { ZP += shfl_xor_d(ZP, off); ZQ += shfl_xor_d(ZQ, off); }
                if (lane == 0) {
                    int bad = sh.bad;
                    // the row's maximum is finite iff its reference is; Z is NaN / inf iff the row
                    // holds a NaN / the sum overflowed
                    if (!(MPr > kNoRef && MPr < INFINITY) || !(ZP < INFINITY)) bad = 1;
                    if (have_q && (!(MQr > kNoRef && MQr < INFINITY) || !(ZQ < INFINITY))) bad = 1;
                    double ratio = 0.0;
                    if (have_q) {
                        if (!x_ok || zq_x == -INFINITY) bad = 1;
                        else ratio = exp2((zp_x - zq_x) * kd - static_cast<double>(MPr - MQr)) * (ZQ / ZP);
                    }
                    double p_r = 1.0;
                    int do2 = 1, last = 0;
                    if (ALGO == kBlockVerify) {
                        p_r = sh.p[r];
                        if (have_q) sh.p[r + 1] = fmin(p_r * ratio, 1.0);
                    } else if (have_q) {
                        const double h = fmin(ratio, 1.0);
                        sh.h[r + 1] = h;
                        if (!bad && h > 0.0 && static_cast<double>(eta) <= h) { sh.tau = r + 1; do2 = 0; }
                        else last = 1;
                        if (bad) {
                            do2 = 0;   // the one candidate this block owes rank 0
                            if (rank == 0) send_b32(map_to_rank(smem_u32(&sh.cand[0]), 0), r_bar_cand, 0xffffffffu);
                        }
                    } else if (bad) {
                        do2 = 0;
                        if (rank == 0) send_b32(map_to_rank(smem_u32(&sh.cand[0]), 0), r_bar_cand, 0xffffffffu);
                    }
                    sh.bad = bad;
                    sh.do_sweep2 = do2;
                    sh.last_row = last;
                    sh.c = have_q ? static_cast<float>(p_r * ZQ / ZP) : 1.f;
                    sh.MP = MPr;
                    sh.MQ = MQr;
                    sh.S[r] = have_q ? 1.0 / ZQ : 1.0 / ZP;   // scale of the segment totals, applied below
                    if (prm.out_lse_t) {
                        const double ln2 = 0.693147180559945309417232;
                        sh.lse_t[r] = (static_cast<double>(MPr) + log2(ZP)) * ln2;
                        if (have_q) sh.lse_d[r] = (static_cast<double>(MQr) + log2(ZQ)) * ln2;
                    }
                    if (do2) mbar_arrive_expect(smem_u32(&sh.bar_seg), bytes_seg);
                }
            }
            ph_ms ^= 1u;
            __syncthreads();
            const bool last_row = sh.last_row != 0;

            if (sh.do_sweep2) {
                const float nMP = -sh.MP, nMQ = -sh.MQ;
                bool use_q = have_q;
                for (int attempt = 0; attempt < 2; ++attempt) {
                    const float cp = use_q ? sh.c : 1.f;
                    const float cq = use_q ? 1.f : 0.f;
                    // ---------------- sweep 2 ----------------
                    float acc = 0.f;
                    {
                        int base = w0;
                        for (; base + 64 <= wfull; base += 64) {
                            float vp0[EPV], vq0[EPV], vp1[EPV], vq1[EPV], t0[EPV], t1[EPV];
                            load_vec<DT>(rowP, base + lane, vp0); load_vec<DT>(rowP, base + 32 + lane, vp1);
                            if (have_q) { load_vec<DT>(rowQ, base + lane, vq0); load_vec<DT>(rowQ, base + 32 + lane, vq1); }
                            else {
#pragma unroll
                                for (int e = 0; e < EPV; ++e) { vq0[e] = -INFINITY; vq1[e] = -INFINITY; }
                            }
                            pair_terms<EPV>(vp0, vq0, kf, cp, cq, nMP, nMQ, t0);
                            pair_terms<EPV>(vp1, vq1, kf, cp, cq, nMP, nMQ, t1);
                            acc += sum_terms<EPV>(t0) + sum_terms<EPV>(t1);
                        }
                        for (; base < w1; base += 32) {
                            float vp[EPV], vq[EPV], t[EPV];
                            load_vec_tail<DT>(rowP, base + lane, w1, vp);
                            if (have_q) load_vec_tail<DT>(rowQ, base + lane, w1, vq);
                            else {
#pragma unroll
                                for (int e = 0; e < EPV; ++e) vq[e] = -INFINITY;
                            }
                            pair_terms<EPV>(vp, vq, kf, cp, cq, nMP, nMQ, t);
                            acc += sum_terms<EPV>(t);
                        }
                    }
                    acc = warp_sum(acc);
                    if (lane < C) send_b32(r_seg, r_bar_seg, __float_as_uint(acc));
                    mbar_wait(smem_u32(&sh.bar_seg), ph_seg, status);
                    ph_seg ^= 1u;

                    // ---------------- locate u * total among the segment totals ----------------
                    const float4 t4 = reinterpret_cast<const float4*>(sh.x_seg)[lane];
                    const float l1 = t4.x, l2 = l1 + t4.y, l3 = l2 + t4.z, l4 = l3 + t4.w;
                    float inc = l4;
#pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const float o = __shfl_up_sync(0xffffffffu, inc, off);
                        if (lane >= off) inc += o;
                    }
                    const float total = __shfl_sync(0xffffffffu, inc, 31);
                    if (attempt == 0 && use_q && warp == 0) {
                        double sd = (static_cast<double>(t4.x) + static_cast<double>(t4.y)) +
                                    (static_cast<double>(t4.z) + static_cast<double>(t4.w));
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) sd += shfl_xor_d(sd, off);
                        if (lane == 0) sh.S[r] = sd * sh.S[r];
                    }
                    const bool empty = !(total > 0.f);
                    // (an empty residual leaves no candidate; should the position be selected all the same,
                    // which the algorithms cannot do, the block ends as a domain error)
                    if (!empty) {
                        const float t = uf * total;
                        float exc = __shfl_up_sync(0xffffffffu, inc, 1);
                        if (lane == 0) exc = 0.f;
                        const float p1 = exc + l1, p2 = exc + l2, p3 = exc + l3, p4 = exc + l4;
                        // first non-empty segment whose inclusive prefix exceeds t, else the last non-empty one
                        const bool h1 = p1 > t && t4.x > 0.f, h2 = p2 > t && t4.y > 0.f;
                        const bool h3 = p3 > t && t4.z > 0.f, h4 = p4 > t && t4.w > 0.f;
                        const unsigned hit = __ballot_sync(0xffffffffu, h1 || h2 || h3 || h4);
                        const unsigned nz = __ballot_sync(0xffffffffu, l4 > 0.f);
                        int sel_seg = -1;
                        float sel_before = 0.f;
                        if (hit) {
                            const int src = __ffs(hit) - 1;
                            int e = 3; float bef = p3;
                            if (h1) { e = 0; bef = exc; }
                            else if (h2) { e = 1; bef = p1; }
                            else if (h3) { e = 2; bef = p2; }
                            sel_seg = __shfl_sync(0xffffffffu, 4 * lane + e, src);
                            sel_before = __shfl_sync(0xffffffffu, bef, src);
                        } else if (nz) {
                            const int src = 31 - __clz(nz);
                            int e = 0; float bef = exc;
                            if (t4.w > 0.f) { e = 3; bef = p3; }
                            else if (t4.z > 0.f) { e = 2; bef = p2; }
                            else if (t4.y > 0.f) { e = 1; bef = p1; }
                            sel_seg = __shfl_sync(0xffffffffu, 4 * lane + e, src);
                            sel_before = __shfl_sync(0xffffffffu, bef, src);
                        }
                        if (sel_seg == myseg) {
                            // ---------------- rescan this warp's segment in index order ----------------
                            const float tw = t - sel_before;
                            float run = 0.f;
                            int found = -1, last_pos = -1;
                            for (int base = w0; base < w1 && found < 0; base += 32) {
                                const int i = base + lane;
                                float vp[EPV], vq[EPV], tt[EPV];
                                load_vec_tail<DT>(rowP, i, w1, vp);
                                if (have_q) load_vec_tail<DT>(rowQ, i, w1, vq);
                                else {
#pragma unroll
                                    for (int e = 0; e < EPV; ++e) vq[e] = -INFINITY;
                                }
                                pair_terms<EPV>(vp, vq, kf, cp, cq, nMP, nMQ, tt);
                                const float ls = sum_terms<EPV>(tt);
#pragma unroll
                                for (int e = 0; e < EPV; ++e) if (tt[e] > 0.f) last_pos = i * EPV + e;
                                float incw = ls;
#pragma unroll
                                for (int off = 1; off < 32; off <<= 1) {
                                    const float o = __shfl_up_sync(0xffffffffu, incw, off);
                                    if (lane >= off) incw += o;
                                }
                                const unsigned bal = __ballot_sync(0xffffffffu, run + incw > tw && ls > 0.f);
                                if (bal) {
                                    const int src = __ffs(bal) - 1;
                                    int f = -1;
                                    if (lane == src) {
                                        float cum = run + incw - ls;
                                        int lp = -1;
#pragma unroll
                                        for (int e = 0; e < EPV; ++e) {
                                            cum += tt[e];
                                            if (tt[e] > 0.f) lp = i * EPV + e;
                                            if (f < 0 && cum > tw && tt[e] > 0.f) f = i * EPV + e;
                                        }
                                        if (f < 0) f = lp;
                                    }
                                    found = __shfl_sync(0xffffffffu, f, src);
                                }
                                run += __shfl_sync(0xffffffffu, incw, 31);
                            }
                            if (found < 0) {
#pragma unroll
                                for (int off = 16; off > 0; off >>= 1)
                                    last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, off));
                                found = last_pos;
                            }
                            const int slot = ALGO == kBlockVerify ? r : 0;
                            if (lane == 0)
                                send_b32(map_to_rank(smem_u32(&sh.cand[slot]), 0), r_bar_cand, static_cast<uint32_t>(found));
                        }
                    } else if (myseg == 0 && lane == 0) {
                        // no candidate at this position: rank 0 is still owed its 4 bytes
                        const int slot = ALGO == kBlockVerify ? r : 0;
                        send_b32(map_to_rank(smem_u32(&sh.cand[slot]), 0), r_bar_cand, 0xffffffffu);
                    }
                    break;
                }
            }
            if (last_row) break;
        }

        // ---------------- end of the block: h, tau, emit (rank 0) ----------------
        if (rank == 0 && tid == 0) {
            mbar_wait(smem_u32(&sh.bar_cand), ph_cand, status);   // every candidate owed has landed
            int32_t* ot = prm.out_tokens + static_cast<size_t>(b) * (g + 1);
            const int32_t* X = prm.tok + static_cast<size_t>(b) * g;
            const float* u = prm.uni + static_cast<size_t>(b) * (g + 2);
            int tau = -1;
            if (!sh.bad) {
                sh.h[0] = 1.0;
                if (ALGO == kBlockVerify) {
                    // h_gamma = p_gamma; h_i = S_i / (S_i + 1 - p_i); tau = max{i : eta_i <= h_i}
                    for (int i = 1; i < g; ++i)
                        sh.h[i] = sh.S[i] > 0.0 ? sh.S[i] / (sh.S[i] + 1.0 - sh.p[i]) : 0.0;
                    sh.h[g] = sh.p[g];
                    tau = 0;
                    for (int i = g; i >= 1; --i)
                        if (sh.h[i] > 0.0 && static_cast<double>(u[i - 1]) <= sh.h[i]) { tau = i; break; }
                } else {
                    tau = sh.tau;
                }
            }
            for (int i = 0; i <= g; ++i) ot[i] = -1;
            // (nothing to sample from at the selected position: a domain error)
            if (tau >= 0 && sh.cand[ALGO == kBlockVerify ? tau : 0] < 0) tau = -1;
            if (tau >= 0) {
                for (int i = 0; i < tau; ++i) ot[i] = X[i];
                ot[tau] = sh.cand[ALGO == kBlockVerify ? tau : 0];
                prm.out_len[b] = tau + 1;
            } else {
                prm.out_len[b] = -1;
            }
            const double nan = __longlong_as_double(0x7ff8000000000000LL);
            for (int i = 0; i <= g; ++i) {
                const size_t o1 = static_cast<size_t>(b) * (g + 1) + i, o0 = static_cast<size_t>(b) * g + i;
                // Algorithm 1 forms S only at tau; other slots hold scales of positions it passed
                const double Si = (ALGO == kBlockVerify || i == tau) ? sh.S[i] : nan;
                if (prm.out_p) prm.out_p[o1] = static_cast<float>(sh.p[i]);
                if (prm.out_h) prm.out_h[o1] = static_cast<float>(sh.h[i]);
                if (prm.out_lse_t) prm.out_lse_t[o1] = static_cast<float>(sh.lse_t[i]);
                if (i < g && prm.out_S) prm.out_S[o0] = static_cast<float>(Si);
                if (i < g && prm.out_lse_d) prm.out_lse_d[o0] = static_cast<float>(sh.lse_d[i]);
            }
        }
        ph_cand ^= 1u;
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
    cluster.sync();   // no CTA exits while a peer may still write into its shared memory
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
using CKernelFn = void (*)(const Params);

static CKernelFn pick_cluster_kernel(int algo, int dtype) {
    if (algo == kBlockVerify)
        return dtype == kF32 ? verify_cluster_kernel<kF32, kBlockVerify> : verify_cluster_kernel<kBF16, kBlockVerify>;
    return dtype == kF32 ? verify_cluster_kernel<kF32, kTokenVerify> : verify_cluster_kernel<kBF16, kTokenVerify>;
}

static void fill_cconfig(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int cluster, int nclusters,
                         cudaStream_t stream) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(static_cast<unsigned>(cluster * nclusters), 1, 1);
    cfg.blockDim = dim3(kCThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

int cluster_max_clusters(int algo, int dtype, int cluster) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_cconfig(cfg, attr, cluster, 1, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, reinterpret_cast<const void*>(pick_cluster_kernel(algo, dtype)), &cfg) !=
        cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t launch_cluster(const Params& prm, int algo, int dtype, int cluster, int nclusters, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_cconfig(cfg, attr, cluster, nclusters, stream);
    return cudaLaunchKernelEx(&cfg, pick_cluster_kernel(algo, dtype), prm);
}

}  // namespace bv
