// Block Verification (Algorithm 2) with each row pair read from HBM exactly once.
//
// A cluster of C CTAs owns one drafted block at a time and walks its positions
// r = 0..gamma.  Every thread owns up to NK 16-byte vectors of P_r and of Q_r
// (contiguous segments per warp, contiguous slices per CTA, so partial sums are
// in vocabulary order).  For each position:
//
//   sweep 1  the thread's vectors arrive through a private ring of cp.async
//            copies that runs NK/2 vectors ahead (across positions and blocks, so
//            HBM stays busy during the reductions).  Each logit is exponentiated
//            ONCE: a_x = 2^{zP k - M} stays in registers, b_x = 2^{zQ k - M'} goes
//            to shared memory as fp32.  Sums of a and b give the normalisers.
//   scalars  cluster-wide combine (DSMEM + cluster barrier), then the drafted
//            token's ratio and p_{r+1} = min(p_r ratio, 1)  (Eq. "def_as").
//   sweep 2  S_r = sum max(p_r P_r(x) - Q_r(x), 0)  (Eq. "pacc_block") from the
//            cached a and b: no global loads, no exponentials.
//   sample   candidate Y_r by inverse CDF over the per-warp segment totals; the
//            one warp that holds u * S_r rescans its cached terms.
//
// References: a warp exponentiates against its own integer reference M, the rounded
// scaled maximum of what it has seen so far, so that the exponent z k - M of every
// large term stays small and its single fp32 rounding is harmless.  M starts as the
// maximum of the warp's first 32 vectors; a later vector whose terms sum to more
// than 12 (some logit lies above M) raises M and rescales the terms cached so far
// by an exact power of two.  References differ between warps by integers, so every
// later rescale is exact as well.
#include "bv_device.cuh"
#include "bv_launch.h"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace bv {

constexpr int kRThreads = 512;
constexpr int kRWarps = kRThreads / 32;
constexpr int kSegs = kMaxCluster * kRWarps;   // warp segments of a row, in vocabulary order
struct ResShared {
    // sweep 1: {reference P, sum P, reference Q, sum Q} of every warp of every CTA, sent by
    // the owners to every CTA of the cluster; index rank * 16 + warp
    float4 x_ms[kSegs];
    // sweep 2: segment totals of every warp of every CTA, same indexing
    float x_seg[kSegs];
    // transaction barriers that count the bytes of the two exchanges and of the candidates
    unsigned long long bar_ms, bar_seg, bar_cand;
    double p[kMaxGamma + 1];
    double S[kMaxGamma + 1];
    double h[kMaxGamma + 1];
    double lse_t[kMaxGamma + 1];
    double lse_d[kMaxGamma + 1];
    int cand[kMaxGamma + 1];
    int bad;
    float c;          // p_r Z_Q / Z_P
    float MP, MQ;     // row references
};

// a_e = 2^{v_e k - M} and their sum (branch-free; -inf logits give 0, NaN stays NaN)
template <int EPV>
__device__ __forceinline__ float expo(const float (&v)[EPV], float kf, float M, float (&a)[EPV]) {
    const float nM = -M;
#pragma unroll
    for (int e = 0; e < EPV; ++e) a[e] = ex2(fmaf(v[e], kf, nM));
    float s0 = a[0] + a[1], s1 = a[2] + a[3];
    if (EPV == 8) { s0 += a[4] + a[5]; s1 += a[6] + a[7]; }
    return s0 + s1;
}

template <int DT, int NK>
__global__ void __launch_bounds__(kRThreads, 1) verify_resident_kernel(const Params prm) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr int HV = EPV / 4;          // float4s per cached vector
    constexpr int L = NK / 2;            // k-steps of lookahead
    constexpr int D = 2 * L;             // ring depth in vectors (P and Q alternate)
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    static_assert(NK % 2 == 0, "NK must be even");

    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int cid = blockIdx.x / C;
    const int ncl = prm.nclusters;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int myseg = rank * kRWarps + warp;

    __shared__ ResShared sh;
    extern __shared__ __align__(16) unsigned char dyn[];
    float4* bcache = reinterpret_cast<float4*>(dyn) + tid;                                   // [NK][HV][512]
    uint4* ring = reinterpret_cast<uint4*>(dyn + sizeof(float4) * NK * HV * kRThreads) + tid;  // [D][512]

    const int g = prm.gamma, V = prm.V, B = prm.B;
    const float kf = prm.kf;
    const double kd = prm.kd;
    const int units = V / EPV;
    const int u0 = static_cast<int>(static_cast<long long>(units) * rank / C);
    const int u1 = static_cast<int>(static_cast<long long>(units) * (rank + 1) / C);
    const int w0 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * warp / kRWarps);
    const int w1 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * (warp + 1) / kRWarps);
    const int v0 = w0 + lane;            // this thread's k-th vector is v0 + 32 k, valid below w1
    unsigned vmask = 0;                  // bit k: vector k exists
#pragma unroll
    for (int k = 0; k < NK; ++k) vmask |= (v0 + 32 * k < w1) ? (1u << k) : 0u;
    const size_t row_bytes = static_cast<size_t>(V) * ESZ;
    const size_t toff = static_cast<size_t>(v0) * 16;   // byte offset of vector 0 inside a row

    // unused slots of the exchange arrays (ranks >= C) stay neutral for the whole kernel
    if (tid < kSegs) {
        sh.x_ms[tid] = make_float4(kNoRef, 0.f, kNoRef, 0.f);
        sh.x_seg[tid] = 0.f;
    }
    if (tid == 0) {
        mbar_init(smem_u32(&sh.bar_ms), 1);
        mbar_init(smem_u32(&sh.bar_seg), 1);
        mbar_init(smem_u32(&sh.bar_cand), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // where this warp's messages go: lane l < C addresses CTA l of the cluster
    const int peer = lane < C ? lane : 0;
    const uint32_t r_ms = map_to_rank(smem_u32(&sh.x_ms[myseg]), peer);
    const uint32_t r_seg = map_to_rank(smem_u32(&sh.x_seg[myseg]), peer);
    const uint32_t r_bar_ms = map_to_rank(smem_u32(&sh.bar_ms), peer);
    const uint32_t r_bar_seg = map_to_rank(smem_u32(&sh.bar_seg), peer);
    const uint32_t r_bar_cand = map_to_rank(smem_u32(&sh.bar_cand), 0);
    const uint32_t bytes_ms = static_cast<uint32_t>(C) * kRWarps * 16u;
    const uint32_t bytes_seg = static_cast<uint32_t>(C) * kRWarps * 4u;
    uint32_t ph_ms = 0, ph_seg = 0, ph_cand = 0;     // phase parities of the three barriers
    int* const status = prm.status;

    auto rowP = [&](int b, int r) -> const char* {
        return static_cast<const char*>(prm.tgt) + (static_cast<size_t>(b) * (g + 1) + r) * row_bytes + toff;
    };
    auto rowQ = [&](int b, int r) -> const char* {
        return static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * row_bytes + toff;
    };
    auto fetch = [&](const char* row, int k, int slot) {
        ring_fetch(ring + slot * kRThreads, row + k * 512, row != nullptr && ((vmask >> k) & 1u), R::kNegInf);
    };

    // prologue: the first L k-steps of the first position
    {
        const char* p0 = cid < B ? rowP(cid, 0) : nullptr;
        const char* q0 = cid < B ? rowQ(cid, 0) : nullptr;
#pragma unroll
        for (int k = 0; k < L; ++k) {
            fetch(p0, k, 2 * k);
            fetch(q0, k, 2 * k + 1);
        }
    }
    cluster.sync();   // barriers and exchange arrays are ready everywhere before any message

    for (int b = cid; b < B; b += ncl) {
        if (tid == 0) {
            sh.bad = 0; sh.p[0] = 1.0;
            if (rank == 0) mbar_arrive_expect(smem_u32(&sh.bar_cand), 4u * static_cast<uint32_t>(g + 1));
        }
        for (int r = 0; r <= g; ++r) {
            const bool have_q = r < g;
            int nb = b, nr = r + 1;
            if (nr > g) { nr = 0; nb = b + ncl; }
            const char* curP = rowP(b, r);
            const char* curQ = have_q ? rowQ(b, r) : nullptr;
            const char* nxtP = nb < B ? rowP(nb, nr) : nullptr;
            const char* nxtQ = (nb < B && nr < g) ? rowQ(nb, nr) : nullptr;

            if (tid == 0) {
                mbar_arrive_expect(smem_u32(&sh.bar_ms), bytes_ms);
                mbar_arrive_expect(smem_u32(&sh.bar_seg), bytes_seg);
            }
            // thread 0 fetches the drafted token's two logits early (used after the combine)
            double zp_x = 0.0, zq_x = 0.0;
            int x_ok = 1;
            if (tid == 0 && have_q) {
                const int x = prm.tok[static_cast<size_t>(b) * g + r];
                x_ok = (x >= 0 && x < V);
                if (x_ok) {
                    zp_x = load_logit<DT>(curP - toff, x);
                    zq_x = load_logit<DT>(curQ - toff, x);
                }
            }

            // ---------------- sweep 1 ----------------
            float a[NK][EPV];
            float MPw = kNoRef, sP = 0.f, MQw = kNoRef, sQ = 0.f;   // references are warp-uniform
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                const int slotP = (2 * k) % D, slotQ = (2 * k + 1) % D;
                cp_async_wait<D - 2>();          // vectors k of both rows have landed
                float vp[EPV], vq[EPV], bq[EPV];
                R::unpack(ring[slotP * kRThreads], vp);
                R::unpack(ring[slotQ * kRThreads], vq);   // -inf pattern when there is no draft row
                if (k == 0) {
                    MPw = fmaxf(rintf(warp_max(vec_max<EPV>(vp)) * kf), kNoRef);
                    MQw = fmaxf(rintf(warp_max(vec_max<EPV>(vq)) * kf), kNoRef);
                }
                float vsP = expo<EPV>(vp, kf, MPw, a[k]);
                float vsQ = expo<EPV>(vq, kf, MQw, bq);
                if (__any_sync(0xffffffffu, vsP > kRaiseBound)) {
                    const float y = rintf(warp_max(vec_max<EPV>(vp)) * kf);
                    if (y > MPw) {
                        const float f = ref_scale(MPw, y);
                        sP *= f;
#pragma unroll
                        for (int kk = 0; kk < k; ++kk)
#pragma unroll
                            for (int e = 0; e < EPV; ++e) a[kk][e] *= f;
                        MPw = y;
                    }
                    vsP = expo<EPV>(vp, kf, MPw, a[k]);
                }
                if (__any_sync(0xffffffffu, vsQ > kRaiseBound)) {
                    const float y = rintf(warp_max(vec_max<EPV>(vq)) * kf);
                    if (y > MQw) {
                        const float f = ref_scale(MQw, y);
                        sQ *= f;
#pragma unroll
                        for (int kk = 0; kk < k; ++kk)
#pragma unroll
                            for (int hv = 0; hv < HV; ++hv) {
                                float4 t4 = bcache[(kk * HV + hv) * kRThreads];
                                t4.x *= f; t4.y *= f; t4.z *= f; t4.w *= f;
                                bcache[(kk * HV + hv) * kRThreads] = t4;
                            }
                        MQw = y;
                    }
                    vsQ = expo<EPV>(vq, kf, MQw, bq);
                }
                sP += vsP;
                sQ += vsQ;
#pragma unroll
                for (int hv = 0; hv < HV; ++hv)
                    bcache[(k * HV + hv) * kRThreads] =
                        make_float4(bq[4 * hv], bq[4 * hv + 1], bq[4 * hv + 2], bq[4 * hv + 3]);
                if (k + L < NK) { fetch(curP, k + L, slotP); fetch(curQ, k + L, slotQ); }
                else            { fetch(nxtP, k + L - NK, slotP); fetch(nxtQ, k + L - NK, slotQ); }
            }

            // ---------------- publish this warp's partials to every CTA ----------------
            sP = warp_sum(sP);
            sQ = warp_sum(sQ);
            if (lane < C) send_v4(r_ms, r_bar_ms, MPw, sP, MQw, sQ);

            // ---------------- row normalisers and the scale of sweep 2 (warp 0) ----------------
            double ZP = 0.0, ZQ = 0.0;     // meaningful in thread 0
            float MPr = 0.f, MQr = 0.f;
            if (warp == 0) {
                mbar_wait(smem_u32(&sh.bar_ms), ph_ms, status);
                // lane l combines segments 4l .. 4l+3
                const float4 e0 = sh.x_ms[4 * lane], e1 = sh.x_ms[4 * lane + 1];
                const float4 e2 = sh.x_ms[4 * lane + 2], e3 = sh.x_ms[4 * lane + 3];
                MPr = warp_max(fmaxf(fmaxf(e0.x, e1.x), fmaxf(e2.x, e3.x)));
                MQr = warp_max(fmaxf(fmaxf(e0.z, e1.z), fmaxf(e2.z, e3.z)));
                ZP = static_cast<double>(e0.y) * ref_scale(e0.x, MPr) + static_cast<double>(e1.y) * ref_scale(e1.x, MPr) +
                     static_cast<double>(e2.y) * ref_scale(e2.x, MPr) + static_cast<double>(e3.y) * ref_scale(e3.x, MPr);
                ZQ = static_cast<double>(e0.w) * ref_scale(e0.z, MQr) + static_cast<double>(e1.w) * ref_scale(e1.z, MQr) +
                     static_cast<double>(e2.w) * ref_scale(e2.z, MQr) + static_cast<double>(e3.w) * ref_scale(e3.z, MQr);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) { ZP += shfl_xor_d(ZP, off); ZQ += shfl_xor_d(ZQ, off); }
                if (lane == 0) {
                    sh.c = have_q ? static_cast<float>(sh.p[r] * ZQ / ZP) : 1.f;
                    sh.MP = MPr;
                    sh.MQ = MQr;
                }
            }
            ph_ms ^= 1u;
            __syncthreads();

            // thread 0, overlapped with sweep 2: data checks and p_{r+1} = min(p_r ratio, 1)
            double invZ = 0.0;
            if (tid == 0) {
                int bad = sh.bad;
                // the row's maximum is finite iff its reference is; Z is NaN / inf iff the row
                // holds a NaN / the sum overflowed
                if (!(MPr > kNoRef && MPr < INFINITY) || !(ZP < INFINITY)) bad = 1;
                if (have_q && (!(MQr > kNoRef && MQr < INFINITY) || !(ZQ < INFINITY))) bad = 1;
                if (have_q) {
                    double ratio = 0.0;
                    if (!x_ok || zq_x == -INFINITY) bad = 1;
                    else ratio = exp2((zp_x - zq_x) * kd - static_cast<double>(MPr - MQr)) * (ZQ / ZP);
                    sh.p[r + 1] = fmin(sh.p[r] * ratio, 1.0);
                }
                sh.bad = bad;
                invZ = have_q ? 1.0 / ZQ : 1.0 / ZP;
                if (prm.out_lse_t) {
                    const double ln2 = 0.693147180559945309417232;
                    sh.lse_t[r] = (static_cast<double>(MPr) + log2(ZP)) * ln2;
                    if (have_q) sh.lse_d[r] = (static_cast<double>(MQr) + log2(ZQ)) * ln2;
                }
            }

            // ---------------- sweep 2 + candidate ----------------
            const float cPw = ref_scale(MPw, sh.MP);      // exact rescale to the row references
            const float cQw = ref_scale(MQw, sh.MQ);
            bool use_q = have_q;
            for (int attempt = 0; attempt < 2; ++attempt) {
                const float cp = use_q ? sh.c * cPw : cPw;
                const float cq = use_q ? cQw : 0.f;
                float acc = 0.f;
                float vsum[NK];      // this thread's residual mass per vector, kept for the rescan
#pragma unroll
                for (int k = 0; k < NK; ++k) {
                    float bq[EPV], tt[EPV];
#pragma unroll
                    for (int hv = 0; hv < HV; ++hv) {
                        const float4 f = bcache[(k * HV + hv) * kRThreads];
                        bq[4 * hv] = f.x; bq[4 * hv + 1] = f.y; bq[4 * hv + 2] = f.z; bq[4 * hv + 3] = f.w;
                    }
#pragma unroll
                    for (int e = 0; e < EPV; ++e) tt[e] = fmaxf(fmaf(cp, a[k][e], -(cq * bq[e])), 0.f);
                    float s0 = tt[0] + tt[1], s1 = tt[2] + tt[3];
                    if (EPV == 8) { s0 += tt[4] + tt[5]; s1 += tt[6] + tt[7]; }
                    vsum[k] = s0 + s1;
                    acc += vsum[k];
                }
                acc = warp_sum(acc);
                if (lane < C) send_b32(r_seg, r_bar_seg, __float_as_uint(acc));
                mbar_wait(smem_u32(&sh.bar_seg), ph_seg, status);
                ph_seg ^= 1u;

                // every warp locates u * total among the 128 segment totals (index order)
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
                    if (lane == 0) sh.S[r] = sd * invZ;
                }
                const bool empty = !(total > 0.f);
                if (empty && use_q && attempt == 0 && r == 0) {
                    use_q = false;   // empty residual at position 0: sample P_0 with the same uniform
                    cluster.sync();  // every warp of every CTA has read x_seg before it is rewritten
                    if (tid == 0) mbar_arrive_expect(smem_u32(&sh.bar_seg), bytes_seg);
                    continue;
                }
                if (!empty) {
                    const float uf = prm.uni[static_cast<size_t>(b) * (g + 2) + (have_q ? g : g + 1)];
                    const float t = uf * total;
                    // exclusive prefix of this lane; p1..p4 = inclusive prefixes of its four segments
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
                        int e = 3; float bef = exc + l3;
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
                        // This warp holds u * S_r.  Its segment is ordered vector-major: step k covers
                        // 32 consecutive vectors, one per lane.  Row totals of the NK steps first,
                        // then a lane scan inside the one step that crosses the target.
                        const float tw = t - sel_before;
                        float rowtot[NK];
#pragma unroll
                        for (int k = 0; k < NK; ++k) rowtot[k] = warp_sum(vsum[k]);
                        int ks = -1, klast = -1;
                        float before = 0.f, ks_before = 0.f, klast_before = 0.f;
#pragma unroll
                        for (int k = 0; k < NK; ++k) {
                            if (rowtot[k] > 0.f) { klast = k; klast_before = before; }
                            if (ks < 0 && rowtot[k] > 0.f && before + rowtot[k] > tw) { ks = k; ks_before = before; }
                            before += rowtot[k];
                        }
                        if (ks < 0) { ks = klast; ks_before = klast_before; }
                        int found = -1;
#pragma unroll
                        for (int k = 0; k < NK; ++k) {
                            if (k == ks) {       // warp-uniform
                                const float tk = tw - ks_before;
                                const float ls = vsum[k];
                                float incw = ls;
#pragma unroll
                                for (int off = 1; off < 32; off <<= 1) {
                                    const float o = __shfl_up_sync(0xffffffffu, incw, off);
                                    if (lane >= off) incw += o;
                                }
                                const unsigned bal = __ballot_sync(0xffffffffu, incw > tk && ls > 0.f);
                                const unsigned nzl = __ballot_sync(0xffffffffu, ls > 0.f);
                                const int src = bal ? __ffs(bal) - 1 : 31 - __clz(nzl);
                                int f = -1;
                                if (lane == src) {
                                    float bq[EPV];
#pragma unroll
                                    for (int hv = 0; hv < HV; ++hv) {
                                        const float4 f4 = bcache[(k * HV + hv) * kRThreads];
                                        bq[4 * hv] = f4.x; bq[4 * hv + 1] = f4.y; bq[4 * hv + 2] = f4.z; bq[4 * hv + 3] = f4.w;
                                    }
                                    float cum = incw - ls;
                                    int lp = -1;
                                    const int i = v0 + 32 * k;
#pragma unroll
                                    for (int e = 0; e < EPV; ++e) {
                                        const float te = fmaxf(fmaf(cp, a[k][e], -(cq * bq[e])), 0.f);
                                        cum += te;
                                        if (te > 0.f) lp = i * EPV + e;
                                        if (f < 0 && cum > tk && te > 0.f) f = i * EPV + e;
                                    }
                                    if (f < 0) f = lp;
                                }
                                found = __shfl_sync(0xffffffffu, f, src);
                            }
                        }
                        if (lane == 0)
                            send_b32(map_to_rank(smem_u32(&sh.cand[r]), 0), r_bar_cand, static_cast<uint32_t>(found));
                    }
                } else if (myseg == 0 && lane == 0) {
                    // no candidate at this position: rank 0 is still owed its 4 bytes
                    send_b32(map_to_rank(smem_u32(&sh.cand[r]), 0), r_bar_cand, 0xffffffffu);
                }
                break;
            }
        }

        // ---------------- end of the block: h, tau, emit (rank 0) ----------------
        if (rank == 0 && tid == 0) {
            mbar_wait(smem_u32(&sh.bar_cand), ph_cand, status);   // all gamma+1 candidates have landed
            int32_t* ot = prm.out_tokens + static_cast<size_t>(b) * (g + 1);
            const int32_t* X = prm.tok + static_cast<size_t>(b) * g;
            const float* u = prm.uni + static_cast<size_t>(b) * (g + 2);
            int tau = -1;
            if (!sh.bad) {
                // h_gamma = p_gamma; h_i = S_i / (S_i + 1 - p_i); tau = max{i : eta_i <= h_i}
                sh.h[0] = 1.0;
                for (int i = 1; i < g; ++i)
                    sh.h[i] = sh.S[i] > 0.0 ? sh.S[i] / (sh.S[i] + 1.0 - sh.p[i]) : 0.0;
                sh.h[g] = sh.p[g];
                tau = 0;
                for (int i = g; i >= 1; --i)
                    if (sh.h[i] > 0.0 && static_cast<double>(u[i - 1]) <= sh.h[i]) { tau = i; break; }
            }
            for (int i = 0; i <= g; ++i) ot[i] = -1;
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
        ph_cand ^= 1u;
    }
    cp_async_wait<0>();
    cluster.sync();   // no CTA exits while a peer may still write into its shared memory
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
using RKernelFn = void (*)(const Params);

static RKernelFn pick_resident(int dtype, int nk) {
    if (dtype == kBF16) {
        switch (nk) {
            case 2: return verify_resident_kernel<kBF16, 2>;
            case 4: return verify_resident_kernel<kBF16, 4>;
            case 8: return verify_resident_kernel<kBF16, 8>;
        }
    } else {
        switch (nk) {
            case 2: return verify_resident_kernel<kF32, 2>;
            case 4: return verify_resident_kernel<kF32, 4>;
            case 8: return verify_resident_kernel<kF32, 8>;
        }
    }
    return nullptr;
}

static size_t resident_smem(int dtype, int nk) {
    const int hv = dtype == kBF16 ? 2 : 1;
    return sizeof(float4) * nk * hv * kRThreads + sizeof(uint4) * nk * kRThreads;
}

int resident_vectors_per_cta(int nk) { return nk * 32 * kRWarps; }

static void fill_rconfig(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int cluster, int nclusters,
                         size_t smem, cudaStream_t stream) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(static_cast<unsigned>(cluster * nclusters), 1, 1);
    cfg.blockDim = dim3(kRThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

int resident_max_clusters(int dtype, int nk, int cluster) {
    RKernelFn fn = pick_resident(dtype, nk);
    if (!fn) return 0;
    const size_t smem = resident_smem(dtype, nk);
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_rconfig(cfg, attr, cluster, 1, smem, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, reinterpret_cast<const void*>(fn), &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

cudaError_t launch_resident(const Params& prm, int dtype, int nk, int cluster, int nclusters,
                            cudaStream_t stream) {
    RKernelFn fn = pick_resident(dtype, nk);
    if (!fn) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_rconfig(cfg, attr, cluster, nclusters, resident_smem(dtype, nk), stream);
    return cudaLaunchKernelEx(&cfg, fn, prm);
}

}  // namespace bv
