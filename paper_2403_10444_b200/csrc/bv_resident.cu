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
// A vector of 8 terms all at the reference sums to at most 8 * 2^0.5 = 11.3; a sum above
// this bound therefore means some term exceeds 2^0.5, i.e. its logit lies above the reference.
// Without a raise every term is below 12, so its exponent is below 4 and is rounded to 1.2e-7.
constexpr float kRaiseBound = 12.f;

struct ResShared {
    float red_M[2][kRWarps];
    double red_s[2][kRWarps];
    float x_M[2][kMaxCluster];
    double x_s[2][kMaxCluster];
    double segtot[kRWarps];
    double x_tot[kMaxCluster];
    double p[kMaxGamma + 1];
    double S[kMaxGamma + 1];
    double h[kMaxGamma + 1];
    double lse_t[kMaxGamma + 1];
    double lse_d[kMaxGamma + 1];
    int cand[kMaxGamma + 1];
    int bad;
    float c;
    float MP, MQ;
    double invZQ;
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int DT> struct Raw;
template <> struct Raw<kBF16> {
    static constexpr int EPV = 8;
    static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[8]) {
        v[0] = __uint_as_float(r.x << 16); v[1] = __uint_as_float(r.x & 0xffff0000u);
        v[2] = __uint_as_float(r.y << 16); v[3] = __uint_as_float(r.y & 0xffff0000u);
        v[4] = __uint_as_float(r.z << 16); v[5] = __uint_as_float(r.z & 0xffff0000u);
        v[6] = __uint_as_float(r.w << 16); v[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};
template <> struct Raw<kF32> {
    static constexpr int EPV = 4;
    static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[4]) {
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y);
        v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
};

template <int EPV> __device__ __forceinline__ float vec_max(const float (&v)[EPV]) {
    float vm = v[0];
#pragma unroll
    for (int e = 1; e < EPV; ++e) vm = fmaxf(vm, v[e]);
    return vm;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, off));
    return x;
}

// a_e = 2^{v_e k - M} and their sum; with no finite reference yet the terms are 0
// (a NaN logit is carried into the sum so that the row is flagged).
template <int EPV>
__device__ __forceinline__ float expo(const float (&v)[EPV], bool valid, float kf, float M, float (&a)[EPV]) {
    float vs = 0.f;
    if (valid && M > -INFINITY) {
        const float nM = -M;
#pragma unroll
        for (int e = 0; e < EPV; ++e) { a[e] = ex2(fmaf(v[e], kf, nM)); vs += a[e]; }
    } else {
#pragma unroll
        for (int e = 0; e < EPV; ++e) { a[e] = 0.f; if (valid && v[e] != v[e]) vs = v[e]; }
    }
    return vs;
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

    __shared__ ResShared sh;
    extern __shared__ __align__(16) unsigned char dyn[];
    float4* bcache = reinterpret_cast<float4*>(dyn);                       // [NK][HV][512]
    uint4* ring = reinterpret_cast<uint4*>(dyn + sizeof(float4) * NK * HV * kRThreads);  // [D][512]

    const int g = prm.gamma, V = prm.V, B = prm.B;
    const float kf = prm.kf;
    const double kd = prm.kd;
    const int units = V / EPV;
    const int u0 = static_cast<int>(static_cast<long long>(units) * rank / C);
    const int u1 = static_cast<int>(static_cast<long long>(units) * (rank + 1) / C);
    const int w0 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * warp / kRWarps);
    const int w1 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * (warp + 1) / kRWarps);
    const int v0 = w0 + lane;            // this thread's k-th vector is v0 + 32 k, valid below w1
    const size_t row_bytes = static_cast<size_t>(V) * ESZ;

    auto rowP = [&](int b, int r) -> const char* {
        return static_cast<const char*>(prm.tgt) + (static_cast<size_t>(b) * (g + 1) + r) * row_bytes;
    };
    auto rowQ = [&](int b, int r) -> const char* {
        return static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * row_bytes;
    };
    // one ring item: vector k of a row (null row: nothing to fetch); always one commit group
    auto fetch = [&](const char* row, int k, int slot) {
        if (row != nullptr && v0 + 32 * k < w1)
            cp_async16(&ring[slot * kRThreads + tid], row + static_cast<size_t>(v0 + 32 * k) * 16);
        cp_async_commit();
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

    for (int b = cid; b < B; b += ncl) {
        if (tid == 0) { sh.bad = 0; sh.p[0] = 1.0; }
        for (int r = 0; r <= g; ++r) {
            const bool have_q = r < g;
            // rows of the next position in this cluster's stream (for the lookahead)
            int nb = b, nr = r + 1;
            if (nr > g) { nr = 0; nb = b + ncl; }
            const char* curP = rowP(b, r);
            const char* curQ = have_q ? rowQ(b, r) : nullptr;
            const char* nxtP = nb < B ? rowP(nb, nr) : nullptr;
            const char* nxtQ = (nb < B && nr < g) ? rowQ(nb, nr) : nullptr;

            // ---------------- sweep 1 ----------------
            float a[NK][EPV];
            float MPw = -INFINITY, sP = 0.f, MQw = -INFINITY, sQ = 0.f;   // references are warp-uniform
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                const bool valid = v0 + 32 * k < w1;
                const int slotP = (2 * k) % D, slotQ = (2 * k + 1) % D;
                // ---- target row ----
                cp_async_wait<D - 1>();
                {
                    float v[EPV];
                    if (valid) R::unpack(ring[slotP * kRThreads + tid], v);
                    else {
#pragma unroll
                        for (int e = 0; e < EPV; ++e) v[e] = -INFINITY;
                    }
                    bool raise;
                    float vs = 0.f;
                    if (MPw > -INFINITY) {
                        vs = expo<EPV>(v, valid, kf, MPw, a[k]);
                        raise = __any_sync(0xffffffffu, vs > kRaiseBound);
                    } else {
                        raise = true;   // no finite logit seen yet: look for one
                    }
                    if (raise) {
                        const float y = rintf(warp_max(vec_max<EPV>(v)) * kf);
                        if (y > MPw) {
                            const float f = pow2_nonpos(MPw - y);
                            sP = (sP != sP) ? sP : sP * f;
#pragma unroll
                            for (int kk = 0; kk < k; ++kk)
#pragma unroll
                                for (int e = 0; e < EPV; ++e) a[kk][e] *= f;
                            MPw = y;
                        }
                        vs = expo<EPV>(v, valid, kf, MPw, a[k]);
                    }
                    sP += vs;
                }
                if (k + L < NK) fetch(curP, k + L, slotP); else fetch(nxtP, k + L - NK, slotP);
                // ---- draft row ----
                cp_async_wait<D - 1>();
                {
                    const bool qvalid = valid && have_q;
                    float v[EPV], bq[EPV];
                    if (qvalid) R::unpack(ring[slotQ * kRThreads + tid], v);
                    else {
#pragma unroll
                        for (int e = 0; e < EPV; ++e) v[e] = -INFINITY;
                    }
                    bool raise;
                    float vs = 0.f;
                    if (MQw > -INFINITY) {
                        vs = expo<EPV>(v, qvalid, kf, MQw, bq);
                        raise = __any_sync(0xffffffffu, vs > kRaiseBound);
                    } else {
                        raise = have_q;
                    }
                    if (raise) {
                        const float y = rintf(warp_max(vec_max<EPV>(v)) * kf);
                        if (y > MQw) {
                            const float f = pow2_nonpos(MQw - y);
                            sQ = (sQ != sQ) ? sQ : sQ * f;
#pragma unroll
                            for (int kk = 0; kk < k; ++kk)
#pragma unroll
                                for (int hv = 0; hv < HV; ++hv) {
                                    float4 t4 = bcache[(kk * HV + hv) * kRThreads + tid];
                                    t4.x *= f; t4.y *= f; t4.z *= f; t4.w *= f;
                                    bcache[(kk * HV + hv) * kRThreads + tid] = t4;
                                }
                            MQw = y;
                        }
                        vs = expo<EPV>(v, qvalid, kf, MQw, bq);
                    }
                    sQ += vs;
#pragma unroll
                    for (int hv = 0; hv < HV; ++hv)
                        bcache[(k * HV + hv) * kRThreads + tid] =
                            make_float4(bq[4 * hv], bq[4 * hv + 1], bq[4 * hv + 2], bq[4 * hv + 3]);
                }
                if (k + L < NK) fetch(curQ, k + L, slotQ); else fetch(nxtQ, k + L - NK, slotQ);
            }

            // ---------------- combine: warp -> CTA -> cluster ----------------
            float sPw = sP, sQw = sQ;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                sPw += __shfl_xor_sync(0xffffffffu, sPw, off);
                sQw += __shfl_xor_sync(0xffffffffu, sQw, off);
            }
            if (lane == 0) {
                sh.red_M[0][warp] = MPw; sh.red_s[0][warp] = static_cast<double>(sPw);
                sh.red_M[1][warp] = MQw; sh.red_s[1][warp] = static_cast<double>(sQw);
            }
            __syncthreads();
            if (warp == 0) {
#pragma unroll
                for (int row = 0; row < 2; ++row) {
                    float M = lane < kRWarps ? sh.red_M[row][lane] : -INFINITY;
                    double s = lane < kRWarps ? sh.red_s[row][lane] : 0.0;
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

            // ---------------- scalars ----------------
            if (warp == 0) {
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
                    if (!(fabsf(MP) < INFINITY) || !(ZP < INFINITY)) bad = 1;   // also catches NaN
                    if (have_q && (!(fabsf(MQ) < INFINITY) || !(ZQ < INFINITY))) bad = 1;
                    const double lse2P = static_cast<double>(MP) + log2(ZP);
                    const double lse2Q = static_cast<double>(MQ) + log2(ZQ);
                    sh.lse_t[r] = lse2P * ln2;
                    if (have_q) sh.lse_d[r] = lse2Q * ln2;
                    const double p_r = sh.p[r];
                    if (have_q) {
                        double ratio = 0.0;
                        const int x = prm.tok[static_cast<size_t>(b) * g + r];
                        if (x < 0 || x >= V) {
                            bad = 1;
                        } else {
                            const double zq = load_logit<DT>(curQ, x), zp = load_logit<DT>(curP, x);
                            if (zq == -INFINITY) bad = 1;
                            else ratio = exp2((zp * kd - lse2P) - (zq * kd - lse2Q));
                        }
                        sh.p[r + 1] = fmin(p_r * ratio, 1.0);
                    }
                    sh.bad = bad;
                    sh.c = have_q ? static_cast<float>(p_r * ZQ / ZP) : 1.f;
                    sh.MP = MP;
                    sh.MQ = MQ;
                    sh.invZQ = have_q ? 1.0 / ZQ : 1.0 / ZP;
                    if (rank == 0) sh.cand[r] = -1;
                }
            }
            __syncthreads();

            // ---------------- sweep 2 + candidate ----------------
            const float c = sh.c;
            const float cPt = c * pow2_nonpos(MPw - sh.MP);     // exact rescale to the row reference
            const float cQt = pow2_nonpos(MQw - sh.MQ);
            bool use_q = have_q;
            for (int attempt = 0; attempt < 2; ++attempt) {
                const float cp = use_q ? cPt : pow2_nonpos(MPw - sh.MP);
                float acc = 0.f;
#pragma unroll
                for (int k = 0; k < NK; ++k) {
                    float bq[EPV];
#pragma unroll
                    for (int hv = 0; hv < HV; ++hv) {
                        const float4 f = bcache[(k * HV + hv) * kRThreads + tid];
                        bq[4 * hv] = f.x; bq[4 * hv + 1] = f.y; bq[4 * hv + 2] = f.z; bq[4 * hv + 3] = f.w;
                    }
                    float v = 0.f;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        const float q = use_q ? cQt * bq[e] : 0.f;
                        v += fmaxf(fmaf(cp, a[k][e], -q), 0.f);
                    }
                    acc += v;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (lane == 0) sh.segtot[warp] = static_cast<double>(acc);
                __syncthreads();
                if (warp == 0) {
                    double v = lane < kRWarps ? sh.segtot[lane] : 0.0;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) v += shfl_xor_d(v, off);
                    if (lane < C) *cluster.map_shared_rank(&sh.x_tot[rank], lane) = v;
                }
                cluster.sync();

                double total = 0.0;
                for (int k = 0; k < C; ++k) total += sh.x_tot[k];
                if (attempt == 0 && use_q && tid == 0) sh.S[r] = total * sh.invZQ;
                const bool empty = !(total > 0.0);
                if (empty && use_q && attempt == 0 && r == 0) {
                    use_q = false;   // empty residual at position 0: sample P_0 with the same uniform
                    cluster.sync();
                    continue;
                }
                if (!empty) {
                    const float uf = prm.uni[static_cast<size_t>(b) * (g + 2) + (have_q ? g : g + 1)];
                    const double t = static_cast<double>(uf) * total;
                    int sel = -1, lastnz = -1;
                    double run = 0.0, sel_before = 0.0, nz_before = 0.0;
                    for (int k = 0; k < C; ++k) {
                        const double v = sh.x_tot[k];
                        if (v > 0.0) { lastnz = k; nz_before = run; }
                        if (sel < 0 && run + v > t) { sel = k; sel_before = run; }
                        run += v;
                    }
                    if (sel < 0) { sel = lastnz; sel_before = nz_before; }
                    if (sel == rank) {
                        const double tc = t - sel_before;
                        int wsel = -1, wlast = -1;
                        double wrun = 0.0, wsel_before = 0.0, wnz_before = 0.0;
                        for (int k = 0; k < kRWarps; ++k) {
                            const double v = sh.segtot[k];
                            if (v > 0.0) { wlast = k; wnz_before = wrun; }
                            if (wsel < 0 && wrun + v > tc) { wsel = k; wsel_before = wrun; }
                            wrun += v;
                        }
                        if (wsel < 0) { wsel = wlast; wsel_before = wnz_before; }
                        if (warp == wsel) {
                            // rescan this warp's cached terms in index order
                            const double tw = tc - wsel_before;
                            double runw = 0.0;
                            int found = -1, last_pos = -1;
#pragma unroll
                            for (int k = 0; k < NK; ++k) {
                                if (found < 0) {
                                    float tt[EPV];
                                    float ls = 0.f;
#pragma unroll
                                    for (int hv = 0; hv < HV; ++hv) {
                                        const float4 f = bcache[(k * HV + hv) * kRThreads + tid];
                                        tt[4 * hv] = f.x; tt[4 * hv + 1] = f.y; tt[4 * hv + 2] = f.z; tt[4 * hv + 3] = f.w;
                                    }
                                    const int i = v0 + 32 * k;
#pragma unroll
                                    for (int e = 0; e < EPV; ++e) {
                                        const float q = use_q ? cQt * tt[e] : 0.f;
                                        tt[e] = fmaxf(fmaf(cp, a[k][e], -q), 0.f);
                                        ls += tt[e];
                                        if (tt[e] > 0.f) last_pos = i * EPV + e;
                                    }
                                    double inc = static_cast<double>(ls);
#pragma unroll
                                    for (int off = 1; off < 32; off <<= 1) {
                                        const double o = shfl_up_d(inc, off);
                                        if (lane >= off) inc += o;
                                    }
                                    const bool hit = runw + inc > tw;
                                    const unsigned bal = __ballot_sync(0xffffffffu, hit);
                                    if (bal) {
                                        const int src = __ffs(bal) - 1;
                                        int f = -1;
                                        if (lane == src) {
                                            double cum = runw + inc - static_cast<double>(ls);
                                            int lp = -1;
#pragma unroll
                                            for (int e = 0; e < EPV; ++e) {
                                                cum += static_cast<double>(tt[e]);
                                                if (tt[e] > 0.f) lp = i * EPV + e;
                                                if (f < 0 && cum > tw && tt[e] > 0.f) f = i * EPV + e;
                                            }
                                            if (f < 0) f = lp;
                                        }
                                        f = __shfl_sync(0xffffffffu, f, src);
                                        if (f >= 0) found = f;
                                    }
                                    runw += shfl_d(inc, 31);
                                }
                            }
                            if (found < 0) {
#pragma unroll
                                for (int off = 16; off > 0; off >>= 1)
                                    last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, off));
                                found = last_pos;
                            }
                            if (lane == 0) *cluster.map_shared_rank(&sh.cand[r], 0) = found;
                        }
                    }
                }
                break;
            }
        }

        // ---------------- end of the block: h, tau, emit (rank 0) ----------------
        cluster.sync();   // every candidate has landed in rank 0's shared memory
        if (rank == 0 && tid == 0) {
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
    }
    cp_async_wait<0>();
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
