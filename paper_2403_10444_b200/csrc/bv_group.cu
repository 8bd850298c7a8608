// Block Verification (Algorithm 2) with every logit read from HBM exactly once.
//
// The CTAs (one per SM, all resident: a cooperative launch) form groups of G.  A group takes
// one row pair (P_r, Q_r) per step and walks through its blocks row by row; CTA j of the group
// owns share j of every row: one 16-byte vector per consumer thread and row.  The share is
// copied into a ring of shared-memory buffers by one bulk asynchronous copy per row (TMA) and
// stays there until both sweeps over it are done:
//
//   sweep 1 (step n)      per lane sum 2^{z k - M} under a warp-wide integer reference M; the
//                         CTA's {M, Z} pair of both rows goes to scratch.
//   between               the release warp of every CTA collects the G pairs of the row as they
//                         appear, forms the normalisers and advances the prefix recursion
//                         p_{r+1} = min(p_r P_r(X)/Q_r(X), 1) (Eq. "def_as") - each CTA for itself,
//                         in the same order, so nobody waits for a designated CTA.
//   sweep 2 (step n + L)  straight from shared memory: per lane sum max(p_r P_r(x) - Q_r(x), 0)
//                         (Eq. "pacc_block"); one total per warp goes to scratch.
//
// The L steps in between hide the exchange through L2 (no cluster is large enough to hold a row
// pair of a 256k vocabulary, so the exchange cannot use distributed shared memory).  One CTA per
// block, the block's owner, adds the totals to S_r, draws the candidate Y_r (Eq. "pres-block")
// and, after the last position, forms h_i, selects tau and emits.
//
// Roles in a CTA: 28 consumer warps (both sweeps; no loads, no reductions), the copy thread, the
// release warp, the post warp (per-lane results -> scratch) and the owner warp.  The order of all
// work is fixed by the launch geometry, so results do not depend on timing.  Every wait is
// bounded; a wait that gives up sets the status word and the role returns.
#include "bv_flow_common.cuh"

#include <climits>

namespace bv {

constexpr int kGWarps = 28;                       // consumer warps
constexpr int kGThreads = kGWarps * 32;
constexpr int kGCopy = kGWarps, kGRel = kGWarps + 1, kGPost = kGWarps + 2, kGOwner = kGWarps + 3;
constexpr int kGAllThreads = (kGWarps + 4) * 32;  // 1024
constexpr int kGShareVecs = kGThreads;            // vectors of one row in a CTA's share
constexpr int kGRowBytes = kGShareVecs * 16;
constexpr int kGBuf = 7;                          // shares resident per CTA
constexpr int kGR = 2;                            // per-lane result slots per sweep
constexpr size_t kGroupSmem = static_cast<size_t>(kGBuf) * 2 * kGRowBytes +
                              static_cast<size_t>(kGR) * 3 * kGShareVecs * sizeof(float);

struct GroupShared {
    unsigned long long bfull[kGBuf];      // the share's bytes have landed
    unsigned long long bfree[kGBuf];      // all consumer warps have read the share for the second time
    unsigned long long s2ready[kGR];      // the release warp has left the scalars of a second sweep
    unsigned long long done1[kGR], free1[kGR];   // sweep-1 results written / read by the post warp
    unsigned long long done2[kGR], free2[kGR];   // sweep-2 results
    float wref[kGR][2][kGWarps];          // sweep 1: warp references of P and Q
    float4 meta2[kGR];                    // sweep 2: p_r Z_Q / Z_P, minus the row references
};

struct GroupGeom {
    int G, NG;        // CTAs per group, groups
    int L;            // steps between the two sweeps of a share
};

// try_wait without a suspend-time hint: the thread resumes as soon as the phase completes
__device__ __forceinline__ bool g_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool g_wait(uint32_t bar, uint32_t parity, int* status) {
    for (uint32_t spins = 0; !g_try(bar, parity); ++spins) {
        if (spins > (1u << 24)) {
            if (status) atomicExch(status, 1);
            return false;
        }
    }
    return true;
}
// bulk copy global -> shared, completion counted in bytes by an mbarrier of this CTA
__device__ __forceinline__ void g_bulk(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void g_sts(uint32_t saddr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(saddr), "f"(v) : "memory");
}
__device__ __forceinline__ unsigned g_ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// counter += 1, ordered after this thread's earlier writes; nothing comes back
__device__ __forceinline__ void g_red_release(unsigned* p) {
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
// warp-wide integer reference of one vector per lane: round(max * k)
template <int EPV> __device__ __forceinline__ float g_ref(const float (&v)[EPV], float kf) {
    const int m = __reduce_max_sync(0xffffffffu, __float2int_rn(vec_max<EPV>(v) * kf));
    return m == INT_MIN ? kNoRef : static_cast<float>(m);
}

// A ring position that advances one slot at a time: slot index and how often it has been used.
struct GRing {
    int idx = 0;
    uint32_t use = 0;
    __device__ __forceinline__ void next(int size) { if (++idx == size) { idx = 0; ++use; } }
    __device__ __forceinline__ uint32_t parity() const { return use & 1u; }               // this use
    __device__ __forceinline__ uint32_t prev_parity() const { return (use & 1u) ^ 1u; }   // the use before
};

// Row statistics from the G pairs in scratch (whole warp; all lanes return the same values).
__device__ __forceinline__ void g_combine(const FlowScratch& fl, size_t rowi, int G, int lane,
                                          double& MP, double& ZP, double& MQ, double& ZQ) {
    MP = kNoRef; MQ = kNoRef;
    for (int ch = lane; ch < G; ch += 32) {
        const RowZ z = load_rowz(&fl.part[rowi * G + ch]);
        MP = fmax(MP, z.MP); MQ = fmax(MQ, z.MQ);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { MP = fmax(MP, shfl_xor_d(MP, off)); MQ = fmax(MQ, shfl_xor_d(MQ, off)); }
    ZP = 0.0; ZQ = 0.0;
    for (int ch = lane; ch < G; ch += 32) {
        const RowZ z = load_rowz(&fl.part[rowi * G + ch]);
        ZP += z.ZP * static_cast<double>(ref_scale(static_cast<float>(z.MP), static_cast<float>(MP)));
        ZQ += z.ZQ * static_cast<double>(ref_scale(static_cast<float>(z.MQ), static_cast<float>(MQ)));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { ZP += shfl_xor_d(ZP, off); ZQ += shfl_xor_d(ZQ, off); }
}

// The drafted token's two logits of row (b, r), r < gamma: what the ratio P_r(X)/Q_r(X) needs
// besides the normalisers.  ok = false: token out of range or impossible under the draft.
template <int DT>
__device__ __forceinline__ void g_token_logits(const Params& prm, const FlowCtx& cx, int b, int r,
                                               double& zp, double& zq, bool& ok) {
    const int g = cx.g;
    const int x = prm.tok[static_cast<size_t>(b) * g + r];
    ok = x >= 0 && x < cx.V;
    zp = 0.0; zq = 0.0;
    if (ok) {
        const char* rowP = static_cast<const char*>(prm.tgt) + (static_cast<size_t>(b) * (g + 1) + r) * cx.row_bytes;
        const char* rowQ = static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes;
        zq = load_logit<DT>(rowQ, x);
        zp = load_logit<DT>(rowP, x);
        if (zq == -INFINITY) ok = false;
    }
}

template <int DT>
__global__ void __launch_bounds__(kGAllThreads, 1)
verify_group_kernel(const Params prm, const FlowScratch fl, const GroupGeom geo) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ GroupShared sh;
    extern __shared__ __align__(128) unsigned char dyn[];
    float* part1 = reinterpret_cast<float*>(dyn + static_cast<size_t>(kGBuf) * 2 * kGRowBytes);   // [kGR][2][share]
    float* part2 = part1 + kGR * 2 * kGShareVecs;                                                 // [kGR][share]

    FlowCtx cx;
    cx.g = prm.gamma; cx.V = prm.V; cx.B = prm.B; cx.nch = geo.G; cx.units = prm.V / EPV;
    cx.row_bytes = static_cast<size_t>(prm.V) * ESZ; cx.kf = prm.kf; cx.kd = prm.kd;
    const int g = cx.g, G = geo.G, NG = geo.NG, L = geo.L;
    const float kf = cx.kf;
    const int grp = blockIdx.x / G, j = blockIdx.x % G;
    const int nblk = grp < cx.B ? (cx.B - grp + NG - 1) / NG : 0;       // blocks grp, grp + NG, ...
    const int N = nblk * (g + 1);                                       // steps (row pairs) of this group
    const int v0 = j * kGShareVecs;
    const int valid = min(kGShareVecs, cx.units - v0);                  // vectors in this CTA's share
    const int nseg = G * kGWarps;

    if (tid == 0) {
        for (int i = 0; i < kGBuf; ++i) {
            mbar_init(smem_u32(&sh.bfull[i]), 1);
            mbar_init(smem_u32(&sh.bfree[i]), kGWarps);
        }
        for (int i = 0; i < kGR; ++i) {
            mbar_init(smem_u32(&sh.s2ready[i]), 1);
            mbar_init(smem_u32(&sh.done1[i]), kGWarps);
            mbar_init(smem_u32(&sh.free1[i]), 1);
            mbar_init(smem_u32(&sh.done2[i]), kGWarps);
            mbar_init(smem_u32(&sh.free2[i]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (N == 0) return;

    if (warp == kGCopy) {
        // =============================== copy thread ===============================
        if (lane != 0) return;
        const uint32_t base = smem_u32(dyn);
        const uint32_t bytes = static_cast<uint32_t>(valid) * 16u;
        GRing buf;
        int q = 0, r = 0;
        for (int n = 0; n < N; ++n) {
            if (buf.use > 0 && !g_wait(smem_u32(&sh.bfree[buf.idx]), buf.prev_parity(), prm.status)) return;
            const int b = grp + q * NG;
            const bool have_q = r < g;
            const uint32_t bar = smem_u32(&sh.bfull[buf.idx]);
            mbar_arrive_expect(bar, have_q ? 2u * bytes : bytes);
            const uint32_t dst = base + static_cast<uint32_t>(buf.idx) * (2u * kGRowBytes);
            g_bulk(dst, static_cast<const char*>(prm.tgt) + (static_cast<size_t>(b) * (g + 1) + r) * cx.row_bytes +
                            static_cast<size_t>(v0) * 16, bytes, bar);
            if (have_q)
                g_bulk(dst + kGRowBytes, static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes +
                                             static_cast<size_t>(v0) * 16, bytes, bar);
            buf.next(kGBuf);
            if (++r > g) { r = 0; ++q; }
        }
        return;
    }

    if (warp == kGRel) {
        // =============================== release warp ===============================
        // Row after row: wait until all G pairs of the row are in scratch, combine them, advance the
        // recursion and hand the scalars of the row's second sweep to the consumers.
        GRing slot;
        int q = 0, r = 0;
        double p = 1.0;
        double zp = 0.0, zq = 0.0;
        bool tok_ok = false;
        if (lane == 0) g_token_logits<DT>(prm, cx, grp, 0, zp, zq, tok_ok);
        for (int n = 0; n < N; ++n) {
            const int b = grp + q * NG;
            const size_t rowi = static_cast<size_t>(b) * (g + 1) + r;
            for (unsigned spins = 0; g_ld_acquire(&fl.row_cnt[rowi]) != static_cast<unsigned>(G); ++spins) {
                if (spins > (1u << 22)) { if (prm.status) atomicExch(prm.status, 1); return; }
            }
            double MP, ZP, MQ, ZQ;
            g_combine(fl, rowi, G, lane, MP, ZP, MQ, ZQ);
            float cs = 1.f;
            if (lane == 0) {
                if (r == 0) p = 1.0;
                if (r < g) {
                    cs = static_cast<float>(p * (ZQ / ZP));
                    const double ratio = tok_ok ? exp2((zp - zq) * cx.kd - (MP - MQ)) * (ZQ / ZP) : 0.0;
                    p = fmin(p * ratio, 1.0);
                }
                // the next row's token logits: on their way while the consumers are being served
                const int rn = r == g ? 0 : r + 1, bn = r == g ? b + NG : b;
                if (n + 1 < N && rn < g) g_token_logits<DT>(prm, cx, bn, rn, zp, zq, tok_ok);
            }
            if (slot.use > 0 && !g_wait(smem_u32(&sh.done2[slot.idx]), slot.prev_parity(), prm.status)) return;
            if (lane == 0) {
                sh.meta2[slot.idx] = make_float4(cs, -static_cast<float>(MP), -static_cast<float>(MQ), 0.f);
                mbar_arrive(smem_u32(&sh.s2ready[slot.idx]));
            }
            __syncwarp();
            slot.next(kGR);
            if (++r > g) { r = 0; ++q; }
        }
        return;
    }

    if (warp == kGPost) {
        // =============================== post warp ===============================
        // per-lane results of the consumers -> the CTA's entries in scratch, in the consumers' order
        GRing s1, s2;
        int q1 = 0, r1 = 0, q2 = 0, r2 = 0;
        for (int n = 0; n < N + L; ++n) {
            if (n < N) {
                if (!g_wait(smem_u32(&sh.done1[s1.idx]), s1.parity(), prm.status)) return;
                const size_t rowi = static_cast<size_t>(grp + q1 * NG) * (g + 1) + r1;
                // lane l adds up consumer warp l (fp64), each lane starting elsewhere: no bank conflicts
                const float* lp = part1 + static_cast<size_t>(s1.idx) * 2 * kGShareVecs + lane * 32;
                double zP = 0.0, zQ = 0.0;
                float mP = kNoRef, mQ = kNoRef;
                if (lane < kGWarps) {
#pragma unroll 8
                    for (int i = 0; i < 32; ++i) {
                        const int k = (i + lane) & 31;
                        zP += static_cast<double>(lp[k]);
                        zQ += static_cast<double>(lp[kGShareVecs + k]);
                    }
                    mP = sh.wref[s1.idx][0][lane]; mQ = sh.wref[s1.idx][1][lane];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.free1[s1.idx]));
                const float MPc = warp_max(mP), MQc = warp_max(mQ);
                zP *= static_cast<double>(ref_scale(mP, MPc));
                zQ *= static_cast<double>(ref_scale(mQ, MQc));
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) { zP += shfl_xor_d(zP, off); zQ += shfl_xor_d(zQ, off); }
                if (lane == 0) {
                    RowZ z; z.MP = MPc; z.ZP = zP; z.MQ = MQc; z.ZQ = zQ;
                    fl.part[rowi * G + j] = z;
                    g_red_release(&fl.row_cnt[rowi]);
                }
                s1.next(kGR);
                if (++r1 > g) { r1 = 0; ++q1; }
            }
            if (n >= L) {
                if (!g_wait(smem_u32(&sh.done2[s2.idx]), s2.parity(), prm.status)) return;
                const size_t rowi = static_cast<size_t>(grp + q2 * NG) * (g + 1) + r2;
                const float* lp = part2 + static_cast<size_t>(s2.idx) * kGShareVecs + lane * 32;
                double t = 0.0;
                if (lane < kGWarps) {
#pragma unroll 8
                    for (int i = 0; i < 32; ++i) t += static_cast<double>(lp[(i + lane) & 31]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.free2[s2.idx]));
                if (lane < kGWarps) {
                    // a segment is one consumer warp's 32 vectors: contiguous in the row
                    fl.seg_tot[rowi * nseg + j * kGWarps + lane] = static_cast<float>(t);
                    g_red_release(&fl.s2_cnt[rowi]);
                }
                s2.next(kGR);
                if (++r2 > g) { r2 = 0; ++q2; }
            }
        }
        return;
    }

    if (warp == kGOwner) {
        // =============================== owner warp ===============================
        // CTA j owns the group's blocks j, j + G, ...: it publishes their normalisers and p_i,
        // completes their positions (S_r, candidate) and finishes them.
        const unsigned all_segs = static_cast<unsigned>(nseg);
        for (int q = j; q < nblk; q += G) {
            const int b = grp + q * NG;
            double* pc = fl.pchain + static_cast<size_t>(b) * (g + 2);
            double p = 1.0, zp = 0.0, zq = 0.0;
            bool tok_ok = false;
            if (lane == 0 && g > 0) g_token_logits<DT>(prm, cx, b, 0, zp, zq, tok_ok);
            int fold_r = 0, pos_r = 0;
            unsigned idle = 0;
            while (pos_r <= g) {
                const size_t row_f = static_cast<size_t>(b) * (g + 1) + min(fold_r, g);
                const size_t row_p = static_cast<size_t>(b) * (g + 1) + pos_r;
                const unsigned c1 = fold_r <= g ? g_ld_acquire(&fl.row_cnt[row_f]) : 0u;
                const unsigned c2 = pos_r < fold_r ? g_ld_acquire(&fl.s2_cnt[row_p]) : 0u;
                bool did = false;
                if (fold_r <= g && c1 == static_cast<unsigned>(G)) {
                    const int r = fold_r;
                    double MP, ZP, MQ, ZQ;
                    g_combine(fl, row_f, G, lane, MP, ZP, MQ, ZQ);
                    if (lane == 0) {
                        RowZ out; out.MP = MP; out.ZP = ZP; out.MQ = MQ; out.ZQ = ZQ;
                        fl.rowZ[row_f] = out;
                        const bool have_q = r < g;
                        // the row's maximum is finite iff its reference is; Z is NaN / inf iff the row holds a NaN / overflowed
                        bool bad = !(MP > kNoRef && MP < INFINITY) || !(ZP < INFINITY);
                        if (have_q) bad = bad || !(MQ > kNoRef && MQ < INFINITY) || !(ZQ < INFINITY) || !tok_ok;
                        if (bad) atomicOr(&fl.bad[b], 1u);
                        pc[r] = p;
                        float cs = 1.f;
                        if (have_q) {
                            cs = static_cast<float>(p * (ZQ / ZP));
                            const double ratio = tok_ok ? exp2((zp - zq) * cx.kd - (MP - MQ)) * (ZQ / ZP) : 0.0;
                            p = fmin(p * ratio, 1.0);
                        }
                        fl.cscale[row_f] = cs;
                        if (r + 1 < g) g_token_logits<DT>(prm, cx, b, r + 1, zp, zq, tok_ok);
                        __threadfence();
                    }
                    __syncwarp();
                    ++fold_r;
                    did = true;
                }
                if (pos_r < fold_r && c2 == all_segs) {
                    const int r = pos_r;
                    const bool have_q = r < g;
                    const char* rowP = static_cast<const char*>(prm.tgt) + row_p * cx.row_bytes;
                    const char* rowQ = have_q ? static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes
                                              : nullptr;
                    const float cs = __ldcg(&fl.cscale[row_p]);
                    const float nMP = -static_cast<float>(__ldcg(&fl.rowZ[row_p].MP));
                    const float nMQ = -static_cast<float>(__ldcg(&fl.rowZ[row_p].MQ));
                    const int units = cx.units;
                    f_position_complete<DT>(prm, fl, cx, static_cast<int>(row_p), have_q, rowP, rowQ, cs, nMP, nMQ, nseg,
                                            fl.seg_tot + row_p * nseg, lane, [units](int sel, int& s0, int& s1) {
                                                s0 = min(sel * 32, units);
                                                s1 = min(sel * 32 + 32, units);
                                            });
                    ++pos_r;
                    did = true;
                }
                if (did) { idle = 0; continue; }
                __nanosleep(100);
                if (++idle > (1u << 23)) { if (prm.status) atomicExch(prm.status, 1); return; }
            }
        }
        return;
    }

    // =============================== consumer warps ===============================
    const uint32_t my = smem_u32(dyn) + static_cast<uint32_t>(tid) * 16u;
    const uint32_t p1 = smem_u32(part1) + static_cast<uint32_t>(tid) * 4u;
    const uint32_t p2 = smem_u32(part2) + static_cast<uint32_t>(tid) * 4u;
    const uint4 ninf = make_uint4(R::kNegInf, R::kNegInf, R::kNegInf, R::kNegInf);
    const bool mine = tid < valid;
    GRing b1, b2, s1, s2;
    int r1 = 0, r2 = 0;
    for (int n = 0; n < N + L; ++n) {
        if (n < N) {
            // ---- sweep 1 of step n ----
            if (!g_wait(smem_u32(&sh.bfull[b1.idx]), b1.parity(), prm.status)) return;
            const bool have_q = r1 < g;
            const uint32_t a = my + static_cast<uint32_t>(b1.idx) * (2u * kGRowBytes);
            uint4 rp = ninf, rq = ninf;
            if (mine) { rp = lds128(a); if (have_q) rq = lds128(a + kGRowBytes); }
            float vp[EPV], vq[EPV];
            R::unpack(rp, vp);
            R::unpack(rq, vq);
            const float MPw = g_ref<EPV>(vp, kf);
            const float MQw = have_q ? g_ref<EPV>(vq, kf) : kNoRef;
            const float vsP = f_exp_sum<EPV>(vp, kf, -MPw);
            const float vsQ = have_q ? f_exp_sum<EPV>(vq, kf, -MQw) : 0.f;
            if (s1.use > 0 && !g_wait(smem_u32(&sh.free1[s1.idx]), s1.prev_parity(), prm.status)) return;
            const uint32_t o = p1 + static_cast<uint32_t>(s1.idx) * (2u * kGShareVecs * 4u);
            g_sts(o, vsP);
            g_sts(o + kGShareVecs * 4u, vsQ);
            if (lane == 0) { sh.wref[s1.idx][0][warp] = MPw; sh.wref[s1.idx][1][warp] = MQw; }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.done1[s1.idx]));
            b1.next(kGBuf);
            s1.next(kGR);
            if (++r1 > g) r1 = 0;
        }
        if (n >= L) {
            // ---- sweep 2 of step n - L, from the same shared-memory share ----
            if (!g_wait(smem_u32(&sh.s2ready[s2.idx]), s2.parity(), prm.status)) return;
            const float4 m = sh.meta2[s2.idx];
            const bool have_q = r2 < g;
            const uint32_t a = my + static_cast<uint32_t>(b2.idx) * (2u * kGRowBytes);
            uint4 rp = ninf, rq = ninf;
            if (mine) { rp = lds128(a); if (have_q) rq = lds128(a + kGRowBytes); }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.bfree[b2.idx]));      // the share may be replaced
            float vp[EPV], vq[EPV], t[EPV];
            R::unpack(rp, vp);
            R::unpack(rq, vq);
            const float acc = have_q ? f_pair_sum<EPV, true>(vp, vq, kf, m.x, m.y, m.z, t)
                                     : f_pair_sum<EPV, false>(vp, vq, kf, m.x, m.y, m.z, t);
            if (s2.use > 0 && !g_wait(smem_u32(&sh.free2[s2.idx]), s2.prev_parity(), prm.status)) return;
            g_sts(p2 + static_cast<uint32_t>(s2.idx) * (kGShareVecs * 4u), acc);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.done2[s2.idx]));
            b2.next(kGBuf);
            s2.next(kGR);
            if (++r2 > g) r2 = 0;
        }
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
using GKernelFn = void (*)(const Params, const FlowScratch, const GroupGeom);
static GKernelFn pick_group(int dtype) {
    return dtype == kF32 ? verify_group_kernel<kF32> : verify_group_kernel<kBF16>;
}

int group_share_vectors() { return kGShareVecs; }
int group_segments_per_share() { return kGWarps; }
int group_max_lag() { return kGBuf - 2; }

int group_max_ctas_per_sm(int dtype) {
    int n = 0;
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(pick_group(dtype)),
                             cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kGroupSmem)) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pick_group(dtype), kGAllThreads, kGroupSmem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

// G CTAs per group, NG groups, L steps between the sweeps; the launch is cooperative because the
// CTAs of a group wait for one another: all of them must be resident.
cudaError_t launch_group(const Params& prm, const FlowScratch& fl, int dtype, int G, int NG, int L,
                         cudaStream_t stream) {
    GroupGeom geo;
    geo.G = G; geo.NG = NG; geo.L = L;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(G * NG));
    cfg.blockDim = dim3(kGAllThreads);
    cfg.dynamicSmemBytes = kGroupSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, pick_group(dtype), prm, fl, geo);
}

}  // namespace bv
