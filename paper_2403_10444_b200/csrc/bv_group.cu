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
// counter += 1; nothing comes back and nothing is ordered: a hint for whoever polls
__device__ __forceinline__ void g_red_relaxed(unsigned* p) {
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
// warp-wide integer reference of one vector per lane: round(max * k)
template <int EPV> __device__ __forceinline__ float g_ref(const float (&v)[EPV], float kf) {
    const int m = __reduce_max_sync(0xffffffffu, __float2int_rn(vec_max<EPV>(v) * kf));
    return m == INT_MIN ? kNoRef : static_cast<float>(m);
}

// Sum of the 32 floats at p as a balanced tree (the same shape as a warp shuffle reduction), read
// in an order that starts at a different element in every lane so that the lanes of a warp, each
// summing its own 32, never meet in a shared-memory bank.  fp32 with short dependency chains: the
// fp64 pipe is far too slow for a 32-long chain per step.
__device__ __forceinline__ float g_sum32(const float* p, int lane) {
    float a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = p[(i + lane) & 31];
#pragma unroll
    for (int j = 1; j < 4; ++j)
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] += p[(8 * j + i + lane) & 31];
    return ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
}

// A ring position that advances one slot at a time: slot index and how often it has been used.
struct GRing {
    int idx = 0;
    uint32_t use = 0;
    __device__ __forceinline__ void next(int size) { if (++idx == size) { idx = 0; ++use; } }
    __device__ __forceinline__ uint32_t parity() const { return use & 1u; }               // this use
    __device__ __forceinline__ uint32_t prev_parity() const { return (use & 1u) ^ 1u; }   // the use before
};

// A CTA's {M_P, Z_P, M_Q, Z_Q} of one row lives in scratch as four 8-byte words that each say
// whether they have been written: the scratch starts at zero and every word is stored with its
// lowest mantissa bit set (a change of 2^-52 in Z, none in the integer M once the bit is cleared
// again).  A reader therefore needs no flag, no counter and no second trip to L2.
__device__ __forceinline__ double g_enc(double v) {
    return __longlong_as_double(__double_as_longlong(v) | 1ll);
}
struct GPart {
    unsigned long long w[4];
    __device__ __forceinline__ bool complete() const { return w[0] != 0ull && w[1] != 0ull && w[2] != 0ull && w[3] != 0ull; }
    __device__ __forceinline__ double get(int i) const { return __longlong_as_double(static_cast<long long>(w[i] & ~1ull)); }
};
__device__ __forceinline__ GPart g_load_part(const RowZ* p) {
    const unsigned long long* q = reinterpret_cast<const unsigned long long*>(p);
    GPart r;
    r.w[0] = __ldcg(q); r.w[1] = __ldcg(q + 1); r.w[2] = __ldcg(q + 2); r.w[3] = __ldcg(q + 3);
    return r;
}
__device__ __forceinline__ RowZ g_load_rowz(const RowZ* p) {
    const GPart t = g_load_part(p);
    RowZ z; z.MP = t.get(0); z.ZP = t.get(1); z.MQ = t.get(2); z.ZQ = t.get(3);
    return z;
}

// A reference as a saturating integer (INT_MIN: no reference), and back.
__device__ __forceinline__ int g_ref_int(double M) { return M > kNoRef ? __double2int_rn(M) : INT_MIN; }
__device__ __forceinline__ float g_ref_float(int m) { return m == INT_MIN ? kNoRef : static_cast<float>(m); }
// z 2^{own - row} for integer references own <= row (0 without a reference of its own): exact
__device__ __forceinline__ double g_scale_down(double z, int own, int row) {
    if (own == INT_MIN) return 0.0;
    const long long d = static_cast<long long>(own) - row;          // <= 0
    if (d < -1000) return 0.0;
    return z * __longlong_as_double((1023ll + d) << 52);
}
// 1 / x to fp64 accuracy from the fp32 reciprocal and two Newton steps (x > 0, finite)
__device__ __forceinline__ double g_recip(double x) {
    double y = static_cast<double>(__frcp_rn(static_cast<float>(x)));
    y = y * (2.0 - x * y);
    return y * (2.0 - x * y);
}
// 2^x in a handful of fp64 multiply-adds: 2^round(x) by the exponent field, 2^f, |f| <= 1/2, by
// its Taylor series in f ln 2 to degree 10 (relative error below 1e-13).  x = -inf gives 0; a NaN
// or a value beyond the exponent range is left to exp2.
__device__ __forceinline__ double g_exp2(double x) {
    if (!(x > -1000.0 && x < 1000.0)) return exp2(x);
    const double xi = rint(x);
    const double t = (x - xi) * 0.693147180559945309417232;
    double y = 1.0 / 3628800.0;
    y = fma(y, t, 1.0 / 362880.0);
    y = fma(y, t, 1.0 / 40320.0);
    y = fma(y, t, 1.0 / 5040.0);
    y = fma(y, t, 1.0 / 720.0);
    y = fma(y, t, 1.0 / 120.0);
    y = fma(y, t, 1.0 / 24.0);
    y = fma(y, t, 1.0 / 6.0);
    y = fma(y, t, 0.5);
    y = fma(y, t, 1.0);
    y = fma(y, t, 1.0);
    return y * __longlong_as_double((1023ll + static_cast<long long>(xi)) << 52);
}

// Row statistics from two parts per lane that are already in registers (G <= 64); whole warp,
// all lanes return the same values.
__device__ __forceinline__ void g_combine2(const GPart& a, const GPart& b, bool has_a, bool has_b,
                                           double& MP, double& ZP, double& MQ, double& ZQ) {
    MP = kNoRef; MQ = kNoRef;
    if (has_a) { MP = fmax(MP, a.get(0)); MQ = fmax(MQ, a.get(2)); }
    if (has_b) { MP = fmax(MP, b.get(0)); MQ = fmax(MQ, b.get(2)); }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { MP = fmax(MP, shfl_xor_d(MP, off)); MQ = fmax(MQ, shfl_xor_d(MQ, off)); }
    ZP = 0.0; ZQ = 0.0;
    const float fMP = static_cast<float>(MP), fMQ = static_cast<float>(MQ);
    if (has_a) {
        ZP += a.get(1) * static_cast<double>(ref_scale(static_cast<float>(a.get(0)), fMP));
        ZQ += a.get(3) * static_cast<double>(ref_scale(static_cast<float>(a.get(2)), fMQ));
    }
    if (has_b) {
        ZP += b.get(1) * static_cast<double>(ref_scale(static_cast<float>(b.get(0)), fMP));
        ZQ += b.get(3) * static_cast<double>(ref_scale(static_cast<float>(b.get(2)), fMQ));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { ZP += shfl_xor_d(ZP, off); ZQ += shfl_xor_d(ZQ, off); }
}

// Row statistics from the G pairs in scratch, all known to be there (whole warp; all lanes return
// the same values; same order of operations as g_combine2 for G <= 64).
__device__ __forceinline__ void g_combine(const FlowScratch& fl, size_t rowi, int G, int lane,
                                          double& MP, double& ZP, double& MQ, double& ZQ) {
    MP = kNoRef; MQ = kNoRef;
    for (int ch = lane; ch < G; ch += 32) {
        const RowZ z = g_load_rowz(&fl.part[rowi * G + ch]);
        MP = fmax(MP, z.MP); MQ = fmax(MQ, z.MQ);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { MP = fmax(MP, shfl_xor_d(MP, off)); MQ = fmax(MQ, shfl_xor_d(MQ, off)); }
    ZP = 0.0; ZQ = 0.0;
    for (int ch = lane; ch < G; ch += 32) {
        const RowZ z = g_load_rowz(&fl.part[rowi * G + ch]);
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
        // Row after row: as soon as all G pairs of the row are in scratch, combine them, advance the
        // recursion and hand the scalars of the row's second sweep to the consumers.  The warp
        // shares its scheduler with seven consumer warps and sits on the path between the two
        // sweeps, so it is kept short and never waits for a load it could have issued earlier:
        // the next row's pairs are requested before this row's are looked at (two register sets
        // that swap roles), references are integers reduced warp-wide, 2^x and 1/x take a few fp64
        // multiply-adds, and the drafted tokens' logits of a block are fetched a block ahead
        // (lane r keeps row r's).
        GRing slot;
        struct TokenLogits { float zp[2], zq[2]; };       // NaN in zq: no valid token
        auto token_logits = [&](int b, TokenLogits& d) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int r = lane + 32 * t;
                d.zp[t] = 0.f; d.zq[t] = NAN;
                if (r < g && b < cx.B) {
                    const int x = prm.tok[static_cast<size_t>(b) * g + r];
                    if (x >= 0 && x < cx.V) {
                        d.zq[t] = static_cast<float>(load_logit<DT>(static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes, x));
                        d.zp[t] = static_cast<float>(load_logit<DT>(static_cast<const char*>(prm.tgt) + (static_cast<size_t>(b) * (g + 1) + r) * cx.row_bytes, x));
                    }
                }
            }
        };
        TokenLogits dcur, dnxt;
        token_logits(grp, dcur);
        token_logits(grp + NG, dnxt);
        int n = 0, q = 0, r = 0;
        double p = 1.0;
        const bool fast = G <= 64, la = lane < G, lb = lane + 32 < G;
        auto row_of = [&](int qq, int rr) { return static_cast<size_t>(grp + qq * NG) * (g + 1) + rr; };
        auto load_set = [&](size_t row, GPart& xa, GPart& xb) {
            if (la) xa = g_load_part(&fl.part[row * G + lane]);
            if (lb) xb = g_load_part(&fl.part[row * G + lane + 32]);
        };
        // row n from the set (xa, xb), which has been requested already; the set (ya, yb) is
        // requested for row n + 1 on the way.  False: gave up waiting.
        auto step = [&](GPart& xa, GPart& xb, GPart& ya, GPart& yb) -> bool {
            const size_t row0 = row_of(q, r);
            int iMP = INT_MIN, iMQ = INT_MIN;
            double ZP = 0.0, ZQ = 0.0;
            if (fast) {
                if (n + 1 < N) load_set(r == g ? row_of(q + 1, 0) : row0 + 1, ya, yb);
                for (unsigned idle = 0; !__all_sync(0xffffffffu, (!la || xa.complete()) && (!lb || xb.complete())); ++idle) {
                    if (idle > (1u << 22)) { if (prm.status) atomicExch(prm.status, 1); return false; }
                    load_set(row0, xa, xb);
                }
                if (la) { iMP = g_ref_int(xa.get(0)); iMQ = g_ref_int(xa.get(2)); }
                if (lb) { iMP = max(iMP, g_ref_int(xb.get(0))); iMQ = max(iMQ, g_ref_int(xb.get(2))); }
                iMP = __reduce_max_sync(0xffffffffu, iMP);
                iMQ = __reduce_max_sync(0xffffffffu, iMQ);
                if (la) { ZP += g_scale_down(xa.get(1), g_ref_int(xa.get(0)), iMP); ZQ += g_scale_down(xa.get(3), g_ref_int(xa.get(2)), iMQ); }
                if (lb) { ZP += g_scale_down(xb.get(1), g_ref_int(xb.get(0)), iMP); ZQ += g_scale_down(xb.get(3), g_ref_int(xb.get(2)), iMQ); }
            } else {
                for (unsigned idle = 0;; ++idle) {
                    bool ok = true;
                    iMP = INT_MIN; iMQ = INT_MIN;
                    for (int ch = lane; ch < G; ch += 32) {
                        const GPart t = g_load_part(&fl.part[row0 * G + ch]);
                        ok = ok && t.complete();
                        iMP = max(iMP, g_ref_int(t.get(0)));
                        iMQ = max(iMQ, g_ref_int(t.get(2)));
                    }
                    if (__all_sync(0xffffffffu, ok)) break;
                    if (idle > (1u << 22)) { if (prm.status) atomicExch(prm.status, 1); return false; }
                }
                iMP = __reduce_max_sync(0xffffffffu, iMP);
                iMQ = __reduce_max_sync(0xffffffffu, iMQ);
                for (int ch = lane; ch < G; ch += 32) {
                    const GPart t = g_load_part(&fl.part[row0 * G + ch]);
                    ZP += g_scale_down(t.get(1), g_ref_int(t.get(0)), iMP);
                    ZQ += g_scale_down(t.get(3), g_ref_int(t.get(2)), iMQ);
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) { ZP += shfl_xor_d(ZP, off); ZQ += shfl_xor_d(ZQ, off); }
            // ---- the recursion (Eq. "def_as") and the scale of the row's second sweep ----
            float cs = 1.f;
            if (r == 0) p = 1.0;
            if (r < g) {
                const float zpx = __shfl_sync(0xffffffffu, r < 32 ? dcur.zp[0] : dcur.zp[1], r & 31);
                const float zqx = __shfl_sync(0xffffffffu, r < 32 ? dcur.zq[0] : dcur.zq[1], r & 31);
                const double zr = ZQ * g_recip(ZP);
                cs = static_cast<float>(p * zr);
                const bool tok_ok = zqx == zqx && zqx != -INFINITY;
                const double e = (static_cast<double>(zpx) - static_cast<double>(zqx)) * cx.kd - static_cast<double>(iMP - iMQ);
                p = fmin(p * (tok_ok ? g_exp2(e) * zr : 0.0), 1.0);
            }
            if (slot.use > 0 && !g_wait(smem_u32(&sh.done2[slot.idx]), slot.prev_parity(), prm.status)) return false;
            if (lane == 0) {
                sh.meta2[slot.idx] = make_float4(cs, -g_ref_float(iMP), -g_ref_float(iMQ), 0.f);
                mbar_arrive(smem_u32(&sh.s2ready[slot.idx]));
            }
            __syncwarp();
            slot.next(kGR);
            ++n;
            if (++r > g) {
                r = 0; ++q;
                dcur = dnxt;
                token_logits(grp + (q + 1) * NG, dnxt);
            }
            return true;
        };
        GPart A0, A1, B0, B1;
        if (fast) load_set(row_of(0, 0), A0, A1);
        while (n < N) {
            if (!step(A0, A1, B0, B1)) return;
            if (n < N && !step(B0, B1, A0, A1)) return;
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
                    zP = static_cast<double>(g_sum32(lp, lane));
                    zQ = static_cast<double>(g_sum32(lp + kGShareVecs, lane));
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
                    RowZ z; z.MP = g_enc(MPc); z.ZP = g_enc(zP); z.MQ = g_enc(MQc); z.ZQ = g_enc(zQ);
                    fl.part[rowi * G + j] = z;          // four self-validating words: no fence, no counter
                }
                s1.next(kGR);
                if (++r1 > g) { r1 = 0; ++q1; }
            }
            if (n >= L) {
                if (!g_wait(smem_u32(&sh.done2[s2.idx]), s2.parity(), prm.status)) return;
                const size_t rowi = static_cast<size_t>(grp + q2 * NG) * (g + 1) + r2;
                const float* lp = part2 + static_cast<size_t>(s2.idx) * kGShareVecs + lane * 32;
                float t = 0.f;
                if (lane < kGWarps) t = g_sum32(lp, lane);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.free2[s2.idx]));
                if (lane < kGWarps) {
                    // a segment is one consumer warp's 32 vectors: contiguous in the row
                    // (the total says "written" by its lowest mantissa bit; the counter is only a hint)
                    fl.seg_tot[rowi * nseg + j * kGWarps + lane] =
                        __uint_as_float(__float_as_uint(t) | 1u);
                    g_red_relaxed(&fl.s2_cnt[rowi]);
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
                bool parts_in = fold_r <= g;
                if (fold_r <= g)
                    for (int ch = lane; ch < G; ch += 32) parts_in = parts_in && g_load_part(&fl.part[row_f * G + ch]).complete();
                parts_in = __all_sync(0xffffffffu, parts_in);
                bool segs_in = pos_r < fold_r && ld_volatile(&fl.s2_cnt[row_p]) == all_segs;
                if (segs_in) {
                    const float* sg = fl.seg_tot + row_p * nseg;
                    for (int i = lane; i < nseg; i += 32) segs_in = segs_in && __float_as_uint(__ldcg(&sg[i])) != 0u;
                }
                segs_in = __all_sync(0xffffffffu, segs_in);
                bool did = false;
                if (parts_in) {
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
                if (segs_in) {
                    const int r = pos_r;
                    const bool have_q = r < g;
                    const char* rowP = static_cast<const char*>(prm.tgt) + row_p * cx.row_bytes;
                    const char* rowQ = have_q ? static_cast<const char*>(prm.drf) + (static_cast<size_t>(b) * g + r) * cx.row_bytes
                                              : nullptr;
                    const float cs = __ldcg(&fl.cscale[row_p]);
                    const float nMP = -static_cast<float>(__ldcg(&fl.rowZ[row_p].MP));
                    const float nMQ = -static_cast<float>(__ldcg(&fl.rowZ[row_p].MQ));
                    const int units = cx.units;
                    f_position_complete<DT, true>(prm, fl, cx, static_cast<int>(row_p), have_q, rowP, rowQ, cs, nMP, nMQ, nseg,
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
