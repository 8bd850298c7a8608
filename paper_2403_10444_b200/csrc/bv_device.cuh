// Device-side building blocks shared by the verification kernels: parameter
// block, 128-bit streaming loads, bf16 widening, (max, sum-exp) reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace bv {

constexpr int kMaxGamma = 64;     // longest drafted block the kernels accept
constexpr int kMaxCluster = 8;    // portable thread-block cluster limit

enum : int { kF32 = 0, kBF16 = 1 };
enum : int { kTokenVerify = 0, kBlockVerify = 1 };

struct Params {
    const void* tgt;          // [B, gamma+1, V]
    const void* drf;          // [B, gamma,   V]
    const int32_t* tok;       // [B, gamma]
    const float* uni;         // [B, gamma+2]
    const float* lse_d;       // [B, gamma] supplied draft log-normalisers ln sum exp(z/T), or null: computed
    int B, gamma, V;
    float kf;                 // log2(e) / T, rounded to float (per-element scale)
    double kd;                // log2(e) / T in double (scalar recursion)
    int32_t* out_tokens;      // [B, gamma+1]
    int32_t* out_len;         // [B]
    float* out_p;             // optional diagnostics, may be null
    float* out_S;
    float* out_h;
    float* out_lse_t;
    float* out_lse_d;
    unsigned int* ticket;     // [2]: next sequence index, clusters that have finished
    int* status;              // set to 1 if a bounded device-side wait gave up
    int nclusters;            // clusters in the grid
    int greedy;               // flow kernel: Greedy Block Verification (Algorithm 4) instead of Algorithm 2
    int algo;                 // flow kernel: kBlockVerify (Algorithms 2, 4) or kTokenVerify (Algorithm 1)
    unsigned wait_limit;      // flow kernel: polls after which a bounded wait gives up (0: the built-in limits)
    int never_signal;         // flow kernel, test switch: workers never report an item as swept, so the waits run out
    int probs;                // flow kernel: tgt / drf hold probabilities, used as stored, instead of logits
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// One "unit" of a logit row: EPV consecutive elements widened to float.
// VEC = true reads 16 bytes at once and needs 16-byte aligned rows.
template <int DT, bool VEC> struct Unit;

template <> struct Unit<kF32, true> {
    static constexpr int EPV = 4;
    static __device__ __forceinline__ void load(const void* row, int i, float (&v)[4]) {
        uint4 r = ld_stream_v4(reinterpret_cast<const uint4*>(row) + i);
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y);
        v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
};
template <> struct Unit<kBF16, true> {
    static constexpr int EPV = 8;
    static __device__ __forceinline__ void load(const void* row, int i, float (&v)[8]) {
        uint4 r = ld_stream_v4(reinterpret_cast<const uint4*>(row) + i);
        v[0] = __uint_as_float(r.x << 16); v[1] = __uint_as_float(r.x & 0xffff0000u);
        v[2] = __uint_as_float(r.y << 16); v[3] = __uint_as_float(r.y & 0xffff0000u);
        v[4] = __uint_as_float(r.z << 16); v[5] = __uint_as_float(r.z & 0xffff0000u);
        v[6] = __uint_as_float(r.w << 16); v[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};
template <> struct Unit<kF32, false> {
    static constexpr int EPV = 1;
    static __device__ __forceinline__ void load(const void* row, int i, float (&v)[1]) {
        v[0] = __ldg(reinterpret_cast<const float*>(row) + i);
    }
};
template <> struct Unit<kBF16, false> {
    static constexpr int EPV = 1;
    static __device__ __forceinline__ void load(const void* row, int i, float (&v)[1]) {
        unsigned short h = __ldg(reinterpret_cast<const unsigned short*>(row) + i);
        v[0] = __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
};

template <int DT> __device__ __forceinline__ double load_logit(const void* row, int x) {
    float v[1];
    Unit<DT, false>::load(row, x, v);
    return static_cast<double>(v[0]);
}

// 2^d for an integer-valued d <= 0 (or -inf): an exact power of two, 0 below 2^-126.
__device__ __forceinline__ float pow2_nonpos(float d) {
    int n = (d < -126.f) ? -127 : static_cast<int>(d);
    return __int_as_float((n + 127) << 23);
}

// Running sum of 2^{z*k - M} over the elements a thread has seen, where the
// reference M is an INTEGER (the rounded scaled maximum so far).  An integer
// reference is exact in fp32, so z*k - M costs one fused multiply-add with a
// single rounding, and changing the reference rescales by an exact power of two.
// A NaN element makes s NaN; M = +inf is caught when the row is combined.
struct MaxSum {
    float M, s;
    __device__ __forceinline__ void init() { M = -INFINITY; s = 0.f; }
    template <int N> __device__ __forceinline__ void add(const float (&v)[N], float kf) {
        float vm = v[0];
#pragma unroll
        for (int e = 1; e < N; ++e) vm = fmaxf(vm, v[e]);
        const float y = rintf(vm * kf);
        if (y > M) { s = (s != s) ? s : s * pow2_nonpos(M - y); M = y; }
        if (M > -INFINITY) {
            const float nM = -M;
#pragma unroll
            for (int e = 0; e < N; ++e) s += ex2(fmaf(v[e], kf, nM));
        } else {
#pragma unroll
            for (int e = 0; e < N; ++e) if (v[e] != v[e]) s = v[e];
        }
    }
};

// Combine the lanes of a warp: afterwards every lane holds the warp's (M, s).
__device__ __forceinline__ void warp_combine(float& M, float& s) {
    float Mw = M;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) Mw = fmaxf(Mw, __shfl_xor_sync(0xffffffffu, Mw, off));
    s = (s != s) ? s : s * pow2_nonpos(M - Mw);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    M = Mw;
}

__device__ __forceinline__ double shfl_xor_d(double v, int off) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(0xffffffffu, lo, off);
    hi = __shfl_xor_sync(0xffffffffu, hi, off);
    return __hiloint2double(hi, lo);
}
__device__ __forceinline__ double warp_sum_d(double x);
__device__ __forceinline__ double shfl_up_d(double v, int off) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_up_sync(0xffffffffu, lo, off);
    hi = __shfl_up_sync(0xffffffffu, hi, off);
    return __hiloint2double(hi, lo);
}
__device__ __forceinline__ double shfl_d(double v, int src) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src);
    hi = __shfl_sync(0xffffffffu, hi, src);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double warp_sum_d(double x) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += shfl_xor_d(x, off);
    return x;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// address of the same shared-memory location in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, int rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Wait for the phase with the given parity.  Each attempt lets the hardware suspend the
// thread for up to about 2 us; the number of attempts is bounded (a few seconds in all),
// after which the wait gives up, records the fact in *status and returns false, so that a
// protocol error cannot hang the GPU.  A caller that gets false must not touch what the
// barrier guards: it leaves its loop and returns.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status, uint32_t limit = 1u << 20) {
    for (uint32_t spins = 0; !mbar_try_wait(bar, parity, 2000u); ++spins) {
        if (spins > limit) {
            if (status) atomicExch(status, 1);
            return false;
        }
    }
    return true;
}
// The same wait without a suspend-time hint: the thread polls and resumes as soon as the phase
// completes (a hinted wait was seen to resume late).  Bounded like mbar_wait.
__device__ __forceinline__ bool mbar_try_wait_now(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_now(uint32_t bar, uint32_t parity, int* status, uint32_t limit = 1u << 24) {
    for (uint32_t spins = 0; !mbar_try_wait_now(bar, parity); ++spins) {
        if (spins > limit) {
            if (status) atomicExch(status, 1);
            return false;
        }
    }
    return true;
}
// The wait of a warp that has nothing else to do and whose wake-up may be a little late: between
// polls it sleeps, so that it takes no issue slots from the warps that stream.  Bounded like the others.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, int* status, uint32_t ns, uint32_t limit = 1u << 22) {
    for (uint32_t spins = 0; !mbar_try_wait_now(bar, parity); ++spins) {
        if (spins > limit) {
            if (status) atomicExch(status, 1);
            return false;
        }
        __nanosleep(ns);
    }
    return true;
}
// 16 or 4 bytes into another CTA's shared memory; the bytes are counted by that CTA's barrier
__device__ __forceinline__ void send_v4(uint32_t raddr, uint32_t rbar, float a, float b, float c, float d) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(raddr), "r"(__float_as_uint(a)), "r"(__float_as_uint(b)), "r"(__float_as_uint(c)),
                   "r"(__float_as_uint(d)), "r"(rbar) : "memory");
}
__device__ __forceinline__ void send_b32(uint32_t raddr, uint32_t rbar, uint32_t v) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(raddr), "r"(v), "r"(rbar) : "memory");
}

template <int DT> struct Raw;
template <> struct Raw<kBF16> {
    static constexpr int EPV = 8;
    static constexpr uint32_t kNegInf = 0xff80ff80u;
    static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[8]) {
        // (the low half by a byte permute: like the mask of the high half it runs on the integer
        // pipe, where a shift would share the pipe of the multiply-adds)
        v[0] = __uint_as_float(__byte_perm(r.x, 0, 0x1044)); v[1] = __uint_as_float(r.x & 0xffff0000u);
        v[2] = __uint_as_float(__byte_perm(r.y, 0, 0x1044)); v[3] = __uint_as_float(r.y & 0xffff0000u);
        v[4] = __uint_as_float(__byte_perm(r.z, 0, 0x1044)); v[5] = __uint_as_float(r.z & 0xffff0000u);
        v[6] = __uint_as_float(__byte_perm(r.w, 0, 0x1044)); v[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};
template <> struct Raw<kF32> {
    static constexpr int EPV = 4;
    static constexpr uint32_t kNegInf = 0xff800000u;
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
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}


__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// One ring item: a 16-byte asynchronous copy when `pred`, else the slot is filled with
// `fill` (the bit pattern of -inf logits); either way one commit group.
__device__ __forceinline__ void ring_fetch(void* slot, const void* src, bool pred, uint32_t fill) {
    const unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(slot));
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t"
        "@p cp.async.cg.shared.global [%0], [%1], 16;\n\t"
        "@!p st.shared.v4.b32 [%0], {%3, %3, %3, %3};\n\t"
        "cp.async.commit_group;\n\t}"
        ::"r"(s), "l"(src), "r"(static_cast<int>(pred)), "r"(fill) : "memory");
}


// 16-byte asynchronous copy and 16-byte load with the shared-memory address given as a
// 32-bit shared-space address (saves the generic-to-shared conversion in inner loops)
__device__ __forceinline__ void cp_async16_s(uint32_t saddr, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(saddr), "l"(gmem) : "memory");
}
// One ring item given by shared-space address: a 16-byte asynchronous copy when `pred`,
// else the slot is filled with `fill` (the bit pattern of -inf logits).  No commit.
__device__ __forceinline__ void ring_fetch_s(uint32_t saddr, const void* src, bool pred, uint32_t fill) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t"
        "@p cp.async.cg.shared.global [%0], [%1], 16;\n\t"
        "@!p st.shared.v4.b32 [%0], {%3, %3, %3, %3};\n\t}"
        ::"r"(saddr), "l"(src), "r"(static_cast<int>(pred)), "r"(fill) : "memory");
}
// L2 eviction-priority policies: rows streamed by the first sweep should outlive the traffic
// that passes before their second sweep; rows read by the second sweep are dead afterwards.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// ring item with an L2 policy (see ring_fetch_s)
__device__ __forceinline__ void ring_fetch_hint(uint32_t saddr, const void* src, bool pred, uint32_t fill, uint64_t pol) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t"
        "@p cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %4;\n\t"
        "@!p st.shared.v4.b32 [%0], {%3, %3, %3, %3};\n\t}"
        ::"r"(saddr), "l"(src), "r"(static_cast<int>(pred)), "r"(fill), "l"(pol) : "memory");
}
// 16-byte asynchronous copy with an L2 policy, shared-space destination address
__device__ __forceinline__ void cp_async16_hint(uint32_t saddr, const void* gmem, uint64_t pol) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(saddr), "l"(gmem), "l"(pol) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr) : "memory");
    return v;
}

// "No reference yet": finite, so that -inf logits still give 2^-inf = 0 and any finite
// logit overflows to +inf, which exceeds the raise bound and installs a real reference.
constexpr float kNoRef = -3.0e38f;
// A vector of 8 terms all at the reference sums to at most 8 * 2^0.5 = 11.3; a sum above
// this bound therefore means some term exceeds 2^0.5, i.e. its logit lies above the reference.
// Without a raise every term is below 12, so its exponent is below 4 and is rounded to 1.2e-7.
constexpr float kRaiseBound = 12.f;

// 2^d for d = (own reference) - (row reference) <= 0, or 0 when there is no own reference
__device__ __forceinline__ float ref_scale(float own, float row) {
    return own > kNoRef ? pow2_nonpos(own - row) : 0.f;
}

}  // namespace bv
