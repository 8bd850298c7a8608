// The drafting step of Algorithm 3 for rows of logits: one token per row drawn from
// softmax(logits / T) by inverse CDF in vocabulary-index order with a supplied uniform, and the
// row's log-normaliser (what the verification needs of a draft row besides the logits).
//
// Persistent CTAs take rows round-robin.  Each of 16 warps streams its contiguous sixteenth of the
// row once, in eight sub-segments, and leaves each sub-segment's {integer reference, sum 2^{z k - M}}
// in shared memory; a seventeenth warp, a row behind, combines the 128 pairs (fp64 for the
// normaliser and for the sampler's prefix sums), finds the sub-segment that holds u * Z and rescans
// that one - a few KB still in L2 - in index order for the token.  Each logit is read from HBM once.
#include <cmath>
#include <cstdint>

#include "bv_flow_common.cuh"

#include "../../include/bv.h"

namespace bv {

constexpr int kSThreads = 512;                    // streaming threads; one more warp draws the samples
constexpr int kSWarps = kSThreads / 32;
constexpr int kSAllThreads = kSThreads + 32;
constexpr int kSSub = 8;                          // sub-segments per warp
constexpr int kSSegs = kSWarps * kSSub;           // 128: four per lane of warp 0
constexpr int kSInFlight = 8;                     // 16-byte loads a thread has in flight

// named barriers of a CTA (hardware barriers 1 .. 15; 0 is __syncthreads): all lanes of a warp take part,
// `threads` is the number of threads that arrive or wait at the barrier per use
constexpr int kBarFull = 1, kBarEmpty = 3;        // ids kBarFull + buffer, kBarEmpty + buffer
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int threads) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// vectors [a0, a1) of sub-segment `sub` of warp `warp` in a row of `units` vectors
__device__ __forceinline__ void s_range(int units, int warp, int sub, int& a0, int& a1) {
    const int u0 = static_cast<int>(static_cast<long long>(units) * warp / kSWarps);
    const int u1 = static_cast<int>(static_cast<long long>(units) * (warp + 1) / kSWarps);
    a0 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * sub / kSSub);
    a1 = u0 + static_cast<int>(static_cast<long long>(u1 - u0) * (sub + 1) / kSSub);
}

// One streaming warp's pass over its sixteenth of a row: the {reference, sum} pair of each of its
// sub-segments goes to sM / sS.
template <int DT>
__device__ __forceinline__ void s_sweep_row(const char* row, int units, float kf, int warp, int lane, float* sM, float* sS) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    // ---- one pass over the warp's part of the row ----
    // (the warp's reference carries over from one sub-segment to the next: a sub-segment's pair is
    // its sum against the reference as it stood at its end, and only the first one has to find one)
    float M = kNoRef;
    for (int sub = 0; sub < kSSub; ++sub) {
        int a0, a1;
        s_range(units, warp, sub, a0, a1);
        float s = 0.f;
        const uint4 ninf = make_uint4(R::kNegInf, R::kNegInf, R::kNegInf, R::kNegInf);
        for (int base = a0; base < a1; base += 32 * kSInFlight) {
            uint4 raw[kSInFlight];                // all loads of the round are issued before any is used
#pragma unroll
            for (int j = 0; j < kSInFlight; ++j) {
                const int i = base + 32 * j + lane;
                raw[j] = i < a1 ? ld_stream_v4(row + static_cast<size_t>(i) * 16) : ninf;
            }
#pragma unroll
            for (int j = 0; j < kSInFlight; ++j) {
                if (base + 32 * j < a1) {
                    float v[EPV];
                    R::unpack(raw[j], v);
                    f_accumulate<EPV>(v, kf, M, s);
                }
            }
        }
        s = warp_sum(s);
        if (lane == 0) { sM[warp * kSSub + sub] = M; sS[warp * kSSub + sub] = s; }
    }
}

// The sampling warp's part: the row's normaliser from the 128 pairs and the token that the uniform u
// selects (inverse CDF in index order; -1 and a NaN normaliser for a row with a NaN or +inf logit or
// without a finite one).  release_pairs >= 0: a named barrier at which the warp arrives once it has
// read the pairs.
template <int DT>
__device__ __forceinline__ int s_draw_row(const char* row, int units, float kf, const float* sM, const float* sS, float u,
                                          int lane, int release_pairs, float* lse_out) {
    // ---- normaliser and the sampled sub-segment (fp64 prefix sums, index order) ----
    float m[4], w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { m[j] = sM[4 * lane + j]; w[j] = sS[4 * lane + j]; }
    const float Mrow = warp_max(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])));
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] *= ref_scale(m[j], Mrow);
    double Z = (static_cast<double>(w[0]) + static_cast<double>(w[1])) +
               (static_cast<double>(w[2]) + static_cast<double>(w[3]));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) Z += shfl_xor_d(Z, off);
    // (the sums over sub-segments that locate the sample are formed in double: a token's cell can
    // be far narrower than fp32 resolves next to the mass before it)
    const double l1 = w[0], l2 = l1 + w[1], l3 = l2 + w[2], l4 = l3 + w[3];
    double inc = l4;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double o = shfl_up_d(inc, off);
        if (lane >= off) inc += o;
    }
    const double total = shfl_d(inc, 31);
    // a row with a NaN or +inf logit has a NaN / infinite sum or reference; one without a finite logit has none
    const bool ok = Mrow > kNoRef && Mrow < INFINITY && Z > 0.0 && Z < INFINITY && total > 0.0 && total < static_cast<double>(INFINITY);
    if (release_pairs >= 0) named_bar_arrive(release_pairs, kSAllThreads);   // (the pairs are in registers: their buffer may be written again)
    int found = -1;
    if (ok) {
        const double t = static_cast<double>(u) * total;
        double exc = shfl_up_d(inc, 1);
        if (lane == 0) exc = 0.0;
        const double p0 = exc, p1 = exc + l1, p2 = exc + l2, p3 = exc + l3, p4 = exc + l4;
        // first non-empty sub-segment whose inclusive prefix exceeds t, else the last non-empty one
        const bool h1 = p1 > t && w[0] > 0.f, h2 = p2 > t && w[1] > 0.f;
        const bool h3 = p3 > t && w[2] > 0.f, h4 = p4 > t && w[3] > 0.f;
        const unsigned hit = __ballot_sync(0xffffffffu, h1 || h2 || h3 || h4);
        const unsigned nz = __ballot_sync(0xffffffffu, l4 > 0.0);
        int e = 3; double bef = p3; int src;
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
        const double before = shfl_d(bef, src);
        int a0, a1;
        s_range(units, sel / kSSub, sel % kSSub, a0, a1);
        found = f_rescan<DT>(row, nullptr, a0, a1, lane, kf, 1.f, -Mrow, 0.f, t - before);
    }
    *lse_out = found >= 0 ? static_cast<float>((static_cast<double>(Mrow) + log2(Z)) * 0.693147180559945309417232)
                          : __int_as_float(0x7fc00000);
    return found;
}

template <int DT>
__global__ void __launch_bounds__(kSAllThreads, 2)
sample_rows_kernel(const char* logits, const float* uni, int rows, int V, float kf, int32_t* tokens, float* lse) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int units = V / EPV;
    const size_t row_bytes = static_cast<size_t>(V) * ESZ;
    __shared__ float sM2[2][kSSegs], sS2[2][kSSegs];

    // The streaming warps sweep the CTA's rows one after the other and leave each row's pairs in one of
    // two buffers; the sampling warp follows, a row behind or so, and draws each row's token from them.
    // Two named barriers per buffer order the two sides, producer and consumer: "full" (the 16 streaming
    // warps arrive when the row's pairs are written, the sampling warp waits) and "empty" (the sampling
    // warp arrives when it has read them, the streaming warps wait before they write that buffer again,
    // two rows later).  The streaming warps never wait for one another: there is no barrier across a row.
    // Every wait ends: the row count is the same for all warps of the CTA, each row has exactly one
    // arrival and one wait per side, and the streaming side waits for row `it - 2` only from row 2 on.
    const int nmine = rows > static_cast<int>(blockIdx.x) ? (rows - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
    if (warp < kSWarps) {
        for (int it = 0; it < nmine; ++it) {
            if (it >= 2) named_bar_sync(kBarEmpty + (it & 1), kSAllThreads);
            const int r = blockIdx.x + it * gridDim.x;
            s_sweep_row<DT>(logits + static_cast<size_t>(r) * row_bytes, units, kf, warp, lane, sM2[it & 1], sS2[it & 1]);
            __threadfence_block();
            named_bar_arrive(kBarFull + (it & 1), kSAllThreads);
        }
    } else {
        for (int it = 0; it < nmine; ++it) {
            named_bar_sync(kBarFull + (it & 1), kSAllThreads);
            const int r = blockIdx.x + it * gridDim.x;
            float l;
            // (row it + 2 waits for the release of this buffer; the last two rows have nobody waiting)
            const int found = s_draw_row<DT>(logits + static_cast<size_t>(r) * row_bytes, units, kf, sM2[it & 1], sS2[it & 1], uni[r],
                                             lane, it + 2 < nmine ? kBarEmpty + (it & 1) : -1, &l);
            if (lane == 0) {
                tokens[r] = found;
                if (lse) lse[r] = l;
            }
        }
    }
}

// The drafting step of Algorithm 3 as a whole for a model whose next-token logits depend on the last
// token only (a table [V, V], row t = logits after token t): X_1 .. X_gamma one after the other, each
// from the row of the token before it.  One CTA per sequence; a step is the sweep of one row by the
// 16 streaming warps, a barrier, the draw by the sampling warp, a barrier.  A token that is not in
// [0, V) (a first token out of range, or a step whose row could not be sampled) ends the sequence's
// chain: the remaining tokens are -1 and their normalisers NaN.
template <int DT>
__global__ void __launch_bounds__(kSAllThreads, 2)
draft_chain_kernel(const char* table, const int32_t* first, const float* uni, int B, int gamma, int V, float kf,
                   int32_t* tokens, float* lse) {
    using R = Raw<DT>;
    constexpr int EPV = R::EPV;
    constexpr size_t ESZ = (DT == kF32) ? 4 : 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int units = V / EPV;
    const size_t row_bytes = static_cast<size_t>(V) * ESZ;
    __shared__ float sM[kSSegs], sS[kSSegs];
    __shared__ int s_next;
    for (int b = blockIdx.x; b < B; b += gridDim.x) {
        int last = first[b];
        for (int i = 0; i < gamma; ++i) {
            const bool ok = last >= 0 && last < V;
            const char* row = table + static_cast<size_t>(ok ? last : 0) * row_bytes;
            if (warp < kSWarps && ok) s_sweep_row<DT>(row, units, kf, warp, lane, sM, sS);
            __syncthreads();
            if (warp == kSWarps) {
                float l = __int_as_float(0x7fc00000);
                int found = -1;
                if (ok) found = s_draw_row<DT>(row, units, kf, sM, sS, uni[static_cast<size_t>(i) * B + b], lane, -1, &l);
                if (lane == 0) {
                    tokens[static_cast<size_t>(b) * gamma + i] = found;
                    if (lse) lse[static_cast<size_t>(b) * gamma + i] = l;
                    s_next = found;
                }
            }
            __syncthreads();
            last = s_next;
            __syncthreads();      // (s_next is written again in the next step)
        }
    }
}

}  // namespace bv

namespace {
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) % 16) == 0; }
}  // namespace

extern "C" int bv_sample_draft(const void* logits, const float* uniforms, int rows, int V, int dtype,
                               float temperature, int32_t* out_tokens, float* out_lse, void* stream) {
    if (!logits || !uniforms || !out_tokens) return BV_ERR_INVALID_ARG;
    if (rows < 0 || V < 1) return BV_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !std::isfinite(temperature)) return BV_ERR_INVALID_ARG;
    if (dtype != BV_DTYPE_F32 && dtype != BV_DTYPE_BF16) return BV_ERR_INVALID_ARG;
    const size_t row_bytes = static_cast<size_t>(V) * (dtype == BV_DTYPE_F32 ? 4 : 2);
    if (row_bytes % 16 != 0 || !aligned16(logits)) return BV_ERR_UNSUPPORTED;
    bv::note_launches(0);
    if (rows == 0) return BV_OK;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return bv::note_cuda_error(e);
    const int grid = rows < 2 * sms ? rows : 2 * sms;
    const float kf = static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == BV_DTYPE_F32)
        bv::sample_rows_kernel<bv::kF32><<<grid, bv::kSAllThreads, 0, st>>>(static_cast<const char*>(logits), uniforms, rows, V, kf, out_tokens, out_lse);
    else
        bv::sample_rows_kernel<bv::kBF16><<<grid, bv::kSAllThreads, 0, st>>>(static_cast<const char*>(logits), uniforms, rows, V, kf, out_tokens, out_lse);
    e = cudaGetLastError();
    if (e != cudaSuccess) return bv::note_cuda_error(e);
    bv::note_launches(1);
    return BV_OK;
}

extern "C" int bv_draft_chain(const void* draft_table, const int32_t* first_tokens, const float* uniforms, int B, int gamma,
                              int V, int dtype, float temperature, int32_t* out_tokens, float* out_lse, void* stream) {
    if (!draft_table || !first_tokens || !uniforms || !out_tokens) return BV_ERR_INVALID_ARG;
    if (B < 0 || gamma < 1 || V < 1) return BV_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !std::isfinite(temperature)) return BV_ERR_INVALID_ARG;
    if (dtype != BV_DTYPE_F32 && dtype != BV_DTYPE_BF16) return BV_ERR_INVALID_ARG;
    const size_t row_bytes = static_cast<size_t>(V) * (dtype == BV_DTYPE_F32 ? 4 : 2);
    if (row_bytes % 16 != 0 || !aligned16(draft_table)) return BV_ERR_UNSUPPORTED;
    bv::note_launches(0);
    if (B == 0) return BV_OK;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return bv::note_cuda_error(e);
    const int grid = B < 2 * sms ? B : 2 * sms;
    const float kf = static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == BV_DTYPE_F32)
        bv::draft_chain_kernel<bv::kF32><<<grid, bv::kSAllThreads, 0, st>>>(static_cast<const char*>(draft_table), first_tokens, uniforms, B, gamma, V, kf, out_tokens, out_lse);
    else
        bv::draft_chain_kernel<bv::kBF16><<<grid, bv::kSAllThreads, 0, st>>>(static_cast<const char*>(draft_table), first_tokens, uniforms, B, gamma, V, kf, out_tokens, out_lse);
    e = cudaGetLastError();
    if (e != cudaSuccess) return bv::note_cuda_error(e);
    bv::note_launches(1);
    return BV_OK;
}
