// C-ABI layer: argument checks, per-device workspace, launch-shape selection and
// the host-buffer entry points.  Declarations and contracts are in include/bv.h.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "../../include/bv.h"
#include "bv_launch.h"

namespace {

constexpr int kMaxDevices = 64;
constexpr int kTicketSlots = 64;  // concurrent calls on one device each need their own slot

struct DeviceState {
    bool ready = false;
    int sm_count = 0;
    int cc_major = 0;
    unsigned int* tickets = nullptr;  // [kTicketSlots][2], zero when idle
    unsigned long long calls = 0;
    int max_clusters[2][2][2][bv::kMaxCluster + 1] = {};  // [algo][dtype][vec][cluster], 0 = not asked yet
    int res_clusters[2][9][bv::kMaxCluster + 1] = {};     // resident kernel: [dtype][nk][cluster]
    int clu_clusters[2][2][bv::kMaxCluster + 1] = {};     // cluster kernel: [algo][dtype][cluster]
    // scratch of the flow kernel: a small ring, so that calls in flight on different streams
    // do not share counters (more than kFlowSlots overlapping calls on one device would)
    void* flow_ws[4] = {};
    size_t flow_bytes[4] = {};
    size_t flow_clean[4] = {};        // leading bytes of each area known to be zero between calls
    unsigned long long flow_calls = 0;
    int flow_ctas_per_sm[2] = {};
    // staging for the host-buffer entry points
    void* stage = nullptr;
    size_t stage_bytes = 0;
    cudaStream_t stream = nullptr;
};

DeviceState g_dev[kMaxDevices];
std::mutex g_mu;

thread_local int t_last_launches = 0;
thread_local int t_last_cuda_error = 0;
thread_local const float* t_given_lse_d = nullptr;   // set by bv_verify_lse around its call of run_device
thread_local int t_greedy = 0;                       // set by gbv_verify around its call of run_device

int cuda_fail(cudaError_t e) {
    t_last_cuda_error = static_cast<int>(e);
    cudaGetLastError();
    return BV_ERR_CUDA;
}

// Per-device set-up on first use: device attributes and the ticket slots.
int device_state(DeviceState** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return BV_ERR_UNSUPPORTED;
    DeviceState& d = g_dev[dev];
    if (!d.ready) {
        if ((e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return cuda_fail(e);
        if ((e = cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess)
            return cuda_fail(e);
        if (d.cc_major < 10) return BV_ERR_UNSUPPORTED;
        // ticket slots, then one status word that a kernel sets if a bounded wait gives up
        if ((e = cudaMalloc(&d.tickets, sizeof(unsigned int) * (2 * kTicketSlots + 1))) != cudaSuccess)
            return cuda_fail(e);
        if ((e = cudaMemset(d.tickets, 0, sizeof(unsigned int) * (2 * kTicketSlots + 1))) != cudaSuccess)
            return cuda_fail(e);
        d.ready = true;
    }
    *out = &d;
    return BV_OK;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_args(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
               int V, int dtype, float T, const int32_t* ot, const int32_t* ol) {
    if (!tgt || !drf || !tok || !uni || !ot || !ol) return BV_ERR_INVALID_ARG;
    if (B < 0 || gamma < 1 || V < 1) return BV_ERR_INVALID_ARG;
    if (!(T > 0.f) || !std::isfinite(T)) return BV_ERR_INVALID_ARG;
    if (dtype != BV_DTYPE_F32 && dtype != BV_DTYPE_BF16) return BV_ERR_INVALID_ARG;
    const size_t esz = dtype == BV_DTYPE_F32 ? 4 : 2;
    if (!aligned(tgt, esz) || !aligned(drf, esz) || !aligned(tok, 4) || !aligned(uni, 4) ||
        !aligned(ot, 4) || !aligned(ol, 4))
        return BV_ERR_INVALID_ARG;
    if (gamma > BV_MAX_GAMMA) return BV_ERR_UNSUPPORTED;
    return BV_OK;
}

// Cluster width for the streaming kernel: wide enough that a CTA's slice of a row
// is at most 64 KB, widened further while the batch alone cannot fill the SMs.
int pick_cluster(const DeviceState& d, int B, size_t row_bytes) {
    if (const char* env = std::getenv("BV_CLUSTER")) {
        int c = std::atoi(env);
        if (c == 1 || c == 2 || c == 4 || c == 8) return c;
    }
    int c = 1;
    while (c < bv::kMaxCluster && row_bytes / c > (64u << 10)) c *= 2;
    while (c < bv::kMaxCluster && static_cast<long long>(B) * c < d.sm_count && row_bytes / (2 * c) >= (8u << 10))
        c *= 2;
    // With several sequences per cluster to go through, narrower clusters (more sequences at a time,
    // cheaper exchanges) win: measured 0.43 against 0.57 ms at B = 256, gamma = 8, V = 152064.
    if (c == 8 && static_cast<long long>(B) * c >= 8LL * d.sm_count) c = 4;
    return c;
}

int run_device(int algo, const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
               int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
               float* out_h, float* out_lse_t, float* out_lse_d, cudaStream_t stream) {
    t_last_launches = 0;
    int rc = check_args(tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
    if (rc != BV_OK) return rc;
    if (B == 0) return BV_OK;

    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState* d = nullptr;
    if ((rc = device_state(&d)) != BV_OK) return rc;

    const size_t esz = dtype == BV_DTYPE_F32 ? 4 : 2;
    const size_t row_bytes = static_cast<size_t>(V) * esz;
    const bool vec = (row_bytes % 16 == 0) && aligned(tgt, 16) && aligned(drf, 16);

    bv::Params prm{};
    prm.tgt = tgt; prm.drf = drf; prm.tok = tok; prm.uni = uni;
    prm.lse_d = t_given_lse_d;
    prm.greedy = t_greedy;
    prm.B = B; prm.gamma = gamma; prm.V = V;
    const double kd = 1.4426950408889634073599246810019 / static_cast<double>(T);
    prm.kd = kd;
    prm.kf = static_cast<float>(kd);
    prm.out_tokens = ot; prm.out_len = ol;
    prm.out_p = out_p; prm.out_S = out_S; prm.out_h = out_h;
    prm.out_lse_t = out_lse_t; prm.out_lse_d = out_lse_d;
    prm.status = reinterpret_cast<int*>(d->tickets + 2 * kTicketSlots);

    // Block Verification on 16-byte rows: the kernel that keeps each row pair on chip,
    // when some cluster width lets a thread hold its share (at most 8 vectors per row).
    const char* force = std::getenv("BV_KERNEL");   // "flow", "cluster", "resident", "stream": experiments and tests
    const bool want = force != nullptr;
    auto forced = [&](const char* name) { return want && std::strcmp(force, name) == 0; };
    if ((prm.lse_d != nullptr || prm.greedy) && !(algo == bv::kBlockVerify && vec && (!want || forced("flow")))) return BV_ERR_UNSUPPORTED;

    // Block Verification on 16-byte rows: the flow of independent work items
    if (algo == bv::kBlockVerify && vec && (!want || forced("flow"))) {
        int& per_sm = d->flow_ctas_per_sm[dtype];
        if (per_sm == 0) {
            per_sm = bv::flow_max_ctas_per_sm(dtype);
            if (per_sm <= 0) per_sm = -1;
        }
        if (per_sm > 0) {
            const long long units = static_cast<long long>(row_bytes / 16);
            long long nctas = static_cast<long long>(d->sm_count) * per_sm;
            if (const char* env = std::getenv("BV_FLOW_CTAS")) {
                const long long v = std::atoll(env);
                if (v >= 1 && v < nctas) nctas = v;
            }
            int chunks = 0, pieces = 0;
            if (const char* env = std::getenv("BV_FLOW_CHUNKS")) {
                const int v = std::atoi(env);
                if (v >= 1 && v <= bv::kFlowMaxChunks) chunks = v;
            }
            if (const char* env = std::getenv("BV_FLOW_PIECES")) {
                const int v = std::atoi(env);
                if (v >= 1 && v <= 8) pieces = v;
            }
            // (with supplied draft normalisers a first-sweep item streams one row, not two)
            const bv::FlowPlan plan = bv::flow_plan(units, B, gamma, nctas, prm.lse_d == nullptr, chunks, pieces);
            size_t zero_bytes = 0;
            const size_t need = bv::flow_scratch_bytes(B, gamma, plan, &zero_bytes);
            const int slot = static_cast<int>(d->flow_calls++ % 4);
            if (d->flow_bytes[slot] < need) {
                if (d->flow_ws[slot]) cudaFree(d->flow_ws[slot]);
                d->flow_ws[slot] = nullptr;
                d->flow_bytes[slot] = 0;
                d->flow_clean[slot] = 0;
                cudaError_t e = cudaMalloc(&d->flow_ws[slot], need);
                if (e != cudaSuccess) return cuda_fail(e);
                d->flow_bytes[slot] = need;
            }
            bv::FlowScratch fl;
            bv::flow_scratch_layout(d->flow_ws[slot], B, gamma, plan, &fl);
            if (const char* env = std::getenv("BV_FLOW_DEPTH")) {
                const int v = std::atoi(env);
                if (v >= 2 && v <= 6) fl.depth = v;
            }
            // The kernel leaves its counters and flags at zero when it ends, so they are cleared here only
            // when the area is new or a larger problem needs more of them than the last launch left clean.
            cudaError_t e = cudaSuccess;
            if (d->flow_clean[slot] < zero_bytes) {
                e = cudaMemsetAsync(d->flow_ws[slot], 0, zero_bytes, stream);
                if (e != cudaSuccess) return cuda_fail(e);
            }
            d->flow_clean[slot] = zero_bytes;
            long long items = static_cast<long long>(fl.total_s1);
            if (nctas > items) nctas = items;
            prm.ticket = nullptr;
            prm.nclusters = 0;
            e = bv::launch_flow(prm, fl, dtype, static_cast<int>(nctas), stream);
            if (e != cudaSuccess) return cuda_fail(e);
            t_last_launches = 1;
            return BV_OK;
        }
    }

    if (prm.lse_d != nullptr || prm.greedy) return BV_ERR_UNSUPPORTED;   // (the flow kernel could not be launched)

    if (algo == bv::kBlockVerify && vec && forced("resident")) {
        const long long units = static_cast<long long>(row_bytes / 16);
        int best_c = 0, best_nk = 0, best_n = 0;
        long long best_sms = -1;
        const char* ec = std::getenv("BV_RES_CLUSTER");
        for (int c = bv::kMaxCluster; c >= 1; c /= 2) {
            if (ec && std::atoi(ec) != c) continue;
            const long long per_warp = ((units + c - 1) / c + 15) / 16;
            int nk = 0;
            for (int cand : {2, 4, 8}) if (per_warp <= 32LL * cand) { nk = cand; break; }
            if (!nk) continue;
            int& cached = d->res_clusters[dtype][nk][c];
            if (cached == 0) {
                cached = bv::resident_max_clusters(dtype, nk, c);
                if (cached <= 0) cached = -1;
            }
            if (cached < 0) continue;
            const int n = B < cached ? B : cached;
            const long long sms = static_cast<long long>(n) * c;
            if (sms >= best_sms) { best_sms = sms; best_c = c; best_nk = nk; best_n = n; }
        }
        if (best_c) {
            prm.ticket = nullptr;
            prm.nclusters = best_n;
            cudaError_t e = bv::launch_resident(prm, dtype, best_nk, best_c, best_n, stream);
            if (e != cudaSuccess) return cuda_fail(e);
            t_last_launches = 1;
            return BV_OK;
        }
    }

    int cluster = pick_cluster(*d, B, row_bytes);
    if (vec && !forced("stream")) {
        int& cc = d->clu_clusters[algo][dtype][cluster];
        if (cc == 0) {
            cc = bv::cluster_max_clusters(algo, dtype, cluster);
            if (cc <= 0) cc = -1;
        }
        if (cc > 0) {
            int n = B < cc ? B : cc;
            if (const char* env = std::getenv("BV_MAX_CLUSTERS")) {
                const int cap = std::atoi(env);
                if (cap > 0 && cap < n) n = cap;
            }
            prm.ticket = d->tickets + 2 * (d->calls++ % kTicketSlots);
            prm.nclusters = n;
            cudaError_t e = bv::launch_cluster(prm, algo, dtype, cluster, n, stream);
            if (e != cudaSuccess) return cuda_fail(e);
            t_last_launches = 1;
            return BV_OK;
        }
    }
    int& cached = d->max_clusters[algo][dtype][vec ? 1 : 0][cluster];
    if (cached == 0) {
        cached = bv::stream_max_clusters(algo, dtype, vec, cluster);
        if (cached <= 0) cached = -1;
    }
    if (cached < 0) return BV_ERR_UNSUPPORTED;
    const int nclusters = B < cached ? B : cached;

    prm.ticket = d->tickets + 2 * (d->calls++ % kTicketSlots);
    prm.nclusters = nclusters;

    cudaError_t e = bv::launch_stream(prm, algo, dtype, vec, cluster, nclusters, stream);
    if (e != cudaSuccess) return cuda_fail(e);
    t_last_launches = 1;
    return BV_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int run_host(int algo, const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
             int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol) {
    int rc = check_args(tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
    if (rc != BV_OK) return rc;
    if (B == 0) return BV_OK;
    const size_t esz = dtype == BV_DTYPE_F32 ? 4 : 2;
    const size_t n_t = static_cast<size_t>(B) * (gamma + 1) * V * esz;
    const size_t n_d = static_cast<size_t>(B) * gamma * V * esz;
    const size_t n_tok = static_cast<size_t>(B) * gamma * 4, n_uni = static_cast<size_t>(B) * (gamma + 2) * 4;
    const size_t n_ot = static_cast<size_t>(B) * (gamma + 1) * 4, n_ol = static_cast<size_t>(B) * 4;
    const size_t o_t = 0, o_d = align_up(o_t + n_t, 256), o_tok = align_up(o_d + n_d, 256);
    const size_t o_uni = align_up(o_tok + n_tok, 256), o_ot = align_up(o_uni + n_uni, 256);
    const size_t o_ol = align_up(o_ot + n_ot, 256), total = align_up(o_ol + n_ol, 256);

    char* base = nullptr;
    cudaStream_t s = nullptr;
    int* status_word = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        DeviceState* d = nullptr;
        if ((rc = device_state(&d)) != BV_OK) return rc;
        cudaError_t e;
        if (!d->stream && (e = cudaStreamCreateWithFlags(&d->stream, cudaStreamNonBlocking)) != cudaSuccess)
            return cuda_fail(e);
        if (d->stage_bytes < total) {
            if (d->stage) cudaFree(d->stage);
            d->stage = nullptr;
            d->stage_bytes = 0;
            if ((e = cudaMalloc(&d->stage, total)) != cudaSuccess) return cuda_fail(e);
            d->stage_bytes = total;
        }
        base = static_cast<char*>(d->stage);
        s = d->stream;
        status_word = reinterpret_cast<int*>(d->tickets + 2 * kTicketSlots);
    }
    cudaError_t e;
    if ((e = cudaMemcpyAsync(base + o_t, tgt, n_t, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(base + o_d, drf, n_d, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(base + o_tok, tok, n_tok, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(base + o_uni, uni, n_uni, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    rc = run_device(algo, base + o_t, base + o_d, reinterpret_cast<const int32_t*>(base + o_tok),
                    reinterpret_cast<const float*>(base + o_uni), B, gamma, V, dtype, T,
                    reinterpret_cast<int32_t*>(base + o_ot), reinterpret_cast<int32_t*>(base + o_ol),
                    nullptr, nullptr, nullptr, nullptr, nullptr, s);
    if (rc != BV_OK) return rc;
    if ((e = cudaMemcpyAsync(ot, base + o_ot, n_ot, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(ol, base + o_ol, n_ol, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    int status = 0;
    if ((e = cudaMemcpyAsync(&status, status_word, sizeof(int), cudaMemcpyDeviceToHost, s)) != cudaSuccess)
        return cuda_fail(e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(e);
    return status ? BV_ERR_TIMEOUT : BV_OK;
}

}  // namespace

extern "C" {

int bv_verify(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
              int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, nullptr, nullptr,
                      nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

int bv_verify_lse(const void* tgt, const void* drf, const int32_t* tok, const float* uni, const float* draft_lse,
                  int B, int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    if (!draft_lse) return BV_ERR_INVALID_ARG;
    t_given_lse_d = draft_lse;
    const int rc = run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, nullptr, nullptr,
                              nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
    t_given_lse_d = nullptr;
    return rc;
}

int bv_verify_lse_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, const float* draft_lse,
                     int B, int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p,
                     float* out_S, float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    if (!draft_lse) return BV_ERR_INVALID_ARG;
    t_given_lse_d = draft_lse;
    const int rc = run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, out_p, out_S,
                              out_h, out_lse_t, out_lse_d, static_cast<cudaStream_t>(stream));
    t_given_lse_d = nullptr;
    return rc;
}

int gbv_verify(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
               int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    t_greedy = 1;
    const int rc = run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, nullptr, nullptr,
                              nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
    t_greedy = 0;
    return rc;
}

int gbv_verify_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                  int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
                  float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    t_greedy = 1;
    const int rc = run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, out_p, out_S,
                              out_h, out_lse_t, out_lse_d, static_cast<cudaStream_t>(stream));
    t_greedy = 0;
    return rc;
}

int tv_verify(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
              int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, nullptr, nullptr,
                      nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

int bv_verify_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                 int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
                 float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, out_p, out_S,
                      out_h, out_lse_t, out_lse_d, static_cast<cudaStream_t>(stream));
}

int tv_verify_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                 int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
                 float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, out_p, out_S,
                      out_h, out_lse_t, out_lse_d, static_cast<cudaStream_t>(stream));
}

int bv_verify_host(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
                   int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol) {
    return run_host(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
}

int tv_verify_host(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
                   int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol) {
    return run_host(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
}

int bv_release(void) {
    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return BV_ERR_UNSUPPORTED;
    DeviceState& d = g_dev[dev];
    if ((e = cudaDeviceSynchronize()) != cudaSuccess) return cuda_fail(e);
    if (d.stage) cudaFree(d.stage);
    if (d.tickets) cudaFree(d.tickets);
    for (void* w : d.flow_ws) if (w) cudaFree(w);
    if (d.stream) cudaStreamDestroy(d.stream);
    d = DeviceState{};
    return BV_OK;
}

int bv_last_launch_count(void) { return t_last_launches; }
int bv_last_cuda_error(void) { return t_last_cuda_error; }

const char* bv_status_string(int status) {
    switch (status) {
        case BV_OK: return "ok";
        case BV_ERR_INVALID_ARG: return "invalid argument";
        case BV_ERR_UNSUPPORTED: return "unsupported shape or device";
        case BV_ERR_CUDA: return "CUDA runtime error";
        case BV_ERR_TIMEOUT: return "device-side wait timed out";
        case BV_ERR_TOO_LARGE: return "problem needs more scratch than the no-allocation entry point has";
        default: return "unknown status";
    }
}

int bv_version(void) { return 100; }

}  // extern "C"
