// C-ABI layer: argument checks, per-device and per-stream workspace, launch-shape selection and
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
constexpr int kTicketSlots = 64;  // concurrent calls of the cluster kernels on one device each need their own slot
// Logit bytes up to which the small-batch kernel is the default (measured against the flow kernel at
// V = 152064, B <= 32: Algorithm 2 gains up to about 90 MB at low and high acceptance alike, Algorithm 1,
// whose one residual sweep per sequence is cheap, up to about 160 MB)
constexpr long long kSmallBytes[2] = {160LL << 20, 90LL << 20};   // [algo]
constexpr int kStreamSlots = 32;  // streams per device that keep a workspace of their own

// Tuning and test options (bv_set_option); their first values come from the environment, read once.
struct Options {
    int kernel = 0;        // 0: chosen by shape; 1 flow, 2 cluster, 3 stream, 4 small-batch
    int small_bytes = 0;   // logit bytes (in MB) up to which the small-batch kernel is chosen; 0: the built-in limit
    int cluster = 0;       // cluster width of the cluster / stream kernels (1, 2, 4, 8); 0: chosen by shape
    int max_clusters = 0;  // cap on the clusters launched; 0: none
    int flow_chunks = 0, flow_pieces = 0, flow_ctas = 0, flow_depth = 0;   // 0: chosen by shape
    int flow_fine = 0;     // > 0: this many blocks at the end of the batch have their rows cut into the finer chunks
    int flow_keep_l2 = 0;  // 1: the lines of a first sweep stay in L2 at normal priority; 0: every load streams past L2
    int wait_limit = 0;    // polls after which a bounded device-side wait gives up; 0: the built-in limits
    int never_signal = 0;  // test switch: the flow kernel's workers never report an item as swept
};
Options g_opt;
std::once_flag g_opt_once;

int env_int(const char* name) {
    const char* v = std::getenv(name);
    return v ? std::atoi(v) : 0;
}
int kernel_code(const char* v) {
    if (!v) return 0;
    if (!std::strcmp(v, "flow")) return 1;
    if (!std::strcmp(v, "cluster")) return 2;
    if (!std::strcmp(v, "stream")) return 3;
    if (!std::strcmp(v, "small")) return 4;
    return 0;
}
void load_env_options() {
    g_opt.kernel = kernel_code(std::getenv("BV_KERNEL"));
    g_opt.cluster = env_int("BV_CLUSTER");
    g_opt.max_clusters = env_int("BV_MAX_CLUSTERS");
    g_opt.flow_chunks = env_int("BV_FLOW_CHUNKS");
    g_opt.flow_pieces = env_int("BV_FLOW_PIECES");
    g_opt.flow_ctas = env_int("BV_FLOW_CTAS");
    g_opt.flow_depth = env_int("BV_FLOW_DEPTH");
}

// The workspace a stream's calls share.  Calls on one stream run one after the other, and the flow
// kernel leaves its counters at zero, so one area per stream serves any number of calls in flight;
// it grows with cudaMallocAsync / cudaFreeAsync on that stream, which do not synchronise the device.
struct StreamSlot {
    cudaStream_t stream = nullptr;
    bool used = false;
    void* ws = nullptr;        // [status word, 256 bytes][flow scratch]
    size_t bytes = 0;
    size_t clean = 0;          // leading bytes of the flow scratch known to be zero between calls
    unsigned long long stamp = 0;
};

struct DeviceState {
    bool ready = false;
    int sm_count = 0;
    int cc_major = 0;
    unsigned int* tickets = nullptr;  // [kTicketSlots][2], zero when idle
    unsigned long long calls = 0;
    int max_clusters[2][2][2][bv::kMaxCluster + 1] = {};  // [algo][dtype][vec][cluster], 0 = not asked yet
    int clu_clusters[2][2][bv::kMaxCluster + 1] = {};     // cluster kernel: [algo][dtype][cluster]
    StreamSlot slots[kStreamSlots];
    unsigned long long clock = 0;
    int flow_ctas_per_sm[2] = {};
    int small_ctas[2] = {};            // small-batch kernel: CTAs of a launch per dtype (0: not asked yet)
    // staging for the host-buffer entry points
    void* stage = nullptr;
    size_t stage_bytes = 0;
    cudaStream_t stream = nullptr;
};

DeviceState g_dev[kMaxDevices];
std::mutex g_mu;

thread_local int t_last_launches = 0;
thread_local int t_last_kernel = 0;     // which kernel the last verification call on this thread launched (the "kernel" option's codes)
thread_local int t_last_cuda_error = 0;

int cuda_fail(cudaError_t e) { return bv::note_cuda_error(e); }

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
        if ((e = cudaMalloc(&d.tickets, sizeof(unsigned int) * 2 * kTicketSlots)) != cudaSuccess)
            return cuda_fail(e);
        if ((e = cudaMemset(d.tickets, 0, sizeof(unsigned int) * 2 * kTicketSlots)) != cudaSuccess)
            return cuda_fail(e);
        d.ready = true;
    }
    *out = &d;
    return BV_OK;
}

// The workspace of `stream` with room for `need` bytes of flow scratch behind its status word.
// A stream seen for the first time takes a free entry, or the one used longest ago (whose area is
// freed in its own stream's order).
int stream_slot(DeviceState& d, cudaStream_t stream, size_t need, StreamSlot** out) {
    StreamSlot* s = nullptr;
    StreamSlot* victim = nullptr;
    for (StreamSlot& c : d.slots) {
        if (c.used && c.stream == stream) { s = &c; break; }
        if (!victim || (victim->used && (!c.used || c.stamp < victim->stamp))) victim = &c;
    }
    cudaError_t e;
    if (!s) {
        s = victim;
        if (s->used && s->ws && (e = cudaFreeAsync(s->ws, s->stream)) != cudaSuccess) return cuda_fail(e);
        *s = StreamSlot{};
        s->used = true;
        s->stream = stream;
    }
    s->stamp = ++d.clock;
    const size_t total = 256 + need;
    if (s->bytes < total) {
        if (s->ws && (e = cudaFreeAsync(s->ws, stream)) != cudaSuccess) return cuda_fail(e);
        s->ws = nullptr; s->bytes = 0; s->clean = 0;
        if ((e = cudaMallocAsync(&s->ws, total, stream)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaMemsetAsync(s->ws, 0, 256, stream)) != cudaSuccess) return cuda_fail(e);   // the status word
        s->bytes = total;
    }
    *out = s;
    return BV_OK;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Cluster width for the streaming kernel: wide enough that a CTA's slice of a row
// is at most 64 KB, widened further while the batch alone cannot fill the SMs.
int pick_cluster(const DeviceState& d, const Options& opt, int B, size_t row_bytes) {
    if (opt.cluster == 1 || opt.cluster == 2 || opt.cluster == 4 || opt.cluster == 8) return opt.cluster;
    int c = 1;
    while (c < bv::kMaxCluster && row_bytes / c > (64u << 10)) c *= 2;
    while (c < bv::kMaxCluster && static_cast<long long>(B) * c < d.sm_count && row_bytes / (2 * c) >= (8u << 10))
        c *= 2;
    // With several sequences per cluster to go through, narrower clusters (more sequences at a time,
    // cheaper exchanges) win: measured 0.43 against 0.57 ms at B = 256, gamma = 8, V = 152064.
    if (c == 8 && static_cast<long long>(B) * c >= 8LL * d.sm_count) c = 4;
    return c;
}

struct Extra {              // what only some entry points pass
    const float* lse_d = nullptr;   // supplied draft log-normalisers (bv_verify_lse)
    int greedy = 0;                 // Algorithm 4 instead of Algorithm 2 (gbv_verify)
    int probs = 0;                  // the rows hold probabilities, not logits (bv_verify_probs, tv_verify_probs)
    float* out_p = nullptr; float* out_S = nullptr; float* out_h = nullptr;
    float* out_lse_t = nullptr; float* out_lse_d = nullptr;
};

int run_device(int algo, const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
               int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, const Extra& ex, cudaStream_t stream) {
    t_last_launches = 0;
    t_last_kernel = 0;
    int rc = bv::check_verify_args(tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
    if (rc != BV_OK) return rc;
    if (B == 0) return BV_OK;
    std::call_once(g_opt_once, load_env_options);

    std::lock_guard<std::mutex> lock(g_mu);
    const Options opt = g_opt;
    DeviceState* d = nullptr;
    if ((rc = device_state(&d)) != BV_OK) return rc;

    const size_t esz = dtype == BV_DTYPE_F32 ? 4 : 2;
    const size_t row_bytes = static_cast<size_t>(V) * esz;
    const bool vec = (row_bytes % 16 == 0) && aligned(tgt, 16) && aligned(drf, 16);

    bv::Params prm{};
    prm.tgt = tgt; prm.drf = drf; prm.tok = tok; prm.uni = uni;
    prm.lse_d = ex.lse_d;
    prm.greedy = ex.greedy;
    prm.probs = ex.probs;
    prm.B = B; prm.gamma = gamma; prm.V = V;
    const double kd = 1.4426950408889634073599246810019 / static_cast<double>(T);
    prm.kd = kd;
    prm.kf = static_cast<float>(kd);
    prm.out_tokens = ot; prm.out_len = ol;
    prm.out_p = ex.out_p; prm.out_S = ex.out_S; prm.out_h = ex.out_h;
    prm.out_lse_t = ex.out_lse_t; prm.out_lse_d = ex.out_lse_d;
    prm.wait_limit = opt.wait_limit > 0 ? static_cast<unsigned>(opt.wait_limit) : 0u;
    prm.never_signal = opt.never_signal;

    prm.algo = algo;
    const bool flow_ok = vec && (opt.kernel == 0 || opt.kernel == 1);

    // A few sequences whose logits fit in L2: the launch is a matter of latency, and the kernel with two
    // grid-wide barriers instead of queues takes half the time of the flow kernel or less.
    const long long logit_bytes = static_cast<long long>(B) * (2 * gamma + 1) * static_cast<long long>(row_bytes);
    const long long small_limit = opt.small_bytes > 0 ? static_cast<long long>(opt.small_bytes) << 20 : kSmallBytes[algo == bv::kBlockVerify ? 1 : 0];
    // (given probabilities only a few row pairs per sequence are read whatever the size of the rest: there the
    // small-batch kernel wins up to 16 sequences, 17 against 33 us for one, 33 against 38 us for sixteen)
    if (vec && bv::small_fits(B, gamma) &&
        (opt.kernel == 4 || (opt.kernel == 0 && (prm.probs ? B <= 16 : logit_bytes <= small_limit)))) {
        int& nc = d->small_ctas[dtype];
        if (nc == 0) {
            nc = bv::small_max_ctas(dtype, d->sm_count);
            if (nc <= 0) nc = -1;
        }
        if (nc > 0) {
            const bv::SmallPlan plan = bv::small_plan(static_cast<long long>(row_bytes / 16), B, gamma, nc);
            StreamSlot* slot = nullptr;
            if ((rc = stream_slot(*d, stream, bv::small_scratch_bytes(B, gamma, plan), &slot)) != BV_OK) return rc;
            slot->clean = 0;                // (the area the flow kernel expects to find zero is written here)
            bv::SmallScratch sc;
            // the barrier words share the 256-byte block of the status word: zero since it was allocated
            bv::small_scratch_layout(static_cast<char*>(slot->ws) + 256, reinterpret_cast<unsigned*>(static_cast<char*>(slot->ws) + 128),
                                     B, gamma, plan, &sc);
            prm.ticket = nullptr;
            prm.nclusters = 0;
            prm.status = static_cast<int*>(slot->ws);
            cudaError_t e = bv::launch_small(prm, sc, dtype, nc, stream);
            if (e != cudaSuccess) return cuda_fail(e);
            t_last_launches = 1; t_last_kernel = 4;
            return BV_OK;
        }
    }

    // (only the two kernels above and below serve these entry points)
    if ((prm.lse_d != nullptr || prm.greedy || prm.probs) && !flow_ok) return BV_ERR_UNSUPPORTED;

    // 16-byte rows: the flow of independent work items (both algorithms)
    if (flow_ok) {
        int& per_sm = d->flow_ctas_per_sm[dtype];
        if (per_sm == 0) {
            per_sm = bv::flow_max_ctas_per_sm(dtype);
            if (per_sm <= 0) per_sm = -1;
        }
        if (per_sm > 0) {
            const long long units = static_cast<long long>(row_bytes / 16);
            long long nctas = static_cast<long long>(d->sm_count) * per_sm;
            if (opt.flow_ctas >= 1 && opt.flow_ctas < nctas) nctas = opt.flow_ctas;
            const int chunks = (opt.flow_chunks >= 1 && opt.flow_chunks <= bv::kFlowMaxChunks) ? opt.flow_chunks : 0;
            const int pieces = (opt.flow_pieces >= 1 && opt.flow_pieces <= 8) ? opt.flow_pieces : 0;
            // (with supplied draft normalisers a first-sweep item streams one row, not two)
            bv::FlowPlan plan = bv::flow_plan(units, B, gamma, nctas, prm.lse_d == nullptr, chunks, pieces, algo == bv::kTokenVerify, prm.probs != 0);
            if (opt.flow_fine > 0 && algo != bv::kTokenVerify && !prm.probs && plan.nch_late > plan.nch) plan.fine_from = opt.flow_fine < B ? B - opt.flow_fine : 0;
            size_t zero_bytes = 0;
            const size_t need = bv::flow_scratch_bytes(B, gamma, plan, &zero_bytes);
            StreamSlot* slot = nullptr;
            if ((rc = stream_slot(*d, stream, need, &slot)) != BV_OK) return rc;
            char* scratch = static_cast<char*>(slot->ws) + 256;
            bv::FlowScratch fl;
            bv::flow_scratch_layout(scratch, B, gamma, plan, &fl);
            // (with every position swept the second sweeps are the larger half of the launch and never wait for one another: deeper measured better)
            if (prm.out_p || prm.out_S || prm.out_h || prm.out_lse_t || prm.out_lse_d) fl.depth = 3;
            if (opt.flow_depth >= 2 && opt.flow_depth <= 6) fl.depth = opt.flow_depth;
            fl.keep_l2 = opt.flow_keep_l2 == 1;
            // The kernel leaves its counters and flags at zero when it ends, so they are cleared here only
            // when the area is new or a larger problem needs more of them than the last launch left clean.
            cudaError_t e = cudaSuccess;
            if (slot->clean < zero_bytes) {
                e = cudaMemsetAsync(scratch, 0, zero_bytes, stream);
                if (e != cudaSuccess) return cuda_fail(e);
            }
            slot->clean = zero_bytes;
            // (given probabilities the items are the pieces of the positions swept: at most all of them)
            long long items = prm.probs ? static_cast<long long>(B) * (gamma + 1) * fl.np : static_cast<long long>(fl.total_s1);
            if (nctas > items) nctas = items;
            prm.ticket = nullptr;
            prm.nclusters = 0;
            prm.status = static_cast<int*>(slot->ws);
            e = bv::launch_flow(prm, fl, dtype, static_cast<int>(nctas), stream);
            if (e != cudaSuccess) return cuda_fail(e);
            t_last_launches = 1; t_last_kernel = 1;
            return BV_OK;
        }
    }

    if (prm.lse_d != nullptr || prm.greedy || prm.probs) return BV_ERR_UNSUPPORTED;   // (the flow kernel could not be launched)

    StreamSlot* slot = nullptr;
    if ((rc = stream_slot(*d, stream, 0, &slot)) != BV_OK) return rc;
    prm.status = static_cast<int*>(slot->ws);

    int cluster = pick_cluster(*d, opt, B, row_bytes);
    if (vec && opt.kernel != 3) {
        int& cc = d->clu_clusters[algo][dtype][cluster];
        if (cc == 0) {
            cc = bv::cluster_max_clusters(algo, dtype, cluster);
            if (cc <= 0) cc = -1;
        }
        if (cc > 0) {
            int n = B < cc ? B : cc;
            if (opt.max_clusters > 0 && opt.max_clusters < n) n = opt.max_clusters;
            prm.ticket = d->tickets + 2 * (d->calls++ % kTicketSlots);
            prm.nclusters = n;
            cudaError_t e = bv::launch_cluster(prm, algo, dtype, cluster, n, stream);
            if (e != cudaSuccess) return cuda_fail(e);
            t_last_launches = 1; t_last_kernel = 2;
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
    t_last_launches = 1; t_last_kernel = 3;
    return BV_OK;
}

// Reads and clears the status word of `stream`'s workspace; waits for the stream.
int take_stream_status(cudaStream_t stream) {
    int* word = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        DeviceState* d = nullptr;
        const int rc = device_state(&d);
        if (rc != BV_OK) return rc;
        for (StreamSlot& c : d->slots)
            if (c.used && c.stream == stream) word = static_cast<int*>(c.ws);
    }
    cudaError_t e;
    if (!word) {
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(e);
        return BV_OK;
    }
    int status = 0;
    if ((e = cudaMemcpyAsync(&status, word, sizeof(int), cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemsetAsync(word, 0, sizeof(int), stream)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(e);
    return status ? BV_ERR_TIMEOUT : BV_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int run_host(int algo, const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
             int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol) {
    int rc = bv::check_verify_args(tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
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
    {
        std::lock_guard<std::mutex> lock(g_mu);
        DeviceState* d = nullptr;
        if ((rc = device_state(&d)) != BV_OK) return rc;
        cudaError_t e;
        if (!d->stream && (e = cudaStreamCreateWithFlags(&d->stream, cudaStreamNonBlocking)) != cudaSuccess)
            return cuda_fail(e);
        // (this entry point waits for its result anyway, so its staging buffer grows with plain cudaMalloc)
        if (d->stage_bytes < total) {
            if (d->stage) cudaFree(d->stage);
            d->stage = nullptr;
            d->stage_bytes = 0;
            if ((e = cudaMalloc(&d->stage, total)) != cudaSuccess) return cuda_fail(e);
            d->stage_bytes = total;
        }
        base = static_cast<char*>(d->stage);
        s = d->stream;
    }
    cudaError_t e;
    if ((e = cudaMemcpyAsync(base + o_t, tgt, n_t, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(base + o_d, drf, n_d, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(base + o_tok, tok, n_tok, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(base + o_uni, uni, n_uni, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    rc = run_device(algo, base + o_t, base + o_d, reinterpret_cast<const int32_t*>(base + o_tok),
                    reinterpret_cast<const float*>(base + o_uni), B, gamma, V, dtype, T,
                    reinterpret_cast<int32_t*>(base + o_ot), reinterpret_cast<int32_t*>(base + o_ol), Extra{}, s);
    if (rc != BV_OK) return rc;
    if ((e = cudaMemcpyAsync(ot, base + o_ot, n_ot, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(ol, base + o_ol, n_ol, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    return take_stream_status(s);
}

Extra diagnostics(float* out_p, float* out_S, float* out_h, float* out_lse_t, float* out_lse_d) {
    Extra ex;
    ex.out_p = out_p; ex.out_S = out_S; ex.out_h = out_h; ex.out_lse_t = out_lse_t; ex.out_lse_d = out_lse_d;
    return ex;
}

}  // namespace

namespace bv {

int note_cuda_error(cudaError_t e) {
    t_last_cuda_error = static_cast<int>(e);
    cudaGetLastError();
    return BV_ERR_CUDA;
}
void note_launches(int n) { t_last_launches = n; }

int check_verify_args(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
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

}  // namespace bv

extern "C" {

int bv_verify(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
              int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, Extra{},
                      static_cast<cudaStream_t>(stream));
}

int bv_verify_lse(const void* tgt, const void* drf, const int32_t* tok, const float* uni, const float* draft_lse,
                  int B, int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    if (!draft_lse) return BV_ERR_INVALID_ARG;
    Extra ex;
    ex.lse_d = draft_lse;
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int bv_verify_lse_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, const float* draft_lse,
                     int B, int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p,
                     float* out_S, float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    if (!draft_lse) return BV_ERR_INVALID_ARG;
    Extra ex = diagnostics(out_p, out_S, out_h, out_lse_t, out_lse_d);
    ex.lse_d = draft_lse;
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int tv_verify_lse(const void* tgt, const void* drf, const int32_t* tok, const float* uni, const float* draft_lse,
                  int B, int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    if (!draft_lse) return BV_ERR_INVALID_ARG;
    Extra ex;
    ex.lse_d = draft_lse;
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int tv_verify_lse_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, const float* draft_lse,
                     int B, int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p,
                     float* out_S, float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    if (!draft_lse) return BV_ERR_INVALID_ARG;
    Extra ex = diagnostics(out_p, out_S, out_h, out_lse_t, out_lse_d);
    ex.lse_d = draft_lse;
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int bv_verify_probs(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                    int V, int dtype, int32_t* ot, int32_t* ol, float* out_p, float* out_S, float* out_h, void* stream) {
    Extra ex = diagnostics(out_p, out_S, out_h, nullptr, nullptr);
    ex.probs = 1;
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, 1.f, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int tv_verify_probs(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                    int V, int dtype, int32_t* ot, int32_t* ol, float* out_p, float* out_S, float* out_h, void* stream) {
    Extra ex = diagnostics(out_p, out_S, out_h, nullptr, nullptr);
    ex.probs = 1;
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, 1.f, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int gbv_verify(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
               int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    Extra ex;
    ex.greedy = 1;
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int gbv_verify_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                  int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
                  float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    Extra ex = diagnostics(out_p, out_S, out_h, out_lse_t, out_lse_d);
    ex.greedy = 1;
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, ex, static_cast<cudaStream_t>(stream));
}

int tv_verify(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
              int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol, Extra{},
                      static_cast<cudaStream_t>(stream));
}

int bv_verify_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                 int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
                 float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    return run_device(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol,
                      diagnostics(out_p, out_S, out_h, out_lse_t, out_lse_d), static_cast<cudaStream_t>(stream));
}

int tv_verify_ex(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B, int gamma,
                 int V, int dtype, float T, int32_t* ot, int32_t* ol, float* out_p, float* out_S,
                 float* out_h, float* out_lse_t, float* out_lse_d, void* stream) {
    return run_device(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol,
                      diagnostics(out_p, out_S, out_h, out_lse_t, out_lse_d), static_cast<cudaStream_t>(stream));
}

int bv_verify_host(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
                   int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol) {
    return run_host(bv::kBlockVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
}

int tv_verify_host(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
                   int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol) {
    return run_host(bv::kTokenVerify, tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
}

int bv_stream_status(void* stream) { return take_stream_status(static_cast<cudaStream_t>(stream)); }

int bv_set_option(const char* name, int value) {
    if (!name) return BV_ERR_INVALID_ARG;
    std::call_once(g_opt_once, load_env_options);
    std::lock_guard<std::mutex> lock(g_mu);
    if (!std::strcmp(name, "kernel")) g_opt.kernel = value;
    else if (!std::strcmp(name, "small_bytes")) g_opt.small_bytes = value;
    else if (!std::strcmp(name, "cluster")) g_opt.cluster = value;
    else if (!std::strcmp(name, "max_clusters")) g_opt.max_clusters = value;
    else if (!std::strcmp(name, "flow_chunks")) g_opt.flow_chunks = value;
    else if (!std::strcmp(name, "flow_pieces")) g_opt.flow_pieces = value;
    else if (!std::strcmp(name, "flow_ctas")) g_opt.flow_ctas = value;
    else if (!std::strcmp(name, "flow_depth")) g_opt.flow_depth = value;
    else if (!std::strcmp(name, "flow_keep_l2")) g_opt.flow_keep_l2 = value;
    else if (!std::strcmp(name, "flow_fine")) g_opt.flow_fine = value;
    else if (!std::strcmp(name, "wait_limit")) g_opt.wait_limit = value;
    else if (!std::strcmp(name, "never_signal")) g_opt.never_signal = value;
    else return BV_ERR_INVALID_ARG;
    return BV_OK;
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
    for (StreamSlot& c : d.slots) if (c.used && c.ws) cudaFree(c.ws);
    if (d.stream) cudaStreamDestroy(d.stream);
    d = DeviceState{};
    return BV_OK;
}

int bv_last_launch_count(void) { return t_last_launches; }
int bv_last_kernel(void) { return t_last_kernel; }
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

int bv_version(void) { return 200; }

}  // extern "C"
