// Block Verification for callers that must not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits at call time: inside a
// serving loop whose memory pool owns every byte of the device and treats a foreign
// allocation as a leak or an out-of-memory risk, inside code that may be under stream
// capture (where an allocation is an error), or in a process whose allocator hooks forbid
// it.  bv_verify() keeps its scratch in buffers it allocates on demand, so it does not
// suit them.  bv_verify_noalloc() runs the same flow kernel with its scratch in a
// fixed array that is part of the library image: nothing is allocated, ever, at the price
// of a hard size limit and of one array shared by every call on a device.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <mutex>

#include "../../include/bv.h"
#include "bv_launch.h"

namespace {

// Every GPU that loads the library holds this array until the process exits.
constexpr size_t kScratchBytes = static_cast<size_t>(BV_NOALLOC_SCRATCH_BYTES);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct NoAllocDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;   // device address of g_noalloc_scratch on this device
    int sm_count = 0;
    int ctas_per_sm[2] = {};
};
NoAllocDevice g_na[kMaxDevices];
std::mutex g_na_mu;

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" int bv_verify_noalloc(const void* tgt, const void* drf, const int32_t* tok, const float* uni, int B,
                                 int gamma, int V, int dtype, float T, int32_t* ot, int32_t* ol, void* stream) {
    bv::note_launches(0);
    const int rc = bv::check_verify_args(tgt, drf, tok, uni, B, gamma, V, dtype, T, ot, ol);
    if (rc != BV_OK) return rc;
    const size_t esz = dtype == BV_DTYPE_F32 ? 4 : 2;
    const size_t row_bytes = static_cast<size_t>(V) * esz;
    // only the 128-bit path exists here: rows of whole 16-byte vectors on 16-byte aligned bases
    if (row_bytes % 16 != 0 || !aligned_to(tgt, 16) || !aligned_to(drf, 16)) return BV_ERR_UNSUPPORTED;
    if (B == 0) return BV_OK;

    std::lock_guard<std::mutex> lock(g_na_mu);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return bv::note_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return BV_ERR_UNSUPPORTED;
    NoAllocDevice& d = g_na[dev];
    if (!d.ready) {
        // Set-up, once per device with that device current.  In host code the array's name only
        // stands for the symbol; the address a kernel can use comes from the runtime.
        void* p = nullptr;
        if ((e = cudaGetSymbolAddress(&p, g_noalloc_scratch)) != cudaSuccess) return bv::note_cuda_error(e);
        if (p == nullptr) return BV_ERR_UNSUPPORTED;
        int major = 0;
        if ((e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess)
            return bv::note_cuda_error(e);
        if (major < 10) return BV_ERR_UNSUPPORTED;
        d.scratch = static_cast<unsigned char*>(p);
        d.ready = true;
    }
    int& per_sm = d.ctas_per_sm[dtype];
    if (per_sm == 0) {
        per_sm = bv::flow_max_ctas_per_sm(dtype);
        if (per_sm <= 0) per_sm = -1;
    }
    if (per_sm < 0) return BV_ERR_UNSUPPORTED;

    // same chunking rule as bv_verify, so both entry points take identical arithmetic paths
    const long long units = static_cast<long long>(row_bytes / 16);
    const bv::FlowPlan plan = bv::flow_plan(units, B, gamma, static_cast<long long>(d.sm_count) * per_sm, true, 0, 0);
    size_t zero_bytes = 0;
    const size_t need = bv::flow_scratch_bytes(B, gamma, plan, &zero_bytes) + 256;   // + the status word
    if (need > kScratchBytes) return BV_ERR_TOO_LARGE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps what the previous call left: counters, flags and the queues must
    // start at zero, and so does the status word at the very end of the used part.
    if ((e = cudaMemsetAsync(d.scratch, 0, zero_bytes, s)) != cudaSuccess) return bv::note_cuda_error(e);
    unsigned char* status_word = d.scratch + (need - 256);
    if ((e = cudaMemsetAsync(status_word, 0, 256, s)) != cudaSuccess) return bv::note_cuda_error(e);

    bv::FlowScratch fl;
    bv::flow_scratch_layout(d.scratch, B, gamma, plan, &fl);
    bv::Params prm{};
    prm.tgt = tgt; prm.drf = drf; prm.tok = tok; prm.uni = uni;
    prm.B = B; prm.gamma = gamma; prm.V = V;
    const double kd = 1.4426950408889634073599246810019 / static_cast<double>(T);
    prm.kd = kd;
    prm.kf = static_cast<float>(kd);
    prm.out_tokens = ot; prm.out_len = ol;
    prm.algo = bv::kBlockVerify;
    prm.status = reinterpret_cast<int*>(status_word);
    long long items = static_cast<long long>(fl.total_s1);
    long long nctas = static_cast<long long>(d.sm_count) * per_sm;
    if (nctas > items) nctas = items;
    if ((e = bv::launch_flow(prm, fl, dtype, static_cast<int>(nctas), s)) != cudaSuccess) return bv::note_cuda_error(e);
    bv::note_launches(1);
    return BV_OK;
}
