// sama_adapt_noalloc: the adaptation + squared-norm kernel for callers that
// must not allocate device memory.
//
// The regular entry point takes a context whose creation calls cudaMalloc for
// the reduction's scratch (one partial sum per block, an arrival counter and
// the total).  Some callers cannot do that: code running under a framework
// whose caching allocator owns all device memory and forbids raw cudaMalloc,
// plug-ins loaded into a process that is already inside a memory-frozen region
// (e.g. after a pool has been sized for a serving engine), or a library
// initialised lazily from a point where a synchronising allocation is not
// permitted.  For them the same scratch lives in the file-scope device array
// below, which every GPU that loads this library holds until the process
// exits.
#include <mutex>

#include "sama_internal.h"

using namespace sama;

namespace {

constexpr int kMaxDevices = 64;

// Scratch: the scalars block (sum, arrival counter) followed by the block partials.
constexpr size_t kHeaderBytes = 256;
constexpr size_t kScratchBytes = kHeaderBytes + sizeof(double) * kMaxPartials;  // 33,024 bytes
static_assert(sizeof(DeviceScalars) <= kHeaderBytes, "header too small");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

struct PerDevice {
    void* scratch = nullptr;  // device address of g_noalloc_scratch on this device
    int sm_count = 0;
};
PerDevice g_dev[kMaxDevices];
std::mutex g_mu;

// First use on a device: resolve the array's device address (its name is only
// a host-side handle in host code) and read the SM count.  No allocation.
int setup_device(int dev, PerDevice** out, int* cuda_err) {
    std::lock_guard<std::mutex> lock(g_mu);
    PerDevice& d = g_dev[dev];
    if (!d.scratch) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) { *cuda_err = (int)e; return SAMA_ERR_CUDA; }
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess || sms < 1) { *cuda_err = (int)e; return SAMA_ERR_CUDA; }
        d.sm_count = sms;
        d.scratch = ptr;
    }
    *out = &d;
    return SAMA_OK;
}

}  // namespace

extern "C" int sama_adapt_noalloc(int64_t n, const float* m, const float* s, const float* g_base,
                                  const float* g_meta, const sama_adam_t* adam, float* p_out, double* sumsq_out,
                                  void* stream) {
    if (!sumsq_out) return SAMA_ERR_NULL;
    AdaptConsts c;
    const int rc = validate_adapt(SAMA_NOALLOC_MAX_N, n, m, s, g_base, g_meta, adam, p_out, sumsq_out, &c);
    if (rc != SAMA_OK) return rc;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SAMA_ERR_CUDA;
    PerDevice* d = nullptr;
    int cuda_err = 0;
    const int rs = setup_device(dev, &d, &cuda_err);
    if (rs != SAMA_OK) return rs;

    // A context on the stack that points at the static scratch; nothing in it is owned.
    sama_ctx ctx = {};
    ctx.device = dev;
    ctx.sm_count = d->sm_count;
    ctx.max_n = SAMA_NOALLOC_MAX_N;
    ctx.scalars = reinterpret_cast<DeviceScalars*>(d->scratch);
    ctx.partials = reinterpret_cast<double*>(static_cast<unsigned char*>(d->scratch) + kHeaderBytes);

    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the last call left: the arrival counter must start at zero.
    if (cudaMemsetAsync(d->scratch, 0, kHeaderBytes, st) != cudaSuccess) return SAMA_ERR_CUDA;
    if (launch_adapt_sumsq(&ctx, n, m, s, c.identity ? nullptr : g_base, g_meta, c, p_out, sumsq_out, st) !=
        cudaSuccess)
        return SAMA_ERR_CUDA;
    return SAMA_OK;
}
