// sysconv1d_host_static: the host-buffer 1-D convolution for callers that cannot
// allocate device memory.  See include/sysconv.h for the contract.
//
// sysconv1d_host stages x and y in a device workspace that the caller allocates.
// Some callers have no way to do that: code that runs after an application has
// handed all device memory to its own arena, plug-ins that are forbidden to call
// the CUDA allocator (cudaMalloc serialises the whole device and may fail late),
// and steady-state loops of real-time pipelines where an allocation is a policy
// violation.  For them the staging area is a fixed array in this library's device
// image.  Every GPU that loads the library pays kStaticScratchBytes for it until
// the process exits.
#include <mutex>

#include "sysconv_common.cuh"

// plain host-buffer sequence, defined beside sysconv1d_host
extern "C" int sysconv1d_host_plain(const void *x_host, long long n, const void *w_host, int q, void *y_host,
                                    int batch, int dtype, int design, void *workspace_dev,
                                    long long workspace_bytes, void *stream);

namespace {

constexpr long long kStaticScratchBytes = 16LL << 20;     // 16 MiB: x and y of up to ~2 Mi fp32 samples

// Staging area for x (first part) and y (second part).  In host code this name is
// only a handle for the runtime, not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the staging area on the current device; resolved once per device.
int static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SYSCONV_ECUDA;
    if (dev < 0 || dev >= kMaxDevices) return SYSCONV_EUNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress((void **)&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr)
            return SYSCONV_ECUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return SYSCONV_OK;
}

}  // namespace

extern "C" {

long long sysconv_static_scratch_bytes(void) { return kStaticScratchBytes; }

int sysconv1d_host_static(const void *x_host, long long n, const void *w_host, int q, void *y_host,
                          int batch, int dtype, int design, void *stream)
{
    if (!x_host || !y_host || !w_host) return SYSCONV_EINVAL;
    const long long need = sysconv1d_host_workspace_bytes(n, q, batch, dtype);
    if (need < 0) return SYSCONV_EINVAL;
    if (need > kStaticScratchBytes) return SYSCONV_ETOOLARGE;
    void *scratch = nullptr;
    const int st = static_scratch(&scratch);
    if (st != SYSCONV_OK) return st;
    // The plain sequence of sysconv1d_host (no helper streams or events are created), with the built-in
    // staging area as the workspace: copy in, convolve, copy out, all on `stream`.  The kernels read x only inside [0, n) and write every
    // one of the n-q+1 outputs, so stale contents of the area from earlier calls are never seen.
    return sysconv1d_host_plain(x_host, n, w_host, q, y_host, batch, dtype, design, scratch, kStaticScratchBytes,
                                stream);
}

}  // extern "C"
