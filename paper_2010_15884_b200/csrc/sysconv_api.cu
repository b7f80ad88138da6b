// C ABI of libsysconv.so: argument validation and dispatch.  See include/sysconv.h
// for the contract of every entry point.  No device memory is allocated here.
#include <atomic>
#include <mutex>

#include "sysconv_common.cuh"

// Raised (set to 1) by a kernel that gave up a bounded wait; read and cleared by sysconv_device_status().
static __device__ unsigned g_status_word;

namespace {

std::atomic<long long> g_launches{0};

// per-device facts resolved on first use: SM count and the device address of g_status_word
constexpr int kMaxDevices = 64;
struct DeviceInfo {
    bool ready = false;
    int sm_count = 0;
    unsigned *status_word = nullptr;
};
std::mutex g_device_mutex;
DeviceInfo g_device[kMaxDevices];

const DeviceInfo *device_info()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_device_mutex);
    DeviceInfo &d = g_device[dev];
    if (!d.ready) {
        void *ptr = nullptr;
        if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
        if (cudaGetSymbolAddress(&ptr, g_status_word) != cudaSuccess || ptr == nullptr) return nullptr;
        d.status_word = static_cast<unsigned *>(ptr);
        d.ready = true;
    }
    return &d;
}

inline size_t in_elt_bytes(int dtype) { return dtype == SYSCONV_F32 ? 4 : 1; }
inline long long align256(long long v) { return (v + 255) & ~255LL; }

int finish(cudaError_t err, int launches)
{
    if (err == sysconv::kNoInstantiation) return SYSCONV_EUNSUPPORTED;
    if (err != cudaSuccess) return SYSCONV_ECUDA;
    g_launches.fetch_add(launches, std::memory_order_relaxed);
    return SYSCONV_OK;
}

bool valid_enums(int dtype, int design)
{
    return (dtype == SYSCONV_F32 || dtype == SYSCONV_U8S8_S32) &&
           (design == SYSCONV_WS || design == SYSCONV_OS || design == SYSCONV_IS);
}

// true if [a, a+an) and [b, b+bn) overlap
bool overlaps(const void *a, unsigned long long an, const void *b, unsigned long long bn)
{
    const unsigned long long pa = reinterpret_cast<unsigned long long>(a);
    const unsigned long long pb = reinterpret_cast<unsigned long long>(b);
    return pa < pb + bn && pb < pa + an;
}

int dispatch2d(const sysconv::Conv2DArgs &a, const void *w_host, int q, int p, int dtype, int design,
               cudaStream_t s)
{
    using namespace sysconv;
    int launches = 0;
    cudaError_t err;
    if (dtype == SYSCONV_F32) {
        const float *w = static_cast<const float *>(w_host);
        err = design == SYSCONV_OS   ? launch_conv2d_f32_os(a, w, q, p, s, &launches)
              : design == SYSCONV_IS ? launch_conv2d_f32_is(a, w, q, p, s, &launches)
                                     : launch_conv2d_f32_ws(a, w, q, p, s, &launches);
    } else {
        const int8_t *w = static_cast<const int8_t *>(w_host);
        err = design == SYSCONV_OS   ? launch_conv2d_u8_os(a, w, q, p, s, &launches)
              : design == SYSCONV_IS ? launch_conv2d_u8_is(a, w, q, p, s, &launches)
                                     : launch_conv2d_u8_ws(a, w, q, p, s, &launches);
    }
    return finish(err, launches);
}

}  // namespace

extern "C" {

int sysconv1d(const void *x_dev, long long n, long long x_batch_stride, const void *w_host, int q,
              void *y_dev, long long y_batch_stride, int batch, int dtype, int design, void *stream)
{
    using namespace sysconv;
    if (!x_dev || !y_dev || !w_host) return SYSCONV_EINVAL;
    if (!valid_enums(dtype, design)) return SYSCONV_EINVAL;
    if (q < 1 || n < q || batch < 1) return SYSCONV_EINVAL;
    const long long n_out = n - q + 1;
    if (batch > 1 && (x_batch_stride < n || y_batch_stride < n_out)) return SYSCONV_EINVAL;
    if (batch == 1) { x_batch_stride = n; y_batch_stride = n_out; }
    const unsigned long long x_bytes = ((unsigned long long)(batch - 1) * x_batch_stride + n) * in_elt_bytes(dtype);
    const unsigned long long y_bytes = ((unsigned long long)(batch - 1) * y_batch_stride + n_out) * 4ull;
    if (overlaps(x_dev, x_bytes, y_dev, y_bytes)) return SYSCONV_EINVAL;
    if (q > kMaxQ1) return SYSCONV_EUNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (dtype == SYSCONV_F32) {
        Conv1DArgs a;
        a.x = x_dev; a.y = y_dev; a.n = n; a.n_out = n_out;
        a.x_bstride = x_batch_stride; a.y_bstride = y_batch_stride; a.batch = batch;
        const float *w = static_cast<const float *>(w_host);
        int launches = 0;
        const DeviceInfo *d = device_info();
        if (!d) return SYSCONV_ECUDA;
        cudaError_t err = design == SYSCONV_OS   ? launch_conv1d_f32_os(a, w, q, d->status_word, s, &launches)
                          : design == SYSCONV_IS ? launch_conv1d_f32_is(a, w, q, d->status_word, s, &launches)
                                                 : launch_conv1d_f32_ws(a, w, q, d->status_word, s, &launches);
        return finish(err, launches);
    }
    // integer signals run as one-row images through the 2-D integer kernels
    if (q > kMaxQ2) return SYSCONV_EUNSUPPORTED;
    if (n > 0x7fffffffLL) return SYSCONV_EUNSUPPORTED;
    Conv2DArgs a;
    a.x = x_dev; a.y = y_dev;
    a.width = static_cast<int>(n); a.height = 1;
    a.out_w = static_cast<int>(n_out); a.out_h = 1;
    a.x_pitch = n; a.y_pitch = n_out;
    a.x_bstride = x_batch_stride; a.y_bstride = y_batch_stride; a.batch = batch;
    return dispatch2d(a, w_host, q, 1, dtype, design, s);
}

int sysconv2d(const void *x_dev, int width, int height, long long x_pitch, long long x_batch_stride,
              const void *w_host, int q, int p, void *y_dev, long long y_pitch, long long y_batch_stride,
              int batch, int dtype, int design, void *stream)
{
    using namespace sysconv;
    if (!x_dev || !y_dev || !w_host) return SYSCONV_EINVAL;
    if (!valid_enums(dtype, design)) return SYSCONV_EINVAL;
    if (q < 1 || p < 1 || width < q || height < p || batch < 1) return SYSCONV_EINVAL;
    const int out_w = width - q + 1, out_h = height - p + 1;
    if (x_pitch < width || y_pitch < out_w) return SYSCONV_EINVAL;
    const long long x_img = (long long)(height - 1) * x_pitch + width;
    const long long y_img = (long long)(out_h - 1) * y_pitch + out_w;
    if (batch > 1 && (x_batch_stride < x_img || y_batch_stride < y_img)) return SYSCONV_EINVAL;
    if (batch == 1) { x_batch_stride = x_img; y_batch_stride = y_img; }
    const unsigned long long x_bytes = ((unsigned long long)(batch - 1) * x_batch_stride + x_img) * in_elt_bytes(dtype);
    const unsigned long long y_bytes = ((unsigned long long)(batch - 1) * y_batch_stride + y_img) * 4ull;
    if (overlaps(x_dev, x_bytes, y_dev, y_bytes)) return SYSCONV_EINVAL;
    if (q > kMaxQ2 || p > kMaxP2) return SYSCONV_EUNSUPPORTED;

    Conv2DArgs a;
    a.x = x_dev; a.y = y_dev;
    a.width = width; a.height = height; a.out_w = out_w; a.out_h = out_h;
    a.x_pitch = x_pitch; a.y_pitch = y_pitch;
    a.x_bstride = x_batch_stride; a.y_bstride = y_batch_stride; a.batch = batch;
    return dispatch2d(a, w_host, q, p, dtype, design, static_cast<cudaStream_t>(stream));
}

long long sysconv1d_host_workspace_bytes(long long n, int q, int batch, int dtype)
{
    if (q < 1 || n < q || batch < 1) return -1;
    if (dtype != SYSCONV_F32 && dtype != SYSCONV_U8S8_S32) return -1;
    return align256(n * batch * (long long)in_elt_bytes(dtype)) + align256((n - q + 1) * batch * 4LL);
}

long long sysconv2d_host_workspace_bytes(int width, int height, int q, int p, int batch, int dtype)
{
    if (q < 1 || p < 1 || width < q || height < p || batch < 1) return -1;
    if (dtype != SYSCONV_F32 && dtype != SYSCONV_U8S8_S32) return -1;
    const long long in = (long long)width * height * batch * (long long)in_elt_bytes(dtype);
    const long long out = (long long)(width - q + 1) * (height - p + 1) * batch * 4LL;
    return align256(in) + align256(out);
}

int sysconv1d_host(const void *x_host, long long n, const void *w_host, int q, void *y_host, int batch,
                   int dtype, int design, void *workspace_dev, long long workspace_bytes, void *stream)
{
    if (!x_host || !y_host || !w_host || !workspace_dev) return SYSCONV_EINVAL;
    const long long need = sysconv1d_host_workspace_bytes(n, q, batch, dtype);
    if (need < 0 || workspace_bytes < need) return SYSCONV_EINVAL;
    if ((reinterpret_cast<unsigned long long>(workspace_dev) & 255ull) != 0) return SYSCONV_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long long x_bytes = n * batch * (long long)in_elt_bytes(dtype);
    const long long y_bytes = (n - q + 1) * batch * 4LL;
    char *xd = static_cast<char *>(workspace_dev);
    char *yd = xd + align256(x_bytes);
    if (cudaMemcpyAsync(xd, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return SYSCONV_ECUDA;
    const int st = sysconv1d(xd, n, n, w_host, q, yd, n - q + 1, batch, dtype, design, stream);
    if (st != SYSCONV_OK) return st;
    if (cudaMemcpyAsync(y_host, yd, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SYSCONV_ECUDA;
    return SYSCONV_OK;
}

int sysconv2d_host(const void *x_host, int width, int height, const void *w_host, int q, int p, void *y_host,
                   int batch, int dtype, int design, void *workspace_dev, long long workspace_bytes,
                   void *stream)
{
    if (!x_host || !y_host || !w_host || !workspace_dev) return SYSCONV_EINVAL;
    const long long need = sysconv2d_host_workspace_bytes(width, height, q, p, batch, dtype);
    if (need < 0 || workspace_bytes < need) return SYSCONV_EINVAL;
    if ((reinterpret_cast<unsigned long long>(workspace_dev) & 255ull) != 0) return SYSCONV_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long long x_img = (long long)width * height;
    const long long y_img = (long long)(width - q + 1) * (height - p + 1);
    const long long x_bytes = x_img * batch * (long long)in_elt_bytes(dtype);
    const long long y_bytes = y_img * batch * 4LL;
    char *xd = static_cast<char *>(workspace_dev);
    char *yd = xd + align256(x_bytes);
    if (cudaMemcpyAsync(xd, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return SYSCONV_ECUDA;
    const int st = sysconv2d(xd, width, height, width, x_img, w_host, q, p, yd, width - q + 1, y_img, batch,
                             dtype, design, stream);
    if (st != SYSCONV_OK) return st;
    if (cudaMemcpyAsync(y_host, yd, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SYSCONV_ECUDA;
    return SYSCONV_OK;
}

const char *sysconv_status_string(int status)
{
    switch (status) {
        case SYSCONV_OK: return "ok";
        case SYSCONV_EINVAL: return "invalid argument";
        case SYSCONV_EUNSUPPORTED: return "unsupported size";
        case SYSCONV_ECUDA: return "CUDA runtime error";
        case SYSCONV_ETIMEOUT: return "device-side wait timed out";
        case SYSCONV_ETOOLARGE: return "problem larger than the built-in staging area";
        default: return "?";
    }
}

const char *sysconv_design_name(int design)
{
    switch (design) {
        case SYSCONV_WS: return "WS/BSM";
        case SYSCONV_OS: return "OS/FBS";
        case SYSCONV_IS: return "IS/SBM";
        default: return "?";
    }
}

int sysconv_device_status(void)
{
    const DeviceInfo *d = device_info();
    if (!d) return SYSCONV_ECUDA;
    unsigned flag = 0;
    if (cudaMemcpy(&flag, d->status_word, sizeof(flag), cudaMemcpyDeviceToHost) != cudaSuccess) return SYSCONV_ECUDA;
    if (flag == 0) return SYSCONV_OK;
    flag = 0;
    if (cudaMemcpy(d->status_word, &flag, sizeof(flag), cudaMemcpyHostToDevice) != cudaSuccess) return SYSCONV_ECUDA;
    return SYSCONV_ETIMEOUT;
}

int sysconv_version(void) { return 101; }

long long sysconv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
