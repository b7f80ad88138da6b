// C ABI of libsysconv.so: argument validation and dispatch.  See include/sysconv.h
// for the contract of every entry point.  No device memory is allocated here.
#include <atomic>
#include <climits>
#include <mutex>

#include "sysconv_common.cuh"
#include "tma_utils.cuh"

#include <cstdlib>

// Raised (set to 1) by a kernel that gave up a bounded wait; read and cleared by sysconv_device_status().
static __device__ unsigned g_status_word;

namespace sysconv {
bool dependent_launch_enabled()
{
    static const bool on = std::getenv("SYSCONV_NO_PDL") == nullptr;
    return on;
}
}  // namespace sysconv

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

// a * b * c for positive factors, or -1 if the product (plus alignment slack) would not fit a long long
long long checked_product(long long a, long long b, long long c)
{
    const long long limit = LLONG_MAX / 4 - 256;
    if (a <= 0 || b <= 0 || c <= 0) return -1;
    if (a > limit / b) return -1;
    const long long ab = a * b;
    if (ab > limit / c) return -1;
    return ab * c;
}

// One CTA that waits, bounded, for bytes nobody sends: it arms a shared-memory barrier with an expected
// byte count, issues NO copy (so nothing is in flight towards the CTA), polls `polls` times, raises the
// status word exactly as the pipelined kernels do when their limit runs out, and returns.
__global__ void wait_timeout_selftest_kernel(unsigned *status_word, unsigned polls)
{
    sysconv::dependent_launch_enter();
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        sysconv::mbar_init(&bar, 1);
        sysconv::mbar_init_fence();
        sysconv::mbar_arrive_expect_tx(&bar, 16);
    }
    __syncthreads();
    const bool ok = sysconv::mbar_wait_bounded(&bar, 0, polls);
    const bool give_up = __syncthreads_or(!ok) != 0;
    if (give_up && threadIdx.x == 0) atomicExch(status_word, 1u);
}

int finish(cudaError_t err, int launches)
{
    if (err == sysconv::kNoInstantiation) return SYSCONV_EUNSUPPORTED;
    if (err != cudaSuccess) return SYSCONV_ECUDA;
    g_launches.fetch_add(launches, std::memory_order_relaxed);
    return SYSCONV_OK;
}

// Helper streams and events of the pipelined host-buffer entry points: one set per device, created on
// first use and kept for the life of the process.  Copies in run on `h2d`, copies out on `d2h`, kernels
// on the caller's stream; fork/join events tie the helpers into the caller's stream order.
constexpr int kMaxPipeChunks = 16;
struct HostPipe {
    bool ready = false;
    std::mutex busy;                            // one pipelined call at a time per device
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t forked = nullptr, joined = nullptr;
    cudaEvent_t in_done[kMaxPipeChunks], k_done[kMaxPipeChunks];
    bool fork(cudaStream_t s)
    {
        return cudaEventRecord(forked, s) == cudaSuccess && cudaStreamWaitEvent(h2d, forked, 0) == cudaSuccess &&
               cudaStreamWaitEvent(d2h, forked, 0) == cudaSuccess;
    }
    bool join(cudaStream_t s)
    {
        bool ok = cudaEventRecord(joined, d2h) == cudaSuccess && cudaStreamWaitEvent(s, joined, 0) == cudaSuccess;
        ok = ok && cudaEventRecord(joined, h2d) == cudaSuccess && cudaStreamWaitEvent(s, joined, 0) == cudaSuccess;
        return ok;
    }
};
HostPipe g_pipe[kMaxDevices];

HostPipe *host_pipe()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_device_mutex);
    HostPipe &p = g_pipe[dev];
    if (!p.ready) {
        bool ok = cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.forked, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.joined, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kMaxPipeChunks; ++i)
            ok = cudaEventCreateWithFlags(&p.in_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.k_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        p.ready = true;
    }
    return &p;
}

bool valid_enums(int dtype, int design)
{
    return (dtype == SYSCONV_F32 || dtype == SYSCONV_U8S8_S32) && design >= SYSCONV_WS && design <= SYSCONV_FFS;
}

bool main_design(int design) { return design == SYSCONV_WS || design == SYSCONV_OS || design == SYSCONV_IS; }

// true if [a, a+an) and [b, b+bn) overlap
bool overlaps(const void *a, unsigned long long an, const void *b, unsigned long long bn)
{
    const unsigned long long pa = reinterpret_cast<unsigned long long>(a);
    const unsigned long long pb = reinterpret_cast<unsigned long long>(b);
    return pa < pb + bn && pb < pa + an;
}

int dispatch2d_once(const sysconv::Conv2DArgs &a, const void *w_host, int q, int p, int dtype, int design,
                    cudaStream_t s);

// The image index is a grid dimension (at most 65535): larger batches go out in slices, one launch each.
constexpr int kMaxBatchPerLaunch = 65535;
int dispatch2d(const sysconv::Conv2DArgs &a, const void *w_host, int q, int p, int dtype, int design,
               cudaStream_t s)
{
    if (a.batch <= kMaxBatchPerLaunch) return dispatch2d_once(a, w_host, q, p, dtype, design, s);
    for (int b0 = 0; b0 < a.batch; b0 += kMaxBatchPerLaunch) {
        sysconv::Conv2DArgs part = a;
        part.batch = a.batch - b0 < kMaxBatchPerLaunch ? a.batch - b0 : kMaxBatchPerLaunch;
        part.x = static_cast<const char *>(a.x) + static_cast<long long>(b0) * a.x_bstride * (long long)in_elt_bytes(dtype);
        part.y = static_cast<char *>(a.y) + static_cast<long long>(b0) * a.y_bstride * 4LL;
        const int st = dispatch2d_once(part, w_host, q, p, dtype, design, s);
        if (st != SYSCONV_OK) return st;
    }
    return SYSCONV_OK;
}

int dispatch2d_once(const sysconv::Conv2DArgs &a, const void *w_host, int q, int p, int dtype, int design,
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
        // a batch of tiny signals (the paper's own experiment shape): small arrays side by side in a warp
        if (conv1d_tiles_eligible(a, design, q)) return finish(launch_conv1d_f32_tiles(design, a, w, q, s, &launches), launches);
        // a batch of SHORT signals: the 1-D kernels give every signal tiles of 1216 or more outputs of its own, so
        // signals of a few hundred samples would leave most of each array idle.  Such a batch is an image with one
        // signal per row and a one-row filter: the 2-D kernels of the same design march down the rows with
        // 128- or 256-PE strips (2^26 samples as signals of 100: 0.9-1.3 ms -> 0.13-0.33 ms; equal at 1000)
        // Filters of 16 to 32 taps: the output- and input-stationary 2-D kernels are compiled for such rows as well.
        const bool long_row = q > kMaxQ2 && (design == SYSCONV_OS || design == SYSCONV_IS);
        if (batch >= 2 && n_out <= kShortSignal1 && main_design(design) && (q <= kMaxQ2 || long_row)) {
            Conv2DArgs g;
            g.x = x_dev; g.y = y_dev;
            g.width = static_cast<int>(n); g.height = batch;
            g.out_w = static_cast<int>(n_out); g.out_h = batch;
            g.x_pitch = x_batch_stride; g.y_pitch = y_batch_stride;
            g.x_bstride = 0; g.y_bstride = 0; g.batch = 1;
            if (long_row) return finish(launch_conv2d_f32_long_rows(design, g, w, q, s, &launches), launches);
            return dispatch2d(g, w_host, q, 1, dtype, design, s);
        }
        const DeviceInfo *d = device_info();
        if (!d) return SYSCONV_ECUDA;
        cudaError_t err = design == SYSCONV_OS   ? launch_conv1d_f32_os(a, w, q, d->status_word, s, &launches)
                          : design == SYSCONV_IS ? launch_conv1d_f32_is(a, w, q, d->status_word, s, &launches)
                          : design == SYSCONV_WS ? launch_conv1d_f32_ws(a, w, q, d->status_word, s, &launches)
                                                 : launch_conv1d_f32_other(design, a, w, q, d->status_word, s, &launches);
        return finish(err, launches);
    }
    // integer signals run as one-row images through the 2-D integer kernels
    if (!main_design(design)) return SYSCONV_EUNSUPPORTED;
    if (q > kMaxQ2) return SYSCONV_EUNSUPPORTED;
    if (n > 0x7fffffffLL) return SYSCONV_EUNSUPPORTED;
    // one signal per image row (the batch stride is the row pitch)
    Conv2DArgs a;
    a.x = x_dev; a.y = y_dev;
    a.width = static_cast<int>(n); a.height = batch;
    a.out_w = static_cast<int>(n_out); a.out_h = batch;
    a.x_pitch = x_batch_stride; a.y_pitch = y_batch_stride;
    a.x_bstride = 0; a.y_bstride = 0; a.batch = 1;
    return dispatch2d(a, w_host, q, 1, dtype, design, s);
}

int sysconv1d_strided(const void *x_dev, long long n, long long x_batch_stride, const void *w_host, int q, int stride,
                      void *y_dev, long long y_batch_stride, int batch, int dtype, int design, void *stream)
{
    using namespace sysconv;
    if (stride < 1) return SYSCONV_EINVAL;
    if (stride == 1)
        return sysconv1d(x_dev, n, x_batch_stride, w_host, q, y_dev, y_batch_stride, batch, dtype, design, stream);
    if (!x_dev || !y_dev || !w_host) return SYSCONV_EINVAL;
    if (!valid_enums(dtype, design)) return SYSCONV_EINVAL;
    if (q < 1 || n < q || batch < 1) return SYSCONV_EINVAL;
    const long long n_out = (n - q) / stride + 1;
    if (batch > 1 && (x_batch_stride < n || y_batch_stride < n_out)) return SYSCONV_EINVAL;
    if (batch == 1) { x_batch_stride = n; y_batch_stride = n_out; }
    const unsigned long long x_bytes = ((unsigned long long)(batch - 1) * x_batch_stride + n) * in_elt_bytes(dtype);
    const unsigned long long y_bytes = ((unsigned long long)(batch - 1) * y_batch_stride + n_out) * 4ull;
    if (overlaps(x_dev, x_bytes, y_dev, y_bytes)) return SYSCONV_EINVAL;
    if (dtype != SYSCONV_F32 || q > kMaxQ1) return SYSCONV_EUNSUPPORTED;
    if (stride != 2) {
        // any other stride: the run-time-stride output-stationary array, the signals as one-row images
        if (design != SYSCONV_OS || batch > 65535 || n > 0x7fffffffLL) return SYSCONV_EUNSUPPORTED;
        Conv2DArgs g;
        g.x = x_dev; g.y = y_dev;
        g.width = static_cast<int>(n); g.height = 1; g.out_w = static_cast<int>(n_out); g.out_h = 1;
        g.x_pitch = n; g.y_pitch = n_out; g.x_bstride = x_batch_stride; g.y_bstride = y_batch_stride; g.batch = batch;
        int launches = 0;
        const cudaError_t err = launch_conv_f32_strided_any(g, static_cast<const float *>(w_host), q, 1, stride, 1,
                                                            static_cast<cudaStream_t>(stream), &launches);
        return finish(err, launches);
    }
    if (design != SYSCONV_OS && design != SYSCONV_IS) return SYSCONV_EUNSUPPORTED;
    Conv1DArgs a;
    a.x = x_dev; a.y = y_dev; a.n = n; a.n_out = n_out;
    a.x_bstride = x_batch_stride; a.y_bstride = y_batch_stride; a.batch = batch;
    int launches = 0;
    const DeviceInfo *d = device_info();
    if (!d) return SYSCONV_ECUDA;
    const cudaError_t err = launch_conv1d_f32_stride2(design, a, static_cast<const float *>(w_host), q, d->status_word,
                                                      static_cast<cudaStream_t>(stream), &launches);
    return finish(err, launches);
}

int sysconv2d_strided(const void *x_dev, int width, int height, long long x_pitch, long long x_batch_stride,
                      const void *w_host, int q, int p, int stride_c, int stride_r, void *y_dev, long long y_pitch,
                      long long y_batch_stride, int batch, int dtype, int design, void *stream)
{
    using namespace sysconv;
    if (stride_c < 1 || stride_r < 1) return SYSCONV_EINVAL;
    if (stride_c == 1 && stride_r == 1)
        return sysconv2d(x_dev, width, height, x_pitch, x_batch_stride, w_host, q, p, y_dev, y_pitch, y_batch_stride,
                         batch, dtype, design, stream);
    if (!x_dev || !y_dev || !w_host) return SYSCONV_EINVAL;
    if (!valid_enums(dtype, design)) return SYSCONV_EINVAL;
    if (q < 1 || p < 1 || width < q || height < p || batch < 1) return SYSCONV_EINVAL;
    const int out_w = (width - q) / stride_c + 1, out_h = (height - p) / stride_r + 1;
    if (x_pitch < width || y_pitch < out_w) return SYSCONV_EINVAL;
    const long long x_img = (long long)(height - 1) * x_pitch + width;
    const long long y_img = (long long)(out_h - 1) * y_pitch + out_w;
    if (batch > 1 && (x_batch_stride < x_img || y_batch_stride < y_img)) return SYSCONV_EINVAL;
    if (batch == 1) { x_batch_stride = x_img; y_batch_stride = y_img; }
    const unsigned long long x_bytes = ((unsigned long long)(batch - 1) * x_batch_stride + x_img) * in_elt_bytes(dtype);
    const unsigned long long y_bytes = ((unsigned long long)(batch - 1) * y_batch_stride + y_img) * 4ull;
    if (overlaps(x_dev, x_bytes, y_dev, y_bytes)) return SYSCONV_EINVAL;
    if (dtype != SYSCONV_F32 || batch > 65535 || q > kMaxQ2 || p > kMaxP2) return SYSCONV_EUNSUPPORTED;
    if (design != SYSCONV_OS && design != SYSCONV_IS) return SYSCONV_EUNSUPPORTED;
    Conv2DArgs a;
    a.x = x_dev; a.y = y_dev;
    a.width = width; a.height = height; a.out_w = out_w; a.out_h = out_h;
    a.x_pitch = x_pitch; a.y_pitch = y_pitch;
    a.x_bstride = x_batch_stride; a.y_bstride = y_batch_stride; a.batch = batch;
    int launches = 0;
    cudaError_t err;
    if (stride_c == 2 && stride_r == 2 && p <= 7 && q <= 7) {
        err = launch_conv2d_f32_stride2(design, a, static_cast<const float *>(w_host), q, p,
                                        static_cast<cudaStream_t>(stream), &launches);
    } else {
        // other strides, mixed strides, larger filters: the run-time-stride output-stationary array
        if (design != SYSCONV_OS) return SYSCONV_EUNSUPPORTED;
        err = launch_conv_f32_strided_any(a, static_cast<const float *>(w_host), q, p, stride_c, stride_r,
                                          static_cast<cudaStream_t>(stream), &launches);
    }
    return finish(err, launches);
}

int sysconv2d_separable(const void *x_dev, int width, int height, long long x_pitch, long long x_batch_stride,
                        const void *u_host, int p, const void *v_host, int q, void *y_dev, long long y_pitch,
                        long long y_batch_stride, int batch, void *stream)
{
    using namespace sysconv;
    if (!x_dev || !y_dev || !u_host || !v_host) return SYSCONV_EINVAL;
    if (q < 1 || p < 1 || width < q || height < p || batch < 1) return SYSCONV_EINVAL;
    const int out_w = width - q + 1, out_h = height - p + 1;
    if (x_pitch < width || y_pitch < out_w) return SYSCONV_EINVAL;
    const long long x_img = (long long)(height - 1) * x_pitch + width;
    const long long y_img = (long long)(out_h - 1) * y_pitch + out_w;
    if (batch > 1 && (x_batch_stride < x_img || y_batch_stride < y_img)) return SYSCONV_EINVAL;
    if (batch == 1) { x_batch_stride = x_img; y_batch_stride = y_img; }
    const unsigned long long x_bytes = ((unsigned long long)(batch - 1) * x_batch_stride + x_img) * 4ull;
    const unsigned long long y_bytes = ((unsigned long long)(batch - 1) * y_batch_stride + y_img) * 4ull;
    if (overlaps(x_dev, x_bytes, y_dev, y_bytes)) return SYSCONV_EINVAL;
    if (q > kMaxQ2 || p > kMaxP2 || batch > 65535) return SYSCONV_EUNSUPPORTED;
    Conv2DArgs a;
    a.x = x_dev; a.y = y_dev;
    a.width = width; a.height = height; a.out_w = out_w; a.out_h = out_h;
    a.x_pitch = x_pitch; a.y_pitch = y_pitch;
    a.x_bstride = x_batch_stride; a.y_bstride = y_batch_stride; a.batch = batch;
    int launches = 0;
    const cudaError_t err = launch_conv2d_f32_separable(a, static_cast<const float *>(u_host), p,
                                                        static_cast<const float *>(v_host), q,
                                                        static_cast<cudaStream_t>(stream), &launches);
    return finish(err, launches);
}

int sysstencil2d(const void *u_dev, int width, int height, long long pitch, long long batch_stride, const void *k_host,
                 int sweeps, void *out_dev, long long out_pitch, long long out_batch_stride, int batch, void *scratch_dev,
                 void *stream)
{
    using namespace sysconv;
    constexpr int kFused = 4;                   // sweeps fused in one launch
    if (!u_dev || !out_dev || !k_host) return SYSCONV_EINVAL;
    if (width < 1 || height < 1 || batch < 1 || sweeps < 1) return SYSCONV_EINVAL;
    if (pitch < width || out_pitch < width) return SYSCONV_EINVAL;
    const long long u_img = (long long)(height - 1) * pitch + width;
    const long long o_img = (long long)(height - 1) * out_pitch + width;
    if (batch > 1 && (batch_stride < u_img || out_batch_stride < o_img)) return SYSCONV_EINVAL;
    if (batch == 1) { batch_stride = u_img; out_batch_stride = o_img; }
    const unsigned long long u_bytes = ((unsigned long long)(batch - 1) * batch_stride + u_img) * 4ull;
    const unsigned long long o_bytes = ((unsigned long long)(batch - 1) * out_batch_stride + o_img) * 4ull;
    if (overlaps(u_dev, u_bytes, out_dev, o_bytes)) return SYSCONV_EINVAL;
    const int launches_needed = (sweeps + kFused - 1) / kFused;
    if (launches_needed > 1) {
        if (!scratch_dev) return SYSCONV_EINVAL;
        if (overlaps(scratch_dev, o_bytes, out_dev, o_bytes) || overlaps(scratch_dev, o_bytes, u_dev, u_bytes)) return SYSCONV_EINVAL;
    }
    if (batch > 65535) return SYSCONV_EUNSUPPORTED;
    // Chain of launches, each fusing up to four sweeps; the intermediate grids alternate between the scratch
    // buffer and the output (both in the output's layout) so that the last launch writes the output.
    const float *k = static_cast<const float *>(k_host);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Conv2DArgs a;
    a.width = width; a.height = height; a.out_w = width; a.out_h = height; a.batch = batch;
    const void *src = u_dev;
    long long src_pitch = pitch, src_bstride = batch_stride;
    int launches = 0, left = sweeps;
    for (int l = 0; l < launches_needed; ++l) {
        const int fused = left < kFused ? left : kFused;
        void *dst = ((launches_needed - 1 - l) % 2 == 0) ? out_dev : scratch_dev;
        a.x = src; a.y = dst;
        a.x_pitch = src_pitch; a.x_bstride = src_bstride;
        a.y_pitch = out_pitch; a.y_bstride = out_batch_stride;
        const cudaError_t err = launch_stencil2d_f32(a, k, fused, s, &launches);
        if (err != cudaSuccess) return finish(err, launches);
        src = dst; src_pitch = out_pitch; src_bstride = out_batch_stride;
        left -= fused;
    }
    return finish(cudaSuccess, launches);
}

int sysconv_spacetime_describe(int p_c, int p_q, int s_c, int s_q, int q, int *info, char *name)
{
    return sysconv::spacetime_describe(p_c, p_q, s_c, s_q, q, info, name);
}

int sysconv1d_spacetime(const void *x_dev, long long n, const void *w_host, int q, void *y_dev, int p_c, int p_q, int s_c,
                        int s_q, void *stream)
{
    using namespace sysconv;
    if (!x_dev || !y_dev || !w_host) return SYSCONV_EINVAL;
    if (q < 1 || n < q) return SYSCONV_EINVAL;
    const long long n_out = n - q + 1;
    if (overlaps(x_dev, (unsigned long long)n * 4ull, y_dev, (unsigned long long)n_out * 4ull)) return SYSCONV_EINVAL;
    if (q > kMaxQ1) return SYSCONV_EUNSUPPORTED;
    const int plan = spacetime_describe(p_c, p_q, s_c, s_q, q, nullptr, nullptr);
    if (plan != SYSCONV_OK) return plan;
    const DeviceInfo *d = device_info();
    if (!d) return SYSCONV_ECUDA;
    int status = SYSCONV_OK, launches = 0;
    const cudaError_t err = launch_spacetime_conv1d(static_cast<const float *>(x_dev), n, static_cast<const float *>(w_host),
                                                    q, static_cast<float *>(y_dev), p_c, p_q, s_c, s_q, d->sm_count,
                                                    static_cast<cudaStream_t>(stream), &status, &launches);
    if (status != SYSCONV_OK) return status;
    return finish(err, launches);
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
    if (q > kMaxQ2 || p > kMaxP2 || !main_design(design)) return SYSCONV_EUNSUPPORTED;

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
    const long long in = checked_product(n, batch, (long long)in_elt_bytes(dtype));
    const long long out = checked_product(n - q + 1, batch, 4LL);
    if (in < 0 || out < 0) return -1;                    // sizes beyond the index type
    return align256(in) + align256(out);
}

long long sysconv2d_host_workspace_bytes(int width, int height, int q, int p, int batch, int dtype)
{
    if (q < 1 || p < 1 || width < q || height < p || batch < 1) return -1;
    if (dtype != SYSCONV_F32 && dtype != SYSCONV_U8S8_S32) return -1;
    const long long in = checked_product((long long)width * height, batch, (long long)in_elt_bytes(dtype));
    const long long out = checked_product((long long)(width - q + 1) * (height - p + 1), batch, 4LL);
    if (in < 0 || out < 0) return -1;                    // sizes beyond the index type
    return align256(in) + align256(out);
}

// ---- host-buffer entry points --------------------------------------------------------------------
// Plain form: one copy in, the kernel, one copy out, all on the caller's stream.
int sysconv1d_host_plain(const void *x_host, long long n, const void *w_host, int q, void *y_host, int batch,
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

int sysconv1d_host(const void *x_host, long long n, const void *w_host, int q, void *y_host, int batch,
                   int dtype, int design, void *workspace_dev, long long workspace_bytes, void *stream)
{
    if (!x_host || !y_host || !w_host || !workspace_dev) return SYSCONV_EINVAL;
    const long long need = sysconv1d_host_workspace_bytes(n, q, batch, dtype);
    if (need < 0 || workspace_bytes < need) return SYSCONV_EINVAL;
    if ((reinterpret_cast<unsigned long long>(workspace_dev) & 255ull) != 0) return SYSCONV_EINVAL;
    const long long n_out = n - q + 1;
    // long single signals: cut into chunks so that the copy in of chunk c+1, the kernel of chunk c and
    // the copy out of chunk c-1 overlap (PCIe is full duplex)
    const long long kChunkMin = 1LL << 20;
    long long chunks = (batch == 1) ? n_out / kChunkMin : 1;
    if (chunks > kMaxPipeChunks) chunks = kMaxPipeChunks;
    if (chunks < 2)
        return sysconv1d_host_plain(x_host, n, w_host, q, y_host, batch, dtype, design, workspace_dev,
                                    workspace_bytes, stream);
    HostPipe *pipe = host_pipe();
    if (!pipe) return SYSCONV_ECUDA;
    std::lock_guard<std::mutex> lock(pipe->busy);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long long esz = (long long)in_elt_bytes(dtype);
    char *xd = static_cast<char *>(workspace_dev);
    char *yd = xd + align256(n * esz);
    long long len = (n_out + chunks - 1) / chunks;
    len = (len + 9727) / 9728 * 9728;                    // whole tiles of every design; keeps 16-byte alignment
    if (!pipe->fork(s)) return SYSCONV_ECUDA;
    int c = 0;
    for (long long o0 = 0; o0 < n_out; o0 += len, ++c) {
        const long long o1 = o0 + len < n_out ? o0 + len : n_out;
        const long long in0 = o0 == 0 ? 0 : o0 + q - 1;           // inputs not yet copied by earlier chunks
        const long long in1 = o1 + q - 1;
        if (cudaMemcpyAsync(xd + in0 * esz, static_cast<const char *>(x_host) + in0 * esz, (in1 - in0) * esz,
                            cudaMemcpyHostToDevice, pipe->h2d) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaEventRecord(pipe->in_done[c], pipe->h2d) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaStreamWaitEvent(s, pipe->in_done[c], 0) != cudaSuccess) return SYSCONV_ECUDA;
        const int st = sysconv1d(xd + o0 * esz, (o1 - o0) + q - 1, 0, w_host, q, yd + o0 * 4, 0, 1, dtype, design, stream);
        if (st != SYSCONV_OK) { pipe->join(s); return st; }
        if (cudaEventRecord(pipe->k_done[c], s) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaStreamWaitEvent(pipe->d2h, pipe->k_done[c], 0) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaMemcpyAsync(static_cast<char *>(y_host) + o0 * 4, yd + o0 * 4, (o1 - o0) * 4,
                            cudaMemcpyDeviceToHost, pipe->d2h) != cudaSuccess) return SYSCONV_ECUDA;
    }
    return pipe->join(s) ? SYSCONV_OK : SYSCONV_ECUDA;
}

long long sysconv1d_host_multi_workspace_bytes(long long n, const int *q, int count, int dtype)
{
    if (!q || count < 1 || count > 64 || dtype != SYSCONV_F32) return -1;
    if (n < 1 || n > (LLONG_MAX / 4 - 256) / (4LL * (count + 1))) return -1;
    long long total = align256(n * 4LL);
    for (int j = 0; j < count; ++j) {
        if (q[j] < 1 || n < q[j]) return -1;
        total += align256((n - q[j] + 1) * 4LL);
    }
    return total;
}

int sysconv1d_host_multi(const void *x_host, long long n, int count, const void *const *w_host, const int *q,
                         const int *design, void *const *y_host, int dtype, void *workspace_dev,
                         long long workspace_bytes, void *stream)
{
    if (!x_host || !w_host || !q || !design || !y_host || !workspace_dev) return SYSCONV_EINVAL;
    if (count < 1 || count > 64) return SYSCONV_EINVAL;
    if (dtype != SYSCONV_F32 && dtype != SYSCONV_U8S8_S32) return SYSCONV_EINVAL;
    if (dtype != SYSCONV_F32) return SYSCONV_EUNSUPPORTED;
    for (int j = 0; j < count; ++j) {
        if (!w_host[j] || !y_host[j] || q[j] < 1 || n < q[j] || !valid_enums(dtype, design[j])) return SYSCONV_EINVAL;
        if (q[j] > sysconv::kMaxQ1) return SYSCONV_EUNSUPPORTED;
    }
    const long long need = sysconv1d_host_multi_workspace_bytes(n, q, count, dtype);
    if (need < 0 || workspace_bytes < need) return SYSCONV_EINVAL;
    if ((reinterpret_cast<unsigned long long>(workspace_dev) & 255ull) != 0) return SYSCONV_EINVAL;
    int q_min = q[0], q_max = q[0];
    for (int j = 1; j < count; ++j) { q_min = q[j] < q_min ? q[j] : q_min; q_max = q[j] > q_max ? q[j] : q_max; }
    char *xd = static_cast<char *>(workspace_dev);
    char *yd[64];
    {
        char *at = xd + align256(n * 4LL);
        for (int j = 0; j < count; ++j) { yd[j] = at; at += align256((n - q[j] + 1) * 4LL); }
    }
    HostPipe *pipe = host_pipe();
    if (!pipe) return SYSCONV_ECUDA;
    std::lock_guard<std::mutex> lock(pipe->busy);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // chunks of output positions, the same for every job (a job's last chunk ends at its own n - q + 1)
    const long long span = n - q_min + 1;
    long long chunks = span / (1LL << 20);
    if (chunks > kMaxPipeChunks) chunks = kMaxPipeChunks;
    if (chunks < 1) chunks = 1;
    long long len = (span + chunks - 1) / chunks;
    len = (len + 9727) / 9728 * 9728;                    // whole tiles of every design; keeps 16-byte alignment
    if (!pipe->fork(s)) return SYSCONV_ECUDA;
    int c = 0;
    long long copied = 0;                                // inputs [0, copied) are on the device
    for (long long o0 = 0; o0 < span; o0 += len, ++c) {
        const long long o1 = o0 + len < span ? o0 + len : span;
        long long in1 = o1 + q_max - 1;
        if (in1 > n) in1 = n;
        if (in1 > copied) {
            if (cudaMemcpyAsync(xd + copied * 4, static_cast<const char *>(x_host) + copied * 4, (in1 - copied) * 4,
                                cudaMemcpyHostToDevice, pipe->h2d) != cudaSuccess) return SYSCONV_ECUDA;
            copied = in1;
        }
        if (cudaEventRecord(pipe->in_done[c], pipe->h2d) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaStreamWaitEvent(s, pipe->in_done[c], 0) != cudaSuccess) return SYSCONV_ECUDA;
        for (int j = 0; j < count; ++j) {
            const long long n_out = n - q[j] + 1;
            const long long e1 = o1 < n_out ? o1 : n_out;
            if (o0 >= e1) continue;
            const int st = sysconv1d(xd + o0 * 4, (e1 - o0) + q[j] - 1, 0, w_host[j], q[j], yd[j] + o0 * 4, 0, 1, dtype,
                                     design[j], stream);
            if (st != SYSCONV_OK) { pipe->join(s); return st; }
        }
        if (cudaEventRecord(pipe->k_done[c], s) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaStreamWaitEvent(pipe->d2h, pipe->k_done[c], 0) != cudaSuccess) return SYSCONV_ECUDA;
        for (int j = 0; j < count; ++j) {
            const long long n_out = n - q[j] + 1;
            const long long e1 = o1 < n_out ? o1 : n_out;
            if (o0 >= e1) continue;
            if (cudaMemcpyAsync(static_cast<char *>(y_host[j]) + o0 * 4, yd[j] + o0 * 4, (e1 - o0) * 4,
                                cudaMemcpyDeviceToHost, pipe->d2h) != cudaSuccess) return SYSCONV_ECUDA;
        }
    }
    return pipe->join(s) ? SYSCONV_OK : SYSCONV_ECUDA;
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
    const long long esz = (long long)in_elt_bytes(dtype);
    const int out_w = width - q + 1, out_h = height - p + 1;
    const long long x_img = (long long)width * height;
    const long long y_img = (long long)out_w * out_h;
    char *xd = static_cast<char *>(workspace_dev);
    char *yd = xd + align256(x_img * batch * esz);

    // chunks: whole images when there are several, else bands of output rows of a large image
    const bool by_image = batch >= 2;
    long long chunks = by_image ? batch : y_img / (1LL << 20);
    if (chunks > kMaxPipeChunks) chunks = kMaxPipeChunks;
    if (chunks < 2) {
        if (cudaMemcpyAsync(xd, x_host, x_img * batch * esz, cudaMemcpyHostToDevice, s) != cudaSuccess) return SYSCONV_ECUDA;
        const int st = sysconv2d(xd, width, height, width, x_img, w_host, q, p, yd, out_w, y_img, batch, dtype, design, stream);
        if (st != SYSCONV_OK) return st;
        if (cudaMemcpyAsync(y_host, yd, y_img * batch * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SYSCONV_ECUDA;
        return SYSCONV_OK;
    }
    HostPipe *pipe = host_pipe();
    if (!pipe) return SYSCONV_ECUDA;
    std::lock_guard<std::mutex> lock(pipe->busy);
    if (!pipe->fork(s)) return SYSCONV_ECUDA;
    const long long unit = by_image ? batch : out_h;             // images, or output rows of the one image
    const long long per = (unit + chunks - 1) / chunks;
    int c = 0;
    for (long long u0 = 0; u0 < unit; u0 += per, ++c) {
        const long long u1 = u0 + per < unit ? u0 + per : unit;
        long long in_off, in_len, y_off, y_len;
        int st;
        if (by_image) {
            in_off = u0 * x_img; in_len = (u1 - u0) * x_img; y_off = u0 * y_img; y_len = (u1 - u0) * y_img;
        } else {
            const long long row0 = u0 == 0 ? 0 : u0 + p - 1;     // input rows not yet copied by earlier chunks
            in_off = row0 * width; in_len = (u1 + p - 1 - row0) * width; y_off = u0 * out_w; y_len = (u1 - u0) * out_w;
        }
        if (cudaMemcpyAsync(xd + in_off * esz, static_cast<const char *>(x_host) + in_off * esz, in_len * esz,
                            cudaMemcpyHostToDevice, pipe->h2d) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaEventRecord(pipe->in_done[c], pipe->h2d) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaStreamWaitEvent(s, pipe->in_done[c], 0) != cudaSuccess) return SYSCONV_ECUDA;
        if (by_image)
            st = sysconv2d(xd + u0 * x_img * esz, width, height, width, x_img, w_host, q, p, yd + u0 * y_img * 4, out_w,
                           y_img, static_cast<int>(u1 - u0), dtype, design, stream);
        else
            st = sysconv2d(xd + u0 * width * esz, width, static_cast<int>(u1 - u0) + p - 1, width, 0, w_host, q, p,
                           yd + u0 * out_w * 4, out_w, 0, 1, dtype, design, stream);
        if (st != SYSCONV_OK) { pipe->join(s); return st; }
        if (cudaEventRecord(pipe->k_done[c], s) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaStreamWaitEvent(pipe->d2h, pipe->k_done[c], 0) != cudaSuccess) return SYSCONV_ECUDA;
        if (cudaMemcpyAsync(static_cast<char *>(y_host) + y_off * 4, yd + y_off * 4, y_len * 4, cudaMemcpyDeviceToHost,
                            pipe->d2h) != cudaSuccess) return SYSCONV_ECUDA;
    }
    return pipe->join(s) ? SYSCONV_OK : SYSCONV_ECUDA;
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
        case SYSCONV_FSM: return "FSM";
        case SYSCONV_BFS: return "BFS";
        case SYSCONV_FFS: return "FFS";
        default: return "?";
    }
}

int sysconv_device_status(void)
{
    const DeviceInfo *d = device_info();
    if (!d) return SYSCONV_ECUDA;
    unsigned flag = 0;
    // every stream of the device, non-blocking ones included: a kernel still running could raise the flag later
    if (cudaDeviceSynchronize() != cudaSuccess) return SYSCONV_ECUDA;
    if (cudaMemcpy(&flag, d->status_word, sizeof(flag), cudaMemcpyDeviceToHost) != cudaSuccess) return SYSCONV_ECUDA;
    if (flag == 0) return SYSCONV_OK;
    flag = 0;
    if (cudaMemcpy(d->status_word, &flag, sizeof(flag), cudaMemcpyHostToDevice) != cudaSuccess) return SYSCONV_ECUDA;
    return SYSCONV_ETIMEOUT;
}

int sysconv_selftest_wait_timeout(void *stream)
{
    const DeviceInfo *d = device_info();
    if (!d) return SYSCONV_ECUDA;
    sysconv::launch_kernel(wait_timeout_selftest_kernel, 1, 64, static_cast<cudaStream_t>(stream), d->status_word, 1u << 10);
    return finish(cudaGetLastError(), 1);
}

int sysconv_version(void) { return 200; }

long long sysconv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
