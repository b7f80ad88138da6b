// Measured denominators for the roofline figures: issue rates of the plain (non-tensor) datapaths the
// convolution kernels run on, and the yardstick kernels for the launch-bound problem sizes.
//
// sysconv_measure_peaks: one block of 1024 threads per SM runs a long, fully unrolled sequence of ONE kind
// of instruction on eight independent register chains per thread and times itself with the SM's cycle
// counter, so the result -- thread-level operations per clock per SM -- does not depend on the clock the
// board happens to run at.  Kinds: fp32 FMA, packed fp32x2 FMA with the multiplicand (x, x) (the form the
// paired passes use), 32-bit integer multiply-add, dp4a (four 8-bit multiply-adds per lane), warp shuffle.
// The streaming figure is a 128-bit copy kernel over the caller's scratch buffer timed with CUDA events.
//
// sysconv_floor_copy: a plain streaming pass with the byte counts of a convolution and none of its
// arithmetic (copy, or uint8 -> int32 widening), launched like the convolution kernels; the benchmark
// times it beside them: what one launch that only moves the bytes costs at that size.
#include <algorithm>
#include <vector>

#include "sysconv_common.cuh"

namespace {

using namespace sysconv;

constexpr int kPeakThreads = 1024;
constexpr int kChains = 8;
constexpr int kUnroll = 16;             // operations per chain and loop trip

enum PeakOp { kOpFfma = 0, kOpFfma2 = 1, kOpImad = 2, kOpDp4a = 3, kOpShfl = 4 };

template <int OP>
__global__ void __launch_bounds__(kPeakThreads) alu_rate_kernel(unsigned long long *cycles, float *sink, int trips, float seed)
{
    float f[kChains];
    float2 f2[kChains];
    int n[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) {
        f[c] = seed + c + threadIdx.x;
        f2[c] = make_float2(seed + c, seed - c);
        n[c] = static_cast<int>(seed) + c + threadIdx.x;
    }
    const float m = 1.0f + seed * 1e-9f, d = seed * 1e-9f;
    const float2 m2 = make_float2(m, m - d);
    const int im = 3 + static_cast<int>(seed);
    __syncthreads();
    const long long t0 = clock64();
#pragma unroll 1
    for (int t = 0; t < trips; ++t) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                if (OP == kOpFfma) f[c] = fmaf(f[c], m, d);
                if (OP == kOpFfma2) f2[c] = __ffma2_rn(make_float2(f[c], f[c]), m2, f2[c]);
                if (OP == kOpImad) n[c] = n[c] * im + c;
                if (OP == kOpDp4a) n[c] = __dp4a(n[c] | 0x01010101, im, n[c]);
                if (OP == kOpShfl) n[c] = __shfl_down_sync(kFullMask, n[c], 1);
            }
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc += f[c] + f2[c].x + f2[c].y + static_cast<float>(n[c]);
    if (acc == 12345.678f) sink[0] = acc;               // keeps the chains alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = static_cast<unsigned long long>(t1 - t0);
}

__global__ void __launch_bounds__(256) stream_copy_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, long long n16)
{
    dependent_launch_enter();
    const long long i = blockIdx.x * static_cast<long long>(blockDim.x) * 4 + threadIdx.x;
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (i + u * blockDim.x < n16) v[u] = src[i + u * blockDim.x];
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (i + u * blockDim.x < n16) dst[i + u * blockDim.x] = v[u];
}

// each thread widens four 32-bit words of pixels into four 128-bit words of int32
__global__ void __launch_bounds__(256) stream_widen_kernel(const unsigned *__restrict__ src, int4 *__restrict__ dst, long long words)
{
    dependent_launch_enter();
    const long long i = blockIdx.x * static_cast<long long>(blockDim.x) * 4 + threadIdx.x;
    unsigned v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = (i + u * blockDim.x < words) ? src[i + u * blockDim.x] : 0u;
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (i + u * blockDim.x < words)
            dst[i + u * blockDim.x] = make_int4(v[u] & 255, (v[u] >> 8) & 255, (v[u] >> 16) & 255, v[u] >> 24);
}

template <int OP>
double measure_alu(unsigned long long *cycles_dev, float *sink_dev, int sms, int ops_per_instruction)
{
    const int trips = 256;
    std::vector<unsigned long long> c(sms);
    double best = 0;
    for (int rep = 0; rep < 3; ++rep) {
        alu_rate_kernel<OP><<<sms, kPeakThreads>>>(cycles_dev, sink_dev, trips, 1.0f + rep);
        if (cudaMemcpy(c.data(), cycles_dev, sms * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
        std::sort(c.begin(), c.end());
        const double med = static_cast<double>(c[sms / 2]);
        const double ops = static_cast<double>(kPeakThreads) * trips * kUnroll * kChains * ops_per_instruction;
        best = std::max(best, ops / med);
    }
    return best;
}

}  // namespace

extern "C" {

int sysconv_measure_peaks(void *scratch_dev, long long scratch_bytes, double *results_host, int count)
{
    if (!scratch_dev || !results_host || count < SYSCONV_PEAK_COUNT) return SYSCONV_EINVAL;
    if (scratch_bytes < (64LL << 20) || (reinterpret_cast<unsigned long long>(scratch_dev) & 255ull) != 0) return SYSCONV_EINVAL;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SYSCONV_ECUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return SYSCONV_ECUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return SYSCONV_ECUDA;
    // the first bytes of the scratch buffer hold the per-SM cycle counts and the sink word
    unsigned long long *cycles = static_cast<unsigned long long *>(scratch_dev);
    float *sink = reinterpret_cast<float *>(cycles + 1024);
    if (sms > 1024) return SYSCONV_EUNSUPPORTED;
    results_host[SYSCONV_PEAK_FFMA] = measure_alu<kOpFfma>(cycles, sink, sms, 1);
    results_host[SYSCONV_PEAK_FFMA2] = measure_alu<kOpFfma2>(cycles, sink, sms, 2);
    results_host[SYSCONV_PEAK_IMAD] = measure_alu<kOpImad>(cycles, sink, sms, 1);
    results_host[SYSCONV_PEAK_DP4A] = measure_alu<kOpDp4a>(cycles, sink, sms, 1);
    results_host[SYSCONV_PEAK_SHFL] = measure_alu<kOpShfl>(cycles, sink, sms, 1);
    // streaming copy of half the scratch buffer into the other half, best of five
    const long long half = (scratch_bytes / 2) & ~255LL;
    const long long n16 = half / 16;
    const uint4 *src = static_cast<const uint4 *>(scratch_dev);
    uint4 *dst = reinterpret_cast<uint4 *>(static_cast<char *>(scratch_dev) + half);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return SYSCONV_ECUDA;
    double best_gbs = 0;
    for (int rep = 0; rep < 6; ++rep) {
        cudaEventRecord(e0, 0);
        stream_copy_kernel<<<static_cast<unsigned>((n16 + 1023) / 1024), 256>>>(src, dst, n16);
        cudaEventRecord(e1, 0);
        if (cudaEventSynchronize(e1) != cudaSuccess) return SYSCONV_ECUDA;
        float ms = 0;
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0) best_gbs = std::max(best_gbs, 2.0 * half / (ms * 1e-3) / 1e9);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    results_host[SYSCONV_PEAK_COPY_GBS] = best_gbs;
    results_host[SYSCONV_PEAK_SM_COUNT] = sms;
    for (int i = 0; i < SYSCONV_PEAK_COUNT; ++i)
        if (results_host[i] < 0) return SYSCONV_ECUDA;
    return cudaGetLastError() == cudaSuccess ? SYSCONV_OK : SYSCONV_ECUDA;
}

int sysconv_floor_copy(const void *src_dev, void *dst_dev, long long bytes_in, int widen, void *stream)
{
    if (!src_dev || !dst_dev || bytes_in < 1 || (widen != 0 && widen != 1)) return SYSCONV_EINVAL;
    const unsigned long long sa = reinterpret_cast<unsigned long long>(src_dev), da = reinterpret_cast<unsigned long long>(dst_dev);
    if ((sa & 15ull) != 0 || (da & 15ull) != 0 || (bytes_in & 15LL) != 0) return SYSCONV_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (widen) {
        const long long words = bytes_in / 4;
        const long long blocks = (words + 1023) / 1024;
        if (blocks > 0x7fffffffLL) return SYSCONV_EUNSUPPORTED;
        launch_kernel(stream_widen_kernel, static_cast<unsigned>(blocks), 256, s, static_cast<const unsigned *>(src_dev),
                      static_cast<int4 *>(dst_dev), words);
    } else {
        const long long n16 = bytes_in / 16;
        const long long blocks = (n16 + 1023) / 1024;
        if (blocks > 0x7fffffffLL) return SYSCONV_EUNSUPPORTED;
        launch_kernel(stream_copy_kernel, static_cast<unsigned>(blocks), 256, s, static_cast<const uint4 *>(src_dev),
                      static_cast<uint4 *>(dst_dev), n16);
    }
    return cudaGetLastError() == cudaSuccess ? SYSCONV_OK : SYSCONV_ECUDA;
}

}  // extern "C"
