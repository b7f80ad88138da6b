// 2-D fp32 kernels of the output-stationary (FBS) design, filter heights 1..10 (all widths 1..15); the taller
// filters are compiled in conv2d_f32_os_hi.cu so that the two halves build in parallel.
#include "conv2d_kernels.cuh"

namespace sysconv {

cudaError_t launch_conv2d_f32_os_hi(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches);

cudaError_t launch_conv2d_f32_os(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches)
{
    if (p > 10) return launch_conv2d_f32_os_hi(a, w, q, p, s, launches);
    return launch_conv2d_range<F32Traits, SYSCONV_OS, 1, 10>(a, w, q, p, s, launches);
}

}  // namespace sysconv
