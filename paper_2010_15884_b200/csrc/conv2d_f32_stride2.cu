// Stride-2 2-D convolution, fp32, filters up to 7 x 7: output-stationary and input-stationary arrays.
#include "conv2d_f32_stride2.cuh"

namespace sysconv {

cudaError_t launch_conv2d_f32_stride2(int design, const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s,
                                      int *launches)
{
    if (design == SYSCONV_OS) return launch_conv2d_s2<SYSCONV_OS>(a, w, q, p, s, launches);
    if (design == SYSCONV_IS) return launch_conv2d_s2<SYSCONV_IS>(a, w, q, p, s, launches);
    return kNoInstantiation;
}

}  // namespace sysconv
