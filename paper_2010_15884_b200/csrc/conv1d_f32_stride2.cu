// Stride-2 1-D convolution, fp32: output-stationary (FBS, Table 2 cell 6) and input-stationary arrays.
#include "conv1d_f32_stride2.cuh"

namespace sysconv {

cudaError_t launch_conv1d_f32_stride2(int design, const Conv1DArgs &a, const float *w, int q, unsigned *status_word,
                                      cudaStream_t s, int *launches)
{
    if (design == SYSCONV_OS) return launch_conv1d_f32_s2<SYSCONV_OS>(a, w, q, status_word, s, launches);
    if (design == SYSCONV_IS) return launch_conv1d_f32_s2<SYSCONV_IS>(a, w, q, status_word, s, launches);
    return kNoInstantiation;
}

}  // namespace sysconv
