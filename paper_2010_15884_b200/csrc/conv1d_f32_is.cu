// 1-D fp32 kernels of the input-stationary (SBM) design, all filter lengths 1..32.
#include "conv1d_f32.cuh"

namespace sysconv {

cudaError_t launch_conv1d_f32_is(const Conv1DArgs &a, const float *w, int q, unsigned *status_word, cudaStream_t s,
                                 int *launches)
{
    return launch_conv1d_f32<SYSCONV_IS>(a, w, q, status_word, s, launches);
}

}  // namespace sysconv
