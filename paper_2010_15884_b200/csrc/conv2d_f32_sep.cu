// Separable 2-D convolution, fp32, vertical and horizontal filters of 1..15 taps.
#include "conv2d_f32_sep.cuh"

namespace sysconv {

cudaError_t launch_conv2d_f32_separable(const Conv2DArgs &a, const float *u, int p, const float *v, int q, cudaStream_t s,
                                        int *launches)
{
    TapsSep taps;
    for (int k = 0; k < kMaxP2; ++k) taps.u[k] = k < p ? u[k] : 0.f;
    for (int k = 0; k < kMaxQ2; ++k) taps.v[k] = k < q ? v[k] : 0.f;
    cudaError_t err = kNoInstantiation;
    switch (p) {
#define SYSCONV_CASE(PP) case PP: err = launch_conv2d_sep_p<PP>(a, taps, q, s); break;
        SYSCONV_CASE(1) SYSCONV_CASE(2) SYSCONV_CASE(3) SYSCONV_CASE(4) SYSCONV_CASE(5)
        SYSCONV_CASE(6) SYSCONV_CASE(7) SYSCONV_CASE(8) SYSCONV_CASE(9) SYSCONV_CASE(10)
        SYSCONV_CASE(11) SYSCONV_CASE(12) SYSCONV_CASE(13) SYSCONV_CASE(14) SYSCONV_CASE(15)
#undef SYSCONV_CASE
        default: break;
    }
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
