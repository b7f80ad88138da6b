// 2-D fp32 kernels of the input-stationary (SBM) design, all filter sizes 1..15 x 1..15.
#include "conv2d_f32_is_pair.cuh"

namespace sysconv {

// the larger filters (more than 25 taps, at least three columns) run the paired packed-FMA kernel
template <int P, int Q>
struct FastPath2D<F32Traits, SYSCONV_IS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s, cudaError_t *err)
    {
        if constexpr (P * Q > 25 && Q >= 3) {
            *err = launch_conv2d_is_pair<P, Q>(a, taps, s);
            return true;
        } else {
            return false;
        }
    }
};

cudaError_t launch_conv2d_f32_is(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches)
{
    return launch_conv2d_range<F32Traits, SYSCONV_IS, 1, kMaxP2>(a, w, q, p, s, launches);
}

}  // namespace sysconv
