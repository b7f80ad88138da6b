// 2-D uint8 x int8 -> int32 kernels of the input-stationary (SBM) design, filter heights 11..15 (all widths 1..15).
#include "conv2d_u8_dp4a.cuh"

namespace sysconv {

cudaError_t launch_conv2d_u8_is_hi(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches)
{
    return launch_conv2d_range<U8Traits, SYSCONV_IS, 11, kMaxP2>(a, w, q, p, s, launches);
}

}  // namespace sysconv
