// 2-D uint8 x int8 -> int32 kernels of the weight-stationary (derived from BSM) design, filter heights 1..10 (all widths 1..15); the taller
// filters are compiled in conv2d_u8_ws_hi.cu so that the two halves build in parallel.
#include "conv2d_u8_ws_dp4a.cuh"

namespace sysconv {

cudaError_t launch_conv2d_u8_ws_hi(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches);

cudaError_t launch_conv2d_u8_ws(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches)
{
    if (p > 10) return launch_conv2d_u8_ws_hi(a, w, q, p, s, launches);
    return launch_conv2d_range<U8Traits, SYSCONV_WS, 1, 10>(a, w, q, p, s, launches);
}

}  // namespace sysconv
