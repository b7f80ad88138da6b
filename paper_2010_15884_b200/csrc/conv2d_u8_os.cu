// 2-D uint8 x int8 -> int32 kernels of the output-stationary (FBS) design, all filter sizes 1..15 x 1..15.
#include "conv2d_u8_dp4a.cuh"

namespace sysconv {

// uint8 rows that start 16-byte aligned run on the packed (dp4a) kernel
template <int P, int Q>
struct FastPath2D<U8Traits, SYSCONV_OS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2DInt &taps, cudaStream_t s, cudaError_t *err)
    {
        if (!u8_dp4a_eligible(a)) return false;
        *err = launch_conv2d_u8_os_dp4a<P, Q>(a, taps, s);
        return true;
    }
};

cudaError_t launch_conv2d_u8_os(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches)
{
    return launch_conv2d_range<U8Traits, SYSCONV_OS, 1, kMaxP2>(a, w, q, p, s, launches);
}

}  // namespace sysconv
