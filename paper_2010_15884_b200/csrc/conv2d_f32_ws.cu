// 2-D fp32 kernels of the weight-stationary (derived from BSM) design, all filter sizes 1..15 x 1..15.
#include "conv2d_f32_ws_lane.cuh"

namespace sysconv {

// fp32 runs the one-lane-per-array paired kernel; the four-lane arrays of conv2d_ws_kernel serve the integer
// data and the images too small to give the one-warp CTAs of the paired kernel a few warps per SM
// (1920 x 1080, 5 x 5: 25 us against 36 us)
template <int P, int Q>
struct FastPath2D<F32Traits, SYSCONV_WS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s, cudaError_t *err)
    {
        const long long bands = (a.out_h + kWlRows - 1) / kWlRows;
        const long long max_segs = (a.out_w + 127) / 128;
        if (bands * max_segs * a.batch < 148LL * 4) return false;
        *err = launch_conv2d_ws_lane<P, Q>(a, taps, s);
        return true;
    }
};

cudaError_t launch_conv2d_f32_ws(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches)
{
    return launch_conv2d_range<F32Traits, SYSCONV_WS, 1, kMaxP2>(a, w, q, p, s, launches);
}

}  // namespace sysconv
