// fp32 one-row filters of 16 to 32 taps on the 2-D output-stationary and input-stationary kernels: the form in which
// batches of SHORT signals with the longer 1-D filters run (an image with one signal per row; the 2-D entry points
// themselves stop at 15 filter columns).
#include "conv2d_f32_is_pair.cuh"

namespace sysconv {

static_assert(kMaxQ1 <= kMaxP2 * kMaxQ2 && kMaxQ1 + 1 <= kMaxP2 * (kMaxQ2 + 1), "a 32-tap row must fit the 2-D tap tables");

template <int DESIGN>
cudaError_t launch_rows(const Conv2DArgs &a, const Taps2D &taps, int q, cudaStream_t s)
{
    switch (q) {
#define SYSCONV_CASE(QQ) case QQ: return launch_conv2d_pq<F32Traits, DESIGN, 1, QQ>(a, taps, s);
        SYSCONV_CASE(16) SYSCONV_CASE(17) SYSCONV_CASE(18) SYSCONV_CASE(19) SYSCONV_CASE(20) SYSCONV_CASE(21)
        SYSCONV_CASE(22) SYSCONV_CASE(23) SYSCONV_CASE(24) SYSCONV_CASE(25) SYSCONV_CASE(26) SYSCONV_CASE(27)
        SYSCONV_CASE(28) SYSCONV_CASE(29) SYSCONV_CASE(30) SYSCONV_CASE(31) SYSCONV_CASE(32)
#undef SYSCONV_CASE
        default: return kNoInstantiation;
    }
}

// design: SYSCONV_OS or SYSCONV_IS; a.batch images of a.height rows (signals) each
cudaError_t launch_conv2d_f32_long_rows(int design, const Conv2DArgs &a, const float *w, int q, cudaStream_t s, int *launches)
{
    Taps2D taps;
    for (int k = 0; k < kMaxP2 * kMaxQ2; ++k) taps.w[k] = k < q ? w[k] : 0.f;
    const cudaError_t err = design == SYSCONV_OS ? launch_rows<SYSCONV_OS>(a, taps, q, s) : launch_rows<SYSCONV_IS>(a, taps, q, s);
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
