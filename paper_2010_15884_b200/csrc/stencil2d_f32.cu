// The iterated 3x3 stencil (second workload): dispatch over the number of sweeps fused in one launch.
#include "stencil2d_f32.cuh"

namespace sysconv {

cudaError_t launch_stencil2d_f32(const Conv2DArgs &a, const float *k9, int fused, cudaStream_t s, int *launches)
{
    StencilCoef coef;
    for (int i = 0; i < 9; ++i) coef.k[i] = k9[i];
    const bool five = k9[0] == 0.f && k9[2] == 0.f && k9[6] == 0.f && k9[8] == 0.f;
    cudaError_t err = kNoInstantiation;
    switch (fused) {
        case 1: err = launch_stencil2d_t<1>(a, coef, five, s); break;
        case 2: err = launch_stencil2d_t<2>(a, coef, five, s); break;
        case 3: err = launch_stencil2d_t<3>(a, coef, five, s); break;
        case 4: err = launch_stencil2d_t<4>(a, coef, five, s); break;
        default: break;
    }
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
