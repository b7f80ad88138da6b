// Many independent tiny 1-D convolutions, all six designs (see conv1d_f32_tiles.cuh).
#include "conv1d_f32_tiles.cuh"

namespace sysconv {

bool conv1d_tiles_eligible(const Conv1DArgs &a, int design, int q) { return tiles_eligible(a, design, q); }

cudaError_t launch_conv1d_f32_tiles(int design, const Conv1DArgs &a, const float *w, int q, cudaStream_t s, int *launches)
{
    Taps1D taps;
    for (int k = 0; k < kMaxQ1; ++k) taps.w[k] = k < q ? w[k] : 0.f;
    cudaError_t err = kNoInstantiation;
    switch (design) {
        case SYSCONV_WS: err = launch_conv1d_tiles_design<SYSCONV_WS>(a, taps, q, s); break;
        case SYSCONV_OS: err = launch_conv1d_tiles_design<SYSCONV_OS>(a, taps, q, s); break;
        case SYSCONV_IS: err = launch_conv1d_tiles_design<SYSCONV_IS>(a, taps, q, s); break;
        case SYSCONV_FSM: err = launch_conv1d_tiles_design<SYSCONV_FSM>(a, taps, q, s); break;
        case SYSCONV_BFS: err = launch_conv1d_tiles_design<SYSCONV_BFS>(a, taps, q, s); break;
        case SYSCONV_FFS: err = launch_conv1d_tiles_design<SYSCONV_FFS>(a, taps, q, s); break;
        default: break;
    }
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
