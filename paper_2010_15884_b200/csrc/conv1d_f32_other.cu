// 1-D fp32 kernels of the paper's other three designs (FSM, BFS, FFS of Table 2), all filter lengths 1..32.
#include "conv1d_f32.cuh"

namespace sysconv {

cudaError_t launch_conv1d_f32_other(int design, const Conv1DArgs &a, const float *w, int q, unsigned *status_word,
                                    cudaStream_t s, int *launches)
{
    switch (design) {
        case SYSCONV_FSM: return launch_conv1d_f32<SYSCONV_FSM>(a, w, q, status_word, s, launches);
        case SYSCONV_BFS: return launch_conv1d_f32<SYSCONV_BFS>(a, w, q, status_word, s, launches);
        case SYSCONV_FFS: return launch_conv1d_f32<SYSCONV_FFS>(a, w, q, status_word, s, launches);
        default: return kNoInstantiation;
    }
}

}  // namespace sysconv
