// Shared declarations of the sysconv CUDA library (sm_100a).
//
// Vocabulary follows the paper: a processing element (PE) is one position of a
// linear systolic array; here R consecutive PEs are folded into one lane of a
// warp, PE registers are lane registers and the PE-to-PE transfer of one time
// step is one warp shuffle plus a static renaming of the lane's own registers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sysconv.h"

namespace sysconv {

constexpr int kLanes = 32;
constexpr unsigned kFullMask = 0xffffffffu;

// ---- 1-D geometry -----------------------------------------------------------
// One warp tile: 32 lanes x R1 PEs = 640 consecutive inputs.  The filter halo is
// budgeted at 32 elements whatever Q (Q <= 32, plus the drain steps of the
// input-stationary design), so every design yields 608 outputs per warp tile.
// R1 = 20 keeps the lane blocks 80 bytes apart, which makes the 128-bit shared
// memory reads and writes of a warp bank-conflict free (odd multiple of 16 B).
constexpr int kMaxQ1 = 32;
constexpr int R1 = 20;
constexpr int kWarpIn1 = kLanes * R1;          // 640
constexpr int kHalo1 = 32;
constexpr int kWarpOut1 = kWarpIn1 - kHalo1;   // 608
// weight-stationary arrays, 1-D: one array per lane, each streaming a 76-output segment
// (76 floats = 19 16-byte words: the lanes' 128-bit reads of their own segments fall in distinct banks)
constexpr int kWsSeg1 = 76;
// weight-stationary arrays, 2-D, integer data and small problems: eight four-lane arrays per warp
constexpr int kWsLanes = 4;
constexpr int kWsArrays = kLanes / kWsLanes;    // 8

struct Taps1D {
    float w[kMaxQ1];
};

// ---- 2-D geometry -----------------------------------------------------------
constexpr int kMaxP2 = 15;
constexpr int kMaxQ2 = 15;

struct Taps2D {
    float w[kMaxP2 * kMaxQ2];   // w[p * Q + q], only the first P*Q used
};

struct Taps2DInt {
    int w[kMaxP2 * kMaxQ2];     // sign-extended int8 taps, w[p * Q + q]
};

struct Conv1DArgs {
    const void *x;
    void *y;
    long long n;          // inputs per signal
    long long n_out;      // n - q + 1
    long long x_bstride;  // elements
    long long y_bstride;
    int batch;
};

struct Conv2DArgs {
    const void *x;
    void *y;
    int width, height;        // input image
    int out_w, out_h;         // width-q+1, height-p+1
    long long x_pitch, y_pitch;
    long long x_bstride, y_bstride;
    int batch;
};

// Launchers implemented in the per-design translation units.  Each returns a
// cudaError_t from the launch and adds the number of kernels it launched to
// *launches.
cudaError_t launch_conv1d_f32_os(const Conv1DArgs &a, const float *w, int q, unsigned *status_word, cudaStream_t s,
                                 int *launches);
cudaError_t launch_conv1d_f32_is(const Conv1DArgs &a, const float *w, int q, unsigned *status_word, cudaStream_t s,
                                 int *launches);
cudaError_t launch_conv1d_f32_ws(const Conv1DArgs &a, const float *w, int q, unsigned *status_word, cudaStream_t s,
                                 int *launches);
// the paper's other three designs (FSM, BFS, FFS): design = SYSCONV_FSM / SYSCONV_BFS / SYSCONV_FFS
cudaError_t launch_conv1d_f32_other(int design, const Conv1DArgs &a, const float *w, int q, unsigned *status_word,
                                    cudaStream_t s, int *launches);

// stride-2 forms (design = SYSCONV_OS or SYSCONV_IS); a.n_out / a.out_w, a.out_h are the strided output sizes
cudaError_t launch_conv1d_f32_stride2(int design, const Conv1DArgs &a, const float *w, int q, unsigned *status_word,
                                      cudaStream_t s, int *launches);
cudaError_t launch_conv2d_f32_stride2(int design, const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s,
                                      int *launches);

// separable 2-D convolution (conv2d_f32_sep.cu): u = p vertical taps, v = q horizontal taps
cudaError_t launch_conv2d_f32_separable(const Conv2DArgs &a, const float *u, int p, const float *v, int q, cudaStream_t s,
                                        int *launches);

// generic space-time executor (spacetime.cu): *status receives the planning result
int spacetime_describe(int pc, int pq, int sc, int sq, int q, int *out10, char *name4);
cudaError_t launch_spacetime_conv1d(const float *x, long long n, const float *w, int q, float *y, int pc, int pq, int sc,
                                    int sq, int sm_count, cudaStream_t s, int *status, int *launches);

cudaError_t launch_conv2d_f32_os(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches);
cudaError_t launch_conv2d_f32_is(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches);
cudaError_t launch_conv2d_f32_ws(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches);

cudaError_t launch_conv2d_u8_os(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches);
cudaError_t launch_conv2d_u8_is(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches);
cudaError_t launch_conv2d_u8_ws(const Conv2DArgs &a, const int8_t *w, int q, int p, cudaStream_t s, int *launches);

// Sentinel returned by a launcher for a filter size it has no instantiation for.
constexpr cudaError_t kNoInstantiation = cudaErrorInvalidKernelImage;

}  // namespace sysconv
