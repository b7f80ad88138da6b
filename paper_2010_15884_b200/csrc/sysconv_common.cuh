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
constexpr int kShortSignal1 = 512;              // batches of signals with at most this many outputs run as images, one signal per row
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

// batches of tiny signals (at most 32 outputs, at most 8 taps): small unfolded arrays side by side in a warp, all six designs
bool conv1d_tiles_eligible(const Conv1DArgs &a, int design, int q);
cudaError_t launch_conv1d_f32_tiles(int design, const Conv1DArgs &a, const float *w, int q, cudaStream_t s, int *launches);

// stride-2 forms (design = SYSCONV_OS or SYSCONV_IS); a.n_out / a.out_w, a.out_h are the strided output sizes
cudaError_t launch_conv1d_f32_stride2(int design, const Conv1DArgs &a, const float *w, int q, unsigned *status_word,
                                      cudaStream_t s, int *launches);
cudaError_t launch_conv2d_f32_stride2(int design, const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s,
                                      int *launches);

// any strides, output-stationary design, fp32, up to 225 taps (conv_f32_strided_any.cu); 1-D = one row, p = 1
cudaError_t launch_conv_f32_strided_any(const Conv2DArgs &a, const float *w, int q, int p, int sc, int sr, cudaStream_t s,
                                        int *launches);

// separable 2-D convolution (conv2d_f32_sep.cu): u = p vertical taps, v = q horizontal taps
cudaError_t launch_conv2d_f32_separable(const Conv2DArgs &a, const float *u, int p, const float *v, int q, cudaStream_t s,
                                        int *launches);

// iterated 3x3 stencil (stencil2d_f32.cu): `fused` sweeps (1..4) in one launch; a.out_w/out_h unused (output = grid size)
cudaError_t launch_conv2d_f32_long_rows(int design, const Conv2DArgs &a, const float *w, int q, cudaStream_t s, int *launches);
cudaError_t launch_stencil2d_f32(const Conv2DArgs &a, const float *k9, int fused, cudaStream_t s, int *launches);

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

// ---- programmatic dependent launch ---------------------------------------------------------------
// Every kernel of the library is launched with the "programmatic stream serialization" attribute and
// starts with dependent_launch_enter(), which waits until the PREVIOUS kernel of the stream has completed
// and its memory is visible (griddepcontrol.wait) before anything touches global memory.  Stream order is
// unchanged; the attribute lets the hardware set up this kernel while the one before it drains, instead of
// after it has signalled completion, which matters for the small, launch-bound problems (measured back to
// back on B200: 1920x1080 fp32 5x5 10.3 -> 8.3 us per launch, 3840x2160 uint8 3x3 12.3 -> 10.5 us).
// No kernel triggers its dependents early (griddepcontrol.launch_dependents): with several kernels queued
// that made the blocks of later kernels resident and waiting beside the running one and cost the
// issue-bound kernels up to 20 %.
__device__ __forceinline__ void dependent_launch_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

bool dependent_launch_enabled();       // false if SYSCONV_NO_PDL is set in the environment (sysconv_api.cu)

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t s, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent_launch_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Blocks of `threads` threads of this kernel that one SM holds at a time (asked of the runtime once per kernel).
template <typename... KArgs>
int resident_blocks_per_sm(void (*kern)(KArgs...), int threads)
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, threads, 0) != cudaSuccess || n < 1) n = 1;
    return n;
}

// Band height (output rows per block) for a 2-D problem SMALL enough that the whole grid is a few waves of blocks.
// There the time is set by the number of waves times the time of one block, and a block's time grows with the
// rows it marches through: its band, the P-1 rows of the window above it, and a fixed start-up worth about
// eight rows (measured on B200: a full-HD 5x5 pass takes 4.4 us + 0.4 us per band row).  The height that
// minimises waves x (band + P - 1 + 8) is taken; a grid that just spills into a second wave costs almost double,
// which the fixed "so many blocks per SM" rules missed (3840x2160 uint8 7x7: 616 blocks on 592 slots, 24.6 us;
// 540 blocks, 16.9 us).  per_band = blocks per band (column tiles x images), slots = blocks resident at once.
inline int pick_band_height_small(int out_h, long long per_band, int p, int lo, int hi, long long slots)
{
    int best = lo;
    double best_cost = 1e300;
    for (int h = lo; h <= hi; ++h) {
        const long long bands = (out_h + h - 1) / h;
        if (bands > 65535) continue;
        const long long waves = (per_band * bands + slots - 1) / slots;
        const double cost = static_cast<double>(waves) * (h + p - 1 + 8);
        if (cost < best_cost) {
            best_cost = cost;
            best = h;
        }
        if (bands == 1) break;
    }
    return best;
}

// true if a problem is "small" in the sense above: even with bands of `lo` rows it is at most four waves of blocks
inline bool small_problem(int out_h, long long per_band, int lo, long long slots)
{
    return per_band * ((out_h + lo - 1) / lo) <= 4 * slots;
}

// Warps per block of the 2-D kernels whose warps take neighbouring column strips: `full` of them, fewer when the image
// has fewer strips -- the spare warps of a block would return at once and leave their share of the SM idle (narrow
// images; batches of short signals, which arrive as images of a few dozen to a few hundred columns).  Such a block is
// the only one of its row of the grid, so the kernels keep computing strip = blockIdx.x * full + warp.
inline int block_warps(long long strips, int full)
{
    return strips >= full ? full : (strips < 1 ? 1 : static_cast<int>(strips));
}

// Sentinel returned by a launcher for a filter size it has no instantiation for.
constexpr cudaError_t kNoInstantiation = cudaErrorInvalidKernelImage;

}  // namespace sysconv
