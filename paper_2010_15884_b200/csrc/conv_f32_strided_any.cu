// Strided convolution with ANY strides, output-stationary (FBS) design, fp32:
//
//   y(r, c) = sum_p sum_q x(sr*r + p, sc*c + q) * w(p, q)          (1-D: one row, P = 1)
//
// Table 2's stride-2 cell, X(c,q) = select(q < 2 || c == C-1, x(2c+q), X(c+1, q-2)), generalises to stride s as
// X(c,q) = select(q < s || c == C-1, x(s*c+q), X(c+1, q-s)): an input reaches PE c exactly s steps after PE c+1
// used it.  Taken residue class by residue class (q = s*a + b) that is s interleaved stride-ONE arrays: for every
// b < s the inputs x(s*c + b) enter the PEs once and move one PE down per step a, meeting the taps w(s*a + b),
// while the sums Z(c) stay in place and collect all classes (and, in 2-D, all filter rows).  This kernel runs
// exactly that: PE c keeps Z(c); lane l holds four consecutive PEs; per class the lane's four inputs come from
// memory, and every further step forwards them by one shuffle (the strip's last PE takes its input from memory,
// as the select says).  Strides, filter size and taps are run-time values: one kernel serves every stride; the
// fully unrolled stride-2 kernels (conv1d_f32_stride2.cuh, conv2d_f32_stride2.cuh) stay the fast path for what
// they cover.
#include "conv2d_kernels.cuh"

namespace sysconv {

namespace {

constexpr int kAnyR = 4;                        // PEs per lane
constexpr int kAnyStrip = kLanes * kAnyR;       // outputs per warp and output row

struct StridedAnyArgs {
    int p, q, sr, sc;
    int rows_per_block;                         // output rows per block (each warp takes every fourth... see kernel)
};

__global__ void __launch_bounds__(kThreads2)
conv_f32_strided_any_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const StridedAnyArgs g)
{
    dependent_launch_enter();
    const int lane = threadIdx.x & (kLanes - 1);
    const int warp = threadIdx.x / kLanes;
    const int c0 = blockIdx.x * kAnyStrip;                          // first output column (PE) of the strip
    const int col = c0 + kAnyR * lane;                              // first PE of this lane
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const int r_begin = blockIdx.y * g.rows_per_block;
    const int r_end = min(r_begin + g.rows_per_block, a.out_h);
    const int classes = min(g.sc, g.q);

    // the four warps of a block take the block's output rows in turn
    for (int r = r_begin + warp; r < r_end; r += kWarps2) {
        float Z[kAnyR] = {0.f, 0.f, 0.f, 0.f};
        for (int p = 0; p < g.p; ++p) {
            const float *xrow = xb + static_cast<long long>(g.sr * r + p) * a.x_pitch;
            const float *wrow = taps.w + p * g.q;
            for (int b = 0; b < classes; ++b) {
                // class b: inputs x(sc*c + b) enter the PEs from memory ...
                float X[kAnyR];
#pragma unroll
                for (int j = 0; j < kAnyR; ++j) {
                    const long long xi = static_cast<long long>(g.sc) * (col + j) + b;
                    X[j] = xi < a.width ? __ldg(xrow + xi) : 0.f;
                }
                const int steps = (g.q - b + g.sc - 1) / g.sc;      // taps w(sc*a + b), a < steps
                for (int s = 0; s < steps; ++s) {
                    const float wt = wrow[g.sc * s + b];
#pragma unroll
                    for (int j = 0; j < kAnyR; ++j) Z[j] = fmaf(X[j], wt, Z[j]);
                    if (s + 1 < steps) {
                        // ... and move one PE down per step; the strip's last PE takes its next input from memory
                        const float fwd = __shfl_down_sync(kFullMask, X[0], 1);
#pragma unroll
                        for (int j = 0; j < kAnyR - 1; ++j) X[j] = X[j + 1];
                        const long long xi = static_cast<long long>(g.sc) * (c0 + kAnyStrip + s) + b;
                        X[kAnyR - 1] = lane == kLanes - 1 ? (xi < a.width ? __ldg(xrow + xi) : 0.f) : fwd;
                    }
                }
            }
        }
        float *orow = yb + static_cast<long long>(r) * a.y_pitch;
#pragma unroll
        for (int j = 0; j < kAnyR; ++j)
            if (col + j < a.out_w) orow[col + j] = Z[j];
    }
}

}  // namespace

cudaError_t launch_conv_f32_strided_any(const Conv2DArgs &a, const float *w, int q, int p, int sc, int sr, cudaStream_t s,
                                        int *launches)
{
    if (p < 1 || q < 1 || p * q > kMaxP2 * kMaxQ2) return kNoInstantiation;
    Taps2D taps;
    for (int k = 0; k < kMaxP2 * kMaxQ2; ++k) taps.w[k] = k < p * q ? w[k] : 0.f;
    StridedAnyArgs g;
    g.p = p; g.q = q; g.sr = sr; g.sc = sc;
    const int strips = (a.out_w + kAnyStrip - 1) / kAnyStrip;
    // blocks of at most 32 output rows, and enough blocks to fill the machine when the image is small
    long long rows = 32;
    while (rows > kWarps2 && static_cast<long long>(strips) * a.batch * ((a.out_h + rows - 1) / rows) < 148LL * 8) rows /= 2;
    if ((a.out_h + rows - 1) / rows > 65535) rows = (a.out_h + 65534) / 65535;
    g.rows_per_block = static_cast<int>(rows);
    dim3 grid(strips, static_cast<unsigned>((a.out_h + rows - 1) / rows), a.batch);
    if (a.batch > 65535) return cudaErrorInvalidConfiguration;
    launch_kernel(conv_f32_strided_any_kernel, grid, kThreads2, s, a, taps, g);
    const cudaError_t err = cudaGetLastError();
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
