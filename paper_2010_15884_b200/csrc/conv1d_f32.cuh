// 1-D fp32 convolution (Eq. 2) as folded linear systolic arrays on a warp.
//
// One CTA handles one tile of kTileOut1 outputs: it stages the kTileIn1 inputs
// the tile needs in shared memory, each of its 8 warps runs one systolic array
// pass over its 640-input slice (608 outputs), the outputs are collected in
// shared memory and leave with coalesced 128-bit stores.
//
// Lane l of a warp holds the R1 = 20 consecutive PEs l*20 .. l*20+19.  A time
// step is R1 fused multiply-adds per lane, one shuffle (the value that crosses
// the lane boundary) and a renaming of the lane's own registers (the loops over
// time are fully unrolled, so "PE j takes PE j-1's value" costs nothing).
// Every PE runs at every step (no CheckTime); PEs whose sums are incomplete are
// not drained.
#pragma once

#include "sysconv_common.cuh"

namespace sysconv {

// ---- tile staging -----------------------------------------------------------

// Copy x[t0 .. t0 + kTileIn1) to shared memory, zeros beyond the signal's end.
__device__ __forceinline__ void stage_in_1d(const float *__restrict__ xg, long long n, long long t0,
                                            float *s_in)
{
    const bool vec_ok = (reinterpret_cast<uintptr_t>(xg) & 15) == 0;   // t0 is a multiple of 4
    if (vec_ok) {
        constexpr int kVec = kTileIn1 / 4;
        constexpr int kIter = (kVec + kThreads1 - 1) / kThreads1;
        float4 v[kIter];
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
            const int i = threadIdx.x + it * kThreads1;
            const long long g = t0 + 4LL * i;
            v[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < kVec) {
                if (g + 3 < n) {
                    v[it] = __ldg(reinterpret_cast<const float4 *>(xg + g));
                } else {
                    if (g < n) v[it].x = xg[g];
                    if (g + 1 < n) v[it].y = xg[g + 1];
                    if (g + 2 < n) v[it].z = xg[g + 2];
                }
            }
        }
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
            const int i = threadIdx.x + it * kThreads1;
            if (i < kVec) reinterpret_cast<float4 *>(s_in)[i] = v[it];
        }
    } else {
        for (int i = threadIdx.x; i < kTileIn1; i += kThreads1) {
            const long long g = t0 + i;
            s_in[i] = g < n ? xg[g] : 0.f;
        }
    }
}

// Copy the tile's outputs from shared memory to y[t0 .. min(t0 + kTileOut1, n_out)).
__device__ __forceinline__ void stage_out_1d(float *__restrict__ yg, long long n_out, long long t0,
                                             const float *s_out)
{
    const bool vec_ok = (reinterpret_cast<uintptr_t>(yg) & 15) == 0;
    if (vec_ok) {
        constexpr int kVec = kTileOut1 / 4;
        for (int i = threadIdx.x; i < kVec; i += kThreads1) {
            const long long g = t0 + 4LL * i;
            const float4 v = reinterpret_cast<const float4 *>(s_out)[i];
            if (g + 3 < n_out) {
                *reinterpret_cast<float4 *>(yg + g) = v;
            } else {
                if (g < n_out) yg[g] = v.x;
                if (g + 1 < n_out) yg[g + 1] = v.y;
                if (g + 2 < n_out) yg[g + 2] = v.z;
            }
        }
    } else {
        for (int i = threadIdx.x; i < kTileOut1; i += kThreads1) {
            const long long g = t0 + i;
            if (g < n_out) yg[g] = s_out[i];
        }
    }
}

__device__ __forceinline__ void load_lane_block(const float *p, float (&v)[R1])
{
#pragma unroll
    for (int g = 0; g < R1 / 4; ++g) {
        const float4 t = reinterpret_cast<const float4 *>(p)[g];
        v[4 * g] = t.x; v[4 * g + 1] = t.y; v[4 * g + 2] = t.z; v[4 * g + 3] = t.w;
    }
}

// ---- output-stationary (FBS, Table 2): PE c keeps Z(c); at step t = q the
// inputs move one PE down:  X_c <- X_{c+1},  Z_c += X_c * w(q). --------------
template <int Q>
__device__ __forceinline__ void os_pass_1d(const float *sx, float *so, const Taps1D &taps, int lane)
{
    float X[R1], Z[R1];
    load_lane_block(sx + lane * R1, X);
#pragma unroll
    for (int t = 0; t < Q; ++t) {
        const float wt = taps.w[t];
#pragma unroll
        for (int j = 0; j < R1; ++j) Z[j] = (t == 0) ? X[j] * wt : fmaf(X[j], wt, Z[j]);
        if (t < Q - 1) {
            const float in = __shfl_down_sync(kFullMask, X[0], 1);   // lane 31 keeps its own: invalid PEs
#pragma unroll
            for (int j = 0; j < R1 - 1; ++j) X[j] = X[j + 1];
            X[R1 - 1] = in;
        }
    }
    // PE c holds y(c); PEs beyond 640-(Q-1) are incomplete and lie outside the 608 drained
#pragma unroll
    for (int g = 0; g < R1 / 4; ++g) {
        const int off = lane * R1 + 4 * g;
        if (off < kWarpOut1)
            *reinterpret_cast<float4 *>(so + off) = make_float4(Z[4 * g], Z[4 * g + 1], Z[4 * g + 2], Z[4 * g + 3]);
    }
}

// ---- input-stationary (SBM, Section 3.1): PE s keeps x(s); at step t = q the
// partial sums move one PE up:  Z_s <- Z_{s-1} + X_s * w(q).  After Q steps PE s
// holds y(s-(Q-1)); up to three more moves without arithmetic (drain) bring the
// offset to a multiple of four so that the sums leave as aligned 128-bit words.
template <int Q>
__device__ __forceinline__ void is_pass_1d(const float *sx, float *so, const Taps1D &taps, int lane)
{
    constexpr int kDrain = (4 - ((Q - 1) & 3)) & 3;
    constexpr int kShift = Q - 1 + kDrain;      // <= 32 = kHalo1
    float X[R1], Z[R1];
    load_lane_block(sx + lane * R1, X);
#pragma unroll
    for (int j = 0; j < R1; ++j) Z[j] = X[j] * taps.w[0];
#pragma unroll
    for (int t = 1; t < Q + kDrain; ++t) {
        const float up = __shfl_up_sync(kFullMask, Z[R1 - 1], 1);    // lane 0 keeps its own: invalid PEs
        if (t < Q) {
            const float wt = taps.w[t];
#pragma unroll
            for (int j = R1 - 1; j > 0; --j) Z[j] = fmaf(X[j], wt, Z[j - 1]);
            Z[0] = fmaf(X[0], wt, up);
        } else {
#pragma unroll
            for (int j = R1 - 1; j > 0; --j) Z[j] = Z[j - 1];
            Z[0] = up;
        }
    }
#pragma unroll
    for (int g = 0; g < R1 / 4; ++g) {
        const int off = lane * R1 + 4 * g - kShift;
        if (off >= 0 && off < kWarpOut1)
            *reinterpret_cast<float4 *>(so + off) = make_float4(Z[4 * g], Z[4 * g + 1], Z[4 * g + 2], Z[4 * g + 3]);
    }
}

// ---- weight-stationary (BSM, Table 2): PE s keeps w(s); at step t the input
// x(t) is broadcast to the array, Z_s <- Z_{s-1} + x(t) * w(s), PE 0 starts a new
// sum and the last PE emits y(t-(Q-1)).  An array has only Q PEs, so a warp holds
// eight arrays of four lanes (RW = ceil(Q/4) PEs per lane, unused PEs keep a zero
// tap); array a streams the 76-output segment a of the warp tile.
template <int Q>
__device__ __forceinline__ void ws_pass_1d(const float *sx, float *so, const Taps1D &taps, int lane)
{
    constexpr int RW = (Q + kWsLanes - 1) / kWsLanes;
    constexpr int QP = RW * kWsLanes;
    constexpr int kGroups = (kWsSeg1 + QP) / 4;       // time steps in groups of four
    const int m = lane & (kWsLanes - 1);
    const int arr = lane / kWsLanes;
    float Wr[RW], Z[RW];
#pragma unroll
    for (int i = 0; i < RW; ++i) {
        const int s = m * RW + i;
        Wr[i] = s < Q ? taps.w[s] : 0.f;
        Z[i] = 0.f;
    }
    const float4 *xs4 = reinterpret_cast<const float4 *>(sx + arr * kWsSeg1);
    float *yo = so + arr * kWsSeg1;

    auto step = [&](float xb) -> float {
        float up = __shfl_up_sync(kFullMask, Z[RW - 1], 1, kWsLanes);
        if (m == 0) up = 0.f;                          // PE 0: Z starts at zero
#pragma unroll
        for (int i = RW - 1; i > 0; --i) Z[i] = fmaf(xb, Wr[i], Z[i - 1]);
        Z[0] = fmaf(xb, Wr[0], up);
        return Z[RW - 1];                              // on the array's last lane: y(t-(QP-1))
    };

    float o0 = 0.f;
#pragma unroll 2
    for (int k = 0; k < kGroups; ++k) {
        const float4 xv = xs4[k];                      // x(4k .. 4k+3) of this array's stream
        const float o1 = step(xv.x);
        const float o2 = step(xv.y);
        const float o3 = step(xv.z);
        const int off = 4 * k - QP;                    // outputs 4k-QP .. 4k-QP+3 are now complete
        if (m == kWsLanes - 1 && off >= 0 && off < kWsSeg1)
            *reinterpret_cast<float4 *>(yo + off) = make_float4(o0, o1, o2, o3);
        o0 = step(xv.w);
    }
}

template <int DESIGN, int Q>
__global__ void __launch_bounds__(kThreads1)
conv1d_f32_kernel(const Conv1DArgs a, const __grid_constant__ Taps1D taps)
{
    __shared__ __align__(16) float s_in[kTileIn1];
    __shared__ __align__(16) float s_out[kTileOut1];
    const int lane = threadIdx.x & (kLanes - 1);
    const int warp = threadIdx.x / kLanes;
    const long long t0 = static_cast<long long>(blockIdx.x) * kTileOut1;

    for (int b = blockIdx.y; b < a.batch; b += gridDim.y) {
        const float *xg = static_cast<const float *>(a.x) + b * a.x_bstride;
        float *yg = static_cast<float *>(a.y) + b * a.y_bstride;
        stage_in_1d(xg, a.n, t0, s_in);
        __syncthreads();
        const float *sx = s_in + warp * kWarpOut1;
        float *so = s_out + warp * kWarpOut1;
        if (DESIGN == SYSCONV_OS) os_pass_1d<Q>(sx, so, taps, lane);
        else if (DESIGN == SYSCONV_IS) is_pass_1d<Q>(sx, so, taps, lane);
        else ws_pass_1d<Q>(sx, so, taps, lane);
        __syncthreads();
        stage_out_1d(yg, a.n_out, t0, s_out);
        // the next batch iteration's stage_in writes s_in only; s_out is rewritten
        // after its __syncthreads, when every thread has finished stage_out
    }
}

template <int DESIGN, int Q>
cudaError_t launch_conv1d_f32_q(const Conv1DArgs &a, const Taps1D &taps, cudaStream_t s)
{
    const long long tiles = (a.n_out + kTileOut1 - 1) / kTileOut1;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(tiles), static_cast<unsigned>(a.batch < 65535 ? a.batch : 65535));
    conv1d_f32_kernel<DESIGN, Q><<<grid, kThreads1, 0, s>>>(a, taps);
    return cudaGetLastError();
}

template <int DESIGN>
cudaError_t launch_conv1d_f32(const Conv1DArgs &a, const float *w, int q, cudaStream_t s, int *launches)
{
    Taps1D taps;
    for (int k = 0; k < kMaxQ1; ++k) taps.w[k] = k < q ? w[k] : 0.f;
    cudaError_t err = kNoInstantiation;
    switch (q) {
#define SYSCONV_CASE(QQ) case QQ: err = launch_conv1d_f32_q<DESIGN, QQ>(a, taps, s); break;
        SYSCONV_CASE(1) SYSCONV_CASE(2) SYSCONV_CASE(3) SYSCONV_CASE(4) SYSCONV_CASE(5) SYSCONV_CASE(6)
        SYSCONV_CASE(7) SYSCONV_CASE(8) SYSCONV_CASE(9) SYSCONV_CASE(10) SYSCONV_CASE(11) SYSCONV_CASE(12)
        SYSCONV_CASE(13) SYSCONV_CASE(14) SYSCONV_CASE(15) SYSCONV_CASE(16) SYSCONV_CASE(17) SYSCONV_CASE(18)
        SYSCONV_CASE(19) SYSCONV_CASE(20) SYSCONV_CASE(21) SYSCONV_CASE(22) SYSCONV_CASE(23) SYSCONV_CASE(24)
        SYSCONV_CASE(25) SYSCONV_CASE(26) SYSCONV_CASE(27) SYSCONV_CASE(28) SYSCONV_CASE(29) SYSCONV_CASE(30)
        SYSCONV_CASE(31) SYSCONV_CASE(32)
#undef SYSCONV_CASE
        default: break;
    }
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
