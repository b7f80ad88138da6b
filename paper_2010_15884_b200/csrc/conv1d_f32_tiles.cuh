// Many independent TINY 1-D convolutions (the shape of the paper's own experiment, Section 6: millions of
// threads, each computing one convolution with 16 outputs and a filter of 2 or 5 taps), for all six designs
// of Section 3.1 / Table 2.
//
// The folded kernels of conv1d_f32.cuh give a warp 608 or more consecutive outputs of ONE signal; a signal with
// 16 outputs would leave 97 % of such an array idle.  Here the arrays are as small as the paper's, unfolded (one
// PE per lane), and a warp holds as many of them side by side as fit its 32 lanes:
//
//   SBM (input-stationary)   PE = c+q   C+Q-1 PEs per array   floor(32 / (C+Q-1)) arrays per warp   Q steps
//   FBS (output-stationary)  PE = c     C PEs                 floor(32 / C)                         Q steps
//   BFS                      PE = c     C PEs                 floor(32 / C)                         C+Q-1 steps
//   FFS                      PE = c     C PEs                 floor(32 / C)                         2(C-1)+Q steps
//   BSM (weight-stationary)  PE = q     Q PEs                 floor(32 / Q)                         C+Q-1 steps
//   FSM                      PE = q     Q PEs                 floor(32 / Q)                         C+Q-1 steps
//
// (C = outputs of a signal.)  These are the PE counts and step counts of the paper's analytical model (Table 4),
// so the measured outputs per second can be read against its outturn and lane utilisation.  The arrays need
// no guard between them: the selects of each design's own recurrences (the first PE starts a sum at zero, the
// last PE takes its input from memory) cut every chain at the array's edge.
//
// Every lane serves U arrays (the same PE of U different signals) per pass, so that U independent chains overlap
// in the pipelines.  The signals of a pass are staged in shared memory ("memory" of the recurrences = this staging
// area) and the outputs go back the same way.  Densely packed signals (the usual case: signal g starts right after
// signal g-1, 16-byte aligned) make one contiguous run per pass, which moves as whole 128-bit words, and the
// words of the NEXT pass are fetched into registers before the current pass is computed, so that the memory
// latency is overlapped with the arithmetic of the same warp.  Any other layout is gathered signal by signal by
// the lanes of each array.
#pragma once

#include "sysconv_common.cuh"

namespace sysconv {

constexpr int kTilesMaxQ = 8;           // filter lengths 1 .. 8
constexpr int kTilesMaxOut = 32;        // outputs per signal 1 .. 32
constexpr int kTilesWarps = 4;
constexpr int kTilesFloatsPerWarp = 2560;   // staging area of one warp (inputs + outputs of a pass)
constexpr int kTilesVecPerLane = 6;         // dense form: 128-bit words of a pass's inputs per lane (at most 768 floats per pass)

// PEs of one array of a design for C outputs and Q taps
inline int tiles_array_pes(int design, int c, int q)
{
    switch (design) {
        case SYSCONV_IS: return c + q - 1;
        case SYSCONV_WS:
        case SYSCONV_FSM: return q;
        default: return c;              // FBS, BFS, FFS
    }
}

template <int DESIGN, int Q, int U, bool DENSE>
__global__ void __launch_bounds__(kTilesWarps *kLanes)
conv1d_tiles_kernel(const Conv1DArgs a, const __grid_constant__ Taps1D taps, const int LA, const int AW, const int warp_floats)
{
    dependent_launch_enter();
    extern __shared__ __align__(16) float tiles_smem[];
    const int C = static_cast<int>(a.n_out), N = static_cast<int>(a.n);     // outputs and inputs of one signal
    const int lane = threadIdx.x & (kLanes - 1);
    const int warp = threadIdx.x / kLanes;
    const int arr = lane / LA;                  // array this lane belongs to (>= AW: the lane idles)
    const int pe = lane - arr * LA;             // its PE in that array
    const bool member = arr < AW;
    float *s_in = tiles_smem + warp * warp_floats;
    float *s_out = s_in + U * AW * N;
    const float *xg = static_cast<const float *>(a.x);
    float *yg = static_cast<float *>(a.y);
    const long long per_pass = static_cast<long long>(U) * AW;              // signals one warp takes per pass
    const long long stride = static_cast<long long>(gridDim.x) * kTilesWarps * per_pass;
    const int in_vec = U * AW * N / 4, out_vec = U * AW * C / 4;            // dense form: 128-bit words per pass

    // dense form: the inputs of a whole pass are one contiguous, 16-byte aligned run
    float4 pre[kTilesVecPerLane];
    auto fetch = [&](long long g) {
        const float4 *src = reinterpret_cast<const float4 *>(xg + g * N);
#pragma unroll
        for (int i = 0; i < kTilesVecPerLane; ++i)
            if (lane + kLanes * i < in_vec) pre[i] = __ldg(src + lane + kLanes * i);
    };
    long long g0 = (static_cast<long long>(blockIdx.x) * kTilesWarps + warp) * per_pass;
    bool have = DENSE && g0 + per_pass <= a.batch;      // a whole pass: its words are in flight or in registers
    if (have) fetch(g0);

    for (; g0 < a.batch; g0 += stride) {
        // ---- the signals of this pass enter the staging area
        if (DENSE && have) {
#pragma unroll
            for (int i = 0; i < kTilesVecPerLane; ++i)
                if (lane + kLanes * i < in_vec) reinterpret_cast<float4 *>(s_in)[lane + kLanes * i] = pre[i];
        } else if (member) {
            // each signal fetched by the lanes of its own array
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long g = g0 + u * AW + arr;
                if (g < a.batch)
                    for (int k = pe; k < N; k += LA) s_in[(u * AW + arr) * N + k] = __ldg(xg + g * a.x_bstride + k);
            }
        }
        bool have_next = false;
        if (DENSE) {
            have_next = g0 + stride + per_pass <= a.batch;
            if (have_next) fetch(g0 + stride);          // in flight while this pass is computed
        }
        __syncwarp();
        // signal u of this lane's array: inputs xin0[u * xu + k], outputs yout0[u * yu + k]
        const float *xin0 = s_in + (member ? arr : 0) * N;
        float *yout0 = s_out + (member ? arr : 0) * C;
        const int xu = AW * N, yu = AW * C;

        if (DESIGN == SYSCONV_OS) {
            // FBS: PE c keeps Z(c); inputs move one PE down per step, the last PE takes x(c+q) from memory
            float X[U], Z[U];
#pragma unroll
            for (int u = 0; u < U; ++u) X[u] = pe < C ? xin0[u * xu + pe] : 0.f;
#pragma unroll
            for (int t = 0; t < Q; ++t) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (t > 0) {
                        const float fwd = __shfl_down_sync(kFullMask, X[u], 1);
                        X[u] = (pe == C - 1) ? xin0[u * xu + pe + t] : fwd;
                    }
                    Z[u] = t == 0 ? X[u] * taps.w[0] : fmaf(X[u], taps.w[t], Z[u]);
                }
            }
            if (member && pe < C) {
#pragma unroll
                for (int u = 0; u < U; ++u) yout0[u * yu + pe] = Z[u];
            }
        } else if (DESIGN == SYSCONV_IS) {
            // SBM: PE s keeps x(s); the sums move one PE up per step; PE s >= Q-1 ends with y(s-(Q-1))
            float X[U], Z[U];
#pragma unroll
            for (int u = 0; u < U; ++u) X[u] = pe < N ? xin0[u * xu + pe] : 0.f;
#pragma unroll
            for (int t = 0; t < Q; ++t) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (t == 0) {
                        Z[u] = X[u] * taps.w[0];
                    } else {
                        const float up = __shfl_up_sync(kFullMask, Z[u], 1);
                        Z[u] = fmaf(X[u], taps.w[t], up);
                    }
                }
            }
            if (member && pe >= Q - 1 && pe < N) {
#pragma unroll
                for (int u = 0; u < U; ++u) yout0[u * yu + pe - (Q - 1)] = Z[u];
            }
        } else if (DESIGN == SYSCONV_WS) {
            // BSM: PE s keeps w(s); x(t) is broadcast to the array; the sums move one PE up; the last PE emits
            const float w = pe < Q ? taps.w[pe] : 0.f;
            float Z[U];
#pragma unroll
            for (int u = 0; u < U; ++u) Z[u] = 0.f;
            for (int t = 0; t < N; ++t) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float up = __shfl_up_sync(kFullMask, Z[u], 1);
                    Z[u] = fmaf(xin0[u * xu + t], w, pe == 0 ? 0.f : up);
                    if (member && pe == Q - 1 && t >= Q - 1) yout0[u * yu + t - (Q - 1)] = Z[u];
                }
            }
        } else if (DESIGN == SYSCONV_FSM) {
            // FSM: PE q keeps w(q); inputs come from PE q+1 two steps late, sums from PE q+1 one step late; t = c - q
            const float w = pe < Q ? taps.w[pe] : 0.f;
            float X[U], Xprev[U], Z[U];
#pragma unroll
            for (int u = 0; u < U; ++u) X[u] = Xprev[u] = Z[u] = 0.f;
            for (int t = -(Q - 1); t < C; ++t) {
                const int c = t + pe;
                const bool active = pe < Q && c >= 0 && c < C;         // CheckTime
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float x_fwd = __shfl_down_sync(kFullMask, Xprev[u], 1);
                    const float z_fwd = __shfl_down_sync(kFullMask, Z[u], 1);
                    Xprev[u] = X[u];
                    if (active) {
                        X[u] = (c == 0 || pe == Q - 1) ? xin0[u * xu + c + pe] : x_fwd;
                        Z[u] = (pe == Q - 1) ? X[u] * w : fmaf(X[u], w, z_fwd);
                        if (member && pe == 0) yout0[u * yu + c] = Z[u];
                    }
                }
            }
        } else if (DESIGN == SYSCONV_BFS) {
            // BFS: PE c keeps Z(c); x(t) is broadcast; the weights move one PE up per step; t = c + q
            float W[U], Z[U];
#pragma unroll
            for (int u = 0; u < U; ++u) W[u] = Z[u] = 0.f;
            for (int t = 0; t < N; ++t) {
                const int q = t - pe;
                const bool active = pe < C && q >= 0 && q < Q;         // CheckTime
                const float w_in = t < Q ? taps.w[t] : 0.f;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float fwd = __shfl_up_sync(kFullMask, W[u], 1);
                    W[u] = pe == 0 ? w_in : fwd;
                    if (active) Z[u] = q == 0 ? xin0[u * xu + t] * W[u] : fmaf(xin0[u * xu + t], W[u], Z[u]);
                }
            }
            if (member && pe < C) {
#pragma unroll
                for (int u = 0; u < U; ++u) yout0[u * yu + pe] = Z[u];
            }
        } else {
            // FFS: PE c keeps Z(c); inputs move one PE up per step, weights one PE up every two steps; t = 2c + q
            float X[U], W[U], Wprev[U], Z[U];
#pragma unroll
            for (int u = 0; u < U; ++u) X[u] = W[u] = Wprev[u] = Z[u] = 0.f;
            for (int t = 0; t < 2 * (C - 1) + Q; ++t) {
                const int q = t - 2 * pe;
                const bool active = pe < C && q >= 0 && q < Q;         // CheckTime
                const float w_in = t < Q ? taps.w[t] : 0.f;             // what PE 0 (q = t) takes from memory
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float x_fwd = __shfl_up_sync(kFullMask, X[u], 1);
                    const float w_fwd = __shfl_up_sync(kFullMask, Wprev[u], 1);
                    Wprev[u] = W[u];
                    if (active) {
                        X[u] = (pe == 0 || q == Q - 1) ? xin0[u * xu + pe + q] : x_fwd;
                        W[u] = pe == 0 ? w_in : w_fwd;
                        Z[u] = q == 0 ? X[u] * W[u] : fmaf(X[u], W[u], Z[u]);
                    }
                }
            }
            if (member && pe < C) {
#pragma unroll
                for (int u = 0; u < U; ++u) yout0[u * yu + pe] = Z[u];
            }
        }
        __syncwarp();
        // ---- the outputs of this pass leave the staging area the way the inputs came
        if (DENSE && have) {
            float4 *dst = reinterpret_cast<float4 *>(yg + g0 * C);
#pragma unroll
            for (int i = 0; i < kTilesVecPerLane; ++i)
                if (lane + kLanes * i < out_vec) dst[lane + kLanes * i] = reinterpret_cast<const float4 *>(s_out)[lane + kLanes * i];
        } else if (member) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long g = g0 + u * AW + arr;
                if (g < a.batch)
                    for (int k = pe; k < C; k += LA) yg[g * a.y_bstride + k] = s_out[(u * AW + arr) * C + k];
            }
        }
        have = have_next;
        // (the next pass refills the staging area only after the barrier that follows its own input stores)
        __syncwarp();
    }
}

// true if the tiny-signal kernels cover this call
inline bool tiles_eligible(const Conv1DArgs &a, int design, int q)
{
    if (a.n_out > kTilesMaxOut || q > kTilesMaxQ || a.batch < 2) return false;
    return tiles_array_pes(design, static_cast<int>(a.n_out), q) <= kLanes;
}

template <int DESIGN, int Q, int U>
cudaError_t launch_conv1d_tiles_u(const Conv1DArgs &a, const Taps1D &taps, int LA, int AW, bool dense, cudaStream_t s)
{
    const int C = static_cast<int>(a.n_out), N = static_cast<int>(a.n);
    const int warp_floats = (U * AW * (N + C) + 3) / 4 * 4;
    const size_t smem = sizeof(float) * kTilesWarps * warp_floats;
    const long long per_block = static_cast<long long>(kTilesWarps) * U * AW;
    long long blocks = (a.batch + per_block - 1) / per_block;
    if (blocks > 148LL * 16) blocks = 148LL * 16;           // the warps loop over the remaining signals
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(kTilesWarps * kLanes);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent_launch_enabled() ? 1 : 0;
    if (dense) cudaLaunchKernelEx(&cfg, conv1d_tiles_kernel<DESIGN, Q, U, true>, a, taps, LA, AW, warp_floats);
    else cudaLaunchKernelEx(&cfg, conv1d_tiles_kernel<DESIGN, Q, U, false>, a, taps, LA, AW, warp_floats);
    return cudaGetLastError();
}

template <int DESIGN, int Q>
cudaError_t launch_conv1d_tiles_q(const Conv1DArgs &a, const Taps1D &taps, cudaStream_t s)
{
    const int C = static_cast<int>(a.n_out), N = static_cast<int>(a.n);
    const int LA = tiles_array_pes(DESIGN, C, Q);
    const int AW = kLanes / LA;
    // signals per lane and pass: as many as the staging area and the registers of the dense form take for the two
    // short-schedule designs (FBS filter 5, 10.5 M signals: 310 / 416 / 483 / 531 Gpix/s with 2 / 4 / 8 / 16); the
    // designs that idle through CheckTime steps run best with two (BFS: 76 against 42 with 16, FFS: 34 against 15)
    int U = (DESIGN == SYSCONV_OS || DESIGN == SYSCONV_IS || DESIGN == SYSCONV_WS) ? 16 : 2;
    while (U > 1 && (U * AW * (N + C) > kTilesFloatsPerWarp || U * AW * N > kTilesVecPerLane * kLanes * 4)) U /= 2;
    // dense form: signals packed back to back, every pass a 16-byte aligned run of whole 128-bit words
    const unsigned long long xa = reinterpret_cast<unsigned long long>(a.x), ya = reinterpret_cast<unsigned long long>(a.y);
    const bool dense = a.x_bstride == N && a.y_bstride == C && (xa & 15ull) == 0 && (ya & 15ull) == 0 &&
                       (U * AW * N) % 4 == 0 && (U * AW * C) % 4 == 0 && U * AW * N <= kTilesVecPerLane * kLanes * 4;
    switch (U) {
        case 16: return launch_conv1d_tiles_u<DESIGN, Q, 16>(a, taps, LA, AW, dense, s);
        case 8: return launch_conv1d_tiles_u<DESIGN, Q, 8>(a, taps, LA, AW, dense, s);
        case 4: return launch_conv1d_tiles_u<DESIGN, Q, 4>(a, taps, LA, AW, dense, s);
        case 2: return launch_conv1d_tiles_u<DESIGN, Q, 2>(a, taps, LA, AW, dense, s);
        default: return launch_conv1d_tiles_u<DESIGN, Q, 1>(a, taps, LA, AW, dense, s);
    }
}

template <int DESIGN>
cudaError_t launch_conv1d_tiles_design(const Conv1DArgs &a, const Taps1D &taps, int q, cudaStream_t s)
{
    switch (q) {
        case 1: return launch_conv1d_tiles_q<DESIGN, 1>(a, taps, s);
        case 2: return launch_conv1d_tiles_q<DESIGN, 2>(a, taps, s);
        case 3: return launch_conv1d_tiles_q<DESIGN, 3>(a, taps, s);
        case 4: return launch_conv1d_tiles_q<DESIGN, 4>(a, taps, s);
        case 5: return launch_conv1d_tiles_q<DESIGN, 5>(a, taps, s);
        case 6: return launch_conv1d_tiles_q<DESIGN, 6>(a, taps, s);
        case 7: return launch_conv1d_tiles_q<DESIGN, 7>(a, taps, s);
        case 8: return launch_conv1d_tiles_q<DESIGN, 8>(a, taps, s);
        default: return kNoInstantiation;
    }
}

}  // namespace sysconv
