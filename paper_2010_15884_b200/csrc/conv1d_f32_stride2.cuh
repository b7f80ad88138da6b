// Stride-2 1-D convolution, y(c) = sum_q x(2c+q) w(q), fp32: the stride-2 FBS design of Table 2 (cell 6)
// and the matching input-stationary (SBM) array, folded onto a warp like their stride-1 forms.
//
// Tile geometry: a warp slice is the same 640 inputs (32 lanes x 20) with the same 32-element halo budget;
// it advances by 608 inputs and therefore yields 304 outputs.
//
//  * OS / FBS, stride 2: PE c keeps Z(c).  Its inputs at steps 0 and 1 come from memory (x(2c), x(2c+1));
//    from step 2 on, X(c, q) = X(c+1, q-2): the value the next PE used two steps earlier.  A lane holds
//    10 PEs; their even inputs and their odd inputs form two register chains, each moved one PE down
//    (one shuffle plus renaming) every second step.
//  * IS / SBM, stride 2: PE s keeps x(s); the sum that started at input 2c sits in PE 2c+q at step q and
//    moves one PE up per step, exactly as with stride 1, but only every second PE holds a live sum, so a
//    step is 10 multiply-adds per lane and the lane-to-lane transfer happens every second step.
#pragma once

#include "conv1d_f32.cuh"

namespace sysconv {

constexpr int kWarpOutS2 = kWarpOut1 / 2;     // 304 outputs per warp slice
constexpr int kPeS2 = R1 / 2;                 // 10 outputs per lane

template <int Q>
__device__ __forceinline__ void os_pass_1d_s2(const float *sx, float *so, const Taps1D &taps, int lane)
{
    float X[R1];
    load_lane_block(sx + lane * R1, X);
    float E[kPeS2], O[kPeS2], Z[kPeS2];
#pragma unroll
    for (int j = 0; j < kPeS2; ++j) {
        E[j] = X[2 * j];
        O[j] = X[2 * j + 1];
    }
#pragma unroll
    for (int t = 0; t < Q; ++t) {
        const float wt = taps.w[t];
        if (t % 2 == 0) {
#pragma unroll
            for (int j = 0; j < kPeS2; ++j) Z[j] = (t == 0) ? E[j] * wt : fmaf(E[j], wt, Z[j]);
            if (t + 2 < Q) {
                const float in = __shfl_down_sync(kFullMask, E[0], 1);   // lane 31 keeps its own: invalid PEs
#pragma unroll
                for (int j = 0; j < kPeS2 - 1; ++j) E[j] = E[j + 1];
                E[kPeS2 - 1] = in;
            }
        } else {
#pragma unroll
            for (int j = 0; j < kPeS2; ++j) Z[j] = fmaf(O[j], wt, Z[j]);
            if (t + 2 < Q) {
                const float in = __shfl_down_sync(kFullMask, O[0], 1);
#pragma unroll
                for (int j = 0; j < kPeS2 - 1; ++j) O[j] = O[j + 1];
                O[kPeS2 - 1] = in;
            }
        }
    }
    // PE c holds y(c); PEs from 304 on are incomplete
#pragma unroll
    for (int g = 0; g < kPeS2 / 2; ++g) {
        const int off = lane * kPeS2 + 2 * g;
        if (off < kWarpOutS2) *reinterpret_cast<float2 *>(so + off) = make_float2(Z[2 * g], Z[2 * g + 1]);
    }
}

// ---- OS / FBS, stride 2, paired form for the longer filters (Q >= 12).  PE c at step t and PE c+1 at step
// t-2 use the SAME input x(2c+t), so the sums of PEs c (even) and c+1 share a 64-bit register pair and ONE
// packed fp32x2 FMA with the multiplicand (x, x) and the aligned tap pair (w(t), w(t-2)) serves both (the odd
// PE lags two steps).  Only the even PEs' inputs are needed: x(2c+t) with c = 2m is element 4m+t of the lane
// block, i.e. four register chains (t mod 4), each moved one pair down every fourth step.  Q+2 steps of 5
// packed FMAs replace Q steps of 10 scalar ones; the first two and the last two steps touch only one sum
// of each pair and stay scalar (no zero tap multiplies an input).
struct Taps1DPairsS2 {
    float2 p[kMaxQ1 + 2];       // p[t] = (w(t), w(t-2)); taps outside 0..Q-1 are zero
};

template <int Q>
__device__ __forceinline__ void os_pass_1d_s2_paired(const float *sx, float *so, const Taps1D &taps,
                                                     const Taps1DPairsS2 &tp, int lane)
{
    constexpr int M = kPeS2 / 2;                // 5 pairs of PEs per lane
    float X[R1];
    load_lane_block(sx + lane * R1, X);
    float S[4][M];                              // S[r][m]: the input pair m uses at the next step t = r mod 4
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int r = 0; r < 4; ++r) S[r][m] = X[4 * m + r];
    float2 Z[M];
#pragma unroll
    for (int t = 0; t < Q + 2; ++t) {
        float(&C)[M] = S[t % 4];
#pragma unroll
        for (int m = 0; m < M; ++m) {
            if (t == 0) Z[m] = make_float2(C[m] * taps.w[0], 0.f);
            else if (t == 1) Z[m].x = fmaf(C[m], taps.w[1], Z[m].x);
            else if (t >= Q) Z[m].y = fmaf(C[m], taps.w[t - 2], Z[m].y);
            else Z[m] = __ffma2_rn(make_float2(C[m], C[m]), tp.p[t], Z[m]);
        }
        if (t + 4 < Q + 2) {
            const float in = __shfl_down_sync(kFullMask, C[0], 1);       // lane 31 keeps its own: invalid PEs
#pragma unroll
            for (int m = 0; m < M - 1; ++m) C[m] = C[m + 1];
            C[M - 1] = in;
        }
    }
    // pair m holds y(10 lane + 2m) and y(10 lane + 2m + 1); PEs from 304 on are incomplete
#pragma unroll
    for (int m = 0; m < M; ++m) {
        const int off = lane * kPeS2 + 2 * m;
        if (off < kWarpOutS2) *reinterpret_cast<float2 *>(so + off) = Z[m];
    }
}

template <int Q>
__device__ __forceinline__ void is_pass_1d_s2(const float *sx, float *so, const Taps1D &taps, int lane)
{
    float X[R1], Z[R1];
    load_lane_block(sx + lane * R1, X);
#pragma unroll
    for (int t = 0; t < Q; ++t) {
        const float wt = taps.w[t];
        // live sums sit in the PEs whose index has the parity of t (20 PEs per lane: lane offsets are even)
        float from_prev = 0.f;
        if (t > 0 && t % 2 == 0) from_prev = __shfl_up_sync(kFullMask, Z[R1 - 1], 1);   // lane 0: its own, invalid
#pragma unroll
        for (int j = R1 - 1; j >= 0; --j) {
            if (j % 2 != t % 2) continue;
            const float z = (t == 0) ? 0.f : (j == 0 ? from_prev : Z[j - 1]);
            Z[j] = (t == 0) ? X[j] * wt : fmaf(X[j], wt, z);
        }
    }
    // PE s (parity of Q-1) holds y((s-(Q-1))/2); the first Q-1 PEs of the slice hold incomplete sums
#pragma unroll
    for (int j = 0; j < R1; ++j) {
        if (j % 2 != (Q - 1) % 2) continue;
        const int start = lane * R1 + j - (Q - 1);
        if (start >= 0 && start < 2 * kWarpOutS2) so[start >> 1] = Z[j];
    }
}

// ---- IS / SBM, stride 2, paired form for the longer filters (Q >= 12).  The sums of outputs c (even) and
// c+1 start two PEs apart and travel together in one 64-bit register pair: PE s adds x(s)*w(t) to the first
// and x(s)*w(t-2) to the second, t = s-2c, with ONE packed fp32x2 FMA.  The pair sits in PE 2c+t at step t,
// so every fourth PE holds a live pair: Q+2 steps of 5 packed FMAs, lane-to-lane transfer every fourth step.
template <int Q>
__device__ __forceinline__ void is_pass_1d_s2_paired(const float *sx, float *so, const Taps1D &taps,
                                                     const Taps1DPairsS2 &tp, int lane)
{
    float X[R1];
    load_lane_block(sx + lane * R1, X);
    constexpr int M = R1 / 4;                   // 5 live pairs per lane
    float2 P[4][M];                             // P[r][i]: the pair in PE 4i+r, live while r = t mod 4
#pragma unroll
    for (int t = 0; t < Q + 2; ++t) {
        const int r = t % 4;
        float2 up = make_float2(0.f, 0.f);
        if (t > 0 && r == 0)                    // lane 0 keeps its own: invalid PEs
            up = make_float2(__shfl_up_sync(kFullMask, P[3][M - 1].x, 1), __shfl_up_sync(kFullMask, P[3][M - 1].y, 1));
#pragma unroll
        for (int i = M - 1; i >= 0; --i) {
            const float x = X[4 * i + r];
            float2 prev = up;
            if (r > 0) prev = P[r - 1][i];
            else if (i > 0) prev = P[3][i - 1];
            if (t == 0) P[r][i] = make_float2(x * taps.w[0], 0.f);
            else if (t == 1) P[r][i] = make_float2(fmaf(x, taps.w[1], prev.x), prev.y);
            else if (t >= Q) P[r][i] = make_float2(prev.x, fmaf(x, taps.w[t - 2], prev.y));
            else P[r][i] = __ffma2_rn(make_float2(x, x), tp.p[t], prev);
        }
    }
    // PE s (s = Q+1 mod 4) holds y((s-Q-1)/2) and the next output; the first PEs of the slice hold incomplete sums
    constexpr int rl = (Q + 1) % 4;
#pragma unroll
    for (int i = 0; i < M; ++i) {
        const int start = lane * R1 + 4 * i + rl - (Q + 1);
        if (start >= 0 && start < 2 * kWarpOutS2) *reinterpret_cast<float2 *>(so + (start >> 1)) = P[rl][i];
    }
}

template <int DESIGN, int Q, int WARPS, int K>
__global__ void __launch_bounds__(WARPS *kLanes)
conv1d_f32_s2_kernel(const Conv1DArgs a, const __grid_constant__ Taps1D taps, const __grid_constant__ Taps1DPairsS2 tpairs,
                     unsigned *status_word)
{
    dependent_launch_enter();
    constexpr int kThreads = WARPS * kLanes;
    constexpr int kTileAdv = WARPS * kWarpOut1;         // inputs a tile advances by
    constexpr int kTileIn = kTileAdv + kHalo1;
    constexpr int kTileOut = WARPS * kWarpOutS2;
    __shared__ __align__(128) float s_in[K][kTileIn];
    __shared__ __align__(128) float s_out[K][kTileOut];
    __shared__ __align__(8) uint64_t full[K];
    const int lane = threadIdx.x & (kLanes - 1);
    const int warp = threadIdx.x / kLanes;
    const long long base_in = static_cast<long long>(blockIdx.x) * (K * kTileAdv);
    const bool x_ok = ((reinterpret_cast<uintptr_t>(a.x) & 15) == 0) && (a.batch == 1 || (a.x_bstride & 3) == 0);
    const bool y_ok = ((reinterpret_cast<uintptr_t>(a.y) & 15) == 0) && (a.batch == 1 || (a.y_bstride & 3) == 0);

    if (threadIdx.x == 0) {
        for (int k = 0; k < K; ++k) mbar_init(&full[k], 1);
        mbar_init_fence();
    }
    // elements of tile k that arrive by bulk copy: the part of the tile inside the signal, in whole 16-byte words.
    // A tile without outputs gets no copy at all (issuer and consumers share this predicate).
    auto bulk_in = [&](int k) -> int {
        const long long t0 = base_in + k * kTileAdv;
        if (!x_ok || t0 >= a.n || t0 / 2 >= a.n_out) return 0;
        const long long valid = a.n - t0 < kTileIn ? a.n - t0 : kTileIn;
        return static_cast<int>(valid) & ~3;
    };
    unsigned phase = 0;
    for (int b = blockIdx.y; b < a.batch; b += gridDim.y) {
        const float *xg = static_cast<const float *>(a.x) + b * a.x_bstride;
        float *yg = static_cast<float *>(a.y) + b * a.y_bstride;
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int be = bulk_in(k);
                if (be > 0) {
                    mbar_arrive_expect_tx(&full[k], be * 4);
                    bulk_load(s_in[k], xg + (base_in + k * kTileAdv), be * 4, &full[k]);
                }
            }
        }
#pragma unroll 1
        for (int k = 0; k < K; ++k) {
            const long long t0 = base_in + k * kTileAdv;    // first input of the tile (even)
            const long long o0 = t0 / 2;                    // first output of the tile
            if (o0 >= a.n_out) break;
            const int be = bulk_in(k);
            if (be > 0) {
                const bool ok = mbar_wait_bounded(&full[k], phase, kWaitPolls);
                const bool give_up = WARPS == 1 ? __any_sync(kFullMask, !ok) != 0 : __syncthreads_or(!ok) != 0;
                if (give_up) {
                    if (threadIdx.x == 0) {
                        atomicExch(status_word, 1u);
                        for (int j = k; j < K; ++j)          // copies still in flight target this CTA's memory
                            if (bulk_in(j) > 0) mbar_wait_bounded(&full[j], phase, kGiveUpPolls);
                    }
                    if (lane == 0) bulk_wait_read<0>();      // every warp's own bulk stores have read their source
                    return;
                }
            }
            if (be < kTileIn) {
                // ragged last tile or unaligned signal: the rest by ordinary loads, zeros beyond the signal's end
                if (be == 0) stage_in_1d(xg, a.n, t0, s_in[k], kTileIn, kThreads);
                else stage_in_1d(xg, a.n, t0, s_in[k], kTileIn, kThreads, be);
                __syncthreads();
            }

            const float *sx = s_in[k] + warp * kWarpOut1;
            float *so = s_out[k] + warp * kWarpOutS2;
            if (DESIGN == SYSCONV_OS && Q >= 12) os_pass_1d_s2_paired<Q>(sx, so, taps, tpairs, lane);
            else if (DESIGN == SYSCONV_OS) os_pass_1d_s2<Q>(sx, so, taps, lane);
            else if (Q >= 12) is_pass_1d_s2_paired<Q>(sx, so, taps, tpairs, lane);
            else is_pass_1d_s2<Q>(sx, so, taps, lane);

            if (y_ok) {
                // the warp's outputs inside the signal: whole 16-byte words by bulk store, up to three more by lanes
                const long long w0 = o0 + warp * kWarpOutS2;
                long long vw = a.n_out - w0;
                vw = vw > kWarpOutS2 ? kWarpOutS2 : (vw < 0 ? 0 : vw);
                const int bo = static_cast<int>(vw) & ~3;
                fence_proxy_async();
                __syncwarp();
                if (lane == 0 && bo > 0) {
                    bulk_store(yg + w0, so, bo * 4);
                    bulk_commit();
                }
                if (bo + lane < vw) yg[w0 + bo + lane] = so[bo + lane];
            } else {
                __syncthreads();
                stage_out_1d(yg, a.n_out, o0, s_out[k], kTileOut, kThreads);
            }
        }
        phase ^= 1u;
        if (lane == 0) bulk_wait_read<0>();
    }
}

template <int DESIGN, int Q>
cudaError_t launch_conv1d_f32_s2_q(const Conv1DArgs &a, const Taps1D &taps, unsigned *status_word, cudaStream_t s)
{
    constexpr int WARPS = 2, K = 2;
    const long long per_cta = static_cast<long long>(K) * WARPS * kWarpOutS2;
    const long long ctas = (a.n_out + per_cta - 1) / per_cta;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(ctas), static_cast<unsigned>(a.batch < 65535 ? a.batch : 65535));
    Taps1DPairsS2 tp;
    for (int t = 0; t < kMaxQ1 + 2; ++t)
        tp.p[t] = make_float2(t < kMaxQ1 ? taps.w[t] : 0.f, t >= 2 ? taps.w[t - 2] : 0.f);
    launch_kernel(conv1d_f32_s2_kernel<DESIGN, Q, WARPS, K>, grid, WARPS * kLanes, s, a, taps, tp, status_word);
    return cudaGetLastError();
}

template <int DESIGN>
cudaError_t launch_conv1d_f32_s2(const Conv1DArgs &a, const float *w, int q, unsigned *status_word, cudaStream_t s,
                                 int *launches)
{
    Taps1D taps;
    for (int k = 0; k < kMaxQ1; ++k) taps.w[k] = k < q ? w[k] : 0.f;
    cudaError_t err = kNoInstantiation;
    switch (q) {
#define SYSCONV_CASE(QQ) case QQ: err = launch_conv1d_f32_s2_q<DESIGN, QQ>(a, taps, status_word, s); break;
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
