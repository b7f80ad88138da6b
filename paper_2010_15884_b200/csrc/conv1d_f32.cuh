// 1-D fp32 convolution (Eq. 2) as folded linear systolic arrays on a warp.
//
// One CTA handles K consecutive tiles of outputs.  Thread 0 fetches the inputs each tile needs with one
// bulk asynchronous copy per tile (global -> shared, completion on the tile's mbarrier), all K copies
// issued up front; every warp waits for a tile, runs its systolic array pass on its slice, collects its
// outputs in shared memory and its lane 0 sends them to global memory with one bulk copy, then moves
// to the next tile, whose copy has meanwhile landed.  No thread spends instructions on staging.
//
// CTAs are small and each takes a fixed, contiguous piece of the signal, on purpose: on B200 the
// in-order CTA dispatcher keeps reads and writes evenly mixed and sustains ~6.2 TB/s, where persistent
// grid-stride loops over the same tiles (bulk copies or plain loads alike) stalled near 5.5 TB/s.
//
// Tiles that touch the end of the signal, and calls whose x or y is not 16-byte aligned, are staged
// with ordinary loads/stores by the threads of the CTA instead (same kernel, same passes).
//
// Lane l of a warp holds R1 = 20 consecutive PEs.  A time step is R1 fused multiply-adds per lane, one
// shuffle (the value that crosses the lane boundary) and a renaming of the lane's own registers (the
// loops over time are fully unrolled, so "PE j takes PE j-1's value" costs nothing).  Every PE runs at
// every step (no CheckTime); PEs whose sums are incomplete are not drained.
//
// The waits on the mbarriers are bounded; if a limit runs out the CTA raises *status_word, gives its
// other copies a bounded chance to land and returns without writing the rest of its tiles.
#pragma once

#include "sysconv_common.cuh"
#include "tma_utils.cuh"

namespace sysconv {

// Tile geometry of a design.  OS and IS: each warp turns 640 inputs into 608 outputs.  WS: each warp
// holds 32 one-lane arrays that stream 76 outputs each (2432 outputs per warp).  A tile is WARPS
// warp slices plus a 32-element halo (the halo budget is 32 whatever Q).
template <int DESIGN, int WARPS>
struct Geo1D {
    static constexpr int kWarps = WARPS;
    static constexpr int kWarpOut = DESIGN == SYSCONV_WS ? kLanes * kWsSeg1 : kWarpOut1;
    static constexpr int kThreads = kWarps * kLanes;
    static constexpr int kTileOut = kWarps * kWarpOut;     // outputs per CTA tile
    static constexpr int kTileIn = kTileOut + kHalo1;      // inputs per CTA tile
};
// shape used by the library (measured best on B200): two warps and two tiles per CTA; WS one warp per CTA
// with one (four times as large) tile
template <int DESIGN, int Q>
struct DefaultShape1D {
    static constexpr int kWarps = DESIGN == SYSCONV_WS ? 1 : 2;
    static constexpr int kTiles = DESIGN == SYSCONV_WS ? 1 : 2;
};

// ---- ordinary-load staging (ragged or unaligned tiles) ------------------------

// Copy x[t0 + first .. t0 + tile_in) to shared memory, zeros beyond the signal's end.
__device__ __forceinline__ void stage_in_1d(const float *__restrict__ xg, long long n, long long t0,
                                            float *__restrict__ s_in, int tile_in, int threads, int first = 0)
{
    for (int i = first + threadIdx.x; i < tile_in; i += threads) {
        const long long g = t0 + i;
        s_in[i] = g < n ? xg[g] : 0.f;
    }
}

// Copy the tile's outputs from shared memory to y[t0 .. min(t0 + tile_out, n_out)).
__device__ __forceinline__ void stage_out_1d(float *__restrict__ yg, long long n_out, long long t0,
                                             const float *s_out, int tile_out, int threads)
{
    for (int i = threadIdx.x; i < tile_out; i += threads) {
        const long long g = t0 + i;
        if (g < n_out) yg[g] = s_out[i];
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

// ---- output-stationary, PE-paired form for the longer filters (Q >= 12).  Same array, same forwarding
// (one shuffle per step).  The partial sums of two neighbouring PEs c (even) and c+1 share a 64-bit
// register pair, and ONE packed fp32x2 FMA (fma.rn.f32x2, sm_100) serves both: the input that PE c uses
// with tap t at step t is the input PE c+1 used with tap t-1, so the multiplicand is (x, x) and the
// multiplier the tap pair (w(t), w(t-1)), which comes straight from the kernel parameters as an aligned
// uniform-register pair (the pairs are laid out by the launcher: built in the kernel from the plain tap
// array they cost almost one uniform move per packed FMA).  Q+1 steps of R1/2 packed FMAs replace Q steps of R1 scalar ones: about half
// the issue slots per MAC (the scalar form is issue-bound at Q = 32).  In the first and the last step
// only one PE of each pair has a tap: those two steps use scalar FMAs, so that no input outside an
// output's window ever enters its sum (a zero tap times a non-finite input would).
struct Taps1DPairs {
    float2 p[kMaxQ1 + 1];       // p[t] = (w(t), w(t-1)); taps outside 0..Q-1 are zero
};

template <int Q>
__device__ __forceinline__ void os_pass_1d_paired(const float *sx, float *so, const Taps1D &taps,
                                                  const Taps1DPairs &tp, int lane)
{
    constexpr int M = R1 / 2;
    float X[R1];
    load_lane_block(sx + lane * R1, X);
    float2 D[R1];                               // the forwarded inputs, each as the pair (x, x)
#pragma unroll
    for (int j = 0; j < R1; ++j) D[j] = make_float2(X[j], X[j]);
    float2 Z[M];                                // Z[m] = partial sums of PEs 2m and 2m+1
#pragma unroll
    for (int t = 0; t <= Q; ++t) {
#pragma unroll
        for (int m = 0; m < M; ++m) {
            if (t == 0) {
                Z[m] = make_float2(D[2 * m].x * taps.w[0], 0.f);
            } else if (t == Q) {
                Z[m].y = fmaf(D[2 * m].x, taps.w[Q - 1], Z[m].y);
            } else {
                Z[m] = __ffma2_rn(D[2 * m], tp.p[t], Z[m]);
            }
        }
        if (t < Q) {
            const float in = __shfl_down_sync(kFullMask, D[0].x, 1);     // lane 31 keeps its own: invalid PEs
#pragma unroll
            for (int j = 0; j < R1 - 1; ++j) D[j] = D[j + 1];
            D[R1 - 1] = make_float2(in, in);
        }
    }
#pragma unroll
    for (int g = 0; g < R1 / 4; ++g) {
        const int off = lane * R1 + 4 * g;
        if (off < kWarpOut1)
            *reinterpret_cast<float4 *>(so + off) = make_float4(Z[2 * g].x, Z[2 * g].y, Z[2 * g + 1].x, Z[2 * g + 1].y);
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

// ---- input-stationary, paired form for the longer filters (Q >= 12).  The sums of two neighbouring outputs
// o (even) and o+1 travel TOGETHER in one 64-bit register pair: PE s adds x(s)*w(s-o) to the first and
// x(s)*w(s-o-1) to the second, i.e. ONE packed fp32x2 FMA with the multiplicand (x(s), x(s)) and the aligned
// tap pair (w(t), w(t-1)), t = s-o, from the kernel parameters.  The pair of outputs (o, o+1) sits in PE
// o+t at step t, so the PEs with the parity of t hold the live pairs: Q+1 steps of R1/2 packed FMAs replace
// Q steps of R1 scalar ones; the pairs move one PE up per step as before (lane-to-lane every second step).
// The first and the last step touch only one sum of each pair and use scalar arithmetic, so that no input
// outside an output's window enters its sum.
template <int Q>
__device__ __forceinline__ void is_pass_1d_paired(const float *sx, float *so, const Taps1D &taps,
                                                  const Taps1DPairs &tp, int lane)
{
    float X[R1];
    load_lane_block(sx + lane * R1, X);
    float2 D[R1], P[R1];
#pragma unroll
    for (int j = 0; j < R1; ++j) D[j] = make_float2(X[j], X[j]);
#pragma unroll
    for (int j = 0; j < R1; j += 2) P[j] = make_float2(X[j] * taps.w[0], 0.f);
#pragma unroll
    for (int t = 1; t <= Q; ++t) {
        float2 up = make_float2(0.f, 0.f);
        if (t % 2 == 0)                                  // lane 0 keeps its own: invalid PEs
            up = make_float2(__shfl_up_sync(kFullMask, P[R1 - 1].x, 1), __shfl_up_sync(kFullMask, P[R1 - 1].y, 1));
#pragma unroll
        for (int j = R1 - 1; j >= 0; --j) {
            if (j % 2 != t % 2) continue;
            const float2 prev = j == 0 ? up : P[j - 1];
            if (t == Q) P[j] = make_float2(prev.x, fmaf(X[j], taps.w[Q - 1], prev.y));
            else P[j] = __ffma2_rn(D[j], tp.p[t], prev);
        }
    }
    // PE s (parity of Q) holds y(s-Q) and y(s-Q+1); the first PEs of the slice hold incomplete sums
#pragma unroll
    for (int j = Q % 2; j < R1; j += 2) {
        const int off = lane * R1 + j - Q;
        if (off >= 0 && off < kWarpOut1) *reinterpret_cast<float2 *>(so + off) = P[j];
    }
}

// ---- weight-stationary (BSM, Table 2): PE s keeps w(s); at step t the input x(t) is broadcast to the
// array, Z_s <- Z_{s-1} + x(t) * w(s), PE 0 starts a new sum and the last PE emits y(t-(Q-1)).
//
// An array has only Q <= 32 PEs, so it is folded ENTIRELY into one lane (PE-to-PE transfer = register
// renaming, no shuffle at all) and a warp holds 32 independent arrays; array a streams the 76-output
// segment a of the warp's 2432-output slice (76 floats = 19 16-byte words: the lanes' 128-bit reads of
// their segments fall in distinct banks).  All arrays hold the same filter, so the stationary weights
// are uniform operands from the kernel parameters rather than a copy per lane.
//
// Paired form: the sums of two neighbouring outputs o (even) and o+1 travel together in one 64-bit
// register pair; PE s adds x(t)*w(s) to the first and x(t)*w(s-1) to the second with ONE packed fp32x2
// FMA (multiplicand (x(t), x(t)), multiplier the aligned tap pair (w(s), w(s-1))).  The pair (o, o+1)
// sits in PE t-o at step t, so the PEs with the parity of t hold the live pairs: a step is Q/2 packed
// FMAs.  PE 0 opens a pair with a scalar multiply, and the pair leaves PE Q-1 with its second sum one tap
// short, which the emission adds with a scalar FMA: no zero tap ever multiplies an input.
//
// Arrays neither fill nor drain separately: every array runs exactly the 76 steps of its segment.  What
// array a+1 emits during its first steps (sums over its own inputs only) are the missing parts of the
// sums still in flight in array a when it stops, so they are stored into segment a's tail and array a
// adds its registers to them afterwards.  Only the last array of the slice has no successor: its tail
// gets the missing taps from a short direct sum over the slice's halo.
constexpr int kWsSlice1 = kLanes * kWsSeg1;     // 2432 outputs per warp slice

template <int Q>
__device__ __forceinline__ void ws_pass_1d(const float *sx, float *so, const Taps1D &taps, const Taps1DPairs &tp,
                                           int lane)
{
    constexpr int kGroups = kWsSeg1 / 4;              // 76 time steps in groups of four
    constexpr int kTail = Q - (Q % 2);                // outputs at the end of a segment still in flight
    static_assert(Q <= kHalo1 && Q <= kWsSeg1, "array longer than the halo or the segment");
    const float4 *xs4 = reinterpret_cast<const float4 *>(sx + lane * kWsSeg1);
    float *yo = so + lane * kWsSeg1;
    float2 P[Q];
#pragma unroll
    for (int s = 0; s < Q; ++s) P[s] = make_float2(0.f, 0.f);

#pragma unroll
    for (int k = 0; k < kGroups; ++k) {
        const float4 xv = xs4[k];                      // x(4k .. 4k+3) of this array's stream
        const float xr[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int t = 4 * k + r;
            const float x = xr[r];
            if (t % 2 == Q % 2) {
                // the pair that left PE Q-1 one step ago: outputs t-Q and t-Q+1 of this segment.  Negative
                // positions are the tail of the previous segment and receive this array's share of those
                // sums (the first array has no predecessor in the slice: the previous slice patches its own tail)
                const float2 e = make_float2(P[Q - 1].x, fmaf(x, taps.w[Q - 1], P[Q - 1].y));
                const int o = t - Q;
                if (o >= 0 || lane > 0) *reinterpret_cast<float2 *>(yo + o) = e;
            }
            const float2 d = make_float2(x, x);
#pragma unroll
            for (int s = Q - 1; s >= 1; --s)
                if (s % 2 == t % 2) P[s] = __ffma2_rn(d, tp.p[s], P[s - 1]);
            if (t % 2 == 0) P[0] = make_float2(x * taps.w[0], 0.f);
        }
    }
    // The last array's tail has no successor: store the taps it is missing, summed directly over the halo
    // (output c = kWsSlice1-1-j lacks the taps k > j; the first position of an even-length tail lacks nothing).
    if (lane < kTail) {
        const int c = kWsSlice1 - 1 - lane;
        float acc = 0.f;
#pragma unroll
        for (int k = 1; k < Q; ++k)
            if (k > lane) acc = fmaf(taps.w[k], sx[c + k], acc);
        so[c] = acc;
    }
    __syncwarp();
    // the odd PEs stopped while holding the pairs of outputs 75-s and 76-s of the segment: add them to what is there
#pragma unroll
    for (int s = 1; s < Q; s += 2) {
        yo[kWsSeg1 - 1 - s] += P[s].x;
        yo[kWsSeg1 - s] += P[s].y;
    }
}

// ---------------------------------------------------------------------------------------------------
// The paper's other three 1-D designs (Table 2): FSM, BFS and FFS.  They are built unfolded, one PE per
// lane, with the CheckTime guard of Table 1 (a PE works only in its own time steps), as a faithful
// rendering rather than a fast one: the paper's own model (Table 4) gives them 25 % (BFS) and 14 % (FFS)
// lane utilisation and a quarter of the outturn of SBM/FBS.  The time loops are run-time loops over
// t = s.z; forwarded values with a two-step delay keep a two-deep register history (Code 2).
// ---------------------------------------------------------------------------------------------------

// BFS: inputs broadcast, weights forwarded, sums stay.  PE c = lane, t = c + q.  Per step every PE takes
// the weight its lower neighbour held one step ago (PE 0 takes w(t)), x(t) is broadcast, and PE c adds
// x(t) * w(t-c) while 0 <= t-c < Q.  A warp slice of 608 outputs is 19 consecutive arrays of 32 PEs.
template <int Q>
__device__ __forceinline__ void bfs_pass_1d(const float *sx, float *so, const Taps1D &taps, int lane)
{
    for (int blk = 0; blk < kWarpOut1 / kLanes; ++blk) {
        const float *xs = sx + blk * kLanes;
        float W = 0.f, Z = 0.f;
        for (int t = 0; t < kLanes + Q - 1; ++t) {
            const float fwd = __shfl_up_sync(kFullMask, W, 1);
            W = lane == 0 ? (t < Q ? taps.w[t] : 0.f) : fwd;
            const float xb = xs[t];                                   // same address in every lane: broadcast
            const int q = t - lane;
            if (q >= 0 && q < Q) Z = (q == 0) ? xb * W : fmaf(xb, W, Z);
        }
        so[blk * kLanes + lane] = Z;
    }
}

// FFS: inputs forwarded (one step), weights forwarded with a two-step delay, sums stay.  PE c = lane,
// t = 2c + q.  X(c,q) comes from PE c-1 one step ago unless c == 0 or q == Q-1 (then x(c+q) is loaded);
// W(c,q) comes from PE c-1 two steps ago (PE 0 takes w(t)).
template <int Q>
__device__ __forceinline__ void ffs_pass_1d(const float *sx, float *so, const Taps1D &taps, int lane)
{
    for (int blk = 0; blk < kWarpOut1 / kLanes; ++blk) {
        const float *xs = sx + blk * kLanes;
        float X = 0.f, W = 0.f, Wprev = 0.f, Z = 0.f;                 // Wprev: this PE's weight one step ago
        for (int t = 0; t < 2 * (kLanes - 1) + Q; ++t) {
            const float x_fwd = __shfl_up_sync(kFullMask, X, 1);      // neighbour's X of one step ago
            const float w_fwd = __shfl_up_sync(kFullMask, Wprev, 1);  // neighbour's W of two steps ago
            const int q = t - 2 * lane;
            const bool active = q >= 0 && q < Q;
            Wprev = W;
            if (active) {
                X = (lane == 0 || q == Q - 1) ? xs[lane + q] : x_fwd;
                W = lane == 0 ? taps.w[q] : w_fwd;
                Z = (q == 0) ? X * W : fmaf(X, W, Z);
            }
        }
        so[blk * kLanes + lane] = Z;
    }
}

// FSM: inputs forwarded with a two-step delay, weights stay, sums migrate.  PE q = lane inside an array of
// LA lanes (LA = Q rounded up to a power of two; lanes beyond Q idle), t = c - q.  The stream enters at PE
// Q-1; X(c,q) comes from PE q+1 two steps ago unless c == 0 or q == Q-1; Z(c,q) comes from PE q+1 one step
// ago (PE Q-1 starts at zero); PE 0 emits y(c) at t = c.  The 32/LA arrays of a warp take consecutive
// segments of the slice.
template <int Q>
__device__ __forceinline__ void fsm_pass_1d(const float *sx, float *so, const Taps1D &taps, int lane)
{
    constexpr int LA = Q <= 1 ? 1 : Q <= 2 ? 2 : Q <= 4 ? 4 : Q <= 8 ? 8 : Q <= 16 ? 16 : 32;
    constexpr int kArrays = kLanes / LA;
    constexpr int kSeg = kWarpOut1 / kArrays;                         // outputs per array
    const int q = lane & (LA - 1);
    const int arr = lane / LA;
    const float *xs = sx + arr * kSeg;
    float *ys = so + arr * kSeg;
    const float w = q < Q ? taps.w[q] : 0.f;
    float X = 0.f, Xprev = 0.f, Z = 0.f;                              // Xprev: this PE's input one step ago
    for (int t = -(Q - 1); t < kSeg; ++t) {
        const float x_fwd = __shfl_down_sync(kFullMask, Xprev, 1, LA);   // neighbour's X of two steps ago
        const float z_fwd = __shfl_down_sync(kFullMask, Z, 1, LA);       // neighbour's Z of one step ago
        const int c = t + q;
        const bool active = q < Q && c >= 0 && c < kSeg;
        Xprev = X;
        if (active) {
            X = (c == 0 || q == Q - 1) ? xs[c + q] : x_fwd;
            Z = (q == Q - 1) ? X * w : fmaf(X, w, z_fwd);
            if (q == 0) ys[c] = Z;
        }
    }
}

template <int DESIGN, int Q, int WARPS, int K>
__global__ void __launch_bounds__(Geo1D<DESIGN, WARPS>::kThreads)
conv1d_f32_kernel(const Conv1DArgs a, const __grid_constant__ Taps1D taps, const __grid_constant__ Taps1DPairs tpairs,
                  unsigned *status_word)
{
    dependent_launch_enter();
    using G = Geo1D<DESIGN, WARPS>;
    __shared__ __align__(128) float s_in[K][G::kTileIn];
    __shared__ __align__(128) float s_out[K][G::kTileOut];
    __shared__ __align__(8) uint64_t full[K];
    const int lane = threadIdx.x & (kLanes - 1);
    const int warp = threadIdx.x / kLanes;
    const long long base = static_cast<long long>(blockIdx.x) * (K * G::kTileOut);
    // bulk copies need 16-byte aligned global addresses (tile starts are multiples of 4 elements)
    const bool x_ok = ((reinterpret_cast<uintptr_t>(a.x) & 15) == 0) && (a.batch == 1 || (a.x_bstride & 3) == 0);
    const bool y_ok = ((reinterpret_cast<uintptr_t>(a.y) & 15) == 0) && (a.batch == 1 || (a.y_bstride & 3) == 0);

    if (threadIdx.x == 0) {
        for (int k = 0; k < K; ++k) mbar_init(&full[k], 1);
        mbar_init_fence();
    }
    // elements of tile k that arrive by bulk copy: the part of the tile inside the signal, in whole 16-byte words.
    // A tile without outputs gets no copy at all: the issuing thread and the consumers use this one predicate,
    // so no copy is ever issued that nobody waits for.
    auto bulk_in = [&](int k) -> int {
        const long long t0 = base + k * G::kTileOut;
        if (!x_ok || t0 >= a.n_out) return 0;
        const long long valid = a.n - t0 < G::kTileIn ? a.n - t0 : G::kTileIn;
        return static_cast<int>(valid) & ~3;
    };
    unsigned phase = 0;
    for (int b = blockIdx.y; b < a.batch; b += gridDim.y) {
        const float *xg = static_cast<const float *>(a.x) + b * a.x_bstride;
        float *yg = static_cast<float *>(a.y) + b * a.y_bstride;
        // the barriers are initialised, and all warps are done with the previous signal's tiles
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int be = bulk_in(k);
                if (be > 0) {
                    mbar_arrive_expect_tx(&full[k], be * 4);
                    bulk_load(s_in[k], xg + (base + k * G::kTileOut), be * 4, &full[k]);
                }
            }
        }
#pragma unroll 1
        for (int k = 0; k < K; ++k) {
            const long long t0 = base + k * G::kTileOut;
            if (t0 >= a.n_out) break;
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
            if (be < G::kTileIn) {
                // ragged last tile or unaligned signal: the rest by ordinary loads, zeros beyond the signal's end
                // (two call sites: with a literal start the loop's trip count is known and its loads are issued together)
                if (be == 0) stage_in_1d(xg, a.n, t0, s_in[k], G::kTileIn, G::kThreads);
                else stage_in_1d(xg, a.n, t0, s_in[k], G::kTileIn, G::kThreads, be);
                __syncthreads();
            }

            const float *sx = s_in[k] + warp * G::kWarpOut;
            float *so = s_out[k] + warp * G::kWarpOut;
            if (DESIGN == SYSCONV_OS && Q >= 12) os_pass_1d_paired<Q>(sx, so, taps, tpairs, lane);
            else if (DESIGN == SYSCONV_OS) os_pass_1d<Q>(sx, so, taps, lane);
            else if (DESIGN == SYSCONV_IS && Q >= 12) is_pass_1d_paired<Q>(sx, so, taps, tpairs, lane);
            else if (DESIGN == SYSCONV_IS) is_pass_1d<Q>(sx, so, taps, lane);
            else if (DESIGN == SYSCONV_WS) ws_pass_1d<Q>(sx, so, taps, tpairs, lane);
            else if (DESIGN == SYSCONV_FSM) fsm_pass_1d<Q>(sx, so, taps, lane);
            else if (DESIGN == SYSCONV_BFS) bfs_pass_1d<Q>(sx, so, taps, lane);
            else ffs_pass_1d<Q>(sx, so, taps, lane);

            if (y_ok) {
                // the warp's outputs inside the signal: whole 16-byte words by bulk store, up to three more by lanes
                const long long w0 = t0 + warp * G::kWarpOut;
                long long vw = a.n_out - w0;
                vw = vw > G::kWarpOut ? G::kWarpOut : (vw < 0 ? 0 : vw);
                const int bo = static_cast<int>(vw) & ~3;
                fence_proxy_async();                     // my shared-memory writes, before the bulk store reads them
                __syncwarp();
                if (lane == 0 && bo > 0) {
                    bulk_store(yg + w0, so, bo * 4);
                    bulk_commit();
                }
                if (bo + lane < vw) yg[w0 + bo + lane] = so[bo + lane];
            } else {
                __syncthreads();
                stage_out_1d(yg, a.n_out, t0, s_out[k], G::kTileOut, G::kThreads);
            }
        }
        phase ^= 1u;
        if (lane == 0) bulk_wait_read<0>();              // shared memory may be reused (or released) after this
    }
}

template <int DESIGN, int Q, int WARPS = DefaultShape1D<DESIGN, Q>::kWarps, int K = DefaultShape1D<DESIGN, Q>::kTiles>
cudaError_t launch_conv1d_f32_q(const Conv1DArgs &a, const Taps1D &taps, unsigned *status_word, cudaStream_t s)
{
    using G = Geo1D<DESIGN, WARPS>;
    const long long per_cta = static_cast<long long>(K) * G::kTileOut;
    const long long ctas = (a.n_out + per_cta - 1) / per_cta;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(ctas), static_cast<unsigned>(a.batch < 65535 ? a.batch : 65535));
    Taps1DPairs tp;
    for (int t = 0; t <= kMaxQ1; ++t)
        tp.p[t] = make_float2(t < kMaxQ1 ? taps.w[t] : 0.f, t > 0 ? taps.w[t - 1] : 0.f);
    launch_kernel(conv1d_f32_kernel<DESIGN, Q, WARPS, K>, grid, G::kThreads, s, a, taps, tp, status_word);
    return cudaGetLastError();
}

template <int DESIGN>
cudaError_t launch_conv1d_f32(const Conv1DArgs &a, const float *w, int q, unsigned *status_word, cudaStream_t s,
                              int *launches)
{
    Taps1D taps;
    for (int k = 0; k < kMaxQ1; ++k) taps.w[k] = k < q ? w[k] : 0.f;
    cudaError_t err = kNoInstantiation;
    switch (q) {
#define SYSCONV_CASE(QQ) case QQ: err = launch_conv1d_f32_q<DESIGN, QQ>(a, taps, status_word, s); break;
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
