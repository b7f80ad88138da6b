/*
 * sysconv -- 1-D and 2-D valid-mode convolution executed as linear software
 * systolic arrays on the lanes of a warp (NVIDIA B200, sm_100a).
 *
 * C ABI of libsysconv.so.  Plain pointers and sizes only.
 *
 * The operation (correlation form, no filter flip, valid mode only):
 *
 *   1-D, Eq. 2 of the paper:   y[c]    = sum_{k<Q}           w[k]    * x[c + k],       c in [0, N-Q]
 *   2-D, Eq. 3 of the paper:   y[r][c] = sum_{p<P} sum_{q<Q} w[p][q] * x[r+p][c+q],
 *                              r in [0, H-P], c in [0, W-Q]
 *
 * Each call picks one of the paper's systolic designs (Section 3.1, Table 2,
 * Section 5); all designs produce the same sums, they differ in which operand
 * stays in a processing element and which one moves between neighbours:
 *
 *   SYSCONV_WS  weight-stationary  = BSM: inputs broadcast, weights stay, partial sums migrate
 *   SYSCONV_OS  output-stationary  = FBS: inputs forwarded, weights broadcast, partial sums stay
 *   SYSCONV_IS  input-stationary   = SBM: inputs stay, weights broadcast, partial sums migrate
 *
 * (The paper gives SBM and FBS in 2-D; the 2-D weight-stationary design is this
 * library's own extension of BSM: PE q keeps filter column q.)
 *
 * Data types:
 *   SYSCONV_F32       x, w, y are float; fp32 fused multiply-add accumulation
 *   SYSCONV_U8S8_S32  x is uint8 (zero-extended), w is int8 (sign-extended),
 *                     y is int32 with exact int32 accumulation
 *
 * Conventions common to every entry point
 *   - Layout: row-major, the column index c is contiguous; pitches and batch
 *     strides are in ELEMENTS of the respective array (not bytes).
 *   - The filter pointer is HOST memory: w[k] in 1-D, w[p*Q + q] in 2-D.  It is
 *     copied by value into the launch, so it may be freed or changed as soon as
 *     the call returns.
 *   - Ownership: the caller owns every buffer.  The library allocates no
 *     device memory.  State kept between calls: a launch counter, one status
 *     word in device memory per GPU (see sysconv_device_status) and, after the
 *     first pipelined host-buffer call on a GPU, two helper streams and a few
 *     events for that GPU.
 *   - Asynchrony: the work is enqueued on `stream` (a cudaStream_t passed as
 *     void*, NULL = the default stream); the call does not synchronise.
 *   - x and y must not overlap.
 *   - Supported sizes: 1-D: 1 <= Q <= 32.  2-D: 1 <= P <= 15 and 1 <= Q <= 15.
 *     Any N, W, H, batch >= 1 that fit the index types; any pitch >= row length.
 *     Pointers need only be aligned to their element type (16-byte aligned
 *     rows run faster).
 *   - Non-finite fp32 inputs (Inf, NaN): an input outside an output's window
 *     never enters its sum, with two exceptions that pad with zero taps and
 *     would multiply them by the non-finite value: the 2-D output-stationary
 *     kernels with 12 or more filter rows (the output rows directly above and
 *     below the affected rows may turn NaN) and the 2-D weight-stationary
 *     kernel used for small problems (fewer than 592 blocks of 128 output rows
 *     x 128 output columns over all images) when q is not a multiple of 4 (up
 *     to three outputs to the left of the affected columns may turn NaN).
 *     Finite data is unaffected.
 *   - Errors: every function returns a sysconv_status; nothing throws, aborts
 *     or traps.  SYSCONV_EINVAL: null pointer, non-positive size, filter larger
 *     than the input, pitch/stride smaller than the row/array, unknown enum.
 *     SYSCONV_EUNSUPPORTED: filter size outside the compiled range, or one of
 *     the designs FSM/BFS/FFS asked for anything but 1-D fp32.
 *     SYSCONV_ECUDA: the CUDA runtime reported an error at launch.
 */
#ifndef SYSCONV_H_
#define SYSCONV_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SYSCONV_OK = 0,
    SYSCONV_EINVAL = 1,
    SYSCONV_EUNSUPPORTED = 2,
    SYSCONV_ECUDA = 3,
    SYSCONV_ETIMEOUT = 4,
    SYSCONV_ETOOLARGE = 5 /* problem exceeds the built-in staging area of sysconv1d_host_static */
} sysconv_status;

typedef enum {
    SYSCONV_WS = 0,  /* BSM */
    SYSCONV_OS = 1,  /* FBS */
    SYSCONV_IS = 2,  /* SBM */
    /* the paper's other three 1-D designs (Table 2); 1-D fp32 only, built unfolded (one PE per lane,
     * CheckTime on) as faithful renderings: expect a fraction of the speed of the three above */
    SYSCONV_FSM = 3, /* inputs forwarded (2-step delay), weights stay, sums migrate */
    SYSCONV_BFS = 4, /* inputs broadcast, weights forwarded, sums stay */
    SYSCONV_FFS = 5  /* inputs forwarded, weights forwarded (2-step delay), sums stay */
} sysconv_design;

typedef enum {
    SYSCONV_F32 = 0,
    SYSCONV_U8S8_S32 = 1
} sysconv_dtype;

/*
 * 1-D convolution, Eq. 2.  `batch` independent signals share one filter:
 * signal b starts at x_dev + b*x_batch_stride and holds n elements; its n-q+1
 * outputs go to y_dev + b*y_batch_stride.
 *   x_dev, y_dev   DEVICE pointers (float/float or uint8/int32 by dtype)
 *   w_host         HOST pointer to q taps (float or int8 by dtype)
 *   strides        in elements; ignored when batch == 1 (pass 0 or anything)
 */
int sysconv1d(const void *x_dev, long long n, long long x_batch_stride,
              const void *w_host, int q,
              void *y_dev, long long y_batch_stride, int batch,
              int dtype, int design, void *stream);

/*
 * 2-D convolution, Eq. 3.  Image b starts at x_dev + b*x_batch_stride, has
 * `height` rows of `width` elements, rows x_pitch elements apart.  The
 * (height-p+1) x (width-q+1) outputs of image b go to y_dev + b*y_batch_stride,
 * rows y_pitch elements apart.  `q` is the filter WIDTH (pairs with columns),
 * `p` the filter HEIGHT; w_host holds p*q taps, w[pp*q + qq].
 */
int sysconv2d(const void *x_dev, int width, int height, long long x_pitch, long long x_batch_stride,
              const void *w_host, int q, int p,
              void *y_dev, long long y_pitch, long long y_batch_stride, int batch,
              int dtype, int design, void *stream);

/*
 * Strided forms: y(c) = sum_q x(stride*c + q) w(q) with (n-q)/stride + 1 outputs per signal (the stride-2
 * FBS design of Table 2), and y(r, c) = sum_p sum_q x(stride_r*r + p, stride_c*c + q) w(p, q) with
 * ((height-p)/stride_r + 1) x ((width-q)/stride_c + 1) outputs per image (Section 5 runs the strided
 * design row by row).  All other arguments as for sysconv1d / sysconv2d.
 * Stride 1 is the unstrided call.  fp32 data only.
 *   - stride 2 (both directions in 2-D), SYSCONV_OS and SYSCONV_IS, q <= 32 in 1-D, p, q <= 7 in 2-D: the
 *     fully unrolled stride-2 arrays.
 *   - any other strides (3, 4, ..., different strides per direction, stride 2 with larger filters up to
 *     15 x 15), SYSCONV_OS only: the same output-stationary array with run-time strides -- the stride-2 cell's
 *     X(c,q) = X(c+1, q-2) read as X(c+1, q-stride).  Slower than the unrolled kernels; 1-D signals need
 *     n < 2^31 there.
 *   batch <= 65535.  Every other combination (integer data, the weight-stationary design, SYSCONV_IS beyond the
 *   first case, the designs FSM/BFS/FFS) returns SYSCONV_EUNSUPPORTED; strides below 1: SYSCONV_EINVAL.
 */
int sysconv1d_strided(const void *x_dev, long long n, long long x_batch_stride,
                      const void *w_host, int q, int stride,
                      void *y_dev, long long y_batch_stride, int batch,
                      int dtype, int design, void *stream);
int sysconv2d_strided(const void *x_dev, int width, int height, long long x_pitch, long long x_batch_stride,
                      const void *w_host, int q, int p, int stride_c, int stride_r,
                      void *y_dev, long long y_pitch, long long y_batch_stride, int batch,
                      int dtype, int design, void *stream);

/*
 * Separable 2-D convolution, a second workload on the same folded array:
 *   y[r][c] = sum_{i<p} sum_{k<q} u[i] * v[k] * x[r+i][c+k]
 * i.e. sysconv2d with the rank-one filter w[i][k] = u[i]*v[k] (Gaussian blur, box, Sobel, ...), computed as one
 * 1-D output-stationary (FBS) pass with the horizontal taps v per input row (Section 6's "multiple FBS 1-D
 * convolutions") whose result feeds the p partial output rows through the vertical taps u: p + q
 * multiply-adds per output instead of p * q.  The intermediate row is rounded to fp32 once.
 *   u_host  HOST pointer to the p vertical taps (filter rows),  v_host  HOST pointer to the q horizontal taps
 *   everything else as for sysconv2d; fp32 only, 1 <= p, q <= 15, batch <= 65535 (SYSCONV_EUNSUPPORTED beyond).
 */
int sysconv2d_separable(const void *x_dev, int width, int height, long long x_pitch, long long x_batch_stride,
                        const void *u_host, int p, const void *v_host, int q,
                        void *y_dev, long long y_pitch, long long y_batch_stride, int batch, void *stream);

/*
 * Iterated 3x3 stencil, a second workload on the same folded array (Section 1 of the paper names stencils
 * beside convolution as what systolic arrays on GPUs are for; it evaluates none).
 *
 *   one sweep:  v[r][c] = sum_{dr,dc in {-1,0,1}} k[dr+1][dc+1] * u[r+dr][c+dc]   for 0 < r < height-1, 0 < c < width-1
 *               v[r][c] = u[r][c]                                                  on the outermost ring (fixed values)
 *   out = the sweep applied `sweeps` times (Jacobi iteration: every sweep reads only the previous sweep's grid).
 *
 * Columns are the PE dimension, inputs are forwarded between neighbouring PEs by shuffles as in the
 * output-stationary convolution, and up to four sweeps are fused in one pass over the grid (time levels kept in
 * PE registers), so the grid is read and written once per four sweeps.  Intermediate levels are rounded to fp32.
 *   u_dev, out_dev   DEVICE pointers, fp32, `batch` grids of height x width, rows pitch / out_pitch elements
 *                    apart, grids batch_stride / out_batch_stride elements apart (ignored when batch == 1)
 *   k_host           HOST pointer to the nine coefficients, row-major k[dr+1][dc+1]; with all four corner
 *                    coefficients zero (five-point stencil) their multiply-adds are skipped
 *   sweeps           >= 1.  More than four sweeps run as a chain of launches whose intermediate grids alternate
 *                    between out_dev and scratch_dev.
 *   scratch_dev      DEVICE buffer with the size and layout of the output; needed only when sweeps > 4 (may be NULL
 *                    otherwise); its contents are overwritten
 * u and out (and scratch) must not overlap.  batch <= 65535 (SYSCONV_EUNSUPPORTED beyond).  Grids with fewer than
 * three rows or columns have no interior: the output is a copy of the input.
 */
int sysstencil2d(const void *u_dev, int width, int height, long long pitch, long long batch_stride,
                 const void *k_host, int sweeps,
                 void *out_dev, long long out_pitch, long long out_batch_stride, int batch,
                 void *scratch_dev, void *stream);

/*
 * Generic space-time-transform executor (Sections 2.1-2.2 and the generic code pattern of Section 4).
 * The 1-D convolution UREs over the iteration space (c, q) are mapped by PE = p_c*c + p_q*q and
 * time = s_c*c + s_q*q; the dependences, delays and PE distances are derived from (P, s) alone, so the six
 * designs of Section 3.1 / Table 2 are (P; s) = SBM (1 1; 0 1), BSM (0 1; 1 1), FSM (0 1; 1 -1),
 * BFS (1 0; 1 1), FFS (1 0; 2 1), FBS (1 0; 0 1), and any other valid transform runs too.  One PE per
 * lane, register histories as deep as the delays, CheckTime on: a reference rendering, a small fraction of
 * the speed of the folded kernels behind sysconv1d.
 *
 * sysconv_spacetime_describe (host only, no CUDA call): checks the validity conditions and reports
 *   info[0..5]  PE distance and delay (in steps; 0 = broadcast) of the input, weight and partial-sum
 *               dependences, info[6] outputs per array, info[7] PEs per array, info[8] time steps per array,
 *               info[9] det(P; s);  name: the design letters (input B/F/S, weight B/F/S, sums M/S) + NUL.
 *   info and name may be NULL.  Returns SYSCONV_EINVAL for a transform that breaks a validity condition
 *   (P and s linearly dependent; sums that would accumulate within one time step) or q outside 1..32,
 *   SYSCONV_EUNSUPPORTED for a valid one the executor does not cover (a delay above 4 steps, more than
 *   32 PEs for one output).
 * sysconv1d_spacetime: y_dev[c] = sum_k w_host[k] * x_dev[c+k], c < n-q+1, fp32, one signal, through that
 *   array.  x_dev, y_dev DEVICE pointers, w_host HOST pointer; asynchronous on `stream`.
 */
int sysconv_spacetime_describe(int p_c, int p_q, int s_c, int s_q, int q, int *info, char *name);
int sysconv1d_spacetime(const void *x_dev, long long n, const void *w_host, int q, void *y_dev,
                        int p_c, int p_q, int s_c, int s_q, void *stream);

/*
 * The same two operations for callers whose data lives in HOST memory
 * (densely packed: pitch = row length, batch stride = array size).  The call
 * enqueues the host-to-device copy of x into the caller's device workspace,
 * the kernel(s), and the device-to-host copy of y, ordered after the work
 * already in `stream` and before work enqueued in `stream` later; it does not
 * synchronise (synchronise the stream before reading y_host).  Large problems
 * (a long single signal, several images, a large single image) are cut into up
 * to 16 chunks whose copy in, kernel and copy out overlap on two helper
 * streams of the library (the kernels run on `stream`); this needs page-locked
 * host buffers to be effective.  sysconv1d_host_plain is the unchunked form:
 * one copy in, one kernel, one copy out, everything on `stream`, no helper
 * streams or events.
 *   workspace_dev / workspace_bytes   DEVICE scratch owned by the caller, at
 *       least sysconv*_host_workspace_bytes(...) bytes, 256-byte aligned.
 * Returns SYSCONV_EINVAL if the workspace is too small.
 */
long long sysconv1d_host_workspace_bytes(long long n, int q, int batch, int dtype);
long long sysconv2d_host_workspace_bytes(int width, int height, int q, int p, int batch, int dtype);

int sysconv1d_host(const void *x_host, long long n, const void *w_host, int q,
                   void *y_host, int batch, int dtype, int design,
                   void *workspace_dev, long long workspace_bytes, void *stream);

int sysconv1d_host_plain(const void *x_host, long long n, const void *w_host, int q,
                         void *y_host, int batch, int dtype, int design,
                         void *workspace_dev, long long workspace_bytes, void *stream);

int sysconv2d_host(const void *x_host, int width, int height, const void *w_host, int q, int p,
                   void *y_host, int batch, int dtype, int design,
                   void *workspace_dev, long long workspace_bytes, void *stream);

/*
 * Several filters / designs over ONE host signal in one call (the shape of an experiment of the paper: the same
 * input through every design and filter size).  The signal crosses to the device once; job j convolves it with
 * the q[j] taps at w_host[j] by design[j] and its n-q[j]+1 outputs go to y_host[j].  Chunked like
 * sysconv1d_host: the copy in of chunk c+1, the kernels of chunk c and the copies out of chunk c-1 overlap.
 *   count                  1 .. 64 jobs;  w_host, y_host: HOST arrays of `count` HOST pointers;  q, design: HOST
 *                          arrays of `count` ints
 *   workspace_dev / bytes  at least sysconv1d_host_multi_workspace_bytes(n, q, count, dtype), 256-byte aligned
 * The y_host[j] must not overlap each other or x_host.  fp32 only (SYSCONV_EUNSUPPORTED otherwise).
 */
long long sysconv1d_host_multi_workspace_bytes(long long n, const int *q, int count, int dtype);
int sysconv1d_host_multi(const void *x_host, long long n, int count,
                         const void *const *w_host, const int *q, const int *design, void *const *y_host,
                         int dtype, void *workspace_dev, long long workspace_bytes, void *stream);

/*
 * sysconv1d_host for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is a packaging variant, not a systolic design.)
 *
 * Who needs it: code that runs where the CUDA allocator is off limits -- a plug-in
 * inside an application that has handed the whole device to its own memory arena,
 * a steady-state real-time loop where cudaMalloc (which serialises the device and
 * can fail late) is banned, a process whose memory budget was fixed at start-up.
 * Such a caller cannot supply the device workspace sysconv1d_host asks for.
 *
 * This entry point takes the same host buffers and stages them in a fixed array
 * that is part of the library's device image, so it allocates nothing: no
 * cudaMalloc/cudaFree, no allocating library call (it runs the plain sequence of
 * sysconv1d_host_plain, so it creates no streams or events either).  Same
 * arguments and results as sysconv1d_host, minus the workspace.
 *   - Limit: sysconv1d_host_workspace_bytes(n, q, batch, dtype) must not exceed
 *     sysconv_static_scratch_bytes() (16 MiB: about 2 Mi fp32 samples in one
 *     signal, or the same total over a batch).  Larger problems return
 *     SYSCONV_ETOOLARGE and enqueue nothing.
 *   - Cost: every GPU on which this library is loaded holds those 16 MiB until
 *     the process exits, whether or not this function is ever called.
 *   - The first call on each device resolves the array's device address (once,
 *     with that device current); make that first call outside any stream capture.
 *   - All calls on one device share the one array: calls whose work overlaps on
 *     the GPU (different streams, or threads, without ordering between them)
 *     race on it.  Issue them on one stream or order them yourself.  Nothing in
 *     the array needs clearing between calls: inputs are fully overwritten and
 *     every output is written before it is copied back.
 */
long long sysconv_static_scratch_bytes(void);
int sysconv1d_host_static(const void *x_host, long long n, const void *w_host, int q,
                          void *y_host, int batch, int dtype, int design, void *stream);

/* Text for a sysconv_status / sysconv_design value ("?" if unknown). Static storage. */
const char *sysconv_status_string(int status);
const char *sysconv_design_name(int design);

/*
 * Device-side health check.  The pipelined kernels wait for their asynchronous
 * copies with a bounded number of polls; a kernel whose limit runs out stops
 * taking work, raises a flag in device memory and returns normally (its outputs
 * are then incomplete).  This call synchronises the current device (every
 * stream, cudaDeviceSynchronize), returns SYSCONV_ETIMEOUT if the flag was
 * raised since the last call (and clears it), SYSCONV_OK otherwise.
 */
int sysconv_device_status(void);

/*
 * Self-test of that mechanism (no counterpart in the paper; for the test suite).
 * Enqueues one small block on `stream` that arms a shared-memory barrier for
 * bytes which are never sent -- it issues no copy, so nothing is in flight
 * towards it -- polls 1024 times, gives up the way the pipelined kernels do
 * (raises the flag, returns normally) and ends.  The next
 * sysconv_device_status() must return SYSCONV_ETIMEOUT, the one after it
 * SYSCONV_OK.  Touches no caller memory.
 */
int sysconv_selftest_wait_timeout(void *stream);

/*
 * Measured denominators for roofline figures (no counterpart in the paper, which reports only ratios to its
 * own baseline; Section 6 explains its results by lane utilisation, which is what these rates normalise).
 *
 * sysconv_measure_peaks runs, on the current device, one block per SM that issues a long unrolled run of one
 * kind of instruction and times itself with the SM's cycle counter, and a 128-bit streaming copy over the
 * scratch buffer timed with CUDA events.  results_host[...] (at least SYSCONV_PEAK_COUNT doubles):
 *   SYSCONV_PEAK_FFMA    fp32 fused multiply-adds per clock per SM
 *   SYSCONV_PEAK_FFMA2   fp32 multiply-adds per clock per SM through the packed fp32x2 FMA, multiplicand (x, x)
 *   SYSCONV_PEAK_IMAD    32-bit integer multiply-adds per clock per SM
 *   SYSCONV_PEAK_DP4A    dp4a instructions per clock per SM (x 4 for 8-bit multiply-adds)
 *   SYSCONV_PEAK_SHFL    warp-shuffle lane transfers per clock per SM
 *   SYSCONV_PEAK_COPY_GBS  bytes read + written per second by the copy, in GB/s
 *   SYSCONV_PEAK_SM_COUNT  SMs of the device
 * scratch_dev: DEVICE memory owned by the caller, 256-byte aligned, at least 64 MiB (use several hundred MiB so
 * that the copy is larger than the L2 cache); its contents are overwritten.  Synchronises the device; takes
 * a few milliseconds.  SYSCONV_EINVAL for a null/small/misaligned buffer or count < SYSCONV_PEAK_COUNT.
 *
 * sysconv_floor_copy enqueues ONE plain streaming kernel on `stream`: widen == 0 copies bytes_in bytes from
 * src_dev to dst_dev; widen == 1 reads bytes_in uint8 values and writes them as int32 (4 * bytes_in bytes).
 * It moves the bytes of a convolution of that size and does none of its arithmetic: timed beside the
 * convolution kernels it shows what a launch of that size costs at best.  Both pointers 16-byte aligned,
 * bytes_in a multiple of 16, buffers must not overlap.
 */
enum {
    SYSCONV_PEAK_FFMA = 0,
    SYSCONV_PEAK_FFMA2 = 1,
    SYSCONV_PEAK_IMAD = 2,
    SYSCONV_PEAK_DP4A = 3,
    SYSCONV_PEAK_SHFL = 4,
    SYSCONV_PEAK_COPY_GBS = 5,
    SYSCONV_PEAK_SM_COUNT = 6,
    SYSCONV_PEAK_COUNT = 7
};
int sysconv_measure_peaks(void *scratch_dev, long long scratch_bytes, double *results_host, int count);
int sysconv_floor_copy(const void *src_dev, void *dst_dev, long long bytes_in, int widen, void *stream);

/* Library version, major*10000 + minor*100 + patch. */
int sysconv_version(void);

/* Number of kernels this library has launched in this process so far. */
long long sysconv_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SYSCONV_H_ */
