/*
 * dsa3d.h - C ABI of the B200 (sm_100a) 3D Deformable Slide Attention library.
 *
 * The operator (paper, section "3D Deformable Slide Attention": Formulation, Eq. 1 second
 * term, and the softmax definition below Eq. 1; sampling as in "Implementation
 * considerations"):
 *
 *   Query token n = (t, y, x) on a (T, H, W) grid, head m, window (kt, kh, kw) with
 *   P = kt*kh*kw cells; cell p = (u*kh + v)*kw + w has the integer displacement
 *   b(p) = (u - kt/2, v - kh/2, w - kw/2) (integer division: a window of 2 covers {-1, 0},
 *   of 3 covers {-1, 0, 1}).  The sample position is
 *       pi = (t, y, x) + b(p) + offsets[n, m, p, :]            in grid-index units,
 *   formed in fp32 as float(coord + b) + offset.  K and V are sampled there by trilinear
 *   interpolation with zero padding: a corner outside the grid contributes nothing and
 *   the other corner weights are not renormalised.  Then
 *       s_p = q[n, m, :] . k_p / sqrt(d),  alpha = softmax over the P samples,
 *       out[n, m, :] = sum_p alpha_p v_p,  lse[n, m] = ln sum_p exp(s_p).
 *   A sample with no corner inside the grid (or a NaN/inf position) has k_p = v_p = 0 and
 *   s_p = 0; it still takes part in the softmax.  With all offsets zero the operator is
 *   fixed 3D sliding-window attention (paper, Ablations, "Effect of offsets").
 *   There is no causal mask.  dsa3d_forward / dsa3d_backward are that operator alone.  The
 *   layers Eq. 1 puts around it are separate entry points further down: the depthwise
 *   convolution (its first term, dsa3d_dwconv3d_* and dsa3d_forward_residual) and the linear
 *   layer of the offset predictor (dsa3d_offsets_linear_*), each with its backward.  The
 *   q/k/v projections are not part of this library.
 *
 * Layouts (row-major, channels last, one video per call; a batch is one call per item):
 *   q, k, v, out, dout, dq, dk, dv : [T, H, W, heads, d]     element type = `dtype`
 *   offsets, doffsets              : [T, H, W, heads, P, 3]  fp32, last axis (t, y, x)
 *   lse                            : [T, H, W, heads]        fp32
 *
 * Pointers.  Unless a parameter says HOST, every pointer is a DEVICE pointer owned by the
 * caller, contiguous and 16-byte aligned.  The library does not allocate, free or keep
 * them.  Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 * default stream); the buffers must stay valid until the stream has run the work.
 * Outputs are fully overwritten.  Inputs and outputs must not alias.
 *
 * Supported: dtype DSA3D_F32 or DSA3D_BF16; d in {32, 64, 128}; 1 <= P <= 256;
 * T, H, W, heads >= 1; T*H*W < 2^31.  Arithmetic is fp32 whatever the storage type.
 *
 * Non-finite values.  dsa3d_forward and dsa3d_backward confine a NaN or infinity in a row of q, k, v or dout to
 * the results that row enters by the definition above.  The tile kernels behind the fixed-window and
 * bounded-offsets entry points form dense products over the region of a 4 x 4 x 8 tile, in which such a row is
 * multiplied by zero weights as well: there it can reach every output of the tiles whose region holds the row.
 * Finite inputs are not affected.
 *
 * Errors.  Every function returns a dsa3d_status (0 = success).  Arguments are checked
 * before anything is launched; nothing aborts, throws or traps.
 *
 * Experiment switches.  A few environment variables, read on each call, select an alternative
 * kernel for the same result (they exist to measure one variant against another; none changes
 * what is computed beyond fp32 summation order):
 *   DSA3D_TILE="tt,ty,tx,halo"     query tiling of the dK/dV pre-reduction of dsa3d_backward
 *                                  (default 4,8,8,6; "0" = no tiling, every contribution is an
 *                                  atomic add); also changes dsa3d_backward_workspace_bytes
 *   DSA3D_KEY_BLOCKS=1             dsa3d_backward (bf16, d = 64 or 128) forms dK/dV per
 *                                  block of 4 x 8 x 8 keys as tensor-core products (coefficient matrix of the
 *                                  block against chunks of 32 queries, tcgen05 in tf32: the coefficients lose
 *                                  the bits below 2^-10 relative, q and dO none) instead of the tile kernel's
 *                                  binning (the gather kernel then lists every sample per key block); slower
 *                                  so far; also changes dsa3d_backward_workspace_bytes; a
 *                                  non-finite q or dO row then reaches every key whose block it lies near
 *   DSA3D_NO_TENSOR_FIXED_WINDOW   dsa3d_forward_fixed_window and dsa3d_forward_bounded_offsets use the general
 *                                  kernel, dsa3d_backward_bounded_offsets the kernels of dsa3d_backward;
 *                                  dsa3d_backward_fixed_window uses its per-row CUDA-core kernels only
 *                                  (no dot-product tables, no tile kernels)
 *   DSA3D_GEMM_ONE_CTA             dsa3d_offsets_linear_forward: one CTA per tile instead of a pair
 *   DSA3D_GEMM_PLAIN_STORES        its epilogue stores from registers instead of by TMA
 *   DSA3D_CONV_GENERAL             dsa3d_dwconv3d_*: the kernel for any size also for 3x3x3
 *   DSA3D_WGRAD_PLAIN              dsa3d_dwconv3d_backward: the unstaged weight-gradient kernel
 */
#ifndef DSA3D_H
#define DSA3D_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DSA3D_OK = 0,
    DSA3D_ERR_NULL_POINTER = 1,   /* a required pointer is NULL */
    DSA3D_ERR_BAD_SHAPE = 2,      /* a size is < 1 or the grid has 2^31 tokens or more */
    DSA3D_ERR_UNSUPPORTED = 3,    /* dtype, head dimension or window outside the supported set */
    DSA3D_ERR_MISALIGNED = 4,     /* a pointer is not 16-byte aligned */
    DSA3D_ERR_WORKSPACE = 5,      /* workspace missing or smaller than required */
    DSA3D_ERR_CUDA = 6,           /* a CUDA runtime call failed; see dsa3d_last_cuda_error */
    DSA3D_ERR_DEVICE_TIMEOUT = 7  /* a bounded wait inside a kernel ran out (dsa3d_check_device_timeout) */
} dsa3d_status;

typedef enum { DSA3D_F32 = 0, DSA3D_BF16 = 1 } dsa3d_dtype;

/*
 * Forward (Eq. 1 second term + softmax definition).  Reads q, k, v, offsets; writes out
 * and lse.  `window` is a HOST pointer to (kt, kh, kw).  No workspace.  dsa3d_forward and
 * dsa3d_backward only enqueue work on `stream` (kernels and a clear of the accumulators; no
 * allocation, no synchronisation), so they may be recorded into a CUDA graph by stream
 * capture and replayed.
 */
int dsa3d_forward(const void* q, const void* k, const void* v, const float* offsets,
                  int T, int H, int W, int heads, int d, const int window[3],
                  void* out, float* lse, int dtype, void* stream);

/*
 * Backward of the forward above (chain rule through sampling, softmax and weighted sum;
 * the paper trains through this operator by automatic differentiation and prints no
 * formulas).  Given dout = dLoss/dout and the lse saved by the forward, writes
 *   dq, dk, dv   same shape and type as q, k, v
 *   doffsets     same shape as offsets; the derivative of the trilinear weights, with the
 *                one-sided convention of the floor at integer positions (cell [i, i+1))
 * The sampling weights are recomputed, nothing of size N*P*d is stored.
 * `workspace` is device scratch of at least dsa3d_backward_workspace_bytes(...) bytes,
 * 16-byte aligned (bf16 storage: fp32 accumulators for dk and dv, two fp32 coefficients per
 * sample, and the bins of the tile pre-reduction; may be NULL when that size is 0).
 * Its contents on entry do not matter.  dk and dv are summed with floating-point atomics,
 * so their last bits can differ from run to run; dq, doffsets are deterministic.
 */
int dsa3d_backward(const void* q, const void* k, const void* v, const float* offsets,
                   const float* lse, const void* dout,
                   int T, int H, int W, int heads, int d, const int window[3],
                   void* dq, void* dk, void* dv, float* doffsets,
                   void* workspace, size_t workspace_bytes, int dtype, void* stream);

/* Scratch bytes dsa3d_backward needs for this problem (0 for DSA3D_F32; 0 also for
 * arguments the library would reject). */
size_t dsa3d_backward_workspace_bytes(int T, int H, int W, int heads, int d,
                                      const int window[3], int dtype);

/*
 * Batched forms (the paper trains with batch 1; a batch here is `batch` independent videos
 * stored back to back, [batch, T, H, W, heads, ...] for every tensor).  Videos never see
 * each other's keys: each is the operator of Eq. 1 on its own grid.  The calls run the
 * single-video kernels once per video on `stream`; the backward reuses one workspace of
 * dsa3d_backward_workspace_bytes(...) bytes for all of them.  Every per-video slice must
 * itself be 16-byte aligned (it is whenever T*H*W*heads is a multiple of 4).
 */
int dsa3d_forward_batch(const void* q, const void* k, const void* v, const float* offsets,
                        int batch, int T, int H, int W, int heads, int d, const int window[3],
                        void* out, float* lse, int dtype, void* stream);
int dsa3d_backward_batch(const void* q, const void* k, const void* v, const float* offsets,
                         const float* lse, const void* dout,
                         int batch, int T, int H, int W, int heads, int d, const int window[3],
                         void* dq, void* dk, void* dv, float* doffsets,
                         void* workspace, size_t workspace_bytes, int dtype, void* stream);

/*
 * One whole step from HOST buffers: copies q, k, v, offsets, dout to the device, runs the
 * forward and the backward above, and copies out, lse, dq, dk, dv, doffsets back.  This is
 * the operator of Eq. 1 (second term) and its gradient exactly as in dsa3d_forward /
 * dsa3d_backward; only the location of the buffers differs.
 * Every *_h pointer is a HOST pointer (page-locked memory makes the copies asynchronous
 * and fast; pageable memory works but serialises).  `arena` is DEVICE scratch of at least
 * dsa3d_step_host_arena_bytes(...) bytes, 256-byte aligned, which holds the device copies
 * and the backward workspace; the library allocates no memory.  The step is pipelined over
 * slabs of whole frames: K and V go up first, then each slab's q, offsets and dout while
 * earlier slabs compute, and each slab's out, lse, dq and doffsets come back while later
 * slabs compute; dk and dv follow the last slab.  This uses two side streams the library
 * creates on the calling thread's first call (with a few dozen events; they are kept for
 * the life of the thread); everything is ordered after the work
 * already in `stream`, and the step is complete when `stream` is.  The host buffers must
 * not be touched until then.  Not for use inside a stream capture.
 */
int dsa3d_step_host(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h,
                    const void* dout_h, int T, int H, int W, int heads, int d, const int window[3],
                    void* out_h, float* lse_h, void* dq_h, void* dk_h, void* dv_h, float* doffsets_h,
                    void* arena, size_t arena_bytes, int dtype, void* stream);

/*
 * dsa3d_step_host_pipelined: the same step, for a sequence of steps on one arena.  It differs
 * in ordering only: its uploads do not wait for the work already in `stream` but only for the
 * device buffers they overwrite, and nothing at its end makes `stream` wait for the downloads.
 * The next call's K and V (the arena holds two copies of each) and first slabs therefore go up
 * while this call's kernels run, and this call's dk and dv come down while the next call's
 * forward runs - the two transfers a single step cannot hide.  The host INPUT buffers must be
 * complete on the host when the call is made (no ordering with earlier work in `stream` is
 * implied for them); all host buffers of a call must stay untouched until
 * dsa3d_step_host_flush(stream) has been called and `stream` has completed, or until a later
 * pipelined call has been flushed.  Results of call i are final on the host no later than that.
 * The arena must not be in use by other work queued in `stream` (the uploads do not wait for it).
 * A call whose arena, shape or dtype differs from the previous one first waits for all of the
 * previous call.  dsa3d_step_host is this call followed by the flush, with the uploads ordered
 * after `stream`.  dsa3d_step_host_flush makes `stream` wait for every transfer the calling
 * thread's earlier steps queued.
 */
int dsa3d_step_host_pipelined(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h,
                              const void* dout_h, int T, int H, int W, int heads, int d, const int window[3],
                              void* out_h, float* lse_h, void* dq_h, void* dk_h, void* dv_h, float* doffsets_h,
                              void* arena, size_t arena_bytes, int dtype, void* stream);
int dsa3d_step_host_flush(void* stream);

/* Device scratch bytes dsa3d_step_host needs (0 for arguments the library would reject). */
size_t dsa3d_step_host_arena_bytes(int T, int H, int W, int heads, int d, const int window[3],
                                   int dtype);

/*
 * dsa3d_forward_host: the forward alone on HOST buffers (sampling / inference): q, k, v,
 * offsets in, out and lse back, pipelined over slabs of frames like dsa3d_step_host (K and V
 * go up first; a slab's q and offsets go up while earlier slabs compute and its out and lse
 * come back while later slabs compute).  `arena`: caller-owned DEVICE scratch of at least
 * dsa3d_forward_host_arena_bytes(...) bytes, 256-byte aligned.  Same side streams, ordering
 * and capture restriction as dsa3d_step_host.
 */
int dsa3d_forward_host(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h, int T, int H, int W,
                       int heads, int d, const int window[3], void* out_h, float* lse_h, void* arena,
                       size_t arena_bytes, int dtype, void* stream);
size_t dsa3d_forward_host_arena_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype);

/*
 * Backward without any caller-provided or allocated scratch (the paper has no counterpart;
 * this exists for deployment reasons only).  Meant for callers that cannot give the
 * library a workspace: code running where all device memory was planned ahead of time,
 * plug-ins whose host application owns the allocator, loops where cudaMalloc's implicit
 * device synchronisation is not acceptable.  Same inputs, outputs and results as
 * dsa3d_backward, but the fp32 dk/dv accumulators live in a fixed 64 MiB array inside the
 * library image (each GPU that loads the library holds it until the process exits), so:
 *   - T*H*W*heads*d must not exceed DSA3D_NOALLOC_MAX_ELEMENTS; larger problems are
 *     rejected with DSA3D_ERR_WORKSPACE before anything is launched;
 *   - the function calls no cudaMalloc / cudaFree and nothing else that allocates;
 *   - the first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current) and caches it for the life of the
 *     process; make that first call outside any stream capture.  The cached address does not
 *     survive a cudaDeviceReset (or any other teardown of the device's primary context): a
 *     process that resets a device must not call this function on it again;
 *   - all calls share the one array, which keeps the previous call's contents; every call
 *     clears it on `stream` before use.  Two calls whose GPU work can overlap (different
 *     streams, or different threads on one device) race on it and give wrong dk/dv:
 *     serialise them.
 */
#define DSA3D_NOALLOC_MAX_ELEMENTS (8u * 1024u * 1024u)
int dsa3d_backward_noalloc(const void* q, const void* k, const void* v, const float* offsets,
                           const float* lse, const void* dout,
                           int T, int H, int W, int heads, int d, const int window[3],
                           void* dq, void* dk, void* dv, float* doffsets, int dtype, void* stream);

/* DSA3D_NOALLOC_MAX_ELEMENTS as the loaded library was built. */
size_t dsa3d_backward_noalloc_max_elements(void);

/* cudaError_t of the most recent failed address lookup of dsa3d_backward_noalloc on the
 * calling thread (0 if none). */
int dsa3d_backward_noalloc_last_cuda_error(void);

/*
 * Timing hook (a measurement aid; the paper has no counterpart).  The six arguments are
 * cudaEvent_t handles created by the caller, or NULL.  While set (per calling thread),
 * dsa3d_forward records fwd_start / fwd_stop on its stream immediately around the forward
 * kernel, and dsa3d_backward records bwd_start / bwd_stop around its gather kernel and
 * scatter_start / scatter_stop around its tile scatter kernel (when that kernel runs), so a
 * caller can time those kernels alone inside a longer step.  Pass NULLs to switch it off.
 */
int dsa3d_set_profile_events(void* fwd_start, void* fwd_stop, void* bwd_start, void* bwd_stop,
                             void* scatter_start, void* scatter_stop);

/*
 * Ceiling probes (measurement aids; the paper has no counterpart).  The operator gathers and
 * scatters rows of a few hundred bytes, so what bounds it on a GPU is the rate of such
 * accesses out of L2 and the FMA issue rate rather than streaming bandwidth.  Each probe
 * launches one kernel on `stream` over a caller-owned DEVICE buffer and stores in its
 * HOST out-parameter the work of that launch; the caller times the launch.
 *   dsa3d_probe_gather : random 256-byte-row reads (16-byte loads, two rows per warp
 *                        step) spread over `working_set_bytes` of `buffer`; `iters` a
 *                        multiple of 8; *bytes_per_launch = bytes read.
 *   dsa3d_probe_red    : red.global.add.v4.f32 of zeros onto random 512-byte rows of
 *                        `buffer` (contents unchanged); *bytes_per_launch = operand bytes.
 *   dsa3d_probe_fma    : 64 FMAs per thread and iteration on registers; kind 0 = fp32 FMA,
 *                        kind 1 = bf16 x bf16 -> fp32 FMA; `seed_1kb` is any 1 KiB of
 *                        device memory; *fma_per_launch = FMAs executed.
 */
int dsa3d_probe_gather(const void* buffer, size_t working_set_bytes, int iters, double* bytes_per_launch,
                       void* stream);
int dsa3d_probe_red(void* buffer, size_t working_set_bytes, int iters, double* bytes_per_launch,
                    void* stream);
int dsa3d_probe_fma(const void* seed_1kb, int iters, int kind, double* fma_per_launch, void* stream);

/*
 * The layers around the operator in Eq. 1 (device pointers, asynchronous on `stream`, same
 * ownership rules as above).  The paper specifies them only as "a lightweight depthwise 3D
 * convolution followed by a linear layer" for the offsets (Formulation section) and as the
 * DWConv3D(X) term of Eq. 1, built from grouped nn.Conv3d and pointwise layers
 * (Implementation considerations); kernel size, padding and parameter layout below are this
 * library's choices.
 *
 * dsa3d_dwconv3d_forward: y[t,y,x,c] = bias[c] + sum over taps (i,j,l) of
 *   weight[(i*kh + j)*kw + l][c] * x[t + i - kt/2, y + j - kh/2, x + l - kw/2][c]
 * (cross-correlation, unit stride, zero outside the grid, integer division in the centring:
 * the same centring as the attention window).  x, y: [T,H,W,C] channels-last in `dtype`,
 * C a multiple of 8; weight fp32 [kt*kh*kw, C]; bias fp32 [C] or NULL; kernel = (kt,kh,kw),
 * HOST pointer, kt,kh <= 15, kw <= 7.  fp32 accumulation in tap order, one rounding to `dtype`.
 * y must not alias x.
 */
int dsa3d_dwconv3d_forward(const void* x, const float* weight, const float* bias, int T, int H, int W, int C,
                           const int kernel[3], void* y, int dtype, void* stream);

/*
 * dsa3d_offsets_linear_forward: offsets[n][o] = bias[o] + sum_c u[n][c] * w[o][c], the linear
 * layer of the offset predictor; with O = heads*P*3 the result is the offsets tensor of
 * dsa3d_forward.  u [tokens, C] and w [O, C] in `dtype` (row-major, C a multiple of 8),
 * bias fp32 [O], offsets fp32 [tokens, O]; tokens < 2^31.  bf16 runs on the tensor cores
 * (exact bf16 products, fp32 accumulation in the hardware's order); fp32 uses fp32 FMAs in
 * channel order.  Its waits on hardware barriers are bounded: if one ever runs out the
 * kernel stops early, the output is incomplete and dsa3d_device_timeout_flag() returns
 * non-zero afterwards.
 */
int dsa3d_offsets_linear_forward(const void* u, const void* w, const float* bias, long long tokens, int C, int O,
                                 float* offsets, int dtype, void* stream);

/*
 * Backward of the two layers above (gradients of a scalar loss L; the paper gives no formulas
 * for them: they follow from the definitions of the two forwards by the chain rule).
 *
 * dsa3d_dwconv3d_backward: with dy = dL/dy [T,H,W,C] in `dtype`,
 *   dx[s]        = sum over taps of weight[tap][c] * dy[s - displacement(tap)]   ([T,H,W,C], `dtype`),
 *   dweight[tap] = sum over positions s of x[s + displacement(tap)] * dy[s]      (fp32 [kt*kh*kw, C]),
 *   dbias[c]     = sum over positions of dy[s][c]                                 (fp32 [C]),
 * zero outside the grid as in the forward.  dx, dweight and dbias may each be NULL (not
 * computed; dbias needs dweight); x is read only for dweight, weight only for dx.  dx is one
 * fp32 accumulation in tap order and one rounding; dweight and dbias are fp32 sums whose order
 * varies from run to run (atomic adds of per-warp partial sums).  workspace: device memory of
 * dsa3d_dwconv3d_backward_workspace_bytes(C, kernel) bytes (needed for dx only), contents
 * undefined afterwards.  dx must not alias dy.
 */
size_t dsa3d_dwconv3d_backward_workspace_bytes(int C, const int kernel[3]);
int dsa3d_dwconv3d_backward(const void* x, const float* weight, const void* dy, int T, int H, int W, int C,
                            const int kernel[3], void* dx, float* dweight, float* dbias, void* workspace,
                            size_t workspace_bytes, int dtype, void* stream);

/*
 * dsa3d_offsets_linear_backward: with doffsets = dL/doffsets (fp32 [tokens, O], e.g. the
 * doffsets of dsa3d_backward),
 *   du[n][c] = sum_o doffsets[n][o] * w[o][c]     ([tokens, C] in `dtype`),
 *   dw[o][c] = sum_n doffsets[n][o] * u[n][c]     (fp32 [O, C]),
 *   dbias[o] = sum_n doffsets[n][o]               (fp32 [O]).
 * Each output may be NULL (not computed).  bf16: doffsets is rounded to bf16 once and both
 * contractions run on the tensor cores with fp32 accumulation (slabs of 262144 tokens, dw
 * accumulated over slabs and k-ranges with fp32 atomic adds, so its summation order varies);
 * dbias is summed from the fp32 doffsets.  fp32: plain fp32 FMAs.  workspace: device memory of
 * dsa3d_offsets_linear_backward_workspace_bytes(...) bytes (0 for fp32), contents undefined
 * afterwards.  Bounded waits as in the forward (dsa3d_device_timeout_flag).
 */
size_t dsa3d_offsets_linear_backward_workspace_bytes(long long tokens, int C, int O, int dtype);
int dsa3d_offsets_linear_backward(const void* u, const void* w, const float* doffsets, long long tokens, int C, int O,
                                  void* du, float* dw, float* dbias, void* workspace, size_t workspace_bytes, int dtype,
                                  void* stream);

/* Synchronises with the device and returns the flag described above (0: no wait ever ran
 * out; -1: the flag could not be read). */
int dsa3d_device_timeout_flag(void);
/* The same check as a status: synchronises with the device and returns DSA3D_OK, or
 * DSA3D_ERR_DEVICE_TIMEOUT if any kernel of the library launched so far gave up a bounded wait
 * (its outputs are then incomplete), or DSA3D_ERR_CUDA if the flag could not be read. */
int dsa3d_check_device_timeout(void);
/* Resets the flag to 0 (synchronises with the device).  The flag is sticky: once a wait has run
 * out, every later check reports it until this is called.  Call it after handling a
 * DSA3D_ERR_DEVICE_TIMEOUT, with no kernel of the library in flight. */
int dsa3d_clear_device_timeout(void);
/* TEST AID, not part of the operator (the paper has no counterpart).  Launches, on `stream`, one
 * warp in which a single thread waits on a hardware barrier that nothing ever arrives at, polling
 * at most `polls` times (1 .. 2^20), exactly like the bounded waits of the tensor-core kernels;
 * the wait then gives up, the thread sets the timeout flag to 99 and the kernel returns normally.
 * Nothing traps or spins without a limit.  It lets a caller (and the test-suite) exercise the
 * path dsa3d_check_device_timeout -> DSA3D_ERR_DEVICE_TIMEOUT -> dsa3d_clear_device_timeout. */
int dsa3d_test_wait_timeout(unsigned polls, void* stream);

/*
 * dsa3d_forward_residual: Eq. 1 with its first term: out = residual + attention output,
 * where `residual` ([T,H,W,heads,d] in `dtype`, e.g. the result of dsa3d_dwconv3d_forward
 * on the layer input with C = heads*d) is added in fp32 before the one rounding to `dtype`.
 * `residual` may be the same buffer as `out`.  Everything else as dsa3d_forward; the
 * gradient of the loss with respect to `residual` is dout itself, so dsa3d_backward is
 * unchanged.
 */
int dsa3d_forward_residual(const void* q, const void* k, const void* v, const float* offsets, const void* residual,
                           int T, int H, int W, int heads, int d, const int window[3], void* out, float* lse,
                           int dtype, void* stream);

/*
 * dsa3d_forward_fixed_window: the operator with every offset equal to zero (the fixed local
 * window of the ablation on the effect of offsets) without an offsets tensor: same out and
 * lse as dsa3d_forward on an all-zero offsets tensor, up to fp32 summation order.  For bf16,
 * d = 64 or 128 it runs as dense tile attention on the tensor cores: windows (3,3,3) and (2,2,2)
 * with the scores of a 4x4x8 query tile against its whole halo region in one tcgen05 tile, window
 * mask, softmax and the weighted sum from shared memory; windows (3,5,5) and (3,7,7) (the paper's
 * own) one region plane at a time with the weighted sum on the tensor cores too, each fp32 weight
 * entering as a bf16 head plus a bf16 remainder.  Every other supported shape runs the general
 * kernel with zero offsets.  The environment variable DSA3D_NO_TENSOR_FIXED_WINDOW forces the
 * general kernel.  The backward of this variant is dsa3d_backward with a zero offsets
 * tensor.  Bounded waits as in dsa3d_offsets_linear_forward (dsa3d_device_timeout_flag).
 */
int dsa3d_forward_fixed_window(const void* q, const void* k, const void* v, int T, int H, int W, int heads, int d,
                               const int window[3], void* out, float* lse, int dtype, void* stream);

/*
 * dsa3d_forward_bounded_offsets: dsa3d_forward for callers whose learned offsets are small perturbations
 * of the fixed window (Formulation: the window positions shifted by learned offsets; the ablation on the
 * effect of offsets compares them with the fixed window).  Same arguments, same out and lse (up to fp32
 * summation order).  A first kernel checks the offsets tensor; if every component is finite and below 1
 * in size, every corner of every sample lies in the box "window grown by one position on each side" and
 * the operator runs as dense tile attention on the tensor cores for bf16, d = 64 or 128 and window (3,3,3):
 * scores of a 4x4x8 query tile against its region by tcgen05, plane by plane; each logit the trilinear
 * combination of eight entries of the score tile; the softmax weights times the corner weights summed
 * per box position; the weighted sum as a second tcgen05 product (weights as bf16 head + remainder).
 * Otherwise - some offset too large, or another shape - the general kernel runs, so the call is correct
 * for any offsets; the decision is taken on the device, the call stays asynchronous.  Calls that are in
 * flight at the same time each use their own gate word (out of 1024).  The environment variable
 * DSA3D_NO_TENSOR_FIXED_WINDOW forces the general kernel.  Bounded waits as in
 * dsa3d_offsets_linear_forward (dsa3d_device_timeout_flag).  The backward of such a call is
 * dsa3d_backward_bounded_offsets (or dsa3d_backward).
 */
int dsa3d_forward_bounded_offsets(const void* q, const void* k, const void* v, const float* offsets, int T, int H, int W,
                                  int heads, int d, const int window[3], void* out, float* lse, int dtype, void* stream);

/*
 * dsa3d_backward_bounded_offsets: dsa3d_backward for the same callers.  Same arguments, same dq, dk, dv and
 * doffsets (up to fp32 summation order; the coefficients of dq, dk and dv enter their products as a bf16
 * head plus a bf16 remainder, relative error 2^-17).  The offsets tensor is checked on the device as in
 * dsa3d_forward_bounded_offsets.  If every component is finite and below 1 in size (bf16, d = 64 or 128,
 * window (3,3,3)) no row is gathered or scattered one by one: a tcgen05 kernel leaves, per (query, head),
 * the dot products q.K_j and dO.V_j of the 6 x 6 x 6 grid positions from query - 2; a second kernel forms
 * every sample's logit, dO.V and their derivatives as trilinear combinations of eight of them (cell and
 * fractions exactly as dsa3d_backward forms them), alpha from `lse`, delta, dS, doffsets, and sums the
 * coefficients of the samples' corners per grid position into a 5 x 5 x 5 box; dq, dk and dv are then the
 * sums of a fixed (5,5,5) window with those coefficients, plane-by-plane tcgen05 products as in
 * dsa3d_backward_fixed_window.  Otherwise the kernels of dsa3d_backward run (they are queued behind the
 * others and do nothing when the check passed), so the call is correct for any offsets and stays
 * asynchronous.  dk and dv of the tile route are written once in `dtype` (no atomics, bitwise deterministic).
 * `workspace`: dsa3d_backward_bounded_offsets_workspace_bytes(...) bytes (for the tile route 2.7 KB per
 * (token, head): the tables and the coefficient boxes), 16-byte aligned, contents undefined afterwards.
 * Other shapes and dtypes, grids of 2^31 / (125 heads) tokens or more, and the switches
 * DSA3D_NO_TENSOR_FIXED_WINDOW and DSA3D_KEY_BLOCKS=1, make it dsa3d_backward.  Bounded waits as in dsa3d_offsets_linear_forward (dsa3d_device_timeout_flag).
 */
int dsa3d_backward_bounded_offsets(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                                   const void* dout, int T, int H, int W, int heads, int d, const int window[3], void* dq,
                                   void* dk, void* dv, float* doffsets, void* workspace, size_t workspace_bytes, int dtype,
                                   void* stream);
size_t dsa3d_backward_bounded_offsets_workspace_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype);

/*
 * dsa3d_backward_fixed_window: backward of the operator with every offset equal to zero, without
 * an offsets tensor: dq, dk, dv (and doffsets, the gradient with respect to the offsets at zero,
 * unless it is NULL) equal those of dsa3d_backward on an all-zero offsets tensor up to fp32
 * summation order.  With a fixed window the contributions to a key's dK/dV come from the P
 * queries around it, so they are gathered instead of scattered: no atomics, results bitwise
 * deterministic, dk/dv written once in `dtype`.  `lse` is the forward's.  `workspace`:
 * dsa3d_backward_fixed_window_workspace_bytes(...) bytes (two fp32 coefficients per sample, plus,
 * for bf16 with d = 64 or 128 and windows (2,2,2), (3,3,3), (3,5,5) or (3,7,7), a table of the dot
 * products q.K_j and dO.V_j of every query's window and its +1 neighbours, which a tcgen05 kernel
 * fills from dense Q.K^T and dO.V^T tiles so that the gradient kernel gathers no K/V rows for them),
 * 16-byte aligned, contents undefined afterwards.  All supported dtypes, head sizes and windows.
 * For those bf16 shapes dq, dk and dv are then formed per tile of 4 x 4 x 8 outputs: from halo
 * regions in shared memory for the two small windows, as plane-by-plane tcgen05 products for the
 * two larger ones (coefficients as a bf16 head plus a bf16 remainder, relative error 2^-17).  The
 * environment variable DSA3D_NO_TENSOR_FIXED_WINDOW switches the table and tile kernels off.
 * Bounded waits as in dsa3d_offsets_linear_forward (dsa3d_device_timeout_flag).
 */
int dsa3d_backward_fixed_window(const void* q, const void* k, const void* v, const float* lse, const void* dout, int T,
                                int H, int W, int heads, int d, const int window[3], void* dq, void* dk, void* dv,
                                float* doffsets, void* workspace, size_t workspace_bytes, int dtype, void* stream);
size_t dsa3d_backward_fixed_window_workspace_bytes(int T, int H, int W, int heads, int d, const int window[3],
                                                   int dtype);

/*
 * Checked build (a debugging aid; the paper has no counterpart).  A library compiled with
 * -DDSA3D_DEBUG (paper_2607_22696_b200.build.build(debug=True) writes it to libdsa3d_debug.so) tests,
 * in dsa3d_forward and dsa3d_backward, every K/V row a sample is about to read, every dK/dV row a
 * contribution is about to be added to and every bin and scratch slot of the dK/dV pre-reduction
 * against the extent of its tensor before the access; the first index out of range is recorded in a
 * device word and that access is skipped - nothing traps, asserts or aborts.  (The tensor-core kernels
 * address memory through TMA tensor maps, whose bounds the hardware enforces.)
 *   dsa3d_debug_build            1 if this library was built with the checks, else 0
 *   dsa3d_debug_first_violation  synchronises with the device; *code = 0 if no violation was recorded
 *                                (always, in a normal build), else the site (1-3 forward gathers, 4-6
 *                                backward gathers, 7 direct dK/dV scatter, 8 bin, 9 scratch slot, 10
 *                                pre-reduced dK/dV row) and *offset = the offending element offset,
 *                                bin, slot or token.  Both HOST pointers.
 *   dsa3d_debug_clear            resets the record
 */
int dsa3d_debug_build(void);
int dsa3d_debug_first_violation(int* code, long long* offset);
int dsa3d_debug_clear(void);

/* Static, NUL-terminated description of a status code. */
const char* dsa3d_status_string(int status);

/* cudaError_t of the most recent DSA3D_ERR_CUDA on the calling thread (0 if none). */
int dsa3d_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DSA3D_H */
