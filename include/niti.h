/*
 * niti.h -- C ABI of the B200 (sm_100a) library for NITI integer training
 * ("NITI: Training Integer Neural Networks Using Integer-only Arithmetic",
 * arXiv 2009.13108).
 *
 * Every tensor pointer below is a DEVICE pointer owned by the caller unless a
 * function says otherwise.  The library allocates no device memory after
 * niti_create(); scratch comes from the caller's workspace `ws` (size from
 * niti_workspace_bytes(), 256-byte aligned; its first 256 KB hold 64 small
 * headers of reduction scalars, see niti_begin_step()).  All work is enqueued on the
 * caller's stream (`stream` is a cudaStream_t passed as void*) and the calls
 * return without synchronising; one workspace must not be used by two calls
 * that can overlap on the GPU.
 *
 * Number format (Section 3.1): a tensor is an int8 payload plus ONE shared
 * exponent s, value = payload * 2^s.  Exponents and effective bit-widths live
 * in device int32 scalars so that a whole training step needs no host sync.
 * The payload value -128 never appears in any output.
 *
 * Layouts: activations / errors are row-major [M][K] (fully connected) or
 * NHWC [B][H][W][C] (convolution); weights are [N_out][K_in] or
 * [Cout][R][S][Cin]; gradients have the layout of the weights.
 *
 * Rounding (Section 3.4): after each matrix multiply the int32 accumulator
 * tensor V is reduced to its effective bit-width b = bit_length(max|V|)
 * (Section 3.2), the binary point is bp = max(0, b - mbits) (Algorithm 1),
 * and every element is rounded by Algorithm 3 (round_mode 0, pseudo-
 * stochastic: the top half of the discarded bits is compared with the bottom
 * half) or to nearest (round_mode 1, magnitude half-up), on the magnitude
 * with the sign re-applied, saturating at 2^mbits - 1.  mbits is 7 for
 * activations and errors and m_u (1..7) for weight gradients.
 *
 * Contract on accumulators (Section 3.2: results are accumulated in int32): the
 * caller guarantees |sum| < 2^31 for every output.  This always holds when the
 * contraction length is <= 133144.  The weight-gradient calls contract over
 * the batch (niti_linear_bwd) or over batch x output pixels (niti_conv_wgrad:
 * 3.2 million on the first layers of a 224 x 224 network), the one place where
 * the contract can really break.  Contractions longer than 131072 are always
 * split over CTAs into pieces that cannot wrap, and the library adds up the
 * largest partial sum of every piece: when that bound reaches 2^31 the device
 * status bit NITI_DEV_ACC_RANGE is raised (the bound is conservative: the bit
 * can be raised for a tensor whose true sums still fit, never the reverse).
 *
 * Return value: NITI_OK or an error code; nothing is enqueued on error.
 */
#ifndef NITI_H_
#define NITI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NITI_OK 0
#define NITI_ERR_ARG 1       /* null pointer, non-positive size, bad flag          */
#define NITI_ERR_SHAPE 2     /* shape not supported by this build                  */
#define NITI_ERR_WORKSPACE 3 /* ws is NULL, misaligned or smaller than required    */
#define NITI_ERR_RANGE 4     /* exponent outside the supported domain              */
#define NITI_ERR_CUDA 5      /* a CUDA call failed; see niti_last_error()          */
#define NITI_ERR_DEVICE 6    /* a kernel raised the device status word             */
#define NITI_ERR_TOO_LARGE 8 /* beyond the fixed capacity of a no-allocation variant */

#define NITI_ROUND_PSR 0
#define NITI_ROUND_NEAREST 1

/* op ids for niti_workspace_bytes(); dims as listed */
#define NITI_OP_LINEAR_FWD 0  /* dims = {M, N, K}                 */
#define NITI_OP_LINEAR_BWD 1  /* dims = {M, N, K}                 */
#define NITI_OP_CONV_FWD 2    /* dims = {B, H, W, Cin, Cout, R, S, pad} or {..., pad, stride} */
#define NITI_OP_CONV_DGRAD 3  /* same                              */
#define NITI_OP_CONV_WGRAD 4  /* same                              */
#define NITI_OP_INT_XENT 5    /* dims = {B, N}                    */
#define NITI_OP_LINEAR_BWD_UPDATE 6 /* dims = {M, N, K}            */
#define NITI_OP_CONV_WGRAD_UPDATE 7 /* dims as NITI_OP_CONV_FWD    */

/* device status bits returned by niti_check() */
#define NITI_DEV_TIMEOUT 1u      /* a bounded wait inside a kernel gave up     */
#define NITI_DEV_EXP_RANGE 2u    /* an exponent left the int8 range            */
#define NITI_DEV_XENT_RANGE 4u   /* s_a outside [-22, 24] in niti_int_xent     */
#define NITI_DEV_BAD_LABEL 8u    /* a label outside [0, N)                     */
#define NITI_DEV_INTERNAL 32u    /* a consistency check inside a kernel failed: outputs of that call are not exact */
#define NITI_DEV_ACC_RANGE 16u   /* an int32 accumulator may have wrapped: in a contraction split over
                                  * CTAs the largest partial sums of the splits add up to 2^31 or more */

typedef struct niti_ctx niti_ctx;

/* Creates a context on CUDA device `device` (the device must be sm_100).
 * Allocates 33 KB of device memory (status words; a table in which the
 * speculative epilogue remembers, per call site, how far its last bit-width
 * estimate was off).  The caller destroys it with niti_destroy().  Not
 * thread-safe per context. */
int niti_create(niti_ctx **out, int device);
int niti_destroy(niti_ctx *ctx);

/* Text of the last host-side error of this context (owned by the context). */
const char *niti_last_error(niti_ctx *ctx);

/* Synchronises `stream`, reads and clears the device status word; returns
 * NITI_OK, NITI_ERR_CUDA or NITI_ERR_DEVICE (bits in *status if non-NULL). */
int niti_check(niti_ctx *ctx, void *stream, uint32_t *status);

/* Bytes of workspace the op needs for these dims (0 on bad arguments). */
size_t niti_workspace_bytes(int op, const int64_t *dims, int ndims);

/* Selects the matrix-multiply engine: 0 = automatic (tensor cores whenever
 * the shape allows; pairs of CTAs on 256-row tiles when there are enough of
 * them; default), 1 = plain CUDA-core kernels only, 2 = tensor cores with the
 * single-CTA kernel only, 3 = tensor cores with the paired-CTA kernel only
 * (falls back to CUDA cores where that kernel does not apply), 4 = tensor
 * cores with the two-pass epilogue (int32 accumulators spilled to the
 * workspace, rounded by a second kernel) instead of the fused one, 5 = tensor
 * cores without the weights-resident mode of small-channel 3x3 convolutions.
 * 1-5 exist so that tests can cross-check the engines.  Returns the previous
 * value. */
int niti_set_engine(niti_ctx *ctx, int engine);

/* Number of kernels / memsets this context has enqueued so far. */
uint64_t niti_launch_count(niti_ctx *ctx);
/* Of those, launches of the tensor-core (tcgen05) matrix-multiply kernel. */
uint64_t niti_tc_launch_count(niti_ctx *ctx);
/* Of those, launches of the paired-CTA (cta_group::2) variant. */
uint64_t niti_tc_pair_launch_count(niti_ctx *ctx);

/* The fused epilogue of the tensor-core kernel rounds with a bit-width guessed from the first
 * tile of every CTA and recomputes the multiply when the whole tensor turns out to need a larger
 * shift (results are exact either way).  A call that passes a bit-width scalar (b_out / b_e / b_g)
 * is recognised by that scalar's address when it comes again (the same layer in the next training
 * step): an estimate that missed by the same amount twice in a row is corrected by that amount, which
 * removes the recomputations of tensors whose extremes the sample systematically misses.  Returns how many recomputations this
 * context has run so far (synchronises `stream`; -1 on error). */
int64_t niti_redo_count(niti_ctx *ctx, void *stream);

/* Self-test of the failure detection: every wait inside the kernels is bounded; this enqueues a
 * one-warp kernel that waits (about 50 ms) on a barrier nothing completes, gives up, raises
 * NITI_DEV_TIMEOUT in the device status word and returns normally.  niti_check() then reports
 * NITI_ERR_DEVICE once, and the context and the GPU remain usable. */
int niti_selftest_timeout(niti_ctx *ctx, void *stream);

/* Timing of the tensor-core matrix-multiply kernel.  While enabled, every launch of that
 * kernel is bracketed by a pair of CUDA events on its stream (up to 8192 launches are kept).
 * niti_profile_read() waits for the recorded events, returns their summed duration in
 * milliseconds, their count and the summed algorithmic int8 operations (2*M*N*K of each
 * multiply), and starts a new record.  Host pointers. */
int niti_profile_enable(niti_ctx *ctx, int on);
int niti_profile_read(niti_ctx *ctx, double *tc_ms, uint64_t *tc_launches, double *tc_ops);
/* Per-launch view of the same record (does not reset it): fills ms[i] and ops[i] for the first
 * min(recorded, max_n) launches in launch order and returns that count (-1 on error). */
int niti_profile_read_launches(niti_ctx *ctx, double *ms, double *ops, int max_n);

/* Fully connected forward (Algorithm 1, forward loop; Section 3.2):
 *   acc[m][n] = sum_k a[m][k] * w[n][k];  b = B(acc);  bp = max(0, b - 7);
 *   out = Round(acc, bp) (then max(.,0) if relu);  *s_out = *s_a + *s_w + bp.
 * a [M][K], w [N][K], out [M][N]; s_a, s_w, s_out, b_out device scalars
 * (s_out, b_out may be NULL). b is taken before the ReLU. */
int niti_linear_fwd(niti_ctx *ctx, void *stream, const int8_t *a, const int32_t *s_a,
                    const int8_t *w, const int32_t *s_w, int8_t *out, int32_t *s_out,
                    int32_t *b_out, int M, int N, int K, int relu, int round_mode, void *ws,
                    size_t ws_bytes);

/* Fully connected backward (Algorithm 1, reverse loop; Section 3.3):
 *   g32[n][k] = sum_m e[m][n] * a[m][k]  -> g = Round(g32, max(0, B(g32) - m_u))
 *   e32[m][k] = sum_n e[m][n] * w[n][k]  -> e_prev = Round(e32, max(0, B(e32) - 7))
 * Both use w as it is on entry (the update is a separate call).  e_prev may be
 * NULL (first layer).  relu_mask_src, if not NULL, is an int8 [M][K] tensor
 * (the ReLU output that fed this layer); e_prev is zeroed where it is <= 0.
 * b_e, b_g: device scalars, may be NULL. */
int niti_linear_bwd(niti_ctx *ctx, void *stream, const int8_t *a, const int8_t *e, const int8_t *w,
                    int8_t *e_prev, const int8_t *relu_mask_src, int8_t *g, int32_t *b_e,
                    int32_t *b_g, int M, int N, int K, int m_u, int round_mode, void *ws,
                    size_t ws_bytes);

/* Convolution forward as an implicit matrix multiply (Section 3.2), stride 1,
 * zero padding `pad`, R x S taps (any R, S, pad; 3 x 3 / pad 1 has tuned modes):
 *   acc[b][i][j][co] = sum_{r,s,ci} x[b][i+r-pad][j+s-pad][ci] * w[co][r][s][ci]
 * followed by the same bit-width / shift / round / exponent rule as
 * niti_linear_fwd.  x [B][H][W][Cin], y [B][H+2pad-R+1][W+2pad-S+1][Cout]. */
int niti_conv_fwd(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x,
                  const int8_t *w, const int32_t *s_w, int8_t *y, int32_t *s_y, int32_t *b_y, int B,
                  int H, int W, int Cin, int Cout, int R, int S, int pad, int relu, int round_mode,
                  void *ws, size_t ws_bytes);

/* niti_conv_fwd followed by the 2 x 2 max-pool of its output, in one call
 * (Sections 3.2-3.3 fuse what follows a multiply into it; the networks of
 * Section 4 pool after a ReLU'd convolution): y as niti_conv_fwd, y_pool
 * [B][Ho/2][Wo/2][Cout] = niti_maxpool2_fwd(y).  Ho and Wo must be even.  With
 * relu != 0, Cout a multiple of 32 and 32-byte aligned y / y_pool the
 * tensor-core kernel's epilogue writes the pooled tile itself (the four pixels
 * of a window sit in one warp and are combined with shuffles); otherwise the
 * pooling kernel runs after the convolution.  Same results either way. */
int niti_conv_fwd_pool(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x, const int8_t *w,
                       const int32_t *s_w, int8_t *y, int8_t *y_pool, int32_t *s_y, int32_t *b_y, int B, int H,
                       int W, int Cin, int Cout, int R, int S, int pad, int relu, int round_mode, void *ws,
                       size_t ws_bytes);

/* Error back-propagation through the convolution (Algorithm 1, reverse loop):
 *   e32[b][i][j][ci] = sum_{r,s,co} e[b][i-r+pad][j-s+pad][co] * w[co][r][s][ci]
 * rounded to 7 bits.  H, W are the INPUT sizes of the forward convolution;
 * e has the forward output's shape.  relu_mask_src as in niti_linear_bwd
 * (shape of e_prev). */
int niti_conv_dgrad(niti_ctx *ctx, void *stream, const int8_t *e, const int8_t *w, int8_t *e_prev,
                    const int8_t *relu_mask_src, int32_t *b_e, int B, int H, int W, int Cin,
                    int Cout, int R, int S, int pad, int round_mode, void *ws, size_t ws_bytes);

/* Weight gradient of the convolution (Algorithm 1, reverse loop; Section 3.3):
 *   g32[co][r][s][ci] = sum_{b,i,j} e[b][i][j][co] * x[b][i+r-pad][j+s-pad][ci]
 * rounded to m_u bits (values in [-(2^m_u - 1), 2^m_u - 1] in an int8). */
int niti_conv_wgrad(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *g,
                    int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S, int pad,
                    int m_u, int round_mode, void *ws, size_t ws_bytes);

/* The same three convolution ops with a stride (the first layer of the paper's
 * AlexNet is 11 x 11 with stride 4, Section 4):
 *   acc[b][i][j][co] = sum_{r,s,ci} x[b][i*stride+r-pad][j*stride+s-pad][ci] * w[co][r][s][ci]
 * with output size Ho = (H + 2 pad - R) / stride + 1 (integer division), Wo
 * likewise; the error and weight-gradient calls are its exact transposes with
 * respect to x and w.  H, W are always the INPUT sizes of the forward
 * convolution; y / e have the [B][Ho][Wo][Cout] shape.  Workspace: the same op
 * ids with the stride as a ninth entry of dims.  stride = 1 is the call
 * without the suffix.  Forward and weight gradient of strided layers with at
 * least 32 channels on both sides run on the tensor cores (the stride becomes
 * the element stride of the operand copies); the error of a strided layer and
 * layers with other channel counts run on the CUDA-core engine. */
int niti_conv_fwd_strided(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x,
                          const int8_t *w, const int32_t *s_w, int8_t *y, int32_t *s_y, int32_t *b_y, int B,
                          int H, int W, int Cin, int Cout, int R, int S, int pad, int stride, int relu,
                          int round_mode, void *ws, size_t ws_bytes);
int niti_conv_dgrad_strided(niti_ctx *ctx, void *stream, const int8_t *e, const int8_t *w, int8_t *e_prev,
                            const int8_t *relu_mask_src, int32_t *b_e, int B, int H, int W, int Cin,
                            int Cout, int R, int S, int pad, int stride, int round_mode, void *ws,
                            size_t ws_bytes);
int niti_conv_wgrad_strided(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *g,
                            int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S, int pad,
                            int stride, int m_u, int round_mode, void *ws, size_t ws_bytes);

/* Weight gradient fused with the weight update (Section 3.3: the gradient is
 * rounded to m_u bits "and fused with the weight update"; Algorithm 1, last two
 * lines of the reverse loop).  Same arithmetic as niti_conv_wgrad followed by
 * niti_int_sgd_update, with w [Cout][R][S][Cin] updated in place,
 *   w <- clamp(w - round(g32), -127, 127),
 * and the int8 gradient never returned: where the contraction is split over
 * CTAs (every convolution of the networks) the rounding pass over the int32
 * sums subtracts from w directly; otherwise the gradient passes through the
 * workspace.  b_g receives the bit-width of g32.  Workspace:
 * NITI_OP_CONV_WGRAD_UPDATE.  w must be 16-byte aligned. */
int niti_conv_wgrad_update(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *w,
                           int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S, int pad,
                           int m_u, int round_mode, void *ws, size_t ws_bytes);

/* niti_linear_bwd with the weight update fused in: e_prev (may be NULL) is
 * computed from the weights as they are on entry, then w [N][K] is updated in
 * place with the rounded weight gradient, which is not returned.  Workspace:
 * NITI_OP_LINEAR_BWD_UPDATE. */
int niti_linear_bwd_update(niti_ctx *ctx, void *stream, const int8_t *a, const int8_t *e, int8_t *w,
                           int8_t *e_prev, const int8_t *relu_mask_src, int32_t *b_e, int32_t *b_g,
                           int M, int N, int K, int m_u, int round_mode, void *ws, size_t ws_bytes);

/* Exact data-parallel training over several GPUs (one process per GPU, each with its share of
 * the batch): the method shards over the batch, and the only quantities that couple the samples
 * are (a) the max magnitude that fixes the bit-width b of a tensor, and (b) the int32 sums of the
 * weight gradient, which contract over the batch (Algorithm 1).  With a hook installed the
 * library calls it, in stream order, wherever one of them must be combined over the ranks before
 * the rounding uses it:
 *   NITI_REDUCE_MAX_U32: dev_ptr -> count (= 1) unsigned 32-bit values, combine with max;
 *   NITI_REDUCE_MAX_U64: the same, 64-bit (integer cross-entropy);
 *   NITI_REDUCE_SUM_I32: dev_ptr -> count int32 sums (a whole weight-gradient tensor), add.
 * dev_ptr points into the workspace of the running call.  The hook must order its work after what
 * is already on `stream` and before what follows (e.g. an NCCL all-reduce on that stream) and
 * return 0.  Every rank must make the same sequence of library calls.  With the combined values
 * every rank rounds exactly as one process holding the whole batch would, so activations, errors
 * and updated weights equal the single-process result bit for bit.  Multiplies that would round
 * in their own epilogue from partial sums (weight gradients) take the int32 path instead.
 * fn == NULL removes the hook.  niti_int_xent_noalloc has no context and calls no hook. */
#define NITI_REDUCE_MAX_U32 0
#define NITI_REDUCE_MAX_U64 1
#define NITI_REDUCE_SUM_I32 2
/* Only after niti_set_dp_shard(ctx, rank, world) with world > 1 (count is a multiple of world):
 *   NITI_REDUCE_SCATTER_SUM_I32: dev_ptr -> count int32; on return the rank's own slice
 *     [rank * count / world, (rank + 1) * count / world) holds the sums over the ranks of that slice
 *     (the other slices are unspecified): a reduce-scatter in place;
 *   NITI_ALLGATHER_I8: dev_ptr -> count bytes; every rank's own slice (same split) is distributed to all
 *     ranks: an all-gather in place. */
#define NITI_REDUCE_SCATTER_SUM_I32 3
#define NITI_ALLGATHER_I8 4
typedef int (*niti_reduce_fn)(void *user, void *stream, void *dev_ptr, int64_t count, int kind);
int niti_set_reduce_hook(niti_ctx *ctx, niti_reduce_fn fn, void *user);
/* Optional, once per training step (or per group of at most 64 calls): clears every header of the
 * workspace `ws` with one memset on `stream`.  The calls that follow on that workspace (in stream
 * order, from this context) then take one zeroed header each instead of clearing their own, which
 * removes a memset node from in front of every multiply of the step.  After 64 calls, or for any other
 * workspace, calls clear their header themselves as they do without this call.  The caller must not
 * use that workspace from two streams at once (as for any workspace) and must call niti_begin_step
 * again before the pattern repeats (each training step; a captured CUDA graph holds it as its first
 * node).  ws = NULL ends the arrangement.  Results do not change. */
int niti_begin_step(niti_ctx *ctx, void *stream, void *ws, size_t ws_bytes);

/* Convolutions with very few input channels (R * S * Cin <= 32: the first layer of an image network)
 * are run as a matrix multiply over rows of gathered taps, 32 bytes per output pixel.  Forward and
 * weight gradient of such a layer read the same rows.  With a tap cache installed (a caller-owned
 * device buffer, 256-byte aligned, at least 32 * B * Ho * Wo bytes) niti_conv_fwd gathers into it
 * and remembers for which input tensor and geometry, and a later niti_conv_wgrad of the same input
 * pointer and geometry reads the rows from there instead of gathering them again (one pass over
 * 103 MB less at 224 x 224, batch 64).  The caller promises that the input tensor is not modified
 * between the two calls; a cached gather serves one weight-gradient call, and the next few-channel
 * forward call overwrites it.  buf = NULL removes the cache.  Results do not change. */
int niti_set_tap_cache(niti_ctx *ctx, void *buf, size_t bytes);

/* Tells the library this process' place among the data-parallel ranks.  With world > 1 a weight
 * gradient is no longer all-reduced as a whole int32 tensor (8 bytes per weight on the wire): its
 * sums are reduce-scattered (4 bytes per weight), every rank takes the max over its shard and the
 * maxima are combined, every rank rounds its shard (or updates its shard of the weights, in the
 * fused-update calls) and the int8 result is all-gathered (1 byte per weight).  Results are the same
 * bit for bit.  world = 1 (the default) keeps the all-reduce. */
int niti_set_dp_shard(niti_ctx *ctx, int rank, int world);

/* Integer cross-entropy gradient (Section 3.5, Eq. 1-4).  Per sample r:
 *   e32[r][i] = T_i - [i == labels[r]] * sum_j T_j
 * with T_i = 2^(1-2s) + a_i 2^(1-s) + a_i^2 when s = *s_a <= -7 (Eq. 2), else
 * T_i = 1 << max(0, xh_i - p), xh_i = (47274 a_i) >> (15 - s) (arithmetic
 * shift; a left shift if 15 - s < 0), p = the smallest xh_i greater than
 * max(xh) - 10 (Eq. 3-4).  The whole [B][N] tensor is then rounded to 7 bits
 * with one shared binary point.  a [B][N] int8, labels [B] int32, e [B][N].
 * n_correct (may be NULL): number of rows whose first arg-max equals the
 * label.  *s_a outside [-22, 24] or a bad label sets the device status word
 * and writes zeros.  N <= 65536. */
int niti_int_xent(niti_ctx *ctx, void *stream, const int8_t *a, const int32_t *s_a,
                  const int32_t *labels, int8_t *e, int32_t *b_e, int32_t *n_correct, int B, int N,
                  int round_mode, void *ws, size_t ws_bytes);

/* Integer cross-entropy gradient for callers that must not allocate device memory (the paper has
 * no counterpart: this is a packaging variant of niti_int_xent, same arithmetic, same outputs).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a latency-critical training loop
 * that forbids allocator calls after start-up, a host process that has already handed all device
 * memory to its own pool, or a plug-in that is given tensors and a stream but no allocator.  Such
 * a caller cannot create a context (niti_create allocates the status word) nor a workspace, so
 * this call takes neither: its scratch (256 bytes of reduction scalars + 16 bytes per sample)
 * lives in a fixed array inside the library image of 512 KiB + 256 B, which every GPU loading the
 * library holds until exit.  Limits: B * N <= NITI_XENT_NOALLOC_MAX_ELEMS (65536 logits) and
 * B <= 32768; anything larger returns NITI_ERR_TOO_LARGE and enqueues nothing.
 *
 * a, labels, e, s_a, b_e, n_correct: device pointers as in niti_int_xent (b_e, n_correct may be
 * NULL); `stream` is the caller's cudaStream_t.  The call allocates nothing and frees nothing.  The
 * first call on each device looks up the array's device address (with the current device); make
 * that first call before any stream capture begins.  All calls on a device share the one array,
 * which keeps the previous call's contents: the call clears the scalars it needs itself, but two
 * calls that can overlap on the GPU (different streams without ordering) race on it.  There is
 * no status word in this variant: an exponent outside [-22, 24] or a label outside [0, N) yields
 * zeros for the affected rows. */
#define NITI_XENT_NOALLOC_MAX_ELEMS 65536
int niti_int_xent_noalloc(void *stream, const int8_t *a, const int32_t *s_a, const int32_t *labels,
                          int8_t *e, int32_t *b_e, int32_t *n_correct, int B, int N, int round_mode);

/* Weight update (Algorithm 1 last line; Section 3.3): w <- clamp(w - g, -127, 127), in place. */
int niti_int_sgd_update(niti_ctx *ctx, void *stream, int8_t *w, const int8_t *g, int64_t n);

/* Support ops on int8 tensors between the layers (implied by the paper's
 * networks, Section 4); exponents are unchanged.
 *   relu_fwd: y = max(x, 0) (y may alias x).
 *   relu_bwd: e_in = e_out where y > 0 else 0 (e_in may alias e_out).
 *   maxpool2_fwd: 2x2 window, stride 2, NHWC, H and W even.
 *   maxpool2_bwd: routes e_out to the first maximum of each window in
 *     (row, col) order, zero elsewhere; if relu != 0 the result is also zeroed
 *     where x <= 0 (x is the pooled ReLU output). */
int niti_relu_fwd(niti_ctx *ctx, void *stream, const int8_t *x, int8_t *y, int64_t n);
int niti_relu_bwd(niti_ctx *ctx, void *stream, const int8_t *y, const int8_t *e_out, int8_t *e_in,
                  int64_t n);
int niti_maxpool2_fwd(niti_ctx *ctx, void *stream, const int8_t *x, int8_t *y, int B, int H, int W,
                      int C);
int niti_maxpool2_bwd(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e_out,
                      int8_t *e_in, int B, int H, int W, int C, int relu);

/* The same max-pool with the routing recorded in the forward pass, so that the
 * backward pass does not read the pooled tensor again (it reads the error and
 * half a byte per output element instead of four input bytes).
 *   maxpool2_fwd_idx: y as niti_maxpool2_fwd, and idx [B][H/2][W/2][C/2]
 *     bytes: per output element a 4-bit code, channel c in the low (c even) or
 *     high (c odd) nibble; bits 0-1 = position of the first maximum in
 *     (row, col) order, bit 2 = that maximum is > 0.
 *   maxpool2_bwd_idx: e_in as niti_maxpool2_bwd(x, e_out, relu) for the x the
 *     codes were recorded from.
 * C must be a multiple of 16, x / y / e_out / e_in 16-byte and idx 8-byte
 * aligned (NITI_ERR_SHAPE otherwise: use the plain calls). */
int niti_maxpool2_fwd_idx(niti_ctx *ctx, void *stream, const int8_t *x, int8_t *y, uint8_t *idx, int B, int H,
                          int W, int C);
int niti_maxpool2_bwd_idx(niti_ctx *ctx, void *stream, const int8_t *e_out, const uint8_t *idx, int8_t *e_in,
                          int B, int H, int W, int C, int relu);

#ifdef __cplusplus
}
#endif
#endif /* NITI_H_ */
