/*
 * patconv — pattern-based sparse 3x3 convolution for NVIDIA B200 (sm_100a).  C ABI.
 *
 * The operations follow "An Image Enhancing Pattern-based Sparsity for Real-time Inference on
 * Mobile Devices" (arXiv 2001.07710):
 *   - pattern pruning: every 3x3 kernel is multiplied element-wise by one binary mask taken from
 *     a small pattern library; every mask keeps exactly four entries (Section 4.1, Section 5.1);
 *   - connectivity pruning: whole kernels are removed according to their L2 norm (Section 6.1);
 *   - filter / kernel re-ordering and compact weight storage for execution (Section 6.2).
 *
 * Conventions used by every entry point
 *   kernel position (r,s): r = row 0..2 (top to bottom), s = column 0..2 (left to right);
 *   mask bit b = 3*r + s; a pattern is a 9-bit integer with exactly four bits set.
 *   weights      [F][C][3][3] fp32, F = filters (output channels), C = input channels.
 *   activations  NHWC, fp32 or fp16; outputs NHWC in the ORIGINAL filter order.
 *   convolution  cross-correlation (no kernel flip), zero padding 1, stride 1 or 2, no bias:
 *                Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1.
 *
 * Memory and execution
 *   "dev" pointers are device memory owned by the caller; "host" pointers are host memory.
 *   The library allocates no device memory unless an entry point says otherwise.  All device
 *   work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *   and the calls return without synchronising.  Arguments are validated on the host before
 *   anything is launched.
 *
 * Errors
 *   Every function that returns int returns PAT_OK (0) or a PAT_ERR_* code; nothing is launched
 *   when a code other than PAT_OK / PAT_ERR_CUDA is returned.  pat_last_error() gives a
 *   thread-local message for the last failing call on the calling thread.
 */
#ifndef PATCONV_H_
#define PATCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PAT_OK               0
#define PAT_ERR_INVALID_ARG  1   /* null pointer, negative size, value out of range          */
#define PAT_ERR_SHAPE        2   /* unsupported tensor shape                                  */
#define PAT_ERR_LIBRARY      3   /* pattern library: mask without 4 bits, duplicate, K range  */
#define PAT_ERR_DTYPE        4   /* dtype is neither PAT_F32 nor PAT_F16                      */
#define PAT_ERR_ALIGN        5   /* pointer alignment                                         */
#define PAT_ERR_BLOB         6   /* packed blob does not match the arguments                  */
#define PAT_ERR_CUDA         7   /* a CUDA runtime call failed                                */
#define PAT_ERR_WORKSPACE    8   /* workspace or blob buffer too small                        */
#define PAT_ERR_TIMEOUT      9   /* a bounded device-side wait expired (reported by pat_query_status) */

#define PAT_F32 0                /* fp32 storage, fp32 accumulation                           */
#define PAT_F16 1                /* fp16 storage (weights, activations), fp32 accumulation    */

#define PAT_PRUNED 0xFF          /* pattern id of a kernel removed by connectivity pruning    */

const char *pat_strerror(int code);
const char *pat_last_error(void);

/* Built-in pattern libraries (Section 4.2 derives the eight patterns; Section 7.1 uses libraries
 * of 12, 8 and 4 patterns).  K = 4: centre + three of the four arms (missing arm: down, up, left,
 * right).  K = 8: those plus the four 2x2 blocks containing the centre (top-left, top-right,
 * bottom-left, bottom-right).  K = 12: those plus {centre, up, down, top-left corner} and its
 * three clockwise quarter-turn rotations (a convention of this library: the paper shows the
 * additional four patterns only in a figure).
 * masks_out: host, K entries.  Returns PAT_ERR_LIBRARY for any other K. */
int pat_library_builtin(int K, uint16_t *masks_out);

/* Bytes of device workspace pat_project needs for an F x C layer (0 on invalid sizes). */
size_t pat_project_workspace(int F, int C);

/* Pattern selection + connectivity pruning of one layer (Sections 4.1, 5.1, 6.1).
 * For every kernel (f,c) the mask of the library that keeps the largest sum of squares is chosen
 * (squares and sums in float64, bits in ascending order; lowest pattern id on ties).  The n_keep
 * kernels with the largest kept sum of squares survive (lower f*C+c on ties); the others are
 * removed.  Results are exact and deterministic.
 *   w           dev, [F][C][3][3] fp32
 *   masks       host, K distinct 9-bit masks with four bits each, 1 <= K <= 255
 *   n_keep      0 .. F*C
 *   pattern_id  dev out, [F*C] bytes: chosen pattern id, PAT_PRUNED for removed kernels
 *   w_masked    dev out, [F][C][3][3] fp32: kept entries bit-identical to w, all others +0.0;
 *               may be the same buffer as w
 *   workspace   dev, at least pat_project_workspace(F, C) bytes, 256-byte aligned; contents are
 *               scratch (no need to clear); concurrent calls must use different workspaces */
int pat_project(const float *w, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
                uint8_t *pattern_id, float *w_masked, void *workspace, size_t workspace_bytes,
                void *stream);

/* pat_project without a caller-supplied workspace, and without any allocation.  (The paper has no counterpart
 * for this entry point: it exists for the way the library is embedded, not for the method.)
 * Who needs it: code that is not allowed to allocate device memory where it runs - a server that gave its
 * whole device budget to a memory pool at start-up, a plug-in living inside another framework's allocator,
 * a real-time loop that cannot accept the device-wide synchronisation an allocation may cause.
 * The scratch space is a fixed array inside the library image (about 3.9 MB on every GPU that loads the
 * library, held until the process exits), sized for layers of up to pat_project_static_max_kernels() =
 * 262144 kernels (F * C; a 512 x 512 layer).  Larger layers are refused with PAT_ERR_WORKSPACE and nothing
 * is launched; use pat_project for them.  Arguments and results are those of pat_project.
 * - The first call on each device looks up the array's device address (no allocation, but a runtime call
 *   that is not stream work): make that first call before any stream capture.
 * - All calls share the one array and it keeps whatever the previous call left there; the kernels
 *   re-initialise every counter they rely on, so stale contents never matter.  Two calls whose kernels
 *   may overlap on the GPU (different streams, no dependency between them) race on the array: order them.
 * - Calls cudaMalloc / cudaFree or any allocating routine: never. */
int pat_project_static(const float *w, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
                       uint8_t *pattern_id, float *w_masked, void *stream);
int64_t pat_project_static_max_kernels(void);

/* Size in bytes of the packed blob of a layer (0 on invalid arguments).  A pure function of its
 * arguments, so no device-to-host transfer is ever needed to size a buffer. */
size_t pat_pack_size(int F, int C, int K, int64_t n_keep, int dtype);

/* Compressed, re-ordered weight storage (Section 6.2: filters with similar kernels are grouped,
 * and inside each filter the kernels of identical pattern are grouped).
 * Canonical section of the blob (host-readable layout given by pat_blob_layout):
 *   perm[F]       i32  new position -> original filter; filters sorted by kept-kernel count
 *                      (descending), then per-pattern count vector (lexicographically
 *                      descending), then original index (ascending)
 *   fptr[F+1]     i32  first kernel of each re-ordered filter; fptr[F] = n_keep
 *   pptr[F][K+1]  i32  first kernel of each pattern segment of the filter
 *   chan[n_keep]  u16  input channel of each kernel; kernels ordered by (pattern id, channel)
 *   w4[n_keep][4]      the four kept entries in ascending bit order, fp32, or fp16 rounded to
 *                      nearest-even when dtype = PAT_F16
 * followed by an execution section (kernels re-sorted by blocks of 16 input channels) that only
 * pat_conv3x3 reads.
 *   w_masked, pattern_id  dev, as written by pat_project; exactly n_keep kernels must be kept
 *   blob        dev out, at least pat_pack_size(...) bytes, 256-byte aligned */
int pat_pack(const float *w_masked, const uint8_t *pattern_id, int F, int C,
             const uint16_t *masks, int K, int64_t n_keep, int dtype,
             void *blob, size_t blob_bytes, void *stream);

/* Byte offsets of the canonical arrays inside a blob (host-side helper; offsets[0..4] =
 * perm, fptr, pptr, chan, w4).  Returns PAT_ERR_* on invalid arguments. */
int pat_blob_layout(int F, int C, int K, int64_t n_keep, int dtype, size_t offsets[5]);

/* Expand a blob back to dense masked weights [F][C][3][3] fp32 (fp16 entries are widened
 * exactly).  Inverse of pat_pack: for dtype PAT_F32 the result is bit-identical to w_masked.
 * (Section 6.2 stores the re-ordered model compactly; this call reads that storage back as the
 * masked kernels of Section 4.1, mask o kernel, which is how the packed layout is verified.) */
int pat_unpack(const void *blob, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
               int dtype, float *w_dense_out, void *stream);

/* The sparse convolution (the execution side of Section 6.2: per-pattern access code with the
 * four tap positions fixed at compile time, no per-weight index decoding, pattern-grouped
 * kernels, filters grouped by load).
 *   Y[n][y][x][f] = sum over kept kernels (f,c) and their four taps (r,s) of
 *                   w[f][c][r][s] * X[n][y*stride + r - 1][x*stride + s - 1][c]
 * Products and sums are fp32 (fp16 inputs are widened exactly); the result is stored in the
 * blob's dtype (fp16: round to nearest even).
 *   blob     dev, written by pat_pack with the same (F, C, masks, K, n_keep, dtype)
 *   masks    host, the library the blob was packed with (selects the compiled tap code)
 *   x        dev, NHWC [N][H][W][C], 16-byte aligned
 *   y        dev out, NHWC [N][Ho][Wo][F], 16-byte aligned, must not overlap x
 * Any F and C in 1..65535 is accepted; shapes outside the tuned kernels' reach (see pat_conv3x3_ws) run a generic
 * kernel. */
int pat_conv3x3(const void *blob, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
                int dtype, const void *x, void *y, int N, int H, int W, int stride, void *stream);

/* The same convolution with a caller-supplied device workspace.  For the layer shapes it covers (fp16 or fp32,
 * stride 1 or 2, C a multiple of 16, F a multiple of 32, W a multiple of 14 with W/14 in {1, 2, 4k} or W < 14,
 * max(ceil(H/4), 4) == 4 or >= 7) the activations are first re-arranged, once per call, into the channel-planar tiles
 * the multiply-add kernel stages in shared memory; the kernel then needs no transposition of its own and runs a deeper
 * pipeline.  Stride 2 is computed like stride 1 and the results at even rows and columns are written.
 * pat_conv3x3_workspace returns the bytes needed (about 1.3 x the size of x, plus 59 MB for partial sums), or 0 for a
 * layer the workspace path does not cover: pat_conv3x3_ws then behaves exactly like pat_conv3x3 and ignores the
 * workspace.
 *   workspace  dev, at least pat_conv3x3_workspace(...) bytes, 256-byte aligned; contents are scratch;
 *              concurrent calls must use different workspaces
 * Results: the same products as pat_conv3x3, added in fp32 in a different order of the kernels of a filter. */
size_t pat_conv3x3_workspace(int F, int C, int dtype, int N, int H, int W, int stride);
int pat_conv3x3_ws(const void *blob, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
                   int dtype, const void *x, void *y, int N, int H, int W, int stride,
                   void *workspace, size_t workspace_bytes, void *stream);

/* pat_conv3x3_ws with the rectifier that follows the layer in the models of Section 7 fused into its epilogue
 * (the graph-level fusion of Section 6.2): act = 1 writes max(result, 0), act = 0 is pat_conv3x3_ws.  The workspace
 * kernels apply it to the fp32 sums before they are rounded and stored, at no extra pass over the output; a layer
 * they do not cover runs the plain convolution and then pat_relu_maxpool in place (same result).
 * act = 2 fuses the 2 x 2 max pooling that follows five of the thirteen layers of the VGG-16 of Section 7 as well:
 * y is then NHWC [N][H/2][W/2][F] and holds max(0, the four results of each 2 x 2 block) - the values of
 * pat_relu_maxpool(pool = 1) on the output of act = 0, bit for bit (rounding is monotone) - and the full-size
 * output is never written.  act = 2 needs stride 1, even H and W and a layer the workspace kernels cover
 * (pat_conv3x3_workspace(...) > 0): PAT_ERR_SHAPE otherwise, nothing launched; such a layer takes act = 1 and a
 * separate pat_relu_maxpool.  Other arguments, errors and workspace as for pat_conv3x3_ws; PAT_ERR_INVALID_ARG for
 * any other `act`. */
int pat_conv3x3_ws_act(const void *blob, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
                       int dtype, const void *x, void *y, int N, int H, int W, int stride, int act,
                       void *workspace, size_t workspace_bytes, void *stream);

/* Dense 3x3 convolution for layers that are not pruned: the first layer of the VGG-16 of Section 7
 * (C = 3 input channels), which stays dense when the other twelve are pattern-pruned.
 *   w   dev, [F][C][3][3] fp32 (converted to the activation type on the fly)
 *   x   dev NHWC [N][H][W][C]; y dev NHWC [N][Ho][Wo][F]; dtype of x and y = `dtype`
 * The case C = 3, F = 64, PAT_F16, stride 1 runs on the tensor cores (fp16 products, fp32 sums, like every
 * other path); all other cases run FMA kernels.
 * Restrictions: 1 <= C <= 16, 1 <= F <= 65535 (PAT_ERR_SHAPE otherwise). */
int pat_conv3x3_dense(const float *w, int F, int C, int dtype, const void *x, void *y,
                      int N, int H, int W, int stride, void *stream);

/* The kernels never trap and never wait without a limit (the paper's execution scheme, Section 6.2, has no
 * counterpart: it generates straight-line code per layer); what they cannot do they report in one status word
 * per device.
 * Synchronises `stream` and returns the device-side status word: PAT_OK, or PAT_ERR_BLOB when a
 * kernel found a blob header that did not match its arguments (the kernel then wrote nothing),
 * or PAT_ERR_TIMEOUT when a bounded wait inside a kernel expired (its output is then incomplete).
 * The word is cleared by the call. */
int pat_query_status(void *stream);

/* Number of CUDA kernels this library has launched from the calling process so far (all threads,
 * all entry points).  Host-side counter; useful to check that work really ran on the GPU. */
uint64_t pat_launch_count(void);

/* Measures the device's multiply-add rate with the instruction the convolution kernels issue (kind 0: fma.rn.f32,
 * kind 1: fma.rn.f32.f16 with an fp32 accumulator): the denominator of their roofline, taken at the clock the device
 * really runs at.  Launches a few short kernels on `stream` and waits for them (this one call synchronises).
 *   scratch     dev, 256-byte aligned, at least 256 + 4 * 8 * 256 * (number of SMs) bytes (2 MiB always suffices)
 *   tflops_out  host out: best of three runs, in TFLOP/s (2 flop per multiply-add)
 * The paper has no counterpart (it reports end-to-end latencies, Section 7.2). */
int pat_measure_fma_peak(int kind, void *scratch, size_t scratch_bytes, double *tflops_out, void *stream);

/* What stands between two convolution layers of the models the paper evaluates (Section 7: VGG-16, ResNet-50; their
 * own definition, the paper adds nothing to it): the rectifier max(x, 0) and, with pool = 1, 2x2 max pooling with
 * stride 2 after it.
 *   x      dev in  NHWC [N][H][W][C], dtype PAT_F32 or PAT_F16, finite values
 *   y      dev out NHWC [N][H][W][C] (pool = 0; may be x itself) or [N][H/2][W/2][C] (pool = 1; H and W even, y must
 *          not overlap x)
 * One pass over the data; 16-byte accesses when C * (element size) is a multiple of 16 and both buffers are 16-byte
 * aligned, element by element otherwise.  Asynchronous on `stream`; allocates nothing.
 * Errors: PAT_ERR_INVALID_ARG, PAT_ERR_DTYPE, PAT_ERR_SHAPE (odd H or W with pool = 1), PAT_ERR_ALIGN, PAT_ERR_CUDA. */
int pat_relu_maxpool(const void *x, int dtype, int N, int H, int W, int C, int pool, void *y, void *stream);

/* ---- Primitives of the pattern-selection ADMM and of the library extraction (training side; the loop around them,
 * the loss and the data are not part of this library).  All pointers are device pointers unless marked host. ---- */

/* Proximal step of Section 5.1: for each of n vectors d of K reals, u = [d - nu 1]_+ where nu is the root of
 * 1^T [d - nu 1]_+ = 1, i.e. the Euclidean projection of d onto the probability simplex.
 *   d   dev in  [n][K] fp32, row-major, 4-byte aligned, finite values
 *   u   dev out [n][K] fp32 (may be d itself); every entry >= 0, every row sums to 1 up to fp32 rounding
 * Arithmetic in fp64, one rounding to fp32.  1 <= K <= 256; n = 0 is accepted and does nothing.  Asynchronous on
 * `stream`; allocates nothing.
 * Errors: PAT_ERR_INVALID_ARG (null), PAT_ERR_SHAPE (K or n out of range), PAT_ERR_ALIGN, PAT_ERR_CUDA. */
int pat_simplex_project(const float *d, int64_t n, int K, float *u, void *stream);

/* Binarisation of Section 5.1: the one-hot vector closest to z has its 1 at argmax_j z_j; among equal maxima the
 * lowest index wins (the paper does not say).
 *   z           dev in  [n][K] fp32, finite values
 *   index_out   dev out [n] u8: the argmax
 *   onehot_out  dev out [n][K] fp32 or NULL: the binary vector itself
 * 1 <= K <= 256.  Asynchronous on `stream`.  Errors as above. */
int pat_argmax_binarize(const float *z, int64_t n, int K, uint8_t *index_out, float *onehot_out, void *stream);

/* One reduction step of the library extraction (Algorithm 1, Section 5.2: "calculate the pattern distribution of the
 * current library; remove the patterns with fewest occurrences"), without the training loop: every kernel is given
 * the mask of the library that keeps most of its energy (as in pat_project), the kernels per mask are counted and
 * the K_out most frequent masks stay.  Among masks of equal count the lower id stays; the survivors keep the order
 * they have in masks_in (both are this library's readings, the paper is silent).  The paper's schedule is
 * 126 -> 12 -> 8 or 4 (Section 5.2, Section 7.1): one call per step, the masks_out of one call (copied to the host)
 * being the masks_in of the next.
 *   w           dev in  [n][3][3] fp32: the kernels of all layers that share the library, one after another
 *   masks_in    HOST in [K_in] 9-bit masks with exactly four bits, distinct; 1 <= K_in <= 255
 *   masks_out   dev out [K_out] u16, 1 <= K_out <= K_in
 *   counts_out  dev out [K_in] u64, 8-byte aligned: kernels per mask of masks_in
 * Asynchronous on `stream` (a memset and two kernels); allocates nothing.
 * Errors: PAT_ERR_INVALID_ARG, PAT_ERR_LIBRARY, PAT_ERR_SHAPE, PAT_ERR_ALIGN, PAT_ERR_CUDA. */
int pat_extract_library(const float *w, int64_t n, const uint16_t *masks_in, int K_in, int K_out,
                        uint16_t *masks_out, uint64_t *counts_out, void *stream);

/* Test hooks of the convolution kernels' bounded waits (host-side, process-wide, not thread safe).  The paper has
 * no counterpart.
 *   what = 0  limit of every device-side wait in nanoseconds (value <= 0: back to the default of 2 s);
 *   what = 1  workspace kernels (pat_conv3x3_ws): in every thread block the copy of pipeline stage number `value`
 *             is never issued, so the wait for it runs out after the limit and the kernel ends, with every other
 *             copy landed and its tensor memory released, leaving PAT_ERR_TIMEOUT in the status word
 *             (value < 0: off, the default).
 * Returns PAT_ERR_INVALID_ARG for any other `what`. */
int pat_debug_set(int what, long long value);

#ifdef __cplusplus
}
#endif
#endif /* PATCONV_H_ */
