/*
 * rosaq.h -- C ABI of the B200 (sm_100a) implementation of the ROSAQ inference
 * hot path: the fused mixed-precision rotated linear  y = (x R) W',  W' = R^T W,
 * with W' stored as one FP16 salient group plus INT4/INT3 groups of 128 input
 * channels (fp16 scale and zero-point per group and output column).
 *
 * Notation follows the paper: X calibration activations [N][d], R rotation
 * (eigenvectors of X^T X sorted by descending eigenvalue), W weight [d][d'],
 * K salient channels.  (The paper writes Q(.) for the quantizer; here the
 * quantizer is always spelled "quantize".)
 *
 * Conventions for every call
 *   - All matrices are row-major.  Unless a parameter is marked HOST, pointers are
 *     DEVICE pointers on the device the context was created for, and stay owned
 *     by the caller; the library never frees or keeps them past the call's
 *     completion on `stream` (exception: none).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls are asynchronous on it unless stated otherwise.
 *   - Return value: ROSAQ_OK (0) or a negative rosaq_status.  Nothing is thrown,
 *     printed or aborted.  Argument errors are detected before any launch.
 *   - Device-side waits are bounded; if one expires the kernel records
 *     ROSAQ_ERR_TIMEOUT in the context's device status word (read it with
 *     rosaq_last_status) and returns, leaving the CUDA context usable.
 *   - Handles (rosaq_ctx, rosaq_weight, rosaq_rotation) are owned by the library
 *     and released with the matching *_destroy / *_free.  They are not
 *     thread-safe; use one context per host thread and device.
 */
#ifndef ROSAQ_H_
#define ROSAQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ROSAQ_OK = 0,
  ROSAQ_ERR_INVALID_ARG = -1,       /* null pointer, non-positive size, bad enum */
  ROSAQ_ERR_UNSUPPORTED_SHAPE = -2, /* size not a multiple of what the layout needs */
  ROSAQ_ERR_ALIGNMENT = -3,         /* pointer or leading dimension not 16-byte aligned */
  ROSAQ_ERR_ALLOC = -4,             /* device or host allocation failed */
  ROSAQ_ERR_CUDA = -5,              /* a CUDA runtime/driver call failed */
  ROSAQ_ERR_TIMEOUT = -6,           /* a bounded device-side wait expired */
  ROSAQ_ERR_UNSUPPORTED_ARCH = -7   /* device is not compute capability 10.x */
} rosaq_status;

typedef enum { ROSAQ_F16 = 0, ROSAQ_F32 = 1 } rosaq_dtype;

typedef struct rosaq_ctx rosaq_ctx;           /* per device: workspace + device status word */
typedef struct rosaq_weight rosaq_weight;     /* one quantized linear in the kernels' tiled layout */
typedef struct rosaq_rotation rosaq_rotation; /* one rotation R prepared for online use */
typedef struct rosaq_plan rosaq_plan;         /* a list of rotations / linears that runs as one launch */

/*
 * Description of a rotation R (Section 3.1, Eq. 4; head-wise: Section 3.1.1, Eq. 6).
 * R = blockdiag(q[0], ..., q[n_blocks-1]) followed by a column permutation:
 * column j of R is column perm[j] of the block-diagonal matrix (perm NULL =
 * identity).  n_blocks = 1 is the layer-wise dense rotation.  Columns are
 * expected in descending-eigenvalue order, so that the first K are the salient
 * ones (Section 3.2); the library does not check orthogonality.
 */
typedef struct {
  int32_t d;           /* total dimension */
  int32_t n_blocks;    /* d % n_blocks == 0 */
  const void *q;       /* DEVICE [n_blocks][d/n_blocks][d/n_blocks] */
  int32_t q_dtype;     /* ROSAQ_F32 for rosaq_quantize, ROSAQ_F16 for rosaq_rotation_create */
  const int32_t *perm; /* DEVICE [d] or NULL; must be a permutation of 0..d-1 */
} rosaq_rot;

/* ---- context ---------------------------------------------------------------- */

/* Creates a context on CUDA device `device` (must be compute capability 10.x, else
 * ROSAQ_ERR_UNSUPPORTED_ARCH).  Allocates a small device status word, the workspace
 * through which the CTAs of one rosaq_linear launch exchange partial output tiles
 * (64 KB per CTA of a two-CTAs-per-SM grid, 19 MB on a 148-SM device, plus 4 KB of
 * counters) and, lazily at the first call that needs it, a workspace for the rotated
 * activations.  A context serves one stream at a time: calls on different streams
 * that overlap in time need a context each.  Synchronous. */
int rosaq_create(rosaq_ctx **out, int device);
int rosaq_destroy(rosaq_ctx *ctx);

/* Static, never-NULL description of a status code. */
const char *rosaq_strerror(int status);

/* Synchronizes `stream`, then returns and clears the device status word
 * (ROSAQ_OK or ROSAQ_ERR_TIMEOUT), or ROSAQ_ERR_CUDA if the stream reports an error. */
int rosaq_last_status(rosaq_ctx *ctx, void *stream);

/* Test hook: upper bound, in polling iterations, of every device-side wait
 * (default 1<<20; a positive value replaces it).  Returns the previous value. */
int64_t rosaq_set_wait_limit(rosaq_ctx *ctx, int64_t iterations);

/* Selects the rosaq_linear / rosaq_rotate implementation: 0 = tensor-core path
 * (tcgen05 + TMEM; default), 1 = plain CUDA-core path (slow; for debugging and
 * cross-checks -- it is still a GPU kernel of this library), 2 = tensor-core path with
 * CTA pairs (tcgen05 cta_group::2: two SMs share one MMA stream) wherever the shape allows
 * it (token tile a multiple of 32, an even number of 128-column tiles); the K splits may
 * differ from those of 0, so results agree to fp32 summation order, not bit for bit;
 * 3 = tensor-core path that always splits K across thread-block clusters (0 prefers,
 * for token counts up to 64 and operands with enough column tiles, an equal share of the
 * weight stream per SM with the partial tiles exchanged through a workspace that
 * rosaq_create allocated; again the same sums in another order); 4 = every call of up to 64 tokens runs as
 * ONE persistent launch, the rotation and the linears that consume it included (the kernel of rosaq_plan;
 * for a single call slower than 0, which is why it is not the default -- see rosaq_plan_create);
 * 5 = every weight, at any token count, on the 256-column x 256-token tiles that 0 picks for large batches
 * (rotations and all-fp16 weights stay on the kernels of 0); 6 = calls of 65 ... 1536 tokens as blocks of 128
 * tokens, one operation of the persistent launch per block, in one launch (slower than 0 for a single
 * call: it exists to test that form of the launch).
 * Returns the previous value. */
int rosaq_set_linear_impl(rosaq_ctx *ctx, int impl);

/* Test hook, host only (no GPU, no context): the cut that implementation 0 uses when it gives every CTA an
 * equal share of a launch.  The launch has n_tiles column tiles of `groups` 128-channel groups each, the
 * first g_fp16 of every tile fp16, the others quantized; the tile-major (tile, group) list is cut into
 * n_ctas contiguous ranges of equal cost.  Writes n_ctas + 1 ascending positions to bounds (HOST memory;
 * range i is [bounds[i], bounds[i + 1])).  Returns ROSAQ_OK, ROSAQ_ERR_INVALID_ARG (a non-positive size,
 * g_fp16 > groups, NULL), or ROSAQ_ERR_UNSUPPORTED_SHAPE when the cut is not usable -- a range would be
 * empty or touch more than two tiles -- in which case rosaq_linear splits K across clusters instead. */
int rosaq_plan_equal_shares(int n_tiles, int groups, int g_fp16, int n_ctas, int32_t *bounds);

/* ---- calibration: Eq. 4, left-hand side ---------------------------------------- */

/*
 * C += X^T X  (uncentred, unnormalised Gram matrix), fp32 accumulation.
 *   X        [n_tokens][ldx] of x_dtype (ROSAQ_F16 or ROSAQ_F32); only the first d columns are read
 *   n_blocks 1: C is [d][d].  H > 1 (head-wise, Section 3.1.1): C is [H][d/H][d/H], the
 *            independent Gram matrices of the column slices [h d/H, (h+1) d/H)
 *   C        fp32, zeroed by the caller before the first chunk; may be called
 *            repeatedly to stream a calibration set through in chunks
 * The full square is written (both triangles).  d % 8 == 0, (d / n_blocks) % 8 == 0, X 16-byte aligned.
 */
int rosaq_calib_cov(rosaq_ctx *ctx, const void *X, int x_dtype, int64_t n_tokens, int d,
                    int64_t ldx, int n_blocks, float *C, void *stream);

/* ---- offline: rotate + quantize + pack (Eq. 3, Section 3.3) -------------------- */

/*
 * Builds the mixed-precision representation of W' = R^T W.
 *   W         fp16 [d_in][d_out]
 *   rot       R with q_dtype ROSAQ_F32, rot->d == d_in; NULL = identity (the paper's
 *             rotation-less "Mixed" baseline)
 *   bits      3 or 4;  group must be 128;  k_salient a multiple of 128 in [0, d_in]
 * W' is accumulated in fp32 as one fused multiply-add per term, input channel
 * ascending, so that its bits (and therefore every code) are reproducible.
 * Rows [0, k_salient) of W' are rounded to fp16 and kept; every further group of
 * 128 rows is quantized per output column with asymmetric min/max round-to-nearest:
 *   s = fp16(max(hi-lo, 1e-5) / (2^bits-1)), with an fp16 result of zero replaced by the smallest
 *       subnormal (bits 0x0001) and an infinite one by the largest finite value (0x7bff),
 *   z = clamp(-rint(lo/s), 0, 2^bits-1), stored as +0 when lo >= 0,
 *   code = clamp(rint(w/s) + z, 0, 2^bits-1), all IEEE fp32, ties to even.
 * Allocates the result (*out, release with rosaq_weight_free) and a temporary fp32
 * W' of d_in*d_out floats that is freed before returning.  Synchronizes `stream`.
 * d_in % 128 == 0 required; d_out >= 1 (padded internally to a multiple of 128).
 */
int rosaq_quantize(rosaq_ctx *ctx, const void *W, int d_in, int d_out, const rosaq_rot *rot,
                   int bits, int group, int k_salient, rosaq_weight **out, void *stream);

/*
 * The same for the scaled weight D W (scaling invariance, X W = (X D^-1)(D W); the weight-splitting appendix
 * quantizes the down projection W_D this way, AWQ-style, without rotating it):
 *   in_scale  DEVICE fp32 [d_in], the diagonal of D; NULL = rosaq_quantize.  The paper gives no rule for D:
 *             it is an input, like R; the caller feeds rosaq_linear the activations x D^-1 (R).
 * W'' = R^T (D W): each product d[i] * W[i][n] is rounded once to fp32, then the chain of rosaq_quantize runs
 * on those values (rot == NULL: W'' = D W).  With rot and in_scale both given a second temporary of
 * d_in*d_out floats is allocated and freed.  Everything else as rosaq_quantize.
 */
int rosaq_quantize_scaled(rosaq_ctx *ctx, const void *W, int d_in, int d_out, const rosaq_rot *rot,
                          const float *in_scale, int bits, int group, int k_salient, rosaq_weight **out,
                          void *stream);

/*
 * Interchange layout of a quantized weight (r = row index inside the non-salient part):
 *   qw       uint32; INT4: [(d_in-K)/8][d_out], code of row r in bits [4(r%8), +4) of qw[r/8][n];
 *            INT3: [(d_in-K)/32*3][d_out], rows in blocks of 32 forming the 96-bit little-endian
 *            string qw[3(r/32)+0..2][n], code of row r in bits [3(r%32), +3)
 *   scales, zeros   fp16 [(d_in-K)/128][d_out]
 *   salient  fp16 [K][d_out]
 * export writes the four arrays (any may be NULL to skip it); import builds a handle
 * from them.  Both run on `stream`; import also allocates and synchronizes.
 */
int rosaq_weight_export(rosaq_ctx *ctx, const rosaq_weight *w, uint32_t *qw, void *scales_f16,
                        void *zeros_f16, void *salient_f16, void *stream);
int rosaq_weight_import(rosaq_ctx *ctx, int d_in, int d_out, int bits, int group, int k_salient,
                        const uint32_t *qw, const void *scales_f16, const void *zeros_f16,
                        const void *salient_f16, rosaq_weight **out, void *stream);
int rosaq_weight_free(rosaq_weight *w);
/* HOST out-parameters (any may be NULL); device_bytes = size of the tiled representation. */
int rosaq_weight_info(const rosaq_weight *w, int *d_in, int *d_out, int *bits, int *group,
                      int *k_salient, int64_t *device_bytes);

/* ---- online: x R, and (x R) W' (Eq. 3; Eq. 6 for block-diagonal R) -------------- */

/*
 * Prepares R (q_dtype ROSAQ_F16) for the online rotation: re-tiles it for the
 * kernels and inverts the permutation.  (d / n_blocks) % 128 == 0 required.
 * Allocates; synchronizes `stream`.
 */
int rosaq_rotation_create(rosaq_ctx *ctx, const rosaq_rot *rot, rosaq_rotation **out, void *stream);
int rosaq_rotation_free(rosaq_rotation *r);

/*
 * x_rot[M][ldxr] (fp16) = x[M][ldx] (fp16) . R, fp32 accumulation, rounded once to fp16.
 * Linears that read the same activation (q/k/v, gate/up) share one rotation, so it
 * is exposed on its own.  ldx, ldxr in elements, multiples of 8; 1 <= M.
 */
int rosaq_rotate(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r,
                 void *x_rot, int64_t ldxr, void *stream);

/*
 * y[M][ldy] (fp16) = (x[M][ldx] (fp16) . R) . W^,  where W^ is the dequantized
 * mixed-precision weight: row i < K is the stored fp16 value, otherwise
 * (code - zero) * scale rounded to fp16; fp32 accumulation; y rounded once to fp16.
 *   r == NULL : x is already rotated (only the GEMM stage runs)
 *   r != NULL : x . R goes through the context workspace (grown on demand: this call
 *               may then allocate and synchronize once), then the GEMM stage runs
 * Only the first d_out columns of each y row are written.  ldx, ldy multiples of 8.
 * Any M >= 1.  The kernel is chosen by size: up to 64 tokens the weight-streaming kernels; large batches
 * (more than 256 tokens, when the launch has at least 40 tiles of 256 columns x 256 tokens and 36
 * 128-channel groups of work per pair of SMs) run on those tiles, each shared by two CTAs on adjacent SMs
 * (tcgen05 cta_group::2, one dequantisation of a weight tile per 256 tokens); everything in between one
 * 128-token tile per CTA.  The choice changes the order of the fp32 sums only; a call gives the same bits
 * every time.  Calls of one context that use the exchange workspace (the large-batch tiles, the
 * equal-share kernel, rosaq_plan_run) must not overlap on the GPU: keep them on one stream.
 */
int rosaq_linear(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r,
                 const rosaq_weight *w, void *y, int64_t ldy, void *stream);

/*
 * Several linears that read the same activation (q/k/v, or gate/up: they share one rotation, Section 3.1)
 * in one launch:  y[i] = (x . R) . W^[i]  for i < n, 1 <= n <= 4.  Each y[i] is the sum rosaq_linear would
 * compute; how K is split among CTAs depends on the number of column tiles in a launch, so the two agree
 * to fp32 summation order -- bit for bit where the splits coincide (small operands), within a few 1e-5
 * relative otherwise.  Repeated launches of the same call always give the same bits.
 * All w[i] must have the same d_in, bits and k_salient; d_out may differ.  w, y and ldy are
 * HOST arrays of n entries (device pointers inside); they are read before the call returns.
 * r as in rosaq_linear (the rotation runs once).  Errors as rosaq_linear.
 */
int rosaq_linear_multi(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r, int n,
                       const rosaq_weight *const *w, void *const *y, const int64_t *ldy, void *stream);

/*
 * A list of operations that runs as ONE persistent launch (up to 128 tokens): every rotation x . R
 * (Eq. 2; Eq. 6 for block-diagonal R) and every GEMM stage x' . W^ (Eq. 3) of, say, a decoder layer.
 * All CTAs of the grid stream the operands of the whole list back to back; an operation whose input is
 * another operation's output starts when that output is complete.  It pays off for long lists (the ten
 * operations of a 7B decoder layer: 66 us against 100 us as seven calls); for one or two operations the
 * single calls are faster (rotation + 4096 -> 4096 linear: 30 us as a plan, 21 us as rosaq_linear).
 *   op.r / op.w  exactly one is non-NULL: the operation is y = x . R, or y = x . W^ (x already rotated)
 *   op.x, ldx    DEVICE [M][ldx] fp16 input; ignored when x_from >= 0
 *   op.x_from    -1, or the index (smaller than this operation's) of the operation whose y is this one's
 *                input (a rotation feeding its linears); that y must have this operation's d_in columns
 *   op.y, ldy    DEVICE [M][ldy] fp16 output; the first d_out columns of each row are written
 * Operations without x_from are independent of each other and may run in any order or at the same time:
 * a y that overlaps another operation's y, or any x other than through x_from (its own operation's x
 * included), is rejected with ROSAQ_ERR_INVALID_ARG (column ranges of one wider buffer with the same row
 * stride do not overlap; views with different row strides must not share any address range).  All quantized weights of a list
 * have the same bit width.  1 <= M <= 128 and 1 <= n_ops <= 12, otherwise ROSAQ_ERR_UNSUPPORTED_SHAPE.
 * From 65 tokens on the launch keeps accumulators of 128 tokens (a 7B decoder layer: 97 us at 128 tokens,
 * 65 us at 64).
 * Each y is the sum rosaq_linear computes, added in an order that depends on how the list is divided
 * among the CTAs: results agree with the separate calls to fp32 summation order (a few 1e-5 relative) and
 * are the same bits on every run of the same plan.
 * rosaq_plan_create reads `ops` (HOST array) before it returns, may allocate device memory and may
 * synchronize the device; create the plans a CUDA graph will replay before capturing it.
 * rosaq_plan_run launches on `stream` and allocates nothing; runs of plans of one context must not
 * overlap on the GPU (they share the context's exchange workspace): keep them on one stream.
 * The pointers inside ops, and the rotation and weight handles, must stay valid while the plan is used.
 */
typedef struct {
  const void *x;
  int64_t ldx;
  int32_t x_from;
  const rosaq_rotation *r;
  const rosaq_weight *w;
  void *y;
  int64_t ldy;
} rosaq_op;
int rosaq_plan_create(rosaq_ctx *ctx, int M, int n_ops, const rosaq_op *ops, rosaq_plan **out);
int rosaq_plan_run(rosaq_ctx *ctx, const rosaq_plan *plan, void *stream);
int rosaq_plan_free(rosaq_plan *plan);

/* Test and tuning hook: the relative cost of an fp16 group, a quantized group and a started tile that
 * rosaq_plan_create (and the single calls, which plan internally) use from now on to cut a phase into
 * equal shares (defaults 12, 7, 1 for single CTAs and 10, 7, 1 for pairs; 1 <= cost <= 1000, tile >= 0).
 * Changes how K is divided among the CTAs, hence the fp32 summation order of later plans; plans already created keep theirs. */
int rosaq_set_plan_costs(rosaq_ctx *ctx, int fp16_group, int quant_group, int tile);

/* Test and tuning hook: enable != 0 lets the persistent launch run as pairs of CTAs that share one
 * MMA stream over two adjacent column tiles (tcgen05 cta_group::2) wherever the operands allow it; 0 (the default)
 * forces single CTAs.  The two cut K differently: results agree to fp32 summation order.  Applies to plans created
 * afterwards.  Returns the previous setting (1 or 0), or a negative status. */
int rosaq_set_plan_pairs(rosaq_ctx *ctx, int enable);

/* Number of CTAs of the persistent launch on the context's device (one per SM), or a negative status. */
int rosaq_plan_ctas(rosaq_ctx *ctx);

/*
 * Test hook, host only (no GPU, no context): how a list of operations is divided among n_ctas CTAs.
 * Operation i has n_tiles[i] column tiles of groups[i] 128-channel groups, the first g_fp16[i] of each
 * tile fp16; x_from[i] as in rosaq_op; copies[i] >= 1 (NULL: all 1) computes every tile of the operation that
 * many times, each copy writing an equal share of the token rows (what the library does, four-fold, for
 * block-diagonal rotations with a column permutation, whose output is a scatter bound by the store rate
 * of one SM).  An operation runs in a later phase than the one it reads from; operations that neither read
 * nor feed another one run in a phase of their own between the producers and their readers (the readers
 * then find the producers' outputs complete instead of waiting for the exchange of shared tiles); inside
 * a phase the (operation, tile, group) list is cut into n_ctas contiguous ranges of equal cost, and a
 * range is a sequence of pieces (the groups of one tile).  Writes piece_begin[0..n_ctas] (CTA c owns pieces
 * piece_begin[c] .. piece_begin[c + 1] - 1, in the order it processes them) and, for the first max_pieces
 * pieces, twelve int32 each: operation, tile, first group, end group, holders of the tile (copy), this
 * piece's position among them (ascending K), first partial-tile slot, arrival counter, closer index (-1: the
 * piece only contributes its partial tile; k >= 0: its CTA adds the partial tiles of token rows k,
 * k + closers, ...), closers, and the token rows [begin, end) out of 64 that the tile (copy) writes.
 * All arrays HOST.  Returns the total number of pieces, or a negative status.
 */
int rosaq_plan_schedule(int n_ops, const int32_t *n_tiles, const int32_t *groups, const int32_t *g_fp16,
                        const int32_t *x_from, const int32_t *copies, int n_ctas, int32_t *piece_begin,
                        int32_t *pieces, int max_pieces);

/*
 * Same result as rosaq_linear, for callers that cannot allocate device memory.  (The paper has
 * no counterpart; this entry point exists for deployment reasons only.)
 *
 * rosaq_linear keeps the rotated activations x . R in a context workspace that it grows with
 * cudaMalloc on demand.  A process whose memory pool already owns all free device memory, a
 * latency-critical loop that cannot take the device-wide synchronisation of an allocation, or a
 * host framework that forbids allocations outside its own allocator cannot use that.  This
 * variant keeps x . R in a fixed 4 MiB array inside the library image instead (every GPU that
 * loads the library holds those 4 MiB until the process exits) and calls neither cudaMalloc nor
 * cudaFree nor any allocating routine.  Inputs and outputs are still the caller's buffers.
 *   - Limit: with r != NULL, M * d_in * 2 bytes must fit in 4 MiB (for example 512 tokens at
 *     d_in = 4096); larger calls return ROSAQ_ERR_UNSUPPORTED_SHAPE and launch nothing.  With
 *     r == NULL no scratch is needed and there is no limit.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device made current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it.
 *     Nothing in it has to start at zero: each call overwrites the [M][d_in] region it then
 *     reads.  Two calls that may overlap on the GPU (different streams, or several host threads)
 *     race on it and corrupt each other; serialise them on one stream.
 * Arguments, alignment rules and status codes otherwise as rosaq_linear.
 */
int rosaq_linear_static(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r,
                        const rosaq_weight *w, void *y, int64_t ldy, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* ROSAQ_H_ */
