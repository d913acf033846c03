/*
 * libsste -- the S-STE 2:4 sparse-training linear layer for NVIDIA B200 (sm_100a).
 *
 * One training iteration of an S-STE linear (Sec. 2: prune, run forward/backward
 * with the sparse weight, update the dense weight) maps onto these calls:
 *
 *   step 0 only   sste_beta_init          beta = <w,S_soft(w)> / ||S_soft(w)||^2      (Eq. 5)
 *   every step    sste_project_compress   w~ = beta * S_soft(w), 2:4 values + metadata (Eq. 4, Sec. 4.2)
 *                 sste_linear_fwd         Z = X w~^T            sparse tensor cores   (Sec. 5.1)
 *                 sste_mvue_sparsify      MVUE(grad_Z^T)        2:4 along tokens      (Sec. 5.1)
 *                 sste_linear_bwd_weight  grad_W = MVUE(grad_Z^T) X   sparse          (Sec. 5.1)
 *                 sste_linear_bwd_input   grad_X = grad_Z w~          dense           (Sec. 5.1)
 *   FP8 variant   sste_amax, sste_project_amax, sste_quantize_fp8 + the E4M3/E5M2 dtypes (Sec. 5.2)
 *
 * Conventions (all entry points)
 *   - Every tensor pointer is DEVICE memory owned by the caller, row-major and
 *     contiguous.  The library allocates no tensor memory and keeps no pointer
 *     after a call returns.  Scalars beta / scales are DEVICE pointers to one
 *     float so that no call needs a host synchronisation.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it.
 *     Kernels are launched with programmatic stream serialisation: a kernel of
 *     this library may be scheduled while the previous kernel of the stream
 *     drains, but reads or writes global memory only once that kernel has
 *     completed, so stream order holds for every caller-visible effect, also
 *     between these calls and the caller's own kernels, copies and captures.
 *   - Two calls that may overlap on the device (different streams) need
 *     different contexts if either is a product: the split-K workspace belongs
 *     to the context.
 *   - O = out features, I = in features, T = tokens.  O, I and T must be
 *     multiples of 128 and tensor pointers 128-byte aligned, otherwise
 *     SSTE_ERR_SHAPE / SSTE_ERR_ALIGN is returned BEFORE anything is launched.
 *   - A device that is not compute capability 10.x gives SSTE_ERR_ARCH.  There
 *     is no CPU or other fallback.
 *   - Kernels never trap.  Every device-side wait is bounded (2 s of wall time,
 *     %globaltimer); one that expires records SSTE_ERR_TIMEOUT in the context's
 *     device status word, read by sste_poll_device_status, and the kernel leaves
 *     with that product's output incomplete: poll before trusting results.
 *   - bf16 tensors hold IEEE bfloat16 bit patterns, E4M3 is the "fn" flavour
 *     (max 448, no infinity), E5M2 is IEEE-like (max finite 57344).
 *   - FP8 per-tensor scaling (Sec. 5.2, "per-tensor rescaling before casting"): a tensor x is quantised as
 *     q = cast(fl32(x * s)), s = fl32(fp8_max / amax(x)) (s = 1 if amax(x) = 0).  The state of a quantised tensor
 *     is its AMAX, one device float: every call that quantises, or that consumes a quantised operand, takes the
 *     `*_amax_dev` pointer and forms s itself with exactly these operations (so no separate kernel computes scales
 *     or their products); a product multiplies its fp32 accumulator by fl32(fl32(1/s_a) * fl32(1/s_b)).  With bf16
 *     operands these pointers are NULL.
 *
 * Compressed 2:4 operand ("vals" + "meta") of a logical [rows, K] matrix whose
 * groups of four run along K:
 *   vals  [rows, K/2]  the two kept values of every group, ascending position, row-major.
 *   meta  one 4-bit code per group: p0 | (p1 << 2), p0 < p1 the kept positions.  Codes are
 *         stored in the image the sparse tensor-core instruction reads from tensor memory,
 *         as 2 KB atoms of 128 rows x 128 logical K, atom (rb, kb) at byte
 *         (rb * (K/128) + kb) * 2048.  Inside an atom, row m and K-offset k (group k/4):
 *           16-bit operands:  byte = 16*(m&7) + 2*((m>>3)&1) + 256*(m>>4) + 128*((k>>4)&1) + 4*(k>>5) + ((k>>3)&1)
 *           8-bit operands:   byte = 16*m + (k>>3)
 *         and the code sits in the low nibble when (k>>2)&1 == 0, else the high nibble.
 *         sste_meta_to_canonical converts to the plain row-major form
 *         uint16 [rows, K/16], group g of a row at bits [4(g%4), 4(g%4)+4) of word g/4.
 */
#ifndef SSTE_H
#define SSTE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sste_ctx sste_ctx;

typedef enum {
    SSTE_OK = 0,
    SSTE_ERR_INVALID_ARG = 1, /* null pointer, bad enum value */
    SSTE_ERR_SHAPE = 2,       /* a dimension is not a positive multiple of 128 */
    SSTE_ERR_DTYPE = 3,       /* dtype combination not supported by this call */
    SSTE_ERR_ALIGN = 4,       /* pointer not 128-byte aligned */
    SSTE_ERR_WORKSPACE = 5,   /* workspace missing or too small */
    SSTE_ERR_ARCH = 6,        /* device is not sm_100 */
    SSTE_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed */
    SSTE_ERR_DEGENERATE = 8,  /* beta: S_soft(W) is identically zero; beta was set to 1 */
    SSTE_ERR_TIMEOUT = 9      /* a bounded device-side wait expired */
} sste_status;

typedef enum { SSTE_BF16 = 0, SSTE_F32 = 1, SSTE_E4M3 = 2, SSTE_E5M2 = 3 } sste_dtype;

/* Bytes of caller-owned device workspace a context needs (status word + reduction scratch). */
size_t sste_workspace_bytes(void);
/* A larger workspace (this many bytes or more) also lets the three products split their reduction
 * dimension over several CTA pairs when a product has fewer output tiles than the GPU has CTA pairs
 * (fp32 partial tiles live in the workspace); with the minimal workspace they never split. */
size_t sste_workspace_bytes_recommended(void);

/*
 * Create a context on `device`.  `workspace` is device memory of at least
 * sste_workspace_bytes() bytes, 256-byte aligned, owned by the caller and kept
 * alive until sste_destroy.  The call zeroes the status word (synchronously).
 * Calls that share a context must be stream-ordered with respect to each other.
 */
sste_status sste_create(sste_ctx **ctx, int device, void *workspace, size_t workspace_bytes);
sste_status sste_destroy(sste_ctx *ctx);
const char *sste_status_string(sste_status s);

/* Synchronise `stream`, read and clear the device status word.  SSTE_OK if nothing was recorded. */
sste_status sste_poll_device_status(sste_ctx *ctx, void *stream);

/* Sizes of a compressed operand of a logical [rows, k] matrix. */
size_t sste_vals_bytes(int rows, int k, sste_dtype dt);
size_t sste_meta_bytes(int rows, int k);

/*
 * Eq. 5 (Sec. 4.2, "Minimizing MSE"): beta = <w, S_soft(w)> / ||S_soft(w)||^2 over the whole
 * tensor, S_soft as in Eq. 4 with groups of four along I.  Products and sums are fp64 in a
 * fixed order (reproducible run to run); the result is rounded once to fp32 into *beta_dev.
 * The paper computes beta in the first iteration only and then freezes it (Sec. 4.2,
 * "Freezing scaling factor"): call this once and keep the scalar.
 * W: bf16 [O, I].  If S_soft(W) == 0 the call stores 1.0 and records SSTE_ERR_DEGENERATE
 * in the status word.  Uses the context workspace as scratch.
 */
sste_status sste_beta_init(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt,
                           float *beta_dev, void *stream);

/*
 * Eq. 4 + Sec. 4.2: w~ = beta * S_soft(w).  Per group of four along I, t = 2nd-smallest |w|,
 * s = sign(w) * max(|w| - t, 0) (one fp32 subtraction), w~ = fl32(s * beta)
 * [FP8: fl32(w~ * s_w)], one round-to-nearest-even cast to `odt` (E4M3: saturating).
 * Pruned entries are +0.  Kept positions: rank by (|w| descending, index ascending), keep two.
 * W: bf16 [O, I].  odt: SSTE_BF16 or SSTE_E4M3.  w_amax_dev: device float holding max|w~| of the bf16
 * projection (from sste_project_amax), from which s_w is formed; NULL for bf16.
 * Outputs: vals [O, I/2] and meta (see top); dense_out (nullable) [O, I] in odt: the dense copy of w~.
 * sste_linear_bwd_input can work from (vals, meta) alone, so the dense copy is optional.
 */
sste_status sste_project_compress(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt,
                                  const float *beta_dev, const float *w_amax_dev, sste_dtype odt,
                                  void *vals, void *meta, void *dense_out, void *stream);

/*
 * Sec. 5.1: Z = X S(W)^T on sparse tensor cores.  X [T, I], (vals, meta) the compressed w~
 * [O, I], both of dtype opdt (SSTE_BF16, or SSTE_E4M3 for the FP8 variant).  fp32 accumulation.
 * Y [T, O] of dtype ydt (SSTE_BF16 or SSTE_F32) = acc [* 1/s_x * 1/s_w for E4M3 operands: x_amax_dev and
 * w_amax_dev are then the amax X and w~ were quantised with; both NULL for bf16, else SSTE_ERR_INVALID_ARG].
 * y_amax_out_dev (nullable, device float): receives max|Y| of the stored output (the call zeroes it on the
 * stream, the epilogue raises it by atomic maximum), so that a following layer that quantises Y needs no
 * separate amax pass.
 */
sste_status sste_linear_fwd(sste_ctx *ctx, const void *X, int T, const void *vals, const void *meta,
                            int O, int I, sste_dtype opdt, const float *x_amax_dev, const float *w_amax_dev,
                            void *Y, sste_dtype ydt, float *y_amax_out_dev, void *stream);

/*
 * Sec. 5.1: minimum-variance unbiased 2:4 sparsification of grad_Z^T (the paper applies MVUE to
 * the output gradient only).  Groups are 4 consecutive tokens of one output column.  Inclusion
 * probabilities p_i = min(1, c|a_i|), sum 2; kept values a_i / p_i; joint law = systematic
 * sampling with one uniform per group.  Group (column j, token group tg) has the GLOBAL index
 * g = (token_offset/4 + tg)*O + j, where token_offset is the number of tokens that precede this
 * call's dY in the whole batch (0 on one GPU; a data-parallel rank passes the start of its token
 * shard, a multiple of 4, so that the draws do not depend on how the batch is sharded).
 * Philox4x32-10 with counter (lo32(g>>2), hi32(g>>2), tensor_id, step) and key
 * (lo32(seed), hi32(seed)); the group uses output word g&3, u = (word >> 8) * 2^-24.
 * dY: bf16 [T, O].  odt: SSTE_BF16, or SSTE_E5M2 with values fl32(v * s_g), s_g formed from
 * *g_amax_dev = max|dY| (non-NULL then).  Outputs: the compressed operand of the TRANSPOSED matrix, logical
 * [O, T]: gvals [O, T/2], gmeta (see top).  dense_q_out (nullable, FP8 only): E5M2(fl32(dY * s_g)) [T, O].
 * counter_cols: the number of columns the group index counts with, g = (token_offset/4 + tg)*counter_cols + j;
 * 0 means O.  A caller that padded O up to a multiple of 128 passes the unpadded column count, so that the draws
 * of the real columns are those of the unpadded problem (columns j >= counter_cols must be all zero: a zero
 * group yields zeros whatever its draw).
 */
sste_status sste_mvue_sparsify(sste_ctx *ctx, const void *dY, int T, int O, sste_dtype gdt,
                               uint64_t seed, uint32_t tensor_id, uint32_t step, uint64_t token_offset,
                               int counter_cols, const float *g_amax_dev, sste_dtype odt,
                               void *gvals, void *gmeta, void *dense_q_out, void *stream);

/*
 * Sec. 5.1: grad_X = grad_Z S(W), a dense product (the 2:4 structure of S(W) lies along I, which
 * is not the reduction dimension here).  dY [T, O] of dtype gdt (SSTE_BF16 / SSTE_E5M2).  S(W) [O, I] of
 * dtype wdt (SSTE_BF16 / SSTE_E4M3) is given EITHER as the dense copy Wt_dense written by
 * sste_project_compress, OR (Wt_dense = NULL) as the forward's compressed operand (vals, meta): the kernel then
 * expands each K slice into the dense shared-memory operand itself (+0 in the pruned positions), the same
 * product bit for bit, and the dense copy need not exist.  dX [T, I] of dtype xdt = acc [* 1/s_g * 1/s_w for FP8
 * operands, from g_amax_dev / w_amax_dev; NULL for bf16].  dx_amax_out_dev: nullable, max|dX| as for the forward.
 */
sste_status sste_linear_bwd_input(sste_ctx *ctx, const void *dY, int T, int O, sste_dtype gdt,
                                  const void *Wt_dense, const void *vals, const void *meta, int I, sste_dtype wdt,
                                  const float *g_amax_dev, const float *w_amax_dev,
                                  void *dX, sste_dtype xdt, float *dx_amax_out_dev, void *stream);

/*
 * Sec. 5.1: grad_W = MVUE(grad_Z^T) X on sparse tensor cores.  (gvals, gmeta) logical [O, T] of
 * dtype gdt (SSTE_BF16 / SSTE_E5M2) from sste_mvue_sparsify, X [T, I] of dtype xdt
 * (SSTE_BF16 / SSTE_E4M3).  dW [O, I] of dtype dwdt (SSTE_BF16 or SSTE_F32) = acc [* 1/s_g * 1/s_x for FP8
 * operands, from g_amax_dev / x_amax_dev; NULL for bf16].
 * Straight-through estimator (Eq. 3): this gradient is applied to the dense weight unchanged.
 */
sste_status sste_linear_bwd_weight(sste_ctx *ctx, const void *gvals, const void *gmeta, int O, int T,
                                   sste_dtype gdt, const void *X, int I, sste_dtype xdt,
                                   const float *g_amax_dev, const float *x_amax_dev,
                                   void *dW, sste_dtype dwdt, void *stream);

/*
 * The same beta as sste_beta_init, for callers that cannot allocate device memory at all (the paper has
 * no counterpart of this call; it exists for deployment).  A serving or training runtime that owns the
 * whole memory pool, a plug-in that is handed only its inputs and outputs, or a job on a full device has
 * no workspace to lend and therefore no sste_ctx.  This call needs neither: its reduction scratch is a
 * fixed array inside the library image (about 129 KB that every GPU loading the library holds until the
 * process exits).  It calls no cudaMalloc / cudaFree or other allocating routine.
 *   device   ordinal of the GPU that W and beta_dev live on (made current for the call); SSTE_ERR_ARCH
 *            unless it is compute capability 10.x.
 *   W        bf16 [O, I], O and I multiples of 128.  One partial per 128 x 128 tile is kept, and the array
 *            holds 8192 of them: (O/128)*(I/128) > 8192 returns SSTE_ERR_WORKSPACE and launches nothing.
 *   beta_dev device float, written asynchronously on `stream`.  If S_soft(W) is identically zero it
 *            receives 1.0 (there is no context, so no status word records it).
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that first
 * call outside any stream capture.  All calls on a device share the one array: each call clears the ticket
 * counter it needs at zero and overwrites the partials, so results never depend on earlier calls, but two
 * calls whose kernels overlap on the GPU (different streams without ordering) race.  Sums are combined in
 * tile order: the result is reproducible, and equals sste_beta_init up to the rounding of a different
 * summation order (about 1e-7 relative).
 */
sste_status sste_beta_init_static(int device, const void *W, int O, int I, sste_dtype wdt, float *beta_dev,
                                  void *stream);

/* ---- FP8 whole-process variant (Sec. 5.2): per-tensor rescaling before the cast ---- */

/* *amax_dev = max |x| over n bf16 elements (n % 8 == 0).  Exact, order-free.  The call first sets
 * *amax_dev to 0 on the stream, then raises it with an atomic maximum. */
sste_status sste_amax(sste_ctx *ctx, const void *x, size_t n, sste_dtype dt, float *amax_dev, void *stream);

/* *amax_dev = max |w~| of the bf16 projection w~ = bf16(beta * S_soft(W)) (what sste_project_compress would
 * write as dense_out with odt = SSTE_BF16), computed from W [O, I] bf16 and *beta_dev without writing w~: the
 * scale of the E4M3 weight operand needs this maximum before the operand can be cast (Sec. 5.2).  Bit-identical
 * to sste_amax of that projection.  The call first sets *amax_dev to 0 on the stream. */
sste_status sste_project_amax(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt, const float *beta_dev,
                              float *amax_dev, void *stream);

/* Inspection helper (no call of the path needs it: they form the scale from the amax themselves):
 * *scale_dev = fl32(fp8_max(odt) / *amax_dev) (1 if amax is 0); *inv_scale_dev (nullable) = fl32(1 / scale). */
sste_status sste_fp8_scale(sste_ctx *ctx, const float *amax_dev, sste_dtype odt, float *scale_dev,
                           float *inv_scale_dev, void *stream);

/* q = cast_rn_satfinite(fl32(x * s)), s formed from *amax_dev = max|x| (see top); x bf16, q E4M3 or E5M2;
 * n % 16 == 0. */
sste_status sste_quantize_fp8(sste_ctx *ctx, const void *x, size_t n, const float *amax_dev,
                              sste_dtype odt, void *q, void *stream);

/* ---- ablation variants of the pruning step (the axes of the paper's ablations; not on the default path) ---- */

typedef enum { SSTE_PRUNE_SOFT = 0, SSTE_PRUNE_HARD = 1 } sste_pruning;

/*
 * sste_project_compress with the paper's knobs.  SSTE_PRUNE_SOFT: soft thresholding (Eq. 4) with the
 * interpolated threshold t = (1 - gamma) |t2| + gamma |t3|, |t2| <= |t3| the second and third smallest
 * magnitudes of the group (Sec. 4.1; gamma in [0, 1], gamma = 0 is the method and runs the same kernel as
 * sste_project_compress); fp32: t = fl(fl(fl(1 - gamma) |t2|) + fl(gamma |t3|)).  SSTE_PRUNE_HARD: hard
 * thresholding (Eq. 2): the two largest magnitudes are kept unchanged, gamma is ignored.  Both are then
 * multiplied by *beta_dev (pass 1.0 for plain hard thresholding) and cast; all other arguments, layouts and
 * errors as sste_project_compress; SSTE_ERR_INVALID_ARG for an unknown pruning or gamma outside [0, 1].
 */
sste_status sste_project_compress_variant(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt,
                                          const float *beta_dev, const float *w_amax_dev, sste_dtype odt,
                                          sste_pruning pruning, float gamma, void *vals, void *meta,
                                          void *dense_out, void *stream);

/* beta = ||w||_1 / ||S_soft(w)||_1: the magnitude-preserving rescaling the method replaces by Eq. 5 (Sec. 4.2,
 * "Minimizing MSE").  Arguments, reduction order and degenerate case as sste_beta_init. */
sste_status sste_beta_init_l1(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt, float *beta_dev,
                              void *stream);

/*
 * Sparse-refined STE (Sec. 3.2): dW += lambda * w on the entries the 2:4 mask prunes, the gradient of
 * (lambda / 2) ||w (1 - m_h(w))||^2; kept entries are left as they are.  W [O, I] bf16 and dW [O, I] bf16
 * (updated in place; fp32 add and multiply, one cast), meta: the metadata image of W written by
 * sste_project_compress[_variant] (meta_dt: the dtype that image was written for, it selects the layout).
 */
sste_status sste_srste_decay(sste_ctx *ctx, const void *W, const void *meta, int O, int I, sste_dtype meta_dt,
                             float lambda, void *dW, void *stream);

/* ---- training diagnostics ---- */

/*
 * Flip count between two iterations (Sec. 3.1, "Flip rate": r_k = || m_h(w_k) xor m_h(w_{k-1}) ||_1 / d).
 * meta_prev, meta_cur: device, the metadata images sste_project_compress wrote for the same [rows, k] weight
 * at two iterations (same dtype, hence same layout; 16-byte aligned).  The 2:4 metadata IS the hard-threshold
 * mask m_h: the kept pair of a group is its two largest magnitudes.  *count_dev (device, 8-byte aligned)
 * receives the number of mask entries that differ; the call first sets it to 0 on the stream.  The flip rate
 * is *count_dev / (rows * k).  Errors: SSTE_ERR_SHAPE unless rows and k are multiples of 128.
 */
sste_status sste_flip_count(sste_ctx *ctx, const void *meta_prev, const void *meta_cur, int rows, int k,
                            unsigned long long *count_dev, void *stream);

/* ---- shapes that are not multiples of 128 ---- */

/*
 * Every call above wants O, I and T to be multiples of 128.  Other shapes (a 50257-row vocabulary projection,
 * a batch of 1000 tokens) are run on zero-padded copies: a group of four zeros is a fixed point of Eq. 4 and of
 * the MVUE rule, contributes nothing to beta (Eq. 5), to an amax or to a product, so the results on the real
 * rows and columns are those of the unpadded problem (for MVUE pass counter_cols = the unpadded column count).
 * sste_padded_dim(n) = the next multiple of 128.  sste_pad_2d copies src [rows, cols] into the top-left corner
 * of dst [rows_p, cols_p] (rows_p >= rows, cols_p >= cols, cols_p % 8 == 0, dst 16-byte aligned) and zero-fills
 * the rest; sste_crop_2d copies the top-left [rows, cols] corner of src [rows_p, cols_p] into dst [rows, cols].
 * Elements are 2 bytes (bf16).  Both are single passes over the larger tensor.
 */
int sste_padded_dim(int n);
sste_status sste_pad_2d(sste_ctx *ctx, const void *src, int rows, int cols, void *dst, int rows_p, int cols_p,
                        void *stream);
sste_status sste_crop_2d(sste_ctx *ctx, const void *src, int rows_p, int cols_p, void *dst, int rows, int cols,
                         void *stream);

/* ---- test / debug helpers ---- */

/* Compressed operand (vals [rows, k/2] + metadata image) -> dense [rows, k] of the same dtype dt (SSTE_BF16,
 * SSTE_E4M3 or SSTE_E5M2), +0 in the pruned positions: the matrix the sparse tensor-core instruction sees. */
sste_status sste_decompress(sste_ctx *ctx, const void *vals, const void *meta, int rows, int k, sste_dtype dt,
                            void *dense_out, void *stream);

/* Operand-image metadata -> canonical uint16 [rows, k/16] (see top).  dt selects the 16-bit or 8-bit image. */
sste_status sste_meta_to_canonical(sste_ctx *ctx, const void *meta, int rows, int k, sste_dtype dt,
                                   void *canonical_out, void *stream);

/* Number of kernels this library has launched in the process so far (all entry points, all contexts; a
 * product that splits its reduction counts its second pass too).  A benchmark reports the difference
 * around its timed region. */
unsigned long long sste_debug_launch_count(void);

/* The three products pick the width of their output tiles (128, 192 or 256 columns) from the problem
 * shape.  This process-wide hook pins it so that tests can cover every variant; widths a product does
 * not support (192 needs a K-major B operand, i.e. the forward) fall back to the automatic choice.
 * bn: 0 (automatic), 128, 192, 224 (forward only) or 256; anything else gives SSTE_ERR_INVALID_ARG. */
sste_status sste_debug_force_tile_width(int bn);
/* Same for the split-K factor: 0 (automatic) or 1..4; a factor the shape or the workspace does not allow
 * falls back to the automatic choice. */
sste_status sste_debug_force_splits(int splits);

/* The products hand their output tiles to the CTA pairs band by band (a band = group_m consecutive rows of
 * 256-row tiles, row index fastest inside a band), with group_m chosen from the operand sizes so that operands
 * are read from HBM about once.  This hook pins group_m (0 = automatic; values above the number of tile rows mean
 * plain column-major order) so that tests can cover every order. */
sste_status sste_debug_force_tile_order(int group_m);

/* The MVUE rule of sste_mvue_sparsify on explicit groups and explicit uniforms, for tests that must reach the cases
 * a random draw almost never produces (u = 1 - 2^-24, sums that round onto a sampling point, zero magnitudes).
 * a: device, n groups of four bf16 values; k24: device, n uint32 whose low 24 bits k give u = k * 2^-24;
 * pos_out: device uint32 [n], q0 | q1 << 2 with q0 < q1 the kept positions; val_out: device float [n][2], the two
 * kept values in fp32 before any cast. */
sste_status sste_debug_mvue_groups(sste_ctx *ctx, const void *a, const void *k24, size_t n, void *pos_out,
                                   void *val_out, void *stream);

/* What the library would decide for a product launch, computed on the host (no device is touched): product 0 =
 * sste_linear_fwd, 1 = sste_linear_bwd_weight, 2 = sste_linear_bwd_input (dense operand), operands of dtype opdt,
 * bf16 output, on a GPU of sm_count SMs with a context workspace of workspace_bytes.  Outputs (each nullable): the
 * tile width, the split-K factor and the first split tile, the band height of the tile order.  The debug hooks
 * above apply.  sste_debug_tile_coords maps a tile number to its (row, column) of tiles under a band height. */
sste_status sste_debug_plan(int product, sste_dtype opdt, int O, int I, int T, int sm_count, size_t workspace_bytes,
                            int *tile_width, int *splits, int *split_from, int *group_m);
sste_status sste_debug_tile_coords(int tile, int m_tiles, int n_tiles, int group_m, int *mt, int *nt);

/* Host-only self-check of the once-per-device bookkeeping behind per-device kernel attributes (a context may live on
 * any device ordinal, and the opt-in to large dynamic shared memory is per device).  SSTE_OK if it behaves. */
sste_status sste_debug_selftest_device_once(void);

/* Test hook for the bounded waits.  While armed (on != 0), a dense sste_linear_bwd_input (Wt_dense given, bf16
 * output) whose output is ONE tile (T <= 256, I <= 256) leaves the last K stage of its operand pipeline unloaded
 * and limits every device-side wait to one millisecond instead of two seconds: the wait for that stage runs out,
 * the kernel records SSTE_ERR_TIMEOUT in the status word, abandons the tile and returns (dX is not written).
 * Nothing traps or spins, the context stays usable.  Any other product call returns SSTE_ERR_INVALID_ARG while
 * the hook is armed.  Process-wide; disarm with 0. */
sste_status sste_debug_inject_stall(int on);

#ifdef __cplusplus
}
#endif
#endif /* SSTE_H */
