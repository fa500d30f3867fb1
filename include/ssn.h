/*
 * libssn -- subspace-network (SSN) stage-boundary codec for NVIDIA B200 (sm_100a).
 *
 * The four operations are the ones the Agora paper defines in Sec. 4.1 ("Pipeline-Parallel
 * Communication with Reparameterized SSNs"); each declaration below cites the passage that
 * defines it.  Notation: n tokens, model width d, subspace rank k,
 *
 *     X, G, Xhat  [n x d]   hidden states / activation-gradients, one row per token
 *     Z, dZ       [n x k]   the coordinates that cross the stage boundary
 *     U           [d x k]   orthonormal basis U_k of the shared subspace
 *     E           [vocab x d]    fixed token embedding T_fixed (row ids[t] belongs to token t)
 *     P           [max_pos x d]  positional embedding PE (row pos[t] belongs to token t)
 *
 * Common rules for every entry point
 *   - All matrices are row-major with a leading dimension `ld*` counted in ELEMENTS
 *     (ld >= number of columns).  One element type (`ssn_dtype_t`) is used for all of
 *     X, G, Xhat, Z, dZ, W, U, E, P of a call; accumulation is always fp32.
 *   - Every data pointer is a DEVICE pointer owned by the caller, except where a parameter is
 *     explicitly called a host array.  The library never allocates, frees or synchronises;
 *     each call only enqueues kernels on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and returns.
 *   - The `ssn_codec_t` struct is read on the host during the call and may be discarded
 *     afterwards; the device buffers it points to must stay valid until the enqueued work
 *     has finished.
 *   - Host-detectable mistakes (NULL pointer, k > d, ld too small, negative sizes, unknown
 *     enum, workspace too small) return an error code before anything is launched.  A launch
 *     the CUDA runtime rejects returns SSN_ERR_CUDA.  n_tokens == 0 (or batch == 0) is a
 *     successful no-op.
 *   - Device-detectable mistakes never trap: a token whose id is outside [0, vocab) or whose
 *     position is outside [0, max_pos) takes a ZERO row for that term, and bit 0 (bad id) or
 *     bit 1 (bad position) is OR-ed into *dev_status when that pointer is not NULL.  The
 *     caller zeroes *dev_status beforehand.
 *   - A tensor-core kernel's internal waits (on its own copies and accumulators) are bounded;
 *     one that runs out ORs SSN_DEV_TIMEOUT into the status word and the kernel still ends.  The
 *     output of that call is invalid then.  The status word is the call's dev_status argument
 *     or, when that is NULL or the call has none, codec->dev_status.
 *   - Inputs and outputs of one call must not overlap, except ssn_weight_reproject, which
 *     works in place.
 *   - Threads and devices: the library keeps no state a call's result depends on.  Its caches
 *     (SM count, kernel attributes, the scratch address of the _static call) are per device,
 *     filled on first use with atomic updates, so calls may come from several host threads and
 *     for several devices (the current device of the calling thread is used, as for any
 *     runtime call).  The diagnostics ssn_launch_count and ssn_last_kernel are informational.
 *   - Stream order: a call's work is ordered after everything enqueued on its stream before it,
 *     as for any kernel launch.  The tensor-core kernels of two consecutive calls may overlap the
 *     SET-UP of the later one (its barriers and tensor memory, nothing in global memory) with the
 *     tail of the earlier one (programmatic dependent launch); what either reads or writes is as
 *     if the calls ran one after the other.
 *   - bf16 buffers whose pointers are 16-byte aligned and whose leading dimensions are
 *     multiples of 8 take the vectorised tensor-core kernels; anything else (fp32, odd
 *     leading dimensions, unaligned views) is still computed, by slower general kernels.
 */
#ifndef SSN_H_
#define SSN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SSN_VERSION 100

typedef enum {
  SSN_OK = 0,
  SSN_ERR_NULL = 1,        /* a required pointer is NULL                                   */
  SSN_ERR_SHAPE = 2,       /* a size, rank or leading dimension is impossible              */
  SSN_ERR_DTYPE = 3,       /* unknown element type / side / mode                           */
  SSN_ERR_WORKSPACE = 4,   /* workspace missing or smaller than the *_workspace_bytes size */
  SSN_ERR_CUDA = 5         /* the CUDA runtime refused a launch                            */
} ssn_status_t;

typedef enum { SSN_F32 = 0, SSN_BF16 = 1 } ssn_dtype_t;

/* Which side of W the subspace lives on (see ssn_weight_reproject). */
typedef enum { SSN_SIDE_LEFT = 0, SSN_SIDE_RIGHT = 1 } ssn_side_t;

/* What ssn_grad_project writes; the two may be OR-ed. */
typedef enum { SSN_GRAD_COEFF = 1, SSN_GRAD_FULL = 2 } ssn_grad_mode_t;

/* Bits of the device status word. */
#define SSN_DEV_BAD_ID 1
#define SSN_DEV_BAD_POS 2
#define SSN_DEV_TIMEOUT 4   /* an internal bounded wait ran out; the output is invalid */

/*
 * The data both ends of a stage boundary share (Sec. 4.1, the paragraph before Eq.
 * ssn_compress: the basis U_k, and the tables PE and T_fixed that sender and receiver both
 * hold).  Plain value struct; nothing is owned.
 */
/*
 * Performance note.  The tensor-core kernels need 16-byte aligned base addresses and leading
 * dimensions that are multiples of 8 elements (bf16) for U, X / G / Xhat, E, P and the weights,
 * and for Z where it is read (decompress).  A rank that is not a multiple of 8 (the paper's 8B
 * run uses ~51) is fine as long as U and Z are STORED with such a leading dimension (ldu = 56,
 * say; the padding columns are never read as data).  Anything else still gives the same results,
 * through the general kernels, two orders of magnitude slower.
 */
typedef struct ssn_codec {
  int32_t d;            /* model width, >= 1                                              */
  int32_t k;            /* subspace rank, 1 <= k <= d                                     */
  int32_t dtype;        /* ssn_dtype_t of every matrix                                    */
  int32_t max_pos;      /* rows of P (ignored when P is NULL)                             */
  const void *U;        /* device [d x k], required                                       */
  int64_t ldu;          /* >= k                                                           */
  const void *E;        /* device [vocab x d] or NULL: no token-embedding term            */
  int64_t lde;          /* >= d                                                           */
  int64_t vocab;        /* rows of E (ignored when E is NULL)                             */
  const void *P;        /* device [max_pos x d] or NULL: no positional term (RoPE models) */
  int64_t ldp;          /* >= d                                                           */
  /* Optional prepared tables (see ssn_prepare_tables), fp32, or NULL.  They are constants of
   * the codec, like U, T_fixed and PE themselves, and only ssn_compress reads them.           */
  const float *EU;      /* device [vocab x k] = E U, or NULL                              */
  int64_t ldeu;         /* >= k                                                           */
  const float *PU;      /* device [max_pos x k] = P U, or NULL                            */
  int64_t ldpu;         /* >= k                                                           */
  /* Optional device status word for the calls that take no dev_status argument (grad-project,
   * re-projection, the reparameterized ops) and for the others when theirs is NULL.          */
  int32_t *dev_status;  /* device int32 or NULL                                           */
} ssn_codec_t;

/*
 * Projects the codec's constant tables once: EU = E U [vocab x k] and PU = P U [max_pos x k],
 * in fp32 (products of the stored values, fp32 accumulation).  Sec. 4.1 makes PE and T_fixed
 * fixed and known to both ends, and U_k is fixed, so by linearity Eq. (ssn_compress) is
 *     Z[t,:] = X[t,:] U - EU[ids[t],:] - PU[pos(t),:]
 * and a codec whose EU / PU fields point at these tables lets ssn_compress read only X, ids
 * and 2k floats per token instead of the E and P rows.  Either output may be NULL (then that
 * table is not made; it must be NULL when the codec has no such term).  The tables must be
 * made again whenever U, E or P change.  The codec passed in is read for U, E, P only.
 */
ssn_status_t ssn_prepare_tables(const ssn_codec_t *codec, float *EU, int64_t ldeu, float *PU,
                                int64_t ldpu, void *stream);

/*
 * Sender side, Eq. (ssn_compress):  Z[t,:] = (X[t,:] - P[pos(t),:] - E[ids[t],:]) U.
 *   X     device [n_tokens x d], ldx >= d.
 *   ids   device int32[n_tokens]; required when codec->E is not NULL, ignored otherwise.
 *   pos   device int32[n_tokens] or NULL; NULL means pos(t) = t mod seq_len, the position of
 *         token t in a batch-major [batch x seq_len] flattening (seq_len >= 1 required then).
 *   Z     device [n_tokens x k] output, ldz >= k, rounded to the element type from fp32.
 *   dev_status  device int32 or NULL (see the common rules).
 */
ssn_status_t ssn_compress(const ssn_codec_t *codec, const void *X, int64_t ldx,
                          const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                          int32_t seq_len, void *Z, int64_t ldz, int32_t *dev_status,
                          void *stream);

/*
 * Receiver side of Eq. (ssn_compress) (Sec. 4.1: the receiving stage expands with U_k^T and
 * adds back the PE and T_fixed it also holds):  Xhat[t,:] = Z[t,:] U^T + E[ids[t],:] + P[pos(t),:].
 * With codec->E == NULL and codec->P == NULL this is the plain expansion Z U^T, which is also
 * how a receiving stage expands an incoming coefficient gradient.
 * Arguments as for ssn_compress with Z the input and Xhat [n_tokens x d] the output.
 */
ssn_status_t ssn_decompress(const ssn_codec_t *codec, const void *Z, int64_t ldz,
                            const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                            int32_t seq_len, void *Xhat, int64_t ldx, int32_t *dev_status,
                            void *stream);

/*
 * ssn_decompress fused with the row statistic of the receiving stage's first block.  Sec. 4.1
 * makes decompress the first operation of a receiving stage, and every block of the paper's
 * models opens with an RMSNorm (model table of the experimental setup), whose only reduction
 * over the row is
 *     rowsumsq[t] = sum_i Xhat[t,i]^2
 * so producing it here leaves the norm a pure scale of Xhat (no second pass over the row).
 *   rowsumsq  device fp32 [n_tokens], written (the call zeroes it on the stream first).  The
 *             squares are of the fp32 values BEFORE Xhat is rounded to the storage type; for
 *             bf16 storage they differ from the squares of the stored row by ~2^-9 / sqrt(d)
 *             relative.  Partial sums of a row are combined with atomic adds, so the last
 *             bits may differ from run to run.
 * Everything else as for ssn_decompress.  Performance note: the tensor-core expansion kernel
 * produces the statistic for bf16 codecs with d a multiple of 128, k <= 128, at least 512
 * tokens and, when the codec has P, implicit positions over whole sequences that tile into g
 * sequences x 128/g positions (g = 8, or 4, 2, 1 with k <= 64); other calls run the general kernel.
 */
ssn_status_t ssn_decompress_rowsumsq(const ssn_codec_t *codec, const void *Z, int64_t ldz,
                                     const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                                     int32_t seq_len, void *Xhat, int64_t ldx, float *rowsumsq,
                                     int32_t *dev_status, void *stream);

/*
 * Backward pass (Sec. 4.1, after Eq. ssn_compress: the activation gradient crosses the boundary
 * compressed the same way; chain rule (grad L) U_k):
 *   mode & SSN_GRAD_COEFF:  dZ   [n_tokens x k] = G U           -- what crosses the link
 *   mode & SSN_GRAD_FULL :  Gpar [n_tokens x d] = (G U) U^T     -- the projected gradient
 * The coordinates are kept in fp32 between the two products of the FULL form.  E and P of the
 * codec are not used.  dZ / Gpar may be NULL when their mode bit is clear.
 */
ssn_status_t ssn_grad_project(const ssn_codec_t *codec, const void *G, int64_t ldg,
                              int64_t n_tokens, int32_t mode, void *dZ, int64_t ldz,
                              void *Gpar, int64_t ldgp, void *stream);

/*
 * Original-SSN weight re-projection (Sec. 4.1: each constrained projection is put back into
 * the subspace after every optimizer step, outside the autograd graph; ablation Sec.
 * "Reparameterized SSN"), in place, for a batch of equally shaped weights:
 *   SSN_SIDE_RIGHT: W is [rows x cols] with cols == d, the layout of Eq. (residual_stream)
 *                   whose ROWS must lie in span(U):      W <- (W U) U^T
 *   SSN_SIDE_LEFT : W is [rows x cols] with rows == d (the transposed storage):
 *                                                        W <- U (U^T W)
 *   W_ptrs   HOST array of `batch` device pointers, each [rows x cols] with leading
 *            dimension ldw >= cols; the weights must be distinct buffers.
 *   workspace  device scratch of at least ssn_weight_reproject_workspace_bytes(...) bytes,
 *              16-byte aligned; may be NULL only when that size is 0.  Its contents are
 *              garbage afterwards; calls that share it must be ordered on one stream.
 * The k coordinates are kept in fp32 between the two products.
 */
size_t ssn_weight_reproject_workspace_bytes(const ssn_codec_t *codec, int64_t rows,
                                            int64_t cols, int32_t side, int32_t batch);

ssn_status_t ssn_weight_reproject(const ssn_codec_t *codec, void *const *W_ptrs, int32_t batch,
                                  int64_t rows, int64_t cols, int64_t ldw, int32_t side,
                                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * The re-projection of `count` weights that may differ in their free extent (all output
 * projections of a block after one optimizer step, Sec. 4.1), in place, with as few launches as
 * possible:
 *   SSN_SIDE_RIGHT: W_i is [extent[i] x d],  W_i <- (W_i U) U^T
 *   SSN_SIDE_LEFT : W_i is [d x extent[i]],  W_i <- U (U^T W_i)
 *   W_ptrs, extent, ldw   HOST arrays of `count` device pointers, extents (>= 1) and leading
 *                         dimensions (>= d for RIGHT, >= extent[i] for LEFT); distinct buffers.
 *   workspace   only read for SSN_SIDE_LEFT weights that the fused tensor-core kernel does not
 *               take (fp32, k > 128, d not a multiple of 128, leading dimension not a multiple of
 *               8 elements, unaligned base): k * max(extent) * 4 bytes, 16-byte aligned; such a
 *               weight without enough workspace gives SSN_ERR_WORKSPACE (weights before it in the
 *               list have been re-projected then).  May be NULL otherwise.
 * Same arithmetic as ssn_weight_reproject.
 */
ssn_status_t ssn_weight_reproject_list(const ssn_codec_t *codec, void *const *W_ptrs,
                                       const int64_t *extent, const int64_t *ldw, int32_t count,
                                       int32_t side, void *workspace, size_t workspace_bytes,
                                       void *stream);

/*
 * Reparameterized SSN (Eq. reparam): an output projection is stored as its low-dimensional
 * factor Zw [m x k], W_p = Zw U_k^T, whose rows lie in the subspace by construction, and the
 * block's output
 *     Y [n x d] = (H [n x m] Zw) U^T
 * is formed from the two skinny products without ever materialising W_p (H: the activations the
 * projection acts on, attention output or MLP inner activation, of width m).
 *   coords     optional [n x k] output of the coordinates H Zw (storage dtype, ldc >= k), or NULL
 * The coordinates stay in fp32 between the two products on every path.
 * H and Y must not overlap.  E and P of the codec are not used.
 * The activation gradient of the same layer, dH [n x m] = (dY U) Zw^T, is this call with the two
 * factors exchanged: a codec whose U is Zw (d = m) and Zw := U ([d x k], m := d), H := dY.
 */
ssn_status_t ssn_reparam_project(const ssn_codec_t *codec, const void *H, int64_t ldh, int64_t m,
                                 const void *Zw, int64_t ldzw, int64_t n_tokens, void *Y,
                                 int64_t ldy, void *coords, int64_t ldc, void *stream);

/*
 * Gradient of a reparameterized projection's factor (the chain rule stated with Eq. reparam:
 * the factor's gradient is the weight gradient times U_k): with Y = (H Zw) U^T and dY = dL/dY,
 *     dZw [m x k] = H^T (dY U)        (fp32 output, written, not accumulated)
 * n_tokens == 0 writes zeros (an empty sum).
 *   workspace  device scratch of n * kpad * sizeof(element) bytes, kpad = k rounded up to 8,
 *              16-byte aligned: the coordinates dY U (in the storage dtype).
 * E and P of the codec are not used.
 */
ssn_status_t ssn_reparam_grad_factor(const ssn_codec_t *codec, const void *H, int64_t ldh,
                                     int64_t m, const void *dY, int64_t lddy, int64_t n_tokens,
                                     float *dZw, int64_t lddz, void *workspace,
                                     size_t workspace_bytes, void *stream);

/*
 * Head-stage input of the reparameterized SSN (Sec. 4.1, after Eq. reparam: the trainable
 * embedding is factored through U_k as well, T_S = Elow U_k^T):
 *     X0[t,:] = E[ids[t],:] + Elow[ids[t],:] U^T + P[pos(t),:]
 * i.e. ssn_decompress applied to the gathered rows of Elow [vocab x k]; compressing X0 gives
 * those rows back exactly.
 *   workspace  device scratch of n * kpad * sizeof(element) bytes, kpad = k rounded up to 8,
 *              16-byte aligned: the gathered coordinates.
 * ids, pos, seq_len, dev_status as for ssn_decompress.  Each table is checked against its own
 * row count: an id outside [0, vocab_low) contributes no Elow row, an id outside
 * [0, codec->vocab) no E row, and either sets SSN_DEV_BAD_ID.  Elow rows are used whether or
 * not the codec has E.
 */
ssn_status_t ssn_head_embed(const ssn_codec_t *codec, const void *Elow, int64_t ldel,
                            int64_t vocab_low, const int32_t *ids, const int32_t *pos,
                            int64_t n_tokens, int32_t seq_len, void *X0, int64_t ldx,
                            void *workspace, size_t workspace_bytes, int32_t *dev_status,
                            void *stream);

/*
 * Wire rows.  The paper's bandwidth estimate (Sec. 3.5, "Stability Under Bandwidth
 * Constraints", the paragraph on the estimated communication) counts the boundary tensors in FP32, and the receiver of a forward activation needs the token ids for
 * T_fixed[ids]; these three calls produce and consume that form directly, whatever the storage
 * dtype of X:
 *     row t of `wire` = k fp32 coordinates, then (with_ids != 0) the token id as one int32 word
 * `wire` is a device buffer of 32-bit words with leading dimension ldw >= k + (with_ids ? 1 : 0)
 * words (any larger pitch leaves room for the caller's own header words; rows 16-byte aligned
 * with ldw % 4 == 0 get vector stores).  The coordinates are the fp32 accumulator values: for a
 * bf16 codec they are NOT rounded to bf16 on the way.
 *
 * ssn_compress_wire       as ssn_compress (prepared tables included); with_ids needs ids.
 * ssn_grad_project_wire   dZ = G U as fp32 rows (no ids).
 * ssn_decompress_wire     as ssn_decompress from wire rows; with_ids != 0: the ids are taken from
 *                         the rows and the `ids` argument is ignored.  A bf16 codec with
 *                         2 * kpad <= 128 (kpad = k rounded up to 8) runs on the tensor cores
 *                         with the fp32 coordinates split into a bf16 head and a bf16 remainder
 *                         (two products against the same basis, or rank 2 * kpad against the
 *                         basis repeated twice), which keeps about 16 of the 24 significand bits
 *                         of a coordinate, far below the single bf16 rounding of X^; for that the
 *                         call needs a 256-byte aligned workspace of
 *                         ssn_decompress_wire_workspace_bytes() bytes.  With a smaller (or
 *                         misaligned) workspace the general kernel runs; with_ids always needs
 *                         at least n_tokens * 4 bytes (rounded up to 256).
 * Errors as for the calls they mirror, plus SSN_ERR_WORKSPACE.
 */
ssn_status_t ssn_compress_wire(const ssn_codec_t *codec, const void *X, int64_t ldx,
                               const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                               int32_t seq_len, void *wire, int64_t ldw, int32_t with_ids,
                               int32_t *dev_status, void *stream);
ssn_status_t ssn_grad_project_wire(const ssn_codec_t *codec, const void *G, int64_t ldg,
                                   int64_t n_tokens, float *dZ, int64_t ldw, void *stream);
size_t ssn_decompress_wire_workspace_bytes(const ssn_codec_t *codec, int64_t n_tokens,
                                           int32_t with_ids);
ssn_status_t ssn_decompress_wire(const ssn_codec_t *codec, const void *wire, int64_t ldw,
                                 int32_t with_ids, const int32_t *ids, const int32_t *pos,
                                 int64_t n_tokens, int32_t seq_len, void *Xhat, int64_t ldx,
                                 void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                 void *stream);

/*
 * Compress fused with the stage's last residual add (Eq. residual_stream: the hidden state that
 * reaches the boundary is the residual stream plus the last block's output; Eq. ssn_compress):
 *     Z = (X + R - P[pos] - E[ids]) U
 * X and R are [n x d] in the storage dtype (leading dimensions ldx, ldr >= d); their sum is never
 * formed in memory nor rounded to the storage dtype.  out_form selects what is written:
 *   SSN_OUT_STORAGE   Z [n x k] in the storage dtype, ldout >= k elements   (as ssn_compress)
 *   SSN_OUT_WIRE      wire rows, ldout >= k words                          (as ssn_compress_wire)
 *   SSN_OUT_WIRE_IDS  wire rows with the id word, ldout >= k + 1 words
 * Everything else as for ssn_compress.  Performance note: the tensor-core kernel takes this call
 * for a codec without E and P or with the prepared tables (ssn_prepare_tables); a codec that has
 * to gather E or P rows runs the general kernel here.
 */
enum { SSN_OUT_STORAGE = 0, SSN_OUT_WIRE = 1, SSN_OUT_WIRE_IDS = 2 };
ssn_status_t ssn_compress_sum(const ssn_codec_t *codec, const void *X, int64_t ldx, const void *R,
                              int64_t ldr, const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                              int32_t seq_len, void *out, int64_t ldout, int32_t out_form,
                              int32_t *dev_status, void *stream);

/*
 * LEFT re-projection of ONE weight, W [d x cols] <- U (U^T W), without a caller workspace.
 * (The paper has no counterpart: this is a packaging variant of ssn_weight_reproject.)
 *
 * Who needs it: processes that gave all their device memory to an arena at start-up, or that
 * sit inside a latency-critical loop, cannot call cudaMalloc (it may fail, and it synchronises
 * the device) and may have no spare buffer to lend as workspace.  For them the k x cols fp32
 * coordinates U^T W are kept in a fixed SSN_STATIC_SCRATCH_BYTES array inside the library
 * (every GPU that loads the library holds it until the process exits).  The call allocates
 * nothing, frees nothing and calls no allocating library routine.
 *
 *   W     device [d x cols], leading dimension ldw >= cols, updated in place.
 *   Limit: k * cols * 4 bytes must not exceed ssn_static_scratch_bytes(); a larger problem is
 *          refused with SSN_ERR_WORKSPACE before anything is launched (use ssn_weight_reproject
 *          with your own workspace for those).
 *   First call on a device: looks up the device address of the scratch array (the device must
 *          be current, as for every call).  Make that first call outside any stream capture.
 *   Sharing: every call on a device uses the same array.  Its contents are rewritten completely
 *          by each call, so nothing has to be cleared, but two calls that overlap on the GPU
 *          (different streams, no ordering between them) race on it: order them.
 * Same arithmetic and results as the general (workspace) form of ssn_weight_reproject(...,
 * SSN_SIDE_LEFT, ...) on one weight; the fused tensor-core form of that call needs no scratch
 * at all and differs from this one only in rounding order.
 */
#define SSN_STATIC_SCRATCH_BYTES (4u << 20)
ssn_status_t ssn_weight_reproject_left_static(const ssn_codec_t *codec, void *W, int64_t cols,
                                              int64_t ldw, void *stream);

/* Size of the fixed scratch array used by ssn_weight_reproject_left_static. */
size_t ssn_static_scratch_bytes(void);

/* Static, never-NULL description of a status code. */
const char *ssn_status_string(ssn_status_t status);

/* SSN_VERSION the library was built from. */
int32_t ssn_version(void);

/*
 * Diagnostic: how many kernels this process has enqueued through the library so far (all
 * entry points, all streams).  No counterpart in the paper; the benchmark uses it to report
 * its launch count.
 */
int64_t ssn_launch_count(void);

/*
 * Diagnostic: which kernel the calling thread's most recent codec launch used, as
 * family | (variant bits << 8); SSN_KERNEL_NONE before the first launch.  No counterpart in
 * the paper; the tests use it to assert that a shape reaches the kernel it is meant to check.
 */
enum {
  SSN_KERNEL_NONE = 0,
  SSN_KERNEL_GENERIC = 1,          /* fp32 FMA kernels: any dtype, shape and alignment         */
  SSN_KERNEL_MMA_SYNC = 2,         /* mma.sync, whole rows per warp                            */
  SSN_KERNEL_MMA_SYNC_DSPLIT = 3,  /* mma.sync, few rows per SM: the warps of a CTA split d    */
  SSN_KERNEL_EXPAND64 = 4,         /* mma.sync expansion, 64-column chunks                     */
  SSN_KERNEL_UMMA_PROJECT = 5,     /* tcgen05 + TMA projection                                 */
  SSN_KERNEL_UMMA_EXPAND = 6,      /* tcgen05 + TMA expansion                                  */
  SSN_KERNEL_UMMA_ROUNDTRIP = 7,   /* tcgen05 + TMA project-then-expand                        */
  SSN_KERNEL_UMMA_TOKENS = 8       /* tcgen05 + TMA contraction over tokens                    */
};
#define SSN_KVAR_E 1      /* the kernel reads E rows                                            */
#define SSN_KVAR_P 2      /* the kernel reads P rows                                            */
#define SSN_KVAR_WIDE 4   /* rank above 64 (two 64-coordinate groups / the wide row tiles)      */
#define SSN_KVAR_ALT 8    /* MMA_SYNC: 32 rows per warp; EXPAND64: one P row per 16-sequence tile;
                             UMMA_PROJECT: positional product shared per block; UMMA_EXPAND:
                             tiles of 8 sequences x 16 positions; UMMA_ROUNDTRIP: LEFT          */
#define SSN_KVAR_ROWSUMSQ 16 /* UMMA_EXPAND / GENERIC: the row statistic is produced              */
#define SSN_KVAR_TWO_RUNS 64  /* UMMA_EXPAND: head and remainder of fp32 wire rows as two runs against one chunk of U */
#define SSN_KVAR_FEWSEQ 32   /* UMMA_EXPAND: tiles of 4, 2 or 1 sequences (a batch that is not groups of 8) */
int32_t ssn_last_kernel(void);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Launches one tiny kernel that
 * waits, with the same helper every tensor-core kernel uses, on a barrier nobody arrives on,
 * for at most max_polls polls (1 <= max_polls <= 1 << 20); the wait gives up, the kernel ORs
 * SSN_DEV_TIMEOUT into *dev_status (device int32, required) and ends normally.  Nothing hangs
 * and the context stays usable; the call exists so that this path can be exercised at all.
 */
ssn_status_t ssn_selftest_bounded_wait(int32_t max_polls, int32_t *dev_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SSN_H_ */
