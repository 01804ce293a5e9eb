/*
 * pd.h -- C ABI of the per-axis 1-bit weight-delta library for NVIDIA B200 (sm_100a).
 *
 * A fine-tuned linear layer W_f is represented as a shared fp16 base W_b plus a
 * bit-packed sign mask B = sign(W_f - W_b) and an fp16 scale vector v that lives on one
 * axis: one entry per output feature ("row" axis, d_out entries) or one per input
 * feature ("col" axis, d_in entries).  The reconstructed weight is
 *
 *        W_hat = W_b + v (.) B                      (paper, Method section, Eq. 1)
 *
 * Conventions shared by every call
 *   - All matrices are row-major.  Weights are [d_out, d_in] (the nn.Linear layout), so the
 *     input axis is the contiguous one.
 *   - mask is uint32 [d_out, d_in/32]: bit k of word w of row o belongs to column 32*w + k;
 *     bit 1 means B = +1 (dW >= 0), bit 0 means B = -1.  d_in must be a multiple of 32.
 *   - fp16 is IEEE binary16, passed as void*.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.
 *     The library never allocates or frees device memory and keeps no pointer after a call
 *     returns.  Scratch space comes from the caller through (workspace, workspace_bytes);
 *     pd_workspace_bytes() tells how much a call needs.  The workspace must be 256-byte aligned,
 *     and its first 256 bytes (the device status words) must be zero when it is first handed to
 *     the library: zero-fill it once after allocating it.  pd_device_status() re-zeroes them.
 *     pd_pack_delta needs ALL of its workspace zero on entry and leaves all of it zero on return
 *     (see there); the linear calls overwrite theirs beyond the status words, so give
 *     pd_pack_delta a workspace of its own or zero-fill it again after another call has used it.
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = the legacy default stream).  Every
 *     call only enqueues work on that stream and returns without synchronising.
 *   - Errors that can be seen on the host (NULL pointers, bad sizes, misalignment, a short
 *     workspace) are returned before anything is launched.  Errors only the device can see
 *     (a variant id out of range, a bounded wait that ran out) are latched in a device status
 *     word inside the workspace and read back by pd_device_status().
 *   - Input matrices, masks and scale vectors must be 16-byte aligned and ldx a multiple of 8
 *     elements; the output y only needs its natural 2-byte alignment and any ldy >= d_out.
 */
#ifndef PD_H_
#define PD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PD_OK = 0,
    PD_ERR_INVALID_ARG = 1,       /* NULL pointer, non-positive size, bad enum value */
    PD_ERR_UNSUPPORTED_SHAPE = 2, /* d_in not a multiple of 32, size beyond a stated maximum */
    PD_ERR_ALIGNMENT = 3,         /* input pointer not 16-byte aligned or ldx not a multiple of 8 */
    PD_ERR_WORKSPACE = 4,         /* workspace NULL, misaligned or smaller than pd_workspace_bytes() */
    PD_ERR_CUDA = 5,              /* a CUDA runtime / driver call failed (launch, attribute, tensor map) */
    PD_ERR_BAD_VARIANT = 6,       /* device saw a variant id outside [-1, V) */
    PD_ERR_DEVICE_TIMEOUT = 7     /* a bounded device-side wait expired */
} pd_status;

typedef enum {
    PD_AXIS_ROW = 0, /* v has d_out entries, W_hat[o,i] = W_b[o,i] + v[o] * B[o,i] */
    PD_AXIS_COL = 1, /* v has d_in  entries, W_hat[o,i] = W_b[o,i] + v[i] * B[o,i] */
    PD_AXIS_SCALAR = 2 /* pd_fit_* only: one scale for the whole matrix (the scalar baseline the paper compares with) */
} pd_axis;

typedef enum {
    PD_OP_PACK = 0,
    PD_OP_LINEAR = 1,
    PD_OP_LINEAR_MULTIVARIANT = 2,
    PD_OP_MERGE = 3,
    PD_OP_FIT = 4,       /* pd_fit_loss_grad: M = tokens of the batch */
    PD_OP_FIT_LAYER = 5  /* pd_fit_layer: M = max(batch, M_val) */
} pd_op;

/*
 * pd_pack_delta -- build the delta of one layer.
 * Paper: Method section (dW = W_f - W_b, B = sign(dW)); Implementation remarks ("1 bit along
 * input axis"); Algorithm "Per-layer compression with Row/Col selection", step 1 (pack) and
 * steps 3 and 5 (initial scales = mean |dW| along the other axis).
 *
 *   w_f, w_b : in,  fp16 [d_out, d_in]
 *   mask     : out, uint32 [d_out, d_in/32]; bit = (w_f >= w_b), i.e. sign(0) reads as +1
 *   v_row    : out, fp16 [d_out], v_row[o] = mean_i |dW[o,i]|; may be NULL
 *   v_col    : out, fp16 [d_in],  v_col[i] = mean_o |dW[o,i]|; may be NULL (not both NULL)
 *
 * The sums of |dW| are accumulated exactly (fixed point, units of 2^-24), divided once in fp64
 * and rounded once to fp16, so the result does not depend on launch shape or summation order.
 * Non-finite inputs are outside the contract.
 * Workspace: pd_workspace_bytes(PD_OP_PACK, ...) bytes that are ALL ZERO when the call is made (zero-fill once
 * after allocation); the sums are added into it and the call puts every byte back to zero before it completes,
 * so calls queued one after another on a stream can share it.  Calls that overlap on the GPU need workspaces of
 * their own.
 */
pd_status pd_pack_delta(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in,
                        uint32_t *mask, void *v_row, void *v_col,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * pd_linear -- y = x . W_hat^T without writing W_hat to memory.
 * Paper: Eq. 1 applied inside the forward pass (the "on-the-fly variant" of the Limitations
 * section, which the paper names but does not build).
 *
 *   x    : in,  fp16 [M, d_in], row stride ldx elements
 *   w_b  : in,  fp16 [d_out, d_in]
 *   mask : in,  uint32 [d_out, d_in/32]; NULL means "base only" (v is ignored)
 *   v    : in,  fp16, d_out entries (PD_AXIS_ROW) or d_in entries (PD_AXIS_COL)
 *   y    : out, fp16 [M, d_out], row stride ldy elements
 *
 * W_hat = W_b +- v is formed on chip in fp16 (one rounding per weight, as pd_merge stores it),
 * products are accumulated in fp32 and y is rounded to fp16 once at the end.  M <= 16 runs the
 * bandwidth-bound decode kernel, larger M the tensor-core (tcgen05) kernel, which needs d_out and
 * d_in to be multiples of 8 and d_in >= 64 (otherwise the rows go through the decode kernel in
 * chunks of 16).  Needs pd_workspace_bytes(PD_OP_LINEAR, M, 0, d_out, d_in) bytes: the status words and, when M is
 * small against the number of SMs (up to about a thousand tokens), fp32 partial sums of a k loop that is dealt to
 * several thread blocks and added in a fixed order by a second kernel (the result does not depend on the schedule).
 */
pd_status pd_linear(const void *x, int64_t M, int64_t ldx,
                    const void *w_b, const uint32_t *mask, const void *v, pd_axis axis,
                    int64_t d_out, int64_t d_in, void *y, int64_t ldy,
                    void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * pd_linear_ex -- pd_linear with flags (same operation, same paper passages).
 *
 *   PD_LINEAR_WEIGHTS_RESIDENT : the caller vouches that w_b, mask and v are not written by any work queued earlier
 *       on cuda_stream that may still be running (the serving case: weights loaded once, then many calls).  The
 *       decode kernel (M <= 16) is launched so that it can start while the previous kernel on the stream drains;
 *       with this flag it streams the weights at once and only x and y wait for that kernel.  Without the flag
 *       (pd_linear) every load waits, so pd_pack_delta -> pd_linear and pd_merge -> pd_linear(w_hat, mask = NULL)
 *       back to back on one stream are always correct.  The flag has no effect for M > 16.
 */
#define PD_LINEAR_WEIGHTS_RESIDENT 1u
pd_status pd_linear_ex(const void *x, int64_t M, int64_t ldx,
                       const void *w_b, const uint32_t *mask, const void *v, pd_axis axis,
                       int64_t d_out, int64_t d_in, void *y, int64_t ldy,
                       void *workspace, size_t workspace_bytes, void *cuda_stream, uint32_t flags);

/*
 * pd_linear_host -- pd_linear for activations that live in HOST memory (same operation and paper passages
 * as pd_linear).  Enqueues, on cuda_stream: copy of x_host -> x_dev, the fused linear, copy of y_dev -> y_host.
 *
 *   x_host : in,  HOST fp16 [M, d_in], dense (row stride d_in); pinned memory makes the copies asynchronous
 *   y_host : out, HOST fp16 [M, d_out], dense
 *   x_dev, y_dev : device staging buffers owned by the caller, at least M*d_in and M*d_out fp16, 16-byte aligned
 *   flags  : as in pd_linear_ex (0 or PD_LINEAR_WEIGHTS_RESIDENT)
 *   everything else as in pd_linear.  The results are in y_host once the stream has been synchronised.
 */
pd_status pd_linear_host(const void *x_host, void *x_dev, int64_t M, const void *w_b, const uint32_t *mask,
                         const void *v, pd_axis axis, int64_t d_out, int64_t d_in, void *y_dev, void *y_host,
                         void *workspace, size_t workspace_bytes, void *cuda_stream, uint32_t flags);

/*
 * pd_linear_multivariant -- one batch, many fine-tunes over one base.
 * Paper: Method section ("multiple fine-tuned models ... all share the same underlying base
 * weights"); the per-row routing is this library's reading of multi-tenant serving.
 *
 *   variant_ids : in, int32 [M] (device); row m uses variant ids[m]; -1 = base weights only.
 *                 Any other value outside [0, V) latches PD_ERR_BAD_VARIANT and leaves that
 *                 output row unspecified.
 *   masks       : in, uint32 [V, d_out, d_in/32]
 *   vs          : in, fp16 [V, v_stride]; variant g's scales start at vs + g*v_stride
 *   axes        : in, HOST array of V bytes, each a pd_axis
 *
 * Everything else as in pd_linear, except that a batch of at most 64 rows (d_in a multiple of 128) keeps the
 * products x.W_b and x.(+-v) apart in exact fp16 x fp16 products (W_hat is not rounded to fp16 first).  V <= 64.
 * Batches of at most 64 rows run as one pass over W_b: HBM traffic is W_b plus the masks of the variants present.
 * Needs pd_workspace_bytes(PD_OP_LINEAR_MULTIVARIANT, M, V, ...).
 */
pd_status pd_linear_multivariant(const void *x, int64_t M, int64_t ldx, const int32_t *variant_ids,
                                 const void *w_b, const uint32_t *masks, const void *vs,
                                 int64_t v_stride, const uint8_t *axes, int32_t V,
                                 int64_t d_out, int64_t d_in, void *y, int64_t ldy,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * pd_merge -- materialise W_hat as dense fp16 weights (cold start / hot swap).
 * Paper: Algorithm "Model-wide application from a saved delta file"; Limitations section
 * ("add all residual terms at once ... inference identical to FP16 weights").
 *
 *   w_hat : out, fp16 [d_out, d_in]; w_hat[o,i] = fp16( fp32(w_b[o,i]) + (+-)fp32(v) ), the sum
 *           rounded to fp32 and then to fp16, both to nearest even.  May alias w_b exactly.
 * Needs no workspace.
 */
pd_status pd_merge(const void *w_b, const uint32_t *mask, const void *v, pd_axis axis,
                   int64_t d_out, int64_t d_in, void *w_hat, void *cuda_stream);

/*
 * pd_load_merged -- cold start of a fine-tuned variant: apply a saved delta to a resident base, module by module.
 * Paper: Algorithm "Model-wide application from a saved delta file" (for every projection module take its mask and
 * scale vector and patch the layer); Implementation remarks (the packed deltas move "in a single operation per
 * module", non-blocking); the load-time paragraph of the experiments (applying the delta on a resident base against
 * loading a full checkpoint).
 *
 * Every module's artifact is ONE contiguous host buffer: d_out * d_in / 32 mask words, then the scale vector (d_out
 * or d_in binary16 values), pd_artifact_bytes() in all.  The call queues, for module i, one host-to-device copy of
 * that buffer into half (i mod 2) of `staging` on copy_stream and one pd_merge on compute_stream; the copy of module
 * i + 1 overlaps the merge of module i, and a staging half is not overwritten before the merge that reads it has
 * finished (events order the two streams).  Nothing is synchronised: when compute_stream has drained, every w_hat
 * holds bf16/fp16( fp32(w_b) +- fp32(v) ) exactly as pd_merge / pd_merge_bf16 would have written it.
 *
 *   modules      : HOST array of n descriptors (read during the call only)
 *   staging      : device, at least 2 * max_i pd_artifact_bytes(module i) rounded up to 256, 256-byte aligned
 *   copy_stream, compute_stream : two different streams for overlap (the same stream works, without overlap);
 *                  artifacts in pinned host memory make the copies asynchronous
 * Errors seen on the host (NULL, bad axis or dtype, d_in not a multiple of 32, short staging) return before anything
 * is queued.
 */
typedef struct {
    const void *w_b;      /* device: base weights [d_out, d_in] */
    void *w_hat;          /* device: merged weights [d_out, d_in]; may be w_b itself */
    const void *artifact; /* HOST: mask words, then scales */
    int64_t d_out, d_in;
    int32_t axis;         /* pd_axis */
    int32_t bf16;         /* 0: weights are binary16, 1: bfloat16 */
} pd_module;
size_t pd_artifact_bytes(int64_t d_out, int64_t d_in, pd_axis axis);
pd_status pd_load_merged(const pd_module *modules, int32_t n, void *staging, size_t staging_bytes,
                         void *copy_stream, void *compute_stream);

/*
 * BF16 variants -- the same four operations with the base, the fine-tuned weights, the activations and the outputs
 * in bfloat16 (the upper 16 bits of an IEEE binary32, passed as void*); masks, ids and the binary16 scale vectors
 * are unchanged.
 * Paper: Implementation remarks -- the base weights are "kept as (in,out) BF16", the calibration inputs and outputs
 * are stored as BF16 tensors and the scale vectors in FP16.
 *
 *   pd_pack_delta_bf16 : bit = (w_f >= w_b), an exact comparison.  The scales are means of floor(|dW| * 2^24)
 *       units of 2^-24 -- bfloat16 differences are not multiples of one small unit, so |dW| is cut down to that grid
 *       before it is summed; the sum is an integer and does not depend on order (for binary16 inputs the grid holds
 *       |dW| exactly, which is what pd_pack_delta sums).  One fp64 division, one rounding to binary16.  Exact while
 *       |w| <= 2^28 and a sum of |dW| stays below 2^29.
 *   pd_merge_bf16      : w_hat = bf16( fp32(w_b) + (+-)fp32(v) ): one binary32 addition, one rounding to bfloat16.
 *   pd_linear_bf16     : as pd_linear_ex.  W_hat = W_b +- v is formed on chip in bfloat16: v is rounded to bfloat16
 *       once, then one bfloat16 addition; bfloat16 products accumulate in fp32 and y is rounded to bfloat16 once.
 *   pd_linear_multivariant_bf16 : as pd_linear_multivariant.
 * Arguments, alignment rules, workspaces and error behaviour are those of the binary16 calls.
 */
pd_status pd_pack_delta_bf16(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in,
                             uint32_t *mask, void *v_row, void *v_col,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);
pd_status pd_merge_bf16(const void *w_b, const uint32_t *mask, const void *v, pd_axis axis,
                        int64_t d_out, int64_t d_in, void *w_hat, void *cuda_stream);
pd_status pd_linear_bf16(const void *x, int64_t M, int64_t ldx,
                         const void *w_b, const uint32_t *mask, const void *v, pd_axis axis,
                         int64_t d_out, int64_t d_in, void *y, int64_t ldy,
                         void *workspace, size_t workspace_bytes, void *cuda_stream, uint32_t flags);
pd_status pd_linear_multivariant_bf16(const void *x, int64_t M, int64_t ldx, const int32_t *variant_ids,
                                      const void *w_b, const uint32_t *masks, const void *vs,
                                      int64_t v_stride, const uint8_t *axes, int32_t V,
                                      int64_t d_out, int64_t d_in, void *y, int64_t ldy,
                                      void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * pd_pack_delta_static -- pd_pack_delta without a workspace argument and without any allocation.
 * The paper has no counterpart: this entry point exists for the library's users, not the method.
 *
 * Some callers have no way to obtain scratch memory at the point where they pack a layer: code
 * that runs inside a memory pool whose budget is already fixed, a plug-in that is handed tensors
 * by a host framework but must not call the CUDA allocator (cudaMalloc synchronises the device
 * and is forbidden while a stream is being captured), or a C program that links no allocator
 * wrapper at all.  For them the exact per-row and per-column sums of |dW| are kept in a fixed
 * 512 KiB array that is part of the library's device image (one copy on every GPU that loads the
 * library, held until the process exits).
 *
 *   arguments : as pd_pack_delta, minus (workspace, workspace_bytes); results are bit-identical.
 *   limit     : d_out + d_in <= 65536, else PD_ERR_UNSUPPORTED_SHAPE (nothing is launched).
 *   set-up    : the first call on each device looks up the array's device address (the device
 *               must be current, as for every call).  Make that first call outside any stream
 *               capture.
 *   sharing   : all calls on one GPU use the same array.  It starts zero-filled and each call puts
 *               what it used back to zero, so back-to-back calls on ONE stream are safe; calls that
 *               may overlap on the GPU (different streams, different threads) race on it and give
 *               wrong scales -- serialise them or use pd_pack_delta with separate workspaces.
 *   It calls no cudaMalloc / cudaFree and no allocating library routine.
 */
pd_status pd_pack_delta_static(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in,
                               uint32_t *mask, void *v_row, void *v_col, void *cuda_stream);

/* Bytes of workspace the given call needs (0 for PD_OP_MERGE).  M and V are ignored where they
 * do not apply.  Returns 0 for an unknown op. */
size_t pd_workspace_bytes(int op, int64_t M, int32_t V, int64_t d_out, int64_t d_in);

/* Synchronises the stream, reads the status word that the last pd_linear* call on this
 * workspace latched, clears it and returns it (PD_OK when nothing was latched). */
pd_status pd_device_status(void *workspace, void *cuda_stream);

/*
 * pd_selftest_bounded_wait -- exercises the device-side failure path without a fault.
 * Every wait inside the kernels (on a TMA copy, on another warp, on the other CTA of a pair) is bounded: when it
 * runs out the kernel latches PD_ERR_DEVICE_TIMEOUT in the workspace status words and returns.  This call launches
 * one warp that waits, with that same routine and a limit of limit_cycles SM clocks (1 .. 1e8), on a barrier that
 * nothing arrives on; afterwards pd_device_status(workspace) returns PD_ERR_DEVICE_TIMEOUT once, then PD_OK.
 * The GPU context stays usable.  workspace: at least 256 bytes, 256-byte aligned, zero-filled.
 */
pd_status pd_selftest_bounded_wait(void *workspace, int64_t limit_cycles, void *cuda_stream);

/*
 * ---- Fitting the scales by output matching ----
 * Paper: section "Calibration cache, training, and stacking" (per layer, only v is trained, on cached pairs (X, Y) of
 * the layer's inputs and the fine-tuned layer's outputs, with L = (1/n) ||Y - Y_hat||_2^2 and AdamW); Algorithm "Train
 * per-row/column scaling vectors via activation matching"; Algorithm "Per-layer compression with Row/Col selection"
 * (both axes are trained from the packed scales with the same budget, the lower validation loss wins, row on a tie).
 * n = M * d_out (the mean over all output entries).  W_b, x, y are fp16; v, gradients and optimiser state are fp32
 * device arrays; every product runs on the tensor cores with fp32 accumulation, W_b and the sign matrix as separate
 * operands.  Sizes: d_in a multiple of 32, d_out a multiple of 8, M >= 1; x [M, d_in] and y [M, d_out] contiguous,
 * x, y and w_b 16-byte aligned.  All calls enqueue on the stream and return; errors the device latches (a bounded wait
 * that ran out) are read with pd_device_status(workspace).
 */

/* mask_t [d_in, ceil(d_out/32)] words: bit (o % 32) of mask_t[i][o / 32] = bit (i % 32) of mask[o][i / 32]; rows past
 * d_out read as 0.  Needed by the col-axis gradient (a contraction over the output rows); computed once per layer. */
pd_status pd_transpose_mask(const uint32_t *mask, int64_t d_out, int64_t d_in, uint32_t *mask_t, void *cuda_stream);

/*
 * pd_fit_loss_grad -- loss of one batch and its gradient with respect to v.
 *   v      : in, fp32, d_out (ROW), d_in (COL) or 1 (SCALAR) entries
 *   mask_t : in, from pd_transpose_mask; only read for PD_AXIS_COL with grad != NULL (may be NULL otherwise)
 *   loss   : out, one fp32 (may be NULL);   grad : out, fp32, as many entries as v (NULL: loss only)
 *   workspace: pd_workspace_bytes(PD_OP_FIT, M, 0, d_out, d_in), 256-byte aligned, status words zero on first use
 * Partial sums are added in a fixed order: the same inputs give the same bits on every call.
 */
pd_status pd_fit_loss_grad(const void *x, const void *y, int64_t M, const void *w_b, const uint32_t *mask,
                           const uint32_t *mask_t, const float *v, pd_axis axis, int64_t d_out, int64_t d_in, float *loss,
                           float *grad, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* AdamW constants (decoupled weight decay; the paper fixes the optimiser and the learning rate, 1e-4, only). */
typedef struct pd_adamw {
    float lr, beta1, beta2, eps, weight_decay;
} pd_adamw;

/* One AdamW step, t = 1, 2, ...:  v *= 1 - lr * wd;  m1 = b1 m1 + (1 - b1) g;  m2 = b2 m2 + (1 - b2) g^2;
 * v -= lr * (m1 / (1 - b1^t)) / (sqrt(m2 / (1 - b2^t)) + eps).  v, m1, m2, grad: fp32 device arrays of len entries. */
pd_status pd_fit_adamw_step(float *v, float *m1, float *m2, const float *grad, int64_t len, int64_t t, const pd_adamw *opt,
                            void *cuda_stream);

/*
 * pd_fit_layer -- the whole per-layer fit with Row/Col selection.
 *   x_tr [M_tr, d_in], y_tr [M_tr, d_out] : training cache, walked in minibatches of `batch` tokens (the last one may
 *                                           be shorter), `epochs` times; batch * d_in must keep x 16-byte aligned
 *   x_val, y_val [M_val, ...]             : held-out cache; the axis with the lower validation loss is kept
 *   v_row0 [d_out], v_col0 [d_in]         : fp16 starting scales (pd_pack_delta's v_row and v_col)
 *   cosine != 0                           : learning rate lr * (1 + cos(pi k / T)) / 2 at step k = 0 .. T-1, T = all steps
 *   v_out    : out, fp16, max(d_out, d_in) entries: the chosen axis' trained scales in its first entries
 *   axis_out : out, device int32: PD_AXIS_ROW or PD_AXIS_COL
 *   val_loss : out, device fp32 [2]: validation loss of the row variant, of the col variant
 *   workspace: pd_workspace_bytes(PD_OP_FIT_LAYER, max(batch, M_val), 0, d_out, d_in)
 */
pd_status pd_fit_layer(const void *x_tr, const void *y_tr, int64_t M_tr, const void *x_val, const void *y_val, int64_t M_val,
                       const void *w_b, const uint32_t *mask, const void *v_row0, const void *v_col0, int64_t d_out,
                       int64_t d_in, int32_t epochs, int64_t batch, const pd_adamw *opt, int32_t cosine, void *v_out,
                       int32_t *axis_out, float *val_loss, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Human-readable name of a status code; never NULL. */
const char *pd_status_string(pd_status status);

/* Number of kernels the library has launched in this process since load (for accounting). */
int64_t pd_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PD_H_ */
