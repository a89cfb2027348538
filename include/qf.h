/* qf — fake-quantization hot path for quantization-aware training on NVIDIA B200 (sm_100a).
 *
 * C ABI of libqf.so. Plain C types only. Unless a parameter says otherwise, EVERY data pointer
 * is a DEVICE pointer owned by the caller; the library never allocates or frees device memory,
 * keeps no state between calls beyond per-device caches of constants (device capability, kernel
 * attributes, the address of one built-in buffer), and enqueues all of its work on the CUDA stream passed as
 * `stream` (a cudaStream_t cast to void*, NULL = the legacy default stream). Calls return as soon
 * as the work is enqueued. Scratch memory comes from the caller through `workspace` /
 * `workspace_bytes`; qf_workspace_bytes() says how much a call needs.
 *
 * Error behaviour: arguments are checked on the host before anything is launched and a non-zero
 * qf_status_t is returned with nothing enqueued. A failed launch maps to QF_ERR_CUDA. Device-side
 * waits are bounded; one that expires records QF_ERR_TIMEOUT in the first 4 bytes of the
 * workspace (readable with qf_read_status() after the stream has been synchronised) and the
 * kernel returns. Inputs must be finite; NaN / Inf give unspecified, non-faulting results.
 *
 * Notation follows the paper (Section 3.2): a quantizer Q maps a BF16 tensor X to low-bit codes C
 * and metadata theta (scales, offsets); Q^-1 maps (C, theta) back to a BF16 tensor X_hat whose
 * values lie on the format's grid (Eq. quantize-dequantize). Tensors are row-major; for a linear
 * layer X is [M,K], W is [N,K], Y is [M,N] = X_hat . W_hat^T. Quantization blocks run along the
 * last (contiguous) dimension.
 */
#ifndef QF_H_
#define QF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Quantization formats (Table "formats"): NVFP4 = E2M1 codes, blocks of 16, E4M3 block scale,
 * FP32 tensor scale; MXFP4 = E2M1 codes, blocks of 32, E8M0 power-of-two block scale; Q4_K =
 * unsigned 4-bit codes, 256-weight super-blocks of 8 sub-blocks, 6-bit sub-block scale and offset
 * under FP16 super-block factors (weight-only). NONE leaves an operand unquantized. */
typedef enum { QF_FMT_NONE = 0, QF_FMT_NVFP4 = 1, QF_FMT_MXFP4 = 2, QF_FMT_Q4_K = 3 } qf_format_t;

typedef enum {
  QF_OK = 0,
  QF_ERR_NULL = 1,      /* a required pointer is NULL */
  QF_ERR_SHAPE = 2,     /* negative size, or a dimension that is not a multiple of what the format / kernel needs */
  QF_ERR_ALIGN = 3,     /* a pointer is not 16-byte aligned */
  QF_ERR_FORMAT = 4,    /* unknown format, or a format not allowed for this operand (Q4_K activations) */
  QF_ERR_WORKSPACE = 5, /* workspace missing or smaller than qf_workspace_bytes() */
  QF_ERR_CUDA = 6,      /* a CUDA runtime or driver call failed */
  QF_ERR_TIMEOUT = 7,   /* a bounded device-side wait expired (reported through the workspace status word) */
  QF_ERR_ARCH = 8,      /* the current device is not compute capability 10.x */
  QF_ERR_DTYPE = 9,     /* unknown output dtype */
  QF_ERR_TOO_LARGE = 10 /* the problem needs more scratch than the built-in buffer of qf_fq_linear_fwd_noalloc */
} qf_status_t;

typedef enum { QF_DT_BF16 = 0, QF_DT_F32 = 1 } qf_dtype_t;

typedef enum {
  QF_OP_QDQ = 0,
  QF_OP_LINEAR_FWD = 1,
  QF_OP_LINEAR_BWD = 2,
  QF_OP_GROUPED_FWD = 3,
  QF_OP_GROUPED_BWD = 4,
  QF_OP_QDQ_BATCHED = 5
} qf_op_t;

/* flags */
#define QF_TENSOR_SCALE_GIVEN 0x1u /* qf_qdq: read *tensor_scale instead of deriving it             */
#define QF_W_TSCALE_GIVEN 0x1u     /* linear calls: *w_tscale is an input (tied / shared scale)      */
#define QF_A_TSCALE_GIVEN 0x2u     /* linear calls: *a_tscale is an input (running activation scale) */
#define QF_ACCUMULATE_DW 0x4u      /* backward: dW += ... instead of dW = ... (gradient accumulation) */
#define QF_REUSE_W_HAT 0x20u       /* linear calls: the workspace still holds the fake-quantized W written by an earlier call */
#define QF_REUSE_X_HAT 0x40u       /* with the same tensor, formats and shapes (e.g. the forward of this step): skip its
                                      recomputation. The paper's layer discards these copies after the forward matmul and
                                      recomputes them; keeping the workspace alive trades that memory for two passes. */
#define QF_AMAX_RUNNING 0x10u      /* qf_nvfp4_tensor_scale: the incoming *amax_state takes part in the maximum        */
#define QF_FUSED_QDQ 0x8u          /* linear calls: quantize-dequantize MXFP4 and NVFP4 operands inside the matmul kernel,
                                      on the tiles staged in shared memory, instead of writing fake-quantized copies to
                                      the workspace first (Eq. fakequant: W_hat and A_hat are transient). Same results
                                      bit for bit. An NVFP4 operand's tensor scale is settled before the launch (supplied,
                                      or derived by a maximum pass over the operand; a speculated scale is derived).
                                      Applies to plain and grouped calls with at least 256 output rows (and at most 256
                                      experts); Q4_K weights (a super-block spans four staged tiles) and anything else
                                      silently take the default path. Slower than the default on B200 at every shape
                                      measured: an option, not the default. */

#define QF_MXFP4_NO_CLIP 0x80u      /* qf_qdq, qf_qdq_lora and the linear calls: MXFP4 block exponent p = the smallest one
                                      with amax <= 6 * 2^p (nothing saturates) instead of floor(log2 amax) - 2, under
                                      which block maxima in (6, 8) * 2^p clamp to 6 * 2^p. The paper leaves the rule
                                      open (Eq. mxfp4 only requires a power-of-two scale); the default follows the
                                      shared-exponent convention of the MX formats. Blocks whose maximum exceeds
                                      3.5 * 2^126 overflow to infinity under this rule. Other formats ignore the flag. */

#define QF_TENSOR_SCALE_SPECULATIVE 0x200u /* qf_qdq, NVFP4, scale not given: *tensor_scale holds a GUESS on entry (for        */
#define QF_W_TSCALE_SPECULATIVE 0x200u    /* a weight in training: the scale of the previous step). The call quantizes with  */
                                          /* the guess while it accumulates the true maximum, then derives the scale, stores */
                                          /* it in *tensor_scale and requantizes unless it equals the guess bit for bit.     */
                                          /* Results are always those of deriving the scale (Section 3.2.3: the tensor scale */
                                          /* comes from the current maximum); a right guess saves the separate pass that     */
                                          /* reads the tensor for its maximum, a wrong one costs a wasted quantize pass.     */
                                          /* Linear calls: the same for *w_tscale (single weight tensors, not grouped).      */

const char* qf_status_string(qf_status_t s);
int qf_version(void);

/* Bytes of caller-provided scratch a call needs (always a multiple of 256, never 0).
 * op = QF_OP_QDQ: M = rows, K = cols, N ignored. Linear ops: M, N, K as in the call; for grouped ops
 * M = rows_padded and `groups` = number of experts. QF_OP_QDQ_BATCHED: `groups` = number of tensors, M, N, K ignored. */
size_t qf_workspace_bytes(qf_op_t op, int64_t M, int64_t N, int64_t K, int groups);

/* Reads the 4-byte status word at the start of a workspace (synchronises `stream` first).
 * host_status_out is a HOST pointer. */
qf_status_t qf_read_status(const void* workspace, void* stream, int* host_status_out);

/* Quantizer interface, both halves in one pass: (C, theta) = Q(in), out = Q^-1(C, theta)
 * (Eq. quantize-dequantize; formats Eq. nvfp4 / Eq. mxfp4 / Eq. q4k; dequantization Eq. nvfp4-dequant /
 * Eq. mxfp4-dequant / Eq. q4k-dequant).
 *   in           BF16 [rows, cols], cols a multiple of the block (16 / 32 / 256).
 *   out_bf16     BF16 [rows, cols]                                   (nullable: skip the dequantized copy)
 *   codes        rows*cols/2 bytes, two 4-bit codes per byte          (nullable)
 *                FP4 formats: element 2j in the low nibble of byte j, element 2j+1 in the high nibble.
 *                Q4_K: 128 bytes per super-block; in each 64-element chunk, byte l holds element l in
 *                the low nibble and element l+32 in the high nibble.
 *   scales       NVFP4: u8 E4M3 [rows, cols/16]; MXFP4: u8 E8M0 [rows, cols/32];
 *                Q4_K: 16 bytes per super-block {fp16 d, fp16 dmin, 12 bytes of packed 6-bit
 *                (scale, offset) pairs}, [rows, cols/256]              (nullable)
 *   tensor_scale NVFP4 only, device float*: read if flags & QF_TENSOR_SCALE_GIVEN, otherwise
 *                written with amax(in)/(6*448) (1.0 for an all-zero tensor). Required for NVFP4.
 * At least one of out_bf16 / codes / scales must be non-NULL. rows*cols == 0 is a no-op.
 * out_bf16 may be the same pointer as in (quantize-dequantize in place); no other overlap between the
 * buffers is allowed. */
qf_status_t qf_qdq(qf_format_t fmt, const void* in, int64_t rows, int64_t cols, void* out_bf16,
                   void* codes, void* scales, float* tensor_scale, uint32_t flags, void* workspace,
                   size_t workspace_bytes, void* stream);

/* qf_qdq for many tensors in one call. A quantization-aware training step quantizes every linear weight of the
 * model (and ships the low-precision payload to the rollout engine, Section 3.4 "Low-precision weight
 * synchronization"); most of those tensors are small enough that a call per tensor is launch-latency bound, and
 * NVFP4 (Eq. nvfp4) needs each tensor's maximum before any of its blocks can be scaled. Results are exactly those
 * of calling qf_qdq on every tensor by itself.
 *   n            number of tensors (n = 0 is a no-op)
 *   in, rows, cols   HOST arrays of n device pointers (BF16 [rows[i], cols[i]]) and their shapes
 *   out_bf16, codes, scales   HOST arrays of n device pointers, layouts as in qf_qdq. Each array may be NULL as a
 *                whole (that output is skipped for every tensor) and entry by entry; every non-empty tensor needs
 *                at least one output. out_bf16[i] may equal in[i].
 *   tensor_scales   NVFP4 only: DEVICE float[n], one tensor scale per tensor: written (derived from each tensor's
 *                maximum), read with QF_TENSOR_SCALE_GIVEN, or guesses on entry and derived values on return with
 *                QF_TENSOR_SCALE_SPECULATIVE (see that flag; a tensor quantized in place is derived directly).
 *   workspace    qf_workspace_bytes(QF_OP_QDQ_BATCHED, 0, 0, 0, n) bytes (needed for NVFP4 without given scales)
 * The host arrays are read during the call only. Errors as for qf_qdq, checked for every tensor before anything
 * is enqueued. */
qf_status_t qf_qdq_batched(qf_format_t fmt, int n, const void* const* in, const int64_t* rows, const int64_t* cols,
                           void* const* out_bf16, void* const* codes, void* const* scales, float* tensor_scales,
                           uint32_t flags, void* workspace, size_t workspace_bytes, void* stream);

/* LoRA-QAD weight path (Eq. qad-lora, Eq. export-lora): quantize-dequantize the MERGED weight
 *     W_hat = Q^-1(Q(W + lora_scale * B A)),
 * with W [rows, cols] BF16 (the frozen base), B [rows, rank] BF16 and A [rank, cols] BF16. The merge is
 * done on the fly inside the quantizer kernels (and inside the amax pre-pass for NVFP4): the merged
 * tensor is never written to memory, which is what lets a mixture-of-experts layer merge and quantize
 * one expert after another without holding merged weights. Arithmetic of the merge, fixed so that results
 * are reproducible: per element acc = W in FP32, then acc = fma(lora_scale * B[n,r], A[r,k], acc) for
 * r = 0 .. rank-1 in that order (each step rounded once), then one rounding to BF16; the quantizer then
 * sees that BF16 value. rank = 0 is qf_qdq. Other arguments as qf_qdq. A must be 16-byte aligned.
 * To run the layer on the result, pass out_bf16 to the linear calls with wq_fmt = QF_FMT_NONE. */
qf_status_t qf_qdq_lora(qf_format_t fmt, const void* W, const void* B, const void* A, int rank, float lora_scale,
                        int64_t rows, int64_t cols, void* out_bf16, void* codes, void* scales, float* tensor_scale,
                        uint32_t flags, void* workspace, size_t workspace_bytes, void* stream);

/* Q^-1 alone (Eq. nvfp4-dequant / Eq. mxfp4-dequant / Eq. q4k-dequant): codes + scales (+ tensor scale)
 * -> BF16 [rows, cols]. Layouts as in qf_qdq. */
qf_status_t qf_dequant(qf_format_t fmt, const void* codes, const void* scales, const float* tensor_scale,
                       int64_t rows, int64_t cols, void* out_bf16, void* stream);

/* Tensor-wide max |x| of a BF16 tensor of n elements, written as FP32 to *amax_out (the statistic
 * the NVFP4 tensor scale and the trainer's running activation maximum are derived from). */
qf_status_t qf_amax(const void* in, int64_t n, float* amax_out, void* stream);

/* NVFP4 tensor scales that span more than one tensor or more than one step ("Engine-specific scale
 * sharing"; the NVFP4 paragraph on the running activation maximum): fused projections (query/key/value,
 * gate/up) share one weight tensor scale computed over their concatenation and one activation scale, and
 * the activation scale exported with the checkpoint is derived from a running absolute maximum.
 *   tensors / sizes  HOST arrays of n device pointers to BF16 tensors and their element counts.
 *   amax_state       device float*, in/out: receives max |x| over all listed tensors; with QF_AMAX_RUNNING
 *                    its previous value takes part in the maximum (running maximum across calls; it must
 *                    then hold a non-negative finite value, e.g. 0 before the first step).
 *   scale_out        device float*, nullable: receives amax_state/(6*448), or 1.0 when the maximum is 0 -
 *                    the value to hand to qf_qdq / the linear calls as a given tensor scale. */
qf_status_t qf_nvfp4_tensor_scale(const void* const* tensors, const int64_t* sizes, int n, float* amax_state, float* scale_out,
                                  uint32_t flags, void* stream);

/* Quantization-aware linear layer, forward (Eq. fakequant):
 *     Y[M,N] = Q_a^-1(Q_a(X[M,K])) . Q_w^-1(Q_w(W[N,K]))^T,   BF16 operands, FP32 accumulation.
 *   wq_fmt in {NONE, NVFP4, MXFP4, Q4_K}; aq_fmt in {NONE, NVFP4, MXFP4}.
 *   Y is BF16 or FP32 per y_dtype. K must be a multiple of the larger block in use (and of 8);
 *   N a multiple of 8.
 *   w_tscale / a_tscale: NVFP4 tensor scales (device float*), given or derived per flags
 *   (derived values are written back); ignored for other formats and may then be NULL.
 *   a_amax_out (nullable): receives amax(X), for the trainer's running activation maximum (taken from the
 *              pass that quantizes X where there is one, so it costs no extra read of X then). */
qf_status_t qf_fq_linear_fwd(const void* X, const void* W, void* Y, qf_dtype_t y_dtype, int64_t M, int64_t N,
                             int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale,
                             float* a_tscale, float* a_amax_out, uint32_t flags, void* workspace,
                             size_t workspace_bytes, void* stream);

/* Straight-through backward (Eq. ste, Eq. activation-ste); both quantizers act as the identity:
 *     dX[M,K] = dY[M,N] . W_hat[N,K]            (nullable: skip)
 *     dW[N,K] = dY[M,N]^T . X_hat[M,K]          (nullable: skip)
 * W_hat and X_hat are recomputed from W and X exactly as in the forward. dY is never quantized.
 * M may be any size (the contraction of dW needs no padding). */
qf_status_t qf_fq_linear_bwd(const void* dY, const void* X, const void* W, void* dX, qf_dtype_t dx_dtype,
                             void* dW, qf_dtype_t dw_dtype, int64_t M, int64_t N, int64_t K,
                             qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale, float* a_tscale,
                             uint32_t flags, void* workspace, size_t workspace_bytes, void* stream);

/* Per-expert variant for mixture-of-experts layers (every expert's latent weights are trained with
 * the same quantization-aware layer). Rows of X are sorted by expert; group_offsets is a device
 * int32[G+1] of segment starts, each a multiple of 128 (the caller pads segments with zero rows;
 * a zero row quantizes to a zero row in every format); rows_padded = group_offsets[G]. The table is device
 * memory, so the host cannot check it: the kernels force every entry to a multiple of 128 in [0, rows_padded],
 * and a table that breaks the contract gives meaningless but finite results, never an out-of-range access.
 * W is [G,N,K], Y is [rows_padded,N]:  Y[r,:] = X_hat[r,:] . W_hat[g(r)]^T.
 * NVFP4 weights: every expert is its own tensor with its own tensor scale, so w_tscale is an array of G
 * floats (required; read if QF_W_TSCALE_GIVEN, otherwise written). An NVFP4 activation scale is a
 * single float for the whole of X (the experts share one input-activation scale). */
qf_status_t qf_fq_grouped_linear_fwd(const void* X, const void* W, void* Y, qf_dtype_t y_dtype,
                                     const int32_t* group_offsets, int G, int64_t rows_padded, int64_t N,
                                     int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale,
                                     float* a_tscale, uint32_t flags, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* dX[r,:] = dY[r,:] . W_hat[g(r)]  (nullable);  dW[g] = dY[seg g]^T . X_hat[seg g], dW is [G,N,K] (nullable). */
qf_status_t qf_fq_grouped_linear_bwd(const void* dY, const void* X, const void* W, void* dX,
                                     qf_dtype_t dx_dtype, void* dW, qf_dtype_t dw_dtype,
                                     const int32_t* group_offsets, int G, int64_t rows_padded, int64_t N,
                                     int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale,
                                     float* a_tscale, uint32_t flags, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* Engine-native packing of quantized weights (Section 3.4 "Low-precision weight synchronization",
 * Section 3.5 "Packing the checkpoint"): a lossless re-layout of what qf_qdq emitted.
 *   QF_LAYOUT_GGUF_Q4_K (fmt = QF_FMT_Q4_K): `packed` receives rows*cols/256 llama.cpp block_q4_K records
 *     of 144 bytes {fp16 d, fp16 dmin, 12 bytes of 6-bit scales/offsets, 128 bytes of codes}, row-major.
 *   QF_LAYOUT_FP4_SWIZZLED_SCALES (fmt = NVFP4 or MXFP4): `packed` receives the block scales in the tiled
 *     layout block-scaled FP4 tensor-core GEMMs read: scales padded with zeros to multiples of 128 rows and
 *     4 scale columns, stored tile by tile (tiles row-major, 512 bytes each), byte (r, c) of a tile at
 *     (r mod 32)*16 + (r div 32)*4 + c. `codes` is ignored: the 4-bit codes are already in the engines'
 *     layout (two per byte, even element in the low nibble, row-major).
 * qf_pack_bytes gives the size of `packed`. qf_unpack is the inverse (for Q4_K it fills both codes and
 * scales; for the FP4 layout only scales). All pointers device, 16-byte aligned. */
typedef enum { QF_LAYOUT_GGUF_Q4_K = 1, QF_LAYOUT_FP4_SWIZZLED_SCALES = 2 } qf_layout_t;
size_t qf_pack_bytes(qf_layout_t layout, qf_format_t fmt, int64_t rows, int64_t cols);
qf_status_t qf_pack(qf_layout_t layout, qf_format_t fmt, const void* codes, const void* scales, int64_t rows, int64_t cols,
                    void* packed, void* stream);
qf_status_t qf_unpack(qf_layout_t layout, qf_format_t fmt, const void* packed, int64_t rows, int64_t cols, void* codes,
                      void* scales, void* stream);

/* The deployment-side product the fake-quantized layer stands for (Section 3.1, goal "Faithfulness to
 * deployment"; Section 3.2: NVFP4 and MXFP4 are W4A4 formats at inference): Y = deq(A) . deq(B)^T computed by
 * the block-scaled FP4 tensor-core instruction directly on the 4-bit codes and block scales that qf_qdq
 * emitted for A [M,K] and B [N,K], FP32 accumulation, FP32 result. For MXFP4 this sums exactly the products
 * the BF16 matmul of the training path sums (Eq. mxfp4-dequant is exact in BF16), so the two may differ only
 * by FP32 summation order; for NVFP4 the training path additionally rounds each dequantized value to BF16
 * (Eq. nvfp4-dequant), the native product does not, and the tensor scales multiply the accumulated sum.
 * It is a checking tool for that equivalence (one CTA per 128x128 tile, not pipelined), not a serving kernel.
 *   fmt          QF_FMT_MXFP4 or QF_FMT_NVFP4 (both operands)
 *   a_codes      device, [M, K/2] bytes;  a_scales device, [M, K/32] E8M0 or [M, K/16] E4M3 bytes (row-major,
 *                as qf_qdq writes them);  likewise b_codes / b_scales with N rows. Codes 16-byte aligned.
 *   a_tscale, b_tscale  NVFP4: device float*, the tensor scales; ignored for MXFP4
 *   Y            device float [M, N], 16-byte aligned
 *   flags        QF_SCALES_TILED: a_scales and b_scales are in the tiled engine layout that qf_pack writes for
 *                QF_LAYOUT_FP4_SWIZZLED_SCALES (16-byte aligned) instead of row-major: the 512-byte tiles are
 *                handed to the tensor cores as they are, which is the hardware's own check of that layout
 *   K % 32 == 0. workspace: at least qf_workspace_bytes(QF_OP_QDQ, ...) bytes; its status word reports an
 *   expired device-side wait (qf_read_status). Errors as for the other calls. */
#define QF_SCALES_TILED 0x100u
qf_status_t qf_fp4_matmul_native(qf_format_t fmt, const void* a_codes, const void* a_scales, const float* a_tscale,
                                 const void* b_codes, const void* b_scales, const float* b_tscale, int64_t M, int64_t N,
                                 int64_t K, float* Y, uint32_t flags, void* workspace, size_t workspace_bytes, void* stream);

/* Allocation-free forward of the quantization-aware linear layer. (The paper has no counterpart:
 * this is a packaging variant of qf_fq_linear_fwd for hosts that cannot hand the library a workspace.)
 *
 * Who needs it: code that runs where nobody may allocate device memory and where no spare buffer
 * was planned for us — for example an extension loaded into a serving or training process whose
 * memory planner reserved the whole device up front and forbids cudaMalloc (and the framework's own
 * allocator) from extension code, or a hot loop that must never enter an allocator because a device
 * allocation can synchronise the GPU. Such a caller still owns X, W and Y; what it lacks is a place
 * for the two transient fake-quantized copies. Here that place is a buffer compiled into the
 * library: QF_NOALLOC_SCRATCH_BYTES (32 MiB) of device memory per GPU, held by every GPU that loads
 * libqf.so until the process exits.
 *
 * Same arithmetic, arguments and results as qf_fq_linear_fwd (no a_amax_out, no workspace;
 * QF_REUSE_W_HAT / QF_REUSE_X_HAT are ignored, since the buffer is shared by every caller). The call
 * itself allocates nothing: no cudaMalloc / cudaFree / allocating library routine on any path. The
 * buffer is part of the library's device image; with CUDA's default lazy module loading the driver
 * places that image on a device the first time something from the library runs there, so the
 * 32 MiB are taken at that moment (for this entry point: at its first call on the device), not at
 * dlopen. A host that is about to reserve all remaining device memory should make one call first
 * (M = 0 is enough), or it will get QF_ERR_CUDA from the first real call.
 *   Limit: 256 + round256(2*N*K) + round256(2*M*K) bytes must fit in QF_NOALLOC_SCRATCH_BYTES; larger
 *          problems are rejected with QF_ERR_TOO_LARGE before anything is enqueued.
 *   First call on each device: looks up the device address of the built-in buffer (once per device,
 *          with that device current; this is also what makes the driver load the image, see above).
 *          Make that first call outside any stream capture.
 *   Sharing: every call on a device uses the same buffer, which keeps the previous call's contents;
 *          the call clears the words that must start at zero itself. Two calls whose GPU work can
 *          overlap (different streams, no dependency between them) race on the buffer — serialise
 *          them. A device-side timeout is not reported by this variant (there is no caller-visible
 *          status word); use qf_fq_linear_fwd when that matters. */
#define QF_NOALLOC_SCRATCH_BYTES (32u << 20)
qf_status_t qf_fq_linear_fwd_noalloc(const void* X, const void* W, void* Y, qf_dtype_t y_dtype, int64_t M, int64_t N,
                                     int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale,
                                     float* a_tscale, uint32_t flags, void* stream);

/* Self-test hook for the hardware number-format conversions the kernels rely on: for each of n FP32
 * inputs (device), writes the E2M1 code (low nibble) into e2m1_out[i] and the E4M3 code of |x|
 * into e4m3_out[i] (device u8 arrays, either nullable). Used by the tests to compare the
 * conversion instructions exhaustively with the oracle's encoders. */
qf_status_t qf_selftest_cvt(const float* in, int64_t n, uint8_t* e2m1_out, uint8_t* e4m3_out, void* stream);

/* Self-test hook for the exact reciprocal-based division the NVFP4 and Q4_K kernels use in place of
 * the per-element IEEE divide: for every pair (xs[i], ys[j]) with ys[j] in [2^-60, 2^60] (device FP32
 * arrays) the quotient is compared bit for bit with the IEEE quotient; *mismatches (device u64)
 * receives the number of differences. */
qf_status_t qf_selftest_div(const float* xs, int64_t nx, const float* ys, int64_t ny, uint64_t* mismatches, void* stream);

/* Self-test hook for the bounded device-side waits: launches one thread that waits, with the given limit
 * in SM clock cycles (at most 2^28), on a barrier nothing ever arrives at. The wait gives up, the kernel
 * returns normally, and the workspace then holds QF_ERR_TIMEOUT in its status word (qf_read_status)
 * and 1 in its 32-bit word 16. Nothing faults or hangs; the context stays usable. */
qf_status_t qf_selftest_timeout(void* workspace, size_t workspace_bytes, int64_t limit_cycles, void* stream);

/* Self-test hook for the conversion-free MXFP4 rounding used inside the fused matmul kernel (packed BF16
 * add/subtract of a magic constant): every BF16 bit pattern against every block-scale code in [8, 240]
 * is compared with the conversion-instruction route; *mismatches (device u64) receives the count. */
qf_status_t qf_selftest_mxfp4_bf16(uint64_t* mismatches, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QF_H_ */
