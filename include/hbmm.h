/*
 * hbmm.h -- C ABI of the B200 (sm_100a) Hadamard Binary Matrix Multiply library.
 *
 * The library implements the inference path of HadaNets ("HadaNets: Flexible
 * Quantization Strategies for Neural Networks"): a tensor X (rows x K, row-major)
 * is represented as the Hadamard product  X~ = delta (.) Sign(X)  of a
 * full-precision tensor delta (the mean absolute value of every run of beta
 * consecutive row elements; Section 3, Eq. 1-4) and a binary tensor that is
 * bit-packed along the row (Section 4).  The product of two such operands is
 * formed from one signed +-1 dot product per K-group (XNOR/popcount) and two
 * full-precision multiplies per group (Section 4.2, Eq. 7).
 *
 * General conventions
 *   - Every data pointer is DEVICE memory owned by the caller unless a comment
 *     says "host".  Operand descriptors and geometry structs are host memory and
 *     are read before the call returns.  The library never allocates, frees or
 *     keeps a pointer, except where an entry point says otherwise.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     All work is enqueued on it; no call synchronises the host.
 *   - Every call returns an hbmm_status.  Argument errors are detected on the
 *     host before anything is launched; a failed launch returns HBMM_ERR_CUDA.
 *   - Matrices are row-major.  A is M x K (rows = samples / output pixels), W is
 *     N x K (rows = filters; the paper's W^f = Reshape(W, (filters, -1))), and
 *     C = A~ * W~^T is M x N in fp32.
 */
#ifndef HBMM_H_
#define HBMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  HBMM_OK = 0,
  HBMM_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, leading dimension too small, K mismatch */
  HBMM_ERR_UNSUPPORTED = 2, /* a beta / dtype / path combination this build does not implement        */
  HBMM_ERR_ALIGNMENT = 3,   /* a pointer or leading dimension violates the stated alignment           */
  HBMM_ERR_WORKSPACE = 4,   /* workspace missing or smaller than the *_workspace_bytes query          */
  HBMM_ERR_CUDA = 5,        /* the CUDA runtime reported an error at launch                            */
  HBMM_ERR_TIMEOUT = 6      /* a bounded device-side wait expired (kernels never spin unbounded)       */
} hbmm_status;

typedef enum { HBMM_F32 = 0, HBMM_BF16 = 1 } hbmm_dtype;

/* Which contraction kernel hbmm_gemm_ex runs.  First meaning: two packed operands (HBMM); second:
 * dense activations x packed weights (HBWN, beta_a == 1). */
typedef enum {
  HBMM_PATH_AUTO = 0,   /* the fastest path that supports the operands (and has its workspace)         */
  HBMM_PATH_POPC = 1,   /* XOR + __popc on the integer pipe, fp32 group-scale epilogue in registers;
                           HBWN: weight sign XOR-ed into fp32 activations on the fp32 pipe              */
  HBMM_PATH_B1MMA = 2,  /* legacy warp-level mma.sync: b1 xor.popc, beta multiple of 128;
                           HBWN: bf16 mma.sync with per-group partial sums (bf16 activations only)      */
  HBMM_PATH_TENSOR = 3, /* tcgen05 with TMEM accumulators: sign bits expanded to +-1 e4m3, group dots
                           scaled in the epilogue; HBWN: bf16 activations x weights written as three
                           bf16 pieces +-d_i (delta = d1 + d2 + d3), one accumulation over all of K     */
  HBMM_PATH_TENSOR_PREPARED = 4, /* HBMM_PATH_TENSOR, and the caller states that the workspace still holds
                           the expanded weight operand an earlier HBMM_PATH_TENSOR / AUTO call with the
                           same W, the same kind of A and this workspace left there (W unchanged
                           since, that call completed without a device-side error): the expansion
                           kernel is skipped.  Results are undefined otherwise.                       */
  HBMM_PATH_FOLDED = 5, /* tcgen05, both operands packed: every group scale, times a power of two chosen
                           per row, is split into two fp16 pieces (22 significant bits) and folded into
                           the +-1 elements, so that Eq. 7's sum over groups is one fp32 accumulation of
                           exact fp16 x fp16 products with no per-group step; the powers of two are
                           divided out once per output.  Scales more than 2^17 below their row's
                           largest lose relative accuracy (absolute error at most 2^-39 of that
                           largest scale).  The K products are summed one by one in fp32, so
                           the error follows sum_k |A~[m,k]| |W~[n,k]| (a few 2^-24 of it) instead of
                           vanishing where group dots cancel.  What HBMM_PATH_AUTO picks when it has
                           the workspace and the finer grouping has at most 128 elements per group.
                           Callers that need Eq. 7's exact cancellation inside a group (integer
                           group dots, error relative to sum_g |dA dW D_g| alone) pass
                           HBMM_PATH_TENSOR.
                           HBWN: bf16 activations x weights written as TWO bf16 pieces (the group
                           scale to 2^-17 instead of 2^-26; activations carry 2^-9), 128-column
                           tiles; what HBMM_PATH_AUTO picks for dense bf16 activations.              */
  HBMM_PATH_FOLDED_PREPARED = 6 /* HBMM_PATH_FOLDED with the expanded weights of an earlier
                           HBMM_PATH_FOLDED / AUTO call reused, as HBMM_PATH_TENSOR_PREPARED (the
                           arrival counters of the shared tiles, which every completed call leaves at
                           zero, are part of what is reused)                                           */
} hbmm_path;

/*
 * One Hadamard-binary operand (Section 3, Fig. 1): rows x K, scale groups of beta
 * consecutive elements along K.
 *   beta >= 2 : packed form.  `bits` and `scales` are used, `dense` is ignored.
 *       bits   : uint32 [rows, ld_words]; element k of a row is bit (k % 32), least significant
 *                first, of word (k / 32); bit 1 <=> Sign = +1 (x >= 0), bit 0 <=> -1 (the paper's
 *                packing example, Section 4).  Bits at positions >= K and words >= ceil(K/32)
 *                are zero.  ld_words is a multiple of 4 (16-byte rows); 16-byte aligned.
 *       scales : [rows, ld_scales] of scale_dtype; entry g is the mean |x| over columns
 *                [g*beta, min((g+1)*beta, K)) (a tail group is averaged over its own length);
 *                entries g >= ceil(K/beta) are zero.  ld_scales is a multiple of 4 (fp32) or 8
 *                (bf16); 16-byte aligned.  bf16 scales are the fp32 scale rounded to nearest even.
 *       Supported beta: multiples of 32; the sub-word powers of two 2, 4, 8 and 16 (the settings of
 *       the paper's experiments, Section 5; a word then holds 32 / beta groups); and any beta >= K
 *       (one group per row, the XNOR-Net case of Section 5).  Anything else returns
 *       HBMM_ERR_UNSUPPORTED.
 *   beta == 1 : the tensor stays at full precision (X~ = X; the paper's first/last layers and the
 *       HBWN mode).  `dense` [rows, ld_dense] of dense_dtype is used, bits/scales are ignored.
 */
typedef struct {
  int64_t rows;
  int64_t K;
  int32_t beta;
  int32_t scale_dtype; /* hbmm_dtype */
  uint32_t *bits;
  int64_t ld_words;
  void *scales;
  int64_t ld_scales;
  const void *dense;
  int64_t ld_dense;
  int32_t dense_dtype; /* hbmm_dtype */
  int32_t reserved;
} hbmm_operand;

/* Convolution geometry: NCHW input [B, C, H, W], kh x kw filters. */
typedef struct {
  int32_t B, C, H, W;
  int32_t kh, kw;
  int32_t stride_h, stride_w;
  int32_t pad_h, pad_w;
} hbmm_conv_geom;

/*
 * Storage of a packed operand (Fig. 1; Section 3.2 and 4.1: a binarized tensor costs about
 * 1 + X/beta bits per element, X the scale width, i.e. beta*X/(beta+X) times less than full
 * precision).  Pure host arithmetic, no CUDA call.  Outputs (host pointers, any may be NULL):
 * bytes of the bit tensor, bytes of the scale tensor, and the two leading dimensions to put in
 * the descriptor.  Errors: INVALID_ARG (rows, K <= 0, beta < 2, bad dtype).
 */
hbmm_status hbmm_operand_bytes(int64_t rows, int64_t K, int32_t beta, int32_t scale_dtype,
                               size_t *bits_bytes, size_t *scales_bytes,
                               int64_t *ld_words, int64_t *ld_scales);

/*
 * Hadamard binarization and bit-packing of a row-major tensor (Section 3, Eq. 1-4; packing
 * Section 4).  x: device, [rows, ldx] of x_dtype, ldx >= K.  out: host descriptor whose rows, K,
 * beta, scale_dtype, bits, ld_words, scales, ld_scales are set by the caller (buffers sized by
 * hbmm_operand_bytes); the call fills bits and scales, including their zero padding.
 * Sign(0) = Sign(-0) = +1.  NaN inputs are outside the contract.
 * Errors: INVALID_ARG, UNSUPPORTED (beta), ALIGNMENT (bits/scales not 16-byte aligned or
 * ld_words / ld_scales not as hbmm_operand_bytes returns), CUDA.
 */
hbmm_status hbmm_quantize(const void *x, int32_t x_dtype, int64_t rows, int64_t K, int64_t ldx,
                          const hbmm_operand *out, void *stream);

/*
 * Training side: gradient through the Hadamard binarization X~ = delta (.) Sign(X) (Section 3.1.3).
 * Given gy = dC/dX~ it returns gx = dC/dX by Eq. 6, with the straight-through estimator of Eq. 5 for the
 * derivative of Sign:
 *     gx[r,i] = (1/n_g) Sign(x_i) sum_{j in group(i)} gy[r,j] Sign(x_j)  +  delta_g gy[r,i] [|x_i| <= 1],
 * group(i) the run of beta consecutive row elements that holds i (a tail group uses its own length n_g),
 * delta_g its mean |x|, Sign(0) = +1.  beta >= 1 (any value; beta >= K: one group per row; beta = 1: X~ = X).
 * x, gy, gx: device fp32 [rows, ld*], ld* >= K, 4-byte aligned (16-byte aligned unpadded rows take the
 * streaming kernel).  gx may not alias x or gy.  The re-binarization of the weights that every training
 * step needs (Algorithm 1) is hbmm_quantize.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
hbmm_status hbmm_binarize_backward(const float *x, int64_t ldx, const float *gy, int64_t ldg,
                                   int64_t rows, int64_t K, int32_t beta, float *gx, int64_t ldo,
                                   void *stream);

/*
 * The binarized tensor itself, dense: out[r,k] = delta_g Sign(x[r,k]) (Eq. 2; Eq. 3-4), g the run of beta
 * consecutive row elements that holds k (a tail run uses its own length), delta_g its mean |x| in fp32,
 * Sign(0) = +1.  beta >= 1 (any value; beta >= K: one group per row; beta = 1: out = x).
 * Called on an NCHW activation map viewed as [batch*channels*height, width] with beta = beta_a <= width it is
 * Eq. 3 as printed -- groups of beta_a neighbours along a row of the map, before the convolution -- and
 * hbmm_conv_im2col with beta_a = 1 on its output is the convolution of Eq. 3's A~ with W~.  (hbmm_conv_im2col
 * with beta_a >= 2 groups along K of the im2col row instead, the form Eq. 7 is stated for.)
 * x: device fp32 [rows, ldx], ldx >= K, 4-byte aligned.  out: device [rows, ldo] of out_dtype (HBMM_F32 or
 * HBMM_BF16, round to nearest even), ldo >= K, aligned to its element; may not alias x.  16-byte aligned
 * unpadded rows with a power-of-two beta <= 128 dividing K take the streaming kernel.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
hbmm_status hbmm_binarize_dense(const float *x, int64_t ldx, int64_t rows, int64_t K, int32_t beta,
                                void *out, int32_t out_dtype, int64_t ldo, void *stream);

/* Bytes of scratch hbmm_gemm wants for these operands (host pointer `bytes`).  The tensor-core
 * contractions keep the weight operand there, expanded once per call into the tile layout their
 * kernels stream (HBMM: 4 K bytes per weight row, two fp16 pieces; HBWN: 6 K bytes per weight row,
 * three bf16 pieces); 0 when no path needs scratch.  For products of few output tiles (fewer than about
 * a thousand tiles of 128 x 128 or 128 x 64 outputs) the packed x packed figure also holds the slots in
 * which CTAs that share a tile's K range exchange partial sums (up to 32 MB).  hbmm_gemm still works
 * without a workspace (NULL or too small): it then runs the integer-pipe path (HBMM) or the warp-level
 * kernels (HBWN).  The workspace must be 16-byte aligned. */
hbmm_status hbmm_gemm_workspace_bytes(const hbmm_operand *A, const hbmm_operand *W, size_t *bytes);

/*
 * C[m,n] = sum_k A~[m,k] * W~[n,k]  (Eq. 7 regrouped: per K-segment one signed +-1 dot product
 * D = n_valid - 2*popcount(xor) and the product of the two segment scales).
 *   A: M x K, packed (beta_a >= 2) or dense bf16/fp32 (beta_a == 1: the HBWN mode, full-precision
 *      activations times Hadamard-binary weights).   W: N x K, packed.  A.K == W.K.
 *   When beta_a != beta_w the larger must be a multiple of the smaller; the work is done on the
 *   finer segmentation (Section 4.2).
 *   C: device fp32 [M, ldc], ldc >= N, 16-byte aligned with ldc % 4 == 0.  Fully overwritten
 *   in columns < N.  workspace may be NULL when the query returns 0.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE, CUDA.
 */
hbmm_status hbmm_gemm(const hbmm_operand *A, const hbmm_operand *W, float *C, int64_t ldc,
                      void *workspace, size_t workspace_bytes, void *stream);

/* Same as hbmm_gemm with the contraction kernel chosen by the caller (hbmm_path); a path that
 * cannot run these operands returns HBMM_ERR_UNSUPPORTED, HBMM_PATH_TENSOR without its workspace
 * HBMM_ERR_WORKSPACE.  For measurement and tests. */
hbmm_status hbmm_gemm_ex(const hbmm_operand *A, const hbmm_operand *W, float *C, int64_t ldc,
                         void *workspace, size_t workspace_bytes, int32_t path, void *stream);

/*
 * Product fused with the next layer's binarization (the layer order of Section 5 is batch normalisation ->
 * binarize -> product, so the consumer of C is a binarizer): inside the contraction's epilogue every output
 * goes through a per-column affine map  z[m,n] = bn_scale[n] * C[m,n] + bn_shift[n]  (a batch normalisation
 * folded to inference form; either pointer may be NULL: 1 and 0) and each row of z is Hadamard-binarized along
 * n with group next->beta (Eq. 3-4).  Only the packed result is written: the fp32 product never reaches
 * memory (4 bytes per output become 1 + 32/beta bits).  `next`: host descriptor of a packed operand with
 * rows = A.rows, K = W.rows, buffers sized by hbmm_operand_bytes; filled like hbmm_quantize fills its output,
 * zero padding included.  It is what a following fully connected layer or 1 x 1 convolution reads as its A.
 * Runs on the folded-scale tensor-core kernel only: A and W packed with K a multiple of 32 and activation
 * groups of whole words; next->beta one of 2, 4, 8, 16, 32, 64, 128, at most 64 when W has at most 64 rows,
 * and smaller than W.rows; workspace as hbmm_gemm_workspace_bytes(A, W) reports.  bn_scale / bn_shift:
 * device fp32 [W.rows].  Where z is within rounding of zero the sign follows the fp32 value the kernel
 * computed.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE, CUDA.
 * (hbmm_gemm_fused with HBMM_OUT_PACKED, no activation, both operands packed.)
 */
hbmm_status hbmm_gemm_binarize_next(const hbmm_operand *A, const hbmm_operand *W, const float *bn_scale,
                                    const float *bn_shift, const hbmm_operand *next, void *workspace,
                                    size_t workspace_bytes, void *stream);

/*
 * What may happen to a product before it leaves the contraction kernel -- the rest of the paper's layer (Section 5:
 * batch normalisation -> binarization -> convolution -> activation -> pooling, then the next block's batch
 * normalisation and binarization), applied in the epilogue while the outputs are in registers:
 *     y = activation(C)                    HBMM_ACT_NONE, or HBMM_ACT_RELU: max(0, C)
 *     z[m,n] = bn_scale[n] * y + bn_shift[n]   the NEXT block's batch normalisation folded to inference form
 *                                              (device fp32 [N]; either pointer may be NULL: 1 and 0)
 * and then one of
 *   HBMM_OUT_DENSE : z stored as out[m * ld_out + n], out_dtype HBMM_F32 or HBMM_BF16 (round to nearest even),
 *                    ld_out >= N, out aligned to its element (16-byte aligned rows take vector stores).  For a
 *                    convolution the rows are output pixels, so this is the NHWC activation tensor of the next
 *                    layer: a dense-activation (beta_a = 1) convolution reads it directly when it is given
 *                    HBMM_CONV_INPUT_NHWC, with no layout copy and no fp32 round trip.
 *   HBMM_OUT_PACKED: every row of z is Hadamard-binarized along n with group next->beta (Eq. 3-4) and only the
 *                    packed result is written (4 bytes per output become 1 + 32/beta bits).  `next`: host
 *                    descriptor of a packed operand with rows = M, K = N, buffers sized by hbmm_operand_bytes;
 *                    filled like hbmm_quantize fills its output, zero padding included.  It is what a following
 *                    fully connected layer or 1 x 1 convolution reads as its A.  next->beta one of 2, 4, 8, 16, 32,
 *                    64, 128, at most 64 when the product has at most 64 columns, and smaller than N.  Where z
 *                    is within rounding of zero the sign follows the fp32 value the kernel computed.
 * Pooling is not part of the chain.  The fp32 product itself is never stored.
 */
typedef enum { HBMM_ACT_NONE = 0, HBMM_ACT_RELU = 1 } hbmm_activation;
typedef enum { HBMM_OUT_DENSE = 1, HBMM_OUT_PACKED = 2 } hbmm_out_kind;
typedef struct {
  int32_t activation;        /* hbmm_activation */
  int32_t out_kind;          /* hbmm_out_kind */
  const float *bn_scale;     /* device fp32 [N] or NULL */
  const float *bn_shift;     /* device fp32 [N] or NULL */
  void *out;                 /* HBMM_OUT_DENSE: device [M, ld_out] */
  int64_t ld_out;
  int32_t out_dtype;         /* hbmm_dtype */
  int32_t reserved;
  const hbmm_operand *next;  /* HBMM_OUT_PACKED: host descriptor, device buffers */
} hbmm_epilogue;

/*
 * hbmm_gemm with the epilogue chain above instead of the fp32 store.  A packed (scale groups of whole K-words,
 * or one group per row; K a multiple of 32): the folded-scale tensor-core kernel; A dense bf16 with rows on
 * 16-byte boundaries (beta_a = 1): the tensor-core HBWN kernel.  workspace as hbmm_gemm_workspace_bytes(A, W)
 * reports (required).  ep: host struct, read before the call returns.
 * Errors: INVALID_ARG, UNSUPPORTED (operands outside the above, next->beta), ALIGNMENT, WORKSPACE, CUDA.
 */
hbmm_status hbmm_gemm_fused(const hbmm_operand *A, const hbmm_operand *W, const hbmm_epilogue *ep, void *workspace,
                            size_t workspace_bytes, void *stream);

/*
 * The integer term of Eq. 7 on its own: D[m,n,t] = signed +-1 dot product of K-segment t
 * (segment length min(beta_a, beta_w); T = ceil(K / segment) segments), int32, device
 * [M, N, T] contiguous.  Both operands packed.  Meant for checking the popcount path
 * bit-exactly; not tuned.  Errors as hbmm_gemm.
 */
hbmm_status hbmm_gemm_partials(const hbmm_operand *A, const hbmm_operand *W, int32_t *D,
                               int32_t path, void *stream);

/* Scratch for hbmm_conv_im2col: the packed (or, for beta_a == 1, bf16 dense) im2col operand
 * followed by the contraction's own workspace.  bytes: host pointer. */
hbmm_status hbmm_conv_workspace_bytes(const hbmm_conv_geom *g, int32_t beta_a, int32_t a_scale_dtype,
                                      const hbmm_operand *W, size_t *bytes);

/*
 * Convolution as HBMM.  Row m = (b, yo, xo) of the implicit activation matrix gathers
 * A[m,k] = x[b, c, yo*stride_h + i - pad_h, xo*stride_w + j - pad_w] (0 outside the image) with
 * k = (c, i, j), c slowest -- the column order of W^f = Reshape(W, (filters, -1)) (Algorithm 1,
 * Section 3.1.1).  beta_a >= 2: every such row is Hadamard-binarized along k (the grouping Eq. 7
 * is stated for), packed into the workspace, and multiplied by W as in hbmm_gemm.  beta_a == 1:
 * HBWN, rows are gathered as bf16.  x: device NCHW of x_dtype.  W: packed, N x (C*kh*kw).
 * C_out: device fp32 [B*Ho*Wo, ldc] (the NHWC output), alignment as in hbmm_gemm.
 * workspace: device, 256-byte aligned, at least hbmm_conv_workspace_bytes.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE, CUDA.
 */
hbmm_status hbmm_conv_im2col(const void *x, int32_t x_dtype, const hbmm_conv_geom *g,
                             int32_t beta_a, int32_t a_scale_dtype, const hbmm_operand *W,
                             float *C_out, int64_t ldc, void *workspace, size_t workspace_bytes,
                             void *stream);

/*
 * hbmm_conv_im2col with flags.  HBMM_CONV_WEIGHTS_PREPARED: the caller states that the part of `workspace`
 * that holds the expanded weight operand (the tile layout the tensor-core contraction streams; Section 4.2:
 * weights are fixed at inference time) was filled by an earlier hbmm_conv_im2col / hbmm_conv_im2col_ex
 * call with the same W, geometry, beta_a, scale type and workspace, and that nothing has written it since.
 * The call then skips the expansion; the activation part of the workspace is rewritten by every call
 * either way.  Results are undefined when the statement is false.  Paths that keep no expanded weights
 * ignore the flag.
 * HBMM_CONV_PACK_ONLY (beta_a >= 2 only, otherwise HBMM_ERR_INVALID_ARG): the call stops once the packed
 * activation operand -- bits [M, ld_words] at the start of the workspace, then, from the next 256-byte
 * boundary, scales [M, ld_scales], both as hbmm_operand_bytes(M, C*kh*kw, beta_a, a_scale_dtype) lays
 * them out -- has been written (gather + Hadamard binarization + packing, Eq. 3-4 on the im2col row);
 * no product is formed and C_out / ldc are ignored (C_out may be NULL).  For callers that multiply one
 * packed activation operand by several weight tensors through hbmm_gemm, and for timing the front end on
 * its own.  On the paths that expand the weights in the front end's launch the expansion still runs unless
 * HBMM_CONV_WEIGHTS_PREPARED is given too.
 * Unknown flag bits: HBMM_ERR_INVALID_ARG.  Everything else as hbmm_conv_im2col (which is this call with
 * flags = 0).
 */
#define HBMM_CONV_WEIGHTS_PREPARED 1u
#define HBMM_CONV_PACK_ONLY 2u
/* beta_a == 1 only: x is an NHWC bf16 tensor [B, H, W, C] (16-byte aligned, C a multiple of 64) instead of NCHW --
 * what HBMM_OUT_DENSE of the layer before wrote.  The layout copy of the dense-activation path is skipped.
 * Otherwise HBMM_ERR_INVALID_ARG (beta_a, dtype) / HBMM_ERR_UNSUPPORTED (channel count) / HBMM_ERR_ALIGNMENT. */
#define HBMM_CONV_INPUT_NHWC 4u
hbmm_status hbmm_conv_im2col_ex(const void *x, int32_t x_dtype, const hbmm_conv_geom *g,
                                int32_t beta_a, int32_t a_scale_dtype, const hbmm_operand *W,
                                float *C_out, int64_t ldc, void *workspace, size_t workspace_bytes,
                                uint32_t flags, void *stream);

/*
 * hbmm_conv_im2col_ex with the epilogue chain of hbmm_epilogue instead of the fp32 NHWC store: the convolution,
 * the activation that follows it, the next block's folded batch normalisation, and the form the next layer
 * reads (dense NHWC bf16 / fp32, or rows binarized along the output channels).  beta_a >= 2: K = C*kh*kw a
 * multiple of 32 and activation groups of whole K-words (or one group per row); beta_a == 1: C a multiple of
 * 64.  Flags as hbmm_conv_im2col_ex except HBMM_CONV_PACK_ONLY.  Workspace as hbmm_conv_workspace_bytes.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE, CUDA.
 */
hbmm_status hbmm_conv_im2col_fused(const void *x, int32_t x_dtype, const hbmm_conv_geom *g, int32_t beta_a,
                                   int32_t a_scale_dtype, const hbmm_operand *W, const hbmm_epilogue *ep,
                                   void *workspace, size_t workspace_bytes, uint32_t flags, void *stream);

/*
 * hbmm_conv_im2col for callers that cannot allocate device memory.  (No counterpart in the
 * paper: this is a deployment convenience, not part of the method.)
 *
 * Who needs it: code that runs inside a host framework or inference server whose allocator
 * already owns all device memory, plugins that are handed nothing but tensor pointers and a
 * stream, and real-time loops where cudaMalloc/cudaFree (which synchronise the device) are
 * not allowed.  Such callers can pass inputs and outputs but have nowhere to get a workspace.
 *
 * Same arguments, results and errors as hbmm_conv_im2col, without the workspace: the packed
 * activation operand is kept in a fixed array of HBMM_STATIC_SCRATCH_BYTES inside the library's
 * device image (every GPU that loads the library holds that much memory until the process
 * exits).  The call allocates and frees nothing.  A problem whose hbmm_conv_workspace_bytes
 * exceeds HBMM_STATIC_SCRATCH_BYTES is rejected with HBMM_ERR_WORKSPACE before anything is
 * launched (this includes every realistic beta_a == 1 problem, whose bf16 row matrix is large).
 *
 * The first call on each device looks up the array's device address (the device must be
 * current); make that first call outside any stream capture, and at start-up: with CUDA's lazy
 * module loading it can be the call that brings the array into device memory, so it is the one
 * call that may synchronise and that can fail for lack of memory (HBMM_ERR_CUDA) when another
 * allocator has already taken the whole device.  Devices with an index of 64 or more are not
 * served (HBMM_ERR_CUDA).  All calls on a device share the
 * one array: it keeps whatever the last call left, which is harmless because each call rewrites
 * all of the region it reads (nothing has to start at zero), but two calls whose kernels can
 * overlap on the GPU (different streams, or different host threads on different streams) race
 * on it -- serialise them on one stream or with events.
 */
#define HBMM_STATIC_SCRATCH_BYTES ((size_t)32 << 20) /* 32 MiB */
hbmm_status hbmm_conv_im2col_static(const void *x, int32_t x_dtype, const hbmm_conv_geom *g,
                                    int32_t beta_a, int32_t a_scale_dtype, const hbmm_operand *W,
                                    float *C_out, int64_t ldc, void *stream);

/*
 * Device-side health word of the kernels that wait on barriers (the tensor-core contractions and the
 * packed convolution front end).  Their kernels never spin without a limit: a wait that does not
 * complete within the limit records a code, makes the kernel drain what it has in flight, free its
 * tensor memory and return, and leaves the output of that launch undefined.  Codes: 1 producer / tile
 * loader waiting for a free stage, 2 / 3 the MMA issuer waiting for a stage / for an accumulator, 4 the
 * final drain of the tensor core, 5 epilogue, 6 weight loader, 7 producer waiting for the row factors,
 * 8 the warps that compute them, 9 the self-test of hbmm_debug_expire_wait; reported as they are for
 * the e4m3 HBMM kernel, 100 + code for the HBWN kernel, 200 + code for the packed convolution front end
 * (201 loader, 202-204 compute warps), 300 + code for the folded-scale HBMM kernel.
 * Lifetime: one word per kernel family and process, holding the FIRST code recorded since it was last
 * cleared; nothing but hbmm_clear_device_error resets it, so after one expiry every later query reports
 * HBMM_ERR_TIMEOUT, whichever call it follows, until the word is cleared.
 * hbmm_last_device_error copies the words back (it synchronises the device) and returns
 * HBMM_ERR_TIMEOUT when one is non-zero, HBMM_OK otherwise.  code: host pointer, may be NULL.
 * hbmm_clear_device_error zeroes them (it synchronises too).
 */
hbmm_status hbmm_last_device_error(int32_t *code);
hbmm_status hbmm_clear_device_error(void);

/*
 * Test hooks for the bounded waits; not for production use.  (Section 4 of the paper has no counterpart:
 * they exist so that the failure path can be exercised without starving a real kernel.)
 * hbmm_debug_set_wait_limit: number of polls after which a device-side wait gives up, for every kernel
 * family, on the current device; 0 restores the default (2^20).  Synchronises.  Errors: INVALID_ARG, CUDA.
 * hbmm_debug_expire_wait: launches one tiny block on `stream` in which a single thread waits, with the
 * library's bounded wait, on a barrier that nobody will ever arrive at and that guards nothing (no copy and
 * no tensor-core work is in flight).  The wait runs out after the limit in force, code 309 is recorded and
 * the kernel returns normally.  Lower the limit first: with the default the launch takes about a second.
 */
hbmm_status hbmm_debug_set_wait_limit(uint32_t polls);
hbmm_status hbmm_debug_expire_wait(void *stream);

/*
 * Measurement aid: a register-only arithmetic loop that times the issue rate of one unit -- kind 0: 32-bit
 * population counts (each fed by an XOR, the inner step of Eq. 7's XNOR/popcount form), 1: fp32 additions
 * (the inner step of the sign-select form of the dense x packed product), 2: fp32 fused multiply-adds.
 * Launches `blocks` blocks of 1024 threads on `stream`; each thread runs `iters` iterations of eight
 * independent operations.  *ops (host, may be NULL) receives the operations per launch; the caller times
 * the launch.  sink: device, at least blocks * 1024 words (the loop's results are never stored in
 * practice).  Errors: INVALID_ARG, CUDA.
 */
hbmm_status hbmm_bench_alu_rate(int32_t kind, int32_t blocks, int32_t iters, uint32_t *sink, int64_t *ops,
                                void *stream);

/* Static, NUL-terminated description of a status code (host). */
const char *hbmm_status_string(int32_t status);

/* Library version, major*10000 + minor*100 + patch. */
int32_t hbmm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HBMM_H_ */
