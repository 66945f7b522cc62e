/*
 * bsp.h -- C ABI of the weight-block-sparse linear operator Y = W*X + b on NVIDIA B200 (sm_100a).
 *
 * Notation is the paper's (Introduction): the kernel W is O x H x K x I, stored with the input
 * channel innermost ([O][H][K][I], Section "Compiler and its Code generation": C_OUT x h x w x C_IN);
 * W-bar[i][j] = W[i,*,*,j] is its O x I abstraction; a block is b_o x b_i entries of W-bar, i.e.
 * b_o x H x K x b_i weights, with b_o x b_i one of 8x8, 4x16, 16x4; Gamma is the 0/1 mask of Eq. (1)
 * with NB_o = O/b_o rows and NB_i = I/b_i columns.  Activations X are N x L x J x I and outputs Y are
 * N x M x N' x O, both channel-innermost (NHWC); the batch dimension N is an addition, the paper
 * describes one image.
 *
 * General rules
 *  - Every tensor pointer is a DEVICE pointer owned by the caller; descriptors (bsp_wdesc, bsp_xdesc,
 *    bsp_bcsr structs) are HOST structs read during the call.  The library allocates no device memory:
 *    scratch comes from the caller's workspace `ws` (device, 256-byte aligned), sized by the matching
 *    *_workspace_bytes() call.  The caller zero-fills the first 256 bytes of a workspace once after
 *    allocating it (they hold the latched status word and the counters of the grid-wide barrier that the
 *    single-launch kernels of small layers use); one workspace sized for the largest request may serve all
 *    calls issued on one stream, and a workspace must not be shared by calls running on different streams.
 *  - Alignment: W and the canonical payload must be 4-byte aligned (the set-up kernels read
 *    32-bit words and use 16-byte accesses when the addresses allow it); X, Y and the packed buffer 16-byte
 *    aligned.  A misaligned pointer is BSP_ERR_SHAPE.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls only enqueue work and
 *    return; results are valid once the stream has been synchronised.
 *  - Every function returns a bsp_status; nothing throws.  Argument errors are detected on the host
 *    before anything is launched.  Device-side problems are latched in a status word inside the
 *    workspace and read back by bsp_check().
 *  - O and I must be multiples of b_o and b_i (Section "Experiments": a layer with fewer channels than a
 *    block, such as a 3-channel first layer, cannot be made block sparse) and, for the product kernels,
 *    multiples of 8 (I a multiple of 16 for int8, so that every row of X is a multiple of 16 bytes).
 */
#ifndef BSP_H
#define BSP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BSP_OK = 0,
    BSP_ERR_NULL = 1,      /* a required pointer is NULL */
    BSP_ERR_SHAPE = 2,     /* sizes <= 0, O % b_o != 0, I % b_i != 0, empty output, unsupported multiple */
    BSP_ERR_BLOCK = 3,     /* b_o x b_i is not 8x8, 4x16 or 16x4 */
    BSP_ERR_DTYPE = 4,     /* element type not valid for this call or combination */
    BSP_ERR_CAPACITY = 5,  /* an output buffer or count is too small */
    BSP_ERR_INDEX = 6,     /* compact structure inconsistent with the descriptor */
    BSP_ERR_CUDA = 7,      /* a CUDA runtime call failed */
    BSP_ERR_TIMEOUT = 8    /* a bounded device-side wait expired (latched in the workspace) */
} bsp_status;

typedef enum { BSP_F32 = 0, BSP_BF16 = 1, BSP_I8 = 2, BSP_I32 = 3 } bsp_dtype;

/* Block importance (Section "Predetermined Sparsity ratio and Full Training Ahead"). */
typedef enum { BSP_NORM_L2 = 0, BSP_NORM_L1 = 1, BSP_NORM_VAR = 2 } bsp_norm;

/* Which blocks compete when the lowest scores are zeroed.  LAYER: all NB_o*NB_i blocks are ranked
 * together (Section "Predetermined Sparsity ratio and Full Training Ahead").  ROW: each row of Gamma is ranked on its own and gets
 * n_zero zeros, the per-row reading of Eq. (2). */
typedef enum { BSP_SCOPE_LAYER = 0, BSP_SCOPE_ROW = 1 } bsp_scope;

/* Weight descriptor: W is [O][H][K][I] of `wtype` (BSP_F32, BSP_BF16 or BSP_I8). */
typedef struct {
    int O, I, H, K, bo, bi;
    bsp_dtype wtype;
} bsp_wdesc;

/* Activation descriptor: X is [N][L][J][I]; output is [N][M][N'][O] with
 * M = (L + 2 pad_h - H) / stride_h + 1 and N' = (J + 2 pad_w - K) / stride_w + 1 (integer division).
 * Zero padding, no dilation, no groups, no kernel flip (cross-correlation). */
typedef struct {
    int N, L, J;
    int stride_h, stride_w, pad_h, pad_w;
} bsp_xdesc;

/* Compacted weights (Section "Block Sparsity in a Matrix": compressed block rows).
 *   row_ptr [NB_o+1]  first stored block of each row of Gamma; row_ptr[NB_o] = nnz
 *   col_idx [nnz]     column of Gamma of each stored block, ascending within a row
 *   payload [nnz][b_o][H][K][b_i]  the surviving weights in canonical order
 *   packed            the same weights in the kernels' own tile order, written by bsp_compact and
 *                     opaque to the caller (bsp_packed_bytes() gives its size)
 *   nnz               number of stored blocks (host copy; used for size checks only)
 * The product kernels read `packed`; row_ptr/col_idx/payload are the portable form. */
typedef struct {
    const int32_t *row_ptr;
    const int32_t *col_idx;
    const void *payload;
    const void *packed;
    int64_t nnz;
} bsp_bcsr;

/* ---- Gamma builder (Eq. (1), Eq. (2); Section "Predetermined Sparsity ratio ...") ------------------
 * score[l][iota] = sum of w^2 (L2, ranked by its square), sum of |w| (L1) or, for float weights, the variance
 * of the block's entries about the block's own mean (VAR, n = b_o H K b_i) over the b_o x H x K x b_i
 * block; the n_zero blocks with the lowest (score, block index) pairs get Gamma = 0, all others 1.
 * Float weights: scores are float64, each product exact, summed over (h, k, c) for each output row r of
 * the block and then over r, always in that order, so that the mask is reproducible bit for bit.
 * int8 weights: scores are exact int64.
 *   W          [O][H][K][I] device, not modified
 *   n_zero     number of blocks to zero: 0..NB (LAYER) or 0..NB_i per row (ROW)
 *   gamma      [NB_o*NB_i] uint8 device, out
 *   scores_opt [NB_o*NB_i] float64 (float W) or int64 (int8 W) device, out; may be NULL
 *   ws         device scratch of bsp_mask_workspace_bytes() bytes
 * Errors: NULL, SHAPE, BLOCK, DTYPE (wtype I32; VAR with int8 weights), CAPACITY (n_zero out of range), CUDA. */
size_t bsp_mask_workspace_bytes(const bsp_wdesc *wd);
bsp_status bsp_mask(const bsp_wdesc *wd, const void *W, bsp_norm norm, bsp_scope scope, int64_t n_zero,
                    uint8_t *gamma, void *scores_opt, void *ws, void *stream);

/* ---- Gamma builder without caller scratch ------------------------------------------------------------
 * (The paper has no counterpart: this entry point exists for the way the library is embedded.)
 * Some hosts of this library may not allocate device memory at the point where a layer is masked: code that
 * runs inside another framework's memory plan or with a fixed, pre-carved device heap, plugins that are
 * handed only their input and output tensors, and real-time loops in which cudaMalloc (a blocking, device-
 * wide call) is banned.  Such callers cannot size and pass the `ws` buffer that bsp_mask() needs for the
 * block scores.  bsp_mask_static() computes exactly what bsp_mask() computes (the same bit-exact Gamma, by the
 * score and selection kernels that need no workspace) but keeps the scores in a fixed array inside the library's device image and allocates nothing: it
 * calls neither cudaMalloc/cudaFree nor any allocating library routine.
 *   - Limit: NB = (O/b_o)*(I/b_i) <= BSP_MASK_STATIC_MAX_BLOCKS; a larger layer returns BSP_ERR_CAPACITY and
 *     launches nothing.  The array (8 bytes per block, 512 KiB) is held on every GPU that loads the library,
 *     for the life of the process.
 *   - The first call on each device looks up the array's device address (with that device current) and
 *     caches it; make that first call outside any stream capture, and from one host thread (the cache is a
 *     plain pointer per device: concurrent first calls would all store the same value, but nothing orders them).
 *   - All calls on a device share the one array, which keeps the previous call's scores; every entry that
 *     is read is rewritten first, so no clearing is needed, but two calls that overlap on the GPU (different
 *     streams, or the same layer masked concurrently) race on it.  Serialise them on one stream.
 *   - There is no scores output and no latched status; arguments are otherwise those of bsp_mask().
 * Errors: NULL, SHAPE, BLOCK, DTYPE, CAPACITY (n_zero out of range, or NB over the limit), CUDA. */
#define BSP_MASK_STATIC_MAX_BLOCKS 65536
bsp_status bsp_mask_static(const bsp_wdesc *wd, const void *W, bsp_norm norm, bsp_scope scope,
                           int64_t n_zero, uint8_t *gamma, void *stream);

/* ---- Compaction (Section "Block Sparsity in a Matrix"; Section "Subvolumes, Data Compression ...") --
 * bsp_packed_bytes: size of the opaque `packed` buffer able to hold `nnz` stored blocks.
 * bsp_compact_nnz : counts the ones of a device Gamma and returns the count on the host; this one call
 *                   synchronises the stream.
 * bsp_compact     : scans Gamma (caller supplied or from bsp_mask) row by row and writes row_ptr, col_idx,
 *                   the canonical payload and the packed form (Gamma (.) W in the layout of W, for the TMA loads of
 *                   the product kernel; its size does not depend on nnz).  `payload` may be NULL (canonical copy
 *                   skipped); `packed` may be NULL (portable form only).  capacity_blocks is the number of
 *                   blocks col_idx/payload/packed were sized for; if Gamma holds more, nothing beyond the
 *                   capacity is written and BSP_ERR_CAPACITY is latched for bsp_check().
 *                   A dense layer is the same call with Gamma == 1.
 *   ws  device scratch of bsp_compact_workspace_bytes() bytes. */
size_t bsp_packed_bytes(const bsp_wdesc *wd, int64_t nnz);
size_t bsp_compact_workspace_bytes(const bsp_wdesc *wd);
bsp_status bsp_compact_nnz(const bsp_wdesc *wd, const uint8_t *gamma, int64_t *nnz_host, void *ws,
                           void *stream);
bsp_status bsp_compact(const bsp_wdesc *wd, const void *W, const uint8_t *gamma, int32_t *row_ptr,
                       int32_t *col_idx, void *payload, void *packed, int64_t capacity_blocks, void *ws,
                       void *stream);

/* ---- Block-sparse products (Introduction; Section "Block Sparsity in a Matrix") ---------------------
 * bsp_gemm  : Y[p][o] = bias[o] + sum over stored blocks (l = o / b_o, iota) sum_c W-bar[o][iota b_i + c]
 *             X[p][iota b_i + c].  X is [P][I], Y is [P][O] (a fully connected layer is a 1x1 convolution
 *             over P pixels); wd->H = wd->K = 1.
 * bsp_conv2d: Y[n,y,x,o] = bias[o] + sum over stored blocks of row o / b_o, over taps (h,k) and channels c of
 *             W[o,h,k,iota b_i + c] X[n, y s_h + h - p_h, x s_w + k - p_w, iota b_i + c], X = 0 out of bounds.
 * Types: BF16 or F32 inputs (wtype = type of X) accumulate in float32, bias float32, ytype F32 or BF16 (round to
 * nearest even after the bias); F32 inputs are multiplied as TF32 (the tensor core reads the upper 19 bits of each
 * operand).  I8 inputs accumulate in int32 (exact), bias int32, ytype I32.
 *   bias may be NULL (treated as zero).  ws: device scratch of bsp_conv_workspace_bytes() bytes.
 * One kernel implements the products ("gemm_tc_kernel": tcgen05 MMAs with the accumulators in tensor memory, both
 * operands staged by tiled TMA loads; a convolution is an implicit GEMM over taps x channel chunks).  It reads
 * `packed`, which holds Gamma (.) W in the layout of W: zeroed blocks cost no arithmetic result and no entry in
 * row_ptr / col_idx / payload, but the tensor-core instruction multiplies them as zeros (an instruction covers
 * 128 x 256 x 16 entries of the operands, far more than a block).
 * The kernel compares the header of `packed` with wd before it loads anything; a buffer that bsp_compact filled for
 * another descriptor latches BSP_ERR_INDEX and leaves Y untouched.  bsp_conv_kernel_name() names the kernel a call
 * with these descriptors takes (static storage; NULL for descriptors no kernel takes).
 * Errors: NULL, SHAPE, BLOCK, DTYPE, INDEX (nnz out of range; packed buffer does not match wd: latched), CUDA. */
size_t bsp_conv_workspace_bytes(const bsp_wdesc *wd, const bsp_xdesc *xd);
bsp_status bsp_gemm(const bsp_wdesc *wd, const bsp_bcsr *w, const void *X, int64_t P, const void *bias,
                    void *Y, bsp_dtype ytype, void *ws, void *stream);
bsp_status bsp_conv2d(const bsp_wdesc *wd, const bsp_bcsr *w, const bsp_xdesc *xd, const void *X,
                      const void *bias, void *Y, bsp_dtype ytype, void *ws, void *stream);
const char *bsp_conv_kernel_name(const bsp_wdesc *wd, const bsp_xdesc *xd);

/* ---- 8-bit products with a requantised int8 output (Section "Compiler and its Code generation": an INT8 tensor
 * carries a power-of-two scale, weights are 8 bits, the bias 32 bits, scales may differ per output channel; the
 * round-to-nearest of Eq. (quant)) -----------------------------------------------------------------------------
 * The same products as bsp_gemm / bsp_conv2d on I8 weights and activations, with the epilogue
 *   Y[.., o] = saturate_int8( round( (accumulator + bias[o]) / 2^shift[o] ) ),
 * rounded to the nearest integer with halves away from zero, saturated to [-128, 127].  With X at scale 2^-f_x, the
 * weights of channel o at 2^-f_w[o] (bias at their product) and Y at 2^-f_y the shift is f_x + f_w[o] - f_y.
 *   bias   int32 [O] device, may be NULL      shift  int32 [O] device, every entry in 0..31 (only the low 5 bits are read)
 *   Y      int8, NHWC / [P][O]; O must be a multiple of 16 (rows of Y are 16-byte multiples)
 * Errors: as bsp_conv2d; NULL shift; DTYPE if the weights are not I8. */
bsp_status bsp_gemm_q8(const bsp_wdesc *wd, const bsp_bcsr *w, const void *X, int64_t P, const int32_t *bias,
                       const int32_t *shift, int8_t *Y, void *ws, void *stream);
bsp_status bsp_conv2d_q8(const bsp_wdesc *wd, const bsp_bcsr *w, const bsp_xdesc *xd, const void *X,
                         const int32_t *bias, const int32_t *shift, int8_t *Y, void *ws, void *stream);

/* ---- Two consecutive layers in one kernel (Section "Depth-wise Tiling": the output is cut into tiles, each tile is
 * carried through the chain of layers, and the tensors between the layers stay on chip) ----------------------------
 * bsp_conv2d_chain: T = act(W1 * X + bias1) rounded to bfloat16 (nearest even), Y = W2 * T + bias2, where layer one is
 *             any convolution that bsp_conv2d takes (taps, strides, zero padding as given by xd) with at most 256
 *             output channels, act is max(., 0) if relu != 0 and the identity otherwise, and layer two is a 1x1
 *             layer on those channels (wd2->H = wd2->K = 1, wd2->I = wd1->O).  Both layers BF16 (weights and X),
 *             accumulation and both biases float32 (device, may be NULL), Y [N][M][N_w][O2] F32 or BF16.  T is never
 *             written to memory: a tile of 128 output positions of layer one is its own input tile of layer two.
 *             w1 / w2: compact forms of the two layers from bsp_compact (`packed` is read; its header is compared with
 *             the descriptors as in bsp_conv2d).  ws: any workspace of at least 256 bytes (status word only).
 * Errors: NULL, SHAPE (second layer not 1x1 on O1 channels, O1 > 256, misaligned buffers), BLOCK, DTYPE (not BF16;
 *         ytype not F32 / BF16), INDEX (nnz out of range; a packed buffer does not match: latched), CUDA. */
bsp_status bsp_conv2d_chain(const bsp_wdesc *wd1, const bsp_bcsr *w1, const bsp_wdesc *wd2, const bsp_bcsr *w2,
                            const bsp_xdesc *xd, const void *X, const float *bias1, int relu, const float *bias2, void *Y,
                            bsp_dtype ytype, void *ws, void *stream);
/* bsp_conv2d_chain_q8: the same chain on I8 layers with the 8-bit tensors of Section "Compiler and its Code generation":
 *             T = act(saturate_int8(round((W1 * X + bias1) / 2^shift1[o]))) is the requantised int8 output of layer one
 *             (the rounding of bsp_conv2d_q8; act = max(., 0) if relu != 0), Y = W2 * T + bias2 as int32, or, when
 *             shift2 is not NULL, requantised to int8 in the same way.  bias1 / bias2 int32 (device, may be NULL),
 *             shift1 [O1] required, shift2 [O2] optional, entries 0..31.  I1 and O1 multiples of 16, O2 a multiple of
 *             16 for an int8 Y.  Exact integer arithmetic: bit-identical to bsp_conv2d_q8 followed by bsp_conv2d
 *             (or bsp_conv2d_q8).
 * Errors: as bsp_conv2d_chain; NULL shift1; DTYPE if the layers are not I8. */
bsp_status bsp_conv2d_chain_q8(const bsp_wdesc *wd1, const bsp_bcsr *w1, const bsp_wdesc *wd2, const bsp_bcsr *w2,
                               const bsp_xdesc *xd, const void *X, const int32_t *bias1, const int32_t *shift1, int relu,
                               const int32_t *bias2, const int32_t *shift2, void *Y, void *ws, void *stream);

/* ---- Block-sparse x block-sparse product (Section "Block-Sparse Matrix-Matrix Multiplication") and the relative column
 * index (Section "Block Sparsity in a Matrix": "a relative row/col index") ------------------------------------------
 * bsp_spgemm: C = (Gamma . A)(Omega . B)^t, i.e. C_{i,j} = sum over the block columns k that row i of A and row j of B
 *             both keep of A_{i,k} B_{j,k}^t.  A is wa->O x wa->I, B is wb->O x wb->I with the same I, both with H = K = 1,
 *             8x8 blocks and the same type (F32 or BF16); `a` and `b` are their compact forms from bsp_compact (row_ptr,
 *             col_idx and the canonical payload are read; `packed` is not).  C is dense float32 [wa->O][wb->O], 8-byte
 *             aligned (the two payloads 16-byte aligned), written in full (blocks without a common column are zero).  Products are accumulated in float32
 *             in ascending order of k.  A column index outside the matrix is skipped and latches BSP_ERR_INDEX.
 *             ws: any workspace of at least 256 bytes (status word only).
 * bsp_index_to_relative / bsp_index_from_relative: within each row of Gamma the first kept block keeps its column, every
 *             further one stores its distance (>= 1) to the previous kept block of the row; and back.  int32 in, int32
 *             out, [nnz] device arrays; row_ptr [NB_o + 1] as written by bsp_compact.
 * Errors: NULL, SHAPE (I differs, H K != 1, more than 12288 block columns), BLOCK (not 8x8), DTYPE, CUDA. */
bsp_status bsp_spgemm(const bsp_wdesc *wa, const bsp_bcsr *a, const bsp_wdesc *wb, const bsp_bcsr *b, float *C, void *ws,
                      void *stream);
bsp_status bsp_index_to_relative(int NBo, const int32_t *row_ptr, const int32_t *col_idx, int32_t *rel, void *stream);
bsp_status bsp_index_from_relative(int NBo, const int32_t *row_ptr, const int32_t *rel, int32_t *col_idx, void *stream);

/* Synchronises `stream` and returns the status latched in the workspace by the kernels that used it
 * (BSP_OK if none), then clears it. */
bsp_status bsp_check(void *ws, void *stream);

/* Text for a status code (static storage). */
const char *bsp_status_string(bsp_status s);

#ifdef __cplusplus
}
#endif
#endif /* BSP_H */
