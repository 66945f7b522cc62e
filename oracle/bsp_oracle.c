/*
 * CPU oracle for the weight-block-sparse operator Y = W*X + b.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the method computes,
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg.  It shares no
 * code, header, table or helper with the CUDA library and must never be linked into it.
 *
 * Notation follows the paper's Introduction: W is O x H x K x I (input channel innermost),
 * W-bar[i][j] = W[i,*,*,j] is the O x I abstraction, a block is b_o x b_i entries of W-bar (so
 * b_o x H x K x b_i weights), Gamma is the NB_o x NB_i 0/1 mask of Eq. (1), NB_o = O / b_o,
 * NB_i = I / b_i.  Activations X are N x L x J x I, outputs Y are N x M x Nw x O (channel
 * innermost); the paper has no batch dimension, N is added here.
 *
 * Floating point is accumulated in double; 8-bit integer paths are accumulated in int64 and
 * checked to fit int32.  Loops are written in the order of the definitions; the only
 * parallelism is an OpenMP loop over output pixels, which does not change any result.
 *
 * Parity pins (tests/test_oracle_*.py): every function below is pinned against something other
 * than itself -- the paper's printed index example, Eq. (2) counts, numpy sort, a numpy/scipy
 * dense correlation of Gamma (.) W, closed forms and brute force on tiny shapes; the requantising
 * epilogue against hand-worked values and an exact rational restatement.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_SHAPE 1
#define ORACLE_ERR_OVERFLOW 2
#define ORACLE_ERR_ALLOC 3

typedef struct {
    int O, I, H, K, bo, bi;
} ref_wdesc;

typedef struct {
    int N, L, J, stride_h, stride_w, pad_h, pad_w;
} ref_xdesc;

static int wdesc_ok(const ref_wdesc *w)
{
    if (w->O <= 0 || w->I <= 0 || w->H <= 0 || w->K <= 0 || w->bo <= 0 || w->bi <= 0) return 0;
    /* Section "Experiments": a layer whose channels do not fill a block cannot be made sparse. */
    if (w->O % w->bo != 0 || w->I % w->bi != 0) return 0;
    return 1;
}

int ref_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
    return omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}

/* ---------------------------------------------------------------------------------------------
 * Block importance (Section "Predetermined Sparsity ratio and Full Training Ahead").
 * norm 0: L2 ranked by its square, sum of w^2 over the b_o x H x K x b_i block.  The square root
 *         is left out because it does not change the order.  Each product of two float values is
 *         exact in double; the sum runs over (h, k, c) for one output row r of the block, then
 *         the b_o row sums are added in order of r.
 * norm 1: L1, sum of |w|, same order.
 * norm 2: variance of the block's entries about the block's own mean, n = b_o*H*K*b_i.
 * ------------------------------------------------------------------------------------------- */
int ref_scores_f32(const ref_wdesc *w, const float *W, int norm, double *score)
{
    if (!wdesc_ok(w)) return ORACLE_ERR_SHAPE;
    const int NBo = w->O / w->bo, NBi = w->I / w->bi;
    const double n_elems = (double)w->bo * w->H * w->K * w->bi;
    for (int l = 0; l < NBo; ++l)
        for (int iota = 0; iota < NBi; ++iota) {
            double mean = 0.0;
            if (norm == 2) {
                double s = 0.0;
                for (int r = 0; r < w->bo; ++r) {
                    double pr = 0.0;
                    for (int h = 0; h < w->H; ++h)
                        for (int k = 0; k < w->K; ++k)
                            for (int c = 0; c < w->bi; ++c)
                                pr += (double)W[(((size_t)(l * w->bo + r) * w->H + h) * w->K + k) * w->I + iota * w->bi + c];
                    s += pr;
                }
                mean = s / n_elems;
            }
            double total = 0.0;
            for (int r = 0; r < w->bo; ++r) {
                double pr = 0.0;
                for (int h = 0; h < w->H; ++h)
                    for (int k = 0; k < w->K; ++k)
                        for (int c = 0; c < w->bi; ++c) {
                            double v = (double)W[(((size_t)(l * w->bo + r) * w->H + h) * w->K + k) * w->I + iota * w->bi + c];
                            if (norm == 0) pr += v * v;
                            else if (norm == 1) pr += (v < 0 ? -v : v);
                            else pr += (v - mean) * (v - mean);
                        }
                total += pr;
            }
            score[(size_t)l * NBi + iota] = (norm == 2) ? total / n_elems : total;
        }
    return ORACLE_OK;
}

/* Integer weights: the sums are exact, so the order is immaterial.  norm 0 (sum w^2), 1 (sum |w|). */
int ref_scores_i8(const ref_wdesc *w, const int8_t *W, int norm, int64_t *score)
{
    if (!wdesc_ok(w)) return ORACLE_ERR_SHAPE;
    if (norm != 0 && norm != 1) return ORACLE_ERR_SHAPE;
    const int NBo = w->O / w->bo, NBi = w->I / w->bi;
    for (int l = 0; l < NBo; ++l)
        for (int iota = 0; iota < NBi; ++iota) {
            int64_t total = 0;
            for (int r = 0; r < w->bo; ++r)
                for (int h = 0; h < w->H; ++h)
                    for (int k = 0; k < w->K; ++k)
                        for (int c = 0; c < w->bi; ++c) {
                            int64_t v = W[(((size_t)(l * w->bo + r) * w->H + h) * w->K + k) * w->I + iota * w->bi + c];
                            total += (norm == 0) ? v * v : (v < 0 ? -v : v);
                        }
            score[(size_t)l * NBi + iota] = total;
        }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Gamma from scores: "sort them in ascending order, set the first [n_zero] to zero".
 * Ties are ordered by block index (lower index first).  scope 0 ranks all NB blocks of the layer
 * together; scope 1 ranks each row of Gamma on its own and zeroes n_zero blocks in every row,
 * the per-row reading of Eq. (2).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    double fs;
    int64_t is;
    int64_t idx;
} rank_item;

static int cmp_f(const void *a, const void *b)
{
    const rank_item *x = (const rank_item *)a, *y = (const rank_item *)b;
    if (x->fs < y->fs) return -1;
    if (x->fs > y->fs) return 1;
    return (x->idx < y->idx) ? -1 : (x->idx > y->idx);
}

static int cmp_i(const void *a, const void *b)
{
    const rank_item *x = (const rank_item *)a, *y = (const rank_item *)b;
    if (x->is < y->is) return -1;
    if (x->is > y->is) return 1;
    return (x->idx < y->idx) ? -1 : (x->idx > y->idx);
}

static int mask_segment(const double *fs, const int64_t *is, int64_t base, int64_t n, int64_t n_zero,
                        uint8_t *gamma)
{
    if (n_zero < 0 || n_zero > n) return ORACLE_ERR_SHAPE;
    rank_item *it = (rank_item *)malloc((size_t)(n > 0 ? n : 1) * sizeof(rank_item));
    if (!it) return ORACLE_ERR_ALLOC;
    for (int64_t i = 0; i < n; ++i) {
        it[i].fs = fs ? fs[base + i] : 0.0;
        it[i].is = is ? is[base + i] : 0;
        it[i].idx = base + i;
    }
    qsort(it, (size_t)n, sizeof(rank_item), fs ? cmp_f : cmp_i);
    for (int64_t i = 0; i < n; ++i) gamma[it[i].idx] = (i < n_zero) ? 0 : 1;
    free(it);
    return ORACLE_OK;
}

int ref_mask(int NBo, int NBi, const double *score_f, const int64_t *score_i, int scope, int64_t n_zero,
             uint8_t *gamma)
{
    if (NBo <= 0 || NBi <= 0 || (!score_f && !score_i)) return ORACLE_ERR_SHAPE;
    if (scope == 0) return mask_segment(score_f, score_i, 0, (int64_t)NBo * NBi, n_zero, gamma);
    for (int l = 0; l < NBo; ++l) {
        int rc = mask_segment(score_f, score_i, (int64_t)l * NBi, NBi, n_zero, gamma);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Compaction to compressed block rows (Section "Block Sparsity in a Matrix": CBR).
 * Gamma is scanned row by row; block n (in scan order) has column index col_idx[n] and payload
 * payload[n][r][h][k][c] = W[l*b_o + r][h][k][iota*b_i + c].  elem is the byte size of a weight.
 * Returns nnz through *nnz_out; capacity_blocks bounds col_idx/payload.
 * ------------------------------------------------------------------------------------------- */
int ref_compact(const ref_wdesc *w, const void *W, int elem, const uint8_t *gamma, int32_t *row_ptr,
                int32_t *col_idx, void *payload, int64_t capacity_blocks, int64_t *nnz_out)
{
    if (!wdesc_ok(w) || elem <= 0) return ORACLE_ERR_SHAPE;
    const int NBo = w->O / w->bo, NBi = w->I / w->bi;
    const size_t blk = (size_t)w->bo * w->H * w->K * w->bi * elem;
    const char *src = (const char *)W;
    char *dst = (char *)payload;
    int64_t n = 0;
    row_ptr[0] = 0;
    for (int l = 0; l < NBo; ++l) {
        for (int iota = 0; iota < NBi; ++iota) {
            if (!gamma[(size_t)l * NBi + iota]) continue;
            if (n >= capacity_blocks) return ORACLE_ERR_SHAPE;
            col_idx[n] = iota;
            size_t q = 0;
            for (int r = 0; r < w->bo; ++r)
                for (int h = 0; h < w->H; ++h)
                    for (int k = 0; k < w->K; ++k)
                        for (int c = 0; c < w->bi; ++c) {
                            size_t s = (((size_t)(l * w->bo + r) * w->H + h) * w->K + k) * w->I + iota * w->bi + c;
                            memcpy(dst + n * blk + q * elem, src + s * elem, (size_t)elem);
                            ++q;
                        }
            ++n;
        }
        row_ptr[l + 1] = (int32_t)n;
    }
    *nnz_out = n;
    return ORACLE_OK;
}

/* Output spatial size: floor((L + 2 pad - H) / stride) + 1. */
static int out_dim(int in, int pad, int k, int stride)
{
    int span = in + 2 * pad - k;
    if (span < 0) return 0;
    return span / stride + 1;
}

/* ---------------------------------------------------------------------------------------------
 * Block-sparse convolution with bias from the compact structure only (Introduction; Section
 * "Block Sparsity in a Matrix": products with a zero block are never formed).
 *
 *   Y[n,y,x,o] = b[o] + sum over the non-zero blocks (l, iota) of block row l = o / b_o,
 *                sum_{h,k} sum_{c<b_i} W[o,h,k,iota*b_i+c] * X[n, y*s_h+h-p_h, x*s_w+k-p_w, iota*b_i+c]
 *
 * with X taken as zero outside its bounds and no kernel flip (cross-correlation).
 * pix lists the flattened output pixels (n*M + y)*Nw + x to evaluate (NULL: all of them);
 * Y holds npix rows of O values.
 * ------------------------------------------------------------------------------------------- */
int ref_conv2d_f32(const ref_wdesc *w, const ref_xdesc *x, const int32_t *row_ptr, const int32_t *col_idx,
                   const float *payload, const float *X, const float *bias, const int64_t *pix,
                   int64_t npix, double *Y)
{
    if (!wdesc_ok(w)) return ORACLE_ERR_SHAPE;
    const int M = out_dim(x->L, x->pad_h, w->H, x->stride_h), Nw = out_dim(x->J, x->pad_w, w->K, x->stride_w);
    const int NBo = w->O / w->bo;
    const int64_t P = (int64_t)x->N * M * Nw;
    const size_t blk = (size_t)w->bo * w->H * w->K * w->bi;
    if (!pix) npix = P;
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < npix; ++q) {
        const int64_t p = pix ? pix[q] : q;
        const int xo = (int)(p % Nw), yo = (int)((p / Nw) % M), n = (int)(p / ((int64_t)Nw * M));
        for (int l = 0; l < NBo; ++l)
            for (int r = 0; r < w->bo; ++r) {
                const int o = l * w->bo + r;
                double acc = bias ? (double)bias[o] : 0.0;
                for (int32_t nb = row_ptr[l]; nb < row_ptr[l + 1]; ++nb) {
                    const int iota = col_idx[nb];
                    for (int h = 0; h < w->H; ++h) {
                        const int yi = yo * x->stride_h + h - x->pad_h;
                        if (yi < 0 || yi >= x->L) continue;
                        for (int k = 0; k < w->K; ++k) {
                            const int xi = xo * x->stride_w + k - x->pad_w;
                            if (xi < 0 || xi >= x->J) continue;
                            const float *xv = X + (((size_t)n * x->L + yi) * x->J + xi) * w->I + (size_t)iota * w->bi;
                            const float *wv = payload + nb * blk + (((size_t)r * w->H + h) * w->K + k) * w->bi;
                            for (int c = 0; c < w->bi; ++c) acc += (double)wv[c] * (double)xv[c];
                        }
                    }
                }
                Y[q * w->O + o] = acc;
            }
    }
    return ORACLE_OK;
}

int ref_conv2d_i8(const ref_wdesc *w, const ref_xdesc *x, const int32_t *row_ptr, const int32_t *col_idx,
                  const int8_t *payload, const int8_t *X, const int32_t *bias, const int64_t *pix,
                  int64_t npix, int32_t *Y)
{
    if (!wdesc_ok(w)) return ORACLE_ERR_SHAPE;
    const int M = out_dim(x->L, x->pad_h, w->H, x->stride_h), Nw = out_dim(x->J, x->pad_w, w->K, x->stride_w);
    const int NBo = w->O / w->bo;
    const int64_t P = (int64_t)x->N * M * Nw;
    const size_t blk = (size_t)w->bo * w->H * w->K * w->bi;
    int overflow = 0;
    if (!pix) npix = P;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t q = 0; q < npix; ++q) {
        const int64_t p = pix ? pix[q] : q;
        const int xo = (int)(p % Nw), yo = (int)((p / Nw) % M), n = (int)(p / ((int64_t)Nw * M));
        for (int l = 0; l < NBo; ++l)
            for (int r = 0; r < w->bo; ++r) {
                const int o = l * w->bo + r;
                int64_t acc = bias ? (int64_t)bias[o] : 0;
                for (int32_t nb = row_ptr[l]; nb < row_ptr[l + 1]; ++nb) {
                    const int iota = col_idx[nb];
                    for (int h = 0; h < w->H; ++h) {
                        const int yi = yo * x->stride_h + h - x->pad_h;
                        if (yi < 0 || yi >= x->L) continue;
                        for (int k = 0; k < w->K; ++k) {
                            const int xi = xo * x->stride_w + k - x->pad_w;
                            if (xi < 0 || xi >= x->J) continue;
                            const int8_t *xv = X + (((size_t)n * x->L + yi) * x->J + xi) * w->I + (size_t)iota * w->bi;
                            const int8_t *wv = payload + nb * blk + (((size_t)r * w->H + h) * w->K + k) * w->bi;
                            for (int c = 0; c < w->bi; ++c) acc += (int64_t)wv[c] * (int64_t)xv[c];
                        }
                    }
                }
                if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
                Y[q * w->O + o] = (int32_t)acc;
            }
    }
    return overflow ? ORACLE_ERR_OVERFLOW : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Block-sparse matrix product for fully connected layers (Section "Block Sparsity in a Matrix"):
 *   Y[p][o] = b[o] + sum over non-zero blocks (l, iota), l = o / b_o, of
 *             sum_{c<b_i} W-bar[o][iota*b_i + c] * X[p][iota*b_i + c]
 * X is stored [P][I], Y [P][O]; H = K = 1, so a payload block is b_o x b_i.
 * Written on its own (not through the convolution) so that each checks the other.
 * ------------------------------------------------------------------------------------------- */
int ref_gemm_f32(int O, int I, int bo, int bi, const int32_t *row_ptr, const int32_t *col_idx,
                 const float *payload, const float *X, int64_t P, const float *bias, const int64_t *pix,
                 int64_t npix, double *Y)
{
    if (O <= 0 || I <= 0 || bo <= 0 || bi <= 0 || O % bo || I % bi) return ORACLE_ERR_SHAPE;
    if (!pix) npix = P;
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < npix; ++q) {
        const int64_t p = pix ? pix[q] : q;
        for (int o = 0; o < O; ++o) {
            const int l = o / bo, r = o % bo;
            double acc = bias ? (double)bias[o] : 0.0;
            for (int32_t nb = row_ptr[l]; nb < row_ptr[l + 1]; ++nb) {
                const float *wv = payload + ((size_t)nb * bo + r) * bi;
                const float *xv = X + (size_t)p * I + (size_t)col_idx[nb] * bi;
                for (int c = 0; c < bi; ++c) acc += (double)wv[c] * (double)xv[c];
            }
            Y[q * O + o] = acc;
        }
    }
    return ORACLE_OK;
}

int ref_gemm_i8(int O, int I, int bo, int bi, const int32_t *row_ptr, const int32_t *col_idx,
                const int8_t *payload, const int8_t *X, int64_t P, const int32_t *bias, const int64_t *pix,
                int64_t npix, int32_t *Y)
{
    if (O <= 0 || I <= 0 || bo <= 0 || bi <= 0 || O % bo || I % bi) return ORACLE_ERR_SHAPE;
    int overflow = 0;
    if (!pix) npix = P;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t q = 0; q < npix; ++q) {
        const int64_t p = pix ? pix[q] : q;
        for (int o = 0; o < O; ++o) {
            const int l = o / bo, r = o % bo;
            int64_t acc = bias ? (int64_t)bias[o] : 0;
            for (int32_t nb = row_ptr[l]; nb < row_ptr[l + 1]; ++nb) {
                const int8_t *wv = payload + ((size_t)nb * bo + r) * bi;
                const int8_t *xv = X + (size_t)p * I + (size_t)col_idx[nb] * bi;
                for (int c = 0; c < bi; ++c) acc += (int64_t)wv[c] * (int64_t)xv[c];
            }
            if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
            Y[q * O + o] = (int32_t)acc;
        }
    }
    return overflow ? ORACLE_ERR_OVERFLOW : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Textbook dense convolution with bias on a full O x H x K x I weight tensor (for the check
 * "sparse result == dense convolution of Gamma (.) W").  Loop order: pixel, o, h, k, i.
 * ------------------------------------------------------------------------------------------- */
int ref_dense_conv2d_f32(const ref_wdesc *w, const ref_xdesc *x, const float *W, const float *X,
                         const float *bias, double *Y)
{
    const int M = out_dim(x->L, x->pad_h, w->H, x->stride_h), Nw = out_dim(x->J, x->pad_w, w->K, x->stride_w);
    const int64_t P = (int64_t)x->N * M * Nw;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        const int xo = (int)(p % Nw), yo = (int)((p / Nw) % M), n = (int)(p / ((int64_t)Nw * M));
        for (int o = 0; o < w->O; ++o) {
            double acc = bias ? (double)bias[o] : 0.0;
            for (int h = 0; h < w->H; ++h) {
                const int yi = yo * x->stride_h + h - x->pad_h;
                if (yi < 0 || yi >= x->L) continue;
                for (int k = 0; k < w->K; ++k) {
                    const int xi = xo * x->stride_w + k - x->pad_w;
                    if (xi < 0 || xi >= x->J) continue;
                    for (int i = 0; i < w->I; ++i)
                        acc += (double)W[(((size_t)o * w->H + h) * w->K + k) * w->I + i] *
                               (double)X[(((size_t)n * x->L + yi) * x->J + xi) * w->I + i];
                }
            }
            Y[p * w->O + o] = acc;
        }
    }
    return ORACLE_OK;
}

int ref_dense_conv2d_i8(const ref_wdesc *w, const ref_xdesc *x, const int8_t *W, const int8_t *X,
                        const int32_t *bias, int64_t *Y)
{
    const int M = out_dim(x->L, x->pad_h, w->H, x->stride_h), Nw = out_dim(x->J, x->pad_w, w->K, x->stride_w);
    const int64_t P = (int64_t)x->N * M * Nw;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        const int xo = (int)(p % Nw), yo = (int)((p / Nw) % M), n = (int)(p / ((int64_t)Nw * M));
        for (int o = 0; o < w->O; ++o) {
            int64_t acc = bias ? (int64_t)bias[o] : 0;
            for (int h = 0; h < w->H; ++h) {
                const int yi = yo * x->stride_h + h - x->pad_h;
                if (yi < 0 || yi >= x->L) continue;
                for (int k = 0; k < w->K; ++k) {
                    const int xi = xo * x->stride_w + k - x->pad_w;
                    if (xi < 0 || xi >= x->J) continue;
                    for (int i = 0; i < w->I; ++i)
                        acc += (int64_t)W[(((size_t)o * w->H + h) * w->K + k) * w->I + i] *
                               (int64_t)X[(((size_t)n * x->L + yi) * x->J + xi) * w->I + i];
                }
            }
            Y[p * w->O + o] = acc;
        }
    }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Requantising epilogue of the 8-bit path (Section "Compiler and its Code generation": an INT8
 * tensor carries a power-of-two scale, "a position where the fraction starts"; weights 8 bits,
 * bias 32 bits, scaling factors may differ per output channel; Eq. (quant) rounds to nearest).
 * The int32 value v = accumulator + bias of output channel o stands at 2^-(f_x + f_w[o]); the int8
 * output stands at 2^-f_y, so it is v / 2^s with s = shift[o] = f_x + f_w[o] - f_y >= 0, rounded
 * to the nearest integer, halves away from zero, then saturated to [-128, 127].
 * ------------------------------------------------------------------------------------------- */
int ref_requant_i8(int64_t rows, int O, const int32_t *y32, const int32_t *shift, int8_t *y8)
{
    if (rows < 0 || O <= 0) return ORACLE_ERR_SHAPE;
    for (int o = 0; o < O; ++o)
        if (shift[o] < 0 || shift[o] > 31) return ORACLE_ERR_SHAPE;
    for (int64_t p = 0; p < rows; ++p)
        for (int o = 0; o < O; ++o) {
            const int64_t v = (int64_t)y32[p * O + o];
            const int s = shift[o];
            int64_t mag = v < 0 ? -v : v;
            if (s > 0) mag = (mag + ((int64_t)1 << (s - 1))) >> s;      /* nearest, halves away from zero */
            int64_t q = v < 0 ? -mag : mag;
            if (q > 127) q = 127;
            if (q < -128) q = -128;
            y8[p * O + o] = (int8_t)q;
        }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Two consecutive layers evaluated tile by tile with the tensor between them kept on chip
 * (Section "Depth-wise Tiling").  The result is that of running the layers one after the other;
 * what the fused evaluation fixes is the precision of the tensor in between, which is stored as
 * bfloat16.  ref_round_bf16 rounds float64 values to the nearest bfloat16 (8 significant bits,
 * ties to the even mantissa) and returns them as float32; ref_relu_f64 is max(v, 0).
 * The chain itself is composed by the caller from ref_conv2d_f32, these two and ref_gemm_f32.
 * Values are assumed finite and inside the normal range of bfloat16.
 * ------------------------------------------------------------------------------------------- */
int ref_round_bf16(int64_t n, const double *in, float *out)
{
    if (n < 0) return ORACLE_ERR_SHAPE;
    for (int64_t i = 0; i < n; ++i) {
        const double v = in[i];
        if (v == 0.0) { out[i] = 0.0f; continue; }
        int e;
        const double m = frexp(fabs(v), &e);              /* |v| = m 2^e, 0.5 <= m < 1 */
        const double scaled = ldexp(m, 8);                /* 128 <= scaled < 256: 8 significant bits */
        double q = floor(scaled);
        const double rest = scaled - q;
        if (rest > 0.5 || (rest == 0.5 && fmod(q, 2.0) == 1.0)) q += 1.0;
        const double r = ldexp(q, e - 8);
        out[i] = (float)(v < 0 ? -r : r);                  /* exact: 8 bits fit a float */
    }
    return ORACLE_OK;
}

int ref_relu_f64(int64_t n, double *v)
{
    if (n < 0) return ORACLE_ERR_SHAPE;
    for (int64_t i = 0; i < n; ++i)
        if (v[i] < 0.0) v[i] = 0.0;
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Block-sparse x block-sparse product (Section "Block-Sparse Matrix-Matrix Multiplication"):
 *   C = (Gamma . A) (Omega . B)^t,   C_{i,j} = sum_k gamma_{i,k} A_{i,k} (omega_{j,k} B_{j,k})^t
 * with kb x kb blocks.  A and B are stored as compressed block rows (only blocks with a one in
 * their mask), so the block-column indices of row i of A and of row j of B are two ascending
 * lists; a product is formed exactly where both lists hold the same k: the lists are merged.
 * C is dense, [NBa*kb][NBb*kb], float64.
 * ------------------------------------------------------------------------------------------- */
int ref_spgemm_f32(int NBa, int NBb, int kb, const int32_t *a_row_ptr, const int32_t *a_col_idx,
                   const float *a_payload, const int32_t *b_row_ptr, const int32_t *b_col_idx,
                   const float *b_payload, double *C)
{
    if (NBa <= 0 || NBb <= 0 || kb <= 0) return ORACLE_ERR_SHAPE;
    const size_t ldc = (size_t)NBb * kb;
    for (int i = 0; i < NBa; ++i)
        for (int j = 0; j < NBb; ++j) {
            for (int r = 0; r < kb; ++r)
                for (int c = 0; c < kb; ++c) C[((size_t)i * kb + r) * ldc + (size_t)j * kb + c] = 0.0;
            int32_t pa = a_row_ptr[i], pb = b_row_ptr[j];
            while (pa < a_row_ptr[i + 1] && pb < b_row_ptr[j + 1]) {
                if (a_col_idx[pa] < b_col_idx[pb]) ++pa;
                else if (a_col_idx[pa] > b_col_idx[pb]) ++pb;
                else {
                    const float *Ab = a_payload + (size_t)pa * kb * kb, *Bb = b_payload + (size_t)pb * kb * kb;
                    for (int r = 0; r < kb; ++r)
                        for (int c = 0; c < kb; ++c) {
                            double acc = 0.0;
                            for (int t = 0; t < kb; ++t) acc += (double)Ab[r * kb + t] * (double)Bb[c * kb + t];
                            C[((size_t)i * kb + r) * ldc + (size_t)j * kb + c] += acc;
                        }
                    ++pa; ++pb;
                }
            }
        }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Relative column index (Section "Block Sparsity in a Matrix": "a relative row/col index"): within
 * each row of Gamma the first kept block keeps its column, every further one stores its distance
 * to the previous kept block of the row.  Distances are >= 1; both directions are given.
 * ------------------------------------------------------------------------------------------- */
int ref_index_to_relative(int NBo, const int32_t *row_ptr, const int32_t *col_idx, int32_t *rel)
{
    if (NBo <= 0) return ORACLE_ERR_SHAPE;
    for (int l = 0; l < NBo; ++l)
        for (int32_t n = row_ptr[l]; n < row_ptr[l + 1]; ++n)
            rel[n] = (n == row_ptr[l]) ? col_idx[n] : col_idx[n] - col_idx[n - 1];
    return ORACLE_OK;
}

int ref_index_from_relative(int NBo, const int32_t *row_ptr, const int32_t *rel, int32_t *col_idx)
{
    if (NBo <= 0) return ORACLE_ERR_SHAPE;
    for (int l = 0; l < NBo; ++l) {
        int32_t at = 0;
        for (int32_t n = row_ptr[l]; n < row_ptr[l + 1]; ++n) {
            at = (n == row_ptr[l]) ? rel[n] : at + rel[n];
            col_idx[n] = at;
        }
    }
    return ORACLE_OK;
}
