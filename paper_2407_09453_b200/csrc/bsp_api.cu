// extern "C" entry points of libbsp: argument validation on the host, then kernel launches on the caller's
// stream.  Declarations and their contracts are in include/bsp.h.
#include <cstdio>
#include <cstdlib>
#include "bsp_internal.cuh"

namespace bsp {
void report_cuda_error(cudaError_t e, const char *expr, const char *file, int line)
{
    if (getenv("BSP_DEBUG")) fprintf(stderr, "libbsp: %s failed at %s:%d: %s\n", expr, file, line, cudaGetErrorString(e));
}
}  // namespace bsp

using namespace bsp;

namespace bsp {
bsp_status check_wdesc(const bsp_wdesc *wd)
{
    if (!wd) return BSP_ERR_NULL;
    if (wd->O <= 0 || wd->I <= 0 || wd->H <= 0 || wd->K <= 0) return BSP_ERR_SHAPE;
    const bool ok_block = (wd->bo == 8 && wd->bi == 8) || (wd->bo == 4 && wd->bi == 16) || (wd->bo == 16 && wd->bi == 4);
    if (!ok_block) return BSP_ERR_BLOCK;
    if (wd->O % wd->bo != 0 || wd->I % wd->bi != 0) return BSP_ERR_SHAPE;
    if (wd->wtype != BSP_F32 && wd->wtype != BSP_BF16 && wd->wtype != BSP_I8) return BSP_ERR_DTYPE;
    if ((long long)wd->H * wd->K > 120) return BSP_ERR_SHAPE;
    return BSP_OK;
}
}  // namespace bsp

namespace {
bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }
bool aligned4(const void *p) { return ((uintptr_t)p & 3u) == 0; }
}  // namespace

extern "C" {

const char *bsp_status_string(bsp_status s)
{
    switch (s) {
        case BSP_OK: return "ok";
        case BSP_ERR_NULL: return "null pointer";
        case BSP_ERR_SHAPE: return "bad shape";
        case BSP_ERR_BLOCK: return "block shape is not 8x8, 4x16 or 16x4";
        case BSP_ERR_DTYPE: return "bad element type";
        case BSP_ERR_CAPACITY: return "buffer or count too small";
        case BSP_ERR_INDEX: return "compact structure does not match the descriptor";
        case BSP_ERR_CUDA: return "CUDA runtime error";
        case BSP_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

size_t bsp_mask_workspace_bytes(const bsp_wdesc *wd)
{
    if (check_wdesc(wd) != BSP_OK) return 0;
    const size_t NB = (size_t)(wd->O / wd->bo) * (wd->I / wd->bi);
    return kWsHeader + align_up(NB * 8, 256) + align_up(kSelectScratch, 256);
}

bsp_status bsp_mask(const bsp_wdesc *wd, const void *W, bsp_norm norm, bsp_scope scope, int64_t n_zero,
                    uint8_t *gamma, void *scores_opt, void *ws, void *stream)
{
    bsp_status rc = check_wdesc(wd);
    if (rc != BSP_OK) return rc;
    if (!W || !gamma || !ws) return BSP_ERR_NULL;
    if (!aligned4(W)) return BSP_ERR_SHAPE;
    if (norm != BSP_NORM_L2 && norm != BSP_NORM_L1 && norm != BSP_NORM_VAR) return BSP_ERR_DTYPE;
    if (norm == BSP_NORM_VAR && wd->wtype == BSP_I8) return BSP_ERR_DTYPE;      // the variance is defined for float weights
    if (scope != BSP_SCOPE_LAYER && scope != BSP_SCOPE_ROW) return BSP_ERR_DTYPE;
    const int64_t NBi = wd->I / wd->bi, NB = (int64_t)(wd->O / wd->bo) * NBi;
    const int64_t limit = (scope == BSP_SCOPE_LAYER) ? NB : NBi;
    if (n_zero < 0 || n_zero > limit) return BSP_ERR_CAPACITY;
    void *scores = scores_opt ? scores_opt : (void *)((char *)ws + kWsHeader);
    return launch_mask(*wd, W, norm, scope, n_zero, gamma, scores, ws, (cudaStream_t)stream);
}

size_t bsp_packed_bytes(const bsp_wdesc *wd, int64_t nnz)
{
    if (check_wdesc(wd) != BSP_OK || nnz < 0) return 0;
    return packed_layout(*wd).total_bytes;
}

size_t bsp_compact_workspace_bytes(const bsp_wdesc *wd)
{
    if (check_wdesc(wd) != BSP_OK) return 0;
    const size_t n = (size_t)(wd->O / wd->bo) + 8;
    return kWsHeader + align_up(n * 4, 256);
}

bsp_status bsp_compact_nnz(const bsp_wdesc *wd, const uint8_t *gamma, int64_t *nnz_host, void *ws, void *stream)
{
    bsp_status rc = check_wdesc(wd);
    if (rc != BSP_OK) return rc;
    if (!gamma || !nnz_host || !ws) return BSP_ERR_NULL;
    const int64_t NB = (int64_t)(wd->O / wd->bo) * (wd->I / wd->bi);
    unsigned long long *cnt = (unsigned long long *)((char *)ws + kWsHeader);
    rc = launch_count(gamma, NB, cnt, (cudaStream_t)stream);
    if (rc != BSP_OK) return rc;
    unsigned long long h = 0;
    BSP_CUDA_OK(cudaMemcpyAsync(&h, cnt, sizeof(h), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    BSP_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    *nnz_host = (int64_t)h;
    return BSP_OK;
}

bsp_status bsp_compact(const bsp_wdesc *wd, const void *W, const uint8_t *gamma, int32_t *row_ptr,
                       int32_t *col_idx, void *payload, void *packed, int64_t capacity_blocks, void *ws,
                       void *stream)
{
    bsp_status rc = check_wdesc(wd);
    if (rc != BSP_OK) return rc;
    if (!W || !gamma || !row_ptr || !col_idx || !ws) return BSP_ERR_NULL;
    if (capacity_blocks < 0) return BSP_ERR_CAPACITY;
    if (packed && (wd->O % 8 != 0 || wd->I % 8 != 0)) return BSP_ERR_SHAPE;
    if (packed && !aligned16(packed)) return BSP_ERR_SHAPE;
    if (!aligned4(W) || (payload && !aligned4(payload))) return BSP_ERR_SHAPE;
    return launch_compact(*wd, W, gamma, row_ptr, col_idx, payload, packed, capacity_blocks, ws, (cudaStream_t)stream);
}

size_t bsp_conv_workspace_bytes(const bsp_wdesc *wd, const bsp_xdesc *xd)
{
    (void)xd;
    if (check_wdesc(wd) != BSP_OK) return 0;
    return kWsHeader;
}

namespace {
// Validation and launch shared by bsp_conv2d and bsp_conv2d_q8 (shift != NULL: int8 output).
bsp_status conv2d_any(const bsp_wdesc *wd, const bsp_bcsr *w, const bsp_xdesc *xd, const void *X, const void *bias,
                      const int32_t *shift, void *Y, bsp_dtype ytype, void *ws, void *stream)
{
    bsp_status rc = check_wdesc(wd);
    if (rc != BSP_OK) return rc;
    if (!w || !xd || !X || !Y || !ws || !w->packed) return BSP_ERR_NULL;
    if (xd->N <= 0 || xd->L <= 0 || xd->J <= 0 || xd->stride_h <= 0 || xd->stride_w <= 0 || xd->pad_h < 0 ||
        xd->pad_w < 0)
        return BSP_ERR_SHAPE;
    if (xd->L + 2 * xd->pad_h < wd->H || xd->J + 2 * xd->pad_w < wd->K) return BSP_ERR_SHAPE;
    if (wd->O % 8 != 0 || wd->I % 8 != 0) return BSP_ERR_SHAPE;
    if (wd->wtype == BSP_I8 && wd->I % 16 != 0) return BSP_ERR_SHAPE;   // rows of X must be 16-byte multiples
    if (wd->wtype == BSP_I8) { if (ytype != BSP_I32 && ytype != BSP_I8) return BSP_ERR_DTYPE; }
    else if (ytype != BSP_F32 && ytype != BSP_BF16) return BSP_ERR_DTYPE;
    if (ytype == BSP_I8 && wd->O % 16 != 0) return BSP_ERR_SHAPE;       // rows of an int8 Y must be 16-byte multiples
    if (!aligned16(X) || !aligned16(Y) || !aligned16(w->packed)) return BSP_ERR_SHAPE;
    if (shift && !aligned4(shift)) return BSP_ERR_SHAPE;
    // the packed header is on the device (the kernel checks it against the descriptor); the host checks the count
    const int64_t NB = (int64_t)(wd->O / wd->bo) * (wd->I / wd->bi);
    if (w->nnz < 0 || w->nnz > NB) return BSP_ERR_INDEX;
    if (!gemm_tc_eligible(*wd, *xd, ytype)) return BSP_ERR_SHAPE;
    return launch_gemm_tc(*wd, *xd, w->packed, X, bias, shift, Y, ytype, ws, (cudaStream_t)stream);
}
}  // namespace

bsp_status bsp_conv2d(const bsp_wdesc *wd, const bsp_bcsr *w, const bsp_xdesc *xd, const void *X,
                      const void *bias, void *Y, bsp_dtype ytype, void *ws, void *stream)
{
    if (ytype == BSP_I8) return BSP_ERR_DTYPE;           // an int8 output needs its shifts: bsp_conv2d_q8
    return conv2d_any(wd, w, xd, X, bias, nullptr, Y, ytype, ws, stream);
}

bsp_status bsp_conv2d_q8(const bsp_wdesc *wd, const bsp_bcsr *w, const bsp_xdesc *xd, const void *X,
                         const int32_t *bias, const int32_t *shift, int8_t *Y, void *ws, void *stream)
{
    if (!shift) return BSP_ERR_NULL;
    if (wd && wd->wtype != BSP_I8) return BSP_ERR_DTYPE;
    return conv2d_any(wd, w, xd, X, bias, shift, Y, BSP_I8, ws, stream);
}

static bsp_status chain_any(const bsp_wdesc *wd1, const bsp_bcsr *w1, const bsp_wdesc *wd2, const bsp_bcsr *w2, const bsp_xdesc *xd,
                            const void *X, const void *bias1, const int32_t *shift1, int relu, const void *bias2,
                            const int32_t *shift2, void *Y, bsp_dtype ytype, void *ws, void *stream)
{
    bsp_status rc = check_wdesc(wd1);
    if (rc != BSP_OK) return rc;
    rc = check_wdesc(wd2);
    if (rc != BSP_OK) return rc;
    if (!w1 || !w2 || !xd || !X || !Y || !ws || !w1->packed || !w2->packed) return BSP_ERR_NULL;
    if (xd->N <= 0 || xd->L <= 0 || xd->J <= 0 || xd->stride_h <= 0 || xd->stride_w <= 0 || xd->pad_h < 0 || xd->pad_w < 0)
        return BSP_ERR_SHAPE;
    if (xd->L + 2 * xd->pad_h < wd1->H || xd->J + 2 * xd->pad_w < wd1->K) return BSP_ERR_SHAPE;
    if (wd2->H != 1 || wd2->K != 1 || wd2->I != wd1->O || wd1->O > 256) return BSP_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(Y) || !aligned16(w1->packed) || !aligned16(w2->packed)) return BSP_ERR_SHAPE;
    if ((bias1 && !aligned4(bias1)) || (bias2 && !aligned4(bias2)) || (shift1 && !aligned4(shift1)) || (shift2 && !aligned4(shift2)))
        return BSP_ERR_SHAPE;
    const int64_t NB1 = (int64_t)(wd1->O / wd1->bo) * (wd1->I / wd1->bi), NB2 = (int64_t)(wd2->O / wd2->bo) * (wd2->I / wd2->bi);
    if (w1->nnz < 0 || w1->nnz > NB1 || w2->nnz < 0 || w2->nnz > NB2) return BSP_ERR_INDEX;
    if (!chain_tc_eligible(*wd1, *wd2, *xd, ytype)) return BSP_ERR_SHAPE;
    return launch_chain_tc(*wd1, w1->packed, *wd2, w2->packed, *xd, X, bias1, shift1, relu, bias2, shift2, Y, ytype, ws,
                           (cudaStream_t)stream);
}

bsp_status bsp_conv2d_chain(const bsp_wdesc *wd1, const bsp_bcsr *w1, const bsp_wdesc *wd2, const bsp_bcsr *w2,
                            const bsp_xdesc *xd, const void *X, const float *bias1, int relu, const float *bias2, void *Y,
                            bsp_dtype ytype, void *ws, void *stream)
{
    if (wd1 && wd2 && (wd1->wtype != BSP_BF16 || wd2->wtype != BSP_BF16)) return BSP_ERR_DTYPE;
    if (ytype != BSP_F32 && ytype != BSP_BF16) return BSP_ERR_DTYPE;
    return chain_any(wd1, w1, wd2, w2, xd, X, bias1, nullptr, relu, bias2, nullptr, Y, ytype, ws, stream);
}

bsp_status bsp_conv2d_chain_q8(const bsp_wdesc *wd1, const bsp_bcsr *w1, const bsp_wdesc *wd2, const bsp_bcsr *w2,
                               const bsp_xdesc *xd, const void *X, const int32_t *bias1, const int32_t *shift1, int relu,
                               const int32_t *bias2, const int32_t *shift2, void *Y, void *ws, void *stream)
{
    if (wd1 && wd2 && (wd1->wtype != BSP_I8 || wd2->wtype != BSP_I8)) return BSP_ERR_DTYPE;
    if (!shift1) return BSP_ERR_NULL;
    return chain_any(wd1, w1, wd2, w2, xd, X, bias1, shift1, relu, bias2, shift2, Y, shift2 ? BSP_I8 : BSP_I32, ws, stream);
}

bsp_status bsp_gemm_q8(const bsp_wdesc *wd, const bsp_bcsr *w, const void *X, int64_t P, const int32_t *bias,
                       const int32_t *shift, int8_t *Y, void *ws, void *stream)
{
    if (!wd) return BSP_ERR_NULL;
    if (wd->H != 1 || wd->K != 1) return BSP_ERR_SHAPE;
    if (P <= 0 || P > 0x7FFFFFFF) return BSP_ERR_SHAPE;
    bsp_xdesc xd = {(int)P, 1, 1, 1, 1, 0, 0};
    return bsp_conv2d_q8(wd, w, &xd, X, bias, shift, Y, ws, stream);
}

const char *bsp_conv_kernel_name(const bsp_wdesc *wd, const bsp_xdesc *xd)
{
    if (check_wdesc(wd) != BSP_OK || !xd) return nullptr;
    return gemm_tc_eligible(*wd, *xd, wd->wtype == BSP_I8 ? BSP_I32 : BSP_F32) ? "gemm_tc_kernel" : nullptr;
}

bsp_status bsp_gemm(const bsp_wdesc *wd, const bsp_bcsr *w, const void *X, int64_t P, const void *bias,
                    void *Y, bsp_dtype ytype, void *ws, void *stream)
{
    if (!wd) return BSP_ERR_NULL;
    if (wd->H != 1 || wd->K != 1) return BSP_ERR_SHAPE;
    if (P <= 0 || P > 0x7FFFFFFF) return BSP_ERR_SHAPE;
    bsp_xdesc xd = {(int)P, 1, 1, 1, 1, 0, 0};
    return bsp_conv2d(wd, w, &xd, X, bias, Y, ytype, ws, stream);
}

bsp_status bsp_check(void *ws, void *stream)
{
    if (!ws) return BSP_ERR_NULL;
    int h = 0;
    BSP_CUDA_OK(cudaMemcpyAsync(&h, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    BSP_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    // a latched status is cleared once read; after a timeout the grid-barrier words are cleared with it, since a
    // launch that gave up may have left arrivals behind
    if (h != 0) BSP_CUDA_OK(cudaMemsetAsync(ws, 0, h == (int)BSP_ERR_TIMEOUT ? (kWsSyncWord + 2) * sizeof(int) : sizeof(int), (cudaStream_t)stream));
    if (h < 0 || h > (int)BSP_ERR_TIMEOUT) return BSP_ERR_CUDA;
    return (bsp_status)h;
}

}  // extern "C"
