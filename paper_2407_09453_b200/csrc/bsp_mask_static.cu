// bsp_mask_static: the Gamma builder for callers that cannot hand the library any scratch memory.
// See include/bsp.h for the contract.  The block scores live in a fixed array in the library's own
// device image instead of a caller workspace.
#include "bsp_internal.cuh"

namespace {

// 65536 blocks x 8 bytes = 512 KiB, resident on every GPU that loads the library until the process exits.
constexpr long long kStaticMaxBlocks = BSP_MASK_STATIC_MAX_BLOCKS;
static __device__ __align__(256) unsigned long long g_static_scores[kStaticMaxBlocks];

constexpr int kMaxDevices = 64;
void *g_scores_ptr[kMaxDevices] = {};      // device address of g_static_scores, looked up once per device

}  // namespace

extern "C" bsp_status bsp_mask_static(const bsp_wdesc *wd, const void *W, bsp_norm norm, bsp_scope scope,
                                      int64_t n_zero, uint8_t *gamma, void *stream)
{
    const bsp_status rc = bsp::check_wdesc(wd);           // the same descriptor rules as bsp_mask()
    if (rc != BSP_OK) return rc;
    if (!W || !gamma) return BSP_ERR_NULL;
    if (((uintptr_t)W & 3u) != 0) return BSP_ERR_SHAPE;
    if (norm != BSP_NORM_L2 && norm != BSP_NORM_L1 && norm != BSP_NORM_VAR) return BSP_ERR_DTYPE;
    if (norm == BSP_NORM_VAR && wd->wtype == BSP_I8) return BSP_ERR_DTYPE;      // the variance is defined for float weights
    if (scope != BSP_SCOPE_LAYER && scope != BSP_SCOPE_ROW) return BSP_ERR_DTYPE;
    const int64_t NBi = wd->I / wd->bi, NB = (int64_t)(wd->O / wd->bo) * NBi;
    if (NB > kStaticMaxBlocks) return BSP_ERR_CAPACITY;          // layer too large for the built-in scratch
    const int64_t limit = (scope == BSP_SCOPE_LAYER) ? NB : NBi;
    if (n_zero < 0 || n_zero > limit) return BSP_ERR_CAPACITY;

    // In host code the array's name is only a handle; kernels need its address on the current device.
    int dev = 0;
    BSP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BSP_ERR_CUDA;
    if (g_scores_ptr[dev] == nullptr) {
        void *p = nullptr;
        BSP_CUDA_OK(cudaGetSymbolAddress(&p, g_static_scores));
        g_scores_ptr[dev] = p;
    }
    // every score the selection reads is rewritten by the score kernel first, so nothing needs clearing
    return bsp::launch_mask(*wd, W, norm, scope, n_zero, gamma, g_scores_ptr[dev], nullptr, (cudaStream_t)stream);
}
