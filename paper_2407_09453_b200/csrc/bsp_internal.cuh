// Internal declarations shared by the CUDA translation units of libbsp.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "bsp.h"

namespace bsp {

constexpr uint32_t kPackedMagic = 0x42535032u;   // "BSP2"

// First 256 bytes of the packed buffer, written on the device by bsp_compact and checked by the product kernel
// before it loads anything.
struct PackedHeader {
    uint32_t magic;
    int32_t dtype, O, I, H, K, bo, bi;
    int32_t forms;           // kForm* bits of what the buffer holds
    int64_t off_payload;     // byte offset of the packed weights
};
static_assert(sizeof(PackedHeader) <= 256, "the packed header is the first 256 bytes");

// The packed form: Gamma (.) W in the layout of W, [O][H][K][I], weights of zeroed blocks written as zeros, so that
// tiles of it arrive by tiled TMA loads.  A K-stage of the product kernel is 128 bytes of the input channels of one
// tap (64 bf16, 128 int8, 32 fp32).
constexpr int kFormDense = 4;

struct PackedLayout {
    bool enabled;            // rows of input channels are multiples of 16 bytes and O a multiple of 8
    size_t off_payload, total_bytes;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int elem_bytes(bsp_dtype t) { return t == BSP_I8 ? 1 : (t == BSP_BF16 ? 2 : 4); }

PackedLayout packed_layout(const bsp_wdesc &wd);

// Workspace: the first 256 bytes hold the latched status word (word 0) and the two words of the grid-wide
// barrier of the single-launch kernels (words kWsSyncWord, kWsSyncWord + 1); scratch starts after them.
constexpr size_t kWsHeader = 256;
constexpr int kWsSyncWord = 2;
// Scratch of the cooperative select after the scores in the mask workspace: 8 x 256 histogram words, 8 counter and key-span words,
// one word per CTA and a list of up to 8192 candidate keys.
constexpr int kSelectMaxCtas = 1024;
constexpr size_t kSelectScratch = (8 * 256 + 8 + kSelectMaxCtas) * 4 + 8192 * 8;

// Host-side validation of a weight descriptor, shared by every entry point.
bsp_status check_wdesc(const bsp_wdesc *wd);

bsp_status launch_mask(const bsp_wdesc &wd, const void *W, bsp_norm norm, bsp_scope scope, int64_t n_zero,
                       uint8_t *gamma, void *scores, void *ws, cudaStream_t st);
bsp_status launch_compact(const bsp_wdesc &wd, const void *W, const uint8_t *gamma, int32_t *row_ptr,
                          int32_t *col_idx, void *payload, void *packed, int64_t capacity_blocks, void *ws,
                          cudaStream_t st);
bsp_status launch_count(const uint8_t *gamma, int64_t n, unsigned long long *out, cudaStream_t st);

// A failed CUDA call becomes BSP_ERR_CUDA; with BSP_DEBUG set in the environment its text goes to stderr.
void report_cuda_error(cudaError_t e, const char *expr, const char *file, int line);

bool gemm_tc_eligible(const bsp_wdesc &wd, const bsp_xdesc &xd, bsp_dtype ytype);
bool chain_tc_eligible(const bsp_wdesc &wd1, const bsp_wdesc &wd2, const bsp_xdesc &xd, bsp_dtype ytype);
bsp_status launch_chain_tc(const bsp_wdesc &wd1, const void *packed1, const bsp_wdesc &wd2, const void *packed2,
                           const bsp_xdesc &xd, const void *X, const void *bias1, const int32_t *shift1, int relu,
                           const void *bias2, const int32_t *shift2, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st);
bsp_status launch_gemm_tc(const bsp_wdesc &wd, const bsp_xdesc &xd, const void *packed, const void *X,
                          const void *bias, const int32_t *shift, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st);
// Output channels per CTA tile of the product kernel (a multiple of 64, at most 256).
inline int gemm_tile_n(int O)
{
    const int tiles = (O + 255) / 256;
    return (((O + tiles - 1) / tiles) + 63) / 64 * 64;
}

#define BSP_CUDA_OK(expr)                                            \
    do {                                                             \
        cudaError_t e_ = (expr);                                     \
        if (e_ != cudaSuccess) {                                     \
            bsp::report_cuda_error(e_, #expr, __FILE__, __LINE__);   \
            return BSP_ERR_CUDA;                                     \
        }                                                            \
    } while (0)

}  // namespace bsp
