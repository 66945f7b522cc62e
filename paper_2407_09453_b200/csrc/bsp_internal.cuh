// Internal declarations shared by the CUDA translation units of libbsp.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "bsp.h"

namespace bsp {

// The product kernels work on 8x8 tiles of W-bar: an 8x8 block is one tile, a 4x16 block covers half of
// two tiles side by side, a 16x4 block covers half of two tiles one above the other.  A tile is stored if
// any block overlapping it has Gamma = 1; weights of zeroed blocks inside a stored tile are written as
// zeros.  Eight tile rows (64 output channels) form a panel; one warp owns one panel.
constexpr int kTile = 8;                 // tile edge in channels
constexpr int kPanelRows = 8;            // tile rows per panel
constexpr int kPanelCh = kTile * kPanelRows;
constexpr uint32_t kPackedMagic = 0x42535031u;   // "BSP1"

// First 256 bytes of the packed buffer.
struct PackedHeader {
    uint32_t magic;
    int32_t dtype, O, I, H, K, bo, bi;
    int32_t n_panels;        // ceil(O / 64)
    int32_t n_cols;          // I / 8 tile columns
    int32_t tile_bytes;      // bytes of one stored tile (all taps)
    int32_t capacity_tiles;  // tiles the payload area can hold
    int32_t n_tiles;         // tiles stored (written on the device)
    int32_t off_colmask;     // byte offsets from the start of the packed buffer
    int32_t off_coloff;
    int32_t off_panelbase;
    int64_t off_payload;
    int64_t off_tc_payload;  // start of the super-tile payload (depends on the capacity the buffer was sized for)
    int32_t forms;           // forms written by the compaction that filled this buffer: kForm* bits
};
static_assert(sizeof(PackedHeader) <= 256, "the packed header is the first 256 bytes");

// Forms of the packed buffer (PackedHeader::forms).
constexpr int kFormTile = 1;     // 8x8 tiles in mma.sync fragment order (warp-MMA kernel)
constexpr int kFormSuper = 2;    // 16-channel super-tiles (tcgen05 convolution kernel)
constexpr int kFormDense = 4;    // Gamma (.) W-bar as a plain matrix (tcgen05 matrix-product kernel)

// Second packed form, for the tcgen05 convolution kernel (bf16 and int8): W-bar is cut into super-tiles of 16 output channels
// (a super-row) by one K-group: 8 input channels and all taps for a convolution, 16 input channels for a 1x1
// layer.  A super-tile is stored if any 8x8 tile inside it is; it holds one 512-byte tcgen05 B operand
// (16 x 16 bf16, K-major core matrices) per K-step of 16: a pair of taps, or the two 8-channel halves.
// Eight super-rows (128 channels) form a group, the N range of one CTA.
constexpr int kTcGroupRows = 8;
constexpr int kTcSuperRow = 16;
constexpr int kTcUnitBytes = 512;

struct TcLayout {
    bool enabled;
    int n_groups, n_kc, kc_ch, n_units, st_bytes;   // K-groups, channels per K-group, K-steps and bytes per super-tile
    int64_t capacity;                                // super-tiles the payload area can hold
    size_t off_mask, off_off, off_gcnt, off_payload, end;
};

// Third packed form, for the persistent tcgen05 kernel (layers of every input type): Gamma (.) W in the layout of W,
// [O][H][K][I], weights of zeroed blocks written as zeros, so that tiles of it arrive by tiled TMA loads.  A K-stage
// of the kernel is 128 bytes of the input channels of one tap (64 bf16, 128 int8, 32 fp32).
struct GemmLayout {
    bool enabled;
    int n_ks;                // K-stages: H K ceil(I * esz / 128)
    size_t off_payload, end;
};

struct PackedLayout {
    int n_panels, n_cols, tile_bytes;
    int64_t capacity_tiles;
    size_t off_colmask, off_coloff, off_panelbase, off_payload, total_bytes;
    TcLayout tc;
    GemmLayout gm;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int elem_bytes(bsp_dtype t) { return t == BSP_I8 ? 1 : (t == BSP_BF16 ? 2 : 4); }

// Bytes of one stored 8x8 tile over all H*K taps, in the order the MMA fragments are read.
inline int tile_bytes_of(bsp_dtype t, int taps)
{
    if (t == BSP_BF16) return 128 * taps;              // 8x8 bf16 per tap
    if (t == BSP_I8) return 128 * ((taps + 1) / 2);    // taps paired into K=16 steps, odd tail zero padded
    return 256 * taps;                                 // 8x8 fp32 per tap
}

PackedLayout packed_layout(const bsp_wdesc &wd, int64_t nnz_blocks);

// Workspace: the first 256 bytes hold the latched status word (word 0) and the two words of the grid-wide
// barrier of the single-launch kernels (words kWsSyncWord, kWsSyncWord + 1); scratch starts after them.
constexpr size_t kWsHeader = 256;
constexpr int kWsSyncWord = 2;
// Scratch of the cooperative select after the scores in the mask workspace: 8 x 256 histogram words and one
// word per CTA.
constexpr int kSelectMaxCtas = 1024;
constexpr size_t kSelectScratch = (8 * 256 + kSelectMaxCtas) * 4;

bsp_status launch_mask(const bsp_wdesc &wd, const void *W, bsp_norm norm, bsp_scope scope, int64_t n_zero,
                       uint8_t *gamma, void *scores, void *ws, cudaStream_t st);
bsp_status launch_compact(const bsp_wdesc &wd, const void *W, const uint8_t *gamma, int32_t *row_ptr,
                          int32_t *col_idx, void *payload, void *packed, int64_t capacity_blocks, void *ws,
                          cudaStream_t st);
bsp_status launch_count(const uint8_t *gamma, int64_t n, unsigned long long *out, cudaStream_t st);
bsp_status launch_conv(const bsp_wdesc &wd, const bsp_xdesc &xd, const void *packed, const void *X,
                       const void *bias, void *Y, bsp_dtype ytype, double density, void *ws, cudaStream_t st);

// A failed CUDA call becomes BSP_ERR_CUDA; with BSP_DEBUG set in the environment its text goes to stderr.
void report_cuda_error(cudaError_t e, const char *expr, const char *file, int line);

bool conv_tc_eligible(const bsp_wdesc &wd, const bsp_xdesc &xd);
bool gemm_tc_eligible(const bsp_wdesc &wd, const bsp_xdesc &xd, bsp_dtype ytype);
bsp_status launch_gemm_tc(const bsp_wdesc &wd, const bsp_xdesc &xd, const void *packed, const void *X,
                          const void *bias, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st);
// Output channels per CTA tile of the matrix-product kernel (a multiple of 64, at most 256).
inline int gemm_tile_n(int O)
{
    const int tiles = (O + 255) / 256;
    return (((O + tiles - 1) / tiles) + 63) / 64 * 64;
}
bsp_status launch_conv_tc(const bsp_wdesc &wd, const bsp_xdesc &xd, const void *packed, const void *X,
                          const void *bias, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st);

#define BSP_CUDA_OK(expr)                                            \
    do {                                                             \
        cudaError_t e_ = (expr);                                     \
        if (e_ != cudaSuccess) {                                     \
            bsp::report_cuda_error(e_, #expr, __FILE__, __LINE__);   \
            return BSP_ERR_CUDA;                                     \
        }                                                            \
    } while (0)

}  // namespace bsp
