// Block-sparse implicit-GEMM convolution / FC product with fused bias: TMA-fed, warp-specialised, warp-level
// tensor-core MMAs.  Introduction (Y = W*X + b) and Section "Block Sparsity in a Matrix" of the paper: only
// stored 8x8 tiles of W-bar are read and multiplied.
//
// Orientation: output pixels are the MMA M dimension, the 8 output channels of a tile row are N, input
// channels (times taps) are K.  A CTA owns a tile of output pixels (nb images x th rows x tw columns) and
// WN panels of 64 output channels; consumer warp (wm, wn) accumulates 64 pixels x 64 channels in registers.
//
// One producer warp feeds two rings of shared-memory stages.  An activation stage holds a 128-byte slab of
// channels (64 bf16, 128 int8 or 32 fp32 channels) of the input patch of the pixel tile: one tiled TMA load
// with 128-byte swizzle, whose out-of-bounds fill supplies the zero padding; rows are patch pixels, so a tap
// is a constant row offset and the swizzle keeps the 8-row fragment loads free of bank conflicts.  A weight
// stage holds, for each of the CTA's panels, the stored tiles of GCW tile columns (8 input channels each),
// which are one contiguous stretch of the packed payload and arrive by one bulk copy.  Loads complete on
// "full" mbarriers; consumer warps release stages through "empty" mbarriers.  The panels' tile masks and
// offsets are copied to shared memory once.  For every tile column a consumer warp loads the activation
// fragments once per K-step and issues MMAs only for the tile rows present in the column's row mask: the mask
// selects, by a warp-uniform jump, straight-line code holding exactly those MMAs.
// Every mbarrier wait is bounded: on expiry the warp latches BSP_ERR_TIMEOUT in the workspace and leaves.
#include <cuda.h>
#include <cstdlib>
#include "bsp_internal.cuh"

namespace bsp {
namespace {

constexpr int kMaxTaps = 128;
constexpr int kMaxSmem = 200 * 1024;      // ceiling of the carved-up shared memory of a launch (+1 KB slack)
constexpr int kMaxDevices = 64;
constexpr int kMaxWStages = 8;            // weight ring depth
constexpr int kMaxAStages = 3;            // activation ring depth
constexpr int kWStageBudget = 16 * 1024;  // target bytes of one weight stage
constexpr int kSlabBytes = 128;           // channel bytes per activation slab row (the TMA swizzle span)
constexpr int kEpiBytes = 16 * (kPanelCh * 4 + 16);   // per-warp epilogue staging: 16 pixels x 64 channels
constexpr uint32_t kSpinLimit = 1u << 22; // bounded mbarrier wait: try_wait attempts before giving up

struct ConvParams {
    CUtensorMap tmap;   // activations: (channel group bytes, x, y, n, group)
    uint8_t *Y;
    const void *bias;
    const uint8_t *colmask;
    const uint32_t *coloff;
    const uint32_t *panel_base;
    const uint8_t *payload;
    int *status;
    int N, L, J, I, O, M, Nw, H, K, sh, sw, ph, pw;
    int nb, th, tw, PH, PW, patch_pix, tile_pix;
    int tiles_x, tiles_y;
    int n_cols, n_panels, tile_bytes;
    int slab_cols, n_slabs, a_stages, a_stage_bytes, a_box_bytes;   // activation ring
    int GCW, w_stages, w_stage_bytes, wseg_cap;                     // weight ring: wseg_cap bytes per panel
    int meta_bytes, a_ring_off, w_ring_off, epi_off;                // byte offsets in dynamic shared memory
    int ytype;
};

// CB: bytes of one tile column (8 channels) inside a 128-byte slab row.
template <int DT> struct Traits;
template <> struct Traits<BSP_BF16> { static constexpr int CB = 16; using acc_t = float; };
template <> struct Traits<BSP_I8> { static constexpr int CB = 8; using acc_t = int; };
template <> struct Traits<BSP_F32> { static constexpr int CB = 32; using acc_t = float; };

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
// Waits for the phase with the given parity; false if the bounded spin ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        uint32_t done;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

__device__ __forceinline__ void mma_bf16_k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_k8(float (&c)[4], const uint32_t (&a)[4], uint32_t b0)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b0));
}
__device__ __forceinline__ void mma_s8_k16(int (&c)[4], const uint32_t (&a)[4], uint32_t b0)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b0));
}
__device__ __forceinline__ void mma_tf32_k8(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t to_tf32(uint32_t fbits)
{
    uint32_t r;
    asm volatile("cvt.rna.tf32.f32 %0, %1;\n" : "=r"(r) : "f"(__uint_as_float(fbits)));
    return r;
}

// Row, in the staged patch, of the top-left input pixel of output pixel q of the CTA's tile (q counts images,
// then rows, then columns of the tile).  Pixels past the tile map to row 0.
__device__ __forceinline__ int patch_row(const ConvParams &p, int q)
{
    if (q >= p.tile_pix) return 0;
    const int ix = q % p.tw;
    const int t = q / p.tw;
    const int iy = t % p.th;
    const int in = t / p.th;
    return (in * p.PH + iy * p.sh) * p.PW + ix * p.sw;
}

// Shared-memory address of 16-byte chunk `chunk` of patch row `row` in a 128-byte-swizzled slab stage
// (1024-byte aligned): the chunk index is XORed with the row index modulo 8.
__device__ __forceinline__ uint32_t slab_addr(uint32_t stage, int row, int chunk)
{
    return stage + (uint32_t)row * kSlabBytes + (uint32_t)((chunk ^ (row & 7)) << 4);
}


// ---- MMAs of the stored tiles of one K-step (general kernel shapes) -----------------------------------------
// KIND: 0 bf16 k16 (two taps), 1 bf16 k8 (odd last tap), 2 int8 k16, 3 tf32 k8.
// The tile rows present in a tile column are known only at run time, but accumulators must be indexed
// statically.  The 8-bit row mask is therefore split into two nibbles and each nibble value jumps (a
// warp-uniform switch) to straight-line code holding exactly the MMAs of its set rows: absent tiles cost no
// issue slot.  Stored tiles follow each other in row order, so the weight pointer just advances.
template <int KIND, int kMT, int R, typename acc_t>
__device__ __forceinline__ void tile_mma(acc_t (&acc)[kMT][kPanelRows][4], const uint32_t (&a)[kMT][4], uint32_t &wp,
                                         int tile_bytes)
{
    if constexpr (KIND == 0) {
        const uint2 b = lds64(wp);
#pragma unroll
        for (int i = 0; i < kMT; ++i) mma_bf16_k16(acc[i][R], a[i], b.x, b.y);
    } else if constexpr (KIND == 1) {
        const uint32_t b = lds32(wp);
#pragma unroll
        for (int i = 0; i < kMT; ++i) mma_bf16_k8(acc[i][R], a[i], b);
    } else if constexpr (KIND == 2) {
        const uint32_t b = lds32(wp);
#pragma unroll
        for (int i = 0; i < kMT; ++i) mma_s8_k16(acc[i][R], a[i], b);
    } else {
        const uint2 b = lds64(wp);
        const uint32_t b0 = to_tf32(b.x), b1 = to_tf32(b.y);
#pragma unroll
        for (int i = 0; i < kMT; ++i) mma_tf32_k8(acc[i][R], a[i], b0, b1);
    }
    wp += tile_bytes;
}

template <int KIND, int kMT, int NIB, int BASE, typename acc_t>
__device__ __forceinline__ void nibble_mma(acc_t (&acc)[kMT][kPanelRows][4], const uint32_t (&a)[kMT][4], uint32_t &wp,
                                           int tile_bytes)
{
    if constexpr ((NIB & 1) != 0) tile_mma<KIND, kMT, BASE + 0>(acc, a, wp, tile_bytes);
    if constexpr ((NIB & 2) != 0) tile_mma<KIND, kMT, BASE + 1>(acc, a, wp, tile_bytes);
    if constexpr ((NIB & 4) != 0) tile_mma<KIND, kMT, BASE + 2>(acc, a, wp, tile_bytes);
    if constexpr ((NIB & 8) != 0) tile_mma<KIND, kMT, BASE + 3>(acc, a, wp, tile_bytes);
}

#define BSP_NIBBLE_SWITCH(FN, ...)                       \
    switch (nib) {                                       \
        case 1: FN<__VA_ARGS__, 1, BASE> ARGS; break;    \
        case 2: FN<__VA_ARGS__, 2, BASE> ARGS; break;    \
        case 3: FN<__VA_ARGS__, 3, BASE> ARGS; break;    \
        case 4: FN<__VA_ARGS__, 4, BASE> ARGS; break;    \
        case 5: FN<__VA_ARGS__, 5, BASE> ARGS; break;    \
        case 6: FN<__VA_ARGS__, 6, BASE> ARGS; break;    \
        case 7: FN<__VA_ARGS__, 7, BASE> ARGS; break;    \
        case 8: FN<__VA_ARGS__, 8, BASE> ARGS; break;    \
        case 9: FN<__VA_ARGS__, 9, BASE> ARGS; break;    \
        case 10: FN<__VA_ARGS__, 10, BASE> ARGS; break;  \
        case 11: FN<__VA_ARGS__, 11, BASE> ARGS; break;  \
        case 12: FN<__VA_ARGS__, 12, BASE> ARGS; break;  \
        case 13: FN<__VA_ARGS__, 13, BASE> ARGS; break;  \
        case 14: FN<__VA_ARGS__, 14, BASE> ARGS; break;  \
        case 15: FN<__VA_ARGS__, 15, BASE> ARGS; break;  \
        default: break;                                  \
    }

template <int KIND, int kMT, int BASE, typename acc_t>
__device__ __forceinline__ void rows_mma(uint32_t nib, acc_t (&acc)[kMT][kPanelRows][4], const uint32_t (&a)[kMT][4],
                                         uint32_t &wp, int tile_bytes)
{
#define ARGS (acc, a, wp, tile_bytes)
    BSP_NIBBLE_SWITCH(nibble_mma, KIND, kMT)
#undef ARGS
}

template <int KIND, int kMT, typename acc_t>
__device__ __forceinline__ void step_mma(uint32_t m, acc_t (&acc)[kMT][kPanelRows][4], const uint32_t (&a)[kMT][4],
                                         uint32_t wp, int tile_bytes)
{
    rows_mma<KIND, kMT, 0>(m & 15u, acc, a, wp, tile_bytes);
    rows_mma<KIND, kMT, 4>(m >> 4, acc, a, wp, tile_bytes);
}

// ---- Columns with a compile-time tap count (1x1 and 3x3 kernels) -------------------------------------------
// With HKT = H*K known, the K-steps of a tile column are unrolled: all activation fragments of the column are
// loaded first (one exposed shared-memory latency per column instead of one per step), the row-mask dispatch
// happens once per column and nibble instead of once per step, and every weight fragment sits at a constant
// offset from the column's first stored tile.
template <int DT, int HKT> struct Steps;
template <int HKT> struct Steps<BSP_BF16, HKT> { static constexpr int N16 = HKT / 2, TAIL = HKT & 1, N = N16 + TAIL; };
template <int HKT> struct Steps<BSP_I8, HKT> { static constexpr int N16 = (HKT + 1) / 2, TAIL = 0, N = N16; };

template <int DT, int HKT, int kMT, int R, typename acc_t>
__device__ __forceinline__ void col_tile(acc_t (&acc)[kMT][kPanelRows][4],
                                         const uint32_t (&a)[Steps<DT, HKT>::N][kMT][4], uint32_t wt, int lane)
{
    using S = Steps<DT, HKT>;
    if constexpr (DT == BSP_BF16) {
        uint2 b[S::N16 > 0 ? S::N16 : 1];
#pragma unroll
        for (int st = 0; st < S::N16; ++st) b[st] = lds64(wt + st * 256 + lane * 8);
        uint32_t bt = 0;
        if constexpr (S::TAIL != 0) bt = lds32(wt + S::N16 * 256 + lane * 4);
#pragma unroll
        for (int st = 0; st < S::N16; ++st)
#pragma unroll
            for (int i = 0; i < kMT; ++i) mma_bf16_k16(acc[i][R], a[st][i], b[st].x, b[st].y);
        if constexpr (S::TAIL != 0) {
#pragma unroll
            for (int i = 0; i < kMT; ++i) mma_bf16_k8(acc[i][R], a[S::N16][i], bt);
        }
    } else {
        uint32_t b[S::N16];
#pragma unroll
        for (int st = 0; st < S::N16; ++st) b[st] = lds32(wt + st * 128 + lane * 4);
#pragma unroll
        for (int st = 0; st < S::N16; ++st)
#pragma unroll
            for (int i = 0; i < kMT; ++i) mma_s8_k16(acc[i][R], a[st][i], b[st]);
    }
}

template <int DT, int HKT, int kMT, int NIB, int BASE, typename acc_t>
__device__ __forceinline__ void col_nibble(acc_t (&acc)[kMT][kPanelRows][4],
                                           const uint32_t (&a)[Steps<DT, HKT>::N][kMT][4], uint32_t wt, int lane)
{
    constexpr int TB = (DT == BSP_BF16) ? 128 * HKT : 128 * ((HKT + 1) / 2);      // bytes of one stored tile
    constexpr int r1 = (NIB & 1), r2 = r1 + ((NIB >> 1) & 1), r3 = r2 + ((NIB >> 2) & 1);
    if constexpr ((NIB & 1) != 0) col_tile<DT, HKT, kMT, BASE + 0>(acc, a, wt, lane);
    if constexpr ((NIB & 2) != 0) col_tile<DT, HKT, kMT, BASE + 1>(acc, a, wt + r1 * TB, lane);
    if constexpr ((NIB & 4) != 0) col_tile<DT, HKT, kMT, BASE + 2>(acc, a, wt + r2 * TB, lane);
    if constexpr ((NIB & 8) != 0) col_tile<DT, HKT, kMT, BASE + 3>(acc, a, wt + r3 * TB, lane);
}

template <int DT, int HKT, int kMT, int BASE, typename acc_t>
__device__ __forceinline__ void col_rows(uint32_t nib, acc_t (&acc)[kMT][kPanelRows][4],
                                         const uint32_t (&a)[Steps<DT, HKT>::N][kMT][4], uint32_t wt, int lane)
{
#define ARGS (acc, a, wt, lane)
    BSP_NIBBLE_SWITCH(col_nibble, DT, HKT, kMT)
#undef ARGS
}

// Threads: WM*WN consumer warps, then one producer warp.  kMT = 16-pixel MMA tiles per consumer warp (a warp
// owns 16*kMT pixels x 64 channels); the smaller warp tile halves the registers so that more warps share an SM.
// HKT = H*K when it is 1 (1x1) or 9 (3x3) and the unrolled column code is used, else 0 (any kernel shape).
template <int DT, int kMT, int WM, int WN, int HKT>
__global__ void __launch_bounds__(32 * (WM * WN + 1), (kMT == 2 && WM * WN <= 4) ? 3 : ((kMT == 2 && HKT != 9) ? 2 : 1))
conv_mma_kernel(const __grid_constant__ ConvParams p)
{
    using T = Traits<DT>;
    using acc_t = typename T::acc_t;
    constexpr int CB = T::CB;
    constexpr int NCW = WM * WN;                 // consumer warps
    constexpr int NT = 32 * (NCW + 1);
    extern __shared__ __align__(16) uint8_t smem_raw[];
    // the swizzled activation stages need 1024-byte alignment; the launch reserves the slack
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ int s_taprow[kMaxTaps];           // patch-row offset of every tap
    __shared__ __align__(8) uint64_t s_afull[kMaxAStages];
    __shared__ __align__(8) uint64_t s_aempty[kMaxAStages];
    __shared__ __align__(8) uint64_t s_wfull[kMaxWStages];
    __shared__ __align__(8) uint64_t s_wempty[kMaxWStages];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int HK = p.H * p.K;
    const int SA = p.a_stages, SW = p.w_stages;

    // tile origin
    int tix = blockIdx.x;
    const int tx = tix % p.tiles_x; tix /= p.tiles_x;
    const int ty = tix % p.tiles_y;
    const int tn = tix / p.tiles_y;
    const int n0 = tn * p.nb, y0 = ty * p.th, x0 = tx * p.tw;

    for (int t = tid; t < kMaxTaps; t += NT) {
        const int tt = t < HK ? t : HK - 1;
        s_taprow[t] = (tt / p.K) * p.PW + (tt % p.K);
    }
    // tile offsets (with an end sentinel) and masks of the CTA's panels -> shared memory
    uint32_t *s_coloff = (uint32_t *)smem;                                   // [WN][n_cols + 1]
    uint8_t *s_mask = smem + (size_t)WN * (p.n_cols + 1) * 4;                // [WN][n_cols]
    for (int i = tid; i < WN * (p.n_cols + 1); i += NT) {
        const int pn = i / (p.n_cols + 1), col = i % (p.n_cols + 1);
        const int pg = blockIdx.y * WN + pn;
        uint32_t v = 0;
        if (pg < p.n_panels)
            v = (col < p.n_cols) ? p.coloff[(size_t)pg * p.n_cols + col] : p.panel_base[pg + 1] - p.panel_base[pg];
        s_coloff[i] = v;
    }
    for (int i = tid; i < WN * p.n_cols; i += NT) {
        const int pg = blockIdx.y * WN + i / p.n_cols;
        s_mask[i] = (pg < p.n_panels) ? p.colmask[(size_t)pg * p.n_cols + i % p.n_cols] : (uint8_t)0;
    }
    if (tid == 0) {
        for (int s = 0; s < SA; ++s) {
            mbar_init(smem_u32(&s_afull[s]), 1);
            mbar_init(smem_u32(&s_aempty[s]), NCW);
        }
        for (int s = 0; s < SW; ++s) {
            mbar_init(smem_u32(&s_wfull[s]), 1);
            mbar_init(smem_u32(&s_wempty[s]), NCW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();

    const uint32_t a_ring = smem_u32(smem) + p.a_ring_off;
    const uint32_t w_ring = smem_u32(smem) + p.w_ring_off;

    if (warp == NCW) {
        // ================= producer warp: one lane issues every copy =================
        if (lane == 0) {
            const int gx0 = x0 * p.sw - p.pw, gy0 = y0 * p.sh - p.ph;
            bool ok = true;
            auto issue_act = [&](int s) {
                if (s >= p.n_slabs || !ok) return;
                const int sa = s % SA;
                if (s >= SA && !mbar_wait(smem_u32(&s_aempty[sa]), (uint32_t)((s / SA - 1) & 1))) { ok = false; return; }
                const uint32_t bar = smem_u32(&s_afull[sa]);
                mbar_expect_tx(bar, (uint32_t)p.a_box_bytes);
                tma_load_4d(a_ring + sa * p.a_stage_bytes, &p.tmap, bar, s * kSlabBytes, gx0, gy0, n0);
            };
            issue_act(0);
            uint32_t pbase[WN];                                  // first stored tile of each of the CTA's panels
#pragma unroll
            for (int pn = 0; pn < WN; ++pn) {
                const int pg = blockIdx.y * WN + pn;
                pbase[pn] = pg < p.n_panels ? p.panel_base[pg] : 0u;
            }
            int wc = 0;
            for (int s = 0; s < p.n_slabs && ok; ++s) {
                issue_act(s + 1);
                const int slab_end = min(p.n_cols, (s + 1) * p.slab_cols);
                for (int col0 = s * p.slab_cols; col0 < slab_end && ok; col0 += p.GCW, ++wc) {
                    const int sw = wc % SW;
                    if (wc >= SW && !mbar_wait(smem_u32(&s_wempty[sw]), (uint32_t)((wc / SW - 1) & 1))) { ok = false; break; }
                    const int ncol = min(p.GCW, slab_end - col0);
                    const uint32_t bar = smem_u32(&s_wfull[sw]);
                    uint32_t tx_bytes = 0;
                    for (int pn = 0; pn < WN; ++pn)
                        tx_bytes += (s_coloff[pn * (p.n_cols + 1) + col0 + ncol] - s_coloff[pn * (p.n_cols + 1) + col0]) *
                                    (uint32_t)p.tile_bytes;
                    mbar_expect_tx(bar, tx_bytes);
#pragma unroll
                    for (int pn = 0; pn < WN; ++pn) {
                        const uint32_t first = s_coloff[pn * (p.n_cols + 1) + col0];
                        const uint32_t bytes = (s_coloff[pn * (p.n_cols + 1) + col0 + ncol] - first) * (uint32_t)p.tile_bytes;
                        if (bytes)      // panels past the last one have no stored tiles
                            bulk_load(w_ring + sw * p.w_stage_bytes + pn * p.wseg_cap,
                                      p.payload + (size_t)(pbase[pn] + first) * p.tile_bytes, bytes, bar);
                    }
                }
            }
            if (!ok) atomicMax(p.status, (int)BSP_ERR_TIMEOUT);
        }
        return;
    }

    // ================= consumer warps =================
    const int wm = warp % WM, wn = warp / WM;
    const int panel = blockIdx.y * WN + wn;
    const bool active = panel < p.n_panels;

    int rowpix[kMT][2];
#pragma unroll
    for (int i = 0; i < kMT; ++i) {
        const int qbase = (wm * kMT + i) * 16;
        if constexpr (DT == BSP_BF16) {
            rowpix[i][0] = patch_row(p, qbase + (lane & 15));
            rowpix[i][1] = 0;
        } else {
            rowpix[i][0] = patch_row(p, qbase + (lane >> 2));
            rowpix[i][1] = patch_row(p, qbase + (lane >> 2) + 8);
        }
    }

    acc_t acc[kMT][kPanelRows][4];
#pragma unroll
    for (int i = 0; i < kMT; ++i)
#pragma unroll
        for (int r = 0; r < kPanelRows; ++r)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][r][e] = 0;

    const uint32_t *my_off = s_coloff + wn * (p.n_cols + 1);
    const uint8_t *my_mask = s_mask + wn * p.n_cols;
    bool ok = true;
    int wc = 0;

    for (int s = 0; s < p.n_slabs && ok; ++s) {
        const int sa = s % SA;
        if (!mbar_wait(smem_u32(&s_afull[sa]), (uint32_t)((s / SA) & 1))) { ok = false; break; }
        const uint32_t a_stage = a_ring + sa * p.a_stage_bytes;
        const int slab_col0 = s * p.slab_cols;
        const int slab_end = min(p.n_cols, slab_col0 + p.slab_cols);
        for (int col0 = slab_col0; col0 < slab_end; col0 += p.GCW, ++wc) {
            const int sw = wc % SW;
            if (!mbar_wait(smem_u32(&s_wfull[sw]), (uint32_t)((wc / SW) & 1))) { ok = false; break; }
            const int ncol = min(p.GCW, slab_end - col0);
            const uint32_t wseg = w_ring + sw * p.w_stage_bytes + wn * p.wseg_cap;
            const uint32_t off0 = my_off[col0];
            for (int v = 0; active && v < ncol; ++v) {
                const uint32_t m = my_mask[col0 + v];
                if (m == 0) continue;
                const uint32_t wt = wseg + (my_off[col0 + v] - off0) * p.tile_bytes;
                const int cbyte = (col0 + v - slab_col0) * CB;     // byte of the tile column inside a slab row
                const int chunk = cbyte >> 4;

                if constexpr (HKT != 0 && DT != BSP_F32) {
                    using S = Steps<DT, HKT>;
                    constexpr int KT = (HKT == 9) ? 3 : 1;          // kernel width of the specialised shapes
                    constexpr int TB = (DT == BSP_BF16) ? 128 * HKT : 128 * ((HKT + 1) / 2);
                    uint32_t a[S::N][kMT][4];
                    if constexpr (DT == BSP_BF16) {
                        const int sel = lane >> 4;
#pragma unroll
                        for (int st = 0; st < S::N16; ++st) {
                            const int tap = 2 * st + sel;
                            const int trow = (tap / KT) * p.PW + tap % KT;
#pragma unroll
                            for (int i = 0; i < kMT; ++i) ldmatrix_x4(slab_addr(a_stage, rowpix[i][0] + trow, chunk), a[st][i]);
                        }
                        if constexpr (S::TAIL != 0) {
                            const int trow = ((HKT - 1) / KT) * p.PW + (HKT - 1) % KT;
#pragma unroll
                            for (int i = 0; i < kMT; ++i) ldmatrix_x2(slab_addr(a_stage, rowpix[i][0] + trow, chunk), a[S::N16][i]);
                        }
                    } else {
                        const int t = lane & 3;
                        const int within = (cbyte & 15) + (t & 1) * 4;
#pragma unroll
                        for (int st = 0; st < S::N16; ++st) {
                            int tap = 2 * st + (t >> 1);
                            if (tap >= HKT) tap = HKT - 1;          // the zero-padded half of an odd last step
                            const int trow = (tap / KT) * p.PW + tap % KT;
#pragma unroll
                            for (int i = 0; i < kMT; ++i) {
                                a[st][i][0] = lds32(slab_addr(a_stage, rowpix[i][0] + trow, chunk) + within);
                                a[st][i][1] = lds32(slab_addr(a_stage, rowpix[i][1] + trow, chunk) + within);
                            }
                        }
                    }
                    col_rows<DT, HKT, kMT, 0>(m & 15u, acc, a, wt, lane);
                    col_rows<DT, HKT, kMT, 4>(m >> 4, acc, a, wt + __popc(m & 15u) * TB, lane);
                } else if constexpr (DT == BSP_BF16) {
                    const int n16 = HK >> 1;
                    const int sel = lane >> 4;
                    for (int st = 0; st < n16; ++st) {
                        uint32_t a[kMT][4];
                        const int trow = s_taprow[2 * st + sel];
#pragma unroll
                        for (int i = 0; i < kMT; ++i) ldmatrix_x4(slab_addr(a_stage, rowpix[i][0] + trow, chunk), a[i]);
                        step_mma<0, kMT>(m, acc, a, wt + st * 256 + lane * 8, p.tile_bytes);
                    }
                    if (HK & 1) {
                        uint32_t a[kMT][4];
                        const int trow = s_taprow[HK - 1];
#pragma unroll
                        for (int i = 0; i < kMT; ++i) ldmatrix_x2(slab_addr(a_stage, rowpix[i][0] + trow, chunk), a[i]);
                        step_mma<1, kMT>(m, acc, a, wt + n16 * 256 + lane * 4, p.tile_bytes);
                    }
                } else if constexpr (DT == BSP_I8) {
                    const int nsteps = (HK + 1) >> 1;
                    const int t = lane & 3;
                    const int within = (cbyte & 15) + (t & 1) * 4;
                    for (int st = 0; st < nsteps; ++st) {
                        uint32_t a[kMT][4];
                        const int trow = s_taprow[2 * st + (t >> 1)];
#pragma unroll
                        for (int i = 0; i < kMT; ++i) {
                            a[i][0] = lds32(slab_addr(a_stage, rowpix[i][0] + trow, chunk) + within);
                            a[i][1] = lds32(slab_addr(a_stage, rowpix[i][1] + trow, chunk) + within);
                        }
                        step_mma<2, kMT>(m, acc, a, wt + st * 128 + lane * 4, p.tile_bytes);
                    }
                } else {
                    const int t = lane & 3;
                    for (int st = 0; st < HK; ++st) {
                        uint32_t a[kMT][4];
                        const int trow = s_taprow[st];
#pragma unroll
                        for (int i = 0; i < kMT; ++i) {
                            a[i][0] = to_tf32(lds32(slab_addr(a_stage, rowpix[i][0] + trow, chunk) + t * 4));
                            a[i][1] = to_tf32(lds32(slab_addr(a_stage, rowpix[i][1] + trow, chunk) + t * 4));
                            a[i][2] = to_tf32(lds32(slab_addr(a_stage, rowpix[i][0] + trow, chunk + 1) + t * 4));
                            a[i][3] = to_tf32(lds32(slab_addr(a_stage, rowpix[i][1] + trow, chunk + 1) + t * 4));
                        }
                        step_mma<3, kMT>(m, acc, a, wt + st * 256 + lane * 8, p.tile_bytes);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_wempty[sw]));
        }
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(smem_u32(&s_aempty[sa]));
    }
    if (!ok) {
        if (lane == 0) atomicMax(p.status, (int)BSP_ERR_TIMEOUT);
        return;
    }
    if (!active) return;

    // ---- epilogue: + bias, convert, stage 16 pixels x 64 channels per warp in shared memory, store rows
    const int oe = (p.ytype == BSP_BF16) ? 2 : 4;               // bytes per output element
    const int pitch = kPanelCh * oe + 16;
    uint8_t *ebuf = smem + p.epi_off + warp * kEpiBytes;
    const int g = lane >> 2, t = lane & 3;
    const int ch0 = panel * kPanelCh;
    acc_t bv[kPanelRows][2];
#pragma unroll
    for (int r = 0; r < kPanelRows; ++r) {
        const int o = ch0 + r * 8 + 2 * t;
        bv[r][0] = 0; bv[r][1] = 0;
        if (p.bias != nullptr && o < p.O) {
            bv[r][0] = ((const acc_t *)p.bias)[o];
            bv[r][1] = ((const acc_t *)p.bias)[o + 1];
        }
    }
    const int cpr = kPanelCh * oe / 16;                      // 16-byte chunks per pixel row
#pragma unroll
    for (int i = 0; i < kMT; ++i) {
#pragma unroll
        for (int r = 0; r < kPanelRows; ++r) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const acc_t v0 = acc[i][r][2 * hh] + bv[r][0];
                const acc_t v1 = acc[i][r][2 * hh + 1] + bv[r][1];
                uint8_t *dst = ebuf + (g + 8 * hh) * pitch + (r * 8 + 2 * t) * oe;
                if constexpr (DT == BSP_I8) {
                    *(int2 *)dst = make_int2(v0, v1);
                } else {
                    if (oe == 2) *(__nv_bfloat162 *)dst = __floats2bfloat162_rn(v0, v1);
                    else *(float2 *)dst = make_float2(v0, v1);
                }
            }
        }
        __syncwarp();
        for (int idx = lane; idx < 16 * cpr; idx += 32) {
            const int row = idx / cpr, chunk = idx % cpr;
            const int q = (wm * kMT + i) * 16 + row;
            const int o = ch0 + chunk * (16 / oe);
            if (q < p.tile_pix && o < p.O) {
                const int ix = q % p.tw;
                const int tq = q / p.tw;
                const int iy = tq % p.th;
                const int in = tq / p.th;
                const int n = n0 + in, y = y0 + iy, x = x0 + ix;
                if (n < p.N && y < p.M && x < p.Nw) {
                    const size_t pix = ((size_t)n * p.M + y) * p.Nw + x;
                    *(uint4 *)(p.Y + (pix * p.O + o) * oe) = *(const uint4 *)(ebuf + row * pitch + chunk * 16);
                }
            }
        }
        __syncwarp();
    }
}

struct Plan {
    int MT, WM, WN, nb, th, tw;
    int slab_cols, n_slabs, a_stages, GCW, w_stages;
    size_t smem, a_stage_bytes, a_box_bytes, w_stage_bytes, wseg_cap, meta_bytes, a_ring_off, w_ring_off, epi_off;
    long long tiles, ctas;
};

// Launch shapes: {kMT, WM, WN, CTAs per SM the shape is compiled for}.
constexpr int kConfigs[][4] = {
    {2, 2, 2, 3}, {2, 4, 1, 3}, {2, 1, 4, 3}, {2, 4, 2, 2}, {2, 8, 1, 2}, {2, 2, 4, 2},
    {4, 2, 2, 1}, {4, 4, 2, 1}, {4, 2, 4, 1},
};

// Output-pixel tile (nb images x th x tw) of at most tpix pixels that needs the fewest tiles; box extents of
// the TMA load are limited to 256 per dimension.
void best_tile(int tpix, int N, int M, int Nw, int sh, int sw, int H, int K, int &nb, int &th, int &tw,
               long long &tiles)
{
    long long best = -1, best_area = 0;
    for (int w = 1; w <= Nw && w <= tpix; ++w) {
        if ((w - 1) * sw + K > 256) break;
        const int hmax = tpix / w < M ? tpix / w : M;
        for (int h = 1; h <= hmax; ++h) {
            if ((h - 1) * sh + H > 256) break;
            int b = 1;
            if (h == M && w == Nw) { b = tpix / (h * w); if (b > N) b = N; if (b > 256) b = 256; if (b < 1) b = 1; }
            const long long cnt = (long long)((N + b - 1) / b) * ((M + h - 1) / h) * ((Nw + w - 1) / w);
            const long long area = (long long)b * h * w;
            if (best < 0 || cnt < best || (cnt == best && area < best_area)) {
                best = cnt; best_area = area; nb = b; th = h; tw = w;
            }
        }
    }
    tiles = best;
}

// Picks the launch shape with the lowest estimated time: the slower of a per-SM issue/tensor-pipe estimate
// and the L2-to-SM traffic (every CTA re-reads its patch and its panels' stored tiles).
Plan make_plan(const bsp_wdesc &wd, const bsp_xdesc &xd, int M, int Nw, int n_panels, int n_cols, double density)
{
    const int CB = 8 * elem_bytes(wd.wtype);
    const int HK = wd.H * wd.K;
    const int tile_bytes = tile_bytes_of(wd.wtype, HK);
    const int steps = wd.wtype == BSP_F32 ? HK : (HK + 1) / 2;
    Plan best = {};
    double best_cost = -1;
    // Each shape is tried with its full pixel tile first; if nothing fits in shared memory (large strides or
    // kernels) the pixel tiles are halved, leaving some MMA rows idle.
    for (int shrink = 1; shrink <= 16 && best_cost < 0; shrink *= 2)
    for (auto &cfg : kConfigs) {
        Plan pl = {};
        pl.MT = cfg[0]; pl.WM = cfg[1]; pl.WN = cfg[2];
        int occ = cfg[3];
        size_t cap = (size_t)kMaxSmem / occ - (occ > 1 ? 2048 : 0);
        pl.tiles = -1;
        const int tpix = pl.WM * pl.MT * 16 / shrink;
        if (tpix < 8) continue;
        best_tile(tpix, xd.N, M, Nw, xd.stride_h, xd.stride_w, wd.H, wd.K, pl.nb, pl.th, pl.tw, pl.tiles);
        if (pl.tiles < 0) continue;
        const int PH = (pl.th - 1) * xd.stride_h + wd.H, PW = (pl.tw - 1) * xd.stride_w + wd.K;
        const long long patch_pix = (long long)pl.nb * PH * PW;
        pl.slab_cols = kSlabBytes / CB;
        pl.n_slabs = (n_cols + pl.slab_cols - 1) / pl.slab_cols;
        pl.a_box_bytes = (size_t)patch_pix * kSlabBytes;
        pl.a_stage_bytes = align_up(pl.a_box_bytes, 1024);
        const long long per_col = (long long)pl.WN * kPanelRows * tile_bytes;
        int GCW = (int)(kWStageBudget / per_col);
        if (GCW > pl.slab_cols) GCW = pl.slab_cols;
        if (GCW < 1) GCW = 1;
        pl.GCW = GCW;
        pl.wseg_cap = (size_t)GCW * kPanelRows * tile_bytes;
        pl.w_stage_bytes = pl.WN * pl.wseg_cap;
        pl.meta_bytes = align_up((size_t)pl.WN * (n_cols + 1) * 4 + (size_t)pl.WN * n_cols, 1024);
        const size_t epi = (size_t)pl.WM * pl.WN * kEpiBytes;
        const size_t fixed = pl.meta_bytes + epi + 1024;          // + slack for aligning the base to 1024 bytes
        // at least two stages in each ring; give up co-residency before giving up the shape
        while (occ > 1 && fixed + 2 * pl.a_stage_bytes + 2 * pl.w_stage_bytes > cap) {
            --occ;
            cap = (size_t)kMaxSmem / occ - (occ > 1 ? 2048 : 0);
        }
        if (fixed + 2 * pl.a_stage_bytes + 2 * pl.w_stage_bytes > cap) continue;
        pl.a_stages = (fixed + 3 * pl.a_stage_bytes + 3 * pl.w_stage_bytes <= cap) ? 3 : 2;
        if (pl.a_stages > pl.n_slabs) pl.a_stages = pl.n_slabs < 2 ? 2 : pl.n_slabs;
        int ws = (int)((cap - fixed - pl.a_stages * pl.a_stage_bytes) / pl.w_stage_bytes);
        if (ws > kMaxWStages) ws = kMaxWStages;
        pl.w_stages = ws;
        pl.a_ring_off = pl.meta_bytes;
        pl.w_ring_off = pl.a_ring_off + pl.a_stages * pl.a_stage_bytes;
        pl.epi_off = pl.w_ring_off + pl.w_stages * pl.w_stage_bytes;
        pl.smem = pl.epi_off + epi + 1024;
        pl.ctas = pl.tiles * ((n_panels + pl.WN - 1) / pl.WN);

        const int warps = pl.WM * pl.WN;
        const double mma_per_warp = (double)n_cols * density * kPanelRows * steps * pl.MT;
        const long long slots = 148LL * occ;
        const long long waves = (pl.ctas + slots - 1) / slots;
        const double resident = (double)warps * (pl.ctas < slots ? (double)((pl.ctas + 147) / 148) : occ);
        // a lone warp issues one MMA per ~8 cycles and pays ~150 cycles of exposed latency per K-step; the SM's
        // tensor pipe takes one MMA per 2 cycles
        const double warp_cycles = mma_per_warp * 8.0 + (double)n_cols * steps * 150.0;
        const double pipe_cycles = resident * mma_per_warp * 2.0 * 1.2;
        const double t_compute = waves * (warp_cycles > pipe_cycles ? warp_cycles : pipe_cycles) / 1.9e9;
        const double bytes = (double)pl.ctas * patch_pix * n_cols * CB +
                             (double)pl.tiles * n_panels * n_cols * kPanelRows * tile_bytes * density;
        const double t_traffic = bytes / 3.0e12;
        const double cost = (t_compute > t_traffic ? t_compute : t_traffic) + 0.25 * (t_compute < t_traffic ? t_compute : t_traffic);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = pl; }
    }
    return best;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

template <int DT, int MT, int WM, int WN, int HKT>
bsp_status launch_hk(const ConvParams &p, const Plan &pl, cudaStream_t st)
{
    auto kern = conv_mma_kernel<DT, MT, WM, WN, HKT>;
    // opt in to large dynamic shared memory once per device and instantiation
    static bool opted[kMaxDevices] = {};
    int dev = 0;
    BSP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BSP_ERR_CUDA;
    if (!opted[dev]) {
        BSP_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem + 1024));
        opted[dev] = true;
    }
    dim3 grid((unsigned)pl.tiles, (unsigned)((p.n_panels + WN - 1) / WN));
    kern<<<grid, 32 * (WM * WN + 1), pl.smem, st>>>(p);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

// 1x1 kernels use the unrolled column code for every shape, 3x3 kernels for the kMT = 2 shapes (at kMT = 4 the
// fragments of all nine taps do not fit in registers); everything else runs the general step loop.
template <int DT, int MT, int WM, int WN>
bsp_status launch_cfg(const ConvParams &p, const Plan &pl, cudaStream_t st)
{
    if constexpr (DT != BSP_F32) {
        if (p.H == 1 && p.K == 1) return launch_hk<DT, MT, WM, WN, 1>(p, pl, st);
        if constexpr (MT == 2) {
            if (p.H == 3 && p.K == 3) return launch_hk<DT, MT, WM, WN, 9>(p, pl, st);
        }
    }
    return launch_hk<DT, MT, WM, WN, 0>(p, pl, st);
}

template <int DT>
bsp_status launch_dt(const ConvParams &p, const Plan &pl, cudaStream_t st)
{
    const int key = pl.MT * 100 + pl.WM * 10 + pl.WN;
    switch (key) {
        case 222: return launch_cfg<DT, 2, 2, 2>(p, pl, st);
        case 241: return launch_cfg<DT, 2, 4, 1>(p, pl, st);
        case 214: return launch_cfg<DT, 2, 1, 4>(p, pl, st);
        case 242: return launch_cfg<DT, 2, 4, 2>(p, pl, st);
        case 281: return launch_cfg<DT, 2, 8, 1>(p, pl, st);
        case 224: return launch_cfg<DT, 2, 2, 4>(p, pl, st);
        case 422: return launch_cfg<DT, 4, 2, 2>(p, pl, st);
        case 442: return launch_cfg<DT, 4, 4, 2>(p, pl, st);
        case 424: return launch_cfg<DT, 4, 2, 4>(p, pl, st);
    }
    return BSP_ERR_SHAPE;
}

}  // namespace

bsp_status launch_conv(const bsp_wdesc &wd, const bsp_xdesc &xd, const void *packed, const void *X,
                       const void *bias, void *Y, bsp_dtype ytype, double density, void *ws, cudaStream_t st)
{
    const PackedLayout L = packed_layout(wd, 0);
    const int M = (xd.L + 2 * xd.pad_h - wd.H) / xd.stride_h + 1;
    const int Nw = (xd.J + 2 * xd.pad_w - wd.K) / xd.stride_w + 1;
    const Plan pl = make_plan(wd, xd, M, Nw, L.n_panels, L.n_cols, density);
    if (pl.MT == 0) return BSP_ERR_SHAPE;
    const int e = elem_bytes(wd.wtype);
    const uint8_t *pk = (const uint8_t *)packed;
    ConvParams p = {};
    p.Y = (uint8_t *)Y; p.bias = bias;
    p.colmask = pk + L.off_colmask;
    p.coloff = (const uint32_t *)(pk + L.off_coloff);
    p.panel_base = (const uint32_t *)(pk + L.off_panelbase);
    p.payload = pk + L.off_payload;
    p.status = (int *)ws;
    p.N = xd.N; p.L = xd.L; p.J = xd.J; p.I = wd.I; p.O = wd.O; p.M = M; p.Nw = Nw; p.H = wd.H; p.K = wd.K;
    p.sh = xd.stride_h; p.sw = xd.stride_w; p.ph = xd.pad_h; p.pw = xd.pad_w;
    p.nb = pl.nb; p.th = pl.th; p.tw = pl.tw;
    p.PH = (pl.th - 1) * xd.stride_h + wd.H; p.PW = (pl.tw - 1) * xd.stride_w + wd.K;
    p.patch_pix = pl.nb * p.PH * p.PW; p.tile_pix = pl.nb * pl.th * pl.tw;
    p.tiles_x = (Nw + pl.tw - 1) / pl.tw; p.tiles_y = (M + pl.th - 1) / pl.th;
    p.n_cols = L.n_cols; p.n_panels = L.n_panels; p.tile_bytes = L.tile_bytes;
    p.slab_cols = pl.slab_cols; p.n_slabs = pl.n_slabs; p.a_stages = pl.a_stages;
    p.a_stage_bytes = (int)pl.a_stage_bytes; p.a_box_bytes = (int)pl.a_box_bytes;
    p.GCW = pl.GCW; p.w_stages = pl.w_stages; p.w_stage_bytes = (int)pl.w_stage_bytes; p.wseg_cap = (int)pl.wseg_cap;
    p.meta_bytes = (int)pl.meta_bytes; p.a_ring_off = (int)pl.a_ring_off; p.w_ring_off = (int)pl.w_ring_off;
    p.epi_off = (int)pl.epi_off;
    p.ytype = ytype;

    // Activations as a rank-4 byte tensor (channel bytes, x, y, n); a box is a 128-byte slab of channels of
    // the tile's input patch, stored with the 128-byte swizzle.
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return BSP_ERR_CUDA;
    const cuuint64_t row = (cuuint64_t)wd.I * e;
    const cuuint64_t gdim[4] = {row, (cuuint64_t)xd.J, (cuuint64_t)xd.L, (cuuint64_t)xd.N};
    const cuuint64_t gstr[3] = {row, row * xd.J, row * xd.J * xd.L};
    const cuuint32_t box[4] = {(cuuint32_t)kSlabBytes, (cuuint32_t)p.PW, (cuuint32_t)p.PH, (cuuint32_t)pl.nb};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (enc(&p.tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(X), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return BSP_ERR_CUDA;

    if (wd.wtype == BSP_BF16) return launch_dt<BSP_BF16>(p, pl, st);
    if (wd.wtype == BSP_I8) return launch_dt<BSP_I8>(p, pl, st);
    return launch_dt<BSP_F32>(p, pl, st);
}

}  // namespace bsp
