// Pieces shared by the tensor-core kernels (tcgen05.mma with accumulators in tensor memory, operands staged by tiled
// TMA loads under the 128-byte swizzle): constants, bounded barrier waits, shared-memory matrix descriptors, the issue of
// one K-stage, tensor-memory loads, the tensor-map encoder and the choice of position tiles.  Every translation unit
// that includes this file gets its own copies (anonymous namespace).
#pragma once
#include <cuda.h>
#include "bsp_internal.cuh"

namespace bsp {
namespace {

constexpr int kGtThreads = 320;                    // producer warp, MMA warp, two groups of four epilogue warps
constexpr int kGtBM = 128;                         // positions per tile (M of the MMA)
constexpr int kGtABytes = kGtBM * 128;             // activation bytes of a stage
constexpr int kGtStageRows = 32;                   // rows of Y per epilogue warp
constexpr int kGtStagingBytes = kGtStageRows * 128;   // one staging buffer of an epilogue warp
constexpr int kGtMaxStages = 8;
constexpr int kGtMaxSmem = 226 * 1024;
constexpr int kGtTmemCols = 512;
constexpr int kGtMaxDevices = 64;
constexpr uint32_t kGtSpin = 1u << 24;             // polls of a barrier before a wait gives up

__device__ __forceinline__ uint32_t sm32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool gt_poll(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < kGtSpin; ++spin) {
        uint32_t done;
        asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
// The same wait for the threads of the epilogue warps: try_wait suspends the thread for a while.
__device__ __forceinline__ bool gt_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < (kGtSpin >> 6); ++spin) {
        uint32_t done;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// Shared-memory matrix descriptor of a K-major operand under the 128-byte swizzle (start address in 16-byte units in
// the low 14 bits): rows of 128 bytes, 8-row groups 1024 bytes apart; a K-step of 32 bytes inside the swizzle span is
// an advance of the start address by 2.
constexpr uint64_t kGtDesc = (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
// The same for rows of 64 bytes under the 64-byte swizzle (layers with at most 64 bytes of input channels): 8-row
// groups 512 bytes apart, two K-steps of 32 bytes.
constexpr uint64_t kGtDesc64 = (1ull << 16) | ((uint64_t)(512u >> 4) << 32) | (1ull << 46) | (4ull << 61);

// The four MMAs of one stage (two when the stage holds 64 bytes of K: `nk`) and the commit that releases the stage,
// issued by one elected lane of a converged warp.  All lanes execute this statement with the same operands; the MMA of
// the first K-step overwrites the accumulator when `acc` is 0.
#define GT_ISSUE_STAGE(KIND, CG, COMMIT_TAIL)                                                                       \
    asm volatile("{\n .reg .pred e, e3, p, t;\n .reg .b64 a1, a2, a3, b1, b2, b3;\n"                                 \
                 " elect.sync _|e, 0xFFFFFFFF;\n setp.ne.b32 p, %5, 0;\n setp.eq.b32 t, %5, %5;\n"                    \
                 " setp.gt.u32 e3, %7, 2;\n and.pred e3, e3, e;\n"                                                    \
                 " add.u64 a1, %1, 2;\n add.u64 a2, %1, 4;\n add.u64 a3, %1, 6;\n"                                    \
                 " add.u64 b1, %2, 2;\n add.u64 b2, %2, 4;\n add.u64 b3, %2, 6;\n"                                    \
                 " @e tcgen05.mma.cta_group::" CG ".kind::" KIND " [%0], %1, %2, %3, p;\n"                                 \
                 " @e tcgen05.mma.cta_group::" CG ".kind::" KIND " [%0], a1, b1, %3, t;\n"                                 \
                 " @e3 tcgen05.mma.cta_group::" CG ".kind::" KIND " [%0], a2, b2, %3, t;\n"                                \
                 " @e3 tcgen05.mma.cta_group::" CG ".kind::" KIND " [%0], a3, b3, %3, t;\n"                                \
                 " @e tcgen05.commit.cta_group::" CG ".mbarrier::arrive::one.shared::cluster" COMMIT_TAIL ";\n}\n"        \
                 ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(bar_empty), "r"(acc), "h"((unsigned short)3), "r"(nk) : "memory")

// kPair: the MMAs span a pair of CTAs (cta_group::2, M = 256: each CTA its own 128 positions and half of the weight
// tile); the commits then arrive on the barrier at the same shared-memory offset in both CTAs.
template <bool kPair>
__device__ __forceinline__ void gt_issue_stage(int wtype, uint32_t d, uint64_t da, uint64_t db, uint32_t idesc,
                                               uint32_t bar_empty, uint32_t acc, uint32_t nk = 4u)
{
    if constexpr (kPair) {
        if (wtype == BSP_BF16) GT_ISSUE_STAGE("f16", "2", ".multicast::cluster.b64 [%4], %6");
        else if (wtype == BSP_I8) GT_ISSUE_STAGE("i8", "2", ".multicast::cluster.b64 [%4], %6");
        else GT_ISSUE_STAGE("tf32", "2", ".multicast::cluster.b64 [%4], %6");
    } else {
        if (wtype == BSP_BF16) GT_ISSUE_STAGE("f16", "1", ".b64 [%4]");
        else if (wtype == BSP_I8) GT_ISSUE_STAGE("i8", "1", ".b64 [%4]");
        else GT_ISSUE_STAGE("tf32", "1", ".b64 [%4]");
    }
}
// All MMAs issued so far by the elected lane complete -> one arrival on `bar` (in both CTAs of a pair).
template <bool kPair>
__device__ __forceinline__ void gt_commit_elected(uint32_t bar)
{
    if constexpr (kPair)
        asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xFFFFFFFF;\n"
                     " @e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n}\n"
                     ::"r"(bar), "h"((unsigned short)3) : "memory");
    else
        asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xFFFFFFFF;\n"
                     " @e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}\n" ::"r"(bar) : "memory");
}

// Synchronises the CTA (the two CTAs of a pair).
template <bool kPair>
__device__ __forceinline__ void gt_sync_all()
{
    if constexpr (kPair) {
        asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
    } else {
        __syncthreads();
    }
}

// n / d and n % d for 0 <= n < 2^31 by the multiplier m = floor(2^32 / d) (0xFFFFFFFF for d = 1): the product's high
// word is the quotient or one less, one correction settles it.
__device__ __forceinline__ void gt_divmod(int n, int d, uint32_t m, int &q, int &r)
{
    q = (int)__umulhi((uint32_t)n, m);
    r = n - q * d;
    if (r >= d) { ++q; r -= d; }
}

// Requantisation of the 8-bit path (Section "Compiler and its Code generation", Eq. (quant)): v / 2^s rounded to the
// nearest integer, halves away from zero, as a 32-bit value that is not yet saturated (|v| + 2^(s-1) < 2^32, so the
// magnitude is formed without overflow; -2^31 with s = 0 comes back as itself) ...
__device__ __forceinline__ int gt_round_shift(int v, uint32_t s)
{
    const uint32_t sg = (uint32_t)(v >> 31);                              // 0 or all ones
    const uint32_t mag = ((uint32_t)v ^ sg) - sg;                        // |v|, at most 2^31
    const uint32_t r = (mag + ((1u << s) >> 1)) >> s;
    return (int)((r ^ sg) - sg);
}
// ... and four such values saturated to int8 and packed, the first in the lowest byte (cvt.pack saturates two 32-bit
// values to bytes, its first source above its second, and shifts the third operand up by 16 bits).
__device__ __forceinline__ uint32_t gt_pack_s8x4(int v0, int v1, int v2, int v3)
{
    uint32_t hi, out;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;\n" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0u));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;\n" : "=r"(out) : "r"(v1), "r"(v0), "r"(hi));
    return out;
}

// Barrier `id` (1..15) over the 128 threads of a group of four warps, and the same with the AND of a flag.
__device__ __forceinline__ void gt_group_sync(int id) { asm volatile("bar.sync %0, 128;\n" ::"r"(id) : "memory"); }
__device__ __forceinline__ bool gt_group_all(int id, bool flag)
{
    uint32_t r;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 p, %1, 0;\n bar.red.and.pred q, %2, 128, p;\n selp.b32 %0, 1, 0, q;\n}\n"
                 : "=r"(r) : "r"((uint32_t)flag), "r"(id) : "memory");
    return r != 0u;
}

// 32 consecutive accumulator columns of this thread's tensor-memory lane.
__device__ __forceinline__ void gt_load32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

typedef CUresult (*GtEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                               const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

GtEncodeFn gt_encode()
{
    static GtEncodeFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (GtEncodeFn)ptr;
    }
    return fn;
}


// Position tile of a layer: Wt x Ht output positions of Nt images, at most 128, chosen for the fewest tiles (ties: the
// smaller box).  Several images share a tile only when a tile holds whole images.  A box of the tensor map spans
// Wt * s_w x Ht * s_h input positions and may not exceed 256 in any extent.
struct GtTile { int Wt, Ht, Nt; long long tiles; };

// A 1x1 layer without padding or stride is a matrix product over all N L J positions: taken as that many 1x1 images,
// so that a tile is 128 consecutive positions whatever the image size.
bsp_xdesc gt_flatten(const bsp_wdesc &wd, const bsp_xdesc &xd)
{
    const long long P = (long long)xd.N * xd.L * xd.J;
    if (wd.H == 1 && wd.K == 1 && xd.pad_h == 0 && xd.pad_w == 0 && xd.stride_h == 1 && xd.stride_w == 1 && P <= 0x7FFFFFFF)
        return bsp_xdesc{(int)P, 1, 1, 1, 1, 0, 0};
    return xd;
}

uint32_t gt_magic(int d) { return d <= 1 ? 0xFFFFFFFFu : (uint32_t)((1ull << 32) / (uint64_t)d); }

GtTile gt_pick_tile(int N, int M, int Nw, int sh, int sw)
{
    GtTile best = {0, 0, 0, -1};
    for (int w = 1; w <= Nw && w <= kGtBM; ++w) {
        if (w * sw > 256) break;
        for (int h = 1; h <= M && h * w <= kGtBM; ++h) {
            if (h * sh > 256) break;
            int b = 1;
            if (w == Nw && h == M) { b = kGtBM / (w * h); if (b > N) b = N; if (b > 256) b = 256; if (b < 1) b = 1; }
            const long long cnt = (long long)((N + b - 1) / b) * ((M + h - 1) / h) * ((Nw + w - 1) / w);
            const long long area = (long long)b * h * w, best_area = (long long)best.Wt * best.Ht * best.Nt;
            if (best.tiles < 0 || cnt < best.tiles || (cnt == best.tiles && area < best_area)) best = {w, h, b, cnt};
        }
    }
    return best;
}

}  // namespace
}  // namespace bsp
