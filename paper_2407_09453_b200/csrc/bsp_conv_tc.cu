// Block-sparse implicit-GEMM convolution / FC product with fused bias on 5th-generation tensor cores
// (tcgen05.mma, accumulators in tensor memory), bf16 (fp32 accumulators) or int8 (int32, exact) inputs, any stride
// whose residues in use number at most four.  Introduction (Y = W*X + b) and Section
// "Block Sparsity in a Matrix" of the paper.
//
// One MMA is D[128 x 16n] += A[128 x 16] * B[16 x 16n]: 128 output positions, n consecutive stored super-rows
// of 16 output channels, 32 bytes of reduction elements (two taps of 8 bf16 / 16 int8 input channels, or 16 / 32
// input channels of a 1x1 layer).  The unit that can be skipped is a 16-channel x K-group super-tile of W-bar; zeroed 8x8 blocks inside
// a stored super-tile are multiplied as zeros.  The stored super-tiles of a run of consecutive super-rows lie
// side by side in the packed payload and in tensor memory, so a run is ONE MMA with N = 16 x (run length): a
// dense layer issues N = 128 MMAs, a sparse one an MMA per run of its mask.
//
// A CTA owns 128 consecutive positions of one image and one group of 8 super-rows (128 channels).  Positions
// are counted over rows of PW = N' + (K-1)/s_w positions (the padded input width at stride 1), so that the input
// of output position m at tap (h, k) is a staged element at a constant offset from m: positions whose column falls
// beyond N' compute garbage and are not stored.  Activations are staged by tiled TMA loads (out-of-bounds fill =
// zero padding) as planes [16-byte chunk][position][16 bytes], the no-swizzle K-major core-matrix layout: 8
// consecutive positions are one core matrix, the two K halves of an MMA are two planes or two tap offsets (the
// descriptor's leading-dimension byte offset).  With strides, each residue (h mod s_h, k mod s_w) in use is staged
// as a stride-1 image of its own through the tensor map's element strides.  An unpadded stride-1 1x1 layer is a
// matrix product over all N*L*J positions: its K-groups are staged as [position][32 bytes] planes under the 32-byte
// swizzle, 256 positions per CTA when the grid stays large.  The stored super-tiles of the group for the stage's
// K-groups are one contiguous stretch of the packed payload (one bulk copy).
// Warps 0-3 issue: issuer s takes the K-groups kc with kc % 4 == s and accumulates them in its own 128 columns
// of tensor memory (an MMA this small costs more to issue than to execute, and MMAs of different threads on one
// accumulator are not ordered, hence four accumulator sets, zeroed at the start and summed at the end; with 256
// positions the issuers split into two position halves x two K phases; the largest products take two channel
// groups per CTA as well, 256 positions x 256 channels, and every issuer then owns one (half, group) quadrant over
// all K-groups).  Warp 4 produces.  The producer and the issuers are single threads whose instruction count per stage
// is on the critical path: the runs of every K-group are decoded once, by all threads, into 8-byte entries in shared
// memory, and the loops advance slot, parity and addresses by additions and poll their barriers.  Then all eight warps
// read their TMEM lanes back, add the sets and the bias, transpose 16-byte chunks inside groups of four lanes and
// store 64-byte pieces of rows.
// Every wait is bounded; on expiry BSP_ERR_TIMEOUT is latched and the CTA winds down.
#include <cuda.h>
#include "bsp_internal.cuh"

namespace bsp {
namespace {

constexpr int kIssuers = 4;                       // issuing warps = accumulator sets (K-groups interleaved over them)
constexpr int kTcThreads = 256;                   // warps 0-3 issue, warp 4 produces, all eight run the epilogue
constexpr int kTcMaxStages = 8;
constexpr int kTcMaxSmem = 200 * 1024;
constexpr int kTcMaxDevices = 64;
constexpr size_t kTcStageBudget = 64 * 1024;      // operand bytes of one stage that the K-groups per stage aim at
constexpr int kTmemCols = 128 * kIssuers;
constexpr uint32_t kTcSpinLimit = 1u << 22;
constexpr uint32_t kOffMask = 0x0FFFFFFFu;          // low bits of a K-group entry's first word: super-tiles before it

struct TcParams {
    CUtensorMap tmap;        // activations as (16 bytes, x, y, n, chunk)
    uint8_t *Y;
    const float *bias;
    const uint8_t *mask;
    const uint32_t *off;
    const uint32_t *gcnt;
    const uint8_t *packed;     // start of the packed buffer; its header gives the super-tile payload's offset
    int *status;
    int N, O, M, Nw, P, H, K, ph, pw;
    int PW, plane_bytes, tiles_per_img, is_gemm;
    int n_kc, n_units, st_bytes, chunks_per_kc;
    int coords_per_kc;        // steps of the tensor map's last coordinate per K-group
    // Strides: the padded input splits into s_h x s_w phase images (rows = a mod s_h, columns = b mod s_w); tap (h, k)
    // reads phase (h mod s_h, k mod s_w) at the constant offset (h / s_h, k / s_w), so every phase in use is staged as a
    // stride-1 plane set of its own (one tiled load each, through the tensor map's element strides).
    int sh, sw, n_phase, phase_bytes;      // phase_bytes: bytes of one phase's planes in a stage
    int ph_a[4], ph_b[4];                  // the phases in use, in the order they lie in a stage
    int mt;                   // 128-position tiles per CTA: 1, or 2 for large matrix products (the weights are then
                              // fetched once for 256 positions); the four issuers split into mt halves x 4/mt K phases
    int ng;                   // channel groups per CTA: 1, or 2 for the largest matrix products (mt == 2 only: the
                              // activations are then fetched once for 256 channels); issuer = (half, group), all K-groups
    int n_groups, w_stride;   // groups of the layer; bytes between the two groups' weights in a stage
    int GK, n_stage_iters, stages, stage_bytes, act_bytes, act_box_bytes;
    int ytype;
};

__device__ __forceinline__ uint32_t s32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin) {
        uint32_t done;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// The same wait by polling: mbarrier.test_wait does not suspend the thread, and on a phase that is already
// complete it answers in a fraction of the ~200 cycles that try_wait takes.  For the single threads that run the
// producer and issue loops, where every cycle of a wait is on the critical path.
__device__ __forceinline__ bool poll_bar(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin) {
        uint32_t done;
        asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// Shared-memory matrix descriptor, no swizzle, K-major: 8 rows x 16 bytes core matrices; `lbo` = bytes between
// the two K halves, `sbo` = bytes between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void commit_to(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}

// Transposes 4x4 blocks of 16-byte chunks inside every group of four lanes: on entry a lane holds the four chunks
// (v[4c .. 4c+3], c = 0..3) of its own row, on exit chunk (lane % 4) of the four rows of its group (v[4j .. 4j+3] =
// row j of the group).  All 32 lanes take part.
__device__ __forceinline__ void transpose_chunks(uint32_t (&v)[16], int lane)
{
    const bool hi2 = (lane & 2) != 0, hi1 = (lane & 1) != 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {          // the 2x2 blocks off the diagonal change places (partner: lane ^ 2)
        const uint32_t s0 = hi2 ? v[k] : v[8 + k], s1 = hi2 ? v[4 + k] : v[12 + k];
        const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, s0, 2), r1 = __shfl_xor_sync(0xFFFFFFFFu, s1, 2);
        if (hi2) { v[k] = r0; v[4 + k] = r1; } else { v[8 + k] = r0; v[12 + k] = r1; }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {          // then the off-diagonal chunks inside every 2x2 block (partner: lane ^ 1)
        const uint32_t s0 = hi1 ? v[k] : v[4 + k], s1 = hi1 ? v[8 + k] : v[12 + k];
        const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, s0, 1), r1 = __shfl_xor_sync(0xFFFFFFFFu, s1, 1);
        if (hi1) { v[k] = r0; v[8 + k] = r1; } else { v[4 + k] = r0; v[12 + k] = r1; }
    }
}

// Stores 16 32-bit outputs per lane (one row of Y each: `dst`, used if `valid`) so that a warp instruction writes whole
// 64-byte pieces of eight rows instead of 16 bytes of thirty-two: the chunks are transposed inside groups of four
// lanes, lane 4q + c then writes chunk c of the rows of lanes 4q .. 4q + 3.  nch: channels present (8 or 16).
__device__ __forceinline__ void store_rows32(uint32_t (&v)[16], uint8_t *dst, bool valid, int nch, int lane)
{
    transpose_chunks(v, lane);
    const int c = lane & 3, first = lane & ~3;
    const unsigned long long d = (unsigned long long)dst;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int ok = __shfl_sync(0xFFFFFFFFu, (int)valid, first + j);
        const unsigned long long dj = __shfl_sync(0xFFFFFFFFu, d, first + j);
        if (ok && 4 * c < nch) *(uint4 *)(dj + 16u * c) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    }
}

// kI8: int8 inputs with int32 accumulators, bias and output (kind::i8); otherwise bf16 with fp32 (kind::f16).
template <bool kI8>
__global__ void __launch_bounds__(kTcThreads, 1) conv_tc_kernel(const __grid_constant__ TcParams p)
{
    extern __shared__ __align__(16) uint8_t tc_smem_raw[];
    uint8_t *smem = tc_smem_raw + ((1024u - (s32(tc_smem_raw) & 1023u)) & 1023u);   // stages of swizzled planes start on 1 KB
    __shared__ __align__(8) uint64_t s_full[kTcMaxStages];
    __shared__ __align__(8) uint64_t s_empty[kTcMaxStages];
    __shared__ __align__(8) uint64_t s_done;
    __shared__ uint32_t s_tmem, s_gbase[2], s_gcnt[2], s_fail;
    __shared__ const uint8_t *s_payload;
    __shared__ uint64_t s_ahi[64];          // per K-step of a super-tile: A descriptor without its address field
    __shared__ uint32_t s_aoff[64];         // ... and the operand's offset from the K-group's first plane, in 16-byte units

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = blockIdx.y * p.ng;
    const int S = p.stages;

    // stored super-tiles of this group: masks and offsets of every K-group -> shared memory
    // (a second group beyond the layer's last reads as empty)
    // One entry per K-group, decoded here by all threads so that the issuing threads need not: .x = stored super-tiles
    // of the group before the K-group (28 bits) and in it (4 bits); .y = its runs of consecutive stored super-rows, a
    // byte each, first run lowest: 0x80 | first row << 3 | (length - 1); a zero byte ends the list.
    uint2 *s_ent = (uint2 *)smem;                                   // [ng][n_kc]
    const int n_meta = (g + p.ng <= p.n_groups ? p.ng : 1) * p.n_kc;
    for (int i = tid; i < p.ng * p.n_kc; i += kTcThreads) {
        uint32_t off = 0u, m = 0u;
        if (i < n_meta) { off = p.off[(size_t)g * p.n_kc + i]; m = p.mask[(size_t)g * p.n_kc + i]; }
        uint32_t runs = 0u, sh = 0u;
        for (uint32_t mm = m; mm;) {
            const uint32_t r0 = (uint32_t)__ffs(mm) - 1u, len = (uint32_t)__ffs(~(mm >> r0)) - 1u;
            mm &= ~(((1u << len) - 1u) << r0);
            runs |= (0x80u | (r0 << 3) | (len - 1u)) << sh;
            sh += 8u;
        }
        s_ent[i] = make_uint2(off | ((uint32_t)__popc(m) << 28), runs);
    }
    if (tid == 0) {
        uint32_t base = 0;
        for (int q = 0; q < g; ++q) base += p.gcnt[q];
        s_gbase[0] = base; s_gcnt[0] = p.gcnt[g];
        const bool second = p.ng == 2 && g + 1 < p.n_groups;
        s_gbase[1] = base + p.gcnt[g]; s_gcnt[1] = second ? p.gcnt[g + 1] : 0u;
        s_fail = 0;
        s_payload = p.packed + ((const PackedHeader *)p.packed)->off_tc_payload;
    }
    // tile geometry
    int n_img = 0, m0 = 0, y_first = 0, rowbase = 0;
    if (p.is_gemm) { m0 = blockIdx.x * 128 * p.mt; }
    else {
        n_img = blockIdx.x / p.tiles_per_img;
        m0 = (blockIdx.x % p.tiles_per_img) * 128;
        y_first = m0 / p.PW;
        rowbase = m0 - y_first * p.PW;
    }
    for (int u = tid; u < p.n_units; u += kTcThreads) {
        uint32_t lbo, off;
        if (p.is_gemm) {
            // matrix product: a K-group's plane is [position][32 bytes = 16 channels] under the 32-byte swizzle,
            // 8 positions (256 bytes) per row group; the leading-dimension offset is not used
            s_aoff[u] = 0;
            s_ahi[u] = smem_desc(0, 16, 256) | (6ull << 61);
            continue;
        }
        if (p.chunks_per_kc == 2) {                 // 1x1 kernel with padding: the K halves are two 8-channel planes
            off = (uint32_t)rowbase;
            lbo = (uint32_t)p.plane_bytes;
        } else {
            // position offset (16-byte units from the stage's first plane) of a tap: its phase's planes, then (h / s_h) rows
            // and k / s_w columns
            auto tap_off = [&](int t) -> int {
                const int h = t / p.K, k = t % p.K;
                if (p.n_phase == 1 && p.sh == 1 && p.sw == 1) return h * p.PW + k;       // stride 1: the tap's row and column
                int ph = 0;
                for (int i = 0; i < p.n_phase; ++i)
                    if (p.ph_a[i] == h % p.sh && p.ph_b[i] == k % p.sw) ph = i;
                return ph * (p.phase_bytes >> 4) + (h / p.sh) * p.PW + k / p.sw;
            };
            const int t0 = 2 * u, t1 = 2 * u + 1;
            const int o0 = tap_off(t0);
            off = (uint32_t)(rowbase + o0);
            // a missing odd tap has zero weights; its K half reads the next position (finite data).  The host orders
            // the phases so that the second tap of a pair lies after the first.
            lbo = (t1 < p.H * p.K) ? (uint32_t)(tap_off(t1) - o0) * 16u : 16u;
        }
        s_aoff[u] = off;
        s_ahi[u] = smem_desc(0, lbo, 128);
    }
    // The producer thread sets the barriers up and starts the activation loads of the first stages at once: they
    // need nothing of the index arrays that the other threads are still fetching.  A full barrier takes two
    // arrivals per phase, one with the activation bytes and one with the weight bytes.
    const int meta_bytes = ((p.ng * p.n_kc * 8 + 1023) / 1024) * 1024;
    const uint32_t ring = s32(smem) + meta_bytes;
    // first input column and row of the tile's phase (0, 0); phase (a, b) starts a rows and b columns further
    const int c1 = p.is_gemm ? 0 : -p.pw, c2 = p.is_gemm ? 0 : y_first * p.sh - p.ph, c3 = p.is_gemm ? m0 : n_img;
    if (warp == kIssuers && lane == 0) {
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmap) : "memory");
        for (int s = 0; s < S; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(s32(&s_full[s])), "r"(2) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(s32(&s_empty[s])), "r"(kIssuers) : "memory");
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(s32(&s_done)), "r"(kIssuers) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        for (int it = 0; it < min(S, p.n_stage_iters); ++it) {
            const uint32_t bar = s32(&s_full[it]);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"((uint32_t)(p.n_phase * p.act_box_bytes)) : "memory");
            for (int ph = 0; ph < p.n_phase; ++ph)
                asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];\n"
                             ::"r"(ring + it * p.stage_bytes + ph * p.phase_bytes), "l"(&p.tmap), "r"(bar), "r"(0), "r"(c1 + p.ph_b[ph]),
                               "r"(c2 + p.ph_a[ph]), "r"(c3), "r"(it * p.GK * p.coords_per_kc) : "memory");
        }
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(s32(&s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem = s_tmem;
    // every accumulator starts at zero, so that every MMA accumulates and super-rows without a stored tile read as
    // zero: warps 0-3 clear the 32 TMEM lanes they can reach, all columns
    if (warp < 4) {
        const uint32_t z = 0u;
        for (int c = 0; c < kTmemCols; c += 16)
            asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};\n"
                         ::"r"(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c), "r"(z) : "memory");
        asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");

    if (warp == kIssuers) {
        // ================= producer (warp 4) =================
        // (one thread runs the whole loop, so its instruction count per stage is on the critical path: the slot, the
        // barrier parity and the addresses advance by additions, loop invariants sit in registers)
        if (lane == 0) {
            const int GK = p.GK, n_kc = p.n_kc, n_it = p.n_stage_iters, n_phase = p.n_phase, ng = p.ng;
            const uint32_t st_bytes = (uint32_t)p.st_bytes, act_tx = (uint32_t)(p.n_phase * p.act_box_bytes);
            const uint32_t stage_bytes = (uint32_t)p.stage_bytes, w_first = (uint32_t)p.act_bytes, w_stride = (uint32_t)p.w_stride;
            const uint32_t full0 = s32(&s_full[0]), empty0 = s32(&s_empty[0]);
            const uint8_t *const pay0 = s_payload + (size_t)s_gbase[0] * st_bytes;
            const uint8_t *const pay1 = s_payload + (size_t)s_gbase[1] * st_bytes;
            const uint32_t gcnt0 = s_gcnt[0], gcnt1 = s_gcnt[1];
            uint32_t slot = 0, wrapped = 0, dst = ring;       // wrapped: times the ring has been filled
            int kc0 = 0, kcoord = 0;
            for (int it = 0; it < n_it; ++it) {
                const uint32_t bar = full0 + slot * 8u;
                if (wrapped && !poll_bar(empty0 + slot * 8u, (wrapped - 1u) & 1u)) { atomicExch(&s_fail, 1u); break; }
                const int kc1 = kc0 + GK;
                const uint32_t lo0 = s_ent[kc0].x & kOffMask, hi0 = kc1 < n_kc ? s_ent[kc1].x & kOffMask : gcnt0;
                uint32_t lo1 = 0u, hi1 = 0u;
                if (ng == 2) { lo1 = s_ent[n_kc + kc0].x & kOffMask; hi1 = kc1 < n_kc ? s_ent[n_kc + kc1].x & kOffMask : gcnt1; }
                const uint32_t wb0 = (hi0 - lo0) * st_bytes, wb1 = (hi1 - lo1) * st_bytes;
                if (wrapped) {          // the first S activation loads were issued before the index arrays arrived
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(act_tx) : "memory");
                    for (int ph = 0; ph < n_phase; ++ph)
                        asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];\n"
                                     ::"r"(dst + ph * p.phase_bytes), "l"(&p.tmap), "r"(bar), "r"(0), "r"(c1 + p.ph_b[ph]), "r"(c2 + p.ph_a[ph]),
                                       "r"(c3), "r"(kcoord) : "memory");
                }
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(wb0 + wb1) : "memory");
                if (wb0)
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                                 ::"r"(dst + w_first), "l"(pay0 + (size_t)lo0 * st_bytes), "r"(wb0), "r"(bar) : "memory");
                if (wb1)
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                                 ::"r"(dst + w_first + w_stride), "l"(pay1 + (size_t)lo1 * st_bytes), "r"(wb1), "r"(bar) : "memory");
                kc0 = kc1; kcoord += GK * p.coords_per_kc;
                if (++slot == (uint32_t)S) { slot = 0; ++wrapped; dst = ring; } else dst += stage_bytes;
            }
        }
    } else if (warp < kIssuers) {
        // ================= MMA issuers: warp s takes the K-groups kc with kc % kIssuers == s =================
        // One thread per issuing warp runs the whole issue loop: a tcgen05.mma is issued by a single thread, and
        // keeping that thread in one long non-divergent stretch avoids a divergence region around every MMA.
        if (lane == 0) {
            // instruction descriptor: D fp32, A and B bf16 (or D int32, A and B signed 8-bit), M = 128; + (N >> 3) << 17
            constexpr bool i8 = kI8;
            const uint32_t idesc0 = ((i8 ? 2u : 1u) << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);
            // Descriptors are sums: the address field (16-byte units, low 14 bits) of an A operand is
            // stage + plane + s_aoff[u]; of a B operand weights + 32 * (tiles before the K-group * n_units
            // + u * tiles of the K-group + tiles before the run).  B: K halves 128 bytes apart, row groups 256.
            const uint64_t b_hi = smem_desc(0, 128, 256);
            const uint32_t plane16 = (uint32_t)((p.plane_bytes >> 4) * p.chunks_per_kc);  // 16-byte units between K-groups' planes
            const uint32_t nu = (uint32_t)p.n_units;
            const uint64_t ahi0 = s_ahi[0];
            const uint32_t aoff0 = s_aoff[0];
            const uint32_t dset = tmem + (uint32_t)warp * 128u;
            // two groups per CTA: issuer = (position half, group), every K-group; its accumulator is its own 128 columns
            const int gq = p.ng == 2 ? (warp & 1) : 0;
            const int kphases = p.ng == 2 ? 1 : kIssuers / p.mt;
            const int kphase = warp % kphases;                                  // K-groups kc with kc % kphases == kphase
            const uint32_t ahalf = (uint32_t)(p.mt == 2 ? warp >> 1 : 0) * 256u;  // second 128 positions: 4096 bytes into the plane
            const uint2 *my_ent = s_ent + gq * p.n_kc;
            // (as in the producer: running slot, parity and addresses, invariants in registers)
            const int GK = p.GK, n_kc = p.n_kc, n_it = p.n_stage_iters;
            const uint32_t ring16 = ring >> 4, stage_step16 = (uint32_t)p.stage_bytes >> 4;
            const uint32_t wofs16 = (uint32_t)(p.act_bytes + gq * p.w_stride) >> 4;
            const uint32_t full0 = s32(&s_full[0]), empty0 = s32(&s_empty[0]);
            uint32_t slot = 0, par = 0, stage16 = ring16;
            int kc0 = 0;
            bool ok = true;
            for (int it = 0; it < n_it; ++it, kc0 += GK) {
                if (!poll_bar(full0 + slot * 8u, par)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const int nk = min(GK, n_kc - kc0);
                const uint32_t w16 = stage16 + wofs16;
                const uint32_t o_lo = my_ent[kc0].x & kOffMask;
                int kl = (kphase - kc0) & (kphases - 1);          // first K-group of the stage that is mine
                for (; kl < nk; kl += kphases) {
                    const uint2 ent = my_ent[kc0 + kl];
                    uint32_t runs = ent.y;
                    if (runs == 0u) continue;
                    const uint32_t cnt = ent.x >> 28;
                    const uint32_t a16 = stage16 + (uint32_t)kl * plane16 + ahalf;
                    const uint64_t a0 = ahi0 | (uint64_t)((a16 + aoff0) & 0x3FFFu);
                    uint32_t b16 = w16 + ((ent.x & kOffMask) - o_lo) * nu * 32u;   // first tile of the K-group, K-step 0
                    for (; runs; runs >>= 8) {
                        const uint32_t r0 = (runs >> 3) & 7u, len = (runs & 7u) + 1u;   // stored super-rows r0 .. r0 + len - 1
                        const uint32_t idesc = idesc0 | (len << 18);                   // N = 16 len, the field holds N / 8
                        const uint32_t d = dset + r0 * 16u;
                        if (nu == 1) {
                            if (i8) mma_i8(d, a0, b_hi | (uint64_t)(b16 & 0x3FFFu), idesc, 1u);
                            else mma_bf16(d, a0, b_hi | (uint64_t)(b16 & 0x3FFFu), idesc, 1u);
                        } else {
                            uint32_t bu = b16;
                            for (uint32_t u = 0; u < nu; ++u) {
                                if (i8) mma_i8(d, s_ahi[u] | (uint64_t)((a16 + s_aoff[u]) & 0x3FFFu), b_hi | (uint64_t)(bu & 0x3FFFu), idesc, 1u);
                                else mma_bf16(d, s_ahi[u] | (uint64_t)((a16 + s_aoff[u]) & 0x3FFFu), b_hi | (uint64_t)(bu & 0x3FFFu), idesc, 1u);
                                bu += cnt * 32u;
                            }
                        }
                        b16 += len * 32u;
                    }
                }
                commit_to(empty0 + slot * 8u);
                if (++slot == (uint32_t)S) { slot = 0; par ^= 1u; stage16 = ring16; } else stage16 += stage_step16;
            }
            if (ok) commit_to(s32(&s_done));
            else atomicExch(&s_fail, 1u);
        }
    }

    // ================= epilogue: all eight warps; warp w reads TMEM lanes 32*(w%4).. (positions) of super-rows 4*(w/4).. =================
    // (threads without a loop of their own park at the block barrier, not in a polling loop, until the loops end)
    __syncwarp();
    __syncthreads();
    bool done = wait_bar(s32(&s_done), 0);
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (s_fail) done = false;
    if (!done && tid == 0) atomicMax(p.status, (int)BSP_ERR_TIMEOUT);
    if (done) {
        const int lq = warp & 3;                 // a warp reaches the TMEM lanes of its quarter only
        // one position tile: warps 0-3 take super-rows 0-3, warps 4-7 rows 4-7, four accumulator sets each;
        // two tiles: warps 0-3 take the first 128 positions (sets 0, 1), warps 4-7 the second (sets 2, 3), all rows
        const int half = p.mt == 2 ? (warp >> 2) : 0;
        // (two groups: one accumulator set per (half, group), nothing to add)
        const int nsets = p.ng == 2 ? 1 : kIssuers / p.mt;
        const int r_lo = p.mt == 2 ? 0 : (warp >> 2) * 4, r_hi = p.mt == 2 ? kTcGroupRows : r_lo + 4;
        const int m = half * 128 + lq * 32 + lane;
        bool valid;
        size_t pix;
        if (p.is_gemm) { valid = m0 + m < p.P; pix = (size_t)(m0 + m); }
        else {
            const int mm = m0 + m, y = mm / p.PW, x = mm % p.PW;
            valid = y < p.M && x < p.Nw;
            pix = ((size_t)n_img * p.M + y) * p.Nw + x;
        }
        const int oe = (p.ytype == BSP_BF16) ? 2 : 4;
#pragma unroll 1
        for (int rr = r_lo; rr < r_hi + (p.ng - 1) * kTcGroupRows; ++rr) {
            const int gq = rr / kTcGroupRows, r = rr % kTcGroupRows;          // group of the CTA, super-row in it
            const int set0 = p.ng == 2 ? 2 * half + gq : (p.mt == 2 ? 2 * half : 0);
            const int ch = ((g + gq) * kTcGroupRows + r) * kTcSuperRow;
            if (ch >= p.O) break;
            // the four accumulator sets of this super-row
            uint32_t v[kIssuers][16];
#pragma unroll
            for (int s = 0; s < kIssuers; ++s) {
                if (s < nsets) {
                    const uint32_t ta = tmem + ((uint32_t)(lq * 32) << 16) + (uint32_t)((set0 + s) * 128 + r * 16);
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
                                 : "=r"(v[s][0]), "=r"(v[s][1]), "=r"(v[s][2]), "=r"(v[s][3]), "=r"(v[s][4]), "=r"(v[s][5]), "=r"(v[s][6]), "=r"(v[s][7]),
                                   "=r"(v[s][8]), "=r"(v[s][9]), "=r"(v[s][10]), "=r"(v[s][11]), "=r"(v[s][12]), "=r"(v[s][13]), "=r"(v[s][14]), "=r"(v[s][15])
                                 : "r"(ta) : "memory");
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[s][e] = 0u;
                }
            }
            asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
            const int nch = min(16, p.O - ch);        // 16, or 8 in a last half super-row
            if constexpr (kI8) {                      // exact: int32 sums of the four sets + int32 bias, int32 out
                uint32_t iv[16];
                const int *ib = (const int *)p.bias;
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    iv[e] = (uint32_t)((int)v[0][e] + (int)v[1][e] + (int)v[2][e] + (int)v[3][e] + ((ib != nullptr && e < nch) ? __ldg(ib + ch + e) : 0));
                store_rows32(iv, p.Y + (pix * p.O + ch) * 4, valid, nch, lane);
                continue;
            } else {
            float f[16];
#pragma unroll
            for (int e = 0; e < 16; ++e)
                f[e] = ((__uint_as_float(v[0][e]) + __uint_as_float(v[1][e])) + (__uint_as_float(v[2][e]) + __uint_as_float(v[3][e]))) +
                       ((p.bias != nullptr && e < nch) ? __ldg(p.bias + ch + e) : 0.f);
            uint8_t *dst = p.Y + (pix * p.O + ch) * oe;
            if (oe == 4) {
                uint32_t fv[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) fv[e] = __float_as_uint(f[e]);
                store_rows32(fv, dst, valid, nch, lane);
            } else {
#pragma unroll
                for (int q = 0; q < 2; ++q)
                    if (valid && q * 8 < nch) {
                        __nv_bfloat162 h0 = __floats2bfloat162_rn(f[8 * q], f[8 * q + 1]), h1 = __floats2bfloat162_rn(f[8 * q + 2], f[8 * q + 3]);
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(f[8 * q + 4], f[8 * q + 5]), h3 = __floats2bfloat162_rn(f[8 * q + 6], f[8 * q + 7]);
                        *(uint4 *)(dst + q * 16) = make_uint4(*(uint32_t *)&h0, *(uint32_t *)&h1, *(uint32_t *)&h2, *(uint32_t *)&h3);
                    }
            }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tc_encode_tiled()
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

}  // namespace

namespace {
// Position geometry of a layer for the tensor-memory kernel.  Output positions are counted over rows of PW = N' + (K-1)/s_w
// positions; a CTA's 128 positions need R rows of every phase image in use.
struct TcGeo {
    bool gemm;
    int M, Nw, PW, R, n_phase, ph_a[4], ph_b[4];
};

bool tc_geometry(const bsp_wdesc &wd, const bsp_xdesc &xd, TcGeo &g)
{
    g = TcGeo{};
    g.gemm = wd.H == 1 && wd.K == 1 && xd.pad_h == 0 && xd.pad_w == 0 && xd.stride_h == 1 && xd.stride_w == 1;
    g.M = (xd.L + 2 * xd.pad_h - wd.H) / xd.stride_h + 1;
    g.Nw = (xd.J + 2 * xd.pad_w - wd.K) / xd.stride_w + 1;
    g.n_phase = 1; g.PW = 1; g.R = 1;
    if (g.gemm) return true;
    const int sh = xd.stride_h, sw = xd.stride_w;
    const int Hq = (wd.H - 1) / sh, Kq = (wd.K - 1) / sw;
    g.PW = g.Nw + Kq;
    g.R = (g.PW - 1 + 127 + Hq * g.PW + Kq) / g.PW + 1;
    if (g.PW * sw > 256 || g.R * sh > 256) return false;          // extents of a tiled load
    // phases (h mod s_h, k mod s_w) that some tap reads
    int n = 0, pa[4], pb[4];
    for (int h = 0; h < wd.H; ++h)
        for (int k = 0; k < wd.K; ++k) {
            bool seen = false;
            for (int i = 0; i < n; ++i) seen |= pa[i] == h % sh && pb[i] == k % sw;
            if (seen) continue;
            if (n == 4) return false;
            pa[n] = h % sh; pb[n] = k % sw; ++n;
        }
    // an MMA multiplies taps 2u and 2u+1, the second at a non-negative byte offset from the first: find an order of
    // the phases in shared memory in which the second tap's phase never lies before the first's
    int perm[4] = {0, 1, 2, 3};
    const int HK = wd.H * wd.K;
    for (int trial = 0; trial < 24; ++trial) {
        int pos[4];                                       // pos[i]: place of phase i in this order
        {   // the trial-th permutation of 0..3 (factorial number system), restricted to the first n entries
            int pool[4] = {0, 1, 2, 3}, t = trial;
            const int f[4] = {6, 2, 1, 1};
            for (int i = 0; i < 4; ++i) {
                const int q = t / f[i]; t %= f[i];
                perm[i] = pool[q];
                for (int j = q; j < 3; ++j) pool[j] = pool[j + 1];
            }
        }
        bool uses_only = true;
        for (int i = 0; i < n; ++i) uses_only &= perm[i] < n;     // the first n places hold the n phases
        if (!uses_only) continue;
        for (int i = 0; i < n; ++i) pos[perm[i]] = i;
        bool ok = true;
        for (int t0 = 0; t0 + 1 < HK && ok; t0 += 2) {
            int i0 = 0, i1 = 0;
            for (int i = 0; i < n; ++i) {
                if (pa[i] == (t0 / wd.K) % sh && pb[i] == (t0 % wd.K) % sw) i0 = i;
                if (pa[i] == ((t0 + 1) / wd.K) % sh && pb[i] == ((t0 + 1) % wd.K) % sw) i1 = i;
            }
            ok = pos[i0] <= pos[i1];
        }
        if (!ok) continue;
        g.n_phase = n;
        for (int i = 0; i < n; ++i) { g.ph_a[i] = pa[perm[i]]; g.ph_b[i] = pb[perm[i]]; }
        return true;
    }
    return false;
}
}  // namespace

// True if the tcgen05 kernel can run this layer: bf16 or int8, super-tile form present, box extents in range.
bool conv_tc_eligible(const bsp_wdesc &wd, const bsp_xdesc &xd)
{
    if (wd.wtype != BSP_BF16 && wd.wtype != BSP_I8) return false;
    const PackedLayout L = packed_layout(wd, 0);
    if (!L.tc.enabled) return false;
    TcGeo g;
    if (!tc_geometry(wd, xd, g)) return false;
    // the per-K-group index of the group plus two stages (one K-group of activations and its dense weights
    // each) must fit the shared memory
    const size_t meta = align_up((size_t)L.tc.n_kc * 8, 1024);
    size_t per_kc;
    if (g.gemm) {
        if ((long long)xd.N * xd.L * xd.J > 0x7FFFFFFF) return false;
        per_kc = (size_t)256 * 32 + (size_t)kTcGroupRows * L.tc.st_bytes;       // up to 256 positions per CTA
    } else {
        per_kc = (size_t)g.n_phase * ((size_t)g.R * g.PW * 16 * (wd.H * wd.K == 1 ? 2 : 1) + 128) + (size_t)kTcGroupRows * L.tc.st_bytes;
    }
    return 2 * (per_kc + 1024) + meta + 1024 <= (size_t)kTcMaxSmem;
}

bsp_status launch_conv_tc(const bsp_wdesc &wd, const bsp_xdesc &xd, const void *packed, const void *X,
                          const void *bias, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st)
{
    const PackedLayout L = packed_layout(wd, 0);
    const TcLayout &T = L.tc;
    const uint8_t *pk = (const uint8_t *)packed;
    TcGeo geo;
    if (!tc_geometry(wd, xd, geo)) return BSP_ERR_SHAPE;
    const bool gemm = geo.gemm;
    const long long n_pos = (long long)xd.N * xd.L * xd.J;      // positions of a 1x1 layer, taken as one long row
    TcParams p = {};
    p.Y = (uint8_t *)Y; p.bias = (const float *)bias;
    p.mask = pk + T.off_mask; p.off = (const uint32_t *)(pk + T.off_off); p.gcnt = (const uint32_t *)(pk + T.off_gcnt);
    p.packed = pk; p.status = (int *)ws;
    p.N = xd.N; p.O = wd.O; p.H = wd.H; p.K = wd.K; p.ph = xd.pad_h; p.pw = xd.pad_w;
    p.M = geo.M; p.Nw = geo.Nw;
    p.sh = xd.stride_h; p.sw = xd.stride_w; p.n_phase = geo.n_phase;
    for (int i = 0; i < 4; ++i) { p.ph_a[i] = geo.ph_a[i]; p.ph_b[i] = geo.ph_b[i]; }
    p.P = xd.N * p.M * p.Nw;
    p.is_gemm = gemm ? 1 : 0;
    const int esz = wd.wtype == BSP_I8 ? 1 : 2;
    p.n_kc = T.n_kc; p.n_units = T.n_units; p.st_bytes = T.st_bytes; p.chunks_per_kc = T.kc_ch * esz / 16;
    p.coords_per_kc = gemm ? 1 : p.chunks_per_kc;
    p.mt = 1;
    int plane_pos, R = 1;
    long long tiles;
    if (gemm) {
        // large products take 256 positions per CTA when that still leaves two waves of CTAs
        p.mt = ((n_pos + 255) / 256) * T.n_groups >= 2 * 148 ? 2 : 1;
        p.PW = 1; plane_pos = 128 * p.mt; p.tiles_per_img = 0; tiles = (n_pos + plane_pos - 1) / plane_pos;
    } else {
        p.PW = geo.PW;
        R = geo.R;
        plane_pos = R * p.PW;
        p.tiles_per_img = (p.M * p.PW + 127) / 128;
        tiles = (long long)xd.N * p.tiles_per_img;
    }
    p.plane_bytes = plane_pos * 16;
    // The largest matrix products take two channel groups per CTA as well (256 positions x 256 channels: every
    // activation byte fetched from L2 then feeds twice the arithmetic), while the grid still fills the SMs twice.
    p.ng = 1; p.n_groups = T.n_groups;
    if (gemm && p.mt == 2 && T.n_groups >= 2 && tiles * ((T.n_groups + 1) / 2) >= 2 * 148) p.ng = 2;
    // (several phases: each plane set is padded to 128 bytes)
    const size_t per_kc = (size_t)p.n_phase * (p.plane_bytes * p.chunks_per_kc + (p.n_phase > 1 ? 128 : 0)) + (size_t)p.ng * kTcGroupRows * T.st_bytes;
    // K-groups per stage: about 64 KB of operands, i.e. three stages in flight; every stage costs the loop threads a
    // wait, a commit and their own bookkeeping, so fewer, larger stages win as long as three remain (measured: 48 KB
    // stages 0.328 ms, 64 KB 0.304 ms, 96 KB 0.343 ms on the 4096x4096x8192 product)
    int GK = (int)(kTcStageBudget / per_kc);
    if (GK < 1) GK = 1;
    if (GK > T.n_kc) GK = T.n_kc;
    if (GK * p.chunks_per_kc > 256) GK = 256 / p.chunks_per_kc;
    p.GK = GK;
    p.act_box_bytes = GK * p.chunks_per_kc * p.plane_bytes;
    // every tiled load must land on a 128-byte boundary of shared memory: the phases' plane sets are padded to that
    p.phase_bytes = (int)align_up((size_t)p.act_box_bytes, 128);
    p.act_bytes = (int)align_up((size_t)p.n_phase * p.phase_bytes + 32, 128);        // + slack read by positions in the padding
    p.w_stride = GK * kTcGroupRows * T.st_bytes;
    p.stage_bytes = (int)align_up((size_t)p.act_bytes + (size_t)p.ng * p.w_stride, 1024);
    p.n_stage_iters = (T.n_kc + GK - 1) / GK;
    const size_t meta = align_up((size_t)p.ng * T.n_kc * 8, 1024);
    int stages = (int)(((size_t)kTcMaxSmem - meta - 1024) / p.stage_bytes);
    if (stages > kTcMaxStages) stages = kTcMaxStages;
    if (stages > p.n_stage_iters) stages = p.n_stage_iters;
    if (stages < 1) return BSP_ERR_SHAPE;
    p.stages = stages;
    p.ytype = ytype;
    const size_t smem = meta + (size_t)stages * p.stage_bytes + 1024;

    EncodeTiledFn enc = tc_encode_tiled();
    if (!enc) return BSP_ERR_CUDA;
    const cuuint64_t row = (cuuint64_t)wd.I * esz;
    const cuuint64_t gJ = gemm ? 1 : (cuuint64_t)xd.J, gL = gemm ? 1 : (cuuint64_t)xd.L, gN = gemm ? (cuuint64_t)n_pos : (cuuint64_t)xd.N;
    // innermost extent: one 8-channel chunk (16 bytes), or for a matrix product a whole K-group (32 bytes, swizzled)
    const cuuint64_t inner = gemm ? 32 : 16;
    const cuuint64_t gdim[5] = {inner, gJ, gL, gN, (cuuint64_t)(row / inner)};
    const cuuint64_t gstr[4] = {row, row * gJ, row * gJ * gL, inner};
    cuuint32_t box[5];
    if (gemm) { box[0] = 32; box[1] = 1; box[2] = 1; box[3] = (cuuint32_t)(128 * p.mt); box[4] = (cuuint32_t)GK; }
    // a box traverses PW * s_w columns and R * s_h rows in steps of the strides: PW x R positions arrive
    else { box[0] = 16; box[1] = (cuuint32_t)(p.PW * p.sw); box[2] = (cuuint32_t)(R * p.sh); box[3] = 1; box[4] = (cuuint32_t)(GK * p.chunks_per_kc); }
    const cuuint32_t estr[5] = {1, gemm ? 1u : (cuuint32_t)p.sw, gemm ? 1u : (cuuint32_t)p.sh, 1, 1};
    if (enc(&p.tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 5, const_cast<void *>(X), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, gemm ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return BSP_ERR_CUDA;

    static bool opted[kTcMaxDevices] = {};
    int dev = 0;
    BSP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kTcMaxDevices) return BSP_ERR_CUDA;
    if (!opted[dev]) {
        BSP_CUDA_OK(cudaFuncSetAttribute(conv_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcMaxSmem));
        BSP_CUDA_OK(cudaFuncSetAttribute(conv_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcMaxSmem));
        opted[dev] = true;
    }
    dim3 grid((unsigned)tiles, (unsigned)((T.n_groups + p.ng - 1) / p.ng));
    if (wd.wtype == BSP_I8) conv_tc_kernel<true><<<grid, kTcThreads, smem, st>>>(p);
    else conv_tc_kernel<false><<<grid, kTcThreads, smem, st>>>(p);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // namespace bsp
