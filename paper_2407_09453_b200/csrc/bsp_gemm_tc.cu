// Block-sparse products Y = W*X + b on 5th-generation tensor cores, one kernel for all of them: the matrix product
// Y[p][o] = b[o] + sum over kept blocks of W-bar X (a fully connected layer, "GEMM is a 1x1 convolution") and the NHWC
// convolution with any taps, strides and zero padding, as an implicit GEMM.  tcgen05.mma with the accumulators in
// tensor memory: bf16 -> fp32 (kind::f16), int8 -> int32 (kind::i8), fp32 as TF32 -> fp32 (kind::tf32); fused bias;
// fp32, bf16, int32 or requantised int8 output.  Introduction (Y = W*X + b), Section "Block Sparsity in a Matrix" and
// Section "Compiler and its Code generation" (8-bit tensors with power-of-two scales) of the paper.
//
// The kernel reads the packed form Gamma (.) W in the layout of W, [O][H][K][I] (zeroed blocks stored as zeros), so
// that both operands arrive by tiled TMA loads under the 128-byte swizzle.  A persistent CTA owns tiles of up to 128
// output positions (a box of Wt x Ht positions of Nt images; 128 consecutive positions for a matrix product) x BN
// output channels (BN <= 256).  The reduction runs over taps x 128-byte chunks of input channels: per K-stage one
// thread issues two loads, the activation box shifted by the tap (out-of-bounds positions arrive as zeros: the
// padding; strides are the tensor map's element strides) and BN x 128 bytes of that tap's weights; one elected lane
// of the MMA warp issues four MMAs of 128 x BN x 32 bytes; two accumulator buffers of 256 columns let the epilogue of
// a tile (tensor memory -> registers -> + bias -> convert -> swizzled shared memory -> global memory, by TMA store
// when the tile's rows are consecutive in Y) overlap the MMAs of the next one.  The arithmetic skips nothing: a
// tensor-core instruction covers 128 x BN x 16 entries of the operands at once, far more than a block, and feeding it
// compact blocks (cp.async expansion of the block-CSR payload in shared memory, or TMA gather loads of 128-byte
// cores) was measured two to five times slower than these dense loads.
//
// Warps: 0 producer and 1 MMA issuer (each runs its loop as a whole, converged warp with warp-uniform values; one
// elected lane issues), 2-9 epilogue in two groups of four (warp w reads the tensor-memory lanes 32 (w % 4) ..; group g
// drains accumulator buffer g, so the epilogues of two consecutive tiles overlap).  Barriers per stage: full (one
// arrival that announces the bytes of both loads) and empty (tcgen05.commit); per accumulator buffer: acc_full (commit)
// and acc_empty (4 warps).  Every wait is bounded; on expiry BSP_ERR_TIMEOUT is latched, the roles wind down, loads
// in flight are awaited (bounded) and tensor memory is freed.
#include "bsp_tc.cuh"

namespace bsp {
namespace {

struct GtParams {
    CUtensorMap tmx;          // X as bytes: (I * esz, J, L, N), box 128 bytes x Wt x Ht x Nt positions (in steps of the strides), 128-byte swizzle
    CUtensorMap tmw;          // Gamma (.) W as bytes: (I * esz, H K, O), box 128 bytes x 1 tap x BN channels, 128-byte swizzle
    CUtensorMap tmy;          // Y as bytes: (O * ey, N_w, M, N), box 128 bytes x Wt x Ht x Nt positions (a tile), 128-byte swizzle
    const void *bias;         // float32 or int32 [O], may be NULL
    const int32_t *shift;     // int8 output only: right shift per output channel, 0..31
    const uint8_t *packed;
    int *status;
    int O, I, P, H, K, bo, bi, wtype, ytype;
    int BN, n_tiles_n, n_tiles, n_tile_pairs, n_ks;
    int stages, stage_bytes;
    // position tiles: Wt x Ht output positions of Nt images (at most 128), tiles_x x tiles_y of them per Nt images
    int N, M, Nw, Wt, Ht, Nt, tiles_x, tiles_y, rows_tile;
    int sh, sw, ph, pw, cpt;          // strides, padding, 128-byte channel chunks per tap
    int a_bytes;                      // bytes of one activation box
    uint8_t *Y;
    int ey;
    uint32_t m_ntn, m_tx, m_ty;       // floor(2^32 / d) of n_tiles_n, tiles_x, tiles_y (division by multiplication)
    int kbytes, a_stride;             // bytes of K per row of a stage: 128, or 64 for layers with at most 64 bytes of input channels; bytes of the activation part of a stage
};

// First output position (image, row, column) of position tile mt.
__device__ __forceinline__ void gt_tile_origin(const GtParams &p, int mt, int &n0, int &y0, int &x0)
{
    int r, tx, ty, ni;
    gt_divmod(mt, p.tiles_x, p.m_tx, r, tx);
    gt_divmod(r, p.tiles_y, p.m_ty, ni, ty);
    x0 = tx * p.Wt; y0 = ty * p.Ht; n0 = ni * p.Nt;
}

// Bias of output channel ch as raw bits (float32 or int32), zero without a bias or past the last channel.
__device__ __forceinline__ uint32_t gt_bias(const GtParams &p, int ch)
{
    return (p.bias != nullptr && ch < p.O) ? __ldg((const uint32_t *)p.bias + ch) : 0u;
}

template <bool kPair>
__global__ void __launch_bounds__(kGtThreads, 1) gemm_tc_kernel(const __grid_constant__ GtParams p)
{
    extern __shared__ __align__(16) uint8_t gt_smem_raw[];
    uint8_t *smem = gt_smem_raw + ((1024u - (sm32(gt_smem_raw) & 1023u)) & 1023u);
    __shared__ __align__(8) uint64_t s_full[kGtMaxStages], s_empty[kGtMaxStages];
    __shared__ __align__(8) uint64_t s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem;
    __shared__ volatile uint32_t s_fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int S = p.stages, n_ks = p.n_ks, BN = p.BN;
    const uint32_t ring = sm32(smem);
    const uint32_t staging = ring + (uint32_t)(S * p.stage_bytes);
    // Work items: tiles, or for CTA pairs two position tiles side by side on one channel tile (CTA r of the pair takes
    // position tile 2 mp + r; a pair past an odd count loads zeros and stores nothing).
    uint32_t rank = 0;
    if constexpr (kPair) asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(rank));
    const int t_first = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, t_step = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int t_count = kPair ? p.n_tile_pairs : p.n_tiles;
    // barriers of the pair's leader (CTA 0), as shared::cluster addresses
    uint32_t lead_full0 = sm32(&s_full[0]), lead_acc_empty0 = sm32(&s_acc_empty[0]);
    if constexpr (kPair) {
        asm volatile("mapa.shared::cluster.u32 %0, %1, 0;\n" : "=r"(lead_full0) : "r"(sm32(&s_full[0])));
        asm volatile("mapa.shared::cluster.u32 %0, %1, 0;\n" : "=r"(lead_acc_empty0) : "r"(sm32(&s_acc_empty[0])));
    }

    if (tid == 0) {
        // the packed buffer must be the one bsp_compact filled for this descriptor, with the masked dense form in it
        const PackedHeader *h = (const PackedHeader *)p.packed;
        const bool ok = h->magic == kPackedMagic && h->dtype == p.wtype && h->O == p.O && h->I == p.I && h->H == p.H &&
                        h->K == p.K && h->bo == p.bo && h->bi == p.bi && (h->forms & kFormDense) != 0;
        s_fail = ok ? 0u : 2u;
        if (!ok) atomicMax(p.status, (int)BSP_ERR_INDEX);
        for (int s = 0; s < S; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_full[s])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_empty[s])), "r"(1) : "memory");
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_acc_full[b])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_acc_empty[b])), "r"(kPair ? 8 : 4) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmx) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmw) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmy) : "memory");
    }
    if (warp == 0) {
        if constexpr (kPair) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(sm32(&s_tmem)), "r"(kGtTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(sm32(&s_tmem)), "r"(kGtTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    gt_sync_all<kPair>();                   // (a pair: both CTAs' barriers are initialised before either signals the other)
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem = s_tmem;
    const bool run = s_fail == 0u;

    if (warp == 0) {
        // ================= producer =================
        // The whole warp runs the loop with warp-uniform values; one elected lane arms the barrier and issues the loads.
        if (run) {
            const uint32_t full0 = sm32(&s_full[0]), empty0 = sm32(&s_empty[0]);
            // (a pair: each CTA loads its own activation box and its half of the weight tile, all four loads announce their
            // bytes on the leader's barrier, which the leader arms with the total)
            const uint32_t stage_bytes = (uint32_t)p.stage_bytes;
            const uint32_t tx = (uint32_t)(p.a_bytes + (BN >> (kPair ? 1 : 0)) * p.kbytes) * (kPair ? 2u : 1u);
            const int cpt128 = p.cpt * 128, Kw = p.K, ntn = p.n_tiles_n;
            // (a fresh barrier counts as released: the wait on parity 1 of the first round returns at once)
            uint32_t slot = 0, epar = 1, issued = 0, dst = ring;
            bool ok = true;
            for (int tile = t_first; tile < t_count && ok; tile += t_step) {
                int mt, tn;
                gt_divmod(tile, ntn, p.m_ntn, mt, tn);
                const int ch0 = tn * BN + (kPair ? (int)rank * (BN >> 1) : 0);
                int n0, y0, x0;
                gt_tile_origin(p, kPair ? 2 * mt + (int)rank : mt, n0, y0, x0);
                // input position of the tile's first output position at tap (0, 0); a tap is a shift of the box, positions
                // outside the image read as zeros (the padding)
                const int xi0 = x0 * p.sw - p.pw;
                int c128 = 0, kx = xi0, hy = y0 * p.sh - p.ph, tap = 0, kk = 0;
                if (s_fail) { ok = false; break; }
                for (int ks = 0; ks < n_ks; ++ks) {
                    bool got = gt_poll(empty0 + slot * 8u, epar);
                    got = __all_sync(0xFFFFFFFFu, got);
                    if (!got) { ok = false; break; }
                    if constexpr (kPair) {
                        asm volatile("{\n .reg .pred e, l;\n elect.sync _|e, 0xFFFFFFFF;\n setp.eq.u32 l, %12, 0;\n and.pred l, l, e;\n"
                                     " @l mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n"
                                     " @e cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%2], [%3, {%4, %5, %6, %7}], [%13];\n"
                                     " @e cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%8], [%9, {%4, %10, %11}], [%13];\n}\n"
                                     ::"r"(full0 + slot * 8u), "r"(tx), "r"(dst), "l"(&p.tmx), "r"(c128), "r"(kx), "r"(hy), "r"(n0),
                                       "r"(dst + (uint32_t)p.a_stride), "l"(&p.tmw), "r"(tap), "r"(ch0), "r"(rank), "r"(lead_full0 + slot * 8u) : "memory");
                    } else {
                        asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xFFFFFFFF;\n"
                                     " @e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n"
                                     " @e cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%2], [%3, {%4, %5, %6, %7}], [%0];\n"
                                     " @e cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%8], [%9, {%4, %10, %11}], [%0];\n}\n"
                                     ::"r"(full0 + slot * 8u), "r"(tx), "r"(dst), "l"(&p.tmx), "r"(c128), "r"(kx), "r"(hy), "r"(n0),
                                       "r"(dst + (uint32_t)p.a_stride), "l"(&p.tmw), "r"(tap), "r"(ch0) : "memory");
                    }
                    ++issued;
                    if (++slot == (uint32_t)S) { slot = 0; epar ^= 1u; dst = ring; } else dst += stage_bytes;
                    // next K-stage: the next 128-byte chunk of channels, then the next tap (columns first)
                    c128 += 128;
                    if (c128 == cpt128) {
                        c128 = 0; ++tap; ++kx;
                        if (++kk == Kw) { kk = 0; kx = xi0; ++hy; }
                    }
                }
            }
            if (!ok && lane == 0) {
                // winding down after a wait that ran out: the loads already issued still write into this CTA's shared
                // memory, so the barriers of the stages in flight are awaited (bounded) before the CTA may leave
                atomicExch((uint32_t *)&s_fail, 1u);
                // (the follower of a pair has no barrier of its own to watch: its loads announce themselves to the leader;
                // both CTAs meet at the cluster barrier before they leave)
                for (uint32_t back = 0; back < (uint32_t)S && back < issued && rank == 0; ++back) {
                    const uint32_t it = issued - 1u - back;
                    gt_poll(full0 + (it % (uint32_t)S) * 8u, (it / (uint32_t)S) & 1u);
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // The whole warp runs the loop (so that its address arithmetic stays warp-uniform); one elected lane issues.
        if (run && rank == 0) {               // (of a pair, the leader issues for both CTAs)
            // instruction descriptor: D fp32 (int32 for int8), A and B bf16 / signed int8 / tf32, K-major both, M = 128
            // (256 over a pair), N = BN
            const uint32_t dfmt = p.wtype == BSP_I8 ? 2u : 1u, abfmt = p.wtype == BSP_F32 ? 2u : 1u;
            const uint32_t idesc = (dfmt << 4) | (abfmt << 7) | (abfmt << 10) | ((uint32_t)(BN >> 3) << 17) | (((kPair ? 256u : 128u) >> 4) << 24);
            const uint32_t full0 = sm32(&s_full[0]), empty0 = sm32(&s_empty[0]);
            const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4, astride16 = (uint32_t)p.a_stride >> 4;
            const uint64_t desc0 = p.kbytes == 64 ? kGtDesc64 : kGtDesc;
            const uint32_t nk = (uint32_t)p.kbytes >> 5;            // MMAs per stage: 32 bytes of K each
            uint32_t slot = 0, par = 0, a16 = ring >> 4, tile_i = 0;
            bool ok = true;
            for (int tile = t_first; tile < t_count && ok; tile += t_step, ++tile_i) {
                const uint32_t buf = tile_i & 1u, use = tile_i >> 1;
                if (!gt_poll(sm32(&s_acc_empty[buf]), (use & 1u) ^ 1u) || s_fail != 0u) ok = false;   // (a fresh barrier counts as released)
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const uint32_t d = tmem + buf * 256u;
                for (int ks = 0; ks < n_ks; ++ks) {
                    bool got = gt_poll(full0 + slot * 8u, par);
                    got = __all_sync(0xFFFFFFFFu, got);
                    if (!got) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                    const uint64_t da = desc0 | (uint64_t)(a16 & 0x3FFFu), db = desc0 | (uint64_t)((a16 + astride16) & 0x3FFFu);
                    gt_issue_stage<kPair>(p.wtype, d, da, db, idesc, empty0 + slot * 8u, ks != 0 ? 1u : 0u, nk);
                    if (++slot == (uint32_t)S) { slot = 0; par ^= 1u; a16 = ring >> 4; } else a16 += stage16;
                }
                if (ok) gt_commit_elected<kPair>(sm32(&s_acc_full[buf]));
            }
            if (!ok && lane == 0) atomicExch((uint32_t *)&s_fail, 1u);
        }
    } else {
        // ================= epilogue (warps 2-9) =================
        // Two groups of four warps: group g drains accumulator buffer g, that is every second tile of the CTA, so the
        // epilogues of two consecutive tiles run side by side.
        if (run) {
            const int q = warp & 3;                              // quarter of the tensor-memory lanes this warp reaches
            const int ew = warp - 2, grp = ew >> 2;
            const int ey = p.ey;
            const int cpr = 128 / ey;                            // output channels per staging round (128 bytes of a row)
            // the group's staging buffer: 128 rows of 128 bytes, this warp's 32 rows at its quarter
            const uint32_t sg = staging + (uint32_t)(grp * 4 * kGtStagingBytes), sb = sg + (uint32_t)(q * kGtStagingBytes);
            const bool issuer = q == 0 && lane == 0;             // one thread of the group issues its stores
            uint32_t tile_i = (uint32_t)grp;
            bool ok = true;
            for (int tile = t_first + grp * t_step; tile < t_count && ok; tile += 2 * t_step, tile_i += 2) {
                const uint32_t buf = tile_i & 1u, use = tile_i >> 1;
                int mt, tn;
                gt_divmod(tile, p.n_tiles_n, p.m_ntn, mt, tn);
                const int n0 = tn * BN;
                int in0, y0, x0;
                gt_tile_origin(p, kPair ? 2 * mt + (int)rank : mt, in0, y0, x0);
                if (!gt_wait(sm32(&s_acc_full[buf]), use & 1u)) ok = false;
                if (s_fail) ok = false;
                ok = gt_group_all(1 + grp, ok);                // the four warps go on or give up as one (they meet at barriers below)
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const uint32_t tbase = tmem + ((uint32_t)(q * 32) << 16) + buf * 256u;
                for (int c0 = 0; c0 < BN; c0 += cpr) {
                    uint32_t out[32];                            // 128 bytes of this lane's row of Y
                    if (ey == 4) {                               // fp32 or int32 output: 32 channels
                        uint32_t v[32];
                        gt_load32(tbase + (uint32_t)c0, v);
                        const uint32_t bl = gt_bias(p, n0 + c0 + lane);      // lane e holds the bias of channel c0 + e
                        if (p.wtype == BSP_I8) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) out[e] = (uint32_t)((int)v[e] + (int)__shfl_sync(0xFFFFFFFFu, bl, e));
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                out[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(__shfl_sync(0xFFFFFFFFu, bl, e)));
                        }
                    } else if (ey == 1) {                        // int8 output: 128 channels, requantised after the bias
#pragma unroll
                        for (int sub = 0; sub < 4; ++sub) {
                            // (32-channel pieces past the tile or past the last channel are not computed: their bytes are clipped by the store)
                            if (c0 + sub * 32 >= BN || n0 + c0 + sub * 32 >= p.O) {
#pragma unroll
                                for (int e = 0; e < 8; ++e) out[sub * 8 + e] = 0u;
                                continue;
                            }
                            uint32_t v[32];
                            gt_load32(tbase + (uint32_t)(c0 + sub * 32), v);
                            const int ch = n0 + c0 + sub * 32 + lane;
                            const uint32_t bl = gt_bias(p, ch);
                            const uint32_t sl = ch < p.O ? (uint32_t)__ldg(p.shift + ch) & 31u : 0u;
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                int r4[4];
#pragma unroll
                                for (int b = 0; b < 4; ++b)
                                    r4[b] = gt_round_shift((int)v[4 * e + b] + (int)__shfl_sync(0xFFFFFFFFu, bl, 4 * e + b),
                                                           __shfl_sync(0xFFFFFFFFu, sl, 4 * e + b));
                                out[sub * 8 + e] = gt_pack_s8x4(r4[0], r4[1], r4[2], r4[3]);
                            }
                        }
                    } else {                                     // bf16 output: 64 channels, rounded to nearest even after the bias
#pragma unroll
                        for (int sub = 0; sub < 2; ++sub) {
                            uint32_t v[32];
                            gt_load32(tbase + (uint32_t)(c0 + sub * 32), v);
                            const uint32_t bl = gt_bias(p, n0 + c0 + sub * 32 + lane);
#pragma unroll
                            for (int e = 0; e < 16; ++e) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(
                                    __uint_as_float(v[2 * e]) + __uint_as_float(__shfl_sync(0xFFFFFFFFu, bl, 2 * e)),
                                    __uint_as_float(v[2 * e + 1]) + __uint_as_float(__shfl_sync(0xFFFFFFFFu, bl, 2 * e + 1)));
                                out[sub * 16 + e] = *(const uint32_t *)&h;
                            }
                        }
                    }
                    // the staging buffer was handed to a TMA store in the previous round: the issuing thread waits until it
                    // has been read (the loads and the arithmetic of this round ran meanwhile), then the group may write
                    if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory");
                    gt_group_sync(1 + grp);
                    const uint32_t srow = sb + (uint32_t)lane * 128u;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};\n"
                                     ::"r"(srow + (uint32_t)((j ^ (lane & 7)) << 4)), "r"(out[4 * j]), "r"(out[4 * j + 1]), "r"(out[4 * j + 2]), "r"(out[4 * j + 3]) : "memory");
                    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    gt_group_sync(1 + grp);
                    // one store of the tile's box: 128 bytes of every row; what lies past the last channel, column, row or image
                    // of Y is clipped (rows of the buffer beyond the box are not part of the store)
                    if (issuer && n0 + c0 < p.O) {
                        asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];\n"
                                     ::"l"(&p.tmy), "r"(sg), "r"((n0 + c0) * ey), "r"(x0), "r"(y0), "r"(in0) : "memory");
                        asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
                    }
                }
                // the accumulator buffer has been read: hand it back to the MMA issuer
                asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    if constexpr (kPair)
                        asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(lead_acc_empty0 + buf * 8u) : "memory");
                    else
                        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(sm32(&s_acc_empty[buf])) : "memory");
                }
            }
            if (issuer) asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory");
            if (!ok && lane == 0) atomicExch((uint32_t *)&s_fail, 1u);
        }
    }

    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    gt_sync_all<kPair>();                   // (a pair: neither CTA leaves while the other may still signal its barriers)
    if (s_fail == 1u && tid == 0) atomicMax(p.status, (int)BSP_ERR_TIMEOUT);
    if (warp == 0) {
        if constexpr (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kGtTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kGtTmemCols) : "memory");
    }
}

}  // namespace


// True if the kernel can run this layer: rows of X, W and Y that are multiples of 16 bytes (tensor-map strides), a
// position count that fits 32 bits, and a position tile whose box the tensor map can express.
bool gemm_tc_eligible(const bsp_wdesc &wd, const bsp_xdesc &xd0, bsp_dtype ytype)
{
    const bsp_xdesc xd = gt_flatten(wd, xd0);
    if (!packed_layout(wd).enabled) return false;
    if (ytype != BSP_F32 && ytype != BSP_BF16 && ytype != BSP_I32 && ytype != BSP_I8) return false;
    const int ey = ytype == BSP_BF16 ? 2 : (ytype == BSP_I8 ? 1 : 4);
    if (((long long)wd.O * ey) % 16 != 0) return false;
    const int M = (xd.L + 2 * xd.pad_h - wd.H) / xd.stride_h + 1, Nw = (xd.J + 2 * xd.pad_w - wd.K) / xd.stride_w + 1;
    if (M <= 0 || Nw <= 0) return false;
    if ((long long)xd.N * M * Nw > 0x7FFFFFFF || (long long)xd.N * xd.L * xd.J > 0x7FFFFFFF) return false;
    if ((long long)xd.N * M * Nw * wd.O * ey >= (1LL << 46)) return false;
    return gt_pick_tile(xd.N, M, Nw, xd.stride_h, xd.stride_w).tiles > 0;
}

bsp_status launch_gemm_tc(const bsp_wdesc &wd, const bsp_xdesc &xd0, const void *packed, const void *X,
                          const void *bias, const int32_t *shift, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st)
{
    const bsp_xdesc xd = gt_flatten(wd, xd0);
    const PackedLayout L = packed_layout(wd);
    if (!L.enabled) return BSP_ERR_SHAPE;
    const int esz = elem_bytes(wd.wtype);
    const int ey = ytype == BSP_BF16 ? 2 : (ytype == BSP_I8 ? 1 : 4);
    const int HK = wd.H * wd.K;
    if (ytype == BSP_I8 && shift == nullptr) return BSP_ERR_NULL;
    GtParams p = {};
    p.bias = bias; p.shift = shift; p.packed = (const uint8_t *)packed;
    p.status = (int *)ws;
    p.O = wd.O; p.I = wd.I; p.H = wd.H; p.K = wd.K; p.bo = wd.bo; p.bi = wd.bi;
    p.wtype = wd.wtype; p.ytype = ytype; p.ey = ey; p.Y = (uint8_t *)Y;
    p.N = xd.N; p.sh = xd.stride_h; p.sw = xd.stride_w; p.ph = xd.pad_h; p.pw = xd.pad_w;
    p.M = (xd.L + 2 * xd.pad_h - wd.H) / xd.stride_h + 1;
    p.Nw = (xd.J + 2 * xd.pad_w - wd.K) / xd.stride_w + 1;
    const long long P = (long long)xd.N * p.M * p.Nw;
    p.P = (int)P;
    const GtTile T = gt_pick_tile(xd.N, p.M, p.Nw, p.sh, p.sw);
    if (T.tiles <= 0) return BSP_ERR_SHAPE;
    p.Wt = T.Wt; p.Ht = T.Ht; p.Nt = T.Nt; p.rows_tile = T.Wt * T.Ht * T.Nt;
    p.tiles_x = (p.Nw + T.Wt - 1) / T.Wt; p.tiles_y = (p.M + T.Ht - 1) / T.Ht;
    // layers with at most 64 bytes of input channels per position stage 64-byte rows (64-byte swizzle, two MMAs a stage)
    p.kbytes = (long long)wd.I * esz <= 64 ? 64 : 128;
    p.a_stride = kGtBM * p.kbytes;
    p.a_bytes = p.rows_tile * p.kbytes;
    static bool opted[kGtMaxDevices] = {};
    static int n_sm[kGtMaxDevices] = {};
    int dev = 0;
    BSP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kGtMaxDevices) return BSP_ERR_CUDA;
    if (!opted[dev]) {
        BSP_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGtMaxSmem));
        BSP_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGtMaxSmem));
        BSP_CUDA_OK(cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev));
        opted[dev] = true;
    }
    // Channels per tile: the widest tile keeps the tensor pipe busiest (a stage costs about 256 + 2 BN cycles of operand
    // fetch from shared memory), but a layer with few position tiles fills more SMs with narrower ones: the width with
    // the lowest waves x stage cost wins.
    {
        const int step = 64;
        const int widest = (gemm_tile_n(wd.O) + step - 1) / step * step;
        long long best_cost = -1;
        for (int bn = widest; bn >= step; bn -= step) {
            if (bn != widest && bn != 128 && bn != 64) continue;
            // (a round of the int8 output stores 128 channels: a tile that is not a multiple of that must be the only one)
            if (ytype == BSP_I8 && bn % 128 != 0 && bn < wd.O) continue;
            const long long tiles = T.tiles * ((wd.O + bn - 1) / bn);
            const long long cost = ((tiles + n_sm[dev] - 1) / n_sm[dev]) * (256 + 2 * bn);
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; p.BN = bn; }
        }
    }
    p.n_tiles_n = (wd.O + p.BN - 1) / p.BN;
    if (T.tiles * p.n_tiles_n > 0x7FFFFFFF - 4096) return BSP_ERR_SHAPE;      // (tile counters step by up to twice the grid)
    p.n_tiles = (int)(T.tiles * p.n_tiles_n);
    // Large products run on CTA pairs: two position tiles side by side on one 256-channel tile, every CTA loading its
    // own activations and half of the weights (the operand fetch per SM and MMA falls from 12 KB to 8 KB).
    // (Tiles of a few K-stages are bound by their epilogue, and there the pair's cross-CTA hand-shakes only cost.)
    p.cpt = (int)(((long long)wd.I * esz + 127) / 128);
    p.n_ks = HK * p.cpt;
    const bool pair = p.kbytes == 128 && p.BN == 256 && p.n_ks >= 8 && (long long)p.n_tiles >= 4LL * n_sm[dev] && n_sm[dev] >= 2;
    p.n_tile_pairs = (int)(((T.tiles + 1) / 2) * p.n_tiles_n);
    p.m_ntn = gt_magic(p.n_tiles_n); p.m_tx = gt_magic(p.tiles_x); p.m_ty = gt_magic(p.tiles_y);
    p.stage_bytes = p.a_stride + (pair ? p.BN / 2 : p.BN) * p.kbytes;
    const int staging = 8 * kGtStagingBytes;
    int stages = (kGtMaxSmem - 1024 - staging) / p.stage_bytes;
    if (stages > kGtMaxStages) stages = kGtMaxStages;
    if (stages < 2) return BSP_ERR_SHAPE;
    p.stages = stages;
    const size_t smem = 1024 + (size_t)stages * p.stage_bytes + staging;

    GtEncodeFn enc = gt_encode();
    if (!enc) return BSP_ERR_CUDA;
    {
        const cuuint64_t row = (cuuint64_t)wd.I * esz;
        const cuuint64_t gdim[4] = {row, (cuuint64_t)xd.J, (cuuint64_t)xd.L, (cuuint64_t)xd.N};
        const cuuint64_t gstr[3] = {row, row * xd.J, row * xd.J * xd.L};
        // a box spans Wt * s_w x Ht * s_h input positions in steps of the strides: Wt x Ht positions arrive
        const cuuint32_t box[4] = {(cuuint32_t)p.kbytes, (cuuint32_t)(T.Wt * p.sw), (cuuint32_t)(T.Ht * p.sh), (cuuint32_t)T.Nt};
        const cuuint32_t estr[4] = {1, (cuuint32_t)p.sw, (cuuint32_t)p.sh, 1};
        if (enc(&p.tmx, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(X), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                p.kbytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }
    {
        const cuuint64_t row = (cuuint64_t)wd.I * esz;
        const cuuint64_t gdim[3] = {row, (cuuint64_t)HK, (cuuint64_t)wd.O};
        const cuuint64_t gstr[2] = {row, row * HK};
        const cuuint32_t box[3] = {(cuuint32_t)p.kbytes, 1, (cuuint32_t)(pair ? p.BN / 2 : p.BN)};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&p.tmw, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>((const uint8_t *)packed + L.off_payload), gdim, gstr, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, p.kbytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }
    {
        const cuuint64_t row = (cuuint64_t)wd.O * ey;
        const cuuint64_t gdim[4] = {row, (cuuint64_t)p.Nw, (cuuint64_t)p.M, (cuuint64_t)xd.N};
        const cuuint64_t gstr[3] = {row, row * p.Nw, row * p.Nw * p.M};
        const cuuint32_t box[4] = {128, (cuuint32_t)T.Wt, (cuuint32_t)T.Ht, (cuuint32_t)T.Nt};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(&p.tmy, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, Y, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }

    if (pair) {
        cudaLaunchConfig_t cfg = {};
        const int pairs = p.n_tile_pairs < n_sm[dev] / 2 ? p.n_tile_pairs : n_sm[dev] / 2;
        cfg.gridDim = dim3((unsigned)(2 * pairs));
        cfg.blockDim = dim3(kGtThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        BSP_CUDA_OK(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<true>, p));
        return BSP_OK;
    }
    const int grid = p.n_tiles < n_sm[dev] ? p.n_tiles : n_sm[dev];
    gemm_tc_kernel<false><<<grid, kGtThreads, smem, st>>>(p);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // namespace bsp
