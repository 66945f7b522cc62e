// Two consecutive block-sparse layers in one kernel: T = act(W1 * X + b1) stored as bfloat16, Y = W2 * T + b2 with a 1x1
// second layer; or the 8-bit chain, where T is the requantised int8 output of layer one (Section "Compiler and its Code
// generation": power-of-two scales) and Y is int32 or requantised int8.  Section "Depth-wise Tiling" of the paper: the output is cut into tiles, every tile is carried through
// the whole chain, and the tensor between the layers never goes to external memory.  A 1x1 second layer needs no
// overlap between tiles (its projection of one output position is one position of T), so the tiles are those of the
// first layer.
//
// Per tile of up to 128 output positions a persistent CTA runs
//   1. the first layer as an implicit GEMM over taps x 128-byte channel chunks (activation box + weight tile per
//      K-stage, both by tiled TMA loads) into accumulator one, all O1 <= 256 channels in tensor memory;
//   2. its epilogue: tensor memory -> registers -> + b1 -> max(., 0) if asked -> bfloat16 (int8: rounding shift, then
//      max(., 0)) -> shared memory, written in the K-major 128-byte-swizzled layout that an MMA reads as its A operand
//      (128 bytes of channels, that is 64 bfloat16 or 128 int8, per 16 KB chunk);
//   3. the second layer: for every tile of 128 output channels, MMAs of that tensor against weight chunks that arrive
//      through the same ring of stages, into one of two 128-column accumulators;
//   4. its epilogue: + b2 -> convert -> global memory, overlapping the MMAs of the next 128 channels.
// Warps: 0 producer, 1 MMA issuer (both converged, one elected lane issues), 2-9 epilogue in two groups of four: the
// groups share the first epilogue (alternate 64-channel chunks) and each drains one of the two second accumulators.
// Every wait is bounded.
#include "bsp_tc.cuh"

namespace bsp {
namespace {

constexpr int kCtThreads = 320;                    // producer warp, MMA warp, two groups of four epilogue warps
constexpr int kCtBN2 = 128;                        // channels of layer two per accumulator buffer
constexpr int kCtChunk = kGtBM * 128;              // bytes of one chunk (128 bytes of channels) of the tensor between the layers

struct CtParams {
    CUtensorMap tmx;          // X as bytes: (I1 * 2, J, L, N), box 128 bytes x Wt x Ht x Nt positions
    CUtensorMap tmw1;         // Gamma1 (.) W1 as bytes: (I1 * 2, H K, O1), box 128 bytes x 1 tap x O1p channels
    CUtensorMap tmw2;         // Gamma2 (.) W2 as bytes: (O1 * 2, 1, O2), box 128 bytes x 1 x 128 channels
    CUtensorMap tmy;          // Y as bytes: (O2 * ey, N_w, M, N), box 128 bytes x Wt x Ht x Nt positions (a tile)
    const void *bias1, *bias2;        // float32, or int32 for the 8-bit chain
    const int32_t *shift1, *shift2;   // 8-bit chain: rounding shifts of T (required) and of an int8 Y
    const uint8_t *packed1, *packed2;
    int *status;
    int O1, I1, H, K, bo1, bi1, O2, bo2, bi2, relu, wtype, ytype, ey;
    int O1p;                  // O1 rounded up to a whole chunk of T (64 or 128 channels): columns of accumulator one
    int tcc;                  // channels per chunk of T: 64 (bfloat16) or 128 (int8)
    int n_ks1, cpt1, n_c2, n_t2;      // K-stages of layer one, its channel chunks per tap; chunks of T; channel tiles of layer two
    int stages, stage_bytes, n_tiles;
    int db;                   // O1p <= 128: accumulator one and the tensor between the layers are double-buffered
    int N, M, Nw, Wt, Ht, Nt, tiles_x, tiles_y, rows_tile, P;
    int sh, sw, ph, pw, a_bytes;
    uint32_t m_tx, m_ty;
    uint8_t *Y;
};

__device__ __forceinline__ void ct_tile_origin(const CtParams &p, int mt, int &n0, int &y0, int &x0)
{
    int r, tx, ty, ni;
    gt_divmod(mt, p.tiles_x, p.m_tx, r, tx);
    gt_divmod(r, p.tiles_y, p.m_ty, ni, ty);
    x0 = tx * p.Wt; y0 = ty * p.Ht; n0 = ni * p.Nt;
}

__device__ __forceinline__ bool ct_header_ok(const uint8_t *packed, int wtype, int O, int I, int H, int K, int bo, int bi)
{
    const PackedHeader *h = (const PackedHeader *)packed;
    return h->magic == kPackedMagic && h->dtype == wtype && h->O == O && h->I == I && h->H == H && h->K == K && h->bo == bo &&
           h->bi == bi && (h->forms & kFormDense) != 0;
}

// kI8: the 8-bit chain (compiled apart, so that neither form carries the other's epilogue code and registers).
template <bool kI8>
__global__ void __launch_bounds__(kCtThreads, 1) chain_tc_kernel(const __grid_constant__ CtParams p)
{
    constexpr int kWt = kI8 ? BSP_I8 : BSP_BF16;
    extern __shared__ __align__(16) uint8_t ct_smem_raw[];
    uint8_t *smem = ct_smem_raw + ((1024u - (sm32(ct_smem_raw) & 1023u)) & 1023u);
    __shared__ __align__(8) uint64_t s_full[kGtMaxStages], s_empty[kGtMaxStages];
    __shared__ __align__(8) uint64_t s_acc1_full[2], s_acc1_empty[2], s_t_full[2], s_t_empty[2], s_acc2_full[2], s_acc2_empty[2];
    __shared__ uint32_t s_tmem;
    __shared__ volatile uint32_t s_fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int S = p.stages;
    const uint32_t ring = sm32(smem);
    const uint32_t tbuf = ring + (uint32_t)(S * p.stage_bytes);          // the tensor between the layers: n_c2 chunks
    const uint32_t tbytes = (uint32_t)(p.n_c2 * kCtChunk);
    const uint32_t staging = tbuf + (p.db ? 2u : 1u) * tbytes;
    const int t_first = (int)blockIdx.x, t_step = (int)gridDim.x, t_count = p.n_tiles;

    if (tid == 0) {
        const bool ok = ct_header_ok(p.packed1, p.wtype, p.O1, p.I1, p.H, p.K, p.bo1, p.bi1) && ct_header_ok(p.packed2, p.wtype, p.O2, p.O1, 1, 1, p.bo2, p.bi2);
        s_fail = ok ? 0u : 2u;
        if (!ok) atomicMax(p.status, (int)BSP_ERR_INDEX);
        for (int s = 0; s < S; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_full[s])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_empty[s])), "r"(1) : "memory");
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_acc1_full[b])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_acc1_empty[b])), "r"(8) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_t_full[b])), "r"(8) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_t_empty[b])), "r"(1) : "memory");
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_acc2_full[b])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(sm32(&s_acc2_empty[b])), "r"(4) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmx) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmw1) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmw2) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&p.tmy) : "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(sm32(&s_tmem)), "r"(kGtTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem = s_tmem;
    const bool run = s_fail == 0u;
    const uint32_t full0 = sm32(&s_full[0]), empty0 = sm32(&s_empty[0]);

    if (warp == 0) {
        // ================= producer =================
        if (run) {
            const uint32_t stage_bytes = (uint32_t)p.stage_bytes;
            const uint32_t tx1 = (uint32_t)(p.a_bytes + p.O1p * 128), tx2 = (uint32_t)(kCtBN2 * 128);
            const int cpt128 = p.cpt1 * 128, Kw = p.K;
            uint32_t slot = 0, epar = 1, issued = 0, dst = ring;      // (a fresh barrier counts as released)
            bool ok = true;
            // layer one of a tile: the activation box shifted by the tap and that tap's weights, per 128-byte chunk of channels
            auto load_layer_one = [&](int tile) {
                int n0, y0, x0;
                ct_tile_origin(p, tile, n0, y0, x0);
                const int xi0 = x0 * p.sw - p.pw;
                int c128 = 0, kx = xi0, hy = y0 * p.sh - p.ph, tap = 0, kk = 0;
                for (int ks = 0; ks < p.n_ks1; ++ks) {
                    bool got = gt_poll(empty0 + slot * 8u, epar);
                    got = __all_sync(0xFFFFFFFFu, got);
                    if (!got) { ok = false; return; }
                    asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xFFFFFFFF;\n"
                                 " @e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n"
                                 " @e cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%2], [%3, {%4, %5, %6, %7}], [%0];\n"
                                 " @e cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%8], [%9, {%4, %10, %11}], [%0];\n}\n"
                                 ::"r"(full0 + slot * 8u), "r"(tx1), "r"(dst), "l"(&p.tmx), "r"(c128), "r"(kx), "r"(hy), "r"(n0),
                                   "r"(dst + (uint32_t)kGtABytes), "l"(&p.tmw1), "r"(tap), "r"(0) : "memory");
                    ++issued;
                    if (++slot == (uint32_t)S) { slot = 0; epar ^= 1u; dst = ring; } else dst += stage_bytes;
                    c128 += 128;
                    if (c128 == cpt128) {
                        c128 = 0; ++tap; ++kx;
                        if (++kk == Kw) { kk = 0; kx = xi0; ++hy; }
                    }
                }
            };
            // layer two: for every tile of 128 output channels, the weight chunk of each 64 channels of T
            auto load_layer_two = [&]() {
                for (int t2 = 0; t2 < p.n_t2; ++t2)
                    for (int c2 = 0; c2 < p.n_c2; ++c2) {
                        bool got = gt_poll(empty0 + slot * 8u, epar);
                        got = __all_sync(0xFFFFFFFFu, got);
                        if (!got) { ok = false; return; }
                        asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xFFFFFFFF;\n"
                                     " @e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n"
                                     " @e cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%2], [%3, {%4, %5, %6}], [%0];\n}\n"
                                     ::"r"(full0 + slot * 8u), "r"(tx2), "r"(dst), "l"(&p.tmw2), "r"(c2 * 128), "r"(0), "r"(t2 * kCtBN2) : "memory");
                        ++issued;
                        if (++slot == (uint32_t)S) { slot = 0; epar ^= 1u; dst = ring; } else dst += stage_bytes;
                    }
            };
            // the stages follow the order in which the MMA warp consumes them: with double buffers, layer one of the next
            // tile goes before layer two of this one
            if (p.db && t_first < t_count) load_layer_one(t_first);
            for (int tile = t_first; tile < t_count && ok; tile += t_step) {
                if (s_fail) { ok = false; break; }
                if (p.db) { if (tile + t_step < t_count) load_layer_one(tile + t_step); }
                else load_layer_one(tile);
                if (ok) load_layer_two();
            }
            if (!ok && lane == 0) {
                // winding down after a wait that ran out: the loads already issued still write into this CTA's shared
                // memory, so the barriers of the stages in flight are awaited (bounded) before the CTA may leave
                atomicExch((uint32_t *)&s_fail, 1u);
                for (uint32_t back = 0; back < (uint32_t)S && back < issued; ++back) {
                    const uint32_t it = issued - 1u - back;
                    gt_poll(full0 + (it % (uint32_t)S) * 8u, (it / (uint32_t)S) & 1u);
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (run) {
            // instruction descriptors: A and B bf16 (signed int8), K-major both, M = 128; N = O1p for layer one, 128 for layer two
            const uint32_t dfmt = kI8 ? 2u : 1u;      // D int32 for int8 operands, fp32 otherwise
            const uint32_t idesc1 = (dfmt << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.O1p >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc2 = (dfmt << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kCtBN2 >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4;
            uint32_t slot = 0, par = 0, a16 = ring >> 4, tile_i = 0, u2 = 0;
            bool ok = true;
            // layer one of the CTA's i-th tile into accumulator one (buffer b, used for the u-th time)
            auto layer_one = [&](uint32_t i) {
                const uint32_t b = p.db ? (i & 1u) : 0u, u = p.db ? (i >> 1) : i;
                // the buffer is free once the first epilogue of its previous tile has read it
                if (!gt_poll(sm32(&s_acc1_empty[b]), (u & 1u) ^ 1u) || s_fail != 0u) ok = false;
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) return;
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const uint32_t d = tmem + b * 128u;
                for (int ks = 0; ks < p.n_ks1; ++ks) {
                    bool got = gt_poll(full0 + slot * 8u, par);
                    got = __all_sync(0xFFFFFFFFu, got);
                    if (!got) { ok = false; return; }
                    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                    const uint64_t da = kGtDesc | (uint64_t)(a16 & 0x3FFFu), db = kGtDesc | (uint64_t)((a16 + (kGtABytes >> 4)) & 0x3FFFu);
                    gt_issue_stage<false>(kWt, d, da, db, idesc1, empty0 + slot * 8u, ks != 0 ? 1u : 0u);
                    if (++slot == (uint32_t)S) { slot = 0; par ^= 1u; a16 = ring >> 4; } else a16 += stage16;
                }
                gt_commit_elected<false>(sm32(&s_acc1_full[b]));
            };
            // layer two of the i-th tile: the tensor between the layers is in shared memory once the first epilogue has written it
            auto layer_two = [&](uint32_t i) {
                const uint32_t b = p.db ? (i & 1u) : 0u, u = p.db ? (i >> 1) : i;
                if (!gt_poll(sm32(&s_t_full[b]), u & 1u)) ok = false;
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) return;
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                for (int t2 = 0; t2 < p.n_t2 && ok; ++t2, ++u2) {
                    const uint32_t buf = u2 & 1u, use = u2 >> 1;
                    if (!gt_poll(sm32(&s_acc2_empty[buf]), (use & 1u) ^ 1u)) ok = false;
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) return;
                    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                    const uint32_t d = tmem + 256u + buf * (uint32_t)kCtBN2;
                    for (int c2 = 0; c2 < p.n_c2; ++c2) {
                        bool got = gt_poll(full0 + slot * 8u, par);
                        got = __all_sync(0xFFFFFFFFu, got);
                        if (!got) { ok = false; return; }
                        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                        const uint64_t da = kGtDesc | (uint64_t)(((tbuf + b * tbytes + (uint32_t)(c2 * kCtChunk)) >> 4) & 0x3FFFu);
                        const uint64_t db = kGtDesc | (uint64_t)(a16 & 0x3FFFu);
                        gt_issue_stage<false>(kWt, d, da, db, idesc2, empty0 + slot * 8u, c2 != 0 ? 1u : 0u);
                        if (++slot == (uint32_t)S) { slot = 0; par ^= 1u; a16 = ring >> 4; } else a16 += stage16;
                    }
                    gt_commit_elected<false>(sm32(&s_acc2_full[buf]));
                }
                // all MMAs that read the tensor have been issued: their completion frees its buffer
                gt_commit_elected<false>(sm32(&s_t_empty[b]));
            };
            if (p.db && t_first < t_count) layer_one(0u);
            for (int tile = t_first; tile < t_count && ok; tile += t_step, ++tile_i) {
                if (p.db) { if (tile + t_step < t_count) layer_one(tile_i + 1u); }
                else layer_one(tile_i);
                if (ok) layer_two(tile_i);
            }
            if (!ok && lane == 0) atomicExch((uint32_t *)&s_fail, 1u);
        }
    } else {
        // ================= epilogues (warps 2-9) =================
        if (run) {
            const int q = warp & 3;                              // quarter of the tensor-memory lanes this warp reaches
            const int grp = (warp - 2) >> 2;
            const int ey = p.ey;
            const int cpr = 128 / ey;                            // output channels per staging round (128 bytes of a row)
            // the group's staging buffer: 128 rows of 128 bytes, this warp's 32 rows at its quarter
            const uint32_t sg = staging + (uint32_t)(grp * 4 * kGtStagingBytes), sb = sg + (uint32_t)(q * kGtStagingBytes);
            const bool issuer = q == 0 && lane == 0;             // one thread of the group issues its stores
            uint32_t tile_i = 0, u2 = 0;
            bool ok = true;
            const int r = q * 32 + lane;                         // this lane's row of a tile
            const uint32_t trow = tbuf + (uint32_t)r * 128u;     // this lane's row of a chunk of T (first buffer)
            for (int tile = t_first; tile < t_count && ok; tile += t_step, ++tile_i) {
                int in0, y0, x0;
                ct_tile_origin(p, tile, in0, y0, x0);
                // ---- first epilogue: accumulator one -> + b1 -> activation -> bfloat16 -> T in shared memory ----
                // (T may be overwritten once the MMAs of the previous tile's second layer have read it)
                const uint32_t b1 = p.db ? (tile_i & 1u) : 0u, u1 = p.db ? (tile_i >> 1) : tile_i;
                if (!gt_wait(sm32(&s_acc1_full[b1]), u1 & 1u) || !gt_wait(sm32(&s_t_empty[b1]), (u1 & 1u) ^ 1u)) ok = false;
                if (s_fail) ok = false;
                ok = gt_group_all(1 + grp, ok);                  // the four warps of a group go on or give up as one
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const uint32_t t1 = tmem + ((uint32_t)(q * 32) << 16);
                const uint32_t a1 = t1 + b1 * 128u;                  // this tile's accumulator one
                for (int c2 = grp; c2 < p.n_c2; c2 += 2) {
                    uint32_t out[32];                            // one chunk (128 bytes of channels) of this lane's row of T
                    if constexpr (kI8) {                         // 128 channels: + b1, rounding shift, activation, int8
#pragma unroll
                        for (int sub = 0; sub < 4; ++sub) {
                            if (c2 * 128 + sub * 32 >= p.O1) {       // (past the last channel of T: zeros, as the weights of layer two there)
#pragma unroll
                                for (int e = 0; e < 8; ++e) out[sub * 8 + e] = 0u;
                                continue;
                            }
                            uint32_t v[32];
                            gt_load32(a1 + (uint32_t)(c2 * 128 + sub * 32), v);
                            const int ch = c2 * 128 + sub * 32 + lane;
                            const int bl = (p.bias1 != nullptr && ch < p.O1) ? __ldg((const int *)p.bias1 + ch) : 0;   // lane e: channel .. + e
                            const uint32_t sl = ch < p.O1 ? (uint32_t)__ldg(p.shift1 + ch) & 31u : 0u;
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                int r4[4];
#pragma unroll
                                for (int b = 0; b < 4; ++b)
                                    r4[b] = gt_round_shift((int)v[4 * e + b] + __shfl_sync(0xFFFFFFFFu, bl, 4 * e + b),
                                                           __shfl_sync(0xFFFFFFFFu, sl, 4 * e + b));
                                uint32_t w = gt_pack_s8x4(r4[0], r4[1], r4[2], r4[3]);
                                if (p.relu) w = __vmaxs4(w, 0u);
                                out[sub * 8 + e] = w;
                            }
                        }
                    } else {
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub) {
                        uint32_t v[32];
                        gt_load32(a1 + (uint32_t)(c2 * 64 + sub * 32), v);
                        const int ch = c2 * 64 + sub * 32 + lane;
                        const float bl = (p.bias1 != nullptr && ch < p.O1) ? __ldg((const float *)p.bias1 + ch) : 0.f;     // lane e: bias of channel .. + e
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            float a = __uint_as_float(v[2 * e]) + __shfl_sync(0xFFFFFFFFu, bl, 2 * e);
                            float b = __uint_as_float(v[2 * e + 1]) + __shfl_sync(0xFFFFFFFFu, bl, 2 * e + 1);
                            if (p.relu) { a = fmaxf(a, 0.f); b = fmaxf(b, 0.f); }
                            const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                            out[sub * 16 + e] = *(const uint32_t *)&h;
                        }
                    }
                    }
                    // K-major rows of 128 bytes under the 128-byte swizzle: the 16-byte piece j of row r sits at piece j ^ (r % 8)
                    const uint32_t dst = trow + b1 * tbytes + (uint32_t)(c2 * kCtChunk);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};\n"
                                     ::"r"(dst + (uint32_t)((j ^ (lane & 7)) << 4)), "r"(out[4 * j]), "r"(out[4 * j + 1]), "r"(out[4 * j + 2]), "r"(out[4 * j + 3]) : "memory");
                }
                // the MMAs read T through the asynchronous proxy
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(sm32(&s_acc1_empty[b1])) : "memory");
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(sm32(&s_t_full[b1])) : "memory");
                }
                // ---- second epilogue, per tile of 128 output channels: + b2 -> convert -> Y ----
                for (int t2 = 0; t2 < p.n_t2 && ok; ++t2, ++u2) {
                    const uint32_t buf = u2 & 1u, use = u2 >> 1;
                    if ((int)buf != grp) continue;               // (the other group drains this accumulator)
                    const int n0 = t2 * kCtBN2;
                    if (!gt_wait(sm32(&s_acc2_full[buf]), use & 1u)) ok = false;
                    if (s_fail) ok = false;
                    ok = gt_group_all(1 + grp, ok);              // the four warps go on or give up as one (they meet at barriers below)
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                    const uint32_t t2base = t1 + 256u + buf * (uint32_t)kCtBN2;
                    for (int c0 = 0; c0 < kCtBN2; c0 += cpr) {
                        uint32_t out[32];                        // 128 bytes of this lane's row of Y
                        if (ey == 4) {                           // float32 or int32 output: 32 channels
                            uint32_t v[32];
                            gt_load32(t2base + (uint32_t)c0, v);
                            const int ch = n0 + c0 + lane;
                            const uint32_t bl = (p.bias2 != nullptr && ch < p.O2) ? __ldg((const uint32_t *)p.bias2 + ch) : 0u;
                            if constexpr (kI8) {
#pragma unroll
                                for (int e = 0; e < 32; ++e) out[e] = (uint32_t)((int)v[e] + (int)__shfl_sync(0xFFFFFFFFu, bl, e));
                            } else {
#pragma unroll
                                for (int e = 0; e < 32; ++e) out[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(__shfl_sync(0xFFFFFFFFu, bl, e)));
                            }
                        } else if (kI8 && ey == 1) {             // int8 output: 128 channels, requantised after the bias
#pragma unroll
                            for (int sub = 0; sub < 4; ++sub) {
                                if (n0 + c0 + sub * 32 >= p.O2) {    // (past the last channel: clipped by the store)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) out[sub * 8 + e] = 0u;
                                    continue;
                                }
                                uint32_t v[32];
                                gt_load32(t2base + (uint32_t)(c0 + sub * 32), v);
                                const int ch = n0 + c0 + sub * 32 + lane;
                                const int bl = (p.bias2 != nullptr && ch < p.O2) ? __ldg((const int *)p.bias2 + ch) : 0;
                                const uint32_t sl = ch < p.O2 ? (uint32_t)__ldg(p.shift2 + ch) & 31u : 0u;
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    int r4[4];
#pragma unroll
                                    for (int b = 0; b < 4; ++b)
                                        r4[b] = gt_round_shift((int)v[4 * e + b] + __shfl_sync(0xFFFFFFFFu, bl, 4 * e + b), __shfl_sync(0xFFFFFFFFu, sl, 4 * e + b));
                                    const uint32_t w = gt_pack_s8x4(r4[0], r4[1], r4[2], r4[3]);
                                    out[sub * 8 + e] = w;
                                }
                            }
                        } else {                                 // bfloat16 output: 64 channels
#pragma unroll
                            for (int sub = 0; sub < 2; ++sub) {
                                uint32_t v[32];
                                gt_load32(t2base + (uint32_t)(c0 + sub * 32), v);
                                const int ch = n0 + c0 + sub * 32 + lane;
                                const float bl = (p.bias2 != nullptr && ch < p.O2) ? __ldg((const float *)p.bias2 + ch) : 0.f;
#pragma unroll
                                for (int e = 0; e < 16; ++e) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * e]) + __shfl_sync(0xFFFFFFFFu, bl, 2 * e),
                                                                                   __uint_as_float(v[2 * e + 1]) + __shfl_sync(0xFFFFFFFFu, bl, 2 * e + 1));
                                    out[sub * 16 + e] = *(const uint32_t *)&h;
                                }
                            }
                        }
                        // staged under the 128-byte swizzle and stored as the tile's box of positions by one TMA store; what lies
                        // past the last channel, column, row or image of Y is clipped
                        if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory");
                        gt_group_sync(1 + grp);
                        const uint32_t srow = sb + (uint32_t)lane * 128u;
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};\n"
                                         ::"r"(srow + (uint32_t)((j ^ (lane & 7)) << 4)), "r"(out[4 * j]), "r"(out[4 * j + 1]), "r"(out[4 * j + 2]), "r"(out[4 * j + 3]) : "memory");
                        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                        gt_group_sync(1 + grp);
                        if (issuer && n0 + c0 < p.O2) {
                            asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];\n"
                                         ::"l"(&p.tmy), "r"(sg), "r"((n0 + c0) * ey), "r"(x0), "r"(y0), "r"(in0) : "memory");
                            asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
                        }
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
                    __syncwarp();
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(sm32(&s_acc2_empty[buf])) : "memory");
                }
            }
            if (issuer) asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory");
            if (!ok && lane == 0) atomicExch((uint32_t *)&s_fail, 1u);
        }
    }

    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (s_fail == 1u && tid == 0) atomicMax(p.status, (int)BSP_ERR_TIMEOUT);
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kGtTmemCols) : "memory");
}

}  // namespace

// True if the fused kernel can run this pair: two bfloat16 or two int8 layers, a 1x1 second layer on the first one's
// output channels, at most 256 of them (accumulator one holds them all), rows of X, of both weights and of Y that are
// multiples of 16 bytes.
bool chain_tc_eligible(const bsp_wdesc &wd1, const bsp_wdesc &wd2, const bsp_xdesc &xd0, bsp_dtype ytype)
{
    if (wd1.wtype != wd2.wtype || (wd1.wtype != BSP_BF16 && wd1.wtype != BSP_I8)) return false;
    if (wd2.H != 1 || wd2.K != 1 || wd2.I != wd1.O) return false;
    if (wd1.O > 256 || wd1.O % 8 != 0 || wd1.I % 8 != 0 || wd2.O % 8 != 0) return false;
    const int esz = elem_bytes(wd1.wtype);
    if (wd1.wtype == BSP_I8) { if (ytype != BSP_I32 && ytype != BSP_I8) return false; }
    else if (ytype != BSP_F32 && ytype != BSP_BF16) return false;
    const int ey = ytype == BSP_BF16 ? 2 : (ytype == BSP_I8 ? 1 : 4);
    if ((wd1.I * esz) % 16 != 0 || (wd1.O * esz) % 16 != 0 || (wd2.O * ey) % 16 != 0) return false;
    if (!packed_layout(wd1).enabled || !packed_layout(wd2).enabled) return false;
    const bsp_xdesc xd = gt_flatten(wd1, xd0);
    const int M = (xd.L + 2 * xd.pad_h - wd1.H) / xd.stride_h + 1, Nw = (xd.J + 2 * xd.pad_w - wd1.K) / xd.stride_w + 1;
    if (M <= 0 || Nw <= 0) return false;
    if ((long long)xd.N * M * Nw > 0x7FFFFFFF - 4096 || (long long)xd.N * xd.L * xd.J > 0x7FFFFFFF) return false;
    return gt_pick_tile(xd.N, M, Nw, xd.stride_h, xd.stride_w).tiles > 0;
}

bsp_status launch_chain_tc(const bsp_wdesc &wd1, const void *packed1, const bsp_wdesc &wd2, const void *packed2,
                           const bsp_xdesc &xd0, const void *X, const void *bias1, const int32_t *shift1, int relu,
                           const void *bias2, const int32_t *shift2, void *Y, bsp_dtype ytype, void *ws, cudaStream_t st)
{
    const bsp_xdesc xd = gt_flatten(wd1, xd0);
    const PackedLayout L1 = packed_layout(wd1), L2 = packed_layout(wd2);
    if (!L1.enabled || !L2.enabled) return BSP_ERR_SHAPE;
    const int ey = ytype == BSP_BF16 ? 2 : (ytype == BSP_I8 ? 1 : 4);
    const int esz = elem_bytes(wd1.wtype);
    if (wd1.wtype == BSP_I8 && (shift1 == nullptr || (ytype == BSP_I8 && shift2 == nullptr))) return BSP_ERR_NULL;
    CtParams p = {};
    p.bias1 = bias1; p.bias2 = bias2; p.shift1 = shift1; p.shift2 = shift2; p.wtype = wd1.wtype; p.packed1 = (const uint8_t *)packed1; p.packed2 = (const uint8_t *)packed2;
    p.status = (int *)ws;
    p.O1 = wd1.O; p.I1 = wd1.I; p.H = wd1.H; p.K = wd1.K; p.bo1 = wd1.bo; p.bi1 = wd1.bi;
    p.O2 = wd2.O; p.bo2 = wd2.bo; p.bi2 = wd2.bi; p.relu = relu ? 1 : 0; p.ytype = ytype; p.ey = ey; p.Y = (uint8_t *)Y;
    p.tcc = 128 / esz;
    p.O1p = (wd1.O + p.tcc - 1) / p.tcc * p.tcc;
    p.N = xd.N; p.sh = xd.stride_h; p.sw = xd.stride_w; p.ph = xd.pad_h; p.pw = xd.pad_w;
    p.M = (xd.L + 2 * xd.pad_h - wd1.H) / xd.stride_h + 1;
    p.Nw = (xd.J + 2 * xd.pad_w - wd1.K) / xd.stride_w + 1;
    const long long P = (long long)xd.N * p.M * p.Nw;
    p.P = (int)P;
    const GtTile T = gt_pick_tile(xd.N, p.M, p.Nw, p.sh, p.sw);
    if (T.tiles <= 0 || T.tiles > 0x7FFFFFFF - 4096) return BSP_ERR_SHAPE;
    p.Wt = T.Wt; p.Ht = T.Ht; p.Nt = T.Nt; p.rows_tile = T.Wt * T.Ht * T.Nt;
    p.tiles_x = (p.Nw + T.Wt - 1) / T.Wt; p.tiles_y = (p.M + T.Ht - 1) / T.Ht;
    p.m_tx = gt_magic(p.tiles_x); p.m_ty = gt_magic(p.tiles_y);
    p.a_bytes = p.rows_tile * 128;
    p.n_tiles = (int)T.tiles;
    p.cpt1 = (wd1.I * esz + 127) / 128;
    p.n_ks1 = wd1.H * wd1.K * p.cpt1;
    p.n_c2 = p.O1p / p.tcc;
    p.n_t2 = (wd2.O + kCtBN2 - 1) / kCtBN2;
    p.stage_bytes = kGtABytes + p.O1p * 128;
    p.db = p.O1p <= 128 ? 1 : 0;
    const int fixed = 1024 + (p.db ? 2 : 1) * p.n_c2 * kCtChunk + 8 * kGtStagingBytes;
    int stages = (kGtMaxSmem - fixed) / p.stage_bytes;
    if (stages > kGtMaxStages) stages = kGtMaxStages;
    if (stages < 2) return BSP_ERR_SHAPE;
    p.stages = stages;
    const size_t smem = (size_t)fixed + (size_t)stages * p.stage_bytes;

    static bool opted[kGtMaxDevices] = {};
    static int n_sm[kGtMaxDevices] = {};
    int dev = 0;
    BSP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kGtMaxDevices) return BSP_ERR_CUDA;
    if (!opted[dev]) {
        BSP_CUDA_OK(cudaFuncSetAttribute(chain_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGtMaxSmem));
        BSP_CUDA_OK(cudaFuncSetAttribute(chain_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGtMaxSmem));
        BSP_CUDA_OK(cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev));
        opted[dev] = true;
    }
    GtEncodeFn enc = gt_encode();
    if (!enc) return BSP_ERR_CUDA;
    {
        const cuuint64_t row = (cuuint64_t)wd1.I * esz;
        const cuuint64_t gdim[4] = {row, (cuuint64_t)xd.J, (cuuint64_t)xd.L, (cuuint64_t)xd.N};
        const cuuint64_t gstr[3] = {row, row * xd.J, row * xd.J * xd.L};
        const cuuint32_t box[4] = {128, (cuuint32_t)(T.Wt * p.sw), (cuuint32_t)(T.Ht * p.sh), (cuuint32_t)T.Nt};
        const cuuint32_t estr[4] = {1, (cuuint32_t)p.sw, (cuuint32_t)p.sh, 1};
        if (enc(&p.tmx, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(X), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }
    {
        const cuuint64_t row = (cuuint64_t)wd1.I * esz;
        const cuuint64_t gdim[3] = {row, (cuuint64_t)(wd1.H * wd1.K), (cuuint64_t)wd1.O};
        const cuuint64_t gstr[2] = {row, row * wd1.H * wd1.K};
        const cuuint32_t box[3] = {128, 1, (cuuint32_t)p.O1p};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&p.tmw1, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>((const uint8_t *)packed1 + L1.off_payload), gdim, gstr, box,
                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }
    {
        const cuuint64_t row = (cuuint64_t)wd2.I * esz;
        const cuuint64_t gdim[3] = {row, 1, (cuuint64_t)wd2.O};
        const cuuint64_t gstr[2] = {row, row};
        const cuuint32_t box[3] = {128, 1, (cuuint32_t)kCtBN2};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&p.tmw2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>((const uint8_t *)packed2 + L2.off_payload), gdim, gstr, box,
                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }
    {
        const cuuint64_t row = (cuuint64_t)wd2.O * ey;
        const cuuint64_t gdim[4] = {row, (cuuint64_t)p.Nw, (cuuint64_t)p.M, (cuuint64_t)xd.N};
        const cuuint64_t gstr[3] = {row, row * p.Nw, row * p.Nw * p.M};
        const cuuint32_t box[4] = {128, (cuuint32_t)T.Wt, (cuuint32_t)T.Ht, (cuuint32_t)T.Nt};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(&p.tmy, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, Y, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return BSP_ERR_CUDA;
    }
    const int grid = p.n_tiles < n_sm[dev] ? p.n_tiles : n_sm[dev];
    if (wd1.wtype == BSP_I8) chain_tc_kernel<true><<<grid, kCtThreads, smem, st>>>(p);
    else chain_tc_kernel<false><<<grid, kCtThreads, smem, st>>>(p);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // namespace bsp
