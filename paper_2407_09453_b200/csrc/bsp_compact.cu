// Compaction of Gamma (.) W: compressed block rows (row_ptr, col_idx, canonical payload) and the packed
// tile form read by the product kernels.  Section "Block Sparsity in a Matrix" (compress block row) and
// Section "Subvolumes, Data Compression, and Data Movements" of the paper.
#include "bsp_internal.cuh"

namespace bsp {

PackedLayout packed_layout(const bsp_wdesc &wd, int64_t nnz_blocks)
{
    PackedLayout L;
    L.n_panels = (wd.O + kPanelCh - 1) / kPanelCh;
    L.n_cols = wd.I / kTile;
    L.tile_bytes = tile_bytes_of(wd.wtype, wd.H * wd.K);
    const int64_t all_tiles = (int64_t)((wd.O + kTile - 1) / kTile) * L.n_cols;
    // a 4x16 or 16x4 block touches two tiles; an 8x8 block is one tile
    const int64_t per_block = (wd.bo == 8 && wd.bi == 8) ? 1 : 2;
    int64_t cap = nnz_blocks * per_block;
    if (cap > all_tiles) cap = all_tiles;
    if (cap < 0) cap = 0;
    L.capacity_tiles = cap;
    L.off_colmask = 256;
    L.off_coloff = align_up(L.off_colmask + (size_t)L.n_panels * L.n_cols, 256);
    L.off_panelbase = align_up(L.off_coloff + (size_t)L.n_panels * L.n_cols * 4, 256);
    // all index arrays come first, at offsets that do not depend on the capacity; the two payloads follow
    size_t meta_end = align_up(L.off_panelbase + (size_t)(L.n_panels + 1) * 4, 256);
    TcLayout &T = L.tc;
    T = TcLayout{};
    const int HK = wd.H * wd.K;
    // a K-step of the tensor-memory kernel is 32 bytes of input channels: 16 bf16 or 32 int8
    const int cpc = wd.wtype == BSP_I8 ? 16 : 8;          // channels per 16-byte chunk
    T.enabled = (wd.wtype == BSP_BF16 || wd.wtype == BSP_I8) && wd.O % 8 == 0 && wd.I % (HK == 1 ? 2 * cpc : cpc) == 0;
    int64_t tcap = 0;
    if (T.enabled) {
        const int n_sr = (wd.O + kTcSuperRow - 1) / kTcSuperRow;
        T.n_groups = (n_sr + kTcGroupRows - 1) / kTcGroupRows;
        T.kc_ch = HK == 1 ? 2 * cpc : cpc;
        T.n_kc = wd.I / T.kc_ch;
        T.n_units = HK == 1 ? 1 : (HK + 1) / 2;
        T.st_bytes = T.n_units * kTcUnitBytes;
        tcap = nnz_blocks * 4;                                // a 4x16 block can touch two super-tiles; gap fillers at most double them
        if (tcap > (int64_t)n_sr * T.n_kc) tcap = (int64_t)n_sr * T.n_kc;
        if (tcap < 0) tcap = 0;
        T.capacity = tcap;
        T.off_mask = meta_end;
        T.off_off = align_up(T.off_mask + (size_t)T.n_groups * T.n_kc, 256);
        T.off_gcnt = align_up(T.off_off + (size_t)T.n_groups * T.n_kc * 4, 256);
        meta_end = align_up(T.off_gcnt + (size_t)(T.n_groups + 1) * 4, 256);
    }
    // third form (layers whose rows of input channels are multiples of 16 bytes): Gamma (.) W as it is laid out,
    // [O][H][K][I]; it comes first among the payloads, so that its offset does not depend on the capacity
    GemmLayout &G = L.gm;
    G = GemmLayout{};
    const int esz = elem_bytes(wd.wtype);
    G.enabled = ((long long)wd.I * esz) % 16 == 0 && wd.O % 8 == 0;
    if (G.enabled) {
        G.n_ks = HK * (int)(((long long)wd.I * esz + 127) / 128);
        G.off_payload = meta_end;
        G.end = align_up(G.off_payload + (size_t)wd.O * HK * wd.I * esz + 256, 256);
        meta_end = G.end;
    }
    L.off_payload = meta_end;
    size_t end = align_up(L.off_payload + (size_t)cap * L.tile_bytes + 256, 256);
    if (T.enabled) {
        T.off_payload = end;
        T.end = align_up(T.off_payload + (size_t)tcap * T.st_bytes + 256, 256);
        end = T.end;
    }
    L.total_bytes = end;
    return L;
}

namespace {

constexpr int kThreads = 256;

// The super-tiles stored for one (group, K-group), given the mask of those that hold a kept block: a missing
// super-row between two present ones is stored too (as zeros), because one MMA over the joined run costs less than
// two MMAs around the gap (every MMA fetches the 128 x 32-byte activation tile again).
__device__ __forceinline__ unsigned tc_fill_gaps(unsigned m) { return (m | ((m << 1) & (m >> 1))) & 0xFFu; }

// b_o and b_i are 4, 8 or 16: divisions by them are shifts by lg().
__device__ __forceinline__ int lg(int b) { return 31 - __clz(b); }

// Exclusive prefix sum of v over the CTA's threads; every thread of the CTA must call it.
__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_sums, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int n = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += n;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    int before = 0, tot = 0;
    for (int w = 0; w < kThreads / 32; ++w) {
        const int s = warp_sums[w];
        if (w < warp) before += s;
        tot += s;
    }
    __syncthreads();
    total = tot;
    return before + inc - v;
}

// Launch 1.  CTAs [0, NBo): ones of one row of Gamma -> row_cnt.  CTAs [NBo, NBo + n_panels): for one panel
// (64 output channels) the byte mask of stored tiles in every tile column, and the running count of stored
// tiles before each column (coloff, relative to the panel).
struct TcIndexArgs {
    int n_panels, n_groups, n_kc, kc_ch;
    uint8_t *mask;        // [n_groups][n_kc]
    uint32_t *off;        // [n_groups][n_kc] stored super-tiles of the group before this K-group
    uint32_t *gcnt;       // [n_groups] stored super-tiles of the group
};

__global__ void __launch_bounds__(kThreads)
count_kernel(const uint8_t *__restrict__ gamma, int NBo, int NBi, int bo, int bi, int O, int n_cols,
             int *__restrict__ row_cnt, uint8_t *__restrict__ colmask, uint32_t *__restrict__ coloff,
             int *__restrict__ panel_cnt, const TcIndexArgs tc)
{
    __shared__ int warp_sums[kThreads / 32];
    __shared__ int s_run;
    if ((int)blockIdx.x >= NBo + tc.n_panels) {
        // CTAs past the panels: one group of super-rows each, for the second packed form
        const int g = (int)blockIdx.x - NBo - tc.n_panels;
        if (threadIdx.x == 0) s_run = 0;
        __syncthreads();
        for (int base = 0; base < tc.n_kc; base += kThreads) {
            const int kc = base + threadIdx.x;
            unsigned m = 0;
            if (kc < tc.n_kc) {
                for (int r = 0; r < kTcGroupRows; ++r) {
                    const int o0 = (g * kTcGroupRows + r) * kTcSuperRow;
                    if (o0 >= O) break;
                    const int o1 = min(O, o0 + kTcSuperRow) - 1;
                    const int c0 = kc * tc.kc_ch, c1 = c0 + tc.kc_ch - 1;
                    bool any = false;
                    for (int lb = o0 >> lg(bo); lb <= (o1 >> lg(bo)) && lb < NBo; ++lb)
                        for (int cb = c0 >> lg(bi); cb <= (c1 >> lg(bi)) && cb < NBi; ++cb) any |= gamma[(size_t)lb * NBi + cb] != 0;
                    if (any) m |= 1u << r;
                }
            }
            m = tc_fill_gaps(m);
            int tot;
            const int before = block_exclusive_scan(__popc(m), warp_sums, tot);
            if (kc < tc.n_kc) {
                tc.mask[(size_t)g * tc.n_kc + kc] = (uint8_t)m;
                tc.off[(size_t)g * tc.n_kc + kc] = (uint32_t)(s_run + before);
            }
            __syncthreads();
            if (threadIdx.x == 0) s_run += tot;
            __syncthreads();
        }
        if (threadIdx.x == 0) tc.gcnt[g] = (uint32_t)s_run;
        return;
    }
    if ((int)blockIdx.x < NBo) {
        const uint8_t *g = gamma + (size_t)blockIdx.x * NBi;
        int c = 0;
        for (int i = threadIdx.x; i < NBi; i += kThreads) c += g[i] ? 1 : 0;
        int tot;
        block_exclusive_scan(c, warp_sums, tot);
        if (threadIdx.x == 0) row_cnt[blockIdx.x] = tot;
        return;
    }
    const int panel = (int)blockIdx.x - NBo;
    if (threadIdx.x == 0) s_run = 0;
    __syncthreads();
    for (int base = 0; base < n_cols; base += kThreads) {
        const int col = base + threadIdx.x;
        unsigned m = 0;
        if (col < n_cols) {
            for (int r = 0; r < kPanelRows; ++r) {
                const int o0 = (panel * kPanelRows + r) * kTile;     // first channel of the tile row
                if (o0 >= O) break;
                // blocks overlapping the tile: rows o0/bo .. (o0+7)/bo, columns (8 col)/bi .. (8 col + 7)/bi
                bool any = false;
                for (int lb = o0 >> lg(bo); lb <= ((o0 + kTile - 1) >> lg(bo)) && lb < NBo; ++lb)
                    for (int cb = (col * kTile) >> lg(bi); cb <= ((col * kTile + kTile - 1) >> lg(bi)) && cb < NBi; ++cb)
                        any |= gamma[(size_t)lb * NBi + cb] != 0;
                if (any) m |= 1u << r;
            }
        }
        int tot;
        const int before = block_exclusive_scan(__popc(m), warp_sums, tot);
        if (col < n_cols) {
            colmask[(size_t)panel * n_cols + col] = (uint8_t)m;
            coloff[(size_t)panel * n_cols + col] = (uint32_t)(s_run + before);
        }
        __syncthreads();
        if (threadIdx.x == 0) s_run += tot;
        __syncthreads();
    }
    if (threadIdx.x == 0) panel_cnt[panel] = s_run;
}

// Launch 2 (one CTA): exclusive scans row_cnt -> row_ptr and panel_cnt -> panel_base, writes the packed
// header, and latches BSP_ERR_CAPACITY if more blocks are stored than the buffers were sized for.
__global__ void __launch_bounds__(kThreads)
scan_kernel(const int *__restrict__ row_cnt, int NBo, int32_t *__restrict__ row_ptr, const int *__restrict__ panel_cnt,
            int n_panels, uint32_t *__restrict__ panel_base, PackedHeader *__restrict__ hdr, PackedHeader hdr_init,
            long long capacity_blocks, long long capacity_tiles, int *__restrict__ status)
{
    __shared__ int warp_sums[kThreads / 32];
    __shared__ int s_run;
    if (threadIdx.x == 0) s_run = 0;
    __syncthreads();
    for (int base = 0; base < NBo; base += kThreads) {
        const int i = base + threadIdx.x;
        const int v = (i < NBo) ? row_cnt[i] : 0;
        int tot;
        const int before = block_exclusive_scan(v, warp_sums, tot);
        if (i < NBo) row_ptr[i] = s_run + before;
        __syncthreads();
        if (threadIdx.x == 0) s_run += tot;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        row_ptr[NBo] = s_run;
        if ((long long)s_run > capacity_blocks) atomicMax(status, (int)BSP_ERR_CAPACITY);
        if (panel_base != nullptr) {
            unsigned run = 0;
            for (int p = 0; p < n_panels; ++p) { panel_base[p] = run; run += (unsigned)panel_cnt[p]; }
            panel_base[n_panels] = run;
            hdr_init.n_tiles = (int)run;
            *hdr = hdr_init;
            if ((long long)run > capacity_tiles) atomicMax(status, (int)BSP_ERR_CAPACITY);
        }
    }
}

// Copies the cnt stored blocks of row l (columns s_cols[]) into the canonical payload in pieces of type V (one or
// several elements; a block row of b_i elements is contiguous in W and in the payload).  Each thread loads four
// pieces before it stores them.
template <typename T, typename V>
__device__ __forceinline__ void fill_copy(int l, int part, int parts, const T *__restrict__ W, int I, int HK, int bo, int bi,
                                          int first, int cnt, const int *s_cols, T *__restrict__ payload,
                                          long long capacity_blocks)
{
    constexpr int per = (int)(sizeof(V) / sizeof(T));
    const int bi_v = bi / per;                          // pieces per block row, a power of two
    const int blk = bo * HK * bi;
    const unsigned blk_v = (unsigned)(bo * HK * bi_v);
    const unsigned total = (unsigned)cnt * blk_v;       // at most I * b_o * H * K: fits 32 bits
    const unsigned stride = (unsigned)parts * kThreads;
    for (unsigned e0 = (unsigned)part * kThreads + threadIdx.x; e0 < total; e0 += 4 * stride) {
        V v[4];
        V *dst[4];
        bool ok[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned e = e0 + u * stride;
            ok[u] = e < total;
            const int n = ok[u] ? (int)(e / blk_v) : 0;
            const int q = ok[u] ? (int)(e - (unsigned)n * blk_v) : 0;
            const int c = q & (bi_v - 1), rt = q >> lg(bi_v);
            const int r = rt / HK, t = rt - r * HK;
            ok[u] = ok[u] && (long long)(first + n) < capacity_blocks;
            dst[u] = (V *)(payload + (size_t)(first + n) * blk + (size_t)rt * bi) + c;
            if (ok[u]) v[u] = *((const V *)(W + ((size_t)(l * bo + r) * HK + t) * I + (size_t)s_cols[n] * bi) + c);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (ok[u]) *dst[u] = v[u];
    }
}

// Final launch, first part.  `parts` CTAs per row of Gamma: column indices in ascending order and the canonical payload
// payload[n][r][h][k][c] = W[l b_o + r][h][k][iota b_i + c].  `first` = stored blocks in the rows above; returns
// the number of stored blocks of row l.
template <typename T>
__device__ __forceinline__ int csr_fill_body(int l, int part, int parts, const T *__restrict__ W,
                                              const uint8_t *__restrict__ gamma, int NBi, int I, int HK, int bo, int bi,
                                              int first, int32_t *__restrict__ col_idx,
                                              T *__restrict__ payload, long long capacity_blocks)
{
    __shared__ int warp_sums[kThreads / 32];
    __shared__ int s_run;
    extern __shared__ int s_cols[];      // NBi ints: columns of this row's stored blocks
    const uint8_t *g = gamma + (size_t)l * NBi;
    if (threadIdx.x == 0) s_run = 0;
    __syncthreads();
    for (int base = 0; base < NBi; base += kThreads) {
        const int i = base + threadIdx.x;
        const int v = (i < NBi && g[i]) ? 1 : 0;
        int tot;
        const int before = block_exclusive_scan(v, warp_sums, tot);
        if (v) {
            const int n = s_run + before;
            s_cols[n] = i;
            if (part == 0 && (long long)(first + n) < capacity_blocks) col_idx[first + n] = i;
        }
        __syncthreads();
        if (threadIdx.x == 0) s_run += tot;
        __syncthreads();
    }
    if (payload == nullptr) return s_run;
    const int cnt = s_run;
    // the CTAs of one row (`parts` of them) all build the column list, then share the copy, in the widest pieces
    // (up to 16 bytes) that the block width, the row pitch of W and the two base addresses allow
    const size_t row_bytes = (size_t)bi * sizeof(T), pitch = (size_t)I * sizeof(T);
    const uintptr_t bases = (uintptr_t)W | (uintptr_t)payload;
    size_t vb = 16;
    while (vb > sizeof(T) && (row_bytes % vb || pitch % vb || bases % vb)) vb >>= 1;
    if (vb == 16) fill_copy<T, uint4>(l, part, parts, W, I, HK, bo, bi, first, cnt, s_cols, payload, capacity_blocks);
    else if (vb == 8) fill_copy<T, uint2>(l, part, parts, W, I, HK, bo, bi, first, cnt, s_cols, payload, capacity_blocks);
    else if (vb == 4 && sizeof(T) < 4) fill_copy<T, uint32_t>(l, part, parts, W, I, HK, bo, bi, first, cnt, s_cols, payload, capacity_blocks);
    else fill_copy<T, T>(l, part, parts, W, I, HK, bo, bi, first, cnt, s_cols, payload, capacity_blocks);
    return cnt;
}

// One 32-bit word of a packed tile.  The tile at (tile row of the panel, tile column) holds, for every K-step
// of the MMA, the B-operand fragment of all 32 lanes: lane = 4 g + t holds output channel g of the tile.
//  bf16 : steps of two taps (m16n8k16): word 2*lane+j of step s = channels 2t, 2t+1 at tap 2s+j;
//         an odd last tap is a step of its own (m16n8k8) with one word per lane.
//  int8 : steps of two taps (m16n8k16): the word of lane (g,t) = channels 4(t&1)..4(t&1)+3 at tap 2s+(t>>1);
//         a missing second tap is written as zeros.
//  fp32 : one tap per step (m16n8k8, tf32): words 2*lane, 2*lane+1 = channel t and channel t+4.
// o0, c0: first output and input channel of the tile.  Weights of blocks with Gamma = 0 read as zero.
template <int DT>
__device__ __forceinline__ uint32_t packed_word(const void *__restrict__ Wv, const uint8_t *__restrict__ gamma,
                                                int word, int o0, int c0, int O, int I, int HK, int bo, int bi,
                                                int NBi)
{
    auto kept = [&](int o, int ch) -> bool { return o < O && gamma[(size_t)(o >> lg(bo)) * NBi + (ch >> lg(bi))] != 0; };
    if constexpr (DT == BSP_BF16) {
        const uint16_t *W = (const uint16_t *)Wv;
        const int pairs = HK / 2;
        int lane, tap;
        if (word < pairs * 64) { const int s = word / 64, w = word % 64; lane = w >> 1; tap = 2 * s + (w & 1); }
        else { lane = word - pairs * 64; tap = HK - 1; }
        const int g = lane >> 2, t = lane & 3;
        const int o = o0 + g, ch = c0 + 2 * t;
        if (!kept(o, ch)) return 0u;              // both channels lie in one block (b_i is even)
        const size_t e = ((size_t)o * HK + tap) * I + ch;
        return (uint32_t)W[e] | ((uint32_t)W[e + 1] << 16);
    } else if constexpr (DT == BSP_I8) {
        const uint8_t *W = (const uint8_t *)Wv;
        const int s = word / 32, lane = word % 32;
        const int g = lane >> 2, t = lane & 3;
        const int tap = 2 * s + (t >> 1);
        const int o = o0 + g, ch = c0 + 4 * (t & 1);
        if (tap >= HK || !kept(o, ch)) return 0u;   // four channels never straddle a block (b_i >= 4)
        const size_t e = ((size_t)o * HK + tap) * I + ch;
        return (uint32_t)W[e] | ((uint32_t)W[e + 1] << 8) | ((uint32_t)W[e + 2] << 16) | ((uint32_t)W[e + 3] << 24);
    } else {
        const uint32_t *W = (const uint32_t *)Wv;
        const int tap = word / 64, w = word % 64;
        const int lane = w >> 1;
        const int g = lane >> 2, t = lane & 3;
        const int o = o0 + g, ch = c0 + t + 4 * (w & 1);
        if (!kept(o, ch)) return 0u;
        return W[((size_t)o * HK + tap) * I + ch];
    }
}

// Sixteen bytes of W[o][tap][ch0 ..] (16 / esz consecutive input channels of esz bytes each), with the channels of
// zeroed blocks cleared; rows past O and taps past HK read as zero.  Needs 16-byte aligned rows of W.
template <int esz>
__device__ __forceinline__ uint4 w_chunk(const void *__restrict__ W, const uint8_t *gamma, int o, int tap, int ch0,
                                         int O, int I, int HK, int bo, int bi, int NBi)
{
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (o >= O || tap >= HK) return v;
    const uint8_t *grow = gamma + (size_t)(o >> lg(bo)) * NBi;
    constexpr int cpc = 16 / esz;
    const int b0 = ch0 >> lg(bi);
    if (bi >= cpc) {
        if (grow[b0] == 0) return v;
        return __ldg((const uint4 *)((const uint8_t *)W + (((size_t)o * HK + tap) * I + ch0) * esz));
    }
    const uint4 *src = (const uint4 *)((const uint8_t *)W + (((size_t)o * HK + tap) * I + ch0) * esz);
    if (cpc == 8 || cpc / bi == 2) {                       // two blocks per chunk (always, for 8-channel chunks and b_i = 4)
        const bool k0 = grow[b0] != 0, k1 = grow[b0 + 1] != 0;
        if (!k0 && !k1) return v;
        v = __ldg(src);
        if (!k0) v.x = v.y = 0u;
        if (!k1) v.z = v.w = 0u;
        return v;
    }
    const bool k0 = grow[b0] != 0, k1 = grow[b0 + 1] != 0, k2 = grow[b0 + 2] != 0, k3 = grow[b0 + 3] != 0;   // four
    if (!k0 && !k1 && !k2 && !k3) return v;
    v = __ldg(src);
    if (!k0) v.x = 0u;
    if (!k1) v.y = 0u;
    if (!k2) v.z = 0u;
    if (!k3) v.w = 0u;
    return v;
}
__device__ __forceinline__ uint4 bf16_chunk(const uint16_t *__restrict__ W, const uint8_t *gamma, int o, int tap, int ch0,
                                            int O, int I, int HK, int bo, int bi, int NBi)
{
    return w_chunk<2>(W, gamma, o, tap, ch0, O, I, HK, bo, bi, NBi);
}

// bf16 tiles of one (panel, tile column) in 16-byte chunks: the 32 bytes of tile row g in a two-tap step are the
// words of its two chunks interleaved (w0 v0 w1 v1 ...), the 16 bytes of an odd last tap are its chunk.
__device__ __forceinline__ void pack_tiles_bf16(unsigned m, unsigned first, int panel, int col, const uint16_t *__restrict__ W,
                                                const uint8_t *gamma, int O, int I, int HK, int bo, int bi, int NBi,
                                                int tile_bytes, uint8_t *__restrict__ payload, long long capacity_tiles,
                                                int part, int parts)
{
    const int pairs = HK >> 1;
    const int ipt = (pairs + (HK & 1)) * 8;             // items per tile: (step, tile row)
    const int total = __popc(m) * ipt;
    const int stride = parts * kThreads;
    for (int e0 = part * kThreads + threadIdx.x; e0 < total; e0 += 2 * stride) {
        uint4 a[2], b[2];
        uint8_t *dst[2];
        bool ok[2], two[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int e = e0 + u * stride;
            ok[u] = e < total;
            const int j = ok[u] ? (int)((unsigned)e / (unsigned)ipt) : 0, rem = ok[u] ? e - j * ipt : 0;
            const int s = rem >> 3, g = rem & 7;
            unsigned mm = m;
            for (int q = 0; q < j; ++q) mm &= mm - 1;
            const int o = (panel * kPanelRows + (__ffs(mm) - 1)) * kTile + g;
            ok[u] = ok[u] && (long long)(first + j) < capacity_tiles;
            two[u] = s < pairs;
            dst[u] = payload + (size_t)(first + j) * tile_bytes + (two[u] ? s * 256 + g * 32 : pairs * 256 + g * 16);
            a[u] = b[u] = make_uint4(0u, 0u, 0u, 0u);
            if (ok[u]) {
                a[u] = bf16_chunk(W, gamma, o, two[u] ? 2 * s : HK - 1, col * kTile, O, I, HK, bo, bi, NBi);
                if (two[u]) b[u] = bf16_chunk(W, gamma, o, 2 * s + 1, col * kTile, O, I, HK, bo, bi, NBi);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (!ok[u]) continue;
            if (two[u]) {
                ((uint4 *)dst[u])[0] = make_uint4(a[u].x, b[u].x, a[u].y, b[u].y);
                ((uint4 *)dst[u])[1] = make_uint4(a[u].z, b[u].z, a[u].w, b[u].w);
            } else {
                *(uint4 *)dst[u] = a[u];
            }
        }
    }
}

// The stored tiles of one (panel, tile column), whose tile rows are the set bits of m, written word by word
// from slot `first` on.  `parts` CTAs share the words; each thread loads four before it stores.
template <int DT>
__device__ __forceinline__ void pack_tiles(unsigned m, unsigned first, int panel, int col, const void *__restrict__ W,
                                           const uint8_t *__restrict__ gamma, int O, int I, int HK, int bo, int bi, int NBi,
                                           int tile_bytes, uint8_t *__restrict__ payload, long long capacity_tiles,
                                           int part, int parts)
{
    if constexpr (DT == BSP_BF16) {
        if ((I & 7) == 0 && (((uintptr_t)W) & 15u) == 0) {
            pack_tiles_bf16(m, first, panel, col, (const uint16_t *)W, gamma, O, I, HK, bo, bi, NBi, tile_bytes, payload,
                            capacity_tiles, part, parts);
            return;
        }
    }
    const int words = tile_bytes / 4;
    const int total = __popc(m) * words;
    const int stride = parts * kThreads;
    for (int e0 = part * kThreads + threadIdx.x; e0 < total; e0 += 4 * stride) {
        uint32_t v[4];
        uint32_t *dst[4];
        bool ok[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = e0 + u * stride;
            ok[u] = e < total;
            const int j = ok[u] ? (int)((unsigned)e / (unsigned)words) : 0, word = ok[u] ? e - j * words : 0;
            unsigned mm = m;                         // j-th set bit of m = tile row
            for (int q = 0; q < j; ++q) mm &= mm - 1;
            const int R = __ffs(mm) - 1;
            ok[u] = ok[u] && (long long)(first + j) < capacity_tiles;
            dst[u] = (uint32_t *)(payload + (size_t)(first + j) * tile_bytes) + word;
            v[u] = ok[u] ? packed_word<DT>(W, gamma, word, (panel * kPanelRows + R) * kTile, col * kTile, O, I, HK, bo, bi, NBi) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (ok[u]) *dst[u] = v[u];
    }
}

// Final launch, second part.  One CTA per (tile-column chunk, panel): every stored tile of the panel in this chunk of columns.
template <int DT>
__device__ __forceinline__ void pack_body(int chunk, int panel, const void *__restrict__ W,
                                          const uint8_t *__restrict__ gamma, int O, int I, int HK, int bo, int bi, int NBi,
                                          int n_cols, int cols_per_cta, int tile_bytes, const uint8_t *__restrict__ colmask,
                                          const uint32_t *__restrict__ coloff, const uint32_t *__restrict__ panel_base,
                                          uint8_t *__restrict__ payload, long long capacity_tiles)
{
    const int col_lo = chunk * cols_per_cta;
    const int col_hi = min(n_cols, col_lo + cols_per_cta);
    const unsigned base = panel_base[panel];
    for (int col = col_lo; col < col_hi; ++col) {
        const unsigned m = colmask[(size_t)panel * n_cols + col];
        if (!m) continue;
        pack_tiles<DT>(m, base + coloff[(size_t)panel * n_cols + col], panel, col, W, gamma, O, I, HK, bo, bi, NBi,
                       tile_bytes, payload, capacity_tiles, 0, 1);
    }
}

// One 32-bit word of a stored super-tile: K-step u, then [8-row group rg][K half h][row][4 words of 2 bf16]:
// 8 rows x 16 bytes are one core matrix of a K-major tcgen05 B operand without swizzle, the K halves are 128
// bytes apart and the row groups 256.  The stored super-tiles of one (group, K-group) are laid out K-step
// major, [u][stored tile][512 bytes], so that for one K-step the tiles of consecutive stored super-rows form ONE
// B operand of 16 x (number of tiles) rows with a uniform 256-byte row-group stride.
// A convolution pairs taps 2u and 2u+1 of the K-group's 8 channels (a missing odd tap reads as zero); a 1x1
// layer pairs the two 8-channel halves.
template <int esz>
__device__ __forceinline__ uint32_t tc_word(const void *__restrict__ W, const uint8_t *__restrict__ gamma, int word,
                                            int o_base, int kc, int O, int I, int HK, int bo, int bi, int NBi)
{
    const int u = word >> 7, w = word & 127;
    const int rg = w >> 6, h = (w >> 5) & 1, row = (w >> 2) & 7, pair = w & 3;
    const int o = o_base + rg * 8 + row;
    constexpr int cpc = 16 / esz, cpw = 4 / esz;          // channels per 16-byte chunk and per 32-bit word
    int tap, ch;
    if (HK == 1) { tap = 0; ch = (2 * kc + h) * cpc + pair * cpw; }
    else { tap = 2 * u + h; ch = kc * cpc + pair * cpw; }
    // the channels of a word lie in one block (b_i is a multiple of 4)
    if (tap >= HK || o >= O || gamma[(size_t)(o >> lg(bo)) * NBi + (ch >> lg(bi))] == 0) return 0u;
    return *(const uint32_t *)((const uint8_t *)W + (((size_t)o * HK + tap) * I + ch) * esz);
}

struct TcPackArgs {
    int n_groups, n_kc, kc_per_cta, chunks, st_bytes;
    const uint8_t *mask;
    const uint32_t *off, *gcnt;
    uint8_t *payload;
    long long capacity;
    int *status;
};

// The stored super-tiles of one (group, K-group), whose super-rows are the set bits of m, from slot `first` on.
// `parts` CTAs share the words; each thread loads four before it stores.
template <int esz>      // bytes per weight: 2 (bf16) or 1 (int8)
__device__ __forceinline__ void tc_pack_tiles(unsigned m, unsigned first, int g, int kc, const TcPackArgs &t,
                                              const void *__restrict__ W, const uint8_t *__restrict__ gamma, int O, int I,
                                              int HK, int bo, int bi, int NBi, int part, int parts)
{
    const int cnt = __popc(m);
    constexpr int cpc = 16 / esz;
    if (((I * esz) & 15) == 0 && (((uintptr_t)W) & 15u) == 0) {
        // 16-byte chunks: one (row group, K half, row) slot of a K-step is one chunk of one weight row and tap
        const int nu = t.st_bytes >> 9;
        const int total = cnt * nu * 32;
        const int stride = parts * kThreads;
        for (int e0 = part * kThreads + threadIdx.x; e0 < total; e0 += 4 * stride) {
            uint4 v[4];
            uint4 *dst[4];
            bool ok[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = e0 + u * stride;
                ok[u] = e < total;
                const int j = ok[u] ? (int)((unsigned)e / (unsigned)(nu * 32)) : 0, rem = ok[u] ? e - j * nu * 32 : 0;
                const int ks = rem >> 5, slot = rem & 31;
                const int rg = slot >> 4, h = (slot >> 3) & 1, row = slot & 7;
                unsigned mm = m;
                for (int q = 0; q < j; ++q) mm &= mm - 1;
                const int o = (g * kTcGroupRows + (__ffs(mm) - 1)) * kTcSuperRow + rg * 8 + row;
                const int tap = HK == 1 ? 0 : 2 * ks + h, ch0 = HK == 1 ? (2 * kc + h) * cpc : kc * cpc;
                ok[u] = ok[u] && (long long)(first + cnt) <= t.capacity;
                dst[u] = (uint4 *)(t.payload + (size_t)first * t.st_bytes + ((size_t)(ks * cnt + j) << 9)) + slot;
                v[u] = ok[u] ? w_chunk<esz>(W, gamma, o, tap, ch0, O, I, HK, bo, bi, NBi) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (ok[u]) *dst[u] = v[u];
        }
        return;
    }
    const int words = t.st_bytes / 4;
    const int total = cnt * words;
    const int stride = parts * kThreads;
    for (int e0 = part * kThreads + threadIdx.x; e0 < total; e0 += 4 * stride) {
        uint32_t v[4];
        uint32_t *dst[4];
        bool ok[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = e0 + u * stride;
            ok[u] = e < total;
            const int j = ok[u] ? (int)((unsigned)e / (unsigned)words) : 0, word = ok[u] ? e - j * words : 0;
            unsigned mm = m;
            for (int q = 0; q < j; ++q) mm &= mm - 1;
            const int R = __ffs(mm) - 1;
            ok[u] = ok[u] && (long long)(first + cnt) <= t.capacity;
            // K-step (word >> 7) major within the K-group, then the stored tile, then the word of the 512-byte unit
            dst[u] = (uint32_t *)(t.payload + (size_t)first * t.st_bytes) + ((size_t)((word >> 7) * cnt + j) << 7) + (word & 127);
            v[u] = ok[u] ? tc_word<esz>(W, gamma, word, (g * kTcGroupRows + R) * kTcSuperRow, kc, O, I, HK, bo, bi, NBi) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (ok[u]) *dst[u] = v[u];
    }
}

template <int esz>
__device__ __forceinline__ void tc_pack_body(int chunk, int g, const TcPackArgs &t, const void *__restrict__ W,
                                             const uint8_t *__restrict__ gamma, int O, int I, int HK, int bo, int bi,
                                             int NBi)
{
    unsigned base = 0;
    for (int q = 0; q < g; ++q) base += t.gcnt[q];
    if (chunk == 0 && threadIdx.x == 0 && (long long)(base + t.gcnt[g]) > t.capacity)
        atomicMax(t.status, (int)BSP_ERR_CAPACITY);
    const int kc_lo = chunk * t.kc_per_cta, kc_hi = min(t.n_kc, kc_lo + t.kc_per_cta);
    for (int kc = kc_lo; kc < kc_hi; ++kc) {
        const unsigned m = t.mask[(size_t)g * t.n_kc + kc];
        if (!m) continue;
        tc_pack_tiles<esz>(m, base + t.off[(size_t)g * t.n_kc + kc], g, kc, t, W, gamma, O, I, HK, bo, bi, NBi, 0, 1);
    }
}

struct FillPackArgs {
    const void *W;
    const uint8_t *gamma;
    int O, I, HK, bo, bi, NBo, NBi;
    const int32_t *row_ptr;
    int32_t *col_idx;
    void *payload;
    long long capacity_blocks;
    int fill_parts;                   // CTAs per row of Gamma in the first part of the grid
    int n_cols, n_panels, cols_per_cta, pack_chunks, tile_bytes;
    const uint8_t *colmask;
    const uint32_t *coloff, *panel_base;
    uint8_t *packed_payload;          // NULL: no packed form
    long long capacity_tiles;
    TcPackArgs tc;                    // tc.n_groups == 0: no second packed form
    // used by the single-launch kernel only, which also writes what the count and scan launches write
    int32_t *row_ptr_out;
    uint8_t *colmask_out;
    uint32_t *coloff_out, *panel_base_out;
    PackedHeader *hdr;
    PackedHeader hdr_init;
    uint8_t *tc_mask_out;
    uint32_t *tc_off_out, *tc_gcnt_out;
    int tc_kc_ch;
    int pack_parts, tc_parts;         // CTAs sharing the words of one tile column / one K-group
    int *status;
};

// The last compaction launch: CTAs [0, NBo * fill_parts) write col_idx and the canonical payload, the rest write
// the packed tiles.  T is the storage type of a weight, DT its bsp_dtype.
template <typename T, int DT>
__global__ void __launch_bounds__(kThreads) fill_pack_kernel(const FillPackArgs a)
{
    const int n_fill = a.NBo * a.fill_parts;
    if ((int)blockIdx.x < n_fill) {
        const int l = (int)blockIdx.x / a.fill_parts;
        csr_fill_body<T>(l, (int)blockIdx.x % a.fill_parts, a.fill_parts, (const T *)a.W, a.gamma, a.NBi, a.I, a.HK, a.bo,
                         a.bi, a.row_ptr[l], a.col_idx, (T *)a.payload, a.capacity_blocks);
    } else {
        const int b = (int)blockIdx.x - n_fill;
        const int n_pack = a.packed_payload ? a.pack_chunks * a.n_panels : 0;
        if (b < n_pack) {
            pack_body<DT>(b % a.pack_chunks, b / a.pack_chunks, a.W, a.gamma, a.O, a.I, a.HK, a.bo, a.bi, a.NBi, a.n_cols,
                          a.cols_per_cta, a.tile_bytes, a.colmask, a.coloff, a.panel_base, a.packed_payload,
                          a.capacity_tiles);
        } else if constexpr (DT != BSP_F32) {
            const int c = b - n_pack;
            tc_pack_body<DT == BSP_I8 ? 1 : 2>(c % a.tc.chunks, c / a.tc.chunks, a.tc, a.W, a.gamma, a.O, a.I, a.HK, a.bo, a.bi, a.NBi);
        }
    }
}

// Layers of up to kSmallBlocks blocks: the whole compaction in ONE launch.  Gamma fits in shared memory, so
// every CTA counts for itself the stored blocks, tiles or super-tiles that precede its share (what the count
// and scan launches hand over through memory in the general path) and writes its part of the index arrays.
constexpr int kSmallBlocks = 4096;

// Sum of v over the CTA's threads; every thread of the CTA must call it.
__device__ __forceinline__ int block_sum(int v, int *warp_sums)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = v;
    __syncthreads();
    int tot = 0;
    for (int w = 0; w < kThreads / 32; ++w) tot += warp_sums[w];
    return tot;
}

// Non-zero bytes among the first n bytes of Gamma in shared memory (the array is 16-byte aligned), four per load:
// this thread's share; the caller adds the shares with block_sum().
__device__ __forceinline__ int ones_share(const uint8_t *g, int n)
{
    int c = 0;
    const int nw = n >> 2;
    for (int i = threadIdx.x; i < nw; i += kThreads) c += __popc(__vsetne4(((const uint32_t *)g)[i], 0u));
    if ((int)threadIdx.x < (n & 3)) c += g[(nw << 2) + threadIdx.x] ? 1 : 0;
    return c;
}

// True if a block of Gamma (in shared memory) with a one overlaps output channels [o_lo, o_hi] x input channels [c_lo, c_hi].
__device__ __forceinline__ bool any_kept(const uint8_t *g, int o_lo, int o_hi, int c_lo, int c_hi, int bo, int bi, int NBo, int NBi)
{
    bool any = false;
    for (int lb = o_lo >> lg(bo); lb <= (o_hi >> lg(bo)) && lb < NBo; ++lb)
        for (int cb = c_lo >> lg(bi); cb <= (c_hi >> lg(bi)) && cb < NBi; ++cb) any |= g[lb * NBi + cb] != 0;
    return any;
}

template <typename T, int DT>
__global__ void __launch_bounds__(kThreads) compact_small_kernel(const FillPackArgs a)
{
    __shared__ __align__(16) uint8_t s_gamma[kSmallBlocks];
    __shared__ int s_sum[kThreads / 32];
    const int NB = a.NBo * a.NBi;
    const bool word_ok = (((uintptr_t)a.gamma) & 3u) == 0;
    for (int i = threadIdx.x * 4; i < NB; i += kThreads * 4) {
        if (i + 4 <= NB && word_ok) *(uint32_t *)(s_gamma + i) = *(const uint32_t *)(a.gamma + i);
        else for (int q = i; q < min(NB, i + 4); ++q) s_gamma[q] = a.gamma[q];
    }
    __syncthreads();
    const int n_fill = a.NBo * a.fill_parts;
    if ((int)blockIdx.x < n_fill) {
        const int l = (int)blockIdx.x / a.fill_parts, part = (int)blockIdx.x % a.fill_parts;
        const int first = block_sum(ones_share(s_gamma, l * a.NBi), s_sum);
        const int cnt = csr_fill_body<T>(l, part, a.fill_parts, (const T *)a.W, a.gamma, a.NBi, a.I, a.HK, a.bo, a.bi, first,
                                         a.col_idx, (T *)a.payload, a.capacity_blocks);
        if (part == 0 && threadIdx.x == 0) {
            a.row_ptr_out[l] = first;
            if (l == a.NBo - 1) {
                a.row_ptr_out[a.NBo] = first + cnt;
                if ((long long)(first + cnt) > a.capacity_blocks) atomicMax(a.status, (int)BSP_ERR_CAPACITY);
            }
        }
        return;
    }
    const int b = (int)blockIdx.x - n_fill;
    const int n_pack = a.packed_payload ? a.pack_chunks * a.n_panels * a.pack_parts : 0;
    if (b < n_pack) {
        const int part = b % a.pack_parts, bc = b / a.pack_parts;
        const int chunk = bc % a.pack_chunks, panel = bc / a.pack_chunks;
        const int col_lo = chunk * a.cols_per_cta, col_hi = min(a.n_cols, col_lo + a.cols_per_cta);
        // stored tiles of the panels above, and of this panel in the columns before col_lo
        int c = 0;
        const int tiles_above = panel * kPanelRows * a.n_cols;
        if (a.bo == kTile && a.bi == kTile) {
            c = ones_share(s_gamma, tiles_above);             // an 8x8 block is a tile
        } else {
            for (int q = threadIdx.x; q < tiles_above; q += kThreads) {
                const int tr = q / a.n_cols, col = q % a.n_cols;
                c += any_kept(s_gamma, tr * kTile, tr * kTile + kTile - 1, col * kTile, col * kTile + kTile - 1, a.bo, a.bi, a.NBo, a.NBi) ? 1 : 0;
            }
        }
        const int base = block_sum(c, s_sum);
        c = 0;
        for (int q = threadIdx.x; q < kPanelRows * col_lo; q += kThreads) {
            const int tr = panel * kPanelRows + q / col_lo, col = q % col_lo;
            if (tr * kTile < a.O)
                c += any_kept(s_gamma, tr * kTile, tr * kTile + kTile - 1, col * kTile, col * kTile + kTile - 1, a.bo, a.bi, a.NBo, a.NBi) ? 1 : 0;
        }
        int before = block_sum(c, s_sum);
        if (chunk == 0 && part == 0 && threadIdx.x == 0) a.panel_base_out[panel] = (uint32_t)base;
        for (int col = col_lo; col < col_hi; ++col) {
            // lane r of every warp looks at tile row r; the ballot is the column's mask
            const int lane = threadIdx.x & 31;
            const int o0 = (panel * kPanelRows + lane) * kTile;
            const bool bit = lane < kPanelRows && o0 < a.O &&
                             any_kept(s_gamma, o0, o0 + kTile - 1, col * kTile, col * kTile + kTile - 1, a.bo, a.bi, a.NBo, a.NBi);
            const unsigned m = __ballot_sync(0xFFFFFFFFu, bit);
            if (part == 0 && threadIdx.x == 0) {
                a.colmask_out[(size_t)panel * a.n_cols + col] = (uint8_t)m;
                a.coloff_out[(size_t)panel * a.n_cols + col] = (uint32_t)before;
            }
            if (m) pack_tiles<DT>(m, (unsigned)(base + before), panel, col, a.W, s_gamma, a.O, a.I, a.HK, a.bo, a.bi, a.NBi,
                                  a.tile_bytes, a.packed_payload, a.capacity_tiles, part, a.pack_parts);
            before += __popc(m);
        }
        if (panel == a.n_panels - 1 && chunk == a.pack_chunks - 1 && part == 0 && threadIdx.x == 0) {
            const int total = base + before;
            a.panel_base_out[a.n_panels] = (uint32_t)total;
            PackedHeader h = a.hdr_init;
            h.n_tiles = total;
            *a.hdr = h;
            if ((long long)total > a.capacity_tiles) atomicMax(a.status, (int)BSP_ERR_CAPACITY);
        }
        return;
    }
    if constexpr (DT != BSP_F32) {
        const TcPackArgs &t = a.tc;
        const int part = (b - n_pack) % a.tc_parts, cidx = (b - n_pack) / a.tc_parts;
        const int chunk = cidx % t.chunks, g = cidx / t.chunks;
        const int kc_lo = chunk * t.kc_per_cta, kc_hi = min(t.n_kc, kc_lo + t.kc_per_cta);
        auto st_kept = [&](int sr, int kc) -> bool {
            const int o0 = sr * kTcSuperRow;
            if (o0 >= a.O) return false;
            return any_kept(s_gamma, o0, min(a.O, o0 + kTcSuperRow) - 1, kc * a.tc_kc_ch, kc * a.tc_kc_ch + a.tc_kc_ch - 1, a.bo,
                            a.bi, a.NBo, a.NBi);
        };
        // Stored super-tiles (gap fillers included) of n_masks (group, K-group) pairs, pair i being (g0 + i / n_kc,
        // i % n_kc): eight consecutive lanes look at the eight super-rows of one pair, a ballot assembles its mask.
        auto count_stored = [&](int g0, int n_masks) -> int {
            int cnt = 0;
            const int lane = threadIdx.x & 31;
            for (int q0 = 0; q0 < n_masks * kTcGroupRows; q0 += kThreads) {
                const int q = q0 + threadIdx.x, i = q >> 3;
                const bool bit = i < n_masks && st_kept((g0 + i / t.n_kc) * kTcGroupRows + (q & 7), i % t.n_kc);
                const unsigned m = (__ballot_sync(0xFFFFFFFFu, bit) >> (lane & 24)) & 0xFFu;
                if ((lane & 7) == 0) cnt += __popc(tc_fill_gaps(m));
            }
            return cnt;
        };
        const int base = block_sum(count_stored(0, g * t.n_kc), s_sum);
        // chunk 0 counts the whole group (it writes gcnt), the others the K-groups before their own
        const int upto = (chunk == 0) ? t.n_kc : kc_lo;
        const int c = count_stored(g, upto);
        const int counted = block_sum(c, s_sum);
        int before = (chunk == 0) ? 0 : counted;
        if (chunk == 0 && part == 0 && threadIdx.x == 0) {
            a.tc_gcnt_out[g] = (uint32_t)counted;
            if ((long long)(base + counted) > t.capacity) atomicMax(a.status, (int)BSP_ERR_CAPACITY);
        }
        for (int kc = kc_lo; kc < kc_hi; ++kc) {
            const int lane = threadIdx.x & 31;           // lane r of every warp looks at super-row r
            const unsigned m = tc_fill_gaps(__ballot_sync(0xFFFFFFFFu, lane < kTcGroupRows && st_kept(g * kTcGroupRows + lane, kc)));
            if (part == 0 && threadIdx.x == 0) {
                a.tc_mask_out[(size_t)g * t.n_kc + kc] = (uint8_t)m;
                a.tc_off_out[(size_t)g * t.n_kc + kc] = (uint32_t)before;
            }
            if (m) tc_pack_tiles<DT == BSP_I8 ? 1 : 2>(m, (unsigned)(base + before), g, kc, t, a.W, s_gamma, a.O, a.I, a.HK, a.bo, a.bi, a.NBi, part, a.tc_parts);
            before += __popc(m);
        }
    }
}

// Third packed form: Gamma (.) W in the layout of W, [O][H][K][I], one 16-byte chunk of input channels per thread and
// step (four loads in flight per thread), the channels of zeroed blocks cleared.  A "row" below is one (o, tap).
template <int esz>
__global__ void __launch_bounds__(kThreads)
masked_dense_kernel(const void *__restrict__ W, const uint8_t *__restrict__ gamma, int O, int I, int HK, int bo, int bi,
                    int NBi, uint8_t *__restrict__ out)
{
    const bool aligned = (((uintptr_t)W) & 15u) == 0;
    const int cpr = I * esz / 16;                     // chunks per row
    constexpr int cpc = 16 / esz;
    const long long total = (long long)O * HK * cpr, stride = (long long)gridDim.x * kThreads;
    for (long long e0 = (long long)blockIdx.x * kThreads + threadIdx.x; e0 < total; e0 += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long e = e0 + u * stride;
            if (e >= total) continue;
            const int ot = (int)(e / cpr), c = (int)(e - (long long)ot * cpr);
            const int o = ot / HK, tap = ot - o * HK;
            if (aligned) {
                v[u] = w_chunk<esz>(W, gamma, o, tap, c * cpc, O, I, HK, bo, bi, NBi);
            } else {
                // W only 4-byte aligned: word by word (the channels of a word lie in one block: b_i is a multiple of 4)
                uint32_t w[4];
                for (int q = 0; q < 4; ++q) {
                    const int ch = c * cpc + q * (4 / esz);
                    const bool on = gamma[(size_t)(o >> lg(bo)) * NBi + (ch >> lg(bi))] != 0;
                    w[q] = on ? *(const uint32_t *)((const uint8_t *)W + ((size_t)ot * I + ch) * esz) : 0u;
                }
                v[u] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long e = e0 + u * stride;
            if (e < total) *(uint4 *)(out + e * 16) = v[u];
        }
    }
}

__global__ void count_ones_kernel(const uint8_t *__restrict__ gamma, long long n, unsigned long long *out)
{
    unsigned long long c = 0;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        c += gamma[i] ? 1 : 0;
    for (int d = 16; d > 0; d >>= 1) c += __shfl_down_sync(0xFFFFFFFFu, c, d);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(out, c);
}

}  // namespace

bsp_status launch_count(const uint8_t *gamma, int64_t n, unsigned long long *out, cudaStream_t st)
{
    BSP_CUDA_OK(cudaMemsetAsync(out, 0, sizeof(unsigned long long), st));
    int64_t grid = (n + 255) / 256;
    if (grid > 296) grid = 296;
    if (grid < 1) grid = 1;
    count_ones_kernel<<<(unsigned)grid, 256, 0, st>>>(gamma, n, out);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

bsp_status launch_compact(const bsp_wdesc &wd, const void *W, const uint8_t *gamma, int32_t *row_ptr,
                          int32_t *col_idx, void *payload, void *packed, int64_t capacity_blocks, void *ws,
                          cudaStream_t st)
{
    const int NBo = wd.O / wd.bo, NBi = wd.I / wd.bi, HK = wd.H * wd.K;
    const PackedLayout L = packed_layout(wd, capacity_blocks);
    int *status = (int *)ws;
    int *row_cnt = (int *)((char *)ws + kWsHeader);
    int *panel_cnt = row_cnt + NBo;
    uint8_t *pk = (uint8_t *)packed;
    uint8_t *colmask = pk ? pk + L.off_colmask : nullptr;
    uint32_t *coloff = pk ? (uint32_t *)(pk + L.off_coloff) : nullptr;
    uint32_t *panel_base = pk ? (uint32_t *)(pk + L.off_panelbase) : nullptr;

    PackedHeader h = {};
    h.magic = kPackedMagic; h.dtype = wd.wtype; h.O = wd.O; h.I = wd.I; h.H = wd.H; h.K = wd.K;
    h.bo = wd.bo; h.bi = wd.bi; h.n_panels = L.n_panels; h.n_cols = L.n_cols; h.tile_bytes = L.tile_bytes;
    h.capacity_tiles = (int32_t)L.capacity_tiles; h.n_tiles = 0;
    h.off_colmask = (int32_t)L.off_colmask; h.off_coloff = (int32_t)L.off_coloff;
    h.off_panelbase = (int32_t)L.off_panelbase; h.off_payload = (int64_t)L.off_payload;
    h.off_tc_payload = (int64_t)L.tc.off_payload;
    const bool gm_on = pk != nullptr && L.gm.enabled;
    h.forms = pk ? (kFormTile | (L.tc.enabled ? kFormSuper : 0) | (gm_on ? kFormDense : 0)) : 0;
    auto pack_dense = [&]() -> bsp_status {
        if (!gm_on) return BSP_OK;
        const long long chunks = (long long)wd.O * HK * wd.I * elem_bytes(wd.wtype) / 16;
        long long g = (chunks + 4LL * kThreads - 1) / (4LL * kThreads);
        if (g > 2368) g = 2368;
        if (g < 1) g = 1;
        uint8_t *out = pk + L.gm.off_payload;
        if (wd.wtype == BSP_I8) masked_dense_kernel<1><<<(unsigned)g, kThreads, 0, st>>>(W, gamma, wd.O, wd.I, HK, wd.bo, wd.bi, NBi, out);
        else if (wd.wtype == BSP_BF16) masked_dense_kernel<2><<<(unsigned)g, kThreads, 0, st>>>(W, gamma, wd.O, wd.I, HK, wd.bo, wd.bi, NBi, out);
        else masked_dense_kernel<4><<<(unsigned)g, kThreads, 0, st>>>(W, gamma, wd.O, wd.I, HK, wd.bo, wd.bi, NBi, out);
        BSP_CUDA_OK(cudaGetLastError());
        return BSP_OK;
    };

    const bool tc_on = pk != nullptr && L.tc.enabled;
    TcIndexArgs ti = {};
    ti.n_panels = pk ? L.n_panels : 0;
    if (tc_on) {
        ti.n_groups = L.tc.n_groups; ti.n_kc = L.tc.n_kc; ti.kc_ch = L.tc.kc_ch;
        ti.mask = pk + L.tc.off_mask; ti.off = (uint32_t *)(pk + L.tc.off_off); ti.gcnt = (uint32_t *)(pk + L.tc.off_gcnt);
    }
    FillPackArgs a = {};
    a.W = W; a.gamma = gamma; a.O = wd.O; a.I = wd.I; a.HK = HK; a.bo = wd.bo; a.bi = wd.bi; a.NBo = NBo; a.NBi = NBi;
    a.row_ptr = row_ptr; a.col_idx = col_idx; a.payload = payload; a.capacity_blocks = capacity_blocks;
    // enough CTAs per row to give every SM some of the payload copy
    a.fill_parts = payload ? (296 + NBo - 1) / NBo : 1;
    if (a.fill_parts > 16) a.fill_parts = 16;
    if (a.fill_parts < 1) a.fill_parts = 1;
    a.n_cols = L.n_cols; a.n_panels = L.n_panels; a.tile_bytes = L.tile_bytes;
    // one tile column per CTA unless that would make a needlessly large grid
    a.cols_per_cta = (int)(((long long)L.n_cols * L.n_panels + 1183) / 1184);
    if (a.cols_per_cta < 1) a.cols_per_cta = 1;
    a.pack_chunks = (L.n_cols + a.cols_per_cta - 1) / a.cols_per_cta;
    a.colmask = colmask; a.coloff = coloff; a.panel_base = panel_base;
    a.packed_payload = pk ? pk + L.off_payload : nullptr;
    a.capacity_tiles = (long long)L.capacity_tiles;
    if (tc_on) {
        a.tc.n_groups = L.tc.n_groups; a.tc.n_kc = L.tc.n_kc; a.tc.st_bytes = L.tc.st_bytes;
        a.tc.kc_per_cta = (int)(((long long)L.tc.n_kc * L.tc.n_groups + 1183) / 1184);
        if (a.tc.kc_per_cta < 1) a.tc.kc_per_cta = 1;
        a.tc.chunks = (L.tc.n_kc + a.tc.kc_per_cta - 1) / a.tc.kc_per_cta;
        a.tc.mask = ti.mask; a.tc.off = ti.off; a.tc.gcnt = ti.gcnt;
        a.tc.payload = pk + L.tc.off_payload; a.tc.capacity = (long long)L.tc.capacity; a.tc.status = status;
    }
    const unsigned grid = (unsigned)(NBo * a.fill_parts + (pk ? a.pack_chunks * L.n_panels : 0) +
                                     (tc_on ? a.tc.chunks * a.tc.n_groups : 0));
    const size_t smem = (size_t)NBi * sizeof(int);
    if ((long long)NBo * NBi <= kSmallBlocks) {
        // enough CTAs per row, tile column and K-group that a thread moves about four pieces: 16-byte chunks for
        // bf16 (two per item in the first packed form), 32-bit words otherwise
        auto parts_for = [](long long items, int per_thread) {
            const long long p = (items + (long long)per_thread * kThreads - 1) / ((long long)per_thread * kThreads);
            return (int)(p < 1 ? 1 : (p > 8 ? 8 : p));
        };
        const bool chunks = wd.wtype == BSP_BF16 && wd.I % 8 == 0 && ((uintptr_t)W & 15u) == 0;
        const bool tc_chunks = wd.wtype != BSP_F32 && (wd.I * (wd.wtype == BSP_I8 ? 1 : 2)) % 16 == 0 && ((uintptr_t)W & 15u) == 0;
        a.pack_parts = chunks ? parts_for((long long)kPanelRows * ((HK + 1) / 2) * 8, 2) : parts_for((long long)kPanelRows * L.tile_bytes / 4, 4);
        a.tc_parts = !tc_on ? 1 : tc_chunks ? parts_for((long long)kTcGroupRows * L.tc.n_units * 32, 4) : parts_for((long long)kTcGroupRows * L.tc.st_bytes / 4, 4);
        if (payload) {
            const size_t esz = wd.wtype == BSP_F32 ? 4 : (wd.wtype == BSP_BF16 ? 2 : 1);
            const long long row_pieces = (long long)NBi * wd.bo * HK * ((wd.bi * esz + 15) / 16);   // a row with every block stored
            a.fill_parts = parts_for(row_pieces / 2, 4);
        }
        const unsigned grid_small = (unsigned)(NBo * a.fill_parts + (pk ? a.pack_chunks * L.n_panels * a.pack_parts : 0) +
                                               (tc_on ? a.tc.chunks * a.tc.n_groups * a.tc_parts : 0));
        a.row_ptr_out = row_ptr; a.colmask_out = colmask; a.coloff_out = coloff; a.panel_base_out = panel_base;
        a.hdr = (PackedHeader *)pk; a.hdr_init = h;
        a.tc_mask_out = ti.mask; a.tc_off_out = ti.off; a.tc_gcnt_out = ti.gcnt; a.tc_kc_ch = ti.kc_ch;
        a.status = status;
        if (wd.wtype == BSP_I8) compact_small_kernel<uint8_t, BSP_I8><<<grid_small, kThreads, smem, st>>>(a);
        else if (wd.wtype == BSP_BF16) compact_small_kernel<uint16_t, BSP_BF16><<<grid_small, kThreads, smem, st>>>(a);
        else compact_small_kernel<uint32_t, BSP_F32><<<grid_small, kThreads, smem, st>>>(a);
        BSP_CUDA_OK(cudaGetLastError());
        return pack_dense();
    }
    count_kernel<<<NBo + ti.n_panels + ti.n_groups, kThreads, 0, st>>>(gamma, NBo, NBi, wd.bo, wd.bi, wd.O, L.n_cols,
                                                                       row_cnt, colmask, coloff, panel_cnt, ti);
    BSP_CUDA_OK(cudaGetLastError());
    scan_kernel<<<1, kThreads, 0, st>>>(row_cnt, NBo, row_ptr, panel_cnt, L.n_panels, panel_base, (PackedHeader *)pk, h,
                                        (long long)capacity_blocks, (long long)L.capacity_tiles, status);
    BSP_CUDA_OK(cudaGetLastError());
    if (wd.wtype == BSP_I8) fill_pack_kernel<uint8_t, BSP_I8><<<grid, kThreads, smem, st>>>(a);
    else if (wd.wtype == BSP_BF16) fill_pack_kernel<uint16_t, BSP_BF16><<<grid, kThreads, smem, st>>>(a);
    else fill_pack_kernel<uint32_t, BSP_F32><<<grid, kThreads, smem, st>>>(a);
    BSP_CUDA_OK(cudaGetLastError());
    return pack_dense();
}

}  // namespace bsp
