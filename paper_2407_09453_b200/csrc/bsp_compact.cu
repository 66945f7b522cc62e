// Compaction of Gamma (.) W: compressed block rows (row_ptr, col_idx, canonical payload) and the packed form read by
// the product kernel.  Section "Block Sparsity in a Matrix" (compress block row) and Section "Subvolumes, Data
// Compression, and Data Movements" of the paper.
#include "bsp_internal.cuh"

namespace bsp {

PackedLayout packed_layout(const bsp_wdesc &wd)
{
    PackedLayout L;
    const int esz = elem_bytes(wd.wtype);
    L.enabled = ((long long)wd.I * esz) % 16 == 0 && wd.O % 8 == 0;
    L.off_payload = 256;
    L.total_bytes = align_up(L.off_payload + (L.enabled ? (size_t)wd.O * wd.H * wd.K * wd.I * esz : 0) + 256, 256);
    return L;
}

namespace {

constexpr int kThreads = 256;

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

// The same count over the first n bytes of Gamma in global memory (layers whose Gamma does not fit shared memory): 16-byte
// loads, eight in flight per thread, when the addresses allow.
__device__ __forceinline__ int ones_share_global(const uint8_t *__restrict__ g, int n)
{
    int c = 0;
    if ((((uintptr_t)g) & 15u) == 0) {
        const uint4 *g4 = (const uint4 *)g;
        const int n4 = n >> 4;
        for (int i0 = threadIdx.x; i0 < n4; i0 += 8 * kThreads) {
            uint4 q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * kThreads;
                q[u] = i < n4 ? __ldg(g4 + i) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                c += __popc(__vsetne4(q[u].x, 0u)) + __popc(__vsetne4(q[u].y, 0u)) + __popc(__vsetne4(q[u].z, 0u)) + __popc(__vsetne4(q[u].w, 0u));
        }
        for (int i = (n4 << 4) + threadIdx.x; i < n; i += kThreads) c += g[i] ? 1 : 0;
    } else {
        for (int i = threadIdx.x; i < n; i += kThreads) c += g[i] ? 1 : 0;
    }
    return c;
}

// The packed form: Gamma (.) W in the layout of W, [O][H][K][I], the channels of zeroed blocks cleared.  CTA `idx` of
// `n_ctas` takes every n_ctas-th stretch of 16-byte chunks, one chunk of input channels per thread and step, four loads
// in flight per thread.  A "row" below is one (o, tap).
template <int esz>
__device__ __forceinline__ void dense_body(int idx, int n_ctas, const void *__restrict__ W, const uint8_t *gamma, int O, int I,
                                           int HK, int bo, int bi, int NBi, uint8_t *__restrict__ out)
{
    const bool aligned = (((uintptr_t)W) & 15u) == 0;
    const int cpr = I * esz / 16;                     // chunks per row
    constexpr int cpc = 16 / esz;
    const long long total = (long long)O * HK * cpr, stride = (long long)n_ctas * kThreads;
    const bool small = total < (1ll << 31);
    for (long long e0 = (long long)idx * kThreads + threadIdx.x; e0 < total; e0 += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long e = e0 + u * stride;
            if (e >= total) continue;
            // (a 64-bit division costs an order of magnitude more than a 32-bit one: taken only by layers that need it)
            const int ot = small ? (int)((unsigned)e / (unsigned)cpr) : (int)(e / cpr);
            const int c = (int)(e - (long long)ot * cpr);
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

struct CompactArgs {
    const void *W;
    const uint8_t *gamma;
    int O, I, HK, bo, bi, NBo, NBi;
    const int32_t *row_ptr;           // multi-launch path: written by the scan launch
    int32_t *row_ptr_out;             // single-launch path
    int32_t *col_idx;
    void *payload;
    long long capacity_blocks;
    int fill_parts;                   // CTAs per row of Gamma in the first part of the grid
    uint8_t *dense;                   // packed form (NULL: none)
    int dense_ctas;                   // CTAs of the second part of the grid
    PackedHeader *hdr;
    PackedHeader hdr_init;
    int *status;
};

// The whole compaction in ONE launch: CTAs [0, NBo * fill_parts) write col_idx and the canonical payload, one row of
// Gamma each, the rest write the packed form.  Every CTA of the first part counts for itself the stored blocks that
// precede its row (no scan launch, nobody waits): from a copy of Gamma in shared memory for layers of up to
// kSmallBlocks blocks, from global memory (through L2, while the other CTAs write the packed form) for larger ones.
// T is the storage type of a weight.
constexpr int kSmallBlocks = 4096;

template <typename T, bool kBig>
__global__ void __launch_bounds__(kThreads, 5) compact_kernel(const CompactArgs a)
{
    __shared__ __align__(16) uint8_t s_gamma[kBig ? 16 : kSmallBlocks];
    __shared__ int s_sum[kThreads / 32];
    const int n_fill = a.NBo * a.fill_parts;
    if ((int)blockIdx.x >= n_fill) {
        if ((int)blockIdx.x == n_fill && threadIdx.x == 0 && a.hdr != nullptr) *a.hdr = a.hdr_init;
        if (a.dense != nullptr)
            dense_body<(int)sizeof(T)>((int)blockIdx.x - n_fill, a.dense_ctas, a.W, a.gamma, a.O, a.I, a.HK, a.bo, a.bi, a.NBi, a.dense);
        return;
    }
    const int l = (int)blockIdx.x / a.fill_parts, part = (int)blockIdx.x % a.fill_parts;
    int first;
    if constexpr (kBig) {
        first = block_sum(ones_share_global(a.gamma, l * a.NBi), s_sum);      // (NB_o NB_i < 2^31: checked by the host)
    } else {
        const int NB = a.NBo * a.NBi;
        const bool word_ok = (((uintptr_t)a.gamma) & 3u) == 0;
        for (int i = threadIdx.x * 4; i < NB; i += kThreads * 4) {
            if (i + 4 <= NB && word_ok) *(uint32_t *)(s_gamma + i) = *(const uint32_t *)(a.gamma + i);
            else for (int q = i; q < min(NB, i + 4); ++q) s_gamma[q] = a.gamma[q];
        }
        __syncthreads();
        first = block_sum(ones_share(s_gamma, l * a.NBi), s_sum);
    }
    const int cnt = csr_fill_body<T>(l, part, a.fill_parts, (const T *)a.W, a.gamma, a.NBi, a.I, a.HK, a.bo, a.bi, first,
                                     a.col_idx, (T *)a.payload, a.capacity_blocks);
    if (part == 0 && threadIdx.x == 0) {
        a.row_ptr_out[l] = first;
        if (l == a.NBo - 1) {
            a.row_ptr_out[a.NBo] = first + cnt;
            if ((long long)(first + cnt) > a.capacity_blocks) atomicMax(a.status, (int)BSP_ERR_CAPACITY);
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
    const PackedLayout L = packed_layout(wd);
    int *status = (int *)ws;
    uint8_t *pk = (uint8_t *)packed;
    const bool dense_on = pk != nullptr && L.enabled;
    const int esz = elem_bytes(wd.wtype);

    CompactArgs a = {};
    a.W = W; a.gamma = gamma; a.O = wd.O; a.I = wd.I; a.HK = HK; a.bo = wd.bo; a.bi = wd.bi; a.NBo = NBo; a.NBi = NBi;
    a.row_ptr = row_ptr; a.row_ptr_out = row_ptr; a.col_idx = col_idx; a.payload = payload; a.capacity_blocks = capacity_blocks;
    a.dense = dense_on ? pk + L.off_payload : nullptr;
    a.hdr = (PackedHeader *)pk; a.status = status;
    PackedHeader &h = a.hdr_init;
    h.magic = kPackedMagic; h.dtype = wd.wtype; h.O = wd.O; h.I = wd.I; h.H = wd.H; h.K = wd.K; h.bo = wd.bo; h.bi = wd.bi;
    h.forms = dense_on ? kFormDense : 0; h.off_payload = (int64_t)L.off_payload;
    // packed form: four 16-byte chunks per thread and pass, at most 16 CTAs per SM's worth of CTAs
    const long long chunks = dense_on ? (long long)wd.O * HK * wd.I * esz / 16 : 0;
    long long dg = (chunks + 4LL * kThreads - 1) / (4LL * kThreads);
    if (dg > 2368) dg = 2368;
    a.dense_ctas = dense_on ? (int)(dg < 1 ? 1 : dg) : (pk ? 1 : 0);      // (a packed buffer without the form still gets its header)
    const size_t smem = (size_t)NBi * sizeof(int);

    if ((long long)NBo * NBi <= kSmallBlocks) {
        // enough CTAs per row that a thread moves about four pieces of the canonical payload
        a.fill_parts = 1;
        if (payload) {
            const long long row_pieces = (long long)NBi * wd.bo * HK * ((wd.bi * esz + 15) / 16);   // a row with every block stored
            const long long p = (row_pieces / 2 + 4LL * kThreads - 1) / (4LL * kThreads);
            a.fill_parts = (int)(p < 1 ? 1 : (p > 8 ? 8 : p));
        }
        const unsigned grid = (unsigned)(NBo * a.fill_parts + a.dense_ctas);
        if (wd.wtype == BSP_I8) compact_kernel<uint8_t, false><<<grid, kThreads, smem, st>>>(a);
        else if (wd.wtype == BSP_BF16) compact_kernel<uint16_t, false><<<grid, kThreads, smem, st>>>(a);
        else compact_kernel<uint32_t, false><<<grid, kThreads, smem, st>>>(a);
        BSP_CUDA_OK(cudaGetLastError());
        return BSP_OK;
    }
    if ((long long)NBo * NBi > 0x7FFFFFFF) return BSP_ERR_SHAPE;
    // enough CTAs per row to give every SM some of the payload copy
    a.fill_parts = payload ? (296 + NBo - 1) / NBo : 1;
    if (a.fill_parts > 16) a.fill_parts = 16;
    if (a.fill_parts < 1) a.fill_parts = 1;
    const unsigned grid = (unsigned)(NBo * a.fill_parts + a.dense_ctas);
    if (wd.wtype == BSP_I8) compact_kernel<uint8_t, true><<<grid, kThreads, smem, st>>>(a);
    else if (wd.wtype == BSP_BF16) compact_kernel<uint16_t, true><<<grid, kThreads, smem, st>>>(a);
    else compact_kernel<uint32_t, true><<<grid, kThreads, smem, st>>>(a);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // namespace bsp
