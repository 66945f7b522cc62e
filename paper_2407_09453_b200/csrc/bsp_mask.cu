// Gamma builder: per-block importance and selection of the n_zero lowest blocks.
// Eq. (1), Eq. (2) and Section "Predetermined Sparsity ratio and Full Training Ahead" of the paper.
#include "bsp_internal.cuh"

namespace bsp {
namespace {

constexpr int kScoreThreads = 256;
constexpr int kSelectThreads = 1024;

// One 4-byte word of W holds 1 fp32, 2 bf16 or 4 int8 values, lowest channel in the lowest bytes.
template <int DT> struct Acc;
template <> struct Acc<BSP_F32> { using type = double; };
template <> struct Acc<BSP_BF16> { using type = double; };
template <> struct Acc<BSP_I8> { using type = long long; };

// Measures of one weight: BSP_NORM_L2 (w^2), BSP_NORM_L1 (|w|), and for the variance two passes over the block:
// kNormSum (w, for the block mean) and BSP_NORM_VAR ((w - mean)^2, with the subtraction, the product and the addition
// each rounded on its own, never fused: the float64 result must not depend on what the compiler contracts).
constexpr int kNormSum = 3;

template <int NORM>
__device__ __forceinline__ void add_value(double v, double &acc, double mean)
{
    if constexpr (NORM == BSP_NORM_L2) acc += v * v;
    else if constexpr (NORM == BSP_NORM_L1) acc += fabs(v);
    else if constexpr (NORM == kNormSum) acc += v;
    else { const double d = __dsub_rn(v, mean); acc = __dadd_rn(acc, __dmul_rn(d, d)); }
}

template <int DT, int NORM>
__device__ __forceinline__ void add_word(uint32_t w, typename Acc<DT>::type &acc, double mean)
{
    if constexpr (DT == BSP_F32) {
        add_value<NORM>((double)__uint_as_float(w), acc, mean);
    } else if constexpr (DT == BSP_BF16) {
        add_value<NORM>((double)__uint_as_float(w << 16), acc, mean);
        add_value<NORM>((double)__uint_as_float(w & 0xFFFF0000u), acc, mean);
    } else {
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const long long v = (long long)(int8_t)((w >> (8 * b)) & 0xFFu);
            acc += (NORM == BSP_NORM_L2) ? v * v : (v < 0 ? -v : v);
        }
    }
}

// One thread sums one output row r of one block over (h, k, c) in that order; the thread with r = 0 then
// adds the b_o row sums in order of r.  The order is part of the definition of the float score: it makes
// the float64 result, and so Gamma, independent of the launch shape.  (Each square of a float or bf16 value
// is exact in float64, so a fused multiply-add rounds like a multiply followed by an add.)
// Threads are laid out with consecutive blocks of one block row on consecutive lanes, so that for a fixed
// (r, h, k) a warp reads one contiguous stretch of input channels.
// Sum of one output row r of block B over (h, k, c) in that order, for a block of WORDS 32-bit words per tap.
// Loads of up to nine taps (a whole 3x3 kernel) are issued together, as 16-byte loads when `vec` says that the
// rows are 16-byte aligned; the adds keep the (h, k, c) order.
template <int DT, int NORM, int WORDS, int kBatch>
__device__ __forceinline__ typename Acc<DT>::type row_sum_w(const uint32_t *__restrict__ src, size_t row_words, int HK, bool vec,
                                                            double mean)
{
    using acc_t = typename Acc<DT>::type;
    acc_t pr = 0;
    for (int t = 0; t < HK; t += kBatch) {
        uint32_t w[kBatch][WORDS];
        if constexpr (WORDS % 4 == 0) {
            if (vec) {
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
#pragma unroll
                    for (int j = 0; j < WORDS; j += 4)
                        if (t + u < HK) {
                            const uint4 q = __ldg((const uint4 *)(src + (size_t)u * row_words + j));
                            w[u][j] = q.x; w[u][j + 1] = q.y; w[u][j + 2] = q.z; w[u][j + 3] = q.w;
                        }
            } else {
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
#pragma unroll
                    for (int j = 0; j < WORDS; ++j)
                        if (t + u < HK) w[u][j] = __ldg(src + (size_t)u * row_words + j);
            }
        } else {
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
#pragma unroll
                for (int j = 0; j < WORDS; ++j)
                    if (t + u < HK) w[u][j] = __ldg(src + (size_t)u * row_words + j);
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
#pragma unroll
            for (int j = 0; j < WORDS; ++j)
                if (t + u < HK) add_word<DT, NORM>(w[u][j], pr, mean);
        src += (size_t)kBatch * row_words;
    }
    return pr;
}

// kBatch = taps whose loads are in flight together: 9 (a 3x3 kernel at once), or 1 in the kernels compiled for
// one-tap layers, which then need few registers and keep many CTAs resident.
template <int DT, int NORM, int kBatch>
__device__ __forceinline__ typename Acc<DT>::type row_sum(const uint32_t *__restrict__ W, int I, int HK, int bo, int bi,
                                                          int NBi, long long B, int r, double mean = 0.0)
{
    constexpr int per_word = (DT == BSP_F32) ? 1 : (DT == BSP_BF16 ? 2 : 4);
    const int l = B < (1ll << 31) ? (int)((unsigned)B / (unsigned)NBi) : (int)(B / NBi);     // (64-bit divisions are slow)
    const int iota = (int)(B - (long long)l * NBi);
    const int words = bi / per_word;
    const size_t row_words = (size_t)I / per_word;
    const uint32_t *src = W + ((size_t)(l * bo + r) * HK) * row_words + (size_t)iota * words;
    const bool vec = (((uintptr_t)W) & 15u) == 0 && row_words % 4 == 0;
    switch (words) {
        case 1: return row_sum_w<DT, NORM, 1, kBatch>(src, row_words, HK, vec, mean);
        case 2: return row_sum_w<DT, NORM, 2, kBatch>(src, row_words, HK, vec, mean);
        case 4: return row_sum_w<DT, NORM, 4, kBatch>(src, row_words, HK, vec, mean);
        case 8: return row_sum_w<DT, NORM, 8, kBatch>(src, row_words, HK, vec, mean);
        default: return row_sum_w<DT, NORM, 16, kBatch>(src, row_words, HK, vec, mean);
    }
}

// OR of the keys' bits and OR of their complements, added to span[0] and span[1] (zeroed by the host): a bit
// position set in both differs between some two keys.  The select starts at the highest such bit.  One thread per
// CTA adds, and only bits that are not there yet (atomics on one address are served one after the other).
// Every thread of the CTA must call it.
__device__ __forceinline__ void publish_span(unsigned long long or1, unsigned long long or0, unsigned long long *span)
{
    __shared__ unsigned long long s_or[2][kScoreThreads / 32];
    for (int o = 16; o > 0; o >>= 1) {
        or1 |= __shfl_xor_sync(0xFFFFFFFFu, or1, o);
        or0 |= __shfl_xor_sync(0xFFFFFFFFu, or0, o);
    }
    if ((threadIdx.x & 31) == 0) { s_or[0][threadIdx.x >> 5] = or1; s_or[1][threadIdx.x >> 5] = or0; }
    __syncthreads();
    if (threadIdx.x < 2) {
        unsigned long long v = 0ull;
        for (int w = 0; w < kScoreThreads / 32; ++w) v |= s_or[threadIdx.x][w];
        if (v & ~__ldcg(span + threadIdx.x)) atomicOr(span + threadIdx.x, v);
    }
}

// One-tap layers (H K = 1) with the L2 or L1 measure: one thread per block (consecutive threads take consecutive blocks of
// a block row, so a warp's load of one row r is one contiguous stretch of input channels).  The rows of a block are
// WORDS words each; kRows rows (eight, or four when b_o = 4 or the rows are long) are loaded at a time, every row is summed over its channels in order and the row sums
// are added in order of r: the same order of additions as row_sum followed by the sum over r.
template <int DT, int NORM, int WORDS, int kRows>
__device__ __forceinline__ void score_one_tap(const uint32_t *__restrict__ W, int I, int bo, int NBo, int NBi,
                                              typename Acc<DT>::type *__restrict__ score, unsigned long long *span)
{
    using acc_t = typename Acc<DT>::type;
    constexpr int per_word = (DT == BSP_F32) ? 1 : (DT == BSP_BF16 ? 2 : 4);
    constexpr int kVec = WORDS % 4 == 0 ? 4 : (WORDS % 2 == 0 ? 2 : 1);       // words per load
    const long long NB = (long long)NBo * NBi;
    const size_t row_words = (size_t)I / per_word;
    const bool vec = kVec > 1 && (((uintptr_t)W) & (4u * kVec - 1u)) == 0 && row_words % kVec == 0;
    const bool small = NB < (1ll << 31);
    unsigned long long or1 = 0ull, or0 = 0ull;
    for (long long B = (long long)blockIdx.x * kScoreThreads + threadIdx.x; B < NB; B += (long long)gridDim.x * kScoreThreads) {
        // (a 64-bit division costs an order of magnitude more than a 32-bit one: taken only by layers that need it)
        const int l = small ? (int)((unsigned)B / (unsigned)NBi) : (int)(B / NBi);
        const int iota = (int)(B - (long long)l * NBi);
        const uint32_t *src = W + (size_t)l * bo * row_words + (size_t)iota * WORDS;
        acc_t total = 0;
        for (int r0 = 0; r0 < bo; r0 += kRows) {             // (b_o is a multiple of kRows)
            uint32_t w[kRows][WORDS];
#pragma unroll
            for (int u = 0; u < kRows; ++u) {
                const uint32_t *row = src + (size_t)(r0 + u) * row_words;
                if (vec && kVec == 4) {
#pragma unroll
                    for (int j = 0; j + 3 < WORDS; j += 4) {
                        const uint4 q = __ldg((const uint4 *)(row + j));
                        w[u][j] = q.x; w[u][j + 1] = q.y; w[u][j + 2] = q.z; w[u][j + 3] = q.w;
                    }
                } else if (vec && kVec == 2) {
#pragma unroll
                    for (int j = 0; j + 1 < WORDS; j += 2) {
                        const uint2 q = __ldg((const uint2 *)(row + j));
                        w[u][j] = q.x; w[u][j + 1] = q.y;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < WORDS; ++j) w[u][j] = __ldg(row + j);
                }
            }
#pragma unroll
            for (int u = 0; u < kRows; ++u) {
                acc_t pr = 0;
#pragma unroll
                for (int j = 0; j < WORDS; ++j) add_word<DT, NORM>(w[u][j], pr, 0.0);
                total += pr;
            }
        }
        score[B] = total;
        unsigned long long key;
        memcpy(&key, &total, 8);
        or1 |= key; or0 |= ~key;
    }
    if (span != nullptr) publish_span(or1, or0, span);
}

// A CTA takes groups of 256 / b_o blocks, every `gridDim.x`-th one (a bounded grid of long-lived CTAs instead of one
// short CTA per group: a layer of 4096 x 4096 weights is 8192 groups).
template <int DT, int NORM, int kBatch>
__global__ void __launch_bounds__(kScoreThreads)
score_kernel(const uint32_t *__restrict__ W, int I, int HK, int bo, int bi, int NBo, int NBi,
             typename Acc<DT>::type *__restrict__ score, unsigned long long *span)
{
    using acc_t = typename Acc<DT>::type;
    if constexpr (kBatch == 1 && NORM != BSP_NORM_VAR) {
        constexpr int per_word = (DT == BSP_F32) ? 1 : (DT == BSP_BF16 ? 2 : 4);
        const bool eight = bo % 8 == 0;
        switch (bi / per_word) {
            case 1: if (eight) score_one_tap<DT, NORM, 1, 8>(W, I, bo, NBo, NBi, score, span); else score_one_tap<DT, NORM, 1, 4>(W, I, bo, NBo, NBi, score, span); break;
            case 2: if (eight) score_one_tap<DT, NORM, 2, 8>(W, I, bo, NBo, NBi, score, span); else score_one_tap<DT, NORM, 2, 4>(W, I, bo, NBo, NBi, score, span); break;
            case 4: if (eight) score_one_tap<DT, NORM, 4, 8>(W, I, bo, NBo, NBi, score, span); else score_one_tap<DT, NORM, 4, 4>(W, I, bo, NBo, NBi, score, span); break;
            case 8: score_one_tap<DT, NORM, 8, 4>(W, I, bo, NBo, NBi, score, span); break;
            default: score_one_tap<DT, NORM, 16, 4>(W, I, bo, NBo, NBi, score, span); break;
        }
        return;
    }
    __shared__ acc_t part[kScoreThreads];
    const int blocks_per_cta = kScoreThreads / bo;
    const int bl = threadIdx.x % blocks_per_cta;
    const int r = threadIdx.x / blocks_per_cta;
    const long long NB = (long long)NBo * NBi;
    const long long n_groups = (NB + blocks_per_cta - 1) / blocks_per_cta;
    unsigned long long or1 = 0ull, or0 = 0ull;
    for (long long grp = blockIdx.x; grp < n_groups; grp += gridDim.x) {
        const long long B = grp * blocks_per_cta + bl;
        if constexpr (NORM == BSP_NORM_VAR) {
            // variance about the block's own mean, n = b_o H K b_i entries: the mean from the row sums added in order of
            // r (every thread of the block adds them the same way), then the squared deviations in the same order, over n
            const double n_elems = (double)bo * HK * bi;
            part[threadIdx.x] = (B < NB) ? row_sum<DT, kNormSum, kBatch>(W, I, HK, bo, bi, NBi, B, r) : (acc_t)0;
            __syncthreads();
            double s = 0.0;
            for (int q = 0; q < bo; ++q) s += (double)part[q * blocks_per_cta + bl];
            const double mean = s / n_elems;
            __syncthreads();
            part[threadIdx.x] = (B < NB) ? row_sum<DT, NORM, kBatch>(W, I, HK, bo, bi, NBi, B, r, mean) : (acc_t)0;
            __syncthreads();
            if (B < NB && r == 0) {
                double total = 0.0;
                for (int q = 0; q < bo; ++q) total += (double)part[q * blocks_per_cta + bl];
                const acc_t out = (acc_t)(total / n_elems);
                score[B] = out;
                unsigned long long key;
                memcpy(&key, &out, 8);
                or1 |= key; or0 |= ~key;
            }
        } else {
            part[threadIdx.x] = (B < NB) ? row_sum<DT, NORM, kBatch>(W, I, HK, bo, bi, NBi, B, r) : (acc_t)0;
            __syncthreads();
            if (B < NB && r == 0) {
                acc_t total = 0;
                for (int q = 0; q < bo; ++q) total += part[q * blocks_per_cta + bl];
                score[B] = total;
                unsigned long long key;
                memcpy(&key, &total, 8);
                or1 |= key; or0 |= ~key;
            }
        }
        __syncthreads();
    }
    if (span != nullptr) publish_span(or1, or0, span);
}

// Scores are non-negative, so the bit pattern of a float64 orders like the value, as does an int64.
// One CTA ranks one segment (the whole layer, or one row of Gamma): an 8-pass most-significant-digit
// radix select finds the key T of the n_zero-th smallest (key, index) pair and how many keys equal to T
// are still to be zeroed; a final pass in index order writes Gamma, zeroing the keys below T and the first
// `ties` keys equal to T.
__global__ void __launch_bounds__(kSelectThreads)
select_kernel(const unsigned long long *__restrict__ key, long long seg_len, long long n_zero,
              uint8_t *__restrict__ gamma)
{
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_k;
    __shared__ unsigned int warp_cnt[kSelectThreads / 32];
    __shared__ long long s_run;

    const unsigned long long *k = key + (size_t)blockIdx.x * seg_len;
    uint8_t *g = gamma + (size_t)blockIdx.x * seg_len;
    const int tid = threadIdx.x;

    if (n_zero <= 0 || n_zero >= seg_len) {
        const uint8_t v = (n_zero <= 0) ? 1 : 0;
        for (long long i = tid; i < seg_len; i += kSelectThreads) g[i] = v;
        return;
    }
    if (tid == 0) { s_prefix = 0ull; s_k = n_zero; }
    for (int pass = 7; pass >= 0; --pass) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const unsigned long long prefix = s_prefix;
        const int shift = 8 * pass;
        for (long long i = tid; i < seg_len; i += kSelectThreads) {
            const unsigned long long v = k[i];
            const bool in = (pass == 7) || ((v >> (shift + 8)) == prefix);
            if (in) atomicAdd(&hist[(unsigned)((v >> shift) & 0xFFull)], 1u);
        }
        __syncthreads();
        if (tid == 0) {
            long long need = s_k, cum = 0;
            int d = 0;
            for (; d < 255; ++d) {
                if (cum + (long long)hist[d] >= need) break;
                cum += hist[d];
            }
            s_k = need - cum;
            s_prefix = (prefix << 8) | (unsigned long long)d;
        }
        __syncthreads();
    }
    const unsigned long long T = s_prefix;
    const long long ties = s_k;        // keys equal to T to zero, lowest indices first
    if (tid == 0) s_run = 0;
    __syncthreads();
    const int lane = tid & 31, warp = tid >> 5;
    for (long long base = 0; base < seg_len; base += kSelectThreads) {
        const long long i = base + tid;
        unsigned long long v = ~0ull;
        if (i < seg_len) v = k[i];
        const bool eq = (i < seg_len) && (v == T);
        const unsigned ball = __ballot_sync(0xFFFFFFFFu, eq);
        if (lane == 0) warp_cnt[warp] = __popc(ball);
        __syncthreads();
        long long before = s_run;
        for (int w = 0; w < warp; ++w) before += warp_cnt[w];
        before += __popc(ball & ((1u << lane) - 1u));
        if (i < seg_len) g[i] = (v < T || (eq && before < ties)) ? 0 : 1;
        __syncthreads();
        if (tid == 0) {
            long long tot = 0;
            for (int w = 0; w < kSelectThreads / 32; ++w) tot += warp_cnt[w];
            s_run += tot;
        }
        __syncthreads();
    }
}

// Grid-wide barrier of a cooperative launch (all CTAs co-resident), reusable within the launch: `sync[0]`
// counts arrivals and is reset by the last arriver, `sync[1]` is a generation that the last arriver bumps.
// Thread 0 of each CTA takes part (release on arrival, acquire on the generation; the CTA barriers around it
// extend both to the other threads); the wait is bounded.  Returns false if it expired.
constexpr unsigned kGridSpinLimit = 1u << 22;
__device__ __forceinline__ bool grid_barrier(unsigned *sync)
{
    __shared__ int s_bar_ok;
    __syncthreads();                         // the CTA's writes are ordered before thread 0's release below
    if (threadIdx.x == 0) {
        unsigned g0, old, g;
        int ok = 1;
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];\n" : "=r"(g0) : "l"(sync + 1) : "memory");
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;\n" : "=r"(old) : "l"(sync) : "memory");
        if (old == gridDim.x - 1) {
            asm volatile("st.relaxed.gpu.global.u32 [%0], %1;\n" ::"l"(sync), "r"(0u) : "memory");
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;\n" ::"l"(sync + 1) : "memory");
        } else {
            unsigned spin = 0;
            do {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(g) : "l"(sync + 1) : "memory");
            } while (g == g0 && ++spin < kGridSpinLimit);
            if (g == g0) ok = 0;
        }
        s_bar_ok = ok;
    }
    __syncthreads();
    return s_bar_ok != 0;
}

// The radix select of select_kernel for one large segment (the whole layer), spread over a cooperative grid:
// CTA c owns a contiguous slice of the keys.  Each of the eight passes adds the CTAs' digit histograms into
// ghist[pass][256] (zeroed by the host before the launch), the CTAs meet at the grid barrier, and every CTA
// derives the digit for itself.  Keys equal to the threshold T are zeroed lowest index first: the CTAs publish
// how many such keys their slices hold (geq[c]), meet again, and each counts those in the slices before its own.
constexpr int kCoopThreads = 512;
constexpr int kLocalMax = 8192;          // candidates that the CTAs finish on their own, in (dynamic) shared memory

// The digit d of a 256-bin histogram with cum(d - 1) < need <= cum(d), found by the first warp: each lane sums eight
// bins, a warp scan finds the lane, the lane walks its bins.  Writes the remaining count, the extended prefix and the
// number of keys in the chosen bin; the caller synchronises the CTA afterwards.
__device__ __forceinline__ void select_digit(const unsigned *hist, int tid, unsigned long long prefix, long long *s_k,
                                             unsigned long long *s_prefix, unsigned *s_left, int width)
{
    if (tid >= 32) return;
    const long long need = *s_k;
    long long mine = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) mine += hist[tid * 8 + q];
    long long inc = mine;
#pragma unroll
    for (int dd = 1; dd < 32; dd <<= 1) {
        const long long n = __shfl_up_sync(0xFFFFFFFFu, inc, dd);
        if (tid >= dd) inc += n;
    }
    const unsigned reach = __ballot_sync(0xFFFFFFFFu, inc >= need);
    const int owner = reach ? __ffs(reach) - 1 : 31;        // need <= total, so some lane reaches it
    if (tid == owner) {
        long long cum = inc - mine;
        int d = tid * 8;
        for (; d < tid * 8 + 7; ++d) {
            if (cum + (long long)hist[d] >= need) break;
            cum += hist[d];
        }
        *s_k = need - cum;
        *s_prefix = (prefix << width) | (unsigned long long)d;
        *s_left = hist[d];
    }
}

// The select starts at the highest bit in which any two keys differ (the score kernel leaves the OR of all keys in
// gcount[2..3] and the OR of their complements in gcount[4..5]: the bits above it are the same in every key, e.g. the
// sign and most of the exponent of float scores, or the leading zero bytes of integer ones) and takes digits of eight
// bits downwards.  Passes run grid-wide (global histograms, a grid barrier
// each) only while more than kLocalMax keys still match the prefix; then the CTAs append their matching keys to one
// list (`cand`, counted in gcount[0], zeroed by the host with the histograms), meet
// once, and every CTA finishes the remaining digits on the list in its own shared memory.
constexpr int kSliceMax = 4096;          // keys of a CTA's slice that are kept in shared memory for all phases
constexpr size_t kCoopSmem = (size_t)(kLocalMax + kSliceMax) * sizeof(unsigned long long);

__global__ void __launch_bounds__(kCoopThreads)
select_coop_kernel(const unsigned long long *__restrict__ key, long long n, long long n_zero, uint8_t *__restrict__ gamma,
                   unsigned *ghist, unsigned *gcount, unsigned long long *cand, unsigned *geq, unsigned *sync, int *status)
{
    __shared__ unsigned hist[256];
    extern __shared__ unsigned long long s_dyn[];
    unsigned long long *s_cand = s_dyn;                  // [kLocalMax]
    unsigned long long *s_keys = s_dyn + kLocalMax;      // [kSliceMax]
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_k;
    __shared__ unsigned s_left, s_n;
    __shared__ unsigned warp_cnt[kCoopThreads / 32];
    __shared__ long long s_run;
    const int tid = threadIdx.x;
    const long long slice = (n + gridDim.x - 1) / gridDim.x;
    const long long lo = min(n, (long long)blockIdx.x * slice), hi = min(n, lo + slice);
    const int len = (int)(hi - lo);                      // (a slice of more than 2^31 keys would need more CTAs than the launch allows)
    const unsigned long long k0 = key[0];
    // bit positions in which some two keys differ (the score kernel accumulated both ORs)
    const unsigned long long diff = __ldcg((const unsigned long long *)(gcount + 2)) & __ldcg((const unsigned long long *)(gcount + 4));
    // the slice is read once: every phase below walks it in shared memory (or in place when it does not fit)
    const unsigned long long *ks = key + lo;
    if (len <= kSliceMax) {
#pragma unroll 4
        for (int i = tid; i < len; i += kCoopThreads) s_keys[i] = key[lo + i];
        ks = s_keys;
    }
    // bits above `top` are common to all keys: they are the prefix so far (all keys equal: nothing left to select)
    int top = diff ? 63 - __clzll((long long)diff) : -1;
    if (tid == 0) { s_prefix = top >= 63 ? 0ull : (k0 >> (top + 1)); s_k = n_zero; s_left = n > 0xFFFFFFFFll ? 0xFFFFFFFFu : (unsigned)n; }
    int pi = 0;
    while (top >= 0) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        if (s_left <= (unsigned)kLocalMax) break;          // few enough candidates: the rest is local
        const unsigned long long prefix = s_prefix;
        const int width = min(8, top + 1), shift = top + 1 - width;
        const unsigned dmask = (1u << width) - 1u;
        for (int i = tid; i < len; i += kCoopThreads) {
            const unsigned long long v = ks[i];
            if (top >= 63 || ((v >> (top + 1)) == prefix)) atomicAdd(&hist[(unsigned)(v >> shift) & dmask], 1u);
        }
        __syncthreads();
        if (tid < 256 && hist[tid]) atomicAdd(&ghist[pi * 256 + tid], hist[tid]);
        if (!grid_barrier(sync)) { if (tid == 0) atomicMax(status, (int)BSP_ERR_TIMEOUT); return; }
        if (tid < 256) hist[tid] = __ldcg(&ghist[pi * 256 + tid]);
        __syncthreads();
        select_digit(hist, tid, prefix, &s_k, &s_prefix, &s_left, width);
        __syncthreads();
        top -= width;
        ++pi;
    }
    if (top >= 0) {
        // bits top .. 0 are still open: gather the keys that match the prefix, then finish locally
        const unsigned long long prefix = s_prefix;
        for (int base = 0; base < len; base += kCoopThreads) {
            const int i = base + tid;
            const unsigned long long v = i < len ? ks[i] : 0ull;
            const bool in = i < len && (top >= 63 || (v >> (top + 1)) == prefix);
            // one addition to the counter per warp
            const unsigned ball = __ballot_sync(0xFFFFFFFFu, in);
            unsigned at = 0u;
            if ((tid & 31) == 0 && ball) at = atomicAdd(gcount, (unsigned)__popc(ball));
            at = __shfl_sync(0xFFFFFFFFu, at, 0) + (unsigned)__popc(ball & ((1u << (tid & 31)) - 1u));
            if (in && at < (unsigned)kLocalMax) cand[at] = v;
        }
        if (!grid_barrier(sync)) { if (tid == 0) atomicMax(status, (int)BSP_ERR_TIMEOUT); return; }
        unsigned cnt = min(__ldcg(gcount), (unsigned)kLocalMax);
        for (unsigned i = tid; i < cnt; i += kCoopThreads) s_cand[i] = __ldcg(&cand[i]);
        __syncthreads();
        constexpr int kMine = kLocalMax / kCoopThreads;    // candidates per thread
        while (top >= 0 && cnt > (unsigned)kCoopThreads) {
            if (tid < 256) hist[tid] = 0u;
            if (tid == 0) s_n = 0u;
            __syncthreads();
            const int width = min(8, top + 1), shift = top + 1 - width;
            const unsigned dmask = (1u << width) - 1u;
            // every candidate matches the prefix so far (the list is thinned after each digit)
            unsigned long long mine[kMine];
#pragma unroll
            for (int u = 0; u < kMine; ++u) {
                const unsigned i = (unsigned)u * kCoopThreads + tid;
                mine[u] = i < cnt ? s_cand[i] : 0ull;
                if (i < cnt) atomicAdd(&hist[(unsigned)(mine[u] >> shift) & dmask], 1u);
            }
            __syncthreads();
            select_digit(hist, tid, s_prefix, &s_k, &s_prefix, &s_left, width);
            __syncthreads();
            top -= width;
            // keep the candidates of the chosen digit (all were read into registers above)
            const unsigned long long pre = s_prefix;
#pragma unroll
            for (int u = 0; u < kMine; ++u) {
                const unsigned i = (unsigned)u * kCoopThreads + tid;
                if (i < cnt && (top < 0 ? mine[u] : (mine[u] >> (top + 1))) == pre) s_cand[atomicAdd(&s_n, 1u)] = mine[u];
            }
            __syncthreads();
            cnt = s_n;
            __syncthreads();
        }
        if (top >= 0) {
            // at most one candidate per thread is left: each counts the candidates below its own and equal to it; the
            // s_k-th smallest is the threshold (threads holding equal keys write the same values)
            const long long need = s_k;
            __syncthreads();
            if ((unsigned)tid < cnt) {
                const unsigned long long v = s_cand[tid];
                unsigned less = 0u, same = 0u;
                for (unsigned j = 0; j < cnt; ++j) {
                    const unsigned long long o = s_cand[j];
                    less += o < v ? 1u : 0u;
                    same += o == v ? 1u : 0u;
                }
                if ((long long)less < need && need <= (long long)(less + same)) { s_prefix = v; s_k = need - less; s_left = same; }
            }
            top = -1;
        }
    }
    __syncthreads();
    const unsigned long long T = s_prefix;
    const long long ties = s_k;        // keys equal to T to zero, lowest indices first
    if (s_left == 1u) {
        // a single key equals T (every CTA derived the same count): it is the last one zeroed, no order among equals
        for (int i = tid; i < len; i += kCoopThreads) gamma[lo + i] = ks[i] <= T ? 0 : 1;
        return;
    }
    // keys equal to T in this slice
    {
        unsigned c = 0;
        for (int i = tid; i < len; i += kCoopThreads) c += ks[i] == T ? 1u : 0u;
        for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, d);
        if ((tid & 31) == 0) warp_cnt[tid >> 5] = c;
        __syncthreads();
        if (tid == 0) {
            unsigned tot = 0;
            for (int w = 0; w < kCoopThreads / 32; ++w) tot += warp_cnt[w];
            geq[blockIdx.x] = tot;
        }
    }
    if (!grid_barrier(sync)) { if (tid == 0) atomicMax(status, (int)BSP_ERR_TIMEOUT); return; }
    if (tid == 0) {
        long long before = 0;
        for (unsigned c = 0; c < blockIdx.x; ++c) before += __ldcg(&geq[c]);
        s_run = before;
    }
    __syncthreads();
    const int lane = tid & 31, warp = tid >> 5;
    for (int base = 0; base < len; base += kCoopThreads) {
        const int i = base + tid;
        unsigned long long v = ~0ull;
        if (i < len) v = ks[i];
        const bool eq = (i < len) && (v == T);
        const unsigned ball = __ballot_sync(0xFFFFFFFFu, eq);
        if (lane == 0) warp_cnt[warp] = __popc(ball);
        __syncthreads();
        long long before = s_run;
        for (int w = 0; w < warp; ++w) before += warp_cnt[w];
        before += __popc(ball & ((1u << lane) - 1u));
        if (i < len) gamma[lo + i] = (v < T || (eq && before < ties)) ? 0 : 1;
        __syncthreads();
        if (tid == 0) {
            long long tot = 0;
            for (int w = 0; w < kCoopThreads / 32; ++w) tot += warp_cnt[w];
            s_run += tot;
        }
        __syncthreads();
    }
}

// Small segments (up to kRankMax keys): the keys sit in shared memory and every thread counts the (key, index)
// pairs below its own, which is its rank in the ascending order; Gamma = 0 for ranks below n_zero.  Same
// result as the radix select, in one pass instead of nine.
constexpr int kRankMax = 4096;
constexpr int kRankThreads = 256;
constexpr int kRankLanes = 8;            // lanes sharing one key; each counts an eighth of the segment
__global__ void __launch_bounds__(kRankThreads)
rank_kernel(const unsigned long long *__restrict__ key, int seg_len, long long n_zero, uint8_t *__restrict__ gamma)
{
    __shared__ unsigned long long s_key[kRankMax];
    const unsigned long long *k = key + (size_t)blockIdx.x * seg_len;
    uint8_t *g = gamma + (size_t)blockIdx.x * seg_len;
    {   // all loads of the segment are issued before the first store, so they share one trip to memory
        unsigned long long v[kRankMax / kRankThreads];
#pragma unroll
        for (int u = 0; u < kRankMax / kRankThreads; ++u) {
            const int i = u * kRankThreads + threadIdx.x;
            v[u] = i < seg_len ? __ldg(k + i) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < kRankMax / kRankThreads; ++u) {
            const int i = u * kRankThreads + threadIdx.x;
            if (i < seg_len) s_key[i] = v[u];
        }
    }
    __syncthreads();
    // gridDim.y CTAs share one segment; the keys are padded to a multiple of the CTA's share so that all
    // lanes of a warp take part in the shuffles
    const int i = (blockIdx.y * kRankThreads + threadIdx.x) / kRankLanes;
    const int part = threadIdx.x % kRankLanes;
    const bool live = i < seg_len;
    const unsigned long long mine = live ? s_key[i] : 0ull;
    const int per = (seg_len + kRankLanes - 1) / kRankLanes;
    const int j0 = part * per, j1 = min(seg_len, j0 + per);
    int rank = 0;
    if (live)
        for (int j = j0; j < j1; ++j) {
            const unsigned long long other = s_key[j];
            rank += (other < mine || (other == mine && j < i)) ? 1 : 0;
        }
#pragma unroll
    for (int d = 1; d < kRankLanes; d <<= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, d);
    if (live && part == 0) g[i] = ((long long)rank < n_zero) ? 0 : 1;
}

// Layers of up to kRankMax blocks: scores and ranks in ONE cooperative launch.  Every CTA scores its blocks,
// the CTAs meet at a grid-wide barrier, then every CTA ranks its own blocks against the keys of their segment
// (b_o lanes per key).  The barrier is two words: arrivals (reset by the last arriver, so the next launch starts
// from zero whatever its grid) and a generation that the last arriver bumps; the wait on the generation is
// bounded and latches BSP_ERR_TIMEOUT.

template <int DT, int NORM, int kBatch>
__global__ void __launch_bounds__(kScoreThreads)
mask_small_kernel(const uint32_t *__restrict__ W, int I, int HK, int bo, int bi, int NBo, int NBi, int BC,
                  typename Acc<DT>::type *score, int seg_len, long long n_zero, uint8_t *__restrict__ gamma,
                  unsigned *sync, int *status)
{
    using acc_t = typename Acc<DT>::type;
    __shared__ acc_t part[kScoreThreads];
    __shared__ unsigned long long s_key[kRankMax];
    const int NB = NBo * NBi;
    // BC blocks per CTA: b_o threads score one block, then 256 / BC lanes rank one key
    {
        const int bl = threadIdx.x % BC, r = threadIdx.x / BC;
        const long long B = (long long)blockIdx.x * BC + bl;
        const bool mine = r < bo && B < NB;
        part[threadIdx.x] = mine ? row_sum<DT, NORM, kBatch>(W, I, HK, bo, bi, NBi, B, r) : (acc_t)0;
        __syncthreads();
        if (mine && r == 0) {
            acc_t total = 0;
            for (int q = 0; q < bo; ++q) total += part[q * BC + bl];
            score[B] = total;
        }
    }
    if (!grid_barrier(sync)) {
        if (threadIdx.x == 0) atomicMax(status, (int)BSP_ERR_TIMEOUT);
        return;
    }
    // every key of the layer -> shared memory (written by other CTAs of this launch: read through L2)
    {
        const unsigned long long *k = (const unsigned long long *)score;
        unsigned long long v[kRankMax / kScoreThreads];
#pragma unroll
        for (int u = 0; u < kRankMax / kScoreThreads; ++u) {
            const int i = u * kScoreThreads + threadIdx.x;
            v[u] = i < NB ? __ldcg(k + i) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < kRankMax / kScoreThreads; ++u) {
            const int i = u * kScoreThreads + threadIdx.x;
            if (i < NB) s_key[i] = v[u];
        }
    }
    __syncthreads();
    const int LK = kScoreThreads / BC;                          // lanes per key, at most 32
    const int i = blockIdx.x * BC + threadIdx.x / LK;
    const int lane_part = threadIdx.x % LK;
    const bool live = i < NB;
    const int seg0 = live ? (i / seg_len) * seg_len : 0;
    const unsigned long long mine = live ? s_key[i] : 0ull;
    int rank = 0;
    if (live)
        for (int j = seg0 + lane_part; j < seg0 + seg_len; j += LK) {   // consecutive lanes, consecutive keys
            const unsigned long long other = s_key[j];
            rank += (other < mine || (other == mine && j < i)) ? 1 : 0;
        }
    for (int d = 1; d < LK; d <<= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, d);
    if (live && lane_part == 0) gamma[i] = ((long long)rank < n_zero) ? 0 : 1;
}

template <int DT, int NORM>
bsp_status run_mask_small(const bsp_wdesc &wd, const void *W, int seg_len, long long n_zero, uint8_t *gamma, void *scores,
                          unsigned *sync, int *status, cudaStream_t st)
{
    using acc_t = typename Acc<DT>::type;
    const uint32_t *Wp = (const uint32_t *)W;
    int I = wd.I, HK = wd.H * wd.K, bo = wd.bo, bi = wd.bi, NBo = wd.O / wd.bo, NBi = wd.I / wd.bi;
    acc_t *sc = (acc_t *)scores;
    // few blocks per CTA spread the layer over the SMs; the grid stays small enough to be co-resident
    int BC = 8;
    while ((NBo * NBi + BC - 1) / BC > 128 && BC * 2 * wd.bo <= kScoreThreads) BC *= 2;
    const unsigned grid = (unsigned)((NBo * NBi + BC - 1) / BC);
    void *args[] = {&Wp, &I, &HK, &bo, &bi, &NBo, &NBi, &BC, &sc, &seg_len, &n_zero, &gamma, &sync, &status};
    const void *kern = HK == 1 ? (const void *)mask_small_kernel<DT, NORM, 1> : (const void *)mask_small_kernel<DT, NORM, 9>;
    const cudaError_t e = cudaLaunchCooperativeKernel(kern, dim3(grid), dim3(kScoreThreads), args, 0, st);
    if (e == cudaErrorCooperativeLaunchTooLarge) {      // fewer SMs than CTAs (a partitioned GPU): the caller takes the multi-launch path
        (void)cudaGetLastError();
        return BSP_ERR_CAPACITY;
    }
    BSP_CUDA_OK(e);
    return BSP_OK;
}

template <int DT>
bsp_status run_scores(const bsp_wdesc &wd, const void *W, bsp_norm norm, void *scores, unsigned long long *span, cudaStream_t st)
{
    using acc_t = typename Acc<DT>::type;
    const int NBo = wd.O / wd.bo, NBi = wd.I / wd.bi;
    const long long NB = (long long)NBo * NBi;
    const int per_cta = kScoreThreads / wd.bo;
    const long long groups = (NB + per_cta - 1) / per_cta;
    const unsigned grid = (unsigned)(groups < 148 * 8 ? groups : 148 * 8);       // eight CTAs per SM's worth, each looping
    const int HK = wd.H * wd.K;
    const uint32_t *Wp = (const uint32_t *)W;
    acc_t *sc = (acc_t *)scores;
    if constexpr (DT != BSP_I8) {
        if (norm == BSP_NORM_VAR) {
            if (HK == 1) score_kernel<DT, BSP_NORM_VAR, 1><<<grid, kScoreThreads, 0, st>>>(Wp, wd.I, HK, wd.bo, wd.bi, NBo, NBi, sc, span);
            else score_kernel<DT, BSP_NORM_VAR, 9><<<grid, kScoreThreads, 0, st>>>(Wp, wd.I, HK, wd.bo, wd.bi, NBo, NBi, sc, span);
            BSP_CUDA_OK(cudaGetLastError());
            return BSP_OK;
        }
    }
    // (one-tap layers: one thread per block)
    const long long ctas1 = (NB + kScoreThreads - 1) / kScoreThreads;
    const unsigned grid1 = (unsigned)(ctas1 < 148 * 8 ? ctas1 : 148 * 8);
    if (norm == BSP_NORM_L2) {
        if (HK == 1) score_kernel<DT, BSP_NORM_L2, 1><<<grid1, kScoreThreads, 0, st>>>(Wp, wd.I, HK, wd.bo, wd.bi, NBo, NBi, sc, span);
        else score_kernel<DT, BSP_NORM_L2, 9><<<grid, kScoreThreads, 0, st>>>(Wp, wd.I, HK, wd.bo, wd.bi, NBo, NBi, sc, span);
    } else {
        if (HK == 1) score_kernel<DT, BSP_NORM_L1, 1><<<grid1, kScoreThreads, 0, st>>>(Wp, wd.I, HK, wd.bo, wd.bi, NBo, NBi, sc, span);
        else score_kernel<DT, BSP_NORM_L1, 9><<<grid, kScoreThreads, 0, st>>>(Wp, wd.I, HK, wd.bo, wd.bi, NBo, NBi, sc, span);
    }
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // namespace

bsp_status launch_mask(const bsp_wdesc &wd, const void *W, bsp_norm norm, bsp_scope scope, int64_t n_zero,
                       uint8_t *gamma, void *scores, void *ws, cudaStream_t st)
{
    bsp_status rc;
    {
        const long long NB = (long long)(wd.O / wd.bo) * (wd.I / wd.bi);
        if (ws != nullptr && NB <= kRankMax && norm != BSP_NORM_VAR) {     // (the variance takes the two-pass score kernel)
            const int seg_len = (int)((scope == BSP_SCOPE_LAYER) ? NB : wd.I / wd.bi);
            int *status = (int *)ws;
            unsigned *sync = (unsigned *)ws + kWsSyncWord;
            const bool l2 = norm == BSP_NORM_L2;
            bsp_status small;
            if (wd.wtype == BSP_F32)
                small = l2 ? run_mask_small<BSP_F32, BSP_NORM_L2>(wd, W, seg_len, n_zero, gamma, scores, sync, status, st)
                           : run_mask_small<BSP_F32, BSP_NORM_L1>(wd, W, seg_len, n_zero, gamma, scores, sync, status, st);
            else if (wd.wtype == BSP_BF16)
                small = l2 ? run_mask_small<BSP_BF16, BSP_NORM_L2>(wd, W, seg_len, n_zero, gamma, scores, sync, status, st)
                           : run_mask_small<BSP_BF16, BSP_NORM_L1>(wd, W, seg_len, n_zero, gamma, scores, sync, status, st);
            else
                small = l2 ? run_mask_small<BSP_I8, BSP_NORM_L2>(wd, W, seg_len, n_zero, gamma, scores, sync, status, st)
                           : run_mask_small<BSP_I8, BSP_NORM_L1>(wd, W, seg_len, n_zero, gamma, scores, sync, status, st);
            if (small != BSP_ERR_CAPACITY) return small;
        }
    }
    const int NBo = wd.O / wd.bo, NBi = wd.I / wd.bi;
    const long long NB = (long long)NBo * NBi;
    const long long seg = (scope == BSP_SCOPE_LAYER) ? NB : NBi;
    const unsigned nseg = (scope == BSP_SCOPE_LAYER) ? 1u : (unsigned)NBo;
    // one large segment: the select runs on a cooperative grid; its histograms, counter and the span of the keys (filled
    // by the score kernel) are zeroed first
    const bool coop = ws != nullptr && nseg == 1 && seg > kRankMax && n_zero > 0 && n_zero < seg;
    unsigned *ghist = coop ? (unsigned *)((char *)ws + kWsHeader + align_up((size_t)NB * 8, 256)) : nullptr;
    unsigned *gcount = coop ? ghist + 8 * 256 : nullptr;     // [0] candidate counter, [2..3] OR of the keys, [4..5] OR of their complements
    if (coop) BSP_CUDA_OK(cudaMemsetAsync(ghist, 0, (8 * 256 + 8) * sizeof(unsigned), st));
    unsigned long long *span = coop ? (unsigned long long *)(gcount + 2) : nullptr;
    if (wd.wtype == BSP_F32) rc = run_scores<BSP_F32>(wd, W, norm, scores, span, st);
    else if (wd.wtype == BSP_BF16) rc = run_scores<BSP_BF16>(wd, W, norm, scores, span, st);
    else rc = run_scores<BSP_I8>(wd, W, norm, scores, span, st);
    if (rc != BSP_OK) return rc;
    if (seg <= kRankMax)
        rank_kernel<<<dim3(nseg, (unsigned)((seg * kRankLanes + kRankThreads - 1) / kRankThreads)), kRankThreads, 0, st>>>(
            (const unsigned long long *)scores, (int)seg, n_zero, gamma);
    else if (coop) {
        // at most one CTA per SM
        static int sm_count[64] = {};
        int dev = 0;
        BSP_CUDA_OK(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return BSP_ERR_CUDA;
        if (sm_count[dev] == 0) {
            BSP_CUDA_OK(cudaFuncSetAttribute(select_coop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCoopSmem));
            BSP_CUDA_OK(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
        }
        long long grid = (seg + 2 * kCoopThreads - 1) / (2 * kCoopThreads);
        if (grid > sm_count[dev]) grid = sm_count[dev];
        if (grid > kSelectMaxCtas) grid = kSelectMaxCtas;
        unsigned *geq = gcount + 8;
        unsigned long long *cand = (unsigned long long *)(geq + kSelectMaxCtas);
        const unsigned long long *keys = (const unsigned long long *)scores;
        long long n = seg, nz = n_zero;
        unsigned *sync = (unsigned *)ws + kWsSyncWord;
        int *status = (int *)ws;
        void *args[] = {&keys, &n, &nz, &gamma, &ghist, &gcount, &cand, &geq, &sync, &status};
        const cudaError_t e = cudaLaunchCooperativeKernel((const void *)select_coop_kernel, dim3((unsigned)grid), dim3(kCoopThreads), args, kCoopSmem, st);
        if (e == cudaErrorCooperativeLaunchTooLarge) {
            (void)cudaGetLastError();
            select_kernel<<<nseg, kSelectThreads, 0, st>>>((const unsigned long long *)scores, seg, n_zero, gamma);
            BSP_CUDA_OK(cudaGetLastError());
            return BSP_OK;
        }
        BSP_CUDA_OK(e);
        return BSP_OK;
    } else
        select_kernel<<<nseg, kSelectThreads, 0, st>>>((const unsigned long long *)scores, seg, n_zero, gamma);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // namespace bsp
