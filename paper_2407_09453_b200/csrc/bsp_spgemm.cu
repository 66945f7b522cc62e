// Block-sparse x block-sparse product C = (Gamma . A)(Omega . B)^t on the compressed block rows of both operands, and the
// relative column index.  Section "Block-Sparse Matrix-Matrix Multiplication" and Section "Block Sparsity in a Matrix"
// ("a relative row/col index") of the paper.
//
// C_{i,j} = sum over the block columns k that row i of A and row j of B both keep of A_{i,k} B_{j,k}^t, 8 x 8 blocks.
// A CTA owns one row i of A: the positions of its kept blocks are spread into a table over the block columns in shared
// memory (the table replaces one side of the paper's merge of two sorted lists), and every warp takes rows j of B in
// turn: 32 entries of B's column list are looked up at once, a ballot gives the common columns in ascending order, and
// for each of them the warp adds the 8 x 8 x 8 product, lane (r, c) holding C[r][2c], C[r][2c + 1] in fp32 (fp32 blocks:
// fused multiply-adds; bfloat16 blocks: one m16n8k16 tensor-core instruction per two common columns).  Work and
// traffic follow the kept blocks only: nothing is read or multiplied where either mask has a zero.
#include "bsp_internal.cuh"

namespace bsp {
namespace {

constexpr int kSpThreads = 256;
constexpr int kSpEdge = 8;

// One row of an 8 x 8 block (8 consecutive values) as floats: two 16-byte loads for fp32, one for bf16.
__device__ __forceinline__ void sp_row(const float *p, float (&v)[8])
{
    const float4 a = __ldg((const float4 *)p), b = __ldg((const float4 *)p + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void sp_row(const __nv_bfloat16 *p, float (&v)[8])
{
    const uint4 q = __ldg((const uint4 *)p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        v[2 * t] = __uint_as_float(w[t] << 16);
        v[2 * t + 1] = __uint_as_float(w[t] & 0xFFFF0000u);
    }
}

template <typename T>
__global__ void __launch_bounds__(kSpThreads)
spgemm_kernel(const int32_t *__restrict__ a_row_ptr, const int32_t *__restrict__ a_col_idx, const T *__restrict__ a_payload,
              const int32_t *__restrict__ b_row_ptr, const int32_t *__restrict__ b_col_idx, const T *__restrict__ b_payload,
              int NBb, int NBk, float *__restrict__ C, int *status)
{
    extern __shared__ int s_pos[];                 // [NBk]: payload position of row i's block in column k, or -1
    const int i = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int k = threadIdx.x; k < NBk; k += kSpThreads) s_pos[k] = -1;
    __syncthreads();
    for (int n = a_row_ptr[i] + threadIdx.x; n < a_row_ptr[i + 1]; n += kSpThreads) {
        const int k = a_col_idx[n];
        if (k >= 0 && k < NBk) s_pos[k] = n;
        else atomicMax(status, (int)BSP_ERR_INDEX);          // a column outside the matrix: skipped
    }
    __syncthreads();
    const int r = lane >> 2, c = (lane & 3) * 2;             // this lane's two entries of the 8 x 8 block of C
    const size_t ldc = (size_t)NBb * kSpEdge;
    for (int j = blockIdx.y * (kSpThreads / 32) + warp; j < NBb; j += gridDim.y * (kSpThreads / 32)) {
        float acc0 = 0.f, acc1 = 0.f;
        const int lo = b_row_ptr[j], hi = b_row_ptr[j + 1];
        for (int base = lo; base < hi; base += 32) {
            const int nb = base + lane;
            int pa = -1;
            if (nb < hi) {
                const int k = b_col_idx[nb];
                if (k >= 0 && k < NBk) pa = s_pos[k];
                else atomicMax(status, (int)BSP_ERR_INDEX);
            }
            unsigned both = __ballot_sync(0xFFFFFFFFu, pa >= 0);
            if constexpr (sizeof(T) == 2) {
                // bfloat16 blocks: two common columns per tensor-core instruction (m16n8k16: the 8 x 8 block of C sits in
                // rows 0-7 of the 16 x 8 result, K = the eight channels of the first column followed by those of the
                // second).  Lane (r, c) holds exactly the words it needs: entries (r, 2c), (r, 2c + 1) of each block of A
                // and of B, so a warp reads each 128-byte block once, four bytes per lane.
                while (both) {
                    const int s1 = __ffs(both) - 1;
                    both &= both - 1;
                    const int s2 = both ? __ffs(both) - 1 : -1;
                    both &= both - 1;                         // (0 & -1 stays 0)
                    const int na1 = __shfl_sync(0xFFFFFFFFu, pa, s1);
                    const int na2 = __shfl_sync(0xFFFFFFFFu, pa, s2 < 0 ? s1 : s2);
                    const uint32_t *Aw = (const uint32_t *)a_payload, *Bw = (const uint32_t *)b_payload;
                    const uint32_t a0 = __ldg(Aw + (size_t)na1 * 32 + lane), b0 = __ldg(Bw + (size_t)(base + s1) * 32 + lane);
                    uint32_t a2 = 0u, b1 = 0u;
                    if (s2 >= 0) { a2 = __ldg(Aw + (size_t)na2 * 32 + lane); b1 = __ldg(Bw + (size_t)(base + s2) * 32 + lane); }
                    float d2 = 0.f, d3 = 0.f;
                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
                                 : "+f"(acc0), "+f"(acc1), "+f"(d2), "+f"(d3) : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
                }
            } else
            while (both) {                                    // common columns, ascending
                const int src = __ffs(both) - 1;
                both &= both - 1;
                const int na = __shfl_sync(0xFFFFFFFFu, pa, src);
                const T *Ab = a_payload + ((size_t)na * kSpEdge + r) * kSpEdge;
                const T *Bb = b_payload + ((size_t)(base + src) * kSpEdge + c) * kSpEdge;
                float av[8], b0[8], b1[8];
                sp_row(Ab, av); sp_row(Bb, b0); sp_row(Bb + kSpEdge, b1);
#pragma unroll
                for (int t = 0; t < kSpEdge; ++t) {
                    acc0 = fmaf(av[t], b0[t], acc0);
                    acc1 = fmaf(av[t], b1[t], acc1);
                }
            }
        }
        *(float2 *)(C + ((size_t)i * kSpEdge + r) * ldc + (size_t)j * kSpEdge + c) = make_float2(acc0, acc1);
    }
}

// One thread per row of Gamma: the first kept block keeps its column, the others store the distance to their predecessor.
__global__ void index_to_relative_kernel(int NBo, const int32_t *__restrict__ row_ptr, const int32_t *__restrict__ col_idx,
                                         int32_t *__restrict__ rel)
{
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= NBo) return;
    int prev = 0;
    for (int n = row_ptr[l]; n < row_ptr[l + 1]; ++n) {
        const int cur = col_idx[n];
        rel[n] = cur - prev;
        prev = cur;
    }
}

__global__ void index_from_relative_kernel(int NBo, const int32_t *__restrict__ row_ptr, const int32_t *__restrict__ rel,
                                           int32_t *__restrict__ col_idx)
{
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= NBo) return;
    int at = 0;
    for (int n = row_ptr[l]; n < row_ptr[l + 1]; ++n) {
        at += rel[n];
        col_idx[n] = at;
    }
}

}  // namespace
}  // namespace bsp

using namespace bsp;

extern "C" {

bsp_status bsp_spgemm(const bsp_wdesc *wa, const bsp_bcsr *a, const bsp_wdesc *wb, const bsp_bcsr *b, float *C, void *ws,
                      void *stream)
{
    bsp_status rc = check_wdesc(wa);
    if (rc != BSP_OK) return rc;
    rc = check_wdesc(wb);
    if (rc != BSP_OK) return rc;
    if (!a || !b || !C || !ws || !a->row_ptr || !a->col_idx || !a->payload || !b->row_ptr || !b->col_idx || !b->payload)
        return BSP_ERR_NULL;
    if (wa->H != 1 || wa->K != 1 || wb->H != 1 || wb->K != 1 || wa->I != wb->I) return BSP_ERR_SHAPE;
    if (wa->bo != kSpEdge || wa->bi != kSpEdge || wb->bo != kSpEdge || wb->bi != kSpEdge) return BSP_ERR_BLOCK;
    if (wa->wtype != wb->wtype || (wa->wtype != BSP_F32 && wa->wtype != BSP_BF16)) return BSP_ERR_DTYPE;
    if (((uintptr_t)C & 7u) != 0 || ((uintptr_t)a->payload & 15u) != 0 || ((uintptr_t)b->payload & 15u) != 0) return BSP_ERR_SHAPE;
    const int NBa = wa->O / kSpEdge, NBb = wb->O / kSpEdge, NBk = wa->I / kSpEdge;
    const size_t smem = (size_t)NBk * sizeof(int);
    if (smem > 48 * 1024) return BSP_ERR_SHAPE;
    // rows of B are dealt over the warps of gridDim.y CTAs per row of A: enough CTAs to fill the GPU a few times over
    int gy = (NBb + kSpThreads / 32 - 1) / (kSpThreads / 32);
    const int want = (148 * 8 + NBa - 1) / NBa;
    if (gy > want) gy = want;
    if (gy < 1) gy = 1;
    const dim3 grid((unsigned)NBa, (unsigned)gy);
    cudaStream_t st = (cudaStream_t)stream;
    if (wa->wtype == BSP_F32)
        spgemm_kernel<float><<<grid, kSpThreads, smem, st>>>(a->row_ptr, a->col_idx, (const float *)a->payload, b->row_ptr, b->col_idx,
                                                             (const float *)b->payload, NBb, NBk, C, (int *)ws);
    else
        spgemm_kernel<__nv_bfloat16><<<grid, kSpThreads, smem, st>>>(a->row_ptr, a->col_idx, (const __nv_bfloat16 *)a->payload, b->row_ptr,
                                                                     b->col_idx, (const __nv_bfloat16 *)b->payload, NBb, NBk, C, (int *)ws);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

bsp_status bsp_index_to_relative(int NBo, const int32_t *row_ptr, const int32_t *col_idx, int32_t *rel, void *stream)
{
    if (!row_ptr || !col_idx || !rel) return BSP_ERR_NULL;
    if (NBo <= 0) return BSP_ERR_SHAPE;
    index_to_relative_kernel<<<(NBo + 127) / 128, 128, 0, (cudaStream_t)stream>>>(NBo, row_ptr, col_idx, rel);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

bsp_status bsp_index_from_relative(int NBo, const int32_t *row_ptr, const int32_t *rel, int32_t *col_idx, void *stream)
{
    if (!row_ptr || !col_idx || !rel) return BSP_ERR_NULL;
    if (NBo <= 0) return BSP_ERR_SHAPE;
    index_from_relative_kernel<<<(NBo + 127) / 128, 128, 0, (cudaStream_t)stream>>>(NBo, row_ptr, rel, col_idx);
    BSP_CUDA_OK(cudaGetLastError());
    return BSP_OK;
}

}  // extern "C"
