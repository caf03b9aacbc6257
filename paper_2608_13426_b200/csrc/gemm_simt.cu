// Reduced product Y = scale * A[:, I] B[I, :] (paper Sec. 3.2) on the plain FMA pipes.
//
// This kernel covers what the tensor-core path does not: fp32 operands (whose 1e-5 accuracy target
// bf16 tensor-core inputs cannot meet) and bf16 operands with strides or alignments outside the TMA
// rules.  Any element strides are accepted.  64 x 64 output tile per block, 16 contraction indices
// per step, 4 x 4 outputs per thread, fp32 accumulation with one partial sum per step of 16 so that
// rounding error grows with k/16 rather than k.
#include "common.cuh"

namespace rmm {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, THREADS = 256;

struct SimtArgs {
    const void *A, *B;
    void *Y;
    const int32_t *idx;
    int64_t M, N, K, k;
    int64_t a_sb, a_sr, a_sc, b_sb, b_sr, b_sc, y_sb, y_sr, y_sc;
    float scale;
    int *status;
};

template <bool BF16>
__device__ __forceinline__ float load_elem(const void *p, int64_t off)
{
    if constexpr (BF16)
        return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p)[off]);
    else
        return reinterpret_cast<const float *>(p)[off];
}

template <bool IN_BF16, bool OUT_BF16>
__global__ void __launch_bounds__(THREADS) reduced_gemm_simt_kernel(SimtArgs a)
{
    __shared__ float sA[BK][BM + 1];
    __shared__ float sB[BK][BN + 1];
    __shared__ int sIdx[BK];
    pdl_wait();

    const int tid = threadIdx.x;
    const int64_t b = blockIdx.z;
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
    const int ty = tid / 16, tx = tid % 16;  // thread owns rows ty*4.., cols tx*4..
    const int32_t *idx = a.idx != nullptr ? a.idx + b * a.k : nullptr;
    const int64_t a0 = b * a.a_sb, b0 = b * a.b_sb;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int64_t kk = 0; kk < a.k; kk += BK) {
        if (tid < BK) {
            int j = -1;
            if (kk + tid < a.k) {
                j = idx != nullptr ? idx[kk + tid] : (int)(kk + tid);
                if (j < 0 || j >= a.K) {  // skip a bad index and report it
                    atomicExch(a.status, (int)RMM_ERR_BOUNDS);
                    j = -1;
                }
            }
            sIdx[tid] = j;
        }
        __syncthreads();
        // A tile: BK x BM gathered columns; consecutive threads take consecutive k (columns of A are close)
        for (int e = tid; e < BK * BM; e += THREADS) {
            int r = e % BK, m = e / BK;
            int j = sIdx[r];
            float v = 0.f;
            if (j >= 0 && m0 + m < a.M) v = load_elem<IN_BF16>(a.A, a0 + (m0 + m) * a.a_sr + (int64_t)j * a.a_sc);
            sA[r][m] = v;
        }
        // B tile: BK x BN gathered rows; consecutive threads take consecutive n
        for (int e = tid; e < BK * BN; e += THREADS) {
            int n = e % BN, r = e / BN;
            int j = sIdx[r];
            float v = 0.f;
            if (j >= 0 && n0 + n < a.N) v = load_elem<IN_BF16>(a.B, b0 + (int64_t)j * a.b_sr + (n0 + n) * a.b_sc);
            sB[r][n] = v;
        }
        __syncthreads();
        float part[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) part[i][j] = 0.f;
#pragma unroll
        for (int r = 0; r < BK; ++r) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = sA[r][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = sB[r][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) part[i][j] = fmaf(av[i], bv[j], part[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] += part[i][j];
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int64_t m = m0 + ty * 4 + i;
        if (m >= a.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int64_t n = n0 + tx * 4 + j;
            if (n >= a.N) continue;
            float v = acc[i][j] * a.scale;
            int64_t off = b * a.y_sb + m * a.y_sr + n * a.y_sc;
            if constexpr (OUT_BF16)
                reinterpret_cast<__nv_bfloat16 *>(a.Y)[off] = __float2bfloat16_rn(v);
            else
                reinterpret_cast<float *>(a.Y)[off] = v;
        }
    }
}

}  // namespace

int launch_gemm_simt(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                     const rmm_mat_t *Y, void *ws, cudaStream_t stream)
{
    SimtArgs a;
    a.A = A->ptr; a.B = B->ptr; a.Y = Y->ptr; a.idx = idx;
    a.M = A->rows; a.K = A->cols; a.N = B->cols; a.k = k;
    a.a_sb = A->stride_batch; a.a_sr = A->stride_row; a.a_sc = A->stride_col;
    a.b_sb = B->stride_batch; a.b_sr = B->stride_row; a.b_sc = B->stride_col;
    a.y_sb = Y->stride_batch; a.y_sr = Y->stride_row; a.y_sc = Y->stride_col;
    a.scale = scale;
    a.status = &reinterpret_cast<WsHeader *>(ws)->status;
    if (A->batch > 65535 || ceil_div(a.M, BM) > 65535)
        return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm (FMA path): batch or M/64 exceeds 65535");
    dim3 grid((unsigned)ceil_div(a.N, BN), (unsigned)ceil_div(a.M, BM), (unsigned)A->batch);
    const bool in_bf16 = A->dtype == RMM_BF16, out_bf16 = Y->dtype == RMM_BF16;
    prof_begin("reduced_gemm_simt_kernel", stream);
    if (in_bf16 && out_bf16) launch_kernel(reduced_gemm_simt_kernel<true, true>, grid, dim3(THREADS), 0, stream, 1, a);
    else if (in_bf16) launch_kernel(reduced_gemm_simt_kernel<true, false>, grid, dim3(THREADS), 0, stream, 1, a);
    else if (out_bf16) launch_kernel(reduced_gemm_simt_kernel<false, true>, grid, dim3(THREADS), 0, stream, 1, a);
    else launch_kernel(reduced_gemm_simt_kernel<false, false>, grid, dim3(THREADS), 0, stream, 1, a);
    return check_launch("reduced_gemm_simt_kernel", stream);
}

}  // namespace rmm
