// Decode-step form of the reduced product (paper App. "Implementation Details" / "Complexity Analysis": at a decoding
// step the activation block has one row, or a few): y = scale * x[:, I] W[I, :] with M <= 4 rows.  This is the one
// regime where RMM cuts BYTES, not only flops: only the kept rows of W are read, so the kernel is HBM-bound on
// k * N * 2 bytes.  No packing, no tensor cores.
//
// A block owns 256 output columns and one slice of the kept rows.  The gathered activations x[m, idx[r]] of a chunk of
// rows are staged in shared memory once; each warp then streams its rows of W (one 512-byte coalesced load per row,
// four rows in flight), every lane keeping MB x 8 fp32 accumulators.  Warps are combined through shared memory, row
// slices through an fp32 partial array summed in slice order by the last block of a column chunk (deterministic).
#include "common.cuh"

namespace rmm {
namespace {

constexpr int kGemvThreads = 256, kGemvCols = 256, kChunk = 256;

struct GemvArgs {
    const __nv_bfloat16 *x, *w;
    void *y;
    const int32_t *idx;
    int64_t N, K, k, x_sr, w_sr, y_sr;
    int M, splits, rows_per_split, y_bf16;
    float scale;
    float *partials;     // [splits, M, N]
    unsigned *counters;  // [N / 256]
    int *status;
};

template <int MB>
__global__ void __launch_bounds__(kGemvThreads) reduced_gemv_kernel(GemvArgs a)
{
    extern __shared__ __align__(16) float s_red[];  // [8 warps][MB][256]
    __shared__ float s_x[MB][kChunk];
    __shared__ int s_row[kChunk];
    __shared__ int s_last;
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t n0 = (int64_t)blockIdx.x * kGemvCols;
    const int split = blockIdx.y;
    const int64_t r_begin = (int64_t)split * a.rows_per_split, r_end = min(a.k, r_begin + a.rows_per_split);
    const bool col_ok = n0 + lane * 8 < a.N;  // N is a multiple of 8

    float acc[MB][8];
#pragma unroll
    for (int m = 0; m < MB; ++m)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[m][e] = 0.f;

    for (int64_t c0 = r_begin; c0 < r_end; c0 += kChunk) {
        const int rows = (int)min((int64_t)kChunk, r_end - c0);
        __syncthreads();
        if (tid < rows) {
            int j = a.idx != nullptr ? __ldg(a.idx + c0 + tid) : (int)(c0 + tid);
            if (j < 0 || j >= a.K) {
                atomicExch(a.status, (int)RMM_ERR_BOUNDS);
                j = -1;
            }
            s_row[tid] = j;
#pragma unroll
            for (int m = 0; m < MB; ++m)
                s_x[m][tid] = (j >= 0 && m < a.M) ? __bfloat162float(a.x[(int64_t)m * a.x_sr + j]) : 0.f;
        }
        __syncthreads();
        constexpr int U = MB <= 2 ? 8 : 4;  // rows of W in flight per warp
        for (int t0 = warp; t0 < rows; t0 += 8 * U) {
            uint4 q[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = t0 + u * 8;
                const int j = t < rows ? s_row[t] : -1;
                q[u] = (j >= 0 && col_ok) ? __ldg(reinterpret_cast<const uint4 *>(a.w + (int64_t)j * a.w_sr + n0) + lane)
                                          : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = t0 + u * 8;
                if (t >= rows) break;
                const unsigned wv[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
                float wf[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    wf[2 * i] = __uint_as_float(wv[i] << 16);
                    wf[2 * i + 1] = __uint_as_float(wv[i] & 0xffff0000u);
                }
#pragma unroll
                for (int m = 0; m < MB; ++m) {
                    const float xv = s_x[m][t];
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[m][e] = fmaf(xv, wf[e], acc[m][e]);
                }
            }
        }
    }
    // combine the 8 warps (fixed order), one thread per output column
#pragma unroll
    for (int m = 0; m < MB; ++m)
#pragma unroll
        for (int e = 0; e < 8; ++e) s_red[(warp * MB + m) * kGemvCols + lane * 8 + e] = acc[m][e];
    __syncthreads();
    const int64_t n = n0 + tid;
    float sum[MB];
#pragma unroll
    for (int m = 0; m < MB; ++m) {
        sum[m] = 0.f;
        for (int w = 0; w < 8; ++w) sum[m] += s_red[(w * MB + m) * kGemvCols + tid];
    }
    bool last = true;
    if (a.splits > 1) {
        if (n < a.N)
#pragma unroll
            for (int m = 0; m < MB; ++m)
                if (m < a.M) a.partials[((int64_t)split * a.M + m) * a.N + n] = sum[m];
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = atomicInc(&a.counters[blockIdx.x], (unsigned)a.splits - 1u) == (unsigned)a.splits - 1u;
        __syncthreads();
        last = s_last != 0;
        if (last) {
            __threadfence();
#pragma unroll
            for (int m = 0; m < MB; ++m) {
                sum[m] = 0.f;
                if (n < a.N && m < a.M)
                    for (int s = 0; s < a.splits; ++s) sum[m] += __ldcg(&a.partials[((int64_t)s * a.M + m) * a.N + n]);
            }
        }
    }
    if (!last || n >= a.N) return;
#pragma unroll
    for (int m = 0; m < MB; ++m) {
        if (m >= a.M) break;
        const float v = sum[m] * a.scale;
        if (a.y_bf16) reinterpret_cast<__nv_bfloat16 *>(a.y)[(int64_t)m * a.y_sr + n] = __float2bfloat16_rn(v);
        else reinterpret_cast<float *>(a.y)[(int64_t)m * a.y_sr + n] = v;
    }
}

}  // namespace

bool gemv_eligible(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y, GemvPlan *plan)
{
    if (A->dtype != RMM_BF16 || B->dtype != RMM_BF16) return false;
    if (A->batch != 1 || A->rows > 4) return false;  // beyond 4 rows the FMA pipes, not HBM, would bound this form
    if (A->stride_col != 1 || B->stride_col != 1 || Y->stride_col != 1) return false;
    const int64_t N = B->cols;
    if (N % 8 != 0 || B->stride_row % 8 != 0 || reinterpret_cast<uintptr_t>(B->ptr) % 16 != 0) return false;
    if (ceil_div(N, kGemvCols) > kHeaderCounters) return false;
    if (plan != nullptr) {
        const int64_t col_blocks = ceil_div(N, kGemvCols);
        int64_t splits = (148 * 4) / col_blocks;  // a few blocks per SM
        const int64_t max_splits = ceil_div(k, 64);
        if (splits > max_splits) splits = max_splits;
        if (splits < 1) splits = 1;
        if (splits > 256) splits = 256;
        plan->rows_per_split = (int)ceil_div(k, splits);
        plan->splits = (int)ceil_div(k, plan->rows_per_split);
        plan->off_partials = RMM_WS_HEADER_BYTES;
        plan->total_bytes = RMM_WS_HEADER_BYTES + (plan->splits > 1 ? align_up((size_t)plan->splits * A->rows * N * 4, 256) : 0);
    }
    return true;
}

int launch_gemv(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale, const rmm_mat_t *Y,
                const GemvPlan &plan, void *ws, cudaStream_t stream)
{
    char *w = static_cast<char *>(ws);
    WsHeader *hdr = reinterpret_cast<WsHeader *>(w);
    GemvArgs a;
    a.x = static_cast<const __nv_bfloat16 *>(A->ptr);
    a.w = static_cast<const __nv_bfloat16 *>(B->ptr);
    a.y = Y->ptr;
    a.idx = idx;
    a.N = B->cols; a.K = A->cols; a.k = k;
    a.x_sr = A->stride_row; a.w_sr = B->stride_row; a.y_sr = Y->stride_row;
    a.M = (int)A->rows; a.splits = plan.splits; a.rows_per_split = plan.rows_per_split;
    a.y_bf16 = Y->dtype == RMM_BF16;
    a.scale = scale;
    a.partials = reinterpret_cast<float *>(w + plan.off_partials);
    a.counters = hdr->counters;
    a.status = &hdr->status;
    dim3 grid((unsigned)ceil_div(a.N, kGemvCols), (unsigned)plan.splits);
    const int mb = a.M <= 1 ? 1 : (a.M <= 2 ? 2 : 4);
    const size_t smem = (size_t)8 * mb * kGemvCols * sizeof(float);
    prof_begin("reduced_gemv_kernel", stream);
    if (mb == 1) launch_kernel(reduced_gemv_kernel<1>, grid, dim3(kGemvThreads), smem, stream, 1, a);
    else if (mb == 2) launch_kernel(reduced_gemv_kernel<2>, grid, dim3(kGemvThreads), smem, stream, 1, a);
    else launch_kernel(reduced_gemv_kernel<4>, grid, dim3(kGemvThreads), smem, stream, 1, a);
    return check_launch("reduced_gemv_kernel", stream);
}

}  // namespace rmm
