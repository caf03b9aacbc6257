// 8-bit operands for the reduced product (the paper's appendix on compatibility with quantisation reports accuracy with
// INT8 and leaves a fused low-bit kernel open; this is the W8A8 form of Y = A[:, I] B[I, :] with e4m3 codes):
//   activations  Aq[i, j] = e4m3(A[i, I_j] / s_i),  s_i = max_j |A[i, I_j]| / 448  (per-row, taken over the KEPT columns
//                only, so the step adapts to what survives the selection; an all-zero row gets s_i = 1)
//   weight       given as e4m3 codes with one scale for the tensor, stored [N, K] (contraction axis contiguous): the kept
//                bytes of every row are gathered
// One block per row: the row is staged in shared memory with 16-byte loads, then gathered (and quantised) from there.
// Every decision that produces a code is taken in fp32 (IEEE division, round-to-nearest-even conversion, saturating).
#include <cuda_fp8.h>

#include "common.cuh"

namespace rmm {
namespace {

constexpr int kThreadsQ = 256;

template <bool QUANT>
__global__ void __launch_bounds__(kThreadsQ) gather_q8_kernel(const void *__restrict__ src, int64_t s_row, int K, const int32_t *__restrict__ idx,
                                                              int k, uint8_t *__restrict__ dst, int64_t ld_dst, float *__restrict__ row_scale,
                                                              int *status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ float s_red[kThreadsQ / 32];
    constexpr int ES = QUANT ? 2 : 1;
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = blockIdx.x;
    {
        const uint4 *g = reinterpret_cast<const uint4 *>(static_cast<const unsigned char *>(src) + row * s_row * ES);
        uint4 *s = reinterpret_cast<uint4 *>(smem);
        const int nvec = (K * ES + 15) / 16;  // the staged row may run a few bytes past K: rows are 16-byte multiples apart
        for (int v = tid; v < nvec; v += kThreadsQ) s[v] = __ldg(g + v);
    }
    __syncthreads();
    auto column = [&](int j) -> int {  // kept column of list position j, or -1
        if (j >= k) return -1;
        const int c = __ldg(idx + j);
        if (c < 0 || c >= K) {
            atomicExch(status, (int)RMM_ERR_BOUNDS);
            return -1;
        }
        return c;
    };
    float inv_step = 1.f, step = 1.f;
    if constexpr (QUANT) {
        const unsigned short *a16 = reinterpret_cast<const unsigned short *>(smem);
        float amax = 0.f;
        for (int j = tid; j < k; j += kThreadsQ) {
            const int c = column(j);
            if (c >= 0) amax = fmaxf(amax, fabsf(__uint_as_float((unsigned)a16[c] << 16)));
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
        if (lane == 0) s_red[warp] = amax;
        __syncthreads();
        amax = s_red[0];
#pragma unroll
        for (int w = 1; w < kThreadsQ / 32; ++w) amax = fmaxf(amax, s_red[w]);
        step = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
        if (tid == 0) row_scale[row] = step;
        (void)inv_step;
    }
    uint32_t *drow = reinterpret_cast<uint32_t *>(dst + row * ld_dst);
    for (int j0 = 4 * tid; j0 < (int)ld_dst; j0 += 4 * kThreadsQ) {
        uint32_t w = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int c = column(j0 + e);
            uint32_t code = 0;
            if (c >= 0) {
                if constexpr (QUANT) {
                    const float x = __uint_as_float((unsigned)reinterpret_cast<const unsigned short *>(smem)[c] << 16);
                    code = __nv_cvt_float_to_fp8(__fdiv_rn(x, step), __NV_SATFINITE, __NV_E4M3);
                } else {
                    code = smem[c];
                }
            }
            w |= code << (8 * e);
        }
        drow[j0 >> 2] = w;
    }
}

}  // namespace

int launch_gather_q8(bool quantise, const void *src, int64_t rows, int64_t s_row, int64_t K, const int32_t *idx, int64_t k, uint8_t *dst,
                     int64_t ld_dst, float *row_scale, int *status, cudaStream_t stream)
{
    const size_t smem = align_up((size_t)K * (quantise ? 2 : 1), 16);
    if (smem > 200 * 1024 || K > INT32_MAX / 4 || rows > INT32_MAX) return fail(RMM_ERR_UNSUPPORTED, "gather_q8: row too long");
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(gather_q8_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gather_q8_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "gather_q8: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    prof_begin("gather_q8_kernel", stream);
    if (quantise)
        launch_kernel(gather_q8_kernel<true>, dim3((unsigned)rows), dim3(kThreadsQ), smem, stream, 1, src, s_row, (int)K, idx, (int)k, dst, ld_dst,
                      row_scale, status);
    else
        launch_kernel(gather_q8_kernel<false>, dim3((unsigned)rows), dim3(kThreadsQ), smem, stream, 1, src, s_row, (int)K, idx, (int)k, dst, ld_dst,
                      row_scale, status);
    return check_launch("gather_q8_kernel", stream);
}

}  // namespace rmm
