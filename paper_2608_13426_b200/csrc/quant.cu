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
#include "sm100_ptx.cuh"

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


// The same gather as a streaming kernel: one persistent 1024-thread block per SM owns a contiguous range of rows, which
// arrive through two shared-memory buffers by bulk asynchronous copies (the next row lands while the current one is
// worked on).  Thread t owns the output words t, t + 1024, ... (four codes each) and keeps the byte offsets of their
// source columns in registers for all its rows, so the index list is read once per block instead of once per row.
constexpr int kThreadsS = 1024;
constexpr int kWordsS = 8;                       // output words per thread: k <= 4 * 8 * 1024
constexpr int kStreamMaxRowBytes = 110 * 1024;   // two such rows (and their zero pads) fit in shared memory
constexpr int kStreamBuffers = 3;                // rows staged at once where three fit (rows up to 73 KB), else two

template <bool QUANT>
__global__ void __launch_bounds__(kThreadsS, 1) gather_q8_stream_kernel(const void *__restrict__ src, int64_t s_row, int K, const int32_t *__restrict__ idx,
                                                                         int k, uint8_t *__restrict__ dst, int64_t ld_dst, float *__restrict__ row_scale,
                                                                         int64_t rows, int64_t per_block, int nbuf, int *status, unsigned long long wait_ns)
{
    using namespace ptx;
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t full[kStreamBuffers];
    __shared__ int abort_flag;
    __shared__ float s_red[kThreadsS / 32];
    constexpr int ES = QUANT ? 2 : 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t row_bytes = (uint32_t)K * ES;           // a multiple of 16
    const uint32_t pitch = row_bytes + 16;                  // 16 zero bytes after each staged row: where missing indices point
    if (tid == 0) {
        for (int b = 0; b < kStreamBuffers; ++b) mbar_init(smem_u32(&full[b]), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 4 * nbuf) reinterpret_cast<uint32_t *>(smem + (size_t)(tid >> 2) * pitch + row_bytes)[tid & 3] = 0;
    __syncthreads();
    pdl_wait();
    const int64_t lo = (int64_t)blockIdx.x * per_block, hi = min(rows, lo + per_block);
    auto issue = [&](int64_t r, int stage) {  // thread 0: one row, global -> shared
        const unsigned char *g = static_cast<const unsigned char *>(src) + r * s_row * ES;
        const uint32_t bar = smem_u32(&full[stage]), d = smem_u32(smem) + (uint32_t)stage * pitch;
        mbar_arrive_expect_tx(bar, row_bytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(d), "l"(g), "r"(row_bytes), "r"(bar) : "memory");
    };
    if (tid == 0)
        for (int b = 0; b < nbuf && lo + b < hi; ++b) issue(lo + b, b);
    // Output j of a row comes from column idx[j].  A warp takes 128 consecutive outputs at a time (group g of the block's
    // 32 x 128): in slot e = 0 .. 3 lane l reads the source of output 32 e + l of them, so the lanes of one instruction read
    // neighbouring kept columns (output words owned whole by a thread made the lanes' reads 16 bytes apart at rho = 1/2:
    // four lanes per bank).  The four bytes of an output word then sit in the four lanes of a quad and are brought
    // together by two shuffle rounds; the warp's 32 words leave as one 128-byte store.
    // Column numbers (column K = the zero pad): bf16 rows hold at most 55 K columns, so two share a register; byte rows
    // keep one per register.
    constexpr int kSlots = 4 * kWordsS;
    constexpr int kRegs = QUANT ? kSlots / 2 : kSlots;
    uint32_t cb[kRegs];
    const int words = (int)(ld_dst / 4);
#pragma unroll
    for (int sl = 0; sl < kSlots; ++sl) {
        const int j = ((sl >> 2) * (kThreadsS / 32) + warp) * 128 + 32 * (sl & 3) + lane;
        uint32_t col = (uint32_t)K;
        if (j < k) {
            const int c = __ldg(idx + j);
            if (c < 0 || c >= K) atomicExch(status, (int)RMM_ERR_BOUNDS);
            else col = (uint32_t)c;
        }
        if constexpr (QUANT) {
            if (sl & 1) cb[sl >> 1] |= col << 16;
            else cb[sl >> 1] = col;
        } else {
            cb[sl] = col;
        }
    }
    auto offset = [&](int sl) -> uint32_t {  // byte offset of the source of slot sl inside the staged row
        if constexpr (QUANT) return ((cb[sl >> 1] >> (16 * (sl & 1))) & 0xffffu) * 2u;
        else return cb[sl];
    };
    const int groups = (int)((ld_dst + 4095) / 4096);  // groups of 4096 outputs (32 warps x 128) that hold any
    const int rr = lane & 3, word_in_warp = 8 * rr + (lane >> 2);  // after the transpose lane 4 m + rr holds word 8 rr + m
    int stage = 0;
    uint32_t parity = 0;
    for (int64_t r = lo; r < hi; ++r) {
        const bool landed = mbar_wait(smem_u32(&full[stage]), parity, &abort_flag, status, wait_ns);
        if (!__syncthreads_and(landed)) break;
        const unsigned char *row = smem + (size_t)stage * pitch;
        // this thread's 32 inputs, read once: bf16 pairs (QUANT) or the bytes themselves, four to a register
        uint32_t val[QUANT ? kSlots / 2 : kSlots / 4];
        float step = 1.f;
        if constexpr (QUANT) {
            float amax = 0.f;
#pragma unroll
            for (int h = 0; h < kSlots / 2; ++h) {
                if ((h >> 1) < groups) {  // (block-uniform: groups of 4096 outputs past k hold nothing)
                    const uint32_t x0 = *reinterpret_cast<const unsigned short *>(row + offset(2 * h));
                    const uint32_t x1 = *reinterpret_cast<const unsigned short *>(row + offset(2 * h + 1));
                    val[h] = x0 | (x1 << 16);
                    amax = fmaxf(amax, fmaxf(fabsf(__uint_as_float(x0 << 16)), fabsf(__uint_as_float(x1 << 16))));
                }
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
            if (lane == 0) s_red[warp] = amax;
            __syncthreads();
            amax = s_red[lane];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
            step = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
            if (tid == 0) row_scale[r] = step;
        } else {
#pragma unroll
            for (int g = 0; g < kSlots / 4; ++g) {
                if (g < groups) {
                    uint32_t word = 0;
#pragma unroll
                    for (int e = 0; e < 4; ++e) word |= (uint32_t)row[offset(4 * g + e)] << (8 * e);
                    val[g] = word;
                }
            }
            __syncthreads();
        }
        // every thread holds what it needs of this buffer (the barrier above): refill it with the row nbuf ahead.  (With
        // rows quantised, s_red is read before the next iteration's barrier and written after it.)
        if (tid == 0 && r + nbuf < hi) issue(r + nbuf, stage);
        uint32_t *drow = reinterpret_cast<uint32_t *>(dst + r * ld_dst);
#pragma unroll
        for (int g = 0; g < kSlots / 4; ++g) {
            if (g >= groups) break;
            uint32_t mine;  // codes of this thread's slots 4 g .. 4 g + 3
            if constexpr (QUANT) {
                // slots 4 g .. 4 g + 3 are val[2 g] (low, high half) and val[2 g + 1]; two codes per conversion
                const float x0 = __uint_as_float(val[2 * g] << 16), x1 = __uint_as_float(val[2 * g] & 0xffff0000u);
                const float x2 = __uint_as_float(val[2 * g + 1] << 16), x3 = __uint_as_float(val[2 * g + 1] & 0xffff0000u);
                const uint32_t lo2 = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(x0, step), __fdiv_rn(x1, step)), __NV_SATFINITE, __NV_E4M3);
                const uint32_t hi2 = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(x2, step), __fdiv_rn(x3, step)), __NV_SATFINITE, __NV_E4M3);
                mine = lo2 | (hi2 << 16);
            } else {
                mine = val[g];
            }
            // 4 x 4 byte transpose among the four lanes of a quad: lane rr ends up with the word of slot 4 g + rr
            uint32_t other = __shfl_xor_sync(0xffffffffu, mine, 1);
            mine = (rr & 1) ? __byte_perm(mine, other, 0x3715) : __byte_perm(mine, other, 0x6240);
            other = __shfl_xor_sync(0xffffffffu, mine, 2);
            mine = (rr & 2) ? __byte_perm(mine, other, 0x3276) : __byte_perm(mine, other, 0x5410);
            const int w = (g * (kThreadsS / 32) + warp) * 32 + word_in_warp;
            if (w < words) drow[w] = mine;
        }
        if (++stage == nbuf) { stage = 0; parity ^= 1u; }
    }
}

}  // namespace

int launch_gather_q8(bool quantise, const void *src, int64_t rows, int64_t s_row, int64_t K, const int32_t *idx, int64_t k, uint8_t *dst,
                     int64_t ld_dst, float *row_scale, int *status, cudaStream_t stream)
{
    const size_t row_bytes = (size_t)K * (quantise ? 2 : 1);
    if (row_bytes % 16 == 0 && row_bytes <= (size_t)kStreamMaxRowBytes && ld_dst <= 4 * kWordsS * kThreadsS && rows >= 32 * (int64_t)sm_count()) {  // (few rows: one block per row keeps every SM busy)
        static PerDeviceOnce stream_configured;
        if (stream_configured.first()) {
            cudaError_t e = cudaFuncSetAttribute(gather_q8_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * (kStreamMaxRowBytes + 16));
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(gather_q8_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * (kStreamMaxRowBytes + 16));
            if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "gather_q8: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        const int64_t per_block = ceil_div(rows, sm_count());
        const unsigned grid = (unsigned)ceil_div(rows, per_block);
        const int nbuf = kStreamBuffers * (row_bytes + 16) <= 2 * (size_t)(kStreamMaxRowBytes + 16) ? kStreamBuffers : 2;
        prof_begin("gather_q8_stream_kernel", stream);
        if (quantise)
            launch_kernel(gather_q8_stream_kernel<true>, dim3(grid), dim3(kThreadsS), nbuf * (row_bytes + 16), stream, 1, src, s_row, (int)K, idx,
                          (int)k, dst, ld_dst, row_scale, rows, per_block, nbuf, status, wait_limit_ns());
        else
            launch_kernel(gather_q8_stream_kernel<false>, dim3(grid), dim3(kThreadsS), nbuf * (row_bytes + 16), stream, 1, src, s_row, (int)K, idx,
                          (int)k, dst, ld_dst, row_scale, rows, per_block, nbuf, status, wait_limit_ns());
        return check_launch("gather_q8_stream_kernel", stream);
    }
    const size_t smem = align_up(row_bytes, 16);
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
