// Column gather dst[b, r, j] = src[b, r, idx[b, j]] (bf16): brings A[:, I] (paper Sec. 3.2) into a
// contiguous K-major operand that a TMA tile load can fetch.  A's contraction axis is its contiguous
// axis, so the gather is element-granular and no bulk-copy engine can do it.
//
// One warp owns 256 adjacent output columns of a few rows.  Lane l produces the output pairs
// (2l, 2l+1) + 64 i, so that the 32 lanes of one load instruction read 64 neighbouring kept columns
// (a few 32-byte sectors) and one store instruction writes 128 contiguous bytes.  The index pairs
// are read once per warp and kept in registers for all of its rows.
#include "common.cuh"

namespace rmm {
namespace {

constexpr int kWarps = 8;
constexpr int kRowsPerBlock = 32;

__global__ void __launch_bounds__(kWarps * 32) pack_cols_kernel(const __nv_bfloat16 *__restrict__ src, int64_t rows,
                                                                int64_t K, int64_t s_batch, int64_t s_row,
                                                                int64_t b_off, int64_t b_div,
                                                                const int32_t *__restrict__ idx, int64_t idx_stride,
                                                                int64_t k, __nv_bfloat16 *__restrict__ dst,
                                                                int64_t ld_dst, int *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t b = blockIdx.z;
    const int64_t j0 = ((int64_t)blockIdx.x * kWarps + warp) * 256;  // first output column of this warp
    if (j0 >= ld_dst) return;
    const int32_t *ix = idx != nullptr ? idx + b * idx_stride : nullptr;  // NULL: columns 0 .. k-1 in order

    int c[8];  // source columns of this lane's 4 output pairs; -1 = write zero
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int64_t j = j0 + 64 * i + 2 * lane + h;
            int v = -1;
            if (j < k) {
                v = ix != nullptr ? __ldg(ix + j) : (int)j;
                if (v < 0 || v >= K) {
                    atomicExch(status, (int)RMM_ERR_BOUNDS);
                    v = -1;
                }
            }
            c[2 * i + h] = v;
        }
    }

    const unsigned short *s16 = reinterpret_cast<const unsigned short *>(src) + ((b + b_off) / b_div) * s_batch;
    unsigned *d32 = reinterpret_cast<unsigned *>(dst + b * rows * ld_dst);
    const int64_t r_begin = (int64_t)blockIdx.y * kRowsPerBlock;
    const int64_t r_end = min(rows, r_begin + kRowsPerBlock);
#pragma unroll 2
    for (int64_t r = r_begin; r < r_end; ++r) {
        const unsigned short *row = s16 + r * s_row;
        unsigned out[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            unsigned lo = c[2 * i] >= 0 ? (unsigned)__ldg(row + c[2 * i]) : 0u;
            unsigned hi = c[2 * i + 1] >= 0 ? (unsigned)__ldg(row + c[2 * i + 1]) : 0u;
            out[i] = lo | (hi << 16);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t j = j0 + 64 * i + 2 * lane;
            if (j < ld_dst) d32[(r * ld_dst + j) >> 1] = out[i];
        }
    }
}

}  // namespace

int launch_pack_cols(const __nv_bfloat16 *src, int64_t batch, int64_t rows, int64_t K, int64_t s_batch, int64_t s_row,
                     int64_t b_off, int64_t b_div, const int32_t *idx, int64_t idx_stride, int64_t k,
                     __nv_bfloat16 *dst, int64_t ld_dst, int *status, cudaStream_t stream)
{
    if (ld_dst % 2 != 0) return fail(RMM_ERR_UNSUPPORTED, "pack: destination pitch must be even");
    dim3 grid((unsigned)ceil_div(ld_dst, 256 * kWarps), (unsigned)ceil_div(rows, kRowsPerBlock), (unsigned)batch);
    if (grid.y > 65535u || grid.z > 65535u) return fail(RMM_ERR_UNSUPPORTED, "pack: rows/32 or batch exceeds 65535");
    pack_cols_kernel<<<grid, kWarps * 32, 0, stream>>>(src, rows, K, s_batch, s_row, b_off, b_div > 0 ? b_div : 1, idx, idx_stride, k, dst,
                                                               ld_dst, status);
    return check_launch("pack_cols_kernel");
}

}  // namespace rmm
