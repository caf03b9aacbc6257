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
constexpr int kRowsPerBlock = 8;   // rows per warp, all in flight at once (the pass is latency-bound otherwise)
constexpr int kRowVecThreads = 256;

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
    unsigned out[kRowsPerBlock][4];
#pragma unroll
    for (int rr = 0; rr < kRowsPerBlock; ++rr) {
        const int64_t r = r_begin + rr;
        const unsigned short *row = s16 + (r < r_end ? r : r_begin) * s_row;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            unsigned lo = c[2 * i] >= 0 ? (unsigned)__ldg(row + c[2 * i]) : 0u;
            unsigned hi = c[2 * i + 1] >= 0 ? (unsigned)__ldg(row + c[2 * i + 1]) : 0u;
            out[rr][i] = lo | (hi << 16);
        }
    }
#pragma unroll
    for (int rr = 0; rr < kRowsPerBlock; ++rr) {
        const int64_t r = r_begin + rr;
        if (r >= r_end) break;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t j = j0 + 64 * i + 2 * lane;
            if (j < ld_dst) d32[(r * ld_dst + j) >> 1] = out[rr][i];
        }
    }
}

// Row gather with 16-byte vectors: one block copies 4 kept rows.
__global__ void __launch_bounds__(kRowVecThreads) pack_rows_kernel(const uint4 *__restrict__ src, int64_t K, int64_t nvec,
                                                                   int64_t s_batch_v, int64_t s_row_v, int64_t b_off,
                                                                   int64_t b_div, const int32_t *__restrict__ idx,
                                                                   int64_t idx_stride, int64_t k, uint4 *__restrict__ dst,
                                                                   int64_t ld_dst_v, int *status)
{
    const int64_t b = blockIdx.z;
    const int64_t j0 = (int64_t)blockIdx.y * 4;
    const uint4 *sbase = src + ((b + b_off) / b_div) * s_batch_v;
    uint4 *dbase = dst + (b * k) * ld_dst_v;
    int rows[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int v = -1;
        if (j0 + i < k) {
            v = idx != nullptr ? __ldg(idx + b * idx_stride + j0 + i) : (int)(j0 + i);
            if (v < 0 || v >= K) {
                if (threadIdx.x == 0) atomicExch(status, (int)RMM_ERR_BOUNDS);
                v = -2;  // write zeros
            }
        }
        rows[i] = v;
    }
    for (int64_t c = (int64_t)blockIdx.x * kRowVecThreads + threadIdx.x; c < nvec; c += (int64_t)gridDim.x * kRowVecThreads) {
        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = rows[i] >= 0 ? __ldg(sbase + rows[i] * s_row_v + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (rows[i] != -1) dbase[(j0 + i) * ld_dst_v + c] = v[i];
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
    prof_begin("pack_cols_kernel", stream);
    pack_cols_kernel<<<grid, kWarps * 32, 0, stream>>>(src, rows, K, s_batch, s_row, b_off, b_div > 0 ? b_div : 1, idx, idx_stride, k, dst,
                                                               ld_dst, status);
    return check_launch("pack_cols_kernel", stream);
}

int launch_pack_rows(const __nv_bfloat16 *src, int64_t batch, int64_t K, int64_t n, int64_t s_batch, int64_t s_row,
                     int64_t b_off, int64_t b_div, const int32_t *idx, int64_t idx_stride, int64_t k,
                     __nv_bfloat16 *dst, int64_t ld_dst, int *status, cudaStream_t stream)
{
    if (n % 8 || s_batch % 8 || s_row % 8 || ld_dst % 8 || reinterpret_cast<uintptr_t>(src) % 16 || reinterpret_cast<uintptr_t>(dst) % 16)
        return fail(RMM_ERR_UNSUPPORTED, "pack_rows: operands must be 16-byte aligned with pitches that are multiples of 8");
    const int64_t nvec = n / 8;
    int64_t gx = ceil_div(nvec, kRowVecThreads);
    if (gx > 8) gx = 8;
    dim3 grid((unsigned)gx, (unsigned)ceil_div(k, 4), (unsigned)batch);
    if (grid.y > 65535u || grid.z > 65535u) return fail(RMM_ERR_UNSUPPORTED, "pack_rows: k/4 or batch exceeds 65535");
    prof_begin("pack_rows_kernel", stream);
    pack_rows_kernel<<<grid, kRowVecThreads, 0, stream>>>(reinterpret_cast<const uint4 *>(src), K, nvec, s_batch / 8, s_row / 8, b_off,
                                                         b_div > 0 ? b_div : 1, idx, idx_stride, k,
                                                         reinterpret_cast<uint4 *>(dst), ld_dst / 8, status);
    return check_launch("pack_rows_kernel", stream);
}

}  // namespace rmm
