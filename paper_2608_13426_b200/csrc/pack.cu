// Gathers that bring the kept slices of the contraction axis (paper Sec. 3.2: A[:, I] and B[I, :]) into
// contiguous operands that TMA tile loads can fetch.  Up to two gathers run in ONE launch (e.g. A[:, I] and
// B[I, :] of a product, or Q[:, I] and K[:, I] of an attention head group): block ranges are split between them.
//
// Column gather  dst[b, r, j] = src[sb, r, idx[b, j]]   (the contraction axis is the contiguous one: element-granular,
//                so no bulk-copy engine can do it).  A block stages R whole source rows in shared memory with
//                coalesced 16-byte loads, then every thread builds pairs of output elements from shared memory and
//                writes 4 bytes; the index pairs are read once per thread and reused for the R rows.  Rows too long
//                for shared memory, or not 16-byte aligned, take the direct form (2-byte gathers from global memory).
//                Long rows (a staged row above 36 KB, e.g. a 28672-wide intermediate axis) take pack_long_kernel: one
//                persistent 1024-thread block per SM streams whole rows through two shared-memory buffers with bulk
//                async copies, so the next row lands while the current one is gathered; every thread keeps its index
//                pairs in registers across all rows (3.1 -> about 5 TB/s on 32768 x 28672).
// Row gather     dst[b, j, :] = src[sb, idx[b, j], :]    16-byte vectors, 8 kept rows per block.
// sb = (b + b_off) / b_div maps a batch entry to its source (grouped-query heads share K and V).
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace rmm {
namespace {

constexpr int kThreadsPack = 256;
constexpr int kThreadsLong = 1024;          // pack_long_kernel
constexpr int kLongPairs = 16;              // output pairs per thread and row it can hold: k <= 2 * 16 * 1024
constexpr int kLongMaxRowBytes = 110 * 1024;  // two such rows (and their zero pads) must fit in shared memory
constexpr int kMaxStageBytes = 96 * 1024;  // longest source row that is staged in shared memory
constexpr int kStageTarget = 36 * 1024;    // preferred staging size (two 8192-column rows with their zero pads): several blocks per SM stay resident
constexpr int kDirectRows = 4;
constexpr int kRowsPerBlock = 8;  // kept rows copied by one block of the row gather

struct PackJob {
    int type;  // 0 none, 1 columns staged, 2 columns direct, 3 rows
    const __nv_bfloat16 *src;
    __nv_bfloat16 *dst;
    const int32_t *idx;
    int64_t batch, rows, K, s_batch, s_row, b_off, b_div, idx_stride, k, ld_dst, n;
    int R;                      // staged rows per block
    int64_t bx, by, blocks;     // block grid of this job: bx * by * batch
};

struct PackArgs {
    PackJob job[2];
    int *status;
};

__device__ __forceinline__ int checked_index(const int32_t *ix, int64_t j, int64_t k, int64_t K, int *status)
{
    if (j >= k) return -1;
    int v = ix != nullptr ? __ldg(ix + j) : (int)j;
    if (v < 0 || v >= K) {
        atomicExch(status, (int)RMM_ERR_BOUNDS);
        return -1;
    }
    return v;
}

__device__ __forceinline__ unsigned lds_u16(uint32_t addr)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}

// Staged rows have a pitch of K + 8 elements; the 8 spare elements are zero, so a missing or bad index simply
// points at column K and the inner loop has no predicates.  All inner-loop addressing is 32-bit.
__device__ void pack_cols_staged(const PackJob &p, int64_t blk, int *status, unsigned char *smem)
{
    const int64_t b = blk / p.bx, r0 = (blk % p.bx) * p.R;
    const int tid = threadIdx.x;
    const int K = (int)p.K, kv = K / 8, pitch_v = kv + 1;  // 16-byte vectors per source row / per staged row
    const unsigned short *s16 = reinterpret_cast<const unsigned short *>(p.src) + ((b + p.b_off) / p.b_div) * p.s_batch;
    uint4 *stage = reinterpret_cast<uint4 *>(smem);
    const int nrows = (int)min((int64_t)p.R, p.rows - r0);
    if (kv >= kThreadsPack) {
        for (int r = 0; r < nrows; ++r) {
            const uint4 *srow = reinterpret_cast<const uint4 *>(s16 + (r0 + r) * p.s_row);
            uint4 *drow = stage + r * pitch_v;
            if (tid == 0) drow[kv] = make_uint4(0, 0, 0, 0);
            for (int c0 = tid; c0 < kv; c0 += 4 * kThreadsPack) {  // four independent loads in flight per thread and row
                uint4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (c0 + i * kThreadsPack < kv) v[i] = __ldg(srow + c0 + i * kThreadsPack);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (c0 + i * kThreadsPack < kv) drow[c0 + i * kThreadsPack] = v[i];
            }
        }
    } else {
        // short rows (attention heads): the block's rows are staged as one flat list of 16-byte vectors
        const int total = nrows * kv;
        const unsigned short *s0 = s16 + r0 * p.s_row;
        for (int r = tid; r < nrows; r += kThreadsPack) stage[r * pitch_v + kv] = make_uint4(0, 0, 0, 0);
        for (int f0 = tid; f0 < total; f0 += 4 * kThreadsPack) {
            uint4 v[4];
            int at[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int f = f0 + i * kThreadsPack;
                if (f < total) {
                    const int r = f / kv, c = f - r * kv;
                    v[i] = __ldg(reinterpret_cast<const uint4 *>(s0 + (int64_t)r * p.s_row) + c);
                    at[i] = r * pitch_v + c;
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (f0 + i * kThreadsPack < total) stage[at[i]] = v[i];
        }
    }
    __syncthreads();
    const uint32_t rows_s = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t pitch_b = (uint32_t)pitch_v * 16u;
    const int32_t *ix = p.idx != nullptr ? p.idx + b * p.idx_stride : nullptr;
    const int half = (int)(p.ld_dst / 2), k = (int)p.k;
    unsigned *drow0 = reinterpret_cast<unsigned *>(p.dst + b * p.rows * p.ld_dst) + ((r0 * p.ld_dst) >> 1);
    if (2 * half <= kThreadsPack) {
        // short rows: thread = (output pair, row phase); every thread keeps its two source columns for all its rows
        const int rows_par = kThreadsPack / half, jp = tid % half, rsub = tid / half;
        if (rsub < rows_par) {
            uint32_t cb[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = 2 * jp + h;
                int c = K;
                if (j < k) {
                    c = ix != nullptr ? __ldg(ix + j) : j;
                    if (c < 0 || c >= K) {
                        atomicExch(status, (int)RMM_ERR_BOUNDS);
                        c = K;
                    }
                }
                cb[h] = (uint32_t)c * 2u;
            }
            for (int r = rsub; r < nrows; r += rows_par) {
                const uint32_t row_s = rows_s + (uint32_t)r * pitch_b;
                drow0[r * half + jp] = lds_u16(row_s + cb[0]) | (lds_u16(row_s + cb[1]) << 16);
            }
        }
        return;
    }
    for (int jp0 = tid; jp0 < half; jp0 += 4 * kThreadsPack) {  // four output pairs per thread: index loads first
        uint32_t cb[8];  // byte offsets of the source columns inside a staged row
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int jp = jp0 + i * kThreadsPack;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = 2 * jp + h;
                int c = K;  // the zero column
                if (jp < half && j < k) {
                    c = ix != nullptr ? __ldg(ix + j) : j;
                    if (c < 0 || c >= K) {
                        atomicExch(status, (int)RMM_ERR_BOUNDS);
                        c = K;
                    }
                }
                cb[2 * i + h] = (uint32_t)c * 2u;
            }
        }
        uint32_t row_s = rows_s;
        unsigned *d = drow0 + jp0;
        for (int r = 0; r < nrows; ++r, row_s += pitch_b, d += half) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const unsigned v = lds_u16(row_s + cb[2 * i]) | (lds_u16(row_s + cb[2 * i + 1]) << 16);
                if (jp0 + i * kThreadsPack < half) d[i * kThreadsPack] = v;
            }
        }
    }
}

// One warp owns 256 adjacent output columns of kDirectRows rows.  Lane l produces the output pairs (2l, 2l+1) + 64 i,
// so the 32 lanes of one load read neighbouring kept columns and one store writes 128 contiguous bytes.
__device__ void pack_cols_direct(const PackJob &p, int64_t blk, int *status)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t b = blk / (p.bx * p.by), rem = blk % (p.bx * p.by);
    const int64_t j0 = ((rem % p.bx) * (kThreadsPack / 32) + warp) * 256;
    const int64_t r_begin = (rem / p.bx) * kDirectRows, r_end = min(p.rows, r_begin + kDirectRows);
    if (j0 >= p.ld_dst) return;
    const int32_t *ix = p.idx != nullptr ? p.idx + b * p.idx_stride : nullptr;
    int c[8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int h = 0; h < 2; ++h) c[2 * i + h] = checked_index(ix, j0 + 64 * i + 2 * lane + h, p.k, p.K, status);
    const unsigned short *s16 = reinterpret_cast<const unsigned short *>(p.src) + ((b + p.b_off) / p.b_div) * p.s_batch;
    unsigned *d32 = reinterpret_cast<unsigned *>(p.dst + b * p.rows * p.ld_dst);
    unsigned out[kDirectRows][4];
#pragma unroll
    for (int rr = 0; rr < kDirectRows; ++rr) {
        const int64_t r = r_begin + rr;
        const unsigned short *row = s16 + (r < r_end ? r : r_begin) * p.s_row;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            unsigned lo = c[2 * i] >= 0 ? (unsigned)__ldg(row + c[2 * i]) : 0u;
            unsigned hi = c[2 * i + 1] >= 0 ? (unsigned)__ldg(row + c[2 * i + 1]) : 0u;
            out[rr][i] = lo | (hi << 16);
        }
    }
#pragma unroll
    for (int rr = 0; rr < kDirectRows; ++rr) {
        const int64_t r = r_begin + rr;
        if (r >= r_end) break;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t j = j0 + 64 * i + 2 * lane;
            if (j < p.ld_dst) d32[(r * p.ld_dst + j) >> 1] = out[rr][i];
        }
    }
}

__device__ void pack_rows(const PackJob &p, int64_t blk, int *status)
{
    const int64_t b = blk / (p.bx * p.by), rem = blk % (p.bx * p.by);
    const int64_t j0 = (rem / p.bx) * kRowsPerBlock, nvec = p.n / 8;
    const uint4 *sbase = reinterpret_cast<const uint4 *>(p.src) + ((b + p.b_off) / p.b_div) * (p.s_batch / 8);
    uint4 *dbase = reinterpret_cast<uint4 *>(p.dst) + (b * p.k) * (p.ld_dst / 8);
    const int32_t *ix = p.idx != nullptr ? p.idx + b * p.idx_stride : nullptr;
    int rows[kRowsPerBlock];
#pragma unroll
    for (int i = 0; i < kRowsPerBlock; ++i) {
        rows[i] = j0 + i < p.k ? checked_index(ix, j0 + i, p.k, p.K, status) : -2;  // -1: bad index, write zeros; -2: no row
    }
    for (int64_t c = (rem % p.bx) * kThreadsPack + threadIdx.x; c < nvec; c += p.bx * kThreadsPack) {
        uint4 v[kRowsPerBlock];
#pragma unroll
        for (int i = 0; i < kRowsPerBlock; ++i)
            v[i] = rows[i] >= 0 ? __ldg(sbase + rows[i] * (p.s_row / 8) + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < kRowsPerBlock; ++i)
            if (rows[i] != -2) dbase[(j0 + i) * (p.ld_dst / 8) + c] = v[i];
    }
}

// Row gather of short rows (fewer 16-byte vectors per row than threads per block): a thread owns one vector position
// and kRowsPerBlock rows, so a block covers (threads / vectors) * kRowsPerBlock rows with every thread busy.
__device__ void pack_rows_short(const PackJob &p, int64_t blk, int *status)
{
    const int nvec = (int)(p.n / 8), rows_par = kThreadsPack / nvec, rows_blk = rows_par * kRowsPerBlock;
    const int64_t b = blk / p.by, j0 = (blk % p.by) * rows_blk;
    const int c = threadIdx.x % nvec, rsub = threadIdx.x / nvec;
    if (rsub >= rows_par) return;
    const uint4 *sbase = reinterpret_cast<const uint4 *>(p.src) + ((b + p.b_off) / p.b_div) * (p.s_batch / 8);
    uint4 *dbase = reinterpret_cast<uint4 *>(p.dst) + (b * p.k) * (p.ld_dst / 8);
    const int32_t *ix = p.idx != nullptr ? p.idx + b * p.idx_stride : nullptr;
    int rows[kRowsPerBlock];
#pragma unroll
    for (int i = 0; i < kRowsPerBlock; ++i) {
        const int64_t j = j0 + rsub + (int64_t)rows_par * i;
        rows[i] = j < p.k ? checked_index(ix, j, p.k, p.K, status) : -2;  // -1: bad index, write zeros; -2: no row
    }
    uint4 v[kRowsPerBlock];
#pragma unroll
    for (int i = 0; i < kRowsPerBlock; ++i) v[i] = rows[i] >= 0 ? __ldg(sbase + rows[i] * (p.s_row / 8) + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int i = 0; i < kRowsPerBlock; ++i)
        if (rows[i] != -2) dbase[(j0 + rsub + (int64_t)rows_par * i) * (p.ld_dst / 8) + c] = v[i];
}

// Column gather of long rows: see the file header.  Block b owns the contiguous (batch, row) range
// [b * per_block, (b + 1) * per_block); rows stream through two buffers filled by cp.async.bulk.
__global__ void __launch_bounds__(kThreadsLong, 1) pack_long_kernel(const __grid_constant__ PackJob p, int64_t per_block, int *status,
                                                                    unsigned long long wait_ns, int withhold)
{
    using namespace ptx;
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t full[2];
    __shared__ int abort_flag;
    const int tid = threadIdx.x;
    const int K = (int)p.K, k = (int)p.k, half = (int)(p.ld_dst / 2);
    const uint32_t pitch = (uint32_t)(K + 8) * 2u;   // 8 zero elements after each staged row: where missing indices point
    if (tid == 0) {
        mbar_init(smem_u32(&full[0]), 1);
        mbar_init(smem_u32(&full[1]), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 8) {
        reinterpret_cast<uint32_t *>(smem + (size_t)K * 2)[tid & 3] = 0;
        reinterpret_cast<uint32_t *>(smem + pitch + (size_t)K * 2)[tid & 3] = 0;
    }
    __syncthreads();
    pdl_wait();
    const int64_t total = p.batch * p.rows;
    const int64_t lo = (int64_t)blockIdx.x * per_block, hi = min(total, lo + per_block);
    auto issue = [&](int64_t g, int stage) {  // thread 0: one row, global -> shared
        const int64_t b = g / p.rows, r = g - b * p.rows;
        const __nv_bfloat16 *src = p.src + ((b + p.b_off) / p.b_div) * p.s_batch + r * p.s_row;
        const uint32_t bar = smem_u32(&full[stage]), dst = smem_u32(smem) + (uint32_t)stage * pitch;
        mbar_arrive_expect_tx(bar, (uint32_t)K * 2u);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst), "l"(src), "r"((uint32_t)K * 2u), "r"(bar) : "memory");
    };
    if (tid == 0 && lo < hi && !(withhold && blockIdx.x == 0)) issue(lo, 0);  // (test switch: block 0's first row is never requested)
    uint32_t cb[2 * kLongPairs];   // byte offsets of this thread's source columns inside a staged row
    int64_t cur_batch = -1;
    for (int64_t g = lo; g < hi; ++g) {
        const int it = (int)(g - lo), stage = it & 1;
        // the other buffer was last read in the previous iteration, which ended with a block-wide barrier
        if (tid == 0 && g + 1 < hi) issue(g + 1, stage ^ 1);
        const int64_t b = g / p.rows, r = g - b * p.rows;
        if (b != cur_batch) {
            cur_batch = b;
            const int32_t *ix = p.idx != nullptr ? p.idx + b * p.idx_stride : nullptr;
#pragma unroll
            for (int i = 0; i < kLongPairs; ++i) {
                const int jp = tid + i * kThreadsLong;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int j = 2 * jp + h;
                    int c = K;
                    if (jp < half && j < k) {
                        c = ix != nullptr ? __ldg(ix + j) : j;
                        if (c < 0 || c >= K) {
                            atomicExch(status, (int)RMM_ERR_BOUNDS);
                            c = K;
                        }
                    }
                    cb[2 * i + h] = (uint32_t)c * 2u;
                }
            }
        }
        // every thread comes out of the wait (landed, timed out, or told to abort) and the block decides together
        const bool landed = mbar_wait(smem_u32(&full[stage]), (uint32_t)(it >> 1) & 1u, &abort_flag, status, wait_ns);
        if (!__syncthreads_and(landed)) break;
        const uint32_t row_s = smem_u32(smem) + (uint32_t)stage * pitch;
        unsigned *d = reinterpret_cast<unsigned *>(p.dst + b * p.rows * p.ld_dst + r * p.ld_dst);
#pragma unroll
        for (int i = 0; i < kLongPairs; ++i) {
            const int jp = tid + i * kThreadsLong;
            if (jp < half) d[jp] = lds_u16(row_s + cb[2 * i]) | (lds_u16(row_s + cb[2 * i + 1]) << 16);
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kThreadsPack, 4) pack_kernel(const __grid_constant__ PackArgs a)
{
    extern __shared__ __align__(16) unsigned char smem[];
    pdl_wait();
    int64_t blk = blockIdx.x;
    const int which = blk < a.job[0].blocks ? 0 : 1;
    if (which == 1) blk -= a.job[0].blocks;
    const PackJob &p = a.job[which];
    if (p.type == 1) pack_cols_staged(p, blk, a.status, smem);
    else if (p.type == 2) pack_cols_direct(p, blk, a.status);
    else if (p.type == 3) pack_rows(p, blk, a.status);
    else if (p.type == 4) pack_rows_short(p, blk, a.status);
}

size_t plan_job(PackJob &p)
{
    size_t smem = 0;
    if (p.type == 1) {
        const bool staged = p.K % 8 == 0 && p.s_row % 8 == 0 && p.s_batch % 8 == 0 && reinterpret_cast<uintptr_t>(p.src) % 16 == 0 &&
                            (p.K + 8) * 2 <= kMaxStageBytes && p.K <= INT32_MAX / 4 && p.ld_dst <= INT32_MAX / 4;
        if (staged) {
            int R = (int)(kStageTarget / ((p.K + 8) * 2));
            if (R < 1) R = 1;
            if (R > 128) R = 128;  // short rows (attention heads): many rows per block
            if (R > p.rows) R = (int)p.rows;
            p.R = R;
            p.bx = ceil_div(p.rows, R);
            p.by = 1;
            smem = (size_t)R * (p.K + 8) * 2;
        } else {
            p.type = 2;
            p.bx = ceil_div(p.ld_dst, 256 * (kThreadsPack / 32));
            p.by = ceil_div(p.rows, kDirectRows);
        }
    } else if (p.type == 3 && p.n / 8 <= kThreadsPack / 2) {
        p.type = 4;  // short rows
        p.bx = 1;
        p.by = ceil_div(p.k, (int64_t)(kThreadsPack / (p.n / 8)) * kRowsPerBlock);
    } else if (p.type == 3) {
        int64_t gx = ceil_div(p.n / 8, kThreadsPack);
        p.bx = gx > 8 ? 8 : gx;
        p.by = ceil_div(p.k, kRowsPerBlock);
    }
    p.blocks = p.type == 0 ? 0 : p.bx * p.by * p.batch;
    return smem;
}

}  // namespace

int launch_pack(const PackSpec *specs, int n, int *status, cudaStream_t stream)
{
    if (n < 1 || n > 2) return fail(RMM_ERR_INVALID_ARG, "pack: one or two gathers per launch");
    PackArgs a = {};
    a.status = status;
    size_t smem = 0;
    int64_t blocks = 0;
    for (int i = 0; i < n; ++i) {
        const PackSpec &s = specs[i];
        PackJob &p = a.job[i];
        p.type = s.rows_gather ? 3 : 1;
        p.src = s.src; p.dst = s.dst; p.idx = s.idx;
        p.batch = s.batch; p.rows = s.rows; p.K = s.K; p.s_batch = s.s_batch; p.s_row = s.s_row;
        p.b_off = s.b_off; p.b_div = s.b_div > 0 ? s.b_div : 1; p.idx_stride = s.idx_stride; p.k = s.k; p.ld_dst = s.ld_dst; p.n = s.n;
        if (s.rows_gather) {
            if (s.n % 8 || s.s_batch % 8 || s.s_row % 8 || s.ld_dst % 8 || reinterpret_cast<uintptr_t>(s.src) % 16 ||
                reinterpret_cast<uintptr_t>(s.dst) % 16)
                return fail(RMM_ERR_UNSUPPORTED, "pack: row gather needs 16-byte aligned operands and pitches that are multiples of 8");
        } else if (s.ld_dst % 2 != 0) {
            return fail(RMM_ERR_UNSUPPORTED, "pack: destination pitch must be even");
        }
        size_t sm = plan_job(p);
        if (sm > smem) smem = sm;
        blocks += p.blocks;
    }
    // long rows leave through their own kernel; what remains (if anything) goes on below
    for (int i = 0; i < n; ++i) {
        PackJob &p = a.job[i];
        const size_t row_bytes = (size_t)(p.K + 8) * 2;
        if (p.type != 1 || row_bytes <= (size_t)kStageTarget || row_bytes > (size_t)kLongMaxRowBytes || p.K % 8 != 0 ||
            p.ld_dst > 2 * kLongPairs * kThreadsLong)
            continue;
        static PerDeviceOnce long_configured;
        if (long_configured.first()) {
            cudaError_t e = cudaFuncSetAttribute(pack_long_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * kLongMaxRowBytes);
            if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "pack: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        int dev = 0, sms = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int64_t total = p.batch * p.rows, per_block = ceil_div(total, sms);
        prof_begin("pack_long_kernel", stream);
        launch_kernel(pack_long_kernel, dim3((unsigned)ceil_div(total, per_block)), dim3(kThreadsLong), 2 * row_bytes, stream, 1, p,
                      per_block, status, wait_limit_ns(), debug_withhold() == WITHHOLD_PACK ? 1 : 0);
        int rc = check_launch("pack_long_kernel", stream);
        if (rc != RMM_OK) return rc;
        blocks -= p.blocks;
        p.type = 0;
        p.blocks = 0;
    }
    if (blocks == 0) return RMM_OK;
    if (a.job[0].type == 0) {  // the block ranges of the merged launch start with job 0
        a.job[0] = a.job[1];
        a.job[1].type = 0;
        a.job[1].blocks = 0;
    }
    if (blocks > INT32_MAX) return fail(RMM_ERR_UNSUPPORTED, "pack: too many blocks");
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxStageBytes);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "pack: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    prof_begin("pack_kernel", stream);
    launch_kernel(pack_kernel, dim3((unsigned)blocks), dim3(kThreadsPack), smem, stream, 1, a);
    return check_launch("pack_kernel", stream);
}

}  // namespace rmm
