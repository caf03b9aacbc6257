// Importance scores and top-k index selection (paper Sec. 3.2: s_j = ||A[:, j]||_2,
// I = TopK({s_j}, ceil(rho d))), as one streaming pass over A whose last-arriving thread block
// selects the index set.
//
// Score pass: HBM-bound.  Each thread owns VEC adjacent columns (one 16-byte load per row) and a
// strided subset of the block's rows; squares of bf16 values are exact in fp32, sums run in fp32
// chains of at most 16 terms that are flushed into fp64, row lanes are combined in fp64 through
// shared memory, row splits through an fp64 partial array combined in split order by the last
// block to arrive (self-resetting atomicInc counter).  Results are therefore run-to-run identical.
//
// Select: radix select on the order-preserving integer image of the fp32 keys (the bits common to all
// keys are skipped, one digit of up to 11 bits over all keys, then 8-bit digits over the keys that share
// the threshold's digit), then one ordered compaction pass that emits the kept indices ascending; among
// keys equal to the threshold the lowest indices are kept.  bf16 matrices that meet the TMA rules are
// streamed by score_tma_kernel (64-column blocks, 256-row tiles through a ring of shared-memory buffers).
#include <cuda.h>
#include <stddef.h>

#include "common.cuh"
#include "select.cuh"

namespace rmm {

namespace {

constexpr int kThreads = 1024;     // one block per SM: its tail (the select) then has 32 warps to work with
constexpr int kUnroll = 4;       // rows in flight per thread (1024 threads x 4 x 16 B = 64 KB in flight per SM)
constexpr int kFlushEvery = 4;   // loop trips between fp32 -> fp64 flushes (kUnroll * kFlushEvery = 16 terms)
constexpr int kFusedSelectMax = 8192;    // largest K whose select runs in the score kernel's tail (32 KB key cache)
constexpr int kCachedSelectMax = 49152;  // largest K the stand-alone select kernel caches in shared memory (192 KB)

using namespace sel;

struct ScoreArgs {
    const void *A;
    int64_t s_batch, s_red, s_n;  // element strides: batch, reduced axis (rows), scored axis (columns)
    int64_t n, m, rows_per_split;
    int row_splits, col_blocks, tx, ty;
    double *partials;    // [batch, row_splits, n]   (unused when row_splits == 1)
    unsigned *counters;  // [batch, col_blocks + 1]
    float *energy;       // [batch, n]  always written (caller's array or workspace)
    float *scores;       // [batch, n]  or null
    int do_select;
    int k;
    int32_t *idx;        // [batch, k]
    float *retained;     // [batch] or null
};

template <int VEC, bool BF16>
__device__ __forceinline__ void load_vec(const void *A, int64_t off, int64_t s_n, float (&v)[VEC])
{
    if constexpr (BF16 && VEC == 8) {
        uint4 q = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(A) + off));
        unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    } else if constexpr (!BF16 && VEC == 4) {
        float4 q = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(A) + off));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    } else {
        static_assert(VEC == 1 || VEC == 4 || VEC == 8, "vector width");
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            if constexpr (BF16)
                v[i] = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(A)[off + i * s_n]);
            else
                v[i] = reinterpret_cast<const float *>(A)[off + i * s_n];
        }
    }
}

// Everything after a block's row loop: combine the row lanes, hand the column sums over (fp64 partials and an arrival
// counter when the rows are split), write energies and scores, and let the last block of a batch element select.
template <int VEC>
__device__ __forceinline__ void score_finish(const ScoreArgs &a, const double (&dacc)[VEC], unsigned char *s_dyn,
                                             SelectSmem &s_sel, int &s_flag)
{
    double *s_part = reinterpret_cast<double *>(s_dyn);
    const int tid = threadIdx.x;
    const int tx = tid % a.tx, ty = tid / a.tx;
    const int64_t b = blockIdx.z;
    const int split = blockIdx.y;
    const int width = a.tx * VEC;  // columns per block
    const int64_t col0 = (int64_t)blockIdx.x * width;
#pragma unroll
    for (int e = 0; e < VEC; ++e) s_part[ty * width + tx * VEC + e] = dacc[e];
    __syncthreads();

    // combine the row lanes in a fixed order, in two levels so that every thread helps: thread (part, c) adds the
    // lanes part, part + parts, ... of column c, then thread c < width (the column's owner) adds the parts in order
    double colsum = 0.0;
    const int64_t mycol = col0 + tid;
    const bool owner = tid < width && mycol < a.n;
    {
        const int parts = kThreads / width;  // width and ty are powers of two with width * ty == kThreads
        const int c = tid % width, part = tid / width;
        double sub = 0.0;
        for (int y = part; y < a.ty; y += parts) sub += s_part[y * width + c];
        __syncthreads();
        s_part[part * width + c] = sub;
        __syncthreads();
        const int np = parts < a.ty ? parts : a.ty;
        if (owner)
            for (int q = 0; q < np; ++q) colsum += s_part[q * width + tid];
    }

    bool finalize = true;
    if (a.row_splits > 1) {
        if (owner) a.partials[(b * a.row_splits + split) * a.n + mycol] = colsum;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            unsigned old = atomicInc(&a.counters[b * (a.col_blocks + 1) + blockIdx.x], (unsigned)a.row_splits - 1u);
            s_flag = (old == (unsigned)a.row_splits - 1u);
        }
        __syncthreads();
        finalize = s_flag != 0;
        if (finalize) {
            __threadfence();
            if (owner) {
                colsum = 0.0;
                for (int s0 = 0; s0 < a.row_splits; s0 += 8) {  // eight independent loads at a time, summed in split order
                    double v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        v[i] = s0 + i < a.row_splits ? __ldcg(&a.partials[(b * a.row_splits + s0 + i) * a.n + mycol]) : 0.0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) colsum += v[i];
                }
            }
        }
    }
    if (!finalize) return;

    if (owner) {
        a.energy[b * a.n + mycol] = (float)colsum;
        if (a.scores != nullptr) a.scores[b * a.n + mycol] = (float)sqrt(colsum);
    }
    if (!a.do_select) return;

    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned old = atomicInc(&a.counters[b * (a.col_blocks + 1) + a.col_blocks], (unsigned)a.col_blocks - 1u);
        s_flag = (old == (unsigned)a.col_blocks - 1u);
    }
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    block_select_any(a.energy + b * a.n, (int)a.n, a.k, a.idx + b * (int64_t)a.k,
                     a.retained ? a.retained + b : nullptr, s_sel, reinterpret_cast<unsigned *>(s_dyn));
}

template <int VEC, bool BF16>
__global__ void __launch_bounds__(kThreads, 1) score_select_kernel(ScoreArgs a)
{
    extern __shared__ __align__(128) unsigned char s_dyn[];  // row-lane partial sums, later the select's key cache
    __shared__ SelectSmem s_sel;
    __shared__ int s_flag;
    pdl_wait();

    const int tid = threadIdx.x;
    const int tx = tid % a.tx, ty = tid / a.tx;
    const int64_t b = blockIdx.z;
    const int split = blockIdx.y;
    const int width = a.tx * VEC;  // columns per block
    const int64_t col0 = (int64_t)blockIdx.x * width;
    const int64_t col = col0 + (int64_t)tx * VEC;
    const int64_t r_begin = (int64_t)split * a.rows_per_split;
    const int64_t r_end = min(a.m, r_begin + a.rows_per_split);

    double dacc[VEC];
    float facc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) { dacc[e] = 0.0; facc[e] = 0.f; }

    if (col < a.n) {
        const int64_t base = b * a.s_batch + col * a.s_n;
        int trips = 0;
        for (int64_t r = r_begin + ty; r < r_end; r += (int64_t)a.ty * kUnroll) {
            float v[kUnroll][VEC];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                int64_t rr = r + (int64_t)u * a.ty;
                if (rr < r_end) {
                    load_vec<VEC, BF16>(a.A, base + rr * a.s_red, a.s_n, v[u]);
                } else {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) v[u][e] = 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
#pragma unroll
                for (int e = 0; e < VEC; ++e) facc[e] = fmaf(v[u][e], v[u][e], facc[e]);
            if (++trips == kFlushEvery) {
                trips = 0;
#pragma unroll
                for (int e = 0; e < VEC; ++e) { dacc[e] += (double)facc[e]; facc[e] = 0.f; }
            }
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) dacc[e] += (double)facc[e];
    }
    score_finish<VEC>(a, dacc, s_dyn, s_sel, s_flag);
}

// ---- the same pass with the rows streamed through shared memory by TMA ------------------------------------------------
// For bf16 matrices that satisfy the TMA rules.  A block owns 64 columns (128 contiguous bytes per row) and streams
// its rows as 256-row tiles (32 KB) through a ring of kTmaStages buffers: the copies in flight cost no registers, so
// about 128 KB per SM are outstanding, against the 64 KB that 1024 threads x 4 register loads allow.  Rows or columns
// outside the matrix arrive as zeros (tensor-map bounds), so the loop has no edge cases.  Thread (tx, ty) reads the
// 16-byte group tx of rows ty and ty + 128 of every tile.
constexpr int kTmaStages = 6, kTmaRows = 256, kTmaCols = 64;
constexpr int kTmaStageBytes = kTmaRows * kTmaCols * 2;
constexpr unsigned long long kScoreWaitNs = 2000000000ull;

__device__ __forceinline__ bool score_wait(uint32_t bar, uint32_t parity, int *status)
{
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 255u) == 255u) {  // bounded: give up after 2 s, report, and let the block finish with what it has
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            if (now - t0 > kScoreWaitNs) {
                atomicExch(status, (int)RMM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1) score_tma_kernel(const __grid_constant__ CUtensorMap map_a, ScoreArgs a, int *status)
{
    extern __shared__ __align__(128) unsigned char s_dyn[];  // the tile ring; afterwards partial sums and the key cache
    __shared__ SelectSmem s_sel;
    __shared__ int s_flag;
    __shared__ __align__(8) unsigned long long s_bar[2 * kTmaStages];

    const int tid = threadIdx.x, lane = tid & 31;
    const int tx = tid & 7, ty = tid >> 3;  // 8 column groups x 128 row lanes
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(s_dyn);
    const uint32_t bars = (uint32_t)__cvta_generic_to_shared(s_bar);
    auto full_bar = [&](int st) { return bars + 8u * st; };
    auto empty_bar = [&](int st) { return bars + 8u * (kTmaStages + st); };
    const int64_t r_begin = (int64_t)blockIdx.y * a.rows_per_split;
    const int64_t r_end = min(a.m, r_begin + a.rows_per_split);
    const int n_tiles = (int)((r_end - r_begin + kTmaRows - 1) / kTmaRows);
    const int col0 = (int)blockIdx.x * kTmaCols;

    if (tid == 0) {
        for (int st = 0; st < kTmaStages; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full_bar(st)), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty_bar(st)), "r"(kThreads / 32) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    }
    __syncthreads();
    pdl_wait();

    auto issue = [&](int t) {  // thread 0 only: fetch tile t into its ring slot
        const int st = t % kTmaStages;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full_bar(st)), "r"(kTmaStageBytes) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
            ::"r"(ring + st * kTmaStageBytes), "l"(&map_a), "r"(col0), "r"((int)(r_begin + (int64_t)t * kTmaRows)),
              "r"((int)blockIdx.z), "r"(full_bar(st))
            : "memory");
    };
    constexpr int kAhead = kTmaStages - 2;  // tiles in flight ahead of the consumers
    if (tid == 0)
        for (int t = 0; t < kAhead && t < n_tiles; ++t) issue(t);

    double dacc[8];
    float facc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { dacc[e] = 0.0; facc[e] = 0.f; }
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
        const int st = t % kTmaStages;
        const uint32_t ph = (uint32_t)(t / kTmaStages) & 1u;
        if (tid == 0 && t + kAhead < n_tiles) {
            // the slot of tile t + kAhead was last used by tile t - 2: wait until every warp has released it
            const int nt = t + kAhead, ns = nt % kTmaStages;
            if (nt >= kTmaStages && !score_wait(empty_bar(ns), (uint32_t)(nt / kTmaStages - 1) & 1u, status)) ok = false;
            if (ok) issue(nt);
        }
        if (!score_wait(full_bar(st), ph, status)) { ok = false; }
        const uint4 *tile = reinterpret_cast<const uint4 *>(s_dyn + st * kTmaStageBytes);
        const uint4 q0 = tile[ty * 8 + tx], q1 = tile[(ty + 128) * 8 + tx];
        const unsigned w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo0 = __uint_as_float(w[i] << 16), hi0 = __uint_as_float(w[i] & 0xffff0000u);
            const float lo1 = __uint_as_float(w[4 + i] << 16), hi1 = __uint_as_float(w[4 + i] & 0xffff0000u);
            facc[2 * i] = fmaf(lo1, lo1, fmaf(lo0, lo0, facc[2 * i]));
            facc[2 * i + 1] = fmaf(hi1, hi1, fmaf(hi0, hi0, facc[2 * i + 1]));
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(st)) : "memory");
        if ((t & 7) == 7) {  // 16 terms per fp32 chain, then fp64
#pragma unroll
            for (int e = 0; e < 8; ++e) { dacc[e] += (double)facc[e]; facc[e] = 0.f; }
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) dacc[e] += (double)facc[e];
    __syncthreads();  // every tile has landed and been read: the ring can be reused for the partial sums
    score_finish<8>(a, dacc, s_dyn, s_sel, s_flag);
}

__global__ void __launch_bounds__(1024) select_kernel(const float *keys, int K, int k, int32_t *idx, float *retained,
                                                      int use_cache)
{
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ SelectSmem s_sel;
    pdl_wait();
    const int64_t b = blockIdx.x;
    block_select_any(keys + b * K, K, k, idx + b * (int64_t)k, retained ? retained + b : nullptr, s_sel,
                     use_cache ? reinterpret_cast<unsigned *>(s_dyn) : nullptr);
}

}  // namespace

int plan_score(const rmm_mat_t *A, int axis, ScorePlan *p)
{
    if (A == nullptr || A->ptr == nullptr) return fail(RMM_ERR_INVALID_ARG, "score: null matrix");
    if (A->batch < 1 || A->rows < 1 || A->cols < 1) return fail(RMM_ERR_INVALID_ARG, "score: non-positive dimension");
    if (axis != 0 && axis != 1) return fail(RMM_ERR_INVALID_ARG, "score: axis must be 0 or 1");
    if (A->dtype != RMM_BF16 && A->dtype != RMM_F32) return fail(RMM_ERR_UNSUPPORTED, "score: dtype");
    if (A->stride_batch < 0 || A->stride_row < 0 || A->stride_col < 0)
        return fail(RMM_ERR_UNSUPPORTED, "score: negative stride");
    p->n = axis == 1 ? A->cols : A->rows;
    p->m = axis == 1 ? A->rows : A->cols;
    p->s_n = axis == 1 ? A->stride_col : A->stride_row;
    p->s_red = axis == 1 ? A->stride_row : A->stride_col;
    p->s_batch = A->stride_batch;
    if (p->n > (int64_t)1 << 30 || p->m > (int64_t)1 << 40 || A->batch > 65535)
        return fail(RMM_ERR_UNSUPPORTED, "score: dimension too large (n <= 2^30, batch <= 65535)");

    const size_t es = dtype_size(A->dtype);
    const int full = A->dtype == RMM_BF16 ? 8 : 4;
    const bool vec_ok = p->s_n == 1 && p->n % full == 0 && (reinterpret_cast<uintptr_t>(A->ptr) % 16 == 0) &&
                        (p->s_red * es) % 16 == 0 && (p->s_batch * es) % 16 == 0;
    p->vec = vec_ok ? full : 1;
    // thread layout: tx column groups x ty row lanes.  Narrow blocks (down to 8 groups = 128 contiguous bytes per
    // row) are preferred as long as the grid stays within one block per SM, because a block that owns all the rows
    // of its columns needs no cross-block combine; row splits only fill the machine when there are few columns.
    const int64_t sms = 148;
    int64_t groups = ceil_div(p->n, p->vec);
    int tx = 32;
    while (tx > 1 && tx / 2 >= groups) tx /= 2;
    const int tx_min = p->vec > 1 ? 8 : 32;
    while (tx > tx_min && ceil_div(groups, tx / 2) * A->batch <= sms) tx /= 2;
    // bf16 matrices that meet the TMA rules stream through shared memory in 64-column blocks (score_tma_kernel)
    p->use_tma = p->vec == 8 && A->dtype == RMM_BF16 && p->n >= kTmaCols && p->m <= INT32_MAX;
    if (p->use_tma) tx = 8;
    p->tx = tx;
    p->ty = kThreads / tx;
    p->col_blocks = (int)ceil_div(p->n, (int64_t)tx * p->vec);
    int64_t splits = sms / ((int64_t)p->col_blocks * A->batch);
    int64_t min_rows = p->use_tma ? 2 * kTmaRows : (int64_t)p->ty * kUnroll * 2;
    int64_t max_splits = p->m / min_rows;
    if (max_splits < 1) max_splits = 1;
    if (splits > max_splits) splits = max_splits;
    if (splits > 64) splits = 64;
    if (splits < 1) splits = 1;
    p->rows_per_split = ceil_div(p->m, splits);
    if (p->use_tma && splits > 1) p->rows_per_split = ceil_div(p->rows_per_split, kTmaRows) * kTmaRows;  // whole tiles
    p->row_splits = (int)ceil_div(p->m, p->rows_per_split);

    int64_t n_counters = A->batch * (p->col_blocks + 1);
    p->counters_in_header = n_counters <= kHeaderCounters;
    size_t off = RMM_WS_HEADER_BYTES;
    p->off_counters = off;
    if (!p->counters_in_header) off += align_up((size_t)n_counters * 4, 256);
    p->off_partials = off;
    if (p->row_splits > 1) off += align_up((size_t)A->batch * p->row_splits * p->n * 8, 256);
    p->off_energy = off;
    off += align_up((size_t)A->batch * p->n * 4, 256);
    p->total_bytes = off;
    return RMM_OK;
}

int launch_score_select(const rmm_mat_t *A, const ScorePlan &p, bool do_select, int64_t k, int32_t *idx,
                        float *scores, float *energy, float *retained, void *ws, cudaStream_t stream)
{
    char *w = static_cast<char *>(ws);
    WsHeader *hdr = reinterpret_cast<WsHeader *>(w);
    ScoreArgs a;
    a.A = A->ptr;
    a.s_batch = p.s_batch; a.s_red = p.s_red; a.s_n = p.s_n;
    a.n = p.n; a.m = p.m; a.rows_per_split = p.rows_per_split;
    a.row_splits = p.row_splits; a.col_blocks = p.col_blocks; a.tx = p.tx; a.ty = p.ty;
    a.partials = reinterpret_cast<double *>(w + p.off_partials);
    if (p.counters_in_header) {
        a.counters = hdr->counters;
    } else {
        a.counters = reinterpret_cast<unsigned *>(w + p.off_counters);
        cudaError_t e = cudaMemsetAsync(a.counters, 0, (size_t)A->batch * (p.col_blocks + 1) * 4, stream);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "score: memset: %s", cudaGetErrorString(e));
    }
    a.energy = energy ? energy : reinterpret_cast<float *>(w + p.off_energy);
    a.scores = scores;
    const bool fused = do_select && p.n <= kFusedSelectMax;
    a.do_select = fused ? 1 : 0;
    a.k = (int)k;
    a.idx = idx;
    a.retained = retained;

    dim3 grid((unsigned)p.col_blocks, (unsigned)p.row_splits, (unsigned)A->batch);
    const bool bf16 = A->dtype == RMM_BF16;
    size_t smem = (size_t)kThreads * p.vec * sizeof(double);
    if (fused && (size_t)p.n * 4 > smem) smem = (size_t)p.n * 4;
    if (p.use_tma) {
        CUtensorMap map;
        const uint64_t dims[3] = {(uint64_t)p.n, (uint64_t)p.m, (uint64_t)A->batch};
        const uint64_t st[2] = {(uint64_t)p.s_red * 2, A->batch > 1 ? (uint64_t)p.s_batch * 2 : (uint64_t)p.s_red * 2 * (uint64_t)p.m};
        const uint32_t box[3] = {kTmaCols, kTmaRows, 1};
        int rc = make_map(&map, const_cast<void *>(a.A), 3, dims, st, box, false);
        if (rc != RMM_OK) return rc;
        static PerDeviceOnce tma_configured;
        if (tma_configured.first()) {
            cudaError_t e = cudaFuncSetAttribute(score_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTmaStages * kTmaStageBytes);
            if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "score: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        prof_begin("score_tma_kernel", stream);
        launch_kernel(score_tma_kernel, grid, dim3(kThreads), kTmaStages * kTmaStageBytes, stream, 1, map, a, &hdr->status);
        int rc2 = check_launch("score_tma_kernel", stream);
        if (rc2 != RMM_OK || !do_select || fused) return rc2;
        return launch_select(a.energy, A->batch, p.n, k, idx, retained, ws, stream);
    }
    static PerDeviceOnce configured;
    if (configured.first()) {
        const int big = kThreads * 8 * (int)sizeof(double);
        cudaError_t e = cudaFuncSetAttribute(score_select_kernel<8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(score_select_kernel<4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(score_select_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(score_select_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "score: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    prof_begin("score_select_kernel", stream);
    if (bf16 && p.vec == 8) launch_kernel(score_select_kernel<8, true>, grid, dim3(kThreads), smem, stream, 1, a);
    else if (bf16) launch_kernel(score_select_kernel<1, true>, grid, dim3(kThreads), smem, stream, 1, a);
    else if (p.vec == 4) launch_kernel(score_select_kernel<4, false>, grid, dim3(kThreads), smem, stream, 1, a);
    else launch_kernel(score_select_kernel<1, false>, grid, dim3(kThreads), smem, stream, 1, a);
    int rc = check_launch("score_select_kernel", stream);
    if (rc != RMM_OK || !do_select || fused) return rc;
    return launch_select(a.energy, A->batch, p.n, k, idx, retained, ws, stream);
}

int launch_select(const float *keys, int64_t batch, int64_t K, int64_t k, int32_t *idx, float *retained, void *ws,
                  cudaStream_t stream)
{
    (void)ws;
    const int threads = 1024;
    const int use_cache = K <= kCachedSelectMax;
    const size_t smem = use_cache ? (size_t)K * 4 : 0;
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCachedSelectMax * 4);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "select: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    prof_begin("select_kernel", stream);
    launch_kernel(select_kernel, dim3((unsigned)batch), dim3(threads), smem, stream, 1, keys, (int)K, (int)k, idx, retained, use_cache);
    return check_launch("select_kernel", stream);
}

}  // namespace rmm

// ------------------------------------------------------------------------------------------------------------------
// rmm_score_select_static: fused score + select for callers that cannot hand the library any scratch memory.
//
// Some callers run where device allocation is off the table: inside a region that must not touch the allocator (a
// real-time loop, a plugin sandbox whose host gives it inputs and outputs only, code that runs after the memory pool
// has been frozen), so they can neither cudaMalloc a workspace nor ask a framework for one.  For them the scratch of
// the score pass (row-split partial sums, arrival counters, the energy keys) lives in the file-scope device array
// below.  Every GPU that loads this library carries the array until the process exits.
// ------------------------------------------------------------------------------------------------------------------
#define RMM_STATIC_SCRATCH_BYTES (4u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[RMM_STATIC_SCRATCH_BYTES];

namespace rmm {
namespace {
constexpr int kMaxDevices = 64;
// Device address of g_static_scratch, per device ordinal; NULL until set up.  Two host threads that make their first
// call at the same time both look the address up and store the same value.  The address belongs to the device's
// primary context: it does not survive cudaDeviceReset() (a process that resets a device must not call these entry
// points on it afterwards).
std::atomic<void *> g_static_scratch_ptr[kMaxDevices];

// In host code `g_static_scratch` names a host-side shadow of the symbol, not device memory: the device address has
// to be asked for, once per device, with that device current.
int static_scratch(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "score_select_static: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(RMM_ERR_UNSUPPORTED, "score_select_static: device index %d is not covered", dev);
    void *p = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || p == nullptr)
            return fail(RMM_ERR_CUDA, "score_select_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        g_static_scratch_ptr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return RMM_OK;
}
}  // namespace
}  // namespace rmm

extern "C" size_t rmm_score_select_static_capacity(void) { return RMM_STATIC_SCRATCH_BYTES; }

extern "C" int rmm_score_select_static(const rmm_mat_t *A, int axis, double rho, int64_t k, int32_t *idx, float *scores,
                                       float *energy, float *retained, void *stream)
{
    using namespace rmm;
    ScorePlan p;
    int rc = plan_score(A, axis, &p);
    if (rc != RMM_OK) return rc;
    if (idx == nullptr) return fail(RMM_ERR_INVALID_ARG, "score_select_static: idx is NULL");
    int64_t kk = k;
    if (k < 0 || k > p.n) return fail(RMM_ERR_INVALID_ARG, "score_select_static: k = %lld is outside [0, n]", (long long)k);
    if (k == 0 && (rc = rmm_keep_count(rho, p.n, &kk)) != RMM_OK)
        return fail(rc, "score_select_static: rho = %g is outside (0, 1]", rho);
    if (p.total_bytes > RMM_STATIC_SCRATCH_BYTES)
        return fail(RMM_ERR_WORKSPACE,
                    "score_select_static: this problem needs %zu bytes of scratch but the built-in array holds %u; "
                    "use rmm_score_select with a caller-provided workspace",
                    p.total_bytes, (unsigned)RMM_STATIC_SCRATCH_BYTES);
    void *ws = nullptr;
    if ((rc = static_scratch(&ws)) != RMM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the arrival counters must start at zero.  The status word in front
    // of them is left alone, so that an error a kernel reported stays there until rmm_score_select_static_status reads it.
    cudaError_t e = cudaMemsetAsync(static_cast<char *>(ws) + offsetof(WsHeader, counters), 0,
                                    RMM_WS_HEADER_BYTES - offsetof(WsHeader, counters), st);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "score_select_static: cudaMemsetAsync: %s", cudaGetErrorString(e));
    return launch_score_select(A, p, true, kk, idx, scores, energy, retained, ws, st);
}

extern "C" int rmm_score_select_static_status(int *device_status)
{
    using namespace rmm;
    if (device_status == nullptr) return fail(RMM_ERR_INVALID_ARG, "score_select_static_status: NULL argument");
    void *ws = nullptr;
    int rc = static_scratch(&ws);
    if (rc != RMM_OK) return rc;
    return rmm_status_read(ws, device_status);  // blocking 4-byte copy; clears the word if it was set
}
