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
#include <stdlib.h>

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
    unsigned long long wait_ns;  // bound of every device-side wait
    int withhold;                // test switch: block 0 never requests its first tile
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

__device__ __forceinline__ bool score_wait(uint32_t bar, uint32_t parity, int *status, unsigned long long limit_ns = kScoreWaitNs)
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
            if (now - t0 > limit_ns) {
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

    const bool withheld = a.withhold && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
    auto issue = [&](int t) {  // thread 0 only: fetch tile t into its ring slot
        const int st = t % kTmaStages;
        if (withheld && t == 0) return;  // (test switch) never requested: the slot's barrier stays incomplete
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
            if (nt >= kTmaStages && !score_wait(empty_bar(ns), (uint32_t)(nt / kTmaStages - 1) & 1u, status, a.wait_ns)) ok = false;
            if (ok) issue(nt);
        }
        if (!score_wait(full_bar(st), ph, status, a.wait_ns)) ok = false;
        ok = __all_sync(0xffffffffu, ok);  // the warp leaves as a whole (thread 0 also waits on behalf of the producer)
        if (!ok) break;
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
    if (!__syncthreads_and(ok)) {
        // A wait ran out (the status word says so).  The ring is not reused (a copy might still land in it) and nothing
        // is published; copies in flight get time to land before shared memory is released.  The arrival counters of this
        // call stay incomplete: rmm_status_read clears them together with the status word.
        unsigned long long t0, now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        do { __nanosleep(2000); asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now)); } while (now - t0 < 200000ull);
        return;
    }
    // every tile has landed and been read: the ring can be reused for the partial sums
    score_finish<8>(a, dacc, s_dyn, s_sel, s_flag);
}

// ---- the front end of a whole product in ONE launch: scores, selection, and both gathers ---------------------------
// For one bf16 product Y = A[:, I] B[I, :] whose score pass needs no row split (every block owns 64 columns and all
// the rows) and whose keys fit in registers (n <= 8192).  Phases of a block:
//   1. stream its 64 columns of A through the ring and sum the squares (as score_tma_kernel), publish 64 energies;
//   2. grid-wide barrier (an arrival counter and a generation word in the workspace header; the grid is at most one
//      block per SM, all resident; the wait is bounded like every other);
//   3. EVERY block runs the selection on all n energies (redundantly: a block-wide select costs the same whether one
//      block or all of them run it, and nobody then waits for a second barrier), so each knows the threshold, the kept
//      columns among its own 64 and their positions in the index list; block 0 writes the list itself;
//   4. (warps 0-15) the kept columns of A go to Ap for the block's share of the ROWS (all kept columns of those rows):
//      chunks of whole rows arrive in the ring by bulk copies (from L2 when A is small; the first chunks are requested
//      before the barrier), a thread builds four consecutive outputs and stores 8 bytes, so Ap is written in full lines;
//   5. (warps 16-31, at the same time) the rows of B that belong to its kept columns, requested into L2 right after the
//      selection, go to Bp[pos0 .. pos0 + cnt, :] as 16-byte vectors.
// The reduced product then reads Ap and Bp with TMA tile loads.  Against separate score, select and gather launches
// this saves two launches, the hand-off to a single selecting block, and the gather kernel's own staging of A.
#ifdef RMM_FRONT_STAMPS
// Debug build: %globaltimer stamps of the front kernel's phases (first start / last end over all blocks), read back by
// rmm_debug_front_stamps.  Slot 0 is a minimum, the others maxima.
__device__ unsigned long long g_fstamps[16];
#define FSTAMP_MIN(i) do { if (threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); atomicMin(&g_fstamps[i], t_); } } while (0)
#define FSTAMP_MAX(i) do { if (threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); atomicMax(&g_fstamps[i], t_); } } while (0)
#else
#define FSTAMP_MIN(i)
#define FSTAMP_MAX(i)
#endif

struct FrontArgs {
    ScoreArgs sc;             // A, n, m, energy, scores, k, idx, retained (row_splits == 1; counters unused)
    unsigned *grid_bar;       // [2] in the workspace header: arrivals, generation
    __nv_bfloat16 *Ap;        // [m, ldp]
    int64_t ldp;
    const __nv_bfloat16 *B;   // [n, N], row pitch b_sr
    int64_t b_sr, N;
    __nv_bfloat16 *Bp;        // [k, N]
    unsigned long long wait_ns;
    int rows_per_chunk;       // rows of A per chunk of the gather: 64 KB / (2 n)
};

// Tall or wide products gather faster through the separate gather launches (whole rows of A per block with full-line
// stores; rows of B spread over every SM) than through this kernel's 64-byte pieces per row and its 16 copying warps
// per block.  Measured at 8192 columns of A, rho = 0.5: ahead by 4 to 6 us up to 8192 rows when B has 2048 columns,
// level at 16384 rows, behind by 15 % at 32768; behind at every row count when B has 8192 columns.
constexpr int64_t kFrontMaxRows = 8192, kFrontMaxCols = 4096;
constexpr int kChunkSlots = 3;                         // row chunks in the ring
constexpr int kChunkBytes = 2 * kTmaStageBytes;        // 64 KB: rows_per_chunk = 64 KB / row bytes
constexpr int kGroupsPerThread = 4;                    // 8-byte output groups per gathering thread and row: k <= 4 * 4 * 512
constexpr int kFrontCombBytes = (kThreads / 32) * kTmaCols * 8;              // per-warp column sums (fp64)
constexpr int kFrontSmemBytes = kTmaStages * kTmaStageBytes + kFrontCombBytes;

__global__ void __launch_bounds__(kThreads, 1) rmm_front_kernel(const __grid_constant__ CUtensorMap map_a, FrontArgs fa, int *status)
{
    extern __shared__ __align__(128) unsigned char s_dyn[];  // the tile ring, then the per-warp column sums
    __shared__ SelectSmem s_sel;
    __shared__ __align__(8) unsigned long long s_bar[2 * kTmaStages];
    __shared__ int s_ok, s_first, s_end;
    __shared__ int s_pos[kTmaCols];           // position in the index list of each own column, or -1
    __shared__ unsigned short s_own[kTmaCols];  // own kept columns (0 .. 63) in list order

    const ScoreArgs &a = fa.sc;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tx = tid & 7, ty = tid >> 3;  // 8 column groups x 128 row lanes
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(s_dyn);
    const uint32_t bars = (uint32_t)__cvta_generic_to_shared(s_bar);
    auto full_bar = [&](int st) { return bars + 8u * st; };
    auto empty_bar = [&](int st) { return bars + 8u * (kTmaStages + st); };
    const int n_tiles = (int)((a.m + kTmaRows - 1) / kTmaRows);
    const int col0 = (int)blockIdx.x * kTmaCols;

    if (tid == 0) {
        for (int st = 0; st < kTmaStages; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full_bar(st)), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty_bar(st)), "r"(kThreads / 32) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        s_ok = 1;
    }
    __syncthreads();
    pdl_wait();
    FSTAMP_MIN(0);
    unsigned gen0 = 0;
    if (tid == 0) gen0 = *reinterpret_cast<volatile unsigned *>(fa.grid_bar + 1);  // before this block can have arrived

    // Ring protocol.  A slot's `full` barrier completes once per fill, its `empty` barrier once every time all 32 warps
    // have released it.  full_par (every thread) and empty_par (thread 0) hold, per slot, the parity of the next
    // completion to wait for; every completion is waited for exactly once, in order.
    uint32_t full_par = 0, empty_par = 0;
    bool withheld = a.withhold && blockIdx.x == 0;
    auto fill = [&](int slot, int tile) {  // thread 0 only: rows of `tile` -> slot
        if (withheld) {  // (test switch) the block's very first request is dropped: the slot's barrier stays incomplete
            withheld = false;
            return;
        }
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full_bar(slot)), "r"(kTmaStageBytes) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
            ::"r"(ring + slot * kTmaStageBytes), "l"(&map_a), "r"(col0), "r"(tile * kTmaRows), "r"(0), "r"(full_bar(slot))
            : "memory");
    };
    auto wait_empty = [&](int slot) -> bool {  // thread 0 only
        const bool done = score_wait(empty_bar(slot), (empty_par >> slot) & 1u, status, fa.wait_ns);
        empty_par ^= 1u << slot;
        return done;
    };
    auto wait_full = [&](int slot) -> bool {
        const bool done = score_wait(full_bar(slot), (full_par >> slot) & 1u, status, fa.wait_ns);
        full_par ^= 1u << slot;
        return done;
    };
    constexpr int kAhead = kTmaStages - 2;
    if (tid == 0)
        for (int t = 0; t < kAhead && t < n_tiles; ++t) fill(t, t);

    // ---- 1. scores
    double dacc[8];
    float facc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { dacc[e] = 0.0; facc[e] = 0.f; }
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
        const int st = t % kTmaStages;
        if (tid == 0 && t + kAhead < n_tiles) {
            const int nt = t + kAhead, ns = nt % kTmaStages;
            if (nt >= kTmaStages && !wait_empty(ns)) ok = false;
            if (ok) fill(ns, nt);
        }
        if (!wait_full(st)) ok = false;
        ok = __all_sync(0xffffffffu, ok);  // the warp leaves as a whole (thread 0 also waits on behalf of the producer)
        if (!ok) break;
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
        if ((t & 7) == 7) {
#pragma unroll
            for (int e = 0; e < 8; ++e) { dacc[e] += (double)facc[e]; facc[e] = 0.f; }
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) dacc[e] += (double)facc[e];
    if (!ok) s_ok = 0;
    __syncthreads();
    FSTAMP_MAX(1);
    // A block that ran out of time leaves the ring alone (a copy may still land in it), lets the others through the
    // grid barrier, gives copies in flight time to land and returns; the status word tells the host.
    const bool alive = s_ok != 0;
    // The gather (step 4) works on ROW chunks of A: this block's rows [row_lo, row_hi), rb rows at a time, every chunk
    // whole (a chunk fills up to a third of the ring).
    const int used_slots = n_tiles < kTmaStages ? n_tiles : kTmaStages;
    const int rows_per_block = (int)((a.m + gridDim.x - 1) / gridDim.x);
    const int64_t row_lo = (int64_t)blockIdx.x * rows_per_block, row_hi = min(a.m, row_lo + rows_per_block);
    const int rb = fa.rows_per_chunk;                                                 // rows per chunk
    const int n_chunks = row_hi > row_lo ? (int)((row_hi - row_lo + rb - 1) / rb) : 0;
    const uint32_t row_bytes = (uint32_t)a.n * 2u;                                    // a multiple of 16
    auto fill_chunk = [&](int c) {  // thread 0: chunk c of the block's rows -> chunk slot c % 3 (two ring slots wide)
        const int cs = c % kChunkSlots;
        const int64_t r0 = row_lo + (int64_t)c * rb;
        const int nr = (int)min((int64_t)rb, row_hi - r0);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full_bar(cs)), "r"((uint32_t)nr * row_bytes) : "memory");
        const unsigned short *g = reinterpret_cast<const unsigned short *>(a.A) + r0 * a.s_red;
        for (int r = 0; r < nr; ++r)  // a row of A is contiguous: one bulk copy per row
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(ring + cs * kChunkBytes + (uint32_t)r * row_bytes), "l"(g + (int64_t)r * a.s_red), "r"(row_bytes), "r"(full_bar(cs))
                         : "memory");
    };
    if (alive) {
        // Row lanes in a fixed order: the four lanes of a column group inside a warp by shuffles, then the 32 warps in
        // order by the column's owner thread.
        double *s_comb = reinterpret_cast<double *>(s_dyn + kTmaStages * kTmaStageBytes);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            dacc[e] += __shfl_xor_sync(0xffffffffu, dacc[e], 8);
            dacc[e] += __shfl_xor_sync(0xffffffffu, dacc[e], 16);
        }
        if (lane < 8) {
#pragma unroll
            for (int e = 0; e < 8; ++e) s_comb[warp * kTmaCols + tx * 8 + e] = dacc[e];
        }
        __syncthreads();
        if (tid < kTmaCols && col0 + tid < a.n) {
            double colsum = 0.0;
#pragma unroll 8
            for (int q = 0; q < kThreads / 32; ++q) colsum += s_comb[q * kTmaCols + tid];
            a.energy[col0 + tid] = (float)colsum;
            if (a.scores != nullptr) a.scores[col0 + tid] = (float)sqrt(colsum);
        }
        if (tid == 0) {
            // every release of the stream is waited for (the ring is free), then the gather's first chunks are requested:
            // they arrive (from L2 when A is small) while the barrier and the selection run
            for (int s2 = 0; s2 < used_slots && ok; ++s2)
                if (!wait_empty(s2)) ok = false;
            if (ok) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                for (int c = 0; c < kChunkSlots && c < n_chunks; ++c) fill_chunk(c);
            }
            if (!ok) s_ok = 0;
        }
    }

    // ---- 2. grid-wide barrier: all energies are visible afterwards.  The block's energy stores are ordered before
    // thread 0's releasing arrival by the block barrier (release is cumulative); the last block to arrive resets the
    // count for the next launch and publishes a new generation, which the others acquire.
    FSTAMP_MAX(2);
    __syncthreads();
    if (tid == 0) {
        const unsigned nblocks = gridDim.x;
        unsigned old;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(fa.grid_bar) : "memory");
        if (old == nblocks - 1u) {
            asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(fa.grid_bar), "r"(0u) : "memory");
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(fa.grid_bar + 1) : "memory");
        } else if (alive) {
            unsigned long long t0 = 0;
            for (uint32_t it = 0;; ++it) {
                unsigned g;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(g) : "l"(fa.grid_bar + 1) : "memory");
                if (g != gen0) break;
                if ((it & 63u) == 63u) {
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                    if (t0 == 0) t0 = now;
                    if (now - t0 > fa.wait_ns) {
                        atomicExch(status, (int)RMM_ERR_TIMEOUT);
                        s_ok = 0;
                        break;
                    }
                }
            }
        }
    }
    __syncthreads();
    if (s_ok == 0) {
        // nothing more is written; copies in flight (if any) get time to land before shared memory is released
        unsigned long long t0, now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        do { __nanosleep(2000); asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now)); } while (now - t0 < 200000ull);
        return;
    }

    // ---- 3. selection, in every block, 8 keys per thread.  (Run by eight warps with 32 keys per thread instead it was
    // slower, 47.6 against 39 us for the kernel at n = 8192: the serial work per thread grows faster than the
    // barriers get cheaper.)
    FSTAMP_MAX(3);
    constexpr int kSelThreads = kThreads, kSelItems = kFusedSelectMax / kSelThreads;
    unsigned short *s_list = reinterpret_cast<unsigned short *>(s_dyn + kTmaStages * kTmaStageBytes);  // position -> column
    if (tid < kSelThreads) {
        unsigned u[kSelItems];
        const int nvalid = load_keys_blocked<kSelItems>(a.energy, (int)a.n, u);
        const Threshold th = block_threshold<kSelItems, kSelThreads>(u, nvalid, a.k, s_sel);
        const unsigned before = block_rank_blocked<kSelItems, kSelThreads>(u, nvalid, th.tau, s_sel);
        unsigned gt_before = before >> 16, eq_before = before & 0xffffu;
        const bool writer = blockIdx.x == 0;
        const int j0 = tid * kSelItems;
        const bool mine = j0 >= col0 && j0 < col0 + kTmaCols;  // the threads that hold this block's columns
        if (mine && j0 == col0) s_first = (int)(gt_before + min(eq_before, th.need_eq));
        double sum_kept = 0.0, sum_all = 0.0;
#pragma unroll
        for (int i = 0; i < kSelItems; ++i) {
            if (i < nvalid) {
                const bool gt = u[i] > th.tau, eq = u[i] == th.tau;
                const bool keep = gt || (eq && eq_before < th.need_eq);
                const unsigned pos = gt_before + min(eq_before, th.need_eq);
                if (keep) s_list[pos] = (unsigned short)(j0 + i);     // the whole list: the gather of A needs every kept column
                if (writer && keep) a.idx[pos] = j0 + i;
                if (mine) s_pos[j0 + i - col0] = keep ? (int)pos : -1;
                if (writer && a.retained != nullptr) {
                    const double f = (double)key_value(u[i]);
                    sum_all += f;
                    if (keep) sum_kept += f;
                }
                gt_before += gt ? 1u : 0u;
                eq_before += eq ? 1u : 0u;
            } else if (mine) {
                s_pos[j0 + i - col0] = -1;
            }
        }
        if (mine && j0 + kSelItems == col0 + kTmaCols) s_end = (int)(gt_before + min(eq_before, th.need_eq));
        if (writer && a.retained != nullptr) {  // uniform over the selecting warps
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                sum_kept += __shfl_down_sync(0xffffffffu, sum_kept, d);
                sum_all += __shfl_down_sync(0xffffffffu, sum_all, d);
            }
            if (lane == 0) {
                s_sel.red[warp] = sum_kept;
                s_sel.red[32 + warp] = sum_all;
            }
            group_sync<kSelThreads>();
            if (tid == 0) {
                double x = 0.0, y = 0.0;
                for (int w2 = 0; w2 < kSelThreads / 32; ++w2) {
                    x += s_sel.red[w2];
                    y += s_sel.red[32 + w2];
                }
                *a.retained = (y > 0.0) ? (float)(x / y) : 1.0f;
            }
        }
    }
    __syncthreads();
    const int pos0 = s_first, cnt = s_end - s_first;
    if (tid < kTmaCols && s_pos[tid] >= 0) s_own[s_pos[tid] - pos0] = (unsigned short)tid;
    __syncthreads();
    {
        // the rows of B that this block copies in step 5 are requested into L2 now, so that they arrive from HBM while
        // the gather of A runs
        const int lines = (int)((fa.N * 2 + 127) / 128);
        const char *b0 = reinterpret_cast<const char *>(fa.B) + (int64_t)col0 * fa.b_sr * 2;
        for (int i = tid; i < cnt * lines; i += kThreads) {
            const int j = i / lines, c = i - j * lines;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(b0 + (int64_t)s_own[j] * fa.b_sr * 2 + (int64_t)c * 128));
        }
    }

    FSTAMP_MAX(4);
    // ---- 4 and 5 run side by side: warps 0 .. 15 gather the block's kept columns of A, warps 16 .. 31 copy its rows
    // of B (requested into L2 above).  A ring slot is still released by 32 arrivals: two lanes of each gathering warp.
    constexpr int kGatherWarps = 16;
    if (warp < kGatherWarps) {
        // ---- 4. kept columns of A -> Ap for this block's ROWS.  What bounds a gather of 2-byte elements is the number of
        // store requests that reach L2 (about 64 G requests/s over the whole GPU, however few bytes each carries: 64-byte
        // pieces per row and column block took 10 us here).  So a block owns whole rows: thread t builds the output
        // groups t, t + 512, ... of four consecutive list positions from four 2-byte shared-memory loads and stores them
        // as one 8-byte word, a warp store is 256 contiguous bytes, and every line of Ap is written once, in full.
        const int gt = tid;                                    // 0 .. 511
        const int n_groups = (int)(fa.ldp / 4);                // groups of four positions per output row
        uint32_t off[kGroupsPerThread][4];                     // byte offset of the source column inside a staged row, or ~0
#pragma unroll
        for (int g = 0; g < kGroupsPerThread; ++g)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = 4 * (gt + g * 32 * kGatherWarps) + e;
                uint32_t o = 0xffffffffu;
                if (j < a.k) o = (uint32_t)s_list[j] * 2u;
                off[g][e] = o;
            }
        for (int c = 0; c < n_chunks && ok; ++c) {
            const int cs = c % kChunkSlots;
            if (tid == 0 && c >= 1 && c - 1 + kChunkSlots < n_chunks) {
                // the slot that chunk c - 1 used is free once all gathering warps have released it
                if (!wait_empty((c - 1) % kChunkSlots)) ok = false;
                if (ok) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    fill_chunk(c - 1 + kChunkSlots);
                }
            }
            if (!wait_full(cs)) ok = false;
            ok = __all_sync(0xffffffffu, ok);  // a warp leaves the loop as a whole
            if (!ok) break;
            const unsigned char *chunk = s_dyn + cs * kChunkBytes;
            const int64_t r0 = row_lo + (int64_t)c * rb;
            const int nr = (int)min((int64_t)rb, row_hi - r0);
            for (int r = 0; r < nr; ++r) {
                const unsigned char *srow = chunk + (uint32_t)r * row_bytes;
                uint2 *drow = reinterpret_cast<uint2 *>(fa.Ap + (r0 + r) * fa.ldp);
#pragma unroll
                for (int g = 0; g < kGroupsPerThread; ++g) {
                    const int grp = gt + g * 32 * kGatherWarps;
                    if (grp < n_groups) {
                        unsigned v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            v[e] = off[g][e] != 0xffffffffu ? (unsigned)*reinterpret_cast<const unsigned short *>(srow + off[g][e]) : 0u;
                        drow[grp] = make_uint2(v[0] | (v[1] << 16), v[2] | (v[3] << 16));
                    }
                }
            }
            __syncwarp();
            if (lane < kThreads / 32 / kGatherWarps) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(cs)) : "memory");
        }
    } else {
        // ---- 5. rows of B of the own kept columns -> Bp[pos0 .. pos0 + cnt, :], 16-byte vectors.  Rows shorter than
        // these warps are wide are copied several at a time (thread = vector c of row j0, j0 + rows_par, ...).
        constexpr int kCopyThreads = kThreads - 32 * kGatherWarps;
        const int ct = tid - 32 * kGatherWarps;
        const int nvec = (int)(fa.N / 8);
        const uint4 *src = reinterpret_cast<const uint4 *>(fa.B) + (int64_t)col0 * (fa.b_sr / 8);
        uint4 *dst = reinterpret_cast<uint4 *>(fa.Bp) + (int64_t)pos0 * nvec;
        const int s_pitch = (int)(fa.b_sr / 8);
        const int rows_par = nvec >= kCopyThreads ? 1 : kCopyThreads / nvec;
        const int c0 = rows_par == 1 ? ct : ct % nvec, j0 = rows_par == 1 ? 0 : ct / nvec;
        if (j0 < rows_par) {
            for (int c = c0; c < nvec; c += kCopyThreads) {
                for (int j = j0; j < cnt; j += 8 * rows_par) {
                    uint4 q[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (j + i * rows_par < cnt) q[i] = __ldg(src + (int)s_own[j + i * rows_par] * s_pitch + c);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (j + i * rows_par < cnt) dst[(j + i * rows_par) * nvec + c] = q[i];
                }
            }
        }
    }
    if (!__syncthreads_and(ok)) {
        unsigned long long t0, now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        do { __nanosleep(2000); asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now)); } while (now - t0 < 200000ull);
        return;
    }
    FSTAMP_MAX(6);
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
    const int64_t sms = sm_count();
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
    a.wait_ns = wait_limit_ns();
    a.withhold = debug_withhold() == WITHHOLD_SCORE;

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

bool front_eligible(const rmm_mat_t *A, const rmm_mat_t *B, const rmm_mat_t *Y, int64_t k, FrontPlan *plan)
{
    TcPlan tc;
    if (A->batch != 1 || !tc_eligible(A, B, k, Y, &tc) || tc.b_kmajor) return false;
    if (A->rows <= 256) return false;  // short outputs: the product fetches the kept rows of B itself
    // RMM_PRODUCT_FUSED=0 / 1 (measurement switch) forces the two-call form / lifts the row limit below
    static const int forced = []() { const char *e = getenv("RMM_PRODUCT_FUSED"); return e ? atoi(e) : -1; }();
    if (forced == 0) return false;
    if (forced != 1 && (A->rows > kFrontMaxRows || B->cols > kFrontMaxCols)) return false;
    ScorePlan sp;
    if (plan_score(A, 1, &sp) != RMM_OK || !sp.use_tma) return false;
    if (sp.n > kFusedSelectMax || sp.n % 8 != 0) return false;
    const int col_blocks = (int)ceil_div(sp.n, kTmaCols);
    // every block owns all the rows of its columns, and the whole grid has to be resident for the grid-wide barrier
    if (col_blocks > sm_count() || col_blocks < sm_count() / 4) return false;
    if (plan != nullptr) {
        plan->col_blocks = col_blocks;
        plan->ldp = (k + 7) / 8 * 8;
        size_t off = RMM_WS_HEADER_BYTES;
        plan->off_energy = off;
        off += align_up((size_t)sp.n * 4, 256);
        plan->off_ap = off;
        off += align_up((size_t)A->rows * plan->ldp * 2, 256);
        plan->off_bp = off;
        off += align_up((size_t)k * B->cols * 2, 256);
        plan->total_bytes = off;
    }
    return true;
}

int launch_front(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, int32_t *idx, float *energy, float *retained,
                 const FrontPlan &plan, void *ws, cudaStream_t stream)
{
    char *w = static_cast<char *>(ws);
    WsHeader *hdr = reinterpret_cast<WsHeader *>(w);
    FrontArgs fa = {};
    ScoreArgs &a = fa.sc;
    a.A = A->ptr;
    a.s_batch = 0; a.s_red = A->stride_row; a.s_n = 1;
    a.n = A->cols; a.m = A->rows; a.rows_per_split = A->rows;
    a.row_splits = 1; a.col_blocks = plan.col_blocks; a.tx = 8; a.ty = kThreads / 8;
    a.partials = nullptr; a.counters = nullptr;
    a.energy = energy != nullptr ? energy : reinterpret_cast<float *>(w + plan.off_energy);
    a.scores = nullptr;
    a.do_select = 1; a.k = (int)k; a.idx = idx; a.retained = retained;
    fa.grid_bar = &hdr->counters[kHeaderCounters - 2];
    fa.Ap = reinterpret_cast<__nv_bfloat16 *>(w + plan.off_ap);
    fa.ldp = plan.ldp;
    fa.B = static_cast<const __nv_bfloat16 *>(B->ptr);
    fa.b_sr = B->stride_row; fa.N = B->cols;
    fa.Bp = reinterpret_cast<__nv_bfloat16 *>(w + plan.off_bp);
    fa.wait_ns = wait_limit_ns();
    a.wait_ns = fa.wait_ns;
    a.withhold = debug_withhold() == WITHHOLD_FRONT;
    CUtensorMap map;
    const uint64_t dims[3] = {(uint64_t)a.n, (uint64_t)a.m, 1};
    const uint64_t st[2] = {(uint64_t)A->stride_row * 2, (uint64_t)A->stride_row * 2 * (uint64_t)a.m};
    const uint32_t box[3] = {kTmaCols, kTmaRows, 1};
    int rc = make_map(&map, const_cast<void *>(a.A), 3, dims, st, box, false);
    if (rc != RMM_OK) return rc;
    // row chunks of the gather: whole rows of A (one bulk copy each), as many as fit 64 KB of the ring
    fa.rows_per_chunk = (int)(kChunkBytes / (a.n * 2));
    if (fa.rows_per_chunk < 1) return fail(RMM_ERR_UNSUPPORTED, "front: row too long");
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(rmm_front_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFrontSmemBytes);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "front: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    prof_begin("rmm_front_kernel", stream);
    launch_kernel(rmm_front_kernel, dim3((unsigned)plan.col_blocks), dim3(kThreads), kFrontSmemBytes, stream, 1, map, fa,
                  &hdr->status);
    return check_launch("rmm_front_kernel", stream);
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

#ifdef RMM_FRONT_STAMPS
// Debug build only: copy the front kernel's phase stamps (nanoseconds of %globaltimer) to out[0 .. 15] and re-arm them.
extern "C" int rmm_debug_front_stamps(unsigned long long *out)
{
    unsigned long long init[16];
    cudaError_t e = cudaMemcpyFromSymbol(out, rmm::g_fstamps, sizeof init);
    for (int i = 0; i < 16; ++i) init[i] = 0;
    init[0] = ~0ull;
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(rmm::g_fstamps, init, sizeof init);
    return e == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}
#endif
