// Reduced product Y = scale * A[:, I] B[I, :] (paper Sec. 3.2) on the sm_100a tensor cores.
//
// Data path per 128 x BN output tile (persistent blocks, one per SM, static round-robin tiles):
//   A[:, I]   packed once by pack_cols_kernel into Ap [b, M, ldp] (K-major); TMA 2-D/3-D tile loads
//             of 128 rows x 64 kept columns into 128-byte-swizzled shared memory.  Columns beyond k
//             are outside the tensor map and arrive as zeros, so k needs no padding.
//   B[I, :]   when B's contraction slices (rows) are contiguous, pack_rows_kernel copies the kept rows into
//             Bp [b, k, N] and 64 x 64 tiles of it are loaded as an MN-major swizzled operand; when B is
//             K-contiguous (K^T in attention) it is packed like A and loaded as K-major tiles.  (Fetching the
//             kept rows inside the producer with TMA gather4 was measured first: at 512 bytes per instruction
//             the copy engine sustained about one instruction per 70 clocks, 2.5x slower than this form.)
//             Outputs of up to 256 rows (small decode batches) skip the packed copy of B: eight gather warps fetch
//             the kept rows straight from B with 16-byte cp.async into the same swizzled layout (one row of the tile
//             = one 512-byte warp request).  There every tile of B is used once, the product is bound by reading the
//             kept rows from HBM, and the copy would triple that traffic.  (For taller outputs the same gather was
//             measured at 1480 clocks per k-block against 590 for TMA tiles of the packed copy: the load/store path
//             does not sustain the L2-to-SM rate that re-used tiles need.)
//   MMA       one elected thread issues tcgen05.mma (bf16 x bf16 -> fp32, M=128, N=BN, K=16 per instruction);
//             accumulators live in TMEM, double buffered (2 x BN columns) so that the epilogue of one tile
//             overlaps the main loop of the next.
//   epilogue  4 warps read TMEM with tcgen05.ld (one accumulator row per thread) and scale.  bf16 output: each warp
//             rounds its 32 x 64 slab into swizzled shared memory and hands it to a TMA tile store (full 128-byte
//             lines per row, edges clipped by the tensor map; direct 64-byte row pieces reached 1.9 TB/s on an
//             output-bound product, the tile stores follow the copy rate).  fp32 output: 128 contiguous bytes per thread.
// Every mbarrier wait is bounded: on expiry the block records RMM_ERR_TIMEOUT in the workspace status
// word, stops issuing work, lets copies in flight land, frees its TMEM and returns.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace rmm {
namespace {

using namespace ptx;

constexpr int BM = 128;
constexpr int BK = 64;           // contraction indices per pipeline stage (128 bytes of bf16)
constexpr int UMMA_K = 16;
constexpr int kThreadsTc = 192;  // warp 0 producer, warp 1 MMA + TMEM owner, warps 2-5 epilogue
constexpr int kThreadsTc2 = 320; // ... and warps 6-9 a second epilogue set, for products with a handful of k-blocks
constexpr int kGatherWarps = 8;  // B_GATHER: warps 6-13 fetch the kept rows of B

#ifdef RMM_GEMM_STAMPS
__device__ unsigned long long g_gstamps[16];
#define GSTAMP_MIN(i) do { unsigned long long t_; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_)); atomicMin(&g_gstamps[i], t_); } while (0)
#define GSTAMP_MAX(i) do { unsigned long long t_; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_)); atomicMax(&g_gstamps[i], t_); } while (0)
#else
#define GSTAMP_MIN(i)
#define GSTAMP_MAX(i)
#endif

struct TcArgs {
    int64_t M, N, k, batch;
    int64_t b_batch_off, b_batch_div, b_batches;  // B batch entry of problem i = min((i + off) / div, b_batches - 1)
    void *Y;
    int64_t y_sb, y_sr;     // element strides of Y (column stride 1)
    float scale;
    int tiles_m, tiles_n;
    int epi_sets;           // 1, or 2: a second set of four epilogue warps takes every other 64-column chunk
    int raster;             // tile columns per raster group (see tile_coords)
    int *status;
    unsigned long long wait_ns;  // bound of every device-side wait
    int withhold;                // test switch: the producer skips its very first stage, so that the waits behind it expire
    int sync_kb;                 // the producers also meet every sync_kb k-blocks inside a tile (0: at tile starts only)
    unsigned *wave_ctr;          // [2] in the workspace header (arrivals, exits) or NULL: keeps the blocks of a wave in step
    float *col_energy;           // [batch, ceil(M / 32), N] or NULL: sum of squares of the rounded outputs per 32-row group
    const float *row_scale;      // 8-bit operands: [batch, M] factor of every output row, or NULL
    // B_GATHER: the unpacked B and the kept row numbers
    const __nv_bfloat16 *b_src;
    const int32_t *b_idx;
    int64_t b_ld, b_sb, b_idx_stride, b_rows;
};

// BN = tile columns (MMA N, accumulator columns); CTAS = CTAs per tile.  With CTAS == 2 a pair of CTAs on one TPC
// shares a 256 x BN tile: each loads its own 128 rows of A and its own half of B's columns, so the operand bytes
// per flop drop by a third against the single-CTA 128 x 256 tile.
template <int BN, int CTAS>
struct SmemLayout {
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = BN / CTAS * BK * 2;
    static constexpr int kStages = (kABytes + kBBytes) > 32768 ? 4 : 6;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kEpiOffset = kStages * kStageBytes;  // epilogue staging: 4 warps x 2 slabs of 32 rows x 128 bytes
    static constexpr int kEpiBytes = 4 * 2 * 4096;
    static constexpr int kBarOffset = kEpiOffset + kEpiBytes;
    static constexpr int kTotal = kBarOffset + 256 + 1024;  // barriers + slack to align the base to 1024 B
};

// Tile order within one batch entry: column groups of `group` tiles, rows within a group, columns fastest.  A wave of
// blocks then shares `group` column slices of B (which stay in L2 while A streams past) instead of all of them; on
// 32768-row outputs the GEMM gained 3 to 23 % over plain row-major order, most where N is largest.  The host picks the
// group width so that the slices of B that a group keeps alive (group * BN columns x k rows) fit well inside L2: 16 for
// short contractions, down to 2 for a 28672-long one.  Outputs with up to `group` tile columns keep the row-major order.
constexpr int kRasterGroupMax = 16;
__device__ __forceinline__ void tile_coords(int64_t t, int tiles_m, int tiles_n, int group, int &tm, int &tn)
{
    const int64_t per_group = (int64_t)group * tiles_m;
    const int grp = (int)(t / per_group);
    const int width = min(group, tiles_n - grp * group);
    const int64_t r = t - grp * per_group;
    tn = grp * group + (int)(r % width);
    tm = (int)(r / width);
}

// FP8: both operands are e4m3 bytes, K-major (tcgen05.mma kind::f8f6f4, 32 contraction indices per instruction); a
// pipeline stage is still 128 bytes per row, i.e. 128 indices instead of 64, and the epilogue multiplies every output
// row by its own scale (the activation row's quantisation step times the weight's).
template <int BN, bool B_KMAJOR, bool OUT_BF16, int CTAS, bool B_GATHER, bool FP8>
__global__ void __launch_bounds__(B_GATHER ? kThreadsTc + 32 * kGatherWarps : kThreadsTc2, 1)
reduced_gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const __grid_constant__ CUtensorMap map_y, TcArgs a)
{
    using L = SmemLayout<BN, CTAS>;
    constexpr int BNL = BN / CTAS;  // columns of B this CTA loads
    const uint32_t rank = CTAS == 2 ? cluster_rank() : 0u;
    constexpr int kStages = L::kStages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_base = base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto tfull_bar = [&](int i) { return bar_base + 8u * (2 * kStages + i); };
    auto tempty_bar = [&](int i) { return bar_base + 8u * (2 * kStages + 2 + i); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kBarOffset + 8 * (2 * kStages + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kBarOffset + 8 * (2 * kStages + 4) + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) { GSTAMP_MIN(0); }
    const int64_t num_tiles = a.batch * a.tiles_m * a.tiles_n;  // tiles of (128 * CTAS) x BN
    const int64_t tile0 = blockIdx.x / CTAS, tile_step = gridDim.x / CTAS;
    constexpr int BKE = FP8 ? 2 * BK : BK;          // contraction indices per stage (128 bytes per row either way)
    constexpr int UK = FP8 ? 2 * UMMA_K : UMMA_K;   // contraction indices per MMA instruction (32 bytes per row)
    static_assert(!FP8 || (B_KMAJOR && !B_GATHER), "8-bit operands: both K-major, packed");
    const int num_kb = (int)((a.k + BKE - 1) / BKE);

    if (threadIdx.x == 32) {  // descriptor fetch overlaps barrier set-up and the TMEM allocation
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        if constexpr (OUT_BF16) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_y) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), B_GATHER ? 1 + 32 * kGatherWarps : 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(tfull_bar(i), 1);
            mbar_init(tempty_bar(i), 4 * CTAS * a.epi_sets);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<CTAS>(smem_u32(const_cast<uint32_t *>(tmem_slot)), 2 * BN);
    tc_fence_before();
    if constexpr (CTAS == 2) cluster_sync_all();
    else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) { GSTAMP_MAX(1); }
    pdl_wait();  // set-up above overlapped the previous kernel's tail; operands are read from here on

    if (warp == 0) {
        // ---------------------------------------------------------------- producer (one thread; the others idle)
        uint32_t s = 0, ph = 0;
        bool ok = true;
        // L2 priority: within a raster group the column slices of B are what every row of tiles comes back to (a row panel
        // of A is shared only by the tiles of one wave and keeps the default priority: marked evict-first it was dropped
        // before its last reader arrived and DRAM traffic went up by two thirds)
        const uint64_t pol_b = l2_policy_evict_last();
        // Blocks start a tile when they finish the last one, so without help the tiles of a wave drift apart along k
        // and a k-slice fetched for one tile of a row or column is gone from L2 when its neighbours ask for it.  The
        // producers therefore meet before every wave: each adds one to a counter and waits, for at most 20 us and
        // without any consequence if the time runs out, until every block with a tile in this wave has done so.
        unsigned wave_target = 0;
        bool meeting = a.wave_ctr != nullptr;
        int64_t wave_first = 0;  // first tile of the current wave
        for (int64_t tile = tile0; lane == 0 && tile < num_tiles && ok; tile += tile_step, wave_first += tile_step) {
            const int64_t in_wave = num_tiles - wave_first < tile_step ? num_tiles - wave_first : tile_step;
            auto meet = [&]() {
                wave_target += (unsigned)(in_wave * CTAS);
                unsigned seen;
                asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(seen) : "l"(a.wave_ctr) : "memory");
                ++seen;
                const unsigned long long t0 = global_ns();
                while (seen < wave_target) {
                    if (global_ns() - t0 >= 20000ull) {  // somebody is missing (a GPU shared with other work): this block
                        meeting = false;                 // stops meeting, and so in turn will those that wait for it
                        break;
                    }
                    __nanosleep(64);
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.wave_ctr) : "memory");
                }
            };
            if (meeting) meet();
            int tm, tn;
            const int64_t b = tile / ((int64_t)a.tiles_n * a.tiles_m);
            tile_coords(tile - b * ((int64_t)a.tiles_n * a.tiles_m), a.tiles_m, a.tiles_n, a.raster, tm, tn);
            int64_t bb = (b + a.b_batch_off) / a.b_batch_div;
            if (bb >= a.b_batches) bb = a.b_batches - 1;
            for (int kb = 0; kb < num_kb; ++kb) {
                if (meeting && a.sync_kb > 0 && kb > 0 && kb % a.sync_kb == 0) meet();
                if (!mbar_wait_lane(empty_bar(s), ph ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                if (a.withhold && blockIdx.x == 0 && tile == tile0 && kb == 0) {
                    // (test switch) this stage is never requested: its barrier stays incomplete
                } else {
                    const uint32_t sa = base + s * L::kStageBytes;
                    const uint32_t sb = sa + L::kABytes;
                    const int row_a = tm * (BM * CTAS) + (int)rank * BM, col_b = tn * BN + (int)rank * BNL;
                    if constexpr (B_GATHER) {
                        mbar_arrive_expect_tx(full_bar(s), L::kABytes);
                        tma_load_3d(sa, &map_a, kb * BKE, row_a, (int)b, full_bar(s));
                    } else if constexpr (CTAS == 1) {
                        mbar_arrive_expect_tx(full_bar(s), L::kStageBytes);
                        tma_load_3d(sa, &map_a, kb * BKE, row_a, (int)b, full_bar(s));
                        if constexpr (B_KMAJOR) {
                            tma_load_3d_hint(sb, &map_b, kb * BKE, col_b, (int)bb, full_bar(s), pol_b);
                        } else {
                            // 64 contraction rows x 64 columns per load; rows past k read as zeros
#pragma unroll
                            for (int c = 0; c < BNL / 64; ++c)
                                tma_load_3d_hint(sb + c * (BK * 128), &map_b, col_b + c * 64, kb * BK, (int)bb, full_bar(s), pol_b);
                        }
                    } else {
                        // both CTAs report their bytes to the leader's barrier; the leader arms it for the pair
                        const uint32_t lead_full = map_to_cta(full_bar(s), 0);
                        if (rank == 0) mbar_arrive_expect_tx(full_bar(s), 2 * L::kStageBytes);
                        tma_load_3d_pair(sa, &map_a, kb * BKE, row_a, (int)b, lead_full);
                        if constexpr (B_KMAJOR) {
                            tma_load_3d_pair_hint(sb, &map_b, kb * BKE, col_b, (int)bb, lead_full, pol_b);
                        } else {
#pragma unroll
                            for (int c = 0; c < BNL / 64; ++c)
                                tma_load_3d_pair_hint(sb + c * (BK * 128), &map_b, col_b + c * 64, kb * BK, (int)bb, lead_full, pol_b);
                        }
                    }
                }
                if (++s == kStages) { s = 0; ph ^= 1u; }
            }
        }
        if (lane == 0 && a.wave_ctr != nullptr) {  // the last block out re-arms the counters for the next launch
            unsigned out;
            asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(out) : "l"(a.wave_ctr + 1) : "memory");
            if (out == gridDim.x - 1) {
                asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(a.wave_ctr), "r"(0u) : "memory");
                asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(a.wave_ctr + 1), "r"(0u) : "memory");
            }
        }
        __syncwarp();
    } else if (warp == 1 && rank == 0) {
        // ---------------------------------------------------------------- MMA issuer (the pair's leader only)
        // instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B K- or MN-major, N = BN, M = 128
        // (operand format fields: 1 = bf16 for kind::f16, 0 = e4m3 for kind::f8f6f4)
        constexpr uint32_t idesc = (1u << 4) | ((FP8 ? 0u : 1u) << 7) | ((FP8 ? 0u : 1u) << 10) | ((B_KMAJOR ? 0u : 1u) << 16) |
                                   ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * CTAS) >> 4) << 24);
        // The issuing thread is the pacemaker of the whole kernel (one thread feeds the tensor cores of one or two
        // SMs), so its loop is kept short: stage and phase are counters, descriptors advance by one add each.
        // A, and a K-major B: 128-byte rows, 8-row groups 1024 B apart; 16 indices = 32 B along the row.
        // MN-major B: 64-column chunks BK*128 B apart, 8-index groups 1024 B apart; 16 indices = 2048 B.
        const uint64_t da0 = smem_desc(base, 16, 1024);
        const uint64_t db0 = B_KMAJOR ? smem_desc(base + L::kABytes, 16, 1024) : smem_desc(base + L::kABytes, BK * 128, 1024);
        const uint32_t a_hi = (uint32_t)(da0 >> 32), b_hi = (uint32_t)(db0 >> 32);
        const uint32_t a_lo0 = (uint32_t)da0, b_lo0 = (uint32_t)db0;
        constexpr uint32_t kStageUnits = L::kStageBytes >> 4, kAStep = 32 >> 4, kBStep = (B_KMAJOR ? 32 : 2048) >> 4;
        const int last_steps = (int)((a.k - (int64_t)(num_kb - 1) * BKE + UK - 1) / UK);  // MMAs of the last k-block
        uint32_t stage = 0, phase = 0, tcount = 0;
        bool ok = true;
        for (int64_t tile = tile0; lane == 0 && tile < num_tiles && ok; tile += tile_step, ++tcount) {
            const uint32_t acc = tcount & 1u, acc_ph = (tcount >> 1) & 1u;
            if (!mbar_wait_lane(tempty_bar(acc), acc_ph ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * BN;
            uint32_t accumulate = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!mbar_wait_lane(full_bar(stage), phase, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                if constexpr (B_GATHER) fence_proxy_async();  // B arrived through the generic proxy (cp.async)
                tc_fence_after();
                if (kb == 0 && tcount == 0) { GSTAMP_MAX(2); }
                const uint32_t a_lo = a_lo0 + stage * kStageUnits, b_lo = b_lo0 + stage * kStageUnits;
                if (kb + 1 < num_kb || last_steps == BK / UMMA_K) {
#pragma unroll
                    for (int ks = 0; ks < BK / UMMA_K; ++ks) {
                        umma_lohi<CTAS, FP8>(d_tmem, a_lo + ks * kAStep, a_hi, b_lo + ks * kBStep, b_hi, idesc, accumulate);
                        accumulate = 1;
                    }
                } else {
                    for (int ks = 0; ks < last_steps; ++ks) {
                        umma_lohi<CTAS, FP8>(d_tmem, a_lo + ks * kAStep, a_hi, b_lo + ks * kBStep, b_hi, idesc, accumulate);
                        accumulate = 1;
                    }
                }
                umma_commit<CTAS>(empty_bar(stage));
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit<CTAS>(tfull_bar(acc));
            GSTAMP_MAX(3);
        }
        __syncwarp();
    } else if (B_GATHER && warp >= 6) {
        // ---------------------------------------------------------------- gather warps: kept rows of B -> MN-major tile
        // Row r of the k-block is one warp request: lane l copies 16 bytes (8 columns) to chunk l / 8, row r, 16-byte
        // unit (l % 8) ^ (r % 8) -- the layout a 128-byte-swizzled TMA tile load would have produced.  The thread does
        // not wait for its copies: the stage's barrier receives this thread's arrival when they have landed, so every
        // free stage has copies in flight.  The MMA thread orders the landed data before the tensor cores'
        // (asynchronous-proxy) reads with a proxy fence.  Row numbers are fetched one k-block ahead.
        static_assert(!B_GATHER || (!B_KMAJOR && CTAS == 1 && BN == 256), "gather form: single-CTA 128 x 256 tiles, row-contiguous B");
        constexpr int kRowsPerWarp = BK / kGatherWarps;
        const int gw = warp - 6;
        uint32_t s = 0, ph = 0;
        bool ok = true;
        for (int64_t tile = tile0; tile < num_tiles && ok; tile += tile_step) {
            int tm, tn;
            const int64_t b = tile / ((int64_t)a.tiles_n * a.tiles_m);
            tile_coords(tile - b * ((int64_t)a.tiles_n * a.tiles_m), a.tiles_m, a.tiles_n, a.raster, tm, tn);
            int64_t bb = (b + a.b_batch_off) / a.b_batch_div;
            if (bb >= a.b_batches) bb = a.b_batches - 1;
            const int32_t *ix = a.b_idx + b * a.b_idx_stride;
            const int64_t col = (int64_t)tn * BN + lane * 8;
            const __nv_bfloat16 *bcol = a.b_src + bb * a.b_sb + (col < a.N ? col : 0);
            const uint32_t col_bytes = col < a.N ? 16u : 0u;
            const uint32_t lane_off = (uint32_t)(lane >> 3) * (BK * 128);
            int rows[kRowsPerWarp], rows_next[kRowsPerWarp];
            auto fetch_rows = [&](int kb, int (&out)[kRowsPerWarp]) {
#pragma unroll
                for (int i = 0; i < kRowsPerWarp; ++i) {
                    const int64_t kk = (int64_t)kb * BK + gw + kGatherWarps * i;
                    out[i] = kk < a.k ? __ldg(ix + kk) : -1;
                }
            };
            fetch_rows(0, rows_next);
            for (int kb = 0; kb < num_kb; ++kb) {
#pragma unroll
                for (int i = 0; i < kRowsPerWarp; ++i) rows[i] = rows_next[i];
                if (kb + 1 < num_kb) fetch_rows(kb + 1, rows_next);
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                const uint32_t sb = base + s * L::kStageBytes + L::kABytes + lane_off;
#pragma unroll
                for (int i = 0; i < kRowsPerWarp; ++i) {
                    const int r = gw + kGatherWarps * i;
                    int row = rows[i];
                    if (row >= a.b_rows || (row < 0 && (int64_t)kb * BK + r < a.k)) {
                        atomicExch(a.status, (int)RMM_ERR_BOUNDS);
                        row = -1;
                    }
                    const uint32_t dst = sb + r * 128 + (((uint32_t)(lane & 7) ^ (uint32_t)(r & 7)) << 4);
                    cp_async_16(dst, row >= 0 ? bcol + (int64_t)row * a.b_ld : bcol, row >= 0 ? col_bytes : 0u);
                }
                cp_async_arrive_noinc(full_bar(s));
                if (++s == kStages) { s = 0; ph ^= 1u; }
            }
        }
        cp_async_commit();
        cp_async_wait<0>();  // nothing of this thread is in flight when the block tears down
    } else if (warp >= 2 && warp < 2 + 4 * a.epi_sets) {
        // ---------------------------------------------------------------- epilogue (warps 2..5, and 6..9 as a second set)
        // With two sets, set s takes the 64-column chunks c with c % 2 == s and every warp has one staging slab
        // instead of two: products with very few k-blocks are bound by this code, and one epilogue warp per scheduler
        // issues too few instructions per clock to keep up with the stores.
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        const int eset = (warp - 2) >> 2, slabs = a.epi_sets == 2 ? 1 : 2;
        uint32_t tcount = 0, ebuf = 0;
        bool ok = true;
        const int slab_id = a.epi_sets == 2 ? eset * 4 + q : q * 2;        // 4 KB slabs; a single set has two per warp
        uint8_t *slab = base_ptr + L::kEpiOffset + slab_id * 4096 + lane * 128;   // this thread's row of the warp's staging slabs
        const uint32_t slab_s = base + L::kEpiOffset + slab_id * 4096;
        for (int64_t tile = tile0; tile < num_tiles && ok; tile += tile_step, ++tcount) {
            int tm, tn;
            const int64_t b = tile / ((int64_t)a.tiles_n * a.tiles_m);
            tile_coords(tile - b * ((int64_t)a.tiles_n * a.tiles_m), a.tiles_m, a.tiles_n, a.raster, tm, tn);
            const uint32_t acc = tcount & 1u, acc_ph = (tcount >> 1) & 1u;
            if (!mbar_wait(tfull_bar(acc), acc_ph, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
            tc_fence_after();
            if (lane == 0) { GSTAMP_MAX(4); }
            const int64_t m_warp = (int64_t)tm * (BM * CTAS) + rank * BM + q * 32, m = m_warp + lane;
            const int64_t n0 = (int64_t)tn * BN;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
            float scale_r = a.scale;  // this thread's output row: the common factor times the row's own (8-bit operands)
            if constexpr (FP8) {
                if (a.row_scale != nullptr && m < a.M) scale_r *= __ldg(a.row_scale + b * a.M + m);
            }
            if constexpr (OUT_BF16) {
                // 64 columns at a time: two TMEM loads, scale and round, one 32 x 64 slab per warp through a TMA store
#pragma unroll 1
                for (int c = eset; c < BN / 64; c += a.epi_sets) {
                    const int64_t n = n0 + c * 64;
                    if (n >= a.N || m_warp >= a.M) break;  // warp-uniform: nothing of this slab lies inside Y
                    uint32_t r0[32], r1[32];
                    tmem_ld32_issue(t_row + c * 64, r0);
                    tmem_ld32_issue(t_row + c * 64 + 32, r1);
                    tmem_ld_wait();
                    if (lane == 0) {  // the slab about to be rewritten has been read by its store
                        if (slabs == 2) bulk_wait_read<1>();
                        else bulk_wait_read<0>();
                    }
                    __syncwarp();
                    uint8_t *row = slab + ebuf * 4096;
                    auto put = [&](const uint32_t (&r)[32], int u0) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint32_t w[4];
#pragma unroll
                            for (int p = 0; p < 4; ++p) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * p]) * scale_r,
                                                                         __uint_as_float(r[8 * v + 2 * p + 1]) * scale_r);
                                w[p] = *reinterpret_cast<uint32_t *>(&h);
                            }
                            *reinterpret_cast<uint4 *>(row + (((u0 + v) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    };
                    put(r0, 0);
                    put(r1, 4);
                    fence_proxy_async();  // generic writes -> visible to the copy engine
                    __syncwarp();
                    if (a.col_energy != nullptr) {
                        // Column energies of the output, where it is produced: lane l sums the squares of columns 2 l and
                        // 2 l + 1 of the slab's 32 rounded rows (two fp32 chains of 16 terms each, exact squares) and stores
                        // the pair; the 32-row groups are added up in fp64, in order, by a small kernel afterwards.
                        const uint8_t *col = base_ptr + L::kEpiOffset + slab_id * 4096 + ebuf * 4096 + (lane & 3) * 4;
                        const int u = lane >> 2;
                        float e0a = 0.f, e0b = 0.f, e1a = 0.f, e1b = 0.f;
#pragma unroll
                        for (int r = 0; r < 32; r += 2) {
                            const uint32_t wa = *reinterpret_cast<const uint32_t *>(col + r * 128 + ((u ^ (r & 7)) << 4));
                            const uint32_t wb = *reinterpret_cast<const uint32_t *>(col + (r + 1) * 128 + ((u ^ ((r + 1) & 7)) << 4));
                            const float a0 = __uint_as_float(wa << 16), a1 = __uint_as_float(wa & 0xffff0000u);
                            const float b0 = __uint_as_float(wb << 16), b1 = __uint_as_float(wb & 0xffff0000u);
                            e0a = fmaf(a0, a0, e0a); e1a = fmaf(a1, a1, e1a);
                            e0b = fmaf(b0, b0, e0b); e1b = fmaf(b1, b1, e1b);
                        }
                        const int64_t cn = n + 2 * lane;
                        if (cn < a.N) {  // N is even for a bf16 tensor-core output
                            const int64_t groups = (a.M + 31) / 32;
                            float2 *dst = reinterpret_cast<float2 *>(a.col_energy + (b * groups + m_warp / 32) * a.N + cn);
                            *dst = make_float2(e0a + e0b, e1a + e1b);
                        }
                    }
                    if (lane == 0) {
                        tma_store_3d(&map_y, slab_s + ebuf * 4096, (int)n, (int)m_warp, (int)b);
                        bulk_commit();
                    }
                    if (slabs == 2) ebuf ^= 1u;
                }
            } else if (eset == 0) {
                // 128 contiguous bytes per thread and 32-column chunk
                auto store_chunk = [&](const uint32_t (&r)[32], int c) {
                    const int64_t n = n0 + c * 32;
                    if (m >= a.M || n >= a.N) return;
                    float *y = reinterpret_cast<float *>(a.Y) + b * a.y_sb + m * a.y_sr + n;
                    if (n + 32 <= a.N) {
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            reinterpret_cast<float4 *>(y)[v] =
                                make_float4(__uint_as_float(r[4 * v]) * scale_r, __uint_as_float(r[4 * v + 1]) * scale_r,
                                            __uint_as_float(r[4 * v + 2]) * scale_r, __uint_as_float(r[4 * v + 3]) * scale_r);
                    } else {
                        for (int e = 0; e < 32 && n + e < a.N; ++e) y[e] = __uint_as_float(r[e]) * scale_r;
                    }
                };
                // four TMEM loads in flight per wait: the load latency is paid BN / 128 times per tile instead of BN / 32
#pragma unroll 1
                for (int c = 0; c < BN / 32; c += 4) {
                    uint32_t r0[32], r1[32], r2[32], r3[32];
                    tmem_ld32_issue(t_row + (c + 0) * 32, r0);
                    tmem_ld32_issue(t_row + (c + 1) * 32, r1);
                    tmem_ld32_issue(t_row + (c + 2) * 32, r2);
                    tmem_ld32_issue(t_row + (c + 3) * 32, r3);
                    tmem_ld_wait();
                    store_chunk(r0, c + 0);
                    store_chunk(r1, c + 1);
                    store_chunk(r2, c + 2);
                    store_chunk(r3, c + 3);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (CTAS == 1) mbar_arrive(tempty_bar(acc));
                else mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));  // the leader's MMA warp waits on it
            }
            if (lane == 0) { GSTAMP_MAX(5); }
        }
        if constexpr (OUT_BF16) {
            if (lane == 0) bulk_wait_read<0>();  // shared memory stays valid until every store has read its slab
            __syncwarp();
        }
    }

    // ---------------------------------------------------------------- teardown
    __syncthreads();
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before shared memory and TMEM are released
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if constexpr (CTAS == 2) {
        tc_fence_before();
        cluster_sync_all();  // the peer may still be reading operands or accumulators that involve this CTA
    }
    tc_fence_after();
    if (warp == 1) tmem_dealloc<CTAS>(tmem_base, 2 * BN);
    if (threadIdx.x == 0) { GSTAMP_MAX(6); }
}

// ----------------------------------------------------------------------------------------------
// host side
// ----------------------------------------------------------------------------------------------
template <int BN, bool B_KMAJOR, bool OUT_BF16, int CTAS, bool B_GATHER = false, bool FP8 = false>
int launch_variant(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &my, const TcArgs &a, cudaStream_t stream)
{
    auto kern = reduced_gemm_tc_kernel<BN, B_KMAJOR, OUT_BF16, CTAS, B_GATHER, FP8>;
    using L = SmemLayout<BN, CTAS>;
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    const int64_t tiles = a.batch * a.tiles_m * a.tiles_n;
    const int64_t slots = sm_count() / CTAS;
    prof_begin("reduced_gemm_tc_kernel", stream);
    cudaError_t e = launch_kernel(kern, dim3((unsigned)((tiles < slots ? tiles : slots) * CTAS)),
                                  dim3(B_GATHER ? kThreadsTc + 32 * kGatherWarps : (a.epi_sets == 2 ? kThreadsTc2 : kThreadsTc)), L::kTotal, stream,
                                  CTAS, ma, mb, my, a);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "reduced_gemm_tc_kernel: launch: %s", cudaGetErrorString(e));
    return check_launch("reduced_gemm_tc_kernel", stream);
}

}  // namespace

bool tc_eligible(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y, TcPlan *plan, bool with_energy)
{
    if (A->dtype != RMM_BF16 || B->dtype != RMM_BF16) return false;
    const int64_t M = A->rows, K = A->cols, N = B->cols, batch = A->batch;
    auto al16 = [](const void *p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; };
    if (A->stride_col != 1) return false;
    if (Y->stride_col != 1 || !al16(Y->ptr)) return false;
    const int64_t yq = Y->dtype == RMM_BF16 ? 8 : 4;
    if (Y->stride_row % yq != 0 || Y->stride_batch % yq != 0) return false;
    if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX || batch > 65535) return false;
    int b_kmajor;
    if (B->stride_col == 1) {
        // rows of B (contraction slices) contiguous: row copies of 16-byte vectors
        b_kmajor = 0;
        if (!al16(B->ptr) || B->stride_row % 8 != 0 || B->stride_batch % 8 != 0 || N % 8 != 0) return false;
    } else if (B->stride_row == 1) {
        b_kmajor = 1;  // K-contiguous: packed like A
    } else {
        return false;
    }
    if (plan != nullptr) {
        plan->b_kmajor = b_kmajor;
        plan->ldp = (k + 7) / 8 * 8;
        size_t off = RMM_WS_HEADER_BYTES;
        plan->off_ap = off;
        off += align_up((size_t)batch * M * plan->ldp * 2, 256);
        plan->off_bp = off;
        off += align_up(b_kmajor ? (size_t)batch * N * plan->ldp * 2 : (size_t)batch * k * N * 2, 256);
        // column energies from the epilogue: bf16 output with an even number of columns (the pairs are stored as float2)
        plan->epilogue_energy = with_energy && Y->dtype == RMM_BF16 && N % 2 == 0;
        plan->off_colen = off;
        if (plan->epilogue_energy) off += align_up((size_t)batch * ceil_div(M, 32) * N * 4, 256);
        plan->total_bytes = off;
    }
    return true;
}

int launch_gemm_tc_problem(const TcProblem &p, cudaStream_t stream)
{
    CUtensorMap ma, mb;
    int rc;
    const int es = p.fp8 ? 1 : 2;             // bytes per operand element
    const uint32_t bke = p.fp8 ? 2 * BK : BK;  // contraction indices per 128-byte stage row
    if (p.fp8 && (!p.b_kmajor || p.b_idx != nullptr))
        return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm_tc: 8-bit operands must both be K-major and packed");
    {
        uint64_t dims[3] = {(uint64_t)p.k, (uint64_t)p.M, (uint64_t)p.batch};
        uint64_t st[2] = {(uint64_t)p.a_ld * es, (uint64_t)p.a_sb * es};
        uint32_t box[3] = {bke, BM, 1};
        rc = make_map(&ma, const_cast<__nv_bfloat16 *>(p.a), 3, dims, st, box, true, es);
        if (rc != RMM_OK) return rc;
    }
    const int BN = p.N <= 128 ? 128 : 256;
    // CTA pairs (256 x 256 tiles, a third fewer operand bytes per flop) pay off once there are enough pair tiles to
    // keep every SM pair busy: measured 1.81-1.87 PFLOP/s against 1.51-1.59 for single CTAs on 8192 x 8192 outputs,
    // while on a 2048 x 2048 output (64 pair tiles for 74 SM pairs) the pair's longer set-up and epilogue lose about
    // 2 us.  RMM_GEMM_CTAS=1 or 2 forces a form (for measurements).
    static const int forced = []() { const char *e = getenv("RMM_GEMM_CTAS"); return e ? atoi(e) : 0; }();
    const int64_t pair_tiles = p.batch * ceil_div(p.M, 2 * BM) * ceil_div(p.N, 256);
    int ctas = (BN == 256 && p.M > BM && pair_tiles >= sm_count() / 2) ? 2 : 1;
    if (forced == 1) ctas = 1;
    if (forced == 2 && BN == 256 && p.M > BM) ctas = 2;
    if (p.b_idx != nullptr) ctas = 1;  // the in-kernel row gather exists for single-CTA tiles
    TcArgs a;
    a.M = p.M; a.N = p.N; a.k = p.k; a.batch = p.batch;
    a.b_batch_off = p.b_batch_off; a.b_batch_div = p.b_batch_div > 0 ? p.b_batch_div : 1; a.b_batches = p.b_batches;
    a.Y = p.y; a.y_sb = p.y_sb; a.y_sr = p.y_sr;
    a.scale = p.scale;
    a.tiles_m = (int)ceil_div(p.M, BM * ctas);
    a.tiles_n = (int)ceil_div(p.N, BN);
    a.status = p.status;
    {
        // column slices of B kept alive by one raster group: group * BN columns x k rows of bf16, held to about 64 MB (half of
        // L2) so that they survive from one wave to the next; where not even eight slices fit, eight all the same: a wave
        // of 74 tiles then reads the fewest bytes when it is about as wide as it is tall
        static const int forced_raster = []() { const char *e = getenv("RMM_GEMM_RASTER"); return e ? atoi(e) : 0; }();
        const int64_t slice = (int64_t)BN * p.k * es;
        int64_t grp = slice > 0 ? (64ll << 20) / slice : kRasterGroupMax;
        if (grp > kRasterGroupMax) grp = kRasterGroupMax;
        if (grp < 8) grp = 8;
        a.raster = forced_raster > 0 ? forced_raster : (int)grp;
    }
    a.wait_ns = wait_limit_ns();
    a.withhold = debug_withhold() == WITHHOLD_GEMM;
    {
        // wave synchronisation: products with several waves of long tiles (measurement switch RMM_GEMM_WAVE_SYNC=0|1)
        static const int forced_sync = []() { const char *e = getenv("RMM_GEMM_WAVE_SYNC"); return e ? atoi(e) : -1; }();
        const int64_t tiles = (int64_t)a.batch * a.tiles_m * a.tiles_n, per_wave = sm_count() / ctas;
        const bool want = forced_sync >= 0 ? forced_sync != 0 : (tiles > per_wave && p.k * es >= 8192);
        static const int sync_kb = []() { const char *e = getenv("RMM_GEMM_SYNC_KB"); return e ? atoi(e) : 128; }();
        a.sync_kb = sync_kb;
        a.wave_ctr = (want && p.status != nullptr)
                         ? &reinterpret_cast<WsHeader *>(reinterpret_cast<char *>(p.status) - offsetof(WsHeader, status))->counters[kHeaderCounters - 4]
                         : nullptr;
    }
    a.col_energy = p.col_energy;
    a.row_scale = p.row_scale;
    // products with at most four k-blocks per tile are bound by the epilogue, and a block with a single tile has no next
    // main loop to hide its epilogue behind: two sets of epilogue warps in both cases
    const int64_t n_tiles = p.batch * ceil_div(p.M, BM * ctas) * ceil_div(p.N, BN);
    a.epi_sets = (p.y_bf16 && p.b_idx == nullptr && (ceil_div(p.k, (int64_t)bke) <= 4 || n_tiles <= sm_count() / ctas)) ? 2 : 1;
    a.b_src = p.b; a.b_idx = p.b_idx; a.b_ld = p.b_ld; a.b_sb = p.b_batches > 1 ? p.b_sb : 0; a.b_idx_stride = p.b_idx_stride;
    a.b_rows = p.b_rows;
    if (p.b_idx != nullptr) {
        if (p.b_kmajor || ctas != 1 || BN != 256)
            return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm_tc: in-kernel row gather needs single-CTA 128 x 256 tiles and row-contiguous B");
        CUtensorMap my_g = ma;  // (the tensor map of B is unused in this form; A's stands in)
        if (p.y_bf16) {
            uint64_t dims[3] = {(uint64_t)p.N, (uint64_t)p.M, (uint64_t)p.batch};
            uint64_t st[2] = {(uint64_t)p.y_sr * 2, p.batch > 1 ? (uint64_t)p.y_sb * 2 : (uint64_t)p.y_sr * 2 * (uint64_t)p.M};
            uint32_t box[3] = {64, 32, 1};
            rc = make_map(&my_g, p.y, 3, dims, st, box, true);
            if (rc != RMM_OK) return rc;
            return launch_variant<256, false, true, 1, true>(ma, ma, my_g, a, stream);
        }
        return launch_variant<256, false, false, 1, true>(ma, ma, my_g, a, stream);
    }
    const uint64_t b_sb = p.b_batches > 1 ? (uint64_t)p.b_sb * es : (uint64_t)p.b_ld * es * (uint64_t)(p.b_kmajor ? p.N : p.k);
    if (p.b_kmajor) {
        uint64_t dims[3] = {(uint64_t)p.k, (uint64_t)p.N, (uint64_t)p.b_batches};
        uint64_t st[2] = {(uint64_t)p.b_ld * es, b_sb};
        uint32_t box[3] = {bke, (uint32_t)(BN / ctas), 1};
        rc = make_map(&mb, const_cast<__nv_bfloat16 *>(p.b), 3, dims, st, box, true, es);
    } else {
        uint64_t dims[3] = {(uint64_t)p.N, (uint64_t)p.k, (uint64_t)p.b_batches};
        uint64_t st[2] = {(uint64_t)p.b_ld * 2, b_sb};
        uint32_t box[3] = {64, BK, 1};
        rc = make_map(&mb, const_cast<__nv_bfloat16 *>(p.b), 3, dims, st, box, true);
    }
    if (rc != RMM_OK) return rc;
    const bool out_bf16 = p.y_bf16 != 0;
    CUtensorMap my = ma;  // fp32 output is stored without a tensor map
    if (out_bf16) {
        // per-warp store slabs: 64 columns x 32 rows; rows and columns past M and N are clipped by the map
        uint64_t dims[3] = {(uint64_t)p.N, (uint64_t)p.M, (uint64_t)p.batch};
        uint64_t st[2] = {(uint64_t)p.y_sr * 2, p.batch > 1 ? (uint64_t)p.y_sb * 2 : (uint64_t)p.y_sr * 2 * (uint64_t)p.M};
        uint32_t box[3] = {64, 32, 1};
        rc = make_map(&my, p.y, 3, dims, st, box, true);
        if (rc != RMM_OK) return rc;
    }
    if (p.fp8) {
        if (ctas == 2) return out_bf16 ? launch_variant<256, true, true, 2, false, true>(ma, mb, my, a, stream) : launch_variant<256, true, false, 2, false, true>(ma, mb, my, a, stream);
        if (BN == 256) return out_bf16 ? launch_variant<256, true, true, 1, false, true>(ma, mb, my, a, stream) : launch_variant<256, true, false, 1, false, true>(ma, mb, my, a, stream);
        return out_bf16 ? launch_variant<128, true, true, 1, false, true>(ma, mb, my, a, stream) : launch_variant<128, true, false, 1, false, true>(ma, mb, my, a, stream);
    }
    if (ctas == 2) {
        if (p.b_kmajor) return out_bf16 ? launch_variant<256, true, true, 2>(ma, mb, my, a, stream) : launch_variant<256, true, false, 2>(ma, mb, my, a, stream);
        return out_bf16 ? launch_variant<256, false, true, 2>(ma, mb, my, a, stream) : launch_variant<256, false, false, 2>(ma, mb, my, a, stream);
    }
    if (BN == 256) {
        if (p.b_kmajor) return out_bf16 ? launch_variant<256, true, true, 1>(ma, mb, my, a, stream) : launch_variant<256, true, false, 1>(ma, mb, my, a, stream);
        return out_bf16 ? launch_variant<256, false, true, 1>(ma, mb, my, a, stream) : launch_variant<256, false, false, 1>(ma, mb, my, a, stream);
    }
    if (p.b_kmajor) return out_bf16 ? launch_variant<128, true, true, 1>(ma, mb, my, a, stream) : launch_variant<128, true, false, 1>(ma, mb, my, a, stream);
    return out_bf16 ? launch_variant<128, false, true, 1>(ma, mb, my, a, stream) : launch_variant<128, false, false, 1>(ma, mb, my, a, stream);
}

int launch_gemm_tc(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                   const rmm_mat_t *Y, const TcPlan &plan, void *ws, cudaStream_t stream, float *energy_out)
{
    if (energy_out != nullptr && plan.epilogue_energy) {
        // the product writes per-group column energies, a small kernel adds the groups up
        int rc0 = launch_gemm_tc(A, B, idx, k, scale, Y, plan, ws, stream, nullptr);
        if (rc0 != RMM_OK) return rc0;
        return launch_energy_combine(reinterpret_cast<const float *>(static_cast<char *>(ws) + plan.off_colen), A->batch,
                                     ceil_div(A->rows, 32), B->cols, energy_out, stream);
    }
    char *w = static_cast<char *>(ws);
    int *status = &reinterpret_cast<WsHeader *>(w)->status;
    const int64_t M = A->rows, K = A->cols, N = B->cols, batch = A->batch;
    const __nv_bfloat16 *a_src = static_cast<const __nv_bfloat16 *>(A->ptr), *b_src = static_cast<const __nv_bfloat16 *>(B->ptr);
    __nv_bfloat16 *Ap = reinterpret_cast<__nv_bfloat16 *>(w + plan.off_ap), *Bp = reinterpret_cast<__nv_bfloat16 *>(w + plan.off_bp);
    int rc;
    TcProblem p = {};
    p.batch = batch; p.M = M; p.N = N; p.k = k;
    p.b_kmajor = plan.b_kmajor;
    p.y = Y->ptr; p.y_bf16 = Y->dtype == RMM_BF16; p.y_sb = Y->stride_batch; p.y_sr = Y->stride_row;
    p.scale = scale; p.status = status;
    p.col_energy = plan.epilogue_energy ? reinterpret_cast<float *>(w + plan.off_colen) : nullptr;
    p.b_batch_off = 0; p.b_batch_div = 1; p.b_batches = batch;

    // the unreduced product (idx NULL, k == K) on TMA-loadable operands needs no gather at all
    const bool in_place = idx == nullptr && !plan.b_kmajor && reinterpret_cast<uintptr_t>(A->ptr) % 16 == 0 &&
                          A->stride_row % 8 == 0 && A->stride_batch % 8 == 0;
    if (in_place) {
        p.a = a_src; p.a_ld = A->stride_row; p.a_sb = batch > 1 ? A->stride_batch : M * A->stride_row;
        p.b = b_src; p.b_ld = B->stride_row;
        if (B->stride_batch == 0) { p.b_batches = 1; p.b_sb = 0; }
        else { p.b_sb = B->stride_batch; }
        return launch_gemm_tc_problem(p, stream);
    }
    // A[:, I] and the kept slices of B are gathered by one launch
    PackSpec specs[2];
    specs[0] = pack_cols_spec(a_src, batch, M, K, A->stride_batch, A->stride_row, 0, 1, idx, k, k, Ap, plan.ldp);
    p.a = Ap; p.a_ld = plan.ldp; p.a_sb = M * plan.ldp;
    if (!plan.b_kmajor && M <= 2 * BM && N > 128) {
        // one or two tile rows: a tile of B is used once or twice (the second time from L2), so the kernel fetches the
        // kept rows itself and only A[:, I] is packed
        p.b = b_src; p.b_ld = B->stride_row; p.b_rows = K;
        if (B->stride_batch == 0) { p.b_batches = 1; p.b_sb = 0; }
        else { p.b_sb = B->stride_batch; }
        p.b_idx = idx; p.b_idx_stride = k;
        rc = launch_pack(specs, 1, status, stream);
        if (rc != RMM_OK) return rc;
        return launch_gemm_tc_problem(p, stream);
    }
    if (plan.b_kmajor) {
        // B is K-contiguous ([N, K] in memory): B[idx, :]^T goes to Bp [batch, N, ldp]; a shared B (stride_batch 0)
        // is packed once per index set
        specs[1] = pack_cols_spec(b_src, batch, N, K, B->stride_batch, B->stride_col, 0, 1, idx, k, k, Bp, plan.ldp);
        p.b = Bp; p.b_ld = plan.ldp; p.b_sb = N * plan.ldp;
    } else {
        specs[1] = pack_rows_spec(b_src, batch, K, N, B->stride_batch, B->stride_row, 0, 1, idx, k, k, Bp, N);
        p.b = Bp; p.b_ld = N; p.b_sb = k * N;
    }
    rc = launch_pack(specs, 2, status, stream);
    if (rc != RMM_OK) return rc;
    return launch_gemm_tc_problem(p, stream);
}

}  // namespace rmm

#ifdef RMM_GEMM_STAMPS
// Debug build only: copy the GEMM kernel's phase stamps (nanoseconds of %globaltimer; slot 0 the first block's start, a
// minimum; 1 set-up done, 2 first tensor-core instruction, 3 last main loop issued, 4 last accumulator complete, 5 last
// epilogue done, 6 last thread out: maxima over blocks) to out[0 .. 15] and re-arm them.
extern "C" int rmm_debug_gemm_stamps(unsigned long long *out)
{
    unsigned long long init[16];
    cudaError_t e = cudaMemcpyFromSymbol(out, rmm::g_gstamps, sizeof init);
    for (int i = 0; i < 16; ++i) init[i] = 0;
    init[0] = ~0ull;
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(rmm::g_gstamps, init, sizeof init);
    return e == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}
#endif
