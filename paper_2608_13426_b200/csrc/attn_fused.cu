// Fused reduced attention (paper Sec. 3.3): S~ = Q[:, I] K[:, I]^T / sqrt(Dh) on packed operands, softmax, and the
// product with V, with S~ and P never leaving the SM (S~ tiles in tensor memory, P tiles in shared memory, O
// accumulated in tensor memory).  One kernel skeleton, four modes:
//
//   FULL      rho_t = 1:  O = softmax(S~ + mask) V in one pass over the keys.
//   STATS     rho_t < 1, sweep 1:  lse_i = log2 sum_t 2^(x_it) per query row (x = S~ * log2(e) / sqrt(Dh)), nothing else.
//   ENERGY    rho_t < 1, sweep 2:  token scores a_t^2 = sum_i P_it^2 with P_it = bf16(2^(x_it - lse_i)), the attention
//             weight rounded once to bf16 as the paper scores it.  The roles are swapped (rows = keys, tiles of
//             queries stream past), so that a thread owns one key and sums over all queries in a register: no
//             cross-thread reduction and no atomics.
//   GATHERED  rho_t < 1, sweep 3:  O = P[:, T] V[T, :] on the kept keys (K[T], V[T] packed), P_it = bf16(2^(x_it -
//             lse_i)) against the full-row normaliser of sweep 1: no renormalisation (Sec. 3.3).
//
// One block owns 256 rows of one head as two groups of 128 and walks the other axis in tiles of 128; both groups
// consume the same tiles, so each crosses from L2 to the SM once per 256 rows.  Per tile and group: S~ on the tensor
// cores (kd of the Dh features; 128 columns of tensor memory, released as soon as the softmax warps hold the tile in
// registers); one thread per row takes p = 2^(x - m) in two chunks of 64 columns, rounds it once to bf16 and writes it
// to shared memory as the A operand of O += P V.  In FULL mode m is the row maximum seen so far, refreshed only when
// the new maximum exceeds it by more than 40 (p up to 2^40 and row sums up to 2^71 are far from the bf16 and fp32
// range limits, and floating point keeps the same relative precision at any scale): then l and the O row in tensor
// memory are multiplied by 2^(m_old - m_new); the epilogue divides by l.  The paper rounds the normalised weight P
// to bf16; in FULL mode the rounded quantity is p = P * l * 2^(m_row - m), the same weight up to a per-row fp32
// factor, so O differs by bf16 rounding noise only (nothing is decided from P when rho_t = 1); the modes that score or
// drop tokens round the normalised P itself.
// Warp 0 feeds TMA, warps 2-5 and 6-9 are the softmax/epilogue warps of the two groups (every scheduler has two of
// them to switch between), and one thread of warp 1 and of warp 10 issues the tcgen05.mma of group 0 and 1: a single
// issuing thread for both groups was the bottleneck.  Every wait is bounded.
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace rmm {
namespace {

using namespace ptx;

enum { MODE_FULL = 0, MODE_STATS = 1, MODE_ENERGY = 2, MODE_GATHERED = 3 };

constexpr int FM = 128, FN = 128;     // rows per group, columns per step
constexpr int kGroups = 2;
constexpr int kFusedThreads = 64 + kGroups * 128 + 32;  // producer, MMA issuer 0, 8 softmax warps, MMA issuer 1
constexpr int kMmaWarp1 = 10;
constexpr int kKvStages = 3;
constexpr int kQChunk = 16384;        // row-side chunk: 128 rows x 64 features (128 bytes per row, 128-byte swizzle)
constexpr int kQTile = 2 * kQChunk;   // up to 128 kept features
constexpr int kKvChunk = 16384;       // column-side chunk: 128 keys x 64 features (or 128 keys x 64 columns of V)
constexpr int kKvTile = 2 * kKvChunk; // ring entry: a K tile (up to 128 kept features) or a V tile (up to 128 columns)
constexpr int kPChunk = 16384;        // P chunk: 128 rows x 64 keys (128 bytes per row, 128-byte swizzle)
constexpr int kPTile = 2 * kPChunk;   // P tile: 128 rows x 128 keys
constexpr int kOffQ = 0, kOffKv = kGroups * kQTile, kOffP = kOffKv + kKvStages * kKvTile, kOffBar = kOffP + kGroups * kPTile;
constexpr int kFusedSmem = kOffBar + 512;
constexpr int kTmemCols = 512;        // per group: S~ (128 columns); then O (128 columns per group)
constexpr uint32_t kTmemO = kGroups * FN;
constexpr float kGrowLimit = 40.f;    // log2 of the largest p taken against a stale maximum

// Debug aid (-DRMM_ATTN_STAMPS): clocks spent per phase by the MMA issuer of group 0 and by one softmax warp of
// block 0, summed over the launch and read back with rmm_debug_attn_stamps().
#ifdef RMM_ATTN_STAMPS
__device__ unsigned long long g_astamps[16];
#define ASTAMP_DECL(cond) long long acc_[8] = {0, 0, 0, 0, 0, 0, 0, 0}, last_ = clock64(); const bool stamp_on = (cond)
#define ASTAMP(i) do { long long t_ = clock64(); acc_[i] += t_ - last_; last_ = t_; } while (0)
#define ASTAMP_FLUSH(off) do { if (stamp_on) for (int k_ = 0; k_ < 8; ++k_) atomicAdd(&g_astamps[(off) + k_], (unsigned long long)acc_[k_]); } while (0)
#else
#define ASTAMP_DECL(cond)
#define ASTAMP(i)
#define ASTAMP_FLUSH(off)
#endif

// "Rows" are what a thread owns (queries; keys in ENERGY mode), "columns" what streams past in tiles.
struct FusedArgs {
    int64_t heads, Lr, Lc;       // rows and columns per head (GATHERED: Lc = kept keys)
    int64_t diag;                // Lk - Lq of the unpacked problem: query i sees key t iff t <= i + diag (causal)
    int kd, Dh, causal;
    int64_t v_off, v_div;        // V batch entry of head h = (h + v_off) / v_div
    __nv_bfloat16 *O;
    int64_t o_sh, o_sr;          // element strides of O: head, row
    float *lse;                  // [heads, lse_ld] log2-domain normalisers: written by STATS, read by ENERGY / GATHERED
    int64_t lse_ld;              // multiple of 64, >= Lq
    float *energy;               // ENERGY: [heads, Lr] squared token scores
    const int32_t *tok;          // GATHERED: [heads, Lc] kept key positions, ascending
    float scale_log2;            // (1 / sqrt(Dh)) * log2(e)
    const float *mask;           // MASK: additive mask M of softmax(S~ + M), fp32, row (head, i) at mask + head m_sh + i m_sr
    int64_t m_sh, m_sr;
    float mask_gain;             // sqrt(Dh): M is added to the unscaled S~ tile as M * sqrt(Dh)
    int *status;
    unsigned long long wait_ns;  // bound of every device-side wait
    int withhold;                // test switch: block 0 never requests its first key tile
};

template <int MODE, bool MASK>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_attn_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, FusedArgs a)
{
    constexpr bool kHasV = MODE == MODE_FULL || MODE == MODE_GATHERED;  // P tiles, P V products and an O accumulator
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    uint8_t *base_ptr = smem_raw;
    if (base & 1023u) {  // the swizzled tiles need a 1024-byte aligned window; nothing has been allocated yet
        if (threadIdx.x == 0) atomicExch(a.status, (int)RMM_ERR_CUDA);
        return;
    }
    const uint32_t bar0 = base + kOffBar;
    // barriers: q_full, q_empty; per group s_full[2], s_empty[2], p_full, p_empty, o_full, o_empty; kv_full[], kv_empty[]
    const uint32_t q_full = bar0, q_empty = bar0 + 8;
    auto s_full = [&](int g, int i) { return bar0 + 64u * (g + 1) + 8u * i; };
    auto s_empty = [&](int g, int i) { return bar0 + 64u * (g + 1) + 16u + 8u * i; };
    auto p_full = [&](int g) { return bar0 + 64u * (g + 1) + 32u; };
    auto p_empty = [&](int g) { return bar0 + 64u * (g + 1) + 40u; };
    auto o_full = [&](int g) { return bar0 + 64u * (g + 1) + 48u; };
    auto o_empty = [&](int g) { return bar0 + 64u * (g + 1) + 56u; };
    auto kv_full = [&](int s) { return bar0 + 256u + 8u * s; };
    auto kv_empty = [&](int s) { return bar0 + 256u + 8u * (kKvStages + s); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + kOffBar + 16);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + kOffBar + 24);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        if constexpr (kHasV) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(q_empty, kGroups);
        for (int s = 0; s < kKvStages; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), kGroups); }
        for (int g = 0; g < kGroups; ++g) {
            for (int i = 0; i < 2; ++i) { mbar_init(s_full(g, i), 1); mbar_init(s_empty(g, i), 4); }
            mbar_init(p_full(g), 4);
            mbar_init(p_empty(g), 1);
            mbar_init(o_full(g), 1);
            mbar_init(o_empty(g), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<1>(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    const int kq = (a.kd + 63) / 64, nv = (a.Dh + 63) / 64;       // 64-column chunks of Q/K and of V
    const int blocks_r = (int)((a.Lr + kGroups * FM - 1) / (kGroups * FM));
    const int64_t items = a.heads * blocks_r;
    // kept keys (GATHERED) with position <= limit: T is ascending
    auto kept_upto = [&](const int32_t *T, int64_t limit) -> int64_t {
        int64_t lo = 0, hi = a.Lc;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if ((int64_t)__ldg(T + mid) <= limit) lo = mid + 1; else hi = mid;
        }
        return lo;
    };
    // Column tiles [jb, je) that the 128 rows starting at r0 need (empty: jb = je = 0).
    auto tile_range = [&](int64_t head, int64_t r0, int *jb, int *je) {
        *jb = 0;
        *je = 0;
        if (r0 >= a.Lr) return;
        if constexpr (MODE == MODE_ENERGY) {
            // row = key t, visible to the queries i >= t - diag: the group's first row reaches furthest back
            const int64_t first = a.causal ? max((int64_t)0, r0 - a.diag) : 0;
            if (first >= a.Lc) return;
            *jb = (int)(first / FN);
            *je = (int)((a.Lc + FN - 1) / FN);
        } else if constexpr (MODE == MODE_GATHERED) {
            const int64_t n = a.causal ? kept_upto(a.tok + head * a.Lc, min(a.Lr - 1, r0 + FM - 1) + a.diag) : a.Lc;
            *je = (int)((n + FN - 1) / FN);
        } else {
            const int64_t last = a.causal ? min(a.Lc - 1, r0 + FM - 1 + a.diag) : a.Lc - 1;
            *je = last < 0 ? 0 : (int)(last / FN) + 1;
        }
    };
    // Tiles the block walks: the union over its groups (a group's range is a prefix or a suffix of it).
    auto block_range = [&](int64_t head, int64_t r0, int *jb, int *je) {
        int b0, e0, b1, e1;
        tile_range(head, r0, &b0, &e0);
        tile_range(head, r0 + FM, &b1, &e1);
        if (e0 <= b0) { *jb = b1; *je = e1; }
        else if (e1 <= b1) { *jb = b0; *je = e0; }
        else { *jb = min(b0, b1); *je = max(e0, e1); }
    };
    // The n-th item of this block: heaviest row blocks first (the last ones when causal; in ENERGY mode, where early
    // keys are seen by most queries, the first ones), and the direction alternates from round to round, so that the
    // block that drew the heaviest item of one round draws the lightest of the next.
    auto item_of = [&](int64_t n, int64_t *head, int64_t *r0) -> bool {
        const int64_t b = (n & 1) ? (int64_t)gridDim.x - 1 - blockIdx.x : blockIdx.x;
        const int64_t item = n * gridDim.x + b;
        if (item >= items) return false;
        *head = item % a.heads;
        const int64_t rb = item / a.heads;
        *r0 = (MODE == MODE_ENERGY ? rb : blocks_r - 1 - rb) * (kGroups * FM);
        return true;
    };
    const int64_t rounds = (items + gridDim.x - 1) / gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer: Q, then K_0, K_1, V_0, K_2, V_1, ...
        uint32_t ks = 0, kph = 0, n_item = 0;
        bool ok = true, first_load = true;
        auto load_kv = [&](const CUtensorMap *map, int chunks, int64_t row, int z) -> bool {
            if (!mbar_wait_sleepy(kv_empty(ks), kph ^ 1u, abort_flag, a.status, a.wait_ns)) return false;
            const uint32_t dst = base + kOffKv + ks * kKvTile;
            if (a.withhold && blockIdx.x == 0 && first_load) {
                first_load = false;  // (test switch) this tile is never requested: its barrier stays incomplete
            } else {
                mbar_arrive_expect_tx(kv_full(ks), (uint32_t)chunks * kKvChunk);
                for (int c = 0; c < chunks; ++c) tma_load_3d(dst + c * kKvChunk, map, c * 64, (int)row, z, kv_full(ks));
            }
            if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
            return true;
        };
        for (int64_t n = 0; lane == 0 && n < rounds && ok; ++n) {
            int64_t head, r0;
            if (!item_of(n, &head, &r0)) continue;
            int jb, je;
            block_range(head, r0, &jb, &je);
            if (je <= jb) continue;
            const int vb = (int)((head + a.v_off) / a.v_div);
            if (!mbar_wait_sleepy(q_empty, (n_item & 1u) ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
            mbar_arrive_expect_tx(q_full, (uint32_t)(kGroups * kq) * kQChunk);
            for (int g = 0; g < kGroups; ++g)
                for (int c = 0; c < kq; ++c)
                    tma_load_3d(base + kOffQ + g * kQTile + c * kQChunk, &map_q, c * 64, (int)(r0 + g * FM), (int)head, q_full);
            ok = load_kv(&map_k, kq, (int64_t)jb * FN, (int)head);
            for (int j = jb; j < je && ok; ++j) {
                if (j + 1 < je) ok = load_kv(&map_k, kq, (int64_t)(j + 1) * FN, (int)head);
                if constexpr (kHasV) {
                    if (ok) ok = load_kv(&map_v, nv, (int64_t)j * FN, vb);
                }
            }
            ++n_item;  // counts the items that reach the tensor cores (those with at least one tile)
        }
        __syncwarp();
    } else if (warp == 1 || warp == kMmaWarp1) {
        // ------------------------------------------------------------------ MMA issuer of group g (one thread)
        // Both issuers walk the same ring entries; each uses the tiles its group needs and releases every entry (a
        // commit arrives once this thread's earlier MMAs are done, at once if there are none).
        const int g = warp == 1 ? 0 : 1;
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(FN >> 3) << 17) | ((uint32_t)(FM >> 4) << 24);
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)((nv * 64) >> 3) << 17) |
                                 ((uint32_t)(FM >> 4) << 24);
        const uint64_t dq0 = smem_desc(base + kOffQ + g * kQTile, 16, 1024), dk0 = smem_desc(base + kOffKv, 16, 1024);
        const uint64_t dp0 = smem_desc(base + kOffP + g * kPTile, 16, 1024), dv0 = smem_desc(base + kOffKv, kKvChunk, 1024);
        const uint32_t q_hi = (uint32_t)(dq0 >> 32), k_hi = (uint32_t)(dk0 >> 32), p_hi = (uint32_t)(dp0 >> 32), v_hi = (uint32_t)(dv0 >> 32);
        const uint32_t q_lo = (uint32_t)dq0, k_lo = (uint32_t)dk0, p_lo = (uint32_t)dp0, v_lo = (uint32_t)dv0;
        const int steps_s = (a.kd + 15) / 16;
        const uint32_t t_s = tmem_base + g * FN, t_o = tmem_base + kTmemO + g * 128;
        uint32_t ks = 0, kph = 0, n_item = 0, s_it = 0, p_it = 0, o_it = 0;
        bool ok = true;
        int gb = 0, ge = 0;  // this group's tile range in the current item
        ASTAMP_DECL(blockIdx.x == 0 && lane == 0 && g == 0);
        auto step_s = [&](int j) -> bool {  // S~ of tile j (if this group needs it); consumes one ring entry
            ASTAMP(7);
            if (!mbar_wait(kv_full(ks), kph, abort_flag, a.status, a.wait_ns)) return false;
            ASTAMP(0);
            if (j >= gb && j < ge) {
                // S~ is single-buffered: the softmax warps release it as soon as they hold the tile in registers
                if (!mbar_wait(s_empty(g, 0), (s_it & 1u) ^ 1u, abort_flag, a.status, a.wait_ns)) return false;
                ASTAMP(1);
                tc_fence_after();
                uint32_t ql = q_lo, kl = k_lo + ks * (kKvTile >> 4), acc = 0;
                if (elect_one()) {
                    for (int left = steps_s; left > 0; left -= 4, ql += kQChunk >> 4, kl += kKvChunk >> 4) {  // 64-feature chunks
                        const int ns = left < 4 ? left : 4;
                        for (int st = 0; st < ns; ++st, acc = 1u)  // 16 features = 32 bytes per step
                            umma_bf16_lohi<1>(t_s, ql + 2 * st, q_hi, kl + 2 * st, k_hi, idesc_s, acc);
                    }
                    umma_commit<1>(s_full(g, 0));
                }
                ++s_it;
            }
            if (elect_one()) umma_commit<1>(kv_empty(ks));
            __syncwarp();
            if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
            ASTAMP(2);
            return true;
        };
        for (int64_t n = 0; n < rounds && ok; ++n) {
            int64_t head, r0;
            if (!item_of(n, &head, &r0)) continue;
            int jb, je;
            block_range(head, r0, &jb, &je);
            if (je <= jb) continue;
            tile_range(head, r0 + g * FM, &gb, &ge);
            if (!mbar_wait(q_full, n_item & 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
            ok = step_s(jb);
            for (int j = jb; j < je && ok; ++j) {
                if (j + 1 < je) ok = step_s(j + 1);                        // S~ of the next tile runs ahead of this P V
                if (!ok) break;
                if constexpr (kHasV) {
                    ASTAMP(7);
                    if (!mbar_wait(kv_full(ks), kph, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                    ASTAMP(3);
                    if (j >= gb && j < ge) {
                        if (j == gb && !mbar_wait(o_empty(g), (o_it & 1u) ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                        ASTAMP(4);
                        if (!mbar_wait(p_full(g), p_it & 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                        ASTAMP(5);
                        tc_fence_after();
                        const uint32_t vl = v_lo + ks * (kKvTile >> 4);
                        if (elect_one()) {
#pragma unroll
                            for (int st = 0; st < FN / 16; ++st)  // P: K-major, 64-key chunks, 32 bytes per step; V: MN-major (rows = keys), 16 keys = 2048 bytes
                                umma_bf16_lohi<1>(t_o, p_lo + (st >> 2) * (kPChunk >> 4) + (st & 3) * 2, p_hi, vl + st * (2048 >> 4), v_hi, idesc_o,
                                                  (j != gb || st != 0) ? 1u : 0u);
                            umma_commit<1>(p_empty(g));   // "P V of this tile is complete": P may be rewritten, O may be rescaled
                            if (j == ge - 1) umma_commit<1>(o_full(g));
                        }
                        ++p_it;
                        if (j == ge - 1) ++o_it;
                    }
                    if (elect_one()) umma_commit<1>(kv_empty(ks));
                    __syncwarp();
                    if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
                    ASTAMP(6);
                }
            }
            if (ok && elect_one()) umma_commit<1>(q_empty);
            __syncwarp();
            ++n_item;
        }
        ASTAMP_FLUSH(0);
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax and epilogue (one row per thread)
        // A step is 128 columns, taken as two chunks of 64 so that a thread never holds more than 64 logits.
        const int g = (warp - 2) >> 2, q = warp & 3, r = q * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t t_s = t_lane + g * FN, t_o = t_lane + kTmemO + g * 128;
        const float c2 = a.scale_log2;
        const uint64_t c22 = pack2(c2, c2);
        uint8_t *prow = base_ptr + kOffP + g * kPTile + r * 128;  // row r of each 64-key chunk: 128 bytes, 16-byte units swizzled
        uint32_t s_it = 0, p_it = 0, o_it = 0;
        bool ok = true;
        ASTAMP_DECL(blockIdx.x == 0 && warp == 2 && lane == 0);
        for (int64_t n = 0; n < rounds && ok; ++n) {
            int64_t head, r0;
            if (!item_of(n, &head, &r0)) continue;
            r0 += g * FM;
            if (r0 >= a.Lr) continue;                  // this group has no rows in the last block
            int jb, je;
            tile_range(head, r0, &jb, &je);
            const int64_t i = r0 + r;                  // this thread's row
            __nv_bfloat16 *orow = a.O + head * a.o_sh + i * a.o_sr;
            if (je <= jb) {  // nothing visible for any row of this group
                if constexpr (kHasV) {
                    if (i < a.Lr)
                        for (int c = 0; c < a.Dh; c += 8) *reinterpret_cast<uint4 *>(orow + c) = make_uint4(0, 0, 0, 0);
                } else if constexpr (MODE == MODE_STATS) {
                    if (i < a.lse_ld) a.lse[head * a.lse_ld + i] = INFINITY;  // 2^(x - inf) = 0 for every later use
                } else {
                    if (i < a.Lr) a.energy[head * a.Lr + i] = 0.f;
                }
                continue;
            }
            // columns this row sees: [first_col, last_col]
            int64_t first_col = 0, last_col = a.Lc - 1;
            if (a.causal) {
                if constexpr (MODE == MODE_ENERGY) first_col = max((int64_t)0, i - a.diag);
                else if constexpr (MODE == MODE_GATHERED) last_col = kept_upto(a.tok + head * a.Lc, i + a.diag) - 1;
                else last_col = min(a.Lc - 1, i + a.diag);
            }
            float m = -INFINITY, l = 0.f;  // FULL / STATS: the maximum that p is taken against (log2 domain), the row sum
            float row_lse = 0.f;           // GATHERED: this row's normaliser
            if constexpr (MODE == MODE_GATHERED) row_lse = i < a.lse_ld ? a.lse[head * a.lse_ld + i] : INFINITY;

            // 64 logits of the current tile (columns c_off .. c_off + 63) into registers; hidden columns become -inf on
            // boundary tiles (the diagonal and the ragged end)
            auto load_chunk = [&](int j, int c_off, uint32_t (&v0)[32], uint32_t (&v1)[32]) {
                tmem_ld32_issue(t_s + c_off, v0);
                tmem_ld32_issue(t_s + c_off + 32, v1);
                tmem_ld_wait();
                const int64_t c0 = (int64_t)j * FN + c_off;
                const int64_t rel_hi = last_col - c0, rel_lo = first_col - c0;
                const int hi = rel_hi > 63 ? 63 : (rel_hi < -1 ? -1 : (int)rel_hi);
                const int lo = rel_lo < 0 ? 0 : (rel_lo > 64 ? 64 : (int)rel_lo);
                if (!__all_sync(0xffffffffu, hi >= 63 && lo <= 0)) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        if (e > hi || e < lo) v0[e] = 0xff800000u;
                        if (e + 32 > hi || e + 32 < lo) v1[e] = 0xff800000u;
                    }
                }
                if constexpr (MASK) {
                    // the caller's additive mask for this row's 64 columns (-inf hides a key); rows past the end and
                    // columns past the last key read nothing
                    if (i < a.Lr) {
                        const float *mrow = a.mask + head * a.m_sh + i * a.m_sr + c0;
                        const float gain = a.mask_gain;
                        auto add4 = [&](uint32_t (&v)[32], int e, int col) {
                            float4 m4;
                            if (c0 + col + 3 < a.Lc) {
                                m4 = __ldg(reinterpret_cast<const float4 *>(mrow + col));
                            } else {
                                m4.x = c0 + col < a.Lc ? __ldg(mrow + col) : 0.f;
                                m4.y = c0 + col + 1 < a.Lc ? __ldg(mrow + col + 1) : 0.f;
                                m4.z = c0 + col + 2 < a.Lc ? __ldg(mrow + col + 2) : 0.f;
                                m4.w = 0.f;
                            }
                            v[e] = __float_as_uint(fmaf(m4.x, gain, __uint_as_float(v[e])));
                            v[e + 1] = __float_as_uint(fmaf(m4.y, gain, __uint_as_float(v[e + 1])));
                            v[e + 2] = __float_as_uint(fmaf(m4.z, gain, __uint_as_float(v[e + 2])));
                            v[e + 3] = __float_as_uint(fmaf(m4.w, gain, __uint_as_float(v[e + 3])));
                        };
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            add4(v0, e, e);
                            add4(v1, e, e + 32);
                        }
                    }
                }
            };
            auto release_s = [&]() {  // this warp holds what it needs of the S~ tile
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(g, 0));
            };
            auto max_chunk = [&](const uint32_t (&v0)[32], const uint32_t (&v1)[32]) -> float {
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    mx0 = fmax3(mx0, __uint_as_float(v0[e]), __uint_as_float(v0[e + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(v0[e + 2]), __uint_as_float(v0[e + 3]));
                    mx2 = fmax3(mx2, __uint_as_float(v1[e]), __uint_as_float(v1[e + 1]));
                    mx3 = fmax3(mx3, __uint_as_float(v1[e + 2]), __uint_as_float(v1[e + 3]));
                }
                return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            };
            // p = 2^(x - m) for 64 logits: row sum (unless GATHERED) and, with V, the bf16 values packed into w
            auto emit_chunk = [&](const uint32_t (&v0)[32], const uint32_t (&v1)[32], float neg_m, uint32_t (&w)[kHasV ? 32 : 1]) {
                const uint64_t nm2 = pack2(neg_m, neg_m);
                uint64_t sum_a = 0, sum_b = 0;
                auto half = [&](const uint32_t (&v)[32], int c) {
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float x0, x1;
                        unpack2(ffma2(pack2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), c22, nm2), x0, x1);
                        const float p0 = ex2(x0), p1 = ex2(x1);
                        if constexpr (MODE != MODE_GATHERED) (e & 2 ? sum_b : sum_a) = fadd2(e & 2 ? sum_b : sum_a, pack2(p0, p1));
                        if constexpr (kHasV) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                            w[(c + e) >> 1] = *reinterpret_cast<uint32_t *>(&h);
                        }
                    }
                };
                half(v0, 0);
                half(v1, 32);
                if constexpr (MODE != MODE_GATHERED) {
                    float s0, s1;
                    unpack2(fadd2(sum_a, sum_b), s0, s1);
                    l += s0 + s1;
                }
            };
            auto store_chunk = [&](int chunk, const uint32_t (&w)[kHasV ? 32 : 1]) {
                if constexpr (kHasV) {
#pragma unroll
                    for (int u = 0; u < 8; ++u)  // 16-byte units of 8 keys
                        *reinterpret_cast<uint4 *>(prow + chunk * kPChunk + ((u ^ (r & 7)) << 4)) =
                            make_uint4(w[4 * u], w[4 * u + 1], w[4 * u + 2], w[4 * u + 3]);
                }
            };
            // m and l follow a new chunk maximum (log2 domain); returns the factor the sums taken so far have to be scaled by
            auto follow_max = [&](float mc, bool *any_grow) -> float {
                const bool grow = mc > m + kGrowLimit;
                *any_grow = __any_sync(0xffffffffu, grow);
                const float alpha = (grow && m > -INFINITY) ? ex2(m - mc) : 1.f;
                l *= alpha;
                if (grow) m = mc;
                return alpha;
            };

            for (int j = jb; j < je; ++j, ++s_it) {
                if constexpr (MODE == MODE_ENERGY) {
                    // the 128 normalisers of the next tile (512 bytes, the same for every thread) are pulled into L1
                    // one step ahead; the first tile's are fetched cold
                    const int64_t nxt = (int64_t)(j + 1) * FN + lane * 32;
                    if (lane < 4 && j + 1 < je && nxt < a.lse_ld)
                        asm volatile("prefetch.global.L1 [%0];" ::"l"(a.lse + head * a.lse_ld + nxt));
                }
                ASTAMP(7);
                if (!mbar_wait(s_full(g, 0), s_it & 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                ASTAMP(0);
                tc_fence_after();
                uint32_t v0[32], v1[32];

                if constexpr (MODE == MODE_ENERGY) {
                    // p = bf16(2^(x - lse_i)); this key's score accumulates p^2 over the tile's 128 queries
                    float acc0 = 0.f, acc1 = 0.f;
                    for (int c_off = 0; c_off < FN; c_off += 64) {
                        float4 cl[16];  // the normalisers of these 64 queries (the same for every thread)
                        const float4 *lp = reinterpret_cast<const float4 *>(a.lse + head * a.lse_ld + (int64_t)j * FN + c_off);
#pragma unroll
                        for (int u = 0; u < 16; ++u) cl[u] = (int64_t)j * FN + c_off + 4 * u < a.lse_ld ? __ldg(lp + u) : make_float4(0.f, 0.f, 0.f, 0.f);
                        load_chunk(j, c_off, v0, v1);
                        if (c_off == 64) release_s();
                        auto fold = [&](const uint32_t (&v)[32], int c) {
#pragma unroll
                            for (int e = 0; e < 32; e += 4) {
                                const float4 ls = cl[(c + e) >> 2];
                                const float p0 = ex2(fmaf(__uint_as_float(v[e]), c2, -ls.x)), p1 = ex2(fmaf(__uint_as_float(v[e + 1]), c2, -ls.y));
                                const float p2 = ex2(fmaf(__uint_as_float(v[e + 2]), c2, -ls.z)), p3 = ex2(fmaf(__uint_as_float(v[e + 3]), c2, -ls.w));
                                const float2 ra = __bfloat1622float2(__floats2bfloat162_rn(p0, p1));
                                const float2 rb = __bfloat1622float2(__floats2bfloat162_rn(p2, p3));
                                acc0 = fmaf(ra.x, ra.x, acc0);
                                acc1 = fmaf(ra.y, ra.y, acc1);
                                acc0 = fmaf(rb.x, rb.x, acc0);
                                acc1 = fmaf(rb.y, rb.y, acc1);
                            }
                        };
                        fold(v0, 0);
                        fold(v1, 32);
                    }
                    l += acc0 + acc1;
                    continue;
                }

                if constexpr (MODE == MODE_STATS) {
                    // no P and no O: the two chunks are folded one after the other, each against its own maximum
                    for (int c_off = 0; c_off < FN; c_off += 64) {
                        load_chunk(j, c_off, v0, v1);
                        if (c_off == 64) release_s();
                        bool any_grow;
                        follow_max(max_chunk(v0, v1) * c2, &any_grow);
                        uint32_t w[1];
                        emit_chunk(v0, v1, m > -INFINITY ? -m : 0.f, w);
                    }
                    continue;
                }

                uint32_t w[kHasV ? 32 : 1];
                if constexpr (MODE == MODE_GATHERED) {
                    const float neg_m = -row_lse;   // +inf normaliser (row sees nothing): p = 0
                    load_chunk(j, 0, v0, v1);
                    emit_chunk(v0, v1, neg_m, w);
                    if (!mbar_wait(p_empty(g), (p_it & 1u) ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                    store_chunk(0, w);
                    load_chunk(j, 64, v0, v1);
                    release_s();
                    emit_chunk(v0, v1, neg_m, w);
                    store_chunk(1, w);
                } else {
                    // FULL: the maximum of all 128 logits decides about a rescale before any p is taken; the second
                    // chunk is still in registers then, the first is read from tensor memory once more
                    load_chunk(j, 0, v0, v1);
                    const float mx_a = max_chunk(v0, v1);
                    load_chunk(j, 64, v0, v1);
                    const float mc = fmaxf(mx_a, max_chunk(v0, v1)) * c2;
                    bool any_grow;
                    const float alpha = follow_max(mc, &any_grow);
                    if (any_grow && j > jb) {  // rows of O already hold sums taken against the old maximum
                        if (!mbar_wait(p_empty(g), (p_it & 1u) ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                        tc_fence_after();
                        for (int c = 0; c < nv * 64; c += 16) {
                            uint32_t o[16];
                            tmem_ld16_issue(t_o + c, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st16_issue(t_o + c, o);
                        }
                        tmem_st_wait();
                    }
                    const float neg_m = m > -INFINITY ? -m : 0.f;
                    ASTAMP(2);
                    emit_chunk(v0, v1, neg_m, w);
                    ASTAMP(3);
                    // (a repeated wait on a completed phase returns at once: the rescale above may have waited already)
                    if (!mbar_wait(p_empty(g), (p_it & 1u) ^ 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                    ASTAMP(4);
                    store_chunk(1, w);
                    load_chunk(j, 0, v0, v1);
                    release_s();
                    emit_chunk(v0, v1, neg_m, w);
                    store_chunk(0, w);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the tensor cores
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(g));
                ++p_it;
                ASTAMP(5);
            }
            if (!ok) break;
            if constexpr (MODE == MODE_STATS) {
                if (i < a.lse_ld) a.lse[head * a.lse_ld + i] = l > 0.f ? m + log2f(l) : INFINITY;
            } else if constexpr (MODE == MODE_ENERGY) {
                if (i < a.Lr) a.energy[head * a.Lr + i] = l;
            } else {
                // ---- epilogue: O row (/ l) -> bf16 -> global
                if (!mbar_wait(o_full(g), o_it & 1u, abort_flag, a.status, a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const float inv_l = MODE == MODE_GATHERED ? 1.f : (l > 0.f ? 1.f / l : 0.f);
                for (int c = 0; c < nv * 64; c += 32) {
                    uint32_t v[32];
                    tmem_ld32_issue(t_o + c, v);
                    tmem_ld_wait();
                    if (i < a.Lr) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (c + 8 * u >= a.Dh) break;
                            uint32_t ww[4];
#pragma unroll
                            for (int pp = 0; pp < 4; ++pp) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * u + 2 * pp]) * inv_l,
                                                                         __uint_as_float(v[8 * u + 2 * pp + 1]) * inv_l);
                                ww[pp] = *reinterpret_cast<uint32_t *>(&h);
                            }
                            *reinterpret_cast<uint4 *>(orow + c + 8 * u) = make_uint4(ww[0], ww[1], ww[2], ww[3]);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(o_empty(g));
                ++o_it;
            }
            ASTAMP(6);
        }
        ASTAMP_FLUSH(8);
    }

    __syncthreads();
    if (*abort_flag) {
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    tc_fence_after();
    if (warp == 1) tmem_dealloc<1>(tmem_base, kTmemCols);
}

template <int MODE, bool MASK = false>
int launch_mode(const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv, const FusedArgs &a, const char *name,
                cudaStream_t stream)
{
    auto kern = fused_attn_kernel<MODE, MASK>;
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "fused_attn: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t items = a.heads * ceil_div(a.Lr, kGroups * FM);
    prof_begin(name, stream);
    cudaError_t e = launch_kernel(kern, dim3((unsigned)(items < sms ? items : sms)), dim3(kFusedThreads), kFusedSmem, stream, 1,
                                  mq, mk, mv, a);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "%s: launch: %s", name, cudaGetErrorString(e));
    return check_launch(name, stream);
}

// 3-D map over a packed [heads, rows, ld] bf16 tensor with `cols` valid columns and a box of 64 columns x box_rows rows.
int packed_map(CUtensorMap *m, const __nv_bfloat16 *p, int64_t cols, int64_t rows, int64_t heads, int64_t ld, uint32_t box_rows)
{
    uint64_t dims[3] = {(uint64_t)cols, (uint64_t)rows, (uint64_t)heads};
    uint64_t st[2] = {(uint64_t)ld * 2, (uint64_t)rows * ld * 2};
    const uint32_t box[3] = {64, box_rows, 1};
    return make_map(m, const_cast<__nv_bfloat16 *>(p), 3, dims, st, box, true);
}

}  // namespace

#ifdef RMM_ATTN_STAMPS
extern "C" void rmm_debug_attn_stamps(unsigned long long *out)
{
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_astamps, sizeof(g_astamps));
    unsigned long long z[16] = {};
    cudaMemcpyToSymbol(g_astamps, z, sizeof(z));
}
#endif

bool fused_attn_eligible(const rmm_attn_desc_t *d, int64_t kd)
{
    // heads of up to 256 columns run as two passes over 128 columns of V and O each (S~ and the weights are taken again)
    return d->Dh % 8 == 0 && d->Dh <= 256 && kd <= 128 && d->Lq <= INT32_MAX && d->Lk <= INT32_MAX;
}

// FULL (lse NULL, tok NULL): O = softmax(Qp Kp^T / sqrt(Dh) + mask) V; `mask` (or NULL) is the caller's additive fp32 mask on
// top of the causal one, row (head, i) at mask + head m_sh + i m_sr (16-byte aligned rows).
// GATHERED (lse and tok given): Kp and V hold the kept keys only (Lk = their count, tok their positions); O = P V with
// P = bf16(2^(x - lse)), no renormalisation.  `diag` = Lk - Lq of the unpacked problem.
// Qp [heads, Lq, ldd], Kp [heads, Lk, ldd] packed; V [v_batches, Lk, Dh] with row pitch v_ld and batch pitch v_sb.
int launch_fused_attn(const __nv_bfloat16 *Qp, const __nv_bfloat16 *Kp, int64_t ldd, int64_t kd, const __nv_bfloat16 *V,
                      int64_t v_ld, int64_t v_sb, int64_t v_batches, int64_t v_off, int64_t v_div, __nv_bfloat16 *O,
                      int64_t o_sh, int64_t o_sr, int64_t heads, int64_t Lq, int64_t Lk, int64_t Dh, int causal, int64_t diag,
                      const float *lse, int64_t lse_ld, const int32_t *tok, const float *mask, int64_t m_sh, int64_t m_sr,
                      int *status, cudaStream_t stream)
{
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = packed_map(&mq, Qp, kd, Lq, heads, ldd, FM)) != RMM_OK) return rc;
    if ((rc = packed_map(&mk, Kp, kd, Lk, heads, ldd, FN)) != RMM_OK) return rc;
    // The O accumulators of a block hold 128 columns per query group: a wider head (up to 256 columns) is produced in
    // two passes, each over its own 128 columns of V and of O; the softmax scale keeps the full head dimension.
    for (int64_t c0 = 0; c0 < Dh; c0 += 128) {
        const int64_t dh = Dh - c0 < 128 ? Dh - c0 : 128;
        {
            uint64_t dims[3] = {(uint64_t)dh, (uint64_t)Lk, (uint64_t)v_batches};
            uint64_t st[2] = {(uint64_t)v_ld * 2, v_batches > 1 ? (uint64_t)v_sb * 2 : (uint64_t)v_ld * 2 * (uint64_t)Lk};
            const uint32_t box[3] = {64, FN, 1};
            if ((rc = make_map(&mv, const_cast<__nv_bfloat16 *>(V + c0), 3, dims, st, box, true)) != RMM_OK) return rc;
        }
        FusedArgs a = {};
        a.heads = heads; a.Lr = Lq; a.Lc = Lk; a.diag = diag;
        a.kd = (int)kd; a.Dh = (int)dh; a.causal = causal;
        a.v_off = v_off; a.v_div = v_div > 0 ? v_div : 1;
        a.O = O + c0; a.o_sh = o_sh; a.o_sr = o_sr;
        a.lse = const_cast<float *>(lse); a.lse_ld = lse_ld; a.tok = tok;
        a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)Dh));
        a.status = status;
        a.wait_ns = wait_limit_ns();
        a.withhold = debug_withhold() == WITHHOLD_ATTN;
        if (tok != nullptr) {
            rc = launch_mode<MODE_GATHERED>(mq, mk, mv, a, "fused_attn_gathered_kernel", stream);
        } else if (mask != nullptr) {
            a.mask = mask; a.m_sh = m_sh; a.m_sr = m_sr;
            a.mask_gain = (float)sqrt((double)Dh);
            rc = launch_mode<MODE_FULL, true>(mq, mk, mv, a, "fused_attn_masked_kernel", stream);
        } else {
            rc = launch_mode<MODE_FULL>(mq, mk, mv, a, "fused_attn_kernel", stream);
        }
        if (rc != RMM_OK) return rc;
    }
    return RMM_OK;
}

// Sweeps 1 and 2 of the token reduction on packed Qp [heads, Lq, ldd], Kp [heads, Lk, ldd]:
//   lse [heads, lse_ld] (lse_ld a multiple of 64, >= Lq): log2-domain row normalisers of softmax(S~ + mask);
//   energy [heads, Lk]: squared token scores sum_i bf16(P_it)^2.
int launch_fused_attn_scores(const __nv_bfloat16 *Qp, const __nv_bfloat16 *Kp, int64_t ldd, int64_t kd, int64_t heads,
                             int64_t Lq, int64_t Lk, int64_t Dh, int causal, float *lse, int64_t lse_ld, float *energy,
                             int *status, cudaStream_t stream)
{
    CUtensorMap mq, mk;
    int rc;
    FusedArgs a = {};
    a.heads = heads; a.diag = Lk - Lq;
    a.kd = (int)kd; a.Dh = (int)Dh; a.causal = causal;
    a.v_div = 1;
    a.lse = lse; a.lse_ld = lse_ld; a.energy = energy;
    a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)Dh));
    a.status = status;
    a.wait_ns = wait_limit_ns();
    a.withhold = debug_withhold() == WITHHOLD_ATTN;
    // sweep 1: rows = queries
    if ((rc = packed_map(&mq, Qp, kd, Lq, heads, ldd, FM)) != RMM_OK) return rc;
    if ((rc = packed_map(&mk, Kp, kd, Lk, heads, ldd, FN)) != RMM_OK) return rc;
    a.Lr = Lq; a.Lc = Lk;
    if ((rc = launch_mode<MODE_STATS>(mq, mk, mk, a, "fused_attn_stats_kernel", stream)) != RMM_OK) return rc;
    // sweep 2: rows = keys, tiles of queries stream past
    if ((rc = packed_map(&mq, Kp, kd, Lk, heads, ldd, FM)) != RMM_OK) return rc;
    if ((rc = packed_map(&mk, Qp, kd, Lq, heads, ldd, FN)) != RMM_OK) return rc;
    a.Lr = Lk; a.Lc = Lq;
    return launch_mode<MODE_ENERGY>(mq, mk, mk, a, "fused_attn_energy_kernel", stream);
}

}  // namespace rmm
