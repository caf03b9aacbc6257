// Fused reduced attention for rho_t = 1 (paper Sec. 3.3 with feature reduction only):
//     O = softmax(Q[:, I] K[:, I]^T / sqrt(Dh) + causal mask) V,
// with Q[:, I] and K[:, I] already packed.  S~ and P never leave the SM: S~ tiles live in tensor memory, P tiles in
// shared memory, O accumulates in tensor memory.
//
// One block owns 256 query rows of one head as two groups of 128 and walks the key axis once; both groups consume
// the same K and V tiles, so each tile crosses from L2 to the SM once per 256 rows.  Per 64-key tile and group:
//   S~ = Qp Kp^T on the tensor cores (kd of the Dh features);
//   one thread per query row takes p = 2^(x - m), x = S~ * log2(e) / sqrt(Dh), rounds p once to bf16 and writes it to
//   shared memory as the A operand of O += P V; the row sum l accumulates in fp32 from the unrounded p;
//   m is the row maximum seen so far, refreshed only when the new maximum exceeds it by more than 40 (p up to 2^40
//   and row sums up to 2^71 are far from the bf16 and fp32 range limits, and floating point keeps the same relative
//   precision at any scale): then l and the O row in tensor memory are multiplied by 2^(m_old - m_new).
// The epilogue divides by l.  The paper rounds the normalised weight P to bf16; here the rounded quantity is
// p = P * l * 2^(m_row - m), the same weight up to a per-row fp32 factor, so O differs by bf16 rounding noise only;
// nothing is decided from P when rho_t = 1.
// Warp 0 feeds TMA, warps 2-5 and 6-9 are the softmax/epilogue warps of the two groups (every scheduler has two of
// them to switch between), and one thread of warp 1 and of warp 10 issues the tcgen05.mma of group 0 and 1: a single
// issuing thread for both groups was the bottleneck.  Every wait is bounded.
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace rmm {
namespace {

using namespace ptx;

constexpr int FM = 128, FN = 64;      // queries per group, keys per step
constexpr int kGroups = 2;
constexpr int kFusedThreads = 64 + kGroups * 128 + 32;  // producer, MMA issuer 0, 8 softmax warps, MMA issuer 1
constexpr int kMmaWarp1 = 10;
constexpr int kKvStages = 8;
constexpr int kQChunk = 16384;        // Q chunk: 128 rows x 64 features (128 bytes per row, 128-byte swizzle)
constexpr int kQTile = 2 * kQChunk;   // up to 128 kept features
constexpr int kKvChunk = 8192;        // K or V chunk: 64 keys x 64 features
constexpr int kKvTile = 2 * kKvChunk; // ring entry: a K tile (up to 128 kept features) or a V tile (up to 128 columns)
constexpr int kPTile = 16384;         // P tile: 128 rows x 64 keys
constexpr int kOffQ = 0, kOffKv = kGroups * kQTile, kOffP = kOffKv + kKvStages * kKvTile, kOffBar = kOffP + kGroups * kPTile;
constexpr int kFusedSmem = kOffBar + 512;
constexpr int kTmemCols = 512;        // per group: S~ double buffer (2 x 64 columns); then O (128 columns per group)
constexpr uint32_t kTmemO = kGroups * 2 * FN;
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

struct FusedArgs {
    int64_t heads, Lq, Lk;
    int kd, Dh, causal;
    int64_t v_off, v_div;        // V batch entry of head h = (h + v_off) / v_div
    __nv_bfloat16 *O;
    int64_t o_sh, o_sr;          // element strides of O: head, row
    float scale_log2;            // (1 / sqrt(Dh)) * log2(e)
    int *status;
};

__global__ void __launch_bounds__(kFusedThreads, 1)
fused_attn_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, FusedArgs a)
{
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
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
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
    const int blocks_q = (int)((a.Lq + kGroups * FM - 1) / (kGroups * FM));
    const int64_t items = a.heads * blocks_q;
    const int64_t diag = a.Lk - a.Lq;                             // query i sees keys t <= i + diag when causal
    auto key_tiles = [&](int64_t i0) -> int {                     // key tiles the 128 rows starting at i0 need
        if (i0 >= a.Lq) return 0;
        int64_t last = a.causal ? min(a.Lk - 1, i0 + FM - 1 + diag) : a.Lk - 1;
        return last < 0 ? 0 : (int)(last / FN) + 1;
    };
    // The n-th item of this block: heaviest query blocks first, and the direction alternates from round to round, so
    // that the block that drew the heaviest item of one round draws the lightest of the next.
    auto item_of = [&](int64_t n, int64_t *head, int64_t *i0) -> bool {
        const int64_t b = (n & 1) ? (int64_t)gridDim.x - 1 - blockIdx.x : blockIdx.x;
        const int64_t item = n * gridDim.x + b;
        if (item >= items) return false;
        *head = item % a.heads;
        *i0 = (int64_t)(blocks_q - 1 - item / a.heads) * (kGroups * FM);
        return true;
    };
    const int64_t rounds = (items + gridDim.x - 1) / gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer: Q, then K_0, K_1, V_0, K_2, V_1, ...
        uint32_t ks = 0, kph = 0, n_item = 0;
        bool ok = true;
        auto load_kv = [&](const CUtensorMap *map, int chunks, int64_t row, int z) -> bool {
            if (!mbar_wait_sleepy(kv_empty(ks), kph ^ 1u, abort_flag, a.status)) return false;
            const uint32_t dst = base + kOffKv + ks * kKvTile;
            mbar_arrive_expect_tx(kv_full(ks), (uint32_t)chunks * kKvChunk);
            for (int c = 0; c < chunks; ++c) tma_load_3d(dst + c * kKvChunk, map, c * 64, (int)row, z, kv_full(ks));
            if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
            return true;
        };
        for (int64_t n = 0; lane == 0 && n < rounds && ok; ++n) {
            int64_t head, i0;
            if (!item_of(n, &head, &i0)) continue;
            const int nt = max(key_tiles(i0), key_tiles(i0 + FM));
            if (nt == 0) continue;
            const int vb = (int)((head + a.v_off) / a.v_div);
            if (!mbar_wait_sleepy(q_empty, (n_item & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
            mbar_arrive_expect_tx(q_full, (uint32_t)(kGroups * kq) * kQChunk);
            for (int g = 0; g < kGroups; ++g)
                for (int c = 0; c < kq; ++c)
                    tma_load_3d(base + kOffQ + g * kQTile + c * kQChunk, &map_q, c * 64, (int)(i0 + g * FM), (int)head, q_full);
            ok = load_kv(&map_k, kq, 0, (int)head);
            for (int j = 0; j < nt && ok; ++j) {
                if (j + 1 < nt) ok = load_kv(&map_k, kq, (int64_t)(j + 1) * FN, (int)head);
                if (ok) ok = load_kv(&map_v, nv, (int64_t)j * FN, vb);
            }
            ++n_item;  // counts the items that reach the tensor cores (those with at least one key tile)
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
        const uint32_t t_s = tmem_base + g * 2 * FN, t_o = tmem_base + kTmemO + g * 128;
        uint32_t ks = 0, kph = 0, n_item = 0, s_it = 0, p_it = 0, o_it = 0;
        bool ok = true;
        int nt = 0;
        ASTAMP_DECL(blockIdx.x == 0 && lane == 0 && g == 0);
        auto step_s = [&](int j) -> bool {  // S~ of key tile j (if this group needs it); consumes one ring entry
            ASTAMP(7);
            if (!mbar_wait_lane(kv_full(ks), kph, abort_flag, a.status)) return false;
            ASTAMP(0);
            if (j < nt) {
                const uint32_t sb = s_it & 1u;
                if (!mbar_wait_lane(s_empty(g, sb), ((s_it >> 1) & 1u) ^ 1u, abort_flag, a.status)) return false;
                ASTAMP(1);
                tc_fence_after();
                uint32_t ql = q_lo, kl = k_lo + ks * (kKvTile >> 4), acc = 0;
                for (int left = steps_s; left > 0; left -= 4, ql += kQChunk >> 4, kl += kKvChunk >> 4) {  // 64-feature chunks
                    const int ns = left < 4 ? left : 4;
                    for (int st = 0; st < ns; ++st, acc = 1u)  // 16 features = 32 bytes per step
                        umma_bf16_lohi<1>(t_s + sb * FN, ql + 2 * st, q_hi, kl + 2 * st, k_hi, idesc_s, acc);
                }
                umma_commit<1>(s_full(g, sb));
                ++s_it;
            }
            umma_commit<1>(kv_empty(ks));
            if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
            ASTAMP(2);
            return true;
        };
        for (int64_t n = 0; lane == 0 && n < rounds && ok; ++n) {
            int64_t head, i0;
            if (!item_of(n, &head, &i0)) continue;
            const int ntmax = max(key_tiles(i0), key_tiles(i0 + FM));
            nt = key_tiles(i0 + g * FM);
            if (ntmax == 0) continue;
            if (!mbar_wait_lane(q_full, n_item & 1u, abort_flag, a.status)) { ok = false; break; }
            ok = step_s(0);
            for (int j = 0; j < ntmax && ok; ++j) {
                if (j + 1 < ntmax) ok = step_s(j + 1);                     // S~ of the next tile runs ahead of this P V
                if (!ok) break;
                ASTAMP(7);
                if (!mbar_wait_lane(kv_full(ks), kph, abort_flag, a.status)) { ok = false; break; }
                ASTAMP(3);
                if (j < nt) {
                    if (j == 0 && !mbar_wait_lane(o_empty(g), (o_it & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
                    ASTAMP(4);
                    if (!mbar_wait_lane(p_full(g), p_it & 1u, abort_flag, a.status)) { ok = false; break; }
                    ASTAMP(5);
                    tc_fence_after();
                    const uint32_t vl = v_lo + ks * (kKvTile >> 4);
#pragma unroll
                    for (int st = 0; st < FN / 16; ++st)  // P: K-major, 32 bytes per step; V: MN-major (rows = keys), 16 keys = 2048 bytes
                        umma_bf16_lohi<1>(t_o, p_lo + st * 2, p_hi, vl + st * (2048 >> 4), v_hi, idesc_o, (j | st) != 0 ? 1u : 0u);
                    umma_commit<1>(p_empty(g));   // "P V of this tile is complete": P may be rewritten, O may be rescaled
                    ++p_it;
                    if (j == nt - 1) {
                        umma_commit<1>(o_full(g));
                        ++o_it;
                    }
                }
                umma_commit<1>(kv_empty(ks));
                if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
                ASTAMP(6);
            }
            if (ok) umma_commit<1>(q_empty);
            ++n_item;
        }
        ASTAMP_FLUSH(0);
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax and epilogue (one query row per thread)
        const int g = (warp - 2) >> 2, q = warp & 3, r = q * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t t_s = t_lane + g * 2 * FN, t_o = t_lane + kTmemO + g * 128;
        const float c2 = a.scale_log2;
        const uint64_t c22 = pack2(c2, c2);
        uint8_t *prow = base_ptr + kOffP + g * kPTile + r * 128;  // row r: 64 keys = 128 bytes, 16-byte units swizzled
        uint32_t s_it = 0, p_it = 0, o_it = 0;
        bool ok = true;
        ASTAMP_DECL(blockIdx.x == 0 && warp == 2 && lane == 0);
        for (int64_t n = 0; n < rounds && ok; ++n) {
            int64_t head, i0;
            if (!item_of(n, &head, &i0)) continue;
            i0 += g * FM;
            if (i0 >= a.Lq) continue;                  // this group has no rows in the last query block
            const int nt = key_tiles(i0);
            const int64_t i = i0 + r;
            __nv_bfloat16 *orow = a.O + head * a.o_sh + i * a.o_sr;
            if (nt == 0) {  // no visible key for any row of this group: the output rows are zero
                if (i < a.Lq)
                    for (int c = 0; c < a.Dh; c += 8) *reinterpret_cast<uint4 *>(orow + c) = make_uint4(0, 0, 0, 0);
                continue;
            }
            const int64_t last_key = a.causal ? min(a.Lk - 1, i + diag) : a.Lk - 1;  // < 0: this row sees nothing
            float m = -INFINITY, l = 0.f;  // m: the maximum that p is taken against (scaled, log2 domain)
            for (int j = 0; j < nt; ++j, ++s_it, ++p_it) {
                const uint32_t sb = s_it & 1u;
                ASTAMP(7);
                if (!mbar_wait(s_full(g, sb), (s_it >> 1) & 1u, abort_flag, a.status)) { ok = false; break; }
                ASTAMP(0);
                tc_fence_after();
                uint32_t v0[32], v1[32];
                tmem_ld32_issue(t_s + sb * FN + 0, v0);
                tmem_ld32_issue(t_s + sb * FN + 32, v1);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(g, sb));
                ASTAMP(1);

                // boundary tiles only (the diagonal and the ragged end): hidden keys become -inf
                const int64_t rel = last_key - (int64_t)j * FN;
                const int lim = rel > FN - 1 ? FN - 1 : (rel < -1 ? -1 : (int)rel);
                if (!__all_sync(0xffffffffu, lim >= FN - 1)) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        if (e > lim) v0[e] = 0xff800000u;
                        if (e + 32 > lim) v1[e] = 0xff800000u;
                    }
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    mx0 = fmax3(mx0, __uint_as_float(v0[e]), __uint_as_float(v0[e + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(v0[e + 2]), __uint_as_float(v0[e + 3]));
                    mx2 = fmax3(mx2, __uint_as_float(v1[e]), __uint_as_float(v1[e + 1]));
                    mx3 = fmax3(mx3, __uint_as_float(v1[e + 2]), __uint_as_float(v1[e + 3]));
                }
                const float mc = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * c2;
                const bool grow = mc > m + kGrowLimit;
                bool p_free = false;  // has this tile's wait for the previous P V been done?
                if (__any_sync(0xffffffffu, grow)) {
                    const float alpha = (grow && m > -INFINITY) ? ex2(m - mc) : 1.f;
                    l *= alpha;
                    if (grow) m = mc;
                    if (j > 0) {  // rows of O already hold sums taken against the old maximum
                        if (!mbar_wait(p_empty(g), (p_it & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
                        p_free = true;
                        tc_fence_after();
                        for (int c = 0; c < nv * 64; c += 32) {
                            uint32_t o[32];
                            tmem_ld32_issue(t_o + c, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st32_issue(t_o + c, o);
                        }
                        tmem_st_wait();
                    }
                }
                const float neg_m = m > -INFINITY ? -m : 0.f;
                const uint64_t nm2 = pack2(neg_m, neg_m);
                ASTAMP(2);

                // p for the 64 keys, rounded and packed in registers; the shared-memory tile is written once the
                // tensor cores are done with the previous one
                uint64_t sum_a = 0, sum_b = 0;  // two packed pairs of partial row sums
                uint32_t w[32];
                auto emit = [&](const uint32_t (&v)[32], int c) {
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float x0, x1;
                        unpack2(ffma2(pack2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), c22, nm2), x0, x1);
                        const float p0 = ex2(x0), p1 = ex2(x1);
                        (e & 2 ? sum_b : sum_a) = fadd2(e & 2 ? sum_b : sum_a, pack2(p0, p1));
                        __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                        w[(c + e) >> 1] = *reinterpret_cast<uint32_t *>(&h);
                    }
                };
                emit(v0, 0);
                emit(v1, 32);
                {
                    float s0, s1;
                    unpack2(fadd2(sum_a, sum_b), s0, s1);
                    l += s0 + s1;
                }
                ASTAMP(3);
                if (!p_free && !mbar_wait(p_empty(g), (p_it & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
                ASTAMP(4);
#pragma unroll
                for (int u = 0; u < 8; ++u)  // 16-byte units of 8 keys
                    *reinterpret_cast<uint4 *>(prow + ((u ^ (r & 7)) << 4)) = make_uint4(w[4 * u], w[4 * u + 1], w[4 * u + 2], w[4 * u + 3]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the tensor cores
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(g));
                ASTAMP(5);
            }
            if (!ok) break;
            // ---- epilogue: O row / l -> bf16 -> global
            if (!mbar_wait(o_full(g), o_it & 1u, abort_flag, a.status)) { ok = false; break; }
            tc_fence_after();
            const float inv_l = l > 0.f ? 1.f / l : 0.f;
            for (int c = 0; c < nv * 64; c += 32) {
                uint32_t v[32];
                tmem_ld32_issue(t_o + c, v);
                tmem_ld_wait();
                if (i < a.Lq) {
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
    return d->rho_t >= 1.0 && d->Dh % 8 == 0 && d->Dh <= 128 && kd <= 128 && d->Lq <= INT32_MAX && d->Lk <= INT32_MAX;
}

// Qp [heads, Lq, ldd], Kp [heads, Lk, ldd] packed; V [v_batches, Lk, Dh] in place with row pitch v_ld and batch pitch v_sb.
int launch_fused_attn(const __nv_bfloat16 *Qp, const __nv_bfloat16 *Kp, int64_t ldd, int64_t kd, const __nv_bfloat16 *V,
                      int64_t v_ld, int64_t v_sb, int64_t v_batches, int64_t v_off, int64_t v_div, __nv_bfloat16 *O,
                      int64_t o_sh, int64_t o_sr, int64_t heads, int64_t Lq, int64_t Lk, int64_t Dh, int causal,
                      int *status, cudaStream_t stream)
{
    CUtensorMap mq, mk, mv;
    int rc;
    const uint32_t box_q[3] = {64, FM, 1}, box_kv[3] = {64, FN, 1};
    {
        uint64_t dims[3] = {(uint64_t)kd, (uint64_t)Lq, (uint64_t)heads};
        uint64_t st[2] = {(uint64_t)ldd * 2, (uint64_t)Lq * ldd * 2};
        if ((rc = make_map(&mq, const_cast<__nv_bfloat16 *>(Qp), 3, dims, st, box_q, true)) != RMM_OK) return rc;
    }
    {
        uint64_t dims[3] = {(uint64_t)kd, (uint64_t)Lk, (uint64_t)heads};
        uint64_t st[2] = {(uint64_t)ldd * 2, (uint64_t)Lk * ldd * 2};
        if ((rc = make_map(&mk, const_cast<__nv_bfloat16 *>(Kp), 3, dims, st, box_kv, true)) != RMM_OK) return rc;
    }
    {
        uint64_t dims[3] = {(uint64_t)Dh, (uint64_t)Lk, (uint64_t)v_batches};
        uint64_t st[2] = {(uint64_t)v_ld * 2, v_batches > 1 ? (uint64_t)v_sb * 2 : (uint64_t)v_ld * 2 * (uint64_t)Lk};
        if ((rc = make_map(&mv, const_cast<__nv_bfloat16 *>(V), 3, dims, st, box_kv, true)) != RMM_OK) return rc;
    }
    FusedArgs a;
    a.heads = heads; a.Lq = Lq; a.Lk = Lk;
    a.kd = (int)kd; a.Dh = (int)Dh; a.causal = causal;
    a.v_off = v_off; a.v_div = v_div > 0 ? v_div : 1;
    a.O = O; a.o_sh = o_sh; a.o_sr = o_sr;
    a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)Dh));
    a.status = status;
    static PerDeviceOnce configured;
    if (configured.first()) {
        cudaError_t e = cudaFuncSetAttribute(fused_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "fused_attn: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t items = heads * ceil_div(Lq, kGroups * FM);
    prof_begin("fused_attn_kernel", stream);
    cudaError_t e = launch_kernel(fused_attn_kernel, dim3((unsigned)(items < sms ? items : sms)), dim3(kFusedThreads), kFusedSmem,
                                  stream, 1, mq, mk, mv, a);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "fused_attn_kernel: launch: %s", cudaGetErrorString(e));
    return check_launch("fused_attn_kernel", stream);
}

}  // namespace rmm
