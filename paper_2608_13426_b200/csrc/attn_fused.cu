// Fused reduced attention for rho_t = 1 (paper Sec. 3.3 with feature reduction only):
//     O = softmax(Q[:, I] K[:, I]^T / sqrt(Dh) + causal mask) V,
// with Q[:, I] and K[:, I] already packed.  S~ and P never leave the SM: S~ tiles live in tensor memory, P tiles in
// shared memory.
//
// One block owns 128 query rows of one head and walks the key axis twice:
//   pass 1  S~ tile = Qp Kp^T on the tensor cores; one thread per query row keeps the running maximum and sum, which
//           give the row's log-sum-exp;
//   pass 2  the same S~ tiles again (the reduced Q K^T is cheap: kd of Dh indices); P = bf16(exp(S~ - lse)) is the
//           FINAL, normalised attention weight rounded once to bf16, so it can be written to shared memory as the
//           A operand of O += P V with no running rescale of O.
// Knowing the normaliser before the first P V product is what removes the correction step of one-pass schemes, at
// the price of a second reduced Q K^T.  Warp 0 feeds TMA, warp 1 issues tcgen05.mma, warps 2-5 do the softmax (one
// query row per thread) and the epilogue.  Every wait is bounded.
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace rmm {
namespace {

using namespace ptx;

constexpr int FM = 128, FN = 128;     // queries per block tile, keys per step
constexpr int kFusedThreads = 192;
constexpr int kKvStages = 3;
constexpr int kTile = 32768;          // bytes of a Q, K, V or P tile (two 64-column chunks of 128 rows)
constexpr int kChunk = 16384;         // one chunk: 128 rows x 128 bytes, 128-byte swizzle
constexpr int kOffQ = 0, kOffKv = kTile, kOffP = kOffKv + kKvStages * kTile, kOffBar = kOffP + 2 * kTile;
constexpr int kFusedSmem = kOffBar + 256 + 1024;

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
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + kOffBar;
    // barriers: q_full, q_empty, kv_full[3], kv_empty[3], s_full[2], s_empty[2], p_full[2], p_empty[2], o_full, o_empty
    const uint32_t q_full = bar0, q_empty = bar0 + 8;
    auto kv_full = [&](int s) { return bar0 + 16u + 8u * s; };
    auto kv_empty = [&](int s) { return bar0 + 16u + 8u * (kKvStages + s); };
    auto s_full = [&](int i) { return bar0 + 64u + 8u * i; };
    auto s_empty = [&](int i) { return bar0 + 80u + 8u * i; };
    auto p_full = [&](int i) { return bar0 + 96u + 8u * i; };
    auto p_empty = [&](int i) { return bar0 + 112u + 8u * i; };
    const uint32_t o_full = bar0 + 128, o_empty = bar0 + 136;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + kOffBar + 144);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + kOffBar + 152);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int s = 0; s < kKvStages; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full(i), 1); mbar_init(s_empty(i), 4);
            mbar_init(p_full(i), 4); mbar_init(p_empty(i), 1);
        }
        mbar_init(o_full, 1);
        mbar_init(o_empty, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<1>(smem_u32(const_cast<uint32_t *>(tmem_slot)), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    const int kq = (a.kd + 63) / 64, nv = (a.Dh + 63) / 64;       // 64-column chunks of Q/K and of V
    const int tiles_q = (int)((a.Lq + FM - 1) / FM);
    const int64_t items = a.heads * tiles_q;
    const int64_t diag = a.Lk - a.Lq;                             // query i sees keys t <= i + diag when causal
    auto key_tiles = [&](int64_t i0) -> int {                     // key tiles a query tile starting at row i0 needs
        int64_t last = a.causal ? min(a.Lk - 1, i0 + FM - 1 + diag) : a.Lk - 1;
        return last < 0 ? 0 : (int)(last / FN) + 1;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        uint32_t ks = 0, kph = 0, n_item = 0;
        bool ok = true;
        auto load_kv = [&](const CUtensorMap *map, int chunks, int64_t row, int z) -> bool {
            if (!mbar_wait_lane(kv_empty(ks), kph ^ 1u, abort_flag, a.status)) return false;
            const uint32_t dst = base + kOffKv + ks * kTile;
            mbar_arrive_expect_tx(kv_full(ks), (uint32_t)chunks * kChunk);
            for (int c = 0; c < chunks; ++c) tma_load_3d(dst + c * kChunk, map, c * 64, (int)row, z, kv_full(ks));
            if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
            return true;
        };
        for (int64_t item = blockIdx.x; lane == 0 && item < items && ok; item += gridDim.x) {
            const int64_t head = item / tiles_q, i0 = (int64_t)(tiles_q - 1 - item % tiles_q) * FM;
            const int nt = key_tiles(i0);
            if (nt == 0) continue;
            const int vb = (int)((head + a.v_off) / a.v_div);
            if (!mbar_wait_lane(q_empty, (n_item & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
            mbar_arrive_expect_tx(q_full, (uint32_t)kq * kChunk);
            for (int c = 0; c < kq; ++c) tma_load_3d(base + kOffQ + c * kChunk, &map_q, c * 64, (int)i0, (int)head, q_full);
            for (int j = 0; j < nt && ok; ++j) ok = load_kv(&map_k, kq, (int64_t)j * FN, (int)head);   // pass 1
            if (ok) ok = load_kv(&map_k, kq, 0, (int)head);                                              // pass 2
            for (int j = 0; j < nt && ok; ++j) {
                if (j + 1 < nt) ok = load_kv(&map_k, kq, (int64_t)(j + 1) * FN, (int)head);
                if (ok) ok = load_kv(&map_v, nv, (int64_t)j * FN, vb);
            }
            ++n_item;  // counts the items that reach the tensor cores (those with at least one key tile)
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(FN >> 3) << 17) | ((uint32_t)(FM >> 4) << 24);
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)((nv * 64) >> 3) << 17) |
                                 ((uint32_t)(FM >> 4) << 24);
        const uint64_t dq0 = smem_desc(base + kOffQ, 16, 1024), dk0 = smem_desc(base + kOffKv, 16, 1024);
        const uint64_t dp0 = smem_desc(base + kOffP, 16, 1024), dv0 = smem_desc(base + kOffKv, kChunk, 1024);
        const uint32_t q_hi = (uint32_t)(dq0 >> 32), k_hi = (uint32_t)(dk0 >> 32), p_hi = (uint32_t)(dp0 >> 32), v_hi = (uint32_t)(dv0 >> 32);
        const uint32_t q_lo = (uint32_t)dq0, k_lo = (uint32_t)dk0, p_lo = (uint32_t)dp0, v_lo = (uint32_t)dv0;
        const int steps_s = (a.kd + 15) / 16;
        uint32_t ks = 0, kph = 0, s_it = 0, p_it = 0, n_item = 0;
        bool ok = true;
        auto issue_s = [&]() -> bool {  // S~[s_it % 2] = Qp Kp_tile^T, consuming the next ring entry
            const uint32_t sb = s_it & 1u;
            if (!mbar_wait_lane(kv_full(ks), kph, abort_flag, a.status)) return false;
            if (!mbar_wait_lane(s_empty(sb), ((s_it >> 1) & 1u) ^ 1u, abort_flag, a.status)) return false;
            tc_fence_after();
            const uint32_t kl = k_lo + ks * (kTile >> 4);
            for (int st = 0; st < steps_s; ++st) {
                const uint32_t off = (uint32_t)((st >> 2) * (kChunk >> 4) + (st & 3) * 2);
                umma_bf16_lohi<1>(tmem_base + sb * FN, q_lo + off, q_hi, kl + off, k_hi, idesc_s, st != 0 ? 1u : 0u);
            }
            umma_commit<1>(kv_empty(ks));
            umma_commit<1>(s_full(sb));
            if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
            ++s_it;
            return true;
        };
        for (int64_t item = blockIdx.x; lane == 0 && item < items && ok; item += gridDim.x) {
            const int64_t i0 = (int64_t)(tiles_q - 1 - item % tiles_q) * FM;
            const int nt = key_tiles(i0);
            if (nt == 0) continue;
            if (!mbar_wait_lane(q_full, n_item & 1u, abort_flag, a.status)) { ok = false; break; }
            for (int j = 0; j < nt && ok; ++j) ok = issue_s();             // pass 1
            if (ok) ok = issue_s();                                        // pass 2: S~ of tile 0
            for (int j = 0; j < nt && ok; ++j) {
                if (j + 1 < nt) ok = issue_s();                            // S~ of the next tile runs ahead of this P V
                if (!ok) break;
                const uint32_t pb = p_it & 1u;
                if (!mbar_wait_lane(p_full(pb), (p_it >> 1) & 1u, abort_flag, a.status)) { ok = false; break; }
                if (!mbar_wait_lane(kv_full(ks), kph, abort_flag, a.status)) { ok = false; break; }
                if (j == 0 && !mbar_wait_lane(o_empty, (n_item & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t pl = p_lo + pb * (kTile >> 4), vl = v_lo + ks * (kTile >> 4);
#pragma unroll
                for (int st = 0; st < FN / 16; ++st) {
                    // P: K-major, 64-key chunks; V: MN-major (rows = keys), 16 keys = 2048 bytes
                    const uint32_t poff = (uint32_t)((st >> 2) * (kChunk >> 4) + (st & 3) * 2);
                    umma_bf16_lohi<1>(tmem_base + 2 * FN, pl + poff, p_hi, vl + st * (2048 >> 4), v_hi, idesc_o, (j | st) != 0 ? 1u : 0u);
                }
                umma_commit<1>(p_empty(pb));
                umma_commit<1>(kv_empty(ks));
                if (++ks == kKvStages) { ks = 0; kph ^= 1u; }
                ++p_it;
            }
            if (ok) {
                umma_commit<1>(o_full);
                umma_commit<1>(q_empty);
            }
            ++n_item;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax and epilogue (one query row per thread)
        const int q = warp & 3, r = q * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        uint32_t s_it = 0, p_it = 0, n_item = 0;
        bool ok = true;
        for (int64_t item = blockIdx.x; item < items && ok; item += gridDim.x) {
            const int64_t head = item / tiles_q, i0 = (int64_t)(tiles_q - 1 - item % tiles_q) * FM;
            const int nt = key_tiles(i0);
            const int64_t i = i0 + r;
            __nv_bfloat16 *orow = a.O + head * a.o_sh + i * a.o_sr;
            if (nt == 0) {  // no visible key for any row of this tile: the output rows are zero
                if (i < a.Lq)
                    for (int c = 0; c < a.Dh; c += 8) *reinterpret_cast<uint4 *>(orow + c) = make_uint4(0, 0, 0, 0);
                continue;
            }
            const int64_t last_key = a.causal ? min(a.Lk - 1, i + diag) : a.Lk - 1;  // < 0: this row sees nothing
            // ---- pass 1: running maximum and sum of 2^(x), x = S~ * scale * log2(e)
            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < nt; ++j, ++s_it) {
                const uint32_t sb = s_it & 1u;
                if (!mbar_wait(s_full(sb), (s_it >> 1) & 1u, abort_flag, a.status)) { ok = false; break; }
                tc_fence_after();
                uint32_t v0[32], v1[32], v2[32], v3[32];
                tmem_ld32_issue(t_lane + sb * FN + 0, v0);
                tmem_ld32_issue(t_lane + sb * FN + 32, v1);
                tmem_ld32_issue(t_lane + sb * FN + 64, v2);
                tmem_ld32_issue(t_lane + sb * FN + 96, v3);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(sb));
                const int64_t t0 = (int64_t)j * FN;
                auto fold = [&](const uint32_t (&v)[32], int c) {
                    float x[32], cm = -INFINITY;
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        x[e] = (t0 + c + e <= last_key) ? __uint_as_float(v[e]) * a.scale_log2 : -INFINITY;
                        cm = fmaxf(cm, x[e]);
                    }
                    const float mn = fmaxf(m, cm);
                    if (mn > -INFINITY) {
                        float sum = 0.f;
#pragma unroll
                        for (int e = 0; e < 32; ++e) sum += exp2f(x[e] - mn);
                        l = l * exp2f(m - mn) + sum;
                        m = mn;
                    }
                };
                fold(v0, 0); fold(v1, 32); fold(v2, 64); fold(v3, 96);
            }
            if (!ok) break;
            const float lse2 = l > 0.f ? m + log2f(l) : INFINITY;  // rows that see nothing give P = 0
            // ---- pass 2: P = bf16(2^(x - lse2)) into shared memory as the K-major A operand of P V
            for (int j = 0; j < nt; ++j, ++s_it, ++p_it) {
                const uint32_t sb = s_it & 1u, pb = p_it & 1u;
                if (!mbar_wait(s_full(sb), (s_it >> 1) & 1u, abort_flag, a.status)) { ok = false; break; }
                tc_fence_after();
                uint32_t v0[32], v1[32], v2[32], v3[32];
                tmem_ld32_issue(t_lane + sb * FN + 0, v0);
                tmem_ld32_issue(t_lane + sb * FN + 32, v1);
                tmem_ld32_issue(t_lane + sb * FN + 64, v2);
                tmem_ld32_issue(t_lane + sb * FN + 96, v3);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(sb));
                if (!mbar_wait(p_empty(pb), ((p_it >> 1) & 1u) ^ 1u, abort_flag, a.status)) { ok = false; break; }
                const int64_t t0 = (int64_t)j * FN;
                uint8_t *prow = base_ptr + kOffP + pb * kTile + r * 128;  // row r of each 64-key chunk
                auto emit = [&](const uint32_t (&v)[32], int c) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {  // four 16-byte units of 8 keys
                        uint32_t w[4];
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp) {
                            const int e = 8 * u + 2 * pp;
                            const float p0 = (t0 + c + e <= last_key) ? exp2f(__uint_as_float(v[e]) * a.scale_log2 - lse2) : 0.f;
                            const float p1 = (t0 + c + e + 1 <= last_key) ? exp2f(__uint_as_float(v[e + 1]) * a.scale_log2 - lse2) : 0.f;
                            __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                            w[pp] = *reinterpret_cast<uint32_t *>(&h);
                        }
                        const int key = c + 8 * u;                  // first key of this unit within the tile
                        const int unit = (key & 63) >> 3;           // 16-byte unit within the 128-byte row of its chunk
                        *reinterpret_cast<uint4 *>(prow + (key >> 6) * kChunk + ((unit ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                };
                emit(v0, 0); emit(v1, 32); emit(v2, 64); emit(v3, 96);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the tensor cores
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(pb));
            }
            if (!ok) break;
            // ---- epilogue: O row -> bf16 -> global
            if (!mbar_wait(o_full, n_item & 1u, abort_flag, a.status)) { ok = false; break; }
            tc_fence_after();
            for (int c = 0; c < nv * 64; c += 32) {
                uint32_t v[32];
                tmem_ld32_issue(t_lane + 2 * FN + c, v);
                tmem_ld_wait();
                if (i < a.Lq) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (c + 8 * u >= a.Dh) break;
                        uint32_t w[4];
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * u + 2 * pp]), __uint_as_float(v[8 * u + 2 * pp + 1]));
                            w[pp] = *reinterpret_cast<uint32_t *>(&h);
                        }
                        *reinterpret_cast<uint4 *>(orow + c + 8 * u) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_empty);
            ++n_item;
        }
    }

    __syncthreads();
    if (*abort_flag) {
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    tc_fence_after();
    if (warp == 1) tmem_dealloc<1>(tmem_base, 512);
}

}  // namespace

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
    const uint32_t box[3] = {64, 128, 1};
    {
        uint64_t dims[3] = {(uint64_t)kd, (uint64_t)Lq, (uint64_t)heads};
        uint64_t st[2] = {(uint64_t)ldd * 2, (uint64_t)Lq * ldd * 2};
        if ((rc = make_map(&mq, const_cast<__nv_bfloat16 *>(Qp), 3, dims, st, box, true)) != RMM_OK) return rc;
    }
    {
        uint64_t dims[3] = {(uint64_t)kd, (uint64_t)Lk, (uint64_t)heads};
        uint64_t st[2] = {(uint64_t)ldd * 2, (uint64_t)Lk * ldd * 2};
        if ((rc = make_map(&mk, const_cast<__nv_bfloat16 *>(Kp), 3, dims, st, box, true)) != RMM_OK) return rc;
    }
    {
        uint64_t dims[3] = {(uint64_t)Dh, (uint64_t)Lk, (uint64_t)v_batches};
        uint64_t st[2] = {(uint64_t)v_ld * 2, v_batches > 1 ? (uint64_t)v_sb * 2 : (uint64_t)v_ld * 2 * (uint64_t)Lk};
        if ((rc = make_map(&mv, const_cast<__nv_bfloat16 *>(V), 3, dims, st, box, true)) != RMM_OK) return rc;
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
    const int64_t items = heads * ceil_div(Lq, FM);
    prof_begin("fused_attn_kernel", stream);
    cudaError_t e = launch_kernel(fused_attn_kernel, dim3((unsigned)(items < sms ? items : sms)), dim3(kFusedThreads), kFusedSmem,
                                  stream, 1, mq, mk, mv, a);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "fused_attn_kernel: launch: %s", cudaGetErrorString(e));
    return check_launch("fused_attn_kernel", stream);
}

}  // namespace rmm
