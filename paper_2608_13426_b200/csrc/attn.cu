// Reduced attention (paper Sec. 3.3) composed from the library's own kernels, one group of query heads
// at a time:
//   score + select on Q          -> I per query head              (score_tma_kernel / score_select_kernel)
//   pack Q[:, I], K_g[:, I]      -> K-major operands              (pack_kernel)
//   S~ = Q[:, I] K[:, I]^T / sqrt(Dh), fp32                        (reduced_gemm_tc_kernel, K-major B)
//   P  = bf16(softmax(S~ + causal mask))                            (softmax_rows_kernel)
//   rho_t < 1: score + select on P -> T; pack P[:, T] and V_g[T, :]; O = P[:, T] V_g[T, :]
//   rho_t = 1: O = P V_g (same kernel, P and V loaded in place)
// S~ and P live in the workspace (materialised), so this form is bound by HBM traffic, not by the tensor cores.
//
// With up to 128 kept features and a head_dim of up to 256 the steps after the packing run fused instead (attn_fused.cu), S~ and P
// staying on the SM:
//   rho_t = 1: one pass, O = softmax(S~ + mask) V;
//   rho_t < 1: row normalisers (sweep 1), token scores of the bf16-rounded P (sweep 2), select T, pack K[T] and V[T],
//              O = P[:, T] V[T, :] (sweep 3).
#include <math.h>
#include <stdlib.h>

#include "common.cuh"

namespace rmm {
namespace {

constexpr int kSoftmaxThreads = 256;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float *sh)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        float o = __shfl_xor_sync(0xffffffffu, v, d);
        v = is_max ? fmaxf(v, o) : v + o;
    }
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    if (warp == 0) {
        float w = lane < (blockDim.x >> 5) ? sh[lane] : (is_max ? -INFINITY : 0.f);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            float o = __shfl_xor_sync(0xffffffffu, w, d);
            w = is_max ? fmaxf(w, o) : w + o;
        }
        if (lane == 0) sh[0] = w;
    }
    __syncthreads();
    return sh[0];
}

// One block per row: max, sum of exp, normalise, round to bf16 (RNE).  Keys t > i + (Lk - Lq) are masked
// when causal; `mask` (or NULL) is the additive M of P = softmax(S~ + M), row (h, i) at mask + h m_sh + i m_sr; a row
// with no visible key is all zeros.
__global__ void __launch_bounds__(kSoftmaxThreads) softmax_rows_kernel(const float *__restrict__ S, int64_t ld_s,
                                                                       int64_t Lq, int64_t Lk, int causal,
                                                                       const float *__restrict__ mask, int64_t m_sh,
                                                                       int64_t m_sr, __nv_bfloat16 *__restrict__ P,
                                                                       int64_t ld_p)
{
    __shared__ float sh[32];
    pdl_wait();
    const int64_t i = blockIdx.x, h = blockIdx.y;
    const float *s = S + (h * Lq + i) * ld_s;
    const float *m = mask != nullptr ? mask + h * m_sh + i * m_sr : nullptr;
    __nv_bfloat16 *p = P + (h * Lq + i) * ld_p;
    int64_t visible = causal ? i + (Lk - Lq) + 1 : Lk;
    if (visible > Lk) visible = Lk;
    if (visible < 0) visible = 0;
    auto logit = [&](int64_t t) { return m != nullptr ? s[t] + m[t] : s[t]; };

    float mx = -INFINITY;
    for (int64_t t = threadIdx.x; t < visible; t += kSoftmaxThreads) mx = fmaxf(mx, logit(t));
    mx = block_reduce(mx, true, sh);
    if (!(mx > -INFINITY)) visible = 0;  // every key hidden
    float sum = 0.f;
    for (int64_t t = threadIdx.x; t < visible; t += kSoftmaxThreads) sum += expf(logit(t) - mx);
    sum = block_reduce(sum, false, sh);
    const float inv = sum > 0.f ? 1.0f / sum : 0.f;
    for (int64_t t = threadIdx.x; t < ld_p; t += kSoftmaxThreads) {
        float v = t < visible ? expf(logit(t) - mx) * inv : 0.f;
        p[t] = __float2bfloat16_rn(v);
    }
}

struct AttnPlan {
    int64_t kd, kt, ldd, ldt, ld_s, ld_p, hg, lse_ld;
    bool fused;
    size_t inner_bytes, off_idxf, off_idxt, off_qp, off_kp, off_s, off_p, off_pp, off_vp, off_lse, off_energy, off_kpt, total;
};

// up to 128 kept features of heads up to 256 wide run fused (RMM_ATTN_FUSED=0 keeps the composed form, for comparison).
bool use_fused(const rmm_attn_desc_t *d, int64_t kd)
{
    static const bool enabled = [] {
        const char *e = getenv("RMM_ATTN_FUSED");
        return e == nullptr || e[0] != '0';
    }();
    return enabled && fused_attn_eligible(d, kd);
}

// A batch of sequences whose (batch, head) pairs are evenly spaced in memory is one sequence with B * Hq heads on
// B * Hkv kv heads (head h of sequence b reads kv head b * Hkv + h / group either way): one pass of launches
// instead of B.
rmm_attn_desc_t fold_batch(const rmm_attn_desc_t &d)
{
    rmm_attn_desc_t f = d;
    const bool even = d.B > 1 && d.Hkv >= 1 && d.Hq % d.Hkv == 0 && d.B * d.Hq <= 65535 &&
                      d.q_stride[0] == d.Hq * d.q_stride[1] && d.k_stride[0] == d.Hkv * d.k_stride[1] &&
                      d.v_stride[0] == d.Hkv * d.v_stride[1] && d.o_stride[0] == d.Hq * d.o_stride[1] &&
                      (d.mask == nullptr || d.mask_stride[0] == d.Hq * d.mask_stride[1]);
    if (even) {
        f.B = 1;
        f.Hq = d.B * d.Hq;
        f.Hkv = d.B * d.Hkv;
        f.q_stride[0] = f.Hq * d.q_stride[1];
        f.k_stride[0] = f.Hkv * d.k_stride[1];
        f.v_stride[0] = f.Hkv * d.v_stride[1];
        f.o_stride[0] = f.Hq * d.o_stride[1];
        f.mask_stride[0] = f.Hq * d.mask_stride[1];
    }
    return f;
}

int plan_attn(const rmm_attn_desc_t *d, AttnPlan *p)
{
    if (d == nullptr) return fail(RMM_ERR_INVALID_ARG, "reduced_attn: NULL description");
    if (d->B < 1 || d->Hq < 1 || d->Hkv < 1 || d->Lq < 1 || d->Lk < 1 || d->Dh < 1)
        return fail(RMM_ERR_INVALID_ARG, "reduced_attn: non-positive dimension");
    if (d->Hq % d->Hkv != 0) return fail(RMM_ERR_INVALID_ARG, "reduced_attn: Hq must be a multiple of Hkv");
    if (rmm_keep_count(d->rho_d, d->Dh, &p->kd) != RMM_OK || rmm_keep_count(d->rho_t, d->Lk, &p->kt) != RMM_OK)
        return fail(RMM_ERR_INVALID_ARG, "reduced_attn: rho_d and rho_t must lie in (0, 1]");
    if (d->Dh % 8 != 0) return fail(RMM_ERR_UNSUPPORTED, "reduced_attn: Dh must be a multiple of 8");
    if (d->Lq > INT32_MAX || d->Lk > INT32_MAX || d->Hq > 65535) return fail(RMM_ERR_UNSUPPORTED, "reduced_attn: too large");
    for (int i = 0; i < 3; ++i)
        if (d->q_stride[i] % 8 || d->k_stride[i] % 8 || d->v_stride[i] % 8 || d->o_stride[i] % 8)
            return fail(RMM_ERR_UNSUPPORTED, "reduced_attn: strides must be multiples of 8 elements");
    if (d->mask != nullptr && (d->mask_stride[0] < 0 || d->mask_stride[1] < 0 || d->mask_stride[2] < 0))
        return fail(RMM_ERR_INVALID_ARG, "reduced_attn: negative mask stride");
    // V's (batch, head) pairs must form one batch axis of the tensor map used when V is read in place
    if (d->v_stride[2] < d->Dh || d->v_stride[0] != d->Hkv * d->v_stride[1])
        return fail(RMM_ERR_UNSUPPORTED, "reduced_attn: V needs batch stride = Hkv * head stride");
    p->ldd = (p->kd + 7) / 8 * 8;
    p->ldt = (p->kt + 7) / 8 * 8;
    p->ld_p = (d->Lk + 7) / 8 * 8;
    p->ld_s = (d->Lk + 3) / 4 * 4;
    // heads per group: keep S~ (fp32) + P (bf16) + P[:, T] within about 6 GiB
    const double per_head = (double)d->Lq * ((double)p->ld_s * 4 + (double)p->ld_p * 2 + (double)p->ldt * 2);
    int64_t hg = (int64_t)(6.0 * 1073741824.0 / per_head);
    if (hg < 1) hg = 1;
    // the one-pass fused kernel also takes the caller's additive mask (rows 16-byte aligned); the three sweeps of the
    // token reduction take the causal mask only (their second sweep walks the mask by columns)
    const bool mask_ok = d->mask == nullptr ||
                         (d->rho_t >= 1.0 && reinterpret_cast<uintptr_t>(d->mask) % 16 == 0 && d->mask_stride[0] % 4 == 0 &&
                          d->mask_stride[1] % 4 == 0 && d->mask_stride[2] % 4 == 0);
    p->fused = mask_ok && use_fused(d, p->kd);
    if (hg > d->Hq || p->fused) hg = d->Hq;  // the fused form materialises neither S~ nor P: all heads at once
    p->hg = hg;

    // workspace of the inner score/select calls (the larger of the Q pass and the P pass)
    rmm_mat_t qm = {reinterpret_cast<void *>(uintptr_t(256)), RMM_BF16, hg, d->Lq, d->Dh, d->q_stride[1], d->q_stride[2], 1};
    rmm_mat_t pm = {reinterpret_cast<void *>(uintptr_t(256)), RMM_BF16, hg, d->Lq, d->Lk, d->Lq * p->ld_p, p->ld_p, 1};
    ScorePlan sq, sp;
    int rc = plan_score(&qm, 1, &sq);
    if (rc != RMM_OK) return rc;
    rc = plan_score(&pm, 1, &sp);
    if (rc != RMM_OK) return rc;
    p->inner_bytes = align_up(sq.total_bytes > sp.total_bytes ? sq.total_bytes : sp.total_bytes, 256);
    size_t off = p->inner_bytes;
    p->off_idxf = off; off += align_up((size_t)hg * p->kd * 4, 256);
    p->off_idxt = off; off += align_up((size_t)hg * p->kt * 4, 256);
    p->off_qp = off; off += align_up((size_t)hg * d->Lq * p->ldd * 2, 256);
    p->off_kp = off; off += align_up((size_t)hg * d->Lk * p->ldd * 2, 256);
    const size_t mat = p->fused ? 0 : 1;
    p->off_s = off; off += mat * align_up((size_t)hg * d->Lq * p->ld_s * 4, 256);
    p->off_p = off; off += mat * align_up((size_t)hg * d->Lq * p->ld_p * 2, 256);
    p->off_pp = off; off += mat * align_up((size_t)hg * d->Lq * p->ldt * 2, 256);
    p->off_vp = off; off += align_up((size_t)hg * p->kt * d->Dh * 2, 256);
    // fused token reduction: row normalisers, token scores, K[T]
    const size_t tokf = p->fused && d->rho_t < 1.0 ? 1 : 0;
    p->lse_ld = (d->Lq + 63) / 64 * 64;
    p->off_lse = off; off += tokf * align_up((size_t)hg * p->lse_ld * 4, 256);
    p->off_energy = off; off += tokf * align_up((size_t)hg * d->Lk * 4, 256);
    p->off_kpt = off; off += tokf * align_up((size_t)hg * p->kt * p->ldd * 2, 256);
    p->total = off;
    return RMM_OK;
}

}  // namespace

int launch_softmax_rows(const float *S, int64_t ld_s, int64_t heads, int64_t Lq, int64_t Lk, int causal, const float *mask,
                        int64_t m_sh, int64_t m_sr, __nv_bfloat16 *P, int64_t ld_p, cudaStream_t stream)
{
    dim3 grid((unsigned)Lq, (unsigned)heads);
    prof_begin("softmax_rows_kernel", stream);
    launch_kernel(softmax_rows_kernel, grid, dim3(kSoftmaxThreads), 0, stream, 1, S, ld_s, Lq, Lk, causal, mask, m_sh, m_sr, P,
                  ld_p);
    return check_launch("softmax_rows_kernel", stream);
}

}  // namespace rmm

using namespace rmm;

extern "C" {

size_t rmm_reduced_attn_workspace_bytes(const rmm_attn_desc_t *desc)
{
    AttnPlan p;
    if (desc == nullptr) return 0;
    const rmm_attn_desc_t folded = fold_batch(*desc);
    if (plan_attn(&folded, &p) != RMM_OK) return 0;
    return p.total;
}

int rmm_reduced_attn(const rmm_attn_desc_t *desc, const void *Q, const void *K, const void *V, void *O, int32_t *idx_feat,
                     int32_t *idx_tok, void *ws, size_t ws_bytes, void *stream)
{
    AttnPlan p;
    if (desc == nullptr) return fail(RMM_ERR_INVALID_ARG, "reduced_attn: NULL description");
    const rmm_attn_desc_t folded = fold_batch(*desc);
    const rmm_attn_desc_t *d = &folded;
    int rc = plan_attn(d, &p);
    if (rc != RMM_OK) return rc;
    if (Q == nullptr || K == nullptr || V == nullptr || O == nullptr) return fail(RMM_ERR_INVALID_ARG, "reduced_attn: NULL tensor");
    for (const void *ptr : {Q, K, V, (const void *)O})
        if (reinterpret_cast<uintptr_t>(ptr) % 16 != 0) return fail(RMM_ERR_UNSUPPORTED, "reduced_attn: tensors must be 16-byte aligned");
    if (ws == nullptr || reinterpret_cast<uintptr_t>(ws) % 256 != 0 || ws_bytes < p.total)
        return fail(RMM_ERR_WORKSPACE, "reduced_attn: workspace must be 256-byte aligned and hold %zu bytes", p.total);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *w = static_cast<char *>(ws);
    int *status = &reinterpret_cast<WsHeader *>(w)->status;
    const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(Q), *kk = static_cast<const __nv_bfloat16 *>(K),
                        *v = static_cast<const __nv_bfloat16 *>(V);
    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(O);
    __nv_bfloat16 *Qp = reinterpret_cast<__nv_bfloat16 *>(w + p.off_qp), *Kp = reinterpret_cast<__nv_bfloat16 *>(w + p.off_kp);
    __nv_bfloat16 *P = reinterpret_cast<__nv_bfloat16 *>(w + p.off_p), *Pp = reinterpret_cast<__nv_bfloat16 *>(w + p.off_pp);
    __nv_bfloat16 *Vp = reinterpret_cast<__nv_bfloat16 *>(w + p.off_vp);
    float *S = reinterpret_cast<float *>(w + p.off_s);
    const int64_t group = d->Hq / d->Hkv;
    const float scale = (float)(1.0 / sqrt((double)d->Dh));
    const bool tok = d->rho_t < 1.0;

    for (int64_t b = 0; b < d->B; ++b) {
        for (int64_t h0 = 0; h0 < d->Hq; h0 += p.hg) {
            const int64_t hg = d->Hq - h0 < p.hg ? d->Hq - h0 : p.hg;
            int32_t *If = idx_feat ? idx_feat + (b * d->Hq + h0) * p.kd : reinterpret_cast<int32_t *>(w + p.off_idxf);
            int32_t *It = idx_tok ? idx_tok + (b * d->Hq + h0) * p.kt : reinterpret_cast<int32_t *>(w + p.off_idxt);

            // feature scores on Q only, one index set per query head
            rmm_mat_t qm = {const_cast<__nv_bfloat16 *>(q + b * d->q_stride[0] + h0 * d->q_stride[1]), RMM_BF16, hg, d->Lq, d->Dh,
                            d->q_stride[1], d->q_stride[2], 1};
            ScorePlan sq;
            if ((rc = plan_score(&qm, 1, &sq)) != RMM_OK) return rc;
            if ((rc = launch_score_select(&qm, sq, true, p.kd, If, nullptr, nullptr, nullptr, w, st)) != RMM_OK) return rc;

            // Q[:, I_h] and K_{g(h)}[:, I_h]
            PackSpec qk[2];
            qk[0] = pack_cols_spec(static_cast<const __nv_bfloat16 *>(qm.ptr), hg, d->Lq, d->Dh, d->q_stride[1], d->q_stride[2], 0, 1,
                                   If, p.kd, p.kd, Qp, p.ldd);
            qk[1] = pack_cols_spec(kk + b * d->k_stride[0], hg, d->Lk, d->Dh, d->k_stride[1], d->k_stride[2], h0, group, If, p.kd,
                                   p.kd, Kp, p.ldd);
            if ((rc = launch_pack(qk, 2, status, st)) != RMM_OK) return rc;

            if (p.fused) {
                __nv_bfloat16 *og = o + b * d->o_stride[0] + h0 * d->o_stride[1];
                if (!tok) {
                    rc = launch_fused_attn(Qp, Kp, p.ldd, p.kd, v, d->v_stride[2], d->v_stride[1], d->B * d->Hkv, b * d->Hq + h0, group,
                                           og, d->o_stride[1], d->o_stride[2], hg, d->Lq, d->Lk, d->Dh, d->causal, d->Lk - d->Lq,
                                           nullptr, 0, nullptr,
                                           d->mask != nullptr ? d->mask + b * d->mask_stride[0] + h0 * d->mask_stride[1] : nullptr,
                                           d->mask_stride[1], d->mask_stride[2], status, st);
                    if (rc != RMM_OK) return rc;
                    continue;
                }
                float *lse = reinterpret_cast<float *>(w + p.off_lse), *energy = reinterpret_cast<float *>(w + p.off_energy);
                __nv_bfloat16 *KpT = reinterpret_cast<__nv_bfloat16 *>(w + p.off_kpt);
                // sweeps 1 and 2: row normalisers, then token scores of the bf16-rounded P; one token set per query head
                rc = launch_fused_attn_scores(Qp, Kp, p.ldd, p.kd, hg, d->Lq, d->Lk, d->Dh, d->causal, lse, p.lse_ld, energy, status, st);
                if (rc != RMM_OK) return rc;
                if ((rc = launch_select(energy, hg, d->Lk, p.kt, It, nullptr, w, st)) != RMM_OK) return rc;
                // K[T] (already reduced to the kept features) and V[T]
                PackSpec kv[2];
                kv[0] = pack_rows_spec(Kp, hg, d->Lk, p.ldd, d->Lk * p.ldd, p.ldd, 0, 1, It, p.kt, p.kt, KpT, p.ldd);
                kv[1] = pack_rows_spec(v + b * d->v_stride[0], hg, d->Lk, d->Dh, d->v_stride[1], d->v_stride[2], h0, group, It, p.kt,
                                       p.kt, Vp, d->Dh);
                if ((rc = launch_pack(kv, 2, status, st)) != RMM_OK) return rc;
                // sweep 3: O = P[:, T] V[T, :] against the full-row normalisers
                rc = launch_fused_attn(Qp, KpT, p.ldd, p.kd, Vp, d->Dh, p.kt * d->Dh, hg, 0, 1, og, d->o_stride[1], d->o_stride[2], hg,
                                       d->Lq, p.kt, d->Dh, d->causal, d->Lk - d->Lq, lse, p.lse_ld, It, nullptr, 0, 0, status, st);
                if (rc != RMM_OK) return rc;
                continue;
            }

            // S~ = Q[:, I] K[:, I]^T / sqrt(Dh)  (the scale keeps the full head dimension)
            TcProblem g1 = {};
            g1.batch = hg; g1.M = d->Lq; g1.N = d->Lk; g1.k = p.kd;
            g1.a = Qp; g1.a_ld = p.ldd; g1.a_sb = d->Lq * p.ldd;
            g1.b_kmajor = 1; g1.b = Kp; g1.b_ld = p.ldd; g1.b_sb = d->Lk * p.ldd;
            g1.b_batches = hg; g1.b_batch_off = 0; g1.b_batch_div = 1;
            g1.y = S; g1.y_bf16 = 0; g1.y_sb = d->Lq * p.ld_s; g1.y_sr = p.ld_s;
            g1.scale = scale; g1.status = status;
            if ((rc = launch_gemm_tc_problem(g1, st)) != RMM_OK) return rc;

            const float *mask = d->mask != nullptr ? d->mask + b * d->mask_stride[0] + h0 * d->mask_stride[1] : nullptr;
            if ((rc = launch_softmax_rows(S, p.ld_s, hg, d->Lq, d->Lk, d->causal, mask, d->mask_stride[1], d->mask_stride[2], P,
                                          p.ld_p, st)) != RMM_OK)
                return rc;

            TcProblem g2 = {};
            g2.batch = hg; g2.M = d->Lq; g2.N = d->Dh;
            g2.b_kmajor = 0;
            g2.y = o + b * d->o_stride[0] + h0 * d->o_stride[1]; g2.y_bf16 = 1; g2.y_sb = d->o_stride[1]; g2.y_sr = d->o_stride[2];
            g2.scale = 1.0f; g2.status = status;
            if (tok) {
                // token scores on the rounded P, one token set per query head, then O = P[:, T] V[T, :]
                rmm_mat_t pm = {P, RMM_BF16, hg, d->Lq, d->Lk, d->Lq * p.ld_p, p.ld_p, 1};
                ScorePlan sp;
                if ((rc = plan_score(&pm, 1, &sp)) != RMM_OK) return rc;
                if ((rc = launch_score_select(&pm, sp, true, p.kt, It, nullptr, nullptr, nullptr, w, st)) != RMM_OK) return rc;
                PackSpec pv[2];
                pv[0] = pack_cols_spec(P, hg, d->Lq, d->Lk, d->Lq * p.ld_p, p.ld_p, 0, 1, It, p.kt, p.kt, Pp, p.ldt);
                pv[1] = pack_rows_spec(v + b * d->v_stride[0], hg, d->Lk, d->Dh, d->v_stride[1], d->v_stride[2], h0, group, It, p.kt,
                                       p.kt, Vp, d->Dh);
                if ((rc = launch_pack(pv, 2, status, st)) != RMM_OK) return rc;
                g2.k = p.kt; g2.a = Pp; g2.a_ld = p.ldt; g2.a_sb = d->Lq * p.ldt;
                g2.b = Vp; g2.b_ld = d->Dh; g2.b_sb = p.kt * d->Dh; g2.b_batches = hg; g2.b_batch_off = 0; g2.b_batch_div = 1;
            } else {
                g2.k = d->Lk; g2.a = P; g2.a_ld = p.ld_p; g2.a_sb = d->Lq * p.ld_p;
                g2.b = v; g2.b_ld = d->v_stride[2]; g2.b_sb = d->v_stride[1]; g2.b_batches = d->B * d->Hkv;
                g2.b_batch_off = b * d->Hq + h0; g2.b_batch_div = group;
            }
            if ((rc = launch_gemm_tc_problem(g2, st)) != RMM_OK) return rc;
        }
    }
    return RMM_OK;
}

}  // extern "C"
