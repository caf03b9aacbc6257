/*
 * rmm_oracle.c — TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of Reduced Matrix Multiplication (RMM) used only to
 * check the CUDA library and to be timed beside it as a CPU baseline.  Only the tests,
 * the smoke check and the benchmark's cpu_baseline / reference arm may call it.  It
 * shares no code, header, table or helper with the CUDA path.
 *
 * What each function follows (section / equation of the paper):
 *   orc_keep_count     Sec. 3.2: |I| = ceil(rho * d), rho in (0, 1]
 *   orc_score          Sec. 3.2 "Activation-aware dimension selection": s_j = ||A[:, j]||_2
 *   orc_select         Sec. 3.2: I = TopK({s_j}, ceil(rho d)); Theorem 1 (App. "Minimax
 *                      Optimality"): the k columns of largest norm
 *   orc_reduced_gemm   Sec. 3.2: RMM_rho(A, B) = A[:, I] B[I, :]   (no rescaling)
 *   orc_dense_gemm     Sec. 3.1: Y = A B (the unreduced product; pins rho = 1)
 *   orc_attn           Sec. 3.3 "Attention": feature scores on Q, S~ = Q[:,I] K[:,I]^T / sqrt(d_h),
 *                      P = softmax(S~ + M), token scores a_t = ||P[:, t]||_2,
 *                      O~ = P[:, T] V[T, :]; grouped-query rule of the same paragraph
 *   orc_attn_sets      the same formulas of Sec. 3.3 evaluated on a feature set I and / or token set T that
 *                      the caller hands in (and, optionally, on a subset of the query rows)
 *
 * Readings taken where the paper is silent (all listed in the design document):
 *   - ties in TopK go to the lower index; the index set is reported ascending;
 *   - ceil(rho*K) is taken on the double product; a product within 4 ulps (4 * 2^-52 * rho*K) of an
 *     integer is that integer, which guards ratios such as 0.07 * 100 that are integral in exact
 *     arithmetic but land a hair above the integer in binary, and nothing else;
 *   - selection compares squared norms (monotone in the norm, no sqrt collapse);
 *   - the softmax scale keeps the full 1/sqrt(d_h); no renormalisation after dropping tokens;
 *   - P is rounded once to bf16 (round-to-nearest-even) before it is scored and multiplied
 *     (switchable, so that the unrounded form can be pinned to textbook attention);
 *   - causal mask aligned to the end: query i sees keys t <= i + (Lk - Lq);
 *   - kv head of query head h is h / (Hq / Hkv).
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py (rho = 1 equals the
 * dense product, brute-force subset enumeration, permutation invariance, rank-one closed
 * form, the error bounds of Eq. 2 / Eq. 4 / Eq. 6, nesting, the printed 70 % / 95 % example,
 * library matmul on pre-gathered operands, textbook attention).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_BF16 = 0, ORC_F32 = 1, ORC_F64 = 2 };

/* Widen one stored element to double, exactly. bf16 is the upper half of an IEEE binary32. */
static double orc_load(const void *base, int dtype, int64_t off)
{
    if (dtype == ORC_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[off] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    if (dtype == ORC_F32)
        return (double)((const float *)base)[off];
    return ((const double *)base)[off];
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0)
        omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Sec. 3.2: |I| = ceil(rho d), rho in (0,1].  Returns -1 for rho outside (0,1] or K < 1. */
int64_t orc_keep_count(double rho, int64_t K)
{
    if (!(rho > 0.0) || !(rho <= 1.0) || K < 1)
        return -1;
    double x = rho * (double)K;
    double r = nearbyint(x);
    int64_t k;
    /* rho and the product each carry at most half an ulp of rounding error, so a product that is integral in exact
     * arithmetic lands within a few ulps of that integer; anything further away is genuinely fractional */
    if (fabs(x - r) <= 4.0 * 2.220446049250313e-16 * x)
        k = (int64_t)r;
    else
        k = (int64_t)ceil(x);
    if (k < 1)
        k = 1;
    if (k > K)
        k = K;
    return k;
}

/*
 * Sec. 3.2: s_j = ||A[:, j]||_2 for a single M x K matrix with element strides (sr, sc).
 * energy[j] = sum_i A[i,j]^2 (Neumaier-compensated fp64), score[j] = sqrt(energy[j]).
 * Either output may be NULL.
 */
static void orc_column_energy(const void *A, int dtype, int64_t off0, int64_t M, int64_t K,
                              int64_t sr, int64_t sc, double *energy)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < K; ++j) {
        double sum = 0.0, comp = 0.0;
        for (int64_t i = 0; i < M; ++i) {
            double a = orc_load(A, dtype, off0 + i * sr + j * sc);
            double term = a * a;
            double t = sum + term;
            if (fabs(sum) >= fabs(term))
                comp += (sum - t) + term;
            else
                comp += (term - t) + sum;
            sum = t;
        }
        energy[j] = sum + comp;
    }
}

void orc_score(const void *A, int dtype, int64_t M, int64_t K, int64_t sr, int64_t sc,
               double *energy, double *score)
{
    double *e = energy ? energy : (double *)malloc((size_t)K * sizeof(double));
    orc_column_energy(A, dtype, 0, M, K, sr, sc, e);
    if (score)
        for (int64_t j = 0; j < K; ++j)
            score[j] = sqrt(e[j]);
    if (!energy)
        free(e);
}

typedef struct {
    double key;
    int32_t index;
} orc_pair;

static int orc_cmp_desc(const void *pa, const void *pb)
{
    const orc_pair *a = (const orc_pair *)pa, *b = (const orc_pair *)pb;
    if (a->key > b->key)
        return -1;
    if (a->key < b->key)
        return 1;
    return (a->index > b->index) - (a->index < b->index);
}

static int orc_cmp_i32(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/*
 * Sec. 3.2 / Theorem 1: the k indices of largest key; equal keys go to the lower index.
 * idx[0..k) is returned ascending.  Returns the retained key mass sum_{j in I} key_j
 * (with key = energy this is the numerator of 1 - eps_A(rho), Eq. 5).
 */
double orc_select(const double *key, int64_t K, int64_t k, int32_t *idx)
{
    orc_pair *p = (orc_pair *)malloc((size_t)K * sizeof *p);
    for (int64_t j = 0; j < K; ++j) {
        p[j].key = key[j];
        p[j].index = (int32_t)j;
    }
    qsort(p, (size_t)K, sizeof *p, orc_cmp_desc);
    double kept = 0.0;
    for (int64_t r = 0; r < k; ++r) {
        idx[r] = p[r].index;
        kept += p[r].key;
    }
    qsort(idx, (size_t)k, sizeof *idx, orc_cmp_i32);
    free(p);
    return kept;
}

/*
 * Sec. 3.2: Y = A[:, I] B[I, :], fp64, summed in the order idx lists the indices.
 * A is M x K with strides (sra, sca); B is K x N with strides (srb, scb); Y is M x N row-major.
 * Rows [row0, row1) only are computed (Y still indexed by absolute row), so that a caller can
 * time or check a sample of rows.
 */
void orc_reduced_gemm_rows(const void *A, int dta, int64_t M, int64_t K, int64_t sra, int64_t sca,
                           const void *B, int dtb, int64_t N, int64_t srb, int64_t scb,
                           const int32_t *idx, int64_t k, double *Y, int64_t row0, int64_t row1)
{
    (void)M;
    (void)K;
#pragma omp parallel for schedule(static)
    for (int64_t i = row0; i < row1; ++i) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t r = 0; r < k; ++r) {
                int64_t j = idx[r];
                acc += orc_load(A, dta, i * sra + j * sca) * orc_load(B, dtb, j * srb + n * scb);
            }
            Y[i * N + n] = acc;
        }
    }
}

void orc_reduced_gemm(const void *A, int dta, int64_t M, int64_t K, int64_t sra, int64_t sca,
                      const void *B, int dtb, int64_t N, int64_t srb, int64_t scb,
                      const int32_t *idx, int64_t k, double *Y)
{
    orc_reduced_gemm_rows(A, dta, M, K, sra, sca, B, dtb, N, srb, scb, idx, k, Y, 0, M);
}

/* Sec. 3.1: Y = A B with no index indirection at all (pins rho = 1). */
void orc_dense_gemm(const void *A, int dta, int64_t M, int64_t K, int64_t sra, int64_t sca,
                    const void *B, int dtb, int64_t N, int64_t srb, int64_t scb, double *Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t j = 0; j < K; ++j)
                acc += orc_load(A, dta, i * sra + j * sca) * orc_load(B, dtb, j * srb + n * scb);
            Y[i * N + n] = acc;
        }
    }
}

/* Round a double to the nearest bf16 (ties to even) and return it widened back to double. */
double orc_round_bf16(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x))
        return x;
    int e;
    double m = frexp(fabs(x), &e); /* |x| = m * 2^e, m in [0.5, 1) */
    /* bf16 has 8 significant bits; normal range down to 2^-126. */
    int shift = 8;
    if (e - 1 < -126)
        shift = 8 - (-126 - (e - 1));
    if (shift < 0)
        return copysign(0.0, x);
    double scaled = ldexp(m, shift);      /* in [2^(shift-1), 2^shift) */
    double r = nearbyint(scaled);         /* default rounding mode: nearest, ties to even */
    double y = ldexp(r, e - shift);
    if (y > 3.3895313892515355e38)        /* largest finite bf16 */
        y = INFINITY;
    return copysign(y, x);
}

/*
 * Sec. 3.3 "Attention", one call for all (batch, query head) pairs.
 *
 * Q  [B, Hq,  Lq, Dh], K,V [B, Hkv, Lk, Dh]: element strides (sb, sh, sl, sd) each.
 * Per (b, h):
 *   1. s_j = ||Q_h[:, j]||_2,  I = TopK(s, ceil(rho_d Dh))               -> idx_feat[b,h,:]
 *   2. S~[i,t] = (sum_{j in I} Q[i,j] K_g[t,j]) / sqrt(Dh), g = h / (Hq/Hkv)
 *   3. causal: t > i + (Lk - Lq) masked out;  P = softmax over t (fp64) of S~ + M
 *   4. if round_p: P <- bf16(P)
 *   5. if rho_t < 1: a_t = ||P[:, t]||_2, T = TopK(a, ceil(rho_t Lk))     -> idx_tok[b,h,:]
 *      O~ = P[:, T] V_g[T, :]  (no renormalisation); else O~ = P V_g
 *
 * Sec. 3.3 defines S~ and O~ for ANY feature set I and token set T; the TopK rule only says which sets RMM
 * picks.  So that a result can be judged on somebody else's sets (the same way orc_reduced_gemm takes idx),
 * either set may be handed in:
 *   idx_feat_in [B,Hq,kd] non-NULL: step 1 is skipped and I = idx_feat_in[b,h,:], used in the order given;
 *   idx_tok_in  [B,Hq,kt] non-NULL (rho_t < 1 only): the scoring of step 5 is skipped and T = idx_tok_in[b,h,:].
 * Every other step is unchanged.  The sets actually used are reported in idx_feat / idx_tok (either may be NULL).
 *
 * rows [n_rows] non-NULL: only these query rows are evaluated (steps 2-4 and the product of step 5 are row by
 * row, so nothing else changes); O is then [B, Hq, n_rows, Dh] and P_out [B, Hq, n_rows, Lk].  Token scores need
 * every row, so with rows given and rho_t < 1 the token set must be handed in; otherwise -1 is returned and
 * nothing is written.  Returns 0 on success.
 * mask non-NULL: the additive mask M of "P = softmax(S~ + M)" (Sec. 3.3), doubles, entry (b, h, i, t) at
 * mask[b sm[0] + h sm[1] + i sm[2] + t] (a stride of 0 shares the mask along that axis); -inf hides a key, and a
 * row whose keys are all hidden gives zeros, as under the causal mask.  It applies on top of `causal`.
 * O [B, Hq, Lq (or n_rows), Dh] contiguous doubles.
 * P_out, if non-NULL, receives P for every (b,h) as [B,Hq,Lq (or n_rows),Lk] doubles (small cases only).
 */
int orc_attn_sets(const void *Q, const void *Kt, const void *V, int dtype,
                  int64_t B, int64_t Hq, int64_t Hkv, int64_t Lq, int64_t Lk, int64_t Dh,
                  const int64_t *sq, const int64_t *sk, const int64_t *sv,
                  int causal, double rho_d, double rho_t, int round_p,
                  const int32_t *idx_feat_in, const int32_t *idx_tok_in,
                  const int64_t *rows, int64_t n_rows,
                  const double *mask, const int64_t *sm,
                  double *O, int32_t *idx_feat, int32_t *idx_tok, double *P_out)
{
    int64_t kd = orc_keep_count(rho_d, Dh);
    int64_t kt = orc_keep_count(rho_t, Lk);
    if (kd < 1 || kt < 1)
        return -1;
    if (rows != NULL && rho_t < 1.0 && idx_tok_in == NULL)
        return -1;
    int64_t nq = rows != NULL ? n_rows : Lq; /* query rows evaluated */
    int64_t group = Hq / Hkv;
    double scale = 1.0 / sqrt((double)Dh);
    double *P = (double *)malloc((size_t)nq * (size_t)Lk * sizeof(double));
    double *e_feat = (double *)malloc((size_t)Dh * sizeof(double));
    double *e_tok = (double *)malloc((size_t)Lk * sizeof(double));
    int32_t *I = (int32_t *)malloc((size_t)kd * sizeof(int32_t));
    int32_t *T = (int32_t *)malloc((size_t)kt * sizeof(int32_t));

    for (int64_t b = 0; b < B; ++b) {
        for (int64_t h = 0; h < Hq; ++h) {
            int64_t g = h / group;
            int64_t q0 = b * sq[0] + h * sq[1];
            int64_t k0 = b * sk[0] + g * sk[1];
            int64_t v0 = b * sv[0] + g * sv[1];

            /* 1. feature scores on Q only (all of its rows), and the feature set */
            if (idx_feat_in != NULL) {
                memcpy(I, idx_feat_in + (b * Hq + h) * kd, (size_t)kd * sizeof(int32_t));
            } else {
                orc_column_energy(Q, dtype, q0, Lq, Dh, sq[2], sq[3], e_feat);
                orc_select(e_feat, Dh, kd, I);
            }
            if (idx_feat)
                memcpy(idx_feat + (b * Hq + h) * kd, I, (size_t)kd * sizeof(int32_t));

            /* 2-4. reduced scores, mask, softmax, rounding */
#pragma omp parallel for schedule(static)
            for (int64_t ii = 0; ii < nq; ++ii) {
                int64_t i = rows != NULL ? rows[ii] : ii;
                double *row = P + ii * Lk;
                int64_t last = causal ? i + (Lk - Lq) : Lk - 1; /* last visible key */
                double mx = -INFINITY;
                for (int64_t t = 0; t < Lk; ++t) {
                    if (t > last) {
                        row[t] = -INFINITY;
                        continue;
                    }
                    double acc = 0.0;
                    for (int64_t r = 0; r < kd; ++r) {
                        int64_t j = I[r];
                        acc += orc_load(Q, dtype, q0 + i * sq[2] + j * sq[3]) *
                               orc_load(Kt, dtype, k0 + t * sk[2] + j * sk[3]);
                    }
                    row[t] = acc * scale;
                    if (mask != NULL) /* S~ + M: an additive mask entry, -inf hides the key */
                        row[t] += mask[b * sm[0] + h * sm[1] + i * sm[2] + t];
                    if (row[t] > mx)
                        mx = row[t];
                }
                double den = 0.0;
                for (int64_t t = 0; t < Lk; ++t) {
                    row[t] = (t > last || mx == -INFINITY) ? 0.0 : exp(row[t] - mx);
                    den += row[t];
                }
                for (int64_t t = 0; t < Lk; ++t) {
                    double p = (den > 0.0) ? row[t] / den : 0.0;
                    row[t] = round_p ? orc_round_bf16(p) : p;
                }
            }
            if (P_out)
                memcpy(P_out + (b * Hq + h) * nq * Lk, P, (size_t)nq * (size_t)Lk * sizeof(double));

            /* 5. token scores on the very P that is multiplied, and the token set */
            int64_t kt_used = Lk;
            if (rho_t < 1.0) {
                if (idx_tok_in != NULL) {
                    memcpy(T, idx_tok_in + (b * Hq + h) * kt, (size_t)kt * sizeof(int32_t));
                } else {
                    orc_column_energy(P, ORC_F64, 0, Lq, Lk, Lk, 1, e_tok);
                    orc_select(e_tok, Lk, kt, T);
                }
                kt_used = kt;
                if (idx_tok)
                    memcpy(idx_tok + (b * Hq + h) * kt, T, (size_t)kt * sizeof(int32_t));
            }

            double *Oh = O + (b * Hq + h) * nq * Dh;
#pragma omp parallel for schedule(static)
            for (int64_t i = 0; i < nq; ++i) {
                for (int64_t c = 0; c < Dh; ++c) {
                    double acc = 0.0;
                    for (int64_t r = 0; r < kt_used; ++r) {
                        int64_t t = (rho_t < 1.0) ? T[r] : r;
                        acc += P[i * Lk + t] * orc_load(V, dtype, v0 + t * sv[2] + c * sv[3]);
                    }
                    Oh[i * Dh + c] = acc;
                }
            }
        }
    }
    free(P);
    free(e_feat);
    free(e_tok);
    free(I);
    free(T);
    return 0;
}

/* The method as the paper states it: both sets chosen by the TopK rule, every query row evaluated. */
void orc_attn(const void *Q, const void *Kt, const void *V, int dtype,
              int64_t B, int64_t Hq, int64_t Hkv, int64_t Lq, int64_t Lk, int64_t Dh,
              const int64_t *sq, const int64_t *sk, const int64_t *sv,
              int causal, double rho_d, double rho_t, int round_p,
              double *O, int32_t *idx_feat, int32_t *idx_tok, double *P_out)
{
    (void)orc_attn_sets(Q, Kt, V, dtype, B, Hq, Hkv, Lq, Lk, Dh, sq, sk, sv, causal, rho_d, rho_t, round_p,
                        NULL, NULL, NULL, 0, NULL, NULL, O, idx_feat, idx_tok, P_out);
}
