// C ABI of the RMM library: argument checks, workspace layout and kernel dispatch.  No entry point
// allocates device memory or synchronises (rmm_status_read excepted, which is a blocking copy).
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace rmm {

static thread_local char t_error[512] = "";
std::atomic<int64_t> g_launches{0};

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_error, sizeof t_error, fmt, ap);
    va_end(ap);
    return code;
}

// Optional timing hook (rmm_profile_kernels): events recorded around launches whose name matches the filter.
static struct {
    cudaEvent_t *start = nullptr, *stop = nullptr;
    int capacity = 0, used = 0, every = 1, seen = 0;
    bool pending = false;
    char filter[64] = "";
    const char *names[4096];
} g_prof;

void prof_begin(const char *name, cudaStream_t stream)
{
    if (g_prof.used >= g_prof.capacity || g_prof.used >= 4096) return;
    if (g_prof.filter[0] != 0 && strstr(name, g_prof.filter) == nullptr) return;
    if (g_prof.seen++ % g_prof.every != 0) return;  // bracket one matching launch in `every`
    cudaEventRecord(g_prof.start[g_prof.used], stream);
    g_prof.names[g_prof.used] = name;
    g_prof.pending = true;
}

int check_launch(const char *what, cudaStream_t stream)
{
    if (g_prof.pending) {
        cudaEventRecord(g_prof.stop[g_prof.used++], stream);
        g_prof.pending = false;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "%s: launch failed: %s", what, cudaGetErrorString(e));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return RMM_OK;
}

int sm_count()
{
    static std::atomic<int> cached[64];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = -1;
    if (dev >= 0 && (n = cached[dev].load(std::memory_order_relaxed)) > 0) return n;
    if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

static std::atomic<unsigned long long> g_wait_override{0};  // rmm_debug_control("wait_limit_ms", ...): 0 = not set
static std::atomic<int> g_withhold_override{-1};             // rmm_debug_control("withhold", ...): -1 = not set

unsigned long long wait_limit_ns()
{
    static const unsigned long long limit = []() -> unsigned long long {
        const char *e = getenv("RMM_SPIN_LIMIT_MS");
        const double ms = e != nullptr ? atof(e) : 0.0;
        return ms > 0.0 ? (unsigned long long)(ms * 1e6) : 2000000000ull;
    }();
    const unsigned long long o = g_wait_override.load(std::memory_order_relaxed);
    return o != 0 ? o : limit;
}

int debug_withhold()
{
    const int o = g_withhold_override.load(std::memory_order_relaxed);
    if (o >= 0) return o;
    static const int which = []() {
        const char *e = getenv("RMM_TEST_WITHHOLD");
        if (e == nullptr) return 0;
        if (strcmp(e, "gemm") == 0) return (int)WITHHOLD_GEMM;
        if (strcmp(e, "score") == 0) return (int)WITHHOLD_SCORE;
        if (strcmp(e, "attn") == 0) return (int)WITHHOLD_ATTN;
        if (strcmp(e, "front") == 0) return (int)WITHHOLD_FRONT;
        if (strcmp(e, "pack") == 0) return (int)WITHHOLD_PACK;
        return 0;
    }();
    return which;
}

static int check_ws(void *ws, size_t ws_bytes, size_t need, const char *who)
{
    if (ws == nullptr) return fail(RMM_ERR_WORKSPACE, "%s: workspace is NULL (need %zu bytes)", who, need);
    if (reinterpret_cast<uintptr_t>(ws) % 256 != 0) return fail(RMM_ERR_WORKSPACE, "%s: workspace is not 256-byte aligned", who);
    if (ws_bytes < need) return fail(RMM_ERR_WORKSPACE, "%s: workspace has %zu bytes, needs %zu", who, ws_bytes, need);
    return RMM_OK;
}

static int check_mat(const rmm_mat_t *X, const char *who, const char *name)
{
    if (X == nullptr || X->ptr == nullptr) return fail(RMM_ERR_INVALID_ARG, "%s: %s is NULL", who, name);
    if (X->batch < 1 || X->rows < 1 || X->cols < 1)
        return fail(RMM_ERR_INVALID_ARG, "%s: %s has a non-positive dimension", who, name);
    if (X->dtype != RMM_BF16 && X->dtype != RMM_F32) return fail(RMM_ERR_UNSUPPORTED, "%s: %s has an unknown dtype", who, name);
    if (X->stride_batch < 0 || X->stride_row < 0 || X->stride_col < 0)
        return fail(RMM_ERR_UNSUPPORTED, "%s: %s has a negative stride", who, name);
    return RMM_OK;
}

static int resolve_k(double rho, int64_t k, int64_t K, int64_t *out, const char *who)
{
    if (k > 0) {
        if (k > K) return fail(RMM_ERR_INVALID_ARG, "%s: k = %lld exceeds K = %lld", who, (long long)k, (long long)K);
        *out = k;
        return RMM_OK;
    }
    if (k < 0) return fail(RMM_ERR_INVALID_ARG, "%s: k is negative", who);
    int rc = rmm_keep_count(rho, K, out);
    if (rc != RMM_OK) return fail(rc, "%s: rho = %g is outside (0, 1]", who, rho);
    return RMM_OK;
}

}  // namespace rmm

using namespace rmm;

extern "C" {

int rmm_keep_count(double rho, int64_t K, int64_t *k)
{
    if (k == nullptr || K < 1 || !(rho > 0.0) || !(rho <= 1.0))
        return fail(RMM_ERR_INVALID_ARG, "keep_count: need rho in (0, 1], K >= 1 and a non-NULL result");
    const double x = rho * (double)K;
    const double r = nearbyint(x);
    // the product of two doubles is off by at most a few ulps: only that close to an integer does it count as integral
    int64_t v = fabs(x - r) <= 4.0 * 2.220446049250313e-16 * x ? (int64_t)r : (int64_t)ceil(x);
    if (v < 1) v = 1;
    if (v > K) v = K;
    *k = v;
    return RMM_OK;
}

size_t rmm_score_workspace_bytes(const rmm_mat_t *A, int axis)
{
    ScorePlan p;
    if (plan_score(A, axis, &p) != RMM_OK) return 0;
    return p.total_bytes;
}

int rmm_score(const rmm_mat_t *A, int axis, float *scores, float *energy, void *ws, size_t ws_bytes, void *stream)
{
    ScorePlan p;
    int rc = plan_score(A, axis, &p);
    if (rc != RMM_OK) return rc;
    if (scores == nullptr && energy == nullptr) return fail(RMM_ERR_INVALID_ARG, "score: both outputs are NULL");
    rc = check_ws(ws, ws_bytes, p.total_bytes, "score");
    if (rc != RMM_OK) return rc;
    return launch_score_select(A, p, false, 0, nullptr, scores, energy, nullptr, ws, static_cast<cudaStream_t>(stream));
}

size_t rmm_select_workspace_bytes(int64_t batch, int64_t K)
{
    // the select keeps its keys in registers or shared memory (or re-reads them): only the header with the status word
    if (batch < 1 || K < 1 || K > (int64_t(1) << 30)) return 0;
    return RMM_WS_HEADER_BYTES;
}

int rmm_select(const float *keys, int64_t batch, int64_t K, double rho, int64_t k, int32_t *idx, float *retained,
               void *ws, size_t ws_bytes, void *stream)
{
    if (keys == nullptr || idx == nullptr) return fail(RMM_ERR_INVALID_ARG, "select: keys or idx is NULL");
    if (batch < 1 || K < 1) return fail(RMM_ERR_INVALID_ARG, "select: non-positive dimension");
    if (K > ((int64_t)1 << 30) || batch > INT32_MAX) return fail(RMM_ERR_UNSUPPORTED, "select: dimension too large");
    int64_t kk;
    int rc = resolve_k(rho, k, K, &kk, "select");
    if (rc != RMM_OK) return rc;
    rc = check_ws(ws, ws_bytes, RMM_WS_HEADER_BYTES, "select");
    if (rc != RMM_OK) return rc;
    return launch_select(keys, batch, K, kk, idx, retained, ws, static_cast<cudaStream_t>(stream));
}

size_t rmm_score_select_workspace_bytes(const rmm_mat_t *A, int axis) { return rmm_score_workspace_bytes(A, axis); }

int rmm_score_select(const rmm_mat_t *A, int axis, double rho, int64_t k, int32_t *idx, float *scores, float *energy,
                     float *retained, void *ws, size_t ws_bytes, void *stream)
{
    ScorePlan p;
    int rc = plan_score(A, axis, &p);
    if (rc != RMM_OK) return rc;
    if (idx == nullptr) return fail(RMM_ERR_INVALID_ARG, "score_select: idx is NULL");
    int64_t kk;
    rc = resolve_k(rho, k, p.n, &kk, "score_select");
    if (rc != RMM_OK) return rc;
    rc = check_ws(ws, ws_bytes, p.total_bytes, "score_select");
    if (rc != RMM_OK) return rc;
    return launch_score_select(A, p, true, kk, idx, scores, energy, retained, ws, static_cast<cudaStream_t>(stream));
}

static int check_gemm(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, const rmm_mat_t *Y)
{
    int rc;
    if ((rc = check_mat(A, "reduced_gemm", "A")) != RMM_OK) return rc;
    if ((rc = check_mat(B, "reduced_gemm", "B")) != RMM_OK) return rc;
    if ((rc = check_mat(Y, "reduced_gemm", "Y")) != RMM_OK) return rc;
    if (idx == nullptr && k != A->cols)
        return fail(RMM_ERR_INVALID_ARG, "reduced_gemm: idx is NULL (allowed only with k == K, the unreduced product)");
    if (A->cols != B->rows) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm: A has %lld columns but B has %lld rows",
                                        (long long)A->cols, (long long)B->rows);
    if (Y->rows != A->rows || Y->cols != B->cols || Y->batch != A->batch)
        return fail(RMM_ERR_INVALID_ARG, "reduced_gemm: Y must be [batch of A, rows of A, columns of B]");
    if (B->batch != A->batch && !(B->batch == 1))
        return fail(RMM_ERR_INVALID_ARG, "reduced_gemm: B must have A's batch or batch 1");
    if (k < 1 || k > A->cols) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm: k = %lld is outside [1, K]", (long long)k);
    if (A->dtype != B->dtype) return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm: A and B must share a dtype");
    if (Y->stride_batch == 0 && Y->batch > 1) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm: Y batches overlap");
    return RMM_OK;
}

// B with batch 1 is shared by every batch element of A: normalise its batch stride to 0.
static rmm_mat_t shared_b(const rmm_mat_t *A, const rmm_mat_t *B)
{
    rmm_mat_t b = *B;
    if (B->batch == 1 && A->batch >= 1) b.stride_batch = 0;
    b.batch = A->batch;
    return b;
}

size_t rmm_reduced_gemm_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y)
{
    if (A == nullptr || B == nullptr || Y == nullptr) return 0;
    rmm_mat_t b = shared_b(A, B);
    GemvPlan gplan;
    if (gemv_eligible(A, &b, k, Y, &gplan)) return gplan.total_bytes;
    TcPlan plan;
    if (tc_eligible(A, &b, k, Y, &plan)) return plan.total_bytes;
    return RMM_WS_HEADER_BYTES;
}

int rmm_reduced_gemm(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                     const rmm_mat_t *Y, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_gemm(A, B, idx, k, Y);
    if (rc != RMM_OK) return rc;
    rmm_mat_t b = shared_b(A, B);
    GemvPlan gplan;
    if (gemv_eligible(A, &b, k, Y, &gplan)) {  // decode-step shapes: only the kept rows of B are read
        rc = check_ws(ws, ws_bytes, gplan.total_bytes, "reduced_gemm");
        if (rc != RMM_OK) return rc;
        return launch_gemv(A, &b, idx, k, scale, Y, gplan, ws, static_cast<cudaStream_t>(stream));
    }
    TcPlan plan;
    if (tc_eligible(A, &b, k, Y, &plan)) {
        rc = check_ws(ws, ws_bytes, plan.total_bytes, "reduced_gemm");
        if (rc != RMM_OK) return rc;
        return launch_gemm_tc(A, &b, idx, k, scale, Y, plan, ws, static_cast<cudaStream_t>(stream));
    }
    rc = check_ws(ws, ws_bytes, RMM_WS_HEADER_BYTES, "reduced_gemm");
    if (rc != RMM_OK) return rc;
    return launch_gemm_simt(A, &b, idx, k, scale, Y, ws, static_cast<cudaStream_t>(stream));
}

// ---- 8-bit operands -------------------------------------------------------------------------------------
struct Q8Plan {
    int64_t ldq;
    size_t off_aq, off_bq, off_scale, total;
};

static int plan_q8(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y, Q8Plan *q)
{
    if (A == nullptr || B == nullptr || Y == nullptr || A->ptr == nullptr || B->ptr == nullptr || Y->ptr == nullptr)
        return fail(RMM_ERR_INVALID_ARG, "reduced_gemm_q8: NULL matrix");
    if (A->batch != 1 || B->batch != 1 || Y->batch != 1) return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm_q8: one product per call (batch 1)");
    if (A->rows < 1 || A->cols < 1 || B->cols < 1) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm_q8: non-positive dimension");
    if (A->dtype != RMM_BF16 || B->dtype != RMM_F8E4M3) return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm_q8: A must be bf16 and B e4m3 codes");
    if (Y->dtype != RMM_BF16 && Y->dtype != RMM_F32) return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm_q8: Y must be bf16 or fp32");
    if (A->cols != B->rows || Y->rows != A->rows || Y->cols != B->cols) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm_q8: shapes do not agree");
    if (k < 1 || k > A->cols) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm_q8: k = %lld is outside [1, K]", (long long)k);
    auto al16 = [](const void *p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; };
    const int64_t yq = Y->dtype == RMM_BF16 ? 8 : 4;
    if (A->stride_col != 1 || A->stride_row % 8 != 0 || !al16(A->ptr) || B->stride_row != 1 || B->stride_col % 16 != 0 || !al16(B->ptr) ||
        Y->stride_col != 1 || Y->stride_row % yq != 0 || !al16(Y->ptr) || A->rows > INT32_MAX || B->cols > INT32_MAX)
        return fail(RMM_ERR_UNSUPPORTED, "reduced_gemm_q8: operands must have contiguous, 16-byte aligned contraction rows");
    q->ldq = (k + 15) / 16 * 16;
    size_t off = RMM_WS_HEADER_BYTES;
    q->off_aq = off; off += align_up((size_t)A->rows * q->ldq, 256);
    q->off_bq = off; off += align_up((size_t)B->cols * q->ldq, 256);
    q->off_scale = off; off += align_up((size_t)A->rows * 4, 256);
    q->total = off;
    return RMM_OK;
}

size_t rmm_reduced_gemm_q8_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y)
{
    Q8Plan q = {};
    return plan_q8(A, B, k, Y, &q) == RMM_OK ? q.total : 0;
}

int rmm_reduced_gemm_q8(const rmm_mat_t *A, const rmm_mat_t *B, float b_scale, const int32_t *idx, int64_t k, float scale,
                        const rmm_mat_t *Y, float *a_scale, void *ws, size_t ws_bytes, void *stream)
{
    Q8Plan q = {};
    int rc = plan_q8(A, B, k, Y, &q);
    if (rc != RMM_OK) return rc;
    if (idx == nullptr) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm_q8: idx is NULL");
    rc = check_ws(ws, ws_bytes, q.total, "reduced_gemm_q8");
    if (rc != RMM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *w = static_cast<char *>(ws);
    int *status = &reinterpret_cast<WsHeader *>(w)->status;
    uint8_t *Aq = reinterpret_cast<uint8_t *>(w + q.off_aq), *Bq = reinterpret_cast<uint8_t *>(w + q.off_bq);
    float *row_scale = a_scale != nullptr ? a_scale : reinterpret_cast<float *>(w + q.off_scale);
    rc = launch_gather_q8(true, A->ptr, A->rows, A->stride_row, A->cols, idx, k, Aq, q.ldq, row_scale, status, st);
    if (rc != RMM_OK) return rc;
    rc = launch_gather_q8(false, B->ptr, B->cols, B->stride_col, B->rows, idx, k, Bq, q.ldq, nullptr, status, st);
    if (rc != RMM_OK) return rc;
    TcProblem p = {};
    p.batch = 1; p.M = A->rows; p.N = B->cols; p.k = k;
    p.fp8 = 1; p.row_scale = row_scale;
    p.a = reinterpret_cast<const __nv_bfloat16 *>(Aq); p.a_ld = q.ldq; p.a_sb = A->rows * q.ldq;
    p.b_kmajor = 1;
    p.b = reinterpret_cast<const __nv_bfloat16 *>(Bq); p.b_ld = q.ldq; p.b_sb = B->cols * q.ldq; p.b_batches = 1;
    p.b_batch_off = 0; p.b_batch_div = 1;
    p.y = Y->ptr; p.y_bf16 = Y->dtype == RMM_BF16; p.y_sb = Y->stride_batch; p.y_sr = Y->stride_row;
    p.scale = scale * b_scale;
    p.status = status;
    return launch_gemm_tc_problem(p, st);
}

// ---- product that also scores its output ---------------------------------------------------------------
size_t rmm_reduced_gemm_scored_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y)
{
    if (A == nullptr || B == nullptr || Y == nullptr) return 0;
    rmm_mat_t b = shared_b(A, B);
    GemvPlan gplan;
    TcPlan plan;
    size_t need;
    if (!gemv_eligible(A, &b, k, Y, &gplan) && tc_eligible(A, &b, k, Y, &plan, true)) {
        if (plan.epilogue_energy) return plan.total_bytes;
        need = plan.total_bytes;
    } else {
        need = rmm_reduced_gemm_workspace_bytes(A, B, k, Y);
    }
    const size_t s = rmm_score_workspace_bytes(Y, 1);  // the output is scored by a pass of its own
    if (need == 0 || s == 0) return 0;
    return need > s ? need : s;
}

int rmm_reduced_gemm_scored(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale, const rmm_mat_t *Y,
                            float *energy_out, void *ws, size_t ws_bytes, void *stream)
{
    if (energy_out == nullptr) return fail(RMM_ERR_INVALID_ARG, "reduced_gemm_scored: energy_out is NULL");
    int rc = check_gemm(A, B, idx, k, Y);
    if (rc != RMM_OK) return rc;
    rmm_mat_t b = shared_b(A, B);
    GemvPlan gplan;
    TcPlan plan;
    if (!gemv_eligible(A, &b, k, Y, &gplan) && tc_eligible(A, &b, k, Y, &plan, true) && plan.epilogue_energy) {
        rc = check_ws(ws, ws_bytes, plan.total_bytes, "reduced_gemm_scored");
        if (rc != RMM_OK) return rc;
        return launch_gemm_tc(A, &b, idx, k, scale, Y, plan, ws, static_cast<cudaStream_t>(stream), energy_out);
    }
    // every other form of the product: the output is scored by the ordinary pass once it has been written
    rc = check_ws(ws, ws_bytes, rmm_reduced_gemm_scored_workspace_bytes(A, B, k, Y), "reduced_gemm_scored");
    if (rc != RMM_OK) return rc;
    rc = rmm_reduced_gemm(A, B, idx, k, scale, Y, ws, ws_bytes, stream);
    if (rc != RMM_OK) return rc;
    return rmm_score(Y, 1, nullptr, energy_out, ws, ws_bytes, stream);
}

// ---- whole operation on device operands ------------------------------------------------------------
struct ProductPlan {
    bool fused;
    FrontPlan front;
    size_t total;
};

static int plan_product(const rmm_mat_t *A, const rmm_mat_t *B, const rmm_mat_t *Y, int64_t k, ProductPlan *pp)
{
    rmm_mat_t b = shared_b(A, B);
    pp->fused = k < A->cols && front_eligible(A, &b, Y, k, &pp->front);
    if (pp->fused) {
        pp->total = pp->front.total_bytes;
        return RMM_OK;
    }
    const size_t s1 = rmm_score_select_workspace_bytes(A, 1);
    const size_t s2 = rmm_reduced_gemm_workspace_bytes(A, B, k, Y);
    if (s1 == 0 || s2 == 0) return RMM_ERR_UNSUPPORTED;
    pp->total = s1 > s2 ? s1 : s2;
    return RMM_OK;
}

size_t rmm_product_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, const rmm_mat_t *Y)
{
    if (A == nullptr || B == nullptr || Y == nullptr || A->cols < 1) return 0;
    // k = K bounds every k, for the two-call form and for the one-launch front end alike
    const size_t s1 = rmm_score_select_workspace_bytes(A, 1), s2 = rmm_reduced_gemm_workspace_bytes(A, B, A->cols, Y);
    if (s1 == 0 || s2 == 0) return 0;
    size_t need = s1 > s2 ? s1 : s2;
    rmm_mat_t b = shared_b(A, B);
    FrontPlan fp;
    if (front_eligible(A, &b, Y, A->cols, &fp) && fp.total_bytes > need) need = fp.total_bytes;
    return need;
}

int rmm_product(const rmm_mat_t *A, const rmm_mat_t *B, double rho, int64_t k, float scale, const rmm_mat_t *Y, int32_t *idx,
                float *retained, void *ws, size_t ws_bytes, void *stream)
{
    if (A == nullptr || A->ptr == nullptr || A->cols < 1) return fail(RMM_ERR_INVALID_ARG, "product: A is NULL or empty");
    if (idx == nullptr) return fail(RMM_ERR_INVALID_ARG, "product: idx is NULL");
    int64_t kk;
    int rc = resolve_k(rho, k, A->cols, &kk, "product");
    if (rc != RMM_OK) return rc;
    rc = check_gemm(A, B, idx, kk, Y);
    if (rc != RMM_OK) return rc;
    ProductPlan pp;
    rc = plan_product(A, B, Y, kk, &pp);
    if (rc != RMM_OK) return fail(rc, "product: operands not covered");
    rc = check_ws(ws, ws_bytes, pp.total, "product");
    if (rc != RMM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (kk == A->cols) {
        // every index is kept: the list is 0 .. K-1 (written by the selection, which also gives `retained`), and the product
        // is the unreduced one, which needs no gather at all
        rc = rmm_score_select(A, 1, rho, kk, idx, nullptr, nullptr, retained, ws, ws_bytes, stream);
        if (rc != RMM_OK) return rc;
        return rmm_reduced_gemm(A, B, nullptr, kk, scale, Y, ws, ws_bytes, stream);
    }
    if (!pp.fused) {
        rc = rmm_score_select(A, 1, rho, kk, idx, nullptr, nullptr, retained, ws, ws_bytes, stream);
        if (rc != RMM_OK) return rc;
        return rmm_reduced_gemm(A, B, idx, kk, scale, Y, ws, ws_bytes, stream);
    }
    rmm_mat_t b = shared_b(A, B);
    rc = launch_front(A, &b, kk, idx, nullptr, retained, pp.front, ws, st);
    if (rc != RMM_OK) return rc;
    char *w = static_cast<char *>(ws);
    TcProblem p = {};
    p.batch = 1; p.M = A->rows; p.N = B->cols; p.k = kk;
    p.a = reinterpret_cast<const __nv_bfloat16 *>(w + pp.front.off_ap); p.a_ld = pp.front.ldp; p.a_sb = A->rows * pp.front.ldp;
    p.b_kmajor = 0;
    p.b = reinterpret_cast<const __nv_bfloat16 *>(w + pp.front.off_bp); p.b_ld = B->cols; p.b_sb = kk * B->cols; p.b_batches = 1;
    p.b_batch_off = 0; p.b_batch_div = 1;
    p.y = Y->ptr; p.y_bf16 = Y->dtype == RMM_BF16; p.y_sb = Y->stride_batch; p.y_sr = Y->stride_row;
    p.scale = scale;
    p.status = &reinterpret_cast<WsHeader *>(w)->status;
    return launch_gemm_tc_problem(p, st);
}

// ---- whole operation on host buffers -------------------------------------------------------------
struct HostPlan {
    size_t off_a, off_b, off_y, off_idx, off_inner, inner_bytes, total;
    rmm_mat_t A, B, Y;
};

static int plan_host(int64_t M, int64_t K, int64_t N, void *ws, HostPlan *h)
{
    if (M < 1 || K < 1 || N < 1) return fail(RMM_ERR_INVALID_ARG, "product_host: non-positive dimension");
    size_t off = 0;
    h->off_inner = off;  // the inner calls' workspace comes first so that its header is the status word
    char *w = static_cast<char *>(ws);
    rmm_mat_t A = {nullptr, RMM_BF16, 1, M, K, M * K, K, 1};
    rmm_mat_t B = {nullptr, RMM_BF16, 1, K, N, K * N, N, 1};
    rmm_mat_t Y = {nullptr, RMM_BF16, 1, M, N, M * N, N, 1};
    // sizes that do not depend on the pointers: use aligned dummies for the planners
    A.ptr = B.ptr = Y.ptr = reinterpret_cast<void *>(uintptr_t(256));
    size_t s1 = rmm_product_workspace_bytes(&A, &B, &Y);
    if (s1 == 0) return RMM_ERR_UNSUPPORTED;
    h->inner_bytes = align_up(s1, 256);
    off += h->inner_bytes;
    h->off_a = off; off += align_up((size_t)M * K * 2, 256);
    h->off_b = off; off += align_up((size_t)K * N * 2, 256);
    h->off_y = off; off += align_up((size_t)M * N * 2, 256);
    h->off_idx = off; off += align_up((size_t)K * 4, 256);
    h->total = off;
    A.ptr = w ? w + h->off_a : nullptr;
    B.ptr = w ? w + h->off_b : nullptr;
    Y.ptr = w ? w + h->off_y : nullptr;
    h->A = A; h->B = B; h->Y = Y;
    return RMM_OK;
}

size_t rmm_product_host_workspace_bytes(int64_t M, int64_t K, int64_t N)
{
    HostPlan h;
    if (plan_host(M, K, N, nullptr, &h) != RMM_OK) return 0;
    return h.total;
}

int rmm_product_host(const void *A_host, const void *B_host, int64_t M, int64_t K, int64_t N, double rho, int copy_B,
                     void *Y_host, int32_t *idx_host, void *ws, size_t ws_bytes, void *stream)
{
    if (A_host == nullptr || Y_host == nullptr || (copy_B && B_host == nullptr))
        return fail(RMM_ERR_INVALID_ARG, "product_host: NULL host buffer");
    HostPlan h;
    int rc = plan_host(M, K, N, ws, &h);
    if (rc != RMM_OK) return rc;
    rc = check_ws(ws, ws_bytes, h.total, "product_host");
    if (rc != RMM_OK) return rc;
    int64_t k;
    rc = resolve_k(rho, 0, K, &k, "product_host");
    if (rc != RMM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *w = static_cast<char *>(ws);
    int32_t *idx = reinterpret_cast<int32_t *>(w + h.off_idx);
    cudaError_t e = cudaMemcpyAsync(h.A.ptr, A_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && copy_B) e = cudaMemcpyAsync(h.B.ptr, B_host, (size_t)K * N * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "product_host: host-to-device copy: %s", cudaGetErrorString(e));
    rc = rmm_product(&h.A, &h.B, rho, k, 1.0f, &h.Y, idx, nullptr, w + h.off_inner, h.inner_bytes, stream);
    if (rc != RMM_OK) return rc;
    e = cudaMemcpyAsync(Y_host, h.Y.ptr, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && idx_host != nullptr)
        e = cudaMemcpyAsync(idx_host, idx, (size_t)k * 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "product_host: device-to-host copy: %s", cudaGetErrorString(e));
    return RMM_OK;
}

int rmm_status_read(void *ws, int *device_status)
{
    if (ws == nullptr || device_status == nullptr) return fail(RMM_ERR_INVALID_ARG, "status_read: NULL argument");
    int v = 0;
    cudaError_t e = cudaMemcpy(&v, ws, sizeof v, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "status_read: %s", cudaGetErrorString(e));
    if (v != 0) {
        // a kernel that gave up may have left arrival counters half way: the whole header starts from zero again
        e = cudaMemset(ws, 0, RMM_WS_HEADER_BYTES);
        if (e != cudaSuccess) return fail(RMM_ERR_CUDA, "status_read: %s", cudaGetErrorString(e));
    }
    *device_status = v;
    return RMM_OK;
}

int rmm_debug_control(const char *key, double value)
{
    if (key == nullptr) return fail(RMM_ERR_INVALID_ARG, "debug_control: NULL key");
    if (strcmp(key, "wait_limit_ms") == 0) {
        if (!(value >= 0.0) || value > 60000.0) return fail(RMM_ERR_INVALID_ARG, "debug_control: wait_limit_ms must be in [0, 60000]");
        g_wait_override.store((unsigned long long)(value * 1e6), std::memory_order_relaxed);
        return RMM_OK;
    }
    if (strcmp(key, "withhold") == 0) {
        const int w = (int)value;
        if (w < -1 || w > WITHHOLD_PACK) return fail(RMM_ERR_INVALID_ARG, "debug_control: withhold must be -1 .. %d", (int)WITHHOLD_PACK);
        g_withhold_override.store(w, std::memory_order_relaxed);
        return RMM_OK;
    }
    return fail(RMM_ERR_INVALID_ARG, "debug_control: unknown key '%s'", key);
}

int rmm_profile_kernels(void **start_events, void **stop_events, int n, const char *name_filter, int every)
{
    if (n < 0 || n > 4096 || ((start_events == nullptr || stop_events == nullptr) && n != 0))
        return fail(RMM_ERR_INVALID_ARG, "profile_kernels: need two event arrays and 0 <= n <= 4096, or NULL, NULL, 0");
    g_prof.every = every > 1 ? every : 1;
    g_prof.seen = 0;
    g_prof.start = reinterpret_cast<cudaEvent_t *>(start_events);
    g_prof.stop = reinterpret_cast<cudaEvent_t *>(stop_events);
    g_prof.capacity = n;
    g_prof.used = 0;
    g_prof.pending = false;
    snprintf(g_prof.filter, sizeof g_prof.filter, "%s", name_filter ? name_filter : "");
    return RMM_OK;
}

int rmm_profile_count(void) { return g_prof.used; }

const char *rmm_profile_name(int i) { return (i >= 0 && i < g_prof.used) ? g_prof.names[i] : ""; }

const char *rmm_last_error(void) { return t_error; }

int64_t rmm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
