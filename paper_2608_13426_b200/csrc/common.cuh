// Shared declarations of the RMM library's translation units (internal; the public ABI is rmm.h).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "rmm.h"

struct CUtensorMap_st;  // the driver API's tensor-map type (cuda.h); opaque here

namespace rmm {

// ---- error text (thread-local) and launch accounting -------------------------------------------
int fail(int code, const char *fmt, ...);
extern std::atomic<int64_t> g_launches;
void prof_begin(const char *kernel_name, cudaStream_t stream);  // call right before a launch (timing hook)
int check_launch(const char *what, cudaStream_t stream);  // right after: cudaGetLastError -> status, counts the launch

// Every kernel is launched with programmatic stream serialization allowed: its blocks may be scheduled, and run
// their set-up (barrier initialisation, descriptor prefetch, TMEM allocation), while the previous kernel on the stream
// drains.  A kernel touches global memory only after pdl_wait(), which returns once the previous grid has completed
// and its writes are visible, so results do not depend on the overlap.  cluster_x > 1 adds a cluster dimension.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                        int cluster_x, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
// Let the next kernel on the stream start its set-up, then wait for the previous kernel's results.
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

// Function attributes (the opt-in to more than 48 KB of dynamic shared memory) belong to a device: a flag per device
// and call site says whether the current device has been set up.  Returns true exactly once per device.
struct PerDeviceOnce {
    std::atomic<bool> done[64];
    bool first()
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;  // unknown: set up every time
        return !done[dev].exchange(true);
    }
};

int sm_count();                      // multiprocessors of the current device
unsigned long long wait_limit_ns();  // bound of every device-side wait: 2 s, or RMM_SPIN_LIMIT_MS from the environment
// Test switch (environment RMM_TEST_WITHHOLD = gemm | score | attn | front | pack, read once): block 0 of that kernel
// family never requests its first tile, so the waits behind it run out and the kernel's give-up path runs.  0 = off.
enum { WITHHOLD_GEMM = 1, WITHHOLD_SCORE = 2, WITHHOLD_ATTN = 3, WITHHOLD_FRONT = 4, WITHHOLD_PACK = 5 };
int debug_withhold();

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline size_t dtype_size(int dt) { return dt == RMM_BF16 ? 2 : (dt == RMM_F8E4M3 ? 1 : 4); }

// ---- TMA tensor map for a bf16 tensor: dims / box innermost first, strides in bytes for dims 1..rank-1; 128-byte
// swizzle or none.  `map` points to a CUtensorMap (opaque here so that only the users include <cuda.h>).
int make_map(::CUtensorMap_st *map, void *ptr, int rank, const uint64_t *dims, const uint64_t *strides_bytes,
             const uint32_t *box, bool swizzle128, int elem_bytes = 2);

// ---- workspace header: status word, then self-resetting arrival counters --------------------------
struct WsHeader {
    int status;  // rmm_status_t written by kernels (0 = ok)
    int pad[15];
    unsigned counters[(RMM_WS_HEADER_BYTES - 64) / 4];
};
static_assert(sizeof(WsHeader) == RMM_WS_HEADER_BYTES, "header size");
constexpr int64_t kHeaderCounters = (RMM_WS_HEADER_BYTES - 64) / 4;

// ---- score + select ---------------------------------------------------------------------------------
struct ScorePlan {
    int vec;         // elements per load: 8 (bf16, 16 B), 4 (fp32, 16 B) or 1 (generic strides)
    int tx, ty;      // thread layout: tx column groups x ty row lanes, tx * ty = 256
    int col_blocks;  // ceil(n / (tx * vec))
    int row_splits;  // row ranges summed by separate blocks
    int64_t rows_per_split;
    int64_t n, m;    // scored axis length, reduced axis length
    int64_t s_batch, s_red, s_n;  // element strides: batch, reduced axis, scored axis
    size_t off_counters, off_partials, off_energy, total_bytes;
    bool counters_in_header;
    bool use_tma;    // rows streamed through shared memory by TMA (bf16, 64-column blocks)
};
int plan_score(const rmm_mat_t *A, int axis, ScorePlan *plan);
int launch_score_select(const rmm_mat_t *A, const ScorePlan &p, bool do_select, int64_t k, int32_t *idx,
                        float *scores, float *energy, float *retained, void *ws, cudaStream_t stream);
int launch_select(const float *keys, int64_t batch, int64_t K, int64_t k, int32_t *idx, float *retained, void *ws,
                  cudaStream_t stream);

// Front end of a whole product in one launch (scores, selection, packed A[:, I] and B[I, :]); see score_select.cu.
struct FrontPlan {
    int col_blocks;
    int64_t ldp;  // row pitch of the packed A (multiple of 8)
    size_t off_energy, off_ap, off_bp, total_bytes;
};
bool front_eligible(const rmm_mat_t *A, const rmm_mat_t *B, const rmm_mat_t *Y, int64_t k, FrontPlan *plan);
int launch_front(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, int32_t *idx, float *energy, float *retained,
                 const FrontPlan &plan, void *ws, cudaStream_t stream);

// ---- reduced GEMM ------------------------------------------------------------------------------------
// Plain FMA kernel: any strides, bf16 or fp32 operands, fp32 accumulation, bf16 or fp32 output.
int launch_gemm_simt(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                     const rmm_mat_t *Y, void *ws, cudaStream_t stream);

// Decode-step path (M <= 4 rows of bf16 activations, B rows contiguous): HBM-bound gathered GEMV, no packing.
struct GemvPlan {
    int splits, rows_per_split;
    size_t off_partials, total_bytes;
};
bool gemv_eligible(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y, GemvPlan *plan);
int launch_gemv(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale, const rmm_mat_t *Y,
                const GemvPlan &plan, void *ws, cudaStream_t stream);

// Tensor-core path (tcgen05, TMEM accumulators).  Operands must satisfy tc_eligible().
struct TcPlan {
    int b_kmajor;       // 0: B rows (contraction slices) contiguous, kept rows copied; 1: B is K-contiguous, packed like A
    int64_t ldp;        // leading dimension of the packed operands (multiple of 8)
    size_t off_ap, off_bp, off_colen, total_bytes;
    bool epilogue_energy;  // the plan reserves the per-group column energies of Y and the epilogue fills them
};
bool tc_eligible(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y, TcPlan *plan, bool with_energy = false);
// energy_out (with a plan made with_energy): also energy_out[b, c] = sum_i Y[b, i, c]^2 of the rounded outputs
int launch_gemm_tc(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                   const rmm_mat_t *Y, const TcPlan &plan, void *ws, cudaStream_t stream, float *energy_out = nullptr);

// A tensor-core problem on operands that are already in TMA-loadable form.
struct TcProblem {
    int64_t batch, M, N, k;
    const __nv_bfloat16 *a;  // K-major A [batch, M, a_ld]: the kept columns are its first k columns
    int64_t a_ld, a_sb;      // row pitch and batch stride in elements (multiples of 8)
    int b_kmajor;
    const __nv_bfloat16 *b;  // K-major: [b_batches, N, b_ld] (kept columns first); MN-major: [b_batches, k, b_ld], rows = kept slices
    int64_t b_ld, b_sb, b_batches;
    int64_t b_batch_off, b_batch_div;  // B batch entry used by problem i = min((i + off) / div, b_batches - 1)
    // MN-major B only: when b_idx is set, b is the UNPACKED matrix [b_batches, b_rows, b_ld] and the kernel fetches the
    // kept rows b_idx[i * b_idx_stride + 0 .. k-1] itself (no packed copy of B; outputs of up to 128 rows)
    const int32_t *b_idx;
    int64_t b_idx_stride, b_rows;
    void *y;
    int y_bf16;
    int64_t y_sb, y_sr;
    float scale;
    int *status;
    // 8-bit operands (e4m3 bytes; a and b then point to bytes, leading dimensions and batch strides count bytes, both
    // K-major): the product of the codes is multiplied by scale * row_scale[batch entry * M + row]
    int fp8;
    const float *row_scale;
    // bf16 output only: when set, the epilogue also writes, per 32-row group g and column c, the sum of the squares of the
    // rounded outputs Y[32 g .. 32 g + 31, c] to col_energy[(batch entry * ceil(M / 32) + g) * N + c]
    float *col_energy;
};
int launch_gemm_tc_problem(const TcProblem &p, cudaStream_t stream);
// energy[b, c] = sum over the 32-row groups of col_energy (fp64, in group order), rounded to fp32
int launch_energy_combine(const float *col_energy, int64_t batch, int64_t groups, int64_t N, float *energy, cudaStream_t stream);

// One gather of kept slices (see pack.cu).  Columns: dst[b, r, j] = src[sb, r, idx[b, j]], j < k, dst row pitch
// ld_dst >= k (columns k .. ld_dst zeroed).  Rows: dst[b, j, 0:n] = src[sb, idx[b, j], 0:n].  NULL idx = 0 .. k-1.
// Source batch sb = (b + b_off) / b_div; idx lists of two batch entries are idx_stride apart.  bf16 only.
struct PackSpec {
    int rows_gather;  // 0: column gather, 1: row gather
    const __nv_bfloat16 *src;
    __nv_bfloat16 *dst;
    const int32_t *idx;
    int64_t batch;
    int64_t rows;     // column gather: rows of src and dst
    int64_t K;        // index range: columns of src (column gather) or rows of src (row gather)
    int64_t n;        // row gather: row length (multiple of 8)
    int64_t s_batch, s_row, b_off, b_div, idx_stride, k, ld_dst;
};
static inline PackSpec pack_cols_spec(const __nv_bfloat16 *src, int64_t batch, int64_t rows, int64_t K, int64_t s_batch,
                                      int64_t s_row, int64_t b_off, int64_t b_div, const int32_t *idx, int64_t idx_stride,
                                      int64_t k, __nv_bfloat16 *dst, int64_t ld_dst)
{
    PackSpec s = {0, src, dst, idx, batch, rows, K, 0, s_batch, s_row, b_off, b_div, idx_stride, k, ld_dst};
    return s;
}
static inline PackSpec pack_rows_spec(const __nv_bfloat16 *src, int64_t batch, int64_t K, int64_t n, int64_t s_batch,
                                      int64_t s_row, int64_t b_off, int64_t b_div, const int32_t *idx, int64_t idx_stride,
                                      int64_t k, __nv_bfloat16 *dst, int64_t ld_dst)
{
    PackSpec s = {1, src, dst, idx, batch, 0, K, n, s_batch, s_row, b_off, b_div, idx_stride, k, ld_dst};
    return s;
}
// One launch for one or two gathers.
int launch_pack(const PackSpec *specs, int n, int *status, cudaStream_t stream);

// Gather of the kept contraction indices into an 8-bit K-major operand (quant.cu): dst[r, j] = code of src[r, idx[j]],
// j < k, zero bytes up to ld_dst (a multiple of 16).  quantise: src is bf16 and every row gets its own step
// row_scale[r] = max_j |src[r, idx[j]]| / 448, codes are e4m3(src / step); otherwise src already holds codes (bytes).
// s_row: elements between two rows of src; rows must start on 16-byte boundaries.
int launch_gather_q8(bool quantise, const void *src, int64_t rows, int64_t s_row, int64_t K, const int32_t *idx, int64_t k, uint8_t *dst,
                     int64_t ld_dst, float *row_scale, int *status, cudaStream_t stream);

// ---- attention helpers --------------------------------------------------------------------------------
// Row softmax of fp32 logits S [heads, Lq, ld_s] with optional end-aligned causal mask and optional additive mask
// (row (h, i) at mask + h m_sh + i m_sr, fp32); writes bf16 P [heads, Lq, ld_p] (columns Lk .. ld_p zeroed).
int launch_softmax_rows(const float *S, int64_t ld_s, int64_t heads, int64_t Lq, int64_t Lk, int causal, const float *mask,
                        int64_t m_sh, int64_t m_sr, __nv_bfloat16 *P, int64_t ld_p, cudaStream_t stream);
// Fused forms (S~ and P stay on the SM; head_dim and kept features up to 128) on packed Qp [heads, Lq, ldd],
// Kp [heads, Lk, ldd] (kd valid columns) and V [v_batches, Lk, Dh] (row pitch v_ld, batch pitch v_sb; head h uses
// batch entry (h + v_off) / v_div).
bool fused_attn_eligible(const rmm_attn_desc_t *d, int64_t kd);
// lse == tok == NULL: O = softmax(Qp Kp^T / sqrt(Dh) + mask) V.  With lse [heads, lse_ld] and tok [heads, Lk] given,
// Kp and V hold the kept keys only (Lk of them, at positions tok): O = P V with P = bf16(2^(x - lse)), not
// renormalised.  diag = Lk - Lq of the unpacked problem (causal: query i sees key t iff t <= i + diag).
int launch_fused_attn(const __nv_bfloat16 *Qp, const __nv_bfloat16 *Kp, int64_t ldd, int64_t kd, const __nv_bfloat16 *V,
                      int64_t v_ld, int64_t v_sb, int64_t v_batches, int64_t v_off, int64_t v_div, __nv_bfloat16 *O,
                      int64_t o_sh, int64_t o_sr, int64_t heads, int64_t Lq, int64_t Lk, int64_t Dh, int causal, int64_t diag,
                      const float *lse, int64_t lse_ld, const int32_t *tok, const float *mask, int64_t m_sh, int64_t m_sr, int *status, cudaStream_t stream);
// Two sweeps: lse [heads, lse_ld] (lse_ld a multiple of 64, >= Lq) = log2-domain row normalisers of softmax(S~ + mask);
// energy [heads, Lk] = squared token scores sum_i bf16(P_it)^2.
int launch_fused_attn_scores(const __nv_bfloat16 *Qp, const __nv_bfloat16 *Kp, int64_t ldd, int64_t kd, int64_t heads,
                             int64_t Lq, int64_t Lk, int64_t Dh, int causal, float *lse, int64_t lse_ld, float *energy,
                             int *status, cudaStream_t stream);

}  // namespace rmm
