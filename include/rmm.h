/*
 * rmm.h — C ABI of the B200 (sm_100a) library for Reduced Matrix Multiplication (RMM).
 *
 * RMM replaces a matrix product Y = A B (A: M x K activations, B: K x N weight or intermediate)
 * by Y~ = A[:, I] B[I, :], where I holds the ceil(rho K) indices of the contraction axis whose
 * activation columns have the largest Euclidean norm (paper Sec. 3.2).  Sec. 3.3 applies the same
 * rule to attention: feature dims of Q K^T chosen per query head from Q, token positions of P V
 * chosen from the columns of P.
 *
 * General rules for every entry point
 *   - every data pointer is a DEVICE pointer owned by the caller, unless a comment says "host";
 *   - the library never allocates, frees or synchronises (rmm_status_read and rmm_product_host excepted,
 *     see there); every launch is asynchronous on `stream` (a cudaStream_t passed as void*, NULL =
 *     legacy default stream);
 *   - scratch memory comes from the caller: `ws` must hold at least the matching
 *     *_workspace_bytes(); it must be 256-byte aligned and its first RMM_WS_HEADER_BYTES must be zero
 *     the first time it is handed to the library (the library leaves them reusable afterwards,
 *     unless a call reported a device-side error); calls that share one workspace must be ordered on one stream;
 *   - the return value is an rmm_status_t; on a host-side error nothing was launched and outputs
 *     are untouched; rmm_last_error() then gives a thread-local message;
 *   - device-side waits are bounded: a kernel that gives up writes RMM_ERR_TIMEOUT to the status
 *     word at the start of the workspace, releases what it holds and returns; read it with
 *     rmm_status_read() after synchronising the stream;
 *   - inputs must be finite; there is no CPU fallback: a shape, stride or dtype the kernels do not
 *     cover is refused with RMM_ERR_UNSUPPORTED.
 */
#ifndef RMM_B200_H
#define RMM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RMM_OK = 0,
    RMM_ERR_INVALID_ARG = 1, /* null pointer, dimension <= 0, rho outside (0,1], k outside [1,K], index out of range */
    RMM_ERR_UNSUPPORTED = 2, /* dtype / stride / alignment / size the kernels do not cover */
    RMM_ERR_WORKSPACE = 3,   /* ws is NULL, misaligned or smaller than *_workspace_bytes() */
    RMM_ERR_CUDA = 4,        /* a CUDA call failed; text kept for rmm_last_error() */
    RMM_ERR_TIMEOUT = 5,     /* device status word: a bounded wait inside a kernel gave up */
    RMM_ERR_BOUNDS = 6       /* device status word: an index outside [0, K) was met and skipped */
} rmm_status_t;

typedef enum { RMM_BF16 = 0, RMM_F32 = 1, RMM_F8E4M3 = 2 /* one byte: 4 exponent bits (bias 7), 3 mantissa bits, no infinities, largest 448; accepted by rmm_reduced_gemm_q8 only */ } rmm_dtype_t;

/* A batch of matrices in device memory.  Element (b, r, c) lives at
 * ptr + (b*stride_batch + r*stride_row + c*stride_col) elements.  stride_batch may be 0 (one matrix
 * shared by every batch element, e.g. a weight).  Strides are in elements and non-negative. */
typedef struct {
    void *ptr;
    int32_t dtype; /* rmm_dtype_t */
    int64_t batch, rows, cols;
    int64_t stride_batch, stride_row, stride_col;
} rmm_mat_t;

#define RMM_WS_HEADER_BYTES 4096

/* |I| = ceil(rho K) (Sec. 3.2), host only.  rho is taken as a double; the product rho*K is snapped
 * to the nearest integer when it lies within 4 ulps (4 * 2^-52 * rho*K) of it (so 0.07*100 gives 7, not 8,
 * while a ratio that is genuinely a little above j/K gives j + 1 at any K), then rounded up and clamped to [1, K].  RMM_ERR_INVALID_ARG if rho is not in (0, 1], K < 1 or k is NULL. */
int rmm_keep_count(double rho, int64_t K, int64_t *k);

/* Importance scores s_j = ||A[:, j]||_2 (Sec. 3.2 "Activation-aware dimension selection"; in
 * attention s_j = ||Q[:, j]||_2 and a_t = ||P[:, t]||_2, Sec. 3.3).  Only A is read.
 *   axis   1: one score per column (the contraction axis of A B); 0: one score per row.
 *   scores fp32 [batch, n] with n = cols (axis 1) or rows (axis 0), or NULL
 *   energy fp32 [batch, n]: the squared scores sum_i A[i,j]^2, which are the selection keys, or NULL
 * Squares of bf16 values are exact in fp32; sums run in short fp32 chains combined in fp64 in a fixed
 * order, so results are deterministic and accurate to about 1e-7 relative. */
size_t rmm_score_workspace_bytes(const rmm_mat_t *A, int axis);
int rmm_score(const rmm_mat_t *A, int axis, float *scores, float *energy, void *ws, size_t ws_bytes, void *stream);

/* I = TopK(keys, k) (Sec. 3.2; Theorem 1 shows it minimises the discarded energy).  One index set per
 * batch element.  k in [1, K] is used as given; k == 0 means k = rmm_keep_count(rho, K); k < 0 or k > K is
 * RMM_ERR_INVALID_ARG.
 *   keys     fp32 [batch, K], non-negative
 *   idx      int32 [batch, k], ASCENDING; among equal keys the lower index is kept
 *   retained fp32 [batch] or NULL: sum of the kept keys / sum of all keys (1 - eps_A(rho) of Eq. 5
 *            when the keys are energies) */
size_t rmm_select_workspace_bytes(int64_t batch, int64_t K);
int rmm_select(const float *keys, int64_t batch, int64_t K, double rho, int64_t k, int32_t *idx, float *retained,
               void *ws, size_t ws_bytes, void *stream);

/* rmm_score followed by rmm_select on the energies, in ONE launch when n <= 8192 (the last thread block to finish
 * a batch element's scores selects its index set; larger n: the select kernel follows as a second launch).
 * scores / energy / retained may be NULL. */
size_t rmm_score_select_workspace_bytes(const rmm_mat_t *A, int axis);
int rmm_score_select(const rmm_mat_t *A, int axis, double rho, int64_t k, int32_t *idx, float *scores, float *energy,
                     float *retained, void *ws, size_t ws_bytes, void *stream);

/* rmm_score_select without a workspace argument (the paper has no counterpart).  For callers that cannot allocate
 * device memory at all (code running where the allocator must not be touched: a frozen memory pool, a plugin that is
 * handed inputs and outputs only, a latency-critical loop), the scratch lives in a device array built into the
 * library: rmm_score_select_static_capacity() bytes (4 MiB), held by every GPU that loads the library until the
 * process exits.  A problem whose scratch (about 8 * row_splits * n + 4 * n bytes per batch element, see
 * rmm_score_select_workspace_bytes) exceeds the capacity is refused with RMM_ERR_WORKSPACE and a message; nothing is
 * launched.  The call allocates nothing and frees nothing.  Its first call on each device looks the array's device
 * address up (with that device current), so make that first call outside any stream capture.  All calls share the
 * one array per device: it keeps the previous call's contents (the part that must start at zero is cleared on the
 * stream by every call), and two calls that overlap on the GPU (different streams) race.  Results are those of
 * rmm_score_select, bit for bit.  idx, scores, energy, retained as there.
 * The device status word of these calls lives in the built-in array, where rmm_status_read cannot reach it:
 * rmm_score_select_static_status copies it to *device_status (an rmm_status_t) and clears it, for the current device.
 * It is a blocking copy: synchronise the stream first.  The word is sticky (a later call does not erase an error an
 * earlier one reported).  The cached address of the array belongs to the device's primary context and does not
 * survive cudaDeviceReset(). */
size_t rmm_score_select_static_capacity(void);
int rmm_score_select_static(const rmm_mat_t *A, int axis, double rho, int64_t k, int32_t *idx, float *scores,
                            float *energy, float *retained, void *stream);
int rmm_score_select_static_status(int *device_status);

/* Y = scale * A[:, I] B[I, :] (Sec. 3.2, RMM_rho(A,B); no rescaling: pass scale = 1).
 *   A    [b, M, K]; B [b or shared, K, N] (stride_batch 0 = shared); Y [b, M, N] (written in full)
 *   idx  int32 [b, k], each entry in [0, K) (NULL with k == K: the unreduced product, nothing is gathered); any set is accepted (so a cached or random set gives
 *        the paper's static / random controls); order fixes the summation order
 *   bf16 operands run on the tensor cores (fp32 accumulation) when A has stride_col 1, B has
 *   stride_col 1 (slices of the contraction axis contiguous) or stride_row 1, Y has stride_col 1, and
 *   pointers / leading strides are 16-byte aligned; Y may be bf16 or fp32.  Every other layout, and
 *   fp32 operands, run on a plain FMA kernel (fp32 accumulation).  A and B must share a dtype.
 *   Decode-step shapes (batch 1, M <= 4, bf16, B with contiguous rows; App. "Complexity Analysis", decoding step)
 *   take a gathered GEMV that reads only the kept rows of B (k N 2 bytes) and packs nothing; outputs of up to 256
 *   rows (small decode batches, B with contiguous rows, N > 128) run on the tensor cores with the kept rows of B
 *   fetched by the kernel itself, so W is read once and never copied. */
size_t rmm_reduced_gemm_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y);
int rmm_reduced_gemm(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                     const rmm_mat_t *Y, void *ws, size_t ws_bytes, void *stream);

/* rmm_reduced_gemm that also scores its output: energy_out fp32 [batch, N] receives sum_i Y[b, i, c]^2 of the outputs as
 * stored (after rounding to bf16 when Y is bf16), i.e. the selection keys of the NEXT product that contracts over Y's
 * columns, so that rmm_select can run on them without a score pass over Y (the paper's closing section names this joint
 * treatment of selection and reduced multiplication as the way to cut memory movement).  On the tensor-core path with a
 * bf16 Y the epilogue accumulates the sums while it holds the rounded tile (exact squares, fp32 chains of 16, 32-row
 * groups added in fp64 in a fixed order: deterministic, about 1e-7 relative); every other form of the product runs
 * rmm_score on Y afterwards.  Arguments otherwise as rmm_reduced_gemm. */
size_t rmm_reduced_gemm_scored_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y);
int rmm_reduced_gemm_scored(const rmm_mat_t *A, const rmm_mat_t *B, const int32_t *idx, int64_t k, float scale,
                            const rmm_mat_t *Y, float *energy_out, void *ws, size_t ws_bytes, void *stream);

/* The reduced product with 8-bit operands (the paper's appendix "Compatibility with quantization" shows that RMM composes
 * with INT8 inference and leaves a fused low-bit kernel as future work; this is the e4m3 form on the fp8 tensor cores):
 *   Y = scale * b_scale * diag(s) * Aq Bq[I, :],  Aq[i, j] = e4m3(A[i, I_j] / s_i),  s_i = max_j |A[i, I_j]| / 448
 * A bf16 [M, K] (batch 1, contiguous rows 16-byte aligned); the activation rows are quantised on the fly, each with its own
 * step taken over the KEPT columns (an all-zero row: s_i = 1); every decision that yields a code is taken in fp32 (IEEE
 * division, round to nearest even, saturating).  B holds e4m3 codes of the weight, dtype RMM_F8E4M3, as a [K, N] matrix
 * with stride_row == 1 (i.e. stored N x K, contraction axis contiguous; stride_col a multiple of 16, base 16-byte
 * aligned), with one scale b_scale for the tensor.  Y bf16 or fp32 [M, N]; a_scale fp32 [M] receives the s_i (or NULL).
 * The index set comes from the bf16 activations as always (rmm_score_select).  Accumulation is exact products in fp32. */
size_t rmm_reduced_gemm_q8_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, int64_t k, const rmm_mat_t *Y);
int rmm_reduced_gemm_q8(const rmm_mat_t *A, const rmm_mat_t *B, float b_scale, const int32_t *idx, int64_t k, float scale,
                        const rmm_mat_t *Y, float *a_scale, void *ws, size_t ws_bytes, void *stream);

/* Reduced attention of Sec. 3.3 for B sequences, Hq query heads, Hkv key/value heads (Hq % Hkv == 0,
 * query head h reads kv head h / (Hq/Hkv)).  Per (sequence, query head):
 *   I  = TopK of ||Q[:, j]||_2, |I| = ceil(rho_d Dh);  S~ = Q[:, I] K[:, I]^T / sqrt(Dh)  (full Dh in the scale)
 *   P  = softmax(S~ + M), M = causal mask aligned to the end (query i sees keys t <= i + Lk - Lq), and / or an
 *        additive mask given by the caller (`mask`), or none;
 *        P is rounded once to bf16 and that rounded P is what is scored and multiplied
 *   rho_t < 1:  T = TopK of ||P[:, t]||_2, |T| = ceil(rho_t Lk);  O = P[:, T] V[T, :]  (no renormalisation)
 *   rho_t == 1: O = P V
 * Q [B,Hq,Lq,Dh], K,V [B,Hkv,Lk,Dh], O [B,Hq,Lq,Dh] are bf16 with explicit element strides
 * (batch, head, row, 1).  idx_feat int32 [B,Hq,kd] and idx_tok int32 [B,Hq,kt] receive the index sets
 * (either may be NULL).  With at most 128 kept features and a head_dim of at most 256, S~ and P stay on the SM (heads wider
 * than 128 columns in two passes over the columns of V; fused kernel: one pass
 * for rho_t == 1; row normalisers, token scores and a gathered P V pass for rho_t < 1, where the normalised P is
 * what is rounded, scored and multiplied; for rho_t == 1 the bf16 rounding is applied to P times a per-row factor,
 * which changes O by rounding noise only).  Wider heads materialise S~ and P in the workspace one group of heads at a
 * time.  An evenly strided batch is processed as B * Hq heads in one pass of launches.
 * mask (device, fp32, or NULL): the additive M of Sec. 3.3, entry (b, h, i, t) at mask[b ms[0] + h ms[1] + i ms[2] + t]
 * with ms = mask_stride in elements (0 shares the mask along that axis; rows contiguous); -inf hides a key; a row with
 * every key hidden gives zeros.  It composes with `causal`.  With rho_t == 1, a fused-eligible shape and mask rows that are
 * 16-byte aligned (base pointer and all three strides multiples of 4 elements) the one-pass fused kernel adds the mask
 * itself; otherwise a call with a mask runs the composed form (S~ and P in the workspace). */
typedef struct {
    int64_t B, Hq, Hkv, Lq, Lk, Dh;
    int32_t causal;
    double rho_d; /* feature retention of Q K^T */
    double rho_t; /* token retention of P V; 1.0 switches token reduction off */
    int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3]; /* batch, head, row (elements); last dim contiguous */
    const float *mask;                                          /* optional additive mask (device) or NULL */
    int64_t mask_stride[3];                                     /* batch, head, query row (elements) */
} rmm_attn_desc_t;
size_t rmm_reduced_attn_workspace_bytes(const rmm_attn_desc_t *desc);
int rmm_reduced_attn(const rmm_attn_desc_t *desc, const void *Q, const void *K, const void *V, void *O,
                     int32_t *idx_feat, int32_t *idx_tok, void *ws, size_t ws_bytes, void *stream);

/* The whole operation of Sec. 3.2 on device operands: I = TopK of the column norms of A with |I| = k (k == 0:
 * ceil(rho K)), Y = scale * A[:, I] B[I, :].  The result is that of rmm_score_select followed by rmm_reduced_gemm
 * (in the one-launch form below the column energies are summed in a different fixed order, which can move a key by one
 * fp64 rounding before it is rounded to fp32); idx [batch, k] and retained [batch] (or NULL) as there.  For one small bf16 product (batch 1, A with 2368 to
 * 8192 columns and 257 to 8192 rows, B with at most 4096 columns) whose operands meet the tensor-core layout rules (the
 * regime where launch and hand-off latencies weigh most), the scores, the selection
 * and both gathers run in ONE launch (every block owns 64 columns of A, a grid-wide barrier makes all column energies
 * visible, every block then selects and gathers its own kept columns and the matching rows of B), followed by the
 * tensor-core product; this form expects the GPU to itself (all of its blocks must be resident at once; if they are
 * not, the barrier's bounded wait expires and RMM_ERR_TIMEOUT is reported).  Everything else runs as the two calls. */
size_t rmm_product_workspace_bytes(const rmm_mat_t *A, const rmm_mat_t *B, const rmm_mat_t *Y);
int rmm_product(const rmm_mat_t *A, const rmm_mat_t *B, double rho, int64_t k, float scale, const rmm_mat_t *Y, int32_t *idx,
                float *retained, void *ws, size_t ws_bytes, void *stream);

/* The whole operation of Sec. 3.2 on one bf16 product held in HOST memory (pinned for speed):
 * copies A [M,K] and B [K,N] (row-major, contiguous) to the device staging area inside ws, runs
 * rmm_product, and copies Y [M,N] bf16 and idx [k] back, all asynchronously on
 * `stream`; the caller synchronises the stream before reading Y_host / idx_host.  copy_B = 0 reuses the
 * B already staged by an earlier call on the same workspace (a resident weight). */
size_t rmm_product_host_workspace_bytes(int64_t M, int64_t K, int64_t N);
int rmm_product_host(const void *A_host, const void *B_host, int64_t M, int64_t K, int64_t N, double rho, int copy_B,
                     void *Y_host, int32_t *idx_host, void *ws, size_t ws_bytes, void *stream);

/* Copy the device status word of a workspace to *device_status (an rmm_status_t) and clear it.  If the word was set,
 * the whole header (the arrival counters too: a kernel that gave up may have left them half way) is zeroed, which
 * makes the workspace usable again.  Synchronous: call it after the stream the workspace was used on has been
 * synchronised. */
int rmm_status_read(void *ws, int *device_status);

/* Testing aid (the paper has no counterpart).  Every wait inside a kernel (on a copy, on another warp, on another block)
 * is bounded: 2 s by default, RMM_SPIN_LIMIT_MS milliseconds if that environment variable is set when the library is
 * first used.  rmm_debug_control("wait_limit_ms", x) overrides the bound for later launches (0 = back to the default);
 * rmm_debug_control("withhold", w) makes block 0 of one kernel family never request its first tile (w = 1 tensor-core
 * product, 2 score pass, 3 fused attention, 4 one-launch front end of rmm_product, 5 streaming column gather; 0 = off,
 * -1 = back to the environment variable RMM_TEST_WITHHOLD = gemm | score | attn | front | pack), so that the waits behind
 * that tile run out: the kernel must then report RMM_ERR_TIMEOUT in the status word, release what it holds and return.
 * Results of such a call are undefined; rmm_status_read clears the workspace header, after which the workspace is
 * usable again.  Not thread-safe against concurrent launches. */
int rmm_debug_control(const char *key, double value);

/* Timing hook for benchmarks (the paper has no counterpart).  After rmm_profile_kernels(start, stop, n, filter, every),
 * launches of library kernels whose name contains `name_filter` (NULL or "" = every kernel) are bracketed by
 * cudaEventRecord(start[i]) and cudaEventRecord(stop[i]) on their stream: one matching launch in `every` (<= 1: all of
 * them), up to n pairs.  (Event records between kernels cost a few microseconds of launch overlap, hence `every`.)  The host arrays
 * hold cudaEvent_t handles created by the caller with timing enabled and must stay alive until the hook is cleared
 * with (NULL, NULL, 0, NULL, 0).  n <= 4096.  Not thread-safe.  rmm_profile_count() tells how many pairs have been
 * recorded, rmm_profile_name(i) the kernel the i-th pair brackets (a static string). */
int rmm_profile_kernels(void **start_events, void **stop_events, int n, const char *name_filter, int every);
int rmm_profile_count(void);
const char *rmm_profile_name(int i);

/* Thread-local text of the last error returned on this thread ("" if none). */
const char *rmm_last_error(void);

/* Number of kernels the library has launched from this process (for launch accounting). */
int64_t rmm_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* RMM_B200_H */
