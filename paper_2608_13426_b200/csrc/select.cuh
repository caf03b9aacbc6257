// Block-wide top-k selection on fp32 keys (paper Sec. 3.2: I = TopK({s_j}, ceil(rho d)); Theorem 1: the k columns of
// largest norm), shared by the kernels that end in a selection.  Device code only.
//
// Radix select on the order-preserving integer image of the keys: the bits common to all keys are skipped, one digit
// of up to 11 bits is histogrammed over all keys, the (few) keys that share the threshold's digit are copied to a
// short list and finished there.  Ties at the threshold go to the lowest indices; indices are emitted ascending.
#pragma once
#include "common.cuh"

namespace rmm {
namespace sel {

constexpr int kBins = 2048;      // first radix digit: up to 11 bits
constexpr int kCandMax = 1024;   // keys that share the threshold's first digit are finished from this list

struct SelectSmem {
    unsigned hist[kBins];
    unsigned cand[kCandMax];
    unsigned warp_a[32], warp_b[32];
    unsigned bin, remaining, count;
    double red[64];
};

__device__ __forceinline__ unsigned key_image(float f)
{
    unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // total order: larger float <=> larger image
}
__device__ __forceinline__ float key_value(unsigned u)
{
    return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}

// Among hist[0..nbins) find the bin b such that (keys in bins above b) < remaining <= (keys in bins >= b); publish it
// in sm.bin and the count still wanted inside that bin in sm.remaining.  Whole block; hist complete before the call.
__device__ __forceinline__ void find_bin(SelectSmem &sm, int nbins, unsigned remaining)
{
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const int per = nbins >= nthr ? nbins / nthr : 1;  // bins owned by a thread, taken from the top down
    const int first = nbins - 1 - tid * per;             // highest bin of this thread (negative: owns none)
    unsigned mine = 0;
    if (first >= 0)
        for (int i = 0; i < per; ++i) mine += sm.hist[first - i];
    unsigned incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        unsigned v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    if (lane == 31) sm.warp_a[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned w = lane < nwarp ? sm.warp_a[lane] : 0u, wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            unsigned v = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += v;
        }
        sm.warp_b[lane] = wi - w;
    }
    __syncthreads();
    incl += sm.warp_b[warp];
    unsigned above = incl - mine;
    if (first >= 0 && above < remaining && remaining <= incl) {
        for (int i = 0; i < per; ++i) {
            unsigned h = sm.hist[first - i];
            if (remaining <= above + h) {
                sm.bin = (unsigned)(first - i);
                sm.remaining = remaining - above;
                break;
            }
            above += h;
        }
    }
    __syncthreads();
}

// Block-wide top-k of keys[0..K): writes idx[0..k) ascending (ties at the threshold go to the lowest indices) and,
// if asked, the kept fraction of the key mass.  Every thread of the block must call it.  Keys are read through L2
// (other blocks may have just written them).  kcache, if not NULL, is shared memory for K key images: the keys
// are then fetched once and every later pass runs out of shared memory.
//
// Radix select on the order-preserving integer image of the keys: the bits common to all keys are skipped, one
// digit of up to 11 bits is histogrammed over all keys, the (few) keys that share the threshold's digit are copied
// to a short list and finished there with 8-bit digits.  The kept indices are then emitted by warps that own
// consecutive chunks of the index range, ranks coming from ballots.
__device__ void block_select(const float *__restrict__ keys, int K, int k, int32_t *__restrict__ idx, float *retained,
                             SelectSmem &sm, unsigned *kcache)
{
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    auto image = [&](int j) -> unsigned { return kcache != nullptr ? kcache[j] : key_image(__ldcg(keys + j)); };
    // ---- fetch the keys, eight independent loads at a time; min and max give the common leading bits
    unsigned lo = 0xffffffffu, hi = 0u;
    for (int j0 = tid; j0 < K; j0 += 8 * nthr) {
        unsigned u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int j = j0 + i * nthr;
            u[i] = j < K ? key_image(__ldcg(keys + j)) : 0u;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int j = j0 + i * nthr;
            if (j < K) {
                if (kcache != nullptr) kcache[j] = u[i];
                lo = min(lo, u[i]);
                hi = max(hi, u[i]);
            }
        }
    }
    lo = __reduce_min_sync(0xffffffffu, lo);
    hi = __reduce_max_sync(0xffffffffu, hi);
    if (lane == 0) {
        sm.warp_a[warp] = lo;
        sm.warp_b[warp] = hi;
    }
    for (int i = tid; i < kBins; i += nthr) sm.hist[i] = 0;
    if (tid == 0) sm.count = 0;
    __syncthreads();
    {
        unsigned l = lane < nwarp ? sm.warp_a[lane] : 0xffffffffu, h = lane < nwarp ? sm.warp_b[lane] : 0u;
        lo = __reduce_min_sync(0xffffffffu, l);
        hi = __reduce_max_sync(0xffffffffu, h);
    }
    __syncthreads();

    const int lcp = (lo ^ hi) ? __clz(lo ^ hi) : 32;  // leading bits common to every key
    unsigned mask = lcp == 0 ? 0u : (lcp == 32 ? 0xffffffffu : ~(0xffffffffu >> lcp));
    unsigned prefix = hi & mask;
    unsigned remaining = (unsigned)k;

    if (lcp < 32) {
        // ---- first digit over all keys
        const int d1 = 32 - lcp < 11 ? 32 - lcp : 11;
        int shift = 32 - lcp - d1;
        const unsigned dmask = (1u << d1) - 1u;
        for (int j = tid; j < K; j += nthr) atomicAdd(&sm.hist[(image(j) >> shift) & dmask], 1u);
        __syncthreads();
        find_bin(sm, 1 << d1, remaining);
        prefix |= sm.bin << shift;
        mask |= dmask << shift;
        remaining = sm.remaining;
        const unsigned n_cand = sm.hist[sm.bin];
        __syncthreads();

        // ---- the keys that share this digit: copy them to the short list if they fit
        const bool listed = n_cand <= (unsigned)kCandMax;
        if (listed && shift > 0) {
            for (int j0 = 0; j0 < K; j0 += nthr) {
                const int j = j0 + tid;
                const unsigned u = j < K ? image(j) : 0u;
                const bool live = j < K && (u & mask) == prefix;
                const unsigned act = __ballot_sync(0xffffffffu, live);
                if (act != 0u) {
                    unsigned base = 0;
                    if (lane == 0) base = atomicAdd(&sm.count, (unsigned)__popc(act));
                    base = __shfl_sync(0xffffffffu, base, 0);
                    if (live) sm.cand[base + __popc(act & ((1u << lane) - 1u))] = u;
                }
            }
            __syncthreads();
        }
        // ---- remaining bits, 8 at a time, over the list (or over all keys if the list would not fit)
        const int n_items = listed ? (int)n_cand : K;
        while (shift > 0) {
            const int d = shift < 8 ? shift : 8;
            shift -= d;
            const unsigned m = (1u << d) - 1u;
            for (int i = tid; i < 256; i += nthr) sm.hist[i] = 0;
            __syncthreads();
            for (int i = tid; i < n_items; i += nthr) {
                const unsigned u = listed ? sm.cand[i] : image(i);
                if ((u & mask) == prefix) atomicAdd(&sm.hist[(u >> shift) & m], 1u);
            }
            __syncthreads();
            find_bin(sm, 1 << d, remaining);
            prefix |= sm.bin << shift;
            mask |= m << shift;
            remaining = sm.remaining;
            __syncthreads();
        }
    }
    const unsigned tau = prefix;          // image of the k-th largest key
    const unsigned need_eq = remaining;   // how many keys equal to tau are kept (lowest indices first)

    // ---- ordered emission: warp w owns indices [w * chunk, (w + 1) * chunk)
    const int chunk = ((K + nwarp - 1) / nwarp + 31) / 32 * 32;
    const int c_begin = warp * chunk, c_end = min(K, c_begin + chunk);
    unsigned n_gt = 0, n_eq = 0;
    for (int j0 = c_begin; j0 < c_end; j0 += 32) {
        const int j = j0 + lane;
        const unsigned u = j < c_end ? image(j) : 0u;
        n_gt += __popc(__ballot_sync(0xffffffffu, j < c_end && u > tau));
        n_eq += __popc(__ballot_sync(0xffffffffu, j < c_end && u == tau));
    }
    if (lane == 0) {
        sm.warp_a[warp] = n_gt;
        sm.warp_b[warp] = n_eq;
    }
    __syncthreads();
    unsigned gt_base = 0, eq_base = 0;
    for (int w = 0; w < warp; ++w) {
        gt_base += sm.warp_a[w];
        eq_base += sm.warp_b[w];
    }
    double sum_kept = 0.0, sum_all = 0.0;
    const unsigned lt = (1u << lane) - 1u;
    for (int j0 = c_begin; j0 < c_end; j0 += 32) {
        const int j = j0 + lane;
        const bool in = j < c_end;
        const unsigned u = in ? image(j) : 0u;
        const bool gt = in && u > tau, eq = in && u == tau;
        const unsigned g = __ballot_sync(0xffffffffu, gt), e = __ballot_sync(0xffffffffu, eq);
        const unsigned gt_before = gt_base + __popc(g & lt), eq_before = eq_base + __popc(e & lt);
        if (in) {
            const bool keep = gt || (eq && eq_before < need_eq);
            if (keep) idx[gt_before + (eq_before < need_eq ? eq_before : need_eq)] = j;
            if (retained != nullptr) {  // the energy sums (fp64 conversions and adds) only when they are asked for
                const double f = (double)key_value(u);
                sum_all += f;
                if (keep) sum_kept += f;
            }
        }
        gt_base += __popc(g);
        eq_base += __popc(e);
    }
    if (retained != nullptr) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            sum_kept += __shfl_down_sync(0xffffffffu, sum_kept, d);
            sum_all += __shfl_down_sync(0xffffffffu, sum_all, d);
        }
        if (lane == 0) {
            sm.red[warp] = sum_kept;
            sm.red[32 + warp] = sum_all;
        }
        __syncthreads();
        if (tid == 0) {
            double a = 0.0, b = 0.0;
            for (int w = 0; w < nwarp; ++w) {
                a += sm.red[w];
                b += sm.red[32 + w];
            }
            *retained = (b > 0.0) ? (float)(a / b) : 1.0f;
        }
    }
    __syncthreads();
}

// The same selection for K <= ITEMS * blockDim.x with every key held in a register of its thread (key j lives in
// item j / blockDim.x of thread j % blockDim.x): all loops unroll, nothing is re-read, and the ordered emission needs
// one scan over ITEMS * 32 per-warp counts.  Requires blockDim.x == 1024.
template <int ITEMS>
__device__ void block_select_reg(const float *__restrict__ keys, int K, int k, int32_t *__restrict__ idx, float *retained,
                                 SelectSmem &sm)
{
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    unsigned u[ITEMS];
    unsigned lo = 0xffffffffu, hi = 0u;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int j = tid + i * nthr;
        u[i] = j < K ? key_image(__ldcg(keys + j)) : 0u;
    }
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        if (tid + i * nthr < K) {
            lo = min(lo, u[i]);
            hi = max(hi, u[i]);
        }
    }
    lo = __reduce_min_sync(0xffffffffu, lo);
    hi = __reduce_max_sync(0xffffffffu, hi);
    if (lane == 0) {
        sm.warp_a[warp] = lo;
        sm.warp_b[warp] = hi;
    }
    for (int i = tid; i < kBins; i += nthr) sm.hist[i] = 0;
    if (tid == 0) sm.count = 0;
    __syncthreads();
    {
        unsigned l = lane < nwarp ? sm.warp_a[lane] : 0xffffffffu, h = lane < nwarp ? sm.warp_b[lane] : 0u;
        lo = __reduce_min_sync(0xffffffffu, l);
        hi = __reduce_max_sync(0xffffffffu, h);
    }
    __syncthreads();

    const int lcp = (lo ^ hi) ? __clz(lo ^ hi) : 32;
    unsigned mask = lcp == 0 ? 0u : (lcp == 32 ? 0xffffffffu : ~(0xffffffffu >> lcp));
    unsigned prefix = hi & mask;
    unsigned remaining = (unsigned)k;
    const unsigned lt = (1u << lane) - 1u;

    if (lcp < 32) {
        const int d1 = 32 - lcp < 11 ? 32 - lcp : 11;
        int shift = 32 - lcp - d1;
        const unsigned dmask = (1u << d1) - 1u;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if (tid + i * nthr < K) atomicAdd(&sm.hist[(u[i] >> shift) & dmask], 1u);
        __syncthreads();
        find_bin(sm, 1 << d1, remaining);
        prefix |= sm.bin << shift;
        mask |= dmask << shift;
        remaining = sm.remaining;
        const unsigned n_cand = sm.hist[sm.bin];
        __syncthreads();
        if (shift > 0) {
            const bool listed = n_cand <= (unsigned)kCandMax;
            if (listed) {
#pragma unroll
                for (int i = 0; i < ITEMS; ++i) {
                    const bool live = tid + i * nthr < K && (u[i] & mask) == prefix;
                    const unsigned act = __ballot_sync(0xffffffffu, live);
                    if (act != 0u) {
                        unsigned base = 0;
                        if (lane == 0) base = atomicAdd(&sm.count, (unsigned)__popc(act));
                        base = __shfl_sync(0xffffffffu, base, 0);
                        if (live) sm.cand[base + __popc(act & lt)] = u[i];
                    }
                }
                __syncthreads();
            }
            while (shift > 0) {
                const int d = shift < 8 ? shift : 8;
                shift -= d;
                const unsigned m = (1u << d) - 1u;
                if (tid < 256) sm.hist[tid] = 0;
                __syncthreads();
                if (listed) {
                    for (int i = tid; i < (int)n_cand; i += nthr) {
                        const unsigned c = sm.cand[i];
                        if ((c & mask) == prefix) atomicAdd(&sm.hist[(c >> shift) & m], 1u);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < ITEMS; ++i)
                        if (tid + i * nthr < K && (u[i] & mask) == prefix) atomicAdd(&sm.hist[(u[i] >> shift) & m], 1u);
                }
                __syncthreads();
                find_bin(sm, 1 << d, remaining);
                prefix |= sm.bin << shift;
                mask |= m << shift;
                remaining = sm.remaining;
                __syncthreads();
            }
        }
    }
    const unsigned tau = prefix, need_eq = remaining;

    // ---- ordered emission.  Index order = (item, warp, lane); per-(item, warp) counts, packed (greater << 16 | equal)
    unsigned *cnt = sm.cand, *cnt_ex = sm.cand + ITEMS * 32;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const bool in = tid + i * nthr < K;
        const unsigned g = __ballot_sync(0xffffffffu, in && u[i] > tau), e = __ballot_sync(0xffffffffu, in && u[i] == tau);
        if (lane == 0) cnt[i * nwarp + warp] = ((unsigned)__popc(g) << 16) | (unsigned)__popc(e);
    }
    __syncthreads();
    if (tid < ITEMS * 32) {
        const unsigned v = cnt[tid];
        unsigned incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            unsigned o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) sm.warp_a[warp] = incl;
        cnt_ex[tid] = incl - v;
    }
    __syncthreads();
    double sum_kept = 0.0, sum_all = 0.0;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int j = tid + i * nthr;
        const bool in = j < K;
        unsigned base = cnt_ex[i * nwarp + warp];
        for (int w = 0; w < i; ++w) base += sm.warp_a[w];  // entries of item i sit in scan warp i (nwarp == 32)
        const bool gt = in && u[i] > tau, eq = in && u[i] == tau;
        const unsigned g = __ballot_sync(0xffffffffu, gt), e = __ballot_sync(0xffffffffu, eq);
        const unsigned gt_before = (base >> 16) + __popc(g & lt), eq_before = (base & 0xffffu) + __popc(e & lt);
        if (in) {
            const bool keep = gt || (eq && eq_before < need_eq);
            if (keep) idx[gt_before + (eq_before < need_eq ? eq_before : need_eq)] = j;
            if (retained != nullptr) {  // the energy sums (fp64 conversions and adds) only when they are asked for
                const double f = (double)key_value(u[i]);
                sum_all += f;
                if (keep) sum_kept += f;
            }
        }
    }
    if (retained != nullptr) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            sum_kept += __shfl_down_sync(0xffffffffu, sum_kept, d);
            sum_all += __shfl_down_sync(0xffffffffu, sum_all, d);
        }
        __syncthreads();
        if (lane == 0) {
            sm.red[warp] = sum_kept;
            sm.red[32 + warp] = sum_all;
        }
        __syncthreads();
        if (tid == 0) {
            double a = 0.0, b = 0.0;
            for (int w = 0; w < nwarp; ++w) {
                a += sm.red[w];
                b += sm.red[32 + w];
            }
            *retained = (b > 0.0) ? (float)(a / b) : 1.0f;
        }
    }
    __syncthreads();
}

// Dispatch on the problem size: keys in registers when they fit (blocks of 1024 threads), else the cached form.
__device__ __forceinline__ void block_select_any(const float *keys, int K, int k, int32_t *idx, float *retained,
                                                 SelectSmem &sm, unsigned *kcache)
{
    if (blockDim.x == 1024 && K <= 1024) block_select_reg<1>(keys, K, k, idx, retained, sm);
    else if (blockDim.x == 1024 && K <= 8192) block_select_reg<8>(keys, K, k, idx, retained, sm);
    else block_select(keys, K, k, idx, retained, sm, kcache);
}

}  // namespace sel
}  // namespace rmm
