// Block-wide top-k selection on fp32 keys (paper Sec. 3.2: I = TopK({s_j}, ceil(rho d)); Theorem 1: the k columns of
// largest norm), shared by the kernels that end in a selection.  Device code only.
//
// Radix select on the order-preserving integer image of the keys: the bits common to all keys are skipped, one digit
// of up to 11 bits is histogrammed over all keys, the (few) keys that share the threshold's digit are copied to a
// short list and finished there.  Ties at the threshold go to the lowest indices; indices are emitted ascending.
#pragma once
#include "common.cuh"

#ifndef SEL_STAMP
#define SEL_STAMP(i)
#endif

namespace rmm {
namespace sel {

constexpr int kBins = 2048;      // first radix digit: up to 11 bits
constexpr int kCandMax = 1024;   // keys that share the threshold's first digit are finished from this list

struct SelectSmem {
    __align__(16) unsigned hist[kBins];
    unsigned cand[kCandMax];
    unsigned warp_a[32], warp_b[32], warp_lo[32], warp_hi[32];
    unsigned bin, remaining, count, n_cand;
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

// ---- blocked form ------------------------------------------------------------------------------------------------
// Thread t of a 1024-thread block holds the ITEMS consecutive keys [t * ITEMS, (t + 1) * ITEMS): the index order is
// the (thread, item) order, so the ordered emission needs one block-wide scan of per-thread counts and every thread
// writes its kept indices next to each other.  Digits after the first are up to 11 bits wide as well.
// The blocked form runs on a group of NTHR threads: the whole block (1024, ordinary block barrier) or its first eight
// warps (256, named barrier 2) while the other warps of the block do something else or wait.
template <int NTHR>
__device__ __forceinline__ void group_sync()
{
    if constexpr (NTHR == 1024) __syncthreads();
    else asm volatile("bar.sync 2, %0;" ::"n"(NTHR) : "memory");
}

struct Threshold {
    unsigned tau;      // image of the k-th largest key
    unsigned need_eq;  // how many keys equal to tau are kept (lowest indices first)
};

template <int ITEMS>
__device__ __forceinline__ int load_keys_blocked(const float *__restrict__ keys, int K, unsigned (&u)[ITEMS])
{
    const int j0 = threadIdx.x * ITEMS;
    const int nvalid = K - j0 >= ITEMS ? ITEMS : (K > j0 ? K - j0 : 0);
    if constexpr (ITEMS % 4 == 0) {
        if (nvalid == ITEMS && (reinterpret_cast<uintptr_t>(keys) & 15) == 0) {
#pragma unroll
            for (int v = 0; v < ITEMS / 4; ++v) {
                const float4 q = __ldcg(reinterpret_cast<const float4 *>(keys + j0) + v);
                u[4 * v] = key_image(q.x); u[4 * v + 1] = key_image(q.y); u[4 * v + 2] = key_image(q.z); u[4 * v + 3] = key_image(q.w);
            }
            return nvalid;
        }
    }
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) u[i] = i < nvalid ? key_image(__ldcg(keys + j0 + i)) : 0u;
    return nvalid;
}

// Among hist[0 .. nbins), nbins = 256 or 2048, find the bin b such that (keys in bins above b) < remaining <= (keys in
// bins >= b); publishes b in sm.bin, the count still wanted inside it in sm.remaining and the bin's own count in
// sm.n_cand.  Every thread of the block calls it (hist complete before the call, results visible after it), but only
// nbins / 256 warps work: a thread owns eight consecutive bins (two 16-byte loads, no bank conflicts), warps scan
// with shuffles, and with eight warps a named barrier among them exchanges the warp totals.  With 32 warps sharing four
// schedulers, instructions issued by every warp are what a block-wide step costs; this keeps them to a few warps.
template <int NTHR>
__device__ __forceinline__ void find_bin8(SelectSmem &sm, int nbins, unsigned remaining)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nw = nbins >> 8;  // 1 or 8 working warps
    if (warp < nw) {
        const int low = nbins - 8 - 8 * tid;  // this thread's lowest bin
        const uint4 qa = *reinterpret_cast<const uint4 *>(&sm.hist[low]), qb = *reinterpret_cast<const uint4 *>(&sm.hist[low + 4]);
        const unsigned h[8] = {qb.w, qb.z, qb.y, qb.x, qa.w, qa.z, qa.y, qa.x};  // from the top bin down
        unsigned mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) mine += h[i];
        unsigned incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        unsigned base = 0;
        if (nw > 1) {
            if (lane == 31) sm.warp_a[warp] = incl;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            const unsigned w = lane < nw ? sm.warp_a[lane] : 0u;
            unsigned wi = w;
#pragma unroll
            for (int d = 1; d < 8; d <<= 1) {
                const unsigned v = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= d) wi += v;
            }
            base = __shfl_sync(0xffffffffu, wi - w, warp);
        }
        unsigned above = base + incl - mine;  // keys in bins above this thread's
        if (above < remaining && remaining <= above + mine) {  // exactly one thread
            bool found = false;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (!found && remaining <= above + h[i]) {
                    sm.bin = (unsigned)(low + 7 - i);
                    sm.remaining = remaining - above;
                    sm.n_cand = h[i];
                    found = true;
                }
                if (!found) above += h[i];
            }
        }
    }
    group_sync<NTHR>();
}

// Image of the k-th largest key and the number of keys equal to it that are kept.  Items 0 .. nvalid-1 of every thread
// take part (entries beyond nvalid must hold 0, which load_keys_blocked guarantees).  Whole block (1024 threads).
// The keys stay in registers for every pass: one digit of up to 11 bits over all keys, then 8-bit digits in which only
// the keys that share the prefix found so far count (a per-thread bit mask of those keys is carried along, and warps
// without any skip the pass).  With 32 warps on four schedulers every instruction that all warps execute costs eight
// issue clocks, so the code paths below are kept short rather than general.
template <int ITEMS, int NTHR = 1024>
__device__ __forceinline__ Threshold block_threshold(const unsigned (&u)[ITEMS], int nvalid, int k, SelectSmem &sm)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nthr = NTHR, nwarp = NTHR / 32;
    unsigned lo = 0xffffffffu, hi = 0u;
    if (nvalid == ITEMS) {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            lo = min(lo, u[i]);
            hi = max(hi, u[i]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            if (i < nvalid) {
                lo = min(lo, u[i]);
                hi = max(hi, u[i]);
            }
        }
    }
    lo = __reduce_min_sync(0xffffffffu, lo);
    hi = __reduce_max_sync(0xffffffffu, hi);
    if (lane == 0) {
        sm.warp_lo[warp] = lo;
        sm.warp_hi[warp] = hi;
    }
    {
        uint4 *h4 = reinterpret_cast<uint4 *>(sm.hist);
        for (int i = tid; i < kBins / 4; i += nthr) h4[i] = make_uint4(0, 0, 0, 0);
    }
    group_sync<NTHR>();
    SEL_STAMP(0);
    {
        const unsigned l = lane < nwarp ? sm.warp_lo[lane] : 0xffffffffu, h = lane < nwarp ? sm.warp_hi[lane] : 0u;
        lo = __reduce_min_sync(0xffffffffu, l);
        hi = __reduce_max_sync(0xffffffffu, h);
    }
    const int lcp = (lo ^ hi) ? __clz(lo ^ hi) : 32;  // leading bits common to every key
    unsigned mask = lcp == 0 ? 0u : (lcp == 32 ? 0xffffffffu : ~(0xffffffffu >> lcp));
    unsigned prefix = hi & mask;
    unsigned remaining = (unsigned)k;
    Threshold t;
    t.tau = prefix;
    t.need_eq = remaining;
    if (lcp == 32) return t;  // every key is the same

    // ---- first digit: every valid key counts
    int d = 32 - lcp < 11 ? 32 - lcp : 11;
    int shift = 32 - lcp - d;
    unsigned m = (1u << d) - 1u;
    if (nvalid == ITEMS) {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) atomicAdd(&sm.hist[(u[i] >> shift) & m], 1u);
    } else {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if (i < nvalid) atomicAdd(&sm.hist[(u[i] >> shift) & m], 1u);
    }
    group_sync<NTHR>();
    SEL_STAMP(1);
    find_bin8<NTHR>(sm, d > 8 ? 2048 : 256, remaining);  // bins beyond 1 << d are zero
    SEL_STAMP(2);
    prefix |= sm.bin << shift;
    mask |= m << shift;
    remaining = sm.remaining;
    unsigned n_same = sm.n_cand;
    unsigned live = 0;  // bit i: key i of this thread shares the prefix
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) live |= (i < nvalid && (u[i] & mask) == prefix) ? (1u << i) : 0u;

    // ---- remaining bits, eight at a time, over the keys that share the prefix
    [[maybe_unused]] int pass = 1;
    while (shift > 0 && n_same != remaining) {
        d = shift < 8 ? shift : 8;
        shift -= d;
        m = (1u << d) - 1u;
        if (tid < 64) reinterpret_cast<uint4 *>(sm.hist)[tid] = make_uint4(0, 0, 0, 0);
        group_sync<NTHR>();
        if (__any_sync(0xffffffffu, live != 0u)) {
#pragma unroll
            for (int i = 0; i < ITEMS; ++i)
                if (live & (1u << i)) atomicAdd(&sm.hist[(u[i] >> shift) & m], 1u);
        }
        group_sync<NTHR>();
        SEL_STAMP(1 + 2 * pass);
        find_bin8<NTHR>(sm, 256, remaining);
        SEL_STAMP(2 + 2 * pass);
        ++pass;
        prefix |= sm.bin << shift;
        mask |= m << shift;
        remaining = sm.remaining;
        n_same = sm.n_cand;
        if (__any_sync(0xffffffffu, live != 0u)) {
#pragma unroll
            for (int i = 0; i < ITEMS; ++i)
                if ((live & (1u << i)) && (u[i] & mask) != prefix) live &= ~(1u << i);
        }
    }
    if (shift > 0) {
        // every key that shares the prefix is kept (n_same == remaining): the threshold is the smallest of them, and
        // need_eq the number of keys equal to it
        unsigned mn = 0xffffffffu;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if (live & (1u << i)) mn = min(mn, u[i]);
        mn = __reduce_min_sync(0xffffffffu, mn);
        if (lane == 0) sm.warp_lo[warp] = mn;
        group_sync<NTHR>();
        mn = __reduce_min_sync(0xffffffffu, lane < nwarp ? sm.warp_lo[lane] : 0xffffffffu);
        unsigned c = 0;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if ((live & (1u << i)) && u[i] == mn) ++c;
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0) sm.warp_hi[warp] = c;
        group_sync<NTHR>();
        t.tau = mn;
        t.need_eq = __reduce_add_sync(0xffffffffu, lane < nwarp ? sm.warp_hi[lane] : 0u);
        return t;
    }
    t.tau = prefix;
    t.need_eq = remaining;
    return t;
}

// Exclusive block-wide scan of this thread's (keys greater than tau, keys equal to tau) counts, packed as
// (greater << 16 | equal): the number of such keys at lower indices.  Whole block (1024 threads), K <= 65535.
// One barrier: every warp scans the 32 warp totals itself.
template <int ITEMS, int NTHR = 1024>
__device__ __forceinline__ unsigned block_rank_blocked(const unsigned (&u)[ITEMS], int nvalid, unsigned tau, SelectSmem &sm)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned mine = 0;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i)
        if (i < nvalid) mine += (u[i] > tau ? 0x10000u : 0u) + (u[i] == tau ? 1u : 0u);
    unsigned incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    if (lane == 31) sm.warp_a[warp] = incl;
    group_sync<NTHR>();
    const unsigned w = lane < NTHR / 32 ? sm.warp_a[lane] : 0u;
    unsigned wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned v = __shfl_up_sync(0xffffffffu, wi, d);
        if (lane >= d) wi += v;
    }
    const unsigned warp_base = __shfl_sync(0xffffffffu, wi - w, warp);
    return incl - mine + warp_base;
}

// Whole selection in the blocked form: K <= ITEMS * 1024 keys, blockDim.x == 1024.
template <int ITEMS>
__device__ void block_select_blocked(const float *__restrict__ keys, int K, int k, int32_t *__restrict__ idx, float *retained,
                                     SelectSmem &sm)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned u[ITEMS];
    const int nvalid = load_keys_blocked<ITEMS>(keys, K, u);
    const Threshold th = block_threshold<ITEMS>(u, nvalid, k, sm);
    const unsigned before = block_rank_blocked<ITEMS>(u, nvalid, th.tau, sm);
    unsigned gt_before = before >> 16, eq_before = before & 0xffffu;
    double sum_kept = 0.0, sum_all = 0.0;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        if (i < nvalid) {
            const bool gt = u[i] > th.tau, eq = u[i] == th.tau;
            const bool keep = gt || (eq && eq_before < th.need_eq);
            if (keep) idx[gt_before + (eq_before < th.need_eq ? eq_before : th.need_eq)] = tid * ITEMS + i;
            if (retained != nullptr) {
                const double f = (double)key_value(u[i]);
                sum_all += f;
                if (keep) sum_kept += f;
            }
            gt_before += gt ? 1u : 0u;
            eq_before += eq ? 1u : 0u;
        }
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
            for (int w = 0; w < 32; ++w) {  // fixed order
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
    if (blockDim.x == 1024 && K <= 1024) block_select_blocked<1>(keys, K, k, idx, retained, sm);
    else if (blockDim.x == 1024 && K <= 4096) block_select_blocked<4>(keys, K, k, idx, retained, sm);
    else if (blockDim.x == 1024 && K <= 8192) block_select_blocked<8>(keys, K, k, idx, retained, sm);
    else block_select(keys, K, k, idx, retained, sm, kcache);
}

}  // namespace sel
}  // namespace rmm
