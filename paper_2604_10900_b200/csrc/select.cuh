// Block-wide exact top-k by radix select on order-preserving uint32 score keys.
// Total order: score descending, then row index ascending (the k-th score may be
// tied; ties are taken in index order).
//
// Three histogram sweeps narrow the key of the k-th greatest row digit by digit (12 + 12 + 8
// bits), a last sweep marks everything above it and the rows equal to it.  The sweeps read the
// unit's scores from global memory; after the first one they are L1/L2 hits.
// Ranges of at most kSmallSpan rows skip the sweeps: their keys sit in shared memory and, up to
// kCountSpan rows, every eligible row counts the rows ahead of it in the total order; above that
// the (key, row) pairs are sorted by a bitonic network (same result, a few microseconds instead
// of a dozen block-wide barriers over global memory).
#pragma once
#include "cask_internal.cuh"

namespace cask {

constexpr int kSelThreads = 1024;
constexpr int kSelBins = 4096;
constexpr int kSmallSpan = 1024;       // rows; keys and eligibility flags fit SelectSmem::hist

// Threads per selection CTA: small units take the counting path, which needs no 4096-bin histogram
// (find_digit wants nbins <= 4 * blockDim.x) and leaves room for several CTAs per SM.
inline int select_threads(int max_rows_per_unit) { return max_rows_per_unit <= kSmallSpan ? 256 : kSelThreads; }

constexpr int kCountSpan = 256;        // rows; up to here every row counts the rows ahead of it, above it the rows are sorted

struct alignas(16) SelectSmem {
    unsigned hist[kSelBins];
    unsigned warp_cnt[kSelThreads / 32];
    unsigned digit, krem, neq;
};

// Sum of `v` over the block, returned to every thread.
__device__ __forceinline__ unsigned block_sum(unsigned v, SelectSmem& sm) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if (lane == 0) sm.warp_cnt[w] = v;
    __syncthreads();
    unsigned t = (lane < (int)(blockDim.x >> 5)) ? sm.warp_cnt[lane] : 0u;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    return t;
}

// Exclusive prefix of `v` over the block in thread order (total returned through `total`).
__device__ __forceinline__ unsigned block_excl_scan(unsigned v, SelectSmem& sm, unsigned& total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    unsigned incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        unsigned o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
    }
    __syncthreads();
    if (lane == 31) sm.warp_cnt[w] = incl;
    __syncthreads();
    unsigned wv = (lane < nw) ? sm.warp_cnt[lane] : 0u;
    unsigned wincl = wv;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        unsigned o = __shfl_up_sync(0xffffffffu, wincl, off);
        if (lane >= off) wincl += o;
    }
    total = __shfl_sync(0xffffffffu, wincl, 31);
    const unsigned wbefore = __shfl_sync(0xffffffffu, wincl - wv, w);
    return wbefore + incl - v;
}

// With sm.hist[0..nbins) filled: the digit d such that fewer than krem keys lie in the bins above d
// and at least krem in the bins >= d.  Leaves d in sm.digit, the rank inside bin d in sm.krem and
// the population of bin d in sm.neq.  nbins <= 4 * blockDim.x.
__device__ __forceinline__ void find_digit(SelectSmem& sm, int nbins, unsigned krem) {
    const int tid = threadIdx.x;
    // thread t owns the four bins nbins-1-4t .. nbins-4-4t, in descending order
    unsigned c[4], tot = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int b = nbins - 1 - 4 * tid - q;
        c[q] = (b >= 0) ? sm.hist[b] : 0u;
        tot += c[q];
    }
    unsigned total;
    const unsigned before = block_excl_scan(tot, sm, total);
    if (before < krem && krem <= before + tot) {
        unsigned run = before;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (run < krem && krem <= run + c[q]) {
                sm.digit = (unsigned)(nbins - 1 - 4 * tid - q);
                sm.krem = krem - run;
                sm.neq = c[q];
            }
            run += c[q];
        }
    }
    __syncthreads();
}

// Rows [lo,hi), at most kSmallSpan of them: among those with kind == 0 the k1 greatest get mark1 and the next k2 get
// mark2 (k2 may be 0).  The (key, row) pairs are sorted in shared memory, in the total order (key descending, row
// ascending), by a bitonic network: counting the rows ahead of every row costs span^2 comparisons, which at a thousand
// rows is ten times the network.
__device__ inline void block_sort_mark(const float* __restrict__ s, uint8_t* kind, int lo, int hi, int k1, uint8_t mark1,
                                       int k2, uint8_t mark2, SelectSmem& sm) {
    const int tid = threadIdx.x, nthr = blockDim.x, span = hi - lo;
    unsigned long long* pk = reinterpret_cast<unsigned long long*>(sm.hist);      // [n2] <= 1024 pairs of 8 bytes
    int n2 = 32;
    while (n2 < span) n2 <<= 1;
    for (int x = tid; x < n2; x += nthr) {
        const bool el = x < span && kind[lo + x] == 0;
        // a greater pair comes earlier: greater key, then lower row; 0 (below every eligible row) for the rest
        pk[x] = el ? ((unsigned long long)order_key(s[lo + x]) << 32) | (unsigned)(0xFFFFFFFFu - (unsigned)x) : 0ull;
    }
    __syncthreads();
    for (int k2b = 2; k2b <= n2; k2b <<= 1)
        for (int j = k2b >> 1; j > 0; j >>= 1) {
            for (int t = tid; t < (n2 >> 1); t += nthr) {
                const int i = 2 * t - (t & (j - 1)), l = i + j;
                const unsigned long long a = pk[i], b = pk[l];
                const bool desc = (i & k2b) == 0;          // this run ends up descending
                if ((a < b) == desc) { pk[i] = b; pk[l] = a; }
            }
            __syncthreads();
        }
    for (int x = tid; x < min(k1 + k2, n2); x += nthr) {
        const unsigned long long v = pk[x];
        if (v != 0ull) kind[lo + (int)(0xFFFFFFFFu - (unsigned)v)] = x < k1 ? mark1 : mark2;
    }
    __syncthreads();
}

// Among rows [lo,hi) with kind == 0, give `mark` to the k greatest.  All threads of the
// block must call it with the same arguments.  s and kind are per-unit pointers.
__device__ inline void block_topk_mark(const float* __restrict__ s, uint8_t* kind, int lo, int hi, int k,
                                       uint8_t mark, SelectSmem& sm) {
    if (k <= 0 || hi <= lo) return;
    const int tid = threadIdx.x, lane = tid & 31, nthr = blockDim.x;
    const int span = hi - lo;
    const int iters = (span + nthr - 1) / nthr;

    if (span > kCountSpan && span <= kSmallSpan) { block_sort_mark(s, kind, lo, hi, k, mark, 0, mark, sm); return; }
    if (span <= kCountSpan) {
        // ---- counting path: rank of every eligible row under (key descending, row ascending) ----
        unsigned* keys = sm.hist;                         // [span] rounded up to a multiple of 4
        unsigned* elig = sm.hist + kSmallSpan;            // one bit per row
        const int span4 = (span + 3) & ~3;
        for (int b = tid; b < (kSmallSpan >> 5); b += nthr) elig[b] = 0u;
        __syncthreads();
        for (int x = tid; x < span4; x += nthr) {
            const bool el = x < span && kind[lo + x] == 0;
            keys[x] = el ? order_key(s[lo + x]) : 0u;
            if (el) atomicOr(&elig[x >> 5], 1u << (x & 31));
        }
        __syncthreads();
        for (int x = tid; x < span; x += nthr) {
            if (!((elig[x >> 5] >> (x & 31)) & 1u)) continue;
            const unsigned ki = keys[x];
            unsigned ahead = 0;
            for (int j = 0; j < span4; j += 4) {
                const uint4 kj = *reinterpret_cast<const uint4*>(keys + j);
                ahead += (kj.x > ki) + (kj.y > ki) + (kj.z > ki) + (kj.w > ki);
                if (kj.x == ki || kj.y == ki || kj.z == ki || kj.w == ki) {
                    // equal keys ahead of this row: lower rows that are eligible themselves
                    const unsigned kk[4] = {kj.x, kj.y, kj.z, kj.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        ahead += (kk[q] == ki && j + q < x && ((elig[(j + q) >> 5] >> ((j + q) & 31)) & 1u));
                }
            }
            if (ahead < (unsigned)k) kind[lo + x] = mark;
        }
        __syncthreads();
        return;
    }

    // ---- sweep 1: top 12 bits ----
    for (int b = tid; b < kSelBins; b += nthr) sm.hist[b] = 0;
    __syncthreads();
    unsigned mine = 0;
    for (int it = 0; it < iters; it += 4) {
        unsigned key[4];
        bool el[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lo + (it + q) * nthr + tid;
            el[q] = (i < hi) && kind[i] == 0;
            key[q] = el[q] ? order_key(s[i]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (el[q]) { atomicAdd(&sm.hist[key[q] >> 20], 1u); ++mine; }
    }
    const unsigned n_elig = block_sum(mine, sm);
    if ((unsigned)k >= n_elig) {
        for (int i = lo + tid; i < hi; i += nthr)
            if (kind[i] == 0) kind[i] = mark;
        __syncthreads();
        return;
    }
    find_digit(sm, kSelBins, (unsigned)k);
    const unsigned d1 = sm.digit;
    unsigned krem = sm.krem;
    __syncthreads();

    // ---- sweep 2: next 12 bits among the keys whose top digit is d1 ----
    for (int b = tid; b < kSelBins; b += nthr) sm.hist[b] = 0;
    __syncthreads();
    for (int it = 0; it < iters; it += 4) {
        unsigned key[4];
        bool el[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lo + (it + q) * nthr + tid;
            el[q] = (i < hi) && kind[i] == 0;
            key[q] = el[q] ? order_key(s[i]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (el[q] && (key[q] >> 20) == d1) atomicAdd(&sm.hist[(key[q] >> 8) & 0xFFFu], 1u);
    }
    __syncthreads();
    find_digit(sm, kSelBins, krem);
    const unsigned d12 = (d1 << 12) | sm.digit;
    krem = sm.krem;
    __syncthreads();

    // ---- sweep 3: last 8 bits ----
    for (int b = tid; b < 256; b += nthr) sm.hist[b] = 0;
    __syncthreads();
    for (int it = 0; it < iters; it += 4) {
        unsigned key[4];
        bool el[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lo + (it + q) * nthr + tid;
            el[q] = (i < hi) && kind[i] == 0;
            key[q] = el[q] ? order_key(s[i]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (el[q] && (key[q] >> 8) == d12) atomicAdd(&sm.hist[key[q] & 0xFFu], 1u);
    }
    __syncthreads();
    find_digit(sm, 256, krem);
    const unsigned thr = (d12 << 8) | sm.digit;     // key of the k-th greatest row
    krem = sm.krem;                                  // how many of the rows equal to it are taken
    const unsigned neq = sm.neq;
    __syncthreads();

    // ---- marking ----
    if (krem == neq) {
        for (int i = lo + tid; i < hi; i += nthr)
            if (kind[i] == 0 && order_key(s[i]) >= thr) kind[i] = mark;
        __syncthreads();
        return;
    }
    // ties at the threshold: the lowest-index krem of them, found by an ordered scan
    unsigned eq_before = 0;
    for (int it = 0; it < iters; ++it) {
        const int i = lo + it * nthr + tid;
        const bool elig = (i < hi) && kind[i] == 0;
        const unsigned key = elig ? order_key(s[i]) : 0u;
        const bool gt = elig && key > thr;
        const bool eq = elig && key == thr;
        const unsigned bal = __ballot_sync(0xffffffffu, eq);
        const unsigned in_warp = __popc(bal & ((1u << lane) - 1u));
        unsigned all;
        const unsigned before = block_excl_scan(lane == 0 ? __popc(bal) : 0u, sm, all);
        const unsigned wbefore = __shfl_sync(0xffffffffu, before, 0);
        if (gt || (eq && eq_before + wbefore + in_warp < krem)) kind[i] = mark;
        eq_before += all;
    }
    __syncthreads();
}

// Two selections in one: among rows [lo,hi) with kind == 0 the k1 greatest get mark1 and the next k2 get mark2, which
// is what block_topk_mark(k1, mark1) followed by block_topk_mark(k2, mark2) gives.  The three histogram sweeps narrow
// both thresholds (rank k1 and rank k1 + k2) at once, with a second histogram where their digit prefixes part; one
// marking sweep follows.  A tie at either threshold, or a selection that takes every row, goes the plain way.
// ALL_OPEN: the caller knows that every row of [lo, hi) is still unmarked (kind 0), so the sweeps need not read the kinds.
template <bool ALL_OPEN = false>
__device__ inline void block_topk2_mark(const float* __restrict__ s, uint8_t* kind, int lo, int hi, int k1, uint8_t mark1,
                                        int k2, uint8_t mark2, SelectSmem& sm, SelectSmem& sm2) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int span = hi - lo;
    auto plain = [&]() {
        block_topk_mark(s, kind, lo, hi, k1, mark1, sm);
        block_topk_mark(s, kind, lo, hi, k2, mark2, sm);
    };
    if (k1 > 0 && k2 > 0 && span > kCountSpan && span <= kSmallSpan) {      // one sort serves both selections
        block_sort_mark(s, kind, lo, hi, k1, mark1, k2, mark2, sm);
        return;
    }
    if (k1 <= 0 || k2 <= 0 || span <= kSmallSpan) { plain(); return; }
    const int iters = (span + nthr - 1) / nthr;
    // ---- sweep 1: top 12 bits, shared by both thresholds ----
    for (int b = tid; b < kSelBins; b += nthr) sm.hist[b] = 0;
    __syncthreads();
    // (the sweeps take four rows a round so that their loads are in flight together: a loop of one load and one
    // shared-memory atomic per round runs at one cache latency per row)
    unsigned mine = 0;
    for (int it = 0; it < iters; it += 4) {
        unsigned key[4];
        bool el[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lo + (it + q) * nthr + tid;
            el[q] = (i < hi) && (ALL_OPEN || kind[i] == 0);
            key[q] = el[q] ? order_key(s[i]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (el[q]) { atomicAdd(&sm.hist[key[q] >> 20], 1u); ++mine; }
    }
    const unsigned n_elig = block_sum(mine, sm);
    if ((unsigned)(k1 + k2) >= n_elig) { __syncthreads(); plain(); return; }
    find_digit(sm, kSelBins, (unsigned)k1);
    const unsigned a1 = sm.digit;
    unsigned ka = sm.krem;
    __syncthreads();
    find_digit(sm, kSelBins, (unsigned)(k1 + k2));
    const unsigned b1 = sm.digit;
    unsigned kb = sm.krem;
    __syncthreads();
    // ---- sweeps 2 and 3: next 12 and last 8 bits; one histogram while the prefixes agree, else one each ----
    unsigned pa = a1, pb = b1;           // prefixes so far
    unsigned neq_a = 0, neq_b = 0;
    for (int pass = 1; pass < 3; ++pass) {
        const int bits = pass == 1 ? 12 : 8, shift = pass == 1 ? 8 : 0, nbins = 1 << bits;
        const bool same = pa == pb;
        for (int b = tid; b < nbins; b += nthr) { sm.hist[b] = 0; sm2.hist[b] = 0; }
        __syncthreads();
        for (int it = 0; it < iters; it += 4) {
            unsigned key[4];
            bool el[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = lo + (it + q) * nthr + tid;
                el[q] = (i < hi) && (ALL_OPEN || kind[i] == 0);
                key[q] = el[q] ? order_key(s[i]) : 0u;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (el[q]) {
                    const unsigned pre = key[q] >> (shift + bits), dg = (key[q] >> shift) & (unsigned)(nbins - 1);
                    if (pre == pa) atomicAdd(&sm.hist[dg], 1u);
                    else if (pre == pb) atomicAdd(&sm2.hist[dg], 1u);
                }
        }
        __syncthreads();
        find_digit(sm, nbins, ka);
        const unsigned da = sm.digit;
        const unsigned ka2 = sm.krem;
        neq_a = sm.neq;
        __syncthreads();
        unsigned db, kb2;
        if (same) {
            find_digit(sm, nbins, kb);
            db = sm.digit; kb2 = sm.krem; neq_b = sm.neq;
        } else {
            find_digit(sm2, nbins, kb);
            db = sm2.digit; kb2 = sm2.krem; neq_b = sm2.neq;
        }
        __syncthreads();
        pa = (pa << bits) | da;
        pb = (pb << bits) | db;
        ka = ka2;
        kb = kb2;
    }
    // pa, pb: keys of the rows of rank k1 and k1 + k2; ka of the neq_a rows equal to pa fall inside the first
    // selection, kb of the neq_b rows equal to pb inside the two together
    if (ka != neq_a || kb != neq_b) { plain(); return; }      // rows tie across a boundary: index order decides
    for (int it = 0; it < iters; it += 4) {
        unsigned key[4];
        bool el[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lo + (it + q) * nthr + tid;
            el[q] = (i < hi) && (ALL_OPEN || kind[i] == 0);
            key[q] = el[q] ? order_key(s[i]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (el[q]) {
                const int i = lo + (it + q) * nthr + tid;
                if (key[q] >= pa) kind[i] = mark1;
                else if (key[q] >= pb) kind[i] = mark2;
            }
    }
    __syncthreads();
}

// Rows of [lo,hi) with kind == want, in ascending order: calls emit(rank, row) for each.  Every
// thread walks one contiguous chunk, so one block scan orders the whole range.
template <typename Emit>
__device__ inline void block_ordered_rows(const uint8_t* kind, int lo, int hi, uint8_t want, SelectSmem& sm,
                                          Emit emit) {
    const int span = hi - lo;
    if (span <= 0) return;
    const int chunk = (span + (int)blockDim.x - 1) / (int)blockDim.x;
    const int b = lo + (int)threadIdx.x * chunk, e = min(hi, b + chunk);
    unsigned cnt = 0;
    for (int i = b; i < e; ++i) cnt += (kind[i] == want);
    unsigned total;
    unsigned rank = block_excl_scan(cnt, sm, total);
    for (int i = b; i < e; ++i)
        if (kind[i] == want) emit(rank++, i);
}

}  // namespace cask
