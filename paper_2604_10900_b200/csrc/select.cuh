// Block-wide exact top-k by radix select on order-preserving uint32 score keys.
// Total order: score descending, then row index ascending (the k-th score may be
// tied; ties are taken in index order).
#pragma once
#include "cask_internal.cuh"

namespace cask {

constexpr int kSelThreads = 1024;

struct SelectSmem {
    unsigned hist[256];
    unsigned warp_cnt[kSelThreads / 32];
    unsigned prefix, krem, total, run;
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

// Among rows [lo,hi) with kind == 0, give `mark` to the k greatest.  All threads of the
// block must call it with the same arguments.  s and kind are per-unit pointers.
__device__ inline void block_topk_mark(const float* __restrict__ s, uint8_t* kind, int lo, int hi, int k,
                                uint8_t mark, SelectSmem& sm) {
    if (k <= 0 || hi <= lo) return;
    const int tid = threadIdx.x, lane = tid & 31, nthr = blockDim.x;
    unsigned mine = 0;
    for (int i = lo + tid; i < hi; i += nthr) mine += (kind[i] == 0);
    const unsigned n_elig = block_sum(mine, sm);
    if ((unsigned)k >= n_elig) {
        for (int i = lo + tid; i < hi; i += nthr)
            if (kind[i] == 0) kind[i] = mark;
        __syncthreads();
        return;
    }
    unsigned prefix = 0, mask = 0, krem = (unsigned)k;
    const int span = hi - lo;
    const int iters = (span + nthr - 1) / nthr;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) sm.hist[tid] = 0;
        __syncthreads();
        for (int it = 0; it < iters; ++it) {
            int i = lo + it * nthr + tid;
            unsigned bucket = 256u + lane;          // unique per lane: matches nobody
            if (i < hi && kind[i] == 0) {
                unsigned key = order_key(s[i]);
                if ((key & mask) == prefix) bucket = (key >> shift) & 255u;
            }
            unsigned peers = __match_any_sync(0xffffffffu, bucket);
            if (bucket < 256u && lane == __ffs(peers) - 1) atomicAdd(&sm.hist[bucket], __popc(peers));
        }
        __syncthreads();
        if (tid < 32) {
            // lane L owns buckets 255-8L .. 248-8L (descending); find where the running count reaches krem
            unsigned c[8], tot = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) { c[t] = sm.hist[255 - 8 * lane - t]; tot += c[t]; }
            unsigned incl = tot;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                unsigned o = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += o;
            }
            unsigned before = incl - tot;           // count in buckets greater than this lane's
            if (before < krem && krem <= incl) {
                unsigned run = before;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    if (run < krem && krem <= run + c[t]) {
                        sm.prefix = prefix | ((unsigned)(255 - 8 * lane - t) << shift);
                        sm.krem = krem - run;
                    }
                    run += c[t];
                }
            }
        }
        __syncthreads();
        prefix = sm.prefix;
        krem = sm.krem;
        mask |= 0xFFu << shift;
        __syncthreads();
    }
    // prefix is now the key of the k-th greatest; krem of the rows equal to it are taken, lowest index first
    unsigned eq_before = 0;
    for (int it = 0; it < iters; ++it) {
        int i = lo + it * nthr + tid;
        bool elig = (i < hi) && kind[i] == 0;
        unsigned key = elig ? order_key(s[i]) : 0u;
        bool gt = elig && key > prefix;
        bool eq = elig && key == prefix;
        unsigned bal = __ballot_sync(0xffffffffu, eq);
        unsigned in_warp = __popc(bal & ((1u << lane) - 1u));
        __syncthreads();
        if (lane == 0) sm.warp_cnt[tid >> 5] = __popc(bal);
        __syncthreads();
        unsigned before = 0, all = 0;
        for (int w = 0; w < (nthr >> 5); ++w) {
            unsigned c = sm.warp_cnt[w];
            if (w < (tid >> 5)) before += c;
            all += c;
        }
        if (gt || (eq && eq_before + before + in_warp < krem)) kind[i] = mark;
        eq_before += all;
    }
    __syncthreads();
}

}  // namespace cask
