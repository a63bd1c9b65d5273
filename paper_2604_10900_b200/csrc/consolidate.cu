// Scratch consolidation (Sec. 2.1, 2.4, 2.5): seed selection, cosine assignment of the
// remaining scratch rows to seeds, group masses and merge weights.
#include <type_traits>

#include "select.cuh"

namespace cask {

namespace {

constexpr int kTile = 64;
constexpr int kThreads = 256;

// ---- 1. seeds: the m greatest scratch rows; ordered list of their rows -------------------
__global__ void __launch_bounds__(kSelThreads) seeds_kernel(const UnitDesc* __restrict__ desc,
                                                            const float* __restrict__ s,
                                                            const int32_t* __restrict__ plan,
                                                            uint8_t* __restrict__ kind,
                                                            int32_t* __restrict__ seed_of,
                                                            float* __restrict__ weight,
                                                            float* __restrict__ sim, int32_t* __restrict__ grp,
                                                            int32_t* __restrict__ seed_rows,
                                                            unsigned long long* __restrict__ mass_fx,
                                                            int32_t* __restrict__ njoin, int max_m) {
    __shared__ SelectSmem sm;
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int T = ud.T, P = ud.P;
    const int64_t o = ud.tok_off;
    int r = max(0, min(plan[u * 8 + CASK_PLAN_R], T - P));
    int m = max(0, min(plan[u * 8 + CASK_PLAN_M], ud.plan[CASK_PLAN_M]));
    // a row left as MERGED/SEED by an earlier call on the same arrays is scratch again
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        uint8_t kd = kind[o + i];
        if (kd == CASK_KIND_SEED || kd == CASK_KIND_MERGED) kind[o + i] = CASK_KIND_DROPPED;
        seed_of[o + i] = -1;
        weight[o + i] = 0.f;
        grp[o + i] = -1;
        if (sim) sim[o + i] = -2.f;
    }
    for (int j = threadIdx.x; j <= max_m; j += blockDim.x) mass_fx[(size_t)u * (max_m + 1) + j] = 0ull;
    if (threadIdx.x == 0) njoin[u] = 0;
    __syncthreads();
    if (m <= 0) return;
    block_topk_mark(s + o, kind + o, P, T - r, m, CASK_KIND_SEED, sm);
    // ordered list of the seed rows
    block_ordered_rows(kind + o, P, T - r, CASK_KIND_SEED, sm, [&](unsigned idx, int i) {
        if (idx < (unsigned)m) {
            seed_rows[ud.seed_base + idx] = i;
            seed_of[o + i] = i;
            grp[o + i] = (int)idx;
        }
    });
}

// ---- 1 for longer units on the event path: prefix eviction, core and seed selection in one CTA per unit ----
// The same result as prefix_evict_kernel, select_core_kernel and seeds_kernel in turn; the core and the seeds come out of
// one pair of thresholds (block_topk2_mark) and the per-row arrays are initialised once.
__global__ void __launch_bounds__(kSelThreads, 2) decide_long_kernel(
    const UnitDesc* __restrict__ desc, const float* __restrict__ s, int32_t* __restrict__ plan,
    uint8_t* __restrict__ kind, int32_t* __restrict__ seed_of, float* __restrict__ weight, float* __restrict__ sim,
    int32_t* __restrict__ grp, int32_t* __restrict__ seed_rows, unsigned long long* __restrict__ mass_fx,
    int32_t* __restrict__ njoin, int max_m) {
    __shared__ SelectSmem sm, sm2;
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int T = ud.T, P = ud.P;
    const int64_t o = ud.tok_off;
    const int pkeep = ud.plan[CASK_PLAN_PKEEP], c = ud.plan[CASK_PLAN_C], m = max(0, ud.plan[CASK_PLAN_M]);
    const int r = max(0, min(ud.plan[CASK_PLAN_R], T - P));
    if (threadIdx.x < 8) plan[u * 8 + threadIdx.x] = ud.plan[threadIdx.x];
    const uint8_t pre = (P <= pkeep) ? CASK_KIND_PREFIX : CASK_KIND_DROPPED;
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        kind[o + i] = (i < P) ? pre : (i >= T - r ? CASK_KIND_RECENT : CASK_KIND_DROPPED);
        seed_of[o + i] = -1;
        weight[o + i] = 0.f;
        grp[o + i] = -1;
        if (sim) sim[o + i] = -2.f;
    }
    for (int j = threadIdx.x; j <= max_m; j += blockDim.x) mass_fx[(size_t)u * (max_m + 1) + j] = 0ull;
    if (threadIdx.x == 0) njoin[u] = 0;
    __syncthreads();
    if (P > pkeep) block_topk_mark(s + o, kind + o, 0, P, pkeep, CASK_KIND_PREFIX, sm);
    // the rows of [P, T - r) were all set to kind 0 above and the prefix eviction touches [0, P) only
    block_topk2_mark<true>(s + o, kind + o, P, T - r, c, CASK_KIND_CORE, m, CASK_KIND_SEED, sm, sm2);
    if (m <= 0) return;
    block_ordered_rows(kind + o, P, T - r, CASK_KIND_SEED, sm, [&](unsigned idx, int i) {
        if (idx < (unsigned)m) {
            seed_rows[ud.seed_base + idx] = i;
            seed_of[o + i] = i;
            grp[o + i] = (int)idx;
        }
    });
}

// ---- 2. gather seed keys, their norms and their own mass ---------------------------------
template <typename T>
__global__ void seed_gather_kernel(const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K,
                                   const float* __restrict__ s, const int32_t* __restrict__ plan,
                                   const int32_t* __restrict__ seed_rows, T* __restrict__ seed_k,
                                   float* __restrict__ seed_norm, unsigned long long* __restrict__ mass_fx,
                                   int max_m, float eps, int split_rows) {
    // one warp per seed, eight seeds per CTA
    const int u = blockIdx.y, j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const UnitDesc& ud = desc[u];
    const int m = max(0, min(plan[u * 8 + CASK_PLAN_M], ud.plan[CASK_PLAN_M]));
    if (j >= m) return;
    const int row = CASK_IDX(seed_rows[ud.seed_base + j], ud.T, sh.err);
    const T* src = K + row_elem_off(sh, ud, ud.k_off, row);
    // Plain copy, or (channel-weighted similarity on the tensor cores) the weighted key w*k as two rows
    // hi + lo of the cache dtype, so that the bf16 contraction sees w*k to about 2^-17.
    T* dst = seed_k + (size_t)(ud.seed_base + j) * (split_rows ? 2 : 1) * sh.d;
    float n2 = 0.f;
    for (int c = lane; c < sh.d; c += 32) {
        T x = src[c];
        float f = Elem<T>::ld(&x);
        const float wc = sh.chan_w ? sh.chan_w[c] : 1.f;
        if (split_rows) {
            const float wf = wc * f;
            Elem<T>::st(dst + c, wf);
            Elem<T>::st(dst + sh.d + c, wf - Elem<T>::ld(dst + c));
        } else {
            dst[c] = x;
        }
        n2 = fmaf(wc * f, f, n2);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, off);
    if (lane == 0) {
        seed_norm[ud.seed_base + j] = sqrtf(n2);
        atomicAdd(&mass_fx[(size_t)u * (max_m + 1) + j], mass_to_fx(row_mass(sh, s, eps, ud.tok_off + row)));
    }
}

// ---- 1+2 for units of at most kSmallSpan rows: prefix eviction, core selection, seed selection and the seed
// gather in one CTA per unit (the event path; the staged calls keep their own kernels and give the same
// result).  Keys and kinds live in shared memory; every row of a range counts the rows ahead of it in the total
// order (score descending, row ascending), so the c greatest rows of the scratch range are the core and the next
// m the seeds, which is what taking the top c and then the top m of the rest gives.
template <typename T>
__global__ void __launch_bounds__(256, 6) decide_small_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const float* __restrict__ s,
    int32_t* __restrict__ plan, uint8_t* __restrict__ kind, int32_t* __restrict__ seed_of,
    float* __restrict__ weight, float* __restrict__ sim, int32_t* __restrict__ grp,
    int32_t* __restrict__ seed_rows, T* __restrict__ seed_k, float* __restrict__ seed_norm,
    unsigned long long* __restrict__ mass_fx, int32_t* __restrict__ njoin, int max_m, float eps, int split_rows) {
    __shared__ __align__(16) unsigned keys[kSmallSpan];
    __shared__ int32_t seed_list[kSmallSpan];
    __shared__ uint8_t kd[kSmallSpan];
    __shared__ unsigned wsum[8];
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const UnitDesc& ud = desc[u];
    const int T_ = ud.T, P = ud.P;
    const int64_t o = ud.tok_off;
    const int pkeep = ud.plan[CASK_PLAN_PKEEP], c = max(0, ud.plan[CASK_PLAN_C]), m = max(0, ud.plan[CASK_PLAN_M]);
    const int r = max(0, min(ud.plan[CASK_PLAN_R], T_ - P));
    if (tid < 8) plan[u * 8 + tid] = ud.plan[tid];
    const uint8_t pre = (P <= pkeep) ? CASK_KIND_PREFIX : CASK_KIND_DROPPED;
    for (int i = tid; i < T_; i += blockDim.x) {
        keys[i] = order_key(s[o + i]);
        kd[i] = (i < P) ? pre : (i >= T_ - r ? CASK_KIND_RECENT : CASK_KIND_DROPPED);
    }
    __syncthreads();
    // rows of [lo, hi) ahead of row i: greater keys, and equal keys at lower rows.  Four keys per shared-memory
    // load wherever the index is a multiple of four (the key array is 16-byte aligned).
    auto count = [&](int a, int b, unsigned ki, auto ge) {       // #{j in [a,b): keys[j] >= ki (ge) or > ki}
        constexpr bool GE = decltype(ge)::value;
        int n = 0, j = a;
        for (; j < b && (j & 3); ++j) n += GE ? keys[j] >= ki : keys[j] > ki;
        for (; j + 4 <= b; j += 4) {
            const uint4 k4 = *reinterpret_cast<const uint4*>(&keys[j]);
            if (GE) n += (k4.x >= ki) + (k4.y >= ki) + (k4.z >= ki) + (k4.w >= ki);
            else n += (k4.x > ki) + (k4.y > ki) + (k4.z > ki) + (k4.w > ki);
        }
        for (; j < b; ++j) n += GE ? keys[j] >= ki : keys[j] > ki;
        return n;
    };
    auto ahead_of = [&](int lo, int hi, int i) {
        const unsigned ki = keys[i];
        return count(lo, i, ki, std::true_type{}) + count(i + 1, hi, ki, std::false_type{});
    };
    if (P > pkeep && pkeep > 0)
        for (int i = tid; i < P; i += blockDim.x)
            if (ahead_of(0, P, i) < pkeep) kd[i] = CASK_KIND_PREFIX;
    const int lo = P, hi = T_ - r;
    if (c + m > 0)
        for (int i = lo + tid; i < hi; i += blockDim.x) {
            const int a = ahead_of(lo, hi, i);
            if (a < c) kd[i] = CASK_KIND_CORE;
            else if (a < c + m) kd[i] = CASK_KIND_SEED;
        }
    __syncthreads();
    for (int i = tid; i < T_; i += blockDim.x) {
        kind[o + i] = kd[i];
        seed_of[o + i] = -1;
        weight[o + i] = 0.f;
        grp[o + i] = -1;
        if (sim) sim[o + i] = -2.f;
    }
    for (int j = tid; j <= max_m; j += blockDim.x) mass_fx[(size_t)u * (max_m + 1) + j] = 0ull;
    if (tid == 0) njoin[u] = 0;
    // ordered list of the seed rows: one contiguous chunk of the scratch range per thread, one block scan
    const int span = max(hi - lo, 0);
    const int chunk = (span + (int)blockDim.x - 1) / (int)blockDim.x;
    const int b = lo + tid * chunk, e = min(hi, b + chunk);
    unsigned cnt = 0;
    for (int i = b; i < e; ++i) cnt += kd[i] == CASK_KIND_SEED;
    unsigned incl = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) wsum[w] = incl;
    __syncthreads();       // also orders the per-row initialisation above before the seed rows' own entries
    unsigned rank = incl - cnt;
    for (int x = 0; x < w; ++x) rank += wsum[x];
    for (int i = b; i < e; ++i)
        if (kd[i] == CASK_KIND_SEED) {
            if (rank < (unsigned)m) {
                seed_list[rank] = i;
                seed_rows[ud.seed_base + rank] = i;
                seed_of[o + i] = i;
                grp[o + i] = (int)rank;
            }
            ++rank;
        }
    __syncthreads();
    unsigned n_seeds = 0;
    for (int x = 0; x < (int)(blockDim.x >> 5); ++x) n_seeds += wsum[x];
    const int ms = min((int)n_seeds, m);
    // gather the seed keys, their norms and their own mass: one warp per seed, four seeds' rows in flight (offsets
    // first, loads after, with no branch between the loads: a branch per row makes every row wait for the one before)
    const int nwarps = (int)(blockDim.x >> 5);
    constexpr int kPerLane = 4;                       // head_dim <= 128: at most four channels per lane
    constexpr int kSeedsInFlight = 4;
    for (int j0 = w; j0 < ms; j0 += kSeedsInFlight * nwarps) {
        T x[kSeedsInFlight][kPerLane];
        int row[kSeedsInFlight];
        int64_t off[kSeedsInFlight];
#pragma unroll
        for (int q = 0; q < kSeedsInFlight; ++q)
            row[q] = CASK_IDX(seed_list[min(j0 + q * nwarps, ms - 1)], T_, sh.err);
        if (sh.page_size == 0) {
#pragma unroll
            for (int q = 0; q < kSeedsInFlight; ++q) off[q] = ud.k_off + (int64_t)row[q] * sh.row_stride;
        } else {
#pragma unroll
            for (int q = 0; q < kSeedsInFlight; ++q) off[q] = row_elem_off(sh, ud, ud.k_off, row[q]);
        }
        float am[kSeedsInFlight];
#pragma unroll
        for (int q = 0; q < kSeedsInFlight; ++q) {
            const T* src = K + off[q];
#pragma unroll
            for (int k = 0; k < kPerLane; ++k)
                if (lane + 32 * k < sh.d) x[q][k] = src[lane + 32 * k];
            am[q] = s[o + row[q]];
        }
        if (sh.mass_in) {
#pragma unroll
            for (int q = 0; q < kSeedsInFlight; ++q) am[q] = (am[q] + eps) + sh.mass_in[o + row[q]];     // row_mass()
        } else {
#pragma unroll
            for (int q = 0; q < kSeedsInFlight; ++q) am[q] += eps;
        }
#pragma unroll
        for (int q = 0; q < kSeedsInFlight; ++q) {
            const int j = j0 + q * nwarps;
            if (j >= ms) break;
            T* dst = seed_k + (size_t)(ud.seed_base + j) * (split_rows ? 2 : 1) * sh.d;
            float n2 = 0.f;
#pragma unroll
            for (int k = 0; k < kPerLane; ++k) {
                const int ch = lane + 32 * k;
                if (ch >= sh.d) break;
                const float f = Elem<T>::ld(&x[q][k]);
                const float wc = sh.chan_w ? sh.chan_w[ch] : 1.f;
                if (split_rows) {
                    const float wf = wc * f;
                    Elem<T>::st(dst + ch, wf);
                    Elem<T>::st(dst + sh.d + ch, wf - Elem<T>::ld(dst + ch));
                } else {
                    dst[ch] = x[q][k];
                }
                n2 = fmaf(wc * f, f, n2);
            }
#pragma unroll
            for (int off2 = 16; off2 >= 1; off2 >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, off2);
            if (lane == 0) {
                seed_norm[ud.seed_base + j] = sqrtf(n2);
                mass_fx[(size_t)u * (max_m + 1) + j] = mass_to_fx(am[q]);
            }
        }
    }
}

// ---- 3. assignment: cosine of every scratch row against every seed, argmax, threshold -----
template <typename T>
__global__ void __launch_bounds__(kThreads) assign_simt_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const float* __restrict__ s,
    const int32_t* __restrict__ plan, const int32_t* __restrict__ seed_rows, const T* __restrict__ seed_k,
    const float* __restrict__ seed_norm, uint8_t* __restrict__ kind, int32_t* __restrict__ seed_of,
    float* __restrict__ sim, int32_t* __restrict__ grp, unsigned long long* __restrict__ mass_fx,
    int32_t* __restrict__ njoin, int max_m, float tau, float eps) {
    extern __shared__ float smem[];
    const int u = blockIdx.y;
    const UnitDesc& ud = desc[u];
    const int T_ = ud.T, P = ud.P;
    const int r = max(0, min(plan[u * 8 + CASK_PLAN_R], T_ - P));
    const int m = max(0, min(plan[u * 8 + CASK_PLAN_M], ud.plan[CASK_PLAN_M]));
    const int lo = P + blockIdx.x * kTile, hi = T_ - r;
    if (m <= 0 || lo >= hi) return;
    const int d = sh.d, pitch = d + 1;
    float* St = smem;
    float* Rt = smem + kTile * pitch;
    float* rnorm = Rt + kTile * pitch;     // [64] norms of the stationary rows
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    const int nrows = min(kTile, hi - lo);

    // stationary tile: 64 candidate rows
    {
        const int vec_per_row = d / 8;
        for (int idx = threadIdx.x; idx < kTile * vec_per_row; idx += kThreads) {
            int rr = idx / vec_per_row, c8 = (idx % vec_per_row) * 8;
#pragma unroll
            for (int t = 0; t < 8; ++t)
                St[rr * pitch + c8 + t] =
                    (rr < nrows) ? Elem<T>::ld(K + row_elem_off(sh, ud, ud.k_off, lo + rr) + c8 + t) : 0.f;
        }
    }
    __syncthreads();
    {
        // 4 threads per row, fixed combination order
        int rr = threadIdx.x / 4, part = threadIdx.x % 4;
        float n2 = 0.f;
        for (int c = part; c < d; c += 4) n2 = fmaf((sh.chan_w ? sh.chan_w[c] : 1.f) * St[rr * pitch + c], St[rr * pitch + c], n2);
        n2 += __shfl_xor_sync(0xffffffffu, n2, 1);
        n2 += __shfl_xor_sync(0xffffffffu, n2, 2);
        if (part == 0) rnorm[rr] = sqrtf(n2);
    }
    float best[4];
    int best_u[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) { best[a] = -INFINITY; best_u[a] = -1; }

    for (int u0 = 0; u0 < m; u0 += kTile) {
        __syncthreads();
        const int vec_per_row = d / 8;
        const int nseed = min(kTile, m - u0);
        for (int idx = threadIdx.x; idx < kTile * vec_per_row; idx += kThreads) {
            int rr = idx / vec_per_row, c8 = (idx % vec_per_row) * 8;
#pragma unroll
            for (int t = 0; t < 8; ++t)
                Rt[rr * pitch + c8 + t] =
                    (rr < nseed) ? (sh.chan_w ? sh.chan_w[c8 + t] : 1.f) *
                                       Elem<T>::ld(seed_k + (size_t)(ud.seed_base + u0 + rr) * d + c8 + t)
                                 : 0.f;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
        for (int c = 0; c < d; ++c) {
            float sa[4], rb[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) sa[a] = St[(ty + 16 * a) * pitch + c];
#pragma unroll
            for (int b = 0; b < 4; ++b) rb[b] = Rt[(tx + 16 * b) * pitch + c];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(sa[a], rb[b], acc[a][b]);
        }
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int su = u0 + tx + 16 * b;
            if (su >= m) continue;
            float nu = seed_norm[ud.seed_base + su];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                float nj = rnorm[ty + 16 * a];
                float sm_ = (nj > 0.f && nu > 0.f) ? acc[a][b] / (nj * nu) : 0.f;
                if (sm_ > best[a]) { best[a] = sm_; best_u[a] = su; }
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
            float ob = __shfl_xor_sync(0xffffffffu, best[a], off);
            int ou = __shfl_xor_sync(0xffffffffu, best_u[a], off);
            if (ou >= 0 && (ob > best[a] || (ob == best[a] && ou < best_u[a]) || best_u[a] < 0)) {
                best[a] = ob;
                best_u[a] = ou;
            }
        }
        int rr = ty + 16 * a;
        int i = lo + rr;
        if (tx == 0 && rr < nrows && kind[ud.tok_off + i] == CASK_KIND_DROPPED) {
            if (sim) sim[ud.tok_off + i] = best[a];
            unsigned long long fx = mass_to_fx(row_mass(sh, s, eps, ud.tok_off + i));
            if (best_u[a] >= 0 && best[a] >= tau) {
                kind[ud.tok_off + i] = CASK_KIND_MERGED;
                seed_of[ud.tok_off + i] = seed_rows[ud.seed_base + CASK_IDX(best_u[a], m, sh.err)];
                grp[ud.tok_off + i] = best_u[a];
                atomicAdd(&mass_fx[(size_t)u * (max_m + 1) + best_u[a]], fx);
                atomicAdd(&njoin[u], 1);
            } else {
                atomicAdd(&mass_fx[(size_t)u * (max_m + 1) + max_m], fx);
            }
        }
    }
}

// ---- 3b. assignment under the un-squared per-band distance of Sec. 2.5 -----------------------------------------
// d_kappa(k_j, k_u) = sum_f w_f ||k_jf - k_uf||_2 over the rotary bands (pairs of channels), used as the similarity
// 1 - d_kappa / (D_j + D_u), D_x = sum_f w_f ||k_xf||_2.  One square root per (row, seed, band), so the special-
// function pipe bounds it; same tiling as assign_simt_kernel (64 rows x 64 seeds per step, 4 x 4 per thread).
__device__ __forceinline__ float sqrt_fast(float x) {
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T>
__global__ void __launch_bounds__(kThreads) assign_band_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const float* __restrict__ s,
    const int32_t* __restrict__ plan, const int32_t* __restrict__ seed_rows, const T* __restrict__ seed_k,
    uint8_t* __restrict__ kind, int32_t* __restrict__ seed_of, float* __restrict__ sim, int32_t* __restrict__ grp,
    unsigned long long* __restrict__ mass_fx, int32_t* __restrict__ njoin, int max_m, float tau, float eps) {
    extern __shared__ float2 smem2[];
    const int u = blockIdx.y;
    const UnitDesc& ud = desc[u];
    const int T_ = ud.T, P = ud.P;
    const int r = max(0, min(plan[u * 8 + CASK_PLAN_R], T_ - P));
    const int m = max(0, min(plan[u * 8 + CASK_PLAN_M], ud.plan[CASK_PLAN_M]));
    const int lo = P + blockIdx.x * kTile, hi = T_ - r;
    if (m <= 0 || lo >= hi) return;
    const int d = sh.d, nb = d / 2, pitch = nb + 1;      // a row is nb bands of (x, y); odd pitch: no bank conflicts
    float2* St = smem2;                                   // [64][pitch] stationary rows
    float2* Rt = St + kTile * pitch;                      // [64][pitch] seeds of the current step
    float* rlen = reinterpret_cast<float*>(Rt + kTile * pitch);   // [64] D of the stationary rows
    float* slen = rlen + kTile;                           // [64] D of the seeds of the current step
    float* bw = slen + kTile;                             // [d/2] band weights
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    const int nrows = min(kTile, hi - lo);
    const int second = sh.band_layout == 0 ? nb : 1, step = sh.band_layout == 0 ? 1 : 2;   // band f: channels (f*step, f*step + second)
    for (int f = threadIdx.x; f < nb; f += kThreads) bw[f] = sh.band_w[f];
    // rows of a tile into band order
    auto stage = [&](float2* dst, const T* base, int64_t row_off, bool valid, int rr, int f) {
        float2 v = make_float2(0.f, 0.f);
        if (valid) {
            v.x = Elem<T>::ld(base + row_off + f * step);
            v.y = Elem<T>::ld(base + row_off + f * step + second);
        }
        dst[rr * pitch + f] = v;
    };
    for (int idx = threadIdx.x; idx < kTile * nb; idx += kThreads) {
        const int rr = idx / nb, f = idx % nb;
        stage(St, K, rr < nrows ? row_elem_off(sh, ud, ud.k_off, lo + rr) : 0, rr < nrows, rr, f);
    }
    __syncthreads();
    // D of a row: four threads per row, a quarter of the bands each, fixed combination order
    auto band_len = [&](const float2* row, int part) {
        float D = 0.f;
        for (int f = part; f < nb; f += 4) {
            const float2 v = row[f];
            D = fmaf(bw[f], sqrt_fast(fmaf(v.x, v.x, v.y * v.y)), D);
        }
        D += __shfl_xor_sync(0xffffffffu, D, 1);
        D += __shfl_xor_sync(0xffffffffu, D, 2);
        return D;
    };
    {
        const int rr = threadIdx.x / 4, part = threadIdx.x % 4;
        const float D = band_len(St + rr * pitch, part);
        if (part == 0) rlen[rr] = D;
    }
    float best[4];
    int best_u[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) { best[a] = -INFINITY; best_u[a] = -1; }

    for (int u0 = 0; u0 < m; u0 += kTile) {
        __syncthreads();
        const int nseed = min(kTile, m - u0);
        for (int idx = threadIdx.x; idx < kTile * nb; idx += kThreads) {
            const int rr = idx / nb, f = idx % nb;
            stage(Rt, seed_k, (int64_t)(ud.seed_base + u0 + rr) * d, rr < nseed, rr, f);
        }
        __syncthreads();
        {
            const int rr = threadIdx.x / 4, part = threadIdx.x % 4;
            const float D = band_len(Rt + rr * pitch, part);
            if (part == 0) slen[rr] = D;
        }
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 2
        for (int f = 0; f < nb; ++f) {
            const float w = bw[f];
            float2 sv[4], rv[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) sv[a] = St[(ty + 16 * a) * pitch + f];
#pragma unroll
            for (int b = 0; b < 4; ++b) rv[b] = Rt[(tx + 16 * b) * pitch + f];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const float dx = sv[a].x - rv[b].x, dy = sv[a].y - rv[b].y;
                    acc[a][b] = fmaf(w, sqrt_fast(fmaf(dx, dx, dy * dy)), acc[a][b]);
                }
        }
        __syncthreads();        // slen is complete
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int su = u0 + tx + 16 * b;
            if (su >= m) continue;
            const float Du = slen[tx + 16 * b];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const float Dj = rlen[ty + 16 * a];
                float sm_ = (Dj > 0.f && Du > 0.f) ? 1.f - acc[a][b] / (Dj + Du) : 0.f;
                if (sm_ > best[a]) { best[a] = sm_; best_u[a] = su; }
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
            float ob = __shfl_xor_sync(0xffffffffu, best[a], off);
            int ou = __shfl_xor_sync(0xffffffffu, best_u[a], off);
            if (ou >= 0 && (ob > best[a] || (ob == best[a] && ou < best_u[a]) || best_u[a] < 0)) {
                best[a] = ob;
                best_u[a] = ou;
            }
        }
        int rr = ty + 16 * a;
        int i = lo + rr;
        if (tx == 0 && rr < nrows && kind[ud.tok_off + i] == CASK_KIND_DROPPED) {
            if (sim) sim[ud.tok_off + i] = best[a];
            unsigned long long fx = mass_to_fx(row_mass(sh, s, eps, ud.tok_off + i));
            if (best_u[a] >= 0 && best[a] >= tau) {
                kind[ud.tok_off + i] = CASK_KIND_MERGED;
                seed_of[ud.tok_off + i] = seed_rows[ud.seed_base + CASK_IDX(best_u[a], m, sh.err)];
                grp[ud.tok_off + i] = best_u[a];
                atomicAdd(&mass_fx[(size_t)u * (max_m + 1) + best_u[a]], fx);
                atomicAdd(&njoin[u], 1);
            } else {
                atomicAdd(&mass_fx[(size_t)u * (max_m + 1) + max_m], fx);
            }
        }
    }
}

// ---- 4. merge weights w_i = a_i / m_G, lost mass, status ---------------------------------
constexpr int kWeightRows = 4;     // rows per thread
__global__ void weights_kernel(const UnitDesc* __restrict__ desc, Shape sh, const float* __restrict__ s,
                               const int32_t* __restrict__ plan, const int32_t* __restrict__ grp,
                               const unsigned long long* __restrict__ mass_fx,
                               const int32_t* __restrict__ njoin, float* __restrict__ weight,
                               int32_t* __restrict__ unit_status, float* __restrict__ lost_mass, int max_m,
                               float eps, const int32_t* __restrict__ err) {
    const int u = blockIdx.y;
    const UnitDesc& ud = desc[u];
    const unsigned long long* mf = mass_fx + (size_t)u * (max_m + 1);
    const int T = ud.T;
    const int64_t o = ud.tok_off;
    // four rows per thread, a block apart (most rows belong to no group and only read their group index; a CTA
    // per 256 rows spent its time being launched)
    const int i0 = blockIdx.x * (kWeightRows * (int)blockDim.x) + threadIdx.x;
    int gidx[kWeightRows];
#pragma unroll
    for (int j = 0; j < kWeightRows; ++j) {
        const int i = i0 + j * (int)blockDim.x;
        gidx[j] = i < T ? grp[o + i] : -1;
    }
#pragma unroll
    for (int j = 0; j < kWeightRows; ++j) {
        const int i = i0 + j * (int)blockDim.x;
        if (gidx[j] >= 0 && gidx[j] < max_m) weight[o + i] = row_mass(sh, s, eps, o + i) / fx_to_mass(mf[gidx[j]]);
    }
    if (i0 == 0) {
        int fl = plan[u * 8 + CASK_PLAN_FLAGS];
        if ((fl & CASK_ST_DECODE_CONSOLIDATED) && njoin[u] == 0) fl |= CASK_ST_MERGE_INACTIVE;
        unit_status[u] = fl | *err;     // device-side flags of this call (bounded wait gave up, bad page id)
        lost_mass[u] = fx_to_mass(mf[max_m]);
    }
}

template <typename T>
cudaError_t run(const Launch& L, const cask_params& prm, const float* s, const int32_t* plan, uint8_t* kind,
                int32_t* seed_of, float* weight, float* sim, int32_t* unit_status, float* lost_mass,
                Workspace& ws, bool fused) {
    const Shape& sh = L.sh;
    const int max_m = L.max_m;
    const bool use_tc = !L.force_simt && L.tmap_encode && assign_tc_supported(L) && !sh.band_w;
    const bool small_units = L.max_T <= kSmallUnitRows && sh.d <= 128;
    if (fused && !small_units) {
        Timed t(L, KID_SEEDS);
        decide_long_kernel<<<sh.n_units, kSelThreads, 0, L.stream>>>(L.desc, s, const_cast<int32_t*>(plan), kind, seed_of,
                                                                     weight, sim, ws.grp, ws.seed_rows, ws.mass_fx, ws.njoin,
                                                                     max_m);
    } else if (fused) {
        Timed t(L, KID_SEEDS);
        decide_small_kernel<T><<<sh.n_units, 256, 0, L.stream>>>(
            L.desc, sh, (const T*)L.k, s, const_cast<int32_t*>(plan), kind, seed_of, weight, sim, ws.grp, ws.seed_rows,
            (T*)ws.seed_k, ws.seed_norm, ws.mass_fx, ws.njoin, max_m, prm.eps, (use_tc && sh.chan_w) ? 1 : 0);
    } else {
        Timed t(L, KID_SEEDS);
        seeds_kernel<<<sh.n_units, select_threads(L.max_T), 0, L.stream>>>(L.desc, s, plan, kind, seed_of, weight, sim,
                                                               ws.grp, ws.seed_rows, ws.mass_fx, ws.njoin, max_m);
    }
    if (max_m > 0) {
        if (!(fused && small_units)) {
            Timed t(L, KID_SEED_GATHER);
            seed_gather_kernel<T><<<dim3((max_m + 7) / 8, sh.n_units), 256, 0, L.stream>>>(
                L.desc, sh, (const T*)L.k, s, plan, ws.seed_rows, (T*)ws.seed_k, ws.seed_norm, ws.mass_fx, max_m,
                prm.eps, (use_tc && sh.chan_w) ? 1 : 0);
        }
        if (use_tc) {
            cudaError_t e = launch_assign_tc(L, prm, s, plan, kind, seed_of, sim, ws, L.tmap_encode);
            if (e != cudaSuccess) return e;
        } else if (sh.band_w) {
            const size_t smem = (size_t)2 * kTile * (sh.d / 2 + 1) * sizeof(float2) + ((size_t)2 * kTile + sh.d / 2) * sizeof(float);
            cudaError_t e = cudaFuncSetAttribute(assign_band_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem);
            if (e != cudaSuccess) return e;
            Timed t(L, KID_ASSIGN);
            assign_band_kernel<T><<<dim3((L.max_T + kTile - 1) / kTile, sh.n_units), kThreads, smem, L.stream>>>(
                L.desc, sh, (const T*)L.k, s, plan, ws.seed_rows, (const T*)ws.seed_k, kind, seed_of, sim, ws.grp,
                ws.mass_fx, ws.njoin, max_m, prm.tau, prm.eps);
        } else {
        const size_t smem = ((size_t)2 * kTile * (sh.d + 1) + kTile) * sizeof(float);
        cudaError_t e = cudaFuncSetAttribute(assign_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
        const int max_nd = L.max_T;   // upper bound on decode rows of any unit
        Timed t(L, KID_ASSIGN);
        assign_simt_kernel<T><<<dim3((max_nd + kTile - 1) / kTile, sh.n_units), kThreads, smem, L.stream>>>(
            L.desc, sh, (const T*)L.k, s, plan, ws.seed_rows, (const T*)ws.seed_k, ws.seed_norm, kind, seed_of,
            sim, ws.grp, ws.mass_fx, ws.njoin, max_m, prm.tau, prm.eps);
        }
    }
    if (!fused) {      // the event path leaves the weights, the status words and the lost mass to the compaction's scan
        Timed t(L, KID_WEIGHTS);
        weights_kernel<<<dim3((L.max_T + 256 * kWeightRows - 1) / (256 * kWeightRows), sh.n_units), 256, 0, L.stream>>>(
            L.desc, sh, s, plan, ws.grp, ws.mass_fx, ws.njoin, weight, unit_status, lost_mass, max_m, prm.eps, ws.err);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_consolidate(const Launch& L, const cask_params& prm, const float* s, const int32_t* plan,
                               uint8_t* kind, int32_t* seed_of, float* weight, float* sim,
                               int32_t* unit_status, float* lost_mass, Workspace& ws, bool fused) {
    if (L.sh.dtype == CASK_DTYPE_BF16)
        return run<__nv_bfloat16>(L, prm, s, plan, kind, seed_of, weight, sim, unit_status, lost_mass, ws, fused);
    return run<float>(L, prm, s, plan, kind, seed_of, weight, sim, unit_status, lost_mass, ws, fused);
}

}  // namespace cask
