// Assignment of scratch rows to seeds on the tensor cores (Sec. 2.5: cosine as the base merge
// geometry): D[row, seed] = <k_row, k_seed> for 128-row tiles of the decode region against the
// unit's m <= 256 gathered seed keys, then per row the argmax of the cosine and the threshold tau.
//
// The contraction is small (2*128*m*128 flop per tile) next to the 32 KB of K it consumes, so the
// kernel is bound by the K stream: a 4-stage TMA ring feeds one persistent CTA per SM.
//   warp 0      TMA producer: seed matrix once per unit, K tiles through the ring
//   warp 1      TMEM allocation, tcgen05.mma issue
//   warps 4-19  epilogue in groups of four warps (one per TMEM lane quadrant); group e takes the
//               tiles e, e+G, e+2G, ... of the CTA and owns one accumulator buffer, so up to G
//               tiles are in flight and the global-memory round trips of a tile (row kind, score,
//               the fixed-point mass atomics) overlap with the next tiles
// With m <= 128 seeds in every unit the TMEM holds four buffers of 128 columns, one per group.  With more
// seeds it holds two buffers of 256 columns and two groups share each: one takes the first seed columns and
// finishes the row, the other takes the rest and hands its best seed over through shared memory.
#include "tc_common.cuh"

namespace cask {

namespace {

using namespace tc;

constexpr int kTileRows = 128;
constexpr int kStages = 4;
constexpr int kEpiWarp0 = 4;
constexpr int kMaxGroups = 4;
constexpr int kThreadsA = (kEpiWarp0 + 4 * kMaxGroups) * 32;
// A parity wait is only sound for a waiter that has seen the phase before the one it waits for complete: a phase
// further behind has the same parity as the one awaited and the wait would pass at once.  Tile t uses key stage
// t % kStages and belongs to epilogue group t % n_bufs (n_bufs = 4 or 2), so with kStages a multiple of n_bufs a group
// meets every phase of the stages it reads, in order.  Any other ring depth lets a fast group reach a stage whose
// previous tile (another group's) has not landed yet, pass the wait and release the stage early.
static_assert(kStages % kMaxGroups == 0, "key ring depth must be a multiple of the epilogue group count");
constexpr uint32_t kSeedRegionBytes = 256 * 128;       // 256 seeds x 64 bf16
constexpr uint32_t kSeedBytes = 2 * kSeedRegionBytes;
constexpr uint32_t kKRegionBytes = 128 * 128;
constexpr uint32_t kKStageBytes = 2 * kKRegionBytes;

struct __align__(8) ABarriers {
    uint64_t b_full[2], b_empty[2];   // seed matrix buffers (two when every unit has at most 128 columns)
    uint64_t k_full[kStages], k_empty[kStages];
    uint64_t d_full[kMaxGroups], d_empty[kMaxGroups];
    uint64_t inv_ready[kMaxGroups];   // a group's table of inverse seed norms is written
    uint64_t x_full[2];      // shared buffers: the second group's best seed of a tile is in shared memory
    uint64_t mma_drain;      // give-up path only: the contractions in flight have completed
};

struct ASmemTail {
    ABarriers bar;
    uint32_t tmem_base;
    int abort;
    alignas(16) float inv_nu[kMaxGroups][2][256];   // 1/|k_seed| (0 for a zero seed): every epilogue group keeps its
                                        // own copy, double-buffered over the units it has tiles in
    int seed_row[kMaxGroups][2][256];   // cache row of every seed of the unit, buffered the same way
    alignas(16) float w[128]; // channel weights of the similarity (1 when none are given)
    float x_val[2][2][128];   // shared buffers: best dot product / seed norm and its seed,
    int x_idx[2][2][128];     //   per buffer, per use parity, per tile row
};

constexpr size_t kSmemBytesA = 1024 + kSeedBytes + kStages * kKStageBytes + sizeof(ASmemTail);

// Walks this CTA's contiguous range of scratch tiles, unit by unit.
struct TileWalk {
    const UnitDesc* desc;
    int g, g_end, u, n_units;
    __device__ void init(const UnitDesc* d, int n_units_, int total) {
        desc = d;
        n_units = n_units_;
        g = (int)(((long long)total * blockIdx.x) / gridDim.x);
        g_end = (int)(((long long)total * (blockIdx.x + 1)) / gridDim.x);
        int lo = 0, hi = n_units - 1;
        while (lo < hi) {                       // last unit with atile0 <= g
            int mid = (lo + hi + 1) >> 1;
            if (d[mid].atile0 <= g) lo = mid; else hi = mid - 1;
        }
        u = lo;
        skip_empty();
    }
    __device__ void skip_empty() {
        while (u < n_units - 1 && g >= desc[u].atile0 + desc[u].n_atiles) ++u;
    }
    __device__ bool valid() const { return g < g_end; }
    __device__ int tile_in_unit() const { return g - desc[u].atile0; }
    // tiles of the current unit that belong to this CTA from g on
    __device__ int run() const { return min(g_end, desc[u].atile0 + desc[u].n_atiles) - g; }
    __device__ void advance(int n) {
        g += n;
        if (g < g_end) { ++u; skip_empty(); }
    }
};

// 16 bytes of shared memory by a shared-space load (through a generic pointer the read takes the path of global loads).
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(a));
    return r;
}

// Squared (channel-weighted) norm of one staged key row as a packed pair of partial sums.  The row's sixteen
// 16-byte pieces are read in a lane-dependent order (no bank conflicts); a bf16 is the upper half of an fp32, so
// two integer operations unpack a pair.  The 128-byte swizzle stores logical piece p of row r at position
// p ^ (r & 7), which matters only for finding the piece's channel weights.  Four running sums, one per 32-bit
// word of a piece, keep the dependent chain of packed multiply-adds at sixteen links instead of sixty-four.
template <bool WEIGHTED>
__device__ __forceinline__ uint64_t row_norm2(const uint8_t* base, int lane, int row, const float* w) {
    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
    const uint32_t b32 = smem_u32(base);
#pragma unroll
    for (int kb = 0; kb < 2; ++kb)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int pos = (c + lane) & 7;
            const uint4 raw = lds128(b32 + kb * kKRegionBytes + (pos << 4));
            const uint32_t wv[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const uint64_t f2 = pack2(__uint_as_float(wv[x] << 16), __uint_as_float(wv[x] & 0xFFFF0000u));
                if (WEIGHTED) {
                    const float2 w2 = *reinterpret_cast<const float2*>(&w[kb * 64 + ((pos ^ (row & 7)) << 3) + 2 * x]);
                    acc[x] = fma2(fma2(f2, pack2(w2.x, w2.y), 0ull), f2, acc[x]);
                } else {
                    acc[x] = fma2(f2, f2, acc[x]);
                }
            }
        }
    return add2(add2(acc[0], acc[1]), add2(acc[2], acc[3]));
}

// Best seed among the accumulator columns [c_lo, c_hi) of this thread's row: the greatest dot * 1/|k_seed|, the
// first seed among equals.  PAIR = 1: a seed owns two adjacent columns (the hi and lo parts of its weighted key)
// whose sum is its dot product.  A block of 32 columns costs a multiply and a maximum per seed; the position of
// the maximum is looked for only in a block that beats everything before it.
template <int PAIR>
__device__ __forceinline__ void best_seed(uint32_t taddr, const float* inv, int c_lo, int c_hi, float& best, int& best_u) {
    constexpr int kPer = PAIR ? 16 : 32;          // seeds per block of 32 columns
    const uint32_t inv32 = smem_u32(inv);        // full blocks read the inverse norms 16 bytes at a time, shared-space
    for (int cc = c_lo; cc < c_hi; cc += 32) {
        float v[32];
        tc_ld32(taddr + cc, v);
        tc_wait_ld_regs(v);
        const int u0 = PAIR ? cc >> 1 : cc, u_hi = PAIR ? c_hi >> 1 : c_hi;
        float bm = -INFINITY;
        if (cc + 32 <= c_hi) {
#pragma unroll
            for (int x = 0; x < kPer; x += 4) {
                const uint4 q = lds128(inv32 + (uint32_t)(u0 + x) * 4u);
                const float nv[4] = {__uint_as_float(q.x), __uint_as_float(q.y), __uint_as_float(q.z), __uint_as_float(q.w)};
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    v[x + y] = (PAIR ? v[2 * (x + y)] + v[2 * (x + y) + 1] : v[x + y]) * nv[y];
                    bm = fmaxf(bm, v[x + y]);
                }
            }
        } else {
#pragma unroll
            for (int x = 0; x < kPer; ++x) {
                const float dot = PAIR ? v[2 * x] + v[2 * x + 1] : v[x];
                v[x] = (u0 + x < u_hi) ? dot * inv[u0 + x] : -INFINITY;
                bm = fmaxf(bm, v[x]);
            }
        }
        if (bm > best) {
            best = bm;
            int at = kPer - 1;
#pragma unroll
            for (int x = kPer - 2; x >= 0; --x)
                if (v[x] == bm) at = x;
            best_u = u0 + at;
        }
    }
}

__global__ void __launch_bounds__(kThreadsA, 1)
assign_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmSeed,
                 const UnitDesc* __restrict__ desc, Shape sh, int total_tiles, int n_bufs, int sub_rows, int wpair,
                 const float* __restrict__ s, const int32_t* __restrict__ plan,
                 const int32_t* __restrict__ seed_rows, const float* __restrict__ seed_norm,
                 uint8_t* __restrict__ kind, int32_t* __restrict__ seed_of, float* __restrict__ sim,
                 int32_t* __restrict__ grp, unsigned long long* __restrict__ mass_fx,
                 int32_t* __restrict__ njoin, int max_m, float tau, float eps, int32_t* __restrict__ err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* b_smem = smem;
    uint8_t* k_smem = smem + kSeedBytes;
    ASmemTail* tail = reinterpret_cast<ASmemTail*>(k_smem + kStages * kKStageBytes);
    ABarriers& bar = tail->bar;
    volatile int* abort_flag = &tail->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int buf_cols = 512 / n_bufs;                   // TMEM columns per accumulator buffer
    const int split = kMaxGroups / n_bufs;               // groups sharing one buffer (1 or 2)
    // At most 128 accumulator columns in every unit: the seed matrix is loaded as 128 rows and the shared-memory
    // area holds two of them, so the next unit's seeds arrive while the tensor pipe still works on this unit's.
    const bool dual = n_bufs == kMaxGroups;
    // n_bufs is 2 or 4: positions among the buffers by mask and shift (a remainder by a run-time value is a division
    // sequence, and the epilogue warps take one per tile, their own or not)
    const uint32_t buf_mask = (uint32_t)n_bufs - 1u, buf_shift = n_bufs == 4 ? 2u : 1u;
    const uint32_t seed_region = dual ? 128u * 128u : kSeedRegionBytes;      // one 64-channel half of a seed buffer

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(&bar.b_full[i], 1); mbar_init(&bar.b_empty[i], 1); }
        for (int i = 0; i < kStages; ++i) { mbar_init(&bar.k_full[i], 1); mbar_init(&bar.k_empty[i], 1 + 4); }
        for (int i = 0; i < kMaxGroups; ++i) { mbar_init(&bar.d_full[i], 1); mbar_init(&bar.d_empty[i], 4 * split); }
        for (int i = 0; i < kMaxGroups; ++i) mbar_init(&bar.inv_ready[i], 128);
        mbar_init(&bar.x_full[0], 4);
        mbar_init(&bar.x_full[1], 4);
        mbar_init(&bar.mma_drain, 1);
        tail->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 128) tail->w[threadIdx.x] = sh.chan_w ? sh.chan_w[threadIdx.x] : 1.f;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tail->tmem_base)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tail->tmem_base;

    TileWalk wk;
    wk.init(desc, sh.n_units, total_tiles);

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t kit = 0, ucount = 0;
            bool ok = true;
            while (wk.valid() && ok) {
                const UnitDesc& ud = desc[wk.u];
                const uint32_t sb = dual ? (ucount & 1u) : 0u, suse = dual ? (ucount >> 1) : ucount;
                ok = mbar_wait(&bar.b_empty[sb], (suse & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                mbar_expect_tx(&bar.b_full[sb], 2 * seed_region);
                uint8_t* bdst = b_smem + sb * 2 * seed_region;
                tma_load_2d(bdst, &tmSeed, &bar.b_full[sb], 0, ud.seed_base << wpair);
                tma_load_2d(bdst + seed_region, &tmSeed, &bar.b_full[sb], 64, ud.seed_base << wpair);
                ++ucount;
                // first cache row of the unit's tile sequence (a page-piece boundary in a paged cache)
                const int a0 = ud.P - (sh.page_size ? ud.P % sub_rows : 0);
                const int lrow0 = a0 + wk.tile_in_unit() * kTileRows;
                const int krow0 = sh.page_size ? 0 : (int)(ud.k_off / sh.row_stride);
                const int nt = wk.run();
                for (int t = 0; t < nt && ok; ++t, ++kit) {
                    const int st = kit % kStages;
                    ok = mbar_wait(&bar.k_empty[st], ((kit / kStages) & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    uint8_t* dst = k_smem + st * kKStageBytes;
                    const int lrow = lrow0 + t * kTileRows;
                    if (sh.page_size == 0) {
                        mbar_expect_tx(&bar.k_full[st], kKStageBytes);
                        tma_load_2d(dst, &tmK, &bar.k_full[st], 0, krow0 + lrow);
                        tma_load_2d(dst + kKRegionBytes, &tmK, &bar.k_full[st], 64, krow0 + lrow);
                    } else {
                        const int n_sub = min(kTileRows / sub_rows, (ud.T - lrow + sub_rows - 1) / sub_rows);
                        mbar_expect_tx(&bar.k_full[st], (uint32_t)n_sub * sub_rows * 256u);
                        for (int sb = 0; sb < n_sub; ++sb) {
                            const int prow = (int)paged_row(sh, ud, lrow + sb * sub_rows);
                            tma_load_2d(dst + sb * sub_rows * 128, &tmK, &bar.k_full[st], 0, prow);
                            tma_load_2d(dst + kKRegionBytes + sb * sub_rows * 128, &tmK, &bar.k_full[st], 64, prow);
                        }
                    }
                }
                wk.advance(nt);
            }
            if (!ok) {
                for (uint32_t j = (kit >= (uint32_t)kStages ? kit - kStages : 0); j < kit; ++j)
                    for (uint32_t it = 0; it < 4096 && !mbar_try(&bar.k_full[j % kStages], (j / kStages) & 1u); ++it) {}
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            uint32_t kit = 0, ucount = 0;
            bool ok = true;
            const uint32_t b_lo = umma_desc_lo(smem_u32(b_smem)), k_lo = umma_desc_lo(smem_u32(k_smem));
            while (wk.valid() && ok) {
                const UnitDesc& ud = desc[wk.u];
                const int m = max(0, min(plan[wk.u * 8 + CASK_PLAN_M], ud.plan[CASK_PLAN_M]));
                const uint32_t idesc = umma_idesc(max(16, ((m << wpair) + 15) & ~15));
                const uint32_t sb = dual ? (ucount & 1u) : 0u, suse = dual ? (ucount >> 1) : ucount;
                ok = mbar_wait(&bar.b_full[sb], suse & 1u, abort_flag);
                if (!ok) break;
                ++ucount;
                const uint32_t bu_lo = b_lo + ((sb * 2 * seed_region) >> 4), half_lo = seed_region >> 4;
                const int nt = wk.run();
                for (int t = 0; t < nt && ok; ++t, ++kit) {
                    const int st = kit % kStages;
                    const uint32_t buf = kit & buf_mask, use = kit >> buf_shift;
                    ok = mbar_wait(&bar.k_full[st], (kit / kStages) & 1u, abort_flag);
                    if (!ok) break;
                    ok = mbar_wait(&bar.d_empty[buf], (use & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t kst_lo = k_lo + st * (kKStageBytes >> 4);
                    const uint32_t d_addr = tmem_base + buf * buf_cols;
                    tc_mma_lo<false>(d_addr, kst_lo, bu_lo, idesc);
#pragma unroll
                    for (int kk = 1; kk < 8; ++kk) {
                        const int kb = kk >> 2, ks = kk & 3;
                        tc_mma_lo<true>(d_addr, kst_lo + ((kb * kKRegionBytes + ks * 32) >> 4),
                                        bu_lo + kb * half_lo + ((ks * 32) >> 4), idesc);
                    }
                    tc_commit(&bar.d_full[buf]);
                    tc_commit(&bar.k_empty[st]);
                }
                wk.advance(nt);
                if (ok) tc_commit(&bar.b_empty[sb]);
            }
            if (!ok) {
                // contractions already issued may still be running: the TMEM they write is freed below, so give them
                // a bounded wait (a commit completes when everything this thread issued before it has)
                tc_commit(&bar.mma_drain);
                for (uint32_t it = 0; it < 4096 && !mbar_try(&bar.mma_drain, 0u); ++it) {}
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ================= epilogue =================
        const int ew = warp - kEpiWarp0;
        const int qd = ew & 3;                               // TMEM lane quadrant (== warp % 4)
        const uint32_t eg = (uint32_t)(ew >> 2) & buf_mask;   // buffer: tiles eg, eg + n_bufs, ...
        const int half = (ew >> 2) >> buf_shift;                 // 0: finishes the row; 1: the later seed columns only
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * qd) << 16) + eg * buf_cols;
        const int my_row = 32 * qd + lane;                   // row of the tile this thread owns
        uint32_t kit = 0, ucount = 0;
        bool ok = true;
        while (wk.valid() && ok) {
            const UnitDesc& ud = desc[wk.u];
            const int u = wk.u;
            const int T = ud.T, P = ud.P;
            const int64_t tok_off = ud.tok_off;
            const int seed_base = ud.seed_base;
            const int r = max(0, min(plan[u * 8 + CASK_PLAN_R], T - P));
            const int m = max(0, min(plan[u * 8 + CASK_PLAN_M], ud.plan[CASK_PLAN_M]));
            const int hi = T - r;
            const int a0 = P - (sh.page_size ? P % sub_rows : 0);
            // shared buffers: the finishing group also computes the row norm, so it takes fewer seed columns
            const int mc = m << wpair;               // accumulator columns in use
            const int c_split = split == 2 ? min(mc, 32 * max(1, (((mc + 31) >> 5) - 2) / 2)) : mc;
            unsigned long long* mass_u = mass_fx + (size_t)u * (max_m + 1);
            const int tile0 = wk.tile_in_unit();
            const int nt = wk.run();
            // Does this group take a tile of the unit?  Only then it needs the table of inverse seed norms; it
            // builds its own copy (two values per thread) and meets on its own barrier, so the groups never
            // wait for one another between units.
            const int first = (int)((eg + (uint32_t)n_bufs - (kit & buf_mask)) & buf_mask);
            if (first >= nt) {
                kit += nt;
                wk.advance(nt);
                continue;
            }
            float* inv = tail->inv_nu[ew >> 2][ucount & 1u];
            int* srow = tail->seed_row[ew >> 2][ucount & 1u];
            {
                const int gt = (ew & 3) * 32 + lane;           // thread of the group
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c = gt + 128 * h;
                    const float nu = (c < m) ? seed_norm[seed_base + c] : 0.f;
                    inv[c] = nu > 0.f ? 1.f / nu : 0.f;
                    srow[c] = (c < m) ? seed_rows[seed_base + c] : 0;
                }
                mbar_arrive(&bar.inv_ready[ew >> 2]);
                ok = mbar_wait(&bar.inv_ready[ew >> 2], ucount & 1u, abort_flag);
                if (!ok) break;
            }
            ++ucount;
            uint8_t kd_n = (uint8_t)CASK_KIND_RECENT;
            float s_n = 0.f, mi_n = 0.f;
            bool pre = false;
            for (int t = 0; t < nt && ok; ++t, ++kit) {
                if ((kit & buf_mask) != eg) continue;
                const int st = kit % kStages;
                const uint32_t use = kit >> buf_shift;
                if (half == 1) {
                    // second group of a shared buffer: best seed among the columns [c_split, m)
                    ok = mbar_wait(&bar.d_full[eg], use & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    float best = -INFINITY;
                    int best_u = -1;
                    if (wpair) best_seed<1>(taddr, inv, c_split, mc, best, best_u);
                    else best_seed<0>(taddr, inv, c_split, mc, best, best_u);
                    tc_fence_before();
                    tail->x_val[eg][use & 1u][my_row] = best;
                    tail->x_idx[eg][use & 1u][my_row] = best_u;
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(&bar.d_empty[eg]);
                        mbar_arrive(&bar.x_full[eg]);
                    }
                    continue;
                }
                // The row's kind and score are used after the contraction.  They were requested during this
                // group's previous tile of the unit (a load issued here would still be waited for before the
                // norm: the cache is saturated by the key stream and a miss costs well over a thousand cycles);
                // only a group's first tile of a unit loads them directly.
                const int i = a0 + (tile0 + t) * kTileRows + my_row;
                const bool in_range = i >= P && i < hi;
                uint8_t kd = (uint8_t)CASK_KIND_RECENT;
                float s_c = 0.f, mi_c = 0.f;
                if (pre) {
                    kd = kd_n; s_c = s_n; mi_c = mi_n;
                } else if (in_range) {
                    kd = kind[tok_off + i];
                    s_c = s[tok_off + i];
                    if (sh.mass_in) mi_c = sh.mass_in[tok_off + i];
                }
                // the same fields of this group's next tile of the unit, in flight during this tile (a row's kind
                // is read and written by the thread that owns the row only, so reading it early sees the same byte)
                pre = t + n_bufs < nt;
                kd_n = (uint8_t)CASK_KIND_RECENT; s_n = 0.f; mi_n = 0.f;
                if (pre) {
                    const int in_ = i + n_bufs * kTileRows;
                    if (in_ >= P && in_ < hi) {
                        kd_n = kind[tok_off + in_];
                        s_n = s[tok_off + in_];
                        if (sh.mass_in) mi_n = sh.mass_in[tok_off + in_];
                    }
                }
                // squared norm of this thread's row, read from the staged tile (any order of the
                // sixteen 16-byte pieces of the row gives the same set of elements)
                ok = mbar_wait(&bar.k_full[st], (kit / kStages) & 1u, abort_flag);
                if (!ok) break;
                uint64_t n2p = 0ull;
                {
                    const uint8_t* base = k_smem + st * kKStageBytes + my_row * 128;
                    if (!sh.chan_w) n2p = row_norm2<false>(base, lane, my_row, tail->w);
                    else n2p = row_norm2<true>(base, lane, my_row, tail->w);
                }
                float n2, n2b;
                unpack2(n2p, n2, n2b);
                n2 += n2b;
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar.k_empty[st]);
                ok = mbar_wait(&bar.d_full[eg], use & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                float best = -INFINITY;
                int best_u = -1;
                if (wpair) best_seed<1>(taddr, inv, 0, c_split, best, best_u);
                else best_seed<0>(taddr, inv, 0, c_split, best, best_u);
                tc_fence_before();
                if (split == 2) {
                    // The other group's candidate has the larger seed indices, so it wins only when strictly
                    // better: the same outcome as one scan over all columns.  The buffer is released after this
                    // read, so the other group cannot start the buffer's next use (and overwrite its hand-over
                    // slot or run a barrier phase ahead) before it.
                    ok = mbar_wait(&bar.x_full[eg], use & 1u, abort_flag);
                    if (!ok) break;
                    const float ov = tail->x_val[eg][use & 1u][my_row];
                    if (ov > best) {
                        best = ov;
                        best_u = tail->x_idx[eg][use & 1u][my_row];
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar.d_empty[eg]);

                const bool cand = in_range && best_u >= 0 && kd == CASK_KIND_DROPPED;
                float sm_ = 0.f;
                if (cand) {
                    const float nj = sqrtf(n2);              // best = <k_row, k_seed> / |k_seed| (0 for a zero seed)
                    sm_ = nj > 0.f ? best / nj : 0.f;
                    if (sim) sim[tok_off + i] = sm_;
                }
                const bool joined = cand && sm_ >= tau;
                float sc = 0.f;                                   // a_i = score + eps (+ the mass it carries)
                if (in_range) { const float a = s_c + eps; sc = sh.mass_in ? a + mi_c : a; }
                const unsigned long long fx = cand ? mass_to_fx(sc) : 0ull;
                if (joined) {
                    const int bu = CASK_IDX(best_u, m, err);
                    kind[tok_off + i] = CASK_KIND_MERGED;
                    seed_of[tok_off + i] = srow[bu];
                    grp[tok_off + i] = bu;
                    atomicAdd(&mass_u[bu], fx);
                }
                // Joiner count and lost mass go out once per warp: the fixed-point sums are exact, so
                // the grouping of the additions does not show in the result.
                const unsigned jb = __ballot_sync(0xffffffffu, joined);
                unsigned long long lost = joined ? 0ull : fx;
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) lost += __shfl_xor_sync(0xffffffffu, lost, off);
                if (lane == 0) {
                    if (jb) atomicAdd(&njoin[u], __popc(jb));
                    if (lost) atomicAdd(&mass_u[max_m], lost);
                }
            }
            wk.advance(nt);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && tail->abort) atomicOr(err, CASK_ST_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace

// Rows per TMA box of the key stream (see the scoring kernel): 128, one page piece, or 0 if unsupported.
int assign_tc_box_rows(const Shape& sh) {
    if (sh.page_size == 0) return kTileRows;
    if (sh.page_size % kTileRows == 0) return kTileRows;
    if (sh.page_size >= 8 && kTileRows % sh.page_size == 0) return sh.page_size;
    return 0;
}

bool assign_tc_supported(const Launch& L) {
    const Shape& sh = L.sh;
    const int cols = L.max_m << (sh.chan_w ? 1 : 0);      // a weighted seed takes two accumulator columns
    if (sh.dtype != CASK_DTYPE_BF16 || sh.d != 128 || cols > 256 || L.max_m < 1 || L.total_atiles < 1)
        return false;
    if (sh.page_size) return assign_tc_box_rows(sh) != 0 && sh.n_pages * sh.page_size < ((int64_t)1 << 31);
    int64_t max_row = 0;
    for (int u = 0; u < sh.n_units; ++u) {
        const UnitDesc& d = L.hdesc[u];
        if (d.k_off % sh.row_stride != 0) return false;
        max_row = std::max<int64_t>(max_row, d.k_off / sh.row_stride + d.T);
    }
    return max_row < (int64_t)1 << 31;
}

cudaError_t launch_assign_tc(const Launch& L, const cask_params& prm, const float* s, const int32_t* plan,
                             uint8_t* kind, int32_t* seed_of, float* sim, Workspace& ws, void* tmap_encode_fn) {
    const Shape& sh = L.sh;
    int64_t k_rows = sh.page_size ? sh.n_pages * sh.page_size : 0, sum_m = 0;
    for (int u = 0; u < sh.n_units; ++u) {
        if (!sh.page_size) k_rows = std::max<int64_t>(k_rows, L.hdesc[u].k_off / sh.row_stride + L.hdesc[u].T);
        sum_m += L.hdesc[u].plan[CASK_PLAN_M];
    }
    const int sub_rows = assign_tc_box_rows(sh);
    CUtensorMap tmK, tmSeed;
    if (!encode_rows_bf16(tmap_encode_fn, &tmK, L.k, (uint64_t)k_rows, (uint64_t)sh.row_stride * 2, sub_rows))
        return cudaErrorInvalidValue;
    // the seed table has 256 spare rows behind the last seed, so a full box never leaves the allocation
    const int wpair = sh.chan_w ? 1 : 0;
    const int n_bufs = (L.max_m << wpair) <= 128 ? 4 : 2;      // accumulator buffers; four: seed boxes of 128 rows
    if (!encode_rows_bf16(tmap_encode_fn, &tmSeed, ws.seed_k, ((uint64_t)sum_m << wpair) + 256, 256, n_bufs == 4 ? 128 : 256))
        return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int grid = std::max(1, std::min(sms, L.total_atiles));
    e = cudaFuncSetAttribute(assign_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytesA);
    if (e != cudaSuccess) return e;
    {
        Timed t(L, KID_ASSIGN);
        assign_tc_kernel<<<grid, kThreadsA, kSmemBytesA, L.stream>>>(
            tmK, tmSeed, L.desc, sh, L.total_atiles, n_bufs, sub_rows, wpair, s, plan, ws.seed_rows, ws.seed_norm, kind, seed_of, sim, ws.grp,
            ws.mass_fx, ws.njoin, L.max_m, prm.tau, prm.eps, ws.err);
    }
    return cudaGetLastError();
}

}  // namespace cask
