// Windowed attention-mass scoring on the 5th-generation tensor cores (bf16 cache, head_dim 128).
//
// Both passes contract the unit's window queries Q_w [rows<=512, 128] with 128-key tiles of K:
//   pass N (normaliser): D[query, key]  -> per query row a reference r and sum of 2^(y - r)
//   pass S (score mass): D[key, query]  -> per key  sum_r roww_r * 2^(y_kr - rowm_r)
// so that the reduction always runs along the TMEM columns a single thread owns.  The two
// passes use the same shared-memory operand tiles (K-major, 128-byte swizzle, written by
// TMA); only the role of the operands (A <-> B) differs.
//
// One persistent CTA per SM, 20 warps:
//   warp 0      TMA producer (one lane): Q once per segment, K tiles through a 2-stage ring
//   warps 1-2   one lane each issues tcgen05.mma and the commits: warp 1 for the even accumulator
//               slots, warp 2 for the odd ones, so that one keeps the tensor pipe fed while the other
//               waits for a slot to be released (warp 1 also owns the TMEM allocation)
//   warps 4-19  epilogue: tcgen05.ld of the fp32 accumulators + the exponentials
// The 512 TMEM columns are four accumulator slots of 128 columns (one 128-row block of
// queries each).  The epilogue warps form two groups of eight (two per TMEM lane quadrant, 64
// columns each); group g drains slots g and g+2 in turn, so while it works on one of its
// slots the tensor pipe refills the other and neither side waits for the other.
//
// The exponentials are the bottleneck (16 ex2 per clock per SM against 65,536 per tile), so a
// fixed share of the columns is evaluated on the FMA pipe instead: round-to-nearest split
// 2^t = 2^n * 2^f, |f| <= 1/2, degree-5 minimax polynomial for 2^f (relative error 2.4e-7,
// the same order as ex2.approx).
//
// Work is split by tiles, not by units: CTA b owns the contiguous tile range
// [total*b/grid, total*(b+1)/grid) of the unit-major tile sequence and walks it segment by
// segment (a segment = its tiles inside one unit).  Pass N leaves one partial per segment
// row and column half at index 2*(unit + CTA) + half; score_tc_combine folds them.  Every mbarrier wait is
// bounded; when one gives up the CTA raises an error flag, drains and frees its TMEM.
#include "tc_common.cuh"

namespace cask {

namespace {

using namespace tc;

constexpr int kTileKeys = 128;
constexpr int kD = 128;
constexpr int kStages = 2;
constexpr int kSlots = 4;                 // accumulator slots of 128 TMEM columns
constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 4 * kSlots;
constexpr int kThreadsTc = (kEpiWarp0 + kEpiWarps) * 32;
constexpr uint32_t kQRegionBytes = 256 * 128;          // 256 rows x 64 bf16
constexpr uint32_t kQBytes = 4 * kQRegionBytes;        // 2 row halves x 2 K blocks
constexpr uint32_t kQBlockBytes = 128 * 128;           // one 128-row query block inside a region
constexpr uint32_t kKRegionBytes = 128 * 128;          // 128 keys x 64 bf16
constexpr uint32_t kKStageBytes = 2 * kKRegionBytes;
constexpr int kMaxSms = 1024;                          // upper bound used when sizing the partial tables

// Columns (of every 32) whose exponential runs on the FMA pipe.
constexpr uint32_t kPolyMaskN = 0x80808080u;
constexpr uint32_t kPolyPairsS = 0x8080u;      // pairs of columns (of the 16 in a block of 32) on the FMA pipe
// the same for the 8 pairs of a 16-column chunk of the streamed path (normaliser pass / score pass)
constexpr uint32_t kPolyPairs16N = 0x80u;
constexpr uint32_t kPolyPairs16S = 0x80u;

struct __align__(8) Barriers {
    uint64_t q_full[kSlots], q_empty[kSlots];   // one pair per 128-row block of the window queries
    uint64_t k_full[kStages], k_empty[kStages];
    uint64_t d_full[kSlots], d_empty[kSlots];
    uint64_t rw_ready;      // pass S: the row table of the segment is written
    uint64_t red_full[8];   // pass S: every warp's partial key sums of a tile are in shared memory
    uint64_t mma_drain[2];  // give-up path only: an issuer's contractions in flight have completed
};

struct TcSmemTail {
    Barriers bar;
    uint32_t tmem_base;
    int abort;
    alignas(16) float rc[3][512];  // pass S: log2(roww) - rowm per query row, one buffer per segment in turn
    float red[8][4][128];         // pass S: partial key sums per (group, column half), eight tiles deep
};

constexpr size_t kSmemBytes = 1024 + kQBytes + kStages * kKStageBytes + sizeof(TcSmemTail);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

// 2^t for t in [-125, 125] on the FMA pipe.
__device__ __forceinline__ float ex2_poly(float t) {
    const float fl = t + 12582912.f;              // 1.5 * 2^23: the integer nearest to t lands in the low mantissa bits
    const float f = t - (fl - 12582912.f);        // |f| <= 1/2
    float p = 1.327644451521337e-3f;
    p = fmaf(p, f, 9.67553723603487e-3f);
    p = fmaf(p, f, 5.550713464617729e-2f);
    p = fmaf(p, f, 2.4022120237350464e-1f);
    p = fmaf(p, f, 6.931469440460205e-1f);
    p = fmaf(p, f, 1.0000001192092896f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(fl) << 23));
}

// 2^t for a pair of t in [-125, 125] on the FMA pipe (packed arithmetic).
__device__ __forceinline__ uint64_t ex2_poly2(uint64_t t2) {
    const uint64_t magic = pack2(12582912.f, 12582912.f);
    const uint64_t fl = add2(t2, magic);
    const uint64_t f = sub2(t2, sub2(fl, magic));
    uint64_t p = pack2(1.327644451521337e-3f, 1.327644451521337e-3f);
    p = fma2(p, f, pack2(9.67553723603487e-3f, 9.67553723603487e-3f));
    p = fma2(p, f, pack2(5.550713464617729e-2f, 5.550713464617729e-2f));
    p = fma2(p, f, pack2(2.4022120237350464e-1f, 2.4022120237350464e-1f));
    p = fma2(p, f, pack2(6.931469440460205e-1f, 6.931469440460205e-1f));
    p = fma2(p, f, pack2(1.0000001192092896f, 1.0000001192092896f));
    float p0, p1, n0, n1;
    unpack2(p, p0, p1);
    unpack2(fl, n0, n1);
    return pack2(__int_as_float(__float_as_int(p0) + (__float_as_int(n0) << 23)),
                 __int_as_float(__float_as_int(p1) + (__float_as_int(n1) << 23)));
}

// 16 bytes of the row table by a shared-space load: through a generic pointer the same read goes the way of
// global loads and comes back later (the score pass is 2.5 % faster this way).
__device__ __forceinline__ float4 lds_f4(uint32_t a) {
    float4 r;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(a));
    return r;
}

// Sum of the n <= 4 partial key sums of one key (one per epilogue group and column half, 128 floats apart), added in
// that order; the four reads are independent shared-space loads, so the fold costs one latency and not four.
__device__ __forceinline__ float fold_partials(const float* p, int n) {
    const uint32_t a = smem_u32(p);
    float v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[k]) : "r"(a + 512u * (uint32_t)min(k, n - 1)));
    float acc = v[0];
#pragma unroll
    for (int k = 1; k < 4; ++k)
        if (k < n) acc += v[k];
    return acc;
}

// Pass S, one block of 32 query columns (rows r0..r0+31 of the window) for the key this thread owns:
// adds sum_r 2^(y_r*scale2 + nc[r]) over the visible rows to the two packed pairs of partial sums.
// Pairs of columns go through packed fp32 instructions; the pairs named by kPolyPairsS take the polynomial.
__device__ __forceinline__ void mass_block(const float (&v)[32], const float* nc, int r0, bool fast, int causal, int W,
                                           int jmin, float scale2, uint64_t& a01, uint64_t& a23) {
    if (fast) {
        const uint32_t nc32 = smem_u32(&nc[r0]);
        const uint64_t s2 = pack2(scale2, scale2);
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const float4 c4 = lds_f4(nc32 + 16u * x);
            const uint64_t tA = fma2(pack2(v[4 * x], v[4 * x + 1]), s2, pack2(c4.x, c4.y));
            const uint64_t tB = fma2(pack2(v[4 * x + 2], v[4 * x + 3]), s2, pack2(c4.z, c4.w));
            float t0, t1, t2, t3;
            unpack2(tA, t0, t1);
            unpack2(tB, t2, t3);
            if ((kPolyPairsS >> (2 * x)) & 1u) a01 = add2(a01, ex2_poly2(pack2(fmaxf(t0, -125.f), fmaxf(t1, -125.f))));
            else a01 = add2(a01, pack2(ex2(t0), ex2(t1)));
            if ((kPolyPairsS >> (2 * x + 1)) & 1u) a23 = add2(a23, ex2_poly2(pack2(fmaxf(t2, -125.f), fmaxf(t3, -125.f))));
            else a23 = add2(a23, pack2(ex2(t2), ex2(t3)));
        }
    } else {
        float a = 0.f;
        if (!causal || (W & 31) == 0) {
            // the 32 rows of the block lie inside one head (r0 is a multiple of 32): one threshold for the block
            const int thr = causal ? jmin - r0 % W : 0;
            // arguments in packed pairs from 16-byte reads of the row table; only the exponentials of the visible
            // columns are issued (the ex2 pipe is the bottleneck), into four independent sums
            const uint32_t nc32 = smem_u32(&nc[r0]);
            const uint64_t s2 = pack2(scale2, scale2);
            float b1 = 0.f, b2 = 0.f, b3 = 0.f;
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const float4 c4 = lds_f4(nc32 + 16u * x);
                float t0, t1, t2, t3;
                unpack2(fma2(pack2(v[4 * x], v[4 * x + 1]), s2, pack2(c4.x, c4.y)), t0, t1);
                unpack2(fma2(pack2(v[4 * x + 2], v[4 * x + 3]), s2, pack2(c4.z, c4.w)), t2, t3);
                if (4 * x >= thr) a += ex2(t0);
                if (4 * x + 1 >= thr) b1 += ex2(t1);
                if (4 * x + 2 >= thr) b2 += ex2(t2);
                if (4 * x + 3 >= thr) b3 += ex2(t3);
            }
            a = (a + b1) + (b2 + b3);
        } else {
#pragma unroll
            for (int x = 0; x < 32; ++x) {
                const int r = r0 + x;
                if ((r % W) >= jmin) a += ex2(fmaf(v[x], scale2, nc[r]));
            }
        }
        a01 = add2(a01, pack2(a, 0.f));
    }
}

// Pass N, one block of 32 key columns for the query row this thread owns: folds them into the
// running (reference, sum of 2^(y*scale2 - reference)).  nvis = visible columns (slow path only).
__device__ __forceinline__ void norm_block(const float (&v)[32], bool fast, int nvis, float scale2, float& mref,
                                           float& lr) {
    if (fast) {
        float b0 = 0.f, b1 = 0.f, b2 = 0.f, b3 = 0.f;
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
            const float t0 = fmaf(v[x], scale2, -mref), t1 = fmaf(v[x + 1], scale2, -mref);
            const float t2 = fmaf(v[x + 2], scale2, -mref), t3 = fmaf(v[x + 3], scale2, -mref);
            b0 += ((kPolyMaskN >> x) & 1u) ? ex2_poly(fminf(fmaxf(t0, -125.f), 125.f)) : ex2(t0);
            b1 += ((kPolyMaskN >> (x + 1)) & 1u) ? ex2_poly(fminf(fmaxf(t1, -125.f), 125.f)) : ex2(t1);
            b2 += ((kPolyMaskN >> (x + 2)) & 1u) ? ex2_poly(fminf(fmaxf(t2, -125.f), 125.f)) : ex2(t2);
            b3 += ((kPolyMaskN >> (x + 3)) & 1u) ? ex2_poly(fminf(fmaxf(t3, -125.f), 125.f)) : ex2(t3);
        }
        float lb = (b0 + b1) + (b2 + b3);
        if (!(lb <= 65536.f)) {
            // A column exceeds the reference by more than 16 (or the reference is still unset): move the
            // reference to the block maximum and redo the block.
            float cm = v[0];
#pragma unroll
            for (int x = 1; x < 32; ++x) cm = fmaxf(cm, v[x]);
            cm *= scale2;
            if (cm > mref) {
                lr *= ex2(mref - cm);
                mref = cm;
            }
            b0 = 0.f; b1 = 0.f;
#pragma unroll
            for (int x = 0; x < 32; x += 2) {
                b0 += ex2(fmaf(v[x], scale2, -mref));
                b1 += ex2(fmaf(v[x + 1], scale2, -mref));
            }
            lb = b0 + b1;
        }
        lr += lb;
    } else {
        float cm = kNegBig;
#pragma unroll
        for (int x = 0; x < 32; ++x)
            if (x < nvis) cm = fmaxf(cm, v[x] * scale2);
        if (cm > mref) {
            lr *= ex2(mref - cm);
            mref = cm;
        }
#pragma unroll
        for (int x = 0; x < 32; ++x)
            if (x < nvis) lr += ex2(fmaf(v[x], scale2, -mref));
    }
}

// Walks this CTA's contiguous range of key tiles, segment by segment.  The next unit's descriptor fields are
// fetched a segment ahead, so a change of segment costs no memory round trip.
struct TileWalk {
    const UnitDesc* desc;
    int t, t_end, u, n_units;
    int tile0, n_tiles, T;
    int nx_tile0, nx_T;
    __device__ void init(const UnitDesc* d, int units, int total_tiles) {
        desc = d;
        n_units = units;
        t = (int)(((long long)total_tiles * blockIdx.x) / gridDim.x);
        t_end = (int)(((long long)total_tiles * (blockIdx.x + 1)) / gridDim.x);
        int lo = 0, hi = n_units - 1;
        while (lo < hi) {                       // last unit with tile0 <= t
            int mid = (lo + hi + 1) >> 1;
            if (d[mid].tile0 <= t) lo = mid; else hi = mid - 1;
        }
        u = lo;
        tile0 = desc[u].tile0;
        T = desc[u].T;
        n_tiles = (T + kTileKeys - 1) / kTileKeys;
        prefetch();
    }
    __device__ void prefetch() {
        const int v = min(u + 1, n_units - 1);
        nx_tile0 = desc[v].tile0;
        nx_T = desc[v].T;
    }
    __device__ bool valid() const { return t < t_end; }
    __device__ int key_begin() const { return (t - tile0) * kTileKeys; }
    __device__ int seg_tiles() const { return min(t_end, tile0 + n_tiles) - t; }
    __device__ bool has_next() const { return t + seg_tiles() < t_end; }
    __device__ void next_segment() {
        t += seg_tiles();
        if (t < t_end) {
            ++u;
            tile0 = nx_tile0;
            T = nx_T;
            n_tiles = (T + kTileKeys - 1) / kTileKeys;
            prefetch();
        }
    }
};

template <int PASS>   // 0: normaliser, 1: score mass
__global__ void __launch_bounds__(kThreadsTc, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                const UnitDesc* __restrict__ desc, Shape sh, int total_tiles, int sub_rows,
                float* __restrict__ part_m, float* __restrict__ part_l, const float* __restrict__ rowm,
                const float* __restrict__ roww, float* __restrict__ s, int32_t* __restrict__ err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_smem = smem;
    uint8_t* k_smem = smem + kQBytes;
    TcSmemTail* tail = reinterpret_cast<TcSmemTail*>(k_smem + kStages * kKStageBytes);
    Barriers& bar = tail->bar;
    volatile int* abort_flag = &tail->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = sh.rows;
    const int n_slots = (rows + 127) >> 7;           // 128-row query blocks in use
    const int n_issuers = min(2, n_slots);
    const int n_groups = n_issuers;                  // epilogue groups of eight warps

    if (threadIdx.x == 0) {
        for (int i = 0; i < kSlots; ++i) { mbar_init(&bar.q_full[i], 1); mbar_init(&bar.q_empty[i], 1); }
        for (int i = 0; i < kStages; ++i) { mbar_init(&bar.k_full[i], 1); mbar_init(&bar.k_empty[i], n_issuers); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(&bar.d_full[i], 1); mbar_init(&bar.d_empty[i], 8); }
        mbar_init(&bar.rw_ready, 256 * n_groups);
        for (int i = 0; i < 8; ++i) mbar_init(&bar.red_full[i], 8 * n_groups);
        mbar_init(&bar.mma_drain[0], 1);
        mbar_init(&bar.mma_drain[1], 1);
        tail->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
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
    // CTA 0 reports the SM clock it ran at (cycles over wall time), so that a pass can be held against the
    // exponential roof at the clock the power limit left it, not only at the nominal one.
    long long clk0 = 0;
    uint64_t ns0 = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) { clk0 = clock64(); ns0 = global_ns(); }

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t kit = 0, seg = 0;
            bool ok = true;
            for (; wk.valid() && ok; wk.next_segment(), ++seg) {
                const UnitDesc& ud = desc[wk.u];
                const int krow0 = sh.page_size ? 0 : (int)(ud.k_off / sh.row_stride);
                const int key_begin = wk.key_begin();
                const int nt = wk.seg_tiles();
                for (int t = 0; t < nt && ok; ++t, ++kit) {
                    const int st = kit % kStages;
                    ok = mbar_wait<true>(&bar.k_empty[st], ((kit / kStages) & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    uint8_t* dst = k_smem + st * kKStageBytes;
                    const int key0 = key_begin + t * kTileKeys;
                    if (sh.page_size == 0) {
                        mbar_expect_tx(&bar.k_full[st], kKStageBytes);
                        tma_load_2d(dst, &tmK, &bar.k_full[st], 0, krow0 + key0);
                        tma_load_2d(dst + kKRegionBytes, &tmK, &bar.k_full[st], 64, krow0 + key0);
                    } else {
                        // one box of sub_rows rows per page piece; pieces past the end of the unit are not read
                        // (their accumulator rows / columns are masked by the epilogue)
                        const int n_sub = min(kTileKeys / sub_rows, (wk.T - key0 + sub_rows - 1) / sub_rows);
                        mbar_expect_tx(&bar.k_full[st], (uint32_t)n_sub * sub_rows * 256u);
                        for (int sb = 0; sb < n_sub; ++sb) {
                            const int prow = (int)paged_row(sh, ud, key0 + sb * sub_rows);
                            tma_load_2d(dst + sb * sub_rows * 128, &tmK, &bar.k_full[st], 0, prow);
                            tma_load_2d(dst + kKRegionBytes + sb * sub_rows * 128, &tmK, &bar.k_full[st], 64, prow);
                        }
                    }
                    if (t == 0) {
                        // The segment's query blocks, each as soon as the previous segment's last contraction
                        // with that block has completed: block 0 is back in shared memory while the tensor pipe
                        // still works on the later blocks of the previous unit.  (The first key tile of the
                        // segment went out before, so it does not wait behind them.)
                        for (int j = 0; j < n_slots && ok; ++j) {
                            ok = mbar_wait<true>(&bar.q_empty[j], (seg & 1u) ^ 1u, abort_flag);
                            if (!ok) break;
                            mbar_expect_tx(&bar.q_full[j], 2 * kQBlockBytes);
                            uint8_t* qd_ = q_smem + (j >> 1) * 2 * kQRegionBytes + (j & 1) * kQBlockBytes;
                            for (int kb = 0; kb < 2; ++kb)
                                tma_load_3d(qd_ + kb * kQRegionBytes, &tmQ, &bar.q_full[j], kb * 64, j * 128, wk.u);
                        }
                    }
                }
            }
            if (!ok) {
                // copies already issued may still be landing: give each armed stage a bounded wait
                for (uint32_t j = (kit >= (uint32_t)kStages ? kit - kStages : 0); j < kit; ++j)
                    for (uint32_t it = 0; it < 4096 && !mbar_try(&bar.k_full[j % kStages], (j / kStages) & 1u); ++it) {}
                for (int j = 0; j < n_slots; ++j)
                    for (uint32_t it = 0; it < 4096 && !mbar_try(&bar.q_full[j], seg & 1u); ++it) {}
            }
        }
    } else if (warp <= n_issuers) {
        // ================= MMA issuers =================
        if (lane == 0) {
            const int j0 = warp - 1;               // this issuer's slots: j0, j0 + 2
            uint32_t kit = 0, seg = 0;
            bool ok = true;
            // Low descriptor words of the two operand bases; every tile of both operands is reached by
            // adding a compile-time constant (the address field counts 16-byte units and cannot carry).
            const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem)), k_lo = umma_desc_lo(smem_u32(k_smem));
            for (; wk.valid() && ok; wk.next_segment(), ++seg) {
                const int nt = wk.seg_tiles();
                for (int t = 0; t < nt && ok; ++t, ++kit) {
                    const int st = kit % kStages;
                    ok = mbar_wait<true>(&bar.k_full[st], (kit / kStages) & 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t kst_lo = k_lo + st * (kKStageBytes >> 4);
#pragma unroll
                    for (int jj = 0; jj < kSlots; jj += 2) {
                        const int j = jj + j0;
                        if (j >= n_slots || !ok) break;
                        ok = mbar_wait<true>(&bar.d_empty[j], (kit & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                        if (t == 0) {                       // the segment's query block j has landed
                            ok = mbar_wait<true>(&bar.q_full[j], seg & 1u, abort_flag);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        const uint32_t qblk_lo = q_lo + (((j >> 1) * 2 * kQRegionBytes + (j & 1) * (128 * 128)) >> 4);
                        const uint32_t idesc = umma_idesc(PASS == 1 ? min(128, rows - 128 * j) : 128);
                        if (PASS == 1) tc_mma_lo<false>(tmem_base + 128 * j, kst_lo, qblk_lo, idesc);
                        else tc_mma_lo<false>(tmem_base + 128 * j, qblk_lo, kst_lo, idesc);
#pragma unroll
                        for (int kk = 1; kk < 8; ++kk) {
                            const int kb = kk >> 2, ks = kk & 3;
                            const uint32_t dq = qblk_lo + ((kb * kQRegionBytes + ks * 32) >> 4);
                            const uint32_t dk = kst_lo + ((kb * kKRegionBytes + ks * 32) >> 4);
                            if (PASS == 1) tc_mma_lo<true>(tmem_base + 128 * j, dk, dq, idesc);
                            else tc_mma_lo<true>(tmem_base + 128 * j, dq, dk, idesc);
                        }
                        tc_commit(&bar.d_full[j]);
                        if (t == nt - 1) tc_commit(&bar.q_empty[j]);      // last use of query block j in this segment
                    }
                    tc_commit(&bar.k_empty[st]);
                }
            }
            if (!ok) {
                // contractions already issued may still be running: the TMEM they write is freed below, so give them
                // a bounded wait (a commit completes when everything this thread issued before it has)
                tc_commit(&bar.mma_drain[j0]);
                for (uint32_t it = 0; it < 4096 && !mbar_try(&bar.mma_drain[j0], 0u); ++it) {}
            }
        }
    } else if (warp >= kEpiWarp0 && ((warp - kEpiWarp0) >> 3) < n_groups) {
        // ================= epilogue =================
        const int ew = warp - kEpiWarp0;
        const int qd = ew & 3;                   // TMEM lane quadrant (== warp % 4)
        const int ch = (ew >> 2) & 1;            // which 64 columns of a slot
        const int g = ew >> 3;                   // group: drains slots g and g + 2 in turn
        const int etid = ew * 32 + lane;
        const float scale2 = kLog2e * rsqrtf((float)kD);
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * qd) << 16) + 64 * ch;
        uint32_t kit = 0, seg = 0;
        bool ok = true;
        // pass S: key offsets of the last two tiles, folded two tiles late by the warps ew < 4
        int64_t pend_off[2] = {-1, -1};
        // pass N: running reference / sum of the two query rows this thread works on
        float mm[2] = {kNegBig, kNegBig}, l_run[2] = {0.f, 0.f};

        if (PASS == 1 && wk.valid()) {
            // roww * 2^(y - rowm) = 2^(y + (log2 roww - rowm)): one constant per query row
            tail->rc[0][etid] = (etid < rows) ? log2f(roww[(size_t)wk.u * rows + etid]) - rowm[(size_t)wk.u * rows + etid]
                                              : -1.0e30f;
            mbar_arrive(&bar.rw_ready);
        }
        for (; wk.valid() && ok; wk.next_segment(), ++seg) {
            const int T = wk.T;
            const int64_t tok_off = desc[wk.u].tok_off;
            const int last_all = sh.causal ? T - sh.W : T - 1;     // last key every query sees
            const float* rc = tail->rc[seg % 3u];
            float nx_w = 0.f, nx_m = 0.f;      // next segment's row weight and offset: loaded now, used after the first tile
            bool has_next = false;
            if (PASS == 1) {
                // The table of this segment was written during the previous one (before the loop for the first).
                ok = mbar_wait<true>(&bar.rw_ready, seg & 1u, abort_flag);
                if (!ok) break;
                // Fetch the next segment's entry now; it goes into the third buffer after this segment's first
                // tile, when the loads have long landed.  Whoever passed the wait above knows that every thread
                // is past the first tile of the previous segment, so nobody still reads the buffer of the segment
                // before that one, which is the one written next.
                has_next = wk.has_next();
                if (has_next && etid < rows)
                    { nx_w = roww[(size_t)(wk.u + 1) * rows + etid]; nx_m = rowm[(size_t)(wk.u + 1) * rows + etid]; }
            } else {
                mm[0] = mm[1] = kNegBig;
                l_run[0] = l_run[1] = 0.f;
            }
            const int key_begin = wk.key_begin();
            const int nt = wk.seg_tiles();
            // The columns of its two slots this warp reads (64 of each, fewer in a ragged last slot).
            const int j0 = g, j1 = g + 2;
            const int cend0 = PASS == 1 ? min(64 * ch + 64, rows - 128 * j0) - 64 * ch : 64;
            const int cend1 = PASS == 1 ? min(64 * ch + 64, rows - 128 * j1) - 64 * ch : 64;
            const bool full_cols = j1 < n_slots && cend0 == 64 && cend1 == 64;
            const int row0 = 128 * j0 + 32 * qd + lane, row1 = 128 * j1 + 32 * qd + lane;      // pass N
            const int lastvis0 = (row0 < rows) ? (sh.causal ? T - sh.W + (row0 % sh.W) : T - 1) : -1;
            const int lastvis1 = (row1 < rows) ? (sh.causal ? T - sh.W + (row1 % sh.W) : T - 1) : -1;
            if (PASS == 0 && full_cols && nt > 0 && key_begin + kTileKeys - 1 <= last_all) {
                // The rows have no reference at the start of a segment, and a streamed tile without one is redone
                // whole.  Once per segment, before its first tile: wait for the tile's two slots (the waits inside
                // the loop then pass at once), read the first chunk of each and take its maximum as the reference.
                float w[16];
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    const int j = p ? j1 : j0;
                    ok = mbar_wait<true>(&bar.d_full[j], kit & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    tc_ld16(taddr + 128 * j, w);
                    tc_wait_ld_regs(w);
                    float cm = w[0];
#pragma unroll
                    for (int x = 1; x < 16; ++x) cm = fmaxf(cm, w[x]);
                    mm[p] = cm * scale2;
                }
                if (!ok) break;
            }
            for (int t = 0; t < nt && ok; ++t, ++kit) {
                const int key0 = key_begin + t * kTileKeys;
                const bool fast = key0 + kTileKeys - 1 <= last_all;
                const int my_key = key0 + 32 * qd + lane;           // pass S: the key this thread owns
                const int jmin = my_key - (T - sh.W);               // pass S: first window position that sees it
                const int kcol = key0 + 64 * ch;                    // pass N: first key column of this warp
                uint64_t a01 = 0ull, a23 = 0ull;      // pass S: two packed pairs of partial key sums
                if (fast && full_cols) {
                    // Streamed form of the common tile: eight chunks of 16 columns.  The arguments of a chunk's
                    // exponentials are formed first; that frees the accumulator registers, so the next chunk's
                    // TMEM load (or the slot's release) is issued before the exponentials and its latency hides
                    // behind them.
                    const uint64_t s2 = pack2(scale2, scale2);
                    float v[16];
                    float lbs[4] = {0.f, 0.f, 0.f, 0.f};      // pass N: the sums of a slot's four chunks
                    ok = mbar_wait<true>(&bar.d_full[j0], kit & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    tc_ld16(taddr + 128 * j0, v);
                    tc_wait_ld_regs(v);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int p = c >> 2, j = p ? j1 : j0, col = 16 * (c & 3);
                        uint64_t t2[8];
                        if (PASS == 1) {
                            const uint32_t nc32 = smem_u32(&rc[128 * j + 64 * ch + col]);
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                const float4 c4 = lds_f4(nc32 + 16u * x);
                                t2[2 * x] = fma2(pack2(v[4 * x], v[4 * x + 1]), s2, pack2(c4.x, c4.y));
                                t2[2 * x + 1] = fma2(pack2(v[4 * x + 2], v[4 * x + 3]), s2, pack2(c4.z, c4.w));
                            }
                        } else {
                            const uint64_t nm2 = pack2(-mm[p], -mm[p]);
#pragma unroll
                            for (int x = 0; x < 8; ++x) t2[x] = fma2(pack2(v[2 * x], v[2 * x + 1]), s2, nm2);
                        }
                        if (PASS == 1 && (c == 3 || c == 7)) {           // the slot's last columns are in registers
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&bar.d_empty[j]);
                        }
                        if (c == 3) {
                            ok = mbar_wait<true>(&bar.d_full[j1], kit & 1u, abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        if (c < 7) tc_ld16(taddr + 128 * (((c + 1) >> 2) ? j1 : j0) + 16 * ((c + 1) & 3), v);
                        if (PASS == 1) {
#pragma unroll
                            for (int x = 0; x < 8; ++x) {
                                float t0, t1;
                                unpack2(t2[x], t0, t1);
                                const uint64_t e2 = ((kPolyPairs16S >> x) & 1u)
                                                        ? ex2_poly2(pack2(fmaxf(t0, -125.f), fmaxf(t1, -125.f)))
                                                        : pack2(ex2(t0), ex2(t1));
                                if (x & 1) a23 = add2(a23, e2); else a01 = add2(a01, e2);
                            }
                        } else {
                            uint64_t b01 = 0ull, b23 = 0ull;
#pragma unroll
                            for (int x = 0; x < 8; ++x) {
                                float t0, t1;
                                unpack2(t2[x], t0, t1);
                                const uint64_t e2 = ((kPolyPairs16N >> x) & 1u)
                                                        ? ex2_poly2(pack2(fminf(fmaxf(t0, -125.f), 125.f), fminf(fmaxf(t1, -125.f), 125.f)))
                                                        : pack2(ex2(t0), ex2(t1));
                                if (x & 1) b23 = add2(b23, e2); else b01 = add2(b01, e2);
                            }
                            float b0, b1;
                            unpack2(add2(b01, b23), b0, b1);
                            lbs[c & 3] = b0 + b1;
                            if (c == 3 || c == 7) {
                                // The four chunk sums of the slot are checked together, once, before the slot is
                                // released: a check per chunk drains the warp's exponentials eight times a tile.
                                const bool redo = !(lbs[0] <= 65536.f) || !(lbs[1] <= 65536.f) || !(lbs[2] <= 65536.f) ||
                                                  !(lbs[3] <= 65536.f);
                                if (__any_sync(0xffffffffu, redo)) {
                                    // Some row of the warp has a column that exceeds its reference by more than 16
                                    // (or its reference is still unset).  The whole warp reads the slot's 64 columns
                                    // again (the loads are warp-wide; the slot is still held); the rows concerned
                                    // move their reference to the maximum of the 64 and redo the four sums.
                                    float w[16];
                                    float cm = kNegBig;
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        tc_ld16(taddr + 128 * j + 16 * k, w);
                                        tc_wait_ld_regs(w);
#pragma unroll
                                        for (int x = 0; x < 16; ++x) cm = fmaxf(cm, w[x]);
                                    }
                                    cm *= scale2;
                                    if (redo && cm > mm[p]) {
                                        l_run[p] *= ex2(mm[p] - cm);
                                        mm[p] = cm;
                                    }
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        tc_ld16(taddr + 128 * j + 16 * k, w);
                                        tc_wait_ld_regs(w);
                                        if (redo) {
                                            float lb = 0.f;
#pragma unroll
                                            for (int x = 0; x < 16; ++x) lb += ex2(fmaf(w[x], scale2, -mm[p]));
                                            lbs[k] = lb;
                                        }
                                    }
                                    __syncwarp();
                                }
#pragma unroll
                                for (int k = 0; k < 4; ++k) l_run[p] += lbs[k];
                                // the slot is no longer needed
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&bar.d_empty[j]);
                            }
                        }
                        if (c < 7) tc_wait_ld_regs(v);
                    }
                    if (!ok) break;
                } else {
#pragma unroll
                    for (int p = 0; p < 2; ++p) {
                        const int j = p ? j1 : j0;
                        if (j >= n_slots || !ok) break;
                        ok = mbar_wait<true>(&bar.d_full[j], kit & 1u, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const int cend = p ? cend1 : cend0;
                        for (int cc = 0; cc < cend; cc += 32) {
                            float v[32];
                            tc_ld32(taddr + 128 * j + cc, v);
                            tc_wait_ld_regs(v);
                            if (PASS == 1) mass_block(v, rc, 128 * j + 64 * ch + cc, fast, sh.causal, sh.W, jmin, scale2, a01, a23);
                            else norm_block(v, fast, (p ? lastvis1 : lastvis0) - (kcol + cc) + 1, scale2, mm[p], l_run[p]);
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bar.d_empty[j]);
                    }
                }
                if (PASS == 1 && t == 0 && has_next && ok) {       // before this tile's global stores
                    tail->rc[(seg + 1) % 3u][etid] = (etid < rows) ? log2f(nx_w) - nx_m : -1.0e30f;
                    mbar_arrive(&bar.rw_ready);
                }
                if (PASS == 1 && ok) {
                    float a0, a1, a2, a3;
                    unpack2(a01, a0, a1);
                    unpack2(a23, a2, a3);
                    tail->red[kit & 7u][ew >> 2][32 * qd + lane] = (a0 + a1) + (a2 + a3);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar.red_full[kit & 7u]);
                    if (ew < 4) {
                        // Fold the tile before the previous one: every warp finished it long ago.  The
                        // two-stage key ring keeps every warp within two tiles of every other, so with
                        // eight buffers the one read here cannot be the one being rewritten.
                        const int64_t off = pend_off[kit & 1u];
                        if (kit >= 2) {
                            const uint32_t pk = kit - 2;
                            ok = mbar_wait<true>(&bar.red_full[pk & 7u], (pk >> 3) & 1u, abort_flag);
                            if (!ok) break;
                            const float acc = fold_partials(&tail->red[pk & 7u][0][32 * qd + lane], 2 * n_groups);
                            if (off >= 0) s[off] = acc;
                        }
                        pend_off[kit & 1u] = (my_key < T) ? tok_off + my_key : -1;
                    }
                }
            }
            if (PASS == 0 && ok) {
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    const int my_row = 128 * (g + 2 * p) + 32 * qd + lane;
                    if (my_row < rows) {
                        const size_t o = ((size_t)(wk.u + blockIdx.x) * 2 + ch) * rows + my_row;
                        part_m[o] = mm[p];
                        part_l[o] = l_run[p];
                    }
                }
            }
        }
        if (PASS == 1 && ew < 4 && ok) {
            // the last two tiles of this CTA
            for (uint32_t pk = (kit >= 2 ? kit - 2 : 0); pk < kit; ++pk) {
                if (!mbar_wait<true>(&bar.red_full[pk & 7u], (pk >> 3) & 1u, abort_flag)) break;
                const float acc = fold_partials(&tail->red[pk & 7u][0][32 * qd + lane], 2 * n_groups);
                const int64_t off = pend_off[pk & 1u];
                if (off >= 0) s[off] = acc;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && tail->abort) atomicOr(err, CASK_ST_TIMEOUT);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const uint64_t ns = global_ns() - ns0;
        const long long clk = clock64() - clk0;
        err[2 + PASS] = ns > 0 ? (int32_t)((double)clk * 1.0e6 / (double)ns) : 0;      // kHz
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// CTA that owns tile x when `total` tiles are split over `grid` CTAs as in TileWalk::init.
template <typename I>
__device__ __forceinline__ int owner_cta_as(I x, I total, I grid) {
    I b = (x * grid) / total;
    while (b + 1 < grid && (total * (b + 1)) / grid <= x) ++b;
    while (b > 0 && (total * b) / grid > x) --b;
    return (int)b;
}
// 32-bit divisions when total * grid fits (a 64-bit division is a sequence of a hundred instructions)
__device__ __forceinline__ int owner_cta(long long x, long long total, long long grid) {
    if (total * grid < (1ll << 31)) return owner_cta_as<uint32_t>((uint32_t)x, (uint32_t)total, (uint32_t)grid);
    return owner_cta_as<long long>(x, total, grid);
}

constexpr int kCombineThreads = 128;      // four rows per thread cover the 512 rows the scoring kernels accept

// Folds the per-segment (reference, sum) pairs of every query row into the row offset and weight
// used by the score pass: rowm = max reference, roww = 1/(rows * sum 2^(y - rowm)).  With
// caller-supplied natural-log normalisers: rowm = lse*log2(e), roww = 1/rows.
__global__ void score_tc_combine(const UnitDesc* __restrict__ desc, int rows, int total_tiles, int grid,
                                 const float* __restrict__ part_m, const float* __restrict__ part_l,
                                 const float* __restrict__ lse_in, float* __restrict__ rowm,
                                 float* __restrict__ roww, float* __restrict__ lse_out) {
    // One block per unit, up to four query rows per thread (rows <= 512), every load of a round independent of the
    // others: the kernel is a chain of cache latencies and nothing else, so it wants as many rows in flight per
    // resident thread as it can have.  The range of CTAs that hold partials of the unit costs a few divisions: one
    // thread finds it for the block.  The additions keep the order of the partials.
    const int u = blockIdx.x;
    __shared__ int b_range[2];
    if (threadIdx.x == 0) {
        const UnitDesc& ud = desc[u];
        const int n_tiles = (ud.T + kTileKeys - 1) / kTileKeys;
        b_range[0] = owner_cta(ud.tile0, total_tiles, grid);
        b_range[1] = owner_cta((long long)ud.tile0 + n_tiles - 1, total_tiles, grid);
    }
    __syncthreads();
    const int lo = 2 * b_range[0], hi = 2 * b_range[1] + 1;
    const float inv_rows = 1.f / (float)rows;
    constexpr int kR = 4;
    const size_t ou = (size_t)u * rows;
    if (lse_in) {
#pragma unroll
        for (int x = 0; x < kR; ++x) {
            const int r = threadIdx.x + x * kCombineThreads;
            if (r >= rows) break;
            const float lse = lse_in[ou + r];
            rowm[ou + r] = lse * kLog2e;
            roww[ou + r] = inv_rows;
            if (lse_out) lse_out[ou + r] = lse;
        }
        return;
    }
    float m[kR], l[kR];
#pragma unroll
    for (int x = 0; x < kR; ++x) { m[x] = kNegBig; l[x] = 0.f; }
    for (int b = lo; b <= hi; b += 2) {
        float pm[kR][2];
#pragma unroll
        for (int x = 0; x < kR; ++x)
#pragma unroll
            for (int y = 0; y < 2; ++y) {
                const int r = threadIdx.x + x * kCombineThreads;
                pm[x][y] = (r < rows && b + y <= hi) ? part_m[((size_t)2 * u + b + y) * rows + r] : kNegBig;
            }
#pragma unroll
        for (int x = 0; x < kR; ++x) m[x] = fmaxf(fmaxf(m[x], pm[x][0]), pm[x][1]);
    }
    for (int b = lo; b <= hi; b += 2) {
        float pm[kR][2], pl[kR][2];
#pragma unroll
        for (int x = 0; x < kR; ++x)
#pragma unroll
            for (int y = 0; y < 2; ++y) {
                const int r = min(threadIdx.x + x * kCombineThreads, rows - 1);
                const size_t p = ((size_t)2 * u + min(b + y, hi)) * rows + r;
                pm[x][y] = part_m[p];
                pl[x][y] = part_l[p];
            }
#pragma unroll
        for (int x = 0; x < kR; ++x)
#pragma unroll
            for (int y = 0; y < 2; ++y)
                if (b + y <= hi) l[x] += pl[x][y] * exp2f(pm[x][y] - m[x]);
    }
#pragma unroll
    for (int x = 0; x < kR; ++x) {
        const int r = threadIdx.x + x * kCombineThreads;
        if (r >= rows) break;
        rowm[ou + r] = m[x];
        roww[ou + r] = inv_rows / l[x];
        if (lse_out) lse_out[ou + r] = (m[x] + log2f(l[x])) * kLn2;
    }
}

}  // namespace

// Entries of each normaliser-partial table the tensor-core path needs (one per unit + CTA).
size_t score_tc_partial_slots(int n_units) { return 2 * ((size_t)n_units + kMaxSms); }

// Rows per TMA box of the key stream: a whole 128-key tile for a contiguous cache, one page piece for
// a paged one (0: the page size does not tile 128 rows).
static int key_box_rows(const Shape& sh) {
    if (sh.page_size == 0) return kTileKeys;
    if (sh.page_size % kTileKeys == 0) return kTileKeys;
    if (sh.page_size >= 8 && kTileKeys % sh.page_size == 0) return sh.page_size;
    return 0;
}

bool score_tc_supported(const Launch& L) {
    const Shape& sh = L.sh;
    if (sh.dtype != CASK_DTYPE_BF16 || sh.d != kD) return false;
    if (sh.rows % 32 != 0 || sh.rows < 32 || sh.rows > 512) return false;
    if (sh.page_size) return key_box_rows(sh) != 0 && sh.n_pages * sh.page_size < ((int64_t)1 << 31);
    int64_t max_row = 0;
    for (int u = 0; u < sh.n_units; ++u) {
        const UnitDesc& d = L.hdesc[u];
        if (d.k_off % sh.row_stride != 0) return false;
        max_row = std::max<int64_t>(max_row, d.k_off / sh.row_stride + d.T);
    }
    return max_row < (int64_t)1 << 31;
}

cudaError_t launch_score_tc(const Launch& L, const float* lse_in, float* s, float* lse_out, Workspace& ws,
                            void* tmap_encode_fn) {
    const Shape& sh = L.sh;
    EncodeTiledFn encode = (EncodeTiledFn)tmap_encode_fn;
    int64_t k_rows = sh.page_size ? sh.n_pages * sh.page_size : 0;
    for (int u = 0; u < sh.n_units && !sh.page_size; ++u)
        k_rows = std::max<int64_t>(k_rows, L.hdesc[u].k_off / sh.row_stride + L.hdesc[u].T);
    const int sub_rows = key_box_rows(sh);
    CUtensorMap tmK, tmQ;
    {
        cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)k_rows};
        cuuint64_t strides[1] = {(cuuint64_t)sh.row_stride * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)sub_rows};
        cuuint32_t estr[2] = {1, 1};
        if (encode(&tmK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(L.k), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)sh.rows, (cuuint64_t)sh.n_units};
        cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)sh.rows * kD * 2};
        cuuint32_t box[3] = {64, 128, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        if (encode(&tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(L.q), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int grid = std::max(1, std::min(std::min(sms, kMaxSms), L.total_tiles));
    e = cudaFuncSetAttribute(score_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    if (!lse_in) {
        Timed t(L, KID_SCORE_NORM);
        score_tc_kernel<0><<<grid, kThreadsTc, kSmemBytes, L.stream>>>(tmK, tmQ, L.desc, sh, L.total_tiles, sub_rows, ws.part_m,
                                                                       ws.part_l, nullptr, nullptr, nullptr, ws.err);
    }
    {
        Timed t(L, KID_ROW_COMBINE);
        score_tc_combine<<<sh.n_units, kCombineThreads, 0, L.stream>>>(
            L.desc, sh.rows, L.total_tiles, grid, ws.part_m, ws.part_l, lse_in, ws.rowm, ws.roww, lse_out);
    }
    {
        Timed t(L, KID_SCORE_MASS);
        score_tc_kernel<1><<<grid, kThreadsTc, kSmemBytes, L.stream>>>(tmK, tmQ, L.desc, sh, L.total_tiles, sub_rows, nullptr,
                                                                       nullptr, ws.rowm, ws.roww, s, ws.err);
    }
    return cudaGetLastError();
}

}  // namespace cask
