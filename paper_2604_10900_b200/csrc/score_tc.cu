// Windowed attention-mass scoring on the 5th-generation tensor cores (bf16 cache, head_dim 128).
//
// Both passes contract the unit's window queries Q_w [rows<=512, 128] with 128-key tiles of K:
//   pass N (normaliser): D[query, key]  -> per query row running max / sum of 2^(y - max)
//   pass S (score mass): D[key, query]  -> per key  sum_r roww_r * 2^(y_kr - rowm_r)
// so that the reduction always runs along the TMEM columns a single thread owns (no
// cross-thread reduction).  The two passes use the same shared-memory operand tiles
// (K-major, 128-byte swizzle, written by TMA); only the role of the operands (A <-> B) and
// the instruction shape differ.
//
// One persistent CTA per SM, 12 warps:
//   warp 0      TMA producer (one lane): Q once per unit, K tiles through a 2-stage ring
//   warp 1      TMEM allocation; one lane issues tcgen05.mma and the commits
//   warps 4-11  epilogue: tcgen05.ld of the fp32 accumulators + exp2 arithmetic
// The 512 TMEM columns hold one 128x512 accumulator split in two 256-column halves that
// ping-pong between the tensor pipe and the epilogue.  Every mbarrier wait is bounded; when
// one gives up the CTA raises an error flag, drains and frees its TMEM.
#include "tc_common.cuh"

namespace cask {

namespace {

using namespace tc;

constexpr int kTileKeys = 128;
constexpr int kD = 128;
constexpr int kStages = 2;
constexpr int kThreadsTc = 384;
constexpr int kEpiWarp0 = 4;
constexpr int kEpiThreads = 256;
constexpr uint32_t kQRegionBytes = 256 * 128;          // 256 rows x 64 bf16
constexpr uint32_t kQBytes = 4 * kQRegionBytes;        // 2 row halves x 2 K blocks
constexpr uint32_t kKRegionBytes = 128 * 128;          // 128 keys x 64 bf16
constexpr uint32_t kKStageBytes = 2 * kKRegionBytes;
constexpr int kTilesPerChunk = kChunkKeys / kTileKeys;

struct __align__(8) Barriers {
    uint64_t q_full, q_empty;
    uint64_t k_full[kStages], k_empty[kStages];
    uint64_t d_full[2], d_empty[2];
    uint64_t rw_ready;      // pass S: all epilogue threads have written the row table of the unit
};

struct TcSmemTail {
    Barriers bar;
    uint32_t tmem_base;
    int abort;
    float2 rw[2][512];     // pass S: {rowm, roww} per query row, double-buffered by unit
};

constexpr size_t kSmemBytes = 1024 + kQBytes + kStages * kKStageBytes + sizeof(TcSmemTail);

// Walks this CTA's contiguous range of key chunks, unit by unit.
struct ChunkWalk {
    const UnitDesc* desc;
    int c, c_end, u;
    int chunk0, n_chunks, T;
    __device__ void init(const UnitDesc* d, int n_units, int total_chunks) {
        desc = d;
        c = (int)(((long long)total_chunks * blockIdx.x) / gridDim.x);
        c_end = (int)(((long long)total_chunks * (blockIdx.x + 1)) / gridDim.x);
        int lo = 0, hi = n_units - 1;
        while (lo < hi) {                       // last unit with chunk0 <= c
            int mid = (lo + hi + 1) >> 1;
            if (d[mid].chunk0 <= c) lo = mid; else hi = mid - 1;
        }
        u = lo;
        load();
    }
    __device__ void load() { chunk0 = desc[u].chunk0; n_chunks = desc[u].n_chunks; T = desc[u].T; }
    __device__ bool valid() const { return c < c_end; }
    __device__ int key_begin() const { return (c - chunk0) * kChunkKeys; }
    __device__ int n_tiles() const {
        int rem = T - key_begin();
        return min(kTilesPerChunk, (rem + kTileKeys - 1) / kTileKeys);
    }
    // returns true when the next chunk belongs to another unit
    __device__ bool advance() {
        ++c;
        if (c >= chunk0 + n_chunks && c < c_end) { ++u; load(); return true; }
        return c >= c_end;
    }
};

template <int PASS>   // 0: normaliser, 1: score mass
__global__ void __launch_bounds__(kThreadsTc, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                const UnitDesc* __restrict__ desc, Shape sh, int total_chunks,
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
    const int n_blocks = (rows + 127) >> 7;          // 128-row query blocks (pass N)
    const int n_halves = (rows + 255) >> 8;          // 256-column accumulator halves in use

    if (threadIdx.x == 0) {
        mbar_init(&bar.q_full, 1);
        mbar_init(&bar.q_empty, 1);
        for (int i = 0; i < kStages; ++i) { mbar_init(&bar.k_full[i], 1); mbar_init(&bar.k_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&bar.d_full[i], 1); mbar_init(&bar.d_empty[i], 8); }
        mbar_init(&bar.rw_ready, kEpiThreads);
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

    ChunkWalk wk;
    wk.init(desc, sh.n_units, total_chunks);

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t kit = 0, qcount = 0;
            bool new_unit = true, ok = true;
            while (wk.valid() && ok) {
                const UnitDesc& ud = desc[wk.u];
                if (new_unit) {
                    ok = mbar_wait(&bar.q_empty, (qcount & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&bar.q_full, n_halves * 2 * kQRegionBytes);
                    for (int nh = 0; nh < n_halves; ++nh)
                        for (int kb = 0; kb < 2; ++kb)
                            tma_load_3d(q_smem + (nh * 2 + kb) * kQRegionBytes, &tmQ, &bar.q_full, kb * 64, nh * 256, wk.u);
                    ++qcount;
                }
                const int krow0 = (int)(ud.k_off / sh.row_stride) + wk.key_begin();
                const int nt = wk.n_tiles();
                for (int t = 0; t < nt && ok; ++t, ++kit) {
                    const int st = kit % kStages;
                    ok = mbar_wait(&bar.k_empty[st], ((kit / kStages) & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&bar.k_full[st], kKStageBytes);
                    uint8_t* dst = k_smem + st * kKStageBytes;
                    tma_load_2d(dst, &tmK, &bar.k_full[st], 0, krow0 + t * kTileKeys);
                    tma_load_2d(dst + kKRegionBytes, &tmK, &bar.k_full[st], 64, krow0 + t * kTileKeys);
                }
                new_unit = wk.advance();
            }
            if (!ok) {
                // copies already issued may still be landing: give each armed stage a bounded wait
                for (uint32_t j = (kit >= (uint32_t)kStages ? kit - kStages : 0); j < kit; ++j)
                    for (uint32_t it = 0; it < 4096 && !mbar_try(&bar.k_full[j % kStages], (j / kStages) & 1u); ++it) {}
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            uint32_t kit = 0, qcount = 0, dcount = 0;
            bool new_unit = true, ok = true;
            const uint32_t q_addr = smem_u32(q_smem), k_addr = smem_u32(k_smem);
            while (wk.valid() && ok) {
                if (new_unit) {
                    ok = mbar_wait(&bar.q_full, qcount & 1u, abort_flag);
                    if (!ok) break;
                    ++qcount;
                }
                const int nt = wk.n_tiles();
                for (int t = 0; t < nt && ok; ++t, ++kit, ++dcount) {
                    const int st = kit % kStages;
                    ok = mbar_wait(&bar.k_full[st], (kit / kStages) & 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t kst = k_addr + st * kKStageBytes;
                    for (int h = 0; h < n_halves && ok; ++h) {
                        ok = mbar_wait(&bar.d_empty[h], (dcount & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        if (PASS == 1) {
                            const int ncols = min(256, rows - 256 * h);
                            const uint32_t idesc = umma_idesc(ncols);
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                const int kb = kk >> 2, ks = kk & 3;
                                uint64_t a = umma_desc(kst + kb * kKRegionBytes + ks * 32);
                                uint64_t b = umma_desc(q_addr + (h * 2 + kb) * kQRegionBytes + ks * 32);
                                tc_mma(tmem_base + 256 * h, a, b, idesc, kk != 0);
                            }
                        } else {
                            const uint32_t idesc = umma_idesc(128);
                            for (int cs = 0; cs < 2; ++cs) {
                                const int mb = 2 * h + cs;
                                if (mb >= n_blocks) break;
#pragma unroll
                                for (int kk = 0; kk < 8; ++kk) {
                                    const int kb = kk >> 2, ks = kk & 3;
                                    uint64_t a = umma_desc(q_addr + (h * 2 + kb) * kQRegionBytes + cs * (128 * 128) + ks * 32);
                                    uint64_t b = umma_desc(kst + kb * kKRegionBytes + ks * 32);
                                    tc_mma(tmem_base + 128 * mb, a, b, idesc, kk != 0);
                                }
                            }
                        }
                        tc_commit(&bar.d_full[h]);
                    }
                    tc_commit(&bar.k_empty[st]);
                }
                new_unit = wk.advance();
                if (new_unit) tc_commit(&bar.q_empty);
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ================= epilogue =================
        const int ew = warp - kEpiWarp0;
        const int qd = warp & 3;                 // TMEM lane quadrant this warp may read
        const int cs = ew >> 2;                  // which 128-column slice of each half
        const int etid = threadIdx.x - kEpiWarp0 * 32;
        const float scale2 = kLog2e * rsqrtf((float)kD);
        const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * qd) << 16);
        uint32_t dcount = 0, ucount = 0;
        bool new_unit = true, ok = true;
        const float2* rw = tail->rw[0];
        while (wk.valid() && ok) {
            const UnitDesc& ud = desc[wk.u];
            const int T = ud.T;
            const int last_all = sh.causal ? T - sh.W : T - 1;     // last key every query sees
            if (PASS == 1 && new_unit) {
                // A thread can be at most one unit ahead of the slowest one (it has passed the previous
                // rw_ready phase), so writing the other buffer never races with a reader.
                float2* dst = tail->rw[ucount & 1u];
                for (int r = etid; r < 512; r += kEpiThreads)
                    dst[r] = (r < rows) ? make_float2(rowm[(size_t)wk.u * rows + r], roww[(size_t)wk.u * rows + r])
                                        : make_float2(0.f, 0.f);
                mbar_arrive(&bar.rw_ready);
                ok = mbar_wait(&bar.rw_ready, ucount & 1u, abort_flag);
                if (!ok) break;
                rw = dst;
                ++ucount;
            }
            // pass N state: the two query rows this thread owns (one per half)
            float m_run[2] = {kNegBig, kNegBig}, l_run[2] = {0.f, 0.f};
            int lastvis[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = 128 * (2 * h + cs) + 32 * qd + lane;
                lastvis[h] = (r < rows) ? (sh.causal ? T - sh.W + (r % sh.W) : T - 1) : -1;
            }
            const int key_begin = wk.key_begin();
            const int nt = wk.n_tiles();
            for (int t = 0; t < nt && ok; ++t, ++dcount) {
                const int key0 = key_begin + t * kTileKeys;
                const bool fast = key0 + kTileKeys - 1 <= last_all;
                float acc = 0.f;
                const int my_key = key0 + 32 * qd + lane;           // pass S: the key this thread owns
                const int jmin = my_key - (T - sh.W);                // pass S: first window position that sees it
                for (int h = 0; h < n_halves && ok; ++h) {
                    ok = mbar_wait(&bar.d_full[h], dcount & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    if (PASS == 1) {
                        const int ncols = min(256, rows - 256 * h);
                        for (int cc = 128 * cs; cc < min(128 * cs + 128, ncols); cc += 32) {
                            float v[32];
                            tc_ld32(lane_addr + 256 * h + cc, v);
                            tc_wait_ld();
                            const float4* rw4 = reinterpret_cast<const float4*>(&rw[256 * h + cc]);
                            if (fast) {
#pragma unroll
                                for (int x = 0; x < 16; ++x) {
                                    const float4 p = rw4[x];
                                    acc = fmaf(ex2(fmaf(v[2 * x], scale2, -p.x)), p.y, acc);
                                    acc = fmaf(ex2(fmaf(v[2 * x + 1], scale2, -p.z)), p.w, acc);
                                }
                            } else {
#pragma unroll
                                for (int x = 0; x < 32; ++x) {
                                    const int r = 256 * h + cc + x;
                                    const float2 p = rw[r];
                                    const bool vis = r < rows && (!sh.causal || (r % sh.W) >= jmin);
                                    if (vis) acc = fmaf(ex2(fmaf(v[x], scale2, -p.x)), p.y, acc);
                                }
                            }
                        }
                    } else {
                        const int mb = 2 * h + cs;
                        if (mb < n_blocks) {
                            for (int cc = 0; cc < 128; cc += 32) {
                                float v[32];
                                tc_ld32(lane_addr + 128 * mb + cc, v);
                                tc_wait_ld();
                                if (fast) {
                                    float cm = v[0];
#pragma unroll
                                    for (int x = 1; x < 32; ++x) cm = fmaxf(cm, v[x]);
                                    cm *= scale2;
                                    if (cm > m_run[h]) {
                                        l_run[h] *= ex2(m_run[h] - cm);
                                        m_run[h] = cm;
                                    }
                                    const float mm = m_run[h];
                                    float l0 = 0.f, l1 = 0.f;
#pragma unroll
                                    for (int x = 0; x < 32; x += 2) {
                                        l0 += ex2(fmaf(v[x], scale2, -mm));
                                        l1 += ex2(fmaf(v[x + 1], scale2, -mm));
                                    }
                                    l_run[h] += l0 + l1;
                                } else {
                                    const int nvis = lastvis[h] - (key0 + cc) + 1;      // visible columns of this chunk
                                    float cm = kNegBig;
#pragma unroll
                                    for (int x = 0; x < 32; ++x)
                                        if (x < nvis) cm = fmaxf(cm, v[x] * scale2);
                                    if (cm > m_run[h]) {
                                        l_run[h] *= ex2(m_run[h] - cm);
                                        m_run[h] = cm;
                                    }
                                    const float mm = m_run[h];
#pragma unroll
                                    for (int x = 0; x < 32; ++x)
                                        if (x < nvis) l_run[h] += ex2(fmaf(v[x], scale2, -mm));
                                }
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar.d_empty[h]);
                }
                // the two column slices of a key meet in the zero-initialised score array; with two
                // addends the sum does not depend on the order of arrival
                if (PASS == 1 && ok && my_key < T) atomicAdd(&s[ud.tok_off + my_key], acc);
            }
            if (PASS == 0 && ok) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int r = 128 * (2 * h + cs) + 32 * qd + lane;
                    if (r < rows) {
                        part_m[(size_t)wk.c * rows + r] = m_run[h];
                        part_l[(size_t)wk.c * rows + r] = l_run[h];
                    }
                }
            }
            new_unit = wk.advance();
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

bool score_tc_supported(const Launch& L) {
    const Shape& sh = L.sh;
    if (sh.dtype != CASK_DTYPE_BF16 || sh.d != kD) return false;
    if (sh.rows % 32 != 0 || sh.rows < 32 || sh.rows > 512) return false;
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
    int64_t k_rows = 0;
    for (int u = 0; u < sh.n_units; ++u)
        k_rows = std::max<int64_t>(k_rows, L.hdesc[u].k_off / sh.row_stride + L.hdesc[u].T);
    CUtensorMap tmK, tmQ;
    {
        cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)k_rows};
        cuuint64_t strides[1] = {(cuuint64_t)sh.row_stride * 2};
        cuuint32_t box[2] = {64, kTileKeys};
        cuuint32_t estr[2] = {1, 1};
        if (encode(&tmK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(L.k), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)sh.rows, (cuuint64_t)sh.n_units};
        cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)sh.rows * kD * 2};
        cuuint32_t box[3] = {64, 256, 1};
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
    const int grid = std::max(1, std::min(sms, L.total_chunks));
    e = cudaFuncSetAttribute(score_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    if (!lse_in) {
        Timed t(L, KID_SCORE_NORM);
        score_tc_kernel<0><<<grid, kThreadsTc, kSmemBytes, L.stream>>>(tmK, tmQ, L.desc, sh, L.total_chunks, ws.part_m,
                                                                       ws.part_l, nullptr, nullptr, nullptr, ws.err);
    }
    e = launch_row_combine(L, lse_in, lse_out, ws);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(s, 0, sizeof(float) * (size_t)L.sum_T, L.stream);
    if (e != cudaSuccess) return e;
    {
        Timed t(L, KID_SCORE_MASS);
        score_tc_kernel<1><<<grid, kThreadsTc, kSmemBytes, L.stream>>>(tmK, tmQ, L.desc, sh, L.total_chunks, nullptr,
                                                                       nullptr, ws.rowm, ws.roww, s, ws.err);
    }
    return cudaGetLastError();
}

}  // namespace cask
