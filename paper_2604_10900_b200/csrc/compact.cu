// Compaction to the budget (Sec. 2.3: |R| <= B) with the weighted K/V merge of Sec. 2.4:
//   slot order = ascending anchor row; kinds 1..3 and lone seeds are byte copies;
//   a seed with joiners holds sum_i w_i k_i, sum_i w_i v_i (members in ascending row order).
#include "tc_common.cuh"

namespace cask {

namespace {

// On the event path the scan also does what weights_kernel does in the staged consolidation call (merge weights
// w_i = a_i / m_G of the rows of kind 4/5, the unit's status word and lost mass): same formulas, same bits, one
// launch fewer.  s == nullptr: not fused, the weights are already there.
struct FusedWeights {
    const float* s;
    const int32_t* grp;
    const unsigned long long* mass_fx;
    const int32_t* njoin;
    const int32_t* plan;
    int32_t* unit_status;
    float* lost_mass;
    const int32_t* err;
    Shape sh;
    int max_m;
    float eps;
};

constexpr int kScanThreads = 1024;
constexpr int kScanMaxIters = 63;      // rows per unit below 64,512: the one-scan path of slot_scan_kernel

// ---- 1. per-unit ordered scan: slots, index map, member list -------------------------------
__global__ void __launch_bounds__(kScanThreads) slot_scan_kernel(
    const UnitDesc* __restrict__ desc, const uint8_t* __restrict__ kind, const int32_t* __restrict__ seed_of,
    float* __restrict__ weight, int Bmax, int32_t* __restrict__ n_out, int32_t* __restrict__ slot_src,
    uint8_t* __restrict__ slot_kind, float* __restrict__ slot_mass, int32_t* __restrict__ assign,
    int32_t* __restrict__ mem_row, int32_t* __restrict__ mem_slot, int32_t* __restrict__ n_mem,
    int32_t* __restrict__ seed_slot, int32_t* __restrict__ n_seed, int max_B, FusedWeights fw,
    int32_t* __restrict__ err) {
    __shared__ unsigned wk[kScanThreads / 32], wm[kScanThreads / 32];
    __shared__ unsigned cell[kScanMaxIters * (kScanThreads / 32)];
    __shared__ int seeds_listed;
    if (threadIdx.x == 0) seeds_listed = 0;
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int T = ud.T;
    const int64_t o = ud.tok_off;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    unsigned base_k = 0, base_m = 0;
    const int iters = (T + (int)blockDim.x - 1) / (int)blockDim.x;
    if (iters <= kScanMaxIters) {
        // Two coalesced sweeps around one scan: per (iteration, warp) cell the number of kept rows and of group
        // members, an exclusive scan over the cells in row order, then every row finds its slot from its cell's
        // base and the lower lanes of its warp.
        // (both sweeps read four rows' kinds a round, so that the loads are in flight together)
        const int cells = iters * nw;
        for (int it0 = 0; it0 < iters; it0 += 4) {
            uint8_t kd4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = (it0 + q) * blockDim.x + threadIdx.x;
                kd4[q] = (it0 + q < iters && i < T) ? kind[o + i] : (uint8_t)0;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (it0 + q >= iters) break;          // uniform over the block
                const uint8_t kd = kd4[q];
                const bool keep = kd >= CASK_KIND_PREFIX && kd <= CASK_KIND_SEED;
                const bool mem = kd == CASK_KIND_SEED || kd == CASK_KIND_MERGED;
                const unsigned bk = __ballot_sync(0xffffffffu, keep), bm = __ballot_sync(0xffffffffu, mem);
                if (lane == 0) cell[(it0 + q) * nw + w] = (unsigned)__popc(bk) | ((unsigned)__popc(bm) << 16);
            }
        }
        __syncthreads();
        // exclusive scan of the packed (kept, member) counts; a cell holds at most 32 of each and a unit fewer
        // than 65,536 kept rows and members in this path, so the halves never carry into each other
        {
            const int per = (cells + (int)blockDim.x - 1) / (int)blockDim.x;
            const int c0 = threadIdx.x * per, c1 = min(cells, c0 + per);
            unsigned sum = 0;
            for (int c = c0; c < c1; ++c) sum += cell[c];
            // block exclusive scan of `sum`
            unsigned incl = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                unsigned v = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += v;
            }
            if (lane == 31) wk[w] = incl;
            __syncthreads();
            unsigned wbase = 0;
            for (int x = 0; x < w; ++x) wbase += wk[x];
            unsigned run = wbase + incl - sum;
            unsigned total = 0;
            for (int x = 0; x < nw; ++x) total += wk[x];
            __syncthreads();
            for (int c = c0; c < c1; ++c) {
                const unsigned v = cell[c];
                cell[c] = run;
                run += v;
            }
            base_k = total & 0xFFFFu;
            base_m = total >> 16;
        }
        __syncthreads();
        for (int it0 = 0; it0 < iters; it0 += 4) {
            uint8_t kd4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = (it0 + q) * blockDim.x + threadIdx.x;
                kd4[q] = (it0 + q < iters && i < T) ? kind[o + i] : (uint8_t)0;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int it = it0 + q;
                if (it >= iters) break;                   // uniform over the block
                const int i = it * blockDim.x + threadIdx.x;
                const uint8_t kd = kd4[q];
                const bool keep = kd >= CASK_KIND_PREFIX && kd <= CASK_KIND_SEED;
                const bool mem = kd == CASK_KIND_SEED || kd == CASK_KIND_MERGED;
                const unsigned bk = __ballot_sync(0xffffffffu, keep), bm = __ballot_sync(0xffffffffu, mem);
                const unsigned cb = cell[it * nw + w];
                const unsigned below = (1u << lane) - 1u;
                if (i < T) {
                    int slot = -1;
                    if (keep) {
                        slot = (int)((cb & 0xFFFFu) + __popc(bk & below));
                        if (slot < Bmax) {
                            slot_src[(size_t)u * Bmax + slot] = i;
                            slot_kind[(size_t)u * Bmax + slot] = kd;
                        } else {
                            slot = -1;        // more kept rows than slots: cannot happen for a valid plan
                        }
                    }
                    assign[o + i] = slot;
                    if (mem) mem_row[o + (cb >> 16) + __popc(bm & below)] = i;
                    if (kd >= CASK_KIND_PREFIX && kd <= CASK_KIND_CORE) weight[o + i] = 1.f;
                    if (kd == CASK_KIND_DROPPED) weight[o + i] = 0.f;
                    if (fw.s && mem) {
                        const int gi = fw.grp[o + i];
                        if (gi >= 0 && gi < fw.max_m)
                            weight[o + i] = row_mass(fw.sh, fw.s, fw.eps, o + i) /
                                            fx_to_mass(fw.mass_fx[(size_t)u * (fw.max_m + 1) + gi]);
                    }
                }
            }
        }
    } else {
    for (int i0 = 0; i0 < T; i0 += blockDim.x) {
            const int i = i0 + threadIdx.x;
            const uint8_t kd = (i < T) ? kind[o + i] : (uint8_t)0;
            const bool keep = kd >= CASK_KIND_PREFIX && kd <= CASK_KIND_SEED;
            const bool mem = kd == CASK_KIND_SEED || kd == CASK_KIND_MERGED;
            const unsigned bk = __ballot_sync(0xffffffffu, keep), bm = __ballot_sync(0xffffffffu, mem);
            __syncthreads();
            if (lane == 0) { wk[w] = __popc(bk); wm[w] = __popc(bm); }
            __syncthreads();
            unsigned pk = 0, pm = 0, ak = 0, am = 0;
            for (int x = 0; x < nw; ++x) {
                if (x < w) { pk += wk[x]; pm += wm[x]; }
                ak += wk[x];
                am += wm[x];
            }
            const unsigned below = (1u << lane) - 1u;
            if (i < T) {
                int slot = -1;
                if (keep) {
                    slot = (int)(base_k + pk + __popc(bk & below));
                    if (slot < Bmax) {
                        slot_src[(size_t)u * Bmax + slot] = i;
                        slot_kind[(size_t)u * Bmax + slot] = kd;
                    } else {
                        slot = -1;        // more kept rows than slots: cannot happen for a valid plan
                    }
                }
                assign[o + i] = slot;
                if (mem) mem_row[o + base_m + pm + __popc(bm & below)] = i;
                if (kd >= CASK_KIND_PREFIX && kd <= CASK_KIND_CORE) weight[o + i] = 1.f;
                if (kd == CASK_KIND_DROPPED) weight[o + i] = 0.f;
                if (fw.s && mem) {
                    const int gi = fw.grp[o + i];
                    if (gi >= 0 && gi < fw.max_m)
                        weight[o + i] = row_mass(fw.sh, fw.s, fw.eps, o + i) /
                                        fx_to_mass(fw.mass_fx[(size_t)u * (fw.max_m + 1) + gi]);
                }
            }
            base_k += ak;
            base_m += am;
        }
    }
    const int nk = min((int)base_k, Bmax), nm = (int)base_m;
    if (threadIdx.x == 0) { n_out[u] = nk; n_mem[u] = nm; }
    if (fw.s && threadIdx.x == 0) {
        int fl = fw.plan[u * 8 + CASK_PLAN_FLAGS];
        if ((fl & CASK_ST_DECODE_CONSOLIDATED) && fw.njoin[u] == 0) fl |= CASK_ST_MERGE_INACTIVE;
        fw.unit_status[u] = fl | *fw.err;     // device-side flags of this call so far
        fw.lost_mass[u] = fx_to_mass(fw.mass_fx[(size_t)u * (fw.max_m + 1) + fw.max_m]);
    }
    for (int t = nk + threadIdx.x; t < Bmax; t += blockDim.x) {
        slot_src[(size_t)u * Bmax + t] = -1;
        slot_kind[(size_t)u * Bmax + t] = 0;
        slot_mass[(size_t)u * Bmax + t] = 0.f;
    }
    __syncthreads();
    // the slots that hold a representative, for the merge kernel (any order)
    for (int t = threadIdx.x; t < nk; t += blockDim.x)
        if (slot_kind[(size_t)u * Bmax + t] == CASK_KIND_SEED) {
            const int at = atomicAdd(&seeds_listed, 1);
            if (at < max_B) seed_slot[(size_t)u * max_B + at] = t;
        }
    __syncthreads();
    if (threadIdx.x == 0) n_seed[u] = min(seeds_listed, max_B);
    // members point at their seed's slot
    for (int e = threadIdx.x; e < nm; e += blockDim.x) {
        const int i = CASK_IDX(mem_row[o + e], T, err);
        int slot = -1;
        if (kind[o + i] == CASK_KIND_SEED) {
            slot = assign[o + i];
        } else {
            const int sd = seed_of[o + i];
            if (sd >= 0 && sd < T && kind[o + sd] == CASK_KIND_SEED) slot = assign[o + sd];
            assign[o + i] = slot;
        }
        mem_slot[o + e] = slot;
    }
}

// ---- 2. byte copy of every slot's anchor row by bulk async copies through shared memory ----
// A warp owns batches of up to 32 consecutive slots of one unit.  Every lane starts the bulk copy of its slot's K
// and V row (row bytes each, any source row) into the warp's staging buffer; when the batch has landed (mbarrier,
// byte count) one lane writes it out with two bulk stores, because consecutive slots are contiguous in k_out and
// v_out.  Two staging buffers per warp, so the loads of a batch run under the stores of the one before.  No
// registers hold data, which leaves enough copies in flight to load HBM with units of a few hundred rows.
constexpr int kCopyWarps = 6;
constexpr int kCopyStageBytes = 16384;       // per warp and stage: K half + V half

struct CopyCtl {
    uint64_t bar[kCopyWarps][2];
    int abort;
};

template <typename T>
__global__ void __launch_bounds__(kCopyWarps * 32) slot_copy_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const T* __restrict__ V,
    const float* __restrict__ s, float eps, int Bmax, int slots, const int32_t* __restrict__ n_out,
    const int32_t* __restrict__ slot_src, T* __restrict__ k_out, T* __restrict__ v_out,
    float* __restrict__ slot_mass) {
    using namespace tc;
    extern __shared__ __align__(128) uint8_t copy_smem[];
    __shared__ CopyCtl ctl;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t row_bytes = (uint32_t)(sh.d * sizeof(T));
    const int sb = min(32, (int)(kCopyStageBytes / 2 / row_bytes));     // slots per batch
    if (threadIdx.x == 0) {
        for (int i = 0; i < kCopyWarps; ++i) { mbar_init(&ctl.bar[i][0], 1); mbar_init(&ctl.bar[i][1], 1); }
        ctl.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int* abort_flag = &ctl.abort;
    uint8_t* my = copy_smem + (size_t)w * 2 * kCopyStageBytes;
    const int bpu = (slots + sb - 1) / sb;                               // batches per unit
    const int64_t total = (int64_t)sh.n_units * bpu;
    uint32_t it = 0;
    bool ok = true;
    for (int64_t bi = (int64_t)blockIdx.x * kCopyWarps + w; bi < total && ok; bi += (int64_t)gridDim.x * kCopyWarps) {
        const int u = (int)(bi / bpu), t0 = (int)(bi - (int64_t)u * bpu) * sb;
        const int nv = min(sb, n_out[u] - t0);
        if (nv <= 0) continue;
        const UnitDesc& ud = desc[u];
        const uint32_t st = it & 1u;
        uint8_t* kbuf = my + st * kCopyStageBytes;
        uint8_t* vbuf = kbuf + kCopyStageBytes / 2;
        // the stores that read this buffer two batches ago must have read it
        if (lane == 0) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            mbar_expect_tx(&ctl.bar[w][st], (uint32_t)nv * 2u * row_bytes);
        }
        __syncwarp();
        if (lane < nv) {
            const int src = CASK_IDX(slot_src[(size_t)u * Bmax + t0 + lane], ud.T, sh.err);
            const T* kr = K + row_elem_off(sh, ud, ud.k_off, src);
            const T* vr = V + v_elem_off(sh, ud, u, src);
            const uint32_t bar = smem_u32(&ctl.bar[w][st]);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(kbuf + lane * row_bytes)), "l"(kr), "r"(row_bytes), "r"(bar) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(vbuf + lane * row_bytes)), "l"(vr), "r"(row_bytes), "r"(bar) : "memory");
            slot_mass[(size_t)u * Bmax + t0 + lane] = row_mass(sh, s, eps, ud.tok_off + src);
        }
        ok = mbar_wait(&ctl.bar[w][st], (it >> 1) & 1u, abort_flag);
        if (!ok) break;
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const size_t dst = ((size_t)u * Bmax + t0) * sh.d;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(k_out + dst), "r"(smem_u32(kbuf)), "r"((uint32_t)nv * row_bytes) : "memory");
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(v_out + dst), "r"(smem_u32(vbuf)), "r"((uint32_t)nv * row_bytes) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        ++it;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (!ok && lane == 0) {
        // a copy that was started may still be landing: give the two barriers a bounded chance to complete
        for (uint32_t k = 0; k < 4096 && !mbar_try(&ctl.bar[w][it & 1u], (it >> 1) & 1u); ++k) {}
        atomicOr(sh.err, CASK_ST_TIMEOUT);
    }
}

// ---- 3. one warp per representative with joiners: ordered weighted merge over its copy -----
// CH > 0: head_dim == 32 * CH, every lane owns CH contiguous channels and reads them with one vector load per row;
// CH == 0: any head_dim up to 256, channels lane, lane + 32, ...  The sums per channel are the same either way.
template <typename T, int CH>
__global__ void __launch_bounds__(256) slot_merge_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const T* __restrict__ V,
    const float* __restrict__ s, const float* __restrict__ weight, float eps, int Bmax,
    const int32_t* __restrict__ seed_slot, const int32_t* __restrict__ n_seed, int max_B,
    const int32_t* __restrict__ mem_row, const int32_t* __restrict__ mem_slot,
    const int32_t* __restrict__ n_mem, T* __restrict__ k_out, T* __restrict__ v_out,
    float* __restrict__ slot_mass, int32_t* __restrict__ unit_status) {
    const int u = blockIdx.y;
    const UnitDesc& ud = desc[u];
    const int lane = threadIdx.x & 31;
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    // Last kernel of an event: flags raised on the device since the status words were written (a bulk copy of the
    // compaction that gave up) join them.  A page id outside the pool was already met by the scoring pass.
    if (unit_status && blockIdx.x == 0 && threadIdx.x == 0 && *sh.err) unit_status[u] |= *sh.err;
    if (j >= n_seed[u]) return;
    const int t = CASK_IDX(seed_slot[(size_t)u * max_B + j], Bmax, sh.err);
    const int d = sh.d;
    const int64_t o = ud.tok_off;
    constexpr int kMaxPerLane = 8;      // d <= 256
    float ak[kMaxPerLane], av[kMaxPerLane];
#pragma unroll
    for (int x = 0; x < kMaxPerLane; ++x) { ak[x] = 0.f; av[x] = 0.f; }
    int count = 0;
    float msum = 0.f;
    const int nm = n_mem[u];
    // A representative nobody joined keeps the byte copy of its row: count the list entries of this slot first (the
    // list is shared by the unit's warps and stays in cache) and leave before any row is requested.
    {
        int total = 0;
        for (int e0 = 0; e0 < nm; e0 += 32) {
            const int e = e0 + lane;
            total += __popc(__ballot_sync(0xffffffffu, e < nm && mem_slot[o + e] == t));
        }
        if (total <= 1) return;
    }
    // The member list of the unit is walked 128 entries at a time (the eight index loads of a round are independent)
    // and the round's own members are listed in shared memory in ascending order; their rows are then read four at a
    // time, so the latency of a row is paid once per four members and not once per member, and added in list order.
    constexpr int kWalk = 4;
    __shared__ int32_t hits[8][32 * kWalk];
    int32_t* my_hits = hits[threadIdx.x >> 5];
    const unsigned below = (1u << lane) - 1u;
    for (int e0 = 0; e0 < nm; e0 += 32 * kWalk) {
        int row[kWalk];
        bool hit[kWalk];
#pragma unroll
        for (int q = 0; q < kWalk; ++q) {
            const int e = e0 + 32 * q + lane;
            row[q] = (e < nm) ? mem_row[o + e] : -1;
            hit[q] = (e < nm) && mem_slot[o + e] == t;
        }
        int n_hits = 0;
#pragma unroll
        for (int q = 0; q < kWalk; ++q) {
            const unsigned bal = __ballot_sync(0xffffffffu, hit[q]);
            if (hit[q]) my_hits[n_hits + __popc(bal & below)] = row[q];
            n_hits += __popc(bal);
        }
        __syncwarp();
        constexpr int kRows = 4;           // member rows in flight per warp
        for (int h0 = 0; h0 < n_hits; h0 += kRows) {
            if (CH > 0) {
                struct alignas((CH > 0 ? CH : 1) * sizeof(T)) Vec { T x[CH > 0 ? CH : 1]; };
                Vec kv[kRows], vv[kRows];
                float wi[kRows], ai[kRows];
                // Offsets first, loads after, uses last, with no branch in between: a branch inside the loop over the
                // rows (paged or not, carried mass or not) makes every row wait for the one before it.
                int64_t io[kRows], ko[kRows], vo[kRows];
#pragma unroll
                for (int q = 0; q < kRows; ++q)
                    io[q] = o + CASK_IDX(my_hits[min(h0 + q, n_hits - 1)], ud.T, sh.err);
                if (sh.page_size == 0 && !sh.v_pos) {
#pragma unroll
                    for (int q = 0; q < kRows; ++q) {
                        ko[q] = ud.k_off + (io[q] - o) * sh.row_stride;
                        vo[q] = ud.v_off + (io[q] - o) * sh.row_stride;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < kRows; ++q) {
                        ko[q] = row_elem_off(sh, ud, ud.k_off, (int)(io[q] - o));
                        vo[q] = v_elem_off(sh, ud, u, (int)(io[q] - o));
                    }
                }
#pragma unroll
                for (int q = 0; q < kRows; ++q) {
                    wi[q] = weight[io[q]];
                    ai[q] = s[io[q]];
                    kv[q] = reinterpret_cast<const Vec*>(K + ko[q])[lane];
                    vv[q] = reinterpret_cast<const Vec*>(V + vo[q])[lane];
                }
                if (sh.mass_in) {
                    float mi[kRows];
#pragma unroll
                    for (int q = 0; q < kRows; ++q) mi[q] = sh.mass_in[io[q]];
#pragma unroll
                    for (int q = 0; q < kRows; ++q) ai[q] = (ai[q] + eps) + mi[q];      // row_mass()
                } else {
#pragma unroll
                    for (int q = 0; q < kRows; ++q) ai[q] += eps;
                }
#pragma unroll
                for (int q = 0; q < kRows; ++q) {
                    if (h0 + q >= n_hits) break;
                    msum += ai[q];
                    ++count;
#pragma unroll
                    for (int x = 0; x < CH; ++x) {
                        ak[x] = fmaf(wi[q], Elem<T>::ld(&kv[q].x[x]), ak[x]);
                        av[x] = fmaf(wi[q], Elem<T>::ld(&vv[q].x[x]), av[x]);
                    }
                }
            } else {
                for (int q = 0; q < kRows && h0 + q < n_hits; ++q) {
                    const int i = CASK_IDX(my_hits[h0 + q], ud.T, sh.err);
                    const float wq = weight[o + i];
                    msum += row_mass(sh, s, eps, o + i);
                    ++count;
                    const T* kr = K + row_elem_off(sh, ud, ud.k_off, i);
                    const T* vr = V + v_elem_off(sh, ud, u, i);
#pragma unroll
                    for (int x = 0; x < kMaxPerLane; ++x) {
                        const int c = lane + 32 * x;
                        if (c < d) {
                            ak[x] = fmaf(wq, Elem<T>::ld(kr + c), ak[x]);
                            av[x] = fmaf(wq, Elem<T>::ld(vr + c), av[x]);
                        }
                    }
                }
            }
        }
        __syncwarp();
    }
    if (count > 1) {       // a lone seed keeps its byte copy
        T* ko = k_out + ((size_t)u * Bmax + t) * d;
        T* vo = v_out + ((size_t)u * Bmax + t) * d;
#pragma unroll
        for (int x = 0; x < kMaxPerLane; ++x) {
            const int c = CH > 0 ? lane * CH + x : lane + 32 * x;
            if ((CH > 0 && x < CH) || (CH == 0 && c < d)) {
                Elem<T>::st(ko + c, ak[x]);
                Elem<T>::st(vo + c, av[x]);
            }
        }
        if (lane == 0) slot_mass[(size_t)u * Bmax + t] = msum;
    }
}

// ---- 3b. units of at most kMergeStageRows rows: one CTA per unit, members sorted by representative in shared memory ----
// Same arithmetic as slot_merge_kernel (members in ascending row order, one fp32 accumulator per channel).  The
// unit's member list is staged once and sorted by representative with a stable counting sort (every member counts
// the earlier members of its group in shared memory), so a warp finds the members of its representative side by side
// and reads their rows four at a time.
constexpr int kMergeStageRows = 1024;

template <typename T, int CH>       // CH = d / 32 contiguous channels per lane
__global__ void __launch_bounds__(256, 4) slot_merge_small_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const T* __restrict__ V,
    const float* __restrict__ s, const float* __restrict__ weight, float eps, int Bmax,
    const int32_t* __restrict__ seed_slot, const int32_t* __restrict__ n_seed, int max_B,
    const int32_t* __restrict__ mem_row, const int32_t* __restrict__ mem_slot,
    const int32_t* __restrict__ n_mem, T* __restrict__ k_out, T* __restrict__ v_out,
    float* __restrict__ slot_mass, int32_t* __restrict__ unit_status) {
    constexpr int R = kMergeStageRows;
    __shared__ int32_t m_row[R], list[R], s_slot[R], start[R + 1], fill[R];
    __shared__ int16_t m_j[R], inv[R];
    __shared__ float m_w[R], m_a[R];
    __shared__ int32_t wsum[8];
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, nw = blockDim.x >> 5;
    const int64_t o = ud.tok_off;
    const int nm = min(n_mem[u], R);
    const int ns = min(n_seed[u], R);
    if (unit_status && tid == 0 && *sh.err) unit_status[u] |= *sh.err;      // see slot_merge_kernel
    for (int t = tid; t < R; t += blockDim.x) { inv[t] = -1; fill[t] = 0; }
    __syncthreads();
    for (int j = tid; j < ns; j += blockDim.x) {
        const int t = seed_slot[(size_t)u * max_B + j];
        s_slot[j] = t;
        if (t >= 0 && t < R) inv[t] = (int16_t)j;
    }
    __syncthreads();
    for (int e = tid; e < nm; e += blockDim.x) {
        const int row = CASK_IDX(mem_row[o + e], ud.T, sh.err), t = mem_slot[o + e];
        const int j = (t >= 0 && t < R) ? inv[t] : -1;
        m_row[e] = row;
        m_j[e] = (int16_t)j;
        m_w[e] = weight[o + row];
        m_a[e] = row_mass(sh, s, eps, o + row);
        if (j >= 0) atomicAdd(&fill[j], 1);
    }
    __syncthreads();
    {   // start[j] = members of the representatives before j (exclusive scan of the counts)
        const int per = (ns + (int)blockDim.x - 1) / (int)blockDim.x;
        const int j0 = tid * per, j1 = min(ns, j0 + per);
        int sum = 0;
        for (int j = j0; j < j1; ++j) sum += fill[j];
        int incl = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += v;
        }
        if (lane == 31) wsum[w] = incl;
        __syncthreads();
        int run = incl - sum;
        for (int x = 0; x < w; ++x) run += wsum[x];
        for (int j = j0; j < j1; ++j) {
            start[j] = run;
            run += fill[j];
            fill[j] = 0;
        }
        if (tid == (int)blockDim.x - 1) start[ns] = run;      // the last thread ends on the total
    }
    __syncthreads();
    // stable placement: a member's position inside its group is the number of earlier members of the same group
    for (int e = tid; e < nm; e += blockDim.x) {
        const int j = m_j[e];
        if (j < 0) continue;
        int before = 0;
        for (int x = 0; x < e; ++x) before += m_j[x] == j;
        list[start[j] + before] = e;
    }
    __syncthreads();
    struct alignas(CH * sizeof(T)) Vec { T x[CH]; };
    for (int j = w; j < ns; j += nw) {
        const int first = start[j], count = start[j + 1] - first;
        if (count <= 1) continue;       // a lone seed keeps its byte copy
        const int t = s_slot[j];
        float ak[CH], av[CH];
#pragma unroll
        for (int x = 0; x < CH; ++x) { ak[x] = 0.f; av[x] = 0.f; }
        float msum = 0.f;
        for (int h0 = 0; h0 < count; h0 += 4) {
            Vec kr[4], vr[4];
            float wi[4], ai[4];
            int64_t ko4[4], vo4[4];       // offsets first, loads after (see slot_merge_kernel)
            int i4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int e = list[first + min(h0 + q, count - 1)];
                i4[q] = m_row[e];
                wi[q] = m_w[e];
                ai[q] = m_a[e];
            }
            if (sh.page_size == 0 && !sh.v_pos) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    ko4[q] = ud.k_off + (int64_t)i4[q] * sh.row_stride;
                    vo4[q] = ud.v_off + (int64_t)i4[q] * sh.row_stride;
                }
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    ko4[q] = row_elem_off(sh, ud, ud.k_off, i4[q]);
                    vo4[q] = v_elem_off(sh, ud, u, i4[q]);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                kr[q] = reinterpret_cast<const Vec*>(K + ko4[q])[lane];
                vr[q] = reinterpret_cast<const Vec*>(V + vo4[q])[lane];
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (h0 + q >= count) break;
                msum += ai[q];
#pragma unroll
                for (int x = 0; x < CH; ++x) {
                    ak[x] = fmaf(wi[q], Elem<T>::ld(&kr[q].x[x]), ak[x]);
                    av[x] = fmaf(wi[q], Elem<T>::ld(&vr[q].x[x]), av[x]);
                }
            }
        }
        Vec ko, vo;
#pragma unroll
        for (int x = 0; x < CH; ++x) {
            Elem<T>::st(&ko.x[x], ak[x]);
            Elem<T>::st(&vo.x[x], av[x]);
        }
        reinterpret_cast<Vec*>(k_out + ((size_t)u * Bmax + t) * sh.d)[lane] = ko;
        reinterpret_cast<Vec*>(v_out + ((size_t)u * Bmax + t) * sh.d)[lane] = vo;
        if (lane == 0) slot_mass[(size_t)u * Bmax + t] = msum;
    }
}

// ---- host-resident caches: which value rows the compaction will read, and where they sit once packed ----
__global__ void __launch_bounds__(kScanThreads) value_rank_kernel(const UnitDesc* __restrict__ desc,
                                                                  const uint8_t* __restrict__ kind,
                                                                  int32_t* __restrict__ v_pos,
                                                                  int32_t* __restrict__ n_need) {
    __shared__ unsigned wsum[kScanThreads / 32];
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int T = ud.T;
    const int64_t o = ud.tok_off;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int chunk = (T + (int)blockDim.x - 1) / (int)blockDim.x;
    const int b = threadIdx.x * chunk, e = min(T, b + chunk);
    unsigned cnt = 0;
    for (int i = b; i < e; ++i) cnt += (kind[o + i] != CASK_KIND_DROPPED);
    unsigned incl = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        unsigned v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) wsum[w] = incl;
    __syncthreads();
    unsigned base = 0, total = 0;
    for (int x = 0; x < nw; ++x) {
        if (x < w) base += wsum[x];
        total += wsum[x];
    }
    unsigned rank = base + incl - cnt;
    for (int i = b; i < e; ++i) {
        const bool need = kind[o + i] != CASK_KIND_DROPPED;
        v_pos[o + i] = need ? (int)rank : -1;
        rank += need;
    }
    if (threadIdx.x == 0) n_need[u] = (int)total;
}

// v_base[u] = value rows needed by the units before u: one CTA, every thread a contiguous run of units.
__global__ void __launch_bounds__(1024) value_base_kernel(int n_units, const int32_t* __restrict__ n_need,
                                                          int64_t* __restrict__ v_base) {
    __shared__ int64_t wsum[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int per = (n_units + (int)blockDim.x - 1) / (int)blockDim.x;
    const int u0 = min(n_units, (int)threadIdx.x * per), u1 = min(n_units, u0 + per);
    int64_t sum = 0;
    for (int u = u0; u < u1; ++u) sum += n_need[u];
    int64_t incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int64_t v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) wsum[w] = incl;
    __syncthreads();
    int64_t run = incl - sum;
    for (int x = 0; x < w; ++x) run += wsum[x];
    for (int u = u0; u < u1; ++u) {
        v_base[u] = run;
        run += n_need[u];
    }
}

// ---- 4. paged cache: the compacted rows go back into the unit's own pages, slot t at logical row t ----
template <typename T>
__global__ void __launch_bounds__(256) writeback_kernel(const UnitDesc* __restrict__ desc, Shape sh, int Bmax,
                                                        const int32_t* __restrict__ n_out, const T* __restrict__ k_out,
                                                        const T* __restrict__ v_out, T* __restrict__ k_pool,
                                                        T* __restrict__ v_pool) {
    const int u = blockIdx.y;
    const UnitDesc& ud = desc[u];
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= n_out[u] || t >= ud.T) return;
    const int d = sh.d, nvec = d * (int)sizeof(T) / 16;
    const int64_t dst = paged_row(sh, ud, t) * sh.row_stride;
    const T* ks = k_out + ((size_t)u * Bmax + t) * d;
    const T* vs = v_out + ((size_t)u * Bmax + t) * d;
    for (int x = lane; x < 2 * nvec; x += 32) {
        const bool isv = x >= nvec;
        const int c = isv ? x - nvec : x;
        reinterpret_cast<uint4*>((isv ? v_pool : k_pool) + dst)[c] = reinterpret_cast<const uint4*>(isv ? vs : ks)[c];
    }
}

template <typename T>
cudaError_t run(const Launch& L, const cask_params& prm, const float* s, const uint8_t* kind,
                const int32_t* seed_of, float* weight, const cask_outputs& out, Workspace& ws, const EventFusion* ev) {
    const Shape& sh = L.sh;
    FusedWeights fw{};
    if (ev) fw = FusedWeights{s, ws.grp, ws.mass_fx, ws.njoin, ev->plan, ev->unit_status, ev->lost_mass, ws.err, sh, L.max_m, prm.eps};
    int32_t* const status = ev ? ev->unit_status : nullptr;
    {
        Timed t(L, KID_SLOT_SCAN);
        slot_scan_kernel<<<sh.n_units, L.max_T <= 2048 ? 256 : kScanThreads, 0, L.stream>>>(L.desc, kind, seed_of, weight, out.Bmax,
                                                                    out.n_out, out.slot_src, out.slot_kind,
                                                                    out.slot_mass, out.assign, ws.mem_row,
                                                                    ws.mem_slot, ws.n_mem, ws.seed_slot, ws.n_seed,
                                                                    ws.max_B, fw, ws.err);
    }
    const int slots = min(out.Bmax, max(L.max_B, 1));
    {
        // the merge kernel overwrites slots the copy kernel wrote: same stream, in order
        Timed t(L, KID_GATHER_MERGE);
        const int sb = std::min(32, (int)(kCopyStageBytes / 2 / (sh.d * sizeof(T))));
        const int64_t batches = (int64_t)sh.n_units * ((slots + sb - 1) / sb);
        const int copy_smem_bytes = kCopyWarps * 2 * kCopyStageBytes;
        cudaError_t ce = cudaFuncSetAttribute(slot_copy_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              copy_smem_bytes);
        if (ce != cudaSuccess) return ce;
        const int copy_grid = (int)std::min<int64_t>((batches + kCopyWarps - 1) / kCopyWarps, L.sms > 0 ? L.sms : 128);   // one CTA per SM
        slot_copy_kernel<T><<<std::max(copy_grid, 1), kCopyWarps * 32, copy_smem_bytes, L.stream>>>(
            L.desc, sh, (const T*)L.k, (const T*)L.v, s, prm.eps, out.Bmax, slots, out.n_out, out.slot_src,
            (T*)out.k_out, (T*)out.v_out, out.slot_mass);
        if (L.max_T <= kMergeStageRows && (sh.d == 64 || sh.d == 128)) {
            auto kern = sh.d == 128 ? slot_merge_small_kernel<T, 4> : slot_merge_small_kernel<T, 2>;
            kern<<<sh.n_units, 256, 0, L.stream>>>(
                L.desc, sh, (const T*)L.k, (const T*)L.v, s, weight, prm.eps, out.Bmax, ws.seed_slot, ws.n_seed,
                ws.max_B, ws.mem_row, ws.mem_slot, ws.n_mem, (T*)out.k_out, (T*)out.v_out, out.slot_mass, status);
        } else {
            auto mk = sh.d == 128 ? slot_merge_kernel<T, 4> : sh.d == 64 ? slot_merge_kernel<T, 2> : slot_merge_kernel<T, 0>;
            // one warp per representative: on the event path no unit has more than max_m of them (the plan's count);
            // a staged call may be handed any kinds, so there the slot count bounds them
            const int reps = ev ? std::max(L.max_m, 1) : std::min(slots, ws.max_B);
            mk<<<dim3((reps + 7) / 8, sh.n_units), 256, 0, L.stream>>>(
                L.desc, sh, (const T*)L.k, (const T*)L.v, s, weight, prm.eps, out.Bmax, ws.seed_slot, ws.n_seed,
                ws.max_B, ws.mem_row, ws.mem_slot, ws.n_mem, (T*)out.k_out, (T*)out.v_out, out.slot_mass, status);
        }
        ++*L.launches;
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_value_ranks(const Launch& L, const uint8_t* kind, int32_t* v_pos, int32_t* n_need, int64_t* v_base) {
    Timed t(L, KID_SLOT_SCAN);
    value_rank_kernel<<<L.sh.n_units, kScanThreads, 0, L.stream>>>(L.desc, kind, v_pos, n_need);
    value_base_kernel<<<1, 1024, 0, L.stream>>>(L.sh.n_units, n_need, v_base);
    ++*L.launches;
    return cudaGetLastError();
}

cudaError_t launch_writeback(const Launch& L, const cask_outputs& out, void* k_pool, void* v_pool) {
    const Shape& sh = L.sh;
    const int slots = min(out.Bmax, max(L.max_B, 1));
    const dim3 grid((slots + 7) / 8, sh.n_units);
    Timed t(L, KID_GATHER_MERGE);
    if (sh.dtype == CASK_DTYPE_BF16)
        writeback_kernel<__nv_bfloat16><<<grid, 256, 0, L.stream>>>(L.desc, sh, out.Bmax, out.n_out,
                                                                   (const __nv_bfloat16*)out.k_out, (const __nv_bfloat16*)out.v_out,
                                                                   (__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool);
    else
        writeback_kernel<float><<<grid, 256, 0, L.stream>>>(L.desc, sh, out.Bmax, out.n_out, (const float*)out.k_out,
                                                            (const float*)out.v_out, (float*)k_pool, (float*)v_pool);
    return cudaGetLastError();
}

cudaError_t launch_compact(const Launch& L, const cask_params& prm, const float* s, const uint8_t* kind,
                           const int32_t* seed_of, float* weight, const cask_outputs& out, Workspace& ws,
                           const EventFusion* ev) {
    if (L.sh.dtype == CASK_DTYPE_BF16) return run<__nv_bfloat16>(L, prm, s, kind, seed_of, weight, out, ws, ev);
    return run<float>(L, prm, s, kind, seed_of, weight, out, ws, ev);
}

}  // namespace cask
