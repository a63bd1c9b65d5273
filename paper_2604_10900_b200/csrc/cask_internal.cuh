// Internal declarations shared by the kernels and the C-ABI layer of libcask.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cask.h"

namespace cask {

// Per-unit descriptor, built on the host for every call and uploaded to the
// head of the workspace.  Offsets are in elements of the cache dtype.
struct UnitDesc {
    int64_t k_off;
    int64_t v_off;
    int64_t q_off;
    int64_t tok_off;
    int32_t T, P, B, reserve;
    int32_t plan[8];
    int32_t chunk0;     // first score-partial chunk of this unit
    int32_t n_chunks;   // key chunks of this unit in the normaliser pass
    int32_t seed_base;  // first entry of this unit in the seed tables
    int32_t atile0;     // first 128-row scratch tile of this unit in the assignment pass
    int32_t n_atiles;   // scratch tiles of this unit: ceil((T - r - P)/128) when m > 0, else 0
    int32_t tile0;      // first 128-key tile of this unit in the unit-major tile sequence of the scoring passes
    int32_t bt0;        // paged cache: first entry of this unit in the block table
    int32_t pad;
};

struct Shape {
    int n_units, d, g, W, rows;   // rows = g*W
    int dtype;
    int64_t row_stride;
    int causal;
    // paged cache (page_size > 0): row i of a unit lives in physical page bt[bt0 + i / page_size]
    int page_size;
    int64_t n_pages;
    const int32_t* bt;   // device
    int32_t* err;        // device flag word (CASK_ST_TIMEOUT, CASK_ST_BOUNDS)
    const float* mass_in;   // device, optional [sumT]: group mass a row already carries
    const float* chan_w;    // device, optional [d]: channel weights of the merge similarity
    const float* band_w;    // device, optional [d/2]: band weights of the un-squared per-band distance (Sec. 2.5)
    int band_layout;        // 0: band f = channels (f, f + d/2); 1: channels (2f, 2f + 1)
    // host-resident caches: only the value rows the compaction reads are on the device, packed unit after unit
    // in ascending row order; v_pos[tok_off + i] is the position of row i inside its unit's run, v_base[u] the
    // first packed row of unit u (both NULL when V is the full cache)
    const int32_t* v_pos;
    const int64_t* v_base;
};

// Kernel ids for the optional per-kernel event timing.
enum KernelId {
    KID_SCORE_NORM = 0, KID_ROW_COMBINE, KID_SCORE_MASS, KID_PREFIX_EVICT, KID_SELECT_CORE, KID_SEEDS,
    KID_SEED_GATHER, KID_ASSIGN, KID_WEIGHTS, KID_SLOT_SCAN, KID_GATHER_MERGE, KID_DIAGNOSTICS, KID_COUNT
};

// Records a CUDA event pair around every launch while switched on (defined in api.cu).
struct Profiler {
    bool on = false;
    void begin(int id, cudaStream_t st);
    void end(cudaStream_t st);
    void* impl = nullptr;
};

// Everything a launch needs, resolved by the API layer.
struct Launch {
    cudaStream_t stream;
    Shape sh;
    const UnitDesc* desc;     // device
    const UnitDesc* hdesc;    // host copy (for grid sizing)
    const void* k;
    const void* v;
    const void* q;
    int max_T, max_m, max_chunks, total_chunks, total_atiles, max_P, max_B, total_tiles;
    int64_t sum_T;
    int64_t* launches;        // counter to bump
    Profiler* prof;
    void* tmap_encode;        // cuTensorMapEncodeTiled or nullptr
    int force_simt;
    int sms;                  // multiprocessors of the context's device (0: not known)
};

// Scope guard around one kernel launch: counts it and, in profiling mode, times it.
struct Timed {
    const Launch& L;
    Timed(const Launch& l, int id) : L(l) {
        ++*L.launches;
        if (L.prof && L.prof->on) L.prof->begin(id, L.stream);
    }
    ~Timed() {
        if (L.prof && L.prof->on) L.prof->end(L.stream);
    }
};

constexpr int kChunkKeys = 2048;    // keys per normaliser-pass chunk
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kNegBig = -1.0e30f;   // finite stand-in for -inf in running maxima

// ---- workspace carving ------------------------------------------------------
struct Workspace {
    UnitDesc* desc;
    float* s;            // [sumT]   scores when the caller keeps none
    float* rowm;         // [units*rows] row offset in log2 units
    float* roww;         // [units*rows] row weight 1/(rows * sum)
    float* part_m;       // [total_chunks*rows]
    float* part_l;       // [total_chunks*rows]
    int32_t* seed_rows;  // [sum m]     seed cache rows, ascending per unit
    float* seed_norm;    // [sum m]
    void* seed_k;        // [sum m_pad, d] gathered seed keys (cache dtype)
    int32_t* grp;        // [sumT] seed slot (0..m) of a joined row, -1
    unsigned long long* mass_fx;  // [units*(max_m+1)] fixed-point group masses (+ lost mass)
    int32_t* njoin;      // [units]
    int32_t* mem_row;    // [sumT] rows of kind 4/5 in ascending order
    int32_t* mem_slot;   // [sumT] slot each of them feeds
    int32_t* n_mem;      // [units]
    int32_t* seed_slot;  // [units*max_B] slots of kind SEED, any order
    int32_t* n_seed;     // [units]
    int32_t max_B;
    int32_t* err;        // [1]
    float* stats_a;      // [units, d] query-statistics scorer: head-pooled mu * kappa per band (re, im)
    size_t bytes;
};

// ---- kernels (defined in the .cu files) --------------------------------------
cudaError_t launch_score_simt(const Launch& L, const float* lse_in, float* s, float* lse_out,
                              Workspace& ws);
cudaError_t launch_row_combine(const Launch& L, const float* lse_in, float* lse_out, Workspace& ws);
cudaError_t launch_prefix_evict(const Launch& L, const float* s, uint8_t* kind, int32_t* plan);
cudaError_t launch_select_core(const Launch& L, const float* s, const int32_t* plan, uint8_t* kind);
cudaError_t launch_consolidate(const Launch& L, const cask_params& prm, const float* s,
                               const int32_t* plan, uint8_t* kind, int32_t* seed_of, float* weight,
                               float* sim, int32_t* unit_status, float* lost_mass, Workspace& ws,
                               bool fused = false);
// fused (the event path only): `plan` and `kind` are still unwritten; one kernel per unit then does the prefix eviction
// and the core and seed selection, and for units of at most kSmallUnitRows rows the seed gather as well.
constexpr int kSmallUnitRows = 1024;
// ev != nullptr (the event path, after launch_consolidate(..., fused = true)): the ordered scan of the compaction also
// writes the merge weights, the status words and the lost mass, which the fused consolidation left out, and the merge
// kernel, the last of the event, ORs late device flags into the status words.
struct EventFusion {
    const int32_t* plan;
    int32_t* unit_status;
    float* lost_mass;
};
cudaError_t launch_compact(const Launch& L, const cask_params& prm, const float* s, const uint8_t* kind,
                           const int32_t* seed_of, float* weight, const cask_outputs& out, Workspace& ws,
                           const EventFusion* ev = nullptr);
// Host-resident caches: rank of every row among the rows of its unit whose values the compaction reads
// (kind != 0), the number of such rows per unit and the exclusive prefix of those numbers.
cudaError_t launch_value_ranks(const Launch& L, const uint8_t* kind, int32_t* v_pos, int32_t* n_need, int64_t* v_base);
// Paged cache: copies the compacted rows into the unit's own pages (slot t -> logical row t).
cudaError_t launch_writeback(const Launch& L, const cask_outputs& out, void* k_pool, void* v_pool);
// rho_core / rho_rep and the within-group dispersion of Sec. 2.6 per unit (any of the pointers may be NULL).
cudaError_t launch_diagnostics(const Launch& L, const cask_params& prm, const float* s, const uint8_t* kind,
                               const cask_outputs& out);

// Tensor-core assignment of scratch rows to seeds (cosine Gram + argmax), same outputs as the SIMT kernel.
bool assign_tc_supported(const Launch& L);
int assign_tc_box_rows(const Shape& sh);   // rows per TMA box of the key stream, 0 if the page size does not fit
cudaError_t launch_assign_tc(const Launch& L, const cask_params& prm, const float* s, const int32_t* plan,
                             uint8_t* kind, int32_t* seed_of, float* sim, Workspace& ws, void* tmap_encode_fn);

// Query-statistics scorer (App. B): horizon kernel and horizon-averaged mean score, one pass over the keys.
cudaError_t launch_score_stats(const Launch& L, const cask_query_stats& qs, float* s, Workspace& ws);

// Tensor-core scoring (tcgen05 + TMA); returns cudaErrorNotSupported when the shape does not fit.
bool score_tc_supported(const Launch& L);
size_t score_tc_partial_slots(int n_units);   // entries per normaliser-partial table
cudaError_t launch_score_tc(const Launch& L, const float* lse_in, float* s, float* lse_out,
                            Workspace& ws, void* tmap_encode_fn);

// ---- small device helpers ------------------------------------------------------
// Physical row (in units of rows of the K/V arrays) of logical row i of a unit in a paged cache.  A
// page id outside the pool raises CASK_ST_BOUNDS and is replaced by page 0, so nothing is read out
// of bounds.
__device__ __forceinline__ int64_t paged_row(const Shape& sh, const UnitDesc& ud, int i) {
    int32_t pg = sh.bt[ud.bt0 + i / sh.page_size];
    if ((uint64_t)(int64_t)pg >= (uint64_t)sh.n_pages) {
        atomicOr(sh.err, CASK_ST_BOUNDS);
        pg = 0;
    }
    return (int64_t)pg * sh.page_size + i % sh.page_size;
}
// Merge weight a_i of the row at per-row index idx (Sec. 2.4): score + eps, plus the mass it already carries.
__device__ __forceinline__ float row_mass(const Shape& sh, const float* __restrict__ s, float eps, int64_t idx) {
    const float a = s[idx] + eps;
    return sh.mass_in ? a + sh.mass_in[idx] : a;
}
// Element offset of logical row i of a unit in the K (unit_off = k_off) or V (v_off) array.
__device__ __forceinline__ int64_t row_elem_off(const Shape& sh, const UnitDesc& ud, int64_t unit_off, int i) {
    if (sh.page_size == 0) return unit_off + (int64_t)i * sh.row_stride;
    return paged_row(sh, ud, i) * sh.row_stride;
}
// Element offset of the value row i of unit u.
__device__ __forceinline__ int64_t v_elem_off(const Shape& sh, const UnitDesc& ud, int u, int i) {
    if (sh.v_pos) return (sh.v_base[u] + sh.v_pos[ud.tok_off + i]) * (int64_t)sh.d;
    return row_elem_off(sh, ud, ud.v_off, i);
}

// Self-checking build (-DCASK_BOUNDS, libcask_bounds.so): every index the kernels take from an array that they or an
// earlier kernel wrote (seed rows, member rows, slots, seed numbers) is checked against its range before it addresses
// memory.  A bad one raises CASK_ST_BOUNDS in the call's flag word and is replaced by 0, so nothing is read or written
// out of bounds and nothing traps.  The ordinary build compiles the checks out.
#ifdef CASK_BOUNDS
__device__ __forceinline__ int checked_index(int i, int n, int32_t* err) {
    if ((unsigned)i >= (unsigned)n) {
        atomicOr(err, CASK_ST_BOUNDS);
        return 0;
    }
    return i;
}
#define CASK_IDX(i, n, err) ::cask::checked_index((i), (n), (err))
#else
#define CASK_IDX(i, n, err) (i)
#endif

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ float ld(const float* p) { return *p; }
    static __device__ __forceinline__ void st(float* p, float x) { *p = x; }
};
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void st(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

// order-preserving map float -> uint32 (greater float <=> greater key)
__device__ __forceinline__ uint32_t order_key(float x) {
    uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// fixed-point image of a mass a in [0, 2^20): 2^43 steps per unit
constexpr double kMassScale = 8796093022208.0;   // 2^43
__device__ __forceinline__ unsigned long long mass_to_fx(float a) {
    return (unsigned long long)__double2ll_rn((double)a * kMassScale);
}
__device__ __forceinline__ float fx_to_mass(unsigned long long f) {
    return (float)((double)f / kMassScale);
}

}  // namespace cask
