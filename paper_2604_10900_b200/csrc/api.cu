// C-ABI layer of libcask: argument checks, budget split, workspace carving, call sequencing.
// Every error is found here, on the host, before anything is launched.
#include <climits>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <thread>
#include <vector>
#if defined(__SSE2__)
#include <emmintrin.h>
#endif

#include "cask_internal.cuh"

using namespace cask;

namespace {
struct ProfRecord { int id; cudaEvent_t a, b; };
struct ProfImpl {
    std::vector<ProfRecord> live;     // recorded, not yet read
    std::vector<cudaEvent_t> pool;    // events ready for reuse
    cudaEvent_t get() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
};
}  // namespace

void cask::Profiler::begin(int id, cudaStream_t st) {
    ProfImpl* pi = (ProfImpl*)impl;
    ProfRecord r{id, pi->get(), pi->get()};
    cudaEventRecord(r.a, st);
    pi->live.push_back(r);
}
void cask::Profiler::end(cudaStream_t st) {
    ProfImpl* pi = (ProfImpl*)impl;
    cudaEventRecord(pi->live.back().b, st);
}

struct cask_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    UnitDesc* pinned = nullptr;      // staging for the per-unit descriptors
    size_t pinned_units = 0;
    cudaEvent_t staged = nullptr;    // recorded after the last descriptor upload
    bool staged_pending = false;
    int64_t launches = 0;
    cudaError_t last_err = cudaSuccess;
    int last_tc = 0;
    const int32_t* flags_dev = nullptr;   // flag word of the last call's workspace
    // host-buffer entry point: pinned staging for the row kinds coming back and the packed value rows going in
    char* hstage = nullptr;
    size_t hstage_bytes = 0;
    // streams and events the slices of a large host batch take turns on; one flag word per slice
    cudaStream_t hs[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaStream_t hs_up = nullptr;    // every host-to-device copy of a sliced call, in the order they are needed
    cudaEvent_t hs_start = nullptr;
    std::vector<cudaEvent_t> hs_ev;  // three per slice: keys up, row kinds down, value rows up
    int32_t* hs_flags = nullptr;     // pinned, kMaxSlices words
    int32_t flags_last = 0;          // flags of a call that has already read them back
    void* tmap_encode = nullptr;     // cuTensorMapEncodeTiled, resolved at creation
    int sms = 0;                     // multiprocessors of the device
    Profiler prof;
    ProfImpl prof_impl;
};

namespace {

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
inline size_t elem_size(int dtype) { return dtype == CASK_DTYPE_BF16 ? 2 : 4; }

// The budget split (Sec. 2.2, 2.3, 5.2); the rule is stated beside cask_plan_host in cask.h.
void plan_unit(int T, int P, int B, int reserve, int W, float gamma, int32_t* pl) {
    const int Nd = T - P;
    const int Bp = B - reserve;
    int Pkeep = std::min(P, Bp), Bd, r = std::min(W, Nd), c = 0, m = 0, flags = 0, nout;
    if (T <= B) {
        flags = CASK_ST_NOOP_UNDER_BUDGET;
        Pkeep = P;
        Bd = B - P;
        c = Nd - r;
        nout = T;
    } else {
        Bd = B - Pkeep;
        if (P > Bp) flags |= CASK_ST_PREFIX_EVICTED;
        if (Nd <= Bd) {
            c = Nd - r;
            nout = Pkeep + Nd;
        } else if (Bd < r + 2) {
            flags |= CASK_ST_PREFIX_BUDGET_EXHAUSTED;
            r = std::min(r, Bd);
            c = Bd - r;
            nout = Pkeep + Bd;
        } else {
            flags |= CASK_ST_DECODE_CONSOLIDATED;
            const int room = Bd - r;
            c = (int)std::ceil((double)gamma * (double)room);
            c = std::max(0, std::min(c, room - 1));
            m = room - c;
            nout = Pkeep + Bd;
        }
    }
    pl[CASK_PLAN_BP] = Bp; pl[CASK_PLAN_PKEEP] = Pkeep; pl[CASK_PLAN_BD] = Bd; pl[CASK_PLAN_R] = r;
    pl[CASK_PLAN_C] = c; pl[CASK_PLAN_M] = m; pl[CASK_PLAN_FLAGS] = flags; pl[CASK_PLAN_NOUT] = nout;
}

int check_batch(const cask_batch* b, const cask_params* p) {
    if (!b || !p) return CASK_ERR_NULL;
    if (b->n_units < 0) return CASK_ERR_SHAPE;
    if (b->page_size < 0) return CASK_ERR_SHAPE;
    if (b->dtype != CASK_DTYPE_BF16 && b->dtype != CASK_DTYPE_FP32) return CASK_ERR_SHAPE;
    if (b->head_dim < 8 || b->head_dim > 256 || b->head_dim % 8) return CASK_ERR_SHAPE;
    if (b->group < 1 || b->window < 1 || (int64_t)b->group * b->window > 65536) return CASK_ERR_SHAPE;
    if (!(p->gamma >= 0.f && p->gamma <= 1.f) || !(p->eps > 0.f) || std::isnan(p->tau) ||
        (p->causal != 0 && p->causal != 1) || (p->score_path != 0 && p->score_path != 1))
        return CASK_ERR_PARAM;
    if (b->n_units == 0) return CASK_OK;
    const bool paged = b->page_size > 0;
    if (!b->k || !b->v || !b->q || !b->T || !b->P || !b->B || !b->reserve || !b->tok_off) return CASK_ERR_NULL;
    if (!paged && (!b->k_off || !b->v_off)) return CASK_ERR_NULL;
    if (paged && (!b->block_table || !b->bt_off)) return CASK_ERR_NULL;
    if (paged && (b->n_pages < 1 || (uintptr_t)b->block_table % 4)) return CASK_ERR_SHAPE;
    const size_t e = elem_size(b->dtype);
    if (b->row_stride < b->head_dim) return CASK_ERR_SHAPE;
    if (((uintptr_t)b->k | (uintptr_t)b->v | (uintptr_t)b->q) % 16 || (b->row_stride * e) % 16)
        return CASK_ERR_ALIGN;
    if (b->lse_in && (uintptr_t)b->lse_in % 4) return CASK_ERR_ALIGN;
    if (b->mass_in && (uintptr_t)b->mass_in % 4) return CASK_ERR_ALIGN;
    if (b->chan_w && (uintptr_t)b->chan_w % 4) return CASK_ERR_ALIGN;
    if (b->band_w) {
        if ((uintptr_t)b->band_w % 4) return CASK_ERR_ALIGN;
        if (b->chan_w || (b->head_dim & 1) || (b->band_layout != 0 && b->band_layout != 1)) return CASK_ERR_SHAPE;
    }
    for (int u = 0; u < b->n_units; ++u) {
        const int T = b->T[u], P = b->P[u], B = b->B[u], R = b->reserve[u];
        if (T < 1 || b->window > T || P < 0 || P > T || B < 1 || R < 0 || R > B) return CASK_ERR_SHAPE;
        if (paged) {
            const int64_t need = ((int64_t)T + b->page_size - 1) / b->page_size;
            if (b->bt_off[u] < 0 || b->bt_off[u + 1] - b->bt_off[u] < need || b->bt_off[u + 1] > INT32_MAX)
                return CASK_ERR_SHAPE;
        } else {
            if (b->k_off[u] < 0 || b->v_off[u] < 0) return CASK_ERR_SHAPE;
            if ((b->k_off[u] * e) % 16 || (b->v_off[u] * e) % 16) return CASK_ERR_ALIGN;
        }
        if (b->tok_off[u] < 0 || b->tok_off[u + 1] - b->tok_off[u] < T) return CASK_ERR_SHAPE;
    }
    return CASK_OK;
}

struct Sizes {
    int64_t sum_T = 0, sum_m = 0;
    int total_chunks = 0, max_chunks = 0, max_m = 0, max_T = 0, max_P = 0, max_B = 0;
};

Sizes batch_sizes(const cask_batch* b, const cask_params* p) {
    Sizes z;
    z.sum_T = b->n_units ? b->tok_off[b->n_units] : 0;
    for (int u = 0; u < b->n_units; ++u) {
        int32_t pl[8];
        plan_unit(b->T[u], b->P[u], b->B[u], b->reserve[u], b->window, p->gamma, pl);
        const int nch = (b->T[u] + kChunkKeys - 1) / kChunkKeys;
        z.total_chunks += nch;
        z.max_chunks = std::max(z.max_chunks, nch);
        z.sum_m += pl[CASK_PLAN_M];
        z.max_m = std::max(z.max_m, pl[CASK_PLAN_M]);
        z.max_T = std::max(z.max_T, b->T[u]);
        z.max_P = std::max(z.max_P, b->P[u]);
        z.max_B = std::max(z.max_B, b->B[u]);
    }
    return z;
}

// Lays the workspace out; with base == nullptr only the size is computed.
Workspace carve(char* base, const cask_batch* b, const Sizes& z) {
    Workspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) -> char* {
        char* p = base ? base + off : nullptr;
        off += align_up(std::max<size_t>(bytes, 16));
        return p;
    };
    const size_t n = (size_t)b->n_units, rows = (size_t)b->group * b->window, sumT = (size_t)z.sum_T;
    w.desc = (UnitDesc*)take(n * sizeof(UnitDesc));
    w.s = (float*)take(sumT * 4);
    w.rowm = (float*)take(n * rows * 4);
    w.roww = (float*)take(n * rows * 4);
    const size_t parts = std::max((size_t)z.total_chunks, score_tc_partial_slots(b->n_units));
    w.part_m = (float*)take(parts * rows * 4);
    w.part_l = (float*)take(parts * rows * 4);
    w.seed_rows = (int32_t*)take((size_t)z.sum_m * 4);
    w.seed_norm = (float*)take((size_t)z.sum_m * 4);
    w.seed_k = take((2 * (size_t)z.sum_m + 256) * b->head_dim * elem_size(b->dtype));   // room for hi/lo rows
    w.grp = (int32_t*)take(sumT * 4);
    w.mass_fx = (unsigned long long*)take(n * ((size_t)z.max_m + 1) * 8);
    w.njoin = (int32_t*)take(n * 4);
    w.mem_row = (int32_t*)take(sumT * 4);
    w.mem_slot = (int32_t*)take(sumT * 4);
    w.n_mem = (int32_t*)take(n * 4);
    w.seed_slot = (int32_t*)take(n * (size_t)std::max(z.max_B, 1) * 4);
    w.n_seed = (int32_t*)take(n * 4);
    w.max_B = std::max(z.max_B, 1);
    w.err = (int32_t*)take(16);
    w.stats_a = (float*)take((n + 4) * (size_t)b->head_dim * 4);      // per-unit coefficients + one table of band constants
    w.bytes = off;
    return w;
}

int fail_cuda(cask_ctx* ctx, cudaError_t e) {
    ctx->last_err = e;
    return CASK_ERR_CUDA;
}

// Validates, builds and uploads the per-unit descriptors, resolves the launch record.
int prepare(cask_ctx* ctx, const cask_batch* b, const cask_params* p, void* ws, size_t ws_bytes, Launch& L,
            Workspace& W) {
    if (!ctx) return CASK_ERR_NULL;
    int rc = check_batch(b, p);
    if (rc != CASK_OK) return rc;
    if (b->n_units == 0) return CASK_OK;
    const Sizes z = batch_sizes(b, p);
    W = carve(nullptr, b, z);
    if (!ws || ws_bytes < W.bytes || (uintptr_t)ws % 256) return CASK_ERR_WORKSPACE;
    W = carve((char*)ws, b, z);

    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    if (ctx->staged_pending) {
        e = cudaEventSynchronize(ctx->staged);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->staged_pending = false;
    }
    if (ctx->pinned_units < (size_t)b->n_units) {
        if (ctx->pinned) cudaFreeHost(ctx->pinned);
        ctx->pinned = nullptr;
        ctx->pinned_units = 0;
        e = cudaMallocHost((void**)&ctx->pinned, sizeof(UnitDesc) * (size_t)b->n_units);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->pinned_units = (size_t)b->n_units;
    }
    Shape shp{};
    shp.page_size = b->page_size;
    const int a_sub = b->page_size ? assign_tc_box_rows(shp) : 0;    // page piece the assignment tiles start on
    int chunk0 = 0, seed_base = 0, atile0 = 0, tile0 = 0;
    const int64_t q_unit = (int64_t)b->group * b->window * b->head_dim;
    for (int u = 0; u < b->n_units; ++u) {
        UnitDesc& d = ctx->pinned[u];
        d.k_off = b->page_size ? 0 : b->k_off[u];
        d.v_off = b->page_size ? 0 : b->v_off[u];
        d.bt0 = b->page_size ? (int32_t)b->bt_off[u] : 0;
        d.pad = 0;
        d.q_off = q_unit * u;
        d.tok_off = b->tok_off[u];
        d.T = b->T[u]; d.P = b->P[u]; d.B = b->B[u]; d.reserve = b->reserve[u];
        plan_unit(d.T, d.P, d.B, d.reserve, b->window, p->gamma, d.plan);
        d.chunk0 = chunk0;
        d.n_chunks = (d.T + kChunkKeys - 1) / kChunkKeys;
        d.seed_base = seed_base;
        d.atile0 = atile0;
        const int a0 = d.P - (a_sub > 0 ? d.P % a_sub : 0);
        d.n_atiles = d.plan[CASK_PLAN_M] > 0 ? (d.T - d.plan[CASK_PLAN_R] - a0 + 127) / 128 : 0;
        d.tile0 = tile0;
        tile0 += (d.T + 127) / 128;
        chunk0 += d.n_chunks;
        seed_base += d.plan[CASK_PLAN_M];
        atile0 += d.n_atiles;
    }
    e = cudaMemcpyAsync(W.desc, ctx->pinned, sizeof(UnitDesc) * (size_t)b->n_units, cudaMemcpyHostToDevice,
                        ctx->stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    e = cudaEventRecord(ctx->staged, ctx->stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->staged_pending = true;
    e = cudaMemsetAsync(W.err, 0, 16, ctx->stream);      // device-side flags of this call
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->flags_dev = W.err;
    ctx->flags_last = 0;

    L.stream = ctx->stream;
    L.sh.n_units = b->n_units; L.sh.d = b->head_dim; L.sh.g = b->group; L.sh.W = b->window;
    L.sh.rows = b->group * b->window; L.sh.dtype = b->dtype; L.sh.row_stride = b->row_stride;
    L.sh.causal = p->causal;
    L.sh.page_size = b->page_size; L.sh.n_pages = b->n_pages; L.sh.bt = b->block_table; L.sh.err = W.err;
    L.sh.mass_in = b->mass_in; L.sh.chan_w = b->chan_w;
    L.sh.band_w = b->band_w; L.sh.band_layout = b->band_layout;
    L.desc = W.desc; L.hdesc = ctx->pinned;
    L.k = b->k; L.v = b->v; L.q = b->q;
    L.max_T = z.max_T; L.max_m = z.max_m; L.max_chunks = z.max_chunks; L.total_chunks = z.total_chunks;
    L.max_P = z.max_P; L.max_B = z.max_B; L.sum_T = z.sum_T;
    L.total_atiles = atile0;
    L.total_tiles = tile0;
    L.tmap_encode = ctx->tmap_encode;
    L.force_simt = p->score_path;
    L.sms = ctx->sms;
    L.launches = &ctx->launches;
    L.prof = &ctx->prof;
    return CASK_OK;
}

int run_score(cask_ctx* ctx, const Launch& L, const cask_batch* b, const cask_params* p, float* s,
              float* lse_out, Workspace& W) {
    cudaError_t e;
    if (p->score_path == 0 && ctx->tmap_encode && score_tc_supported(L)) {
        ctx->last_tc = 1;
        e = launch_score_tc(L, b->lse_in, s, lse_out, W, ctx->tmap_encode);
    } else {
        ctx->last_tc = 0;
        e = launch_score_simt(L, b->lse_in, s, lse_out, W);
    }
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

}  // namespace

namespace cask {
// The host-side argument check, for entry points that live in other files.
int check_batch_host(const cask_batch* b, const cask_params* p) { return check_batch(b, p); }
// The self-tests: their flag word (if any) becomes the one cask_last_device_flags reads, their launches are counted.
int selftest_set_flags_source(cask_ctx* ctx, const int32_t* flags_dev, int n_launches, cudaStream_t* stream, int* device) {
    if (!ctx) return CASK_ERR_NULL;
    ctx->flags_dev = flags_dev;
    ctx->flags_last = 0;
    ctx->last_tc = 0;
    ctx->launches += n_launches;
    *stream = ctx->stream;
    *device = ctx->device;
    return CASK_OK;
}
}  // namespace cask

extern "C" {

int cask_create(cask_ctx** out, int device, void* cuda_stream) {
    if (!out) return CASK_ERR_NULL;
    *out = nullptr;
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return CASK_ERR_CUDA;
    cask_ctx* c = new (std::nothrow) cask_ctx();
    if (!c) return CASK_ERR_CUDA;
    c->device = device;
    c->stream = (cudaStream_t)cuda_stream;
    c->prof.impl = &c->prof_impl;
    e = cudaEventCreateWithFlags(&c->staged, cudaEventDisableTiming);
    if (e != cudaSuccess) { delete c; return CASK_ERR_CUDA; }
    if (cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) c->sms = 0;
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        c->tmap_encode = fn;
    else
        cudaGetLastError();
    *out = c;
    return CASK_OK;
}

int cask_destroy(cask_ctx* ctx) {
    if (!ctx) return CASK_ERR_NULL;
    cudaSetDevice(ctx->device);
    if (ctx->staged_pending) cudaEventSynchronize(ctx->staged);
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    if (ctx->hstage) cudaFreeHost(ctx->hstage);
    if (ctx->staged) cudaEventDestroy(ctx->staged);
    for (cudaStream_t st : ctx->hs)
        if (st) cudaStreamDestroy(st);
    if (ctx->hs_start) cudaEventDestroy(ctx->hs_start);
    if (ctx->hs_flags) cudaFreeHost(ctx->hs_flags);
    if (ctx->hs_up) cudaStreamDestroy(ctx->hs_up);
    for (cudaEvent_t ev : ctx->hs_ev) cudaEventDestroy(ev);
    for (ProfRecord& r : ctx->prof_impl.live) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (cudaEvent_t e : ctx->prof_impl.pool) cudaEventDestroy(e);
    delete ctx;
    return CASK_OK;
}

int cask_set_stream(cask_ctx* ctx, void* cuda_stream) {
    if (!ctx) return CASK_ERR_NULL;
    ctx->stream = (cudaStream_t)cuda_stream;
    return CASK_OK;
}

const char* cask_strerror(int code) {
    switch (code) {
        case CASK_OK: return "ok";
        case CASK_ERR_NULL: return "a required pointer is NULL";
        case CASK_ERR_SHAPE: return "shape out of range (head_dim, group, window, T, P, B, reserve, offsets)";
        case CASK_ERR_ALIGN: return "pointer, offset or row stride is not a multiple of 16 bytes";
        case CASK_ERR_WORKSPACE: return "workspace missing, misaligned (256 B) or too small";
        case CASK_ERR_UNSUPPORTED: return "mode not built (paged cache through the host-buffer or no-allocation entry point, or a capturing stream there)";
        case CASK_ERR_CUDA: return "CUDA runtime error";
        case CASK_ERR_PARAM: return "policy parameter out of range";
        case CASK_ERR_TOO_LARGE: return "batch exceeds the fixed capacity of the no-allocation entry point";
        default: return "unknown error";
    }
}

const char* cask_last_cuda_error(const cask_ctx* ctx) {
    if (!ctx || ctx->last_err == cudaSuccess) return "";
    return cudaGetErrorName(ctx->last_err);
}

int64_t cask_launch_count(const cask_ctx* ctx) { return ctx ? ctx->launches : 0; }

int cask_profile_enable(cask_ctx* ctx, int on) {
    if (!ctx) return CASK_ERR_NULL;
    ctx->prof.on = on != 0;
    return CASK_OK;
}

int cask_kernel_count(void) { return KID_COUNT; }

const char* cask_kernel_name(int id) {
    static const char* names[KID_COUNT] = {"score_norm", "row_combine", "score_mass", "prefix_evict",
                                           "select_core", "seeds", "seed_gather", "assign", "weights",
                                           "slot_scan", "gather_merge", "diagnostics"};
    return (id >= 0 && id < KID_COUNT) ? names[id] : "";
}

int cask_profile_read(cask_ctx* ctx, float* ms, int64_t* launches) {
    if (!ctx || !ms || !launches) return CASK_ERR_NULL;
    for (int i = 0; i < KID_COUNT; ++i) { ms[i] = 0.f; launches[i] = 0; }
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    for (ProfRecord& r : ctx->prof_impl.live) {
        e = cudaEventSynchronize(r.b);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        float t = 0.f;
        e = cudaEventElapsedTime(&t, r.a, r.b);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ms[r.id] += t;
        launches[r.id] += 1;
        ctx->prof_impl.pool.push_back(r.a);
        ctx->prof_impl.pool.push_back(r.b);
    }
    ctx->prof_impl.live.clear();
    return CASK_OK;
}
int cask_last_score_path_tensor(const cask_ctx* ctx) { return ctx ? ctx->last_tc : 0; }

int cask_last_score_clock_khz(cask_ctx* ctx, int32_t* khz_host) {
    if (!ctx || !khz_host) return CASK_ERR_NULL;
    khz_host[0] = khz_host[1] = 0;
    if (!ctx->flags_dev || !ctx->last_tc) return CASK_OK;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(khz_host, ctx->flags_dev + 2, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

int cask_last_device_flags(cask_ctx* ctx, int32_t* flags_host) {
    if (!ctx || !flags_host) return CASK_ERR_NULL;
    *flags_host = ctx->flags_last;
    if (!ctx->flags_dev) return CASK_OK;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(flags_host, ctx->flags_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

size_t cask_workspace_bytes(const cask_batch* batch, const cask_params* params) {
    if (check_batch(batch, params) != CASK_OK || batch->n_units == 0) return 0;
    return carve(nullptr, batch, batch_sizes(batch, params)).bytes;
}

int cask_plan_host(const cask_batch* b, const cask_params* p, int32_t* plan_host) {
    if (!b || !p || !plan_host) return CASK_ERR_NULL;
    if (b->n_units > 0 && (!b->T || !b->P || !b->B || !b->reserve)) return CASK_ERR_NULL;
    if (!(p->gamma >= 0.f && p->gamma <= 1.f)) return CASK_ERR_PARAM;
    for (int u = 0; u < b->n_units; ++u) {
        const int T = b->T[u], P = b->P[u], B = b->B[u], R = b->reserve[u];
        if (T < 1 || b->window < 1 || b->window > T || P < 0 || P > T || B < 1 || R < 0 || R > B)
            return CASK_ERR_SHAPE;
        plan_unit(T, P, B, R, b->window, p->gamma, plan_host + (size_t)u * 8);
    }
    return CASK_OK;
}

int cask_score(cask_ctx* ctx, const cask_batch* b, const cask_params* p, float* s, float* lse_out, void* ws,
               size_t ws_bytes) {
    if (!s) return CASK_ERR_NULL;
    Launch L{};
    Workspace W{};
    int rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    return run_score(ctx, L, b, p, s, lse_out, W);
}

int cask_score_stats(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const cask_query_stats* qs, float* s,
                     void* ws, size_t ws_bytes) {
    if (!s || !qs || !qs->mu || !qs->pi || !qs->delta_grid || !qs->omega) return CASK_ERR_NULL;
    if (qs->n_delta < 1 || qs->n_delta > 4096 || (qs->band_layout != 0 && qs->band_layout != 1)) return CASK_ERR_SHAPE;
    if (((uintptr_t)qs->mu | (uintptr_t)qs->pi | (uintptr_t)qs->delta_grid | (uintptr_t)qs->omega |
         (uintptr_t)qs->delta) % 4)
        return CASK_ERR_ALIGN;
    Launch L{};
    Workspace W{};
    int rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    if (b->head_dim & 1) return CASK_ERR_SHAPE;
    cudaError_t e = launch_score_stats(L, *qs, s, W);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

int cask_prefix_evict(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const float* s, uint8_t* kind,
                      int32_t* plan, void* ws, size_t ws_bytes) {
    if (!s || !kind || !plan) return CASK_ERR_NULL;
    Launch L{};
    Workspace W{};
    int rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    cudaError_t e = launch_prefix_evict(L, s, kind, plan);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

int cask_select_core(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const float* s,
                     const int32_t* plan, uint8_t* kind, void* ws, size_t ws_bytes) {
    if (!s || !kind || !plan) return CASK_ERR_NULL;
    Launch L{};
    Workspace W{};
    int rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    cudaError_t e = launch_select_core(L, s, plan, kind);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

int cask_consolidate_scratch(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const float* s,
                             const int32_t* plan, uint8_t* kind, int32_t* seed_of, float* weight, float* sim,
                             int32_t* unit_status, float* lost_mass, void* ws, size_t ws_bytes) {
    if (!s || !kind || !plan || !seed_of || !weight || !unit_status || !lost_mass) return CASK_ERR_NULL;
    Launch L{};
    Workspace W{};
    int rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    cudaError_t e = launch_consolidate(L, *p, s, plan, kind, seed_of, weight, sim, unit_status, lost_mass, W);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

static int max_budget(const cask_batch* b) {
    int mb = 0;
    if (b && b->B)
        for (int u = 0; u < b->n_units; ++u) mb = std::max(mb, b->B[u]);
    return mb;
}

static int check_compact_out(const cask_outputs* o, int max_B) {
    if (!o) return CASK_ERR_NULL;
    if (!o->k_out || !o->v_out || !o->n_out || !o->slot_src || !o->slot_kind || !o->slot_mass || !o->assign)
        return CASK_ERR_NULL;
    if (o->Bmax < max_B) return CASK_ERR_SHAPE;
    if (((uintptr_t)o->k_out | (uintptr_t)o->v_out) % 16) return CASK_ERR_ALIGN;
    return CASK_OK;
}

int cask_compact(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const float* s, const uint8_t* kind,
                 const int32_t* seed_of, float* weight, const cask_outputs* out, void* ws, size_t ws_bytes) {
    if (!s || !kind || !seed_of || !weight) return CASK_ERR_NULL;
    int rc = check_compact_out(out, max_budget(b));
    if (rc != CASK_OK) return rc;
    Launch L{};
    Workspace W{};
    rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    cudaError_t e = launch_compact(L, *p, s, kind, seed_of, weight, *out, W);
    if (e == cudaSuccess) e = launch_diagnostics(L, *p, s, kind, *out);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

// The event up to the point where every row's fate is known (score, selections, group assignment, weights);
// only keys are read.
static int event_decide(cask_ctx* ctx, Launch& L, Workspace& W, const cask_batch* b, const cask_params* p,
                        const cask_outputs* out) {
    float* s = out->s ? out->s : W.s;
    int rc = run_score(ctx, L, b, p, s, out->lse, W);
    if (rc != CASK_OK) return rc;
    // the event leaves prefix eviction and core selection to the fused selection kernel of the consolidation step
    cudaError_t e = launch_consolidate(L, *p, s, out->plan, out->kind, out->seed_of, out->weight, out->sim,
                                       out->unit_status, out->lost_mass, W, true);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

// The rest: compaction (the only step that reads values) and the optional diagnostics.
static int event_compact(cask_ctx* ctx, Launch& L, Workspace& W, const cask_params* p, const cask_outputs* out) {
    float* s = out->s ? out->s : W.s;
    const EventFusion ev{out->plan, out->unit_status, out->lost_mass};
    cudaError_t e = launch_compact(L, *p, s, out->kind, out->seed_of, out->weight, *out, W, &ev);
    if (e == cudaSuccess) e = launch_diagnostics(L, *p, s, out->kind, *out);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

int cask_compress_event(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const cask_outputs* out,
                        void* ws, size_t ws_bytes) {
    int rc = check_compact_out(out, max_budget(b));
    if (rc != CASK_OK) return rc;
    if (!out->weight || !out->kind || !out->seed_of || !out->plan || !out->unit_status || !out->lost_mass)
        return CASK_ERR_NULL;
    Launch L{};
    Workspace W{};
    rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    rc = event_decide(ctx, L, W, b, p, out);
    if (rc != CASK_OK) return rc;
    return event_compact(ctx, L, W, p, out);
}

int cask_writeback_paged(cask_ctx* ctx, const cask_batch* b, const cask_params* p, const cask_outputs* out,
                         void* k_pool, void* v_pool, void* ws, size_t ws_bytes) {
    if (!out || !k_pool || !v_pool) return CASK_ERR_NULL;
    if (!out->k_out || !out->v_out || !out->n_out) return CASK_ERR_NULL;
    if (b && b->page_size <= 0) return CASK_ERR_SHAPE;
    if (((uintptr_t)k_pool | (uintptr_t)v_pool | (uintptr_t)out->k_out | (uintptr_t)out->v_out) % 16) return CASK_ERR_ALIGN;
    if (out->Bmax < max_budget(b)) return CASK_ERR_SHAPE;
    Launch L{};
    Workspace W{};
    int rc = prepare(ctx, b, p, ws, ws_bytes, L, W);
    if (rc != CASK_OK || b->n_units == 0) return rc;
    cudaError_t e = launch_writeback(L, *out, k_pool, v_pool);
    return e == cudaSuccess ? CASK_OK : fail_cuda(ctx, e);
}

}  // extern "C"

// ---- host-resident caches ------------------------------------------------------------------

namespace {
struct HostStage {
    char *k, *v, *q, *lse_in, *mass_in, *chan_w, *band_w;
    cask_outputs o;
    char* ws;
    size_t ws_bytes, bytes;
    size_t kv_bytes, q_bytes, lse_bytes;
    int32_t *v_pos, *n_need;
    int64_t* v_base;
};

HostStage stage_layout(char* base, const cask_batch* b, const cask_params* p, int32_t Bmax) {
    HostStage h{};
    size_t off = 0;
    auto take = [&](size_t bytes) -> char* {
        char* ptr = base ? base + off : nullptr;
        off += align_up(std::max<size_t>(bytes, 16));
        return ptr;
    };
    const size_t e = elem_size(b->dtype), n = (size_t)b->n_units, d = (size_t)b->head_dim;
    const size_t sumT = (size_t)b->tok_off[b->n_units], rows = (size_t)b->group * b->window;
    h.kv_bytes = sumT * d * e;
    h.q_bytes = n * rows * d * e;
    h.lse_bytes = n * rows * 4;
    h.k = take(h.kv_bytes);
    h.v = take(h.kv_bytes);
    h.q = take(h.q_bytes);
    h.lse_in = take(h.lse_bytes);
    h.mass_in = take(sumT * 4);
    h.chan_w = take(d * 4);
    h.band_w = take(d * 2);
    h.v_pos = (int32_t*)take(sumT * 4);
    h.n_need = (int32_t*)take(n * 4);
    h.v_base = (int64_t*)take(n * 8);
    h.o.Bmax = Bmax;
    h.o.k_out = take(n * Bmax * d * e);
    h.o.v_out = take(n * Bmax * d * e);
    h.o.n_out = (int32_t*)take(n * 4);
    h.o.slot_src = (int32_t*)take(n * Bmax * 4);
    h.o.slot_kind = (uint8_t*)take(n * Bmax);
    h.o.slot_mass = (float*)take(n * Bmax * 4);
    h.o.assign = (int32_t*)take(sumT * 4);
    h.o.weight = (float*)take(sumT * 4);
    h.o.kind = (uint8_t*)take(sumT);
    h.o.seed_of = (int32_t*)take(sumT * 4);
    h.o.plan = (int32_t*)take(n * 32);
    h.o.unit_status = (int32_t*)take(n * 4);
    h.o.lost_mass = (float*)take(n * 4);
    h.o.s = (float*)take(sumT * 4);
    h.o.lse = (float*)take(n * rows * 4);
    h.o.sim = (float*)take(sumT * 4);
    h.o.rho_core = (float*)take(n * 4);
    h.o.rho_rep = (float*)take(n * 4);
    h.o.dispersion = (float*)take(n * 4);
    h.ws_bytes = carve(nullptr, b, batch_sizes(b, p)).bytes;
    h.ws = take(h.ws_bytes);
    h.bytes = off;
    return h;
}

int check_host_layout(const cask_batch* b) {
    if (b->row_stride != b->head_dim) return CASK_ERR_SHAPE;
    for (int u = 0; u < b->n_units; ++u)
        if (b->k_off[u] != b->tok_off[u] * b->head_dim || b->v_off[u] != b->k_off[u]) return CASK_ERR_SHAPE;
    return CASK_OK;
}

// A large batch goes through the device in slices of consecutive units, so that one slice's upload runs while
// the one before it is being decided, packed and read back.  A slice is a batch of its own: offsets rebased to
// zero, host pointers moved to its first unit, its own staging area and workspace on the device.
constexpr size_t kSliceMinBytes = (size_t)16 << 20;   // of keys; below this the copies are too short to hide anything
constexpr int kSliceTarget = 10;                      // slices a large batch is cut into
constexpr int kSliceStreams = 4;
constexpr size_t kMaxSlices = 64;

struct HostSlice {
    int u0 = 0, u1 = 0;
    int64_t r0 = 0;                      // first row (caller's tok_off) of the slice
    std::vector<int64_t> tok, off;       // rebased offsets
    cask_batch hb;                       // host pointers of the slice
    cask_outputs ho;
    HostStage h;                         // device staging
    Launch L;
    Workspace W;
    size_t v_row0 = 0, need_rows = 0;    // place of the packed value rows in the pinned staging
    std::vector<int64_t> vbase;
};

std::vector<int> slice_bounds(const cask_batch* b) {
    const size_t row_bytes = (size_t)b->head_dim * elem_size(b->dtype);
    const size_t total = (size_t)b->tok_off[b->n_units] * row_bytes;
    const size_t target = std::max(kSliceMinBytes, total / kSliceTarget);
    std::vector<int> bounds{0};
    size_t acc = 0;
    for (int u = 0; u < b->n_units; ++u) {
        acc += (size_t)(b->tok_off[u + 1] - b->tok_off[u]) * row_bytes;
        const size_t left = (size_t)(b->tok_off[b->n_units] - b->tok_off[u + 1]) * row_bytes;
        if (acc >= target && left >= target / 2) {
            bounds.push_back(u + 1);
            acc = 0;
        }
    }
    if (bounds.back() != b->n_units) bounds.push_back(b->n_units);
    return bounds;
}

template <typename T>
T* moved(T* p, size_t n) { return p ? p + n : nullptr; }
inline void* moved_bytes(const void* p, size_t n) { return p ? (char*)p + n : nullptr; }

void make_slice(HostSlice& s, const cask_batch* hb, const cask_outputs* ho, int u0, int u1) {
    const size_t es = elem_size(hb->dtype), d = (size_t)hb->head_dim, rows = (size_t)hb->group * hb->window;
    s.u0 = u0; s.u1 = u1; s.r0 = hb->tok_off[u0];
    const size_t n = (size_t)(u1 - u0), r0 = (size_t)s.r0;
    s.tok.resize(n + 1);
    s.off.resize(n);
    for (size_t u = 0; u <= n; ++u) s.tok[u] = hb->tok_off[u0 + u] - s.r0;
    for (size_t u = 0; u < n; ++u) s.off[u] = s.tok[u] * (int64_t)d;
    s.hb = *hb;
    s.hb.n_units = (int32_t)n;
    s.hb.T = hb->T + u0; s.hb.P = hb->P + u0; s.hb.B = hb->B + u0; s.hb.reserve = hb->reserve + u0;
    s.hb.tok_off = s.tok.data();
    s.hb.k_off = s.off.data();
    s.hb.v_off = s.off.data();
    s.hb.k = moved_bytes(hb->k, r0 * d * es);
    s.hb.v = moved_bytes(hb->v, r0 * d * es);
    s.hb.q = moved_bytes(hb->q, (size_t)u0 * rows * d * es);
    s.hb.lse_in = moved(hb->lse_in, (size_t)u0 * rows);
    s.hb.mass_in = moved(hb->mass_in, r0);
    if (!ho) return;
    const size_t Bm = (size_t)ho->Bmax;
    s.ho = *ho;
    s.ho.k_out = moved_bytes(ho->k_out, (size_t)u0 * Bm * d * es);
    s.ho.v_out = moved_bytes(ho->v_out, (size_t)u0 * Bm * d * es);
    s.ho.n_out = moved(ho->n_out, (size_t)u0);
    s.ho.slot_src = moved(ho->slot_src, (size_t)u0 * Bm);
    s.ho.slot_kind = moved(ho->slot_kind, (size_t)u0 * Bm);
    s.ho.slot_mass = moved(ho->slot_mass, (size_t)u0 * Bm);
    s.ho.assign = moved(ho->assign, r0);
    s.ho.weight = moved(ho->weight, r0);
    s.ho.kind = moved(ho->kind, r0);
    s.ho.seed_of = moved(ho->seed_of, r0);
    s.ho.plan = moved(ho->plan, (size_t)u0 * 8);
    s.ho.unit_status = moved(ho->unit_status, (size_t)u0);
    s.ho.lost_mass = moved(ho->lost_mass, (size_t)u0);
    s.ho.s = moved(ho->s, r0);
    s.ho.lse = moved(ho->lse, (size_t)u0 * rows);
    s.ho.sim = moved(ho->sim, r0);
    s.ho.rho_core = moved(ho->rho_core, (size_t)u0);
    s.ho.rho_rep = moved(ho->rho_rep, (size_t)u0);
    s.ho.dispersion = moved(ho->dispersion, (size_t)u0);
}

// Copies one value row into the pinned staging with stores that go past the caches where the CPU has them: the
// next reader is the GPU's copy engine, and lines left dirty in the caches of sixteen cores made its read of a
// 4 MB slice take 0.5 ms instead of 0.1 ms.
inline void stage_row(char* dst, const char* src, size_t bytes) {
#if defined(__SSE2__)
    if ((((uintptr_t)dst | bytes) & 15) == 0) {
        for (size_t o = 0; o < bytes; o += 16)
            _mm_stream_si128((__m128i*)(dst + o), _mm_loadu_si128((const __m128i*)(src + o)));
        return;
    }
#endif
    memcpy(dst, src, bytes);
}
inline void stage_fence() {
#if defined(__SSE2__)
    _mm_sfence();
#endif
}

// Runs fn(u) for u in [0, n) on up to 16 host threads.
template <typename F>
void over_units(size_t n, F fn) {
    const unsigned nthr = (unsigned)std::min<size_t>(n, std::max(1u, std::min(16u, std::thread::hardware_concurrency())));
    if (nthr <= 1) {
        for (size_t u = 0; u < n; ++u) fn(u);
        return;
    }
    std::vector<std::thread> th;
    for (unsigned t = 0; t < nthr; ++t)
        th.emplace_back([&, t] {
            for (size_t u = t; u < n; u += nthr) fn(u);
        });
    for (auto& x : th) x.join();
}

// Upload of a slice's keys, queries and per-row inputs.  Values do not go up here: only the compaction reads
// them, and only the rows that are kept or merged, so they follow later, packed, once the rows' fates are known.
cudaError_t slice_upload(HostSlice& s, cudaStream_t st) {
    const cask_batch& hb = s.hb;
    HostStage& h = s.h;
    // the small arrays first: one of them in pageable memory then holds the host only until the stream's earlier
    // work is done, not until the keys queued here have arrived
    cudaError_t e = cudaMemcpyAsync(h.q, hb.q, h.q_bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && hb.lse_in) e = cudaMemcpyAsync(h.lse_in, hb.lse_in, h.lse_bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && hb.mass_in)
        e = cudaMemcpyAsync(h.mass_in, hb.mass_in, (size_t)hb.tok_off[hb.n_units] * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && hb.chan_w)
        e = cudaMemcpyAsync(h.chan_w, hb.chan_w, (size_t)hb.head_dim * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && hb.band_w)
        e = cudaMemcpyAsync(h.band_w, hb.band_w, (size_t)(hb.head_dim / 2) * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h.k, hb.k, h.kv_bytes, cudaMemcpyHostToDevice, st);
    return e;
}
}  // namespace

extern "C" {

size_t cask_host_event_device_bytes(const cask_batch* b, const cask_params* p, int32_t Bmax) {
    if (check_batch(b, p) != CASK_OK || b->n_units == 0 || Bmax < 1) return 0;
    const std::vector<int> bounds = slice_bounds(b);
    size_t bytes = 0;
    for (size_t i = 0; i + 1 < bounds.size(); ++i) {
        HostSlice s;
        make_slice(s, b, nullptr, bounds[i], bounds[i + 1]);
        bytes += stage_layout(nullptr, &s.hb, p, Bmax).bytes;
    }
    return bytes;
}

int cask_compress_event_host(cask_ctx* ctx, const cask_batch* hb, const cask_params* p,
                             const cask_outputs* ho, void* dev_buf, size_t dev_bytes) {
    if (!ctx || !ho) return CASK_ERR_NULL;
    int rc = check_batch(hb, p);
    if (rc != CASK_OK) return rc;
    if (hb->page_size != 0) return CASK_ERR_UNSUPPORTED;
    if (hb->n_units == 0) return CASK_OK;
    rc = check_host_layout(hb);
    if (rc != CASK_OK) return rc;
    if (ho->Bmax < 1) return CASK_ERR_SHAPE;
    if (!dev_buf || (uintptr_t)dev_buf % 256) return CASK_ERR_WORKSPACE;

    const std::vector<int> bounds = slice_bounds(hb);
    const size_t C = bounds.size() - 1;
    if (C > kMaxSlices) return CASK_ERR_SHAPE;      // cannot happen: a slice holds a tenth of the batch or more
    std::vector<HostSlice> sl(C);
    size_t used = 0;
    for (size_t i = 0; i < C; ++i) {
        make_slice(sl[i], hb, ho, bounds[i], bounds[i + 1]);
        const size_t need = stage_layout(nullptr, &sl[i].hb, p, ho->Bmax).bytes;
        if (used + need > dev_bytes) return CASK_ERR_WORKSPACE;
        sl[i].h = stage_layout((char*)dev_buf + used, &sl[i].hb, p, ho->Bmax);
        used += need;
        // optional diagnostics are computed only when the caller has a place for them
        if (!ho->rho_core) sl[i].h.o.rho_core = nullptr;
        if (!ho->rho_rep) sl[i].h.o.rho_rep = nullptr;
        if (!ho->dispersion) sl[i].h.o.dispersion = nullptr;
    }
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return fail_cuda(ctx, e);

    // One slice runs on the caller's stream.  Several use streams of the context, which start after the work
    // already queued on the caller's stream and are drained before the call returns: one stream for every copy
    // to the device, in the order the copies are needed (copies queued on different streams are served in turns
    // per stream, not in the order they were queued: a slice's few value rows then wait behind the keys of three
    // later slices), and four that the slices take turns on for their kernels and their copies to the host.
    cudaStream_t const user = ctx->stream;
    const bool sliced = C > 1;
    if (sliced) {
        for (int j = 0; j < kSliceStreams && e == cudaSuccess; ++j)
            if (!ctx->hs[j]) e = cudaStreamCreateWithFlags(&ctx->hs[j], cudaStreamNonBlocking);
        if (e == cudaSuccess && !ctx->hs_up) e = cudaStreamCreateWithFlags(&ctx->hs_up, cudaStreamNonBlocking);
        if (e == cudaSuccess && !ctx->hs_start) e = cudaEventCreateWithFlags(&ctx->hs_start, cudaEventDisableTiming);
        while (e == cudaSuccess && ctx->hs_ev.size() < 3 * C) {
            cudaEvent_t ev = nullptr;
            e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            if (e == cudaSuccess) ctx->hs_ev.push_back(ev);
        }
        if (e == cudaSuccess) e = cudaEventRecord(ctx->hs_start, user);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->hs_up, ctx->hs_start, 0);
        for (int j = 0; j < kSliceStreams && e == cudaSuccess; ++j) e = cudaStreamWaitEvent(ctx->hs[j], ctx->hs_start, 0);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    cudaStream_t const up = sliced ? ctx->hs_up : user;
    auto stream_of = [&](size_t i) { return sliced ? ctx->hs[i % kSliceStreams] : user; };
    auto ev_keys = [&](size_t i) { return ctx->hs_ev[3 * i]; };
    auto ev_kinds = [&](size_t i) { return ctx->hs_ev[3 * i + 1]; };
    auto ev_values = [&](size_t i) { return ctx->hs_ev[3 * i + 2]; };
    auto drain = [&]() {
        cudaError_t first = cudaSuccess;
        if (sliced) {
            first = cudaStreamSynchronize(ctx->hs_up);
            for (int j = 0; j < kSliceStreams; ++j) {
                const cudaError_t x = cudaStreamSynchronize(ctx->hs[j]);
                if (first == cudaSuccess) first = x;
            }
        } else
            first = cudaStreamSynchronize(user);
        return first;
    };
    // leaves with the context's stream restored and nothing of this call still in flight
    auto leave = [&](int code, cudaError_t ce) {
        ctx->stream = user;
        const cudaError_t de = drain();
        if (code == CASK_OK && ce == cudaSuccess && de != cudaSuccess) ce = de;
        if (ce != cudaSuccess) return fail_cuda(ctx, ce);
        return code;
    };

    const size_t es = elem_size(hb->dtype), d = (size_t)hb->head_dim, row_bytes = d * es;
    const size_t sumT = (size_t)hb->tok_off[hb->n_units], rows = (size_t)hb->group * hb->window;
    const size_t Bm = (size_t)ho->Bmax;
    const size_t v_stage0 = align_up(sumT);      // the row kinds first, the packed value rows behind them
    if (ctx->hstage_bytes < v_stage0 + 4096 * row_bytes) {
        if (ctx->hstage) cudaFreeHost(ctx->hstage);
        ctx->hstage = nullptr;
        ctx->hstage_bytes = 0;
        const size_t nb = v_stage0 + (sumT / 8 + 4096) * row_bytes;
        e = cudaMallocHost((void**)&ctx->hstage, nb);
        if (e != cudaSuccess) return leave(CASK_OK, e);
        ctx->hstage_bytes = nb;
    }

    // keys up, the rows' fates decided, the row kinds on their way back
    auto decide = [&](size_t i) -> int {
        HostSlice& s = sl[i];
        cudaStream_t st = stream_of(i);
        cask_batch db = s.hb;
        db.k = s.h.k; db.v = s.h.v; db.q = s.h.q;
        db.lse_in = s.hb.lse_in ? (const float*)s.h.lse_in : nullptr;
        db.mass_in = s.hb.mass_in ? (const float*)s.h.mass_in : nullptr;
        db.chan_w = s.hb.chan_w ? (const float*)s.h.chan_w : nullptr;
        db.band_w = s.hb.band_w ? (const float*)s.h.band_w : nullptr;
        ctx->stream = up;               // the descriptors go up behind the slice's keys
        int r = prepare(ctx, &db, p, s.h.ws, s.h.ws_bytes, s.L, s.W);
        ctx->stream = user;
        if (r != CASK_OK) return r;
        s.L.stream = st;
        if (sliced) {
            cudaError_t we = cudaEventRecord(ev_keys(i), up);
            if (we == cudaSuccess) we = cudaStreamWaitEvent(st, ev_keys(i), 0);
            if (we != cudaSuccess) return fail_cuda(ctx, we);
        }
        r = event_decide(ctx, s.L, s.W, &db, p, &s.h.o);
        if (r != CASK_OK) return r;
        cudaError_t ce = launch_value_ranks(s.L, s.h.o.kind, s.h.v_pos, s.h.n_need, s.h.v_base);
        // the rows with a kind other than 0 are the ones whose values are read
        if (ce == cudaSuccess)
            ce = cudaMemcpyAsync(ctx->hstage + s.r0, s.h.o.kind, (size_t)s.tok.back(), cudaMemcpyDeviceToHost, st);
        if (ce == cudaSuccess && sliced) ce = cudaEventRecord(ev_kinds(i), st);
        return ce == cudaSuccess ? CASK_OK : fail_cuda(ctx, ce);
    };

    size_t v_rows_used = 0;
    // the needed value rows packed and sent up, the compaction
    auto compact = [&](size_t i) -> int {
        HostSlice& s = sl[i];
        cudaStream_t st = stream_of(i);
        cudaError_t ce = sliced ? cudaEventSynchronize(ev_kinds(i)) : cudaStreamSynchronize(st);
        if (ce != cudaSuccess) return fail_cuda(ctx, ce);
        const size_t n = (size_t)s.hb.n_units;
        const uint8_t* hkind = (const uint8_t*)ctx->hstage + s.r0;
        s.vbase.assign(n + 1, 0);
        over_units(n, [&](size_t u) {
            const uint8_t* kd = hkind + s.tok[u];
            int64_t c = 0;
            for (int r = 0; r < s.hb.T[u]; ++r) c += kd[r] != CASK_KIND_DROPPED;
            s.vbase[u + 1] = c;
        });
        for (size_t u = 0; u < n; ++u) s.vbase[u + 1] += s.vbase[u];
        s.need_rows = (size_t)s.vbase[n];
        s.v_row0 = v_rows_used;
        if (ctx->hstage_bytes < v_stage0 + (v_rows_used + s.need_rows) * row_bytes) {
            // Grow, keeping the kinds.  Earlier slices may still be reading their packed rows: wait for them first.
            ce = drain();
            if (ce != cudaSuccess) return fail_cuda(ctx, ce);
            char* bigger = nullptr;
            const size_t want = v_rows_used + s.need_rows;
            const size_t nb = v_stage0 + (want + want / 4 + 4096) * row_bytes;
            ce = cudaMallocHost((void**)&bigger, nb);
            if (ce != cudaSuccess) return fail_cuda(ctx, ce);
            memcpy(bigger, ctx->hstage, sumT);
            cudaFreeHost(ctx->hstage);
            ctx->hstage = bigger;
            ctx->hstage_bytes = nb;
            hkind = (const uint8_t*)ctx->hstage + s.r0;
        }
        v_rows_used += s.need_rows;
        char* hv = ctx->hstage + v_stage0 + s.v_row0 * row_bytes;
        over_units(n, [&](size_t u) {
            const uint8_t* kd = hkind + s.tok[u];
            const char* src = (const char*)s.hb.v + (size_t)s.off[u] * es;
            char* dst = hv + (size_t)s.vbase[u] * row_bytes;
            for (int r = 0; r < s.hb.T[u]; ++r)
                if (kd[r] != CASK_KIND_DROPPED) {
                    stage_row(dst, src + (size_t)r * row_bytes, row_bytes);
                    dst += row_bytes;
                }
            stage_fence();
        });
        ce = cudaMemcpyAsync(s.h.v, hv, s.need_rows * row_bytes, cudaMemcpyHostToDevice, up);
        if (ce == cudaSuccess && sliced) ce = cudaEventRecord(ev_values(i), up);
        if (ce == cudaSuccess && sliced) ce = cudaStreamWaitEvent(st, ev_values(i), 0);
        if (ce != cudaSuccess) return fail_cuda(ctx, ce);
        s.L.v = s.h.v;
        s.L.sh.v_pos = s.h.v_pos;
        s.L.sh.v_base = s.h.v_base;
        return event_compact(ctx, s.L, s.W, p, &s.h.o);
    };
    auto results = [&](size_t i) -> int {
        HostSlice& s = sl[i];
        cudaStream_t st = stream_of(i);
        cudaError_t ce = cudaSuccess;
        const size_t n = (size_t)s.hb.n_units, sT = (size_t)s.tok.back();
        struct Cp { void* dst; const void* src; size_t bytes; };
        const cask_outputs &o = s.ho, &g = s.h.o;
        const Cp cps[] = {
            {o.k_out, g.k_out, n * Bm * d * es}, {o.v_out, g.v_out, n * Bm * d * es},
            {o.n_out, g.n_out, n * 4}, {o.slot_src, g.slot_src, n * Bm * 4},
            {o.slot_kind, g.slot_kind, n * Bm}, {o.slot_mass, g.slot_mass, n * Bm * 4},
            {o.assign, g.assign, sT * 4}, {o.weight, g.weight, sT * 4},
            {o.kind, g.kind, sT}, {o.seed_of, g.seed_of, sT * 4},
            {o.plan, g.plan, n * 32}, {o.unit_status, g.unit_status, n * 4},
            {o.lost_mass, g.lost_mass, n * 4}, {o.s, g.s, sT * 4},
            {o.lse, g.lse, n * rows * 4}, {o.sim, g.sim, sT * 4},
            {o.rho_core, g.rho_core, n * 4}, {o.rho_rep, g.rho_rep, n * 4},
            {o.dispersion, g.dispersion, n * 4},
        };
        for (const Cp& c : cps) {
            if (!c.dst) continue;
            ce = cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyDeviceToHost, st);
            if (ce != cudaSuccess) return fail_cuda(ctx, ce);
        }
        // the slice's flag word joins the call's
        ce = cudaMemcpyAsync(&ctx->hs_flags[i], s.W.err, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
        return ce == cudaSuccess ? CASK_OK : fail_cuda(ctx, ce);
    };

    // Order of the host's work for slice i: pack and compact it, decide slice i+1, queue slice i+2's upload, then
    // queue slice i's results.  The descriptor staging of the context serves one slice at a time, so slice i+1 is
    // decided only after slice i's compaction has been queued; the results come last because a copy into pageable
    // memory holds the host until the slice is done, and by then the next upload and decision are already queued.
    if (!ctx->hs_flags) {
        e = cudaMallocHost((void**)&ctx->hs_flags, kMaxSlices * sizeof(int32_t));
        if (e != cudaSuccess) return leave(CASK_OK, e);
    }
    e = slice_upload(sl[0], up);
    if (e != cudaSuccess) return leave(CASK_OK, e);
    rc = decide(0);
    if (rc != CASK_OK) return leave(rc, cudaSuccess);
    if (C > 1) {
        e = slice_upload(sl[1], up);
        if (e != cudaSuccess) return leave(CASK_OK, e);
    }
    for (size_t i = 0; i < C; ++i) {
        rc = compact(i);
        if (rc != CASK_OK) return leave(rc, cudaSuccess);
        if (i + 1 < C) {
            rc = decide(i + 1);
            if (rc != CASK_OK) return leave(rc, cudaSuccess);
        }
        if (i + 2 < C) {
            e = slice_upload(sl[i + 2], up);
            if (e != cudaSuccess) return leave(CASK_OK, e);
        }
        rc = results(i);
        if (rc != CASK_OK) return leave(rc, cudaSuccess);
    }
    rc = leave(CASK_OK, cudaSuccess);
    if (rc != CASK_OK) return rc;
    int32_t flags = 0;
    for (size_t i = 0; i < C; ++i) flags |= ctx->hs_flags[i];
    ctx->flags_dev = nullptr;
    ctx->flags_last = flags;
    return CASK_OK;
}

}  // extern "C"
