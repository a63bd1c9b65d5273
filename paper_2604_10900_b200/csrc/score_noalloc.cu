// cask_score_noalloc: the scoring step for callers that cannot allocate.
//
// Some hosts of this library may not call cudaMalloc at the point where they need a score pass:
// code running inside an inference engine that has handed all device memory to its own pool, a
// plugin loaded after the memory budget was frozen, or a caller inside a region where allocation
// is forbidden.  Everything cask_score takes from the caller's workspace (unit descriptors, the
// per-chunk normaliser partials, the per-row offset/weight tables) lives here in one fixed array
// in device global memory instead.  The array is part of the library image: every GPU that loads
// the library holds CASK_NOALLOC_SCRATCH_BYTES until the process exits.
//
// The kernels are the SIMT scoring kernels of score_simt.cu, unchanged; only the origin of their
// scratch differs.  No cudaMalloc / cudaFree / cudaMallocHost / event or stream creation happens
// in this file, and nothing from torch is involved.
#include <mutex>

#include "cask_internal.cuh"

namespace cask {
int check_batch_host(const cask_batch* b, const cask_params* p);   // api.cu
}

using namespace cask;

namespace {

constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; the
// kernels are given the address that call returns.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CASK_NOALLOC_SCRATCH_BYTES];

std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// Makes `device` current for the duration of a call and puts the caller's device back on every way out.
struct DeviceGuard {
    int prev = -1;
    bool enter(int device) {
        if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; return false; }
        if (prev == device) { prev = -1; return true; }
        return cudaSetDevice(device) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" int cask_score_noalloc(int device, void* cuda_stream, const cask_batch* b, const cask_params* p,
                                  float* s, float* lse_out) {
    if (!s) return CASK_ERR_NULL;
    int rc = check_batch_host(b, p);
    if (rc != CASK_OK) return rc;
    if (b->page_size != 0) return CASK_ERR_UNSUPPORTED;     // contiguous caches only
    if (b->n_units == 0) return CASK_OK;
    if (device < 0 || device >= kMaxDevices) return CASK_ERR_SHAPE;
    if (b->n_units > CASK_NOALLOC_MAX_UNITS) return CASK_ERR_TOO_LARGE;

    // layout of the fixed array for this batch
    const size_t rows = (size_t)b->group * b->window, n = (size_t)b->n_units;
    size_t total_chunks = 0;
    int max_chunks = 0, max_T = 0;
    for (int u = 0; u < b->n_units; ++u) {
        const int nch = (b->T[u] + kChunkKeys - 1) / kChunkKeys;
        total_chunks += (size_t)nch;
        max_chunks = nch > max_chunks ? nch : max_chunks;
        max_T = b->T[u] > max_T ? b->T[u] : max_T;
    }
    const size_t off_desc = 0;
    const size_t off_rowm = off_desc + up256(sizeof(UnitDesc) * CASK_NOALLOC_MAX_UNITS);
    const size_t off_roww = off_rowm + up256(n * rows * 4);
    const size_t off_pm = off_roww + up256(n * rows * 4);
    const size_t off_pl = off_pm + up256(total_chunks * rows * 4);
    const size_t need = off_pl + up256(total_chunks * rows * 4);
    if (need > (size_t)CASK_NOALLOC_SCRATCH_BYTES) return CASK_ERR_TOO_LARGE;

    // The calling thread keeps the current device it came with.
    DeviceGuard guard;
    if (!guard.enter(device)) return CASK_ERR_CUDA;
    // A stream that is being captured is refused: the descriptor upload below reads a host array that is gone
    // when this call returns, so a recorded copy of it could never be replayed.
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    cudaError_t e = cudaStreamIsCapturing(st, &cap);
    if (e != cudaSuccess) return CASK_ERR_CUDA;
    if (cap != cudaStreamCaptureStatusNone) return CASK_ERR_UNSUPPORTED;
    unsigned char* base = nullptr;
    {
        // first call on this device: resolve the array's device address (once per device, with that
        // device current)
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_addr[device]) {
            void* ptr = nullptr;
            e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
            if (e != cudaSuccess || !ptr) return CASK_ERR_CUDA;
            g_scratch_addr[device] = ptr;
        }
        base = (unsigned char*)g_scratch_addr[device];
    }

    UnitDesc hd[CASK_NOALLOC_MAX_UNITS];
    int chunk0 = 0;
    const int64_t q_unit = (int64_t)b->group * b->window * b->head_dim;
    for (int u = 0; u < b->n_units; ++u) {
        UnitDesc& d = hd[u];
        d = UnitDesc{};
        d.k_off = b->k_off[u];
        d.v_off = b->v_off[u];
        d.q_off = q_unit * u;
        d.tok_off = b->tok_off[u];
        d.T = b->T[u]; d.P = b->P[u]; d.B = b->B[u]; d.reserve = b->reserve[u];
        d.chunk0 = chunk0;
        d.n_chunks = (d.T + kChunkKeys - 1) / kChunkKeys;
        chunk0 += d.n_chunks;
    }
    // pageable source: the runtime has taken its copy of hd[] when this returns
    e = cudaMemcpyAsync(base + off_desc, hd, sizeof(UnitDesc) * n, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return CASK_ERR_CUDA;

    int64_t launches = 0;
    Launch L{};
    L.stream = st;
    L.sh.n_units = b->n_units; L.sh.d = b->head_dim; L.sh.g = b->group; L.sh.W = b->window;
    L.sh.rows = (int)rows; L.sh.dtype = b->dtype; L.sh.row_stride = b->row_stride; L.sh.causal = p->causal;
    L.desc = (const UnitDesc*)(base + off_desc);
    L.hdesc = hd;
    L.k = b->k; L.v = b->v; L.q = b->q;
    L.max_T = max_T; L.max_chunks = max_chunks; L.total_chunks = (int)total_chunks;
    L.sum_T = b->tok_off[b->n_units];
    L.launches = &launches;
    L.prof = nullptr;
    Workspace W{};
    W.desc = (UnitDesc*)(base + off_desc);
    W.rowm = (float*)(base + off_rowm);
    W.roww = (float*)(base + off_roww);
    W.part_m = (float*)(base + off_pm);
    W.part_l = (float*)(base + off_pl);
    // Nothing in the array has to start at zero: every word a kernel of this call reads (descriptors,
    // partials, row tables) is written earlier in the same call, so the contents left by the previous
    // call are never observed.
    e = launch_score_simt(L, b->lse_in, s, lse_out, W);
    return e == cudaSuccess ? CASK_OK : CASK_ERR_CUDA;
}
