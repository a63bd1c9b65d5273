// Representative-set mass diagnostics (Sec. 2.6): per unit
//   rho_core = sum_{k in C} s_k / sum_{k in TopB} s_k,   rho_rep = (mass carried by the output slots) / same,
// with TopB the B greatest rows of the whole cache under the score of this event, C = recent + core rows.
// One CTA per unit: the B-th greatest score by the same radix narrowing as the selections, then fixed-order
// double-precision sums.
#include "select.cuh"

namespace cask {

namespace {

// Key of the k-th greatest score of rows [lo,hi) (every row counts) and how many rows equal to it fall inside
// the top k.  1 <= k <= hi - lo.
__device__ inline void block_kth_key(const float* __restrict__ s, int lo, int hi, int k, SelectSmem& sm, unsigned& thr,
                                     unsigned& krem) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    unsigned prefix = 0, rem = (unsigned)k;
    for (int pass = 0; pass < 3; ++pass) {
        const int bits = pass == 2 ? 8 : 12, shift = pass == 0 ? 20 : (pass == 1 ? 8 : 0);
        const int nbins = 1 << bits;
        for (int b = tid; b < nbins; b += nthr) sm.hist[b] = 0;
        __syncthreads();
        for (int i = lo + tid; i < hi; i += nthr) {
            const unsigned key = order_key(s[i]);
            const bool match = pass == 0 || (key >> (shift + bits)) == prefix;
            if (match) atomicAdd(&sm.hist[(key >> shift) & (unsigned)(nbins - 1)], 1u);
        }
        __syncthreads();
        find_digit(sm, nbins, rem);
        prefix = (prefix << bits) | sm.digit;
        rem = sm.krem;
        __syncthreads();
    }
    thr = prefix;
    krem = rem;
}

__device__ __forceinline__ float key_to_float(unsigned key) {
    return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}

__device__ inline double block_sum_f64(double v, double* red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    double t = 0.0;
    for (int x = 0; x < (int)(blockDim.x >> 5); ++x) t += red[x];
    return t;
}

__global__ void __launch_bounds__(kSelThreads) diagnostics_kernel(
    const UnitDesc* __restrict__ desc, const float* __restrict__ s, const uint8_t* __restrict__ kind,
    const float* __restrict__ slot_mass, const int32_t* __restrict__ n_out, int Bmax, float* __restrict__ rho_core,
    float* __restrict__ rho_rep) {
    __shared__ SelectSmem sm;
    __shared__ double red[kSelThreads / 32];
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int T = ud.T;
    const float* su = s + ud.tok_off;
    const uint8_t* kd = kind + ud.tok_off;
    const int k = min(ud.B, T);
    unsigned thr, krem;
    block_kth_key(su, 0, T, k, sm, thr, krem);
    double top = 0.0, core = 0.0, rep = 0.0;
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        const float x = su[i];
        if (order_key(x) > thr) top += (double)x;
        if (kd[i] == CASK_KIND_RECENT || kd[i] == CASK_KIND_CORE) core += (double)x;
    }
    const int n = n_out[u];
    for (int t = threadIdx.x; t < n; t += blockDim.x) rep += (double)slot_mass[(size_t)u * Bmax + t];
    top = block_sum_f64(top, red) + (double)krem * (double)key_to_float(thr);
    core = block_sum_f64(core, red);
    rep = block_sum_f64(rep, red);
    if (threadIdx.x == 0) {
        if (rho_core) rho_core[u] = top > 0.0 ? (float)(core / top) : 0.f;
        if (rho_rep) rho_rep[u] = top > 0.0 ? (float)(rep / top) : 0.f;
    }
}

}  // namespace

cudaError_t launch_diagnostics(const Launch& L, const float* s, const uint8_t* kind, const cask_outputs& out) {
    if (!out.rho_core && !out.rho_rep) return cudaSuccess;
    Timed t(L, KID_DIAGNOSTICS);
    diagnostics_kernel<<<L.sh.n_units, kSelThreads, 0, L.stream>>>(L.desc, s, kind, out.slot_mass, out.n_out, out.Bmax,
                                                                  out.rho_core, out.rho_rep);
    return cudaGetLastError();
}

}  // namespace cask
