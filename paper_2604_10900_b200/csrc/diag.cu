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

// Within-group dispersion (Sec. 2.6, first term of the bound): sum_i a_i ||k_i - k~_G|| over the rows of kind 4/5, k~_G
// read back from k_out.  One CTA per unit, one warp per member row in turn; a lane takes the bands lane, lane + 32, ...
// (both channels of a band, so the per-band norm needs no exchange); fixed-order double-precision sums.
template <typename T>
__global__ void __launch_bounds__(256) dispersion_kernel(
    const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K, const float* __restrict__ s, float eps,
    const uint8_t* __restrict__ kind, const int32_t* __restrict__ assign, const T* __restrict__ k_out, int Bmax,
    float* __restrict__ dispersion) {
    __shared__ double red[8];
    const int u = blockIdx.x;
    const UnitDesc& ud = desc[u];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int nb = sh.d / 2;
    const int second = (sh.band_w && sh.band_layout == 1) ? 1 : nb, step = (sh.band_w && sh.band_layout == 1) ? 2 : 1;
    double acc = 0.0;
    for (int i = w; i < ud.T; i += nw) {
        const uint8_t kd = kind[ud.tok_off + i];
        if (kd != CASK_KIND_SEED && kd != CASK_KIND_MERGED) continue;      // the same for the whole warp
        const int slot = assign[ud.tok_off + i];
        if (slot < 0 || slot >= Bmax) continue;
        const T* kr = K + row_elem_off(sh, ud, ud.k_off, i);
        const T* rep = k_out + ((size_t)u * Bmax + slot) * sh.d;
        float part = 0.f;
        for (int f = lane; f < nb; f += 32) {
            const int c0 = f * step, c1 = c0 + second;
            const float dx = Elem<T>::ld(kr + c0) - Elem<T>::ld(rep + c0), dy = Elem<T>::ld(kr + c1) - Elem<T>::ld(rep + c1);
            if (sh.band_w) part = fmaf(sh.band_w[f], sqrtf(fmaf(dx, dx, dy * dy)), part);
            else if (sh.chan_w) part = fmaf(sh.chan_w[c0] * dx, dx, fmaf(sh.chan_w[c1] * dy, dy, part));
            else part = fmaf(dx, dx, fmaf(dy, dy, part));
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        const float norm = sh.band_w ? part : sqrtf(part);
        acc += (double)row_mass(sh, s, eps, ud.tok_off + i) * (double)norm;
    }
    if (lane == 0) red[w] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int x = 0; x < nw; ++x) t += red[x];
        dispersion[u] = (float)t;
    }
}

}  // namespace

cudaError_t launch_diagnostics(const Launch& L, const cask_params& prm, const float* s, const uint8_t* kind,
                               const cask_outputs& out) {
    if (out.rho_core || out.rho_rep) {
        Timed t(L, KID_DIAGNOSTICS);
        diagnostics_kernel<<<L.sh.n_units, kSelThreads, 0, L.stream>>>(L.desc, s, kind, out.slot_mass, out.n_out,
                                                                      out.Bmax, out.rho_core, out.rho_rep);
    }
    if (out.dispersion) {
        Timed t(L, KID_DIAGNOSTICS);
        if (L.sh.dtype == CASK_DTYPE_BF16)
            dispersion_kernel<__nv_bfloat16><<<L.sh.n_units, 256, 0, L.stream>>>(
                L.desc, L.sh, (const __nv_bfloat16*)L.k, s, prm.eps, kind, out.assign, (const __nv_bfloat16*)out.k_out,
                out.Bmax, out.dispersion);
        else
            dispersion_kernel<float><<<L.sh.n_units, 256, 0, L.stream>>>(L.desc, L.sh, (const float*)L.k, s, prm.eps, kind,
                                                                        out.assign, (const float*)out.k_out, out.Bmax,
                                                                        out.dispersion);
    }
    return cudaGetLastError();
}

}  // namespace cask
