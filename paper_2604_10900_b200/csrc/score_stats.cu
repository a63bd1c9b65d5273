// Query-statistics scorer of the Phase-1 archive (App. B): horizon kernel of a discrete horizon distribution and
// the horizon-averaged mean score
//     S_h(k, Delta) = Re sum_f mu_{h,f} conj(k_f) kappa_{pi_h}(omega_f) e^{i omega_f Delta},   s_i = mean_h S_h(k_i, Delta_i).
// The sum over heads is linear, so a first small kernel folds mu and kappa into one complex coefficient per unit and
// band, A_f = (1/g) sum_h mu_{h,f} kappa_{h,f}; the main kernel then needs one pass over the keys:
// s_i = sum_f Re(A_f conj(k_if) e^{i omega_f Delta_i}).  Phases are counted in turns in 64-bit fixed point: omega_f / 2 pi
// as a 0.64 fraction times the integer part of Delta wraps around by itself, so a distance of tens of thousands of
// rows costs no accuracy and no double-precision arithmetic in the inner loop; the fractional part of Delta is added
// in single precision.
#include "cask_internal.cuh"

namespace cask {

namespace {

constexpr double kTwoPi = 6.283185307179586476925286766559;
constexpr int kRowsPerCta = 64;

// Per-band constants shared by all units (global memory, read through the L1): omega / 2 pi in turns and in 0.64 fixed
// point, and e^{i omega} for the row-to-row phase step.
struct BandTable {
    float* om_t;
    float* rot_c;
    float* rot_s;
    unsigned long long* om_fx;
};

// A[u][f] = (1/g) sum_h mu[u][h][f] * kappa[u][h][f],  kappa = sum_n pi[u][h][n] e^{i omega_f delta_n}.
// One CTA per unit; four threads per band, each a quarter of the horizon offsets, combined in a fixed order.
__global__ void __launch_bounds__(256) stats_fold_kernel(int g, int nb, cask_query_stats qs, float* __restrict__ A,
                                                         BandTable tab) {
    const int u = blockIdx.x;
    const int part = threadIdx.x & 3;
    if (u == 0)
        for (int f = threadIdx.x; f < nb; f += blockDim.x) {
            const double turns = (double)qs.omega[f] * (1.0 / kTwoPi);   // whole turns per unit offset drop out of the integer part
            const double fr = turns - floor(turns);
            tab.om_t[f] = (float)turns;
            tab.om_fx[f] = (unsigned long long)(fr * 18446744073709551616.0);
            float sn, cs;
            sincosf((float)(kTwoPi * (fr > 0.5 ? fr - 1.0 : fr)), &sn, &cs);
            tab.rot_c[f] = cs;
            tab.rot_s[f] = sn;
        }
    for (int f0 = 0; f0 < nb; f0 += 64) {
        const int f = f0 + (threadIdx.x >> 2);
        // omega_f / 2 pi in turns (float) and as a 0.64 fixed-point fraction: the phase of an offset is formed from its
        // integer part by two 32-bit multiplies (whole turns wrap away) and from its fractional part in single precision,
        // so the loop below needs no double-precision arithmetic
        const double tr = f < nb ? (double)qs.omega[f] * (1.0 / kTwoPi) : 0.0;
        const double frt = tr - floor(tr);
        const float ot = (float)tr;
        const unsigned long long ofx = (unsigned long long)(frt * 18446744073709551616.0);
        const unsigned fx_hi = (unsigned)(ofx >> 32), fx_lo = (unsigned)ofx;
        float ar = 0.f, ai = 0.f;
        // e^{i omega_f delta_n} does not depend on the head: one sine and cosine per offset serve eight heads at a time
        for (int h0 = 0; h0 < g; h0 += 8) {
            float kr[8], ki[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) { kr[k] = 0.f; ki[k] = 0.f; }
            for (int n = part; n < qs.n_delta; n += 4) {
                float sn, cs;
                const float dv = qs.delta_grid[n], fl = floorf(dv);
                const int di = (int)fl;
                const unsigned dm = (unsigned)abs(di);
                const int hi = (int)(fx_hi * dm + __umulhi(fx_lo, dm));
                const float turns = fmaf((float)hi, di < 0 ? -2.3283064365386963e-10f : 2.3283064365386963e-10f, ot * (dv - fl));
                sincosf(6.2831853071795865f * turns, &sn, &cs);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (h0 + k < g) {
                        const float pv = qs.pi[((size_t)u * g + h0 + k) * qs.n_delta + n];
                        kr[k] = fmaf(pv, cs, kr[k]);
                        ki[k] = fmaf(pv, sn, ki[k]);
                    }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                kr[k] += __shfl_xor_sync(0xffffffffu, kr[k], 1);
                ki[k] += __shfl_xor_sync(0xffffffffu, ki[k], 1);
                kr[k] += __shfl_xor_sync(0xffffffffu, kr[k], 2);
                ki[k] += __shfl_xor_sync(0xffffffffu, ki[k], 2);
                if (f < nb && h0 + k < g) {
                    const float* mu = qs.mu + (((size_t)u * g + h0 + k) * nb + f) * 2;
                    ar += fmaf(mu[0], kr[k], -mu[1] * ki[k]);
                    ai += fmaf(mu[0], ki[k], mu[1] * kr[k]);
                }
            }
        }
        if (part == 0 && f < nb) {
            A[((size_t)u * nb + f) * 2] = ar / (float)g;
            A[((size_t)u * nb + f) * 2 + 1] = ai / (float)g;
        }
    }
}

// One pass over the keys.  A CTA takes a run of up to kTilesPerCta tiles of 64 rows of one unit and streams them
// through a ring of shared-memory stages with 16-byte asynchronous copies (cp.async), so several tiles are in flight
// per CTA while it computes; the data stays in the cache dtype in shared memory.  A thread owns four consecutive rows
// of a tile and a quad of four bands; sixteen threads cover a row.  The quad's constants sit in registers; the row
// sums meet by shuffles.  Without caller-supplied offsets Delta falls by one from a row to the next, so after the
// first of its rows a thread turns the phase by e^{-i omega} (four multiply-adds) instead of forming it anew.
constexpr int kTilesPerCta = 8;

template <typename T> struct Quad;       // four consecutive elements of a row as floats
template <> struct Quad<__nv_bfloat16> {
    static __device__ __forceinline__ void ld(const __nv_bfloat16* p, float (&x)[4]) {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
    }
};
template <> struct Quad<float> {
    static __device__ __forceinline__ void ld(const float* p, float (&x)[4]) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
};

template <typename T, bool STEP, int LAYOUT>      // STEP: no caller-supplied offsets, Delta falls by one per row
__global__ void __launch_bounds__(256) score_stats_kernel(const UnitDesc* __restrict__ desc, Shape sh, const T* __restrict__ K,
                                                             cask_query_stats qs, const float* __restrict__ A, BandTable tab,
                                                             int n_stages, float* __restrict__ s) {
    extern __shared__ __align__(16) uint8_t ring[];
    const int u = blockIdx.y;
    const UnitDesc& ud = desc[u];
    const int first_row = blockIdx.x * kTilesPerCta * kRowsPerCta;
    // descriptor fields in registers: the asynchronous copies below are memory barriers to the compiler, which
    // would otherwise read them again after every one
    const int T_u = ud.T;
    const int64_t tok_u = ud.tok_off, koff_u = ud.k_off;
    if (first_row >= T_u) return;
    const int d = sh.d, nb = d / 2, nq = nb / 4;
    const int n_tiles = min(kTilesPerCta, (T_u - first_row + kRowsPerCta - 1) / kRowsPerCta);
    constexpr int kPer = 16 / (int)sizeof(T);                 // elements per 16-byte vector
    const int vec_per_row = d / kPer;
    const size_t stage_elems = (size_t)kRowsPerCta * d;
    T* stages = reinterpret_cast<T*>(ring);
    auto issue = [&](int k) {                                  // tile k of this CTA into stage k % n_stages
        if (k < n_tiles) {
            const int row0 = first_row + k * kRowsPerCta, nrows = min(kRowsPerCta, T_u - row0);
            T* dst = stages + (size_t)(k % n_stages) * stage_elems;
            if (sh.page_size == 0 && sh.row_stride == d) {
                // rows back to back in the cache: the tile is one contiguous run of 16-byte vectors
                const T* src = K + koff_u + (int64_t)row0 * d;
                const unsigned sa0 = (unsigned)__cvta_generic_to_shared(dst);
                for (int v = threadIdx.x; v < nrows * vec_per_row; v += blockDim.x)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa0 + 16u * v), "l"(src + (size_t)v * kPer) : "memory");
            } else {
                for (int v = threadIdx.x; v < nrows * vec_per_row; v += blockDim.x) {
                    const int rr = v / vec_per_row, c = (v - rr * vec_per_row) * kPer;
                    const T* src = K + row_elem_off(sh, ud, ud.k_off, row0 + rr) + c;
                    const unsigned sa = (unsigned)__cvta_generic_to_shared(dst + (size_t)rr * d + c);
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(src) : "memory");
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    for (int k = 0; k < n_stages - 1; ++k) issue(k);

    const int q = threadIdx.x & 15, rg = threadIdx.x >> 4;       // band quad (and its multiples of 16), row group
    const int r_first = 4 * rg;
    // constants of a quad: coefficient A, omega in turns (float and the two halves of the 0.64 fixed-point value),
    // e^{i omega}
    struct QuadConst { float ar[4], ai[4], ot[4], rc[4], rs[4]; unsigned fx_hi[4], fx_lo[4]; };
    auto load_const = [&](int qq, QuadConst& c) {
        const float4 ot4 = *reinterpret_cast<const float4*>(tab.om_t + 4 * qq);
        const float4 rc4 = *reinterpret_cast<const float4*>(tab.rot_c + 4 * qq), rs4 = *reinterpret_cast<const float4*>(tab.rot_s + 4 * qq);
        const float4 a01 = *reinterpret_cast<const float4*>(A + ((size_t)u * nb + 4 * qq) * 2);
        const float4 a23 = *reinterpret_cast<const float4*>(A + ((size_t)u * nb + 4 * qq) * 2 + 4);
        c.ar[0] = a01.x; c.ar[1] = a01.z; c.ar[2] = a23.x; c.ar[3] = a23.z;
        c.ai[0] = a01.y; c.ai[1] = a01.w; c.ai[2] = a23.y; c.ai[3] = a23.w;
        c.ot[0] = ot4.x; c.ot[1] = ot4.y; c.ot[2] = ot4.z; c.ot[3] = ot4.w;
        c.rc[0] = rc4.x; c.rc[1] = rc4.y; c.rc[2] = rc4.z; c.rc[3] = rc4.w;
        c.rs[0] = rs4.x; c.rs[1] = rs4.y; c.rs[2] = rs4.z; c.rs[3] = rs4.w;
#pragma unroll
        for (int b4 = 0; b4 < 4; ++b4) {
            const unsigned long long fx = tab.om_fx[4 * qq + b4];
            c.fx_hi[b4] = (unsigned)(fx >> 32);
            c.fx_lo[b4] = (unsigned)fx;
        }
    };
    const bool one_quad = nq <= 16;          // head_dim <= 128: a thread has at most one quad, its constants load once
    QuadConst c0 = {};
    if (one_quad && q < nq) load_const(q, c0);
    for (int k = 0; k < n_tiles; ++k) {
        issue(k + n_stages - 1);
        // all but the newest n_stages - 1 groups have landed: tile k is in shared memory
        if (n_stages == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
        else if (n_stages == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        const int row0 = first_row + k * kRowsPerCta, nrows = min(kRowsPerCta, T_u - row0);
        const T* tile = stages + (size_t)(k % n_stages) * stage_elems;
        // offsets of this thread's rows: magnitude of the integer part, its sign, the fractional part
        unsigned Dm[4];
        float Dsg[4], Df[4];
        int rloc[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            rloc[j] = min(r_first + j, nrows - 1);                // rows past the end repeat the last one; not stored
            const int i = row0 + rloc[j];
            int Di = T_u - 1 - i;
            Df[j] = 0.f;
            if (!STEP) {
                const float dv = qs.delta[tok_u + i], fl = floorf(dv);
                Di = (int)fl;
                Df[j] = dv - fl;
            }
            Dm[j] = (unsigned)abs(Di);
            Dsg[j] = Di < 0 ? -2.3283064365386963e-10f : 2.3283064365386963e-10f;      // +-2^-32
        }
        // Without caller offsets Delta falls by exactly one per row: rows 1..3 turn the phase of row 0.  (Rows past
        // the end of the unit get a phase that means nothing; they are not stored.)
        constexpr bool rotate = STEP;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int qq = q; qq < nq; qq += 16) {
            QuadConst c = c0;
            if (!one_quad) load_const(qq, c);
            float cs[4], sn[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const T* row = tile + (size_t)rloc[j] * d;
                float kx[4], ky[4];
                if (LAYOUT == 0) {
                    Quad<T>::ld(row + 4 * qq, kx);
                    Quad<T>::ld(row + nb + 4 * qq, ky);
                } else {
                    float v0[4], v1[4];
                    Quad<T>::ld(row + 8 * qq, v0);
                    Quad<T>::ld(row + 8 * qq + 4, v1);
                    kx[0] = v0[0]; ky[0] = v0[1]; kx[1] = v0[2]; ky[1] = v0[3];
                    kx[2] = v1[0]; ky[2] = v1[1]; kx[3] = v1[2]; ky[3] = v1[3];
                }
#pragma unroll
                for (int b4 = 0; b4 < 4; ++b4) {
                    if (j == 0 || !rotate) {
                        // frac(omega / 2 pi * |Di|) as a signed 32-bit fraction of a turn (the 64-bit product modulo one
                        // turn from two 32-bit multiplies), signed by Di, plus the fractional offset's share
                        const int hi = (int)(c.fx_hi[b4] * Dm[j] + __umulhi(c.fx_lo[b4], Dm[j]));
                        const float turns = fmaf((float)hi, Dsg[j], c.ot[b4] * Df[j]);
                        __sincosf(6.2831853071795865f * turns, &sn[b4], &cs[b4]);
                    } else {
                        const float c2 = fmaf(cs[b4], c.rc[b4], sn[b4] * c.rs[b4]);      // (c + i s) e^{-i omega}
                        sn[b4] = fmaf(sn[b4], c.rc[b4], -cs[b4] * c.rs[b4]);
                        cs[b4] = c2;
                    }
                    // conj(k) e^{i theta} = (kx cs + ky sn) + i (kx sn - ky cs)
                    const float wr = fmaf(kx[b4], cs[b4], ky[b4] * sn[b4]), wi = fmaf(kx[b4], sn[b4], -ky[b4] * cs[b4]);
                    acc[j] += fmaf(c.ar[b4], wr, -c.ai[b4] * wi);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int off = 1; off < 16; off <<= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], off);
            if (q == 0 && r_first + j < nrows) s[tok_u + row0 + r_first + j] = acc[j];
        }
        __syncthreads();            // the stage is free for the tile issued at the top of the next round
    }
}

}  // namespace

cudaError_t launch_score_stats(const Launch& L, const cask_query_stats& qs, float* s, Workspace& ws) {
    const Shape& sh = L.sh;
    const int nb = sh.d / 2;
    // the table of per-band constants sits behind the per-unit coefficients in the same workspace array
    float* tbase = ws.stats_a + (size_t)sh.n_units * sh.d;
    BandTable tab{tbase, tbase + nb, tbase + 2 * nb, reinterpret_cast<unsigned long long*>(tbase + 4 * nb)};
    {
        Timed t(L, KID_ROW_COMBINE);
        stats_fold_kernel<<<sh.n_units, 256, 0, L.stream>>>(sh.g, nb, qs, ws.stats_a, tab);
    }
    const size_t stage_bytes = (size_t)kRowsPerCta * sh.d * (sh.dtype == CASK_DTYPE_BF16 ? 2 : 4);
    const int n_stages = (int)std::max<size_t>(1, std::min<size_t>(3, (96 * 1024) / stage_bytes));
    const size_t smem = n_stages * stage_bytes;
    const int rows_per_cta = kTilesPerCta * kRowsPerCta;
    const dim3 grid((L.max_T + rows_per_cta - 1) / rows_per_cta, sh.n_units);
    Timed t(L, KID_SCORE_MASS);
    auto launch = [&](auto kern, const auto* kptr) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, 256, smem, L.stream>>>(L.desc, sh, kptr, qs, ws.stats_a, tab, n_stages, s);
        return cudaSuccess;
    };
    const bool step = qs.delta == nullptr;
    cudaError_t e;
    if (sh.dtype == CASK_DTYPE_BF16) {
        const __nv_bfloat16* kp = (const __nv_bfloat16*)L.k;
        if (qs.band_layout == 0) e = step ? launch(score_stats_kernel<__nv_bfloat16, true, 0>, kp) : launch(score_stats_kernel<__nv_bfloat16, false, 0>, kp);
        else e = step ? launch(score_stats_kernel<__nv_bfloat16, true, 1>, kp) : launch(score_stats_kernel<__nv_bfloat16, false, 1>, kp);
    } else {
        const float* kp = (const float*)L.k;
        if (qs.band_layout == 0) e = step ? launch(score_stats_kernel<float, true, 0>, kp) : launch(score_stats_kernel<float, false, 0>, kp);
        else e = step ? launch(score_stats_kernel<float, true, 1>, kp) : launch(score_stats_kernel<float, false, 1>, kp);
    }
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace cask
