// Query-statistics scorer of the Phase-1 archive (App. B): horizon kernel of a discrete horizon distribution and
// the horizon-averaged mean score
//     S_h(k, Delta) = Re sum_f mu_{h,f} conj(k_f) kappa_{pi_h}(omega_f) e^{i omega_f Delta},   s_i = mean_h S_h(k_i, Delta_i).
// The sum over heads is linear, so a first small kernel folds mu and kappa into one complex coefficient per unit and
// band, A_f = (1/g) sum_h mu_{h,f} kappa_{h,f}; the main kernel then needs one pass over the keys:
// s_i = sum_f Re(A_f conj(k_if) e^{i omega_f Delta_i}).  Phases are counted in turns in 64-bit fixed point: omega_f / 2 pi
// as a 0.64 fraction times the integer part of Delta wraps around by itself, so a distance of tens of thousands of
// rows costs no accuracy and no double-precision arithmetic in the inner loop; the fractional part of Delta is added
// in single precision.
#include "tc_common.cuh"

namespace cask {

namespace {

using tc::pack2;
using tc::unpack2;
using tc::fma2;

constexpr double kTwoPi = 6.283185307179586476925286766559;
constexpr int kRowsPerCta = 64;

// Per-band constants shared by all units (global memory, read through the L1): omega / 2 pi in turns and in 0.64 fixed
// point, e^{i omega} for the row-to-row phase step and e^{i 64 omega} for the step from a tile to the next.
struct BandTable {
    float* om_t;
    float* rot_c;
    float* rot_s;
    float* r64_c;
    float* r64_s;
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
            const double t64 = fr * (double)kRowsPerCta, f64 = t64 - floor(t64);
            sincosf((float)(kTwoPi * (f64 > 0.5 ? f64 - 1.0 : f64)), &sn, &cs);
            tab.r64_c[f] = cs;
            tab.r64_s[f] = sn;
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
// through a ring of shared-memory stages, so several tiles are in flight per CTA while it computes; the data stays in
// the cache dtype in shared memory.  A thread owns four consecutive rows of a tile and a quad of four bands; sixteen
// threads cover a row and the row sums meet by shuffles.
// With caller-supplied offsets every (row, band) pair gets its own sine and cosine.  Without them Delta falls by one
// from a row to the next and by 64 from a tile to the next, and the thread keeps the whole factor A e^{i omega Delta} of
// its sixteen pairs in registers, turned by e^{-i 64 omega} once per tile (head_dim <= 128; larger heads form the
// first row's phase per tile and turn it by e^{-i omega} from row to row).
constexpr int kTilesPerCta = 16;

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

// The real parts (kx) and imaginary parts (ky) of a quad of bands as two packed pairs each, straight from shared
// memory: a bf16 pair becomes a packed fp32 pair by one shift and one mask into the two halves of a 64-bit register.
__device__ __forceinline__ uint64_t widen_pair(unsigned w) {            // (lo, hi) halves of w as two floats
    uint64_t r;
    asm("{\n\t.reg .b32 lo, hi;\n\tshl.b32 lo, %1, 16;\n\tand.b32 hi, %1, 0xffff0000;\n\tmov.b64 %0, {lo, hi};\n\t}" : "=l"(r) : "r"(w));
    return r;
}
__device__ __forceinline__ uint64_t widen_lows(unsigned w0, unsigned w1) {      // low halves of w0 and w1
    uint64_t r;
    asm("{\n\t.reg .b32 a, b;\n\tshl.b32 a, %1, 16;\n\tshl.b32 b, %2, 16;\n\tmov.b64 %0, {a, b};\n\t}" : "=l"(r) : "r"(w0), "r"(w1));
    return r;
}
__device__ __forceinline__ uint64_t widen_highs(unsigned w0, unsigned w1) {     // high halves of w0 and w1
    uint64_t r;
    asm("{\n\t.reg .b32 a, b;\n\tand.b32 a, %1, 0xffff0000;\n\tand.b32 b, %2, 0xffff0000;\n\tmov.b64 %0, {a, b};\n\t}" : "=l"(r) : "r"(w0), "r"(w1));
    return r;
}
template <typename T, int LAYOUT> struct QuadPairs;
template <int LAYOUT> struct QuadPairs<__nv_bfloat16, LAYOUT> {
    static __device__ __forceinline__ void ld(const __nv_bfloat16* row, int nb, int q, uint64_t (&kx)[2], uint64_t (&ky)[2]) {
        if (LAYOUT == 0) {
            const uint2 x = *reinterpret_cast<const uint2*>(row + 4 * q), y = *reinterpret_cast<const uint2*>(row + nb + 4 * q);
            kx[0] = widen_pair(x.x); kx[1] = widen_pair(x.y);
            ky[0] = widen_pair(y.x); ky[1] = widen_pair(y.y);
        } else {
            const uint4 v = *reinterpret_cast<const uint4*>(row + 8 * q);      // (x0 y0)(x1 y1)(x2 y2)(x3 y3)
            kx[0] = widen_lows(v.x, v.y); kx[1] = widen_lows(v.z, v.w);
            ky[0] = widen_highs(v.x, v.y); ky[1] = widen_highs(v.z, v.w);
        }
    }
};
template <int LAYOUT> struct QuadPairs<float, LAYOUT> {
    static __device__ __forceinline__ void ld(const float* row, int nb, int q, uint64_t (&kx)[2], uint64_t (&ky)[2]) {
        if (LAYOUT == 0) {
            const float4 x = *reinterpret_cast<const float4*>(row + 4 * q), y = *reinterpret_cast<const float4*>(row + nb + 4 * q);
            kx[0] = pack2(x.x, x.y); kx[1] = pack2(x.z, x.w);
            ky[0] = pack2(y.x, y.y); ky[1] = pack2(y.z, y.w);
        } else {
            const float4 a = *reinterpret_cast<const float4*>(row + 8 * q), b = *reinterpret_cast<const float4*>(row + 8 * q + 4);
            kx[0] = pack2(a.x, a.z); kx[1] = pack2(b.x, b.z);
            ky[0] = pack2(a.y, a.w); ky[1] = pack2(b.y, b.w);
        }
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
    // Stages are used in turn; the positions are counted along (a remainder by the run-time number of stages in every
    // round costs a division sequence per thread).
    int f_stage = 0;                                           // stage of the next tile to be requested
    auto issue = [&](int k) {                                  // tile k of this CTA into the next stage
        if (k < n_tiles) {
            const int row0 = first_row + k * kRowsPerCta, nrows = min(kRowsPerCta, T_u - row0);
            T* dst = stages + (size_t)f_stage * stage_elems;
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
    // Rows back to back in the cache: a tile is one run of bytes, fetched by one bulk copy that one thread
    // issues and a barrier of the stage reports (no per-thread copy instructions, one CTA-wide barrier less
    // per tile).  Any other layout goes through the per-thread 16-byte copies.
    __shared__ uint64_t full_bar[3];
    __shared__ int gave_up;
    const bool bulk = sh.page_size == 0 && sh.row_stride == d;
    if (bulk) {
        if (threadIdx.x == 0) {
            for (int i = 0; i < 3; ++i) tc::mbar_init(&full_bar[i], 1);
            gave_up = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
    }
    auto fetch = [&](int k) {
        if (!bulk) issue(k);
        else if (threadIdx.x == 0 && k < n_tiles) {
            const int row0 = first_row + k * kRowsPerCta, nrows = min(kRowsPerCta, T_u - row0);
            const uint32_t bytes = (uint32_t)nrows * (uint32_t)d * (uint32_t)sizeof(T);
            uint64_t* bar = &full_bar[f_stage];
            tc::mbar_expect_tx(bar, bytes);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(tc::smem_u32(stages + (size_t)f_stage * stage_elems)),
                           "l"(K + koff_u + (int64_t)row0 * d), "r"(bytes), "r"(tc::smem_u32(bar)) : "memory");
        }
        if (++f_stage == n_stages) f_stage = 0;
    };
    // Tile k is in shared memory for every thread of the CTA; false when the bounded wait ran out.
    int c_stage = 0;                      // stage of the tile being consumed and the parity of its barrier phase
    uint32_t c_phase = 0;
    auto landed = [&](int k) -> bool {
        if (bulk) {
            if (!tc::mbar_wait(&full_bar[c_stage], c_phase, &gave_up)) {
                // The wait ran out (about a second).  Copies already started may still land in this CTA's shared
                // memory: the issuing thread gives their barriers a bounded chance before it leaves.
                if (threadIdx.x == 0) {
                    for (int kk = k; kk < min(n_tiles, k + n_stages); ++kk)
                        for (uint32_t it = 0; it < 4096 && !tc::mbar_try(&full_bar[kk % n_stages], (uint32_t)(kk / n_stages) & 1u); ++it) {}
                    atomicOr(sh.err, CASK_ST_TIMEOUT);
                }
                return false;
            }
        } else {
            // all but the newest n_stages - 1 groups have landed
            if (n_stages == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
            else if (n_stages == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
            else asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();
        }
        return true;
    };
    // The four row sums meet over the sixteen lanes of a row group: the first two exchanges halve what a
    // lane carries (a lane keeps the rows whose index bit matches its own), the last two add the rest;
    // lane l of the group ends with the whole sum of row r_first + (l & 3) in its bit-reversed order.
    auto reduce_store = [&](const float (&acc)[4], int row0, int nrows) {
        const bool up1 = (q & 1) != 0;
        const float give0 = up1 ? acc[0] : acc[1], give1 = up1 ? acc[2] : acc[3];
        const float keep0 = up1 ? acc[1] : acc[0], keep1 = up1 ? acc[3] : acc[2];
        const float h0 = keep0 + __shfl_xor_sync(0xffffffffu, give0, 1);       // rows (0|1), (2|3) by bit 0
        const float h1 = keep1 + __shfl_xor_sync(0xffffffffu, give1, 1);
        const bool up2 = (q & 2) != 0;
        float t = (up2 ? h1 : h0) + __shfl_xor_sync(0xffffffffu, up2 ? h0 : h1, 2);
        t += __shfl_xor_sync(0xffffffffu, t, 4);
        t += __shfl_xor_sync(0xffffffffu, t, 8);
        const int jr = (q & 1) + 2 * ((q >> 1) & 1);                          // the row this lane holds
        if (q < 4 && r_first + jr < nrows) s[tok_u + row0 + r_first + jr] = t;
    };
    if constexpr (STEP) {
        if (one_quad) {
            // Delta falls by one per row and by 64 per tile, so the whole factor G = A e^{i omega Delta} of each of the
            // thread's sixteen (row, band) pairs lives in registers: formed once per CTA (one sine and cosine per
            // band for the first row, the other rows by turning it by e^{-i omega}), turned by e^{-i 64 omega} from
            // tile to tile, and a row's score is sum_f Gr kx + Gi ky.  Two bands per instruction (packed fp32).
            const bool active = q < nq;
            uint64_t Gr[4][2], Gi[4][2], Rc[2], Rs[2], Rn[2];
            {
                float gr[4][4], gi[4][4];
#pragma unroll
                for (int b4 = 0; b4 < 4; ++b4) {
                    const int Di = T_u - 1 - (first_row + r_first);       // negative only for rows past the end, never stored
                    const unsigned dm = (unsigned)abs(Di);
                    const int hi = (int)(c0.fx_hi[b4] * dm + __umulhi(c0.fx_lo[b4], dm));
                    float sn, cs;
                    __sincosf(6.2831853071795865f * ((float)hi * (Di < 0 ? -2.3283064365386963e-10f : 2.3283064365386963e-10f)), &sn, &cs);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (j > 0) {
                            const float c2 = fmaf(cs, c0.rc[b4], sn * c0.rs[b4]);      // (c + i s) e^{-i omega}
                            sn = fmaf(sn, c0.rc[b4], -cs * c0.rs[b4]);
                            cs = c2;
                        }
                        gr[j][b4] = fmaf(c0.ar[b4], cs, -c0.ai[b4] * sn);              // A e^{i theta}
                        gi[j][b4] = fmaf(c0.ar[b4], sn, c0.ai[b4] * cs);
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int pp = 0; pp < 2; ++pp) {
                        Gr[j][pp] = pack2(gr[j][2 * pp], gr[j][2 * pp + 1]);
                        Gi[j][pp] = pack2(gi[j][2 * pp], gi[j][2 * pp + 1]);
                    }
                float4 c64 = make_float4(1.f, 1.f, 1.f, 1.f), s64 = make_float4(0.f, 0.f, 0.f, 0.f);
                if (active) {
                    c64 = *reinterpret_cast<const float4*>(tab.r64_c + 4 * q);
                    s64 = *reinterpret_cast<const float4*>(tab.r64_s + 4 * q);
                }
                Rc[0] = pack2(c64.x, c64.y); Rc[1] = pack2(c64.z, c64.w);
                Rs[0] = pack2(s64.x, s64.y); Rs[1] = pack2(s64.z, s64.w);
                Rn[0] = pack2(-s64.x, -s64.y); Rn[1] = pack2(-s64.z, -s64.w);
            }
            const uint64_t zero2 = pack2(0.f, 0.f);
            for (int k = 0; k < n_stages - 1; ++k) fetch(k);
            for (int k = 0; k < n_tiles; ++k) {
                fetch(k + n_stages - 1);
                if (!landed(k)) return;
                const int row0 = first_row + k * kRowsPerCta, nrows = min(kRowsPerCta, T_u - row0);
                const T* tile = stages + (size_t)c_stage * stage_elems;
                if (++c_stage == n_stages) { c_stage = 0; c_phase ^= 1u; }
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                if (active) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // rows past the end of the unit repeat the last one (their sums are not stored)
                        const T* row = tile + (size_t)(nrows == kRowsPerCta ? r_first + j : min(r_first + j, nrows - 1)) * d;
                        uint64_t kx[2], ky[2];
                        QuadPairs<T, LAYOUT>::ld(row, nb, q, kx, ky);
                        uint64_t a2 = zero2;
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            a2 = fma2(Gr[j][pp], kx[pp], a2);
                            a2 = fma2(Gi[j][pp], ky[pp], a2);
                            // on to the next tile: G e^{-i 64 omega} = (Gr c + Gi s) + i (Gi c - Gr s)
                            const uint64_t nr = fma2(Gr[j][pp], Rc[pp], fma2(Gi[j][pp], Rs[pp], zero2));
                            Gi[j][pp] = fma2(Gi[j][pp], Rc[pp], fma2(Gr[j][pp], Rn[pp], zero2));
                            Gr[j][pp] = nr;
                        }
                        float lo, hi2;
                        unpack2(a2, lo, hi2);
                        acc[j] = lo + hi2;
                    }
                }
                reduce_store(acc, row0, nrows);
                __syncthreads();        // the stage is free for the tile issued at the top of the next round
            }
            return;
        }
    }
    for (int k = 0; k < n_stages - 1; ++k) fetch(k);
    for (int k = 0; k < n_tiles; ++k) {
        fetch(k + n_stages - 1);
        if (!landed(k)) return;
        const int row0 = first_row + k * kRowsPerCta, nrows = min(kRowsPerCta, T_u - row0);
        const T* tile = stages + (size_t)c_stage * stage_elems;
        if (++c_stage == n_stages) { c_stage = 0; c_phase ^= 1u; }
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
        reduce_store(acc, row0, nrows);
        __syncthreads();            // the stage is free for the tile issued at the top of the next round
    }
}

}  // namespace

cudaError_t launch_score_stats(const Launch& L, const cask_query_stats& qs, float* s, Workspace& ws) {
    const Shape& sh = L.sh;
    const int nb = sh.d / 2;
    // the table of per-band constants sits behind the per-unit coefficients in the same workspace array
    float* tbase = ws.stats_a + (size_t)sh.n_units * sh.d;
    BandTable tab{tbase, tbase + nb, tbase + 2 * nb, tbase + 3 * nb, tbase + 6 * nb,
                  reinterpret_cast<unsigned long long*>(tbase + 4 * nb)};
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
