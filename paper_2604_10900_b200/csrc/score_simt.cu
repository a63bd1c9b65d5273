// Windowed attention-mass scoring, SIMT fp32 path (any head_dim, bf16 or fp32 cache).
//
//   x_ri = <q_r, k_i>/sqrt(d),  visible(r,i) = i <= T-W+(r mod W)  (causal)
//   pass N ("normaliser"): per query row r, running max and sum of 2^(y - max) over visible keys
//   pass S ("score"):      s_i = sum_r roww_r * 2^(y_ri - rowm_r)
// with y = x*log2(e).  Both passes are the same 64x64 tile product between a
// stationary tile (kept in shared memory) and streaming tiles, followed by a
// reduction over the streaming side; only the epilogue differs.
#include "cask_internal.cuh"

namespace cask {

namespace {

constexpr int kTile = 64;
constexpr int kThreads = 256;

// Tile of 64 rows starting at row0 of `src` with a fixed row pitch (the dense query block).
template <typename T>
__device__ __forceinline__ void load_tile(float* dst, int pitch, const T* src, int64_t row_stride,
                                          int row0, int n_valid_rows, int d);

// Tile of 64 cache rows of a unit (contiguous or paged keys).
template <typename T>
__device__ __forceinline__ void load_key_tile(float* dst, int pitch, const T* K, const Shape& sh, const UnitDesc& ud,
                                              int row0, int n_valid_rows, int d) {
    if (sh.page_size == 0) {
        load_tile<T>(dst, pitch, K + ud.k_off, sh.row_stride, row0, n_valid_rows, d);
        return;
    }
    const int vec_per_row = d / 8;
    for (int idx = threadIdx.x; idx < kTile * vec_per_row; idx += kThreads) {
        int r = idx / vec_per_row, c8 = (idx % vec_per_row) * 8;
#pragma unroll
        for (int t = 0; t < 8; ++t)
            dst[r * pitch + c8 + t] =
                (r < n_valid_rows) ? Elem<T>::ld(K + row_elem_off(sh, ud, ud.k_off, row0 + r) + c8 + t) : 0.f;
    }
}

template <typename T>
__device__ __forceinline__ void load_tile(float* dst, int pitch, const T* src, int64_t row_stride,
                                          int row0, int n_valid_rows, int d) {
    // 64 rows x d elements, 8 elements (16 or 32 bytes) per step; rows past n_valid_rows are zeroed
    const int vec_per_row = d / 8;
    for (int idx = threadIdx.x; idx < kTile * vec_per_row; idx += kThreads) {
        int r = idx / vec_per_row, c8 = (idx % vec_per_row) * 8;
        float v[8];
        if (r < n_valid_rows) {
            const T* p = src + (int64_t)(row0 + r) * row_stride + c8;
            if constexpr (sizeof(T) == 2) {
                uint4 raw = *reinterpret_cast<const uint4*>(p);
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float2 f = __bfloat1622float2(h[t]);
                    v[2 * t] = f.x;
                    v[2 * t + 1] = f.y;
                }
            } else {
                float4 a = *reinterpret_cast<const float4*>(p);
                float4 b = *reinterpret_cast<const float4*>(p + 4);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
                v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            }
        } else {
#pragma unroll
            for (int t = 0; t < 8; ++t) v[t] = 0.f;
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) dst[r * pitch + c8 + t] = v[t];
    }
}

__device__ __forceinline__ void tile_product(const float* St, const float* Rt, int pitch, int d, int ty,
                                             int tx, float acc[4][4]) {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
    for (int c = 0; c < d; ++c) {
        float sa[4], rb[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) sa[a] = St[(ty + 16 * a) * pitch + c];
#pragma unroll
        for (int b = 0; b < 4; ++b) rb[b] = Rt[(tx + 16 * b) * pitch + c];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(sa[a], rb[b], acc[a][b]);
    }
}

// pass N: grid (chunk within unit, row block, unit)
template <typename T>
__global__ void __launch_bounds__(kThreads) score_norm_simt(const UnitDesc* __restrict__ desc, Shape sh,
                                                            const T* __restrict__ K,
                                                            const T* __restrict__ Q,
                                                            float* __restrict__ part_m,
                                                            float* __restrict__ part_l) {
    extern __shared__ float smem[];
    const UnitDesc& ud = desc[blockIdx.z];
    const int kc = blockIdx.x;
    if (kc >= ud.n_chunks) return;
    const int d = sh.d, pitch = d + 1, rows = sh.rows;
    float* St = smem;
    float* Rt = smem + kTile * pitch;
    const int row0 = blockIdx.y * kTile;
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    const float scale2 = kLog2e * rsqrtf((float)d);
    const int Tn = ud.T;

    load_tile<T>(St, pitch, Q + ud.q_off, d, row0, min(kTile, rows - row0), d);
    float m[4], l[4];
    int lastvis[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        m[a] = kNegBig;
        l[a] = 0.f;
        int r = row0 + ty + 16 * a;
        lastvis[a] = (r < rows) ? (sh.causal ? Tn - sh.W + (r % sh.W) : Tn - 1) : -1;
    }
    const int key_end = min(Tn, (kc + 1) * kChunkKeys);
    for (int key0 = kc * kChunkKeys; key0 < key_end; key0 += kTile) {
        __syncthreads();
        load_key_tile<T>(Rt, pitch, K, sh, ud, key0, min(kTile, Tn - key0), d);
        __syncthreads();
        float acc[4][4];
        tile_product(St, Rt, pitch, d, ty, tx, acc);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float tm = kNegBig;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                int i = key0 + tx + 16 * b;
                acc[a][b] *= scale2;
                if (i <= lastvis[a]) tm = fmaxf(tm, acc[a][b]);
            }
            if (tm > m[a]) {
                l[a] *= exp2f(m[a] - tm);
                m[a] = tm;
            }
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                int i = key0 + tx + 16 * b;
                if (i <= lastvis[a]) l[a] += exp2f(acc[a][b] - m[a]);
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
            float m2 = __shfl_xor_sync(0xffffffffu, m[a], off);
            float l2 = __shfl_xor_sync(0xffffffffu, l[a], off);
            float mn = fmaxf(m[a], m2);
            l[a] = l[a] * exp2f(m[a] - mn) + l2 * exp2f(m2 - mn);
            m[a] = mn;
        }
        int r = row0 + ty + 16 * a;
        if (tx == 0 && r < rows) {
            size_t o = (size_t)(ud.chunk0 + kc) * rows + r;
            part_m[o] = m[a];
            part_l[o] = l[a];
        }
    }
}

// pass S: grid (key tile within unit, unit)
template <typename T>
__global__ void __launch_bounds__(kThreads) score_mass_simt(const UnitDesc* __restrict__ desc, Shape sh,
                                                            const T* __restrict__ K,
                                                            const T* __restrict__ Q,
                                                            const float* __restrict__ rowm,
                                                            const float* __restrict__ roww,
                                                            float* __restrict__ s) {
    extern __shared__ float smem[];
    const UnitDesc& ud = desc[blockIdx.y];
    const int key0 = blockIdx.x * kTile;
    const int Tn = ud.T;
    if (key0 >= Tn) return;
    const int d = sh.d, pitch = d + 1, rows = sh.rows;
    float* St = smem;
    float* Rt = smem + kTile * pitch;
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    const float scale2 = kLog2e * rsqrtf((float)d);
    const float* rm = rowm + (size_t)blockIdx.y * rows;
    const float* rw = roww + (size_t)blockIdx.y * rows;

    load_key_tile<T>(St, pitch, K, sh, ud, key0, min(kTile, Tn - key0), d);
    float accs[4] = {0.f, 0.f, 0.f, 0.f};
    for (int row0 = 0; row0 < rows; row0 += kTile) {
        __syncthreads();
        load_tile<T>(Rt, pitch, Q + ud.q_off, d, row0, min(kTile, rows - row0), d);
        __syncthreads();
        float acc[4][4];
        tile_product(St, Rt, pitch, d, ty, tx, acc);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int r = row0 + tx + 16 * b;
            if (r >= rows) continue;
            int lastvis = sh.causal ? Tn - sh.W + (r % sh.W) : Tn - 1;
            float mr = rm[r], wr = rw[r];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                int i = key0 + ty + 16 * a;
                if (i <= lastvis) accs[a] = fmaf(exp2f(fmaf(acc[a][b], scale2, -mr)), wr, accs[a]);
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) accs[a] += __shfl_xor_sync(0xffffffffu, accs[a], off);
        int i = key0 + ty + 16 * a;
        if (tx == 0 && i < Tn) s[ud.tok_off + i] = accs[a];
    }
}

// Combine the per-chunk (max, sum) pairs of every query row into the row offset and row
// weight used by the score pass:  rowm = max,  roww = 1/(rows * sum 2^(y-max)).
// With caller-supplied natural-log normalisers: rowm = lse*log2(e), roww = 1/rows.
__global__ void row_combine(const UnitDesc* __restrict__ desc, int rows, const float* __restrict__ part_m,
                            const float* __restrict__ part_l, const float* __restrict__ lse_in,
                            float* __restrict__ rowm, float* __restrict__ roww,
                            float* __restrict__ lse_out) {
    const UnitDesc& ud = desc[blockIdx.x];
    const float inv_rows = 1.f / (float)rows;
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        size_t o = (size_t)blockIdx.x * rows + r;
        if (lse_in) {
            float lse = lse_in[o];
            rowm[o] = lse * kLog2e;
            roww[o] = inv_rows;
            if (lse_out) lse_out[o] = lse;
            continue;
        }
        float m = kNegBig;
        for (int c = 0; c < ud.n_chunks; ++c) m = fmaxf(m, part_m[(size_t)(ud.chunk0 + c) * rows + r]);
        float l = 0.f;
        for (int c = 0; c < ud.n_chunks; ++c) {
            size_t p = (size_t)(ud.chunk0 + c) * rows + r;
            l += part_l[p] * exp2f(part_m[p] - m);
        }
        rowm[o] = m;
        roww[o] = inv_rows / l;
        if (lse_out) lse_out[o] = (m + log2f(l)) * kLn2;
    }
}

template <typename T>
cudaError_t run_simt(const Launch& L, const float* lse_in, float* s, float* lse_out, Workspace& ws) {
    const Shape& sh = L.sh;
    const size_t smem = (size_t)2 * kTile * (sh.d + 1) * sizeof(float);
    cudaError_t e;
    e = cudaFuncSetAttribute(score_norm_simt<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_mass_simt<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int row_blocks = (sh.rows + kTile - 1) / kTile;
    if (!lse_in) {
        dim3 g(L.max_chunks, row_blocks, sh.n_units);
        Timed t(L, KID_SCORE_NORM);
        score_norm_simt<T><<<g, kThreads, smem, L.stream>>>(L.desc, sh, (const T*)L.k, (const T*)L.q,
                                                            ws.part_m, ws.part_l);
    }
    e = launch_row_combine(L, lse_in, lse_out, ws);
    if (e != cudaSuccess) return e;
    dim3 g2((L.max_T + kTile - 1) / kTile, sh.n_units);
    {
        Timed t(L, KID_SCORE_MASS);
        score_mass_simt<T><<<g2, kThreads, smem, L.stream>>>(L.desc, sh, (const T*)L.k, (const T*)L.q, ws.rowm,
                                                             ws.roww, s);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_row_combine(const Launch& L, const float* lse_in, float* lse_out, Workspace& ws) {
    Timed t(L, KID_ROW_COMBINE);
    row_combine<<<L.sh.n_units, 128, 0, L.stream>>>(L.desc, L.sh.rows, ws.part_m, ws.part_l, lse_in,
                                                   ws.rowm, ws.roww, lse_out);
    return cudaGetLastError();
}

cudaError_t launch_score_simt(const Launch& L, const float* lse_in, float* s, float* lse_out,
                              Workspace& ws) {
    if (L.sh.dtype == CASK_DTYPE_BF16) return run_simt<__nv_bfloat16>(L, lse_in, s, lse_out, ws);
    return run_simt<float>(L, lse_in, s, lse_out, ws);
}

}  // namespace cask
