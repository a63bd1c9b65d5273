// Stage 1 prefix eviction and protected-core selection: one CTA per unit.
#include "select.cuh"

namespace cask {

namespace {

// kind[0:T) = 0; plan written out; kept prefix rows -> CASK_KIND_PREFIX (Sec. 2.2, Stage 1).
__global__ void __launch_bounds__(kSelThreads) prefix_evict_kernel(const UnitDesc* __restrict__ desc,
                                                                   const float* __restrict__ s,
                                                                   uint8_t* __restrict__ kind,
                                                                   int32_t* __restrict__ plan) {
    __shared__ SelectSmem sm;
    const UnitDesc& ud = desc[blockIdx.x];
    uint8_t* kd = kind + ud.tok_off;
    const float* su = s + ud.tok_off;
    if (threadIdx.x < 8) plan[blockIdx.x * 8 + threadIdx.x] = ud.plan[threadIdx.x];
    const int P = ud.P, pkeep = ud.plan[CASK_PLAN_PKEEP];
    const uint8_t pre = (P <= pkeep) ? CASK_KIND_PREFIX : CASK_KIND_DROPPED;
    for (int i = threadIdx.x; i < ud.T; i += blockDim.x) kd[i] = (i < P) ? pre : CASK_KIND_DROPPED;
    __syncthreads();
    if (P > pkeep) block_topk_mark(su, kd, 0, P, pkeep, CASK_KIND_PREFIX, sm);
}

// decode rows: last r -> RECENT, the c greatest of [P, T-r) -> CORE (Sec. 2.1, 2.3).
__global__ void __launch_bounds__(kSelThreads) select_core_kernel(const UnitDesc* __restrict__ desc,
                                                                  const float* __restrict__ s,
                                                                  const int32_t* __restrict__ plan,
                                                                  uint8_t* __restrict__ kind) {
    __shared__ SelectSmem sm;
    const UnitDesc& ud = desc[blockIdx.x];
    uint8_t* kd = kind + ud.tok_off;
    const float* su = s + ud.tok_off;
    const int T = ud.T, P = ud.P;
    int r = plan[blockIdx.x * 8 + CASK_PLAN_R], c = plan[blockIdx.x * 8 + CASK_PLAN_C];
    r = max(0, min(r, T - P));
    for (int i = P + threadIdx.x; i < T; i += blockDim.x)
        kd[i] = (i >= T - r) ? CASK_KIND_RECENT : CASK_KIND_DROPPED;
    __syncthreads();
    block_topk_mark(su, kd, P, T - r, c, CASK_KIND_CORE, sm);
}

}  // namespace

cudaError_t launch_prefix_evict(const Launch& L, const float* s, uint8_t* kind, int32_t* plan) {
    Timed t(L, KID_PREFIX_EVICT);
    prefix_evict_kernel<<<L.sh.n_units, select_threads(L.max_T), 0, L.stream>>>(L.desc, s, kind, plan);
    return cudaGetLastError();
}

cudaError_t launch_select_core(const Launch& L, const float* s, const int32_t* plan, uint8_t* kind) {
    Timed t(L, KID_SELECT_CORE);
    select_core_kernel<<<L.sh.n_units, select_threads(L.max_T), 0, L.stream>>>(L.desc, s, plan, kind);
    return cudaGetLastError();
}

}  // namespace cask
