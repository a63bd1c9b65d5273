// Self-test of the bounded device waits: every mbarrier wait of the tensor-core and bulk-copy kernels goes through
// tc::mbar_wait, which gives up after a wall-time limit, raises an abort flag and lets the kernel end with
// CASK_ST_TIMEOUT instead of hanging.  In a healthy run no wait ever runs out, so that path would never execute; this
// entry point makes one run out on purpose, harmlessly: a single CTA waits, with a caller-chosen limit, on a
// barrier that nobody arrives at, then reports the flag exactly as the real kernels do and returns.
#include "tc_common.cuh"

namespace cask {
int selftest_set_flags_source(cask_ctx* ctx, const int32_t* flags_dev, int n_launches, cudaStream_t* stream, int* device);   // api.cu
}

using namespace cask;

namespace {

__global__ void __launch_bounds__(96) wait_timeout_kernel(unsigned long long limit_ns, int32_t* __restrict__ err,
                                                          unsigned long long* __restrict__ waited_ns) {
    using namespace tc;
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    __shared__ unsigned long long followed[2];
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // warp 0 waits for a phase that never completes; warps 1 and 2 wait on the same barrier with the default limit
    // and leave as soon as the first one has given up (the abort flag), the way the other roles of a kernel follow
    // the one that timed out: warp 1 with the form that reads the flag after every probe, warp 2 with the form that
    // reads it with the clock only
    const unsigned long long t0 = global_ns();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(&bar, 0u, &abort_flag, limit_ns);
    if (threadIdx.x == 32) ok = mbar_wait<false>(&bar, 0u, &abort_flag);
    if (threadIdx.x == 64) ok = mbar_wait<true>(&bar, 0u, &abort_flag);
    const unsigned long long t1 = global_ns();
    if (threadIdx.x == 32 || threadIdx.x == 64) followed[threadIdx.x / 32 - 1] = ok ? 0ull : t1 - t0;
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!ok && abort_flag) atomicOr(err, CASK_ST_TIMEOUT);
        waited_ns[0] = t1 - t0;
        // 0 unless both followers left on the flag; else the later of the two
        waited_ns[1] = (followed[0] && followed[1]) ? max(followed[0], followed[1]) : 0ull;
    }
}

// Throughput of the special-function unit in the instruction mix of the scoring epilogue: per element one FFMA (the
// argument), one ex2.approx, one FADD (the sum) and one FMUL, eight independent chains per thread, sixteen warps per
// SM.  Every CTA reports the clocks its loop took.
constexpr int kEx2Threads = 512, kEx2Chains = 8;
__global__ void __launch_bounds__(kEx2Threads) ex2_rate_kernel(int iters, unsigned long long* __restrict__ clk,
                                                               float* __restrict__ sink) {
    float x[kEx2Chains], acc[kEx2Chains];
#pragma unroll
    for (int j = 0; j < kEx2Chains; ++j) { x[j] = 0.25f + 0.001f * (float)((threadIdx.x + 7 * j) & 63); acc[j] = 0.f; }
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < kEx2Chains; ++j) {
            const float e = tc::ex2(fmaf(x[j], 0.5f, -1.f));
            acc[j] += e;
            x[j] = e * 1.0001f;
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < kEx2Chains; ++j) t += acc[j] + x[j];
    if (t == 12345.678f) sink[0] = t;          // keeps the loop alive; never true in practice
    if (threadIdx.x == 0) clk[blockIdx.x] = (unsigned long long)(t1 - t0);
}

}  // namespace

extern "C" int cask_selftest_exp_rate(cask_ctx* ctx, int32_t iters, void* ws, size_t ws_bytes, double* rate_host) {
    if (!ctx || !rate_host) return CASK_ERR_NULL;
    if (iters < 16 || iters > (1 << 20)) return CASK_ERR_PARAM;
    cudaStream_t st = nullptr;
    int device = 0;
    int rc = selftest_set_flags_source(ctx, nullptr, 2, &st, &device);
    if (rc != CASK_OK) return rc;
    int sms = 0;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess || sms < 1) return CASK_ERR_CUDA;
    sms = sms > 1024 ? 1024 : sms;
    if (!ws || ws_bytes < 16 + 8 * (size_t)sms || (uintptr_t)ws % 16) return CASK_ERR_WORKSPACE;
    float* sink = (float*)ws;
    unsigned long long* clk = (unsigned long long*)((char*)ws + 16);
    unsigned long long hclk[1024];
    for (int rep = 0; rep < 2 && e == cudaSuccess; ++rep) {      // the second launch is the measurement
        ex2_rate_kernel<<<sms, kEx2Threads, 0, st>>>(iters, clk, sink);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(hclk, clk, 8 * (size_t)sms, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return CASK_ERR_CUDA;
    // median over the SMs of exponentials per clock
    for (int i = 1; i < sms; ++i)
        for (int j = i; j > 0 && hclk[j] < hclk[j - 1]; --j) { unsigned long long t = hclk[j]; hclk[j] = hclk[j - 1]; hclk[j - 1] = t; }
    const double clocks = (double)hclk[sms / 2];
    *rate_host = clocks > 0 ? (double)kEx2Threads * kEx2Chains * (double)iters / clocks : 0.0;
    return CASK_OK;
}

extern "C" int cask_selftest_wait_timeout(cask_ctx* ctx, uint64_t limit_ns, void* ws, size_t ws_bytes,
                                          int32_t* flags_host, uint64_t* waited_ns_host) {
    if (!ctx || !flags_host) return CASK_ERR_NULL;
    if (limit_ns < 1000ull || limit_ns > 100000000ull) return CASK_ERR_PARAM;       // 1 us .. 100 ms
    if (!ws || ws_bytes < 64 || (uintptr_t)ws % 16) return CASK_ERR_WORKSPACE;
    int32_t* err = (int32_t*)ws;
    unsigned long long* waited = (unsigned long long*)((char*)ws + 16);
    cudaStream_t st = nullptr;
    int device = 0;
    int rc = selftest_set_flags_source(ctx, err, 1, &st, &device);
    if (rc != CASK_OK) return rc;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaMemsetAsync(ws, 0, 64, st);
    if (e == cudaSuccess) {
        wait_timeout_kernel<<<1, 96, 0, st>>>((unsigned long long)limit_ns, err, waited);
        e = cudaGetLastError();
    }
    unsigned long long w2[2] = {0, 0};
    if (e == cudaSuccess) e = cudaMemcpyAsync(flags_host, err, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(w2, waited, sizeof(w2), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return CASK_ERR_CUDA;
    if (waited_ns_host) { waited_ns_host[0] = w2[0]; waited_ns_host[1] = w2[1]; }
    return CASK_OK;
}
