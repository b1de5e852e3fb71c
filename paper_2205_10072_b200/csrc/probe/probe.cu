// Integer instruction rate probe (measurement helper of the benchmark; see bcs_probe.h; built into a library of its own).
#include "bcs_common.cuh"
#include "bcs_probe.h"

namespace bcs {
namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeCtas = 148 * 8;
constexpr int kChains = 8;        // independent dependency chains per thread
constexpr int kOpsPerIter = 32;   // instructions per loop round: 4 steps over all chains

template <int kMix>
__global__ void __launch_bounds__(kProbeThreads)
int_rate_kernel(uint32_t iters, uint32_t seed, uint32_t *sink)
{
    uint32_t a[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) a[c] = seed + threadIdx.x * 7u + blockIdx.x * 13u + c;
    const uint32_t m = seed | 1u, n = ~seed;
#pragma unroll 2
    for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
        for (int step = 0; step < kOpsPerIter / kChains; ++step) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                // one machine instruction each (inline PTX); the neighbouring chain's value is
                // the second operand
                const uint32_t v = a[c], w = a[(c + 1) % kChains];
                uint32_t d;
                if (kMix == 0 || (step & 1) == 0)                    // (v ^ w) | (v & m)
                    asm volatile("lop3.b32 %0, %1, %2, %3, 0xBC;" : "=r"(d) : "r"(v), "r"(w), "r"(m));
                else if (kMix == 1)                                  // v * w + n
                    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(v), "r"(w), "r"(n));
                else                                                 // v + w
                    asm volatile("add.u32 %0, %1, %2;" : "=r"(d) : "r"(v), "r"(w));
                a[c] = d;
            }
        }
    }
    uint32_t r = 0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) r ^= a[c];
    if (r == 0x9e3779b9u) atomicAdd(sink, r);   // practically never: keeps the results alive
}

}  // namespace
}  // namespace bcs

using namespace bcs;

extern "C" {

bcs_status bcs_probe_int_rate(int mix, uint32_t iters, uint32_t *sink_dev, double *ops_out,
                              float *ms_out, void *cuda_stream)
{
    if (sink_dev == nullptr || ops_out == nullptr || ms_out == nullptr || iters == 0 ||
        mix < 0 || mix > 2)
        return BCS_ERR_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaEvent_t t0, t1;
    if (cudaEventCreate(&t0) != cudaSuccess) return BCS_ERR_CUDA;
    if (cudaEventCreate(&t1) != cudaSuccess) {
        cudaEventDestroy(t0);
        return BCS_ERR_CUDA;
    }
    bcs_status st = BCS_OK;
    for (int pass = 0; pass < 2 && st == BCS_OK; ++pass) {          // first pass warms up
        cudaEventRecord(t0, stream);
        if (mix == 0)
            int_rate_kernel<0><<<kProbeCtas, kProbeThreads, 0, stream>>>(iters, 12345u + pass, sink_dev);
        else if (mix == 1)
            int_rate_kernel<1><<<kProbeCtas, kProbeThreads, 0, stream>>>(iters, 12345u + pass, sink_dev);
        else
            int_rate_kernel<2><<<kProbeCtas, kProbeThreads, 0, stream>>>(iters, 12345u + pass, sink_dev);
        st = launch_status();
        cudaEventRecord(t1, stream);
        if (cudaEventSynchronize(t1) != cudaSuccess) st = BCS_ERR_CUDA;
    }
    float ms = 0.f;
    if (st == BCS_OK && cudaEventElapsedTime(&ms, t0, t1) != cudaSuccess) st = BCS_ERR_CUDA;
    cudaEventDestroy(t0);
    cudaEventDestroy(t1);
    *ms_out = ms;
    *ops_out = (double)kProbeCtas * kProbeThreads * (double)iters * kOpsPerIter;
    return st;
}

}  // extern "C"
