// Measurement helpers declared in include/nbos_probe.h.
#include "nbos_internal.h"
#include "nbos_ptx.cuh"
#include "nbos_probe.h"

namespace nbos {
namespace {

constexpr int kChains = 8;

template <int MIX>
__global__ void __launch_bounds__(1024) issue_probe_kernel(int iters, int a, int b, int c, int d,
                                                           int *sink)
{
    int x[kChains];
#pragma unroll
    for (int j = 0; j < kChains; ++j) x[j] = (int)(threadIdx.x * 2654435761u) + j * 97 + blockIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < kChains; ++j) {
            if (MIX == NBOS_PROBE_MIX_ALU) {
                asm volatile("xor.b32 %0, %0, %1;" : "+r"(x[j]) : "r"(a));
                asm volatile("min.s32 %0, %0, %1;" : "+r"(x[j]) : "r"(b));
                asm volatile("xor.b32 %0, %0, %1;" : "+r"(x[j]) : "r"(c));
                asm volatile("max.s32 %0, %0, %1;" : "+r"(x[j]) : "r"(d));
            } else if (MIX == NBOS_PROBE_MIX_IMAD) {
                asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(x[j]) : "r"(a), "r"(b));
                asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(x[j]) : "r"(c), "r"(d));
                asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(x[j]) : "r"(b), "r"(a));
                asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(x[j]) : "r"(d), "r"(c));
            } else {
                asm volatile("xor.b32 %0, %0, %1;" : "+r"(x[j]) : "r"(a));
                asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(x[j]) : "r"(c), "r"(d));
                asm volatile("min.s32 %0, %0, %1;" : "+r"(x[j]) : "r"(b));
                asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(x[j]) : "r"(d), "r"(c));
            }
        }
    }
    int acc = 0;
#pragma unroll
    for (int j = 0; j < kChains; ++j) acc ^= x[j];
    if (acc == 0x7fffffff) sink[0] = acc;  // keeps the chains alive; practically never taken
}

// Two warps wait, with the placement kernel's own bounded wait, for a phase of a shared-memory
// barrier that nothing ever completes. The warp whose wait runs out first raises the block's abort
// flag, the other leaves through that flag; each reports in `status` the way the placement kernel
// reports in a snapshot's status word (bit 0), plus bit 1 + warp index for the test to see that
// both warps came back.
__global__ void wait_timeout_kernel(unsigned long long limit_ns, unsigned int *status)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ unsigned int abort_flag;
    const uint32_t addr = smem_addr(&bar);
    if (threadIdx.x == 0) {
        mbar_init(addr, 1u);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool done = mbar_wait(addr, 0u, &abort_flag, limit_ns);
    if (!done && (threadIdx.x & 31) == 0) atomicOr(status, STATUS_WAIT_TIMEOUT | (2u << (threadIdx.x >> 5)));
}

}  // namespace
}  // namespace nbos

using namespace nbos;

extern "C" int nbos_probe_int32_issue(int mix, int iters, int blocks, int threads, void *cuda_stream,
                                      double *out_thread_ops, float *out_ms)
{
    if (!out_thread_ops || !out_ms) return fail(NBOS_ERR_INVALID_ARG, "NULL output");
    if (mix < 0 || mix > 2 || iters < 1 || blocks < 1 || threads < 32 || threads > 1024 || (threads & 31))
        return fail(NBOS_ERR_INVALID_ARG, "probe arguments out of range");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int *sink = nullptr;
    NBOS_CUDA_TRY(cudaMalloc(&sink, sizeof(int)));
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    // operands come in as runtime values so nothing folds at compile time
    const int a = 0x5bd1e995, b = 0x3fffffff, c = 0x27d4eb2f, d = -0x40000000;
    cudaEventRecord(e0, stream);
    if (mix == NBOS_PROBE_MIX_ALU)
        issue_probe_kernel<NBOS_PROBE_MIX_ALU><<<blocks, threads, 0, stream>>>(iters, a, b, c, d, sink);
    else if (mix == NBOS_PROBE_MIX_IMAD)
        issue_probe_kernel<NBOS_PROBE_MIX_IMAD><<<blocks, threads, 0, stream>>>(iters, a, b, c, d, sink);
    else
        issue_probe_kernel<NBOS_PROBE_MIX_BOTH><<<blocks, threads, 0, stream>>>(iters, a, b, c, d, sink);
    cudaError_t e = cudaGetLastError();
    cudaEventRecord(e1, stream);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(sink);
    if (e != cudaSuccess) return cuda_fail(e, "issue probe");
    *out_ms = ms;
    *out_thread_ops = (double)iters * kChains * 4.0 * (double)threads * (double)blocks;
    return NBOS_OK;
}

static int run_wait_timeout(uint64_t limit_ns, cudaStream_t stream, unsigned int *d_status, float *out_ms)
{
    if (limit_ns < 1000000ull) limit_ns = 1000000ull;
    if (limit_ns > 5000000000ull) limit_ns = 5000000000ull;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    cudaEventRecord(e0, stream);
    wait_timeout_kernel<<<1, 64, 0, stream>>>(limit_ns, d_status);
    cudaError_t e = cudaGetLastError();
    cudaEventRecord(e1, stream);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return cuda_fail(e, "wait-timeout self-test");
    *out_ms = ms;
    return NBOS_OK;
}

extern "C" int nbos_probe_wait_timeout(uint64_t limit_ns, void *cuda_stream, int *out_gave_up,
                                       float *out_ms)
{
    if (!out_gave_up || !out_ms) return fail(NBOS_ERR_INVALID_ARG, "NULL output");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned int *flag = nullptr;
    NBOS_CUDA_TRY(cudaMalloc(&flag, sizeof(unsigned int)));
    cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(unsigned int), stream);
    int rc = e == cudaSuccess ? run_wait_timeout(limit_ns, stream, flag, out_ms) : cuda_fail(e, "cudaMemsetAsync");
    unsigned int word = 0;
    if (rc == NBOS_OK) {
        e = cudaMemcpy(&word, flag, sizeof(word), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) rc = cuda_fail(e, "reading the self-test's status word");
    }
    cudaFree(flag);
    if (rc) return rc;
    *out_gave_up = (word & STATUS_WAIT_TIMEOUT) ? (int)(word >> 1) : 0;
    return NBOS_OK;
}

extern "C" int nbos_probe_wait_timeout_on_snapshot(nbos_snapshot *snap, uint64_t limit_ns,
                                                   void *cuda_stream, float *out_ms)
{
    if (!snap || !out_ms) return fail(NBOS_ERR_INVALID_ARG, "NULL argument");
    int device = -1;
    NBOS_CUDA_TRY(cudaGetDevice(&device));
    if (device != snap->device) return fail(NBOS_ERR_INVALID_ARG, "the snapshot belongs to device %d", snap->device);
    return run_wait_timeout(limit_ns, static_cast<cudaStream_t>(cuda_stream), snap->d_status, out_ms);
}
