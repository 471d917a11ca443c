// Cluster-wide reductions next to the placement path: the sums behind the dynamic SR limit and
// the auto-scaler rule (Sections 3.4.1, 3.4.2), and the scale-out deficit of a placed batch
// (Sections 3.2.1, 3.4.2).
#include "nbos_internal.h"

namespace nbos {
namespace {

// out[n] = (sum over the batch of 3 - found, number of requests with found < 3); grid (bx, N).
__global__ void __launch_bounds__(256) deficit_kernel(const int32_t *found, long long B,
                                                      unsigned long long *out)
{
    __shared__ unsigned long long s_acc[2];
    if (threadIdx.x < 2) s_acc[threadIdx.x] = 0ull;
    __syncthreads();
    const size_t base = (size_t)blockIdx.y * (size_t)B;
    unsigned long long deficit = 0, shortc = 0;
    for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < B;
         r += (long long)gridDim.x * blockDim.x) {
        const int f = __ldg(found + base + r);
        if (f < NBOS_REPLICAS_PLACED) {
            deficit += (unsigned long long)(NBOS_REPLICAS_PLACED - (f < 0 ? 0 : f));
            shortc += 1;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        deficit += __shfl_xor_sync(0xFFFFFFFFu, deficit, off);
        shortc += __shfl_xor_sync(0xFFFFFFFFu, shortc, off);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&s_acc[0], deficit);
        atomicAdd(&s_acc[1], shortc);
    }
    __syncthreads();
    if (threadIdx.x < 2 && s_acc[threadIdx.x]) atomicAdd(&out[(size_t)blockIdx.y * 2 + threadIdx.x], s_acc[threadIdx.x]);
}

int check_sm100()
{
    int device = 0, major = 0;
    NBOS_CUDA_TRY(cudaGetDevice(&device));
    NBOS_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    if (major != 10) return fail(NBOS_ERR_UNSUPPORTED_DEVICE, "device %d has compute capability %d.x", device, major);
    return NBOS_OK;
}

}  // namespace
}  // namespace nbos

using namespace nbos;

extern "C" int nbos_cluster_sums(const int32_t *gpus_total, const int32_t *gpus_subscribed,
                                 const int32_t *gpus_committed, int32_t n_snapshots, int32_t n_hosts,
                                 int32_t f_num, int32_t f_den, int64_t *out_sums, void *cuda_stream)
{
    if (!gpus_total || !gpus_subscribed || !gpus_committed || !out_sums) return fail(NBOS_ERR_INVALID_ARG, "NULL pointer");
    if (n_snapshots < 1 || n_snapshots > 65535) return fail(NBOS_ERR_INVALID_ARG, "n_snapshots must be in 1..65535");
    if (n_hosts < 1 || n_hosts > NBOS_MAX_HOSTS) return fail(NBOS_ERR_INVALID_ARG, "n_hosts must be in 1..%d", NBOS_MAX_HOSTS);
    if (f_num < 0 || f_den < 1) return fail(NBOS_ERR_INVALID_ARG, "f = f_num / f_den needs f_num >= 0, f_den >= 1");
    if (reinterpret_cast<uintptr_t>(out_sums) & 7) return fail(NBOS_ERR_INVALID_ARG, "out_sums is not 8-byte aligned");
    int rc = check_sm100();
    if (rc) return rc;
    return launch_cluster_sums(gpus_total, gpus_subscribed, gpus_committed, n_snapshots, n_hosts, f_num, f_den,
                               reinterpret_cast<long long *>(out_sums), static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int nbos_scale_out_deficit(const int32_t *found, int32_t n_snapshots, int64_t batch_per_snapshot,
                                      int64_t *out_deficit, void *cuda_stream)
{
    if (!out_deficit || (!found && batch_per_snapshot != 0)) return fail(NBOS_ERR_INVALID_ARG, "NULL pointer");
    if (n_snapshots < 1 || n_snapshots > 65535) return fail(NBOS_ERR_INVALID_ARG, "n_snapshots must be in 1..65535");
    if (batch_per_snapshot < 0 || batch_per_snapshot > ((int64_t)1 << 40) / n_snapshots)
        return fail(NBOS_ERR_INVALID_ARG, "batch_per_snapshot out of range");
    if (reinterpret_cast<uintptr_t>(out_deficit) & 7) return fail(NBOS_ERR_INVALID_ARG, "out_deficit is not 8-byte aligned");
    int rc = check_sm100();
    if (rc) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    NBOS_CUDA_TRY(cudaMemsetAsync(out_deficit, 0, sizeof(int64_t) * 2 * (size_t)n_snapshots, stream));
    if (batch_per_snapshot == 0) return NBOS_OK;
    long long bx = (batch_per_snapshot + 1023) / 1024;
    const long long cap = n_snapshots >= 64 ? 16 : 592;
    if (bx > cap) bx = cap;
    deficit_kernel<<<dim3((unsigned int)bx, n_snapshots), 256, 0, stream>>>(
        found, batch_per_snapshot, reinterpret_cast<unsigned long long *>(out_deficit));
    NBOS_CUDA_TRY(cudaGetLastError());
    return NBOS_OK;
}
