// Executor selection for a batch of cell executions (Section 3.2.2): for each kernel, which of
// its three replica hosts has the idle resources to run the cell now, and which one the
// scheduler designates (default policy order of Section 3.4.1 among those that can run).
// One thread per kernel: a 128-bit request load, three host ids, three gathers from the
// cluster-state arrays (which stay in L2), two 32-bit results. HBM-bound: 36 bytes per kernel.
#include "nbos_internal.h"

namespace nbos {
namespace {

struct ExecArgs {
    const int4 *fit;        // [H] (idle GPUs or -1 if the host has none, vram_gb, millicpus, mem_mb)
    const int2 *rank;       // [H] (G, S): what the order among runnable replicas needs
    const int4 *requests;
    const int32_t *replica_hosts;
    int32_t *out_executor, *out_can_run;
    long long n_kernels;
    int H;
};

// Gathering six separate arrays per replica costs 18 scattered loads per kernel; two packed
// records per host make it 3 (+ up to 3 when more than one replica can run).
__global__ void __launch_bounds__(256) pack_state_kernel(const int32_t *G, const int32_t *S, const int32_t *C,
                                                         const int32_t *AV, const int32_t *AC,
                                                         const int32_t *AM, int H, int4 *fit, int2 *rank)
{
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= H) return;
    const int g = G[h];
    fit[h] = make_int4(g >= 1 ? g - C[h] : -1, AV[h], AC[h], AM[h]);
    rank[h] = make_int2(g, S[h]);
}

// One kernel per thread and iteration. SMEM = true: the packed tables are first copied into
// shared memory (scattered 16-byte reads from shared memory are several times cheaper than from
// L1, whose tag stage handles one cache line per cycle); SMEM = false: gathers go to global
// memory (tables too large for shared memory, or too few kernels to pay for the copy).
template <bool SMEM>
__global__ void __launch_bounds__(512) select_executors_kernel(const ExecArgs a)
{
    extern __shared__ __align__(16) unsigned char exec_smem[];
    const int4 *fit = a.fit;
    const int2 *rank = a.rank;
    if (SMEM) {
        int4 *s_fit = reinterpret_cast<int4 *>(exec_smem);
        int2 *s_rank = reinterpret_cast<int2 *>(exec_smem + (size_t)a.H * sizeof(int4));
        for (int i = threadIdx.x; i < a.H; i += blockDim.x) {
            s_fit[i] = a.fit[i];
            s_rank[i] = a.rank[i];
        }
        __syncthreads();
        fit = s_fit;
        rank = s_rank;
    }
    // the streams of the next iteration are requested before this iteration's records are
    // gathered, so that every thread always has a request and three host ids in flight
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    int4 r_next = make_int4(-1, 0, 0, 0);
    int h_next[3] = {-1, -1, -1};
    if (k < a.n_kernels) {
        r_next = __ldg(a.requests + k);
#pragma unroll
        for (int slot = 0; slot < 3; ++slot) h_next[slot] = __ldg(a.replica_hosts + 3 * k + slot);
    }
    for (; k < a.n_kernels; k += stride) {
        const int4 r = r_next;
        int h[3] = {h_next[0], h_next[1], h_next[2]};
        if (k + stride < a.n_kernels) {
            r_next = __ldg(a.requests + k + stride);
#pragma unroll
            for (int slot = 0; slot < 3; ++slot) h_next[slot] = __ldg(a.replica_hosts + 3 * (k + stride) + slot);
        }
        const bool sane = (r.x | r.y | r.z | r.w) >= 0;
        int4 f[3];
        bool ok[3];
#pragma unroll
        for (int slot = 0; slot < 3; ++slot) {
            const bool valid = sane && h[slot] >= 0 && h[slot] < a.H;
            f[slot] = valid ? fit[h[slot]] : make_int4(-1, 0, 0, 0);
            ok[slot] = valid && r.x <= f[slot].x && r.y <= f[slot].y && r.z <= f[slot].z && r.w <= f[slot].w;
        }
        const int mask = (int)ok[0] | ((int)ok[1] << 1) | ((int)ok[2] << 2);
        int best = -1;
        if (mask != 0 && (mask & (mask - 1)) == 0) {
            best = ok[0] ? h[0] : ok[1] ? h[1] : h[2];  // a single runnable replica: no ranking needed
        } else if (mask != 0) {
            int best_idle = 0, best_slot = 0;
            int2 best_gs = make_int2(1, 0);
            bool have_gs = false;  // (G, S) of the current best is fetched only when idle GPUs tie
#pragma unroll
            for (int slot = 0; slot < 3; ++slot) {
                if (!ok[slot]) continue;
                const int idle = f[slot].x;
                bool before = best < 0 || idle > best_idle;
                if (best >= 0 && idle == best_idle) {
                    if (!have_gs) best_gs = rank[best];
                    const int2 gs = rank[h[slot]];
                    // S / (G R) against best_S / (best_G R): R cancels, cross-multiply exactly
                    const long long lhs = (long long)gs.y * best_gs.x, rhs = (long long)best_gs.y * gs.x;
                    before = lhs != rhs ? lhs < rhs : h[slot] < best;
                    if (before) best_gs = gs;
                    have_gs = true;
                } else if (before) {
                    have_gs = false;
                }
                if (before) {
                    best = h[slot];
                    best_idle = idle;
                    best_slot = slot;
                }
            }
            (void)best_slot;
        }
        a.out_executor[k] = best;
        a.out_can_run[k] = mask;
    }
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace nbos

using namespace nbos;

extern "C" int nbos_select_executors(const nbos_cluster_state *state, const int32_t *requests,
                                     const int32_t *replica_hosts, int64_t n_kernels,
                                     int32_t *out_executor, int32_t *out_can_run, void *cuda_stream)
{
    if (!state) return fail(NBOS_ERR_INVALID_ARG, "state is NULL");
    if (state->n_hosts < 1 || state->n_hosts > NBOS_MAX_HOSTS)
        return fail(NBOS_ERR_INVALID_ARG, "n_hosts must be in 1..%d", NBOS_MAX_HOSTS);
    if (state->replicas_R < 1 || state->replicas_R > NBOS_MAX_REPLICAS)
        return fail(NBOS_ERR_INVALID_ARG, "replicas_R must be in 1..%d", NBOS_MAX_REPLICAS);
    if (n_kernels < 0 || n_kernels > ((int64_t)1 << 40)) return fail(NBOS_ERR_INVALID_ARG, "n_kernels out of range");
    if (n_kernels == 0) return NBOS_OK;
    const void *arrays[6] = {state->gpus_total, state->gpus_subscribed, state->gpus_committed,
                             state->vram_gb, state->millicpus, state->mem_mb};
    for (int i = 0; i < 6; ++i)
        if (!arrays[i]) return fail(NBOS_ERR_INVALID_ARG, "cluster-state array %d is NULL", i);
    if (!requests || !replica_hosts || !out_executor || !out_can_run)
        return fail(NBOS_ERR_INVALID_ARG, "NULL request / replica / output pointer");
    if (!aligned16(requests)) return fail(NBOS_ERR_INVALID_ARG, "requests is not 16-byte aligned");
    int device = 0, major = 0, sms = 0;
    NBOS_CUDA_TRY(cudaGetDevice(&device));
    NBOS_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    if (major != 10) return fail(NBOS_ERR_UNSUPPORTED_DEVICE, "device %d has compute capability %d.x", device, major);
    NBOS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int H = state->n_hosts;
    char *packed = nullptr;  // stream-ordered temporary: 24 bytes per host
    const size_t fit_bytes = ((size_t)H * sizeof(int4) + 255) & ~(size_t)255;
    cudaMemPool_t pool = nullptr;
    int rc = library_pool(device, &pool);
    if (rc) return rc;
    cudaError_t e = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&packed), fit_bytes + (size_t)H * sizeof(int2), pool, stream);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(NBOS_ERR_NO_MEMORY, "device allocation failed: %s", cudaGetErrorString(e));
    }
    int4 *fit = reinterpret_cast<int4 *>(packed);
    int2 *rank = reinterpret_cast<int2 *>(packed + fit_bytes);
    pack_state_kernel<<<(H + 255) / 256, 256, 0, stream>>>(state->gpus_total, state->gpus_subscribed,
                                                           state->gpus_committed, state->vram_gb,
                                                           state->millicpus, state->mem_mb, H, fit, rank);
    e = cudaGetLastError();
    if (e == cudaSuccess) {
        ExecArgs a{fit, rank, reinterpret_cast<const int4 *>(requests), replica_hosts,
                   out_executor, out_can_run, n_kernels, H};
        const size_t table_bytes = (size_t)H * (sizeof(int4) + sizeof(int2));
        const bool use_smem = table_bytes <= 96 * 1024 && n_kernels >= (long long)sms * 2 * 8 * H;
        if (use_smem) {
            e = cudaFuncSetAttribute(select_executors_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)table_bytes);
            const int per_sm = table_bytes <= 56 * 1024 ? 3 : 2;
            if (e == cudaSuccess)
                select_executors_kernel<true><<<sms * per_sm, 512, table_bytes, stream>>>(a);
        } else {
            long long blocks = (n_kernels + 511) / 512;
            if (blocks > (long long)sms * 4) blocks = (long long)sms * 4;
            select_executors_kernel<false><<<(unsigned int)blocks, 512, 0, stream>>>(a);
        }
        e = cudaGetLastError();
    }
    cudaFreeAsync(packed, stream);
    if (e != cudaSuccess) return cuda_fail(e, "executor selection launch");
    return NBOS_OK;
}
