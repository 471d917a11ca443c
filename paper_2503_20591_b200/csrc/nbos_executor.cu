// Executor selection for a batch of cell executions (Section 3.2.2): for each kernel, which of
// its three replica hosts has the idle resources to run the cell now, and which one the
// scheduler designates (default policy order of Section 3.4.1 among those that can run).
// One thread per kernel: a 128-bit request load, three host ids, three gathers from a packed
// host table in shared memory, two 32-bit results. HBM-bound: 36 bytes per kernel.
#include <limits.h>

#include "nbos_internal.h"
#include "nbos_ptx.cuh"

namespace nbos {
namespace {

// Packed form of a host: the four capacities of "can run now" in 8 bytes, each field under a
// guard bit, so that one subtraction per word tests two capacities at once (host - ask keeps a
// guard exactly when capacity >= ask in that field; a field never borrows from its neighbour
// because an ask is first clamped to 2^width, which clears the field's own guard and nothing else).
//   word x: bits 0..25 memory MB, bit 26 guard, bits 27..30 idle GPUs + 1, bit 31 guard
//   word y: bits 0..10 VRAM GB,   bit 11 guard, bits 12..30 millicpus,    bit 31 guard
// GPUs are stored as idle + 1 against ask + 1, so that a host that can run nothing (no GPUs, or a
// negative component) is the record with GPU field 0: below every ask. Index H of the table holds
// such a record; invalid host indices are redirected there.
constexpr int kMemBits = 26, kIdleShift = 27, kIdleBits = 4, kVramBits = 11, kCpuShift = 12, kCpuBits = 19;
constexpr unsigned int kGuardsX = (1u << kMemBits) | (1u << 31);
constexpr unsigned int kGuardsY = (1u << kVramBits) | (1u << 31);
// Order among runnable replicas (Section 3.4.1) as one 32-bit key per host, smaller first: 14 - idle
// GPUs in the top four bits, below it S / (G R) as the integer S * (840 / G) -- R cancels, and for
// 1 <= G <= 8 that integer orders the ratios exactly. Equal keys: the lower host index.
constexpr int kRatioLcm = 840, kRatioBits = 28;
constexpr int kPackBlock = 256;

struct ExecArgs {
    const int4 *fit;        // [H] (idle GPUs or -1 if the host has none, vram_gb, millicpus, mem_mb)
    const int2 *rank;       // [H] (G, S): what the order among runnable replicas needs
    const uint2 *rec;       // [H + 1] packed form (above)
    const unsigned int *ratio;  // [H + 1] designation key (above)
    const int *wide;        // [ceil(H / kPackBlock)] non-zero: some host of that block does not fit the packed form
    const int4 *requests;
    const int32_t *replica_hosts;
    int32_t *out_executor, *out_can_run;
    long long n_kernels;
    int H;
};

// Gathering six separate arrays per replica costs 18 scattered loads per kernel; packed records
// per host make it 3 (+ the ratio keys when replicas tie on idle GPUs). Both forms are written:
// the 8-byte one and, for cluster states it cannot hold, the general one.
__global__ void __launch_bounds__(kPackBlock) pack_state_kernel(const int32_t *G, const int32_t *S, const int32_t *C,
                                                                const int32_t *AV, const int32_t *AC,
                                                                const int32_t *AM, int H, int4 *fit, int2 *rank,
                                                                uint2 *rec, unsigned int *ratio, int *wide)
{
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    bool too_wide = false;
    if (h <= H) {
        uint2 r = make_uint2(kGuardsX, kGuardsY);
        unsigned int q = 0u;
        if (h < H) {
            const int g = G[h], s = S[h];
            const int4 f = make_int4(g >= 1 ? g - C[h] : -1, AV[h], AC[h], AM[h]);
            fit[h] = f;
            rank[h] = make_int2(g, s);
            if ((f.x | f.y | f.z | f.w) >= 0) {   // otherwise the host runs nothing: GPU field 0
                too_wide = f.x + 1 >= (1 << kIdleBits) || f.y >= (1 << kVramBits) || f.z >= (1 << kCpuBits) ||
                           f.w >= (1 << kMemBits) || g > 8 || s < 0 ||
                           (long long)s * (kRatioLcm / g) >= (1ll << kRatioBits);
                if (!too_wide) {
                    r.x |= (unsigned int)f.w | ((unsigned int)(f.x + 1) << kIdleShift);
                    r.y |= (unsigned int)f.y | ((unsigned int)f.z << kCpuShift);
                    q = ((unsigned int)((1 << kIdleBits) - 2 - f.x) << kRatioBits) | ((unsigned int)s * (unsigned int)(kRatioLcm / g));
                }
            }
        }
        rec[h] = r;
        ratio[h] = q;
    }
    const int any = __syncthreads_or(too_wide);
    if (threadIdx.x == 0 && blockIdx.x * kPackBlock < H) wide[blockIdx.x] = any;
}

// The general form of one kernel's decision: 16-byte capacity records, (G, S) pairs compared by
// cross-multiplication. Gathers go wherever fit / rank point (shared or global memory).
__device__ __forceinline__ void decide_general(const int4 *fit, const int2 *rank, int H, const int4 r, const int (&h)[3],
                                               int &best, int &mask)
{
    const bool sane = (r.x | r.y | r.z | r.w) >= 0;
    int4 f[3];
    bool ok[3];
#pragma unroll
    for (int slot = 0; slot < 3; ++slot) {
        const bool valid = sane && h[slot] >= 0 && h[slot] < H;
        f[slot] = valid ? fit[h[slot]] : make_int4(-1, 0, 0, 0);
        ok[slot] = valid && r.x <= f[slot].x && r.y <= f[slot].y && r.z <= f[slot].z && r.w <= f[slot].w;
    }
    mask = (int)ok[0] | ((int)ok[1] << 1) | ((int)ok[2] << 2);
    best = -1;
    if (mask != 0 && (mask & (mask - 1)) == 0) {
        best = ok[0] ? h[0] : ok[1] ? h[1] : h[2];  // a single runnable replica: no ranking needed
    } else if (mask != 0) {
        int best_idle = 0;
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
            }
        }
    }
}

// The packed form of the same decision. rec / ratio have H + 1 entries.
__device__ __forceinline__ void decide_packed(const uint2 *rec, const unsigned int *ratio, int H, const int4 r,
                                              const int (&h)[3], int &best, int &mask)
{
    // asks as fields; a negative or oversized ask becomes 2^width: it clears the field's guard on
    // every host. (A GPU ask of 15 or more cannot be met by a host that fits the packed form.)
    const unsigned int qx = min((unsigned int)r.w, 1u << kMemBits) + ((min((unsigned int)r.x, (1u << kIdleBits) - 1u) + 1u) << kIdleShift);
    const unsigned int qy = min((unsigned int)r.y, 1u << kVramBits) + (min((unsigned int)r.z, 1u << kCpuBits) << kCpuShift);
    unsigned int key[3];
    mask = 0;
#pragma unroll
    for (int slot = 0; slot < 3; ++slot) {
        const unsigned int idx = min((unsigned int)h[slot], (unsigned int)H);
        const uint2 w = rec[idx];
        const unsigned int dk = ratio[idx];
        const unsigned int lost = (~(w.x - qx) & kGuardsX) | (~(w.y - qy) & kGuardsY);
        key[slot] = lost == 0u ? dk : 0xFFFFFFFFu;   // designation keys are below 15 << 28
        mask |= (lost == 0u ? 1 : 0) << slot;
    }
    // smallest key, then smallest host index among those that have it (runnable slots hold valid indices)
    const unsigned int m = min(min(key[0], key[1]), key[2]);
    const int c0 = key[0] == m ? h[0] : INT_MAX, c1 = key[1] == m ? h[1] : INT_MAX, c2 = key[2] == m ? h[2] : INT_MAX;
    best = mask != 0 ? min(min(c0, c1), c2) : -1;
}

// One kernel per thread and iteration, gathers from the packed tables in global memory (they stay
// in L1 / L2). Used for small batches, for tables too large for shared memory, and for host-id
// arrays that are not 16-byte aligned; large batches take the ring form below. A cluster state
// that the packed form cannot hold (flagged by the packing kernel) takes the general form.
__global__ void __launch_bounds__(512, 2) select_executors_kernel(const ExecArgs a)
{
    const uint2 *rec = a.rec;
    const unsigned int *ratio = a.ratio;
    int wide = 0;
    for (int i = threadIdx.x; i * kPackBlock < a.H; i += blockDim.x) wide |= a.wide[i];
    wide = __syncthreads_or(wide);
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
        const int h[3] = {h_next[0], h_next[1], h_next[2]};
        if (k + stride < a.n_kernels) {
            r_next = __ldg(a.requests + k + stride);
#pragma unroll
            for (int slot = 0; slot < 3; ++slot) h_next[slot] = __ldg(a.replica_hosts + 3 * (k + stride) + slot);
        }
        int best, mask;
        if (wide)
            decide_general(a.fit, a.rank, a.H, r, h, best, mask);
        else
            decide_packed(rec, ratio, a.H, r, h, best, mask);
        a.out_executor[k] = best;
        a.out_can_run[k] = mask;
    }
}

// The same with the two input streams brought in by bulk asynchronous copies: per tile of 512
// kernels one lane of a copy warp issues two copies (8 KiB of requests, 6 KiB of host ids) into a
// ring of shared-memory stages, several tiles ahead of the 512 threads that consume them, so that
// the bytes in flight do not depend on registers or on occupancy. Waits are bounded; a wait that
// runs out makes the block read its remaining tiles with plain loads instead (same results), and
// the copy lane stays until what it issued has landed. The last, partial tile is read with plain
// loads too (a bulk copy's size must be a multiple of 16 bytes).
constexpr int kRingThreads = 512;        // consumers; + one copy warp
constexpr int kRingTile = kRingThreads;  // kernels per stage, one per consumer thread
constexpr int kRingStages = 4;
constexpr uint32_t kRingStageBytes = kRingTile * (16u + 12u);

__global__ void __launch_bounds__(kRingThreads + 32, 2) select_executors_ring_kernel(const ExecArgs a, const int table_bytes)
{
    extern __shared__ __align__(128) unsigned char exec_smem[];
    uint2 *s_rec = reinterpret_cast<uint2 *>(exec_smem);
    unsigned int *s_ratio = reinterpret_cast<unsigned int *>(exec_smem + (size_t)(a.H + 1) * sizeof(uint2));
    unsigned char *ring = exec_smem + table_bytes;   // table_bytes is a multiple of 128
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(ring + (size_t)kRingStages * kRingStageBytes);
    volatile unsigned int *abort_flag = reinterpret_cast<volatile unsigned int *>(bars + 2 * kRingStages);
    const uint32_t full_bar = smem_addr(bars), empty_bar = smem_addr(bars + kRingStages);
    const int tid = threadIdx.x;

    int wide = 0;
    for (int i = tid; i * kPackBlock < a.H; i += blockDim.x) wide |= a.wide[i];
    if (tid == 0) {
        for (int s = 0; s < kRingStages; ++s) {
            mbar_init(full_bar + 8u * s, 1u);
            mbar_init(empty_bar + 8u * s, (uint32_t)(kRingThreads / 32));
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    wide = __syncthreads_or(wide);
    const long long full_tiles = wide ? 0 : a.n_kernels / kRingTile;   // tiles that go through the ring

    if (tid >= kRingThreads) {
        // ---- copy warp: one lane keeps the ring full ----
        if (tid != kRingThreads) return;
        const uint32_t stage0 = smem_addr(ring);
        uint32_t issued = 0;
        bool ok = true;
        for (long long t = blockIdx.x; t < full_tiles; t += gridDim.x, ++issued) {
            const uint32_t s = issued % kRingStages;
            if (issued >= (uint32_t)kRingStages) {
                const uint32_t parity = ((issued / kRingStages) - 1u) & 1u;
                if (!mbar_wait(empty_bar + 8u * s, parity, abort_flag)) {
                    ok = false;
                    break;
                }
            }
            const uint32_t dst = stage0 + s * kRingStageBytes;
            mbar_arrive_expect_tx(full_bar + 8u * s, kRingStageBytes);
            bulk_copy_g2s(dst, a.requests + t * kRingTile, kRingTile * 16u, full_bar + 8u * s);
            bulk_copy_g2s(dst + kRingTile * 16u, a.replica_hosts + t * kRingTile * 3, kRingTile * 12u, full_bar + 8u * s);
        }
        if (!ok) {
            // copies already issued still write into this block's shared memory: stay until they
            // have landed (bounded), so the memory is not handed to another block early
            const uint32_t from = issued > (uint32_t)kRingStages ? issued - kRingStages : 0u;
            const unsigned long long t0 = global_timer_ns();
            for (uint32_t i = from; i < issued; ++i) {
                const uint32_t s = i % kRingStages, parity = (i / kRingStages) & 1u;
                while (!mbar_try_wait(full_bar + 8u * s, parity))
                    if (global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
        return;
    }

    // ---- consumers ----
    if (!wide) {
        for (int i = tid; i <= a.H; i += kRingThreads) {
            s_rec[i] = a.rec[i];
            s_ratio[i] = a.ratio[i];
        }
    }
    // consumers only (the copy lane is already at work): named barrier 1
    asm volatile("bar.sync 1, %0;" ::"n"(kRingThreads) : "memory");

    bool ring_ok = true;
    uint32_t parity = 0u;
    const uint32_t tiles = (uint32_t)full_tiles;   // n_kernels <= 2^40: at most 2^31 tiles
    for (uint32_t t0 = blockIdx.x; t0 < tiles; t0 += kRingStages * gridDim.x, parity ^= 1u) {
#pragma unroll
        for (int s = 0; s < kRingStages; ++s) {
            const uint32_t t = t0 + (uint32_t)s * gridDim.x;
            if (t >= tiles) break;
            const long long k = (long long)t * kRingTile + tid;
            int4 r;
            int h[3];
            // the whole warp takes the same path
            if (ring_ok) ring_ok = __all_sync(0xFFFFFFFFu, mbar_wait(full_bar + 8u * s, parity, abort_flag));
            if (ring_ok) {
                const unsigned char *stage = ring + (size_t)s * kRingStageBytes;
                r = reinterpret_cast<const int4 *>(stage)[tid];
                const int *ids = reinterpret_cast<const int *>(stage + kRingTile * 16u) + 3 * tid;
                h[0] = ids[0];
                h[1] = ids[1];
                h[2] = ids[2];
                __syncwarp();
                if ((tid & 31) == 0) mbar_arrive(empty_bar + 8u * s);
            } else {
                r = __ldg(a.requests + k);
#pragma unroll
                for (int slot = 0; slot < 3; ++slot) h[slot] = __ldg(a.replica_hosts + 3 * k + slot);
            }
            int best, mask;
            decide_packed(s_rec, s_ratio, a.H, r, h, best, mask);
            a.out_executor[k] = best;
            a.out_can_run[k] = mask;
        }
    }
    // what did not go through the ring: the partial last tile, or everything when the cluster
    // state needs the general form
    for (long long k = full_tiles * kRingTile + (long long)blockIdx.x * kRingThreads + tid; k < a.n_kernels;
         k += (long long)gridDim.x * kRingThreads) {
        const int4 r = __ldg(a.requests + k);
        int h[3];
#pragma unroll
        for (int slot = 0; slot < 3; ++slot) h[slot] = __ldg(a.replica_hosts + 3 * k + slot);
        int best, mask;
        if (wide)
            decide_general(a.fit, a.rank, a.H, r, h, best, mask);
        else
            decide_packed(s_rec, s_ratio, a.H, r, h, best, mask);
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
    // stream-ordered temporary: both forms of the host table (36 bytes per host) and the flags
    const int pack_blocks = (H + 1 + kPackBlock - 1) / kPackBlock;
    auto round256 = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t fit_bytes = round256((size_t)H * sizeof(int4));
    const size_t rank_bytes = round256((size_t)H * sizeof(int2));
    const size_t rec_bytes = round256((size_t)(H + 1) * sizeof(uint2));
    const size_t ratio_bytes = round256((size_t)(H + 1) * sizeof(unsigned int));
    const size_t wide_bytes = round256((size_t)pack_blocks * sizeof(int));
    char *packed = nullptr;
    cudaMemPool_t pool = nullptr;
    int rc = library_pool(device, &pool);
    if (rc) return rc;
    cudaError_t e = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&packed),
                                            fit_bytes + rank_bytes + rec_bytes + ratio_bytes + wide_bytes, pool, stream);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(NBOS_ERR_NO_MEMORY, "device allocation failed: %s", cudaGetErrorString(e));
    }
    int4 *fit = reinterpret_cast<int4 *>(packed);
    int2 *rank = reinterpret_cast<int2 *>(packed + fit_bytes);
    uint2 *rec = reinterpret_cast<uint2 *>(packed + fit_bytes + rank_bytes);
    unsigned int *ratio = reinterpret_cast<unsigned int *>(packed + fit_bytes + rank_bytes + rec_bytes);
    int *wide = reinterpret_cast<int *>(packed + fit_bytes + rank_bytes + rec_bytes + ratio_bytes);
    pack_state_kernel<<<pack_blocks, kPackBlock, 0, stream>>>(state->gpus_total, state->gpus_subscribed,
                                                              state->gpus_committed, state->vram_gb,
                                                              state->millicpus, state->mem_mb, H, fit, rank, rec, ratio, wide);
    e = cudaGetLastError();
    if (e == cudaSuccess) {
        ExecArgs a{fit, rank, rec, ratio, wide, reinterpret_cast<const int4 *>(requests), replica_hosts,
                   out_executor, out_can_run, n_kernels, H};
        // the ring form pays from about half a million kernels on (measured: never slower than
        // the plain form from 2^20 kernels, 15 - 25 % faster at 2^22 and above)
        const size_t table_bytes = ((size_t)(H + 1) * (sizeof(uint2) + sizeof(unsigned int)) + 127) & ~(size_t)127;
        const size_t ring_smem = table_bytes + (size_t)kRingStages * kRingStageBytes + 2 * kRingStages * 8 + 16;
        const bool use_ring = ring_smem <= 110 * 1024 && aligned16(replica_hosts) && n_kernels >= (1ll << 19);
        if (use_ring) {
            e = cudaFuncSetAttribute(select_executors_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring_smem);
            if (e == cudaSuccess)
                select_executors_ring_kernel<<<sms * 2, kRingThreads + 32, ring_smem, stream>>>(a, (int)table_bytes);
        } else {
            long long blocks = (n_kernels + 511) / 512;
            if (blocks > (long long)sms * 4) blocks = (long long)sms * 4;
            select_executors_kernel<<<(unsigned int)blocks, 512, 0, stream>>>(a);
        }
        e = cudaGetLastError();
    }
    cudaFreeAsync(packed, stream);
    if (e != cudaSuccess) return cuda_fail(e, "executor selection launch");
    return NBOS_OK;
}
