// Batched placement kernel for sm_100a.
//
// For every (request, host) pair: the feasibility test (Section 3.2.1 capacity in four
// resources; Section 3.4.1 SR limit and Section 3.2.3 idle test, both folded into the host's
// `gmax` when the snapshot was derived) and the ranking key A + g * B of Section 3.4.1's default
// policy; per request the three smallest keys among feasible hosts. The key carries the host id
// in its low bits, so keys are unique, ties go to the lower id, and any evaluation order gives
// the same three hosts.
//
// Shape of one thread block (256 compute threads + 1 copy warp):
//   - the copy warp streams host tiles (feasibility quads + key pairs) from global memory into
//     a ring of shared-memory stages with cp.async.bulk, completion signalled on mbarriers;
//   - the compute threads are cut into groups of L lanes (L = 1..32, a power of two). A group
//     owns Q requests at a time (request fields live in registers, loaded with one 128-bit
//     load each); its lanes stride the hosts of each tile, every lane keeps a sorted best-three
//     per request in registers; after the last tile the L lanes are merged with xor-shuffles.
//     With L = 1 every lane of a warp reads the same host record (a shared-memory broadcast)
//     and no shuffle is needed; with L = 32 a warp serves one request group.
//   - optionally the hosts are cut into K slices handled by different blocks; those write their
//     best-three keys to a candidate buffer that a second kernel merges.
// Every wait on an mbarrier is bounded; when one runs out the block raises the snapshot's
// sticky status word and leaves without touching the barrier again.
#include <limits.h>

#include <mutex>

#include "nbos_internal.h"

namespace nbos {
namespace {

constexpr int kComputeThreads = 256;
constexpr int kComputeWarps = kComputeThreads / 32;
constexpr int kThreads = kComputeThreads + 32;  // + the copy warp
constexpr int kStages = 3;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

struct PlaceParams {
    const int4 *feas;       // [N][Hpad]
    const void *ab;         // [N][Hpad] pairs (A, B)
    const int4 *requests;   // [N * B]
    int32_t *out_hosts;     // [N * B * 3]
    int32_t *out_found;     // [N * B] or null
    void *cand;             // [K][N * B][3] keys, only when K > 1
    unsigned int *status;
    long long B, total;     // requests per snapshot, N * B
    int N, Hpad;
    int tile_hosts, tiles_total, K, req_ctas;
    unsigned int id_mask;
    int max_q;
};

template <typename KeyT> struct KeyTraits;
template <> struct KeyTraits<unsigned int> {
    using Pair = uint2;
    static constexpr unsigned int kInf = 0xFFFFFFFFu;
};
template <> struct KeyTraits<unsigned long long> {
    using Pair = ulonglong2;
    static constexpr unsigned long long kInf = 0xFFFFFFFFFFFFFFFFull;
};

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bulk asynchronous copy global -> shared of `bytes` (multiple of 16, both addresses 16-byte
// aligned); completion is counted on `bar`. No multicast.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes,
                                              uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

// Bounded wait. Returns false when the wait ran out or another thread of the block gave up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity,
                                            volatile unsigned int *abort_flag)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > kWaitLimitNs) {
            *abort_flag = 1u;
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity,
                                          volatile unsigned int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag);
}

// ---- best-three bookkeeping ---------------------------------------------------------------
// (t1 <= t2 <= t3) := the three smallest of {t1, t2, t3, k}
template <typename KeyT>
__device__ __forceinline__ void insert3(KeyT &t1, KeyT &t2, KeyT &t3, KeyT k)
{
    const KeyT hi1 = max(t1, k);
    t1 = min(t1, k);
    const KeyT hi2 = max(t2, hi1);
    t2 = min(t2, hi1);
    t3 = min(t3, hi2);
}

// ---- the list of passes a block makes over its share of the requests ----------------------
// A block owns the flattened request range [lo, hi) of [0, N * B). It is cut at snapshot
// boundaries and then into passes of Q * groups requests, Q the largest power of two <= max_q
// that still fills every lane (or 1 for the ragged tail). Copy warp and compute threads walk
// the same list.
struct PassList {
    long long cursor, hi, B;
    int groups, max_q;
    __device__ bool next(int &n, long long &first, int &count, int &q)
    {
        if (cursor >= hi) return false;
        n = (int)(cursor / B);
        long long end = (long long)(n + 1) * B;
        if (end > hi) end = hi;
        const long long rem = end - cursor;
        q = max_q;
        while (q > 1 && (long long)q * groups > rem) q >>= 1;
        const long long cap = (long long)q * groups;
        count = (int)(rem < cap ? rem : cap);
        first = cursor;  // flattened index n * B + r
        cursor += count;
        return true;
    }
};

__device__ __forceinline__ void block_request_range(const PlaceParams &p, int cr, long long &lo,
                                                    long long &hi)
{
    // split in units of 32 requests so that a warp's 128-bit loads start on a 512-byte line
    const long long units = (p.total + 31) >> 5;
    lo = (units * cr / p.req_ctas) << 5;
    hi = (units * (cr + 1) / p.req_ctas) << 5;
    if (lo > p.total) lo = p.total;
    if (hi > p.total) hi = p.total;
}

// ---- one pass: Q requests per group through all tiles of the block's host slice ------------
template <int Q, int L, typename KeyT>
__device__ __forceinline__ bool run_pass(const PlaceParams &p, unsigned char *stages,
                                         uint32_t stage_bytes, uint32_t full_bar,
                                         uint32_t empty_bar, volatile unsigned int *abort_flag,
                                         uint32_t &ring_pos, int tile_begin, int tile_end,
                                         int slice, int n, long long first, int count)
{
    using Pair = typename KeyTraits<KeyT>::Pair;
    constexpr KeyT kInf = KeyTraits<KeyT>::kInf;
    constexpr int kGroups = kComputeThreads / L;
    const int tid = threadIdx.x;
    const int sub = tid % L;
    const int grp = tid / L;
    const int lane = tid & 31;

    int g[Q], v[Q], c[Q], m[Q];
    KeyT t1[Q], t2[Q], t3[Q];
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        const int idx = q * kGroups + grp;
        int4 r = make_int4(INT_MAX, 0, 0, 0);
        if (idx < count) {
            r = __ldg(p.requests + first + idx);
            if ((r.x | r.y | r.z | r.w) < 0) r.x = INT_MAX;  // a negative ask fits nowhere
        }
        g[q] = r.x; v[q] = r.y; c[q] = r.z; m[q] = r.w;
        t1[q] = kInf; t2[q] = kInf; t3[q] = kInf;
    }

    const int T = p.tile_hosts;
    for (int t = tile_begin; t < tile_end; ++t, ++ring_pos) {
        const uint32_t s = ring_pos % kStages;
        const uint32_t parity = (ring_pos / kStages) & 1u;
        if (!mbar_wait(full_bar + 8u * s, parity, abort_flag)) return false;
        const int4 *F = reinterpret_cast<const int4 *>(stages + (size_t)s * stage_bytes);
        const Pair *AB = reinterpret_cast<const Pair *>(stages + (size_t)s * stage_bytes + (size_t)T * 16);
        int hosts = p.Hpad - t * T;
        if (hosts > T) hosts = T;
#pragma unroll 2
        for (int i = sub; i < hosts; i += L) {
            const int4 f = F[i];
            const Pair ab = AB[i];
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                const bool ok = (g[q] <= f.x) & (v[q] <= f.y) & (c[q] <= f.z) & (m[q] <= f.w);
                const KeyT key = (KeyT)(unsigned int)g[q] * ab.y + ab.x;
                if (ok && key < t3[q]) {
                    t3[q] = max(t2[q], key);
                    t2[q] = min(t2[q], max(t1[q], key));
                    t1[q] = min(t1[q], key);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + 8u * s);
    }

    // merge the L lanes of a group (keys are unique, so the order of merging does not matter)
#pragma unroll
    for (int mask = 1; mask < L; mask <<= 1) {
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const KeyT o1 = __shfl_xor_sync(0xFFFFFFFFu, t1[q], mask);
            const KeyT o2 = __shfl_xor_sync(0xFFFFFFFFu, t2[q], mask);
            const KeyT o3 = __shfl_xor_sync(0xFFFFFFFFu, t3[q], mask);
            insert3(t1[q], t2[q], t3[q], o1);
            insert3(t1[q], t2[q], t3[q], o2);
            insert3(t1[q], t2[q], t3[q], o3);
        }
    }

    if (sub == 0) {
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int idx = q * kGroups + grp;
            if (idx >= count) continue;
            const long long r = first + idx;
            if (p.K > 1) {
                KeyT *cand = reinterpret_cast<KeyT *>(p.cand) + ((long long)slice * p.total + r) * 3;
                cand[0] = t1[q]; cand[1] = t2[q]; cand[2] = t3[q];
            } else {
                int32_t *o = p.out_hosts + r * 3;
                o[0] = t1[q] == kInf ? -1 : (int)((unsigned int)t1[q] & p.id_mask);
                o[1] = t2[q] == kInf ? -1 : (int)((unsigned int)t2[q] & p.id_mask);
                o[2] = t3[q] == kInf ? -1 : (int)((unsigned int)t3[q] & p.id_mask);
                if (p.out_found)
                    p.out_found[r] = (t1[q] != kInf) + (t2[q] != kInf) + (t3[q] != kInf);
            }
        }
    }
    (void)n;
    return true;
}

template <int L, typename KeyT, int MAXQ>
__global__ void __launch_bounds__(kThreads, 2) place_kernel(const __grid_constant__ PlaceParams p)
{
    using Pair = typename KeyTraits<KeyT>::Pair;
    extern __shared__ __align__(128) unsigned char smem[];
    const int T = p.tile_hosts;
    const uint32_t stage_bytes = (uint32_t)T * (16u + (uint32_t)sizeof(Pair));
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + (size_t)kStages * stage_bytes);
    volatile unsigned int *abort_flag = reinterpret_cast<volatile unsigned int *>(bars + 2 * kStages);
    const uint32_t full_bar = smem_addr(bars);
    const uint32_t empty_bar = smem_addr(bars + kStages);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar + 8u * s, 1u);
            mbar_init(empty_bar + 8u * s, (uint32_t)kComputeWarps);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int slice = blockIdx.x / p.req_ctas;
    const int cr = blockIdx.x % p.req_ctas;
    const int tile_begin = (int)((long long)p.tiles_total * slice / p.K);
    const int tile_end = (int)((long long)p.tiles_total * (slice + 1) / p.K);
    PassList passes;
    block_request_range(p, cr, passes.cursor, passes.hi);
    passes.B = p.B;
    passes.groups = kComputeThreads / L;
    passes.max_q = p.max_q < MAXQ ? p.max_q : MAXQ;

    int n, count, q;
    long long first;

    if (threadIdx.x >= kComputeThreads) {
        // ---- copy warp: one lane walks the same pass list and keeps the ring full ----
        if (threadIdx.x != kComputeThreads) return;
        const uint32_t stage0 = smem_addr(smem);
        uint32_t issued = 0;
        bool ok = true;
        while (ok && passes.next(n, first, count, q)) {
            const int4 *feas_n = p.feas + (size_t)n * p.Hpad;
            const Pair *ab_n = reinterpret_cast<const Pair *>(p.ab) + (size_t)n * p.Hpad;
            for (int t = tile_begin; t < tile_end; ++t, ++issued) {
                const uint32_t s = issued % kStages;
                if (issued >= (uint32_t)kStages) {
                    const uint32_t parity = ((issued / kStages) - 1u) & 1u;
                    if (!mbar_wait(empty_bar + 8u * s, parity, abort_flag)) {
                        ok = false;
                        break;
                    }
                }
                int hosts = p.Hpad - t * T;
                if (hosts > T) hosts = T;
                const uint32_t bytes_f = (uint32_t)hosts * 16u;
                const uint32_t bytes_k = (uint32_t)hosts * (uint32_t)sizeof(Pair);
                const uint32_t dst = stage0 + s * stage_bytes;
                mbar_arrive_expect_tx(full_bar + 8u * s, bytes_f + bytes_k);
                bulk_copy_g2s(dst, feas_n + (size_t)t * T, bytes_f, full_bar + 8u * s);
                bulk_copy_g2s(dst + (uint32_t)T * 16u, ab_n + (size_t)t * T, bytes_k, full_bar + 8u * s);
            }
        }
        if (!ok) {
            atomicOr(p.status, 1u);
            // copies already issued still write into this block's shared memory: stay until
            // they have landed (bounded), so the memory is not handed to another block early
            const uint32_t from = issued > (uint32_t)kStages ? issued - kStages : 0u;
            const unsigned long long t0 = global_timer_ns();
            for (uint32_t i = from; i < issued; ++i) {
                const uint32_t s = i % kStages, parity = (i / kStages) & 1u;
                while (!mbar_try_wait(full_bar + 8u * s, parity))
                    if (global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
        return;
    }

    // ---- compute threads ----
    uint32_t ring_pos = 0;
    bool ok = true;
    while (ok && passes.next(n, first, count, q)) {
#define NBOS_PASS(QV)                                                                         \
    ok = run_pass<QV, L, KeyT>(p, smem, stage_bytes, full_bar, empty_bar, abort_flag, ring_pos, \
                               tile_begin, tile_end, slice, n, first, count)
        if (MAXQ >= 8 && q == 8) NBOS_PASS(8);
        else if (MAXQ >= 4 && q == 4) NBOS_PASS(4);
        else if (MAXQ >= 2 && q == 2) NBOS_PASS(2);
        else NBOS_PASS(1);
#undef NBOS_PASS
    }
    if (!ok) atomicOr(p.status, 1u);
}

// a7: merge the K per-slice candidate triples of each request.
template <typename KeyT>
__global__ void __launch_bounds__(256) merge_kernel(const KeyT *cand, int K, long long total,
                                                    unsigned int id_mask, int32_t *out_hosts,
                                                    int32_t *out_found)
{
    constexpr KeyT kInf = KeyTraits<KeyT>::kInf;
    for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < total;
         r += (long long)gridDim.x * blockDim.x) {
        KeyT t1 = kInf, t2 = kInf, t3 = kInf;
        for (int k = 0; k < K; ++k) {
            const KeyT *c = cand + ((long long)k * total + r) * 3;
            insert3(t1, t2, t3, c[0]);
            insert3(t1, t2, t3, c[1]);
            insert3(t1, t2, t3, c[2]);
        }
        int32_t *o = out_hosts + r * 3;
        o[0] = t1 == kInf ? -1 : (int)((unsigned int)t1 & id_mask);
        o[1] = t2 == kInf ? -1 : (int)((unsigned int)t2 & id_mask);
        o[2] = t3 == kInf ? -1 : (int)((unsigned int)t3 & id_mask);
        if (out_found) out_found[r] = (t1 != kInf) + (t2 != kInf) + (t3 != kInf);
    }
}

using KernelFn = void (*)(const PlaceParams);

template <typename KeyT, int MAXQ>
KernelFn pick_kernel(int L)
{
    switch (L) {
        case 1: return place_kernel<1, KeyT, MAXQ>;
        case 2: return place_kernel<2, KeyT, MAXQ>;
        case 4: return place_kernel<4, KeyT, MAXQ>;
        case 8: return place_kernel<8, KeyT, MAXQ>;
        case 16: return place_kernel<16, KeyT, MAXQ>;
        case 32: return place_kernel<32, KeyT, MAXQ>;
    }
    return nullptr;
}

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

}  // namespace

int launch_place(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                 int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                 const nbos_launch_config *cfg)
{
    const long long total = (long long)s->N * batch;
    if (total == 0) return NBOS_OK;
    const bool k64 = s->key.key_bits == 64;
    const int max_q_kernel = k64 ? 4 : 8;
    const int pair_bytes = k64 ? 16 : 8;

    nbos_launch_config c = {};
    if (cfg) c = *cfg;
    if (c.reserved[0] | c.reserved[1] | c.reserved[2]) return fail(NBOS_ERR_INVALID_ARG, "launch config: reserved fields must be 0");
    if (c.lanes_per_request && !(is_pow2(c.lanes_per_request) && c.lanes_per_request <= 32))
        return fail(NBOS_ERR_INVALID_ARG, "lanes_per_request must be 1,2,4,8,16 or 32");
    if (c.requests_per_lane && !(is_pow2(c.requests_per_lane) && c.requests_per_lane <= 8))
        return fail(NBOS_ERR_INVALID_ARG, "requests_per_lane must be 1,2,4 or 8");
    if (c.host_split < 0 || c.grid_blocks < 0 || c.tile_hosts < 0 || (c.tile_hosts & 31))
        return fail(NBOS_ERR_INVALID_ARG, "launch config: negative field or tile_hosts not a multiple of 32");

    // tile: as many hosts as fit the stage budget, at most the whole (padded) table
    int T = c.tile_hosts ? c.tile_hosts : 1024;
    if (T > s->Hpad) T = s->Hpad;
    const int max_tile = (64 * 1024) / (16 + pair_bytes) / 32 * 32;  // <= 64 KB per stage
    if (T > max_tile) T = max_tile;
    const int tiles_total = (s->Hpad + T - 1) / T;

    // lanes per request: as few as still give every SM enough resident threads
    const long long want_threads = (long long)s->sm_count * 2 * kComputeThreads;
    int L = c.lanes_per_request;
    if (!L) {
        L = 1;
        while (L < 32 && total * L < want_threads) L <<= 1;
    }
    int K = c.host_split;
    if (!K) {
        K = 1;
        if (total * L < want_threads) {
            long long k = (want_threads + total * L - 1) / (total * L);
            K = (int)(k < tiles_total ? k : tiles_total);
        }
    }
    if (K > tiles_total) K = tiles_total;
    if (K < 1) K = 1;

    int max_q = c.requests_per_lane ? c.requests_per_lane : max_q_kernel;
    if (max_q > max_q_kernel) max_q = max_q_kernel;

    KernelFn fn = k64 ? pick_kernel<unsigned long long, 4>(L) : pick_kernel<unsigned int, 8>(L);
    if (!fn) return fail(NBOS_ERR_INVALID_ARG, "no kernel for this launch shape");
    const size_t smem = (size_t)kStages * T * (16 + pair_bytes) + 2 * kStages * 8 + 16;
    NBOS_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    NBOS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, smem));
    if (per_sm < 1) return fail(NBOS_ERR_CUDA, "placement kernel does not fit on an SM (%zu bytes of shared memory)", smem);

    const int groups = kComputeThreads / L;
    long long req_ctas = (total + groups - 1) / groups;  // at least one request per group
    long long cap = (long long)s->sm_count * per_sm / K;
    if (cap < 1) cap = 1;
    if (c.grid_blocks) cap = c.grid_blocks;
    if (req_ctas > cap) req_ctas = cap;

    PlaceParams p;
    p.feas = s->d_feas;
    p.ab = s->d_ab;
    p.requests = reinterpret_cast<const int4 *>(d_requests);
    p.out_hosts = d_out_hosts;
    p.out_found = d_out_found;
    p.cand = nullptr;
    p.status = s->d_status;
    p.B = batch;
    p.total = total;
    p.N = s->N;
    p.Hpad = s->Hpad;
    p.tile_hosts = T;
    p.tiles_total = tiles_total;
    p.K = K;
    p.req_ctas = (int)req_ctas;
    p.id_mask = (1u << s->key.bits_id) - 1u;
    p.max_q = max_q;

    if (K > 1) {
        const size_t cand_bytes = (size_t)K * (size_t)total * 3 * (k64 ? 8 : 4);
        cudaError_t e = cudaMallocAsync(&p.cand, cand_bytes, stream);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(NBOS_ERR_NO_MEMORY, "could not allocate %zu bytes for slice candidates: %s", cand_bytes,
                        cudaGetErrorString(e));
        }
    }
    fn<<<(unsigned int)(req_ctas * K), kThreads, smem, stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && K > 1) {
        long long blocks = (total + 255) / 256;
        if (blocks > (long long)s->sm_count * 8) blocks = (long long)s->sm_count * 8;
        if (k64)
            merge_kernel<unsigned long long><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned long long *>(p.cand), K, total, p.id_mask, d_out_hosts, d_out_found);
        else
            merge_kernel<unsigned int><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned int *>(p.cand), K, total, p.id_mask, d_out_hosts, d_out_found);
        e = cudaGetLastError();
    }
    if (p.cand) cudaFreeAsync(p.cand, stream);
    if (e != cudaSuccess) return cuda_fail(e, "placement launch");
    return NBOS_OK;
}


// ---- placement without any allocation ------------------------------------------------------
// The host-split launch shape needs a candidate buffer (K slices x requests x 3 keys). The
// ordinary entry points take it from the stream-ordered allocator; this variant keeps it in a
// fixed array that is part of the loaded module, for callers that must not allocate.
namespace {

constexpr size_t kStaticCandBytes = NBOS_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_cand[kStaticCandBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_cand_ptr[kMaxDevices] = {};  // device address of g_static_cand, per device

// Host code cannot use the name g_static_cand as a pointer: on the host it only stands for the
// symbol. The device address is looked up once per device, with that device current.
int static_cand_address(int device, void **out)
{
    if (device < 0 || device >= kMaxDevices) return fail(NBOS_ERR_INVALID_ARG, "device index %d not supported", device);
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_cand_ptr[device]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_cand);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static candidate buffer)");
        if (!ptr) return fail(NBOS_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_static_cand_ptr[device] = ptr;
    }
    *out = g_static_cand_ptr[device];
    return NBOS_OK;
}

}  // namespace

int launch_place_static(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                        int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                        int host_split)
{
    const long long total = (long long)s->N * batch;
    if (total == 0) return NBOS_OK;
    int device = -1;
    NBOS_CUDA_TRY(cudaGetDevice(&device));
    if (device != s->device)
        return fail(NBOS_ERR_INVALID_ARG, "snapshot was created on device %d, current device is %d", s->device, device);
    const bool k64 = s->key.key_bits == 64;
    const int key_bytes = k64 ? 8 : 4;
    const int pair_bytes = k64 ? 16 : 8;

    // host slices: K tiles-aligned slices of the padded host table
    int K = host_split ? host_split : 4;
    if (K > s->Hpad / 32) K = s->Hpad / 32;
    if (K < 1) K = 1;
    int T = (s->Hpad / K) / 32 * 32;
    if (T > 1024) T = 1024;
    if (T < 32) T = 32;
    const int tiles_total = (s->Hpad + T - 1) / T;
    if (K > tiles_total) K = tiles_total;

    const size_t cand_bytes = (size_t)K * (size_t)total * 3 * key_bytes;
    if (K > 1 && cand_bytes > kStaticCandBytes)
        return fail(NBOS_ERR_NO_MEMORY,
                    "nbos_place_batch_noalloc: %lld requests x %d host slices need %zu bytes of candidates, "
                    "the built-in buffer holds %zu; use fewer slices, a smaller batch, or nbos_place_batch",
                    total, K, cand_bytes, kStaticCandBytes);
    void *cand = nullptr;
    int rc = static_cand_address(device, &cand);
    if (rc) return rc;

    const int L = 32;  // small batches are what this shape is for: one warp per request group
    KernelFn fn = k64 ? pick_kernel<unsigned long long, 4>(L) : pick_kernel<unsigned int, 8>(L);
    const size_t smem = (size_t)kStages * T * (16 + pair_bytes) + 2 * kStages * 8 + 16;
    NBOS_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    NBOS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, smem));
    if (per_sm < 1) return fail(NBOS_ERR_CUDA, "placement kernel does not fit on an SM");
    const int groups = kComputeThreads / L;
    long long req_ctas = (total + groups - 1) / groups;
    long long cap = (long long)s->sm_count * per_sm / K;
    if (cap < 1) cap = 1;
    if (req_ctas > cap) req_ctas = cap;

    PlaceParams p;
    p.feas = s->d_feas;
    p.ab = s->d_ab;
    p.requests = reinterpret_cast<const int4 *>(d_requests);
    p.out_hosts = d_out_hosts;
    p.out_found = d_out_found;
    p.cand = K > 1 ? cand : nullptr;
    p.status = s->d_status;
    p.B = batch;
    p.total = total;
    p.N = s->N;
    p.Hpad = s->Hpad;
    p.tile_hosts = T;
    p.tiles_total = tiles_total;
    p.K = K;
    p.req_ctas = (int)req_ctas;
    p.id_mask = (1u << s->key.bits_id) - 1u;
    p.max_q = k64 ? 4 : 8;

    // Nothing in the buffer has to start at zero: the placement kernel writes all K * total * 3
    // candidate slots of this call before the merge kernel (next on the stream) reads them.
    fn<<<(unsigned int)(req_ctas * K), kThreads, smem, stream>>>(p);
    NBOS_CUDA_TRY(cudaGetLastError());
    if (K > 1) {
        long long blocks = (total + 255) / 256;
        if (blocks > (long long)s->sm_count * 8) blocks = (long long)s->sm_count * 8;
        if (k64)
            merge_kernel<unsigned long long><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned long long *>(cand), K, total, p.id_mask, d_out_hosts, d_out_found);
        else
            merge_kernel<unsigned int><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned int *>(cand), K, total, p.id_mask, d_out_hosts, d_out_found);
        NBOS_CUDA_TRY(cudaGetLastError());
    }
    return NBOS_OK;
}

}  // namespace nbos
