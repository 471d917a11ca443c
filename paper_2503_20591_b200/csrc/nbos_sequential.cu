// Sequential placement with commits (Sections 3.2.1, 3.4.1): requests of a snapshot are placed one
// after the other, and a request that found three hosts adds its GPUs to their subscribed count
// before the next request is looked at. The dependence is serial over requests, so the
// parallelism is over hosts (all hosts of the snapshot are evaluated for one request at a time)
// and over snapshots (one thread block each).
//
// One block of T = 256, 512 or 1,024 threads owns a snapshot (about four hosts per thread; up to
// eight at 8,192 hosts). Thread t owns hosts t, t + T, ...: the fields a commit changes (room under
// the SR limit, key intercept A) live in registers, the static ones in shared memory. Per
// request: every thread ranks its own hosts, each warp extracts its three smallest keys with
// three warp-wide integer minimum reductions (keys are unique, the lane that held the minimum
// pops it) and writes them to shared memory; behind one block barrier every warp does the same
// over the warps' triples for itself, thread 0 writes the result, and the owners of the three
// winning hosts update them. One block barrier per request.
//
// Tables beyond 8,192 hosts (what one block's registers and shared memory hold) are spread over a
// thread-block cluster of 2, 4 or 8 blocks, each owning a contiguous run of the hosts. Per request
// every block finds the best three of its hosts as above, writes them into the shared memory of
// every block of the cluster (distributed shared memory: plain remote stores, no multicast), one
// cluster-wide barrier follows, and every block merges the 2 to 8 triples for itself; the owners of
// the three winners update them. The cost per request is that of the one-block form plus the
// cluster barrier; what the cluster buys is room (up to 65,536 hosts), not speed.
#include <limits.h>

#include <cooperative_groups.h>

#include "nbos_internal.h"
#include "nbos_ptx.cuh"

namespace nbos {
namespace {

constexpr int kSeqThreads = 1024;
constexpr int kSeqWarps = kSeqThreads / 32;

struct SeqParams {
    const int4 *feas;   // [N][Hpad] host order: (gmax, vram, cpu, mem)
    const void *ab;     // [N][Hpad] host order: (A, B)
    const int4 *seq;    // [N][Hpad] host order: (min(G, idle), cap - S, S, 0)
    const int4 *requests;
    int32_t *out_hosts, *out_found, *out_subscribed;
    long long B;
    int H, Hpad;
    unsigned int id_mask;
};

template <typename KeyT> struct SeqKey;
template <> struct SeqKey<unsigned int> {
    using Pair = uint2;
    static constexpr unsigned int kInf = 0xFFFFFFFFu;
    static __device__ __forceinline__ unsigned int warp_min(unsigned int k) { return __reduce_min_sync(0xFFFFFFFFu, k); }
};
template <> struct SeqKey<unsigned long long> {
    using Pair = ulonglong2;
    static constexpr unsigned long long kInf = 0xFFFFFFFFFFFFFFFFull;
    static __device__ __forceinline__ unsigned long long warp_min(unsigned long long k)
    {
        const unsigned int hi = __reduce_min_sync(0xFFFFFFFFu, (unsigned int)(k >> 32));
        const unsigned int lo = __reduce_min_sync(0xFFFFFFFFu, (unsigned int)(k >> 32) == hi ? (unsigned int)k : 0xFFFFFFFFu);
        return ((unsigned long long)hi << 32) | lo;
    }
};


// The three smallest of the warp's keys (each lane brings a sorted triple); every lane returns them.
template <typename KeyT>
__device__ __forceinline__ void warp_best3(KeyT k1, KeyT k2, KeyT k3, KeyT &w1, KeyT &w2, KeyT &w3)
{
    constexpr KeyT kInf = SeqKey<KeyT>::kInf;
    KeyT w[3];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        const KeyT m = SeqKey<KeyT>::warp_min(k1);
        w[i] = m;
        if (k1 == m && m != kInf) {  // unique keys: exactly one lane pops
            k1 = k2;
            k2 = k3;
            k3 = kInf;
        }
    }
    w1 = w[0]; w2 = w[1]; w3 = w[2];
}

// T threads, HPT hosts per thread (1..8). Static per-host fields in shared memory: (vram, cpu, mem,
// g_cap) as int4 and B; dynamic in registers: room = cap - S, A, and the GPUs added so far.
// One block barrier per request: every warp writes its best three, and behind the barrier every
// warp reduces the T / 32 triples for itself (the buffer alternates with the request's parity, so
// a warp that runs ahead never overwrites what a slower one still reads).
template <typename KeyT, int HPT, int T>
__global__ void __launch_bounds__(T) place_sequential_kernel(const SeqParams p)
{
    using Pair = typename SeqKey<KeyT>::Pair;
    constexpr KeyT kInf = SeqKey<KeyT>::kInf;
    constexpr int W = T / 32;
    extern __shared__ __align__(16) unsigned char seq_smem[];
    int4 *s_cap = reinterpret_cast<int4 *>(seq_smem);                              // [HPT * T]
    KeyT *s_B = reinterpret_cast<KeyT *>(seq_smem + (size_t)HPT * T * sizeof(int4));  // [HPT * T]
    __shared__ KeyT s_warp[2][W][3];

    const int n = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t row = (size_t)n * p.Hpad;

    int gmax_now[HPT], room[HPT], added[HPT];  // gmax_now = min(g_cap, room): largest ask that fits now
    KeyT A[HPT];
#pragma unroll
    for (int u = 0; u < HPT; ++u) {
        const int h = tid + u * T;
        int4 cap = make_int4(0, 0, 0, -1);
        KeyT b = 0;
        room[u] = -1;
        added[u] = 0;
        A[u] = kInf;
        if (h < p.Hpad) {
            const int4 f = p.feas[row + h];
            const int4 sq = p.seq[row + h];
            const Pair ab = reinterpret_cast<const Pair *>(p.ab)[row + h];
            cap = make_int4(f.y, f.z, f.w, sq.x);
            room[u] = sq.y;
            // a host that takes nothing now has no key yet (A = h, B = 0): it can never take anything
            // later either, because commits only shrink the room
            A[u] = f.x >= 0 ? (KeyT)ab.x : kInf;
            b = ab.y;
            if (f.x < 0) room[u] = -1;
        }
        gmax_now[u] = min(cap.w, room[u]);
        s_cap[h] = cap;
        s_B[h] = b;
    }
    __syncthreads();

    const int4 *req = p.requests + (size_t)n * p.B;
    int4 next = p.B > 0 ? __ldg(req) : make_int4(-1, 0, 0, 0);
    for (long long r = 0; r < p.B; ++r) {
        const int4 q = next;
        if (r + 1 < p.B) next = __ldg(req + r + 1);
        const int par = (int)(r & 1);
        const bool sane = (q.x | q.y | q.z | q.w) >= 0;
        KeyT k1 = kInf, k2 = kInf, k3 = kInf;
        if (sane) {
#pragma unroll
            for (int u = 0; u < HPT; ++u) {
                const int h = tid + u * T;
                const int4 cap = s_cap[h];
                const bool ok = q.x <= gmax_now[u] && q.y <= cap.x && q.z <= cap.y && q.w <= cap.z;
                const KeyT key = ok ? (KeyT)(A[u] + (KeyT)(unsigned int)q.x * s_B[h]) : kInf;
                insert3(k1, k2, k3, key);
            }
        }
        KeyT b1, b2, b3;
        warp_best3(k1, k2, k3, b1, b2, b3);
        if (W > 1) {
            if (lane == 0) {
                s_warp[par][warp][0] = b1;
                s_warp[par][warp][1] = b2;
                s_warp[par][warp][2] = b3;
            }
            __syncthreads();
            const bool has = lane < W;
            warp_best3(has ? s_warp[par][has ? lane : 0][0] : kInf, has ? s_warp[par][has ? lane : 0][1] : kInf,
                       has ? s_warp[par][has ? lane : 0][2] : kInf, b1, b2, b3);
        }
        if (tid == 0) {
            const long long o = (long long)n * p.B + r;
            p.out_hosts[o * 3 + 0] = b1 == kInf ? -1 : (int)((unsigned int)b1 & p.id_mask);
            p.out_hosts[o * 3 + 1] = b2 == kInf ? -1 : (int)((unsigned int)b2 & p.id_mask);
            p.out_hosts[o * 3 + 2] = b3 == kInf ? -1 : (int)((unsigned int)b3 & p.id_mask);
            if (p.out_found) p.out_found[o] = (b1 != kInf) + (b2 != kInf) + (b3 != kInf);
        }
        // commit: only a kernel that got all three replicas is created
        if (b3 != kInf && q.x > 0) {
            const KeyT best[3] = {b1, b2, b3};
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const int h = (int)((unsigned int)best[i] & p.id_mask);
                if ((h & (T - 1)) == tid) {
                    const int u0 = h / T;
#pragma unroll
                    for (int u = 0; u < HPT; ++u)
                        if (u == u0) {
                            room[u] -= q.x;
                            gmax_now[u] = min(s_cap[h].w, room[u]);
                            added[u] += q.x;
                            A[u] += (KeyT)(unsigned int)q.x * s_B[h];
                        }
                }
            }
        }
    }
    if (p.out_subscribed) {
#pragma unroll
        for (int u = 0; u < HPT; ++u) {
            const int h = tid + u * T;
            if (h < p.H) p.out_subscribed[(size_t)n * p.H + h] = p.seq[row + h].z + added[u];
        }
    }
}

// The cluster form: blockIdx.x = snapshot * C + rank; block `rank` of the cluster owns hosts
// [rank * kClusterHosts, (rank + 1) * kClusterHosts). Every thread of every block executes the same
// number of cluster barriers (one per request and one before leaving), whatever the data.
constexpr int kClusterHpt = 8;
constexpr int kClusterHosts = kClusterHpt * kSeqThreads;   // hosts per block
constexpr int kMaxCluster = 8;

template <typename KeyT>
__global__ void __launch_bounds__(kSeqThreads, 1) place_sequential_cluster_kernel(const SeqParams p)
{
    namespace cg = cooperative_groups;
    using Pair = typename SeqKey<KeyT>::Pair;
    constexpr KeyT kInf = SeqKey<KeyT>::kInf;
    constexpr int HPT = kClusterHpt;
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    extern __shared__ __align__(16) unsigned char seq_smem[];
    int4 *s_cap = reinterpret_cast<int4 *>(seq_smem);                                          // [kClusterHosts]
    KeyT *s_B = reinterpret_cast<KeyT *>(seq_smem + (size_t)kClusterHosts * sizeof(int4));      // [kClusterHosts]
    __shared__ KeyT s_warp[kSeqWarps][3];
    __shared__ KeyT s_best[3];
    __shared__ KeyT s_all[2][kMaxCluster][3];   // every block's triple of a request, double-buffered by request parity

    const int n = blockIdx.x / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t row = (size_t)n * p.Hpad;
    const int h_base = rank * kClusterHosts;

    int gmax_now[HPT], room[HPT], added[HPT];
    KeyT A[HPT];
#pragma unroll
    for (int u = 0; u < HPT; ++u) {
        const int hl = tid + u * kSeqThreads;   // index inside this block's run of hosts
        const int h = h_base + hl;
        int4 cap = make_int4(0, 0, 0, -1);
        KeyT b = 0;
        room[u] = -1;
        added[u] = 0;
        A[u] = kInf;
        if (h < p.Hpad) {
            const int4 f = p.feas[row + h];
            const int4 sq = p.seq[row + h];
            const Pair ab = reinterpret_cast<const Pair *>(p.ab)[row + h];
            cap = make_int4(f.y, f.z, f.w, sq.x);
            room[u] = sq.y;
            A[u] = f.x >= 0 ? (KeyT)ab.x : kInf;
            b = ab.y;
            if (f.x < 0) room[u] = -1;
        }
        gmax_now[u] = min(cap.w, room[u]);
        s_cap[hl] = cap;
        s_B[hl] = b;
    }
    // all blocks of the cluster are running before anyone writes into another's shared memory
    cluster.sync();

    const int4 *req = p.requests + (size_t)n * p.B;
    int4 next = p.B > 0 ? __ldg(req) : make_int4(-1, 0, 0, 0);
    for (long long r = 0; r < p.B; ++r) {
        const int4 q = next;
        if (r + 1 < p.B) next = __ldg(req + r + 1);
        const int par = (int)(r & 1);
        const bool sane = (q.x | q.y | q.z | q.w) >= 0;
        KeyT k1 = kInf, k2 = kInf, k3 = kInf;
        if (sane) {
#pragma unroll
            for (int u = 0; u < HPT; ++u) {
                const int hl = tid + u * kSeqThreads;
                const int4 cap = s_cap[hl];
                const bool ok = q.x <= gmax_now[u] && q.y <= cap.x && q.z <= cap.y && q.w <= cap.z;
                const KeyT key = ok ? (KeyT)(A[u] + (KeyT)(unsigned int)q.x * s_B[hl]) : kInf;
                insert3(k1, k2, k3, key);
            }
        }
        KeyT w1, w2, w3;
        warp_best3(k1, k2, k3, w1, w2, w3);
        if (lane == 0) {
            s_warp[warp][0] = w1;
            s_warp[warp][1] = w2;
            s_warp[warp][2] = w3;
        }
        __syncthreads();
        if (warp == 0) {
            KeyT b1, b2, b3;
            const bool has = lane < kSeqWarps;
            warp_best3(has ? s_warp[lane][0] : kInf, has ? s_warp[lane][1] : kInf, has ? s_warp[lane][2] : kInf, b1, b2, b3);
            // this block's triple goes into slot `rank` of every block's exchange buffer
            if (lane < C) {
                KeyT *remote = cluster.map_shared_rank(&s_all[par][rank][0], lane);
                remote[0] = b1;
                remote[1] = b2;
                remote[2] = b3;
            }
        }
        // one barrier per request for the whole cluster (release / acquire: the remote stores above
        // are visible to every block behind it). The buffer of the other parity is written again
        // only behind the next barrier, which no block passes before all have merged this one.
        cluster.sync();
        if (warp == 0) {
            KeyT b1, b2, b3;
            const bool has = lane < C;
            warp_best3(has ? s_all[par][lane][0] : kInf, has ? s_all[par][lane][1] : kInf, has ? s_all[par][lane][2] : kInf, b1, b2, b3);
            if (lane == 0) {
                s_best[0] = b1;
                s_best[1] = b2;
                s_best[2] = b3;
                if (rank == 0) {
                    const long long o = (long long)n * p.B + r;
                    p.out_hosts[o * 3 + 0] = b1 == kInf ? -1 : (int)((unsigned int)b1 & p.id_mask);
                    p.out_hosts[o * 3 + 1] = b2 == kInf ? -1 : (int)((unsigned int)b2 & p.id_mask);
                    p.out_hosts[o * 3 + 2] = b3 == kInf ? -1 : (int)((unsigned int)b3 & p.id_mask);
                    if (p.out_found) p.out_found[o] = (b1 != kInf) + (b2 != kInf) + (b3 != kInf);
                }
            }
        }
        __syncthreads();
        // commit: only a kernel that got all three replicas is created; a winner is updated by the
        // thread of the block that owns it
        if (s_best[2] != kInf && q.x > 0) {
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const int hl = (int)((unsigned int)s_best[i] & p.id_mask) - h_base;
                if (hl >= 0 && hl < kClusterHosts && (hl & (kSeqThreads - 1)) == tid) {
                    const int u0 = hl / kSeqThreads;
#pragma unroll
                    for (int u = 0; u < HPT; ++u)
                        if (u == u0) {
                            room[u] -= q.x;
                            gmax_now[u] = min(s_cap[hl].w, room[u]);
                            added[u] += q.x;
                            A[u] += (KeyT)(unsigned int)q.x * s_B[hl];
                        }
                }
            }
        }
        // s_best is rewritten only behind the next request's cluster barrier, which every thread
        // reaches after having read it here
    }
    if (p.out_subscribed) {
#pragma unroll
        for (int u = 0; u < HPT; ++u) {
            const int h = h_base + tid + u * kSeqThreads;
            if (h < p.H) p.out_subscribed[(size_t)n * p.H + h] = p.seq[row + h].z + added[u];
        }
    }
    // no block leaves while another may still write into its shared memory
    cluster.sync();
}

template <typename KeyT>
int launch_seq_cluster(const SeqParams &p, int N, int C, cudaStream_t stream)
{
    const size_t smem = (size_t)kClusterHosts * (sizeof(int4) + sizeof(KeyT));
    void (*fn)(const SeqParams) = place_sequential_cluster_kernel<KeyT>;
    NBOS_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned int)(N * C));
    cfg.blockDim = dim3(kSeqThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned int)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    NBOS_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, p));
    return NBOS_OK;
}

template <typename KeyT, int T>
int launch_seq_t(const SeqParams &p, int N, int hpt, cudaStream_t stream)
{
    const size_t smem = (size_t)hpt * T * (sizeof(int4) + sizeof(KeyT));
    void (*fn)(const SeqParams) = hpt == 1 ? place_sequential_kernel<KeyT, 1, T>
                                  : hpt == 2 ? place_sequential_kernel<KeyT, 2, T>
                                  : hpt == 4 ? place_sequential_kernel<KeyT, 4, T>
                                             : place_sequential_kernel<KeyT, 8, T>;
    NBOS_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    fn<<<N, T, smem, stream>>>(p);
    NBOS_CUDA_TRY(cudaGetLastError());
    return NBOS_OK;
}

template <typename KeyT>
int launch_seq(const SeqParams &p, int N, int threads, int hpt, cudaStream_t stream)
{
    switch (threads) {
    case 256: return launch_seq_t<KeyT, 256>(p, N, hpt, stream);
    case 512: return launch_seq_t<KeyT, 512>(p, N, hpt, stream);
    default: return launch_seq_t<KeyT, 1024>(p, N, hpt, stream);
    }
}

}  // namespace

int launch_place_sequential(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                            int32_t *d_out_hosts, int32_t *d_out_found, int32_t *d_out_subscribed,
                            cudaStream_t stream)
{
    SeqParams p;
    p.feas = s->d_host_feas;
    p.ab = s->d_host_ab;
    p.seq = s->d_host_seq;
    p.requests = reinterpret_cast<const int4 *>(d_requests);
    p.out_hosts = d_out_hosts;
    p.out_found = d_out_found;
    p.out_subscribed = d_out_subscribed;
    p.B = batch;
    p.H = s->H;
    p.Hpad = s->Hpad;
    p.id_mask = (1u << s->key.bits_id) - 1u;
    if (batch == 0 && !d_out_subscribed) return NBOS_OK;
    if (s->Hpad > kClusterHosts) {
        int C = 2;
        while (C * kClusterHosts < s->Hpad) C <<= 1;
        if (C > kMaxCluster) return fail(NBOS_ERR_RANGE, "sequential placement supports at most %d hosts", NBOS_SEQUENTIAL_MAX_HOSTS);
        return s->key.key_bits == 64 ? launch_seq_cluster<unsigned long long>(p, s->N, C, stream)
                                     : launch_seq_cluster<unsigned int>(p, s->N, C, stream);
    }
    // about four hosts per thread is fastest (measured at 256 to 8,192 hosts, one snapshot and 256):
    // fewer warps make the two reductions and the barrier cheaper, more hosts per thread lengthen
    // the evaluation; small blocks also let several snapshots share an SM
    const int threads = s->Hpad <= 1024 ? 256 : s->Hpad <= 2048 ? 512 : 1024;
    int hpt = 1;
    while (hpt * threads < s->Hpad) hpt <<= 1;
    return s->key.key_bits == 64 ? launch_seq<unsigned long long>(p, s->N, threads, hpt, stream)
                                 : launch_seq<unsigned int>(p, s->N, threads, hpt, stream);
}

}  // namespace nbos
