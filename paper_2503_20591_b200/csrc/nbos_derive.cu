// Snapshot derivation: cluster state (Section 3.4.1: G, S, C per server, plus the capacities of
// Section 3.2.1) -> one record per host that the placement kernel can test with four compares
// and rank with one multiply-add.
//
//   cap   = floor(limit_num * G * R / limit_den)      largest S+g with (S+g)/(G*R) <= limit
//   gmax  = min(G, cap - S [, G - C])                 largest GPU ask the host can take; -1 = none
//   key(g) = A + g * B, an integer that orders hosts exactly like
//            (G-C desc, (S+g)/(G*R) asc, host id asc)   [or with the first two swapped]:
//            the ratio field is (S+g) * (Lambda / G), Lambda = lcm of the distinct G of the
//            snapshot, which is (S+g)/(G*R) times the constant Lambda*R.
#include <limits.h>

#include "nbos_internal.h"

namespace nbos {
namespace {

struct ScanArgs {
    const int32_t *G, *S, *C, *AV, *AC, *AM;
    const longlong2 *limits;  // per snapshot (num * R, den): cap = floor(limits.x * G / limits.y)
    longlong2 limit0;         // used instead of limits[0] when `limits` is null (single snapshot)
    SnapStats *stats;
    int H, R, flags;
};

// `num_r` is the limit's numerator times R (R already cancelled for the dynamic limit).
__device__ __forceinline__ int derive_gmax(long long G, long long S, long long C, long long num_r,
                                           long long den, int flags)
{
    if (G < 1 || den < 1) return -1;
    long long cap = (num_r * G) / den;
    long long gm = cap - S;
    if (gm > G) gm = G;
    if ((flags & NBOS_REQUIRE_IDLE_GPUS) && gm > G - C) gm = G - C;
    return gm < 0 ? -1 : (int)gm;
}

// Cluster sums of Sections 3.4.1 / 3.4.2: sums[n] = (sum G, sum S, sum C, unused) per snapshot.
// grid (blocks_per_snapshot, N); `sums` must be zeroed before the launch.
__global__ void __launch_bounds__(256) sums_kernel(const int32_t *G, const int32_t *S, const int32_t *C,
                                                   int H, unsigned long long *sums)
{
    __shared__ unsigned long long s_sum[3];
    if (threadIdx.x < 3) s_sum[threadIdx.x] = 0ull;
    __syncthreads();
    const int n = blockIdx.y;
    unsigned long long g = 0, s = 0, c = 0;
    for (int h = blockIdx.x * blockDim.x + threadIdx.x; h < H; h += gridDim.x * blockDim.x) {
        const size_t i = (size_t)n * H + h;
        g += (unsigned long long)(long long)G[i];
        s += (unsigned long long)(long long)S[i];
        c += (unsigned long long)(long long)C[i];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        g += __shfl_xor_sync(0xFFFFFFFFu, g, off);
        s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        c += __shfl_xor_sync(0xFFFFFFFFu, c, off);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&s_sum[0], g);
        atomicAdd(&s_sum[1], s);
        atomicAdd(&s_sum[2], c);
    }
    __syncthreads();
    if (threadIdx.x < 3) atomicAdd(&sums[(size_t)n * 4 + threadIdx.x], s_sum[threadIdx.x]);
}

// Dynamic cluster-wide limit (Section 3.4.1, third factor): sum S / (sum G * R). R cancels against
// the R of the per-host ratio, so the stored pair is (sum S, sum G).
__global__ void limits_from_sums_kernel(const unsigned long long *sums, longlong2 *limits, int N)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n < N) limits[n] = make_longlong2((long long)sums[(size_t)n * 4 + 1], (long long)sums[(size_t)n * 4 + 0]);
}

// Per-snapshot values travel to the device inside kernel arguments (captured at launch, so no
// host buffer has to outlive the call and no stream synchronisation is implied).
struct LimitChunk {
    longlong2 v[128];
    int first, count;
};
__global__ void set_limits_kernel(longlong2 *limits, const LimitChunk c)
{
    const int i = threadIdx.x;
    if (i < c.count) limits[c.first + i] = c.v[i];
}

// Auto-scaler rule (Section 3.4.2) next to the sums: sums[n*4+3] = +1 if sum G < f * sum C (scale
// out), -1 if f * sum C < sum G (servers may be released), 0 if equal; f = f_num / f_den.
__global__ void autoscale_kernel(unsigned long long *sums, int N, long long f_num, long long f_den)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    const long long have = f_den * (long long)sums[(size_t)n * 4 + 0];
    const long long expected = f_num * (long long)sums[(size_t)n * 4 + 2];
    sums[(size_t)n * 4 + 3] = (unsigned long long)(long long)((have < expected) - (expected < have));
}

// grid (blocks_per_snapshot, N). Validates the value ranges and reduces what the key layout
// depends on. `stats` must be zeroed before the launch (every field is a max- or or-reduction).
__global__ void __launch_bounds__(256) scan_kernel(const ScanArgs a)
{
    __shared__ unsigned long long s_mask[16];
    __shared__ unsigned int s_err;
    __shared__ int s_idle_max, s_g_min_inv;
    __shared__ unsigned long long s_sub_max;
    __shared__ int s_max4[4];
    const int n = blockIdx.y;
    if (threadIdx.x < 4) s_max4[threadIdx.x] = 0;
    if (threadIdx.x < 16) s_mask[threadIdx.x] = 0ull;
    if (threadIdx.x == 0) {
        s_err = 0u;
        s_idle_max = 0;
        s_g_min_inv = 0;
        s_sub_max = 0ull;
    }
    __syncthreads();
    const longlong2 lim = a.limits ? a.limits[n] : a.limit0;
    unsigned int err = 0u;
    int idle_max = 0, g_min_inv = 0;  // INT_MAX - smallest G seen, 0 = none
    unsigned long long sub_max = 0ull;
    int max_gcap1 = 0, max_av = 0, max_ac = 0, max_am = 0;  // max_gcap1 = largest gmax + 1
    for (int h = blockIdx.x * blockDim.x + threadIdx.x; h < a.H; h += gridDim.x * blockDim.x) {
        const size_t i = (size_t)n * a.H + h;
        const int G = a.G[i], S = a.S[i], C = a.C[i];
        if ((G | S | C | a.AV[i] | a.AC[i] | a.AM[i]) < 0) err |= ERR_NEGATIVE;
        if (C > G) err |= ERR_COMMITTED_GT_TOTAL;
        if (G > NBOS_MAX_GPUS_PER_HOST) err |= ERR_G_TOO_LARGE;
        if (err) continue;
        if (G >= 1) {
            atomicOr(&s_mask[G >> 6], 1ull << (G & 63));
            g_min_inv = max(g_min_inv, INT_MAX - G);
        }
        idle_max = max(idle_max, G - C);
        const int gm = derive_gmax(G, S, C, lim.x, lim.y, a.flags);
        if (gm >= 0) {
            // largest S + g the ratio field has to hold: what fits now, or -- when later commits may
            // add to S (NBOS_ROOM_FOR_COMMITS) -- everything up to the host's cap
            unsigned long long top = (unsigned long long)S + (unsigned long long)gm;
            if (a.flags & NBOS_ROOM_FOR_COMMITS) top = max(top, (unsigned long long)((lim.x * (long long)G) / lim.y));
            sub_max = max(sub_max, top);
        }
        max_gcap1 = max(max_gcap1, gm + 1);
        max_av = max(max_av, a.AV[i]);
        max_ac = max(max_ac, a.AC[i]);
        max_am = max(max_am, a.AM[i]);
    }
    if (err) atomicOr(&s_err, err);
    atomicMax(&s_idle_max, idle_max);
    atomicMax(&s_g_min_inv, g_min_inv);
    atomicMax(&s_sub_max, sub_max);
    atomicMax(&s_max4[0], max_gcap1);
    atomicMax(&s_max4[1], max_av);
    atomicMax(&s_max4[2], max_ac);
    atomicMax(&s_max4[3], max_am);
    __syncthreads();
    SnapStats *st = a.stats + n;
    if (threadIdx.x < 16 && s_mask[threadIdx.x]) atomicOr(&st->g_mask[threadIdx.x], s_mask[threadIdx.x]);
    if (threadIdx.x == 0) {
        if (s_err) atomicOr(&st->err, s_err);
        atomicMax(&st->idle_max, s_idle_max);
        atomicMax(&st->g_min_inv, s_g_min_inv);
        atomicMax(&st->sub_max, s_sub_max);
        atomicMax(&st->max_gcap1, s_max4[0]);
        atomicMax(&st->max_av, s_max4[1]);
        atomicMax(&st->max_ac, s_max4[2]);
        atomicMax(&st->max_am, s_max4[3]);
    }
}

struct EmitArgs {
    const int32_t *G, *S, *C, *AV, *AC, *AM;
    const longlong2 *limits;
    longlong2 limit0;         // used when `limits` is null (single snapshot)
    const long long *lambda;  // per snapshot; null = every host has w = 1 (one GPU count per snapshot)
    unsigned int *rank;       // [N][Hpad], cleared here for rank_kernel (null = no visiting order)
    int4 *feas;                 // records in host-index order (staging)
    int4 *seq;                  // (min(G, idle), cap - S, S, 0) per host, for sequential placement
    void *ab;
    unsigned long long *sortkey;  // [N][Hpad] visiting-order key: A, or near-max for hosts that take nothing
    int H, Hpad, R, flags, key_order;
    int idle_max;             // over all snapshots: the idle field stores idle_max - (G - C)
    int bits_idle, bits_sr, bits_id;
    int group_major;          // 1: visiting order is (GPU count, key at g = 0) instead of the key alone
    unsigned int *done;       // [N][ceil(Hpad / 256)] counters of rank_kernel, cleared here (null = unused)
    // update mode (null status = create mode, where scan_kernel has validated the state): the new
    // state must be valid and fit the layout chosen when the snapshot was created; a host that is
    // not or does not raises the status word instead
    unsigned int *status;
    const int *g_single;       // per snapshot: the one GPU count of a static-key snapshot (0 = none)
    unsigned long long sr_field_max;
    int check_fmax, fmax[4];
};

constexpr int kMaxGpuCountGroups = kGroupSlices;  // distinct GPU counts per snapshot up to which the table is grouped
constexpr int kSortMaxHosts = 65536;  // larger tables keep host order (ranking is quadratic in the host count)
constexpr unsigned long long kSortNever = 0xFFFFFFFF00000000ull;  // hosts that take nothing go last (| host index)

// grid (ceil(Hpad / 256), N). One record per (padded) host.
template <typename KeyT, typename PairT>
__global__ void __launch_bounds__(256) emit_kernel(const EmitArgs a)
{
    const int n = blockIdx.y;
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= a.Hpad) return;
    if (a.done && h < (a.Hpad + 255) / 256) a.done[(size_t)n * ((a.Hpad + 255) / 256) + h] = 0u;
    int4 f = make_int4(-1, 0, 0, 0);  // padding host: takes nothing
    int4 sq = make_int4(-1, -1, 0, 0);
    KeyT A = (KeyT)h, B = 0;
    unsigned long long sk = kSortNever | (unsigned int)h;
    if (h < a.H) {
        const size_t i = (size_t)n * a.H + h;
        const int G = a.G[i], S = a.S[i], C = a.C[i];
        const longlong2 lim = a.limits ? a.limits[n] : a.limit0;
        int gm = derive_gmax(G, S, C, lim.x, lim.y, a.flags);
        if (a.status) {
            // the checks scan_kernel makes at creation, against the stored layout
            unsigned int upd = 0u;
            if ((G | S | C | a.AV[i] | a.AC[i] | a.AM[i]) < 0 || C > G || G > NBOS_MAX_GPUS_PER_HOST) {
                upd = STATUS_BAD_VALUES;
                gm = -1;   // the tables are undefined after such an update; keep the arithmetic in range
            } else {
                bool stale = G - C > a.idle_max;
                long long w = 1;
                if (G >= 1) {
                    if (a.lambda) {
                        const long long lam = a.lambda[n];
                        if (lam % G) stale = true; else w = lam / G;
                    } else if (G != a.g_single[n]) {
                        stale = true;
                    }
                }
                if (gm >= 0) {
                    unsigned long long top = (unsigned long long)S + (unsigned long long)gm;
                    if (a.flags & NBOS_ROOM_FOR_COMMITS) top = max(top, (unsigned long long)((lim.x * (long long)G) / lim.y));
                    if (top > a.sr_field_max / (unsigned long long)w) stale = true;
                }
                if (a.check_fmax && (gm > a.fmax[0] || a.AV[i] > a.fmax[1] || a.AC[i] > a.fmax[2] || a.AM[i] > a.fmax[3]))
                    stale = true;
                if (stale) {
                    upd = STATUS_STALE_LAYOUT;
                    gm = -1;
                }
            }
            if (upd) atomicOr(a.status, upd);
        }
        f = make_int4(gm, a.AV[i], a.AC[i], a.AM[i]);
        sq.z = S;
        if (G >= 1 && lim.y >= 1) {
            long long room = (lim.x * (long long)G) / lim.y - S;   // cap - S
            room = room > INT_MAX ? INT_MAX : room < -1 ? -1 : room;
            const int g_cap = (a.flags & NBOS_REQUIRE_IDLE_GPUS) ? min(G, G - C) : G;
            sq = make_int4(g_cap, (int)room, S, 0);
        }
        if (gm >= 0) {
            const KeyT w = a.lambda ? (KeyT)(a.lambda[n] / G) : (KeyT)1;
            const KeyT idle_inv = (KeyT)(a.idle_max - (G - C));
            const KeyT sr0 = (KeyT)S * w;
            if (a.key_order == NBOS_KEY_SR_FIRST) {
                A = (sr0 << (a.bits_idle + a.bits_id)) + (idle_inv << a.bits_id) + (KeyT)h;
                B = w << (a.bits_idle + a.bits_id);
            } else {
                A = (idle_inv << (a.bits_sr + a.bits_id)) + (sr0 << a.bits_id) + (KeyT)h;
                B = w << a.bits_id;
            }
            // A carries the host index in its low bits, so both forms are unique
            if (a.group_major) sk = ((unsigned long long)(unsigned int)G << 32) | (unsigned long long)(unsigned int)A;
            else sk = sizeof(KeyT) == 4 ? ((unsigned long long)A << 32) | (unsigned int)h : (unsigned long long)A;
        }
    }
    a.sortkey[(size_t)n * a.Hpad + h] = sk;
    a.seq[(size_t)n * a.Hpad + h] = sq;
    if (a.rank) a.rank[(size_t)n * a.Hpad + h] = 0u;
    a.feas[(size_t)n * a.Hpad + h] = f;
    PairT p;
    p.x = A;
    p.y = B;
    reinterpret_cast<PairT *>(a.ab)[(size_t)n * a.Hpad + h] = p;
}

struct FinalizeArgs {
    const int4 *tmp_feas;
    const void *tmp_ab;
    const unsigned int *rank;   // position of each host in visiting order, or null = host order
    int4 *feas;
    void *ab;
    uint4 *pk;
    uint2 *rk;
    unsigned int *rk1;
    int Hpad;
    PackLayout pack;
    RankLayout ranked;
};

// Move the record of host `src` of snapshot `n` to its place in visiting order and build the
// packed and ranked forms there.
template <typename PairT>
__device__ __forceinline__ void finalize_host(const FinalizeArgs &a, int n, int src)
{
    const size_t base = (size_t)n * a.Hpad;
    const unsigned int j = a.rank ? a.rank[base + src] : (unsigned int)src;
    const int4 f = a.tmp_feas[base + src];
    const PairT p = reinterpret_cast<const PairT *>(a.tmp_ab)[base + src];
    a.feas[base + j] = f;
    reinterpret_cast<PairT *>(a.ab)[base + j] = p;
    if (a.pack.enabled) {
        const unsigned int cap[4] = {(unsigned int)(f.x + 1), (unsigned int)f.y, (unsigned int)f.z,
                                     (unsigned int)f.w};
        unsigned int w[2] = {a.pack.guards, a.pack.guards1};
#pragma unroll
        for (int c = 0; c < 4; ++c) w[a.pack.fword[c]] |= cap[c] << a.pack.fshift[c];
        a.pk[base + j] = make_uint4(w[0], w[1], (unsigned int)p.x, (unsigned int)p.y);
    }
    if (a.ranked.enabled) {
        // ranked form: coarse capacities and the host's position in key order, two words
        const unsigned int cap[4] = {(unsigned int)(f.x + 1), (unsigned int)f.y, (unsigned int)f.z,
                                     (unsigned int)f.w};
        unsigned int w[2] = {a.ranked.guards, a.ranked.guards};
#pragma unroll
        for (int c = 0; c < 4; ++c) w[a.ranked.fword[c]] |= (cap[c] >> a.ranked.fdrop[c]) << a.ranked.fshift[c];
        w[a.ranked.fword[4]] |= (a.ranked.rank_top - j) << a.ranked.fshift[4];
        a.rk[base + j] = make_uint2(w[0], w[1]);
        if (a.ranked.l1_enabled) {
            unsigned int w1 = a.ranked.l1_guards;
#pragma unroll
            for (int c = 0; c < 4; ++c) w1 |= (cap[c] >> a.ranked.l1_drop[c]) << a.ranked.l1_shift[c];
            w1 |= (a.ranked.rank_top - j) << a.ranked.l1_shift[4];
            a.rk1[base + j] = w1;
        }
    }
}

// grid (ceil(Hpad / 256), N): tables that keep host order (too large to rank).
template <typename PairT>
__global__ void __launch_bounds__(256) finalize_kernel(const FinalizeArgs a)
{
    const int src = blockIdx.x * blockDim.x + threadIdx.x;
    if (src < a.Hpad) finalize_host<PairT>(a, blockIdx.y, src);
}

// Visiting order: hosts are visited in ascending order of their key at g = 0 (hosts that take
// nothing last), which makes later hosts rarely displace an earlier best-three entry. The sort
// keys are unique, so the position of host i is the number of hosts with a smaller key. Each
// block counts, for 256 hosts, the smaller keys inside one chunk of kRankChunk keys staged in
// shared memory, and adds its partial count to rank[i]; the block that is the last of its 256
// hosts' blocks to finish (a counter per group of 256 hosts tells) finds their positions
// complete and moves their records into place (finalize_host) in the same launch.
// grid (ceil(Hpad/256), ceil(Hpad/chunk), N); rank[] and done[] must be zero.
constexpr int kRankChunk = 256;
template <typename PairT>
__global__ void __launch_bounds__(256) rank_finalize_kernel(const unsigned long long *sortkey, unsigned int *rank,
                                                            unsigned int *done, const FinalizeArgs fa)
{
    __shared__ unsigned long long chunk[kRankChunk];
    __shared__ unsigned int s_last;
    const int Hpad = fa.Hpad;
    const size_t base = (size_t)blockIdx.z * Hpad;
    const int j0 = blockIdx.y * kRankChunk;
    const int nj = min(kRankChunk, Hpad - j0);
    for (int j = threadIdx.x; j < nj; j += blockDim.x) chunk[j] = sortkey[base + j0 + j];
    __syncthreads();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < Hpad) {
        const unsigned long long ki = sortkey[base + i];
        unsigned int smaller = 0;
#pragma unroll 8
        for (int j = 0; j < nj; ++j) smaller += chunk[j] < ki ? 1u : 0u;
        if (smaller) atomicAdd(&rank[base + i], smaller);
    }
    // every thread's additions are visible device-wide before the block signs off
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0)
        s_last = atomicAdd(&done[(size_t)blockIdx.z * gridDim.x + blockIdx.x], 1u) == gridDim.y - 1 ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();   // the other blocks' additions, published before their sign-off, are read below
    if (i < Hpad) finalize_host<PairT>(fa, blockIdx.z, i);
}

// Grouped tables (hosts stored GPU count by GPU count): where each group starts. A position
// starts a group when its key slope differs from its predecessor's; the hosts that take nothing
// are stored last and end the last group. One block per snapshot; bounds[n][k] = start of group k
// for k < number of groups, = end of the last group after that.
__global__ void __launch_bounds__(256) group_bounds_kernel(const int4 *feas, const uint2 *ab, int Hpad, int *bounds)
{
    __shared__ int s_start[kGroupSlices + 1];
    __shared__ int s_count, s_end;
    const size_t base = (size_t)blockIdx.x * Hpad;
    if (threadIdx.x == 0) {
        s_count = 0;
        s_end = Hpad;
    }
    __syncthreads();
    for (int pos = threadIdx.x; pos < Hpad; pos += blockDim.x) {
        const bool live = feas[base + pos].x >= 0;
        const bool prev_live = pos > 0 && feas[base + pos - 1].x >= 0;
        if (!live) {
            if (pos == 0 || prev_live) atomicMin(&s_end, pos);
        } else if (pos == 0 || ab[base + pos].y != ab[base + pos - 1].y) {
            const int slot = atomicAdd(&s_count, 1);
            if (slot <= kGroupSlices) s_start[slot] = pos;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int n = s_count < kGroupSlices ? s_count : kGroupSlices;
        for (int i = 1; i < n; ++i) {       // a handful of entries: insertion sort
            const int v = s_start[i];
            int j = i - 1;
            for (; j >= 0 && s_start[j] > v; --j) s_start[j + 1] = s_start[j];
            s_start[j + 1] = v;
        }
        int *out = bounds + (size_t)blockIdx.x * (kGroupSlices + 1);
        for (int k = 0; k <= kGroupSlices; ++k) out[k] = k < n ? s_start[k] : s_end;
    }
}

int bits_for(unsigned long long max_value)
{
    int b = 0;
    while (max_value) {
        ++b;
        max_value >>= 1;
    }
    return b;
}

unsigned long long gcd_u64(unsigned long long a, unsigned long long b)
{
    while (b) {
        unsigned long long t = a % b;
        a = b;
        b = t;
    }
    return a;
}

}  // namespace

Layout workspace_layout(int N, int Hpad)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    Layout l;
    size_t o = 0;
    l.off_status = o;  o = up(o + 256);
    l.off_limits = o;  o = up(o + (size_t)N * sizeof(longlong2));
    l.off_sums = o;    o = up(o + (size_t)N * 4 * sizeof(unsigned long long));
    l.off_stats = o;   o = up(o + (size_t)N * sizeof(SnapStats));
    l.off_lambda = o;  o = up(o + (size_t)N * sizeof(long long));
    l.off_g_single = o; o = up(o + (size_t)N * sizeof(int));
    l.off_feas = o;    o = up(o + (size_t)N * Hpad * sizeof(int4));
    l.off_ab = o;      o = up(o + (size_t)N * Hpad * sizeof(ulonglong2));
    l.off_pk = o;      o = up(o + (size_t)N * Hpad * sizeof(uint4));
    l.off_rk = o;      o = up(o + (size_t)N * Hpad * sizeof(uint2));
    l.off_rk1 = o;     o = up(o + (size_t)N * Hpad * sizeof(unsigned int));
    l.off_tmp_feas = o; o = up(o + (size_t)N * Hpad * sizeof(int4));
    l.off_tmp_ab = o;  o = up(o + (size_t)N * Hpad * sizeof(ulonglong2));
    l.off_tmp_seq = o; o = up(o + (size_t)N * Hpad * sizeof(int4));
    l.off_sortkey = o; o = up(o + (size_t)N * Hpad * sizeof(unsigned long long));
    l.off_perm = o;    o = up(o + (size_t)N * Hpad * sizeof(unsigned int));
    l.off_done = o;    o = up(o + (size_t)N * ((Hpad + 255) / 256) * sizeof(unsigned int));
    l.off_gbounds = o; o = up(o + (size_t)N * (kGroupSlices + 1) * sizeof(int));
    l.total = o;
    return l;
}

int launch_cluster_sums(const int32_t *d_G, const int32_t *d_S, const int32_t *d_C, int N, int H,
                        long long f_num, long long f_den, long long *d_out, cudaStream_t stream)
{
    unsigned long long *sums = reinterpret_cast<unsigned long long *>(d_out);
    NBOS_CUDA_TRY(cudaMemsetAsync(sums, 0, sizeof(unsigned long long) * 4 * (size_t)N, stream));
    int bx = (H + 255) / 256;
    if (bx > 64) bx = 64;
    sums_kernel<<<dim3(bx, N), 256, 0, stream>>>(d_G, d_S, d_C, H, sums);
    autoscale_kernel<<<(N + 255) / 256, 256, 0, stream>>>(sums, N, f_num, f_den);
    NBOS_CUDA_TRY(cudaGetLastError());
    return NBOS_OK;
}

namespace {

struct DeriveCtx {
    nbos_snapshot *s;
    const int32_t *G, *S, *C, *AV, *AC, *AM;
    cudaStream_t stream;
    Layout lay;
    char *ws;
    longlong2 *d_limits;
    const longlong2 *limits_arg;
    longlong2 limit0;
    int bx;
};

// Clear the per-derivation state and put the limits on the device (or compute them there).
// `first_time` also clears the word that kernels raise when a bounded wait runs out; a later
// derivation of the same snapshot leaves that word alone.
int stage_limits(DeriveCtx &c, const nbos_snapshot_desc *d, bool first_time)
{
    nbos_snapshot *s = c.s;
    const int N = s->N, H = s->H;
    const bool dynamic_limit = (s->flags & NBOS_LIMIT_CLUSTER_SR) != 0;
    // status word, limits, sums and scan statistics are contiguous: one clear (lambda and g_single,
    // which an update keeps, lie behind them)
    const size_t from = c.lay.off_status + (first_time ? 0 : kUpdateStatusOffset);
    NBOS_CUDA_TRY(cudaMemsetAsync(c.ws + from, 0, c.lay.off_lambda - from, c.stream));
    c.limits_arg = c.d_limits;
    c.limit0 = make_longlong2(0, 1);
    if (dynamic_limit) {
        unsigned long long *d_sums = reinterpret_cast<unsigned long long *>(c.ws + c.lay.off_sums);
        sums_kernel<<<dim3(c.bx, N), 256, 0, c.stream>>>(c.G, c.S, c.C, H, d_sums);
        limits_from_sums_kernel<<<(N + 255) / 256, 256, 0, c.stream>>>(d_sums, c.d_limits, N);
    } else if (N == 1) {
        // a single snapshot's fixed limit travels in the kernel arguments
        c.limits_arg = nullptr;
        c.limit0 = make_longlong2((long long)d->limit_num[0] * s->R, d->limit_den[0]);
    } else {
        for (int first = 0; first < N; first += 128) {
            LimitChunk chunk;
            chunk.first = first;
            chunk.count = N - first < 128 ? N - first : 128;
            for (int i = 0; i < chunk.count; ++i)
                chunk.v[i] = make_longlong2((long long)d->limit_num[first + i] * s->R, d->limit_den[first + i]);
            set_limits_kernel<<<1, 128, 0, c.stream>>>(c.d_limits, chunk);
        }
    }
    NBOS_CUDA_TRY(cudaGetLastError());
    return NBOS_OK;
}

// emit -> rank + finalize with the layout stored in the handle. `check_state` (refresh of an
// existing snapshot): the emit kernel also validates the new state against that layout.
int emit_tables(DeriveCtx &c, bool check_state)
{
    nbos_snapshot *s = c.s;
    const int N = s->N, H = s->H, Hpad = s->Hpad;
    const KeyLayout &k = s->key;
    long long *d_lambda = reinterpret_cast<long long *>(c.ws + c.lay.off_lambda);
    int4 *tmp_feas = reinterpret_cast<int4 *>(c.ws + c.lay.off_tmp_feas);
    void *tmp_ab = c.ws + c.lay.off_tmp_ab;
    unsigned long long *sortkey = reinterpret_cast<unsigned long long *>(c.ws + c.lay.off_sortkey);
    unsigned int *perm = reinterpret_cast<unsigned int *>(c.ws + c.lay.off_perm);
    int4 *tmp_seq = reinterpret_cast<int4 *>(c.ws + c.lay.off_tmp_seq);
    unsigned int *done = reinterpret_cast<unsigned int *>(c.ws + c.lay.off_done);
    const int *fm = s->pack.enabled ? s->pack.fmax : s->rank.fmax;  // the same values in both layouts
    EmitArgs ea{c.G, c.S, c.C, c.AV, c.AC, c.AM, c.limits_arg, c.limit0, k.static_key ? nullptr : d_lambda,
                s->presorted ? perm : nullptr, tmp_feas, tmp_seq, tmp_ab, sortkey,
                H, Hpad, s->R, s->flags, s->key_order, s->idle_max, k.bits_idle, k.bits_sr, k.bits_id,
                k.grouped, s->presorted ? done : nullptr,
                check_state ? s->d_update_status : nullptr,
                reinterpret_cast<const int *>(c.ws + c.lay.off_g_single),
                k.bits_sr >= 64 ? ~0ull : ((1ull << k.bits_sr) - 1ull),
                (s->pack.enabled || s->rank.enabled) ? 1 : 0, {fm[0], fm[1], fm[2], fm[3]}};
    dim3 grid((Hpad + 255) / 256, N);
    if (k.key_bits == 32)
        emit_kernel<unsigned int, uint2><<<grid, 256, 0, c.stream>>>(ea);
    else
        emit_kernel<unsigned long long, ulonglong2><<<grid, 256, 0, c.stream>>>(ea);
    FinalizeArgs fa{tmp_feas, tmp_ab, s->presorted ? perm : nullptr, reinterpret_cast<int4 *>(c.ws + c.lay.off_feas),
                    c.ws + c.lay.off_ab, reinterpret_cast<uint4 *>(c.ws + c.lay.off_pk),
                    reinterpret_cast<uint2 *>(c.ws + c.lay.off_rk),
                    reinterpret_cast<unsigned int *>(c.ws + c.lay.off_rk1), Hpad, s->pack, s->rank};
    if (s->presorted) {
        const dim3 rgrid((Hpad + 255) / 256, (Hpad + kRankChunk - 1) / kRankChunk, N);
        if (k.key_bits == 32)
            rank_finalize_kernel<uint2><<<rgrid, 256, 0, c.stream>>>(sortkey, perm, done, fa);
        else
            rank_finalize_kernel<ulonglong2><<<rgrid, 256, 0, c.stream>>>(sortkey, perm, done, fa);
    } else if (k.key_bits == 32) {
        finalize_kernel<uint2><<<grid, 256, 0, c.stream>>>(fa);
    } else {
        finalize_kernel<ulonglong2><<<grid, 256, 0, c.stream>>>(fa);
    }
    if (k.grouped)
        group_bounds_kernel<<<N, 256, 0, c.stream>>>(fa.feas, reinterpret_cast<const uint2 *>(fa.ab), Hpad,
                                                     reinterpret_cast<int *>(c.ws + c.lay.off_gbounds));
    NBOS_CUDA_TRY(cudaGetLastError());
    return NBOS_OK;
}

DeriveCtx make_ctx(nbos_snapshot *s, const int32_t *d_G, const int32_t *d_S, const int32_t *d_C,
                   const int32_t *d_AV, const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream)
{
    DeriveCtx c;
    c.s = s;
    c.G = d_G; c.S = d_S; c.C = d_C; c.AV = d_AV; c.AC = d_AC; c.AM = d_AM;
    c.stream = stream;
    c.lay = workspace_layout(s->N, s->Hpad);
    c.ws = static_cast<char *>(s->workspace);
    c.d_limits = reinterpret_cast<longlong2 *>(c.ws + c.lay.off_limits);
    c.limits_arg = c.d_limits;
    c.limit0 = make_longlong2(0, 1);
    c.bx = (s->H + 255) / 256;
    if (c.bx > 64) c.bx = 64;
    return c;
}

}  // namespace

int derive_snapshot(nbos_snapshot *s, const nbos_snapshot_desc *d, const int32_t *d_G,
                    const int32_t *d_S, const int32_t *d_C, const int32_t *d_AV,
                    const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream)
{
    const int N = s->N, H = s->H, Hpad = s->Hpad;
    DeriveCtx c = make_ctx(s, d_G, d_S, d_C, d_AV, d_AC, d_AM, stream);
    long long *d_lambda = reinterpret_cast<long long *>(c.ws + c.lay.off_lambda);
    int *d_g_single = reinterpret_cast<int *>(c.ws + c.lay.off_g_single);
    SnapStats *d_stats = reinterpret_cast<SnapStats *>(c.ws + c.lay.off_stats);

    SnapStats *h_stats = static_cast<SnapStats *>(malloc(sizeof(SnapStats) * (size_t)N));
    long long *h_lambda = static_cast<long long *>(malloc(sizeof(long long) * (size_t)N));
    int *h_g_single = static_cast<int *>(malloc(sizeof(int) * (size_t)N));
    struct Free {
        void *a, *b, *c;
        ~Free() { free(a); free(b); free(c); }
    } guard{h_stats, h_lambda, h_g_single};
    if (!h_stats || !h_lambda || !h_g_single) return fail(NBOS_ERR_NO_MEMORY, "host allocation failed");

    int rc = stage_limits(c, d, true);
    if (rc) return rc;
    ScanArgs sa{d_G, d_S, d_C, d_AV, d_AC, d_AM, c.limits_arg, c.limit0, d_stats, H, s->R, s->flags};
    scan_kernel<<<dim3(c.bx, N), 256, 0, stream>>>(sa);
    NBOS_CUDA_TRY(cudaGetLastError());
    NBOS_CUDA_TRY(cudaMemcpyAsync(h_stats, d_stats, sizeof(SnapStats) * (size_t)N,
                                  cudaMemcpyDeviceToHost, stream));
    NBOS_CUDA_TRY(cudaStreamSynchronize(stream));

    // value ranges, Lambda per snapshot, field widths
    int idle_max = 0;
    unsigned long long sr_max = 0;
    for (int n = 0; n < N; ++n) {
        const SnapStats &st = h_stats[n];
        if (st.err & ERR_NEGATIVE) return fail(NBOS_ERR_RANGE, "snapshot %d: negative value in a host array", n);
        if (st.err & ERR_COMMITTED_GT_TOTAL)
            return fail(NBOS_ERR_RANGE, "snapshot %d: committed GPUs exceed total GPUs on some host", n);
        if (st.err & ERR_G_TOO_LARGE)
            return fail(NBOS_ERR_RANGE, "snapshot %d: more than %d GPUs on some host", n, NBOS_MAX_GPUS_PER_HOST);
        unsigned long long lambda = 1;
        int distinct = 0, single = 0;
        for (int G = 1; G <= NBOS_MAX_GPUS_PER_HOST; ++G) {
            if (!(st.g_mask[G >> 6] >> (G & 63) & 1ull)) continue;
            ++distinct;
            single = G;
            lambda = lambda / gcd_u64(lambda, (unsigned long long)G) * (unsigned long long)G;
            if (lambda > (1ull << 40))
                return fail(NBOS_ERR_RANGE, "snapshot %d: GPU counts per host too diverse for an exact 63-bit key", n);
        }
        h_lambda[n] = (long long)lambda;
        h_g_single[n] = distinct == 1 ? single : 0;
        if (st.idle_max > idle_max) idle_max = st.idle_max;
        if (st.g_min_inv != 0) {
            const unsigned long long w_max = lambda / (unsigned long long)(INT_MAX - st.g_min_inv);
            if (st.sub_max > (1ull << 62) / (w_max ? w_max : 1))
                return fail(NBOS_ERR_RANGE, "snapshot %d: subscription values too large for a 63-bit key", n);
            const unsigned long long m = st.sub_max * w_max;
            if (m > sr_max) sr_max = m;
        }
    }
    KeyLayout k = {};
    k.bits_idle = bits_for((unsigned long long)idle_max);
    k.bits_sr = bits_for(sr_max);
    k.bits_id = bits_for((unsigned long long)(Hpad - 1));
    const int total_bits = k.bits_idle + k.bits_sr + k.bits_id;
    if (total_bits > 63) return fail(NBOS_ERR_RANGE, "ranking key needs %d bits (max 63)", total_bits);
    k.key_bits = (total_bits <= 31 && !(s->flags & NBOS_FORCE_KEY64)) ? 32 : 64;
    k.static_key = 1;
    int fmax[4] = {0, 0, 0, 0};
    int max_distinct_g = 0;
    for (int n = 0; n < N; ++n) {
        const SnapStats &st = h_stats[n];
        int distinct_g = 0;
        for (int w = 0; w < 16; ++w) distinct_g += __builtin_popcountll(st.g_mask[w]);
        if (distinct_g > 1) k.static_key = 0;
        if (distinct_g > max_distinct_g) max_distinct_g = distinct_g;
        if (st.max_gcap1 - 1 > fmax[0]) fmax[0] = st.max_gcap1 - 1;
        if (st.max_av > fmax[1]) fmax[1] = st.max_av;
        if (st.max_ac > fmax[2]) fmax[2] = st.max_ac;
        if (st.max_am > fmax[3]) fmax[3] = st.max_am;
    }
    s->key = k;
    // the idle field can hold up to 2^bits - 1: use all of it, so that a later update may bring
    // hosts with more idle GPUs than any host has now
    idle_max = (int)((1u << k.bits_idle) - 1u);
    s->idle_max = idle_max;

    // field widths of the four capacity components, from the scanned maxima
    int width[4];
    width[0] = bits_for((unsigned long long)fmax[0] + 2);  // stored +1, and one more for "fits nowhere"
    for (int c2 = 1; c2 < 4; ++c2) width[c2] = fmax[c2] ? bits_for((unsigned long long)fmax[c2]) : 1;
    // largest value each field can take (not merely the largest present now): asks up to it are
    // compared exactly, and a later update may raise capacities up to it
    int field_max[4];
    field_max[0] = (int)((1u << width[0]) - 3u);
    for (int c2 = 1; c2 < 4; ++c2) field_max[c2] = (int)((1u << width[c2]) - 1u);

    // packed capacity test: the two widest components become the high fields of the two words
    PackLayout pk = {};
    if (k.key_bits == 32) {
        int order[4] = {0, 1, 2, 3};
        for (int i = 0; i < 4; ++i)
            for (int j = i + 1; j < 4; ++j)
                if (width[order[j]] > width[order[i]]) { int t = order[i]; order[i] = order[j]; order[j] = t; }
        // widest with narrowest in word 0, the middle two in word 1
        const int hi0 = width[order[0]], lo0 = width[order[3]], hi1 = width[order[1]], lo1 = width[order[2]];
        int lo_a = -1, lo_b = -1;
        if (hi0 + lo1 + 2 <= 32) lo_a = lo_b = lo1;                              // same guard positions in both words
        else if (hi0 + lo0 + 2 <= 32 && hi1 + lo1 + 2 <= 32) { lo_a = lo0; lo_b = lo1; }  // each word its own
        if (lo_a >= 0) {
            pk.enabled = 1;
            pk.guards = 0x80000000u | (1u << lo_a);
            pk.guards1 = 0x80000000u | (1u << lo_b);
            for (int c2 = 0; c2 < 4; ++c2) pk.fmax[c2] = field_max[c2];
            pk.fword[order[0]] = 0; pk.fshift[order[0]] = lo_a + 1;
            pk.fword[order[3]] = 0; pk.fshift[order[3]] = 0;
            pk.fword[order[1]] = 1; pk.fshift[order[1]] = lo_b + 1;
            pk.fword[order[2]] = 1; pk.fshift[order[2]] = 0;
        }
    }
    s->pack = pk;
    s->presorted = Hpad <= kSortMaxHosts;
    // Hosts with different GPU counts rank differently for different asks, but within one GPU
    // count the order is the same for every ask. With few distinct counts the table is stored
    // count by count, each group in key order, and the placement kernel treats every group like
    // a table in key order.
    s->key.grouped = (!k.static_key && k.key_bits == 32 && pk.enabled && s->presorted &&
                      max_distinct_g <= kMaxGpuCountGroups) ? 1 : 0;

    // Ranked form (see RankLayout): six slots -- three per word at the same bit positions -- for
    // the four capacities, the rank and one unused slot. Components are paired by width (the two
    // narrowest share the lowest slot, and so on); a slot is as wide as its wider member, and
    // while the three widths exceed the 29 bits left beside the guards the widest slot that may
    // shrink does: the GPU component and the rank stay exact, the others lose low bits.
    RankLayout rl = {};
    if (k.key_bits == 32 && (k.static_key || s->key.grouped) && s->presorted) {
        int w6[6] = {width[0], width[1], width[2], width[3], bits_for((unsigned long long)(Hpad - 1)), 0};
        int order[6] = {0, 1, 2, 3, 4, 5};
        for (int i = 0; i < 6; ++i)
            for (int j = i + 1; j < 6; ++j)
                if (w6[order[j]] < w6[order[i]]) { int t = order[i]; order[i] = order[j]; order[j] = t; }
        int slot_w[3], slot_min[3];
        for (int sl = 0; sl < 3; ++sl) {
            const int a = order[2 * sl], b = order[2 * sl + 1];
            slot_w[sl] = w6[a] > w6[b] ? w6[a] : w6[b];
            slot_min[sl] = 1;
            if ((a == 0 || a == 4) && w6[a] > slot_min[sl]) slot_min[sl] = w6[a];
            if ((b == 0 || b == 4) && w6[b] > slot_min[sl]) slot_min[sl] = w6[b];
            if (slot_w[sl] < slot_min[sl]) slot_w[sl] = slot_min[sl];
        }
        bool fits = true;
        while (slot_w[0] + slot_w[1] + slot_w[2] > 29) {
            int pick = -1;
            for (int sl = 0; sl < 3; ++sl)
                if (slot_w[sl] > slot_min[sl] && (pick < 0 || slot_w[sl] > slot_w[pick])) pick = sl;
            if (pick < 0) { fits = false; break; }
            --slot_w[pick];
        }
        if (fits) {
            slot_w[2] = 29 - slot_w[0] - slot_w[1];  // the top slot takes what is left
            const int slot_shift[3] = {0, slot_w[0] + 1, slot_w[0] + slot_w[1] + 2};
            rl.enabled = 1;
            rl.guards = 0x80000000u | (1u << slot_w[0]) | (1u << (slot_w[0] + slot_w[1] + 1));
            for (int sl = 0; sl < 3; ++sl)
                for (int half = 0; half < 2; ++half) {
                    const int comp = order[2 * sl + half];
                    if (comp == 5) continue;  // the unused slot: host field 0 against request field 0
                    rl.fword[comp] = half;
                    rl.fshift[comp] = slot_shift[sl];
                    rl.fdrop[comp] = w6[comp] > slot_w[sl] ? w6[comp] - slot_w[sl] : 0;
                }
            for (int c2 = 0; c2 < 4; ++c2) rl.fmax[c2] = field_max[c2];
            rl.rank_top = (unsigned int)(Hpad - 1);
            rl.rank_mask = ((1u << w6[4]) - 1u) << rl.fshift[4];
            // first level: five fields + five guards in 32 bits. The GPU component and the rank
            // keep their widths; the three other capacities share what is left as evenly as
            // their widths allow (a component narrower than its share passes the rest on).
            int left = 32 - 5 - w6[0] - w6[4];
            if (left >= 3) {
                int give[4] = {w6[0], 0, 0, 0};
                int need[4] = {0, w6[1], w6[2], w6[3]};
                while (left > 0) {
                    int pick = -1;  // the component that still lacks the most bits
                    for (int c2 = 1; c2 < 4; ++c2)
                        if (need[c2] > give[c2] && (pick < 0 || give[c2] < give[pick] ||
                                                    (give[c2] == give[pick] && need[c2] > need[pick])))
                            pick = c2;
                    if (pick < 0) break;
                    ++give[pick];
                    --left;
                }
                int at = 0;
                rl.l1_enabled = 1;
                rl.l1_guards = 0u;
                for (int c2 = 1; c2 <= 5; ++c2) {      // order: VRAM, millicpus, memory, GPUs, rank
                    const int comp = c2 <= 3 ? c2 : c2 == 4 ? 0 : 4;
                    const int wdt = comp == 4 ? w6[4] : give[comp];
                    rl.l1_shift[comp] = at;
                    rl.l1_drop[comp] = comp == 4 ? 0 : w6[comp] - wdt;
                    at += wdt;
                    rl.l1_guards |= 1u << at;
                    ++at;
                }
                rl.l1_rank_mask = ((1u << w6[4]) - 1u) << rl.l1_shift[4];
            }
        }
    }
    s->rank = rl;
    // what a later nbos_snapshot_update checks the new state against
    if (!k.static_key)
        NBOS_CUDA_TRY(cudaMemcpyAsync(d_lambda, h_lambda, sizeof(long long) * (size_t)N, cudaMemcpyHostToDevice, stream));
    NBOS_CUDA_TRY(cudaMemcpyAsync(d_g_single, h_g_single, sizeof(int) * (size_t)N, cudaMemcpyHostToDevice, stream));

    rc = emit_tables(c, false);
    if (rc) return rc;
    s->d_status = reinterpret_cast<unsigned int *>(c.ws + c.lay.off_status);
    s->d_update_status = reinterpret_cast<unsigned int *>(c.ws + c.lay.off_status + kUpdateStatusOffset);
    s->d_feas = reinterpret_cast<const int4 *>(c.ws + c.lay.off_feas);
    s->d_ab = c.ws + c.lay.off_ab;
    s->d_pk = reinterpret_cast<const uint4 *>(c.ws + c.lay.off_pk);
    s->d_rk = reinterpret_cast<const uint2 *>(c.ws + c.lay.off_rk);
    s->d_rk1 = reinterpret_cast<const unsigned int *>(c.ws + c.lay.off_rk1);
    s->d_group_bounds = reinterpret_cast<const int *>(c.ws + c.lay.off_gbounds);
    s->d_host_feas = reinterpret_cast<const int4 *>(c.ws + c.lay.off_tmp_feas);
    s->d_host_ab = c.ws + c.lay.off_tmp_ab;
    s->d_host_seq = reinterpret_cast<const int4 *>(c.ws + c.lay.off_tmp_seq);
    return NBOS_OK;
}

// Re-derive the tables of an existing snapshot from new state, keeping the key and packing layout
// chosen at creation: two kernels (emit, which also validates the state against that layout, and
// rank + finalize). Nothing is read back: a state that is invalid or does not fit the layout is
// reported through the status word.
int update_snapshot(nbos_snapshot *s, const nbos_snapshot_desc *d, const int32_t *d_G,
                    const int32_t *d_S, const int32_t *d_C, const int32_t *d_AV,
                    const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream)
{
    DeriveCtx c = make_ctx(s, d_G, d_S, d_C, d_AV, d_AC, d_AM, stream);
    int rc = stage_limits(c, d, false);
    if (rc) return rc;
    return emit_tables(c, true);
}

}  // namespace nbos
