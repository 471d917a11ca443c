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
    const int2 *limits;  // per snapshot (num, den)
    SnapStats *stats;
    int H, R, flags;
};

__device__ __forceinline__ int derive_gmax(long long G, long long S, long long C, long long num,
                                           long long den, long long R, int flags)
{
    if (G < 1) return -1;
    long long cap = (num * G * R) / den;
    long long gm = cap - S;
    if (gm > G) gm = G;
    if ((flags & NBOS_REQUIRE_IDLE_GPUS) && gm > G - C) gm = G - C;
    return gm < 0 ? -1 : (int)gm;
}

// grid (blocks_per_snapshot, N). Validates the value ranges and reduces what the key layout
// depends on. `stats` must be zeroed (g_min preset to INT_MAX) before the launch.
__global__ void __launch_bounds__(256) scan_kernel(const ScanArgs a)
{
    __shared__ unsigned long long s_mask[16];
    __shared__ unsigned int s_err;
    __shared__ int s_idle_max, s_g_min;
    __shared__ unsigned long long s_sub_max;
    const int n = blockIdx.y;
    if (threadIdx.x < 16) s_mask[threadIdx.x] = 0ull;
    if (threadIdx.x == 0) {
        s_err = 0u;
        s_idle_max = 0;
        s_g_min = INT_MAX;
        s_sub_max = 0ull;
    }
    __syncthreads();
    const int2 lim = a.limits[n];
    unsigned int err = 0u;
    int idle_max = 0, g_min = INT_MAX;
    unsigned long long sub_max = 0ull;
    for (int h = blockIdx.x * blockDim.x + threadIdx.x; h < a.H; h += gridDim.x * blockDim.x) {
        const size_t i = (size_t)n * a.H + h;
        const int G = a.G[i], S = a.S[i], C = a.C[i];
        if ((G | S | C | a.AV[i] | a.AC[i] | a.AM[i]) < 0) err |= ERR_NEGATIVE;
        if (C > G) err |= ERR_COMMITTED_GT_TOTAL;
        if (G > NBOS_MAX_GPUS_PER_HOST) err |= ERR_G_TOO_LARGE;
        if (err) continue;
        if (G >= 1) {
            atomicOr(&s_mask[G >> 6], 1ull << (G & 63));
            g_min = min(g_min, G);
        }
        idle_max = max(idle_max, G - C);
        const int gm = derive_gmax(G, S, C, lim.x, lim.y, a.R, a.flags);
        if (gm >= 0) sub_max = max(sub_max, (unsigned long long)S + (unsigned long long)gm);
    }
    if (err) atomicOr(&s_err, err);
    atomicMax(&s_idle_max, idle_max);
    atomicMin(&s_g_min, g_min);
    atomicMax(&s_sub_max, sub_max);
    __syncthreads();
    SnapStats *st = a.stats + n;
    if (threadIdx.x < 16 && s_mask[threadIdx.x]) atomicOr(&st->g_mask[threadIdx.x], s_mask[threadIdx.x]);
    if (threadIdx.x == 0) {
        if (s_err) atomicOr(&st->err, s_err);
        atomicMax(&st->idle_max, s_idle_max);
        atomicMin(&st->g_min, s_g_min);
        atomicMax(&st->sub_max, s_sub_max);
    }
}

__global__ void init_stats_kernel(SnapStats *stats, int n)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        SnapStats z = {};
        z.g_min = INT_MAX;
        stats[i] = z;
    }
}

struct EmitArgs {
    const int32_t *G, *S, *C, *AV, *AC, *AM;
    const int2 *limits;
    const long long *lambda;  // per snapshot
    int4 *feas;
    void *ab;
    int H, Hpad, R, flags, key_order;
    int idle_max;             // over all snapshots: the idle field stores idle_max - (G - C)
    int bits_idle, bits_sr, bits_id;
};

// grid (ceil(Hpad / 256), N). One record per (padded) host.
template <typename KeyT, typename PairT>
__global__ void __launch_bounds__(256) emit_kernel(const EmitArgs a)
{
    const int n = blockIdx.y;
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= a.Hpad) return;
    int4 f = make_int4(-1, 0, 0, 0);  // padding host: takes nothing
    KeyT A = (KeyT)h, B = 0;
    if (h < a.H) {
        const size_t i = (size_t)n * a.H + h;
        const int G = a.G[i], S = a.S[i], C = a.C[i];
        const int2 lim = a.limits[n];
        const int gm = derive_gmax(G, S, C, lim.x, lim.y, a.R, a.flags);
        f = make_int4(gm, a.AV[i], a.AC[i], a.AM[i]);
        if (gm >= 0) {
            const KeyT w = (KeyT)(a.lambda[n] / G);
            const KeyT idle_inv = (KeyT)(a.idle_max - (G - C));
            const KeyT sr0 = (KeyT)S * w;
            if (a.key_order == NBOS_KEY_SR_FIRST) {
                A = (sr0 << (a.bits_idle + a.bits_id)) + (idle_inv << a.bits_id) + (KeyT)h;
                B = w << (a.bits_idle + a.bits_id);
            } else {
                A = (idle_inv << (a.bits_sr + a.bits_id)) + (sr0 << a.bits_id) + (KeyT)h;
                B = w << a.bits_id;
            }
        }
    }
    a.feas[(size_t)n * a.Hpad + h] = f;
    PairT p;
    p.x = A;
    p.y = B;
    reinterpret_cast<PairT *>(a.ab)[(size_t)n * a.Hpad + h] = p;
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
    l.off_limits = o;  o = up(o + (size_t)N * sizeof(int2));
    l.off_lambda = o;  o = up(o + (size_t)N * sizeof(long long));
    l.off_stats = o;   o = up(o + (size_t)N * sizeof(SnapStats));
    l.off_feas = o;    o = up(o + (size_t)N * Hpad * sizeof(int4));
    l.off_ab = o;      o = up(o + (size_t)N * Hpad * sizeof(ulonglong2));
    l.total = o;
    return l;
}

int derive_snapshot(nbos_snapshot *s, const nbos_snapshot_desc *d, const int32_t *d_G,
                    const int32_t *d_S, const int32_t *d_C, const int32_t *d_AV,
                    const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream)
{
    const int N = s->N, H = s->H, Hpad = s->Hpad;
    const Layout lay = workspace_layout(N, Hpad);
    char *ws = static_cast<char *>(s->workspace);
    int2 *d_limits = reinterpret_cast<int2 *>(ws + lay.off_limits);
    long long *d_lambda = reinterpret_cast<long long *>(ws + lay.off_lambda);
    SnapStats *d_stats = reinterpret_cast<SnapStats *>(ws + lay.off_stats);

    // limits -> device
    int2 *h_limits = static_cast<int2 *>(malloc(sizeof(int2) * (size_t)N));
    SnapStats *h_stats = static_cast<SnapStats *>(malloc(sizeof(SnapStats) * (size_t)N));
    long long *h_lambda = static_cast<long long *>(malloc(sizeof(long long) * (size_t)N));
    struct Free {
        void *a, *b, *c;
        ~Free() { free(a); free(b); free(c); }
    } guard{h_limits, h_stats, h_lambda};
    if (!h_limits || !h_stats || !h_lambda) return fail(NBOS_ERR_NO_MEMORY, "host allocation failed");
    for (int n = 0; n < N; ++n) h_limits[n] = make_int2(d->limit_num[n], d->limit_den[n]);

    NBOS_CUDA_TRY(cudaMemsetAsync(ws + lay.off_status, 0, 256, stream));
    NBOS_CUDA_TRY(cudaMemcpyAsync(d_limits, h_limits, sizeof(int2) * (size_t)N,
                                  cudaMemcpyHostToDevice, stream));
    init_stats_kernel<<<(N + 255) / 256, 256, 0, stream>>>(d_stats, N);

    ScanArgs sa{d_G, d_S, d_C, d_AV, d_AC, d_AM, d_limits, d_stats, H, s->R, s->flags};
    int bx = (H + 255) / 256;
    if (bx > 64) bx = 64;
    scan_kernel<<<dim3(bx, N), 256, 0, stream>>>(sa);
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
        for (int G = 1; G <= NBOS_MAX_GPUS_PER_HOST; ++G) {
            if (!(st.g_mask[G >> 6] >> (G & 63) & 1ull)) continue;
            lambda = lambda / gcd_u64(lambda, (unsigned long long)G) * (unsigned long long)G;
            if (lambda > (1ull << 40))
                return fail(NBOS_ERR_RANGE, "snapshot %d: GPU counts per host too diverse for an exact 63-bit key", n);
        }
        h_lambda[n] = (long long)lambda;
        if (st.idle_max > idle_max) idle_max = st.idle_max;
        if (st.g_min != INT_MAX) {
            const unsigned long long w_max = lambda / (unsigned long long)st.g_min;
            if (st.sub_max > (1ull << 62) / (w_max ? w_max : 1))
                return fail(NBOS_ERR_RANGE, "snapshot %d: subscription values too large for a 63-bit key", n);
            const unsigned long long m = st.sub_max * w_max;
            if (m > sr_max) sr_max = m;
        }
    }
    KeyLayout k;
    k.bits_idle = bits_for((unsigned long long)idle_max);
    k.bits_sr = bits_for(sr_max);
    k.bits_id = bits_for((unsigned long long)(Hpad - 1));
    const int total_bits = k.bits_idle + k.bits_sr + k.bits_id;
    if (total_bits > 63) return fail(NBOS_ERR_RANGE, "ranking key needs %d bits (max 63)", total_bits);
    k.key_bits = (total_bits <= 31 && !(s->flags & NBOS_FORCE_KEY64)) ? 32 : 64;
    s->key = k;

    NBOS_CUDA_TRY(cudaMemcpyAsync(d_lambda, h_lambda, sizeof(long long) * (size_t)N,
                                  cudaMemcpyHostToDevice, stream));
    EmitArgs ea{d_G, d_S, d_C, d_AV, d_AC, d_AM, d_limits, d_lambda,
                reinterpret_cast<int4 *>(ws + lay.off_feas), ws + lay.off_ab,
                H, Hpad, s->R, s->flags, s->key_order, idle_max, k.bits_idle, k.bits_sr, k.bits_id};
    dim3 grid((Hpad + 255) / 256, N);
    if (k.key_bits == 32)
        emit_kernel<unsigned int, uint2><<<grid, 256, 0, stream>>>(ea);
    else
        emit_kernel<unsigned long long, ulonglong2><<<grid, 256, 0, stream>>>(ea);
    NBOS_CUDA_TRY(cudaGetLastError());
    s->d_status = reinterpret_cast<unsigned int *>(ws + lay.off_status);
    s->d_feas = reinterpret_cast<const int4 *>(ws + lay.off_feas);
    s->d_ab = ws + lay.off_ab;
    return NBOS_OK;
}

}  // namespace nbos
