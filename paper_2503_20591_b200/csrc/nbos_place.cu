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
#include <type_traits>

#include "nbos_internal.h"
#include "nbos_ptx.cuh"
#include "nbos_ranked_chunk.cuh"
#include "nbos_sorted_chunk.cuh"

namespace nbos {
namespace {

constexpr int kComputeThreads = 224;
constexpr int kComputeWarps = kComputeThreads / 32;
constexpr int kThreads = kComputeThreads + 32;  // + the copy warp = 256

// How a (request, host) pair is evaluated; chosen per snapshot when it is derived.
enum : int {
    MODE_KEY64 = 0,          // 64-bit keys, plain C++ compares                (records: feas + ab)
    MODE_PLAIN = 1,          // 32-bit keys, four compares + multiply-add       (records: feas + ab)
    MODE_PACKED = 2,         // 32-bit keys, two packed subtractions + multiply-add   (records: pk)
    MODE_PACKED_STATIC = 3,  // as 2, but B is the same on every host: rank by A alone (records: pk)
    MODE_PACKED2 = 4,        // as 2, the two words have their low guard bit at different positions
    MODE_PACKED2_STATIC = 5, // as 3, likewise
    MODE_SORTED = 6,         // as 3, and the records are stored in ascending key order: a feasible host
                             // enters the best three exactly while the request has fewer than three,
                             // so the key compare is replaced by retiring the request's packed words
    MODE_SORTED2 = 7,        // as 6 with two guard masks
    MODE_GROUPED = 8,        // hosts differ in key slope (GPU count) but the table is stored count by count,
                             // each group in ascending key order: every group is treated like a table in
                             // key order (a request is retired for the rest of a group once it has three
                             // hosts of that group), keys are computed only for the hosts that fit
    MODE_GROUPED2 = 9,       // as 8 with two guard masks
    MODE_RANKED = 10,        // static key, table in key order: capacities and rank in one 64-bit value per
                             // host and per request, one subtraction + one logic operation per pair;
                             // pairs that pass are re-tested exactly          (records: rk, then feas + ab)
    MODE_RANKED2 = 11,       // as 10 behind a first level: one 32-bit word per host and per request, one
                             // subtraction + one logic operation per pair; chunks in which a pair passes
                             // go through the two-word test               (records: rk + rk1, then feas + ab)
    MODE_RANKED_GROUPS = 12,   // as 10 for a table stored GPU count by GPU count: a block walks the groups one
                               // after the other, each like a table in key order; best three kept as keys
    MODE_RANKED2_GROUPS = 13,  // as 11, likewise
    MODE_COUNT = 14,
};
__host__ __device__ constexpr bool mode_is_ranked(int mode) { return mode >= MODE_RANKED && mode <= MODE_RANKED2_GROUPS; }
__host__ __device__ constexpr bool mode_ranked_two_levels(int mode) { return mode == MODE_RANKED2 || mode == MODE_RANKED2_GROUPS; }
__host__ __device__ constexpr bool mode_ranked_by_group(int mode) { return mode == MODE_RANKED_GROUPS || mode == MODE_RANKED2_GROUPS; }
__host__ __device__ constexpr bool mode_is_packed(int mode) { return mode >= MODE_PACKED && mode <= MODE_GROUPED2; }
__host__ __device__ constexpr bool mode_is_sorted(int mode) { return mode == MODE_SORTED || mode == MODE_SORTED2; }
__host__ __device__ constexpr bool mode_is_grouped(int mode) { return mode == MODE_GROUPED || mode == MODE_GROUPED2; }
// modes whose pair step is the capacity test alone (chained predicate, no key work per pair)
__host__ __device__ constexpr bool mode_is_chained(int mode) { return mode_is_sorted(mode) || mode_is_grouped(mode); }
__host__ __device__ constexpr bool mode_is_static(int mode) { return mode == MODE_PACKED_STATIC || mode == MODE_PACKED2_STATIC || mode_is_sorted(mode); }
__host__ __device__ constexpr bool mode_two_masks(int mode) { return mode == MODE_PACKED2 || mode == MODE_PACKED2_STATIC || mode == MODE_SORTED2 || mode == MODE_GROUPED2; }
__host__ __device__ constexpr int mode_record_bytes(int mode) { return mode == MODE_KEY64 ? 32 : mode == MODE_PLAIN ? 24 : mode_is_ranked(mode) ? (mode_ranked_two_levels(mode) ? 12 : 8) : 16; }
__host__ __device__ constexpr int mode_max_q(int mode) { return mode == MODE_KEY64 ? 4 : 8; }
// Resident blocks per SM the kernels are compiled for. The modes that rank hosts by their own key
// touch most best-three registers only on the rare update path, so 64 registers (a few spills
// there) buy a fourth block; with the key computed per pair the same limit spills in the loop
// (measured slower), so those modes stay at two blocks.
__host__ __device__ constexpr int mode_blocks_per_sm(int mode) { return (mode_is_chained(mode) || mode_is_static(mode) || mode_is_ranked(mode)) ? 4 : 2; }
constexpr int kStages = 3;

struct PlaceParams {
    const int4 *feas;       // [N][Hpad]
    const void *ab;         // [N][Hpad] pairs (A, B)
    const uint4 *pk;        // [N][Hpad] (word0, word1, A, B), packed modes
    const uint2 *rk;        // [N][Hpad] (word0, word1), ranked modes
    const unsigned int *rk1;  // [N][Hpad] first-level word, MODE_RANKED2
    PackLayout pack;
    RankLayout rank;
    const int4 *requests;   // [N * B]
    int32_t *out_hosts;     // [N * B * 3]
    int32_t *out_found;     // [N * B] or null
    void *cand;             // [K][N * B][3] keys, only when K > 1
    unsigned int *status;
    long long B, total;     // requests per snapshot, N * B
    long long first_req, n_req;  // this launch handles flattened requests [first_req, first_req + n_req)
    int N, Hpad;
    int tile_hosts, tiles_total, K, req_ctas;
    int per_snapshot;       // > 0: blocks do not share snapshots, each snapshot's requests go to this many blocks
    const int *group_bounds;  // non-null: the K host slices are the GPU-count groups of each snapshot,
                              // [N][kGroupSlices + 1] table positions (ranked form of grouped tables)
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


// ---- the list of passes a block makes over its share of the requests ----------------------
// A block owns the flattened request range [lo, hi) of [0, N * B). It is cut at snapshot
// boundaries and then into passes of up to Q * groups requests: full passes of max_q, then one
// pass with the smallest power of two that covers the rest. Copy warp and compute threads walk
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
        // the smallest power of two that covers what is left, but at least 2 requests per lane: a
        // half-empty pass of 2 is cheaper than a full pass of 1 (per-host overhead dominates there)
        q = max_q;
        while (q > 2 && (long long)(q >> 1) * groups >= rem) q >>= 1;
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
    if (p.per_snapshot > 0) {
        // snapshot cr / per_snapshot, part cr % per_snapshot of its requests (units of 32)
        const long long n = cr / p.per_snapshot, part = cr % p.per_snapshot;
        const long long units_b = (p.B + 31) >> 5;
        lo = (units_b * part / p.per_snapshot) << 5;
        hi = (units_b * (part + 1) / p.per_snapshot) << 5;
        if (lo > p.B) lo = p.B;
        if (hi > p.B) hi = p.B;
        lo += n * p.B;
        hi += n * p.B;
        return;
    }
    // split in units of 32 requests so that a warp's 128-bit loads start on a 512-byte line
    const long long units = (p.n_req + 31) >> 5;
    lo = (units * cr / p.req_ctas) << 5;
    hi = (units * (cr + 1) / p.req_ctas) << 5;
    if (lo > p.n_req) lo = p.n_req;
    if (hi > p.n_req) hi = p.n_req;
    lo += p.first_req;
    hi += p.first_req;
}

// ---- the host slice of a block -----------------------------------------------------------------
// Hosts [lo, hi) of the table are staged (tile by tile), of which [real_lo, real_hi) are the
// block's to evaluate. Ordinary slices are runs of whole tiles and the two ranges coincide. The
// slices of a grouped table are its GPU-count groups, which start anywhere: the staged range is
// widened to multiples of four hosts (16-byte copies), and what lies outside the group is ignored.
struct SliceRange {
    int lo, hi, real_lo, real_hi;
};
__device__ __forceinline__ SliceRange slice_range(const PlaceParams &p, int n, int slice)
{
    SliceRange r;
    if (p.group_bounds) {
        const int *b = p.group_bounds + (size_t)n * (kGroupSlices + 1);
        r.real_lo = b[slice];
        r.real_hi = b[slice + 1];
        if (r.real_hi <= r.real_lo) {
            r.lo = r.hi = r.real_lo = r.real_hi = 0;
        } else {
            r.lo = r.real_lo & ~3;
            r.hi = (r.real_hi + 3) & ~3;
        }
    } else {
        const int T = p.tile_hosts;
        r.lo = (p.tiles_total * slice / p.K) * T;          // tiles_total * K stays far below 2^31
        r.hi = (p.tiles_total * (slice + 1) / p.K) * T;
        if (r.hi > p.Hpad) r.hi = p.Hpad;
        r.real_lo = r.lo;
        r.real_hi = r.hi;
    }
    return r;
}

// ---- the pair step --------------------------------------------------------------------------
// Fast path of the 32-bit modes: decide whether this pair would enter the request's best three
// and, if so, bump a per-thread counter (a predicated FADD, off the integer pipe). The update
// itself is rare and happens once per host behind a single branch (see run_pass). The inline
// PTX pins the instruction selection: compares chained through one predicate, the subtractions
// and the key on the multiply pipe.
__device__ __forceinline__ void pair_plain(float &cnt, unsigned int t3, int g, int v, int c, int m,
                                           const int4 &f, const uint2 &ab)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .u32 key;\n\t"
        "setp.le.s32 p, %2, %6;\n\t"
        "setp.le.and.s32 p, %3, %7, p;\n\t"
        "setp.le.and.s32 p, %4, %8, p;\n\t"
        "setp.le.and.s32 p, %5, %9, p;\n\t"
        "mad.lo.u32 key, %2, %11, %10;\n\t"
        "setp.lt.and.u32 p, key, %1, p;\n\t"
        "@p add.f32 %0, %0, 0f3F800000;\n\t}"
        : "+f"(cnt)
        : "r"(t3), "r"(g), "r"(v), "r"(c), "r"(m), "r"(f.x), "r"(f.y), "r"(f.z), "r"(f.w), "r"(ab.x), "r"(ab.y));
}
// Packed capacity test: both words are subtracted; a guard bit that fell means some capacity is
// smaller than the ask. lop3 0x2a = ~(a & b) & c, with the "result != 0" predicate.
__device__ __forceinline__ void pair_packed(float &cnt, unsigned int t3, unsigned int r0, unsigned int r1,
                                            unsigned int g, const uint4 &h, unsigned int guards)
{
    asm volatile(
        "{\n\t.reg .pred p, bad;\n\t.reg .u32 d0, d1, e, key;\n\t"
        "mad.lo.u32 d0, %2, 0xffffffff, %5;\n\t"
        "mad.lo.u32 d1, %3, 0xffffffff, %6;\n\t"
        "lop3.and.b32 e|bad, d0, d1, %9, 0x2a, 1;\n\t"
        "mad.lo.u32 key, %4, %8, %7;\n\t"
        "setp.lt.and.u32 p, key, %1, !bad;\n\t"
        "@p add.f32 %0, %0, 0f3F800000;\n\t}"
        : "+f"(cnt)
        : "r"(t3), "r"(r0), "r"(r1), "r"(g), "r"(h.x), "r"(h.y), "r"(h.z), "r"(h.w), "r"(guards));
}
__device__ __forceinline__ void pair_packed_static(float &cnt, unsigned int t3, unsigned int r0,
                                                   unsigned int r1, const uint4 &h, unsigned int guards)
{
    asm volatile(
        "{\n\t.reg .pred p, bad;\n\t.reg .u32 d0, d1, e;\n\t"
        "mad.lo.u32 d0, %2, 0xffffffff, %4;\n\t"
        "mad.lo.u32 d1, %3, 0xffffffff, %5;\n\t"
        "lop3.and.b32 e|bad, d0, d1, %7, 0x2a, 1;\n\t"
        "setp.lt.and.u32 p, %6, %1, !bad;\n\t"
        "@p add.f32 %0, %0, 0f3F800000;\n\t}"
        : "+f"(cnt)
        : "r"(t3), "r"(r0), "r"(r1), "r"(h.x), "r"(h.y), "r"(h.z), "r"(guards));
}

// Two-mask forms: 0x0c = ~a & b on (d0, guards0); 0xf2 = a | (~b & c) on (e0, d1, guards1).
__device__ __forceinline__ void pair_packed2(float &cnt, unsigned int t3, unsigned int r0, unsigned int r1,
                                             unsigned int g, const uint4 &h, unsigned int guards0,
                                             unsigned int guards1)
{
    asm volatile(
        "{\n\t.reg .pred p, bad;\n\t.reg .u32 d0, d1, e0, e, key;\n\t"
        "mad.lo.u32 d0, %2, 0xffffffff, %5;\n\t"
        "mad.lo.u32 d1, %3, 0xffffffff, %6;\n\t"
        "lop3.b32 e0, d0, %9, 0, 0x0c;\n\t"
        "lop3.and.b32 e|bad, e0, d1, %10, 0xf2, 1;\n\t"
        "mad.lo.u32 key, %4, %8, %7;\n\t"
        "setp.lt.and.u32 p, key, %1, !bad;\n\t"
        "@p add.f32 %0, %0, 0f3F800000;\n\t}"
        : "+f"(cnt)
        : "r"(t3), "r"(r0), "r"(r1), "r"(g), "r"(h.x), "r"(h.y), "r"(h.z), "r"(h.w), "r"(guards0), "r"(guards1));
}
__device__ __forceinline__ void pair_packed2_static(float &cnt, unsigned int t3, unsigned int r0,
                                                    unsigned int r1, const uint4 &h, unsigned int guards0,
                                                    unsigned int guards1)
{
    asm volatile(
        "{\n\t.reg .pred p, bad;\n\t.reg .u32 d0, d1, e0, e;\n\t"
        "mad.lo.u32 d0, %2, 0xffffffff, %4;\n\t"
        "mad.lo.u32 d1, %3, 0xffffffff, %5;\n\t"
        "lop3.b32 e0, d0, %7, 0, 0x0c;\n\t"
        "lop3.and.b32 e|bad, e0, d1, %8, 0xf2, 1;\n\t"
        "setp.lt.and.u32 p, %6, %1, !bad;\n\t"
        "@p add.f32 %0, %0, 0f3F800000;\n\t}"
        : "+f"(cnt)
        : "r"(t3), "r"(r0), "r"(r1), "r"(h.x), "r"(h.y), "r"(h.z), "r"(guards0), "r"(guards1));
}

template <int MODE> struct ModeTraits {
    using Key = unsigned int;
    using Pair = uint2;
};
template <> struct ModeTraits<MODE_KEY64> {
    using Key = unsigned long long;
    using Pair = ulonglong2;
};

// ---- one pass: Q requests per group through all tiles of the block's host slice ------------
template <int Q, int L, int MODE>
__device__ __forceinline__ bool run_pass(const PlaceParams &p, unsigned char *stages,
                                         uint32_t stage_bytes, uint32_t full_bar,
                                         uint32_t empty_bar, volatile unsigned int *abort_flag,
                                         uint32_t &ring_pos, int tile_begin, int tile_end,
                                         int slice, long long first, int count)
{
    using KeyT = typename ModeTraits<MODE>::Key;
    using Pair = typename ModeTraits<MODE>::Pair;
    constexpr KeyT kInf = KeyTraits<KeyT>::kInf;
    constexpr bool kPacked = mode_is_packed(MODE);
    constexpr int kGroups = kComputeThreads / L;
    const int tid = threadIdx.x;
    const int sub = tid % L;
    const int grp = tid / L;
    const int lane = tid & 31;

    // request registers: plain modes keep the four asks, packed modes the two packed words
    int g[Q], v[kPacked ? 1 : Q], c[kPacked ? 1 : Q], m[kPacked ? 1 : Q];
    unsigned int r0[kPacked ? Q : 1], r1[kPacked ? Q : 1];
    // grouped modes: the key slope of the group the lane is in, and hosts found in that group
    // (4 bits per request)
    unsigned int group_slope = 0xFFFFFFFFu, group_found = 0u;
    (void)group_slope; (void)group_found;
    KeyT t1[Q], t2[Q], t3[Q];
    // request q of this lane, packed into the two words of the packed capacity test
    auto load_packed = [&](int q, unsigned int &w0, unsigned int &w1, int &gpus) {
        const int idx = q * kGroups + grp;
        int4 r = make_int4(-1, 0, 0, 0);
        if (idx < count) r = __ldg(p.requests + first + idx);
        // an ask that is negative or larger than every host's capacity fits nowhere: encode it
        // as a GPU ask above every host's gmax and keep the other fields inside their widths
        const bool bad = ((r.x | r.y | r.z | r.w) < 0) | (r.x > p.pack.fmax[0]) | (r.y > p.pack.fmax[1]) |
                         (r.z > p.pack.fmax[2]) | (r.w > p.pack.fmax[3]);
        const unsigned int val[4] = {bad ? (unsigned int)p.pack.fmax[0] + 2u : (unsigned int)r.x + 1u,
                                     bad ? 0u : (unsigned int)r.y, bad ? 0u : (unsigned int)r.z,
                                     bad ? 0u : (unsigned int)r.w};
        w0 = 0u; w1 = 0u;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned int piece = val[k] << p.pack.fshift[k];
            if (p.pack.fword[k]) w1 |= piece; else w0 |= piece;
        }
        gpus = bad ? 0 : r.x;
    };
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        if (kPacked) {
            load_packed(q, r0[q], r1[q], g[q]);
        } else {
            const int idx = q * kGroups + grp;
            int4 r = make_int4(-1, 0, 0, 0);
            if (idx < count) r = __ldg(p.requests + first + idx);
            if ((r.x | r.y | r.z | r.w) < 0) r.x = INT_MAX;  // a negative ask fits nowhere
            g[q] = r.x; v[q] = r.y; c[q] = r.z; m[q] = r.w;
        }
        t1[q] = kInf; t2[q] = kInf; t3[q] = kInf;
    }

    const int T = p.tile_hosts;
    for (int t = tile_begin; t < tile_end; ++t, ++ring_pos) {
        const uint32_t s = ring_pos % kStages;
        const uint32_t parity = (ring_pos / kStages) & 1u;
        if (!mbar_wait(full_bar + 8u * s, parity, abort_flag)) return false;
        const unsigned char *stage = stages + (size_t)s * stage_bytes;
        int hosts = p.Hpad - t * T;
        if (hosts > T) hosts = T;
        if (MODE == MODE_KEY64) {
            const int4 *F = reinterpret_cast<const int4 *>(stage);
            const Pair *AB = reinterpret_cast<const Pair *>(stage + (size_t)T * 16);
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
        } else if (MODE == MODE_PLAIN) {
            const int4 *F = reinterpret_cast<const int4 *>(stage);
            const uint2 *AB = reinterpret_cast<const uint2 *>(stage + (size_t)T * 16);
            float cnt = 0.f, seen = 0.f;
            auto chunk = [&](auto width, int i0) {
                constexpr int W = decltype(width)::value;
                int4 f[W];
                uint2 ab[W];
#pragma unroll
                for (int u = 0; u < W; ++u) { f[u] = F[i0 + u * L]; ab[u] = AB[i0 + u * L]; }
#pragma unroll
                for (int u = 0; u < W; ++u)
#pragma unroll
                    for (int q = 0; q < Q; ++q) pair_plain(cnt, (unsigned int)t3[q], g[q], v[q], c[q], m[q], f[u], ab[u]);
                if (cnt != seen) {  // rare: some request of this lane takes one of these hosts
                    seen = cnt;
#pragma unroll
                    for (int u = 0; u < W; ++u)
#pragma unroll
                        for (int q = 0; q < Q; ++q) {
                            const bool ok = (g[q] <= f[u].x) & (v[q] <= f[u].y) & (c[q] <= f[u].z) & (m[q] <= f[u].w);
                            const KeyT key = ok ? (KeyT)((unsigned int)g[q] * ab[u].y + ab[u].x) : kInf;
                            insert3(t1[q], t2[q], t3[q], key);
                        }
                }
            };
            int i = sub;
            for (; i + 3 * L < hosts; i += 4 * L) chunk(std::integral_constant<int, 4>{}, i);
            for (; i < hosts; i += L) chunk(std::integral_constant<int, 1>{}, i);
        } else {
            const uint4 *R = reinterpret_cast<const uint4 *>(stage);
            const unsigned int guards0 = p.pack.guards, guards1 = p.pack.guards1;
            float cnt = 0.f, seen = 0.f;
            (void)cnt; (void)seen;
            auto chunk = [&](auto width, int i0) {
                constexpr int W = decltype(width)::value;
                uint4 h[W];
#pragma unroll
                for (int u = 0; u < W; ++u) h[u] = R[i0 + u * L];
                if constexpr (mode_is_grouped(MODE)) {
                    // a new GPU-count group begins somewhere in this chunk: every request is live again
                    // (the lane's hosts are in table order, so the last host of the chunk tells)
                    const unsigned int slope = h[W - 1].w;
                    if (slope != group_slope) {
                        group_slope = slope;
                        group_found = 0u;
                        // retired requests carry the guard mask in word 0: fetch the requests again
                        // (a handful of times per pass; keeping a copy would cost 8 registers)
#pragma unroll
                        for (int q = 0; q < Q; ++q) {
                            unsigned int w1_same;
                            int gpus_same;
                            load_packed(q, r0[q], w1_same, gpus_same);
                        }
                    }
                }
                bool hit;  // some pair of the chunk may enter its request's best three
                if constexpr (mode_is_chained(MODE)) {
                    // table in key order: the capacity test alone decides (chained predicate)
                    hit = sorted_chunk_any_fit<Q, W, mode_two_masks(MODE)>(r0, r1, h, guards0, guards1);
                } else {
#pragma unroll
                    for (int u = 0; u < W; ++u)
#pragma unroll
                        for (int q = 0; q < Q; ++q) {
                            if (MODE == MODE_PACKED) pair_packed(cnt, (unsigned int)t3[q], r0[q], r1[q], (unsigned int)g[q], h[u], guards0);
                            else if (MODE == MODE_PACKED_STATIC) pair_packed_static(cnt, (unsigned int)t3[q], r0[q], r1[q], h[u], guards0);
                            else if (MODE == MODE_PACKED2) pair_packed2(cnt, (unsigned int)t3[q], r0[q], r1[q], (unsigned int)g[q], h[u], guards0, guards1);
                            else pair_packed2_static(cnt, (unsigned int)t3[q], r0[q], r1[q], h[u], guards0, guards1);
                        }
                    hit = cnt != seen;
                    seen = cnt;
                }
                if (hit) {
#pragma unroll
                    for (int u = 0; u < W; ++u) {
#pragma unroll
                        for (int q = 0; q < Q; ++q) {
                            const unsigned int d0 = h[u].x - r0[q], d1 = h[u].y - r1[q];
                            const bool bad = ((~d0 & guards0) | (~d1 & guards1)) != 0u;
                            const unsigned int key = mode_is_static(MODE) ? h[u].z : (unsigned int)g[q] * h[u].w + h[u].z;
                            insert3(t1[q], t2[q], t3[q], (KeyT)(bad ? 0xFFFFFFFFu : key));
                            // hosts of the current group that fit this request, 4 bits per request
                            if (mode_is_grouped(MODE) && !bad && h[u].w == group_slope) group_found += 1u << (4 * q);
                        }
                    }
                    if (mode_is_grouped(MODE)) {
                        // three hosts of this group found: its later hosts all have larger keys
#pragma unroll
                        for (int q = 0; q < Q; ++q)
                            if (((group_found >> (4 * q)) & 15u) >= 3u) r0[q] = guards0;
                    }
                    if (mode_is_sorted(MODE)) {
                        // three hosts found: every later host has a larger key. Retire the request
                        // with a word equal to the guard mask, which clears every guard of any host
#pragma unroll
                        for (int q = 0; q < Q; ++q)
                            if (t3[q] != kInf) r0[q] = guards0;
                    }
                }
            };
            int i = sub;
            for (; i + 3 * L < hosts; i += 4 * L) chunk(std::integral_constant<int, 4>{}, i);
            for (; i < hosts; i += L) chunk(std::integral_constant<int, 1>{}, i);
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
                KeyT *cand = reinterpret_cast<KeyT *>(p.cand) + ((long long)slice * p.n_req + (r - p.first_req)) * 3;
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
    return true;
}

// ---- one pass in ranked form ------------------------------------------------------------------
// Same contract as run_pass. Inside one host slice (a run of tiles of a table in key order, or
// one GPU-count group of a grouped table) a smaller position is a smaller key, so "would this
// host enter the best three" is a compare of positions, which the packed words carry. A block
// walks its slices [slice_first, slice_last) one after the other. With a single slice the best
// three of a request are kept as positions (turned into keys after the last tile) and double as
// the rank threshold; a block that walks the groups of a grouped table keeps them as keys across
// the groups, and per group the positions of the first three hosts that fit give the threshold.
//
// Hosts are dealt to the L lanes of a request group in groups of four consecutive hosts (lane s
// takes groups s, s + L, ...), so that a lane's host words come in 128-bit shared-memory loads
// whatever L is.
//
// Opening. The first 16 hosts of a slice are compared exactly (four compares on the exact
// records) against every request of the pass, in table order, until a request has three hosts:
// in a table in key order most requests find their three right there, and the pair loop then
// starts with the rank thresholds already in the request words instead of going through the
// second level and the exact test for its first chunks. Every lane of a group does this (they all
// need the thresholds); lane 0 of the group keeps the finds.
//
// Pair loop, from the end of the opening on. Per pair: one subtraction and one logic operation
// on the first-level words (TWO_LEVELS), or directly the two-word test. A group of four hosts in
// which some pair passed the first level goes through the two-word test; pairs that pass that
// one too are re-tested with the exact records, fitting hosts enter the best three, and the
// request's rank fields are set from the slice's new third fit (or from the opening's,
// whichever is earlier).
constexpr int kOpeningHosts = 16;

template <int Q, int L, bool TWO_LEVELS, bool BY_GROUP>
__device__ __forceinline__ bool run_pass_ranked(const PlaceParams &p, unsigned char *stages,
                                                uint32_t stage_bytes, uint32_t full_bar,
                                                uint32_t empty_bar, volatile unsigned int *abort_flag,
                                                uint32_t &ring_pos, int slice_first, int slice_last,
                                                const SliceRange &own_slice, long long first, int count, int n)
{
    constexpr unsigned int kNone = 0xFFFFFFFFu;
    constexpr int kGroups = kComputeThreads / L;
    const int tid = threadIdx.x;
    const int sub = tid % L;
    const int grp = tid / L;
    const int lane = tid & 31;
    const size_t row = (size_t)n * p.Hpad;
    const unsigned int guards = p.rank.guards;
    const unsigned int guards1 = p.rank.l1_guards;
    const int rank_shift = p.rank.fshift[4] + 32 * p.rank.fword[4];
    const unsigned long long rank_mask = (unsigned long long)p.rank.rank_mask << (32 * p.rank.fword[4]);
    const int T = p.tile_hosts;

    // the ask as given, with a GPU count no host has when it fits nowhere (negative field)
    auto load_request = [&](int q) -> int4 {
        const int idx = q * kGroups + grp;
        int4 r = make_int4(-1, 0, 0, 0);
        if (idx < count) r = __ldg(p.requests + first + idx);
        if ((r.x | r.y | r.z | r.w) < 0) r.x = INT_MAX;
        return r;
    };
    // key of the host at table position `pos` for a request of g GPUs: A + g * B (low bits = host id)
    auto key_at = [&](unsigned int pos, int g) -> unsigned int {
        const uint2 ab = __ldg(reinterpret_cast<const uint2 *>(p.ab) + row + pos);
        return ab.x + (unsigned int)g * ab.y;
    };

    // Two-word form of each request. With two levels it is needed only in the chunks that pass
    // the first level, and is kept in local memory (indexed dynamically below) so that the pair
    // loop has its registers for first-level words; otherwise it stays in registers.
    unsigned long long rq_keep[Q];
    unsigned int r1[TWO_LEVELS ? Q : 1];   // first-level word
    constexpr bool by_group = BY_GROUP;
    unsigned int best[3 * Q];  // the best three, [0, Q) best, [Q, 2Q) second, [2Q, 3Q) third: positions, or
                               // (by_group) keys over all groups
    unsigned int fits[BY_GROUP ? 3 * Q : 1];  // by_group: positions of the first three hosts of the current group that fit
    unsigned int field[Q];     // rank field of each request after an update
    unsigned int opened[Q];    // position of the third host the opening found (kNone: fewer than three)

#pragma unroll
    for (int q = 0; q < Q; ++q) {
        best[q] = kNone; best[Q + q] = kNone; best[2 * Q + q] = kNone;
    }
    bool words_built = false;

    // slice after slice: the opening, then the pair loop over the slice's tiles. (A block with one
    // slice has the same host range in every pass, computed once by the caller; its loop below runs
    // once.)
    int sl = slice_first;
    do {
        const SliceRange sr = BY_GROUP ? slice_range(p, n, sl) : own_slice;
        if (BY_GROUP && sr.hi <= sr.lo) continue;
        // ---- opening: the first hosts of the slice, exactly, eight at a time ----
        const int open_pos = sr.real_lo;
        const int open_end = min(sr.real_lo + kOpeningHosts, sr.real_hi);
        {
            unsigned int o1[Q], o2[Q], o3[Q];
            int4 ask[Q];
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                ask[q] = load_request(q);
                o1[q] = kNone; o2[q] = kNone; o3[q] = kNone;
            }
#pragma unroll 1
            for (int base = 0; base < kOpeningHosts; base += 8) {
                bool need = false;
#pragma unroll
                for (int q = 0; q < Q; ++q) need |= o3[q] == kNone;
                if (!need) break;
                int4 f[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)   // hosts past the end of a group take nothing (ordinary slices have 32 hosts or more)
                    f[u] = (!BY_GROUP || open_pos + base + u < open_end) ? __ldg(p.feas + row + open_pos + base + u)
                                                                          : make_int4(-1, 0, 0, 0);
#pragma unroll
                for (int q = 0; q < Q; ++q)
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const bool ok = (ask[q].x <= f[u].x) & (ask[q].y <= f[u].y) & (ask[q].z <= f[u].z) & (ask[q].w <= f[u].w);
                        // positions come in ascending order: a fitting host takes the first free slot
                        const unsigned int pos = (unsigned int)(open_pos + base + u);
                        const bool take3 = ok & (o2[q] != kNone) & (o3[q] == kNone);
                        const bool take2 = ok & (o1[q] != kNone) & (o2[q] == kNone);
                        const bool take1 = ok & (o1[q] == kNone);
                        o3[q] = take3 ? pos : o3[q];
                        o2[q] = take2 ? pos : o2[q];
                        o1[q] = take1 ? pos : o1[q];
                    }
            }
            if (!BY_GROUP || !words_built) {
                // the packed forms of the requests, once per pass (rank fields 0 so far)
                words_built = true;
#pragma unroll
                for (int q = 0; q < Q; ++q) {
                    const int4 r = ask[q];
                    // an ask above every host's capacity in some resource fits nowhere either: encode both
                    // cases as a GPU ask above every gmax and keep the other fields inside their widths
                    const bool bad = (r.x > p.rank.fmax[0]) | (r.y > p.rank.fmax[1]) | (r.z > p.rank.fmax[2]) |
                                     (r.w > p.rank.fmax[3]);
                    const unsigned int val[4] = {bad ? (unsigned int)p.rank.fmax[0] + 2u : (unsigned int)r.x + 1u,
                                                 bad ? 0u : (unsigned int)r.y, bad ? 0u : (unsigned int)r.z,
                                                 bad ? 0u : (unsigned int)r.w};
                    unsigned int w0 = 0u, w1 = 0u, l1 = 0u;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const unsigned int piece = (val[k] >> p.rank.fdrop[k]) << p.rank.fshift[k];
                        if (p.rank.fword[k]) w1 |= piece; else w0 |= piece;
                        l1 |= (val[k] >> p.rank.l1_drop[k]) << p.rank.l1_shift[k];
                    }
                    rq_keep[q] = (unsigned long long)w0 | ((unsigned long long)w1 << 32);
                    if constexpr (TWO_LEVELS) r1[q] = l1;
                }
            }
            const bool keeper = sub == 0;   // one lane of the group carries the opening's finds to the merge
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                // rank field from the opening's third host (0 = every rank passes)
                const unsigned int fld = o3[q] == kNone ? 0u : p.rank.rank_top + 1u - o3[q];
                rq_keep[q] = (rq_keep[q] & ~rank_mask) | ((unsigned long long)fld << rank_shift);
                if constexpr (TWO_LEVELS) r1[q] = (r1[q] & ~p.rank.l1_rank_mask) | (fld << p.rank.l1_shift[4]);
                field[q] = fld;
                opened[q] = o3[q];
                if constexpr (!BY_GROUP) {
                    best[q] = keeper ? o1[q] : kNone; best[Q + q] = keeper ? o2[q] : kNone; best[2 * Q + q] = keeper ? o3[q] : kNone;
                } else {
                    fits[q] = keeper ? o1[q] : kNone; fits[Q + q] = keeper ? o2[q] : kNone; fits[2 * Q + q] = keeper ? o3[q] : kNone;
                    if (keeper && o1[q] != kNone) {
                        unsigned int a1 = best[q], a2 = best[Q + q], a3 = best[2 * Q + q];
                        insert3(a1, a2, a3, key_at(o1[q], ask[q].x));
                        if (o2[q] != kNone) insert3(a1, a2, a3, key_at(o2[q], ask[q].x));
                        if (o3[q] != kNone) insert3(a1, a2, a3, key_at(o3[q], ask[q].x));
                        best[q] = a1; best[Q + q] = a2; best[2 * Q + q] = a3;
                    }
                }
            }
        }

        for (int pos0 = sr.lo; pos0 < sr.hi; pos0 += T, ++ring_pos) {
            const uint32_t s = ring_pos % kStages;
            const uint32_t parity = (ring_pos / kStages) & 1u;
            if (!mbar_wait(full_bar + 8u * s, parity, abort_flag)) return false;
            const unsigned long long *R = reinterpret_cast<const unsigned long long *>(stages + (size_t)s * stage_bytes);
            const unsigned int *R1 = reinterpret_cast<const unsigned int *>(R + T);
            int hosts = sr.hi - pos0;
            if (hosts > T) hosts = T;
            const int n_groups = hosts >> 2;   // groups of four hosts in this tile (hosts is a multiple of 4)

            // two-word test of host group gi (hosts 4 gi .. 4 gi + 3 of the tile) against the Q
            // requests, then the exact part
            auto group2 = [&](int gi) {
                unsigned long long h[4];
                {
                    const ulonglong2 a = *reinterpret_cast<const ulonglong2 *>(R + 4 * gi);
                    const ulonglong2 b = *reinterpret_cast<const ulonglong2 *>(R + 4 * gi + 2);
                    h[0] = a.x; h[1] = a.y; h[2] = b.x; h[3] = b.y;
                }
                unsigned long long rq[Q];
#pragma unroll
                for (int q = 0; q < Q; ++q) rq[q] = rq_keep[q];
                if (!ranked_chunk_any_pass<Q, 4>(rq, h, guards)) return;
                // rare. Which pairs passed (bit 4 q + u), with static register indices ...
                unsigned int passed = 0u;
#pragma unroll
                for (int q = 0; q < Q; ++q)
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const unsigned long long d = h[u] - rq[q];
                        const unsigned int fell = ~((unsigned int)d & (unsigned int)(d >> 32)) & guards;
                        passed |= (fell == 0u ? 1u : 0u) << (q * 4 + u);
                    }
                // ... then one pair after the other: exact test against the request as given; the
                // best-three arrays are indexed dynamically here and therefore live in local memory,
                // which keeps their registers out of the pair loop
                unsigned int touched = 0u;
                while (passed) {
                    const int bit = __ffs(passed) - 1;
                    passed &= passed - 1u;
                    const int q = bit >> 2, u = bit & 3;
                    const unsigned int pos = (unsigned int)(pos0 + 4 * gi + u);
                    // the opening has dealt with the group's first hosts; what was staged beyond the
                    // group's ends belongs to a neighbouring group. (Ordinary slices are whole tiles
                    // and the pair loop starts right behind the opening: nothing to leave out.)
                    if constexpr (BY_GROUP)
                        if ((int)pos < open_end || (int)pos >= sr.real_hi) continue;
                    const int4 r = load_request(q);
                    const int4 f = __ldg(p.feas + row + pos);
                    if ((r.x <= f.x) & (r.y <= f.y) & (r.z <= f.z) & (r.w <= f.w)) {
                        unsigned int a1 = best[q], a2 = best[Q + q], a3 = best[2 * Q + q];
                        insert3(a1, a2, a3, by_group ? key_at(pos, r.x) : pos);
                        best[q] = a1; best[Q + q] = a2; best[2 * Q + q] = a3;
                        unsigned int f3 = a3;
                        if constexpr (BY_GROUP) {
                            unsigned int f1 = fits[q], f2 = fits[Q + q];
                            f3 = fits[2 * Q + q];
                            insert3(f1, f2, f3, pos);
                            fits[q] = f1; fits[Q + q] = f2; fits[2 * Q + q] = f3;
                        }
                        const unsigned int third = min(f3, opened[q]);   // the other lanes' opening finds count too
                        field[q] = third == kNone ? 0u : p.rank.rank_top + 1u - third;
                        if constexpr (TWO_LEVELS)
                            rq_keep[q] = (rq_keep[q] & ~rank_mask) | ((unsigned long long)field[q] << rank_shift);
                        touched = 1u;
                    }
                }
                if (touched) {
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        if constexpr (TWO_LEVELS) r1[q] = (r1[q] & ~p.rank.l1_rank_mask) | (field[q] << p.rank.l1_shift[4]);
                        else rq_keep[q] = (rq_keep[q] & ~rank_mask) | ((unsigned long long)field[q] << rank_shift);
                    }
                }
            };

            // this lane's host groups: sub, sub + L, ...; the groups that lie entirely inside the
            // opening's range are left out
            int g = sub;
            if (pos0 == sr.lo)
                while (g < ((open_end - sr.lo) >> 2)) g += L;
            if constexpr (TWO_LEVELS) {
                // first level of W / 4 host groups (g0, g0 + L, ...) against the Q requests
                auto chunk1 = [&](auto width, int g0) {
                    constexpr int W = decltype(width)::value;
                    unsigned int h1[W];
#pragma unroll
                    for (int v = 0; v < W / 4; ++v) {
                        const uint4 a = *reinterpret_cast<const uint4 *>(R1 + 4 * (g0 + v * L));
                        h1[4 * v] = a.x; h1[4 * v + 1] = a.y; h1[4 * v + 2] = a.z; h1[4 * v + 3] = a.w;
                    }
                    unsigned int groups_passed = ranked_l1_chunk_groups_passed<Q, W>(r1, h1, guards1);
                    // second level only for the groups of four hosts in which a pair passed
                    while (groups_passed) {
                        const int v = __ffs(groups_passed) - 1;
                        groups_passed &= groups_passed - 1u;
                        group2(g0 + v * L);
                    }
                };
                for (; g + 3 * L < n_groups; g += 4 * L) chunk1(std::integral_constant<int, 16>{}, g);
                for (; g < n_groups; g += L) chunk1(std::integral_constant<int, 4>{}, g);
            } else {
                for (; g < n_groups; g += L) group2(g);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar + 8u * s);
        }
    } while (BY_GROUP && ++sl < slice_last);

    // merge the L lanes of a group (keys and positions are unique, so the order of merging does not matter)
    unsigned int t1[Q], t2[Q], t3[Q];
#pragma unroll
    for (int q = 0; q < Q; ++q) { t1[q] = best[q]; t2[q] = best[Q + q]; t3[q] = best[2 * Q + q]; }
#pragma unroll
    for (int mask = 1; mask < L; mask <<= 1) {
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const unsigned int o1 = __shfl_xor_sync(0xFFFFFFFFu, t1[q], mask);
            const unsigned int o2 = __shfl_xor_sync(0xFFFFFFFFu, t2[q], mask);
            const unsigned int o3 = __shfl_xor_sync(0xFFFFFFFFu, t3[q], mask);
            insert3(t1[q], t2[q], t3[q], o1);
            insert3(t1[q], t2[q], t3[q], o2);
            insert3(t1[q], t2[q], t3[q], o3);
        }
    }

    if (sub == 0) {
        const uint2 *AB = reinterpret_cast<const uint2 *>(p.ab) + row;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int idx = q * kGroups + grp;
            if (idx >= count) continue;
            const long long r = first + idx;
            // single slice: position -> key (its low bits are the host id; all hosts of the slice
            // share the key slope, so the intercepts order like the keys)
            const unsigned int k1 = by_group || t1[q] == kNone ? t1[q] : __ldg(&AB[t1[q]].x);
            const unsigned int k2 = by_group || t2[q] == kNone ? t2[q] : __ldg(&AB[t2[q]].x);
            const unsigned int k3 = by_group || t3[q] == kNone ? t3[q] : __ldg(&AB[t3[q]].x);
            if (p.K > 1) {
                unsigned int *cand = reinterpret_cast<unsigned int *>(p.cand) + ((long long)slice_first * p.n_req + (r - p.first_req)) * 3;
                cand[0] = k1; cand[1] = k2; cand[2] = k3;
            } else {
                int32_t *o = p.out_hosts + r * 3;
                o[0] = k1 == kNone ? -1 : (int)(k1 & p.id_mask);
                o[1] = k2 == kNone ? -1 : (int)(k2 & p.id_mask);
                o[2] = k3 == kNone ? -1 : (int)(k3 & p.id_mask);
                if (p.out_found) p.out_found[r] = (k1 != kNone) + (k2 != kNone) + (k3 != kNone);
            }
        }
    }
    return true;
}

template <int L, int MODE>
__global__ void __launch_bounds__(kThreads, mode_blocks_per_sm(MODE))
place_kernel(const __grid_constant__ PlaceParams p)
{
    constexpr int MAXQ = mode_max_q(MODE);
    constexpr int kRecord = mode_record_bytes(MODE);
    constexpr bool kPacked = mode_is_packed(MODE);
    extern __shared__ __align__(128) unsigned char smem[];
    const int T = p.tile_hosts;
    const uint32_t stage_bytes = (uint32_t)T * (uint32_t)kRecord;
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
    // a block has one host slice, except for grouped tables in the ranked form, whose blocks walk
    // all GPU-count groups (K = 1 there)
    const int slice_first = mode_ranked_by_group(MODE) ? 0 : slice;
    const int slice_last = mode_ranked_by_group(MODE) ? kGroupSlices : slice + 1;
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
        SliceRange copy_slice = {0, 0, 0, 0};
        if (!mode_ranked_by_group(MODE)) copy_slice = slice_range(p, 0, slice);
        while (ok && passes.next(n, first, count, q)) {
            const size_t row = (size_t)n * p.Hpad;
            for (int sl = slice_first; ok && sl < slice_last; ++sl) {
            const SliceRange sr = mode_ranked_by_group(MODE) ? slice_range(p, n, sl) : copy_slice;
            for (int pos0 = sr.lo; pos0 < sr.hi; pos0 += T, ++issued) {
                const uint32_t s = issued % kStages;
                if (issued >= (uint32_t)kStages) {
                    const uint32_t parity = ((issued / kStages) - 1u) & 1u;
                    if (!mbar_wait(empty_bar + 8u * s, parity, abort_flag)) {
                        ok = false;
                        break;
                    }
                }
                int hosts = sr.hi - pos0;
                if (hosts > T) hosts = T;
                const uint32_t dst = stage0 + s * stage_bytes;
                if (mode_is_ranked(MODE)) {
                    // pos0 and hosts are multiples of four: 16-byte aligned sources and sizes
                    const uint32_t bytes = (uint32_t)hosts * 8u;
                    const uint32_t bytes1 = mode_ranked_two_levels(MODE) ? (uint32_t)hosts * 4u : 0u;
                    mbar_arrive_expect_tx(full_bar + 8u * s, bytes + bytes1);
                    bulk_copy_g2s(dst, p.rk + row + pos0, bytes, full_bar + 8u * s);
                    if (mode_ranked_two_levels(MODE))
                        bulk_copy_g2s(dst + (uint32_t)T * 8u, p.rk1 + row + pos0, bytes1, full_bar + 8u * s);
                } else if (kPacked) {
                    const uint32_t bytes = (uint32_t)hosts * 16u;
                    mbar_arrive_expect_tx(full_bar + 8u * s, bytes);
                    bulk_copy_g2s(dst, p.pk + row + pos0, bytes, full_bar + 8u * s);
                } else {
                    const uint32_t pair_bytes = (uint32_t)kRecord - 16u;
                    const uint32_t bytes_f = (uint32_t)hosts * 16u;
                    const uint32_t bytes_k = (uint32_t)hosts * pair_bytes;
                    mbar_arrive_expect_tx(full_bar + 8u * s, bytes_f + bytes_k);
                    bulk_copy_g2s(dst, p.feas + row + pos0, bytes_f, full_bar + 8u * s);
                    bulk_copy_g2s(dst + (uint32_t)T * 16u,
                                  static_cast<const unsigned char *>(p.ab) + (row + (size_t)pos0) * pair_bytes,
                                  bytes_k, full_bar + 8u * s);
                }
            }
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
    // an ordinary slice (whole tiles) is the same for every snapshot
    SliceRange own_slice = {0, 0, 0, 0};
    if (!mode_ranked_by_group(MODE)) own_slice = slice_range(p, 0, slice);
    const int tile_begin = own_slice.lo / T, tile_end = (own_slice.hi + T - 1) / T;
    (void)tile_begin; (void)tile_end;
    while (ok && passes.next(n, first, count, q)) {
#define NBOS_PASS(QV)                                                                                 \
    if constexpr (mode_is_ranked(MODE))                                                               \
        ok = run_pass_ranked<QV, L, mode_ranked_two_levels(MODE), mode_ranked_by_group(MODE)>(p, smem, stage_bytes, full_bar, empty_bar, abort_flag, ring_pos,  \
                                    slice_first, slice_last, own_slice, first, count, n);             \
    else                                                                                              \
        ok = run_pass<QV, L, MODE>(p, smem, stage_bytes, full_bar, empty_bar, abort_flag, ring_pos,   \
                                   tile_begin, tile_end, slice, first, count)
        if (MAXQ >= 8 && q == 8) { NBOS_PASS(8); }
        else if (MAXQ >= 4 && q == 4) { NBOS_PASS(4); }
        else if (MAXQ >= 2 && q == 2) { NBOS_PASS(2); }
        else { NBOS_PASS(1); }
#undef NBOS_PASS
    }
    if (!ok) atomicOr(p.status, 1u);
}

// a7: merge the K per-slice candidate triples of each request.
template <typename KeyT>
__global__ void __launch_bounds__(256) merge_kernel(const KeyT *cand, int K, long long total,
                                                    long long first_req, unsigned int id_mask,
                                                    int32_t *out_hosts, int32_t *out_found)
{
    constexpr KeyT kInf = KeyTraits<KeyT>::kInf;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long r = first_req + i;
        KeyT t1 = kInf, t2 = kInf, t3 = kInf;
        for (int k = 0; k < K; ++k) {
            const KeyT *c = cand + ((long long)k * total + i) * 3;
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

// ---- first-fit variant -------------------------------------------------------------------------
// When every host has the same key slope (static key) and the table is stored in ascending key
// order, the best three feasible hosts of a request are simply the first three feasible ones in
// table order, and the scan can stop there. Same outputs as place_kernel, far fewer pairs looked
// at; reported separately from the full evaluation. 8 lanes share a request and test 8 hosts per
// step; a lane whose host fits computes its position among the group's fitting lanes from the
// ballot and writes its own output slot.
struct FirstFitParams {
    const int4 *feas;
    const void *ab;
    const uint4 *pk;
    PackLayout pack;
    const int4 *requests;
    int32_t *out_hosts, *out_found;
    long long B, first_req, n_req;
    int Hpad, key64;
    unsigned int id_mask;
};

__global__ void __launch_bounds__(256) place_first_fit_kernel(const FirstFitParams p)
{
    constexpr int kLanes = 8;
    constexpr int kGroupHosts = 32;  // hosts a group looks at before the warp takes over
    constexpr int kWide = 4;         // 32-host rows the warp loads per step once it has taken over
    const int lane = threadIdx.x & 31;
    const int sub = lane & (kLanes - 1);
    const int grp_in_warp = lane / kLanes;
    const long long groups_total = (long long)gridDim.x * (blockDim.x / kLanes);
    const long long my_group = (long long)blockIdx.x * (blockDim.x / kLanes) + threadIdx.x / kLanes;
    // all four groups of a warp make the same number of rounds, so that the ballots stay warp-wide
    const long long rounds = (p.n_req + groups_total - 1) / groups_total;
    // the next round's request is fetched while this round walks its hosts
    int4 q_next = my_group < p.n_req ? __ldg(p.requests + p.first_req + my_group) : make_int4(-1, 0, 0, 0);
    for (long long round = 0; round < rounds; ++round) {
        const long long idx = round * groups_total + my_group;
        const bool live = idx < p.n_req;
        const long long r = p.first_req + (live ? idx : 0);
        const int4 q = q_next;
        if (idx + groups_total < p.n_req) q_next = __ldg(p.requests + r + groups_total);
        else q_next = make_int4(-1, 0, 0, 0);
        const size_t row = (size_t)(r / p.B) * p.Hpad;
        bool sane = (q.x | q.y | q.z | q.w) >= 0;
        unsigned int w0 = 0u, w1 = 0u;
        if (p.pack.enabled) {
            sane = sane && q.x <= p.pack.fmax[0] && q.y <= p.pack.fmax[1] && q.z <= p.pack.fmax[2] && q.w <= p.pack.fmax[3];
            const unsigned int val[4] = {(unsigned int)q.x + 1u, (unsigned int)q.y, (unsigned int)q.z, (unsigned int)q.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned int piece = sane ? val[k] << p.pack.fshift[k] : 0u;
                if (p.pack.fword[k]) w1 |= piece; else w0 |= piece;
            }
        }
        // one host test, shared by both phases
        auto fits_host = [&](const int4 &qq, unsigned int ww0, unsigned int ww1, size_t rrow, int i,
                             unsigned int &id) -> bool {
            if (p.pack.enabled) {
                const uint4 h = __ldg(p.pk + rrow + i);
                const unsigned int d0 = h.x - ww0, d1 = h.y - ww1;
                id = h.z & p.id_mask;
                return ((~d0 & p.pack.guards) | (~d1 & p.pack.guards1)) == 0u;
            }
            const int4 f = __ldg(p.feas + rrow + i);
            id = (p.key64 ? (unsigned int)__ldg(reinterpret_cast<const ulonglong2 *>(p.ab) + rrow + i).x
                          : __ldg(reinterpret_cast<const uint2 *>(p.ab) + rrow + i).x) & p.id_mask;
            return qq.x <= f.x && qq.y <= f.y && qq.z <= f.z && qq.w <= f.w;
        };

        // phase 1: the group's 8 lanes test 8 hosts per step over the first kGroupHosts hosts;
        // most requests find their three hosts there
        int found = 0;
        bool need = live && sane;
        for (int base = 0; base < kGroupHosts && __ballot_sync(0xFFFFFFFFu, need) != 0u; base += kLanes) {
            const int i = base + sub;
            unsigned int id = 0u;
            const bool ok = need && i < p.Hpad && fits_host(q, w0, w1, row, i, id);
            const unsigned int fits = (__ballot_sync(0xFFFFFFFFu, ok) >> (grp_in_warp * kLanes)) & ((1u << kLanes) - 1u);
            const int slot = found + __popc(fits & ((1u << sub) - 1u));
            if (ok && slot < NBOS_REPLICAS_PLACED) p.out_hosts[r * 3 + slot] = (int)id;
            found += __popc(fits);
            need = need && found < NBOS_REPLICAS_PLACED && base + kLanes < p.Hpad;
        }
        // phase 2: requests that are still short get the whole warp, 32 hosts per step, one
        // request after the other (a long walk with 8 lanes would hold up the other three groups)
#pragma unroll 1
        for (int g = 0; g < 32 / kLanes; ++g) {
            const int src = g * kLanes;
            if (!__shfl_sync(0xFFFFFFFFu, (int)need, src)) continue;      // uniform across the warp
            const int4 qq = make_int4(__shfl_sync(0xFFFFFFFFu, q.x, src), __shfl_sync(0xFFFFFFFFu, q.y, src),
                                      __shfl_sync(0xFFFFFFFFu, q.z, src), __shfl_sync(0xFFFFFFFFu, q.w, src));
            const unsigned int ww0 = __shfl_sync(0xFFFFFFFFu, w0, src), ww1 = __shfl_sync(0xFFFFFFFFu, w1, src);
            const long long rr = __shfl_sync(0xFFFFFFFFu, r, src);
            const size_t rrow = (size_t)(rr / p.B) * p.Hpad;
            int ff = __shfl_sync(0xFFFFFFFFu, found, src);
            // four independent loads per step: the walk is bound by load latency, and looking at
            // up to 96 hosts too many costs nothing
            for (int base = kGroupHosts; base < p.Hpad && ff < NBOS_REPLICAS_PLACED; base += 32 * kWide) {
                bool ok[kWide];
                unsigned int id[kWide];
#pragma unroll
                for (int u = 0; u < kWide; ++u) {
                    const int i = base + u * 32 + lane;
                    id[u] = 0u;
                    ok[u] = i < p.Hpad && fits_host(qq, ww0, ww1, rrow, i, id[u]);
                }
#pragma unroll
                for (int u = 0; u < kWide; ++u) {
                    const unsigned int fits = __ballot_sync(0xFFFFFFFFu, ok[u]);
                    const int slot = ff + __popc(fits & ((1u << lane) - 1u));
                    if (ok[u] && slot < NBOS_REPLICAS_PLACED) p.out_hosts[rr * 3 + slot] = (int)id[u];
                    ff += __popc(fits);
                }
            }
            if (grp_in_warp == g) found = ff;
        }
        if (found > NBOS_REPLICAS_PLACED) found = NBOS_REPLICAS_PLACED;
        if (live) {
            if (sub < NBOS_REPLICAS_PLACED && sub >= found) p.out_hosts[r * 3 + sub] = -1;
            if (sub == 0 && p.out_found) p.out_found[r] = found;
        }
    }
}

using KernelFn = void (*)(const PlaceParams);

template <int MODE>
KernelFn pick_kernel_l(int L)
{
    switch (L) {
        case 1: return place_kernel<1, MODE>;
        case 2: return place_kernel<2, MODE>;
        case 4: return place_kernel<4, MODE>;
        case 8: return place_kernel<8, MODE>;
        case 16: return place_kernel<16, MODE>;
        case 32: return place_kernel<32, MODE>;
    }
    return nullptr;
}

KernelFn pick_kernel(int mode, int L)
{
    switch (mode) {
        case MODE_KEY64: return pick_kernel_l<MODE_KEY64>(L);
        case MODE_PLAIN: return pick_kernel_l<MODE_PLAIN>(L);
        case MODE_PACKED: return pick_kernel_l<MODE_PACKED>(L);
        case MODE_PACKED_STATIC: return pick_kernel_l<MODE_PACKED_STATIC>(L);
        case MODE_PACKED2: return pick_kernel_l<MODE_PACKED2>(L);
        case MODE_PACKED2_STATIC: return pick_kernel_l<MODE_PACKED2_STATIC>(L);
        case MODE_SORTED: return pick_kernel_l<MODE_SORTED>(L);
        case MODE_SORTED2: return pick_kernel_l<MODE_SORTED2>(L);
        case MODE_GROUPED: return pick_kernel_l<MODE_GROUPED>(L);
        case MODE_GROUPED2: return pick_kernel_l<MODE_GROUPED2>(L);
        case MODE_RANKED: return pick_kernel_l<MODE_RANKED>(L);
        case MODE_RANKED2: return pick_kernel_l<MODE_RANKED2>(L);
        case MODE_RANKED_GROUPS: return pick_kernel_l<MODE_RANKED_GROUPS>(L);
        case MODE_RANKED2_GROUPS: return pick_kernel_l<MODE_RANKED2_GROUPS>(L);
    }
    return nullptr;
}

// Resident blocks per SM of a placement kernel with `smem` bytes of dynamic shared memory, with
// the kernel's shared-memory limit raised accordingly. Both runtime calls cost microseconds, which
// is most of the host time of a small launch, so the answers are kept per (kernel, device, size).
int kernel_occupancy(KernelFn fn, int device, size_t smem, int *per_sm)
{
    struct Entry { KernelFn fn; int device; size_t smem; int per_sm; };
    static std::mutex mutex;
    static Entry cache[256];
    static int n_cached = 0;
    std::lock_guard<std::mutex> lock(mutex);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].fn == fn && cache[i].device == device && cache[i].smem == smem) {
            *per_sm = cache[i].per_sm;
            return NBOS_OK;
        }
    NBOS_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    NBOS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(per_sm, fn, kThreads, smem));
    // the attribute is per kernel: entries of the same kernel with a smaller size stay valid
    // only while the limit is not lowered, so it is only ever raised
    size_t largest = smem;
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].fn == fn && cache[i].device == device && cache[i].smem > largest) largest = cache[i].smem;
    if (largest > smem)
        NBOS_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)largest));
    if (n_cached < 256) cache[n_cached++] = Entry{fn, device, smem, *per_sm};
    return NBOS_OK;
}

int snapshot_mode(const nbos_snapshot *s, int forced)
{
    if (s->key.key_bits == 64) return MODE_KEY64;
    if ((forced == 0 || forced == 5) && s->rank.enabled) {
        const bool two = forced == 0 && s->rank.l1_enabled;
        if (s->key.grouped) return two ? MODE_RANKED2_GROUPS : MODE_RANKED_GROUPS;
        return two ? MODE_RANKED2 : MODE_RANKED;
    }
    if (forced == 1 || !s->pack.enabled) return MODE_PLAIN;
    const bool two = s->pack.guards != s->pack.guards1;
    if ((forced == 0 || forced == 4) && s->key.grouped) return two ? MODE_GROUPED2 : MODE_GROUPED;
    if (forced == 2 || !s->key.static_key) return two ? MODE_PACKED2 : MODE_PACKED;
    if (forced == 3 || !s->presorted) return two ? MODE_PACKED2_STATIC : MODE_PACKED_STATIC;
    return two ? MODE_SORTED2 : MODE_SORTED;
}

void fill_params(PlaceParams &p, const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                 int32_t *d_out_hosts, int32_t *d_out_found)
{
    p.feas = s->d_feas;
    p.ab = s->d_ab;
    p.pk = s->d_pk;
    p.rk = s->d_rk;
    p.rk1 = s->d_rk1;
    p.pack = s->pack;
    p.rank = s->rank;
    p.requests = reinterpret_cast<const int4 *>(d_requests);
    p.out_hosts = d_out_hosts;
    p.out_found = d_out_found;
    p.cand = nullptr;
    p.status = s->d_status;
    p.B = batch;
    p.total = (long long)s->N * batch;
    p.first_req = 0;
    p.n_req = p.total;
    p.per_snapshot = 0;
    p.group_bounds = nullptr;
    p.N = s->N;
    p.Hpad = s->Hpad;
    p.id_mask = (1u << s->key.bits_id) - 1u;
}

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }


// What launch_place decides before it looks at the host split: evaluation mode, tile size,
// shared memory, resident blocks per SM and lanes per request.
struct LaunchPlan {
    int mode, T, tiles_total, per_sm, blocks_per_sm, L;
    int per_snapshot;  // > 0: that many blocks per snapshot, no block works on two snapshots
    size_t smem;
};

int make_plan(const nbos_snapshot *s, long long total, long long batch, const nbos_launch_config &c,
              bool whole_batch, LaunchPlan &plan)
{
    const int mode = snapshot_mode(s, c.pair_mode);
    const int host_div = 1;
    const int record = mode_record_bytes(mode);
    const int max_q_kernel = mode_max_q(mode);

    // tile: as many hosts as fit the stage budget, at most the whole (padded) table
    int T = c.tile_hosts ? c.tile_hosts : 1024;
    if (T > s->Hpad) T = s->Hpad;
    const int max_tile = (64 * 1024) / record / 32 * 32;  // <= 64 KB per stage
    if (T > max_tile) T = max_tile;
    const int tiles_total = (s->Hpad + T - 1) / T;

    KernelFn fn1 = pick_kernel(mode, 1);
    const size_t smem = (size_t)kStages * T * record + 2 * kStages * 8 + 16;
    int per_sm = 0;
    int rc_occ = kernel_occupancy(fn1, s->device, smem, &per_sm);
    if (rc_occ) return rc_occ;
    if (per_sm < 1) return fail(NBOS_ERR_CUDA, "placement kernel does not fit on an SM (%zu bytes of shared memory)", smem);

    // Lanes per request and resident blocks per SM: for each choice, estimate the instructions a
    // compute warp of the busiest SM issues -- per pass a fixed part, a part per request of a lane
    // (load, packing, best-three updates, result store), a part per host of a lane and the pair
    // steps proper, plus the shuffle merges -- and divide by the issue rate the SM reaches with
    // that many resident blocks. The constants were fitted to timings of the five benchmark
    // shapes and of shrunk batches over all (lanes, blocks per SM) choices. Large batches end up
    // with one lane per request, small ones with a whole warp; fewer blocks than fit can win
    // because each block then gets more requests and its last pass is fuller.
    int L = c.lanes_per_request;
    int blocks_per_sm = per_sm;
    plan.per_snapshot = 0;
    {
        const bool two_level = mode_ranked_two_levels(mode);
        const double pair_cost = two_level ? 1.8 : (mode_is_sorted(mode) || mode_is_ranked(mode)) ? 3.0 : mode_is_grouped(mode) ? 3.3
                                 : mode_is_static(mode) ? 4.0 : mode_is_packed(mode) ? 5.0 : mode == MODE_PLAIN ? 7.0 : 12.0;
        // The two-level ranked form has a cheap pair step and a dearer start of every request (its
        // first hosts go through the second level and the exact test until the best three are
        // full); its constants were fitted on their own.
        const double kPassCost = two_level ? 3000.0 : 490.0, kRequestCost = two_level ? 930.0 : 190.0,
                     kHostCost = two_level ? 1.7 : 1.6, kMergeCost = 12.0;
        const double issue_rate_general[4] = {0.376, 0.472, 0.499, 0.529};  // per scheduler, by resident blocks
        const double issue_rate_two_level[4] = {0.543, 0.654, 0.774, 0.835};
        const double *issue_rate = two_level ? issue_rate_two_level : issue_rate_general;
        const long long B = batch > 0 ? batch : total;
        double best = 0.0;
        bool have = false;
        for (int cand = 1, lg = 0; cand <= 32; cand <<= 1, ++lg) {
            if (c.lanes_per_request && cand != c.lanes_per_request) continue;
            const long long groups = kComputeThreads / cand;
            const double per_host = (double)s->Hpad / host_div / cand;
            for (int j = per_sm; j >= 1; --j) {
                const long long slots = (long long)s->sm_count * j;
                // (grouped ranked form: every request is looked at by host_div blocks)
                long long ctas = (total * host_div + groups - 1) / groups;
                if (ctas > slots) ctas = slots;
                long long n_req = (total * host_div + ctas - 1) / ctas;
                n_req = (n_req + 31) / 32 * 32;
                auto pass = [&](int qq) {
                    return kPassCost + qq * kRequestCost + per_host * (kHostCost + pair_cost * qq) + lg * qq * kMergeCost;
                };
                // instructions for `len` requests of one snapshot: full passes, then one that covers the rest
                auto piece = [&](long long len) {
                    if (len <= 0) return 0.0;
                    const long long full = len / (groups * max_q_kernel), rem = len % (groups * max_q_kernel);
                    int q = max_q_kernel;
                    while (q > 2 && (long long)(q >> 1) * groups >= rem) q >>= 1;
                    return (double)full * pass(max_q_kernel) + (rem ? pass(q) : 0.0);
                };
                // the block's range is cut at snapshot boundaries, each piece into passes
                double instr = 0.0;
                if (n_req > B) {
                    instr = (double)(n_req / B) * piece(B) + piece(n_req % B);
                    if (B % n_req != 0) instr += pass(2);
                } else if (total > B && (B % n_req != 0)) {
                    // ranges that do not line up with the snapshots: some block gets the end of one
                    // snapshot and the start of the next, two partial pieces; the launch takes as long
                    // as the unluckiest split
                    for (int num = 1; num <= 4; ++num) {
                        const long long a = (n_req * num / 5 + 31) / 32 * 32;
                        const double two = piece(a) + piece(n_req - a);
                        if (two > instr) instr = two;
                    }
                } else {
                    instr = piece(n_req);
                }
                auto consider = [&](double instr_block, long long blocks, int per_snapshot) {
                    const long long on_sm = (blocks + s->sm_count - 1) / s->sm_count;
                    const int resident = (int)(on_sm < j ? on_sm : j);
                    const double cost = (double)on_sm * instr_block / issue_rate[resident > 4 ? 3 : resident - 1];
                    // candidates come with the most resident blocks first; a later one must be
                    // clearly cheaper (the estimate is good to a few per cent, and more resident
                    // warps hide the second-level and exact work of sparse workloads better)
                    if (!have || cost < best * 0.97) {
                        have = true;
                        best = cost;
                        L = cand;
                        blocks_per_sm = j;
                        plan.per_snapshot = per_snapshot;
                    }
                };
                consider(instr, ctas, 0);
                // several snapshots: also blocks that stay inside one snapshot, k per snapshot, all
                // resident at once
                if (whole_batch && total > B && !c.grid_blocks) {
                    const long long n_snap = total / B;
                    for (int k = 1; k <= 16 && n_snap * k <= slots; ++k) {
                        const long long nb = (((B + 31) / 32 + k - 1) / k) * 32;
                        if (nb < groups && k > 1) break;   // less than one request per group
                        consider(piece(nb), n_snap * k, k);
                    }
                }
            }
        }
    }
    plan.mode = mode;
    plan.T = T;
    plan.tiles_total = tiles_total;
    plan.per_sm = per_sm;
    plan.blocks_per_sm = blocks_per_sm;
    plan.L = L;
    plan.smem = smem;
    return NBOS_OK;
}

}  // namespace

int launch_place(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                 int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                 const nbos_launch_config *cfg, long long range_first, long long range_count)
{
    if (range_count < 0) range_count = (long long)s->N * batch - range_first;
    const long long total = range_count;  // requests of this launch
    if (total <= 0) return NBOS_OK;

    nbos_launch_config c = {};
    if (cfg) c = *cfg;
    if (c.reserved != 0) return fail(NBOS_ERR_INVALID_ARG, "launch config: reserved field must be 0");
    // The ranked form of a grouped table slices the hosts by GPU-count group; a caller who asks for
    // a host split of his own gets the form that can take any split.
    if (s->key.grouped && c.host_split > 0 && c.pair_mode == 0) c.pair_mode = 4;
    if (c.first_fit < 0 || c.first_fit > 1) return fail(NBOS_ERR_INVALID_ARG, "first_fit must be 0 or 1");
    if (c.lanes_per_request && !(is_pow2(c.lanes_per_request) && c.lanes_per_request <= 32))
        return fail(NBOS_ERR_INVALID_ARG, "lanes_per_request must be 1,2,4,8,16 or 32");
    if (c.requests_per_lane && !(is_pow2(c.requests_per_lane) && c.requests_per_lane <= 8))
        return fail(NBOS_ERR_INVALID_ARG, "requests_per_lane must be 1,2,4 or 8");
    if (c.host_split < 0 || c.grid_blocks < 0 || c.tile_hosts < 0 || (c.tile_hosts & 31))
        return fail(NBOS_ERR_INVALID_ARG, "launch config: negative field or tile_hosts not a multiple of 32");
    if (c.pair_mode < 0 || c.pair_mode > 5)
        return fail(NBOS_ERR_INVALID_ARG, "pair_mode must be 0 (automatic), 1 (plain compares), 2 (packed, key computed per pair), 3 (packed, host key compared per pair), 4 (key-order forms that retire requests) or 5 (ranked form without its first level)");

    if (c.first_fit && s->key.static_key && s->presorted) {
        FirstFitParams fp;
        fp.feas = s->d_feas;
        fp.ab = s->d_ab;
        fp.pk = s->d_pk;
        fp.pack = s->pack;
        fp.requests = reinterpret_cast<const int4 *>(d_requests);
        fp.out_hosts = d_out_hosts;
        fp.out_found = d_out_found;
        fp.B = batch;
        fp.first_req = range_first;
        fp.n_req = total;
        fp.Hpad = s->Hpad;
        fp.key64 = s->key.key_bits == 64;
        fp.id_mask = (1u << s->key.bits_id) - 1u;
        long long blocks = (total + 31) / 32;  // 32 groups of 8 lanes per block
        if (blocks > (long long)s->sm_count * 8) blocks = (long long)s->sm_count * 8;
        place_first_fit_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(fp);
        NBOS_CUDA_TRY(cudaGetLastError());
        return NBOS_OK;
    }

    LaunchPlan plan;
    const bool whole_batch = range_first == 0 && total == (long long)s->N * batch;
    int rc = make_plan(s, total, batch, c, whole_batch, plan);
    if (rc) return rc;
    const int mode = plan.mode, T = plan.T, tiles_total = plan.tiles_total;
    const int max_q_kernel = mode_max_q(mode);
    const bool k64 = mode == MODE_KEY64;
    const size_t smem = plan.smem;
    int per_sm = plan.per_sm;
    // Hosts are cut into slices only when the batch is so small that even a warp per request
    // leaves SMs without a block.
    const long long one_block_per_sm = (long long)s->sm_count * kComputeThreads;
    const bool by_group = mode_ranked_by_group(mode);
    int K = c.host_split;
    if (by_group) {
        K = 1;   // a block walks all GPU-count groups itself
    } else {
        if (!K) {
            K = 1;
            if (total * 32 < one_block_per_sm && !c.lanes_per_request) {
                const long long k = (one_block_per_sm + total * 32 - 1) / (total * 32);
                K = (int)(k < tiles_total ? k : tiles_total);
            }
        }
        if (K > tiles_total) K = tiles_total;
        if (K < 1) K = 1;
    }
    const int L = (K > 1 && !by_group && !c.lanes_per_request) ? 32 : plan.L;

    int max_q = c.requests_per_lane ? c.requests_per_lane : max_q_kernel;
    if (max_q > max_q_kernel) max_q = max_q_kernel;

    KernelFn fn = pick_kernel(mode, L);
    if (!fn) return fail(NBOS_ERR_INVALID_ARG, "no kernel for this launch shape");
    rc = kernel_occupancy(fn, s->device, smem, &per_sm);
    if (rc) return rc;
    if (per_sm < 1) return fail(NBOS_ERR_CUDA, "placement kernel does not fit on an SM (%zu bytes of shared memory)", smem);

    const int groups = kComputeThreads / L;
    long long req_ctas = (total + groups - 1) / groups;  // at least one request per group
    if (per_sm > plan.blocks_per_sm && (K == 1 || by_group)) per_sm = plan.blocks_per_sm;
    long long cap = (long long)s->sm_count * per_sm / K;
    if (cap < 1) cap = 1;
    if (c.grid_blocks) cap = c.grid_blocks;
    if (req_ctas > cap) req_ctas = cap;
    const int per_snapshot = (K == 1 && !c.grid_blocks) ? plan.per_snapshot : 0;
    if (per_snapshot > 0) req_ctas = (long long)s->N * per_snapshot;

    PlaceParams p;
    fill_params(p, s, d_requests, batch, d_out_hosts, d_out_found);
    p.per_snapshot = per_snapshot;
    p.group_bounds = by_group ? s->d_group_bounds : nullptr;
    p.first_req = range_first;
    p.n_req = range_count;
    p.tile_hosts = T;
    p.tiles_total = tiles_total;
    p.K = K;
    p.req_ctas = (int)req_ctas;
    p.max_q = max_q;

    if (K > 1) {
        const size_t cand_bytes = (size_t)K * (size_t)total * 3 * (k64 ? 8 : 4);
        cudaMemPool_t pool = nullptr;
        rc = library_pool(s->device, &pool);
        if (rc) return rc;
        cudaError_t e = cudaMallocFromPoolAsync(&p.cand, cand_bytes, pool, stream);
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
                static_cast<const unsigned long long *>(p.cand), K, total, p.first_req, p.id_mask, d_out_hosts, d_out_found);
        else
            merge_kernel<unsigned int><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned int *>(p.cand), K, total, p.first_req, p.id_mask, d_out_hosts, d_out_found);
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
    // (a grouped table's ranked form slices the hosts its own way; this entry point's slices are
    // the caller's, so it takes the grouped form that works with any slice)
    const int mode = snapshot_mode(s, s->key.grouped ? 4 : 0);
    const bool k64 = mode == MODE_KEY64;
    const int key_bytes = k64 ? 8 : 4;
    const int record = mode_record_bytes(mode);

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
    KernelFn fn = pick_kernel(mode, L);
    const size_t smem = (size_t)kStages * T * record + 2 * kStages * 8 + 16;
    int per_sm = 0;
    rc = kernel_occupancy(fn, device, smem, &per_sm);
    if (rc) return rc;
    if (per_sm < 1) return fail(NBOS_ERR_CUDA, "placement kernel does not fit on an SM");
    const int groups = kComputeThreads / L;
    long long req_ctas = (total + groups - 1) / groups;
    long long cap = (long long)s->sm_count * per_sm / K;
    if (cap < 1) cap = 1;
    if (req_ctas > cap) req_ctas = cap;

    PlaceParams p;
    fill_params(p, s, d_requests, batch, d_out_hosts, d_out_found);
    p.cand = K > 1 ? cand : nullptr;
    p.tile_hosts = T;
    p.tiles_total = tiles_total;
    p.K = K;
    p.req_ctas = (int)req_ctas;
    p.max_q = mode_max_q(mode);

    // Nothing in the buffer has to start at zero: the placement kernel writes all K * total * 3
    // candidate slots of this call before the merge kernel (next on the stream) reads them.
    fn<<<(unsigned int)(req_ctas * K), kThreads, smem, stream>>>(p);
    NBOS_CUDA_TRY(cudaGetLastError());
    if (K > 1) {
        long long blocks = (total + 255) / 256;
        if (blocks > (long long)s->sm_count * 8) blocks = (long long)s->sm_count * 8;
        if (k64)
            merge_kernel<unsigned long long><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned long long *>(cand), K, total, p.first_req, p.id_mask, d_out_hosts, d_out_found);
        else
            merge_kernel<unsigned int><<<(unsigned int)blocks, 256, 0, stream>>>(
                static_cast<const unsigned int *>(cand), K, total, p.first_req, p.id_mask, d_out_hosts, d_out_found);
        NBOS_CUDA_TRY(cudaGetLastError());
    }
    return NBOS_OK;
}

}  // namespace nbos
