// Internal declarations shared by the translation units of libnbos.so.
#ifndef NBOS_INTERNAL_H_
#define NBOS_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>

#include "nbos.h"

namespace nbos {

// ---- error plumbing -----------------------------------------------------------------------
int fail(int code, const char *fmt, ...);  // records the detail string, returns `code`
int cuda_fail(cudaError_t e, const char *what);

#define NBOS_CUDA_TRY(expr)                                          \
    do {                                                             \
        cudaError_t nbos_e_ = (expr);                                \
        if (nbos_e_ != cudaSuccess) return ::nbos::cuda_fail(nbos_e_, #expr); \
    } while (0)

// ---- workspace layout ---------------------------------------------------------------------
// All sections start on 256-byte boundaries.
struct SnapStats {                 // one per snapshot, filled by the scan kernel
    unsigned int err;              // bit mask of ERR_* below
    int idle_max;                  // max over hosts of G - C
    int g_min_inv;                 // INT_MAX - (min over hosts with G >= 1 of G); 0 if none
    int pad;
    unsigned long long sub_max;    // max over hosts that can take something of S + gmax
    int max_gcap1, max_av, max_ac, max_am;  // maxima of gmax + 1 and of the three capacities
    unsigned long long g_mask[16]; // bit G set if some host has G GPUs (G in 1..1023)
};
// The status section of the workspace holds two words: at offset 0 what kernels report while they
// run (kept for the life of the snapshot), at kUpdateStatusOffset what the last derivation
// reported (cleared by the next one).
constexpr size_t kUpdateStatusOffset = 128;
enum : unsigned int {  // bits of the snapshot's device status words
    STATUS_WAIT_TIMEOUT = 1u,   // a kernel gave up on a bounded wait
    STATUS_STALE_LAYOUT = 2u,   // nbos_snapshot_update: the new state does not fit the stored layout
    STATUS_BAD_VALUES = 4u,     // nbos_snapshot_update: a value outside the supported range
};
enum : unsigned int {
    ERR_NEGATIVE = 1u,        // some value < 0
    ERR_COMMITTED_GT_TOTAL = 2u,
    ERR_G_TOO_LARGE = 4u,
};

struct Layout {
    size_t off_status, off_limits, off_sums, off_stats, off_lambda, off_g_single, off_feas, off_ab, off_pk, off_rk, off_rk1;
    size_t off_tmp_feas, off_tmp_ab, off_tmp_seq, off_sortkey, off_perm, off_done, off_gbounds, total;
};
Layout workspace_layout(int n_snapshots, int hosts_padded);
inline int pad_hosts(int h) { return (h + 31) & ~31; }

constexpr int kGroupSlices = 8;   // distinct GPU counts per snapshot up to which a table is stored count by count

struct KeyLayout {
    int key_bits;  // 32 or 64
    int bits_idle, bits_sr, bits_id;
    int static_key;  // 1 if B is the same for every host that can take a request: order = order of A
    int grouped;     // 1 if B differs between hosts and the table is stored GPU count by GPU count,
                     // each group in ascending order of A (set only with a packed test and 32-bit keys)
};

// Two-compares-per-subtraction encoding of the four capacity tests. Components: 0 = GPUs
// (stored as gmax + 1 against ask + 1, so that 0 means "takes nothing"), 1 = VRAM, 2 = millicpus,
// 3 = memory. Each 32-bit word holds a low field [0, lo_bits) with its guard bit at lo_bits and
// a high field from lo_bits + 1 with its guard bit at 31. host_word - request_word keeps a
// guard bit set exactly when capacity >= ask in that field.
struct PackLayout {
    int enabled;
    int fmax[4];    // largest ask that any host could satisfy, per component
    int fword[4];   // which word (0 / 1) holds the component
    int fshift[4];  // bit position of the component inside its word
    unsigned int guards;    // guard bits of word 0
    unsigned int guards1;   // guard bits of word 1 (equal to `guards` when the layouts coincide)
};

// One-subtraction encoding of the whole pair step for snapshots whose hosts rank the same for
// every ask (static key) and whose table is stored in key order. A host is a pair of 32-bit words
// (one 64-bit value); each word has three fields at the same bit positions in both words, every
// field with a guard bit right above it (the top one at bit 31). Five of the six fields are used:
// the four capacities of Section 3.2.1 (component 0 stored as gmax + 1 against ask + 1) and the
// host's rank in the order of Section 3.4.1, stored as rank_top - position against the request's
// rank_top + 1 - (position of its current third best), so that the guard survives exactly when
// the host ranks before the third best. host - request (one 64-bit subtraction, or two 32-bit
// ones) keeps every guard set exactly when the host fits the ask in all four resources and would
// enter the request's best three. Capacities wider than their field lose their low `fdrop` bits
// on both sides: floor(ask / 2^d) <= floor(capacity / 2^d) whenever ask <= capacity, so the coarse
// test never rejects a feasible host; pairs that pass it are re-tested exactly before the best
// three change. The GPU component and the rank are always exact.
struct RankLayout {
    int enabled;
    int fmax[4];     // largest ask that any host could satisfy, per component (as PackLayout::fmax)
    int fword[5];    // word (0 / 1) of components 0..3 and of the rank (index 4)
    int fshift[5];   // bit position inside that word
    int fdrop[5];    // low bits dropped before the component is stored (0 = exact)
    unsigned int guards;    // guard bits, the same in both words
    unsigned int rank_top;  // host field = rank_top - position in the table
    unsigned int rank_mask; // bits of the rank field inside its word
    // First level: the same five fields once more in a single 32-bit word per host (each under its
    // own guard bit; the GPU component and the rank exact, the three other capacities with as many
    // of their high bits as are left). One 32-bit subtraction and one logic operation per pair
    // answer "cannot enter the best three" for most pairs; only chunks in which some pair
    // passes go on to the two-word test above.
    int l1_enabled;
    int l1_shift[5], l1_drop[5];
    unsigned int l1_guards, l1_rank_mask;
};

}  // namespace nbos

struct nbos_snapshot {
    int N, H, Hpad, R, key_order, flags;
    nbos::KeyLayout key;
    void *workspace;
    size_t workspace_bytes;
    bool owns_workspace;
    unsigned int *d_status;         // raised by kernels that gave up on a bounded wait
    unsigned int *d_update_status;  // raised by nbos_snapshot_update's scan of the new state
    // tables in visiting order (hosts sorted by ascending A when the table is small enough)
    const int4 *d_feas;   // [N][Hpad] (gmax, vram_gb, millicpus, mem_mb)
    const void *d_ab;     // [N][Hpad] uint2 (32-bit keys) or ulonglong2 (64-bit keys): (A, B)
    const uint4 *d_pk;    // [N][Hpad] (word0, word1, A, B), only when pack.enabled
    nbos::PackLayout pack;
    const uint2 *d_rk;    // [N][Hpad] (word0, word1) of the ranked form, only when rank.enabled
    const unsigned int *d_rk1;  // [N][Hpad] first-level word of the ranked form, only when rank.l1_enabled
    // [N][kGroupSlices + 1] table positions at which the GPU-count groups of a grouped snapshot
    // start (entry k = start of group k; the entries after the last group = where the hosts that
    // can take something end), only when key.grouped
    const int *d_group_bounds;
    nbos::RankLayout rank;
    int presorted;
    int idle_max;             // the key's idle field stores idle_max - (G - C)
    // the same records in host-index order (what the derivation staged), for sequential placement
    const int4 *d_host_feas;
    const void *d_host_ab;
    const int4 *d_host_seq;   // (min(G, idle GPUs), cap - S, S, 0)
    int device, sm_count;
    cudaStream_t owner_stream;  // stream the owned workspace was allocated on (create_host)
};

namespace nbos {

// a0: scan + emit kernels (nbos_derive.cu). `d_*` are device arrays [N*H].
int derive_snapshot(nbos_snapshot *s, const nbos_snapshot_desc *host_desc, const int32_t *d_G,
                    const int32_t *d_S, const int32_t *d_C, const int32_t *d_AV,
                    const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream);

// Cluster sums + auto-scaler sign per snapshot into d_out [N][4] (nbos_derive.cu).
int launch_cluster_sums(const int32_t *d_G, const int32_t *d_S, const int32_t *d_C, int N, int H,
                        long long f_num, long long f_den, long long *d_out, cudaStream_t stream);

int update_snapshot(nbos_snapshot *s, const nbos_snapshot_desc *host_desc, const int32_t *d_G,
                    const int32_t *d_S, const int32_t *d_C, const int32_t *d_AV,
                    const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream);

// a1-a9: the placement launch (nbos_place.cu). The pointers are those of the whole batch; the
// launch handles the flattened requests [range_first, range_first + range_count) of the N * batch
// (range_count < 0: all that follow range_first).
int launch_place(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                 int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                 const nbos_launch_config *cfg, long long range_first = 0, long long range_count = -1);

// Host-split placement whose candidate buffer is a fixed array inside the module (no allocation).
int launch_place_static(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                        int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                        int host_split);

// The library's own stream-ordered memory pool of a device (nbos_api.cu). Its release threshold
// is unlimited: temporaries come back from it at once, whereas the device's default pool hands
// its memory back to the driver at every synchronisation and has to map it again on the next
// call (measured: a 0.16 ms call then takes 0.3 to 7 ms now and then).
int library_pool(int device, cudaMemPool_t *out);

// Sequential placement with commits (nbos_sequential.cu).
int launch_place_sequential(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                            int32_t *d_out_hosts, int32_t *d_out_found, int32_t *d_out_subscribed,
                            cudaStream_t stream);

}  // namespace nbos
#endif
