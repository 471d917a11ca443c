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
    int g_min;                     // min over hosts with G >= 1 of G (INT_MAX if none)
    int pad;
    unsigned long long sub_max;    // max over hosts that can take something of S + gmax
    unsigned long long g_mask[16]; // bit G set if some host has G GPUs (G in 1..1023)
};
enum : unsigned int {
    ERR_NEGATIVE = 1u,        // some value < 0
    ERR_COMMITTED_GT_TOTAL = 2u,
    ERR_G_TOO_LARGE = 4u,
};

struct Layout {
    size_t off_status, off_limits, off_lambda, off_stats, off_feas, off_ab, total;
};
Layout workspace_layout(int n_snapshots, int hosts_padded);
inline int pad_hosts(int h) { return (h + 31) & ~31; }

struct KeyLayout {
    int key_bits;  // 32 or 64
    int bits_idle, bits_sr, bits_id;
};

}  // namespace nbos

struct nbos_snapshot {
    int N, H, Hpad, R, key_order, flags;
    nbos::KeyLayout key;
    void *workspace;
    size_t workspace_bytes;
    bool owns_workspace;
    unsigned int *d_status;
    const int4 *d_feas;   // [N][Hpad] (gmax, vram_gb, millicpus, mem_mb)
    const void *d_ab;     // [N][Hpad] uint2 (32-bit keys) or ulonglong2 (64-bit keys): (A, B)
    int device, sm_count;
};

namespace nbos {

// a0: scan + emit kernels (nbos_derive.cu). `d_*` are device arrays [N*H].
int derive_snapshot(nbos_snapshot *s, const nbos_snapshot_desc *host_desc, const int32_t *d_G,
                    const int32_t *d_S, const int32_t *d_C, const int32_t *d_AV,
                    const int32_t *d_AC, const int32_t *d_AM, cudaStream_t stream);

// a1-a9: the placement launch (nbos_place.cu).
int launch_place(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                 int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                 const nbos_launch_config *cfg);

// Host-split placement whose candidate buffer is a fixed array inside the module (no allocation).
int launch_place_static(const nbos_snapshot *s, const int32_t *d_requests, int64_t batch,
                        int32_t *d_out_hosts, int32_t *d_out_found, cudaStream_t stream,
                        int host_split);

}  // namespace nbos
#endif
