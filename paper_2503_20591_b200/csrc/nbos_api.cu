// Host side of the C ABI declared in include/nbos.h: argument checks, handle life cycle,
// staging for the host-buffer entry points. All arithmetic of the method runs in the kernels of
// nbos_derive.cu and nbos_place.cu.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>

#include "nbos_internal.h"

namespace nbos {

static thread_local char g_detail[512] = "";

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_detail, sizeof(g_detail), fmt, ap);
    va_end(ap);
    return code;
}

int cuda_fail(cudaError_t e, const char *what)
{
    cudaGetLastError();  // clear the non-sticky error state
    return fail(NBOS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

namespace {

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_desc_scalars(const nbos_snapshot_desc *d)
{
    if (!d) return fail(NBOS_ERR_INVALID_ARG, "desc is NULL");
    if (d->n_snapshots < 1 || d->n_snapshots > 65535)
        return fail(NBOS_ERR_INVALID_ARG, "n_snapshots must be in 1..65535 (got %d)", d->n_snapshots);
    if (d->n_hosts < 1 || d->n_hosts > NBOS_MAX_HOSTS)
        return fail(NBOS_ERR_INVALID_ARG, "n_hosts must be in 1..%d (got %d)", NBOS_MAX_HOSTS, d->n_hosts);
    if (d->flags & ~(NBOS_REQUIRE_IDLE_GPUS | NBOS_FORCE_KEY64 | NBOS_LIMIT_CLUSTER_SR | NBOS_ROOM_FOR_COMMITS))
        return fail(NBOS_ERR_INVALID_ARG, "unknown bits in flags (0x%x)", d->flags);
    return NBOS_OK;
}

int check_desc_full(const nbos_snapshot_desc *d)
{
    int rc = check_desc_scalars(d);
    if (rc) return rc;
    if (d->replicas_R < 1 || d->replicas_R > NBOS_MAX_REPLICAS)
        return fail(NBOS_ERR_INVALID_ARG, "replicas_R must be in 1..%d (got %d)", NBOS_MAX_REPLICAS, d->replicas_R);
    if (d->key_order != NBOS_KEY_IDLE_FIRST && d->key_order != NBOS_KEY_SR_FIRST)
        return fail(NBOS_ERR_INVALID_ARG, "unknown key_order %d", d->key_order);
    if (d->reserved != 0) return fail(NBOS_ERR_INVALID_ARG, "reserved must be 0");
    const bool own_limit = (d->flags & NBOS_LIMIT_CLUSTER_SR) != 0;
    if (!own_limit && (!d->limit_num || !d->limit_den)) return fail(NBOS_ERR_INVALID_ARG, "limit_num / limit_den is NULL");
    const void *arrays[6] = {d->gpus_total, d->gpus_subscribed, d->gpus_committed,
                             d->vram_gb, d->millicpus, d->mem_mb};
    for (int i = 0; i < 6; ++i)
        if (!arrays[i]) return fail(NBOS_ERR_INVALID_ARG, "host-state array %d is NULL", i);
    for (int n = 0; n < d->n_snapshots && !own_limit; ++n) {
        if (d->limit_den[n] < 1) return fail(NBOS_ERR_INVALID_ARG, "limit_den[%d] must be >= 1", n);
        if (d->limit_num[n] < 0) return fail(NBOS_ERR_INVALID_ARG, "limit_num[%d] must be >= 0", n);
    }
    return NBOS_OK;
}

int check_device(int *device, int *sm_count)
{
    NBOS_CUDA_TRY(cudaGetDevice(device));
    int major = 0;
    NBOS_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, *device));
    if (major != 10)
        return fail(NBOS_ERR_UNSUPPORTED_DEVICE, "device %d has compute capability %d.x; this library is built for 10.x only",
                    *device, major);
    NBOS_CUDA_TRY(cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, *device));
    return NBOS_OK;
}

// Streams, events and device staging used by the host-buffer entry points, per device, created on
// first use: one stream for the copies in, one for the kernels, one for the copies out (each kind
// of work is serial on the hardware anyway), and two sets of staging buffers taken in turn by
// successive calls, so that the copies in of one call run beside the kernels of the call before
// it and the copies out of the one before that.
struct HostPipe {
    static constexpr int kSets = 2, kMaxChunks = 4;
    std::mutex mutex;
    bool ready = false;
    cudaStream_t s_in = nullptr, s_kernel = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr;
    cudaEvent_t h2d_done[kSets][kMaxChunks] = {}, kernel_done[kSets][kMaxChunks] = {};
    cudaEvent_t kernels_done[kSets] = {};   // the last kernel that reads / writes the set's staging
    cudaEvent_t out_done[kSets] = {};       // the last copy out of the set's staging
    bool set_used[kSets] = {};
    unsigned int turn = 0;
    // The library's own stream-ordered pool for temporaries. Its release threshold is
    // unlimited, so the buffers of one call are reused by the next instead of going back to the
    // driver at every synchronisation (which costs more than the placement itself).
    cudaMemPool_t pool = nullptr;
    // Device staging (requests in, results out) of each set, kept between calls and grown when a
    // larger batch comes.
    char *stage[kSets] = {};
    size_t stage_bytes[kSets] = {};
    // Device staging of the cluster-state arrays of nbos_snapshot_update_host, also two sets:
    // they are copied on the copy-in stream, in call order with the request copies (a copy
    // queued on another stream would wait behind whatever bulk copies are already running).
    char *state_stage[kSets] = {};
    size_t state_bytes[kSets] = {};
    cudaEvent_t state_in[kSets] = {}, state_consumed[kSets] = {};
    bool state_used[kSets] = {};
    unsigned int state_turn = 0;
};
HostPipe g_pipes[64];
std::mutex g_pipes_mutex;

int host_pipe(int device, HostPipe **out)
{
    if (device < 0 || device >= 64) return fail(NBOS_ERR_INVALID_ARG, "device index %d not supported", device);
    std::lock_guard<std::mutex> lock(g_pipes_mutex);
    HostPipe &p = g_pipes[device];
    if (!p.ready) {
        NBOS_CUDA_TRY(cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking));
        NBOS_CUDA_TRY(cudaStreamCreateWithFlags(&p.s_kernel, cudaStreamNonBlocking));
        NBOS_CUDA_TRY(cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking));
        for (int k = 0; k < HostPipe::kSets; ++k) {
            for (int c = 0; c < HostPipe::kMaxChunks; ++c) {
                NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.h2d_done[k][c], cudaEventDisableTiming));
                NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.kernel_done[k][c], cudaEventDisableTiming));
            }
            NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.kernels_done[k], cudaEventDisableTiming));
            NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.out_done[k], cudaEventDisableTiming));
            NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.state_in[k], cudaEventDisableTiming));
            NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.state_consumed[k], cudaEventDisableTiming));
        }
        NBOS_CUDA_TRY(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = device;
        NBOS_CUDA_TRY(cudaMemPoolCreate(&p.pool, &props));
        unsigned long long keep = ~0ull;
        NBOS_CUDA_TRY(cudaMemPoolSetAttribute(p.pool, cudaMemPoolAttrReleaseThreshold, &keep));
        p.ready = true;
    }
    *out = &p;
    return NBOS_OK;
}

}  // namespace

int library_pool(int device, cudaMemPool_t *out)
{
    HostPipe *pipe = nullptr;
    int rc = host_pipe(device, &pipe);
    if (rc) return rc;
    *out = pipe->pool;
    return NBOS_OK;
}

namespace {

nbos_snapshot *new_handle(const nbos_snapshot_desc *d)
{
    nbos_snapshot *s = new (std::nothrow) nbos_snapshot();
    if (!s) return nullptr;
    s->N = d->n_snapshots;
    s->H = d->n_hosts;
    s->Hpad = pad_hosts(d->n_hosts);
    s->R = d->replicas_R;
    s->key_order = d->key_order;
    s->flags = d->flags;
    s->owns_workspace = false;
    s->owner_stream = nullptr;
    return s;
}

}  // namespace
}  // namespace nbos

using namespace nbos;

extern "C" {

int nbos_snapshot_workspace_bytes(const nbos_snapshot_desc *desc, size_t *out_bytes)
{
    if (!out_bytes) return fail(NBOS_ERR_INVALID_ARG, "out_bytes is NULL");
    int rc = check_desc_scalars(desc);
    if (rc) return rc;
    *out_bytes = workspace_layout(desc->n_snapshots, pad_hosts(desc->n_hosts)).total;
    return NBOS_OK;
}

int nbos_snapshot_create(const nbos_snapshot_desc *desc, void *workspace, size_t workspace_bytes,
                         void *cuda_stream, nbos_snapshot **out)
{
    if (!out) return fail(NBOS_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    int rc = check_desc_full(desc);
    if (rc) return rc;
    const void *arrays[6] = {desc->gpus_total, desc->gpus_subscribed, desc->gpus_committed,
                             desc->vram_gb, desc->millicpus, desc->mem_mb};
    for (int i = 0; i < 6; ++i)
        if (!aligned(arrays[i], 16)) return fail(NBOS_ERR_INVALID_ARG, "host-state array %d is not 16-byte aligned", i);
    if (!workspace || !aligned(workspace, 256)) return fail(NBOS_ERR_INVALID_ARG, "workspace is NULL or not 256-byte aligned");
    const size_t need = workspace_layout(desc->n_snapshots, pad_hosts(desc->n_hosts)).total;
    if (workspace_bytes < need)
        return fail(NBOS_ERR_NO_MEMORY, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    int device = 0, sms = 0;
    rc = check_device(&device, &sms);
    if (rc) return rc;
    nbos_snapshot *s = new_handle(desc);
    if (!s) return fail(NBOS_ERR_NO_MEMORY, "host allocation failed");
    s->workspace = workspace;
    s->workspace_bytes = need;
    s->device = device;
    s->sm_count = sms;
    rc = derive_snapshot(s, desc, desc->gpus_total, desc->gpus_subscribed, desc->gpus_committed,
                         desc->vram_gb, desc->millicpus, desc->mem_mb,
                         static_cast<cudaStream_t>(cuda_stream));
    if (rc) {
        delete s;
        return rc;
    }
    *out = s;
    return NBOS_OK;
}

int nbos_snapshot_create_host(const nbos_snapshot_desc *desc, void *cuda_stream, nbos_snapshot **out)
{
    if (!out) return fail(NBOS_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    int rc = check_desc_full(desc);
    if (rc) return rc;
    int device = 0, sms = 0;
    rc = check_device(&device, &sms);
    if (rc) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t cells = (size_t)desc->n_snapshots * desc->n_hosts;
    const size_t arr_bytes = (cells * sizeof(int32_t) + 255) & ~(size_t)255;
    const size_t need = workspace_layout(desc->n_snapshots, pad_hosts(desc->n_hosts)).total;
    HostPipe *pipe = nullptr;
    rc = host_pipe(device, &pipe);
    if (rc) return rc;
    void *ws = nullptr, *staging = nullptr;
    cudaError_t e = cudaMallocFromPoolAsync(&ws, need, pipe->pool, stream);
    if (e == cudaSuccess) e = cudaMallocFromPoolAsync(&staging, 6 * arr_bytes, pipe->pool, stream);
    if (e != cudaSuccess) {
        if (ws) cudaFreeAsync(ws, stream);
        cudaGetLastError();
        return fail(NBOS_ERR_NO_MEMORY, "device allocation failed: %s", cudaGetErrorString(e));
    }
    nbos_snapshot *s = new_handle(desc);
    if (!s) {
        cudaFreeAsync(ws, stream);
        cudaFreeAsync(staging, stream);
        return fail(NBOS_ERR_NO_MEMORY, "host allocation failed");
    }
    s->workspace = ws;
    s->workspace_bytes = need;
    s->owns_workspace = true;
    s->owner_stream = stream;
    s->device = device;
    s->sm_count = sms;
    const int32_t *src[6] = {desc->gpus_total, desc->gpus_subscribed, desc->gpus_committed,
                             desc->vram_gb, desc->millicpus, desc->mem_mb};
    const int32_t *dev[6];
    for (int i = 0; i < 6 && e == cudaSuccess; ++i) {
        dev[i] = reinterpret_cast<const int32_t *>(static_cast<char *>(staging) + i * arr_bytes);
        e = cudaMemcpyAsync(const_cast<int32_t *>(dev[i]), src[i], cells * sizeof(int32_t),
                            cudaMemcpyHostToDevice, stream);
    }
    rc = e == cudaSuccess ? derive_snapshot(s, desc, dev[0], dev[1], dev[2], dev[3], dev[4], dev[5], stream)
                          : cuda_fail(e, "copying host-state arrays to the device");
    cudaFreeAsync(staging, stream);  // stream-ordered: after the kernels that read it
    if (rc) {
        cudaFreeAsync(ws, stream);
        delete s;
        return rc;
    }
    *out = s;
    return NBOS_OK;
}

// A snapshot's tables live on the device it was created on; kernels launched from another
// current device would be handed pointers that mean nothing there.
static int check_current_device(const nbos_snapshot *snap)
{
    int device = -1;
    NBOS_CUDA_TRY(cudaGetDevice(&device));
    if (device != snap->device)
        return fail(NBOS_ERR_INVALID_ARG, "the snapshot belongs to device %d, the current device is %d", snap->device, device);
    return NBOS_OK;
}

static int check_update_desc(const nbos_snapshot *snap, const nbos_snapshot_desc *desc)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    int rc = check_desc_full(desc);
    if (rc) return rc;
    if (desc->n_snapshots != snap->N || desc->n_hosts != snap->H || desc->replicas_R != snap->R ||
        desc->key_order != snap->key_order || desc->flags != snap->flags)
        return fail(NBOS_ERR_INVALID_ARG, "update: shape, R, key order and flags must be those the snapshot was created with");
    int device = -1;
    NBOS_CUDA_TRY(cudaGetDevice(&device));
    if (device != snap->device) return fail(NBOS_ERR_INVALID_ARG, "update: the snapshot belongs to device %d", snap->device);
    return NBOS_OK;
}

int nbos_snapshot_update(nbos_snapshot *snap, const nbos_snapshot_desc *desc, void *cuda_stream)
{
    int rc = check_update_desc(snap, desc);
    if (rc) return rc;
    const void *arrays[6] = {desc->gpus_total, desc->gpus_subscribed, desc->gpus_committed,
                             desc->vram_gb, desc->millicpus, desc->mem_mb};
    for (int i = 0; i < 6; ++i)
        if (!aligned(arrays[i], 16)) return fail(NBOS_ERR_INVALID_ARG, "host-state array %d is not 16-byte aligned", i);
    snap->owner_stream = static_cast<cudaStream_t>(cuda_stream);
    return update_snapshot(snap, desc, desc->gpus_total, desc->gpus_subscribed, desc->gpus_committed,
                           desc->vram_gb, desc->millicpus, desc->mem_mb, static_cast<cudaStream_t>(cuda_stream));
}

int nbos_snapshot_update_host(nbos_snapshot *snap, const nbos_snapshot_desc *desc, void *cuda_stream)
{
    int rc = check_update_desc(snap, desc);
    if (rc) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    HostPipe *pipe = nullptr;
    rc = host_pipe(snap->device, &pipe);
    if (rc) return rc;
    const size_t cells = (size_t)snap->N * snap->H;
    const size_t arr_bytes = (cells * sizeof(int32_t) + 255) & ~(size_t)255;
    std::lock_guard<std::mutex> lock(pipe->mutex);
    const int k = (int)(pipe->state_turn++ % HostPipe::kSets);
    if (pipe->state_bytes[k] < 6 * arr_bytes) {
        // the update that used this set last may still be reading it
        if (pipe->state_used[k]) NBOS_CUDA_TRY(cudaEventSynchronize(pipe->state_consumed[k]));
        if (pipe->state_stage[k]) cudaFree(pipe->state_stage[k]);
        pipe->state_stage[k] = nullptr;
        pipe->state_bytes[k] = 0;
        cudaError_t ea = cudaMalloc(reinterpret_cast<void **>(&pipe->state_stage[k]), 6 * arr_bytes);
        if (ea != cudaSuccess) {
            cudaGetLastError();
            return fail(NBOS_ERR_NO_MEMORY, "device allocation failed: %s", cudaGetErrorString(ea));
        }
        pipe->state_bytes[k] = 6 * arr_bytes;
    }
    char *staging = pipe->state_stage[k];
    const int32_t *src[6] = {desc->gpus_total, desc->gpus_subscribed, desc->gpus_committed,
                             desc->vram_gb, desc->millicpus, desc->mem_mb};
    const int32_t *dev[6];
    cudaError_t e = pipe->state_used[k] ? cudaStreamWaitEvent(pipe->s_in, pipe->state_consumed[k], 0) : cudaSuccess;
    for (int i = 0; i < 6 && e == cudaSuccess; ++i) {
        dev[i] = reinterpret_cast<const int32_t *>(staging + i * arr_bytes);
        e = cudaMemcpyAsync(const_cast<int32_t *>(dev[i]), src[i], cells * sizeof(int32_t), cudaMemcpyHostToDevice, pipe->s_in);
    }
    if (e == cudaSuccess) e = cudaEventRecord(pipe->state_in[k], pipe->s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, pipe->state_in[k], 0);
    rc = e == cudaSuccess ? update_snapshot(snap, desc, dev[0], dev[1], dev[2], dev[3], dev[4], dev[5], stream)
                          : cuda_fail(e, "copying host-state arrays to the device");
    // also after an error: whatever was queued on `stream` comes before the set is written again
    if (cudaEventRecord(pipe->state_consumed[k], stream) == cudaSuccess) pipe->state_used[k] = true;
    snap->owner_stream = stream;
    return rc;
}

int nbos_snapshot_destroy(nbos_snapshot *snap)
{
    if (!snap) return NBOS_OK;
    int rc = NBOS_OK;
    if (snap->owns_workspace) {
        // in the order of the stream whose kernels last wrote the workspace (creation or update)
        cudaError_t e = cudaFreeAsync(snap->workspace, snap->owner_stream);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaFreeAsync");
    }
    delete snap;
    return rc;
}

int nbos_snapshot_get_info(const nbos_snapshot *s, nbos_snapshot_info *out)
{
    if (!s || !out) return fail(NBOS_ERR_INVALID_ARG, "NULL argument");
    out->n_snapshots = s->N;
    out->n_hosts = s->H;
    out->hosts_padded = s->Hpad;
    out->key_bits = s->key.key_bits;
    out->bits_idle = s->key.bits_idle;
    out->bits_sr = s->key.bits_sr;
    out->bits_id = s->key.bits_id;
    out->key_order = s->key_order;
    out->flags = s->flags;
    out->replicas_R = s->R;
    out->packed_test = !s->pack.enabled ? 0 : s->pack.guards == s->pack.guards1 ? 1 : 2;
    out->static_key = s->key.static_key;
    out->presorted = s->presorted;
    out->grouped = s->key.grouped;
    out->workspace_bytes = (int64_t)s->workspace_bytes;
    out->ranked = s->rank.enabled;
    for (int c = 0; c < 4; ++c) out->ranked_dropped_bits[c] = s->rank.enabled ? s->rank.fdrop[c] : 0;
    out->reserved = 0;
    return NBOS_OK;
}

int nbos_place_batch_ex(const nbos_snapshot *snap, const int32_t *requests,
                        int64_t batch_per_snapshot, int32_t *out_hosts, int32_t *out_found,
                        void *cuda_stream, const nbos_launch_config *cfg)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    if (batch_per_snapshot < 0 || batch_per_snapshot > ((int64_t)1 << 40) / snap->N)
        return fail(NBOS_ERR_INVALID_ARG, "batch_per_snapshot out of range");
    if (batch_per_snapshot == 0) return NBOS_OK;
    if (!requests || !out_hosts) return fail(NBOS_ERR_INVALID_ARG, "requests / out_hosts is NULL");
    if (!aligned(requests, 16)) return fail(NBOS_ERR_INVALID_ARG, "requests is not 16-byte aligned");
    if (!aligned(out_hosts, 4) || !aligned(out_found, 4)) return fail(NBOS_ERR_INVALID_ARG, "output not 4-byte aligned");
    int rc = check_current_device(snap);
    if (rc) return rc;
    return launch_place(snap, requests, batch_per_snapshot, out_hosts, out_found,
                        static_cast<cudaStream_t>(cuda_stream), cfg);
}

int nbos_place_batch(const nbos_snapshot *snap, const int32_t *requests, int64_t batch_per_snapshot,
                     int32_t *out_hosts, int32_t *out_found, void *cuda_stream)
{
    return nbos_place_batch_ex(snap, requests, batch_per_snapshot, out_hosts, out_found, cuda_stream,
                               nullptr);
}

namespace {

// chunks of an asynchronous call (measured at the largest benchmark shape, calls in a row with a
// snapshot refresh between them: 1 / 2 / 3 / 4 chunks -> 0.53 / 0.44 / 0.51 / 0.52 ms per call)
constexpr long long kAsyncChunks = 2;

int place_batch_host(const nbos_snapshot *snap, const int32_t *requests_host, int64_t batch_per_snapshot,
                     int32_t *out_hosts_host, int32_t *out_found_host, void *cuda_stream, bool synchronise)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    if (batch_per_snapshot < 0 || batch_per_snapshot > ((int64_t)1 << 40) / snap->N)
        return fail(NBOS_ERR_INVALID_ARG, "batch_per_snapshot out of range");
    if (batch_per_snapshot == 0) return NBOS_OK;
    if (!requests_host || !out_hosts_host) return fail(NBOS_ERR_INVALID_ARG, "requests / out_hosts is NULL");
    int rc_dev = check_current_device(snap);
    if (rc_dev) return rc_dev;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const long long total = (long long)snap->N * batch_per_snapshot;
    const size_t req_bytes = (size_t)total * 16, out_bytes = (size_t)total * 12,
                 found_bytes = out_found_host ? (size_t)total * 4 : 0;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };

    HostPipe *pipe = nullptr;
    int rc = host_pipe(snap->device, &pipe);
    if (rc) return rc;
    std::lock_guard<std::mutex> lock(pipe->mutex);
    const int set = (int)(pipe->turn++ % HostPipe::kSets);

    const size_t need = up(req_bytes) + up(out_bytes) + up(found_bytes);
    if (pipe->stage_bytes[set] < need) {
        // the call that used this set last may still be running: wait for it before the buffer goes
        if (pipe->set_used[set]) NBOS_CUDA_TRY(cudaEventSynchronize(pipe->out_done[set]));
        if (pipe->stage[set]) cudaFree(pipe->stage[set]);
        pipe->stage[set] = nullptr;
        pipe->stage_bytes[set] = 0;
        cudaError_t ea = cudaMalloc(reinterpret_cast<void **>(&pipe->stage[set]), need);
        if (ea != cudaSuccess) {
            cudaGetLastError();
            return fail(NBOS_ERR_NO_MEMORY, "device staging allocation of %zu bytes failed: %s", need, cudaGetErrorString(ea));
        }
        pipe->stage_bytes[set] = need;
    }
    char *buf = pipe->stage[set];
    int32_t *d_req = reinterpret_cast<int32_t *>(buf);
    int32_t *d_out = reinterpret_cast<int32_t *>(buf + up(req_bytes));
    int32_t *d_found = out_found_host ? reinterpret_cast<int32_t *>(buf + up(req_bytes) + up(out_bytes)) : nullptr;

    // Chunks of the flattened request list: copy in, place, copy out. A chunk carries at least
    // 2^30 (request, host) pairs: smaller launches lose more in kernel efficiency than the finer
    // overlap gains (measured with 2, 4, 8, 16 and 32 chunks of the largest benchmark shape);
    // at most four chunks. Every chunk launch plans itself. The copies in depend on nothing
    // queued on the caller's stream and start as soon as the set's request buffer is free (the
    // kernels of the call that used it last have finished); only the kernels wait for the caller's
    // stream, because the snapshot may still be in the making there; and the caller's stream in
    // turn waits for the kernels (not for the copies out), so that a later snapshot update does
    // not overtake them.
    const long long pairs = total * (long long)snap->Hpad;
    long long n_chunks = pairs >> 30;
    if (n_chunks < 1) n_chunks = 1;
    if (n_chunks > HostPipe::kMaxChunks) n_chunks = HostPipe::kMaxChunks;
    // calls in a row have their requests on the device before their kernels' turn comes: fewer,
    // larger launches then
    if (!synchronise && n_chunks > kAsyncChunks) n_chunks = kAsyncChunks;
    const long long chunk = (((total + n_chunks - 1) / n_chunks) + 31) & ~31ll;
    cudaError_t e = cudaEventRecord(pipe->start, stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->s_kernel, pipe->start, 0);
    if (e == cudaSuccess && pipe->set_used[set]) {
        e = cudaStreamWaitEvent(pipe->s_in, pipe->kernels_done[set], 0);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->s_kernel, pipe->out_done[set], 0);
    }
    for (long long lo = 0, c = 0; lo < total && e == cudaSuccess && rc == NBOS_OK; lo += chunk, ++c) {
        const long long n = total - lo < chunk ? total - lo : chunk;
        e = cudaMemcpyAsync(d_req + lo * 4, requests_host + lo * 4, (size_t)n * 16, cudaMemcpyHostToDevice, pipe->s_in);
        if (e == cudaSuccess) e = cudaEventRecord(pipe->h2d_done[set][c], pipe->s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->s_kernel, pipe->h2d_done[set][c], 0);
        if (e != cudaSuccess) break;
        rc = launch_place(snap, d_req, batch_per_snapshot, d_out, d_found, pipe->s_kernel, nullptr, lo, n);
        if (rc) break;
        e = cudaEventRecord(pipe->kernel_done[set][c], pipe->s_kernel);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->s_out, pipe->kernel_done[set][c], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(out_hosts_host + lo * 3, d_out + lo * 3, (size_t)n * 12, cudaMemcpyDeviceToHost, pipe->s_out);
        if (e == cudaSuccess && d_found)
            e = cudaMemcpyAsync(out_found_host + lo, d_found + lo, (size_t)n * 4, cudaMemcpyDeviceToHost, pipe->s_out);
    }
    // what was queued is accounted for also on the error paths, so that the set can be taken again
    cudaError_t e3 = cudaEventRecord(pipe->kernels_done[set], pipe->s_kernel);
    if (e3 == cudaSuccess) e3 = cudaStreamWaitEvent(stream, pipe->kernels_done[set], 0);
    if (e3 == cudaSuccess) e3 = cudaStreamWaitEvent(pipe->s_out, pipe->kernels_done[set], 0);
    if (e3 == cudaSuccess) e3 = cudaEventRecord(pipe->out_done[set], pipe->s_out);
    if (e3 == cudaSuccess) pipe->set_used[set] = true;
    const bool failed = rc != NBOS_OK || e != cudaSuccess || e3 != cudaSuccess;
    cudaError_t e2 = cudaSuccess;
    if (failed) {
        cudaStreamSynchronize(pipe->s_in);
        cudaStreamSynchronize(pipe->s_kernel);
        cudaStreamSynchronize(pipe->s_out);
    } else if (synchronise) {
        e2 = cudaEventSynchronize(pipe->out_done[set]);
    }
    if (rc) return rc;
    if (e != cudaSuccess) return cuda_fail(e, "host <-> device copy");
    if (e3 != cudaSuccess) return cuda_fail(e3, "cudaEventRecord");
    if (e2 != cudaSuccess) return cuda_fail(e2, "cudaEventSynchronize");
    return NBOS_OK;
}

}  // namespace

int nbos_place_batch_host(const nbos_snapshot *snap, const int32_t *requests_host,
                          int64_t batch_per_snapshot, int32_t *out_hosts_host,
                          int32_t *out_found_host, void *cuda_stream)
{
    return place_batch_host(snap, requests_host, batch_per_snapshot, out_hosts_host, out_found_host, cuda_stream, true);
}

int nbos_place_batch_host_async(const nbos_snapshot *snap, const int32_t *requests_host,
                                int64_t batch_per_snapshot, int32_t *out_hosts_host,
                                int32_t *out_found_host, void *cuda_stream)
{
    return place_batch_host(snap, requests_host, batch_per_snapshot, out_hosts_host, out_found_host, cuda_stream, false);
}

int nbos_place_batch_host_wait(const nbos_snapshot *snap)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    HostPipe *pipe = nullptr;
    int rc = host_pipe(snap->device, &pipe);
    if (rc) return rc;
    std::lock_guard<std::mutex> lock(pipe->mutex);
    for (int k = 0; k < HostPipe::kSets; ++k)
        if (pipe->set_used[k]) NBOS_CUDA_TRY(cudaEventSynchronize(pipe->out_done[k]));
    return NBOS_OK;
}

int nbos_place_batch_noalloc(const nbos_snapshot *snap, const int32_t *requests,
                             int64_t batch_per_snapshot, int32_t *out_hosts, int32_t *out_found,
                             void *cuda_stream, int32_t host_split)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    if (batch_per_snapshot < 0 || batch_per_snapshot > ((int64_t)1 << 40) / snap->N)
        return fail(NBOS_ERR_INVALID_ARG, "batch_per_snapshot out of range");
    if (host_split < 0 || host_split > NBOS_NOALLOC_MAX_SPLIT)
        return fail(NBOS_ERR_INVALID_ARG, "host_split must be 0 (default) or 1..%d", NBOS_NOALLOC_MAX_SPLIT);
    if (batch_per_snapshot == 0) return NBOS_OK;
    if (!requests || !out_hosts) return fail(NBOS_ERR_INVALID_ARG, "requests / out_hosts is NULL");
    if (!aligned(requests, 16)) return fail(NBOS_ERR_INVALID_ARG, "requests is not 16-byte aligned");
    if (!aligned(out_hosts, 4) || !aligned(out_found, 4)) return fail(NBOS_ERR_INVALID_ARG, "output not 4-byte aligned");
    return launch_place_static(snap, requests, batch_per_snapshot, out_hosts, out_found,
                               static_cast<cudaStream_t>(cuda_stream), host_split);
}

int nbos_place_batch_sequential(const nbos_snapshot *snap, const int32_t *requests,
                                int64_t batch_per_snapshot, int32_t *out_hosts, int32_t *out_found,
                                int32_t *out_subscribed, void *cuda_stream)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    if (!(snap->flags & NBOS_ROOM_FOR_COMMITS))
        return fail(NBOS_ERR_INVALID_ARG, "the snapshot was not created with NBOS_ROOM_FOR_COMMITS");
    if (snap->Hpad > NBOS_SEQUENTIAL_MAX_HOSTS)
        return fail(NBOS_ERR_RANGE, "sequential placement supports at most %d hosts (snapshot has %d)",
                    NBOS_SEQUENTIAL_MAX_HOSTS, snap->H);
    if (batch_per_snapshot < 0 || batch_per_snapshot > ((int64_t)1 << 40) / snap->N)
        return fail(NBOS_ERR_INVALID_ARG, "batch_per_snapshot out of range");
    if (batch_per_snapshot != 0 && (!requests || !out_hosts)) return fail(NBOS_ERR_INVALID_ARG, "requests / out_hosts is NULL");
    if (!aligned(requests, 16)) return fail(NBOS_ERR_INVALID_ARG, "requests is not 16-byte aligned");
    int rc = check_current_device(snap);
    if (rc) return rc;
    return launch_place_sequential(snap, requests, batch_per_snapshot, out_hosts, out_found, out_subscribed,
                                   static_cast<cudaStream_t>(cuda_stream));
}

int nbos_snapshot_status(const nbos_snapshot *snap, void *cuda_stream)
{
    if (!snap) return fail(NBOS_ERR_INVALID_ARG, "snapshot is NULL");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned int words[kUpdateStatusOffset / sizeof(unsigned int) + 1] = {};
    NBOS_CUDA_TRY(cudaMemcpyAsync(words, snap->d_status, sizeof(words), cudaMemcpyDeviceToHost, stream));
    NBOS_CUDA_TRY(cudaStreamSynchronize(stream));
    const unsigned int word = words[0] | words[kUpdateStatusOffset / sizeof(unsigned int)];
    if (word & STATUS_WAIT_TIMEOUT) return fail(NBOS_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (status word 0x%x)", word);
    if (word & STATUS_BAD_VALUES) return fail(NBOS_ERR_RANGE, "the last update brought a value outside the supported range (status word 0x%x)", word);
    if (word & STATUS_STALE_LAYOUT) return fail(NBOS_ERR_STALE_LAYOUT, "the last update does not fit the snapshot's layout (status word 0x%x)", word);
    if (word) return fail(NBOS_ERR_CUDA, "unknown status word 0x%x", word);
    return NBOS_OK;
}

const char *nbos_strerror(int status)
{
    switch (status) {
        case NBOS_OK: return "ok";
        case NBOS_ERR_INVALID_ARG: return "invalid argument";
        case NBOS_ERR_RANGE: return "value out of the supported range";
        case NBOS_ERR_CUDA: return "CUDA runtime error";
        case NBOS_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs compute capability 10.x)";
        case NBOS_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case NBOS_ERR_NO_MEMORY: return "out of memory or workspace too small";
        case NBOS_ERR_STALE_LAYOUT: return "updated state does not fit the snapshot's layout";
    }
    return "unknown status";
}

const char *nbos_last_error_detail(void) { return g_detail; }

}  // extern "C"
