/*
 * nbos -- batched replica placement for an oversubscribing notebook scheduler,
 * for NVIDIA B200 (sm_100a).  C ABI.
 *
 * The operation is the placement decision of NotebookOS (arXiv 2503.20591):
 *   Section 3.2.1  For a kernel's resource request (GPUs, VRAM GB, millicpus, memory MB) the
 *                  scheduler walks over all servers, keeps those with enough capacity, and
 *                  needs three of them, one per replica; with more than three a policy ranks
 *                  them; with fewer the caller has to scale out.
 *   Section 3.4.1  Default policy: more idle GPUs first, then the subscription ratio
 *                  SR = S / (G * R) (S subscribed GPUs, G server GPUs, R replicas per kernel);
 *                  a server whose SR would exceed the limit after placement is rejected.
 *   Section 3.2.3  A migration target must have the GPUs idle now (NBOS_REQUIRE_IDLE_GPUS).
 *
 * This library evaluates that rule for a whole batch of requests against a frozen snapshot of
 * the cluster (or against many independent snapshots at once): for every (request, host) pair
 * the feasibility test and an exact integer ranking key, then the three best distinct feasible
 * hosts per request.
 *
 * Exact definition of the result, per request (g, v, c, m) and snapshot n:
 *   host h is feasible  <=>  g,v,c,m >= 0  and  G[h] >= 1  and  g <= G[h]  and  v <= vram_gb[h]
 *                            and c <= millicpus[h] and m <= mem_mb[h]
 *                            and (S[h] + g) * limit_den[n] <= limit_num[n] * G[h] * R
 *                            and (flags & NBOS_REQUIRE_IDLE_GPUS ? g <= G[h] - C[h] : true)
 *   feasible hosts are ordered by (G-C descending, (S+g)/(G*R) ascending, h ascending)
 *   [NBOS_KEY_IDLE_FIRST, the paper's order] or by ((S+g)/(G*R) ascending, G-C descending,
 *   h ascending) [NBOS_KEY_SR_FIRST]; ratios are compared exactly.
 *   out_hosts = the first three of that order, best first, -1 where fewer exist;
 *   out_found = how many exist, capped at 3.
 *
 * Conventions
 *   - Every function returns an int status: NBOS_OK (0) or a negative NBOS_ERR_* code. Nothing
 *     throws, aborts or prints. nbos_strerror() names a code; nbos_last_error_detail() gives the
 *     calling thread's most recent failure in words.
 *   - "DEVICE" pointers are device memory of the current CUDA device; "HOST" pointers are
 *     ordinary host memory. The caller owns every buffer it passes. The library owns only the
 *     snapshot handle (host memory) and, for the *_host entry points and the host-split launch
 *     shape, stream-ordered temporary device memory that it frees itself.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Only devices of compute capability 10.x are accepted (NBOS_ERR_UNSUPPORTED_DEVICE).
 *   - There is no CPU fallback anywhere.
 */
#ifndef NBOS_H_
#define NBOS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NBOS_OK 0
#define NBOS_ERR_INVALID_ARG (-1)        /* NULL / misaligned pointer, size out of range        */
#define NBOS_ERR_RANGE (-2)              /* a value in the arrays is outside what is supported  */
#define NBOS_ERR_CUDA (-3)               /* a CUDA runtime call failed                          */
#define NBOS_ERR_UNSUPPORTED_DEVICE (-4) /* current device is not compute capability 10.x       */
#define NBOS_ERR_DEVICE_TIMEOUT (-5)     /* a bounded wait inside a kernel ran out              */
#define NBOS_ERR_NO_MEMORY (-6)          /* host or device allocation failed / workspace small  */
#define NBOS_ERR_STALE_LAYOUT (-7)       /* nbos_snapshot_update: new state does not fit the key /
                                          * packing layout chosen at creation; create a new one  */

/* key_order */
#define NBOS_KEY_IDLE_FIRST 0 /* Section 3.4.1: idle GPUs, then SR, then host id (default) */
#define NBOS_KEY_SR_FIRST 1   /* SR, then idle GPUs, then host id                           */

/* flags */
#define NBOS_REQUIRE_IDLE_GPUS 1 /* Section 3.2.3: also require g <= G - C                   */
#define NBOS_FORCE_KEY64 2       /* build the 64-bit key table even if 32 bits would do      */
#define NBOS_LIMIT_CLUSTER_SR 4  /* Section 3.4.1, third factor: ignore limit_num / limit_den (they may
                                  * be NULL) and use each snapshot's own cluster-wide SR,
                                  * sum(S) / (sum(G) * R), as its limit. An empty cluster (sum S = 0)
                                  * then admits only g = 0; the paper gives no floor.          */

#define NBOS_ROOM_FOR_COMMITS 8   /* size the key's ratio field for subscribed counts growing up to each
                                  * host's cap; required by nbos_place_batch_sequential          */

#define NBOS_MAX_HOSTS (1 << 20)   /* per snapshot                          */
#define NBOS_MAX_GPUS_PER_HOST 1023
#define NBOS_MAX_REPLICAS 1024
#define NBOS_REPLICAS_PLACED 3     /* hosts returned per request (Section 3.2.1) */

typedef struct nbos_snapshot nbos_snapshot; /* opaque */

/*
 * Cluster state, structure of arrays. N snapshots of H hosts each; array element [n*H + h].
 *   gpus_total       G  (0 .. NBOS_MAX_GPUS_PER_HOST; a host with G = 0 is never feasible)
 *   gpus_subscribed  S  (>= 0)  sum of GPUs requested by all replicas scheduled on the host
 *   gpus_committed   C  (0 .. G) GPUs bound to replicas that are executing now
 *   vram_gb, millicpus, mem_mb  (>= 0) the capacity a request's ask is compared with. Pass total
 *                    capacity for the creation reading of Section 3.2.1, or what is left
 *                    unbound for the migration reading of Section 3.2.3.
 *   limit_num/limit_den  per-snapshot SR limit as a rational in the paper's units S/(G*R);
 *                    limit_num >= 0, limit_den >= 1.
 */
typedef struct nbos_snapshot_desc {
    int32_t n_snapshots; /* N >= 1                                   */
    int32_t n_hosts;     /* 1 <= H <= NBOS_MAX_HOSTS                  */
    int32_t replicas_R;  /* 1 .. NBOS_MAX_REPLICAS; the paper uses 3  */
    int32_t key_order;   /* NBOS_KEY_*                                */
    int32_t flags;       /* NBOS_REQUIRE_IDLE_GPUS | NBOS_FORCE_KEY64 | NBOS_LIMIT_CLUSTER_SR |
                          * NBOS_ROOM_FOR_COMMITS */
    int32_t reserved;    /* must be 0                                 */
    const int32_t *limit_num; /* HOST [N] in both create variants     */
    const int32_t *limit_den; /* HOST [N]                             */
    /* [N*H] each. DEVICE for nbos_snapshot_create (read by work queued on the stream: keep them
     * valid until that work has finished), HOST for nbos_snapshot_create_host (read before it
     * returns). */
    const int32_t *gpus_total, *gpus_subscribed, *gpus_committed;
    const int32_t *vram_gb, *millicpus, *mem_mb;
} nbos_snapshot_desc;

typedef struct nbos_snapshot_info {
    int32_t n_snapshots, n_hosts, hosts_padded;
    int32_t key_bits;                    /* 32 or 64: width of the ranking key in use       */
    int32_t bits_idle, bits_sr, bits_id; /* field widths inside the key                     */
    int32_t key_order, flags, replicas_R;
    int32_t packed_test; /* 0: capacities too wide for the packed test; 1: packed, one guard
                          * mask; 2: packed, one guard mask per word                        */
    int32_t static_key;  /* 1: every host has the same key slope, hosts rank the same for all g */
    int32_t presorted;   /* 1: the host table is stored in ascending key order              */
    int32_t grouped;     /* 1: hosts differ in GPU count; the table is stored count by count,
                          * each group in ascending key order                               */
    int64_t workspace_bytes;
    int32_t ranked;      /* 1: the ranked form is available (static_key and presorted): capacities and
                          * the host's rank in the order of Section 3.4.1 packed into one 64-bit
                          * value per host, compared with one subtraction per pair               */
    int32_t ranked_dropped_bits[4]; /* low bits of (GPUs, VRAM, millicpus, memory) the ranked form
                          * leaves out of its per-pair test; pairs that pass are re-tested exactly */
    int32_t reserved;
} nbos_snapshot_info;

/*
 * Launch shape for nbos_place_batch_ex. 0 in a field = choose automatically.
 *   lanes_per_request  1,2,4,8,16,32: lanes of one warp that share a request; each strides the
 *                      hosts and keeps its own best three, merged by xor-shuffles at the end.
 *   requests_per_lane  1,2,4,8: upper bound on requests one lane carries through the host loop.
 *   host_split         K >= 1: hosts are cut into K slices handled by different thread blocks;
 *                      K > 1 writes per-slice candidates to temporary device memory and runs a
 *                      merge kernel.
 *   tile_hosts         hosts per shared-memory tile (multiple of 32).
 *   grid_blocks        thread blocks along the request dimension (per host slice).
 *   pair_mode          how a (request, host) pair is evaluated when the snapshot has 32-bit keys:
 *                      0 = the fastest form the snapshot allows; 1 = four separate capacity
 *                      compares; 2 = packed capacity test with the key computed per pair (even if
 *                      the snapshot would allow ranking by the host part of the key alone);
 *                      3 = packed capacity test with the host part of the key compared per pair
 *                      (even if the table is stored in key order, where 0 drops that compare:
 *                      a feasible host then enters a request's best three exactly while the
 *                      request has fewer than three). Every form gives the same outputs.
 *   first_fit          1 = stop scanning a request's hosts at the third feasible one. Possible
 *                      when every host has the same key slope and the table is stored in key
 *                      order (nbos_snapshot_info: static_key and presorted), because then the
 *                      first three feasible hosts in table order are the best three; otherwise
 *                      the flag is ignored. Same outputs, far fewer (request, host) pairs looked
 *                      at: throughput of this variant is not a pairs/s figure.
 */
typedef struct nbos_launch_config {
    int32_t lanes_per_request;
    int32_t requests_per_lane;
    int32_t host_split;
    int32_t tile_hosts;
    int32_t grid_blocks;
    int32_t pair_mode;
    int32_t first_fit;
    int32_t reserved; /* must be 0 */
} nbos_launch_config;

/* Device bytes nbos_snapshot_create needs in `workspace` for this N and H (Section 3.4.1 state
 * turned into per-host records). Only n_snapshots, n_hosts and flags of `desc` are read. */
int nbos_snapshot_workspace_bytes(const nbos_snapshot_desc *desc, size_t *out_bytes);

/*
 * Build a snapshot from DEVICE arrays: validates, then derives one record per host -- the
 * largest GPU ask that passes the capacity test, the SR limit test of Section 3.4.1 and (if
 * asked) the idle test of Section 3.2.3, the three other capacities, and the two integers
 * (A, B) with  key(g) = A + g * B  that order hosts exactly as Section 3.4.1 does.
 *   workspace        DEVICE, 256-byte aligned, >= nbos_snapshot_workspace_bytes; caller-owned;
 *                    must stay valid and untouched until nbos_snapshot_destroy.
 *   arrays           DEVICE, 16-byte aligned.
 * Synchronises `cuda_stream` once (value-range validation needs a small read-back).
 * Errors: INVALID_ARG (NULL, alignment, N/H/R out of range, bad limit), RANGE (negative value,
 * C > G, G too large, key would not fit 63 bits), NO_MEMORY, CUDA, UNSUPPORTED_DEVICE.
 * On error *out is NULL and nothing is leaked.
 */
int nbos_snapshot_create(const nbos_snapshot_desc *desc, void *workspace, size_t workspace_bytes,
                         void *cuda_stream, nbos_snapshot **out);

/* Same operation from HOST arrays (any alignment). The library takes the workspace and a staging
 * buffer from a stream-ordered memory pool of its own (one per device, kept for the life of the
 * process so that repeated calls reuse the same memory) and gives them back to that pool in
 * nbos_snapshot_destroy / when the derivation has run. The host arrays have been read when the
 * call returns. */
int nbos_snapshot_create_host(const nbos_snapshot_desc *desc, void *cuda_stream,
                              nbos_snapshot **out);

/*
 * Refresh an existing snapshot from new cluster state of the same shape (same N, H, R, key order
 * and flags as at creation; `desc` carries the new arrays and limits): the per-host records of
 * Sections 3.2.1 / 3.4.1 are derived again with the key widths, packing layout and visiting-order
 * machinery chosen at creation. Unlike creation this reads nothing back and never synchronises:
 * it only queues work on `cuda_stream`, so a scheduler tick can queue "update, place, update,
 * place ..." without waiting. The price is that problems are reported late: if the new state
 * has a value outside the supported range, or does not fit the stored layout (more idle GPUs,
 * a larger subscription or capacity than the widths allow, a GPU count per host the snapshot did
 * not have), the device status word is raised, the tables and every placement made from them are
 * undefined, and nbos_snapshot_status returns NBOS_ERR_RANGE / NBOS_ERR_STALE_LAYOUT; destroy the
 * snapshot and create a new one then. A successful update clears what an earlier update reported;
 * a device-side wait that ran out (NBOS_ERR_DEVICE_TIMEOUT) stays reported until the snapshot is
 * destroyed.
 * The caller must make sure that no placement on ANOTHER stream is still using the snapshot;
 * work queued earlier on the same stream is ordered before the update.
 *   nbos_snapshot_update       arrays are DEVICE memory (16-byte aligned), read by the queued work
 *   nbos_snapshot_update_host  arrays are HOST memory; copied into device staging the library
 *                              keeps per device (two sets, taken in turn) on its copy-in stream,
 *                              in call order with the request copies of the host-buffer placement
 *                              calls; the derivation queued on `cuda_stream` waits for the copies.
 *                              Pageable arrays have been read when the call returns; PINNED arrays
 *                              are read asynchronously: keep them unchanged until `cuda_stream`
 *                              has reached the end of the update.
 * Errors at call time: INVALID_ARG (shape / flags differ, NULL or misaligned pointers, bad limit),
 * NO_MEMORY, CUDA.
 */
int nbos_snapshot_update(nbos_snapshot *snap, const nbos_snapshot_desc *desc, void *cuda_stream);
int nbos_snapshot_update_host(nbos_snapshot *snap, const nbos_snapshot_desc *desc, void *cuda_stream);

/* Frees the handle (and what nbos_snapshot_create_host allocated: that memory goes back to the
 * library's pool in the order of the stream the snapshot was created or last updated on). The
 * caller must make sure no nbos_place_batch on this snapshot is still running. NULL is accepted. */
int nbos_snapshot_destroy(nbos_snapshot *snap);

int nbos_snapshot_get_info(const nbos_snapshot *snap, nbos_snapshot_info *out);

/*
 * The placement decision of Sections 3.2.1 / 3.4.1 for a batch (definition at the top).
 *   requests   DEVICE [N * batch_per_snapshot * 4] int32, 16-byte aligned; request i of
 *              snapshot n at ((n * batch + i) * 4): GPUs, VRAM GB, millicpus, memory MB.
 *              A request with a negative field fits nowhere (all -1); that is not an error.
 *   out_hosts  DEVICE [N * batch * 3] int32: host indices (0 .. H-1) best first, -1 padding.
 *   out_found  DEVICE [N * batch] int32 or NULL: number of hosts found (0..3).
 * Asynchronous on `cuda_stream`; outputs are valid once the stream has been synchronised. The
 * snapshot is read-only here, so calls on different streams may overlap. batch == 0 is a no-op.
 * Errors: INVALID_ARG, CUDA, NO_MEMORY. A device-side wait that ran out is reported later by
 * nbos_snapshot_status.
 */
int nbos_place_batch(const nbos_snapshot *snap, const int32_t *requests, int64_t batch_per_snapshot,
                     int32_t *out_hosts, int32_t *out_found, void *cuda_stream);

/* Same, with an explicit launch shape (NULL = automatic). Every shape gives identical output. */
int nbos_place_batch_ex(const nbos_snapshot *snap, const int32_t *requests,
                        int64_t batch_per_snapshot, int32_t *out_hosts, int32_t *out_found,
                        void *cuda_stream, const nbos_launch_config *cfg);

/*
 * Same operation with HOST buffers (pinned memory makes the copies asynchronous and faster, but
 * any host memory works). The batch is cut into up to 4 chunks whose host-to-device copy, kernel
 * and device-to-host copy overlap on three internal streams (copies in, kernels, copies out;
 * created once per device, with two sets of device staging that successive calls take in turn and
 * that grow when a larger batch comes). The copies in start as soon as staging is free; the
 * kernels wait for the work queued on `cuda_stream` before the call (a snapshot update, say), and
 * `cuda_stream` in turn waits for the kernels, so that a later update of the snapshot queued on it
 * does not overtake them. Calls on the same device take their turns in the order they are made.
 *   nbos_place_batch_host        returns after the results are in the host buffers.
 *   nbos_place_batch_host_async  returns once the work is queued. Calls in a row overlap: the
 *                                copies in of one run beside the kernels of the one before and
 *                                the copies out of the one before that. The request and result
 *                                buffers belong to the library until nbos_place_batch_host_wait
 *                                (or a later nbos_place_batch_host on the same device) has
 *                                returned. With pageable host memory the copies block the caller
 *                                and nothing overlaps (still correct).
 *   nbos_place_batch_host_wait   blocks until every host-buffer call made so far on the
 *                                snapshot's device has delivered its results. Call it before
 *                                destroying a snapshot that asynchronous calls still use.
 * Errors: INVALID_ARG, NO_MEMORY, CUDA (after an error the internal streams are synchronised
 * before the call returns).
 */
int nbos_place_batch_host(const nbos_snapshot *snap, const int32_t *requests_host,
                          int64_t batch_per_snapshot, int32_t *out_hosts_host,
                          int32_t *out_found_host, void *cuda_stream);
int nbos_place_batch_host_async(const nbos_snapshot *snap, const int32_t *requests_host,
                                int64_t batch_per_snapshot, int32_t *out_hosts_host,
                                int32_t *out_found_host, void *cuda_stream);
int nbos_place_batch_host_wait(const nbos_snapshot *snap);

/*
 * Placement for callers that are not allowed to allocate device memory. (The paper has no
 * counterpart; this is a deployment variant of nbos_place_batch with the host-split launch
 * shape.)
 *
 * Who needs it: a scheduler that shares its GPU with a training or serving job which has
 * already handed all free device memory to its own pool, so that a cudaMalloc here can fail or
 * evict; and control loops with a latency budget, where the device-wide synchronisation and
 * the driver lock an allocation may take are not acceptable. nbos_place_batch allocates a
 * temporary candidate buffer whenever it cuts the hosts into slices (small batches against many
 * hosts). This entry point computes the same result with that buffer placed in a fixed array
 * of NBOS_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU on which the
 * library is loaded holds those bytes until the process exits. It calls no cudaMalloc,
 * cudaFree or other allocating routine. Inputs and outputs are still the caller's.
 *
 *   host_split   K, number of host slices (1..NBOS_NOALLOC_MAX_SPLIT; 0 = 4). It is lowered to
 *                what the host count allows. K = 1 uses no candidate buffer at all.
 *   limit        K * N * batch_per_snapshot * 3 keys (4 bytes each, 8 when the snapshot uses
 *                64-bit keys) must fit NBOS_NOALLOC_SCRATCH_BYTES; otherwise the call returns
 *                NBOS_ERR_NO_MEMORY, says so in nbos_last_error_detail(), and launches nothing.
 *   first call   The first call on each device looks up the array's device address
 *                (cudaGetSymbolAddress, with that device current). Make that first call during
 *                start-up, before any stream capture begins.
 *   sharing      All calls in the process, on all streams, use the same array, and it keeps
 *                whatever the previous call left. Nothing in it needs clearing: each call writes
 *                every slot it later reads. But two calls that overlap on the GPU (different
 *                streams, no dependency between them) race on it and give wrong results: order
 *                them on one stream or with events.
 * Other arguments, output and asynchrony as for nbos_place_batch; the snapshot must belong to
 * the current device.
 */
#define NBOS_NOALLOC_SCRATCH_BYTES (8u << 20)
#define NBOS_NOALLOC_MAX_SPLIT 64
int nbos_place_batch_noalloc(const nbos_snapshot *snap, const int32_t *requests,
                             int64_t batch_per_snapshot, int32_t *out_hosts, int32_t *out_found,
                             void *cuda_stream, int32_t host_split);

/*
 * Executor selection for a batch of cell executions (Section 3.2.2). When a cell is submitted,
 * the scheduler looks at the servers hosting the kernel's three replicas: a replica whose server
 * lacks the resources to run the cell now is told to yield, and with the resource information at
 * hand the scheduler designates the executor itself; if all three must yield, a replica has to
 * migrate (Section 3.2.3 -- find the target with nbos_place_batch on a snapshot created with
 * NBOS_REQUIRE_IDLE_GPUS and the idle capacities; its first column is the best target).
 *
 *   can run now   <=>  g,v,c,m >= 0 and G >= 1 and g <= G - C and v <= vram_gb and c <= millicpus
 *                      and m <= mem_mb  (pass the idle capacities). The SR limit is not tested:
 *                      the replica is already subscribed on its server.
 *   designated    =    among the replicas that can run, the first by (G - C descending,
 *                      S / (G * R) ascending -- compared exactly --, host index ascending, replica
 *                      slot ascending). The paper does not say which runnable replica is picked;
 *                      this is the default placement policy's order (Section 3.4.1).
 *
 *   state          DEVICE arrays [n_hosts] int32 of one cluster snapshot (not validated; a host
 *                  index outside 0..n_hosts-1 in replica_hosts, e.g. -1, means "no such replica")
 *   requests       DEVICE [n_kernels * 4] int32, 16-byte aligned: GPUs, VRAM GB, millicpus, MB
 *   replica_hosts  DEVICE [n_kernels * 3] int32 (any 4-byte alignment; when it is 16-byte aligned,
 *                  batches of 2^19 kernels and more are streamed through bulk asynchronous copies)
 *   out_executor   DEVICE [n_kernels] int32: host index of the designated executor, -1 = all yield
 *   out_can_run    DEVICE [n_kernels] int32: bit k set = the replica in slot k can run now
 * Asynchronous on `cuda_stream`; a per-call temporary of 36 bytes per host comes from the
 * library's stream-ordered pool. Errors: INVALID_ARG, NO_MEMORY, CUDA, UNSUPPORTED_DEVICE.
 */
typedef struct nbos_cluster_state {
    int32_t n_hosts;
    int32_t replicas_R;
    const int32_t *gpus_total, *gpus_subscribed, *gpus_committed;
    const int32_t *vram_gb, *millicpus, *mem_mb;
} nbos_cluster_state;

int nbos_select_executors(const nbos_cluster_state *state, const int32_t *requests,
                          const int32_t *replica_hosts, int64_t n_kernels, int32_t *out_executor,
                          int32_t *out_can_run, void *cuda_stream);

/*
 * Sequential placement with commits: the paper's scheduler places one kernel at a time, and a
 * placed kernel's replicas subscribe its GPUs on their three servers before the next kernel is
 * looked at (Sections 3.2.1, 3.4.1). For request i = 0, 1, ... of each snapshot, in order: the
 * same decision as nbos_place_batch against the current state; if three hosts were found, S of
 * each grows by the request's GPU count (its key and its remaining room under the SR limit move
 * accordingly); if fewer were found nothing changes (the kernel is not created). Committed GPUs
 * and the other capacities stay as they are. Snapshots are independent and run in parallel; the
 * snapshot object itself is not modified.
 *   snap            must have been created with NBOS_ROOM_FOR_COMMITS; at most
 *                   NBOS_SEQUENTIAL_MAX_HOSTS hosts (the evolving state lives on one SM up to
 *                   8,192 hosts, on the 2 to 8 SMs of a thread-block cluster beyond that);
 *                   otherwise INVALID_ARG / RANGE
 *   requests, out_hosts, out_found   as for nbos_place_batch
 *   out_subscribed  DEVICE [N * H] int32 or NULL: S of every host after the last request
 * Asynchronous on `cuda_stream`.
 */
#define NBOS_SEQUENTIAL_MAX_HOSTS 65536
int nbos_place_batch_sequential(const nbos_snapshot *snap, const int32_t *requests,
                                int64_t batch_per_snapshot, int32_t *out_hosts, int32_t *out_found,
                                int32_t *out_subscribed, void *cuda_stream);

/*
 * Cluster sums and the auto-scaler rule (Sections 3.4.1, 3.4.2), per snapshot:
 *   out_sums[4n + 0] = sum of G   (GPUs provisioned)
 *   out_sums[4n + 1] = sum of S   (GPUs subscribed; sum S / (sum G * R) is the cluster-wide SR)
 *   out_sums[4n + 2] = sum of C   (GPUs in active use)
 *   out_sums[4n + 3] = +1 if sum G < f * sum C   (capacity below the expected f * sum C: scale out)
 *                      -1 if f * sum C < sum G   (more provisioned than expected: servers may go)
 *                       0 if equal;   f = f_num / f_den, compared exactly (the paper uses 1.05 = 21/20)
 * Arrays: DEVICE [n_snapshots * n_hosts] int32 (not validated); out_sums: DEVICE [n_snapshots * 4]
 * int64. Asynchronous on `cuda_stream`.
 */
int nbos_cluster_sums(const int32_t *gpus_total, const int32_t *gpus_subscribed,
                      const int32_t *gpus_committed, int32_t n_snapshots, int32_t n_hosts,
                      int32_t f_num, int32_t f_den, int64_t *out_sums, void *cuda_stream);

/*
 * Scale-out deficit of a placed batch (Sections 3.2.1, 3.4.2: when fewer than three candidate
 * servers exist, as many additional servers as are missing get provisioned), per snapshot:
 *   out_deficit[2n + 0] = sum over the batch of (3 - found)
 *   out_deficit[2n + 1] = number of requests with found < 3
 * found: DEVICE [n_snapshots * batch_per_snapshot] int32 as written by nbos_place_batch;
 * out_deficit: DEVICE [n_snapshots * 2] int64. Asynchronous on `cuda_stream`.
 */
int nbos_scale_out_deficit(const int32_t *found, int32_t n_snapshots, int64_t batch_per_snapshot,
                           int64_t *out_deficit, void *cuda_stream);

/* Synchronises `cuda_stream` and returns the sticky device status of this snapshot: NBOS_OK, or
 * NBOS_ERR_DEVICE_TIMEOUT if some kernel gave up on a bounded wait (its outputs are then
 * undefined), NBOS_ERR_RANGE / NBOS_ERR_STALE_LAYOUT after an nbos_snapshot_update whose new state
 * was invalid / did not fit the snapshot's layout. */
int nbos_snapshot_status(const nbos_snapshot *snap, void *cuda_stream);

const char *nbos_strerror(int status);
const char *nbos_last_error_detail(void);

#ifdef __cplusplus
}
#endif
#endif /* NBOS_H_ */
