/*
 * CPU checker for batched replica placement -- TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition of what the placement path computes.
 * It exists so that tests and the benchmark's CPU-baseline leg have something
 * independent to compare the CUDA library with. It shares no code, header,
 * table or constant with the CUDA library, and the library never calls it.
 *
 * What it computes (NotebookOS, arXiv 2503.20591):
 *
 *   Section 3.2.1  The scheduler walks over all servers; a server that has enough
 *                  capacity for the resource request (millicpus, memory MB, GPUs,
 *                  VRAM GB) is a candidate. Three candidates are needed, one per
 *                  replica. With more than three, a policy ranks them. With fewer,
 *                  the caller has to scale out, so the count found is reported.
 *   Section 3.4.1  Default policy. First: more idle GPUs is better. Second: the
 *                  subscription ratio SR = S / (G * R), S = subscribed GPUs,
 *                  G = GPUs of the server, R = replicas per kernel. A server is
 *                  rejected if adding the replica would push its SR above the
 *                  limit.
 *   Section 3.2.3  A migration target additionally needs enough idle GPUs to bind
 *                  them at once (flag NBOS_ORACLE_REQUIRE_IDLE_GPUS).
 *
 * Readings where the paper is silent (the project's design notes list them all):
 *   - "idle GPUs" of a server is G - C, C = GPUs bound to running replicas.
 *   - the SR used for ranking and for the limit is the one AFTER placement,
 *     (S + g) / (G * R); lower is better; the limit is exceeded only by a strictly greater SR.
 *   - remaining ties go to the lower host index.
 *   - a request with a negative field fits nowhere; a server with G < 1 is not a
 *     GPU server and is never a candidate.
 *   - every request of a batch sees the same frozen snapshot.
 *
 * All ratio comparisons are exact: 64-bit cross-multiplication, never floating
 * point, never a packed key. One thread, no blocking, no early exit.
 */
#include <stdint.h>
#include <stdlib.h>

#define NBOS_ORACLE_KEY_IDLE_FIRST 0 /* Section 3.4.1 order: idle GPUs, then SR   */
#define NBOS_ORACLE_KEY_SR_FIRST 1   /* the two ranking fields swapped            */
#define NBOS_ORACLE_REQUIRE_IDLE_GPUS 1

#define NBOS_ORACLE_REPLICAS_PLACED 3 /* Section 3.2.1: three candidate servers */

typedef struct {
    int32_t n_hosts;
    int32_t replicas_R;
    int32_t key_order;
    int32_t flags;
    int64_t limit_num, limit_den; /* SR limit = limit_num / limit_den, limit_den > 0 */
    const int32_t *G, *S, *C;     /* [n_hosts] total / subscribed / committed GPUs  */
    const int32_t *AV, *AC, *AM;  /* [n_hosts] VRAM GB / millicpus / memory MB capacity */
} nbos_oracle_cluster;

/* SR = S / (G * R), Section 3.4.1. Only used to pin the paper's printed example. */
double nbos_oracle_subscription_ratio(int64_t S, int64_t G, int64_t R)
{
    return (double)S / ((double)G * (double)R);
}

/* Sign of (Sa + g) / (Ga * R) - (Sb + g) / (Gb * R), exactly. Ga, Gb, R >= 1. */
int nbos_oracle_compare_sr_after(int64_t Sa, int64_t Ga, int64_t Sb, int64_t Gb, int64_t g,
                                 int64_t R)
{
    int64_t lhs = (Sa + g) * (Gb * R);
    int64_t rhs = (Sb + g) * (Ga * R);
    return (lhs > rhs) - (lhs < rhs);
}

/* Is server h a candidate for the request (g, v, c, m)? Sections 3.2.1, 3.4.1, 3.2.3. */
int nbos_oracle_feasible(const nbos_oracle_cluster *cl, int32_t h, int32_t g, int32_t v, int32_t c,
                         int32_t m)
{
    int64_t G = cl->G[h], S = cl->S[h], C = cl->C[h], R = cl->replicas_R;
    if (g < 0 || v < 0 || c < 0 || m < 0) return 0;
    if (G < 1) return 0;
    /* enough capacity in each of the four resources (Section 3.2.1) */
    if (g > G) return 0;
    if (v > cl->AV[h]) return 0;
    if (c > cl->AC[h]) return 0;
    if (m > cl->AM[h]) return 0;
    /* SR after placement must not exceed the limit (Section 3.4.1):
     *   (S + g) / (G * R) <= num / den   <=>   (S + g) * den <= num * G * R   */
    if ((S + (int64_t)g) * cl->limit_den > cl->limit_num * G * R) return 0;
    /* migration reading (Section 3.2.3): the GPUs must be idle right now */
    if ((cl->flags & NBOS_ORACLE_REQUIRE_IDLE_GPUS) && (int64_t)g > G - C) return 0;
    return 1;
}

/* Does candidate a rank strictly before candidate b for a request of g GPUs? */
int nbos_oracle_ranks_before(const nbos_oracle_cluster *cl, int32_t a, int32_t b, int32_t g)
{
    int64_t idle_a = (int64_t)cl->G[a] - cl->C[a];
    int64_t idle_b = (int64_t)cl->G[b] - cl->C[b];
    int sr = nbos_oracle_compare_sr_after(cl->S[a], cl->G[a], cl->S[b], cl->G[b], g,
                                          cl->replicas_R);
    if (cl->key_order == NBOS_ORACLE_KEY_SR_FIRST) {
        if (sr != 0) return sr < 0;             /* lower SR first            */
        if (idle_a != idle_b) return idle_a > idle_b; /* then more idle GPUs */
    } else {
        if (idle_a != idle_b) return idle_a > idle_b; /* more idle GPUs first */
        if (sr != 0) return sr < 0;             /* then lower SR             */
    }
    return a < b; /* then lower host index */
}

/*
 * Place `batch` requests against one snapshot.
 *   requests  [batch][4] = (GPUs, VRAM GB, millicpus, memory MB)
 *   out_hosts [batch][3] best first, -1 where fewer than three servers fit
 *   out_found [batch]    number of servers found, 0..3 (may be NULL)
 * Returns 0, or -1 on a bad argument / allocation failure.
 */
int nbos_oracle_place(const nbos_oracle_cluster *cl, const int32_t *requests, int64_t batch,
                      int32_t *out_hosts, int32_t *out_found)
{
    if (!cl || cl->n_hosts < 0 || cl->limit_den <= 0 || cl->limit_num < 0 || cl->replicas_R < 1 ||
        batch < 0)
        return -1;
    int32_t H = cl->n_hosts;
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)(H > 0 ? H : 1));
    char *taken = (char *)malloc((size_t)(H > 0 ? H : 1));
    if (!cand || !taken) {
        free(cand);
        free(taken);
        return -1;
    }
    for (int64_t r = 0; r < batch; ++r) {
        int32_t g = requests[4 * r + 0], v = requests[4 * r + 1];
        int32_t c = requests[4 * r + 2], m = requests[4 * r + 3];
        /* 1. collect every candidate */
        int32_t n_cand = 0;
        for (int32_t h = 0; h < H; ++h)
            if (nbos_oracle_feasible(cl, h, g, v, c, m)) cand[n_cand++] = h;
        for (int32_t i = 0; i < n_cand; ++i) taken[i] = 0;
        /* 2. three times: take the best candidate not taken yet */
        int32_t found = 0;
        for (int k = 0; k < NBOS_ORACLE_REPLICAS_PLACED; ++k) {
            int32_t best = -1;
            for (int32_t i = 0; i < n_cand; ++i) {
                if (taken[i]) continue;
                if (best < 0 || nbos_oracle_ranks_before(cl, cand[i], cand[best], g)) best = i;
            }
            if (best >= 0) {
                taken[best] = 1;
                out_hosts[3 * r + k] = cand[best];
                ++found;
            } else {
                out_hosts[3 * r + k] = -1;
            }
        }
        if (out_found) out_found[r] = found;
    }
    free(cand);
    free(taken);
    return 0;
}

/*
 * Executor selection for a cell execution (Section 3.2.2). The scheduler looks at the servers
 * that host the kernel's three replicas. A replica whose server lacks the resources to run the
 * cell now is told to yield; when the scheduler has the resource information it designates the
 * executor itself. If all three must yield, the election fails and a replica has to migrate
 * (Section 3.2.3).
 *
 * "Can run now" = the server has the idle resources to bind at once: g <= G - C idle GPUs, and
 * the three other asks within the capacities passed in (the caller passes what is idle). The SR
 * limit is not tested here: the replica is already subscribed on its server.
 * Reading where the paper is silent: among the replicas that can run, the designated executor is
 * the first in the default policy's order (Section 3.4.1): more idle GPUs, then lower current
 * SR = S / (G * R), then lower host index, then lower replica slot.
 *
 *   requests       [n_kernels][4]  (GPUs, VRAM GB, millicpus, memory MB)
 *   replica_hosts  [n_kernels][3]  host index of each replica, -1 = no such replica
 *   out_executor   [n_kernels]     host index of the designated executor, -1 = all yield
 *   out_can_run    [n_kernels]     bit k set: replica k could run now
 */
int nbos_oracle_select_executors(const nbos_oracle_cluster *cl, const int32_t *requests,
                                 const int32_t *replica_hosts, int64_t n_kernels,
                                 int32_t *out_executor, int32_t *out_can_run)
{
    if (!cl || n_kernels < 0 || cl->replicas_R < 1) return -1;
    for (int64_t k = 0; k < n_kernels; ++k) {
        int32_t g = requests[4 * k + 0], v = requests[4 * k + 1];
        int32_t c = requests[4 * k + 2], m = requests[4 * k + 3];
        int32_t best = -1, mask = 0;
        for (int slot = 0; slot < 3; ++slot) {
            int32_t h = replica_hosts[3 * k + slot];
            if (h < 0 || h >= cl->n_hosts) continue;
            int64_t G = cl->G[h], C = cl->C[h];
            if (g < 0 || v < 0 || c < 0 || m < 0) continue;
            if (G < 1) continue;
            if ((int64_t)g > G - C) continue;          /* idle GPUs, bound at once */
            if (v > cl->AV[h] || c > cl->AC[h] || m > cl->AM[h]) continue;
            mask |= 1 << slot;
            if (best < 0) {
                best = h;
                continue;
            }
            /* does h come before the current best? */
            int64_t idle_h = G - C, idle_b = (int64_t)cl->G[best] - cl->C[best];
            int before;
            if (idle_h != idle_b) {
                before = idle_h > idle_b;
            } else {
                int sr = nbos_oracle_compare_sr_after(cl->S[h], cl->G[h], cl->S[best], cl->G[best], 0,
                                                      cl->replicas_R);
                before = sr != 0 ? sr < 0 : h < best;   /* equal host: keep the earlier slot */
            }
            if (before) best = h;
        }
        out_executor[k] = best;
        out_can_run[k] = mask;
    }
    return 0;
}

/*
 * Cluster-wide quantities of Sections 3.4.1 and 3.4.2.
 *   sums[0] = sum of G (GPUs of all servers), sums[1] = sum of S (subscribed GPUs),
 *   sums[2] = sum of C (GPUs in active use).
 */
void nbos_oracle_cluster_sums(const nbos_oracle_cluster *cl, int64_t *sums)
{
    sums[0] = sums[1] = sums[2] = 0;
    for (int32_t h = 0; h < cl->n_hosts; ++h) {
        sums[0] += cl->G[h];
        sums[1] += cl->S[h];
        sums[2] += cl->C[h];
    }
}

/* Section 3.4.1, third factor: the dynamic cluster-wide SR limit is sum(S) / (sum(G) * R).
 * Returned as the rational num / den. den = 0 when the cluster has no GPUs (then no server is a
 * candidate anyway and the caller must not place against it). */
void nbos_oracle_cluster_limit(const nbos_oracle_cluster *cl, int64_t *num, int64_t *den)
{
    int64_t sums[3];
    nbos_oracle_cluster_sums(cl, sums);
    *num = sums[1];
    *den = sums[0] * cl->replicas_R;
}

/* Section 3.4.2: the expected capacity is f * sum(C), f = f_num / f_den (the paper uses 1.05).
 * +1: current capacity sum(G) is smaller than that -> scale out.
 * -1: the expected capacity is smaller than what is provisioned -> servers may be released.
 *  0: equal. Exact integer comparison. */
int nbos_oracle_autoscale(int64_t sum_G, int64_t sum_C, int64_t f_num, int64_t f_den)
{
    int64_t expected_scaled = f_num * sum_C; /* f * sum(C) * f_den */
    int64_t have_scaled = f_den * sum_G;
    return (have_scaled < expected_scaled) - (expected_scaled < have_scaled);
}

/* Sections 3.2.1 / 3.4.2: a kernel for which fewer than three servers were found needs as many
 * additional servers as it is short of. deficit = sum of (3 - found),
 * short_requests = number of requests with found < 3. */
void nbos_oracle_scale_out_deficit(const int32_t *found, int64_t batch, int64_t *deficit,
                                   int64_t *short_requests)
{
    *deficit = 0;
    *short_requests = 0;
    for (int64_t r = 0; r < batch; ++r) {
        if (found[r] < NBOS_ORACLE_REPLICAS_PLACED) {
            *deficit += NBOS_ORACLE_REPLICAS_PLACED - found[r];
            *short_requests += 1;
        }
    }
}

/*
 * Sequential placement: the paper's scheduler places one kernel at a time, and the replicas of a
 * placed kernel subscribe to its GPUs on their three servers before the next kernel is looked at
 * (Section 3.2.1: a kernel's replicas subscribe to the resources it requested; Section 3.4.1: S is
 * the sum of the GPUs requested by all replicas scheduled on the server).
 *
 * For request r = 0, 1, ... in order: place it against the current state exactly as
 * nbos_oracle_place does; if three servers were found, add g to S on each of them; if fewer were
 * found the kernel is not created (the scheduler scales out and retries later, Section 3.2.1) and
 * nothing changes. Committed GPUs C and the other capacities are not touched: a new replica is
 * idle until a cell runs.
 *   S_final [n_hosts] receives the subscribed GPUs after the last request (may be NULL).
 */
int nbos_oracle_place_sequential(const nbos_oracle_cluster *cl, const int32_t *requests,
                                 int64_t batch, int32_t *out_hosts, int32_t *out_found,
                                 int32_t *S_final)
{
    if (!cl || cl->n_hosts < 0 || batch < 0) return -1;
    int32_t *S_now = (int32_t *)malloc(sizeof(int32_t) * (size_t)(cl->n_hosts > 0 ? cl->n_hosts : 1));
    if (!S_now) return -1;
    for (int32_t h = 0; h < cl->n_hosts; ++h) S_now[h] = cl->S[h];
    nbos_oracle_cluster now = *cl;
    now.S = S_now;
    int rc = 0;
    for (int64_t r = 0; r < batch && rc == 0; ++r) {
        int32_t found = 0;
        rc = nbos_oracle_place(&now, requests + 4 * r, 1, out_hosts + 3 * r, &found);
        if (out_found) out_found[r] = found;
        if (rc == 0 && found == NBOS_ORACLE_REPLICAS_PLACED)
            for (int k = 0; k < NBOS_ORACLE_REPLICAS_PLACED; ++k) S_now[out_hosts[3 * r + k]] += requests[4 * r];
    }
    if (S_final)
        for (int32_t h = 0; h < cl->n_hosts; ++h) S_final[h] = S_now[h];
    free(S_now);
    return rc;
}
