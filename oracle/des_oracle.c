/*
 * CPU oracle for the InferLine Estimator -- TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, literal statement of what the Estimator computes.  It
 * exists so that tests can check the CUDA path against it; nothing in the
 * product path may call it, and it shares no code with the CUDA sources.
 *
 * What it follows (InferLine, arXiv 1812.01776):
 *   - Section 4.2 (Estimator): a discrete-event simulator with one global
 *     logical clock that is advanced from one event to the next, events being
 *     processed in temporal order; it takes a pipeline configuration, the
 *     model profiles and a sample arrival trace, simulates the whole pipeline
 *     including queueing, and yields a latency for every query of the trace.
 *   - Section 3 (requirements on the serving system): one centralized batched
 *     queue per model hands batches of at most the configured maximum batch
 *     size to that model's replicas; this behaviour is deterministic.
 *   - Section 2.1 (Combinatorial Configuration Space): a batch returns as a
 *     whole -- no query of a batch is done before the last one is; and a
 *     pipeline configuration is, per model, a hardware type, a maximum batch
 *     size and a replication factor.
 *   - Section 2 / Section 4.1: conditional control flow -- only a subset of the
 *     models is visited by a given query.
 *   - Section 2 (P99 objective): 99% of the query latencies must lie below the
 *     objective.
 *
 * Readings taken where the paper is silent (each is pinned by a test):
 *   - Everything that happens at one timestamp happens in three phases: all
 *     completions (stage by stage, within a stage in the order their batches
 *     were dispatched), then all external arrivals (in trace order), then
 *     dispatching, stage by stage.
 *   - An idle replica with a non-empty queue takes min(queue length, max
 *     batch) queries from the front of the FIFO queue at once; the lowest-id
 *     idle replica goes first.
 *   - Batch-mates enter the next stage's queue in the order they had in the
 *     batch.  A query follows EVERY child edge whose condition its branch bits
 *     satisfy (Section 2: the pipeline is a DAG whose edges are dataflow; two
 *     unconditional children are two branches that work on the query in
 *     parallel); where it follows none, that copy of the query leaves the
 *     pipeline.  The query is answered when its last copy has left, and its
 *     latency is that instant - arrival time (Section 4.3 measures the service
 *     time along the LONGEST path of the DAG).  With mutually exclusive
 *     conditions (the conditional control flow of Section 2) there is one copy
 *     and one path.  There is no delay between stages.
 *   - A stage may have a SECOND incoming edge (a join: Section 2 draws pipelines as DAGs whose edges
 *     are dataflow, so a model that consumes two models' outputs needs both).  A query enters the
 *     join's queue at the instant the last of the incoming edges it follows delivers it -- one edge if
 *     its branch bits switch the other one off -- and is processed there once.
 *   - Batch time is a dense table lookup lat[stage][hw][b-1] for the actual
 *     batch size b.
 *   - P99 is the k-th smallest latency, k = ceil(0.99 n) computed in integers
 *     as (99 n + 99) / 100; a query misses the objective iff latency > slo.
 *
 * Single-threaded, plain C, all times int64 microseconds.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK            0
#define ORC_ERR_ARG      -1
#define ORC_ERR_TOPOLOGY -2
#define ORC_ERR_PROFILE  -3
#define ORC_ERR_TRACE    -4
#define ORC_ERR_CONFIG   -5
#define ORC_ERR_NOMEM    -6
#define ORC_ERR_INTERNAL -7

enum { EV_COMPLETION = 0, EV_ARRIVAL = 1 };

typedef struct {
    int64_t time;
    int64_t seq;
    int32_t kind;    /* EV_COMPLETION sorts before EV_ARRIVAL at equal time */
    int32_t stage;   /* completion: stage; arrival: unused */
    int32_t replica; /* completion: replica id; arrival: unused */
    int32_t query;   /* arrival: trace index */
} event_t;

/* Completions of one instant are taken stage by stage (lower stage index first) and, within a stage, in
 * the order their batches were dispatched.  While every stage has one parent the order between stages
 * cannot matter; with a join it decides who enters the join's queue first, and a rule that a stage-wise
 * formulation can follow as well is needed. */
static int ev_less(const event_t *a, const event_t *b)
{
    if (a->time != b->time) return a->time < b->time;
    if (a->kind != b->kind) return a->kind < b->kind;
    if (a->kind == EV_COMPLETION && a->stage != b->stage) return a->stage < b->stage;
    return a->seq < b->seq;
}

typedef struct { event_t *e; int64_t size, cap; } heap_t;

static void heap_push(heap_t *h, event_t v)
{
    int64_t i = h->size++;
    while (i > 0) {
        int64_t p = (i - 1) / 2;
        if (!ev_less(&v, &h->e[p])) break;
        h->e[i] = h->e[p];
        i = p;
    }
    h->e[i] = v;
}

static event_t heap_pop(heap_t *h)
{
    event_t top = h->e[0];
    event_t last = h->e[--h->size];
    int64_t i = 0, n = h->size;
    for (;;) {
        int64_t c = 2 * i + 1;
        if (c >= n) break;
        if (c + 1 < n && ev_less(&h->e[c + 1], &h->e[c])) c++;
        if (!ev_less(&h->e[c], &last)) break;
        h->e[i] = h->e[c];
        i = c;
    }
    if (n > 0) h->e[i] = last;
    return top;
}

/* One record per dispatched batch, for tests that check invariants. */
typedef struct {
    int32_t stage, replica, batch, reserved;
    int64_t t_dispatch, t_finish;
} orc_dispatch_t;

static int cmp_i64(const void *a, const void *b)
{
    int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
    return (x > y) - (x < y);
}

/* Checks the graph: parent[0] = -1, parent[s] < s, an optional second parent with
 * parent[s] < parent2[s] < s, at most two outgoing edges per stage, each edge
 * unconditional or guarded by one branch bit. */
static int check_topology(int S, const int32_t *parent, const int8_t *cond_bit,
                          const uint8_t *cond_val, const int32_t *parent2,
                          const int8_t *cond_bit2, const uint8_t *cond_val2)
{
    if (parent[0] != -1) return ORC_ERR_TOPOLOGY;
    if (parent2 && parent2[0] != -1) return ORC_ERR_TOPOLOGY;
    for (int s = 1; s < S; s++) {
        if (parent[s] < 0 || parent[s] >= s) return ORC_ERR_TOPOLOGY;
        if (cond_bit[s] < -1 || cond_bit[s] > 7) return ORC_ERR_TOPOLOGY;
        if (cond_bit[s] >= 0 && cond_val[s] > 1) return ORC_ERR_TOPOLOGY;
        if (parent2 && parent2[s] != -1) {
            if (parent2[s] <= parent[s] || parent2[s] >= s) return ORC_ERR_TOPOLOGY;
            if (cond_bit2[s] < -1 || cond_bit2[s] > 7) return ORC_ERR_TOPOLOGY;
            if (cond_bit2[s] >= 0 && cond_val2[s] > 1) return ORC_ERR_TOPOLOGY;
        }
    }
    for (int p = 0; p < S; p++) {
        int nchild = 0;
        for (int c = 1; c < S; c++) {
            if (parent[c] == p && ++nchild > 2) return ORC_ERR_TOPOLOGY;
            if (parent2 && parent2[c] == p && ++nchild > 2) return ORC_ERR_TOPOLOGY;
        }
    }
    return ORC_OK;
}

static int edge_on(int8_t bit, uint8_t val, const uint8_t *branch_bits, int64_t q)
{
    return bit < 0 || (uint8_t)((branch_bits[q] >> bit) & 1) == val;
}

/*
 * Simulates ONE candidate configuration over the whole trace.
 *
 *   config          [S][4] bytes: hw, max_batch, replicas, reserved
 *   replica_pref    0: the lowest-id idle replica dispatches first (the rule);
 *                   1: the highest-id idle replica does (only for the test that
 *                      shows the choice cannot change any latency)
 *   out_latency     NULL or int64[n]: latency of every query, by trace index
 *   out_log         NULL or room for log_cap dispatch records; *out_nlog gets
 *                   the number of batches dispatched (may exceed log_cap)
 *   parent2, cond_bit2, cond_val2
 *                   NULL (no joins), or per stage the second incoming edge: its
 *                   source stage (-1: none) and its guard
 */
int orc_estimate_one_dag(int32_t S, int32_t H, int32_t Bmax,
                     const int32_t *parent, const int8_t *cond_bit, const uint8_t *cond_val,
                     const int32_t *parent2, const int8_t *cond_bit2, const uint8_t *cond_val2,
                     const int32_t *latency_us,
                     int64_t n, const int64_t *arrival_us, const uint8_t *branch_bits,
                     const uint8_t *config, int64_t slo_us, int32_t replica_pref,
                     int64_t *out_p99_us, int64_t *out_miss,
                     int64_t *out_latency,
                     orc_dispatch_t *out_log, int64_t log_cap, int64_t *out_nlog)
{
    if (S < 1 || S > 16 || H < 1 || H > 8 || Bmax < 1 || Bmax > 64 || n < 1) return ORC_ERR_ARG;
    if (!parent || !cond_bit || !cond_val || !latency_us || !arrival_us || !config) return ORC_ERR_ARG;
    if (parent2 && (!cond_bit2 || !cond_val2)) return ORC_ERR_ARG;
    int rc = check_topology(S, parent, cond_bit, cond_val, parent2, cond_bit2, cond_val2);
    if (rc) return rc;
    int any_cond = 0, any_join = 0;
    for (int s = 1; s < S; s++) {
        any_cond |= (cond_bit[s] >= 0);
        if (parent2 && parent2[s] >= 0) { any_join = 1; any_cond |= (cond_bit2[s] >= 0); }
    }
    if (any_cond && !branch_bits) return ORC_ERR_ARG;
    for (int64_t i = 0; i < (int64_t)S * H * Bmax; i++)
        if (latency_us[i] < 1) return ORC_ERR_PROFILE;
    if (arrival_us[0] < 0) return ORC_ERR_TRACE;
    for (int64_t i = 1; i < n; i++)
        if (arrival_us[i] < arrival_us[i - 1]) return ORC_ERR_TRACE;
    int R[16], MB[16], HW[16], total_R = 0;
    for (int s = 0; s < S; s++) {
        HW[s] = config[4 * s + 0];
        MB[s] = config[4 * s + 1];
        R[s]  = config[4 * s + 2];
        if (HW[s] >= H || MB[s] < 1 || MB[s] > Bmax || R[s] < 1 || R[s] > 32) return ORC_ERR_CONFIG;
        total_R += R[s];
    }

    /* state */
    heap_t heap = { NULL, 0, n + total_R + 1 };
    int32_t *queue[16];          /* Q_s: ids in arrival order; each query enters a stage once */
    int64_t qhead[16], qtail[16];
    uint8_t *busy[16];
    int32_t *inflight[16];       /* [R_s][MB_s] ids of the batch a replica is working on */
    int32_t *inflight_n[16];
    int64_t *lat = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    uint8_t *done = (uint8_t *)calloc((size_t)n, 1);
    int32_t *copies = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);   /* copies of the query still in the pipeline */
    heap.e = (event_t *)malloc(sizeof(event_t) * (size_t)heap.cap);
    /* joins only: reach[s][q] = the query visits stage s; need[s][q] = how many of the stage's incoming
     * edges deliver it; arrived[s][q] = how many have so far */
    uint8_t *reach = any_join ? (uint8_t *)calloc((size_t)n * S, 1) : NULL;
    uint8_t *need = any_join ? (uint8_t *)calloc((size_t)n * S, 1) : NULL;
    uint8_t *arrived = any_join ? (uint8_t *)calloc((size_t)n * S, 1) : NULL;
    int ok = lat && done && copies && heap.e && (!any_join || (reach && need && arrived));
    for (int s = 0; s < S; s++) {
        queue[s] = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        busy[s] = (uint8_t *)calloc((size_t)R[s], 1);
        inflight[s] = (int32_t *)malloc(sizeof(int32_t) * (size_t)R[s] * MB[s]);
        inflight_n[s] = (int32_t *)calloc((size_t)R[s], sizeof(int32_t));
        qhead[s] = qtail[s] = 0;
        ok = ok && queue[s] && busy[s] && inflight[s] && inflight_n[s];
    }
    int64_t nlog = 0, n_done = 0, seq = 0;
    rc = ORC_OK;
    if (!ok) { rc = ORC_ERR_NOMEM; goto cleanup; }

    for (int64_t i = 0; i < n; i++) {
        event_t ev = { arrival_us[i], i, EV_ARRIVAL, 0, 0, (int32_t)i };
        heap_push(&heap, ev);
        copies[i] = 1;
    }
    if (any_join) {
        /* which stages a query visits follows from its branch bits alone; parents come first in index order */
        for (int64_t q = 0; q < n; q++) {
            reach[q] = 1;
            for (int c = 1; c < S; c++) {
                int a = reach[(size_t)parent[c] * n + q] && edge_on(cond_bit[c], cond_val[c], branch_bits, q);
                int b = parent2[c] >= 0 && reach[(size_t)parent2[c] * n + q] &&
                        edge_on(cond_bit2[c], cond_val2[c], branch_bits, q);
                need[(size_t)c * n + q] = (uint8_t)(a + b);
                reach[(size_t)c * n + q] = (uint8_t)(a || b);
            }
        }
    }

    while (heap.size > 0) {
        const int64_t clock = heap.e[0].time;

        /* phase 1: every completion at this instant: by stage, then earliest-dispatched batch first */
        while (heap.size > 0 && heap.e[0].time == clock && heap.e[0].kind == EV_COMPLETION) {
            event_t ev = heap_pop(&heap);
            int s = ev.stage, r = ev.replica;
            busy[s][r] = 0;
            for (int j = 0; j < inflight_n[s][r]; j++) {
                int32_t q = inflight[s][r * MB[s] + j];
                int taken = 0;       /* copies that enter a queue now */
                for (int c = s + 1; c < S; c++) {
                    int on = (parent[c] == s && edge_on(cond_bit[c], cond_val[c], branch_bits, q)) ||
                             (any_join && parent2[c] == s && edge_on(cond_bit2[c], cond_val2[c], branch_bits, q));
                    if (!on) continue;
                    /* at a join the copy waits for the other input; the one that completes the set goes on */
                    if (any_join && ++arrived[(size_t)c * n + q] < need[(size_t)c * n + q]) continue;
                    queue[c][qtail[c]++] = q;
                    taken++;
                }
                if (done[q]) { rc = ORC_ERR_INTERNAL; goto cleanup; }
                copies[q] += taken - 1;      /* this copy went on as `taken` copies, was absorbed, or left */
                if (copies[q] == 0) {        /* the last copy has left: the query is answered now */
                    done[q] = 1;
                    lat[q] = clock - arrival_us[q];
                    n_done++;
                }
            }
            inflight_n[s][r] = 0;
        }
        /* phase 2: every external arrival at this instant, in trace order */
        while (heap.size > 0 && heap.e[0].time == clock && heap.e[0].kind == EV_ARRIVAL) {
            event_t ev = heap_pop(&heap);
            queue[0][qtail[0]++] = ev.query;
        }
        /* phase 3: dispatch, stage by stage */
        for (int s = 0; s < S; s++) {
            while (qtail[s] > qhead[s]) {
                int r = -1;
                if (replica_pref == 0) { for (int i = 0; i < R[s]; i++) if (!busy[s][i]) { r = i; break; } }
                else { for (int i = R[s] - 1; i >= 0; i--) if (!busy[s][i]) { r = i; break; } }
                if (r < 0) break;
                int64_t waiting = qtail[s] - qhead[s];
                int b = (int)(waiting < MB[s] ? waiting : MB[s]);
                for (int j = 0; j < b; j++) inflight[s][r * MB[s] + j] = queue[s][qhead[s]++];
                inflight_n[s][r] = b;
                busy[s][r] = 1;
                int64_t d = latency_us[((int64_t)s * H + HW[s]) * Bmax + (b - 1)];
                event_t ev = { clock + d, ++seq, EV_COMPLETION, s, r, -1 };
                heap_push(&heap, ev);
                if (out_log && nlog < log_cap) {
                    orc_dispatch_t rec = { s, r, b, 0, clock, clock + d };
                    out_log[nlog] = rec;
                }
                nlog++;
            }
        }
    }
    if (n_done != n) { rc = ORC_ERR_INTERNAL; goto cleanup; }

    if (out_latency) memcpy(out_latency, lat, sizeof(int64_t) * (size_t)n);
    if (out_nlog) *out_nlog = nlog;
    {
        int64_t miss = 0;
        for (int64_t i = 0; i < n; i++) miss += (lat[i] > slo_us);
        qsort(lat, (size_t)n, sizeof(int64_t), cmp_i64);
        int64_t k = (99 * n + 99) / 100;   /* ceil(0.99 n), 1-indexed rank */
        if (out_p99_us) *out_p99_us = lat[k - 1];
        if (out_miss) *out_miss = miss;
    }

cleanup:
    free(lat); free(done); free(copies); free(heap.e); free(reach); free(need); free(arrived);
    for (int s = 0; s < S; s++) { free(queue[s]); free(busy[s]); free(inflight[s]); free(inflight_n[s]); }
    return rc;
}

/* The same for a pipeline without joins. */
int orc_estimate_one(int32_t S, int32_t H, int32_t Bmax,
                     const int32_t *parent, const int8_t *cond_bit, const uint8_t *cond_val,
                     const int32_t *latency_us,
                     int64_t n, const int64_t *arrival_us, const uint8_t *branch_bits,
                     const uint8_t *config, int64_t slo_us, int32_t replica_pref,
                     int64_t *out_p99_us, int64_t *out_miss,
                     int64_t *out_latency,
                     orc_dispatch_t *out_log, int64_t log_cap, int64_t *out_nlog)
{
    return orc_estimate_one_dag(S, H, Bmax, parent, cond_bit, cond_val, NULL, NULL, NULL, latency_us,
                                n, arrival_us, branch_bits, config, slo_us, replica_pref,
                                out_p99_us, out_miss, out_latency, out_log, log_cap, out_nlog);
}

/* Plain loop over candidates [0, C): configs is [C][S][4] bytes.  Stops at the
 * first error and returns it. */
int orc_estimate_many_dag(int32_t S, int32_t H, int32_t Bmax,
                      const int32_t *parent, const int8_t *cond_bit, const uint8_t *cond_val,
                      const int32_t *parent2, const int8_t *cond_bit2, const uint8_t *cond_val2,
                      const int32_t *latency_us,
                      int64_t n, const int64_t *arrival_us, const uint8_t *branch_bits,
                      const uint8_t *configs, int64_t C, int64_t slo_us,
                      int64_t *out_p99_us, int64_t *out_miss)
{
    for (int64_t c = 0; c < C; c++) {
        int rc = orc_estimate_one_dag(S, H, Bmax, parent, cond_bit, cond_val, parent2, cond_bit2, cond_val2,
                                      latency_us, n, arrival_us, branch_bits, configs + c * S * 4, slo_us, 0,
                                      out_p99_us + c, out_miss + c, NULL, NULL, 0, NULL);
        if (rc) return rc;
    }
    return ORC_OK;
}

int orc_estimate_many(int32_t S, int32_t H, int32_t Bmax,
                      const int32_t *parent, const int8_t *cond_bit, const uint8_t *cond_val,
                      const int32_t *latency_us,
                      int64_t n, const int64_t *arrival_us, const uint8_t *branch_bits,
                      const uint8_t *configs, int64_t C, int64_t slo_us,
                      int64_t *out_p99_us, int64_t *out_miss)
{
    for (int64_t c = 0; c < C; c++) {
        int rc = orc_estimate_one(S, H, Bmax, parent, cond_bit, cond_val, latency_us,
                                  n, arrival_us, branch_bits, configs + c * S * 4, slo_us, 0,
                                  out_p99_us + c, out_miss + c, NULL, NULL, 0, NULL);
        if (rc) return rc;
    }
    return ORC_OK;
}

/* The percentile rule on its own: k-th smallest with k = ceil(0.99 n), and the
 * number of entries above slo_us.  The input is not modified. */
int orc_p99_miss(const int64_t *latency, int64_t n, int64_t slo_us,
                 int64_t *out_p99_us, int64_t *out_miss)
{
    if (!latency || n < 1) return ORC_ERR_ARG;
    int64_t *tmp = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    if (!tmp) return ORC_ERR_NOMEM;
    memcpy(tmp, latency, sizeof(int64_t) * (size_t)n);
    int64_t miss = 0;
    for (int64_t i = 0; i < n; i++) miss += (tmp[i] > slo_us);
    qsort(tmp, (size_t)n, sizeof(int64_t), cmp_i64);
    int64_t k = (99 * n + 99) / 100;
    *out_p99_us = tmp[k - 1];
    *out_miss = miss;
    free(tmp);
    return ORC_OK;
}

/*
 * Traffic envelope of the trace (Section 5, "High-Frequency Tuning"): for a
 * window of length window_us[i], the largest number of arrivals that fall into
 * any window of that length anywhere on the trace.  A window that maximises
 * the count can be moved right until it starts at an arrival, so it is enough
 * to look at the half-open windows [a_j, a_j + window_us[i]) for every arrival
 * j.  Plain two-pointer sweep per window length.
 */
int orc_traffic_envelope(int64_t n, const int64_t *arrival_us, int32_t n_windows,
                         const int64_t *window_us, int64_t *out_max_count)
{
    if (n < 1 || !arrival_us || n_windows < 0 || (n_windows > 0 && (!window_us || !out_max_count)))
        return ORC_ERR_ARG;
    for (int64_t i = 1; i < n; i++)
        if (arrival_us[i] < arrival_us[i - 1]) return ORC_ERR_TRACE;
    for (int32_t w = 0; w < n_windows; w++) {
        if (window_us[w] < 1) return ORC_ERR_ARG;
        int64_t best = 0, hi = 0;
        for (int64_t j = 0; j < n; j++) {
            if (hi < j) hi = j;
            while (hi < n && arrival_us[hi] - arrival_us[j] < window_us[w]) hi++;
            if (hi - j > best) best = hi - j;
        }
        out_max_count[w] = best;
    }
    return ORC_OK;
}
