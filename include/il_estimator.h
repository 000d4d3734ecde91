/*
 * il_estimator.h -- C ABI of the batched InferLine Estimator for NVIDIA B200 (sm_100a).
 *
 * The Estimator (InferLine, arXiv 1812.01776, Section 4.2) is a discrete-event
 * simulation: given a pipeline configuration, the per-model profiles and a
 * sample arrival trace it replays the trace through the pipeline, queueing
 * included, and yields the latency of every query.  The Planner (Section 4.3,
 * Algorithms 1 and 2) asks it one question per candidate configuration --
 * "does this configuration meet the latency objective at P99?" (Feasible) --
 * and asks it for many candidates against the same profiles and trace.  This
 * library answers that question for a whole batch of candidates per call:
 * profiles and trace are bound once (create), candidates are evaluated many
 * times (estimate).
 *
 * Simulated system (Section 3: centralized batched queue; Section 2.1: batches
 * complete as a whole; configuration = per model a hardware type, a maximum
 * batch size and a replication factor):
 *   - every stage has one FIFO queue and R identical replicas;
 *   - a replica that is idle while the queue is non-empty takes
 *     min(queue length, max batch) queries from the front at once (the
 *     lowest-id idle replica first) and is busy for
 *     latency_us[stage][hw][b-1] microseconds, b being the batch it took;
 *   - all queries of the batch leave the stage together; each follows every
 *     child edge whose condition its branch bits satisfy (with conditional
 *     control flow: at most one), with zero delay, in batch order; a copy with
 *     no such edge leaves the pipeline, and the query's latency is the instant
 *     its last copy leaves minus its arrival time;
 *   - everything at one timestamp happens as: all completions (batches
 *     dispatched earlier first), then all trace arrivals (in trace order), then
 *     dispatching;
 *   - per candidate the result is the k-th smallest latency, k = ceil(0.99 n)
 *     = (99 n + 99) / 100 in integers (Section 2: P99 objective), and the
 *     number of queries with latency > slo_us.
 * All times are int64 microseconds.  Results are exact integers; there is no
 * floating point on the path.
 *
 * There is no CPU fallback: every entry point that computes needs a CUDA
 * device of compute capability 10.x and fails with IL_ERR_CUDA otherwise.
 *
 * Threading: calls on ONE handle must not overlap.  Different handles may be
 * used from different threads.  Unless said otherwise a call returns after all
 * work it enqueued has completed.
 */
#ifndef IL_ESTIMATOR_H
#define IL_ESTIMATOR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define IL_API __attribute__((visibility("default")))
#else
#define IL_API
#endif

#define IL_MAX_STAGES     16
#define IL_MAX_HW          8
#define IL_MAX_BATCH      64
#define IL_MAX_REPLICAS   32

/* Return codes.  0 is success; on any error no output element is defined. */
#define IL_OK                 0
#define IL_ERR_INVALID_ARG   -1  /* NULL pointer, n < 0, sizes out of the limits above      */
#define IL_ERR_BAD_TOPOLOGY  -2  /* not a tree in the accepted form (see il_profiles)      */
#define IL_ERR_BAD_PROFILE   -3  /* a latency table entry < 1                              */
#define IL_ERR_BAD_TRACE     -4  /* arrival times negative, decreasing, or too large       */
#define IL_ERR_BAD_CONFIG    -5  /* a candidate with hw >= H, max_batch or replicas out of range */
#define IL_ERR_NOMEM         -6  /* host or device allocation failed / workspace too small */
#define IL_ERR_CUDA          -7  /* a CUDA runtime call failed; see il_last_cuda_error     */
#define IL_ERR_ITER_LIMIT    -8  /* a device loop hit its iteration bound (internal error) */
#define IL_ERR_TOO_LARGE     -9  /* il_estimate_device_static: needs more than IL_STATIC_SCRATCH_BYTES */
#define IL_ERR_BOUNDS       -10  /* checked build only (-DIL_CHECKED): a device index left its array; the access
                                    was skipped and recorded instead (internal error)                        */

typedef struct il_estimator il_estimator;   /* opaque; owns its device copies */

/*
 * Pipeline shape and model profiles (Section 4.1: a profile gives, per
 * hardware type and batch size, how long the model takes for that batch).
 * All pointers are HOST pointers, read during il_estimator_create only.
 *
 * The pipeline is a tree.  Stage 0 is the root, parent[s] < s, and a stage has
 * at most two children.  The edge parent[s] -> s is taken by query q iff
 * cond_bit[s] < 0, or ((branch_bits[q] >> cond_bit[s]) & 1) == cond_val[s].
 * A query goes down EVERY edge of a stage whose condition it satisfies, and
 * where it satisfies none, that copy of it leaves the pipeline; the query is
 * answered when its last copy has left, and its latency is that instant minus
 * its arrival time (Section 2: a pipeline is a DAG whose edges are dataflow;
 * Section 4.3: the service time is taken along the longest path).  Two children
 * guarded by the SAME bit with different values are alternatives (conditional
 * control flow: one path per query), and a guarded edge without sibling is a
 * cascade (the other queries leave there).  Two children that are not
 * alternatives -- both unconditional, or guarded by different bits -- are
 * fan-out: parallel branches.  Handles with fan-out run on the lane kernel
 * (whole streams) or the kernel with separate streams; the other kernel
 * choices, prefix sharing and the early exit of il_feasible fall back to those.
 * A stage that waits for the outputs of TWO stages (a join) is described with
 * il_join_edges and il_estimator_create_dag below.
 */
typedef struct {
    int32_t        n_stages;    /* S, 1..IL_MAX_STAGES                                  */
    int32_t        n_hw;        /* H, 1..IL_MAX_HW                                      */
    int32_t        max_batch;   /* Bmax, 1..IL_MAX_BATCH; tables are dense in b = 1..Bmax */
    const int32_t *parent;      /* [S], parent[0] = -1                                  */
    const int8_t  *cond_bit;    /* [S], -1 or 0..7                                      */
    const uint8_t *cond_val;    /* [S], 0 or 1 (ignored where cond_bit < 0)             */
    const int32_t *latency_us;  /* [S][H][Bmax] row-major, every entry >= 1             */
} il_profiles;

/*
 * The sample arrival trace (Section 3: provided by the developer; Section 4.2:
 * input of the Estimator).  HOST pointers, copied by il_estimator_create.
 */
typedef struct {
    int64_t        n_queries;   /* n, 1 .. 2^31 - 1                                     */
    const int64_t *arrival_us;  /* [n], >= 0 and non-decreasing; equal stamps keep trace order */
    const uint8_t *branch_bits; /* [n]; may be NULL when no stage has cond_bit >= 0     */
} il_trace;

/* One stage of one candidate configuration (Section 2.1: hardware type,
 * maximum batch size, replication factor).  A candidate is S of these in a
 * row; a batch of candidates is an array [n_candidates][S]. */
typedef struct {
    uint8_t hw;         /* 0 .. H-1                     */
    uint8_t max_batch;  /* 1 .. Bmax                    */
    uint8_t replicas;   /* 1 .. IL_MAX_REPLICAS         */
    uint8_t reserved;   /* ignored                      */
} il_stage_config;

/* Counters of the most recent il_estimate / il_estimate_device call. */
typedef struct {
    int64_t candidates;      /* candidates evaluated                                     */
    int64_t query_events;    /* candidates * sum over stages of queries visiting the stage */
    int64_t batches;         /* batches dispatched, all candidates, all stages           */
    int64_t algorithmic_ops; /* integer operations the method needs: per batch R + max_batch + 4
                                (replica min, queue count, table add, slot update), per query-event 3 */
    int64_t chunks;          /* how many (simulate, select) launch groups the call made (the
                                warp-per-candidate kernels add an ordering launch to each)  */
    int64_t kernel_launches; /* kernels of this library launched by the call             */
    double  sim_ms;          /* device time of the simulation kernels (CUDA events)      */
    double  select_ms;       /* device time of the percentile kernels (CUDA events)      */
    double  total_ms;        /* device time of all stream work of the call               */
    int64_t fallback_candidates; /* candidates the lane kernel gave up on (stream ring overflow) and the
                                warp-per-candidate kernel evaluated instead; results are the same     */
    int64_t stage_runs;      /* (stage, candidate) simulations carried out: candidates * S unless
                                candidates with a common configuration prefix shared them            */
    int64_t error_detail;    /* diagnostic for IL_ERR_ITER_LIMIT: which device check gave up (bit 0: the
                                lane kernel's iteration bound, bit 1: its count of leaving queries, bit 3:
                                the warp-per-candidate kernel's count of leaving queries); 0 otherwise */
    int64_t early_exits;     /* il_feasible*: candidates dropped before the end of the trace because more
                                queries had missed the objective than the P99 rule allows             */
} il_stats;

/*
 * Binds profiles and trace (Section 4.2: the Estimator's fixed inputs) on the
 * current CUDA device: validates them, copies them to device memory, and
 * precomputes from the branch bits how many queries visit each stage.
 *   profiles, trace   host structs with host pointers (see above)
 *   out               receives the handle; untouched on error
 * Errors: INVALID_ARG, BAD_TOPOLOGY, BAD_PROFILE, BAD_TRACE (also when
 * last arrival + (sum over stages of n * largest table entry) would not fit in
 * 62 bits), NOMEM, CUDA.
 */
IL_API int il_estimator_create(const il_profiles *profiles, const il_trace *trace, il_estimator **out);

/*
 * Joins (Section 2: the pipeline is a DAG whose edges are dataflow, so a model
 * may consume the outputs of two models).  Per stage s an optional SECOND
 * incoming edge parent2[s] -> s, with parent[s] < parent2[s] < s, guarded like
 * the first one by (cond_bit2[s], cond_val2[s]); parent2[s] = -1: none.  A query
 * enters the queue of stage s at the instant the LAST of the incoming edges it
 * follows delivers it (both, or the only one its branch bits leave on) and is
 * processed there once.  Queries that become ready in the same instant queue in
 * the order (delivering stage, that stage's completion order).  A stage still
 * has at most two outgoing edges, counting both kinds.  HOST pointers, [S] each,
 * read during the call only.
 */
typedef struct {
    const int32_t *parent2;     /* [S], -1 or parent[s] < parent2[s] < s                */
    const int8_t  *cond_bit2;   /* [S], -1 or 0..7                                      */
    const uint8_t *cond_val2;   /* [S], 0 or 1 (ignored where cond_bit2 < 0)            */
} il_join_edges;

/*
 * il_estimator_create for a pipeline with joins; `joins` may be NULL (then the
 * two calls are the same).  A handle with a join runs on the kernel with
 * separate streams (kernel name "des_kernel") whatever variant is set: that
 * kernel builds the join's arrival stream from the two incoming streams before
 * it simulates the stage.  Every entry point works on such a handle and gives
 * the same results as on any other; il_feasible* evaluate it without early exit.
 * Errors: as il_estimator_create; BAD_TOPOLOGY also for a second edge outside
 * the form above or a third outgoing edge; TOO_LARGE if the streams of one
 * candidate exceed 2^31 - 1 elements.
 */
IL_API int il_estimator_create_dag(const il_profiles *profiles, const il_join_edges *joins,
                                   const il_trace *trace, il_estimator **out);

/* Frees the handle and everything the library allocated for it.  Memory given
 * through il_set_workspace stays the caller's.  NULL is allowed. */
IL_API void il_estimator_destroy(il_estimator *est);

/*
 * Evaluates n candidate configurations against the bound profiles and trace
 * (Section 4.2 run once per candidate; Section 4.3 "Feasible" is
 * out_p99_us[c] <= slo_us, equivalently out_miss[c] <= n_queries - k).
 *   configs      HOST pointer, [n][S] il_stage_config
 *   n            number of candidates, >= 0 (0 is a no-op)
 *   slo_us       latency objective for the miss count
 *   out_p99_us   HOST pointer, [n]: k-th smallest latency of candidate c
 *   out_miss     HOST pointer, [n]: number of queries with latency > slo_us
 * Candidates are validated on the host before anything is launched
 * (BAD_CONFIG names no index; nothing is written).  Copies to and from the
 * device happen inside the call, on the handle's stream.
 */
IL_API int il_estimate(il_estimator *est, const il_stage_config *configs, int64_t n, int64_t slo_us,
                       int64_t *out_p99_us, int64_t *out_miss);

/*
 * Same computation with DEVICE pointers (memory of the handle's device, e.g.
 * owned by a torch tensor): configs [n][S], out_p99_us [n], out_miss [n].
 * Work is enqueued on the handle's stream and the call waits for it.
 * Candidates are validated on the device; an invalid one makes the call return
 * BAD_CONFIG after the stream has drained, and outputs are then undefined.
 *
 * Shared prefixes.  The completion stream of a stage depends only on the
 * configurations of the stages on its path from the root, so candidates that
 * agree there need that part simulated once.  With the default kernel choice
 * (IL_VARIANT_AUTO), a batch of at least 2,048 candidates, n - ceil(0.99 n) <
 * 16,384 and enough workspace, the call first builds the set of distinct (stage,
 * configuration, parent) nodes on the device; if there are at most a quarter as
 * many nodes as candidates x stages (an exhaustive sweep over per-stage choices,
 * not a uniform random draw) it simulates the nodes instead of the candidates --
 * through a small set of whole candidates that between them contain every node
 * queries leave after, or node by node -- and assembles each candidate's P99 and
 * miss count from the nodes where its queries leave.  Results are the same
 * integers; il_stats.stage_runs tells how many stage simulations were carried out.
 */
IL_API int il_estimate_device(il_estimator *est, const il_stage_config *d_configs, int64_t n,
                              int64_t slo_us, int64_t *d_out_p99_us, int64_t *d_out_miss);

/*
 * Feasibility only (Section 4.3: the one question the Planner asks in Algorithms 1 and 2,
 * "Feasible(pipeline, slo)": does the configuration meet the objective at P99?).
 *   out_feasible[c] = 1  iff  the k-th smallest latency of candidate c is <= slo_us, k = ceil(0.99 n),
 *                        equivalently iff at most n - k queries have latency > slo_us;  else 0.
 * Exactly the answer out_p99_us[c] <= slo_us of il_estimate, but cheaper to get: the lane kernel
 * compares each query with the objective as it leaves the pipeline, writes no latencies and runs no
 * percentile pass, and drops a candidate as soon as more than n - k of its queries have missed the
 * objective (an overloaded candidate is decided within the first few per cent of the trace;
 * il_stats.early_exits counts them).  A feasible candidate is simulated to the end, so its answer is
 * exact too.  The warp-per-candidate kernels have no early exit: with them this call computes P99
 * and compares.
 *   il_feasible         configs HOST [n][S], out_feasible HOST [n] bytes; candidates validated on the host
 *   il_feasible_device  DEVICE pointers; an invalid candidate makes the call return BAD_CONFIG
 * Work on the handle's stream; returns after completion.  Errors as il_estimate / il_estimate_device.
 * If the lane kernel gives candidates up on stream ring overflow (see il_set_variant), they are
 * evaluated by the warp-per-candidate kernel in the same call, which then allocates temporaries.
 */
IL_API int il_feasible(il_estimator *est, const il_stage_config *configs, int64_t n, int64_t slo_us,
                       uint8_t *out_feasible);
IL_API int il_feasible_device(il_estimator *est, const il_stage_config *d_configs, int64_t n, int64_t slo_us,
                              uint8_t *d_out_feasible);

/*
 * The Estimator's full answer for ONE configuration: the latency of every
 * query of the trace (Section 4.2: it "returns accurate estimates of the
 * latency for each query in the trace"; P99 and miss count are reductions of
 * this vector).
 *   d_config          DEVICE pointer, [S] il_stage_config (one candidate)
 *   d_out_latency_us  DEVICE pointer, [n_queries]: latency of query i of the trace
 * Runs one warp; meant for inspection and tests, not for throughput.  Errors
 * as il_estimate_device.
 */
IL_API int il_estimate_latencies(il_estimator *est, const il_stage_config *d_config,
                                 int64_t *d_out_latency_us);

/*
 * Traffic envelope of the bound trace (Section 5: the Planner builds it for the
 * sample trace and hands it to the Tuner): for each window length
 * window_us[i] >= 1, the largest number of arrivals in any half-open window
 * [t, t + window_us[i]) on the trace; the maximum arrival rate at that time
 * scale is out_max_count[i] / window_us[i].  The paper takes the lengths from
 * the pipeline's service time, doubling up to 60 s; the caller chooses them.
 *   window_us       HOST pointer, [n_windows], n_windows <= 64
 *   out_max_count   HOST pointer, [n_windows]
 * Errors: INVALID_ARG, CUDA.
 */
IL_API int il_traffic_envelope(il_estimator *est, const int64_t *window_us, int32_t n_windows,
                               int64_t *out_max_count);

/*
 * Allocation-free variant of il_estimate_device (the paper has no counterpart;
 * this is a deployment convenience of this library).
 *
 * Who needs it: a Planner that runs inside a serving process usually shares
 * its GPU with a model server whose memory pool has already claimed the
 * device's memory, so a cudaMalloc made by this library can fail there, and
 * even when it succeeds it synchronises the whole device and stalls the
 * inference kernels running next to it.  Such callers create the handle once
 * at start-up (creation does allocate the device copies of trace and profiles)
 * and afterwards use this call, which never calls cudaMalloc, cudaFree or any
 * other allocating routine: the simulation kernel's scratch (inter-stage
 * streams, latency slab, counters) lives in one static device array of
 * IL_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that
 * loads the library holds that much memory until the process exits.
 *
 * Arguments and results are those of il_estimate_device (DEVICE pointers,
 * work on the handle's stream, returns after completion, same values bit for
 * bit).  A workspace set with il_set_workspace is ignored, and il_get_stats is
 * not updated.  The call runs on the handle's device and leaves the caller's
 * current device as it found it; after an error it has still waited for whatever
 * it had enqueued, and il_last_cuda_error names the failing CUDA call.
 *
 * Limit: the whole batch is evaluated in one pass, with at most 32 warps
 * resident, and must fit the array:
 *     256 + r * slot * min(32, n rounded up to 4) + (8 * n_queries' + 4) * n
 *         <= IL_STATIC_SCRATCH_BYTES
 * where n_queries' is n_queries rounded up to 32, slot is the number of
 * stream elements one warp keeps between stages (for a linear pipeline about
 * 2 * n_queries; never more than the query-events per candidate), and r is 8
 * bytes per element (12 when the times are too large for packed records, see
 * il_set_variant, or IL_VARIANT_WIDE is set).  A larger
 * request returns IL_ERR_TOO_LARGE and launches nothing; split the batch or use
 * il_estimate_device.
 *
 * The first call on a device looks up the array's device address; make that
 * first call during start-up, before any stream capture begins.  All calls, on
 * all handles, share the one array: it keeps the previous call's contents (the
 * call clears the counters it needs to start at zero), and two calls that
 * overlap on the same GPU, from different handles or streams, race on it and
 * give wrong results.  Serialise them.
 */
#define IL_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
IL_API int il_estimate_device_static(il_estimator *est, const il_stage_config *d_configs, int64_t n,
                                     int64_t slo_us, int64_t *d_out_p99_us, int64_t *d_out_miss);

/* Stream all later calls on this handle use (a cudaStream_t passed as void*;
 * NULL = the default stream).  The stream stays the caller's. */
IL_API int il_set_stream(il_estimator *est, void *cuda_stream);

/*
 * Scratch memory.  The simulation keeps, per resident warp, the streams of
 * (time, query) pairs that flow between stages, and per candidate of a chunk
 * its n latencies for the percentile kernel.
 *   il_workspace_bytes  size that lets a call of n_candidates run at full
 *                       occupancy (for large n_candidates: the size beyond
 *                       which more memory no longer helps)
 *   il_workspace_min_bytes  smallest size il_set_workspace accepts
 *   il_set_workspace    hands the library a DEVICE buffer (256-byte aligned) of
 *                       the given size; it stays the caller's and must outlive
 *                       its use.  NULL/0 returns to library-owned scratch.
 * Without il_set_workspace the library allocates its own scratch with
 * cudaMalloc inside the first estimate call that needs it: il_workspace_bytes
 * for that call's candidate count, but never more than 80 % of the memory that
 * is free on the device at that moment.  A later call that wants more makes the
 * library synchronise the stream, free the buffer and allocate a larger one (by
 * the same rule); it is kept until destroy.  Callers that share the device with
 * other allocators should size and own the buffer themselves (il_set_workspace),
 * or use il_estimate_device_static.
 */
IL_API int il_workspace_bytes(const il_estimator *est, int64_t n_candidates, size_t *bytes);
IL_API int il_workspace_min_bytes(const il_estimator *est, size_t *bytes);
IL_API int il_set_workspace(il_estimator *est, void *d_workspace, size_t bytes);

/*
 * Chooses the simulation kernel.  All variants give identical results.
 *
 * Records.  When every time the simulation can reach (last arrival + sum over
 * stages of n * largest table entry) fits in 63 - q bits, q = max(5, ceil(log2 n)),
 * a stream element is one 64-bit word (time << q) | query ("packed"); otherwise
 * only IL_VARIANT_WIDE applies and every other choice falls back to it.
 *
 * IL_VARIANT_AUTO (default): the lane kernel.
 * IL_VARIANT_LANES: one lane per (candidate, stage); the stages of a candidate
 *   run side by side as a pipeline inside one warp, floor(32 / S) candidates per
 *   warp; a group of lanes takes its next candidate as soon as it has finished
 *   one.  While the inter-stage streams of all resident candidates fit 48 GiB
 *   every stage keeps its whole arrival stream in the workspace.  Beyond that
 *   (long traces through deep pipelines) a stage's stream lives in a ring of
 *   8,192 records, so the scratch per resident candidate does not grow with the
 *   trace, and a parent stage waits when it would overrun its child's ring.  A
 *   candidate in which one batch stays in flight while more than a ring of later
 *   records passes through the other replicas of its stage cannot be finished
 *   that way: it is evaluated by the IL_VARIANT_PACKED kernel in the same call
 *   (il_stats.fallback_candidates counts them).
 * IL_VARIANT_PACKED: one candidate per warp, stages one after the other, replica
 *   slots across the lanes, warp-level primitives for the queue count and the
 *   slot to reuse.
 * IL_VARIANT_STAGED: IL_VARIANT_PACKED with the shared trace staged through
 *   shared memory once per CTA (bulk asynchronous copies into a ring of tiles
 *   that the CTA's four warps consume together) instead of every warp reading
 *   it through L1/L2 on its own; on B200 it measured slower (the warps of a CTA
 *   must then move through the root stage within one ring length of each other).
 * IL_VARIANT_WIDE: one candidate per warp with separate 64-bit time and 32-bit
 *   query streams; always valid.
 * il_workspace_bytes depends on the variant in force: set the variant first.
 */
#define IL_VARIANT_AUTO 0
#define IL_VARIANT_WIDE 1
#define IL_VARIANT_STAGED 2
#define IL_VARIANT_LANES 3
#define IL_VARIANT_PACKED 4
IL_API int il_set_variant(il_estimator *est, int variant);

/*
 * Hooks for the library's own tests; not for production use.
 *   IL_KNOB_LANE_RING_LOG2  value 6..24: the lane kernel keeps its streams in rings of at most 2^value
 *                           records whatever the sizes (by default the library chooses between whole
 *                           streams and rings of 2^13).  Small rings force the overflow path.
 *   IL_KNOB_ITER_LIMIT      value >= 0: iteration bound of the simulation kernels' loops; 0 restores
 *                           the bound each loop derives from its input.  A small bound makes a call
 *                           return IL_ERR_ITER_LIMIT; the handle stays usable.
 *   IL_KNOB_SHARE_PREFIXES  0: the library decides per call whether to evaluate a batch through shared
 *                           configuration prefixes (see il_estimate_device); 1: always, when the
 *                           preconditions hold; 2: never; 3: always, and the distinct stage runs are
 *                           simulated one by one even where a covering set of whole candidates on
 *                           the lane kernel would do.
 *   IL_KNOB_LANE_CTAS       value 0..16: resident CTAs (of two warps) per SM of the lane kernel; 0 restores
 *                           the library's choice (4).  For measurements.
 *   IL_KNOB_BITS_IN_RECORDS value 0 or 1: whether the lane kernel's stream records carry the queries' branch
 *                           bits (1, the default where the time range leaves room) or every stage looks
 *                           them up by query index (0).  Same results either way.
 * Set a knob before il_workspace_bytes / il_set_workspace: sizes depend on the ring length.
 */
#define IL_KNOB_LANE_RING_LOG2 1
#define IL_KNOB_ITER_LIMIT 2
#define IL_KNOB_SHARE_PREFIXES 3
#define IL_KNOB_LANE_CTAS 4
#define IL_KNOB_BITS_IN_RECORDS 5
IL_API int il_set_test_knob(il_estimator *est, int knob, int64_t value);

/* Name of the simulation kernel the handle's next estimate call will launch
 * (the choice il_set_variant describes, resolved for the bound inputs);
 * a static string, never NULL. */
IL_API const char *il_kernel_name(const il_estimator *est);

/* Counters of the last estimate call on this handle. */
IL_API int il_get_stats(const il_estimator *est, il_stats *out);

/* Queries visiting stage s (n_s), derived from the branch bits at create;
 * out_visits is a HOST pointer to S int64. */
IL_API int il_stage_visits(const il_estimator *est, int64_t *out_visits);

/* Text for a return code; never NULL. */
IL_API const char *il_strerror(int code);

/* cudaError_t value of the last failing CUDA call in this thread (0 if none). */
IL_API int il_last_cuda_error(void);

/*
 * Measures how many warp-instructions per second the device issues on a
 * dependency-free 32-bit integer stream (every SM, every scheduler busy): the
 * denominator for the simulation kernel's instruction-issue roofline.  Runs a
 * few milliseconds on the current device.  out_* are HOST pointers.
 */
IL_API int il_measure_int_issue(void *cuda_stream, double *out_warp_inst_per_s, double *out_ms);

#ifdef __cplusplus
}
#endif
#endif /* IL_ESTIMATOR_H */
