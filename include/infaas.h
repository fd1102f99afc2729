/* infaas.h -- C ABI of the batched model-variant selection library (CUDA, sm_100a).
 *
 * The library answers, for a batch of queries, the question the paper's dispatcher asks on
 * the arrival of every query (Section 4.1, "Case I"): which profiled model-variant of the
 * query's application should serve it, given a latency requirement and an accuracy
 * requirement (Section 3.1, Table 4).  Between batches it folds the decisions back into
 * per-variant load (Section 4.2.2) so that the next batch sees load-adjusted latencies
 * (Section 4, the list of dynamic aspects a static profile misses).
 *
 * Units: latency in microseconds (u32), accuracy in basis points (u16, 0..10000), cost in
 * integer units (u32).  All arithmetic is unsigned integer arithmetic; results are exact.
 *
 * Every function returns 0 on success or a negative INFAAS_E_* code.  No function throws,
 * aborts, or makes the GPU fault on bad *values* inside the query arrays.
 */
#ifndef INFAAS_H_
#define INFAAS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct infaas_catalog infaas_catalog; /* opaque; owns all catalog device memory */

/* One profiled model-variant (Section 2.1 lists what defines a variant; Section 3.2,
 * "Variant-Generator and Variant-Profiler", lists what is recorded for it).  The variant
 * id is the row's index in the array given to infaas_catalog_load. */
typedef struct {
  uint16_t task;     /* application / task index, < n_tasks                              */
  uint16_t arch;     /* model architecture code (carried, not used by selection)         */
  uint8_t hw;        /* hardware platform code   (carried, not used by selection)        */
  uint8_t opt;       /* framework / graph-optimiser code (carried, not used)             */
  uint16_t batch;    /* batch size the variant is optimised for, >= 1                    */
  uint32_t lat_us;   /* profiled latency of one batch, microseconds, >= 1                */
  uint16_t acc_bp;   /* accuracy, basis points, 0..10000                                 */
  uint16_t reserved; /* must be 0                                                        */
  uint32_t cost;     /* cost, integer units                                              */
  uint32_t queued;   /* queries already queued on this variant (initial load snapshot)   */
} infaas_variant;    /* 24 bytes */

/* Decision encoding (one u32 per query):
 *   0 .. 2^31-2          id of the chosen variant (it meets both requirements)
 *   bit 31 set           no variant meets the requirements; low 31 bits = nearest miss
 *   0xFFFFFFFF           invalid query: task >= n_tasks or the task has no variant      */
#define INFAAS_NO_FEASIBLE 0x80000000u
#define INFAAS_INVALID 0xFFFFFFFFu

#define INFAAS_OK 0
#define INFAAS_E_NULL (-1)      /* a required pointer is NULL                             */
#define INFAAS_E_BAD_TASK (-2)  /* a row's task >= n_tasks, or n_tasks == 0 / > 65535     */
#define INFAAS_E_BAD_BATCH (-3) /* a row's batch == 0                                     */
#define INFAAS_E_BAD_LAT (-4)   /* a row's lat_us == 0                                    */
#define INFAAS_E_BAD_ACC (-5)   /* a row's acc_bp > 10000 or reserved != 0                */
#define INFAAS_E_TOO_LARGE (-6) /* a size limit is exceeded (see each function)           */
#define INFAAS_E_CUDA (-7)      /* a CUDA call failed; infaas_last_cuda_error() has text  */
#define INFAAS_E_ALIGN (-8)     /* a device array is not 16-byte aligned                  */
#define INFAAS_E_DEVICE (-9)    /* a kernel reported an internal error (a bounded wait ran
                                   out); the catalog is unchanged by that call            */
#define INFAAS_E_BAD_STATE (-10) /* a variant state is not one of INFAAS_STATE_*          */
#define INFAAS_E_BAD_ARG (-11)   /* a scalar argument is out of range (see the function)  */

/* Limits. */
#define INFAAS_MAX_VARIANTS 0x7FFFFFFEu   /* ids must fit below bit 31                     */
#define INFAAS_MAX_TASK_VARIANTS 8192u    /* variants of one task (sorted in shared memory) */

/* Build the device catalog (Section 3.2, "Metadata Store": static profiles plus dynamic
 * load, organised for fast lookup).  Validates the rows, buckets them by task, uploads
 * them as a struct of arrays, computes each variant's load-adjusted latency
 *     pred_lat = min(2^32-1, lat_us + floor(queued * lat_us / batch))
 * and builds, per task, the list of non-dominated variants in (cost, pred_lat, -acc, id)
 * order that the selection kernel scans.
 *   rows         HOST pointer, n_variants rows, copied; the caller keeps ownership.
 *   n_variants   1 .. INFAAS_MAX_VARIANTS; at most INFAAS_MAX_TASK_VARIANTS per task.
 *   n_tasks      1 .. 65535.  Tasks without rows are allowed (their queries are INVALID).
 *   cuda_device  device ordinal; all later calls on this catalog run on it.
 *   out          receives the handle; release it with infaas_catalog_free.
 * Allocates device memory and synchronises the device.  Errors: E_NULL, E_BAD_*,
 * E_TOO_LARGE, E_CUDA.  On error *out is NULL and nothing is leaked. */
int infaas_catalog_load(const infaas_variant *rows, uint32_t n_variants, uint32_t n_tasks,
                        int cuda_device, infaas_catalog **out);

/* Decide n queries against the catalog's current load snapshot (Section 4.1, Case I; the
 * cost objective is the one of Section 2.2's worked example around Table 2).
 * For query q over the variants v of task d_task[q]:
 *     feasible(v)  <=>  pred_lat(v) <= d_slo_us[q]  and  acc_bp(v) >= d_min_acc_bp[q]
 *   - some v feasible: d_decision[q] = the feasible v smallest in (cost, pred_lat,
 *     10000-acc_bp, id), lexicographically;
 *   - none feasible (Section 4.1: suggest the closest variant): with
 *     d(v) = 10000*max(0, pred_lat-slo) + slo*max(0, min_acc-acc_bp)  (64-bit),
 *     d_decision[q] = INFAAS_NO_FEASIBLE | the v smallest in (d, cost, pred_lat,
 *     10000-acc_bp, id);
 *   - task out of range or without variants: INFAAS_INVALID.
 * All queries of one call see the same snapshot.
 *   d_task, d_slo_us, d_min_acc_bp   DEVICE arrays of n elements, 16-byte aligned, read only.
 *   d_decision                       DEVICE array of n u32, 16-byte aligned, written.
 *   cuda_stream                      a cudaStream_t (NULL = default stream).
 * Asynchronous and stream-ordered; allocates nothing.  n == 0 is a successful no-op.
 * Errors: E_NULL, E_ALIGN, E_CUDA (launch failure).  A kernel-internal error is reported by
 * the next infaas_catalog_get_state as E_DEVICE. */
int infaas_select_batch(infaas_catalog *c, const uint16_t *d_task, const uint32_t *d_slo_us,
                        const uint16_t *d_min_acc_bp, uint64_t n, uint32_t *d_decision,
                        void *cuda_stream);

/* Close a window (Section 4.2.2: load per variant from the queries it serves and its batch
 * size; Section 5: load statistics are refreshed periodically).  Tallies the window's
 * decisions per variant, advances every variant's queue by one window and rebuilds the
 * load-adjusted latencies and the per-task scan lists:
 *     count(v)   = #{q : d_decision[q] == v}          (bit 31 clear and v < n_variants)
 *     drain(v)   = min(2^32-1, floor(window_us * batch / lat_us))
 *     queued(v)  = max(0, min(2^32-1, queued + count) - drain)
 *     served_total(v) += count(v)
 * Decisions with bit 31 set add no load; INFAAS_INVALID and ids >= n_variants are counted
 * as invalid and otherwise ignored.
 *   d_decision   DEVICE array of n u32 (16-byte aligned), read only; n <= 2^32-1.
 * Asynchronous, stream-ordered, allocates nothing; must be ordered (same stream or an
 * event) before the next infaas_select_batch that should see the new load.
 * Errors: E_NULL, E_ALIGN, E_TOO_LARGE, E_CUDA. */
int infaas_load_update(infaas_catalog *c, const uint32_t *d_decision, uint64_t n,
                       uint32_t window_us, void *cuda_stream);

/* The two halves of infaas_load_update, for windows whose queries are shared out over several
 * GPUs (Section 4.2.2 and Section 5: every worker's monitoring daemon reports the load it saw;
 * the load of a variant is the sum over the workers).  Each GPU holds the same catalog and
 * decides its share of the window; then
 *     infaas_tally           adds the share's decisions to the pending per-variant counts,
 *     infaas_pending_counts  copies the pending counts out (set = 0) -- sum them over the
 *                            GPUs, e.g. with an all-reduce -- and back in (set = 1),
 *     infaas_advance         applies the queue recursion with the pending counts, clears
 *                            them and rebuilds the scan lists, as infaas_load_update does.
 * infaas_load_update(c, d, n, w, s) equals infaas_tally(c, d, n, s); infaas_advance(c, w, s).
 * With the same summed counts every GPU reaches the same load state.  The counters of
 * infaas_catalog_get_state stay local to each GPU (they count the decisions it tallied).
 *   d_decision   as for infaas_load_update.
 *   d_counts     DEVICE array of n_variants u32 indexed by variant id, 16-byte aligned;
 *                written (set = 0) or read (set = 1).
 * Asynchronous, stream-ordered, allocate nothing.  Errors: E_NULL, E_ALIGN, E_TOO_LARGE, E_CUDA. */
int infaas_tally(infaas_catalog *c, const uint32_t *d_decision, uint64_t n, void *cuda_stream);

/* infaas_select_batch followed by infaas_load_update over the same n queries, as one call
 * (the arrival of a window of queries and the refresh of the load that follows it:
 * Section 4.1 "Case I", then Section 4.2.2 / Section 5).  Same arguments, layouts, results and
 * errors as the two calls; n <= 2^32-1.  For windows below 2^18 queries the selection kernel
 * counts its own decisions, which saves the pass over d_decision and one kernel launch. */
int infaas_select_update(infaas_catalog *c, const uint16_t *d_task, const uint32_t *d_slo_us,
                         const uint16_t *d_min_acc_bp, uint64_t n, uint32_t *d_decision,
                         uint32_t window_us, void *cuda_stream);
int infaas_pending_counts(infaas_catalog *c, uint32_t *d_counts, int set, void *cuda_stream);
int infaas_advance(infaas_catalog *c, uint32_t window_us, void *cuda_stream);

/* Life cycle of a variant (Section 4, "State machine for the lifecycle of model-variants"):
 * Inactive = not loaded, Active = loaded and below its peak throughput, Overloaded = serving
 * at its peak throughput, Interfered = slower than profiled because of co-located work. */
#define INFAAS_STATE_INACTIVE 0
#define INFAAS_STATE_ACTIVE 1
#define INFAAS_STATE_OVERLOADED 2
#define INFAAS_STATE_INTERFERED 3

/* Give every variant a state and a loading latency, and switch the catalog to state-aware
 * selection (Section 4.1, Case I and "Mitigating performance degradation").  From then on
 * infaas_select_batch answers a query in this order:
 *   1. among the Active variants of its task that meet both requirements, the one with the
 *      smallest (cost, pred_lat, 10000-acc, id) -- Active variants carry no loading latency;
 *   2. otherwise, among the Inactive variants with  eff = min(2^32-1, pred_lat + load_lat)
 *      <= slo and acc >= min_acc, the one with the lowest combined loading and inference
 *      latency: smallest (eff, 10000-acc, id);
 *   3. otherwise bit 31 set and the nearest miss over the Active and Inactive variants:
 *      smallest d = 10000*max(0,L-slo) + slo*max(0,min_acc-acc) with L = pred_lat (Active) or
 *      eff (Inactive); equal d goes to an Active variant first, then by the order of 1. / 2.
 * Overloaded and Interfered variants are neither chosen nor suggested; a task without an
 * Active or Inactive variant answers INFAAS_INVALID.  And infaas_load_update / infaas_advance,
 * after the queue recursion, move the states with the load:
 *     Inactive and count(v) > 0                      -> Active   (it was loaded to serve them)
 *     then, Active or Overloaded: queued(v) > 0      -> Overloaded, else Active
 *     Interfered is left alone (set it from outside with this call).
 * A catalog on which this was never called behaves as if every variant were Active and
 * never changes a state.
 *   h_state        HOST, n_variants bytes indexed by variant id, each an INFAAS_STATE_* value.
 *   h_load_lat_us  HOST, n_variants u32 indexed by variant id (time to load the variant,
 *                  microseconds), or NULL for all zero.  Both are copied.
 * Rebuilds the scan lists; synchronises cuda_stream.  Errors: E_NULL, E_BAD_STATE (nothing is
 * changed), E_CUDA. */
int infaas_catalog_set_states(infaas_catalog *c, const uint8_t *h_state,
                              const uint32_t *h_load_lat_us, void *cuda_stream);

/* Copy the variants' states to HOST: h_state[n_variants] indexed by variant id (all Active
 * if infaas_catalog_set_states was never called).  Synchronises cuda_stream. */
int infaas_catalog_get_states(infaas_catalog *c, uint8_t *h_state, void *cuda_stream);

/* Model-Autoscaler, scaling-up step (Section 4.2.2, "A Greedy Heuristic"; cost function and
 * constraints (1), (2), (4) of Section 4.2.1).  For every task it compares the saturation
 * throughput of the running variants with the load the window's tallies show and, when the
 * headroom is below the slack threshold, picks the cheaper of replicating the running variant
 * and adding a faster variant of the same architecture:
 *     Q(v)  = floor(10^9 * batch / lat_us)                   milli-queries/s, profiled
 *     L     = floor(10^9 * min(2^32-1, sum_v count(v)) / window_us)
 *     cap   = sum over variants with instances > 0 of instances * Q      (saturating, 64 bit)
 *     need  = ceil(L * slack_pct / 100)                      (saturating)
 *   cap >= need: no action, variant = INFAAS_AUTOSCALE_NONE, delta = 0.  Otherwise, with
 *   deficit = need - cap and r = the running variant with the largest count (ties: lower id;
 *   none if nothing runs), the candidates are r itself (replicate) and every v != r of r's
 *   architecture with Q(v) > Q(r) (upgrade; if nothing runs: every v), each only if
 *   lat_us(v) <= the task's SLO and Q(v) > 0, with delta = ceil(deficit / Q(v)) <= 2^32-1
 *   instances added.  The smallest  cost * delta * (10^9 + lambda_milli * load_lat_us)  wins
 *   (the paper's C (delta + lambda T_load delta) in units of 10^-9), replication first on
 *   equal cost, then the lower id.  No candidate: variant = INFAAS_AUTOSCALE_ESCALATE (the
 *   case the paper hands to the VM-level autoscaler), delta = 0.
 * count(v) are the pending tallies: call this after infaas_tally and before infaas_advance
 * (infaas_load_update does both at once and leaves nothing pending).  The loading latencies are
 * those of infaas_catalog_set_states (zero if never set).  The actions are only reported; apply
 * them with infaas_autoscale_config.
 *   infaas_autoscale_config: h_instances HOST n_variants u32 by variant id (running instances
 *     N of each variant), h_task_slo_us HOST n_tasks u32 (each application's SLO); copied;
 *     synchronises cuda_stream.  Errors: E_NULL, E_CUDA.
 *   infaas_autoscale_step: window_us >= 1 (else E_BAD_ARG); slack_pct = the slack threshold in
 *     percent (the paper uses 1.05 = 105); lambda_milli = the weight lambda in 1/1000 per second;
 *     d_variant, d_delta DEVICE, n_tasks u32 each, overwritten.  Asynchronous, stream-ordered,
 *     allocates nothing.  Errors: E_NULL, E_BAD_ARG (also: config never called), E_CUDA. */
#define INFAAS_AUTOSCALE_NONE 0xFFFFFFFFu
#define INFAAS_AUTOSCALE_ESCALATE 0xFFFFFFFEu
int infaas_autoscale_config(infaas_catalog *c, const uint32_t *h_instances,
                            const uint32_t *h_task_slo_us, void *cuda_stream);
int infaas_autoscale_step(infaas_catalog *c, uint32_t window_us, uint32_t slack_pct,
                          uint32_t lambda_milli, uint32_t *d_variant, uint32_t *d_delta,
                          void *cuda_stream);

/* Worker choice (Section 4.1, Case I; Section 5: an instance is a {variant, worker} pair).  A
 * decided query goes to the least-loaded worker that runs an instance of the chosen variant;
 * if the variant is not loaded anywhere, to the worker with the lowest utilisation among those
 * whose hardware is the variant's (the row's hw code).  All queries of a call see one snapshot
 * of the two tables:
 *     worker(q) = the worker of the instance of v = d_decision[q] with the smallest
 *                 (load, worker);  if v has no instance, the w with the smallest (util, w) among
 *                 worker_hw[w] == hw(v);  if there is none, or the decision has bit 31 set or is
 *                 >= n_variants, 0xFFFFFFFF.
 *   infaas_workers_config: HOST arrays, copied: the instance table h_inst_variant /
 *     h_inst_worker / h_inst_load (n_inst entries each; rows whose variant or worker is out of
 *     range are ignored; may be NULL if n_inst == 0) and the worker table h_worker_hw (u8) /
 *     h_worker_util (n_workers entries; worker ids are the indices).  Replaces the previous
 *     tables (the paper's monitoring daemons refresh them every 2 s).  Allocates and frees a
 *     temporary device buffer; synchronises cuda_stream.  Errors: E_NULL, E_CUDA.
 *   infaas_assign_workers: d_decision DEVICE n u32 (read), d_worker DEVICE n u32 (written),
 *     both 16-byte aligned; asynchronous, stream-ordered, allocates nothing.  Errors: E_NULL,
 *     E_ALIGN, E_BAD_ARG (infaas_workers_config never called), E_CUDA. */
int infaas_workers_config(infaas_catalog *c, const uint32_t *h_inst_variant,
                          const uint32_t *h_inst_worker, const uint32_t *h_inst_load,
                          uint32_t n_inst, const uint8_t *h_worker_hw,
                          const uint32_t *h_worker_util, uint32_t n_workers, void *cuda_stream);
int infaas_assign_workers(infaas_catalog *c, const uint32_t *d_decision, uint64_t n,
                          uint32_t *d_worker, void *cuda_stream);

/* Copy the load state to HOST arrays (any of the four may be NULL to skip it):
 *   h_queued[n_variants], h_pred_lat_us[n_variants], h_served_total[n_variants] indexed by
 *   variant id; h_counters[3] = feasible decisions tallied, NO_FEASIBLE decisions seen,
 *   invalid decisions seen, summed over all infaas_load_update calls.
 * Synchronises cuda_stream.  Returns E_DEVICE if any kernel of this catalog recorded an
 * internal error since the last call. */
int infaas_catalog_get_state(infaas_catalog *c, uint32_t *h_queued, uint32_t *h_pred_lat_us,
                             uint64_t *h_served_total, uint64_t h_counters[3],
                             void *cuda_stream);

/* Copy one task's scan list to HOST: the ids of its non-dominated variants in scan order
 * (state-aware catalogs: the Active list, then the Inactive list).
 * h_ids may be NULL to query the length only; at most `cap` ids are written.
 * *h_len receives the list's length.  Synchronises cuda_stream.  For inspection/tests. */
int infaas_catalog_get_frontier(infaas_catalog *c, uint32_t task, uint32_t *h_ids,
                                uint32_t cap, uint32_t *h_len, void *cuda_stream);

/* Sizes of the structures built for the current load state, for reporting (HOST array):
 *   h_info[0] bytes of the packed lookup image the selection kernel reads
 *   h_info[1] longest per-task scan list        h_info[2] sum of the list lengths
 *   h_info[3] tasks whose list has no rank index (longer than the index supports)
 *   h_info[4] shared memory (bytes) the next infaas_select_batch reserves for the image;
 *             if h_info[0] is larger the kernel reads the image from global memory
 *   h_info[5..7] reserved (0).
 * Synchronises cuda_stream. */
int infaas_catalog_get_info(infaas_catalog *c, uint32_t h_info[8], void *cuda_stream);

/* (No counterpart in the paper: an addition for callers that cannot allocate.)
 * Per-variant tallies of a decision array, as the first step of infaas_load_update computes
 * them, for callers that must not trigger a device allocation: a serving process that has
 * handed all free device memory to its own pool (a cudaMalloc there fails), or a dispatch
 * loop that cannot afford the device-wide stall an allocation causes.  It needs no catalog
 * handle and calls no cudaMalloc / cudaFree nor any allocating routine: its scratch (the
 * counters it accumulates into) is a fixed array inside the library's device image, which
 * every GPU that loads the library holds until the process exits (256 KB + 32 B).
 *     d_count[v]    = #{q : d_decision[q] == v}      for v < n_variants (bit 31 clear)
 *     d_counters[3] = decisions tallied, decisions with bit 31 set (not INFAAS_INVALID),
 *                     invalid decisions (INFAAS_INVALID or an id >= n_variants)
 *   d_decision   DEVICE, n u32, 16-byte aligned, read only; n <= 2^32-1.
 *   n_variants   1 .. INFAAS_STATIC_MAX_VARIANTS, else INFAAS_E_TOO_LARGE.
 *   d_count      DEVICE, n_variants u32, overwritten.   d_counters  DEVICE, 3 u64, overwritten.
 *   cuda_device  device the arrays live on (0..63).      cuda_stream a cudaStream_t on it.
 * Asynchronous and stream-ordered.  The first call on each device looks up the array's
 * device address (a set-up step): make that first call outside any stream capture.  All
 * calls on a device share the one array and each call clears what it uses before counting,
 * so two calls whose work overlaps on the GPU (different streams, no ordering) race and give
 * wrong counts; order them.  Errors: E_NULL, E_ALIGN, E_TOO_LARGE, E_CUDA. */
#define INFAAS_STATIC_MAX_VARIANTS 65536u
int infaas_tally_static(const uint32_t *d_decision, uint64_t n, uint32_t n_variants,
                        uint32_t *d_count, uint64_t *d_counters, int cuda_device,
                        void *cuda_stream);

/* Measurement aid, not a step of the path: runs a kernel of independent 32-bit integer
 * add / xor / compare / conditional-add chains on every multiprocessor of `cuda_device`
 * (`iters` steps per chain, 1 .. 2^24) and reports in *h_lane_ops (HOST) how many
 * lane-operations the launch executes.  Timed by the caller with CUDA events on
 * `cuda_stream`, it gives the integer-pipe rate against which the feasibility scan of
 * Section 4.1's per-query search (2 compares and 1 AND per variant examined) is put.
 * d_sink: DEVICE, one u32, never written in practice.  Asynchronous, allocates nothing.
 * Errors: E_NULL, E_BAD_ARG, E_CUDA. */
int infaas_intpipe_probe(uint32_t iters, uint32_t *d_sink, int cuda_device, uint64_t *h_lane_ops,
                         void *cuda_stream);

/* Release the catalog and its device memory.  NULL is allowed. */
void infaas_catalog_free(infaas_catalog *c);

/* Text for an INFAAS_E_* code; never NULL. */
const char *infaas_strerror(int code);

/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char *infaas_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* INFAAS_H_ */
