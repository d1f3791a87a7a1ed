/*
 * hfx.h -- C ABI of the multi-SLO scheduler hot path (one GPU, sm_100a).
 *
 * The library evaluates, for a whole request table at once, the decision
 * primitives of the paper's dispatcher (Sec. 3.3.1 "Dispatching Mechanism and
 * Policy"): the latency predictor E_p / E_d, the safe token budget (Eq. 3),
 * slack and the priority key, the per-replica priority order, the budgeted
 * greedy admission ("most urgent requests that fit", dispatching step 3) and
 * the maturity-time update (dispatching step 4).  hfx_sim_run steps many
 * independent replicas through that scheduler over arrival traces and reports
 * the attainment metric (Eq. 2) and latency percentiles.
 *
 * Conventions
 *   - Every time is an int64 count of nanoseconds.  There is no floating point
 *     anywhere in the library.
 *   - "device" pointers are CUDA device pointers of the current device, each
 *     16-byte aligned; "host" pointers are ordinary host memory.
 *   - The caller owns every table, state and output buffer.  The library owns
 *     only the workspace it allocates in hfx_sched_create.
 *   - Calls are asynchronous on the stream given at create; only
 *     hfx_sched_status synchronises.
 *   - Return value: HFX_OK (0) or a negative HFX_E_* code.  Argument errors are
 *     reported before anything is launched.  Bad data found on the device (an
 *     id out of range, a length outside the domain) never traps: the row is
 *     treated as inactive and a bit is set in a sticky status word that
 *     hfx_sched_status returns.
 *   - There is no CPU fallback: without a CUDA device every entry point that
 *     would launch work returns HFX_E_CUDA.
 *
 * Domain (checked at create for the configuration, per row on the device for
 * lengths and ids; timestamps are not checked):
 *   rows            1 .. 2^27 per call (0 rows is a no-op)
 *   replicas        1 .. 65536, classes 1 .. 64
 *   prompt_len, gen 0 .. 2^24      token_cap 1 .. 2^24
 *   c0, d0 0 .. 2^40   c1, d1 0 .. 2^30   c2 0 .. 2^12   d2 0 .. 2^8
 *   ttft_slo <= 2^44, tpot_slo <= 2^34 (<= 0 means unbounded), prio 0 .. 62
 *   timestamps      -2^56 .. 2^56
 */
#ifndef HFX_H
#define HFX_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes --------------------------------------------------------- */
#define HFX_OK            0
#define HFX_E_ARG        -1   /* NULL or out-of-domain argument              */
#define HFX_E_ALIGN      -2   /* a device pointer is not 16-byte aligned     */
#define HFX_E_CAPACITY   -3   /* more rows / replicas than created for       */
#define HFX_E_CUDA       -4   /* a CUDA runtime call failed (no device, ...) */
#define HFX_E_TIMEOUT    -5   /* reserved: no kernel of this version waits on another block, so none can run out */
#define HFX_E_NOMEM      -6   /* workspace allocation failed                 */

/* bits of the sticky device status word */
#define HFX_ST_BAD_REPLICA  1u  /* replica_id outside [0, n_replicas); not raised for -1
                                   on a QUEUED row: that request is still in the global
                                   queue, bound to no instance yet                     */
#define HFX_ST_BAD_CLASS    2u  /* class_id >= n_classes                      */
#define HFX_ST_BAD_LEN      4u  /* prompt_len or gen outside [0, 2^24]        */
#define HFX_ST_TIMEOUT      8u  /* reserved (see HFX_E_TIMEOUT)               */

/* request states (column `state`) */
#define HFX_QUEUED    0
#define HFX_RUNNING   1
#define HFX_DONE      2
#define HFX_REJECTED  3

/* replica modes */
#define HFX_COLOCATED 0   /* prefill and decode share the instance            */
#define HFX_PREFILL   1   /* P-stage instance of the disaggregated mode       */
#define HFX_DECODE    2   /* D-stage instance of the disaggregated mode       */

/* budget modes */
#define HFX_BUDGET_SAFE      0  /* Eq. 3 (generalised to the quadratic E_p)   */
#define HFX_BUDGET_CAP_ONLY  1  /* capacity caps only, no SLO-derived bound   */

/* hfx_options.flags */
#define HFX_OPT_FIRST_FIT 1u    /* admission by first fit: dispatching step 3 ("the most urgent
                                   requests that fit") read as "try every request in priority
                                   order against what is left of the budget and the batch cap,
                                   take it if it fits, pass it over if not", instead of the
                                   default longest prefix of the requests that fit alone; applies
                                   to hfx_sched_step and hfx_sim_run                          */

/* hfx_sched_step flags */
#define HFX_COMMIT 1u           /* apply the admitted batch to the table      */

#define HFX_INF        INT64_MAX              /* "unbounded" budget / minimum */
#define HFX_TIME_MAX   (INT64_C(1) << 62)     /* saturation of maturity       */
#define HFX_SLACK_MAX  ((INT64_C(1) << 39) - 1)
#define HFX_SLACK_MIN  (-(INT64_C(1) << 39))
#define HFX_MAX_TOKENS (1 << 24)

typedef struct hfx_sched hfx_sched; /* opaque */

/* Latency predictor (Sec. 3.3.1: E_p of a prefill batch of t tokens, E_d of one
 * decode iteration of a running batch; the quadratic term of the cited
 * prefill model is kept as c2, the paper's linear model is c2 = 0):
 *   E_p(t)     = c0 + c1*t + c2*t*t
 *   E_d(b, kv) = d0 + d1*b + d2*kv     b = batch size, kv = sum of context
 *                                       lengths (prompt_len + gen) of the batch */
typedef struct hfx_latency_model { int64_t c0, c1, c2, d0, d1, d2; } hfx_latency_model;

/* One SLO class: TTFT and TPOT targets (Problem Definition: each request
 * carries heterogeneous SLOs) and the class priority, 0 = highest
 * (Sec. 3.3.2, "Priority as input"). */
typedef struct hfx_slo_class {
  int64_t ttft_slo_ns;  /* <= 0 : no TTFT bound */
  int64_t tpot_slo_ns;  /* <= 0 : no TPOT bound */
  int32_t prio;         /* 0 .. 62 */
  int32_t reserved;
} hfx_slo_class;

typedef struct hfx_replica_cfg {
  int32_t mode;       /* HFX_COLOCATED / HFX_PREFILL / HFX_DECODE           */
  int32_t token_cap;  /* tokens one iteration can take                       */
  int32_t batch_cap;  /* sequences in the running batch; 0 = unlimited       */
} hfx_replica_cfg;

typedef struct hfx_options {
  int32_t  budget_mode; /* HFX_BUDGET_*                                       */
  int32_t  weight_max;  /* 0: prio = class prio; >0: prio = clamp(weight_max -
                           weight, 0, 62) and the table's `weight` is read    */
  uint32_t flags;       /* HFX_OPT_* bits                                     */
  uint32_t reserved;
} hfx_options;

/* Request table, structure of arrays, all columns device pointers of n_rows
 * elements (Problem Definition: a request has an arrival timestamp, a prompt,
 * an output length and TTFT / TPOT SLOs).  Columns the call does not need may
 * be NULL: `weight` unless weight_max > 0; `output_len`, `last_token_ns`,
 * `finish_ns` unless HFX_COMMIT is given or the call is hfx_sim_run. */
typedef struct hfx_table {
  int64_t        n_rows;
  const int32_t *replica_id;     /* instance the request is bound to; -1 on a
                                    QUEUED row: still in the global queue     */
  const uint8_t *class_id;       /* index into the SLO class table            */
  uint8_t       *state;          /* HFX_QUEUED .. HFX_REJECTED (written by
                                    COMMIT and by hfx_sim_run)                */
  const int32_t *prompt_len;     /* tokens                                    */
  const int32_t *output_len;     /* true output length; read only to detect
                                    completion, never by the scheduler        */
  int32_t       *gen;            /* decode steps completed after the first
                                    token                                     */
  const int64_t *arrival_ns;
  int64_t       *first_token_ns; /* valid once RUNNING (and for QUEUED rows of
                                    a DECODE replica, which are prefilled)    */
  int64_t       *last_token_ns;
  int64_t       *finish_ns;
  const int32_t *req_id;         /* unique; final tie-break of the order      */
  const int32_t *weight;         /* priority weight, higher = served first    */
} hfx_table;

/* Per-replica clock and maturity time (Sec. 3.3.1: the earliest time an
 * instance may take new load), device arrays of n_replicas elements.  Read by
 * every step; written only by HFX_COMMIT (clock advanced, maturity replaced by
 * maturity_next).  Without HFX_COMMIT a step changes neither the table nor
 * this state. */
typedef struct hfx_replica_state {
  int64_t *now_ns;
  int64_t *maturity_ns;
} hfx_replica_state;

/* Outputs of one step.  Device pointers.  Required: order, seg_off, admit,
 * slack_ns, budget, adm_cost, adm_count, maturity_next.  Optional (NULL =
 * skip): the rest. */
typedef struct hfx_step_out {
  int64_t  *slack_ns;      /* [n_rows] remaining SLO budget, unclamped; 0 for
                              inactive rows                                   */
  int64_t  *pred_ttft_ns;  /* [n_rows] optional                               */
  int64_t  *pred_tpot_ns;  /* [n_rows] optional                               */
  uint64_t *key;           /* [n_rows] optional: replica<16> | phase<2> |
                              prio<6> | (clamp(slack)+2^39)<40>               */
  int32_t  *order;         /* [n_rows] row indices, replica-major, each
                              replica's rows ascending by (key, req_id); rows
                              with a bad replica_id follow seg_off[R], by
                              req_id                                          */
  int32_t  *seg_off;       /* [n_replicas+1] start of each replica in order   */
  uint8_t  *admit;         /* [n_rows] 1 = in the next batch (running rows and
                              admitted queued rows)                           */
  int32_t  *admitted_rows; /* [n_rows] optional: for replica r the first
                              adm_count[r] entries after seg_off[r] are the
                              newly admitted rows in priority order, the rest
                              of the replica's range is -1                    */
  int64_t  *budget;        /* [n_replicas] tokens (COLOCATED, PREFILL) or ns
                              of decode-step latency (DECODE); HFX_INF if
                              unbounded                                       */
  int64_t  *e_d_ns;        /* [n_replicas] optional: decode-iteration latency
                              of the current running batch                    */
  int32_t  *n_run;         /* [n_replicas] optional                           */
  int64_t  *sum_kv;        /* [n_replicas] optional                           */
  int64_t  *adm_cost;      /* [n_replicas] total cost of newly admitted rows  */
  int32_t  *adm_count;     /* [n_replicas] number of newly admitted rows      */
  int64_t  *maturity_next; /* [n_replicas] maturity time after this dispatch
                              (dispatching step 4); the old one if nothing
                              was admitted                                    */
} hfx_step_out;

/* Outputs of the simulator, device arrays of n_traces elements; all required
 * except now_ns. */
typedef struct hfx_sim_out {
  int32_t *iters_executed; /* iterations that did work or advanced the clock  */
  int32_t *finished;       /* rows that ended DONE                            */
  int32_t *rejected;       /* rows that ended REJECTED                        */
  int32_t *attained;       /* DONE rows that met both SLOs (numerator of
                              Eq. 2; the denominator is the trace length)     */
  int64_t *ttft_p50_ns;    /* nearest-rank percentiles; -1 if no sample       */
  int64_t *ttft_p99_ns;
  int64_t *tpot_p50_ns;
  int64_t *tpot_p99_ns;
  int64_t *now_ns;         /* optional: final clock of the trace              */
} hfx_sim_out;

/* Create a scheduler.  `model`, `classes[n_classes]`, `replicas[n_replicas]`
 * and `opts` are host pointers, copied.  `max_rows` bounds n_rows of later
 * calls and sizes the workspace (about 51 bytes per row of device memory, 67
 * for tables of more than 16384 rows, plus 8 bytes per replica and tile of the
 * table -- a tile is about 1/148 of the rows, at most 8192 -- for up to 4095
 * replicas).  `cuda_stream` is a cudaStream_t (NULL = the default stream).  Errors: HFX_E_ARG (NULL pointer, value outside the domain
 * above), HFX_E_CUDA, HFX_E_NOMEM.  On error *out is NULL. */
int hfx_sched_create(hfx_sched **out, const hfx_latency_model *model,
                     const hfx_slo_class *classes, int n_classes,
                     const hfx_replica_cfg *replicas, int n_replicas,
                     int64_t max_rows, const hfx_options *opts,
                     void *cuda_stream);

/* One scheduling iteration over the whole table (dispatching steps 2-4 of
 * Sec. 3.3.1 for every replica at once, and its P-stage / D-stage variants of
 * the paragraph "Disaggregated Mode"): per-replica aggregates of the running
 * batch, E_d, the safe budget (Eq. 3), per-row predicted TTFT / TPOT, slack and
 * key, the per-replica order, admission under the budget by a segmented prefix
 * sum, the new maturity time.  With HFX_COMMIT the admitted batch is applied:
 * admitted rows become RUNNING with their first-token time, running rows
 * advance one decode step, finished rows become DONE, oversize prompts become
 * REJECTED, and the replica clock advances by the iteration's latency (or, when
 * the replica is idle, to its next event).
 * `table`, `state`, `out` are host structs holding device pointers.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_CUDA. */
int hfx_sched_step(hfx_sched *s, const hfx_table *table,
                   const hfx_replica_state *state, const hfx_step_out *out,
                   uint32_t flags);

/* Outputs of hfx_dispatch_step; every member is a device pointer.  n = rows of
 * the table, R = replicas of the scheduler. */
typedef struct hfx_dispatch_out {
  int32_t *assign;         /* [n] instance a queued row (or, D stage, a prefilled request) is dispatched to, else -1 */
  int32_t *queue_order;    /* [n] rows of the global queue, most urgent first, then the rows of the queue of
                              prefilled requests; -1 behind them */
  int32_t *n_queue;        /* [2] length of the global queue; of the queue of prefilled requests */
  int32_t *inst_order;     /* [R] matured instances in dispatch order: colocated and P stage, then D stage; -1 behind */
  int32_t *n_mature;       /* [2] matured colocated and P-stage instances; matured D-stage instances */
  int64_t *slack_ns;       /* [n] slack of the rows of either queue, 0 elsewhere */
  int64_t *budget;         /* [R] safe budget: tokens (colocated, P stage), ns (D stage); 0 for an instance not matured */
  int64_t *e_d_ns;         /* [R] */
  int32_t *n_run;          /* [R] */
  int64_t *sum_kv;         /* [R] */
  int64_t *adm_cost;       /* [R] what was dispatched to the instance, in the unit of its budget */
  int32_t *adm_count;      /* [R] requests dispatched to the instance */
  int64_t *maturity_next;  /* [R] */
} hfx_dispatch_out;

/* The four dispatching steps of Sec. 3.3.1 (colocated mode, and the P stage of
 * the disaggregated mode) over a shared
 * global queue, for the decisions due at time now_ns: (1) the instances whose
 * maturity time (maturity_ns, device, [R]) has come take their turn once each,
 * earliest maturity first, ties in index order; (2) each gets its safe token
 * budget (Eq. 3) from the strictest TTFT in the queue as it stands when the
 * call begins and the strictest TPOT among its own in-flight requests;
 * (3) the queue -- every QUEUED row that has arrived, whatever its replica_id,
 * ordered by (priority, slack, req_id) with slack = TTFT - (now - arrival) -
 * E_p(prompt_len) -- is handed out in order: an instance takes entries from
 * where the previous one stopped while their total stays within its budget
 * and batch room, and stops at the first that does not fit (it waits at the
 * head for the next instance); an entry larger than the largest budget of
 * the call fits nowhere now and is passed over; (4) an instance that took
 * requests gets the maturity time E_p + k E_d of the per-replica step.
 * RUNNING rows count for the instance in their replica_id.  A prompt longer
 * than every instance's token_cap can never be served and is left out of the
 * queue.  The table is not changed; the caller binds the dispatched rows
 * (replica_id := assign) before the next hfx_sched_step.
 * HFX_PREFILL replicas take part the same way with the budget and maturity
 * update of their stage (the "P-stage Dispatcher": no decode batch, maturity =
 * end of the prefill batch).
 * On a scheduler with HFX_DECODE replicas the same call then runs the four
 * steps for the D stage (Sec. 3.3.1, "D-stage Migrator"): (1) the DECODE
 * instances whose maturity has come, earliest first; (2) each gets a budget in
 * time, T - E_d(its running batch), T the strictest TPOT among its in-flight
 * requests or, when it has none, in the queue of prefilled requests as the
 * call begins (unbounded when no TPOT applies or in HFX_BUDGET_CAP_ONLY mode);
 * (3) the queue of prefilled requests -- every RUNNING row on an HFX_PREFILL
 * replica whose first_token_ns has come (the end of its prefill batch; a KV
 * transfer time is not modelled here), ordered by (priority, slack, req_id)
 * with slack = first_token + (gen + 1) TPOT - now - E_d(1, prompt_len + gen)
 * -- is handed out as above, an entry costing d1 + d2 (prompt_len + gen) of
 * the budget; (4) a matured instance that then has a batch gets maturity =
 * now + E_d of the enlarged batch.  A dispatched prefilled request stays
 * RUNNING; binding it (replica_id := assign) puts it in flight on the D
 * instance.  DECODE replicas also keep their own queue (QUEUED rows bound to
 * them, e.g. by hfx_pd_migrate), which hfx_sched_step serves.
 * The scheduler may have at most 4096 replicas.  The first call allocates the call's workspace (44 bytes
 * per row of max_rows) with cudaMalloc, so it should not be made inside a
 * stream capture; hfx_sched_destroy frees it.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_NOMEM, HFX_E_CUDA. */
int hfx_dispatch_step(hfx_sched *s, const hfx_table *table, int64_t now_ns,
                      const int64_t *maturity_ns, const hfx_dispatch_out *out);

/* Binding what a dispatching call decided (Sec. 3.3.1, "dispatch them"): replica_id[i] = assign[i] for
 * every request that hfx_dispatch_step assigned (out->assign, out->adm_count as it wrote them), and the
 * clock now_ns[r] of an instance that was given requests is raised to now_ns if it was behind (an idle
 * instance's clock stands where its last iteration ended; it cannot start the requests before the call
 * that dispatched them).  replica_id must be table->replica_id (passed separately because the table
 * is otherwise read-only here); device pointers; asynchronous on the scheduler's stream.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_CUDA. */
int hfx_dispatch_bind(hfx_sched *s, const hfx_table *table, int32_t *replica_id, int64_t now_ns,
                      const hfx_dispatch_out *out, int64_t *clock_ns);

/* Hand-off from the P stage to the D stage of the disaggregated mode
 * (Sec. 3.3.1 "Disaggregated Mode": the Dispatcher serves the P instances, the
 * Migrator the D instances over the queue of prefilled requests).  With
 * hfx_sched_step + HFX_COMMIT on a scheduler that has HFX_PREFILL and
 * HFX_DECODE replicas this couples the two stages: a committed P-stage step
 * leaves an admitted request RUNNING on its P instance with first_token_ns =
 * the end of its prefill batch; this call moves it to the partner D instance
 * pair[r] (device, [n_replicas]; read for PREFILL replicas only) once its KV
 * transfer, xfer_c0_ns + xfer_c1_ns * prompt_len after the first token, has
 * ended by the partner's clock: replica_id := pair[r], state := HFX_QUEUED,
 * first_token_ns stands, so the next step of the D instance sees it in its
 * queue of prefilled requests.  A D instance with nothing in flight and
 * nothing arrived in its queue is woken: its now_ns becomes the earliest end
 * of a transfer to it.  `replica_id` must be table->replica_id (the column is
 * written, which the const in hfx_table does not allow); state and now_ns are
 * written too.  n_moved (device, [1]) may be NULL.  A partner that is not a
 * DECODE replica sets HFX_ST_BAD_REPLICA and the row stays.
 * Errors: HFX_E_ARG (NULL, negative transfer coefficients, replica_id not the
 * table's column), HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_CUDA. */
int hfx_pd_migrate(hfx_sched *s, const hfx_table *table, int32_t *replica_id, const hfx_replica_state *state,
                   const int32_t *pair, int64_t xfer_c0_ns, int64_t xfer_c1_ns, int32_t *n_moved);

/* SLO attainment over the table (Problem Definition, Eq. 2: the fraction of
 * requests that meet both their TTFT and their TPOT target; E2E = completion -
 * arrival of the same section), per SLO class and in total.  `out` is a device
 * array of (n_classes + 1) x 6 int64, row c = class c, the last row the totals:
 * requests, DONE, attained, REJECTED, sum of TTFT (first_token - arrival over
 * RUNNING and DONE requests), sum of E2E (finish - arrival over DONE ones).
 * TPOT = floor((last_token - first_token) / (output_len - 1)), 0 for output_len
 * <= 1; a target <= 0 is always met; a request that is not DONE is a miss, as
 * Eq. 2 sums over all requests.  Rows with a class or a length outside the
 * domain are left out and flagged.  Attainment = attained / requests.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_CUDA. */
int hfx_attainment(hfx_sched *s, const hfx_table *table, int64_t *out);

/* Priority-based SLO mapping (Sec. 3.3.2 "Priority-Based SLO Mapping", its five
 * steps): requests that carry only a priority p in [0, n_prio), 0 highest, get
 * their TTFT and TPOT targets from recent history.  `win` is the sliding window
 * of completed requests (device arrays of `w` records, w <= 4096, in any
 * order): priority, measured TTFT, measured TPOT, queueing delay.  With C_i the
 * window records of priority i, base = C_0 + ... + C_{p-1} and offset =
 * floor((p + 1) C_p / (n_prio + 1)); the provisional targets are the
 * (base + offset)-th smallest TTFT and TPOT of the window (ties by record
 * position; an index past the end means the last record; an empty window gives
 * the upper bounds of the priority's range).  The TTFT is then reduced by the
 * reference record's queueing delay in excess of last_queue_ns[p] (device,
 * [n_prio], in/out: it becomes the reference's delay), so within one call only
 * the first request of a priority (lowest row) sees a correction.  Both targets
 * are clamped into the priority's range; the lower bound is the strict one
 * while some higher priority has pending[i] > 0 (device, [n_prio]), the relaxed
 * one otherwise.  new_prio [n_new] and the outputs [n_new] are device arrays;
 * a request or window record whose priority is outside [0, n_prio) is ignored
 * and sets HFX_ST_BAD_CLASS (the request gets 0, 0).
 * Errors: HFX_E_ARG (n_prio outside 1..64, w < 0, NULL), HFX_E_CAPACITY
 * (w > 4096), HFX_E_ALIGN, HFX_E_CUDA. */
typedef struct hfx_slo_window {
  const int32_t *prio;      /* [w] */
  const int64_t *ttft_ns;   /* [w] */
  const int64_t *tpot_ns;   /* [w] */
  const int64_t *queue_ns;  /* [w] */
  int32_t w;
  int32_t reserved;
} hfx_slo_window;

typedef struct hfx_slo_bounds {   /* device arrays of n_prio entries */
  const int64_t *ttft_min_ns;
  const int64_t *ttft_max_ns;
  const int64_t *ttft_min_relaxed_ns;
  const int64_t *tpot_min_ns;
  const int64_t *tpot_max_ns;
  const int64_t *tpot_min_relaxed_ns;
} hfx_slo_bounds;

int hfx_slo_map(hfx_sched *s, int32_t n_prio, const hfx_slo_window *win, const hfx_slo_bounds *bounds,
                int64_t *last_queue_ns, const int32_t *pending, const int32_t *new_prio, int64_t n_new,
                int64_t *ttft_slo_ns, int64_t *tpot_slo_ns);

/* Trace-driven simulation (events are request arrivals and iteration
 * completions, Problem Definition; metrics are Eq. 2 and the TTFT / TPOT
 * definitions).  `table` holds n_traces traces back to back, trace j being
 * rows trace_off[j] .. trace_off[j+1]-1 (HOST int32 array of n_traces+1
 * offsets, copied before the call returns), sorted by arrival within a trace;
 * trace j runs on replica j of the scheduler, which must be COLOCATED.  replica_id is not read.  Every trace
 * starts at time 0 with all rows QUEUED (the incoming state, gen and time
 * columns are overwritten) and runs `iters` iterations of step + commit, or
 * until nothing is left to happen.  Written: state, gen, first_token_ns,
 * last_token_ns, finish_ns and `out`.
 * A trace of up to 10240 rows is kept in shared memory; a longer one (at most 65535 rows) works in a scratch
 * buffer in device memory (15 bytes per row for two traces per SM), which the first call that needs it
 * allocates with cudaMalloc after synchronising the stream, so such a call should not be made inside a stream
 * capture; hfx_sched_destroy frees it.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY (n_traces > n_replicas, or a
 * trace longer than 65535 rows), HFX_E_NOMEM, HFX_E_CUDA. */
int hfx_sim_run(hfx_sched *s, const hfx_table *table, const int32_t *trace_off,
                int32_t n_traces, int32_t iters, const hfx_sim_out *out);

/* Scaling indicators and threshold policy of one Scaler tick (Sec. 3.3.3 "Scaling Mechanism and
 * Policy"), evaluated per pool of instances (0 colocated, 1 prefill, 2 decode) over the whole
 * table at time now_ns:
 *   f1 = completions / arrivals inside the window (now - window_ns, now]   (used once at least
 *        min_samples arrivals were seen),
 *   f2 = mean over visible queued requests with a TTFT SLO of waiting_time / TTFT SLO, each ratio
 *        in 16.16 fixed point (floor), saturated at 2^15,
 *   f3 = used_blocks / total_blocks per instance: ceil((prompt_len + gen) / block_tokens) of every
 *        in-flight request plus ceil(prompt_len / block_tokens) of every visible queued one.
 * A QUEUED request with replica_id -1 is still in the global queue, bound to no instance: the global
 * queue feeds the colocated instances and the P stage, so it counts as an arrival and as a waiting
 * request for pools 0 and 1 and holds no KV block (any other row with a replica_id outside
 * [0, n_replicas) is skipped and sets HFX_ST_BAD_REPLICA).
 * Decision per pool: scale out (+1) if f1 < eps_out or f2 > eps_wait; else scale in (-1) if
 * f1 > eps_in and more than one instance of the pool is active (total_blocks > 0), removing the
 * active instance with the smallest f3 (lowest id on ties); else hold (0).  Thresholds are the
 * rationals num/den; the paper's defaults are window 10 s, 7/10, 11/10 and 1/4.
 * `total_blocks` [n_replicas] and the outputs are device pointers; `params` is a host pointer.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_CUDA. */
typedef struct hfx_scale_params {
  int64_t window_ns;
  int32_t block_tokens;   /* tokens per KV block, > 0 */
  int32_t min_samples;
  int32_t eps_out_num, eps_out_den, eps_in_num, eps_in_den, eps_wait_num, eps_wait_den;   /* > 0 */
} hfx_scale_params;

typedef struct hfx_scale_out {
  int64_t *counts;       /* [3][4] per pool: arrivals, completions, queued requests, sum of 16.16 ratios */
  int64_t *used_blocks;  /* [n_replicas] */
  int32_t *decision;     /* [3][2] per pool: action, instance to remove (-1 unless scaling in) */
} hfx_scale_out;

int hfx_scale_tick(hfx_sched *s, const hfx_table *table, int64_t now_ns, const int32_t *total_blocks,
                   const hfx_scale_params *params, const hfx_scale_out *out);
/* The decision of a tick alone, from counters that are already there: out->counts and out->used_blocks are
 * READ (as hfx_scale_tick writes them, or sums of what it wrote for the shards of a table: a Scaler that
 * watches instances on several GPUs adds up their counters first -- integer sums, the decision is the same
 * on every rank), out->decision is written.  window_ns and block_tokens of `params` are not used.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CUDA. */
int hfx_scale_decide(hfx_sched *s, const int32_t *total_blocks, const hfx_scale_params *params,
                     const hfx_scale_out *out);

/* Carrying out the decisions of a Scaler tick: the life of an instance and the cost of the fleet
 * (Sec. 3.3.3 for the decisions, Eq. 1 of the Problem Definition for the cost; the time to bring an
 * instance up is a constant per pool).  An instance is HFX_INST_OFF, STARTING (decided, not yet
 * serving), ACTIVE or DRAINING (chosen for removal, finishing what it holds).  At time now_ns, in
 * this order:
 *   1. every instance that is not OFF is charged for (since_ns, now_ns];
 *   2. a STARTING instance whose ready_ns has come turns ACTIVE; its clock and maturity in `state`
 *      (the arrays hfx_sched_step works on) are raised to ready_ns: it serves nothing earlier;
 *   3. a DRAINING instance with used_blocks == 0 turns OFF;
 *   4. per pool (0 colocated, 1 prefill, 2 decode) the decision {action, instance}: scale out (+1)
 *      does nothing while an instance of the pool is STARTING; else the lowest-id DRAINING instance
 *      of the pool is taken back (ACTIVE at once); else the lowest-id OFF one turns STARTING with
 *      ready_ns = now_ns + cold_start_ns[pool]; else nothing.  Scale in (-1) turns the named
 *      instance DRAINING if it is ACTIVE and of this pool, and does nothing otherwise;
 *   5. due_ns[r] = maturity of an ACTIVE instance, INT64_MAX for any other (the maturity array to
 *      give hfx_dispatch_step: only ACTIVE instances receive requests); total_blocks[r] =
 *      blocks_cap[r] if ACTIVE else 0 (the input of the next hfx_scale_tick); cost_ns[pool] = sum of
 *      billed_ns, Eq. 1 up to the factor UnitCost.
 * `decision` ([3][2]) and `used_blocks` ([n_replicas]) are what hfx_scale_tick wrote; all arrays are
 * device pointers of n_replicas entries owned by the caller (cost_ns: 3), cold_start_ns is a HOST
 * array of 3 values >= 0.  An inst_state outside 0..3 is read as OFF.  Role switching between pools
 * is not modelled.  Asynchronous on the scheduler's stream.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CUDA. */
#define HFX_INST_OFF 0
#define HFX_INST_STARTING 1
#define HFX_INST_ACTIVE 2
#define HFX_INST_DRAINING 3
typedef struct hfx_fleet {
  int32_t *inst_state;        /* read and written */
  int64_t *ready_ns;          /* written when an instance starts */
  int64_t *billed_ns;         /* read and written: time charged so far */
  int64_t *since_ns;          /* read and written: time up to which billed_ns is settled */
  int32_t *total_blocks;      /* written */
  int64_t *due_ns;            /* written */
  const int32_t *blocks_cap;  /* KV blocks of the instance when it is on */
} hfx_fleet;
int hfx_scale_apply(hfx_sched *s, int64_t now_ns, const int32_t *decision, const int64_t *used_blocks,
                    const int64_t *cold_start_ns, const hfx_fleet *fleet, const hfx_replica_state *state,
                    int64_t *cost_ns);

/* Synchronise the scheduler's stream and return the sticky status word
 * (HFX_ST_* bits) in *status_word (host pointer); the word is then cleared.
 * Returns HFX_E_CUDA if the stream reports an error, else HFX_OK. */
int hfx_sched_status(hfx_sched *s, uint32_t *status_word);

/* Number of kernels the library has launched on behalf of `s` so far. */
int64_t hfx_sched_launch_count(const hfx_sched *s);

/* Per-kernel timing (a measurement aid; the paper has no counterpart).  While
 * profiling is on, every kernel the library launches is bracketed by CUDA
 * events on the scheduler's stream.  hfx_sched_get_profile synchronises the
 * stream, adds the elapsed times of all brackets recorded since the last call
 * to *out (host pointer) and forgets them.  Kernel slots: 0 count, 2 offsets and 3 regroup (the fallback
 * front end), 4 the per-replica kernel k_replicas, 7 simulator, 8 scaler tick and hfx_scale_apply, 9 the tile
 * front end k_front, 10 the kernels of hfx_dispatch_step and hfx_dispatch_bind together, 11 those of hfx_slo_map,
 * 12 those of hfx_pd_migrate, 13 hfx_attainment (1, 5, 6 unused); hfx_kernel_name gives the name of a slot
 * (NULL past the end).  While profiling is on the per-replica kernel is not set up ahead of the front end's end
 * (the brackets sit between them), so a step takes a little longer than without. */
#define HFX_N_KERNELS 14
typedef struct hfx_profile {
  double  ms[HFX_N_KERNELS];        /* total device time per kernel slot      */
  int64_t launches[HFX_N_KERNELS];  /* launches per kernel slot               */
} hfx_profile;
int hfx_sched_set_profiling(hfx_sched *s, int on);
/* The front end of a step normally is the tile kernel k_front (one pass over the table, one block per tile;
 * slot 9), for schedulers of at most 4095 replicas whose tile matrix fits the workspace; `on` = 0 makes the
 * following steps use the fallback front end instead (three kernels with global counters, slots 0, 2, 3), which
 * is what larger schedulers always use.  Results are identical either way.  Host call, takes effect at the next
 * hfx_sched_step.  The paper has no counterpart (an execution switch). */
int hfx_sched_set_fused_front(hfx_sched *s, int on);
/* Commit horizon, for callers that advance many instances in rounds of one global clock (the events of
 * the Problem Definition happen in one global time): in the following steps with HFX_COMMIT an
 * instance whose clock now_ns[r] is past horizon_ns has nothing due yet and sits the commit out --
 * its decisions are reported as usual, its rows, clock and maturity stay as they are.  A clock equal
 * to the horizon still acts.  The default, INT64_MAX, gates nothing.  Host call, takes effect at the
 * next hfx_sched_step; the simulator is not affected. */
int hfx_sched_set_horizon(hfx_sched *s, int64_t horizon_ns);
int hfx_sched_get_profile(hfx_sched *s, hfx_profile *out);
const char *hfx_kernel_name(int slot);

void hfx_sched_destroy(hfx_sched *s);

/* Rows per replica without any allocation (the paper has no counterpart; this
 * is a service entry for callers that cannot call cudaMalloc: a process whose
 * device memory is owned entirely by a framework's allocator, a plugin inside
 * another component's memory budget, a path where an allocation's implicit
 * synchronisation is not acceptable).  It needs no hfx_sched.
 * Computes what hfx_sched_step returns in seg_off: seg_off[r] is the number of
 * rows whose replica_id is below r (the start of replica r in a replica-major
 * order) for r = 0 .. n_replicas, so seg_off[n_replicas] counts the rows with a
 * valid id; *n_bad (optional) receives the number of rows whose id is outside
 * [0, n_replicas).  `replica_id` [n_rows], `seg_off` [n_replicas+1] and `n_bad`
 * are device pointers (4-byte aligned) owned by the caller; the call is
 * asynchronous on `cuda_stream`.
 * The counters live in a fixed 16 KiB array inside the library image, held by
 * every GPU that loads the library until the process exits; hence the limit
 * n_replicas <= HFX_NOALLOC_MAX_REPLICAS (HFX_E_CAPACITY beyond it, and for
 * n_rows > 2^27).  The first call on each device looks up the array's device
 * address (make that first call outside any stream capture); no call allocates
 * or frees memory.  All calls on a device share the array and each call clears
 * what it uses, so two calls whose kernels overlap on the GPU (different
 * streams, different threads) race: serialise them.
 * Errors: HFX_E_ARG, HFX_E_ALIGN, HFX_E_CAPACITY, HFX_E_CUDA. */
#define HFX_NOALLOC_MAX_REPLICAS 4096
int hfx_count_rows_noalloc(const int32_t *replica_id, int64_t n_rows, int32_t n_replicas,
                           int32_t *seg_off, uint32_t *n_bad, void *cuda_stream);

/* Static, never NULL. */
const char *hfx_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* HFX_H */
