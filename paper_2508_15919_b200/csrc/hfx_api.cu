// C ABI of the scheduler library: argument checking, workspace, launch sequencing.
#include <new>
#include <string.h>

#include "hfx_internal.cuh"

int hfx_front_configure();
int hfx_segment_configure();
int hfx_sim_configure();
int hfx_dispatch_configure();
int hfx_slomap_configure();
int hfx_launch_sim_kernel(hfx_sched *s, const hfx_table *t, const int32_t *d_trace_off, int32_t n_traces,
                          int32_t max_trace_rows, int32_t iters, const hfx_sim_out *o, uint32_t *d_work_counter);

#define SIM_MAX_ROWS 65535      // rows of a trace are numbered with 16 bits inside the simulator

struct hfx_sched_host {
  hfx_sched core;
  hfx_replica_cfg *h_cfg;
  int32_t *d_trace_off;     // [R+1]
  uint32_t *d_work_counter;
};

static inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

extern "C" const char *hfx_strerror(int code) {
  switch (code) {
    case HFX_OK: return "ok";
    case HFX_E_ARG: return "invalid argument";
    case HFX_E_ALIGN: return "device pointer not 16-byte aligned";
    case HFX_E_CAPACITY: return "more rows, replicas or trace rows than the scheduler was created for";
    case HFX_E_CUDA: return "CUDA runtime error (no device, launch or copy failure)";
    case HFX_E_TIMEOUT: return "a bounded device-side wait ran out";
    case HFX_E_NOMEM: return "device workspace allocation failed";
    default: return "unknown error";
  }
}

static bool in_range(int64_t v, int64_t lo, int64_t hi) { return v >= lo && v <= hi; }

extern "C" int hfx_sched_create(hfx_sched **out, const hfx_latency_model *model, const hfx_slo_class *classes,
                                int n_classes, const hfx_replica_cfg *replicas, int n_replicas, int64_t max_rows,
                                const hfx_options *opts, void *cuda_stream) {
  if (!out) return HFX_E_ARG;
  *out = nullptr;
  if (!model || !classes || !replicas || !opts) return HFX_E_ARG;
  if (n_classes < 1 || n_classes > HFX_MAX_CLASSES || n_replicas < 1 || n_replicas > HFX_MAX_REPLICAS) return HFX_E_ARG;
  if (max_rows < 1 || max_rows > HFX_MAX_ROWS) return HFX_E_ARG;
  if (!in_range(model->c0, 0, INT64_C(1) << 40) || !in_range(model->d0, 0, INT64_C(1) << 40) ||
      !in_range(model->c1, 0, INT64_C(1) << 30) || !in_range(model->d1, 0, INT64_C(1) << 30) ||
      !in_range(model->c2, 0, INT64_C(1) << 12) || !in_range(model->d2, 0, INT64_C(1) << 8))
    return HFX_E_ARG;
  for (int c = 0; c < n_classes; c++) {
    if (classes[c].ttft_slo_ns > (INT64_C(1) << 44) || classes[c].tpot_slo_ns > (INT64_C(1) << 34)) return HFX_E_ARG;
    if (classes[c].prio < 0 || classes[c].prio > 62) return HFX_E_ARG;
  }
  for (int r = 0; r < n_replicas; r++) {
    if (replicas[r].mode < HFX_COLOCATED || replicas[r].mode > HFX_DECODE) return HFX_E_ARG;
    if (replicas[r].token_cap < 1 || replicas[r].token_cap > HFX_MAX_TOKENS || replicas[r].batch_cap < 0) return HFX_E_ARG;
  }
  if (opts->budget_mode != HFX_BUDGET_SAFE && opts->budget_mode != HFX_BUDGET_CAP_ONLY) return HFX_E_ARG;
  if (opts->weight_max < 0 || opts->weight_max > (1 << 20) || (opts->flags & ~HFX_OPT_FIRST_FIT) != 0) return HFX_E_ARG;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return HFX_E_CUDA; }
  int n_sm = 0;
  if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1) {
    cudaGetLastError();
    return HFX_E_CUDA;
  }
  if (hfx_front_configure() != HFX_OK || hfx_segment_configure() != HFX_OK || hfx_sim_configure() != HFX_OK || hfx_dispatch_configure() != HFX_OK || hfx_slomap_configure() != HFX_OK) { cudaGetLastError(); return HFX_E_CUDA; }

  hfx_sched_host *h = new (std::nothrow) hfx_sched_host();
  if (!h) return HFX_E_NOMEM;
  memset(h, 0, sizeof(*h));
  hfx_sched *s = &h->core;
  s->p.c0 = model->c0; s->p.c1 = model->c1; s->p.c2 = model->c2;
  s->p.d0 = model->d0; s->p.d1 = model->d1; s->p.d2 = model->d2;
  for (int c = 0; c < HFX_MAX_CLASSES; c++) {
    s->p.ttft[c] = c < n_classes ? classes[c].ttft_slo_ns : 0;
    s->p.tpot[c] = c < n_classes ? classes[c].tpot_slo_ns : 0;
    s->p.prio[c] = c < n_classes ? (uint8_t)classes[c].prio : 63;
  }
  s->p.n_classes = n_classes; s->p.n_replicas = n_replicas;
  s->p.budget_mode = opts->budget_mode; s->p.weight_max = opts->weight_max;
  s->p.first_fit = (opts->flags & HFX_OPT_FIRST_FIT) ? 1 : 0;
  s->opts = *opts; s->max_rows = max_rows; s->n_sm = n_sm;
  s->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  s->launches = 0;
  s->profiling = 0;
  s->brackets = new (std::nothrow) std::vector<HfxBracket>();

  const size_t R2 = (size_t)n_replicas + 2;
  bool ok = true;
  ok = ok && cudaMalloc(&s->d_cfg, sizeof(hfx_replica_cfg) * n_replicas) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_status, 256) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_mode, (size_t)n_replicas + 16) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_seg_count, sizeof(uint32_t) * R2) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_seg_begin, sizeof(uint32_t) * R2) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_cursor, sizeof(uint32_t) * 2 * R2) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_act_count, sizeof(uint32_t) * R2) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_rowflag, (size_t)max_rows + 16) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_flags, 256) == cudaSuccess;
  {
    // the tile front end: slabs for every tile of the largest table, one matrix row per tile
    int32_t tile_rows = 0, n_tiles = 0;
    hfx_front_shape(s, max_rows, &tile_rows, &n_tiles);
    if (n_tiles < n_sm + 1) n_tiles = n_sm + 1;      // smaller tables have lower tiles, about one per SM
    s->tiles_max = 0;
    if (n_replicas <= HFX_TILE_REPLICAS_MAX && (int64_t)n_tiles * (n_replicas + 1) <= HFX_TILE_MATRIX_MAX) {
      const size_t slots = (size_t)max_rows + HFX_TILE_ROWS_MAX;
      ok = ok && cudaMalloc(&s->d_M, sizeof(uint2) * (size_t)n_tiles * ((size_t)n_replicas + 1)) == cudaSuccess;
      ok = ok && cudaMalloc(&s->d_slab_rec, sizeof(uint4) * slots) == cudaSuccess;
      ok = ok && cudaMalloc(&s->d_slab_idx, sizeof(uint16_t) * slots) == cudaSuccess;
      ok = ok && cudaMalloc(&s->d_tot, sizeof(unsigned long long) * 2 * R2) == cudaSuccess;
      ok = ok && cudaMemset(s->d_tot, 0, sizeof(unsigned long long) * 2 * R2) == cudaSuccess;
      s->tiles_max = n_tiles;
    }
  }
  ok = ok && cudaMalloc(&s->d_rec, sizeof(HfxRec) * (size_t)max_rows) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_slo, hfx_slomap_workspace_bytes()) == cudaSuccess;
  ok = ok && cudaMalloc(&s->d_pd, hfx_pd_workspace_bytes(n_replicas)) == cudaSuccess;
  s->horizon = INT64_MAX;
  s->front_enabled = 1; s->tot_parity = 0;
  ok = ok && cudaMalloc(&h->d_trace_off, sizeof(int32_t) * R2) == cudaSuccess;
  ok = ok && cudaMalloc(&h->d_work_counter, 256) == cudaSuccess;
  if (ok && max_rows > 16384) {   // scratch of the global sort: only tables that can hold an oversize segment
    ok = ok && cudaMalloc(&s->d_big_hi, sizeof(uint64_t) * (size_t)max_rows) == cudaSuccess;
    ok = ok && cudaMalloc(&s->d_big_lo, sizeof(uint32_t) * 2 * (size_t)max_rows) == cudaSuccess;
  }
  h->h_cfg = new (std::nothrow) hfx_replica_cfg[n_replicas];
  ok = ok && h->h_cfg != nullptr;
  if (ok) {
    memcpy(h->h_cfg, replicas, sizeof(hfx_replica_cfg) * n_replicas);
    ok = ok && cudaMemcpy(s->d_cfg, replicas, sizeof(hfx_replica_cfg) * n_replicas, cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(s->d_status, 0, 256) == cudaSuccess;
    {
      std::vector<uint8_t> modes((size_t)n_replicas);
      for (int r = 0; r < n_replicas; r++) modes[r] = (uint8_t)replicas[r].mode;
      ok = ok && cudaMemcpy(s->d_mode, modes.data(), (size_t)n_replicas, cudaMemcpyHostToDevice) == cudaSuccess;
    }
    const uint32_t init_flags[8] = {0u, 0u, 0u, 0u, 1u, 1u, 0u, 0u};
    ok = ok && cudaMemcpy(s->d_flags, init_flags, sizeof(init_flags), cudaMemcpyHostToDevice) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    hfx_sched_destroy(s);
    return HFX_E_NOMEM;
  }
  *out = s;
  return HFX_OK;
}

extern "C" void hfx_sched_destroy(hfx_sched *s) {
  if (!s) return;
  hfx_sched_host *h = reinterpret_cast<hfx_sched_host *>(s);
  cudaStreamSynchronize(s->stream);
  hfx_dispatch_release(s);
  hfx_sim_release(s);
  cudaFree(s->d_cfg); cudaFree(s->d_mode); cudaFree(s->d_status); cudaFree(s->d_seg_count); cudaFree(s->d_seg_begin);
  cudaFree(s->d_cursor); cudaFree(s->d_flags); cudaFree(s->d_rec);
  cudaFree(s->d_act_count); cudaFree(s->d_rowflag);
  cudaFree(s->d_M); cudaFree(s->d_slab_rec); cudaFree(s->d_slab_idx); cudaFree(s->d_tot);
  cudaFree(s->d_big_hi); cudaFree(s->d_big_lo); cudaFree(s->d_slo); cudaFree(s->d_pd);
  cudaFree(h->d_trace_off); cudaFree(h->d_work_counter);
  cudaGetLastError();
  if (s->brackets) {
    for (HfxBracket &b : *s->brackets) { cudaEventDestroy(b.a); cudaEventDestroy(b.b); }
    delete s->brackets;
  }
  delete[] h->h_cfg;
  delete h;
}

extern "C" int hfx_sched_step(hfx_sched *s, const hfx_table *t, const hfx_replica_state *st, const hfx_step_out *o,
                              uint32_t flags) {
  if (!s || !t || !st || !o) return HFX_E_ARG;
  if (flags & ~HFX_COMMIT) return HFX_E_ARG;
  if (t->n_rows < 0) return HFX_E_ARG;
  if (t->n_rows > s->max_rows) return HFX_E_CAPACITY;
  const bool commit = (flags & HFX_COMMIT) != 0;
  const void *need_rep[] = {st->now_ns, st->maturity_ns, o->seg_off, o->budget, o->adm_cost, o->adm_count,
                            o->maturity_next};
  for (const void *p : need_rep) if (!p) return HFX_E_ARG;
  if (t->n_rows > 0) {   // per-row buffers may be NULL for an empty table
    const void *need_row[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->gen, t->arrival_ns,
                              t->first_token_ns, t->req_id, o->slack_ns, o->order, o->admit};
    for (const void *p : need_row) if (!p) return HFX_E_ARG;
    if (s->p.weight_max > 0 && !t->weight) return HFX_E_ARG;
    if (commit && (!t->output_len || !t->last_token_ns || !t->finish_ns)) return HFX_E_ARG;
  }
  const void *all[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->output_len, t->gen, t->arrival_ns,
                       t->first_token_ns, t->last_token_ns, t->finish_ns, t->req_id, t->weight, st->now_ns,
                       st->maturity_ns, o->slack_ns, o->pred_ttft_ns, o->pred_tpot_ns, o->key, o->order, o->seg_off,
                       o->admit, o->admitted_rows, o->budget, o->e_d_ns, o->n_run, o->sum_kv, o->adm_cost,
                       o->adm_count, o->maturity_next};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  return hfx_launch_step(s, t, st, o, flags);
}

extern "C" int hfx_dispatch_step(hfx_sched *s, const hfx_table *t, int64_t now_ns, const int64_t *maturity_ns,
                                 const hfx_dispatch_out *o) {
  if (!s || !t || !maturity_ns || !o) return HFX_E_ARG;
  hfx_sched_host *h = reinterpret_cast<hfx_sched_host *>(s);
  if (t->n_rows < 0) return HFX_E_ARG;
  if (t->n_rows > s->max_rows || s->p.n_replicas > 4096) return HFX_E_CAPACITY;
  const void *need_rep[] = {o->n_queue, o->inst_order, o->n_mature, o->budget, o->e_d_ns, o->n_run, o->sum_kv, o->adm_cost,
                            o->adm_count, o->maturity_next};
  for (const void *p : need_rep) if (!p) return HFX_E_ARG;
  if (t->n_rows > 0) {
    const void *need_row[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->gen, t->arrival_ns, t->req_id,
                              o->assign, o->queue_order, o->slack_ns};
    for (const void *p : need_row) if (!p) return HFX_E_ARG;
    if (s->p.weight_max > 0 && !t->weight) return HFX_E_ARG;
  }
  const void *all[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->gen, t->arrival_ns, t->req_id, t->weight,
                       maturity_ns, o->assign, o->queue_order, o->n_queue, o->inst_order, o->n_mature, o->slack_ns, o->budget,
                       o->e_d_ns, o->n_run, o->sum_kv, o->adm_cost, o->adm_count, o->maturity_next};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  int32_t cap_max = 0;
  bool d_stage = false;      // the scheduler has D-stage instances: the Migrator's stage runs too
  for (int r = 0; r < s->p.n_replicas; r++) {
    if (h->h_cfg[r].mode != HFX_DECODE && h->h_cfg[r].token_cap > cap_max) cap_max = h->h_cfg[r].token_cap;
    d_stage = d_stage || h->h_cfg[r].mode == HFX_DECODE;
  }
  if (d_stage && t->n_rows > 0 && !t->first_token_ns) return HFX_E_ARG;
  if (misaligned(t->first_token_ns)) return HFX_E_ALIGN;
  return hfx_launch_dispatch(s, t, now_ns, maturity_ns, o, cap_max, d_stage);
}

extern "C" int hfx_pd_migrate(hfx_sched *s, const hfx_table *t, int32_t *replica_id, const hfx_replica_state *st,
                              const int32_t *pair, int64_t xfer_c0_ns, int64_t xfer_c1_ns, int32_t *n_moved) {
  if (!s || !t || !st || !st->now_ns || !pair) return HFX_E_ARG;
  if (t->n_rows < 0 || xfer_c0_ns < 0 || xfer_c1_ns < 0 || xfer_c0_ns > (INT64_C(1) << 40) || xfer_c1_ns > (INT64_C(1) << 30)) return HFX_E_ARG;
  if (t->n_rows > s->max_rows) return HFX_E_CAPACITY;
  if (t->n_rows > 0) {
    const void *need[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->gen, t->arrival_ns, t->first_token_ns};
    for (const void *p : need) if (!p) return HFX_E_ARG;
    if (replica_id != t->replica_id) return HFX_E_ARG;
  }
  const void *all[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->gen, t->arrival_ns, t->first_token_ns, st->now_ns,
                       pair, n_moved};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  return hfx_launch_pd_migrate(s, t, replica_id, st->now_ns, pair, xfer_c0_ns, xfer_c1_ns, n_moved);
}

extern "C" int hfx_attainment(hfx_sched *s, const hfx_table *t, int64_t *out) {
  if (!s || !t || !out || t->n_rows < 0) return HFX_E_ARG;
  if (t->n_rows > s->max_rows) return HFX_E_CAPACITY;
  if (t->n_rows > 0) {
    const void *need[] = {t->class_id, t->state, t->prompt_len, t->output_len, t->gen, t->arrival_ns, t->first_token_ns,
                          t->last_token_ns, t->finish_ns};
    for (const void *p : need) if (!p) return HFX_E_ARG;
  }
  const void *all[] = {t->class_id, t->state, t->prompt_len, t->output_len, t->gen, t->arrival_ns, t->first_token_ns,
                       t->last_token_ns, t->finish_ns, out};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  return hfx_launch_attainment(s, t, out);
}

extern "C" int hfx_slo_map(hfx_sched *s, int32_t n_prio, const hfx_slo_window *win, const hfx_slo_bounds *b,
                           int64_t *last_queue_ns, const int32_t *pending, const int32_t *new_prio, int64_t n_new,
                           int64_t *ttft_slo_ns, int64_t *tpot_slo_ns) {
  if (!s || !win || !b || !last_queue_ns || !pending) return HFX_E_ARG;
  if (n_prio < 1 || n_prio > HFX_MAX_CLASSES || win->w < 0 || n_new < 0) return HFX_E_ARG;
  if (win->w > 4096) return HFX_E_CAPACITY;
  if (win->w > 0 && (!win->prio || !win->ttft_ns || !win->tpot_ns || !win->queue_ns)) return HFX_E_ARG;
  if (n_new > 0 && (!new_prio || !ttft_slo_ns || !tpot_slo_ns)) return HFX_E_ARG;
  const void *bp[] = {b->ttft_min_ns, b->ttft_max_ns, b->ttft_min_relaxed_ns, b->tpot_min_ns, b->tpot_max_ns, b->tpot_min_relaxed_ns};
  for (const void *p : bp) if (!p) return HFX_E_ARG;
  const void *all[] = {win->prio, win->ttft_ns, win->tpot_ns, win->queue_ns, b->ttft_min_ns, b->ttft_max_ns, b->ttft_min_relaxed_ns,
                       b->tpot_min_ns, b->tpot_max_ns, b->tpot_min_relaxed_ns, last_queue_ns, pending, new_prio, ttft_slo_ns,
                       tpot_slo_ns};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  return hfx_launch_slo_map(s, n_prio, win, b, last_queue_ns, pending, new_prio, n_new, ttft_slo_ns, tpot_slo_ns);
}

extern "C" int hfx_sim_run(hfx_sched *s, const hfx_table *t, const int32_t *trace_off, int32_t n_traces, int32_t iters,
                           const hfx_sim_out *o) {
  if (!s || !t || !trace_off || !o) return HFX_E_ARG;
  hfx_sched_host *h = reinterpret_cast<hfx_sched_host *>(s);
  if (n_traces < 0 || iters < 0 || iters > (1 << 29)) return HFX_E_ARG;
  if (n_traces > s->p.n_replicas) return HFX_E_CAPACITY;
  const void *need[] = {t->class_id, t->state, t->prompt_len, t->output_len, t->gen, t->arrival_ns, t->first_token_ns,
                        t->last_token_ns, t->finish_ns, t->req_id, o->iters_executed, o->finished, o->rejected,
                        o->attained, o->ttft_p50_ns, o->ttft_p99_ns, o->tpot_p50_ns, o->tpot_p99_ns};
  for (const void *p : need) if (!p) return HFX_E_ARG;
  if (s->p.weight_max > 0 && !t->weight) return HFX_E_ARG;
  const void *all[] = {t->class_id, t->state, t->prompt_len, t->output_len, t->gen, t->arrival_ns, t->first_token_ns,
                       t->last_token_ns, t->finish_ns, t->req_id, t->weight, o->iters_executed, o->finished,
                       o->rejected, o->attained, o->ttft_p50_ns, o->ttft_p99_ns, o->tpot_p50_ns, o->tpot_p99_ns,
                       o->now_ns};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  if (n_traces == 0) return HFX_OK;
  int32_t longest = 0;
  if (trace_off[0] < 0) return HFX_E_ARG;
  for (int32_t j = 0; j < n_traces; j++) {
    const int64_t len = (int64_t)trace_off[j + 1] - trace_off[j];
    if (len < 0) return HFX_E_ARG;
    if (len > SIM_MAX_ROWS) return HFX_E_CAPACITY;
    if (h->h_cfg[j].mode != HFX_COLOCATED) return HFX_E_ARG;
    if (len > longest) longest = (int32_t)len;
  }
  if (trace_off[n_traces] > t->n_rows || t->n_rows > s->max_rows) return HFX_E_CAPACITY;
  if (cudaMemcpyAsync(h->d_trace_off, trace_off, sizeof(int32_t) * ((size_t)n_traces + 1), cudaMemcpyHostToDevice,
                      s->stream) != cudaSuccess) {
    cudaGetLastError();
    return HFX_E_CUDA;
  }
  return hfx_launch_sim_kernel(s, t, h->d_trace_off, n_traces, longest, iters, o, h->d_work_counter);
}

extern "C" int hfx_sched_status(hfx_sched *s, uint32_t *status_word) {
  if (!s || !status_word) return HFX_E_ARG;
  uint32_t w = 0;
  if (cudaMemcpyAsync(&w, s->d_status, sizeof(w), cudaMemcpyDeviceToHost, s->stream) != cudaSuccess ||
      cudaMemsetAsync(s->d_status, 0, sizeof(w), s->stream) != cudaSuccess ||
      cudaStreamSynchronize(s->stream) != cudaSuccess) {
    cudaGetLastError();
    return HFX_E_CUDA;
  }
  *status_word = w;
  return (w & HFX_ST_TIMEOUT) ? HFX_E_TIMEOUT : HFX_OK;
}

extern "C" int64_t hfx_sched_launch_count(const hfx_sched *s) { return s ? s->launches : 0; }

extern "C" int hfx_sched_set_profiling(hfx_sched *s, int on) {
  if (!s) return HFX_E_ARG;
  s->profiling = on ? 1 : 0;
  return HFX_OK;
}

extern "C" int hfx_sched_set_fused_front(hfx_sched *s, int on) {
  if (!s) return HFX_E_ARG;
  s->front_enabled = on ? 1 : 0;
  return HFX_OK;
}

extern "C" int hfx_sched_set_horizon(hfx_sched *s, int64_t horizon_ns) {
  if (!s) return HFX_E_ARG;
  s->horizon = horizon_ns;
  return HFX_OK;
}

extern "C" int hfx_scale_apply(hfx_sched *s, int64_t now_ns, const int32_t *decision, const int64_t *used_blocks,
                               const int64_t *cold_start_ns, const hfx_fleet *f, const hfx_replica_state *st, int64_t *cost_ns) {
  if (!s || !decision || !used_blocks || !cold_start_ns || !f || !st || !st->now_ns || !st->maturity_ns || !cost_ns) return HFX_E_ARG;
  if (!f->inst_state || !f->ready_ns || !f->billed_ns || !f->since_ns || !f->total_blocks || !f->due_ns || !f->blocks_cap) return HFX_E_ARG;
  for (int q = 0; q < 3; q++) if (cold_start_ns[q] < 0 || cold_start_ns[q] > (INT64_C(1) << 50)) return HFX_E_ARG;
  const void *all[] = {decision, used_blocks, f->inst_state, f->ready_ns, f->billed_ns, f->since_ns, f->total_blocks, f->due_ns,
                       f->blocks_cap, st->now_ns, st->maturity_ns, cost_ns};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  return hfx_launch_fleet_apply(s, now_ns, decision, used_blocks, cold_start_ns, f, st->now_ns, st->maturity_ns, cost_ns);
}

extern "C" int hfx_dispatch_bind(hfx_sched *s, const hfx_table *t, int32_t *replica_id, int64_t now_ns,
                                 const hfx_dispatch_out *o, int64_t *clock_ns) {
  if (!s || !t || !o || !o->assign || !o->adm_count || !clock_ns || t->n_rows < 0) return HFX_E_ARG;
  if (t->n_rows > s->max_rows) return HFX_E_CAPACITY;
  if (t->n_rows > 0 && (!replica_id || replica_id != t->replica_id)) return HFX_E_ARG;
  const void *all[] = {replica_id, o->assign, o->adm_count, clock_ns};
  for (const void *p : all) if (misaligned(p)) return HFX_E_ALIGN;
  return hfx_launch_dispatch_bind(s, t->n_rows, now_ns, o->assign, o->adm_count, replica_id, clock_ns);
}

extern "C" int hfx_sched_get_profile(hfx_sched *s, hfx_profile *out) {
  if (!s || !out) return HFX_E_ARG;
  if (cudaStreamSynchronize(s->stream) != cudaSuccess) { cudaGetLastError(); return HFX_E_CUDA; }
  if (!s->brackets) return HFX_OK;
  for (HfxBracket &b : *s->brackets) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, b.a, b.b) == cudaSuccess && b.slot >= 0 && b.slot < HFX_N_KERNELS) {
      out->ms[b.slot] += ms;
      out->launches[b.slot] += 1;
    }
    cudaEventDestroy(b.a); cudaEventDestroy(b.b);
  }
  s->brackets->clear();
  cudaGetLastError();
  return HFX_OK;
}

extern "C" const char *hfx_kernel_name(int slot) {
  static const char *names[] = {"k_count", "(unused)", "k_offsets", "k_regroup_atomic", "k_replicas", "(unused)",
                                "(unused)", "k_sim", "k_scale", "k_front", "k_dispatch", "k_slo_map", "k_pd_migrate", "k_attainment"};
  return (slot >= 0 && slot < 14) ? names[slot] : nullptr;
}
