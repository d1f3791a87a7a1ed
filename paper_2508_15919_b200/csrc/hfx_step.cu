// hfx_sched_step: one scheduling iteration over the whole request table.
//
// Two launches on one stream, no host synchronisation, no wait between blocks:
//   k_front     one pass over the table, one block per tile: per-row latency model, slack base and
//               priority, the per-row outputs, and the tile's rows grouped by replica in a slab of
//               its own (hfx_front.cu)
//   k_replicas  one persistent block per SM: every replica's rows gathered from the slabs in row
//               order, aggregates of the running batch, E_d, safe budget (Eq. 3), final slack and key,
//               sort, segmented-scan admission, maturity update, optional commit (hfx_segment.cu);
//               launched so that its set-up overlaps the tail of k_front
// Tables with more replicas than the tile front end takes go through the fallback front end
// (hfx_regroup.cu: three kernels with global counters) and the same k_replicas.
#include "hfx_internal.cuh"

int hfx_launch_step(hfx_sched *s, const hfx_table *t, const hfx_replica_state *st, const hfx_step_out *o,
                    uint32_t flags) {
  SegArgs sa;
  sa.arrival = t->arrival_ns; sa.req_id = t->req_id; sa.output_len = t->output_len;
  sa.state = t->state; sa.gen = t->gen; sa.first_token = t->first_token_ns; sa.last_token = t->last_token_ns;
  sa.finish = t->finish_ns; sa.now = st->now_ns; sa.mat = st->maturity_ns; sa.cfg = s->d_cfg;
  sa.slack = o->slack_ns; sa.pred_tpot = o->pred_tpot_ns; sa.key = o->key; sa.order = o->order; sa.seg_off = o->seg_off;
  sa.admit = o->admit;
  sa.admitted_rows = o->admitted_rows; sa.budget = o->budget; sa.e_d = o->e_d_ns; sa.n_run = o->n_run;
  sa.sum_kv = o->sum_kv; sa.adm_cost = o->adm_cost; sa.adm_count = o->adm_count; sa.maturity_next = o->maturity_next;
  sa.flags = flags; sa.horizon = s->horizon;

  bool slabs = s->tiles_max > 0 && s->front_enabled;
  if (slabs) {
    int32_t tile_rows, n_tiles;
    hfx_front_shape(s, t->n_rows, &tile_rows, &n_tiles);
    slabs = n_tiles <= s->tiles_max;
  }
  int rc;
  if (slabs) {
    FrontArgs fa;
    fa.replica_id = t->replica_id; fa.class_id = t->class_id; fa.state = t->state; fa.prompt_len = t->prompt_len;
    fa.gen = t->gen; fa.arrival = t->arrival_ns; fa.first_token = t->first_token_ns; fa.req_id = t->req_id;
    fa.weight = s->p.weight_max > 0 ? t->weight : nullptr;
    fa.now = st->now_ns; fa.mat = st->maturity_ns; fa.mode = s->d_mode; fa.n = t->n_rows;
    fa.slack = o->slack_ns; fa.pred_ttft = o->pred_ttft_ns; fa.pred_tpot = o->pred_tpot_ns; fa.key = o->key; fa.admit = o->admit;
    rc = hfx_launch_front(s, fa);
    if (rc == HFX_OK) rc = hfx_launch_replicas(s, sa, t->n_rows, true);
    s->tot_parity ^= 1u;
  } else {
    RegroupArgs ra;
    ra.replica_id = t->replica_id; ra.class_id = t->class_id; ra.state = t->state; ra.prompt_len = t->prompt_len;
    ra.output_len = t->output_len; ra.gen = t->gen; ra.arrival = t->arrival_ns; ra.first_token = t->first_token_ns;
    ra.req_id = t->req_id; ra.weight = s->p.weight_max > 0 ? t->weight : nullptr;
    ra.now = st->now_ns; ra.mat = st->maturity_ns; ra.cfg = s->d_cfg; ra.mode = s->d_mode; ra.pred_ttft = o->pred_ttft_ns; ra.n = t->n_rows;
    ra.slack = o->slack_ns; ra.pred_tpot = o->pred_tpot_ns; ra.key = o->key; ra.order = o->order; ra.admit = o->admit;
    ra.admitted_rows = o->admitted_rows; ra.commit = flags & HFX_COMMIT;
    rc = hfx_launch_regroup(s, ra, o->seg_off);
    if (rc == HFX_OK) rc = hfx_launch_replicas(s, sa, t->n_rows, false);
  }
  if (rc != HFX_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
