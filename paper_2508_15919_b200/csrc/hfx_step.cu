// hfx_sched_step: one scheduling iteration over the whole request table.
//
// Pipeline (all on one stream, no host synchronisation).  The first four stages run as ONE cooperative
// kernel, k_front, when every tile's block can be resident at once; otherwise as kernels of their own:
//   k_count     per-tile histogram of replica_id (shared memory), one matrix row per tile
//   k_colscan   column-wise exclusive scan of the tile histograms: where each tile's rows of each
//               replica start inside the replica's range; per-replica totals
//   k_offsets   exclusive scan of the totals -> seg_off, range starts
//   k_regroup   the one streaming pass over the table: per-row latency model, slack base and
//               priority; every row becomes a 32-byte record written to its replica's range at a
//               position that keeps row order (a stable partition without global atomics)
//   k_segment   one block per replica: aggregates of the running batch, E_d, safe budget (Eq. 3),
//               final slack and key, shared-memory sort, segmented-scan admission, maturity
//               update, optional commit
//   k_big       the same for replicas whose rows do not fit in shared memory (global sort)
// The kernels live in hfx_regroup.cu and hfx_segment.cu; this file sequences them.
#include "hfx_internal.cuh"

void hfx_tile_shape(int64_t n, int32_t *tile_rows, int32_t *n_tiles) {
  int64_t t = (n + HFX_TILE_BLOCKS - 1) / HFX_TILE_BLOCKS;
  t = (t + 3) & ~INT64_C(3);
  if (t < 1024) t = 1024;
  if (t > HFX_TILE_ROWS_MAX) t = HFX_TILE_ROWS_MAX;
  *tile_rows = (int32_t)t;
  int64_t k = (n + t - 1) / t;
  if (k < 1) k = 1;
  *n_tiles = (int32_t)k;
}

int hfx_launch_step(hfx_sched *s, const hfx_table *t, const hfx_replica_state *st, const hfx_step_out *o,
                    uint32_t flags) {
  RegroupArgs ra;
  ra.replica_id = t->replica_id; ra.class_id = t->class_id; ra.state = t->state; ra.prompt_len = t->prompt_len;
  ra.output_len = t->output_len; ra.gen = t->gen; ra.arrival = t->arrival_ns; ra.first_token = t->first_token_ns;
  ra.req_id = t->req_id; ra.weight = s->p.weight_max > 0 ? t->weight : nullptr;
  ra.now = st->now_ns; ra.mat = st->maturity_ns; ra.cfg = s->d_cfg; ra.mode = s->d_mode; ra.pred_ttft = o->pred_ttft_ns; ra.n = t->n_rows;
  ra.slack = o->slack_ns; ra.pred_tpot = o->pred_tpot_ns; ra.key = o->key; ra.order = o->order; ra.admit = o->admit;
  ra.admitted_rows = o->admitted_rows; ra.commit = flags & HFX_COMMIT;
  int rc = hfx_launch_regroup(s, ra, o->seg_off);
  if (rc != HFX_OK) return rc;

  SegArgs sa;
  sa.arrival = t->arrival_ns; sa.state = t->state; sa.gen = t->gen; sa.first_token = t->first_token_ns; sa.last_token = t->last_token_ns;
  sa.finish = t->finish_ns; sa.now = st->now_ns; sa.mat = st->maturity_ns; sa.cfg = s->d_cfg;
  sa.slack = o->slack_ns; sa.pred_tpot = o->pred_tpot_ns; sa.key = o->key; sa.order = o->order; sa.admit = o->admit;
  sa.admitted_rows = o->admitted_rows; sa.budget = o->budget; sa.e_d = o->e_d_ns; sa.n_run = o->n_run;
  sa.sum_kv = o->sum_kv; sa.adm_cost = o->adm_cost; sa.adm_count = o->adm_count; sa.maturity_next = o->maturity_next;
  sa.flags = flags; sa.horizon = s->horizon;
  rc = hfx_launch_segments(s, sa, t->n_rows);
  s->step_parity ^= 1u;
  if (rc != HFX_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
