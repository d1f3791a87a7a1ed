/*
 * hfx_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-threaded statement of what the scheduler hot path
 * computes, written from the paper's Sec. 3.3.1 (dispatching steps 2-4, slack,
 * maturity time, Eq. 3, the P-stage / D-stage variants) and the Problem
 * Definition (events, Eq. 2).  The paper's Algorithm 1 is not printed in the
 * paper body, so the steps below follow its prose in the paper's order and
 * notation; every reading of a point the paper leaves open is marked
 * "reading:".  Integer nanoseconds throughout, one 128-bit product, a library
 * qsort on explicit tuples, no blocking or fusion.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use this
 * file.  It shares no code, header, table or constant with the CUDA library.
 *
 * Parity status: the arithmetic below is pinned by hand-worked values, the
 * closed form of Eq. 3 in exact rationals, closed forms of the simulator,
 * invariants and brute force on tiny inputs (tests/test_oracle_*.py).  Against the
 * behaviour of the paper's own system it is "parity unpinned": the paper
 * prints no scheduler trace or worked numeric example.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef __int128 i128;

#define ORA_INF INT64_MAX
#define ORA_TIME_MAX ((int64_t)1 << 62)
#define ORA_SLACK_MAX (((int64_t)1 << 39) - 1)
#define ORA_SLACK_MIN (-((int64_t)1 << 39))
#define ORA_MAX_LEN (1 << 24)

enum { ST_QUEUED = 0, ST_RUNNING = 1, ST_DONE = 2, ST_REJECTED = 3 };
enum { MODE_COLOCATED = 0, MODE_PREFILL = 1, MODE_DECODE = 2 };
enum { BUDGET_SAFE = 0, BUDGET_CAP_ONLY = 1 };
enum { PH_RUNNING = 0, PH_QUEUED = 1, PH_INACTIVE = 3 };
enum { BAD_REPLICA = 1, BAD_CLASS = 2, BAD_LEN = 4 };
enum { FLAG_COMMIT = 1 };

typedef struct { int64_t c0, c1, c2, d0, d1, d2; } ora_model;
typedef struct { int64_t ttft, tpot; int32_t prio, pad; } ora_class;
typedef struct { int32_t mode, token_cap, batch_cap; } ora_replica;

typedef struct {
  ora_model model;
  const ora_class *classes;
  int32_t n_classes;
  const ora_replica *replicas;
  int32_t n_replicas;
  int32_t budget_mode;
  int32_t weight_max;
  int32_t first_fit;   /* admission variant, see step 6 */
  int64_t horizon;     /* a committed step leaves a replica whose clock is past it untouched, see step 8 */
} ora_config;

typedef struct {
  int64_t n;
  const int32_t *replica_id;
  const uint8_t *class_id;
  uint8_t *state;
  const int32_t *prompt_len;
  const int32_t *output_len;
  int32_t *gen;
  const int64_t *arrival;
  int64_t *first_token;
  int64_t *last_token;
  int64_t *finish;
  const int32_t *req_id;
  const int32_t *weight;
} ora_table;

typedef struct {
  int64_t *slack;      /* [n] */
  int64_t *pred_ttft;  /* [n] */
  int64_t *pred_tpot;  /* [n] */
  uint64_t *key;       /* [n] */
  int32_t *order;      /* [n] */
  int32_t *seg_off;    /* [R+1] */
  uint8_t *admit;      /* [n] */
  int32_t *admitted_rows; /* [n] */
  int64_t *budget;     /* [R] */
  int64_t *e_d;        /* [R] */
  int32_t *n_run;      /* [R] */
  int64_t *sum_kv;     /* [R] */
  int64_t *adm_cost;   /* [R] */
  int32_t *adm_count;  /* [R] */
  int64_t *maturity_next; /* [R] */
  /* extra, for the pins */
  int64_t *epmax;      /* [R] largest safe prefill latency (ORA_INF, or -1)  */
  int64_t *n_safe;     /* [R] */
} ora_step_out;

/* ---- latency predictor (Sec. 3.3.1; quadratic prefill model of the cited
 *      work, linear when c2 = 0; decode latency from the running batch) ------ */
int64_t ora_Ep(const ora_model *m, int64_t t) { return m->c0 + m->c1 * t + m->c2 * t * t; }
int64_t ora_Ed(const ora_model *m, int64_t b, int64_t kv) { return m->d0 + m->d1 * b + m->d2 * kv; }

static int64_t clamp_slack(int64_t s) {
  if (s < ORA_SLACK_MIN) return ORA_SLACK_MIN;
  if (s > ORA_SLACK_MAX) return ORA_SLACK_MAX;
  return s;
}

/* 64-bit priority key: replica<16> | phase<2> | prio<6> | (clamp(slack)+2^39)<40>.
 * Smaller = more urgent (in-flight first, priority 0 highest, least remaining
 * SLO budget first). */
uint64_t ora_key(int32_t replica, int32_t phase, int32_t prio, int64_t slack) {
  uint64_t f = (uint64_t)(clamp_slack(slack) + ((int64_t)1 << 39));
  return ((uint64_t)replica << 48) | ((uint64_t)phase << 46) | ((uint64_t)prio << 40) | f;
}

/* Largest prefill latency E_p that keeps the worst-case TTFT bound of
 * Sec. 3.3.1: a request arriving right after this dispatch waits one maturity
 * time plus its own prefill, 2*E_p + k*E_d <= TTFT with k = E_p/(TPOT - E_d)
 * real, i.e. E_p*(2*TPOT - E_d)/(TPOT - E_d) <= TTFT.  Returns ORA_INF when no
 * TTFT bound applies, -1 when TPOT <= E_d (no slack can accumulate; reading:
 * nothing is safe). `decoding` = the instance has a running batch with a
 * bounded TPOT. */
int64_t ora_epmax(int64_t min_ttft, int decoding, int64_t min_tpot, int64_t e_d) {
  if (min_ttft == ORA_INF) return ORA_INF;
  if (!decoding) return min_ttft / 2;            /* E_d = 0: 2*E_p <= TTFT    */
  if (min_tpot <= e_d) return -1;
  i128 num = (i128)min_ttft * (i128)(min_tpot - e_d);
  i128 den = (i128)2 * min_tpot - e_d;
  return (int64_t)(num / den);
}

/* Eq. 3 solved on the general E_p: the largest n in [0, token_cap] with
 * E_p(n) <= epmax, 0 if there is none.  E_p is non-decreasing for non-negative
 * coefficients, so a binary search finds it. */
int64_t ora_nsafe(const ora_model *m, int64_t epmax, int64_t token_cap) {
  if (epmax == ORA_INF) return token_cap;
  if (ora_Ep(m, 0) > epmax) return 0;
  int64_t lo = 0, hi = token_cap;              /* E_p(lo) <= epmax always      */
  while (lo < hi) {
    int64_t mid = lo + (hi - lo + 1) / 2;
    if (ora_Ep(m, mid) <= epmax) lo = mid; else hi = mid - 1;
  }
  return lo;
}

typedef struct {
  int32_t phase, prio;
  int64_t cslack;     /* clamped slack */
  int32_t req_id;
  int64_t row;        /* global row index */
} sort_tuple;

static int cmp_tuple(const void *pa, const void *pb) {
  const sort_tuple *a = (const sort_tuple *)pa, *b = (const sort_tuple *)pb;
  if (a->phase != b->phase) return a->phase < b->phase ? -1 : 1;
  if (a->prio != b->prio) return a->prio < b->prio ? -1 : 1;
  if (a->cslack != b->cslack) return a->cslack < b->cslack ? -1 : 1;
  if (a->req_id != b->req_id) return a->req_id < b->req_id ? -1 : 1;
  return 0;
}

static int cmp_i64(const void *pa, const void *pb) {
  int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
  return a < b ? -1 : (a > b ? 1 : 0);
}

static int row_valid(const ora_config *c, const ora_table *t, int64_t i, uint32_t *status) {
  int ok = 1;
  if (t->class_id[i] >= c->n_classes) { *status |= BAD_CLASS; ok = 0; }
  if (t->prompt_len[i] < 0 || t->prompt_len[i] > ORA_MAX_LEN || t->gen[i] < 0 || t->gen[i] > ORA_MAX_LEN) {
    *status |= BAD_LEN; ok = 0;
  }
  return ok;
}

/* result of the commit of one replica */
enum { CM_WORKED = 0, CM_JUMPED = 1, CM_STUCK = 2 };

/*
 * One scheduling iteration of one replica over the rows `rows[0..m)` (global
 * row indices).  `r` selects the replica configuration; `key_replica` is the
 * replica field of the key; `order_base` is where this replica's order starts.
 * Steps are numbered as the dispatching steps of Sec. 3.3.1 are refined here.
 */
static int step_replica(const ora_config *c, const ora_table *t, int32_t r, int32_t key_replica,
                        const int64_t *rows, int64_t m, int64_t order_base, int64_t *now_p,
                        int64_t *mat_p, const ora_step_out *o, uint32_t flags, uint32_t *status) {
  const ora_model *M = &c->model;
  const ora_replica *cfg = &c->replicas[r];
  const int64_t now = *now_p, mat = *mat_p;
  int32_t *phase = (int32_t *)malloc(sizeof(int32_t) * (size_t)(m + 1));
  int64_t *cost = (int64_t *)malloc(sizeof(int64_t) * (size_t)(m + 1));
  sort_tuple *tup = (sort_tuple *)malloc(sizeof(sort_tuple) * (size_t)(m + 1));

  /* 1. visibility and phase: a request exists for the scheduler once it has
   *    arrived; in-flight requests are phase 0, the visible queue phase 1. */
  for (int64_t j = 0; j < m; j++) {
    int64_t i = rows[j];
    int ph = PH_INACTIVE;
    if (row_valid(c, t, i, status)) {
      if (t->state[i] == ST_RUNNING) ph = PH_RUNNING;
      else if (t->state[i] == ST_QUEUED && t->arrival[i] <= now) ph = PH_QUEUED;
    }
    phase[j] = ph;
  }

  /* 2. aggregates of the running batch and the strictest SLOs ("use current
   *    running batch to estimate a constant E_d"; strictest TTFT of the queue;
   *    strictest TPOT among in-flight).  reading: sum_kv = sum of prompt_len +
   *    gen over running rows; classes without a bound are skipped in a minimum. */
  int64_t n_run = 0, sum_kv = 0, min_tpot = ORA_INF, min_ttft = ORA_INF, min_tpot_q = ORA_INF;
  for (int64_t j = 0; j < m; j++) {
    int64_t i = rows[j];
    if (phase[j] == PH_RUNNING) {
      const ora_class *k = &c->classes[t->class_id[i]];
      n_run += 1;
      sum_kv += (int64_t)t->prompt_len[i] + t->gen[i];
      if (k->tpot > 0 && k->tpot < min_tpot) min_tpot = k->tpot;
    } else if (phase[j] == PH_QUEUED) {
      const ora_class *k = &c->classes[t->class_id[i]];
      if (k->ttft > 0 && k->ttft < min_ttft) min_ttft = k->ttft;
      if (k->tpot > 0 && k->tpot < min_tpot_q) min_tpot_q = k->tpot;
    }
  }
  /* a P-stage instance starts from an empty instance: it has no decode batch */
  const int64_t n_eff = cfg->mode == MODE_PREFILL ? 0 : n_run;
  const int64_t kv_eff = cfg->mode == MODE_PREFILL ? 0 : sum_kv;
  const int64_t tpot_eff = cfg->mode == MODE_PREFILL ? ORA_INF : min_tpot;
  const int64_t e_d = n_eff > 0 ? ora_Ed(M, n_eff, kv_eff) : 0;

  /* 3. safe budget (dispatching step 2).  Before maturity the instance is
   *    protected: budget 0. */
  int64_t epmax = ORA_INF, n_safe = 0, budget = 0;
  const int64_t cap_left = cfg->token_cap - n_eff > 0 ? cfg->token_cap - n_eff : 0;
  if (cfg->mode == MODE_DECODE) {
    /* D-stage: strictest TPOT among in-flight, else of the queue of prefilled
     * requests.  reading: the budget is the decode-step latency still
     * available, E_d(batch) <= TPOT, and a request costs d1 + d2*kv of it. */
    int64_t T = (n_run > 0 && min_tpot < ORA_INF) ? min_tpot : min_tpot_q;
    if (c->budget_mode == BUDGET_CAP_ONLY || T == ORA_INF) budget = ORA_INF;
    else {
      int64_t room = T - ora_Ed(M, n_run, sum_kv);
      budget = room > 0 ? room : 0;
    }
    epmax = ORA_INF; n_safe = 0;
  } else {
    if (c->budget_mode == BUDGET_CAP_ONLY) { epmax = ORA_INF; n_safe = cfg->token_cap; }
    else {
      epmax = ora_epmax(min_ttft, n_eff > 0 && tpot_eff < ORA_INF, tpot_eff, e_d);
      n_safe = ora_nsafe(M, epmax, cfg->token_cap);
    }
    budget = n_safe < cap_left ? n_safe : cap_left;
  }
  if (now < mat) budget = 0;

  /* 4. per-row predicted TTFT / TPOT, slack ("remaining SLO budget"), cost;
   * 5. priority and key. */
  const int64_t start = now > mat ? now : mat;
  for (int64_t j = 0; j < m; j++) {
    int64_t i = rows[j];
    int64_t sl = 0, pt = 0, pp = 0, cst = 0;
    int32_t prio = 63;
    if (phase[j] != PH_INACTIVE) {
      const ora_class *k = &c->classes[t->class_id[i]];
      const int64_t kv_i = (int64_t)t->prompt_len[i] + t->gen[i];
      if (c->weight_max > 0) {
        int64_t p = (int64_t)c->weight_max - t->weight[i];
        prio = (int32_t)(p < 0 ? 0 : (p > 62 ? 62 : p));
      } else prio = k->prio;
      if (phase[j] == PH_RUNNING) {
        /* accumulated slack of an in-flight request, net of the coming step:
         * its next-token deadline is first_token + (gen+1)*TPOT */
        pp = e_d;
        pt = t->first_token[i] - t->arrival[i];
        sl = k->tpot > 0 ? t->first_token[i] + ((int64_t)t->gen[i] + 1) * k->tpot - now - e_d : ORA_SLACK_MAX;
        cst = 0;
      } else if (cfg->mode == MODE_DECODE) {
        /* prefilled request waiting to be migrated to this D-stage instance */
        pp = ora_Ed(M, n_eff + 1, kv_eff + kv_i);
        pt = t->first_token[i] - t->arrival[i];
        sl = k->tpot > 0 ? t->first_token[i] + ((int64_t)t->gen[i] + 1) * k->tpot - start - pp : ORA_SLACK_MAX;
        cst = M->d1 + M->d2 * kv_i;
      } else {
        /* queued request: earliest start is max(now, maturity) */
        pt = (start - t->arrival[i]) + ora_Ep(M, t->prompt_len[i]);
        pp = ora_Ed(M, n_eff + 1, kv_eff + kv_i);
        sl = k->ttft > 0 ? k->ttft - pt : ORA_SLACK_MAX;
        cst = t->prompt_len[i];
      }
    }
    cost[j] = cst;
    o->slack[i] = sl;
    if (o->pred_ttft) o->pred_ttft[i] = pt;
    if (o->pred_tpot) o->pred_tpot[i] = pp;
    tup[j].phase = phase[j];
    tup[j].prio = prio;
    tup[j].cslack = phase[j] == PH_INACTIVE ? ORA_SLACK_MAX : clamp_slack(sl);
    tup[j].req_id = t->req_id[i];
    tup[j].row = j; /* local index for now */
    if (o->key) o->key[i] = ora_key(key_replica, phase[j], prio, tup[j].cslack);
  }

  /* order within the replica: in-flight first, then by priority, then by
   * remaining slack; reading: req_id breaks ties, inactive rows last. */
  qsort(tup, (size_t)m, sizeof(sort_tuple), cmp_tuple);

  /* 6. admission (dispatching step 3): the most urgent requests that fit.
   *    reading: a request that could not fit even alone is skipped; among the
   *    rest admission is the longest prefix whose running totals stay within
   *    the budget and the batch cap (totals keep growing after a failure).
   *    Variant (first_fit): the other reading of "requests that fit" -- every
   *    request is tried in order against what is left of the budget and the
   *    batch cap, taken if it fits and passed over if not, so a large request
   *    never shuts out the smaller ones behind it. */
  int64_t s_cost = 0, s_count = 0, adm_cost = 0, adm_count = 0, adm_kv = 0;
  for (int64_t q = 0; q < m; q++) {
    int64_t j = tup[q].row, i = rows[j];
    o->order[order_base + q] = (int32_t)i;
    if (o->admitted_rows) o->admitted_rows[order_base + q] = -1;
    uint8_t a = 0;
    if (phase[j] == PH_RUNNING) a = 1;
    else if (c->first_fit) {
      if (phase[j] == PH_QUEUED && adm_cost + cost[j] <= budget &&
          (cfg->batch_cap == 0 || n_eff + adm_count + 1 <= cfg->batch_cap)) {
        a = 1;
        if (o->admitted_rows) o->admitted_rows[order_base + adm_count] = (int32_t)i;
        adm_cost += cost[j];
        adm_count += 1;
        adm_kv += (int64_t)t->prompt_len[i] + t->gen[i];
      }
    } else if (phase[j] == PH_QUEUED && cost[j] <= budget) {
      s_cost += cost[j];
      s_count += 1;
      if (s_cost <= budget && (cfg->batch_cap == 0 || n_eff + s_count <= cfg->batch_cap)) {
        a = 1;
        if (o->admitted_rows) o->admitted_rows[order_base + adm_count] = (int32_t)i;
        adm_cost += cost[j];
        adm_count += 1;
        adm_kv += (int64_t)t->prompt_len[i] + t->gen[i];
      }
    }
    o->admit[i] = a;
  }

  /* 7. maturity time after the dispatch (dispatching step 4). */
  int64_t mat_next = mat;
  int64_t lp = 0;
  if (cfg->mode == MODE_DECODE) {
    /* end of the next decode iteration of the enlarged batch; reading: before
     * maturity an iteration is still in flight and its end stands */
    if (now >= mat && n_run + adm_count > 0) mat_next = now + ora_Ed(M, n_run + adm_count, sum_kv + adm_kv);
  } else if (adm_count > 0) {
    lp = ora_Ep(M, adm_cost);   /* reading: E_p of a batch = model at its total tokens */
    if (cfg->mode == MODE_PREFILL) mat_next = now + lp;  /* completion of the batch */
    else {
      /* Maturity = E_p + k*E_d, k decode iterations accumulate E_p of slack;
       * reading: k is rounded up here, and is 0 without a bounded running batch */
      i128 k = 0;
      if (n_eff > 0 && tpot_eff < ORA_INF && tpot_eff > e_d) k = ((i128)lp + (tpot_eff - e_d) - 1) / (tpot_eff - e_d);
      i128 v = (i128)now + lp + k * e_d;
      mat_next = v > ORA_TIME_MAX ? ORA_TIME_MAX : (int64_t)v;
    }
  }

  o->budget[r] = budget;
  if (o->e_d) o->e_d[r] = e_d;
  if (o->n_run) o->n_run[r] = (int32_t)n_run;
  if (o->sum_kv) o->sum_kv[r] = sum_kv;
  o->adm_cost[r] = adm_cost;
  o->adm_count[r] = (int32_t)adm_count;
  o->maturity_next[r] = mat_next;
  if (o->epmax) o->epmax[r] = epmax;
  if (o->n_safe) o->n_safe[r] = n_safe;

  /* 8. commit: the iteration happens.  Colocated: the new prefill batch runs
   *    first (prefill preempts ongoing decoding), then one decode iteration of
   *    the batch that was running. */
  /*    reading (coupling replicas to a global clock): the events of the paper
   *    happen in one global time; when a caller advances many replicas in
   *    rounds, a replica whose own clock is already past the round's horizon
   *    has nothing due yet and sits the commit out (its decisions are still
   *    reported).  The horizon is "never" unless the caller sets one. */
  int result = CM_WORKED;
  if ((flags & FLAG_COMMIT) && now <= c->horizon) {
    int worked;
    int64_t t1 = now, t2 = now;
    if (cfg->mode == MODE_COLOCATED) {
      worked = adm_count > 0 || n_run > 0;
      t1 = now + (adm_count > 0 ? lp : 0);
      t2 = t1 + (n_run > 0 ? e_d : 0);
    } else if (cfg->mode == MODE_PREFILL) {
      worked = adm_count > 0;
      t1 = t2 = now + (adm_count > 0 ? lp : 0);
    } else {
      worked = now >= mat && n_run + adm_count > 0;
      t1 = now;
      t2 = worked ? mat_next : now;
    }
    int64_t next_arrival = ORA_INF;
    for (int64_t j = 0; j < m; j++) {
      int64_t i = rows[j];
      if (phase[j] == PH_RUNNING) {
        if (cfg->mode == MODE_PREFILL) continue;   /* a P-stage instance does not decode */
        if (cfg->mode == MODE_DECODE && !worked) continue;
        t->gen[i] += 1;
        t->last_token[i] = t2;
        if ((int64_t)t->gen[i] + 1 >= t->output_len[i]) { t->state[i] = ST_DONE; t->finish[i] = t2; }
      } else if (phase[j] == PH_QUEUED) {
        if (o->admit[i]) {
          t->state[i] = ST_RUNNING;
          if (cfg->mode == MODE_DECODE) {
            t->gen[i] += 1;
            t->last_token[i] = t2;
            if ((int64_t)t->gen[i] + 1 >= t->output_len[i]) { t->state[i] = ST_DONE; t->finish[i] = t2; }
          } else {
            t->gen[i] = 0;
            t->first_token[i] = t1;
            t->last_token[i] = t1;
            if (t->output_len[i] <= 1) { t->state[i] = ST_DONE; t->finish[i] = t1; }
          }
        } else if (cfg->mode != MODE_DECODE && t->prompt_len[i] > cfg->token_cap) {
          t->state[i] = ST_REJECTED;   /* reading: an oversize prompt can never be served */
        }
      } else if (t->state[i] == ST_QUEUED && t->arrival[i] > now && row_valid(c, t, i, status)) {
        if (t->arrival[i] < next_arrival) next_arrival = t->arrival[i];
      }
    }
    if (worked) { *now_p = t2; result = CM_WORKED; }
    else {
      /* idle: jump to the next event (maturity or the next arrival), if any */
      int64_t ev = ORA_INF;
      if (mat > now) ev = mat;
      if (next_arrival < ev) ev = next_arrival;
      if (ev == ORA_INF) result = CM_STUCK;
      else { *now_p = ev; result = CM_JUMPED; }
    }
    *mat_p = mat_next;
  }
  free(phase); free(cost); free(tup);
  return result;
}

/*
 * One scheduling iteration over the whole table.  now[R], maturity[R] are read,
 * and written when flags has FLAG_COMMIT.  Returns the status bits.
 */
uint32_t ora_step(const ora_config *c, const ora_table *t, int64_t *now, int64_t *maturity,
                  const ora_step_out *o, uint32_t flags) {
  const int32_t R = c->n_replicas;
  uint32_t status = 0;
  int64_t *cnt = (int64_t *)calloc((size_t)R + 2, sizeof(int64_t));
  for (int64_t i = 0; i < t->n; i++) {
    int32_t r = t->replica_id[i];
    /* reading: replica_id -1 on a QUEUED request means "still in the global queue" (the dispatcher has not
     * bound it yet): no replica looks at it, it is listed behind the last replica, and it is no error */
    if (r == -1 && t->state[i] == ST_QUEUED) r = R;
    else if (r < 0 || r >= R) { status |= BAD_REPLICA; r = R; }
    cnt[r + 1]++;
  }
  for (int32_t r = 0; r <= R; r++) cnt[r + 1] += cnt[r];
  for (int32_t r = 0; r <= R; r++) o->seg_off[r] = (int32_t)cnt[r];
  int64_t *rows = (int64_t *)malloc(sizeof(int64_t) * (size_t)(t->n + 1));
  int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * ((size_t)R + 2));
  memcpy(fill, cnt, sizeof(int64_t) * ((size_t)R + 2));
  for (int64_t i = 0; i < t->n; i++) {
    int32_t r = t->replica_id[i];
    if (r < 0 || r >= R) r = R;
    rows[fill[r]++] = i;
  }
  for (int32_t r = 0; r < R; r++)
    step_replica(c, t, r, r, rows + cnt[r], cnt[r + 1] - cnt[r], cnt[r], &now[r], &maturity[r], o, flags, &status);
  /* rows bound to no replica: inactive, listed after every replica by req_id */
  {
    int64_t m = cnt[R + 1] - cnt[R];
    sort_tuple *tup = (sort_tuple *)malloc(sizeof(sort_tuple) * (size_t)(m + 1));
    for (int64_t j = 0; j < m; j++) {
      int64_t i = rows[cnt[R] + j];
      tup[j].phase = PH_INACTIVE; tup[j].prio = 63; tup[j].cslack = ORA_SLACK_MAX;
      tup[j].req_id = t->req_id[i]; tup[j].row = i;
      o->slack[i] = 0;
      if (o->pred_ttft) o->pred_ttft[i] = 0;
      if (o->pred_tpot) o->pred_tpot[i] = 0;
      if (o->key) o->key[i] = ora_key(R & 0xFFFF, PH_INACTIVE, 63, ORA_SLACK_MAX);
      o->admit[i] = 0;
    }
    qsort(tup, (size_t)m, sizeof(sort_tuple), cmp_tuple);
    for (int64_t j = 0; j < m; j++) {
      o->order[cnt[R] + j] = (int32_t)tup[j].row;
      if (o->admitted_rows) o->admitted_rows[cnt[R] + j] = -1;
    }
    free(tup);
  }
  free(cnt); free(rows); free(fill);
  return status;
}

typedef struct {
  int32_t *iters_executed, *finished, *rejected, *attained;
  int64_t *ttft_p50, *ttft_p99, *tpot_p50, *tpot_p99, *now;
} ora_sim_out;

static int64_t nearest_rank(int64_t *v, int64_t n, int p) {
  if (n == 0) return -1;
  qsort(v, (size_t)n, sizeof(int64_t), cmp_i64);
  int64_t k = (p * n + 99) / 100;   /* ceil(p*n/100) */
  if (k < 1) k = 1;
  return v[k - 1];
}

/*
 * Discrete-event simulation of traces [j0, j1): trace j = rows trace_off[j] ..
 * trace_off[j+1]-1 on replica j (colocated).  Events are arrivals and iteration
 * completions (Problem Definition).  Each iteration is one step + commit at
 * the replica's clock.  Metrics: attainment numerator (Eq. 2; unfinished and
 * rejected requests count as misses), TTFT = first token - arrival, TPOT =
 * floor((last token - first token)/(output_len - 1)), nearest-rank percentiles.
 */
uint32_t ora_sim(const ora_config *c, const ora_table *t, const int32_t *trace_off, int32_t j0,
                 int32_t j1, int32_t iters, const ora_sim_out *so) {
  uint32_t status = 0;
  int64_t max_m = 0;
  for (int32_t j = j0; j < j1; j++) {
    int64_t m = trace_off[j + 1] - trace_off[j];
    if (m > max_m) max_m = m;
  }
  int64_t *rows = (int64_t *)malloc(sizeof(int64_t) * (size_t)(max_m + 1));
  int64_t *va = (int64_t *)malloc(sizeof(int64_t) * (size_t)(max_m + 1));
  int64_t *vb = (int64_t *)malloc(sizeof(int64_t) * (size_t)(max_m + 1));
  /* scratch outputs of the step, indexed by global row / by replica */
  ora_step_out o;
  memset(&o, 0, sizeof(o));
  const int32_t R = c->n_replicas;
  o.slack = (int64_t *)malloc(sizeof(int64_t) * (size_t)(t->n + 1));
  o.order = (int32_t *)malloc(sizeof(int32_t) * (size_t)(t->n + 1));
  o.admit = (uint8_t *)malloc((size_t)(t->n + 1));
  o.budget = (int64_t *)malloc(sizeof(int64_t) * (size_t)R);
  o.adm_cost = (int64_t *)malloc(sizeof(int64_t) * (size_t)R);
  o.adm_count = (int32_t *)malloc(sizeof(int32_t) * (size_t)R);
  o.maturity_next = (int64_t *)malloc(sizeof(int64_t) * (size_t)R);
  for (int32_t j = j0; j < j1; j++) {
    const int64_t b = trace_off[j], m = trace_off[j + 1] - trace_off[j];
    for (int64_t q = 0; q < m; q++) {
      int64_t i = b + q;
      rows[q] = i;
      t->state[i] = ST_QUEUED; t->gen[i] = 0;
      t->first_token[i] = -1; t->last_token[i] = -1; t->finish[i] = -1;
    }
    int64_t now = 0, mat = 0;
    int32_t executed = 0;
    for (int32_t it = 0; it < iters; it++) {
      int res = step_replica(c, t, j, j, rows, m, b, &now, &mat, &o, FLAG_COMMIT, &status);
      if (res == CM_STUCK) break;
      executed++;
    }
    int32_t fin = 0, rej = 0, att = 0;
    int64_t na = 0, nb = 0;
    for (int64_t q = 0; q < m; q++) {
      int64_t i = b + q;
      if (t->class_id[i] >= c->n_classes) continue;
      const ora_class *k = &c->classes[t->class_id[i]];
      if (t->state[i] == ST_REJECTED) rej++;
      if (t->state[i] == ST_RUNNING || t->state[i] == ST_DONE) va[na++] = t->first_token[i] - t->arrival[i];
      if (t->state[i] == ST_DONE) {
        fin++;
        int64_t ttft = t->first_token[i] - t->arrival[i];
        int64_t tpot = t->output_len[i] > 1 ? (t->last_token[i] - t->first_token[i]) / (t->output_len[i] - 1) : 0;
        if (t->output_len[i] > 1) vb[nb++] = tpot;
        if ((k->ttft <= 0 || ttft <= k->ttft) && (k->tpot <= 0 || tpot <= k->tpot)) att++;
      }
    }
    so->iters_executed[j] = executed;
    so->finished[j] = fin;
    so->rejected[j] = rej;
    so->attained[j] = att;
    so->ttft_p50[j] = nearest_rank(va, na, 50);
    so->ttft_p99[j] = nearest_rank(va, na, 99);
    so->tpot_p50[j] = nearest_rank(vb, nb, 50);
    so->tpot_p99[j] = nearest_rank(vb, nb, 99);
    if (so->now) so->now[j] = now;
  }
  free(rows); free(va); free(vb);
  free(o.slack); free(o.order); free(o.admit); free(o.budget); free(o.adm_cost); free(o.adm_count);
  free(o.maturity_next);
  return status;
}

/* ---- scaling indicators and the threshold policy (Sec. 3.3.3 "Scaling Mechanism and Policy") -------
 * At a tick at time `now` the Scaler computes, per pool of instances (colocated, prefill, decode; the
 * paper evaluates the stages of the disaggregated mode independently):
 *   f1 = lambda_out / lambda_in over the window (now - W, now]: arrivals in and completions in the
 *        window (the window length cancels); used only once enough arrivals were seen;
 *   f2 = (1/N) * sum over queued requests of waiting_time / SLO;
 *   f3 = used_blocks / total_blocks per instance: KV blocks of in-flight requests plus blocks
 *        reserved for the requests waiting in the instance's queue.
 * f1 < eps_out or f2 > eps_wait -> scale out; else f1 > eps_in with more than one active instance ->
 * scale in, removing the instance with the smallest f3.
 * reading: waiting time is measured against the TTFT SLO, requests without one are left out of N;
 * each ratio waiting/SLO is taken in 16.16 fixed point (floor), saturated at 2^15; thresholds are
 * rationals num/den compared by cross-multiplication; an instance with total_blocks <= 0 is not
 * active; ties for the smallest f3 go to the lowest instance id.
 * reading: a QUEUED request with replica_id -1 waits in the global queue, bound to no instance yet; the
 * global queue feeds the colocated instances and the P stage, so such a request counts as an arrival
 * and as a waiting request for both of those pools (and holds no KV block anywhere). */
typedef struct {
  int64_t window;
  int32_t block_tokens, min_samples;
  int32_t eps_out_num, eps_out_den, eps_in_num, eps_in_den, eps_wait_num, eps_wait_den;
} ora_scale_params;

typedef struct {
  int64_t *counts;       /* [3][4]: per pool n_in, n_out, n_queue, sum of waiting/SLO in 16.16 */
  int64_t *used_blocks;  /* [R] */
  int32_t *decision;     /* [3][2]: per pool action (+1 out, -1 in, 0 hold), instance to remove or -1 */
} ora_scale_out;

/* The decision alone, from counters and used blocks that are already there (a Scaler that watches
 * several shards of the table sums their counters first; integer sums, so the result is the same). */
void ora_scale_decide(const ora_config *c, const int32_t *total_blocks, const ora_scale_params *sp, const ora_scale_out *o) {
  const int32_t R = c->n_replicas;
  for (int pool = 0; pool < 3; pool++) {
    const int64_t *cnt = o->counts + 4 * pool;
    int32_t n_active = 0, victim = -1;
    for (int32_t r = 0; r < R; r++) {
      if (c->replicas[r].mode != pool || total_blocks[r] <= 0) continue;
      n_active++;
      /* smallest used/total: compare by cross-multiplication */
      if (victim < 0 || (i128)o->used_blocks[r] * total_blocks[victim] < (i128)o->used_blocks[victim] * total_blocks[r]) victim = r;
    }
    const int f1_valid = cnt[0] >= sp->min_samples;
    int action = 0;
    if ((f1_valid && (i128)sp->eps_out_den * cnt[1] < (i128)sp->eps_out_num * cnt[0]) ||
        (cnt[2] > 0 && (i128)sp->eps_wait_den * cnt[3] > ((i128)sp->eps_wait_num * cnt[2] << 16)))
      action = 1;
    else if (f1_valid && (i128)sp->eps_in_den * cnt[1] > (i128)sp->eps_in_num * cnt[0] && n_active > 1)
      action = -1;
    o->decision[2 * pool] = action;
    o->decision[2 * pool + 1] = action == -1 ? victim : -1;
  }
}

uint32_t ora_scale(const ora_config *c, const ora_table *t, int64_t now, const int32_t *total_blocks,
                   const ora_scale_params *sp, const ora_scale_out *o) {
  const int32_t R = c->n_replicas;
  uint32_t status = 0;
  for (int k = 0; k < 12; k++) o->counts[k] = 0;
  for (int32_t r = 0; r < R; r++) o->used_blocks[r] = 0;
  const int64_t B = sp->block_tokens;
  for (int64_t i = 0; i < t->n; i++) {
    const int32_t r = t->replica_id[i];
    if (r == -1 && t->state[i] == ST_QUEUED) {
      /* still in the global queue: it feeds the colocated pool and the P stage, so it counts for both */
      if (!row_valid(c, t, i, &status)) continue;
      const ora_class *k = &c->classes[t->class_id[i]];
      for (int pool = 0; pool < 2; pool++) {
        int64_t *cnt = o->counts + 4 * pool;
        if (t->arrival[i] > now - sp->window && t->arrival[i] <= now) cnt[0] += 1;
        if (t->arrival[i] <= now && k->ttft > 0) {
          i128 q = ((i128)(now - t->arrival[i]) << 16) / k->ttft;
          if (q > ((i128)1 << 31)) q = (i128)1 << 31;
          cnt[2] += 1;
          cnt[3] += (int64_t)q;
        }
      }
      continue;
    }
    if (r < 0 || r >= R) { status |= BAD_REPLICA; continue; }
    if (!row_valid(c, t, i, &status)) continue;
    int64_t *cnt = o->counts + 4 * c->replicas[r].mode;
    const ora_class *k = &c->classes[t->class_id[i]];
    if (t->arrival[i] > now - sp->window && t->arrival[i] <= now) cnt[0] += 1;               /* enqueued in the window */
    if (t->state[i] == ST_DONE && t->finish[i] > now - sp->window && t->finish[i] <= now) cnt[1] += 1;  /* completed in it */
    if (t->state[i] == ST_RUNNING) o->used_blocks[r] += ((int64_t)t->prompt_len[i] + t->gen[i] + B - 1) / B;
    if (t->state[i] == ST_QUEUED && t->arrival[i] <= now) {
      o->used_blocks[r] += ((int64_t)t->prompt_len[i] + B - 1) / B;
      if (k->ttft > 0) {
        const int64_t wait = now - t->arrival[i];
        i128 q = ((i128)wait << 16) / k->ttft;
        if (q > ((i128)1 << 31)) q = (i128)1 << 31;
        cnt[2] += 1;
        cnt[3] += (int64_t)q;
      }
    }
  }
  ora_scale_decide(c, total_blocks, sp, o);
  return status;
}

/* ==========================================================================
 * Dispatching over a shared global queue (Sec. 3.3.1, colocated mode, the four
 * dispatching steps as the paper lists them): (1) take the instance whose
 * maturity time arrives first, (2) compute its safe token budget, (3) scan the
 * global request queue for the most urgent requests that fit within it,
 * (4) dispatch them and update the instance's maturity time; repeat with the
 * next instance.  Here one call makes the decisions that are due at time `now`:
 * every instance that has matured takes its turn once, in maturity order.
 *
 * reading: a request belongs to the global queue while it is QUEUED and has
 *   arrived (its replica_id is not looked at); in-flight requests count for the
 *   instance they run on.
 * reading: the queue is ordered by (priority, remaining slack, req_id) with
 *   slack = TTFT - (now - arrival) - E_p(prompt_len), the request starting at
 *   once on an instance that has matured.
 * reading: the TTFT of Eq. 3 is the strictest TTFT in the queue as it stands
 *   when the call begins; the TPOT is the strictest among the instance's
 *   in-flight requests.
 * reading: "requests that fit" -- each instance takes queue entries in order,
 *   from where the previous instance stopped, while their total stays within
 *   its budget and batch cap, and stops at the first that does not fit (that
 *   request waits at the head for the next instance).  An entry larger than
 *   the largest budget any matured instance has in this call fits nowhere now:
 *   it is passed over and stays queued, so it never blocks the entries behind
 *   it.  A prompt longer than every instance's token cap can never be served
 *   and is left out of the queue.
 * reading: instances tie on maturity in index order.
 * The same four steps serve the P stage of the disaggregated mode ("P-stage
 * Dispatcher"): a PREFILL instance takes part with the budget and the maturity
 * update of its stage (no decode batch: E_d = 0, maturity = end of the prefill
 * batch).
 * The D stage ("D-stage Migrator") runs the four steps once more in the same
 * call, for the DECODE instances over the queue of prefilled requests:
 * reading: a prefilled request is one in flight on a PREFILL instance whose
 *   first token has been produced by `now` (the end of its prefill batch); what
 *   the KV transfer adds is not modelled by this call.
 * reading: that queue is ordered by (priority, slack, req_id) with slack =
 *   first_token + (gen + 1) TPOT - now - E_d(1, prompt + gen): the time to the
 *   request's next-token deadline, net of a decode iteration on its own.
 * reading: step 2 as in the per-instance step of a DECODE replica: the budget
 *   is a time, T - E_d(running batch), T the strictest TPOT in flight on the
 *   instance, or, when it has none, of the queue of prefilled requests; a
 *   request costs d1 + d2 (prompt + gen) of it.  Step 3 hands the queue out as
 *   in the P stage (in order, stop at the first entry that does not fit, pass
 *   over what exceeds every D budget of the call).  Step 4: a matured instance
 *   with a batch gets maturity = now + E_d of the enlarged batch.
 * The caller binds a dispatched prefilled request by replica_id := assign; it
 * stays in flight, now on the D instance.
 * ========================================================================== */
typedef struct {
  int32_t *assign;        /* [n] instance a queued row is dispatched to, else -1         */
  int32_t *queue_order;   /* [n] rows of the queue, most urgent first; -1 past n_queue   */
  int32_t *n_queue;       /* [2] global queue; queue of prefilled requests (listed behind it in queue_order) */
  int32_t *inst_order;    /* [R] matured instances in dispatch order, colocated / P stage first, then D stage; -1 behind */
  int32_t *n_mature;      /* [2] colocated and P-stage instances; D-stage instances      */
  int64_t *slack;         /* [n] slack of queue rows, 0 elsewhere                        */
  int64_t *budget;        /* [R] safe token budget (0 for an instance not matured)       */
  int64_t *e_d;           /* [R] */
  int32_t *n_run;         /* [R] */
  int64_t *sum_kv;        /* [R] */
  int64_t *adm_cost;      /* [R] tokens dispatched to the instance                       */
  int32_t *adm_count;     /* [R] requests dispatched to the instance                     */
  int64_t *maturity_next; /* [R] */
} ora_dispatch_out;

typedef struct { int64_t mat; int32_t id; } inst_tuple;
static int cmp_inst(const void *pa, const void *pb) {
  const inst_tuple *a = (const inst_tuple *)pa, *b = (const inst_tuple *)pb;
  if (a->mat != b->mat) return a->mat < b->mat ? -1 : 1;
  return a->id < b->id ? -1 : (a->id > b->id ? 1 : 0);
}

uint32_t ora_dispatch(const ora_config *c, const ora_table *t, int64_t now, const int64_t *maturity,
                      const ora_dispatch_out *o) {
  const ora_model *M = &c->model;
  const int32_t R = c->n_replicas;
  const int64_t n = t->n;
  uint32_t status = 0;
  int64_t *n_run = (int64_t *)calloc((size_t)R + 1, sizeof(int64_t));
  int64_t *sum_kv = (int64_t *)calloc((size_t)R + 1, sizeof(int64_t));
  int64_t *min_tpot = (int64_t *)malloc(sizeof(int64_t) * ((size_t)R + 1));
  sort_tuple *q = (sort_tuple *)malloc(sizeof(sort_tuple) * (size_t)(n + 1));
  inst_tuple *inst = (inst_tuple *)malloc(sizeof(inst_tuple) * ((size_t)R + 1));
  int32_t cap_max = 0;
  for (int32_t r = 0; r < R; r++) {
    min_tpot[r] = ORA_INF;
    if (c->replicas[r].mode != MODE_DECODE && c->replicas[r].token_cap > cap_max) cap_max = c->replicas[r].token_cap;
  }

  /* in-flight requests: the running batch of each instance; the queue */
  int64_t nq = 0, min_ttft = ORA_INF;
  for (int64_t i = 0; i < n; i++) {
    o->assign[i] = -1;
    o->slack[i] = 0;
    o->queue_order[i] = -1;
    if (!row_valid(c, t, i, &status)) continue;
    const ora_class *k = &c->classes[t->class_id[i]];
    if (t->state[i] == ST_RUNNING) {
      const int32_t r = t->replica_id[i];
      if (r < 0 || r >= R) { status |= BAD_REPLICA; continue; }
      n_run[r] += 1;
      sum_kv[r] += (int64_t)t->prompt_len[i] + t->gen[i];
      if (k->tpot > 0 && k->tpot < min_tpot[r]) min_tpot[r] = k->tpot;
    } else if (t->state[i] == ST_QUEUED && t->arrival[i] <= now && t->prompt_len[i] <= cap_max) {
      const int64_t pred_ttft = (now - t->arrival[i]) + ora_Ep(M, t->prompt_len[i]);
      const int64_t sl = k->ttft > 0 ? k->ttft - pred_ttft : ORA_SLACK_MAX;
      int32_t prio;
      if (c->weight_max > 0) {
        int64_t p = (int64_t)c->weight_max - t->weight[i];
        prio = (int32_t)(p < 0 ? 0 : (p > 62 ? 62 : p));
      } else prio = k->prio;
      o->slack[i] = sl;
      q[nq].phase = PH_QUEUED; q[nq].prio = prio; q[nq].cslack = clamp_slack(sl);
      q[nq].req_id = t->req_id[i]; q[nq].row = i;
      nq++;
      if (k->ttft > 0 && k->ttft < min_ttft) min_ttft = k->ttft;
    }
  }
  qsort(q, (size_t)nq, sizeof(sort_tuple), cmp_tuple);
  for (int64_t j = 0; j < nq; j++) o->queue_order[j] = (int32_t)q[j].row;
  o->n_queue[0] = (int32_t)nq;

  /* step 2 for every instance that has matured; step 1: their order */
  int32_t nm = 0;
  for (int32_t r = 0; r < R; r++) {
    const ora_replica *cfg = &c->replicas[r];
    /* a P-stage instance starts from an empty instance: it has no decode batch */
    const int64_t n_eff = cfg->mode == MODE_PREFILL ? 0 : n_run[r];
    const int64_t tpot_eff = cfg->mode == MODE_PREFILL ? ORA_INF : min_tpot[r];
    const int64_t e_d = n_eff > 0 ? ora_Ed(M, n_eff, sum_kv[r]) : 0;
    int64_t budget = 0;
    if (cfg->mode == MODE_DECODE) {
      /* takes no part: reported with the decode latency of its batch, budget 0 */
    } else if (maturity[r] <= now) {
      int64_t n_safe;
      if (c->budget_mode == BUDGET_CAP_ONLY) n_safe = cfg->token_cap;
      else n_safe = ora_nsafe(M, ora_epmax(min_ttft, n_eff > 0 && tpot_eff < ORA_INF, tpot_eff, e_d), cfg->token_cap);
      const int64_t cap_left = cfg->token_cap - n_eff > 0 ? cfg->token_cap - n_eff : 0;
      budget = n_safe < cap_left ? n_safe : cap_left;
      inst[nm].mat = maturity[r]; inst[nm].id = r; nm++;
    }
    o->budget[r] = budget;
    o->e_d[r] = e_d;
    o->n_run[r] = (int32_t)n_run[r];
    o->sum_kv[r] = sum_kv[r];
    o->adm_cost[r] = 0;
    o->adm_count[r] = 0;
    o->maturity_next[r] = maturity[r];
    o->inst_order[r] = -1;
  }
  qsort(inst, (size_t)nm, sizeof(inst_tuple), cmp_inst);
  for (int32_t k = 0; k < nm; k++) o->inst_order[k] = inst[k].id;
  o->n_mature[0] = nm;

  /* steps 3 and 4, instance by instance */
  int64_t budget_max = 0;
  for (int32_t k = 0; k < nm; k++) if (o->budget[inst[k].id] > budget_max) budget_max = o->budget[inst[k].id];
  int64_t cursor = 0;
  for (int32_t k = 0; k < nm; k++) {
    const int32_t r = inst[k].id;
    const ora_replica *cfg = &c->replicas[r];
    int64_t cost = 0, count = 0;
    while (cursor < nq) {
      const int64_t i = q[cursor].row;
      if (t->prompt_len[i] > budget_max) { cursor++; continue; }   /* fits no instance in this call */
      if (cost + t->prompt_len[i] > o->budget[r]) break;
      if (cfg->batch_cap != 0 && (cfg->mode == MODE_PREFILL ? 0 : n_run[r]) + count + 1 > cfg->batch_cap) break;
      cost += t->prompt_len[i];
      count += 1;
      o->assign[i] = r;
      cursor++;
    }
    o->adm_cost[r] = cost;
    o->adm_count[r] = (int32_t)count;
    if (count > 0) {
      /* Maturity = E_p + k*E_d as in the per-instance step */
      const int64_t lp = ora_Ep(M, cost), e_d = o->e_d[r];
      i128 kk = 0;      /* a P-stage instance has E_d = 0 and no decode batch: maturity = end of the prefill batch */
      if (cfg->mode != MODE_PREFILL && n_run[r] > 0 && min_tpot[r] < ORA_INF && min_tpot[r] > e_d)
        kk = ((i128)lp + (min_tpot[r] - e_d) - 1) / (min_tpot[r] - e_d);
      i128 v = (i128)now + lp + kk * e_d;
      o->maturity_next[r] = v > ORA_TIME_MAX ? ORA_TIME_MAX : (int64_t)v;
    }
  }

  /* ---- the D stage: the same four steps, by the Migrator (Sec. 3.3.1, "D-stage Migrator") ---- */
  /* the queue of prefilled requests, priority-ordered */
  sort_tuple *dq = (sort_tuple *)malloc(sizeof(sort_tuple) * (size_t)(n + 1));
  int64_t ndq = 0, min_tpot_dq = ORA_INF;
  for (int64_t i = 0; i < n; i++) {
    uint32_t again = 0;
    if (!row_valid(c, t, i, &again) || t->state[i] != ST_RUNNING) continue;
    const int32_t r = t->replica_id[i];
    if (r < 0 || r >= R || c->replicas[r].mode != MODE_PREFILL || t->first_token[i] > now) continue;
    const ora_class *k = &c->classes[t->class_id[i]];
    const int64_t kv_i = (int64_t)t->prompt_len[i] + t->gen[i];
    const int64_t sl = k->tpot > 0 ? t->first_token[i] + ((int64_t)t->gen[i] + 1) * k->tpot - now - ora_Ed(M, 1, kv_i) : ORA_SLACK_MAX;
    int32_t prio;
    if (c->weight_max > 0) {
      int64_t pw = (int64_t)c->weight_max - t->weight[i];
      prio = (int32_t)(pw < 0 ? 0 : (pw > 62 ? 62 : pw));
    } else prio = k->prio;
    o->slack[i] = sl;
    dq[ndq].phase = PH_QUEUED; dq[ndq].prio = prio; dq[ndq].cslack = clamp_slack(sl);
    dq[ndq].req_id = t->req_id[i]; dq[ndq].row = i;
    ndq++;
    if (k->tpot > 0 && k->tpot < min_tpot_dq) min_tpot_dq = k->tpot;
  }
  qsort(dq, (size_t)ndq, sizeof(sort_tuple), cmp_tuple);
  for (int64_t j = 0; j < ndq; j++) o->queue_order[nq + j] = (int32_t)dq[j].row;
  o->n_queue[1] = (int32_t)ndq;

  /* step 1: the D-stage instances that have matured, earliest first; step 2: their budget, a time */
  int32_t nmd = 0;
  int64_t dbudget_max = 0;
  for (int32_t r = 0; r < R; r++) {
    if (c->replicas[r].mode != MODE_DECODE || maturity[r] > now) continue;
    const int64_t T = (n_run[r] > 0 && min_tpot[r] < ORA_INF) ? min_tpot[r] : min_tpot_dq;
    int64_t budget;
    if (c->budget_mode == BUDGET_CAP_ONLY || T == ORA_INF) budget = ORA_INF;
    else {
      const int64_t room = T - ora_Ed(M, n_run[r], sum_kv[r]);
      budget = room > 0 ? room : 0;
    }
    o->budget[r] = budget;
    if (budget > dbudget_max) dbudget_max = budget;
    inst[nmd].mat = maturity[r]; inst[nmd].id = r; nmd++;
  }
  qsort(inst, (size_t)nmd, sizeof(inst_tuple), cmp_inst);
  for (int32_t k = 0; k < nmd; k++) o->inst_order[nm + k] = inst[k].id;
  o->n_mature[1] = nmd;

  /* steps 3 and 4, instance by instance */
  cursor = 0;
  for (int32_t k = 0; k < nmd; k++) {
    const int32_t r = inst[k].id;
    const ora_replica *cfg = &c->replicas[r];
    int64_t cost = 0, count = 0, adm_kv = 0;
    while (cursor < ndq) {
      const int64_t i = dq[cursor].row;
      const int64_t kv_i = (int64_t)t->prompt_len[i] + t->gen[i];
      const int64_t c_i = M->d1 + M->d2 * kv_i;
      if (c_i > dbudget_max) { cursor++; continue; }          /* fits no instance in this call */
      if (c_i > o->budget[r] - cost) break;
      if (cfg->batch_cap != 0 && n_run[r] + count + 1 > cfg->batch_cap) break;
      cost += c_i; count += 1; adm_kv += kv_i;
      o->assign[i] = r;
      cursor++;
    }
    o->adm_cost[r] = cost;
    o->adm_count[r] = (int32_t)count;
    /* maturity = end of the next decoding iteration of the enlarged batch */
    if (n_run[r] + count > 0) o->maturity_next[r] = now + ora_Ed(M, n_run[r] + count, sum_kv[r] + adm_kv);
  }
  free(dq);
  free(n_run); free(sum_kv); free(min_tpot); free(q); free(inst);
  return status;
}

/* ==========================================================================
 * Priority-based SLO mapping (Sec. 3.3.2, steps (1)-(5)): a request that
 * carries only a priority p in [0, N) gets its TTFT and TPOT targets from the
 * recent history.  The history is a sliding window of completed requests
 * (priority, measured TTFT, measured TPOT, queueing delay).  With C_i the
 * number of window records of priority i,
 *     base = C_0 + ... + C_{p-1},   offset = floor((p + 1) * C_p / (N + 1)),
 * and the provisional targets are the (base + offset)-th smallest TTFT and
 * TPOT of the window (step 3).  Step 4 subtracts from the TTFT the queueing
 * delay of the chosen reference record in excess of the queueing delay last
 * seen for this priority, and remembers the reference's delay.  Step 5 clamps
 * both targets into the priority's range; while requests of a higher priority
 * are pending the strict lower bound applies, otherwise the relaxed one.
 * Requests are served in row order, so the second request of a priority in
 * one call sees the delay the first one left behind.
 *
 * reading: the two windows are ordered by value, ties by record position.
 * reading: an index past the end of the window means its last record; with an
 *   empty window the targets are the upper bounds of the range.
 * reading: "higher-priority requests are pending" = some priority below p has
 *   a positive pending count; the relaxed lower bound is a second per-priority
 *   parameter.
 * reading: window records and requests whose priority is outside [0, N) are
 *   ignored (flagged); such a request gets 0, 0.
 * ========================================================================== */
typedef struct {
  int32_t w;
  const int32_t *prio;
  const int64_t *ttft, *tpot, *queue;
} ora_slo_window;

typedef struct {
  const int64_t *ttft_min, *ttft_max, *ttft_min_relaxed, *tpot_min, *tpot_max, *tpot_min_relaxed;
} ora_slo_bounds;

typedef struct { int64_t v; int32_t pos; } val_pos;
static int cmp_val_pos(const void *pa, const void *pb) {
  const val_pos *a = (const val_pos *)pa, *b = (const val_pos *)pb;
  if (a->v != b->v) return a->v < b->v ? -1 : 1;
  return a->pos < b->pos ? -1 : (a->pos > b->pos ? 1 : 0);
}

static int64_t clamp_i64(int64_t x, int64_t lo, int64_t hi) { return x < lo ? lo : (x > hi ? hi : x); }

uint32_t ora_slo_map(int32_t n_prio, const ora_slo_window *win, const ora_slo_bounds *b, int64_t *last_queue,
                     const int32_t *pending, int64_t n_new, const int32_t *new_prio, int64_t *ttft_out,
                     int64_t *tpot_out) {
  uint32_t status = 0;
  val_pos *by_ttft = (val_pos *)malloc(sizeof(val_pos) * (size_t)(win->w + 1));
  val_pos *by_tpot = (val_pos *)malloc(sizeof(val_pos) * (size_t)(win->w + 1));
  int64_t *C = (int64_t *)calloc((size_t)n_prio + 1, sizeof(int64_t));
  int32_t w = 0;
  for (int32_t j = 0; j < win->w; j++) {
    if (win->prio[j] < 0 || win->prio[j] >= n_prio) { status |= BAD_CLASS; continue; }
    C[win->prio[j]] += 1;
    by_ttft[w].v = win->ttft[j]; by_ttft[w].pos = j;
    by_tpot[w].v = win->tpot[j]; by_tpot[w].pos = j;
    w++;
  }
  qsort(by_ttft, (size_t)w, sizeof(val_pos), cmp_val_pos);
  qsort(by_tpot, (size_t)w, sizeof(val_pos), cmp_val_pos);
  for (int64_t r = 0; r < n_new; r++) {
    const int32_t p = new_prio[r];
    if (p < 0 || p >= n_prio) { status |= BAD_CLASS; ttft_out[r] = 0; tpot_out[r] = 0; continue; }
    int64_t ttft = b->ttft_max[p], tpot = b->tpot_max[p];
    if (w > 0) {
      int64_t base = 0;
      for (int32_t i = 0; i < p; i++) base += C[i];
      const int64_t offset = ((int64_t)(p + 1) * C[p]) / (n_prio + 1);
      int64_t idx = base + offset;
      if (idx > w - 1) idx = w - 1;
      const int64_t q_ref = win->queue[by_ttft[idx].pos];
      ttft = by_ttft[idx].v - (q_ref - last_queue[p]);
      last_queue[p] = q_ref;
      tpot = by_tpot[idx].v;
    }
    int higher_pending = 0;
    for (int32_t i = 0; i < p; i++) if (pending[i] > 0) higher_pending = 1;
    ttft_out[r] = clamp_i64(ttft, higher_pending ? b->ttft_min[p] : b->ttft_min_relaxed[p], b->ttft_max[p]);
    tpot_out[r] = clamp_i64(tpot, higher_pending ? b->tpot_min[p] : b->tpot_min_relaxed[p], b->tpot_max[p]);
  }
  free(by_ttft); free(by_tpot); free(C);
  return status;
}

/* ==========================================================================
 * Hand-off from the P stage to the D stage in the disaggregated mode
 * (Sec. 3.3.1 "Disaggregated Mode": prefill and decode run on separate
 * instance pools, the Migrator makes the D-stage decisions over the queue of
 * prefilled requests; the Overview has the Migrator coordinate the KV-cache
 * transfers).  Together with the per-replica step and its commit this couples
 * the two stages: a request is prefilled on a P instance (step, commit: it is
 * RUNNING there with its first-token time = the end of its prefill batch), its
 * KV cache is transferred, and it joins the queue of its partner D instance.
 *
 * reading: every P instance r has one partner D instance pair[r].
 * reading: the transfer of a request takes x0 + x1 * prompt_len ns and starts
 *   when its prefill batch ends; the request can be handed over once the D
 *   instance's clock has reached that time.  It then becomes QUEUED on the D
 *   instance (prefilled: its first-token time stands).
 * reading: a D instance with nothing in flight and nothing in its queue would
 *   never move its clock; it is woken at the earliest time a transfer to it
 *   completes.
 * Requests that finished at their first token (output_len <= 1) are DONE on
 * the P instance and stay there.
 * ========================================================================== */
uint32_t ora_pd_migrate(const ora_config *c, const ora_table *t, int64_t *now, const int32_t *pair, int64_t x0,
                        int64_t x1, int32_t *n_moved) {
  const int32_t R = c->n_replicas;
  uint32_t status = 0;
  int32_t *rid = (int32_t *)t->replica_id;      /* the binding is rewritten here */
  int64_t *wake = (int64_t *)malloc(sizeof(int64_t) * (size_t)R);
  int32_t *busy = (int32_t *)calloc((size_t)R, sizeof(int32_t));
  int32_t moved = 0;
  for (int32_t r = 0; r < R; r++) wake[r] = ORA_INF;
  for (int64_t i = 0; i < t->n; i++) {
    const int32_t r = rid[i];
    if (r == -1 && t->state[i] == ST_QUEUED) continue;      /* still in the global queue */
    if (r < 0 || r >= R) { status |= BAD_REPLICA; continue; }
    if (!row_valid(c, t, i, &status)) continue;
    if (c->replicas[r].mode != MODE_PREFILL || t->state[i] != ST_RUNNING) continue;
    const int32_t d = pair[r];
    if (d < 0 || d >= R || c->replicas[d].mode != MODE_DECODE) { status |= BAD_REPLICA; continue; }
    const int64_t ready = t->first_token[i] + x0 + x1 * (int64_t)t->prompt_len[i];
    if (ready <= now[d]) { rid[i] = d; t->state[i] = ST_QUEUED; moved++; }
    else if (ready < wake[d]) wake[d] = ready;
  }
  for (int64_t i = 0; i < t->n; i++) {
    const int32_t r = rid[i];
    if (r < 0 || r >= R || c->replicas[r].mode != MODE_DECODE) continue;
    uint32_t ignore = 0;
    if (!row_valid(c, t, i, &ignore)) continue;
    if (t->state[i] == ST_RUNNING || (t->state[i] == ST_QUEUED && t->arrival[i] <= now[r])) busy[r] = 1;
  }
  for (int32_t d = 0; d < R; d++)
    if (c->replicas[d].mode == MODE_DECODE && !busy[d] && wake[d] != ORA_INF && wake[d] > now[d]) now[d] = wake[d];
  if (n_moved) *n_moved = moved;
  free(wake); free(busy);
  return status;
}

/* ==========================================================================
 * SLO attainment over a request table (Problem Definition, Eq. 2: the
 * fraction of requests that meet both their TTFT and their TPOT target), per
 * SLO class and in total, with the sums behind the mean TTFT and the mean
 * end-to-end time E2E = T_complete - T_arrival of the same section.
 *   TTFT = first_token - arrival (requests RUNNING or DONE),
 *   TPOT = floor((last_token - first_token) / (output_len - 1)), 0 for
 *          output_len <= 1 (DONE requests),
 * a target <= 0 is unbounded and always met; requests that are not DONE count
 * as misses (Eq. 2 sums over all M requests).
 * out[(c)*6 + k], c = class (row n_classes = total), k = 0 requests, 1 DONE,
 * 2 attained, 3 REJECTED, 4 sum of TTFT, 5 sum of E2E over DONE requests.
 * ========================================================================== */
uint32_t ora_attainment(const ora_config *c, const ora_table *t, int64_t *out) {
  uint32_t status = 0;
  const int32_t K = c->n_classes;
  for (int32_t k = 0; k < (K + 1) * 6; k++) out[k] = 0;
  for (int64_t i = 0; i < t->n; i++) {
    if (!row_valid(c, t, i, &status)) continue;
    const int32_t cl = t->class_id[i];
    const ora_class *k = &c->classes[cl];
    int64_t v[6] = {1, 0, 0, 0, 0, 0};
    if (t->state[i] == ST_REJECTED) v[3] = 1;
    if (t->state[i] == ST_RUNNING || t->state[i] == ST_DONE) v[4] = t->first_token[i] - t->arrival[i];
    if (t->state[i] == ST_DONE) {
      const int64_t ttft = t->first_token[i] - t->arrival[i];
      const int64_t tpot = t->output_len[i] > 1 ? (t->last_token[i] - t->first_token[i]) / (t->output_len[i] - 1) : 0;
      v[1] = 1;
      v[5] = t->finish[i] - t->arrival[i];
      if ((k->ttft <= 0 || ttft <= k->ttft) && (k->tpot <= 0 || tpot <= k->tpot)) v[2] = 1;
    }
    for (int q = 0; q < 6; q++) { out[cl * 6 + q] += v[q]; out[K * 6 + q] += v[q]; }
  }
  return status;
}

/* ==========================================================================
 * Carrying out the Scaler's decisions: the life of an instance and the cost of
 * the fleet (Sec. 3.3.3 "Scaling Mechanism and Policy" for the decisions, the
 * Problem Definition's Eq. 1 for the cost; the time to bring an instance up is
 * a constant per pool, the quantity the paper's scaling-time table measures).
 * An instance is OFF (0), STARTING (1: decided, not yet serving), ACTIVE (2)
 * or DRAINING (3: chosen for removal, finishing what it holds).  At a tick at
 * time `now`, in this order:
 *   1. every instance that is not OFF is charged for (since, now];
 *   2. a STARTING instance whose ready time has come turns ACTIVE: its clock
 *      and its maturity (the per-instance arrays of the scheduling step) are
 *      brought up to the ready time, it serves nothing earlier;
 *   3. a DRAINING instance that holds no KV block any more turns OFF;
 *   4. per pool, the decision of this tick: scale out -> the pool gets one
 *      more instance; scale in -> the named instance starts DRAINING;
 *   5. due[r], the maturity the dispatcher sees, is the instance's maturity
 *      if it is ACTIVE and "never" otherwise (only ACTIVE instances are given
 *      new requests); total_blocks (what the next tick reads) is the capacity
 *      of an ACTIVE instance and 0 for every other one; cost[pool] = sum of
 *      charged time.
 * reading: Eq. 1's "active time" runs from the decision to start an instance
 *   until it is turned off: starting up and draining hold the device too.
 * reading: while an instance of the pool is STARTING a further scale-out does
 *   nothing (the capacity already on its way is not ordered twice).  Otherwise
 *   a DRAINING instance of the pool, lowest id first, is taken back into
 *   service at once (no start-up), else the lowest-id OFF instance of the pool
 *   starts and is ready at now + cold_start[pool]; with none left, nothing.
 * reading: a scale-in that names an instance which is not ACTIVE, or of
 *   another pool, does nothing.  Role switching between pools is not modelled.
 * ========================================================================== */
#define INST_OFF 0
#define INST_STARTING 1
#define INST_ACTIVE 2
#define INST_DRAINING 3
#define T_NEVER INT64_MAX

typedef struct {
  int32_t *inst_state;       /* [R] */
  int64_t *ready;            /* [R] */
  int64_t *billed;           /* [R] */
  int64_t *since;            /* [R] */
  int32_t *total_blocks;     /* [R] out */
  int64_t *due;              /* [R] out */
  const int32_t *blocks_cap; /* [R] */
} ora_fleet;

void ora_scale_apply(const ora_config *c, int64_t now, const int32_t *decision, const int64_t *used_blocks,
                     const int64_t *cold_start, const ora_fleet *f, int64_t *clock, int64_t *maturity, int64_t *cost) {
  const int32_t R = c->n_replicas;
  for (int32_t r = 0; r < R; r++) {
    if (f->inst_state[r] != INST_OFF && now > f->since[r]) { f->billed[r] += now - f->since[r]; f->since[r] = now; }
    if (f->inst_state[r] == INST_STARTING && f->ready[r] <= now) {
      f->inst_state[r] = INST_ACTIVE;
      if (clock[r] < f->ready[r]) clock[r] = f->ready[r];
      if (maturity[r] < f->ready[r]) maturity[r] = f->ready[r];
    }
    if (f->inst_state[r] == INST_DRAINING && used_blocks[r] == 0) f->inst_state[r] = INST_OFF;
  }
  for (int pool = 0; pool < 3; pool++) {
    const int action = decision[2 * pool], victim = decision[2 * pool + 1];
    if (action > 0) {
      int32_t first[4] = {-1, -1, -1, -1};      /* lowest id of the pool in each state */
      for (int32_t r = R - 1; r >= 0; r--)
        if (c->replicas[r].mode == pool) first[f->inst_state[r]] = r;
      if (first[INST_STARTING] >= 0) {
        /* capacity is already on its way */
      } else if (first[INST_DRAINING] >= 0) {
        f->inst_state[first[INST_DRAINING]] = INST_ACTIVE;
      } else if (first[INST_OFF] >= 0) {
        const int32_t r = first[INST_OFF];
        f->inst_state[r] = INST_STARTING; f->ready[r] = now + cold_start[pool]; f->since[r] = now;
      }
    } else if (action < 0 && victim >= 0 && victim < R && c->replicas[victim].mode == pool &&
               f->inst_state[victim] == INST_ACTIVE) {
      f->inst_state[victim] = INST_DRAINING;
    }
  }
  cost[0] = cost[1] = cost[2] = 0;
  for (int32_t r = 0; r < R; r++) {
    const int on = f->inst_state[r] == INST_ACTIVE;
    f->total_blocks[r] = on ? f->blocks_cap[r] : 0;
    f->due[r] = on ? maturity[r] : T_NEVER;
    cost[c->replicas[r].mode] += f->billed[r];
  }
}

/* Binding what a dispatching call decided (Sec. 3.3.1, step "dispatch them"): each request the call
 * assigned now belongs to its instance (replica_id), and an instance that was given requests cannot
 * have started them before the call was made: its clock is brought up to `now` if it was behind
 * (an idle instance's clock stands where its last iteration ended). */
void ora_dispatch_bind(const ora_config *c, const ora_table *t, int64_t now, const int32_t *assign,
                       const int32_t *adm_count, int32_t *replica_id, int64_t *clock) {
  for (int64_t i = 0; i < t->n; i++)
    if (assign[i] >= 0) replica_id[i] = assign[i];
  for (int32_t r = 0; r < c->n_replicas; r++)
    if (adm_count[r] > 0 && clock[r] < now) clock[r] = now;
}
