// hfx_sim_run: batched trace-driven simulation, one persistent thread block per trace.
//
// A trace is staged once into shared memory; then the block runs the scheduler iteration
// (visible set, aggregates of the running batch, E_d, safe budget, most-urgent-first admission,
// maturity, commit, clock advance) `iters` times without leaving the chip.  Work per iteration
// scales with the live set (queue + running batch), not with the trace length:
//   - rows are sorted by arrival, so the visible queue grows from a head pointer;
//   - the running batch and the strictest SLOs are kept as incremental counters;
//   - a running request's completion iteration is fixed at admission (every iteration with a
//     running batch advances each of its requests by one token);
//   - admission extracts the most urgent eligible request repeatedly (block-wide arg-min on
//     (prio, clamp(slack), req_id)) and stops at the first one that does not fit, which is
//     exactly the prefix-closed rule of the sorted formulation.
// Shared memory is what bounds the number of resident traces, so a row takes 15 bytes: one 8-byte slot
// (arrival, then the slack base while queued, then the finish iteration while running), a word (prompt
// length and priority), a byte (class and state) and one list entry (the queue from the front of the list array, the running batch
// from its back: a row is in one of them at most); the rows
// admitted in an iteration are parked in the part of the queue array that their extraction frees, and the
// running list is kept in place (a finished request's place is filled from the tail).  A scan of the queue is
// only made when the budget reaches the shortest queued prompt (a bound kept beside the queue).
#include "hfx_internal.cuh"

#define SIM_THREADS 128
#define SIM_WARPS (SIM_THREADS / 32)
#define SIM_SMEM_ROWS 10240          // longest trace whose rows are kept in shared memory (15 bytes each); longer ones work in global scratch
#define SIM_BYTES_PER_ROW 15
#define SIM_CLASS_BYTES(nc) ((((size_t)(nc) * 24) + 15) & ~(size_t)15)     // per-class tables in dynamic shared memory: TTFT, TPOT, two counters
#define SIM_HOLES 32                 // finished requests of one iteration whose places in the running list are noted
#define SIM_OUTLEN_CAP (1 << 30)   // output lengths are clamped here when the finish iteration is formed

// the byte of a row: class<6> | state<2>; the word of a row: prompt_len<25> | prio<6>, prio 63 marks a row with bad data
#define ROW_CLS(x) ((x) & 0x3fu)
#define ROW_STATE(x) ((x) >> 6)
#define ROW_BYTE(cls, st) ((uint8_t)((cls) | ((st) << 6)))
#define ROW_PROMPT(w) ((int32_t)((w) & 0x1ffffffu))
#define ROW_PRIO(w) ((w) >> 25)
#define ROW_INVALID_PRIO 63u

struct SimArgs {
  const uint8_t *class_id; const int32_t *prompt_len; const int32_t *output_len; const int64_t *arrival;
  const int32_t *req_id; const int32_t *weight;
  uint8_t *state; int32_t *gen; int64_t *first_token; int64_t *last_token; int64_t *finish;
  const int32_t *trace_off; const hfx_replica_cfg *cfg;
  int32_t n_traces, iters, cap_rows;
  // outputs
  int32_t *iters_executed, *finished, *rejected, *attained;
  int64_t *ttft_p50, *ttft_p99, *tpot_p50, *tpot_p99, *now_out;
};

struct SimShared {
  ReplicaPlan plan;
  int64_t now, mat, sum_kv;
  int64_t t1, t2, lp, mat_next;
  int64_t d_kv;                 // change of sum_kv collected during commit
  int32_t head, head_prev, nq, nr, na, no, arrived;
  int32_t worked, stop, trace, zero_prompt;
  int32_t min_prompt;           // a lower bound of the shortest prompt in the queue: lowered by every arrival, made exact by
                                // every scan of the queue (an admission can only raise the true value)
  int32_t best_min[2][SIM_WARPS];
  int32_t n_holes;              // requests of the running list that finished in this iteration
  uint16_t holes[SIM_HOLES];    // their places in the list (the first SIM_HOLES of them)
  // arg-min scratch, double buffered
  uint64_t best_key[2][SIM_WARPS];
  uint32_t best_id[2][SIM_WARPS];
  int32_t best_slot[2][SIM_WARPS];
  // end-of-trace counters
  int32_t n_fin, n_rej, n_att, n_a, n_b;
};

__device__ __forceinline__ void sort_i64(int64_t *v, int n) {
  int n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  const int half = n_pad >> 1;
  for (int k = 2; k <= n_pad; k <<= 1) {
    const int hk = k >> 1;
    for (int t = threadIdx.x; t < half; t += blockDim.x) {
      const int blk = t / hk, off = t - blk * hk;
      const int i = blk * k + off, j = blk * k + k - 1 - off;
      if (j < n) { const int64_t x = v[i], y = v[j]; if (x > y) { v[i] = y; v[j] = x; } }
    }
    __syncthreads();
    for (int j = k >> 2; j > 0; j >>= 1) {
      for (int t = threadIdx.x; t < half; t += blockDim.x) {
        const int i = 2 * t - (t & (j - 1));
        if (i + j < n) { const int64_t x = v[i], y = v[i + j]; if (x > y) { v[i] = y; v[i + j] = x; } }
      }
      __syncthreads();
    }
  }
}

__device__ __forceinline__ int64_t nearest_rank(const int64_t *sorted, int n, int pct) {
  if (n == 0) return -1;
  int64_t k = ((int64_t)pct * n + 99) / 100;
  if (k < 1) k = 1;
  return sorted[k - 1];
}

// SCRATCH: the per-row arrays of a block live in its part of a global scratch buffer instead of shared memory (traces
// too long for it); the code is the same.
template <bool SCRATCH>
__global__ void __launch_bounds__(SIM_THREADS) k_sim(const HfxParams p, const SimArgs a, uint32_t *__restrict__ work_counter,
                                                     uint32_t *__restrict__ status, unsigned char *__restrict__ scratch) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int cap = a.cap_rows;
  // per class, in front of the rows: TTFT and TPOT bounds, requests in flight, requests in the queue
  const int nc = p.n_classes;
  int64_t *c_ttft = reinterpret_cast<int64_t *>(smem_raw), *c_tpot = c_ttft + nc;
  int32_t *c_run = reinterpret_cast<int32_t *>(c_tpot + nc), *c_q = c_run + nc;
  unsigned char *rows_mem = SCRATCH ? scratch + (size_t)blockIdx.x * cap * SIM_BYTES_PER_ROW : smem_raw + SIM_CLASS_BYTES(nc);
  int64_t *s_arr = reinterpret_cast<int64_t *>(rows_mem);              // arrival; the slack base once arrived; the finish iteration once running; later the TTFT, then the TPOT samples
  uint32_t *s_word = reinterpret_cast<uint32_t *>(s_arr + cap);        // prompt_len | prio << 25
  // One list array for both lists (a row is in one of them at most): from the front the visible queue (row indices,
  // unordered) and behind it the rows admitted in this iteration; from the back the running batch (RUN(s), unordered;
  // 0xffff: a request that just finished)
  uint16_t *s_q = reinterpret_cast<uint16_t *>(s_word + cap);
  uint8_t *s_byte = reinterpret_cast<uint8_t *>(s_q + cap);            // class | state << 6
#define RUN(s) s_q[cap - 1 - (s)]
  __shared__ SimShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (;;) {
    __syncthreads();
    if (tid == 0) S.trace = (int32_t)atomicAdd(work_counter, 1u);
    __syncthreads();
    const int j = S.trace;
    if (j >= a.n_traces) return;
    const int32_t b = a.trace_off[j];
    const int m = a.trace_off[j + 1] - b;
    const hfx_replica_cfg cfg = a.cfg[j];

    // ---- stage the trace ----------------------------------------------------------------
    if (tid == 0) {
      S.now = 0; S.mat = 0; S.sum_kv = 0; S.head = 0; S.head_prev = 0; S.nq = 0; S.nr = 0; S.stop = 0;
      S.n_fin = 0; S.n_rej = 0; S.n_att = 0; S.n_a = 0; S.n_b = 0; S.zero_prompt = 0; S.min_prompt = INT32_MAX; S.n_holes = 0;
      S.arrived = 0; S.no = 0; S.na = 0; S.d_kv = 0;
    }
    __syncthreads();
    for (int c = tid; c < nc; c += SIM_THREADS) { c_run[c] = 0; c_q[c] = 0; c_ttft[c] = p.ttft[c]; c_tpot[c] = p.tpot[c]; }
    uint32_t bad = 0;
    for (int i = tid; i < m; i += SIM_THREADS) {
      const int64_t g = (int64_t)b + i;
      const uint32_t cls = a.class_id[g];
      const int32_t prompt = a.prompt_len[g];
      const int64_t arr = a.arrival[g];
      bool ok = true;
      if (cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
      if (prompt < 0 || prompt > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
      s_arr[i] = arr;
      if (prompt == 0) S.zero_prompt = 1;   // a zero-token prompt fits a zero budget
      uint32_t prio = ROW_INVALID_PRIO;
      if (ok) {
        if (p.weight_max > 0) {
          const int64_t w = (int64_t)p.weight_max - a.weight[g];
          prio = (uint32_t)(w < 0 ? 0 : (w > 62 ? 62 : w));
        } else prio = p.prio[cls];
      }
      s_word[i] = (ok ? (uint32_t)prompt : 0u) | (prio << 25);
      s_byte[i] = ROW_BYTE(ok ? cls : 0u, HFX_QUEUED);
      a.first_token[g] = -1; a.last_token[g] = -1; a.finish[g] = -1;
    }
    if (bad) atomicOr(status, bad);
    // A trace that is not sorted by arrival is a caller error; it is simulated as given (the head
    // pointer stops at the first row that has not arrived) and cannot fault.
    __syncthreads();

    int executed = 0;
    PlanMemo memo;          // of the planning warp: the trace's replica is planned every iteration
    plan_memo_reset(memo);
    for (int it = 0; it < a.iters; it++) {
      // ---- 1. arrivals: rows [head, head + k) with arrival <= now join the queue -----------
      // (the iteration's counters were cleared by the thread that closed the previous one)
      {
        const int64_t now = S.now;
        const int head = S.head;
        int local = 0;
        for (int i = head + tid; i < m && s_arr[i] <= now; i += SIM_THREADS) {
          local++;
          const uint32_t w = s_word[i];
          if (ROW_PRIO(w) == ROW_INVALID_PRIO) continue;
          const uint32_t cls = ROW_CLS(s_byte[i]);
          atomicAdd(&c_q[cls], 1);
          if (ROW_PROMPT(w) > cfg.token_cap) {
            // can never be served: visible for this one iteration, rejected at its commit (which looks through
            // the rows that arrived in the iteration again)
            atomicAdd(&S.no, 1);
          } else {
            const int slot = atomicAdd(&S.nq, 1);
            s_q[slot] = (uint16_t)i;
            atomicMin(&S.min_prompt, (int32_t)ROW_PROMPT(w));
            // from here on the row's slot holds its slack base, ttft_slo + arrival - E_p(prompt_len):
            // the slack at any later decision is the base minus the earliest start
            const int64_t ttft = c_ttft[cls];
            s_arr[i] = ttft > 0 ? ttft + s_arr[i] - dev_Ep(p, ROW_PROMPT(w)) : BASE_UNBOUNDED;
          }
        }
        if (local) atomicAdd(&S.arrived, local);
      }
      __syncthreads();

      // ---- 2. plan: E_d of the running batch and the safe budget (the first warp) ----------------
      if (warp == 0) {
        if (lane == 0) { S.head_prev = S.head; S.head += S.arrived; }
        const uint32_t r0 = __ballot_sync(0xffffffffu, lane < p.n_classes && c_run[lane] > 0);
        const uint32_t r1 = __ballot_sync(0xffffffffu, lane + 32 < p.n_classes && c_run[lane + 32] > 0);
        const uint32_t q0 = __ballot_sync(0xffffffffu, lane < p.n_classes && c_q[lane] > 0);
        const uint32_t q1 = __ballot_sync(0xffffffffu, lane + 32 < p.n_classes && c_q[lane + 32] > 0);
        ReplicaPlan pl0;
        // the budget only matters if it reaches the shortest queued prompt (a queue without requests admits nothing)
        memo.need = S.zero_prompt ? 0 : (S.nq > 0 ? (int64_t)S.min_prompt : (int64_t)cfg.token_cap + 1);
        warp_plan(p, c_ttft, c_tpot, cfg, S.now, S.mat, S.nr, S.sum_kv, ((uint64_t)r1 << 32) | r0, ((uint64_t)q1 << 32) | q0, pl0, lane, &memo);
        if (lane == 0) S.plan = pl0;
      }
      __syncthreads();
      const int64_t budget = S.plan.budget, start = S.plan.start;
      const int nr = S.nr;
      const int32_t min_prompt = S.min_prompt;

      // ---- 3. admission: extract the most urgent request that fits alone, until one fails ----
      int64_t s_cost = 0, adm_cost = 0;
      int s_cnt = 0, adm_cnt = 0;
      int nq = S.nq;
      // (a budget below the shortest queued prompt admits nothing: the scan of the queue would come back empty)
      if ((budget > 0 || S.zero_prompt) && (int64_t)min_prompt <= budget) {
        int buf = 0;
        for (;;) {
          uint64_t bk = ~0ull; uint32_t bid = ~0u; int bslot = -1;
          int32_t lmin = INT32_MAX;
          for (int s = tid; s < nq; s += SIM_THREADS) {
            const int i = s_q[s];
            const uint32_t wd = s_word[i];
            lmin = (int32_t)ROW_PROMPT(wd) < lmin ? (int32_t)ROW_PROMPT(wd) : lmin;
            if ((int64_t)ROW_PROMPT(wd) > (p.first_fit ? budget - adm_cost : budget)) continue;      // first fit: against what is left
            // slack of a queued request: ttft_slo - (start - arrival) - E_p(prompt_len) = base - start
            const int64_t base = s_arr[i];
            const int64_t sl = base != BASE_UNBOUNDED ? dev_clamp_slack(base - start) : HFX_SLACK_MAX;
            const uint64_t k = ((uint64_t)ROW_PRIO(wd) << 40) | (uint64_t)(sl + (INT64_C(1) << 39));
            if (k < bk) { bk = k; bslot = s; bid = ~0u; }
            else if (k == bk) {      // equal keys are rare: only then fetch the request ids that break the tie
              if (bid == ~0u) bid = (uint32_t)__ldg(a.req_id + b + s_q[bslot]) ^ 0x80000000u;
              const uint32_t id = (uint32_t)__ldg(a.req_id + b + i) ^ 0x80000000u;
              if (id < bid) { bid = id; bslot = s; }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const uint64_t k2 = __shfl_xor_sync(0xffffffffu, bk, o);
            uint32_t i2 = __shfl_xor_sync(0xffffffffu, bid, o);
            const int s2 = __shfl_xor_sync(0xffffffffu, bslot, o);
            if (k2 == bk && bslot >= 0 && s2 >= 0 && s2 != bslot) {
              if (bid == ~0u) bid = (uint32_t)__ldg(a.req_id + b + s_q[bslot]) ^ 0x80000000u;
              if (i2 == ~0u) i2 = (uint32_t)__ldg(a.req_id + b + s_q[s2]) ^ 0x80000000u;
            }
            if (k2 < bk || (k2 == bk && i2 < bid)) { bk = k2; bid = i2; bslot = s2; }
          }
          lmin = __reduce_min_sync(0xffffffffu, lmin);
          if (lane == 0) { S.best_key[buf][warp] = bk; S.best_id[buf][warp] = bid; S.best_slot[buf][warp] = bslot; S.best_min[buf][warp] = lmin; }
          __syncthreads();
          if (tid == 0) {      // the shortest prompt of the queue as it stood for this scan
            int32_t mn = S.best_min[buf][0];
#pragma unroll
            for (int w = 1; w < SIM_WARPS; w++) mn = S.best_min[buf][w] < mn ? S.best_min[buf][w] : mn;
            S.min_prompt = mn;
          }
          bk = S.best_key[buf][0]; bid = S.best_id[buf][0]; bslot = S.best_slot[buf][0];
#pragma unroll
          for (int w = 1; w < SIM_WARPS; w++) {
            const uint64_t k2 = S.best_key[buf][w]; uint32_t i2 = S.best_id[buf][w];
            const int s2 = S.best_slot[buf][w];
            if (k2 == bk && bslot >= 0 && s2 >= 0) {
              if (bid == ~0u) bid = (uint32_t)__ldg(a.req_id + b + s_q[bslot]) ^ 0x80000000u;
              if (i2 == ~0u) i2 = (uint32_t)__ldg(a.req_id + b + s_q[s2]) ^ 0x80000000u;
            }
            if (k2 < bk || (k2 == bk && i2 < bid)) { bk = k2; bid = i2; bslot = s2; }
          }
          buf ^= 1;
          if (bslot < 0) break;                       // no eligible request left
          const int i = s_q[bslot];
          const int32_t pr_i = ROW_PROMPT(s_word[i]);
          s_cost += pr_i; s_cnt += 1;
          if (!(s_cost <= budget && (cfg.batch_cap == 0 || nr + s_cnt <= cfg.batch_cap))) break;
          adm_cost += pr_i; adm_cnt += 1;
          __syncthreads();                            // everyone has read s_q[bslot]
          // the queue shrinks by one; the place it frees behind its end takes the admitted row
          if (tid == 0) { s_q[bslot] = s_q[nq - 1]; s_q[nq - 1] = (uint16_t)i; }
          nq -= 1;
          __syncthreads();
        }
      }
      const int nq_adm = nq;      // the rows admitted in this iteration are s_q[nq_adm .. nq_adm + adm_cnt), last admitted first

      // ---- 4. maturity and the iteration's clock -------------------------------------------
      // every thread knows what was admitted, so every thread forms the iteration's two times itself; the
      // new maturity (a division) is left to one thread, beside the commit
      const int64_t t1 = S.now + (adm_cnt > 0 ? dev_Ep(p, adm_cost) : 0);
      const int64_t t2 = t1 + (nr > 0 ? S.plan.e_d : 0);
      if (tid == 0) {
        int64_t lp = 0;
        S.mat_next = dev_maturity_next(p, S.plan, adm_cnt, adm_cost, 0, &lp);
        S.worked = adm_cnt > 0 || nr > 0;
        S.nq = nq; S.na = adm_cnt;
      }

      // ---- 5. commit ---------------------------------------------------------------------------
      int64_t d_kv = 0;
      // running batch: one more token each; a request finishes when gen + 1 reaches output_len
      for (int s = tid; s < nr; s += SIM_THREADS) {
        const int i = RUN(s);
        if (it >= (int32_t)s_arr[i]) {       // gen + 1 reaches output_len in this iteration
          RUN(s) = 0xffffu;                // its place is free
          const int h = atomicAdd(&S.n_holes, 1);
          if (h < SIM_HOLES) S.holes[h] = (uint16_t)s;
          const uint32_t cls = ROW_CLS(s_byte[i]);
          s_byte[i] = ROW_BYTE(cls, HFX_DONE);
          a.finish[(int64_t)b + i] = t2;
          atomicSub(&c_run[cls], 1);
          const int32_t outlen = __ldg(a.output_len + b + i);
          d_kv -= (int64_t)ROW_PROMPT(s_word[i]) + outlen - 2;       // leaves with the context it had before this step
        } else d_kv += 1;
      }
      // admitted requests: first token at t1
      for (int s = tid; s < adm_cnt; s += SIM_THREADS) {
        const int i = s_q[nq_adm + s];
        a.first_token[(int64_t)b + i] = t1;
        const int32_t outlen = __ldg(a.output_len + b + i);
        s_arr[i] = it + (outlen < SIM_OUTLEN_CAP ? outlen : SIM_OUTLEN_CAP) - 1;      // the slot now holds the finish iteration
        const uint32_t cls = ROW_CLS(s_byte[i]);
        atomicSub(&c_q[cls], 1);
        if (outlen <= 1) {
          s_byte[i] = ROW_BYTE(cls, HFX_DONE);
          a.finish[(int64_t)b + i] = t1;
        } else {
          s_byte[i] = ROW_BYTE(cls, HFX_RUNNING);      // (joins the running list below)
          atomicAdd(&c_run[cls], 1);
          d_kv += ROW_PROMPT(s_word[i]);
        }
      }
      // oversize prompts seen for the first time: among the rows that arrived in this iteration
      if (S.no > 0) {
        for (int i = S.head_prev + tid; i < S.head; i += SIM_THREADS) {
          const uint32_t w = s_word[i];
          if (ROW_PRIO(w) != ROW_INVALID_PRIO && ROW_PROMPT(w) > cfg.token_cap) {
            const uint32_t cls = ROW_CLS(s_byte[i]);
            s_byte[i] = ROW_BYTE(cls, HFX_REJECTED);
            atomicSub(&c_q[cls], 1);
          }
        }
      }
      d_kv = warp_sum_i64(d_kv);
      if (lane == 0 && d_kv) atomicAdd(reinterpret_cast<unsigned long long *>(&S.d_kv), (unsigned long long)d_kv);
      __syncthreads();
      if (tid == 0) {
        S.sum_kv += S.d_kv;
        {   // the running list, in place: free places below the new length are filled from the tail, then the
            // admitted requests that go on decoding join (the list has no order)
          int n = S.nr;
          const int k = S.n_holes;
          if (k > 0) {
            if (k <= SIM_HOLES) {
              for (int e = 1; e < k; e++) {      // the noted places in ascending order (k is small)
                const uint16_t x = S.holes[e];
                int f = e - 1;
                while (f >= 0 && S.holes[f] > x) { S.holes[f + 1] = S.holes[f]; f--; }
                S.holes[f + 1] = x;
              }
              int tail = n - 1;
              for (int e = 0; e < k; e++) {
                const int h = S.holes[e];
                while (tail > h && RUN(tail) == 0xffffu) tail--;
                if (h >= tail) break;          // this place and the ones after it lie beyond the new length
                RUN(h) = RUN(tail); tail--;
              }
            } else {                             // many at once: one pass from both ends
              int lo = 0, hi = n - 1;
              for (;;) {
                while (lo < hi && RUN(lo) != 0xffffu) lo++;
                while (hi > lo && RUN(hi) == 0xffffu) hi--;
                if (lo >= hi) break;
                RUN(lo) = RUN(hi); RUN(hi) = 0xffffu;
              }
            }
            n -= k;
          }
          const int na = S.na, q0 = S.nq;
          for (int e = na - 1; e >= 0; e--) {      // from the last parked row down: the list grows towards them and may take
            const int i = s_q[q0 + e];              // the place of a row already read, never of one still to be read
            if ((s_byte[i] >> 6) == HFX_RUNNING) RUN(n++) = (uint16_t)i;
          }
          S.nr = n;
        }
        S.mat = S.mat_next;
        S.arrived = 0; S.no = 0; S.na = 0; S.n_holes = 0; S.d_kv = 0;      // for the next iteration
        if (S.worked) S.now = t2;
        else {
          int64_t ev = HFX_INF;
          if (S.plan.mat > S.plan.now) ev = S.plan.mat;
          int h = S.head;
          while (h < m && ROW_PRIO(s_word[h]) == ROW_INVALID_PRIO) h++;     // rows with bad data never arrive
          if (h < m && s_arr[h] < ev) ev = s_arr[h];
          if (ev == HFX_INF) S.stop = 1; else S.now = ev;
        }
      }
      __syncthreads();
      if (S.stop) break;
      executed++;
    }

    // ---- per-request outputs and per-trace metrics ------------------------------------------
    __syncthreads();
    const int64_t now_final = S.now;
    int fin = 0, rej = 0, att = 0;
    for (int i = tid; i < m; i += SIM_THREADS) {
      const int64_t g = (int64_t)b + i;
      const int st = ROW_STATE(s_byte[i]);
      const bool valid = ROW_PRIO(s_word[i]) != ROW_INVALID_PRIO;
      const uint32_t cls = ROW_CLS(s_byte[i]);
      const int32_t outlen = a.output_len[g];
      int32_t gen = 0;
      int64_t first = -1, last = -1;
      if (st == HFX_RUNNING || st == HFX_DONE) {
        first = a.first_token[g];
        if (st == HFX_DONE) { gen = outlen > 1 ? outlen - 1 : 0; last = a.finish[g]; }
        else {
          const int admit_it = (int32_t)s_arr[i] - (outlen < SIM_OUTLEN_CAP ? outlen : SIM_OUTLEN_CAP) + 1;
          gen = executed - 1 - admit_it;
          last = gen > 0 ? now_final : first;
        }
        a.last_token[g] = last;
      }
      a.state[g] = (uint8_t)st;
      a.gen[g] = gen;
      const int64_t arr = a.arrival[g];      // (the shared-memory slot holds other things by now)
      int64_t ttft = -1;
      if (valid) {
        if (st == HFX_REJECTED) rej++;
        if (st == HFX_RUNNING || st == HFX_DONE) ttft = first - arr;
        if (st == HFX_DONE) {
          fin++;
          const int64_t tp = outlen > 1 ? (last - first) / (outlen - 1) : 0;
          const int64_t ttft_slo = p.ttft[cls], tpot_slo = p.tpot[cls];
          if ((ttft_slo <= 0 || ttft <= ttft_slo) && (tpot_slo <= 0 || tp <= tpot_slo)) att++;
        }
      }
      s_arr[i] = ttft;     // park the TTFT sample; negative = none
    }
    fin = (int)warp_sum_i64(fin); rej = (int)warp_sum_i64(rej); att = (int)warp_sum_i64(att);
    if (lane == 0) { atomicAdd(&S.n_fin, fin); atomicAdd(&S.n_rej, rej); atomicAdd(&S.n_att, att); }
    __syncthreads();
    // Compact the samples (their order is irrelevant before the sort), sort, take the ranks; then the
    // same array takes the TPOT samples.  The arrays are small: one thread compacts serially.
    if (tid == 0) { int k = 0; for (int i = 0; i < m; i++) { const int64_t v = s_arr[i]; if (v >= 0) s_arr[k++] = v; } S.n_a = k; }
    __syncthreads();
    const int na = S.n_a;
    sort_i64(s_arr, na);
    if (tid == 0) { S.t1 = nearest_rank(s_arr, na, 50); S.t2 = nearest_rank(s_arr, na, 99); }
    __syncthreads();
    for (int i = tid; i < m; i += SIM_THREADS) {
      const int64_t g = (int64_t)b + i;
      int64_t tpot = -1;
      if (ROW_STATE(s_byte[i]) == HFX_DONE && ROW_PRIO(s_word[i]) != ROW_INVALID_PRIO) {
        const int32_t outlen = a.output_len[g];
        if (outlen > 1) tpot = (a.finish[g] - a.first_token[g]) / (outlen - 1);
      }
      s_arr[i] = tpot;
    }
    __syncthreads();
    if (tid == 0) { int k = 0; for (int i = 0; i < m; i++) { const int64_t v = s_arr[i]; if (v >= 0) s_arr[k++] = v; } S.n_b = k; }
    __syncthreads();
    const int nb = S.n_b;
    sort_i64(s_arr, nb);
    if (tid == 0) {
      a.iters_executed[j] = executed;
      a.finished[j] = S.n_fin;
      a.rejected[j] = S.n_rej;
      a.attained[j] = S.n_att;
      a.ttft_p50[j] = S.t1;
      a.ttft_p99[j] = S.t2;
      a.tpot_p50[j] = nearest_rank(s_arr, nb, 50);
      a.tpot_p99[j] = nearest_rank(s_arr, nb, 99);
      if (a.now_out) a.now_out[j] = now_final;
    }
  }
}

int hfx_sim_configure() {
  if (cudaFuncSetAttribute(k_sim<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SIM_SMEM_ROWS * SIM_BYTES_PER_ROW + (int)SIM_CLASS_BYTES(HFX_MAX_CLASSES)) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}

void hfx_sim_release(hfx_sched *s) {
  cudaFree(s->d_sim_scratch);
  s->d_sim_scratch = nullptr; s->sim_scratch_bytes = 0;
}

// `trace_off` is already on the device (copied by the caller of this launcher); max_rows is the
// longest trace, known on the host.
int hfx_launch_sim_kernel(hfx_sched *s, const hfx_table *t, const int32_t *d_trace_off, int32_t n_traces,
                          int32_t max_trace_rows, int32_t iters, const hfx_sim_out *o, uint32_t *d_work_counter) {
  SimArgs a;
  a.class_id = t->class_id; a.prompt_len = t->prompt_len; a.output_len = t->output_len; a.arrival = t->arrival_ns;
  a.req_id = t->req_id; a.weight = s->p.weight_max > 0 ? t->weight : nullptr;
  a.state = t->state; a.gen = t->gen; a.first_token = t->first_token_ns; a.last_token = t->last_token_ns;
  a.finish = t->finish_ns; a.trace_off = d_trace_off; a.cfg = s->d_cfg;
  a.n_traces = n_traces; a.iters = iters;
  int cap = (max_trace_rows + 15) & ~15;
  if (cap < 16) cap = 16;
  a.cap_rows = cap;
  a.iters_executed = o->iters_executed; a.finished = o->finished; a.rejected = o->rejected; a.attained = o->attained;
  a.ttft_p50 = o->ttft_p50_ns; a.ttft_p99 = o->ttft_p99_ns; a.tpot_p50 = o->tpot_p50_ns; a.tpot_p99 = o->tpot_p99_ns;
  a.now_out = o->now_ns;
  const size_t rows_bytes = (size_t)cap * SIM_BYTES_PER_ROW, class_bytes = SIM_CLASS_BYTES(s->p.n_classes);
  if (cudaMemsetAsync(d_work_counter, 0, sizeof(uint32_t), s->stream) != cudaSuccess) return HFX_E_CUDA;
  if (cap <= SIM_SMEM_ROWS) {
    int per_sm = (int)((224 * 1024) / (rows_bytes + class_bytes + 1792));      // (static shared memory and the per-block reserve)
    if (per_sm < 1) per_sm = 1;
    if (per_sm > 8) per_sm = 8;
    int grid = s->n_sm * per_sm;
    if (grid > n_traces) grid = n_traces;
    KernelScope ks(s, KSLOT_SIM);
    k_sim<false><<<grid, SIM_THREADS, rows_bytes + class_bytes, s->stream>>>(s->p, a, d_work_counter, s->d_status, nullptr);
  } else {
    // long traces: the rows of every resident block in a scratch buffer (two blocks per SM), allocated when first needed
    int grid = s->n_sm * 2;
    if (grid > n_traces) grid = n_traces;
    const size_t need = rows_bytes * (size_t)grid;
    if (s->sim_scratch_bytes < need) {
      if (cudaStreamSynchronize(s->stream) != cudaSuccess) return HFX_E_CUDA;
      cudaFree(s->d_sim_scratch);
      s->d_sim_scratch = nullptr; s->sim_scratch_bytes = 0;
      if (cudaMalloc(&s->d_sim_scratch, need) != cudaSuccess) { cudaGetLastError(); return HFX_E_NOMEM; }
      s->sim_scratch_bytes = need;
    }
    KernelScope ks(s, KSLOT_SIM);
    k_sim<true><<<grid, SIM_THREADS, class_bytes, s->stream>>>(s->p, a, d_work_counter, s->d_status, s->d_sim_scratch);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
