// hfx_sched_step: one scheduling iteration over the whole request table.
//
// Pipeline (all on one stream, no host synchronisation):
//   k_count     histogram of replica_id                      -> rows per replica
//   k_offsets   exclusive scan, seg_off, work lists by segment size
//   k_regroup   one streaming pass over the table: per-row latency model, slack base,
//               priority; each row becomes a 32-byte record scattered into its replica's
//               range (the only data-permuting pass over HBM)
//   k_segment   one block per replica: aggregates of the running batch, E_d, safe budget
//               (Eq. 3), final slack and key, shared-memory sort by (key, req_id), segmented
//               scan admission, maturity update, optional commit
//   k_big_*     the same for replicas whose rows do not fit in shared memory (global sort)
#include <cooperative_groups.h>

#include "hfx_internal.cuh"

namespace cg = cooperative_groups;

#define SEG_SMALL 2048    // rows a small-segment block sorts in shared memory
#define SEG_MED 16384     // rows a medium-segment block sorts in shared memory
#define THREADS_SMALL 256
#define THREADS_MED 1024
#define HIST_SMEM_MAX 8192

// ------------------------------------------------------------------------------------------------
// k_count: rows per replica.  Bad replica ids go to bucket R and raise a status bit.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) k_count(const int32_t *__restrict__ replica_id, int64_t n, int32_t R,
                                               uint32_t *__restrict__ seg_count, uint32_t *__restrict__ status) {
  extern __shared__ uint32_t hist[];
  const bool use_smem = R + 1 <= HIST_SMEM_MAX;
  if (use_smem) {
    for (int i = threadIdx.x; i <= R; i += blockDim.x) hist[i] = 0;
    __syncthreads();
  }
  uint32_t bad = 0;
  const int64_t n4 = n >> 2;
  const int4 *rid4 = reinterpret_cast<const int4 *>(replica_id);
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
    const int4 r = __ldg(rid4 + v);
    const int rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; k++) {
      int b = rr[k];
      if (b < 0 || b >= R) { b = R; bad = 1; }
      if (use_smem) atomicAdd(&hist[b], 1u); else atomicAdd(&seg_count[b], 1u);
    }
  }
  if (blockIdx.x == 0) {
    for (int64_t i = (n4 << 2) + threadIdx.x; i < n; i += blockDim.x) {
      int b = replica_id[i];
      if (b < 0 || b >= R) { b = R; bad = 1; }
      if (use_smem) atomicAdd(&hist[b], 1u); else atomicAdd(&seg_count[b], 1u);
    }
  }
  if (bad) atomicOr(status, HFX_ST_BAD_REPLICA);
  if (use_smem) {
    __syncthreads();
    for (int i = threadIdx.x; i <= R; i += blockDim.x) {
      const uint32_t c = hist[i];
      if (c) atomicAdd(&seg_count[i], c);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// k_offsets: exclusive scan of the counts (one block), user-visible seg_off, fill cursors and
// the work lists of small / medium / oversize segments.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) k_offsets(const uint32_t *__restrict__ seg_count, int32_t R,
                                                  uint32_t *__restrict__ seg_begin, uint32_t *__restrict__ cursor,
                                                  int32_t *__restrict__ seg_off, int32_t *__restrict__ list,
                                                  uint32_t *__restrict__ list_n) {
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  if (threadIdx.x < 4) list_n[threadIdx.x] = 0;
  __syncthreads();
  const int total = R + 1;  // buckets 0..R
  for (int base = 0; base < total; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const uint32_t c = i < total ? seg_count[i] : 0;
    uint32_t v = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
      uint32_t w = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { uint32_t x = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += x; }
      warp_tot[lane] = w;
    }
    __syncthreads();
    const uint32_t excl = carry_s + (warp ? warp_tot[warp - 1] : 0) + v - c;
    if (i < total) {
      seg_begin[i] = excl;
      cursor[i] = excl;
      seg_off[i] = (int32_t)excl;   // seg_off[R] = number of rows bound to a valid replica
      if (c > 0 || i < R) {   // replicas without rows still get their budget and clock
        const int cls = c <= SEG_SMALL ? 0 : (c <= SEG_MED ? 1 : 2);
        const uint32_t slot = atomicAdd(&list_n[cls], 1u);
        list[(size_t)cls * (R + 1) + slot] = i;
      }
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = excl + c;
    __syncthreads();
  }
  if (threadIdx.x == 0) seg_begin[total] = carry_s;
}

// ------------------------------------------------------------------------------------------------
// k_regroup: the streaming pass.  Each thread takes 4 consecutive rows with 16-byte loads,
// evaluates what does not depend on the replica's aggregates (prefill model of the prompt,
// slack base, priority), and scatters one record per row into the replica's range.
// ------------------------------------------------------------------------------------------------
struct RegroupArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len;
  const int32_t *output_len; const int32_t *gen; const int64_t *arrival; const int64_t *first_token;
  const int32_t *req_id; const int32_t *weight;
  const int64_t *now; const int64_t *mat; const hfx_replica_cfg *cfg;
  int64_t *pred_ttft;    // optional output
  int64_t n;
};

__device__ __forceinline__ void regroup_row(const HfxParams &p, const RegroupArgs &a, const int64_t *s_ttft,
                                            const int64_t *s_tpot, const uint8_t *s_prio, int64_t i, int32_t rid,
                                            uint32_t cls, uint32_t st, int32_t prompt, int32_t gen, int64_t arrival,
                                            int64_t first_token, int32_t req_id, int32_t weight, int32_t out_len,
                                            uint32_t *cursor, HfxRec *rec, uint32_t &bad) {
  const int32_t R = p.n_replicas;
  HfxRec r;
  r.req_id = req_id; r.row = (int32_t)i; r.prompt = prompt; r.gen = gen; r.output_len = out_len;
  r.cls = (uint8_t)cls; r.kind = KIND_DEAD; r.prio = 63; r.pad = 0; r.base = 0;
  int64_t pred_ttft = 0;
  int bucket = rid;
  if (rid < 0 || rid >= R) bucket = R;   // status bit already raised by k_count
  else {
    bool ok = true;
    if (cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
    if (prompt < 0 || prompt > HFX_MAX_TOKENS || gen < 0 || gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
    if (ok) {
      const int64_t now = __ldg(a.now + rid), mat = __ldg(a.mat + rid);
      const int32_t mode = __ldg(&a.cfg[rid].mode);
      const int64_t start = now > mat ? now : mat;
      int prio;
      if (p.weight_max > 0) {
        const int64_t w = (int64_t)p.weight_max - weight;
        prio = (int)(w < 0 ? 0 : (w > 62 ? 62 : w));
      } else prio = s_prio[cls];
      const int64_t ttft = s_ttft[cls], tpot = s_tpot[cls];
      if (st == HFX_RUNNING) {
        r.kind = KIND_RUNNING; r.prio = (uint8_t)prio;
        r.base = tpot > 0 ? first_token + ((int64_t)gen + 1) * tpot - now : BASE_UNBOUNDED;
        pred_ttft = first_token - arrival;
      } else if (st == HFX_QUEUED) {
        if (arrival <= now) {
          r.kind = KIND_QUEUED; r.prio = (uint8_t)prio;
          if (mode == HFX_DECODE) {
            r.base = tpot > 0 ? first_token + ((int64_t)gen + 1) * tpot - start - p.d2 * ((int64_t)prompt + gen) : BASE_UNBOUNDED;
            pred_ttft = first_token - arrival;
          } else {
            pred_ttft = (start - arrival) + dev_Ep(p, prompt);
            r.base = ttft > 0 ? ttft - pred_ttft : BASE_UNBOUNDED;
          }
        } else {
          r.kind = KIND_FUTURE;
          r.base = arrival;
        }
      }
    }
  }
  if (a.pred_ttft) a.pred_ttft[i] = pred_ttft;
  const uint32_t pos = atomicAdd(&cursor[bucket], 1u);
  // two 16-byte stores
  uint4 *dst = reinterpret_cast<uint4 *>(rec + pos);
  const uint4 *src = reinterpret_cast<const uint4 *>(&r);
  dst[0] = src[0];
  dst[1] = src[1];
}

__global__ void __launch_bounds__(256) k_regroup(const HfxParams p, const RegroupArgs a, uint32_t *__restrict__ cursor,
                                                 HfxRec *__restrict__ rec, uint32_t *__restrict__ status) {
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  for (int c = threadIdx.x; c < HFX_MAX_CLASSES; c += blockDim.x) {
    s_ttft[c] = c < p.n_classes ? p.ttft[c] : 0;
    s_tpot[c] = c < p.n_classes ? p.tpot[c] : 0;
    s_prio[c] = c < p.n_classes ? p.prio[c] : 63;
  }
  __syncthreads();
  uint32_t bad = 0;
  const int64_t n4 = a.n >> 2;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
    const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + v);
    const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + v);
    const uchar4 st = __ldg(reinterpret_cast<const uchar4 *>(a.state) + v);
    const int4 pr = __ldg(reinterpret_cast<const int4 *>(a.prompt_len) + v);
    const int4 ge = __ldg(reinterpret_cast<const int4 *>(a.gen) + v);
    const int4 id = __ldg(reinterpret_cast<const int4 *>(a.req_id) + v);
    const longlong2 ar0 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * v);
    const longlong2 ar1 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * v + 1);
    const longlong2 ft0 = __ldg(reinterpret_cast<const longlong2 *>(a.first_token) + 2 * v);
    const longlong2 ft1 = __ldg(reinterpret_cast<const longlong2 *>(a.first_token) + 2 * v + 1);
    int4 we = make_int4(0, 0, 0, 0), ol = make_int4(0, 0, 0, 0);
    if (a.weight) we = __ldg(reinterpret_cast<const int4 *>(a.weight) + v);
    if (a.output_len) ol = __ldg(reinterpret_cast<const int4 *>(a.output_len) + v);
    const int64_t i0 = v << 2;
    regroup_row(p, a, s_ttft, s_tpot, s_prio, i0 + 0, rid.x, cls.x, st.x, pr.x, ge.x, ar0.x, ft0.x, id.x, we.x, ol.x, cursor, rec, bad);
    regroup_row(p, a, s_ttft, s_tpot, s_prio, i0 + 1, rid.y, cls.y, st.y, pr.y, ge.y, ar0.y, ft0.y, id.y, we.y, ol.y, cursor, rec, bad);
    regroup_row(p, a, s_ttft, s_tpot, s_prio, i0 + 2, rid.z, cls.z, st.z, pr.z, ge.z, ar1.x, ft1.x, id.z, we.z, ol.z, cursor, rec, bad);
    regroup_row(p, a, s_ttft, s_tpot, s_prio, i0 + 3, rid.w, cls.w, st.w, pr.w, ge.w, ar1.y, ft1.y, id.w, we.w, ol.w, cursor, rec, bad);
  }
  if (blockIdx.x == 0) {   // ragged tail, scalar
    for (int64_t i = (n4 << 2) + threadIdx.x; i < a.n; i += blockDim.x)
      regroup_row(p, a, s_ttft, s_tpot, s_prio, i, a.replica_id[i], a.class_id[i], a.state[i], a.prompt_len[i], a.gen[i],
                  a.arrival[i], a.first_token[i], a.req_id[i], a.weight ? a.weight[i] : 0,
                  a.output_len ? a.output_len[i] : 0, cursor, rec, bad);
  }
  if (bad) atomicOr(status, bad);
}

// ------------------------------------------------------------------------------------------------
// k_segment: one block per replica (taken from a work list), everything after the regroup.
// ------------------------------------------------------------------------------------------------
struct SegArgs {
  // table columns written by COMMIT
  uint8_t *state; int32_t *gen; int64_t *first_token; int64_t *last_token; int64_t *finish;
  // replica state
  int64_t *now; int64_t *mat; const hfx_replica_cfg *cfg;
  // outputs
  int64_t *slack; int64_t *pred_tpot; uint64_t *key; int32_t *order; uint8_t *admit; int32_t *admitted_rows;
  int64_t *budget; int64_t *e_d; int32_t *n_run; int64_t *sum_kv; int64_t *adm_cost; int32_t *adm_count;
  int64_t *maturity_next;
  uint32_t flags;
};

struct BlockShared {
  int64_t red_a[32], red_b[32], red_c[32];
  uint64_t red_m0[32], red_m1[32];
  ReplicaPlan plan;
  int64_t carry_cost, carry_kv;
  int32_t carry_count;
  int64_t adm_cost, adm_kv, t1, t2, next_arrival;
  int32_t adm_count, worked;
};

// ascending compare-exchange on (hi, lo)
__device__ __forceinline__ void cmp_swap(uint64_t *hi, uint32_t *lo, int i, int j) {
  const uint64_t hi_i = hi[i], hi_j = hi[j];
  const uint32_t lo_i = lo[i], lo_j = lo[j];
  if (hi_i > hi_j || (hi_i == hi_j && lo_i > lo_j)) {
    hi[i] = hi_j; hi[j] = hi_i;
    lo[i] = lo_j; lo[j] = lo_i;
  }
}

// Bitonic sorting network with ascending comparators only, so that the virtual +inf padding
// beyond n never moves: any n, in place, no ties between distinct items (req_id is unique).
__device__ void block_sort(uint64_t *hi, uint32_t *lo, int n) {
  int n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  const int half = n_pad >> 1;
  for (int k = 2; k <= n_pad; k <<= 1) {
    const int hk = k >> 1;
    for (int t = threadIdx.x; t < half; t += blockDim.x) {
      const int blk = t / hk, off = t - blk * hk;
      const int i = blk * k + off, j = blk * k + k - 1 - off;
      if (j < n) cmp_swap(hi, lo, i, j);
    }
    __syncthreads();
    for (int j = k >> 2; j > 0; j >>= 1) {
      for (int t = threadIdx.x; t < half; t += blockDim.x) {
        const int i = 2 * t - (t & (j - 1));
        if (i + j < n) cmp_swap(hi, lo, i, i + j);
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(1024) k_segment(const HfxParams p, const SegArgs a, const HfxRec *__restrict__ rec,
                          const uint32_t *__restrict__ seg_begin, const int32_t *__restrict__ list,
                          const uint32_t *__restrict__ list_n, int seg_cap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t *s_hi = reinterpret_cast<uint64_t *>(smem_raw);
  uint32_t *s_lo = reinterpret_cast<uint32_t *>(smem_raw + (size_t)seg_cap * 8);
  __shared__ BlockShared sh;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int R = p.n_replicas;
  const uint32_t n_work = *list_n;

  for (uint32_t w = blockIdx.x; w < n_work; w += gridDim.x) {
    const int r = list[w];
    const uint32_t b = seg_begin[r];
    const int n = (int)(seg_begin[r + 1] - b);
    const HfxRec *seg = rec + b;
    const bool real = r < R;    // bucket R holds rows bound to no replica

    // ---- aggregates of the running batch and the strictest SLOs present -------------------
    int64_t n_run = 0, sum_kv = 0, next_arr = HFX_INF;
    uint64_t m_run = 0, m_q = 0;
    for (int q = threadIdx.x; q < n; q += blockDim.x) {
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);   // prompt, gen, output_len, bytes
      const int kind = (w1.w >> 8) & 0xff, cls = w1.w & 0xff;
      if (kind == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(int32_t)w1.x + (int32_t)w1.y; m_run |= 1ull << cls; }
      else if (kind == KIND_QUEUED) m_q |= 1ull << cls;
      else if (kind == KIND_FUTURE) { const int64_t arr = seg[q].base; next_arr = arr < next_arr ? arr : next_arr; }
    }
    n_run = warp_sum_i64(n_run); sum_kv = warp_sum_i64(sum_kv); next_arr = warp_min_i64(next_arr);
    m_run = warp_or_u64(m_run); m_q = warp_or_u64(m_q);
    if (lane == 0) { sh.red_a[warp] = n_run; sh.red_b[warp] = sum_kv; sh.red_c[warp] = next_arr; sh.red_m0[warp] = m_run; sh.red_m1[warp] = m_q; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int k = 1; k < nwarp; k++) {
        n_run += sh.red_a[k]; sum_kv += sh.red_b[k];
        next_arr = sh.red_c[k] < next_arr ? sh.red_c[k] : next_arr;
        m_run |= sh.red_m0[k]; m_q |= sh.red_m1[k];
      }
      hfx_replica_cfg cfg; cfg.mode = HFX_COLOCATED; cfg.token_cap = 1; cfg.batch_cap = 0;
      int64_t now = 0, mat = 0;
      if (real) { cfg = a.cfg[r]; now = a.now[r]; mat = a.mat[r]; }
      dev_plan(p, cfg, now, mat, n_run, sum_kv, m_run, m_q, sh.plan);
      sh.next_arrival = next_arr;
      sh.carry_cost = 0; sh.carry_kv = 0; sh.carry_count = 0;
      sh.adm_cost = 0; sh.adm_kv = 0; sh.adm_count = 0;
    }
    __syncthreads();
    const ReplicaPlan pl = sh.plan;

    // ---- final slack, key, sort items -----------------------------------------------------
    for (int q = threadIdx.x; q < n; q += blockDim.x) {
      const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + q));
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
      const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
      const int32_t req_id = (int32_t)w0.z, row = (int32_t)w0.w;
      const int32_t prompt = (int32_t)w1.x, gen = (int32_t)w1.y;
      const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
      int64_t slack = 0, pred_tpot = 0;
      int phase = PH_INACTIVE, kprio = 63;
      int64_t kslack = HFX_SLACK_MAX;
      if (kind == KIND_RUNNING) {
        phase = PH_RUNNING; kprio = prio;
        slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - pl.shift_run;
        pred_tpot = pl.e_d; kslack = slack;
      } else if (kind == KIND_QUEUED) {
        phase = PH_QUEUED; kprio = prio;
        pred_tpot = pl.shift_dq + p.d2 * ((int64_t)prompt + gen);
        if (pl.mode == HFX_DECODE) slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - pl.shift_dq;
        else slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base;
        kslack = slack;
      }
      const uint64_t k48 = dev_key48(phase, kprio, kslack);
      const uint32_t uid = (uint32_t)req_id ^ 0x80000000u;      // signed order as unsigned
      s_hi[q] = (k48 << 16) | (uid >> 16);
      s_lo[q] = (uid << 16) | (uint32_t)q;
      a.slack[row] = slack;
      if (a.pred_tpot) a.pred_tpot[row] = pred_tpot;
      if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | k48;
    }
    __syncthreads();

    block_sort(s_hi, s_lo, n);

    // ---- admission: segmented scan along the order ---------------------------------------
    for (int tile = 0; tile < n; tile += blockDim.x) {
      const int q = tile + threadIdx.x;
      int64_t cost = 0, kv = 0;
      int32_t cnt = 0, row = -1, kind = KIND_DEAD;
      if (q < n) {
        const int li = s_lo[q] & 0xffff;
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
        const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
        row = (int32_t)w0.w;
        kind = (w1.w >> 8) & 0xff;
        if (kind == KIND_QUEUED) {
          kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
          const int64_t c = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
          if (c <= pl.budget) { cost = c; cnt = 1; } else kv = 0;
        }
        a.order[b + q] = row;
      }
      // block-wide inclusive scan of (cost, cnt) with carry
      int64_t sc = warp_incl_scan_i64(cost, lane);
      int32_t sn = warp_incl_scan_i32(cnt, lane);
      if (lane == 31) { sh.red_a[warp] = sc; sh.red_b[warp] = sn; }
      __syncthreads();
      if (warp == 0) {
        int64_t x = lane < nwarp ? sh.red_a[lane] : 0;
        int32_t y = lane < nwarp ? (int32_t)sh.red_b[lane] : 0;
        x = warp_incl_scan_i64(x, lane); y = warp_incl_scan_i32(y, lane);
        sh.red_a[lane] = x; sh.red_b[lane] = y;
      }
      __syncthreads();
      const int64_t pre_c = sh.carry_cost + (warp ? sh.red_a[warp - 1] : 0);
      const int32_t pre_n = sh.carry_count + (warp ? (int32_t)sh.red_b[warp - 1] : 0);
      sc += pre_c; sn += pre_n;
      bool adm = false;
      if (cnt) adm = sc <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + sn <= pl.batch_cap);
      if (q < n) {
        a.admit[row] = (uint8_t)((kind == KIND_RUNNING || adm) ? 1 : 0);
        if (adm && a.admitted_rows) a.admitted_rows[b + sn - 1] = row;
        s_lo[q] = (s_lo[q] & 0xffffu) | (adm ? 0x10000u : 0u);   // keep the decision for the commit pass
      }
      // totals over admitted rows (admission is prefix-closed, so a block reduction suffices)
      int64_t ac = adm ? cost : 0, ak = adm ? kv : 0;
      int32_t an = adm ? 1 : 0;
      ac = warp_sum_i64(ac); ak = warp_sum_i64(ak); an = (int32_t)warp_sum_i64(an);
      __syncthreads();     // everyone has read red_a / red_b / carry
      if (lane == 0) { sh.red_a[warp] = ac; sh.red_b[warp] = ak; sh.red_c[warp] = an; }
      if (threadIdx.x == blockDim.x - 1) { sh.carry_cost = sc; sh.carry_count = sn; }
      __syncthreads();
      if (threadIdx.x == 0) {
        for (int k = 0; k < nwarp; k++) { sh.adm_cost += sh.red_a[k]; sh.adm_kv += sh.red_b[k]; sh.adm_count += (int32_t)sh.red_c[k]; }
      }
      __syncthreads();
    }

    // ---- maturity, per-replica outputs, commit decisions --------------------------------
    if (threadIdx.x == 0) {
      int64_t lp = 0;
      const int64_t mat_next = dev_maturity_next(p, pl, sh.adm_count, sh.adm_cost, sh.adm_kv, &lp);
      int worked; int64_t t1 = pl.now, t2 = pl.now;
      if (pl.mode == HFX_COLOCATED) {
        worked = sh.adm_count > 0 || pl.n_run > 0;
        t1 = pl.now + (sh.adm_count > 0 ? lp : 0);
        t2 = t1 + (pl.n_run > 0 ? pl.e_d : 0);
      } else if (pl.mode == HFX_PREFILL) {
        worked = sh.adm_count > 0;
        t1 = t2 = pl.now + (sh.adm_count > 0 ? lp : 0);
      } else {
        worked = pl.now >= pl.mat && pl.n_run + sh.adm_count > 0;
        t2 = worked ? mat_next : pl.now;
      }
      sh.worked = worked; sh.t1 = t1; sh.t2 = t2;
      if (real) {
        a.budget[r] = pl.budget;
        if (a.e_d) a.e_d[r] = pl.e_d;
        if (a.n_run) a.n_run[r] = (int32_t)pl.n_run;
        if (a.sum_kv) a.sum_kv[r] = pl.sum_kv;
        a.adm_cost[r] = sh.adm_cost;
        a.adm_count[r] = sh.adm_count;
        a.maturity_next[r] = mat_next;
        if (a.flags & HFX_COMMIT) {
          int64_t now_next = pl.now;
          if (worked) now_next = t2;
          else {
            int64_t ev = HFX_INF;
            if (pl.mat > pl.now) ev = pl.mat;
            if (sh.next_arrival < ev) ev = sh.next_arrival;
            if (ev != HFX_INF) now_next = ev;
          }
          a.now[r] = now_next;
          a.mat[r] = mat_next;
        }
      }
    }
    __syncthreads();

    // ---- second pass: compacted list padding and commit ---------------------------------
    const bool commit = real && (a.flags & HFX_COMMIT);
    if (a.admitted_rows || commit) {
      const int adm_count = sh.adm_count, worked = sh.worked;
      const int64_t t1 = sh.t1, t2 = sh.t2;
      for (int q = threadIdx.x; q < n; q += blockDim.x) {
        if (a.admitted_rows && q >= adm_count) a.admitted_rows[b + q] = -1;
        if (!commit) continue;
        const uint32_t lo = s_lo[q];
        const int li = lo & 0xffff;
        const bool adm = (lo & 0x10000u) != 0;
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
        const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
        const int32_t row = (int32_t)w0.w, prompt = (int32_t)w1.x, gen = (int32_t)w1.y, out_len = (int32_t)w1.z;
        const int kind = (w1.w >> 8) & 0xff;
        if (kind == KIND_RUNNING) {
          if (pl.mode == HFX_PREFILL || (pl.mode == HFX_DECODE && !worked)) continue;
          a.gen[row] = gen + 1;
          a.last_token[row] = t2;
          if ((int64_t)gen + 2 >= out_len) { a.state[row] = HFX_DONE; a.finish[row] = t2; }
        } else if (kind == KIND_QUEUED) {
          if (adm) {
            uint8_t st = HFX_RUNNING;
            if (pl.mode == HFX_DECODE) {
              a.gen[row] = gen + 1;
              a.last_token[row] = t2;
              if ((int64_t)gen + 2 >= out_len) { st = HFX_DONE; a.finish[row] = t2; }
            } else {
              a.gen[row] = 0;
              a.first_token[row] = t1;
              a.last_token[row] = t1;
              if (out_len <= 1) { st = HFX_DONE; a.finish[row] = t1; }
            }
            a.state[row] = st;
          } else if (pl.mode != HFX_DECODE && prompt > pl.token_cap) {
            a.state[row] = HFX_REJECTED;
          }
        }
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// Oversize segments (more rows than a block can sort in shared memory): one cooperative kernel.
// Blocks share the work of each oversize replica: aggregates and keys by block 0 of the grid in a
// loop, sort by a global bitonic network with grid barriers, admission by one block walking the
// order with a carried prefix.  Slow but exact; it only exists so that any table is handled.
// ------------------------------------------------------------------------------------------------
struct BigShared {
  ReplicaPlan plan;
  int64_t red_a[32], red_b[32], red_c[32];
  uint64_t red_m0[32], red_m1[32];
  int64_t carry_cost, adm_cost, adm_kv, t1, t2, next_arrival;
  int32_t carry_count, adm_count, worked;
};

// Bounded grid barrier (all blocks of a cooperative launch are resident).  Returns false if the
// wait ran out; the caller then raises HFX_ST_TIMEOUT and leaves.
__device__ bool grid_barrier(uint32_t *bar, uint32_t *status, uint32_t &epoch) {
  __syncthreads();
  __shared__ int ok_s;
  if (threadIdx.x == 0) {
    epoch++;
    __threadfence();
    const uint32_t target = epoch * gridDim.x;
    atomicAdd(bar, 1u);
    int ok = 0;
    for (long long spin = 0; spin < (1ll << 26); spin++) {
      if (*((volatile uint32_t *)bar) >= target) { ok = 1; break; }
      if (*((volatile uint32_t *)status) & HFX_ST_TIMEOUT) break;
      __nanosleep(64);
    }
    if (!ok) atomicOr(status, HFX_ST_TIMEOUT);
    __threadfence();
    ok_s = ok;
  }
  __syncthreads();
  return ok_s != 0;
}

__global__ void __launch_bounds__(512) k_big(const HfxParams p, const SegArgs a, const HfxRec *__restrict__ rec,
                                             const uint32_t *__restrict__ seg_begin, const int32_t *__restrict__ list,
                                             const uint32_t *__restrict__ list_n, uint64_t *__restrict__ g_hi,
                                             uint32_t *__restrict__ g_lo, uint32_t *__restrict__ g_idx,
                                             uint32_t *bar, uint32_t *status) {
  __shared__ BigShared sh;
  const uint32_t n_work = *list_n;
  if (n_work == 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int R = p.n_replicas;
  uint32_t epoch = 0;
  const int64_t gtid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t gsize = (int64_t)gridDim.x * blockDim.x;

  for (uint32_t w = 0; w < n_work; w++) {
    const int r = list[w];
    const uint32_t b = seg_begin[r];
    const int64_t n = (int64_t)(seg_begin[r + 1] - b);
    const HfxRec *seg = rec + b;
    const bool real = r < R;
    uint64_t *hi = g_hi + b;
    uint32_t *lo = g_lo + b, *idx = g_idx + b;

    // every block computes the aggregates redundantly (reads come from L2 after the first)
    int64_t n_run = 0, sum_kv = 0, next_arr = HFX_INF;
    uint64_t m_run = 0, m_q = 0;
    for (int64_t q = threadIdx.x; q < n; q += blockDim.x) {
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
      const int kind = (w1.w >> 8) & 0xff, cls = w1.w & 0xff;
      if (kind == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(int32_t)w1.x + (int32_t)w1.y; m_run |= 1ull << cls; }
      else if (kind == KIND_QUEUED) m_q |= 1ull << cls;
      else if (kind == KIND_FUTURE) { const int64_t arr = seg[q].base; next_arr = arr < next_arr ? arr : next_arr; }
    }
    n_run = warp_sum_i64(n_run); sum_kv = warp_sum_i64(sum_kv); next_arr = warp_min_i64(next_arr);
    m_run = warp_or_u64(m_run); m_q = warp_or_u64(m_q);
    if (lane == 0) { sh.red_a[warp] = n_run; sh.red_b[warp] = sum_kv; sh.red_c[warp] = next_arr; sh.red_m0[warp] = m_run; sh.red_m1[warp] = m_q; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int k = 1; k < nwarp; k++) {
        n_run += sh.red_a[k]; sum_kv += sh.red_b[k];
        next_arr = sh.red_c[k] < next_arr ? sh.red_c[k] : next_arr;
        m_run |= sh.red_m0[k]; m_q |= sh.red_m1[k];
      }
      hfx_replica_cfg cfg; cfg.mode = HFX_COLOCATED; cfg.token_cap = 1; cfg.batch_cap = 0;
      int64_t now = 0, mat = 0;
      if (real) { cfg = a.cfg[r]; now = a.now[r]; mat = a.mat[r]; }
      dev_plan(p, cfg, now, mat, n_run, sum_kv, m_run, m_q, sh.plan);
      sh.next_arrival = next_arr;
      sh.carry_cost = 0; sh.carry_count = 0; sh.adm_cost = 0; sh.adm_kv = 0; sh.adm_count = 0;
    }
    __syncthreads();
    const ReplicaPlan pl = sh.plan;

    // keys, spread over the grid
    for (int64_t q = gtid; q < n; q += gsize) {
      const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + q));
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
      const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
      const int32_t req_id = (int32_t)w0.z, row = (int32_t)w0.w;
      const int32_t prompt = (int32_t)w1.x, gen = (int32_t)w1.y;
      const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
      int64_t slack = 0, pred_tpot = 0, kslack = HFX_SLACK_MAX;
      int phase = PH_INACTIVE, kprio = 63;
      if (kind == KIND_RUNNING) {
        phase = PH_RUNNING; kprio = prio;
        slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - pl.shift_run;
        pred_tpot = pl.e_d; kslack = slack;
      } else if (kind == KIND_QUEUED) {
        phase = PH_QUEUED; kprio = prio;
        pred_tpot = pl.shift_dq + p.d2 * ((int64_t)prompt + gen);
        if (pl.mode == HFX_DECODE) slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - pl.shift_dq;
        else slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base;
        kslack = slack;
      }
      const uint64_t k48 = dev_key48(phase, kprio, kslack);
      hi[q] = k48;
      lo[q] = (uint32_t)req_id ^ 0x80000000u;
      idx[q] = (uint32_t)q;
      a.slack[row] = slack;
      if (a.pred_tpot) a.pred_tpot[row] = pred_tpot;
      if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | k48;
    }
    if (!grid_barrier(bar, status, epoch)) return;

    // global bitonic network (ascending comparators, virtual padding), idx travels with the item
    int64_t n_pad = 1;
    while (n_pad < n) n_pad <<= 1;
    const int64_t half = n_pad >> 1;
    for (int64_t k = 2; k <= n_pad; k <<= 1) {
      const int64_t hk = k >> 1;
      for (int64_t t = gtid; t < half; t += gsize) {
        const int64_t blk = t / hk, off = t - blk * hk;
        const int64_t i = blk * k + off, j = blk * k + k - 1 - off;
        if (j < n) {
          const uint64_t hi_i = hi[i], hi_j = hi[j];
          const uint32_t lo_i = lo[i], lo_j = lo[j];
          if (hi_i > hi_j || (hi_i == hi_j && lo_i > lo_j)) {
            hi[i] = hi_j; hi[j] = hi_i; lo[i] = lo_j; lo[j] = lo_i;
            const uint32_t x = idx[i]; idx[i] = idx[j]; idx[j] = x;
          }
        }
      }
      if (!grid_barrier(bar, status, epoch)) return;
      for (int64_t j = k >> 2; j > 0; j >>= 1) {
        for (int64_t t = gtid; t < half; t += gsize) {
          const int64_t i = 2 * t - (t & (j - 1));
          if (i + j < n) {
            const uint64_t hi_i = hi[i], hi_j = hi[i + j];
            const uint32_t lo_i = lo[i], lo_j = lo[i + j];
            if (hi_i > hi_j || (hi_i == hi_j && lo_i > lo_j)) {
              hi[i] = hi_j; hi[i + j] = hi_i; lo[i] = lo_j; lo[i + j] = lo_i;
              const uint32_t x = idx[i]; idx[i] = idx[i + j]; idx[i + j] = x;
            }
          }
        }
        if (!grid_barrier(bar, status, epoch)) return;
      }
    }

    // admission walk by block 0 with a carried prefix, then commit by the whole grid
    if (blockIdx.x == 0) {
      for (int64_t tile = 0; tile < n; tile += blockDim.x) {
        const int64_t q = tile + threadIdx.x;
        int64_t cost = 0, kv = 0;
        int32_t cnt = 0, row = -1, kind = KIND_DEAD;
        if (q < n) {
          const uint32_t li = idx[q];
          const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
          const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
          row = (int32_t)w0.w;
          kind = (w1.w >> 8) & 0xff;
          if (kind == KIND_QUEUED) {
            kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
            const int64_t c = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
            if (c <= pl.budget) { cost = c; cnt = 1; } else kv = 0;
          }
          a.order[b + q] = row;
        }
        int64_t sc = warp_incl_scan_i64(cost, lane);
        int32_t sn = warp_incl_scan_i32(cnt, lane);
        if (lane == 31) { sh.red_a[warp] = sc; sh.red_b[warp] = sn; }
        __syncthreads();
        if (warp == 0) {
          int64_t x = lane < nwarp ? sh.red_a[lane] : 0;
          int32_t y = lane < nwarp ? (int32_t)sh.red_b[lane] : 0;
          x = warp_incl_scan_i64(x, lane); y = warp_incl_scan_i32(y, lane);
          sh.red_a[lane] = x; sh.red_b[lane] = y;
        }
        __syncthreads();
        sc += sh.carry_cost + (warp ? sh.red_a[warp - 1] : 0);
        sn += sh.carry_count + (warp ? (int32_t)sh.red_b[warp - 1] : 0);
        bool adm = false;
        if (cnt) adm = sc <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + sn <= pl.batch_cap);
        if (q < n) {
          a.admit[row] = (uint8_t)((kind == KIND_RUNNING || adm) ? 1 : 0);
          if (adm && a.admitted_rows) a.admitted_rows[b + sn - 1] = row;
          lo[q] = adm ? 1u : 0u;      // the sort is over: lo now carries the decision
        }
        int64_t ac = adm ? cost : 0, ak = adm ? kv : 0;
        int32_t an = adm ? 1 : 0;
        ac = warp_sum_i64(ac); ak = warp_sum_i64(ak); an = (int32_t)warp_sum_i64(an);
        __syncthreads();
        if (lane == 0) { sh.red_a[warp] = ac; sh.red_b[warp] = ak; sh.red_c[warp] = an; }
        if (threadIdx.x == blockDim.x - 1) { sh.carry_cost = sc; sh.carry_count = sn; }
        __syncthreads();
        if (threadIdx.x == 0)
          for (int k = 0; k < nwarp; k++) { sh.adm_cost += sh.red_a[k]; sh.adm_kv += sh.red_b[k]; sh.adm_count += (int32_t)sh.red_c[k]; }
        __syncthreads();
      }
      if (threadIdx.x == 0) {
        int64_t lp = 0;
        const int64_t mat_next = dev_maturity_next(p, pl, sh.adm_count, sh.adm_cost, sh.adm_kv, &lp);
        int worked; int64_t t1 = pl.now, t2 = pl.now;
        if (pl.mode == HFX_COLOCATED) {
          worked = sh.adm_count > 0 || pl.n_run > 0;
          t1 = pl.now + (sh.adm_count > 0 ? lp : 0);
          t2 = t1 + (pl.n_run > 0 ? pl.e_d : 0);
        } else if (pl.mode == HFX_PREFILL) {
          worked = sh.adm_count > 0;
          t1 = t2 = pl.now + (sh.adm_count > 0 ? lp : 0);
        } else {
          worked = pl.now >= pl.mat && pl.n_run + sh.adm_count > 0;
          t2 = worked ? mat_next : pl.now;
        }
        // hand the decisions to the other blocks through the head of the sort scratch's
        // barrier area: words 2.. of `bar`
        volatile int64_t *mail = reinterpret_cast<volatile int64_t *>(bar + 4);
        mail[0] = t1; mail[1] = t2; mail[2] = worked; mail[3] = sh.adm_count;
        if (real) {
          a.budget[r] = pl.budget;
          if (a.e_d) a.e_d[r] = pl.e_d;
          if (a.n_run) a.n_run[r] = (int32_t)pl.n_run;
          if (a.sum_kv) a.sum_kv[r] = pl.sum_kv;
          a.adm_cost[r] = sh.adm_cost;
          a.adm_count[r] = sh.adm_count;
          a.maturity_next[r] = mat_next;
          if (a.flags & HFX_COMMIT) {
            int64_t now_next = pl.now;
            if (worked) now_next = t2;
            else {
              int64_t ev = HFX_INF;
              if (pl.mat > pl.now) ev = pl.mat;
              if (sh.next_arrival < ev) ev = sh.next_arrival;
              if (ev != HFX_INF) now_next = ev;
            }
            a.now[r] = now_next;
            a.mat[r] = mat_next;
          }
        }
      }
    }
    if (!grid_barrier(bar, status, epoch)) return;
    {
      volatile int64_t *mail = reinterpret_cast<volatile int64_t *>(bar + 4);
      const int64_t t1 = mail[0], t2 = mail[1];
      const int worked = (int)mail[2], adm_count = (int)mail[3];
      const bool commit = real && (a.flags & HFX_COMMIT);
      for (int64_t q = gtid; q < n; q += gsize) {
        if (a.admitted_rows && q >= adm_count) a.admitted_rows[b + q] = -1;
        if (!commit) continue;
        const bool adm = lo[q] != 0;
        const uint32_t li = idx[q];
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
        const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
        const int32_t row = (int32_t)w0.w, prompt = (int32_t)w1.x, gen = (int32_t)w1.y, out_len = (int32_t)w1.z;
        const int kind = (w1.w >> 8) & 0xff;
        if (kind == KIND_RUNNING) {
          if (pl.mode == HFX_PREFILL || (pl.mode == HFX_DECODE && !worked)) continue;
          a.gen[row] = gen + 1;
          a.last_token[row] = t2;
          if ((int64_t)gen + 2 >= out_len) { a.state[row] = HFX_DONE; a.finish[row] = t2; }
        } else if (kind == KIND_QUEUED) {
          if (adm) {
            uint8_t st = HFX_RUNNING;
            if (pl.mode == HFX_DECODE) {
              a.gen[row] = gen + 1;
              a.last_token[row] = t2;
              if ((int64_t)gen + 2 >= out_len) { st = HFX_DONE; a.finish[row] = t2; }
            } else {
              a.gen[row] = 0;
              a.first_token[row] = t1;
              a.last_token[row] = t1;
              if (out_len <= 1) { st = HFX_DONE; a.finish[row] = t1; }
            }
            a.state[row] = st;
          } else if (pl.mode != HFX_DECODE && prompt > pl.token_cap) {
            a.state[row] = HFX_REJECTED;
          }
        }
      }
    }
    if (!grid_barrier(bar, status, epoch)) return;
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
int hfx_launch_step(hfx_sched *s, const hfx_table *t, const hfx_replica_state *st, const hfx_step_out *o,
                    uint32_t flags) {
  const int R = s->p.n_replicas;
  const int64_t n = t->n_rows;
  cudaStream_t stream = s->stream;

  if (cudaMemsetAsync(s->d_seg_count, 0, sizeof(uint32_t) * (R + 2), stream) != cudaSuccess) return HFX_E_CUDA;
  if (o->admitted_rows == nullptr) { /* nothing to pre-fill */ }

  const int grid_stream = s->n_sm * 4;
  {
    const size_t sm = (R + 1 <= HIST_SMEM_MAX) ? sizeof(uint32_t) * (R + 1) : 0;
    KernelScope ks(s, KSLOT_COUNT);
    k_count<<<grid_stream, 512, sm, stream>>>(t->replica_id, n, R, s->d_seg_count, s->d_status);
  }
  {
    KernelScope ks(s, KSLOT_OFFSETS);
    k_offsets<<<1, 1024, 0, stream>>>(s->d_seg_count, R, s->d_seg_begin, s->d_cursor, o->seg_off, s->d_list, s->d_list_n);
  }
  {
    RegroupArgs a;
    a.replica_id = t->replica_id; a.class_id = t->class_id; a.state = t->state; a.prompt_len = t->prompt_len;
    a.output_len = t->output_len; a.gen = t->gen; a.arrival = t->arrival_ns; a.first_token = t->first_token_ns;
    a.req_id = t->req_id; a.weight = s->p.weight_max > 0 ? t->weight : nullptr;
    a.now = st->now_ns; a.mat = st->maturity_ns; a.cfg = s->d_cfg; a.pred_ttft = o->pred_ttft_ns; a.n = n;
    KernelScope ks(s, KSLOT_REGROUP);
    k_regroup<<<s->n_sm * 8, 256, 0, stream>>>(s->p, a, s->d_cursor, s->d_rec, s->d_status);
  }
  SegArgs sa;
  sa.state = t->state; sa.gen = t->gen; sa.first_token = t->first_token_ns; sa.last_token = t->last_token_ns;
  sa.finish = t->finish_ns; sa.now = st->now_ns; sa.mat = st->maturity_ns; sa.cfg = s->d_cfg;
  sa.slack = o->slack_ns; sa.pred_tpot = o->pred_tpot_ns; sa.key = o->key; sa.order = o->order; sa.admit = o->admit;
  sa.admitted_rows = o->admitted_rows; sa.budget = o->budget; sa.e_d = o->e_d_ns; sa.n_run = o->n_run;
  sa.sum_kv = o->sum_kv; sa.adm_cost = o->adm_cost; sa.adm_count = o->adm_count; sa.maturity_next = o->maturity_next;
  sa.flags = flags;
  {
    const int grid = R + 1 < s->n_sm * 8 ? R + 1 : s->n_sm * 8;
    KernelScope ks(s, KSLOT_SEG_SMALL);
    k_segment<<<grid, THREADS_SMALL, SEG_SMALL * 12, stream>>>(s->p, sa, s->d_rec, s->d_seg_begin, s->d_list,
                                                                s->d_list_n, SEG_SMALL);
  }
  if (n > SEG_SMALL) {
    const int grid = R + 1 < s->n_sm ? R + 1 : s->n_sm;
    KernelScope ks(s, KSLOT_SEG_MED);
    k_segment<<<grid, THREADS_MED, SEG_MED * 12, stream>>>(s->p, sa, s->d_rec, s->d_seg_begin, s->d_list + (R + 1),
                                                            s->d_list_n + 1, SEG_MED);
  }
  if (n > SEG_MED) {
    const int32_t *list = s->d_list + 2 * (size_t)(R + 1);
    const uint32_t *list_n = s->d_list_n + 2;
    uint32_t *big_idx = reinterpret_cast<uint32_t *>(s->d_big_lo + s->max_rows);
    if (cudaMemsetAsync(s->d_barrier, 0, 64, stream) != cudaSuccess) return HFX_E_CUDA;
    void *args[] = {(void *)&s->p, (void *)&sa, (void *)&s->d_rec, (void *)&s->d_seg_begin, (void *)&list,
                    (void *)&list_n, (void *)&s->d_big_hi, (void *)&s->d_big_lo, (void *)&big_idx,
                    (void *)&s->d_barrier, (void *)&s->d_status};
    KernelScope ks(s, KSLOT_BIG);
    if (cudaLaunchCooperativeKernel((void *)k_big, dim3(s->n_sm), dim3(512), args, 0, stream) != cudaSuccess)
      return HFX_E_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}

int hfx_step_configure() {
  if (cudaFuncSetAttribute(k_segment, cudaFuncAttributeMaxDynamicSharedMemorySize, SEG_MED * 12) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}
