// Per-replica work after the regroup: aggregates of the running batch, E_d, the safe budget
// (Eq. 3), final slack and key, the sort, segmented-scan admission, maturity, commit.
//   k_segment  one block per replica whose rows fit in shared memory (two size classes)
//   k_big      cooperative kernel for larger replicas (global sort with bounded grid barriers)
#include "hfx_internal.cuh"

#define SEG_SMALL 2048    // rows a small-segment block sorts in shared memory
#define SEG_MED 16384     // rows a medium-segment block sorts in shared memory
#define THREADS_SMALL 256
#define TINY_BLOCKS_PER_SM 4
#define THREADS_MED 1024
#define SMEM_SMALL (SEG_SMALL * 20 + (2 * 1024 + 8) * 4)   // sort items, their order, scatter buffer, bins

struct BlockShared {
  int64_t red_a[32], red_b[32], red_c[32];
  uint64_t red_m0[32], red_m1[32];
  int32_t red_n[32];
  ReplicaPlan plan;
  int64_t carry_cost;
  int32_t carry_count, carry_act, carry_inact;
  int64_t adm_cost, adm_kv, t1, t2, next_arrival;
  int32_t adm_count, worked, n_act;
};

// Distribution sort of distinct 64-bit items for small segments: items are binned by their offset
// from the smallest item (a shift makes at most SORT_BINS bins, so bins are in key order), scattered
// bin by bin, and ranked inside their bin by counting smaller items.  Writes the low 16 bits of the
// items, in ascending item order, to s_lo.  Returns false (uniformly, nothing written) when a bin is
// too crowded for the counting to pay; the caller then runs the sorting network instead.
// Needs blockDim.x <= SORT_BINS and SORT_BINS % blockDim.x == 0.  Block-synchronised on entry by the
// caller and on return.
#define SORT_BINS 1024
#define SORT_BIN_MAX 48
__device__ bool block_bucket_order(const uint64_t *s_hi, uint64_t *s_tmp, uint32_t *s_lo, uint32_t *s_bin,
                                   uint32_t *s_cur, int n, BlockShared &sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  uint64_t mn = ~0ull, mx = 0;
  for (int q = threadIdx.x; q < n; q += blockDim.x) { const uint64_t v = s_hi[q]; mn = v < mn ? v : mn; mx = v > mx ? v : mx; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const uint64_t a = __shfl_xor_sync(0xffffffffu, mn, o), b = __shfl_xor_sync(0xffffffffu, mx, o);
    mn = a < mn ? a : mn; mx = b > mx ? b : mx;
  }
  if (lane == 0) { sh.red_m0[warp] = mn; sh.red_m1[warp] = mx; }
  for (int i = threadIdx.x; i <= SORT_BINS; i += blockDim.x) s_bin[i] = 0;
  __syncthreads();
  for (int k = 0; k < nwarp; k++) { const uint64_t a = sh.red_m0[k], b = sh.red_m1[k]; mn = a < mn ? a : mn; mx = b > mx ? b : mx; }
  const uint64_t range = mx - mn;
  int sft = 0;
  if (range >> 10) sft = 64 - __clzll((long long)range) - 10;     // (range >> sft) < SORT_BINS
  for (int q = threadIdx.x; q < n; q += blockDim.x) atomicAdd(&s_bin[(uint32_t)((s_hi[q] - mn) >> sft)], 1u);
  __syncthreads();
  // exclusive scan of the bin counts; the largest bin
  const int per = SORT_BINS / blockDim.x;
  const int i0 = threadIdx.x * per;
  uint32_t sum = 0, big = 0;
  for (int i = 0; i < per; i++) { const uint32_t c = s_bin[i0 + i]; sum += c; big = c > big ? c : big; }
  uint32_t v = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const uint32_t x = __shfl_xor_sync(0xffffffffu, big, o); big = x > big ? x : big; }
  if (lane == 31) sh.red_n[warp] = (int32_t)v;
  if (lane == 0) sh.red_a[warp] = big;
  __syncthreads();
  uint32_t pre = 0, bigall = 0;
  for (int k = 0; k < nwarp; k++) { if (k < warp) pre += (uint32_t)sh.red_n[k]; const uint32_t x = (uint32_t)sh.red_a[k]; bigall = x > bigall ? x : bigall; }
  if (bigall > SORT_BIN_MAX) { __syncthreads(); return false; }
  uint32_t run = pre + v - sum;
  for (int i = 0; i < per; i++) { const uint32_t c = s_bin[i0 + i]; s_bin[i0 + i] = run; s_cur[i0 + i] = run; run += c; }
  __syncthreads();
  for (int q = threadIdx.x; q < n; q += blockDim.x) {
    const uint64_t x = s_hi[q];
    s_tmp[atomicAdd(&s_cur[(uint32_t)((x - mn) >> sft)], 1u)] = x;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < n; e += blockDim.x) {
    const uint64_t x = s_tmp[e];
    const uint32_t b = (uint32_t)((x - mn) >> sft);
    const uint32_t g0 = s_bin[b], g1 = s_cur[b];
    uint32_t rank = 0;
    for (uint32_t g = g0; g < g1; g++) rank += s_tmp[g] < x ? 1u : 0u;
    s_lo[g0 + rank] = (uint32_t)(x & 0xffffu);
  }
  __syncthreads();
  return true;
}

// what a record says about its row once the replica's plan is known
struct RowEval { int64_t slack, pred_tpot; uint64_t k48; int phase; };

__device__ __forceinline__ RowEval eval_row(const HfxParams &p, const ReplicaPlan &pl, int64_t base, int kind, int prio,
                                            int32_t prompt, int32_t gen) {
  RowEval e;
  e.slack = 0; e.pred_tpot = 0; e.phase = PH_INACTIVE;
  int kprio = 63;
  int64_t kslack = HFX_SLACK_MAX;
  if (kind == KIND_RUNNING) {
    e.phase = PH_RUNNING; kprio = prio;
    e.slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - pl.shift_run;
    e.pred_tpot = pl.e_d; kslack = e.slack;
  } else if (kind == KIND_QUEUED) {
    e.phase = PH_QUEUED; kprio = prio;
    e.pred_tpot = pl.tpot_q0 + p.d2 * ((int64_t)prompt + gen);
    e.slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - pl.shift_q;
    kslack = e.slack;
  }
  e.k48 = dev_key48(e.phase, kprio, kslack);
  return e;
}

// iteration clock of a replica once its admission is known (the commit rules)
__device__ __forceinline__ void iteration_clock(const ReplicaPlan &pl, int32_t adm_count, int64_t lp, int64_t mat_next,
                                                int &worked, int64_t &t1, int64_t &t2) {
  t1 = pl.now; t2 = pl.now;
  if (pl.mode == HFX_COLOCATED) {
    worked = adm_count > 0 || pl.n_run > 0;
    t1 = pl.now + (adm_count > 0 ? lp : 0);
    t2 = t1 + (pl.n_run > 0 ? pl.e_d : 0);
  } else if (pl.mode == HFX_PREFILL) {
    worked = adm_count > 0;
    t1 = t2 = pl.now + (adm_count > 0 ? lp : 0);
  } else {
    worked = pl.now >= pl.mat && pl.n_run + adm_count > 0;
    t2 = worked ? mat_next : pl.now;
  }
}

__device__ __forceinline__ void write_replica_outputs(const SegArgs &a, int r, const ReplicaPlan &pl, int64_t adm_cost,
                                                      int32_t adm_count, int64_t mat_next, int worked, int64_t t2,
                                                      int64_t next_arrival) {
  a.budget[r] = pl.budget;
  if (a.e_d) a.e_d[r] = pl.e_d;
  if (a.n_run) a.n_run[r] = (int32_t)pl.n_run;
  if (a.sum_kv) a.sum_kv[r] = pl.sum_kv;
  a.adm_cost[r] = adm_cost;
  a.adm_count[r] = adm_count;
  a.maturity_next[r] = mat_next;
  if ((a.flags & HFX_COMMIT) && pl.now <= a.horizon) {
    int64_t now_next = pl.now;
    if (worked) now_next = t2;
    else {   // idle: jump to the next event, if any
      int64_t ev = HFX_INF;
      if (pl.mat > pl.now) ev = pl.mat;
      if (next_arrival < ev) ev = next_arrival;
      if (ev != HFX_INF) now_next = ev;
    }
    a.now[r] = now_next;
    a.mat[r] = mat_next;
  }
}

// the table update of one row at commit
__device__ __forceinline__ void commit_row(const SegArgs &a, const ReplicaPlan &pl, int kind, bool adm, int worked,
                                           int64_t t1, int64_t t2, int32_t row, int32_t prompt, int32_t gen, int32_t out_len) {
  if (kind == KIND_RUNNING) {
    if (pl.mode == HFX_PREFILL || (pl.mode == HFX_DECODE && !worked)) return;
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

// where a kernel finds the regrouped table
struct SegCtx {
  const HfxRec *rec; const uint32_t *seg_begin; const uint32_t *tot_act; const uint32_t *flags;
  const uint8_t *rowflag; uint32_t parity;
};

// Earliest arrival among a replica's rows that have not arrived yet, for the clock jump of an idle
// replica in an ordered step: the regroup has listed the replica's inactive rows in
// order[b + n_act .. b + n); their kind bytes say which of them are still to come.
__device__ __forceinline__ int64_t next_arrival_listed(const SegArgs &a, const SegCtx &c, uint32_t b, int64_t n_act, int64_t n,
                                                       int64_t first, int64_t stride) {
  int64_t v = HFX_INF;
  for (int64_t q = n_act + first; q < n; q += stride) {
    const int32_t row = a.order[b + q];
    if (c.rowflag[row] == KIND_FUTURE) { const int64_t x = a.arrival[row]; v = x < v ? x : v; }
  }
  return v;
}

// aggregates of a replica's active records into the block's plan (all threads call; result in
// sh.plan; sh.next_arrival is left at "none")
__device__ __forceinline__ void segment_plan(const HfxParams &p, const SegArgs &a, const HfxRec *seg, int64_t n_act, int r,
                                             bool real, BlockShared &sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  int64_t n_run = 0, sum_kv = 0;
  uint64_t m_run = 0, m_q = 0;
  for (int64_t q = threadIdx.x; q < n_act; q += blockDim.x) {
    const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);   // prompt, gen, output_len, bytes
    const int kind = (w1.w >> 8) & 0xff, cls = w1.w & 0xff;
    if (kind == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(int32_t)w1.x + (int32_t)w1.y; m_run |= 1ull << cls; }
    else m_q |= 1ull << cls;
  }
  n_run = warp_sum_i64(n_run); sum_kv = warp_sum_i64(sum_kv);
  m_run = warp_or_u64(m_run); m_q = warp_or_u64(m_q);
  if (lane == 0) { sh.red_a[warp] = n_run; sh.red_b[warp] = sum_kv; sh.red_m0[warp] = m_run; sh.red_m1[warp] = m_q; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < nwarp; k++) { n_run += sh.red_a[k]; sum_kv += sh.red_b[k]; m_run |= sh.red_m0[k]; m_q |= sh.red_m1[k]; }
    hfx_replica_cfg cfg; cfg.mode = HFX_COLOCATED; cfg.token_cap = 1; cfg.batch_cap = 0;
    int64_t now = 0, mat = 0;
    if (real) { cfg = a.cfg[r]; now = a.now[r]; mat = a.mat[r]; }
    dev_plan(p, cfg, now, mat, n_run, sum_kv, m_run, m_q, sh.plan);
    sh.next_arrival = HFX_INF;
    sh.carry_cost = 0; sh.carry_count = 0;
    sh.adm_cost = 0; sh.adm_kv = 0; sh.adm_count = 0;
  }
  __syncthreads();
}

// block-wide minimum into sh.next_arrival (all threads call)
__device__ __forceinline__ void block_min_arrival(int64_t v, BlockShared &sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  v = warp_min_i64(v);
  __syncthreads();
  if (lane == 0) sh.red_c[warp] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    int64_t m = sh.next_arrival;
    for (int k = 0; k < nwarp; k++) m = sh.red_c[k] < m ? sh.red_c[k] : m;
    sh.next_arrival = m;
  }
  __syncthreads();
}


// Block-wide admission over the sorted items s_lo[0..n_sorted) (low 16 bits = position of the
// record inside the segment): writes order, admit and the compacted admitted list, keeps each
// decision in bit 16 of s_lo, accumulates the totals in sh.
__device__ __forceinline__ void segment_admit(const HfxParams &p, const SegArgs &a, const ReplicaPlan &pl,
                                              const HfxRec *seg, uint32_t b, uint32_t *s_lo, int n_sorted,
                                              BlockShared &sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  if (p.first_fit) {       // the first warp walks the order and marks what it takes (bit 17)
    if (warp == 0) {
      const int64_t room = pl.batch_cap == 0 ? HFX_INF : (pl.batch_cap > pl.n_eff ? pl.batch_cap - pl.n_eff : 0);
      warp_first_fit(n_sorted, pl.budget, room, lane,
                     [&](int64_t q) -> int64_t {
                       const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + (s_lo[q] & 0xffffu)) + 1);
                       if (((w1.w >> 8) & 0xff) != KIND_QUEUED) return -1;
                       return pl.mode == HFX_DECODE ? p.d1 + p.d2 * ((int64_t)(int32_t)w1.x + (int32_t)w1.y) : (int64_t)(int32_t)w1.x;
                     },
                     [&](int64_t q, bool taken) { if (taken) s_lo[q] |= 0x20000u; });
    }
    __syncthreads();
  }
  // The order begins with the requests in flight (phase 0 sorts first): they are listed and marked, no
  // prefix is needed for them.  Whole tiles of them are passed here; the scan starts at the tile that
  // reaches the queue.
  const int n_front = (int)((pl.n_run < n_sorted ? pl.n_run : n_sorted) / blockDim.x) * blockDim.x;
  for (int q = threadIdx.x; q < n_front; q += blockDim.x) {
    const uint32_t li = s_lo[q] & 0xffffu;
    const int32_t row = (int32_t)__ldg(reinterpret_cast<const uint4 *>(seg + li)).w;
    a.order[b + q] = row;
    a.admit[row] = 1;
    s_lo[q] = li;
  }
  for (int tile = n_front; tile < n_sorted; tile += blockDim.x) {
    const int q = tile + threadIdx.x;
    int64_t cost = 0, kv = 0;
    int32_t cnt = 0, row = -1, kind = KIND_DEAD;
    if (q < n_sorted) {
      const int li = s_lo[q] & 0xffff;
      const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
      row = (int32_t)w0.w;
      kind = (w1.w >> 8) & 0xff;
      if (kind == KIND_QUEUED) {
        kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
        const int64_t c = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
        if (p.first_fit ? (s_lo[q] & 0x20000u) != 0 : c <= pl.budget) { cost = c; cnt = 1; } else kv = 0;
      }
      a.order[b + q] = row;
    }
    if (!__syncthreads_or(cnt)) {      // no candidate in this tile (a spent budget, requests in flight): nothing to add up
      if (q < n_sorted) {
        if (kind == KIND_RUNNING) a.admit[row] = 1;
        s_lo[q] &= 0xffffu;
      }
      continue;
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
    sc += sh.carry_cost + (warp ? sh.red_a[warp - 1] : 0);
    sn += sh.carry_count + (warp ? (int32_t)sh.red_b[warp - 1] : 0);
    bool adm = false;
    if (cnt) adm = p.first_fit || (sc <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + sn <= pl.batch_cap));
    if (q < n_sorted) {
      if (kind == KIND_RUNNING || adm) a.admit[row] = 1;
      if (adm && a.admitted_rows) a.admitted_rows[b + sn - 1] = row;
      s_lo[q] = (s_lo[q] & 0xffffu) | (adm ? 0x10000u : 0u);
    }
    // totals over admitted rows (admission is prefix-closed, so a block reduction suffices)
    int64_t ac = adm ? cost : 0, ak = adm ? kv : 0;
    int32_t an = adm ? 1 : 0;
    ac = warp_sum_i64(ac); ak = warp_sum_i64(ak); an = (int32_t)warp_sum_i64(an);
    __syncthreads();     // everyone has read red_a / red_b / carry
    if (lane == 0) { sh.red_a[warp] = ac; sh.red_b[warp] = ak; sh.red_c[warp] = an; }
    if (threadIdx.x == blockDim.x - 1) { sh.carry_cost = sc; sh.carry_count = sn; sh.carry_act = kind == KIND_QUEUED; }
    __syncthreads();
    if (threadIdx.x == 0)
      for (int k = 0; k < nwarp; k++) { sh.adm_cost += sh.red_a[k]; sh.adm_kv += sh.red_b[k]; sh.adm_count += (int32_t)sh.red_c[k]; }
    __syncthreads();
    // Admission along the order is closed under prefixes: once the running cost is over the budget, or the
    // batch is full, nothing behind is admitted; and once the order has reached the queue, nothing behind is
    // in flight.  The rest of the order then only has to be written out.
    if (!p.first_fit && sh.carry_act &&
        (sh.carry_cost > pl.budget || (pl.batch_cap != 0 && pl.n_eff + sh.carry_count >= pl.batch_cap))) {
      for (int q = tile + blockDim.x + threadIdx.x; q < n_sorted; q += blockDim.x) {
        const uint32_t li = s_lo[q] & 0xffffu;
        a.order[b + q] = (int32_t)__ldg(reinterpret_cast<const uint4 *>(seg + li)).w;
        s_lo[q] = li;
      }
      break;
    }
  }
}

// The sorting network of block_sort for items of one 64-bit word (ordered steps), with the items held in
// registers: thread t of the 1024 owns the items IPT*t .. IPT*t + IPT-1 (IPT * 1024 = the padded length).
// Every pair of the network is (i, i ^ mask): mask = k-1 in the mirrored first sub-stage of merge size k,
// a single bit j afterwards; the lower index keeps the smaller item.  Masks below IPT stay inside a
// thread (no memory traffic), thread distances below 32 go through warp shuffles, the rest (15 of the
// 105 sub-stages at 16384 items) through shared memory, striped by item slot so that neither side has
// bank conflicts.  `hi` holds the items on entry and is the exchange buffer afterwards; on return
// pos_out[i] is the low 16 bits (the item's tie-break position) of the i-th smallest item.
// The block is synchronised on entry by the caller; the caller synchronises before reading pos_out.
__device__ __forceinline__ void cx64(uint64_t &a, uint64_t &b) {
  const uint64_t lo = a < b ? a : b, hi = a < b ? b : a;
  a = lo; b = hi;
}

template <int IPT>
__device__ void block_sort_reg(uint64_t *hi, uint32_t *pos_out, int n) {
  const int t = threadIdx.x;
  uint64_t v[IPT];
#pragma unroll
  for (int e = 0; e < IPT; e++) { const int i = t * IPT + e; v[e] = i < n ? hi[i] : ~UINT64_C(0); }
  __syncthreads();
  // merge sizes up to IPT: inside the thread
#pragma unroll
  for (int k = 2; k <= IPT; k <<= 1) {
#pragma unroll
    for (int e = 0; e < IPT; e++) if (e < (e ^ (k - 1))) cx64(v[e], v[e ^ (k - 1)]);
#pragma unroll
    for (int j = k >> 2; j > 0; j >>= 1)
#pragma unroll
      for (int e = 0; e < IPT; e++) if (!(e & j)) cx64(v[e], v[e | j]);
  }
  // merge sizes kt * IPT: kt threads per merged run
  for (int kt = 2; kt <= 1024; kt <<= 1) {
    {   // mirrored sub-stage: partner thread t ^ (kt-1), partner slot IPT-1-e
      const int mt = kt - 1;
      const bool lower = (t & (kt >> 1)) == 0;
      if (mt < 32) {
#pragma unroll
        for (int e = 0; e < (IPT + 1) / 2; e++) {
          const int f = IPT - 1 - e;
          const uint64_t pa = __shfl_xor_sync(0xffffffffu, v[f], mt);     // the partner's slot f pairs with my slot e
          const uint64_t pb = __shfl_xor_sync(0xffffffffu, v[e], mt);     // and its slot e with my slot f
          v[e] = lower ? (v[e] < pa ? v[e] : pa) : (v[e] < pa ? pa : v[e]);
          if (f != e) v[f] = lower ? (v[f] < pb ? v[f] : pb) : (v[f] < pb ? pb : v[f]);
        }
      } else {
#pragma unroll
        for (int e = 0; e < IPT; e++) hi[e * 1024 + t] = v[e];
        __syncthreads();
#pragma unroll
        for (int e = 0; e < IPT; e++) {
          const uint64_t w = hi[(IPT - 1 - e) * 1024 + (t ^ mt)];
          v[e] = lower ? (v[e] < w ? v[e] : w) : (v[e] < w ? w : v[e]);
        }
        __syncthreads();
      }
    }
    for (int jt = kt >> 2; jt > 0; jt >>= 1) {     // partner thread t ^ jt, same slot
      const bool lower = (t & jt) == 0;
      if (jt < 32) {
#pragma unroll
        for (int e = 0; e < IPT; e++) {
          const uint64_t w = __shfl_xor_sync(0xffffffffu, v[e], jt);
          v[e] = lower ? (v[e] < w ? v[e] : w) : (v[e] < w ? w : v[e]);
        }
      } else {
#pragma unroll
        for (int e = 0; e < IPT; e++) hi[e * 1024 + t] = v[e];
        __syncthreads();
#pragma unroll
        for (int e = 0; e < IPT; e++) {
          const uint64_t w = hi[e * 1024 + (t ^ jt)];
          v[e] = lower ? (v[e] < w ? v[e] : w) : (v[e] < w ? w : v[e]);
        }
        __syncthreads();
      }
    }
#pragma unroll
    for (int j = IPT >> 1; j > 0; j >>= 1)          // the remaining distances are inside the thread
#pragma unroll
      for (int e = 0; e < IPT; e++) if (!(e & j)) cx64(v[e], v[e | j]);
  }
#pragma unroll
  for (int e = 0; e < IPT; e++) { const int i = t * IPT + e; if (i < n) pos_out[i] = (uint32_t)(v[e] & 0xffffu); }
}

// Sort n distinct 64-bit items (block-synchronised on entry) and write their low 16 bits, in ascending item
// order, to pos_out; the caller synchronises before reading pos_out.  1024-thread blocks keep the items in
// registers (1, 2, 4, 8 or 16 per thread) for more than 512 items.
__device__ __forceinline__ void sort64_positions(uint64_t *hi, uint32_t *pos_out, int n) {
  if (blockDim.x == 1024 && n > 512) {
    if (n <= 1024) block_sort_reg<1>(hi, pos_out, n);
    else if (n <= 2048) block_sort_reg<2>(hi, pos_out, n);
    else if (n <= 4096) block_sort_reg<4>(hi, pos_out, n);
    else if (n <= 8192) block_sort_reg<8>(hi, pos_out, n);
    else block_sort_reg<16>(hi, pos_out, n);
  } else {
    block_sort<false>(hi, nullptr, n);
    for (int q = threadIdx.x; q < n; q += blockDim.x) pos_out[q] = (uint32_t)(hi[q] & 0xffffu);
  }
}

__global__ void __launch_bounds__(1024) k_segment(const HfxParams p, const SegArgs a, const SegCtx c, int seg_min,
                                                  int seg_cap, int bucket) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t *s_hi = reinterpret_cast<uint64_t *>(smem_raw);
  uint32_t *s_lo = reinterpret_cast<uint32_t *>(smem_raw + (size_t)seg_cap * 8);
  // only with `bucket`: scratch of the distribution sort
  uint64_t *s_tmp = reinterpret_cast<uint64_t *>(smem_raw + (size_t)seg_cap * 12);
  uint32_t *s_bin = reinterpret_cast<uint32_t *>(smem_raw + (size_t)seg_cap * 20);
  uint32_t *s_cur = s_bin + SORT_BINS + 4;
  __shared__ BlockShared sh;
  const int R = p.n_replicas;
  if (c.flags[2] < (uint32_t)seg_min) return;     // no replica of this kernel's size class exists
  const bool ordered = c.flags[c.parity] != 0;

  for (int r = blockIdx.x; r <= R; r += gridDim.x) {
    const uint32_t b = c.seg_begin[r];
    const int n = (int)(c.seg_begin[r + 1] - b);
    const int n_act = (int)c.tot_act[r];
    const int n_in = n - n_act;
    const int need = ordered ? n_act : (n_act > n_in ? n_act : n_in);
    if (need < seg_min || need > seg_cap) continue;
    if (r == R && n == 0) continue;
    const HfxRec *seg = c.rec + b;
    const bool real = r < R;    // bucket R holds rows bound to no replica

    // ---- inactive rows of a step that is not ordered: listed by req_id behind the active ones ----
    if (!ordered && n_in > 0) {
      const HfxRec *sin = seg + n_act;
      int64_t next_arr = HFX_INF;
      for (int q = threadIdx.x; q < n_in; q += blockDim.x) {
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(sin + q));
        const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(sin + q) + 1);
        if (((w1.w >> 8) & 0xff) == KIND_FUTURE) { const int64_t arr = (int64_t)(((uint64_t)w0.y << 32) | w0.x); next_arr = arr < next_arr ? arr : next_arr; }
        s_hi[q] = ((uint64_t)(w0.z ^ 0x80000000u) << 16) | (uint32_t)q;     // signed req_id order, then position
      }
      __syncthreads();
      if (!(bucket && n_in > 64 && block_bucket_order(s_hi, s_tmp, s_lo, s_bin, s_cur, n_in, sh))) {
        sort64_positions(s_hi, s_lo, n_in);
        __syncthreads();
      }
      for (int q = threadIdx.x; q < n_in; q += blockDim.x) a.order[b + n_act + q] = sin[s_lo[q]].row;
      __syncthreads();
      segment_plan(p, a, seg, n_act, r, real, sh);
      block_min_arrival(next_arr, sh);
    } else {
      segment_plan(p, a, seg, n_act, r, real, sh);
    }
    const ReplicaPlan pl = sh.plan;

    // ---- sort items of the active rows ---------------------------------------------------------------
    for (int q = threadIdx.x; q < n_act; q += blockDim.x) {
      const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + q));
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
      const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
      const int32_t row = (int32_t)w0.w;
      const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
      const RowEval e = eval_row(p, pl, base, kind, prio, (int32_t)w1.x, (int32_t)w1.y);
      if (ordered) s_hi[q] = (e.k48 << 16) | (uint32_t)q;     // records are in req_id order: position breaks ties
      else {
        const uint32_t uid = w0.z ^ 0x80000000u;               // signed req_id order as unsigned
        s_hi[q] = (e.k48 << 16) | (uid >> 16);
        s_lo[q] = (uid << 16) | (uint32_t)q;
      }
      if (kind == KIND_RUNNING || pl.mode == HFX_DECODE) {    // (the regroup wrote the slack of the other queued rows)
        a.slack[row] = e.slack;
        if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | e.k48;
      }
      if (a.pred_tpot) a.pred_tpot[row] = e.pred_tpot;
    }
    __syncthreads();
    if (ordered) {
      if (!(bucket && n_act > 64 && block_bucket_order(s_hi, s_tmp, s_lo, s_bin, s_cur, n_act, sh))) {
        sort64_positions(s_hi, s_lo, n_act);
      }
    } else {
      block_sort<true>(s_hi, s_lo, n_act);
      for (int q = threadIdx.x; q < n_act; q += blockDim.x) s_lo[q] &= 0xffffu;
    }
    __syncthreads();

    segment_admit(p, a, pl, seg, b, s_lo, n_act, sh);

    // ---- maturity, iteration clock ------------------------------------------------------------------
    if (threadIdx.x == 0) {
      int64_t lp = 0;
      const int64_t mat_next = dev_maturity_next(p, pl, sh.adm_count, sh.adm_cost, sh.adm_kv, &lp);
      int worked; int64_t t1, t2;
      iteration_clock(pl, sh.adm_count, lp, mat_next, worked, t1, t2);
      sh.worked = worked; sh.t1 = t1; sh.t2 = t2; sh.red_c[0] = mat_next;
    }
    __syncthreads();
    const bool commit = real && (a.flags & HFX_COMMIT) && pl.now <= a.horizon;
    const int worked = sh.worked;
    const int64_t mat_next = sh.red_c[0];
    if (commit && !worked && ordered) {
      // idle replica of an ordered step: its next arrival is looked up among its listed inactive rows
      block_min_arrival(next_arrival_listed(a, c, b, n_act, n, threadIdx.x, blockDim.x), sh);
    }
    if (threadIdx.x == 0 && real)
      write_replica_outputs(a, r, pl, sh.adm_cost, sh.adm_count, mat_next, worked, sh.t2, sh.next_arrival);

    // ---- padding of the compacted list, commit ----------------------------------------------------
    if (a.admitted_rows)
      for (int q = sh.adm_count + threadIdx.x; q < n; q += blockDim.x) a.admitted_rows[b + q] = -1;
    if (commit) {
      const int64_t t1 = sh.t1, t2 = sh.t2;
      for (int q = threadIdx.x; q < n_act; q += blockDim.x) {
        const uint32_t lo = s_lo[q];
        const int li = lo & 0xffff;
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
        const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
        commit_row(a, pl, (w1.w >> 8) & 0xff, (lo & 0x10000u) != 0, worked, t1, t2, (int32_t)w0.w, (int32_t)w1.x,
                   (int32_t)w1.y, (int32_t)w1.z);
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// k_segment_small: replicas with at most SEG_TINY items to sort.  What later passes need of the
// replica's active records (lengths, kind, row) is staged once into shared memory; sort items live
// in registers until they are scattered into their bins.
// ------------------------------------------------------------------------------------------------
#define SEG_TINY 768
#define TINY_IPT ((SEG_TINY + THREADS_SMALL - 1) / THREADS_SMALL)     // items per thread
#define TINY_BINS 512
#define TINY_BIN_MAX 48
#define SMEM_TINY (SEG_TINY * (16 + 4 + 8 + 4) + (2 * TINY_BINS + 8) * 4)

__global__ void __launch_bounds__(THREADS_SMALL, TINY_BLOCKS_PER_SM) k_segment_small(const HfxParams p, const SegArgs a, const SegCtx c) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4 *s_w1 = reinterpret_cast<uint4 *>(smem_raw);                                   // [SEG_TINY] prompt, gen, output_len, bytes
  uint64_t *s_key = reinterpret_cast<uint64_t *>(smem_raw + (size_t)SEG_TINY * 16);    // [SEG_TINY] sort items, binned
  int32_t *s_row = reinterpret_cast<int32_t *>(s_key + SEG_TINY);                      // [SEG_TINY]
  uint32_t *s_lo = reinterpret_cast<uint32_t *>(s_row + SEG_TINY);                     // [SEG_TINY] order (+ tie-break words)
  uint32_t *s_bin = s_lo + SEG_TINY;                                                   // [TINY_BINS + 4]
  uint32_t *s_cur = s_bin + TINY_BINS + 4;                                             // [TINY_BINS]
  __shared__ BlockShared sh;
  __shared__ int64_t s_cls_ttft[HFX_MAX_CLASSES], s_cls_tpot[HFX_MAX_CLASSES];     // class tables for the planning warp
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int R = p.n_replicas;
  const bool ordered = c.flags[c.parity] != 0;
  for (int k = threadIdx.x; k < HFX_MAX_CLASSES; k += blockDim.x) {
    s_cls_ttft[k] = k < p.n_classes ? p.ttft[k] : 0;
    s_cls_tpot[k] = k < p.n_classes ? p.tpot[k] : 0;
  }

  for (int r = blockIdx.x; r <= R; r += gridDim.x) {
    const uint32_t b = c.seg_begin[r];
    const int n = (int)(c.seg_begin[r + 1] - b);
    const int n_act = (int)c.tot_act[r];
    const int n_in = n - n_act;
    const int need = ordered ? n_act : (n_act > n_in ? n_act : n_in);
    if (need > SEG_TINY) continue;
    if (r == R && n == 0) continue;
    const HfxRec *seg = c.rec + b;
    const bool real = r < R;    // bucket R holds rows bound to no replica

    int64_t next_arr = HFX_INF;
    if (!ordered && n_in > 0) {
      // inactive rows of a step that is not ordered: listed by req_id behind the active ones
      const HfxRec *sin = seg + n_act;
      for (int q = threadIdx.x; q < n_in; q += blockDim.x) {
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(sin + q));
        const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(sin + q) + 1);
        if (((w1.w >> 8) & 0xff) == KIND_FUTURE) { const int64_t arr = (int64_t)(((uint64_t)w0.y << 32) | w0.x); next_arr = arr < next_arr ? arr : next_arr; }
        s_key[q] = ((uint64_t)(w0.z ^ 0x80000000u) << 16) | (uint32_t)q;
      }
      __syncthreads();
      block_sort<false>(s_key, nullptr, n_in);
      for (int q = threadIdx.x; q < n_in; q += blockDim.x) a.order[b + n_act + q] = sin[s_key[q] & 0xffffu].row;
      __syncthreads();
    }

    // ---- stage what later passes need of the active records; aggregates --------------------------
    uint4 w0r[TINY_IPT];
    {
      int64_t n_run = 0, sum_kv = 0;
      uint64_t m_run = 0, m_q = 0;
#pragma unroll
      for (int k = 0; k < TINY_IPT; k++) {
        const int q = threadIdx.x + k * THREADS_SMALL;
        if (q < n_act) {
          w0r[k] = __ldg(reinterpret_cast<const uint4 *>(seg + q));
          const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
          s_w1[q] = w1;
          s_row[q] = (int32_t)w0r[k].w;
          const int kind = (w1.w >> 8) & 0xff, cls = w1.w & 0xff;
          if (kind == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(int32_t)w1.x + (int32_t)w1.y; m_run |= 1ull << cls; }
          else m_q |= 1ull << cls;
        }
      }
      n_run = warp_sum_i64(n_run); sum_kv = warp_sum_i64(sum_kv); next_arr = warp_min_i64(next_arr);
      m_run = warp_or_u64(m_run); m_q = warp_or_u64(m_q);
      if (lane == 0) { sh.red_a[warp] = n_run; sh.red_b[warp] = sum_kv; sh.red_c[warp] = next_arr; sh.red_m0[warp] = m_run; sh.red_m1[warp] = m_q; }
      for (int i = threadIdx.x; i <= TINY_BINS; i += blockDim.x) s_bin[i] = 0;
      __syncthreads();
      if (warp == 0) {     // the whole first warp finishes the reduction and plans
        const bool has = lane < nwarp;
        n_run = warp_sum_i64(has ? sh.red_a[lane] : 0); sum_kv = warp_sum_i64(has ? sh.red_b[lane] : 0);
        next_arr = warp_min_i64(has ? sh.red_c[lane] : HFX_INF);
        m_run = warp_or_u64(has ? sh.red_m0[lane] : 0); m_q = warp_or_u64(has ? sh.red_m1[lane] : 0);
        hfx_replica_cfg cfg; cfg.mode = HFX_COLOCATED; cfg.token_cap = 1; cfg.batch_cap = 0;
        int64_t now = 0, mat = 0;
        if (real) { cfg = a.cfg[r]; now = a.now[r]; mat = a.mat[r]; }
        ReplicaPlan pl0;
        warp_plan(p, s_cls_ttft, s_cls_tpot, cfg, now, mat, n_run, sum_kv, m_run, m_q, pl0, lane);
        if (lane == 0) { sh.plan = pl0; sh.next_arrival = next_arr; }
      }
      __syncthreads();
    }
    const ReplicaPlan pl = sh.plan;

    // ---- keys (in registers), their range ---------------------------------------------------------
    uint64_t item[TINY_IPT];
    uint64_t mn = ~0ull, mx = 0;
#pragma unroll
    for (int k = 0; k < TINY_IPT; k++) {
      const int q = threadIdx.x + k * THREADS_SMALL;
      item[k] = ~0ull;
      if (q < n_act) {
        const uint4 w0 = w0r[k], w1 = s_w1[q];
        const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
        const int32_t row = (int32_t)w0.w;
        const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
        const RowEval e = eval_row(p, pl, base, kind, prio, (int32_t)w1.x, (int32_t)w1.y);
        if (ordered) {
          item[k] = (e.k48 << 16) | (uint32_t)q;     // records are in req_id order: position breaks ties
          mn = item[k] < mn ? item[k] : mn; mx = item[k] > mx ? item[k] : mx;
        } else {
          const uint32_t uid = w0.z ^ 0x80000000u;
          s_key[q] = (e.k48 << 16) | (uid >> 16);
          s_lo[q] = (uid << 16) | (uint32_t)q;
        }
        if (kind == KIND_RUNNING || pl.mode == HFX_DECODE) {    // (the regroup wrote the slack of the other queued rows)
          a.slack[row] = e.slack;
          if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | e.k48;
        }
        if (a.pred_tpot) a.pred_tpot[row] = e.pred_tpot;
      }
    }
    bool sorted_done = false;
    if (ordered && n_act > 0) {
      // ---- distribution sort: bins by offset from the smallest item, rank inside the bin by counting ----
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const uint64_t x = __shfl_xor_sync(0xffffffffu, mn, o), y = __shfl_xor_sync(0xffffffffu, mx, o);
        mn = x < mn ? x : mn; mx = y > mx ? y : mx;
      }
      if (lane == 0) { sh.red_m0[warp] = mn; sh.red_m1[warp] = mx; }
      __syncthreads();
      for (int k = 0; k < nwarp; k++) { const uint64_t x = sh.red_m0[k], y = sh.red_m1[k]; mn = x < mn ? x : mn; mx = y > mx ? y : mx; }
      const uint64_t range = mx - mn;
      int sft = 0;
      if (range >= TINY_BINS) sft = 64 - __clzll((long long)range) - 9;     // (range >> sft) < TINY_BINS
#pragma unroll
      for (int k = 0; k < TINY_IPT; k++)
        if (threadIdx.x + k * THREADS_SMALL < n_act) atomicAdd(&s_bin[(uint32_t)((item[k] - mn) >> sft)], 1u);
      __syncthreads();
      if (warp == 0) {     // exclusive scan of the bin counts by one warp; the largest bin
        const int per = TINY_BINS / 32;
        uint32_t cnt[TINY_BINS / 32];
        uint32_t sum = 0, big = 0;
#pragma unroll
        for (int i = 0; i < per; i++) { cnt[i] = s_bin[lane * per + i]; sum += cnt[i]; big = cnt[i] > big ? cnt[i] : big; }
        uint32_t v = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const uint32_t x = __shfl_xor_sync(0xffffffffu, big, o); big = x > big ? x : big; }
        uint32_t run = v - sum;
#pragma unroll
        for (int i = 0; i < per; i++) { s_bin[lane * per + i] = run; s_cur[lane * per + i] = run; run += cnt[i]; }
        if (lane == 0) sh.red_n[0] = (int32_t)big;
      }
      __syncthreads();
      if (sh.red_n[0] <= TINY_BIN_MAX) {
#pragma unroll
        for (int k = 0; k < TINY_IPT; k++)
          if (threadIdx.x + k * THREADS_SMALL < n_act) s_key[atomicAdd(&s_cur[(uint32_t)((item[k] - mn) >> sft)], 1u)] = item[k];
        __syncthreads();
        for (int e = threadIdx.x; e < n_act; e += blockDim.x) {
          const uint64_t x = s_key[e];
          const uint32_t bi = (uint32_t)((x - mn) >> sft);
          const uint32_t g0 = s_bin[bi], g1 = s_cur[bi];
          uint32_t rank = 0;
          for (uint32_t g = g0; g < g1; g++) rank += s_key[g] < x ? 1u : 0u;
          s_lo[g0 + rank] = (uint32_t)(x & 0xffffu);
        }
        sorted_done = true;
      } else {
#pragma unroll
        for (int k = 0; k < TINY_IPT; k++) { const int q = threadIdx.x + k * THREADS_SMALL; if (q < n_act) s_key[q] = item[k]; }
      }
    }
    __syncthreads();
    if (!sorted_done) {
      if (ordered) {
        block_sort<false>(s_key, nullptr, n_act);
        for (int q = threadIdx.x; q < n_act; q += blockDim.x) s_lo[q] = (uint32_t)(s_key[q] & 0xffffu);
      } else {
        block_sort<true>(s_key, s_lo, n_act);
        for (int q = threadIdx.x; q < n_act; q += blockDim.x) s_lo[q] &= 0xffffu;
      }
      __syncthreads();
    }

    // ---- first-fit variant: the first warp walks the order and marks what it takes (bit 17) -----------
    if (p.first_fit) {
      if (warp == 0) {
        const int64_t room = pl.batch_cap == 0 ? HFX_INF : (pl.batch_cap > pl.n_eff ? pl.batch_cap - pl.n_eff : 0);
        warp_first_fit(n_act, pl.budget, room, lane,
                       [&](int64_t q) -> int64_t {
                         const uint4 w1 = s_w1[s_lo[q] & 0xffffu];
                         if (((w1.w >> 8) & 0xff) != KIND_QUEUED) return -1;
                         return pl.mode == HFX_DECODE ? p.d1 + p.d2 * ((int64_t)(int32_t)w1.x + (int32_t)w1.y) : (int64_t)(int32_t)w1.x;
                       },
                       [&](int64_t q, bool taken) { if (taken) s_lo[q] |= 0x20000u; });
      }
      __syncthreads();
    }

    // ---- admission: each thread walks TINY_IPT consecutive places of the order ---------------------
    const int q0 = threadIdx.x * TINY_IPT;
    int64_t cost[TINY_IPT], kvs[TINY_IPT];
    int32_t rows[TINY_IPT], kinds[TINY_IPT];
    int64_t my_cost = 0;
    int32_t my_cnt = 0;
#pragma unroll
    for (int k = 0; k < TINY_IPT; k++) {
      const int q = q0 + k;
      cost[k] = -1; kvs[k] = 0; rows[k] = -1; kinds[k] = KIND_DEAD;
      if (q < n_act) {
        const int li = s_lo[q] & 0xffffu;
        const uint4 w1 = s_w1[li];
        rows[k] = s_row[li];
        kinds[k] = (w1.w >> 8) & 0xff;
        if (kinds[k] == KIND_QUEUED) {
          const int64_t kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
          const int64_t cc = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
          // what counts towards the totals: rows that fit alone, or (first fit) exactly the rows taken
          if (p.first_fit ? (s_lo[q] & 0x20000u) != 0 : cc <= pl.budget) { cost[k] = cc; kvs[k] = kv; my_cost += cc; my_cnt++; }
        }
        a.order[b + q] = rows[k];
      }
    }
    int64_t sc = warp_incl_scan_i64(my_cost, lane);
    int32_t sn = warp_incl_scan_i32(my_cnt, lane);
    if (lane == 31) { sh.red_a[warp] = sc; sh.red_n[warp] = sn; }
    __syncthreads();
    int64_t run_c = sc - my_cost;
    int32_t run_n = sn - my_cnt;
    for (int k = 0; k < warp; k++) { run_c += sh.red_a[k]; run_n += sh.red_n[k]; }
    int64_t ac = 0, ak = 0;
    int32_t an = 0;
#pragma unroll
    for (int k = 0; k < TINY_IPT; k++) {
      const int q = q0 + k;
      if (q < n_act) {
        bool adm = false;
        if (cost[k] >= 0) {
          run_c += cost[k]; run_n += 1;
          adm = p.first_fit || (run_c <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + run_n <= pl.batch_cap));
          if (adm) { ac += cost[k]; ak += kvs[k]; an++; if (a.admitted_rows) a.admitted_rows[b + run_n - 1] = rows[k]; }
        }
        if (kinds[k] == KIND_RUNNING || adm) a.admit[rows[k]] = 1;
        s_lo[q] = (s_lo[q] & 0xffffu) | (adm ? 0x10000u : 0u);
      }
    }
    ac = warp_sum_i64(ac); ak = warp_sum_i64(ak); an = (int32_t)warp_sum_i64(an);
    __syncthreads();
    if (lane == 0) { sh.red_a[warp] = ac; sh.red_b[warp] = ak; sh.red_n[warp] = an; }
    __syncthreads();
    if (threadIdx.x == 0) {
      int64_t adm_cost = 0, adm_kv = 0; int32_t adm_count = 0;
      for (int k = 0; k < nwarp; k++) { adm_cost += sh.red_a[k]; adm_kv += sh.red_b[k]; adm_count += sh.red_n[k]; }
      int64_t lp = 0;
      const int64_t mat_next = dev_maturity_next(p, pl, adm_count, adm_cost, adm_kv, &lp);
      int worked; int64_t t1, t2;
      iteration_clock(pl, adm_count, lp, mat_next, worked, t1, t2);
      sh.adm_cost = adm_cost; sh.adm_count = adm_count;
      sh.worked = worked; sh.t1 = t1; sh.t2 = t2; sh.red_c[0] = mat_next;
    }
    __syncthreads();
    const bool commit = real && (a.flags & HFX_COMMIT) && pl.now <= a.horizon;
    const int worked = sh.worked;
    const int64_t mat_next = sh.red_c[0];
    if (commit && !worked && ordered) {
      // idle replica of an ordered step: its next arrival is looked up among its listed inactive rows
      block_min_arrival(next_arrival_listed(a, c, b, n_act, n, threadIdx.x, blockDim.x), sh);
    }
    if (threadIdx.x == 0 && real)
      write_replica_outputs(a, r, pl, sh.adm_cost, sh.adm_count, mat_next, worked, sh.t2, sh.next_arrival);
    if (a.admitted_rows)
      for (int q = sh.adm_count + threadIdx.x; q < n; q += blockDim.x) a.admitted_rows[b + q] = -1;
    if (commit) {
      const int64_t t1 = sh.t1, t2 = sh.t2;
      for (int q = threadIdx.x; q < n_act; q += blockDim.x) {
        const uint32_t lo = s_lo[q];
        const int li = lo & 0xffff;
        const uint4 w1 = s_w1[li];
        commit_row(a, pl, (w1.w >> 8) & 0xff, (lo & 0x10000u) != 0, worked, t1, t2, s_row[li], (int32_t)w1.x,
                   (int32_t)w1.y, (int32_t)w1.z);
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// Oversize replicas (more items than a block can sort in shared memory): one cooperative kernel.
// All blocks walk the replicas in the same order and share the work of each oversize one: keys
// spread over the grid, a global bitonic network with bounded grid barriers, admission by block 0
// walking the order with a carried prefix, commit by the grid.  Slow but exact; it only exists so
// that any table is handled.
// ------------------------------------------------------------------------------------------------

// Bounded grid barrier (all blocks of a cooperative launch are resident).  Returns false if the
// wait ran out; the caller then leaves, and HFX_ST_TIMEOUT is raised.
__device__ bool grid_barrier(uint32_t *bar, uint32_t *status, uint32_t &epoch) {
  __shared__ int ok_s;
  __syncthreads();
  epoch++;
  if (threadIdx.x == 0) {
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

__device__ __forceinline__ void global_cmp_swap(uint64_t *hi, uint32_t *lo, uint32_t *idx, int64_t i, int64_t j) {
  const uint64_t hi_i = hi[i], hi_j = hi[j];
  const uint32_t lo_i = lo[i], lo_j = lo[j];
  if (hi_i > hi_j || (hi_i == hi_j && lo_i > lo_j)) {
    hi[i] = hi_j; hi[j] = hi_i; lo[i] = lo_j; lo[j] = lo_i;
    const uint32_t x = idx[i]; idx[i] = idx[j]; idx[j] = x;
  }
}

// Global bitonic network over n items (hi, lo) with idx travelling along: ascending comparators,
// virtual padding.  The items must be visible grid-wide on entry (a grid barrier precedes it).
__device__ bool grid_sort(uint64_t *hi, uint32_t *lo, uint32_t *idx, int64_t n, uint32_t *bar, uint32_t *status,
                          uint32_t &epoch) {
  const int64_t gtid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t gsize = (int64_t)gridDim.x * blockDim.x;
  int64_t n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  const int64_t half = n_pad >> 1;
  for (int64_t k = 2; k <= n_pad; k <<= 1) {
    const int64_t hk = k >> 1;
    for (int64_t t = gtid; t < half; t += gsize) {
      const int64_t blk = t / hk, off = t - blk * hk;
      const int64_t i = blk * k + off, j = blk * k + k - 1 - off;
      if (j < n) global_cmp_swap(hi, lo, idx, i, j);
    }
    if (!grid_barrier(bar, status, epoch)) return false;
    for (int64_t j = k >> 2; j > 0; j >>= 1) {
      for (int64_t t = gtid; t < half; t += gsize) {
        const int64_t i = 2 * t - (t & (j - 1));
        if (i + j < n) global_cmp_swap(hi, lo, idx, i, i + j);
      }
      if (!grid_barrier(bar, status, epoch)) return false;
    }
  }
  return true;
}

__global__ void __launch_bounds__(512) k_big(const HfxParams p, const SegArgs a, const SegCtx c,
                                             uint64_t *__restrict__ g_hi, uint32_t *__restrict__ g_lo,
                                             uint32_t *__restrict__ g_idx, uint32_t *bar, uint32_t *status) {
  __shared__ BlockShared sh;
  if (c.flags[2] <= SEG_MED) return;
  const bool ordered = c.flags[c.parity] != 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int R = p.n_replicas;
  uint32_t epoch = 0;
  const int64_t gtid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t gsize = (int64_t)gridDim.x * blockDim.x;
  volatile int64_t *mail = reinterpret_cast<volatile int64_t *>(bar + 4);

  for (int r = 0; r <= R; r++) {
    const uint32_t b = c.seg_begin[r];
    const int64_t n = (int64_t)(c.seg_begin[r + 1] - b);
    const int64_t n_act = c.tot_act[r], n_in = n - n_act;
    const int64_t need = ordered ? n_act : (n_act > n_in ? n_act : n_in);
    if (need <= SEG_MED) continue;
    const HfxRec *seg = c.rec + b;
    const bool real = r < R;

    // ---- inactive rows of a step that is not ordered: by req_id behind the active ones -----------
    if (!ordered && n_in > 0) {
      const HfxRec *sin = seg + n_act;
      uint64_t *hi = g_hi + b + n_act;
      uint32_t *lo = g_lo + b + n_act, *idx = g_idx + b + n_act;
      for (int64_t q = gtid; q < n_in; q += gsize) {
        const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(sin + q));
        hi[q] = w0.z ^ 0x80000000u; lo[q] = 0; idx[q] = (uint32_t)q;
      }
      if (!grid_barrier(bar, status, epoch)) return;
      if (!grid_sort(hi, lo, idx, n_in, bar, status, epoch)) return;
      for (int64_t q = gtid; q < n_in; q += gsize) a.order[b + n_act + q] = sin[idx[q]].row;
    }

    // every block computes the aggregates redundantly (reads come from L2 after the first)
    segment_plan(p, a, seg, n_act, r, real, sh);
    const ReplicaPlan pl = sh.plan;
    uint64_t *hi = g_hi + b;
    uint32_t *lo = g_lo + b, *idx = g_idx + b;

    // keys of the active rows, spread over the grid
    for (int64_t q = gtid; q < n_act; q += gsize) {
      const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + q));
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
      const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
      const int32_t row = (int32_t)w0.w;
      const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
      const RowEval e = eval_row(p, pl, base, kind, prio, (int32_t)w1.x, (int32_t)w1.y);
      hi[q] = e.k48;
      lo[q] = w0.z ^ 0x80000000u;
      idx[q] = (uint32_t)q;
      if (kind == KIND_RUNNING || pl.mode == HFX_DECODE) {    // (the regroup wrote the slack of the other queued rows)
        a.slack[row] = e.slack;
        if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | e.k48;
      }
      if (a.pred_tpot) a.pred_tpot[row] = e.pred_tpot;
    }
    if (!grid_barrier(bar, status, epoch)) return;
    if (!grid_sort(hi, lo, idx, n_act, bar, status, epoch)) return;

    // admission walk by block 0 with a carried prefix, then commit by the whole grid
    if (blockIdx.x == 0) {
      if (p.first_fit) {     // the first warp walks the order; lo (free now that the sort is over) says what it took
        if (warp == 0) {
          const int64_t room = pl.batch_cap == 0 ? HFX_INF : (pl.batch_cap > pl.n_eff ? pl.batch_cap - pl.n_eff : 0);
          warp_first_fit(n_act, pl.budget, room, lane,
                         [&](int64_t q) -> int64_t {
                           const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + idx[q]) + 1);
                           if (((w1.w >> 8) & 0xff) != KIND_QUEUED) return -1;
                           return pl.mode == HFX_DECODE ? p.d1 + p.d2 * ((int64_t)(int32_t)w1.x + (int32_t)w1.y) : (int64_t)(int32_t)w1.x;
                         },
                         [&](int64_t q, bool taken) { lo[q] = taken ? 2u : 0u; });
        }
        __syncthreads();
      }
      for (int64_t tile = 0; tile < n_act; tile += blockDim.x) {
        const int64_t q = tile + threadIdx.x;
        int64_t cost = 0, kv = 0;
        int32_t cnt = 0, row = -1, kind = KIND_DEAD;
        if (q < n_act) {
          const uint32_t li = idx[q];
          const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
          const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
          row = (int32_t)w0.w;
          kind = (w1.w >> 8) & 0xff;
          if (kind == KIND_QUEUED) {
            kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
            const int64_t cc = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
            if (p.first_fit ? lo[q] == 2u : cc <= pl.budget) { cost = cc; cnt = 1; } else kv = 0;
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
        if (cnt) adm = p.first_fit || (sc <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + sn <= pl.batch_cap));
        if (q < n_act) {
          if (kind == KIND_RUNNING || adm) a.admit[row] = 1;
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
      // the replica's next arrival, should it turn out idle
      int64_t v = HFX_INF;
      if (ordered) {
        v = next_arrival_listed(a, c, b, n_act, n, threadIdx.x, blockDim.x);
      } else {
        const HfxRec *sin = seg + n_act;
        for (int64_t q = threadIdx.x; q < n_in; q += blockDim.x) {
          const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(sin + q));
          const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(sin + q) + 1);
          if (((w1.w >> 8) & 0xff) == KIND_FUTURE) { const int64_t arr = (int64_t)(((uint64_t)w0.y << 32) | w0.x); v = arr < v ? arr : v; }
        }
      }
      block_min_arrival(v, sh);
      if (threadIdx.x == 0) {
        int64_t lp = 0;
        const int64_t mat_next = dev_maturity_next(p, pl, sh.adm_count, sh.adm_cost, sh.adm_kv, &lp);
        int worked; int64_t t1, t2;
        iteration_clock(pl, sh.adm_count, lp, mat_next, worked, t1, t2);
        mail[0] = t1; mail[1] = t2; mail[2] = worked; mail[3] = sh.adm_count;   // for the other blocks
        if (real) write_replica_outputs(a, r, pl, sh.adm_cost, sh.adm_count, mat_next, worked, t2, sh.next_arrival);
      }
    }
    if (!grid_barrier(bar, status, epoch)) return;
    {
      const int64_t t1 = mail[0], t2 = mail[1];
      const int worked = (int)mail[2], adm_count = (int)mail[3];
      const bool commit = real && (a.flags & HFX_COMMIT) && pl.now <= a.horizon;
      if (a.admitted_rows)
        for (int64_t q = adm_count + gtid; q < n; q += gsize) a.admitted_rows[b + q] = -1;
      if (commit)
        for (int64_t q = gtid; q < n_act; q += gsize) {
          const uint32_t li = idx[q];
          const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + li));
          const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + li) + 1);
          commit_row(a, pl, (w1.w >> 8) & 0xff, lo[q] != 0, worked, t1, t2, (int32_t)w0.w, (int32_t)w1.x, (int32_t)w1.y,
                     (int32_t)w1.z);
        }
    }
    if (!grid_barrier(bar, status, epoch)) return;
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
int hfx_launch_segments(hfx_sched *s, const SegArgs &sa, int64_t n) {
  const int R1 = s->p.n_replicas + 1;
  cudaStream_t stream = s->stream;
  SegCtx c;
  c.rec = s->d_rec; c.seg_begin = s->d_seg_begin; c.tot_act = s->d_act_count; c.flags = s->d_flags;
  c.rowflag = s->d_rowflag; c.parity = s->step_parity;
  // Replicas too large for the small kernel are rare; their kernels (which leave at once when there is
  // nothing for them) run on a second stream beside the small-replica kernel, forked and joined by events.
  const bool larger = n > SEG_TINY;
  const bool beside = larger && !s->profiling;
  cudaStream_t st2 = beside ? s->side : stream;
  if (beside) {
    if (cudaEventRecord(s->ev_fork, stream) != cudaSuccess || cudaStreamWaitEvent(s->side, s->ev_fork, 0) != cudaSuccess)
      return HFX_E_CUDA;
  }
  if (!beside) {
    KernelScope ks(s, KSLOT_SEG_SMALL);
    const int grid = R1 < s->n_sm * 16 ? R1 : s->n_sm * 16;
    k_segment_small<<<grid, THREADS_SMALL, SMEM_TINY, stream>>>(s->p, sa, c);
  }
  if (larger) {
    KernelScope ks(s, KSLOT_SEG_MED, st2);
    const int grid = R1 < s->n_sm ? R1 : s->n_sm;
    k_segment<<<grid, THREADS_MED, SEG_MED * 12, st2>>>(s->p, sa, c, SEG_TINY + 1, SEG_MED, 0);
  }
  if (n > SEG_MED) {
    uint32_t *big_idx = reinterpret_cast<uint32_t *>(s->d_big_lo + s->max_rows);
    if (cudaMemsetAsync(s->d_barrier, 0, 64, st2) != cudaSuccess) return HFX_E_CUDA;
    void *args[] = {(void *)&s->p, (void *)&sa, (void *)&c, (void *)&s->d_big_hi, (void *)&s->d_big_lo, (void *)&big_idx,
                    (void *)&s->d_barrier, (void *)&s->d_status};
    KernelScope ks(s, KSLOT_BIG, st2);
    if (cudaLaunchCooperativeKernel((void *)k_big, dim3(s->n_sm), dim3(512), args, 0, st2) != cudaSuccess)
      return HFX_E_CUDA;
  }
  if (beside) {
    {
      KernelScope ks(s, KSLOT_SEG_SMALL);
      const int grid = R1 < s->n_sm * 16 ? R1 : s->n_sm * 16;
      k_segment_small<<<grid, THREADS_SMALL, SMEM_TINY, stream>>>(s->p, sa, c);
    }
    if (cudaEventRecord(s->ev_join, s->side) != cudaSuccess || cudaStreamWaitEvent(stream, s->ev_join, 0) != cudaSuccess)
      return HFX_E_CUDA;
  }
  return HFX_OK;
}

int hfx_segment_configure() {
  if (cudaFuncSetAttribute(k_segment, cudaFuncAttributeMaxDynamicSharedMemorySize, SEG_MED * 12) != cudaSuccess ||
      cudaFuncSetAttribute(k_segment_small, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TINY) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}
