// Per-replica work of a step, one persistent kernel (k_replicas, one block of 1024 threads per SM):
// the replica's rows are gathered from the tile slabs in tile order (= row order), then aggregates of
// the running batch, E_d, the safe budget (Eq. 3), final slack and key, the sort, segmented-scan
// admission, maturity, commit.  Three size classes share the kernel:
//   small    (<= SEG_TINY items to sort)  a group of 128 threads per replica, eight groups per block, each on
//                                         its own hardware barrier; records staged in shared memory
//   medium   (<= SEG_MED items)           the whole block; records gathered into a contiguous scratch range
//   oversize                              the whole block with a sorting network in global memory; slow, it
//                                         only exists so that any table is handled
// No block ever waits for another: the only cross-block data are the slabs and totals that the front end
// finished before this kernel reads them.
#include <string.h>

#include "hfx_internal.cuh"

#define SEG_TINY 768      // items a 128-thread group sorts
#define SEG_MED 16384     // items a block sorts in shared memory
#define REP_THREADS 1024
#define REP_GROUPS 8
#define GROUP_THREADS 128
#define TINY_IPT ((SEG_TINY + GROUP_THREADS - 1) / GROUP_THREADS)     // items per thread
#define TINY_BINS 1024    // bins of the distribution sort (16-bit counters, two to a word)
#define TINY_BIN_MAX 48
#define TINY_CLASSES 128  // (phase, priority) classes of the sort items of active rows: phase<1> | prio<6>
#define GROUP_TPT 2       // tiles per thread and round when a group gathers
#define LIST_MAX 2048     // inactive rows a replica's own threads list while they gather; longer lists are shared by the grid
#define SMEM_MED (SEG_MED * 12)
#define SMEM_GROUP (SMEM_MED / REP_GROUPS)

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

// where the kernel finds the rows of a replica
struct SegCtx {
  // tile front end: slabs
  const uint4 *slab_rec; const uint16_t *slab_idx; const uint2 *M; const unsigned long long *tot;
  int32_t tile_rows, n_tiles;
  // fallback front end: contiguous records, counts and range starts
  const uint32_t *seg_count; const uint32_t *act_count; const uint32_t *seg_begin;
  HfxRec *rec;            // contiguous records (fallback: input; slabs: scratch of the larger replicas)
  const uint32_t *ordered; const uint8_t *rowflag;
  uint64_t *big_hi; uint32_t *big_lo; uint32_t *big_idx;
  int32_t slabs;
};

// A set of threads of the block that synchronise on a hardware barrier of their own (0 = the whole block).
struct Grp {
  int tid, n, bar;
  __device__ __forceinline__ void sync() const { asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(n) : "memory"); }
  __device__ __forceinline__ int any(int pred) const {
    int r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.s32 p, %3, 0;\n\tbar.red.or.pred q, %1, %2, p;\n\tselp.s32 %0, 1, 0, q;\n\t}"
                 : "=r"(r) : "r"(bar), "r"(n), "r"(pred) : "memory");
    return r;
  }
};

// ---- sorting networks ---------------------------------------------------------------------------
// Bitonic network with ascending comparators only (mirrored first sub-stage), so the virtual +inf
// padding beyond n never moves: any n, in place.  Items are distinct, so the result is unique.  Each
// warp owns a contiguous chunk of E items; stages whose pairs stay inside a chunk need only a warp
// barrier.  Callers synchronise the group before the call; it is synchronised on return.
template <bool WIDE>
__device__ void group_sort(uint64_t *hi, uint32_t *lo, int n, const Grp &G) {
  if (n > 1) {
    int n_pad = 2;
    while (n_pad < n) n_pad <<= 1;
    const int lane = G.tid & 31, warp = G.tid >> 5, nwarp = G.n >> 5;
    int E = n_pad / nwarp;
    if (E < 64) E = 64;
    if (E > n_pad) E = n_pad;
    const int c0 = warp * E;
    const bool has_chunk = c0 < n_pad;
    const int half = n_pad >> 1;
    bool local = true;    // the previous stage was chunk-local (or there was none)
    for (int k = 2; k <= n_pad; k <<= 1) {
      const int hk = k >> 1;
      if (k <= E) {   // mirrored sub-stage of merge size k, inside the chunk
        if (has_chunk)
          for (int t = lane; t < (E >> 1); t += 32) {
            const int blk = t / hk, off = t - blk * hk;
            const int i = c0 + blk * k + off, j = c0 + blk * k + k - 1 - off;
            if (j < n) cmp_swap<WIDE>(hi, lo, i, j);
          }
        __syncwarp();
      } else {
        if (local) { G.sync(); local = false; }
        for (int t = G.tid; t < half; t += G.n) {
          const int blk = t / hk, off = t - blk * hk;
          const int i = blk * k + off, j = blk * k + k - 1 - off;
          if (j < n) cmp_swap<WIDE>(hi, lo, i, j);
        }
        G.sync();
      }
      for (int j = k >> 2; j > 0; j >>= 1) {
        if (2 * j <= E) {   // pairs (i, i+j) stay inside an aligned block of 2j <= E items
          local = true;
          if (has_chunk)
            for (int t = lane; t < (E >> 1); t += 32) {
              const int i = c0 + 2 * t - (t & (j - 1));
              if (i + j < n) cmp_swap<WIDE>(hi, lo, i, i + j);
            }
          __syncwarp();
        } else {
          if (local) { G.sync(); local = false; }
          for (int t = G.tid; t < half; t += G.n) {
            const int i = 2 * t - (t & (j - 1));
            if (i + j < n) cmp_swap<WIDE>(hi, lo, i, i + j);
          }
          G.sync();
        }
      }
    }
  }
  G.sync();
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

// does the commit of this row read its output length?  (rows in flight that advance, and admitted rows)
__device__ __forceinline__ bool commit_needs_out_len(const ReplicaPlan &pl, int kind, bool adm, int worked) {
  if (kind == KIND_RUNNING) return !(pl.mode == HFX_PREFILL || (pl.mode == HFX_DECODE && !worked));
  return kind == KIND_QUEUED && adm;
}

// Earliest arrival among a replica's rows that have not arrived yet, for the clock jump of an idle
// replica: the replica's inactive rows are listed in order[b + n_act .. b + n); their kind bytes say
// which of them are still to come.
__device__ __forceinline__ int64_t next_arrival_listed(const SegArgs &a, const SegCtx &c, uint32_t b, int64_t n_act, int64_t n,
                                                       int64_t first, int64_t stride) {
  int64_t v = HFX_INF;
  for (int64_t q = n_act + first; q < n; q += stride) {
    const int32_t row = a.order[b + q];
    if (c.rowflag[row] == KIND_FUTURE) { const int64_t x = a.arrival[row]; v = x < v ? x : v; }
  }
  return v;
}

// The same when the inactive rows are not listed yet (a long list that the grid writes at the end of the kernel):
// read from the slabs.  The warps of the group share the tiles; a warp reads the descriptors of 32 of its tiles at
// once (a lane each), then walks them one by one, its lanes over the replica's inactive rows of the tile, the row
// kind and the arrival of a row asked for together.  All threads of the group call.
__device__ __forceinline__ int64_t next_arrival_slabs(const SegArgs &a, const SegCtx &c, int R1, int r, const Grp &G) {
  const int lane = G.tid & 31, warp = G.tid >> 5, nwarp = G.n >> 5;
  int64_t v = HFX_INF;
  for (int t0 = warp; t0 < c.n_tiles; t0 += 32 * nwarp) {      // this warp's tiles t0, t0 + nwarp, ...: 32 at a time
    const int t = t0 + lane * nwarp;
    uint32_t ci = 0, src = 0;
    if (t < c.n_tiles) {
      const uint2 m = __ldcg(c.M + (size_t)t * R1 + r);
      const uint32_t ca = m.y >> 16;
      ci = (m.x >> 16) - ca; src = (m.x & 0xffffu) + ca;
    }
    uint32_t some = __ballot_sync(0xffffffffu, ci != 0);
    while (some) {
      const int l = __ffs(some) - 1;
      some &= some - 1;
      const uint32_t src_l = __shfl_sync(0xffffffffu, src, l), ci_l = __shfl_sync(0xffffffffu, ci, l);
      const size_t tb = (size_t)(t0 + l * nwarp) * c.tile_rows;
#pragma unroll 2
      for (uint32_t k = lane; k < ci_l; k += 32) {
        const size_t row = tb + __ldcg(c.slab_idx + tb + src_l + k);
        const uint8_t kind = c.rowflag[row];
        const int64_t x = a.arrival[row];
        if (kind == KIND_FUTURE && x < v) v = x;
      }
    }
  }
  return v;
}

// minimum of v over the group into sh.next_arrival (all threads of the group call)
__device__ __forceinline__ void group_min_arrival(int64_t v, BlockShared &sh, const Grp &G) {
  const int lane = G.tid & 31, warp = G.tid >> 5, nwarp = G.n >> 5;
  v = warp_min_i64(v);
  G.sync();
  if (lane == 0) sh.red_c[warp] = v;
  G.sync();
  if (G.tid == 0) {
    int64_t m = sh.next_arrival;
    for (int k = 0; k < nwarp; k++) m = sh.red_c[k] < m ? sh.red_c[k] : m;
    sh.next_arrival = m;
  }
  G.sync();
}

// ---- gathering a replica's rows from the tile slabs -------------------------------------------------
// Replica r's chunks are taken in tile order, TPT * G.n tiles per round: a thread reads the chunk
// descriptors of TPT neighbouring tiles, an exclusive scan over the round's tiles gives each chunk's
// place inside the replica (row order, since tiles and the rows inside a chunk are in row order); then
// the round's rows are spread evenly over the threads, each finding its chunk by a binary search over the
// round's prefixes, a few rows at a time so that their loads are in flight together.
// emit_act(pos, rec, row) is called once for the pos-th active row, emit_in(pos, row) for the pos-th
// inactive row (only if list_in; active rows only if take_act).
// Shared memory: GatherTiles for TPT * G.n tiles.  The slabs were written by the previous kernel: L2 loads.
struct GatherTiles {
  uint32_t *pa, *pi;          // [n] active / inactive rows of the replica in the round's earlier tiles
  uint16_t *oa, *oall, *ca;   // [n] chunk descriptor: first record, first row index, active rows
  uint32_t *scan;             // [2 * warps + 2]
  uint8_t *own_a, *own_i;     // optional (small replicas, n <= 256): the tile of every active / inactive row of the round
};
__host__ __device__ constexpr size_t gather_tiles_bytes(int n_tiles, int n_threads) { return (size_t)n_tiles * 14 + 4 * (2 * (size_t)(n_threads / 32) + 2); }
__device__ __forceinline__ GatherTiles gather_tiles_at(unsigned char *smem, int n_tiles, int n_threads) {
  GatherTiles g;
  g.pa = reinterpret_cast<uint32_t *>(smem); g.pi = g.pa + n_tiles; g.scan = g.pi + n_tiles;
  g.oa = reinterpret_cast<uint16_t *>(g.scan + 2 * (n_threads / 32) + 2); g.oall = g.oa + n_tiles; g.ca = g.oall + n_tiles;
  g.own_a = nullptr; g.own_i = nullptr;
  return g;
}

__device__ __forceinline__ void cp_async8(void *smem_dst, const void *gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// where an asynchronous gather puts the active rows (shared memory): slack base, record words z and w, row index
struct GatherDst { uint64_t *bk; uint2 *zw; int32_t *row; };

// ASYNC: the records of the active rows are copied global -> shared memory without passing through registers (two
// 8-byte cp.async per row, all of a round in flight together; the caller waits for them with cp_async_wait_all and
// a barrier) and emit_act is not called.
template <int NT, int TPT, bool OWNER, bool ASYNC, class ActF, class InF>      // NT = G.n threads, TPT tiles per thread and round; NT * TPT a power of two
__device__ __forceinline__ void gather_replica(const SegCtx &c, int R1, int r, const Grp &G, const GatherTiles &gt, bool take_act,
                                               bool list_in, ActF emit_act, InF emit_in, const GatherDst dst = GatherDst()) {
  const int lane = G.tid & 31, w = G.tid >> 5, nw = G.n >> 5;
  constexpr int round_tiles = NT * TPT;
  uint32_t base_a = 0, base_i = 0;
  for (int t0 = 0; t0 < c.n_tiles; t0 += round_tiles) {
    uint32_t ca[TPT], ci[TPT], oa[TPT], oall[TPT];
    uint32_t sa = 0, si = 0;
#pragma unroll
    for (int e = 0; e < TPT; e++) {
      const int t = t0 + G.tid * TPT + e;
      ca[e] = 0; ci[e] = 0; oa[e] = 0; oall[e] = 0;
      if (t < c.n_tiles) {
        const uint2 m = __ldcg(c.M + (size_t)t * R1 + r);
        oall[e] = m.x & 0xffffu; oa[e] = m.y & 0xffffu; ca[e] = m.y >> 16; ci[e] = (m.x >> 16) - ca[e];
      }
      sa += ca[e]; si += ci[e];
    }
    const uint32_t mine_a = sa, mine_i = si;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t x = __shfl_up_sync(0xffffffffu, sa, o), y = __shfl_up_sync(0xffffffffu, si, o);
      if (lane >= o) { sa += x; si += y; }
    }
    if (t0 > 0) G.sync();      // the previous round still reads the tile arrays
    if (lane == 31) { gt.scan[2 * w] = sa; gt.scan[2 * w + 1] = si; }
    G.sync();
    uint32_t pa = sa - mine_a, pi = si - mine_i, ta = 0, ti = 0;
    for (int k = 0; k < nw; k++) {
      const uint32_t x = gt.scan[2 * k], y = gt.scan[2 * k + 1];
      if (k < w) { pa += x; pi += y; }
      ta += x; ti += y;
    }
#pragma unroll
    for (int e = 0; e < TPT; e++) {
      const int lt = G.tid * TPT + e;
      const bool in = t0 + lt < c.n_tiles;
      gt.pa[lt] = in ? pa : 0xffffffffu; gt.pi[lt] = in ? pi : 0xffffffffu;
      gt.oa[lt] = (uint16_t)oa[e]; gt.oall[lt] = (uint16_t)oall[e]; gt.ca[lt] = (uint16_t)ca[e];
      if (OWNER) {      // which tile every row of the round comes from (rows are few: a small replica)
        if (take_act) for (uint32_t k = 0; k < ca[e]; k++) gt.own_a[pa + k] = (uint8_t)lt;
        if (list_in) for (uint32_t k = 0; k < ci[e]; k++) gt.own_i[pi + k] = (uint8_t)lt;
      }
      pa += ca[e]; pi += ci[e];
    }
    G.sync();
    // the chunk that holds the q-th row of the round: the last tile whose prefix is <= q
    auto chunk_of = [&](const uint32_t *pre, uint32_t q) -> int {
      int lo = 0;
#pragma unroll
      for (int s = round_tiles >> 1; s > 0; s >>= 1) if (pre[lo + s] <= q) lo += s;
      return lo;
    };
    if (ASYNC && take_act) {
      for (uint32_t q = G.tid; q < ta; q += G.n) {
        const int lt = OWNER ? (int)gt.own_a[q] : chunk_of(gt.pa, q);
        const uint4 *src = c.slab_rec + (size_t)(t0 + lt) * c.tile_rows + gt.oa[lt] + (q - gt.pa[lt]);
        cp_async8(&dst.bk[base_a + q], src);
        cp_async8(&dst.zw[base_a + q], reinterpret_cast<const uint2 *>(src) + 1);
      }
      for (uint32_t q0 = G.tid; q0 < ta; q0 += 4 * G.n) {      // their row indices, four loads in flight per thread
        int32_t row[4];
#pragma unroll
        for (int e = 0; e < 4; e++) {
          const uint32_t q = q0 + e * G.n;
          if (q < ta) {
            const int lt = OWNER ? (int)gt.own_a[q] : chunk_of(gt.pa, q);
            const size_t tb = (size_t)(t0 + lt) * c.tile_rows;
            row[e] = (int32_t)(tb + __ldcg(c.slab_idx + tb + gt.oall[lt] + (q - gt.pa[lt])));
          }
        }
#pragma unroll
        for (int e = 0; e < 4; e++) { const uint32_t q = q0 + e * G.n; if (q < ta) dst.row[base_a + q] = row[e]; }
      }
    } else if (take_act) {
      int lt_c = 0;            // the chunk of my previous row and where it ends: my rows rise, so large chunks are searched once
      uint32_t lim_c = 0;
      for (uint32_t q0 = G.tid; q0 < ta; q0 += 3 * G.n) {
        uint4 rec[3];
        int32_t row[3];
#pragma unroll
        for (int e = 0; e < 3; e++) {
          const uint32_t q = q0 + e * G.n;
          if (q < ta) {
            if (!OWNER && q >= lim_c) { lt_c = chunk_of(gt.pa, q); lim_c = gt.pa[lt_c] + gt.ca[lt_c]; }
            const int lt = OWNER ? (int)gt.own_a[q] : lt_c;
            const uint32_t k = q - gt.pa[lt];
            const size_t tb = (size_t)(t0 + lt) * c.tile_rows;
            rec[e] = __ldcg(c.slab_rec + tb + gt.oa[lt] + k);
            row[e] = (int32_t)(tb + __ldcg(c.slab_idx + tb + gt.oall[lt] + k));
          }
        }
#pragma unroll
        for (int e = 0; e < 3; e++) { const uint32_t q = q0 + e * G.n; if (q < ta) emit_act(base_a + q, rec[e], row[e]); }
      }
    }
    if (list_in)
      for (uint32_t q0 = G.tid; q0 < ti; q0 += 4 * G.n) {
        int32_t row[4];
#pragma unroll
        for (int e = 0; e < 4; e++) {
          const uint32_t q = q0 + e * G.n;
          if (q < ti) {
            const int lt = OWNER ? (int)gt.own_i[q] : chunk_of(gt.pi, q);
            const uint32_t k = q - gt.pi[lt];
            const size_t tb = (size_t)(t0 + lt) * c.tile_rows;
            row[e] = (int32_t)(tb + __ldcg(c.slab_idx + tb + gt.oall[lt] + gt.ca[lt] + k));
          }
        }
#pragma unroll
        for (int e = 0; e < 4; e++) { const uint32_t q = q0 + e * G.n; if (q < ti) emit_in(base_i + q, row[e]); }
      }
    base_a += ta; base_i += ti;
  }
}

// First-fit admission along the order by the first warp of G; marks what it takes in bit 17 of s_lo.
template <class CostF>
__device__ __forceinline__ void first_fit_marks(const ReplicaPlan &pl, uint32_t *s_lo, int n_sorted, const Grp &G, CostF cost_of) {
  if ((G.tid >> 5) == 0) {
    const int64_t room = pl.batch_cap == 0 ? HFX_INF : (pl.batch_cap > pl.n_eff ? pl.batch_cap - pl.n_eff : 0);
    warp_first_fit(n_sorted, pl.budget, room, G.tid & 31, cost_of, [&](int64_t q, bool taken) { if (taken) s_lo[q] |= 0x20000u; });
  }
  G.sync();
}

// Distribution sort, bin layout (one warp; all 32 lanes call): every (phase, priority) class gets a share of the
// n_bins bins in proportion to its items (a power of two; the shares add up to at most n_bins - TINY_CLASSES) and
// the shift that maps its range of sub-keys onto its bins.  cinfo[class] = (smallest sub-key, first bin | shift << 16).
template <int N_BINS>
__device__ __forceinline__ void layout_class_bins(const uint32_t *s_ccnt, const uint32_t *s_cmin, const uint32_t *s_cmax, uint2 *s_cinfo,
                                                  uint32_t n_items, int lane) {
  uint32_t nb[TINY_CLASSES / 32], sft[TINY_CLASSES / 32], lo_[TINY_CLASSES / 32];
  uint32_t sum = 0;
#pragma unroll
  for (int e = 0; e < TINY_CLASSES / 32; e++) {
    const int cl = lane * (TINY_CLASSES / 32) + e;
    const uint32_t cnt = s_ccnt[cl], lo = s_cmin[cl], hi = s_cmax[cl];
    uint32_t want = cnt * (uint32_t)(N_BINS - TINY_CLASSES) / n_items;
    nb[e] = cnt ? (want > 1 ? 1u << (31 - __clz(want)) : 1u) : 0u;
    const uint32_t range = cnt ? hi - lo : 0u;
    const int bits = 32 - __clz(range), lg = 31 - __clz(nb[e] | 1u);
    sft[e] = bits > lg ? (uint32_t)(bits - lg) : 0u;       // (range >> sft) < nb
    lo_[e] = lo;
    sum += nb[e];
  }
  uint32_t v = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
  uint32_t run = v - sum;
#pragma unroll
  for (int e = 0; e < TINY_CLASSES / 32; e++) { s_cinfo[lane * (TINY_CLASSES / 32) + e] = make_uint2(lo_[e], run | (sft[e] << 16)); run += nb[e]; }
}

// ------------------------------------------------------------------------------------------------
// Small replicas: one group of 128 threads.  What later passes need of the replica's active rows
// (slack base, record words, row) is staged once in shared memory; sort items live in registers
// until they are scattered into their bins.
// ------------------------------------------------------------------------------------------------
#define SMALL_SMEM (SEG_TINY * 24 + (TINY_BINS + 4) * 4 + TINY_CLASSES * 8)
static_assert(SMALL_SMEM <= SMEM_GROUP, "a group's arrays fit its share of the block's shared memory");

template <bool SLABS, bool FF>
__device__ void small_replica(const HfxParams &p, const SegArgs &a, const SegCtx &c, const Grp &G, int r, uint32_t b, int n,
                              int n_act, bool ordered, bool list_in, unsigned char *smem, BlockShared &sh,
                              const int64_t *s_cls_ttft, const int64_t *s_cls_tpot) {
  uint64_t *s_bk = reinterpret_cast<uint64_t *>(smem);                     // [SEG_TINY] slack base of every active row; then the sort items, binned
  uint2 *s_zw = reinterpret_cast<uint2 *>(s_bk + SEG_TINY);                // [SEG_TINY] record words z, w; bit 31 of w: admitted
  int32_t *s_row = reinterpret_cast<int32_t *>(s_zw + SEG_TINY);           // [SEG_TINY]
  uint32_t *s_lo = reinterpret_cast<uint32_t *>(s_row + SEG_TINY);         // [SEG_TINY] order (+ tie-break words)
  uint32_t *s_bin = s_lo + SEG_TINY;                                       // [TINY_BINS / 2 + 4] bin counts, then bin starts; two 16-bit values to a word
  uint32_t *s_cur = s_bin + TINY_BINS / 2 + 4;                             // [TINY_BINS / 2] fill cursors, then bin ends
  uint2 *s_cinfo = reinterpret_cast<uint2 *>(s_cur + TINY_BINS / 2);       // [TINY_CLASSES] per class: smallest sub-key; first bin | shift << 16
  // over s_lo .. s_cur while the gather runs: the round's tile descriptors
  GatherTiles gt = gather_tiles_at(reinterpret_cast<unsigned char *>(s_lo), GROUP_THREADS * GROUP_TPT, GROUP_THREADS);
  gt.own_a = reinterpret_cast<uint8_t *>(s_lo) + ((gather_tiles_bytes(GROUP_THREADS * GROUP_TPT, GROUP_THREADS) + 15) & ~(size_t)15);
  gt.own_i = gt.own_a + SEG_TINY;
  static_assert(((gather_tiles_bytes(GROUP_THREADS * GROUP_TPT, GROUP_THREADS) + 15) & ~(size_t)15) + SEG_TINY + LIST_MAX <=
                (size_t)SEG_TINY * 4 + (TINY_BINS + 4) * 4, "the gather's scratch fits over the order and bin arrays");
  // over s_lo until the ranks are written: per class the smallest and largest sub-key and the number of items
  uint32_t *s_cmin = s_lo, *s_cmax = s_lo + TINY_CLASSES, *s_ccnt = s_lo + 2 * TINY_CLASSES;
  const int R = p.n_replicas, R1 = R + 1;
  const int lane = G.tid & 31, warp = G.tid >> 5, nwarp = G.n >> 5;
  const int n_in = n - n_act;
  const bool real = r < R;    // bucket R holds rows bound to no replica
  const HfxRec *seg = c.rec + b;   // (fallback layout only)

  // the replica's state, asked for early by the planning warp and used after the gather
  hfx_replica_cfg cfg; cfg.mode = HFX_COLOCATED; cfg.token_cap = 1; cfg.batch_cap = 0;
  int64_t now = 0, mat = 0;
  if (warp == 0 && real) { cfg = a.cfg[r]; now = a.now[r]; mat = a.mat[r]; }

  // ---- a step that is not ordered: the inactive rows, listed by req_id behind the active ones --------
  if (!ordered && n_in > 0) {
    if (SLABS)
      gather_replica<GROUP_THREADS, GROUP_TPT, true, false>(c, R1, r, G, gt, false, true, [](uint32_t, const uint4, int32_t) {},
                                                            [&](uint32_t pos, int32_t row) { s_row[pos] = row; });
    else
      for (int q = G.tid; q < n_in; q += G.n) s_row[q] = (int32_t)__ldg(reinterpret_cast<const uint4 *>(seg + n_act + q)).w;
    G.sync();
    for (int q = G.tid; q < n_in; q += G.n) s_bk[q] = ((uint64_t)((uint32_t)__ldg(a.req_id + s_row[q]) ^ 0x80000000u) << 16) | (uint32_t)q;
    G.sync();
    group_sort<false>(s_bk, nullptr, n_in, G);
    for (int q = G.tid; q < n_in; q += G.n) a.order[b + n_act + q] = s_row[s_bk[q] & 0xffffu];
    G.sync();
  }

  // ---- gather: base, record words and row of the active rows; the inactive rows' places ----------------------
  if (SLABS) {
    GatherDst dst; dst.bk = s_bk; dst.zw = s_zw; dst.row = s_row;
    gather_replica<GROUP_THREADS, GROUP_TPT, true, true>(c, R1, r, G, gt, true, ordered && list_in, [](uint32_t, const uint4, int32_t) {},
                                                         [&](uint32_t pos, int32_t row) { a.order[b + n_act + pos] = row; }, dst);
    cp_async_wait_all();
  } else {
    for (int q = G.tid; q < n_act; q += G.n) {
      const uint4 w0 = __ldg(reinterpret_cast<const uint4 *>(seg + q));
      const uint4 w1 = __ldg(reinterpret_cast<const uint4 *>(seg + q) + 1);
      s_bk[q] = ((uint64_t)w0.y << 32) | w0.x;
      s_zw[q] = make_uint2(w1.x | (((w1.w >> 8) & 1u) << CREC_KIND_SHIFT) | (((w1.w >> 16) & 0x3fu) << CREC_PRIO_SHIFT),
                           w1.y | ((w1.w & 0x3fu) << CREC_CLS_SHIFT));
      s_row[q] = (int32_t)w0.w;
    }
  }
  G.sync();       // the gather is over: its tile descriptors may be overwritten

  // ---- aggregates -> plan ----------------------------------------------------------------------------
  uint32_t n_run = 0;
  int64_t sum_kv = 0;
  uint64_t m_run = 0, m_q = 0;
#pragma unroll
  for (int k = 0; k < TINY_IPT; k++) {
    const int q = G.tid + k * GROUP_THREADS;
    if (q < n_act) {
      const uint2 zw = s_zw[q];
      const uint32_t cls = zw.y >> CREC_CLS_SHIFT;
      if (((zw.x >> CREC_KIND_SHIFT) & 1u) == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(zw.x & CREC_LEN_MASK) + (zw.y & CREC_LEN_MASK); m_run |= 1ull << cls; }
      else m_q |= 1ull << cls;
    }
  }
  n_run = __reduce_add_sync(0xffffffffu, n_run);
  sum_kv = warp_sum_i64(sum_kv);
  m_run = ((uint64_t)__reduce_or_sync(0xffffffffu, (uint32_t)(m_run >> 32)) << 32) | __reduce_or_sync(0xffffffffu, (uint32_t)m_run);
  m_q = ((uint64_t)__reduce_or_sync(0xffffffffu, (uint32_t)(m_q >> 32)) << 32) | __reduce_or_sync(0xffffffffu, (uint32_t)m_q);
  if (lane == 0) { sh.red_a[warp] = n_run; sh.red_b[warp] = sum_kv; sh.red_m0[warp] = m_run; sh.red_m1[warp] = m_q; }
  for (int i = G.tid; i < TINY_BINS / 2 + 2; i += G.n) s_bin[i] = 0;
  for (int i = G.tid; i < TINY_CLASSES; i += G.n) { s_cmin[i] = 0xffffffffu; s_cmax[i] = 0; s_ccnt[i] = 0; }
  G.sync();
  if (warp == 0) {     // the whole first warp finishes the reduction and plans
    int64_t nr = 0, kv = 0;
    uint64_t mr = 0, mq = 0;
    for (int k = 0; k < nwarp; k++) { nr += sh.red_a[k]; kv += sh.red_b[k]; mr |= sh.red_m0[k]; mq |= sh.red_m1[k]; }
    ReplicaPlan pl0;
    warp_plan(p, s_cls_ttft, s_cls_tpot, cfg, now, mat, nr, kv, mr, mq, pl0, lane);
    if (lane == 0) { sh.plan = pl0; sh.next_arrival = HFX_INF; }
  }
  G.sync();
  const ReplicaPlan pl = sh.plan;

  // ---- keys (in registers); per class their range ---------------------------------------------------
  uint64_t item[TINY_IPT];
  int32_t out_len[TINY_IPT];       // of my rows in flight, asked for now and used by the commit
  const bool will_commit = real && (a.flags & HFX_COMMIT) && pl.now <= a.horizon;
#pragma unroll
  for (int k = 0; k < TINY_IPT; k++) {
    const int q = G.tid + k * GROUP_THREADS;
    item[k] = ~0ull;
    out_len[k] = 0;
    if (q < n_act) {
      if (will_commit && ((s_zw[q].x >> CREC_KIND_SHIFT) & 1u) == KIND_RUNNING) out_len[k] = __ldg(a.output_len + s_row[q]);
      const int64_t base = (int64_t)s_bk[q];
      const uint2 zw = s_zw[q];
      const int kind = (zw.x >> CREC_KIND_SHIFT) & 1, prio = zw.x >> CREC_PRIO_SHIFT;
      const bool given = kind == KIND_QUEUED && pl.mode != HFX_DECODE;      // the front end has put the row's final key in place of the base
      RowEval e;
      if (given) { e.k48 = (uint64_t)base; e.slack = 0; e.pred_tpot = a.pred_tpot ? pl.tpot_q0 + p.d2 * ((int64_t)(zw.x & CREC_LEN_MASK) + (zw.y & CREC_LEN_MASK)) : 0; }
      else e = eval_row(p, pl, base, kind, prio, (int32_t)(zw.x & CREC_LEN_MASK), (int32_t)(zw.y & CREC_LEN_MASK));
      if (ordered) {
        item[k] = (e.k48 << 16) | (uint32_t)q;     // rows were gathered in req_id order: position breaks ties
        const uint32_t cl = (uint32_t)(item[k] >> 56), sub = (uint32_t)(item[k] >> 24);
        atomicMin(&s_cmin[cl], sub); atomicMax(&s_cmax[cl], sub); atomicAdd(&s_ccnt[cl], 1u);
      } else {
        const uint32_t uid = (uint32_t)__ldg(a.req_id + s_row[q]) ^ 0x80000000u;
        s_bk[q] = (e.k48 << 16) | (uid >> 16);
        s_lo[q] = (uid << 16) | (uint32_t)q;
      }
      if (kind == KIND_RUNNING || pl.mode == HFX_DECODE) {    // (the front end wrote the slack of the other queued rows)
        const int32_t row = s_row[q];
        a.slack[row] = e.slack;
        if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | e.k48;
      }
      if (a.pred_tpot) a.pred_tpot[s_row[q]] = e.pred_tpot;
    }
  }

  // ---- sort --------------------------------------------------------------------------------------------
  // Distribution sort.  The top 8 bits of an item are its class (phase, priority); inside a class items are
  // spread over the class's share of the bins by their sub-key (slack >> 8) between the class's smallest and
  // largest, so bins stay in item order; an item's place inside its bin comes from counting the smaller
  // items of the bin.
  bool sorted_done = false;
  if (ordered && n_act > 0) {
    G.sync();
    if (warp == 0) layout_class_bins<TINY_BINS>(s_ccnt, s_cmin, s_cmax, s_cinfo, (uint32_t)n_act, lane);
    G.sync();
    auto bin_of = [&](uint64_t x) -> uint32_t {
      const uint2 ci = s_cinfo[(uint32_t)(x >> 56)];
      return (ci.y & 0xffffu) + (((uint32_t)(x >> 24) - ci.x) >> (ci.y >> 16));
    };
    uint32_t bins[TINY_IPT];
#pragma unroll
    for (int k = 0; k < TINY_IPT; k++) {
      bins[k] = 0;
      if (G.tid + k * GROUP_THREADS < n_act) { bins[k] = bin_of(item[k]); atomicAdd(&s_bin[bins[k] >> 1], 1u << ((bins[k] & 1u) * 16)); }
    }
    G.sync();
    {   // exclusive scan of the 1024 bin counts: 8 per thread; the largest bin
      const uint4 wd = reinterpret_cast<const uint4 *>(s_bin)[G.tid];
      const uint32_t ww[4] = {wd.x, wd.y, wd.z, wd.w};
      uint32_t cnt[8], sum = 0, big = 0;
#pragma unroll
      for (int i = 0; i < 4; i++) { cnt[2 * i] = ww[i] & 0xffffu; cnt[2 * i + 1] = ww[i] >> 16; }
#pragma unroll
      for (int i = 0; i < 8; i++) { sum += cnt[i]; big = cnt[i] > big ? cnt[i] : big; }
      uint32_t v = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
      big = __reduce_max_sync(0xffffffffu, big);
      if (lane == 31) sh.red_n[warp] = (int32_t)v;
      if (lane == 0) sh.red_n[8 + warp] = (int32_t)big;
      G.sync();
      uint32_t run = v - sum, bigall = 0;
      for (int k = 0; k < nwarp; k++) { if (k < warp) run += (uint32_t)sh.red_n[k]; const uint32_t x = (uint32_t)sh.red_n[8 + k]; bigall = x > bigall ? x : bigall; }
      if (bigall <= TINY_BIN_MAX) {
        uint32_t st[8];
#pragma unroll
        for (int i = 0; i < 8; i++) { st[i] = run; run += cnt[i]; }
        const uint4 o4 = make_uint4(st[0] | (st[1] << 16), st[2] | (st[3] << 16), st[4] | (st[5] << 16), st[6] | (st[7] << 16));
        reinterpret_cast<uint4 *>(s_bin)[G.tid] = o4;
        reinterpret_cast<uint4 *>(s_cur)[G.tid] = o4;
        sorted_done = true;
      }
    }
    G.sync();
    if (sorted_done) {
#pragma unroll
      for (int k = 0; k < TINY_IPT; k++)
        if (G.tid + k * GROUP_THREADS < n_act) {
          const uint32_t sh16 = (bins[k] & 1u) * 16;
          const uint32_t pos = (atomicAdd(&s_cur[bins[k] >> 1], 1u << sh16) >> sh16) & 0xffffu;
          s_bk[pos] = item[k];
        }
      G.sync();
#pragma unroll
      for (int k = 0; k < TINY_IPT; k++) {
        const int e = G.tid + k * GROUP_THREADS;
        if (e < n_act) {
          const uint64_t x = s_bk[e];
          const uint32_t bi = bin_of(x), sh16 = (bi & 1u) * 16;
          const uint32_t g0 = (s_bin[bi >> 1] >> sh16) & 0xffffu, g1 = (s_cur[bi >> 1] >> sh16) & 0xffffu;
          uint32_t rank = 0;
          for (uint32_t g = g0; g < g1; g++) rank += s_bk[g] < x ? 1u : 0u;
          s_lo[g0 + rank] = (uint32_t)(x & 0xffffu);      // (the class ranges that s_lo overlays were last read when the bins were laid out)
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < TINY_IPT; k++) { const int q = G.tid + k * GROUP_THREADS; if (q < n_act) s_bk[q] = item[k]; }
    }
  }
  G.sync();
  if (!sorted_done) {
    if (ordered) {
      group_sort<false>(s_bk, nullptr, n_act, G);
      for (int q = G.tid; q < n_act; q += G.n) s_lo[q] = (uint32_t)(s_bk[q] & 0xffffu);
    } else {
      group_sort<true>(s_bk, s_lo, n_act, G);
      for (int q = G.tid; q < n_act; q += G.n) s_lo[q] &= 0xffffu;
    }
    G.sync();
  }

  auto cost_at = [&](uint32_t li, int64_t &kv) -> int64_t {      // cost of the queued row at record li, -1 if it is in flight
    const uint2 zw = s_zw[li];
    if (((zw.x >> CREC_KIND_SHIFT) & 1u) != KIND_QUEUED) return -1;
    kv = (int64_t)(zw.x & CREC_LEN_MASK) + (zw.y & CREC_LEN_MASK);
    return pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(zw.x & CREC_LEN_MASK);
  };

  // ---- first-fit variant: the first warp walks the order and marks what it takes (bit 17) -----------
  if (FF)
    first_fit_marks(pl, s_lo, n_act, G, [&](int64_t q) -> int64_t { int64_t kv; return cost_at(s_lo[q] & 0xffffu, kv); });

  // ---- admission: each thread walks TINY_IPT consecutive places of the order ---------------------
  const int q0 = G.tid * TINY_IPT;
  uint32_t cand[TINY_IPT];      // record position of the candidate at each of my places | 0x80000000, or 0
  uint64_t mine = 0;            // cost | count << 48 of the candidates of this thread (costs stay below 2^44 in total)
#pragma unroll
  for (int k = 0; k < TINY_IPT; k++) {
    const int q = q0 + k;
    cand[k] = 0;
    if (q < n_act) {
      const uint32_t li = s_lo[q] & 0xffffu;
      int64_t kv = 0;
      const int64_t cc = cost_at(li, kv);
      // what counts towards the totals: rows that fit alone, or (first fit) exactly the rows taken
      if (cc >= 0 && (FF ? (s_lo[q] & 0x20000u) != 0 : cc <= pl.budget)) { cand[k] = li | 0x80000000u; mine += (uint64_t)cc + (1ull << 48); }
      a.order[b + q] = s_row[li];
    }
  }
  uint64_t sc = (uint64_t)warp_incl_scan_i64((int64_t)mine, lane);
  if (lane == 31) sh.red_m0[warp] = sc;
  G.sync();
  uint64_t run = sc - mine;
  for (int k = 0; k < warp; k++) run += sh.red_m0[k];
  int64_t run_c = (int64_t)(run & ((1ull << 48) - 1));
  int32_t run_n = (int32_t)(run >> 48);
  int64_t ac = 0, ak = 0;
  int32_t an = 0;
#pragma unroll
  for (int k = 0; k < TINY_IPT; k++) {
    if (cand[k]) {
      const uint32_t li = cand[k] & 0xffffu;
      int64_t kv = 0;
      const int64_t cc = cost_at(li, kv);
      run_c += cc; run_n += 1;
      if (FF || (run_c <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + run_n <= pl.batch_cap))) {
        ac += cc; ak += kv; an++;
        const int32_t row = s_row[li];
        a.admit[row] = 1;
        if (a.admitted_rows) a.admitted_rows[b + run_n - 1] = row;
        s_zw[li].y |= 0x80000000u;
      }
    }
  }

  // ---- totals, maturity, replica outputs, commit ---------------------------------------------------------
  ac = warp_sum_i64(ac); ak = warp_sum_i64(ak); an = (int32_t)__reduce_add_sync(0xffffffffu, (uint32_t)an);
  if (lane == 0) { sh.red_a[warp] = ac; sh.red_b[warp] = ak; sh.red_n[warp] = an; }
  G.sync();
  if (G.tid == 0) {
    int64_t adm_cost = 0, adm_kv = 0; int32_t adm_count = 0;
    for (int k = 0; k < nwarp; k++) { adm_cost += sh.red_a[k]; adm_kv += sh.red_b[k]; adm_count += sh.red_n[k]; }
    int64_t lp = 0;
    const int64_t mat_next = dev_maturity_next(p, pl, adm_count, adm_cost, adm_kv, &lp);
    int worked; int64_t t1, t2;
    iteration_clock(pl, adm_count, lp, mat_next, worked, t1, t2);
    sh.adm_cost = adm_cost; sh.adm_count = adm_count;
    sh.worked = worked; sh.t1 = t1; sh.t2 = t2; sh.red_c[0] = mat_next;
  }
  G.sync();
  const bool commit = real && (a.flags & HFX_COMMIT) && pl.now <= a.horizon;
  const int worked = sh.worked;
  const int64_t mat_next = sh.red_c[0];
  if (commit && !worked) {
    // idle replica: its next arrival is looked up among its listed inactive rows (unless the grid lists them later)
    group_min_arrival(list_in || !ordered ? next_arrival_listed(a, c, b, n_act, n, G.tid, G.n) : next_arrival_slabs(a, c, R1, r, G), sh, G);
  }
  if (G.tid == 0 && real)
    write_replica_outputs(a, r, pl, sh.adm_cost, sh.adm_count, mat_next, worked, sh.t2, sh.next_arrival);
  if (a.admitted_rows)
    for (int q = sh.adm_count + G.tid; q < n; q += G.n) a.admitted_rows[b + q] = -1;
  if (commit) {      // every thread its own rows; an admitted row's output length is fetched now (there are few)
    const int64_t t1 = sh.t1, t2 = sh.t2;
#pragma unroll
    for (int k = 0; k < TINY_IPT; k++) {
      const int q = G.tid + k * GROUP_THREADS;
      if (q < n_act) {
        const uint2 zw = s_zw[q];
        const int kind = (zw.x >> CREC_KIND_SHIFT) & 1;
        const bool adm = (zw.y >> 31) != 0;
        const int32_t ol = adm ? __ldg(a.output_len + s_row[q]) : out_len[k];
        commit_row(a, pl, kind, adm, worked, t1, t2, s_row[q], (int32_t)(zw.x & CREC_LEN_MASK), (int32_t)(zw.y & CREC_LEN_MASK), ol);
      }
    }
  }
  G.sync();
}

// ------------------------------------------------------------------------------------------------
// Larger replicas: the whole block.  Their records are first gathered into the contiguous scratch range
// [b, b + n) of c.rec (32-byte records, active rows first), which the passes below read by position.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_rec(const HfxRec *rec, int half) { return *(reinterpret_cast<const uint4 *>(rec) + half); }

__device__ void gather_to_records(const SegArgs &a, const SegCtx &c, int R1, int r, uint32_t b, int64_t n_act, bool ordered,
                                  bool list_in, unsigned char *smem) {
  const Grp B = {(int)threadIdx.x, (int)blockDim.x, 0};
  HfxRec *seg = c.rec + b;
  gather_replica<REP_THREADS, 1, false, false>(c, R1, r, B, gather_tiles_at(smem, REP_THREADS, REP_THREADS), true, list_in || !ordered,
                 [&](uint32_t pos, const uint4 rec, int32_t row) {
                   uint4 w0, w1;
                   w0.x = rec.x; w0.y = rec.y; w0.z = ordered ? 0u : (uint32_t)__ldg(a.req_id + row); w0.w = (uint32_t)row;
                   w1.x = rec.z & CREC_LEN_MASK; w1.y = rec.w & CREC_LEN_MASK; w1.z = 0;
                   w1.w = (rec.w >> CREC_CLS_SHIFT) | (((rec.z >> CREC_KIND_SHIFT) & 1u) << 8) | ((rec.z >> CREC_PRIO_SHIFT) << 16);
                   uint4 *dst = reinterpret_cast<uint4 *>(seg + pos);
                   dst[0] = w0; dst[1] = w1;
                 },
                 [&](uint32_t pos, int32_t row) {
                   if (ordered) a.order[b + n_act + pos] = row;
                   else {
                     uint4 *dst = reinterpret_cast<uint4 *>(seg + n_act + pos);
                     dst[0] = make_uint4(0u, 0u, (uint32_t)__ldg(a.req_id + row), (uint32_t)row);
                     dst[1] = make_uint4(0u, 0u, 0u, KIND_DEAD << 8);
                   }
                 });
  __syncthreads();
}

// the block's partial aggregates of a replica's active rows -> its plan (all threads call; result in sh.plan)
__device__ __forceinline__ void block_plan(const HfxParams &p, const SegArgs &a, int r, bool real, BlockShared &sh,
                                           int64_t n_run, int64_t sum_kv, uint64_t m_run, uint64_t m_q) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
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

// aggregates of a replica's active records into the block's plan (all threads call; result in sh.plan)
__device__ __forceinline__ void segment_plan(const HfxParams &p, const SegArgs &a, const HfxRec *seg, int64_t n_act, int r,
                                             bool real, BlockShared &sh) {
  int64_t n_run = 0, sum_kv = 0;
  uint64_t m_run = 0, m_q = 0;
#pragma unroll 4
  for (int64_t q = threadIdx.x; q < n_act; q += blockDim.x) {
    const uint4 w1 = ld_rec(seg + q, 1);   // prompt, gen, -, bytes
    const int kind = (w1.w >> 8) & 0xff, cls = w1.w & 0xff;
    if (kind == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(int32_t)w1.x + (int32_t)w1.y; m_run |= 1ull << cls; }
    else m_q |= 1ull << cls;
  }
  block_plan(p, a, r, real, sh, n_run, sum_kv, m_run, m_q);
}

// Block-wide admission over the sorted items s_lo[0..n_sorted) (low 16 bits = position of the
// record inside the segment): writes order, admit and the compacted admitted list, keeps each
// decision in bit 16 of s_lo, accumulates the totals in sh.
template <bool FF>
__device__ __forceinline__ void segment_admit(const HfxParams &p, const SegArgs &a, const ReplicaPlan &pl,
                                              const HfxRec *seg, uint32_t b, uint32_t *s_lo, int n_sorted,
                                              BlockShared &sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  if (FF) {
    const Grp B = {(int)threadIdx.x, (int)blockDim.x, 0};
    first_fit_marks(pl, s_lo, n_sorted, B, [&](int64_t q) -> int64_t {
      const uint4 w1 = ld_rec(seg + (s_lo[q] & 0xffffu), 1);
      if (((w1.w >> 8) & 0xff) != KIND_QUEUED) return -1;
      return pl.mode == HFX_DECODE ? p.d1 + p.d2 * ((int64_t)(int32_t)w1.x + (int32_t)w1.y) : (int64_t)(int32_t)w1.x;
    });
  }
  // The order begins with the requests in flight (phase 0 sorts first): they are only listed, no
  // prefix is needed for them.  Whole tiles of them are passed here; the scan starts at the tile that
  // reaches the queue.
  const int n_front = (int)((pl.n_run < n_sorted ? pl.n_run : n_sorted) / blockDim.x) * blockDim.x;
  for (int q = threadIdx.x; q < n_front; q += blockDim.x) {
    const uint32_t li = s_lo[q] & 0xffffu;
    a.order[b + q] = (int32_t)ld_rec(seg + li, 0).w;
    s_lo[q] = li;
  }
  for (int tile = n_front; tile < n_sorted; tile += blockDim.x) {
    const int q = tile + threadIdx.x;
    int64_t cost = 0, kv = 0;
    int32_t cnt = 0, row = -1, kind = KIND_DEAD;
    if (q < n_sorted) {
      const int li = s_lo[q] & 0xffff;
      const uint4 w0 = ld_rec(seg + li, 0);
      const uint4 w1 = ld_rec(seg + li, 1);
      row = (int32_t)w0.w;
      kind = (w1.w >> 8) & 0xff;
      if (kind == KIND_QUEUED) {
        kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
        const int64_t c = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
        if (FF ? (s_lo[q] & 0x20000u) != 0 : c <= pl.budget) { cost = c; cnt = 1; } else kv = 0;
      }
      a.order[b + q] = row;
    }
    if (!__syncthreads_or(cnt)) {      // no candidate in this tile (a spent budget, requests in flight): nothing to add up
      if (q < n_sorted) s_lo[q] &= 0xffffu;
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
    if (cnt) adm = FF || (sc <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + sn <= pl.batch_cap));
    if (q < n_sorted) {
      if (adm) a.admit[row] = 1;
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
    if (!FF && sh.carry_act &&
        (sh.carry_cost > pl.budget || (pl.batch_cap != 0 && pl.n_eff + sh.carry_count >= pl.batch_cap))) {
      for (int q = tile + blockDim.x + threadIdx.x; q < n_sorted; q += blockDim.x) {
        const uint32_t li = s_lo[q] & 0xffffu;
        a.order[b + q] = (int32_t)ld_rec(seg + li, 0).w;
        s_lo[q] = li;
      }
      break;
    }
  }
}

// The sorting network for items of one 64-bit word (ordered steps), with the items held in
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
// order, to pos_out; the caller synchronises before reading pos_out.
__device__ __forceinline__ void sort64_positions(uint64_t *hi, uint32_t *pos_out, int n) {
  if (n > 512) {
    if (n <= 1024) block_sort_reg<1>(hi, pos_out, n);
    else if (n <= 2048) block_sort_reg<2>(hi, pos_out, n);
    else if (n <= 4096) block_sort_reg<4>(hi, pos_out, n);
    else if (n <= 8192) block_sort_reg<8>(hi, pos_out, n);
    else block_sort_reg<16>(hi, pos_out, n);
  } else {
    const Grp B = {(int)threadIdx.x, (int)blockDim.x, 0};
    group_sort<false>(hi, nullptr, n, B);
    for (int q = threadIdx.x; q < n; q += blockDim.x) pos_out[q] = (uint32_t)(hi[q] & 0xffffu);
  }
}

template <bool SLABS, bool FF>
__device__ void medium_replica(const HfxParams &p, const SegArgs &a, const SegCtx &c, int r, uint32_t b, int n, int n_act,
                               bool ordered, bool list_in, unsigned char *smem, BlockShared &sh) {
  uint64_t *s_hi = reinterpret_cast<uint64_t *>(smem);
  uint32_t *s_lo = reinterpret_cast<uint32_t *>(smem + (size_t)SEG_MED * 8);
  const int R = p.n_replicas;
  const Grp B = {(int)threadIdx.x, (int)blockDim.x, 0};
  const int n_in = n - n_act;
  const HfxRec *seg = c.rec + b;
  const bool real = r < R;    // bucket R holds rows bound to no replica
  // ---- gather into contiguous records -----------------------------------------------------------------
  if (SLABS) gather_to_records(a, c, R + 1, r, b, n_act, ordered, list_in, smem);

  // ---- inactive rows of a step that is not ordered: listed by req_id behind the active ones ----
  if (!ordered && n_in > 0) {
    const HfxRec *sin = seg + n_act;
    for (int q = threadIdx.x; q < n_in; q += blockDim.x)
      s_hi[q] = ((uint64_t)(ld_rec(sin + q, 0).z ^ 0x80000000u) << 16) | (uint32_t)q;     // signed req_id order, then position
    __syncthreads();
    sort64_positions(s_hi, s_lo, n_in);
    __syncthreads();
    for (int q = threadIdx.x; q < n_in; q += blockDim.x) a.order[b + n_act + q] = (int32_t)ld_rec(sin + s_lo[q], 0).w;
    __syncthreads();
  }
  // ---- aggregates, plan ---------------------------------------------------------------------------------
  segment_plan(p, a, seg, n_act, r, real, sh);
  const ReplicaPlan pl = sh.plan;

  // ---- sort items of the active rows ---------------------------------------------------------------
#pragma unroll 4
  for (int q = threadIdx.x; q < n_act; q += blockDim.x) {
    const uint4 w0 = ld_rec(seg + q, 0);
    const uint4 w1 = ld_rec(seg + q, 1);
    const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
    const int32_t row = (int32_t)w0.w;
    const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
    RowEval e = eval_row(p, pl, base, kind, prio, (int32_t)w1.x, (int32_t)w1.y);
    if (kind == KIND_QUEUED && pl.mode != HFX_DECODE) e.k48 = (uint64_t)base;      // the front end has put the row's final key in place of the base
    if (ordered) s_hi[q] = (e.k48 << 16) | (uint32_t)q;     // records are in req_id order: position breaks ties
    else {
      const uint32_t uid = w0.z ^ 0x80000000u;               // signed req_id order as unsigned
      s_hi[q] = (e.k48 << 16) | (uid >> 16);
      s_lo[q] = (uid << 16) | (uint32_t)q;
    }
    if (kind == KIND_RUNNING || pl.mode == HFX_DECODE) {    // (the front end wrote the slack of the other queued rows)
      a.slack[row] = e.slack;
      if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | e.k48;
    }
    if (a.pred_tpot) a.pred_tpot[row] = e.pred_tpot;
  }
  __syncthreads();
  // ---- sort ------------------------------------------------------------------------------------------------
  if (ordered) sort64_positions(s_hi, s_lo, n_act);
  else {
    group_sort<true>(s_hi, s_lo, n_act, B);
    for (int q = threadIdx.x; q < n_act; q += blockDim.x) s_lo[q] &= 0xffffu;
  }
  __syncthreads();

  // ---- admission -------------------------------------------------------------------------------------------
  segment_admit<FF>(p, a, pl, seg, b, s_lo, n_act, sh);

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
  if (commit && !worked)      // idle replica: its next arrival is looked up among its listed inactive rows
    group_min_arrival(list_in || !ordered ? next_arrival_listed(a, c, b, n_act, n, threadIdx.x, blockDim.x) : next_arrival_slabs(a, c, p.n_replicas + 1, r, B), sh, B);
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
      const uint4 w0 = ld_rec(seg + li, 0);
      const uint4 w1 = ld_rec(seg + li, 1);
      const int kind = (w1.w >> 8) & 0xff;
      const bool adm = (lo & 0x10000u) != 0;
      const int32_t out_len = commit_needs_out_len(pl, kind, adm, worked) ? __ldg(a.output_len + (int32_t)w0.w) : 0;
      commit_row(a, pl, kind, adm, worked, t1, t2, (int32_t)w0.w, (int32_t)w1.x, (int32_t)w1.y, out_len);
    }
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// Larger replicas of an ordered step on the slab layout: the whole block with a distribution sort.
// The replica's scratch range of c.rec (32 bytes per row, of which 20 per active row are used) holds three
// arrays by position q in row order: slack base, then sort item (8 bytes); record words z, w (8); row (4).
// Every pass reads them front to back; shared memory holds the binned items (afterwards the record words), the
// order as 16-bit positions and the bin counters.
// ------------------------------------------------------------------------------------------------
#define MED_BINS 8192     // bins of the block's distribution sort (16-bit counters, two to a word)
#define MED_BIN_MAX 160   // fuller bins send the replica to the sorting network
static_assert((size_t)SEG_MED * 10 + MED_BINS * 4 <= SMEM_MED, "items, order and bins of a medium replica fit the block's shared memory");
static_assert(MED_BINS / 8 == REP_THREADS, "every thread scans eight bins");

template <bool FF>
__device__ void medium_ordered(const HfxParams &p, const SegArgs &a, const SegCtx &c, int r, uint32_t b, int n, int n_act,
                               bool list_in, unsigned char *smem, BlockShared &sh, uint64_t *s_cinfo,
                               const int64_t *s_cls_ttft, const int64_t *s_cls_tpot) {
  uint64_t *s_item = reinterpret_cast<uint64_t *>(smem);                          // [SEG_MED] items by bin
  uint2 *s_zw = reinterpret_cast<uint2 *>(smem);                                  // [SEG_MED] afterwards: record words by position; bit 31 of x: taken by first fit, of y: admitted
  uint16_t *s_ord = reinterpret_cast<uint16_t *>(smem + (size_t)SEG_MED * 8);     // [SEG_MED] position of the i-th row of the order
  uint32_t *s_bin = reinterpret_cast<uint32_t *>(smem + (size_t)SEG_MED * 10);    // [MED_BINS / 2] bin counts, then bin starts
  uint32_t *s_cur = s_bin + MED_BINS / 2;                                         // [MED_BINS / 2] fill cursors, then bin ends
  uint32_t *s_lo = reinterpret_cast<uint32_t *>(s_ord);                           // (sorting network only: 32-bit positions over order and bins)
  // until the bins are laid out: per class the smallest and largest of the slack's upper 32 bits and of its low 8 bits, the items
  uint32_t *s_cmin = reinterpret_cast<uint32_t *>(s_ord), *s_cmax = s_cmin + TINY_CLASSES, *s_lmin = s_cmax + TINY_CLASSES,
           *s_lmax = s_lmin + TINY_CLASSES, *s_ccnt = s_lmax + TINY_CLASSES;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int R = p.n_replicas;
  const bool real = r < R;    // bucket R holds rows bound to no replica
  const Grp B = {tid, REP_THREADS, 0};
  unsigned char *g = reinterpret_cast<unsigned char *>(c.rec + b);
  uint64_t *g_item = reinterpret_cast<uint64_t *>(g);
  uint2 *g_zw = reinterpret_cast<uint2 *>(g + (size_t)n_act * 8);
  int32_t *g_row = reinterpret_cast<int32_t *>(g + (size_t)n_act * 16);

  // ---- gather into the scratch arrays; the inactive rows go straight to their places -------------------
  gather_replica<REP_THREADS, 1, false, false>(c, R + 1, r, B, gather_tiles_at(smem, REP_THREADS, REP_THREADS), true, list_in,
                 [&](uint32_t pos, const uint4 rec, int32_t row) {
                   g_item[pos] = ((uint64_t)rec.y << 32) | rec.x; g_zw[pos] = make_uint2(rec.z, rec.w); g_row[pos] = row;
                 },
                 [&](uint32_t pos, int32_t row) { a.order[b + n_act + pos] = row; });
  __syncthreads();

  // ---- aggregates, plan ---------------------------------------------------------------------------------
  {
    int64_t n_run = 0, sum_kv = 0;
    uint64_t m_run = 0, m_q = 0;
#pragma unroll 4
    for (int q = tid; q < n_act; q += REP_THREADS) {
      const uint2 zw = g_zw[q];
      const uint32_t cls = zw.y >> CREC_CLS_SHIFT;
      if (((zw.x >> CREC_KIND_SHIFT) & 1u) == KIND_RUNNING) { n_run++; sum_kv += (int64_t)(zw.x & CREC_LEN_MASK) + (zw.y & CREC_LEN_MASK); m_run |= 1ull << cls; }
      else m_q |= 1ull << cls;
    }
    for (int i = tid; i < MED_BINS / 2; i += REP_THREADS) s_bin[i] = 0;
    for (int i = tid; i < TINY_CLASSES; i += REP_THREADS) { s_cmin[i] = 0xffffffffu; s_cmax[i] = 0; s_lmin[i] = 0xffu; s_lmax[i] = 0; s_ccnt[i] = 0; }
    n_run = warp_sum_i64(n_run); sum_kv = warp_sum_i64(sum_kv);
    m_run = warp_or_u64(m_run); m_q = warp_or_u64(m_q);
    if (lane == 0) { sh.red_a[warp] = n_run; sh.red_b[warp] = sum_kv; sh.red_m0[warp] = m_run; sh.red_m1[warp] = m_q; }
    __syncthreads();
    if (warp == 0) {     // the first warp finishes the reduction and plans
      n_run = warp_sum_i64(sh.red_a[lane]); sum_kv = warp_sum_i64(sh.red_b[lane]);
      m_run = warp_or_u64(sh.red_m0[lane]); m_q = warp_or_u64(sh.red_m1[lane]);
      hfx_replica_cfg cfg; cfg.mode = HFX_COLOCATED; cfg.token_cap = 1; cfg.batch_cap = 0;
      int64_t now = 0, mat = 0;
      if (real) { cfg = a.cfg[r]; now = a.now[r]; mat = a.mat[r]; }
      ReplicaPlan pl0;
      warp_plan(p, s_cls_ttft, s_cls_tpot, cfg, now, mat, n_run, sum_kv, m_run, m_q, pl0, lane);
      if (lane == 0) { sh.plan = pl0; sh.next_arrival = HFX_INF; }
    }
    __syncthreads();
  }
  const ReplicaPlan pl = sh.plan;

  // ---- sort items (into the scratch, over the bases); per class their range ------------------------
  {
    const int n_rounds = (n_act + REP_THREADS - 1) / REP_THREADS;
    int64_t base_n = 0; uint2 zw_n = make_uint2(0u, 0u); int32_t row_n = 0;      // the next round's row, asked for a round ahead
    if (tid < n_act) { base_n = (int64_t)g_item[tid]; zw_n = g_zw[tid]; row_n = g_row[tid]; }
    for (int q0 = 0; q0 < n_act; q0 += REP_THREADS) {
      if (q0 + (tid & ~31) >= n_act) break;      // (whole warps leave)
      const int q = q0 + tid;
      const bool in = q < n_act;
      const int64_t base = base_n; const uint2 zw = zw_n; const int32_t row = row_n;
      if (q + REP_THREADS < n_act) { base_n = (int64_t)g_item[q + REP_THREADS]; zw_n = g_zw[q + REP_THREADS]; row_n = g_row[q + REP_THREADS]; }
      uint64_t item = ~0ull;
      if (in) {
        const int kind = (zw.x >> CREC_KIND_SHIFT) & 1, prio = zw.x >> CREC_PRIO_SHIFT;
        const bool given = kind == KIND_QUEUED && pl.mode != HFX_DECODE;      // the front end has put the row's final key in place of the base
        RowEval ev;
        if (given) { ev.k48 = (uint64_t)base; ev.slack = 0; ev.pred_tpot = a.pred_tpot ? pl.tpot_q0 + p.d2 * ((int64_t)(zw.x & CREC_LEN_MASK) + (zw.y & CREC_LEN_MASK)) : 0; }
        else ev = eval_row(p, pl, base, kind, prio, (int32_t)(zw.x & CREC_LEN_MASK), (int32_t)(zw.y & CREC_LEN_MASK));
        item = (ev.k48 << 16) | (uint32_t)q;     // rows were gathered in req_id order: position breaks ties
        g_item[q] = item;
        if (!given) {    // (the front end wrote the slack of the other queued rows)
          a.slack[row] = ev.slack;
          if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | ev.k48;
        }
        if (a.pred_tpot) a.pred_tpot[row] = ev.pred_tpot;
      }
      // Ranges of the slacks per class, from a sample: in every round one warp in n_rounds looks (a different one each
      // round, so the sample is spread over the replica's rows).  The warp's rows of one class update the class's range
      // together.  The smallest upper part joined to the smallest low part is a lower bound of the sampled slacks of
      // the class, likewise an upper bound; both are exact when they are all equal (requests without a bound).
      if ((warp + (q0 >> 10)) % n_rounds == 0) {
        const uint32_t cl = in ? (uint32_t)(item >> 56) : 0xffu, up = (uint32_t)(item >> 24), low = (uint32_t)(item >> 16) & 0xffu;
        const uint32_t same = __match_any_sync(0xffffffffu, cl);
        const uint32_t mn = __reduce_min_sync(same, up), mx = __reduce_max_sync(same, up);
        const uint32_t mn_low = __reduce_min_sync(same, low), mx_low = __reduce_max_sync(same, low);
        if (in && lane == __ffs(same) - 1) {
          atomicMin(&s_cmin[cl], mn); atomicMax(&s_cmax[cl], mx); atomicMin(&s_lmin[cl], mn_low); atomicMax(&s_lmax[cl], mx_low);
          atomicAdd(&s_ccnt[cl], (uint32_t)__popc(same));
        }
      }
    }
  }
  __syncthreads();

  // ---- sort: bins by class and sub-key, places inside a bin by counting ------------------------------
  // An item's place in its class's order is (slack - smallest slack of the class) << 16 | position, at most
  // (range of slacks) << 16 | (n_act - 1); the class's bins divide that evenly, so equal slacks spread by position.
  // Every class has a bin, sampled or not; what falls outside the sampled range goes to the class's first or last
  // bin, which keeps the bins in item order.
  if (warp == 0) {
    uint32_t cnt[TINY_CLASSES / 32], seen = 0;
#pragma unroll
    for (int e = 0; e < TINY_CLASSES / 32; e++) { cnt[e] = s_ccnt[lane * (TINY_CLASSES / 32) + e]; seen += cnt[e]; }
    seen = __reduce_add_sync(0xffffffffu, seen);
    uint32_t lg[TINY_CLASSES / 32], sum = 0;
#pragma unroll
    for (int e = 0; e < TINY_CLASSES / 32; e++) {
      const uint32_t want = seen ? cnt[e] * (uint32_t)(MED_BINS - TINY_CLASSES) / seen : 0u;      // the shares add up to at most MED_BINS - TINY_CLASSES, plus one bin per class
      lg[e] = want > 1 ? 31 - __clz(want) : 0;
      sum += 1u << lg[e];
    }
    uint32_t v = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
    uint32_t run = v - sum;
#pragma unroll
    for (int e = 0; e < TINY_CLASSES / 32; e++) {
      const int cl = lane * (TINY_CLASSES / 32) + e;
      unsigned long long lo = 0, range = 0;
      if (cnt[e]) {
        lo = ((unsigned long long)s_cmin[cl] << 8) | s_lmin[cl];
        range = (((((unsigned long long)s_cmax[cl] << 8) | s_lmax[cl]) - lo) << 16) | (unsigned long long)(n_act - 1);
      }
      const int bits = 64 - __clzll((long long)range);
      const unsigned long long sft = bits > (int)lg[e] ? (unsigned long long)(bits - (int)lg[e]) : 0ull;       // (range >> sft) < number of bins
      s_cinfo[cl] = lo | ((unsigned long long)run << 40) | (sft << 53) | ((unsigned long long)lg[e] << 59);
      run += 1u << lg[e];
    }
  }
  __syncthreads();
  auto bin_of = [&](uint64_t x) -> uint32_t {
    const uint64_t ci = s_cinfo[(uint32_t)(x >> 56)];
    const uint64_t v = x & ((1ull << 56) - 1), lo = (ci & ((1ull << 40) - 1)) << 16;
    const uint32_t last = (1u << ((uint32_t)(ci >> 59) & 15u)) - 1u;
    const uint64_t d = v > lo ? (v - lo) >> ((uint32_t)(ci >> 53) & 63u) : 0ull;
    return ((uint32_t)(ci >> 40) & 0x1fffu) + (d < last ? (uint32_t)d : last);
  };
#pragma unroll 4
  for (int q = tid; q < n_act; q += REP_THREADS) {
    const uint32_t bi = bin_of(g_item[q]);
    atomicAdd(&s_bin[bi >> 1], 1u << ((bi & 1u) * 16));
  }
  __syncthreads();
  bool binned = false;
  {   // exclusive scan of the bin counts, eight per thread; the fullest bin
    const uint4 wd = reinterpret_cast<const uint4 *>(s_bin)[tid];
    const uint32_t ww[4] = {wd.x, wd.y, wd.z, wd.w};
    uint32_t cnt[8], sum = 0, big = 0;
#pragma unroll
    for (int i = 0; i < 4; i++) { cnt[2 * i] = ww[i] & 0xffffu; cnt[2 * i + 1] = ww[i] >> 16; }
#pragma unroll
    for (int i = 0; i < 8; i++) { sum += cnt[i]; big = cnt[i] > big ? cnt[i] : big; }
    uint32_t v = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
    big = __reduce_max_sync(0xffffffffu, big);
    if (lane == 31) sh.red_n[warp] = (int32_t)v;
    if (lane == 0) sh.red_a[warp] = (int64_t)big;
    __syncthreads();
    uint32_t run = v - sum, bigall = 0;
    for (int k = 0; k < REP_THREADS / 32; k++) { if (k < warp) run += (uint32_t)sh.red_n[k]; const uint32_t x = (uint32_t)sh.red_a[k]; bigall = x > bigall ? x : bigall; }
    if (bigall <= MED_BIN_MAX) {
      uint32_t st[8];
#pragma unroll
      for (int i = 0; i < 8; i++) { st[i] = run; run += cnt[i]; }
      const uint4 o4 = make_uint4(st[0] | (st[1] << 16), st[2] | (st[3] << 16), st[4] | (st[5] << 16), st[6] | (st[7] << 16));
      reinterpret_cast<uint4 *>(s_bin)[tid] = o4;
      reinterpret_cast<uint4 *>(s_cur)[tid] = o4;
      binned = true;
    }
  }
  __syncthreads();
  if (binned) {
#pragma unroll 4
    for (int q = tid; q < n_act; q += REP_THREADS) {
      const uint64_t x = g_item[q];
      const uint32_t bi = bin_of(x), sh16 = (bi & 1u) * 16;
      const uint32_t pos = (atomicAdd(&s_cur[bi >> 1], 1u << sh16) >> sh16) & 0xffffu;
      s_item[pos] = x;
    }
    __syncthreads();
    for (int e = tid; e < n_act; e += REP_THREADS) {
      const uint64_t x = s_item[e];
      const uint32_t bi = bin_of(x), sh16 = (bi & 1u) * 16;
      const uint32_t g0 = (s_bin[bi >> 1] >> sh16) & 0xffffu, g1 = (s_cur[bi >> 1] >> sh16) & 0xffffu;
      uint32_t rank = 0;
      for (uint32_t k = g0; k < g1; k++) rank += s_item[k] < x ? 1u : 0u;
      s_ord[g0 + rank] = (uint16_t)(x & 0xffffu);      // (the class ranges that s_ord overlays were last read when the bins were laid out)
    }
  } else {      // a bin is too full: the sorting network
    for (int q = tid; q < n_act; q += REP_THREADS) s_item[q] = g_item[q];
    __syncthreads();
    sort64_positions(s_item, s_lo, n_act);
    __syncthreads();
    for (int q0 = 0; q0 < n_act; q0 += REP_THREADS) {      // 32-bit positions -> 16-bit, in place: a chunk's writes land on words already read
      const int q = q0 + tid;
      const uint32_t v = q < n_act ? s_lo[q] : 0u;
      __syncthreads();
      if (q < n_act) s_ord[q] = (uint16_t)v;
    }
  }
  __syncthreads();

  // ---- the order; the record words by position, over the items -----------------------------------------
#pragma unroll 4
  for (int q = tid; q < n_act; q += REP_THREADS) {
    a.order[b + q] = g_row[s_ord[q]];
    const uint2 zw = g_zw[q];
    s_zw[q] = make_uint2(zw.x & ((1u << CREC_PRIO_SHIFT) - 1u), zw.y);      // (the priority has served; its bits make room for the marks)
  }
  __syncthreads();

  auto cost_at = [&](uint32_t li, int64_t &kv) -> int64_t {      // cost of the queued row at position li, -1 if it is in flight
    const uint2 zw = s_zw[li];
    if (((zw.x >> CREC_KIND_SHIFT) & 1u) != KIND_QUEUED) return -1;
    kv = (int64_t)(zw.x & CREC_LEN_MASK) + (zw.y & CREC_LEN_MASK);
    return pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(zw.x & CREC_LEN_MASK);
  };
  if (FF) {     // first fit: the first warp walks the order and marks what it takes
    if (warp == 0) {
      const int64_t room = pl.batch_cap == 0 ? HFX_INF : (pl.batch_cap > pl.n_eff ? pl.batch_cap - pl.n_eff : 0);
      warp_first_fit(n_act, pl.budget, room, lane, [&](int64_t q) -> int64_t { int64_t kv; return cost_at(s_ord[q], kv); },
                     [&](int64_t q, bool taken) { if (taken) s_zw[s_ord[q]].x |= 0x80000000u; });
    }
    __syncthreads();
  }

  // ---- admission: every thread walks consecutive places of the order, twice -------------------------------
  const int ipt = (n_act + REP_THREADS - 1) / REP_THREADS;
  const int qa = tid * ipt < n_act ? tid * ipt : n_act, qb = qa + ipt < n_act ? qa + ipt : n_act;
  int64_t my_cost = 0;
  int32_t my_cnt = 0;
  for (int q = qa; q < qb; q++) {      // what counts towards the running totals: rows that fit alone, or (first fit) exactly the rows taken
    const uint32_t li = s_ord[q];
    int64_t kv = 0;
    const int64_t cc = cost_at(li, kv);
    if (cc >= 0 && (FF ? (s_zw[li].x >> 31) != 0 : cc <= pl.budget)) { my_cost += cc; my_cnt++; }
  }
  int64_t run_c = warp_incl_scan_i64(my_cost, lane);
  int32_t run_n = warp_incl_scan_i32(my_cnt, lane);
  if (lane == 31) { sh.red_a[warp] = run_c; sh.red_n[warp] = run_n; }
  __syncthreads();
  run_c -= my_cost; run_n -= my_cnt;
  for (int k = 0; k < warp; k++) { run_c += sh.red_a[k]; run_n += sh.red_n[k]; }
  int64_t ac = 0, ak = 0;
  int32_t an = 0;
  if (my_cnt)
    for (int q = qa; q < qb; q++) {
      const uint32_t li = s_ord[q];
      int64_t kv = 0;
      const int64_t cc = cost_at(li, kv);
      if (cc >= 0 && (FF ? (s_zw[li].x >> 31) != 0 : cc <= pl.budget)) {
        run_c += cc; run_n += 1;
        if (FF || (run_c <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + run_n <= pl.batch_cap))) {
          ac += cc; ak += kv; an++;
          const int32_t row = g_row[li];
          a.admit[row] = 1;
          if (a.admitted_rows) a.admitted_rows[b + run_n - 1] = row;
          s_zw[li].y |= 0x80000000u;
        }
      }
    }
  __syncthreads();      // (the scan's partial sums have been read)

  // ---- totals, maturity, iteration clock ---------------------------------------------------------
  ac = warp_sum_i64(ac); ak = warp_sum_i64(ak); an = (int32_t)__reduce_add_sync(0xffffffffu, (uint32_t)an);
  if (lane == 0) { sh.red_a[warp] = ac; sh.red_b[warp] = ak; sh.red_n[warp] = an; }
  __syncthreads();
  if (tid == 0) {
    int64_t adm_cost = 0, adm_kv = 0; int32_t adm_count = 0;
    for (int k = 0; k < REP_THREADS / 32; k++) { adm_cost += sh.red_a[k]; adm_kv += sh.red_b[k]; adm_count += sh.red_n[k]; }
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
  if (commit && !worked)      // idle replica: its next arrival is looked up among its listed inactive rows
    group_min_arrival(list_in ? next_arrival_listed(a, c, b, n_act, n, tid, REP_THREADS) : next_arrival_slabs(a, c, R + 1, r, B), sh, B);
  if (tid == 0 && real)
    write_replica_outputs(a, r, pl, sh.adm_cost, sh.adm_count, mat_next, worked, sh.t2, sh.next_arrival);

  // ---- padding of the compacted list, commit ----------------------------------------------------
  if (a.admitted_rows)
    for (int q = sh.adm_count + tid; q < n; q += REP_THREADS) a.admitted_rows[b + q] = -1;
  if (commit) {
    const int64_t t1 = sh.t1, t2 = sh.t2;
#pragma unroll 2
    for (int q = tid; q < n_act; q += REP_THREADS) {
      const uint2 zw = s_zw[q];
      const int kind = (zw.x >> CREC_KIND_SHIFT) & 1;
      const bool adm = (zw.y >> 31) != 0;
      const int32_t row = g_row[q];
      const int32_t out_len = commit_needs_out_len(pl, kind, adm, worked) ? __ldg(a.output_len + row) : 0;
      commit_row(a, pl, kind, adm, worked, t1, t2, row, (int32_t)(zw.x & CREC_LEN_MASK), (int32_t)(zw.y & CREC_LEN_MASK), out_len);
    }
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// Oversize replicas (more items than a block sorts in shared memory): the block runs the sorting
// network in global memory (items in c.big_hi / big_lo, the record positions travelling in big_idx),
// then admission with a carried prefix.  Slow but exact.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void global_cmp_swap(uint64_t *hi, uint32_t *lo, uint32_t *idx, int64_t i, int64_t j) {
  const uint64_t hi_i = hi[i], hi_j = hi[j];
  const uint32_t lo_i = lo[i], lo_j = lo[j];
  if (hi_i > hi_j || (hi_i == hi_j && lo_i > lo_j)) {
    hi[i] = hi_j; hi[j] = hi_i; lo[i] = lo_j; lo[j] = lo_i;
    const uint32_t x = idx[i]; idx[i] = idx[j]; idx[j] = x;
  }
}

// Bitonic network over n items (hi, lo) in global memory with idx travelling along: ascending comparators,
// virtual padding.  Block-synchronised on entry by the caller and on return.
__device__ void block_global_sort(uint64_t *hi, uint32_t *lo, uint32_t *idx, int64_t n) {
  int64_t n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  const int64_t half = n_pad >> 1;
  for (int64_t k = 2; k <= n_pad; k <<= 1) {
    const int64_t hk = k >> 1;
    for (int64_t t = threadIdx.x; t < half; t += blockDim.x) {
      const int64_t blk = t / hk, off = t - blk * hk;
      const int64_t i = blk * k + off, j = blk * k + k - 1 - off;
      if (j < n) global_cmp_swap(hi, lo, idx, i, j);
    }
    __syncthreads();
    for (int64_t j = k >> 2; j > 0; j >>= 1) {
      for (int64_t t = threadIdx.x; t < half; t += blockDim.x) {
        const int64_t i = 2 * t - (t & (j - 1));
        if (i + j < n) global_cmp_swap(hi, lo, idx, i, i + j);
      }
      __syncthreads();
    }
  }
}

template <bool SLABS, bool FF>
__device__ void oversize_replica(const HfxParams &p, const SegArgs &a, const SegCtx &c, int r, uint32_t b, int64_t n, int64_t n_act,
                                 bool ordered, bool list_in, unsigned char *smem, BlockShared &sh) {
  const int R = p.n_replicas;
  const Grp B = {(int)threadIdx.x, (int)blockDim.x, 0};
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int64_t n_in = n - n_act;
  const HfxRec *seg = c.rec + b;
  const bool real = r < R;
  if (SLABS) gather_to_records(a, c, R + 1, r, b, n_act, ordered, list_in, smem);

  // ---- inactive rows of a step that is not ordered: by req_id behind the active ones -----------
  if (!ordered && n_in > 0) {
    const HfxRec *sin = seg + n_act;
    uint64_t *hi = c.big_hi + b + n_act;
    uint32_t *lo = c.big_lo + b + n_act, *idx = c.big_idx + b + n_act;
    for (int64_t q = threadIdx.x; q < n_in; q += blockDim.x) { hi[q] = ld_rec(sin + q, 0).z ^ 0x80000000u; lo[q] = 0; idx[q] = (uint32_t)q; }
    __syncthreads();
    block_global_sort(hi, lo, idx, n_in);
    for (int64_t q = threadIdx.x; q < n_in; q += blockDim.x) a.order[b + n_act + q] = (int32_t)ld_rec(sin + idx[q], 0).w;
    __syncthreads();
  }

  segment_plan(p, a, seg, n_act, r, real, sh);
  const ReplicaPlan pl = sh.plan;
  uint64_t *hi = c.big_hi + b;
  uint32_t *lo = c.big_lo + b, *idx = c.big_idx + b;

  for (int64_t q = threadIdx.x; q < n_act; q += blockDim.x) {
    const uint4 w0 = ld_rec(seg + q, 0);
    const uint4 w1 = ld_rec(seg + q, 1);
    const int64_t base = (int64_t)(((uint64_t)w0.y << 32) | w0.x);
    const int32_t row = (int32_t)w0.w;
    const int kind = (w1.w >> 8) & 0xff, prio = (w1.w >> 16) & 0xff;
    RowEval e = eval_row(p, pl, base, kind, prio, (int32_t)w1.x, (int32_t)w1.y);
    if (kind == KIND_QUEUED && pl.mode != HFX_DECODE) e.k48 = (uint64_t)base;      // the front end has put the row's final key in place of the base
    hi[q] = e.k48;
    lo[q] = ordered ? (uint32_t)q : (w0.z ^ 0x80000000u);     // ties: position (rows in req_id order) or the request id
    idx[q] = (uint32_t)q;
    if (kind == KIND_RUNNING || pl.mode == HFX_DECODE) {
      a.slack[row] = e.slack;
      if (a.key) a.key[row] = ((uint64_t)(r & 0xffff) << 48) | e.k48;
    }
    if (a.pred_tpot) a.pred_tpot[row] = e.pred_tpot;
  }
  __syncthreads();
  block_global_sort(hi, lo, idx, n_act);

  // admission walk with a carried prefix
  if (FF) {     // the first warp walks the order; lo (free now that the sort is over) says what it took
    if (warp == 0) {
      const int64_t room = pl.batch_cap == 0 ? HFX_INF : (pl.batch_cap > pl.n_eff ? pl.batch_cap - pl.n_eff : 0);
      warp_first_fit(n_act, pl.budget, room, lane,
                     [&](int64_t q) -> int64_t {
                       const uint4 w1 = ld_rec(seg + idx[q], 1);
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
      const uint4 w0 = ld_rec(seg + li, 0);
      const uint4 w1 = ld_rec(seg + li, 1);
      row = (int32_t)w0.w;
      kind = (w1.w >> 8) & 0xff;
      if (kind == KIND_QUEUED) {
        kv = (int64_t)(int32_t)w1.x + (int32_t)w1.y;
        const int64_t cc = pl.mode == HFX_DECODE ? p.d1 + p.d2 * kv : (int64_t)(int32_t)w1.x;
        if (FF ? lo[q] == 2u : cc <= pl.budget) { cost = cc; cnt = 1; } else kv = 0;
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
    if (cnt) adm = FF || (sc <= pl.budget && (pl.batch_cap == 0 || pl.n_eff + sn <= pl.batch_cap));
    if (q < n_act) {
      if (adm) a.admit[row] = 1;
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
    int worked; int64_t t1, t2;
    iteration_clock(pl, sh.adm_count, lp, mat_next, worked, t1, t2);
    sh.worked = worked; sh.t1 = t1; sh.t2 = t2; sh.red_c[0] = mat_next;
  }
  __syncthreads();
  const bool commit = real && (a.flags & HFX_COMMIT) && pl.now <= a.horizon;
  const int worked = sh.worked;
  const int64_t mat_next = sh.red_c[0];
  if (commit && !worked)
    group_min_arrival(list_in || !ordered ? next_arrival_listed(a, c, b, n_act, n, threadIdx.x, blockDim.x) : next_arrival_slabs(a, c, p.n_replicas + 1, r, B), sh, B);
  if (threadIdx.x == 0 && real)
    write_replica_outputs(a, r, pl, sh.adm_cost, sh.adm_count, mat_next, worked, sh.t2, sh.next_arrival);
  if (a.admitted_rows)
    for (int64_t q = sh.adm_count + threadIdx.x; q < n; q += blockDim.x) a.admitted_rows[b + q] = -1;
  if (commit) {
    const int64_t t1 = sh.t1, t2 = sh.t2;
    for (int64_t q = threadIdx.x; q < n_act; q += blockDim.x) {
      const uint32_t li = idx[q];
      const uint4 w0 = ld_rec(seg + li, 0);
      const uint4 w1 = ld_rec(seg + li, 1);
      const int kind = (w1.w >> 8) & 0xff;
      const bool adm = lo[q] != 0;
      const int32_t out_len = commit_needs_out_len(pl, kind, adm, worked) ? __ldg(a.output_len + (int32_t)w0.w) : 0;
      commit_row(a, pl, kind, adm, worked, t1, t2, (int32_t)w0.w, (int32_t)w1.x, (int32_t)w1.y, out_len);
    }
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <bool SLABS, bool FF>
__global__ void __launch_bounds__(REP_THREADS, 1) k_replicas(const HfxParams p, const SegArgs a, const SegCtx c) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ BlockShared sh_g[REP_GROUPS];
  __shared__ int64_t s_cls_ttft[HFX_MAX_CLASSES], s_cls_tpot[HFX_MAX_CLASSES];     // class tables for the planning warps
  __shared__ uint32_t s_scan[2 * 32 + 2];      // (also the scratch of the block-wide scans below)
  __shared__ uint64_t s_cinfo_med[TINY_CLASSES];  // bin layout of a medium replica's distribution sort: smallest slack<40> | first bin<13> | shift<6> | log2 bins<4>
  __shared__ uint32_t s_long[(HFX_TILE_REPLICAS_MAX + 1 + 31) / 32 + 1];           // replicas whose inactive rows the grid lists together
  uint32_t *s_begin = reinterpret_cast<uint32_t *>(smem_raw + SMEM_MED);           // [R+2] range starts (slabs only)
  const int R = p.n_replicas, R1 = R + 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int k = tid; k < HFX_MAX_CLASSES; k += blockDim.x) {
    s_cls_ttft[k] = k < p.n_classes ? p.ttft[k] : 0;
    s_cls_tpot[k] = k < p.n_classes ? p.tpot[k] : 0;
  }
  for (int k = tid; k < (int)(sizeof(s_long) / sizeof(uint32_t)); k += blockDim.x) s_long[k] = 0;

  // everything below reads what the front end wrote
  cudaGridDependencySynchronize();

  const bool ordered = SLABS ? __ldcg(c.ordered) != 0 : false;
  const uint32_t *begin = c.seg_begin;
  int larger = 1, longer = 0;       // does any replica need the whole block?  does any list of inactive rows need the grid?
  __syncthreads();
  if (SLABS) {
    // range starts: exclusive prefix of the rows per replica, every block its own copy
    const int per = (R1 + blockDim.x - 1) / blockDim.x;
    const int i0 = tid * per < R1 ? tid * per : R1, i1 = (i0 + per < R1) ? i0 + per : R1;
    uint32_t sum = 0;
    larger = 0;
    for (int i = i0; i < i1; i++) {
      const unsigned long long t = __ldcg(c.tot + i);
      const uint32_t n_all = (uint32_t)t, n_act = (uint32_t)(t >> 32), n_in = n_all - n_act;
      sum += n_all;
      if ((ordered ? n_act : (n_act > n_in ? n_act : n_in)) > SEG_TINY) larger = 1;
      if (ordered && n_in > LIST_MAX) { atomicOr(&s_long[i >> 5], 1u << (i & 31)); longer = 1; }
    }
    uint32_t v = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
    if (lane == 31) s_scan[warp] = v;
    larger = __syncthreads_or(larger);
    longer = __syncthreads_or(longer);
    if (warp == 0) {      // the warps' totals, scanned by the first warp
      uint32_t w = s_scan[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += x; }
      s_scan[32 + lane] = w;
    }
    __syncthreads();
    uint32_t run = v - sum + (warp ? s_scan[32 + warp - 1] : 0u);
    for (int i = i0; i < i1; i++) {
      s_begin[i] = run;
      if (blockIdx.x == 0) a.seg_off[i] = (int32_t)run;
      run += (uint32_t)__ldcg(c.tot + i);
    }
    if (tid == 0) s_begin[R1] = s_scan[63];
    begin = s_begin;
    __syncthreads();
  }
  auto counts = [&](int r, uint32_t &n_all, uint32_t &n_act) {
    if (SLABS) { const unsigned long long t = __ldcg(c.tot + r); n_all = (uint32_t)t; n_act = (uint32_t)(t >> 32); }
    else { n_all = c.seg_count[r]; n_act = c.act_count[r]; }
  };
  auto need_of = [&](uint32_t n_all, uint32_t n_act) -> uint32_t {
    const uint32_t n_in = n_all - n_act;
    return ordered ? n_act : (n_act > n_in ? n_act : n_in);
  };

  // ---- small replicas: eight groups of 128 threads, each on a barrier of its own ---------------------
  {
    const int g = tid / GROUP_THREADS;
    const Grp G = {tid - g * GROUP_THREADS, GROUP_THREADS, g + 1};
    for (int r = g * gridDim.x + blockIdx.x; r <= R; r += gridDim.x * REP_GROUPS) {      // consecutive replicas on different SMs: few replicas still use them all
      uint32_t n_all, n_act;
      counts(r, n_all, n_act);
      if (need_of(n_all, n_act) > SEG_TINY) continue;
      if (r == R && n_all == 0) continue;
      const bool list_in = !ordered || n_all - n_act <= LIST_MAX;
      small_replica<SLABS, FF>(p, a, c, G, r, begin[r], (int)n_all, (int)n_act, ordered, list_in, smem_raw + (size_t)g * SMEM_GROUP, sh_g[g],
                    s_cls_ttft, s_cls_tpot);
    }
  }
  __syncthreads();

  // ---- larger replicas: the whole block -------------------------------------------------------------
  if (larger)
  for (int r = blockIdx.x; r <= R; r += gridDim.x) {
    uint32_t n_all, n_act;
    counts(r, n_all, n_act);
    const uint32_t need = need_of(n_all, n_act);
    if (need <= SEG_TINY) continue;
    const bool list_in = !ordered || n_all - n_act <= LIST_MAX;
    if (SLABS && ordered && need <= SEG_MED) medium_ordered<FF>(p, a, c, r, begin[r], (int)n_all, (int)n_act, list_in, smem_raw, sh_g[0], s_cinfo_med, s_cls_ttft, s_cls_tpot);
    else if (need <= SEG_MED) medium_replica<SLABS, FF>(p, a, c, r, begin[r], (int)n_all, (int)n_act, ordered, list_in, smem_raw, sh_g[0]);
    else oversize_replica<SLABS, FF>(p, a, c, r, begin[r], n_all, n_act, ordered, list_in, smem_raw, sh_g[0]);
  }

  // ---- long lists of inactive rows (ordered steps): every block lists a range of tiles ----------------
  // The replicas with a long list are collected in shared memory; a thread per replica adds up the replica's
  // inactive rows in the tiles before the block's, then a warp per replica copies the rows of the block's tiles.
  if (longer) {
    __syncthreads();      // the larger replicas are done with the block's shared memory
    uint16_t *s_lr = reinterpret_cast<uint16_t *>(smem_raw);                                   // [R1] the replicas
    uint32_t *s_lpre = reinterpret_cast<uint32_t *>(smem_raw + (((size_t)R1 * 2 + 15) & ~(size_t)15));   // [R1] rows in earlier tiles
    if (tid == 0) s_scan[0] = 0;
    __syncthreads();
    for (int r = tid; r < R1; r += blockDim.x)
      if ((s_long[r >> 5] >> (r & 31)) & 1u) s_lr[atomicAdd(&s_scan[0], 1u)] = (uint16_t)r;
    __syncthreads();
    const int n_long = (int)s_scan[0];
    const int per = (c.n_tiles + gridDim.x - 1) / gridDim.x;
    const int tA = blockIdx.x * per < c.n_tiles ? blockIdx.x * per : c.n_tiles;
    const int tB = tA + per < c.n_tiles ? tA + per : c.n_tiles;
    if (tA < tB) {
      for (int j = tid; j < n_long; j += blockDim.x) {
        const int r = s_lr[j];
        uint32_t pre = 0;
#pragma unroll 8
        for (int t = 0; t < tA; t++) { const uint2 m = __ldcg(c.M + (size_t)t * R1 + r); pre += (m.x >> 16) - (m.y >> 16); }
        s_lpre[j] = pre;
      }
      __syncthreads();
      // many long lists: a warp per replica; few (one bucket of unbound rows, say): the whole block on each
      const bool by_warp = n_long >= (int)(blockDim.x >> 5);
      const int first = by_warp ? warp : 0, step = by_warp ? (int)(blockDim.x >> 5) : 1;
      const uint32_t k0 = by_warp ? (uint32_t)lane : (uint32_t)tid, kstep = by_warp ? 32u : blockDim.x;
      for (int j = first; j < n_long; j += step) {
        const int r = s_lr[j];
        uint32_t dst = begin[r] + (uint32_t)(__ldcg(c.tot + r) >> 32) + s_lpre[j];
        for (int t = tA; t < tB; t++) {
          const uint2 m = __ldcg(c.M + (size_t)t * R1 + r);
          const uint32_t ca = m.y >> 16, ci = (m.x >> 16) - ca, src = (m.x & 0xffffu) + ca;
          const size_t tb = (size_t)t * c.tile_rows;
#pragma unroll 4
          for (uint32_t k = k0; k < ci; k += kstep) a.order[dst + k] = (int32_t)(tb + __ldcg(c.slab_idx + tb + src + k));
          dst += ci;
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
int hfx_launch_replicas(hfx_sched *s, const SegArgs &sa, int64_t n, bool slabs) {
  const int R1 = s->p.n_replicas + 1;
  SegCtx c;
  memset(&c, 0, sizeof(c));
  c.slabs = slabs ? 1 : 0;
  c.rec = s->d_rec; c.rowflag = s->d_rowflag;
  c.big_hi = s->d_big_hi; c.big_lo = s->d_big_lo; c.big_idx = s->d_big_lo ? s->d_big_lo + s->max_rows : nullptr;
  if (slabs) {
    const uint32_t par = s->tot_parity;
    c.slab_rec = s->d_slab_rec; c.slab_idx = s->d_slab_idx; c.M = s->d_M;
    c.tot = s->d_tot + (size_t)par * (R1 + 1);
    c.ordered = s->d_flags + 4 + par;
    hfx_front_shape(s, n, &c.tile_rows, &c.n_tiles);
  } else {
    c.seg_count = s->d_seg_count; c.act_count = s->d_act_count; c.seg_begin = s->d_seg_begin;
    c.ordered = s->d_flags;
  }
  // one block per SM; the fallback layout has nothing that every block shares, so it needs no more blocks than replicas
  const int grid = slabs ? s->n_sm : (R1 < s->n_sm ? R1 : s->n_sm);
  const size_t smem = SMEM_MED + (slabs ? sizeof(uint32_t) * ((size_t)R1 + 2) : 0);
  KernelScope ks(s, KSLOT_SEG_SMALL);
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(REP_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = s->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (slabs && !s->profiling) ? 1 : 0;      // the kernel may be set up while the tile front end drains
  cudaError_t e;
  if (slabs) e = s->p.first_fit ? cudaLaunchKernelEx(&cfg, k_replicas<true, true>, s->p, sa, c) : cudaLaunchKernelEx(&cfg, k_replicas<true, false>, s->p, sa, c);
  else e = s->p.first_fit ? cudaLaunchKernelEx(&cfg, k_replicas<false, true>, s->p, sa, c) : cudaLaunchKernelEx(&cfg, k_replicas<false, false>, s->p, sa, c);
  return e == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}

int hfx_segment_configure() {
  const int smem = (int)(SMEM_MED + sizeof(uint32_t) * (HFX_TILE_REPLICAS_MAX + 3));
  if (cudaFuncSetAttribute(k_replicas<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(k_replicas<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(k_replicas<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(k_replicas<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}
