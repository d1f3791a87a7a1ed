// Internal declarations shared by the kernels of the scheduler library.
// Integer nanoseconds everywhere; nothing here is floating point.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "hfx.h"

#define HFX_MAX_CLASSES 64
#define HFX_MAX_REPLICAS 65536
#define HFX_MAX_ROWS (INT64_C(1) << 27)

// phases of the key (2 bits)
#define PH_RUNNING 0
#define PH_QUEUED 1
#define PH_INACTIVE 3

// kinds of a regrouped record
#define KIND_RUNNING 0  // in flight
#define KIND_QUEUED 1   // arrived and waiting
#define KIND_FUTURE 2   // QUEUED but not arrived yet (only matters for the idle clock jump)
#define KIND_DEAD 3     // DONE, REJECTED or a row with bad data

#define ROWFLAG_BADREP 4  // row bound to no replica (bucket R)

// how a tile's rows get their rank inside their (replica, class) group, in row order
#define TILE_SORTED 0     // tile already sorted by replica: ranks from positions
#define TILE_GROUPS 1     // small groups: counting sort of the tile, rank by scanning the group
#define TILE_ANY 2        // large unsorted groups: any order (clears "ordered")

// "no bound" marker of a slack base
#define BASE_UNBOUNDED INT64_MAX

// Scheduler constants, passed by value to every kernel (lives in the constant bank).
struct HfxParams {
  int64_t c0, c1, c2, d0, d1, d2;
  int64_t ttft[HFX_MAX_CLASSES];
  int64_t tpot[HFX_MAX_CLASSES];
  uint8_t prio[HFX_MAX_CLASSES];
  int32_t n_classes;
  int32_t n_replicas;
  int32_t budget_mode;
  int32_t weight_max;
  int32_t first_fit;      // admission variant: every request is tried against what is left of the budget
};

// One row after regrouping by replica: everything the per-replica kernel needs, 32 bytes
// (one L2 sector), so that kernel never goes back to the table for reads.
struct __align__(32) HfxRec {
  int64_t base;      // slack before the per-replica shift (see ReplicaPlan); the final 48-bit key for a queued row on a
                     // colocated / prefill replica; arrival for KIND_FUTURE
  int32_t req_id;
  int32_t row;
  int32_t prompt;
  int32_t gen;
  int32_t output_len;
  uint8_t cls, kind, prio, pad;
};
static_assert(sizeof(HfxRec) == 32, "record is one 32-byte sector");

// Compact record of an ACTIVE row as the tile front end leaves it (16 bytes, a uint4):
//   x, y  slack base (int64, as HfxRec::base); for a queued row on a colocated / prefill replica the row's final
//         48-bit key (phase | prio | clamped slack) instead, which needs nothing from the running batch
//   z     prompt_len<25> | kind<1> (KIND_RUNNING / KIND_QUEUED) | prio<6>
//   w     gen<25> | class<6>
// The row index travels beside it (16-bit index inside the tile); req_id and output_len are fetched
// from the table by the few paths that need them.
#define CREC_LEN_MASK 0x1ffffffu
#define CREC_KIND_SHIFT 25
#define CREC_PRIO_SHIFT 26
#define CREC_CLS_SHIFT 25
#define HFX_FRONT_SMEM (220 * 1024)      // dynamic shared memory the tile kernel may use

#include <vector>

enum { KSLOT_COUNT = 0, KSLOT_COLSCAN, KSLOT_OFFSETS, KSLOT_REGROUP, KSLOT_SEG_SMALL, KSLOT_SEG_MED, KSLOT_BIG, KSLOT_SIM, KSLOT_SCALE, KSLOT_FRONT, KSLOT_DISPATCH, KSLOT_SLOMAP, KSLOT_PD, KSLOT_METRICS };

// tiling of the front end: one tile per block, at most 8192 rows (16-bit indices inside a tile)
#define HFX_TILE_ROWS_MAX 8192
#define HFX_TILE_MATRIX_MAX (INT64_C(8) << 20)   // entries of the tile matrix (64 MiB)
#define HFX_TILE_REPLICAS_MAX 4095               // replicas whose counters fit in shared memory (12-bit bucket ids)
#define HFX_COUNT_TILE_ROWS 4096                 // rows per block of the counting pass of the fallback front end

struct HfxBracket { cudaEvent_t a, b; int slot; };

struct hfx_sched {
  HfxParams p;
  hfx_options opts;
  int64_t max_rows;
  int n_sm;
  cudaStream_t stream;
  int64_t launches;
  int profiling;
  std::vector<HfxBracket> *brackets;
  // device
  hfx_replica_cfg *d_cfg;   // [R]
  uint8_t *d_mode;          // [R] replica modes, one byte each
  uint32_t *d_status;       // sticky status word
  uint32_t *d_seg_count;    // [R+2] rows per replica (+ the bad-replica bucket R)      (fallback front end)
  uint32_t *d_act_count;    // [R+2] active rows (in flight or in the visible queue) per replica    (fallback)
  uint32_t *d_seg_begin;    // [R+2] exclusive prefix of d_seg_count                      (fallback)
  uint32_t *d_cursor;       // [2][R+2] fill cursors of the fallback regroup (active, inactive)
  uint8_t *d_rowflag;       // [max_rows] kind of every row (KIND_*), ROWFLAG_BADREP for a bad replica id
  uint32_t *d_flags;        // [0] "ordered" of the fallback front end (never), [4],[5] "ordered" of the tile front end by parity
  HfxRec *d_rec;            // [max_rows] contiguous records: written by the fallback regroup, or gathered from the
                            // slabs by the blocks of larger replicas
  uint64_t *d_big_hi;       // sort scratch of oversize segments
  uint32_t *d_big_lo;
  // tile front end (see hfx_front.cu)
  uint4 *d_slab_rec;        // [tiles_max * tile_rows] records of active rows, tile-major
  uint16_t *d_slab_idx;     // [tiles_max * tile_rows] local row indices, tile-major, grouped by replica
  uint2 *d_M;               // [tiles_max][R+1] where each replica's rows sit in a tile's slabs
  unsigned long long *d_tot;// [2][R+2] rows | active rows << 32 per replica, by parity
  int32_t tiles_max;        // matrix rows allocated (0: fallback front end only)
  uint32_t tot_parity;      // which half of d_tot / which "ordered" word the next tile front end uses
  int64_t horizon;          // commit horizon of the following steps (INT64_MAX: none)
  int front_enabled;        // 0: use the fallback front end (global counters) even where the tile front end fits
  void *dispatch_ws;                   // workspace of hfx_dispatch_step, allocated by its first call
  unsigned char *d_sim_scratch;        // rows of long traces in hfx_sim_run (allocated by the first call that needs it)
  size_t sim_scratch_bytes;
  void *d_slo;                         // per-priority table of hfx_slo_map
  void *d_pd;                          // moved counter, wake-up times and busy flags of hfx_pd_migrate
};

// ---- latency predictor -------------------------------------------------------------------
__device__ __forceinline__ int64_t dev_Ep(const HfxParams &p, int64_t t) { return p.c0 + p.c1 * t + p.c2 * t * t; }
__device__ __forceinline__ int64_t dev_Ed(const HfxParams &p, int64_t b, int64_t kv) { return p.d0 + p.d1 * b + p.d2 * kv; }

__device__ __forceinline__ int64_t dev_clamp_slack(int64_t s) {
  return s < HFX_SLACK_MIN ? HFX_SLACK_MIN : (s > HFX_SLACK_MAX ? HFX_SLACK_MAX : s);
}

// phase<2> | prio<6> | (clamp(slack) + 2^39)<40>  -- the low 48 bits of the key
__device__ __forceinline__ uint64_t dev_key48(int phase, int prio, int64_t slack) {
  return ((uint64_t)phase << 46) | ((uint64_t)prio << 40) | (uint64_t)(dev_clamp_slack(slack) + (INT64_C(1) << 39));
}

// Per-replica quantities of one step, computed once per replica.
struct ReplicaPlan {
  int64_t now, mat, start;
  int64_t n_run, sum_kv, n_eff, kv_eff;
  int64_t tpot_eff;   // strictest TPOT of the running batch (HFX_INF if none)
  int64_t e_d;
  int64_t budget;
  int64_t shift_run;  // slack of a running row = base - shift_run      (now + E_d)
  int64_t shift_q;    // slack of a queued row  = base - shift_q        (earliest start; + predicted TPOT base on DECODE)
  int64_t tpot_q0;    // predicted TPOT of a queued row = tpot_q0 + d2 * (prompt_len + gen)
  int32_t mode, token_cap, batch_cap;
};

// Largest E_p with 2 E_p + k E_d <= TTFT, k = E_p / (TPOT - E_d)  (worst-case TTFT bound
// behind Eq. 3).  HFX_INF without a TTFT bound, -1 when TPOT <= E_d.
__device__ inline int64_t dev_epmax(int64_t min_ttft, bool decoding, int64_t min_tpot, int64_t e_d) {
  if (min_ttft == HFX_INF) return HFX_INF;
  if (!decoding) return min_ttft / 2;
  if (min_tpot <= e_d) return -1;
  const uint64_t x = (uint64_t)min_ttft, y = (uint64_t)(min_tpot - e_d), den = (uint64_t)(2 * min_tpot - e_d);
  if (__umul64hi(x, y) == 0) return (int64_t)((x * y) / den);     // the product fits 64 bits (the usual case)
  return (int64_t)(((unsigned __int128)x * y) / den);
}

// Largest n in [0, cap] with E_p(n) <= epmax (Eq. 3 on the general prefill model), 0 if none.
__device__ inline int64_t dev_nsafe(const HfxParams &p, int64_t epmax, int64_t cap) {
  if (epmax == HFX_INF) return cap;
  if (dev_Ep(p, 0) > epmax) return 0;
  int64_t lo = 0, hi = cap;
  while (lo < hi) {
    int64_t mid = lo + (hi - lo + 1) / 2;
    if (dev_Ep(p, mid) <= epmax) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ inline int64_t dev_min_over_mask(const int64_t *v, uint64_t mask) {
  int64_t m = HFX_INF;
  while (mask) {
    int c = __ffsll((long long)mask) - 1;
    mask &= mask - 1;
    if (v[c] > 0 && v[c] < m) m = v[c];
  }
  return m;
}

// Dispatching step 2 for one replica: E_d of the running batch and the safe budget.
__device__ inline void dev_plan(const HfxParams &p, const hfx_replica_cfg &cfg, int64_t now, int64_t mat,
                                int64_t n_run, int64_t sum_kv, uint64_t mask_run, uint64_t mask_q,
                                ReplicaPlan &pl) {
  pl.now = now; pl.mat = mat; pl.start = now > mat ? now : mat;
  pl.mode = cfg.mode; pl.token_cap = cfg.token_cap; pl.batch_cap = cfg.batch_cap;
  pl.n_run = n_run; pl.sum_kv = sum_kv;
  const int64_t min_tpot = dev_min_over_mask(p.tpot, mask_run);
  const int64_t min_ttft = dev_min_over_mask(p.ttft, mask_q);
  const int64_t min_tpot_q = dev_min_over_mask(p.tpot, mask_q);
  const bool prefill = cfg.mode == HFX_PREFILL;
  pl.n_eff = prefill ? 0 : n_run;
  pl.kv_eff = prefill ? 0 : sum_kv;
  pl.tpot_eff = prefill ? HFX_INF : min_tpot;
  pl.e_d = pl.n_eff > 0 ? dev_Ed(p, pl.n_eff, pl.kv_eff) : 0;
  int64_t budget;
  if (cfg.mode == HFX_DECODE) {
    const int64_t T = (n_run > 0 && min_tpot < HFX_INF) ? min_tpot : min_tpot_q;
    if (p.budget_mode == HFX_BUDGET_CAP_ONLY || T == HFX_INF) budget = HFX_INF;
    else {
      const int64_t room = T - dev_Ed(p, n_run, sum_kv);
      budget = room > 0 ? room : 0;
    }
  } else {
    const int64_t cap_left = cfg.token_cap - pl.n_eff > 0 ? cfg.token_cap - pl.n_eff : 0;
    int64_t n_safe;
    if (p.budget_mode == HFX_BUDGET_CAP_ONLY) n_safe = cfg.token_cap;
    else n_safe = dev_nsafe(p, dev_epmax(min_ttft, pl.n_eff > 0 && pl.tpot_eff < HFX_INF, pl.tpot_eff, pl.e_d), cfg.token_cap);
    budget = n_safe < cap_left ? n_safe : cap_left;
  }
  if (now < mat) budget = 0;
  pl.budget = budget;
  pl.tpot_q0 = dev_Ed(p, pl.n_eff + 1, pl.kv_eff);
  pl.shift_run = now + pl.e_d;
  pl.shift_q = pl.start + (cfg.mode == HFX_DECODE ? pl.tpot_q0 : 0);
}

// The same plan computed by a whole warp (all 32 lanes call with the same arguments and get the same
// result).  The class minima are taken by lanes from a copy of the class tables in shared memory
// (cls_ttft / cls_tpot, HFX_MAX_CLASSES entries each); the largest safe n comes from a 32-way search
// on the bound itself, E_p(n) * (2 TPOT - E_d) <= TTFT * (TPOT - E_d), compared in 128 bits: for
// integer E_p that is the same set of n as E_p(n) <= floor(TTFT (TPOT - E_d) / (2 TPOT - E_d)), and no
// division is needed.
__device__ inline int64_t warp_min_over_mask(const int64_t *cls_v, uint64_t mask, int lane) {
  int64_t m = HFX_INF;
#pragma unroll
  for (int c = lane; c < HFX_MAX_CLASSES; c += 32)
    if ((mask >> c) & 1ull) { const int64_t x = cls_v[c]; if (x > 0 && x < m) m = x; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const int64_t w = __shfl_xor_sync(0xffffffffu, m, o); m = w < m ? w : m; }
  return m;
}

// What a caller that plans the same replica again and again keeps between its calls (one copy per lane
// of the planning warp, all lanes equal): the class sets seen last with their minima, and the last
// answer of the search, around which the next one starts.  None of it changes a result.
struct PlanMemo {
  uint64_t m_run, m_q;
  int64_t min_tpot, min_ttft;
  int64_t n_safe;           // < 0: none yet
  int64_t need;             // > 0: the caller only wants the budget if at least this many tokens are safe (the shortest
                            // prompt it could admit); otherwise the budget it gets is 0.  <= 0: always the exact budget
  int have_run, have_q;
};
__device__ __forceinline__ void plan_memo_reset(PlanMemo &m) { m.m_run = 0; m.m_q = 0; m.min_tpot = 0; m.min_ttft = 0; m.n_safe = -1; m.need = 0; m.have_run = 0; m.have_q = 0; }

// Largest n in [0, cap] with E_p(n) * den <= num (num = nh:nl as 128 bits, den > 0), 0 if none.
// `hint` >= 0: a value the answer is probably close to (tried first: 32 neighbours in one round).
// `need` > 0: return -1 at once when fewer than `need` tokens are safe.
__device__ inline int64_t warp_nsafe(const HfxParams &p, uint64_t nh, uint64_t nl, uint64_t den, int64_t cap, int lane,
                                     int64_t hint = -1, int64_t need = 0) {
  auto fits = [&](int64_t n) {
    const uint64_t ep = (uint64_t)dev_Ep(p, n);
    const uint64_t ph = __umul64hi(ep, den), pl = ep * den;
    return ph < nh || (ph == nh && pl <= nl);
  };
  if (need > 0) { if (need > cap || !fits(need)) return -1; }
  else if (!fits(0)) return 0;
  int64_t lo = need > 0 ? need : 0, hi = cap;          // fits(lo); the answer lies in [lo, hi]
  if (hint >= 0) {
    int64_t base = hint - 15;
    if (base < 1) base = 1;
    if (base > cap) base = cap;
    const int64_t cand = base + lane;
    const int f = __popc(__ballot_sync(0xffffffffu, cand <= cap && fits(cand)));    // a prefix of the lanes
    if (f == 0) hi = base - 1;                    // the answer lies below the neighbourhood
    else if (f == 32) lo = base + 31 > lo ? base + 31 : lo;      // at or above its top
    else return base + f - 1;
  }
  while (lo < hi) {
    const int64_t step = (int64_t)(((uint64_t)(hi - lo) + 31u) >> 5);
    const int64_t cand = lo + (int64_t)(lane + 1) * step;
    const int m = __popc(__ballot_sync(0xffffffffu, cand <= hi && fits(cand)));     // E_p is monotone: the ones that fit are a prefix
    const int64_t nlo = lo + (int64_t)m * step;
    int64_t nhi = lo + (int64_t)(m + 1) * step - 1;
    if (nhi > hi) nhi = hi;
    lo = nlo; hi = nhi;
  }
  return lo;
}

__device__ inline void warp_plan(const HfxParams &p, const int64_t *cls_ttft, const int64_t *cls_tpot,
                                 const hfx_replica_cfg &cfg, int64_t now, int64_t mat, int64_t n_run, int64_t sum_kv,
                                 uint64_t mask_run, uint64_t mask_q, ReplicaPlan &pl, int lane, PlanMemo *memo = nullptr) {
  pl.now = now; pl.mat = mat; pl.start = now > mat ? now : mat;
  pl.mode = cfg.mode; pl.token_cap = cfg.token_cap; pl.batch_cap = cfg.batch_cap;
  pl.n_run = n_run; pl.sum_kv = sum_kv;
  int64_t min_tpot;
  if (memo && memo->have_run && memo->m_run == mask_run) min_tpot = memo->min_tpot;
  else {
    min_tpot = warp_min_over_mask(cls_tpot, mask_run, lane);
    if (memo) { memo->m_run = mask_run; memo->min_tpot = min_tpot; memo->have_run = 1; }
  }
  const bool prefill = cfg.mode == HFX_PREFILL;
  pl.n_eff = prefill ? 0 : n_run;
  pl.kv_eff = prefill ? 0 : sum_kv;
  pl.tpot_eff = prefill ? HFX_INF : min_tpot;
  pl.e_d = pl.n_eff > 0 ? dev_Ed(p, pl.n_eff, pl.kv_eff) : 0;
  int64_t budget = 0;
  if (now >= mat) {      // before maturity the instance is protected: no budget to work out
    if (cfg.mode == HFX_DECODE) {
      const int64_t T = (n_run > 0 && min_tpot < HFX_INF) ? min_tpot : warp_min_over_mask(cls_tpot, mask_q, lane);
      if (p.budget_mode == HFX_BUDGET_CAP_ONLY || T == HFX_INF) budget = HFX_INF;
      else {
        const int64_t room = T - dev_Ed(p, n_run, sum_kv);
        budget = room > 0 ? room : 0;
      }
    } else {
      const int64_t cap_left = cfg.token_cap - pl.n_eff > 0 ? cfg.token_cap - pl.n_eff : 0;
      int64_t n_safe;
      if (p.budget_mode == HFX_BUDGET_CAP_ONLY) n_safe = cfg.token_cap;
      else {
        int64_t min_ttft;
        if (memo && memo->have_q && memo->m_q == mask_q) min_ttft = memo->min_ttft;
        else {
          min_ttft = warp_min_over_mask(cls_ttft, mask_q, lane);
          if (memo) { memo->m_q = mask_q; memo->min_ttft = min_ttft; memo->have_q = 1; }
        }
        const bool decoding = pl.n_eff > 0 && pl.tpot_eff < HFX_INF;
        const int64_t hint = memo ? memo->n_safe : -1, need = memo ? memo->need : 0;
        if (min_ttft == HFX_INF) n_safe = cfg.token_cap;
        else if (!decoding) n_safe = warp_nsafe(p, 0, (uint64_t)min_ttft, 2, cfg.token_cap, lane, hint, need);     // 2 E_p <= TTFT
        else if (pl.tpot_eff <= pl.e_d) n_safe = 0;
        else {
          const uint64_t x = (uint64_t)min_ttft, y = (uint64_t)(pl.tpot_eff - pl.e_d);
          n_safe = warp_nsafe(p, __umul64hi(x, y), x * y, (uint64_t)(2 * pl.tpot_eff - pl.e_d), cfg.token_cap, lane, hint, need);
        }
        if (n_safe < 0) n_safe = 0;      // fewer than `need` tokens are safe: the caller admits nothing
        else if (memo) memo->n_safe = n_safe;
      }
      budget = n_safe < cap_left ? n_safe : cap_left;
    }
  }
  pl.budget = budget;
  pl.tpot_q0 = dev_Ed(p, pl.n_eff + 1, pl.kv_eff);
  pl.shift_run = now + pl.e_d;
  pl.shift_q = pl.start + (cfg.mode == HFX_DECODE ? pl.tpot_q0 : 0);
}

// Dispatching step 4: maturity time after admitting adm_count requests of adm_cost in total.
__device__ inline int64_t dev_maturity_next(const HfxParams &p, const ReplicaPlan &pl, int64_t adm_count,
                                            int64_t adm_cost, int64_t adm_kv, int64_t *lp_out) {
  int64_t lp = 0, mat_next = pl.mat;
  if (pl.mode == HFX_DECODE) {
    if (pl.now >= pl.mat && pl.n_run + adm_count > 0)
      mat_next = pl.now + dev_Ed(p, pl.n_run + adm_count, pl.sum_kv + adm_kv);
  } else if (adm_count > 0) {
    lp = dev_Ep(p, adm_cost);
    if (pl.mode == HFX_PREFILL) mat_next = pl.now + lp;
    else {
      uint64_t k = 0;
      if (pl.n_eff > 0 && pl.tpot_eff < HFX_INF && pl.tpot_eff > pl.e_d) {
        const uint64_t d = (uint64_t)(pl.tpot_eff - pl.e_d);
        k = ((uint64_t)lp + d - 1) / d;
      }
      // now + lp + k * e_d, saturating at HFX_TIME_MAX (the product may need more than 64 bits)
      const uint64_t ed = (uint64_t)pl.e_d, prod = k * ed;
      const int64_t t = pl.now + lp;                              // |now| <= 2^56, lp < 2^61
      if (__umul64hi(k, ed) != 0 || prod >= (UINT64_C(1) << 63)) mat_next = HFX_TIME_MAX;
      else mat_next = (int64_t)prod > HFX_TIME_MAX - t ? HFX_TIME_MAX : t + (int64_t)prod;
    }
  }
  *lp_out = lp;
  return mat_next;
}

// ---- warp / block primitives ----------------------------------------------------------------
__device__ __forceinline__ int64_t warp_sum_i64(int64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int64_t warp_min_i64(int64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { int64_t w = __shfl_xor_sync(0xffffffffu, v, o); v = w < v ? w : v; }
  return v;
}
__device__ __forceinline__ uint64_t warp_or_u64(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v |= __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int64_t warp_incl_scan_i64(int64_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { int64_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
  return v;
}
__device__ __forceinline__ int32_t warp_incl_scan_i32(int32_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { int32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
  return v;
}

// Compare-exchange of sort items, ascending: `hi` alone (items carry their tie-break in the low
// bits) or the 96-bit pair (hi, lo).
template <bool WIDE>
__device__ __forceinline__ void cmp_swap(uint64_t *hi, uint32_t *lo, int i, int j) {
  const uint64_t hi_i = hi[i], hi_j = hi[j];
  if (WIDE) {
    const uint32_t lo_i = lo[i], lo_j = lo[j];
    if (hi_i > hi_j || (hi_i == hi_j && lo_i > lo_j)) { hi[i] = hi_j; hi[j] = hi_i; lo[i] = lo_j; lo[j] = lo_i; }
  } else if (hi_i > hi_j) { hi[i] = hi_j; hi[j] = hi_i; }
}

// Bitonic sorting network with ascending comparators only (mirrored first sub-stage), so the virtual
// +inf padding beyond n never moves: any n, in place.  Items are distinct, so the result is unique.
// Each warp owns a contiguous chunk of E items; stages whose pairs stay inside a chunk need only a
// warp barrier, the others a block barrier.  Callers synchronise the block before the call; the
// block is synchronised on return.
template <bool WIDE>
__device__ void block_sort(uint64_t *hi, uint32_t *lo, int n) {
  if (n > 1) {
    int n_pad = 2;
    while (n_pad < n) n_pad <<= 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
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
        if (local) { __syncthreads(); local = false; }
        for (int t = threadIdx.x; t < half; t += blockDim.x) {
          const int blk = t / hk, off = t - blk * hk;
          const int i = blk * k + off, j = blk * k + k - 1 - off;
          if (j < n) cmp_swap<WIDE>(hi, lo, i, j);
        }
        __syncthreads();
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
          if (local) { __syncthreads(); local = false; }
          for (int t = threadIdx.x; t < half; t += blockDim.x) {
            const int i = 2 * t - (t & (j - 1));
            if (i + j < n) cmp_swap<WIDE>(hi, lo, i, i + j);
          }
          __syncthreads();
        }
      }
    }
  }
  __syncthreads();
}

// First-fit admission along an order of n places, by one warp (all 32 lanes call).  cost_of(q) is the
// cost of the candidate at place q, or -1 where there is none; every candidate is tried in order against
// what is left of `budget` and of `room` (how many more may be taken) and taken if it fits; decide(q, taken)
// is called once for every place.  32 places at a time: the first lane that still fits starts a run, the
// run ends at the first lane that no longer fits behind it (that lane is refused for good), the lanes after
// it are tried again with what is left then.
template <typename CostF, typename DecideF>
__device__ __forceinline__ void warp_first_fit(int64_t n, int64_t budget, int64_t room, int lane, CostF cost_of, DecideF decide) {
  int64_t used = 0, taken = 0;
  for (int64_t base = 0; base < n; base += 32) {
    const int64_t q = base + lane;
    const int64_t c = q < n ? cost_of(q) : -1;
    uint32_t pending = __ballot_sync(0xffffffffu, c >= 0);
    bool mine = false;
    while (pending) {
      const int64_t rem = budget - used, left = room - taken;
      const bool me = (pending >> lane) & 1u;
      const uint32_t fit = left > 0 ? __ballot_sync(0xffffffffu, me && c <= rem) : 0u;
      if (!fit) break;
      const int l0 = __ffs(fit) - 1;
      const bool in = me && lane >= l0;
      const int64_t pre = warp_incl_scan_i64(in ? c : 0, lane);
      const int32_t pcnt = warp_incl_scan_i32(in ? 1 : 0, lane);
      const bool ok = in && pre <= rem && (int64_t)pcnt <= left;
      const uint32_t bad = __ballot_sync(0xffffffffu, in && !ok);
      const int l1 = bad ? __ffs(bad) - 1 : 32;            // the run is the pending lanes in [l0, l1)
      const bool take = in && lane < l1;
      if (take) mine = true;
      const uint32_t tm = __ballot_sync(0xffffffffu, take);
      const int last = 31 - __clz(tm);                      // tm has lane l0 at least
      used += __shfl_sync(0xffffffffu, pre, last);
      taken += __shfl_sync(0xffffffffu, pcnt, last);
      pending = l1 >= 31 ? 0u : (pending & ~((2u << l1) - 1u));
    }
    if (q < n) decide(q, mine);
  }
}

// Brackets one kernel launch with events when profiling is on; counts the launch either way.
struct KernelScope {
  hfx_sched *s; HfxBracket br; bool on; cudaStream_t st;
  KernelScope(hfx_sched *s_, int slot, cudaStream_t stream = nullptr) : s(s_), on(false), st(stream ? stream : s_->stream) {
    s->launches++;
    if (s->profiling && s->brackets) {
      br.slot = slot;
      if (cudaEventCreate(&br.a) == cudaSuccess && cudaEventCreate(&br.b) == cudaSuccess) {
        cudaEventRecord(br.a, st);
        on = true;
      }
    }
  }
  ~KernelScope() {
    if (on) { cudaEventRecord(br.b, st); s->brackets->push_back(br); }
  }
};

// ---- kernel argument blocks ------------------------------------------------------------------
// the fallback front end (global counters; tables with more replicas than the tile front end takes)
struct RegroupArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len;
  const int32_t *output_len; const int32_t *gen; const int64_t *arrival; const int64_t *first_token;
  const int32_t *req_id; const int32_t *weight;
  const int64_t *now; const int64_t *mat; const hfx_replica_cfg *cfg; const uint8_t *mode;
  int64_t *pred_ttft;    // optional output
  int64_t n;
  // per-row outputs written by the regroup itself
  int64_t *slack; int64_t *pred_tpot; uint64_t *key; int32_t *order; uint8_t *admit; int32_t *admitted_rows;
  uint32_t commit;
};

// the tile front end
struct FrontArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len; const int32_t *gen;
  const int64_t *arrival; const int64_t *first_token; const int32_t *req_id; const int32_t *weight;
  const int64_t *now; const int64_t *mat; const uint8_t *mode;
  int64_t n; int32_t tile_rows; int32_t n_tiles;
  // per-row outputs, written in row order
  int64_t *slack; int64_t *pred_ttft; int64_t *pred_tpot; uint64_t *key; uint8_t *admit; uint8_t *rowflag;
  // the slabs
  uint4 *slab_rec; uint16_t *slab_idx; uint2 *M; unsigned long long *tot; unsigned long long *tot_next;
  uint32_t *ordered; uint32_t *ordered_next; uint32_t *status;
};

struct SegArgs {
  // read-only table columns (fetched by row where a path needs them)
  const int64_t *arrival; const int32_t *req_id; const int32_t *output_len;
  // table columns written by COMMIT
  uint8_t *state; int32_t *gen; int64_t *first_token; int64_t *last_token; int64_t *finish;
  // replica state
  int64_t *now; int64_t *mat; const hfx_replica_cfg *cfg;
  // outputs
  int64_t *slack; int64_t *pred_tpot; uint64_t *key; int32_t *order; int32_t *seg_off; uint8_t *admit; int32_t *admitted_rows;
  int64_t *budget; int64_t *e_d; int32_t *n_run; int64_t *sum_kv; int64_t *adm_cost; int32_t *adm_count;
  int64_t *maturity_next;
  uint32_t flags;
  int64_t horizon;           // a replica whose clock is past it sits the commit out
};

// host-side launchers implemented in the .cu files
void hfx_front_shape(const hfx_sched *s, int64_t n, int32_t *tile_rows, int32_t *n_tiles);
int hfx_launch_front(hfx_sched *s, const FrontArgs &fa);
int hfx_launch_regroup(hfx_sched *s, const RegroupArgs &ra, int32_t *seg_off);
int hfx_launch_replicas(hfx_sched *s, const SegArgs &sa, int64_t n, bool slabs);
int hfx_launch_step(hfx_sched *s, const hfx_table *t, const hfx_replica_state *st, const hfx_step_out *o, uint32_t flags);
int hfx_launch_dispatch(hfx_sched *s, const hfx_table *t, int64_t now_ns, const int64_t *maturity, const hfx_dispatch_out *o,
                        int32_t cap_max, bool d_stage);
void hfx_dispatch_release(hfx_sched *s);
void hfx_sim_release(hfx_sched *s);
int hfx_launch_slo_map(hfx_sched *s, int32_t n_prio, const hfx_slo_window *win, const hfx_slo_bounds *b, int64_t *last_queue,
                       const int32_t *pending, const int32_t *new_prio, int64_t n_new, int64_t *ttft_out, int64_t *tpot_out);
size_t hfx_slomap_workspace_bytes();
int hfx_launch_pd_migrate(hfx_sched *s, const hfx_table *t, int32_t *replica_id, int64_t *now, const int32_t *pair, int64_t x0,
                          int64_t x1, int32_t *n_moved);
size_t hfx_pd_workspace_bytes(int n_replicas);
int hfx_launch_attainment(hfx_sched *s, const hfx_table *t, int64_t *out);
int hfx_launch_fleet_apply(hfx_sched *s, int64_t now, const int32_t *decision, const int64_t *used_blocks,
                           const int64_t *cold, const hfx_fleet *f, int64_t *clock, int64_t *maturity, int64_t *cost);
int hfx_launch_dispatch_bind(hfx_sched *s, int64_t n, int64_t now, const int32_t *assign, const int32_t *adm_count,
                             int32_t *replica_id, int64_t *clock);
int hfx_launch_sim(hfx_sched *s, const hfx_table *t, const int32_t *trace_off, int32_t n_traces, int32_t iters,
                   const hfx_sim_out *o);
