// Grouping the request table by replica: classify and count, scan, and the one streaming pass that
// turns every row the scheduler has to look at into a 32-byte record inside its replica's range.
//
// A row is ACTIVE when it is in flight or in the visible queue; everything else (not yet arrived,
// finished, rejected, bad data) is inactive: it only needs a place at the end of its replica's
// order.  Each replica's range [seg_begin[r], seg_begin[r+1]) holds its active rows first.
//
// Matrix mode (default): the table is cut into tiles; k_count classifies every row once (one flag
// byte per row) and writes two histogram rows per tile (all rows, active rows); k_colscan turns the
// columns into exclusive prefixes; k_regroup places each row at
//   range start + (rows of its replica and class in earlier tiles) + (rank inside the tile, row order)
// which is a stable partition without a single global atomic.  When additionally req_id rises with
// the row index (the step is then "ordered"), inactive rows need no record at all: the regroup
// writes their outputs and their place in the order directly.
// Atomic mode (very many replicas, so the tile matrices would be too large): global counters and
// global fill cursors; rows land in any order inside their class, which the sort repairs.
#include "hfx_internal.cuh"

#define THREADS_TILE 512

// dynamic shared memory of the regroup's arrays (multiple of 16 bytes)
__host__ __device__ inline size_t hfx_regroup_smem_dev(int R1, int tile_rows) {
  const size_t b = sizeof(int64_t) * (size_t)R1 + sizeof(uint32_t) * (4 * (size_t)R1 + 1) +
                   sizeof(uint16_t) * (2 * (size_t)tile_rows + 1) + (size_t)R1 + 32;
  return (b + 15) & ~(size_t)15;
}
#define COLSCAN_REG 16
#define GROUP_MAX 64      // largest same-replica group of an unsorted tile that is ranked by scanning

__device__ __forceinline__ int bucket_of(int rid, int R) { return (rid < 0 || rid >= R) ? R : rid; }

// Kind of a row (KIND_*), with ROWFLAG_BADREP for a row bound to no replica; raises status bits.
__device__ __forceinline__ uint32_t classify_row(const HfxParams &p, int32_t rid, uint32_t cls, uint32_t st, int32_t prompt,
                                                 int32_t gen, int64_t arrival, const int64_t *now, uint32_t &bad) {
  if (rid < 0 || rid >= p.n_replicas) {
    if (!(rid == -1 && st == HFX_QUEUED)) bad |= HFX_ST_BAD_REPLICA;      // -1 on a QUEUED row: still in the global queue, no error
    return KIND_DEAD | ROWFLAG_BADREP;
  }
  bool ok = true;
  if (cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
  if (prompt < 0 || prompt > HFX_MAX_TOKENS || gen < 0 || gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
  if (!ok) return KIND_DEAD;
  if (st == HFX_RUNNING) return KIND_RUNNING;
  if (st == HFX_QUEUED) return arrival <= __ldg(now + rid) ? KIND_QUEUED : KIND_FUTURE;
  return KIND_DEAD;
}

// ------------------------------------------------------------------------------------------------
// k_count: classify the rows of one tile, count them per replica (all / active), note how the
// regroup will rank the tile's rows, and whether the step can be "ordered".
// Matrix mode: M[tile][0][0..R] = all rows, M[tile][1][0..R] = active rows (plain stores).
// Atomic mode (M == nullptr): global counters tot_all / tot_act; never ordered.
// ------------------------------------------------------------------------------------------------
struct CountArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len;
  const int32_t *gen; const int64_t *arrival; const int32_t *req_id; const int64_t *now;
  int64_t n; int32_t tile_rows;
  uint32_t *M; uint8_t *tile_mode; uint32_t *tot_all; uint32_t *tot_act;
  uint8_t *rowflag; uint32_t *status; uint32_t *ordered;
};

// s_hist: [2][R1] words of shared memory (matrix mode only)
__device__ __forceinline__ void count_tile(const HfxParams &p, const CountArgs &a, uint32_t *s_hist) {
  const int R = p.n_replicas, R1 = R + 1;
  const bool matrix = a.M != nullptr;
  uint32_t *h_all = s_hist, *h_act = s_hist + R1;
  if (matrix) {
    for (int i = threadIdx.x; i < 2 * R1; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
  }
  const int64_t lo = (int64_t)blockIdx.x * a.tile_rows;
  const int64_t hi = lo + a.tile_rows < a.n ? lo + a.tile_rows : a.n;
  const int nt = hi > lo ? (int)(hi - lo) : 0;
  const int nvec = nt >> 2;
  const int64_t v0 = lo >> 2;
  uint32_t bad = 0;
  int sorted = 1, rising = 1;
  for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
    const int64_t gv = v0 + v;
    const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + gv);
    const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + gv);
    const uchar4 st = __ldg(reinterpret_cast<const uchar4 *>(a.state) + gv);
    const int4 pr = __ldg(reinterpret_cast<const int4 *>(a.prompt_len) + gv);
    const int4 ge = __ldg(reinterpret_cast<const int4 *>(a.gen) + gv);
    const int4 id = __ldg(reinterpret_cast<const int4 *>(a.req_id) + gv);
    const longlong2 ar0 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * gv);
    const longlong2 ar1 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * gv + 1);
    const int rr[4] = {rid.x, rid.y, rid.z, rid.w};
    const uint32_t cc[4] = {cls.x, cls.y, cls.z, cls.w}, ss[4] = {st.x, st.y, st.z, st.w};
    const int pp[4] = {pr.x, pr.y, pr.z, pr.w}, gg[4] = {ge.x, ge.y, ge.z, ge.w};
    const int64_t aa[4] = {ar0.x, ar0.y, ar1.x, ar1.y};
    uint32_t fl[4];
    int b[5];
#pragma unroll
    for (int k = 0; k < 4; k++) {
      fl[k] = classify_row(p, rr[k], cc[k], ss[k], pp[k], gg[k], aa[k], a.now, bad);
      b[k] = bucket_of(rr[k], R);
      if (matrix) { atomicAdd(&h_all[b[k]], 1u); if (fl[k] <= KIND_QUEUED) atomicAdd(&h_act[b[k]], 1u); }
      else { atomicAdd(&a.tot_all[b[k]], 1u); if (fl[k] <= KIND_QUEUED) atomicAdd(&a.tot_act[b[k]], 1u); }
    }
    *reinterpret_cast<uchar4 *>(a.rowflag + (gv << 2)) = make_uchar4(fl[0], fl[1], fl[2], fl[3]);
    // sorted by replica inside the tile?  req_id rising along the table (also across tiles)?
    const int64_t nxt = (gv << 2) + 4;
    b[4] = nxt < hi ? bucket_of(__ldg(a.replica_id + nxt), R) : b[3];
    if (b[0] > b[1] || b[1] > b[2] || b[2] > b[3] || b[3] > b[4]) sorted = 0;
    if (!(id.x < id.y && id.y < id.z && id.z < id.w && (nxt >= a.n || id.w < __ldg(a.req_id + nxt)))) rising = 0;
  }
  for (int i = (nvec << 2) + threadIdx.x; i < nt; i += blockDim.x) {
    const int64_t g = lo + i;
    const int32_t rid = a.replica_id[g];
    const uint32_t fl = classify_row(p, rid, a.class_id[g], a.state[g], a.prompt_len[g], a.gen[g], a.arrival[g], a.now, bad);
    const int b = bucket_of(rid, R);
    if (matrix) { atomicAdd(&h_all[b], 1u); if (fl <= KIND_QUEUED) atomicAdd(&h_act[b], 1u); }
    else { atomicAdd(&a.tot_all[b], 1u); if (fl <= KIND_QUEUED) atomicAdd(&a.tot_act[b], 1u); }
    a.rowflag[g] = (uint8_t)fl;
    if (g + 1 < hi && b > bucket_of(a.replica_id[g + 1], R)) sorted = 0;
    if (g + 1 < a.n && !(a.req_id[g] < a.req_id[g + 1])) rising = 0;
  }
  if (bad) atomicOr(a.status, bad);
  if (!matrix) return;
  sorted = __syncthreads_and(sorted);      // also orders the histogram updates before the reads below
  rising = __syncthreads_and(rising);
  uint32_t *row = a.M + (size_t)blockIdx.x * 2 * R1;
  uint32_t mx = 0;
  for (int i = threadIdx.x; i < 2 * R1; i += blockDim.x) {
    const uint32_t c = s_hist[i];
    row[i] = c;
    if (i < R) mx = c > mx ? c : mx;      // rows bound to no replica are ranked by a scan, whatever their number
  }
  const int small_groups = __syncthreads_and(mx <= GROUP_MAX);
  if (threadIdx.x == 0) {
    const int mode = sorted ? TILE_SORTED : (small_groups ? TILE_GROUPS : TILE_ANY);
    a.tile_mode[blockIdx.x] = (uint8_t)mode;
    if (mode == TILE_ANY || !rising) *a.ordered = 0;
  }
}

__global__ void __launch_bounds__(THREADS_TILE) k_count(const HfxParams p, const CountArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  count_tile(p, a, reinterpret_cast<uint32_t *>(smem_raw));
}

// ------------------------------------------------------------------------------------------------
// k_offsets: exclusive scan of the per-replica totals (one block) -> seg_begin and the user-visible
// seg_off; zeroes the fill cursors of the atomic mode; flags[2] = the largest number of items any
// replica has to sort (its active rows; without "ordered" also its inactive rows); re-arms the
// "ordered" word of the next step.
// ------------------------------------------------------------------------------------------------
struct OffsetArgs {
  const uint32_t *tot_all; const uint32_t *tot_act; int32_t R; uint32_t *seg_begin; uint32_t *cursor; int32_t *seg_off;
  uint32_t *flags; uint32_t parity; uint32_t force_unordered;
};

// one block of 1024 threads
__device__ void offsets_block(const OffsetArgs &oa) {
  const uint32_t *__restrict__ tot_all = oa.tot_all; const uint32_t *__restrict__ tot_act = oa.tot_act;
  const int32_t R = oa.R;
  uint32_t *__restrict__ seg_begin = oa.seg_begin; uint32_t *__restrict__ cursor = oa.cursor;
  int32_t *__restrict__ seg_off = oa.seg_off; uint32_t *__restrict__ flags = oa.flags;
  const uint32_t parity = oa.parity, force_unordered = oa.force_unordered;
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry_s, max_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { carry_s = 0; max_s = 0; if (force_unordered) flags[parity] = 0; }
  __syncthreads();
  const bool ordered = __ldcg(flags + parity) != 0;
  const int total = R + 1;  // buckets 0..R
  uint32_t mx = 0;
  for (int base = 0; base < total; base += blockDim.x) {
    const int i = base + threadIdx.x;
    // (L2 loads: in the fused kernel other blocks wrote these totals a moment ago)
    const uint32_t c = i < total ? __ldcg(tot_all + i) : 0;
    if (i < total) {
      const uint32_t act = __ldcg(tot_act + i);
      const uint32_t need = ordered ? act : (act > c - act ? act : c - act);
      mx = need > mx ? need : mx;
    }
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
      cursor[i] = 0;
      cursor[R + 2 + i] = 0;
      seg_off[i] = (int32_t)excl;   // seg_off[R] = number of rows bound to a valid replica
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = excl + c;
    __syncthreads();
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const uint32_t x = __shfl_xor_sync(0xffffffffu, mx, o); mx = x > mx ? x : mx; }
  if (lane == 0) atomicMax(&max_s, mx);
  __syncthreads();
  if (threadIdx.x == 0) { seg_begin[total] = carry_s; flags[2] = max_s; flags[parity ^ 1u] = 1u; }
}

__global__ void __launch_bounds__(1024) k_offsets(const OffsetArgs oa) { offsets_block(oa); }

// ------------------------------------------------------------------------------------------------
// k_colscan: for each column of the tile matrix (2 x (R+1) columns: all rows, active rows) the
// exclusive prefix of its counts over the tiles, in place, and the column total.
// Block = 32 columns x 32 chunks of tiles.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) k_colscan(uint32_t *__restrict__ M, int32_t n_tiles, int32_t R1,
                                                  uint32_t *__restrict__ tot_all, uint32_t *__restrict__ tot_act,
                                                  uint32_t *__restrict__ done, const OffsetArgs oa) {
  __shared__ uint32_t part[32][33];
  __shared__ uint32_t s_last;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int C = 2 * R1;
  const int col = blockIdx.x * 32 + lane;
  const int cb = (n_tiles + 31) / 32;
  const int t0 = w * cb < n_tiles ? w * cb : n_tiles;
  const int t1 = (t0 + cb < n_tiles) ? t0 + cb : n_tiles;
  // Up to COLSCAN_REG tiles per thread are held in registers (independent loads, one pass);
  // longer chunks take the two-pass loop.
  uint32_t v[COLSCAN_REG];
  const bool in_regs = cb <= COLSCAN_REG;
  uint32_t sum = 0;
  if (col < C) {
    if (in_regs) {
#pragma unroll
      for (int k = 0; k < COLSCAN_REG; k++) v[k] = t0 + k < t1 ? M[(size_t)(t0 + k) * C + col] : 0u;
#pragma unroll
      for (int k = 0; k < COLSCAN_REG; k++) sum += v[k];
    } else {
      for (int t = t0; t < t1; t++) sum += M[(size_t)t * C + col];
    }
  }
  part[w][lane] = sum;
  __syncthreads();
  uint32_t pre = 0;
  for (int k = 0; k < w; k++) pre += part[k][lane];
  if (col < C) {
    uint32_t run = pre;
    if (in_regs) {
#pragma unroll
      for (int k = 0; k < COLSCAN_REG; k++)
        if (t0 + k < t1) { M[(size_t)(t0 + k) * C + col] = run; run += v[k]; }
    } else {
      for (int t = t0; t < t1; t++) {
        const size_t idx = (size_t)t * C + col;
        const uint32_t x = M[idx];
        M[idx] = run;
        run += x;
      }
    }
    if (w == 31) { if (col < R1) tot_all[col] = pre + sum; else tot_act[col - R1] = pre + sum; }
  }
  // the block that finishes last turns the totals into offsets (no block waits for another)
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(done, 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (s_last) {
    __threadfence();
    offsets_block(oa);
    if (threadIdx.x == 0) *done = 0;
  }
}


// ------------------------------------------------------------------------------------------------
// Per-row work of the streaming pass: what does not depend on the replica's aggregates (prefill
// model of the prompt, slack base, priority) is evaluated here and packed into the record.
// ------------------------------------------------------------------------------------------------
struct RowIn {
  int32_t rid, prompt, gen, req_id, weight, out_len;
  uint32_t cls, kind;      // kind: the row's flag byte from k_count
  int64_t arrival, first_token;
};

// Fills the record of a row of kind in.kind.  The slack base is free of per-replica quantities (the
// replica's clock, earliest start and E_d are subtracted later, once per replica):
//   in flight                base = first_token + (gen+1) * tpot_slo              (next-token deadline)
//   queued, colocated/prefill base = ttft_slo + arrival - E_p(prompt_len)
//   queued on a decode replica base = first_token + (gen+1) * tpot_slo - d2 * (prompt_len + gen)
//   not yet arrived          base = arrival
__device__ __forceinline__ void make_record(const HfxParams &p, const int64_t *s_ttft, const int64_t *s_tpot,
                                            const uint8_t *s_prio, int64_t i, const RowIn &in, int mode, HfxRec &r) {
  r.req_id = in.req_id; r.row = (int32_t)i; r.prompt = in.prompt; r.gen = in.gen; r.output_len = in.out_len;
  r.cls = (uint8_t)in.cls; r.kind = (uint8_t)(in.kind & 3u); r.prio = 63; r.pad = 0; r.base = 0;
  if (in.kind == KIND_FUTURE) r.base = in.arrival;
  else if (in.kind <= KIND_QUEUED) {
    int prio;
    if (p.weight_max > 0) {
      const int64_t w = (int64_t)p.weight_max - in.weight;
      prio = (int)(w < 0 ? 0 : (w > 62 ? 62 : w));
    } else prio = s_prio[in.cls];
    r.prio = (uint8_t)prio;
    const int64_t ttft = s_ttft[in.cls], tpot = s_tpot[in.cls];
    if (in.kind == KIND_RUNNING) r.base = tpot > 0 ? in.first_token + ((int64_t)in.gen + 1) * tpot : BASE_UNBOUNDED;
    else if (mode == HFX_DECODE)
      r.base = tpot > 0 ? in.first_token + ((int64_t)in.gen + 1) * tpot - p.d2 * ((int64_t)in.prompt + in.gen) : BASE_UNBOUNDED;
    else r.base = ttft > 0 ? ttft + in.arrival - dev_Ep(p, in.prompt) : BASE_UNBOUNDED;
  }
}

// predicted TTFT of a row (optional output)
__device__ __forceinline__ int64_t row_pred_ttft(const HfxParams &p, const RowIn &in, int mode, int64_t start) {
  if (in.kind > KIND_QUEUED) return 0;
  if (in.kind == KIND_RUNNING || mode == HFX_DECODE) return in.first_token - in.arrival;
  return (start - in.arrival) + dev_Ep(p, in.prompt);
}

// One 32-byte store per record: a whole L2 sector at once (two 16-byte stores would each be a
// partial-sector write).
__device__ __forceinline__ void store_record(HfxRec *rec, uint32_t pos, const HfxRec &r) {
  const uint64_t *w = reinterpret_cast<const uint64_t *>(&r);
  asm volatile("st.global.v4.b64 [%0], {%1, %2, %3, %4};" ::"l"(rec + pos), "l"(w[0]), "l"(w[1]), "l"(w[2]), "l"(w[3]) : "memory");
}

// rows 4v .. 4v+3 with 16-byte loads
__device__ __forceinline__ void load_rows4(const RegroupArgs &a, const uint8_t *rowflag, int64_t v, RowIn in[4]) {
  const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + v);
  const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + v);
  const uchar4 kd = reinterpret_cast<const uchar4 *>(rowflag)[v];     // (not a read-only load: the fused kernel wrote it)
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
  in[0] = {rid.x, pr.x, ge.x, id.x, we.x, ol.x, cls.x, kd.x, ar0.x, ft0.x};
  in[1] = {rid.y, pr.y, ge.y, id.y, we.y, ol.y, cls.y, kd.y, ar0.y, ft0.y};
  in[2] = {rid.z, pr.z, ge.z, id.z, we.z, ol.z, cls.z, kd.z, ar1.x, ft1.x};
  in[3] = {rid.w, pr.w, ge.w, id.w, we.w, ol.w, cls.w, kd.w, ar1.y, ft1.y};
}

__device__ __forceinline__ void load_row1(const RegroupArgs &a, const uint8_t *rowflag, int64_t i, RowIn &in) {
  in = {a.replica_id[i], a.prompt_len[i], a.gen[i], a.req_id[i], a.weight ? a.weight[i] : 0,
        a.output_len ? a.output_len[i] : 0, a.class_id[i], rowflag[i], a.arrival[i], a.first_token[i]};
}

__device__ __forceinline__ void stage_classes(const HfxParams &p, int64_t *s_ttft, int64_t *s_tpot, uint8_t *s_prio) {
  for (int c = threadIdx.x; c < HFX_MAX_CLASSES; c += blockDim.x) {
    s_ttft[c] = c < p.n_classes ? p.ttft[c] : 0;
    s_tpot[c] = c < p.n_classes ? p.tpot[c] : 0;
    s_prio[c] = c < p.n_classes ? p.prio[c] : 63;
  }
}

// Per-row outputs that the regroup can finish by itself: slack 0 / admit 0 / inactive key for rows
// the scheduler does not look at, and the final slack and key of queued rows on colocated and
// prefill replicas (slack = base - earliest start needs nothing from the running batch).  Rows in
// flight and queued rows of decode replicas get their slack from the replica kernels afterwards;
// those kernels also set admit = 1 where it applies.
struct RowOut { int64_t slack; uint64_t k48; };

__device__ __forceinline__ RowOut row_out(const HfxRec &r, int mode, int64_t start) {
  RowOut o;
  o.slack = 0;
  o.k48 = dev_key48(PH_INACTIVE, 63, HFX_SLACK_MAX);
  if (r.kind == KIND_QUEUED && mode != HFX_DECODE) {
    o.slack = r.base == BASE_UNBOUNDED ? HFX_SLACK_MAX : r.base - start;
    o.k48 = dev_key48(PH_QUEUED, r.prio, o.slack);
  }
  return o;
}

// rows 4v .. 4v+3 with vector stores
__device__ __forceinline__ void write_outputs4(const RegroupArgs &a, int64_t v, const int bkt[4], const RowOut o[4]) {
  longlong2 *sl = reinterpret_cast<longlong2 *>(a.slack) + 2 * v;
  sl[0] = make_longlong2(o[0].slack, o[1].slack); sl[1] = make_longlong2(o[2].slack, o[3].slack);
  reinterpret_cast<uint32_t *>(a.admit)[v] = 0u;
  if (a.pred_tpot) {
    longlong2 *pt = reinterpret_cast<longlong2 *>(a.pred_tpot) + 2 * v;
    pt[0] = make_longlong2(0, 0); pt[1] = make_longlong2(0, 0);
  }
  if (a.key) {
    ulonglong2 *kp = reinterpret_cast<ulonglong2 *>(a.key) + 2 * v;
    kp[0] = make_ulonglong2(((uint64_t)(bkt[0] & 0xffff) << 48) | o[0].k48, ((uint64_t)(bkt[1] & 0xffff) << 48) | o[1].k48);
    kp[1] = make_ulonglong2(((uint64_t)(bkt[2] & 0xffff) << 48) | o[2].k48, ((uint64_t)(bkt[3] & 0xffff) << 48) | o[3].k48);
  }
}

__device__ __forceinline__ void write_outputs1(const RegroupArgs &a, int64_t i, int bkt, const RowOut &o) {
  a.slack[i] = o.slack;
  a.admit[i] = 0;
  if (a.pred_tpot) a.pred_tpot[i] = 0;
  if (a.key) a.key[i] = ((uint64_t)(bkt & 0xffff) << 48) | o.k48;
}

// atomic mode: positions from global fill cursors (any order inside a replica's two classes)
__global__ void __launch_bounds__(256) k_regroup_atomic(const HfxParams p, const RegroupArgs a, const uint8_t *__restrict__ rowflag,
                                                        const uint32_t *__restrict__ seg_begin,
                                                        const uint32_t *__restrict__ tot_act, uint32_t *__restrict__ cursor,
                                                        HfxRec *__restrict__ rec) {
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  stage_classes(p, s_ttft, s_tpot, s_prio);
  __syncthreads();
  const int R = p.n_replicas;
  auto emit = [&](int64_t i, const RowIn &in) {
    HfxRec r;
    const int bkt = bucket_of(in.rid, R);
    int mode = 0;
    int64_t start = 0;
    if (bkt < R) {
      mode = __ldg(a.mode + bkt);
      const int64_t now = __ldg(a.now + bkt), mat = __ldg(a.mat + bkt);
      start = now > mat ? now : mat;
    }
    make_record(p, s_ttft, s_tpot, s_prio, i, in, mode, r);
    if (a.pred_ttft) a.pred_ttft[i] = row_pred_ttft(p, in, mode, start);
    write_outputs1(a, i, bkt, row_out(r, mode, start));
    const uint32_t pos = in.kind <= KIND_QUEUED ? seg_begin[bkt] + atomicAdd(&cursor[bkt], 1u)
                                                : seg_begin[bkt] + tot_act[bkt] + atomicAdd(&cursor[R + 2 + bkt], 1u);
    store_record(rec, pos, r);
  };
  const int64_t n4 = a.n >> 2;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
    RowIn in[4];
    load_rows4(a, rowflag, v, in);
#pragma unroll
    for (int k = 0; k < 4; k++) emit((v << 2) + k, in[k]);
  }
  if (blockIdx.x == 0) {
    for (int64_t i = (n4 << 2) + threadIdx.x; i < a.n; i += blockDim.x) {
      RowIn in;
      load_row1(a, rowflag, i, in);
      emit(i, in);
    }
  }
}

// matrix mode: see the head of this file
struct TileArgs {
  const uint32_t *M; const uint8_t *tile_mode; const uint32_t *seg_begin; const uint32_t *tot_act;
  const uint8_t *rowflag; const uint32_t *ordered; HfxRec *rec; int32_t tile_rows;
};

// ta.seg_begin and ta.tot_act may point to shared memory (the fused kernel keeps its own copy there).
__device__ __forceinline__ void regroup_tile(const HfxParams &p, const RegroupArgs &a, const TileArgs &ta, unsigned char *smem_raw) {
  const int R = p.n_replicas, R1 = R + 1, T = ta.tile_rows;
  int64_t *s_start = reinterpret_cast<int64_t *>(smem_raw);          // [R1]   earliest start max(now, maturity)
  uint32_t *s_cnt = reinterpret_cast<uint32_t *>(s_start + R1);      // [R1]   rows of each replica in the tile / cursors
  uint32_t *s_off = s_cnt + R1;                                      // [R1+1] exclusive prefix of s_cnt / cursors
  uint32_t *s_bact = s_off + R1 + 1;                                 // [R1]   where the tile's active rows of r start
  uint32_t *s_bin = s_bact + R1;                                     // [R1]   where its inactive rows start
  uint16_t *s_stage = reinterpret_cast<uint16_t *>(s_bin + R1);      // [T]    tile rows grouped by replica (+ class bit)
  uint16_t *s_P = s_stage + T;                                       // [T+1]  active rows before each tile position
  uint8_t *s_mode = reinterpret_cast<uint8_t *>(s_P + T + 1);        // [R1]   replica modes
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  __shared__ uint32_t s_warp[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
  const int mode = ta.tile_mode[blockIdx.x];
  const bool ordered = __ldcg(ta.ordered) != 0;

  stage_classes(p, s_ttft, s_tpot, s_prio);
  for (int i = tid; i < R1; i += blockDim.x) {
    s_cnt[i] = 0; s_off[i] = 0; s_mode[i] = i < R ? a.mode[i] : 0;
    { int64_t st = 0; if (i < R) { const int64_t nw = a.now[i], mt = a.mat[i]; st = nw > mt ? nw : mt; } s_start[i] = st; }
  }
  __syncthreads();

  const int64_t lo = (int64_t)blockIdx.x * T;
  const int64_t hi = lo + T < a.n ? lo + T : a.n;
  const int nt = hi > lo ? (int)(hi - lo) : 0;
  const int nvec = nt >> 2;
  const int64_t v0 = lo >> 2;
  const size_t mrow = (size_t)blockIdx.x * 2 * R1;

  bool tail_scan = false;
  if (mode != TILE_ANY) {
    // ---- A: histogram of the tile; active flag of every position ------------------------------------
    for (int v = tid; v < nvec; v += blockDim.x) {
      const int4 r4 = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + v0 + v);
      const uchar4 k4 = reinterpret_cast<const uchar4 *>(ta.rowflag)[v0 + v];
      atomicAdd(&s_cnt[bucket_of(r4.x, R)], 1u); atomicAdd(&s_cnt[bucket_of(r4.y, R)], 1u);
      atomicAdd(&s_cnt[bucket_of(r4.z, R)], 1u); atomicAdd(&s_cnt[bucket_of(r4.w, R)], 1u);
      s_P[4 * v] = k4.x <= KIND_QUEUED; s_P[4 * v + 1] = k4.y <= KIND_QUEUED;
      s_P[4 * v + 2] = k4.z <= KIND_QUEUED; s_P[4 * v + 3] = k4.w <= KIND_QUEUED;
    }
    for (int i = (nvec << 2) + tid; i < nt; i += blockDim.x) {
      atomicAdd(&s_cnt[bucket_of(a.replica_id[lo + i], R)], 1u);
      s_P[i] = ta.rowflag[lo + i] <= KIND_QUEUED;
    }
    __syncthreads();
    // ---- B: exclusive scan of the histogram ---------------------------------------------------------
    {
      const int per = (R1 + blockDim.x - 1) / blockDim.x;
      const int i0 = tid * per < R1 ? tid * per : R1, i1 = (i0 + per < R1) ? i0 + per : R1;
      uint32_t sum = 0;
      for (int i = i0; i < i1; i++) sum += s_cnt[i];
      uint32_t v = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
      if (lane == 31) s_warp[warp] = v;
      __syncthreads();
      if (warp == 0) {
        uint32_t w = lane < nwarp ? s_warp[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += x; }
        s_warp[lane] = w;
      }
      __syncthreads();
      uint32_t run = (warp ? s_warp[warp - 1] : 0) + v - sum;
      for (int i = i0; i < i1; i++) { s_off[i] = run; run += s_cnt[i]; }
      if (tid == 0) s_off[R1] = (uint32_t)nt;
    }
    __syncthreads();
    // exclusive scan of s_P[0 .. nt) in place, the total in s_P[nt]
    auto scan_P = [&]() {
      const int per = (nt + blockDim.x - 1) / blockDim.x;
      const int i0 = tid * per < nt ? tid * per : nt, i1 = (i0 + per < nt) ? i0 + per : nt;
      uint32_t sum = 0;
      for (int i = i0; i < i1; i++) sum += s_P[i];
      uint32_t v = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
      if (lane == 31) s_warp[warp] = v;
      __syncthreads();
      if (warp == 0) {
        uint32_t w = lane < nwarp ? s_warp[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += x; }
        s_warp[lane] = w;
      }
      __syncthreads();
      uint32_t run = (warp ? s_warp[warp - 1] : 0) + v - sum;
      for (int i = i0; i < i1; i++) { const uint32_t f = s_P[i]; s_P[i] = (uint16_t)run; run += f; }
      if (i1 == nt && i0 < nt) s_P[nt] = (uint16_t)run;
      if (nt == 0 && tid == 0) s_P[0] = 0;
    };
    if (mode == TILE_SORTED) {
      // ---- C0: s_P := number of active rows before each position ----------------------------------------
      scan_P();
    } else {
      // ---- C1: tile rows grouped by replica (counting sort of local indices, class in bit 15) ---------
      tail_scan = s_off[R1] - s_off[R] > GROUP_MAX;
      for (int i = tid; i < R1; i += blockDim.x) s_cnt[i] = 0;
      __syncthreads();
      for (int i = tid; i < nt; i += blockDim.x) {
        const int b = bucket_of(__ldg(a.replica_id + lo + i), R);
        if (b == R && tail_scan) continue;
        s_stage[s_off[b] + atomicAdd(&s_cnt[b], 1u)] = (uint16_t)(i | (s_P[i] ? 0x8000 : 0));
      }
      if (tail_scan) {
        // ---- C2: many rows bound to no replica (none of them active): s_P := how many precede each position
        __syncthreads();
        for (int i = tid; i < nt; i += blockDim.x) s_P[i] = bucket_of(__ldg(a.replica_id + lo + i), R) == R;
        __syncthreads();
        scan_P();
      }
    }
  }
  for (int i = tid; i < R1; i += blockDim.x) {
    const uint32_t m_all = __ldcg(ta.M + mrow + i), m_act = __ldcg(ta.M + mrow + R1 + i), sb = ta.seg_begin[i];
    s_bact[i] = sb + m_act;
    s_bin[i] = sb + ta.tot_act[i] + (m_all - m_act);
  }
  __syncthreads();

  // ---- D: records of active rows; inactive rows: their outputs (ordered) or their records ----------
  auto emit = [&](int64_t i, int il, const RowIn &in) -> RowOut {
    const int bkt = bucket_of(in.rid, R);
    const bool act = in.kind <= KIND_QUEUED;
    uint32_t rank;
    if (mode == TILE_SORTED) {
      const uint32_t o = s_off[bkt];
      const uint32_t ra = (uint32_t)s_P[il] - (uint32_t)s_P[o];
      rank = act ? ra : (uint32_t)il - o - ra;
    } else if (mode == TILE_GROUPS && bkt == R && tail_scan) {
      rank = s_P[il];
    } else if (mode == TILE_GROUPS) {
      rank = 0;
      const uint32_t g0 = s_off[bkt], g1 = s_off[bkt + 1];
      const uint32_t me = (uint32_t)il | (act ? 0x8000u : 0u);
      for (uint32_t g = g0; g < g1; g++) { const uint32_t e = s_stage[g]; rank += ((e ^ me) < 0x8000u && e < me) ? 1u : 0u; }
    } else rank = atomicAdd(act ? &s_cnt[bkt] : &s_off[bkt], 1u);
    const int rmode = s_mode[bkt];
    const int64_t start = s_start[bkt];
    if (a.pred_ttft) a.pred_ttft[i] = row_pred_ttft(p, in, rmode, start);
    RowOut o;
    o.slack = 0; o.k48 = dev_key48(PH_INACTIVE, 63, HFX_SLACK_MAX);
    if (act || !ordered) {
      HfxRec r;
      make_record(p, s_ttft, s_tpot, s_prio, i, in, rmode, r);
      o = row_out(r, rmode, start);
      store_record(ta.rec, (act ? s_bact[bkt] : s_bin[bkt]) + rank, r);
    } else {
      a.order[s_bin[bkt] + rank] = (int32_t)i;
    }
    return o;
  };
  for (int v = tid; v < nvec; v += blockDim.x) {
    RowIn in[4];
    load_rows4(a, ta.rowflag, v0 + v, in);
    const int bk[4] = {bucket_of(in[0].rid, R), bucket_of(in[1].rid, R), bucket_of(in[2].rid, R), bucket_of(in[3].rid, R)};
    RowOut o[4];
#pragma unroll
    for (int k = 0; k < 4; k++) o[k] = emit(lo + 4 * (int64_t)v + k, 4 * v + k, in[k]);
    write_outputs4(a, v0 + v, bk, o);
  }
  for (int i = (nvec << 2) + tid; i < nt; i += blockDim.x) {
    RowIn in;
    load_row1(a, ta.rowflag, lo + i, in);
    const RowOut o = emit(lo + i, i, in);
    write_outputs1(a, lo + i, bucket_of(in.rid, R), o);
  }
}

__global__ void __launch_bounds__(THREADS_TILE, 2) k_regroup(const HfxParams p, const RegroupArgs a, const TileArgs ta) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  regroup_tile(p, a, ta, smem_raw);
}

// ------------------------------------------------------------------------------------------------
// k_front: count, column scan, offsets and regroup as ONE cooperative kernel (one block per tile,
// all blocks resident), separated by two grid barriers.  The barriers count arrivals on a 64-bit
// word that only ever grows: the host passes the value it must reach, so nothing is reset
// between launches.  Every wait is bounded; a block whose wait runs out raises HFX_ST_TIMEOUT and
// leaves.
// ------------------------------------------------------------------------------------------------
__device__ bool front_barrier(unsigned long long *bar, unsigned long long target, uint32_t *status) {
  __shared__ int ok_s;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(bar, 1ull);
    int ok = 0;
    for (int spin = 0; spin < (1 << 22); spin++) {
      if (*((volatile unsigned long long *)bar) >= target) { ok = 1; break; }
      if (spin > 64) __nanosleep(spin > 4096 ? 256 : 20);
    }
    if (!ok) atomicOr(status, HFX_ST_TIMEOUT);
    __threadfence();
    ok_s = ok;
  }
  __syncthreads();
  return ok_s != 0;
}

// Column scan of the tile matrix by the whole grid.  A block takes 8 neighbouring columns (one
// 32-byte sector of every matrix row): its 16 warps load them for all tiles (a lane = one of 4 tiles
// x 8 columns, so every load instruction reads whole sectors), the block transposes them through
// shared memory, one warp per column scans its tiles, and the prefixes go back the way they came.
// M was written by other blocks of this kernel: L2 loads.  At most FRONT_TILES_MAX tiles.
#define FRONT_TILES_MAX 512
#define FRONT_LD (FRONT_TILES_MAX / (THREADS_TILE / 8))     // loads per thread
__device__ __forceinline__ void colscan_grid(uint32_t *M, int32_t n_tiles, int32_t R1, uint32_t *tot_all, uint32_t *tot_act,
                                             uint32_t *s_t /* [n_tiles][9] */) {
  const int C = 2 * R1;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = threadIdx.x & 7, tsub = threadIdx.x >> 3;          // tsub in [0, 64)
  for (int g = blockIdx.x; g * 8 < C; g += gridDim.x) {
    const int col = g * 8 + c;
    uint32_t x[FRONT_LD];
#pragma unroll
    for (int k = 0; k < FRONT_LD; k++) {
      const int t = tsub + 64 * k;
      x[k] = (t < n_tiles && col < C) ? __ldcg(M + (size_t)t * C + col) : 0u;
    }
#pragma unroll
    for (int k = 0; k < FRONT_LD; k++) { const int t = tsub + 64 * k; if (t < n_tiles) s_t[t * 9 + c] = x[k]; }
    __syncthreads();
    if (warp < 8) {       // warp = column of the group; a lane scans a run of consecutive tiles
      const int per = (n_tiles + 31) / 32;
      const int t0 = lane * per < n_tiles ? lane * per : n_tiles, t1 = (t0 + per < n_tiles) ? t0 + per : n_tiles;
      uint32_t sum = 0;
      for (int t = t0; t < t1; t++) sum += s_t[t * 9 + warp];
      uint32_t v = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
      uint32_t run = v - sum;
      for (int t = t0; t < t1; t++) { const uint32_t y = s_t[t * 9 + warp]; s_t[t * 9 + warp] = run; run += y; }
      const int wc = g * 8 + warp;
      if (lane == 31 && wc < C) { if (wc < R1) tot_all[wc] = v; else tot_act[wc - R1] = v; }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < FRONT_LD; k++) {
      const int t = tsub + 64 * k;
      if (t < n_tiles && col < C) M[(size_t)t * C + col] = s_t[t * 9 + c];
    }
    __syncthreads();
  }
}

// Exclusive scan of the per-replica totals into shared memory (every block computes its own copy);
// block 0 also publishes what the replica kernels and the caller read: seg_begin, seg_off, the
// largest sort size, and it re-arms the next step's "ordered" word.
__device__ __forceinline__ void offsets_local(const OffsetArgs &oa, uint32_t *s_segb /* [R+2] */, uint32_t *s_act /* [R+1] */) {
  __shared__ uint32_t warp_tot[32], warp_max[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const bool pub = blockIdx.x == 0;
  const bool ordered = __ldcg(oa.flags + oa.parity) != 0;
  const int total = oa.R + 1;
  // each thread owns a run of consecutive replicas
  const int per = (total + blockDim.x - 1) / blockDim.x;
  const int i0 = threadIdx.x * per < total ? threadIdx.x * per : total, i1 = (i0 + per < total) ? i0 + per : total;
  for (int i = threadIdx.x; i < total; i += blockDim.x) { s_segb[i] = __ldcg(oa.tot_all + i); s_act[i] = __ldcg(oa.tot_act + i); }
  __syncthreads();
  uint32_t sum = 0, mx = 0;
  for (int i = i0; i < i1; i++) {
    const uint32_t c = s_segb[i], act = s_act[i];
    sum += c;
    const uint32_t need = ordered ? act : (act > c - act ? act : c - act);
    mx = need > mx ? need : mx;
  }
  uint32_t v = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const uint32_t x = __shfl_xor_sync(0xffffffffu, mx, o); mx = x > mx ? x : mx; }
  if (lane == 31) warp_tot[warp] = v;
  if (lane == 0) warp_max[warp] = mx;
  __syncthreads();
  uint32_t run = v - sum, all = 0, mxall = 0;
  for (int k = 0; k < nwarp; k++) { const uint32_t w = warp_tot[k]; if (k < warp) run += w; all += w; mxall = warp_max[k] > mxall ? warp_max[k] : mxall; }
  for (int i = i0; i < i1; i++) {
    const uint32_t c = s_segb[i];
    s_segb[i] = run;
    if (pub) { oa.seg_begin[i] = run; oa.seg_off[i] = (int32_t)run; }
    run += c;
  }
  if (threadIdx.x == 0) {
    s_segb[total] = all;
    if (pub) { oa.seg_begin[total] = all; oa.flags[2] = mxall; oa.flags[oa.parity ^ 1u] = 1u; }
  }
  __syncthreads();
}

struct FrontArgs { unsigned long long *bar; unsigned long long target; uint32_t *status; int32_t n_tiles; };

__global__ void __launch_bounds__(THREADS_TILE, 2) k_front(const HfxParams p, const CountArgs ca, const OffsetArgs oa,
                                                           const RegroupArgs ra, const TileArgs ta0, const FrontArgs fa) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R1 = p.n_replicas + 1;
  count_tile(p, ca, reinterpret_cast<uint32_t *>(smem_raw));
  if (!front_barrier(fa.bar, fa.target, fa.status)) return;
  colscan_grid(ca.M, fa.n_tiles, R1, ca.tot_all, ca.tot_act, reinterpret_cast<uint32_t *>(smem_raw));
  if (!front_barrier(fa.bar, fa.target + gridDim.x, fa.status)) return;
  // the block's own copy of the range starts and active counts sits behind the regroup's arrays
  uint32_t *s_segb = reinterpret_cast<uint32_t *>(smem_raw + hfx_regroup_smem_dev(R1, ta0.tile_rows));
  uint32_t *s_act = s_segb + R1 + 1;
  offsets_local(oa, s_segb, s_act);
  TileArgs ta = ta0;
  ta.seg_begin = s_segb; ta.tot_act = s_act;
  regroup_tile(p, ra, ta, smem_raw);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
size_t hfx_regroup_smem(int R1, int tile_rows) { return hfx_regroup_smem_dev(R1, tile_rows); }

// shared memory of the fused kernel: the regroup's arrays (the count's histograms reuse their space)
// plus the block's copy of the offsets, or the column scan's slab if that is larger
static size_t hfx_front_smem(int R1, int tile_rows, int n_tiles) {
  const size_t regroup = hfx_regroup_smem_dev(R1, tile_rows) + sizeof(uint32_t) * (2 * (size_t)R1 + 2);
  const size_t colscan = sizeof(uint32_t) * 9 * (size_t)n_tiles;      // the transposed 8-column slab of the column scan
  return regroup > colscan ? regroup : colscan;
}

int hfx_launch_regroup(hfx_sched *s, const RegroupArgs &ra, int32_t *seg_off) {
  const int R = s->p.n_replicas, R1 = R + 1;
  const int64_t n = ra.n;
  cudaStream_t stream = s->stream;
  int32_t tile_rows, n_tiles;
  hfx_tile_shape(n, &tile_rows, &n_tiles);
  const bool matrix = s->d_tile_hist != nullptr && n_tiles <= s->tile_blocks_max;
  uint32_t *ordered = s->d_flags + s->step_parity;
  CountArgs ca;
  ca.replica_id = ra.replica_id; ca.class_id = ra.class_id; ca.state = ra.state; ca.prompt_len = ra.prompt_len;
  ca.gen = ra.gen; ca.arrival = ra.arrival; ca.req_id = ra.req_id; ca.now = ra.now; ca.n = n; ca.tile_rows = tile_rows;
  ca.M = matrix ? s->d_tile_hist : nullptr; ca.tile_mode = s->d_tile_mode; ca.tot_all = s->d_seg_count;
  ca.tot_act = s->d_act_count; ca.rowflag = s->d_rowflag; ca.status = s->d_status; ca.ordered = ordered;
  const size_t front_smem = hfx_front_smem(R1, tile_rows, n_tiles);
  bool fused = matrix && s->front_enabled && front_smem <= 200 * 1024 && n_tiles <= FRONT_TILES_MAX;
  if (fused) {     // every tile's block must be resident at once
    if (s->front_smem_cached != front_smem) {
      int per_sm = 0;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_front, THREADS_TILE, front_smem) != cudaSuccess) per_sm = 0;
      s->front_smem_cached = front_smem;
      s->front_capacity = per_sm * s->n_sm;
    }
    fused = n_tiles <= s->front_capacity;
  }
  if (fused) {
    OffsetArgs oa = {s->d_seg_count, s->d_act_count, R, s->d_seg_begin, s->d_cursor, seg_off, s->d_flags, s->step_parity, 0u};
    TileArgs ta;
    ta.M = s->d_tile_hist; ta.tile_mode = s->d_tile_mode; ta.seg_begin = nullptr; ta.tot_act = nullptr;
    ta.rowflag = s->d_rowflag; ta.ordered = ordered; ta.rec = s->d_rec; ta.tile_rows = tile_rows;
    FrontArgs fa;
    fa.bar = s->d_front_bar; fa.target = s->front_arrivals + (unsigned long long)n_tiles; fa.status = s->d_status; fa.n_tiles = n_tiles;
    s->front_arrivals += 2ull * (unsigned long long)n_tiles;
    void *args[] = {(void *)&s->p, (void *)&ca, (void *)&oa, (void *)&ra, (void *)&ta, (void *)&fa};
    KernelScope ks(s, KSLOT_FRONT);
    if (cudaLaunchCooperativeKernel((void *)k_front, dim3(n_tiles), dim3(THREADS_TILE), args, front_smem, stream) != cudaSuccess)
      return HFX_E_CUDA;
  } else if (matrix) {
    {
      KernelScope ks(s, KSLOT_COUNT);
      k_count<<<n_tiles, THREADS_TILE, sizeof(uint32_t) * 2 * R1, stream>>>(s->p, ca);
    }
    {
      KernelScope ks(s, KSLOT_COLSCAN);
      const OffsetArgs oa = {s->d_seg_count, s->d_act_count, R, s->d_seg_begin, s->d_cursor, seg_off, s->d_flags,
                             s->step_parity, 0u};
      k_colscan<<<(2 * R1 + 31) / 32, 1024, 0, stream>>>(s->d_tile_hist, n_tiles, R1, s->d_seg_count, s->d_act_count,
                                                          s->d_flags + 3, oa);
    }
    {
      KernelScope ks(s, KSLOT_REGROUP);
      TileArgs ta;
      ta.M = s->d_tile_hist; ta.tile_mode = s->d_tile_mode; ta.seg_begin = s->d_seg_begin; ta.tot_act = s->d_act_count;
      ta.rowflag = s->d_rowflag; ta.ordered = ordered; ta.rec = s->d_rec; ta.tile_rows = tile_rows;
      k_regroup<<<n_tiles, THREADS_TILE, hfx_regroup_smem(R1, tile_rows), stream>>>(s->p, ra, ta);
    }
  } else {
    if (cudaMemsetAsync(s->d_seg_count, 0, sizeof(uint32_t) * (R + 2), stream) != cudaSuccess ||
        cudaMemsetAsync(s->d_act_count, 0, sizeof(uint32_t) * (R + 2), stream) != cudaSuccess)
      return HFX_E_CUDA;
    {
      KernelScope ks(s, KSLOT_COUNT);
      k_count<<<n_tiles, THREADS_TILE, 0, stream>>>(s->p, ca);
    }
    {
      KernelScope ks(s, KSLOT_OFFSETS);
      const OffsetArgs oa = {s->d_seg_count, s->d_act_count, R, s->d_seg_begin, s->d_cursor, seg_off, s->d_flags,
                             s->step_parity, 1u};
      k_offsets<<<1, 1024, 0, stream>>>(oa);
    }
    {
      KernelScope ks(s, KSLOT_REGROUP);
      k_regroup_atomic<<<s->n_sm * 8, 256, 0, stream>>>(s->p, ra, s->d_rowflag, s->d_seg_begin, s->d_act_count, s->d_cursor,
                                                        s->d_rec);
    }
  }
  return HFX_OK;
}

int hfx_regroup_configure() {
  if (cudaFuncSetAttribute(k_regroup, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(k_front, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}
