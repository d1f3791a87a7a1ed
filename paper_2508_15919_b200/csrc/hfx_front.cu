// Front end of a step: ONE pass over the request table, no wait between blocks.
//
// The table is cut into tiles; one block per tile.  The block loads its rows once (16-byte vector
// loads), classifies them, evaluates what does not depend on the replica's running batch (prefill model
// of the prompt, slack base, priority; final slack and key of queued rows on colocated / prefill
// replicas), writes the per-row outputs in row order, and leaves the tile's rows grouped by replica in a
// slab of its own:
//   slab_idx[t*T + j]   local row indices of ALL rows of tile t, by replica; inside a replica the active
//                       rows (in flight or visible queue) first, each part in row order
//   slab_rec[t*T + k]   16-byte records of the ACTIVE rows, in the same order
//   M[t][r]             where replica r's rows sit in the two slabs (offsets and counts)
//   tot[r]              rows / active rows per replica over all tiles (one 64-bit atomic add per tile
//                       and replica)
// The cross-tile prefix (where tile t's rows of replica r go inside the replica's range) is left to
// the replica's block in the next kernel, which reads column r of M and gathers its chunks in tile
// order: that order is row order, so the grouping is stable without any grid-wide wait.
#include "hfx_rows.cuh"

#define FRONT_THREADS 1024
#define FRONT_PER 8                 // rows per thread in the scans over tile positions: T <= 8192
#define FRONT_GROUP_MAX 1024        // largest group that is put in row order by counting (a row costs its group's size; the network over the
                                    // whole tile that larger groups need costs as much as groups of about a thousand rows)
#define FRONT_TAIL_MAX 64           // more rows bound to no replica than this are ranked by a scan
#define FRONT_ROW_BYTES 24          // shared memory per row of the tile
#define FRONT_REP_BYTES 31          // shared memory per replica

// shared memory of the tile kernel
__host__ __device__ inline size_t front_smem_bytes(int R1, int T) {
  size_t b = 16 * (size_t)T;                       // s_rec
  b += 16 * (size_t)R1;                            // s_now, s_start
  b += 8 * (size_t)R1;                             // s_cnt
  b += 4 * (size_t)T;                              // s_bkt
  b += 4 * (size_t)R1 + 2 * (size_t)R1;            // s_base, s_offact
  b += 2 * 2 * ((size_t)T + 8);                    // s_perm, s_fin
  b += (size_t)R1 + 64;                            // s_mode
  return (b + 15) & ~(size_t)15;
}

// exclusive prefix of `mine` over the threads of the block (two barriers); *total = block sum
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t mine, uint32_t *s_warp, uint32_t *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  uint32_t v = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
  __syncthreads();                 // s_warp may still be read from a previous call
  if (lane == 31) s_warp[warp] = v;
  __syncthreads();
  uint32_t pre = 0, all = 0;
  for (int k = 0; k < nwarp; k++) { const uint32_t w = s_warp[k]; if (k < warp) pre += w; all += w; }
  if (total) *total = all;
  return pre + v - mine;
}

// EXTRA: the optional per-row outputs (predicted TTFT, predicted TPOT default, key) are wanted
template <bool EXTRA>
__global__ void __launch_bounds__(FRONT_THREADS, 1) k_front(const HfxParams p, const FrontArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = p.n_replicas, R1 = R + 1, T = a.tile_rows;
  uint4 *s_rec = reinterpret_cast<uint4 *>(smem_raw);                    // [T]    record of every active row, by local index
  int64_t *s_now = reinterpret_cast<int64_t *>(s_rec + T);               // [R1]
  int64_t *s_start = s_now + R1;                                         // [R1]   earliest start max(now, maturity)
  uint32_t *s_cnt = reinterpret_cast<uint32_t *>(s_start + R1);          // [2 R1] rows per group = (replica, active / inactive)
  uint32_t *s_bkt = s_cnt + 2 * R1;                                      // [T]    replica bucket | 0x8000 if active | arrival rank in the group << 16
  uint16_t *s_base = reinterpret_cast<uint16_t *>(s_bkt + T);            // [2 R1] first slot of each group in slab_idx order
  uint16_t *s_offact = s_base + 2 * R1;                                  // [R1]   first slot of the replica's records in slab_rec
  uint16_t *s_perm = s_offact + R1;                                      // [T+8]  local index of the row in each slot, groups in arrival order
  uint16_t *s_fin = s_perm + T + 8;                                      // [T+8]  the same with every group in row order
  uint8_t *s_mode = reinterpret_cast<uint8_t *>(s_fin + T + 8);          // [R1]
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  __shared__ uint32_t s_warp[32];
  const int tid = threadIdx.x;

  // the dependent kernel may be scheduled as soon as SMs free up; it waits for this whole grid before it reads
  cudaTriggerProgrammaticLaunchCompletion();

  const int64_t lo = (int64_t)blockIdx.x * T;
  const int64_t hi = lo + T < a.n ? lo + T : a.n;
  const int nt = hi > lo ? (int)(hi - lo) : 0;
  // The tile's column ranges are asked into L2 right away, one bulk prefetch per column (the tile starts on a
  // multiple of 16 rows and the columns are 16-byte aligned; a ragged end is rounded down): DRAM then streams
  // at its own pace while the block sets up and works through the rows.
  if (tid < 9 && nt >= 16) {
    const void *col; uint32_t esz;
    switch (tid) {
      case 0: col = a.replica_id; esz = 4; break;
      case 1: col = a.arrival; esz = 8; break;
      case 2: col = a.first_token; esz = 8; break;
      case 3: col = a.prompt_len; esz = 4; break;
      case 4: col = a.gen; esz = 4; break;
      case 5: col = a.req_id; esz = 4; break;
      case 6: col = a.weight; esz = 4; break;
      case 7: col = a.class_id; esz = 1; break;
      default: col = a.state; esz = 1; break;
    }
    if (col) {
      const uint32_t bytes = ((uint32_t)(nt & ~15)) * esz;
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char *>(col) + lo * esz), "r"(bytes) : "memory");
    }
  }

  stage_classes(p, s_ttft, s_tpot, s_prio);
  for (int i = tid; i < R1; i += blockDim.x) {
    const int64_t nw = i < R ? a.now[i] : 0, mt = i < R ? a.mat[i] : 0;
    s_now[i] = nw; s_start[i] = nw > mt ? nw : mt;
    s_mode[i] = i < R ? a.mode[i] : 0;
    s_cnt[2 * i] = 0; s_cnt[2 * i + 1] = 0;
  }
  if (blockIdx.x == 0) {      // re-arm what the next step accumulates into
    for (int i = tid; i < R1; i += blockDim.x) a.tot_next[i] = 0ull;
    if (tid == 0) *a.ordered_next = 1u;
  }
  __syncthreads();

  const int nvec = nt >> 2;
  const int64_t v0 = lo >> 2;
  uint32_t bad = 0;
  int sorted = 1, rising = 1;

  // ---- pass 1: every row once -------------------------------------------------------------------
  // returns the row's kind; slack = what the slack output gets; bkt = its bucket
  auto do_row = [&](int il, int32_t rid, uint32_t cls, uint32_t st, int32_t prompt, int32_t gen, int32_t weight,
                    int64_t arrival, int64_t first_token, int64_t &slack, int &bkt, uint64_t &k48, int64_t &pttft) -> uint32_t {
    const uint32_t kind = classify_row(p, rid, cls, st, prompt, gen, arrival, s_now, bad);
    bkt = (uint32_t)rid < (uint32_t)R ? rid : R;
    slack = 0;
    if (EXTRA) { pttft = 0; k48 = dev_key48(PH_INACTIVE, 63, HFX_SLACK_MAX); }
    const bool act = kind <= KIND_QUEUED;
    if (act) {
      const int mode = s_mode[bkt];
      int prio;
      if (p.weight_max > 0) prio = weight >= p.weight_max ? 0 : (weight <= p.weight_max - 62 ? 62 : p.weight_max - weight);
      else prio = s_prio[cls];
      int64_t base = row_base(p, s_ttft[cls], s_tpot[cls], kind, mode, prompt, gen, arrival, first_token);
      if (kind == KIND_QUEUED && mode != HFX_DECODE) {
        // the slack of such a row needs nothing from the running batch: it is final here, and the record carries
        // the row's final key in place of the base
        const int64_t start = s_start[bkt];
        slack = base == BASE_UNBOUNDED ? HFX_SLACK_MAX : base - start;
        base = (int64_t)dev_key48(PH_QUEUED, prio, slack);
        if (EXTRA) {
          k48 = (uint64_t)base;
          pttft = (start - arrival) + dev_Ep_prompt(p, prompt);
        }
      } else if (EXTRA) pttft = first_token - arrival;
      s_rec[il] = make_uint4((uint32_t)(uint64_t)base, (uint32_t)((uint64_t)base >> 32),
                             (uint32_t)prompt | (kind << CREC_KIND_SHIFT) | ((uint32_t)prio << CREC_PRIO_SHIFT),
                             (uint32_t)gen | (cls << CREC_CLS_SHIFT));
    }
    const uint32_t g = 2u * (uint32_t)bkt + (act ? 0u : 1u);
    s_bkt[il] = (uint32_t)bkt | (act ? 0x8000u : 0u) | (atomicAdd(&s_cnt[g], 1u) << 16);
    return kind;
  };

  for (int v = tid; v < nvec; v += blockDim.x) {
    const int64_t gv = v0 + v;
    const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + gv);
    const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + gv);
    const uchar4 st = __ldg(reinterpret_cast<const uchar4 *>(a.state) + gv);
    const int4 pr = __ldg(reinterpret_cast<const int4 *>(a.prompt_len) + gv);
    const int4 ge = __ldg(reinterpret_cast<const int4 *>(a.gen) + gv);
    const int4 id = __ldg(reinterpret_cast<const int4 *>(a.req_id) + gv);
    const longlong2 ar0 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * gv);
    const longlong2 ar1 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * gv + 1);
    const longlong2 ft0 = __ldg(reinterpret_cast<const longlong2 *>(a.first_token) + 2 * gv);
    const longlong2 ft1 = __ldg(reinterpret_cast<const longlong2 *>(a.first_token) + 2 * gv + 1);
    int4 we = make_int4(0, 0, 0, 0);
    if (a.weight) we = __ldg(reinterpret_cast<const int4 *>(a.weight) + gv);
    int64_t sl[4], pt[4];
    uint64_t kk[4];
    int bk[4];
    uint32_t kd[4];
    kd[0] = do_row(4 * v, rid.x, cls.x, st.x, pr.x, ge.x, we.x, ar0.x, ft0.x, sl[0], bk[0], kk[0], pt[0]);
    kd[1] = do_row(4 * v + 1, rid.y, cls.y, st.y, pr.y, ge.y, we.y, ar0.y, ft0.y, sl[1], bk[1], kk[1], pt[1]);
    kd[2] = do_row(4 * v + 2, rid.z, cls.z, st.z, pr.z, ge.z, we.z, ar1.x, ft1.x, sl[2], bk[2], kk[2], pt[2]);
    kd[3] = do_row(4 * v + 3, rid.w, cls.w, st.w, pr.w, ge.w, we.w, ar1.y, ft1.y, sl[3], bk[3], kk[3], pt[3]);
    // per-row outputs in row order
    longlong2 *slp = reinterpret_cast<longlong2 *>(a.slack) + 2 * gv;
    slp[0] = make_longlong2(sl[0], sl[1]); slp[1] = make_longlong2(sl[2], sl[3]);
    reinterpret_cast<uchar4 *>(a.admit)[gv] = make_uchar4(kd[0] == KIND_RUNNING, kd[1] == KIND_RUNNING, kd[2] == KIND_RUNNING, kd[3] == KIND_RUNNING);
    reinterpret_cast<uchar4 *>(a.rowflag)[gv] = make_uchar4(kd[0], kd[1], kd[2], kd[3]);
    if (EXTRA) {
      if (a.pred_ttft) {
        longlong2 *q = reinterpret_cast<longlong2 *>(a.pred_ttft) + 2 * gv;
        q[0] = make_longlong2(pt[0], pt[1]); q[1] = make_longlong2(pt[2], pt[3]);
      }
      if (a.pred_tpot) {
        longlong2 *q = reinterpret_cast<longlong2 *>(a.pred_tpot) + 2 * gv;
        q[0] = make_longlong2(0, 0); q[1] = make_longlong2(0, 0);
      }
      if (a.key) {
        ulonglong2 *kp = reinterpret_cast<ulonglong2 *>(a.key) + 2 * gv;
        kp[0] = make_ulonglong2(((uint64_t)(bk[0] & 0xffff) << 48) | kk[0], ((uint64_t)(bk[1] & 0xffff) << 48) | kk[1]);
        kp[1] = make_ulonglong2(((uint64_t)(bk[2] & 0xffff) << 48) | kk[2], ((uint64_t)(bk[3] & 0xffff) << 48) | kk[3]);
      }
    }
    // sorted by replica inside the tile?  req_id rising along the table (also across tiles)?
    const int64_t nxt = (gv << 2) + 4;
    const int bn = nxt < hi ? bucket_of(__ldg(a.replica_id + nxt), R) : bk[3];
    if (bk[0] > bk[1] || bk[1] > bk[2] || bk[2] > bk[3] || bk[3] > bn) sorted = 0;
    if (!(id.x < id.y && id.y < id.z && id.z < id.w && (nxt >= a.n || id.w < __ldg(a.req_id + nxt)))) rising = 0;
  }
  for (int i = (nvec << 2) + tid; i < nt; i += blockDim.x) {
    const int64_t g = lo + i;
    int64_t sl, pt; uint64_t kk; int bk;
    const uint32_t kd = do_row(i, a.replica_id[g], a.class_id[g], a.state[g], a.prompt_len[g], a.gen[g], a.weight ? a.weight[g] : 0,
                               a.arrival[g], a.first_token[g], sl, bk, kk, pt);
    a.slack[g] = sl;
    a.admit[g] = kd == KIND_RUNNING;
    a.rowflag[g] = (uint8_t)kd;
    if (EXTRA) {
      if (a.pred_ttft) a.pred_ttft[g] = pt;
      if (a.pred_tpot) a.pred_tpot[g] = 0;
      if (a.key) a.key[g] = ((uint64_t)(bk & 0xffff) << 48) | kk;
    }
    if (g + 1 < hi && bk > bucket_of(a.replica_id[g + 1], R)) sorted = 0;
    if (g + 1 < a.n && !(a.req_id[g] < a.req_id[g + 1])) rising = 0;
  }
  if (bad) atomicOr(a.status, bad);
  sorted = __syncthreads_and(sorted);        // also orders the shared-memory writes of pass 1 before pass 2
  rising = __syncthreads_and(rising);
  if (tid == 0 && !rising) *a.ordered = 0u;

  // ---- pass 2: where each group starts inside the slabs; the tile's matrix row; totals -----------
  int big = 0;
  {
    const int per = (R1 + blockDim.x - 1) / blockDim.x;
    const int i0 = tid * per < R1 ? tid * per : R1, i1 = (i0 + per < R1) ? i0 + per : R1;
    uint32_t pack = 0;       // rows | active rows << 16 (each at most T <= 8192: the fields cannot carry into each other)
    for (int i = i0; i < i1; i++) {
      const uint32_t cA = s_cnt[2 * i], cI = s_cnt[2 * i + 1];
      pack += (cA + cI) | (cA << 16);
      if (i < R && (cA > FRONT_GROUP_MAX || cI > FRONT_GROUP_MAX)) big = 1;
    }
    uint32_t run = block_excl_scan(pack, s_warp, nullptr);
    uint2 *mrow = a.M + (size_t)blockIdx.x * R1;
    for (int i = i0; i < i1; i++) {
      const uint32_t cA = s_cnt[2 * i], cI = s_cnt[2 * i + 1];
      const uint32_t off_all = run & 0xffffu, off_act = run >> 16;
      s_base[2 * i] = (uint16_t)off_all; s_base[2 * i + 1] = (uint16_t)(off_all + cA); s_offact[i] = (uint16_t)off_act;
      mrow[i] = make_uint2(off_all | ((cA + cI) << 16), off_act | (cA << 16));
      if (cA + cI) atomicAdd(a.tot + i, (unsigned long long)(cA + cI) | ((unsigned long long)cA << 32));
      run += (cA + cI) | (cA << 16);
    }
  }
  const bool tail_scan = s_cnt[2 * R + 1] > FRONT_TAIL_MAX;    // many rows bound to no replica: ranked by a scan
  const int any_big = __syncthreads_or(big);          // (also publishes s_base / s_offact)
  uint16_t *fin = s_fin;

  // ---- pass 3: the slot of every row -----------------------------------------------------------------
  const int c0 = tid * FRONT_PER < nt ? tid * FRONT_PER : nt, c1 = (c0 + FRONT_PER < nt) ? c0 + FRONT_PER : nt;
  if (sorted) {
    // rows of a replica are contiguous: ranks from positions.  s_perm[il] = active rows before position il.
    uint32_t cnt = 0;
    for (int il = c0; il < c1; il++) cnt += (s_bkt[il] >> 15) & 1u;
    uint32_t run = block_excl_scan(cnt, s_warp, nullptr);
    for (int il = c0; il < c1; il++) { s_perm[il] = (uint16_t)run; run += (s_bkt[il] >> 15) & 1u; }
    __syncthreads();
    for (int il = c0; il < c1; il++) {
      const uint32_t bk = s_bkt[il], b = bk & 0xfffu, act = (bk >> 15) & 1u;
      const uint32_t g0 = s_base[2 * b];
      const uint32_t ra = (uint32_t)s_perm[il] - (uint32_t)s_perm[g0];
      s_fin[act ? g0 + ra : (uint32_t)s_base[2 * b + 1] + ((uint32_t)il - g0 - ra)] = (uint16_t)il;
    }
  } else {
    if (any_big) fin = s_perm;      // the network below works in place
    if (tail_scan) {      // (uniform) rows bound to no replica: slot from the number of such rows before each position
      uint32_t cnt = 0;
      for (int il = c0; il < c1; il++) cnt += (s_bkt[il] & 0xfffu) == (uint32_t)R;
      uint32_t run = block_excl_scan(cnt, s_warp, nullptr);
      const uint32_t tb = s_base[2 * R + 1];
      for (int il = c0; il < c1; il++)
        if ((s_bkt[il] & 0xfffu) == (uint32_t)R) { fin[tb + run] = (uint16_t)il; run++; }
    }
    // every other row: the slot inside its group in arrival order (any order) ...
    for (int il = tid; il < nt; il += blockDim.x) {
      const uint32_t bk = s_bkt[il], b = bk & 0xfffu;
      if (tail_scan && b == (uint32_t)R) continue;
      s_perm[s_base[2 * b + (((bk >> 15) & 1u) ^ 1u)] + (bk >> 16)] = (uint16_t)il;
    }
    __syncthreads();
    const int n_slots = tail_scan ? (int)s_base[2 * R + 1] : nt;      // (the group of unbound rows is the last one)
    if (!any_big) {
      // ... then every group in row order: the place of a row is the number of smaller rows in its group
      for (int j = tid; j < n_slots; j += blockDim.x) {
        const uint32_t il = s_perm[j];
        const uint32_t bk = s_bkt[il];
        const uint32_t g = 2 * (bk & 0xfffu) + (((bk >> 15) & 1u) ^ 1u);
        const uint32_t g0 = s_base[g], g1 = g0 + s_cnt[g];
        uint32_t rank = 0;
        for (uint32_t i = g0; i < g1; i++) rank += s_perm[i] < il ? 1u : 0u;
        s_fin[g0 + rank] = (uint16_t)il;
      }
    } else {
      // large unsorted groups: a sorting network over all slots that only exchanges rows of the same group
      // (groups are contiguous in slot order, so this sorts by (group, local index)); ascending comparators
      // with virtual padding
      int n_pad = 2;
      while (n_pad < n_slots) n_pad <<= 1;
      const int half = n_pad >> 1;
      auto cx = [&](int i, int j) {
        const uint16_t x = s_perm[i], y = s_perm[j];
        if (x > y && (s_bkt[x] & 0xffffu) == (s_bkt[y] & 0xffffu)) { s_perm[i] = y; s_perm[j] = x; }
      };
      for (int k = 2; k <= n_pad; k <<= 1) {
        const int hk = k >> 1;
        for (int t = tid; t < half; t += blockDim.x) {
          const int blk = t / hk, off = t - blk * hk;
          const int i = blk * k + off, j = blk * k + k - 1 - off;
          if (j < n_slots) cx(i, j);
        }
        __syncthreads();
        for (int j = k >> 2; j > 0; j >>= 1) {
          for (int t = tid; t < half; t += blockDim.x) {
            const int i = 2 * t - (t & (j - 1));
            if (i + j < n_slots) cx(i, i + j);
          }
          __syncthreads();
        }
      }
    }
  }
  __syncthreads();

  // ---- pass 4: the slabs ---------------------------------------------------------------------------------
  uint16_t *idx_out = a.slab_idx + lo;
  uint4 *rec_out = a.slab_rec + lo;
  for (int j = tid; j < nt; j += blockDim.x) {
    const uint32_t il = fin[j];
    idx_out[j] = (uint16_t)il;
    const uint32_t bk = s_bkt[il];
    if (bk & 0x8000u) {
      const uint32_t b = bk & 0xfffu;
      rec_out[(uint32_t)s_offact[b] + ((uint32_t)j - (uint32_t)s_base[2 * b])] = s_rec[il];
    }
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// Tile height: about one tile per SM, a multiple of 4 rows, at most 8192 (16-bit local indices) and what
// the block's shared memory holds beside its per-replica arrays.
void hfx_front_shape(const hfx_sched *s, int64_t n, int32_t *tile_rows, int32_t *n_tiles) {
  const int R1 = s->p.n_replicas + 1;
  int64_t t = (n + s->n_sm - 1) / s->n_sm;
  t = (t + 15) & ~INT64_C(15);       // (a multiple of 16 rows: every tile starts on a 16-byte boundary of every column)
  if (t < 1024) t = 1024;
  int64_t cap = ((int64_t)HFX_FRONT_SMEM - (int64_t)front_smem_bytes(R1, 0)) / FRONT_ROW_BYTES;
  cap &= ~INT64_C(15);
  if (cap > 8192) cap = 8192;
  if (t > cap) t = cap;
  *tile_rows = (int32_t)t;
  int64_t k = (n + t - 1) / t;
  if (k < 1) k = 1;
  *n_tiles = (int32_t)k;
}

int hfx_launch_front(hfx_sched *s, const FrontArgs &fa0) {
  FrontArgs fa = fa0;
  hfx_front_shape(s, fa.n, &fa.tile_rows, &fa.n_tiles);
  const int R1 = s->p.n_replicas + 1;
  const uint32_t par = s->tot_parity;
  fa.slab_rec = s->d_slab_rec; fa.slab_idx = s->d_slab_idx; fa.M = s->d_M;
  fa.tot = s->d_tot + (size_t)par * (R1 + 1); fa.tot_next = s->d_tot + (size_t)(par ^ 1u) * (R1 + 1);
  fa.ordered = s->d_flags + 4 + par; fa.ordered_next = s->d_flags + 4 + (par ^ 1u);
  fa.status = s->d_status; fa.rowflag = s->d_rowflag;
  KernelScope ks(s, KSLOT_FRONT);
  if (fa.pred_ttft || fa.pred_tpot || fa.key) k_front<true><<<fa.n_tiles, FRONT_THREADS, front_smem_bytes(R1, fa.tile_rows), s->stream>>>(s->p, fa);
  else k_front<false><<<fa.n_tiles, FRONT_THREADS, front_smem_bytes(R1, fa.tile_rows), s->stream>>>(s->p, fa);
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}

int hfx_front_configure() {
  if (cudaFuncSetAttribute(k_front<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, HFX_FRONT_SMEM) != cudaSuccess ||
      cudaFuncSetAttribute(k_front<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, HFX_FRONT_SMEM) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}
