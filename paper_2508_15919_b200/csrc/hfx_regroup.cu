// Grouping the request table by replica: count, scan, and the one streaming pass that turns every
// row into a 32-byte record inside its replica's range.
//
// Matrix mode (default): the table is cut into tiles; k_count writes one histogram row per tile,
// k_colscan turns the columns into exclusive prefixes, and k_regroup places each row at
//   seg_begin[replica] + (rows of that replica in earlier tiles) + (rank inside the tile, row order)
// which is a stable partition without a single global atomic.
// Atomic mode (very many replicas, so the tile matrix would be too large): global counters and
// global fill cursors; rows land in any order inside a replica's range, which the sort repairs.
#include "hfx_internal.cuh"

#define THREADS_TILE 512
#define GROUP_MAX 64      // largest same-replica group of an unsorted tile that is ranked by scanning

// ------------------------------------------------------------------------------------------------
// k_count: rows per replica of one tile.  Bad replica ids go to bucket R and raise a status bit.
// M != nullptr: M[tile][0..R] = the tile's histogram (plain stores).  M == nullptr: global counters.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS_TILE) k_count(const int32_t *__restrict__ replica_id, int64_t n, int32_t R,
                                                        int32_t tile_rows, uint32_t *__restrict__ M,
                                                        uint32_t *__restrict__ seg_count, uint32_t *__restrict__ status) {
  extern __shared__ uint32_t hist[];
  const int R1 = R + 1;
  const bool use_smem = M != nullptr;
  if (use_smem) {
    for (int i = threadIdx.x; i < R1; i += blockDim.x) hist[i] = 0;
    __syncthreads();
  }
  const int64_t lo = (int64_t)blockIdx.x * tile_rows;
  const int64_t hi = lo + tile_rows < n ? lo + tile_rows : n;
  uint32_t bad = 0;
  const int64_t nvec = hi > lo ? (hi - lo) >> 2 : 0;
  const int4 *rid4 = reinterpret_cast<const int4 *>(replica_id + lo);
  for (int64_t v = threadIdx.x; v < nvec; v += blockDim.x) {
    const int4 r = __ldg(rid4 + v);
    const int rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; k++) {
      int b = rr[k];
      if (b < 0 || b >= R) { b = R; bad = 1; }
      if (use_smem) atomicAdd(&hist[b], 1u); else atomicAdd(&seg_count[b], 1u);
    }
  }
  for (int64_t i = lo + (nvec << 2) + threadIdx.x; i < hi; i += blockDim.x) {
    int b = replica_id[i];
    if (b < 0 || b >= R) { b = R; bad = 1; }
    if (use_smem) atomicAdd(&hist[b], 1u); else atomicAdd(&seg_count[b], 1u);
  }
  if (bad) atomicOr(status, HFX_ST_BAD_REPLICA);
  if (use_smem) {
    __syncthreads();
    uint32_t *row = M + (size_t)blockIdx.x * R1;
    for (int i = threadIdx.x; i < R1; i += blockDim.x) row[i] = hist[i];
  }
}

// ------------------------------------------------------------------------------------------------
// k_colscan: for each replica (column) the exclusive prefix of its counts over the tiles, in place,
// and the column total.  Block = 32 columns x 32 chunks of tiles.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) k_colscan(uint32_t *__restrict__ M, int32_t n_tiles, int32_t R1,
                                                  uint32_t *__restrict__ tot) {
  __shared__ uint32_t part[32][33];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int col = blockIdx.x * 32 + lane;
  const int cb = (n_tiles + 31) / 32;
  const int t0 = w * cb < n_tiles ? w * cb : n_tiles;
  const int t1 = (t0 + cb < n_tiles) ? t0 + cb : n_tiles;
  uint32_t sum = 0;
  if (col < R1)
    for (int t = t0; t < t1; t++) sum += M[(size_t)t * R1 + col];
  part[w][lane] = sum;
  __syncthreads();
  uint32_t pre = 0;
  for (int k = 0; k < w; k++) pre += part[k][lane];
  if (col < R1) {
    uint32_t run = pre;
    for (int t = t0; t < t1; t++) {
      const size_t idx = (size_t)t * R1 + col;
      const uint32_t v = M[idx];
      M[idx] = run;
      run += v;
    }
    if (w == 31) tot[col] = pre + sum;
  }
}

// ------------------------------------------------------------------------------------------------
// k_offsets: exclusive scan of the per-replica totals (one block) -> seg_begin, the user-visible
// seg_off, the fill cursors of the atomic mode, and the step's flags:
// flags[0] = 1 says "records of a replica are in row order and req_id rises with the row index"
// (k_regroup clears it when it finds otherwise); flags[1] = largest segment.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) k_offsets(const uint32_t *__restrict__ tot, int32_t R,
                                                  uint32_t *__restrict__ seg_begin, uint32_t *__restrict__ cursor,
                                                  int32_t *__restrict__ seg_off, uint32_t *__restrict__ flags,
                                                  uint32_t ordered_init) {
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry_s, max_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { carry_s = 0; max_s = 0; }
  __syncthreads();
  const int total = R + 1;  // buckets 0..R
  uint32_t mx = 0;
  for (int base = 0; base < total; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const uint32_t c = i < total ? tot[i] : 0;
    mx = c > mx ? c : mx;
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
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = excl + c;
    __syncthreads();
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const uint32_t x = __shfl_xor_sync(0xffffffffu, mx, o); mx = x > mx ? x : mx; }
  if (lane == 0) atomicMax(&max_s, mx);
  __syncthreads();
  if (threadIdx.x == 0) { seg_begin[total] = carry_s; flags[0] = ordered_init; flags[1] = max_s; }
}

// ------------------------------------------------------------------------------------------------
// Per-row work of the streaming pass: what does not depend on the replica's aggregates (prefill
// model of the prompt, slack base, priority) is evaluated here and packed into the record.
// ------------------------------------------------------------------------------------------------
struct RowIn {
  int32_t rid, prompt, gen, req_id, weight, out_len;
  uint32_t cls, st;
  int64_t arrival, first_token;
};

__device__ __forceinline__ void make_record(const HfxParams &p, const RegroupArgs &a, const int64_t *s_ttft,
                                            const int64_t *s_tpot, const uint8_t *s_prio, int64_t i, const RowIn &in,
                                            HfxRec &r, uint32_t &bad) {
  const int32_t R = p.n_replicas;
  r.req_id = in.req_id; r.row = (int32_t)i; r.prompt = in.prompt; r.gen = in.gen; r.output_len = in.out_len;
  r.cls = (uint8_t)in.cls; r.kind = KIND_DEAD; r.prio = 63; r.pad = 0; r.base = 0;
  int64_t pred_ttft = 0;
  if (in.rid >= 0 && in.rid < R) {   // a bad replica id was flagged by k_count
    bool ok = true;
    if (in.cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
    if (in.prompt < 0 || in.prompt > HFX_MAX_TOKENS || in.gen < 0 || in.gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
    if (ok) {
      const int64_t now = __ldg(a.now + in.rid), mat = __ldg(a.mat + in.rid);
      const int32_t mode = __ldg(&a.cfg[in.rid].mode);
      const int64_t start = now > mat ? now : mat;
      int prio;
      if (p.weight_max > 0) {
        const int64_t w = (int64_t)p.weight_max - in.weight;
        prio = (int)(w < 0 ? 0 : (w > 62 ? 62 : w));
      } else prio = s_prio[in.cls];
      const int64_t ttft = s_ttft[in.cls], tpot = s_tpot[in.cls];
      if (in.st == HFX_RUNNING) {
        r.kind = KIND_RUNNING; r.prio = (uint8_t)prio;
        r.base = tpot > 0 ? in.first_token + ((int64_t)in.gen + 1) * tpot - now : BASE_UNBOUNDED;
        pred_ttft = in.first_token - in.arrival;
      } else if (in.st == HFX_QUEUED) {
        if (in.arrival <= now) {
          r.kind = KIND_QUEUED; r.prio = (uint8_t)prio;
          if (mode == HFX_DECODE) {
            r.base = tpot > 0 ? in.first_token + ((int64_t)in.gen + 1) * tpot - start - p.d2 * ((int64_t)in.prompt + in.gen)
                              : BASE_UNBOUNDED;
            pred_ttft = in.first_token - in.arrival;
          } else {
            pred_ttft = (start - in.arrival) + dev_Ep(p, in.prompt);
            r.base = ttft > 0 ? ttft - pred_ttft : BASE_UNBOUNDED;
          }
        } else {
          r.kind = KIND_FUTURE;
          r.base = in.arrival;
        }
      }
    }
  }
  if (a.pred_ttft) a.pred_ttft[i] = pred_ttft;
}

__device__ __forceinline__ void store_record(HfxRec *rec, uint32_t pos, const HfxRec &r) {
  uint4 *dst = reinterpret_cast<uint4 *>(rec + pos);
  const uint4 *src = reinterpret_cast<const uint4 *>(&r);
  dst[0] = src[0];
  dst[1] = src[1];
}

// rows 4v .. 4v+3 with 16-byte loads
__device__ __forceinline__ void load_rows4(const RegroupArgs &a, int64_t v, RowIn in[4]) {
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
  in[0] = {rid.x, pr.x, ge.x, id.x, we.x, ol.x, cls.x, st.x, ar0.x, ft0.x};
  in[1] = {rid.y, pr.y, ge.y, id.y, we.y, ol.y, cls.y, st.y, ar0.y, ft0.y};
  in[2] = {rid.z, pr.z, ge.z, id.z, we.z, ol.z, cls.z, st.z, ar1.x, ft1.x};
  in[3] = {rid.w, pr.w, ge.w, id.w, we.w, ol.w, cls.w, st.w, ar1.y, ft1.y};
}

__device__ __forceinline__ void load_row1(const RegroupArgs &a, int64_t i, RowIn &in) {
  in = {a.replica_id[i], a.prompt_len[i], a.gen[i], a.req_id[i], a.weight ? a.weight[i] : 0,
        a.output_len ? a.output_len[i] : 0, a.class_id[i], a.state[i], a.arrival[i], a.first_token[i]};
}

__device__ __forceinline__ void stage_classes(const HfxParams &p, int64_t *s_ttft, int64_t *s_tpot, uint8_t *s_prio) {
  for (int c = threadIdx.x; c < HFX_MAX_CLASSES; c += blockDim.x) {
    s_ttft[c] = c < p.n_classes ? p.ttft[c] : 0;
    s_tpot[c] = c < p.n_classes ? p.tpot[c] : 0;
    s_prio[c] = c < p.n_classes ? p.prio[c] : 63;
  }
}

// atomic mode: positions from global fill cursors (any order inside a replica's range)
__global__ void __launch_bounds__(256) k_regroup_atomic(const HfxParams p, const RegroupArgs a, uint32_t *__restrict__ cursor,
                                                        HfxRec *__restrict__ rec, uint32_t *__restrict__ status) {
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  stage_classes(p, s_ttft, s_tpot, s_prio);
  __syncthreads();
  uint32_t bad = 0;
  const int R = p.n_replicas;
  const int64_t n4 = a.n >> 2;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
    RowIn in[4];
    load_rows4(a, v, in);
#pragma unroll
    for (int k = 0; k < 4; k++) {
      HfxRec r;
      make_record(p, a, s_ttft, s_tpot, s_prio, (v << 2) + k, in[k], r, bad);
      const int bucket = (in[k].rid < 0 || in[k].rid >= R) ? R : in[k].rid;
      store_record(rec, atomicAdd(&cursor[bucket], 1u), r);
    }
  }
  if (blockIdx.x == 0) {
    for (int64_t i = (n4 << 2) + threadIdx.x; i < a.n; i += blockDim.x) {
      RowIn in; HfxRec r;
      load_row1(a, i, in);
      make_record(p, a, s_ttft, s_tpot, s_prio, i, in, r, bad);
      const int bucket = (in.rid < 0 || in.rid >= R) ? R : in.rid;
      store_record(rec, atomicAdd(&cursor[bucket], 1u), r);
    }
  }
  if (bad) atomicOr(status, bad);
}

// clamp of a replica id to its bucket (bad ids share bucket R)
__device__ __forceinline__ int bucket_of(int rid, int R) { return (rid < 0 || rid >= R) ? R : rid; }

// matrix mode: tile t writes its rows of replica r at seg_begin[r] + M[t][r] + (rank of the row
// among the tile's rows of r, in row order).  The rank comes from the tile being sorted by replica
// already (grouped tables), or from a small shared-memory counting sort of the tile.
__global__ void __launch_bounds__(THREADS_TILE, 2) k_regroup(const HfxParams p, const RegroupArgs a, int32_t tile_rows,
                                                          const uint32_t *__restrict__ M,
                                                          const uint32_t *__restrict__ seg_begin, HfxRec *__restrict__ rec,
                                                          uint32_t *__restrict__ status, uint32_t *__restrict__ flags) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = p.n_replicas, R1 = R + 1;
  uint32_t *s_cnt = reinterpret_cast<uint32_t *>(smem_raw);           // [R1]   rows of each replica in the tile
  uint32_t *s_off = s_cnt + R1;                                        // [R1+1] exclusive prefix of s_cnt
  uint32_t *s_base = s_off + R1 + 1;                                   // [R1]   global position of the tile's first row of r
  uint16_t *s_stage = reinterpret_cast<uint16_t *>(s_base + R1);       // [tile_rows] tile rows grouped by replica
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_maxcnt;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;

  stage_classes(p, s_ttft, s_tpot, s_prio);
  for (int i = tid; i < R1; i += blockDim.x) s_cnt[i] = 0;
  if (tid == 0) s_maxcnt = 0;
  __syncthreads();

  const int64_t lo = (int64_t)blockIdx.x * tile_rows;
  const int64_t hi = lo + tile_rows < a.n ? lo + tile_rows : a.n;
  const int nt = hi > lo ? (int)(hi - lo) : 0;
  const int nvec = nt >> 2;
  const int4 *rid4 = reinterpret_cast<const int4 *>(a.replica_id + lo);
  const uint32_t *Mrow = M + (size_t)blockIdx.x * R1;

  // ---- A: histogram of the tile; is the tile already sorted by replica? ----------------------------
  int sorted = 1;
  for (int v = tid; v < nvec; v += blockDim.x) {
    const int4 r4 = __ldg(rid4 + v);
    int b[5] = {bucket_of(r4.x, R), bucket_of(r4.y, R), bucket_of(r4.z, R), bucket_of(r4.w, R), 0};
#pragma unroll
    for (int k = 0; k < 4; k++) atomicAdd(&s_cnt[b[k]], 1u);
    const int nxt = 4 * v + 4;
    b[4] = nxt < nt ? bucket_of(__ldg(a.replica_id + lo + nxt), R) : b[3];
    if (b[0] > b[1] || b[1] > b[2] || b[2] > b[3] || b[3] > b[4]) sorted = 0;
  }
  for (int i = (nvec << 2) + tid; i < nt; i += blockDim.x) {
    const int x = bucket_of(a.replica_id[lo + i], R);
    atomicAdd(&s_cnt[x], 1u);
    if (i + 1 < nt && x > bucket_of(a.replica_id[lo + i + 1], R)) sorted = 0;
  }
  sorted = __syncthreads_and(sorted);

  // ---- B: exclusive scan of the histogram; global bases; largest group ---------------------------
  {
    const int per = (R1 + blockDim.x - 1) / blockDim.x;
    const int i0 = tid * per < R1 ? tid * per : R1, i1 = (i0 + per < R1) ? i0 + per : R1;
    uint32_t sum = 0, mx = 0;
    for (int i = i0; i < i1; i++) { const uint32_t c = s_cnt[i]; sum += c; mx = c > mx ? c : mx; }
    uint32_t v = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const uint32_t x = __shfl_xor_sync(0xffffffffu, mx, o); mx = x > mx ? x : mx; }
    if (lane == 31) s_warp[warp] = v;
    if (lane == 0) atomicMax(&s_maxcnt, mx);
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
    for (int i = tid; i < R1; i += blockDim.x) s_base[i] = seg_begin[i] + Mrow[i];
  }
  __syncthreads();
  // how the rank of a row inside its (tile, replica) group is found:
  // 0 by position (tile sorted by replica), 1 by scanning the group, 2 any order (huge groups)
  const int mode = sorted ? 0 : (s_maxcnt <= GROUP_MAX ? 1 : 2);
  if (mode != 0) {
    for (int i = tid; i < R1; i += blockDim.x) s_cnt[i] = 0;
    __syncthreads();
    if (mode == 1) {
      // ---- C: tile rows grouped by replica (counting sort of the local indices) ----------------
      for (int v = tid; v < nvec; v += blockDim.x) {
        const int4 r4 = __ldg(rid4 + v);
        const int b[4] = {bucket_of(r4.x, R), bucket_of(r4.y, R), bucket_of(r4.z, R), bucket_of(r4.w, R)};
#pragma unroll
        for (int k = 0; k < 4; k++) s_stage[s_off[b[k]] + atomicAdd(&s_cnt[b[k]], 1u)] = (uint16_t)(4 * v + k);
      }
      for (int i = (nvec << 2) + tid; i < nt; i += blockDim.x) {
        const int x = bucket_of(a.replica_id[lo + i], R);
        s_stage[s_off[x] + atomicAdd(&s_cnt[x], 1u)] = (uint16_t)i;
      }
      __syncthreads();
    }
  }

  // ---- D: records -----------------------------------------------------------------------------------
  uint32_t bad = 0;
  int ordered = mode != 2;
  auto place = [&](int rid, int il) -> uint32_t {
    const int bkt = bucket_of(rid, R);
    uint32_t rank;
    if (mode == 0) rank = (uint32_t)il - s_off[bkt];
    else if (mode == 1) {
      rank = 0;
      const uint32_t g0 = s_off[bkt], g1 = s_off[bkt + 1];
      for (uint32_t g = g0; g < g1; g++) rank += s_stage[g] < (uint32_t)il ? 1u : 0u;
    } else rank = atomicAdd(&s_cnt[bkt], 1u);
    return s_base[bkt] + rank;
  };
  const int64_t v0 = lo >> 2;
  for (int v = tid; v < nvec; v += blockDim.x) {
    RowIn in[4];
    load_rows4(a, v0 + v, in);
    // req_id must rise with the row index for the order of equal keys to come for free
    const int64_t nxt = lo + 4 * (int64_t)v + 4;
    const bool has_next = nxt < a.n;
    const int32_t id_next = has_next ? __ldg(a.req_id + nxt) : 0;
    if (!(in[0].req_id < in[1].req_id && in[1].req_id < in[2].req_id && in[2].req_id < in[3].req_id &&
          (!has_next || in[3].req_id < id_next))) ordered = 0;
#pragma unroll
    for (int k = 0; k < 4; k++) {
      HfxRec r;
      make_record(p, a, s_ttft, s_tpot, s_prio, lo + 4 * (int64_t)v + k, in[k], r, bad);
      store_record(rec, place(in[k].rid, 4 * v + k), r);
    }
  }
  for (int i = (nvec << 2) + tid; i < nt; i += blockDim.x) {
    RowIn in; HfxRec r;
    load_row1(a, lo + i, in);
    if (lo + i + 1 < a.n && !(in.req_id < a.req_id[lo + i + 1])) ordered = 0;
    make_record(p, a, s_ttft, s_tpot, s_prio, lo + i, in, r, bad);
    store_record(rec, place(in.rid, i), r);
  }
  if (bad) atomicOr(status, bad);
  if (!ordered) flags[0] = 0;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
int hfx_launch_regroup(hfx_sched *s, const RegroupArgs &ra, int32_t *seg_off) {
  const int R = s->p.n_replicas, R1 = R + 1;
  const int64_t n = ra.n;
  cudaStream_t stream = s->stream;
  int32_t tile_rows, n_tiles;
  hfx_tile_shape(n, &tile_rows, &n_tiles);
  const bool matrix = s->d_tile_hist != nullptr && n_tiles <= s->tile_blocks_max;
  if (matrix) {
    {
      KernelScope ks(s, KSLOT_COUNT);
      k_count<<<n_tiles, THREADS_TILE, sizeof(uint32_t) * R1, stream>>>(ra.replica_id, n, R, tile_rows, s->d_tile_hist,
                                                                          nullptr, s->d_status);
    }
    {
      KernelScope ks(s, KSLOT_COLSCAN);
      k_colscan<<<(R1 + 31) / 32, 1024, 0, stream>>>(s->d_tile_hist, n_tiles, R1, s->d_seg_count);
    }
    {
      KernelScope ks(s, KSLOT_OFFSETS);
      k_offsets<<<1, 1024, 0, stream>>>(s->d_seg_count, R, s->d_seg_begin, s->d_cursor, seg_off, s->d_flags, 1u);
    }
    {
      KernelScope ks(s, KSLOT_REGROUP);
      const size_t sm = sizeof(uint32_t) * (3 * (size_t)R1 + 1) + sizeof(uint16_t) * (size_t)tile_rows + 16;
      k_regroup<<<n_tiles, THREADS_TILE, sm, stream>>>(s->p, ra, tile_rows, s->d_tile_hist, s->d_seg_begin, s->d_rec,
                                                        s->d_status, s->d_flags);
    }
  } else {
    if (cudaMemsetAsync(s->d_seg_count, 0, sizeof(uint32_t) * (R + 2), stream) != cudaSuccess) return HFX_E_CUDA;
    {
      KernelScope ks(s, KSLOT_COUNT);
      k_count<<<n_tiles, THREADS_TILE, 0, stream>>>(ra.replica_id, n, R, tile_rows, nullptr, s->d_seg_count, s->d_status);
    }
    {
      KernelScope ks(s, KSLOT_OFFSETS);
      k_offsets<<<1, 1024, 0, stream>>>(s->d_seg_count, R, s->d_seg_begin, s->d_cursor, seg_off, s->d_flags, 0u);
    }
    {
      KernelScope ks(s, KSLOT_REGROUP);
      k_regroup_atomic<<<s->n_sm * 8, 256, 0, stream>>>(s->p, ra, s->d_cursor, s->d_rec, s->d_status);
    }
  }
  return HFX_OK;
}

int hfx_regroup_configure() {
  if (cudaFuncSetAttribute(k_regroup, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}
