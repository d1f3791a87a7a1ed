// hfx_dispatch_step: the four dispatching steps of Sec. 3.3.1 over a shared global queue, for every
// colocated or P-stage instance whose maturity time has come, in maturity order; then, on a scheduler with
// D-stage instances, the same steps once more for the D stage (the Migrator): the queue of prefilled
// requests, the D instances in maturity order, budgets and costs in time.  One scan of the table finds both
// queues; the kernels from the compaction on run once per stage (stage 0, then stage 1 on the same buffers).
//
//   k_disp_scan     one streaming pass over the table: the running batch of every instance (count,
//                   context tokens, classes), slack and priority key of the visible queue's rows
//   k_disp_compact  the queue's rows in row order as (sort word, row) pairs
//   radix passes    the queue ordered by (priority, slack, request id): a stable least-significant-
//                   digit radix sort, 8 bits a pass, on the 48-bit key; before that on the request id,
//                   unless the ids rise with the rows (then row order already is id order)
//   k_disp_plan     E_d and the safe token budget (Eq. 3) of every instance; the largest budget
//   k_disp_prefix   the queue's rows in order, and the running totals (tokens, entries) of those that
//                   fit some instance; larger entries are passed over
//   k_disp_chain    matured instances sorted by (maturity, index); one warp hands consecutive runs of
//                   the queue to them, each run found by a probe of the next 32 entries of the running totals
//                   (a search for the longer ones) and only noted; all threads then write what each took
//   k_disp_assign   the request -> instance binding of every dispatched row, the new maturity times
#include <new>
#include <string.h>

#include "hfx_internal.cuh"

#define DISP_THREADS 256
#define RADIX_ITEMS 8                               // items a thread holds in the scatter pass
#define RADIX_TILE (DISP_THREADS * RADIX_ITEMS)     // 2048
#define DISP_MAX_INSTANCES 4096                     // instances the chain kernel orders in shared memory
#define DISP_SCAN_BLOCKS_MAX 4096                   // blocks of the scan / compaction pair

struct DispWork {
  // queue, ping-pong
  uint64_t *key[2]; uint32_t *val[2];
  uint64_t *rowkey;          // [rows] the 48-bit key of a queue row, by row
  int64_t *prefix;           // [rows] running total of prompt lengths along the queue (entries that fit some instance)
  int32_t *prefix_cnt;       // [rows] running count of those entries
  uint32_t *hist;            // [tiles][256] digit counts of the current pass
  int64_t *tile_sum;         // [2][tiles] totals of the prefix pass: tokens, entries
  uint32_t *n_run;           // [R]
  unsigned long long *sum_kv;    // [R]
  unsigned long long *mask_run;  // [R]
  unsigned long long *ctl;   // per stage, 8 words each: [0] classes present in the queue  [1] queue length  [2], [3] last-block
                             // counters  [4] largest budget among the matured instances;  [5] (first stage's only) request
                             // ids do not rise with the rows
  uint32_t *blk_cnt;         // [2][DISP_SCAN_BLOCKS_MAX] queue rows of each stage found by each block of the scan
  ReplicaPlan *plan;         // [R]
  int32_t *run_start;        // [R] where an instance's run starts in the queue
  int32_t *run_len;          // [R] queue positions the run covers (passed-over entries included)
  int64_t max_rows; int32_t R;
};

struct DispArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len; const int32_t *gen;
  const int64_t *arrival; const int32_t *req_id; const int32_t *weight; const int64_t *first_token;
  int64_t n; int64_t now; int32_t cap_max;
  int32_t d_stage;           // the scheduler has D-stage instances: the Migrator's stage runs too
  const int64_t *maturity; const hfx_replica_cfg *cfg; const uint8_t *mode;
  // outputs
  int32_t *assign; int32_t *queue_order; int32_t *n_queue; int32_t *inst_order; int32_t *n_mature; int64_t *slack;
  int64_t *budget; int64_t *e_d; int32_t *n_run; int64_t *sum_kv; int64_t *adm_cost; int32_t *adm_count; int64_t *maturity_next;
  uint32_t *status;
};

#define DQ_TAG (UINT64_C(1) << 63)      // on a row's key: the row belongs to the queue of prefilled requests
#define KEY48 ((UINT64_C(1) << 48) - 1)

// what a queue entry takes of an instance's budget: prompt tokens (first stage), decode time d1 + d2 kv (D stage)
struct DispCost {
  const int32_t *prompt_len, *gen; int64_t d1, d2; int32_t stage;
  __device__ __forceinline__ int64_t of(uint32_t row) const {
    const int64_t x = prompt_len[row];
    return stage ? d1 + d2 * (x + gen[row]) : x;
  }
};

// rows per block of the scan / compaction pair: equal contiguous runs, whole warps
__host__ __device__ inline int64_t disp_chunk(int64_t n, int blocks) {
  int64_t c = (n + blocks - 1) / blocks;
  return (c + 31) & ~INT64_C(31);
}

// ------------------------------------------------------------------------------------------------
// k_disp_scan
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DISP_THREADS) k_disp_scan(const HfxParams p, const DispArgs a, const DispWork w) {
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES], s_tpot[HFX_MAX_CLASSES];
  __shared__ uint8_t s_prio[HFX_MAX_CLASSES];
  for (int c = threadIdx.x; c < HFX_MAX_CLASSES; c += blockDim.x) {
    s_ttft[c] = c < p.n_classes ? p.ttft[c] : 0;
    s_tpot[c] = c < p.n_classes ? p.tpot[c] : 0;
    s_prio[c] = c < p.n_classes ? p.prio[c] : 63;
  }
  __syncthreads();
  const int lane = threadIdx.x & 31;
  uint32_t bad = 0;
  unsigned long long qmask = 0, dmask = 0;
  __shared__ uint32_t s_count, s_dcount;
  if (threadIdx.x == 0) { s_count = 0; s_dcount = 0; }
  __syncthreads();
  // every block takes a contiguous run of rows, so that the compaction that follows keeps row order
  const int64_t chunk = disp_chunk(a.n, gridDim.x);
  const int64_t lo = (int64_t)blockIdx.x * chunk, hi = lo + chunk < a.n ? lo + chunk : a.n;
  uint32_t mine = 0, dmine = 0;
  bool falls = false;
  for (int64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    bool in_queue = false;
    uint64_t k48 = 0;
    {
      const uint32_t cls = a.class_id[i], st = a.state[i];
      const int32_t prompt = a.prompt_len[i], gen = a.gen[i];
      bool ok = true;
      if (cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
      if (prompt < 0 || prompt > HFX_MAX_TOKENS || gen < 0 || gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
      int64_t slack = 0;
      if (ok && st == HFX_RUNNING) {
        const int32_t r = a.replica_id[i];
        if (r < 0 || r >= p.n_replicas) bad |= HFX_ST_BAD_REPLICA;
        else {
          atomicAdd(&w.n_run[r], 1u);
          atomicAdd(&w.sum_kv[r], (unsigned long long)((int64_t)prompt + gen));
          atomicOr(&w.mask_run[r], 1ull << cls);
          // a prefilled request: in flight on a P-stage instance, its first token produced by now
          if (a.d_stage && a.mode[r] == HFX_PREFILL) {
            const int64_t ft = a.first_token[i];
            if (ft <= a.now) {
              const int64_t tpot = s_tpot[cls];
              slack = tpot > 0 ? ft + ((int64_t)gen + 1) * tpot - a.now - dev_Ed(p, 1, (int64_t)prompt + gen) : HFX_SLACK_MAX;
              int prio;
              if (p.weight_max > 0) {
                const int64_t x = (int64_t)p.weight_max - a.weight[i];
                prio = (int)(x < 0 ? 0 : (x > 62 ? 62 : x));
              } else prio = s_prio[cls];
              k48 = dev_key48(PH_QUEUED, prio, slack) | DQ_TAG;
              dmask |= 1ull << cls;
              dmine += 1u;
            }
          }
        }
      } else if (ok && st == HFX_QUEUED && a.arrival[i] <= a.now && prompt <= a.cap_max) {
        const int64_t ttft = s_ttft[cls];
        slack = ttft > 0 ? ttft - ((a.now - a.arrival[i]) + dev_Ep(p, prompt)) : HFX_SLACK_MAX;
        int prio;
        if (p.weight_max > 0) {
          const int64_t x = (int64_t)p.weight_max - a.weight[i];
          prio = (int)(x < 0 ? 0 : (x > 62 ? 62 : x));
        } else prio = s_prio[cls];
        k48 = dev_key48(PH_QUEUED, prio, slack);           // never 0: the phase bits are set
        qmask |= 1ull << cls;
        in_queue = true;
      }
      a.slack[i] = slack;
      a.assign[i] = -1;
      a.queue_order[i] = -1;
      w.rowkey[i] = k48;
      mine += in_queue ? 1u : 0u;
      if (i + 1 < a.n && !(a.req_id[i] < a.req_id[i + 1])) falls = true;
    }
  }
  qmask = warp_or_u64(qmask);
  if (lane == 0 && qmask) atomicOr(&w.ctl[0], qmask);
  if (a.d_stage) {
    dmask = warp_or_u64(dmask);
    if (lane == 0 && dmask) atomicOr(&w.ctl[8], dmask);
    dmine = (uint32_t)warp_sum_i64(dmine);
    if (lane == 0 && dmine) atomicAdd(&s_dcount, dmine);
  }
  if (bad) atomicOr(a.status, bad);
  if (falls) atomicExch(&w.ctl[5], 1ull);
  mine = (uint32_t)warp_sum_i64(mine);
  if (lane == 0 && mine) atomicAdd(&s_count, mine);
  __syncthreads();
  if (threadIdx.x == 0) { w.blk_cnt[blockIdx.x] = s_count; w.blk_cnt[DISP_SCAN_BLOCKS_MAX + blockIdx.x] = s_dcount; }
}

// k_disp_compact: the queue rows in row order, as (sort word, row) pairs.  A block starts where the blocks
// before it end (it adds up their counts) and places its own rows by a block-wide prefix of the "in the
// queue" flags.  When the request ids rise with the rows the pairs carry the 48-bit key at once (row
// order is id order, and the radix passes keep it among equal keys); otherwise they carry the request id,
// which is ordered first.
__global__ void __launch_bounds__(DISP_THREADS) k_disp_compact(const DispArgs a, const DispWork w, const int stage) {
  __shared__ uint32_t s_warp[DISP_THREADS / 32];
  __shared__ unsigned long long s_base;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_base = 0;
  __syncthreads();
  {
    unsigned long long part = 0;
    for (int bb = threadIdx.x; bb < (int)blockIdx.x; bb += blockDim.x) part += w.blk_cnt[stage * DISP_SCAN_BLOCKS_MAX + bb];
    part = (unsigned long long)warp_sum_i64((int64_t)part);
    if (lane == 0 && part) atomicAdd(&s_base, part);
  }
  __syncthreads();
  unsigned long long run = s_base;
  const bool by_id = w.ctl[5] != 0;
  const int64_t chunk = disp_chunk(a.n, gridDim.x);
  const int64_t lo = (int64_t)blockIdx.x * chunk, hi = lo + chunk < a.n ? lo + chunk : a.n;
  for (int64_t i0 = lo; i0 < hi; i0 += blockDim.x) {
    const int64_t i = i0 + threadIdx.x;
    uint64_t k48 = i < hi ? w.rowkey[i] : 0;
    k48 = (k48 != 0 && (int)(k48 >> 63) == stage) ? (k48 & KEY48) : 0;      // this stage's queue only
    const uint32_t m = __ballot_sync(0xffffffffu, k48 != 0);
    if (lane == 0) s_warp[warp] = __popc(m);
    __syncthreads();
    uint32_t before = 0, all = 0;
    for (int k = 0; k < DISP_THREADS / 32; k++) { const uint32_t c = s_warp[k]; if (k < warp) before += c; all += c; }
    if (k48 != 0) {
      const unsigned long long pos = run + before + __popc(m & ((1u << lane) - 1u));
      w.key[0][pos] = by_id ? (uint64_t)((uint32_t)a.req_id[i] ^ 0x80000000u) : k48;      // signed id order as unsigned
      w.val[0][pos] = (uint32_t)i;
    }
    run += all;
    __syncthreads();
  }
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) w.ctl[8 * stage + 1] = run;      // the queue's length
}

// ------------------------------------------------------------------------------------------------
// Radix sort pass, 8 bits.  k_radix_hist counts the digits of every tile (hist[tile][digit]).
// k_radix_scatter first works out where its tile's items of each digit go -- thread d adds up digit
// d's counts over all tiles (coalesced rows of the histogram), the part from earlier tiles and the
// total, and a block scan of the totals gives the digit's start -- then orders the tile by the
// digit (stable one-bit splits of packed (digit, position) words in shared memory) and writes the
// items out.  The item count lives on the device (ctl[1]); tiles beyond it leave at once.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DISP_THREADS) k_radix_hist(const uint64_t *__restrict__ keys, const unsigned long long *ctl_n,
                                                             int shift, uint32_t *__restrict__ hist,
                                                             const unsigned long long *only_if) {
  __shared__ uint32_t s_h[256];
  if (only_if && *only_if == 0) return;      // a pass on the request id, and the ids already rise with the rows
  const int64_t n = (int64_t)*ctl_n;
  const int32_t tiles = (int32_t)((n + RADIX_TILE - 1) / RADIX_TILE);
  const int tile = blockIdx.x;
  if (tile >= tiles) return;
  s_h[threadIdx.x] = 0;
  __syncthreads();
  const int64_t lo = (int64_t)tile * RADIX_TILE;
  const int64_t hi = lo + RADIX_TILE < n ? lo + RADIX_TILE : n;
  for (int64_t j = lo + threadIdx.x; j < hi; j += DISP_THREADS) atomicAdd(&s_h[(uint32_t)(keys[j] >> shift) & 255u], 1u);
  __syncthreads();
  hist[(size_t)tile * 256 + threadIdx.x] = s_h[threadIdx.x];
}

__global__ void __launch_bounds__(DISP_THREADS) k_radix_scatter(const uint64_t *__restrict__ keys_in, const uint32_t *__restrict__ vals_in,
                                                                uint64_t *__restrict__ keys_out, uint32_t *__restrict__ vals_out,
                                                                const unsigned long long *ctl_n, int shift,
                                                                const uint32_t *__restrict__ hist, const unsigned long long *only_if) {
  __shared__ uint64_t s_key[RADIX_TILE];
  if (only_if && *only_if == 0) return;
  __shared__ uint32_t s_base[256];               // where the tile's items of each digit go
  __shared__ uint32_t s_val[RADIX_TILE];
  __shared__ uint32_t s_item[2][RADIX_TILE];     // digit << 16 | position in the tile
  __shared__ uint32_t s_start[257];              // where each digit starts in the ordered tile
  __shared__ uint32_t s_warp[32];
  const int64_t n = (int64_t)*ctl_n;
  const int32_t tiles = (int32_t)((n + RADIX_TILE - 1) / RADIX_TILE);
  const int tile = blockIdx.x;
  if (tile >= tiles) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t lo = (int64_t)tile * RADIX_TILE;
  const int nt = (int)((lo + RADIX_TILE < n ? lo + RADIX_TILE : n) - lo);
  {   // digit threadIdx.x: items in earlier tiles, items in all tiles; exclusive scan of the totals over the digits
    uint32_t before = 0, total = 0;
    const uint32_t *col = hist + threadIdx.x;
    int t = 0;
    for (; t + 8 <= tiles; t += 8) {
      uint32_t x[8];
#pragma unroll
      for (int k = 0; k < 8; k++) x[k] = col[(size_t)(t + k) * 256];
#pragma unroll
      for (int k = 0; k < 8; k++) { total += x[k]; if (t + k < tile) before += x[k]; }
    }
    for (; t < tiles; t++) { const uint32_t x = col[(size_t)t * 256]; total += x; if (t < tile) before += x; }
    uint32_t inc = total;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += y; }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t start = inc - total;
    for (int k = 0; k < warp; k++) start += s_warp[k];
    s_base[threadIdx.x] = start + before;
    __syncthreads();
  }
  for (int q = threadIdx.x; q < RADIX_TILE; q += DISP_THREADS) {
    uint32_t item = (256u << 16) | (uint32_t)q;           // padding sorts behind every digit
    if (q < nt) {
      const uint64_t k = keys_in[lo + q];
      s_key[q] = k; s_val[q] = vals_in[lo + q];
      item = (((uint32_t)(k >> shift) & 255u) << 16) | (uint32_t)q;
    }
    s_item[0][q] = item;
  }
  __syncthreads();
  int src = 0;
  for (int bit = 16; bit < 25; bit++) {                    // 8 digit bits and the padding bit
    uint32_t it[RADIX_ITEMS];
    uint32_t zeros = 0;
#pragma unroll
    for (int k = 0; k < RADIX_ITEMS; k++) { it[k] = s_item[src][threadIdx.x * RADIX_ITEMS + k]; zeros += ((it[k] >> bit) & 1u) ^ 1u; }
    uint32_t inc = zeros;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += x; }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t zbase = inc - zeros, ztotal = 0;
    for (int k = 0; k < DISP_THREADS / 32; k++) { const uint32_t x = s_warp[k]; if (k < warp) zbase += x; ztotal += x; }
    uint32_t obase = ztotal + (uint32_t)threadIdx.x * RADIX_ITEMS - zbase;
#pragma unroll
    for (int k = 0; k < RADIX_ITEMS; k++) {
      if ((it[k] >> bit) & 1u) s_item[src ^ 1][obase++] = it[k];
      else s_item[src ^ 1][zbase++] = it[k];
    }
    src ^= 1;
    __syncthreads();
  }
  // digit starts inside the ordered tile: first position of each digit
  for (int d = threadIdx.x; d <= 256; d += DISP_THREADS) s_start[d] = (uint32_t)nt;
  __syncthreads();
  for (int q = threadIdx.x; q < nt; q += DISP_THREADS) {
    const uint32_t d = s_item[src][q] >> 16;
    if (q == 0 || (s_item[src][q - 1] >> 16) != d) s_start[d] = (uint32_t)q;
  }
  __syncthreads();
  for (int q = threadIdx.x; q < nt; q += DISP_THREADS) {
    const uint32_t item = s_item[src][q];
    const uint32_t d = item >> 16, from = item & 0xffffu;
    const uint32_t pos = s_base[d] + ((uint32_t)q - s_start[d]);
    keys_out[pos] = s_key[from];
    vals_out[pos] = s_val[from];
  }
}

// after the request-id passes: the 48-bit key of every queue entry, in the order reached so far
__global__ void __launch_bounds__(DISP_THREADS) k_disp_gather(uint64_t *__restrict__ keys, const uint32_t *__restrict__ vals,
                                                              const uint64_t *__restrict__ rowkey, const unsigned long long *ctl_n,
                                                              const unsigned long long *only_if) {
  if (*only_if == 0) return;
  const int64_t n = (int64_t)*ctl_n;
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += (int64_t)gridDim.x * blockDim.x)
    keys[j] = rowkey[vals[j]] & KEY48;
}

// ------------------------------------------------------------------------------------------------
// Running total of prompt lengths along the ordered queue: per-tile totals, the last block scans
// them; then every tile scans its own items on top of its offset and lists the queue's rows.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DISP_THREADS) k_disp_tilesum(const uint32_t *__restrict__ vals, const DispCost cost,
                                                               const unsigned long long *ctl, int64_t *__restrict__ tile_sum,
                                                               int32_t tiles_max, unsigned long long *done) {
  __shared__ int64_t s_red[32], s_redc[32];
  __shared__ uint32_t s_last;
  const int64_t n = (int64_t)ctl[1];
  const int64_t bmax = (int64_t)ctl[4];
  const int32_t tiles = (int32_t)((n + RADIX_TILE - 1) / RADIX_TILE);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if ((int)blockIdx.x < tiles) {
    const int64_t lo = (int64_t)blockIdx.x * RADIX_TILE;
    const int64_t hi = lo + RADIX_TILE < n ? lo + RADIX_TILE : n;
    int64_t s = 0, c = 0;
    for (int64_t j = lo + threadIdx.x; j < hi; j += DISP_THREADS) { const int64_t x = cost.of(vals[j]); if (x <= bmax) { s += x; c += 1; } }
    s = warp_sum_i64(s); c = warp_sum_i64(c);
    if (lane == 0) { s_red[warp] = s; s_redc[warp] = c; }
    __syncthreads();
    if (threadIdx.x == 0) {
      int64_t t = 0, u = 0;
      for (int k = 0; k < DISP_THREADS / 32; k++) { t += s_red[k]; u += s_redc[k]; }
      tile_sum[blockIdx.x] = t;
      tile_sum[tiles_max + blockIdx.x] = u;
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(done, 1ull) == (unsigned long long)gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // exclusive scan of the tile totals, DISP_THREADS tiles at a time with a carry
  __shared__ int64_t s_carry[2];
  if (threadIdx.x == 0) { s_carry[0] = 0; s_carry[1] = 0; *done = 0; }
  __syncthreads();
  for (int32_t t0 = 0; t0 < tiles; t0 += DISP_THREADS) {
    const int32_t t = t0 + threadIdx.x;
    const int64_t x = t < tiles ? __ldcg(tile_sum + t) : 0, y = t < tiles ? __ldcg(tile_sum + tiles_max + t) : 0;
    const int64_t ix = warp_incl_scan_i64(x, lane), iy = warp_incl_scan_i64(y, lane);
    if (lane == 31) { s_red[warp] = ix; s_redc[warp] = iy; }
    __syncthreads();
    int64_t rx = s_carry[0] + ix - x, ry = s_carry[1] + iy - y;
    for (int k = 0; k < warp; k++) { rx += s_red[k]; ry += s_redc[k]; }
    if (t < tiles) { tile_sum[t] = rx; tile_sum[tiles_max + t] = ry; }
    __syncthreads();
    if (threadIdx.x == DISP_THREADS - 1) { s_carry[0] = rx + x; s_carry[1] = ry + y; }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(DISP_THREADS) k_disp_prefix(const uint32_t *__restrict__ vals, const DispCost cost,
                                                              const unsigned long long *ctl, const int64_t *__restrict__ tile_sum,
                                                              int32_t tiles_max, int64_t *__restrict__ prefix,
                                                              int32_t *__restrict__ prefix_cnt, int32_t *__restrict__ queue_order,
                                                              int32_t *__restrict__ n_queue, const unsigned long long *listed_before) {
  __shared__ int64_t s_warp[32];
  __shared__ int32_t s_warpc[32];
  const int64_t n = (int64_t)ctl[1];
  const int64_t bmax = (int64_t)ctl[4];
  const int32_t tiles = (int32_t)((n + RADIX_TILE - 1) / RADIX_TILE);
  if (blockIdx.x == 0 && threadIdx.x == 0) *n_queue = (int32_t)n;
  if ((int)blockIdx.x >= tiles) return;
  const int64_t q0 = listed_before ? (int64_t)*listed_before : 0;      // the D stage's queue is listed behind the first stage's
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t lo = (int64_t)blockIdx.x * RADIX_TILE + (int64_t)threadIdx.x * RADIX_ITEMS;
  int64_t c[RADIX_ITEMS], sum = 0;
  int32_t e[RADIX_ITEMS], cnt = 0;
#pragma unroll
  for (int k = 0; k < RADIX_ITEMS; k++) {
    c[k] = 0; e[k] = 0;
    if (lo + k < n) {
      const uint32_t row = vals[lo + k];
      const int64_t x = cost.of(row);
      if (x <= bmax) { c[k] = x; e[k] = 1; }      // larger than every budget of this call: passed over
      queue_order[q0 + lo + k] = (int32_t)row;
    }
    sum += c[k]; cnt += e[k];
  }
  const int64_t inc = warp_incl_scan_i64(sum, lane);
  const int32_t incc = warp_incl_scan_i32(cnt, lane);
  if (lane == 31) { s_warp[warp] = inc; s_warpc[warp] = incc; }
  __syncthreads();
  int64_t run = tile_sum[blockIdx.x] + inc - sum;
  int32_t runc = (int32_t)tile_sum[tiles_max + blockIdx.x] + incc - cnt;
  for (int k = 0; k < warp; k++) { run += s_warp[k]; runc += s_warpc[k]; }
#pragma unroll
  for (int k = 0; k < RADIX_ITEMS; k++) {     // inclusive
    run += c[k]; runc += e[k];
    if (lo + k < n) { prefix[lo + k] = run; prefix_cnt[lo + k] = runc; }
  }
}

// ------------------------------------------------------------------------------------------------
// k_disp_plan: dispatching step 2 for every instance (E_d of its running batch, the safe budget from
// the strictest TTFT in the queue and the strictest TPOT in flight); resets the per-instance results.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DISP_THREADS) k_disp_plan(const HfxParams p, const DispArgs a, const DispWork w, const int stage) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.n_replicas) return;
  ReplicaPlan pl;
  if (stage) {     // the D stage: the time budget of a DECODE instance, from its batch or the queue of prefilled requests
    if (a.cfg[r].mode != HFX_DECODE) return;
    dev_plan(p, a.cfg[r], a.now, a.maturity[r], (int64_t)w.n_run[r], (int64_t)w.sum_kv[r], w.mask_run[r], w.ctl[8], pl);
    w.plan[r] = pl;
    a.budget[r] = pl.budget;
    if (pl.now >= pl.mat && pl.budget > 0) atomicMax(&w.ctl[8 + 4], (unsigned long long)pl.budget);
    return;
  }
  if (r == 0) { a.n_queue[1] = 0; a.n_mature[1] = 0; }
  dev_plan(p, a.cfg[r], a.now, a.maturity[r], (int64_t)w.n_run[r], (int64_t)w.sum_kv[r], w.mask_run[r], w.ctl[0], pl);
  if (pl.mode == HFX_DECODE) pl.budget = 0;      // a D-stage instance takes nothing from this queue
  w.plan[r] = pl;
  a.budget[r] = pl.budget;
  a.e_d[r] = pl.e_d;
  a.n_run[r] = (int32_t)pl.n_run;
  a.sum_kv[r] = pl.sum_kv;
  a.adm_cost[r] = 0;
  a.adm_count[r] = 0;
  a.maturity_next[r] = pl.mat;
  a.inst_order[r] = -1;
  w.run_start[r] = 0;
  w.run_len[r] = 0;
  if (pl.now >= pl.mat && pl.budget > 0) atomicMax(&w.ctl[4], (unsigned long long)pl.budget);
}

// ------------------------------------------------------------------------------------------------
// k_disp_chain: one block.  Dispatching step 1: the matured instances ordered by (maturity, index)
// in shared memory.  Step 3: the first warp walks them; each takes the longest stretch of the queue,
// from where the previous one stopped, whose entries stay within its budget and batch room (a
// gallop and a 32-way search on the running totals).  The totals are read through a window in
// shared memory that the whole block refills from the current position whenever a search reaches
// its end; a run longer than the window finishes its search in global memory.
// ------------------------------------------------------------------------------------------------
#define CHAIN_WINDOW 2048

// longest m in [lo0, hi0] with fits(m), given fits(lo0) (or lo0 = 0) and fits monotone; whole warp
template <typename F>
__device__ __forceinline__ int64_t warp_longest(int64_t lo0, const int64_t hi0, int lane, F fits) {
  {   // short stretches first: lane l tries lo0 + l + 1
    const int64_t m = lo0 + lane + 1;
    const int f = __popc(__ballot_sync(0xffffffffu, m <= hi0 && fits(m)));      // the lanes that fit are a prefix
    if (f < 32) return lo0 + f;
    lo0 += 32;
  }
  int64_t lo = lo0, hi = hi0;
  {   // gallop: lane l tries lo0 + 2^l
    const int64_t m = lo0 + (INT64_C(1) << lane);
    const bool ok = m <= hi0 && fits(m);
    const int f = __popc(__ballot_sync(0xffffffffu, ok));      // the lanes that fit are a prefix
    if (f > 0) lo = lo0 + (INT64_C(1) << (f - 1));
    if (f < 32) { const int64_t t = lo0 + (INT64_C(1) << f) - 1; hi = t < hi ? t : hi; }
  }
  while (lo < hi) {
    const int64_t step = (hi - lo + 31) / 32;
    const int64_t cand = lo + (int64_t)(lane + 1) * step;
    const bool ok = cand <= hi && fits(cand);
    const int f = __popc(__ballot_sync(0xffffffffu, ok));
    const int64_t nlo = lo + (int64_t)f * step;
    int64_t nhi = lo + (int64_t)(f + 1) * step - 1;
    if (nhi > hi) nhi = hi;
    lo = nlo; hi = nhi;
  }
  return lo;
}

__global__ void __launch_bounds__(1024) k_disp_chain(const HfxParams p, const DispArgs a, const DispWork w, const int stage) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = p.n_replicas;
  uint64_t *s_mat = reinterpret_cast<uint64_t *>(smem_raw);     // [R] maturity, biased to unsigned order; then the budgets
  uint32_t *s_id = reinterpret_cast<uint32_t *>(s_mat + R);     // [R]
  int32_t *s_room = reinterpret_cast<int32_t *>(s_id + R);      // [R] entries the batch cap still allows
  int32_t *s_rs = s_room + R;                                   // [R] where the k-th instance's run starts in the queue
  int32_t *s_rl = s_rs + R;                                     // [R] and how many positions it covers
  __shared__ int64_t s_pre[CHAIN_WINDOW + 32];                  // running totals of the window; behind them entries that fit nothing
  __shared__ int32_t s_cnt[CHAIN_WINDOW + 32];
  __shared__ int32_t s_nm, s_k, s_done;
  __shared__ int64_t s_cursor, s_base, s_basec;
  if (threadIdx.x == 0) { s_nm = 0; s_k = 0; s_done = 0; s_cursor = 0; s_base = 0; s_basec = 0; }
  __syncthreads();
  for (int r = threadIdx.x; r < R; r += blockDim.x)
    if (a.maturity[r] <= a.now && (a.cfg[r].mode == HFX_DECODE) == (stage != 0)) {
      const int k = atomicAdd(&s_nm, 1);
      s_mat[k] = (uint64_t)a.maturity[r] ^ (1ull << 63);
      s_id[k] = (uint32_t)r;
    }
  __syncthreads();
  const int nm = s_nm;
  block_sort<true>(s_mat, s_id, nm);
  int64_t *s_bud = reinterpret_cast<int64_t *>(s_mat);
  const int listed = stage ? a.n_mature[0] : 0;      // the D instances are listed behind the first stage's
  for (int k = threadIdx.x; k < nm; k += blockDim.x) {
    const int r = (int)s_id[k];
    a.inst_order[listed + k] = r;
    const ReplicaPlan *pl = w.plan + r;
    s_bud[k] = pl->budget < (INT64_C(1) << 62) ? pl->budget : (INT64_C(1) << 62);     // (a D-stage budget may be unbounded; the totals stay far below)
    int64_t room = INT32_MAX;
    if (pl->batch_cap != 0) { const int64_t left = (int64_t)pl->batch_cap - pl->n_eff; room = left > 0 ? left : 0; }
    s_room[k] = (int32_t)(room < INT32_MAX ? room : INT32_MAX);
    s_rs[k] = 0; s_rl[k] = 0;
  }
  if (threadIdx.x == 0) a.n_mature[stage] = nm;
  const int lane = threadIdx.x & 31;
  const int64_t nq = (int64_t)w.ctl[8 * stage + 1];
  for (int guard = 0; guard < 2 * nm + 4; guard++) {      // every round finishes an instance or refills for one
    __syncthreads();
    if (s_done || s_k >= nm || s_cursor >= nq) break;
    // refill the window from the current position
    const int64_t w0 = s_cursor;
    const int64_t wn = nq - w0 < CHAIN_WINDOW ? nq - w0 : CHAIN_WINDOW;
    for (int i = threadIdx.x; i < wn; i += blockDim.x) { s_pre[i] = w.prefix[w0 + i]; s_cnt[i] = w.prefix_cnt[w0 + i]; }
    if (threadIdx.x < 32) { s_pre[wn + threadIdx.x] = INT64_MAX; s_cnt[wn + threadIdx.x] = INT32_MAX; }
    __syncthreads();
    if (threadIdx.x < 32) {
      int k = s_k;
      int64_t cursor = s_cursor, base = s_base, base_cnt = s_basec;
      const bool last_window = w0 + wn >= nq;
      for (; k < nm && cursor < nq; k++) {
        const int64_t limit = base + s_bud[k], limit_cnt = base_cnt + s_room[k];
        const int i0 = (int)(cursor - w0);
        {   // most runs are short: probes of the next 32 entries, up to eight in a row, settle them (the entries that
            // fit are a prefix); the first entry that does not fit must have been looked at, or the queue must end
          int i1 = i0;
          int64_t e_pre = base, e_cnt = base_cnt;
          bool settled = false;
          for (int it = 0; it < 8; it++) {
            const int64_t pre = s_pre[i1 + lane];
            const int32_t cn = s_cnt[i1 + lane];
            const int f = __popc(__ballot_sync(0xffffffffu, pre <= limit && (int64_t)cn <= limit_cnt));
            if (f > 0) {
              e_pre = __shfl_sync(0xffffffffu, pre, f - 1);
              e_cnt = __shfl_sync(0xffffffffu, cn, f - 1);
              i1 += f;
            }
            if (f < 32) { settled = i1 < (int)wn || last_window; break; }
            if (i1 >= (int)wn && !last_window) break;      // the window is used up and the queue goes on: the search below decides
          }
          if (settled) {
            if (i1 > i0) {
              s_rs[k] = (int32_t)cursor; s_rl[k] = i1 - i0;
              cursor += i1 - i0; base = e_pre; base_cnt = e_cnt;
              if (cursor >= w0 + wn) { k++; break; }      // the window is used up
            }
            continue;
          }
        }
        // longer runs, and runs that may leave the window: a gallop and a 32-way search on the running totals
        const int64_t span = nq - cursor, avail = w0 + wn - cursor;
        const int64_t off = cursor - w0 - 1;
        const int64_t hiw = span < avail ? span : avail;
        int64_t m = warp_longest(0, hiw, lane, [&](int64_t x) { return s_pre[off + x] <= limit && (int64_t)s_cnt[off + x] <= limit_cnt; });
        if (m == hiw && hiw < span) {          // the stretch may go on past the window
          if (cursor != w0) break;              // refill from here and search again
          m = warp_longest(m, span, lane, [&](int64_t x) {
            return w.prefix[cursor + x - 1] <= limit && (int64_t)w.prefix_cnt[cursor + x - 1] <= limit_cnt; });
        }
        if (m > 0) {
          int64_t e_pre, e_cnt;
          if (m <= avail) { e_pre = s_pre[off + m]; e_cnt = s_cnt[off + m]; }
          else { e_pre = w.prefix[cursor + m - 1]; e_cnt = w.prefix_cnt[cursor + m - 1]; }
          s_rs[k] = (int32_t)cursor; s_rl[k] = (int32_t)m;
          cursor += m; base = e_pre; base_cnt = e_cnt;
          if (cursor >= w0 + wn) { k++; break; }      // the window is used up
        }
      }
      if (lane == 0) { s_k = k; s_cursor = cursor; s_base = base; s_basec = base_cnt; }
    }
  }
  __syncthreads();
  // what every instance took, from the running totals at the ends of its run
  for (int k = threadIdx.x; k < nm; k += blockDim.x) {
    const int32_t m = s_rl[k];
    if (m > 0) {
      const int32_t st = s_rs[k];
      const int r = (int)s_id[k];
      const int64_t b0 = st > 0 ? w.prefix[st - 1] : 0, b1 = w.prefix[st + m - 1];
      const int32_t c0 = st > 0 ? w.prefix_cnt[st - 1] : 0, c1 = w.prefix_cnt[st + m - 1];
      w.run_start[r] = st;
      w.run_len[r] = m;
      a.adm_cost[r] = b1 - b0;
      a.adm_count[r] = c1 - c0;
    }
  }
}

// the request -> instance binding of every dispatched row, and dispatching step 4 (the new maturity
// time of an instance that took requests): one block per instance
__global__ void __launch_bounds__(DISP_THREADS) k_disp_assign(const HfxParams p, const DispArgs a, const DispWork w, int slot,
                                                              const DispCost cost, const int stage) {
  const int r = blockIdx.x;
  if ((a.cfg[r].mode == HFX_DECODE) != (stage != 0)) return;      // the other stage's instance
  const int32_t m = w.run_len[r], s0 = w.run_start[r];
  const int64_t bmax = (int64_t)w.ctl[8 * stage + 4];
  int64_t kv = 0;
  for (int32_t q = threadIdx.x; q < m; q += blockDim.x) {
    const uint32_t row = w.val[slot][s0 + q];
    if (cost.of(row) <= bmax) {       // the others were passed over
      a.assign[row] = r;
      kv += (int64_t)a.prompt_len[row] + a.gen[row];
    }
  }
  if (stage) {      // maturity = end of the next decode iteration of the enlarged batch: the context the run brings
    __shared__ int64_t s_kv[DISP_THREADS / 32];
    kv = warp_sum_i64(kv);
    if ((threadIdx.x & 31) == 0) s_kv[threadIdx.x >> 5] = kv;
    __syncthreads();
    if (threadIdx.x == 0) {
      kv = 0;
      for (int k = 0; k < DISP_THREADS / 32; k++) kv += s_kv[k];
      int64_t lp = 0;
      a.maturity_next[r] = dev_maturity_next(p, w.plan[r], a.adm_count[r], a.adm_cost[r], kv, &lp);
    }
  } else if (threadIdx.x == 0 && a.adm_count[r] > 0) {
    int64_t lp = 0;
    a.maturity_next[r] = dev_maturity_next(p, w.plan[r], a.adm_count[r], a.adm_cost[r], 0, &lp);
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct hfx_dispatch_ws { DispWork w; int ready; };

int hfx_dispatch_configure() {
  if (cudaFuncSetAttribute(k_disp_chain, cudaFuncAttributeMaxDynamicSharedMemorySize, 24 * DISP_MAX_INSTANCES) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}

static void disp_free(DispWork &w) {
  cudaFree(w.key[0]); cudaFree(w.key[1]); cudaFree(w.val[0]); cudaFree(w.val[1]); cudaFree(w.rowkey); cudaFree(w.prefix);
  cudaFree(w.hist); cudaFree(w.tile_sum); cudaFree(w.n_run); cudaFree(w.sum_kv); cudaFree(w.mask_run); cudaFree(w.ctl);
  cudaFree(w.plan); cudaFree(w.run_start); cudaFree(w.run_len); cudaFree(w.prefix_cnt); cudaFree(w.blk_cnt);
  cudaGetLastError();
}

void hfx_dispatch_release(hfx_sched *s) {
  if (!s->dispatch_ws) return;
  hfx_dispatch_ws *d = reinterpret_cast<hfx_dispatch_ws *>(s->dispatch_ws);
  disp_free(d->w);
  delete d;
  s->dispatch_ws = nullptr;
}

static int disp_workspace(hfx_sched *s, hfx_dispatch_ws **out) {
  if (s->dispatch_ws) { *out = reinterpret_cast<hfx_dispatch_ws *>(s->dispatch_ws); return HFX_OK; }
  hfx_dispatch_ws *d = new (std::nothrow) hfx_dispatch_ws();
  if (!d) return HFX_E_NOMEM;
  memset(d, 0, sizeof(*d));
  DispWork &w = d->w;
  const size_t rows = (size_t)s->max_rows, R = (size_t)s->p.n_replicas;
  const size_t tiles = (rows + RADIX_TILE - 1) / RADIX_TILE;
  w.max_rows = s->max_rows; w.R = s->p.n_replicas;
  bool ok = true;
  for (int k = 0; k < 2; k++) {
    ok = ok && cudaMalloc(&w.key[k], sizeof(uint64_t) * rows) == cudaSuccess;
    ok = ok && cudaMalloc(&w.val[k], sizeof(uint32_t) * rows) == cudaSuccess;
  }
  ok = ok && cudaMalloc(&w.rowkey, sizeof(uint64_t) * rows) == cudaSuccess;
  ok = ok && cudaMalloc(&w.prefix, sizeof(int64_t) * rows) == cudaSuccess;
  ok = ok && cudaMalloc(&w.hist, sizeof(uint32_t) * 256 * tiles) == cudaSuccess;
  ok = ok && cudaMalloc(&w.tile_sum, sizeof(int64_t) * 2 * tiles) == cudaSuccess;
  ok = ok && cudaMalloc(&w.prefix_cnt, sizeof(int32_t) * rows) == cudaSuccess;
  ok = ok && cudaMalloc(&w.n_run, sizeof(uint32_t) * R) == cudaSuccess;
  ok = ok && cudaMalloc(&w.sum_kv, sizeof(unsigned long long) * R) == cudaSuccess;
  ok = ok && cudaMalloc(&w.mask_run, sizeof(unsigned long long) * R) == cudaSuccess;
  ok = ok && cudaMalloc(&w.ctl, 256) == cudaSuccess;
  ok = ok && cudaMalloc(&w.blk_cnt, sizeof(uint32_t) * 2 * DISP_SCAN_BLOCKS_MAX) == cudaSuccess;
  ok = ok && cudaMalloc(&w.plan, sizeof(ReplicaPlan) * R) == cudaSuccess;
  ok = ok && cudaMalloc(&w.run_start, sizeof(int32_t) * R) == cudaSuccess;
  ok = ok && cudaMalloc(&w.run_len, sizeof(int32_t) * R) == cudaSuccess;
  if (!ok) { cudaGetLastError(); disp_free(w); delete d; return HFX_E_NOMEM; }
  s->dispatch_ws = d;
  *out = d;
  return HFX_OK;
}

int hfx_launch_dispatch(hfx_sched *s, const hfx_table *t, int64_t now_ns, const int64_t *maturity, const hfx_dispatch_out *o,
                        int32_t cap_max, bool d_stage) {
  hfx_dispatch_ws *d = nullptr;
  int rc = disp_workspace(s, &d);
  if (rc != HFX_OK) return rc;
  const DispWork &w = d->w;
  cudaStream_t st = s->stream;
  const int R = s->p.n_replicas;
  const int64_t n = t->n_rows;
  DispArgs a;
  a.replica_id = t->replica_id; a.class_id = t->class_id; a.state = t->state; a.prompt_len = t->prompt_len; a.gen = t->gen;
  a.arrival = t->arrival_ns; a.req_id = t->req_id; a.weight = s->p.weight_max > 0 ? t->weight : nullptr;
  a.first_token = t->first_token_ns; a.d_stage = d_stage ? 1 : 0; a.mode = s->d_mode;
  a.n = n; a.now = now_ns; a.cap_max = cap_max; a.maturity = maturity; a.cfg = s->d_cfg;
  a.assign = o->assign; a.queue_order = o->queue_order; a.n_queue = o->n_queue; a.inst_order = o->inst_order;
  a.n_mature = o->n_mature; a.slack = o->slack_ns; a.budget = o->budget; a.e_d = o->e_d_ns; a.n_run = o->n_run;
  a.sum_kv = o->sum_kv; a.adm_cost = o->adm_cost; a.adm_count = o->adm_count; a.maturity_next = o->maturity_next;
  a.status = s->d_status;
  if (cudaMemsetAsync(w.n_run, 0, sizeof(uint32_t) * R, st) != cudaSuccess ||
      cudaMemsetAsync(w.sum_kv, 0, sizeof(unsigned long long) * R, st) != cudaSuccess ||
      cudaMemsetAsync(w.mask_run, 0, sizeof(unsigned long long) * R, st) != cudaSuccess ||
      cudaMemsetAsync(w.ctl, 0, 128, st) != cudaSuccess)
    return HFX_E_CUDA;
  const int tiles_max = (int)((s->max_rows + RADIX_TILE - 1) / RADIX_TILE);
  const int tiles = n > 0 ? (int)((n + RADIX_TILE - 1) / RADIX_TILE) : 1;      // tiles the queue can fill in this call
  int grid = (int)((n + DISP_THREADS - 1) / DISP_THREADS);
  if (grid > s->n_sm * 8) grid = s->n_sm * 8;
  if (grid > DISP_SCAN_BLOCKS_MAX) grid = DISP_SCAN_BLOCKS_MAX;
  if (grid < 1) grid = 1;
  { KernelScope ks(s, KSLOT_DISPATCH); k_disp_scan<<<grid, DISP_THREADS, 0, st>>>(s->p, a, w); }
  for (int stage = 0; stage < (d_stage ? 2 : 1); stage++) {
    unsigned long long *ctl = w.ctl + 8 * stage;
    DispCost cost;
    cost.prompt_len = t->prompt_len; cost.gen = t->gen; cost.d1 = s->p.d1; cost.d2 = s->p.d2; cost.stage = stage;
    { KernelScope ks(s, KSLOT_DISPATCH); k_disp_compact<<<grid, DISP_THREADS, 0, st>>>(a, w, stage); }
    int slot = 0;
    auto pass = [&](int shift, const unsigned long long *only_if) {
      { KernelScope ks(s, KSLOT_DISPATCH); k_radix_hist<<<tiles, DISP_THREADS, 0, st>>>(w.key[slot], ctl + 1, shift, w.hist, only_if); }
      { KernelScope ks(s, KSLOT_DISPATCH); k_radix_scatter<<<tiles, DISP_THREADS, 0, st>>>(w.key[slot], w.val[slot], w.key[slot ^ 1], w.val[slot ^ 1], ctl + 1, shift, w.hist, only_if); }
      slot ^= 1;
    };
    // by request id, only when the ids do not rise with the rows (the kernels leave at once otherwise; an even
    // number of passes, so the pairs are back in the first buffer either way)
    for (int shift = 0; shift < 32; shift += 8) pass(shift, w.ctl + 5);
    {
      KernelScope ks(s, KSLOT_DISPATCH);
      k_disp_gather<<<tiles, DISP_THREADS, 0, st>>>(w.key[slot], w.val[slot], w.rowkey, ctl + 1, w.ctl + 5);
    }
    for (int shift = 0; shift < 48; shift += 8) pass(shift, nullptr);   // by (priority, slack)
    { KernelScope ks(s, KSLOT_DISPATCH); k_disp_plan<<<(R + DISP_THREADS - 1) / DISP_THREADS, DISP_THREADS, 0, st>>>(s->p, a, w, stage); }
    { KernelScope ks(s, KSLOT_DISPATCH); k_disp_tilesum<<<tiles, DISP_THREADS, 0, st>>>(w.val[slot], cost, ctl, w.tile_sum, tiles_max, ctl + 3); }
    { KernelScope ks(s, KSLOT_DISPATCH); k_disp_prefix<<<tiles, DISP_THREADS, 0, st>>>(w.val[slot], cost, ctl, w.tile_sum, tiles_max, w.prefix, w.prefix_cnt, o->queue_order, o->n_queue + stage, stage ? w.ctl + 1 : nullptr); }
    { KernelScope ks(s, KSLOT_DISPATCH); k_disp_chain<<<1, 1024, 24 * (size_t)R, st>>>(s->p, a, w, stage); }
    { KernelScope ks(s, KSLOT_DISPATCH); k_disp_assign<<<R, DISP_THREADS, 0, st>>>(s->p, a, w, slot, cost, stage); }
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
