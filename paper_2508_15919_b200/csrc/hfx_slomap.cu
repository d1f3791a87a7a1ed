// hfx_slo_map: priority-based SLO mapping (Sec. 3.3.2).  Requests that carry only a priority get
// their TTFT / TPOT targets from a sliding window of completed requests.
//
//   k_slo_window   one block: per-priority counts C_i of the window, the window ordered by TTFT and
//                  by TPOT (shared-memory sorting network on (value, position)), and for every
//                  priority p the record at index base + offset, base = C_0 + ... + C_{p-1},
//                  offset = floor((p + 1) C_p / (N + 1)): its TTFT, its queueing delay, the TPOT of
//                  the same index; whether a higher priority is pending
//   k_slo_first    the first request (lowest row) of every priority in this call: only it sees the
//                  queueing-delay correction, the later ones find the delay it left behind
//   k_slo_assign   per request: correction, contention-aware clamp, the two targets
#include "hfx_internal.cuh"

#define SLO_WINDOW_MAX 4096
#define SLO_THREADS 256

struct SloTable {          // per priority, HFX_MAX_CLASSES entries each
  int64_t ref_ttft[HFX_MAX_CLASSES], ref_tpot[HFX_MAX_CLASSES], ref_queue[HFX_MAX_CLASSES], delta[HFX_MAX_CLASSES];
  int64_t first_row[HFX_MAX_CLASSES];
  int32_t higher_pending[HFX_MAX_CLASSES];
  int32_t w_valid;
};

struct SloArgs {
  const int32_t *win_prio; const int64_t *win_ttft; const int64_t *win_tpot; const int64_t *win_queue; int32_t w;
  const int64_t *ttft_min, *ttft_max, *ttft_min_relaxed, *tpot_min, *tpot_max, *tpot_min_relaxed;
  int64_t *last_queue; const int32_t *pending; const int32_t *new_prio; int64_t n_new;
  int64_t *ttft_out, *tpot_out;
  int32_t n_prio; SloTable *tab; uint32_t *status;
};

__global__ void __launch_bounds__(1024) k_slo_window(const SloArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t *s_val = reinterpret_cast<uint64_t *>(smem_raw);              // [w] value, biased to unsigned order
  uint32_t *s_pos = reinterpret_cast<uint32_t *>(s_val + a.w);           // [w] record position
  __shared__ uint32_t s_C[HFX_MAX_CLASSES + 1];
  __shared__ uint32_t s_idx[HFX_MAX_CLASSES];
  __shared__ uint32_t s_n;
  const int N = a.n_prio;
  for (int i = threadIdx.x; i <= HFX_MAX_CLASSES; i += blockDim.x) s_C[i] = 0;
  if (threadIdx.x == 0) s_n = 0;
  __syncthreads();
  // valid records, their counts per priority; the TTFT items
  uint32_t bad = 0;
  for (int j = threadIdx.x; j < a.w; j += blockDim.x) {
    const int32_t pr = a.win_prio[j];
    if (pr < 0 || pr >= N) { bad |= HFX_ST_BAD_CLASS; continue; }
    atomicAdd(&s_C[pr], 1u);
    const uint32_t k = atomicAdd(&s_n, 1u);
    s_val[k] = (uint64_t)a.win_ttft[j] ^ (1ull << 63);
    s_pos[k] = (uint32_t)j;
  }
  if (bad) atomicOr(a.status, bad);
  __syncthreads();
  const int w = (int)s_n;
  if (threadIdx.x < N) {      // index of priority threadIdx.x; a higher priority pending?
    const int pr = threadIdx.x;
    uint32_t base = 0;
    int hp = 0;
    for (int i = 0; i < pr; i++) { base += s_C[i]; hp |= a.pending[i] > 0; }
    const uint32_t offset = (uint32_t)(((uint64_t)(pr + 1) * s_C[pr]) / (uint64_t)(N + 1));
    uint32_t idx = base + offset;
    if (w > 0 && idx > (uint32_t)(w - 1)) idx = (uint32_t)(w - 1);
    s_idx[pr] = idx;
    a.tab->higher_pending[pr] = hp;
    a.tab->first_row[pr] = INT64_MAX;
  }
  if (threadIdx.x == 0) a.tab->w_valid = w;
  __syncthreads();
  block_sort<true>(s_val, s_pos, w);
  if (threadIdx.x < N && w > 0) {
    const int pr = threadIdx.x;
    const uint32_t idx = s_idx[pr];
    const int64_t q = a.win_queue[s_pos[idx]];
    a.tab->ref_ttft[pr] = (int64_t)(s_val[idx] ^ (1ull << 63));
    a.tab->ref_queue[pr] = q;
    a.tab->delta[pr] = q - a.last_queue[pr];
  }
  __syncthreads();
  // the same records by TPOT
  for (int k = threadIdx.x; k < w; k += blockDim.x) s_val[k] = (uint64_t)a.win_tpot[s_pos[k]] ^ (1ull << 63);
  __syncthreads();
  block_sort<true>(s_val, s_pos, w);
  if (threadIdx.x < N && w > 0) a.tab->ref_tpot[threadIdx.x] = (int64_t)(s_val[s_idx[threadIdx.x]] ^ (1ull << 63));
}

__global__ void __launch_bounds__(SLO_THREADS) k_slo_first(const SloArgs a) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < a.n_new; i += (int64_t)gridDim.x * blockDim.x) {
    const int32_t pr = a.new_prio[i];
    if (pr >= 0 && pr < a.n_prio) atomicMin(reinterpret_cast<long long *>(&a.tab->first_row[pr]), (long long)i);
  }
}

__global__ void __launch_bounds__(SLO_THREADS) k_slo_assign(const SloArgs a) {
  const int w = a.tab->w_valid;
  uint32_t bad = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < a.n_new; i += (int64_t)gridDim.x * blockDim.x) {
    const int32_t pr = a.new_prio[i];
    int64_t ttft = 0, tpot = 0;
    if (pr < 0 || pr >= a.n_prio) bad |= HFX_ST_BAD_CLASS;
    else {
      ttft = a.ttft_max[pr]; tpot = a.tpot_max[pr];
      if (w > 0) {
        const bool first = a.tab->first_row[pr] == i;
        ttft = a.tab->ref_ttft[pr] - (first ? a.tab->delta[pr] : 0);
        tpot = a.tab->ref_tpot[pr];
        if (first) a.last_queue[pr] = a.tab->ref_queue[pr];      // (the others read the delay from the table)
      }
      const bool hp = a.tab->higher_pending[pr] != 0;
      const int64_t lo_t = hp ? a.ttft_min[pr] : a.ttft_min_relaxed[pr], hi_t = a.ttft_max[pr];
      const int64_t lo_p = hp ? a.tpot_min[pr] : a.tpot_min_relaxed[pr], hi_p = a.tpot_max[pr];
      ttft = ttft < lo_t ? lo_t : (ttft > hi_t ? hi_t : ttft);
      tpot = tpot < lo_p ? lo_p : (tpot > hi_p ? hi_p : tpot);
    }
    a.ttft_out[i] = ttft;
    a.tpot_out[i] = tpot;
  }
  if (bad) atomicOr(a.status, bad);
}

int hfx_slomap_configure() {
  if (cudaFuncSetAttribute(k_slo_window, cudaFuncAttributeMaxDynamicSharedMemorySize, 12 * SLO_WINDOW_MAX) != cudaSuccess)
    return HFX_E_CUDA;
  return HFX_OK;
}

int hfx_launch_slo_map(hfx_sched *s, int32_t n_prio, const hfx_slo_window *win, const hfx_slo_bounds *b, int64_t *last_queue,
                       const int32_t *pending, const int32_t *new_prio, int64_t n_new, int64_t *ttft_out, int64_t *tpot_out) {
  SloArgs a;
  a.win_prio = win->prio; a.win_ttft = win->ttft_ns; a.win_tpot = win->tpot_ns; a.win_queue = win->queue_ns; a.w = win->w;
  a.ttft_min = b->ttft_min_ns; a.ttft_max = b->ttft_max_ns; a.ttft_min_relaxed = b->ttft_min_relaxed_ns;
  a.tpot_min = b->tpot_min_ns; a.tpot_max = b->tpot_max_ns; a.tpot_min_relaxed = b->tpot_min_relaxed_ns;
  a.last_queue = last_queue; a.pending = pending; a.new_prio = new_prio; a.n_new = n_new;
  a.ttft_out = ttft_out; a.tpot_out = tpot_out; a.n_prio = n_prio;
  a.tab = reinterpret_cast<SloTable *>(s->d_slo); a.status = s->d_status;
  cudaStream_t st = s->stream;
  {
    KernelScope ks(s, KSLOT_SLOMAP);
    k_slo_window<<<1, 1024, 12 * (size_t)(win->w > 0 ? win->w : 1), st>>>(a);
  }
  if (n_new > 0) {
    int grid = (int)((n_new + SLO_THREADS - 1) / SLO_THREADS);
    if (grid > s->n_sm * 8) grid = s->n_sm * 8;
    { KernelScope ks(s, KSLOT_SLOMAP); k_slo_first<<<grid, SLO_THREADS, 0, st>>>(a); }
    { KernelScope ks(s, KSLOT_SLOMAP); k_slo_assign<<<grid, SLO_THREADS, 0, st>>>(a); }
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}

size_t hfx_slomap_workspace_bytes() { return sizeof(SloTable); }
