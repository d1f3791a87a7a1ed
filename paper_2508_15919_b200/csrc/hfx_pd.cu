// hfx_pd_migrate: hand-off of prefilled requests from the P instances to their partner D instances in
// the disaggregated mode (Sec. 3.3.1 "Disaggregated Mode"); with hfx_sched_step + HFX_COMMIT it couples
// the two stages.
//
//   k_pd_rows    one streaming pass: a request RUNNING on a P instance whose KV transfer
//                (x0 + x1 * prompt_len after its first token) has ended by its partner's clock becomes
//                QUEUED on the partner; otherwise it bids for the partner's wake-up time.  Rows that
//                keep a D instance occupied (in flight, or queued and arrived) mark it busy.
//   k_pd_clock   a D instance that is not busy is woken at the earliest end of a transfer to it.
// A row that moves makes its new instance busy in the same pass, so the two kernels need no third.
#include "hfx_internal.cuh"

#define PD_THREADS 256

struct PdArgs {
  int32_t *replica_id; const uint8_t *class_id; uint8_t *state; const int32_t *prompt_len; const int32_t *gen;
  const int64_t *arrival; const int64_t *first_token; int64_t n;
  int64_t *now; const int32_t *pair; const uint8_t *mode; int64_t x0, x1;
  long long *wake; uint32_t *busy; uint32_t *moved; int32_t *n_moved; uint32_t *status;
};

__global__ void __launch_bounds__(PD_THREADS) k_pd_rows(const HfxParams p, const PdArgs a) {
  const int R = p.n_replicas;
  uint32_t bad = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < a.n; i += (int64_t)gridDim.x * blockDim.x) {
    const int32_t r = a.replica_id[i];
    if (r == -1 && a.state[i] == HFX_QUEUED) continue;       // still in the global queue
    if (r < 0 || r >= R) { bad |= HFX_ST_BAD_REPLICA; continue; }
    const uint32_t cls = a.class_id[i], st = a.state[i];
    const int32_t prompt = a.prompt_len[i], gen = a.gen[i];
    bool ok = true;
    if (cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
    if (prompt < 0 || prompt > HFX_MAX_TOKENS || gen < 0 || gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
    if (!ok) continue;
    const int mode = a.mode[r];
    if (mode == HFX_DECODE) {
      if ((st == HFX_RUNNING || (st == HFX_QUEUED && a.arrival[i] <= a.now[r])) && a.busy[r] == 0) atomicExch(&a.busy[r], 1u);
    } else if (mode == HFX_PREFILL && st == HFX_RUNNING) {
      const int32_t d = a.pair[r];
      if (d < 0 || d >= R || a.mode[d] != HFX_DECODE) { bad |= HFX_ST_BAD_REPLICA; continue; }
      const int64_t ready = a.first_token[i] + a.x0 + a.x1 * (int64_t)prompt;
      if (ready <= a.now[d]) {
        a.replica_id[i] = d;
        a.state[i] = HFX_QUEUED;
        if (a.arrival[i] <= a.now[d]) atomicExch(&a.busy[d], 1u);      // prefilled and arrived: it occupies the D instance's queue
        atomicAdd(a.moved, 1u);
      } else atomicMin(&a.wake[d], (long long)ready);
    }
  }
  if (bad) atomicOr(a.status, bad);
}

__global__ void __launch_bounds__(PD_THREADS) k_pd_clock(const HfxParams p, const PdArgs a) {
  const int d = blockIdx.x * blockDim.x + threadIdx.x;
  if (d == 0 && a.n_moved) *a.n_moved = (int32_t)*a.moved;
  if (d >= p.n_replicas || a.mode[d] != HFX_DECODE) return;
  const long long w = a.wake[d];
  if (a.busy[d] == 0 && w != INT64_MAX && w > a.now[d]) a.now[d] = w;
}

// wake-up times start at "never", nothing is busy, nothing has moved
__global__ void __launch_bounds__(PD_THREADS) k_pd_init(long long *wake, uint32_t *busy, uint32_t *moved, int R) {
  const int d = blockIdx.x * blockDim.x + threadIdx.x;
  if (d < R) { wake[d] = INT64_MAX; busy[d] = 0; }
  if (d == 0) *moved = 0;
}

size_t hfx_pd_workspace_bytes(int n_replicas) { return 16 + (size_t)n_replicas * 16; }

int hfx_launch_pd_migrate(hfx_sched *s, const hfx_table *t, int32_t *replica_id, int64_t *now, const int32_t *pair, int64_t x0,
                          int64_t x1, int32_t *n_moved) {
  const int R = s->p.n_replicas;
  PdArgs a;
  unsigned char *ws = reinterpret_cast<unsigned char *>(s->d_pd);
  a.moved = reinterpret_cast<uint32_t *>(ws);
  a.wake = reinterpret_cast<long long *>(ws + 16);
  a.busy = reinterpret_cast<uint32_t *>(ws + 16 + (size_t)R * 8);
  a.replica_id = replica_id; a.class_id = t->class_id; a.state = t->state; a.prompt_len = t->prompt_len; a.gen = t->gen;
  a.arrival = t->arrival_ns; a.first_token = t->first_token_ns; a.n = t->n_rows;
  a.now = now; a.pair = pair; a.mode = s->d_mode; a.x0 = x0; a.x1 = x1; a.n_moved = n_moved; a.status = s->d_status;
  cudaStream_t st = s->stream;
  {
    KernelScope ks(s, KSLOT_PD);
    k_pd_init<<<(R + PD_THREADS - 1) / PD_THREADS, PD_THREADS, 0, st>>>(a.wake, a.busy, a.moved, R);
  }
  {
    KernelScope ks(s, KSLOT_PD);
    int grid = (int)((t->n_rows + PD_THREADS - 1) / PD_THREADS);
    if (grid > s->n_sm * 8) grid = s->n_sm * 8;
    if (grid < 1) grid = 1;
    k_pd_rows<<<grid, PD_THREADS, 0, st>>>(s->p, a);
  }
  {
    KernelScope ks(s, KSLOT_PD);
    k_pd_clock<<<(R + PD_THREADS - 1) / PD_THREADS, PD_THREADS, 0, st>>>(s->p, a);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
