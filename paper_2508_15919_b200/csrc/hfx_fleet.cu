// The Scaler's decisions carried out, and the dispatcher's decisions bound (Sec. 3.3.3 "Scaling Mechanism
// and Policy", Sec. 3.3.1 step "dispatch them"; cost as in Eq. 1 of the Problem Definition).
//
//   k_fleet_apply  one block walks the instance records three times:
//                    A  charge (since, now] to every instance that is on; a STARTING instance whose ready
//                       time has come turns ACTIVE (clock and maturity brought up to it); a DRAINING
//                       instance that holds no KV block turns OFF; the lowest id of each pool in each
//                       state is collected with shared-memory atomicMin
//                    B  three threads, one per pool, carry out the pool's decision on one instance
//                    C  due time and capacity per instance, charged time summed per pool
//                  A and B touch different instances' records only through the block barrier between them.
//   k_disp_bind    grid-stride: replica_id[i] = assign[i] where a request was dispatched; the clock of an
//                  instance that was given requests is brought up to the time of the call.
#include "hfx_internal.cuh"

#define FLEET_THREADS 1024
#define BIND_THREADS 256

struct FleetArgs {
  int32_t *inst_state; int64_t *ready; int64_t *billed; int64_t *since; int32_t *total_blocks; int64_t *due;
  const int32_t *blocks_cap;
  const int32_t *decision; const int64_t *used_blocks; const uint8_t *mode;
  int64_t *clock; int64_t *maturity; int64_t *cost;
  int64_t now; int64_t cold[3];
};

__global__ void __launch_bounds__(FLEET_THREADS) k_fleet_apply(const HfxParams p, const FleetArgs a) {
  __shared__ int s_first[3][4];                  // lowest id of the pool in each state, INT_MAX if none
  __shared__ unsigned long long s_cost[3];
  const int R = p.n_replicas;
  if (threadIdx.x < 12) s_first[threadIdx.x >> 2][threadIdx.x & 3] = INT_MAX;
  if (threadIdx.x < 3) s_cost[threadIdx.x] = 0;
  __syncthreads();
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    int st = a.inst_state[r];
    if (st < HFX_INST_OFF || st > HFX_INST_DRAINING) st = HFX_INST_OFF;      // a record out of range counts as OFF
    if (st != HFX_INST_OFF && a.now > a.since[r]) { a.billed[r] += a.now - a.since[r]; a.since[r] = a.now; }
    if (st == HFX_INST_STARTING && a.ready[r] <= a.now) {
      st = HFX_INST_ACTIVE;
      const int64_t rd = a.ready[r];
      if (a.clock[r] < rd) a.clock[r] = rd;
      if (a.maturity[r] < rd) a.maturity[r] = rd;
    } else if (st == HFX_INST_DRAINING && a.used_blocks[r] == 0) st = HFX_INST_OFF;
    a.inst_state[r] = st;
    const int pool = a.mode[r];
    if (pool < 3) atomicMin(&s_first[pool][st], r);
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    const int pool = threadIdx.x;
    const int action = a.decision[2 * pool], victim = a.decision[2 * pool + 1];
    if (action > 0) {
      if (s_first[pool][HFX_INST_STARTING] != INT_MAX) {
        // capacity is already on its way
      } else if (s_first[pool][HFX_INST_DRAINING] != INT_MAX) {
        a.inst_state[s_first[pool][HFX_INST_DRAINING]] = HFX_INST_ACTIVE;
      } else if (s_first[pool][HFX_INST_OFF] != INT_MAX) {
        const int r = s_first[pool][HFX_INST_OFF];
        a.inst_state[r] = HFX_INST_STARTING; a.ready[r] = a.now + a.cold[pool]; a.since[r] = a.now;
      }
    } else if (action < 0 && victim >= 0 && victim < R && a.mode[victim] == pool && a.inst_state[victim] == HFX_INST_ACTIVE) {
      a.inst_state[victim] = HFX_INST_DRAINING;
    }
  }
  __syncthreads();
  unsigned long long c[3] = {0, 0, 0};
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const bool on = a.inst_state[r] == HFX_INST_ACTIVE;
    a.total_blocks[r] = on ? a.blocks_cap[r] : 0;
    a.due[r] = on ? a.maturity[r] : INT64_MAX;
    const int pool = a.mode[r];
    const unsigned long long b = (unsigned long long)a.billed[r];
#pragma unroll
    for (int q = 0; q < 3; q++) if (pool == q) c[q] += b;
  }
#pragma unroll
  for (int q = 0; q < 3; q++) {
    unsigned long long x = c[q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) == 0 && x) atomicAdd(&s_cost[q], x);
  }
  __syncthreads();
  if (threadIdx.x < 3) a.cost[threadIdx.x] = (int64_t)s_cost[threadIdx.x];
}

int hfx_launch_fleet_apply(hfx_sched *s, int64_t now, const int32_t *decision, const int64_t *used_blocks,
                           const int64_t *cold, const hfx_fleet *f, int64_t *clock, int64_t *maturity, int64_t *cost) {
  FleetArgs a;
  a.inst_state = f->inst_state; a.ready = f->ready_ns; a.billed = f->billed_ns; a.since = f->since_ns;
  a.total_blocks = f->total_blocks; a.due = f->due_ns; a.blocks_cap = f->blocks_cap;
  a.decision = decision; a.used_blocks = used_blocks; a.mode = s->d_mode;
  a.clock = clock; a.maturity = maturity; a.cost = cost; a.now = now;
  for (int q = 0; q < 3; q++) a.cold[q] = cold[q];
  {
    KernelScope ks(s, KSLOT_SCALE);
    k_fleet_apply<<<1, FLEET_THREADS, 0, s->stream>>>(s->p, a);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}

__global__ void __launch_bounds__(BIND_THREADS) k_disp_bind(const HfxParams p, const int32_t *__restrict__ assign,
                                                            const int32_t *__restrict__ adm_count, int32_t *replica_id,
                                                            int64_t *clock, int64_t n, int64_t now) {
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = tid; i < n; i += stride) {
    const int32_t r = assign[i];
    if (r >= 0) replica_id[i] = r;
  }
  for (int64_t r = tid; r < p.n_replicas; r += stride)
    if (adm_count[r] > 0 && clock[r] < now) clock[r] = now;
}

int hfx_launch_dispatch_bind(hfx_sched *s, int64_t n, int64_t now, const int32_t *assign, const int32_t *adm_count,
                             int32_t *replica_id, int64_t *clock) {
  int64_t want = ((n > s->p.n_replicas ? n : s->p.n_replicas) + BIND_THREADS - 1) / BIND_THREADS;
  int grid = (int)(want < (int64_t)s->n_sm * 8 ? want : (int64_t)s->n_sm * 8);
  if (grid < 1) grid = 1;
  {
    KernelScope ks(s, KSLOT_DISPATCH);
    k_disp_bind<<<grid, BIND_THREADS, 0, s->stream>>>(s->p, assign, adm_count, replica_id, clock, n, now);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
