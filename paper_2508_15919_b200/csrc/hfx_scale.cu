// hfx_scale_tick: the Scaler's indicators f1, f2, f3 and its threshold policy (Sec. 3.3.3) as one
// streaming reduction over the request table plus a one-block decision.
//   k_scale        4 rows per thread with 16-byte loads; per-pool counters by warp reduction and one
//                  atomic per block; used KV blocks per instance in shared memory, flushed with one
//                  integer atomic per (block, instance) -- integer sums, so the order of the atomics
//                  cannot change any result
//   k_scale_decide one block: per pool the instance with the smallest used/total, the thresholds
#include "hfx_internal.cuh"

#define SCALE_THREADS 512
#define SCALE_SMEM_REPLICAS 8192

struct ScaleArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len;
  const int32_t *gen; const int64_t *arrival; const int64_t *finish;
  const uint8_t *mode; const int32_t *total_blocks;
  int64_t n, now, window;
  int32_t block_tokens;
  unsigned long long *counts;        // [3][4]
  unsigned long long *used_blocks;   // [R]
  int32_t *decision;                 // [3][2]
  uint32_t *status;
  hfx_scale_params sp;
};

// floor(wait * 2^16 / slo), saturated at 2^31, without a 128-bit division
__device__ __forceinline__ uint64_t ratio_q16(int64_t wait, int64_t slo) {
  if (wait <= 0) return 0;
  const uint64_t w = (uint64_t)wait, s = (uint64_t)slo;
  const uint64_t qh = w / s;
  if (qh >= (1u << 15)) return UINT64_C(1) << 31;
  const uint64_t rem = w - qh * s;                       // < slo <= 2^44, so rem << 16 fits
  const uint64_t q = (qh << 16) + ((rem << 16) / s);
  return q > (UINT64_C(1) << 31) ? (UINT64_C(1) << 31) : q;
}

__global__ void __launch_bounds__(SCALE_THREADS) k_scale(const HfxParams p, const ScaleArgs a) {
  extern __shared__ unsigned int s_used[];      // [R] when it fits
  __shared__ unsigned long long s_cnt[12];
  __shared__ int64_t s_ttft[HFX_MAX_CLASSES];
  const int R = p.n_replicas;
  const bool use_smem = R <= SCALE_SMEM_REPLICAS;
  if (use_smem) for (int i = threadIdx.x; i < R; i += blockDim.x) s_used[i] = 0;
  if (threadIdx.x < 12) s_cnt[threadIdx.x] = 0;
  for (int c = threadIdx.x; c < HFX_MAX_CLASSES; c += blockDim.x) s_ttft[c] = c < p.n_classes ? p.ttft[c] : 0;
  __syncthreads();
  const int64_t lo_t = a.now - a.window, now = a.now, B = a.block_tokens;
  uint32_t bad = 0;
  unsigned long long cnt[12];
#pragma unroll
  for (int k = 0; k < 12; k++) cnt[k] = 0;

  auto row = [&](int32_t rid, uint32_t cls, uint32_t st, int32_t prompt, int32_t gen, int64_t arrival, int64_t finish) {
    const bool unbound = rid == -1 && st == HFX_QUEUED;     // still in the global queue
    if (!unbound && (rid < 0 || rid >= R)) { bad |= HFX_ST_BAD_REPLICA; return; }
    bool ok = true;
    if (cls >= (uint32_t)p.n_classes) { bad |= HFX_ST_BAD_CLASS; ok = false; }
    if (prompt < 0 || prompt > HFX_MAX_TOKENS || gen < 0 || gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
    if (!ok) return;
    if (unbound) {
      // the global queue feeds the colocated pool and the P stage: the request counts for both, holds no block
      const unsigned long long c0 = arrival > lo_t && arrival <= now ? 1 : 0;
      const int64_t ttft = s_ttft[cls];
      const bool waits = arrival <= now && ttft > 0;
      const unsigned long long c3 = waits ? ratio_q16(now - arrival, ttft) : 0;
      cnt[0] += c0; cnt[4] += c0;
      cnt[2] += waits; cnt[6] += waits;
      cnt[3] += c3; cnt[7] += c3;
      return;
    }
    const int pool = __ldg(a.mode + rid);
    unsigned long long c0 = 0, c1 = 0, c2 = 0, c3 = 0;
    if (arrival > lo_t && arrival <= now) c0 = 1;
    if (st == HFX_DONE && finish > lo_t && finish <= now) c1 = 1;
    uint32_t blocks = 0;
    if (st == HFX_RUNNING) blocks = (uint32_t)(((int64_t)prompt + gen + B - 1) / B);
    else if (st == HFX_QUEUED && arrival <= now) {
      blocks = (uint32_t)(((int64_t)prompt + B - 1) / B);
      const int64_t ttft = s_ttft[cls];
      if (ttft > 0) { c2 = 1; c3 = ratio_q16(now - arrival, ttft); }
    }
    if (blocks) { if (use_smem) atomicAdd(&s_used[rid], blocks); else atomicAdd(&a.used_blocks[rid], (unsigned long long)blocks); }
#pragma unroll
    for (int q = 0; q < 3; q++)
      if (pool == q) { cnt[4 * q] += c0; cnt[4 * q + 1] += c1; cnt[4 * q + 2] += c2; cnt[4 * q + 3] += c3; }
  };

  const int64_t n4 = a.n >> 2;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
    const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + v);
    const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + v);
    const uchar4 st = __ldg(reinterpret_cast<const uchar4 *>(a.state) + v);
    const int4 pr = __ldg(reinterpret_cast<const int4 *>(a.prompt_len) + v);
    const int4 ge = __ldg(reinterpret_cast<const int4 *>(a.gen) + v);
    const longlong2 ar0 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * v);
    const longlong2 ar1 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * v + 1);
    const longlong2 fi0 = __ldg(reinterpret_cast<const longlong2 *>(a.finish) + 2 * v);
    const longlong2 fi1 = __ldg(reinterpret_cast<const longlong2 *>(a.finish) + 2 * v + 1);
    row(rid.x, cls.x, st.x, pr.x, ge.x, ar0.x, fi0.x);
    row(rid.y, cls.y, st.y, pr.y, ge.y, ar0.y, fi0.y);
    row(rid.z, cls.z, st.z, pr.z, ge.z, ar1.x, fi1.x);
    row(rid.w, cls.w, st.w, pr.w, ge.w, ar1.y, fi1.y);
  }
  if (blockIdx.x == 0)
    for (int64_t i = (n4 << 2) + threadIdx.x; i < a.n; i += blockDim.x)
      row(a.replica_id[i], a.class_id[i], a.state[i], a.prompt_len[i], a.gen[i], a.arrival[i], a.finish[i]);

  // per-pool counters: warp reduction, shared memory, one atomic per block and counter
#pragma unroll
  for (int k = 0; k < 12; k++) {
    unsigned long long x = cnt[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) == 0 && x) atomicAdd(&s_cnt[k], x);
  }
  if (bad) atomicOr(a.status, bad);
  __syncthreads();
  if (threadIdx.x < 12 && s_cnt[threadIdx.x]) atomicAdd(&a.counts[threadIdx.x], s_cnt[threadIdx.x]);
  if (use_smem)
    for (int i = threadIdx.x; i < R; i += blockDim.x) { const unsigned int u = s_used[i]; if (u) atomicAdd(&a.used_blocks[i], (unsigned long long)u); }
}

// 128-bit-free comparison a*b < c*d for non-negative 64-bit operands
__device__ __forceinline__ bool mul_less(uint64_t a, uint64_t b, uint64_t c, uint64_t d) {
  const uint64_t h1 = __umul64hi(a, b), h2 = __umul64hi(c, d);
  return h1 != h2 ? h1 < h2 : a * b < c * d;
}

__global__ void __launch_bounds__(1024) k_scale_decide(const HfxParams p, const ScaleArgs a) {
  __shared__ int s_victim[3][32];
  __shared__ int s_active[3][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int R = p.n_replicas;
  // per pool: number of active instances and the one with the smallest used/total (lowest id on ties)
  for (int pool = 0; pool < 3; pool++) {
    int best = -1, n_act = 0;
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
      if (a.mode[r] != pool || a.total_blocks[r] <= 0) continue;
      n_act++;
      if (best < 0 || mul_less(a.used_blocks[r], (uint64_t)a.total_blocks[best], a.used_blocks[best], (uint64_t)a.total_blocks[r])) best = r;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const int b2 = __shfl_xor_sync(0xffffffffu, best, o);
      n_act += __shfl_xor_sync(0xffffffffu, n_act, o);
      if (b2 >= 0) {
        if (best < 0) best = b2;
        else {
          const bool lt = mul_less(a.used_blocks[b2], (uint64_t)a.total_blocks[best], a.used_blocks[best], (uint64_t)a.total_blocks[b2]);
          const bool eq = !lt && !mul_less(a.used_blocks[best], (uint64_t)a.total_blocks[b2], a.used_blocks[b2], (uint64_t)a.total_blocks[best]);
          if (lt || (eq && b2 < best)) best = b2;
        }
      }
    }
    if (lane == 0) { s_victim[pool][warp] = best; s_active[pool][warp] = n_act; }
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    const int pool = threadIdx.x;
    int best = -1, n_act = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); w++) {
      n_act += s_active[pool][w];
      const int b2 = s_victim[pool][w];
      if (b2 < 0) continue;
      if (best < 0) { best = b2; continue; }
      const bool lt = mul_less(a.used_blocks[b2], (uint64_t)a.total_blocks[best], a.used_blocks[best], (uint64_t)a.total_blocks[b2]);
      const bool eq = !lt && !mul_less(a.used_blocks[best], (uint64_t)a.total_blocks[b2], a.used_blocks[b2], (uint64_t)a.total_blocks[best]);
      if (lt || (eq && b2 < best)) best = b2;
    }
    const uint64_t n_in = a.counts[4 * pool], n_out = a.counts[4 * pool + 1], n_q = a.counts[4 * pool + 2], f2 = a.counts[4 * pool + 3];
    const hfx_scale_params &sp = a.sp;
    const bool f1_valid = n_in >= (uint64_t)(sp.min_samples > 0 ? sp.min_samples : 0);
    int action = 0;
    if ((f1_valid && mul_less((uint64_t)sp.eps_out_den, n_out, (uint64_t)sp.eps_out_num, n_in)) ||
        (n_q > 0 && mul_less((uint64_t)sp.eps_wait_num << 16, n_q, (uint64_t)sp.eps_wait_den, f2)))
      action = 1;
    else if (f1_valid && mul_less((uint64_t)sp.eps_in_num, n_in, (uint64_t)sp.eps_in_den, n_out) && n_act > 1)
      action = -1;
    a.decision[2 * pool] = action;
    a.decision[2 * pool + 1] = action == -1 ? best : -1;
  }
}

static inline bool misaligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

extern "C" int hfx_scale_tick(hfx_sched *s, const hfx_table *t, int64_t now_ns, const int32_t *total_blocks,
                              const hfx_scale_params *sp, const hfx_scale_out *o) {
  if (!s || !t || !total_blocks || !sp || !o || !o->counts || !o->used_blocks || !o->decision) return HFX_E_ARG;
  if (t->n_rows < 0 || sp->window_ns <= 0 || sp->block_tokens <= 0 || sp->eps_out_num <= 0 || sp->eps_out_den <= 0 ||
      sp->eps_in_num <= 0 || sp->eps_in_den <= 0 || sp->eps_wait_num <= 0 || sp->eps_wait_den <= 0)
    return HFX_E_ARG;
  if (t->n_rows > s->max_rows) return HFX_E_CAPACITY;
  if (t->n_rows > 0 && (!t->replica_id || !t->class_id || !t->state || !t->prompt_len || !t->gen || !t->arrival_ns || !t->finish_ns))
    return HFX_E_ARG;
  const void *all[] = {t->replica_id, t->class_id, t->state, t->prompt_len, t->gen, t->arrival_ns, t->finish_ns,
                       total_blocks, o->counts, o->used_blocks, o->decision};
  for (const void *q : all) if (misaligned16(q)) return HFX_E_ALIGN;
  const int R = s->p.n_replicas;
  cudaStream_t stream = s->stream;
  if (cudaMemsetAsync(o->counts, 0, sizeof(int64_t) * 12, stream) != cudaSuccess ||
      cudaMemsetAsync(o->used_blocks, 0, sizeof(int64_t) * (size_t)R, stream) != cudaSuccess) {
    cudaGetLastError();
    return HFX_E_CUDA;
  }
  ScaleArgs a;
  a.replica_id = t->replica_id; a.class_id = t->class_id; a.state = t->state; a.prompt_len = t->prompt_len; a.gen = t->gen;
  a.arrival = t->arrival_ns; a.finish = t->finish_ns; a.mode = s->d_mode; a.total_blocks = total_blocks;
  a.n = t->n_rows; a.now = now_ns; a.window = sp->window_ns; a.block_tokens = sp->block_tokens;
  a.counts = reinterpret_cast<unsigned long long *>(o->counts);
  a.used_blocks = reinterpret_cast<unsigned long long *>(o->used_blocks);
  a.decision = o->decision; a.status = s->d_status; a.sp = *sp;
  {
    KernelScope ks(s, KSLOT_SCALE);
    int64_t want = (t->n_rows / 4 + SCALE_THREADS - 1) / SCALE_THREADS;
    int grid = (int)(want < s->n_sm * 4 ? want : s->n_sm * 4);
    if (grid < 1) grid = 1;
    const size_t sm = R <= SCALE_SMEM_REPLICAS ? sizeof(unsigned int) * (size_t)R : 0;
    k_scale<<<grid, SCALE_THREADS, sm, stream>>>(s->p, a);
  }
  {
    KernelScope ks(s, KSLOT_SCALE);
    k_scale_decide<<<1, 1024, 0, stream>>>(s->p, a);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}

extern "C" int hfx_scale_decide(hfx_sched *s, const int32_t *total_blocks, const hfx_scale_params *sp, const hfx_scale_out *o) {
  if (!s || !total_blocks || !sp || !o || !o->counts || !o->used_blocks || !o->decision) return HFX_E_ARG;
  if (sp->eps_out_num <= 0 || sp->eps_out_den <= 0 || sp->eps_in_num <= 0 || sp->eps_in_den <= 0 || sp->eps_wait_num <= 0 ||
      sp->eps_wait_den <= 0)
    return HFX_E_ARG;
  const void *all[] = {total_blocks, o->counts, o->used_blocks, o->decision};
  for (const void *q : all) if (misaligned16(q)) return HFX_E_ALIGN;
  ScaleArgs a = {};
  a.mode = s->d_mode; a.total_blocks = total_blocks;
  a.counts = reinterpret_cast<unsigned long long *>(o->counts);
  a.used_blocks = reinterpret_cast<unsigned long long *>(o->used_blocks);
  a.decision = o->decision; a.status = s->d_status; a.sp = *sp;
  {
    KernelScope ks(s, KSLOT_SCALE);
    k_scale_decide<<<1, 1024, 0, s->stream>>>(s->p, a);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
