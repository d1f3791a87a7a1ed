// hfx_attainment: SLO attainment over a request table (Problem Definition, Eq. 2) per SLO class and in
// total, with the sums behind the mean TTFT and the mean end-to-end time.  One streaming pass: every
// block accumulates its rows in shared memory and adds its non-zero totals to the output once.
#include "hfx_internal.cuh"

#define ATT_THREADS 256
#define ATT_FIELDS 6

struct AttArgs {
  const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len; const int32_t *output_len; const int32_t *gen;
  const int64_t *arrival; const int64_t *first_token; const int64_t *last_token; const int64_t *finish;
  int64_t n; unsigned long long *out; uint32_t *status;
};

__global__ void __launch_bounds__(ATT_THREADS) k_attainment(const HfxParams p, const AttArgs a) {
  __shared__ unsigned long long s_acc[(HFX_MAX_CLASSES + 1) * ATT_FIELDS];
  const int K = p.n_classes;
  for (int k = threadIdx.x; k < (K + 1) * ATT_FIELDS; k += blockDim.x) s_acc[k] = 0;
  __syncthreads();
  uint32_t bad = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < a.n; i += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t cls = a.class_id[i], st = a.state[i];
    const int32_t prompt = a.prompt_len[i], gen = a.gen[i];
    bool ok = true;
    if (cls >= (uint32_t)K) { bad |= HFX_ST_BAD_CLASS; ok = false; }
    if (prompt < 0 || prompt > HFX_MAX_TOKENS || gen < 0 || gen > HFX_MAX_TOKENS) { bad |= HFX_ST_BAD_LEN; ok = false; }
    if (!ok) continue;
    long long v[ATT_FIELDS] = {1, 0, 0, 0, 0, 0};
    if (st == HFX_REJECTED) v[3] = 1;
    if (st == HFX_RUNNING || st == HFX_DONE) v[4] = a.first_token[i] - a.arrival[i];
    if (st == HFX_DONE) {
      const int64_t first = a.first_token[i], ttft = first - a.arrival[i];
      const int32_t outlen = a.output_len[i];
      const int64_t tpot = outlen > 1 ? (a.last_token[i] - first) / (outlen - 1) : 0;
      const int64_t ttft_slo = p.ttft[cls], tpot_slo = p.tpot[cls];
      v[1] = 1;
      v[5] = a.finish[i] - a.arrival[i];
      if ((ttft_slo <= 0 || ttft <= ttft_slo) && (tpot_slo <= 0 || tpot <= tpot_slo)) v[2] = 1;
    }
#pragma unroll
    for (int q = 0; q < ATT_FIELDS; q++)
      if (v[q]) { atomicAdd(&s_acc[cls * ATT_FIELDS + q], (unsigned long long)v[q]); atomicAdd(&s_acc[K * ATT_FIELDS + q], (unsigned long long)v[q]); }
  }
  if (bad) atomicOr(a.status, bad);
  __syncthreads();
  for (int k = threadIdx.x; k < (K + 1) * ATT_FIELDS; k += blockDim.x)
    if (s_acc[k]) atomicAdd(&a.out[k], s_acc[k]);
}

int hfx_launch_attainment(hfx_sched *s, const hfx_table *t, int64_t *out) {
  AttArgs a;
  a.class_id = t->class_id; a.state = t->state; a.prompt_len = t->prompt_len; a.output_len = t->output_len; a.gen = t->gen;
  a.arrival = t->arrival_ns; a.first_token = t->first_token_ns; a.last_token = t->last_token_ns; a.finish = t->finish_ns;
  a.n = t->n_rows; a.out = reinterpret_cast<unsigned long long *>(out); a.status = s->d_status;
  if (cudaMemsetAsync(out, 0, sizeof(int64_t) * (size_t)(s->p.n_classes + 1) * ATT_FIELDS, s->stream) != cudaSuccess) return HFX_E_CUDA;
  if (t->n_rows > 0) {
    KernelScope ks(s, KSLOT_METRICS);
    int grid = (int)((t->n_rows + ATT_THREADS - 1) / ATT_THREADS);
    if (grid > s->n_sm * 8) grid = s->n_sm * 8;
    k_attainment<<<grid, ATT_THREADS, 0, s->stream>>>(s->p, a);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
