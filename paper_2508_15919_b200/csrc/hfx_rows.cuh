// Per-row work shared by the front ends of a step: the kind of a row, its priority, the part of its
// slack that does not depend on the replica's running batch (Sec. 3.3.1: slack = remaining SLO budget).
#pragma once

#include "hfx_internal.cuh"

__device__ __forceinline__ int bucket_of(int rid, int R) { return (rid < 0 || rid >= R) ? R : rid; }

// Kind of a row (KIND_*), with ROWFLAG_BADREP for a row bound to no replica; raises status bits.
// `now` is indexed by replica (global or shared memory).
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
  if (st == HFX_QUEUED) return arrival <= now[rid] ? KIND_QUEUED : KIND_FUTURE;
  return KIND_DEAD;
}

// E_p of one prompt with the narrow products the domain allows (c1 <= 2^30, c2 <= 2^12, t <= 2^24).
__device__ __forceinline__ int64_t dev_Ep_prompt(const HfxParams &p, int32_t t) {
  const uint64_t lin = (uint64_t)(uint32_t)p.c1 * (uint32_t)t;
  const uint64_t c2t = (uint64_t)(uint32_t)p.c2 * (uint32_t)t;       // <= 2^36
  return p.c0 + (int64_t)lin + (int64_t)(c2t * (uint64_t)(uint32_t)t);
}

__device__ __forceinline__ int row_prio(const HfxParams &p, const uint8_t *s_prio, uint32_t cls, int32_t weight) {
  if (p.weight_max > 0) {
    const int64_t w = (int64_t)p.weight_max - weight;
    return (int)(w < 0 ? 0 : (w > 62 ? 62 : w));
  }
  return s_prio[cls];
}

// Slack base of an active row, free of per-replica quantities (the replica's clock, earliest start and
// E_d are subtracted later, once per replica):
//   in flight                  base = first_token + (gen+1) * tpot_slo              (next-token deadline)
//   queued, colocated/prefill  base = ttft_slo + arrival - E_p(prompt_len)
//   queued on a decode replica base = first_token + (gen+1) * tpot_slo - d2 * (prompt_len + gen)
__device__ __forceinline__ int64_t row_base(const HfxParams &p, int64_t ttft, int64_t tpot, uint32_t kind, int mode,
                                            int32_t prompt, int32_t gen, int64_t arrival, int64_t first_token) {
  if (kind == KIND_RUNNING) return tpot > 0 ? first_token + ((int64_t)gen + 1) * tpot : BASE_UNBOUNDED;
  if (mode == HFX_DECODE)
    return tpot > 0 ? first_token + ((int64_t)gen + 1) * tpot - p.d2 * ((int64_t)prompt + gen) : BASE_UNBOUNDED;
  return ttft > 0 ? ttft + arrival - dev_Ep_prompt(p, prompt) : BASE_UNBOUNDED;
}

__device__ __forceinline__ void stage_classes(const HfxParams &p, int64_t *s_ttft, int64_t *s_tpot, uint8_t *s_prio) {
  for (int c = threadIdx.x; c < HFX_MAX_CLASSES; c += blockDim.x) {
    s_ttft[c] = c < p.n_classes ? p.ttft[c] : 0;
    s_tpot[c] = c < p.n_classes ? p.tpot[c] : 0;
    s_prio[c] = c < p.n_classes ? p.prio[c] : 63;
  }
}
