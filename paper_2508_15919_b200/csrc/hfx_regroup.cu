// Fallback front end of a step, for tables the tile front end (hfx_front.cu) does not take: more
// replicas than fit a block's shared-memory counters, or a tile matrix that would be too large.
// Three kernels with global counters:
//   k_count           classify every row (one flag byte per row), count rows / active rows per replica
//   k_offsets         exclusive scan of the totals -> range starts, seg_off; zeroes the fill cursors
//   k_regroup_atomic  every row becomes a 32-byte record inside its replica's range, active rows
//                     first, at a position taken from a global fill cursor (any order inside the two
//                     classes: the per-replica sort breaks ties by req_id, so the step is never "ordered")
// A row is ACTIVE when it is in flight or in the visible queue; everything else (not yet arrived,
// finished, rejected, bad data) is inactive and only needs a place at the end of its replica's order.
#include "hfx_rows.cuh"

// ------------------------------------------------------------------------------------------------
// k_count
// ------------------------------------------------------------------------------------------------
struct CountArgs {
  const int32_t *replica_id; const uint8_t *class_id; const uint8_t *state; const int32_t *prompt_len;
  const int32_t *gen; const int64_t *arrival; const int64_t *now;
  int64_t n;
  uint32_t *tot_all; uint32_t *tot_act; uint8_t *rowflag; uint32_t *status;
};

__global__ void __launch_bounds__(256) k_count(const HfxParams p, const CountArgs a) {
  const int R = p.n_replicas;
  uint32_t bad = 0;
  const int64_t n4 = a.n >> 2;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
    const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + v);
    const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + v);
    const uchar4 st = __ldg(reinterpret_cast<const uchar4 *>(a.state) + v);
    const int4 pr = __ldg(reinterpret_cast<const int4 *>(a.prompt_len) + v);
    const int4 ge = __ldg(reinterpret_cast<const int4 *>(a.gen) + v);
    const longlong2 ar0 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * v);
    const longlong2 ar1 = __ldg(reinterpret_cast<const longlong2 *>(a.arrival) + 2 * v + 1);
    const int rr[4] = {rid.x, rid.y, rid.z, rid.w};
    const uint32_t cc[4] = {cls.x, cls.y, cls.z, cls.w}, ss[4] = {st.x, st.y, st.z, st.w};
    const int pp[4] = {pr.x, pr.y, pr.z, pr.w}, gg[4] = {ge.x, ge.y, ge.z, ge.w};
    const int64_t aa[4] = {ar0.x, ar0.y, ar1.x, ar1.y};
    uint32_t fl[4];
#pragma unroll
    for (int k = 0; k < 4; k++) {
      fl[k] = classify_row(p, rr[k], cc[k], ss[k], pp[k], gg[k], aa[k], a.now, bad);
      const int b = bucket_of(rr[k], R);
      atomicAdd(&a.tot_all[b], 1u);
      if (fl[k] <= KIND_QUEUED) atomicAdd(&a.tot_act[b], 1u);
    }
    *reinterpret_cast<uchar4 *>(a.rowflag + (v << 2)) = make_uchar4(fl[0], fl[1], fl[2], fl[3]);
  }
  if (blockIdx.x == 0) {
    for (int64_t g = (n4 << 2) + threadIdx.x; g < a.n; g += blockDim.x) {
      const int32_t rid = a.replica_id[g];
      const uint32_t fl = classify_row(p, rid, a.class_id[g], a.state[g], a.prompt_len[g], a.gen[g], a.arrival[g], a.now, bad);
      const int b = bucket_of(rid, R);
      atomicAdd(&a.tot_all[b], 1u);
      if (fl <= KIND_QUEUED) atomicAdd(&a.tot_act[b], 1u);
      a.rowflag[g] = (uint8_t)fl;
    }
  }
  if (bad) atomicOr(a.status, bad);
}

// ------------------------------------------------------------------------------------------------
// k_offsets: exclusive scan of the per-replica totals (one block) -> seg_begin and the user-visible
// seg_off; zeroes the fill cursors.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) k_offsets(const uint32_t *__restrict__ tot_all, int32_t R, uint32_t *__restrict__ seg_begin,
                                                  uint32_t *__restrict__ cursor, int32_t *__restrict__ seg_off) {
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  const int total = R + 1;  // buckets 0..R
  for (int base = 0; base < total; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const uint32_t c = i < total ? tot_all[i] : 0;
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
  if (threadIdx.x == 0) seg_begin[total] = carry_s;
}

// ------------------------------------------------------------------------------------------------
// k_regroup_atomic
// ------------------------------------------------------------------------------------------------
struct RowIn {
  int32_t rid, prompt, gen, req_id, weight, out_len;
  uint32_t cls, kind;      // kind: the row's flag byte from k_count
  int64_t arrival, first_token;
};

// The record of a row of kind in.kind; base = arrival for a row that has not arrived yet.
__device__ __forceinline__ void make_record(const HfxParams &p, const int64_t *s_ttft, const int64_t *s_tpot,
                                            const uint8_t *s_prio, int64_t i, const RowIn &in, int mode, HfxRec &r) {
  r.req_id = in.req_id; r.row = (int32_t)i; r.prompt = in.prompt; r.gen = in.gen; r.output_len = in.out_len;
  r.cls = (uint8_t)in.cls; r.kind = (uint8_t)(in.kind & 3u); r.prio = 63; r.pad = 0; r.base = 0;
  if (in.kind == KIND_FUTURE) r.base = in.arrival;
  else if (in.kind <= KIND_QUEUED) {
    r.prio = (uint8_t)row_prio(p, s_prio, in.cls, in.weight);
    r.base = row_base(p, s_ttft[in.cls], s_tpot[in.cls], in.kind, mode, in.prompt, in.gen, in.arrival, in.first_token);
  }
}

// predicted TTFT of a row (optional output)
__device__ __forceinline__ int64_t row_pred_ttft(const HfxParams &p, const RowIn &in, int mode, int64_t start) {
  if (in.kind > KIND_QUEUED) return 0;
  if (in.kind == KIND_RUNNING || mode == HFX_DECODE) return in.first_token - in.arrival;
  return (start - in.arrival) + dev_Ep_prompt(p, in.prompt);
}

// One 32-byte store per record: a whole L2 sector at once.
__device__ __forceinline__ void store_record(HfxRec *rec, uint32_t pos, const HfxRec &r) {
  const uint64_t *w = reinterpret_cast<const uint64_t *>(&r);
  asm volatile("st.global.v4.b64 [%0], {%1, %2, %3, %4};" ::"l"(rec + pos), "l"(w[0]), "l"(w[1]), "l"(w[2]), "l"(w[3]) : "memory");
}

// rows 4v .. 4v+3 with 16-byte loads
__device__ __forceinline__ void load_rows4(const RegroupArgs &a, const uint8_t *rowflag, int64_t v, RowIn in[4]) {
  const int4 rid = __ldg(reinterpret_cast<const int4 *>(a.replica_id) + v);
  const uchar4 cls = __ldg(reinterpret_cast<const uchar4 *>(a.class_id) + v);
  const uchar4 kd = __ldg(reinterpret_cast<const uchar4 *>(rowflag) + v);
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

// Per-row outputs that the regroup can finish by itself: slack 0 / inactive key for rows the scheduler
// does not look at, admit = 1 exactly for rows in flight (they are always in the batch), and the final
// slack and key of queued rows on colocated and prefill replicas (slack = base - earliest start needs
// nothing from the running batch).  Rows in flight and queued rows of decode replicas get their slack
// from the replica kernel afterwards, which also sets admit = 1 for what it admits.
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
    int64_t slack = 0;
    uint64_t k48 = dev_key48(PH_INACTIVE, 63, HFX_SLACK_MAX);
    if (r.kind == KIND_QUEUED && mode != HFX_DECODE) {
      slack = r.base == BASE_UNBOUNDED ? HFX_SLACK_MAX : r.base - start;
      k48 = dev_key48(PH_QUEUED, r.prio, slack);
      r.base = (int64_t)k48;      // final here: the record carries the row's key in place of the base
    }
    a.slack[i] = slack;
    a.admit[i] = in.kind == KIND_RUNNING;
    if (a.pred_tpot) a.pred_tpot[i] = 0;
    if (a.key) a.key[i] = ((uint64_t)(bkt & 0xffff) << 48) | k48;
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

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
int hfx_launch_regroup(hfx_sched *s, const RegroupArgs &ra, int32_t *seg_off) {
  const int R = s->p.n_replicas;
  cudaStream_t stream = s->stream;
  CountArgs ca;
  ca.replica_id = ra.replica_id; ca.class_id = ra.class_id; ca.state = ra.state; ca.prompt_len = ra.prompt_len;
  ca.gen = ra.gen; ca.arrival = ra.arrival; ca.now = ra.now; ca.n = ra.n;
  ca.tot_all = s->d_seg_count; ca.tot_act = s->d_act_count; ca.rowflag = s->d_rowflag; ca.status = s->d_status;
  if (cudaMemsetAsync(s->d_seg_count, 0, sizeof(uint32_t) * (R + 2), stream) != cudaSuccess ||
      cudaMemsetAsync(s->d_act_count, 0, sizeof(uint32_t) * (R + 2), stream) != cudaSuccess)
    return HFX_E_CUDA;
  {
    KernelScope ks(s, KSLOT_COUNT);
    k_count<<<s->n_sm * 8, 256, 0, stream>>>(s->p, ca);
  }
  {
    KernelScope ks(s, KSLOT_OFFSETS);
    k_offsets<<<1, 1024, 0, stream>>>(s->d_seg_count, R, s->d_seg_begin, s->d_cursor, seg_off);
  }
  {
    KernelScope ks(s, KSLOT_REGROUP);
    k_regroup_atomic<<<s->n_sm * 8, 256, 0, stream>>>(s->p, ra, s->d_rowflag, s->d_seg_begin, s->d_act_count, s->d_cursor,
                                                      s->d_rec);
  }
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
