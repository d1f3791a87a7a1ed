// hfx_count_rows_noalloc: rows per replica and their exclusive prefix (the seg_off output of a
// step) for callers that must not allocate device memory.
//
// The regular path keeps its per-replica counters in a workspace that hfx_sched_create obtains
// with cudaMalloc.  Some callers cannot do that: a serving process that has handed all device
// memory to its framework's caching allocator, a plugin that runs inside someone else's memory
// budget, or code on a latency-critical path where an allocation would synchronise the device.
// For them the counters live in a fixed array that is part of the library image itself.  Every GPU
// that loads the library holds this array (16 KiB) until the process exits.
#include <cuda_runtime.h>
#include <stdint.h>

#include "hfx.h"

#define NOALLOC_WORDS (HFX_NOALLOC_MAX_REPLICAS + 2)
#define NOALLOC_MAX_DEVICES 64

// The scratch: one counter per replica plus the bucket of rows with a bad replica id.
static __device__ __align__(256) uint32_t g_noalloc_counts[NOALLOC_WORDS];

// In host code `g_noalloc_counts` is only a handle for the runtime, not an address a kernel can
// use; the device address is looked up once per device and kept here.
static uint32_t *g_noalloc_ptr[NOALLOC_MAX_DEVICES];

static __global__ void __launch_bounds__(512) k_noalloc_count(const int32_t *__restrict__ replica_id, int64_t n, int32_t R,
                                                              uint32_t *__restrict__ counts) {
  extern __shared__ uint32_t hist[];
  for (int i = threadIdx.x; i <= R; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    int b = replica_id[i];
    if (b < 0 || b >= R) b = R;
    atomicAdd(&hist[b], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i <= R; i += blockDim.x) {
    const uint32_t c = hist[i];
    if (c) atomicAdd(&counts[i], c);
  }
}

// One block: exclusive prefix of counts[0..R] into seg_off[0..R]; optionally the number of rows
// with a bad replica id.
static __global__ void __launch_bounds__(1024) k_noalloc_scan(const uint32_t *__restrict__ counts, int32_t R,
                                                              int32_t *__restrict__ seg_off, uint32_t *__restrict__ n_bad) {
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base <= R; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const uint32_t c = i <= R ? counts[i] : 0;
    uint32_t v = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t w = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += w; }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
      uint32_t w = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += x; }
      warp_tot[lane] = w;
    }
    __syncthreads();
    const uint32_t excl = carry + (warp ? warp_tot[warp - 1] : 0) + v - c;
    if (i <= R) seg_off[i] = (int32_t)excl;
    if (i == R && n_bad) *n_bad = c;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry = excl + c;
    __syncthreads();
  }
}

extern "C" int hfx_count_rows_noalloc(const int32_t *replica_id, int64_t n_rows, int32_t n_replicas,
                                      int32_t *seg_off, uint32_t *n_bad, void *cuda_stream) {
  if (n_replicas < 1 || n_rows < 0 || !seg_off || (n_rows > 0 && !replica_id)) return HFX_E_ARG;
  if (n_replicas > HFX_NOALLOC_MAX_REPLICAS || n_rows > (INT64_C(1) << 27)) return HFX_E_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(replica_id) | reinterpret_cast<uintptr_t>(seg_off) | reinterpret_cast<uintptr_t>(n_bad)) & 3u) return HFX_E_ALIGN;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return HFX_E_CUDA; }
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return HFX_E_CAPACITY;
  if (!g_noalloc_ptr[dev]) {   // set-up, once per device, with that device current
    uint32_t *ptr = nullptr;
    if (cudaGetSymbolAddress((void **)&ptr, g_noalloc_counts) != cudaSuccess || !ptr) { cudaGetLastError(); return HFX_E_CUDA; }
    g_noalloc_ptr[dev] = ptr;
  }
  uint32_t *counts = g_noalloc_ptr[dev];
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  // the array keeps what the previous call left: clear the part this call uses
  if (cudaMemsetAsync(counts, 0, sizeof(uint32_t) * ((size_t)n_replicas + 1), stream) != cudaSuccess) {
    cudaGetLastError();
    return HFX_E_CUDA;
  }
  if (n_rows > 0) {
    int64_t want = (n_rows + 511) / 512;
    const int grid = (int)(want < 592 ? want : 592);
    k_noalloc_count<<<grid, 512, sizeof(uint32_t) * ((size_t)n_replicas + 1), stream>>>(replica_id, n_rows, n_replicas, counts);
  }
  k_noalloc_scan<<<1, 1024, 0, stream>>>(counts, n_replicas, seg_off, n_bad);
  return cudaGetLastError() == cudaSuccess ? HFX_OK : HFX_E_CUDA;
}
