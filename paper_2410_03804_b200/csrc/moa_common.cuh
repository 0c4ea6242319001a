// Shared device helpers for the Mixture-of-Attentions drafter kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace moa {

typedef __nv_bfloat16 bf16;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// Programmatic dependent launch. A kernel launched with that attribute may begin while the kernel before it in
// the stream still runs. pdl_trigger() lets the NEXT kernel begin; pdl_wait() blocks until the PREVIOUS kernel has
// completed and its writes are visible. Every kernel of a chain calls pdl_wait() before it reads or overwrites
// anything another kernel of the chain touches (so completion stays transitive); both are no-ops otherwise.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum for blocks of up to 1024 threads; every thread gets the result.
__device__ __forceinline__ float block_sum(float v, float* red /* >= 33 floats of shared memory */) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[wid] = v;
  __syncthreads();
  if (wid == 0) {
    float t = lane < nw ? red[lane] : 0.f;
    t = warp_sum(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}
__device__ __forceinline__ float block_max(float v, float* red) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) red[wid] = v;
  __syncthreads();
  if (wid == 0) {
    float t = lane < nw ? red[lane] : -INFINITY;
    t = warp_max(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}

// Which sequence a flat token index belongs to: tokens of the sequences lie back to back.
struct SeqSplit {
  int n_seq;
  int off[65];   // off[b] = first token of sequence b; off[n_seq] = total
  __host__ __device__ int seq_of(int t) const {
    int b = 0;
    while (b + 1 < n_seq && t >= off[b + 1]) ++b;
    return b;
  }
};

// Device-side status word values (mirrors moa_status where it matters).
enum : int { DEV_OK = 0, DEV_ERR_BOUNDS = 6, DEV_ERR_TIMEOUT = 10 };

}  // namespace moa
