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
// Kernel ids of the optional stage trace (library built with -DMOA_TRACE; see moa_trace_begin).
enum : int { KID_OTHER = 0, KID_EMBED, KID_GEMM, KID_ATTN, KID_ATTN_MERGE, KID_LM_MERGE, KID_EXPAND, KID_NORM, KID_RESNORM,
             KID_SILU, KID_SUMCAST, KID_ROPE, KID_APPEND, KID_MEAN, KID_COUNT };
#ifdef MOA_TRACE
__device__ unsigned long long* g_moa_trace_buf = nullptr;   // [cap][2]: %globaltimer, kernel id << 32 | gridDim.x
__device__ int g_moa_trace_cap = 0;
__device__ int g_moa_trace_n = 0;
#endif
__device__ __forceinline__ void pdl_wait(int kid = KID_OTHER) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef MOA_TRACE
  // one stamp per kernel, at the moment its first thread is released by its predecessor's completion
  if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && g_moa_trace_buf) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    const int i = atomicAdd(&g_moa_trace_n, 1);
    if (i < g_moa_trace_cap) {
      g_moa_trace_buf[2 * i] = t;
      g_moa_trace_buf[2 * i + 1] = ((unsigned long long)kid << 32) | (unsigned long long)gridDim.x;
    }
  }
#else
  (void)kid;
#endif
}

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

// Optional per-row bound on the cache positions a query row may attend (causal / K-step-bounded masks of the
// whole-sequence drafter pass): row r sees positions 0 .. of(r) - 1. Non-decreasing in r within a launch.
struct RowLimit {
  const int* ptr;      // explicit limits, one per row, or nullptr
  int base, inc;       // else base + r * inc when inc != 0; no bound when inc == 0
  __host__ __device__ bool active() const { return ptr != nullptr || inc != 0; }
  __device__ __forceinline__ int of(int r) const { return ptr ? ptr[r] : (inc ? base + r * inc : 0x7fffffff); }
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ---- vector helpers of the glue kernels: fp32 split planes in, bf16 (one or two terms) out ----
__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// 8 consecutive fp32 values: sum of `splits` planes (plane elements apart), read past L1. The loads of four
// planes are issued before any of them is used, so a row costs one memory round trip per four planes.
__device__ __forceinline__ void load8_planes(const float* p, int splits, size_t plane, float* v) {
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = 0.f;
  int s = 0;
  for (; s + 4 <= splits; s += 4) {
    float4 a[4], b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) { a[u] = ldcg4(p + (size_t)(s + u) * plane); b[u] = ldcg4(p + (size_t)(s + u) * plane + 4); }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      v[0] += a[u].x; v[1] += a[u].y; v[2] += a[u].z; v[3] += a[u].w;
      v[4] += b[u].x; v[5] += b[u].y; v[6] += b[u].z; v[7] += b[u].w;
    }
  }
  float4 a[3], b[3];
#pragma unroll
  for (int u = 0; u < 3; ++u)
    if (s + u < splits) { a[u] = ldcg4(p + (size_t)(s + u) * plane); b[u] = ldcg4(p + (size_t)(s + u) * plane + 4); }
#pragma unroll
  for (int u = 0; u < 3; ++u)
    if (s + u < splits) {
      v[0] += a[u].x; v[1] += a[u].y; v[2] += a[u].z; v[3] += a[u].w;
      v[4] += b[u].x; v[5] += b[u].y; v[6] += b[u].z; v[7] += b[u].w;
    }
}

// One fp32 value as the sum of its split planes, loads issued four at a time.
__device__ __forceinline__ float load1_planes(const float* p, int splits, size_t plane) {
  float acc = 0.f;
  int s = 0;
  for (; s + 4 <= splits; s += 4) {
    const float a = __ldcg(p + (size_t)s * plane), b = __ldcg(p + (size_t)(s + 1) * plane);
    const float c = __ldcg(p + (size_t)(s + 2) * plane), d = __ldcg(p + (size_t)(s + 3) * plane);
    acc += a; acc += b; acc += c; acc += d;
  }
  float t[3] = {0.f, 0.f, 0.f};
#pragma unroll
  for (int u = 0; u < 3; ++u)
    if (s + u < splits) t[u] = __ldcg(p + (size_t)(s + u) * plane);
  return acc + t[0] + t[1] + t[2];
}

__device__ __forceinline__ void bf16x8_to_float(const uint4 u, float* v) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// Stores 8 values into an X buffer row as bf16: hi at row r, and (lo_rows > 0) the remainder at row lo_rows + r.
__device__ __forceinline__ void xbuf_store8(bf16* xb, size_t K, int r, int k, int lo_rows, const float* v) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const bf16 h0 = __float2bfloat16_rn(v[2 * e]), h1 = __float2bfloat16_rn(v[2 * e + 1]);
    hi[e] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
    lo[e] = pack_bf16(v[2 * e] - __bfloat162float(h0), v[2 * e + 1] - __bfloat162float(h1));
  }
  *reinterpret_cast<uint4*>(xb + (size_t)r * K + k) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  if (lo_rows > 0) *reinterpret_cast<uint4*>(xb + (size_t)(lo_rows + r) * K + k) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
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
enum : int { DEV_OK = 0, DEV_ERR_BOUNDS = 6, DEV_ERR_TIMEOUT = 10, DEV_ERR_NONFINITE = 11 };

// Debug build (-DMOA_CHECKS): indices that the host logic guarantees (token ids, tree slots, cache lengths) are
// checked where they are used; a violation raises the status word and the access is skipped or clamped as in the
// normal build. Without the flag the macro costs nothing.
#ifdef MOA_CHECKS
#define MOA_DEV_CHECK(cond, status_ptr)                                          \
  do {                                                                           \
    if (!(cond) && (status_ptr) != nullptr) atomicMax((status_ptr), DEV_ERR_BOUNDS); \
  } while (0)
#else
#define MOA_DEV_CHECK(cond, status_ptr) do { } while (0)
#endif

}  // namespace moa
