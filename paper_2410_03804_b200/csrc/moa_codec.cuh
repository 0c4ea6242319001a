// Client-server message codec (Section 4.2 "Client-Server"): draft-tree nodes as 3 bytes of token id + 1 byte
// of tree position (4 bytes per node), and 8-bit quantisation of activation rows. Byte and index work; the
// quantiser decides its codes in fp32.
#pragma once
#include "moa_common.cuh"

namespace moa {

// node i -> bytes [4i .. 4i+3]: token id little endian (ff ff ff for a negative id), parent slot (255 for none)
__global__ void pack_tree_kernel(const int* __restrict__ tok, const int* __restrict__ parent, size_t total,
                                 uint32_t* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int t = tok[i], q = parent[i];
  const uint32_t tb = t < 0 ? 0xFFFFFFu : ((uint32_t)t & 0xFFFFFFu);
  const uint32_t pb = q < 0 ? 255u : ((uint32_t)q & 0xFFu);
  out[i] = tb | (pb << 24);                      // little-endian store: token bytes first, position byte last
}

__global__ void unpack_tree_kernel(const uint32_t* __restrict__ in, size_t total, int* __restrict__ tok,
                                   int* __restrict__ parent) {
  pdl_trigger();
  pdl_wait();
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const uint32_t w = in[i];
  const uint32_t tb = w & 0xFFFFFFu, pb = w >> 24;
  tok[i] = tb == 0xFFFFFFu ? -1 : (int)tb;
  parent[i] = pb == 255u ? -1 : (int)pb;
}

// One warp per row: scale = max|x| / 127 (fp32), code = round-half-even(x / scale) clamped to [-127, 127];
// an all-zero row has scale 0 and codes 0. The row is read twice (the second pass hits L1/L2). 16-byte loads
// and 8- or 4-byte code stores when the width and the base pointers allow it (vec), scalar accesses otherwise.
template <typename T>
__device__ __forceinline__ void load_vec(const T* p, float* x) {       // 16 bytes: 4 floats or 8 bf16
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  if constexpr (sizeof(T) == 4) {
    x[0] = __uint_as_float(raw.x); x[1] = __uint_as_float(raw.y);
    x[2] = __uint_as_float(raw.z); x[3] = __uint_as_float(raw.w);
  } else {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      x[2 * e] = __uint_as_float(w[e] << 16);
      x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
  }
}

__device__ __forceinline__ int code_of(float v, float scale) {
  return scale > 0.f ? (int)fminf(127.f, fmaxf(-127.f, rintf(v / scale))) : 0;
}

template <typename T>
__global__ void __launch_bounds__(256) quantize_rows_kernel(const T* __restrict__ x, long long rows, int width, int vec,
                                                            int8_t* __restrict__ codes, float* __restrict__ scales) {
  pdl_trigger();
  pdl_wait();
  constexpr int PER = 16 / sizeof(T);
  const int lane = threadIdx.x & 31;
  const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const T* row = x + (size_t)r * width;
  int8_t* out = codes + (size_t)r * width;
  const int nvec = vec ? width / PER : 0;
  float amax = 0.f;
  for (int c = lane; c < nvec; c += 32) {
    float v[PER];
    load_vec<T>(row + c * PER, v);
#pragma unroll
    for (int e = 0; e < PER; ++e) amax = fmaxf(amax, fabsf(v[e]));
  }
  for (int i = nvec * PER + lane; i < width; i += 32) amax = fmaxf(amax, fabsf(to_f(row[i])));
  amax = warp_max(amax);
  const float scale = amax / 127.f;
  if (lane == 0) scales[r] = scale;
  for (int c = lane; c < nvec; c += 32) {
    float v[PER];
    load_vec<T>(row + c * PER, v);
    uint32_t w[PER / 4];
#pragma unroll
    for (int e4 = 0; e4 < PER / 4; ++e4) {
      w[e4] = 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e) w[e4] |= ((uint32_t)code_of(v[e4 * 4 + e], scale) & 0xFFu) << (8 * e);
    }
    if constexpr (PER == 8) *reinterpret_cast<uint2*>(out + c * PER) = make_uint2(w[0], w[1]);
    else *reinterpret_cast<uint32_t*>(out + c * PER) = w[0];
  }
  for (int i = nvec * PER + lane; i < width; i += 32) out[i] = (int8_t)code_of(to_f(row[i]), scale);
}

template <typename T>
__global__ void dequantize_rows_kernel(const int8_t* __restrict__ codes, const float* __restrict__ scales, long long rows,
                                       int width, T* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)rows * width) return;
  out[i] = from_f<T>((float)codes[i] * scales[i / width]);
}

}  // namespace moa
