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

// One warp per row: scale = max|x| / 127 (fp32), code = round-half-even(x * (127 / max|x|)) clamped to [-127, 127];
// an all-zero row has scale 0 and codes 0. The row is read twice (the second pass hits L1/L2). 16-byte loads
// and 8- or 4-byte code stores when the width and the base pointers allow it (vec), scalar accesses otherwise.
template <typename T>
__device__ __forceinline__ void unpack_vec(const uint4& raw, float* x) {       // 16 bytes: 4 floats or 8 bf16
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

__device__ __forceinline__ int code_of(float v, float inv) {        // inv = 127 / max|x| of the row, 0 for a zero row
  return max(-127, min(127, __float2int_rn(v * inv)));
}

template <typename T>
__device__ __forceinline__ void store_codes(int8_t* dst, const uint4& raw, float inv) {
  constexpr int PER = 16 / sizeof(T);
  float v[PER];
  unpack_vec<T>(raw, v);
  uint32_t w[PER / 4];
#pragma unroll
  for (int e4 = 0; e4 < PER / 4; ++e4) {
    w[e4] = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) w[e4] |= ((uint32_t)code_of(v[e4 * 4 + e], inv) & 0xFFu) << (8 * e);
  }
  if constexpr (PER == 8) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
  else *reinterpret_cast<uint32_t*>(dst) = w[0];
}

// The first QZ_KEEP 16-byte vectors of every lane stay in registers between the two passes (rows of up to
// 2048 bf16 / 1024 floats are read from memory once); what is beyond them is read again (from L1 / L2). Kept
// small on purpose: many resident warps hide the latency of the two dependent passes.
constexpr int QZ_KEEP = 8;

template <typename T>
__global__ void __launch_bounds__(256, 3) quantize_rows_kernel(const T* __restrict__ x, long long rows, int width, int vec,
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
  const uint4* rv = reinterpret_cast<const uint4*>(row);
  uint4 keep[QZ_KEEP];
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < QZ_KEEP; ++j) {
    const int c = lane + 32 * j;
    keep[j] = c < nvec ? __ldcs(rv + c) : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int j = 0; j < QZ_KEEP; ++j) {
    float v[PER];
    unpack_vec<T>(keep[j], v);
#pragma unroll
    for (int e = 0; e < PER; ++e) amax = fmaxf(amax, fabsf(v[e]));      // vectors beyond the row are zeros
  }
#pragma unroll 4
  for (int c = lane + 32 * QZ_KEEP; c < nvec; c += 32) {
    float v[PER];
    unpack_vec<T>(rv[c], v);
#pragma unroll
    for (int e = 0; e < PER; ++e) amax = fmaxf(amax, fabsf(v[e]));
  }
  for (int i = nvec * PER + lane; i < width; i += 32) amax = fmaxf(amax, fabsf(to_f(row[i])));
  amax = warp_max(amax);
  const float scale = amax / 127.f;
  const float inv = amax > 0.f ? 127.f / amax : 0.f;
  if (lane == 0) scales[r] = scale;
#pragma unroll
  for (int j = 0; j < QZ_KEEP; ++j) {
    const int c = lane + 32 * j;
    if (c < nvec) store_codes<T>(out + c * PER, keep[j], inv);
  }
#pragma unroll 4
  for (int c = lane + 32 * QZ_KEEP; c < nvec; c += 32) store_codes<T>(out + c * PER, rv[c], inv);
  for (int i = nvec * PER + lane; i < width; i += 32) out[i] = (int8_t)code_of(to_f(row[i]), inv);
}

// vec: every thread turns 16 codes of one row (width % 16 == 0, 16-byte aligned pointers) into 16 values;
// otherwise one element per thread.
template <typename T>
__global__ void __launch_bounds__(256) dequantize_rows_kernel(const int8_t* __restrict__ codes, const float* __restrict__ scales,
                                                              long long rows, int width, int vec, T* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  const size_t total = (size_t)rows * width;
  if (vec) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 16;
    if (i >= total) return;
    const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(codes + i));
    const float sc = scales[i / width];
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    float v[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) v[e] = (float)(int8_t)((w[e >> 2] >> (8 * (e & 3))) & 0xFFu) * sc;
    if constexpr (sizeof(T) == 4) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        *reinterpret_cast<float4*>(out + i + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    } else {
#pragma unroll
      for (int q = 0; q < 2; ++q)
        *reinterpret_cast<uint4*>(out + i + 8 * q) = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                                                               pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
    }
    return;
  }
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  out[i] = from_f<T>((float)codes[i] * scales[i / width]);
}

}  // namespace moa
